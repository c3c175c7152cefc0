"""The allocation-free decode entry point against the regular one.

snap_decode_attn_static exists for callers that cannot hand the library a scratch buffer
(memory pool frozen at start-up, running inside another runtime's callback, a no-late-
allocation policy): its scratch is a fixed array inside the library.  It must produce exactly
what snap_decode_attn produces, call after call, although the array still holds the previous
call's partial results.  This file is named to be collected last."""
import pytest
import torch

from paper_2511_03092_b200 import binding as B
from paper_2511_03092_b200 import synth
from tests import _harness as H

pytestmark = pytest.mark.gpu


def _pair_of_layers(wl, lengths, seed):
    prompts = [synth.make_prompt(wl, L, seed + i) for i, L in enumerate(lengths)]
    a, b = H.GpuLayer(wl, len(lengths)), H.GpuLayer(wl, len(lengths))
    slots = list(range(len(lengths)))
    a.compress(prompts, slots)
    b.compress(prompts, slots)
    return a, b


@pytest.mark.parametrize("wl_name", ["gqa_bf16", "f32"])
def test_static_scratch_decode_matches_regular_decode_twice_in_a_row(wl_name):
    wl = synth.Workload("gqa_bf16", 16, 4, 128, 128, "bf16", 4, 48, 96, 16, 7, batch=1,
                        prompt_len=(700, 700), decode_steps=2, salience="zipf")
    if wl_name == "f32":
        wl = wl.scaled(name="f32", dtype="f32", n_q_heads=8, n_kv_heads=2)
    lengths = [700, 30, 333, 2]
    a, b = _pair_of_layers(wl, lengths, seed=31)
    n = len(lengths)
    slots_dev = torch.arange(n, dtype=torch.int32, device="cuda")
    out_b = torch.empty(n, wl.n_q_heads, wl.d_v, dtype=wl.torch_dtype, device="cuda")
    for step in range(2):                                   # two calls in a row share the array
        d = synth.make_decode_inputs(wl, n, 31, step)
        q, kn, vn = d["q"].cuda(), d["k_new"].cuda(), d["v_new"].cuda()
        out_a = a.decode(q, kn, vn, slots_dev)
        c = b.cache
        B.snap_decode_attn_static(b.cfg, b.layout, q, kn, vn, slots_dev, n, c.k_cache, c.v_cache, c.seq_len,
                                  c.valid_topk, out_b, c.status)
        torch.cuda.synchronize()
        tol = 2e-2 if wl.dtype == "bf16" else 1e-5
        assert float((out_a.float() - out_b.float()).abs().max()) <= tol
        assert torch.equal(out_a, out_b)                    # same kernels, same split count
        assert torch.equal(a.cache.k_cache, b.cache.k_cache)
        assert torch.equal(a.cache.seq_len, b.cache.seq_len)
    assert b.status() == 0


def test_static_scratch_rejects_oversized_batches():
    wl = synth.CONFIGS[1]
    cfg = H.snap_config(wl, max_seqs=512)
    lay = B.snap_cache_layout(cfg)
    one = torch.zeros(16, dtype=torch.int32, device="cuda")   # never dereferenced: refused before any launch
    with pytest.raises(B.SnapError) as e:
        B.snap_decode_attn_static(cfg, lay, one, None, None, one, 512, one, one, one, one, one)
    assert e.value.code == -6
    assert "static scratch" in B.status_string(-6)
