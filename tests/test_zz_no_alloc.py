"""The allocation-free decode entry point against the regular one.

snap_decode_attn_static exists for callers that cannot hand the library a scratch buffer
(memory pool frozen at start-up, running inside another runtime's callback, a no-late-
allocation policy): its scratch is a fixed array inside the library.  It must produce exactly
what snap_decode_attn produces, call after call, although the array still holds the previous
call's partial results, and both must agree with the oracle.  This file is named to be
collected last."""
import numpy as np
import pytest
import torch

from oracle import snapstream_oracle as orc
from paper_2511_03092_b200 import binding as B
from paper_2511_03092_b200 import synth
from tests import _harness as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("wl_name", ["gqa_bf16", "f32", "latent_128_heads", "latent_64_heads"])
def test_static_scratch_decode_matches_regular_decode_twice_in_a_row(wl_name):
    """The same inputs through snap_decode_attn and snap_decode_attn_static, two steps in a row:
    equal bit for bit (same kernels, same split count: GQA tensor-core, generic fp32, and both
    latent-layout kernels), and both within the test tolerances of the oracle's decode steps."""
    wl = synth.Workload("gqa_bf16", 16, 4, 128, 128, "bf16", 4, 48, 96, 16, 7, batch=1,
                        prompt_len=(700, 700), decode_steps=2, salience="zipf")
    if wl_name == "f32":
        wl = wl.scaled(name="f32", dtype="f32", n_q_heads=8, n_kv_heads=2)
    elif wl_name.startswith("latent"):
        wl = synth.Workload(wl_name, 128 if "128" in wl_name else 64, 1, 576, 512, "bf16", 3, 40, 64, 8, 5, batch=1,
                            prompt_len=(700, 700), decode_steps=2, salience="planted", n_planted=8,
                            v_aliases_k=True, softmax_scale=2.0 ** -0.5)
    lengths = [700, 30, 333, 2]
    prompts = [synth.make_prompt(wl, L, 31 + i) for i, L in enumerate(lengths)]
    a, b = H.GpuLayer(wl, len(lengths)), H.GpuLayer(wl, len(lengths))
    idx = a.compress(prompts, list(range(len(lengths))))
    b.compress(prompts, list(range(len(lengths))))
    seqs = [H.oracle_compress(wl, p) for p in prompts]
    for i, seq in enumerate(seqs):
        H.check_selection(idx[i], seq, wl)
        seq.topk_pos = [idx[i][h][idx[i][h] >= 0].astype(np.int64) for h in range(wl.n_kv_heads)]
    n = len(lengths)
    slots_dev = torch.arange(n, dtype=torch.int32, device="cuda")
    out_b = torch.empty(n, wl.n_q_heads, wl.d_v, dtype=wl.torch_dtype, device="cuda")
    for step in range(2):                                   # two calls in a row share the array
        d = synth.make_decode_inputs(wl, n, 31, step)
        q, kn = d["q"].cuda(), d["k_new"].cuda()
        vn = None if d["v_new"] is None else d["v_new"].cuda()
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
        for i, seq in enumerate(seqs):
            ref = orc.decode_step(seq, synth.to_f64(d["q"][i]), synth.to_f64(d["k_new"][i]),
                                  None if d["v_new"] is None else synth.to_f64(d["v_new"][i]))
            H.check_output(out_b[i], ref, wl, f"{wl_name} seq {i} step {step}")
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
