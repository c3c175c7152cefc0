"""The benchmark configurations at their full sizes (where one sequence's oracle finishes in
seconds) and sampled units of the larger ones, through the same C-ABI calls bench.py times."""
import numpy as np
import pytest
import torch

from oracle import snapstream_oracle as orc
from paper_2511_03092_b200 import synth
from tests import _harness as H

pytestmark = pytest.mark.gpu


def _run(wl, lengths, seed, steps, sample_steps=None):
    n = len(lengths)
    layer = H.GpuLayer(wl, max_seqs=n)
    prompts = [synth.make_prompt(wl, L, seed + 101 * i) for i, L in enumerate(lengths)]
    idx = layer.compress(prompts, list(range(n)))
    assert layer.status() == 0
    seqs = [H.oracle_compress(wl, p) for p in prompts]
    swaps = 0
    for i, seq in enumerate(seqs):
        swaps += H.check_selection(idx[i], seq, wl)
        seq.topk_pos = [idx[i][h][idx[i][h] >= 0].astype(np.int64) for h in range(wl.n_kv_heads)]
        H.check_cache_image(layer, seq, i, wl)
    slots_dev = torch.arange(n, dtype=torch.int32, device="cuda")
    check = set(range(steps)) if sample_steps is None else set(sample_steps)
    for step in range(steps):
        d = synth.make_decode_inputs(wl, n, seed, step)
        out = layer.decode(d["q"].cuda(), d["k_new"].cuda(), None if d["v_new"] is None else d["v_new"].cuda(),
                           slots_dev)
        for i, seq in enumerate(seqs):
            ref = orc.decode_step(seq, synth.to_f64(d["q"][i]), synth.to_f64(d["k_new"][i]),
                                  synth.to_f64(d["v_new"][i]) if d["v_new"] is not None else None)
            if step in check:
                H.check_output(out[i], ref, wl, f"seq {i} step {step}")
    for i, seq in enumerate(seqs):
        H.check_cache_image(layer, seq, i, wl)
    assert layer.status() == 0
    return swaps


def test_config0_full():
    """GQA 8/2 heads, fp32, prompt 4096, 16 decode steps."""
    wl = synth.CONFIGS[0]
    _run(wl, [4096], seed=100, steps=wl.decode_steps)


def test_config1_full_size_prompt():
    """Llama-shaped bf16 layer, prompt 32768; decode outputs checked on sampled steps."""
    wl = synth.CONFIGS[1]
    _run(wl, [32768], seed=200, steps=40, sample_steps=[0, 1, 7, 20, 39])


def test_config2_ragged_batch_sample():
    """Continuous-batching shape: a ragged batch (lengths drawn like config 2's, capped so the
    oracle stays within seconds) compressed in one call and decoded together."""
    wl = synth.CONFIGS[2]
    lengths = [8192, 11000, 20011, 16384 + 5]
    _run(wl, lengths, seed=300, steps=6)


def test_config2_decode_in_the_benchmark_launch_shape():
    """32 resident sequences with full caches: the decode launch bench.py times (same grid, same
    number of splits).  The oracle follows a sample of the sequences; the others only have to
    leave the status word clean."""
    wl = synth.CONFIGS[2]
    n = wl.batch
    assert n == 32
    lengths = [8192] * n
    lengths[17], lengths[29], lengths[31] = 12000, 20000, 32768
    sample = [0, 17, 29, 31]
    layer = H.GpuLayer(wl, max_seqs=n)
    prompts = [synth.make_prompt(wl, L, 600 + 7 * i) for i, L in enumerate(lengths)]
    idx = layer.compress(prompts, list(range(n)))
    assert layer.status() == 0
    seqs = {}
    for i in sample:
        seqs[i] = H.oracle_compress(wl, prompts[i])
        H.check_selection(idx[i], seqs[i], wl)
        seqs[i].topk_pos = [idx[i][h][idx[i][h] >= 0].astype(np.int64) for h in range(wl.n_kv_heads)]
        H.check_cache_image(layer, seqs[i], i, wl)
    slots_dev = torch.arange(n, dtype=torch.int32, device="cuda")
    for step in range(3):
        d = synth.make_decode_inputs(wl, n, 600, step)
        out = layer.decode(d["q"].cuda(), d["k_new"].cuda(), d["v_new"].cuda(), slots_dev)
        for i in sample:
            ref = orc.decode_step(seqs[i], synth.to_f64(d["q"][i]), synth.to_f64(d["k_new"][i]),
                                  synth.to_f64(d["v_new"][i]))
            H.check_output(out[i], ref, wl, f"seq {i} step {step}")
    for i in sample:
        H.check_cache_image(layer, seqs[i], i, wl)
    assert layer.status() == 0
    assert [int(x) for x in layer.cache.seq_len.cpu()] == [L + 3 for L in lengths]


def test_config3_latent_sample():
    """Latent-attention shape (128 heads over one 576-wide KV row, V = first 512 dims), prompt cut
    to 16k tokens so that the oracle finishes in seconds."""
    wl = synth.CONFIGS[3].scaled(topk=2048, l_recent=512)
    _run(wl, [16384], seed=400, steps=3)


def test_config3_full_size_unit():
    """Config 3 at its real size: eight 131072-token latent prompts (Ls 4, Lr 2048, K 8192, Lo 32,
    w 7, 128 heads over one 576-wide row) compressed by one call into a batch-8 layer, then decoded
    together, so that the wide score kernel runs its full split count and 32 row blocks, the
    selection sees 129020 candidates at K = 8192 and the latent decode kernel its 10244-slot,
    batch-8 grid and split rule.  The oracle follows one of the eight sequences (units are
    independent); the others only have to leave the status word clean and their cache sections in
    place.  Oracle wall time: about 11 s for the compression of the followed prompt (8 host cores)
    and 0.3 s per decode step."""
    wl = synth.CONFIGS[3]
    n, L, followed = wl.batch, 131072, 5
    assert (n, wl.topk, wl.l_recent, wl.l_obs, wl.pool_kernel, wl.slots) == (8, 8192, 2048, 32, 7, 10244)
    layer = H.GpuLayer(wl, max_seqs=n)
    prompts = [synth.make_prompt(wl, L, 400 + 13 * i) for i in range(n)]
    idx = layer.compress(prompts, list(range(n)))
    assert layer.status() == 0
    seq = H.oracle_compress(wl, prompts[followed])
    swaps = H.check_selection(idx[followed], seq, wl)
    assert swaps <= 2
    seq.topk_pos = [idx[followed][0].astype(np.int64)]
    H.check_cache_image(layer, seq, followed, wl)
    for i in range(n):                                      # every planted heavy hitter is kept (sanity, all prompts)
        assert np.isin(prompts[i]["planted"][0], idx[i][0]).all()
        assert (np.diff(idx[i][0]) > 0).all() and idx[i][0][0] >= wl.l_sink and idx[i][0][-1] < L - wl.l_recent
    assert [int(x) for x in layer.cache.seq_len.cpu()] == [L] * n
    assert [int(x) for x in layer.cache.valid_topk.cpu()] == [wl.topk] * n
    slots_dev = torch.arange(n, dtype=torch.int32, device="cuda")
    for step in range(3):
        d = synth.make_decode_inputs(wl, n, 400, step)
        out = layer.decode(d["q"].cuda(), d["k_new"].cuda(), None, slots_dev)
        ref = orc.decode_step(seq, synth.to_f64(d["q"][followed]), synth.to_f64(d["k_new"][followed]), None)
        H.check_output(out[followed], ref, wl, f"step {step}")
        assert torch.isfinite(out.float()).all()
    H.check_cache_image(layer, seq, followed, wl)
    assert layer.status() == 0
    assert [int(x) for x in layer.cache.seq_len.cpu()] == [L + 3] * n


def test_config2_ragged_batch_with_a_128k_prompt():
    """Config 2's compress call as bench.py issues it: one call over a ragged batch that holds a
    prompt near the 131072-token end of the range next to short ones (the candidate splits of the
    score kernel are cut to the batch as a whole).  Every sequence is followed by the oracle
    (about 4 s for the long prompt's compression)."""
    wl = synth.CONFIGS[2]
    swaps = _run(wl, [9000, 126000 + 77, 30011, 8192], seed=700, steps=3)
    assert swaps <= 2


def test_config4_one_sequence_layer_unit():
    """One (sequence, layer) unit of the 32-layer, 128k-prompt configuration: units are independent,
    so parity on a unit at full prompt length covers the kernels in the launch shape bench.py uses."""
    wl = synth.CONFIGS[4]
    swaps = _run(wl, [131072], seed=500, steps=4)
    assert swaps <= 2


def test_config1_prompt_attention_hands_its_normalisers_to_the_compression():
    """Llama-shaped bf16 layer, prompt 32768, the launch shape bench.py's prefill extra uses: the
    prompt's causal attention checked on sampled (position, head) pairs the oracle computes one by
    one, every normaliser of the observation window, and the selection made from them."""
    from paper_2511_03092_b200 import binding as B
    wl = synth.CONFIGS[1]
    L = 32768
    p = synth.make_prompt(wl, L, 200)
    q = synth.make_prompt_queries(wl, p, 200)
    layer = H.GpuLayer(wl, max_seqs=1)
    qd, kd, vd = q.cuda(), p["k"].cuda(), p["v"].cuda()
    out = torch.empty(L, wl.n_q_heads, wl.d_v, dtype=wl.torch_dtype, device="cuda")
    mu = torch.full((1, wl.n_q_heads, wl.l_obs), float("nan"), dtype=torch.float32, device="cuda")
    c = layer.cache
    B.snap_prefill_attn(layer.cfg, qd, kd, vd, [0, L], out, mu, c.status)
    assert layer.status() == 0
    ocfg = H.oracle_config(wl)
    k64, v64 = synth.to_f64(p["k"]), synth.to_f64(p["v"])
    rng = np.random.default_rng(201)
    rows = [0, 1, 127, 128, 129, 4095, 4096, L - wl.l_obs - 1, L - wl.l_obs, L - 1] + [int(x) for x in rng.integers(0, L, 6)]
    for t in rows:
        for h in (0, int(rng.integers(0, wl.n_q_heads)), wl.n_q_heads - 1):
            kvh = h // (wl.n_q_heads // wl.n_kv_heads)
            ref = orc.attention_over(synth.to_f64(q[t, h]), k64[: t + 1, kvh], v64[: t + 1, kvh], ocfg.softmax_scale)
            H.check_output(out[t, h], ref, wl, f"position {t} head {h}")
    want = orc.candidate_log2_normalisers(synth.to_f64(p["q_obs"]), k64, ocfg)
    np.testing.assert_allclose(mu[0].cpu().numpy().astype(np.float64), want, rtol=0, atol=1e-3)
    ws = torch.empty(B.snap_compress_workspace_bytes(layer.cfg, [0, L]), dtype=torch.uint8, device="cuda")
    idx = torch.full((1, wl.n_kv_heads, wl.topk), -7, dtype=torch.int32, device="cuda")
    B.snap_compress_with_row_stats(layer.cfg, layer.layout, p["q_obs"][None].cuda(), mu, kd, vd, [0, L], [0], c.k_cache,
                                   c.v_cache, c.seq_len, c.valid_topk, idx, ws, c.status)
    assert layer.status() == 0
    seq = H.oracle_compress(wl, p)
    H.check_selection(idx.cpu().numpy()[0], seq, wl)


@pytest.mark.parametrize("row", ["llama", "deepseek"])
def test_paper_hyperparameter_rows(row):
    """The two rows of the appendix table "SnapStream Hyperparameters" (sink, top-K, recent, observation
    window, pooling kernel) on their own attention shapes, with prompts just long enough to need scoring."""
    if row == "llama":        # sink 768, top-K 6400, recent 1024 (8192 slots), window 32, kernel 13
        wl = synth.CONFIGS[1].scaled(name="paper_llama", l_sink=768, topk=6400, l_recent=1024, l_obs=32, pool_kernel=13)
        lengths, steps = [20000, 9000], 4
    else:                     # sink 512, top-K 512, recent 31744 (32768 slots), latent attention
        wl = synth.CONFIGS[3].scaled(name="paper_deepseek", l_sink=512, topk=512, l_recent=31744, l_obs=32, pool_kernel=13)
        lengths, steps = [36000], 3
    assert wl.slots in (8192, 32768)
    _run(wl, lengths, seed=500, steps=steps)


def test_head_sharded_compress_reassembles_to_the_full_head_result():
    """The library's side of a head-sharded deployment (compression with the KV heads spread over
    ranks, decode with whole sequences per rank): each shard calls snap_compress with its share of
    the heads -- n_kv_heads and n_q_heads of the shard, q_obs of its query heads, K/V pointers
    offset to its first head with the strides of the full tensors -- into a cache of its own.
    Both shards run here on one device, one after the other; their caches, concatenated along the
    head axis (what the hand-off's all-to-all delivers to a decode rank), must equal byte for byte
    the cache of one full-head call, the oracle's image, and decode like it."""
    from paper_2511_03092_b200 import binding as B
    wl = synth.CONFIGS[1]
    lengths = [9000, 20000 + 3]
    n, shards = len(lengths), 2
    prompts = [synth.make_prompt(wl, L, 900 + i) for i, L in enumerate(lengths)]
    full = H.GpuLayer(wl, max_seqs=n)
    idx_full = full.compress(prompts, list(range(n)))
    assert full.status() == 0
    hk, g = wl.n_kv_heads // shards, wl.n_q_heads // wl.n_kv_heads
    wl_shard = wl.scaled(n_kv_heads=hk, n_q_heads=hk * g)
    cu = [0, lengths[0], lengths[0] + lengths[1]]
    k_all = torch.cat([p["k"] for p in prompts]).cuda()                     # [T, Hkv, d]: the full tensors
    v_all = torch.cat([p["v"] for p in prompts]).cuda()
    q_all = torch.stack([p["q_obs"] for p in prompts]).cuda()               # [n, Hq, Lo, d]
    parts_k, parts_v, parts_idx = [], [], []
    for r in range(shards):
        layer = H.GpuLayer(wl_shard, max_seqs=n)
        c = layer.cache
        ws = torch.empty(B.snap_compress_workspace_bytes(layer.cfg, cu), dtype=torch.uint8, device="cuda")
        idx = torch.full((n, hk, wl.topk), -7, dtype=torch.int32, device="cuda")
        q_r = q_all[:, r * hk * g:(r + 1) * hk * g].contiguous()
        k_r, v_r = k_all[:, r * hk:(r + 1) * hk], v_all[:, r * hk:(r + 1) * hk]   # views: offset pointer, full strides
        assert k_r.stride(0) == wl.n_kv_heads * wl.d_qk and not k_r.is_contiguous()
        B.snap_compress(layer.cfg, layer.layout, q_r, k_r, v_r, cu, list(range(n)), c.k_cache, c.v_cache, c.seq_len,
                        c.valid_topk, idx, ws, c.status)
        assert layer.status() == 0
        assert torch.equal(c.seq_len, full.cache.seq_len) and torch.equal(c.valid_topk, full.cache.valid_topk)
        parts_k.append(c.k_cache); parts_v.append(c.v_cache); parts_idx.append(idx)
    k_cat, v_cat = torch.cat(parts_k, dim=1), torch.cat(parts_v, dim=1)
    assert torch.equal(k_cat, full.cache.k_cache) and torch.equal(v_cat, full.cache.v_cache)
    assert np.array_equal(torch.cat(parts_idx, dim=1).cpu().numpy(), idx_full)
    # the reassembled cache in a decode layer of its own, against the oracle
    dec = H.GpuLayer(wl, max_seqs=n)
    dec.cache.k_cache.copy_(k_cat); dec.cache.v_cache.copy_(v_cat)
    dec.cache.seq_len.copy_(full.cache.seq_len); dec.cache.valid_topk.copy_(full.cache.valid_topk)
    seqs = [H.oracle_compress(wl, p) for p in prompts]
    for i, seq in enumerate(seqs):
        H.check_selection(idx_full[i], seq, wl)
        seq.topk_pos = [idx_full[i][h].astype(np.int64) for h in range(wl.n_kv_heads)]
        H.check_cache_image(dec, seq, i, wl)
    slots_dev = torch.arange(n, dtype=torch.int32, device="cuda")
    for step in range(2):
        d = synth.make_decode_inputs(wl, n, 900, step)
        out = dec.decode(d["q"].cuda(), d["k_new"].cuda(), d["v_new"].cuda(), slots_dev)
        for i, seq in enumerate(seqs):
            ref = orc.decode_step(seq, synth.to_f64(d["q"][i]), synth.to_f64(d["k_new"][i]), synth.to_f64(d["v_new"][i]))
            H.check_output(out[i], ref, wl, f"seq {i} step {step}")
    assert dec.status() == 0
