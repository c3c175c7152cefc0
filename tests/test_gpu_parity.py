"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, element by
element on the same seeded inputs.  Sizes span several tiles and ragged tails."""
import numpy as np
import pytest
import torch

from oracle import snapstream_oracle as orc
from paper_2511_03092_b200 import binding as B
from paper_2511_03092_b200 import synth
from tests import _harness as H

pytestmark = pytest.mark.gpu

SMALL_F32 = synth.Workload("small_f32", 8, 2, 128, 128, "f32", 4, 48, 96, 16, 7, batch=1,
                           prompt_len=(700, 700), decode_steps=8, salience="planted", n_planted=12)
SMALL_BF16 = SMALL_F32.scaled(name="small_bf16", dtype="bf16", n_q_heads=16, n_kv_heads=4, salience="zipf")
SMALL_MLA = synth.Workload("small_mla", 16, 1, 96, 64, "bf16", 3, 40, 64, 8, 5, batch=1,
                           prompt_len=(500, 500), decode_steps=6, salience="planted", n_planted=8,
                           v_aliases_k=True, softmax_scale=2.0 ** -0.5)


def _run_compress_and_decode(wl, lengths, seed, steps, sharp=1.0, check_ring_every=1):
    n = len(lengths)
    layer = H.GpuLayer(wl, max_seqs=n + 2)
    slots = [int(x) for x in np.random.default_rng(seed).permutation(n + 2)[:n]]   # not the identity map
    prompts = [synth.make_prompt(wl, L, seed + i) for i, L in enumerate(lengths)]
    idx = layer.compress(prompts, slots)
    assert layer.status() == 0
    seqs = [H.oracle_compress(wl, p) for p in prompts]
    seq_len = layer.cache.seq_len.cpu().numpy()
    vt = layer.cache.valid_topk.cpu().numpy()
    for i, (seq, L) in enumerate(zip(seqs, lengths)):
        assert seq_len[slots[i]] == L
        assert vt[slots[i]] == orc.valid_topk(L, wl.l_sink, wl.l_recent, wl.topk)
        if wl.topk > 0:
            H.check_selection(idx[i], seq, wl)
            seq.topk_pos = [idx[i][h][idx[i][h] >= 0].astype(np.int64) for h in range(wl.n_kv_heads)]
        H.check_cache_image(layer, seq, slots[i], wl)
    slots_dev = torch.tensor(slots, dtype=torch.int32, device="cuda")
    for step in range(steps):
        d = synth.make_decode_inputs(wl, n, seed, step)
        q = (d["q"].float() * sharp).to(wl.torch_dtype)
        out = layer.decode(q.cuda(), d["k_new"].cuda(), None if d["v_new"] is None else d["v_new"].cuda(),
                           slots_dev)
        for i, seq in enumerate(seqs):
            ref = orc.decode_step(seq, synth.to_f64(q[i]), synth.to_f64(d["k_new"][i]),
                                  synth.to_f64(d["v_new"][i]) if d["v_new"] is not None else None)
            H.check_output(out[i], ref, wl, f"seq {i} step {step}")
        if (step + 1) % check_ring_every == 0:
            for i, seq in enumerate(seqs):
                H.check_cache_image(layer, seq, slots[i], wl)
    assert layer.status() == 0
    np.testing.assert_array_equal(layer.cache.seq_len.cpu().numpy()[slots], [L + steps for L in lengths])
    return layer, seqs


@pytest.mark.parametrize("wl", [SMALL_F32, SMALL_BF16, SMALL_MLA], ids=lambda w: w.name)
def test_compress_then_decode_matches_oracle(wl):
    Lsr, K = wl.l_sink + wl.l_recent, wl.topk
    # one prompt of every case: L<Ls, Ls<=L<Lsr, L==Lsr, Lsr<L<=Lsr+K, L==Lsr+K+1, long ragged ones
    lengths = [2, wl.l_sink + 5, Lsr, Lsr + K // 2, Lsr + K, Lsr + K + 1, 333, wl.prompt_len[0], 1031]
    _run_compress_and_decode(wl, lengths, seed=11, steps=wl.decode_steps)


@pytest.mark.parametrize("wl", [SMALL_F32, SMALL_BF16], ids=lambda w: w.name)
def test_sharp_softmax_outputs(wl):
    """Queries scaled x4 make the decode softmax peaked, so outputs are O(1) and the absolute
    tolerance bites."""
    _run_compress_and_decode(wl, [wl.prompt_len[0], 260], seed=5, steps=4, sharp=4.0)


@pytest.mark.parametrize("hq,l_obs,sharp", [(16, 32, 4.0), (32, 32, 8.0), (16, 16, 6.0)],
                         ids=["rows128_x4", "rows256_x8", "rows64_x6"])
def test_scores_with_large_logits(hq, l_obs, sharp):
    """Observation queries scaled up: logits of +-30 and more, normalisers far from zero.  The second score
    pass carries the normalisers inside the contraction, so their magnitude must not cost precision."""
    wl = SMALL_BF16.scaled(n_q_heads=hq, n_kv_heads=4, l_obs=l_obs, l_recent=48)
    lengths = [700, 1500, 149]
    layer = H.GpuLayer(wl, max_seqs=len(lengths))
    prompts = [synth.make_prompt(wl, L, 91 + i) for i, L in enumerate(lengths)]
    for p in prompts:
        p["q_obs"] = (p["q_obs"].float() * sharp).to(wl.torch_dtype)
    idx = layer.compress(prompts, list(range(len(lengths))))
    assert layer.status() == 0
    for i, p in enumerate(prompts):
        seq = H.oracle_compress(wl, p)
        H.check_selection(idx[i], seq, wl)
        seq.topk_pos = [idx[i][h][idx[i][h] >= 0].astype(np.int64) for h in range(wl.n_kv_heads)]
        H.check_cache_image(layer, seq, i, wl)


def test_ring_wraps_many_times():
    wl = SMALL_BF16.scaled(l_recent=9, l_obs=4, topk=20, l_sink=2)
    _run_compress_and_decode(wl, [5, 11, 40, 300], seed=3, steps=40, check_ring_every=5)


@pytest.mark.parametrize("kw", [dict(topk=0), dict(l_sink=0), dict(pool_kernel=1), dict(pool_mode="max"),
                                dict(l_obs=1, pool_kernel=1), dict(pool_kernel=13, l_obs=32), dict(pool_kernel=19)],
                         ids=lambda k: "-".join(f"{a}{b}" for a, b in k.items()))
def test_degenerate_hyperparameters(kw):
    wl = SMALL_BF16.scaled(**kw)
    _run_compress_and_decode(wl, [wl.l_sink + wl.l_recent + wl.topk + 300, 77], seed=7, steps=3)


@pytest.mark.parametrize("mode", ["avg", "max"])
def test_all_equal_scores_tie_break(mode):
    """Zero observation queries make every candidate score identical: average pooling then
    favours candidates [r, r+K) (zero padding lowers the edges), max pooling [0, K)."""
    wl = SMALL_BF16.scaled(pool_mode=mode)
    L = 900
    p = synth.make_prompt(wl, L, seed=1)
    p["q_obs"] = torch.zeros_like(p["q_obs"])
    layer = H.GpuLayer(wl, max_seqs=1)
    idx = layer.compress([p], [0])
    # every candidate lies in the re-scoring band: it overflows, says so, and the order stands
    assert layer.status() == B.SNAP_DEV_BAND_OVERFLOW
    r = wl.pool_kernel // 2 if mode == "avg" else 0
    for h in range(wl.n_kv_heads):
        np.testing.assert_array_equal(idx[0][h], wl.l_sink + r + np.arange(wl.topk))
    seq = H.oracle_compress(wl, p)
    H.check_selection(idx[0], seq, wl)


def test_duplicate_scores_and_exact_ties_at_the_boundary():
    """Keys repeated verbatim give exactly equal scores; the lower index must win."""
    wl = SMALL_BF16.scaled(pool_kernel=1, topk=50)
    L = 600
    p = synth.make_prompt(wl, L, seed=2)
    lo = wl.l_sink
    block = p["k"][lo:lo + 40].clone()
    for rep in range(1, 12):                     # 12 identical copies of a 40-token block
        p["k"][lo + 40 * rep: lo + 40 * (rep + 1)] = block
    layer = H.GpuLayer(wl, max_seqs=1)
    idx = layer.compress([p], [0])
    seq = H.oracle_compress(wl, p)
    for h in range(wl.n_kv_heads):
        np.testing.assert_array_equal(idx[0][h], seq.topk_pos[h])


@pytest.mark.parametrize("copies, take", [(200, 100), (40, 17)])
def test_many_exact_ties_at_the_threshold_spread_over_the_selection_cluster(copies, take):
    """One key repeated at scattered positions of a long prompt: its copies score exactly alike, and the
    budget is set so that the threshold falls among them (`take` of them are kept).  With 200 copies
    the equal keys outnumber what the selection kernel's CTAs pass around as a list, so every radix
    digit is resolved by histograms and the copies are shared out among the CTAs by index order; with 40
    the list short-cut ends the selection.  Either way the lowest positions win, as in the oracle."""
    base = SMALL_BF16.scaled(n_q_heads=4, n_kv_heads=1, pool_kernel=1)
    L = 40000
    p = synth.make_prompt(base, L, seed=5)
    rng = np.random.default_rng(3)
    cand = np.arange(base.l_sink, L - base.l_recent)
    pos = np.sort(rng.choice(cand, size=copies, replace=False))
    p["k"][pos] = p["k"][pos[0]].clone()
    scores = H.oracle_compress(base, p).pooled[0]
    dup = scores[pos[0] - base.l_sink]
    assert (scores[pos - base.l_sink] == dup).all()
    above = int((scores > dup).sum())
    wl = base.scaled(topk=above + take)
    layer = H.GpuLayer(wl, max_seqs=1)
    idx = layer.compress([p], [0])
    seq = H.oracle_compress(wl, p)
    np.testing.assert_array_equal(idx[0][0], seq.topk_pos[0])
    kept = np.isin(pos, idx[0][0])
    assert kept[:take].all() and not kept[take:].any()


def test_budget_covers_prompt_equals_dense_attention():
    """K >= number of candidates and no new token: the compressed cache attends like the full one."""
    wl = SMALL_F32.scaled(topk=1024)
    L = 700
    p = synth.make_prompt(wl, L, seed=9)
    layer = H.GpuLayer(wl, max_seqs=1)
    layer.compress([p], [0])
    seq = H.oracle_compress(wl, p)
    d = synth.make_decode_inputs(wl, 1, 9, 0)
    slots_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = layer.decode(d["q"].cuda(), None, None, slots_dev)
    H.check_output(out[0], orc.dense_attention(seq, synth.to_f64(d["q"][0])), wl, "dense")
    assert int(layer.cache.seq_len[0]) == L          # attend-only leaves the length alone


def test_append_kv_then_attend_equals_fused_step():
    wl = SMALL_BF16
    lengths = [3, 60, 400]
    prompts = [synth.make_prompt(wl, L, 21 + i) for i, L in enumerate(lengths)]
    a, b = H.GpuLayer(wl, 3), H.GpuLayer(wl, 3)
    a.compress(prompts, [0, 1, 2]); b.compress(prompts, [0, 1, 2])
    slots_dev = torch.arange(3, dtype=torch.int32, device="cuda")
    for step in range(5):
        d = synth.make_decode_inputs(wl, 3, 21, step)
        q, kn, vn = d["q"].cuda(), d["k_new"].cuda(), d["v_new"].cuda()
        out_a = a.decode(q, kn, vn, slots_dev)
        B.snap_append_kv(b.cfg, b.layout, kn, vn, slots_dev, 3, b.cache.k_cache, b.cache.v_cache,
                         b.cache.seq_len, b.cache.status)
        out_b = b.decode(q, None, None, slots_dev)
        torch.cuda.synchronize()
        assert torch.equal(out_a, out_b)
        assert torch.equal(a.cache.k_cache, b.cache.k_cache) and torch.equal(a.cache.v_cache, b.cache.v_cache)
        assert torch.equal(a.cache.seq_len, b.cache.seq_len)


def test_empty_sequence_and_bad_slot_are_reported_not_fatal():
    wl = SMALL_BF16
    layer = H.GpuLayer(wl, 2)
    d = synth.make_decode_inputs(wl, 2, 1, 0)
    slots_dev = torch.tensor([0, 5], dtype=torch.int32, device="cuda")      # slot 5 does not exist
    out = layer.decode(d["q"].cuda(), None, None, slots_dev)
    assert layer.status() & B.SNAP_DEV_BAD_SLOT
    assert float(out.float().abs().max()) == 0.0                            # empty cache -> zeros


def test_strided_prompt_layout():
    """Prompt K/V that sit inside a fused [tokens, (Hq + 2 Hkv), d] QKV activation."""
    wl = SMALL_BF16
    L = 500
    p = synth.make_prompt(wl, L, seed=4)
    Hq, Hkv, d = wl.n_q_heads, wl.n_kv_heads, wl.d_qk
    qkv = torch.zeros(L, Hq + 2 * Hkv, d, dtype=wl.torch_dtype, device="cuda")
    qkv[:, Hq:Hq + Hkv] = p["k"].cuda(); qkv[:, Hq + Hkv:] = p["v"].cuda()
    layer = H.GpuLayer(wl, 1)
    cu = [0, L]
    ws = torch.empty(B.snap_compress_workspace_bytes(layer.cfg, cu), dtype=torch.uint8, device="cuda")
    c = layer.cache
    B.snap_compress(layer.cfg, layer.layout, p["q_obs"].cuda(), qkv[:, Hq:Hq + Hkv], qkv[:, Hq + Hkv:], cu, [0],
                    c.k_cache, c.v_cache, c.seq_len, c.valid_topk, None, ws, c.status)
    ref = H.GpuLayer(wl, 1)
    ref.compress([p], [0])
    assert torch.equal(c.k_cache, ref.cache.k_cache) and torch.equal(c.v_cache, ref.cache.v_cache)


def test_slot_reuse_overwrites_everything():
    """A finished sequence's slot is simply compressed into again (continuous batching)."""
    wl = SMALL_BF16
    layer = H.GpuLayer(wl, 1)
    layer.compress([synth.make_prompt(wl, 800, 1)], [0])
    p = synth.make_prompt(wl, 30, 2)
    layer.compress([p], [0])
    H.check_cache_image(layer, H.oracle_compress(wl, p), 0, wl)


@pytest.mark.parametrize("hq,hkv", [(4, 4), (8, 4), (12, 4), (20, 4), (24, 4), (28, 4), (32, 4), (18, 2), (24, 2), (32, 2)],
                         ids=["g1", "g2", "g3", "g5", "g6", "g7", "g8", "g9", "g12", "g16"])
def test_group_sizes(hq, hkv):
    """Numbers of query heads per KV head from 1 to 16 (up to 8 in one group of MMA columns, beyond in two)."""
    wl = SMALL_BF16.scaled(n_q_heads=hq, n_kv_heads=hkv)
    _run_compress_and_decode(wl, [wl.prompt_len[0], 50, 3], seed=13, steps=5)


@pytest.mark.parametrize("hq,hkv,d", [(4, 4, 128), (16, 4, 128), (20, 4, 128), (32, 4, 128), (8, 2, 64), (8, 2, 256)],
                         ids=["g1", "g4", "g5", "g8", "d64", "d256"])
def test_decode_with_the_merge_inside_the_kernel(hq, hkv, d, snap_option):
    """Small batches captured into a CUDA graph merge their splits inside the decode kernel (one cluster per
    sequence and KV head, the lengths advanced by a launch of their own); the option takes that path outside
    a capture too: ragged lengths, a ring that wraps, sequences shorter than one tile, every head size."""
    snap_option(B.SNAP_OPT_DECODE_GQA_KERNEL, 3)
    wl = SMALL_BF16.scaled(n_q_heads=hq, n_kv_heads=hkv, d_qk=d, d_v=d)
    _run_compress_and_decode(wl, [wl.prompt_len[0], 50, 3], seed=19, steps=wl.l_recent + 5, check_ring_every=16)


@pytest.mark.parametrize("hq,hkv", [(4, 4), (16, 4), (20, 4), (32, 4)], ids=["g1", "g4", "g5", "g8"])
def test_packed_fp32_decode_kernel_stays_selectable(hq, hkv, snap_option):
    """The packed-FP32 decode kernel (the default before the tensor-core one) on the same cases."""
    snap_option(B.SNAP_OPT_DECODE_GQA_KERNEL, 1)
    wl = SMALL_BF16.scaled(n_q_heads=hq, n_kv_heads=hkv)
    _run_compress_and_decode(wl, [wl.prompt_len[0], 50, 3], seed=13, steps=5)
    _run_compress_and_decode(wl, [300], seed=17, steps=2 * wl.l_recent + 5, check_ring_every=16)


def test_many_sequences_ragged_decode():
    """More sequences than one launch chunk holds, lengths from empty-ish to several tiles."""
    wl = SMALL_BF16.scaled(topk=64, l_recent=32)
    rng = np.random.default_rng(0)
    lengths = [int(x) for x in rng.integers(1, 400, size=70)]
    _run_compress_and_decode(wl, lengths, seed=17, steps=3, check_ring_every=3)


def test_prompt_longer_than_the_register_resident_topk_path():
    """More than 16 candidates per thread of the top-K cluster: keys are re-read from scratch."""
    wl = SMALL_BF16.scaled(n_q_heads=4, n_kv_heads=2, topk=300)
    _run_compress_and_decode(wl, [140000, 131072 + 60], seed=23, steps=2)


def test_late_outlier_logits_refresh_the_running_reference():
    """Keys far down the candidate range that give huge logits to single observation rows only:
    the score kernels must refresh their per-row softmax reference mid-stream (rows of one warp
    disagree about needing it)."""
    wl = SMALL_BF16.scaled(l_obs=32, topk=200)          # 4 heads per KV head x 32 rows = 128 window rows
    L = 5000
    p = synth.make_prompt(wl, L, seed=41)
    q = p["q_obs"].float()
    k = p["k"].float()
    for n, (hq, row, pos, c) in enumerate([(0, 0, 1500, 30.0), (5, 17, 2600, 45.0), (9, 31, 4000, 25.0), (14, 3, 4700, 60.0)]):
        qv = q[hq, row]
        k[pos, hq // 4] = qv * (c / (wl.scale * float(qv @ qv)))
    p["k"] = k.to(wl.torch_dtype)
    layer = H.GpuLayer(wl, max_seqs=1)
    idx = layer.compress([p], [0])
    assert layer.status() == 0
    seq = H.oracle_compress(wl, p)
    H.check_selection(idx[0], seq, wl)
    for pos, kvh in [(1500, 0), (2600, 1), (4000, 2), (4700, 3)]:
        assert pos in idx[0][kvh]


@pytest.mark.parametrize("hq", [64, 128])
def test_latent_attention_kernel_shapes(hq):
    """The 576/512 latent layout (tensor-core decode kernels: tcgen05 for 128 heads, mma.sync for
    64): short and ragged sequences, ring wrap, sharp softmax."""
    wl = synth.Workload("mla_small", hq, 1, 576, 512, "bf16", 3, 40, 64, 8, 5, batch=1,
                        prompt_len=(500, 500), decode_steps=6, salience="planted", n_planted=8,
                        v_aliases_k=True, softmax_scale=2.0 ** -0.5)
    _run_compress_and_decode(wl, [2, 30, 43, 44, 107, 500, 333], seed=29, steps=6)
    _run_compress_and_decode(wl, [500, 70], seed=31, steps=45, sharp=3.0, check_ring_every=9)


def test_latent_attention_mma_sync_decode_kernel_with_128_heads(snap_option):
    """The mma.sync decode kernel for the latent layout stays selectable at 128 heads, where the
    tcgen05 kernel is the default: same cases."""
    snap_option(B.SNAP_OPT_DECODE_LATENT_KERNEL, 1)
    wl = synth.Workload("mla_small", 128, 1, 576, 512, "bf16", 3, 40, 64, 8, 5, batch=1,
                        prompt_len=(500, 500), decode_steps=6, salience="planted", n_planted=8,
                        v_aliases_k=True, softmax_scale=2.0 ** -0.5)
    _run_compress_and_decode(wl, [2, 30, 43, 44, 107, 500, 333], seed=29, steps=6)
    _run_compress_and_decode(wl, [500, 70], seed=31, steps=45, sharp=3.0, check_ring_every=9)


def test_late_outlier_logits_latent_shape():
    """Same hazard as above on the wide-row score kernel (576-wide keys, 512 window rows)."""
    wl = synth.Workload("mla_outlier", 64, 1, 576, 512, "bf16", 3, 40, 100, 8, 5, batch=1,
                        prompt_len=(3000, 3000), decode_steps=2, salience="planted", n_planted=8,
                        v_aliases_k=True, softmax_scale=2.0 ** -0.5)
    L = 3000
    p = synth.make_prompt(wl, L, seed=43)
    q = p["q_obs"].float()
    k = p["k"].float()
    for hq, row, pos, c in [(0, 0, 900, 30.0), (17, 5, 1700, 45.0), (40, 7, 2500, 25.0), (63, 3, 2900, 60.0)]:
        qv = q[hq, row]
        k[pos, 0] = qv * (c / (wl.scale * float(qv @ qv)))
    p["k"] = k.to(wl.torch_dtype)
    layer = H.GpuLayer(wl, max_seqs=1)
    idx = layer.compress([p], [0])
    assert layer.status() == 0
    seq = H.oracle_compress(wl, p)
    H.check_selection(idx[0], seq, wl)
    for pos in (900, 1700, 2500, 2900):
        assert pos in idx[0][0]


@pytest.mark.parametrize("hq,hkv,lo,d", [(128, 1, 8, 576), (64, 1, 8, 576), (32, 2, 32, 320), (24, 1, 16, 192)],
                         ids=["latent_8_row_blocks", "latent_4_row_blocks", "gqa_320_wide_4_row_blocks", "odd_3_row_blocks"])
def test_wide_score_kernel_with_cta_pairs_and_with_single_ctas(snap_option, hq, hkv, lo, d):
    """The wide-row score kernel pairs the CTAs of adjacent row blocks when their number is even (each
    loads half of every key tile, M = 256 instructions over both) and keeps single CTAs when it is
    odd or when asked to: both forms against the oracle on one ragged call (a partly filled last
    candidate tile, a prompt shorter than one tile of candidates), and the same selection from both."""
    latent = d == 576
    wl = synth.Workload("wide_pairs", hq, hkv, d, 512 if latent else d, "bf16", 3, 40, 96, lo, 5, batch=1,
                        prompt_len=(3000, 3000), decode_steps=1, salience="planted", n_planted=8,
                        v_aliases_k=latent, softmax_scale=2.0 ** -0.5 if latent else None)
    prompts = [synth.make_prompt(wl, L, seed=61 + i) for i, L in enumerate([3000, 1777, 150])]
    seqs = [H.oracle_compress(wl, p) for p in prompts]
    picked = []
    for single in (0, 3):
        snap_option(B.SNAP_OPT_SCORE_KERNEL, single)
        layer = H.GpuLayer(wl, max_seqs=3)
        idx = layer.compress(prompts, [2, 0, 1])
        assert layer.status() == 0
        for i, seq in enumerate(seqs):
            H.check_selection(idx[i], seq, wl)
        picked.append(idx)
    assert (picked[0] == picked[1]).all()


@pytest.mark.parametrize("wl,lengths", [(SMALL_BF16, [3, 30, 4 + 5 * 48]), (SMALL_MLA, [2, 3 + 2 * 40])])
def test_concat_update_baseline_matches_oracle(wl, lengths):
    """The slice-and-concatenate update (position-ordered window, new cache every step) gives
    the oracle's outputs and, row for row, the oracle's position-ordered cache image."""
    n = len(lengths)
    prompts = [synth.make_prompt(wl, L, 51 + i) for i, L in enumerate(lengths)]
    layer = H.GpuLayer(wl, n)
    layer.compress(prompts, list(range(n)))
    seqs = [H.oracle_compress(wl, p) for p in prompts]
    c = layer.cache
    cur_k, cur_v = c.k_cache, c.v_cache
    alt_k = torch.zeros_like(cur_k)
    alt_v = None if cur_v is None else torch.zeros_like(cur_v)
    slots_dev = torch.arange(n, dtype=torch.int32, device="cuda")
    ws = torch.empty(B.snap_decode_workspace_bytes(layer.cfg, n), dtype=torch.uint8, device="cuda")
    for step in range(wl.l_recent + 12):
        d = synth.make_decode_inputs(wl, n, 51, step)
        q, kn = d["q"].cuda(), d["k_new"].cuda()
        vn = None if wl.v_aliases_k else d["v_new"].cuda()
        B.snap_append_kv_concat(layer.cfg, layer.layout, kn, vn, slots_dev, n, cur_k, cur_v, alt_k, alt_v,
                                c.seq_len, c.status)
        cur_k, alt_k, cur_v, alt_v = alt_k, cur_k, alt_v, cur_v
        out = torch.empty(n, wl.n_q_heads, wl.d_v, dtype=wl.torch_dtype, device="cuda")
        B.snap_decode_attn(layer.cfg, layer.layout, q, None, None, slots_dev, n, cur_k, cur_v, c.seq_len,
                           c.valid_topk, out, ws, c.status)
        for i in range(n):
            ref = orc.decode_step(seqs[i], synth.to_f64(d["q"][i]), synth.to_f64(d["k_new"][i]),
                                  None if wl.v_aliases_k else synth.to_f64(d["v_new"][i]))
            if step % 8 == 0 or step >= wl.l_recent:
                H.check_output(out[i], ref, wl, f"step {step} seq {i}")
    assert layer.status() == 0
    for i in range(n):
        assert int(c.seq_len[i]) == seqs[i].n_tokens
        Kc, Vc, _ = orc.expected_cache_position_order(seqs[i])
        np.testing.assert_array_equal(cur_k[i].to("cpu", torch.float64).numpy(), Kc)
        if Vc is not None:
            np.testing.assert_array_equal(cur_v[i].to("cpu", torch.float64).numpy(), Vc)


def test_concat_update_refuses_in_place():
    wl = SMALL_BF16
    layer = H.GpuLayer(wl, 1)
    c = layer.cache
    d = synth.make_decode_inputs(wl, 1, 1, 0)
    slots_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(B.SnapError):
        B.snap_append_kv_concat(layer.cfg, layer.layout, d["k_new"].cuda(), d["v_new"].cuda(), slots_dev, 1,
                                c.k_cache, c.v_cache, c.k_cache, c.v_cache, c.seq_len, c.status)


LATENT_128 = synth.Workload("mla_graph", 128, 1, 576, 512, "bf16", 3, 40, 64, 8, 5, batch=1,
                            prompt_len=(500, 500), decode_steps=6, salience="planted", n_planted=8,
                            v_aliases_k=True, softmax_scale=2.0 ** -0.5)


@pytest.mark.parametrize("wl", [SMALL_BF16, LATENT_128], ids=lambda w: w.name)
def test_decode_step_replayed_from_a_cuda_graph(wl):
    """A decode step (append + attention + merge, programmatic dependent launches included) is
    captured once into a CUDA graph and replayed with new inputs: same outputs, cache and
    lengths as issuing the calls directly.  The first call happens before the capture."""
    lengths = [60, 400, 150]
    n = len(lengths)
    prompts = [synth.make_prompt(wl, L, 71 + i) for i, L in enumerate(lengths)]
    a, b = H.GpuLayer(wl, n), H.GpuLayer(wl, n)
    a.compress(prompts, list(range(n))); b.compress(prompts, list(range(n)))
    slots_dev = torch.arange(n, dtype=torch.int32, device="cuda")
    d0 = synth.make_decode_inputs(wl, n, 71, 0)
    q_s, kn_s = d0["q"].cuda(), d0["k_new"].cuda()
    vn_s = None if wl.v_aliases_k else d0["v_new"].cuda()
    a.decode(q_s, kn_s, vn_s, slots_dev); b.decode(q_s, kn_s, vn_s, slots_dev)      # step 0, direct on both
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        out_s = b.decode(q_s, kn_s, vn_s, slots_dev)
    for step in range(1, 6):
        d = synth.make_decode_inputs(wl, n, 71, step)
        q, kn = d["q"].cuda(), d["k_new"].cuda()
        vn = None if wl.v_aliases_k else d["v_new"].cuda()
        q_s.copy_(q); kn_s.copy_(kn)
        if vn is not None:
            vn_s.copy_(vn)
        graph.replay()
        out_a = a.decode(q, kn, vn, slots_dev)
        torch.cuda.synchronize()
        assert torch.equal(out_a, out_s)
        assert torch.equal(a.cache.k_cache, b.cache.k_cache)
        assert torch.equal(a.cache.seq_len, b.cache.seq_len)
    assert a.status() == 0 and b.status() == 0
    assert [int(x) for x in b.cache.seq_len.cpu()] == [L + 6 for L in lengths]


def _run_multi(wl, lengths, q_len, steps, seed):
    """Multi-token steps through snap_decode_attn_multi against q_len oracle steps each."""
    n = len(lengths)
    layer = H.GpuLayer(wl, max_seqs=n)
    prompts = [synth.make_prompt(wl, L, seed + i) for i, L in enumerate(lengths)]
    layer.compress(prompts, list(range(n)))
    seqs = [H.oracle_compress(wl, p) for p in prompts]
    slots_dev = torch.arange(n, dtype=torch.int32, device="cuda")
    ws = torch.empty(B.snap_decode_multi_workspace_bytes(layer.cfg, n, q_len), dtype=torch.uint8, device="cuda")
    c = layer.cache
    for step in range(steps):
        ds = [synth.make_decode_inputs(wl, n, seed, step * q_len + u) for u in range(q_len)]
        q = torch.stack([d["q"] for d in ds], dim=1).contiguous().cuda()            # [n][q_len][Hq][d]
        kn = torch.stack([d["k_new"] for d in ds], dim=1).contiguous().cuda()
        vn = None if wl.v_aliases_k else torch.stack([d["v_new"] for d in ds], dim=1).contiguous().cuda()
        out = torch.empty(n, q_len, wl.n_q_heads, wl.d_v, dtype=wl.torch_dtype, device="cuda")
        B.snap_decode_attn_multi(layer.cfg, layer.layout, q, kn, vn, slots_dev, n, q_len, c.k_cache, c.v_cache,
                                 c.seq_len, c.valid_topk, out, ws, c.status)
        for i in range(n):
            for u in range(q_len):
                ref = orc.decode_step(seqs[i], synth.to_f64(ds[u]["q"][i]), synth.to_f64(ds[u]["k_new"][i]),
                                      None if wl.v_aliases_k else synth.to_f64(ds[u]["v_new"][i]))
                H.check_output(out[i, u], ref, wl, f"step {step} seq {i} token {u}")
    assert layer.status() == 0
    for i in range(n):
        assert int(c.seq_len[i]) == seqs[i].n_tokens
        H.check_cache_image(layer, seqs[i], i, wl)


@pytest.mark.parametrize("hq,hkv,q_len", [(16, 4, 2), (8, 4, 4), (8, 4, 3), (4, 4, 8), (32, 4, 1),
                                          (16, 4, 4), (16, 4, 3), (8, 4, 7), (12, 4, 5), (4, 4, 13),
                                          (32, 4, 3), (16, 4, 7), (12, 4, 11)],
                         ids=["g4x2", "g2x4", "g2x3", "g1x8", "g8x1",
                              "g4x4_16_columns", "g4x3_12_columns", "g2x7_14_columns", "g3x5_15_columns", "g1x13_13_columns",
                              "g8x3_two_passes", "g4x7_two_passes", "g3x11_three_passes"])
def test_multi_token_decode_steps(hq, hkv, q_len):
    """q_len tokens per step: each query sees the cache as it is after its own token -- window rows
    evicted by later tokens of the step included, those evicted by earlier ones not.  Sequences that
    are still filling the sinks, filling the window, and wrapping the ring."""
    wl = SMALL_BF16.scaled(n_q_heads=hq, n_kv_heads=hkv)
    _run_multi(wl, [1, 3, 45, 50, 51, 52, 300, wl.prompt_len[0]], q_len, steps=max(4, 60 // q_len), seed=83)


@pytest.mark.parametrize("wl,q_len", [(SMALL_BF16, 3), (SMALL_F32, 2), (SMALL_MLA, 3), (LATENT_128, 2)],
                         ids=["bf16_g4x3", "f32_g4x2", "latent_x3", "latent_128_heads_x2"])
def test_multi_token_decode_on_shapes_served_step_by_step(wl, q_len):
    """Shapes the tensor-core grouped-query kernel does not take (fp32, the latent layout) go through
    q_len single steps inside the library, and a step with more than 16 query rows per KV head through
    several passes of that kernel: same definition, same results."""
    _run_multi(wl, [1, 3, 45, 50, 51, 52, 300, wl.prompt_len[0]], q_len, steps=6, seed=87)


def test_multi_token_decode_rejects_invalid_token_counts():
    wl = SMALL_BF16
    layer = H.GpuLayer(wl, 1)
    for q_len in (0, wl.l_recent + 1):                # at least one token, at most a window's worth
        with pytest.raises(B.SnapError) as e:
            B.snap_decode_multi_workspace_bytes(layer.cfg, 1, q_len)
        assert e.value.code == -1
    assert B.snap_decode_multi_workspace_bytes(layer.cfg, 4, 3) > B.snap_decode_workspace_bytes(layer.cfg, 4)


@pytest.mark.parametrize("wl", [SMALL_BF16, LATENT_128, SMALL_F32], ids=lambda w: w.name)
def test_decode_from_empty_slots_in_memory_full_of_nans(wl):
    """Sequences built by decode steps alone, in cache memory that was never cleared: rows past
    the end of a ragged tile must not leak into the result (0 x NaN is NaN)."""
    n = 2
    layer = H.GpuLayer(wl, n)
    c = layer.cache
    c.k_cache.fill_(float("nan"))
    if c.v_cache is not None:
        c.v_cache.fill_(float("nan"))
    ocfg = H.oracle_config(wl)
    seqs = []
    for _ in range(n):
        seq = orc.OracleSequence(ocfg)
        seq.topk_pos = [np.zeros(0, dtype=np.int64) for _ in range(wl.n_kv_heads)]
        seqs.append(seq)
    slots_dev = torch.arange(n, dtype=torch.int32, device="cuda")
    for step in range(wl.l_sink + wl.l_recent + 9):
        d = synth.make_decode_inputs(wl, n, 91, step)
        vn = None if wl.v_aliases_k else d["v_new"].cuda()
        out = layer.decode(d["q"].cuda(), d["k_new"].cuda(), vn, slots_dev)
        for i in range(n):
            ref = orc.decode_step(seqs[i], synth.to_f64(d["q"][i]), synth.to_f64(d["k_new"][i]),
                                  None if wl.v_aliases_k else synth.to_f64(d["v_new"][i]))
            if step < 20 or step % 7 == 0:
                H.check_output(out[i], ref, wl, f"step {step} seq {i}")
    assert layer.status() == 0


@pytest.mark.parametrize("d,hq,hkv", [(64, 16, 4), (64, 4, 4), (256, 8, 4), (256, 32, 4)],
                         ids=["d64g4", "d64g1", "d256g2", "d256g8"])
def test_head_sizes_64_and_256(d, hq, hkv):
    """The tensor-core decode kernel and the wide score kernel at the other common head sizes."""
    wl = SMALL_BF16.scaled(d_qk=d, d_v=d, n_q_heads=hq, n_kv_heads=hkv)
    _run_compress_and_decode(wl, [wl.prompt_len[0], 50, 3], seed=19, steps=5)
    _run_compress_and_decode(wl, [300], seed=23, steps=2 * wl.l_recent + 5, check_ring_every=16)


def test_multi_token_decode_with_64_wide_heads():
    wl = SMALL_BF16.scaled(d_qk=64, d_v=64, n_q_heads=8, n_kv_heads=4)
    _run_multi(wl, [3, 50, 52, 300], 3, steps=20, seed=89)
