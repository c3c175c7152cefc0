"""Per-step block top-K through the C ABI against the oracle: block statistics byte for byte, the
per-step selection (exact, up to blocks whose oracle scores lie within 1e-12 relative of the last
selected one: the kernel re-scores the blocks near its threshold in double precision, the oracle
sums in double throughout, in another order), and the attention over sinks, window and the
selected blocks, on ragged batches with prompts that have no middle, a short last block, more
budget than blocks, and rings that wrap."""
import numpy as np
import pytest
import torch

from oracle import snapstream_oracle as orc
from paper_2511_03092_b200 import binding as B
from paper_2511_03092_b200 import synth
from tests import _harness as H

pytestmark = pytest.mark.gpu

SCORE_REL = 1e-12


def _workload(hq, hkv, d, topk, l_recent=48, l_sink=4):
    return synth.Workload("blocks", hq, hkv, d, d, "bf16", l_sink, l_recent, topk, 8, 5, batch=1, prompt_len=(1000, 1000),
                          decode_steps=4, salience="planted", n_planted=16)


def _check_blocks(got, n_got, U, n_blocks):
    """One KV head's selection against the oracle's scores U: exact, or differing only in near ties."""
    want = orc.select_blocks(U, n_blocks)
    assert n_got == len(want)
    got = got[:n_got]
    assert (np.diff(got) > 0).all(), "blocks must be ascending and distinct"
    if np.array_equal(got, want):
        return 0
    tau = np.sort(U)[-len(want)]
    tol = SCORE_REL * max(abs(tau), np.abs(U).max() * 1e-3)
    sel = np.zeros(len(U), dtype=bool)
    sel[got] = True
    assert sel[U > tau + tol].all(), "a clear winner was not selected"
    assert not sel[U < tau - tol].any(), "a clear loser was selected"
    return int((sel != np.isin(np.arange(len(U)), want)).sum() // 2)


def _run(wl, lengths, bs, n_blocks, steps, seed):
    n = len(lengths)
    layer = H.GpuLayer(wl, max_seqs=n + 1)
    slots = [int(x) for x in np.random.default_rng(seed).permutation(n + 1)[:n]]
    prompts = [synth.make_prompt(wl, L, seed + i) for i, L in enumerate(lengths)]
    layer.compress(prompts, slots, want_idx=False)
    assert layer.status() == 0
    cfg = H.oracle_config(wl)
    seqs = [H.oracle_compress(wl, p) for p in prompts]
    for i, seq in enumerate(seqs):                      # the whole middle is kept, in position order
        Le = max(lengths[i] - cfg.l_sr, 0)
        assert all(np.array_equal(t, cfg.l_sink + np.arange(Le)) for t in seq.topk_pos)
        H.check_cache_image(layer, seq, slots[i], wl)
    c = layer.cache
    slots_dev = torch.tensor(slots, dtype=torch.int32, device="cuda")
    # ---- statistics, once per prompt ----
    nb_max = -(-wl.topk // bs)
    nbytes = B.snap_block_stats_bytes(layer.cfg, bs)
    assert nbytes == (n + 1) * wl.n_kv_heads * nb_max * 2 * wl.d_qk * 2
    stats = torch.full((n + 1, wl.n_kv_heads, nb_max, 2, wl.d_qk), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.snap_block_stats(layer.cfg, layer.layout, slots_dev, n, c.k_cache, c.valid_topk, bs, stats, c.status)
    torch.cuda.synchronize()
    ref_stats = [orc.block_statistics(synth.to_f64(p["k"]), cfg, bs) for p in prompts]
    got_stats = stats.to("cpu", torch.float64).numpy()
    for i, (kmin, kmax) in enumerate(ref_stats):
        nb = kmin.shape[1]
        np.testing.assert_array_equal(got_stats[slots[i], :, :nb, 0], kmin)
        np.testing.assert_array_equal(got_stats[slots[i], :, :nb, 1], kmax)
        assert np.isnan(got_stats[slots[i], :, nb:]).all()          # blocks past the prompt's last one: untouched
    # ---- steps: select, then attend ----
    block_idx = torch.full((n, wl.n_kv_heads, n_blocks), -9, dtype=torch.int32, device="cuda")
    n_sel = torch.full((n, wl.n_kv_heads), -9, dtype=torch.int32, device="cuda")
    ws = torch.empty(B.snap_decode_blocks_workspace_bytes(layer.cfg, n, bs, n_blocks), dtype=torch.uint8, device="cuda")
    sws = torch.empty(B.snap_block_select_workspace_bytes(layer.cfg, n, bs), dtype=torch.uint8, device="cuda")
    out = torch.empty(n, wl.n_q_heads, wl.d_v, dtype=torch.bfloat16, device="cuda")
    swaps = 0
    for step in range(steps):
        d = synth.make_decode_inputs(wl, n, seed, step)
        q = d["q"]
        if step % 2 == 1:                                # every other step: a query aligned with some prompt key
            for i, L in enumerate(lengths):
                if L > cfg.l_sr + 3:
                    pos = cfg.l_sink + (step * 37 + i * 11) % (L - cfg.l_sr)
                    q[i] = (prompts[i]["k"][pos].float().repeat_interleave(cfg.group, dim=0) * 3.0).to(torch.bfloat16)
        B.snap_block_select(layer.cfg, layer.layout, q.cuda(), slots_dev, n, stats, c.valid_topk, bs, n_blocks, block_idx,
                            n_sel, sws, c.status)
        B.snap_decode_attn_blocks(layer.cfg, layer.layout, q.cuda(), d["k_new"].cuda(), d["v_new"].cuda(), slots_dev, n,
                                  c.k_cache, c.v_cache, c.seq_len, c.valid_topk, bs, n_blocks, block_idx, n_sel, out, ws,
                                  c.status)
        torch.cuda.synchronize()
        bi, ns = block_idx.cpu().numpy(), n_sel.cpu().numpy()
        for i, seq in enumerate(seqs):
            kmin, kmax = ref_stats[i]
            U = orc.block_upper_bounds(synth.to_f64(q[i]), kmin, kmax, cfg)
            chosen = []
            for h in range(wl.n_kv_heads):
                swaps += _check_blocks(bi[i, h], int(ns[i, h]), U[h], n_blocks)
                chosen.append(bi[i, h, :ns[i, h]])
            # the attention is checked on the set the kernel chose (validated above)
            seq.topk_pos = [orc.block_positions(chosen[h], lengths[i], cfg, bs) for h in range(wl.n_kv_heads)]
            ref = orc.decode_step(seq, synth.to_f64(q[i]), synth.to_f64(d["k_new"][i]), synth.to_f64(d["v_new"][i]))
            H.check_output(out[i], ref, wl, f"seq {i} step {step}")
    assert layer.status() == 0
    np.testing.assert_array_equal(c.seq_len.cpu().numpy()[slots], [L + steps for L in lengths])
    for i, seq in enumerate(seqs):                      # the ring advanced, the middle is untouched
        seq.topk_pos = [cfg.l_sink + np.arange(max(lengths[i] - cfg.l_sr, 0)) for _ in range(wl.n_kv_heads)]
        H.check_cache_image(layer, seq, slots[i], wl)
    return swaps


@pytest.mark.parametrize("hq,hkv,d,bs,n_blocks", [(8, 2, 128, 64, 6), (4, 4, 128, 16, 9), (16, 2, 64, 32, 4), (8, 1, 256, 128, 3)],
                         ids=["g4_d128_b64", "g1_d128_b16", "g8_d64_b32", "g8_d256_b128"])
def test_block_lookup_steps_match_the_oracle(hq, hkv, d, bs, n_blocks):
    wl = _workload(hq, hkv, d, topk=2100)
    # no middle at all, a middle shorter than one block, a short last block, exact multiples, long ones
    lengths = [30, 52 + 5, 52 + bs, 52 + 2 * bs + 3, 700, 2052, 1999]
    _run(wl, lengths, bs, n_blocks, steps=6, seed=201)


@pytest.mark.parametrize("seed", [5, 6])
def test_random_block_lookup_configurations(seed):
    """Seeded random layers (group size 1..8, head size 64/128/256, blocks of 16..256 tokens, budgets of 1..40 blocks, sink
    and window sizes, one to four ragged prompts): statistics, selections, outputs and the final cache image."""
    rng = np.random.default_rng(seed)
    for case in range(20):
        hkv = int(rng.choice([1, 2, 4])); g = int(rng.choice([1, 2, 3, 4, 8])); d = int(rng.choice([64, 128, 256]))
        bs = int(rng.choice([16, 32, 48, 64, 128, 256])); nblk = int(rng.choice([1, 2, 5, 16, 40]))
        Ls = int(rng.integers(0, 9)); Lr = int(rng.integers(8, 200)); topk = int(rng.choice([500, 2100, 5000]))
        lengths = [int(rng.integers(1, Ls + Lr + topk)) for _ in range(int(rng.integers(1, 5)))]
        wl = synth.Workload("blocks_random", g * hkv, hkv, d, d, "bf16", Ls, Lr, topk, 8, 5, batch=1, prompt_len=(100, 100),
                            decode_steps=1, salience=str(rng.choice(["zipf", "planted"])), n_planted=8)
        _run(wl, lengths, bs, nblk, steps=int(rng.integers(1, 6)), seed=1000 * seed + case)


def test_block_lookup_with_the_merge_inside_the_decode_kernel(snap_option):
    """The block list and the in-kernel merge of small batches (taken under stream capture; the option takes it here)
    together: ragged prompts, several steps."""
    snap_option(B.SNAP_OPT_DECODE_GQA_KERNEL, 3)
    wl = _workload(8, 2, 128, topk=2100)
    _run(wl, [30, 52 + 64, 700, 2052], 64, 6, steps=6, seed=231)


def test_more_budget_than_blocks_attends_everything_and_the_ring_wraps():
    wl = _workload(8, 2, 128, topk=600, l_recent=16)
    _run(wl, [300, 616, 90], 64, 12, steps=40, seed=207)       # 12 blocks of budget, at most 10 blocks of middle


def test_block_lookup_at_the_benchmark_shape():
    """Llama-shaped layer, one 131072-token prompt kept whole (2048 blocks of 64 tokens) next to a
    40000-token one; 64 blocks per step and KV head, as many rows as the one-time top-K keeps."""
    wl = synth.Workload("blocks_128k", 32, 8, 128, 128, "bf16", 4, 1024, 131072, 64, 7, batch=1, prompt_len=(131072, 131072),
                        decode_steps=3, salience="zipf")
    _run(wl, [131072, 40000], 64, 64, steps=3, seed=211)


def _near_tie_case(gap_dim_q, seed):
    """Blocks of identical keys (minimum = maximum, so a block's score is the group-summed logit itself): three strong
    ones, many weak ones, and a pair of equal strength whose second member is one bf16 step larger in one dim; the query
    is tiny in that dim, so the pair's scores differ by 1e-9 .. 1e-8 relative -- below what a 256-term single-precision
    sum resolves, far above what double precision does."""
    bs, n_blocks, nb = 16, 4, 40
    wl = _workload(4, 1, 128, topk=nb * bs, l_recent=16, l_sink=0)
    g = torch.Generator().manual_seed(seed)
    base = (torch.randn(128, generator=g).abs() + 0.5).to(torch.bfloat16)
    L = nb * bs + wl.l_recent
    p = synth.make_prompt(wl, L, seed)
    k = torch.zeros(L, 1, 128, dtype=torch.bfloat16)
    strength = torch.ones(nb)
    strong = [5, 17, 33]
    pair = (11, 26)
    strength[strong] = 3.0
    strength[list(pair)] = 2.0
    for b in range(nb):
        k[b * bs:(b + 1) * bs, 0] = (base.float() * strength[b]).to(torch.bfloat16)
    d_star = 77
    row = k[pair[1] * bs, 0].clone()
    step = torch.tensor(row[d_star].view(torch.int16).item() + 1, dtype=torch.int16).view(torch.bfloat16)   # next bf16 up
    k[pair[1] * bs:(pair[1] + 1) * bs, 0, d_star] = step
    k[L - wl.l_recent:] = p["k"][L - wl.l_recent:]
    p["k"] = k
    q = base.float().repeat(4, 1)
    q[:, d_star] = gap_dim_q
    return wl, p, q.to(torch.bfloat16), bs, n_blocks, strong, pair


@pytest.mark.parametrize("gap_dim_q,winner", [(2.0 ** -12, 1), (-(2.0 ** -12), 0), (2.0 ** -15, 1), (-(2.0 ** -15), 0)],
                         ids=["second_larger_q_2^-12", "first_larger_q_2^-12", "second_larger_q_2^-15", "first_larger_q_2^-15"])
def test_blocks_nearly_tied_at_the_threshold_are_ranked_by_their_exact_scores(snap_option, gap_dim_q, winner):
    """The last place goes to the member of the pair whose exact score is larger, whichever its block number.  With the
    re-scoring switched off the single-precision order (a tie, hence the lower block number) must get at least one of
    the four cases wrong; that run is the evidence that the cases bite."""
    wl, p, q, bs, n_blocks, strong, pair = _near_tie_case(gap_dim_q, seed=301)
    cfg = H.oracle_config(wl)
    kmin, kmax = orc.block_statistics(synth.to_f64(p["k"]), cfg, bs)
    U = orc.block_upper_bounds(synth.to_f64(q), kmin, kmax, cfg)[0]
    gap = abs(U[pair[0]] - U[pair[1]]) / abs(U[pair[0]])
    assert 1e-10 < gap < 1e-7
    want = sorted(strong + [pair[winner]])
    assert orc.select_blocks(U, n_blocks).tolist() == want
    layer = H.GpuLayer(wl, 1)
    layer.compress([p], [0], want_idx=False)
    c = layer.cache
    slots = torch.zeros(1, dtype=torch.int32, device="cuda")
    stats = torch.zeros(B.snap_block_stats_bytes(layer.cfg, bs), dtype=torch.uint8, device="cuda")
    B.snap_block_stats(layer.cfg, layer.layout, slots, 1, c.k_cache, c.valid_topk, bs, stats, c.status)
    idx = torch.zeros(1, 1, n_blocks, dtype=torch.int32, device="cuda")
    nsel = torch.zeros(1, 1, dtype=torch.int32, device="cuda")
    sws = torch.empty(B.snap_block_select_workspace_bytes(layer.cfg, 1, bs), dtype=torch.uint8, device="cuda")
    B.snap_block_select(layer.cfg, layer.layout, q[None].cuda(), slots, 1, stats, c.valid_topk, bs, n_blocks, idx, nsel, sws,
                        c.status)
    torch.cuda.synchronize()
    assert layer.status() == 0
    assert idx.cpu().numpy()[0, 0].tolist() == want


def test_without_rescoring_the_near_ties_are_not_all_resolved(snap_option):
    snap_option(B.SNAP_OPT_REFINE_OFF, 1)
    wrong = 0
    for gap_dim_q, winner in [(2.0 ** -12, 1), (-(2.0 ** -12), 0), (2.0 ** -15, 1), (-(2.0 ** -15), 0)]:
        wl, p, q, bs, n_blocks, strong, pair = _near_tie_case(gap_dim_q, seed=301)
        layer = H.GpuLayer(wl, 1)
        layer.compress([p], [0], want_idx=False)
        c = layer.cache
        slots = torch.zeros(1, dtype=torch.int32, device="cuda")
        stats = torch.zeros(B.snap_block_stats_bytes(layer.cfg, bs), dtype=torch.uint8, device="cuda")
        B.snap_block_stats(layer.cfg, layer.layout, slots, 1, c.k_cache, c.valid_topk, bs, stats, c.status)
        idx = torch.zeros(1, 1, n_blocks, dtype=torch.int32, device="cuda")
        nsel = torch.zeros(1, 1, dtype=torch.int32, device="cuda")
        sws = torch.empty(B.snap_block_select_workspace_bytes(layer.cfg, 1, bs), dtype=torch.uint8, device="cuda")
        B.snap_block_select(layer.cfg, layer.layout, q[None].cuda(), slots, 1, stats, c.valid_topk, bs, n_blocks, idx, nsel,
                            sws, c.status)
        torch.cuda.synchronize()
        got = idx.cpu().numpy()[0, 0].tolist()
        assert sorted(strong) == [b for b in got if b in strong]          # the clear winners are always there
        wrong += got != sorted(strong + [pair[winner]])
    assert wrong >= 1


def test_block_entry_points_reject_what_they_do_not_serve():
    wl = _workload(8, 2, 128, topk=2100)
    layer = H.GpuLayer(wl, 2)
    for bad_bs in (0, 8, 24, 2048):
        with pytest.raises(B.SnapError):
            B.snap_block_stats_bytes(layer.cfg, bad_bs)
    f32 = synth.Workload("f", 8, 2, 128, 128, "f32", 4, 48, 2100, 8, 5, batch=1, prompt_len=(100, 100), decode_steps=1,
                         salience="zipf")
    with pytest.raises(B.SnapError) as e:
        B.snap_block_stats_bytes(H.snap_config(f32, 2), 64)
    assert e.value.code == -2                                   # unsupported, not invalid
    with pytest.raises(B.SnapError):
        B.snap_decode_blocks_workspace_bytes(layer.cfg, 2, 64, 0)
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    z = torch.zeros(2, 2, 4, dtype=torch.int32, device="cuda")
    q = torch.zeros(2, 8, 128, dtype=torch.bfloat16, device="cuda")
    c = layer.cache
    with pytest.raises(B.SnapError) as e:
        B.snap_decode_attn_blocks(layer.cfg, layer.layout, q, None, None, torch.zeros(2, dtype=torch.int32, device="cuda"), 2,
                                  c.k_cache, c.v_cache, c.seq_len, c.valid_topk, 64, 4, z, z[:, :, 0].contiguous(), q.clone(),
                                  small, c.status)
    assert e.value.code == -3                                   # workspace too small
