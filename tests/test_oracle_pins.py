"""Pins for the CPU oracle: values the paper prints, closed forms, invariants, special
cases that reduce to library routines, brute force on tiny inputs.  No GPU needed."""
import itertools
import math
import os

import numpy as np
import pytest
import scipy.special

from oracle import snapstream_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _cfg(**kw):
    base = dict(n_q_heads=4, n_kv_heads=2, d_qk=16, d_v=16, l_sink=2, l_recent=8, topk=6,
                l_obs=4, pool_kernel=3, softmax_scale=0.25)
    base.update(kw)
    return orc.OracleConfig(**base)


def _rand_prompt(cfg, L, seed, sharp=1.0):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((cfg.n_q_heads, cfg.l_obs, cfg.d_qk)) * sharp
    k = rng.standard_normal((L, cfg.n_kv_heads, cfg.d_qk))
    v = None if cfg.v_aliases_k else rng.standard_normal((L, cfg.n_kv_heads, cfg.d_v))
    return q, k, v


# ------------------------------------------------------------------ paper-printed values

def _read_golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def test_fig4_ring_example():
    """Fig. 4 caption + Eq. 3: L=26, Ls=1, Lr=4."""
    rows = _read_golden("fig4_ring_example.txt")
    kv = {r[0]: r[1:] for r in rows if r[0] not in ("eq3",)}
    Ls, Lr, L = int(kv["l_sink"][0]), int(kv["l_recent"][0]), int(kv["prompt_len"][0])
    r1 = (int(kv["range1"][0]), int(kv["range1"][1]))
    r2 = (int(kv["range2"][0]), int(kv["range2"][1]))
    # both ranges are ring-aligned: position p of a range sits at ring index p - start
    for start, end in (r1, r2):
        assert end - start + 1 == Lr
        for p in range(start, end + 1):
            assert orc.slot_of_position(p, Ls, Lr) - Ls == p - start
    # ring indices 0-1 hold range-2 positions, 2-3 hold range-1 positions (prompt tokens only)
    ring = {orc.slot_of_position(p, Ls, Lr) - Ls: p for p in range(L - Lr, L)}
    assert ring[0] == r2[0] and ring[2] == r1[0] + 2 and ring[3] == r1[0] + 3
    # token 27 replaces token 23
    new, old = (int(x) for x in kv["replaced_by"])
    assert orc.ring_write_slot(new, Ls, Lr) == orc.slot_of_position(old, Ls, Lr)
    # Eq. 3 values
    for r in rows:
        if r[0] == "eq3":
            assert orc.ring_write_slot(int(r[1]), Ls, Lr) == int(r[2])


def test_fig4_deque_evicts_what_ring_overwrites():
    """The rolling-window deque (naive update) and Eq. 3 agree on who is evicted."""
    cfg = _cfg(n_q_heads=1, n_kv_heads=1, l_sink=1, l_recent=4, topk=0, l_obs=1, pool_kernel=1)
    q, k, v = _rand_prompt(cfg, 26, 0)
    seq = orc.compress(q, k, v, cfg)
    assert list(seq.recents) == [22, 23, 24, 25]
    rng = np.random.default_rng(1)
    orc.decode_step(seq, rng.standard_normal((1, 16)), rng.standard_normal((1, 16)), rng.standard_normal((1, 16)))
    assert list(seq.recents) == [23, 24, 25, 26]        # 22 evicted by 26
    orc.decode_step(seq, rng.standard_normal((1, 16)), rng.standard_normal((1, 16)), rng.standard_normal((1, 16)))
    assert list(seq.recents) == [24, 25, 26, 27]        # 23 evicted by 27 (the caption's statement)


def test_hyperparameter_table_totals():
    for model, sink, topk, recent, total, obs, kern in _read_golden("hyperparameters_table.txt"):
        lay = orc.cache_layout(int(sink), int(recent), int(topk))
        assert lay["slots"] == int(total)
        assert lay["ring_off"] == int(sink) and lay["topk_off"] == int(sink) + int(recent)
        assert int(obs) <= int(recent) and int(kern) % 2 == 1


# ------------------------------------------------------------------ closed forms

def test_valid_topk_cases():
    Ls, Lr, K = 4, 16, 10
    assert orc.valid_topk(2, Ls, Lr, K) == 0            # L < Ls
    assert orc.valid_topk(12, Ls, Lr, K) == 0           # Ls <= L < Lsr
    assert orc.valid_topk(20, Ls, Lr, K) == 0           # L == Lsr
    assert orc.valid_topk(25, Ls, Lr, K) == 5           # Lsr < L < Lsr + K
    assert orc.valid_topk(30, Ls, Lr, K) == 10          # L == Lsr + K
    assert orc.valid_topk(1000, Ls, Lr, K) == 10        # L > Lsr + K


@pytest.mark.parametrize("Ls,Lr", [(0, 1), (0, 5), (1, 4), (4, 256), (768, 1024), (3, 7)])
def test_eq3_matches_closed_form_and_is_a_ring(Ls, Lr):
    for t in range(0, Ls + 5 * Lr + 3):
        s = orc.ring_write_slot(t, Ls, Lr)
        assert s == orc.slot_of_position(t, Ls, Lr)
        if t < Ls:
            assert s == t
        else:
            assert Ls <= s < Ls + Lr
            # period Lr, and consecutive tokens take consecutive ring slots
            assert orc.ring_write_slot(t + Lr, Ls, Lr) == s
            assert (orc.ring_write_slot(t + 1, Ls, Lr) - Ls) == (s - Ls + 1) % Lr
    # Case 1: while L < Lsr the layout is the plain one, slot == position
    for t in range(Ls + Lr):
        assert orc.ring_write_slot(t, Ls, Lr) == t


def test_ring_holds_exactly_the_deque_after_every_step():
    cfg = _cfg(n_q_heads=2, n_kv_heads=2, l_sink=3, l_recent=5, topk=4, l_obs=2, pool_kernel=3)
    for L in (1, 2, 3, 4, 7, 8, 9, 13, 30):
        q, k, v = _rand_prompt(cfg, L, L)
        seq = orc.compress(q, k, v, cfg)
        ring = {}       # slot -> position, maintained with Eq. 3 only
        for p in range(L):
            ring[orc.ring_write_slot(p, cfg.l_sink, cfg.l_recent)] = p
        rng = np.random.default_rng(L)
        for step in range(14):
            Kc, Vc, pos_map = orc.expected_cache(seq)
            held = sorted(p for s, p in ring.items())
            assert held == sorted(list(seq.sinks) + list(seq.recents))
            for s, p in ring.items():
                assert pos_map[0, s] == p
                np.testing.assert_array_equal(Kc[1, s], seq.k_hist[p][1])
            t = seq.n_tokens
            orc.decode_step(seq, rng.standard_normal((2, 16)), rng.standard_normal((2, 16)),
                            rng.standard_normal((2, 16)))
            ring[orc.ring_write_slot(t, cfg.l_sink, cfg.l_recent)] = t


# ------------------------------------------------------------------ score invariants

@pytest.mark.parametrize("seed,sharp", [(0, 1.0), (1, 4.0), (2, 0.1)])
def test_scores_sum_to_window_times_group(seed, sharp):
    cfg = _cfg(n_q_heads=6, n_kv_heads=2, l_obs=5, topk=3)
    q, k, _ = _rand_prompt(cfg, 60, seed, sharp)
    C = orc.observation_scores(q, k, cfg)
    assert C.shape == (2, 60 - 10)
    np.testing.assert_allclose(C.sum(axis=1), cfg.l_obs * cfg.group, rtol=1e-12)
    assert (C >= 0).all()


def test_avg_pool_weighted_sum_identity():
    rng = np.random.default_rng(3)
    for n, w in [(50, 7), (9, 3), (5, 13), (1, 5), (40, 1)]:
        C = rng.random((3, n))
        P = orc.pool_scores(C, w, "avg")
        r = w // 2
        i = np.arange(n)
        cover = np.minimum(i, r) + np.minimum(n - 1 - i, r) + 1
        np.testing.assert_allclose(P.sum(axis=1), (C * cover).sum(axis=1) / w, rtol=1e-12)
    np.testing.assert_array_equal(orc.pool_scores(C, 1, "avg"), C)
    np.testing.assert_array_equal(orc.pool_scores(C, 1, "max"), C)


def test_pool_against_direct_window_loops():
    rng = np.random.default_rng(4)
    C = rng.random(23)
    for w in (3, 5, 7):
        r = w // 2
        avg = [sum(C[j + t] for t in range(-r, r + 1) if 0 <= j + t < 23) / w for j in range(23)]
        mx = [max(C[j + t] for t in range(-r, r + 1) if 0 <= j + t < 23) for j in range(23)]
        np.testing.assert_allclose(orc.pool_scores(C[None], w, "avg")[0], avg, rtol=1e-14)
        np.testing.assert_array_equal(orc.pool_scores(C[None], w, "max")[0], mx)


def test_avg_pool_commutes_with_group_sum():
    rng = np.random.default_rng(5)
    parts = rng.random((4, 37))
    a = orc.pool_scores(parts.sum(axis=0, keepdims=True), 7, "avg")[0]
    b = orc.pool_scores(parts, 7, "avg").sum(axis=0)
    np.testing.assert_allclose(a, b, rtol=1e-13)


def test_zero_queries_give_edge_and_tie_pattern():
    """Q_obs = 0 makes every candidate score equal; zero-padded averaging lowers the first
    and last w//2 entries, so the K winners are candidates [r, r+K); max pooling keeps all
    equal, so the winners are [0, K) by the lower-index rule."""
    cfg = _cfg(n_q_heads=2, n_kv_heads=1, l_sink=3, l_recent=8, topk=5, l_obs=4, pool_kernel=5)
    L = 40
    _, k, v = _rand_prompt(cfg, L, 6)
    q0 = np.zeros((2, 4, 16))
    idx, _ = orc.snapkv_select(q0, k, cfg)
    r = cfg.pool_kernel // 2
    np.testing.assert_array_equal(idx[0], cfg.l_sink + r + np.arange(cfg.topk))
    cfg_max = _cfg(n_q_heads=2, n_kv_heads=1, l_sink=3, l_recent=8, topk=5, l_obs=4, pool_kernel=5,
                   pool_mode="max")
    idx, _ = orc.snapkv_select(q0, k, cfg_max)
    np.testing.assert_array_equal(idx[0], cfg.l_sink + np.arange(cfg.topk))


def test_single_row_case_matches_scipy_softmax():
    """w=1, Lo=1, g=1: the score of a head is one softmax row over the candidates."""
    cfg = _cfg(n_q_heads=2, n_kv_heads=2, l_obs=1, pool_kernel=1, topk=4, l_sink=2, l_recent=3)
    L = 31
    q, k, _ = _rand_prompt(cfg, L, 7, sharp=2.0)
    C = orc.observation_scores(q, k, cfg)
    for h in range(2):
        logits = cfg.softmax_scale * np.einsum("d,jd->j", q[h, 0], k[cfg.l_sink:L - cfg.l_recent, h])
        ref = scipy.special.softmax(logits)
        np.testing.assert_allclose(C[h], ref, rtol=1e-12)
        idx, _ = orc.snapkv_select(q, k, cfg)
        np.testing.assert_array_equal(idx[h], cfg.l_sink + np.sort(np.argsort(-ref, kind="stable")[:4]))


def test_scores_use_last_obs_queries_and_right_kv_head():
    """A key aligned with the queries of one query head raises only its KV head's score
    at exactly that candidate; keys outside the candidate range never appear."""
    cfg = _cfg(n_q_heads=4, n_kv_heads=2, l_sink=2, l_recent=6, l_obs=3, pool_kernel=1, topk=1,
               softmax_scale=1.0)
    L = 30
    rng = np.random.default_rng(8)
    q = np.zeros((4, 3, 16))
    k = rng.standard_normal((L, 2, 16)) * 0.01
    d = np.zeros(16); d[5] = 1.0
    q[3] = 10.0 * d                       # query head 3 belongs to KV head 1
    k[11, 1] = 3.0 * d                    # candidate position 11, KV head 1
    k[1, 1] = 50.0 * d                    # a sink: not a candidate
    k[L - 6, 1] = 50.0 * d                # first recent token: not a candidate
    k[11, 0] = -3.0 * d                   # other KV head must not see head 3's queries
    C = orc.observation_scores(q, k, cfg)
    assert C.shape == (2, L - 8)
    assert np.argmax(C[1]) == 11 - cfg.l_sink
    assert C[1].max() > 3.0 - 1e-6        # three obs rows of head 3 put ~all weight there (+ head 2 uniform)
    np.testing.assert_allclose(C[0], cfg.l_obs * cfg.group / (L - 8), rtol=1e-3)
    idx, _ = orc.snapkv_select(q, k, cfg)
    assert list(idx[1]) == [11]


def test_candidate_range_boundaries_are_selectable():
    cfg = _cfg(n_q_heads=1, n_kv_heads=1, l_sink=2, l_recent=6, l_obs=2, pool_kernel=1, topk=2,
               softmax_scale=1.0)
    L = 25
    q = np.zeros((1, 2, 16)); q[..., 0] = 5.0
    k = np.zeros((L, 1, 16))
    k[cfg.l_sink, 0, 0] = 2.0             # first candidate
    k[L - cfg.l_recent - 1, 0, 0] = 2.0   # last candidate
    idx, _ = orc.snapkv_select(q, k, cfg)
    assert list(idx[0]) == [cfg.l_sink, L - cfg.l_recent - 1]


def test_scores_against_pure_python_brute_force():
    cfg = _cfg(n_q_heads=4, n_kv_heads=2, d_qk=3, d_v=3, l_sink=1, l_recent=2, l_obs=2, topk=2,
               pool_kernel=3, softmax_scale=0.7)
    L = 9
    q, k, _ = _rand_prompt(cfg, L, 9)
    C = orc.observation_scores(q, k, cfg)
    for kvh in range(2):
        for j in range(1, L - 2):
            tot = 0.0
            for h in (2 * kvh, 2 * kvh + 1):
                for i in range(2):
                    logit = lambda jj: 0.7 * sum(q[h, i, c] * k[jj, kvh, c] for c in range(3))
                    z = sum(math.exp(logit(jj)) for jj in range(1, L - 2))
                    tot += math.exp(logit(j)) / z
            assert abs(C[kvh, j - 1] - tot) < 1e-13


# ------------------------------------------------------------------ top-k

def test_topk_equals_brute_force_with_duplicates():
    rng = np.random.default_rng(10)
    for trial in range(200):
        n = int(rng.integers(1, 12))
        K = int(rng.integers(0, 8))
        P = rng.integers(0, 4, size=n).astype(np.float64)     # many exact duplicates
        got = list(orc.select_topk(P, K))
        if n <= K:
            assert got == list(range(n))
            continue
        # brute force: among all K-subsets take the one maximising (sum of scores, then lexicographically
        # smallest indices) -- equivalent to "largest first, ties to the lower index"
        best = None
        for comb in itertools.combinations(range(n), K):
            key = (-sum(P[list(comb)]), comb)
            if best is None or key < best:
                best = key
        assert got == list(best[1])


def test_topk_plain_cases():
    np.testing.assert_array_equal(orc.select_topk(np.array([0.1, 0.9, 0.5, 0.7]), 2), [1, 3])
    np.testing.assert_array_equal(orc.select_topk(np.array([1.0, 1.0, 1.0, 1.0]), 2), [0, 1])
    np.testing.assert_array_equal(orc.select_topk(np.array([0.0, 2.0, 2.0, 1.0, 2.0]), 2), [1, 2])
    assert len(orc.select_topk(np.array([3.0, 1.0]), 0)) == 0


# ------------------------------------------------------------------ retained set and attention

def test_sinks_and_window_always_retained_and_topk_never_changes():
    cfg = _cfg()
    L = 50
    q, k, v = _rand_prompt(cfg, L, 11)
    seq = orc.compress(q, k, v, cfg)
    top0 = [p.copy() for p in seq.topk_pos]
    rng = np.random.default_rng(12)
    for step in range(20):
        for kvh in range(cfg.n_kv_heads):
            ret = seq.retained(kvh)
            assert len(set(ret)) == len(ret) == cfg.l_sink + cfg.l_recent + cfg.topk
            assert set(range(cfg.l_sink)) <= set(ret)
            assert set(range(seq.n_tokens - cfg.l_recent, seq.n_tokens)) <= set(ret)
            np.testing.assert_array_equal(seq.topk_pos[kvh], top0[kvh])
            assert all(cfg.l_sink <= p < L - cfg.l_recent for p in seq.topk_pos[kvh])
        orc.decode_step(seq, rng.standard_normal((4, 16)), rng.standard_normal((2, 16)),
                        rng.standard_normal((2, 16)))


def test_budget_at_least_prompt_equals_dense_attention():
    """(i) L + steps <= Lsr: nothing is ever evicted; (ii) K >= Le: attend-only equals dense."""
    rng = np.random.default_rng(13)
    cfg = _cfg(l_sink=4, l_recent=40, topk=3)
    q, k, v = _rand_prompt(cfg, 20, 13)
    seq = orc.compress(q, k, v, cfg)
    for step in range(10):
        qd = rng.standard_normal((4, 16)) * 3
        out = orc.decode_step(seq, qd, rng.standard_normal((2, 16)), rng.standard_normal((2, 16)))
        np.testing.assert_allclose(out, orc.dense_attention(seq, qd), rtol=1e-12, atol=1e-14)
    cfg2 = _cfg(l_sink=2, l_recent=8, topk=64)
    q, k, v = _rand_prompt(cfg2, 50, 14)
    seq = orc.compress(q, k, v, cfg2)
    assert all(len(p) == 40 for p in seq.topk_pos)
    qd = rng.standard_normal((4, 16)) * 3
    np.testing.assert_allclose(orc.attend(seq, qd), orc.dense_attention(seq, qd), rtol=1e-12, atol=1e-14)


def test_attention_matches_masked_dense_and_is_order_invariant():
    cfg = _cfg()
    q, k, v = _rand_prompt(cfg, 64, 15)
    seq = orc.compress(q, k, v, cfg)
    rng = np.random.default_rng(16)
    qd = rng.standard_normal((4, 16)) * 2
    out = orc.decode_step(seq, qd, rng.standard_normal((2, 16)), rng.standard_normal((2, 16)))
    K_all = np.stack(seq.k_hist); V_all = np.stack(seq.v_hist)
    for h in range(4):
        kvh = h // 2
        mask = np.full(seq.n_tokens, -np.inf)
        mask[seq.retained(kvh)] = 0.0
        w = scipy.special.softmax(cfg.softmax_scale * (K_all[:, kvh] @ qd[h]) + mask)
        np.testing.assert_allclose(out[h], w @ V_all[:, kvh], rtol=1e-12, atol=1e-14)
    # order of the rows does not matter
    pos = seq.retained(0)
    perm = rng.permutation(len(pos))
    Kr = np.stack([seq.k_hist[p][0] for p in pos]); Vr = np.stack([seq.v_hist[p][0] for p in pos])
    a = orc.attention_over(qd[0], Kr, Vr, cfg.softmax_scale)
    b = orc.attention_over(qd[0], Kr[perm], Vr[perm], cfg.softmax_scale)
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-14)


def test_single_valid_slot_returns_its_value():
    cfg = _cfg(n_q_heads=2, n_kv_heads=1, l_sink=2, l_recent=4, topk=2, l_obs=1)
    rng = np.random.default_rng(17)
    seq = orc.OracleSequence(cfg, topk_pos=[np.zeros(0, dtype=np.int64)])
    k0, v0 = rng.standard_normal((1, 16)), rng.standard_normal((1, 16))
    out = orc.decode_step(seq, rng.standard_normal((2, 16)), k0, v0)
    np.testing.assert_allclose(out, np.repeat(v0, 2, axis=0), rtol=1e-14)


def test_latent_layout_value_is_prefix_of_key_row():
    cfg = _cfg(n_q_heads=4, n_kv_heads=1, d_qk=24, d_v=16, v_aliases_k=True, l_obs=2)
    q, k, _ = _rand_prompt(cfg, 40, 18)
    seq = orc.compress(q, k, None, cfg)
    rng = np.random.default_rng(19)
    qd = rng.standard_normal((4, 24))
    out = orc.decode_step(seq, qd, rng.standard_normal((1, 24)), None)
    pos = seq.retained(0)
    Kr = np.stack([seq.k_hist[p][0] for p in pos])
    for h in range(4):
        w = scipy.special.softmax(cfg.softmax_scale * Kr @ qd[h])
        np.testing.assert_allclose(out[h], w @ Kr[:, :16], rtol=1e-12)
    Kc, Vc, pos_map = orc.expected_cache(seq)
    assert Vc is None and Kc.shape == (1, cfg.l_sr + cfg.topk, 24)


def test_expected_cache_sections():
    cfg = _cfg(l_sink=3, l_recent=5, topk=6)
    # Case 1 (L < Lsr): plain layout, slot == position, top-K section all padding
    q, k, v = _rand_prompt(cfg, 6, 20)
    seq = orc.compress(q, k, v, cfg)
    Kc, Vc, pos_map = orc.expected_cache(seq)
    assert list(pos_map[0]) == [0, 1, 2, 3, 4, 5, -1, -1] + [-1] * 6
    assert not Kc[:, 6:].any()
    # Lsr < L <= Lsr + K: all candidates kept, valid rows first, pads after
    q, k, v = _rand_prompt(cfg, 12, 21)
    seq = orc.compress(q, k, v, cfg)
    Kc, Vc, pos_map = orc.expected_cache(seq)
    assert orc.valid_topk(12, 3, 5, 6) == 4
    assert list(pos_map[1][8:]) == [3, 4, 5, 6, -1, -1]
    assert sorted(pos_map[1][3:8]) == [7, 8, 9, 10, 11]
    np.testing.assert_array_equal(Vc[1, 8], v[3, 1])
    # L > Lsr + K: exactly K selected, ascending
    q, k, v = _rand_prompt(cfg, 40, 22)
    seq = orc.compress(q, k, v, cfg)
    _, _, pos_map = orc.expected_cache(seq)
    top = pos_map[0][8:]
    assert (top >= 0).all() and (np.diff(top) > 0).all()


def test_planted_heavy_hitters_are_selected():
    """Statistical sanity on the synthetic recipe used by the benchmark configs."""
    from paper_2511_03092_b200 import synth
    wl = synth.CONFIGS[0].scaled(prompt_len=(1024, 1024), topk=128, l_recent=64, n_planted=16)
    p = synth.make_prompt(wl, 1024, seed=5)
    cfg = orc.OracleConfig(wl.n_q_heads, wl.n_kv_heads, wl.d_qk, wl.d_v, wl.l_sink, wl.l_recent,
                           wl.topk, wl.l_obs, wl.pool_kernel, wl.scale)
    idx, P = orc.snapkv_select(synth.to_f64(p["q_obs"]), synth.to_f64(p["k"]), cfg)
    for h in range(wl.n_kv_heads):
        hit = len(set(p["planted"][h]) & set(idx[h])) / len(p["planted"][h])
        assert hit >= 0.7          # chance level would be topk / candidates = 0.13


def test_position_order_image_equals_repeated_array_concatenation():
    """Section 3.2.1's slice-and-concatenate update, done literally on arrays, step by step,
    gives the position-ordered cache image; it holds the same rows as the ring image, and the
    two images coincide when the ring's write pointer is back at the window start."""
    cfg = _cfg()
    Ls, Lr, Lsr = cfg.l_sink, cfg.l_recent, cfg.l_sr
    L = Ls + 3 * Lr                              # ring pointer at the window start
    q, k, v = _rand_prompt(cfg, L, seed=21)
    seq = orc.compress(q, k, v, cfg)
    K0, V0, _ = orc.expected_cache(seq)
    Kp, Vp, _ = orc.expected_cache_position_order(seq)
    np.testing.assert_array_equal(K0, Kp)
    np.testing.assert_array_equal(V0, Vp)
    rng = np.random.default_rng(5)
    Kc, Vc = K0.copy(), V0.copy()
    for step in range(2 * Lr + 3):
        kn = rng.standard_normal((cfg.n_kv_heads, cfg.d_qk))
        vn = rng.standard_normal((cfg.n_kv_heads, cfg.d_v))
        orc.decode_step(seq, rng.standard_normal((cfg.n_q_heads, cfg.d_qk)), kn, vn)
        Kc = np.concatenate([Kc[:, :Ls], Kc[:, Ls + 1:Lsr], kn[:, None], Kc[:, Lsr:]], axis=1)
        Vc = np.concatenate([Vc[:, :Ls], Vc[:, Ls + 1:Lsr], vn[:, None], Vc[:, Lsr:]], axis=1)
        Kp, Vp, pm = orc.expected_cache_position_order(seq)
        np.testing.assert_array_equal(Kc, Kp)
        np.testing.assert_array_equal(Vc, Vp)
        Kr, Vr, pr = orc.expected_cache(seq)
        for kvh in range(cfg.n_kv_heads):
            assert sorted(pm[kvh].tolist()) == sorted(pr[kvh].tolist())
        if (seq.n_tokens - Ls) % Lr == 0:
            np.testing.assert_array_equal(Kr, Kp)


# ------------------------------------------------------------------ prefill attention + Eq. 4 normalisers

def test_prefill_attention_matches_the_library_causal_routine_and_closed_forms():
    import torch
    cfg = _cfg()
    rng = np.random.default_rng(71)
    L = 37
    q = rng.standard_normal((L, cfg.n_q_heads, cfg.d_qk))
    k = rng.standard_normal((L, cfg.n_kv_heads, cfg.d_qk))
    v = rng.standard_normal((L, cfg.n_kv_heads, cfg.d_v))
    out = orc.prefill_attention(q, k, v, cfg)
    # library routine: torch's fused causal attention in double precision, heads expanded
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(cfg.group, dim=0)[None]
    tv = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(cfg.group, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=cfg.softmax_scale)
    np.testing.assert_allclose(out, ref[0].permute(1, 0, 2).numpy(), rtol=1e-12, atol=1e-13)
    # the first token sees only itself
    for h in range(cfg.n_q_heads):
        np.testing.assert_allclose(out[0, h], v[0, h // cfg.group], rtol=0, atol=1e-15)
    # equal keys: uniform weights, the output is the running mean of the values
    k_same = np.broadcast_to(k[:1], k.shape)
    out_same = orc.prefill_attention(q, k_same, v, cfg)
    running = np.cumsum(v, axis=0) / np.arange(1, L + 1)[:, None, None]
    for h in range(cfg.n_q_heads):
        np.testing.assert_allclose(out_same[:, h], running[:, h // cfg.group], rtol=1e-12, atol=1e-13)
    # a future token cannot change an earlier row
    k2, v2 = k.copy(), v.copy()
    k2[20:] += 3.0
    v2[20:] -= 5.0
    np.testing.assert_array_equal(orc.prefill_attention(q, k2, v2, cfg)[:20], out[:20])


def test_candidate_normalisers_are_the_library_logsumexp_and_rebuild_eq1():
    cfg = _cfg()
    L = 61
    q, k, _ = _rand_prompt(cfg, L, seed=72, sharp=2.0)
    mu = orc.candidate_log2_normalisers(q, k, cfg)
    lo, hi = cfg.l_sink, L - cfg.l_recent
    C = np.zeros((cfg.n_kv_heads, hi - lo))
    for h in range(cfg.n_q_heads):
        S = cfg.softmax_scale * np.einsum("id,jd->ij", q[h], k[lo:hi, h // cfg.group])
        np.testing.assert_allclose(mu[h], scipy.special.logsumexp(S, axis=1) / math.log(2.0), rtol=1e-13)
        C[h // cfg.group] += np.exp2(S * math.log2(math.e) - mu[h][:, None]).sum(axis=0)
    # weights rebuilt from the normalisers are Eq. 4's, so their window sum is Eq. 1
    np.testing.assert_allclose(C, orc.observation_scores(q, k, cfg), rtol=1e-11)
    # a prompt that fits the budget has no candidate
    assert np.all(np.isneginf(orc.candidate_log2_normalisers(q, k[: cfg.l_sink + cfg.l_recent], cfg)))
