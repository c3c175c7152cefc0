"""Pins of the oracle's per-step block top-K functions (no GPU): the bound property that defines the
block score, values worked by hand, the one-token-block special case against a brute-force top-k by
logit, equality with attention over everything kept when every block is selected, what the
statistics may and may not see, and the tie rule."""
import numpy as np
import pytest

from oracle import snapstream_oracle as orc


def _cfg(hq=4, hkv=2, d=8, ls=2, lr=4, **kw):
    base = dict(n_q_heads=hq, n_kv_heads=hkv, d_qk=d, d_v=d, l_sink=ls, l_recent=lr, topk=10 ** 6, l_obs=2,
                pool_kernel=1, softmax_scale=0.37)
    base.update(kw)
    return orc.OracleConfig(**base)


def test_block_scores_worked_by_hand():
    """One head, two dims, blocks of two tokens; every number below is pencil arithmetic on the definition:
    block 0 = keys (1, -2), (3, 0): min (1, -2), max (3, 0); q = (2, -1): max(2, 6) + max(2, 0) = 8.
    block 1 = keys (-1, 4), (-3, 5): min (-3, 4), max (-1, 5); q = (2, -1): max(-6, -2) + max(-4, -5) = -6.
    block 2 (one token left) = key (0.5, 0.5): 1 - 0.5 = 0.5."""
    cfg = _cfg(hq=1, hkv=1, d=2, ls=1, lr=1)
    k = np.array([[9, 9], [1, -2], [3, 0], [-1, 4], [-3, 5], [0.5, 0.5], [-9, -9]], dtype=np.float64)[:, None, :]
    kmin, kmax = orc.block_statistics(k, cfg, 2)
    assert kmin.shape == (1, 3, 2)
    assert kmin[0].tolist() == [[1, -2], [-3, 4], [0.5, 0.5]]
    assert kmax[0].tolist() == [[3, 0], [-1, 5], [0.5, 0.5]]
    U = orc.block_upper_bounds(np.array([[2.0, -1.0]]), kmin, kmax, cfg)
    assert U[0].tolist() == [8.0, -6.0, 0.5]
    assert orc.select_blocks(U[0], 2).tolist() == [0, 2]
    assert orc.block_positions(np.array([0, 2]), 7, cfg, 2).tolist() == [1, 2, 5]   # the short last block has one token


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_block_score_bounds_every_key_of_the_block_and_is_tight_for_constant_blocks(seed):
    rng = np.random.default_rng(seed)
    cfg = _cfg()
    L, bs = 61, 8
    k = rng.normal(size=(L, cfg.n_kv_heads, cfg.d_qk))
    k[cfg.l_sink + 16:cfg.l_sink + 24] = k[cfg.l_sink + 16]    # block 2: eight identical keys
    q = rng.normal(size=(cfg.n_q_heads, cfg.d_qk))
    kmin, kmax = orc.block_statistics(k, cfg, bs)
    U = orc.block_upper_bounds(q, kmin, kmax, cfg)
    Le = L - cfg.l_sr
    for kvh in range(cfg.n_kv_heads):
        qs = q[kvh * cfg.group:(kvh + 1) * cfg.group]
        for j in range(Le):
            logit = float(sum(qh @ k[cfg.l_sink + j, kvh] for qh in qs))
            assert logit <= U[kvh, j // bs] + 1e-12
        exact = float(sum(qh @ k[cfg.l_sink + 16, kvh] for qh in qs))
        assert abs(U[kvh, 2] - exact) < 1e-12          # min = max: the bound is the logit itself


def test_one_token_blocks_reduce_to_top_k_by_group_summed_logit():
    rng = np.random.default_rng(7)
    cfg = _cfg(hq=6, hkv=2, d=5, ls=3, lr=5)
    L = 40
    k = rng.normal(size=(L, cfg.n_kv_heads, cfg.d_qk))
    q = rng.normal(size=(cfg.n_q_heads, cfg.d_qk))
    kmin, kmax = orc.block_statistics(k, cfg, 1)
    U = orc.block_upper_bounds(q, kmin, kmax, cfg)
    for kvh in range(cfg.n_kv_heads):
        logits = [sum(float(q[h] @ k[p, kvh]) for h in range(kvh * cfg.group, (kvh + 1) * cfg.group))
                  for p in range(cfg.l_sink, L - cfg.l_recent)]
        assert np.allclose(U[kvh], logits, atol=1e-12)
        brute = sorted(sorted(range(len(logits)), key=lambda j: (-logits[j], j))[:7])
        chosen = orc.select_blocks(U[kvh], 7)
        assert chosen.tolist() == brute
        assert orc.block_positions(chosen, L, cfg, 1).tolist() == [cfg.l_sink + j for j in brute]


def test_statistics_see_only_the_middle_of_the_prompt():
    rng = np.random.default_rng(3)
    cfg = _cfg()
    L = 30
    k = rng.normal(size=(L, cfg.n_kv_heads, cfg.d_qk))
    ref = orc.block_statistics(k, cfg, 4)
    k2 = k.copy()
    k2[:cfg.l_sink] = 1e6                               # sinks
    k2[L - cfg.l_recent:] = -1e6                        # recent window
    got = orc.block_statistics(k2, cfg, 4)
    assert np.array_equal(ref[0], got[0]) and np.array_equal(ref[1], got[1])
    assert ref[0].shape[1] == -(-(L - cfg.l_sr) // 4)
    k3 = k.copy()
    k3[cfg.l_sink + 5, 1, 2] = 77.0                     # a middle token: block 1 of KV head 1, dim 2 only
    got = orc.block_statistics(k3, cfg, 4)
    assert got[1][1, 1, 2] == 77.0 and np.array_equal(got[0], ref[0])
    changed = got[1] != ref[1]
    assert changed.sum() == 1 and changed[1, 1, 2]
    assert orc.block_statistics(k[:cfg.l_sr], cfg, 4)[0].shape[1] == 0   # nothing between sinks and window


def test_equal_scores_go_to_the_lower_block_index():
    assert orc.select_blocks(np.array([1.0, 3.0, 3.0, 3.0, 0.0]), 2).tolist() == [1, 2]
    assert orc.select_blocks(np.zeros(6), 3).tolist() == [0, 1, 2]
    assert orc.select_blocks(np.array([2.0, 1.0]), 5).tolist() == [0, 1]      # fewer blocks than the budget: all


def test_all_blocks_selected_is_attention_over_everything_kept():
    """With every block selected a query attends over sinks, the whole middle and the window: dense
    attention as long as nothing has left the window (i.e. on the prompt itself), and afterwards
    exactly `decode_step` on a sequence that kept the whole middle."""
    rng = np.random.default_rng(11)
    cfg = _cfg(hq=4, hkv=2, d=6, ls=2, lr=5)
    L, bs = 37, 4
    k = rng.normal(size=(L, cfg.n_kv_heads, cfg.d_qk))
    v = rng.normal(size=(L, cfg.n_kv_heads, cfg.d_v))
    q_obs = rng.normal(size=(cfg.n_q_heads, cfg.l_obs, cfg.d_qk))
    kmin, kmax = orc.block_statistics(k, cfg, bs)
    nb = kmin.shape[1]
    a = orc.compress(q_obs, k, v, cfg)
    b = orc.compress(q_obs, k, v, cfg)
    q0 = rng.normal(size=(cfg.n_q_heads, cfg.d_qk))
    a.topk_pos = [orc.block_positions(np.arange(nb), L, cfg, bs) for _ in range(cfg.n_kv_heads)]
    assert np.allclose(orc.attend(a, q0), orc.dense_attention(a, q0), atol=1e-12)
    for step in range(8):
        q = rng.normal(size=(cfg.n_q_heads, cfg.d_qk))
        kn = rng.normal(size=(cfg.n_kv_heads, cfg.d_qk))
        vn = rng.normal(size=(cfg.n_kv_heads, cfg.d_v))
        out_a, chosen = orc.block_decode_step(a, L, kmin, kmax, nb, bs, q, kn, vn)
        out_b = orc.decode_step(b, q, kn, vn)
        assert [c.tolist() for c in chosen] == [list(range(nb))] * cfg.n_kv_heads
        assert np.allclose(out_a, out_b, atol=1e-13)


def test_block_lookup_changes_the_retained_set_per_step_only_in_its_middle_part():
    rng = np.random.default_rng(5)
    cfg = _cfg(hq=2, hkv=1, d=4, ls=1, lr=3)
    L, bs = 26, 4
    k = rng.normal(size=(L, 1, 4))
    k[9:13] *= 30.0                                     # block 2 (positions 9..12) dominates for an aligned query
    v = rng.normal(size=(L, 1, 4))
    seq = orc.compress(rng.normal(size=(2, 2, 4)), k, v, cfg)
    kmin, kmax = orc.block_statistics(k, cfg, bs)
    q = np.stack([k[10, 0], k[10, 0]])
    out, chosen = orc.block_decode_step(seq, L, kmin, kmax, 1, bs, q, rng.normal(size=(1, 4)), rng.normal(size=(1, 4)))
    assert chosen[0].tolist() == [2]
    assert seq.retained(0) == [0] + [9, 10, 11, 12] + [24, 25, 26]
