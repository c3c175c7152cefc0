"""CPU oracle for the SnapStream hot path.  TEST INFRASTRUCTURE ONLY.

This file is a plain, slow, double-precision restatement of what the SnapStream
paper (arXiv 2511.03092) computes.  It exists so that the CUDA library can be
checked against something that can be compared with the paper by eye.  It is
imported only by the tests, by the smoke check and by the benchmark's
``cpu_baseline`` / ``--impl reference`` legs; the product path never calls it
and shares no code, table or helper with it.

Everything is numpy float64.  Library primitives used as steps: ``np.matmul``
(the Q K^T products), ``np.exp``, ``np.lexsort`` (the full sort behind top-k).
There is no blocking, fusion or reordering beyond what the paper states.

Notation (0-indexed token positions, prompt = positions 0..L-1):
  Ls = L_sink, Lr = L_recent, K = top-K budget, Lo = L_obs, w = pooling kernel,
  Lsr = Ls + Lr, Sc = Ls + Lr + K cache slots, Le = L - Lsr eviction candidates,
  Hq / Hkv query / KV heads, g = Hq // Hkv.

Readings of the paper adopted here (the paper is silent or inconsistent on them):
  * the observation window is exactly the last Lo prompt queries, positions
    [L-Lo, L)  (Section 3.2.2 writes q_{L-Lo}..q_L, Eq. 1 sums Lo+1 terms);
  * the recent window is exactly the last Lr tokens, candidates are positions
    [Ls, L-Lr)  -- their count L - Lsr is what Section 3 and the appendix's
    valid_topk expression use;
  * the softmax of Eq. 4 normalises over the eviction candidates only;
  * with grouped-query attention the g query heads of one KV head are summed
    before pooling, and one index set is chosen per KV head;
  * pooling is 1-D along the sequence over the candidate array only (stride 1,
    pad w//2; average divides by w with zero padding, max pads with -inf);
  * ties in the top-k go to the lower token index; the selected rows are stored
    in ascending position order, valid rows first, zero rows after;
  * the ring keeps all Lr prompt recents; position p >= Ls lives in cache slot
    Ls + (p - Ls) mod Lr, which is Eq. 3 evaluated at p;
  * a decode step writes the new token first and attends afterwards.

Parity pins (tests/test_oracle_*.py): Fig. 4's worked ring example, Eq. 3 against
the closed-form slot map, the appendix's valid_topk expression, the
hyper-parameter table totals, sum_j C = Lo*g, the weighted pooled-sum identity,
the all-equal tie pattern, brute-force top-k, the single-row softmax special case
against scipy, dense-attention equalities, permutation invariance; prefill attention
against torch's double-precision causal routine, the running-mean closed form and
causality; the Eq. 4 normalisers against scipy's logsumexp and by rebuilding Eq. 1.
Parity unpinned by the paper (fixed only by the readings above): which softmax
domain, pooling domain, GQA reduction order and ring-fill convention the
authors' own implementation uses; and the whole per-step block top-K section at
the end of this file, which the paper only names as future work (its definition
and its pins -- hand-worked values, the bound property, the one-token-block
special case, all blocks = everything kept -- are stated there and in
tests/test_oracle_blocks.py).
"""
from __future__ import annotations

from collections import deque
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np


@dataclass(frozen=True)
class OracleConfig:
    """Hyper-parameters of one attention layer (Table "SnapStream Hyperparameters")."""

    n_q_heads: int
    n_kv_heads: int
    d_qk: int
    d_v: int
    l_sink: int
    l_recent: int
    topk: int
    l_obs: int
    pool_kernel: int
    softmax_scale: float
    pool_mode: str = "avg"          # "avg" (Eq. 2) or "max"
    v_aliases_k: bool = False       # latent attention: V row = first d_v dims of K row

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def l_sr(self) -> int:
        return self.l_sink + self.l_recent


# ----------------------------------------------------------------------------
# Section 3.1: cache structure
# ----------------------------------------------------------------------------

def cache_layout(l_sink: int, l_recent: int, topk: int) -> dict:
    """Section 3 / 3.1: the cache is sink | recent ring | top-K, L_snapstream slots."""
    return {
        "slots": l_sink + l_recent + topk,
        "sink_off": 0,
        "ring_off": l_sink,
        "topk_off": l_sink + l_recent,
    }


def valid_topk(L: int, l_sink: int, l_recent: int, topk: int) -> int:
    """Number of real (non-padding) rows in the top-K section (Section 3.2.2, last
    paragraph; the appendix's prefill listings give min(max(L - Lsr, 0), K))."""
    return min(max(L - (l_sink + l_recent), 0), topk)


def ring_write_slot(t: int, l_sink: int, l_recent: int) -> int:
    """Eq. 3: cache slot that receives the token at 0-indexed position t.
    While the sink region is still filling (t < Ls) the token goes to slot t."""
    if t < l_sink:
        return t
    return (t - l_sink + l_recent) % l_recent + l_sink


def slot_of_position(p: int, l_sink: int, l_recent: int) -> int:
    """Closed form of where a retained non-top-K position lives: sinks at their own
    index, everything later at Ls + (p - Ls) mod Lr (ring, Section 3.2.1)."""
    if p < l_sink:
        return p
    return l_sink + (p - l_sink) % l_recent


# ----------------------------------------------------------------------------
# Section 3.2.2: SnapKV scoring on the eviction candidates (Eq. 4, Eq. 1, Eq. 2)
# ----------------------------------------------------------------------------

def observation_scores(q_obs: np.ndarray, k: np.ndarray, cfg: OracleConfig) -> np.ndarray:
    """C[kvh, j] for candidates j in [Ls, L-Lr)  (Eq. 4 then Eq. 1, summed over the
    query heads of each KV head).

    q_obs: [Hq, Lo, d_qk]  queries of prompt positions L-Lo .. L-1 (post-RoPE).
    k:     [L, Hkv, d_qk]  prompt keys.
    returns float64 [Hkv, Le].
    """
    q_obs = np.asarray(q_obs, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    L = k.shape[0]
    lo, hi = cfg.l_sink, L - cfg.l_recent
    assert hi > lo, "no eviction candidates"
    assert q_obs.shape == (cfg.n_q_heads, cfg.l_obs, cfg.d_qk)
    C = np.zeros((cfg.n_kv_heads, hi - lo), dtype=np.float64)
    for h in range(cfg.n_q_heads):
        kvh = h // cfg.group
        k_evict = k[lo:hi, kvh, :]                       # [Le, d]
        S = cfg.softmax_scale * (q_obs[h] @ k_evict.T)   # [Lo, Le]      Eq. 4 logits
        S = S - S.max(axis=1, keepdims=True)
        E = np.exp(S)
        W = E / E.sum(axis=1, keepdims=True)             # softmax over candidates
        C[kvh] += W.sum(axis=0)                          # Eq. 1: sum over the window
    return C


def pool_scores(C: np.ndarray, w: int, mode: str = "avg") -> np.ndarray:
    """Eq. 2's pooling: 1-D, kernel w, stride 1, padding w//2, along the sequence."""
    assert w >= 1 and w % 2 == 1
    C = np.asarray(C, dtype=np.float64)
    r = w // 2
    n = C.shape[-1]
    if mode == "avg":
        pad = np.zeros(C.shape[:-1] + (r,), dtype=np.float64)
        Cp = np.concatenate([pad, C, pad], axis=-1)
        P = np.zeros_like(C)
        for t in range(w):
            P += Cp[..., t:t + n]
        return P / w
    if mode == "max":
        pad = np.full(C.shape[:-1] + (r,), -np.inf, dtype=np.float64)
        Cp = np.concatenate([pad, C, pad], axis=-1)
        P = np.full_like(C, -np.inf)
        for t in range(w):
            P = np.maximum(P, Cp[..., t:t + n])
        return P
    raise ValueError(mode)


def select_topk(P_row: np.ndarray, K: int) -> np.ndarray:
    """Eq. 2's Top_K on one KV head: indices (into the candidate array) of the K
    largest pooled scores, ties to the lower index, returned in ascending order.
    Definition by full sort."""
    n = P_row.shape[0]
    if n <= K:
        return np.arange(n, dtype=np.int64)
    order = np.lexsort((np.arange(n), -P_row))   # primary -P ascending, then index
    return np.sort(order[:K]).astype(np.int64)


def snapkv_select(q_obs: np.ndarray, k: np.ndarray, cfg: OracleConfig):
    """Selected absolute prompt positions per KV head, plus the pooled scores.

    returns (idx, P): idx is a list of Hkv int64 arrays (ascending positions),
    P is float64 [Hkv, Le] or None when no scoring is needed (Le <= K)."""
    L = k.shape[0]
    Le = L - cfg.l_sr
    if Le <= 0 or cfg.topk == 0:
        return [np.zeros(0, dtype=np.int64) for _ in range(cfg.n_kv_heads)], None
    if Le <= cfg.topk:
        all_pos = cfg.l_sink + np.arange(Le, dtype=np.int64)
        return [all_pos.copy() for _ in range(cfg.n_kv_heads)], None
    C = observation_scores(q_obs, k, cfg)
    P = pool_scores(C, cfg.pool_kernel, cfg.pool_mode)
    idx = [cfg.l_sink + select_topk(P[kvh], cfg.topk) for kvh in range(cfg.n_kv_heads)]
    return idx, P


# ----------------------------------------------------------------------------
# Retained-set state: explicit lists (rolling window by deque), NOT a ring.
# ----------------------------------------------------------------------------

@dataclass
class OracleSequence:
    """Everything the method retains for one sequence of one layer.

    The rolling window is a deque that drops its oldest entry (the appendix's
    naive update), so the ring arithmetic of Eq. 3 is checked against it rather
    than reused.  All keys/values ever seen are kept in ``k_hist``/``v_hist`` so
    that retained positions can be looked up and dense attention computed."""

    cfg: OracleConfig
    k_hist: List[np.ndarray] = field(default_factory=list)   # each [Hkv, d_qk]
    v_hist: List[np.ndarray] = field(default_factory=list)   # each [Hkv, d_v]
    sinks: List[int] = field(default_factory=list)
    recents: deque = field(default_factory=deque)
    topk_pos: List[np.ndarray] = field(default_factory=list)  # per KV head
    pooled: Optional[np.ndarray] = None

    @property
    def n_tokens(self) -> int:
        return len(self.k_hist)

    def retained(self, kvh: int) -> List[int]:
        return list(self.sinks) + [int(p) for p in self.topk_pos[kvh]] + list(self.recents)

    def _push(self, k_row: np.ndarray, v_row: np.ndarray) -> int:
        cfg = self.cfg
        t = self.n_tokens
        self.k_hist.append(np.asarray(k_row, dtype=np.float64))
        self.v_hist.append(np.asarray(v_row, dtype=np.float64))
        if t < cfg.l_sink:
            self.sinks.append(t)                 # sink region still filling
        else:
            self.recents.append(t)
            if len(self.recents) > cfg.l_recent:
                self.recents.popleft()           # evict the least recent (Section 3.1, Case 2)
        return t


def _v_rows(k: np.ndarray, v: Optional[np.ndarray], cfg: OracleConfig) -> np.ndarray:
    if cfg.v_aliases_k:
        return np.asarray(k, dtype=np.float64)[..., :cfg.d_v]
    return np.asarray(v, dtype=np.float64)


def compress(q_obs: np.ndarray, k: np.ndarray, v: Optional[np.ndarray],
             cfg: OracleConfig) -> OracleSequence:
    """Prefill compression of one sequence (Section 3.2): keep the first Ls tokens,
    the last Lr tokens, and the SnapKV top-K of what lies between."""
    k = np.asarray(k, dtype=np.float64)
    vv = _v_rows(k, v, cfg)
    L = k.shape[0]
    seq = OracleSequence(cfg)
    for p in range(L):
        seq._push(k[p], vv[p])
    idx, P = snapkv_select(q_obs, k, cfg)
    seq.topk_pos = idx
    seq.pooled = P
    return seq


def attention_over(q: np.ndarray, K_rows: np.ndarray, V_rows: np.ndarray, scale: float) -> np.ndarray:
    """softmax(scale * q K^T) V for one query vector; plain definition."""
    s = scale * (K_rows @ q)
    s = s - s.max()
    e = np.exp(s)
    return (e / e.sum()) @ V_rows


def attend(seq: OracleSequence, q: np.ndarray) -> np.ndarray:
    """Attention of one query token [Hq, d_qk] over the retained set. -> [Hq, d_v]."""
    cfg = seq.cfg
    q = np.asarray(q, dtype=np.float64)
    out = np.zeros((cfg.n_q_heads, cfg.d_v), dtype=np.float64)
    for kvh in range(cfg.n_kv_heads):
        pos = seq.retained(kvh)
        K_rows = np.stack([seq.k_hist[p][kvh] for p in pos])
        V_rows = np.stack([seq.v_hist[p][kvh] for p in pos])
        for h in range(kvh * cfg.group, (kvh + 1) * cfg.group):
            out[h] = attention_over(q[h], K_rows, V_rows, cfg.softmax_scale)
    return out


def decode_step(seq: OracleSequence, q: np.ndarray, k_new: np.ndarray,
                v_new: Optional[np.ndarray]) -> np.ndarray:
    """One decode step (Section 3.3): the new token's K/V enter the rolling window
    (evicting its oldest entry once it is full), then the query attends over the
    retained set, the new token included."""
    cfg = seq.cfg
    k_new = np.asarray(k_new, dtype=np.float64)
    seq._push(k_new, _v_rows(k_new, v_new, cfg))
    return attend(seq, q)


def dense_attention(seq: OracleSequence, q: np.ndarray) -> np.ndarray:
    """Uncompressed attention over every token seen so far (the full-KV baseline)."""
    cfg = seq.cfg
    q = np.asarray(q, dtype=np.float64)
    K_all = np.stack(seq.k_hist)      # [T, Hkv, d]
    V_all = np.stack(seq.v_hist)
    out = np.zeros((cfg.n_q_heads, cfg.d_v), dtype=np.float64)
    for h in range(cfg.n_q_heads):
        kvh = h // cfg.group
        out[h] = attention_over(q[h], K_all[:, kvh], V_all[:, kvh], cfg.softmax_scale)
    return out


# ----------------------------------------------------------------------------
# Expected cache image: where each retained position must sit in the fixed cache.
# ----------------------------------------------------------------------------

def expected_cache(seq: OracleSequence):
    """Cache contents implied by the retained set: K image [Hkv, Sc, d_qk], V image
    [Hkv, Sc, d_v] (None when V aliases K), slot->position map [Hkv, Sc] (-1 = pad).
    Sinks and ring positions sit at slot_of_position(p); the i-th selected position
    (ascending) sits at Lsr + i; every other slot is zero."""
    cfg = seq.cfg
    lay = cache_layout(cfg.l_sink, cfg.l_recent, cfg.topk)
    Sc = lay["slots"]
    Kc = np.zeros((cfg.n_kv_heads, Sc, cfg.d_qk), dtype=np.float64)
    Vc = np.zeros((cfg.n_kv_heads, Sc, cfg.d_v), dtype=np.float64)
    pos_map = -np.ones((cfg.n_kv_heads, Sc), dtype=np.int64)
    for kvh in range(cfg.n_kv_heads):
        for p in list(seq.sinks) + list(seq.recents):
            s = slot_of_position(p, cfg.l_sink, cfg.l_recent)
            assert pos_map[kvh, s] == -1, "two retained positions map to one slot"
            pos_map[kvh, s] = p
        for i, p in enumerate(seq.topk_pos[kvh]):
            pos_map[kvh, lay["topk_off"] + i] = int(p)
        for s in range(Sc):
            p = pos_map[kvh, s]
            if p >= 0:
                Kc[kvh, s] = seq.k_hist[p][kvh]
                Vc[kvh, s] = seq.v_hist[p][kvh]
    return Kc, (None if cfg.v_aliases_k else Vc), pos_map


def expected_cache_position_order(seq: OracleSequence):
    """Cache image under the slice-and-concatenate update that Section 3.2.1 describes as the
    naive alternative to the ring: sinks at [0, Ls), the rolling window in position order
    (its i-th oldest entry at Ls + i), the i-th selected position at Lsr + i, zeros elsewhere.
    Same return values as expected_cache."""
    cfg = seq.cfg
    lay = cache_layout(cfg.l_sink, cfg.l_recent, cfg.topk)
    Sc = lay["slots"]
    Kc = np.zeros((cfg.n_kv_heads, Sc, cfg.d_qk), dtype=np.float64)
    Vc = np.zeros((cfg.n_kv_heads, Sc, cfg.d_v), dtype=np.float64)
    pos_map = -np.ones((cfg.n_kv_heads, Sc), dtype=np.int64)
    for kvh in range(cfg.n_kv_heads):
        for p in seq.sinks:
            pos_map[kvh, p] = p
        for i, p in enumerate(seq.recents):
            pos_map[kvh, cfg.l_sink + i] = p
        for i, p in enumerate(seq.topk_pos[kvh]):
            pos_map[kvh, lay["topk_off"] + i] = int(p)
        for s in range(Sc):
            p = pos_map[kvh, s]
            if p >= 0:
                Kc[kvh, s] = seq.k_hist[p][kvh]
                Vc[kvh, s] = seq.v_hist[p][kvh]
    return Kc, (None if cfg.v_aliases_k else Vc), pos_map


# ----------------------------------------------------------------------------
# Prefill attention that also yields Eq. 4's normalisers (the step Section 3.2.2
# leaves to future optimisation: the scores' denominators are by-products of the
# prompt's own causal attention pass).
# ----------------------------------------------------------------------------

def prefill_attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, cfg: OracleConfig) -> np.ndarray:
    """Causal attention of a whole prompt, plain definition: query position t of head h
    attends over key positions 0..t of KV head h // g.

    q: [L, Hq, d_qk], k: [L, Hkv, d_qk], v: [L, Hkv, d_v]  ->  float64 [L, Hq, d_v].
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    L = q.shape[0]
    out = np.zeros((L, cfg.n_q_heads, v.shape[2]), dtype=np.float64)
    for h in range(cfg.n_q_heads):
        kvh = h // cfg.group
        for t in range(L):
            out[t, h] = attention_over(q[t, h], k[: t + 1, kvh], v[: t + 1, kvh], cfg.softmax_scale)
    return out


def candidate_log2_normalisers(q_obs: np.ndarray, k: np.ndarray, cfg: OracleConfig) -> np.ndarray:
    """mu[h, i] = log2 sum_{j in [Ls, L-Lr)} exp(scale * q_obs[h, i] . k_j): the denominator of
    Eq. 4 for window row i of head h, as a base-2 logarithm, so that the Eq. 4 weight of
    candidate j is 2 ** (log2(e) * scale * q.k_j - mu).  -> float64 [Hq, Lo]; -inf where the
    prompt has no candidate."""
    q_obs = np.asarray(q_obs, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    L = k.shape[0]
    lo, hi = cfg.l_sink, L - cfg.l_recent
    mu = np.full((cfg.n_q_heads, cfg.l_obs), -np.inf, dtype=np.float64)
    if hi <= lo:
        return mu
    for h in range(cfg.n_q_heads):
        kvh = h // cfg.group
        S = cfg.softmax_scale * (q_obs[h] @ k[lo:hi, kvh].T)           # [Lo, Le]
        m = S.max(axis=1)
        mu[h] = (m + np.log(np.exp(S - m[:, None]).sum(axis=1))) / np.log(2.0)
    return mu


# ----------------------------------------------------------------------------
# Per-step block top-K over the evictable middle of the prompt (the alternative the paper's
# related-work section leaves to future work: KV blocks with pre-computed statistics, of
# which the top ones are looked up for every newly decoded token, "in the style of Quest
# and InfLLM").  The paper fixes nothing beyond that sentence, so everything here is a
# reading, stated in full:
#   * the middle of the prompt, positions [Ls, L - Lr), is kept whole and cut into blocks
#     of `block_tokens` consecutive positions (the last block may be shorter);
#   * a block's statistics are the element-wise minimum and maximum of its keys per KV
#     head (the published query-aware page criterion);
#   * a decode query scores block b of KV head kvh by
#         U[kvh, b] = sum_{h in group(kvh)} sum_d max(q[h, d] * kmin[kvh, b, d], q[h, d] * kmax[kvh, b, d]),
#     an upper bound of the group-summed logit q_h . k_j of every key j of the block (the
#     g query heads of a KV head are summed as in Eq. 1's group reading above);
#   * the `n_blocks` highest-scoring blocks are attended, ties to the lower block index,
#     together with the sinks and the rolling window of Eq. 3, which behave as before;
#     tokens that leave the rolling window during decoding are dropped as in SnapStream.
# Parity unpinned by the paper: all of the above.  Pinned by the mathematics: the bound
# property, the one-token-block special case (exact top-k by logit), and equality with
# attention over everything kept when all blocks are selected.
# ----------------------------------------------------------------------------

def block_statistics(k: np.ndarray, cfg: OracleConfig, block_tokens: int):
    """Per-block key minima and maxima over the prompt's middle.  k: [L, Hkv, d_qk].
    returns (kmin, kmax), each [Hkv, n_blocks, d_qk]; n_blocks = ceil((L - Lsr) / block_tokens)."""
    k = np.asarray(k, dtype=np.float64)
    L = k.shape[0]
    Le = max(L - cfg.l_sr, 0)
    nb = -(-Le // block_tokens)
    kmin = np.zeros((cfg.n_kv_heads, nb, cfg.d_qk))
    kmax = np.zeros((cfg.n_kv_heads, nb, cfg.d_qk))
    for b in range(nb):
        lo = cfg.l_sink + b * block_tokens
        hi = min(lo + block_tokens, cfg.l_sink + Le)
        kmin[:, b, :] = k[lo:hi].min(axis=0)
        kmax[:, b, :] = k[lo:hi].max(axis=0)
    return kmin, kmax


def block_upper_bounds(q: np.ndarray, kmin: np.ndarray, kmax: np.ndarray, cfg: OracleConfig) -> np.ndarray:
    """U[kvh, b] for one decode query q: [Hq, d_qk]. -> [Hkv, n_blocks]."""
    q = np.asarray(q, dtype=np.float64)
    nb = kmin.shape[1]
    U = np.zeros((cfg.n_kv_heads, nb))
    for kvh in range(cfg.n_kv_heads):
        for h in range(kvh * cfg.group, (kvh + 1) * cfg.group):
            U[kvh] += np.maximum(q[h][None, :] * kmin[kvh], q[h][None, :] * kmax[kvh]).sum(axis=1)
    return U


def select_blocks(U_row: np.ndarray, n_blocks: int) -> np.ndarray:
    """The n_blocks highest-scoring blocks of one KV head, ties to the lower index, ascending."""
    return select_topk(U_row, n_blocks)


def block_positions(blocks: np.ndarray, prompt_len: int, cfg: OracleConfig, block_tokens: int) -> np.ndarray:
    """Absolute prompt positions covered by the given blocks (ascending)."""
    end = prompt_len - cfg.l_recent
    out = []
    for b in blocks:
        lo = cfg.l_sink + int(b) * block_tokens
        out.extend(range(lo, min(lo + block_tokens, end)))
    return np.asarray(out, dtype=np.int64)


def block_decode_step(seq: OracleSequence, prompt_len: int, kmin: np.ndarray, kmax: np.ndarray, n_blocks: int,
                      block_tokens: int, q: np.ndarray, k_new: np.ndarray, v_new: Optional[np.ndarray]):
    """One decode step with a per-step block lookup: score the blocks with this token's
    query, keep the top n_blocks per KV head in place of the prefill top-K set, then
    append and attend as in `decode_step`.  returns (out [Hq, d_v], blocks per KV head)."""
    cfg = seq.cfg
    U = block_upper_bounds(q, kmin, kmax, cfg)
    chosen = [select_blocks(U[kvh], n_blocks) for kvh in range(cfg.n_kv_heads)]
    seq.topk_pos = [block_positions(chosen[kvh], prompt_len, cfg, block_tokens) for kvh in range(cfg.n_kv_heads)]
    return decode_step(seq, q, k_new, v_new), chosen
