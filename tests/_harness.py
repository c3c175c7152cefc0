"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI and the
oracle on the same seeded inputs and compare them."""
import numpy as np
import torch

from oracle import snapstream_oracle as orc
from paper_2511_03092_b200 import binding as B
from paper_2511_03092_b200 import synth

BF16_ABS, BF16_REL_L2 = 2e-2, 1e-2          # output tolerances, bf16
F32_REL, F32_REL_L2 = 1e-4, 1e-5            # output tolerances, fp32
BOUNDARY_REL = 1e-6                         # allowance on pooled scores at the K-th boundary


def oracle_config(wl):
    return orc.OracleConfig(wl.n_q_heads, wl.n_kv_heads, wl.d_qk, wl.d_v, wl.l_sink, wl.l_recent, wl.topk,
                            wl.l_obs, wl.pool_kernel, wl.scale, wl.pool_mode, wl.v_aliases_k)


def snap_config(wl, max_seqs):
    return B.make_config(n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, d_qk=wl.d_qk, d_v=wl.d_v,
                         dtype=wl.torch_dtype, l_sink=wl.l_sink, l_recent=wl.l_recent, topk=wl.topk,
                         l_obs=wl.l_obs, pool_kernel=wl.pool_kernel, softmax_scale=wl.scale,
                         max_seqs=max_seqs, pool_mode=wl.pool_mode, v_aliases_k=wl.v_aliases_k)


class GpuLayer:
    """One layer's cache plus scratch on the GPU, driven only through the C ABI binding."""

    def __init__(self, wl, max_seqs, device="cuda"):
        self.wl, self.device = wl, device
        self.cfg = snap_config(wl, max_seqs)
        self.layout = B.snap_cache_layout(self.cfg)
        self.cache = B.alloc_cache(self.cfg, self.layout, device)
        self.dec_ws = None

    def compress(self, prompts, slots, want_idx=True):
        wl = self.wl
        lens = [p["k"].shape[0] for p in prompts]
        cu = [0]
        for L in lens:
            cu.append(cu[-1] + L)
        q_obs = torch.stack([p["q_obs"] for p in prompts]).to(self.device)
        k = torch.cat([p["k"] for p in prompts]).to(self.device)
        v = None if wl.v_aliases_k else torch.cat([p["v"] for p in prompts]).to(self.device)
        ws = torch.empty(B.snap_compress_workspace_bytes(self.cfg, cu), dtype=torch.uint8, device=self.device)
        idx = None
        if want_idx:
            idx = torch.full((len(prompts), wl.n_kv_heads, max(wl.topk, 1)), -7, dtype=torch.int32,
                             device=self.device)
        c = self.cache
        B.snap_compress(self.cfg, self.layout, q_obs, k, v, cu, slots, c.k_cache, c.v_cache, c.seq_len,
                        c.valid_topk, idx, ws, c.status)
        torch.cuda.synchronize()
        return None if idx is None else idx.cpu().numpy()[:, :, :wl.topk]

    def decode(self, q, k_new, v_new, slots_dev):
        n = q.shape[0]
        need = B.snap_decode_workspace_bytes(self.cfg, n)
        if self.dec_ws is None or self.dec_ws.numel() < need:
            self.dec_ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        out = torch.empty(n, self.wl.n_q_heads, self.wl.d_v, dtype=self.wl.torch_dtype, device=self.device)
        c = self.cache
        B.snap_decode_attn(self.cfg, self.layout, q, k_new, v_new, slots_dev, n, c.k_cache, c.v_cache,
                           c.seq_len, c.valid_topk, out, self.dec_ws, c.status)
        return out

    def status(self):
        torch.cuda.synchronize()
        return int(self.cache.status.item())


def check_selection(idx_gpu, seq, wl):
    """Selected positions of one sequence [Hkv, K] against the oracle.  Bit-exact, except that a
    candidate whose oracle pooled score is within BOUNDARY_REL (relative) of the K-th largest may
    be swapped for another such candidate.  Returns the number of such swaps."""
    swaps = 0
    for h in range(wl.n_kv_heads):
        want = np.asarray(seq.topk_pos[h])
        got = idx_gpu[h]
        nv = len(want)
        assert (got[nv:] == -1).all(), "padding entries must be -1"
        got = got[:nv]
        assert (np.diff(got) > 0).all(), "selected positions must be ascending and distinct"
        if np.array_equal(got, want):
            continue
        assert seq.pooled is not None, "selection differs although no scoring was needed"
        P = seq.pooled[h]
        tau = np.sort(P)[-wl.topk]
        sel = np.zeros(P.shape[0], dtype=bool)
        sel[got - wl.l_sink] = True
        assert sel.sum() == wl.topk
        must = P > tau * (1 + BOUNDARY_REL)
        never = P < tau * (1 - BOUNDARY_REL)
        assert sel[must].all(), f"head {h}: {(must & ~sel).sum()} clear winners not selected"
        assert not sel[never].any(), f"head {h}: {(never & sel).sum()} clear losers selected"
        swaps += int((sel != np.isin(np.arange(P.shape[0]) + wl.l_sink, want)).sum() // 2)
    return swaps


def check_output(out_gpu, out_ref, wl, what=""):
    got = out_gpu.detach().to("cpu", torch.float64).numpy()
    err = np.abs(got - out_ref)
    rel_l2 = np.linalg.norm(got - out_ref) / max(np.linalg.norm(out_ref), 1e-300)
    if wl.dtype == "bf16":
        assert err.max() <= BF16_ABS, f"{what} max abs err {err.max():.3e}"
        assert rel_l2 <= BF16_REL_L2, f"{what} rel L2 err {rel_l2:.3e}"
    else:
        tol = F32_REL * np.abs(out_ref) + 1e-6 * np.abs(out_ref).max()
        assert (err <= tol).all(), f"{what} max rel err {(err / (np.abs(out_ref) + 1e-30)).max():.3e}"
        assert rel_l2 <= F32_REL_L2, f"{what} rel L2 err {rel_l2:.3e}"


def check_cache_image(layer, seq, slot, wl):
    """Cache bytes of one slot against the oracle's expected image (exact: rows are copies)."""
    Kc, Vc, _ = orc.expected_cache(seq)
    got_k = layer.cache.k_cache[slot].to("cpu", torch.float64).numpy()
    np.testing.assert_array_equal(got_k, Kc)
    if Vc is not None:
        got_v = layer.cache.v_cache[slot].to("cpu", torch.float64).numpy()
        np.testing.assert_array_equal(got_v, Vc)


def oracle_compress(wl, prompt):
    return orc.compress(synth.to_f64(prompt["q_obs"]), synth.to_f64(prompt["k"]), synth.to_f64(prompt["v"]),
                        oracle_config(wl))
