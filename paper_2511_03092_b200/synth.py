"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random tensors; it contains none of the method's arithmetic
(no scoring, pooling, selection, cache indexing or attention).  The CUDA path and the
CPU oracle both consume what it produces: the oracle reads host copies of exactly
the buffers handed to the GPU.

Recipe (one family for every configuration).  Per KV head draw a unit vector ``u``.
Observation-window queries are ``q = n_q + u / scale`` and prompt keys are
``k_t = n_t + s_t * u`` with ``n`` i.i.d. Gaussian noise, so a token with salience
``s_t`` gains about ``s_t`` logits on every observation row.  Values are noise only.
Salience patterns: ``planted`` (a fixed number of candidate positions get s_t = 3),
``zipf`` (per head a random ranking r_t gets s_t = 8 * r_t**-1.1), ``none``.
For the latent-attention shape the key row is 512 latent dims with variance 1/512
followed by 64 rotary dims with variance 1/64, queries have unit variance, and the
value is the latent part of the key row (no separate V tensor).

These stand in for Llama-3.1-8B and DeepSeek-R1 attention layers at up to 128k
context (the models the paper evaluates); no model weights, datasets or benchmark
items are used.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, List, Optional, Tuple

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    n_q_heads: int
    n_kv_heads: int
    d_qk: int
    d_v: int
    dtype: str                      # "f32" | "bf16"
    l_sink: int
    l_recent: int
    topk: int
    l_obs: int
    pool_kernel: int
    batch: int
    prompt_len: Tuple[int, int]     # inclusive range; equal ends = fixed length
    decode_steps: int
    salience: str                   # "planted" | "zipf" | "none"
    n_planted: int = 0
    pool_mode: str = "avg"
    v_aliases_k: bool = False
    n_layers: int = 1
    replace_prob: float = 0.0       # continuous batching: per-slot, per-step finish probability
    softmax_scale: Optional[float] = None

    @property
    def scale(self) -> float:
        s = self.softmax_scale if self.softmax_scale is not None else 1.0 / math.sqrt(self.d_qk)
        return float(np.float32(s))

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def slots(self) -> int:
        return self.l_sink + self.l_recent + self.topk

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five benchmark configurations (attention-layer shapes of Llama-3.1-8B and of
# DeepSeek's latent attention, prompts up to 128k tokens).
CONFIGS: Dict[int, Workload] = {
    0: Workload("cfg0_gqa_f32_4k", 8, 2, 128, 128, "f32", 4, 256, 512, 32, 7,
                batch=1, prompt_len=(4096, 4096), decode_steps=16,
                salience="planted", n_planted=64),
    1: Workload("cfg1_llama_bf16_32k", 32, 8, 128, 128, "bf16", 4, 1024, 4096, 64, 7,
                batch=1, prompt_len=(32768, 32768), decode_steps=256, salience="zipf"),
    2: Workload("cfg2_llama_bf16_cb32_8k-128k", 32, 8, 128, 128, "bf16", 4, 1024, 4096, 64, 7,
                batch=32, prompt_len=(8192, 131072), decode_steps=512, salience="zipf",
                replace_prob=0.02),
    3: Workload("cfg3_mla_bf16_128k", 128, 1, 576, 512, "bf16", 4, 2048, 8192, 32, 7,
                batch=8, prompt_len=(131072, 131072), decode_steps=256,
                salience="planted", n_planted=64, v_aliases_k=True,
                softmax_scale=1.0 / math.sqrt(2.0)),
    4: Workload("cfg4_llama_bf16_32layers_128k", 32, 8, 128, 128, "bf16", 4, 1024, 4096, 64, 7,
                batch=16, prompt_len=(131072, 131072), decode_steps=1024, salience="none",
                n_layers=32),
}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _noise_std(wl: Workload, device) -> torch.Tensor:
    """Per-dimension standard deviation of key noise."""
    if wl.v_aliases_k:
        n_rope = wl.d_qk - wl.d_v
        std = torch.cat([torch.full((wl.d_v,), wl.d_v ** -0.5),
                         torch.full((n_rope,), n_rope ** -0.5)])
        return std.to(device)
    return torch.ones(wl.d_qk, device=device)


def make_prompt(wl: Workload, L: int, seed: int, device="cpu") -> dict:
    """One prompt of length L: observation queries, keys, values (None if V aliases K).

    returns dict(q_obs [Hq, Lo, d_qk], k [L, Hkv, d_qk], v [L, Hkv, d_v] | None,
                 planted list of positions per KV head | None)."""
    dev = torch.device(device)
    g = _gen(seed, dev)
    Hq, Hkv, d = wl.n_q_heads, wl.n_kv_heads, wl.d_qk
    grp = Hq // Hkv
    u = torch.randn(Hkv, d, generator=g, device=dev)
    u = u / u.norm(dim=1, keepdim=True)
    q = torch.randn(Hq, wl.l_obs, d, generator=g, device=dev)
    q = q + (u / wl.scale).repeat_interleave(grp, dim=0)[:, None, :]
    k = torch.randn(L, Hkv, d, generator=g, device=dev)
    k.mul_(_noise_std(wl, dev))
    lo, hi = wl.l_sink, L - wl.l_recent
    planted = None
    rng = np.random.default_rng(seed + 7919)
    if hi > lo and wl.salience == "planted":
        planted = []
        for h in range(Hkv):
            pos = np.sort(rng.choice(np.arange(lo, hi), size=min(wl.n_planted, hi - lo), replace=False))
            planted.append(pos)
            k[torch.as_tensor(pos, device=dev), h] += 3.0 * u[h]
    elif hi > lo and wl.salience == "zipf":
        for h in range(Hkv):
            rank = torch.as_tensor(rng.permutation(L) + 1, device=dev, dtype=torch.float32)
            k[:, h] += (8.0 * rank.pow(-1.1))[:, None] * u[h]
    v = None
    if not wl.v_aliases_k:
        v = torch.randn(L, Hkv, wl.d_v, generator=g, device=dev).to(wl.torch_dtype)
    return {"q_obs": q.to(wl.torch_dtype).contiguous(), "k": k.to(wl.torch_dtype).contiguous(),
            "v": v, "planted": planted}


def make_decode_inputs(wl: Workload, n: int, seed: int, step: int, device="cpu") -> dict:
    """New-token tensors for one decode step of n sequences: q [n, Hq, d_qk],
    k_new [n, Hkv, d_qk], v_new [n, Hkv, d_v] | None."""
    dev = torch.device(device)
    g = _gen(seed * 1000003 + step + 1, dev)
    q = torch.randn(n, wl.n_q_heads, wl.d_qk, generator=g, device=dev)
    k = torch.randn(n, wl.n_kv_heads, wl.d_qk, generator=g, device=dev) * _noise_std(wl, dev)
    v = None
    if not wl.v_aliases_k:
        v = torch.randn(n, wl.n_kv_heads, wl.d_v, generator=g, device=dev).to(wl.torch_dtype)
    return {"q": q.to(wl.torch_dtype).contiguous(), "k_new": k.to(wl.torch_dtype).contiguous(),
            "v_new": v}


def make_prompt_queries(wl: Workload, prompt: dict, seed: int, device="cpu") -> torch.Tensor:
    """Queries of every prompt position, [L, Hq, d_qk], for the prefill attention pass: random
    rows whose last Lo positions are the prompt's observation queries."""
    dev = torch.device(device)
    L = prompt["k"].shape[0]
    g = _gen(seed * 7 + 13, dev)
    q = torch.randn(L, wl.n_q_heads, wl.d_qk, generator=g, device=dev).to(wl.torch_dtype)
    n = min(L, wl.l_obs)
    if n > 0:
        q[L - n:] = prompt["q_obs"][:, wl.l_obs - n:].transpose(0, 1).to(dev)
    return q.contiguous()


def draw_prompt_lengths(wl: Workload, n: int, seed: int) -> List[int]:
    lo, hi = wl.prompt_len
    rng = np.random.default_rng(seed + 104729)
    return [int(x) for x in rng.integers(lo, hi + 1, size=n)]


def continuous_batching_schedule(wl: Workload, steps: int, seed: int) -> List[List[int]]:
    """For each decode step, the cache slots whose sequence finishes after that step
    and is replaced by a fresh prompt before the next one (seeded Bernoulli per slot)."""
    rng = np.random.default_rng(seed + 15485863)
    out = []
    for _ in range(steps):
        fin = np.nonzero(rng.random(wl.batch) < wl.replace_prob)[0]
        out.append([int(s) for s in fin])
    return out


def to_f64(t: Optional[torch.Tensor]) -> Optional[np.ndarray]:
    """Exact float64 host copy of a tensor (bf16/fp32 values are representable)."""
    if t is None:
        return None
    return t.detach().to("cpu", torch.float64).numpy()
