"""Seeded random small configurations through the C ABI against the oracle: head size, group size,
sink / window / budget sizes, pooling width, ragged prompt lengths, one or several tokens per step,
the latent layout with 64, 128 and 256 heads, and the prompt attention that feeds the compression
its normalisers.  Every case checks the selected indices, every
decode output, the sequence lengths and the final cache image."""
import numpy as np
import pytest
import torch

from oracle import snapstream_oracle as orc
from paper_2511_03092_b200 import binding as B
from paper_2511_03092_b200 import synth
from tests import _harness as H

pytestmark = pytest.mark.gpu


def _compress_and_check(wl, lengths, seed):
    n = len(lengths)
    layer = H.GpuLayer(wl, n)
    prompts = [synth.make_prompt(wl, L, seed + i) for i, L in enumerate(lengths)]
    idx = layer.compress(prompts, list(range(n)))
    seqs = [H.oracle_compress(wl, p) for p in prompts]
    for i in range(n):
        H.check_selection(idx[i], seqs[i], wl)
        seqs[i].topk_pos = [idx[i][h][idx[i][h] >= 0].astype(np.int64) for h in range(wl.n_kv_heads)]
    return layer, seqs


def _finish(layer, seqs, wl):
    assert layer.status() == 0
    for i, seq in enumerate(seqs):
        assert int(layer.cache.seq_len[i]) == seq.n_tokens
        H.check_cache_image(layer, seq, i, wl)


@pytest.mark.parametrize("seed", [3, 4])
def test_random_grouped_query_configurations(seed):
    rng = np.random.default_rng(seed)
    for case in range(40):
        d = int(rng.choice([64, 128, 256]))
        hkv = int(rng.choice([1, 2, 4]))
        g = int(rng.integers(1, 9))
        Ls, Lr, K = int(rng.integers(0, 6)), int(rng.integers(1, 40)), int(rng.choice([0, 5, 16, 33, 64]))
        Lo, w = int(rng.integers(1, min(Lr, 16) + 1)), int(rng.choice([1, 3, 7]))
        wl = synth.Workload("rnd", g * hkv, hkv, d, d, "bf16", Ls, Lr, K, Lo, w, batch=1, prompt_len=(100, 100),
                            decode_steps=4, salience="zipf")
        n = int(rng.integers(1, 4))
        lengths = [int(rng.integers(1, 200)) for _ in range(n)]
        q_len = int(rng.integers(1, max(1, min(8 // g, Lr)) + 1))
        steps = int(rng.integers(1, 2 * Lr // q_len + 4))
        what = f"case {case}: d{d} hkv{hkv} g{g} Ls{Ls} Lr{Lr} K{K} Lo{Lo} w{w} L{lengths} q_len{q_len}"
        layer, seqs = _compress_and_check(wl, lengths, 1000 * case + seed)
        c = layer.cache
        slots = torch.arange(n, dtype=torch.int32, device="cuda")
        ws = torch.empty(B.snap_decode_multi_workspace_bytes(layer.cfg, n, q_len), dtype=torch.uint8, device="cuda")
        for st in range(steps):
            ds = [synth.make_decode_inputs(wl, n, case, st * q_len + u) for u in range(q_len)]
            if q_len == 1:
                out = layer.decode(ds[0]["q"].cuda(), ds[0]["k_new"].cuda(), ds[0]["v_new"].cuda(), slots).unsqueeze(1)
            else:
                q = torch.stack([x["q"] for x in ds], 1).contiguous().cuda()
                kn = torch.stack([x["k_new"] for x in ds], 1).contiguous().cuda()
                vn = torch.stack([x["v_new"] for x in ds], 1).contiguous().cuda()
                out = torch.empty(n, q_len, wl.n_q_heads, d, dtype=torch.bfloat16, device="cuda")
                B.snap_decode_attn_multi(layer.cfg, layer.layout, q, kn, vn, slots, n, q_len, c.k_cache, c.v_cache,
                                         c.seq_len, c.valid_topk, out, ws, c.status)
            for i in range(n):
                for u in range(q_len):
                    ref = orc.decode_step(seqs[i], synth.to_f64(ds[u]["q"][i]), synth.to_f64(ds[u]["k_new"][i]),
                                          synth.to_f64(ds[u]["v_new"][i]))
                    H.check_output(out[i, u], ref, wl, f"{what} step {st} seq {i} token {u}")
        _finish(layer, seqs, wl)


def test_random_latent_configurations():
    rng = np.random.default_rng(5)
    for case in range(16):
        hq = int(rng.choice([64, 128, 256]))
        Ls, Lr, K = int(rng.integers(0, 6)), int(rng.integers(1, 300)), int(rng.choice([0, 7, 64, 200]))
        Lo, w = int(rng.integers(1, min(Lr, 8) + 1)), int(rng.choice([1, 5]))
        wl = synth.Workload("rnd_latent", hq, 1, 576, 512, "bf16", Ls, Lr, K, Lo, w, batch=1, prompt_len=(100, 100),
                            decode_steps=4, salience="planted", n_planted=4, v_aliases_k=True,
                            softmax_scale=2.0 ** -0.5)
        n = int(rng.integers(1, 3))
        lengths = [int(rng.integers(1, 700)) for _ in range(n)]
        what = f"case {case}: hq{hq} Ls{Ls} Lr{Lr} K{K} Lo{Lo} w{w} L{lengths}"
        layer, seqs = _compress_and_check(wl, lengths, 1000 * case)
        slots = torch.arange(n, dtype=torch.int32, device="cuda")
        for st in range(int(rng.integers(1, 12))):
            d = synth.make_decode_inputs(wl, n, case, st)
            out = layer.decode(d["q"].cuda(), d["k_new"].cuda(), None, slots)
            for i in range(n):
                ref = orc.decode_step(seqs[i], synth.to_f64(d["q"][i]), synth.to_f64(d["k_new"][i]), None)
                H.check_output(out[i], ref, wl, f"{what} step {st} seq {i}")
        _finish(layer, seqs, wl)


def test_random_compress_configurations():
    """Prompts of a few thousand tokens through each score kernel family (128-wide tcgen05, wide tcgen05 at
    other head and group sizes, latent layout), both pooling modes, several pooling widths and budgets."""
    rng = np.random.default_rng(1)
    for case in range(18):
        kind = case % 3
        if kind == 0:
            hkv, g, d = int(rng.choice([1, 2])), int(rng.choice([2, 4])), 128
            Lo = int(rng.choice([32, 64])) if g == 4 else int(rng.choice([64, 128]))
        elif kind == 1:
            hkv, g = int(rng.choice([1, 2])), int(rng.choice([1, 3, 5, 8]))
            Lo, d = int(rng.choice([8, 16, 48])), int(rng.choice([64, 128, 256]))
        else:
            hkv, g, Lo, d = 1, int(rng.choice([64, 128])), int(rng.choice([4, 16])), 576
        Ls, Lr = int(rng.integers(0, 8)), int(rng.integers(max(Lo, 8), 600))
        K, w = int(rng.choice([0, 64, 500, 2048])), int(rng.choice([1, 3, 7, 13]))
        mode = str(rng.choice(["avg", "max"]))
        L = int(rng.integers(Ls + Lr + 1, 20000))
        if kind == 2:
            wl = synth.Workload("rnd", g, 1, 576, 512, "bf16", Ls, Lr, K, Lo, w, batch=1, prompt_len=(L, L),
                                decode_steps=1, salience="planted", n_planted=16, v_aliases_k=True,
                                softmax_scale=2.0 ** -0.5, pool_mode=mode)
        else:
            wl = synth.Workload("rnd", g * hkv, hkv, d, d, "bf16", Ls, Lr, K, Lo, w, batch=1, prompt_len=(L, L),
                                decode_steps=1, salience=str(rng.choice(["zipf", "planted"])), n_planted=16,
                                pool_mode=mode)
        layer, seqs = _compress_and_check(wl, [L], 77 * case + 1)
        assert layer.status() == 0, f"case {case}"
        H.check_cache_image(layer, seqs[0], 0, wl)


@pytest.mark.parametrize("seed", [11, 12])
def test_random_prefill_configurations(seed):
    """Prompt attention, its Eq. 4 normalisers, and the compression that takes them: random head size (the
    tensor-core kernel for 128, the portable one otherwise), group size, hyper-parameters and ragged batches."""
    rng = np.random.default_rng(seed)
    for case in range(14):
        d = int(rng.choice([128, 128, 128, 64, 256]))
        hkv = int(rng.choice([1, 2, 4]))
        g = int(rng.integers(1, 9))
        Ls, Lr, K = int(rng.integers(0, 6)), int(rng.integers(1, 70)), int(rng.choice([5, 16, 33, 64]))
        Lo, w = int(rng.integers(1, min(Lr, 40) + 1)), int(rng.choice([1, 3, 7]))
        wl = synth.Workload("rnd", g * hkv, hkv, d, d, "bf16", Ls, Lr, K, Lo, w, batch=1, prompt_len=(100, 100),
                            decode_steps=1, salience="zipf")
        n = int(rng.integers(1, 5))
        lengths = [int(rng.integers(1, 420)) for _ in range(n)]
        what = f"case {case}: d{d} hkv{hkv} g{g} Ls{Ls} Lr{Lr} K{K} Lo{Lo} w{w} L{lengths}"
        prompts = [synth.make_prompt(wl, L, 1000 * case + seed + i) for i, L in enumerate(lengths)]
        qs = [synth.make_prompt_queries(wl, p, 1000 * case + seed + i) for i, p in enumerate(prompts)]
        cu = [0]
        for L in lengths:
            cu.append(cu[-1] + L)
        layer = H.GpuLayer(wl, n)
        q = torch.cat(qs).cuda()
        k = torch.cat([p["k"] for p in prompts]).cuda()
        v = torch.cat([p["v"] for p in prompts]).cuda()
        out = torch.full((cu[-1], wl.n_q_heads, d), float("nan"), dtype=torch.bfloat16, device="cuda")
        mu = torch.full((n, wl.n_q_heads, Lo), float("nan"), dtype=torch.float32, device="cuda")
        c = layer.cache
        B.snap_prefill_attn(layer.cfg, q, k, v, cu, out, mu, c.status)
        ocfg = H.oracle_config(wl)
        mu_host = mu.cpu().numpy().astype(np.float64)
        for i, (p, qq, L) in enumerate(zip(prompts, qs, lengths)):
            ref = orc.prefill_attention(synth.to_f64(qq), synth.to_f64(p["k"]), synth.to_f64(p["v"]), ocfg)
            H.check_output(out[cu[i]:cu[i + 1]], ref, wl, f"{what} prompt {i}")
            m = min(L, Lo)
            want = orc.candidate_log2_normalisers(synth.to_f64(p["q_obs"]), synth.to_f64(p["k"]), ocfg)[:, Lo - m:]
            got = mu_host[i][:, Lo - m:]
            if np.isneginf(want).all():
                assert np.isneginf(got).all(), what
            else:
                np.testing.assert_allclose(got, want, rtol=0, atol=1e-3, err_msg=what)
        ws = torch.empty(B.snap_compress_workspace_bytes(layer.cfg, cu), dtype=torch.uint8, device="cuda")
        idx = torch.full((n, hkv, K), -7, dtype=torch.int32, device="cuda")
        B.snap_compress_with_row_stats(layer.cfg, layer.layout, torch.stack([p["q_obs"] for p in prompts]).cuda(), mu, k, v,
                                       cu, list(range(n)), c.k_cache, c.v_cache, c.seq_len, c.valid_topk, idx, ws, c.status)
        assert layer.status() == 0, what
        idx = idx.cpu().numpy()
        for i, p in enumerate(prompts):
            seq = H.oracle_compress(wl, p)
            H.check_selection(idx[i], seq, wl)
            seq.topk_pos = [idx[i][h][idx[i][h] >= 0].astype(np.int64) for h in range(hkv)]
            H.check_cache_image(layer, seq, i, wl)
