"""GPU parity of the prefill attention kernel and of the compression that consumes the Eq. 4
normalisers it emits, through the C ABI, against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import snapstream_oracle as orc
from paper_2511_03092_b200 import binding as B
from paper_2511_03092_b200 import synth
from tests import _harness as H

pytestmark = pytest.mark.gpu

MU_ATOL = 1e-3      # log2 units: fp32 accumulation of bf16 products and the hardware exp2 give ~1e-5

# g * Lo = 64 rows per KV head (wide score kernel) and 128 (128-row score kernel)
WL64 = synth.Workload("prefill_g4", 8, 2, 128, 128, "bf16", 4, 48, 96, 16, 7, batch=1,
                      prompt_len=(700, 700), decode_steps=1, salience="zipf")
WL128 = WL64.scaled(name="prefill_g8", n_q_heads=16, n_kv_heads=2)
WL_MHA = WL64.scaled(name="prefill_g1", n_q_heads=4, n_kv_heads=4)       # odd group: one head per CTA
WL_G3 = WL64.scaled(name="prefill_g3", n_q_heads=6, n_kv_heads=2)
# an observation window longer than a 128-row tile: its rows sit in two or three CTAs
WL_LONGWIN = WL64.scaled(name="prefill_lo160", n_q_heads=4, n_kv_heads=2, l_sink=3, l_recent=200, topk=64, l_obs=160)


def _prefill(wl, lengths, seed, want_mu=True):
    n = len(lengths)
    prompts = [synth.make_prompt(wl, L, seed + i) for i, L in enumerate(lengths)]
    qs = [synth.make_prompt_queries(wl, p, seed + i) for i, p in enumerate(prompts)]
    cu = [0]
    for L in lengths:
        cu.append(cu[-1] + L)
    layer = H.GpuLayer(wl, max_seqs=n + 1)
    q = torch.cat(qs).cuda()
    k = torch.cat([p["k"] for p in prompts]).cuda()
    v = torch.cat([p["v"] for p in prompts]).cuda()
    out = torch.full((cu[-1], wl.n_q_heads, wl.d_v), float("nan"), dtype=torch.bfloat16, device="cuda")
    mu = torch.full((n, wl.n_q_heads, wl.l_obs), float("nan"), dtype=torch.float32, device="cuda") if want_mu else None
    B.snap_prefill_attn(layer.cfg, q, k, v, cu, out, mu, layer.cache.status)
    assert layer.status() == 0
    return layer, prompts, qs, cu, (q, k, v), out, mu


def _check_prefill(wl, lengths, seed):
    layer, prompts, qs, cu, _, out, mu = _prefill(wl, lengths, seed)
    ocfg = H.oracle_config(wl)
    mu_host = mu.cpu().numpy().astype(np.float64)
    for i, (p, q, L) in enumerate(zip(prompts, qs, lengths)):
        if L == 0:
            continue
        ref = orc.prefill_attention(synth.to_f64(q), synth.to_f64(p["k"]), synth.to_f64(p["v"]), ocfg)
        H.check_output(out[cu[i]:cu[i + 1]], ref, wl, f"prompt {i} (L={L})")
        n = min(L, wl.l_obs)
        want = orc.candidate_log2_normalisers(synth.to_f64(p["q_obs"]), synth.to_f64(p["k"]), ocfg)[:, wl.l_obs - n:]
        got = mu_host[i][:, wl.l_obs - n:]
        if np.isneginf(want).all():
            assert np.isneginf(got).all(), f"prompt {i}: no candidate, normalisers must be -inf"
        else:
            np.testing.assert_allclose(got, want, rtol=0, atol=MU_ATOL, err_msg=f"prompt {i} (L={L})")
        assert np.isnan(mu_host[i][:, :wl.l_obs - n]).all(), "entries of positions before the prompt are left alone"
    return layer, prompts, cu, mu


@pytest.mark.parametrize("wl", [WL64, WL128, WL_MHA, WL_G3, WL_LONGWIN], ids=lambda w: w.name)
def test_prefill_attention_and_normalisers_match_oracle(wl):
    # one row, shorter than the window, around one tile, several tiles with ragged tails, the
    # window straddling a tile boundary (L = 520: rows 504..519), neighbours in one ragged batch
    _check_prefill(wl, [1, 5, 127, 128, 129, 300, 520, 700], seed=310)


def test_single_head_kernel_stays_selectable_for_even_groups(snap_option):
    snap_option(B.SNAP_OPT_PREFILL_SINGLE_HEADS, 1)
    _check_prefill(WL64, [129, 700], seed=315)


def test_prefill_handles_empty_prompts_and_no_normaliser_buffer():
    wl = WL64
    layer, prompts, qs, cu, _, out, _ = _prefill(wl, [0, 200, 0], seed=320, want_mu=False)
    ref = orc.prefill_attention(synth.to_f64(qs[1]), synth.to_f64(prompts[1]["k"]), synth.to_f64(prompts[1]["v"]),
                                H.oracle_config(wl))
    H.check_output(out, ref, wl)


def test_prefill_isolates_prompts_from_nan_neighbours():
    """The tail tile of a prompt reaches into the next prompt's rows; they must not leak."""
    wl = WL64
    lengths = [150, 130]
    layer, prompts, qs, cu, (q, k, v), out, mu = _prefill(wl, lengths, seed=330)
    k2, v2, q2 = k.clone(), v.clone(), q.clone()
    k2[cu[1]:] = float("nan")
    v2[cu[1]:] = float("nan")
    q2[cu[1]:] = float("nan")
    out2 = torch.empty_like(out)
    B.snap_prefill_attn(layer.cfg, q2, k2, v2, cu, out2, None, layer.cache.status)
    assert layer.status() == 0
    assert torch.equal(out2[:cu[1]], out[:cu[1]])


@pytest.mark.parametrize("wl", [WL64, WL128, WL_LONGWIN], ids=lambda w: w.name)
def test_compress_with_prefill_normalisers_matches_oracle(wl):
    lengths = [700, 100, 149, 1300]          # scored, unscored (fits the budget), just scored, many tiles
    layer, prompts, cu, mu = _check_prefill(wl, lengths, seed=340)
    n = len(lengths)
    slots = [2, 0, 4, 1]
    layer2 = H.GpuLayer(wl, max_seqs=n + 1)
    q_obs = torch.stack([p["q_obs"] for p in prompts]).cuda()
    k = torch.cat([p["k"] for p in prompts]).cuda()
    v = torch.cat([p["v"] for p in prompts]).cuda()
    ws = torch.empty(B.snap_compress_workspace_bytes(layer2.cfg, cu), dtype=torch.uint8, device="cuda")
    idx = torch.full((n, wl.n_kv_heads, wl.topk), -7, dtype=torch.int32, device="cuda")
    c = layer2.cache
    launches = B.snap_kernel_launch_count()
    B.snap_compress_with_row_stats(layer2.cfg, layer2.layout, q_obs, mu, k, v, cu, slots, c.k_cache, c.v_cache,
                                   c.seq_len, c.valid_topk, idx, ws, c.status)
    with_stats = B.snap_kernel_launch_count() - launches
    assert layer2.status() == 0
    idx = idx.cpu().numpy()
    for i, p in enumerate(prompts):
        seq = H.oracle_compress(wl, p)
        H.check_selection(idx[i], seq, wl)
        seq.topk_pos = [idx[i][h][idx[i][h] >= 0].astype(np.int64) for h in range(wl.n_kv_heads)]
        H.check_cache_image(layer2, seq, slots[i], wl)
    # one pass over the keys instead of two: fewer launches than the plain call
    launches = B.snap_kernel_launch_count()
    B.snap_compress(layer2.cfg, layer2.layout, q_obs, k, v, cu, slots, c.k_cache, c.v_cache, c.seq_len,
                    c.valid_topk, None, ws, c.status)
    assert with_stats < B.snap_kernel_launch_count() - launches


def test_more_prompts_than_one_launch_takes():
    """Prompts are launched in groups of 64: the normalisers of a later group land in its own rows."""
    wl = WL64
    lengths = [int(x) for x in np.random.default_rng(350).integers(1, 260, size=70)]
    lengths[66] = 400                                  # a scored prompt in the second group
    _check_prefill(wl, lengths, seed=351)


def test_prefill_reads_strided_keys_and_values():
    """K and V as slices of one fused [T, 2 * Hkv, d] buffer (token and head strides differ from dense)."""
    wl = WL64
    lengths = [300, 131]
    layer, prompts, qs, cu, (q, k, v), out, mu = _prefill(wl, lengths, seed=360)
    fused = torch.full((cu[-1], 2 * wl.n_kv_heads + 1, wl.d_qk), float("nan"), dtype=torch.bfloat16, device="cuda")
    fused[:, 0:wl.n_kv_heads] = k
    fused[:, wl.n_kv_heads + 1:] = v
    kv, vv = fused[:, 0:wl.n_kv_heads], fused[:, wl.n_kv_heads + 1:]
    assert not kv.is_contiguous() and kv.stride(0) == (2 * wl.n_kv_heads + 1) * wl.d_qk
    out2 = torch.empty_like(out)
    mu2 = torch.full_like(mu, float("nan"))
    B.snap_prefill_attn(layer.cfg, q, kv, vv, cu, out2, mu2, layer.cache.status)
    assert layer.status() == 0
    assert torch.equal(out2, out)
    assert torch.equal(mu2, mu)


WL_F32 = WL64.scaled(name="prefill_f32", dtype="f32", salience="planted", n_planted=12)
WL_D64 = WL64.scaled(name="prefill_d64", d_qk=64, d_v=64)
WL_LATENT = synth.Workload("prefill_latent", 16, 1, 96, 64, "bf16", 3, 40, 64, 8, 5, batch=1, prompt_len=(500, 500),
                           decode_steps=1, salience="planted", n_planted=8, v_aliases_k=True,
                           softmax_scale=2.0 ** -0.5)


def _prefill_any(wl, lengths, seed):
    """Like _prefill, for layouts without a separate V as well."""
    n = len(lengths)
    prompts = [synth.make_prompt(wl, L, seed + i) for i, L in enumerate(lengths)]
    qs = [synth.make_prompt_queries(wl, p, seed + i) for i, p in enumerate(prompts)]
    cu = [0]
    for L in lengths:
        cu.append(cu[-1] + L)
    layer = H.GpuLayer(wl, max_seqs=n + 1)
    q = torch.cat(qs).cuda()
    k = torch.cat([p["k"] for p in prompts]).cuda()
    v = None if wl.v_aliases_k else torch.cat([p["v"] for p in prompts]).cuda()
    out = torch.full((cu[-1], wl.n_q_heads, wl.d_v), float("nan"), dtype=wl.torch_dtype, device="cuda")
    mu = torch.full((n, wl.n_q_heads, wl.l_obs), float("nan"), dtype=torch.float32, device="cuda")
    B.snap_prefill_attn(layer.cfg, q, k, v, cu, out, mu, layer.cache.status)
    assert layer.status() == 0
    return layer, prompts, qs, cu, (k, v), out, mu


@pytest.mark.parametrize("wl", [WL_F32, WL_D64, WL_LATENT], ids=lambda w: w.name)
def test_portable_prefill_kernel_and_every_score_path_take_the_normalisers(wl):
    """fp32, 64-wide heads and the latent layout: the portable prefill kernel, then compression with its
    normalisers through the SIMT, mma.sync-free and wide tcgen05 score paths these shapes select."""
    lengths = [1, 5, 33, 150, 420]
    layer, prompts, qs, cu, (k, v), out, mu = _prefill_any(wl, lengths, seed=370)
    ocfg = H.oracle_config(wl)
    mu_host = mu.cpu().numpy().astype(np.float64)
    for i, (p, q, L) in enumerate(zip(prompts, qs, lengths)):
        kk = synth.to_f64(p["k"])
        vv = kk[:, :, :wl.d_v] if wl.v_aliases_k else synth.to_f64(p["v"])
        ref = orc.prefill_attention(synth.to_f64(q), kk, vv, ocfg)
        H.check_output(out[cu[i]:cu[i + 1]], ref, wl, f"prompt {i} (L={L})")
        n = min(L, wl.l_obs)
        want = orc.candidate_log2_normalisers(synth.to_f64(p["q_obs"]), kk, ocfg)[:, wl.l_obs - n:]
        got = mu_host[i][:, wl.l_obs - n:]
        if np.isneginf(want).all():
            assert np.isneginf(got).all()
        else:
            np.testing.assert_allclose(got, want, rtol=0, atol=MU_ATOL, err_msg=f"prompt {i} (L={L})")
    n = len(lengths)
    slots = list(range(n))
    q_obs = torch.stack([p["q_obs"] for p in prompts]).cuda()
    ws = torch.empty(B.snap_compress_workspace_bytes(layer.cfg, cu), dtype=torch.uint8, device="cuda")
    idx = torch.full((n, wl.n_kv_heads, wl.topk), -7, dtype=torch.int32, device="cuda")
    c = layer.cache
    B.snap_compress_with_row_stats(layer.cfg, layer.layout, q_obs, mu, k, v, cu, slots, c.k_cache, c.v_cache, c.seq_len,
                                   c.valid_topk, idx, ws, c.status)
    assert layer.status() == 0
    idx = idx.cpu().numpy()
    for i, p in enumerate(prompts):
        seq = H.oracle_compress(wl, p)
        H.check_selection(idx[i], seq, wl)
        seq.topk_pos = [idx[i][h][idx[i][h] >= 0].astype(np.int64) for h in range(wl.n_kv_heads)]
        H.check_cache_image(layer, seq, slots[i], wl)


def test_normalisers_through_the_mma_sync_score_path(snap_option):
    snap_option(B.SNAP_OPT_SCORE_KERNEL, 1)
    test_compress_with_prefill_normalisers_matches_oracle(WL128)


def test_portable_prefill_kernel_matches_the_tensor_core_one(snap_option):
    wl = WL64
    lengths = [129, 300]
    _, _, _, cu, _, out_t, mu_t = _prefill(wl, lengths, seed=380)
    snap_option(B.SNAP_OPT_PREFILL_KERNEL, 1)
    _, _, _, _, _, out_s, mu_s = _prefill(wl, lengths, seed=380)
    assert (out_t.float() - out_s.float()).abs().max().item() <= 2e-2
    assert (mu_t - mu_s).abs().max().item() <= 2 * MU_ATOL
