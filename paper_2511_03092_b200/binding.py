"""ctypes binding of libsnapstream.so: argument marshalling only.

Every function mirrors one entry point of include/snapstream.h and takes torch tensors
(used purely as device memory) or raw integers.  Nothing is computed here; if the shared
library is missing the import of this module's symbols fails loudly -- there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import torch

# SNAP_LIBRARY names another build of the library in this directory (the checked build, libsnapstream_dbg.so)
_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)),
                         os.path.basename(os.environ.get("SNAP_LIBRARY", "libsnapstream.so")))

SNAP_F32, SNAP_BF16 = 0, 1
SNAP_POOL_AVG, SNAP_POOL_MAX = 0, 1
SNAP_DEV_BAD_SLOT, SNAP_DEV_WAIT_TIMEOUT, SNAP_DEV_BAND_OVERFLOW, SNAP_DEV_INDEX_CHECK = 1, 2, 4, 8


class SnapConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_q_heads", "n_kv_heads", "d_qk", "d_v", "v_aliases_k", "dtype",
                                         "l_sink", "l_recent", "topk", "l_obs", "pool_kernel", "pool_mode")]
    _fields_ += [("softmax_scale", C.c_float), ("max_seqs", C.c_int32)]


class SnapLayout(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("slots", "sink_off", "ring_off", "topk_off")]
    _fields_ += [(n, C.c_int64) for n in ("k_row_bytes", "v_row_bytes", "k_head_stride_bytes",
                                          "v_head_stride_bytes", "k_seq_stride_bytes", "v_seq_stride_bytes",
                                          "k_cache_bytes", "v_cache_bytes")]


class SnapError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


_lib = None


def lib() -> C.CDLL:
    """Load libsnapstream.so (built by paper_2511_03092_b200.build); raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2511_03092_b200.build` "
                           "(there is no CPU fallback)")
    L = C.CDLL(_LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    pcfg, play = C.POINTER(SnapConfig), C.POINTER(SnapLayout)
    L.snap_status_string.restype = C.c_char_p
    L.snap_status_string.argtypes = [C.c_int]
    L.snap_kernel_launch_count.restype = i64
    L.snap_kernel_launch_count.argtypes = []
    L.snap_cache_layout.restype = C.c_int
    L.snap_cache_layout.argtypes = [pcfg, play]
    L.snap_compress_workspace_bytes.restype = i64
    L.snap_compress_workspace_bytes.argtypes = [pcfg, C.POINTER(i32), i32]
    L.snap_decode_workspace_bytes.restype = i64
    L.snap_decode_workspace_bytes.argtypes = [pcfg, i32]
    L.snap_compress.restype = C.c_int
    L.snap_compress.argtypes = [pcfg, play, vp, vp, i64, i64, vp, i64, i64, C.POINTER(i32), C.POINTER(i32), i32,
                                vp, vp, vp, vp, vp, vp, sz, vp, vp]
    L.snap_compress_with_row_stats.restype = C.c_int
    L.snap_compress_with_row_stats.argtypes = [pcfg, play, vp, vp, vp, i64, i64, vp, i64, i64, C.POINTER(i32),
                                               C.POINTER(i32), i32, vp, vp, vp, vp, vp, vp, sz, vp, vp]
    L.snap_prefill_attn.restype = C.c_int
    L.snap_prefill_attn.argtypes = [pcfg, vp, vp, i64, i64, vp, i64, i64, C.POINTER(i32), i32, vp, vp, vp, vp]
    L.snap_append_kv.restype = C.c_int
    L.snap_append_kv.argtypes = [pcfg, play, vp, vp, vp, i32, vp, vp, vp, vp, vp]
    L.snap_append_kv_concat.restype = C.c_int
    L.snap_append_kv_concat.argtypes = [pcfg, play, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp]
    L.snap_decode_attn.restype = C.c_int
    L.snap_decode_attn.argtypes = [pcfg, play, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp, sz, vp, vp]
    L.snap_decode_multi_workspace_bytes.restype = i64
    L.snap_decode_multi_workspace_bytes.argtypes = [pcfg, i32, i32]
    L.snap_decode_attn_multi.restype = C.c_int
    L.snap_decode_attn_multi.argtypes = [pcfg, play, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp, sz, vp, vp]
    L.snap_decode_attn_static.restype = C.c_int
    L.snap_decode_attn_static.argtypes = [pcfg, play, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp]
    L.snap_debug_set_option.restype = C.c_int
    L.snap_debug_set_option.argtypes = [C.c_int, C.c_int]
    L.snap_block_stats_bytes.restype = i64
    L.snap_block_stats_bytes.argtypes = [pcfg, i32]
    L.snap_block_stats.restype = C.c_int
    L.snap_block_stats.argtypes = [pcfg, play, vp, i32, vp, vp, i32, vp, vp, vp]
    L.snap_block_select.restype = C.c_int
    L.snap_block_select.argtypes = [pcfg, play, vp, vp, i32, vp, vp, i32, i32, vp, vp, vp, sz, vp, vp]
    L.snap_block_select_workspace_bytes.restype = i64
    L.snap_block_select_workspace_bytes.argtypes = [pcfg, i32, i32]
    L.snap_decode_blocks_workspace_bytes.restype = i64
    L.snap_decode_blocks_workspace_bytes.argtypes = [pcfg, i32, i32, i32]
    L.snap_decode_attn_blocks.restype = C.c_int
    L.snap_decode_attn_blocks.argtypes = [pcfg, play, vp, vp, vp, vp, i32, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, sz, vp, vp]
    _lib = L
    return L


EXPORTS = ("snap_cache_layout", "snap_compress_workspace_bytes", "snap_decode_workspace_bytes",
           "snap_compress", "snap_append_kv", "snap_append_kv_concat", "snap_decode_attn",
           "snap_decode_multi_workspace_bytes", "snap_decode_attn_multi", "snap_decode_attn_static", "snap_status_string",
           "snap_kernel_launch_count", "snap_prefill_attn", "snap_compress_with_row_stats", "snap_debug_set_option",
           "snap_block_stats_bytes", "snap_block_stats", "snap_block_select", "snap_block_select_workspace_bytes",
           "snap_decode_blocks_workspace_bytes",
           "snap_decode_attn_blocks")

# testing / tuning options of snap_debug_set_option
(SNAP_OPT_SCORE_KERNEL, SNAP_OPT_DECODE_GQA_KERNEL, SNAP_OPT_DECODE_LATENT_KERNEL, SNAP_OPT_DECODE_NSPLIT,
 SNAP_OPT_SCORE_NSPLIT, SNAP_OPT_WIDE_STAGES, SNAP_OPT_PREFILL_KERNEL, SNAP_OPT_PREFILL_SINGLE_HEADS,
 SNAP_OPT_REFINE_OFF) = range(9)


def status_string(code: int) -> str:
    return lib().snap_status_string(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != 0:
        raise SnapError(int(code), where)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _i32_array(xs: Sequence[int]):
    return (C.c_int32 * len(xs))(*[int(x) for x in xs])


def make_config(*, n_q_heads, n_kv_heads, d_qk, d_v, dtype, l_sink, l_recent, topk, l_obs, pool_kernel,
                softmax_scale, max_seqs, pool_mode=SNAP_POOL_AVG, v_aliases_k=False) -> SnapConfig:
    if isinstance(dtype, torch.dtype):
        dtype = {torch.float32: SNAP_F32, torch.bfloat16: SNAP_BF16}[dtype]
    if isinstance(pool_mode, str):
        pool_mode = {"avg": SNAP_POOL_AVG, "max": SNAP_POOL_MAX}[pool_mode]
    return SnapConfig(n_q_heads, n_kv_heads, d_qk, d_v, int(bool(v_aliases_k)), dtype, l_sink, l_recent, topk,
                      l_obs, pool_kernel, pool_mode, float(softmax_scale), max_seqs)


def snap_debug_set_option(option: int, value: int) -> int:
    """Set a process-wide testing / tuning option; returns its previous value."""
    old = lib().snap_debug_set_option(int(option), int(value))
    if old < 0:
        raise SnapError(int(old), "snap_debug_set_option")
    return int(old)


def snap_kernel_launch_count() -> int:
    return int(lib().snap_kernel_launch_count())


def snap_cache_layout(cfg: SnapConfig) -> SnapLayout:
    lay = SnapLayout()
    _check(lib().snap_cache_layout(C.byref(cfg), C.byref(lay)), "snap_cache_layout")
    return lay


def snap_compress_workspace_bytes(cfg: SnapConfig, cu_seqlens: Sequence[int]) -> int:
    cu = _i32_array(cu_seqlens)
    n = lib().snap_compress_workspace_bytes(C.byref(cfg), cu, len(cu_seqlens) - 1)
    if n < 0:
        raise SnapError(int(n), "snap_compress_workspace_bytes")
    return int(n)


def snap_decode_workspace_bytes(cfg: SnapConfig, n_active: int) -> int:
    n = lib().snap_decode_workspace_bytes(C.byref(cfg), int(n_active))
    if n < 0:
        raise SnapError(int(n), "snap_decode_workspace_bytes")
    return int(n)


def snap_compress(cfg: SnapConfig, layout: SnapLayout, q_obs, k, v, cu_seqlens: Sequence[int],
                  slot_ids: Sequence[int], k_cache, v_cache, seq_len, valid_topk, topk_idx=None,
                  workspace=None, status=None, stream=None, k_strides=None, v_strides=None) -> None:
    """k, v: [total_tokens, Hkv, d] tensors (any strides with a dense last dim), or pass
    k_strides/v_strides = (token_stride, head_stride) in elements explicitly."""
    ks = k_strides if k_strides is not None else (k.stride(0), k.stride(1))
    if v is not None:
        vs = v_strides if v_strides is not None else (v.stride(0), v.stride(1))
    else:
        vs = (0, 0)
    cu = _i32_array(cu_seqlens)
    sl = _i32_array(slot_ids)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().snap_compress(C.byref(cfg), C.byref(layout), _ptr(q_obs), _ptr(k), ks[0], ks[1], _ptr(v),
                               vs[0], vs[1], cu, sl, len(slot_ids), _ptr(k_cache), _ptr(v_cache),
                               _ptr(seq_len), _ptr(valid_topk), _ptr(topk_idx), _ptr(workspace), ws_bytes,
                               _ptr(status), _stream(stream)), "snap_compress")


def snap_compress_with_row_stats(cfg: SnapConfig, layout: SnapLayout, q_obs, row_mu, k, v, cu_seqlens: Sequence[int],
                                 slot_ids: Sequence[int], k_cache, v_cache, seq_len, valid_topk, topk_idx=None,
                                 workspace=None, status=None, stream=None) -> None:
    """snap_compress with the Eq. 4 normalisers (row_mu: [n_seq, Hq, Lo] float32, as written by
    snap_prefill_attn) supplied instead of computed."""
    vs = (v.stride(0), v.stride(1)) if v is not None else (0, 0)
    cu = _i32_array(cu_seqlens)
    sl = _i32_array(slot_ids)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().snap_compress_with_row_stats(C.byref(cfg), C.byref(layout), _ptr(q_obs), _ptr(row_mu), _ptr(k),
                                              k.stride(0), k.stride(1), _ptr(v), vs[0], vs[1], cu, sl, len(slot_ids),
                                              _ptr(k_cache), _ptr(v_cache), _ptr(seq_len), _ptr(valid_topk),
                                              _ptr(topk_idx), _ptr(workspace), ws_bytes, _ptr(status),
                                              _stream(stream)), "snap_compress_with_row_stats")


def snap_prefill_attn(cfg: SnapConfig, q, k, v, cu_seqlens: Sequence[int], out, row_mu=None, status=None,
                      stream=None) -> None:
    """Causal attention of whole prompts.  q: [T, Hq, d] dense; k, v: [T, Hkv, d] (dense last dim; v None for
    the latent layout);
    out: [T, Hq, d_v]; row_mu: None or [n_seq, Hq, Lo] float32 receiving the Eq. 4 normalisers."""
    cu = _i32_array(cu_seqlens)
    vs = (v.stride(0), v.stride(1)) if v is not None else (0, 0)
    _check(lib().snap_prefill_attn(C.byref(cfg), _ptr(q), _ptr(k), k.stride(0), k.stride(1), _ptr(v), vs[0], vs[1], cu,
                                   len(cu_seqlens) - 1, _ptr(out), _ptr(row_mu), _ptr(status), _stream(stream)),
           "snap_prefill_attn")


def snap_append_kv(cfg: SnapConfig, layout: SnapLayout, k_new, v_new, slot_ids_dev, n_active: int, k_cache,
                   v_cache, seq_len, status=None, stream=None) -> None:
    _check(lib().snap_append_kv(C.byref(cfg), C.byref(layout), _ptr(k_new), _ptr(v_new), _ptr(slot_ids_dev),
                                int(n_active), _ptr(k_cache), _ptr(v_cache), _ptr(seq_len), _ptr(status),
                                _stream(stream)), "snap_append_kv")


def snap_append_kv_concat(cfg: SnapConfig, layout: SnapLayout, k_new, v_new, slot_ids_dev, n_active: int,
                          k_cache_in, v_cache_in, k_cache_out, v_cache_out, seq_len, status=None,
                          stream=None) -> None:
    """Baseline update by slicing and concatenating into a second cache (position-ordered window)."""
    _check(lib().snap_append_kv_concat(C.byref(cfg), C.byref(layout), _ptr(k_new), _ptr(v_new),
                                       _ptr(slot_ids_dev), int(n_active), _ptr(k_cache_in), _ptr(v_cache_in),
                                       _ptr(k_cache_out), _ptr(v_cache_out), _ptr(seq_len), _ptr(status),
                                       _stream(stream)), "snap_append_kv_concat")


def snap_decode_attn(cfg: SnapConfig, layout: SnapLayout, q, k_new, v_new, slot_ids_dev, n_active: int,
                     k_cache, v_cache, seq_len, valid_topk, out, workspace, status=None, stream=None) -> None:
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().snap_decode_attn(C.byref(cfg), C.byref(layout), _ptr(q), _ptr(k_new), _ptr(v_new),
                                  _ptr(slot_ids_dev), int(n_active), _ptr(k_cache), _ptr(v_cache),
                                  _ptr(seq_len), _ptr(valid_topk), _ptr(out), _ptr(workspace), ws_bytes,
                                  _ptr(status), _stream(stream)), "snap_decode_attn")


def snap_decode_multi_workspace_bytes(cfg: SnapConfig, n_active: int, q_len: int) -> int:
    n = lib().snap_decode_multi_workspace_bytes(C.byref(cfg), int(n_active), int(q_len))
    if n < 0:
        raise SnapError(int(n), "snap_decode_multi_workspace_bytes")
    return int(n)


def snap_decode_attn_multi(cfg: SnapConfig, layout: SnapLayout, q, k_new, v_new, slot_ids_dev, n_active: int,
                           q_len: int, k_cache, v_cache, seq_len, valid_topk, out, workspace, status=None,
                           stream=None) -> None:
    """q_len new tokens per sequence in one pass over the cache (q [n][q_len][Hq][d], out alike)."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().snap_decode_attn_multi(C.byref(cfg), C.byref(layout), _ptr(q), _ptr(k_new), _ptr(v_new),
                                        _ptr(slot_ids_dev), int(n_active), int(q_len), _ptr(k_cache),
                                        _ptr(v_cache), _ptr(seq_len), _ptr(valid_topk), _ptr(out),
                                        _ptr(workspace), ws_bytes, _ptr(status), _stream(stream)),
           "snap_decode_attn_multi")


def snap_decode_attn_static(cfg: SnapConfig, layout: SnapLayout, q, k_new, v_new, slot_ids_dev, n_active: int,
                            k_cache, v_cache, seq_len, valid_topk, out, status=None, stream=None) -> None:
    """Decode step without a workspace argument: scratch is a fixed array inside the library, for
    callers that must not allocate.  Raises SnapError(-6) when the batch does not fit that array."""
    _check(lib().snap_decode_attn_static(C.byref(cfg), C.byref(layout), _ptr(q), _ptr(k_new), _ptr(v_new),
                                         _ptr(slot_ids_dev), int(n_active), _ptr(k_cache), _ptr(v_cache),
                                         _ptr(seq_len), _ptr(valid_topk), _ptr(out), _ptr(status),
                                         _stream(stream)), "snap_decode_attn_static")


@dataclass
class CacheBuffers:
    """Device buffers of one layer's compressed cache (torch is used only as the allocator)."""
    k_cache: torch.Tensor
    v_cache: Optional[torch.Tensor]
    seq_len: torch.Tensor
    valid_topk: torch.Tensor
    status: torch.Tensor


def alloc_cache(cfg: SnapConfig, layout: SnapLayout, device="cuda") -> CacheBuffers:
    dt = torch.float32 if cfg.dtype == SNAP_F32 else torch.bfloat16
    kc = torch.zeros(cfg.max_seqs, cfg.n_kv_heads, layout.slots, cfg.d_qk, dtype=dt, device=device)
    vc = None
    if not cfg.v_aliases_k:
        vc = torch.zeros(cfg.max_seqs, cfg.n_kv_heads, layout.slots, cfg.d_v, dtype=dt, device=device)
    return CacheBuffers(kc, vc, torch.zeros(cfg.max_seqs, dtype=torch.int32, device=device),
                        torch.zeros(cfg.max_seqs, dtype=torch.int32, device=device),
                        torch.zeros(1, dtype=torch.int32, device=device))


def snap_block_stats_bytes(cfg: SnapConfig, block_tokens: int) -> int:
    n = lib().snap_block_stats_bytes(C.byref(cfg), int(block_tokens))
    if n < 0:
        raise SnapError(int(n), "snap_block_stats_bytes")
    return int(n)


def snap_block_stats(cfg: SnapConfig, layout: SnapLayout, slot_ids_dev, n_seqs: int, k_cache, valid_topk,
                     block_tokens: int, stats, status=None, stream=None) -> None:
    """Per-block key minima and maxima of the third section of the given slots' caches."""
    _check(lib().snap_block_stats(C.byref(cfg), C.byref(layout), _ptr(slot_ids_dev), int(n_seqs), _ptr(k_cache),
                                  _ptr(valid_topk), int(block_tokens), _ptr(stats), _ptr(status), _stream(stream)),
           "snap_block_stats")


def snap_block_select(cfg: SnapConfig, layout: SnapLayout, q, slot_ids_dev, n_active: int, stats, valid_topk,
                      block_tokens: int, n_blocks: int, block_idx, n_selected, workspace, status=None, stream=None) -> None:
    """The n_blocks highest-scoring blocks per (sequence, KV head) for this step's queries."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().snap_block_select(C.byref(cfg), C.byref(layout), _ptr(q), _ptr(slot_ids_dev), int(n_active), _ptr(stats),
                                   _ptr(valid_topk), int(block_tokens), int(n_blocks), _ptr(block_idx), _ptr(n_selected),
                                   _ptr(workspace), ws_bytes, _ptr(status), _stream(stream)), "snap_block_select")


def snap_block_select_workspace_bytes(cfg: SnapConfig, n_active: int, block_tokens: int) -> int:
    n = lib().snap_block_select_workspace_bytes(C.byref(cfg), int(n_active), int(block_tokens))
    if n < 0:
        raise SnapError(int(n), "snap_block_select_workspace_bytes")
    return int(n)


def snap_decode_blocks_workspace_bytes(cfg: SnapConfig, n_active: int, block_tokens: int, n_blocks: int) -> int:
    n = lib().snap_decode_blocks_workspace_bytes(C.byref(cfg), int(n_active), int(block_tokens), int(n_blocks))
    if n < 0:
        raise SnapError(int(n), "snap_decode_blocks_workspace_bytes")
    return int(n)


def snap_decode_attn_blocks(cfg: SnapConfig, layout: SnapLayout, q, k_new, v_new, slot_ids_dev, n_active: int, k_cache,
                            v_cache, seq_len, valid_topk, block_tokens: int, n_blocks: int, block_idx, n_selected, out,
                            workspace, status=None, stream=None) -> None:
    """snap_decode_attn over the sinks, the window and the listed blocks of the third section."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().snap_decode_attn_blocks(C.byref(cfg), C.byref(layout), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(slot_ids_dev),
                                         int(n_active), _ptr(k_cache), _ptr(v_cache), _ptr(seq_len), _ptr(valid_topk),
                                         int(block_tokens), int(n_blocks), _ptr(block_idx), _ptr(n_selected), _ptr(out),
                                         _ptr(workspace), ws_bytes, _ptr(status), _stream(stream)), "snap_decode_attn_blocks")
