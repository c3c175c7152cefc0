"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every declared
symbol, its layout arithmetic matches the oracle's, and it rejects bad arguments."""
import ctypes as C
import os
import re

import pytest

from oracle import snapstream_oracle as orc
from paper_2511_03092_b200 import binding as B
from paper_2511_03092_b200 import build as snap_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    snap_build.build()


def _cfg(**kw):
    base = dict(n_q_heads=32, n_kv_heads=8, d_qk=128, d_v=128, dtype=B.SNAP_BF16, l_sink=4, l_recent=1024,
                topk=4096, l_obs=64, pool_kernel=7, softmax_scale=0.088, max_seqs=3)
    base.update(kw)
    return B.make_config(**base)


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "snapstream.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(snap_[a-z_0-9]+)\s*\(", header))
    assert {"snap_cache_layout", "snap_compress", "snap_append_kv", "snap_decode_attn"} <= declared
    lib = B.lib()
    for name in declared:
        assert hasattr(lib, name), name
    assert set(B.EXPORTS) == declared


def test_layout_matches_oracle_and_paper_totals():
    for Ls, K, Lr, total in [(768, 6400, 1024, 8192), (512, 512, 31744, 32768), (4, 4096, 1024, 5124)]:
        cfg = _cfg(l_sink=Ls, l_recent=Lr, topk=K, l_obs=32)
        lay = B.snap_cache_layout(cfg)
        ref = orc.cache_layout(Ls, Lr, K)
        assert (lay.slots, lay.sink_off, lay.ring_off, lay.topk_off) == (
            ref["slots"], ref["sink_off"], ref["ring_off"], ref["topk_off"])
        assert lay.slots == total
        assert lay.k_row_bytes == 256 and lay.k_head_stride_bytes == 256 * total
        assert lay.k_seq_stride_bytes == 8 * 256 * total and lay.k_cache_bytes == 3 * 8 * 256 * total
    lay = B.snap_cache_layout(_cfg(n_q_heads=128, n_kv_heads=1, d_qk=576, d_v=512, v_aliases_k=True,
                                   l_recent=2048, topk=8192, l_obs=32))
    assert lay.slots == 10244 and lay.k_row_bytes == 1152 and lay.v_cache_bytes == 0
    lay = B.snap_cache_layout(_cfg(dtype=B.SNAP_F32))
    assert lay.k_row_bytes == 512


@pytest.mark.parametrize("kw,code", [
    (dict(n_q_heads=30), -1), (dict(l_recent=0), -1), (dict(l_obs=2000), -1), (dict(l_obs=0), -1),
    (dict(pool_kernel=4), -1), (dict(pool_kernel=0), -1), (dict(topk=-1), -1), (dict(l_sink=-1), -1),
    (dict(dtype=5), -1), (dict(pool_mode=3), -1), (dict(softmax_scale=0.0), -1), (dict(max_seqs=0), -1),
    (dict(d_qk=120), -2), (dict(d_v=1024, d_qk=1024), -2), (dict(v_aliases_k=True, d_v=256), -1),
])
def test_invalid_configs_are_rejected(kw, code):
    with pytest.raises(B.SnapError) as e:
        B.snap_cache_layout(_cfg(**kw))
    assert e.value.code == code
    assert B.status_string(code) != "unknown status"


def test_workspace_queries_and_argument_errors_without_gpu():
    cfg = _cfg()
    lay = B.snap_cache_layout(cfg)
    assert B.snap_compress_workspace_bytes(cfg, [0, 100, 8000]) > 0
    small = B.snap_compress_workspace_bytes(cfg, [0, 6000])
    big = B.snap_compress_workspace_bytes(cfg, [0, 60000])
    assert big > small
    assert B.snap_decode_workspace_bytes(cfg, 32) >= 32 * 32 * 130 * 4
    with pytest.raises(B.SnapError):
        B.snap_compress_workspace_bytes(cfg, [0, 10, 5])            # decreasing offsets
    lib = B.lib()
    cu = (C.c_int32 * 2)(0, 9000)
    bad_slot = (C.c_int32 * 1)(7)
    ok_slot = (C.c_int32 * 1)(0)
    one = C.c_void_p(256)   # never dereferenced: validation fails first
    args = lambda slots, ws_bytes, kts=1024: (C.byref(cfg), C.byref(lay), one, one, kts, 128, one, 1024, 128,
                                              cu, slots, 1, one, one, one, one, None, one, ws_bytes, None, None)
    assert lib.snap_compress(*args(bad_slot, 1 << 40)) == -1                 # slot out of range
    assert lib.snap_compress(*args(ok_slot, 16)) == -3                       # workspace too small
    assert lib.snap_compress(*args(ok_slot, 1 << 40, kts=1023)) == -1        # stride not 16-byte multiple
    assert lib.snap_compress(C.byref(cfg), C.byref(lay), one, None, 1024, 128, one, 1024, 128, cu, ok_slot, 1,
                             one, one, one, one, None, one, 1 << 40, None, None) == -4
    assert lib.snap_decode_attn(C.byref(cfg), C.byref(lay), one, None, None, one, 4, one, one, one, one, one,
                                one, 8, None, None) == -3
    assert lib.snap_decode_attn(C.byref(cfg), C.byref(lay), None, None, None, one, 4, one, one, one, one, one,
                                one, 1 << 40, None, None) == -4
    assert lib.snap_append_kv(C.byref(cfg), C.byref(lay), one, None, one, 2, one, one, one, None, None) == -4
    assert lib.snap_append_kv(C.byref(cfg), C.byref(lay), one, one, one, -1, one, one, one, None, None) == -1
    assert lib.snap_decode_attn(C.byref(cfg), C.byref(lay), one, None, None, one, 0, one, one, one, one, one,
                                one, 0, None, None) == 0                     # nothing to do
    # device buffers that do not start on a 16-byte boundary are refused before anything is launched
    odd = C.c_void_p(264)
    assert lib.snap_compress(C.byref(cfg), C.byref(lay), one, odd, 1024, 128, one, 1024, 128, cu, ok_slot, 1,
                             one, one, one, one, None, one, 1 << 40, None, None) == -1
    assert lib.snap_compress(C.byref(cfg), C.byref(lay), one, one, 1024, 128, one, 1024, 128, cu, ok_slot, 1,
                             one, one, one, one, None, odd, 1 << 40, None, None) == -1
    assert lib.snap_decode_attn(C.byref(cfg), C.byref(lay), odd, None, None, one, 4, one, one, one, one, one,
                                one, 1 << 40, None, None) == -1
    assert lib.snap_decode_attn(C.byref(cfg), C.byref(lay), one, None, None, one, 4, one, one, one, one, one,
                                odd, 1 << 40, None, None) == -1
    assert lib.snap_append_kv(C.byref(cfg), C.byref(lay), one, one, one, 2, odd, one, one, None, None) == -1
    two = C.c_void_p(512)
    cc = lambda *a: lib.snap_append_kv_concat(C.byref(cfg), C.byref(lay), *a)
    assert cc(one, one, one, 2, one, one, one, one, one, None, None) == -1   # in place: output must differ from input
    assert cc(one, one, one, 2, one, one, None, two, one, None, None) == -4  # missing output buffer
    assert cc(one, None, one, 2, one, one, two, two, one, None, None) == -4  # missing new values
    assert cc(one, one, one, -3, one, one, two, two, one, None, None) == -1
    assert cc(one, one, one, 0, one, one, two, two, one, None, None) == 0    # nothing to do


def test_prefill_entry_points_validate_before_touching_memory():
    cfg = _cfg()
    lay = B.snap_cache_layout(cfg)
    lib = B.lib()
    one = C.c_void_p(256)   # never dereferenced: validation fails first
    cu_bad = (C.c_int32 * 3)(0, 10, 5)
    cu = (C.c_int32 * 2)(0, 9000)
    pre = lambda c, cup, n: lib.snap_prefill_attn(c, one, one, 1024, 128, one, 1024, 128, cup, n, one, None, None, None)
    assert pre(None, cu, 1) == -4                                            # no config
    assert pre(C.byref(cfg), cu_bad, 2) == -1                                # decreasing offsets
    assert pre(C.byref(cfg), None, 1) == -4
    assert pre(C.byref(_cfg(softmax_scale=-1.0)), cu, 1) == -1
    assert lib.snap_prefill_attn(C.byref(cfg), one, one, 1023, 128, one, 1024, 128, cu, 1, one, None, None, None) == -1
    assert lib.snap_prefill_attn(C.byref(cfg), one, one, 1024, 128, None, 1024, 128, cu, 1, one, None, None, None) == -4
    empty = (C.c_int32 * 3)(0, 0, 0)
    assert pre(C.byref(cfg), empty, 2) == 0                                  # nothing to do
    # the compress variant shares snap_compress's validation
    ok_slot = (C.c_int32 * 1)(0)
    bad_slot = (C.c_int32 * 1)(7)
    crs = lambda slots, ws_bytes, kts=1024, mu=one: lib.snap_compress_with_row_stats(
        C.byref(cfg), C.byref(lay), one, mu, one, kts, 128, one, 1024, 128, cu, slots, 1, one, one, one, one, None, one,
        ws_bytes, None, None)
    assert crs(bad_slot, 1 << 40) == -1
    assert crs(ok_slot, 1 << 40, kts=1023) == -1
    assert crs(ok_slot, 16, mu=None) == -3                                   # without normalisers it is snap_compress


def test_header_is_plain_c99(tmp_path):
    """The boundary is a C ABI: the header must compile as C99 on its own, and a C caller must be able to
    link against the library and use the host-only entry points."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = tmp_path / "use_header.c"
    src.write_text(
        '#include "snapstream.h"\n'
        "#include <stdio.h>\n"
        "int main(void) {\n"
        "  snap_config_t cfg = {32, 8, 128, 128, 0, SNAP_BF16, 4, 1024, 4096, 64, 7, SNAP_POOL_AVG, 0.088388f, 32};\n"
        "  snap_layout_t lay;\n"
        "  int rc = snap_cache_layout(&cfg, &lay);\n"
        '  printf("%d %d %d %d %d %s\\n", rc, lay.slots, lay.sink_off, lay.ring_off, lay.topk_off, snap_status_string(-3));\n'
        "  cfg.l_obs = 0;\n"
        "  return snap_cache_layout(&cfg, &lay) == SNAP_ERR_INVALID_ARG ? 0 : 1;\n"
        "}\n")
    obj = tmp_path / "use_header.o"
    subprocess.run([gcc, "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(root, "include"),
                    "-c", str(src), "-o", str(obj)], check=True)
    libdir = os.path.join(root, "paper_2511_03092_b200")
    exe = tmp_path / "use_header"
    subprocess.run([gcc, str(obj), "-L", libdir, "-lsnapstream", "-Wl,-rpath," + libdir, "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()
    assert out[:5] == ["0", "5124", "0", "4", "1028"]


def test_debug_options_are_process_wide_integers():
    """snap_debug_set_option: returns the previous value, rejects unknown options and negative
    values, and what it sets changes the library's planning (host arithmetic only, no GPU)."""
    before = B.snap_debug_set_option(B.SNAP_OPT_REFINE_OFF, 1)
    try:
        assert B.snap_debug_set_option(B.SNAP_OPT_REFINE_OFF, 1) == 1
        cfg = _cfg()
        cu = [0, 40000]
        without = B.snap_compress_workspace_bytes(cfg, cu)
        B.snap_debug_set_option(B.SNAP_OPT_REFINE_OFF, 0)
        with_refine = B.snap_compress_workspace_bytes(cfg, cu)
        assert with_refine > without                      # band entries, column sums, normalisers, verdict lists
    finally:
        B.snap_debug_set_option(B.SNAP_OPT_REFINE_OFF, before)
    for bad in ((-1, 0), (99, 0), (B.SNAP_OPT_REFINE_OFF, -3)):
        with pytest.raises(B.SnapError) as e:
            B.snap_debug_set_option(*bad)
        assert e.value.code == -1
