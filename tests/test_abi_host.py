"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and rejects bad arguments before anything is launched."""
import ctypes as C
import os
import re

import pytest

from paper_2511_11641_b200 import binding as B
from paper_2511_11641_b200 import build as lib_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    lib_build.build()
    return B.lib()


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(ecospa_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert "ecospa_score_pairs" in names and "ecospa_select_aligned_topk" in names and "ecospa_compact_pair" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/ but not exported"


def test_status_strings(lib):
    assert lib.ecospa_status_string(0) == b"ok"
    assert b"invalid" in lib.ecospa_status_string(1)
    assert lib.ecospa_status_string(99) == b"unknown status"


def _fake_mat(ptr, dtype=B.BF16, layout=B.SHARED_COLS, other=64, ld=64):
    return B.Mat(ptr, dtype, layout, other, ld)


def test_score_rejects_bad_arguments_without_launching(lib):
    null = B.Mat(None, 0, 0, 0, 0)
    good = _fake_mat(0x1000)
    p = B.Pair(B.PAIR_PLAIN, 1, 64, 0, good, null, _fake_mat(0x2000, layout=B.SHARED_ROWS), null, null, null)
    arr = (B.Pair * 1)(p)
    ups = C.c_void_p(0x3000)
    ws = C.c_void_p(0x4000)
    # null pair array / null upsilon / non-positive n_samples
    assert lib.ecospa_score_pairs(None, 1, 1.0, ups, None, None, ws, 1 << 20, None) == 1
    assert lib.ecospa_score_pairs(C.addressof(arr), 1, 1.0, None, None, None, ws, 1 << 20, None) == 1
    assert lib.ecospa_score_pairs(C.addressof(arr), 1, 0.0, ups, None, None, ws, 1 << 20, None) == 1
    # missing workspace, too-small workspace, misaligned workspace
    assert lib.ecospa_score_pairs(C.addressof(arr), 1, 1.0, ups, None, None, None, 0, None) == 6
    assert lib.ecospa_score_pairs(C.addressof(arr), 1, 1.0, ups, None, None, ws, 16, None) == 6
    assert lib.ecospa_score_pairs(C.addressof(arr), 1, 1.0, ups, None, None, C.c_void_p(0x4004), 1 << 20, None) == 2
    # Fisher requested but gradients absent
    assert lib.ecospa_score_pairs(C.addressof(arr), 1, 1.0, ups, None, C.c_void_p(0x5000), ws, 1 << 20, None) == 1
    # ld smaller than the shared extent; weights of different dtypes; SwiGLU without the up matrix
    bad = B.Pair(B.PAIR_PLAIN, 1, 64, 0, _fake_mat(0x1000, ld=32), null, _fake_mat(0x2000, layout=B.SHARED_ROWS), null, null, null)
    assert lib.ecospa_score_pairs(C.addressof((B.Pair * 1)(bad)), 1, 1.0, ups, None, None, ws, 1 << 20, None) == 1
    bad = B.Pair(B.PAIR_PLAIN, 1, 64, 0, good, null, _fake_mat(0x2000, dtype=B.F32, layout=B.SHARED_ROWS), null, null, null)
    assert lib.ecospa_score_pairs(C.addressof((B.Pair * 1)(bad)), 1, 1.0, ups, None, None, ws, 1 << 20, None) == 1
    bad = B.Pair(B.PAIR_SWIGLU, 1, 64, 0, good, null, _fake_mat(0x2000, layout=B.SHARED_ROWS), null, null, null)
    assert lib.ecospa_score_pairs(C.addressof((B.Pair * 1)(bad)), 1, 1.0, ups, None, None, ws, 1 << 20, None) == 1
    # odd element pointer
    bad = B.Pair(B.PAIR_PLAIN, 1, 64, 0, _fake_mat(0x1001), null, _fake_mat(0x2000, layout=B.SHARED_ROWS), null, null, null)
    assert lib.ecospa_score_pairs(C.addressof((B.Pair * 1)(bad)), 1, 1.0, ups, None, None, ws, 1 << 20, None) == 2
    assert lib.ecospa_score_workspace_bytes(C.addressof(arr), 1) > 0
    assert lib.ecospa_score_workspace_bytes(None, 1) == 0


def test_select_rejects_bad_arguments_without_launching(lib):
    ups = C.c_void_p(0x1000)
    kept = C.c_void_p(0x2000)
    one = (C.c_int32 * 1)(1)
    slen = (C.c_int32 * 1)(64)
    for k, expect in ((65, 1), (-1, 1)):
        kk = (C.c_int32 * 1)(k)
        assert lib.ecospa_select_aligned_topk(ups, C.addressof(one), C.addressof(slen), C.addressof(kk), 1, kept, None, None) == expect
    kk = (C.c_int32 * 1)(32)
    assert lib.ecospa_select_aligned_topk(None, C.addressof(one), C.addressof(slen), C.addressof(kk), 1, kept, None, None) == 1
    assert lib.ecospa_select_aligned_topk(ups, C.addressof(one), C.addressof(slen), C.addressof(kk), 1, None, None, None) == 1
    big = (C.c_int32 * 1)((1 << 20) + 1)
    assert lib.ecospa_select_aligned_topk(ups, C.addressof(one), C.addressof(big), C.addressof(kk), 1, kept, None, None) == 3


def test_compact_rejects_bad_arguments_without_launching(lib):
    kept = 0x9000
    m_in = _fake_mat(0x10000, other=8, ld=64)
    # output overlapping the input
    g = B.Gather(m_in, _fake_mat(0x10010, other=8, ld=32), kept, 32, 64)
    assert lib.ecospa_compact_tensors(C.addressof((B.Gather * 1)(g)), 1, None) == 1
    # output pitch smaller than n_kept
    g = B.Gather(m_in, _fake_mat(0x20000, other=8, ld=16), kept, 32, 64)
    assert lib.ecospa_compact_tensors(C.addressof((B.Gather * 1)(g)), 1, None) == 1
    # dtype mismatch, n_kept > D, null kept
    g = B.Gather(m_in, _fake_mat(0x20000, dtype=B.F32, other=8, ld=32), kept, 32, 64)
    assert lib.ecospa_compact_tensors(C.addressof((B.Gather * 1)(g)), 1, None) == 1
    g = B.Gather(m_in, _fake_mat(0x20000, other=8, ld=128), kept, 65, 64)
    assert lib.ecospa_compact_tensors(C.addressof((B.Gather * 1)(g)), 1, None) == 1
    g = B.Gather(m_in, _fake_mat(0x20000, other=8, ld=32), None, 32, 64)
    assert lib.ecospa_compact_tensors(C.addressof((B.Gather * 1)(g)), 1, None) == 1
    assert lib.ecospa_compact_tensors(None, 1, None) == 1


def test_threshold_selection_rejects_bad_arguments_without_launching(lib):
    fn = lib.ecospa_select_aligned_threshold
    fn.restype = C.c_int
    fn.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_double, C.c_int32, C.c_int32, C.c_void_p,
                   C.c_void_p, C.c_void_p, C.c_void_p]
    ups, kept, kout = C.c_void_p(0x1000), C.c_void_p(0x2000), C.c_void_p(0x3000)
    one = (C.c_int32 * 1)(1)
    slen = (C.c_int32 * 1)(64)
    a = (C.addressof(one), C.addressof(slen), None, 1)
    odd = (C.c_int32 * 1)(63)
    mode = (C.c_int32 * 1)(2)
    assert fn(ups, C.addressof(one), C.addressof(odd), C.addressof(mode), 1, 0.9, 1, 1, None, kept, kout, None) == 1
    bad = (C.c_int32 * 1)(5)
    assert fn(ups, C.addressof(one), C.addressof(slen), C.addressof(bad), 1, 0.9, 1, 1, None, kept, kout, None) == 1
    assert fn(None, *a, 0.9, 1, 1, None, kept, kout, None) == 1
    assert fn(ups, *a, 0.9, 1, 1, None, None, kout, None) == 1
    assert fn(ups, *a, 0.9, 1, 1, None, kept, None, None) == 1
    assert fn(ups, *a, -0.1, 1, 1, None, kept, kout, None) == 1
    assert fn(ups, *a, float("nan"), 1, 1, None, kept, kout, None) == 1
    assert fn(ups, *a, 0.9, 1, -1, None, kept, kout, None) == 1
    big = (C.c_int32 * 1)((1 << 20) + 1)
    assert fn(ups, C.addressof(one), C.addressof(big), None, 1, 0.9, 1, 1, None, kept, kout, None) == 3
    ch = lib.ecospa_choose_pairs
    ch.restype = C.c_int
    ch.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
    assert ch(None, 4, 1, kept, None) == 1
    assert ch(ups, 0, 1, kept, None) == 1
    assert ch(ups, 4, -1, kept, None) == 1
    assert ch(ups, 1 << 15, 1, kept, None) == 3


def test_rotation_pair_selection_rejects_bad_arguments_without_launching(lib):
    fn = lib.ecospa_select_rotation_pairs
    fn.restype = C.c_int
    fn.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    ups, kept = C.c_void_p(0x1000), C.c_void_p(0x2000)
    one = (C.c_int32 * 1)(1)

    def call(seg_len, k, mode, rope_null=False):
        sl, kk, rp = (C.c_int32 * 1)(seg_len), (C.c_int32 * 1)(k), (C.c_int32 * 1)(mode)
        return fn(ups, C.addressof(one), C.addressof(sl), C.addressof(kk), None if rope_null else C.addressof(rp), 1,
                  kept, None, None)

    assert call(64, 31, 1) == 1          # an odd count would split a rotation pair
    assert call(63, 30, 2) == 1          # a segment of odd length has no pairing
    assert call(64, 32, 3) == 1          # unknown pairing
    assert call(64, 66, 1) == 1          # more than the segment holds
    assert call(64, 32, 1, rope_null=True) == 1


def test_pack_kept_rejects_bad_arguments_without_launching(lib):
    fn = lib.ecospa_pack_kept
    fn.restype = C.c_int
    fn.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
    slots, out = C.c_void_p(0x1000), C.c_void_p(0x2000)
    z, neg = (C.c_int32 * 1)(0), (C.c_int32 * 1)(-1)
    a = C.addressof
    assert fn(None, a(z), a(z), a(z), a(z), 1, out, None) == 1
    assert fn(slots, a(z), a(z), a(z), a(z), 1, None, None) == 1
    assert fn(slots, a(z), a(z), a(z), a(z), 0, out, None) == 1
    assert fn(slots, a(neg), a(z), a(z), a(z), 1, out, None) == 1
    assert fn(slots, a(z), a(z), a(neg), a(z), 1, out, None) == 1


# ---------------------------------------------------------------------------------------------
# step 4 (compacted-pair forward/backward): everything below is rejected on the host, before any
# CUDA call, so it runs without a GPU.  Pointers are fake addresses that are never dereferenced.
# ---------------------------------------------------------------------------------------------

def _w(ptr, layout=B.SHARED_COLS, d_m=64, ld=64, dtype=B.BF16):
    return B.Mat(ptr, dtype, layout, d_m, ld)


def test_layer_calls_reject_bad_arguments_without_launching(lib):
    f = B._fn
    a = C.addressof
    X, Q, K, V, ws = 0x10000, 0x20000, 0x30000, 0x40000, 0x50000
    T, d_m, n = 128, 64, 32
    wq, wk, wv = _w(0x1000), _w(0x2000), _w(0x3000)
    wo = _w(0x4000, layout=B.SHARED_ROWS)
    big = 1 << 24
    qk_fwd = f("ecospa_coupled_qk_fwd")
    # null weight descriptor / null output / null weight pointer
    assert qk_fwd(X, d_m, T, d_m, None, a(wk), n, None, None, Q, K, 32, ws, big, None) == 1
    assert qk_fwd(X, d_m, T, d_m, a(wq), a(wk), n, None, None, None, K, 32, ws, big, None) == 1
    assert qk_fwd(X, d_m, T, d_m, a(_w(None)), a(wk), n, None, None, Q, K, 32, ws, big, None) == 1
    # K requested (weight given) without an output for it; sizes < 1; weight of another width or dtype
    assert qk_fwd(X, d_m, T, d_m, a(wq), a(wk), n, None, None, Q, None, 32, ws, big, None) == 1
    assert qk_fwd(X, d_m, 0, d_m, a(wq), a(wk), n, None, None, Q, K, 32, ws, big, None) == 1
    assert qk_fwd(X, d_m, T, d_m, a(wq), a(wk), 0, None, None, Q, K, 32, ws, big, None) == 1
    assert qk_fwd(X, d_m, T, d_m, a(_w(0x1000, d_m=128)), a(wk), n, None, None, Q, K, 32, ws, big, None) == 1
    assert qk_fwd(X, d_m, T, d_m, a(wq), a(_w(0x2000, dtype=B.F32)), n, None, None, Q, K, 32, ws, big, None) == 1
    assert qk_fwd(X, d_m, T, d_m, a(_w(0x1000, ld=16)), a(wk), n, None, None, Q, K, 32, ws, big, None) == 1
    assert qk_fwd(X, d_m, T, d_m, a(_w(0x1000, layout=7)), a(wk), n, None, None, Q, K, 32, ws, big, None) == 1
    # X missing; X narrower than d_m
    assert qk_fwd(None, d_m, T, d_m, a(wq), a(wk), n, None, None, Q, K, 32, ws, big, None) == 1
    assert qk_fwd(X, 32, T, d_m, a(wq), a(wk), n, None, None, Q, K, 32, ws, big, None) == 1
    # alignment: workspace, output pointer, output pitch, X pitch, weight pointer, weight pitch, bias pointer
    assert qk_fwd(X, d_m, T, d_m, a(wq), a(wk), n, None, None, Q, K, 32, ws + 4, big, None) == 2
    assert qk_fwd(X, d_m, T, d_m, a(wq), a(wk), n, None, None, Q + 2, K, 32, ws, big, None) == 2
    assert qk_fwd(X, d_m, T, d_m, a(wq), a(wk), n, None, None, Q, K, 36, ws, big, None) == 2
    assert qk_fwd(X, d_m + 4, T, d_m, a(wq), a(wk), n, None, None, Q, K, 32, ws, big, None) == 2
    assert qk_fwd(X, d_m, T, d_m, a(_w(0x1008)), a(wk), n, None, None, Q, K, 32, ws, big, None) == 2
    assert qk_fwd(X, d_m, T, d_m, a(_w(0x1000, ld=68)), a(wk), n, None, None, Q, K, 32, ws, big, None) == 2
    assert qk_fwd(X, d_m, T, d_m, a(wq), a(wk), n, 0x7002, None, Q, K, 32, ws, big, None) == 2
    # the other forward calls share the checks
    assert f("ecospa_coupled_vo_fwd_v")(X, d_m, T, d_m, None, n, None, V, 32, ws, big, None) == 1
    assert f("ecospa_coupled_vo_fwd_o")(X, 32, T, d_m, a(wo), n, None, None, d_m, ws, big, None) == 1
    assert f("ecospa_coupled_vo_fwd_o")(X, 32, T, d_m, a(_w(0x4000, layout=B.SHARED_ROWS, ld=32)), n, None, Q, d_m, ws, big, None) == 1
    assert f("ecospa_coupled_qkv_fwd")(X, d_m, T, d_m, a(wq), a(wk), None, n, n, None, None, None, Q, K, V, 32, 32, ws, big,
                                       None) == 1
    assert f("ecospa_coupled_qkv_fwd")(X, d_m, T, d_m, a(wq), a(wk), a(wv), n, n, None, None, None, Q, K, V, 32, 36, ws, big,
                                       None) == 2

    # backward calls: missing gradient inputs / outputs, short or missing workspace
    dQ, dK, dX, dWq, dWk, db = 0x60000, 0x70000, 0x80000, 0x90000, 0xA0000, 0xB0000
    qk_bwd = f("ecospa_coupled_qk_bwd")
    assert qk_bwd(X, d_m, T, d_m, a(wq), a(wk), n, None, dK, 32, dX, d_m, 0, dWq, dWk, 32, None, None, ws, big, None) == 1
    assert qk_bwd(X, d_m, T, d_m, a(wq), a(wk), n, dQ, dK, 32, None, d_m, 0, dWq, dWk, 32, None, None, ws, big, None) == 1
    assert qk_bwd(X, d_m, T, d_m, a(wq), a(wk), n, dQ, dK, 32, dX, d_m, 0, dWq, None, 32, None, None, ws, big, None) == 1
    # bias gradients need column-sum scratch: no workspace, or one that is too small -> nothing is launched
    assert qk_bwd(X, d_m, T, d_m, a(wq), a(wk), n, dQ, dK, 32, dX, d_m, 0, dWq, dWk, 32, db, db + 256, None, 0, None) == 6
    assert qk_bwd(X, d_m, T, d_m, a(wq), a(wk), n, dQ, dK, 32, dX, d_m, 0, dWq, dWk, 32, db, db + 256, ws, 64, None) == 6
    need = lib.ecospa_proj_workspace_bytes(T, d_m, n, B.BF16)
    assert need > 0
    # misaligned gradient pitch
    assert qk_bwd(X, d_m, T, d_m, a(wq), a(wk), n, dQ, dK, 36, dX, d_m, 0, dWq, dWk, 32, None, None, ws, big, None) == 2
    vo_bwd_o = f("ecospa_coupled_vo_bwd_o")
    assert vo_bwd_o(None, 32, T, d_m, a(wo), n, dQ, d_m, dK, 32, dWq, d_m, None, ws, big, None) == 1
    assert vo_bwd_o(X, 32, T, d_m, a(wo), n, dQ, d_m, dK, 32, dWq, d_m, db, None, 0, None) == 6
    qkv_bwd = f("ecospa_coupled_qkv_bwd")
    assert qkv_bwd(X, d_m, T, d_m, a(wq), a(wk), a(wv), n, n, dQ, dK, None, 32, 32, dX, d_m, 1, dWq, dWk, dWk + 0x8000, 32,
                   32, None, None, None, ws, big, None) == 1
    assert qkv_bwd(X, d_m, T, d_m, a(wq), a(wk), a(wv), n, n, dQ, dK, dK + 0x8000, 32, 32, dX, d_m, 1, dWq, dWk,
                   dWk + 0x8000, 32, 32, db, db + 256, db + 512, ws, 128, None) == 6

    # fp32 models stage their operands in the workspace: without one the call stops before the first launch
    wq32 = _w(0x1000, dtype=B.F32)
    assert qk_fwd(X, d_m, T, d_m, a(wq32), None, n, None, None, Q, None, 32, None, 0, None) == 6
    assert lib.ecospa_proj_workspace_bytes(T, d_m, n, B.F32) > need


def test_ffn_calls_reject_bad_arguments_without_launching(lib):
    f = B._fn
    a = C.addressof
    X, Y, H, Hb, A, ws = 0x10000, 0x20000, 0x30000, 0x40000, 0x50000, 0x60000
    T, d_m, k = 128, 64, 48
    w1, w1b = _w(0x1000), _w(0x2000)
    w2 = _w(0x3000, layout=B.SHARED_ROWS)
    big = 1 << 24
    fwd = f("ecospa_coupled_ffn_fwd")
    ok_args = lambda act, w1b_, Hb_: (X, d_m, T, d_m, act, a(w1), w1b_, a(w2), k, None, None, Y, d_m, H, Hb_, A, 48, ws, big, None)
    # unknown activation; ACT_NONE is not an FFN; SwiGLU without the up matrix or without its saved tensor
    assert fwd(*ok_args(9, None, None)) == 1
    assert fwd(*ok_args(B.ACT_NONE, None, None)) == 1
    assert fwd(*ok_args(B.ACT_SWIGLU, None, Hb)) == 1
    assert fwd(*ok_args(B.ACT_SWIGLU, a(w1b), None)) == 1
    # saved-activation pitch: smaller than k, or not a multiple of 16 bytes
    assert fwd(X, d_m, T, d_m, B.ACT_GELU_ERF, a(w1), None, a(w2), k, None, None, Y, d_m, H, None, A, 40, ws, big, None) == 1
    assert fwd(X, d_m, T, d_m, B.ACT_GELU_ERF, a(w1), None, a(w2), k, None, None, Y, d_m, H, None, A, 50, ws, big, None) == 2
    # null outputs
    assert fwd(X, d_m, T, d_m, B.ACT_GELU_ERF, a(w1), None, a(w2), k, None, None, None, d_m, H, None, A, 48, ws, big, None) == 1
    assert fwd(X, d_m, T, d_m, B.ACT_GELU_ERF, a(w1), None, a(w2), k, None, None, Y, d_m, None, None, A, 48, ws, big, None) == 1
    # misaligned output
    assert fwd(X, d_m, T, d_m, B.ACT_GELU_ERF, a(w1), None, a(w2), k, None, None, Y + 8, d_m, H, None, A, 48, ws, big, None) == 2
    bwd = f("ecospa_coupled_ffn_bwd")
    dY, dX, dW1, dW2, db = 0x70000, 0x80000, 0x90000, 0xA0000, 0xB0000
    # the backward pass always needs scratch for dH: none, or too little
    assert bwd(X, d_m, T, d_m, B.ACT_GELU_ERF, a(w1), None, a(w2), k, H, None, A, 48, dY, d_m, dX, d_m, dW1, None, 48, dW2,
               d_m, None, None, None, 0, None) == 6
    assert bwd(X, d_m, T, d_m, B.ACT_GELU_ERF, a(w1), None, a(w2), k, H, None, A, 48, dY, d_m, dX, d_m, dW1, None, 48, dW2,
               d_m, db, db + 256, ws, 1024, None) == 6
    assert bwd(X, d_m, T, d_m, B.ACT_SWIGLU, a(w1), a(w1b), a(w2), k, H, Hb, A, 48, dY, d_m, dX, d_m, dW1, None, 48, dW2,
               d_m, None, None, ws, big, None) == 1          # SwiGLU without an output for dW_up
    assert bwd(X, d_m, T, d_m, B.ACT_GELU_ERF, a(w1), None, a(w2), k, H, None, A, 48, None, d_m, dX, d_m, dW1, None, 48, dW2,
               d_m, None, None, ws, big, None) == 1
    assert lib.ecospa_ffn_workspace_bytes(T, d_m, k, B.ACT_SWIGLU, B.BF16) > lib.ecospa_ffn_workspace_bytes(
        T, d_m, k, B.ACT_GELU_ERF, B.BF16) > 0


def test_wait_limit_setter(lib):
    fn = lib.ecospa_set_device_wait_limit_ns
    fn.restype = C.c_int
    fn.argtypes = [C.c_uint64]
    assert fn(0) == 1
    assert fn(2_000_000_000) == 0


def test_shared_dimension_limit(lib):
    null = B.Mat(None, 0, 0, 0, 0)
    D = (1 << 22) + 64
    p = B.Pair(B.PAIR_PLAIN, 1, D, 0, _fake_mat(0x1000, dtype=B.F32, other=4, ld=D), null,
               _fake_mat(0x40000000, dtype=B.F32, layout=B.SHARED_ROWS, other=4, ld=4), null, null, null)
    assert lib.ecospa_score_pairs(C.addressof((B.Pair * 1)(p)), 1, 1.0, C.c_void_p(0x3000), None, None,
                                  C.c_void_p(0x4000), 1 << 30, None) == 3
    g = B.Gather(_fake_mat(0x10000, other=2, ld=D), _fake_mat(0x80000000, other=2, ld=64), 0x9000, 32, D)
    assert lib.ecospa_compact_tensors(C.addressof((B.Gather * 1)(g)), 1, None) == 3


def test_grouped_pairs_are_validated_on_the_host(lib):
    null = B.Mat(None, 0, 0, 0, 0)
    ups, ws = C.c_void_p(0x3000), C.c_void_p(0x4000)
    wq = _fake_mat(0x100000, other=64, ld=256)                 # 4 query heads of 64 side by side
    wk = _fake_mat(0x200000, other=64, ld=64)
    ok = B.Pair(B.PAIR_PLAIN, 1, 64, 0, wq, null, wk, null, null, null, 4, 1)
    assert lib.ecospa_score_workspace_bytes(C.addressof((B.Pair * 1)(ok)), 1) > 0
    # the stacked side must cover rep * D shared indices
    short = B.Pair(B.PAIR_PLAIN, 1, 64, 0, _fake_mat(0x100000, other=64, ld=128), null, wk, null, null, null, 4, 1)
    assert lib.ecospa_score_pairs(C.addressof((B.Pair * 1)(short)), 1, 1.0, ups, None, None, ws, 1 << 24, None) == 1
    # grouped heads with rotation pairs or with a gated FFN pair are not defined
    rope = B.Pair(B.PAIR_PLAIN, 1, 64, 1, wq, null, wk, null, null, null, 4, 1)
    assert lib.ecospa_score_pairs(C.addressof((B.Pair * 1)(rope)), 1, 1.0, ups, None, None, ws, 1 << 24, None) == 1
    sw = B.Pair(B.PAIR_SWIGLU, 1, 64, 0, wq, wq, wk, null, null, null, 4, 1)
    assert lib.ecospa_score_pairs(C.addressof((B.Pair * 1)(sw)), 1, 1.0, ups, None, None, ws, 1 << 24, None) == 1
    neg = B.Pair(B.PAIR_PLAIN, 1, 64, 0, wq, null, wk, null, null, null, -2, 1)
    assert lib.ecospa_score_pairs(C.addressof((B.Pair * 1)(neg)), 1, 1.0, ups, None, None, ws, 1 << 24, None) == 1


def test_in_place_compaction_rejects_jobs_that_are_not_in_place(lib):
    fn = lib.ecospa_compact_tensors_inplace
    fn.restype = C.c_int
    fn.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
    kept = 0x9000
    m = _fake_mat(0x10000, other=8, ld=64)
    ok_shape = B.Gather(m, _fake_mat(0x20000, other=8, ld=64), kept, 32, 64)          # another buffer
    assert fn(C.addressof((B.Gather * 1)(ok_shape)), 1, None) == 1
    other_pitch = B.Gather(m, _fake_mat(0x10000, other=8, ld=32), kept, 32, 64)       # same base, other pitch
    assert fn(C.addressof((B.Gather * 1)(other_pitch)), 1, None) == 1
    assert fn(None, 1, None) == 1
    too_many = B.Gather(m, m, kept, 65, 64)
    assert fn(C.addressof((B.Gather * 1)(too_many)), 1, None) == 1


def test_algorithm1_pass_rejects_bad_arguments_without_launching(lib):
    null = B.Mat(None, 0, 0, 0, 0)
    w1 = _fake_mat(0x10000, ld=128)
    w2 = _fake_mat(0x20000, layout=B.SHARED_ROWS)
    g1 = _fake_mat(0x30000, ld=128)
    g2 = _fake_mat(0x40000, layout=B.SHARED_ROWS)
    widths = (C.c_int32 * 2)(64, 64)

    def grp(w1=w1, w2=w2, g1=g1, g2=g2, n_pairs=2, wptr=C.addressof(widths), n_aux=0, aux=None):
        return B.Group(w1, null, w2, g1, null, g2, aux, n_aux, n_pairs, wptr, 0, 0)

    def arr(g):
        a = (B.Group * 1)(g)
        return a, C.addressof(a)

    size = lib.ecospa_alg1_workspace_bytes
    size.restype, size.argtypes = C.c_size_t, [C.c_void_p, C.c_int32]
    plan = lib.ecospa_alg1_plan
    plan.restype = C.c_int
    plan.argtypes = [C.c_void_p, C.c_int32, C.c_double, C.c_int32, C.c_double, C.c_int32, C.c_int32, C.c_void_p, C.c_size_t,
                     C.c_void_p, C.c_void_p]
    apply_ = lib.ecospa_alg1_apply
    apply_.restype = C.c_int
    apply_.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t, C.c_void_p]
    offs = lib.ecospa_alg1_offsets
    offs.restype, offs.argtypes = C.c_int, [C.c_void_p, C.c_int32, C.c_void_p]

    keep, good = arr(grp())
    need = size(good, 1)
    assert need > 6 * 128 * 4 and need % 256 == 0
    out6 = (C.c_int64 * 6)()
    assert offs(good, 1, C.addressof(out6)) == 0 and out6[4] == 128 and out6[5] == 2 and out6[0] == 0
    assert offs(good, 1, None) == 1
    k = (C.c_int32 * 2)(32, 32)
    ws = 0x100000
    # no groups / no counts / negative pair count to choose
    assert plan(None, 1, 8.0, 1, 0.5, 1, 1, ws, need, C.addressof(k), None) == 1
    assert plan(good, 1, 8.0, 1, 0.5, 1, 1, ws, need, None, None) == 1
    assert plan(good, 1, 8.0, -1, 0.5, 1, 1, ws, need, C.addressof(k), None) == 1
    # importance needs the gradients
    kp, nograd = arr(grp(g1=null))
    assert plan(nograd, 1, 8.0, 1, 0.5, 1, 1, ws, need, C.addressof(k), None) == 1
    # a group without widths, with a negative width, with aux announced but absent
    kp, bad = arr(grp(wptr=None))
    assert size(bad, 1) == 0 and plan(bad, 1, 8.0, 1, 0.5, 1, 1, ws, need, C.addressof(k), None) == 1
    neg = (C.c_int32 * 2)(64, -1)
    kp, bad = arr(grp(wptr=C.addressof(neg)))
    assert size(bad, 1) == 0
    kp, bad = arr(grp(n_aux=1))
    assert size(bad, 1) == 0
    # every pair empty: nothing to describe
    zero = (C.c_int32 * 2)(0, 0)
    kp, bad = arr(grp(wptr=C.addressof(zero)))
    assert size(bad, 1) == 0
    # workspace too small / absent / misaligned
    assert plan(good, 1, 8.0, 1, 0.5, 1, 1, ws, need - 1, C.addressof(k), None) != 0
    assert plan(good, 1, 8.0, 1, 0.5, 1, 1, None, need, C.addressof(k), None) != 0
    assert plan(good, 1, 8.0, 1, 0.5, 1, 1, ws + 4, need, C.addressof(k), None) != 0
    # apply: out of place without outputs, counts larger than the pair, workspace too small
    assert apply_(good, 1, C.addressof(k), None, 0, ws, need, None) == 1
    big = (C.c_int32 * 2)(65, 1)
    assert apply_(good, 1, C.addressof(big), None, 1, ws, need, None) == 1
    assert apply_(good, 1, C.addressof(k), None, 1, ws, need - 1, None) != 0
    assert apply_(good, 1, None, None, 1, ws, need, None) == 1


def test_attention_calls_reject_bad_arguments_without_launching(lib):
    fwd = lib.ecospa_coupled_attn_fwd
    fwd.restype = C.c_int
    fwd.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_float,
                    C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
    bwd = lib.ecospa_coupled_attn_bwd
    bwd.restype = C.c_int
    bwd.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64,
                    C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_float, C.c_int32, C.c_void_p, C.c_void_p, C.c_int64,
                    C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p]
    wsb = lib.ecospa_attn_workspace_bytes
    wsb.restype, wsb.argtypes = C.c_size_t, [C.c_int64, C.c_int64, C.c_int32]
    assert wsb(2, 128, 4) >= 2 * 128 * 4 * 4 and wsb(0, 128, 4) == 0 and wsb(2, 0, 4) == 0 and wsb(2, 128, 0) == 0
    Q, K, V, Ctx, lse = 0x10000, 0x20000, 0x30000, 0x40000, 0x50000

    def f(hd, q=Q, k=K, ld_qk=64, v=V, ld_v=64, batch=2, seq=128, scale=0.125, ctx=Ctx, ld_ctx=64, l=lse):
        return fwd(q, k, ld_qk, v, ld_v, batch, seq, C.addressof(hd) if hd is not None else None, scale, 0, ctx, ld_ctx, l, None)

    good = B.heads([0, 32], [32, 32], [0, 32], [32, 32])
    # every check below fails before the first CUDA call; the good descriptor itself is used for the pointer / pitch cases
    assert f(None) == 1
    assert f(B.heads([0, 32], [32, 24], [0, 32], [32, 32])) == 2          # width not a multiple of 16
    assert f(B.heads([0, 36], [32, 32], [0, 32], [32, 32])) == 2          # offset not a multiple of 8
    assert f(B.heads([0, 32], [32, 144], [0, 32], [32, 32])) == 3         # wider than 128
    assert f(B.heads([0, 32], [32, 0], [0, 32], [32, 32])) == 1
    assert f(B.heads([0, -8], [32, 32], [0, 32], [32, 32])) == 1
    assert f(B.heads(list(range(0, 16 * 129, 16)), [16] * 129, list(range(0, 16 * 129, 16)), [16] * 129), ld_qk=4096, ld_v=4096, ld_ctx=4096) == 3
    assert f(good, batch=0) == 1 and f(good, seq=0) == 1 and f(good, l=None) == 1
    assert f(good, scale=0.0) == 1 and f(good, scale=float("nan")) == 1 and f(good, scale=-1.0) == 1
    assert f(good, q=None) == 1 and f(good, ctx=None) == 1
    assert f(good, ld_qk=60) == 1                                         # pitch smaller than the heads' columns
    assert f(good, ld_v=68) == 2 and f(good, q=Q + 2) == 2 and f(good, l=lse + 2) == 2
    # grouped-query descriptors
    assert f(B.heads([0, 32, 64], [32] * 3, [0, 32, 64], [32] * 3, k_off=[0, 32], v_off=[0, 32]), ld_qk=96, ld_v=96, ld_ctx=96) == 1   # 3 % 2
    assert f(B.heads([0, 32], [32, 16], [0, 32], [32, 32], k_off=[0], v_off=[0])) == 1     # widths differ inside a group
    assert f(B.heads([0, 32], [32, 32], [0, 32], [32, 32], k_off=[4], v_off=[0])) == 2
    h = B.heads([0, 32], [32, 32], [0, 32], [32, 32], k_off=[0], v_off=[0])
    h.k_off = None
    assert f(h) == 1
    h = B.heads([0, 32], [32, 32], [0, 32], [32, 32])
    h.n_kv_heads = -1
    assert f(h) == 1

    def g(hd, ws=0x90000, ws_bytes=1 << 20, dq=0x60000, dk=0x70000, dv=0x80000, ld_dqk=64, ld_dv=64, dctx=0xa0000):
        return bwd(Q, K, 64, V, 64, Ctx, 64, dctx, 64, lse, 2, 128, C.addressof(hd), 0.125, 1, dq, dk, ld_dqk, dv, ld_dv, ws, ws_bytes, None)

    assert g(good, ws=None) == 6 and g(good, ws_bytes=16) == 6 and g(good, ws=0x90004) == 2
    assert g(good, dq=None) == 1 and g(good, dctx=None) == 1 and g(good, ld_dqk=62) == 1 and g(good, ld_dv=68) == 2
