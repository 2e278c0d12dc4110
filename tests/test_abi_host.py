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
