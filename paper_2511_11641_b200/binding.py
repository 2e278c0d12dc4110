"""Thin ctypes binding of libecospa: argument marshalling only.

Every function has the name of the C entry point it calls (without the ``ecospa_``
prefix where that reads better in Python is NOT done: names are kept identical).
torch supplies device memory and the current stream; every step runs in the CUDA
kernels of the shared library.  There is no CPU fallback: if the library is missing
or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libecospa.so")

F32, BF16 = 0, 1
SHARED_COLS, SHARED_ROWS = 0, 1
PAIR_PLAIN, PAIR_SWIGLU = 0, 1
ACT_NONE, ACT_GELU_ERF, ACT_GELU_TANH, ACT_SWIGLU = 0, 1, 2, 3
ROPE_NONE, ROPE_INTERLEAVED, ROPE_HALF = 0, 1, 2


class EcospaError(RuntimeError):
    def __init__(self, status: int, where: str):
        l = lib()
        msg = l.ecospa_status_string(status).decode()
        cuda = l.ecospa_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} (status {status})" + (f" [{cuda}]" if status in (3, 4) and cuda else ""))
        self.status = status


class Mat(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("dtype", C.c_int32), ("layout", C.c_int32),
                ("other_dim", C.c_int64), ("ld", C.c_int64)]


class Pair(C.Structure):
    _fields_ = [("kind", C.c_int32), ("n_seg", C.c_int32), ("seg_len", C.c_int32), ("rope", C.c_int32),
                ("w1", Mat), ("w1b", Mat), ("w2", Mat), ("g1", Mat), ("g1b", Mat), ("g2", Mat),
                ("w1_rep", C.c_int32), ("w2_rep", C.c_int32)]


class Gather(C.Structure):
    _fields_ = [("in_", Mat), ("out", Mat), ("kept", C.c_void_p), ("n_kept", C.c_int32), ("shared_dim", C.c_int32)]


_lib = None


def lib() -> C.CDLL:
    """Load libecospa.so (built in-tree by build.py); raises if it is not there."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_2511_11641_b200.build` (needs nvcc)")
        l = C.CDLL(LIB_PATH)
        l.ecospa_status_string.restype = C.c_char_p
        l.ecospa_status_string.argtypes = [C.c_int]
        l.ecospa_last_cuda_error.restype = C.c_char_p
        l.ecospa_score_workspace_bytes.restype = C.c_size_t
        l.ecospa_score_workspace_bytes.argtypes = [C.c_void_p, C.c_int32]
        l.ecospa_score_pairs.restype = C.c_int
        l.ecospa_score_pairs.argtypes = [C.c_void_p, C.c_int32, C.c_double, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_size_t, C.c_void_p]
        l.ecospa_select_aligned_topk.restype = C.c_int
        l.ecospa_select_aligned_topk.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                                 C.c_void_p, C.c_void_p, C.c_void_p]
        l.ecospa_compact_tensors.restype = C.c_int
        l.ecospa_compact_tensors.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
        l.ecospa_compact_pair.restype = C.c_int
        l.ecospa_compact_pair.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32,
                                          C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib = l
    return _lib


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def mat(t: Optional[torch.Tensor], layout: int) -> Mat:
    """Descriptor of a row-major 2-D tensor (or a 1-D vector over the shared axis)."""
    if t is None:
        return Mat(None, 0, 0, 0, 0)
    if t.dim() == 1:
        assert t.stride(0) == 1
        return Mat(t.data_ptr(), _dtype_code(t), SHARED_COLS, 1, t.numel())
    assert t.dim() == 2 and t.stride(1) == 1, "row-major tensors only"
    other = t.shape[0] if layout == SHARED_COLS else t.shape[1]
    return Mat(t.data_ptr(), _dtype_code(t), layout, other, t.stride(0))


def pair(kind: int, n_seg: int, seg_len: int, w1, w2, layout1: int, layout2: int, w1b=None,
         g1=None, g2=None, g1b=None, rope: int = 0, w1_rep: int = 1, w2_rep: int = 1) -> Pair:
    """w1_rep / w2_rep > 1: grouped-query attention, that many heads per segment stacked on the W_1 / W_2 side."""
    p = Pair(kind, n_seg, seg_len, rope, mat(w1, layout1), mat(w1b, layout1), mat(w2, layout2),
             mat(g1, layout1), mat(g1b, layout1), mat(g2, layout2), w1_rep, w2_rep)
    p._keep = (w1, w2, w1b, g1, g2, g1b)   # keep the tensors alive as long as the descriptor
    return p


def _pair_array(pairs: Sequence[Pair]):
    arr = (Pair * len(pairs))(*pairs)
    return arr


def ecospa_score_workspace_bytes(pairs: Sequence[Pair]) -> int:
    arr = _pair_array(pairs)
    return int(lib().ecospa_score_workspace_bytes(C.addressof(arr), len(pairs)))


def ecospa_score_pairs(pairs: Sequence[Pair], n_samples: float, upsilon: torch.Tensor,
                       raw: Optional[torch.Tensor] = None, fisher: Optional[torch.Tensor] = None,
                       workspace: Optional[torch.Tensor] = None, stream=None) -> None:
    """upsilon/raw: fp32 [sum D]; fisher: fp32 [sum n_seg] or None; workspace: uint8 device buffer."""
    arr = _pair_array(pairs)
    if workspace is None:
        workspace = torch.empty(ecospa_score_workspace_bytes(pairs), dtype=torch.uint8, device=upsilon.device)
    st = lib().ecospa_score_pairs(C.addressof(arr), len(pairs), float(n_samples), _ptr(upsilon), _ptr(raw),
                                  _ptr(fisher), _ptr(workspace), workspace.numel(), _stream(stream))
    if st != 0:
        raise EcospaError(st, "ecospa_score_pairs")


def ecospa_score_pair_static_max_bytes() -> int:
    f = lib().ecospa_score_pair_static_max_bytes
    f.restype = C.c_size_t
    return int(f())


def ecospa_score_pair_static(p: Pair, n_samples: float, upsilon: torch.Tensor, raw: Optional[torch.Tensor] = None,
                             fisher: Optional[torch.Tensor] = None, stream=None) -> None:
    """Scores of one pair group using the library's built-in scratch array; allocates nothing."""
    f = lib().ecospa_score_pair_static
    f.restype = C.c_int
    f.argtypes = [C.c_void_p, C.c_double, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    st = f(C.addressof(p), float(n_samples), _ptr(upsilon), _ptr(raw), _ptr(fisher), _stream(stream))
    if st != 0:
        raise EcospaError(st, "ecospa_score_pair_static")


def ecospa_select_aligned_topk(upsilon: torch.Tensor, n_seg: Sequence[int], seg_len: Sequence[int],
                               k_per_seg: Sequence[int], kept: torch.Tensor,
                               seg_offsets: Optional[torch.Tensor] = None, stream=None) -> None:
    n_pairs = len(n_seg)
    a_nseg = (C.c_int32 * n_pairs)(*n_seg)
    a_slen = (C.c_int32 * n_pairs)(*seg_len)
    a_k = (C.c_int32 * len(k_per_seg))(*k_per_seg)
    assert len(k_per_seg) == sum(n_seg)
    assert kept.dtype == torch.int32 and kept.numel() >= sum(k_per_seg)
    st = lib().ecospa_select_aligned_topk(_ptr(upsilon), C.addressof(a_nseg), C.addressof(a_slen), C.addressof(a_k),
                                          n_pairs, _ptr(kept), _ptr(seg_offsets), _stream(stream))
    if st != 0:
        raise EcospaError(st, "ecospa_select_aligned_topk")


def ecospa_select_rotation_pairs(upsilon: torch.Tensor, n_seg: Sequence[int], seg_len: Sequence[int],
                                 k_per_seg: Sequence[int], rope: Sequence[int], kept: torch.Tensor,
                                 seg_offsets: Optional[torch.Tensor] = None, stream=None) -> None:
    n_pairs = len(n_seg)
    a_nseg = (C.c_int32 * n_pairs)(*n_seg)
    a_slen = (C.c_int32 * n_pairs)(*seg_len)
    a_rope = (C.c_int32 * n_pairs)(*rope)
    a_k = (C.c_int32 * len(k_per_seg))(*k_per_seg)
    assert len(k_per_seg) == sum(n_seg) and len(rope) == n_pairs
    assert kept.dtype == torch.int32 and kept.numel() >= sum(k_per_seg)
    fn = lib().ecospa_select_rotation_pairs
    fn.restype = C.c_int
    fn.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    st = fn(_ptr(upsilon), C.addressof(a_nseg), C.addressof(a_slen), C.addressof(a_k), C.addressof(a_rope), n_pairs,
            _ptr(kept), _ptr(seg_offsets), _stream(stream))
    if st != 0:
        raise EcospaError(st, "ecospa_select_rotation_pairs")


def ecospa_pack_kept(slots: torch.Tensor, src: Sequence[int], dst: Sequence[int], k: Sequence[int], add: Sequence[int],
                     out: torch.Tensor, stream=None) -> None:
    n = len(src)
    assert len(dst) == n and len(k) == n and len(add) == n and slots.dtype == torch.int32 and out.dtype == torch.int32
    arr = lambda v: (C.c_int32 * n)(*v)
    a_src, a_dst, a_k, a_add = arr(src), arr(dst), arr(k), arr(add)
    fn = lib().ecospa_pack_kept
    fn.restype = C.c_int
    fn.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
    st = fn(_ptr(slots), C.addressof(a_src), C.addressof(a_dst), C.addressof(a_k), C.addressof(a_add), n, _ptr(out),
            _stream(stream))
    if st != 0:
        raise EcospaError(st, "ecospa_pack_kept")


def ecospa_choose_pairs(fisher: torch.Tensor, m: int, chosen: torch.Tensor, stream=None) -> None:
    assert fisher.dtype == torch.float32 and chosen.dtype == torch.int32 and chosen.numel() >= fisher.numel()
    fn = lib().ecospa_choose_pairs
    fn.restype = C.c_int
    fn.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
    st = fn(_ptr(fisher), fisher.numel(), int(m), _ptr(chosen), _stream(stream))
    if st != 0:
        raise EcospaError(st, "ecospa_choose_pairs")


def ecospa_select_aligned_threshold(upsilon: torch.Tensor, n_seg: Sequence[int], seg_len: Sequence[int], theta: float,
                                    kept: torch.Tensor, k_out: torch.Tensor, l1: bool = True, k_min: int = 1,
                                    chosen: Optional[torch.Tensor] = None, rope: Optional[Sequence[int]] = None,
                                    stream=None) -> None:
    n_pairs = len(n_seg)
    a_nseg = (C.c_int32 * n_pairs)(*n_seg)
    a_slen = (C.c_int32 * n_pairs)(*seg_len)
    a_rope = (C.c_int32 * n_pairs)(*rope) if rope is not None else None
    assert kept.dtype == torch.int32 and kept.numel() >= sum(a * b for a, b in zip(n_seg, seg_len))
    assert k_out.dtype == torch.int32 and k_out.numel() >= sum(n_seg)
    fn = lib().ecospa_select_aligned_threshold
    fn.restype = C.c_int
    fn.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_double, C.c_int32, C.c_int32, C.c_void_p,
                   C.c_void_p, C.c_void_p, C.c_void_p]
    st = fn(_ptr(upsilon), C.addressof(a_nseg), C.addressof(a_slen), C.addressof(a_rope) if a_rope is not None else None,
            n_pairs, float(theta), int(bool(l1)), int(k_min), _ptr(chosen), _ptr(kept), _ptr(k_out), _stream(stream))
    if st != 0:
        raise EcospaError(st, "ecospa_select_aligned_threshold")


def gather(inp: torch.Tensor, out: torch.Tensor, layout: int, kept: torch.Tensor, n_kept: int, shared_dim: int) -> Gather:
    g = Gather(mat(inp, layout), mat(out, layout), kept.data_ptr(), n_kept, shared_dim)
    g._keep = (inp, out, kept)
    return g


def ecospa_compact_tensors(jobs: Sequence[Gather], stream=None) -> None:
    arr = (Gather * len(jobs))(*jobs)
    st = lib().ecospa_compact_tensors(C.addressof(arr), len(jobs), _stream(stream))
    if st != 0:
        raise EcospaError(st, "ecospa_compact_tensors")


def ecospa_compact_tensors_inplace(jobs: Sequence[Gather], stream=None) -> None:
    """Jobs whose output is their input (same pointer and pitch): the kept part moves to the front."""
    arr = (Gather * len(jobs))(*jobs)
    fn = lib().ecospa_compact_tensors_inplace
    fn.restype = C.c_int
    fn.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
    st = fn(C.addressof(arr), len(jobs), _stream(stream))
    if st != 0:
        raise EcospaError(st, "ecospa_compact_tensors_inplace")


def ecospa_compact_pair(p: Pair, kept: torch.Tensor, n_kept: int, w1_out: torch.Tensor, w2_out: torch.Tensor,
                        w1b_out: Optional[torch.Tensor] = None,
                        aux: Sequence[Tuple[torch.Tensor, torch.Tensor, int]] = (), stream=None) -> None:
    """aux: (in, out, layout) triples compacted with the same kept list (bias, grads, optimizer moments)."""
    n_aux = len(aux)
    a_in = (Mat * max(1, n_aux))(*[mat(a[0], a[2]) for a in aux])
    a_out = (Mat * max(1, n_aux))(*[mat(a[1], a[2]) for a in aux])
    m1 = mat(w1_out, p.w1.layout)
    m1b = mat(w1b_out, p.w1.layout) if w1b_out is not None else None
    m2 = mat(w2_out, p.w2.layout)
    st = lib().ecospa_compact_pair(C.addressof(p), _ptr(kept), n_kept, C.addressof(a_in), C.addressof(a_out), n_aux,
                                   C.addressof(m1), C.addressof(m1b) if m1b is not None else None, C.addressof(m2),
                                   _stream(stream))
    if st != 0:
        raise EcospaError(st, "ecospa_compact_pair")


# ---------------------------------------------------------------------------------------------
# compacted-pair forward / backward
# ---------------------------------------------------------------------------------------------

_LAYER_SIGS = {
    "ecospa_proj_workspace_bytes": (C.c_size_t, [C.c_int64, C.c_int64, C.c_int64, C.c_int32]),
    "ecospa_ffn_workspace_bytes": (C.c_size_t, [C.c_int64, C.c_int64, C.c_int64, C.c_int32, C.c_int32]),
    "ecospa_coupled_qk_fwd": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_int64,
                                        C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                        C.c_void_p, C.c_size_t, C.c_void_p]),
    "ecospa_coupled_qk_bwd": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_int64,
                                        C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_int32,
                                        C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_size_t, C.c_void_p]),
    "ecospa_coupled_vo_fwd_v": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p,
                                          C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p]),
    "ecospa_coupled_vo_fwd_o": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p,
                                          C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p]),
    "ecospa_coupled_vo_bwd": (C.c_int, [C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_int64, C.c_int64,
                                        C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64,
                                        C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64,
                                        C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "ecospa_coupled_ffn_fwd": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                         C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p]),
    "ecospa_coupled_ffn_bwd": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                         C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_int64,
                                         C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "ecospa_coupled_qkv_fwd": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p]),
    "ecospa_coupled_qkv_bwd": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64,
                                         C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                         C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "ecospa_coupled_vo_bwd_o": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p,
                                          C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p,
                                          C.c_void_p, C.c_size_t, C.c_void_p]),
    "ecospa_coupled_vo_bwd_v": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p,
                                          C.c_int64, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p,
                                          C.c_void_p, C.c_size_t, C.c_void_p]),
    "ecospa_device_status": (C.c_int, [C.c_void_p, C.c_void_p]),
}
_sigs_done = False


def _fn(name: str):
    global _sigs_done
    l = lib()
    if not _sigs_done:
        for n, (res, args) in _LAYER_SIGS.items():
            f = getattr(l, n)
            f.restype, f.argtypes = res, args
        _sigs_done = True
    return getattr(l, name)


def _ws(ws: Optional[torch.Tensor]):
    return (None, 0) if ws is None else (ws.data_ptr(), ws.numel() * ws.element_size())


def _ref(m: Optional[Mat]):
    return None if m is None else C.addressof(m)


def _check(st: int, where: str) -> None:
    if st != 0:
        raise EcospaError(st, where)


def ecospa_proj_workspace_bytes(T: int, d_m: int, n: int, dtype: int) -> int:
    return int(_fn("ecospa_proj_workspace_bytes")(T, d_m, n, dtype))


def ecospa_ffn_workspace_bytes(T: int, d_m: int, k: int, act: int, dtype: int) -> int:
    return int(_fn("ecospa_ffn_workspace_bytes")(T, d_m, k, act, dtype))


# Layer calls.  Weights may be stored in either orientation: `w_in_layout` is the orientation of W_Q, W_K, W_V, W_1,
# W_gate, W_up (default SHARED_COLS = d_m x n; SHARED_ROWS = n x d_m, the nn.Linear layout of those weights),
# `w_out_layout` that of W_O, W_2, W_down (default SHARED_ROWS = n x d_m; SHARED_COLS = d_m x n, their nn.Linear
# layout).  Weight gradients are written in the orientation of their weight.
def ecospa_coupled_qk_fwd(X, wq_c, wk_c, n: int, Qc, Kc, bq_c=None, bk_c=None, workspace=None, stream=None,
        w_in_layout: int = SHARED_COLS, w_out_layout: int = SHARED_ROWS) -> None:
    """wq_c / wk_c: compacted weight buffers of shape (d_m, pitch); Qc / Kc: (T, pitch_out)."""
    T, d_m = X.shape
    mq = mat(wq_c, w_in_layout)
    mk = mat(wk_c, w_in_layout) if wk_c is not None else None
    wp, wb = _ws(workspace)
    _check(_fn("ecospa_coupled_qk_fwd")(X.data_ptr(), X.stride(0), T, d_m, _ref(mq), _ref(mk), n, _ptr(bq_c), _ptr(bk_c),
                                        Qc.data_ptr(), _ptr(Kc), Qc.stride(0), wp, wb, _stream(stream)),
           "ecospa_coupled_qk_fwd")


def ecospa_coupled_qk_bwd(X, wq_c, wk_c, n: int, dQc, dKc, dX, dWq_c, dWk_c, dbq_c=None, dbk_c=None,
                          accumulate_dX: bool = False, workspace=None, stream=None,
        w_in_layout: int = SHARED_COLS, w_out_layout: int = SHARED_ROWS) -> None:
    T, d_m = X.shape
    mq = mat(wq_c, w_in_layout)
    mk = mat(wk_c, w_in_layout) if wk_c is not None else None
    wp, wb = _ws(workspace)
    _check(_fn("ecospa_coupled_qk_bwd")(X.data_ptr(), X.stride(0), T, d_m, _ref(mq), _ref(mk), n, dQc.data_ptr(), _ptr(dKc),
                                        dQc.stride(0), dX.data_ptr(), dX.stride(0), int(accumulate_dX), dWq_c.data_ptr(),
                                        _ptr(dWk_c), dWq_c.stride(0), _ptr(dbq_c), _ptr(dbk_c), wp, wb, _stream(stream)),
           "ecospa_coupled_qk_bwd")


def ecospa_coupled_vo_fwd_v(X, wv_c, n: int, Vc, bv_c=None, workspace=None, stream=None,
        w_in_layout: int = SHARED_COLS, w_out_layout: int = SHARED_ROWS) -> None:
    T, d_m = X.shape
    mv = mat(wv_c, w_in_layout)
    wp, wb = _ws(workspace)
    _check(_fn("ecospa_coupled_vo_fwd_v")(X.data_ptr(), X.stride(0), T, d_m, _ref(mv), n, _ptr(bv_c), Vc.data_ptr(),
                                          Vc.stride(0), wp, wb, _stream(stream)), "ecospa_coupled_vo_fwd_v")


def ecospa_coupled_vo_fwd_o(Ctx, wo_c, n: int, Out, bo=None, workspace=None, stream=None,
        w_in_layout: int = SHARED_COLS, w_out_layout: int = SHARED_ROWS) -> None:
    T = Ctx.shape[0]
    d_m = wo_c.shape[1] if w_out_layout == SHARED_ROWS else wo_c.shape[0]
    mo = mat(wo_c, w_out_layout)
    wp, wb = _ws(workspace)
    _check(_fn("ecospa_coupled_vo_fwd_o")(Ctx.data_ptr(), Ctx.stride(0), T, d_m, _ref(mo), n, _ptr(bo), Out.data_ptr(),
                                          Out.stride(0), wp, wb, _stream(stream)), "ecospa_coupled_vo_fwd_o")


def ecospa_coupled_vo_bwd(X, Ctx, wv_c, wo_c, n: int, dVc, dOut, dX, dCtx, dWv_c, dWo_c, dbv_c=None, dbo=None,
                          accumulate_dX: bool = False, workspace=None, stream=None,
        w_in_layout: int = SHARED_COLS, w_out_layout: int = SHARED_ROWS) -> None:
    T, d_m = X.shape
    mv, mo = mat(wv_c, w_in_layout), mat(wo_c, w_out_layout)
    wp, wb = _ws(workspace)
    _check(_fn("ecospa_coupled_vo_bwd")(X.data_ptr(), X.stride(0), Ctx.data_ptr(), Ctx.stride(0), T, d_m, _ref(mv), _ref(mo),
                                        n, dVc.data_ptr(), dVc.stride(0), dOut.data_ptr(), dOut.stride(0), dX.data_ptr(),
                                        dX.stride(0), int(accumulate_dX), dCtx.data_ptr(), dCtx.stride(0), dWv_c.data_ptr(),
                                        dWv_c.stride(0), dWo_c.data_ptr(), dWo_c.stride(0), _ptr(dbv_c), _ptr(dbo), wp, wb,
                                        _stream(stream)), "ecospa_coupled_vo_bwd")


def ecospa_coupled_qkv_fwd(X, wq_c, wk_c, wv_c, n_qk: int, n_vo: int, Qc, Kc, Vc, bq_c=None, bk_c=None, bv_c=None,
                           workspace=None, stream=None,
        w_in_layout: int = SHARED_COLS, w_out_layout: int = SHARED_ROWS) -> None:
    T, d_m = X.shape
    mq, mk, mv = mat(wq_c, w_in_layout), mat(wk_c, w_in_layout), mat(wv_c, w_in_layout)
    wp, wb = _ws(workspace)
    _check(_fn("ecospa_coupled_qkv_fwd")(X.data_ptr(), X.stride(0), T, d_m, _ref(mq), _ref(mk), _ref(mv), n_qk, n_vo,
                                         _ptr(bq_c), _ptr(bk_c), _ptr(bv_c), Qc.data_ptr(), Kc.data_ptr(), Vc.data_ptr(),
                                         Qc.stride(0), Vc.stride(0), wp, wb, _stream(stream)), "ecospa_coupled_qkv_fwd")


def ecospa_coupled_qkv_bwd(X, wq_c, wk_c, wv_c, n_qk: int, n_vo: int, dQc, dKc, dVc, dX, dWq_c, dWk_c, dWv_c,
                           dbq_c=None, dbk_c=None, dbv_c=None, accumulate_dX: bool = False, workspace=None, stream=None,
        w_in_layout: int = SHARED_COLS, w_out_layout: int = SHARED_ROWS) -> None:
    T, d_m = X.shape
    mq, mk, mv = mat(wq_c, w_in_layout), mat(wk_c, w_in_layout), mat(wv_c, w_in_layout)
    wp, wb = _ws(workspace)
    _check(_fn("ecospa_coupled_qkv_bwd")(X.data_ptr(), X.stride(0), T, d_m, _ref(mq), _ref(mk), _ref(mv), n_qk, n_vo,
                                         dQc.data_ptr(), dKc.data_ptr(), dVc.data_ptr(), dQc.stride(0), dVc.stride(0),
                                         dX.data_ptr(), dX.stride(0), int(accumulate_dX), dWq_c.data_ptr(),
                                         dWk_c.data_ptr(), dWv_c.data_ptr(), dWq_c.stride(0), dWv_c.stride(0),
                                         _ptr(dbq_c), _ptr(dbk_c), _ptr(dbv_c), wp, wb, _stream(stream)),
           "ecospa_coupled_qkv_bwd")


def ecospa_coupled_vo_bwd_o(Ctx, wo_c, n: int, dOut, dCtx, dWo_c, dbo=None, workspace=None, stream=None,
        w_in_layout: int = SHARED_COLS, w_out_layout: int = SHARED_ROWS) -> None:
    T = Ctx.shape[0]
    d_m = wo_c.shape[1] if w_out_layout == SHARED_ROWS else wo_c.shape[0]
    mo = mat(wo_c, w_out_layout)
    wp, wb = _ws(workspace)
    _check(_fn("ecospa_coupled_vo_bwd_o")(Ctx.data_ptr(), Ctx.stride(0), T, d_m, _ref(mo), n, dOut.data_ptr(),
                                          dOut.stride(0), dCtx.data_ptr(), dCtx.stride(0), dWo_c.data_ptr(),
                                          dWo_c.stride(0), _ptr(dbo), wp, wb, _stream(stream)), "ecospa_coupled_vo_bwd_o")


def ecospa_coupled_vo_bwd_v(X, wv_c, n: int, dVc, dX, dWv_c, dbv_c=None, accumulate_dX: bool = False, workspace=None, stream=None,
        w_in_layout: int = SHARED_COLS, w_out_layout: int = SHARED_ROWS) -> None:
    T, d_m = X.shape
    mv = mat(wv_c, w_in_layout)
    wp, wb = _ws(workspace)
    _check(_fn("ecospa_coupled_vo_bwd_v")(X.data_ptr(), X.stride(0), T, d_m, _ref(mv), n, dVc.data_ptr(), dVc.stride(0),
                                          dX.data_ptr(), dX.stride(0), int(accumulate_dX), dWv_c.data_ptr(),
                                          dWv_c.stride(0), _ptr(dbv_c), wp, wb, _stream(stream)), "ecospa_coupled_vo_bwd_v")


def ecospa_coupled_ffn_fwd(X, act: int, w1_c, w2_c, k: int, Y, H, A, w1b_c=None, Hb=None, b1_c=None, b2=None,
                           workspace=None, stream=None,
        w_in_layout: int = SHARED_COLS, w_out_layout: int = SHARED_ROWS) -> None:
    T, d_m = X.shape
    m1 = mat(w1_c, w_in_layout)
    m1b = mat(w1b_c, w_in_layout) if w1b_c is not None else None
    m2 = mat(w2_c, w_out_layout)
    wp, wb = _ws(workspace)
    _check(_fn("ecospa_coupled_ffn_fwd")(X.data_ptr(), X.stride(0), T, d_m, act, _ref(m1), _ref(m1b), _ref(m2), k, _ptr(b1_c),
                                         _ptr(b2), Y.data_ptr(), Y.stride(0), H.data_ptr(), _ptr(Hb), A.data_ptr(),
                                         H.stride(0), wp, wb, _stream(stream)), "ecospa_coupled_ffn_fwd")


def ecospa_coupled_ffn_bwd(X, act: int, w1_c, w2_c, k: int, H, A, dY, dX, dW1_c, dW2_c, w1b_c=None, Hb=None,
                           dW1b_c=None, db1_c=None, db2=None, workspace=None, stream=None,
        w_in_layout: int = SHARED_COLS, w_out_layout: int = SHARED_ROWS) -> None:
    T, d_m = X.shape
    m1 = mat(w1_c, w_in_layout)
    m1b = mat(w1b_c, w_in_layout) if w1b_c is not None else None
    m2 = mat(w2_c, w_out_layout)
    wp, wb = _ws(workspace)
    _check(_fn("ecospa_coupled_ffn_bwd")(X.data_ptr(), X.stride(0), T, d_m, act, _ref(m1), _ref(m1b), _ref(m2), k, H.data_ptr(),
                                         _ptr(Hb), A.data_ptr(), H.stride(0), dY.data_ptr(), dY.stride(0), dX.data_ptr(),
                                         dX.stride(0), dW1_c.data_ptr(), _ptr(dW1b_c), dW1_c.stride(0), dW2_c.data_ptr(),
                                         dW2_c.stride(0), _ptr(db1_c), _ptr(db2), wp, wb, _stream(stream)),
           "ecospa_coupled_ffn_bwd")


# ---------------------------------------------------------------------------------------------
# attention core on compacted heads
# ---------------------------------------------------------------------------------------------

class Heads(C.Structure):
    _fields_ = [("n_heads", C.c_int32), ("qk_off", C.c_void_p), ("qk_w", C.c_void_p), ("vo_off", C.c_void_p),
                ("vo_w", C.c_void_p), ("n_kv_heads", C.c_int32), ("k_off", C.c_void_p), ("v_off", C.c_void_p)]


def heads(qk_off: Sequence[int], qk_w: Sequence[int], vo_off: Sequence[int], vo_w: Sequence[int],
          k_off: Optional[Sequence[int]] = None, v_off: Optional[Sequence[int]] = None) -> Heads:
    """Descriptor of the per-head column blocks of Qc / Kc (qk_*) and of Vc / Ctx (vo_*).  Grouped-query models: k_off,
    v_off = first columns of the K/V heads in Kc and Vc (len(qk_off) // len(k_off) query heads read each of them)."""
    n = len(qk_off)
    assert len(qk_w) == n and len(vo_off) == n and len(vo_w) == n
    arrs = [(C.c_int32 * n)(*[int(x) for x in v]) for v in (qk_off, qk_w, vo_off, vo_w)]
    if k_off is None:
        h = Heads(n, *[C.addressof(a) for a in arrs], 0, None, None)
    else:
        assert v_off is not None and len(v_off) == len(k_off)
        kv = [(C.c_int32 * len(k_off))(*[int(x) for x in v]) for v in (k_off, v_off)]
        h = Heads(n, *[C.addressof(a) for a in arrs], len(k_off), C.addressof(kv[0]), C.addressof(kv[1]))
        arrs += kv
    h._keep = arrs
    return h


def ecospa_attn_workspace_bytes(batch: int, seq: int, n_heads: int) -> int:
    f = lib().ecospa_attn_workspace_bytes
    f.restype = C.c_size_t
    f.argtypes = [C.c_int64, C.c_int64, C.c_int32]
    return int(f(batch, seq, n_heads))


def ecospa_coupled_attn_fwd(Qc, Kc, Vc, batch: int, seq: int, hd: Heads, scale: float, causal: bool, Ctx, lse,
                            stream=None) -> None:
    """Ctx_h = softmax(scale * Q_h K_h^T) V_h per sequence and head; lse: fp32 [n_heads * T]."""
    f = lib().ecospa_coupled_attn_fwd
    f.restype = C.c_int
    f.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_float,
                  C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
    assert Qc.stride(0) == Kc.stride(0)
    _check(f(Qc.data_ptr(), Kc.data_ptr(), Qc.stride(0), Vc.data_ptr(), Vc.stride(0), batch, seq, C.addressof(hd),
             float(scale), int(bool(causal)), Ctx.data_ptr(), Ctx.stride(0), lse.data_ptr(), _stream(stream)),
           "ecospa_coupled_attn_fwd")


def ecospa_coupled_attn_bwd(Qc, Kc, Vc, Ctx, dCtx, lse, batch: int, seq: int, hd: Heads, scale: float, causal: bool,
                            dQc, dKc, dVc, workspace, stream=None) -> None:
    f = lib().ecospa_coupled_attn_bwd
    f.restype = C.c_int
    f.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64,
                  C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_float, C.c_int32, C.c_void_p, C.c_void_p, C.c_int64,
                  C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p]
    assert Qc.stride(0) == Kc.stride(0) and dQc.stride(0) == dKc.stride(0)
    wp, wb = _ws(workspace)
    _check(f(Qc.data_ptr(), Kc.data_ptr(), Qc.stride(0), Vc.data_ptr(), Vc.stride(0), Ctx.data_ptr(), Ctx.stride(0),
             dCtx.data_ptr(), dCtx.stride(0), lse.data_ptr(), batch, seq, C.addressof(hd), float(scale),
             int(bool(causal)), dQc.data_ptr(), dKc.data_ptr(), dQc.stride(0), dVc.data_ptr(), dVc.stride(0), wp, wb,
             _stream(stream)), "ecospa_coupled_attn_bwd")


def ecospa_pad_kept(kept: torch.Tensor, src: Sequence[int], dst: Sequence[int], k: Sequence[int],
                    k_padded: Sequence[int], out: torch.Tensor, stream=None) -> None:
    n = len(src)
    assert len(dst) == n and len(k) == n and len(k_padded) == n and kept.dtype == torch.int32 and out.dtype == torch.int32
    arr = lambda v: (C.c_int32 * n)(*[int(x) for x in v])
    a_src, a_dst, a_k, a_kp = arr(src), arr(dst), arr(k), arr(k_padded)
    fn = lib().ecospa_pad_kept
    fn.restype = C.c_int
    fn.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
    _check(fn(_ptr(kept), C.addressof(a_src), C.addressof(a_dst), C.addressof(a_k), C.addressof(a_kp), n, _ptr(out),
              _stream(stream)), "ecospa_pad_kept")


# ---------------------------------------------------------------------------------------------
# one pass of Algorithm 1's body over groups of pairs
# ---------------------------------------------------------------------------------------------

class Group(C.Structure):
    _fields_ = [("w1", Mat), ("w1b", Mat), ("w2", Mat), ("g1", Mat), ("g1b", Mat), ("g2", Mat), ("aux", C.c_void_p),
                ("n_aux", C.c_int32), ("n_pairs", C.c_int32), ("widths", C.c_void_p), ("rope", C.c_int32),
                ("reserved_", C.c_int32)]


def group(w1, w2, layout1: int, layout2: int, widths: Sequence[int], w1b=None, g1=None, g2=None, g1b=None,
          aux: Sequence[Tuple[Optional[torch.Tensor], int]] = (), rope: int = 0) -> Group:
    """Descriptor of the tensors on one shared axis; aux = (tensor, layout) pairs (a 1-D tensor is a bias)."""
    n_aux = len(aux)
    a_arr = (Mat * max(1, n_aux))(*[mat(t, lay) for t, lay in aux])
    w_arr = (C.c_int32 * len(widths))(*[int(v) for v in widths])
    g = Group(mat(w1, layout1), mat(w1b, layout1), mat(w2, layout2), mat(g1, layout1), mat(g1b, layout1), mat(g2, layout2),
              C.addressof(a_arr) if n_aux else None, n_aux, len(widths), C.addressof(w_arr), rope, 0)
    g._keep = (a_arr, w_arr, w1, w2, w1b, g1, g2, g1b, [t for t, _ in aux])
    return g


def _alg1(name, restype, argtypes):
    f = getattr(lib(), name)
    f.restype, f.argtypes = restype, argtypes
    return f


def ecospa_alg1_workspace_bytes(groups: Sequence[Group]) -> int:
    arr = (Group * len(groups))(*groups)
    return int(_alg1("ecospa_alg1_workspace_bytes", C.c_size_t, [C.c_void_p, C.c_int32])(C.addressof(arr), len(groups)))


def ecospa_alg1_offsets(groups: Sequence[Group]) -> List[int]:
    arr = (Group * len(groups))(*groups)
    out = (C.c_int64 * 6)()
    _check(_alg1("ecospa_alg1_offsets", C.c_int, [C.c_void_p, C.c_int32, C.c_void_p])(C.addressof(arr), len(groups), C.addressof(out)),
           "ecospa_alg1_offsets")
    return [int(v) for v in out]


def ecospa_alg1_plan(groups: Sequence[Group], n_samples: float, n_choose: int, theta: float, l1: bool, k_min: int,
                     workspace: torch.Tensor, stream=None) -> List[int]:
    """Returns the new width of every pair of every group (synchronises the stream)."""
    arr = (Group * len(groups))(*groups)
    n = sum(g.n_pairs for g in groups)
    k = (C.c_int32 * n)()
    f = _alg1("ecospa_alg1_plan", C.c_int, [C.c_void_p, C.c_int32, C.c_double, C.c_int32, C.c_double, C.c_int32, C.c_int32,
                                            C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p])
    _check(f(C.addressof(arr), len(groups), float(n_samples), int(n_choose), float(theta), int(bool(l1)), int(k_min),
             workspace.data_ptr(), workspace.numel(), C.addressof(k), _stream(stream)), "ecospa_alg1_plan")
    return list(k)


def ecospa_alg1_apply(groups: Sequence[Group], k: Sequence[int], out: Optional[Sequence[Group]], workspace: torch.Tensor,
                      in_place: bool = False, stream=None) -> None:
    arr = (Group * len(groups))(*groups)
    oarr = (Group * len(out))(*out) if out is not None else None
    ka = (C.c_int32 * len(k))(*[int(v) for v in k])
    f = _alg1("ecospa_alg1_apply", C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t,
                                             C.c_void_p])
    _check(f(C.addressof(arr), len(groups), C.addressof(ka), C.addressof(oarr) if oarr is not None else None,
             int(bool(in_place)), workspace.data_ptr(), workspace.numel(), _stream(stream)), "ecospa_alg1_apply")


def ecospa_launch_count() -> int:
    f = lib().ecospa_launch_count
    f.restype = C.c_uint64
    return int(f())


def ecospa_set_device_wait_limit_ns(ns: int) -> None:
    """How long a device-side wait of the layer kernels may last before the kernel gives up (default 2 s)."""
    f = lib().ecospa_set_device_wait_limit_ns
    f.restype = C.c_int
    f.argtypes = [C.c_uint64]
    _check(f(int(ns)), "ecospa_set_device_wait_limit_ns")


def ecospa_gemm_resident_pairs() -> int:
    f = lib().ecospa_gemm_resident_pairs
    f.restype = C.c_int32
    return int(f())


def ecospa_device_status(stream=None) -> int:
    """Synchronises the stream; returns 0 or raises EcospaError(ERR_TIMEOUT) carrying the wait code."""
    code = C.c_int32(0)
    st = _fn("ecospa_device_status")(_stream(stream), C.addressof(code))
    if st != 0:
        e = EcospaError(st, f"ecospa_device_status (wait code {code.value})")
        e.code = code.value
        raise e
    return 0
