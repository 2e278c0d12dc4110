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


class EcospaError(RuntimeError):
    def __init__(self, status: int, where: str):
        l = lib()
        msg = l.ecospa_status_string(status).decode()
        cuda = l.ecospa_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} (status {status})" + (f" [{cuda}]" if status == 4 and cuda else ""))
        self.status = status


class Mat(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("dtype", C.c_int32), ("layout", C.c_int32),
                ("other_dim", C.c_int64), ("ld", C.c_int64)]


class Pair(C.Structure):
    _fields_ = [("kind", C.c_int32), ("n_seg", C.c_int32), ("seg_len", C.c_int32), ("reserved", C.c_int32),
                ("w1", Mat), ("w1b", Mat), ("w2", Mat), ("g1", Mat), ("g1b", Mat), ("g2", Mat)]


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
         g1=None, g2=None, g1b=None) -> Pair:
    p = Pair(kind, n_seg, seg_len, 0, mat(w1, layout1), mat(w1b, layout1), mat(w2, layout2),
             mat(g1, layout1), mat(g1b, layout1), mat(g2, layout2))
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


def gather(inp: torch.Tensor, out: torch.Tensor, layout: int, kept: torch.Tensor, n_kept: int, shared_dim: int) -> Gather:
    g = Gather(mat(inp, layout), mat(out, layout), kept.data_ptr(), n_kept, shared_dim)
    g._keep = (inp, out, kept)
    return g


def ecospa_compact_tensors(jobs: Sequence[Gather], stream=None) -> None:
    arr = (Gather * len(jobs))(*jobs)
    st = lib().ecospa_compact_tensors(C.addressof(arr), len(jobs), _stream(stream))
    if st != 0:
        raise EcospaError(st, "ecospa_compact_tensors")


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
