"""ctypes front end of the CPU oracle (ecospa_oracle.cpp) -- TEST INFRASTRUCTURE ONLY.

Nothing in the product package imports this module.  It marshals numpy / torch CPU
tensors into the plain-C oracle and returns numpy fp64 (or int32 / raw byte) results.
It performs no arithmetic of the method itself.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ecospa_oracle.cpp")
_LIB = os.path.join(_HERE, "libecospa_oracle.so")

F32, BF16, F64 = 0, 1, 2
SHARED_COLS, SHARED_ROWS = 0, 1
ACT_GELU_ERF, ACT_GELU_TANH, ACT_SWIGLU = 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (plain -O2, no fast-math) if it is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-o", _LIB, _SRC])
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.eco_coupled_single.restype = C.c_int32
        _lib.eco_frob_removed.restype = C.c_double
    return _lib


# ---------------------------------------------------------------------------
# marshalling helpers
# ---------------------------------------------------------------------------

class _Buf:
    """Keeps a contiguous CPU buffer alive and exposes (pointer, dtype code, leading dim)."""

    def __init__(self, t):
        if t is None:
            self.arr, self.ptr, self.dtype, self.ld = None, None, F64, 0
            return
        if isinstance(t, torch.Tensor):
            t = t.detach().cpu().contiguous()
            assert t.dim() <= 2, "2-D or 1-D tensors only"
            ld = t.shape[1] if t.dim() == 2 else t.numel()
            if t.dtype == torch.bfloat16:
                arr, code = t.view(torch.int16).numpy(), BF16
            elif t.dtype == torch.float32:
                arr, code = t.numpy(), F32
            elif t.dtype == torch.float64:
                arr, code = t.numpy(), F64
            else:
                raise TypeError(t.dtype)
        else:
            arr = np.ascontiguousarray(t)
            ld = arr.shape[1] if arr.ndim == 2 else arr.size
            code = {np.dtype(np.float32): F32, np.dtype(np.float64): F64}[arr.dtype]
        self.arr, self.dtype, self.ld = arr, code, int(ld)
        self.ptr = C.c_void_p(arr.ctypes.data)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _p(a: Optional[np.ndarray]):
    return None if a is None else C.c_void_p(a.ctypes.data)


def _shared_dims(t, layout):
    """(other, D) of a matrix with a shared axis."""
    r, c = t.shape
    return (r, c) if layout == SHARED_COLS else (c, r)


# ---------------------------------------------------------------------------
# scores, Fisher, selection, compaction
# ---------------------------------------------------------------------------

def sumsq_shared(w, layout: int) -> np.ndarray:
    b = _Buf(w)
    other, D = _shared_dims(w, layout)
    out = np.empty(D, dtype=np.float64)
    lib().eco_sumsq_shared(b.ptr, b.dtype, layout, C.c_int64(other), C.c_int64(D), C.c_int64(b.ld), _p(out))
    return out


def sumsq_shared_hadamard(gate, up, layout: int) -> np.ndarray:
    g, u = _Buf(gate), _Buf(up)
    assert g.dtype == u.dtype and gate.shape == up.shape
    other, D = _shared_dims(gate, layout)
    out = np.empty(D, dtype=np.float64)
    lib().eco_sumsq_shared_hadamard(g.ptr, u.ptr, g.dtype, layout, C.c_int64(other), C.c_int64(D),
                                    C.c_int64(g.ld), C.c_int64(u.ld), _p(out))
    return out


def upsilon(c1: np.ndarray, c2: np.ndarray, n_seg: int, seg_len: int, rope: int = 0):
    c1 = np.ascontiguousarray(c1, dtype=np.float64)
    c2 = np.ascontiguousarray(c2, dtype=np.float64)
    assert c1.size == c2.size == n_seg * seg_len
    raw = np.empty_like(c1)
    ups = np.empty_like(c1)
    if rope:
        assert seg_len % 2 == 0
        lib().eco_upsilon_rope(_p(c1), _p(c2), n_seg, seg_len, int(rope), _p(raw), _p(ups))
    else:
        lib().eco_upsilon(_p(c1), _p(c2), n_seg, seg_len, _p(raw), _p(ups))
    return raw, ups


def score_pair(w1, w2, layout1: int, layout2: int, n_seg: int, seg_len: int, w1b=None, rope: int = 0):
    """(raw, upsilon) of a coupled pair; w1b given = SwiGLU pair with W_1 = w1 (.) w1b; rope = 1 / 2: rotation
    pairs (2u, 2u+1) / (u, u + seg_len/2) of shared indices are the scored unit."""
    c1 = sumsq_shared(w1, layout1) if w1b is None else sumsq_shared_hadamard(w1, w1b, layout1)
    c2 = sumsq_shared(w2, layout2)
    return upsilon(c1, c2, n_seg, seg_len, rope)


def select_rotation_pairs(ups, n_seg: int, seg_len: int, k: Sequence[int], rope: int) -> np.ndarray:
    """Ascending kept indices, whole rotation pairs only (k even), fp32 scores ranked as stored."""
    k = _i32(k)
    assert k.size == n_seg and (k % 2 == 0).all() and (k <= seg_len).all() and rope in (1, 2)
    ups = np.ascontiguousarray(ups, dtype=np.float32)
    kept = np.empty(int(k.sum()), dtype=np.int32)
    lib().eco_select_rotation_pairs_f32(_p(ups), n_seg, seg_len, _p(k), int(rope), _p(kept))
    return kept


def fisher_pair(g1, g2, layout1: int, layout2: int, n_seg: int, seg_len: int, n_samples: float, g1b=None):
    a, b, ab = _Buf(g1), _Buf(g2), _Buf(g1b)
    other1, D1 = _shared_dims(g1, layout1)
    other2, D2 = _shared_dims(g2, layout2)
    assert D1 == D2 == n_seg * seg_len and a.dtype == b.dtype
    out = np.empty(n_seg, dtype=np.float64)
    lib().eco_fisher_pair(a.ptr, ab.ptr, b.ptr, a.dtype, layout1, layout2, C.c_int64(other1), C.c_int64(other2),
                          C.c_int64(a.ld), C.c_int64(ab.ld), C.c_int64(b.ld), n_seg, seg_len,
                          C.c_double(n_samples), _p(out))
    return out


def select_topk(ups, n_seg: int, seg_len: int, k: Sequence[int]) -> np.ndarray:
    """Ascending global kept indices, segment after segment.  fp32 input is ranked as fp32."""
    k = _i32(k)
    assert k.size == n_seg and (k >= 0).all() and (k <= seg_len).all()
    kept = np.empty(int(k.sum()), dtype=np.int32)
    ups = np.ascontiguousarray(ups)
    assert ups.size == n_seg * seg_len
    if ups.dtype == np.float32:
        lib().eco_select_topk_f32(_p(ups), n_seg, seg_len, _p(k), _p(kept))
    else:
        ups = ups.astype(np.float64, copy=False)
        lib().eco_select_topk_f64(_p(ups), n_seg, seg_len, _p(k), _p(kept))
    return kept


def threshold_counts(ups, n_seg: int, seg_len: int, theta: float, l1: bool = True, k_min: int = 1,
                     chosen=None, rope: int = 0) -> np.ndarray:
    """Kept count per segment after Algorithm 1's cumulative-threshold loop (fp32 scores as stored)."""
    ups = np.ascontiguousarray(ups, dtype=np.float32)
    assert ups.size == n_seg * seg_len
    k = np.empty(n_seg, dtype=np.int32)
    ch = _i32(chosen) if chosen is not None else None
    lib().eco_threshold_counts_f32(_p(ups), n_seg, seg_len, int(rope), C.c_double(theta), int(l1), int(k_min), _p(ch), _p(k))
    return k


def choose_pairs(fisher, m: int) -> np.ndarray:
    """Flags of the m pairs with the smallest importance (ties: lower index first)."""
    f = np.ascontiguousarray(fisher, dtype=np.float32)
    out = np.empty(f.size, dtype=np.int32)
    lib().eco_choose_pairs_f32(_p(f), f.size, int(m), _p(out))
    return out


def compact(t: torch.Tensor, layout: int, kept, ld_out: Optional[int] = None) -> torch.Tensor:
    """Gather the kept shared indices of `t` (2-D, or 1-D = a bias over the shared axis)."""
    kept = _i32(kept)
    vec = t.dim() == 1
    t2 = t.reshape(1, -1) if vec else t
    if vec:
        layout = SHARED_COLS
    t2 = t2.detach().cpu().contiguous()
    other, D = _shared_dims(t2, layout)
    eb = t2.element_size()
    n_kept = kept.size
    if layout == SHARED_COLS:
        ld = ld_out if ld_out is not None else n_kept
        out = torch.empty((other, ld), dtype=t2.dtype)
    else:
        ld = ld_out if ld_out is not None else other
        out = torch.empty((n_kept, ld), dtype=t2.dtype)
    src = t2.view(torch.uint8).numpy() if eb == 1 else t2.view(torch.int16 if eb == 2 else torch.int32 if eb == 4 else torch.int64).numpy()
    dst_t = out.view(torch.int16 if eb == 2 else torch.int32 if eb == 4 else torch.int64)
    dst = dst_t.numpy()
    lib().eco_compact_bytes(_p(src), eb, layout, C.c_int64(other), C.c_int64(t2.stride(0)), _p(kept),
                            C.c_int64(n_kept), _p(dst), C.c_int64(ld))
    return out.reshape(-1) if vec else out


# ---------------------------------------------------------------------------
# Appendix A comparators
# ---------------------------------------------------------------------------

def coupled_single(A: np.ndarray, B: np.ndarray) -> int:
    A = np.ascontiguousarray(A, dtype=np.float64)
    B = np.ascontiguousarray(B, dtype=np.float64)
    m, n = A.shape
    p = B.shape[1]
    return int(lib().eco_coupled_single(_p(A), _p(B), C.c_int64(m), C.c_int64(n), C.c_int64(p)))


def individual_single(A: np.ndarray, B: np.ndarray):
    A = np.ascontiguousarray(A, dtype=np.float64)
    B = np.ascontiguousarray(B, dtype=np.float64)
    m, n = A.shape
    p = B.shape[1]
    ks, ls = C.c_int32(0), C.c_int32(0)
    lib().eco_individual_single(_p(A), _p(B), C.c_int64(m), C.c_int64(n), C.c_int64(p), C.byref(ks), C.byref(ls))
    return int(ks.value), int(ls.value)


def frob_removed(A: np.ndarray, B: np.ndarray, keptA, keptB) -> float:
    A = np.ascontiguousarray(A, dtype=np.float64)
    B = np.ascontiguousarray(B, dtype=np.float64)
    ka, kb = _i32(keptA), _i32(keptB)
    assert ka.size == kb.size
    m, n = A.shape
    p = B.shape[1]
    return float(lib().eco_frob_removed(_p(A), _p(B), C.c_int64(m), C.c_int64(n), C.c_int64(p), _p(ka), _p(kb),
                                        C.c_int64(ka.size)))


# ---------------------------------------------------------------------------
# layer math
# ---------------------------------------------------------------------------

def _wdims(w, layout):
    other, D = _shared_dims(w, layout)
    return other, D


def proj_fwd(X, W, wlayout: int, n: int, bias=None) -> np.ndarray:
    """Y = X W^c + b with W^c a (d_m x n) shared-cols or (n x d_m) shared-rows matrix (n real columns)."""
    x, w, b = _Buf(X), _Buf(W), _Buf(bias)
    T, d_m = X.shape
    Y = np.empty((T, n), dtype=np.float64)
    lib().eco_proj_fwd(x.ptr, x.dtype, C.c_int64(T), C.c_int64(d_m), C.c_int64(x.ld), w.ptr, w.dtype, wlayout,
                       C.c_int64(n), C.c_int64(w.ld), b.ptr, _p(Y))
    return Y


def proj_bwd(X, W, wlayout: int, n: int, dY, want_db: bool = False, dX: Optional[np.ndarray] = None):
    x, w, dy = _Buf(X), _Buf(W), _Buf(dY)
    assert x.dtype == dy.dtype
    T, d_m = X.shape
    if dX is None:
        dX = np.zeros((T, d_m), dtype=np.float64)
    dW = np.empty((d_m, n), dtype=np.float64)
    db = np.empty(n, dtype=np.float64) if want_db else None
    lib().eco_proj_bwd(x.ptr, x.dtype, C.c_int64(T), C.c_int64(d_m), C.c_int64(x.ld), w.ptr, w.dtype, wlayout,
                       C.c_int64(n), C.c_int64(w.ld), dy.ptr, C.c_int64(dy.ld), _p(dX), _p(dW), _p(db))
    return dX, dW, db


def outproj_fwd(Ctx, W, wlayout: int, n: int, d_m: int, bias=None) -> np.ndarray:
    c, w, b = _Buf(Ctx), _Buf(W), _Buf(bias)
    T = Ctx.shape[0]
    Out = np.empty((T, d_m), dtype=np.float64)
    lib().eco_outproj_fwd(c.ptr, c.dtype, C.c_int64(T), C.c_int64(n), C.c_int64(c.ld), w.ptr, w.dtype, wlayout,
                          C.c_int64(d_m), C.c_int64(w.ld), b.ptr, _p(Out))
    return Out


def outproj_bwd(Ctx, W, wlayout: int, n: int, d_m: int, dOut, want_db: bool = False):
    c, w, do = _Buf(Ctx), _Buf(W), _Buf(dOut)
    T = Ctx.shape[0]
    dCtx = np.empty((T, n), dtype=np.float64)
    dW = np.empty((d_m, n), dtype=np.float64)
    db = np.empty(d_m, dtype=np.float64) if want_db else None
    lib().eco_outproj_bwd(c.ptr, c.dtype, C.c_int64(T), C.c_int64(n), C.c_int64(c.ld), w.ptr, w.dtype, wlayout,
                          C.c_int64(d_m), C.c_int64(w.ld), do.ptr, C.c_int64(do.ld), _p(dCtx), _p(dW), _p(db))
    return dCtx, dW, db


def ffn_fwd(X, act: int, W1, W2, layout1: int, layout2: int, k: int, W1b=None, b1=None, b2=None):
    """Returns dict(Y, H, Hb, A) in fp64."""
    x, w1, w1b, w2, bb1, bb2 = _Buf(X), _Buf(W1), _Buf(W1b), _Buf(W2), _Buf(b1), _Buf(b2)
    T, d_m = X.shape
    Y = np.empty((T, d_m), dtype=np.float64)
    H = np.empty((T, k), dtype=np.float64)
    A = np.empty((T, k), dtype=np.float64)
    Hb = np.empty((T, k), dtype=np.float64) if act == ACT_SWIGLU else None
    lib().eco_ffn_fwd(x.ptr, x.dtype, C.c_int64(T), C.c_int64(d_m), C.c_int64(x.ld), act, w1.ptr, w1b.ptr, w2.ptr,
                      w1.dtype, layout1, layout2, C.c_int64(k), C.c_int64(w1.ld), C.c_int64(w1b.ld),
                      C.c_int64(w2.ld), bb1.ptr, bb2.ptr, _p(Y), _p(H), _p(Hb), _p(A))
    return {"Y": Y, "H": H, "Hb": Hb, "A": A}


def ffn_bwd(X, act: int, W1, W2, layout1: int, layout2: int, k: int, dY, W1b=None, b1=None, want_bias: bool = False):
    """Returns dict(dX, dW1, dW1b, dW2, db1, db2); weight grads in math orientation (d_m x k)."""
    x, w1, w1b, w2, bb1, dy = _Buf(X), _Buf(W1), _Buf(W1b), _Buf(W2), _Buf(b1), _Buf(dY)
    assert x.dtype == dy.dtype
    T, d_m = X.shape
    dX = np.empty((T, d_m), dtype=np.float64)
    dW1 = np.empty((d_m, k), dtype=np.float64)
    dW2 = np.empty((d_m, k), dtype=np.float64)
    dW1b = np.empty((d_m, k), dtype=np.float64) if act == ACT_SWIGLU else None
    db1 = np.empty(k, dtype=np.float64) if want_bias else None
    db2 = np.empty(d_m, dtype=np.float64) if want_bias else None
    lib().eco_ffn_bwd(x.ptr, x.dtype, C.c_int64(T), C.c_int64(d_m), C.c_int64(x.ld), act, w1.ptr, w1b.ptr, w2.ptr,
                      w1.dtype, layout1, layout2, C.c_int64(k), C.c_int64(w1.ld), C.c_int64(w1b.ld),
                      C.c_int64(w2.ld), bb1.ptr, dy.ptr, C.c_int64(dy.ld), _p(dX), _p(dW1), _p(dW1b), _p(dW2),
                      _p(db1), _p(db2))
    return {"dX": dX, "dW1": dW1, "dW1b": dW1b, "dW2": dW2, "db1": db1, "db2": db2}


# ---------------------------------------------------------------------------
# attention on compacted heads
# ---------------------------------------------------------------------------

def attn_fwd(Q, K, V, batch: int, seq: int, qk_off, qk_w, vo_off, vo_w, scale: float, causal: bool = False,
             want_p: bool = False):
    """Returns dict(Ctx (T x V.shape[1], fp64; columns outside the heads are zero), lse (n_heads x T), P or None)."""
    q, k, v = _Buf(Q), _Buf(K), _Buf(V)
    assert q.dtype == k.dtype == v.dtype
    T = batch * seq
    assert Q.shape[0] == T and K.shape[0] == T and V.shape[0] == T
    qo, qw, vo, vw = _i32(qk_off), _i32(qk_w), _i32(vo_off), _i32(vo_w)
    H = qo.size
    assert qw.size == H and vo.size == H and vw.size == H
    Ctx = np.zeros((T, V.shape[1]), dtype=np.float64)
    lse = np.empty((H, T), dtype=np.float64)
    P = np.empty((H, batch, seq, seq), dtype=np.float64) if want_p else None
    lib().eco_attn_fwd(q.ptr, k.ptr, v.ptr, q.dtype, C.c_int64(batch), C.c_int64(seq), H, _p(qo), _p(qw), _p(vo), _p(vw),
                       C.c_int64(q.ld), C.c_int64(k.ld), C.c_int64(v.ld), C.c_double(scale), int(causal), _p(Ctx),
                       C.c_int64(Ctx.shape[1]), _p(lse), _p(P))
    return {"Ctx": Ctx, "lse": lse, "P": P}


def attn_bwd(Q, K, V, dCtx, batch: int, seq: int, qk_off, qk_w, vo_off, vo_w, scale: float, causal: bool = False):
    """Returns dict(dQ, dK (T x Q.shape[1]), dV (T x V.shape[1])) in fp64, zero outside the heads' columns."""
    q, k, v, dc = _Buf(Q), _Buf(K), _Buf(V), _Buf(dCtx)
    assert q.dtype == k.dtype == v.dtype == dc.dtype
    T = batch * seq
    qo, qw, vo, vw = _i32(qk_off), _i32(qk_w), _i32(vo_off), _i32(vo_w)
    H = qo.size
    dQ = np.zeros((T, Q.shape[1]), dtype=np.float64)
    dK = np.zeros((T, Q.shape[1]), dtype=np.float64)
    dV = np.zeros((T, V.shape[1]), dtype=np.float64)
    lib().eco_attn_bwd(q.ptr, k.ptr, v.ptr, dc.ptr, q.dtype, C.c_int64(batch), C.c_int64(seq), H, _p(qo), _p(qw), _p(vo),
                       _p(vw), C.c_int64(q.ld), C.c_int64(k.ld), C.c_int64(v.ld), C.c_int64(dc.ld), C.c_double(scale),
                       int(causal), _p(dQ), _p(dK), C.c_int64(dQ.shape[1]), _p(dV), C.c_int64(dV.shape[1]))
    return {"dQ": dQ, "dK": dK, "dV": dV}


# ---------------------------------------------------------------------------
# grouped-query attention: the pairs W_i^Q W_g(i)^K^T and W_g(i)^V W_i^O of "Extension to GQA"
# ---------------------------------------------------------------------------

def group_sum(c: np.ndarray, n_groups: int, rep: int, seg_len: int) -> np.ndarray:
    """c holds one value per shared index of `n_groups * rep` heads stored side by side, the heads of a group next to
    each other; returns, per group and index, the sum over the group's heads (length n_groups * seg_len)."""
    c = np.asarray(c, dtype=np.float64)
    assert c.size == n_groups * rep * seg_len
    return c.reshape(n_groups, rep, seg_len).sum(axis=1).reshape(-1)


def score_pair_gqa(w1, w2, layout1: int, layout2: int, n_groups: int, seg_len: int, rep1: int = 1, rep2: int = 1):
    """(raw, upsilon) per K/V group.  The heads that share a K (or V) head share its removable index: removing index
    j of group g removes it from every pair of the group at once, so the group is scored as ONE coupled pair whose
    W_1 (rep1 > 1: the group's query heads, stacked) or W_2 (rep2 > 1: the group's W^O row blocks, side by side) is
    the stack of the group's heads: the norm of index j on that side is the l2 norm over the whole stack."""
    c1 = group_sum(sumsq_shared(w1, layout1), n_groups, rep1, seg_len)
    c2 = group_sum(sumsq_shared(w2, layout2), n_groups, rep2, seg_len)
    return upsilon(c1, c2, n_groups, seg_len)


def fisher_pair_gqa(g1, g2, layout1: int, layout2: int, n_groups: int, seg_len: int, n_samples: float, rep1: int = 1,
                    rep2: int = 1) -> np.ndarray:
    """Eq. "importance" of the group's stacked pair: each side's mean squared gradient is taken over the whole stack."""
    s1 = group_sum(sumsq_shared(g1, layout1), n_groups, rep1, seg_len).reshape(n_groups, seg_len).sum(axis=1)
    s2 = group_sum(sumsq_shared(g2, layout2), n_groups, rep2, seg_len).reshape(n_groups, seg_len).sum(axis=1)
    other1, _ = _shared_dims(g1, layout1)
    other2, _ = _shared_dims(g2, layout2)
    return 0.5 * (s1 / (other1 * rep1 * seg_len) + s2 / (other2 * rep2 * seg_len)) / n_samples


# ---------------------------------------------------------------------------
# attention core for grouped-query models (Sec. 3.1, "Extension to GQA"): the query heads of a group read the K and V
# columns of the group's one K/V head.  Written as the definition: every query head is given a copy of its group's K and V
# columns and the per-head routines above are called; the gradients of the copies of a group are added.
# ---------------------------------------------------------------------------

def _expand_kv(K, V, rep, qk_off, qk_w, vo_off, vo_w, k_off, v_off, n_q, n_v):
    import torch
    T = K.shape[0]
    Ke = torch.zeros((T, n_q), dtype=K.dtype)
    Ve = torch.zeros((T, n_v), dtype=V.dtype)
    for h in range(len(qk_off)):
        g = h // rep
        Ke[:, qk_off[h]: qk_off[h] + qk_w[h]] = K[:, k_off[g]: k_off[g] + qk_w[h]]
        Ve[:, vo_off[h]: vo_off[h] + vo_w[h]] = V[:, v_off[g]: v_off[g] + vo_w[h]]
    return Ke, Ve


def attn_fwd_gqa(Q, K, V, batch: int, seq: int, qk_off, qk_w, vo_off, vo_w, k_off, v_off, scale: float, causal: bool = False):
    """Q (T x n_q) and the returned Ctx hold one block per query head (qk_off / vo_off), K and V one block per K/V head
    (k_off / v_off; head h reads group h // rep, rep = query heads per K/V head, and has the widths qk_w[h], vo_w[h])."""
    rep = len(qk_off) // len(k_off)
    n_v = max(o + w for o, w in zip(vo_off, vo_w))
    Ke, Ve = _expand_kv(K, V, rep, qk_off, qk_w, vo_off, vo_w, k_off, v_off, Q.shape[1], n_v)
    return attn_fwd(Q, Ke, Ve, batch, seq, qk_off, qk_w, vo_off, vo_w, scale, causal)


def attn_bwd_gqa(Q, K, V, dCtx, batch: int, seq: int, qk_off, qk_w, vo_off, vo_w, k_off, v_off, scale: float, causal: bool = False):
    """dQ in Q's layout; dK, dV in the layout of K and V: the sum over the query heads of each group."""
    rep = len(qk_off) // len(k_off)
    n_v = max(o + w for o, w in zip(vo_off, vo_w))
    Ke, Ve = _expand_kv(K, V, rep, qk_off, qk_w, vo_off, vo_w, k_off, v_off, Q.shape[1], n_v)
    dC = dCtx[:, :n_v].contiguous() if dCtx.shape[1] != n_v else dCtx
    r = attn_bwd(Q, Ke, Ve, dC, batch, seq, qk_off, qk_w, vo_off, vo_w, scale, causal)
    dK = np.zeros((K.shape[0], K.shape[1]), dtype=np.float64)
    dV = np.zeros((V.shape[0], V.shape[1]), dtype=np.float64)
    for h in range(len(qk_off)):
        g = h // rep
        dK[:, k_off[g]: k_off[g] + qk_w[h]] += r["dK"][:, qk_off[h]: qk_off[h] + qk_w[h]]
        dV[:, v_off[g]: v_off[g] + vo_w[h]] += r["dV"][:, vo_off[h]: vo_off[h] + vo_w[h]]
    return {"dQ": r["dQ"], "dK": dK, "dV": dV}
