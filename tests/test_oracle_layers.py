"""Pins for the oracle's layer math (Eq. 2, 3, 5 on compacted pairs and their gradients).

Checked against library routines on special cases, mathematical constants, central
finite differences and the masked-full-layer identity.
"""
import math

import numpy as np
import pytest
import torch

from oracle import oracle as O

COLS, ROWS = O.SHARED_COLS, O.SHARED_ROWS


def rng(seed):
    return np.random.default_rng(seed)


def test_projection_matches_library_matmul_in_both_layouts():
    r = rng(1)
    T, dm, n = 7, 6, 5
    X = r.standard_normal((T, dm)); W = r.standard_normal((dm, n)); b = r.standard_normal(n)
    Y = O.proj_fwd(X, W, COLS, n, bias=b)
    np.testing.assert_allclose(Y, X @ W + b, rtol=1e-13, atol=1e-13)
    Yt = O.proj_fwd(X, np.ascontiguousarray(W.T), ROWS, n, bias=b)
    np.testing.assert_allclose(Yt, Y, rtol=1e-13, atol=1e-13)
    # padded leading dimension: extra columns are ignored
    Wp = np.concatenate([W, 99.0 * np.ones((dm, 3))], axis=1)
    np.testing.assert_allclose(O.proj_fwd(X, Wp, COLS, n, bias=b), Y, rtol=1e-13, atol=1e-13)


def test_projection_backward_matches_library_and_accumulates_dx():
    r = rng(2)
    T, dm, n = 8, 5, 4
    X = r.standard_normal((T, dm)); Wq = r.standard_normal((dm, n)); Wk = r.standard_normal((dm, n))
    dQ = r.standard_normal((T, n)); dK = r.standard_normal((T, n))
    dX, dWq, dbq = O.proj_bwd(X, Wq, COLS, n, dQ, want_db=True)
    dX, dWk, dbk = O.proj_bwd(X, Wk, COLS, n, dK, want_db=True, dX=dX)
    np.testing.assert_allclose(dX, dQ @ Wq.T + dK @ Wk.T, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dWq, X.T @ dQ, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dWk, X.T @ dK, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dbq, dQ.sum(0), rtol=1e-12)
    np.testing.assert_allclose(dbk, dK.sum(0), rtol=1e-12)


def test_output_projection_fwd_bwd_match_library():
    r = rng(3)
    T, n, dm = 6, 5, 7
    Ctx = r.standard_normal((T, n)); Wo = r.standard_normal((n, dm)); b = r.standard_normal(dm)
    dOut = r.standard_normal((T, dm))
    Out = O.outproj_fwd(Ctx, Wo, ROWS, n, dm, bias=b)
    np.testing.assert_allclose(Out, Ctx @ Wo + b, rtol=1e-13, atol=1e-13)
    dCtx, dW, db = O.outproj_bwd(Ctx, Wo, ROWS, n, dm, dOut, want_db=True)
    np.testing.assert_allclose(dCtx, dOut @ Wo.T, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dW, (Ctx.T @ dOut).T, rtol=1e-12, atol=1e-12)   # math orientation d_m x n
    np.testing.assert_allclose(db, dOut.sum(0), rtol=1e-12)


def test_activation_values_are_the_textbook_constants():
    xs = np.array([[-2.0, -1.0, 0.0, 0.5, 1.0, 3.0]])
    k = xs.shape[1]
    I = np.eye(k)
    X = np.diag(xs[0])        # row t has x_t in column t -> H[t, t] = x_t
    out = O.ffn_fwd(X, O.ACT_GELU_ERF, I, I, COLS, ROWS, k)
    Phi = np.array([0.5 * (1 + math.erf(v / math.sqrt(2))) for v in xs[0]])
    np.testing.assert_allclose(np.diag(out["A"]), xs[0] * Phi, rtol=1e-15, atol=1e-16)
    assert abs(out["A"][4, 4] - 0.8413447460685429) < 1e-15      # GELU(1) = Phi(1)
    lib = torch.nn.functional.gelu(torch.from_numpy(xs[0]), approximate="none").numpy()
    np.testing.assert_allclose(np.diag(out["A"]), lib, rtol=1e-14, atol=1e-16)
    out_t = O.ffn_fwd(X, O.ACT_GELU_TANH, I, I, COLS, ROWS, k)
    lib_t = torch.nn.functional.gelu(torch.from_numpy(xs[0]), approximate="tanh").numpy()
    np.testing.assert_allclose(np.diag(out_t["A"]), lib_t, rtol=1e-14, atol=1e-16)
    # SwiGLU: A = silu(X W_gate) . (X W_up); with W_up = 2 I the up branch is 2 x
    out_s = O.ffn_fwd(X, O.ACT_SWIGLU, I, I, COLS, ROWS, k, W1b=2 * I)
    silu = xs[0] / (1 + np.exp(-xs[0]))
    np.testing.assert_allclose(np.diag(out_s["A"]), silu * 2 * xs[0], rtol=1e-15, atol=1e-16)
    assert abs(out_s["A"][4, 4] - 2 * 0.7310585786300049) < 1e-15  # silu(1) = sigmoid(1)
    np.testing.assert_allclose(np.diag(out_s["Hb"]), 2 * xs[0])


@pytest.mark.parametrize("act", [O.ACT_GELU_ERF, O.ACT_GELU_TANH, O.ACT_SWIGLU])
def test_ffn_forward_matches_library_composition(act):
    r = rng(4)
    T, dm, k = 9, 6, 7
    X = r.standard_normal((T, dm)); W1 = r.standard_normal((dm, k)); W2 = r.standard_normal((k, dm))
    W1b = r.standard_normal((dm, k)) if act == O.ACT_SWIGLU else None
    b1 = None if act == O.ACT_SWIGLU else r.standard_normal(k)
    b2 = None if act == O.ACT_SWIGLU else r.standard_normal(dm)
    out = O.ffn_fwd(X, act, W1, W2, COLS, ROWS, k, W1b=W1b, b1=b1, b2=b2)
    tx = torch.from_numpy
    if act == O.ACT_SWIGLU:
        A = torch.nn.functional.silu(tx(X) @ tx(W1)) * (tx(X) @ tx(W1b))
        Y = A @ tx(W2)
    else:
        H = tx(X) @ tx(W1) + tx(b1)
        A = torch.nn.functional.gelu(H, approximate="none" if act == O.ACT_GELU_ERF else "tanh")
        Y = A @ tx(W2) + tx(b2)
    np.testing.assert_allclose(out["A"], A.numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(out["Y"], Y.numpy(), rtol=1e-12, atol=1e-12)
    # the transposed storage of both weights gives the same layer
    out_t = O.ffn_fwd(X, act, np.ascontiguousarray(W1.T), np.ascontiguousarray(W2.T), ROWS, COLS, k,
                      W1b=None if W1b is None else np.ascontiguousarray(W1b.T), b1=b1, b2=b2)
    np.testing.assert_allclose(out_t["Y"], out["Y"], rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("act", [O.ACT_GELU_ERF, O.ACT_GELU_TANH, O.ACT_SWIGLU])
def test_ffn_backward_by_central_finite_differences(act):
    r = rng(5)
    T, dm, k = 4, 3, 5
    X = r.standard_normal((T, dm)); W1 = r.standard_normal((dm, k)); W2 = r.standard_normal((k, dm))
    W1b = r.standard_normal((dm, k)) if act == O.ACT_SWIGLU else None
    b1 = None if act == O.ACT_SWIGLU else r.standard_normal(k)
    b2 = None if act == O.ACT_SWIGLU else r.standard_normal(dm)
    dY = r.standard_normal((T, dm))

    def loss(X_, W1_, W1b_, W2_, b1_, b2_):
        return float((O.ffn_fwd(X_, act, W1_, W2_, COLS, ROWS, k, W1b=W1b_, b1=b1_, b2=b2_)["Y"] * dY).sum())

    g = O.ffn_bwd(X, act, W1, W2, COLS, ROWS, k, dY, W1b=W1b, b1=b1, want_bias=True)
    eps = 1e-6
    args = [X, W1, W1b, W2, b1, b2]
    names = ["dX", "dW1", "dW1b", "dW2", "db1", "db2"]
    for ai, name in enumerate(names):
        if args[ai] is None:
            continue
        base = args[ai]
        num = np.zeros_like(base)
        it = np.nditer(base, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            plus = [a if a is None else a.copy() for a in args]; minus = [a if a is None else a.copy() for a in args]
            plus[ai][idx] += eps; minus[ai][idx] -= eps
            num[idx] = (loss(*plus) - loss(*minus)) / (2 * eps)
        got = g[name]
        if name == "dW2":
            got = got.T            # oracle returns d_m x k (math orientation); W2 here is k x d_m
        np.testing.assert_allclose(got, num, rtol=2e-6, atol=2e-7, err_msg=name)


def test_projection_backward_by_finite_differences():
    r = rng(6)
    T, dm, n = 4, 3, 5
    X = r.standard_normal((T, dm)); W = r.standard_normal((dm, n)); b = r.standard_normal(n)
    dY = r.standard_normal((T, n))

    def loss(X_, W_, b_):
        return float((O.proj_fwd(X_, W_, COLS, n, bias=b_) * dY).sum())

    dX, dW, db = O.proj_bwd(X, W, COLS, n, dY, want_db=True)
    eps = 1e-6
    for base, got, pos in ((X, dX, 0), (W, dW, 1), (b, db, 2)):
        num = np.zeros_like(base)
        it = np.nditer(base, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            args_p = [X.copy(), W.copy(), b.copy()]; args_m = [X.copy(), W.copy(), b.copy()]
            args_p[pos][idx] += eps; args_m[pos][idx] -= eps
            num[idx] = (loss(*args_p) - loss(*args_m)) / (2 * eps)
        np.testing.assert_allclose(got, num, rtol=2e-6, atol=2e-7)


@pytest.mark.parametrize("act", [O.ACT_GELU_ERF, O.ACT_SWIGLU])
def test_masked_full_layer_identity(act):
    """The compacted FFN equals the full FFN whose dropped hidden units are zeroed after the
    activation (here: rows of W_2 zeroed), and every compacted gradient is the matching slice."""
    r = rng(7)
    T, dm, d = 6, 5, 12
    X = r.standard_normal((T, dm)); W1 = r.standard_normal((dm, d)); W2 = r.standard_normal((d, dm))
    W1b = r.standard_normal((dm, d)) if act == O.ACT_SWIGLU else None
    b1 = None if act == O.ACT_SWIGLU else r.standard_normal(d)
    dY = r.standard_normal((T, dm))
    _, ups = O.score_pair(W1, W2, COLS, ROWS, 1, d, w1b=W1b)
    kept = O.select_topk(ups, 1, d, [7])
    tw = torch.from_numpy
    W1c = O.compact(tw(W1), COLS, kept, ld_out=8).numpy()        # padded to 8 columns
    W2c = O.compact(tw(W2), ROWS, kept).numpy()
    W1bc = None if W1b is None else O.compact(tw(W1b), COLS, kept, ld_out=8).numpy()
    b1c = None if b1 is None else O.compact(tw(b1), COLS, kept).numpy()
    k = len(kept)
    fc = O.ffn_fwd(X, act, W1c, W2c, COLS, ROWS, k, W1b=W1bc, b1=b1c)
    W2m = np.zeros_like(W2); W2m[kept] = W2[kept]
    ff = O.ffn_fwd(X, act, W1, W2m, COLS, ROWS, d, W1b=W1b, b1=b1)
    np.testing.assert_allclose(fc["Y"], ff["Y"], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(fc["A"], ff["A"][:, kept], rtol=1e-12, atol=1e-12)
    gc = O.ffn_bwd(X, act, W1c, W2c, COLS, ROWS, k, dY, W1b=W1bc, b1=b1c, want_bias=True)
    gf = O.ffn_bwd(X, act, W1, W2m, COLS, ROWS, d, dY, W1b=W1b, b1=b1, want_bias=True)
    np.testing.assert_allclose(gc["dX"], gf["dX"], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(gc["dW1"], gf["dW1"][:, kept], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(gc["dW2"], gf["dW2"][:, kept], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(gc["db1"], gf["db1"][kept], rtol=1e-12, atol=1e-12)
    dropped = np.setdiff1d(np.arange(d), kept)
    assert np.all(gf["dW1"][:, dropped] == 0.0)                  # dropped units get no gradient
    if act == O.ACT_SWIGLU:
        np.testing.assert_allclose(gc["dW1b"], gf["dW1b"][:, kept], rtol=1e-12, atol=1e-12)


def test_compacted_qk_scores_equal_restricted_full_scores():
    # Q^c K^c^T = Q[:, kept] K[:, kept]^T per head: the attention logits of the compacted pair
    r = rng(8)
    T, h, dh = 5, 2, 6
    dm = h * dh
    X = r.standard_normal((T, dm)); WQ = r.standard_normal((dm, dm)); WK = r.standard_normal((dm, dm))
    _, ups = O.score_pair(WQ, WK, COLS, COLS, h, dh)
    k = [4, 3]
    kept = O.select_topk(ups, h, dh, k)
    tw = torch.from_numpy
    WQc = O.compact(tw(WQ), COLS, kept, ld_out=8).numpy(); WKc = O.compact(tw(WK), COLS, kept, ld_out=8).numpy()
    Qc = O.proj_fwd(X, WQc, COLS, sum(k)); Kc = O.proj_fwd(X, WKc, COLS, sum(k))
    Q = X @ WQ; K = X @ WK
    off = 0
    for i in range(h):
        ki = kept[off:off + k[i]]
        np.testing.assert_allclose(Qc[:, off:off + k[i]] @ Kc[:, off:off + k[i]].T, Q[:, ki] @ K[:, ki].T,
                                   rtol=1e-12, atol=1e-12)
        off += k[i]
