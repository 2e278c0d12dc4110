"""GPU parity of the grouped attention-side calls a training step uses (Q/K/V in one launch, output projection,
its backward, and the backward of the three projections with dX accumulated) at the full token count, vs the fp64
oracle, plus run-to-run bit-identity of the backward calls.

At T = 8192 these calls take paths the small cases do not: weight gradients split over the tokens into fp32
partials that a finishing launch adds up, the dX product over three K segments leaving through reducing tile
stores onto a non-zero dX, and schedules of more than a hundred tiles.  Sampling is stratified: one token row in
every block of 256 rows (each row of an output depends on its input row only, and a sampled row crosses every
column tile) and one kept column / unit in every block of 256 (each weight-gradient column depends on that
column's upstream gradient only, and crosses every row tile), so every 256 x 256 output tile is touched.  The
error is asserted per sampled row and per sampled column (relative l2 <= 2e-2 each), not per tensor.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2511_11641_b200 import binding as B
from paper_2511_11641_b200 import block as BL
from paper_2511_11641_b200 import layers as L
from paper_2511_11641_b200 import workloads as WL

pytestmark = pytest.mark.gpu
DEV = "cuda"
TOL = 2e-2


def stratified(n, block, rng):
    """One index out of every `block` consecutive ones (the last block may be short)."""
    return np.array([rng.integers(a, min(a + block, n)) for a in range(0, n, block)], dtype=np.int64)


def assert_rows(name, got, ref, tol=TOL):
    """Relative l2 error of every row of `got` (torch, device) against `ref` (numpy fp64)."""
    got = got.double().cpu().numpy()
    assert got.shape == ref.shape, (name, got.shape, ref.shape)
    num = np.linalg.norm(got - ref, axis=-1)
    den = np.linalg.norm(ref, axis=-1)
    bad = np.nonzero(~(num <= tol * den))[0]
    assert bad.size == 0, f"{name}: rows {bad[:8].tolist()} off by {(num[bad] / np.maximum(den[bad], 1e-300))[:8]}"


def setup_attention_side(wl, sparsity, transposed, seed=11):
    """Compacted attention weights of layer 0 on the device (compacted by the library from seeded kept sets) in the
    equations' orientation or the transposed one, plus oracle-side CPU copies in the equations' orientation."""
    w = WL.layer_weights(wl, 0, device=DEV)
    kh = WL.kept_count(wl.d_h, sparsity)
    r = np.random.default_rng(seed)
    kept = np.concatenate([np.sort(r.choice(wl.d_h, size=kh, replace=False)) + h * wl.d_h
                           for h in range(wl.n_heads)]).astype(np.int32)
    n = len(kept)
    kd = torch.from_numpy(kept).to(DEV)
    D = wl.n_heads * wl.d_h
    c, jobs = {}, []
    names = [("wq", 0), ("wk", 0), ("wv", 0), ("wo", 1)] + ([("bq", 0), ("bk", 0), ("bv", 0)] if wl.bias else [])
    for nm, lay in names:
        c[nm] = BL.alloc_compacted(w[nm], lay, n)
        jobs.append(B.gather(w[nm], c[nm], lay, kd, n, D))
    B.ecospa_compact_tensors(jobs)
    cpu = {nm: t.cpu() for nm, t in c.items()}
    if transposed:
        npad = BL.pad8(n)
        for nm in ("wq", "wk", "wv"):
            c[nm] = c[nm][:, :n].t().contiguous()                 # n x d_m
        wo_t = torch.zeros((wl.d_m, npad), dtype=c["wo"].dtype, device=DEV)
        wo_t[:, :n] = c["wo"].t()
        c["wo"] = wo_t                                            # d_m x pitch
    return w, c, cpu, n


@pytest.mark.parametrize("name,sparsity,transposed", [
    ("gpt2m", 0.5, False), ("gpt2m", 0.5, True), ("llama1b", 0.5, False), ("llama1b", 0.5, True),
    ("llama7b_layer", 0.75, False), ("llama7b_layer", 0.25, True)])
def test_grouped_attention_side_calls_full_size(name, sparsity, transposed):
    wl = WL.WORKLOADS[name]
    T, d_m = wl.tokens, wl.d_m
    w, c, cpu, n = setup_attention_side(wl, sparsity, transposed)
    npad = BL.pad8(n)
    lay = dict(w_in_layout=B.SHARED_ROWS, w_out_layout=B.SHARED_COLS) if transposed else {}
    acts = WL.activations(wl, 0, kinds=["x", "dout", "dq", "dk", "dv", "ctx"],
                          widths={"dq": npad, "dk": npad, "dv": npad, "ctx": npad}, device=DEV)
    dt = wl.torch_dtype
    e = lambda *shape: torch.full(shape, 3.0, dtype=dt, device=DEV)
    ws = torch.empty(B.ecospa_proj_workspace_bytes(T, d_m, n, B.BF16) + 16, dtype=torch.uint8, device=DEV)
    bo = w.get("b2")                                              # a d_m-wide bias for the output projection
    Q, K, V, Out = e(T, npad), e(T, npad), e(T, npad), e(T, d_m)
    B.ecospa_coupled_qkv_fwd(acts["x"], c["wq"], c["wk"], c["wv"], n, n, Q, K, V, bq_c=c.get("bq"), bk_c=c.get("bk"),
                             bv_c=c.get("bv"), workspace=ws, **lay)
    B.ecospa_coupled_vo_fwd_o(acts["ctx"], c["wo"], n, Out, bo=bo, workspace=ws, **lay)
    dCtx = e(T, npad)
    dWo = e(d_m, npad) if transposed else e(n, d_m)
    dbo = e(d_m)
    B.ecospa_coupled_vo_bwd_o(acts["ctx"], c["wo"], n, acts["dout"], dCtx, dWo, dbo, workspace=ws, **lay)
    g = torch.Generator(device=DEV).manual_seed(5)
    dX0 = torch.randn((T, d_m), generator=g, device=DEV, dtype=torch.float32).to(dt)
    dX = dX0.clone()
    dW = {nm: (e(n, d_m) if transposed else e(d_m, npad)) for nm in ("q", "k", "v")}
    db = {nm: e(n) for nm in ("q", "k", "v")}
    B.ecospa_coupled_qkv_bwd(acts["x"], c["wq"], c["wk"], c["wv"], n, n, acts["dq"], acts["dk"], acts["dv"], dX,
                             dW["q"], dW["k"], dW["v"], db["q"], db["k"], db["v"], accumulate_dX=True, workspace=ws, **lay)
    B.ecospa_device_status()

    r = np.random.default_rng(21)
    rows = stratified(T, 256, r)
    cols = stratified(n, 256, r)
    rows_t, cols_t = torch.from_numpy(rows), torch.from_numpy(cols)
    rows_d, cols_d = rows_t.to(DEV), cols_t.to(DEV)
    Xc = acts["x"].cpu()
    Xr = Xc[rows_t].contiguous()
    up = {nm: acts["d" + nm].cpu()[:, :n].contiguous() for nm in ("q", "k", "v")}
    ctx_c = acts["ctx"].cpu()[:, :n].contiguous()
    dout_c = acts["dout"].cpu()
    # ---- sampled token rows: Q, K, V, Out, dCtx, dX (every column tile of those row blocks)
    for nm, out in (("q", Q), ("k", K), ("v", V)):
        assert_rows(nm.upper() + "[rows]", out[rows_d][:, :n], O.proj_fwd(Xr, cpu["w" + nm], O.SHARED_COLS, n, bias=cpu.get("b" + nm)))
    assert_rows("Out[rows]", Out[rows_d], O.outproj_fwd(ctx_c[rows_t].contiguous(), cpu["wo"], O.SHARED_ROWS, n, d_m,
                                                        bias=bo.cpu() if bo is not None else None))
    rdCtx, _, _ = O.outproj_bwd(ctx_c[rows_t].contiguous(), cpu["wo"], O.SHARED_ROWS, n, d_m, dout_c[rows_t].contiguous())
    assert_rows("dCtx[rows]", dCtx[rows_d][:, :n], rdCtx)
    rdX = dX0[rows_d].double().cpu().numpy()          # accumulate_dX: the product is added to what dX held
    for nm in ("q", "k", "v"):
        rdX, _, _ = O.proj_bwd(Xr, cpu["w" + nm], O.SHARED_COLS, n, up[nm][rows_t].contiguous(), dX=rdX)
    assert_rows("dX[rows]", dX[rows_d], rdX)
    # ---- sampled kept columns: dW_Q, dW_K, dW_V columns and bias gradients (every row tile of those column blocks)
    for nm in ("q", "k", "v"):
        wsub = cpu["w" + nm][:, cols_t].contiguous()
        _, rdW, rdb = O.proj_bwd(Xc, wsub, O.SHARED_COLS, len(cols), up[nm][:, cols_t].contiguous(), want_db=True)
        got = dW[nm][cols_d] if transposed else dW[nm][:, cols_d].t()
        assert_rows(f"dW{nm}[cols]", got, rdW.T)
        np.testing.assert_allclose(db[nm][cols_d].double().cpu().numpy(), rdb, rtol=TOL, atol=TOL * np.abs(rdb).max())
    # ---- sampled units of the output projection: rows of dW_O (n x d_m)
    _, rdWo, rdbo = O.outproj_bwd(ctx_c[:, cols_t].contiguous(), cpu["wo"][cols_t].contiguous(), O.SHARED_ROWS, len(cols),
                                  d_m, dout_c, want_db=True)
    got = dWo[:, cols_d].t() if transposed else dWo[cols_d]
    assert_rows("dWo[units]", got, rdWo.T)
    np.testing.assert_allclose(dbo.double().cpu().numpy(), rdbo, rtol=TOL, atol=TOL * np.abs(rdbo).max())
    # pad columns of the outputs keep what the buffers held
    if npad > n:
        assert torch.all(Q[:, n:] == 3.0) and torch.all(dCtx[:, n:] == 3.0)


@pytest.mark.parametrize("name", ["gpt2m", "llama1b"])
def test_backward_calls_are_bit_identical_from_run_to_run(name):
    """Split-K partials are added in split order and accumulated outputs receive one reducing store per element, so
    two runs on the same inputs must agree bit for bit."""
    wl = WL.WORKLOADS[name]
    T, d_m = wl.tokens, wl.d_m
    w, c, _, n = setup_attention_side(wl, 0.5, False)
    npad = BL.pad8(n)
    acts = WL.activations(wl, 0, kinds=["x", "dy", "dout", "dq", "dk", "dv", "ctx"],
                          widths={"dq": npad, "dk": npad, "dv": npad, "ctx": npad}, device=DEV)
    dt = wl.torch_dtype
    ws = torch.empty(B.ecospa_proj_workspace_bytes(T, d_m, n, B.BF16) + 16, dtype=torch.uint8, device=DEV)
    k = WL.kept_count(wl.d_ffn, 0.5)
    act = B.ACT_SWIGLU if wl.ffn == "swiglu" else B.ACT_GELU_ERF
    r = np.random.default_rng(3)
    kept_f = torch.from_numpy(np.sort(r.choice(wl.d_ffn, size=k, replace=False)).astype(np.int32)).to(DEV)
    f = {}
    jobs = []
    for nm, lay_ in (("w1", 0), ("w1b", 0), ("w2", 1), ("b1", 0)):
        if nm in w:
            f[nm] = BL.alloc_compacted(w[nm], lay_, k)
            jobs.append(B.gather(w[nm], f[nm], lay_, kept_f, k, wl.d_ffn))
    B.ecospa_compact_tensors(jobs)

    def once():
        z = lambda *shape: torch.zeros(shape, dtype=dt, device=DEV)
        o = {"dCtx": z(T, npad), "dWo": z(n, d_m), "dbo": z(d_m), "dX": torch.ones((T, d_m), dtype=dt, device=DEV),
             "dWq": z(d_m, npad), "dWk": z(d_m, npad), "dWv": z(d_m, npad), "dbq": z(n), "dbk": z(n), "dbv": z(n)}
        B.ecospa_coupled_vo_bwd_o(acts["ctx"], c["wo"], n, acts["dout"], o["dCtx"], o["dWo"], o["dbo"], workspace=ws)
        B.ecospa_coupled_qkv_bwd(acts["x"], c["wq"], c["wk"], c["wv"], n, n, acts["dq"], acts["dk"], acts["dv"], o["dX"],
                                 o["dWq"], o["dWk"], o["dWv"], o["dbq"], o["dbk"], o["dbv"], accumulate_dX=True, workspace=ws)
        buf = L.ffn_buffers(T, d_m, k, act, dt, DEV)
        for t in buf.values():
            t.zero_()
        L.ffn_fwd_bwd(acts["x"], acts["dy"], act, f["w1"], f["w2"], k, buf, w1bc=f.get("w1b"), b1c=f.get("b1"),
                      b2=w.get("b2"))
        B.ecospa_device_status()
        o.update({"ffn." + kk: v for kk, v in buf.items() if kk != "ws"})
        return o

    a, b = once(), once()
    for kk in a:
        assert torch.equal(a[kk].view(torch.int16), b[kk].view(torch.int16)), kk
