"""GPU parity of the compacted-pair forward/backward calls (through the C ABI) vs the fp64 oracle.

Tolerance: relative Frobenius error <= 2e-2 per output tensor (bf16 tensor-core operands, fp32
accumulation, bf16 rounding of the saved activations; the oracle keeps everything in fp64).
Small workloads are compared in full; full-size workloads on sampled token rows (every output row
is an independent function of its input row) and sampled hidden units / kept columns (every
weight-gradient column is an independent function of that unit's weights).
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


def rel(got, ref, th=32, tw=64):
    """Relative Frobenius error of the whole tensor, and for 2-D outputs also of every th x tw tile (the unit one
    epilogue warp stores), so that a single wrong tile cannot hide in the norm of a large tensor; returns the larger.
    A tile's denominator is floored at half of what a tile of average magnitude would have (edge tiles with a few
    columns, tiles that happen to be small)."""
    got = got.double().cpu().numpy() if isinstance(got, torch.Tensor) else got
    whole = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))
    if got.ndim != 2:
        return whole
    R, Cn = ref.shape
    rp, cp = -(-R // th) * th, -(-Cn // tw) * tw
    d2 = np.zeros((rp, cp)); d2[:R, :Cn] = (got - ref) ** 2
    r2 = np.zeros((rp, cp)); r2[:R, :Cn] = ref ** 2
    num = np.sqrt(d2.reshape(rp // th, th, cp // tw, tw).sum(axis=(1, 3)))
    den = np.sqrt(r2.reshape(rp // th, th, cp // tw, tw).sum(axis=(1, 3)))
    floor = 0.5 * np.sqrt(r2.sum() / max(R * Cn, 1) * th * tw)
    tiles = float((num / np.maximum(den, max(floor, 1e-300))).max())
    return max(whole, tiles)


def check(errs):
    bad = {k: v for k, v in errs.items() if not v <= TOL}
    assert not bad, f"relative Frobenius error above {TOL}: {bad} (all: {errs})"


def compact_cpu(w, kept, ld_elems):
    """Oracle-side compaction of the tensors of a block for given kept lists (dict of torch CPU tensors)."""
    out = {}
    for nm in ("wq", "wk", "wv"):
        out[nm] = O.compact(w[nm], O.SHARED_COLS, kept["attn"], ld_out=ld_elems(len(kept["attn"])))
    out["wo"] = O.compact(w["wo"], O.SHARED_ROWS, kept["attn"])
    out["w1"] = O.compact(w["w1"], O.SHARED_COLS, kept["ffn"], ld_out=ld_elems(len(kept["ffn"])))
    if "w1b" in w:
        out["w1b"] = O.compact(w["w1b"], O.SHARED_COLS, kept["ffn"], ld_out=ld_elems(len(kept["ffn"])))
    out["w2"] = O.compact(w["w2"], O.SHARED_ROWS, kept["ffn"])
    for nm, key in (("bq", "attn"), ("bk", "attn"), ("bv", "attn"), ("b1", "ffn")):
        if nm in w:
            out[nm] = O.compact(w[nm], O.SHARED_COLS, kept[key], ld_out=ld_elems(len(kept[key])))
    if "b2" in w:
        out["b2"] = w["b2"]
    return out


def random_kept(wl, k_heads, k_ffn, seed):
    r = np.random.default_rng(seed)
    attn = np.concatenate([np.sort(r.choice(wl.d_h, size=kh, replace=False)) + h * wl.d_h
                           for h, kh in enumerate(k_heads)]).astype(np.int32)
    ffn = np.sort(r.choice(wl.d_ffn, size=k_ffn, replace=False)).astype(np.int32)
    return {"attn": attn, "ffn": ffn}


def run_block_full(wl, k_heads, k_ffn, act, T=None, seed=0):
    """All layer calls on one block, compared in full against the oracle."""
    eb = wl.elem_bytes
    w = WL.layer_weights(wl, 0)
    kept = random_kept(wl, k_heads, k_ffn, seed)
    n, k = len(kept["attn"]), len(kept["ffn"])
    wc = compact_cpu(w, kept, lambda m: BL.pad8(m, eb))
    T = T or wl.tokens
    npad = BL.pad8(n, eb)
    acts = WL.activations(wl, 0, tokens=T, kinds=["x", "dy", "dout", "dq", "dk", "dv", "ctx"],
                          widths={"dq": npad, "dk": npad, "dv": npad, "ctx": npad})
    d = {kk: v.to(DEV) for kk, v in wc.items()}
    a = {kk: v.to(DEV) for kk, v in acts.items()}
    dt = wl.torch_dtype
    code = B.F32 if dt == torch.float32 else B.BF16
    ws = torch.empty(B.ecospa_proj_workspace_bytes(T, wl.d_m, n, code) + 16, dtype=torch.uint8, device=DEV)
    errs = {}

    # ---- QK
    Q = torch.full((T, npad), 5.0, dtype=dt, device=DEV); K = torch.full((T, npad), 5.0, dtype=dt, device=DEV)
    B.ecospa_coupled_qk_fwd(a["x"], d["wq"], d["wk"], n, Q, K, bq_c=d.get("bq"), bk_c=d.get("bk"), workspace=ws)
    errs["Q"] = rel(Q[:, :n], O.proj_fwd(acts["x"], wc["wq"], O.SHARED_COLS, n, bias=wc.get("bq")))
    errs["K"] = rel(K[:, :n], O.proj_fwd(acts["x"], wc["wk"], O.SHARED_COLS, n, bias=wc.get("bk")))
    assert torch.all(torch.isfinite(Q.float())), "pad columns may be rewritten, but only with finite values"
    dX = torch.empty((T, wl.d_m), dtype=dt, device=DEV)
    dWq = torch.zeros_like(d["wq"]); dWk = torch.zeros_like(d["wk"])
    dbq = torch.empty(n, dtype=dt, device=DEV); dbk = torch.empty(n, dtype=dt, device=DEV)
    B.ecospa_coupled_qk_bwd(a["x"], d["wq"], d["wk"], n, a["dq"], a["dk"], dX, dWq, dWk, dbq, dbk, workspace=ws)
    dq_c, dk_c = acts["dq"][:, :n].contiguous(), acts["dk"][:, :n].contiguous()
    rdX, rdWq, rdbq = O.proj_bwd(acts["x"], wc["wq"], O.SHARED_COLS, n, dq_c, want_db=True)
    rdX, rdWk, rdbk = O.proj_bwd(acts["x"], wc["wk"], O.SHARED_COLS, n, dk_c, want_db=True, dX=rdX)
    errs["qk.dX"] = rel(dX, rdX); errs["dWq"] = rel(dWq[:, :n], rdWq); errs["dWk"] = rel(dWk[:, :n], rdWk)
    errs["dbq"] = rel(dbq, rdbq); errs["dbk"] = rel(dbk, rdbk)
    # accumulate_dX adds on top of what is there
    dX2 = dX.clone()
    B.ecospa_coupled_qk_bwd(a["x"], d["wq"], d["wk"], n, a["dq"], a["dk"], dX2, dWq, dWk, accumulate_dX=True, workspace=ws)
    errs["qk.dX(acc)"] = rel(dX2, 2 * rdX)

    # ---- VO
    V = torch.empty((T, npad), dtype=dt, device=DEV)
    B.ecospa_coupled_vo_fwd_v(a["x"], d["wv"], n, V, bv_c=d.get("bv"), workspace=ws)
    errs["V"] = rel(V[:, :n], O.proj_fwd(acts["x"], wc["wv"], O.SHARED_COLS, n, bias=wc.get("bv")))
    Out = torch.empty((T, wl.d_m), dtype=dt, device=DEV)
    B.ecospa_coupled_vo_fwd_o(a["ctx"], d["wo"], n, Out, workspace=ws)
    ctx_cpu = acts["ctx"][:, :n].contiguous()
    errs["Out"] = rel(Out, O.outproj_fwd(ctx_cpu, wc["wo"], O.SHARED_ROWS, n, wl.d_m))
    dCtx = torch.full((T, npad), 5.0, dtype=dt, device=DEV)
    dWv = torch.zeros_like(d["wv"]); dWo = torch.empty_like(d["wo"])
    dbv = torch.empty(n, dtype=dt, device=DEV); dbo = torch.empty(wl.d_m, dtype=dt, device=DEV)
    B.ecospa_coupled_vo_bwd(a["x"], a["ctx"], d["wv"], d["wo"], n, a["dv"], a["dout"], dX, dCtx, dWv, dWo, dbv, dbo,
                            workspace=ws)
    rdCtx, rdWo, rdbo = O.outproj_bwd(ctx_cpu, wc["wo"], O.SHARED_ROWS, n, wl.d_m, acts["dout"], want_db=True)
    rdXv, rdWv, rdbv = O.proj_bwd(acts["x"], wc["wv"], O.SHARED_COLS, n, acts["dv"][:, :n].contiguous(), want_db=True)
    errs["dCtx"] = rel(dCtx[:, :n], rdCtx); errs["dWo"] = rel(dWo, rdWo.T); errs["dbo"] = rel(dbo, rdbo)
    errs["vo.dX"] = rel(dX, rdXv); errs["dWv"] = rel(dWv[:, :n], rdWv); errs["dbv"] = rel(dbv, rdbv)

    # ---- the same attention-side products through the grouped calls (one launch each)
    Q2 = torch.empty_like(Q); K2 = torch.empty_like(K); V2 = torch.empty_like(V)
    B.ecospa_coupled_qkv_fwd(a["x"], d["wq"], d["wk"], d["wv"], n, n, Q2, K2, V2, bq_c=d.get("bq"), bk_c=d.get("bk"),
                             bv_c=d.get("bv"), workspace=ws)
    errs["qkv.Q"] = rel(Q2[:, :n], O.proj_fwd(acts["x"], wc["wq"], O.SHARED_COLS, n, bias=wc.get("bq")))
    errs["qkv.K"] = rel(K2[:, :n], O.proj_fwd(acts["x"], wc["wk"], O.SHARED_COLS, n, bias=wc.get("bk")))
    errs["qkv.V"] = rel(V2[:, :n], O.proj_fwd(acts["x"], wc["wv"], O.SHARED_COLS, n, bias=wc.get("bv")))
    dCtx2 = torch.empty_like(dCtx); dWo2 = torch.empty_like(dWo); dbo2 = torch.empty_like(dbo)
    B.ecospa_coupled_vo_bwd_o(a["ctx"], d["wo"], n, a["dout"], dCtx2, dWo2, dbo2, workspace=ws)
    errs["vo_o.dCtx"] = rel(dCtx2[:, :n], rdCtx); errs["vo_o.dWo"] = rel(dWo2, rdWo.T); errs["vo_o.dbo"] = rel(dbo2, rdbo)
    dX3 = torch.empty_like(dX)
    dWq3 = torch.zeros_like(dWq); dWk3 = torch.zeros_like(dWk); dWv3 = torch.zeros_like(dWv)
    dbq3 = torch.empty_like(dbq); dbk3 = torch.empty_like(dbk); dbv3 = torch.empty_like(dbv)
    B.ecospa_coupled_qkv_bwd(a["x"], d["wq"], d["wk"], d["wv"], n, n, a["dq"], a["dk"], a["dv"], dX3, dWq3, dWk3, dWv3,
                             dbq3, dbk3, dbv3, workspace=ws)
    errs["qkv.dX"] = rel(dX3, rdX + rdXv)
    errs["qkv.dWq"] = rel(dWq3[:, :n], rdWq); errs["qkv.dWk"] = rel(dWk3[:, :n], rdWk); errs["qkv.dWv"] = rel(dWv3[:, :n], rdWv)
    errs["qkv.dbq"] = rel(dbq3, rdbq); errs["qkv.dbk"] = rel(dbk3, rdbk); errs["qkv.dbv"] = rel(dbv3, rdbv)
    dX4 = torch.empty_like(dX); dWv4 = torch.zeros_like(dWv)
    B.ecospa_coupled_vo_bwd_v(a["x"], d["wv"], n, a["dv"], dX4, dWv4, workspace=ws)
    errs["vo_v.dX"] = rel(dX4, rdXv); errs["vo_v.dWv"] = rel(dWv4[:, :n], rdWv)

    # ---- FFN
    sw = act == B.ACT_SWIGLU
    buf = L.ffn_buffers(T, wl.d_m, k, act, dt, DEV)
    L.ffn_fwd_bwd(a["x"], a["dy"], act, d["w1"], d["w2"], k, buf, w1bc=d.get("w1b"),
                  b1c=None if sw else d.get("b1"), b2=None if sw else d.get("b2"))
    B.ecospa_device_status()
    b1 = None if sw else wc.get("b1")
    b2 = None if sw else wc.get("b2")
    rf = O.ffn_fwd(acts["x"], act, wc["w1"], wc["w2"], O.SHARED_COLS, O.SHARED_ROWS, k, W1b=wc.get("w1b"), b1=b1, b2=b2)
    rb = O.ffn_bwd(acts["x"], act, wc["w1"], wc["w2"], O.SHARED_COLS, O.SHARED_ROWS, k, acts["dy"], W1b=wc.get("w1b"),
                   b1=b1, want_bias=True)
    errs["Y"] = rel(buf["Y"], rf["Y"]); errs["H"] = rel(buf["H"][:, :k], rf["H"]); errs["A"] = rel(buf["A"][:, :k], rf["A"])
    errs["ffn.dX"] = rel(buf["dX"], rb["dX"]); errs["dW1"] = rel(buf["dW1"][:, :k], rb["dW1"])
    errs["dW2"] = rel(buf["dW2"], rb["dW2"].T); errs["db2"] = rel(buf["db2"], rb["db2"])
    if sw:
        errs["Hb"] = rel(buf["Hb"][:, :k], rf["Hb"]); errs["dW1b"] = rel(buf["dW1b"][:, :k], rb["dW1b"])
    else:
        errs["db1"] = rel(buf["db1"], rb["db1"])
    check(errs)
    return errs


def test_block_f32_full_forward_backward():
    wl = WL.WORKLOADS["block_f32"]
    kh = WL.kept_count(wl.d_h, 0.5)
    run_block_full(wl, [kh] * wl.n_heads, WL.kept_count(wl.d_ffn, 0.5), B.ACT_GELU_ERF)


def test_tiny_swiglu_full_forward_backward():
    wl = WL.WORKLOADS["tiny_swiglu"]
    run_block_full(wl, [16, 16], 80, B.ACT_SWIGLU)
    run_block_full(wl, [13, 6], 77, B.ACT_SWIGLU, seed=1)      # kept counts that are not multiples of 8


@pytest.mark.parametrize("k_ffn", [1073, 1337])
def test_ragged_kept_counts_gelu(k_ffn):
    """Per-head widths and FFN widths the paper's compressed GPT-2-Small shows; T spans 2.5 row tiles."""
    wl = WL.WORKLOADS["tails768"]
    k_heads = [WL.RAGGED_HEAD_KEPT[i % len(WL.RAGGED_HEAD_KEPT)] for i in range(wl.n_heads)]
    run_block_full(wl, k_heads, k_ffn, B.ACT_GELU_ERF)


def test_token_counts_that_end_inside_a_row_block():
    """T = 333 and T = 77 end inside a 32-row warp block: the tile stores clip the rows past T, the saved
    activations of the last block are fetched element by element, and accumulation must not touch them."""
    wl = WL.WORKLOADS["tails768"]
    k_heads = [WL.RAGGED_HEAD_KEPT[i % len(WL.RAGGED_HEAD_KEPT)] for i in range(wl.n_heads)]
    run_block_full(wl, k_heads, 1073, B.ACT_GELU_ERF, T=333)
    wl = WL.WORKLOADS["tiny_swiglu"]
    run_block_full(wl, [13, 6], 77, B.ACT_SWIGLU, T=77, seed=2)


def run_block_other_orientation(wl, k_heads, k_ffn, act, T=None, seed=0):
    """The same products with every weight stored the other way round (W_Q, W_K, W_V, W_1 as n x d_m, i.e. the
    nn.Linear layout; W_O, W_2 as d_m x n): outputs must not change and weight gradients come back in the
    orientation of their weight."""
    eb = wl.elem_bytes
    w = WL.layer_weights(wl, 0)
    kept = random_kept(wl, k_heads, k_ffn, seed)
    n, k = len(kept["attn"]), len(kept["ffn"])
    wc = compact_cpu(w, kept, lambda m: BL.pad8(m, eb))
    T = T or wl.tokens
    npad, kpad = BL.pad8(n, eb), BL.pad8(k, eb)
    acts = WL.activations(wl, 0, tokens=T, kinds=["x", "dy", "dout", "dq", "dk", "dv", "ctx"],
                          widths={"dq": npad, "dk": npad, "dv": npad, "ctx": npad})
    a = {kk: v.to(DEV) for kk, v in acts.items()}
    dt = wl.torch_dtype

    def rows(t, m):            # d_m x pitch  ->  m x d_m
        return t[:, :m].t().contiguous().to(DEV)

    def cols(t, m, pad):       # m x d_m  ->  d_m x pitch, pad columns zero
        o = torch.zeros((t.shape[1], pad), dtype=t.dtype)
        o[:, :m] = t.t()
        return o.to(DEV)

    d = {"wq": rows(wc["wq"], n), "wk": rows(wc["wk"], n), "wv": rows(wc["wv"], n), "wo": cols(wc["wo"], n, npad),
         "w1": rows(wc["w1"], k), "w2": cols(wc["w2"], k, kpad)}
    if "w1b" in wc:
        d["w1b"] = rows(wc["w1b"], k)
    bias = {nm: wc[nm].to(DEV) for nm in ("bq", "bk", "bv", "b1", "b2") if nm in wc}
    code = B.F32 if dt == torch.float32 else B.BF16
    ws = torch.empty(B.ecospa_proj_workspace_bytes(T, wl.d_m, n, code) + 16, dtype=torch.uint8, device=DEV)
    lay = dict(w_in_layout=B.SHARED_ROWS, w_out_layout=B.SHARED_COLS)
    errs = {}
    e = lambda *shape: torch.full(shape, 3.0, dtype=dt, device=DEV)

    Q, K, V = e(T, npad), e(T, npad), e(T, npad)
    B.ecospa_coupled_qkv_fwd(a["x"], d["wq"], d["wk"], d["wv"], n, n, Q, K, V, bq_c=bias.get("bq"), bk_c=bias.get("bk"),
                             bv_c=bias.get("bv"), workspace=ws, **lay)
    for nm, out in (("q", Q), ("k", K), ("v", V)):
        errs[nm.upper()] = rel(out[:, :n], O.proj_fwd(acts["x"], wc["w" + nm], O.SHARED_COLS, n, bias=wc.get("b" + nm)))
    Out = e(T, wl.d_m)
    B.ecospa_coupled_vo_fwd_o(a["ctx"], d["wo"], n, Out, workspace=ws, **lay)
    ctx_cpu = acts["ctx"][:, :n].contiguous()
    errs["Out"] = rel(Out, O.outproj_fwd(ctx_cpu, wc["wo"], O.SHARED_ROWS, n, wl.d_m))

    dCtx, dWo, dbo = e(T, npad), e(wl.d_m, npad), e(wl.d_m)
    B.ecospa_coupled_vo_bwd_o(a["ctx"], d["wo"], n, a["dout"], dCtx, dWo, dbo, workspace=ws, **lay)
    rdCtx, rdWo, rdbo = O.outproj_bwd(ctx_cpu, wc["wo"], O.SHARED_ROWS, n, wl.d_m, acts["dout"], want_db=True)
    errs["dCtx"] = rel(dCtx[:, :n], rdCtx); errs["dWo"] = rel(dWo[:, :n], rdWo); errs["dbo"] = rel(dbo, rdbo)

    dX = e(T, wl.d_m)
    dWq, dWk, dWv = e(n, wl.d_m), e(n, wl.d_m), e(n, wl.d_m)
    B.ecospa_coupled_qkv_bwd(a["x"], d["wq"], d["wk"], d["wv"], n, n, a["dq"], a["dk"], a["dv"], dX, dWq, dWk, dWv,
                             workspace=ws, **lay)
    ref_dx = None
    for nm, dW in (("q", dWq), ("k", dWk), ("v", dWv)):
        up = acts["d" + nm][:, :n].contiguous()
        ref_dx, rdW, _ = O.proj_bwd(acts["x"], wc["w" + nm], O.SHARED_COLS, n, up, dX=ref_dx)
        errs["dW" + nm] = rel(dW, rdW.T)
    errs["dX"] = rel(dX, ref_dx)

    sw = act == B.ACT_SWIGLU
    buf = L.ffn_buffers(T, wl.d_m, k, act, dt, DEV)
    buf["dW1"] = e(k, wl.d_m); buf["dW2"] = e(wl.d_m, kpad)
    if sw:
        buf["dW1b"] = e(k, wl.d_m)
    B.ecospa_coupled_ffn_fwd(a["x"], act, d["w1"], d["w2"], k, buf["Y"], buf["H"], buf["A"], w1b_c=d.get("w1b"),
                             Hb=buf.get("Hb"), b1_c=None if sw else bias.get("b1"), b2=None if sw else bias.get("b2"),
                             workspace=buf["ws"], **lay)
    B.ecospa_coupled_ffn_bwd(a["x"], act, d["w1"], d["w2"], k, buf["H"], buf["A"], a["dy"], buf["dX"], buf["dW1"],
                             buf["dW2"], w1b_c=d.get("w1b"), Hb=buf.get("Hb"), dW1b_c=buf.get("dW1b"),
                             db1_c=buf.get("db1"), db2=buf["db2"], workspace=buf["ws"], **lay)
    B.ecospa_device_status()
    b1 = None if sw else wc.get("b1")
    b2 = None if sw else wc.get("b2")
    rf = O.ffn_fwd(acts["x"], act, wc["w1"], wc["w2"], O.SHARED_COLS, O.SHARED_ROWS, k, W1b=wc.get("w1b"), b1=b1, b2=b2)
    rb = O.ffn_bwd(acts["x"], act, wc["w1"], wc["w2"], O.SHARED_COLS, O.SHARED_ROWS, k, acts["dy"], W1b=wc.get("w1b"),
                   b1=b1, want_bias=True)
    errs["Y"] = rel(buf["Y"], rf["Y"]); errs["A"] = rel(buf["A"][:, :k], rf["A"])
    errs["ffn.dX"] = rel(buf["dX"], rb["dX"]); errs["dW1"] = rel(buf["dW1"], rb["dW1"].T)
    errs["dW2"] = rel(buf["dW2"][:, :k], rb["dW2"])
    if sw:
        errs["dW1b"] = rel(buf["dW1b"], rb["dW1b"].T)
    else:
        errs["db1"] = rel(buf["db1"], rb["db1"])
    check(errs)


def test_weights_stored_the_other_way_round():
    wl = WL.WORKLOADS["tails768"]
    k_heads = [WL.RAGGED_HEAD_KEPT[i % len(WL.RAGGED_HEAD_KEPT)] for i in range(wl.n_heads)]
    run_block_other_orientation(wl, k_heads, 1337, B.ACT_GELU_ERF)
    wl = WL.WORKLOADS["tiny_swiglu"]
    run_block_other_orientation(wl, [13, 6], 77, B.ACT_SWIGLU, seed=1)
    wl = WL.WORKLOADS["block_f32"]
    run_block_other_orientation(wl, [32] * wl.n_heads, 512, B.ACT_GELU_ERF)


def test_gelu_tanh_variant_small():
    wl = WL.WORKLOADS["tails768"]
    run_block_full(wl, [32] * wl.n_heads, 264, B.ACT_GELU_TANH, T=96)


# ---------------------------------------------------------------------------------------------
# full-size layers, sampled outputs
# ---------------------------------------------------------------------------------------------

def run_ffn_sampled(wl, sparsity, layer=0, n_rows=12, n_units=6):
    act = B.ACT_SWIGLU if wl.ffn == "swiglu" else B.ACT_GELU_ERF
    w = WL.layer_weights(wl, layer, device=DEV)
    k = WL.kept_count(wl.d_ffn, sparsity)
    r = np.random.default_rng(7)
    kept = np.sort(r.choice(wl.d_ffn, size=k, replace=False)).astype(np.int32)
    kept_d = torch.from_numpy(kept).to(DEV)
    sw = act == B.ACT_SWIGLU
    p = B.pair(B.PAIR_SWIGLU if sw else B.PAIR_PLAIN, 1, wl.d_ffn, w["w1"], w["w2"], B.SHARED_COLS, B.SHARED_ROWS,
               w1b=w.get("w1b"))
    w1c = BL.alloc_compacted(w["w1"], B.SHARED_COLS, k); w2c = BL.alloc_compacted(w["w2"], B.SHARED_ROWS, k)
    w1bc = BL.alloc_compacted(w["w1b"], B.SHARED_COLS, k) if sw else None
    aux = []
    b1c = None
    if wl.bias:
        b1c = BL.alloc_compacted(w["b1"], B.SHARED_COLS, k)
        aux.append((w["b1"], b1c, B.SHARED_COLS))
    B.ecospa_compact_pair(p, kept_d, k, w1c, w2c, w1b_out=w1bc, aux=aux)
    T = wl.tokens
    acts = WL.activations(wl, layer, kinds=["x", "dy"], device=DEV)
    buf = L.ffn_buffers(T, wl.d_m, k, act, wl.torch_dtype, DEV)
    b2 = w.get("b2")
    L.ffn_fwd_bwd(acts["x"], acts["dy"], act, w1c, w2c, k, buf, w1bc=w1bc, b1c=b1c, b2=b2)
    B.ecospa_device_status()

    rows = np.sort(r.choice(T, size=n_rows, replace=False))
    units = np.sort(r.choice(k, size=n_units, replace=False))
    Xc, dYc = acts["x"].cpu(), acts["dy"].cpu()
    w1c_c, w2c_c = w1c.cpu(), w2c.cpu()
    w1bc_c = w1bc.cpu() if sw else None
    b1_c = b1c.cpu() if b1c is not None else None
    b2_c = b2.cpu() if b2 is not None else None
    errs = {}
    # sampled token rows: Y, A, dX
    rows_t = torch.from_numpy(rows)
    Xr, dYr = Xc[rows_t].contiguous(), dYc[rows_t].contiguous()
    rf = O.ffn_fwd(Xr, act, w1c_c, w2c_c, O.SHARED_COLS, O.SHARED_ROWS, k, W1b=w1bc_c, b1=b1_c, b2=b2_c)
    rb = O.ffn_bwd(Xr, act, w1c_c, w2c_c, O.SHARED_COLS, O.SHARED_ROWS, k, dYr, W1b=w1bc_c, b1=b1_c)
    rows_d = rows_t.to(DEV)
    errs["Y[rows]"] = rel(buf["Y"][rows_d], rf["Y"])
    errs["A[rows]"] = rel(buf["A"][rows_d][:, :k], rf["A"])
    errs["dX[rows]"] = rel(buf["dX"][rows_d], rb["dX"])
    # sampled hidden units: dW1[:, u], dW2[u, :] need every token
    units_t = torch.from_numpy(units)
    w1u = w1c_c[:, units_t].contiguous(); w2u = w2c_c[units_t].contiguous()
    w1bu = w1bc_c[:, units_t].contiguous() if sw else None
    b1u = b1_c[units_t].contiguous() if b1_c is not None else None
    ru = O.ffn_bwd(Xc, act, w1u, w2u, O.SHARED_COLS, O.SHARED_ROWS, len(units), dYc, W1b=w1bu, b1=b1u, want_bias=True)
    units_d = units_t.to(DEV)
    errs["dW1[:,units]"] = rel(buf["dW1"][:, units_d], ru["dW1"])
    errs["dW2[units]"] = rel(buf["dW2"][units_d], ru["dW2"].T)
    errs["db2"] = rel(buf["db2"], ru["db2"])
    if sw:
        errs["dW1b[:,units]"] = rel(buf["dW1b"][:, units_d], ru["dW1b"])
    else:
        errs["db1[units]"] = rel(buf["db1"][units_d], ru["db1"])
    check(errs)


def run_qk_sampled(wl, sparsity, layer=0, n_rows=12, n_cols=6):
    w = WL.layer_weights(wl, layer, device=DEV)
    kh = WL.kept_count(wl.d_h, sparsity)
    r = np.random.default_rng(9)
    kept = np.concatenate([np.sort(r.choice(wl.d_h, size=kh, replace=False)) + h * wl.d_h
                           for h in range(wl.n_heads)]).astype(np.int32)
    n = len(kept)
    kept_d = torch.from_numpy(kept).to(DEV)
    D = wl.n_heads * wl.d_h
    wqc = BL.alloc_compacted(w["wq"], B.SHARED_COLS, n); wkc = BL.alloc_compacted(w["wk"], B.SHARED_COLS, n)
    B.ecospa_compact_tensors([B.gather(w["wq"], wqc, B.SHARED_COLS, kept_d, n, D),
                              B.gather(w["wk"], wkc, B.SHARED_COLS, kept_d, n, D)])
    T = wl.tokens
    npad = BL.pad8(n)
    acts = WL.activations(wl, layer, kinds=["x", "dq", "dk"], widths={"dq": npad, "dk": npad}, device=DEV)
    dt = wl.torch_dtype
    Q = torch.empty((T, npad), dtype=dt, device=DEV); K = torch.empty((T, npad), dtype=dt, device=DEV)
    ws = torch.empty(B.ecospa_proj_workspace_bytes(T, wl.d_m, n, B.BF16) + 16, dtype=torch.uint8, device=DEV)
    B.ecospa_coupled_qk_fwd(acts["x"], wqc, wkc, n, Q, K, workspace=ws)
    dX = torch.empty((T, wl.d_m), dtype=dt, device=DEV)
    dWq = torch.zeros_like(wqc); dWk = torch.zeros_like(wkc)
    B.ecospa_coupled_qk_bwd(acts["x"], wqc, wkc, n, acts["dq"], acts["dk"], dX, dWq, dWk, workspace=ws)
    B.ecospa_device_status()
    rows = np.sort(r.choice(T, size=n_rows, replace=False)); cols = np.sort(r.choice(n, size=n_cols, replace=False))
    rows_t, cols_t = torch.from_numpy(rows), torch.from_numpy(cols)
    Xc = acts["x"].cpu(); wq_c, wk_c = wqc.cpu(), wkc.cpu()
    dq_c, dk_c = acts["dq"].cpu()[:, :n].contiguous(), acts["dk"].cpu()[:, :n].contiguous()
    errs = {}
    Xr = Xc[rows_t].contiguous()
    errs["Q[rows]"] = rel(Q[rows_t.to(DEV)][:, :n], O.proj_fwd(Xr, wq_c, O.SHARED_COLS, n))
    errs["K[rows]"] = rel(K[rows_t.to(DEV)][:, :n], O.proj_fwd(Xr, wk_c, O.SHARED_COLS, n))
    rdX, _, _ = O.proj_bwd(Xr, wq_c, O.SHARED_COLS, n, dq_c[rows_t].contiguous())
    rdX, _, _ = O.proj_bwd(Xr, wk_c, O.SHARED_COLS, n, dk_c[rows_t].contiguous(), dX=rdX)
    errs["dX[rows]"] = rel(dX[rows_t.to(DEV)], rdX)
    _, rdWq, _ = O.proj_bwd(Xc, wq_c[:, cols_t].contiguous(), O.SHARED_COLS, n_cols, dq_c[:, cols_t].contiguous())
    _, rdWk, _ = O.proj_bwd(Xc, wk_c[:, cols_t].contiguous(), O.SHARED_COLS, n_cols, dk_c[:, cols_t].contiguous())
    errs["dWq[:,cols]"] = rel(dWq[:, cols_t.to(DEV)], rdWq)
    errs["dWk[:,cols]"] = rel(dWk[:, cols_t.to(DEV)], rdWk)
    check(errs)


@pytest.mark.parametrize("name,sparsity", [("gpt2m", 0.5), ("llama1b", 0.5), ("llama7b_layer", 0.25),
                                           ("llama7b_layer", 0.5), ("llama7b_layer", 0.75)])
def test_full_size_ffn_sampled(name, sparsity):
    run_ffn_sampled(WL.WORKLOADS[name], sparsity)


@pytest.mark.parametrize("name,sparsity", [("gpt2m", 0.5), ("llama1b", 0.5), ("llama7b_layer", 0.75)])
def test_full_size_qk_sampled(name, sparsity):
    run_qk_sampled(WL.WORKLOADS[name], sparsity)
