"""GPU parity of the attention core on compacted heads (through the C ABI) vs the fp64 oracle.

Tolerance: relative Frobenius error <= 2e-2 per head and sequence for Ctx and for dQ, dK, dV (bf16 operands and bf16
probabilities on the tensor cores, fp32 accumulation and softmax; the oracle works in fp64 on the same bf16 inputs);
the log-sum-exp within 2e-3 absolute.  Small cases are compared in full; the LLaMA-1B-sized case on sampled
(sequence, head) pairs, each of which is an independent sub-problem.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2511_11641_b200 import binding as B
from paper_2511_11641_b200 import block as BL
from paper_2511_11641_b200 import workloads as WL

pytestmark = pytest.mark.gpu
DEV = "cuda"
TOL = 2e-2


def make_inputs(batch, seq, k_qk, k_vo, seed=0, with_grad=False):
    """bf16 Q, K, V (and dCtx) in the padded layout: head h has k real columns followed by zero columns up to the
    next multiple of 16; a few extra columns of pitch beyond the last head hold a canary value."""
    qo, qw, nq = BL.padded_head_layout(k_qk)
    vo, vw, nv = BL.padded_head_layout(k_vo)
    T = batch * seq
    g = torch.Generator().manual_seed(seed)

    def fill(n, off, k):
        t = torch.zeros((T, n + 8), dtype=torch.bfloat16)
        for h in range(len(k)):
            t[:, off[h]: off[h] + k[h]] = torch.randn((T, k[h]), generator=g).to(torch.bfloat16)
        return t

    d = {"Q": fill(nq, qo, k_qk), "K": fill(nq, qo, k_qk), "V": fill(nv, vo, k_vo)}
    if with_grad:
        d["dCtx"] = fill(nv, vo, k_vo)
    return d, (qo, qw, nq), (vo, vw, nv)


def rel(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def run_forward(batch, seq, k_qk, k_vo, causal, seed=0, d_h=64):
    d, (qo, qw, nq), (vo, vw, nv) = make_inputs(batch, seq, k_qk, k_vo, seed)
    T = batch * seq
    dd = {k: v.to(DEV) for k, v in d.items()}
    Ctx = torch.full((T, nv + 8), 7.0, dtype=torch.bfloat16, device=DEV)
    lse = torch.full((len(k_qk) * T + 16,), -3.0, dtype=torch.float32, device=DEV)
    hd = B.heads(qo, qw, vo, vw)
    scale = 1.0 / np.sqrt(d_h)
    B.ecospa_coupled_attn_fwd(dd["Q"], dd["K"], dd["V"], batch, seq, hd, scale, causal, Ctx, lse)
    B.ecospa_device_status()
    ref = O.attn_fwd(d["Q"], d["K"], d["V"], batch, seq, qo, k_qk, vo, k_vo, scale, causal)
    got = Ctx.double().cpu().numpy()
    for h in range(len(k_qk)):
        for b in range(batch):
            rows = slice(b * seq, (b + 1) * seq)
            cols = slice(vo[h], vo[h] + k_vo[h])
            e = rel(got[rows, cols], ref["Ctx"][rows, cols])
            assert e <= TOL, f"Ctx head {h} sequence {b}: {e}"
            per_row = np.linalg.norm(got[rows, cols] - ref["Ctx"][rows, cols], axis=1) / np.linalg.norm(ref["Ctx"][rows, cols], axis=1)
            assert per_row.max() <= 3 * TOL, f"Ctx head {h} sequence {b}: worst row {per_row.argmax()} {per_row.max()}"
        # pad columns of the head come out as zeros (zero V columns), nothing else is written
        assert np.all(got[:, vo[h] + k_vo[h]: vo[h] + vw[h]] == 0)
    assert torch.all(Ctx[:, nv:] == 7.0), "columns past the last head must stay untouched"
    got_lse = lse[: len(k_qk) * T].double().cpu().numpy().reshape(len(k_qk), T)
    np.testing.assert_allclose(got_lse, ref["lse"], rtol=0, atol=2e-3)
    assert torch.all(lse[len(k_qk) * T:] == -3.0)
    return dd, d, Ctx, lse, hd, scale


RAGGED = WL.RAGGED_HEAD_KEPT      # 20, 21, 25, 26, 30, 37, 64: widths the paper's compressed GPT-2-Small shows


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("seq", [77, 128, 300])
def test_forward_ragged_heads_small(seq, causal):
    k_qk = [RAGGED[i % len(RAGGED)] for i in range(9)]
    k_vo = [RAGGED[(i + 3) % len(RAGGED)] for i in range(9)]
    run_forward(2, seq, k_qk, k_vo, causal, seed=seq)


@pytest.mark.parametrize("causal", [False, True])
def test_forward_wide_heads(causal):
    """Heads of a 128-wide architecture (LLaMA-7B shape): widths above 64 take two column blocks per tile."""
    run_forward(2, 200, [96, 128, 72, 33, 64], [128, 17, 100, 64, 80], causal, seed=5, d_h=128)


def test_forward_block_config_in_full():
    """The one-block configuration (4 heads x 64, batch 4 x seq 128, 50 %: 32 of 64 kept) in full."""
    for causal in (False, True):
        run_forward(4, 128, [32] * 4, [32] * 4, causal, seed=1)


@pytest.mark.parametrize("causal", [False, True])
def test_forward_llama1b_sized_sampled_heads(causal):
    """batch 4 x seq 2048, 32 heads with the paper's ragged widths: sampled (sequence, head) pairs in full."""
    batch, seq, H = 4, 2048, 32
    k_qk = [RAGGED[i % len(RAGGED)] for i in range(H)]
    k_vo = [RAGGED[(i + 2) % len(RAGGED)] for i in range(H)]
    d, (qo, qw, nq), (vo, vw, nv) = make_inputs(batch, seq, k_qk, k_vo, seed=11)
    T = batch * seq
    dd = {k: v.to(DEV) for k, v in d.items()}
    Ctx = torch.zeros((T, nv + 8), dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(H * T, dtype=torch.float32, device=DEV)
    scale = 0.125
    B.ecospa_coupled_attn_fwd(dd["Q"], dd["K"], dd["V"], batch, seq, B.heads(qo, qw, vo, vw), scale, causal, Ctx, lse)
    B.ecospa_device_status()
    got = Ctx.double().cpu().numpy()
    got_lse = lse.double().cpu().numpy().reshape(H, T)
    for b, h in ((0, 0), (3, 6), (1, 17), (2, 31)):
        rows = slice(b * seq, (b + 1) * seq)
        q = d["Q"][rows, qo[h]: qo[h] + k_qk[h]].contiguous()
        k = d["K"][rows, qo[h]: qo[h] + k_qk[h]].contiguous()
        v = d["V"][rows, vo[h]: vo[h] + k_vo[h]].contiguous()
        ref = O.attn_fwd(q, k, v, 1, seq, [0], [k_qk[h]], [0], [k_vo[h]], scale, causal)
        e = rel(got[rows, vo[h]: vo[h] + k_vo[h]], ref["Ctx"])
        assert e <= TOL, (b, h, e)
        np.testing.assert_allclose(got_lse[h, rows], ref["lse"][0], rtol=0, atol=2e-3)


NARROW = [20, 21, 25, 26, 30, 16, 32]      # output heads at most 32 wide take the kernel with independent key streams


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("seq", [77, 192, 500, 1000])
def test_forward_narrow_heads_several_items_per_block(seq, causal):
    """Output heads up to 32 wide, Q/K heads up to 64 wide: sequences that are not multiples of the 192-key tile, more
    (sequence, head, query tile) items than the GPU has blocks (so every block walks several items and its pipelines
    cross item boundaries), causal and not."""
    H = 40
    k_qk = [RAGGED[i % len(RAGGED)] for i in range(H)]
    k_vo = [NARROW[i % len(NARROW)] for i in range(H)]
    run_forward(3, seq, k_qk, k_vo, causal, seed=seq + 1)


@pytest.mark.parametrize("causal", [False, True])
def test_forward_scores_that_grow_along_the_sequence(causal):
    """Logits that rise by far more than 32 binary orders of magnitude along the keys (and from one 64-key slice to the
    next), so that the kernel's reference exponent has to move many times, in the middle of a slice too, with the running
    sums, the output accumulator and the probabilities already written rescaled each time; rows 3 mod 4 fall instead."""
    batch, seq, H, w = 2, 600, 5, 32
    k_qk, k_vo = [w] * H, [w] * H
    d, (qo, qw, nq), (vo, vw, nv) = make_inputs(batch, seq, k_qk, k_vo, seed=21)
    T = batch * seq
    pos = torch.arange(T) % seq
    ramp = (pos.double() / seq * 40.0 + ((pos % 97) == 0) * 25.0).to(torch.float32)        # steps and isolated spikes
    for h in range(H):
        u = torch.zeros(w)
        u[h % w] = 1.0
        d["Q"][:, qo[h]: qo[h] + w] = (torch.where((torch.arange(T) % 4 == 3)[:, None], -3.0, 3.0) * u[None, :]).to(torch.bfloat16)
        d["K"][:, qo[h]: qo[h] + w] = (d["K"][:, qo[h]: qo[h] + w].float() * 0.1 + ramp[:, None] * u[None, :]).to(torch.bfloat16)
    dd = {k: v.to(DEV) for k, v in d.items()}
    Ctx = torch.zeros((T, nv + 8), dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(H * T, dtype=torch.float32, device=DEV)
    scale = 1.0
    B.ecospa_coupled_attn_fwd(dd["Q"], dd["K"], dd["V"], batch, seq, B.heads(qo, qw, vo, vw), scale, causal, Ctx, lse)
    B.ecospa_device_status()
    ref = O.attn_fwd(d["Q"], d["K"], d["V"], batch, seq, qo, k_qk, vo, k_vo, scale, causal)
    assert np.ptp(ref["lse"]) > 100                      # the case does span far more than 2^32
    got = Ctx.double().cpu().numpy()
    assert np.all(np.isfinite(got))
    for h in range(H):
        cols = slice(vo[h], vo[h] + w)
        per_row = np.linalg.norm(got[:, cols] - ref["Ctx"][:, cols], axis=1) / np.linalg.norm(ref["Ctx"][:, cols], axis=1)
        assert per_row.max() <= 3 * TOL, (h, per_row.argmax(), per_row.max())
    np.testing.assert_allclose(lse.double().cpu().numpy().reshape(H, T), ref["lse"], rtol=2e-4, atol=2e-3)


@pytest.mark.parametrize("causal", [False, True])
def test_forward_llama1b_step_shape_sampled_heads(causal):
    """batch 4 x seq 2048, 32 heads of 32 kept columns (the benchmark's attention shape): sampled (sequence, head) pairs."""
    batch, seq, H = 4, 2048, 32
    d, (qo, qw, nq), (vo, vw, nv) = make_inputs(batch, seq, [32] * H, [32] * H, seed=12)
    T = batch * seq
    dd = {k: v.to(DEV) for k, v in d.items()}
    Ctx = torch.zeros((T, nv + 8), dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(H * T, dtype=torch.float32, device=DEV)
    scale = 0.125
    B.ecospa_coupled_attn_fwd(dd["Q"], dd["K"], dd["V"], batch, seq, B.heads(qo, qw, vo, vw), scale, causal, Ctx, lse)
    B.ecospa_device_status()
    got = Ctx.double().cpu().numpy()
    got_lse = lse.double().cpu().numpy().reshape(H, T)
    for b, h in ((0, 0), (3, 31), (1, 13)):
        rows = slice(b * seq, (b + 1) * seq)
        q = d["Q"][rows, qo[h]: qo[h] + 32].contiguous()
        k = d["K"][rows, qo[h]: qo[h] + 32].contiguous()
        v = d["V"][rows, vo[h]: vo[h] + 32].contiguous()
        ref = O.attn_fwd(q, k, v, 1, seq, [0], [32], [0], [32], scale, causal)
        assert rel(got[rows, vo[h]: vo[h] + 32], ref["Ctx"]) <= TOL, (b, h)
        np.testing.assert_allclose(got_lse[h, rows], ref["lse"][0], rtol=0, atol=2e-3)


# ---------------------------------------------------------------------------------------------
# backward
# ---------------------------------------------------------------------------------------------

def run_backward(batch, seq, k_qk, k_vo, causal, seed=0, d_h=64):
    d, (qo, qw, nq), (vo, vw, nv) = make_inputs(batch, seq, k_qk, k_vo, seed, with_grad=True)
    T, H = batch * seq, len(k_qk)
    dd = {k: v.to(DEV) for k, v in d.items()}
    Ctx = torch.zeros((T, nv + 8), dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(H * T, dtype=torch.float32, device=DEV)
    hd = B.heads(qo, qw, vo, vw)
    scale = 1.0 / np.sqrt(d_h)
    B.ecospa_coupled_attn_fwd(dd["Q"], dd["K"], dd["V"], batch, seq, hd, scale, causal, Ctx, lse)
    full = lambda n: torch.full((T, n + 8), 7.0, dtype=torch.bfloat16, device=DEV)
    dQ, dK, dV = full(nq), full(nq), full(nv)
    ws = torch.empty(B.ecospa_attn_workspace_bytes(batch, seq, H), dtype=torch.uint8, device=DEV)
    B.ecospa_coupled_attn_bwd(dd["Q"], dd["K"], dd["V"], Ctx, dd["dCtx"], lse, batch, seq, hd, scale, causal, dQ, dK, dV, ws)
    B.ecospa_device_status()
    ref = O.attn_bwd(d["Q"], d["K"], d["V"], d["dCtx"], batch, seq, qo, k_qk, vo, k_vo, scale, causal)
    for name, got_t, off, k, wpad, n in (("dQ", dQ, qo, k_qk, qw, nq), ("dK", dK, qo, k_qk, qw, nq), ("dV", dV, vo, k_vo, vw, nv)):
        got = got_t.double().cpu().numpy()
        for h in range(H):
            for b in range(batch):
                rows = slice(b * seq, (b + 1) * seq)
                cols = slice(off[h], off[h] + k[h])
                e = rel(got[rows, cols], ref[name][rows, cols])
                assert e <= TOL, f"{name} head {h} sequence {b}: {e}"
            assert np.all(got[:, off[h] + k[h]: off[h] + wpad[h]] == 0), f"{name}: pad columns of head {h}"
        assert torch.all(got_t[:, n:] == 7.0), f"{name}: columns past the last head must stay untouched"
    return dQ, dK, dV


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("seq", [77, 128, 300])
def test_backward_ragged_heads_small(seq, causal):
    k_qk = [RAGGED[i % len(RAGGED)] for i in range(9)]
    k_vo = [RAGGED[(i + 3) % len(RAGGED)] for i in range(9)]
    run_backward(2, seq, k_qk, k_vo, causal, seed=seq + 1)


@pytest.mark.parametrize("causal", [False, True])
def test_backward_wide_heads(causal):
    run_backward(2, 200, [96, 128, 72, 33, 64], [128, 17, 100, 64, 80], causal, seed=6, d_h=128)


@pytest.mark.parametrize("causal", [False, True])
def test_backward_wide_heads_several_items_per_block(causal):
    """Heads wider than 64 (the key-block kernel takes their queries 64 at a time): 3 x 9 x 6 key blocks are more items
    than resident blocks, and 650 positions leave a ragged last half block of queries."""
    k_qk = [96, 128, 72, 65, 128, 80, 112, 128, 100]
    k_vo = [128, 70, 100, 128, 66, 128, 96, 120, 128]
    a = run_backward(3, 650, k_qk, k_vo, causal, seed=11, d_h=128)
    b = run_backward(3, 650, k_qk, k_vo, causal, seed=11, d_h=128)
    for x, y in zip(a, b):
        assert torch.equal(x.view(torch.int16), y.view(torch.int16))


def test_backward_block_config_in_full_and_bit_identical_reruns():
    for causal in (False, True):
        a = run_backward(4, 128, [32] * 4, [32] * 4, causal, seed=2)
        b = run_backward(4, 128, [32] * 4, [32] * 4, causal, seed=2)
        for x, y in zip(a, b):
            assert torch.equal(x.view(torch.int16), y.view(torch.int16))


@pytest.mark.parametrize("causal", [False, True])
def test_backward_llama1b_sized_sampled_heads(causal):
    batch, seq, H = 4, 2048, 32
    k_qk = [RAGGED[i % len(RAGGED)] for i in range(H)]
    k_vo = [RAGGED[(i + 2) % len(RAGGED)] for i in range(H)]
    d, (qo, qw, nq), (vo, vw, nv) = make_inputs(batch, seq, k_qk, k_vo, seed=12, with_grad=True)
    T = batch * seq
    dd = {k: v.to(DEV) for k, v in d.items()}
    Ctx = torch.zeros((T, nv + 8), dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(H * T, dtype=torch.float32, device=DEV)
    hd = B.heads(qo, qw, vo, vw)
    scale = 0.125
    B.ecospa_coupled_attn_fwd(dd["Q"], dd["K"], dd["V"], batch, seq, hd, scale, causal, Ctx, lse)
    z = lambda n: torch.zeros((T, n + 8), dtype=torch.bfloat16, device=DEV)
    dQ, dK, dV = z(nq), z(nq), z(nv)
    ws = torch.empty(B.ecospa_attn_workspace_bytes(batch, seq, H), dtype=torch.uint8, device=DEV)
    B.ecospa_coupled_attn_bwd(dd["Q"], dd["K"], dd["V"], Ctx, dd["dCtx"], lse, batch, seq, hd, scale, causal, dQ, dK, dV, ws)
    B.ecospa_device_status()
    g = {"dQ": dQ.double().cpu().numpy(), "dK": dK.double().cpu().numpy(), "dV": dV.double().cpu().numpy()}
    for b, h in ((0, 1), (3, 13), (2, 31)):
        rows = slice(b * seq, (b + 1) * seq)
        cq, cv = slice(qo[h], qo[h] + k_qk[h]), slice(vo[h], vo[h] + k_vo[h])
        sub = lambda t, c: t[rows, c].contiguous()
        ref = O.attn_bwd(sub(d["Q"], cq), sub(d["K"], cq), sub(d["V"], cv), sub(d["dCtx"], cv), 1, seq, [0], [k_qk[h]], [0],
                         [k_vo[h]], scale, causal)
        for name, c in (("dQ", cq), ("dK", cq), ("dV", cv)):
            e = rel(g[name][rows, c], ref[name])
            assert e <= TOL, (name, b, h, e)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("seq", [50, 77, 192, 500, 1000])
def test_backward_narrow_heads_several_items_per_block(seq, causal):
    """Heads at most 32 wide: sequences that are not multiples of 64 or 128, more (sequence, head, block) items than
    resident blocks (so that a block's products run on into its next item), causal and not."""
    H = 40 if seq < 1000 else 12
    k_qk = [NARROW[(i + 1) % len(NARROW)] for i in range(H)]
    k_vo = [NARROW[i % len(NARROW)] for i in range(H)]
    run_backward(3, seq, k_qk, k_vo, causal, seed=seq + 2)


@pytest.mark.parametrize("causal", [False, True])
def test_backward_llama1b_step_shape_sampled_heads_and_reruns(causal):
    """batch 4 x seq 2048, 32 heads of 32 kept columns (the benchmark's attention shape): sampled (sequence, head) pairs
    against the oracle, and a second run bit-identical to the first."""
    batch, seq, H = 4, 2048, 32
    d, (qo, qw, nq), (vo, vw, nv) = make_inputs(batch, seq, [32] * H, [32] * H, seed=13, with_grad=True)
    T = batch * seq
    dd = {k: v.to(DEV) for k, v in d.items()}
    Ctx = torch.zeros((T, nv + 8), dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(H * T, dtype=torch.float32, device=DEV)
    hd = B.heads(qo, qw, vo, vw)
    scale = 0.125
    B.ecospa_coupled_attn_fwd(dd["Q"], dd["K"], dd["V"], batch, seq, hd, scale, causal, Ctx, lse)
    ws = torch.empty(B.ecospa_attn_workspace_bytes(batch, seq, H), dtype=torch.uint8, device=DEV)
    runs = []
    for _ in range(2):
        z = lambda n: torch.zeros((T, n + 8), dtype=torch.bfloat16, device=DEV)
        dQ, dK, dV = z(nq), z(nq), z(nv)
        B.ecospa_coupled_attn_bwd(dd["Q"], dd["K"], dd["V"], Ctx, dd["dCtx"], lse, batch, seq, hd, scale, causal, dQ, dK, dV, ws)
        B.ecospa_device_status()
        runs.append((dQ, dK, dV))
    for x, y in zip(*runs):
        assert torch.equal(x.view(torch.int16), y.view(torch.int16))
    dQ, dK, dV = runs[0]
    g = {"dQ": dQ.double().cpu().numpy(), "dK": dK.double().cpu().numpy(), "dV": dV.double().cpu().numpy()}
    for b, h in ((0, 0), (3, 31), (2, 14)):
        rows = slice(b * seq, (b + 1) * seq)
        cq, cv = slice(qo[h], qo[h] + 32), slice(vo[h], vo[h] + 32)
        sub = lambda t, c: t[rows, c].contiguous()
        ref = O.attn_bwd(sub(d["Q"], cq), sub(d["K"], cq), sub(d["V"], cv), sub(d["dCtx"], cv), 1, seq, [0], [32], [0], [32],
                         scale, causal)
        for name, c in (("dQ", cq), ("dK", cq), ("dV", cv)):
            e = rel(g[name][rows, c], ref[name])
            assert e <= TOL, (name, b, h, e)


# ---------------------------------------------------------------------------------------------
# grouped-query models: several query heads read one K/V head
# ---------------------------------------------------------------------------------------------

def run_gqa(batch, seq, k_qk_g, k_vo_g, rep, causal, seed=0, d_h=64):
    """k_qk_g / k_vo_g: kept widths per K/V group (its query heads share them).  Forward and backward against the oracle."""
    G = len(k_qk_g)
    k_qk = [k_qk_g[h // rep] for h in range(G * rep)]
    k_vo = [k_vo_g[h // rep] for h in range(G * rep)]
    qo, qw, nq = BL.padded_head_layout(k_qk)
    vo, vw, nvo = BL.padded_head_layout(k_vo)
    ko, kw, nk = BL.padded_head_layout(k_qk_g)
    vko, vkw, nv = BL.padded_head_layout(k_vo_g)
    T = batch * seq
    g = torch.Generator().manual_seed(seed)

    def fill(n, off, k):
        t = torch.zeros((T, n + 8), dtype=torch.bfloat16)
        for h in range(len(k)):
            t[:, off[h]: off[h] + k[h]] = torch.randn((T, k[h]), generator=g).to(torch.bfloat16)
        return t

    Q, dC = fill(nq, qo, k_qk), fill(nvo, vo, k_vo)
    K = torch.zeros((T, nq + 8), dtype=torch.bfloat16)          # K^c shares the pitch of Q^c
    K[:, :nk + 8] = fill(nk, ko, k_qk_g)
    V = fill(nv, vko, k_vo_g)
    dev = lambda t: t.to(DEV)
    Qd, Kd, Vd, dCd = dev(Q), dev(K), dev(V), dev(dC)
    Ctx = torch.full((T, nvo + 8), 7.0, dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(G * rep * T, dtype=torch.float32, device=DEV)
    hd = B.heads(qo, qw, vo, vw, k_off=ko, v_off=vko)
    scale = 1.0 / np.sqrt(d_h)
    B.ecospa_coupled_attn_fwd(Qd, Kd, Vd, batch, seq, hd, scale, causal, Ctx, lse)
    dQ = torch.full((T, nq + 8), 7.0, dtype=torch.bfloat16, device=DEV)
    dK = torch.full((T, nq + 8), 7.0, dtype=torch.bfloat16, device=DEV)
    dV = torch.full((T, nv + 8), 7.0, dtype=torch.bfloat16, device=DEV)
    ws = torch.empty(B.ecospa_attn_workspace_bytes(batch, seq, G * rep), dtype=torch.uint8, device=DEV)
    B.ecospa_coupled_attn_bwd(Qd, Kd, Vd, Ctx, dCd, lse, batch, seq, hd, scale, causal, dQ, dK, dV, ws)
    B.ecospa_device_status()
    ref = O.attn_fwd_gqa(Q, K, V, batch, seq, qo, k_qk, vo, k_vo, ko, vko, scale, causal)
    rb = O.attn_bwd_gqa(Q, K, V, dC, batch, seq, qo, k_qk, vo, k_vo, ko, vko, scale, causal)
    got = Ctx.double().cpu().numpy()
    for h in range(G * rep):
        for b in range(batch):
            rows = slice(b * seq, (b + 1) * seq)
            assert rel(got[rows, vo[h]: vo[h] + k_vo[h]], ref["Ctx"][rows, vo[h]: vo[h] + k_vo[h]]) <= TOL, ("Ctx", h, b)
            assert rel(dQ.double().cpu().numpy()[rows, qo[h]: qo[h] + k_qk[h]], rb["dQ"][rows, qo[h]: qo[h] + k_qk[h]]) <= TOL, ("dQ", h, b)
    np.testing.assert_allclose(lse.double().cpu().numpy().reshape(G * rep, T), ref["lse"], rtol=0, atol=2e-3)
    gK, gV = dK.double().cpu().numpy(), dV.double().cpu().numpy()
    for gi in range(G):
        for b in range(batch):
            rows = slice(b * seq, (b + 1) * seq)
            assert rel(gK[rows, ko[gi]: ko[gi] + k_qk_g[gi]], rb["dK"][rows, ko[gi]: ko[gi] + k_qk_g[gi]]) <= TOL, ("dK", gi, b)
            assert rel(gV[rows, vko[gi]: vko[gi] + k_vo_g[gi]], rb["dV"][rows, vko[gi]: vko[gi] + k_vo_g[gi]]) <= TOL, ("dV", gi, b)
    assert torch.all(dK[:, nk:] == 7.0) and torch.all(dV[:, nv:] == 7.0) and torch.all(Ctx[:, nvo:] == 7.0)
    return dQ, dK, dV


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("rep,seq", [(2, 77), (4, 300), (8, 200)])
def test_grouped_query_attention_narrow_heads(rep, seq, causal):
    """4 or 5 K/V heads with ragged kept widths up to 32 (the kernel with key streams in the forward pass)."""
    run_gqa(2, seq, [20, 32, 26, 16, 30][: 5 if rep < 8 else 4], [25, 16, 32, 21, 30][: 5 if rep < 8 else 4], rep, causal, seed=rep + seq)


@pytest.mark.parametrize("causal", [False, True])
def test_grouped_query_attention_wide_heads(causal):
    """Widths up to 64 and up to 128: the kernels with one and two 64-column blocks per tile."""
    run_gqa(2, 200, [64, 37, 48], [30, 64, 50], 4, causal, seed=3)
    run_gqa(1, 260, [128, 96], [72, 128], 2, causal, seed=4, d_h=128)


def test_grouped_query_attention_llama_shape_rerun_bit_identical():
    """8 K/V heads x 4 query heads of 32 kept columns, 2 x 1024 tokens, causal: more items than CTAs; two runs agree bit
    for bit (the sums over a group's query heads are taken by one CTA in a fixed order)."""
    a = run_gqa(2, 1024, [32] * 8, [32] * 8, 4, True, seed=5)
    b = run_gqa(2, 1024, [32] * 8, [32] * 8, 4, True, seed=5)
    for x, y in zip(a, b):
        assert torch.equal(x.view(torch.int16), y.view(torch.int16))


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("seq", [63, 65, 129])
def test_short_sequences_all_kernels(seq, causal):
    """Lengths around the 64- and 128-position block sizes; one call per kernel family: narrow (key streams), up to 64
    wide, up to 128 wide (half blocks of queries in the backward pass)."""
    for k_qk, k_vo, d_h in (([16, 30], [32, 16], 64), ([64, 40], [48, 64], 64), ([128, 80], [96, 128], 128)):
        run_forward(2, seq, k_qk, k_vo, causal, seed=100 + seq, d_h=d_h)
        run_backward(2, seq, k_qk, k_vo, causal, seed=200 + seq, d_h=d_h)


@pytest.mark.parametrize("causal", [False, True])
def test_two_positions(causal):
    """seq = 2.  dS = P (dP - D) cancels when one key dominates (dP of that key ~ D), and the kernels take D from the
    bf16 context rows the forward call stored, the oracle from its own fp64 ones: each D_i is off by up to 2^-8 of
    sum_c |dCtx_ic Ctx_ic|, which moves dQ_i by scale |dD_i| |sum_j P_ij K_j| <= scale |dD_i| max_j |K_j| and dK_j by
    scale |dD_i| P_ij |Q_i|.  The comparison allows for that on top of the relative tolerance; dV does not involve D."""
    for k_qk, k_vo, d_h in (([16, 30], [32, 16], 64), ([64, 40], [48, 64], 64), ([128, 80], [96, 128], 128)):
        batch, seq, H = 8, 2, len(k_qk)
        run_forward(batch, seq, k_qk, k_vo, causal, seed=7, d_h=d_h)
        d, (qo, qw, nq), (vo, vw, nv) = make_inputs(batch, seq, k_qk, k_vo, 8, with_grad=True)
        dd = {k: v.to(DEV) for k, v in d.items()}
        T = batch * seq
        Ctx = torch.zeros((T, nv), dtype=torch.bfloat16, device=DEV)
        lse = torch.zeros(H * T, dtype=torch.float32, device=DEV)
        hd = B.heads(qo, qw, vo, vw)
        scale = 1.0 / np.sqrt(d_h)
        B.ecospa_coupled_attn_fwd(dd["Q"], dd["K"], dd["V"], batch, seq, hd, scale, causal, Ctx, lse)
        dQ, dK, dV = (torch.zeros((T, n), dtype=torch.bfloat16, device=DEV) for n in (nq, nq, nv))
        ws = torch.empty(B.ecospa_attn_workspace_bytes(batch, seq, H), dtype=torch.uint8, device=DEV)
        B.ecospa_coupled_attn_bwd(dd["Q"], dd["K"], dd["V"], Ctx, dd["dCtx"], lse, batch, seq, hd, scale, causal, dQ, dK, dV, ws)
        B.ecospa_device_status()
        ref = O.attn_bwd(d["Q"], d["K"], d["V"], d["dCtx"], batch, seq, qo, k_qk, vo, k_vo, scale, causal)
        fwd = O.attn_fwd(d["Q"], d["K"], d["V"], batch, seq, qo, k_qk, vo, k_vo, scale, causal)
        Qn, Kn, dCn = (d[k].double().numpy() for k in ("Q", "K", "dCtx"))
        for h in range(H):
            cq, cv = slice(qo[h], qo[h] + k_qk[h]), slice(vo[h], vo[h] + k_vo[h])
            dD = 2.0 ** -8 * np.abs(dCn[:, cv] * fwd["Ctx"][:, cv]).sum(axis=1)          # per query position
            slack = scale * np.linalg.norm(dD) * max(np.linalg.norm(Kn[:, cq], axis=1).max(), np.linalg.norm(Qn[:, cq], axis=1).max())
            for name, got_t in (("dQ", dQ), ("dK", dK)):
                got = got_t.double().cpu().numpy()[:, cq]
                err = np.linalg.norm(got - ref[name][:, cq])
                assert err <= TOL * np.linalg.norm(ref[name][:, cq]) + slack, (name, h, err, slack)
            assert rel(dV.double().cpu().numpy()[:, cv], ref["dV"][:, cv]) <= TOL, ("dV", h)


@pytest.mark.parametrize("causal", [False, True])
def test_single_position(causal):
    """seq = 1: the softmax is over one key, so Ctx = V, dV = dCtx and dQ = dK = 0 (dS = P (dP - D) with P = 1 and
    D = dP); the kernels get the zeros only up to the rounding of two differently ordered fp32 sums."""
    for k_qk, k_vo, d_h in (([16, 30], [32, 16], 64), ([64, 40], [48, 64], 64), ([128, 80], [96, 128], 128)):
        batch, seq, H = 3, 1, len(k_qk)
        run_forward(batch, seq, k_qk, k_vo, causal, seed=5, d_h=d_h)
        d, (qo, qw, nq), (vo, vw, nv) = make_inputs(batch, seq, k_qk, k_vo, 6, with_grad=True)
        dd = {k: v.to(DEV) for k, v in d.items()}
        T = batch * seq
        Ctx = torch.zeros((T, nv), dtype=torch.bfloat16, device=DEV)
        lse = torch.zeros(H * T, dtype=torch.float32, device=DEV)
        hd = B.heads(qo, qw, vo, vw)
        scale = 1.0 / np.sqrt(d_h)
        B.ecospa_coupled_attn_fwd(dd["Q"], dd["K"], dd["V"], batch, seq, hd, scale, causal, Ctx, lse)
        dQ, dK, dV = (torch.zeros((T, n), dtype=torch.bfloat16, device=DEV) for n in (nq, nq, nv))
        ws = torch.empty(B.ecospa_attn_workspace_bytes(batch, seq, H), dtype=torch.uint8, device=DEV)
        B.ecospa_coupled_attn_bwd(dd["Q"], dd["K"], dd["V"], Ctx, dd["dCtx"], lse, batch, seq, hd, scale, causal, dQ, dK, dV, ws)
        B.ecospa_device_status()
        for h in range(H):
            cv = slice(vo[h], vo[h] + k_vo[h])
            assert torch.equal(Ctx[:, cv].cpu(), d["V"][:, cv]), "Ctx = V"
            assert torch.equal(dV[:, cv].cpu(), d["dCtx"][:, cv]), "dV = dCtx"
        big = float(d["dCtx"].double().abs().max() * d["V"].double().abs().max() * max(max(k_vo), 1))
        assert float(dQ.double().abs().max()) <= 1e-5 * big and float(dK.double().abs().max()) <= 1e-5 * big


@pytest.mark.parametrize("causal", [False, True])
def test_long_sequence_and_many_heads(causal):
    """One sequence of 6000 positions (not a multiple of any tile size; 32 slices per stream in the narrow-head forward
    kernel, 47 blocks in the others) on two heads, forward and backward, in full; and 128 heads (the most the descriptor
    takes) on a short one."""
    run_backward(1, 6000, [32, 20], [32, 26], causal, seed=31)
    run_forward(1, 6000, [64, 37], [64, 48], causal, seed=32)
    run_forward(1, 130, [16] * 128, [16] * 128, causal, seed=33)
    run_backward(1, 130, [16] * 128, [16] * 128, causal, seed=34)
