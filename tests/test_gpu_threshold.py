"""GPU parity of Algorithm 1's variable-count steps through the C ABI vs the CPU oracle.

Kept counts and kept index sets are integers: they must match the oracle exactly, except where the decision
falls inside the fp64 summation noise (the GPU adds the scores of a segment in a different order): a count may
then differ by one, and only if the sum of the kept scores is within 1e-9 (relative to the segment total) of
the budget.  Such a case is not expected on these inputs and is reported by the assertion message.
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


def run_case(ups_np, n_seg, seg_len, theta, l1, k_min, chosen_np=None, rope=None):
    """ups_np: concatenated scores; n_seg / seg_len: per pair.  Returns nothing; asserts parity."""
    ups = torch.from_numpy(ups_np).to(DEV)
    total_segs = sum(n_seg)
    D = sum(a * b for a, b in zip(n_seg, seg_len))
    kept = torch.full((D,), -7, dtype=torch.int32, device=DEV)
    k_out = torch.full((total_segs,), -1, dtype=torch.int32, device=DEV)
    chosen = torch.from_numpy(chosen_np).to(DEV) if chosen_np is not None else None
    B.ecospa_select_aligned_threshold(ups, n_seg, seg_len, theta, kept, k_out, l1=l1, k_min=k_min, chosen=chosen, rope=rope)
    torch.cuda.synchronize()
    k_gpu = k_out.cpu().numpy()
    kept_gpu = kept.cpu().numpy()
    off, seg = 0, 0
    for pi, (ns, sl) in enumerate(zip(n_seg, seg_len)):
        u = ups_np[off:off + ns * sl]
        ch = chosen_np[seg:seg + ns] if chosen_np is not None else None
        rp = rope[pi] if rope is not None else 0
        k_ref = O.threshold_counts(u, ns, sl, theta, l1=l1, k_min=k_min, chosen=ch, rope=rp)
        for s in range(ns):
            kg, kr = int(k_gpu[seg + s]), int(k_ref[s])
            if kg != kr:
                assert rp == 0, (seg + s, kg, kr)
                v = np.sort(u[s * sl:(s + 1) * sl].astype(np.float64))[::-1]
                total = v.sum() if l1 else 1.0
                gap = min(abs(v[:kk].sum() - theta * total) for kk in (kg, kr))
                assert abs(kg - kr) == 1 and gap <= 1e-9 * max(total, 1e-300), (seg + s, kg, kr, gap)
            # the kept indices are the top-k of the segment, ascending, relative to the pair group
            if rp:
                want = O.select_rotation_pairs(u[s * sl:(s + 1) * sl], 1, sl, [kg], rp) + s * sl
            else:
                want = O.select_topk(u[s * sl:(s + 1) * sl], 1, sl, [kg]) + s * sl
            got = kept_gpu[off + s * sl: off + s * sl + kg]
            assert np.array_equal(got, want), (seg + s, kg)
            assert (kept_gpu[off + s * sl + kg: off + (s + 1) * sl] == -7).all()     # rest of the slot untouched
        off += ns * sl
        seg += ns


def test_threshold_on_scored_llama_layer():
    """Scores of a LLaMA-1B-shaped layer (32 heads of 64 twice, one 5632-wide FFN pair), theta = 0.9 and 0.5."""
    wl = WL.WORKLOADS["llama1b"]
    w = WL.layer_weights(wl, 0, device=DEV)
    pairs = BL.block_pairs(w, wl.n_heads, wl.d_h, wl.d_ffn, None)
    D = 2 * wl.n_heads * wl.d_h + wl.d_ffn
    ups = torch.empty(D, dtype=torch.float32, device=DEV)
    B.ecospa_score_pairs(pairs, float(wl.tokens), ups, None, None)
    u = ups.cpu().numpy()
    n_seg, seg_len = [wl.n_heads, wl.n_heads, 1], [wl.d_h, wl.d_h, wl.d_ffn]
    for theta in (0.9, 0.5):
        run_case(u, n_seg, seg_len, theta, True, 1)
    run_case(u, n_seg, seg_len, 0.9, False, 8)           # l2-normalised scores compared as stored: strips to k_min or so
    r = np.random.default_rng(1)
    chosen = (r.random(2 * wl.n_heads + 1) < 0.3).astype(np.int32)
    run_case(u, n_seg, seg_len, 0.85, True, 1, chosen)


def test_threshold_degenerate_segments():
    r = np.random.default_rng(2)
    # all-equal scores (every removal is a tie), a zero segment, a heavy-tailed one, a wide one with repeats
    eq = np.full(64, 0.125, dtype=np.float32)
    zero = np.zeros(64, dtype=np.float32)
    heavy = (r.random(64).astype(np.float32) * np.where(r.random(64) < 0.05, 100.0, 1.0)).astype(np.float32)
    wide = r.integers(0, 50, size=11008).astype(np.float32) / 64.0
    u = np.concatenate([eq, zero, heavy, wide])
    for theta in (0.0, 0.3, 0.75, 0.999, 1.0, 1.5):
        run_case(u, [3, 1], [64, 11008], theta, True, 1)
        run_case(u, [3, 1], [64, 11008], theta, True, 0)
    run_case(u, [3, 1], [64, 11008], 2.0, False, 4)


def test_choose_pairs_matches_oracle():
    r = np.random.default_rng(3)
    for n in (1, 7, 792, 5000):
        f = r.random(n).astype(np.float32)
        if n > 10:
            f[5] = f[2]; f[9] = f[2]
        fd = torch.from_numpy(f).to(DEV)
        for m in (0, 1, int(round(0.3 * n)), n):
            ch = torch.full((n,), -1, dtype=torch.int32, device=DEV)
            B.ecospa_choose_pairs(fd, m, ch)
            assert np.array_equal(ch.cpu().numpy(), O.choose_pairs(f, m))


@pytest.mark.parametrize("mode", [B.ROPE_INTERLEAVED, B.ROPE_HALF])
def test_threshold_on_rotation_pairs(mode):
    """Q/K group scored with rotation pairs, V/O group plain, in one call."""
    wl = WL.WORKLOADS["llama1b"]
    w = WL.layer_weights(wl, 0, device=DEV)
    h, d_h = wl.n_heads, wl.d_h
    pairs = [B.pair(B.PAIR_PLAIN, h, d_h, w["wq"], w["wk"], B.SHARED_COLS, B.SHARED_COLS, rope=mode),
             B.pair(B.PAIR_PLAIN, h, d_h, w["wv"], w["wo"], B.SHARED_COLS, B.SHARED_ROWS)]
    ups = torch.empty(2 * h * d_h, dtype=torch.float32, device=DEV)
    B.ecospa_score_pairs(pairs, float(wl.tokens), ups, None, None)
    u = ups.cpu().numpy()
    for theta, k_min in ((0.9, 1), (0.6, 5), (1e-6, 3)):
        run_case(u, [h, h], [d_h, d_h], theta, True, k_min, rope=[mode, B.ROPE_NONE])
