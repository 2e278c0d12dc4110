"""GPU parity of rotation-pair (rotary position embedding) scoring and selection vs the CPU oracle.

Scores within 1e-5 relative (floor 1e-5 of the segment maximum); kept index sets bit-exact when both sides
rank the same fp32 score vector.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2511_11641_b200 import binding as B
from paper_2511_11641_b200 import workloads as WL

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("name", ["llama1b", "llama7b_layer", "tiny_swiglu"])
@pytest.mark.parametrize("mode", [B.ROPE_INTERLEAVED, B.ROPE_HALF])
def test_rotation_pair_scores_and_selection(name, mode):
    wl = WL.WORKLOADS[name]
    w = WL.layer_weights(wl, 0)
    wq, wk = w["wq"].to(DEV), w["wk"].to(DEV)
    h, d_h = wl.n_heads, wl.d_h
    D = h * d_h
    p_rope = B.pair(B.PAIR_PLAIN, h, d_h, wq, wk, B.SHARED_COLS, B.SHARED_COLS, rope=mode)
    p_vo = B.pair(B.PAIR_PLAIN, h, d_h, w["wv"].to(DEV), w["wo"].to(DEV), B.SHARED_COLS, B.SHARED_ROWS)   # a plain group beside it
    ups = torch.empty(2 * D, dtype=torch.float32, device=DEV)
    raw = torch.empty(2 * D, dtype=torch.float32, device=DEV)
    B.ecospa_score_pairs([p_rope, p_vo], float(wl.tokens), ups, raw, None)
    torch.cuda.synchronize()
    raw_o, ups_o = O.score_pair(w["wq"], w["wk"], O.SHARED_COLS, O.SHARED_COLS, h, d_h, rope=mode)
    raw_v, ups_v = O.score_pair(w["wv"], w["wo"], O.SHARED_COLS, O.SHARED_ROWS, h, d_h)
    for got, ref in ((ups[:D], ups_o), (raw[:D], raw_o), (ups[D:], ups_v), (raw[D:], raw_v)):
        g = got.double().cpu().numpy().reshape(h, d_h)
        r = ref.reshape(h, d_h)
        tol = 1e-5 * np.abs(r) + 1e-5 * np.abs(r).max(axis=1, keepdims=True)
        assert (np.abs(g - r) <= tol).all()
    # whole pairs only, a different count per head
    ks = [2 * ((3 + 5 * i) % (d_h // 2 + 1)) for i in range(h)]
    k_vo = [(7 * i + 1) % (d_h + 1) for i in range(h)]
    kept = torch.full((sum(ks) + sum(k_vo),), -1, dtype=torch.int32, device=DEV)
    offs = torch.empty(2 * h + 1, dtype=torch.int32, device=DEV)
    B.ecospa_select_rotation_pairs(ups, [h, h], [d_h, d_h], ks + k_vo, [mode, B.ROPE_NONE], kept, offs)
    torch.cuda.synchronize()
    u_cpu = ups.cpu().numpy()
    want = np.concatenate([O.select_rotation_pairs(u_cpu[:D], h, d_h, ks, mode), O.select_topk(u_cpu[D:], h, d_h, k_vo)])
    assert np.array_equal(kept.cpu().numpy(), want)
    assert np.array_equal(offs.cpu().numpy(), np.concatenate([[0], np.cumsum(ks + k_vo)]).astype(np.int32))


def test_rotation_pair_requests_that_are_rejected():
    wl = WL.WORKLOADS["tiny_swiglu"]
    w = WL.layer_weights(wl, 0)
    wq, wk = w["wq"].to(DEV), w["wk"].to(DEV)
    ups = torch.zeros(wl.n_heads * wl.d_h, dtype=torch.float32, device=DEV)
    kept = torch.zeros(64, dtype=torch.int32, device=DEV)
    with pytest.raises(B.EcospaError):          # an odd count would split a rotation pair
        B.ecospa_select_rotation_pairs(ups, [wl.n_heads], [wl.d_h], [3] * wl.n_heads, [B.ROPE_HALF], kept)
    with pytest.raises(B.EcospaError):          # unknown pairing
        B.ecospa_score_pairs([B.pair(B.PAIR_PLAIN, wl.n_heads, wl.d_h, wq, wk, 0, 0, rope=7)], 1.0, ups, None, None)
