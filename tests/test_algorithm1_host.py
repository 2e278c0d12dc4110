"""Host-side logic of the Algorithm 1 pass (no GPU): how groups are described to the scoring call."""
import torch

from paper_2511_11641_b200 import algorithm1 as A1
from paper_2511_11641_b200 import binding as B


def test_uniform_group_is_one_descriptor_and_ragged_group_one_per_pair():
    d_m, h, dh = 16, 3, 8
    wq = torch.zeros(d_m, h * dh, dtype=torch.bfloat16)
    wo = torch.zeros(h * dh, d_m, dtype=torch.bfloat16)
    g = A1.Group(wq, wo, B.SHARED_COLS, B.SHARED_ROWS, [dh] * h)
    pairs, n_seg, seg_len, where, rope = A1.describe([g])
    assert (n_seg, seg_len, where, rope) == ([h], [dh], [(0, 0)], [0])
    assert pairs[0].w1.ptr == wq.data_ptr() and pairs[0].w2.ptr == wo.data_ptr()
    assert g.n_params() == 2 * d_m * h * dh

    # after a pass: widths 6, 2, 4 in a buffer whose pitch is still padded
    buf1 = torch.zeros(d_m, 16, dtype=torch.bfloat16)         # 12 real columns + 4 pad columns
    buf2 = torch.zeros(12, d_m, dtype=torch.bfloat16)
    r = A1.Group(buf1, buf2, B.SHARED_COLS, B.SHARED_ROWS, [6, 2, 4], rope=B.ROPE_HALF)
    pairs, n_seg, seg_len, where, rope = A1.describe([g, r])
    assert n_seg == [h, 1, 1, 1] and seg_len == [dh, 6, 2, 4]
    assert where == [(0, 0), (1, 0), (1, 6), (1, 8)] and rope == [0, 2, 2, 2]
    eb = 2
    assert [p.w1.ptr - buf1.data_ptr() for p in pairs[1:]] == [0, 6 * eb, 8 * eb]              # column offsets
    assert [p.w2.ptr - buf2.data_ptr() for p in pairs[1:]] == [0, 6 * d_m * eb, 8 * d_m * eb]  # row offsets
    assert all(p.w1.ld == 16 and p.w2.ld == d_m for p in pairs[1:])                            # pitches stay
    assert [p.rope for p in pairs] == [0, 2, 2, 2]
    assert r.n_params() == 12 * 2 * d_m


def test_run_to_budget_stops_without_a_pass_when_the_model_is_small_enough():
    import torch
    from paper_2511_11641_b200 import algorithm1 as A1
    g = A1.Group(torch.zeros(4, 6), torch.zeros(6, 4), 0, 1, [3, 3])
    assert A1.total_params([g]) == 6 * (4 + 4)
    out, hist = A1.run_to_budget([g], 48, 1.0, 0.3, 0.9)          # already at the target: nothing is launched
    assert hist == [] and out[0] is g
