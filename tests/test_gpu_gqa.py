"""GPU parity of grouped-query scoring (w1_rep / w2_rep of the pair descriptor), selection per K/V group and the
compaction of the grouped tensors with kept lists expanded per query head, vs the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2511_11641_b200 import binding as B
from paper_2511_11641_b200 import block as BL

pytestmark = pytest.mark.gpu
DEV = "cuda"


def rand(shape, seed, std=0.02):
    return (torch.randn(shape, generator=torch.Generator().manual_seed(seed)) * std).to(torch.bfloat16)


@pytest.mark.parametrize("d_m,n_groups,rep,d_h", [(256, 2, 4, 64), (2048, 8, 4, 64), (512, 4, 8, 128)])
def test_grouped_query_scores_selection_compaction(d_m, n_groups, rep, d_h):
    H = n_groups * rep
    w = {"wq": rand((d_m, H * d_h), 0), "wk": rand((d_m, n_groups * d_h), 1), "wv": rand((d_m, n_groups * d_h), 2),
         "wo": rand((H * d_h, d_m), 3)}
    g = {"gq": rand((d_m, H * d_h), 4, 1e-3), "gk": rand((d_m, n_groups * d_h), 5, 1e-3),
         "gv": rand((d_m, n_groups * d_h), 6, 1e-3), "go": rand((H * d_h, d_m), 7, 1e-3)}
    d = {k: v.to(DEV) for k, v in {**w, **g}.items()}
    pairs = [B.pair(B.PAIR_PLAIN, n_groups, d_h, d["wq"], d["wk"], B.SHARED_COLS, B.SHARED_COLS, g1=d["gq"], g2=d["gk"], w1_rep=rep),
             B.pair(B.PAIR_PLAIN, n_groups, d_h, d["wv"], d["wo"], B.SHARED_COLS, B.SHARED_ROWS, g1=d["gv"], g2=d["go"], w2_rep=rep)]
    D = n_groups * d_h
    ups = torch.full((2 * D + 16,), -7.0, dtype=torch.float32, device=DEV)
    raw = torch.empty(2 * D, dtype=torch.float32, device=DEV)
    fis = torch.empty(2 * n_groups, dtype=torch.float32, device=DEV)
    n_samples = 4096.0
    B.ecospa_score_pairs(pairs, n_samples, ups, raw, fis)
    torch.cuda.synchronize()
    assert torch.all(ups[2 * D:] == -7.0)
    refs = [O.score_pair_gqa(w["wq"], w["wk"], 0, 0, n_groups, d_h, rep1=rep),
            O.score_pair_gqa(w["wv"], w["wo"], 0, 1, n_groups, d_h, rep2=rep)]
    fref = np.concatenate([O.fisher_pair_gqa(g["gq"], g["gk"], 0, 0, n_groups, d_h, n_samples, rep1=rep),
                           O.fisher_pair_gqa(g["gv"], g["go"], 0, 1, n_groups, d_h, n_samples, rep2=rep)])
    got_u, got_r = ups[:2 * D].double().cpu().numpy(), raw.double().cpu().numpy()
    for p in range(2):
        for s in range(n_groups):
            a, b = p * D + s * d_h, p * D + (s + 1) * d_h
            for got, ref in ((got_u[a:b], refs[p][1][s * d_h:(s + 1) * d_h]), (got_r[a:b], refs[p][0][s * d_h:(s + 1) * d_h])):
                assert np.all(np.abs(got - ref) <= 1e-5 * np.abs(ref) + 1e-5 * np.abs(ref).max())
    np.testing.assert_allclose(fis.double().cpu().numpy(), fref, rtol=1e-5)

    # selection per K/V group on the GPU's scores vs the oracle's ranking of the same vector
    k = [d_h // 2] * n_groups
    kept = torch.empty(2 * sum(k), dtype=torch.int32, device=DEV)
    B.ecospa_select_aligned_topk(ups[:2 * D], [n_groups, n_groups], [d_h, d_h], k + k, kept)
    u = ups[:2 * D].cpu().numpy()
    kept_qk = O.select_topk(u[:D], n_groups, d_h, k)
    kept_vo = O.select_topk(u[D:], n_groups, d_h, k)
    np.testing.assert_array_equal(kept.cpu().numpy(), np.concatenate([kept_qk, kept_vo]))

    # compaction: K and V with the group lists; Q and O with the same within-head indices in every head of the group
    # (the lists are expanded on the device by ecospa_pack_kept: one segment per query head, shifted by its offset)
    nk = sum(k)
    src, dst, kk, add = [], [], [], []
    for h in range(H):
        grp = h // rep
        src.append(sum(k[:grp])); dst.append(h * k[0]); kk.append(k[grp]); add.append((h - grp) * d_h)
    kept_q = torch.empty(H * k[0], dtype=torch.int32, device=DEV)
    kept_o = torch.empty(H * k[0], dtype=torch.int32, device=DEV)
    B.ecospa_pack_kept(kept[:nk], src, dst, kk, add, kept_q)
    B.ecospa_pack_kept(kept[nk:], src, dst, kk, add, kept_o)
    exp_q = np.concatenate([kept_qk[sum(k[:h // rep]):sum(k[:h // rep + 1])] + (h - h // rep) * d_h for h in range(H)])
    exp_o = np.concatenate([kept_vo[sum(k[:h // rep]):sum(k[:h // rep + 1])] + (h - h // rep) * d_h for h in range(H)])
    np.testing.assert_array_equal(kept_q.cpu().numpy(), exp_q)
    np.testing.assert_array_equal(kept_o.cpu().numpy(), exp_o)
    jobs, outs = [], {}
    for nm, lay, kd, Dt in (("wq", 0, kept_q, H * d_h), ("wk", 0, kept[:nk], D), ("wv", 0, kept[nk:], D), ("wo", 1, kept_o, H * d_h)):
        o = BL.alloc_compacted(d[nm], lay, kd.numel()).fill_(7)
        outs[nm] = (o, lay, kd)
        jobs.append(B.gather(d[nm], o, lay, kd, kd.numel(), Dt))
    B.ecospa_compact_tensors(jobs)
    torch.cuda.synchronize()
    for nm, (o, lay, kd) in outs.items():
        ref = O.compact(w[nm], lay, kd.cpu().numpy(), ld_out=o.shape[1])
        assert torch.equal(o.cpu().view(torch.int16), ref.view(torch.int16)), nm
    # ecospa_compact_pair does not take grouped pairs (the two sides have different kept lists)
    with pytest.raises(B.EcospaError):
        B.ecospa_compact_pair(pairs[0], kept[:nk], nk, outs["wq"][0], outs["wk"][0])
