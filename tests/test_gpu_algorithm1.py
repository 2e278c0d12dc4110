"""Two consecutive passes of Algorithm 1's body on the GPU (paper_2511_11641_b200.algorithm1.step) vs the oracle.

Per pass: importance and scores within 1e-5 of the oracle's; the pair choice, the kept counts and the kept lists
equal to what the oracle decides on the same fp32 importance / score vectors; every tensor of every group
(weights, gradients, fp32 moments, biases) byte-exact against the oracle's compaction.  The second pass runs on
groups whose pairs have different widths.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2511_11641_b200 import algorithm1 as A1
from paper_2511_11641_b200 import binding as B
from paper_2511_11641_b200 import workloads as WL

pytestmark = pytest.mark.gpu
DEV = "cuda"


def make_groups(wl, with_moments=True, rope=0, galore_rank=0):
    w = WL.layer_weights(wl, 0)
    g = WL.layer_grads(wl, 0)
    gen = torch.Generator().manual_seed(11)
    h, dh = wl.n_heads, wl.d_h

    def mom(t):
        return torch.rand(t.shape, generator=gen, dtype=torch.float32)

    qk = dict(w1=w["wq"], w2=w["wk"], layout1=0, layout2=0, widths=[dh] * h, g1=g["gq"], g2=g["gk"], aux=[], rope=rope)
    vo = dict(w1=w["wv"], w2=w["wo"], layout1=0, layout2=1, widths=[dh] * h, g1=g["gv"], g2=g["go"], aux=[])
    ffn = dict(w1=w["w1"], w2=w["w2"], layout1=0, layout2=1, widths=[wl.d_ffn], g1=g["g1"], g2=g["g2"], aux=[])
    if "w1b" in w:
        ffn.update(w1b=w["w1b"], g1b=g["g1b"])
    if with_moments:
        qk["aux"] += [(mom(w["wq"]), 0), (mom(w["wk"]), 0)]
        ffn["aux"] += [(mom(w["w1"]), 0), (mom(w["w2"]), 1)]
    if galore_rank:
        # Optimizer states kept in a rank-r projected space (the memory-saving optimizer of the paper's LLaMA runs): the
        # projection acts on the short side of a weight, so the moments keep the shared axis: r x D beside a d_m x D
        # weight (shared columns), D x r beside a D x d_m weight (shared rows).  First and second moment each.
        r_ = galore_rank
        D_attn, D_ffn = h * dh, wl.d_ffn
        for _ in range(2):
            qk["aux"] += [(torch.rand((r_, D_attn), generator=gen), 0), (torch.rand((r_, D_attn), generator=gen), 0)]
            vo["aux"] += [(torch.rand((r_, D_attn), generator=gen), 0), (torch.rand((D_attn, r_), generator=gen), 1)]
            ffn["aux"] += [(torch.rand((r_, D_ffn), generator=gen), 0), (torch.rand((D_ffn, r_), generator=gen), 1)]
    if wl.bias:
        qk["aux"] += [(w["bq"], 0), (w["bk"], 0)]
        vo["aux"] += [(w["bv"], 0)]
        ffn["aux"] += [(w["b1"], 0)]
    return [qk, vo, ffn]


def to_gpu(spec):
    kw = {k: (v.to(DEV) if isinstance(v, torch.Tensor) else v) for k, v in spec.items() if k != "aux"}
    kw["aux"] = [(t.to(DEV), lay) for t, lay in spec["aux"]]
    return A1.Group(**kw)


def cut(t, layout, off, width):
    if t.dim() == 1:
        return t[off:off + width].contiguous()
    return (t[:, off:off + width] if layout == 0 else t[off:off + width, :]).contiguous()


def oracle_pass(specs, info, n_samples, ratio, theta, k_min):
    """Checks info against the oracle and returns the specs (CPU tensors) after the oracle's own removal."""
    ups = info["upsilon"].cpu().numpy(); fis = info["fisher"].cpu().numpy()
    # 1. importance and scores, pair by pair
    u_ref, f_ref = [], []
    for sp in specs:
        off = 0
        for wd in sp["widths"]:
            s = lambda nm, lay: cut(sp[nm], lay, off, wd) if sp.get(nm) is not None else None
            _, u = O.score_pair(s("w1", sp["layout1"]), s("w2", sp["layout2"]), sp["layout1"], sp["layout2"], 1, wd,
                                w1b=s("w1b", sp["layout1"]), rope=sp.get("rope", 0))
            f = O.fisher_pair(s("g1", sp["layout1"]), s("g2", sp["layout2"]), sp["layout1"], sp["layout2"], 1, wd, n_samples,
                              g1b=s("g1b", sp["layout1"]))
            u_ref.append(u); f_ref.append(f)
            off += wd
    f_ref = np.concatenate([np.atleast_1d(f) for f in f_ref])
    assert np.allclose(fis, f_ref, rtol=1e-5, atol=0)
    pos = 0
    for u in u_ref:
        got = ups[pos:pos + u.size]
        assert np.allclose(got, u, rtol=1e-5, atol=1e-5 * u.max())
        pos += u.size
    # 2. decisions on the fp32 vectors the GPU produced
    n = fis.size
    m = min(n, int(ratio * n + 0.5))
    chosen = O.choose_pairs(fis, m)
    assert np.array_equal(info["chosen"].cpu().numpy(), chosen) and info["n_chosen"] == m
    out, seg, pos = [], 0, 0
    for gi, sp in enumerate(specs):
        kept_g, new_w, off = [], [], 0
        for wd in sp["widths"]:
            u = ups[pos:pos + wd]
            rp = sp.get("rope", 0)
            k = int(O.threshold_counts(u, 1, wd, theta, l1=True, k_min=k_min, chosen=[int(chosen[seg])], rope=rp)[0])
            kept_g.append((O.select_rotation_pairs(u, 1, wd, [k], rp) if rp else O.select_topk(u, 1, wd, [k])) + off)
            new_w.append(k)
            pos += wd; off += wd; seg += 1
        kept_g = np.concatenate(kept_g).astype(np.int32)
        assert info["k"][gi] == new_w
        assert np.array_equal(info["kept"][gi].cpu().numpy(), kept_g)
        ns = dict(sp)
        ns["widths"] = new_w
        for nm, lay in (("w1", sp["layout1"]), ("w1b", sp["layout1"]), ("g1", sp["layout1"]), ("g1b", sp["layout1"]),
                        ("w2", sp["layout2"]), ("g2", sp["layout2"])):
            if sp.get(nm) is not None:
                ns[nm] = O.compact(sp[nm], lay, kept_g)
        ns["aux"] = [(O.compact(t, lay, kept_g), lay) for t, lay in sp["aux"]]
        out.append(ns)
    return out


def same_bytes(gpu_t, ref, layout, D):
    g = A1._trim(gpu_t, layout, D).cpu().contiguous()
    view = {1: torch.uint8, 2: torch.int16, 4: torch.int32}[ref.element_size()]
    return torch.equal(g.view(view), ref.contiguous().view(view))


@pytest.mark.parametrize("name,rope,in_place", [("tails768", 0, False), ("tiny_swiglu", 0, False), ("tails768", B.ROPE_HALF, False),
                                                ("tiny_swiglu", B.ROPE_INTERLEAVED, False), ("tails768", 0, True),
                                                ("tiny_swiglu", 0, True)])
def test_two_passes_match_the_oracle(name, rope, in_place):
    """in_place: the tensors (weights, gradients, fp32 moments, biases) shrink inside their own storage."""
    wl = WL.WORKLOADS[name]
    specs = make_groups(wl, rope=rope)
    groups = [to_gpu(sp) for sp in specs]
    n_samples = float(wl.tokens)
    ptrs = [g.w1.data_ptr() for g in groups]
    for ratio, theta in ((0.5, 0.9), (0.6, 0.8)):
        groups, info = A1.step(groups, n_samples, ratio, theta, l1=True, k_min=2, in_place=in_place)
        assert [g.w1.data_ptr() for g in groups] == ptrs or not in_place
        torch.cuda.synchronize()
        specs = oracle_pass(specs, info, n_samples, ratio, theta, 2)
        for g, sp in zip(groups, specs):
            assert g.widths == sp["widths"]
            D = sum(sp["widths"])
            for nm, lay in (("w1", sp["layout1"]), ("w1b", sp["layout1"]), ("g1", sp["layout1"]), ("g1b", sp["layout1"]),
                            ("w2", sp["layout2"]), ("g2", sp["layout2"])):
                if sp.get(nm) is not None:
                    assert same_bytes(getattr(g, nm), sp[nm], lay, D), nm
            for (tg, lay), (tr, _) in zip(g.aux, sp["aux"]):
                assert same_bytes(tg, tr, lay, D)
    assert any(len(set(g.widths)) > 1 for g in groups)          # the second pass did run on ragged groups


def spec_params(specs):
    n = 0
    for sp in specs:
        D = sum(sp["widths"])
        o1 = sp["w1"].shape[0] if sp["layout1"] == 0 else sp["w1"].shape[1]
        o2 = sp["w2"].shape[0] if sp["layout2"] == 0 else sp["w2"].shape[1]
        n += D * (o1 * (2 if sp.get("w1b") is not None else 1) + o2)
    return n


@pytest.mark.parametrize("name", ["tails768", "tiny_swiglu"])
def test_run_to_budget_matches_the_oracle_loop(name):
    """Algorithm 1's `if Param(W_t) > c` rule as a loop: the GPU driver and an oracle-side loop (same decisions on the
    same fp32 vectors, oracle compaction) shrink two copies of the model pass by pass to the same sizes and bytes,
    and stop at the same pass."""
    wl = WL.WORKLOADS[name]
    specs = make_groups(wl)
    groups = [to_gpu(sp) for sp in specs]
    n_samples = float(wl.tokens)
    start = spec_params(specs)
    assert A1.total_params(groups) == start
    budget = int(0.72 * start)
    ratio, theta, k_min = 0.4, 0.9, 2
    groups, hist = A1.run_to_budget(groups, budget, n_samples, ratio, theta, k_min=k_min)
    torch.cuda.synchronize()
    assert len(hist) >= 2, "the budget must take more than one pass"
    for h in hist:                                   # replay the same passes on the oracle's copy
        assert spec_params(specs) == h["params_before"] and h["params_before"] > budget
        specs = oracle_pass(specs, h["info"], n_samples, ratio, theta, k_min)
        assert spec_params(specs) == h["params_after"]
    assert A1.total_params(groups) == spec_params(specs)
    assert A1.total_params(groups) <= budget or hist[-1]["params_after"] == hist[-1]["params_before"]
    assert hist[-1]["params_before"] > budget            # no pass ran once the target was met
    for g, sp in zip(groups, specs):
        assert g.widths == sp["widths"]
        D = sum(sp["widths"])
        for nm, lay in (("w1", sp["layout1"]), ("w1b", sp["layout1"]), ("w2", sp["layout2"])):
            if sp.get(nm) is not None:
                assert same_bytes(getattr(g, nm), sp[nm], lay, D), nm
        for (tg, lay), (tr, _) in zip(g.aux, sp["aux"]):
            assert same_bytes(tg, tr, lay, D)


@pytest.mark.parametrize("in_place", [False, True])
def test_projected_optimizer_states_follow_the_pass(in_place):
    """Rank-24 projected first and second moments (r x D and D x r, fp32) ride along as further tensors of their groups:
    after two passes they hold exactly the kept columns / rows, like the weights."""
    wl = WL.WORKLOADS["tails768"]
    specs = make_groups(wl, with_moments=False, galore_rank=24)
    groups = [to_gpu(sp) for sp in specs]
    n_samples = float(wl.tokens)
    for ratio, theta in ((0.5, 0.9), (0.7, 0.85)):
        groups, info = A1.step(groups, n_samples, ratio, theta, l1=True, k_min=2, in_place=in_place)
        torch.cuda.synchronize()
        specs = oracle_pass(specs, info, n_samples, ratio, theta, 2)
        for g, sp in zip(groups, specs):
            D = sum(sp["widths"])
            assert len(g.aux) == len(sp["aux"]) >= 4
            for (tg, lay), (tr, _) in zip(g.aux, sp["aux"]):
                assert same_bytes(tg, tr, lay, D)


def test_a_pair_that_lost_every_index_takes_no_part():
    """A group described with an empty pair in the middle gives the same pass as the group without it (the empty
    pair keeps width 0 and is neither scored nor chosen); the reference pass is the oracle-checked one above."""
    wl = WL.WORKLOADS["tails768"]
    specs = make_groups(wl)
    n_samples = float(wl.tokens)
    ref_groups, ref_info = A1.step([to_gpu(sp) for sp in specs], n_samples, 0.5, 0.85, k_min=2)
    holed = []
    for sp in specs:
        sp = dict(sp)
        w = list(sp["widths"])
        sp["widths"] = w[:1] + [0] + w[1:]
        holed.append(to_gpu(sp))
    groups, info = A1.step(holed, n_samples, 0.5, 0.85, k_min=2)
    torch.cuda.synchronize()
    assert info["n_chosen"] == ref_info["n_chosen"]
    assert torch.allclose(info["fisher"], ref_info["fisher"], rtol=1e-6, atol=0)
    assert torch.equal(info["chosen"], ref_info["chosen"])
    for g, r in zip(groups, ref_groups):
        assert g.widths == r.widths[:1] + [0] + r.widths[1:]
        D = g.D
        for nm, lay in (("w1", g.layout1), ("w2", g.layout2), ("g1", g.layout1), ("g2", g.layout2)):
            assert torch.equal(A1._trim(getattr(g, nm), lay, D), A1._trim(getattr(r, nm), lay, D)), nm
        for (a, lay), (b, _) in zip(g.aux, r.aux):
            assert torch.equal(A1._trim(a, lay, D), A1._trim(b, lay, D))
