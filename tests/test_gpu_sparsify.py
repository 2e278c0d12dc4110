"""GPU parity: score / Fisher / aligned top-k / compaction through the C ABI vs the CPU oracle.

Tolerances (fp32 arithmetic on the GPU, fp64 in the oracle):
  scores and Fisher  : 1e-5 relative (absolute floor 1e-5 * max of the segment)
  kept index sets    : bit-exact when both sides rank the same fp32 score vector
  compacted tensors  : byte-exact
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
REL = 1e-5


def to_dev(d):
    return {k: v.to(DEV) for k, v in d.items()}


def oracle_block_scores(w, g, wl, n_samples):
    """Oracle upsilon / raw / fisher for the three groups of a block, concatenated like the ABI."""
    sw = "w1b" in w
    groups = [
        (w["wq"], None, w["wk"], O.SHARED_COLS, O.SHARED_COLS, wl.n_heads, wl.d_h, g and (g["gq"], None, g["gk"])),
        (w["wv"], None, w["wo"], O.SHARED_COLS, O.SHARED_ROWS, wl.n_heads, wl.d_h, g and (g["gv"], None, g["go"])),
        (w["w1"], w.get("w1b"), w["w2"], O.SHARED_COLS, O.SHARED_ROWS, 1, wl.d_ffn,
         g and (g["g1"], g.get("g1b") if sw else None, g["g2"])),
    ]
    raws, upss, fish = [], [], []
    for w1, w1b, w2, l1, l2, n_seg, seg_len, gg in groups:
        raw, ups = O.score_pair(w1, w2, l1, l2, n_seg, seg_len, w1b=w1b)
        raws.append(raw); upss.append(ups)
        if gg:
            fish.append(O.fisher_pair(gg[0], gg[2], l1, l2, n_seg, seg_len, n_samples, g1b=gg[1]))
    return np.concatenate(raws), np.concatenate(upss), (np.concatenate(fish) if fish else None)


def gpu_block_scores(w_d, g_d, wl, n_samples, want_fisher=True):
    pairs = BL.block_pairs(w_d, wl.n_heads, wl.d_h, wl.d_ffn, g_d)
    total_d = 2 * wl.n_heads * wl.d_h + wl.d_ffn
    total_seg = 2 * wl.n_heads + 1
    ups = torch.full((total_d + 64,), -7.0, dtype=torch.float32, device=DEV)   # canary tail
    raw = torch.full((total_d + 64,), -7.0, dtype=torch.float32, device=DEV)
    fis = torch.full((total_seg + 64,), -7.0, dtype=torch.float32, device=DEV) if want_fisher else None
    B.ecospa_score_pairs(pairs, n_samples, ups, raw, fis)
    torch.cuda.synchronize()
    assert torch.all(ups[total_d:] == -7.0) and torch.all(raw[total_d:] == -7.0)
    if fis is not None:
        assert torch.all(fis[total_seg:] == -7.0)
        fis = fis[:total_seg]
    return pairs, ups[:total_d], raw[:total_d], fis


def assert_close_per_segment(got, ref, seg_bounds, rel=REL):
    got = got.double().cpu().numpy()
    for a, b in seg_bounds:
        floor = rel * np.abs(ref[a:b]).max()
        err = np.abs(got[a:b] - ref[a:b])
        assert np.all(err <= rel * np.abs(ref[a:b]) + floor), f"segment [{a},{b}) max err {err.max():.3e}"


def seg_bounds_of(wl):
    out, off = [], 0
    for n_seg, seg_len in ((wl.n_heads, wl.d_h), (wl.n_heads, wl.d_h), (1, wl.d_ffn)):
        for s in range(n_seg):
            out.append((off + s * seg_len, off + (s + 1) * seg_len))
        off += n_seg * seg_len
    return out


@pytest.mark.parametrize("name", ["block_f32", "tiny_swiglu", "tails768"])
def test_scores_and_fisher_match_oracle_small(name):
    wl = WL.WORKLOADS[name]
    w = WL.layer_weights(wl, 0); g = WL.layer_grads(wl, 0)
    raw_o, ups_o, fis_o = oracle_block_scores(w, g, wl, wl.tokens)
    _, ups, raw, fis = gpu_block_scores(to_dev(w), to_dev(g), wl, wl.tokens)
    sb = seg_bounds_of(wl)
    assert_close_per_segment(ups, ups_o, sb)
    assert_close_per_segment(raw, raw_o, sb)
    np.testing.assert_allclose(fis.double().cpu().numpy(), fis_o, rtol=REL)


@pytest.mark.parametrize("name", ["gpt2m", "llama1b"])
def test_scores_match_oracle_one_full_size_layer(name):
    wl = WL.WORKLOADS[name]
    w = WL.layer_weights(wl, 3); g = WL.layer_grads(wl, 3)
    raw_o, ups_o, fis_o = oracle_block_scores(w, g, wl, wl.tokens)
    _, ups, raw, fis = gpu_block_scores(to_dev(w), to_dev(g), wl, wl.tokens)
    assert_close_per_segment(ups, ups_o, seg_bounds_of(wl))
    np.testing.assert_allclose(fis.double().cpu().numpy(), fis_o, rtol=REL)


def test_scores_without_fisher_and_runs_are_bit_identical():
    wl = WL.WORKLOADS["tails768"]
    w_d = to_dev(WL.layer_weights(wl, 0))
    _, u1, r1, f1 = gpu_block_scores(w_d, None, wl, 1.0, want_fisher=False)
    _, u2, r2, _ = gpu_block_scores(w_d, None, wl, 1.0, want_fisher=False)
    assert f1 is None
    assert torch.equal(u1, u2) and torch.equal(r1, r2)


def test_scores_other_storage_orientation_and_unaligned_views():
    """Every tensor stored the other way round (nn.Linear style), then odd pitches / offset bases."""
    wl = WL.WORKLOADS["tiny_swiglu"]
    w = WL.layer_weights(wl, 0)
    raw_o, ups_o, _ = oracle_block_scores(w, None, wl, 1.0)
    wt = {k: v.t().contiguous().to(DEV) for k, v in w.items()}
    flip = {B.SHARED_COLS: B.SHARED_ROWS, B.SHARED_ROWS: B.SHARED_COLS}
    pairs = [
        B.pair(B.PAIR_PLAIN, wl.n_heads, wl.d_h, wt["wq"], wt["wk"], B.SHARED_ROWS, B.SHARED_ROWS),
        B.pair(B.PAIR_PLAIN, wl.n_heads, wl.d_h, wt["wv"], wt["wo"], B.SHARED_ROWS, B.SHARED_COLS),
        B.pair(B.PAIR_SWIGLU, 1, wl.d_ffn, wt["w1"], wt["w2"], B.SHARED_ROWS, B.SHARED_COLS, w1b=wt["w1b"]),
    ]
    total_d = 2 * wl.n_heads * wl.d_h + wl.d_ffn
    ups = torch.empty(total_d, dtype=torch.float32, device=DEV)
    B.ecospa_score_pairs(pairs, 1.0, ups)
    assert_close_per_segment(ups, ups_o, seg_bounds_of(wl))
    # unaligned: views with an odd pitch and a base that is only 2-byte aligned
    def odd_view(t):
        buf = torch.zeros((t.shape[0], t.shape[1] + 3), dtype=t.dtype, device=DEV).reshape(-1)
        v = buf[1:1 + t.shape[0] * (t.shape[1] + 3) - 3].as_strided(t.shape, (t.shape[1] + 3, 1))
        v.copy_(t)
        return v
    wd = {k: odd_view(v.to(DEV)) for k, v in w.items()}
    pairs = BL.block_pairs(wd, wl.n_heads, wl.d_h, wl.d_ffn)
    ups2 = torch.empty(total_d, dtype=torch.float32, device=DEV)
    B.ecospa_score_pairs(pairs, 1.0, ups2)
    assert_close_per_segment(ups2, ups_o, seg_bounds_of(wl))


def test_zero_segment_scores_zero():
    wl = WL.WORKLOADS["tiny_swiglu"]
    w = WL.layer_weights(wl, 0)
    w["wq"][:, : wl.d_h] = 0      # head 0 of QK is dead
    _, ups_o, _ = oracle_block_scores(w, None, wl, 1.0)
    _, ups, _, _ = gpu_block_scores(to_dev(w), None, wl, 1.0, want_fisher=False)
    assert torch.all(ups[: wl.d_h] == 0) and torch.all(torch.isfinite(ups))
    assert_close_per_segment(ups, ups_o, seg_bounds_of(wl))


# ---------------------------------------------------------------------------
# selection
# ---------------------------------------------------------------------------

def run_select(ups_cpu: np.ndarray, n_seg, seg_len, k):
    ups = torch.from_numpy(ups_cpu).to(DEV)
    total_k = int(sum(k)); total_seg = int(sum(n_seg))
    kept = torch.full((total_k + 16,), -1, dtype=torch.int32, device=DEV)
    offs = torch.full((total_seg + 1 + 16,), -1, dtype=torch.int32, device=DEV)
    B.ecospa_select_aligned_topk(ups, n_seg, seg_len, k, kept, offs)
    torch.cuda.synchronize()
    assert torch.all(kept[total_k:] == -1) and torch.all(offs[total_seg + 1:] == -1)
    np.testing.assert_array_equal(offs[: total_seg + 1].cpu().numpy(), np.concatenate([[0], np.cumsum(k)]))
    return kept[:total_k].cpu().numpy()


def oracle_select(ups_cpu, n_seg, seg_len, k):
    out, d_off, s_off = [], 0, 0
    for ns, sl in zip(n_seg, seg_len):
        out.append(O.select_topk(ups_cpu[d_off:d_off + ns * sl], ns, sl, k[s_off:s_off + ns]))
        d_off += ns * sl; s_off += ns
    return np.concatenate(out)


def test_select_bit_exact_on_random_scores_all_shapes():
    r = np.random.default_rng(0)
    n_seg = [16, 32, 1, 1, 3]
    seg_len = [64, 128, 4096, 11008, 777]
    k = []
    for ns, sl in zip(n_seg, seg_len):
        k += list(r.integers(0, sl + 1, size=ns))
    k[0], k[1], k[2] = 0, 64, 1
    ups = r.random(sum(a * b for a, b in zip(n_seg, seg_len))).astype(np.float32)
    got = run_select(ups, n_seg, seg_len, k)
    np.testing.assert_array_equal(got, oracle_select(ups, n_seg, seg_len, k))


def test_select_ties_keep_lowest_index():
    r = np.random.default_rng(1)
    n_seg, seg_len = [40, 2], [64, 5000]
    total = 40 * 64 + 2 * 5000
    ups = (r.integers(0, 5, size=total) / 8).astype(np.float32)       # heavy ties
    ups[:64] = 0.25                                                    # an all-equal segment
    ups[64:128] = np.where(np.arange(64) % 2 == 0, 0.0, -0.0)         # +0 / -0 are equal
    ups[128:192] = -ups[128:192]                                       # negative scores rank too
    k = list(r.integers(1, 64, size=40)) + [2500, 4999]
    got = run_select(ups, n_seg, seg_len, k)
    exp = oracle_select(ups, n_seg, seg_len, k)
    np.testing.assert_array_equal(got, exp)
    assert got[: k[0]].tolist() == list(range(k[0]))


@pytest.mark.parametrize("sparsity", [0.1, 0.5, 0.9])
def test_select_on_gpu_scores_matches_oracle_ranking_of_same_vector(sparsity):
    wl = WL.WORKLOADS["llama1b"]
    w_d = to_dev(WL.layer_weights(wl, 1))
    _, ups, _, _ = gpu_block_scores(w_d, None, wl, 1.0, want_fisher=False)
    plan = WL.kept_plan(wl, sparsity)
    n_seg = [wl.n_heads, wl.n_heads, 1]; seg_len = [wl.d_h, wl.d_h, wl.d_ffn]
    k = plan["qk"] + plan["vo"] + plan["ffn"]
    ups_cpu = ups.cpu().numpy()
    got = run_select(ups_cpu, n_seg, seg_len, k)
    np.testing.assert_array_equal(got, oracle_select(ups_cpu, n_seg, seg_len, k))
    assert len(got) == sum(k)


def test_select_from_own_scores_differs_from_oracle_scores_only_at_near_ties():
    wl = WL.WORKLOADS["gpt2m"]
    w = WL.layer_weights(wl, 2)
    _, ups_o, _ = oracle_block_scores(w, None, wl, 1.0)
    _, ups, _, _ = gpu_block_scores(to_dev(w), None, wl, 1.0, want_fisher=False)
    plan = WL.kept_plan(wl, 0.5)
    n_seg = [wl.n_heads, wl.n_heads, 1]; seg_len = [wl.d_h, wl.d_h, wl.d_ffn]
    k = plan["qk"] + plan["vo"] + plan["ffn"]
    got = run_select(ups.cpu().numpy(), n_seg, seg_len, k)
    exp = oracle_select(ups_o, n_seg, seg_len, k)        # fp64 scores ranked in fp64
    # kept lists are per pair group, indices relative to the group
    d_offs = [0, wl.n_heads * wl.d_h, 2 * wl.n_heads * wl.d_h]
    ks = [sum(plan["qk"]), sum(plan["vo"]), sum(plan["ffn"])]
    o = 0
    for gi in range(3):
        a = set(got[o:o + ks[gi]].tolist()); b = set(exp[o:o + ks[gi]].tolist())
        for j in a ^ b:
            # a disagreement must sit within 2e-5 (relative) of the segment's k-th score
            seg = j // seg_len[gi]
            seg_scores = ups_o[d_offs[gi] + seg * seg_len[gi]: d_offs[gi] + (seg + 1) * seg_len[gi]]
            kth = np.sort(seg_scores)[::-1][k[sum(n_seg[:gi]) + seg] - 1]
            assert abs(ups_o[d_offs[gi] + j] - kth) <= 2e-5 * kth
        o += ks[gi]


# ---------------------------------------------------------------------------
# compaction
# ---------------------------------------------------------------------------

def compact_block_gpu(w_d, aux_d, wl, kept_d, ks):
    """Compacts the three groups with ecospa_compact_pair; returns dict name -> padded output buffer."""
    pairs = BL.block_pairs(w_d, wl.n_heads, wl.d_h, wl.d_ffn)
    names = [("wq", "wk", None), ("wv", "wo", None), ("w1", "w2", "w1b")]
    out = {}
    o = 0
    for gi, p in enumerate(pairs):
        n1, n2, n1b = names[gi]
        nk = ks[gi]
        kept = kept_d[o:o + nk]
        o1 = BL.alloc_compacted(w_d[n1], p.w1.layout, nk).fill_(7)
        o2 = BL.alloc_compacted(w_d[n2], p.w2.layout, nk).fill_(7)
        o1b = BL.alloc_compacted(w_d[n1b], p.w1.layout, nk).fill_(7) if (n1b and n1b in w_d) else None
        aux = []
        for a_name, a_layout in aux_d.get(gi, []):
            ao = BL.alloc_compacted(w_d[a_name], a_layout, nk).fill_(7)
            aux.append((w_d[a_name], ao, a_layout))
            out[a_name] = ao
        B.ecospa_compact_pair(p, kept, nk, o1, o2, w1b_out=o1b, aux=aux)
        out[n1], out[n2] = o1, o2
        if o1b is not None:
            out[n1b] = o1b
        o += nk
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("name,sparsity", [("block_f32", 0.5), ("tiny_swiglu", 0.3), ("gpt2m", 0.5), ("llama1b", 0.9)])
def test_compaction_byte_exact(name, sparsity):
    wl = WL.WORKLOADS[name]
    w = WL.layer_weights(wl, 0)
    g = WL.layer_grads(wl, 0)
    allt = dict(w); allt.update(g)
    w_d = to_dev(allt)
    _, ups, _, _ = gpu_block_scores(w_d, None, wl, 1.0, want_fisher=False)
    plan = WL.kept_plan(wl, sparsity)
    n_seg = [wl.n_heads, wl.n_heads, 1]; seg_len = [wl.d_h, wl.d_h, wl.d_ffn]
    k = plan["qk"] + plan["vo"] + plan["ffn"]
    ks = [sum(plan["qk"]), sum(plan["vo"]), sum(plan["ffn"])]
    kept_d = torch.empty(sum(k), dtype=torch.int32, device=DEV)
    B.ecospa_select_aligned_topk(ups, n_seg, seg_len, k, kept_d)
    kept = kept_d.cpu().numpy()
    aux = {0: [("gq", B.SHARED_COLS), ("gk", B.SHARED_COLS)], 1: [("gv", B.SHARED_COLS), ("go", B.SHARED_ROWS)],
           2: [("g1", B.SHARED_COLS), ("g2", B.SHARED_ROWS)]}
    if wl.bias:
        aux[0] += [("bq", B.SHARED_COLS), ("bk", B.SHARED_COLS)]
        aux[1] += [("bv", B.SHARED_COLS)]
        aux[2] += [("b1", B.SHARED_COLS)]
    got = compact_block_gpu(w_d, aux, wl, kept_d, ks)
    layouts = {"wq": 0, "wk": 0, "wv": 0, "wo": 1, "w1": 0, "w1b": 0, "w2": 1,
               "gq": 0, "gk": 0, "gv": 0, "go": 1, "g1": 0, "g2": 1, "bq": 0, "bk": 0, "bv": 0, "b1": 0}
    group_of = {"wq": 0, "wk": 0, "gq": 0, "gk": 0, "bq": 0, "bk": 0, "wv": 1, "wo": 1, "gv": 1, "go": 1, "bv": 1,
                "w1": 2, "w1b": 2, "w2": 2, "g1": 2, "g2": 2, "b1": 2}
    starts = [0, ks[0], ks[0] + ks[1]]
    for nm, buf in got.items():
        gi = group_of[nm]
        kk = kept[starts[gi]: starts[gi] + ks[gi]]
        src = allt[nm]
        if src.dim() == 1:
            ref = O.compact(src, O.SHARED_COLS, kk, ld_out=buf.numel())
        else:
            ref = O.compact(src, layouts[nm], kk, ld_out=buf.shape[1])
        g_cpu = buf.cpu()
        view = torch.int16 if src.element_size() == 2 else torch.int32
        assert torch.equal(g_cpu.view(view), ref.view(view)), nm


def test_compaction_ragged_kept_counts_and_tensors_entry():
    """Per-head kept counts that the paper's compressed models show (not multiples of 8), through
    ecospa_compact_tensors with one job per tensor."""
    wl = WL.WORKLOADS["tails768"]
    w = WL.layer_weights(wl, 0)
    w_d = to_dev(w)
    r = np.random.default_rng(3)
    k_heads = [WL.RAGGED_HEAD_KEPT[i % len(WL.RAGGED_HEAD_KEPT)] for i in range(wl.n_heads)]
    for k_ffn in WL.RAGGED_FFN_KEPT:
        kept_qk = np.concatenate([np.sort(r.choice(wl.d_h, size=kh, replace=False)) + h * wl.d_h
                                  for h, kh in enumerate(k_heads)]).astype(np.int32)
        kept_ffn = np.sort(r.choice(wl.d_ffn, size=k_ffn, replace=False)).astype(np.int32)
        kq_d = torch.from_numpy(kept_qk).to(DEV); kf_d = torch.from_numpy(kept_ffn).to(DEV)
        jobs, outs = [], {}
        for nm, layout, kd, D in (("wq", 0, kq_d, wl.n_heads * wl.d_h), ("wo", 1, kq_d, wl.n_heads * wl.d_h),
                                  ("w1", 0, kf_d, wl.d_ffn), ("w2", 1, kf_d, wl.d_ffn), ("b1", 0, kf_d, wl.d_ffn)):
            o = BL.alloc_compacted(w_d[nm], layout, kd.numel()).fill_(7)
            outs[nm] = (o, layout, kd)
            jobs.append(B.gather(w_d[nm], o, layout, kd, kd.numel(), D))
        B.ecospa_compact_tensors(jobs)
        torch.cuda.synchronize()
        for nm, (o, layout, kd) in outs.items():
            src = w[nm]
            ld = o.numel() if src.dim() == 1 else o.shape[1]
            ref = O.compact(src, layout, kd.cpu().numpy(), ld_out=ld)
            assert torch.equal(o.cpu().view(torch.int16), ref.view(torch.int16)), (nm, k_ffn)


def test_fp32_optimizer_moments_follow_bf16_weights():
    """Algorithm 1 removes the same rows/columns of the optimizer moments: fp32 first and second moments of a
    bf16 FFN pair go through the same launch as the weights, with the same kept list, byte for byte."""
    wl = WL.WORKLOADS["tails768"]
    w = WL.layer_weights(wl, 0)
    gen = torch.Generator().manual_seed(5)
    mom = {"m1": torch.randn(w["w1"].shape, generator=gen), "v1": torch.rand(w["w1"].shape, generator=gen),
           "m2": torch.randn(w["w2"].shape, generator=gen), "v2": torch.rand(w["w2"].shape, generator=gen)}
    allt = {"w1": w["w1"], "w2": w["w2"], **mom}
    d = to_dev(allt)
    r = np.random.default_rng(4)
    for k_ffn in (1337, 2044):
        kept = np.sort(r.choice(wl.d_ffn, size=k_ffn, replace=False)).astype(np.int32)
        kd = torch.from_numpy(kept).to(DEV)
        jobs, outs = [], {}
        for nm, layout in (("w1", 0), ("m1", 0), ("v1", 0), ("w2", 1), ("m2", 1), ("v2", 1)):
            o = BL.alloc_compacted(d[nm], layout, k_ffn).fill_(7)
            outs[nm] = (o, layout)
            jobs.append(B.gather(d[nm], o, layout, kd, k_ffn, wl.d_ffn))
        B.ecospa_compact_tensors(jobs)
        torch.cuda.synchronize()
        for nm, (o, layout) in outs.items():
            ref = O.compact(allt[nm], layout, kept, ld_out=o.shape[1])
            view = torch.int16 if allt[nm].element_size() == 2 else torch.int32
            assert torch.equal(o.cpu().view(view), ref.view(view)), nm


# ---------------------------------------------------------------------------
# heavy-tailed single layer (LLaMA-7B shape) and the re-estimation sweep (LLaMA-1B shape)
# ---------------------------------------------------------------------------

_LAYOUTS = {"wq": 0, "wk": 0, "wv": 0, "wo": 1, "w1": 0, "w1b": 0, "w2": 1,
            "gq": 0, "gk": 0, "gv": 0, "go": 1, "g1": 0, "g1b": 0, "g2": 1, "bq": 0, "bk": 0, "bv": 0, "b1": 0}
_GROUP_OF = {"wq": 0, "wk": 0, "gq": 0, "gk": 0, "bq": 0, "bk": 0, "wv": 1, "wo": 1, "gv": 1, "go": 1, "bv": 1,
             "w1": 2, "w1b": 2, "w2": 2, "g1": 2, "g1b": 2, "g2": 2, "b1": 2}


def select_and_compact_vs_oracle(wl, allt, w_d, ups, sparsity, names):
    """Selection on the GPU's own fp32 scores vs the oracle's ranking of the same vector (bit-exact), then
    compaction of `names` by the library vs the oracle's byte copy with that kept list."""
    plan = WL.kept_plan(wl, sparsity)
    n_seg = [wl.n_heads, wl.n_heads, 1]; seg_len = [wl.d_h, wl.d_h, wl.d_ffn]
    k = plan["qk"] + plan["vo"] + plan["ffn"]
    ks = [sum(plan["qk"]), sum(plan["vo"]), sum(plan["ffn"])]
    kept_d = torch.empty(sum(k), dtype=torch.int32, device=DEV)
    B.ecospa_select_aligned_topk(ups, n_seg, seg_len, k, kept_d)
    kept = kept_d.cpu().numpy()
    np.testing.assert_array_equal(kept, oracle_select(ups.cpu().numpy(), n_seg, seg_len, k))
    if not names:
        return kept
    starts = [0, ks[0], ks[0] + ks[1]]
    dims = [wl.n_heads * wl.d_h, wl.n_heads * wl.d_h, wl.d_ffn]
    jobs, outs = [], {}
    for nm in names:
        gi = _GROUP_OF[nm]
        o = BL.alloc_compacted(w_d[nm], _LAYOUTS[nm], ks[gi]).fill_(7)
        outs[nm] = o
        jobs.append(B.gather(w_d[nm], o, _LAYOUTS[nm], kept_d[starts[gi]: starts[gi] + ks[gi]], ks[gi], dims[gi]))
    B.ecospa_compact_tensors(jobs)
    torch.cuda.synchronize()
    for nm, o in outs.items():
        gi = _GROUP_OF[nm]
        kk = kept[starts[gi]: starts[gi] + ks[gi]]
        ref = O.compact(allt[nm], _LAYOUTS[nm], kk, ld_out=o.shape[1] if o.dim() == 2 else o.numel())
        assert torch.equal(o.cpu().view(torch.int16), ref.view(torch.int16)), (nm, sparsity)
    return kept


def test_heavy_tailed_layer_scores_selection_compaction():
    """The LLaMA-7B-shaped layer whose shared-index vectors carry a x10 tail: scores and pair-level importance
    against the oracle, then kept sets and compacted tensors at 25 / 50 / 75 %."""
    wl = WL.WORKLOADS["llama7b_layer"]
    w = WL.layer_weights(wl, 0); g = WL.layer_grads(wl, 0)
    raw_o, ups_o, fis_o = oracle_block_scores(w, g, wl, wl.tokens)
    allt = dict(w); allt.update(g)
    w_d = to_dev(allt)
    _, ups, raw, fis = gpu_block_scores(w_d, w_d, wl, wl.tokens)
    sb = seg_bounds_of(wl)
    assert_close_per_segment(ups, ups_o, sb)
    assert_close_per_segment(raw, raw_o, sb)
    np.testing.assert_allclose(fis.double().cpu().numpy(), fis_o, rtol=REL)
    # the tail is what decides: the scores of a head span more than an order of magnitude
    head0 = ups_o[: wl.d_h]
    assert head0.max() > 10 * np.median(head0)
    for s in (0.25, 0.5, 0.75):
        select_and_compact_vs_oracle(wl, allt, w_d, ups, s, ["wq", "wk", "wv", "wo", "w1", "w1b", "w2"])


def test_reestimation_sweep_one_layer():
    """Re-estimation as Algorithm 1 repeats it: weights fixed, gradients redrawn per step.  One LLaMA-1B-shaped layer,
    three of the ten gradient draws: importance vs the oracle for every draw; kept sets at all nine sparsities
    (10 ... 90 %) bit-exact on the same fp32 scores; compaction of weights and of the redrawn gradients byte-exact
    at 10 / 50 / 90 %."""
    wl = WL.WORKLOADS["llama1b"]
    layer = 5
    w = WL.layer_weights(wl, layer)
    w_d = to_dev(w)
    _, ups_o, _ = oracle_block_scores(w, None, wl, wl.tokens)
    ups_first = None
    for seed in (0, 4, 9):
        g = WL.layer_grads(wl, layer, step=seed)
        g_d = to_dev(g)
        _, ups, _, fis = gpu_block_scores(w_d, g_d, wl, wl.tokens)
        fis_o = np.concatenate([
            O.fisher_pair(g["gq"], g["gk"], 0, 0, wl.n_heads, wl.d_h, wl.tokens),
            O.fisher_pair(g["gv"], g["go"], 0, 1, wl.n_heads, wl.d_h, wl.tokens),
            O.fisher_pair(g["g1"], g["g2"], 0, 1, 1, wl.d_ffn, wl.tokens, g1b=g["g1b"])])
        np.testing.assert_allclose(fis.double().cpu().numpy(), fis_o, rtol=REL)
        assert_close_per_segment(ups, ups_o, seg_bounds_of(wl))
        if ups_first is None:
            ups_first = ups.clone()
        else:
            assert torch.equal(ups, ups_first)          # the scores do not depend on the gradients
        allt = dict(w); allt.update(g)
        d_all = dict(w_d); d_all.update(g_d)
        for s10 in range(1, 10):
            s = s10 / 10.0
            names = ["wq", "wk", "wo", "w1", "w1b", "w2", "gq", "go", "g1", "g1b", "g2"] if s10 in (1, 5, 9) else []
            kept = select_and_compact_vs_oracle(wl, allt, d_all, ups, s, names)
            assert len(kept) == 2 * wl.n_heads * WL.kept_count(wl.d_h, s) + WL.kept_count(wl.d_ffn, s)


def test_in_place_compaction_equals_out_of_place():
    """ecospa_compact_tensors_inplace moves the kept part to the front of each tensor's own storage: same bytes as the
    out-of-place call (and the oracle) on the kept part, for bf16 and fp32, both layouts, a 1-D bias, odd pitches, and a
    kept list with "no index" entries."""
    wl = WL.WORKLOADS["tails768"]
    w = WL.layer_weights(wl, 0)
    gen = torch.Generator().manual_seed(6)
    t = {"w1": w["w1"], "w2": w["w2"], "b1": w["b1"], "m1": torch.randn(w["w1"].shape, generator=gen),
         "m2": torch.randn(w["w2"].shape, generator=gen)}
    lay = {"w1": 0, "w2": 1, "b1": 0, "m1": 0, "m2": 1}
    r = np.random.default_rng(8)
    for k_ffn, pads in ((1337, 0), (2044, 0), (1073, 7), (150, 0)):      # 150: sources too far apart to stage a chunk
        kept = np.sort(r.choice(wl.d_ffn, size=k_ffn, replace=False)).astype(np.int32)
        if pads:                                          # "no index" entries that pad two blocks, as for padded heads:
            half = wl.d_ffn // 2                          # every real entry still satisfies kept[c] >= c
            lo, hi = kept[kept < half], kept[kept >= half]
            kept = np.concatenate([lo, -np.ones(3, np.int32), hi, -np.ones(pads - 3, np.int32)]).astype(np.int32)
        n = len(kept)
        kd = torch.from_numpy(kept).to(DEV)
        jobs, bufs = [], {}
        for nm, src in t.items():
            d = src.to(DEV).clone()
            bufs[nm] = d
            jobs.append(B.gather(d, d, lay[nm], kd, n, wl.d_ffn))
        B.ecospa_compact_tensors_inplace(jobs)
        torch.cuda.synchronize()
        for nm, src in t.items():
            ref = O.compact(src, lay[nm], kept)
            d = bufs[nm].cpu()
            got = d[:n] if src.dim() == 1 else (d[:, :n] if lay[nm] == 0 else d[:n])
            view = torch.int16 if src.element_size() == 2 else torch.int32
            assert torch.equal(got.contiguous().view(view), ref.contiguous().view(view)), (nm, k_ffn)
    # an odd pitch and a base that is only 2-byte aligned (element-wise path of the shared-rows stripe)
    src = w["w2"][:, :701].contiguous()
    buf = torch.zeros(src.shape[0] * 705 + 1, dtype=src.dtype, device=DEV)
    v = buf[1:].as_strided(src.shape, (705, 1))
    v.copy_(src)
    kept = np.sort(r.choice(wl.d_ffn, size=900, replace=False)).astype(np.int32)
    kd = torch.from_numpy(kept).to(DEV)
    B.ecospa_compact_tensors_inplace([B.gather(v, v, 1, kd, 900, wl.d_ffn)])
    ref = O.compact(src, 1, kept)
    assert torch.equal(v[:900].cpu().contiguous().view(torch.int16), ref.view(torch.int16))
    # the same for a shared-cols tensor (element-wise loads and stores of the staged path)
    src = w["w1"][:37].contiguous()
    pitch = wl.d_ffn + 3
    buf = torch.zeros(src.shape[0] * pitch + 1, dtype=src.dtype, device=DEV)
    v = buf[1:].as_strided(src.shape, (pitch, 1))
    v.copy_(src)
    B.ecospa_compact_tensors_inplace([B.gather(v, v, 0, kd, 900, wl.d_ffn)])
    ref = O.compact(src, 0, kept)
    assert torch.equal(v[:, :900].cpu().contiguous().view(torch.int16), ref.view(torch.int16))
