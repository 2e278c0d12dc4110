// One pass of the body of Algorithm 1 behind two C entry points (host-side bookkeeping only: every arithmetic
// step is one of the library's own calls).  ecospa_alg1_plan: importance of every pair (Eq. "importance"), choice
// of the least important pairs, their scores (Eq. "l2norm"), the kept count of every pair under the
// cumulative-threshold rule and the kept indices; the counts come back to the host, because they size the
// compacted tensors.  ecospa_alg1_apply: the physical removal from every tensor of every group (weights, gradients,
// and whatever else lives on the same shared axis: optimizer moments, biases), out of place or in place.
// Between the two calls the workspace keeps the scores, importance values, choice flags, slots and kept lists.

#include <cstring>
#include <vector>

#include "common.cuh"

namespace ecospa {

namespace {

struct Layout {          // where things sit in the workspace, in bytes
    int64_t total_d = 0, total_pairs = 0;
    size_t ups = 0, fisher = 0, chosen = 0, slots = 0, k_out = 0, kept = 0, score_ws = 0, end = 0;
};

struct Described {       // the pair descriptors of all groups, as the scoring call wants them
    std::vector<ecospa_pair_t> pairs;
    std::vector<int32_t> n_seg, seg_len, rope;
    std::vector<int32_t> group, offset;      // of every descriptor: its group and its first shared index inside the group
};

ecospa_mat_t slice(const ecospa_mat_t& m, int64_t off) {
    ecospa_mat_t s = m;
    if (!m.ptr) return s;
    const int64_t eb = elem_bytes(m.dtype);
    s.ptr = static_cast<char*>(m.ptr) + (m.layout == ECOSPA_SHARED_COLS ? off : off * m.ld) * eb;
    return s;
}

ecospa_status_t check_group(const ecospa_group_t& g) {
    if (g.n_pairs < 1 || !g.widths || g.n_aux < 0 || (g.n_aux > 0 && !g.aux)) return ECOSPA_ERR_INVALID;
    if (!g.w1.ptr || !g.w2.ptr) return ECOSPA_ERR_INVALID;
    for (int i = 0; i < g.n_pairs; ++i)
        if (g.widths[i] < 0) return ECOSPA_ERR_INVALID;
    return ECOSPA_OK;
}

// A group whose pairs all have one width is one descriptor (n_pairs segments side by side); a ragged group is one
// descriptor per pair on slices of its tensors; a pair that has lost every index takes no part.
ecospa_status_t describe(const ecospa_group_t* groups, int n_groups, bool with_grads, Described& D) {
    for (int gi = 0; gi < n_groups; ++gi) {
        const ecospa_group_t& g = groups[gi];
        ecospa_status_t st = check_group(g);
        if (st != ECOSPA_OK) return st;
        if (with_grads && (!g.g1.ptr || !g.g2.ptr || (g.w1b.ptr && !g.g1b.ptr))) return ECOSPA_ERR_INVALID;
        bool uniform = true;
        for (int i = 1; i < g.n_pairs; ++i) uniform = uniform && g.widths[i] == g.widths[0];
        auto add = [&](int64_t off, int32_t ns, int32_t sl) {
            if (sl == 0) return;
            ecospa_pair_t p;
            std::memset(&p, 0, sizeof(p));
            p.kind = g.w1b.ptr ? ECOSPA_PAIR_SWIGLU : ECOSPA_PAIR_PLAIN;
            p.n_seg = ns; p.seg_len = sl; p.rope = g.rope;
            p.w1 = slice(g.w1, off); p.w1b = slice(g.w1b, off); p.w2 = slice(g.w2, off);
            p.g1 = slice(g.g1, off); p.g1b = slice(g.g1b, off); p.g2 = slice(g.g2, off);
            D.pairs.push_back(p);
            D.n_seg.push_back(ns); D.seg_len.push_back(sl); D.rope.push_back(g.rope);
            D.group.push_back(gi); D.offset.push_back(static_cast<int32_t>(off));
        };
        if (uniform) {
            add(0, g.n_pairs, g.widths[0]);
        } else {
            int64_t off = 0;
            for (int i = 0; i < g.n_pairs; ++i) {
                add(off, 1, g.widths[i]);
                off += g.widths[i];
            }
        }
    }
    return D.pairs.empty() ? ECOSPA_ERR_INVALID : ECOSPA_OK;
}

Layout lay_out(const Described& D) {
    Layout L;
    for (size_t i = 0; i < D.pairs.size(); ++i) {
        L.total_d += static_cast<int64_t>(D.n_seg[i]) * D.seg_len[i];
        L.total_pairs += D.n_seg[i];
    }
    auto up = [](size_t v) { return (v + 255) & ~size_t(255); };
    size_t o = 0;
    L.ups = o; o = up(o + L.total_d * 4);
    L.fisher = o; o = up(o + L.total_pairs * 4);
    L.chosen = o; o = up(o + L.total_pairs * 4);
    L.slots = o; o = up(o + L.total_d * 4);
    L.k_out = o; o = up(o + L.total_pairs * 4);
    L.kept = o; o = up(o + L.total_d * 4);
    L.score_ws = o;
    o = up(o + ecospa_score_workspace_bytes(D.pairs.data(), static_cast<int32_t>(D.pairs.size())));
    L.end = o;
    return L;
}

}  // namespace

}  // namespace ecospa

using namespace ecospa;

extern "C" size_t ecospa_alg1_workspace_bytes(const ecospa_group_t* groups, int32_t n_groups) {
    if (!groups || n_groups < 1) return 0;
    Described D;
    if (describe(groups, n_groups, false, D) != ECOSPA_OK) return 0;
    return lay_out(D).end;
}

extern "C" ecospa_status_t ecospa_alg1_offsets(const ecospa_group_t* groups, int32_t n_groups, int64_t* offsets) {
    if (!groups || n_groups < 1 || !offsets) return ECOSPA_ERR_INVALID;
    Described D;
    ecospa_status_t st = describe(groups, n_groups, false, D);
    if (st != ECOSPA_OK) return st;
    const Layout L = lay_out(D);
    offsets[0] = static_cast<int64_t>(L.ups); offsets[1] = static_cast<int64_t>(L.fisher);
    offsets[2] = static_cast<int64_t>(L.chosen); offsets[3] = static_cast<int64_t>(L.kept);
    offsets[4] = L.total_d; offsets[5] = L.total_pairs;
    return ECOSPA_OK;
}

extern "C" ecospa_status_t ecospa_alg1_plan(const ecospa_group_t* groups, int32_t n_groups, double n_samples,
                                            int32_t n_choose, double theta, int32_t l1, int32_t k_min, void* workspace,
                                            size_t workspace_bytes, int32_t* k_host, void* stream) {
    if (!groups || n_groups < 1 || !k_host || n_choose < 0) return ECOSPA_ERR_INVALID;
    Described D;
    ecospa_status_t st = describe(groups, n_groups, true, D);
    if (st != ECOSPA_OK) return st;
    const Layout L = lay_out(D);
    if (!workspace || workspace_bytes < L.end) return ECOSPA_ERR_WORKSPACE;
    if (!aligned16(workspace)) return ECOSPA_ERR_ALIGNMENT;
    char* ws = static_cast<char*>(workspace);
    float* ups = reinterpret_cast<float*>(ws + L.ups);
    float* fisher = reinterpret_cast<float*>(ws + L.fisher);
    int32_t* chosen = reinterpret_cast<int32_t*>(ws + L.chosen);
    int32_t* slots = reinterpret_cast<int32_t*>(ws + L.slots);
    int32_t* k_out = reinterpret_cast<int32_t*>(ws + L.k_out);
    const int32_t n_desc = static_cast<int32_t>(D.pairs.size());
    if ((st = ecospa_score_pairs(D.pairs.data(), n_desc, n_samples, ups, nullptr, fisher, ws + L.score_ws,
                                 L.end - L.score_ws, stream)) != ECOSPA_OK)
        return st;
    const int32_t m = static_cast<int32_t>(std::min<int64_t>(n_choose, L.total_pairs));
    if ((st = ecospa_choose_pairs(fisher, static_cast<int32_t>(L.total_pairs), m, chosen, stream)) != ECOSPA_OK) return st;
    bool any_rope = false;
    for (int32_t r : D.rope) any_rope = any_rope || r != ECOSPA_ROPE_NONE;
    if ((st = ecospa_select_aligned_threshold(ups, D.n_seg.data(), D.seg_len.data(), any_rope ? D.rope.data() : nullptr, n_desc,
                                              theta, l1, k_min, chosen, slots, k_out, stream)) != ECOSPA_OK)
        return st;
    // the one read-back of the pass: the counts size everything that follows
    std::vector<int32_t> k(static_cast<size_t>(L.total_pairs));
    cudaError_t e = cudaMemcpyAsync(k.data(), k_out, k.size() * 4, cudaMemcpyDeviceToHost, static_cast<cudaStream_t>(stream));
    if (e == cudaSuccess) e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        set_cuda_error(e, "ecospa_alg1_plan (read-back of the kept counts)");
        return ECOSPA_ERR_CUDA;
    }
    // per (group, pair) in the caller's order; pairs of width 0 stay at 0
    size_t pos = 0, seg = 0;
    for (int gi = 0; gi < n_groups; ++gi)
        for (int i = 0; i < groups[gi].n_pairs; ++i) k_host[pos++] = groups[gi].widths[i] == 0 ? 0 : k[seg++];
    return ECOSPA_OK;
}

extern "C" ecospa_status_t ecospa_alg1_apply(const ecospa_group_t* groups, int32_t n_groups, const int32_t* k_host,
                                             const ecospa_group_t* out, int32_t in_place, void* workspace,
                                             size_t workspace_bytes, void* stream) {
    if (!groups || n_groups < 1 || !k_host || (!in_place && !out)) return ECOSPA_ERR_INVALID;
    Described D;
    ecospa_status_t st = describe(groups, n_groups, false, D);
    if (st != ECOSPA_OK) return st;
    const Layout L = lay_out(D);
    if (!workspace || workspace_bytes < L.end) return ECOSPA_ERR_WORKSPACE;
    char* ws = static_cast<char*>(workspace);
    const int32_t* slots = reinterpret_cast<const int32_t*>(ws + L.slots);
    int32_t* kept_all = reinterpret_cast<int32_t*>(ws + L.kept);
    // kept list of every group: its pairs' slots one after the other, shifted to indices of the group's shared axis
    std::vector<int32_t> src, dst, kk, add;
    std::vector<int64_t> group_kept_off(n_groups), group_n_kept(n_groups), group_D(n_groups);
    std::vector<int64_t> k_base(n_groups);
    {
        int64_t kb = 0;
        for (int gi = 0; gi < n_groups; ++gi) { k_base[gi] = kb; kb += groups[gi].n_pairs; }
    }
    int64_t d_off = 0, kept_off = 0;
    size_t di = 0;
    for (int gi = 0; gi < n_groups; ++gi) {
        const ecospa_group_t& g = groups[gi];
        group_kept_off[gi] = kept_off;
        int64_t run = 0, Dg = 0;
        int pair_i = 0;
        for (int i = 0; i < g.n_pairs; ++i) Dg += g.widths[i];
        group_D[gi] = Dg;
        for (; di < D.pairs.size() && D.group[di] == gi; ++di) {
            for (int s = 0; s < D.n_seg[di]; ++s) {
                while (g.widths[pair_i] == 0) ++pair_i;                    // pairs of width 0 were not described
                const int32_t k = k_host[k_base[gi] + pair_i];
                if (k < 0 || k > D.seg_len[di]) return ECOSPA_ERR_INVALID;
                src.push_back(static_cast<int32_t>(d_off + static_cast<int64_t>(s) * D.seg_len[di]));
                dst.push_back(static_cast<int32_t>(kept_off + run));
                kk.push_back(k);
                add.push_back(D.offset[di]);
                run += k;
                ++pair_i;
            }
            d_off += static_cast<int64_t>(D.n_seg[di]) * D.seg_len[di];
        }
        group_n_kept[gi] = run;
        kept_off += run;
    }
    if (!src.empty() && (st = ecospa_pack_kept(slots, src.data(), dst.data(), kk.data(), add.data(), static_cast<int32_t>(src.size()),
                                               kept_all, stream)) != ECOSPA_OK)
        return st;
    std::vector<ecospa_gather_t> jobs;
    for (int gi = 0; gi < n_groups; ++gi) {
        const ecospa_group_t& g = groups[gi];
        if (group_n_kept[gi] == 0) continue;
        auto add_job = [&](const ecospa_mat_t& in, const ecospa_mat_t* o) {
            if (!in.ptr) return ECOSPA_OK;
            ecospa_gather_t j;
            std::memset(&j, 0, sizeof(j));
            j.in = in;
            if (in_place) j.out = in;
            else {
                if (!o || !o->ptr) return ECOSPA_ERR_INVALID;
                j.out = *o;
            }
            j.kept = kept_all + group_kept_off[gi];
            j.n_kept = static_cast<int32_t>(group_n_kept[gi]);
            j.shared_dim = static_cast<int32_t>(group_D[gi]);
            jobs.push_back(j);
            return ECOSPA_OK;
        };
        const ecospa_group_t* og = in_place ? nullptr : &out[gi];
        if (og && og->n_aux != g.n_aux) return ECOSPA_ERR_INVALID;
        if ((st = add_job(g.w1, og ? &og->w1 : nullptr)) != ECOSPA_OK || (st = add_job(g.w1b, og ? &og->w1b : nullptr)) != ECOSPA_OK ||
            (st = add_job(g.w2, og ? &og->w2 : nullptr)) != ECOSPA_OK || (st = add_job(g.g1, og ? &og->g1 : nullptr)) != ECOSPA_OK ||
            (st = add_job(g.g1b, og ? &og->g1b : nullptr)) != ECOSPA_OK || (st = add_job(g.g2, og ? &og->g2 : nullptr)) != ECOSPA_OK)
            return st;
        for (int a = 0; a < g.n_aux; ++a)
            if ((st = add_job(g.aux[a], og ? &og->aux[a] : nullptr)) != ECOSPA_OK) return st;
    }
    if (jobs.empty()) return ECOSPA_OK;
    return in_place ? ecospa_compact_tensors_inplace(jobs.data(), static_cast<int32_t>(jobs.size()), stream)
                    : ecospa_compact_tensors(jobs.data(), static_cast<int32_t>(jobs.size()), stream);
}
