// Coupled importance scores: per-shared-index sums of squares of weights and gradients
// (streaming, HBM-bound), then the per-segment finalisation of Eq. "l2norm" and Eq. "importance".
//
// Three launches per call, no host synchronisation:
//   1. sumsq_kernel      one CTA per 64 KB-class tile of any tensor of any pair (job table in kernel
//                        parameters); shared-cols tensors produce per-row-chunk partial column sums,
//                        shared-rows tensors produce final row sums.
//   2. reduce_kernel     adds the row-chunk partials in a fixed order.
//   3. finalize_kernel   one CTA per segment: raw = sqrt(c1) sqrt(c2), upsilon = raw/||raw||, Fisher.
// Everything is summed in a fixed order, so results are bit-identical run to run.

#include <algorithm>
#include <mutex>
#include <vector>

#include "common.cuh"

namespace ecospa {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxJobs = 400;      // per launch; 72 B each -> 28.8 KB of kernel parameters (limit 32764)
constexpr int kMaxPairs = 256;     // per finalize launch; 64 B each
constexpr int kRowTile = 32;       // shared-rows tile: rows per CTA
constexpr int kUnroll = 4;

struct SumsqJob {
    const void* a;       // tensor
    const void* b;       // second factor of an element-wise product (gate (.) up) or nullptr
    float* partial;      // [n_chunks][D]; equals `stat` when n_chunks == 1
    float* stat;         // [D] final sums
    int32_t lda, ldb;    // row pitch in elements
    int32_t other, D;
    int32_t rows_per_chunk;
    int32_t tile_start;  // first sumsq tile of this job
    int32_t red_start;   // first reduce block of this job
    uint16_t col_tiles;  // shared-cols: tiles along D
    uint16_t n_chunks;
    uint8_t dtype, layout, aligned, pad_[5];
};
static_assert(sizeof(SumsqJob) == 72, "job descriptor size");

struct SumsqParams {
    int32_t n_jobs;
    int32_t pad_;
    SumsqJob jobs[kMaxJobs];
};

struct PairDesc {
    const float* c1;
    const float* c2;
    const float* gs1;
    const float* gs1b;
    const float* gs2;
    int32_t n_seg, seg_len;
    int32_t d_off;      // offset of this pair in upsilon / raw
    int32_t seg_start;  // first global segment index (also offset into fisher)
    float inv_numel1, inv_numel2;
    int32_t rope;       // ecospa_rope_t: the scored unit is a rotation pair of shared indices
    int16_t rep1, rep2; // heads stacked per segment on the W_1 / W_2 side (grouped-query attention); 1 = ordinary pair
};
static_assert(sizeof(PairDesc) == 72, "pair descriptor size");

struct FinalizeParams {
    int32_t n_pairs;
    int32_t pad_;
    float* upsilon;
    float* raw;
    float* fisher;
    double inv_n_samples;
    PairDesc pairs[kMaxPairs];
};

// Largest i with start(i) <= x.
template <typename F>
__device__ __forceinline__ int find_owner(int n, int x, F start) {
    int lo = 0, hi = n - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (start(mid) <= x) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// ---------------------------------------------------------------------------------------------
// shared-cols tile: rows [r0, r1) x columns [c0, c0 + 32*kVec); lane owns kVec adjacent columns,
// warp w takes rows r0 + w, r0 + w + 8, ...  Column sums of squares of a (or of a.*b).
// ---------------------------------------------------------------------------------------------
template <typename Tag>
__device__ __forceinline__ void cols_tile(const SumsqJob& J, int local, float* smem) {
    using TR = ElemTraits<Tag>;
    constexpr int V = TR::kVec;
    constexpr int CW = 32 * V;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int ct = local % J.col_tiles, chunk = local / J.col_tiles;
    const int col = ct * CW + lane * V;
    const int r0 = chunk * J.rows_per_chunk;
    const int r1 = min(J.other, r0 + J.rows_per_chunk);
    const bool has_b = J.b != nullptr;
    float acc[V];
#pragma unroll
    for (int e = 0; e < V; ++e) acc[e] = 0.f;

    if (col < J.D) {
        const bool vec = J.aligned && (col + V <= J.D);
        if (vec) {
            constexpr int EB = 16 / V;  // bytes per element
            const char* pa = static_cast<const char*>(J.a) + static_cast<int64_t>(col) * EB;
            const char* pb = has_b ? static_cast<const char*>(J.b) + static_cast<int64_t>(col) * EB : nullptr;
            const int64_t sa = static_cast<int64_t>(J.lda) * EB, sb = static_cast<int64_t>(J.ldb) * EB;  // bytes per row
            for (int r = r0 + warp; r < r1; r += kWarps * kUnroll) {
                uint4 va[kUnroll], vb[kUnroll];
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    const int rr = r + u * kWarps;
                    va[u] = make_uint4(0, 0, 0, 0);
                    vb[u] = make_uint4(0, 0, 0, 0);
                    if (rr < r1) {
                        va[u] = ldg_stream16(pa + rr * sa);
                        if (has_b) vb[u] = ldg_stream16(pb + rr * sb);
                    }
                }
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    float fa[V], fb[V];
                    TR::unpack(va[u], fa);
                    if (has_b) {
                        TR::unpack(vb[u], fb);
#pragma unroll
                        for (int e = 0; e < V; ++e) fa[e] *= fb[e];
                    }
#pragma unroll
                    for (int e = 0; e < V; ++e) acc[e] = fmaf(fa[e], fa[e], acc[e]);
                }
            }
        } else {
            for (int r = r0 + warp; r < r1; r += kWarps) {
#pragma unroll
                for (int e = 0; e < V; ++e) {
                    if (col + e < J.D) {
                        float x = TR::load1(J.a, static_cast<int64_t>(r) * J.lda + col + e);
                        if (has_b) x *= TR::load1(J.b, static_cast<int64_t>(r) * J.ldb + col + e);
                        acc[e] = fmaf(x, x, acc[e]);
                    }
                }
            }
        }
    }
    // cross-warp sum in warp order
    float* mine = smem + warp * (CW + 4) + lane * V;
#pragma unroll
    for (int e = 0; e < V; ++e) mine[e] = acc[e];
    __syncthreads();
    if (threadIdx.x < CW) {
        const int c = ct * CW + threadIdx.x;
        if (c < J.D) {
            float s = 0.f;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) s += smem[w * (CW + 4) + threadIdx.x];
            J.partial[static_cast<int64_t>(chunk) * J.D + c] = s;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// shared-rows tile: kRowTile rows (shared indices); a warp sums one row at a time.
// ---------------------------------------------------------------------------------------------
template <typename Tag>
__device__ __forceinline__ void rows_tile(const SumsqJob& J, int local) {
    using TR = ElemTraits<Tag>;
    constexpr int V = TR::kVec;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool has_b = J.b != nullptr;
    const int j0 = local * kRowTile;
    for (int jj = warp; jj < kRowTile; jj += kWarps) {
        const int j = j0 + jj;
        if (j >= J.D) break;
        float acc = 0.f;
        if (J.aligned) {
            const int nvec = J.other / V;
            const uint4* pa = reinterpret_cast<const uint4*>(static_cast<const char*>(J.a) + static_cast<int64_t>(j) * J.lda * (16 / V));
            const uint4* pb = has_b ? reinterpret_cast<const uint4*>(static_cast<const char*>(J.b) + static_cast<int64_t>(j) * J.ldb * (16 / V)) : nullptr;
            for (int v = lane; v < nvec; v += 32 * kUnroll) {
                uint4 va[kUnroll], vb[kUnroll];
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    const int vv = v + u * 32;
                    va[u] = make_uint4(0, 0, 0, 0);
                    vb[u] = make_uint4(0, 0, 0, 0);
                    if (vv < nvec) {
                        va[u] = ldg_stream16(pa + vv);
                        if (has_b) vb[u] = ldg_stream16(pb + vv);
                    }
                }
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    float fa[V], fb[V];
                    TR::unpack(va[u], fa);
                    if (has_b) {
                        TR::unpack(vb[u], fb);
#pragma unroll
                        for (int e = 0; e < V; ++e) fa[e] *= fb[e];
                    }
#pragma unroll
                    for (int e = 0; e < V; ++e) acc = fmaf(fa[e], fa[e], acc);
                }
            }
            for (int i = nvec * V + lane; i < J.other; i += 32) {  // ragged tail of the row
                float x = TR::load1(J.a, static_cast<int64_t>(j) * J.lda + i);
                if (has_b) x *= TR::load1(J.b, static_cast<int64_t>(j) * J.ldb + i);
                acc = fmaf(x, x, acc);
            }
        } else {
            for (int i = lane; i < J.other; i += 32) {
                float x = TR::load1(J.a, static_cast<int64_t>(j) * J.lda + i);
                if (has_b) x *= TR::load1(J.b, static_cast<int64_t>(j) * J.ldb + i);
                acc = fmaf(x, x, acc);
            }
        }
        acc = warp_sum(acc);
        if (lane == 0) J.partial[j] = acc;
    }
}

__global__ void __launch_bounds__(kThreads) sumsq_kernel(const __grid_constant__ SumsqParams P) {
    __shared__ float smem[kWarps * (256 + 4)];
    const int tile = blockIdx.x;
    const int ji = find_owner(P.n_jobs, tile, [&](int i) { return P.jobs[i].tile_start; });
    const SumsqJob& J = P.jobs[ji];
    const int local = tile - J.tile_start;
    if (J.layout == ECOSPA_SHARED_COLS) {
        if (J.dtype == ECOSPA_BF16) cols_tile<bf16_tag>(J, local, smem); else cols_tile<float>(J, local, smem);
    } else {
        if (J.dtype == ECOSPA_BF16) rows_tile<bf16_tag>(J, local); else rows_tile<float>(J, local);
    }
}

// stat[c] = sum over chunks of partial[chunk][c], chunk order fixed.
__global__ void __launch_bounds__(kThreads) reduce_kernel(const __grid_constant__ SumsqParams P) {
    const int blk = blockIdx.x;
    const int ji = find_owner(P.n_jobs, blk, [&](int i) { return P.jobs[i].red_start; });
    const SumsqJob& J = P.jobs[ji];
    const int c = (blk - J.red_start) * kThreads + threadIdx.x;
    if (J.n_chunks <= 1 || c >= J.D) return;
    float s = 0.f;
    for (int k = 0; k < J.n_chunks; ++k) s += J.partial[static_cast<int64_t>(k) * J.D + c];
    J.stat[c] = s;
}

__global__ void __launch_bounds__(kThreads) finalize_kernel(const __grid_constant__ FinalizeParams P) {
    __shared__ float scratch[kWarps];
    const int seg = blockIdx.x;
    const int pi = find_owner(P.n_pairs, seg, [&](int i) { return P.pairs[i].seg_start; });
    const PairDesc& Q = P.pairs[pi];
    const int s = seg - Q.seg_start;
    const int base = s * Q.seg_len;
    if (Q.rep1 > 1 || Q.rep2 > 1) {
        // Grouped heads: the statistic of index j on a stacked side is the sum over the group's heads, in head order.
        auto stacked = [&](const float* v, int rep, int j) {
            float t = 0.f;
            for (int r = 0; r < rep; ++r) t += v[(s * rep + r) * Q.seg_len + j];
            return t;
        };
        float ss = 0.f;
        for (int j = threadIdx.x; j < Q.seg_len; j += kThreads) {
            const float r = sqrtf(stacked(Q.c1, Q.rep1, j)) * sqrtf(stacked(Q.c2, Q.rep2, j));
            ss = fmaf(r, r, ss);
        }
        const float nrm = sqrtf(block_sum<kWarps>(ss, scratch));
        for (int j = threadIdx.x; j < Q.seg_len; j += kThreads) {
            const float r = sqrtf(stacked(Q.c1, Q.rep1, j)) * sqrtf(stacked(Q.c2, Q.rep2, j));
            if (P.raw) P.raw[Q.d_off + base + j] = r;
            P.upsilon[Q.d_off + base + j] = nrm > 0.f ? __fdiv_rn(r, nrm) : 0.f;
        }
        if (P.fisher) {
            float a = 0.f, b = 0.f;
            for (int j = threadIdx.x; j < Q.seg_len; j += kThreads) {
                a += stacked(Q.gs1, Q.rep1, j);
                b += stacked(Q.gs2, Q.rep2, j);
            }
            a = block_sum<kWarps>(a, scratch);
            b = block_sum<kWarps>(b, scratch);
            if (threadIdx.x == 0)
                P.fisher[seg] = static_cast<float>(0.5 * (static_cast<double>(a) * Q.inv_numel1 + static_cast<double>(b) * Q.inv_numel2) *
                                                   P.inv_n_samples);
        }
        return;
    }
    const float* c1 = Q.c1 + base;
    const float* c2 = Q.c2 + base;

    // raw score of index j: its own column/row norms, or those of its rotation pair (both members get the
    // pair's value; the pair is counted once in the normaliser)
    const int half = Q.seg_len >> 1;
    auto raw_of = [&](int j) -> float {
        if (Q.rope == ECOSPA_ROPE_NONE) return sqrtf(c1[j]) * sqrtf(c2[j]);
        const int a = Q.rope == ECOSPA_ROPE_INTERLEAVED ? (j & ~1) : (j < half ? j : j - half);
        const int b = Q.rope == ECOSPA_ROPE_INTERLEAVED ? (a | 1) : a + half;
        return sqrtf(c1[a] + c1[b]) * sqrtf(c2[a] + c2[b]);
    };
    float ss = 0.f;
    for (int j = threadIdx.x; j < Q.seg_len; j += kThreads) {
        const float r = raw_of(j);
        ss = fmaf(r, r, ss);
    }
    const float total = block_sum<kWarps>(ss, scratch);
    const float nrm = sqrtf(Q.rope == ECOSPA_ROPE_NONE ? total : 0.5f * total);
    for (int j = threadIdx.x; j < Q.seg_len; j += kThreads) {
        const float r = raw_of(j);
        if (P.raw) P.raw[Q.d_off + base + j] = r;
        P.upsilon[Q.d_off + base + j] = nrm > 0.f ? __fdiv_rn(r, nrm) : 0.f;
    }
    if (P.fisher) {
        float a = 0.f, ab = 0.f, b = 0.f;
        for (int j = threadIdx.x; j < Q.seg_len; j += kThreads) {
            a += Q.gs1[base + j];
            if (Q.gs1b) ab += Q.gs1b[base + j];
            b += Q.gs2[base + j];
        }
        a = block_sum<kWarps>(a, scratch);
        ab = block_sum<kWarps>(ab, scratch);
        b = block_sum<kWarps>(b, scratch);
        if (threadIdx.x == 0) {
            double t1 = static_cast<double>(a) * Q.inv_numel1;
            if (Q.gs1b) t1 = 0.5 * (t1 + static_cast<double>(ab) * Q.inv_numel1);
            const double t2 = static_cast<double>(b) * Q.inv_numel2;
            P.fisher[seg] = static_cast<float>(0.5 * (t1 + t2) * P.inv_n_samples);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// host side: validation, workspace plan, job tables
// ---------------------------------------------------------------------------------------------

struct StatPlan {        // one per-index statistic of one pair
    const ecospa_mat_t* a;
    const ecospa_mat_t* b;
    size_t partial_off, stat_off;  // in floats, relative to the workspace
    int n_chunks, rows_per_chunk;
    int32_t D;
};

int chunks_for(const ecospa_mat_t& m) {
    if (m.layout != ECOSPA_SHARED_COLS) return 1;
    return static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(4, m.other_dim / 64)));
}

ecospa_status_t validate_mat(const ecospa_mat_t& m, int64_t D, int want_dtype, int want_layout, int64_t want_other) {
    if (!m.ptr) return ECOSPA_ERR_INVALID;
    if (m.dtype != ECOSPA_F32 && m.dtype != ECOSPA_BF16) return ECOSPA_ERR_INVALID;
    if (m.layout != ECOSPA_SHARED_COLS && m.layout != ECOSPA_SHARED_ROWS) return ECOSPA_ERR_INVALID;
    if (m.other_dim < 1 || m.other_dim > INT32_MAX || m.ld > INT32_MAX) return ECOSPA_ERR_INVALID;
    if (m.ld < mat_cols(m, D)) return ECOSPA_ERR_INVALID;
    if (want_dtype >= 0 && m.dtype != want_dtype) return ECOSPA_ERR_INVALID;
    if (want_layout >= 0 && m.layout != want_layout) return ECOSPA_ERR_INVALID;
    if (want_other >= 0 && m.other_dim != want_other) return ECOSPA_ERR_INVALID;
    if (reinterpret_cast<uintptr_t>(m.ptr) % elem_bytes(m.dtype)) return ECOSPA_ERR_ALIGNMENT;
    return ECOSPA_OK;
}

ecospa_status_t validate_pair(const ecospa_pair_t& p, bool need_grads) {
    if (p.kind != ECOSPA_PAIR_PLAIN && p.kind != ECOSPA_PAIR_SWIGLU) return ECOSPA_ERR_INVALID;
    if (p.n_seg < 1 || p.seg_len < 1) return ECOSPA_ERR_INVALID;
    if (p.rope != ECOSPA_ROPE_NONE && p.rope != ECOSPA_ROPE_INTERLEAVED && p.rope != ECOSPA_ROPE_HALF) return ECOSPA_ERR_INVALID;
    if (p.rope != ECOSPA_ROPE_NONE && (p.kind != ECOSPA_PAIR_PLAIN || (p.seg_len & 1))) return ECOSPA_ERR_INVALID;
    const int64_t D = static_cast<int64_t>(p.n_seg) * p.seg_len;
    if (p.w1_rep < 0 || p.w2_rep < 0 || p.w1_rep > 1024 || p.w2_rep > 1024) return ECOSPA_ERR_INVALID;
    const int64_t r1 = std::max(1, p.w1_rep), r2 = std::max(1, p.w2_rep);
    if ((r1 > 1 || r2 > 1) && (p.kind != ECOSPA_PAIR_PLAIN || p.rope != ECOSPA_ROPE_NONE)) return ECOSPA_ERR_INVALID;
    if (D * std::max(r1, r2) > (1 << 22)) return ECOSPA_ERR_UNSUPPORTED;   // tile counts along D are 16-bit
    ecospa_status_t st;
    if ((st = validate_mat(p.w1, D * r1, -1, -1, -1)) != ECOSPA_OK) return st;
    if ((st = validate_mat(p.w2, D * r2, p.w1.dtype, -1, -1)) != ECOSPA_OK) return st;
    if (p.kind == ECOSPA_PAIR_SWIGLU &&
        (st = validate_mat(p.w1b, D, p.w1.dtype, p.w1.layout, p.w1.other_dim)) != ECOSPA_OK) return st;
    if (need_grads) {
        if ((st = validate_mat(p.g1, D * r1, -1, p.w1.layout, p.w1.other_dim)) != ECOSPA_OK) return st;
        if ((st = validate_mat(p.g2, D * r2, -1, p.w2.layout, p.w2.other_dim)) != ECOSPA_OK) return st;
        if (p.kind == ECOSPA_PAIR_SWIGLU &&
            (st = validate_mat(p.g1b, D, -1, p.w1.layout, p.w1.other_dim)) != ECOSPA_OK) return st;
    }
    return ECOSPA_OK;
}

// Lays the statistics of every pair out in the workspace.  Returns floats needed.
size_t plan_stats(const ecospa_pair_t* pairs, int n_pairs, bool grads, std::vector<StatPlan>* out) {
    size_t off = 0;
    auto add = [&](const ecospa_mat_t* a, const ecospa_mat_t* b, int64_t D) {
        StatPlan s{};
        s.a = a;
        s.b = b;
        s.D = static_cast<int32_t>(D);
        s.n_chunks = chunks_for(*a);
        s.rows_per_chunk = static_cast<int>(round_up(ceil_div(a->other_dim, s.n_chunks), kWarps));
        s.n_chunks = static_cast<int>(ceil_div(a->other_dim, s.rows_per_chunk));
        s.stat_off = off;
        off += round_up(D, 4);
        if (s.n_chunks > 1) {
            s.partial_off = off;
            off += static_cast<size_t>(s.n_chunks) * round_up(D, 4);
        } else {
            s.partial_off = s.stat_off;
        }
        if (out) out->push_back(s);
    };
    for (int i = 0; i < n_pairs; ++i) {
        const ecospa_pair_t& p = pairs[i];
        const int64_t D = static_cast<int64_t>(p.n_seg) * p.seg_len;
        const int64_t D1 = D * std::max(1, p.w1_rep), D2 = D * std::max(1, p.w2_rep);   // grouped heads: the stacked extent
        const bool sw = p.kind == ECOSPA_PAIR_SWIGLU;
        add(&p.w1, sw ? &p.w1b : nullptr, D1);  // c1
        add(&p.w2, nullptr, D2);                // c2
        if (grads) {
            add(&p.g1, nullptr, D1);
            if (sw) add(&p.g1b, nullptr, D);
            add(&p.g2, nullptr, D2);
        }
    }
    return off;
}

bool mat_aligned(const ecospa_mat_t& m) {
    return aligned16(m.ptr) && (m.ld * elem_bytes(m.dtype)) % 16 == 0;
}

}  // namespace

}  // namespace ecospa

using namespace ecospa;

extern "C" size_t ecospa_score_workspace_bytes(const ecospa_pair_t* pairs, int32_t n_pairs) {
    if (!pairs || n_pairs < 1) return 0;
    for (int i = 0; i < n_pairs; ++i)
        if (validate_pair(pairs[i], false) != ECOSPA_OK) return 0;
    bool grads = true;  // size for the larger (with-gradients) plan whenever gradients are present
    for (int i = 0; i < n_pairs; ++i) grads = grads && pairs[i].g1.ptr && pairs[i].g2.ptr;
    return plan_stats(pairs, n_pairs, grads, nullptr) * sizeof(float) + 256;
}

extern "C" ecospa_status_t ecospa_score_pairs(const ecospa_pair_t* pairs, int32_t n_pairs, double n_samples,
                                              float* upsilon, float* raw, float* fisher, void* workspace,
                                              size_t workspace_bytes, void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!pairs || n_pairs < 1 || !upsilon) return ECOSPA_ERR_INVALID;
    if (!(n_samples > 0.0)) return ECOSPA_ERR_INVALID;
    const bool grads = fisher != nullptr;
    for (int i = 0; i < n_pairs; ++i) {
        ecospa_status_t st = validate_pair(pairs[i], grads);
        if (st != ECOSPA_OK) return st;
    }
    if (!workspace || !aligned16(workspace)) return workspace ? ECOSPA_ERR_ALIGNMENT : ECOSPA_ERR_WORKSPACE;
    std::vector<StatPlan> stats;
    const size_t need = plan_stats(pairs, n_pairs, grads, &stats) * sizeof(float);
    if (workspace_bytes < need) return ECOSPA_ERR_WORKSPACE;
    float* ws = static_cast<float*>(workspace);

    // --- sumsq + reduce, in launches of at most kMaxJobs jobs
    static thread_local SumsqParams sp;
    size_t si = 0;
    while (si < stats.size()) {
        int nj = 0, tiles = 0, red = 0;
        for (; si < stats.size() && nj < kMaxJobs; ++si, ++nj) {
            const StatPlan& s = stats[si];
            const ecospa_mat_t& a = *s.a;
            SumsqJob& J = sp.jobs[nj];
            J = SumsqJob{};
            J.a = a.ptr;
            J.b = s.b ? s.b->ptr : nullptr;
            J.partial = ws + s.partial_off;
            J.stat = ws + s.stat_off;
            J.lda = static_cast<int32_t>(a.ld);
            J.ldb = s.b ? static_cast<int32_t>(s.b->ld) : 0;
            J.other = static_cast<int32_t>(a.other_dim);
            J.D = s.D;
            J.rows_per_chunk = s.rows_per_chunk;
            J.n_chunks = static_cast<uint16_t>(s.n_chunks);
            J.dtype = static_cast<uint8_t>(a.dtype);
            J.layout = static_cast<uint8_t>(a.layout);
            J.aligned = mat_aligned(a) && (!s.b || mat_aligned(*s.b));
            J.tile_start = tiles;
            J.red_start = red;
            if (J.layout == ECOSPA_SHARED_COLS) {
                const int cw = 32 * (16 / elem_bytes(J.dtype));
                J.col_tiles = static_cast<uint16_t>(ceil_div(J.D, cw));
                tiles += J.col_tiles * J.n_chunks;
            } else {
                tiles += static_cast<int>(ceil_div(J.D, kRowTile));
            }
            if (J.n_chunks > 1) red += static_cast<int>(ceil_div(J.D, kThreads));
        }
        sp.n_jobs = nj;
        sumsq_kernel<<<tiles, kThreads, 0, stream>>>(sp);
        ecospa_status_t st = check_launch("sumsq_kernel");
        if (st != ECOSPA_OK) return st;
        if (red > 0) {
            reduce_kernel<<<red, kThreads, 0, stream>>>(sp);
            if ((st = check_launch("reduce_kernel")) != ECOSPA_OK) return st;
        }
    }

    // --- finalize, in launches of at most kMaxPairs pairs
    static thread_local FinalizeParams fp;
    size_t stat_i = 0;
    int32_t d_off = 0, seg_off = 0;
    int p = 0;
    while (p < n_pairs) {
        int np = 0, segs = 0;
        const int32_t seg_base = seg_off;
        for (; p < n_pairs && np < kMaxPairs; ++p, ++np) {
            const ecospa_pair_t& pr = pairs[p];
            const bool sw = pr.kind == ECOSPA_PAIR_SWIGLU;
            PairDesc& Q = fp.pairs[np];
            Q = PairDesc{};
            Q.c1 = ws + stats[stat_i++].stat_off;
            Q.c2 = ws + stats[stat_i++].stat_off;
            if (grads) {
                Q.gs1 = ws + stats[stat_i++].stat_off;
                if (sw) Q.gs1b = ws + stats[stat_i++].stat_off;
                Q.gs2 = ws + stats[stat_i++].stat_off;
            }
            Q.n_seg = pr.n_seg;
            Q.seg_len = pr.seg_len;
            Q.rope = pr.rope;
            Q.d_off = d_off;
            Q.seg_start = segs;
            Q.rep1 = static_cast<int16_t>(std::max(1, pr.w1_rep));
            Q.rep2 = static_cast<int16_t>(std::max(1, pr.w2_rep));
            Q.inv_numel1 = static_cast<float>(1.0 / (static_cast<double>(pr.w1.other_dim) * pr.seg_len * Q.rep1));
            Q.inv_numel2 = static_cast<float>(1.0 / (static_cast<double>(pr.w2.other_dim) * pr.seg_len * Q.rep2));
            d_off += pr.n_seg * pr.seg_len;
            segs += pr.n_seg;
            seg_off += pr.n_seg;
        }
        fp.n_pairs = np;
        fp.upsilon = upsilon;
        fp.raw = raw;
        fp.fisher = fisher ? fisher + seg_base : nullptr;
        fp.inv_n_samples = 1.0 / n_samples;
        finalize_kernel<<<segs, kThreads, 0, stream>>>(fp);
        ecospa_status_t st = check_launch("finalize_kernel");
        if (st != ECOSPA_OK) return st;
    }
    return ECOSPA_OK;
}

// ---------------------------------------------------------------------------------------------
// Allocation-free variant: scores of ONE pair group with the scratch taken from a fixed array that
// lives in the library's device image instead of from a caller-provided workspace.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr size_t kStaticScratchBytes = size_t(4) << 20;  // 4 MiB, held by every GPU that loads the library

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void* g_static_ptr[kMaxDevices] = {};

// Device address of g_static_scratch on the current device (looked up once per device).
ecospa_status_t static_scratch_ptr(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        set_cuda_error(e == cudaSuccess ? cudaErrorInvalidDevice : e, "ecospa_score_pair_static: cudaGetDevice");
        return ECOSPA_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);   // the symbol itself is not a device pointer on the host
        if (e != cudaSuccess || !p) {
            set_cuda_error(e, "ecospa_score_pair_static: cudaGetSymbolAddress");
            return ECOSPA_ERR_CUDA;
        }
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return ECOSPA_OK;
}

}  // namespace

extern "C" size_t ecospa_score_pair_static_max_bytes(void) { return kStaticScratchBytes; }

extern "C" ecospa_status_t ecospa_score_pair_static(const ecospa_pair_t* pair, double n_samples, float* upsilon,
                                                    float* raw, float* fisher, void* stream) {
    if (!pair || !upsilon) return ECOSPA_ERR_INVALID;
    const ecospa_status_t vs = validate_pair(*pair, fisher != nullptr);
    if (vs != ECOSPA_OK) return vs;
    std::vector<StatPlan> stats;
    const size_t need = plan_stats(pair, 1, fisher != nullptr, &stats) * sizeof(float);
    if (need > kStaticScratchBytes) {
        set_cuda_error(cudaErrorMemoryAllocation,
                       "ecospa_score_pair_static: this pair needs more scratch than the built-in 4 MiB array; "
                       "use ecospa_score_pairs with a workspace");
        return ECOSPA_ERR_UNSUPPORTED;
    }
    void* scratch = nullptr;
    const ecospa_status_t st = static_scratch_ptr(&scratch);
    if (st != ECOSPA_OK) return st;
    return ecospa_score_pairs(pair, 1, n_samples, upsilon, raw, fisher, scratch, kStaticScratchBytes, stream);
}
