// Aligned top-k per segment (Definition 1 applied to the lowest-scored indices).
//
// One CTA per segment.  The k-th largest score is found by a 4-pass radix select over an
// order-preserving 32-bit key; the kept indices are then emitted in ascending order with a
// block-wide stream compaction, taking equal-to-threshold scores lowest index first.  The score
// vector of a segment (<= 44 KB at the shapes of interest) is re-read from L1/L2 in each pass.

#include <vector>

#include "common.cuh"

namespace ecospa {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxSegs = 4096;   // per launch (16 KB of offsets)
constexpr int kMaxPairs = 256;   // per launch

struct SelPair {
    int32_t seg_start;  // first segment (within this launch) of the pair
    int32_t seg_len;
    int32_t d_off;      // offset of the pair's scores in upsilon, and base added to nothing: kept
                        // indices are relative to the pair group (segment offset included)
    int32_t rope;       // ecospa_rope_t: units of two shared indices are ranked and kept together
};

struct SelectParams {
    const float* upsilon;
    int32_t* kept;
    int32_t* seg_offsets;   // may be null; global prefix sums of k
    int32_t n_pairs, n_segs;
    int32_t seg_base;       // global index of this launch's first segment
    int32_t is_last;        // this launch writes the final seg_offsets entry
    const int32_t* k_dev;   // non-null: kept counts are read from the device (indexed by global segment) and
                            // segment s of a pair writes at the pair's score offset + s * seg_len
    SelPair pairs[kMaxPairs];
    int32_t out_off[kMaxSegs + 1];  // global offsets into kept
};

// fp32 -> uint32 whose unsigned order is the float order; -0 and +0 map to the same key.
__device__ __forceinline__ uint32_t order_key(float f) {
    uint32_t u = __float_as_uint(f);
    if (u == 0x80000000u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// ROPE = false: no pair group of the launch has rotation pairs (the common case, compiled without the unit logic).
template <bool ROPE>
__global__ void __launch_bounds__(kThreads) select_kernel(const __grid_constant__ SelectParams P) {
    __shared__ int hist[256];
    __shared__ int warp_tot[kWarps];
    __shared__ uint32_t sh_prefix;
    __shared__ int sh_want, sh_cnt_eq;

    const int seg = blockIdx.x;
    int lo = 0, hi = P.n_pairs - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (P.pairs[mid].seg_start <= seg) lo = mid; else hi = mid - 1;
    }
    const SelPair& Q = P.pairs[lo];
    const int seg_len = Q.seg_len;
    const int seg_in_pair = seg - Q.seg_start;
    // With rotation pairs the ranked units are the seg_len/2 pairs; both members carry the pair's score, so
    // unit u is read at index 2u (interleaved pairs) or u (pairs of the two halves).
    const int rope = ROPE ? Q.rope : ECOSPA_ROPE_NONE;
    const int n = rope ? seg_len >> 1 : seg_len;
    const int stride = rope == ECOSPA_ROPE_INTERLEAVED ? 2 : 1;
    const float* sc = P.upsilon + Q.d_off + static_cast<int64_t>(seg_in_pair) * seg_len;
    const int out0 = P.k_dev ? Q.d_off + seg_in_pair * seg_len : P.out_off[seg];
    const int k_idx = P.k_dev ? min(max(P.k_dev[P.seg_base + seg], 0), seg_len) : P.out_off[seg + 1] - out0;
    const int k = rope ? k_idx >> 1 : k_idx;     // units to keep
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (P.seg_offsets && tid == 0) {
        P.seg_offsets[P.seg_base + seg] = out0;
        if (P.is_last && seg == P.n_segs - 1) P.seg_offsets[P.seg_base + seg + 1] = out0 + k_idx;
    }
    if (k <= 0) return;

    // ---- radix select: key of the k-th largest element
    uint32_t prefix = 0, mask = 0;
    int want = k, cnt_eq = 0;
    for (int shift = 24; shift >= 0; shift -= 8) {
        hist[tid] = 0;
        __syncthreads();
        for (int j = tid; j < n; j += kThreads) {
            const uint32_t key = order_key(__ldg(sc + j * stride));
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255], 1);
        }
        __syncthreads();
        if (warp == 0) {
            // lane l owns bins 255-8l ... 248-8l (descending)
            int local[8], s = 0;
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                local[b] = hist[255 - 8 * lane - b];
                s += local[b];
            }
            int incl = s;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            const int excl = incl - s;
            if (excl < want && want <= incl) {
                int cum = excl;
#pragma unroll
                for (int b = 0; b < 8; ++b) {
                    if (cum < want && want <= cum + local[b]) {
                        sh_prefix = prefix | (static_cast<uint32_t>(255 - 8 * lane - b) << shift);
                        sh_want = want - cum;
                        sh_cnt_eq = local[b];
                    }
                    cum += local[b];
                }
            }
        }
        __syncthreads();
        prefix = sh_prefix;
        want = sh_want;
        cnt_eq = sh_cnt_eq;
        mask |= 255u << shift;
        __syncthreads();
    }
    const uint32_t thr = prefix;            // key of the k-th largest
    const bool all_eq = (want == cnt_eq);   // every element equal to the threshold is kept

    // ---- emit ascending: key > thr, plus the first `want` elements with key == thr
    const int seg_first = seg_in_pair * seg_len;  // kept indices are shared indices of the pair group
    int run_eq = 0, run_out = 0;
    for (int base = 0; base < n; base += kThreads) {
        const int j = base + tid;
        uint32_t key = 0;
        bool valid = j < n;
        if (valid) key = order_key(__ldg(sc + j * stride));
        const bool gt = valid && key > thr;
        const bool eq = valid && key == thr;
        bool sel;
        if (all_eq) {
            sel = gt || eq;
        } else {
            const unsigned beq = __ballot_sync(0xffffffffu, eq);
            if (lane == 0) warp_tot[warp] = __popc(beq);
            __syncthreads();
            int rank = run_eq + __popc(beq & ((1u << lane) - 1u));
            int tot = 0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                if (w < warp) rank += warp_tot[w];
                tot += warp_tot[w];
            }
            run_eq += tot;
            sel = gt || (eq && rank < want);
            __syncthreads();
        }
        const unsigned bs = __ballot_sync(0xffffffffu, sel);
        if (lane == 0) warp_tot[warp] = __popc(bs);
        __syncthreads();
        int pos = run_out + __popc(bs & ((1u << lane) - 1u));
        int tot = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            if (w < warp) pos += warp_tot[w];
            tot += warp_tot[w];
        }
        run_out += tot;
        if (sel && pos < k) {
            if (rope == ECOSPA_ROPE_NONE) {
                P.kept[out0 + pos] = seg_first + j;
            } else if (rope == ECOSPA_ROPE_INTERLEAVED) {           // members 2j, 2j + 1
                P.kept[out0 + 2 * pos] = seg_first + 2 * j;
                P.kept[out0 + 2 * pos + 1] = seg_first + 2 * j + 1;
            } else {                                                // members j, j + seg_len/2: both halves ascending
                P.kept[out0 + pos] = seg_first + j;
                P.kept[out0 + k + pos] = seg_first + n + j;
            }
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------------
// Algorithm 1's stopping rule: how many indices of a segment stay when the smallest scores are removed
// while the sum of what is left exceeds theta * total.
// ---------------------------------------------------------------------------------------------
// Sum over the block in a fixed order (thread partial -> shuffle tree -> warps in order); all threads get it.
__device__ __forceinline__ double block_sum_f64(double v, double* scratch) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) t += scratch[w];
    return t;
}

struct ThresholdParams {
    const float* upsilon;
    const int32_t* chosen;  // per global segment, may be null
    int32_t* k_out;         // per global segment
    double theta;
    int32_t l1, k_min;
    int32_t n_pairs, seg_base;
    SelPair pairs[kMaxPairs];
};

// One CTA per segment.  The kept set is {key >= t} plus the first e elements of the tie group just below t,
// where t is the smallest key threshold whose scores sum to at most the budget: found by bisection over
// the 32-bit key space, every sum taken in fp64 over the whole segment.
__global__ void __launch_bounds__(kThreads) threshold_count_kernel(const __grid_constant__ ThresholdParams P) {
    __shared__ double scratch[kWarps];
    __shared__ uint32_t sh_max[kWarps];
    const int seg = blockIdx.x;
    int lo_p = 0, hi_p = P.n_pairs - 1;
    while (lo_p < hi_p) {
        const int mid = (lo_p + hi_p + 1) >> 1;
        if (P.pairs[mid].seg_start <= seg) lo_p = mid; else hi_p = mid - 1;
    }
    const SelPair& Q = P.pairs[lo_p];
    // with rotation pairs the units are the seg_len/2 pairs, each counted once (its score sits at its first member)
    const int unit = Q.rope ? 2 : 1;
    const int n = Q.seg_len / unit;
    const int stride = Q.rope == ECOSPA_ROPE_INTERLEAVED ? 2 : 1;
    const float* sc = P.upsilon + Q.d_off + static_cast<int64_t>(seg - Q.seg_start) * Q.seg_len;
    const int tid = threadIdx.x;
    const int gseg = P.seg_base + seg;
    if (P.chosen && P.chosen[gseg] == 0) {
        if (tid == 0) P.k_out[gseg] = Q.seg_len;
        return;
    }
    // sum of the scores whose key is at least t, and how many there are
    auto mass_ge = [&](uint64_t t, int* count) -> double {
        double s = 0.0;
        int c = 0;
        for (int j = tid; j < n; j += kThreads) {
            const float f = __ldg(sc + j * stride);
            if (static_cast<uint64_t>(order_key(f)) >= t) {
                s += static_cast<double>(f);
                ++c;
            }
        }
        if (count) *count = static_cast<int>(block_sum_f64(static_cast<double>(c), scratch));
        return block_sum_f64(s, scratch);
    };
    const double all = mass_ge(0, nullptr);
    const double budget = P.theta * (P.l1 ? all : 1.0);
    int k = n;
    if (all > budget) {
        uint64_t lo = 0, hi = 1ull << 32;        // the empty set (t = 2^32) always fits
        while (lo < hi) {
            const uint64_t mid = (lo + hi) >> 1;
            if (mass_ge(mid, nullptr) <= budget) hi = mid; else lo = mid + 1;
        }
        int cnt = 0;
        double s = mass_ge(hi, &cnt);
        // tie group just below the threshold: its largest key, its size and its (common) value
        uint32_t below = 0;
        bool any = false;
        for (int j = tid; j < n; j += kThreads) {
            const uint32_t key = order_key(__ldg(sc + j * stride));
            if (static_cast<uint64_t>(key) < hi) {
                below = any ? max(below, key) : key;
                any = true;
            }
        }
        // block maximum of (any, below): encode "none" as 0 with a flag bit in 64 bits
        unsigned long long enc = any ? (1ull << 32) | below : 0ull;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) enc = max(enc, __shfl_xor_sync(0xffffffffu, enc, o));
        __syncthreads();
        if ((tid & 31) == 0) {
            sh_max[tid >> 5] = static_cast<uint32_t>(enc);
            scratch[tid >> 5] = static_cast<double>(enc >> 32);
        }
        __syncthreads();
        bool have = false;
        uint32_t tkey = 0;
        for (int w = 0; w < kWarps; ++w)
            if (scratch[w] != 0.0) {
                tkey = have ? max(tkey, sh_max[w]) : sh_max[w];
                have = true;
            }
        __syncthreads();
        int e = 0;
        if (have) {
            double val = 0.0;
            int c = 0;
            for (int j = tid; j < n; j += kThreads) {
                const float f = __ldg(sc + j * stride);
                if (order_key(f) == tkey) {
                    val = static_cast<double>(f);
                    ++c;
                }
            }
            const int ties = static_cast<int>(block_sum_f64(static_cast<double>(c), scratch));
            // every thread that saw one holds the same value; take the maximum over the block
            double vmax = val;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) vmax = fmax(vmax, __shfl_xor_sync(0xffffffffu, vmax, o));
            __syncthreads();
            if ((tid & 31) == 0) scratch[tid >> 5] = vmax;
            __syncthreads();
            double v = scratch[0];
            for (int w = 1; w < kWarps; ++w) v = fmax(v, scratch[w]);
            __syncthreads();
            // (scores below zero do not occur: they are norms; a zero tie group adds nothing and always fits)
            for (int j = 1; j <= ties; ++j) {
                s += v;
                if (s <= budget) e = j; else break;
            }
        }
        k = cnt + e;
    }
    k = max(k, min((P.k_min + unit - 1) / unit, n));
    if (tid == 0) P.k_out[gseg] = k * unit;
}

// chosen[i] = 1 for the m smallest values (equal values: lower index first): rank by counting.
__global__ void __launch_bounds__(1024) choose_pairs_kernel(const float* __restrict__ fisher, int n, int m,
                                                            int32_t* __restrict__ chosen) {
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const float fi = fisher[i];
        int rank = 0;
        for (int j = 0; j < n; ++j) {
            const float fj = __ldg(fisher + j);
            rank += (fj < fi || (fj == fi && j < i)) ? 1 : 0;
        }
        chosen[i] = rank < m ? 1 : 0;
    }
}

// Packs the per-segment slots of the variable-count selection into one ascending list per pair group:
// out[dst[s] + i] = slots[src[s] + i] + add[s] for i < k[s].
constexpr int kPackSegs = 512;
struct PackParams {
    const int32_t* slots;
    int32_t* out;
    int32_t n;
    int32_t src[kPackSegs], dst[kPackSegs], k[kPackSegs], add[kPackSegs];
};
__global__ void __launch_bounds__(128) pack_kept_kernel(const __grid_constant__ PackParams P) {
    const int s = blockIdx.x;
    for (int i = threadIdx.x; i < P.k[s]; i += blockDim.x) P.out[P.dst[s] + i] = P.slots[P.src[s] + i] + P.add[s];
}

// Kept list with padded segments: the k[s] entries of segment s, then -1 ("no index") up to its padded count
// (carried in the `add` slot of the parameters).
__global__ void __launch_bounds__(128) pad_kept_kernel(const __grid_constant__ PackParams P) {
    const int s = blockIdx.x;
    for (int i = threadIdx.x; i < P.add[s]; i += blockDim.x) P.out[P.dst[s] + i] = i < P.k[s] ? P.slots[P.src[s] + i] : -1;
}

}  // namespace

}  // namespace ecospa

using namespace ecospa;

extern "C" ecospa_status_t ecospa_pad_kept(const int32_t* kept, const int32_t* src, const int32_t* dst, const int32_t* k,
                                           const int32_t* k_padded, int32_t n_segs, int32_t* out, void* stream) {
    if (!kept || !src || !dst || !k || !k_padded || !out || n_segs < 1) return ECOSPA_ERR_INVALID;
    for (int i = 0; i < n_segs; ++i)
        if (src[i] < 0 || dst[i] < 0 || k[i] < 0 || k_padded[i] < k[i]) return ECOSPA_ERR_INVALID;
    static thread_local PackParams pp;
    for (int base = 0; base < n_segs; base += kPackSegs) {
        const int n = std::min(kPackSegs, n_segs - base);
        pp.slots = kept; pp.out = out; pp.n = n;
        for (int i = 0; i < n; ++i) {
            pp.src[i] = src[base + i]; pp.dst[i] = dst[base + i]; pp.k[i] = k[base + i]; pp.add[i] = k_padded[base + i];
        }
        pad_kept_kernel<<<n, 128, 0, static_cast<cudaStream_t>(stream)>>>(pp);
        const ecospa_status_t st = check_launch("pad_kept_kernel");
        if (st != ECOSPA_OK) return st;
    }
    return ECOSPA_OK;
}

extern "C" ecospa_status_t ecospa_pack_kept(const int32_t* slots, const int32_t* src, const int32_t* dst, const int32_t* k,
                                            const int32_t* add, int32_t n_segs, int32_t* out, void* stream) {
    if (!slots || !src || !dst || !k || !add || !out || n_segs < 1) return ECOSPA_ERR_INVALID;
    for (int i = 0; i < n_segs; ++i)
        if (src[i] < 0 || dst[i] < 0 || k[i] < 0) return ECOSPA_ERR_INVALID;
    static thread_local PackParams pp;
    for (int base = 0; base < n_segs; base += kPackSegs) {
        const int n = std::min(kPackSegs, n_segs - base);
        pp.slots = slots; pp.out = out; pp.n = n;
        for (int i = 0; i < n; ++i) {
            pp.src[i] = src[base + i]; pp.dst[i] = dst[base + i]; pp.k[i] = k[base + i]; pp.add[i] = add[base + i];
        }
        pack_kept_kernel<<<n, 128, 0, static_cast<cudaStream_t>(stream)>>>(pp);
        const ecospa_status_t st = check_launch("pack_kept_kernel");
        if (st != ECOSPA_OK) return st;
    }
    return ECOSPA_OK;
}

static ecospa_status_t select_fixed_counts(const float* upsilon, const int32_t* n_seg, const int32_t* seg_len,
                                           const int32_t* k_per_seg, const int32_t* rope, int32_t n_pairs,
                                           int32_t* kept, int32_t* seg_offsets, void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!upsilon || !n_seg || !seg_len || !k_per_seg || n_pairs < 1 || !kept) return ECOSPA_ERR_INVALID;
    int64_t total_segs = 0, total_d = 0, total_k = 0;
    for (int p = 0; p < n_pairs; ++p) {
        if (n_seg[p] < 1 || seg_len[p] < 1) return ECOSPA_ERR_INVALID;
        if (seg_len[p] > (1 << 20)) return ECOSPA_ERR_UNSUPPORTED;
        const int32_t rp = rope ? rope[p] : ECOSPA_ROPE_NONE;
        if (rp != ECOSPA_ROPE_NONE && rp != ECOSPA_ROPE_INTERLEAVED && rp != ECOSPA_ROPE_HALF) return ECOSPA_ERR_INVALID;
        if (rp != ECOSPA_ROPE_NONE && (seg_len[p] & 1)) return ECOSPA_ERR_INVALID;
        for (int s = 0; s < n_seg[p]; ++s) {
            const int32_t k = k_per_seg[total_segs + s];
            if (k < 0 || k > seg_len[p]) return ECOSPA_ERR_INVALID;
            if (rp != ECOSPA_ROPE_NONE && (k & 1)) return ECOSPA_ERR_INVALID;   // whole rotation pairs only
            total_k += k;
        }
        total_segs += n_seg[p];
        total_d += static_cast<int64_t>(n_seg[p]) * seg_len[p];
    }
    if (total_d > INT32_MAX || total_k > INT32_MAX) return ECOSPA_ERR_UNSUPPORTED;

    static thread_local SelectParams sp;
    int p = 0, s_in_p = 0;          // walk position: pair, segment inside pair
    int32_t d_off = 0, out = 0, seg_global = 0;
    while (p < n_pairs) {
        int np = 0, ns = 0;
        sp.seg_base = seg_global;
        // a pair can be split across launches; each launch sees it as a pair starting at s_in_p
        while (p < n_pairs && np < kMaxPairs && ns < kMaxSegs) {
            const int take = std::min(n_seg[p] - s_in_p, kMaxSegs - ns);
            SelPair& Q = sp.pairs[np++];
            Q.seg_start = ns - s_in_p;   // so that (seg - seg_start) is the segment index inside the pair
            Q.seg_len = seg_len[p];
            Q.d_off = d_off;
            Q.rope = rope ? rope[p] : ECOSPA_ROPE_NONE;
            for (int s = 0; s < take; ++s) {
                sp.out_off[ns++] = out;
                out += k_per_seg[seg_global++];
            }
            s_in_p += take;
            if (s_in_p == n_seg[p]) {
                d_off += n_seg[p] * seg_len[p];
                ++p;
                s_in_p = 0;
            }
        }
        sp.out_off[ns] = out;
        sp.upsilon = upsilon;
        sp.kept = kept;
        sp.k_dev = nullptr;
        sp.seg_offsets = seg_offsets;
        sp.n_pairs = np;
        sp.n_segs = ns;
        sp.is_last = (p >= n_pairs) ? 1 : 0;
        bool any_rope = false;
        for (int i = 0; i < np; ++i) any_rope = any_rope || sp.pairs[i].rope != ECOSPA_ROPE_NONE;
        if (any_rope) select_kernel<true><<<ns, kThreads, 0, stream>>>(sp);
        else select_kernel<false><<<ns, kThreads, 0, stream>>>(sp);
        ecospa_status_t st = check_launch("select_kernel");
        if (st != ECOSPA_OK) return st;
    }
    return ECOSPA_OK;
}

extern "C" ecospa_status_t ecospa_select_aligned_topk(const float* upsilon, const int32_t* n_seg,
                                                      const int32_t* seg_len, const int32_t* k_per_seg,
                                                      int32_t n_pairs, int32_t* kept, int32_t* seg_offsets,
                                                      void* stream) {
    return select_fixed_counts(upsilon, n_seg, seg_len, k_per_seg, nullptr, n_pairs, kept, seg_offsets, stream);
}

extern "C" ecospa_status_t ecospa_select_rotation_pairs(const float* upsilon, const int32_t* n_seg,
                                                        const int32_t* seg_len, const int32_t* k_per_seg,
                                                        const int32_t* rope, int32_t n_pairs, int32_t* kept,
                                                        int32_t* seg_offsets, void* stream) {
    if (!rope) return ECOSPA_ERR_INVALID;
    return select_fixed_counts(upsilon, n_seg, seg_len, k_per_seg, rope, n_pairs, kept, seg_offsets, stream);
}

extern "C" ecospa_status_t ecospa_select_aligned_threshold(const float* upsilon, const int32_t* n_seg,
                                                           const int32_t* seg_len, const int32_t* rope, int32_t n_pairs,
                                                           double theta, int32_t l1, int32_t k_min, const int32_t* chosen,
                                                           int32_t* kept, int32_t* k_out, void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!upsilon || !n_seg || !seg_len || n_pairs < 1 || !kept || !k_out) return ECOSPA_ERR_INVALID;
    if (!(theta >= 0.0) || k_min < 0) return ECOSPA_ERR_INVALID;
    int64_t total_d = 0;
    for (int p = 0; p < n_pairs; ++p) {
        if (n_seg[p] < 1 || seg_len[p] < 1) return ECOSPA_ERR_INVALID;
        if (seg_len[p] > (1 << 20)) return ECOSPA_ERR_UNSUPPORTED;
        const int32_t rp = rope ? rope[p] : ECOSPA_ROPE_NONE;
        if (rp != ECOSPA_ROPE_NONE && rp != ECOSPA_ROPE_INTERLEAVED && rp != ECOSPA_ROPE_HALF) return ECOSPA_ERR_INVALID;
        if (rp != ECOSPA_ROPE_NONE && (seg_len[p] & 1)) return ECOSPA_ERR_INVALID;
        total_d += static_cast<int64_t>(n_seg[p]) * seg_len[p];
    }
    if (total_d > INT32_MAX) return ECOSPA_ERR_UNSUPPORTED;

    static thread_local ThresholdParams tp;
    static thread_local SelectParams sp;
    int p = 0, s_in_p = 0;
    int32_t d_off = 0, seg_global = 0;
    while (p < n_pairs) {
        int np = 0, ns = 0;
        const int32_t seg_base = seg_global;
        while (p < n_pairs && np < kMaxPairs && ns < kMaxSegs) {
            const int take = std::min(n_seg[p] - s_in_p, kMaxSegs - ns);
            SelPair& Q = sp.pairs[np];
            Q.seg_start = ns - s_in_p;
            Q.seg_len = seg_len[p];
            Q.d_off = d_off;
            Q.rope = rope ? rope[p] : ECOSPA_ROPE_NONE;
            tp.pairs[np] = Q;
            ++np;
            ns += take;
            seg_global += take;
            s_in_p += take;
            if (s_in_p == n_seg[p]) {
                d_off += n_seg[p] * seg_len[p];
                ++p;
                s_in_p = 0;
            }
        }
        tp.upsilon = upsilon; tp.chosen = chosen; tp.k_out = k_out;
        tp.theta = theta; tp.l1 = l1 ? 1 : 0; tp.k_min = k_min;
        tp.n_pairs = np; tp.seg_base = seg_base;
        threshold_count_kernel<<<ns, kThreads, 0, stream>>>(tp);
        ecospa_status_t st = check_launch("threshold_count_kernel");
        if (st != ECOSPA_OK) return st;
        // the fixed-count selection, with the counts just written and one slot of seg_len entries per segment
        sp.upsilon = upsilon; sp.kept = kept; sp.seg_offsets = nullptr;
        sp.n_pairs = np; sp.n_segs = ns; sp.seg_base = seg_base; sp.is_last = 0;
        sp.k_dev = k_out;
        bool any_rope = false;
        for (int i = 0; i < np; ++i) any_rope = any_rope || sp.pairs[i].rope != ECOSPA_ROPE_NONE;
        if (any_rope) select_kernel<true><<<ns, kThreads, 0, stream>>>(sp);
        else select_kernel<false><<<ns, kThreads, 0, stream>>>(sp);
        if ((st = check_launch("select_kernel")) != ECOSPA_OK) return st;
    }
    return ECOSPA_OK;
}

extern "C" ecospa_status_t ecospa_choose_pairs(const float* fisher, int32_t n, int32_t m, int32_t* chosen, void* stream_) {
    if (!fisher || !chosen || n < 1 || m < 0) return ECOSPA_ERR_INVALID;
    if (n > 16384) return ECOSPA_ERR_UNSUPPORTED;
    const int grid = (n + 1023) / 1024;
    choose_pairs_kernel<<<grid, 1024, 0, static_cast<cudaStream_t>(stream_)>>>(fisher, n, m, chosen);
    return check_launch("choose_pairs_kernel");
}
