// Physical removal (Definition 1): gather of the kept shared indices of any number of tensors.
//
// shared-rows tensors: whole-row copies (out row r <- in row kept[r]), 16-byte vectors.
// shared-cols tensors: each thread owns 16 bytes of an output row (kVec adjacent kept columns,
//   indices held in registers) and walks down the rows of its tile; the gathered 2/4-byte reads
//   of neighbouring threads fall into the same 32-byte sectors (every sector of the input row
//   holds a kept element at moderate sparsity), the writes are full 16-byte vectors.
// Pad columns [n_kept, round_up(n_kept, 16 bytes)) of shared-cols outputs are zero-filled.

#include <vector>

#include "common.cuh"

namespace ecospa {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxJobs = 400;
constexpr int kColRows = 64;   // shared-cols tile: rows per CTA
constexpr int kRowTile = 32;   // shared-rows tile: output rows per CTA

struct GatherJob {
    const void* in;
    void* out;
    const int32_t* kept;
    int32_t ld_in, ld_out;   // elements
    int32_t other, D;
    int32_t n_kept;
    int32_t out_cols;        // shared-cols: columns written (n_kept + zero pad)
    int32_t tile_start;
    uint16_t col_tiles;
    uint8_t esize, layout, aligned, pad_[7];
};
static_assert(sizeof(GatherJob) == 64, "job descriptor size");

struct GatherParams {
    int32_t n_jobs;
    int32_t pad_;
    GatherJob jobs[kMaxJobs];
};

template <typename E>  // E = uint16_t or uint32_t (element as raw bits)
__device__ __forceinline__ void cols_tile(const GatherJob& J, int local) {
    constexpr int V = 16 / sizeof(E);
    constexpr int CW = 32 * V;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int ct = local % J.col_tiles, rt = local / J.col_tiles;
    const int c0 = ct * CW + lane * V;
    if (c0 >= J.out_cols) return;
    const int r0 = rt * kColRows, r1 = min(J.other, r0 + kColRows);
    int idx[V];
#pragma unroll
    for (int e = 0; e < V; ++e) {
        const int c = c0 + e;
        const int kc = c < J.n_kept ? __ldg(J.kept + c) : -1;      // -1 = no index: a zero column
        idx[e] = kc < 0 ? -1 : min(kc, J.D - 1);
    }
    const E* in = static_cast<const E*>(J.in);
    E* out = static_cast<E*>(J.out);
    const bool vec = J.aligned && (c0 + V <= J.ld_out);
    for (int r = r0 + warp; r < r1; r += 2 * kWarps) {
        E v[2][V];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int rr = r + u * kWarps;
            const E* row = in + static_cast<int64_t>(rr) * J.ld_in;
#pragma unroll
            for (int e = 0; e < V; ++e) v[u][e] = (rr < r1 && idx[e] >= 0) ? __ldg(row + idx[e]) : E(0);
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int rr = r + u * kWarps;
            if (rr >= r1) continue;
            E* orow = out + static_cast<int64_t>(rr) * J.ld_out + c0;
            if (vec) {
                uint4 pk;
                if (sizeof(E) == 2) {
                    pk.x = static_cast<uint32_t>(v[u][0]) | (static_cast<uint32_t>(v[u][1 % V]) << 16);
                    pk.y = static_cast<uint32_t>(v[u][2 % V]) | (static_cast<uint32_t>(v[u][3 % V]) << 16);
                    pk.z = static_cast<uint32_t>(v[u][4 % V]) | (static_cast<uint32_t>(v[u][5 % V]) << 16);
                    pk.w = static_cast<uint32_t>(v[u][6 % V]) | (static_cast<uint32_t>(v[u][7 % V]) << 16);
                } else {
                    pk.x = v[u][0];
                    pk.y = v[u][1 % V];
                    pk.z = v[u][2 % V];
                    pk.w = v[u][3 % V];
                }
                *reinterpret_cast<uint4*>(orow) = pk;
            } else {
#pragma unroll
                for (int e = 0; e < V; ++e)
                    if (c0 + e < J.out_cols) orow[e] = v[u][e];
            }
        }
    }
}

__device__ __forceinline__ void rows_tile(const GatherJob& J, int local) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row_bytes = static_cast<int64_t>(J.other) * J.esize;
    const int64_t pitch_in = static_cast<int64_t>(J.ld_in) * J.esize, pitch_out = static_cast<int64_t>(J.ld_out) * J.esize;
    const int64_t row_up = (row_bytes + 15) / 16 * 16;
    const int64_t pad_bytes = (pitch_out < row_up ? pitch_out : row_up) - row_bytes;
    for (int rr = warp; rr < kRowTile; rr += kWarps) {
        const int r = local * kRowTile + rr;
        if (r >= J.n_kept) break;
        const int kr = __ldg(J.kept + r);
        char* dst = static_cast<char*>(J.out) + r * pitch_out;
        if (kr < 0) {                                              // no index: a zero row
            for (int64_t b = 2 * lane; b < row_bytes + pad_bytes; b += 64) *reinterpret_cast<uint16_t*>(dst + b) = 0;
            continue;
        }
        const int src_row = min(kr, J.D - 1);
        const char* src = static_cast<const char*>(J.in) + src_row * pitch_in;
        int64_t done = 0;
        if (J.aligned) {
            const int nvec = static_cast<int>(row_bytes / 16);
            for (int v = lane; v < nvec; v += 128) {
                uint4 t[4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (v + u * 32 < nvec) t[u] = ldg_stream16(src + static_cast<int64_t>(v + u * 32) * 16);
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (v + u * 32 < nvec) *reinterpret_cast<uint4*>(dst + static_cast<int64_t>(v + u * 32) * 16) = t[u];
            }
            done = static_cast<int64_t>(nvec) * 16;
        }
        // tail (or everything when unaligned): 2-byte units, every element size is a multiple of 2
        for (int64_t b = done + 2 * lane; b < row_bytes; b += 64)
            *reinterpret_cast<uint16_t*>(dst + b) = __ldg(reinterpret_cast<const uint16_t*>(src + b));
        for (int64_t b = 2 * lane; b < pad_bytes; b += 64) *reinterpret_cast<uint16_t*>(dst + row_bytes + b) = 0;
    }
}

__global__ void __launch_bounds__(kThreads) gather_kernel(const __grid_constant__ GatherParams P) {
    const int tile = blockIdx.x;
    int lo = 0, hi = P.n_jobs - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (P.jobs[mid].tile_start <= tile) lo = mid; else hi = mid - 1;
    }
    const GatherJob& J = P.jobs[lo];
    const int local = tile - J.tile_start;
    if (J.layout == ECOSPA_SHARED_COLS) {
        if (J.esize == 2) cols_tile<uint16_t>(J, local); else cols_tile<uint32_t>(J, local);
    } else {
        rows_tile(J, local);
    }
}

bool ranges_overlap(const void* a, int64_t na, const void* b, int64_t nb) {
    const char* pa = static_cast<const char*>(a);
    const char* pb = static_cast<const char*>(b);
    return pa < pb + nb && pb < pa + na;
}

ecospa_status_t validate_job(const ecospa_gather_t& g) {
    const ecospa_mat_t& in = g.in;
    const ecospa_mat_t& out = g.out;
    if (!in.ptr || !out.ptr || !g.kept) return ECOSPA_ERR_INVALID;
    if (in.dtype != out.dtype || in.layout != out.layout || in.other_dim != out.other_dim) return ECOSPA_ERR_INVALID;
    if (in.dtype != ECOSPA_F32 && in.dtype != ECOSPA_BF16) return ECOSPA_ERR_INVALID;
    if (in.layout != ECOSPA_SHARED_COLS && in.layout != ECOSPA_SHARED_ROWS) return ECOSPA_ERR_INVALID;
    if (in.other_dim < 1 || in.other_dim > INT32_MAX || in.ld > INT32_MAX || out.ld > INT32_MAX) return ECOSPA_ERR_INVALID;
    if (g.n_kept < 0 || g.shared_dim < 1 || g.n_kept > g.shared_dim) return ECOSPA_ERR_INVALID;
    if (g.shared_dim > (1 << 22)) return ECOSPA_ERR_UNSUPPORTED;   // tile counts along the shared axis are 16-bit
    const int eb = elem_bytes(in.dtype);
    if (reinterpret_cast<uintptr_t>(in.ptr) % eb || reinterpret_cast<uintptr_t>(out.ptr) % eb) return ECOSPA_ERR_ALIGNMENT;
    int64_t in_bytes, out_bytes;
    if (in.layout == ECOSPA_SHARED_COLS) {
        if (out.ld < g.n_kept || in.ld < g.shared_dim) return ECOSPA_ERR_INVALID;
        in_bytes = in.other_dim * in.ld * eb;
        out_bytes = in.other_dim * out.ld * eb;
    } else {
        if (in.ld < in.other_dim || out.ld < in.other_dim) return ECOSPA_ERR_INVALID;
        in_bytes = static_cast<int64_t>(g.shared_dim) * in.ld * eb;
        out_bytes = static_cast<int64_t>(g.n_kept) * out.ld * eb;
    }
    if (ranges_overlap(in.ptr, in_bytes, out.ptr, out_bytes)) return ECOSPA_ERR_INVALID;
    return ECOSPA_OK;
}

}  // namespace

ecospa_status_t compact_impl(const ecospa_gather_t* jobs, int32_t n_jobs, cudaStream_t stream) {
    if (!jobs || n_jobs < 1) return ECOSPA_ERR_INVALID;
    for (int i = 0; i < n_jobs; ++i) {
        ecospa_status_t st = validate_job(jobs[i]);
        if (st != ECOSPA_OK) return st;
    }
    static thread_local GatherParams gp;
    int i = 0;
    while (i < n_jobs) {
        int nj = 0, tiles = 0;
        for (; i < n_jobs && nj < kMaxJobs; ++i) {
            const ecospa_gather_t& g = jobs[i];
            if (g.n_kept == 0) continue;
            GatherJob& J = gp.jobs[nj++];
            J = GatherJob{};
            const int eb = elem_bytes(g.in.dtype);
            J.in = g.in.ptr;
            J.out = g.out.ptr;
            J.kept = g.kept;
            J.ld_in = static_cast<int32_t>(g.in.ld);
            J.ld_out = static_cast<int32_t>(g.out.ld);
            J.other = static_cast<int32_t>(g.in.other_dim);
            J.D = g.shared_dim;
            J.n_kept = g.n_kept;
            J.esize = static_cast<uint8_t>(eb);
            J.layout = static_cast<uint8_t>(g.in.layout);
            J.tile_start = tiles;
            if (g.in.layout == ECOSPA_SHARED_COLS) {
                const int v = 16 / eb, cw = 32 * v;
                J.out_cols = static_cast<int32_t>(std::min<int64_t>(g.out.ld, round_up(g.n_kept, v)));
                J.col_tiles = static_cast<uint16_t>(ceil_div(J.out_cols, cw));
                J.aligned = aligned16(g.out.ptr) && (g.out.ld * eb) % 16 == 0;
                tiles += J.col_tiles * static_cast<int>(ceil_div(J.other, kColRows));
            } else {
                J.aligned = aligned16(g.out.ptr) && aligned16(g.in.ptr) && (g.out.ld * eb) % 16 == 0 && (g.in.ld * eb) % 16 == 0;
                tiles += static_cast<int>(ceil_div(g.n_kept, kRowTile));
            }
        }
        if (nj == 0) continue;
        gp.n_jobs = nj;
        gather_kernel<<<tiles, kThreads, 0, stream>>>(gp);
        ecospa_status_t st = check_launch("gather_kernel");
        if (st != ECOSPA_OK) return st;
    }
    return ECOSPA_OK;
}

// ------------------------------------------------------------------------------------------------
// In-place variant: out == in (same base, same pitch); the kept part moves to the front of the shared axis.
// Kept indices are ascending, so kept[c] >= c: a destination is never a source that is still needed later, as long
// as one owner walks the shared axis front to back and reads a batch before it writes it.
//   shared-cols: a warp owns a row; it gathers a batch of columns into registers, then writes the batch.
//   shared-rows: a warp owns a 512-byte stripe of columns of every row; it reads the stripe of 8 source rows, then
//                writes them to their destination rows.
// One job per launch grid slice; far fewer bytes in flight than the out-of-place kernel (memory saved, not time).
// ------------------------------------------------------------------------------------------------
struct InplaceJob {
    void* base;
    const int32_t* kept;
    int64_t ld;            // elements
    int32_t other, D, n_kept, esize, layout, warp_start, n_warps, pad_;
};
constexpr int kMaxInplaceJobs = 512;      // (28 KB of kernel parameters)
struct InplaceParams {
    int32_t n_jobs, pad_;
    InplaceJob jobs[kMaxInplaceJobs];
};

constexpr int kInplaceRows = 4;          // rows a warp compacts with one read of the kept list
constexpr int kInplaceStageBytes = 2048; // staging space per row and chunk of 256 outputs

// Shared-cols tensor, rows [row0, row0 + n_rows) of one warp.  The kept list is walked in chunks of 256 outputs (8 per
// lane); the sources of a chunk span kept[first] .. kept[last], which is read into shared memory with wide loads (all of
// the warp's rows at once, to have enough bytes in flight) and written back compacted with wide stores.  In place this
// is safe because every output index of a chunk is below every source index of the chunks after it (kept[c] >= c) and
// the chunk's own sources are all staged before its first store.  A chunk whose sources span more than the staging
// space (about one kept column in four or fewer) falls back to element-wise moves, read before written in the same way.
template <typename E>
__device__ __forceinline__ void inplace_cols_rows(const InplaceJob& J, int row0, int n_rows, int lane, uint8_t* stage_raw) {
    constexpr int V = 16 / static_cast<int>(sizeof(E));          // elements per 16-byte vector
    constexpr int kWindow = kInplaceStageBytes / static_cast<int>(sizeof(E));
    constexpr int kPer = 8;
    const int64_t padded = static_cast<int64_t>((J.n_kept + V - 1) / V) * V;
    const int out_cols = static_cast<int>(padded < J.ld ? padded : J.ld);   // kept columns + zero pad
    E* base = static_cast<E*>(J.base);
    const bool aligned = (reinterpret_cast<uintptr_t>(base) & 15u) == 0 && (J.ld * sizeof(E)) % 16 == 0;
    for (int c0 = 0; c0 < out_cols; c0 += 32 * kPer) {
        int k[kPer];
        int lo = INT32_MAX, hi = -1;
#pragma unroll
        for (int e = 0; e < kPer; ++e) {
            const int c = c0 + lane * kPer + e;
            int v = c < J.n_kept ? __ldg(J.kept + c) : -1;
            v = v < 0 ? -1 : min(v, J.D - 1);
            k[e] = v;
            if (v >= 0) {
                lo = min(lo, v);
                hi = max(hi, v);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, o));
            hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, o));
        }
        const int s0 = hi >= 0 ? (lo / V) * V : 0;               // window start, on a vector boundary of the row
        const int span = hi >= 0 ? hi + 1 - s0 : 0;
        const bool staged = span <= kWindow;
        alignas(16) E val[kInplaceRows][kPer];
        if (staged) {
#pragma unroll
            for (int r = 0; r < kInplaceRows; ++r) {
                if (r < n_rows) {
                    const E* p = base + static_cast<int64_t>(row0 + r) * J.ld + s0;
                    E* st = reinterpret_cast<E*>(stage_raw + r * kInplaceStageBytes);
                    if (aligned) {
                        for (int v = lane * V; v < span; v += 32 * V)   // (the pitch is a whole number of vectors)
                            *reinterpret_cast<uint4*>(st + v) = *reinterpret_cast<const uint4*>(p + v);
                    } else {
                        for (int v = lane; v < span; v += 32) st[v] = p[v];
                    }
                }
            }
            __syncwarp();
#pragma unroll
            for (int r = 0; r < kInplaceRows; ++r) {
                const E* st = reinterpret_cast<const E*>(stage_raw + r * kInplaceStageBytes);
#pragma unroll
                for (int e = 0; e < kPer; ++e) val[r][e] = (r < n_rows && k[e] >= 0) ? st[k[e] - s0] : E(0);
            }
        } else {
#pragma unroll
            for (int r = 0; r < kInplaceRows; ++r) {
                const E* p = base + static_cast<int64_t>(row0 + (r < n_rows ? r : 0)) * J.ld;
#pragma unroll
                for (int e = 0; e < kPer; ++e) val[r][e] = (r < n_rows && k[e] >= 0) ? p[k[e]] : E(0);
            }
        }
        __syncwarp();                                            // every source of the chunk is read before any of it is written
        const int c = c0 + lane * kPer;
#pragma unroll
        for (int r = 0; r < kInplaceRows; ++r) {
            if (r >= n_rows) continue;
            E* p = base + static_cast<int64_t>(row0 + r) * J.ld;
            if (aligned && c + kPer <= out_cols) {
                *reinterpret_cast<uint4*>(p + c) = *reinterpret_cast<const uint4*>(val[r]);
                if (sizeof(E) == 4) *reinterpret_cast<uint4*>(p + c + 4) = *reinterpret_cast<const uint4*>(val[r] + 4);
            } else {
#pragma unroll
                for (int e = 0; e < kPer; ++e)
                    if (c + e < out_cols) p[c + e] = val[r][e];
            }
        }
        __syncwarp();
    }
}

__global__ void __launch_bounds__(128) gather_inplace_kernel(const __grid_constant__ InplaceParams P) {
    const int gw = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    int ji = 0;
    while (ji + 1 < P.n_jobs && P.jobs[ji + 1].warp_start <= gw) ++ji;
    const InplaceJob& J = P.jobs[ji];
    const int w = gw - J.warp_start;
    if (w >= J.n_warps) return;
    if (J.layout == ECOSPA_SHARED_COLS) {
        __shared__ __align__(16) uint8_t stage_all[4][kInplaceRows * kInplaceStageBytes];
        const int row0 = w * kInplaceRows, n_rows = min(kInplaceRows, J.other - row0);
        if (J.esize == 2) inplace_cols_rows<uint16_t>(J, row0, n_rows, lane, stage_all[threadIdx.x >> 5]);
        else inplace_cols_rows<uint32_t>(J, row0, n_rows, lane, stage_all[threadIdx.x >> 5]);
        return;
    }
    // shared rows: this warp's stripe = bytes [128 w, 128 w + 128) of every row (4 bytes per lane; 2-byte units at a ragged
    // end: every element size divides them).  Rows move in batches of 32, each batch read before it is written; narrow
    // stripes because the batches of a stripe must follow one another, so the stripes are where the parallelism is.
    constexpr int kBatch = 32;
    const int64_t row_bytes = static_cast<int64_t>(J.other) * J.esize, pitch = J.ld * J.esize;
    const int64_t b0 = 128ll * w + 4 * lane;
    char* base = static_cast<char*>(J.base);
    if (b0 >= row_bytes) return;
    const bool vec = (reinterpret_cast<uintptr_t>(base) & 3u) == 0 && pitch % 4 == 0 && b0 + 4 <= row_bytes;
    for (int r0 = 0; r0 < J.n_kept; r0 += kBatch) {
        uint32_t v[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            v[u] = 0;
            if (r0 + u < J.n_kept) {
                const int k = __ldg(J.kept + r0 + u);
                if (k >= 0) {
                    const char* src = base + static_cast<int64_t>(min(k, J.D - 1)) * pitch + b0;
                    if (vec) {
                        v[u] = *reinterpret_cast<const uint32_t*>(src);
                    } else {                                     // unaligned tensor or the 2-byte tail of a row: halves
                        v[u] = *reinterpret_cast<const uint16_t*>(src);
                        if (b0 + 4 <= row_bytes) v[u] |= static_cast<uint32_t>(*reinterpret_cast<const uint16_t*>(src + 2)) << 16;
                    }
                }
            }
        }
        __syncwarp();
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            if (r0 + u < J.n_kept) {
                char* dst = base + static_cast<int64_t>(r0 + u) * pitch + b0;
                if (vec) {
                    *reinterpret_cast<uint32_t*>(dst) = v[u];
                } else {
                    *reinterpret_cast<uint16_t*>(dst) = static_cast<uint16_t>(v[u]);
                    if (b0 + 4 <= row_bytes) *reinterpret_cast<uint16_t*>(dst + 2) = static_cast<uint16_t>(v[u] >> 16);
                }
            }
        }
        __syncwarp();
    }
}

ecospa_status_t compact_inplace_impl(const ecospa_gather_t* jobs, int32_t n_jobs, cudaStream_t stream) {
    if (!jobs || n_jobs < 1) return ECOSPA_ERR_INVALID;
    for (int i = 0; i < n_jobs; ++i) {
        const ecospa_gather_t& g = jobs[i];
        if (!g.in.ptr || !g.kept || g.out.ptr != g.in.ptr || g.out.ld != g.in.ld) return ECOSPA_ERR_INVALID;
        if (g.in.dtype != g.out.dtype || g.in.layout != g.out.layout || g.in.other_dim != g.out.other_dim) return ECOSPA_ERR_INVALID;
        if (g.in.dtype != ECOSPA_F32 && g.in.dtype != ECOSPA_BF16) return ECOSPA_ERR_INVALID;
        if (g.in.layout != ECOSPA_SHARED_COLS && g.in.layout != ECOSPA_SHARED_ROWS) return ECOSPA_ERR_INVALID;
        if (g.in.other_dim < 1 || g.in.other_dim > INT32_MAX || g.in.ld > INT32_MAX) return ECOSPA_ERR_INVALID;
        if (g.n_kept < 0 || g.shared_dim < 1 || g.n_kept > g.shared_dim) return ECOSPA_ERR_INVALID;
        if (g.in.ld < (g.in.layout == ECOSPA_SHARED_COLS ? g.shared_dim : g.in.other_dim)) return ECOSPA_ERR_INVALID;
        if (reinterpret_cast<uintptr_t>(g.in.ptr) % elem_bytes(g.in.dtype)) return ECOSPA_ERR_ALIGNMENT;
    }
    static thread_local InplaceParams ip;
    int i = 0;
    while (i < n_jobs) {
        int nj = 0, warps = 0;
        for (; i < n_jobs && nj < kMaxInplaceJobs; ++i) {
            const ecospa_gather_t& g = jobs[i];
            if (g.n_kept == 0) continue;
            InplaceJob& J = ip.jobs[nj++];
            J = InplaceJob{};
            const int eb = elem_bytes(g.in.dtype);
            J.base = g.in.ptr; J.kept = g.kept; J.ld = g.in.ld;
            J.other = static_cast<int32_t>(g.in.other_dim); J.D = g.shared_dim; J.n_kept = g.n_kept;
            J.esize = eb; J.layout = g.in.layout; J.warp_start = warps;
            J.n_warps = g.in.layout == ECOSPA_SHARED_COLS ? static_cast<int32_t>(ceil_div(static_cast<int64_t>(J.other), static_cast<int64_t>(kInplaceRows)))
                                                           : static_cast<int32_t>(ceil_div(static_cast<int64_t>(J.other) * eb, 128));
            warps += J.n_warps;
        }
        if (nj == 0) continue;
        ip.n_jobs = nj;
        gather_inplace_kernel<<<static_cast<unsigned>(ceil_div(warps, 4)), 128, 0, stream>>>(ip);
        ecospa_status_t st = check_launch("gather_inplace_kernel");
        if (st != ECOSPA_OK) return st;
    }
    return ECOSPA_OK;
}

}  // namespace ecospa

using namespace ecospa;

extern "C" ecospa_status_t ecospa_compact_tensors(const ecospa_gather_t* jobs, int32_t n_jobs, void* stream) {
    return compact_impl(jobs, n_jobs, static_cast<cudaStream_t>(stream));
}

extern "C" ecospa_status_t ecospa_compact_tensors_inplace(const ecospa_gather_t* jobs, int32_t n_jobs, void* stream) {
    return compact_inplace_impl(jobs, n_jobs, static_cast<cudaStream_t>(stream));
}

extern "C" ecospa_status_t ecospa_compact_pair(const ecospa_pair_t* pair, const int32_t* kept, int32_t n_kept,
                                               const ecospa_mat_t* aux_in, const ecospa_mat_t* aux_out,
                                               int32_t n_aux, const ecospa_mat_t* w1_out,
                                               const ecospa_mat_t* w1b_out, const ecospa_mat_t* w2_out,
                                               void* stream) {
    if (!pair || !kept || n_kept < 0 || n_aux < 0 || !w1_out || !w2_out) return ECOSPA_ERR_INVALID;
    if (n_aux > 0 && (!aux_in || !aux_out)) return ECOSPA_ERR_INVALID;
    const bool sw = pair->kind == ECOSPA_PAIR_SWIGLU;
    if (sw && !w1b_out) return ECOSPA_ERR_INVALID;
    if (pair->n_seg < 1 || pair->seg_len < 1) return ECOSPA_ERR_INVALID;
    // grouped heads: the two sides have different shared extents and kept lists; use ecospa_compact_tensors
    if (pair->w1_rep > 1 || pair->w2_rep > 1) return ECOSPA_ERR_UNSUPPORTED;
    const int64_t D = static_cast<int64_t>(pair->n_seg) * pair->seg_len;
    if (n_kept > D) return ECOSPA_ERR_INVALID;
    std::vector<ecospa_gather_t> jobs;
    auto add = [&](const ecospa_mat_t& in, const ecospa_mat_t& out) {
        ecospa_gather_t g{};
        g.in = in;
        g.out = out;
        g.kept = kept;
        g.n_kept = n_kept;
        g.shared_dim = static_cast<int32_t>(D);
        jobs.push_back(g);
    };
    add(pair->w1, *w1_out);
    if (sw) add(pair->w1b, *w1b_out);
    add(pair->w2, *w2_out);
    for (int i = 0; i < n_aux; ++i) add(aux_in[i], aux_out[i]);
    return compact_impl(jobs.data(), static_cast<int32_t>(jobs.size()), static_cast<cudaStream_t>(stream));
}
