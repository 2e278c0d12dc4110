// Forward / backward of the compacted coupled pairs (Eq. 2, 3, 5 after aligned removal), expressed as
// grouped launches of the tcgen05 GEMM engine plus two small helper kernels (fp32 -> bf16 staging for
// fp32 models, and column sums for the bias gradients).
//
// Storage: every compacted weight is accepted as d_m x n (ECOSPA_SHARED_COLS) or n x d_m (ECOSPA_SHARED_ROWS),
// row-major; the equations' orientation is d_m x n for W_Q^c, W_K^c, W_V^c, W_1^c (gate/up) and n x d_m for
// W_O^c, W_2^c (down).  Every product below consumes its operands as stored (K-major or MN-major UMMA
// operands, chosen from the weight's layout); nothing is transposed in memory, and a weight gradient is
// written in the orientation of its weight.

#include <cuda_bf16.h>

#include <algorithm>

#include "common.cuh"
#include "gemm.cuh"

namespace ecospa {

namespace {

constexpr int kThreads = 256;

// ------------------------------------------------------------------------------------------------
// helper kernels
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) cast_f32_bf16_kernel(const float* __restrict__ in, int64_t ld_in,
                                                                 uint16_t* __restrict__ out, int64_t ld_out, int64_t rows,
                                                                 int64_t cols, int64_t cols_out) {
    // one thread per 4 output columns; columns [cols, cols_out) are zero-filled
    const int64_t per_row = (cols_out + 3) / 4;
    const int64_t total = rows * per_row;
    for (int64_t i = blockIdx.x * static_cast<int64_t>(kThreads) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * kThreads) {
        const int64_t r = i / per_row, c = (i % per_row) * 4;
        for (int e = 0; e < 4; ++e) {
            if (c + e < cols_out) {
                const float v = (c + e < cols) ? in[r * ld_in + c + e] : 0.f;
                __nv_bfloat16 b = __float2bfloat16_rn(v);
                out[r * ld_out + c + e] = *reinterpret_cast<uint16_t*>(&b);
            }
        }
    }
}

// These helpers are launched with programmatic stream serialization, like the GEMM engine: their blocks may be
// placed while the previous kernel drains, and touch no global memory before pdl_wait().
__device__ __forceinline__ void pdl_start() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename Params>
cudaError_t launch_pdl(void (*kernel)(Params), dim3 grid, cudaStream_t stream, const Params& p) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

// Column sums (bias gradients) of up to two bf16 matrices with the same number of rows, two launches:
// partial[chunk][c] over tiles of kSumRows rows x 64 columns (8 lanes cover a row's 128 bytes with
// 16-byte loads, the block covers 32 rows per pass, all 4 passes in flight at once: the kernel is one round
// of loads deep and its grid is large), then a fixed-order sum of the chunks.
constexpr int kSumRows = 128;
constexpr int kSumCols = 64;
struct ColsumJob {
    const uint16_t* M;
    float* partial;
    void* out;
    int64_t ld, cols;
    int32_t col_tiles, vec_ok;
};
struct ColsumParams {
    ColsumJob job[3];
    int64_t rows;
    int32_t n_jobs, chunks, out_f32;
};

__global__ void __launch_bounds__(kThreads) colsum_partial_kernel(const __grid_constant__ ColsumParams P) {
    __shared__ float red[32][kSumCols + 1];
    pdl_start();
    pdl_wait();
    int ji = 0, ct = blockIdx.x;
    while (ji + 1 < P.n_jobs && ct >= P.job[ji].col_tiles) {
        ct -= P.job[ji].col_tiles;
        ++ji;
    }
    const ColsumJob& J = P.job[ji];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int rowoff = (lane >> 3) + 4 * warp;              // 0..31
    const int64_t c0 = static_cast<int64_t>(ct) * kSumCols + (lane & 7) * 8;
    const int64_t r0 = static_cast<int64_t>(blockIdx.y) * kSumRows;
    const int64_t r1 = r0 + kSumRows < P.rows ? r0 + kSumRows : P.rows;
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    if (c0 < J.cols) {
        if (J.vec_ok && c0 + 8 <= J.cols) {
            const uint16_t* p = J.M + c0;
            for (int64_t r = r0 + rowoff; r < r1; r += 128) {
                uint4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int64_t rr = r + 32 * u;
                    v[u] = rr < r1 ? ldg_stream16(p + rr * J.ld) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    acc[0] += bf16_lo(v[u].x); acc[1] += bf16_hi(v[u].x);
                    acc[2] += bf16_lo(v[u].y); acc[3] += bf16_hi(v[u].y);
                    acc[4] += bf16_lo(v[u].z); acc[5] += bf16_hi(v[u].z);
                    acc[6] += bf16_lo(v[u].w); acc[7] += bf16_hi(v[u].w);
                }
            }
        } else {
            for (int64_t r = r0 + rowoff; r < r1; r += 32)
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if (c0 + e < J.cols) acc[e] += __uint_as_float(static_cast<uint32_t>(J.M[r * J.ld + c0 + e]) << 16);
        }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) red[rowoff][(lane & 7) * 8 + e] = acc[e];
    __syncthreads();
    if (threadIdx.x < kSumCols) {
        const int64_t c = static_cast<int64_t>(ct) * kSumCols + threadIdx.x;
        if (c < J.cols) {
            float s = 0.f;
#pragma unroll
            for (int w = 0; w < 32; ++w) s += red[w][threadIdx.x];
            J.partial[static_cast<int64_t>(blockIdx.y) * J.cols + c] = s;
        }
    }
}
// One launch that finishes a call: out[r][c] = sum over s of partial[s][r][c] for up to three split-K weight
// gradients (summed in split order), and the fixed-order sum of the column-sum chunks.
struct ReduceJob {
    const float* partial;
    void* out;
    int64_t rows, cols, ldp, ld_out;
    int32_t splits, blk_start, n_blk, pad_;
};
struct PostParams {
    ReduceJob red[3];
    ColsumParams cs;
    int32_t n_red, red_blocks, out_f32, pad_;
};
__host__ __device__ inline int64_t round_up32(int64_t v) { return (v + 31) & ~int64_t(31); }
__global__ void __launch_bounds__(kThreads) post_kernel(const __grid_constant__ PostParams P) {
    __shared__ float part[8][32];
    pdl_start();
    pdl_wait();
    if (static_cast<int>(blockIdx.x) < P.red_blocks) {
        int ji = 0;
        while (ji + 1 < P.n_red && static_cast<int>(blockIdx.x) >= P.red[ji + 1].blk_start) ++ji;
        const ReduceJob& J = P.red[ji];
        const int64_t per_row = (J.cols + 3) / 4;
        const int64_t total = J.rows * per_row;
        const int64_t plane = J.rows * J.ldp;
        for (int64_t i = (blockIdx.x - J.blk_start) * static_cast<int64_t>(kThreads) + threadIdx.x; i < total;
             i += static_cast<int64_t>(J.n_blk) * kThreads) {
            const int64_t r = i / per_row, c = (i % per_row) * 4;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int s2 = 0; s2 < J.splits; ++s2) {
                const float4 v = *reinterpret_cast<const float4*>(J.partial + s2 * plane + r * J.ldp + c);
                acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
            }
            const float a[4] = {acc.x, acc.y, acc.z, acc.w};
            for (int e = 0; e < 4; ++e) {
                if (c + e < J.cols) {
                    if (P.out_f32) static_cast<float*>(J.out)[r * J.ld_out + c + e] = a[e];
                    else static_cast<__nv_bfloat16*>(J.out)[r * J.ld_out + c + e] = __float2bfloat16_rn(a[e]);
                }
            }
        }
        return;
    }
    // column-sum finals: a block takes 32 columns; warp g adds chunks g, g + 8, ... and warp 0 adds the 8 sums
    const int g = threadIdx.x >> 5;
    int64_t c = static_cast<int64_t>(blockIdx.x - P.red_blocks) * 32 + (threadIdx.x & 31);
    int ji = 0;
    while (ji < P.cs.n_jobs && c >= round_up32(P.cs.job[ji].cols)) {
        c -= round_up32(P.cs.job[ji].cols);
        ++ji;
    }
    const bool live = ji < P.cs.n_jobs && c < P.cs.job[ji].cols;
    float s = 0.f;
    if (live) {
        const float* p = P.cs.job[ji].partial + c;
        const int64_t cols = P.cs.job[ji].cols;
        for (int k = g; k < P.cs.chunks; k += 8) s += p[static_cast<int64_t>(k) * cols];
    }
    part[g][threadIdx.x & 31] = s;
    __syncthreads();
    if (g == 0 && live) {
        float t = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) t += part[i][threadIdx.x];
        if (P.out_f32) static_cast<float*>(P.cs.job[ji].out)[c] = t;
        else static_cast<__nv_bfloat16*>(P.cs.job[ji].out)[c] = __float2bfloat16_rn(t);
    }
}

// ------------------------------------------------------------------------------------------------
// workspace bump allocator and operand staging
// ------------------------------------------------------------------------------------------------
struct Arena {
    char* base = nullptr;
    size_t size = 0, used = 0;
    void* take(size_t bytes) {
        const size_t a = (used + 255) & ~size_t(255);
        if (!base || a + bytes > size) return nullptr;
        used = a + bytes;
        return base + a;
    }
};
inline size_t arena_need(size_t bytes) { return ((bytes + 255) & ~size_t(255)) + 256; }

struct Ctx {
    cudaStream_t stream = nullptr;
    Arena arena;
    int dtype = ECOSPA_BF16;  // of the model (activations, weights, outputs)
    ecospa_status_t st = ECOSPA_OK;
};

// A (rows x cols, pitch ld) matrix of the model dtype as a bf16 Stored operand (staged if fp32).
Stored as_bf16(Ctx& cx, const void* p, int64_t rows, int64_t cols, int64_t ld) {
    Stored s;
    if (cx.st != ECOSPA_OK) return s;
    if (!p || rows < 1 || cols < 1 || ld < cols) {
        cx.st = ECOSPA_ERR_INVALID;
        return s;
    }
    if (cx.dtype == ECOSPA_BF16) {
        s.ptr = p; s.rows = rows; s.cols = cols; s.ld = ld;
        return s;
    }
    const int64_t ldo = round_up(cols, 8);
    void* buf = cx.arena.take(static_cast<size_t>(rows) * ldo * 2);
    if (!buf) {
        cx.st = ECOSPA_ERR_WORKSPACE;
        return s;
    }
    const int64_t total = rows * ((ldo + 3) / 4);
    const int grid = static_cast<int>(std::min<int64_t>(ceil_div(total, kThreads), 148 * 16));
    cast_f32_bf16_kernel<<<grid, kThreads, 0, cx.stream>>>(static_cast<const float*>(p), ld, static_cast<uint16_t*>(buf), ldo,
                                                           rows, cols, ldo);
    cx.st = check_launch("cast_f32_bf16_kernel");
    s.ptr = buf; s.rows = rows; s.cols = cols; s.ld = ldo;
    return s;
}

// bf16 scratch matrix (rows x cols) from the workspace.
Stored scratch_bf16(Ctx& cx, int64_t rows, int64_t cols) {
    Stored s;
    if (cx.st != ECOSPA_OK) return s;
    const int64_t ld = round_up(cols, 8);
    void* buf = cx.arena.take(static_cast<size_t>(rows) * ld * 2);
    if (!buf) {
        cx.st = ECOSPA_ERR_WORKSPACE;
        return s;
    }
    s.ptr = buf; s.rows = rows; s.cols = cols; s.ld = ld;
    return s;
}

// Column sums of up to three bf16 matrices with the same row count.  colsum_plan takes the scratch of the chunk
// partials from the workspace (so that a short workspace is reported before anything is launched) and returns the
// description that colsum_begin (launch of the chunk-partial kernel) and the finishing launch need.  A null output
// skips that matrix.
ColsumParams colsum_plan(Ctx& cx, const Stored& M1, void* out1, const Stored& M2 = Stored(), void* out2 = nullptr,
                         const Stored& M3 = Stored(), void* out3 = nullptr) {
    ColsumParams P = {};
    if (cx.st != ECOSPA_OK) return P;
    const Stored* mats[3] = {&M1, &M2, &M3};
    void* outs[3] = {out1, out2, out3};
    for (int i = 0; i < 3; ++i) {
        if (!outs[i] || !mats[i]->ptr) continue;
        ColsumJob& J = P.job[P.n_jobs++];
        J.M = static_cast<const uint16_t*>(mats[i]->ptr);
        J.out = outs[i];
        J.ld = mats[i]->ld;
        J.cols = mats[i]->cols;
        J.col_tiles = static_cast<int32_t>(ceil_div(J.cols, kSumCols));
        J.vec_ok = aligned16(J.M) && J.ld % 8 == 0;
        P.rows = mats[i]->rows;
    }
    if (P.n_jobs == 0) return P;
    P.chunks = static_cast<int32_t>(ceil_div(P.rows, kSumRows));
    P.out_f32 = cx.dtype == ECOSPA_F32;
    for (int i = 0; i < P.n_jobs; ++i) {
        P.job[i].partial = static_cast<float*>(cx.arena.take(static_cast<size_t>(P.chunks) * P.job[i].cols * 4));
        if (!P.job[i].partial) {
            cx.st = ECOSPA_ERR_WORKSPACE;
            P.n_jobs = 0;
            return P;
        }
    }
    return P;
}
const ColsumParams& colsum_begin(Ctx& cx, const ColsumParams& P) {
    if (cx.st != ECOSPA_OK || P.n_jobs == 0) return P;
    int tiles = 0;
    for (int i = 0; i < P.n_jobs; ++i) tiles += P.job[i].col_tiles;
    const cudaError_t e = launch_pdl(colsum_partial_kernel, dim3(tiles, P.chunks), cx.stream, P);
    if (e != cudaSuccess) {
        set_cuda_error(e, "colsum_partial_kernel launch");
        cudaGetLastError();
        cx.st = ECOSPA_ERR_CUDA;
        return P;
    }
    cx.st = check_launch("colsum_partial_kernel");
    return P;
}

// Compacted weight with n real shared indices, as stored: shared-cols d_m x n, or shared-rows n x d_m.  Either
// orientation is accepted for every weight: the engine consumes K-major and MN-major operands alike, so a
// stored orientation only decides which of the two a product sees (and in which orientation the weight
// gradient is written: the same as the weight).
ecospa_status_t check_weight(const ecospa_mat_t* w, int64_t d_m, int64_t n, int dtype) {
    if (!w || !w->ptr) return ECOSPA_ERR_INVALID;
    if (w->dtype != dtype || w->other_dim != d_m) return ECOSPA_ERR_INVALID;
    if (w->layout != ECOSPA_SHARED_COLS && w->layout != ECOSPA_SHARED_ROWS) return ECOSPA_ERR_INVALID;
    if (w->ld < (w->layout == ECOSPA_SHARED_COLS ? n : d_m)) return ECOSPA_ERR_INVALID;
    return ECOSPA_OK;
}
// Is the weight an MN-major B operand ([K][N] in memory) of a product that contracts over d_m (output = shared
// index), respectively over the shared index (output = d_m)?
bool mn_over_other(const ecospa_mat_t* w) { return w->layout == ECOSPA_SHARED_COLS; }
bool mn_over_shared(const ecospa_mat_t* w) { return w->layout == ECOSPA_SHARED_ROWS; }
Stored weight_bf16(Ctx& cx, const ecospa_mat_t* w, int64_t d_m, int64_t n) {
    if (w->layout == ECOSPA_SHARED_COLS) return as_bf16(cx, w->ptr, d_m, n, w->ld);
    return as_bf16(cx, w->ptr, n, d_m, w->ld);
}

ecospa_status_t begin(Ctx& cx, int dtype, void* workspace, size_t workspace_bytes, void* stream, int64_t T, int64_t d_m, int64_t n) {
    if (dtype != ECOSPA_F32 && dtype != ECOSPA_BF16) return ECOSPA_ERR_INVALID;
    if (T < 1 || d_m < 1 || n < 1) return ECOSPA_ERR_INVALID;
    if (workspace && !aligned16(workspace)) return ECOSPA_ERR_ALIGNMENT;
    cx.stream = static_cast<cudaStream_t>(stream);
    cx.arena.base = static_cast<char*>(workspace);
    cx.arena.size = workspace ? workspace_bytes : 0;
    cx.dtype = dtype;
    return ECOSPA_OK;
}

size_t staged(int dtype, int64_t rows, int64_t cols) {  // bytes as_bf16 takes from the arena
    return dtype == ECOSPA_F32 ? arena_need(static_cast<size_t>(rows) * round_up(cols, 8) * 2) : 0;
}
size_t scratch(int64_t rows, int64_t cols) { return arena_need(static_cast<size_t>(rows) * round_up(cols, 8) * 2); }
size_t colsum_need(int64_t rows, int64_t cols) { return arena_need(static_cast<size_t>(ceil_div(rows, kSumRows)) * cols * 4); }

// C (T x n) = X (stored T x d_m, K-major) * W (d_m x n consumed MN-major, or n x d_m consumed K-major) [+ bias]
GemmOp proj_op(const Stored& X, const Stored& W, bool w_mn, int64_t T, int64_t d_m, int64_t n, const void* bias, void* out, int64_t ld_out, int dtype) {
    GemmOp op;
    op.M = T; op.N = n; op.n_kseg = 1;
    op.seg[0].a = X; op.seg[0].a_mn = false;
    op.seg[0].b[0] = W; op.seg[0].b_mn = w_mn;
    op.seg[0].K = d_m;
    op.epi = EPI_STORE;
    op.C = out; op.ldc = ld_out; op.out_f32 = dtype == ECOSPA_F32;
    op.bias = bias; op.bias_f32 = dtype == ECOSPA_F32;
    return op;
}
// Weight gradients contract over the T tokens and have few output tiles, so on their own they would keep
// most SMs idle behind one long tile.  The token range is therefore cut into `splits` ranges computed as
// separate ops of the same launch into fp32 partial buffers, which the finishing launch (post_kernel) adds up in split order.
// Workers of a launch: the CTA pairs the engine keeps resident on the current device (74 on a 148-SM part, which is
// also what the size queries assume when no device can be asked).
int64_t engine_workers() {
    static thread_local int cached = 0;
    if (cached <= 0) {
        const int n = gemm_resident_pairs();
        if (n <= 0) return 74;
        cached = n;
    }
    return cached;
}
// Cost of a product in k-blocks of 256x256 tiles (what one worker spends on it if it ran alone).
int64_t gemm_cost(int64_t M, int64_t N, int64_t K) { return ceil_div(M, 256) * ceil_div(N, 256) * ceil_div(K, 64); }
// `launch_cost` = cost of every product of the launch.  The scheduler hands tiles out longest first, so a
// tile much longer than a worker's fair share of the launch sets the duration: cut the tokens until it is
// not (a tile up to 1.3 shares is left whole: the partial sums and their reduction cost more than they save).
int wgrad_splits(int64_t rows_out, int64_t cols_out, int64_t T, int64_t launch_cost) {
    const int64_t share = std::max<int64_t>(launch_cost / engine_workers(), 1);
    int64_t s = ceil_div(10 * ceil_div(T, 64), 13 * share);
    s = std::min<int64_t>(s, T / 1024);            // at least 16 k-blocks per range
    s = std::min<int64_t>(s, 6);
    return static_cast<int>(std::max<int64_t>(s, 1));
}
// Upper bound of the partial buffers over every launch this product can be part of (its own cost alone).
size_t wgrad_need_one(int64_t rows_out, int64_t cols_out, int64_t T) {
    const int S = wgrad_splits(rows_out, cols_out, T, gemm_cost(rows_out, cols_out, T));
    return S > 1 ? arena_need(static_cast<size_t>(S) * rows_out * round_up(cols_out, 4) * 4) : 0;
}
// the gradient is written in the weight's orientation, which the size query does not know
size_t wgrad_need(int64_t rows_out, int64_t cols_out, int64_t T) {
    return std::max(wgrad_need_one(rows_out, cols_out, T), wgrad_need_one(cols_out, rows_out, T));
}
struct PendingReduce {
    const float* partial = nullptr;
    int splits = 0;
    int64_t rows = 0, cols = 0, ldp = 0, ld_out = 0;
    void* out = nullptr;
};
// dW (rows_out x cols_out) = Xs^T dYs  with Xs stored T x rows_out and dYs stored T x cols_out.
// Appends 1 or `splits` ops to ops[n_ops...] and returns the new op count.  `reserve` = ops the caller
// still has to append after this one; the split count is reduced so that everything fits kMaxGemmOps.
int add_wgrad(Ctx& cx, GemmOp* ops, int n_ops, const Stored& Xs, const Stored& dYs, int64_t rows_out, int64_t cols_out,
              int64_t T, void* out, int64_t ld_out, PendingReduce* red, int reserve, int64_t launch_cost) {
    GemmOp op;
    op.M = rows_out; op.N = cols_out; op.n_kseg = 1;
    op.seg[0].a = Xs; op.seg[0].a_mn = true;
    op.seg[0].b[0] = dYs; op.seg[0].b_mn = true;
    op.epi = EPI_STORE;
    int S = wgrad_splits(rows_out, cols_out, T, launch_cost);
    S = std::max(1, std::min(S, (kMaxGemmOps - n_ops - reserve) / std::max(1, reserve)));
    if (cx.st != ECOSPA_OK) return n_ops;
    if (n_ops + 1 + reserve > kMaxGemmOps) {
        cx.st = ECOSPA_ERR_INVALID;
        return n_ops;
    }
    if (S == 1) {
        op.seg[0].K = T;
        op.C = out; op.ldc = ld_out; op.out_f32 = cx.dtype == ECOSPA_F32;
        ops[n_ops++] = op;
        return n_ops;
    }
    const int64_t ldp = round_up(cols_out, 4);
    float* partial = static_cast<float*>(cx.arena.take(static_cast<size_t>(S) * rows_out * ldp * 4));
    if (!partial) {
        cx.st = ECOSPA_ERR_WORKSPACE;
        return n_ops;
    }
    const int64_t per = round_up(ceil_div(T, S), 64);
    int used = 0;
    for (int i = 0; i < S; ++i) {
        const int64_t k0 = i * per;
        if (k0 >= T) break;
        op.seg[0].k_begin = k0;
        op.seg[0].K = std::min<int64_t>(per, T - k0);
        op.C = partial + static_cast<int64_t>(i) * rows_out * ldp;
        op.ldc = ldp;
        op.out_f32 = true;
        ops[n_ops++] = op;
        ++used;
    }
    red->partial = partial; red->splits = used; red->rows = rows_out; red->cols = cols_out; red->ldp = ldp;
    red->out = out; red->ld_out = ld_out;
    return n_ops;
}
// Gradient of a weight stored like `w`: d_m x n = other^T shared for a shared-cols weight, n x d_m = shared^T other
// for a shared-rows one (other_act: T x d_m on the d_m side of the weight, shared_act: T x n on its shared side).
int add_wgrad_w(Ctx& cx, GemmOp* ops, int n_ops, const ecospa_mat_t* w, const Stored& other_act, const Stored& shared_act,
                int64_t d_m, int64_t n, int64_t T, void* out, int64_t ld_out, PendingReduce* red, int reserve,
                int64_t launch_cost) {
    if (w->layout == ECOSPA_SHARED_COLS)
        return add_wgrad(cx, ops, n_ops, other_act, shared_act, d_m, n, T, out, ld_out, red, reserve, launch_cost);
    return add_wgrad(cx, ops, n_ops, shared_act, other_act, n, d_m, T, out, ld_out, red, reserve, launch_cost);
}

// The finishing launch of a call: split-K reductions and column-sum finals together.
void finish(Ctx& cx, const PendingReduce* red, int n_red, const ColsumParams& cs) {
    if (cx.st != ECOSPA_OK) return;
    PostParams P = {};
    P.cs = cs;
    P.out_f32 = cx.dtype == ECOSPA_F32;
    int blocks = 0;
    for (int i = 0; i < n_red; ++i) {
        const PendingReduce& r = red[i];
        if (r.splits == 0) continue;
        ReduceJob& J = P.red[P.n_red++];
        J.partial = r.partial; J.out = r.out; J.rows = r.rows; J.cols = r.cols; J.ldp = r.ldp; J.ld_out = r.ld_out;
        J.splits = r.splits;
        const int64_t total = r.rows * ((r.cols + 3) / 4);
        J.n_blk = static_cast<int32_t>(std::min<int64_t>(ceil_div(total, kThreads), 148 * 4));
        J.blk_start = blocks;
        blocks += J.n_blk;
    }
    P.red_blocks = blocks;
    for (int i = 0; i < cs.n_jobs; ++i) blocks += static_cast<int>(round_up32(cs.job[i].cols) / 32);
    if (blocks == 0) return;
    const cudaError_t e = launch_pdl(post_kernel, dim3(blocks), cx.stream, P);
    if (e != cudaSuccess) {
        set_cuda_error(e, "post_kernel launch");
        cudaGetLastError();
        cx.st = ECOSPA_ERR_CUDA;
        return;
    }
    cx.st = check_launch("post_kernel");
}

}  // namespace

}  // namespace ecospa

using namespace ecospa;

extern "C" size_t ecospa_proj_workspace_bytes(int64_t T, int64_t d_m, int64_t n, int32_t dtype) {
    // worst case over the qk / vo calls: staged X, Ctx, upstream grads, weights, and the column-sum partials
    const size_t w = std::max(staged(dtype, d_m, n), staged(dtype, n, d_m));   // a weight in either orientation
    return staged(dtype, T, d_m) * 2 + w * 4 + staged(dtype, T, n) * 4 + colsum_need(T, n) * 3 + colsum_need(T, d_m) +
           wgrad_need(d_m, n, T) * 4 + 1024;
}

extern "C" size_t ecospa_ffn_workspace_bytes(int64_t T, int64_t d_m, int64_t k, int32_t act, int32_t dtype) {
    const int nw = act == ECOSPA_ACT_SWIGLU ? 2 : 1;
    const size_t w = std::max(staged(dtype, d_m, k), staged(dtype, k, d_m));   // a weight in either orientation
    return staged(dtype, T, d_m) * 2 + w * (nw + 1) + scratch(T, k) * nw + colsum_need(T, k) + colsum_need(T, d_m) +
           wgrad_need(d_m, k, T) * (nw + 1) + 1024;
}

extern "C" ecospa_status_t ecospa_coupled_qk_fwd(const void* X, int64_t ldx, int64_t T, int64_t d_m,
                                                 const ecospa_mat_t* wq_c, const ecospa_mat_t* wk_c, int64_t n,
                                                 const void* bq_c, const void* bk_c, void* Qc, void* Kc, int64_t ld_out,
                                                 void* workspace, size_t workspace_bytes, void* stream) {
    if (!wq_c || !Qc) return ECOSPA_ERR_INVALID;
    Ctx cx;
    ecospa_status_t st = begin(cx, wq_c->dtype, workspace, workspace_bytes, stream, T, d_m, n);
    if (st != ECOSPA_OK) return st;
    if ((st = check_weight(wq_c, d_m, n, cx.dtype)) != ECOSPA_OK) return st;
    if (wk_c && (st = check_weight(wk_c, d_m, n, cx.dtype)) != ECOSPA_OK) return st;
    if (wk_c && !Kc) return ECOSPA_ERR_INVALID;
    const Stored Xs = as_bf16(cx, X, T, d_m, ldx);
    GemmOp ops[2];
    int n_ops = 0;
    ops[n_ops++] = proj_op(Xs, weight_bf16(cx, wq_c, d_m, n), mn_over_other(wq_c), T, d_m, n, bq_c, Qc, ld_out, cx.dtype);
    if (wk_c) ops[n_ops++] = proj_op(Xs, weight_bf16(cx, wk_c, d_m, n), mn_over_other(wk_c), T, d_m, n, bk_c, Kc, ld_out, cx.dtype);
    if (cx.st != ECOSPA_OK) return cx.st;
    return launch_grouped_gemm(ops, n_ops, cx.stream);
}

extern "C" ecospa_status_t ecospa_coupled_qk_bwd(const void* X, int64_t ldx, int64_t T, int64_t d_m,
                                                 const ecospa_mat_t* wq_c, const ecospa_mat_t* wk_c, int64_t n,
                                                 const void* dQc, const void* dKc, int64_t ld_dqk, void* dX, int64_t ld_dx,
                                                 int32_t accumulate_dX, void* dWq_c, void* dWk_c, int64_t ld_dw,
                                                 void* dbq_c, void* dbk_c, void* workspace, size_t workspace_bytes,
                                                 void* stream) {
    if (!wq_c || !dQc || !dX || !dWq_c) return ECOSPA_ERR_INVALID;
    if (wk_c && (!dKc || !dWk_c)) return ECOSPA_ERR_INVALID;
    Ctx cx;
    ecospa_status_t st = begin(cx, wq_c->dtype, workspace, workspace_bytes, stream, T, d_m, n);
    if (st != ECOSPA_OK) return st;
    if ((st = check_weight(wq_c, d_m, n, cx.dtype)) != ECOSPA_OK) return st;
    if (wk_c && (st = check_weight(wk_c, d_m, n, cx.dtype)) != ECOSPA_OK) return st;
    const bool f32 = cx.dtype == ECOSPA_F32;
    const Stored Xs = as_bf16(cx, X, T, d_m, ldx);
    const Stored dQs = as_bf16(cx, dQc, T, n, ld_dqk);
    const Stored Wq = weight_bf16(cx, wq_c, d_m, n);
    Stored dKs, Wk;
    if (wk_c) {
        dKs = as_bf16(cx, dKc, T, n, ld_dqk);
        Wk = weight_bf16(cx, wk_c, d_m, n);
    }
    if (cx.st != ECOSPA_OK) return cx.st;
    GemmOp ops[kMaxGemmOps];
    PendingReduce red[2];
    int n_ops = 0;
    const int64_t cost = (wk_c ? 2 : 1) * (gemm_cost(d_m, n, T) + gemm_cost(T, d_m, n));
    n_ops = add_wgrad_w(cx, ops, n_ops, wq_c, Xs, dQs, d_m, n, T, dWq_c, ld_dw, &red[0], wk_c ? 2 : 1, cost);
    if (wk_c) n_ops = add_wgrad_w(cx, ops, n_ops, wk_c, Xs, dKs, d_m, n, T, dWk_c, ld_dw, &red[1], 1, cost);
    if (cx.st != ECOSPA_OK) return cx.st;
    // dX = dQ W_Q^T (+ dK W_K^T): weights stored d_m x n are K-major B operands here
    GemmOp& dx = ops[n_ops++];
    dx.M = T; dx.N = d_m; dx.n_kseg = wk_c ? 2 : 1;
    dx.seg[0].a = dQs; dx.seg[0].b[0] = Wq; dx.seg[0].b_mn = mn_over_shared(wq_c); dx.seg[0].K = n;
    if (wk_c) {
        dx.seg[1].a = dKs; dx.seg[1].b[0] = Wk; dx.seg[1].b_mn = mn_over_shared(wk_c); dx.seg[1].K = n;
    }
    dx.epi = EPI_STORE; dx.C = dX; dx.ldc = ld_dx; dx.out_f32 = f32; dx.accumulate = accumulate_dX != 0;
    const ColsumParams cs = colsum_plan(cx, dQs, dbq_c, dKs, wk_c ? dbk_c : nullptr);
    if (cx.st != ECOSPA_OK) return cx.st;
    if ((st = launch_grouped_gemm(ops, n_ops, cx.stream)) != ECOSPA_OK) return st;
    finish(cx, red, 2, colsum_begin(cx, cs));
    return cx.st;
}

extern "C" ecospa_status_t ecospa_coupled_vo_fwd_v(const void* X, int64_t ldx, int64_t T, int64_t d_m,
                                                   const ecospa_mat_t* wv_c, int64_t n, const void* bv_c, void* Vc,
                                                   int64_t ld_out, void* workspace, size_t workspace_bytes, void* stream) {
    return ecospa_coupled_qk_fwd(X, ldx, T, d_m, wv_c, nullptr, n, bv_c, nullptr, Vc, nullptr, ld_out, workspace,
                                 workspace_bytes, stream);
}

extern "C" ecospa_status_t ecospa_coupled_vo_fwd_o(const void* Ctxm, int64_t ld_ctx, int64_t T, int64_t d_m,
                                                   const ecospa_mat_t* wo_c, int64_t n, const void* bo, void* Out,
                                                   int64_t ld_out, void* workspace, size_t workspace_bytes, void* stream) {
    if (!wo_c || !Out) return ECOSPA_ERR_INVALID;
    Ctx cx;
    ecospa_status_t st = begin(cx, wo_c->dtype, workspace, workspace_bytes, stream, T, d_m, n);
    if (st != ECOSPA_OK) return st;
    if ((st = check_weight(wo_c, d_m, n, cx.dtype)) != ECOSPA_OK) return st;
    GemmOp op;
    op.M = T; op.N = d_m; op.n_kseg = 1;
    op.seg[0].a = as_bf16(cx, Ctxm, T, n, ld_ctx);
    op.seg[0].b[0] = weight_bf16(cx, wo_c, d_m, n);   // stored n x d_m = [K][N], or d_m x n = [N][K]
    op.seg[0].b_mn = mn_over_shared(wo_c);
    op.seg[0].K = n;
    op.epi = EPI_STORE; op.C = Out; op.ldc = ld_out; op.out_f32 = cx.dtype == ECOSPA_F32;
    op.bias = bo; op.bias_f32 = cx.dtype == ECOSPA_F32;
    if (cx.st != ECOSPA_OK) return cx.st;
    return launch_grouped_gemm(&op, 1, cx.stream);
}

extern "C" ecospa_status_t ecospa_coupled_vo_bwd(const void* X, int64_t ldx, const void* Ctxm, int64_t ld_ctx, int64_t T,
                                                 int64_t d_m, const ecospa_mat_t* wv_c, const ecospa_mat_t* wo_c, int64_t n,
                                                 const void* dVc, int64_t ld_dv, const void* dOut, int64_t ld_dout,
                                                 void* dX, int64_t ld_dx, int32_t accumulate_dX, void* dCtx, int64_t ld_dctx,
                                                 void* dWv_c, int64_t ld_dwv, void* dWo_c, int64_t ld_dwo, void* dbv_c,
                                                 void* dbo, void* workspace, size_t workspace_bytes, void* stream) {
    if (!wv_c || !wo_c || !dVc || !dOut || !dX || !dCtx || !dWv_c || !dWo_c) return ECOSPA_ERR_INVALID;
    Ctx cx;
    ecospa_status_t st = begin(cx, wv_c->dtype, workspace, workspace_bytes, stream, T, d_m, n);
    if (st != ECOSPA_OK) return st;
    if ((st = check_weight(wv_c, d_m, n, cx.dtype)) != ECOSPA_OK) return st;
    if ((st = check_weight(wo_c, d_m, n, cx.dtype)) != ECOSPA_OK) return st;
    const bool f32 = cx.dtype == ECOSPA_F32;
    const Stored Xs = as_bf16(cx, X, T, d_m, ldx);
    const Stored Cs = as_bf16(cx, Ctxm, T, n, ld_ctx);
    const Stored dVs = as_bf16(cx, dVc, T, n, ld_dv);
    const Stored dOs = as_bf16(cx, dOut, T, d_m, ld_dout);
    const Stored Wv = weight_bf16(cx, wv_c, d_m, n);
    const Stored Wo = weight_bf16(cx, wo_c, d_m, n);
    if (cx.st != ECOSPA_OK) return cx.st;
    GemmOp ops[kMaxGemmOps];
    PendingReduce red[2];
    int n_ops = 0;
    // dW_O (n x d_m) = Ctx^T dOut ; dW_V (d_m x n) = X^T dV
    const int64_t cost = gemm_cost(n, d_m, T) + gemm_cost(d_m, n, T) + gemm_cost(T, n, d_m) + gemm_cost(T, d_m, n);
    n_ops = add_wgrad_w(cx, ops, n_ops, wo_c, dOs, Cs, d_m, n, T, dWo_c, ld_dwo, &red[0], 3, cost);
    n_ops = add_wgrad_w(cx, ops, n_ops, wv_c, Xs, dVs, d_m, n, T, dWv_c, ld_dwv, &red[1], 2, cost);
    if (cx.st != ECOSPA_OK) return cx.st;
    // dCtx (T x n) = dOut W_O^T : W_O stored n x d_m = [N][K]
    GemmOp& dc = ops[n_ops++];
    dc.M = T; dc.N = n; dc.n_kseg = 1;
    dc.seg[0].a = dOs; dc.seg[0].b[0] = Wo; dc.seg[0].b_mn = mn_over_other(wo_c); dc.seg[0].K = d_m;
    dc.epi = EPI_STORE; dc.C = dCtx; dc.ldc = ld_dctx; dc.out_f32 = f32;
    // dX (T x d_m) = dV W_V^T : W_V stored d_m x n = [N][K]
    GemmOp& dx = ops[n_ops++];
    dx.M = T; dx.N = d_m; dx.n_kseg = 1;
    dx.seg[0].a = dVs; dx.seg[0].b[0] = Wv; dx.seg[0].b_mn = mn_over_shared(wv_c); dx.seg[0].K = n;
    dx.epi = EPI_STORE; dx.C = dX; dx.ldc = ld_dx; dx.out_f32 = f32; dx.accumulate = accumulate_dX != 0;
    const ColsumParams cs = colsum_plan(cx, dVs, dbv_c, dOs, dbo);
    if (cx.st != ECOSPA_OK) return cx.st;
    if ((st = launch_grouped_gemm(ops, n_ops, cx.stream)) != ECOSPA_OK) return st;
    finish(cx, red, 2, colsum_begin(cx, cs));
    return cx.st;
}

// Q^c, K^c and V^c in one launch (the QK and VO pairs of a block read the same X).
extern "C" ecospa_status_t ecospa_coupled_qkv_fwd(const void* X, int64_t ldx, int64_t T, int64_t d_m,
                                                  const ecospa_mat_t* wq_c, const ecospa_mat_t* wk_c,
                                                  const ecospa_mat_t* wv_c, int64_t n_qk, int64_t n_vo, const void* bq_c,
                                                  const void* bk_c, const void* bv_c, void* Qc, void* Kc, void* Vc,
                                                  int64_t ld_qk, int64_t ld_v, void* workspace, size_t workspace_bytes,
                                                  void* stream) {
    if (!wq_c || !wk_c || !wv_c || !Qc || !Kc || !Vc) return ECOSPA_ERR_INVALID;
    Ctx cx;
    ecospa_status_t st = begin(cx, wq_c->dtype, workspace, workspace_bytes, stream, T, d_m, std::min(n_qk, n_vo));
    if (st != ECOSPA_OK) return st;
    if ((st = check_weight(wq_c, d_m, n_qk, cx.dtype)) != ECOSPA_OK) return st;
    if ((st = check_weight(wk_c, d_m, n_qk, cx.dtype)) != ECOSPA_OK) return st;
    if ((st = check_weight(wv_c, d_m, n_vo, cx.dtype)) != ECOSPA_OK) return st;
    const Stored Xs = as_bf16(cx, X, T, d_m, ldx);
    GemmOp ops[3];
    ops[0] = proj_op(Xs, weight_bf16(cx, wq_c, d_m, n_qk), mn_over_other(wq_c), T, d_m, n_qk, bq_c, Qc, ld_qk, cx.dtype);
    ops[1] = proj_op(Xs, weight_bf16(cx, wk_c, d_m, n_qk), mn_over_other(wk_c), T, d_m, n_qk, bk_c, Kc, ld_qk, cx.dtype);
    ops[2] = proj_op(Xs, weight_bf16(cx, wv_c, d_m, n_vo), mn_over_other(wv_c), T, d_m, n_vo, bv_c, Vc, ld_v, cx.dtype);
    if (cx.st != ECOSPA_OK) return cx.st;
    return launch_grouped_gemm(ops, 3, cx.stream);
}

// Backward of the three projections in one launch: dW_Q^c, dW_K^c, dW_V^c (split over the tokens when they
// have few tiles) and dX = dQ W_Q^cT + dK W_K^cT + dV W_V^cT as one product over three K segments.
extern "C" ecospa_status_t ecospa_coupled_qkv_bwd(const void* X, int64_t ldx, int64_t T, int64_t d_m,
                                                  const ecospa_mat_t* wq_c, const ecospa_mat_t* wk_c,
                                                  const ecospa_mat_t* wv_c, int64_t n_qk, int64_t n_vo, const void* dQc,
                                                  const void* dKc, const void* dVc, int64_t ld_dqk, int64_t ld_dv,
                                                  void* dX, int64_t ld_dx, int32_t accumulate_dX, void* dWq_c,
                                                  void* dWk_c, void* dWv_c, int64_t ld_dwqk, int64_t ld_dwv, void* dbq_c,
                                                  void* dbk_c, void* dbv_c, void* workspace, size_t workspace_bytes,
                                                  void* stream) {
    if (!wq_c || !wk_c || !wv_c || !dQc || !dKc || !dVc || !dX || !dWq_c || !dWk_c || !dWv_c) return ECOSPA_ERR_INVALID;
    Ctx cx;
    ecospa_status_t st = begin(cx, wq_c->dtype, workspace, workspace_bytes, stream, T, d_m, std::min(n_qk, n_vo));
    if (st != ECOSPA_OK) return st;
    if ((st = check_weight(wq_c, d_m, n_qk, cx.dtype)) != ECOSPA_OK) return st;
    if ((st = check_weight(wk_c, d_m, n_qk, cx.dtype)) != ECOSPA_OK) return st;
    if ((st = check_weight(wv_c, d_m, n_vo, cx.dtype)) != ECOSPA_OK) return st;
    const Stored Xs = as_bf16(cx, X, T, d_m, ldx);
    const Stored dQs = as_bf16(cx, dQc, T, n_qk, ld_dqk);
    const Stored dKs = as_bf16(cx, dKc, T, n_qk, ld_dqk);
    const Stored dVs = as_bf16(cx, dVc, T, n_vo, ld_dv);
    const Stored Wq = weight_bf16(cx, wq_c, d_m, n_qk);
    const Stored Wk = weight_bf16(cx, wk_c, d_m, n_qk);
    const Stored Wv = weight_bf16(cx, wv_c, d_m, n_vo);
    if (cx.st != ECOSPA_OK) return cx.st;
    GemmOp ops[kMaxGemmOps];
    PendingReduce red[3];
    int n_ops = 0;
    const int64_t cost = 2 * gemm_cost(d_m, n_qk, T) + gemm_cost(d_m, n_vo, T) + gemm_cost(T, d_m, 2 * n_qk + n_vo);
    n_ops = add_wgrad_w(cx, ops, n_ops, wq_c, Xs, dQs, d_m, n_qk, T, dWq_c, ld_dwqk, &red[0], 3, cost);
    n_ops = add_wgrad_w(cx, ops, n_ops, wk_c, Xs, dKs, d_m, n_qk, T, dWk_c, ld_dwqk, &red[1], 2, cost);
    n_ops = add_wgrad_w(cx, ops, n_ops, wv_c, Xs, dVs, d_m, n_vo, T, dWv_c, ld_dwv, &red[2], 1, cost);
    if (cx.st != ECOSPA_OK) return cx.st;
    GemmOp& dx = ops[n_ops++];
    dx.M = T; dx.N = d_m; dx.n_kseg = 3;
    dx.seg[0].a = dQs; dx.seg[0].b[0] = Wq; dx.seg[0].b_mn = mn_over_shared(wq_c); dx.seg[0].K = n_qk;
    dx.seg[1].a = dKs; dx.seg[1].b[0] = Wk; dx.seg[1].b_mn = mn_over_shared(wk_c); dx.seg[1].K = n_qk;
    dx.seg[2].a = dVs; dx.seg[2].b[0] = Wv; dx.seg[2].b_mn = mn_over_shared(wv_c); dx.seg[2].K = n_vo;
    dx.epi = EPI_STORE; dx.C = dX; dx.ldc = ld_dx; dx.out_f32 = cx.dtype == ECOSPA_F32; dx.accumulate = accumulate_dX != 0;
    const ColsumParams cs = colsum_plan(cx, dQs, dbq_c, dKs, dbk_c, dVs, dbv_c);
    if (cx.st != ECOSPA_OK) return cx.st;
    if ((st = launch_grouped_gemm(ops, n_ops, cx.stream)) != ECOSPA_OK) return st;
    finish(cx, red, 3, colsum_begin(cx, cs));
    return cx.st;
}

// Output-projection half of the VO backward: everything that only needs dOut (dCtx feeds the caller's
// attention backward, which produces the dV^c that ecospa_coupled_qkv_bwd / _vo_bwd_v consume).
extern "C" ecospa_status_t ecospa_coupled_vo_bwd_o(const void* Ctxm, int64_t ld_ctx, int64_t T, int64_t d_m,
                                                   const ecospa_mat_t* wo_c, int64_t n, const void* dOut, int64_t ld_dout,
                                                   void* dCtx, int64_t ld_dctx, void* dWo_c, int64_t ld_dwo, void* dbo,
                                                   void* workspace, size_t workspace_bytes, void* stream) {
    if (!wo_c || !Ctxm || !dOut || !dCtx || !dWo_c) return ECOSPA_ERR_INVALID;
    Ctx cx;
    ecospa_status_t st = begin(cx, wo_c->dtype, workspace, workspace_bytes, stream, T, d_m, n);
    if (st != ECOSPA_OK) return st;
    if ((st = check_weight(wo_c, d_m, n, cx.dtype)) != ECOSPA_OK) return st;
    const Stored Cs = as_bf16(cx, Ctxm, T, n, ld_ctx);
    const Stored dOs = as_bf16(cx, dOut, T, d_m, ld_dout);
    const Stored Wo = weight_bf16(cx, wo_c, d_m, n);
    if (cx.st != ECOSPA_OK) return cx.st;
    GemmOp ops[kMaxGemmOps];
    PendingReduce red;
    const int64_t cost = gemm_cost(n, d_m, T) + gemm_cost(T, n, d_m);
    int n_ops = add_wgrad_w(cx, ops, 0, wo_c, dOs, Cs, d_m, n, T, dWo_c, ld_dwo, &red, 1, cost);   // dW_O, stored like W_O
    if (cx.st != ECOSPA_OK) return cx.st;
    GemmOp& dc = ops[n_ops++];                                                        // dCtx = dOut W_O^T
    dc.M = T; dc.N = n; dc.n_kseg = 1;
    dc.seg[0].a = dOs; dc.seg[0].b[0] = Wo; dc.seg[0].b_mn = mn_over_other(wo_c); dc.seg[0].K = d_m;
    dc.epi = EPI_STORE; dc.C = dCtx; dc.ldc = ld_dctx; dc.out_f32 = cx.dtype == ECOSPA_F32;
    const ColsumParams cs = colsum_plan(cx, dOs, dbo);
    if (cx.st != ECOSPA_OK) return cx.st;
    if ((st = launch_grouped_gemm(ops, n_ops, cx.stream)) != ECOSPA_OK) return st;
    finish(cx, &red, 1, colsum_begin(cx, cs));
    return cx.st;
}

// Value-projection half of the VO backward: dW_V^c = X^T dV^c, dX (+)= dV^c W_V^cT, dbv = colsum(dV^c).
extern "C" ecospa_status_t ecospa_coupled_vo_bwd_v(const void* X, int64_t ldx, int64_t T, int64_t d_m,
                                                   const ecospa_mat_t* wv_c, int64_t n, const void* dVc, int64_t ld_dv,
                                                   void* dX, int64_t ld_dx, int32_t accumulate_dX, void* dWv_c,
                                                   int64_t ld_dwv, void* dbv_c, void* workspace, size_t workspace_bytes,
                                                   void* stream) {
    return ecospa_coupled_qk_bwd(X, ldx, T, d_m, wv_c, nullptr, n, dVc, nullptr, ld_dv, dX, ld_dx, accumulate_dX, dWv_c,
                                 nullptr, ld_dwv, dbv_c, nullptr, workspace, workspace_bytes, stream);
}

extern "C" ecospa_status_t ecospa_coupled_ffn_fwd(const void* X, int64_t ldx, int64_t T, int64_t d_m, int32_t act,
                                                  const ecospa_mat_t* w1_c, const ecospa_mat_t* w1b_c,
                                                  const ecospa_mat_t* w2_c, int64_t k, const void* b1_c, const void* b2,
                                                  void* Y, int64_t ld_y, void* H, void* Hb, void* A, int64_t ld_h,
                                                  void* workspace, size_t workspace_bytes, void* stream) {
    if (!w1_c || !w2_c || !Y || !H || !A) return ECOSPA_ERR_INVALID;
    if (act != ECOSPA_ACT_GELU_ERF && act != ECOSPA_ACT_GELU_TANH && act != ECOSPA_ACT_SWIGLU) return ECOSPA_ERR_INVALID;
    const bool sw = act == ECOSPA_ACT_SWIGLU;
    if (sw && (!w1b_c || !Hb)) return ECOSPA_ERR_INVALID;
    Ctx cx;
    ecospa_status_t st = begin(cx, w1_c->dtype, workspace, workspace_bytes, stream, T, d_m, k);
    if (st != ECOSPA_OK) return st;
    if ((st = check_weight(w1_c, d_m, k, cx.dtype)) != ECOSPA_OK) return st;
    if (sw && (st = check_weight(w1b_c, d_m, k, cx.dtype)) != ECOSPA_OK) return st;
    if ((st = check_weight(w2_c, d_m, k, cx.dtype)) != ECOSPA_OK) return st;
    if (ld_h < k || (ld_h * 2) % 16) return ld_h < k ? ECOSPA_ERR_INVALID : ECOSPA_ERR_ALIGNMENT;
    const bool f32 = cx.dtype == ECOSPA_F32;
    const Stored Xs = as_bf16(cx, X, T, d_m, ldx);
    GemmOp up;   // H = X W_1 (+ b_1), A = act(H): activation fused into the W_1 epilogue
    up.M = T; up.N = k; up.n_kseg = 1;
    up.seg[0].a = Xs;
    up.seg[0].b[0] = weight_bf16(cx, w1_c, d_m, k);
    if (sw) up.seg[0].b[1] = weight_bf16(cx, w1b_c, d_m, k);
    up.seg[0].b_mn = mn_over_other(w1_c);
    up.seg[0].K = d_m;
    up.epi = sw ? EPI_SWIGLU : (act == ECOSPA_ACT_GELU_ERF ? EPI_GELU_ERF : EPI_GELU_TANH);
    up.C = H; up.C2 = sw ? Hb : A; up.C3 = sw ? A : nullptr; up.ldc = ld_h;
    up.bias = sw ? nullptr : b1_c; up.bias_f32 = f32;
    GemmOp down;  // Y = A W_2 (+ b_2)
    down.M = T; down.N = d_m; down.n_kseg = 1;
    down.seg[0].a.ptr = A; down.seg[0].a.rows = T; down.seg[0].a.cols = k; down.seg[0].a.ld = ld_h;
    down.seg[0].b[0] = weight_bf16(cx, w2_c, d_m, k);  // stored k x d_m = [K][N], or d_m x k = [N][K]
    down.seg[0].b_mn = mn_over_shared(w2_c);
    down.seg[0].K = k;
    down.epi = EPI_STORE; down.C = Y; down.ldc = ld_y; down.out_f32 = f32;
    down.bias = b2; down.bias_f32 = f32;
    if (cx.st != ECOSPA_OK) return cx.st;
    if ((st = validate_gemm_ops(&up, 1)) != ECOSPA_OK || (st = validate_gemm_ops(&down, 1)) != ECOSPA_OK) return st;
    if ((st = launch_grouped_gemm(&up, 1, cx.stream)) != ECOSPA_OK) return st;
    return launch_grouped_gemm(&down, 1, cx.stream);
}

extern "C" ecospa_status_t ecospa_coupled_ffn_bwd(const void* X, int64_t ldx, int64_t T, int64_t d_m, int32_t act,
                                                  const ecospa_mat_t* w1_c, const ecospa_mat_t* w1b_c,
                                                  const ecospa_mat_t* w2_c, int64_t k, const void* H, const void* Hb,
                                                  const void* A, int64_t ld_h, const void* dY, int64_t ld_dy, void* dX,
                                                  int64_t ld_dx, void* dW1_c, void* dW1b_c, int64_t ld_dw1, void* dW2_c,
                                                  int64_t ld_dw2, void* db1_c, void* db2, void* workspace,
                                                  size_t workspace_bytes, void* stream) {
    if (!w1_c || !w2_c || !H || !A || !dY || !dX || !dW1_c || !dW2_c) return ECOSPA_ERR_INVALID;
    if (act != ECOSPA_ACT_GELU_ERF && act != ECOSPA_ACT_GELU_TANH && act != ECOSPA_ACT_SWIGLU) return ECOSPA_ERR_INVALID;
    const bool sw = act == ECOSPA_ACT_SWIGLU;
    if (sw && (!w1b_c || !Hb || !dW1b_c)) return ECOSPA_ERR_INVALID;
    Ctx cx;
    ecospa_status_t st = begin(cx, w1_c->dtype, workspace, workspace_bytes, stream, T, d_m, k);
    if (st != ECOSPA_OK) return st;
    if ((st = check_weight(w1_c, d_m, k, cx.dtype)) != ECOSPA_OK) return st;
    if (sw && (st = check_weight(w1b_c, d_m, k, cx.dtype)) != ECOSPA_OK) return st;
    if ((st = check_weight(w2_c, d_m, k, cx.dtype)) != ECOSPA_OK) return st;
    if (ld_h < k || (ld_h * 2) % 16) return ld_h < k ? ECOSPA_ERR_INVALID : ECOSPA_ERR_ALIGNMENT;
    const bool f32 = cx.dtype == ECOSPA_F32;
    const Stored Xs = as_bf16(cx, X, T, d_m, ldx);
    const Stored dYs = as_bf16(cx, dY, T, d_m, ld_dy);
    const Stored W1 = weight_bf16(cx, w1_c, d_m, k);
    Stored W1b;
    if (sw) W1b = weight_bf16(cx, w1b_c, d_m, k);
    const Stored W2 = weight_bf16(cx, w2_c, d_m, k);
    const Stored dH = scratch_bf16(cx, T, k);
    Stored dHb;
    if (sw) dHb = scratch_bf16(cx, T, k);
    if (cx.st != ECOSPA_OK) return cx.st;
    Stored As;
    As.ptr = A; As.rows = T; As.cols = k; As.ld = ld_h;

    // Two launches of about equal length.  First: dH = (dY W_2^T) (.) act'(H) (W_2 stored k x d_m = [N][K], the
    // derivative fused into the epilogue) together with dW_2 = A^T dY, which does not need dH.  Both launches are
    // described (and all their scratch is taken from the workspace) before the first one is enqueued.
    const int nw = sw ? 2 : 1;
    GemmOp ops[kMaxGemmOps], ops2[kMaxGemmOps];
    PendingReduce red[3];
    int n_ops = 0;
    n_ops = add_wgrad_w(cx, ops, n_ops, w2_c, dYs, As, d_m, k, T, dW2_c, ld_dw2, &red[0], 1,
                        gemm_cost(k, d_m, T) + nw * gemm_cost(T, k, d_m));                                   // dW_2, stored like W_2
    if (cx.st != ECOSPA_OK) return cx.st;
    GemmOp& da = ops[n_ops++];
    da.M = T; da.N = k; da.n_kseg = 1;
    da.seg[0].a = dYs; da.seg[0].b[0] = W2; da.seg[0].b_mn = mn_over_other(w2_c); da.seg[0].K = d_m;
    da.epi = sw ? EPI_DSWIGLU : (act == ECOSPA_ACT_GELU_ERF ? EPI_DGELU_ERF : EPI_DGELU_TANH);
    da.C = const_cast<void*>(dH.ptr); da.C2 = sw ? const_cast<void*>(dHb.ptr) : nullptr; da.ldc = dH.ld;
    da.H = H; da.Hb = Hb; da.ldh = ld_h;

    // Second: dW_1 = X^T dH (and dW_up = X^T dH_up), dX = dH W_1^T (+ dH_up W_up^T)
    int n_ops2 = 0;
    const int64_t cost = nw * gemm_cost(d_m, k, T) + gemm_cost(T, d_m, nw * k);
    n_ops2 = add_wgrad_w(cx, ops2, n_ops2, w1_c, Xs, dH, d_m, k, T, dW1_c, ld_dw1, &red[1], sw ? 2 : 1, cost);   // dW_1, stored like W_1
    if (sw) n_ops2 = add_wgrad_w(cx, ops2, n_ops2, w1b_c, Xs, dHb, d_m, k, T, dW1b_c, ld_dw1, &red[2], 1, cost); // dW_up
    if (cx.st != ECOSPA_OK) return cx.st;
    GemmOp& dx = ops2[n_ops2++];
    dx = GemmOp();
    dx.M = T; dx.N = d_m; dx.n_kseg = sw ? 2 : 1;
    dx.seg[0].a = dH; dx.seg[0].b[0] = W1; dx.seg[0].b_mn = mn_over_shared(w1_c); dx.seg[0].K = k;
    if (sw) {
        dx.seg[1].a = dHb; dx.seg[1].b[0] = W1b; dx.seg[1].b_mn = mn_over_shared(w1b_c); dx.seg[1].K = k;
    }
    dx.epi = EPI_STORE; dx.C = dX; dx.ldc = ld_dx; dx.out_f32 = f32;
    const ColsumParams cs = colsum_plan(cx, dYs, db2, dH, sw ? nullptr : db1_c);
    if (cx.st != ECOSPA_OK) return cx.st;
    if ((st = validate_gemm_ops(ops, n_ops)) != ECOSPA_OK || (st = validate_gemm_ops(ops2, n_ops2)) != ECOSPA_OK) return st;
    if ((st = launch_grouped_gemm(ops, n_ops, cx.stream)) != ECOSPA_OK) return st;
    if ((st = launch_grouped_gemm(ops2, n_ops2, cx.stream)) != ECOSPA_OK) return st;
    finish(cx, red, 3, colsum_begin(cx, cs));
    return cx.st;
}
