// Attention core on compacted heads (Eq. 2 per head, with the heads of the coupled-matrix reformulation of Sec. 3.1
// restricted to their kept indices): Ctx_h = softmax(scale * Q_h K_h^T) V_h for heads whose Q/K width and V width
// differ from head to head, forward and backward.  sm_100a: TMA tile loads -> shared memory -> tcgen05.mma with the
// score tiles and the output tile in TMEM; the softmax runs in registers, one thread per query row.
//
// Layout: Q^c, K^c (T x n_qk) and V^c, Ctx (T x n_vo) hold head h in columns [off_h, off_h + w_h) with w_h a multiple of
// 16 (the compaction step pads every head's block with zero columns: a zero column of Q^c / K^c adds nothing to
// Q K^T, and a zero column of V^c gives a zero column of Ctx) and off_h a multiple of 8, so that every tile load starts
// on a 16-byte boundary and every contraction is a whole number of 16-deep MMA steps.
//
// Two forward kernels, one CTA per SM.  Output heads up to 32 wide (with Q/K heads up to 64) take the kernel of
// independent key streams further down (attn_fwd_ms_kernel); wider heads take the kernel described here, 320 threads.
// A work item is (sequence b, head h, two neighbouring tiles of 128 query rows); a CTA walks a static list of items
// (for causal attention the long ones first).  The two query tiles are two streams that share the K / V tiles and run
// half a step apart.
//   warp 0      producer: one lane issues the TMA loads of the item's two Q tiles and of every K / V tile (rings of 2
//               stages); a tile is one or two 64-column blocks of 128 rows x 128 bytes, 128-byte swizzle
//   warp 1      owns TMEM (512 columns: a 128-column score tile and an output tile per stream, and the probabilities as
//               packed bf16); one lane issues S = Q K^T (K-major operands from shared memory) and O_tile = P V (P read
//               from TMEM, V as stored = MN-major) for both streams
//   warps 2..5  softmax of stream 0, warps 6..9 of stream 1; thread = query row = TMEM lane, all 128 key columns, so
//               nothing is exchanged between threads.  Per key block: pass 1 reads the score tile for the row maximum,
//               folds the previous output tile (O = O * 2^(m_old - m_new) + O_tile, in registers); pass 2 reads the
//               scores again, p = 2^(s*c - m), packs P to bf16 and writes it to TMEM for the second product.
// Pass 2 is bound by the exponential unit, pass 1 and the waits on the tensor pipe are not: a token (two mbarriers)
// lets only one stream at a time through pass 2, so one stream exponentiates while the other reads maxima, folds and
// waits for its products.  Every mbarrier wait is bounded; on expiry the CTA records a code (11 producer, 12 MMA
// issuer, 13 softmax) in the device status word, lets copies land, frees TMEM and returns.

#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <mutex>

#include "common.cuh"
#include "gemm.cuh"
#include "tc.cuh"

namespace ecospa {

namespace {

using namespace tc;

constexpr int kTile = 128;                  // query rows and key rows per tile
constexpr int kBlockBytes = kTile * 128;    // one 64-column block of a 128-row tile
constexpr int kMaxHeads = 128;
constexpr int kFwdThreads = 64 + 2 * 128;   // producer warp, MMA warp, two streams of four softmax warps
constexpr int kBwdComputeWarps = 16;
constexpr int kBwdThreads = 64 + 4 * 128 + 64;   // producer warp, MMA warp, four sets of four compute warps, two more MMA warps
constexpr int kTmemCols = 512;

struct HeadLayout {
    int32_t qk_off[kMaxHeads], qk_w[kMaxHeads], vo_off[kMaxHeads], vo_w[kMaxHeads];   // per query head: Q^c and Ctx columns, widths
    int32_t k_off[kMaxHeads], v_off[kMaxHeads];   // per query head: first column of its K/V head in K^c and in V^c
    int32_t rep;                                   // query heads per K/V head (1: every head its own)
};

struct AttnFwdParams {
    alignas(64) CUtensorMap map_q, map_k, map_v;
    HeadLayout heads;
    int32_t batch, seq, n_heads, n_qt, causal, n_items;
    float scale_log2e;                      // scale * log2(e): scores are exponentiated in base 2
    uint16_t* ctx;
    int64_t ld_ctx;
    float* lse;                             // [n_heads][T], natural logarithm
    int* status;
    unsigned long long wait_limit_ns;
};

struct Item {
    int b, h, qp, n_a, n_b, n;   // query tiles 2 qp and 2 qp + 1 with n_a and n_b key blocks (0: no such tile), n = the larger
};
__device__ __forceinline__ Item decode_item(int it, int n_qt, int n_heads, int batch, int n_kt, int causal) {
    Item I;
    const int per = n_heads * batch;
    const int n_qp = (n_qt + 1) >> 1;
    I.qp = n_qp - 1 - it / per;             // long (late) query tiles first
    const int rem = it % per;
    I.h = rem / batch;
    I.b = rem % batch;
    const int qa = 2 * I.qp, qb = qa + 1;
    I.n_a = causal ? min(n_kt, qa + 1) : n_kt;
    I.n_b = qb < n_qt ? (causal ? min(n_kt, qb + 1) : n_kt) : 0;
    I.n = max(I.n_a, I.n_b);
    return I;
}

template <int NB>   // 64-column blocks per tile: 1 (every head at most 64 wide) or 2
struct FwdCfg {
    static constexpr int kTileBytes = NB * kBlockBytes;
    static constexpr int QS = NB == 1 ? 2 : 1;                     // buffers of the pair of Q tiles
    static constexpr int kSmem = (2 * QS + 4) * kTileBytes + 1024 + 256;
    static constexpr int kOCols = NB * 64;                          // columns of an output tile
    static constexpr int CH = NB == 1 ? 32 : 16;                    // score columns a thread holds at a time (two such buffers)
    // TMEM columns of stream x: scores, output tile, probabilities (narrow heads: a region of their own, so that the
    // next score tile never waits for the second product; wide heads: over the scores they were made from)
    static __device__ __forceinline__ uint32_t col_s(uint32_t x) { return 128u * x; }
    static __device__ __forceinline__ uint32_t col_o(uint32_t x) { return 256u + kOCols * x; }
    static __device__ __forceinline__ uint32_t col_p(uint32_t x) { return NB == 1 ? 384u + 64u * x : 128u * x; }
};

template <int NB>
__global__ void __launch_bounds__(kFwdThreads, 1) attn_fwd_kernel(const __grid_constant__ AttnFwdParams P) {
    using Cfg = FwdCfg<NB>;
    constexpr int kTileBytes = Cfg::kTileBytes;
    constexpr int QS = Cfg::QS;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw_addr);
    const uint32_t sQ = base, sK = sQ + 2 * QS * kTileBytes, sV = sK + 2 * kTileBytes;
    uint8_t* tail = smem + (2 * QS + 4) * kTileBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(tail + 24 * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 24 * 8 + 8);
    const uint32_t bar0 = smem_u32(bars);
    auto q_full = [&](uint32_t s) { return bar0 + 8u * s; };
    auto q_empty = [&](uint32_t s) { return bar0 + 8u * (2 + s); };
    // K and V tiles have rings of their own: a K stage is free as soon as the score products that read it are done
    // (one step earlier than the V stage), so the load of the next K tile is not held up by the second products
    auto k_full = [&](uint32_t s) { return bar0 + 8u * (4 + s); };
    auto k_empty = [&](uint32_t s) { return bar0 + 8u * (6 + s); };
    auto v_full = [&](uint32_t s) { return bar0 + 8u * (8 + s); };
    auto v_empty = [&](uint32_t s) { return bar0 + 8u * (10 + s); };
    // per stream: score tile complete, probabilities written, output tile complete, pass-2 token
    auto s_full = [&](uint32_t x) { return bar0 + 8u * (12 + x); };
    auto p_full = [&](uint32_t x) { return bar0 + 8u * (14 + x); };
    auto o_full = [&](uint32_t x) { return bar0 + 8u * (16 + x); };
    auto token = [&](uint32_t x) { return bar0 + 8u * (18 + x); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_kt = (P.seq + kTile - 1) / kTile;
    if (threadIdx.x == 0) {
        for (uint32_t s = 0; s < 2; ++s) {
            mbar_init(q_full(s), 1);
            mbar_init(q_empty(s), 1);
            mbar_init(k_full(s), 1);
            mbar_init(k_empty(s), 1);
            mbar_init(v_full(s), 1);
            mbar_init(v_empty(s), 1);
            mbar_init(s_full(s), 1);
            mbar_init(p_full(s), 128);
            mbar_init(o_full(s), 1);
            mbar_init(token(s), 128);
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&P.map_q);
        prefetch_tensormap(&P.map_k);
        prefetch_tensormap(&P.map_v);
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_holder), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t g = 0, qi = 0;
            bool ok = true;
            for (int it = blockIdx.x; ok && it < P.n_items; it += gridDim.x, ++qi) {
                const Item I = decode_item(it, P.n_qt, P.n_heads, P.batch, n_kt, P.causal);
                const int qoff = P.heads.qk_off[I.h], koff = P.heads.k_off[I.h], voff = P.heads.v_off[I.h];
                const int nbq = (P.heads.qk_w[I.h] + 63) >> 6, nbv = (P.heads.vo_w[I.h] + 63) >> 6;
                const int row0 = I.b * P.seq;
                const uint32_t qs = qi % QS;
                if (!(ok = mbar_wait(q_empty(qs), ((qi / QS) & 1u) ^ 1u, abort_flag, 11, P.status, P.wait_limit_ns))) break;
                const int n_tiles = I.n_b > 0 ? 2 : 1;
                mbar_expect_tx(q_full(qs), n_tiles * nbq * kBlockBytes);
                for (int x = 0; x < n_tiles; ++x)
                    for (int blk = 0; blk < nbq; ++blk)
                        tma_load_2d(sQ + (2 * qs + x) * kTileBytes + blk * kBlockBytes, &P.map_q, qoff + 64 * blk,
                                    row0 + (2 * I.qp + x) * kTile, q_full(qs));
                for (int j = 0; j < I.n; ++j, ++g) {
                    const uint32_t st = g & 1;
                    if (!(ok = mbar_wait(k_empty(st), ((g >> 1) & 1u) ^ 1u, abort_flag, 11, P.status, P.wait_limit_ns))) break;
                    mbar_expect_tx(k_full(st), nbq * kBlockBytes);
                    for (int blk = 0; blk < nbq; ++blk)
                        tma_load_2d(sK + st * kTileBytes + blk * kBlockBytes, &P.map_k, koff + 64 * blk, row0 + j * kTile, k_full(st));
                    if (!(ok = mbar_wait(v_empty(st), ((g >> 1) & 1u) ^ 1u, abort_flag, 11, P.status, P.wait_limit_ns))) break;
                    mbar_expect_tx(v_full(st), nbv * kBlockBytes);
                    for (int blk = 0; blk < nbv; ++blk)
                        tma_load_2d(sV + st * kTileBytes + blk * kBlockBytes, &P.map_v, voff + 64 * blk, row0 + j * kTile, v_full(st));
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t g = 0, qi = 0, cp[2] = {0, 0};       // cp[x]: probability tiles of stream x consumed so far
            bool ok = true;
            for (int it = blockIdx.x; ok && it < P.n_items; it += gridDim.x, ++qi) {
                const Item I = decode_item(it, P.n_qt, P.n_heads, P.batch, n_kt, P.causal);
                const int wq = P.heads.qk_w[I.h], wv = P.heads.vo_w[I.h];
                const uint32_t qs = qi % QS;
                if (!(ok = mbar_wait(q_full(qs), (qi / QS) & 1u, abort_flag, 12, P.status, P.wait_limit_ns))) break;
                const uint32_t idesc_s = make_idesc(kTile, kTile, 0, 0);
                const uint32_t idesc_o = make_idesc(kTile, wv, 0, 1);
                // S_x = Q_x K^T with the K tile in ring stage st
                auto scores = [&](uint32_t x, uint32_t st) {
                    for (int ks = 0; ks < (wq >> 4); ++ks) {
                        const uint32_t o = (ks >> 2) * kBlockBytes + (ks & 3) * 32;
                        tc_mma_bf16(tmem_base + Cfg::col_s(x), make_smem_desc(sQ + (2 * qs + x) * kTileBytes + o, 16, 1024),
                                    make_smem_desc(sK + st * kTileBytes + o, 16, 1024), idesc_s, ks != 0 ? 1u : 0u);
                    }
                    tc_commit(s_full(x));
                };
                // O_tile_x = P_x V over the 128 keys of the block in ring stage st
                auto outputs = [&](uint32_t x, uint32_t st) -> bool {
                    if (!mbar_wait(p_full(x), cp[x] & 1u, abort_flag, 12, P.status, P.wait_limit_ns)) return false;
                    ++cp[x];
                    tc_fence_after();
                    for (int ks = 0; ks < kTile / 16; ++ks)
                        tc_mma_bf16_ts(tmem_base + Cfg::col_o(x), tmem_base + Cfg::col_p(x) + 8 * ks,
                                       make_smem_desc(sV + st * kTileBytes + ks * 2048, kBlockBytes, 1024), idesc_o, ks != 0 ? 1u : 0u);
                    tc_commit(o_full(x));
                    return true;
                };
                if (!(ok = mbar_wait(k_full(g & 1), (g >> 1) & 1u, abort_flag, 12, P.status, P.wait_limit_ns))) break;
                tc_fence_after();
                scores(0, g & 1);
                if (I.n_b > 0) scores(1, g & 1);
                tc_commit(k_empty(g & 1));
                for (int j = 0; j < I.n; ++j, ++g) {
                    const uint32_t st = g & 1, nx = (g + 1) & 1;
                    if (!(ok = mbar_wait(v_full(st), (g >> 1) & 1u, abort_flag, 12, P.status, P.wait_limit_ns))) break;
                    if (j + 1 < I.n && !(ok = mbar_wait(k_full(nx), ((g + 1) >> 1) & 1u, abort_flag, 12, P.status, P.wait_limit_ns))) break;
                    tc_fence_after();
                    if (j < I.n_a && !(ok = outputs(0, st))) break;
                    if (j + 1 < I.n_a) scores(0, nx);
                    if (j < I.n_b && !(ok = outputs(1, st))) break;
                    tc_commit(v_empty(st));
                    if (j + 1 < I.n_b) scores(1, nx);
                    if (j + 1 < I.n) tc_commit(k_empty(nx));
                }
                if (ok) tc_commit(q_empty(qs));
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax
        const uint32_t x = static_cast<uint32_t>(warp - 2) >> 2;           // stream
        const int row = (warp & 3) * 32 + lane;
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        const uint32_t tS = t_lane + Cfg::col_s(x), tO = t_lane + Cfg::col_o(x), tP = t_lane + Cfg::col_p(x);
        constexpr int CH = Cfg::CH, NC = kTile / CH;
        constexpr int kOwn = Cfg::kOCols;
        uint32_t cs = 0, turn = 0;                                          // tiles of this stream so far; turns of the token
        bool ok = true;
        const int64_t T = static_cast<int64_t>(P.batch) * P.seq;
        for (int it = blockIdx.x; ok && it < P.n_items; it += gridDim.x) {
            const Item I = decode_item(it, P.n_qt, P.n_heads, P.batch, n_kt, P.causal);
            const int n_own = x == 0 ? I.n_a : I.n_b;
            const int wv = P.heads.vo_w[I.h];
            const int q_pos = (2 * I.qp + static_cast<int>(x)) * kTile + row;   // position of this row in its sequence
            const int limit = P.causal ? min(P.seq, q_pos + 1) : P.seq;     // keys [0, limit) are visible
            float m = -INFINITY, l = 0.f, alpha_prev = 0.f;
            float o[kOwn];
#pragma unroll
            for (int i = 0; i < kOwn; ++i) o[i] = 0.f;
            // O = O * a + O_tile (the output tile of the previous key block)
            auto fold_output = [&](float a) {
                const f32x2 a2 = pack2(a, a);
#pragma unroll
                for (int c = 0; c < kOwn / 16; ++c) {
                    if (c * 16 < wv) {
                        uint32_t r[16];
                        tc_ld16(tO + c * 16, r);
                        tc_wait_ld(r);
#pragma unroll
                        for (int i = 0; i < 16; i += 2)     // (packed fp32: half the issue slots)
                            unpack2(fma2(pack2(o[c * 16 + i], o[c * 16 + i + 1]), a2, pack2(r[i], r[i + 1])), o[c * 16 + i], o[c * 16 + i + 1]);
                    }
                }
            };
            for (int j = 0; j < I.n; ++j, ++turn) {
                const bool active = j < n_own;
                const int kv_base = j * kTile;
                const bool masked = kv_base + kTile > limit;               // keys past the limit count as -inf
                float m_new = m, alpha = 1.f;
                if (active) {
                    if (!(ok = mbar_wait(s_full(x), cs & 1u, abort_flag, 13, P.status, P.wait_limit_ns))) break;
                    tc_fence_after();
                    // pass 1: row maximum (four independent chains); the next chunk is in flight while one is reduced
                    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                    uint32_t ra[CH], rb[CH];
                    tc_ld(tS, ra);
#pragma unroll
                    for (int c = 0; c < NC; ++c) {
                        uint32_t(&cur)[CH] = (c & 1) ? rb : ra;
                        uint32_t(&nxt)[CH] = (c & 1) ? ra : rb;
                        tc_wait_ld(cur);
                        if (c + 1 < NC) tc_ld(tS + (c + 1) * CH, nxt);
                        if (masked) {
#pragma unroll
                            for (int i = 0; i < CH; ++i)
                                if (kv_base + c * CH + i >= limit) cur[i] = 0xff800000u;
                        }
#pragma unroll
                        for (int i = 0; i < CH; i += 2) mx4[(i >> 1) & 3] = max3(mx4[(i >> 1) & 3], __uint_as_float(cur[i]), __uint_as_float(cur[i + 1]));
                    }
                    const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                    m_new = fmaxf(m, mx * P.scale_log2e);
                    alpha = ex2(m - m_new);
                    if (j > 0) {
                        if (!(ok = mbar_wait(o_full(x), (cs - 1) & 1u, abort_flag, 13, P.status, P.wait_limit_ns))) break;
                        tc_fence_after();
                        fold_output(alpha_prev);
                    }
                }
                // the token: stream 0 goes first, then the streams alternate
                if (!(ok = mbar_wait(token(x), x == 0 ? (turn & 1u) ^ 1u : turn & 1u, abort_flag, 13, P.status, P.wait_limit_ns))) break;
                float rs4[4] = {0.f, 0.f, 0.f, 0.f};
                if (active) {
                    // pass 2: p = 2^(s * c - m_new) (2^-inf = 0 for the masked keys), row sum, P as packed bf16 into TMEM
                    uint32_t ra[CH], rb[CH];
                    const f32x2 c2 = pack2(P.scale_log2e, P.scale_log2e), nm2 = pack2(-m_new, -m_new);
                    f32x2 acc2[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
                    tc_ld(tS, ra);
#pragma unroll
                    for (int c = 0; c < NC; ++c) {
                        uint32_t(&cur)[CH] = (c & 1) ? rb : ra;
                        uint32_t(&nxt)[CH] = (c & 1) ? ra : rb;
                        tc_wait_ld(cur);
                        if (c + 1 < NC) tc_ld(tS + (c + 1) * CH, nxt);
                        if (masked) {
#pragma unroll
                            for (int i = 0; i < CH; ++i)
                                if (kv_base + c * CH + i >= limit) cur[i] = 0xff800000u;
                        }
                        uint32_t pk[CH / 2];
#pragma unroll
                        for (int i = 0; i < CH; i += 2) {
                            float x0, x1;
                            unpack2(fma2(pack2(cur[i], cur[i + 1]), c2, nm2), x0, x1);
                            const float p0 = ex2(x0), p1 = ex2(x1);
                            acc2[(i >> 1) & 1] = add2(acc2[(i >> 1) & 1], pack2(p0, p1));
                            pk[i >> 1] = pack_bf16(p0, p1);
                        }
                        tc_st(tP + c * (CH / 2), pk);
                    }
                    unpack2(acc2[0], rs4[0], rs4[1]);
                    unpack2(acc2[1], rs4[2], rs4[3]);
                }
                mbar_arrive(token(x ^ 1u));
                if (active) {
                    tc_wait_st();
                    tc_fence_before();
                    mbar_arrive(p_full(x));
                    l = fmaf(l, alpha, (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]));
                    m = m_new;
                    alpha_prev = alpha;
                    ++cs;
                }
            }
            if (!ok) break;
            if (n_own > 0) {
                if (!(ok = mbar_wait(o_full(x), (cs - 1) & 1u, abort_flag, 13, P.status, P.wait_limit_ns))) break;
                tc_fence_after();
                fold_output(alpha_prev);
                if (q_pos < P.seq) {
                    const int64_t t = static_cast<int64_t>(I.b) * P.seq + q_pos;
                    const float inv = 1.f / l;
                    uint16_t* dst = P.ctx + t * P.ld_ctx + P.heads.vo_off[I.h];
#pragma unroll
                    for (int c = 0; c < kOwn / 8; ++c) {
                        if (c * 8 < wv) {
                            uint4 v;
                            v.x = pack_bf16(o[c * 8 + 0] * inv, o[c * 8 + 1] * inv);
                            v.y = pack_bf16(o[c * 8 + 2] * inv, o[c * 8 + 3] * inv);
                            v.z = pack_bf16(o[c * 8 + 4] * inv, o[c * 8 + 5] * inv);
                            v.w = pack_bf16(o[c * 8 + 6] * inv, o[c * 8 + 7] * inv);
                            *reinterpret_cast<uint4*>(dst + c * 8) = v;
                        }
                    }
                    P.lse[static_cast<int64_t>(I.h) * T + t] = m * 0.6931471805599453f + logf(l);
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    if (*abort_flag) {
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);   // copies still in flight land before the memory is released
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------------
// forward, heads up to 64 wide: NS independent streams per CTA
// ------------------------------------------------------------------------------------------------
// A work item is (sequence b, head h, one tile of 128 query rows).  A K / V tile holds NS slices of 64 keys; stream x
// (four warps, thread = query row) owns slice x of every tile and keeps a softmax of its own over its keys: reference
// exponent m_x, sum l_x, and the output O_x = sum_j P_x(j) V_x(j) accumulating in TMEM.  At the end of the item the NS
// partial results of a row are merged (M = max m_x, weights 2^(m_x - M)).  The streams never wait for one another inside
// an item, so while one waits for its products the others keep the exponential unit busy.
// One pass per score slice: p = 2^(s*c - m) with the reference m the stream already has; m moves only when a score
// exceeds it by more than 32 (2^32 headroom in fp32 / bf16, whose relative precision does not depend on the scale), in
// which case the row's l, O and the probabilities already written for the slice are rescaled first, so no exponent
// can overflow.  The first slice of an item starts from m = -1e30 and takes that path once.
// A stream has two score buffers: S_x of slice G + 1 is computed while the stream exponentiates slice G, so a stream goes
// from one slice to the next without waiting for the tensor pipe.  The probabilities of a slice overwrite the first half
// of the score buffer they were made from (chunk c of 32 scores becomes 16 packed columns at 16 c, inside columns
// that are already in registers).  TMEM columns of stream x: score buffers at 128 x and 128 x + 64, output 128 NS + OC x.
template <int NS, int OC>
struct MsCfg {
    // per stream: one warp that loads the stream's K / V slices and issues its products, and four softmax warps
    static constexpr int kThreads = 32 * NS + 128 * NS;
    static constexpr int kSlice = 64;
    static constexpr int kKeys = NS * kSlice;                 // keys per K / V tile
    static constexpr int kSliceBytes = kSlice * 128;          // one slice: 64 rows x 128 bytes
    static constexpr int kStages = 3;                         // K and V slices per stream: slice s uses stage s % 3
    static constexpr int kRingBytes = NS * 2 * kStages * kSliceBytes;
    static constexpr int kMergeBytes = 2 * NS * kTile * 4;    // m and l of every stream and row
    static constexpr int kSmem = 2 * kBlockBytes + kRingBytes + kMergeBytes + 1024 + 512;
    static __device__ __forceinline__ uint32_t col_s(uint32_t x, uint32_t buf) { return 128u * x + 64u * buf; }
    static __device__ __forceinline__ uint32_t col_o(uint32_t x) { return 128u * NS + OC * x; }
    static_assert(128 * NS + OC * NS <= kTmemCols, "TMEM columns");
};

struct MsItem {
    int b, h, qt, lim;          // lim: last key position any row of the tile sees
};
__device__ __forceinline__ MsItem ms_decode(int it, int n_qt, int n_heads, int batch, int seq, int causal) {
    MsItem I;
    const int per = n_heads * batch;
    I.qt = n_qt - 1 - it / per;             // long (late) query tiles first
    const int rem = it % per;
    I.h = rem / batch;
    I.b = rem % batch;
    I.lim = causal ? min(I.qt * kTile + kTile - 1, seq - 1) : seq - 1;
    return I;
}
// K / V tiles in which slice x has a visible key
__device__ __forceinline__ int ms_steps(int lim, int x, int keys_per_tile) {
    const int first = 64 * x;
    return lim >= first ? (lim - first) / keys_per_tile + 1 : 0;
}

struct RowState {
    float m, l, rs;
};
// The rare path of a slice: a score exceeds the row's reference exponent by more than 32.  Moves the reference to that
// score and rescales what was computed with the old one: the sums, the output row in TMEM (o_groups 16-column groups; 0
// while the stream has no output yet) and the probability chunks of this slice written so far.  Called by whole warps.
__device__ __forceinline__ RowState rescale_row(RowState s, float cm, uint32_t tO, int o_groups, uint32_t tP, int chunks_done) {
    const bool need = cm - s.m > 32.f;
    const float m_new = need ? cm : s.m;
    const float f = need ? ex2(s.m - m_new) : 1.f;
    tc_wait_st();                            // the chunks written so far are read back below
    for (int g = 0; g < o_groups; ++g) {
        uint32_t r[16];
        tc_ld16(tO + 16 * g, r);
        tc_wait_ld(r);
#pragma unroll
        for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
        tc_st(tO + 16 * g, r);
    }
    for (int c = 0; c < chunks_done; ++c) {
        uint32_t r[16];
        tc_ld16(tP + 16 * c, r);
        tc_wait_ld(r);
#pragma unroll
        for (int i = 0; i < 16; ++i) r[i] = pack_bf16(bf16_lo(r[i]) * f, bf16_hi(r[i]) * f);
        tc_st(tP + 16 * c, r);
    }
    tc_wait_st();
    RowState o;
    o.m = m_new;
    o.l = s.l * f;
    o.rs = s.rs * f;
    return o;
}

template <int NS, int OC>
__global__ void __launch_bounds__(MsCfg<NS, OC>::kThreads, 1) attn_fwd_ms_kernel(const __grid_constant__ AttnFwdParams P) {
    using Cfg = MsCfg<NS, OC>;
    constexpr int kSliceB = Cfg::kSliceBytes, kKeys = Cfg::kKeys, ST = Cfg::kStages;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw_addr);
    const uint32_t sQ = base, sK = sQ + 2 * kBlockBytes, sV = sK + NS * ST * kSliceB;   // K / V: [stream][stage] slices
    float* merge = reinterpret_cast<float*>(smem + 2 * kBlockBytes + Cfg::kRingBytes);   // [m | l][stream][row]
    uint8_t* tail = smem + 2 * kBlockBytes + Cfg::kRingBytes + Cfg::kMergeBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(tail + 60 * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 60 * 8 + 8);
    const uint32_t bar0 = smem_u32(bars);
    auto q_full = [&](uint32_t s) { return bar0 + 8u * s; };
    auto q_empty = [&](uint32_t s) { return bar0 + 8u * (2 + s); };     // one arrival per stream and item
    // Per stream and score buffer (slice G uses buffer G & 1): probabilities written; the product that read them done.
    // Two barriers each, because a stream runs ahead of its issuer by one slice: with one barrier the phases of slices
    // G and G + 1 could both complete before the waiter has looked at the first.
    auto p_full = [&](uint32_t x, uint32_t buf) { return bar0 + 8u * (4 + 2 * x + buf); };
    auto pv_done = [&](uint32_t x, uint32_t buf) { return bar0 + 8u * (42 + 2 * x + buf); };
    auto s_full = [&](uint32_t x, uint32_t buf) { return bar0 + 8u * (12 + 2 * x + buf); };   // scores in buffer buf of stream x
    auto kv_full = [&](uint32_t x, uint32_t b) { return bar0 + 8u * (20 + 2 * x + b); };      // the loads event G needs (b = G & 1) landed
    const uint32_t merge_a = bar0 + 8u * 40, merge_b = bar0 + 8u * 41;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (uint32_t s = 0; s < 2; ++s) {
            mbar_init(q_full(s), 1);
            mbar_init(q_empty(s), NS);
            for (uint32_t x = 0; x < NS; ++x) {
                mbar_init(kv_full(x, s), 1);
                mbar_init(s_full(x, s), 1);
                mbar_init(p_full(x, s), 128);
                mbar_init(pv_done(x, s), 1);
            }
        }
        mbar_init(merge_a, 128 * NS);
        mbar_init(merge_b, 128 * NS);
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&P.map_q);
        prefetch_tensormap(&P.map_k);
        prefetch_tensormap(&P.map_v);
    }
    if (warp == 0) tmem_alloc(smem_u32(tmem_holder), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    if (warp < NS) {
        // ------------------------------------------------------------------ loader and MMA issuer of stream x
        // The stream's slices form one sequence G = 0, 1, ... across the CTA's items (items in which the stream has no
        // visible key are skipped).  Event G: the probabilities of slice G are written -> O_x += P_x V_x (slice G), then
        // S_x of slice G + 2 into the score buffer that slice G occupied, then the loads of the K slice G + 3 and of the V
        // slice G + 1.  Their stages (slice s uses stage s % 3) are free: S(G) was read by the softmax, and P V(G - 2) was
        // issued before S(G), whose completion signal covers it.  Both loads report to the barrier event G + 1 waits on.
        // This thread shares its scheduler with the stream's softmax warps, so the loop is kept short: slices are
        // described by three packed registers produced once (next()) and handed from stage to stage.
        if (lane == 0) {
            const uint32_t x = warp;
            const uint32_t tS = tmem_base + Cfg::col_s(x, 0), tO = tmem_base + Cfg::col_o(x);
            const uint32_t idesc_s = make_idesc(kTile, 64, 0, 0);
            const uint32_t sKx = sK + x * ST * kSliceB, sVx = sV + x * ST * kSliceB;
            const uint64_t dq0 = make_smem_desc(sQ, 16, 1024), dk0 = make_smem_desc(sKx, 16, 1024),
                           dv0 = make_smem_desc(sVx, kBlockBytes, 1024);
            // meta bits: 0 valid, 1 first slice of its item, 2 last, 3 Q buffer, 4 phase of that buffer, 5-7 contraction
            // steps of the scores, 8-11 output width / 16, 12-.. items skipped just before (first slices and the end mark)
            struct SD {
                int row;            // first key row of the slice in the K / V tensors
                int qrow;           // first row of the item's query tile
                uint32_t qcol;      // first column of the head in Q^c
                uint32_t cols;      // first column of the head's K/V head in K^c | in V^c << 16
                uint32_t meta;
            };
            // generator of the stream's slice sequence
            int g_it = static_cast<int>(blockIdx.x) - static_cast<int>(gridDim.x), g_J = 0, g_n = 0, g_row = 0, g_qrow = 0;
            uint32_t g_cols = 0, g_qcol = 0, g_meta = 0, g_qi = ~0u, g_skip = 0;
            auto next = [&]() {
                SD d;
                if (g_J >= g_n) {
                    for (;;) {
                        g_it += gridDim.x;
                        ++g_qi;
                        if (g_it >= P.n_items) {   // end mark; it carries the Q buffers still to hand back
                            d.row = 0;
                            d.cols = 0;
                            d.qcol = 0;
                            d.meta = ((g_qi & 1u) << 3) | (g_skip << 12);
                            g_skip = 0;
                            g_it -= gridDim.x;      // stay at the end: later calls give the mark again, with no count
                            --g_qi;
                            g_J = g_n = 0;
                            d.qrow = 0;
                            return d;
                        }
                        const MsItem I = ms_decode(g_it, P.n_qt, P.n_heads, P.batch, P.seq, P.causal);
                        g_n = ms_steps(I.lim, x, kKeys);
                        if (g_n == 0) {
                            ++g_skip;
                            continue;
                        }
                        g_J = 0;
                        g_row = I.b * P.seq + 64 * static_cast<int>(x);
                        g_qrow = I.b * P.seq + I.qt * kTile;
                        g_cols = static_cast<uint32_t>(P.heads.k_off[I.h]) | (static_cast<uint32_t>(P.heads.v_off[I.h]) << 16);
                        g_qcol = static_cast<uint32_t>(P.heads.qk_off[I.h]);
                        g_meta = 1u | ((g_qi & 1u) << 3) | (((g_qi >> 1) & 1u) << 4) | (static_cast<uint32_t>(P.heads.qk_w[I.h] >> 4) << 5) |
                                 (static_cast<uint32_t>(P.heads.vo_w[I.h] >> 4) << 8);
                        break;
                    }
                }
                d.row = g_row + g_J * kKeys;
                d.qrow = g_qrow;
                d.qcol = g_qcol;
                d.cols = g_cols;
                d.meta = g_meta | (g_J == 0 ? 2u | (g_skip << 12) : 0u) | (g_J == g_n - 1 ? 4u : 0u);
                if (g_J == 0) g_skip = 0;
                ++g_J;
                return d;
            };
            bool ok = true;
            // K slice of d into stage st (stream 0: with the Q tile of the item when d is its first slice)
            auto load_k = [&](const SD& d, uint32_t st, uint32_t bar) -> bool {
                if (x == 0 && (d.meta & 2u)) {
                    const uint32_t qs = (d.meta >> 3) & 1u, ph = (d.meta >> 4) & 1u;
                    if (!mbar_wait(q_empty(qs), ph ^ 1u, abort_flag, 11, P.status, P.wait_limit_ns)) return false;
                    mbar_expect_tx(q_full(qs), kBlockBytes);
                    tma_load_2d(sQ + qs * kBlockBytes, &P.map_q, d.qcol, d.qrow, q_full(qs));
                }
                tma_load_2d(sKx + st * kSliceB, &P.map_k, d.cols & 0xffffu, d.row, bar);
                return true;
            };
            auto load_v = [&](const SD& d, uint32_t st, uint32_t bar) {
                tma_load_2d(sVx + st * kSliceB, &P.map_v, d.cols >> 16, d.row, bar);
            };
            auto hand_back = [&](uint32_t qs_of_item, uint32_t n) {   // Q buffers of the n items before the one whose buffer is given
                for (uint32_t k = 1; k <= n; ++k) tc_commit(q_empty((qs_of_item + k) & 1u));
            };
            // S_x of slice d (its K slice in stage st) into score buffer buf
            auto scores = [&](SD& d, uint32_t st, uint32_t buf) -> bool {
                const uint32_t qs = (d.meta >> 3) & 1u;
                if (!(d.meta & 1u)) {               // the end mark: only the hand-backs, once
                    hand_back(qs, d.meta >> 12);
                    d.meta &= 0xfffu;
                    return true;
                }
                if (d.meta & 2u) {
                    hand_back(qs, d.meta >> 12);
                    if (!mbar_wait(q_full(qs), (d.meta >> 4) & 1u, abort_flag, 12, P.status, P.wait_limit_ns)) return false;
                    tc_fence_after();
                }
                const uint64_t dq = dq0 + qs * (kBlockBytes >> 4), dk = dk0 + st * (kSliceB >> 4);
                const uint32_t ksteps = (d.meta >> 5) & 7u, t = tS + 64 * buf;
                tc_mma_bf16(t, dq, dk, idesc_s, 0u);
                if (ksteps > 1) tc_mma_bf16(t, dq + 2, dk + 2, idesc_s, 1u);
                if (ksteps > 2) tc_mma_bf16(t, dq + 4, dk + 4, idesc_s, 1u);
                if (ksteps > 3) tc_mma_bf16(t, dq + 6, dk + 6, idesc_s, 1u);
                tc_commit(s_full(x, buf));
                if (d.meta & 4u) tc_commit(q_empty(qs));
                return true;
            };
            SD d0 = next(), d1 = next(), d2 = next(), d3;
            {   // start: K slices 0..2 and V slice 0 on the barrier event 0 waits on
                const uint32_t nk = (d0.meta & 1u) + (d1.meta & 1u) + (d2.meta & 1u);
                if (nk) mbar_expect_tx(kv_full(x, 0), (nk + 1) * kSliceB);
                if (d0.meta & 1u) {
                    ok = load_k(d0, 0, kv_full(x, 0));
                    load_v(d0, 0, kv_full(x, 0));
                }
                if (ok && (d1.meta & 1u)) ok = load_k(d1, 1, kv_full(x, 0));
                if (ok && (d2.meta & 1u)) ok = load_k(d2, 2, kv_full(x, 0));
                if (ok && nk) ok = mbar_wait(kv_full(x, 0), 0u, abort_flag, 12, P.status, P.wait_limit_ns);
                tc_fence_after();
                ok = ok && scores(d0, 0, 0) && scores(d1, 1, 1);
            }
            uint32_t G = 0, st0 = 0;                // st0 = G % 3
            while (ok && (d0.meta & 1u)) {
                const uint32_t buf = G & 1u, ph = (G >> 1) & 1u;
                const uint32_t st1 = st0 == 2 ? 0 : st0 + 1, st2 = st1 == 2 ? 0 : st1 + 1;
                if (!(ok = mbar_wait(p_full(x, buf), ph, abort_flag, 12, P.status, P.wait_limit_ns))) break;
                if (G > 0 && !(ok = mbar_wait(kv_full(x, buf), ph, abort_flag, 12, P.status, P.wait_limit_ns))) break;
                tc_fence_after();
                {   // O_x += P_x V_x over the slice's 64 keys
                    const uint32_t idesc_o = make_idesc(kTile, ((d0.meta >> 8) & 15u) << 4, 0, 1);
                    const uint64_t dv = dv0 + st0 * (kSliceB >> 4);
                    const uint32_t tP = tS + 64 * buf;
                    tc_mma_bf16_ts(tO, tP, dv, idesc_o, (d0.meta & 2u) ? 0u : 1u);
                    tc_mma_bf16_ts(tO, tP + 8, dv + 128, idesc_o, 1u);
                    tc_mma_bf16_ts(tO, tP + 16, dv + 256, idesc_o, 1u);
                    tc_mma_bf16_ts(tO, tP + 24, dv + 384, idesc_o, 1u);
                    tc_commit(pv_done(x, buf));
                }
                if (!(ok = scores(d2, st2, buf))) break;      // slice G + 2
                d3 = next();                                   // slice G + 3
                {
                    const uint32_t nb = (d3.meta & 1u) + (d1.meta & 1u), bar = kv_full(x, buf ^ 1u);
                    if (nb) mbar_expect_tx(bar, nb * kSliceB);
                    if ((d3.meta & 1u) && !(ok = load_k(d3, st0, bar))) break;
                    if (d1.meta & 1u) load_v(d1, st1, bar);
                }
                d0 = d1;
                d1 = d2;
                d2 = d3;
                st0 = st1;
                ++G;
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax streams
        const uint32_t x = static_cast<uint32_t>(warp - NS) >> 2;
        const int row = (warp & 3) * 32 + lane;
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        const uint32_t tS0 = t_lane + Cfg::col_s(x, 0), tO = t_lane + Cfg::col_o(x);
        constexpr int CH = 32, NC = 64 / CH;
        uint32_t cs = 0, mi = 0;             // slices of this stream so far, items
        bool ok = true, pending_b = false;
        const int64_t T = static_cast<int64_t>(P.batch) * P.seq;
        for (int it = blockIdx.x; ok && it < P.n_items; it += gridDim.x, ++mi) {
            const MsItem I = ms_decode(it, P.n_qt, P.n_heads, P.batch, P.seq, P.causal);
            const int n_own = ms_steps(I.lim, x, kKeys);
            const int wv = P.heads.vo_w[I.h];
            const int q_pos = I.qt * kTile + row;
            const int limit = P.causal ? min(P.seq, q_pos + 1) : P.seq;     // keys [0, limit) are visible
            RowState rsx;
            rsx.m = -1e30f;
            rsx.l = 0.f;
            for (int j = 0; j < n_own; ++j) {
                if (!(ok = mbar_wait(s_full(x, cs & 1), (cs >> 1) & 1u, abort_flag, 13, P.status, P.wait_limit_ns))) break;
                tc_fence_after();
                const uint32_t tS = tS0 + 64 * (cs & 1), tP = tS;    // the probabilities go over the scores they came from
                const int kv_base = j * kKeys + 64 * static_cast<int>(x);
                const bool masked = kv_base + 64 > limit;                   // keys past the limit count as -inf
                float rs4[4] = {0.f, 0.f, 0.f, 0.f};
                uint32_t ra[CH], rb[CH];
                tc_ld(tS, ra);
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    uint32_t(&cur)[CH] = (c & 1) ? rb : ra;
                    uint32_t(&nxt)[CH] = (c & 1) ? ra : rb;
                    tc_wait_ld(cur);
                    if (c + 1 < NC) tc_ld(tS + (c + 1) * CH, nxt);
                    if (masked) {
#pragma unroll
                        for (int i = 0; i < CH; ++i)
                            if (kv_base + c * CH + i >= limit) cur[i] = 0xff800000u;
                    }
                    // The chunk's maximum and its exponentials (with the reference the row has) have no dependence on one
                    // another, so they can be interleaved; only if some score exceeds the reference by more than 32 (rare) is
                    // the row rescaled and the chunk exponentiated again.
                    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int i = 0; i < CH; i += 2) mx4[(i >> 1) & 3] = max3(mx4[(i >> 1) & 3], __uint_as_float(cur[i]), __uint_as_float(cur[i + 1]));
                    const float cm = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * P.scale_log2e;
                    uint32_t pk[CH / 2];
                    float cs4[4] = {0.f, 0.f, 0.f, 0.f};
                    auto exponentiate = [&](float neg_m) {   // (packed fp32 multiply-adds and sums: half the issue slots)
                        const f32x2 c2 = pack2(P.scale_log2e, P.scale_log2e), nm2 = pack2(neg_m, neg_m);
                        f32x2 acc2[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
#pragma unroll
                        for (int i = 0; i < CH; i += 2) {
                            float x0, x1;
                            unpack2(fma2(pack2(cur[i], cur[i + 1]), c2, nm2), x0, x1);
                            const float p0 = ex2(x0), p1 = ex2(x1);
                            acc2[(i >> 1) & 1] = add2(acc2[(i >> 1) & 1], pack2(p0, p1));
                            pk[i >> 1] = pack_bf16(p0, p1);
                        }
                        unpack2(acc2[0], cs4[0], cs4[1]);
                        unpack2(acc2[1], cs4[2], cs4[3]);
                    };
                    exponentiate(-rsx.m);
                    if (__any_sync(0xffffffffu, cm - rsx.m > 32.f)) {
                        // the output row is touched: the product of the previous slice must have landed
                        if (j > 0 && !(ok = mbar_wait(pv_done(x, (cs - 1) & 1), ((cs - 1) >> 1) & 1u, abort_flag, 13, P.status, P.wait_limit_ns))) break;
                        tc_fence_after();
                        rsx.rs = (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]);
                        rsx = rescale_row(rsx, cm, tO, j > 0 ? wv >> 4 : 0, tP, c);
                        rs4[0] = rsx.rs;
                        rs4[1] = rs4[2] = rs4[3] = 0.f;
                        exponentiate(-rsx.m);
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) rs4[q] += cs4[q];
                    tc_st(tP + c * (CH / 2), pk);
                }
                if (!ok) break;
                tc_wait_st();
                tc_fence_before();
                if (pending_b) {   // the output regions of the previous item have been read by every stream
                    if (!(ok = mbar_wait(merge_b, (mi - 1) & 1u, abort_flag, 13, P.status, P.wait_limit_ns))) break;
                    pending_b = false;
                }
                mbar_arrive(p_full(x, cs & 1));
                rsx.l += (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]);
                ++cs;
            }
            if (!ok) break;
            if (n_own > 0) {   // the stream's last product of the item
                if (!(ok = mbar_wait(pv_done(x, (cs - 1) & 1), ((cs - 1) >> 1) & 1u, abort_flag, 13, P.status, P.wait_limit_ns))) break;
                tc_fence_after();
            }
            if (pending_b) {       // (a stream without slices in this item)
                if (!(ok = mbar_wait(merge_b, (mi - 1) & 1u, abort_flag, 13, P.status, P.wait_limit_ns))) break;
                pending_b = false;
            }
            // merge of the row's NS partial results
            merge[x * kTile + row] = rsx.m;
            merge[(NS + x) * kTile + row] = rsx.l;
            mbar_arrive(merge_a);
            if (!(ok = mbar_wait(merge_a, mi & 1u, abort_flag, 13, P.status, P.wait_limit_ns))) break;
            float gk[NS], M = -INFINITY, L = 0.f;
#pragma unroll
            for (int k = 0; k < NS; ++k)
                if (ms_steps(I.lim, k, kKeys) > 0) M = fmaxf(M, merge[k * kTile + row]);
#pragma unroll
            for (int k = 0; k < NS; ++k) {
                gk[k] = 0.f;
                if (ms_steps(I.lim, k, kKeys) > 0) {
                    gk[k] = ex2(merge[k * kTile + row] - M);
                    L = fmaf(merge[(NS + k) * kTile + row], gk[k], L);
                }
            }
            const float inv = 1.f / L;
            const bool live = q_pos < P.seq;
            const int64_t t = static_cast<int64_t>(I.b) * P.seq + q_pos;
            for (int grp = x; grp < (wv >> 4); grp += NS) {   // this stream's share of the output columns
                float acc[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[i] = 0.f;
#pragma unroll
                for (int k = 0; k < NS; ++k) {
                    if (ms_steps(I.lim, k, kKeys) > 0) {
                        uint32_t r[16];
                        tc_ld16(t_lane + Cfg::col_o(k) + 16 * grp, r);
                        tc_wait_ld(r);
#pragma unroll
                        for (int i = 0; i < 16; ++i) acc[i] = fmaf(__uint_as_float(r[i]), gk[k], acc[i]);
                    }
                }
                if (live) {
                    uint16_t* dst = P.ctx + t * P.ld_ctx + P.heads.vo_off[I.h] + 16 * grp;
                    uint4 v0, v1;
                    v0.x = pack_bf16(acc[0] * inv, acc[1] * inv);
                    v0.y = pack_bf16(acc[2] * inv, acc[3] * inv);
                    v0.z = pack_bf16(acc[4] * inv, acc[5] * inv);
                    v0.w = pack_bf16(acc[6] * inv, acc[7] * inv);
                    v1.x = pack_bf16(acc[8] * inv, acc[9] * inv);
                    v1.y = pack_bf16(acc[10] * inv, acc[11] * inv);
                    v1.z = pack_bf16(acc[12] * inv, acc[13] * inv);
                    v1.w = pack_bf16(acc[14] * inv, acc[15] * inv);
                    *reinterpret_cast<uint4*>(dst) = v0;
                    *reinterpret_cast<uint4*>(dst + 8) = v1;
                }
            }
            if (x == 0 && live) P.lse[static_cast<int64_t>(I.h) * T + t] = M * 0.6931471805599453f + logf(L);
            tc_fence_before();
            mbar_arrive(merge_b);
            pending_b = true;
        }
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    if (*abort_flag) {
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);   // copies still in flight land before the memory is released
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------------
// backward
// ------------------------------------------------------------------------------------------------
// Reverse mode of Ctx_h = P V_h, P = softmax(scale * Q_h K_h^T), with P recomputed from the saved log-sum-exp:
//     dV = P^T dCtx,  dP = dCtx V^T,  dS = P (.) (dP - D),  D_t = sum_c dCtx[t, c] Ctx[t, c],
//     dQ = scale * dS K,  dK = scale * dS^T Q.
// Three launches: the row dots D with the log-sum-exp in the form the other two use (memory-bound), then one launch that
// owns key blocks (dK and dV accumulate in TMEM over the query blocks) and one that owns query blocks (dQ accumulates
// over the key blocks).  Nothing is added across CTAs, so the results do not depend on timing.

// D[h][t] for every head: a warp takes a row, every lane multiplies 16-byte vectors (8 columns, which never straddle a
// head because offsets and widths are multiples of 8), and the per-vector partial sums are added per head in order.
constexpr int kDotWarps = 4;
constexpr int kDotMaxVecs = 2048;      // 16384 columns
struct DotParams {
    HeadLayout heads;
    const uint16_t* ctx;
    const uint16_t* dctx;
    const float* lse;                  // [n_heads][T], natural logarithm (from the forward call)
    float* vecs;                       // [2][n_heads][batch][seq_pad]: -lse * log2(e), then the row dots D; zero past seq
    int64_t ld_ctx, ld_dctx, T;
    int32_t n_heads, n_vecs, batch, seq, seq_pad;
};
// One warp per position of the padded sequences: the per-head row dots D_t = sum_c dCtx[t, c] Ctx[t, c] and the
// log-sum-exp in the form the backward kernels use, in a layout whose 128-position blocks are whole, 512-byte aligned
// runs (so that a block's vectors can be copied to shared memory in bulk).
__global__ void __launch_bounds__(32 * kDotWarps) attn_rowdot_kernel(const __grid_constant__ DotParams P) {
    __shared__ float part[kDotWarps][kDotMaxVecs];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t tp = static_cast<int64_t>(blockIdx.x) * kDotWarps + warp;      // position in the padded layout
    if (tp >= static_cast<int64_t>(P.batch) * P.seq_pad) return;
    const int b = static_cast<int>(tp / P.seq_pad), pos = static_cast<int>(tp % P.seq_pad);
    const int64_t per_arr = static_cast<int64_t>(P.n_heads) * P.batch * P.seq_pad;
    if (pos >= P.seq) {
        for (int h = lane; h < P.n_heads; h += 32) {
            const int64_t o = (static_cast<int64_t>(h) * P.batch + b) * P.seq_pad + pos;
            P.vecs[o] = 0.f;
            P.vecs[per_arr + o] = 0.f;
        }
        return;
    }
    const int64_t t = static_cast<int64_t>(b) * P.seq + pos;
    const uint16_t* a = P.ctx + t * P.ld_ctx;
    const uint16_t* bb = P.dctx + t * P.ld_dctx;
    for (int v = lane; v < P.n_vecs; v += 32) {
        const uint4 x = *reinterpret_cast<const uint4*>(a + 8 * v);
        const uint4 y = *reinterpret_cast<const uint4*>(bb + 8 * v);
        float s = bf16_lo(x.x) * bf16_lo(y.x);
        s = fmaf(bf16_hi(x.x), bf16_hi(y.x), s);
        s = fmaf(bf16_lo(x.y), bf16_lo(y.y), s);
        s = fmaf(bf16_hi(x.y), bf16_hi(y.y), s);
        s = fmaf(bf16_lo(x.z), bf16_lo(y.z), s);
        s = fmaf(bf16_hi(x.z), bf16_hi(y.z), s);
        s = fmaf(bf16_lo(x.w), bf16_lo(y.w), s);
        s = fmaf(bf16_hi(x.w), bf16_hi(y.w), s);
        part[warp][v] = s;
    }
    __syncwarp();
    for (int h = lane; h < P.n_heads; h += 32) {
        const int v0 = P.heads.vo_off[h] >> 3, nv = P.heads.vo_w[h] >> 3;
        float s = 0.f;
        for (int i = 0; i < nv; ++i) s += part[warp][v0 + i];
        const int64_t o = (static_cast<int64_t>(h) * P.batch + b) * P.seq_pad + pos;
        P.vecs[o] = -P.lse[static_cast<int64_t>(h) * P.T + t] * 1.4426950408889634f;
        P.vecs[per_arr + o] = s;
    }
}

struct AttnBwdParams {
    alignas(64) CUtensorMap map_q, map_k, map_v, map_do;
    HeadLayout heads;
    int32_t batch, seq, n_heads, n_t, causal, n_items;
    float scale_log2e, scale;
    const float* lse;                  // [n_heads][T], natural logarithm
    const float* vecs;                 // [2][n_heads][batch][seq_pad]: -lse * log2(e) and the row dots D (attn_rowdot_kernel)
    int32_t seq_pad;
    uint16_t* dq;
    uint16_t* dk;
    uint16_t* dv;
    int64_t ld_dqk, ld_dv;
    int* status;
    unsigned long long wait_limit_ns;
};

// MODE 0: a CTA owns a key block of a (sequence, K/V head) and walks the query blocks of the query heads that read it:
//         K, V resident, Q_i and dCtx_i streamed (with the step's queries' -lse*log2e and D, bulk-copied on the same
//         barrier); X = S^T = K Q_i^T and Y = dP^T = V dCtx_i^T (thread = key row, columns = queries); P^T and dS^T are
//         the A operands of dV += P^T dCtx_i and dK += dS^T Q_i, which accumulate in TMEM.
// MODE 1: a CTA owns a query block and walks the key blocks: Q, dCtx resident, K_j and V_j streamed; X = S = Q K_j^T and
//         Y = dP = dCtx V_j^T (thread = query row); dS is the A operand of dQ += dS K_j, which accumulates in TMEM.
// Streamed tiles serve twice: as K-major B operands of the score products and as MN-major B operands of the
// accumulating ones (same bytes, other descriptor).  Warp 0 loads, warps 2..17 compute (thread = row, quarter of the
// columns), and three threads issue products: a thread gets a tcgen05 instruction (product or commit) accepted every
// 70-130 clocks, so the 25-40 of a step are spread evenly over them, and the score products of a step are issued as soon
// as every compute thread has the previous score tiles in registers.
// Heads up to 64 wide (NB = 1): warp 1 issues the score products; warps 18 and 19 the accumulating ones: dV and dK in the
// key-block kernel, the two halves of the contraction of dQ (into two accumulators that are added at the end) in the
// query-block kernel; their A operands go through TMEM as packed bf16; three stages of streamed tiles.
// Wider heads (NB = 2): warp 1 issues X, warp 18 Y, warp 19 the accumulating products, whose A operands go through shared
// memory; the key-block kernel takes the queries 64 at a time (three stages of half-size tiles, two buffers of score
// tiles and of operands), the query-block kernel has two stages.
// Wait codes: 14 / 15 / 16 (MODE 0 loads, products, compute) and 17 / 18 / 19 (MODE 1).
template <int NB, int MODE>
struct BwdCfg {
    static constexpr int kTileBytes = NB * kBlockBytes;
    // rows of a streamed block.  The key-block kernel on wide heads walks the queries in half blocks: its two wide
    // accumulators fill the tensor memory beside the score tiles, so P^T and dS^T go through shared memory, and only with
    // half-size streamed tiles and operands is there room for more than one stage
    static constexpr int kStep = (NB == 2 && MODE == 0) ? 64 : kTile;
    static constexpr int kStrBlockBytes = kStep * 128;                         // 64 columns of a streamed block
    static constexpr int kStrTileBytes = NB * kStrBlockBytes;
    static constexpr int kResStages = NB == 1 ? 2 : 1;                         // buffers of the resident pair of tiles
    // stages of the streamed pair of tiles.  Three where they fit (a fourth changes nothing): a stage is free again only when the accumulating
    // products that read it are done, a whole step after the score products, and the next load must be under way by then
    static constexpr int kStrStages = (NB == 1 || MODE == 0) ? 3 : 2;
    static constexpr int kOutTileBytes = (kStep / 64) * kBlockBytes;            // 128 rows x kStep columns of bf16
    static constexpr int kOutTiles = NB == 1 ? 0 : (MODE == 0 ? 2 : 1);        // P^T and dS^T, or dS (narrow heads: in TMEM)
    static constexpr int kOutBufs = kStep == 64 ? 2 : 1;                       // half-block steps: room for two sets of them
    static constexpr int kVecBytes = MODE == 0 ? kStrStages * 2 * kStep * 4 : 0;   // -lse2 and D of a query block, per streamed stage
    static constexpr int kSmem = 2 * kTileBytes * kResStages + 2 * kStrTileBytes * kStrStages + kOutBufs * kOutTiles * kOutTileBytes +
                                 kVecBytes + 1024 + 256;
    static_assert(kSmem <= 232448, "shared memory of a block");
};

template <int NB, int MODE, int NACC = 1>   // NACC = 2: every head at most 32 wide, the accumulators of two items side by side
__global__ void __launch_bounds__(kBwdThreads, 1) attn_bwd_kernel(const __grid_constant__ AttnBwdParams P) {
    using Cfg = BwdCfg<NB, MODE>;
    constexpr int kTileBytes = Cfg::kTileBytes, kStrTileBytes = Cfg::kStrTileBytes, kStrBlockBytes = Cfg::kStrBlockBytes;
    constexpr int kStep = Cfg::kStep, kOutTileBytes = Cfg::kOutTileBytes;
    constexpr int RS = Cfg::kResStages, SS = Cfg::kStrStages;
    // TMEM columns.  Heads up to 64 wide: the accumulators take 64 columns each and the bf16 operands of the
    // accumulating products (P^T and dS^T, or dS) live in TMEM too, two values per column; wider heads: accumulators of
    // 128 columns, those operands in shared memory.
    constexpr bool kOpsInTmem = NB == 1;
    constexpr uint32_t kAccIssuers = NB == 1 ? 2 : 1, kScoreIssuers = NB == 1 ? 1 : 2;
    constexpr uint32_t kColX = 0, kColY = 128, kColAcc1 = 256, kColAcc2 = kOpsInTmem ? 320 : 384, kColP = 384, kColDS = 448;
    constexpr int kCodeBase = MODE == 0 ? 14 : 17;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw_addr);
    // resident: [stage][a | b], streamed: [stage][a | b], out tiles, vectors, barriers
    const uint32_t sRes = base, sStr = sRes + 2 * kTileBytes * RS, sOut = sStr + 2 * kStrTileBytes * SS;
    uint8_t* vec_raw = smem + 2 * kTileBytes * RS + 2 * kStrTileBytes * SS + Cfg::kOutBufs * Cfg::kOutTiles * kOutTileBytes;
    float* vec = reinterpret_cast<float*>(vec_raw);                               // [stage][-lse2 | D][128]
    uint8_t* tail = vec_raw + Cfg::kVecBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(tail + 24 * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 24 * 8 + 8);
    const uint32_t bar0 = smem_u32(bars);
    auto r_full = [&](uint32_t s) { return bar0 + 8u * s; };
    auto r_empty = [&](uint32_t s) { return bar0 + 8u * (2 + s); };
    auto t_full = [&](uint32_t s) { return bar0 + 8u * (4 + s); };
    auto t_empty = [&](uint32_t s) { return bar0 + 8u * (8 + s); };
    // accumulators: one set, or two (heads at most 32 wide) that the items take in turn, each with its own pair of barriers
    auto acc_full = [&](uint32_t a) { return bar0 + 8u * (a ? 22 : 15); };
    auto acc_empty = [&](uint32_t a) { return bar0 + 8u * (a ? 23 : 16); };
    constexpr uint32_t n_acc = NACC;
    static_assert(NACC == 1 || NB == 1, "two sets of accumulators need the narrow layout");
    constexpr uint32_t kOB = Cfg::kOutBufs, kOutSetBytes = Cfg::kOutTiles * kOutTileBytes;
    auto out_full = [&](uint32_t b) { return bar0 + 8u * (b ? 20 : 13); };
    auto out_empty = [&](uint32_t b) { return bar0 + 8u * (b ? 21 : 14); };
    // score tiles: one buffer of 128 columns each, or (half-block steps) two of 64, each with its own pair of barriers
    constexpr uint32_t kXY = kStep == 64 ? 2 : 1;
    auto x_full = [&](uint32_t b) { return bar0 + 8u * (b ? 18 : 12); };
    auto xy_free = [&](uint32_t b) { return bar0 + 8u * (b ? 19 : 17); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (uint32_t s = 0; s < 2; ++s) {
            mbar_init(r_full(s), 1);
            mbar_init(r_empty(s), kScoreIssuers);
        }
        for (uint32_t s = 0; s < 4; ++s) {
            mbar_init(t_full(s), 1);
            mbar_init(t_empty(s), kAccIssuers);
        }
        for (uint32_t b = 0; b < 2; ++b) {
            mbar_init(x_full(b), kScoreIssuers);
            mbar_init(xy_free(b), kBwdComputeWarps);
            mbar_init(out_full(b), kBwdComputeWarps);     // barriers the compute threads arrive on: one arrival per warp (its lanes meet first)
            mbar_init(out_empty(b), kAccIssuers);
        }
        for (uint32_t a = 0; a < 2; ++a) {
            mbar_init(acc_full(a), kAccIssuers);
            mbar_init(acc_empty(a), kBwdComputeWarps);
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&P.map_q);
        prefetch_tensormap(&P.map_k);
        prefetch_tensormap(&P.map_v);
        prefetch_tensormap(&P.map_do);
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_holder), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    // item -> (sequence, head, owned block, steps, first streamed block).  MODE 0 owns a key block of a K/V head and
    // walks the query blocks of every query head that reads it, one head after the other (h = the first of them).
    struct BItem {
        int b, h, own, n_steps, n_per, first;
    };
    const int grp = MODE == 0 ? P.heads.rep : 1;
    auto decode = [&](int it) {
        BItem I;
        const int per = (P.n_heads / grp) * P.batch;
        const int a = it / per;
        I.own = MODE == 0 ? a : P.n_t - 1 - a;                 // causal: the blocks with the most steps first
        const int rem = it % per;
        I.h = (rem / P.batch) * grp;
        I.b = rem % P.batch;
        if (MODE == 0) {
            I.first = P.causal ? I.own * (kTile / kStep) : 0;  // query blocks (of kStep queries) at or after the key block
            I.n_per = (P.seq + kStep - 1) / kStep - I.first;
        } else {
            I.first = 0;
            I.n_per = P.causal ? I.own + 1 : P.n_t;            // key blocks up to the query block
        }
        I.n_steps = I.n_per * grp;
        return I;
    };
    // which tensor maps / head columns the resident and streamed "a" (Q/K side) and "b" (V/dCtx side) tiles use
    const CUtensorMap* map_ra = MODE == 0 ? &P.map_k : &P.map_q;
    const CUtensorMap* map_rb = MODE == 0 ? &P.map_v : &P.map_do;
    const CUtensorMap* map_sa = MODE == 0 ? &P.map_q : &P.map_k;
    const CUtensorMap* map_sb = MODE == 0 ? &P.map_do : &P.map_v;

    // The score products X = Ra Sa^T (contraction over the Q/K width) and / or Y = Rb Sb^T (over the V width) of every step:
    // those of a step as soon as every compute thread has the previous scores of the same buffer in registers (it says so
    // half way through its step), also across the boundary between two items.
    auto score_role = [&](bool do_x, bool do_y) {
        uint32_t g = 0, ri = 0;
        bool ok = true;
        for (int it = blockIdx.x; ok && it < P.n_items; it += gridDim.x, ++ri) {
            const BItem I = decode(it);
            const int wa = P.heads.qk_w[I.h], wb = P.heads.vo_w[I.h];
            const uint32_t rs = ri % RS;
            if (!(ok = mbar_wait(r_full(rs), (ri / RS) & 1u, abort_flag, kCodeBase + 1, P.status, P.wait_limit_ns))) break;
            const uint32_t idesc_x = make_idesc(kTile, kStep, 0, 0);
            const uint64_t d_ra = make_smem_desc(sRes + (2 * rs) * kTileBytes, 16, 1024),
                           d_rb = make_smem_desc(sRes + (2 * rs + 1) * kTileBytes, 16, 1024);
            for (int i = 0; ok && i < I.n_steps; ++i, ++g) {
                const uint32_t use = g / kXY, st = g % SS, xb = g % kXY;
                if (use > 0 && !(ok = mbar_wait(xy_free(xb), (use - 1) & 1u, abort_flag, kCodeBase + 1, P.status, P.wait_limit_ns))) break;
                if (!(ok = mbar_wait(t_full(st), (g / SS) & 1u, abort_flag, kCodeBase + 1, P.status, P.wait_limit_ns))) break;
                tc_fence_after();
                const uint64_t d_sa = make_smem_desc(sStr + (2 * st) * kStrTileBytes, 16, 1024),
                               d_sb = make_smem_desc(sStr + (2 * st + 1) * kStrTileBytes, 16, 1024);
                if (do_x) {
                    for (int ks = 0; ks < (wa >> 4); ++ks) {
                        const uint32_t o = ((ks >> 2) * kBlockBytes + (ks & 3) * 32) >> 4, os = ((ks >> 2) * kStrBlockBytes + (ks & 3) * 32) >> 4;
                        tc_mma_bf16(tmem_base + kColX + xb * kStep, d_ra + o, d_sa + os, idesc_x, ks != 0 ? 1u : 0u);
                    }
                }
                if (do_y) {
                    for (int ks = 0; ks < (wb >> 4); ++ks) {
                        const uint32_t o = ((ks >> 2) * kBlockBytes + (ks & 3) * 32) >> 4, os = ((ks >> 2) * kStrBlockBytes + (ks & 3) * 32) >> 4;
                        tc_mma_bf16(tmem_base + kColY + xb * kStep, d_rb + o, d_sb + os, idesc_x, ks != 0 ? 1u : 0u);
                    }
                }
                tc_commit(x_full(xb));
            }
            if (ok) tc_commit(r_empty(rs));
        }
    };
    // The accumulating products number w0 .. w1 - 1 of every step.  Key-block kernel: 0 is dV += P^T dCtx_i (B = streamed b
    // tile), 1 is dK += dS^T Q_i (B = streamed a tile), all steps of the contraction over the step's queries; query-block
    // kernel: dQ += dS K_j (B = streamed a tile), 0 is steps 0-3 of the contraction, 1 is steps 4-7 (two accumulators).
    auto acc_role = [&](int w0, int w1) {
        uint32_t g = 0, ri = 0;
        bool ok = true;
        for (int it = blockIdx.x; ok && it < P.n_items; it += gridDim.x, ++ri) {
            const BItem I = decode(it);
            const uint32_t as = ri % n_acc;
            const uint32_t acc1 = n_acc == 2 ? kColAcc1 + 64 * as : kColAcc1, acc2 = n_acc == 2 ? kColAcc1 + 64 * as + 32 : kColAcc2;
            for (int i = 0; i < I.n_steps; ++i, ++g) {
                const uint32_t st = g % SS;
                if (!(ok = mbar_wait(t_full(st), (g / SS) & 1u, abort_flag, kCodeBase + 1, P.status, P.wait_limit_ns))) break;
                const uint32_t ob = g % kOB;
                if (!(ok = mbar_wait(out_full(ob), (g / kOB) & 1u, abort_flag, kCodeBase + 1, P.status, P.wait_limit_ns))) break;
                if (i == 0 && !(ok = mbar_wait(acc_empty(as), ((ri / n_acc) & 1u) ^ 1u, abort_flag, kCodeBase + 1, P.status, P.wait_limit_ns))) break;
                tc_fence_after();
                for (int which = w0; which < w1; ++which) {
                    const int wn = (MODE == 0 && which == 0) ? P.heads.vo_w[I.h] : P.heads.qk_w[I.h];
                    const uint32_t idesc = make_idesc(kTile, wn, 0, 1);
                    const uint32_t acc_col = (MODE == 0) == (which == 0) ? acc1 : acc2;
                    const uint32_t a_col = (MODE == 0 && which == 0) ? kColP : kColDS;                 // narrow heads: A operand in TMEM
                    const uint32_t sA = sOut + ob * kOutSetBytes + ((MODE == 0 && which == 1) ? kOutTileBytes : 0);   // wide heads: in shared memory
                    const int ks0 = MODE == 0 ? 0 : 4 * which, ks1 = MODE == 0 ? kStep / 16 : 4 * which + 4;
                    const uint64_t db = make_smem_desc(sStr + (2 * st + ((MODE == 0 && which == 0) ? 1 : 0)) * kStrTileBytes, kStrBlockBytes, 1024);
                    for (int ks = ks0; ks < ks1; ++ks) {
                        if (kOpsInTmem)
                            tc_mma_bf16_ts(tmem_base + acc_col, tmem_base + a_col + 8 * ks, db + 128 * ks, idesc, (i != 0 || ks != ks0) ? 1u : 0u);
                        else
                            tc_mma_bf16(tmem_base + acc_col, make_smem_desc(sA + (ks >> 2) * kBlockBytes + (ks & 3) * 32, 16, 1024),
                                        db + 128 * ks, idesc, (i != 0 || ks != ks0) ? 1u : 0u);
                    }
                }
                tc_commit(out_empty(ob));
                tc_commit(t_empty(st));
            }
            if (ok) tc_commit(acc_full(as));
        }
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t g = 0, ri = 0;
            bool ok = true;
            for (int it = blockIdx.x; ok && it < P.n_items; it += gridDim.x, ++ri) {
                const BItem I = decode(it);
                // columns of the resident tiles: MODE 0 the K/V head's block of K^c and V^c, MODE 1 the query head's of Q^c and dCtx
                const int ra_off = MODE == 0 ? P.heads.k_off[I.h] : P.heads.qk_off[I.h];
                const int rb_off = MODE == 0 ? P.heads.v_off[I.h] : P.heads.vo_off[I.h];
                const int nba = (P.heads.qk_w[I.h] + 63) >> 6, nbb = (P.heads.vo_w[I.h] + 63) >> 6;
                const int row0 = I.b * P.seq;
                const uint32_t rs = ri % RS;
                if (!(ok = mbar_wait(r_empty(rs), ((ri / RS) & 1u) ^ 1u, abort_flag, kCodeBase, P.status, P.wait_limit_ns))) break;
                mbar_expect_tx(r_full(rs), (nba + nbb) * kBlockBytes);
                for (int blk = 0; blk < nba; ++blk)
                    tma_load_2d(sRes + (2 * rs) * kTileBytes + blk * kBlockBytes, map_ra, ra_off + 64 * blk, row0 + I.own * kTile, r_full(rs));
                for (int blk = 0; blk < nbb; ++blk)
                    tma_load_2d(sRes + (2 * rs + 1) * kTileBytes + blk * kBlockBytes, map_rb, rb_off + 64 * blk, row0 + I.own * kTile, r_full(rs));
                for (int i = 0; i < I.n_steps; ++i, ++g) {
                    const uint32_t st = g % SS;
                    if (!(ok = mbar_wait(t_empty(st), ((g / SS) & 1u) ^ 1u, abort_flag, kCodeBase, P.status, P.wait_limit_ns))) break;
                    mbar_expect_tx(t_full(st), (nba + nbb) * kStrBlockBytes + (MODE == 0 ? 2 * kStep * 4 : 0));
                    // streamed tiles: MODE 0 the query block of query head h + i / n_per, MODE 1 the key block of the K/V head
                    const int hq = I.h + i / I.n_per;
                    if (MODE == 0) {   // with the query block's per-query vectors
                        const int64_t o = (static_cast<int64_t>(hq) * P.batch + I.b) * P.seq_pad + (I.first + i % I.n_per) * kStep;
                        const int64_t per_arr = static_cast<int64_t>(P.n_heads) * P.batch * P.seq_pad;
                        const uint32_t dst = smem_u32(vec) + st * 2 * kStep * 4;
                        bulk_load(dst, P.vecs + o, kStep * 4, t_full(st));
                        bulk_load(dst + kStep * 4, P.vecs + per_arr + o, kStep * 4, t_full(st));
                    }
                    const int sa_off = MODE == 0 ? P.heads.qk_off[hq] : P.heads.k_off[I.h];
                    const int sb_off = MODE == 0 ? P.heads.vo_off[hq] : P.heads.v_off[I.h];
                    const int y = row0 + (I.first + i % I.n_per) * kStep;
                    for (int blk = 0; blk < nba; ++blk)
                        tma_load_2d(sStr + (2 * st) * kStrTileBytes + blk * kStrBlockBytes, map_sa, sa_off + 64 * blk, y, t_full(st));
                    for (int blk = 0; blk < nbb; ++blk)
                        tma_load_2d(sStr + (2 * st + 1) * kStrTileBytes + blk * kStrBlockBytes, map_sb, sb_off + 64 * blk, y, t_full(st));
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ issuer of the score products
        if (lane == 0) score_role(true, NB == 1);
    } else if (warp >= 2 + kBwdComputeWarps) {
        // ------------------------------------------------------------------ issuers of the accumulating products (wide heads: of Y, and of all accumulating products)
        if (lane == 0) {
            const int which = warp - (2 + kBwdComputeWarps);
            if (NB == 1) acc_role(which, which + 1);
            else if (which == 0) score_role(false, true);
            else acc_role(0, 2);
        }
    } else {
        // ------------------------------------------------------------------ compute
        // Thread = (row of the owned block = TMEM lane, quarter of the streamed block's 128 columns): warps 2..5 take
        // columns [0, 32), warps 6..9 [32, 64), and so on, so every scheduler has four compute warps to interleave.
        const int part = (warp - 2) >> 2;
        const int row = (warp & 3) * 32 + lane;
        constexpr int kHalves = kStep / 64;                            // 16-column halves of this thread's columns
        const int col0 = part * (kStep / 4);                           // this thread's columns of the streamed block
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        // 32 columns = four 16-byte chunks of block col0 / 64 of the row's image
        const uint32_t out_row = sOut + (col0 >> 6) * kBlockBytes + row * 128;
        const int chunk0 = (col0 & 63) >> 3;
        const int swz = row & 7;
        uint32_t g = 0, ri = 0;
        bool ok = true;
        const int64_t T = static_cast<int64_t>(P.batch) * P.seq;
        struct Pend {
            int h, b, own;
            uint32_t ri;
            bool on;
        };
        Pend pend = {0, 0, 0, 0, false};
        // writes an item's accumulators out once they are complete (every thread its quarter of the columns) and releases them
        auto flush = [&](const Pend& d) -> bool {
            const uint32_t as = d.ri % n_acc;
            const uint32_t acc1 = n_acc == 2 ? kColAcc1 + 64 * as : kColAcc1, acc2 = n_acc == 2 ? kColAcc1 + 64 * as + 32 : kColAcc2;
            if (!mbar_wait(acc_full(as), (d.ri / n_acc) & 1u, abort_flag, kCodeBase + 2, P.status, P.wait_limit_ns)) return false;
            tc_fence_after();
            const int pos = d.own * kTile + row;
            const bool live = pos < P.seq;
            const int64_t t = static_cast<int64_t>(d.b) * P.seq + pos;
            auto write_acc = [&](uint32_t colbase, int w, uint16_t* dst, float mul, bool two = false, uint32_t colbase2 = 0) {
#pragma unroll
                for (int c = 0; c < NB; ++c) {
                    const int col = part * (NB * 16) + c * 16;
                    if (col < w) {
                        uint32_t r[16];
                        tc_ld16(t_lane + colbase + col, r);
                        tc_wait_ld();
                        if (two) {                               // the contraction was split over two accumulators
                            uint32_t r2[16];
                            tc_ld16(t_lane + colbase2 + col, r2);
                            tc_wait_ld();
#pragma unroll
                            for (int e = 0; e < 16; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) + __uint_as_float(r2[e]));
                        }
                        if (live) {
                            uint4 v0, v1;
                            v0.x = pack_bf16(__uint_as_float(r[0]) * mul, __uint_as_float(r[1]) * mul);
                            v0.y = pack_bf16(__uint_as_float(r[2]) * mul, __uint_as_float(r[3]) * mul);
                            v0.z = pack_bf16(__uint_as_float(r[4]) * mul, __uint_as_float(r[5]) * mul);
                            v0.w = pack_bf16(__uint_as_float(r[6]) * mul, __uint_as_float(r[7]) * mul);
                            v1.x = pack_bf16(__uint_as_float(r[8]) * mul, __uint_as_float(r[9]) * mul);
                            v1.y = pack_bf16(__uint_as_float(r[10]) * mul, __uint_as_float(r[11]) * mul);
                            v1.z = pack_bf16(__uint_as_float(r[12]) * mul, __uint_as_float(r[13]) * mul);
                            v1.w = pack_bf16(__uint_as_float(r[14]) * mul, __uint_as_float(r[15]) * mul);
                            *reinterpret_cast<uint4*>(dst + col) = v0;
                            *reinterpret_cast<uint4*>(dst + col + 8) = v1;
                        }
                    }
                }
            };
            if (MODE == 0) {
                write_acc(acc1, P.heads.vo_w[d.h], P.dv + t * P.ld_dv + P.heads.v_off[d.h], 1.f);
                write_acc(acc2, P.heads.qk_w[d.h], P.dk + t * P.ld_dqk + P.heads.k_off[d.h], P.scale);
            } else {
                write_acc(acc2, P.heads.qk_w[d.h], P.dq + t * P.ld_dqk + P.heads.qk_off[d.h], P.scale, true, acc1);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(as));
            return true;
        };
        for (int it = blockIdx.x; ok && it < P.n_items; it += gridDim.x, ++ri) {
            const BItem I = decode(it);
            const int own_pos = I.own * kTile + row;                 // position of this thread's row in the sequence
            // MODE 1: this row's -log-sum-exp (base 2) and row dot (zeros past the end of the sequence).  MODE 0: the values of
            // the step's 128 queries arrive in shared memory with the step's tiles.
            float lse_r = 0.f, d_r = 0.f;
            if (MODE == 1) {
                const int64_t o = (static_cast<int64_t>(I.h) * P.batch + I.b) * P.seq_pad + own_pos;
                lse_r = P.vecs[o];
                d_r = P.vecs[static_cast<int64_t>(P.n_heads) * P.batch * P.seq_pad + o];
            }
            for (int i = 0; i < I.n_steps; ++i, ++g) {
                const int other0 = (I.first + i % I.n_per) * kStep;  // first position of the streamed block
                const float* vb = vec + (g % SS) * 2 * kStep;
                const uint32_t xb = g % kXY;
                if (!(ok = mbar_wait(x_full(xb), (g / kXY) & 1u, abort_flag, kCodeBase + 2, P.status, P.wait_limit_ns))) break;
                tc_fence_after();
                // (the step's loads landed long ago; this thread reads the vectors among them, so it looks at their barrier itself)
                if (MODE == 0 && !(ok = mbar_wait(t_full(g % SS), (g / SS) & 1u, abort_flag, kCodeBase + 2, P.status, P.wait_limit_ns))) break;
                // (query position, key position) of element (row, column c): MODE 0 rows are keys, MODE 1 rows are queries
                const int q0 = MODE == 0 ? other0 : I.own * kTile, k0 = MODE == 0 ? I.own * kTile : other0;
                const bool masked = q0 + (MODE == 0 ? kStep : kTile) > P.seq || k0 + kTile > P.seq || (P.causal && q0 < k0 + kTile);
                // two halves of 16 columns: probabilities and dS are packed to bf16 pairs as soon as they exist
                uint32_t pk_p[16], pk_ds[16];
                const f32x2 c2 = pack2(P.scale_log2e, P.scale_log2e), neg1 = pack2(-1.f, -1.f);
#pragma unroll
                for (int hh = 0; hh < kHalves; ++hh) {
                    uint32_t rx[16], ry[16];
                    tc_ld16(t_lane + kColX + xb * kStep + col0 + 16 * hh, rx);
                    tc_ld16(t_lane + kColY + xb * kStep + col0 + 16 * hh, ry);
                    tc_wait_ld();
                    if (hh == kHalves - 1) {                          // this thread's last read of the step's score tiles
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(xy_free(xb));
                    }
                    if (masked) {                                     // pairs outside the mask count as -inf (p = 0)
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const int c = col0 + 16 * hh + e;
                            const int qp = MODE == 0 ? q0 + c : own_pos;
                            const int kp = MODE == 0 ? own_pos : k0 + c;
                            if (!(qp < P.seq && kp < P.seq && (!P.causal || kp <= qp))) rx[e] = 0xff800000u;
                        }
                    }
#pragma unroll
                    for (int e = 0; e < 16; e += 4) {
                        // packed fp32 arithmetic around the exponentials: the step is bound by issue slots as much as by the
                        // exponential unit.  l2 = -lse * log2(e); p = 2^(s * c + l2); dS = p * (dP - D)
                        f32x2 l2a = pack2(lse_r, lse_r), l2b = l2a, dda = pack2(d_r, d_r), ddb = dda;
                        if (MODE == 0) {
                            const float4 a4 = *reinterpret_cast<const float4*>(vb + col0 + 16 * hh + e);
                            const float4 b4 = *reinterpret_cast<const float4*>(vb + kStep + col0 + 16 * hh + e);
                            l2a = pack2(a4.x, a4.y); l2b = pack2(a4.z, a4.w);
                            dda = pack2(b4.x, b4.y); ddb = pack2(b4.z, b4.w);
                        }
                        float x0, x1, x2, x3;
                        unpack2(fma2(pack2(rx[e], rx[e + 1]), c2, l2a), x0, x1);
                        unpack2(fma2(pack2(rx[e + 2], rx[e + 3]), c2, l2b), x2, x3);
                        const float p0 = ex2(x0), p1 = ex2(x1), p2 = ex2(x2), p3 = ex2(x3);
                        float d0, d1, d2, d3;
                        unpack2(mul2(pack2(p0, p1), fma2(dda, neg1, pack2(ry[e], ry[e + 1]))), d0, d1);
                        unpack2(mul2(pack2(p2, p3), fma2(ddb, neg1, pack2(ry[e + 2], ry[e + 3]))), d2, d3);
                        pk_p[8 * hh + (e >> 1)] = pack_bf16(p0, p1);
                        pk_p[8 * hh + (e >> 1) + 1] = pack_bf16(p2, p3);
                        pk_ds[8 * hh + (e >> 1)] = pack_bf16(d0, d1);
                        pk_ds[8 * hh + (e >> 1) + 1] = pack_bf16(d2, d3);
                    }
                }
                // the products that read the previous step's tiles from shared memory are done
                const uint32_t ob = g % kOB;
                if (!(ok = mbar_wait(out_empty(ob), ((g / kOB) & 1u) ^ 1u, abort_flag, kCodeBase + 2, P.status, P.wait_limit_ns))) break;
                if (kOpsInTmem) {   // this thread's 32 columns = 16 packed columns of its TMEM lane
                    if (MODE == 0) tc_st(t_lane + kColP + 16 * part, pk_p);
                    tc_st(t_lane + kColDS + 16 * part, pk_ds);
                    tc_wait_st();
                } else {
#pragma unroll
                    for (int q = 0; q < 2 * kHalves; ++q) {
                        const int chunk = chunk0 + q;
                        if (MODE == 0)
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(out_row + ob * kOutSetBytes + ((chunk ^ swz) << 4)),
                                         "r"(pk_p[4 * q + 0]), "r"(pk_p[4 * q + 1]), "r"(pk_p[4 * q + 2]), "r"(pk_p[4 * q + 3]) : "memory");
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(out_row + ob * kOutSetBytes + (MODE == 0 ? kOutTileBytes : 0) + ((chunk ^ swz) << 4)),
                                     "r"(pk_ds[4 * q + 0]), "r"(pk_ds[4 * q + 1]), "r"(pk_ds[4 * q + 2]), "r"(pk_ds[4 * q + 3]) : "memory");
                    }
                    fence_async_smem();
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(out_full(ob));
                if (i == 0 && pend.on) {   // the previous item's accumulators, now that this item's first step is on its way
                    if (!(ok = flush(pend))) break;
                    pend.on = false;
                }
            }
            if (!ok) break;
            // the accumulators of this item: written out now, or (two sets) after the first step of the CTA's next item, when
            // the last products into them have long landed
            const Pend cur = {I.h, I.b, I.own, ri, true};
            if (n_acc == 2) pend = cur;
            else if (!(ok = flush(cur))) break;
        }
        if (ok && pend.on) flush(pend);
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    if (*abort_flag) {
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn attn_encode_fn() {
    static EncodeFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeFn>(p);
    });
    return fn;
}
// bf16 row-major (rows x cols, pitch ld) as tiles of 64 columns x box_rows rows, 128-byte swizzle, zero fill outside
ecospa_status_t encode_tile_map(CUtensorMap* out, const void* ptr, int64_t rows, int64_t cols, int64_t ld, int box_rows = kTile) {
    EncodeFn enc = attn_encode_fn();
    if (!enc) {
        set_cuda_error(cudaErrorNotSupported, "cuTensorMapEncodeTiled entry point");
        return ECOSPA_ERR_CUDA;
    }
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * 2};
    const cuuint32_t box[2] = {64, static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
        set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled (attention)");
        return ECOSPA_ERR_CUDA;
    }
    return ECOSPA_OK;
}

// Host-only checks shared by the forward and the backward call; fills the layout and the widths of the tensors: Q^c
// (n_qk), Ctx (n_vo), K^c (n_k) and V^c (n_v; the last two equal the first two unless K/V heads are shared).
ecospa_status_t check_heads(const ecospa_heads_t* heads, HeadLayout& L, int64_t& n_qk, int64_t& n_vo, int64_t& n_k, int64_t& n_v,
                            int& max_w) {
    if (!heads || !heads->qk_off || !heads->qk_w || !heads->vo_off || !heads->vo_w) return ECOSPA_ERR_INVALID;
    if (heads->n_heads < 1 || heads->n_kv_heads < 0) return ECOSPA_ERR_INVALID;
    if (heads->n_heads > kMaxHeads) return ECOSPA_ERR_UNSUPPORTED;
    const int n_kv = heads->n_kv_heads;
    if (n_kv > 0 && (!heads->k_off || !heads->v_off || heads->n_heads % n_kv != 0)) return ECOSPA_ERR_INVALID;
    const int rep = n_kv > 0 ? heads->n_heads / n_kv : 1;
    L.rep = rep;
    n_qk = n_vo = n_k = n_v = 0;
    max_w = 0;
    for (int h = 0; h < heads->n_heads; ++h) {
        const int32_t qo = heads->qk_off[h], qw = heads->qk_w[h], vo = heads->vo_off[h], vw = heads->vo_w[h];
        const int32_t ko = n_kv > 0 ? heads->k_off[h / rep] : qo, vko = n_kv > 0 ? heads->v_off[h / rep] : vo;
        if (qo < 0 || vo < 0 || ko < 0 || vko < 0 || qw < 1 || vw < 1) return ECOSPA_ERR_INVALID;
        if (qw > 128 || vw > 128) return ECOSPA_ERR_UNSUPPORTED;
        if ((qw & 15) || (vw & 15) || (qo & 7) || (vo & 7) || (ko & 7) || (vko & 7)) return ECOSPA_ERR_ALIGNMENT;
        // the query heads of a group share the group's kept indices, hence its widths
        if (h % rep != 0 && (qw != heads->qk_w[h - h % rep] || vw != heads->vo_w[h - h % rep])) return ECOSPA_ERR_INVALID;
        L.qk_off[h] = qo; L.qk_w[h] = qw; L.vo_off[h] = vo; L.vo_w[h] = vw; L.k_off[h] = ko; L.v_off[h] = vko;
        n_qk = std::max<int64_t>(n_qk, qo + qw);
        n_vo = std::max<int64_t>(n_vo, vo + vw);
        n_k = std::max<int64_t>(n_k, ko + qw);
        n_v = std::max<int64_t>(n_v, vko + vw);
        max_w = std::max(max_w, std::max(qw, vw));
    }
    return ECOSPA_OK;
}
ecospa_status_t check_mat(const void* p, int64_t ld, int64_t cols) {
    if (!p || ld < cols) return ECOSPA_ERR_INVALID;
    if (!aligned16(p) || (ld * 2) % 16) return ECOSPA_ERR_ALIGNMENT;
    return ECOSPA_OK;
}

}  // namespace

}  // namespace ecospa

using namespace ecospa;

extern "C" ecospa_status_t ecospa_coupled_attn_fwd(const void* Qc, const void* Kc, int64_t ld_qk, const void* Vc, int64_t ld_v,
                                                   int64_t batch, int64_t seq, const ecospa_heads_t* heads, float scale,
                                                   int32_t causal, void* Ctx, int64_t ld_ctx, float* lse, void* stream) {
    static thread_local AttnFwdParams P;
    int64_t n_qk = 0, n_vo = 0, n_k = 0, n_v = 0;
    int max_w = 0;
    ecospa_status_t st = check_heads(heads, P.heads, n_qk, n_vo, n_k, n_v, max_w);
    if (st != ECOSPA_OK) return st;
    if (batch < 1 || seq < 1 || batch * seq > INT32_MAX || !lse) return ECOSPA_ERR_INVALID;
    if (!(scale > 0.f) || !std::isfinite(scale)) return ECOSPA_ERR_INVALID;
    if ((st = check_mat(Qc, ld_qk, n_qk)) != ECOSPA_OK || (st = check_mat(Kc, ld_qk, n_k)) != ECOSPA_OK ||
        (st = check_mat(Vc, ld_v, n_v)) != ECOSPA_OK || (st = check_mat(Ctx, ld_ctx, n_vo)) != ECOSPA_OK)
        return st;
    if (reinterpret_cast<uintptr_t>(lse) & 3u) return ECOSPA_ERR_ALIGNMENT;
    int* status = engine_status_ptr(&st);
    if (!status) return st;
    const int64_t T = batch * seq;
    // output heads up to 32 wide (and Q/K heads up to 64): the stream kernel (K / V tiles as slices of 64 keys); wider
    // heads: two query tiles per CTA, with one or two 64-column blocks per tile
    int max_vo = 0;
    for (int h = 0; h < heads->n_heads; ++h) max_vo = std::max<int>(max_vo, heads->vo_w[h]);
    const bool streams = max_w <= 64 && max_vo <= 32;
    if ((st = encode_tile_map(&P.map_q, Qc, T, n_qk, ld_qk)) != ECOSPA_OK) return st;
    if ((st = encode_tile_map(&P.map_k, Kc, T, n_k, ld_qk, streams ? 64 : kTile)) != ECOSPA_OK) return st;
    if ((st = encode_tile_map(&P.map_v, Vc, T, n_v, ld_v, streams ? 64 : kTile)) != ECOSPA_OK) return st;
    P.batch = static_cast<int32_t>(batch);
    P.seq = static_cast<int32_t>(seq);
    P.n_heads = heads->n_heads;
    P.n_qt = static_cast<int32_t>(ceil_div(seq, kTile));
    P.causal = causal != 0;
    const int64_t items = static_cast<int64_t>(streams ? P.n_qt : (P.n_qt + 1) / 2) * P.n_heads * batch;
    if (items > INT32_MAX) return ECOSPA_ERR_UNSUPPORTED;
    P.n_items = static_cast<int32_t>(items);
    P.scale_log2e = scale * 1.4426950408889634f;
    P.ctx = static_cast<uint16_t*>(Ctx);
    P.ld_ctx = ld_ctx;
    P.lse = lse;
    P.status = status;
    P.wait_limit_ns = engine_wait_limit_ns();
    static std::once_flag once[64];
    int dev = 0;
    cudaGetDevice(&dev);
    cudaError_t e = cudaSuccess;
    std::call_once(once[dev & 63], [&] {
        e = cudaFuncSetAttribute(attn_fwd_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdCfg<1>::kSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_fwd_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdCfg<2>::kSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_fwd_ms_kernel<3, 32>, cudaFuncAttributeMaxDynamicSharedMemorySize, MsCfg<3, 32>::kSmem);
    });
    if (e != cudaSuccess) {
        set_cuda_error(e, "attention setup");
        cudaGetLastError();
        return ECOSPA_ERR_CUDA;
    }
    const int grid = std::min<int>(P.n_items, std::max(1, engine_num_sms()));
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (streams) attn_fwd_ms_kernel<3, 32><<<grid, MsCfg<3, 32>::kThreads, MsCfg<3, 32>::kSmem, cs>>>(P);
    else if (max_w <= 64) attn_fwd_kernel<1><<<grid, kFwdThreads, FwdCfg<1>::kSmem, cs>>>(P);
    else attn_fwd_kernel<2><<<grid, kFwdThreads, FwdCfg<2>::kSmem, cs>>>(P);
    return check_launch("attn_fwd_kernel");
}

extern "C" size_t ecospa_attn_workspace_bytes(int64_t batch, int64_t seq, int32_t n_heads) {
    if (batch < 1 || seq < 1 || n_heads < 1) return 0;
    // two fp32 per (head, position of the sequences padded to whole blocks of 128): -lse * log2(e) and the row dots D
    return static_cast<size_t>(batch) * ceil_div(seq, static_cast<int64_t>(kTile)) * kTile * n_heads * 8 + 256;
}

extern "C" ecospa_status_t ecospa_coupled_attn_bwd(const void* Qc, const void* Kc, int64_t ld_qk, const void* Vc, int64_t ld_v,
                                                   const void* Ctx, int64_t ld_ctx, const void* dCtx, int64_t ld_dctx,
                                                   const float* lse, int64_t batch, int64_t seq, const ecospa_heads_t* heads,
                                                   float scale, int32_t causal, void* dQc, void* dKc, int64_t ld_dqk,
                                                   void* dVc, int64_t ld_dv, void* workspace, size_t workspace_bytes,
                                                   void* stream_) {
    static thread_local AttnBwdParams P;
    static thread_local DotParams D;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int64_t n_qk = 0, n_vo = 0, n_k = 0, n_v = 0;
    int max_w = 0;
    ecospa_status_t st = check_heads(heads, P.heads, n_qk, n_vo, n_k, n_v, max_w);
    if (st != ECOSPA_OK) return st;
    if (batch < 1 || seq < 1 || batch * seq > INT32_MAX || !lse) return ECOSPA_ERR_INVALID;
    if (!(scale > 0.f) || !std::isfinite(scale)) return ECOSPA_ERR_INVALID;
    if ((st = check_mat(Qc, ld_qk, n_qk)) != ECOSPA_OK || (st = check_mat(Kc, ld_qk, n_k)) != ECOSPA_OK ||
        (st = check_mat(Vc, ld_v, n_v)) != ECOSPA_OK || (st = check_mat(Ctx, ld_ctx, n_vo)) != ECOSPA_OK ||
        (st = check_mat(dCtx, ld_dctx, n_vo)) != ECOSPA_OK || (st = check_mat(dQc, ld_dqk, n_qk)) != ECOSPA_OK ||
        (st = check_mat(dKc, ld_dqk, n_k)) != ECOSPA_OK || (st = check_mat(dVc, ld_dv, n_v)) != ECOSPA_OK)
        return st;
    if (reinterpret_cast<uintptr_t>(lse) & 3u) return ECOSPA_ERR_ALIGNMENT;
    if (n_vo / 8 > kDotMaxVecs) return ECOSPA_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < ecospa_attn_workspace_bytes(batch, seq, heads->n_heads)) return ECOSPA_ERR_WORKSPACE;
    if (!aligned16(workspace)) return ECOSPA_ERR_ALIGNMENT;
    int* status = engine_status_ptr(&st);
    if (!status) return st;
    const int64_t T = batch * seq;
    if ((st = encode_tile_map(&P.map_q, Qc, T, n_qk, ld_qk)) != ECOSPA_OK) return st;
    if ((st = encode_tile_map(&P.map_k, Kc, T, n_k, ld_qk)) != ECOSPA_OK) return st;
    if ((st = encode_tile_map(&P.map_v, Vc, T, n_v, ld_v)) != ECOSPA_OK) return st;
    if ((st = encode_tile_map(&P.map_do, dCtx, T, n_vo, ld_dctx)) != ECOSPA_OK) return st;
    float* vecs = static_cast<float*>(workspace);
    P.batch = static_cast<int32_t>(batch);
    P.seq = static_cast<int32_t>(seq);
    P.n_heads = heads->n_heads;
    P.n_t = static_cast<int32_t>(ceil_div(seq, kTile));
    P.causal = causal != 0;
    const int64_t items = static_cast<int64_t>(P.n_t) * P.n_heads * batch;
    if (items > INT32_MAX) return ECOSPA_ERR_UNSUPPORTED;
    P.n_items = static_cast<int32_t>(items);
    P.scale = scale;
    P.scale_log2e = scale * 1.4426950408889634f;
    P.lse = lse;
    P.vecs = vecs;
    P.seq_pad = static_cast<int32_t>(ceil_div(seq, static_cast<int64_t>(kTile)) * kTile);
    P.dq = static_cast<uint16_t*>(dQc);
    P.dk = static_cast<uint16_t*>(dKc);
    P.dv = static_cast<uint16_t*>(dVc);
    P.ld_dqk = ld_dqk;
    P.ld_dv = ld_dv;
    P.status = status;
    P.wait_limit_ns = engine_wait_limit_ns();
    static std::once_flag once[64];
    int dev = 0;
    cudaGetDevice(&dev);
    cudaError_t e = cudaSuccess;
    std::call_once(once[dev & 63], [&] {
        e = cudaFuncSetAttribute(attn_bwd_kernel<1, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<1, 0>::kSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_bwd_kernel<1, 0, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<1, 0>::kSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_bwd_kernel<1, 1, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<1, 1>::kSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_bwd_kernel<2, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<2, 0>::kSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_bwd_kernel<1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<1, 1>::kSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_bwd_kernel<2, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<2, 1>::kSmem);
    });
    if (e != cudaSuccess) {
        set_cuda_error(e, "attention backward setup");
        cudaGetLastError();
        return ECOSPA_ERR_CUDA;
    }
    // row dots D
    D.heads = P.heads;
    D.ctx = static_cast<const uint16_t*>(Ctx);
    D.dctx = static_cast<const uint16_t*>(dCtx);
    D.vecs = vecs;
    D.lse = lse;
    D.batch = static_cast<int32_t>(batch);
    D.seq = static_cast<int32_t>(seq);
    D.seq_pad = P.seq_pad;
    D.ld_ctx = ld_ctx;
    D.ld_dctx = ld_dctx;
    D.T = T;
    D.n_heads = heads->n_heads;
    D.n_vecs = static_cast<int32_t>(n_vo / 8);
    attn_rowdot_kernel<<<static_cast<unsigned>(ceil_div(batch * D.seq_pad, static_cast<int64_t>(kDotWarps))), 32 * kDotWarps, 0, stream>>>(D);
    if ((st = check_launch("attn_rowdot_kernel")) != ECOSPA_OK) return st;
    const int nb = max_w > 64 ? 2 : 1;
    // dK, dV: one item per (sequence, K/V head, key block); dQ: one per (sequence, query head, query block)
    const int items_q = P.n_items;
    P.n_items = items_q / P.heads.rep;
    int grid = std::min<int>(P.n_items, std::max(1, engine_num_sms()));
    if (nb == 1) {
        if (max_w <= 32) attn_bwd_kernel<1, 0, 2><<<grid, kBwdThreads, BwdCfg<1, 0>::kSmem, stream>>>(P);
        else attn_bwd_kernel<1, 0><<<grid, kBwdThreads, BwdCfg<1, 0>::kSmem, stream>>>(P);
    } else {   // wide heads: the streamed query blocks are half blocks
        AttnBwdParams P0 = P;
        if ((st = encode_tile_map(&P0.map_q, Qc, T, n_qk, ld_qk, BwdCfg<2, 0>::kStep)) != ECOSPA_OK) return st;
        if ((st = encode_tile_map(&P0.map_do, dCtx, T, n_vo, ld_dctx, BwdCfg<2, 0>::kStep)) != ECOSPA_OK) return st;
        attn_bwd_kernel<2, 0><<<grid, kBwdThreads, BwdCfg<2, 0>::kSmem, stream>>>(P0);
    }
    if ((st = check_launch("attn_bwd_kernel (dK, dV)")) != ECOSPA_OK) return st;
    P.n_items = items_q;
    grid = std::min<int>(P.n_items, std::max(1, engine_num_sms()));
    if (nb == 1 && max_w <= 32) attn_bwd_kernel<1, 1, 2><<<grid, kBwdThreads, BwdCfg<1, 1>::kSmem, stream>>>(P);
    else if (nb == 1) attn_bwd_kernel<1, 1><<<grid, kBwdThreads, BwdCfg<1, 1>::kSmem, stream>>>(P);
    else attn_bwd_kernel<2, 1><<<grid, kBwdThreads, BwdCfg<2, 1>::kSmem, stream>>>(P);
    return check_launch("attn_bwd_kernel (dQ)");
}
