// Grouped persistent bf16 GEMM for sm_100a: TMA -> shared memory ring -> tcgen05.mma (fp32 accumulators
// in TMEM, double buffered) -> fused epilogues.  Two forms of the same kernel:
//   single  cta_group::1, one CTA per SM computes 128x256 tiles (2 stages of 2 x (16 KB A + 32 KB B))
//   pair    cta_group::2, a cluster of two CTAs computes 256x256 tiles: each CTA loads its 128 rows of A
//           and its half of B (3 stages of 2 x (16 KB + 16 KB)), the leader CTA issues the MMAs for both,
//           so every SM fetches a third less operand data per flop.  Every CTA issues its own loads: the
//           peer's loads signal the leader's barrier, and completion is committed to each CTA's barrier.
//
// One launch computes up to kMaxGemmOps independent products ("ops"), each C = sum over one to three
// K segments of A_seg * B_seg with K-major or MN-major operands (chosen per segment, so that weights
// and activations are consumed in whatever row-major orientation they are stored).  Warp roles:
//   warp 0      producer: one elected lane issues the TMA loads of a stage (two 64-deep k-blocks)
//   warp 1      owns the 512 TMEM columns; one elected lane issues the MMAs and the commits
//   warps 2..9  epilogue: two warps per TMEM lane quadrant, each takes half of the tile's columns; a warp
//               converts its rows, stages them in swizzled shared memory and one lane issues a TMA tile
//               store (a reducing store when the output is added to what C holds)
// Tiles are numbered op by op, longest contraction first; the host hands them out longest first to the
// least-loaded worker and passes the lists as a table in the kernel parameters (a plain stride when
// there are many tiles per worker).  The kernel is launched with programmatic stream serialization and
// touches no global memory before griddepcontrol.wait, so its set-up overlaps the previous kernel's tail.
// Every mbarrier wait is bounded in time; on expiry the CTA records an error code in a device
// status word, waits for its copies in flight, frees its TMEM and returns.

#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "common.cuh"
#include "gemm.cuh"

namespace ecospa {

namespace {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int kAStage = BM * BK * 2;        // 16 KB
constexpr int kBStage = BN * BK * 2;        // 32 KB
constexpr int kBHalf = kBStage / 2;
constexpr int kRingBytes = 4 * (kAStage + kBStage);   // = 6 * (kAStage + kBHalf) = 192 KB
constexpr int kMaxStages = 6;
constexpr int kAtomBytes = 64 * 64 * 2;     // one 64x64 bf16 swizzle atom of an MN-major operand
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kTmemCols = 512;
constexpr int kMaxSeg = 3;
constexpr int kOperandMaps = 3 * kMaxSeg;   // per K segment: one A map and two B (half) maps
constexpr int kMapsPerOp = kOperandMaps + 3; // + one store map per output (C, C2, C3)
constexpr int kEpiSlotBytes = 32 * 32 * 2;  // one 32-row x 64-byte staging image; a warp owns two (= one 32 x 128-byte image)
constexpr int kEpiBytes = kEpiWarps * 2 * kEpiSlotBytes;
constexpr int kSmemBytes = kRingBytes + kEpiBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr unsigned long long kDefaultWaitLimitNs = 2000000000ull;  // 2 s

struct DevProblem {
    int32_t M, N;
    int32_t kb_end[kMaxSeg];     // cumulative k-blocks: segment s covers [kb_end[s-1], kb_end[s])
    int32_t kblocks;             // k-blocks of all segments
    int32_t tiles_m, tiles_n, tile_start;
    int32_t n_per_tile;          // output columns per tile: 256, or 128 hidden units for EPI_SWIGLU
    int32_t half1_n_off;         // n-coordinate of B half 1 relative to half 0
    int32_t epi;
    int32_t k_off[kMaxSeg];      // first contraction index of each segment
    uint8_t a_mn[kMaxSeg], b_mn[kMaxSeg];
    uint8_t map_a[kMaxSeg], map_b[kMaxSeg][2];
    uint8_t a_3d[kMaxSeg], b_3d[kMaxSeg];   // MN-major operand fetched as one 3-D box (both 64-wide atoms)
    uint8_t a_big[kMaxSeg], b_big[kMaxSeg]; // pair mode: one box brings both k-blocks of a stage
    uint8_t map_c[3];            // store maps of C, C2, C3
    uint8_t pad2_[2];
    uint8_t out_f32, accumulate, bias_f32, pad_[5];
    void* C;
    void* C2;
    void* C3;
    const void* bias;
    const void* H;
    const void* Hb;
    int64_t ldc, ldh;
};

constexpr int kMaxOrder = 2048;              // entries of the explicit tile schedule
constexpr uint16_t kNoTile = 0xffff;
struct GemmParams {
    alignas(64) CUtensorMap maps[kMaxGemmOps * kMapsPerOp];
    DevProblem prob[kMaxGemmOps];
    // Worker w runs, in round i, tile order[w + i * workers] (kNoTile = nothing) when use_order is set,
    // otherwise tile w + i * workers.
    uint16_t order[kMaxOrder];
    int32_t n_problems, total_tiles, rounds, use_order;
    int* status;
    unsigned long long wait_limit_ns;   // every mbarrier wait of the launch gives up after this long
};

__device__ int g_gemm_status = 0;

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  Returns false if the wait gave up (or another thread of the CTA already did).
template <bool CLUSTER>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int code, int* status,
                                          unsigned long long limit_ns) {
    // Fast path: plain polling.  The (slow) global timer is only consulted every 1024 failed polls,
    // so a wait that completes normally never touches it (limits under a millisecond look at it on
    // every failed poll, so that they are kept to within a poll).
    unsigned long long t0 = 0;
    uint32_t spins = 0;
    const uint32_t mask = limit_ns < 1000000ull ? 0u : 1023u;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & mask) == 0) {
            if (*abort_flag) return false;
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            if (now - t0 > limit_ns) {
                *abort_flag = 1;
                atomicCAS(status, 0, code);
                return false;
            }
        }
    }
}

// --- cluster (CTA pair) helpers
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of `addr` (a shared::cta address of this CTA) in the CTA of rank `rank`
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load issued by one CTA of a pair; the completion may be signalled on the peer's (leader's) barrier.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar_cluster) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_cluster) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int y, int z, int w, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(0), "r"(y), "r"(z), "r"(w)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, int y, int z, int w, uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(0), "r"(y), "r"(z), "r"(w)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}

// --- TMA tile stores (shared memory -> global), tracked per issuing thread in bulk groups
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
}
// C += tile: the addition is done by the memory system in the output's type, once per element
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all but the newest N stores of this thread have finished reading their shared-memory source
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((addr >> 4) & 0x3fffu);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3fffu) << 16;
    d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3fffu) << 32;
    d |= 1ull << 46;   // descriptor version of this architecture
    d |= 2ull << 61;   // 128-byte swizzle
    return d;
}

// ------------------------------------------------------------------------------------------------
// epilogue math (fp32)
// ------------------------------------------------------------------------------------------------
// The erf-form GELU needs Phi(x), the standard normal CDF, for 32768 outputs per tile, which makes the
// epilogue ALU-bound if it is evaluated with exponentials and divisions.  Here
//   Phi(x) ~= 1/2 + xc * Q(xc^2),   xc = clamp(x, -4.5, 4.5),
// with Q a degree-8 polynomial fitted (weighted least squares on Chebyshev nodes, refitted towards the
// minimax error) to (Phi(x) - 1/2)/x on [0, 4.5]; |error| <= 2.1e-5 everywhere (the clamp contributes
// 3.4e-6), far below the bf16 rounding of the outputs.  Two elements are evaluated per instruction with
// the packed fp32 pair arithmetic of this architecture.
typedef unsigned long long f32x2;   // two fp32 values in one 64-bit register
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float ex2_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Phi of two values
__device__ __forceinline__ f32x2 normal_cdf2(float x0, float x1) {
    const f32x2 xc = pack2(fminf(fmaxf(x0, -4.5f), 4.5f), fminf(fmaxf(x1, -4.5f), 4.5f));
    const f32x2 t = mul2(xc, xc);
    f32x2 q = pack2(3.80569048497037e-11f, 3.80569048497037e-11f);
    q = fma2(q, t, pack2(-4.0023149239232225e-09f, -4.0023149239232225e-09f));
    q = fma2(q, t, pack2(1.8461658157775673e-07f, 1.8461658157775673e-07f));
    q = fma2(q, t, pack2(-4.959736997989239e-06f, -4.959736997989239e-06f));
    q = fma2(q, t, pack2(8.72766540851444e-05f, 8.72766540851444e-05f));
    q = fma2(q, t, pack2(-0.0010767392814159393f, -0.0010767392814159393f));
    q = fma2(q, t, pack2(0.009729491546750069f, 0.009729491546750069f));
    q = fma2(q, t, pack2(-0.06624043732881546f, -0.06624043732881546f));
    q = fma2(q, t, pack2(0.3988664746284485f, 0.3988664746284485f));
    return fma2(xc, q, pack2(0.5f, 0.5f));
}
// v[i] <- GELU(v[i]) = v[i] Phi(v[i])
__device__ __forceinline__ void gelu_erf32(float (&v)[32]) {
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        const f32x2 g = mul2(pack2(v[i], v[i + 1]), normal_cdf2(v[i], v[i + 1]));
        unpack2(g, v[i], v[i + 1]);
    }
}
// v[i] <- v[i] * GELU'(h[i]),  GELU'(h) = Phi(h) + h phi(h),  phi(h) = exp(-h^2/2)/sqrt(2 pi).
// With hc = clamp(h, -4.5, 4.5) and t = hc^2:  Phi ~= 1/2 + hc Q6(t) (degree-6 fit of the same kind as above,
// |error| <= 3.0e-4, an order of magnitude below the bf16 rounding of the result) and
// phi = 2^(-t log2(e)/2 - log2(sqrt(2 pi))); beyond the clamp both terms are within 1e-4 of their limits.
__device__ __forceinline__ void dgelu_erf32(float (&v)[32], const float (&h)[32]) {
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        const f32x2 hc = pack2(fminf(fmaxf(h[i], -4.5f), 4.5f), fminf(fmaxf(h[i + 1], -4.5f), 4.5f));
        const f32x2 t = mul2(hc, hc);
        const f32x2 ex = fma2(t, pack2(-0.72134752044448170f, -0.72134752044448170f),
                              pack2(-1.3257480647361593f, -1.3257480647361593f));
        float e0, e1;
        unpack2(ex, e0, e1);
        f32x2 q = pack2(1.431838114740458e-08f, 1.431838114740458e-08f);
        q = fma2(q, t, pack2(-1.1645848871921771e-06f, -1.1645848871921771e-06f));
        q = fma2(q, t, pack2(3.9588092477060854e-05f, 3.9588092477060854e-05f));
        q = fma2(q, t, pack2(-0.0007395460270345211f, -0.0007395460270345211f));
        q = fma2(q, t, pack2(0.008474125526845455f, 0.008474125526845455f));
        q = fma2(q, t, pack2(-0.06415736675262451f, -0.06415736675262451f));
        q = fma2(q, t, pack2(0.39786770939826965f, 0.39786770939826965f));
        // Phi + h phi = 1/2 + hc (Q6 + phi)
        const f32x2 qp = add2(pack2(ex2_fast(e0), ex2_fast(e1)), q);
        const f32x2 d = fma2(hc, qp, pack2(0.5f, 0.5f));
        const f32x2 r = mul2(pack2(v[i], v[i + 1]), d);
        unpack2(r, v[i], v[i + 1]);
    }
}
// tanh(u) = 1 - 2 / (1 + exp(2u)); saturates correctly for large |u|
__device__ __forceinline__ float tanh_fast(float u) { return 1.f - __fdividef(2.f, 1.f + __expf(2.f * u)); }
__device__ __forceinline__ float gelu_tanh(float x) {
    const float u = 0.79788456080286536f * (x + 0.044715f * x * x * x);
    return 0.5f * x * (1.f + tanh_fast(u));
}
__device__ __forceinline__ float dgelu_tanh(float x) {
    const float u = 0.79788456080286536f * (x + 0.044715f * x * x * x);
    const float t = tanh_fast(u);
    const float du = 0.79788456080286536f * (1.f + 3.f * 0.044715f * x * x);
    return 0.5f * (1.f + t) + 0.5f * x * (1.f - t * t) * du;
}
__device__ __forceinline__ float sigmoidf_(float x) { return __fdividef(1.f, 1.f + __expf(-x)); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Staging images for the TMA tile stores.  A warp owns 4 KB: either one image of 32 rows x 128 bytes in the
// 128-byte swizzle (64 bf16 or 32 fp32 columns; 16-byte chunk j of row r sits at chunk j ^ (r & 7)), or two
// "slots" of 32 rows x 64 bytes in the 64-byte swizzle (32 bf16 columns; chunk j of row r at j ^ ((r >> 1) & 3)).
// Lane = row (what tcgen05.ld delivers); both layouts are bank-conflict free for that access.
// Before an image is overwritten the issuing lane waits until the stores that still read it are done
// (KEEP = stores that may stay in flight because they read the other slot).
template <int KEEP>
__device__ __forceinline__ void stage_begin(int lane) {
    if (lane == 0) bulk_wait_read<KEEP>();
    __syncwarp();
}
__device__ __forceinline__ void stage_commit(const CUtensorMap* map, uint32_t buf, int x, int y, int lane, bool add = false) {
    fence_async_smem();
    __syncwarp();
    if (lane == 0) {
        if (add) tma_reduce_add_2d(map, buf, x, y);
        else tma_store_2d(map, buf, x, y);
        bulk_commit();
    }
}
// 32 words (128 bytes) per lane
__device__ __forceinline__ void stage_row128(uint32_t buf, int lane, const uint32_t (&w)[32]) {
#pragma unroll
    for (int j = 0; j < 8; ++j)
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(buf + lane * 128 + ((j ^ (lane & 7)) << 4)),
                     "r"(w[4 * j]), "r"(w[4 * j + 1]), "r"(w[4 * j + 2]), "r"(w[4 * j + 3]) : "memory");
}
// 64 fp32 values of one row -> 64 bf16 columns (one 128-byte image row)
__device__ __forceinline__ void stage_bf16x64(uint32_t buf, int lane, const float (&v0)[32], const float (&v1)[32]) {
    uint32_t w[32];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        w[i] = pack_bf16(v0[2 * i], v0[2 * i + 1]);
        w[16 + i] = pack_bf16(v1[2 * i], v1[2 * i + 1]);
    }
    stage_row128(buf, lane, w);
}
// 32 fp32 values of one row -> 32 fp32 columns (one 128-byte image row)
__device__ __forceinline__ void stage_f32x32(uint32_t buf, int lane, const float (&v)[32]) {
    uint32_t w[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) w[i] = __float_as_uint(v[i]);
    stage_row128(buf, lane, w);
}
// 32 fp32 values of one row -> 32 bf16 columns (one 64-byte slot row)
__device__ __forceinline__ void stage_bf16x32(uint32_t slot, int lane, const float (&v)[32]) {
#pragma unroll
    for (int c = 0; c < 4; ++c)
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(slot + lane * 64 + ((c ^ ((lane >> 1) & 3)) << 4)),
                     "r"(pack_bf16(v[8 * c + 0], v[8 * c + 1])), "r"(pack_bf16(v[8 * c + 2], v[8 * c + 3])),
                     "r"(pack_bf16(v[8 * c + 4], v[8 * c + 5])), "r"(pack_bf16(v[8 * c + 6], v[8 * c + 7]))
                     : "memory");
}

// Landing buffer of the saved activations: 32 rows x 32 bf16 columns, 64 bytes per row, the four 16-byte
// chunks of a row permuted by (chunk ^ ((row >> 1) & 3)) so that both access patterns are conflict-free:
//   "line" pattern: 4 lanes per row, 8 rows per instruction (coalesced 64-byte global segments);
//   "row" pattern:  lane = row, a lane touches the four chunks of its row (the layout of tcgen05.ld).
__device__ __forceinline__ uint32_t epi_chunk_addr(uint32_t buf, int row, int chunk) {
    return buf + row * 64 + ((chunk ^ ((row >> 1) & 3)) << 4);
}

// global (bf16, rows m_warp.. x columns n..n+31) -> registers in the coalesced "line" pattern.  Split in
// two so that the global loads of the next chunk are in flight while the current one is processed.
__device__ __forceinline__ void staged_load32_issue(const unsigned short* H, int64_t ldh, int m_warp, int n, int M, int N,
                                                    uint4 (&q)[4], int lane) {
    const int c = lane & 3;
    const int col = n + 8 * c;
    if (m_warp + 32 <= M && n + 32 <= N) {      // the whole block is inside: four plain vector loads
        const unsigned short* g0 = H + static_cast<int64_t>(m_warp + (lane >> 2)) * ldh + col;
#pragma unroll
        for (int i = 0; i < 4; ++i) q[i] = *reinterpret_cast<const uint4*>(g0 + static_cast<int64_t>(8 * i) * ldh);
        return;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = 8 * i + (lane >> 2);
        q[i] = make_uint4(0, 0, 0, 0);
        if (m_warp + row < M && col < N) {
            const unsigned short* g = H + static_cast<int64_t>(m_warp + row) * ldh + col;
            if (col + 8 <= N) {
                q[i] = *reinterpret_cast<const uint4*>(g);
            } else {
                uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if (col + e < N) w[e >> 1] |= static_cast<uint32_t>(g[e]) << ((e & 1) * 16);
                q[i] = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
    }
}
// registers ("line" pattern) -> buffer -> registers (one row per lane, fp32)
__device__ __forceinline__ void staged_load32_finish(uint32_t buf, const uint4 (&q)[4], float (&v)[32], int lane) {
    const int c = lane & 3;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = 8 * i + (lane >> 2);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(epi_chunk_addr(buf, row, c)), "r"(q[i].x), "r"(q[i].y), "r"(q[i].z), "r"(q[i].w) : "memory");
    }
    __syncwarp();
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
        uint4 t;
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(t.x), "=r"(t.y), "=r"(t.z), "=r"(t.w) : "r"(epi_chunk_addr(buf, lane, cc)));
        v[8 * cc + 0] = bf16_lo(t.x); v[8 * cc + 1] = bf16_hi(t.x);
        v[8 * cc + 2] = bf16_lo(t.y); v[8 * cc + 3] = bf16_hi(t.y);
        v[8 * cc + 4] = bf16_lo(t.z); v[8 * cc + 5] = bf16_hi(t.z);
        v[8 * cc + 6] = bf16_lo(t.w); v[8 * cc + 7] = bf16_hi(t.w);
    }
    __syncwarp();
}

// tile of worker `worker` in round `i`, or -1
__device__ __forceinline__ int scheduled_tile(const GemmParams& P, int worker, int n_workers, int i) {
    const int pos = worker + i * n_workers;
    if (P.use_order) {
        const int t = P.order[pos];
        return t == kNoTile ? -1 : t;
    }
    return pos < P.total_tiles ? pos : -1;
}

// v[i] += bias of column i, where lane i of the warp holds that column's bias
__device__ __forceinline__ void add_bias32(float (&v)[32], float b) {
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] += __shfl_sync(0xffffffffu, b, i);
}

__device__ __forceinline__ const DevProblem& find_problem(const GemmParams& P, int tile) {
    int pi = 0;
#pragma unroll
    for (int i = 1; i < kMaxGemmOps; ++i)
        if (i < P.n_problems && P.prob[i].tile_start <= tile) pi = i;
    return P.prob[pi];
}

// ------------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------------
template <bool PAIR>
__global__ void __launch_bounds__(kThreads, 1) gemm_kernel(const __grid_constant__ GemmParams P) {
    constexpr int kSub = 2;                                  // 64-deep k-blocks per pipeline stage
    constexpr int kStages = PAIR ? 3 : 2;
    constexpr int kBLocal = PAIR ? kBHalf : kBStage;        // B bytes this CTA holds per k-block
    constexpr int kTileM = PAIR ? 2 * BM : BM;               // rows of one scheduled tile
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;       // 1024-byte aligned stage memory
    uint8_t* smem = smem_raw + (base - raw_addr);
    const uint32_t sA = base, sB = base + kStages * kSub * kAStage;
    const uint32_t sEpi = base + kRingBytes;
    uint8_t* tail = smem + kRingBytes + kEpiBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);        // full[S], empty[S], tmem_full[2], tmem_empty[2]
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(tail + (2 * kMaxStages + 4) * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + (2 * kMaxStages + 4) * 8 + 8);
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kStages + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kStages + 2 + a); };

    // Launched with programmatic stream serialization: the next launch of this engine may place its CTAs as
    // soon as SMs free up and set itself up; it reads or writes no global memory before the wait below.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta_rank = PAIR ? cluster_ctarank() : 0u;   // 0 = leader: issues the MMAs, owns full/tmem_empty
    const bool leader = cta_rank == 0;
    const int worker = PAIR ? blockIdx.x >> 1 : blockIdx.x;
    const int n_workers = PAIR ? gridDim.x >> 1 : gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar(s), 1);                // the leader's producer announces the bytes of both CTAs
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), PAIR ? 2 * kEpiWarps : kEpiWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const int tile0 = P.rounds > 0 ? scheduled_tile(P, worker, n_workers, 0) : -1;
        if (tile0 >= 0) {
            // warm the descriptors of the first tile while TMEM is allocated and the CTAs meet
            const DevProblem& Q0 = find_problem(P, tile0);
            prefetch_tensormap(&P.maps[Q0.map_a[0]]);
            prefetch_tensormap(&P.maps[Q0.map_b[0][cta_rank]]);
        }
    }
    if (warp == 1) {
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)), "r"(kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)), "r"(kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();     // the peer's barriers are initialised before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    // everything earlier in the stream has completed and its writes are visible after this
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp == 0) {
        // ------------------------------------------------------------------ producer (both CTAs of a pair)
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int round = 0; ok && round < P.rounds; ++round) {
                const int tile = scheduled_tile(P, worker, n_workers, round);
                if (tile < 0) continue;
                const DevProblem& Q = find_problem(P, tile);
                const int local = tile - Q.tile_start;
                const int m0 = (local % Q.tiles_m) * kTileM + static_cast<int>(cta_rank) * BM;
                const int n0 = (local / Q.tiles_m) * Q.n_per_tile;
                // a stage carries up to kSub k-blocks of one K segment
                for (int seg = 0; ok && seg < kMaxSeg; ++seg) {
                const int kb_lo = seg ? Q.kb_end[seg - 1] : 0, kb_hi = Q.kb_end[seg];
                for (int kb0 = kb_lo; kb0 < kb_hi; kb0 += kSub) {
                    const int nsub = min(kSub, kb_hi - kb0);
                    if (!(ok = mbar_wait<PAIR>(empty_bar(stage), phase ^ 1u, abort_flag, 1, P.status, P.wait_limit_ns))) break;
                    // "big" operands arrive as one box holding both k-blocks (zero-filled past the end of K)
                    const bool a_big = PAIR && Q.a_big[seg], b_big = PAIR && Q.b_big[seg];
                    const uint32_t tx = (a_big ? kSub : nsub) * kAStage + (b_big ? kSub : nsub) * kBLocal;
                    if (PAIR) {
                        if (leader) mbar_expect_tx(full_bar(stage), 2 * tx);   // both CTAs' bytes
                    } else {
                        mbar_expect_tx(full_bar(stage), tx);
                    }
                    if (PAIR && (a_big || b_big)) {
                        const int k0 = (kb0 - kb_lo) * BK + Q.k_off[seg];
                        const uint32_t fb = map_to_cta(full_bar(stage), 0);
                        if (a_big) {
                            const uint32_t dst = sA + stage * kSub * kAStage;
                            const CUtensorMap* ma = &P.maps[Q.map_a[seg]];
                            if (!Q.a_mn[seg]) {           // (64 k, 128 rows, 2 k-blocks)
                                if (leader) tma_load_3d(dst, ma, 0, m0, k0 >> 6, full_bar(stage));
                                else tma_load_3d_pair(dst, ma, 0, m0, k0 >> 6, fb);
                            } else {                      // (64 m, 64 k, 2 atoms, 2 k-blocks)
                                if (leader) tma_load_4d(dst, ma, 0, m0 >> 6, k0 >> 6, full_bar(stage));
                                else tma_load_4d_pair(dst, ma, 0, m0 >> 6, k0 >> 6, fb);
                            }
                        }
                        if (b_big) {
                            const uint32_t dst = sB + stage * kSub * kBLocal;
                            const CUtensorMap* mb = &P.maps[Q.map_b[seg][cta_rank]];
                            const int nc = n0 + static_cast<int>(cta_rank) * Q.half1_n_off;
                            if (!Q.b_mn[seg]) {
                                if (leader) tma_load_3d(dst, mb, 0, nc, k0 >> 6, full_bar(stage));
                                else tma_load_3d_pair(dst, mb, 0, nc, k0 >> 6, fb);
                            } else {
                                if (leader) tma_load_4d(dst, mb, 0, nc >> 6, k0 >> 6, full_bar(stage));
                                else tma_load_4d_pair(dst, mb, 0, nc >> 6, k0 >> 6, fb);
                            }
                        }
                    }
#pragma unroll
                    for (int sub = 0; sub < kSub; ++sub) {
                    if (sub >= nsub) break;
                    const int kb = kb0 + sub;
                    const int k0 = (kb - kb_lo) * BK + Q.k_off[seg];
                    const uint32_t a_dst = sA + (stage * kSub + sub) * kAStage, b_dst = sB + (stage * kSub + sub) * kBLocal;
                    const CUtensorMap* ma = &P.maps[Q.map_a[seg]];
                    if (PAIR) {
                        // This CTA's share of the stage, completed on the leader's barrier: the leader uses the
                        // plain form on its own barrier (measurably cheaper), the peer the pair form that may
                        // signal the other CTA's barrier.
                        const uint32_t fb = map_to_cta(full_bar(stage), 0);
                        auto load = [&](uint32_t dst, const CUtensorMap* map, int x, int y) {
                            if (leader) tma_load_2d(dst, map, x, y, full_bar(stage));
                            else tma_load_2d_pair(dst, map, x, y, fb);
                        };
                        auto load3 = [&](uint32_t dst, const CUtensorMap* map, int y, int z) {
                            if (leader) tma_load_3d(dst, map, 0, y, z, full_bar(stage));
                            else tma_load_3d_pair(dst, map, 0, y, z, fb);
                        };
                        if (a_big) {
                        } else if (!Q.a_mn[seg]) {
                            load(a_dst, ma, k0, m0);
                        } else if (Q.a_3d[seg]) {
                            load3(a_dst, ma, k0, m0 >> 6);
                        } else {
                            load(a_dst, ma, m0, k0);
                            load(a_dst + kAtomBytes, ma, m0 + 64, k0);
                        }
                        const CUtensorMap* mb = &P.maps[Q.map_b[seg][cta_rank]];
                        const int nc = n0 + static_cast<int>(cta_rank) * Q.half1_n_off;
                        if (b_big) {
                        } else if (!Q.b_mn[seg]) {
                            load(b_dst, mb, k0, nc);
                        } else if (Q.b_3d[seg]) {
                            load3(b_dst, mb, k0, nc >> 6);
                        } else {
                            load(b_dst, mb, nc, k0);
                            load(b_dst + kAtomBytes, mb, nc + 64, k0);
                        }
                    } else {
                        if (!Q.a_mn[seg]) {
                            tma_load_2d(a_dst, ma, k0, m0, full_bar(stage));                    // box 64(k) x 128(m)
                        } else if (Q.a_3d[seg]) {
                            tma_load_3d(a_dst, ma, 0, k0, m0 >> 6, full_bar(stage));            // box 64 x 64(k) x 2 atoms
                        } else {
                            tma_load_2d(a_dst, ma, m0, k0, full_bar(stage));                    // box 64(m) x 64(k)
                            tma_load_2d(a_dst + kAtomBytes, ma, m0 + 64, k0, full_bar(stage));
                        }
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const CUtensorMap* mb = &P.maps[Q.map_b[seg][h]];
                            const int nc = n0 + h * Q.half1_n_off;
                            const uint32_t dst = b_dst + h * kBHalf;
                            if (!Q.b_mn[seg]) {
                                tma_load_2d(dst, mb, k0, nc, full_bar(stage));                  // box 64(k) x 128(n)
                            } else if (Q.b_3d[seg]) {
                                tma_load_3d(dst, mb, 0, k0, nc >> 6, full_bar(stage));
                            } else {
                                tma_load_2d(dst, mb, nc, k0, full_bar(stage));                  // box 64(n) x 64(k)
                                tma_load_2d(dst + kAtomBytes, mb, nc + 64, k0, full_bar(stage));
                            }
                        }
                    }
                    }   // sub
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }   // kb0
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && leader) {
            int stage = 0;
            uint32_t phase = 0;
            int it = 0;
            bool ok = true;
            for (int round = 0; ok && round < P.rounds; ++round) {
                const int tile = scheduled_tile(P, worker, n_workers, round);
                if (tile < 0) continue;
                const DevProblem& Q = find_problem(P, tile);
                const int acc = it & 1;
                const uint32_t acc_phase = (it >> 1) & 1u;
                if (!(ok = mbar_wait<PAIR>(tempty_bar(acc), acc_phase ^ 1u, abort_flag, 2, P.status, P.wait_limit_ns))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int seg = 0; ok && seg < kMaxSeg; ++seg) {
                const int kb_lo = seg ? Q.kb_end[seg - 1] : 0, kb_hi = Q.kb_end[seg];
                for (int kb0 = kb_lo; kb0 < kb_hi; kb0 += kSub) {
                    const int nsub = min(kSub, kb_hi - kb0);
                    if (!(ok = mbar_wait<PAIR>(full_bar(stage), phase, abort_flag, 3, P.status, P.wait_limit_ns))) break;
                    tc_fence_after();
#pragma unroll
                    for (int sub = 0; sub < kSub; ++sub) {
                        if (sub >= nsub) break;
                        const int kb = kb0 + sub;
                        const uint32_t a_mn = Q.a_mn[seg], b_mn = Q.b_mn[seg];
                        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (a_mn << 15) | (b_mn << 16) |
                                               (static_cast<uint32_t>(BN >> 3) << 17) | (static_cast<uint32_t>(kTileM >> 4) << 24);
                        const uint64_t a_desc = make_smem_desc(sA + (stage * kSub + sub) * kAStage, a_mn ? kAtomBytes : 16, 1024);
                        const uint64_t b_desc = make_smem_desc(sB + (stage * kSub + sub) * kBLocal, b_mn ? kAtomBytes : 16, 1024);
                        const uint64_t a_step = a_mn ? (2048 >> 4) : (32 >> 4);   // per 16 k: two 8-row groups, or 32 bytes
                        const uint64_t b_step = b_mn ? (2048 >> 4) : (32 >> 4);
#pragma unroll
                        for (int ks = 0; ks < BK / 16; ++ks) {
                            if (PAIR) tc_mma_bf16_pair(d_tmem, a_desc + ks * a_step, b_desc + ks * b_step, idesc, (kb | ks) != 0 ? 1u : 0u);
                            else tc_mma_bf16(d_tmem, a_desc + ks * a_step, b_desc + ks * b_step, idesc, (kb | ks) != 0 ? 1u : 0u);
                        }
                    }
                    // the stage is free (in both CTAs) once these MMAs have read it
                    if (PAIR) {
                        tc_commit_pair(map_to_cta(empty_bar(stage), 0));
                        tc_commit_pair(map_to_cta(empty_bar(stage), 1));
                    } else {
                        tc_commit(empty_bar(stage));
                    }
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                }   // seg
                if (ok) {                              // accumulator complete (in both CTAs)
                    if (PAIR) {
                        tc_commit_pair(map_to_cta(tfull_bar(acc), 0));
                        tc_commit_pair(map_to_cta(tfull_bar(acc), 1));
                    } else {
                        tc_commit(tfull_bar(acc));
                    }
                }
                ++it;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int ew = warp - 2;
        const int quad = warp & 3;            // TMEM lanes this warp may read: [32*quad, 32*quad + 32)
        const int half = ew >> 2;             // which half of the tile's columns
        const uint32_t buf_out = sEpi + ew * 2 * kEpiSlotBytes, buf_in = buf_out + kEpiSlotBytes;
        int it = 0;
        bool ok = true;
        for (int round = 0; ok && round < P.rounds; ++round) {
            const int tile = scheduled_tile(P, worker, n_workers, round);
            if (tile < 0) continue;
            const DevProblem& Q = find_problem(P, tile);
            const int local = tile - Q.tile_start;
            const int m_warp = (local % Q.tiles_m) * kTileM + static_cast<int>(cta_rank) * BM + quad * 32;   // first row of this warp
            const int n0 = (local / Q.tiles_m) * Q.n_per_tile;
            const int acc = it & 1;
            const uint32_t acc_phase = (it >> 1) & 1u;
            const int epi = Q.epi;
            const int QM = Q.M, QN = Q.N;
            const CUtensorMap* mc0 = &P.maps[Q.map_c[0]];
            const CUtensorMap* mc1 = &P.maps[Q.map_c[1]];
            const CUtensorMap* mc2 = &P.maps[Q.map_c[2]];
            // saved activations of the derivative epilogues: first chunk requested before the accumulator is ready
            const bool need_h = epi >= EPI_DGELU_ERF;
            const bool need_hb = epi == EPI_DSWIGLU;
            const unsigned short* Hp = static_cast<const unsigned short*>(Q.H);
            const unsigned short* Hbp = static_cast<const unsigned short*>(Q.Hb);
            uint4 hq[4], hbq[4];
            if (need_h) staged_load32_issue(Hp, Q.ldh, m_warp, n0 + half * 128, QM, QN, hq, lane);
            if (need_hb) staged_load32_issue(Hbp, Q.ldh, m_warp, n0 + half * 128, QM, QN, hbq, lane);
            // the second slot doubles as the landing buffer of those loads: no store of an earlier tile may still read it
            if (need_h) stage_begin<0>(lane);
            // bias of this warp's 128 columns, one column per lane and 32-column chunk (fetched while the tile is computed)
            float breg[4] = {0.f, 0.f, 0.f, 0.f};
            const bool has_bias = Q.bias != nullptr;
            if (has_bias) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int col = n0 + half * 128 + 32 * j + lane;
                    if (col < QN)
                        breg[j] = Q.bias_f32 ? static_cast<const float*>(Q.bias)[col]
                                             : __uint_as_float(static_cast<uint32_t>(static_cast<const unsigned short*>(Q.bias)[col]) << 16);
                }
            }
            if (!(ok = mbar_wait<PAIR>(tfull_bar(acc), acc_phase, abort_flag, 4, P.status, P.wait_limit_ns))) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + acc * BN + (static_cast<uint32_t>(quad * 32) << 16);
            const bool warp_rows = m_warp < QM;          // any row of this warp inside the output
            if (epi == EPI_SWIGLU) {
                // accumulator columns [0,128) = gate, [128,256) = up for hidden units n0 .. n0+127.
                // The three outputs of a chunk alternate between the two slots, one store may stay in flight.
                int slot = 0;
                bool fresh = true;
                auto put = [&](const CUtensorMap* map, int n, const float (&v)[32]) {
                    if (fresh) stage_begin<0>(lane); else stage_begin<1>(lane);
                    fresh = false;
                    const uint32_t sb = buf_out + slot * kEpiSlotBytes;
                    stage_bf16x32(sb, lane, v);
                    stage_commit(map, sb, n, m_warp, lane);
                    slot ^= 1;
                };
#pragma unroll 1
                for (int c = 0; c < 2; ++c) {
                    const int hc = half * 64 + c * 32;
                    uint32_t rg[32], ru[32];
                    tc_ld32(t_row + hc, rg);
                    tc_ld32(t_row + 128 + hc, ru);
                    tc_wait_ld();
                    const int n = n0 + hc;
                    if (n >= QN || !warp_rows) continue;
                    float g[32], u[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        g[i] = __uint_as_float(rg[i]);
                        u[i] = __uint_as_float(ru[i]);
                    }
                    put(mc0, n, g);
                    put(mc1, n, u);
#pragma unroll
                    for (int i = 0; i < 32; ++i) g[i] = g[i] * sigmoidf_(g[i]) * u[i];
                    put(mc2, n, g);
                }
            } else if (epi == EPI_STORE && !Q.out_f32) {
                // bf16 output: two chunks of 64 columns, each one 32 x 128-byte image
#pragma unroll 1
                for (int c = 0; c < 2; ++c) {
                    const int col = half * 128 + c * 64;
                    uint32_t r0[32], r1[32];
                    tc_ld32(t_row + col, r0);
                    tc_ld32(t_row + col + 32, r1);
                    tc_wait_ld();
                    const int n = n0 + col;
                    if (n >= QN || !warp_rows) continue;
                    float v0[32], v1[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        v0[i] = __uint_as_float(r0[i]);
                        v1[i] = __uint_as_float(r1[i]);
                    }
                    if (has_bias) {
                        add_bias32(v0, c ? breg[2] : breg[0]);
                        add_bias32(v1, c ? breg[3] : breg[1]);
                    }
                    stage_begin<0>(lane);
                    stage_bf16x64(buf_out, lane, v0, v1);
                    stage_commit(mc0, buf_out, n, m_warp, lane, Q.accumulate != 0);
                }
            } else if (epi == EPI_GELU_ERF || epi == EPI_GELU_TANH) {
                // H = acc + bias and A = GELU(H), 64 columns at a time
#pragma unroll 1
                for (int c = 0; c < 2; ++c) {
                    const int col = half * 128 + c * 64;
                    uint32_t r0[32], r1[32];
                    tc_ld32(t_row + col, r0);
                    tc_ld32(t_row + col + 32, r1);
                    tc_wait_ld();
                    const int n = n0 + col;
                    if (n >= QN || !warp_rows) continue;
                    float v0[32], v1[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        v0[i] = __uint_as_float(r0[i]);
                        v1[i] = __uint_as_float(r1[i]);
                    }
                    if (has_bias) {
                        add_bias32(v0, c ? breg[2] : breg[0]);
                        add_bias32(v1, c ? breg[3] : breg[1]);
                    }
                    stage_begin<0>(lane);
                    stage_bf16x64(buf_out, lane, v0, v1);
                    stage_commit(mc0, buf_out, n, m_warp, lane);
                    if (epi == EPI_GELU_ERF) {
                        gelu_erf32(v0);
                        gelu_erf32(v1);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            v0[i] = gelu_tanh(v0[i]);
                            v1[i] = gelu_tanh(v1[i]);
                        }
                    }
                    stage_begin<0>(lane);
                    stage_bf16x64(buf_out, lane, v0, v1);
                    stage_commit(mc1, buf_out, n, m_warp, lane);
                }
            } else {
                // 32 columns at a time: fp32 outputs and the derivative epilogues
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    const int col = half * 128 + c * 32;
                    uint32_t r[32];
                    tc_ld32(t_row + col, r);
                    tc_wait_ld();
                    const int n = n0 + col;
                    const int nv = min(32, QN - n);
                    if (nv <= 0) continue;
                    float v[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
                    if (has_bias) add_bias32(v, c == 0 ? breg[0] : c == 1 ? breg[1] : c == 2 ? breg[2] : breg[3]);
                    if (epi == EPI_STORE) {                // fp32 output: one 32 x 128-byte image
                        if (warp_rows) {
                            stage_begin<0>(lane);
                            stage_f32x32(buf_out, lane, v);
                            stage_commit(mc0, buf_out, n, m_warp, lane, Q.accumulate != 0);
                        }
                    } else if (epi == EPI_DGELU_ERF || epi == EPI_DGELU_TANH) {
                        float h[32];
                        staged_load32_finish(buf_in, hq, h, lane);
                        if (c < 3) staged_load32_issue(Hp, Q.ldh, m_warp, n + 32, QM, QN, hq, lane);
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (epi != EPI_DGELU_ERF) v[i] *= dgelu_tanh(h[i]);
                        if (epi == EPI_DGELU_ERF) dgelu_erf32(v, h);
                        if (warp_rows) {
                            stage_begin<0>(lane);
                            stage_bf16x32(buf_out, lane, v);
                            stage_commit(mc0, buf_out, n, m_warp, lane);
                        }
                    } else {  // EPI_DSWIGLU
                        float hg[32], hu[32];
                        staged_load32_finish(buf_in, hq, hg, lane);
                        staged_load32_finish(buf_in, hbq, hu, lane);
                        if (c < 3) {
                            staged_load32_issue(Hp, Q.ldh, m_warp, n + 32, QM, QN, hq, lane);
                            staged_load32_issue(Hbp, Q.ldh, m_warp, n + 32, QM, QN, hbq, lane);
                        }
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const float s = sigmoidf_(hg[i]);
                            hu[i] = v[i] * hu[i] * s * (1.f + hg[i] * (1.f - s));   // dH_gate
                            v[i] = v[i] * hg[i] * s;                                // dH_up
                        }
                        if (warp_rows) {
                            stage_begin<0>(lane);
                            stage_bf16x32(buf_out, lane, hu);
                            stage_commit(mc0, buf_out, n, m_warp, lane);
                            stage_begin<0>(lane);
                            stage_bf16x32(buf_out, lane, v);
                            stage_commit(mc1, buf_out, n, m_warp, lane);
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {                       // the accumulator may be overwritten: tell the MMA issuer
                if (PAIR) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));
                else mbar_arrive(tempty_bar(acc));
            }
            ++it;
        }
        if (lane == 0) bulk_wait_all();            // this warp's tile stores have landed
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    if (*abort_flag) {
        // give copies that are still in flight time to land before the shared memory is released
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();     // neither CTA leaves while the other may still signal its barriers
    if (warp == 1) {
        tc_fence_after();
        if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn get_encode() {
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

// MN-major operand whose row length is a multiple of 64: the matrix [K][MN] viewed as (64, K, MN/64) with strides
// (2 B, pitch, 128 B), so that one box of 64 x 64 x 2 brings both 64-wide swizzle atoms of a 128-wide slab
// in the atom-major order the MMA descriptor expects.  Returns false when the view cannot be encoded.
bool encode_map_mn3d(CUtensorMap* out, const Stored& s) {
    EncodeFn enc = get_encode();
    if (!enc || !s.ptr || s.cols % 64 != 0 || !aligned16(s.ptr) || (s.ld * 2) % 16 != 0) return false;
    const cuuint64_t dims[3] = {64, static_cast<cuuint64_t>(s.rows), static_cast<cuuint64_t>(s.cols / 64)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(s.ld) * 2, 128};
    const cuuint32_t box[3] = {64, 64, 2};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(s.ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Pair mode, one box per operand per stage (two 64-deep k-blocks), when the extents are multiples of 64:
//   K-major  [rows][K]  viewed as (64, rows, K/64)          box 64 x 128 x 2        -> [k-block][row][64 k]
//   MN-major [K][MN]    viewed as (64, 64, MN/64, K/64)     box 64 x 64 x 2 x 2     -> [k-block][atom][k][64 mn]
// Both orders are exactly two consecutive k-block images of the per-k-block layout.
bool encode_map_big(CUtensorMap* out, const Stored& s, bool mn) {
    EncodeFn enc = get_encode();
    if (!enc || !s.ptr || s.cols % 64 != 0 || !aligned16(s.ptr) || (s.ld * 2) % 16 != 0) return false;
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    if (!mn) {
        const cuuint64_t dims[3] = {64, static_cast<cuuint64_t>(s.rows), static_cast<cuuint64_t>(s.cols / 64)};
        const cuuint64_t strides[2] = {static_cast<cuuint64_t>(s.ld) * 2, 128};
        const cuuint32_t box[3] = {64, 128, 2};
        return enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(s.ptr), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    }
    if (s.rows % 64 != 0) return false;
    const cuuint64_t dims[4] = {64, 64, static_cast<cuuint64_t>(s.cols / 64), static_cast<cuuint64_t>(s.rows / 64)};
    const cuuint64_t strides[3] = {static_cast<cuuint64_t>(s.ld) * 2, 128, static_cast<cuuint64_t>(s.ld) * 128};
    const cuuint32_t box[4] = {64, 64, 2, 2};
    return enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(s.ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map of a stored row-major bf16 matrix; box = 64 elements along the row x box_rows rows
// (128-byte swizzle, operand loads), or 32 x 32 with the 64-byte swizzle (epilogue stores).
ecospa_status_t encode_map(CUtensorMap* out, const Stored& s, int box_rows, bool store_box = false) {
    EncodeFn enc = get_encode();
    if (!enc) {
        set_cuda_error(cudaErrorNotSupported, "cuTensorMapEncodeTiled entry point");
        return ECOSPA_ERR_CUDA;
    }
    if (!s.ptr || s.rows < 1 || s.cols < 1 || s.ld < s.cols) return ECOSPA_ERR_INVALID;
    if (!aligned16(s.ptr) || (s.ld * 2) % 16 != 0) return ECOSPA_ERR_ALIGNMENT;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(s.cols), static_cast<cuuint64_t>(s.rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(s.ld) * 2};
    const cuuint32_t box[2] = {store_box ? 32u : 64u, static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(s.ptr), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, store_box ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
        return ECOSPA_ERR_CUDA;
    }
    return ECOSPA_OK;
}

// Store map of an output (rows x cols, pitch ld elements): boxes of 32 rows x 64 bf16 or 32 fp32 columns
// (128-byte swizzle) or 32 rows x 32 bf16 columns (64-byte swizzle), matching the staging images.
ecospa_status_t encode_out_map(CUtensorMap* out, void* ptr, int64_t rows, int64_t cols, int64_t ld, bool f32, bool wide) {
    EncodeFn enc = get_encode();
    if (!enc) {
        set_cuda_error(cudaErrorNotSupported, "cuTensorMapEncodeTiled entry point");
        return ECOSPA_ERR_CUDA;
    }
    const int eb = f32 ? 4 : 2;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * eb};
    const cuuint32_t box[2] = {(f32 || !wide) ? 32u : 64u, 32u};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(out, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ptr, dims, strides, box,
                           estr, CU_TENSOR_MAP_INTERLEAVE_NONE, (f32 || wide) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                           CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled (output)");
        return ECOSPA_ERR_CUDA;
    }
    return ECOSPA_OK;
}

// Per-device facts of the engine, looked up the first time a device is used (with that device current).
constexpr int kMaxDevices = 64;
struct DeviceState {
    std::once_flag once;
    ecospa_status_t st = ECOSPA_OK;
    int num_sms = 0;
    int max_pairs = 0;      // CTA pairs that can be resident at once (clusters must fit inside a GPC)
    int* status_ptr = nullptr;   // this device's copy of g_gemm_status
};
DeviceState g_dev[kMaxDevices];
int g_pair_mode = 1;   // 1: CTA pairs (cta_group::2) whenever an op has more than one 128-row tile; 0: never
std::atomic<unsigned long long> g_wait_limit_ns{kDefaultWaitLimitNs};

// State of the current device (set up on first use), or nullptr with *st set.
DeviceState* gemm_setup(ecospa_status_t* st_out) {
    int dev = 0;
    cudaError_t e0 = cudaGetDevice(&dev);
    if (e0 != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        if (e0 != cudaSuccess) {
            set_cuda_error(e0, "gemm setup (cudaGetDevice)");
            cudaGetLastError();
        }
        *st_out = e0 != cudaSuccess ? ECOSPA_ERR_CUDA : ECOSPA_ERR_UNSUPPORTED;
        return nullptr;
    }
    DeviceState& D = g_dev[dev];
    std::call_once(D.once, [&D, dev] {
        cudaError_t e = cudaDeviceGetAttribute(&D.num_sms, cudaDevAttrMultiProcessorCount, dev);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (const char* v = std::getenv("ECOSPA_GEMM_PAIR")) g_pair_mode = std::atoi(v);
        if (e == cudaSuccess) {
            // the tile schedule is static, so only as many pairs as can run at the same time are launched
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(2 * (D.num_sms / 2));
            cfg.blockDim = dim3(kThreads);
            cfg.dynamicSmemBytes = kSmemBytes;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 2;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, gemm_kernel<true>, &cfg) == cudaSuccess && n > 0) D.max_pairs = n;
            else cudaGetLastError();
        }
        if (e == cudaSuccess) e = cudaGetSymbolAddress(reinterpret_cast<void**>(&D.status_ptr), g_gemm_status);
        if (e != cudaSuccess) {
            set_cuda_error(e, "gemm setup");
            cudaGetLastError();
            D.st = ECOSPA_ERR_CUDA;
        }
    });
    *st_out = D.st;
    return D.st == ECOSPA_OK ? &D : nullptr;
}

// Tile schedule.  Tiles are numbered op by op, longest contraction first.  With few tiles per worker the
// plain stride (worker w takes w, w + workers, ...) can leave one worker with several long tiles, so the
// tiles are handed out longest first to the least-loaded worker (ties: lowest worker) and the result is
// written as a table; with many tiles per worker the stride is balanced enough and needs no table.
void build_schedule(GemmParams& gp, int workers) {
    const int tiles = gp.total_tiles;
    gp.use_order = 0;
    gp.rounds = static_cast<int32_t>(ceil_div(tiles, workers));
    if (tiles <= workers || tiles > kMaxOrder || tiles >= kNoTile) return;
    static thread_local int64_t load[256];
    static thread_local int32_t len[256];
    static thread_local uint16_t lists[256][64];
    if (workers > 256) return;
    for (int w = 0; w < workers; ++w) load[w] = len[w] = 0;
    int max_len = 0;
    int pi = 0;
    for (int t = 0; t < tiles; ++t) {
        while (pi + 1 < gp.n_problems && gp.prob[pi + 1].tile_start <= t) ++pi;
        // main loop, or the epilogue where that is the longer of the two (measured, in k-block times), + a fixed share
        static const int kEpiCost[7] = {5, 14, 14, 16, 20, 20, 26};
        const int64_t cost = std::max<int64_t>(gp.prob[pi].kblocks, kEpiCost[gp.prob[pi].epi]) + 4;
        int best = 0;
        for (int w = 1; w < workers; ++w)
            if (load[w] < load[best]) best = w;
        if (len[best] >= 64) return;                       // not expected; keep the stride
        lists[best][len[best]++] = static_cast<uint16_t>(t);
        load[best] += cost;
        max_len = std::max(max_len, static_cast<int>(len[best]));
    }
    if (static_cast<int64_t>(max_len) * workers > kMaxOrder) return;
    for (int i = 0; i < max_len; ++i)
        for (int w = 0; w < workers; ++w) gp.order[w + i * workers] = i < len[w] ? lists[w][i] : kNoTile;
    gp.rounds = max_len;
    gp.use_order = 1;
}

}  // namespace

// Host-only checks of a launch (no CUDA call): shapes, pointers, 16-byte alignment of every base and pitch.
ecospa_status_t validate_gemm_ops(const GemmOp* ops, int n_ops) {
    if (!ops || n_ops < 1 || n_ops > kMaxGemmOps) return ECOSPA_ERR_INVALID;
    for (int i = 0; i < n_ops; ++i) {
        const GemmOp& op = ops[i];
        if (op.M < 1 || op.N < 1 || op.n_kseg < 1 || op.n_kseg > kMaxSeg || !op.C || op.ldc < 1) return ECOSPA_ERR_INVALID;
        if (op.M > INT32_MAX || op.N > INT32_MAX) return ECOSPA_ERR_INVALID;
        if (op.epi < EPI_STORE || op.epi > EPI_DSWIGLU) return ECOSPA_ERR_INVALID;
        const int out_eb = op.out_f32 ? 4 : 2;
        if (!aligned16(op.C) || (op.ldc * out_eb) % 16) return ECOSPA_ERR_ALIGNMENT;
        if (op.ldc < op.N) return ECOSPA_ERR_INVALID;
        if (op.bias && !aligned16(op.bias)) return ECOSPA_ERR_ALIGNMENT;
        for (int s = 0; s < op.n_kseg; ++s) {
            const KSegment& ks = op.seg[s];
            if (ks.K < 1 || ks.k_begin < 0 || ks.k_begin % BK) return ECOSPA_ERR_INVALID;
            const Stored* mats[3] = {&ks.a, &ks.b[0], op.epi == EPI_SWIGLU ? &ks.b[1] : nullptr};
            for (const Stored* m : mats) {
                if (!m) continue;
                if (!m->ptr || m->rows < 1 || m->cols < 1 || m->ld < m->cols) return ECOSPA_ERR_INVALID;
                if (!aligned16(m->ptr) || (m->ld * 2) % 16) return ECOSPA_ERR_ALIGNMENT;
            }
        }
    }
    return ECOSPA_OK;
}

ecospa_status_t launch_grouped_gemm(const GemmOp* ops, int n_ops, cudaStream_t stream) {
    ecospa_status_t st = validate_gemm_ops(ops, n_ops);
    if (st != ECOSPA_OK) return st;
    DeviceState* dev = gemm_setup(&st);
    if (!dev) return st;
    const int g_max_pairs = dev->max_pairs, g_num_sms = dev->num_sms;

    // longest contraction first
    int order[kMaxGemmOps];
    int64_t ktot[kMaxGemmOps];
    for (int i = 0; i < n_ops; ++i) {
        order[i] = i;
        ktot[i] = 0;
        for (int s = 0; s < ops[i].n_kseg; ++s) ktot[i] += ceil_div(ops[i].seg[s].K, BK);
    }
    std::stable_sort(order, order + n_ops, [&](int a, int b) { return ktot[a] > ktot[b]; });

    // CTA pairs pay off as soon as there is more than one 128-row tile to share a B tile between
    bool pair = g_pair_mode != 0 && g_max_pairs >= 1;
    if (pair) {
        bool any_tall = false;
        for (int i = 0; i < n_ops; ++i) any_tall = any_tall || ops[i].M > BM;
        pair = any_tall;
    }
    const int tile_m = pair ? 2 * BM : BM;

    static thread_local GemmParams gp;
    int tiles = 0;
    for (int oi = 0; oi < n_ops; ++oi) {
        const GemmOp& op = ops[order[oi]];
        DevProblem& Q = gp.prob[oi];
        std::memset(&Q, 0, sizeof(Q));
        if (op.M < 1 || op.N < 1 || op.n_kseg < 1 || op.n_kseg > kMaxSeg || !op.C || op.ldc < 1) return ECOSPA_ERR_INVALID;
        if (op.M > INT32_MAX || op.N > INT32_MAX) return ECOSPA_ERR_INVALID;
        const bool swiglu = op.epi == EPI_SWIGLU;
        const int out_eb = op.out_f32 ? 4 : 2;
        if (!aligned16(op.C) || (op.ldc * out_eb) % 16) return ECOSPA_ERR_ALIGNMENT;
        if ((op.epi == EPI_GELU_ERF || op.epi == EPI_GELU_TANH || op.epi == EPI_DSWIGLU || swiglu) && (!op.C2 || !aligned16(op.C2)))
            return op.C2 ? ECOSPA_ERR_ALIGNMENT : ECOSPA_ERR_INVALID;
        if (swiglu && (!op.C3 || !aligned16(op.C3))) return op.C3 ? ECOSPA_ERR_ALIGNMENT : ECOSPA_ERR_INVALID;
        if (op.epi >= EPI_DGELU_ERF) {
            if (!op.H || (op.epi == EPI_DSWIGLU && !op.Hb)) return ECOSPA_ERR_INVALID;
            if (!aligned16(op.H) || (op.Hb && !aligned16(op.Hb)) || (op.ldh * 2) % 16) return ECOSPA_ERR_ALIGNMENT;
        }
        if (op.out_f32 && op.epi != EPI_STORE) return ECOSPA_ERR_UNSUPPORTED;
        if (op.bias && !aligned16(op.bias)) return ECOSPA_ERR_ALIGNMENT;
        Q.M = static_cast<int32_t>(op.M);
        Q.N = static_cast<int32_t>(op.N);
        Q.n_per_tile = swiglu ? 128 : BN;
        Q.half1_n_off = swiglu ? 0 : 128;
        Q.epi = op.epi;
        Q.out_f32 = op.out_f32;
        Q.accumulate = op.accumulate;
        Q.bias_f32 = op.bias_f32;
        Q.C = op.C; Q.C2 = op.C2; Q.C3 = op.C3;
        Q.bias = op.bias; Q.H = op.H; Q.Hb = op.Hb;
        Q.ldc = op.ldc; Q.ldh = op.ldh;
        for (int s = 0; s < op.n_kseg; ++s) {
            const KSegment& ks = op.seg[s];
            if (ks.K < 1 || ks.k_begin < 0 || ks.k_begin % BK) return ECOSPA_ERR_INVALID;
            // stored shapes must cover the logical (M, N, [k_begin, k_begin + K))
            const int64_t k_end = ks.k_begin + ks.K;
            const Stored& a = ks.a;
            // a range that stops before the end of the stored tensor must end on a k-block boundary
            if (k_end < (ks.a_mn ? a.rows : a.cols) && ks.K % BK) return ECOSPA_ERR_INVALID;
            if (ks.a_mn ? (a.rows < k_end || a.cols != op.M) : (a.rows != op.M || a.cols < k_end)) return ECOSPA_ERR_INVALID;
            const int mi = oi * kMapsPerOp;
            Q.a_big[s] = pair && encode_map_big(&gp.maps[mi + 3 * s], a, ks.a_mn);
            Q.a_3d[s] = !Q.a_big[s] && ks.a_mn && encode_map_mn3d(&gp.maps[mi + 3 * s], a);
            if (!Q.a_big[s] && !Q.a_3d[s] && (st = encode_map(&gp.maps[mi + 3 * s], a, ks.a_mn ? 64 : 128)) != ECOSPA_OK) return st;
            Q.map_a[s] = static_cast<uint8_t>(mi + 3 * s);
            for (int h = 0; h < 2; ++h) {
                const Stored& b = (swiglu && h == 1) ? ks.b[1] : ks.b[0];
                if (ks.b_mn ? (b.rows < k_end || b.cols != op.N) : (b.rows != op.N || b.cols < k_end)) return ECOSPA_ERR_INVALID;
                const bool bb = pair && encode_map_big(&gp.maps[mi + 3 * s + 1 + h], b, ks.b_mn);
                const bool b3 = !bb && ks.b_mn && encode_map_mn3d(&gp.maps[mi + 3 * s + 1 + h], b);
                if (h == 0) {
                    Q.b_big[s] = bb;
                    Q.b_3d[s] = b3;
                } else if (bb != (Q.b_big[s] != 0) || b3 != (Q.b_3d[s] != 0)) {
                    return ECOSPA_ERR_UNSUPPORTED;   // both halves take the same path
                }
                if (!bb && !b3 && (st = encode_map(&gp.maps[mi + 3 * s + 1 + h], b, ks.b_mn ? 64 : 128)) != ECOSPA_OK) return st;
                Q.map_b[s][h] = static_cast<uint8_t>(mi + 3 * s + 1 + h);
            }
            Q.a_mn[s] = ks.a_mn;
            Q.b_mn[s] = ks.b_mn;
            Q.k_off[s] = static_cast<int32_t>(ks.k_begin);
            Q.kblocks += static_cast<int32_t>(ceil_div(ks.K, BK));
            Q.kb_end[s] = Q.kblocks;
        }
        // outputs leave through TMA tile stores (a reducing store when they are added to what C holds)
        {
            const bool wide = op.epi == EPI_STORE || op.epi == EPI_GELU_ERF || op.epi == EPI_GELU_TANH;
            void* outs[3] = {op.C, op.C2, op.C3};
            for (int o = 0; o < 3; ++o) {
                Q.map_c[o] = static_cast<uint8_t>(oi * kMapsPerOp + kOperandMaps + o);
                if (!outs[o]) continue;
                if ((st = encode_out_map(&gp.maps[Q.map_c[o]], outs[o], op.M, op.N, op.ldc, op.out_f32, wide)) != ECOSPA_OK) return st;
            }
        }
        for (int s2 = op.n_kseg; s2 < kMaxSeg; ++s2) Q.kb_end[s2] = Q.kblocks;
        Q.tiles_m = static_cast<int32_t>(ceil_div(op.M, tile_m));
        Q.tiles_n = static_cast<int32_t>(ceil_div(op.N, Q.n_per_tile));
        Q.tile_start = tiles;
        tiles += Q.tiles_m * Q.tiles_n;
    }
    gp.n_problems = n_ops;
    gp.total_tiles = tiles;
    gp.status = dev->status_ptr;
    gp.wait_limit_ns = g_wait_limit_ns.load(std::memory_order_relaxed);
    const int workers = pair ? std::min(tiles, g_max_pairs) : std::min(tiles, g_num_sms);
    build_schedule(gp, workers);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(pair ? 2 * workers : workers);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pair ? 2 : 1;
    const cudaError_t e = pair ? cudaLaunchKernelEx(&cfg, gemm_kernel<true>, gp) : cudaLaunchKernelEx(&cfg, gemm_kernel<false>, gp);
    if (e != cudaSuccess) {
        set_cuda_error(e, "gemm_kernel launch");
        cudaGetLastError();
        return ECOSPA_ERR_CUDA;
    }
    return check_launch("gemm_kernel");
}

int* engine_status_ptr(ecospa_status_t* st) {
    DeviceState* dev = gemm_setup(st);
    return dev ? dev->status_ptr : nullptr;
}
int engine_num_sms() {
    ecospa_status_t st;
    DeviceState* dev = gemm_setup(&st);
    return dev ? dev->num_sms : 0;
}
unsigned long long engine_wait_limit_ns() { return g_wait_limit_ns.load(std::memory_order_relaxed); }

int gemm_resident_pairs() {
    ecospa_status_t st;
    DeviceState* dev = gemm_setup(&st);
    if (!dev) return -1;
    return g_pair_mode ? dev->max_pairs : 0;
}

}  // namespace ecospa

extern "C" ecospa_status_t ecospa_device_status(void* stream, int32_t* code) {
    if (!code) return ECOSPA_ERR_INVALID;
    ecospa_status_t st;
    ecospa::DeviceState* dev = ecospa::gemm_setup(&st);
    if (!dev) return st;
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    int v = 0;
    if (e == cudaSuccess) e = cudaMemcpy(&v, dev->status_ptr, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) {
        ecospa::set_cuda_error(e, "ecospa_device_status");
        return ECOSPA_ERR_CUDA;
    }
    *code = v;
    if (v != 0) {
        cudaMemset(dev->status_ptr, 0, sizeof(int));
        return ECOSPA_ERR_TIMEOUT;
    }
    return ECOSPA_OK;
}

// Number of CTA pairs the GEMM engine runs at once on the current device (0 = pair mode off).
extern "C" int32_t ecospa_gemm_resident_pairs(void) { return ecospa::gemm_resident_pairs(); }

extern "C" ecospa_status_t ecospa_set_device_wait_limit_ns(uint64_t ns) {
    if (ns == 0) return ECOSPA_ERR_INVALID;
    ecospa::g_wait_limit_ns.store(ns, std::memory_order_relaxed);
    return ECOSPA_OK;
}
