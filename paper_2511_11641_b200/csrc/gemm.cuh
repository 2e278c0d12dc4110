// Internal interface of the grouped tcgen05 GEMM engine (see gemm.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "ecospa.h"

namespace ecospa {

// A bf16 row-major matrix as stored in memory.
struct Stored {
    const void* ptr = nullptr;
    int64_t rows = 0, cols = 0, ld = 0;
};

enum Epilogue : int {
    EPI_STORE = 0,        // C = acc (+ bias[n]) (+ C_old)
    EPI_GELU_ERF = 1,     // C = H = acc + bias, C2 = GELU(H)
    EPI_GELU_TANH = 2,
    EPI_SWIGLU = 3,       // acc = [gate | up] for 128 hidden units: C = H_gate, C2 = H_up, C3 = silu(gate) * up
    EPI_DGELU_ERF = 4,    // C = acc * GELU'(H)
    EPI_DGELU_TANH = 5,
    EPI_DSWIGLU = 6       // C = acc * H_up * silu'(H_gate), C2 = acc * silu(H_gate)
};

// One K segment of a contraction: C += A_seg * B_seg.
//   a_mn == false: A stored [M][K] (K-major);  true: stored [K][M].
//   b_mn == false: B stored [N][K] (K-major);  true: stored [K][N].
// b[1] is only used by EPI_SWIGLU (b[0] = gate weights, b[1] = up weights).
struct KSegment {
    Stored a;
    Stored b[2];
    bool a_mn = false, b_mn = false;
    int64_t K = 0;        // length of this segment's contraction
    int64_t k_begin = 0;  // first contraction index used (multiple of 64): lets several ops split one K range
};

struct GemmOp {
    int64_t M = 0, N = 0;     // output extent (EPI_SWIGLU: N = hidden units)
    int n_kseg = 1;           // 1..3 segments accumulated into the same output
    KSegment seg[3];
    int epi = EPI_STORE;
    void* C = nullptr;
    void* C2 = nullptr;
    void* C3 = nullptr;
    int64_t ldc = 0;          // pitch of C, C2, C3 (elements)
    bool out_f32 = false;     // C is fp32 (EPI_STORE only); otherwise bf16
    bool accumulate = false;  // EPI_STORE: add the previous contents of C
    const void* bias = nullptr;
    bool bias_f32 = false;
    const void* H = nullptr;  // saved pre-activations for the derivative epilogues (bf16)
    const void* Hb = nullptr;
    int64_t ldh = 0;
};

constexpr int kMaxGemmOps = 16;

// Enqueues one persistent launch that computes every op (tiles of the ops with the longest
// contraction are scheduled first).  Operands must be 16-byte aligned with 16-byte pitches.
ecospa_status_t launch_grouped_gemm(const GemmOp* ops, int n_ops, cudaStream_t stream);

// The host-only checks launch_grouped_gemm starts with (shapes, null pointers, 16-byte alignment of every base and
// pitch); makes no CUDA call.  Calls that enqueue several launches check all of them before the first.
ecospa_status_t validate_gemm_ops(const GemmOp* ops, int n_ops);

// What the other tensor-core kernels of the library share with the engine: the current device's status word (device
// pointer; nullptr with *st set when no device can be used), its SM count, and the limit of device-side waits.
int* engine_status_ptr(ecospa_status_t* st);
int engine_num_sms();
unsigned long long engine_wait_limit_ns();

// CTA pairs the engine keeps resident on the current device (0: pair mode off, -1: no usable device).
int gemm_resident_pairs();

}  // namespace ecospa
