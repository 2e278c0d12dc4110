// Shared device/host helpers of libecospa (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "ecospa.h"

namespace ecospa {

// Thread-local record of the last CUDA failure, for ecospa_last_cuda_error().
void set_cuda_error(cudaError_t e, const char* where);
ecospa_status_t check_launch(const char* where);

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline int64_t round_up(int64_t a, int64_t b) { return ceil_div(a, b) * b; }
inline int elem_bytes(int dtype) { return dtype == ECOSPA_F32 ? 4 : 2; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Extent (in elements) of the memory a tensor with shared dimension D touches.
inline int64_t mat_rows(const ecospa_mat_t& m, int64_t D) { return m.layout == ECOSPA_SHARED_COLS ? m.other_dim : D; }
inline int64_t mat_cols(const ecospa_mat_t& m, int64_t D) { return m.layout == ECOSPA_SHARED_COLS ? D : m.other_dim; }

#ifdef __CUDACC__

__device__ __forceinline__ uint4 ldg_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

template <typename T>
struct ElemTraits;
template <>
struct ElemTraits<float> {
    static constexpr int kVec = 4;  // elements per 16 bytes
    __device__ static __forceinline__ void unpack(const uint4& v, float (&f)[4]) {
        f[0] = __uint_as_float(v.x);
        f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z);
        f[3] = __uint_as_float(v.w);
    }
    __device__ static __forceinline__ float load1(const void* base, int64_t i) {
        return __ldg(static_cast<const float*>(base) + i);
    }
};
struct bf16_tag {};
template <>
struct ElemTraits<bf16_tag> {
    static constexpr int kVec = 8;
    __device__ static __forceinline__ void unpack(const uint4& v, float (&f)[8]) {
        f[0] = bf16_lo(v.x);
        f[1] = bf16_hi(v.x);
        f[2] = bf16_lo(v.y);
        f[3] = bf16_hi(v.y);
        f[4] = bf16_lo(v.z);
        f[5] = bf16_hi(v.z);
        f[6] = bf16_lo(v.w);
        f[7] = bf16_hi(v.w);
    }
    __device__ static __forceinline__ float load1(const void* base, int64_t i) {
        return __uint_as_float(static_cast<uint32_t>(__ldg(static_cast<const unsigned short*>(base) + i)) << 16);
    }
};

// Sum over a warp, fixed order.
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum over a block of NW warps; every thread gets the result.  `scratch` holds >= NW floats.
template <int NW>
__device__ __forceinline__ float block_sum(float v, float* scratch) {
    v = warp_sum(v);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) t += scratch[w];
    return t;
}

#endif  // __CUDACC__

}  // namespace ecospa
