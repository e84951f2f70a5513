// Shared host/device helpers of libmpq (CUDA side only).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "mpq.h"

namespace mpq {

constexpr int kMaxBits = 8;

__host__ __device__ inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Words per packed row: ceil(k/32) rounded up to 4 words (16 bytes).
__host__ __device__ inline int64_t row_words(int64_t k) { return ceil_div(ceil_div(k, 32), 4) * 4; }

inline bool bits_ok(int b) { return b >= 1 && b <= kMaxBits; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int launch_status() { return cudaGetLastError() == cudaSuccess ? MPQ_OK : MPQ_ERR_CUDA; }

// 1/s, or 0 when s is not a finite positive number (every code then becomes the level above zero).
__device__ __forceinline__ float inverse_scale(float s) {
    return (s > 0.0f && s < __int_as_float(0x7f800000)) ? __fdiv_rn(1.0f, s) : 0.0f;
}

// Quantizer of Eq. 15 (round half up) as a level index u in [0, 2^bits - 1].
// Two separately rounded multiplies, then floor: no add before the floor, nothing to contract.
template <int ACT>
__device__ __forceinline__ int level_index(float x, float inv_s, float half_L, float lo, float hi, int H) {
    float y = __fmul_rn(__fmul_rn(x, inv_s), half_L);
    if (!(y == y)) y = 0.0f;                 // NaN -> level just above zero
    if (ACT == MPQ_ACT_HRELU) y = fmaxf(y, 0.0f);
    y = fminf(fmaxf(y, lo), hi);             // HTanh clamp: [-H, H - 1/2]
    return __float2int_rd(y) + H;
}

}  // namespace mpq
