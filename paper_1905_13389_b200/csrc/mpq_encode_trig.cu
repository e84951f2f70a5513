// The Encoder in its trigonometric form (Section 3.2 "M-bit Encoding Functions", Eq. 11): every
// bit of the code is the sign of a sine of x/s,
//     bit b-1 (highest)   = sign( sin((2^b-1)/2^b * pi * y)),
//     bit m-1, 1 <= m < b = sign(-sin((2^b-1)/2^m * pi * y)),       y = clamp(x/s)  (HTanh / HReLU),
// the family that Eq. 11 prints for b = 2, continued to 1..8 bits (the highest bit has half a
// period on [-1,1], every lower bit doubles the frequency and flips the sign).  At a zero of a
// sine -- a level boundary -- the sign is that of the sine just above the zero, so the tie goes
// to the upper level like the rounding of Eq. 15; x = 0 therefore lands on the level above zero.
// This is the form the paper differentiates for training; for inference it spells the same level
// index as mpq_encode except within one fp32 rounding of a level boundary.  It is a selectable
// mode, not the fast path: one sinpi per bit and element, warp-ballot packing, no tuning.
#include "mpq_common.cuh"

namespace mpq {

// Level index of one element through the sine encoders; t = y * (2^b-1)/2^m is one rounded fp32
// multiply by an exact constant, sinpif/cospif reduce their argument exactly.
template <int ACT>
__device__ __forceinline__ uint32_t trig_level_index(float x, float inv_s, int bits) {
    float y = __fmul_rn(x, inv_s);
    if (!(y == y)) y = 0.0f;
    if (ACT == MPQ_ACT_HRELU) y = fmaxf(y, 0.0f);
    y = fminf(fmaxf(y, -1.0f), 1.0f);
    const float L = (float)((1 << bits) - 1);
    uint32_t u = 0u;
    for (int m = 1; m <= bits; ++m) {
        const float t = __fmul_rn(y, __fdiv_rn(L, (float)(1 << m)));
        float sine = (t == floorf(t)) ? cospif(t) : sinpif(t);      // at a zero: the sign of the slope
        if (m < bits) sine = -sine;
        if (sine > 0.0f) u |= 1u << (m - 1);
    }
    return u;
}

// One warp packs 1024 consecutive elements of a row: in step j lane L encodes element 32 j + L
// and one ballot per plane transposes that bit across the warp into word j.
template <int ACT>
__global__ void __launch_bounds__(256)
encode_rows_trig_kernel(const float* __restrict__ x, int64_t rows, int64_t k, int64_t ldx,
                        const float* __restrict__ scale, int per_row, int bits,
                        uint32_t* __restrict__ planes, int64_t rw, int64_t segs_per_row) {
    chain_entry();
    const int64_t warp = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (warp >= rows * segs_per_row) return;
    const int lane = threadIdx.x & 31;
    const int64_t row = warp / segs_per_row, seg = warp % segs_per_row;
    const float* xr = x + row * ldx;
    const int64_t e0 = seg * 1024;
    const float inv = inverse_scale(__ldg(scale + (per_row ? row : 0)));
    uint32_t mine[kMaxBits];
#pragma unroll
    for (int p = 0; p < kMaxBits; ++p) mine[p] = 0u;
    const int64_t remaining = k - e0;
    const int steps = remaining >= 1024 ? 32 : (int)((remaining + 31) / 32);    // warp-uniform; 0 for pad words
    for (int j = 0; j < steps; ++j) {
        const int64_t idx = e0 + (int64_t)j * 32 + lane;
        const uint32_t u = idx < k ? trig_level_index<ACT>(__ldg(xr + idx), inv, bits) : 0u;
#pragma unroll
        for (int p = 0; p < kMaxBits; ++p) {
            if (p < bits) {                                                       // warp-uniform
                const uint32_t word = __ballot_sync(0xffffffffu, (u >> p) & 1u);
                if (lane == j) mine[p] = word;
            }
        }
    }
    const int64_t word_idx = seg * 32 + lane;
    if (word_idx < rw) {
#pragma unroll
        for (int p = 0; p < kMaxBits; ++p)
            if (p < bits) planes[((int64_t)p * rows + row) * rw + word_idx] = mine[p];
    }
}

}  // namespace mpq

using namespace mpq;

extern "C" int mpq_encode_with(int encoder, const float* x, int64_t rows, int64_t k, int64_t ldx,
                               const float* scale, int mode, int act, int bits,
                               uint32_t* planes, void* stream) {
    if (encoder == MPQ_ENC_LEVELS) return mpq_encode(x, rows, k, ldx, scale, mode, act, bits, planes, stream);
    if (encoder != MPQ_ENC_TRIG) return MPQ_ERR_UNSUPPORTED;
    if (!x || !scale || !planes) return MPQ_ERR_NULL;
    if (rows <= 0 || k <= 0 || ldx < k) return MPQ_ERR_BAD_SHAPE;
    if (!bits_ok(bits) || (mode != MPQ_SCALE_PER_TENSOR && mode != MPQ_SCALE_PER_ROW) ||
        (act != MPQ_ACT_HTANH && act != MPQ_ACT_HRELU)) return MPQ_ERR_UNSUPPORTED;
    if (!aligned16(planes)) return MPQ_ERR_ALIGN;
    const int64_t rw = row_words(k);
    const int64_t segs = ceil_div(rw, 32);
    const int64_t blocks = ceil_div(rows * segs, 8);
    if (blocks > 0x7fffffffLL) return MPQ_ERR_BAD_SHAPE;
    const int per_row = mode == MPQ_SCALE_PER_ROW;
    cudaStream_t st = (cudaStream_t)stream;
    if (act == MPQ_ACT_HRELU)
        return launch_chained(encode_rows_trig_kernel<MPQ_ACT_HRELU>, (unsigned)blocks, 256, 0, st,
                              x, rows, k, ldx, scale, per_row, bits, planes, rw, segs);
    return launch_chained(encode_rows_trig_kernel<MPQ_ACT_HTANH>, (unsigned)blocks, 256, 0, st,
                          x, rows, k, ldx, scale, per_row, bits, planes, rw, segs);
}
