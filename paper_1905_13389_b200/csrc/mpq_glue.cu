// Full-precision glue around the quantized layers of a ResNet-shaped stack: the 7x7 stride-2
// stem convolution (the first layer stays fp32) and the 3x3 stride-2 max-pool.  Neither is part
// of the paper's method; they only produce the activations that the encoded layers consume.
#include "mpq_common.cuh"

namespace mpq {

// ------------------------------------------------------------------------------------------
// Stem: y[n][o][oh][ow] = relu?( sum_{c,kh,kw} x[n][c][2 oh + kh - 3][2 ow + kw - 3] * w[o][c][kh][kw] )
// C = 3, O = 64, 7x7, stride 2, pad 3 (zero).  A CTA owns 16 rows x 56 columns of output pixels of
// one image (224 threads: 16 rows x 14 groups of 4 adjacent pixels); the 37 x 117 x 3 input patch
// and all 64 x 147 weights sit in shared memory.  Per (c, kh) a thread reads the 13 inputs its four
// pixels share and the weights of 16 output channels (broadcast 16-byte vectors) and issues
// 7 x 4 x 16 fused multiply-adds from registers, so the loop is bound by the FP32 pipe, not by
// shared-memory reads.  Accumulation order per output: c, then kh, then kw.
// ------------------------------------------------------------------------------------------
constexpr int kStemRows = 16;                       // output rows per CTA
constexpr int kStemGroups = 14;                     // groups of 4 output columns per CTA
constexpr int kStemCols = 4 * kStemGroups;          // 56
constexpr int kStemThreads = kStemRows * kStemGroups;   // 224
constexpr int kStemPatchH = 2 * kStemRows + 5;      // 37
constexpr int kStemPatchW = 2 * kStemCols + 5;      // 117
constexpr int kStemPatchStride = 120;               // >= 117, rows 16-byte aligned: a thread's 13 inputs are three vector loads + one
constexpr int kStemTaps = 3 * 7 * 7;                // 147
constexpr int kStemO = 64;
constexpr int kStemWRow = 68;                      // floats per staged weight row (64 + 4: spreads the transposing stores over banks)

__global__ void __launch_bounds__(kStemThreads)
stem_conv7x7_kernel(const float* __restrict__ x, const float* __restrict__ w, float* __restrict__ y,
                    int N, int H, int W, int Ho, int Wo, int relu) {
    extern __shared__ __align__(16) float smem[];
    chain_entry();
    float* ws = smem;                                   // [147][68]
    float* xs = smem + kStemTaps * kStemWRow;           // [3][37][120]
    const int tid = threadIdx.x;
    const int tiles_w = (Wo + kStemCols - 1) / kStemCols;
    const int tiles_h = (Ho + kStemRows - 1) / kStemRows;
    const int n = blockIdx.x / (tiles_w * tiles_h);
    const int trem = blockIdx.x % (tiles_w * tiles_h);
    const int oh0 = (trem / tiles_w) * kStemRows, ow0 = (trem % tiles_w) * kStemCols;

    for (int i = tid; i < kStemTaps * kStemO; i += kStemThreads) {
        const int o = i / kStemTaps, t = i % kStemTaps;  // global order [o][c][kh][kw]
        ws[t * kStemWRow + o] = __ldg(w + i);
    }
    const int ih0 = oh0 * 2 - 3, iw0 = ow0 * 2 - 3;
    for (int i = tid; i < 3 * kStemPatchH * kStemPatchW; i += kStemThreads) {
        const int c = i / (kStemPatchH * kStemPatchW);
        const int r = (i / kStemPatchW) % kStemPatchH, q = i % kStemPatchW;
        const int ih = ih0 + r, iw = iw0 + q;
        float v = 0.0f;
        if (ih >= 0 && ih < H && iw >= 0 && iw < W) v = __ldg(x + (((int64_t)n * 3 + c) * H + ih) * W + iw);
        xs[(c * kStemPatchH + r) * kStemPatchStride + q] = v;
    }
    __syncthreads();

    const int ty = tid / kStemGroups, tg = tid % kStemGroups;
    const int oh = oh0 + ty, ow = ow0 + 4 * tg;
    for (int o0 = 0; o0 < kStemO; o0 += 16) {
        float acc[4][16];
#pragma unroll
        for (int p = 0; p < 4; ++p)
#pragma unroll
            for (int j = 0; j < 16; ++j) acc[p][j] = 0.0f;
        for (int c = 0; c < 3; ++c) {
#pragma unroll 1
            for (int kh = 0; kh < 7; ++kh) {
                const float* xrow = xs + (c * kStemPatchH + 2 * ty + kh) * kStemPatchStride + 8 * tg;
                float xv[13];
                {
                    const float4* xq = reinterpret_cast<const float4*>(xrow);     // 8 * tg floats into an aligned row
                    const float4 a = xq[0], b = xq[1], d = xq[2];
                    xv[0] = a.x; xv[1] = a.y; xv[2] = a.z; xv[3] = a.w;
                    xv[4] = b.x; xv[5] = b.y; xv[6] = b.z; xv[7] = b.w;
                    xv[8] = d.x; xv[9] = d.y; xv[10] = d.z; xv[11] = d.w;
                    xv[12] = xrow[12];
                }
                const float* wrow = ws + ((c * 7 + kh) * 7) * kStemWRow + o0;
#pragma unroll
                for (int kw = 0; kw < 7; ++kw) {
                    const float4* wv = reinterpret_cast<const float4*>(wrow + kw * kStemWRow);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float4 f = wv[q];
#pragma unroll
                        for (int p = 0; p < 4; ++p) {
                            const float xin = xv[2 * p + kw];
                            acc[p][4 * q + 0] = fmaf(xin, f.x, acc[p][4 * q + 0]);
                            acc[p][4 * q + 1] = fmaf(xin, f.y, acc[p][4 * q + 1]);
                            acc[p][4 * q + 2] = fmaf(xin, f.z, acc[p][4 * q + 2]);
                            acc[p][4 * q + 3] = fmaf(xin, f.w, acc[p][4 * q + 3]);
                        }
                    }
                }
            }
        }
        if (oh < Ho) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                float* dst = y + (((int64_t)n * kStemO + o0 + j) * Ho + oh) * Wo + ow;
#pragma unroll
                for (int p = 0; p < 4; ++p)
                    if (ow + p < Wo) dst[p] = relu ? fmaxf(acc[p][j], 0.0f) : acc[p][j];
            }
        }
    }
}

// 3x3 max-pool, stride 2, pad 1 (padding never wins: the window always holds a real element).
// A thread produces four adjacent outputs of a row from the 3 x 9 inputs they share, so that
// 27 loads are in flight per thread and neighbouring threads read neighbouring columns.
// VEC: W is a multiple of 8 and x is 16-byte aligned -- the eight inputs 8g .. 8g+7 of a group are
// two aligned 16-byte loads, and the ninth (8g - 1) is the left neighbour's last element, taken
// from the neighbouring lane when that lane holds the same row's previous group.
template <bool VEC>
__global__ void maxpool3x3s2_kernel(const float* __restrict__ x, float* __restrict__ y,
                                    int64_t planes, int H, int W, int Ho, int Wo, float* out_max) {
    chain_entry();
    float seen_max = 0.0f;
    const int groups = (Wo + 3) / 4;                       // groups of 4 outputs per row
    const int64_t total = planes * Ho * groups;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const float ninf = -__int_as_float(0x7f800000);
    // (VEC: every lane of a warp runs the same number of iterations up to the last one, where the
    // shuffle below names the lanes that are still in the loop)
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int g = (int)(i % groups), oh = (int)((i / groups) % Ho);
        const int64_t pl = i / ((int64_t)groups * Ho);
        const float* xp = x + pl * H * W;
        const int ow0 = 4 * g, iw0 = 2 * ow0 - 1;
        float col[9];                                      // column maxima over the three rows
#pragma unroll
        for (int q = 0; q < 9; ++q) col[q] = ninf;
        if (VEC) {
            const unsigned live = __activemask();
            float4 lo[3], hi[3];
#pragma unroll
            for (int kh = 0; kh < 3; ++kh) {
                const int ih = 2 * oh + kh - 1;
                const bool in = ih >= 0 && ih < H;
                const float4* row = reinterpret_cast<const float4*>(xp + (int64_t)(in ? ih : 0) * W + 8 * g);
                lo[kh] = in ? __ldg(row) : make_float4(ninf, ninf, ninf, ninf);
                hi[kh] = in ? __ldg(row + 1) : make_float4(ninf, ninf, ninf, ninf);
            }
#pragma unroll
            for (int kh = 0; kh < 3; ++kh) {
                col[1] = fmaxf(col[1], lo[kh].x); col[2] = fmaxf(col[2], lo[kh].y);
                col[3] = fmaxf(col[3], lo[kh].z); col[4] = fmaxf(col[4], lo[kh].w);
                col[5] = fmaxf(col[5], hi[kh].x); col[6] = fmaxf(col[6], hi[kh].y);
                col[7] = fmaxf(col[7], hi[kh].z); col[8] = fmaxf(col[8], hi[kh].w);
            }
            // column 8g - 1: the left neighbour's column 8(g-1) + 7, already reduced over the three rows
            const float left = __shfl_up_sync(live, col[8], 1);
            const int lane = (int)(threadIdx.x & 31);
            if (g > 0) {
                if (lane > 0 && ((live >> (lane - 1)) & 1u)) {
                    col[0] = left;                         // lane - 1 holds item i - 1: same row, group g - 1
                } else {
#pragma unroll
                    for (int kh = 0; kh < 3; ++kh) {
                        const int ih = 2 * oh + kh - 1;
                        if (ih >= 0 && ih < H) col[0] = fmaxf(col[0], __ldg(xp + (int64_t)ih * W + iw0));
                    }
                }
            }
        } else {
#pragma unroll
            for (int kh = 0; kh < 3; ++kh) {
                const int ih = 2 * oh + kh - 1;
                if (ih < 0 || ih >= H) continue;
                const float* row = xp + (int64_t)ih * W;
#pragma unroll
                for (int q = 0; q < 9; ++q) {
                    const int iw = iw0 + q;
                    if (iw >= 0 && iw < W) col[q] = fmaxf(col[q], __ldg(row + iw));
                }
            }
        }
        float* dst = y + (pl * Ho + oh) * Wo + ow0;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            if (ow0 + t < Wo) {
                const float m = fmaxf(fmaxf(col[2 * t], col[2 * t + 1]), col[2 * t + 2]);
                dst[t] = m;
                seen_max = fmaxf(seen_max, m);
            }
        }
    }
    if (out_max) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) seen_max = fmaxf(seen_max, __shfl_xor_sync(0xffffffffu, seen_max, off));
        if ((threadIdx.x & 31) == 0 && seen_max > 0.0f) atomicMax(reinterpret_cast<int*>(out_max), __float_as_int(seen_max));
    }
}

}  // namespace mpq

using namespace mpq;

extern "C" int mpq_stem_conv7x7(const float* x, const float* w, float* y, int N, int H, int W, int relu,
                                void* stream) {
    if (!x || !w || !y) return MPQ_ERR_NULL;
    if (N <= 0 || H <= 0 || W <= 0) return MPQ_ERR_BAD_SHAPE;
    const int Ho = (H + 6 - 7) / 2 + 1, Wo = (W + 6 - 7) / 2 + 1;
    const int64_t blocks = (int64_t)N * ceil_div(Ho, kStemRows) * ceil_div(Wo, kStemCols);
    if (blocks > 0x7fffffffLL) return MPQ_ERR_BAD_SHAPE;
    const size_t smem = (size_t)(kStemTaps * kStemWRow + 3 * kStemPatchH * kStemPatchStride) * sizeof(float);
    static PerDeviceOnce configured;
    if (configured.raise_smem_limit(stem_conv7x7_kernel, smem) != MPQ_OK) return MPQ_ERR_CUDA;
    return launch_chained(stem_conv7x7_kernel, (unsigned)blocks, kStemThreads, smem, (cudaStream_t)stream,
                          x, w, y, N, H, W, Ho, Wo, relu);
}

extern "C" int mpq_maxpool3x3s2(const float* x, float* y, int N, int C, int H, int W, float* out_max,
                                void* stream) {
    if (!x || !y) return MPQ_ERR_NULL;
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0) return MPQ_ERR_BAD_SHAPE;
    const int Ho = (H + 2 - 3) / 2 + 1, Wo = (W + 2 - 3) / 2 + 1;
    const int64_t total = (int64_t)N * C * Ho * ((Wo + 3) / 4);
    const int sms = sm_count();
    if (sms <= 0) return MPQ_ERR_CUDA;
    const int64_t blocks = min((int64_t)sms * 32, ceil_div(total, 256));
    const bool vec = W % 8 == 0 && aligned16(x);
    return launch_chained(vec ? maxpool3x3s2_kernel<true> : maxpool3x3s2_kernel<false>, (unsigned)blocks, 256, 0,
                          (cudaStream_t)stream, x, y, (int64_t)N * C, H, W, Ho, Wo, out_max);
}

extern "C" int mpq_zero(void* p, int64_t bytes, void* stream) {
    if (!p) return MPQ_ERR_NULL;
    if (bytes <= 0) return MPQ_ERR_BAD_SHAPE;
    return cudaMemsetAsync(p, 0, (size_t)bytes, (cudaStream_t)stream) == cudaSuccess ? MPQ_OK : MPQ_ERR_CUDA;
}
