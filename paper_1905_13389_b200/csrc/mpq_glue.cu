// Full-precision glue around the quantized layers of a ResNet-shaped stack: the 7x7 stride-2
// stem convolution (the first layer stays fp32) and the 3x3 stride-2 max-pool.  Neither is part
// of the paper's method; they only produce the activations that the encoded layers consume.
#include "mpq_common.cuh"

namespace mpq {

// ------------------------------------------------------------------------------------------
// Stem: y[n][o][oh][ow] = relu?( sum_{c,kh,kw} x[n][c][2 oh + kh - 3][2 ow + kw - 3] * w[o][c][kh][kw] )
// C = 3, O = 64, 7x7, stride 2, pad 3 (zero).  A CTA owns a 16 x 16 tile of output pixels of one
// image: the 37 x 37 x 3 input patch and all 64 x 147 weights sit in shared memory; each thread
// computes its pixel for 16 output channels at a time (weights read as broadcast 16-byte vectors).
// Accumulation order per output: c, then kh, then kw, one fused multiply-add each.
// ------------------------------------------------------------------------------------------
constexpr int kStemTile = 16;
constexpr int kStemPatch = 2 * kStemTile + 5;      // 37
constexpr int kStemTaps = 3 * 7 * 7;               // 147
constexpr int kStemO = 64;

__global__ void __launch_bounds__(kStemTile* kStemTile)
stem_conv7x7_kernel(const float* __restrict__ x, const float* __restrict__ w, float* __restrict__ y,
                    int N, int H, int W, int Ho, int Wo, int relu) {
    extern __shared__ __align__(16) float smem[];
    chain_entry();
    float* ws = smem;                                   // [147][64]
    float* xs = smem + kStemTaps * kStemO;              // [3][37][38]
    constexpr int kRow = kStemPatch + 1;
    const int tid = threadIdx.x;
    const int tiles_w = (Wo + kStemTile - 1) / kStemTile;
    const int tiles_h = (Ho + kStemTile - 1) / kStemTile;
    const int n = blockIdx.x / (tiles_w * tiles_h);
    const int trem = blockIdx.x % (tiles_w * tiles_h);
    const int oh0 = (trem / tiles_w) * kStemTile, ow0 = (trem % tiles_w) * kStemTile;

    for (int i = tid; i < kStemTaps * kStemO; i += blockDim.x) {
        const int o = i / kStemTaps, t = i % kStemTaps;  // global order [o][c][kh][kw]
        ws[t * kStemO + o] = __ldg(w + i);
    }
    const int ih0 = oh0 * 2 - 3, iw0 = ow0 * 2 - 3;
    for (int i = tid; i < 3 * kStemPatch * kStemPatch; i += blockDim.x) {
        const int c = i / (kStemPatch * kStemPatch);
        const int r = (i / kStemPatch) % kStemPatch, q = i % kStemPatch;
        const int ih = ih0 + r, iw = iw0 + q;
        float v = 0.0f;
        if (ih >= 0 && ih < H && iw >= 0 && iw < W) v = __ldg(x + (((int64_t)n * 3 + c) * H + ih) * W + iw);
        xs[(c * kStemPatch + r) * kRow + q] = v;
    }
    __syncthreads();

    const int ty = tid / kStemTile, tx = tid % kStemTile;
    const int oh = oh0 + ty, ow = ow0 + tx;
    const bool live = oh < Ho && ow < Wo;
    for (int o0 = 0; o0 < kStemO; o0 += 16) {
        float acc[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) acc[j] = 0.0f;
        for (int c = 0; c < 3; ++c) {
            for (int kh = 0; kh < 7; ++kh) {
                const float* xrow = xs + (c * kStemPatch + 2 * ty + kh) * kRow + 2 * tx;
                const float* wrow = ws + ((c * 7 + kh) * 7) * kStemO + o0;
#pragma unroll
                for (int kw = 0; kw < 7; ++kw) {
                    const float xv = xrow[kw];
                    const float4* wv = reinterpret_cast<const float4*>(wrow + kw * kStemO);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float4 f = wv[q];
                        acc[4 * q + 0] = fmaf(xv, f.x, acc[4 * q + 0]);
                        acc[4 * q + 1] = fmaf(xv, f.y, acc[4 * q + 1]);
                        acc[4 * q + 2] = fmaf(xv, f.z, acc[4 * q + 2]);
                        acc[4 * q + 3] = fmaf(xv, f.w, acc[4 * q + 3]);
                    }
                }
            }
        }
        if (live) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const float v = relu ? fmaxf(acc[j], 0.0f) : acc[j];
                y[(((int64_t)n * kStemO + o0 + j) * Ho + oh) * Wo + ow] = v;
            }
        }
    }
}

// 3x3 max-pool, stride 2, pad 1 (padding never wins: the window always holds a real element).
__global__ void maxpool3x3s2_kernel(const float* __restrict__ x, float* __restrict__ y,
                                    int64_t planes, int H, int W, int Ho, int Wo, float* out_max) {
    chain_entry();
    float seen_max = 0.0f;
    const int64_t total = planes * Ho * Wo;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int ow = (int)(i % Wo), oh = (int)((i / Wo) % Ho);
        const int64_t pl = i / ((int64_t)Wo * Ho);
        const float* xp = x + pl * H * W;
        float m = -__int_as_float(0x7f800000);
        for (int kh = 0; kh < 3; ++kh) {
            const int ih = 2 * oh + kh - 1;
            if (ih < 0 || ih >= H) continue;
            for (int kw = 0; kw < 3; ++kw) {
                const int iw = 2 * ow + kw - 1;
                if (iw < 0 || iw >= W) continue;
                m = fmaxf(m, __ldg(xp + (int64_t)ih * W + iw));
            }
        }
        y[i] = m;
        seen_max = fmaxf(seen_max, m);
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
    const int64_t blocks = (int64_t)N * ceil_div(Ho, kStemTile) * ceil_div(Wo, kStemTile);
    if (blocks > 0x7fffffffLL) return MPQ_ERR_BAD_SHAPE;
    const size_t smem = (size_t)(kStemTaps * kStemO + 3 * kStemPatch * (kStemPatch + 1)) * sizeof(float);
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MPQ_ERR_CUDA;
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(stem_conv7x7_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return MPQ_ERR_CUDA;
        configured[dev] = true;
    }
    return launch_chained(stem_conv7x7_kernel, (unsigned)blocks, kStemTile * kStemTile, smem, (cudaStream_t)stream,
                          x, w, y, N, H, W, Ho, Wo, relu);
}

extern "C" int mpq_maxpool3x3s2(const float* x, float* y, int N, int C, int H, int W, float* out_max,
                                void* stream) {
    if (!x || !y) return MPQ_ERR_NULL;
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0) return MPQ_ERR_BAD_SHAPE;
    const int Ho = (H + 2 - 3) / 2 + 1, Wo = (W + 2 - 3) / 2 + 1;
    const int64_t total = (int64_t)N * C * Ho * Wo;
    const int64_t blocks = min((int64_t)148 * 16, ceil_div(total, 256));
    return launch_chained(maxpool3x3s2_kernel, (unsigned)blocks, 256, 0, (cudaStream_t)stream,
                          x, y, (int64_t)N * C, H, W, Ho, Wo, out_max);
}

extern "C" int mpq_zero(void* p, int64_t bytes, void* stream) {
    if (!p) return MPQ_ERR_NULL;
    if (bytes <= 0) return MPQ_ERR_BAD_SHAPE;
    return cudaMemsetAsync(p, 0, (size_t)bytes, (cudaStream_t)stream) == cudaSuccess ? MPQ_OK : MPQ_ERR_CUDA;
}
