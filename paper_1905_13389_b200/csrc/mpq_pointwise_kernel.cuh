// 1 x 1 convolution over few channels (C <= 256, no padding): the pixel-stationary form of the
// branch-fused product.
//
// With k = C of at most 8 words a tile of the general kernel has a single, partly filled k-stage and
// its per-tile set-up outweighs the branch arithmetic (a 64-channel shortcut convolution ran at 0.46
// of the instruction-mix peak).  Here a thread owns ONE output pixel: it reads that pixel's SB x C/32
// plane words once, keeps them in registers, and walks over the output channels of its CTA, whose
// weight planes sit in shared memory and are read as broadcasts.  No staging ring, no k-loop, no
// barrier after the set-up; per output there are only the branch arithmetic (the same carry-save
// levels as the general kernel), HB x NQ shared-memory loads and the store.
//
// Grid: x = blocks of 256 output pixels, y = blocks of kPointwiseChannels output channels.
// NQ = 16-byte chunks per pixel and plane (1: C <= 128, 2: C = 256); NW = words of a chunk that hold
// data (2 for C = 32 / 64, whose chunk is zero-filled, else 4).
#pragma once
#include "mpq_branch_kernel.cuh"

namespace mpq {

constexpr int kPointwiseChannels = 32;

template <int HB, int SB, int NQ, int NW>
__global__ void __launch_bounds__(256)
pointwise_kernel(const BranchParams p) {
    __shared__ uint4 wq[kPointwiseChannels * HB * NQ];      // [channel][plane][chunk]
    __shared__ float alpha_s[kPointwiseChannels];
    chain_entry();
    const int tid = (int)threadIdx.x;
    const int o_base = (int)blockIdx.y * kPointwiseChannels;
    const int oc = min(kPointwiseChannels, p.O - o_base);
    const bool want_f32 = p.out_f32 != nullptr;
    // weights of this CTA's channels: rows are zero-padded to whole 16-byte chunks
    for (int i = tid; i < oc * HB * NQ; i += 256) {
        const int q = i % NQ, plane = (i / NQ) % HB, o = i / (NQ * HB);
        wq[i] = __ldg(reinterpret_cast<const uint4*>(p.held + ((int64_t)plane * p.held_plane_rows + o_base + o) * p.rw) + q);
    }
    if (tid < oc && want_f32) {
        const float fa = __fdiv_rn(__ldg(p.a_scale), (float)((1 << SB) - 1));
        alpha_s[tid] = __fmul_rn(fa, __fdiv_rn(__ldg(p.w_scale + (p.w_per_row ? o_base + tid : 0)), (float)((1 << HB) - 1)));
    }
    __syncthreads();

    const int64_t g = (int64_t)blockIdx.x * 256 + tid;      // output pixel (n, oh, ow)
    const int64_t hw = (int64_t)p.Ho * p.Wo;
    float seen_max = 0.0f;
    if (g < p.streamed_rows) {
        const int n = (int)(g / hw);
        const int rem = (int)(g % hw);
        const int64_t pix = ((int64_t)n * p.H + (rem / p.Wo) * p.stride) * p.W + (rem % p.Wo) * p.stride;
        const int64_t plane_words = (int64_t)p.N * p.H * p.W * p.Cw;
        uint4 s[NQ][SB];
#pragma unroll
        for (int j = 0; j < SB; ++j) {
            const uint32_t* src = p.streamed + j * plane_words + pix * p.Cw;
            if (NQ == 2) {
                s[0][j] = __ldg(reinterpret_cast<const uint4*>(src));
                s[NQ - 1][j] = __ldg(reinterpret_cast<const uint4*>(src) + 1);
            } else if (NW == 4) {
                s[0][j] = __ldg(reinterpret_cast<const uint4*>(src));
            } else if (p.Cw == 2) {
                const uint2 v = __ldg(reinterpret_cast<const uint2*>(src));
                s[0][j] = make_uint4(v.x, v.y, 0u, 0u);
            } else {
                s[0][j] = make_uint4(__ldg(src), 0u, 0u, 0u);
            }
        }
        constexpr uint32_t LL = (uint32_t)(((1 << HB) - 1) * ((1 << SB) - 1));
        const uint32_t full = LL * (uint32_t)p.k;
        const uint32_t none[1] = {0u};
        const int64_t out0 = ((int64_t)n * p.O + o_base) * hw + rem;
#pragma unroll 1
        for (int o = 0; o < oc; ++o) {
            uint32_t acc = 0u;
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                uint4 h[HB];
#pragma unroll
                for (int i = 0; i < HB; ++i) h[i] = wq[(o * HB + i) * NQ + q];
                BranchLevel<HB, SB, 1, NW, 0, 0, (2 * HB * SB * NW) / 4>::run(h, s[q], none, acc, p);
            }
            const int32_t v = (int32_t)(full - 2u * acc);
            const int64_t idx = out0 + (int64_t)o * hw;
            if (p.out_i32) p.out_i32[idx] = v;
            if (want_f32) {
                float f = __fmul_rn((float)v, alpha_s[o]);
                if (p.residual) f = __fadd_rn(f, __ldg(p.residual + idx));
                if (p.relu) f = fmaxf(f, 0.0f);
                p.out_f32[idx] = f;
                seen_max = fmaxf(seen_max, f);
            }
        }
    }
    if (p.out_max) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) seen_max = fmaxf(seen_max, __shfl_xor_sync(0xffffffffu, seen_max, off));
        if ((tid & 31) == 0 && seen_max > 0.0f) atomicMax(reinterpret_cast<int*>(p.out_max), __float_as_int(seen_max));
    }
}

// ------------------------------------------------------------------------------------------
// 3 x 3 convolution over 64 channels, pixel-stationary.  k = 576 is 18 words: the general kernel's
// tile runs two and a quarter k-stages and pays its set-up, ring and gather for them (0.82 of the
// instruction-mix peak).  A thread keeps the 9 taps x 2 words x SB planes of its output pixel in
// registers (taps outside the image as zero bits, i.e. as the code -L_a, taken out again through the
// tap sums exactly as in the general kernel) and walks over up to 64 output channels whose weight
// rows -- five 16-byte chunks per plane, the last one half filled -- are broadcast from shared memory.
// ------------------------------------------------------------------------------------------
constexpr int kWindowChannels = 64;

// PLANES: the store also runs the consumer's Encoder (a variant of its own: the plain store keeps
// its registers).
template <int HB, int SB, bool PLANES>
__global__ void __launch_bounds__(256)
window3x3c64_kernel(const BranchParams p) {
    constexpr int NQ = 5;                                    // 18 words = four chunks and a half
    extern __shared__ uint4 window_smem[];
    uint4* wq = window_smem;                                 // [channel][plane][chunk]
    float* alpha_s = reinterpret_cast<float*>(wq + kWindowChannels * HB * NQ);
    int* tap_s = reinterpret_cast<int*>(alpha_s + kWindowChannels);          // [tap][channel]
    // consumer's Encoder in the store: level indices [channel][thread], one byte each (16 KB); a thread
    // reads back only its own column, so no barrier is needed
    unsigned char* code_s = reinterpret_cast<unsigned char*>(tap_s + 9 * kWindowChannels);
    chain_entry();
    const int tid = (int)threadIdx.x;
    const int o_base = (int)blockIdx.y * kWindowChannels;
    const int oc = min(kWindowChannels, p.O - o_base);
    constexpr bool want_planes = PLANES;
    const bool want_f32 = p.out_f32 != nullptr || want_planes;
    for (int i = tid; i < oc * HB * NQ; i += 256) {
        const int q = i % NQ, plane = (i / NQ) % HB, o = i / (NQ * HB);
        wq[i] = __ldg(reinterpret_cast<const uint4*>(p.held + ((int64_t)plane * p.held_plane_rows + o_base + o) * p.rw) + q);
    }
    if (p.tap_sums)
        for (int i = tid; i < 9 * oc; i += 256) tap_s[(i / oc) * kWindowChannels + i % oc] = __ldg(p.tap_sums + (int64_t)(i / oc) * p.O + o_base + i % oc);
    if (tid < oc && want_f32) {
        const float fa = __fdiv_rn(__ldg(p.a_scale), (float)((1 << SB) - 1));
        alpha_s[tid] = __fmul_rn(fa, __fdiv_rn(__ldg(p.w_scale + (p.w_per_row ? o_base + tid : 0)), (float)((1 << HB) - 1)));
    }
    __syncthreads();

    const int64_t g = (int64_t)blockIdx.x * 256 + tid;      // output pixel (n, oh, ow)
    const int64_t hw = (int64_t)p.Ho * p.Wo;
    float seen_max = 0.0f;
    if (g < p.streamed_rows) {
        const int n = (int)(g / hw);
        const int rem = (int)(g % hw);
        const int ih0 = (rem / p.Wo) * p.stride - p.pad, iw0 = (rem % p.Wo) * p.stride - p.pad;
        const int64_t plane_words = (int64_t)p.N * p.H * p.W * 2;
        uint4 s[NQ][SB];
        unsigned outside = 0u;
#pragma unroll
        for (int t = 0; t < 9; ++t) {
            const int ih = ih0 + t / 3, iw = iw0 + t % 3;
            const bool in = ih >= 0 && ih < p.H && iw >= 0 && iw < p.W;
            if (!in) outside |= 1u << t;
            const uint32_t* src = p.streamed + (in ? (((int64_t)n * p.H + ih) * p.W + iw) * 2 : 0);
#pragma unroll
            for (int j = 0; j < SB; ++j) {
                const uint2 v = in ? __ldg(reinterpret_cast<const uint2*>(src + j * plane_words)) : make_uint2(0u, 0u);
                if (t % 2 == 0) { s[t / 2][j].x = v.x; s[t / 2][j].y = v.y; }
                else { s[t / 2][j].z = v.x; s[t / 2][j].w = v.y; }
            }
        }
#pragma unroll
        for (int j = 0; j < SB; ++j) { s[NQ - 1][j].z = 0u; s[NQ - 1][j].w = 0u; }
        constexpr uint32_t LL = (uint32_t)(((1 << HB) - 1) * ((1 << SB) - 1));
        const uint32_t full = LL * (uint32_t)p.k;
        const uint32_t none[1] = {0u};
        const int64_t out0 = ((int64_t)n * p.O + o_base) * hw + rem;
        float next_inv = 0.0f, next_half_L = 0.0f, next_lo = 0.0f, next_hi = 0.0f;
        int next_H = 0;
        if (want_planes) {
            next_inv = inverse_scale(__ldg(p.next_scale));
            next_H = 1 << (p.next_bits - 1);
            next_half_L = 0.5f * (float)((1 << p.next_bits) - 1);
            next_lo = (float)(-next_H); next_hi = (float)next_H - 0.5f;
        }
#pragma unroll 1
        for (int o = 0; o < oc; ++o) {
            uint32_t acc = 0u;
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                uint4 h[HB];
#pragma unroll
                for (int i = 0; i < HB; ++i) h[i] = wq[(o * HB + i) * NQ + q];
                if (q < NQ - 1) BranchLevel<HB, SB, 1, 4, 0, 0, 2 * HB * SB>::run(h, s[q], none, acc, p);
                else BranchLevel<HB, SB, 1, 2, 0, 0, HB * SB>::run(h, s[q], none, acc, p);
            }
            int32_t v = (int32_t)(full - 2u * acc);
            if (outside) {
                uint32_t fix = 0u;
                for (int t = 0; t < 9; ++t)
                    if (outside & (1u << t)) fix += (uint32_t)tap_s[t * kWindowChannels + o];
                v = (int32_t)((uint32_t)v + (uint32_t)((1 << SB) - 1) * fix);
            }
            const int64_t idx = out0 + (int64_t)o * hw;
            if (p.out_i32) p.out_i32[idx] = v;
            if (want_f32) {
                float f = __fmul_rn((float)v, alpha_s[o]);
                if (p.residual) f = __fadd_rn(f, __ldg(p.residual + idx));
                if (p.relu) f = fmaxf(f, 0.0f);
                if (p.out_f32) p.out_f32[idx] = f;
                seen_max = fmaxf(seen_max, f);
                if (want_planes) {
                    const int u = p.next_act == MPQ_ACT_HRELU
                                      ? level_index<MPQ_ACT_HRELU>(f, next_inv, next_half_L, next_lo, next_hi, next_H)
                                      : level_index<MPQ_ACT_HTANH>(f, next_inv, next_half_L, next_lo, next_hi, next_H);
                    code_s[o * 256 + tid] = (unsigned char)u;
                }
            }
        }
        if (want_planes) {
            // the pixel's level indices, 32 channels at a time, through the 8 x 8 bit-block transpose:
            // word i of a group holds channels i, 8 + i, 16 + i, 24 + i (O is a multiple of 32)
            const int Ow = p.O / 32;
            const int64_t plane_words_out = (int64_t)p.N * hw * Ow;
            for (int grp = 0; grp < oc / 32; ++grp) {
                uint32_t w8[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const unsigned char* c = code_s + (32 * grp + i) * 256 + tid;
                    w8[i] = (uint32_t)c[0] | ((uint32_t)c[8 * 256] << 8) | ((uint32_t)c[16 * 256] << 16) | ((uint32_t)c[24 * 256] << 24);
                }
#pragma unroll
                for (int d = 1; d <= 4; d *= 2) {
                    const uint32_t mask = d == 1 ? 0x55555555u : d == 2 ? 0x33333333u : 0x0F0F0F0Fu;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        if ((i & d) == 0) {
                            const uint32_t x = ((w8[i] >> d) ^ w8[i + d]) & mask;
                            w8[i + d] ^= x;
                            w8[i] ^= x << d;
                        }
                    }
                }
                const int64_t at0 = ((int64_t)n * hw + rem) * Ow + (o_base / 32 + grp);
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    if (q < p.next_bits) p.next_planes[(int64_t)q * plane_words_out + at0] = w8[q];
            }
        }
    }
    if (p.out_max) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) seen_max = fmaxf(seen_max, __shfl_xor_sync(0xffffffffu, seen_max, off));
        if ((tid & 31) == 0 && seen_max > 0.0f) atomicMax(reinterpret_cast<int*>(p.out_max), __float_as_int(seen_max));
    }
}

// (activations of up to 4 bits: 18 words per plane must stay in registers)
inline bool window3x3c64_applies(const BranchParams& p, int a_bits) {
    return p.KH == 3 && p.KW == 3 && p.Cw == 2 && a_bits <= 4 && (p.pad == 0 || p.tap_sums != nullptr);
}

template <int HB, int SB>
static int launch_window3x3c64(const BranchParams& p, cudaStream_t st) {
    const int64_t bx = ceil_div(p.streamed_rows, 256), by = ceil_div(p.O, kWindowChannels);
    if (bx <= 0 || bx > 0x7fffffffLL || by > 65535) return MPQ_ERR_BAD_SHAPE;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)bx, (unsigned)by, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = bx * by >= 1024 ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // weights, decoder factors, tap sums, level-index tile
    constexpr size_t smem_bytes = (size_t)kWindowChannels * (HB * 5 * sizeof(uint4) + sizeof(float) + 9 * sizeof(int) + 256);
    static PerDeviceOnce configured[2];
    const bool planes = p.next_planes != nullptr;
    auto kern = planes ? window3x3c64_kernel<HB, SB, true> : window3x3c64_kernel<HB, SB, false>;
    if (configured[planes ? 1 : 0].raise_smem_limit(kern, smem_bytes) != MPQ_OK) return MPQ_ERR_CUDA;
    cfg.dynamicSmemBytes = smem_bytes;
    if (cudaLaunchKernelEx(&cfg, kern, p) != cudaSuccess) {
        cudaGetLastError();
        return MPQ_ERR_CUDA;
    }
    return launch_status();
}

template <int HB>
int launch_window3x3c64_hb(int sb, const BranchParams& p, cudaStream_t st);

// Takes the layers that mpq_conv would otherwise run as tiles with a single k-stage.
inline bool pointwise_applies(const BranchParams& p) {
    return p.KH == 1 && p.KW == 1 && p.pad == 0 && p.Cw <= 8 && p.next_planes == nullptr;
}

template <int HB, int SB>
static int launch_pointwise(const BranchParams& p, cudaStream_t st) {
    const int64_t bx = ceil_div(p.streamed_rows, 256), by = ceil_div(p.O, kPointwiseChannels);
    if (bx <= 0 || bx > 0x7fffffffLL || by > 65535) return MPQ_ERR_BAD_SHAPE;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)bx, (unsigned)by, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = bx * by >= 1024 ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e;
    if (p.Cw == 8) e = cudaLaunchKernelEx(&cfg, pointwise_kernel<HB, SB, 2, 4>, p);
    else if (p.Cw == 4) e = cudaLaunchKernelEx(&cfg, pointwise_kernel<HB, SB, 1, 4>, p);
    else e = cudaLaunchKernelEx(&cfg, pointwise_kernel<HB, SB, 1, 2>, p);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return MPQ_ERR_CUDA;
    }
    return launch_status();
}

template <int HB>
int launch_pointwise_hb(int sb, const BranchParams& p, cudaStream_t st);

}  // namespace mpq
