// Range (max-abs) and Encoder kernels: fp32 -> packed {-1,+1} bit-planes.
//
// Encoder = quantizer of Eq. 15 (round half up) + the code of Table 2 / Eq. 10, stored one bit
// per element.  All three layouts are HBM-bound: 4 bytes read and bits/8 bytes written per
// element, so the kernels are organised around coalesced reads with many loads in flight.
#include "mpq_common.cuh"

namespace mpq {

// ------------------------------------------------------------------------------------------
// Range: max |x| (HTanh) or max of the positive side (HReLU); NaNs are ignored by fmaxf.
// Non-negative floats order like their bit patterns, so the cross-CTA step is an integer atomicMax.
// ------------------------------------------------------------------------------------------
constexpr int kAbsmaxThreads = 256;
constexpr int kAbsmaxChunk = 8192;  // elements per CTA and step
constexpr int kAbsmaxPerSm = 6;     // CTAs per multiprocessor: 6 x 32 KiB of loads in flight

__global__ void zero_floats_kernel(float* __restrict__ p, int64_t n) {
    chain_entry();
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) p[i] = 0.0f;
}

// The grid is at most a few CTAs per multiprocessor; every CTA walks the chunks of the tensor in
// a grid-stride loop, so all multiprocessors finish together whatever the tensor's size.
template <int ACT, bool VEC4>
__global__ void __launch_bounds__(kAbsmaxThreads, kAbsmaxPerSm)
absmax_kernel(const float* __restrict__ x, int64_t k, int64_t ldx, int64_t chunks_per_row,
              int64_t total_chunks, int per_row, float* __restrict__ out) {
    chain_entry();
    __shared__ float warp_max[kAbsmaxThreads / 32];
    auto publish = [&](float m, int64_t row) {               // CTA-wide maximum -> one atomic
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
        __syncthreads();
        if (threadIdx.x == 0) {
#pragma unroll
            for (int w = 1; w < kAbsmaxThreads / 32; ++w) m = fmaxf(m, warp_max[w]);
            if (m > 0.0f) atomicMax(reinterpret_cast<int*>(out + row), __float_as_int(m));
        }
        __syncthreads();
    };
    float running = 0.0f;
    for (int64_t chunk = blockIdx.x; chunk < total_chunks; chunk += gridDim.x) {
        const int64_t row = chunk / chunks_per_row;
        const int64_t e0 = (chunk % chunks_per_row) * kAbsmaxChunk;
        const float* xr = x + row * ldx;
        const int64_t e1 = min(e0 + (int64_t)kAbsmaxChunk, k);
        float m = 0.0f;
        if (VEC4) {
            // row starts are 16-byte aligned and the chunk start is a multiple of 4 elements
            const int64_t nvec = (e1 - e0) / 4;
            const float4* xv = reinterpret_cast<const float4*>(xr + e0);
            // eight 16-byte loads of every thread are issued before the first one is used
            for (int64_t i0 = threadIdx.x; i0 < nvec; i0 += 8 * kAbsmaxThreads) {
                float4 v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int64_t i = i0 + j * kAbsmaxThreads;
                    v[j] = i < nvec ? __ldcs(xv + i) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);   // read once: streaming load
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (ACT == MPQ_ACT_HRELU) {
                        m = fmaxf(m, fmaxf(fmaxf(v[j].x, v[j].y), fmaxf(v[j].z, v[j].w)));
                    } else {
                        m = fmaxf(m, fmaxf(fmaxf(fabsf(v[j].x), fabsf(v[j].y)), fmaxf(fabsf(v[j].z), fabsf(v[j].w))));
                    }
                }
            }
            for (int64_t i = e0 + nvec * 4 + threadIdx.x; i < e1; i += kAbsmaxThreads) {
                float v = __ldg(xr + i);
                m = fmaxf(m, ACT == MPQ_ACT_HRELU ? v : fabsf(v));
            }
        } else {
            for (int64_t i = e0 + threadIdx.x; i < e1; i += kAbsmaxThreads) {
                float v = __ldg(xr + i);
                m = fmaxf(m, ACT == MPQ_ACT_HRELU ? v : fabsf(v));
            }
        }
        if (per_row) publish(m, row);
        else running = fmaxf(running, m);
    }
    if (!per_row) publish(running, 0);
}

// ------------------------------------------------------------------------------------------
// Row-major encoder.  One warp packs 1024 consecutive elements of a row (32 words per plane).
//
// Full, 16-byte aligned segments take the lane-local path: the 4 KiB segment is copied into
// shared memory with coalesced 16-byte asynchronous copies (rows of 32 floats, padded to 36 so
// that the later 16-byte reads of a quarter-warp fall in distinct banks), then lane L owns
// elements 32 L .. 32 L + 31, i.e. word L of every plane, and builds its words with LaneWords:
// the quantizer and the bit split run on the floating-point pipe, the integer ALU sees one min
// per element, and the plane stores are coalesced 128-byte rows.  The kernel is then limited by
// HBM, not by issue slots.  A lane that meets a NaN (HTanh) or a degenerate range rebuilds its
// words with the plain quantizer (so does every lane when 1/s overflows to infinity, which a
// positive subnormal range does: a zero element then gives 0 * inf = NaN without being one).
//
// Ragged or unaligned segments take the ballot path: in step j lane L quantizes element
// 32 j + L and one __ballot_sync per plane transposes that bit across the warp into word j.
// ------------------------------------------------------------------------------------------
constexpr int kEncodeThreads = 256;
constexpr int kStageRow = 36;          // floats per staged 32-float row (16 bytes of padding)

__device__ __forceinline__ void copy_async_16(void* smem_dst, const void* gsrc) {
    const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void copy_async_wait_all() {
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
}


// ---- Plane words of 32 elements held by one thread, wide codes (5..8 bits) -------------------
// LaneWords costs two floating-point-pipe operations per element and PLANE, which makes an 8-bit
// encoder issue-bound.  For wide codes the level index of every element is taken once (one
// round-down multiply-add leaves it in the low byte of the result, see LaneWords), the 32 bytes are
// laid out as eight words W_i = [u_i, u_(8+i), u_(16+i), u_(24+i)] (byte j of word i = element
// 8 j + i), and the eight 8 x 8 bit blocks that the four byte lanes of W_0..W_7 form are transposed
// in place by three rounds of masked swaps (distance 1, 2, 4).  Afterwards bit 8 j + i of word b is
// bit b of element 8 j + i: word b is the plane word.  About five integer operations per element
// instead of sixteen floating-point ones.
constexpr int kByteBuilderFromBits = 3;       // narrower codes keep LaneWords (measured)
template <int BITS, int ACT>
struct LaneBytes {
    uint32_t t[32];                                // 0x4B000000 + level index, per element
    __device__ __forceinline__ void set(int e, float z) {
        const float magic = 8388608.0f + (ACT == MPQ_ACT_HRELU ? (float)(1 << (BITS - 1)) : 0.0f);
        t[e] = __float_as_uint(__fmaf_rd(z, (float)(1 << BITS), magic));
    }
    __device__ __forceinline__ void words(uint32_t (&out)[BITS]) const {
        uint32_t w[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
            w[i] = __byte_perm(__byte_perm(t[i], t[8 + i], 0x0040), __byte_perm(t[16 + i], t[24 + i], 0x0040), 0x5410);
#pragma unroll
        for (int d = 1; d <= 4; d *= 2) {
            const uint32_t mask = d == 1 ? 0x55555555u : d == 2 ? 0x33333333u : 0x0F0F0F0Fu;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if ((i & d) == 0) {
                    const uint32_t x = ((w[i] >> d) ^ w[i + d]) & mask;
                    w[i + d] ^= x;
                    w[i] ^= x << d;
                }
            }
        }
#pragma unroll
        for (int p = 0; p < BITS; ++p) out[p] = w[p];
    }
};

// The 32 staged elements of one lane (eight consecutive 16-byte chunks at lane_row) -> its BITS plane
// words: quantizer on the floating-point pipe, builder by code width, and the plain quantizer again
// for a lane that met a NaN under HTanh or a range whose inverse is 0 or infinite.
template <int BITS, int ACT>
__device__ __forceinline__ void staged_lane_words(const float* lane_row, float inv, uint32_t two, uint32_t (&word)[BITS]) {
    constexpr int H = 1 << (BITS - 1);
    const float half_L = 0.5f * (float)((1 << BITS) - 1);
    const float lo = (float)(-H), hi = (float)H - 0.5f;
    const float4* own = reinterpret_cast<const float4*>(lane_row);
    float probe = 0.0f;                                 // turns NaN if any element is NaN
    if constexpr (BITS >= kByteBuilderFromBits) {
        LaneBytes<BITS, ACT> lb;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const float4 v = own[c];
            if (ACT == MPQ_ACT_HTANH) probe = fmaf(v.x, v.y, fmaf(v.z, v.w, probe));
            lb.set(4 * c + 0, level_fraction<BITS, ACT>(v.x, inv, half_L));
            lb.set(4 * c + 1, level_fraction<BITS, ACT>(v.y, inv, half_L));
            lb.set(4 * c + 2, level_fraction<BITS, ACT>(v.z, inv, half_L));
            lb.set(4 * c + 3, level_fraction<BITS, ACT>(v.w, inv, half_L));
        }
        lb.words(word);
    } else {
        LaneWords<BITS, ACT> lw;
        lw.clear();
#pragma unroll
        for (int c = 7; c >= 0; --c) {
            const float4 v = own[c];
            if (ACT == MPQ_ACT_HTANH) probe = fmaf(v.x, v.y, fmaf(v.z, v.w, probe));
            lw.push(level_fraction<BITS, ACT>(v.w, inv, half_L), two);
            lw.push(level_fraction<BITS, ACT>(v.z, inv, half_L), two);
            lw.push(level_fraction<BITS, ACT>(v.y, inv, half_L), two);
            lw.push(level_fraction<BITS, ACT>(v.x, inv, half_L), two);
        }
#pragma unroll
        for (int p = 0; p < BITS; ++p) word[p] = lw.word(p);
    }
    if (ACT == MPQ_ACT_HTANH && (probe != probe || inv == 0.0f || inv == __int_as_float(0x7f800000))) {
#pragma unroll
        for (int p = 0; p < BITS; ++p) word[p] = 0u;
        for (int t = 0; t < 32; ++t) {
            const uint32_t u = (uint32_t)level_index<ACT>(lane_row[t], inv, half_L, lo, hi, H);
#pragma unroll
            for (int p = 0; p < BITS; ++p) word[p] |= ((u >> p) & 1u) << t;
        }
    }
}

template <int BITS, int ACT>
__global__ void __launch_bounds__(kEncodeThreads)
encode_rows_kernel(const float* __restrict__ x, int64_t rows, int64_t k, int64_t ldx,
                   const float* __restrict__ scale, int per_row,
                   uint32_t* __restrict__ planes, int64_t rw, int64_t segs_per_row,
                   int vec_ok, uint32_t two) {
    __shared__ __align__(16) float stage[kEncodeThreads / 32][32 * kStageRow];
    chain_entry();
    const int64_t warp = (int64_t)blockIdx.x * (kEncodeThreads / 32) + (threadIdx.x >> 5);
    if (warp >= rows * segs_per_row) return;
    const int lane = threadIdx.x & 31;
    const int64_t row = warp / segs_per_row;
    const int64_t seg = warp % segs_per_row;
    const float* xr = x + row * ldx;
    const int64_t e0 = seg * 1024;

    constexpr int H = 1 << (BITS - 1);
    const float half_L = 0.5f * (float)((1 << BITS) - 1);
    const float lo = (float)(-H), hi = (float)H - 0.5f;
    const float inv = inverse_scale(__ldg(scale + (per_row ? row : 0)));
    const int64_t remaining = k - e0;                       // > 0 only for words that hold data

    if (vec_ok && remaining >= 1024) {
        float* mine = stage[threadIdx.x >> 5];
        const float* src = xr + e0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int chunk = 32 * i + lane;                // 16-byte chunk of the segment
            copy_async_16(mine + (chunk >> 3) * kStageRow + (chunk & 7) * 4, src + chunk * 4);
        }
        copy_async_wait_all();
        __syncwarp();
        uint32_t word[BITS];
        staged_lane_words<BITS, ACT>(mine + lane * kStageRow, inv, two, word);
        uint32_t* dst = planes + row * rw + seg * 32 + lane;
        const int64_t plane_stride = rows * rw;
#pragma unroll
        for (int p = 0; p < BITS; ++p) dst[p * plane_stride] = word[p];
        return;
    }

    uint32_t mine[BITS];
#pragma unroll
    for (int p = 0; p < BITS; ++p) mine[p] = 0u;
    const int steps = remaining >= 1024 ? 32 : (int)((remaining + 31) / 32);   // warp-uniform
    for (int j0 = 0; j0 < steps; j0 += 8) {
        float v[8];
        bool ok[8];
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
            const int64_t idx = e0 + (int64_t)(j0 + jj) * 32 + lane;
            ok[jj] = idx < k;
            v[jj] = ok[jj] ? __ldg(xr + idx) : 0.0f;
        }
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
            const int u = ok[jj] ? level_index<ACT>(v[jj], inv, half_L, lo, hi, H) : 0;
#pragma unroll
            for (int p = 0; p < BITS; ++p) {
                const uint32_t word = __ballot_sync(0xffffffffu, (u >> p) & 1);
                if (lane == j0 + jj) mine[p] = word;
            }
        }
    }
    const int64_t word_idx = seg * 32 + lane;
    if (word_idx < rw) {
#pragma unroll
        for (int p = 0; p < BITS; ++p) planes[((int64_t)p * rows + row) * rw + word_idx] = mine[p];
    }
}

// ------------------------------------------------------------------------------------------
// Per-row range AND encode in one pass over HBM (weights with one range per output channel): one
// CTA stages a whole row in shared memory (the same 32 x 36 layout per 1024-element segment),
// takes the row's maximum there, publishes it, and encodes the segments from the staged copy, so
// the row is read from HBM once instead of twice.  Rows of up to kRangedMaxK elements.
// ------------------------------------------------------------------------------------------
constexpr int64_t kRangedMaxK = 48 * 1024;                      // 48 segments x 4608 bytes = 216 KiB staged

template <int BITS, int ACT>
__global__ void __launch_bounds__(kEncodeThreads)
encode_rows_ranged_kernel(const float* __restrict__ x, int64_t rows, int64_t k, int64_t ldx,
                          float* __restrict__ scale_out, uint32_t* __restrict__ planes, int64_t rw, uint32_t two) {
    extern __shared__ __align__(16) float staged[];             // [segments][32 * kStageRow]
    __shared__ float warp_max[kEncodeThreads / 32];
    chain_entry();
    const int64_t row = blockIdx.x;
    const float* xr = x + row * ldx;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t full_chunks = k / 4;                          // 16-byte chunks that lie wholly inside the row
    const int segs = (int)ceil_div(k, 1024);
    // stage: chunk c -> segment c / 256, row (c % 256) / 8 of the segment, 16-byte slot (c % 8)
    for (int64_t c = tid; c < full_chunks; c += kEncodeThreads) {
        const int cc = (int)(c & 255);
        copy_async_16(staged + (c >> 8) * (32 * kStageRow) + (cc >> 3) * kStageRow + (cc & 7) * 4, xr + c * 4);
    }
    // the ragged end of the row and the rest of its last segment: plain stores (zeros past the end)
    for (int64_t e = full_chunks * 4 + tid; e < (int64_t)segs * 1024; e += kEncodeThreads) {
        const int ee = (int)(e & 1023);
        staged[(e >> 10) * (32 * kStageRow) + (ee >> 5) * kStageRow + (ee & 31)] = e < k ? __ldg(xr + e) : 0.0f;
    }
    copy_async_wait_all();
    __syncthreads();
    // range of the row
    float m = 0.0f;
    for (int64_t c = tid; c < (int64_t)segs * 256; c += kEncodeThreads) {
        const int cc = (int)(c & 255);
        const float4 v = *reinterpret_cast<const float4*>(staged + (c >> 8) * (32 * kStageRow) + (cc >> 3) * kStageRow + (cc & 7) * 4);
        if (ACT == MPQ_ACT_HRELU) m = fmaxf(m, fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)));
        else m = fmaxf(m, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) warp_max[warp] = m;
    __syncthreads();
    m = warp_max[0];
#pragma unroll
    for (int w = 1; w < kEncodeThreads / 32; ++w) m = fmaxf(m, warp_max[w]);
    if (tid == 0) scale_out[row] = m;
    const float inv = inverse_scale(m);
    // encode: warp w takes segments w, w + 8, ...; lane L owns word L of every plane of the segment
    constexpr int H = 1 << (BITS - 1);
    const float half_L = 0.5f * (float)((1 << BITS) - 1);
    const float lo = (float)(-H), hi = (float)H - 0.5f;
    const int64_t plane_stride = rows * rw;
    for (int seg = warp; seg < segs; seg += kEncodeThreads / 32) {
        const float* lane_row = staged + (size_t)seg * (32 * kStageRow) + lane * kStageRow;
        const int64_t e0 = (int64_t)seg * 1024 + 32 * lane;    // first element of this lane's word
        uint32_t word[BITS];
        if (e0 + 32 <= k) {
            staged_lane_words<BITS, ACT>(lane_row, inv, two, word);
        } else {                                                // the word holding the end of the row, and pad words
#pragma unroll
            for (int p = 0; p < BITS; ++p) word[p] = 0u;
            for (int t = 0; t < 32 && e0 + t < k; ++t) {
                const uint32_t u = (uint32_t)level_index<ACT>(lane_row[t], inv, half_L, lo, hi, H);
#pragma unroll
                for (int p = 0; p < BITS; ++p) word[p] |= ((u >> p) & 1u) << t;
            }
        }
        const int64_t word_idx = (int64_t)seg * 32 + lane;
        if (word_idx < rw) {
#pragma unroll
            for (int p = 0; p < BITS; ++p) planes[p * plane_stride + row * rw + word_idx] = word[p];
        }
    }
}

// ------------------------------------------------------------------------------------------
// NCHW activations -> planes[bits][N][H][W][C/32].  A warp takes 32 pixels x G adjacent channel
// words (G = 1, 2 or 4: all of them for C = 32 and 64): lane = pixel, so each channel read is a
// coalesced 128-byte row of one channel -- the 32 reads of a word are all in flight together --
// and every lane builds the G words of its own pixel (channel c -> bit c) and stores them as one
// 4-, 8- or 16-byte vector, so that the warp's stores cover whole 32-byte sectors.
// ------------------------------------------------------------------------------------------
constexpr int kNchwPerSm = 3;          // 80 registers per thread: 32 loads in flight and the words built so far

template <int BITS, int ACT, int G>
__global__ void __launch_bounds__(kEncodeThreads, kNchwPerSm)
encode_nchw_kernel(const float* __restrict__ x, int N, int C, int64_t HW,
                   const float* __restrict__ scale, uint32_t* __restrict__ planes,
                   int64_t pix_blocks, int64_t total_warps, uint32_t two) {
    chain_entry();
    const int64_t warp = (int64_t)blockIdx.x * (kEncodeThreads / 32) + (threadIdx.x >> 5);
    if (warp >= total_warps) return;
    const int lane = threadIdx.x & 31;
    const int Cw = C / 32;
    const int groups = Cw / G;
    const int64_t pb = warp % pix_blocks;
    const int64_t rest = warp / pix_blocks;
    const int cw0 = (int)(rest % groups) * G;
    const int64_t n = rest / groups;
    const int64_t pixel = pb * 32 + lane;
    if (pixel >= HW) return;

    constexpr int H = 1 << (BITS - 1);
    const float half_L = 0.5f * (float)((1 << BITS) - 1);
    const float lo = (float)(-H), hi = (float)H - 0.5f;
    const float inv = inverse_scale(__ldg(scale));

    uint32_t word[G][BITS];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const float* base = x + ((n * C + (int64_t)(cw0 + g) * 32) * HW + pixel);
        float v[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) v[c] = __ldg(base + (int64_t)c * HW);
        float probe = 0.0f;                                 // turns NaN if any element is NaN
        if (ACT == MPQ_ACT_HTANH) {
#pragma unroll
            for (int c = 0; c < 32; c += 2) probe = fmaf(v[c], v[c + 1], probe);
        }
        if constexpr (BITS >= kByteBuilderFromBits) {
            LaneBytes<BITS, ACT> lb;
#pragma unroll
            for (int c = 0; c < 32; ++c) lb.set(c, level_fraction<BITS, ACT>(v[c], inv, half_L));
            lb.words(word[g]);
        } else {
            LaneWords<BITS, ACT> lw;
            lw.clear();
#pragma unroll
            for (int c = 31; c >= 0; --c) lw.push(level_fraction<BITS, ACT>(v[c], inv, half_L), two);
#pragma unroll
            for (int p = 0; p < BITS; ++p) word[g][p] = lw.word(p);
        }
        if (ACT == MPQ_ACT_HTANH && (probe != probe || inv == 0.0f || inv == __int_as_float(0x7f800000))) {
#pragma unroll
            for (int p = 0; p < BITS; ++p) word[g][p] = 0u;
            for (int c = 0; c < 32; ++c) {
                const uint32_t u = (uint32_t)level_index<ACT>(__ldg(base + (int64_t)c * HW), inv, half_L, lo, hi, H);
#pragma unroll
                for (int p = 0; p < BITS; ++p) word[g][p] |= ((u >> p) & 1u) << c;
            }
        }
    }
#pragma unroll
    for (int p = 0; p < BITS; ++p) {
        uint32_t* dst = planes + (((int64_t)p * N + n) * HW + pixel) * Cw + cw0;     // G words: G * 4-byte aligned
        if constexpr (G == 4) *reinterpret_cast<uint4*>(dst) = make_uint4(word[0][p], word[1][p], word[2][p], word[3][p]);
        else if constexpr (G == 2) *reinterpret_cast<uint2*>(dst) = make_uint2(word[0][p], word[1][p]);
        else dst[0] = word[0][p];
    }
}

// ------------------------------------------------------------------------------------------
// OIHW weights -> planes[bits][O][row_words(KH*KW*C)], k ordered (kh, kw, c); plus tap sums.
// Weights are encoded once, offline: one thread per output word, no tuning.
// ------------------------------------------------------------------------------------------
template <int ACT>
__device__ __forceinline__ int level_index_rt(float x, float inv, int bits) {
    const int H = 1 << (bits - 1);
    return level_index<ACT>(x, inv, 0.5f * (float)((1 << bits) - 1), (float)(-H), (float)H - 0.5f, H);
}

// The row of output channel o holds `taps` filter taps; tap t of the row is tap map.from[t] of the
// filter's KH*KW (the identity for a convolution, one phase's taps for a deconvolution).
struct TapMap {
    int filter_taps;          // KH * KW
    int from[16];
};
static TapMap identity_taps(int taps) {
    TapMap m;
    m.filter_taps = taps;
    for (int t = 0; t < 16; ++t) m.from[t] = t < taps ? t : 0;
    return m;
}

__global__ void encode_oihw_kernel(const float* __restrict__ w, int O, int C, int taps, const TapMap map,
                                   const float* __restrict__ scale, int per_row, int bits,
                                   uint32_t* __restrict__ planes, int64_t rw) {
    const int64_t id = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= (int64_t)O * rw) return;
    const int64_t o = id / rw;
    const int64_t word = id % rw;
    const int64_t K = (int64_t)taps * C;
    const float inv = inverse_scale(__ldg(scale + (per_row ? o : 0)));
    uint32_t out[kMaxBits];
    for (int p = 0; p < kMaxBits; ++p) out[p] = 0u;
    for (int t = 0; t < 32; ++t) {
        const int64_t kidx = word * 32 + t;
        if (kidx >= K) break;
        const int64_t tap = kidx / C, c = kidx % C;
        const uint32_t u = (uint32_t)level_index_rt<MPQ_ACT_HTANH>(__ldg(w + (o * C + c) * map.filter_taps + map.from[tap]), inv, bits);
        for (int p = 0; p < kMaxBits; ++p) out[p] |= ((u >> p) & 1u) << t;
    }
    for (int p = 0; p < bits; ++p) planes[((int64_t)p * O + o) * rw + word] = out[p];
}

__global__ void tap_sums_kernel(const float* __restrict__ w, int O, int C, int taps, const TapMap map,
                                const float* __restrict__ scale, int per_row, int bits,
                                int32_t* __restrict__ tap_sums) {
    const int64_t id = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= (int64_t)O * taps) return;
    const int64_t tap = id / O, o = id % O;
    const float inv = inverse_scale(__ldg(scale + (per_row ? o : 0)));
    const int L = (1 << bits) - 1;
    int32_t s = 0;
    for (int c = 0; c < C; ++c)
        s += 2 * level_index_rt<MPQ_ACT_HTANH>(__ldg(w + (o * C + c) * map.filter_taps + map.from[tap]), inv, bits) - L;
    tap_sums[tap * O + o] = s;
}

__global__ void add_relu_kernel(const float* __restrict__ a, const float* __restrict__ b,
                                float* __restrict__ y, int64_t n) {
    chain_entry();
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        const float v = b ? __fadd_rn(a[i], b[i]) : a[i];
        y[i] = fmaxf(v, 0.0f);
    }
}

template <template <int, int> class Launcher, typename... Args>
static int dispatch_bits_act(int bits, int act, Args... args) {
#define MPQ_CASE(B)                                                              \
    case B:                                                                      \
        return act == MPQ_ACT_HRELU ? Launcher<B, MPQ_ACT_HRELU>::run(args...)   \
                                    : Launcher<B, MPQ_ACT_HTANH>::run(args...);
    switch (bits) {
        MPQ_CASE(1) MPQ_CASE(2) MPQ_CASE(3) MPQ_CASE(4) MPQ_CASE(5) MPQ_CASE(6) MPQ_CASE(7) MPQ_CASE(8)
    }
#undef MPQ_CASE
    return MPQ_ERR_UNSUPPORTED;
}

template <int BITS, int ACT>
struct EncodeRowsLauncher {
    static int run(const float* x, int64_t rows, int64_t k, int64_t ldx, const float* scale, int per_row,
                   uint32_t* planes, cudaStream_t st) {
        const int64_t rw = row_words(k);
        const int64_t segs = ceil_div(rw, 32);
        const int64_t warps = rows * segs;
        const int64_t blocks = ceil_div(warps, kEncodeThreads / 32);
        if (blocks > 0x7fffffffLL) return MPQ_ERR_BAD_SHAPE;
        // the lane-local path copies 16-byte chunks: every row start must be 16-byte aligned
        const int vec_ok = aligned16(x) && (ldx % 4 == 0 || rows == 1);
        return launch_chained(encode_rows_kernel<BITS, ACT>, (unsigned)blocks, kEncodeThreads, 0, st,
                              x, rows, k, ldx, scale, per_row, planes, rw, segs, vec_ok, 2u);
    }
};

template <int BITS, int ACT>
struct EncodeNchwLauncher {
    template <int G>
    static int go(const float* x, int N, int C, int64_t HW, const float* scale, uint32_t* planes, cudaStream_t st) {
        const int64_t pix_blocks = ceil_div(HW, 32);
        const int64_t warps = pix_blocks * (C / 32 / G) * N;
        const int64_t blocks = ceil_div(warps, kEncodeThreads / 32);
        if (blocks > 0x7fffffffLL) return MPQ_ERR_BAD_SHAPE;
        return launch_chained(encode_nchw_kernel<BITS, ACT, G>, (unsigned)blocks, kEncodeThreads, 0, st,
                              x, N, C, HW, scale, planes, pix_blocks, warps, 2u);
    }
    static int run(const float* x, int N, int C, int64_t HW, const float* scale, uint32_t* planes, cudaStream_t st) {
        // C is 32, 64 or a multiple of 128 (checked by the caller): 1, 2 or 4 words per lane
        return C == 32 ? go<1>(x, N, C, HW, scale, planes, st)
             : C == 64 ? go<2>(x, N, C, HW, scale, planes, st) : go<4>(x, N, C, HW, scale, planes, st);
    }
};

template <int BITS, int ACT>
struct EncodeRangedLauncher {
    static int run(const float* x, int64_t rows, int64_t k, int64_t ldx, float* scale_out, uint32_t* planes, cudaStream_t st) {
        const int64_t rw = row_words(k);
        const size_t smem = (size_t)ceil_div(k, 1024) * 32 * kStageRow * sizeof(float);
        auto kern = encode_rows_ranged_kernel<BITS, ACT>;
        static PerDeviceOnce configured;
        if (configured.raise_smem_limit(kern, (size_t)ceil_div(kRangedMaxK, 1024) * 32 * kStageRow * sizeof(float)) != MPQ_OK)
            return MPQ_ERR_CUDA;
        if (rows > 0x7fffffffLL) return MPQ_ERR_BAD_SHAPE;
        return launch_chained(kern, (unsigned)rows, kEncodeThreads, smem, st, x, rows, k, ldx, scale_out, planes, rw, 2u);
    }
};

}  // namespace mpq

using namespace mpq;

extern "C" int mpq_absmax(const float* x, int64_t rows, int64_t k, int64_t ldx, int mode, int act,
                          float* scale_out, void* stream) {
    if (!x || !scale_out) return MPQ_ERR_NULL;
    if (rows <= 0 || k <= 0 || ldx < k) return MPQ_ERR_BAD_SHAPE;
    if ((mode != MPQ_SCALE_PER_TENSOR && mode != MPQ_SCALE_PER_ROW) ||
        (act != MPQ_ACT_HTANH && act != MPQ_ACT_HRELU)) return MPQ_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    const int per_row = mode == MPQ_SCALE_PER_ROW;
    // zeroed by a kernel of the chain rather than a memset node: the range kernel's blocks are then
    // already resident (waiting at their chain entry) when the zeroes land
    {
        const int64_t n = per_row ? rows : 1;
        const int rc = launch_chained_as(true, zero_floats_kernel, (unsigned)min(ceil_div(n, 256), (int64_t)1024), 256, 0, st, scale_out, n);
        if (rc != MPQ_OK) return rc;
    }
    if (!per_row && ldx == k) { k = rows * k; ldx = k; rows = 1; }   // contiguous tensor: one long row
    const int64_t chunks = ceil_div(k, kAbsmaxChunk);
    const int64_t total = rows * chunks;
    const int sms = sm_count();
    if (sms <= 0) return MPQ_ERR_CUDA;
    const int64_t blocks = min(total, (int64_t)sms * kAbsmaxPerSm);
    const bool vec4 = aligned16(x) && (ldx % 4 == 0);
#define MPQ_LAUNCH(A, V) launch_chained_as(blocks == (int64_t)sms * kAbsmaxPerSm, absmax_kernel<A, V>, (unsigned)blocks, kAbsmaxThreads, 0, st, x, k, ldx, chunks, total, per_row, scale_out)
    if (act == MPQ_ACT_HRELU) return vec4 ? MPQ_LAUNCH(MPQ_ACT_HRELU, true) : MPQ_LAUNCH(MPQ_ACT_HRELU, false);
    return vec4 ? MPQ_LAUNCH(MPQ_ACT_HTANH, true) : MPQ_LAUNCH(MPQ_ACT_HTANH, false);
#undef MPQ_LAUNCH
}

extern "C" int mpq_encode(const float* x, int64_t rows, int64_t k, int64_t ldx,
                          const float* scale, int mode, int act, int bits,
                          uint32_t* planes, void* stream) {
    if (!x || !scale || !planes) return MPQ_ERR_NULL;
    if (rows <= 0 || k <= 0 || ldx < k) return MPQ_ERR_BAD_SHAPE;
    if (!bits_ok(bits) || (mode != MPQ_SCALE_PER_TENSOR && mode != MPQ_SCALE_PER_ROW) ||
        (act != MPQ_ACT_HTANH && act != MPQ_ACT_HRELU)) return MPQ_ERR_UNSUPPORTED;
    if (!aligned16(planes)) return MPQ_ERR_ALIGN;
    return dispatch_bits_act<EncodeRowsLauncher>(bits, act, x, rows, k, ldx, scale,
                                                 (int)(mode == MPQ_SCALE_PER_ROW), planes, (cudaStream_t)stream);
}

extern "C" int mpq_encode_ranged(const float* x, int64_t rows, int64_t k, int64_t ldx, int act, int bits,
                                 float* scale_out, uint32_t* planes, void* stream) {
    if (!x || !scale_out || !planes) return MPQ_ERR_NULL;
    if (rows <= 0 || k <= 0 || ldx < k) return MPQ_ERR_BAD_SHAPE;
    if (!bits_ok(bits) || (act != MPQ_ACT_HTANH && act != MPQ_ACT_HRELU)) return MPQ_ERR_UNSUPPORTED;
    if (!aligned16(planes)) return MPQ_ERR_ALIGN;
    // one pass when a row fits the staging buffer and its start is 16-byte aligned; else range, then encode
    if (k <= kRangedMaxK && aligned16(x) && (ldx % 4 == 0 || rows == 1))
        return dispatch_bits_act<EncodeRangedLauncher>(bits, act, x, rows, k, ldx, scale_out, planes, (cudaStream_t)stream);
    const int rc = mpq_absmax(x, rows, k, ldx, MPQ_SCALE_PER_ROW, act, scale_out, stream);
    if (rc != MPQ_OK) return rc;
    return mpq_encode(x, rows, k, ldx, scale_out, MPQ_SCALE_PER_ROW, act, bits, planes, stream);
}

static bool conv_channels_ok(int C) { return C == 32 || C == 64 || (C > 0 && C % 128 == 0); }

extern "C" int mpq_encode_nchw(const float* x, int N, int C, int H, int W, const float* scale, int act,
                               int bits, uint32_t* planes, void* stream) {
    if (!x || !scale || !planes) return MPQ_ERR_NULL;
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0) return MPQ_ERR_BAD_SHAPE;
    if (!bits_ok(bits) || !conv_channels_ok(C) || (act != MPQ_ACT_HTANH && act != MPQ_ACT_HRELU)) return MPQ_ERR_UNSUPPORTED;
    if (!aligned16(planes)) return MPQ_ERR_ALIGN;
    return dispatch_bits_act<EncodeNchwLauncher>(bits, act, x, N, C, (int64_t)H * W, scale, planes, (cudaStream_t)stream);
}

static int encode_filter_rows(const float* w, int O, int C, int taps, const TapMap& map, const float* scale,
                              int per_row, int bits, uint32_t* planes, int32_t* tap_sums, cudaStream_t st) {
    const int64_t rw = row_words((int64_t)taps * C);
    encode_oihw_kernel<<<(unsigned)ceil_div((int64_t)O * rw, 128), 128, 0, st>>>(w, O, C, taps, map, scale, per_row, bits, planes, rw);
    if (launch_status() != MPQ_OK) return MPQ_ERR_CUDA;
    tap_sums_kernel<<<(unsigned)ceil_div((int64_t)O * taps, 128), 128, 0, st>>>(w, O, C, taps, map, scale, per_row, bits, tap_sums);
    return launch_status();
}

extern "C" int mpq_encode_oihw(const float* w, int O, int C, int KH, int KW, const float* scale, int mode,
                               int bits, uint32_t* planes, int32_t* tap_sums, void* stream) {
    if (!w || !scale || !planes || !tap_sums) return MPQ_ERR_NULL;
    if (O <= 0 || C <= 0 || KH <= 0 || KW <= 0) return MPQ_ERR_BAD_SHAPE;
    if (!bits_ok(bits) || !conv_channels_ok(C) || (mode != MPQ_SCALE_PER_TENSOR && mode != MPQ_SCALE_PER_ROW)) return MPQ_ERR_UNSUPPORTED;
    if (!aligned16(planes)) return MPQ_ERR_ALIGN;
    if (KH * KW > 16) return MPQ_ERR_UNSUPPORTED;
    return encode_filter_rows(w, O, C, KH * KW, identity_taps(KH * KW), scale, mode == MPQ_SCALE_PER_ROW, bits,
                              planes, tap_sums, (cudaStream_t)stream);
}

extern "C" int64_t mpq_deconv_weight_words(int O, int C, int KH, int KW, int stride, int bits) {
    if (O <= 0 || C <= 0 || KH <= 0 || KW <= 0 || !bits_ok(bits) || !deconv_filter_ok(KH, KW, stride)) return 0;
    DeconvPhase ph[4];
    return deconv_phases(O, C, KH, KW, stride, bits, ph);
}

extern "C" int mpq_encode_deconv_weights(const float* w, int O, int C, int KH, int KW, int stride,
                                         const float* scale, int mode, int bits,
                                         uint32_t* planes, int32_t* tap_sums, void* stream) {
    if (!w || !scale || !planes || !tap_sums) return MPQ_ERR_NULL;
    if (O <= 0 || C <= 0 || KH <= 0 || KW <= 0) return MPQ_ERR_BAD_SHAPE;
    if (!bits_ok(bits) || !conv_channels_ok(C) || !deconv_filter_ok(KH, KW, stride) ||
        (mode != MPQ_SCALE_PER_TENSOR && mode != MPQ_SCALE_PER_ROW)) return MPQ_ERR_UNSUPPORTED;
    if (!aligned16(planes)) return MPQ_ERR_ALIGN;
    DeconvPhase ph[4];
    deconv_phases(O, C, KH, KW, stride, bits, ph);
    for (int g = 0; g < stride * stride; ++g) {
        TapMap map;
        map.filter_taps = KH * KW;
        for (int t = 0; t < 16; ++t) map.from[t] = 0;
        for (int t_h = 0; t_h < ph[g].T_h; ++t_h)
            for (int t_w = 0; t_w < ph[g].T_w; ++t_w)
                map.from[t_h * ph[g].T_w + t_w] = (ph[g].r_h + stride * t_h) * KW + ph[g].r_w + stride * t_w;
        const int rc = encode_filter_rows(w, O, C, ph[g].T_h * ph[g].T_w, map, scale, mode == MPQ_SCALE_PER_ROW, bits,
                                          planes + ph[g].word_offset, tap_sums + (int64_t)ph[g].tap_start * O,
                                          (cudaStream_t)stream);
        if (rc != MPQ_OK) return rc;
    }
    return MPQ_OK;
}

extern "C" int mpq_add_relu(const float* a, const float* b, float* y, int64_t n, void* stream) {
    if (!a || !y) return MPQ_ERR_NULL;
    if (n <= 0) return MPQ_ERR_BAD_SHAPE;
    const int sms = sm_count();
    if (sms <= 0) return MPQ_ERR_CUDA;
    const int64_t blocks = min((int64_t)sms * 16, ceil_div(n, 256));
    return launch_chained(add_relu_kernel, (unsigned)blocks, 256, 0, (cudaStream_t)stream, a, b, y, n);
}
