// Branch-fused binary GEMM / implicit-im2col convolution on packed {-1,+1} bit-planes.
//
// One kernel computes, for a tile of outputs, ALL a_bits x w_bits binary-branch products of
// Eq. 7-10 at once: every bit-plane of the two operand tiles is staged once in shared memory
// (cp.async, multi-stage ring) and each thread accumulates
//     S[r][c] = sum_{i,j} 2^(i+j) * popcount(A_i[r] xor B_j[c])
// for a small register tile of outputs, then applies the decoder
//     acc = L_a L_w k - 2 S,   out = float(acc) * alpha[c]           (Eq. 18)
// in the store.  The arithmetic is XOR, bitwise full adders (carry-save) and POPC on the integer
// pipes, with the weighted adds as integer multiply-adds: the B200's 5th-generation tensor cores
// have no 1-bit kind, and the legacy 1-bit mma.sync form measured slower than this path.
//
// Roles.  The "held" operand (HB planes, TH items per thread) lives in registers as 128-bit
// k-quads; the "streamed" operand (SB planes, TS items per thread) is read quad by quad from
// shared memory.  Threads form a 16 x 16 grid: ty indexes held items, tx streamed items, so
// streamed reads are conflict-free 16-byte accesses and held reads are broadcasts.
//   GEMM mode: held = A rows (activations), streamed = B rows (weights / output columns).
//   CONV mode: held = weight rows (output channels), streamed = output pixels, gathered on the
//              fly from planes[bits][N][H][W][C/32]; consecutive tx = consecutive pixels, which
//              is the contiguous direction of the NCHW output.
#pragma once
#include <type_traits>
#include "mpq_common.cuh"

namespace mpq {

enum { kModeGemm = 0, kModeConv = 1 };

struct BranchParams {
    const uint32_t* held;      // GEMM: A planes [HB][m][rw];      CONV: weight planes [HB][O][rw]
    const uint32_t* streamed;  // GEMM: B planes [SB][n][rw];      CONV: x planes [SB][N][H][W][Cw]
    int64_t held_rows;         // GEMM: m (rows computed by this launch);  CONV: O
    int64_t held_plane_rows;   // rows between two planes of the held operand in memory (>= held_rows)
    int64_t streamed_rows;     // GEMM: n;  CONV: N*Ho*Wo
    int64_t rw;                // words per packed row (GEMM: both operands; CONV: weight rows)
    int64_t k;                 // elements per dot product (CONV: KH*KW*C)
    int32_t* out_i32;
    float* out_f32;
    int64_t ldc;               // GEMM only
    const float* a_scale;      // activation range, 1 value (may be null when out_f32 is null)
    const float* w_scale;      // weight range, 1 or per-output-channel values
    int w_per_row;
    // CONV only
    int N, C, H, W, O, KH, KW, stride, pad, Ho, Wo, Cw;
    int granule;               // words gathered per copy: 1 (C=32), 2 (C=64) or 4 (C % 128 == 0)
    int granule_shift;         // log2(4 / granule): copies per k-quad
    int tap_granules;          // copies per filter tap = Cw / granule
    uint32_t tap_magic;        // ceil(2^32 / tap_granules): copy index / tap_granules by one multiply
    const int32_t* tap_sums;   // [KH*KW][O]
    const float* bias;         // optional: one value per output channel / column, added first (one rounded add)
    const float* residual;     // optional: added to the scaled output (same layout as the output), one rounded add
    int relu;                  // store max(value, 0)
    float* out_max;            // CONV, optional: raised (never lowered) to the largest stored max(value, 0)
    // CONV, optional: the consumer's Encoder folded into the store.  The value that would be stored
    // as fp32 is quantized with the consumer's range and written as packed planes
    // next_planes[next_bits][N][Ho][Wo][O/32] (the layout mpq_encode_nchw produces for that tensor).
    uint32_t* next_planes;
    const float* next_scale;   // 1 value: the consumer's range, known before this layer runs
    int next_bits, next_act;
    int half_tail;             // CONV: the last k-quad of a row holds data in its first two words only
    int tap_offset[16];        // CONV: dh * W + dw of filter tap t (pixels from the window origin); 0 past the last tap
    // CONV: the pixels of this launch form a sub_h x sub_w grid per image.  Grid point (a, b) has its window
    // origin at input pixel (a * in_step + in_h0, b * in_step + in_w0), tap t reads the pixel (tap_dh[t],
    // tap_dw[t]) away from it, and the result goes to output pixel (out_h0 + a * out_step, out_w0 + b * out_step)
    // of the Ho x Wo output.  A convolution: in_step = stride, in_h0 = -pad, taps (kh, kw), the whole output.
    // A deconvolution runs one launch per output phase: in_step = 1, taps (-th, -tw), out_step = stride.
    int sub_h, sub_w, in_step, in_h0, in_w0, out_h0, out_w0, out_step;
    int window3x3;             // taps are (kh, kw) of a 3 x 3 window that sticks out by at most one pixel
    signed char tap_dh[16], tap_dw[16];
    uint32_t pow2[24];         // pow2[e] = 2^e: branch weights read from the constant bank, so that
                               // "popcount * 2^e + acc" stays one integer multiply-add (FMA pipe)
};

__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gsrc, bool valid) {
    const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    const int src_bytes = valid ? 16 : 0;   // 0 => the 16 bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(gsrc), "r"(src_bytes) : "memory");
}
template <int BYTES>
__device__ __forceinline__ void cp_async_small(void* smem_dst, const void* gsrc, bool valid) {
    const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    const int src_bytes = valid ? BYTES : 0;
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2, %3;\n" ::"r"(dst), "l"(gsrc), "n"(BYTES), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

// fp32 value of one GEMM output: decoder scale (Eq. 18), then the optional glue of a chained layer
// (bias, residual, max(.,0)), one rounded operation each.
__device__ __forceinline__ float gemm_store_value(const BranchParams& p, int32_t v, float alpha, int64_t row, int64_t col) {
    float f = __fmul_rn((float)v, alpha);
    if (p.bias) f = __fadd_rn(f, __ldg(p.bias + col));
    if (p.residual) f = __fadd_rn(f, __ldg(p.residual + row * p.ldc + col));
    if (p.relu) f = fmaxf(f, 0.0f);
    return f;
}

// ---- The branch products of one output over one k-quad, with carry-save compression ---------
// S += sum_{i,j} 2^(i+j) * popcount(h_i xor s_j) over the four words of a k-quad.  The 4*HB*SB
// xor words are grouped by weight exponent e = i + j ("level").  Within a level three words of
// equal weight are replaced by their bitwise sum (weight 2^e, one 3-input xor) and their bitwise
// carry (weight 2^(e+1), one 3-input majority) -- a full adder on 32 bit positions at once, since
// popc(a) + popc(b) + popc(c) = popc(a^b^c) + 2 popc(maj(a,b,c)).  Each such step trades one
// population count (the narrow pipe of the SM: 16 lanes per clock) for two logic operations
// (64 lanes per clock).  Spending about one adder per two xor words leaves half as many
// population counts as xor words, which balances the two pipes; the weighted add of each count
// is an integer multiply-add with 2^e taken from the constant bank, i.e. it runs on the FMA pipe.
// All counts and array sizes are compile-time constants; the arrays live in registers.
__host__ __device__ constexpr int pairs_at_level(int hb, int sb, int e) {
    int n = 0;
    for (int i = 0; i < hb; ++i) {
        const int j = e - i;
        if (j >= 0 && j < sb) ++n;
    }
    return n;
}
__device__ __forceinline__ uint32_t quad_word(const uint4& v, int c) {
    return c == 0 ? v.x : c == 1 ? v.y : c == 2 ? v.z : v.w;
}
// Full adder on 32 bit positions: each half is exactly one 3-input logic operation (written as
// lop3 with its truth table so that the compiler cannot split it into 2-input steps).
__device__ __forceinline__ uint32_t majority3(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xE8;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t parity3(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// One level's working set: up to BUDGET full adders, applied in rounds of disjoint triples
// (independent of one another, so they pipeline); what is left after the last round is counted.
template <int N, int BUDGET>
struct CarrySave {
    static constexpr int K = (N / 3 < BUDGET) ? N / 3 : BUDGET;            // adders of this round
    static constexpr int REST = N - 2 * K;                                  // words after the round
    static constexpr int TOTAL = K == 0 ? 0 : K + CarrySave<(K == 0 ? 0 : REST), (K == 0 ? 0 : BUDGET - K)>::TOTAL;
    // w: the N words; carry[at ...] receives the TOTAL carries; the counts go to acc with `weight`
    template <int NCARRY>
    __device__ __forceinline__ static void run(const uint32_t (&w)[N > 0 ? N : 1], uint32_t (&carry)[NCARRY], int at,
                                               uint32_t& acc, uint32_t weight) {
        if constexpr (K == 0) {
#pragma unroll
            for (int q = 0; q < N; ++q) acc = (uint32_t)__popc(w[q]) * weight + acc;
        } else {
            uint32_t r[REST];
#pragma unroll
            for (int q = 0; q < K; ++q) {
                const uint32_t a = w[3 * q], b = w[3 * q + 1], c = w[3 * q + 2];
                carry[at + q] = majority3(a, b, c);
                r[q] = parity3(a, b, c);
            }
#pragma unroll
            for (int q = 3 * K; q < N; ++q) r[K + q - 3 * K] = w[q];
            CarrySave<REST, BUDGET - K>::run(r, carry, at + K, acc, weight);
        }
    }
};
template <>
struct CarrySave<0, 0> {
    static constexpr int TOTAL = 0;
    template <int NCARRY>
    __device__ __forceinline__ static void run(const uint32_t (&)[1], uint32_t (&)[NCARRY], int, uint32_t&, uint32_t) {}
};

// Level E of one output: NC carries from the level below plus the fresh xor words of GQ k-quads;
// BUDGET is the number of full adders still to be spent on this and the higher levels (lower
// levels first).  h and s hold the planes of the GQ k-quads, quad-major: h[g * HB + i].
// NW = words of each k-quad that hold data (4, or 2 for the half-filled last quad of a short k).
template <int HB, int SB, int GQ, int NW, int E, int NC, int BUDGET>
struct BranchLevel {
    static constexpr int NF = NW * GQ * pairs_at_level(HB, SB, E);  // fresh xor words of this level
    static constexpr int N = NF + NC;
    using CS = CarrySave<N, (N >= 3 ? BUDGET : 0)>;
    static constexpr int K = CS::TOTAL;
    __device__ __forceinline__ static void run(const uint4 (&h)[GQ * HB], const uint4 (&s)[GQ * SB],
                                               const uint32_t (&carry_in)[NC > 0 ? NC : 1],
                                               uint32_t& acc, const BranchParams& p) {
        if constexpr (N > 0) {
            uint32_t w[N];
#pragma unroll
            for (int q = 0; q < NC; ++q) w[q] = carry_in[q];
            int n = NC;
#pragma unroll
            for (int g = 0; g < GQ; ++g) {
#pragma unroll
                for (int i = 0; i < HB; ++i) {
                    const int j = E - i;
                    if (j >= 0 && j < SB) {
#pragma unroll
                        for (int c = 0; c < NW; ++c) w[n++] = quad_word(h[g * HB + i], c) ^ quad_word(s[g * SB + j], c);
                    }
                }
            }
            uint32_t carry[K > 0 ? K : 1];
            CS::run(w, carry, 0, acc, p.pow2[E]);
            BranchLevel<HB, SB, GQ, NW, E + 1, K, BUDGET - K>::run(h, s, carry, acc, p);
        }
    }
};

template <int HB, int SB>
struct BranchTile {
    // k-quads whose xor words are compressed together.  A product with a 1-bit operand has one plane
    // pair per weight, i.e. only 4 xor words of equal weight per k-quad: a chain of adders over so few
    // words leaves 3 of 4 (1 x 1) or 5 of 8 (1 x 2) population counts standing where half is the
    // balance of the two pipes.  Two k-quads at once give every weight 8 words and the full budget of
    // adders finds work (1 x 2 bits: 0.84 -> 0.90 of the instruction-mix peak).  From 1 x 3 bits on the
    // gain (7 of 12 counts -> 6) no longer pays for the registers of a second k-quad.
    static constexpr int GQ = (HB * SB <= 2) ? 2 : 1;
    static constexpr int TH = ((HB == 1) ? 8 : (HB == 2) ? 4 : (HB <= 4) ? 2 : 1) / GQ;   // TH*HB*GQ <= 8 quads held
    static constexpr int KQ = (SB == 1) ? 8 : (SB == 2) ? 4 : (SB <= 4) ? 2 : 1;   // k-quads per stage
    static constexpr int STAGES = 3;
    static constexpr int THREADS = 256;
    // full adders per output and k-quad: half of the 4*HB*SB xor words balances the two pipes
    // (each adder costs two logic operations and saves one population count)
    static constexpr int CSA_BUDGET = 2 * HB * SB * GQ;
    // the k-quads of a stage are unrolled only while the loop body stays small enough for the
    // instruction cache (about 12 instructions per plane pair per output)
    static constexpr bool UNROLL_KQ = HB * SB <= 9;
    // CTAs per SM: the 64-wide tile (TS = 4) fits three times with 80 registers per thread as long
    // as the product has at most 16 plane pairs; a third resident CTA gives the two integer pipes
    // more warps to interleave (W4A4: 0.92 -> 0.94 of the instruction-mix peak).
    static constexpr int resident(int ts) { return (ts == 4 && HB * SB <= 16) ? 3 : 2; }
    // 16-byte chunks of one k-group's shared-memory region: its ring, or the 256 x TH x TS partial
    // sums it parks there at the end, whichever is larger
    __host__ __device__ static constexpr int group_quads(int ts, int ring_quads) {
        return ring_quads > TH * ts * 64 ? ring_quads : TH * ts * 64;
    }
};

// KS > 1 (GEMM only): the CTA has KS groups of 256 threads that share the tile and take its k-stages
// in turn (group g computes stages g, g + KS, ...), each with its own staging ring and its own
// barrier; at the end the groups' partial sums meet in shared memory and group 0 decodes and
// stores.  For grids of at most one CTA per multiprocessor (a fully-connected layer at small
// batch) this doubles the warps that interleave on the two integer pipes without splitting the
// tile any finer; the sums are integers, so the result is the same bit for bit.
template <int HB, int SB, int TS, int MODE, int KS = 1>
__global__ void __launch_bounds__(256 * KS, KS == 1 ? BranchTile<HB, SB>::resident(TS) : 1)
branch_kernel(const BranchParams p) {
    static_assert(KS == 1 || MODE == kModeGemm, "k-groups are a GEMM variant");
    using T = BranchTile<HB, SB>;
    constexpr int TH = T::TH, KQ = T::KQ, STAGES = T::STAGES;
    constexpr int BH = 16 * TH, BS = 16 * TS;
    constexpr int H_QUADS = HB * KQ * BH;          // 16-byte chunks per stage, held operand
    constexpr int S_QUADS = SB * KQ * BS;          // ... streamed operand
    constexpr int STAGE_QUADS = H_QUADS + S_QUADS;

    extern __shared__ uint4 smem_all[];
    __shared__ int row_n[MODE == kModeConv ? BS : 1];      // image index, or -1 for rows past the end
    __shared__ int row_pix[MODE == kModeConv ? BS : 1];    // (n*H + ih0)*W + iw0: pixel index of the window origin
    __shared__ int row_rem[MODE == kModeConv ? BS : 1];    // oh*Wo + ow: offset of the output pixel in its plane
    __shared__ unsigned row_out[MODE == kModeConv ? BS : 1];   // bit t set: filter tap t falls outside the image (all set: no such row)

    chain_entry();
    const int grp = KS == 1 ? 0 : (int)threadIdx.x / 256;                 // k-group of this thread
    const int tid = (int)threadIdx.x - 256 * grp;
    // the group's own region: its ring, which later parks its partial sums
    constexpr int GROUP_QUADS = T::group_quads(TS, STAGES * STAGE_QUADS);
    uint4* smem = smem_all + (size_t)grp * GROUP_QUADS;
    auto group_sync = [&]() {
        if (KS == 1) __syncthreads();
        else asm volatile("bar.sync %0, 256;" ::"r"(1 + grp) : "memory");
    };
    const int tx = tid & 15, ty = tid >> 4;
    const int64_t s_tiles = ceil_div(p.streamed_rows, BS);
    const int64_t s0 = (int64_t)(blockIdx.x % s_tiles) * BS;
    const int64_t h0 = (int64_t)(blockIdx.x / s_tiles) * BH;
    const int64_t kq_total = p.rw / 4;
    const int n_iters_all = (int)ceil_div(kq_total, KQ);
    const int n_iters = (n_iters_all - grp + KS - 1) / KS;               // k-stages grp, grp + KS, ... are mine

    if (MODE == kModeConv) {
        for (int r = tid; r < BS; r += 256) {
            const int64_t g = s0 + r;
            if (g < p.streamed_rows) {
                const uint32_t shw = (uint32_t)(p.sub_h * p.sub_w);  // pixels fit 32 bits (checked by the host)
                const int n = (int)((uint32_t)g / shw);
                const int srem = (int)((uint32_t)g % shw);
                const int ga = srem / p.sub_w, gb = srem % p.sub_w;
                const int ih0 = ga * p.in_step + p.in_h0;             // input coordinate of the window origin
                const int iw0 = gb * p.in_step + p.in_w0;
                row_n[r] = n;
                row_pix[r] = (n * p.H + ih0) * p.W + iw0;
                row_rem[r] = (p.out_h0 + ga * p.out_step) * p.Wo + p.out_w0 + gb * p.out_step;
                // taps outside the image, bit t = tap t.  A 3 x 3 window with padding of at most one pixel: only
                // its first / last row and column can stick out, whole rows or columns of taps at once
                unsigned outside = 0u;
                if (p.window3x3) {
                    outside = (ih0 < 0 ? 0x007u : 0u) | (ih0 + 2 >= p.H ? 0x1C0u : 0u) |
                              (iw0 < 0 ? 0x049u : 0u) | (iw0 + 2 >= p.W ? 0x124u : 0u);
                } else {
                    for (int t = 0; t < p.KH * p.KW; ++t) {
                        const int ih = ih0 + p.tap_dh[t], iw = iw0 + p.tap_dw[t];
                        if (ih < 0 || ih >= p.H || iw < 0 || iw >= p.W) outside |= 1u << t;
                    }
                }
                row_out[r] = outside;
            } else {
                row_n[r] = -1; row_pix[r] = 0; row_rem[r] = 0; row_out[r] = 0xFFFFFFFFu;   // never inside the image
            }
        }
        __syncthreads();
    }

    auto load_stage = [&](int stage, int64_t kq0) {
        uint4* hs = smem + (size_t)stage * STAGE_QUADS;
        uint4* ss = hs + H_QUADS;
        // held operand: [plane][kq][row], consecutive threads -> consecutive kq of one row
#pragma unroll
        for (int base = 0; base < H_QUADS; base += 256) {
            const int id = base + tid;
            if (H_QUADS % 256 == 0 || id < H_QUADS) {
                const int kq = id % KQ, row = (id / KQ) % BH, plane = id / (KQ * BH);
                const int64_t grow = h0 + row, gkq = kq0 + kq;
                const bool ok = grow < p.held_rows && gkq < kq_total;
                const uint32_t* src = ok ? p.held + ((int64_t)plane * p.held_plane_rows + grow) * p.rw + gkq * 4 : p.held;
                cp_async_16(hs + (plane * KQ + kq) * BH + row, src, ok);
            }
        }
        if (MODE == kModeGemm) {
#pragma unroll
            for (int base = 0; base < S_QUADS; base += 256) {
                const int id = base + tid;
                if (S_QUADS % 256 == 0 || id < S_QUADS) {
                    const int kq = id % KQ, row = (id / KQ) % BS, plane = id / (KQ * BS);
                    const int64_t grow = s0 + row, gkq = kq0 + kq;
                    const bool ok = grow < p.streamed_rows && gkq < kq_total;
                    const uint32_t* src = ok ? p.streamed + ((int64_t)plane * p.streamed_rows + grow) * p.rw + gkq * 4 : p.streamed;
                    cp_async_16(ss + (plane * KQ + kq) * BS + row, src, ok);
                }
            }
        } else {
            // implicit im2col: one copy = `granule` words of one tap of one pixel (never crosses a tap).
            // A thread owns one (pixel, k-quad) of the stage -- consecutive threads = consecutive
            // pixels, which are contiguous in memory for a fixed tap -- works out the tap and its
            // bounds once per copy position, and then only steps through the planes.  Index
            // arithmetic is kept to shifts, compile-time divisors and one multiply-high.
            const int G = p.granule;
            const int gs = p.granule_shift;                 // copies per k-quad = 1 << gs
            const int64_t plane_words = (int64_t)p.N * p.H * p.W * p.Cw;
            constexpr int PS = (KQ * BS >= 256) ? 1 : (256 / (KQ * BS) < SB ? 256 / (KQ * BS) : SB);   // plane split
            for (int item = tid; item < KQ * BS * PS; item += 256) {
                const int row = item % BS, kq = (item / BS) % KQ, ps = item / (BS * KQ);
                const int pix0 = row_pix[row];
                const unsigned inside = ~row_out[row] & ((1u << (p.KH * p.KW)) - 1u);   // bit t: tap t is in the image
                for (int part = 0; part < (1 << gs); ++part) {
                    const uint32_t copy = (uint32_t)(((kq0 + kq) << gs) + part);   // copy index along k
                    const uint32_t tap = p.tap_granules == 1 ? copy : __umulhi(copy, p.tap_magic);
                    const int cw = (int)(copy - tap * p.tap_granules) * G;
                    const bool ok = tap < 16u && ((inside >> tap) & 1u) != 0u;      // also false past the last tap
                    const uint32_t* src = p.streamed + (ok ? (int64_t)(pix0 + p.tap_offset[tap & 15u]) * p.Cw + cw + ps * plane_words : 0);
                    uint32_t* dst = reinterpret_cast<uint32_t*>(ss + (ps * KQ + kq) * BS + row) + part * G;
#pragma unroll
                    for (int plane = ps; plane < SB; plane += PS) {
                        if (G == 4) cp_async_16(dst, src, ok);
                        else if (G == 2) cp_async_small<8>(dst, src, ok);
                        else cp_async_small<4>(dst, src, ok);
                        if (ok) src += PS * plane_words;
                        dst += PS * KQ * BS * 4;
                    }
                }
            }
        }
    };

    uint32_t acc[TH][TS];
#pragma unroll
    for (int a = 0; a < TH; ++a)
#pragma unroll
        for (int b = 0; b < TS; ++b) acc[a][b] = 0u;

#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < n_iters) load_stage(s, (int64_t)(s * KS + grp) * KQ);
        cp_async_commit();
    }

    for (int it = 0; it < n_iters; ++it) {
        cp_async_wait<STAGES - 2>();
        group_sync();
        {
            const int nxt = it + STAGES - 1;
            if (nxt < n_iters) load_stage(nxt % STAGES, (int64_t)(nxt * KS + grp) * KQ);
            cp_async_commit();
        }
        const uint4* hs = smem + (size_t)(it % STAGES) * STAGE_QUADS;
        const uint4* ss = hs + H_QUADS;
        constexpr int GQ = T::GQ;
        auto one_group = [&](int kq, auto words_tag) {       // k-quads kq .. kq + GQ - 1 of this stage
            constexpr int NW = decltype(words_tag)::value;
            uint4 h[TH][GQ * HB];
#pragma unroll
            for (int a = 0; a < TH; ++a)
#pragma unroll
                for (int g = 0; g < GQ; ++g)
#pragma unroll
                    for (int i = 0; i < HB; ++i) h[a][g * HB + i] = hs[(i * KQ + kq + g) * BH + ty + 16 * a];
#pragma unroll
            for (int b = 0; b < TS; ++b) {
                uint4 s[GQ * SB];
#pragma unroll
                for (int g = 0; g < GQ; ++g)
#pragma unroll
                    for (int j = 0; j < SB; ++j) s[g * SB + j] = ss[(j * KQ + kq + g) * BS + tx + 16 * b];
                const uint32_t none[1] = {0u};
#pragma unroll
                for (int a = 0; a < TH; ++a)
                    BranchLevel<HB, SB, GQ, NW, 0, 0, (T::CSA_BUDGET * NW) / 4>::run(h[a], s, none, acc[a][b], p);
            }
        };
        // the last stage may hold fewer than KQ k-quads of data: skip the rest (they are all zero;
        // a group that is only partly live reads zero-filled quads, which add nothing)
        const int kq_live = (int)min((int64_t)KQ, kq_total - (int64_t)(it * KS + grp) * KQ);
        // (conv only) a short k whose last k-quad is half empty: that quad is computed on two words
        const bool half_tail = MODE == kModeConv && GQ == 1 && p.half_tail && it == n_iters - 1;
        using Full = std::integral_constant<int, 4>;
        using Half = std::integral_constant<int, (MODE == kModeConv && GQ == 1) ? 2 : 4>;
        if (T::UNROLL_KQ) {
#pragma unroll
            for (int kq = 0; kq < KQ; kq += GQ) {
                if (kq < kq_live) {
                    if (half_tail && kq == kq_live - 1) one_group(kq, Half());
                    else one_group(kq, Full());
                }
            }
        } else {
            const int full_quads = half_tail ? kq_live - 1 : kq_live;
#pragma unroll 1
            for (int kq = 0; kq < full_quads; kq += GQ) one_group(kq, Full());
            if (half_tail) one_group(kq_live - 1, Half());
        }
    }
    cp_async_wait<0>();

    if (KS > 1) {
        // the groups' partial sums meet in shared memory (each group parks its own in its own ring)
        group_sync();
        uint32_t* parked = reinterpret_cast<uint32_t*>(smem);
        if (grp != 0) {
#pragma unroll
            for (int a = 0; a < TH; ++a)
#pragma unroll
                for (int b = 0; b < TS; ++b) parked[(a * TS + b) * 256 + tid] = acc[a][b];
        }
        __syncthreads();
        if (grp != 0) return;
#pragma unroll
        for (int g = 1; g < KS; ++g) {
            const uint32_t* theirs = reinterpret_cast<const uint32_t*>(smem_all + (size_t)g * GROUP_QUADS);
#pragma unroll
            for (int a = 0; a < TH; ++a)
#pragma unroll
                for (int b = 0; b < TS; ++b) acc[a][b] += theirs[(a * TS + b) * 256 + tid];
        }
    }

    // ---- decoder: acc = L_a L_w k - 2 S, then the fused scale of Eq. 18 -------------------
    constexpr uint32_t LL = (uint32_t)(((1 << HB) - 1) * ((1 << SB) - 1));
    const uint32_t full = LL * (uint32_t)p.k;
    const bool want_f32 = p.out_f32 != nullptr || p.next_planes != nullptr;
    // activation bits: GEMM held = A; CONV streamed = x
    constexpr int A_BITS = (MODE == kModeGemm) ? HB : SB;
    constexpr int W_BITS = (MODE == kModeGemm) ? SB : HB;
    float fa = 0.0f;
    if (want_f32) fa = __fdiv_rn(__ldg(p.a_scale), (float)((1 << A_BITS) - 1));
    const float Lw = (float)((1 << W_BITS) - 1);

    if (MODE == kModeGemm) {
#pragma unroll
        for (int b = 0; b < TS; ++b) {
            const int64_t col = s0 + tx + 16 * b;
            if (col >= p.streamed_rows) continue;
            float alpha = 0.0f;
            if (want_f32) alpha = __fmul_rn(fa, __fdiv_rn(__ldg(p.w_scale + (p.w_per_row ? col : 0)), Lw));
#pragma unroll
            for (int a = 0; a < TH; ++a) {
                const int64_t row = h0 + ty + 16 * a;
                if (row >= p.held_rows) continue;
                const int32_t v = (int32_t)(full - 2u * acc[a][b]);
                if (p.out_i32) p.out_i32[row * p.ldc + col] = v;
                if (want_f32) p.out_f32[row * p.ldc + col] = gemm_store_value(p, v, alpha, row, col);
            }
        }
    } else {
        const int taps = p.KH * p.KW;
        const int64_t hw = (int64_t)p.Ho * p.Wo;
        float alpha[TH];
#pragma unroll
        for (int a = 0; a < TH; ++a) {
            const int64_t o = h0 + ty + 16 * a;
            alpha[a] = 0.0f;
            if (want_f32 && o < p.held_rows)
                alpha[a] = __fmul_rn(fa, __fdiv_rn(__ldg(p.w_scale + (p.w_per_row ? o : 0)), Lw));
        }
        float seen_max = 0.0f;
        // consumer's Encoder in the store: its level indices go through a [pixel][channel] byte tile in the
        // (drained) staging ring; one thread per pixel and 32-channel group then turns 32 bytes into plane
        // words with an 8 x 8 bit-block transpose.  Channel c of a group sits at byte 4 (c % 8) + c / 8, so
        // 32-bit word i of the pixel holds channels i, 8 + i, 16 + i, 24 + i: the transpose's input order
        // (a 16-channel tile keeps channels i, 8 + i in 16-bit half i and fills half a plane word).
        // A pixel takes BH + 4 bytes (an odd number of words: neighbouring pixels fall into distinct banks).
        const bool want_planes = p.next_planes != nullptr;
        unsigned char* code_tile = reinterpret_cast<unsigned char*>(smem);
        constexpr int PIXEL_BYTES = BH + 4;
        float next_inv = 0.0f, next_half_L = 0.0f, next_lo = 0.0f, next_hi = 0.0f;
        int next_H = 0;
        if (want_planes) {
            next_inv = inverse_scale(__ldg(p.next_scale));
            next_H = 1 << (p.next_bits - 1);
            next_half_L = 0.5f * (float)((1 << p.next_bits) - 1);
            next_lo = (float)(-next_H); next_hi = (float)next_H - 0.5f;
            __syncthreads();                         // every warp is done reading the last k-stage
        }
#pragma unroll
        for (int b = 0; b < TS; ++b) {
            const int r = tx + 16 * b;
            const int n = row_n[r];
            // taps of this pixel that fall outside the image were staged as all-zero bits, i.e. as the
            // code -L_a; what they added, -L_a * tap_sum[tap][o], is taken out again so they count as 0
            const unsigned outside = row_out[r];
            const int64_t rem = row_rem[r];
#pragma unroll
            for (int a = 0; a < TH; ++a) {
                const int64_t o = h0 + ty + 16 * a;
                if (n < 0 || o >= p.held_rows) continue;
                int32_t v = (int32_t)(full - 2u * acc[a][b]);
                if (outside) {
                    // modular arithmetic: the staged value may leave the int32 range, the corrected one does not
                    uint32_t fix = 0u;
                    for (int t = 0; t < taps; ++t)
                        if (outside & (1u << t)) fix += (uint32_t)__ldg(p.tap_sums + (int64_t)t * p.O + o);
                    v = (int32_t)((uint32_t)v + (uint32_t)((1 << A_BITS) - 1) * fix);
                }
                const int64_t idx = ((int64_t)n * p.O + o) * hw + rem;
                if (p.out_i32) p.out_i32[idx] = v;
                if (want_f32) {
                    float f = __fmul_rn((float)v, alpha[a]);
                    if (p.residual) f = __fadd_rn(f, __ldg(p.residual + idx));
                    if (p.relu) f = fmaxf(f, 0.0f);
                    if (p.out_f32) p.out_f32[idx] = f;
                    seen_max = fmaxf(seen_max, f);
                    if (want_planes) {
                        const int u = p.next_act == MPQ_ACT_HRELU
                                          ? level_index<MPQ_ACT_HRELU>(f, next_inv, next_half_L, next_lo, next_hi, next_H)
                                          : level_index<MPQ_ACT_HTANH>(f, next_inv, next_half_L, next_lo, next_hi, next_H);
                        const int c = ty + 16 * a;
                        const int at = BH >= 32 ? (c & ~31) + 4 * (c & 7) + ((c >> 3) & 3) : 2 * (c & 7) + (c >> 3);
                        code_tile[r * PIXEL_BYTES + at] = (unsigned char)u;
                    }
                }
            }
        }
        if (want_planes) {
            __syncthreads();
            // (pixel, 32-channel group) pairs of the tile, one per thread
            constexpr int GROUPS = BH >= 32 ? BH / 32 : 1;
            const int Ow = p.O / 32;
            const int64_t plane_words = (int64_t)p.N * hw * Ow;
            for (int task = tid; task < BS * GROUPS; task += 256) {
                const int r = task / GROUPS, grp = task % GROUPS;
                const int n = row_n[r];
                const int64_t o0 = h0 + 32 * grp;
                if (n < 0 || o0 >= p.held_rows) continue;
                const uint32_t* mine = reinterpret_cast<const uint32_t*>(code_tile + r * PIXEL_BYTES + 32 * grp);
                uint32_t w[8];
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    w[i] = BH >= 32 ? mine[i] : (mine[i >> 1] >> (16 * (i & 1))) & 0x0000FFFFu;
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
                const int64_t at0 = ((int64_t)n * hw + row_rem[r]) * Ow + o0 / 32;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (q < p.next_bits) {
                        const int64_t at = (int64_t)q * plane_words + at0;
                        if (BH >= 32) p.next_planes[at] = w[q];
                        else reinterpret_cast<unsigned short*>(p.next_planes)[2 * at + ((o0 >> 4) & 1)] = (unsigned short)w[q];
                    }
                }
            }
        }
        if (p.out_max) {
            // range of the next layer's encoder, taken while the outputs are still in registers:
            // non-negative floats order like their bit patterns, so an integer atomicMax is exact
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) seen_max = fmaxf(seen_max, __shfl_xor_sync(0xffffffffu, seen_max, off));
            if ((tid & 31) == 0 && seen_max > 0.0f) atomicMax(reinterpret_cast<int*>(p.out_max), __float_as_int(seen_max));
        }
    }
}

template <int HB, int SB, int TS, int MODE, int KS = 1>
static int launch_branch(const BranchParams& p, cudaStream_t st) {
    using T = BranchTile<HB, SB>;
    constexpr int BH = 16 * T::TH, BS = 16 * TS;
    constexpr int ring_quads = T::STAGES * (HB * T::KQ * BH + SB * T::KQ * BS);
    constexpr size_t smem_bytes = (KS == 1 ? (size_t)ring_quads : (size_t)KS * T::group_quads(TS, ring_quads)) * sizeof(uint4);
    static_assert(smem_bytes <= 227 * 1024, "shared memory of one CTA");
    auto kern = branch_kernel<HB, SB, TS, MODE, KS>;
    static PerDeviceOnce configured;   // per instantiation: the attribute belongs to (function, device)
    if (configured.raise_smem_limit(kern, smem_bytes) != MPQ_OK) return MPQ_ERR_CUDA;
    const int64_t blocks = ceil_div(p.streamed_rows, BS) * ceil_div(p.held_rows, BH);
    if (blocks <= 0 || blocks > 0x7fffffffLL) return MPQ_ERR_BAD_SHAPE;
    return launch_chained(kern, (unsigned)blocks, 256 * KS, smem_bytes, st, p);
}

// One translation unit per held-operand width instantiates all eight streamed widths.
template <int HB>
int launch_gemm_hb(int sb, const BranchParams& p, cudaStream_t st);
template <int HB>
int launch_conv_hb(int sb, const BranchParams& p, cudaStream_t st);

}  // namespace mpq
