// Shared host/device helpers of libmpq (CUDA side only).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <atomic>
#include "mpq.h"

namespace mpq {

constexpr int kMaxBits = 8;

__host__ __device__ inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Words per packed row: ceil(k/32) rounded up to 4 words (16 bytes).
__host__ __device__ inline int64_t row_words(int64_t k) { return ceil_div(ceil_div(k, 32), 4) * 4; }

// Deconvolution weights are stored as one packed matrix per filter phase (r_h, r_w) = (kh mod stride,
// kw mod stride): the taps kh = r_h + stride * t_h, kw = r_w + stride * t_w that reach the same output
// phase, k ordered (t_h, t_w, c).  Phases in the order r_h * stride + r_w, each [bits][O][rw].
inline bool deconv_filter_ok(int KH, int KW, int stride) {
    return (stride == 1 || stride == 2) && KH >= stride && KW >= stride && KH <= 4 && KW <= 4;
}
struct DeconvPhase {
    int r_h, r_w, T_h, T_w;      // phase and its tap counts
    int tap_start;               // first row of its tap sums (taps counted phase by phase)
    int64_t rw;                  // words per packed row = row_words(T_h * T_w * C)
    int64_t word_offset;         // where its planes start
};
inline int64_t deconv_phases(int O, int C, int KH, int KW, int stride, int bits, DeconvPhase (&ph)[4]) {
    int64_t words = 0;
    int taps = 0, n = 0;
    for (int r_h = 0; r_h < stride; ++r_h)
        for (int r_w = 0; r_w < stride; ++r_w) {
            DeconvPhase& g = ph[n++];
            g.r_h = r_h; g.r_w = r_w;
            g.T_h = (KH - r_h + stride - 1) / stride; g.T_w = (KW - r_w + stride - 1) / stride;
            g.tap_start = taps; taps += g.T_h * g.T_w;
            g.rw = row_words((int64_t)g.T_h * g.T_w * C);
            g.word_offset = words; words += (int64_t)bits * O * g.rw;
        }
    return words;
}

inline bool bits_ok(int b) { return b >= 1 && b <= kMaxBits; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int launch_status() { return cudaGetLastError() == cudaSuccess ? MPQ_OK : MPQ_ERR_CUDA; }

// ---- Per-device host state ------------------------------------------------------------------
// The only things the library remembers between calls are facts about a device that never change
// while the process lives: its multiprocessor count and "this kernel's shared-memory limit has
// been raised on this device".  Both sit in tables indexed by device ordinal and are written with
// atomics, so concurrent host threads and processes that alternate between devices are safe
// (a lost race only repeats an idempotent query or attribute call).
constexpr int kMaxDevices = 64;

inline int current_device() {
    int dev = -1;
    return (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices) ? dev : -1;
}

// Multiprocessors of the current device (0 if it cannot be read).
inline int sm_count() {
    static std::atomic<int> cached[kMaxDevices];
    const int dev = current_device();
    if (dev < 0) return 0;
    int n = cached[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cached[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

// One flag per device for one kernel: set once that kernel's dynamic shared-memory limit has been
// raised there.  A kernel's launcher keeps one static instance.
struct PerDeviceOnce {
    std::atomic<bool> done[kMaxDevices];
    template <typename Kernel>
    int raise_smem_limit(Kernel kernel, size_t bytes) {
        const int dev = current_device();
        if (dev < 0) return MPQ_ERR_CUDA;
        if (!done[dev].load(std::memory_order_acquire)) {
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess)
                return MPQ_ERR_CUDA;
            done[dev].store(true, std::memory_order_release);
        }
        return MPQ_OK;
    }
};

// Rows [row0, row0 + rows) of the layer product (mpq_gemm on a row block of A): lets a caller
// overlap the copy-out of finished rows with the product of the next ones.
// `glue`: what may ride in the store (bias per column, residual with the output's layout, max(.,0)).
struct GemmGlue {
    const float* bias = nullptr;
    const float* residual = nullptr;
    bool relu = false;
};
int gemm_rows(const uint32_t* a_planes, int a_bits, const uint32_t* b_planes, int b_bits,
              int64_t m_total, int64_t row0, int64_t rows, int64_t n, int64_t k,
              int32_t* c_i32, float* c_f32, int64_t ldc,
              const float* a_scale, const float* b_scale, int b_mode, cudaStream_t stream,
              const GemmGlue& glue = GemmGlue());

// ---- Chained launches (programmatic dependent launch) --------------------------------------
// A layer is a chain of short kernels on one stream (range, encode, product, add).  Launched
// with the programmatic-serialization attribute, a kernel's blocks may become resident while the
// kernel before it in the stream drains its last wave, which hides the launch latency between
// them.  Every kernel launched this way calls chain_entry() before it touches global memory:
// it first lets its own successor start launching, then waits until the predecessor grid has
// completed and its writes are visible.  (On a launch without the attribute both are no-ops.)
// Grids of less than a few waves are launched without the attribute: their blocks would be placed
// early on whichever SMs happen to be free, several to one SM, and that imbalance costs more
// than the hidden latency (a 128-block product ran 1.7 x slower).
__device__ __forceinline__ void chain_entry() {
    asm volatile("griddepcontrol.launch_dependents;\n\tgriddepcontrol.wait;\n" ::: "memory");
}
// `whole_device`: the grid is exactly one CTA per resident slot of the device (a persistent kernel),
// so early placement cannot unbalance it and the attribute is set whatever the grid size.
template <typename... Params, typename... Args>
inline int launch_chained_as(bool whole_device, void (*kernel)(Params...), unsigned blocks, unsigned threads,
                             size_t smem_bytes, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks, 1, 1);
    cfg.blockDim = dim3(threads, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = (whole_device || blocks >= 1024u) ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...) != cudaSuccess) {
        cudaGetLastError();
        return MPQ_ERR_CUDA;
    }
    return launch_status();
}
template <typename... Params, typename... Args>
inline int launch_chained(void (*kernel)(Params...), unsigned blocks, unsigned threads, size_t smem_bytes,
                          cudaStream_t st, Args... args) {
    return launch_chained_as(false, kernel, blocks, threads, smem_bytes, st, args...);
}

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

// ---- The quantizer and the bit-plane split on the floating-point pipe ---------------------
// level_fraction() returns z in [0, 1) with  u = floor(2^BITS * z)  (HReLU: u = H + floor(2^BITS * z)),
// H = 2^(BITS-1), u the level index of level_index():
//   HTanh: z = min(sat(RD(y/2H + 1/2)), 1 - 1/4H)        HReLU: z = min(sat(y/2H), 1/2 - 1/4H)
// sat() clamps to [0,1] inside the multiply-add; the round-down addition keeps a value that lies
// just below a level boundary below it (n/2H is representable, so floor(2H*RD(t)) = floor(2H*t)).
// Equal to level_index() for every input except a NaN under HTanh (sat() sends a NaN to 0, not
// to the level above zero): callers look for NaNs themselves and fall back to level_index().
template <int BITS, int ACT>
__device__ __forceinline__ float level_fraction(float x, float inv_s, float half_L) {
    constexpr float kInvTwoH = 1.0f / (float)(1 << BITS);
    const float y = __fmul_rn(__fmul_rn(x, inv_s), half_L);
    float z;
    if (ACT == MPQ_ACT_HRELU) {
        asm("mul.rn.sat.f32 %0, %1, %2;" : "=f"(z) : "f"(y), "f"(kInvTwoH));
        return fminf(z, 0.5f - 0.5f * kInvTwoH);
    }
    asm("fma.rm.sat.f32 %0, %1, %2, %3;" : "=f"(z) : "f"(y), "f"(kInvTwoH), "f"(0.5f));
    return fminf(z, 1.0f - 0.5f * kInvTwoH);
}

// Builds, in one thread, the BITS plane words of 32 elements pushed from element 31 down to
// element 0, without a per-bit test: for plane p the value floor(u / 2^p) drops out of one
// round-down multiply-add (2^23 is added so that the integer sits in the low mantissa bits),
//     t_p = bits(RD(z * 2^(BITS-p) + 2^23 + (H >> p)))  =  0x4B000000 + floor(u / 2^p),
// it is shifted in with  acc_p = 2 acc_p + t_p  (arithmetic mod 2^32, so the running sums may
// wrap), and since bit p of u is floor(u/2^p) - 2 floor(u/2^(p+1)) the plane words are
//     word_p = T_p - 2 T_(p+1),   T_p = acc_p + 0x4B000000,   T_BITS = 0
// (the 32 added constants sum to 0x4B000000 * (2^32 - 1) = -0x4B000000).  `two` is the number 2
// passed in a register: a multiplier the compiler cannot see keeps the doubling an integer
// multiply-add on the FMA pipe instead of a shift-add on the (busier) integer ALU.
template <int BITS, int ACT>
struct LaneWords {
    uint32_t acc[BITS];
    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int p = 0; p < BITS; ++p) acc[p] = 0u;
    }
    __device__ __forceinline__ void push(float z, uint32_t two) {
#pragma unroll
        for (int p = 0; p < BITS; ++p) {
            const float magic = 8388608.0f + (ACT == MPQ_ACT_HRELU ? (float)((1 << (BITS - 1)) >> p) : 0.0f);
            const uint32_t t = __float_as_uint(__fmaf_rd(z, (float)(1 << (BITS - p)), magic));
            acc[p] = acc[p] * two + t;
        }
    }
    __device__ __forceinline__ uint32_t word(int p) const {
        const uint32_t T = acc[p] + 0x4B000000u;
        return p + 1 < BITS ? T - 2u * (acc[p + 1] + 0x4B000000u) : T;
    }
};

}  // namespace mpq
