// Roofline denominators measured on the GPU the library runs on: register-only loops (no memory
// traffic) that issue one kind of instruction, or one instruction mix, as fast as the SM accepts
// it.  Three probes: the plain population-count rate, the carry-save instruction mix of the
// branch kernel (L three-input logic operations + 1 population count + 1 integer multiply-add per
// group), and the legacy one-bit tensor instruction mma.sync.m16n8k256 (xor.popc / and.popc).
#include "mpq_common.cuh"

using namespace mpq;

namespace {
constexpr int kProbeChains = 8;
constexpr int kProbeThreads = 512;
constexpr int kProbeBlocksPerSm = 2;
// The probes' few result words live in the module so that the calls need no buffer from the caller.
__device__ unsigned long long probe_clk[2];
__device__ uint32_t probe_sink[1];

struct ProbeClock {
    long long c0;
    unsigned long long g0;
    __device__ __forceinline__ void start() {
        c0 = clock64();
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g0));
    }
    __device__ __forceinline__ void stop(unsigned long long* clk) {
        const long long c1 = clock64();
        unsigned long long g1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g1));
        if (threadIdx.x == 0 && blockIdx.x == 0) { clk[0] = (unsigned long long)(c1 - c0); clk[1] = g1 - g0; }
    }
};

__global__ void popc_rate_kernel(uint32_t seed, int iters, uint32_t* sink, unsigned long long* clk) {
    uint32_t x[kProbeChains];
    const uint32_t s = seed ^ (threadIdx.x * 0x9E3779B9u);
#pragma unroll
    for (int i = 0; i < kProbeChains; ++i) x[i] = s * (uint32_t)(i + 3);
    ProbeClock pc;
    pc.start();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < kProbeChains; ++i) x[i] = __popc(x[i]) + s;   // independent chains
    }
    pc.stop(clk);
    uint32_t r = 0;
#pragma unroll
    for (int i = 0; i < kProbeChains; ++i) r += x[i];
    if (r == 0xFFFFFFFFu) sink[0] = r;          // never true: keeps the loop alive
}

// The instruction mix of the carry-save branch kernel: per group L three-input logic operations,
// one population count and one integer multiply-add (L = 4 when one full adder is spent per two
// xor words: per word 1 xor + 1 adder half-pair).
template <int L>
__global__ void mix_rate_kernel(uint32_t seed, uint32_t weight, int iters, uint32_t* sink, unsigned long long* clk) {
    uint32_t a[kProbeChains], b[kProbeChains], c[kProbeChains];
    const uint32_t s = seed ^ (threadIdx.x * 0x9E3779B9u);
#pragma unroll
    for (int i = 0; i < kProbeChains; ++i) { a[i] = s * (uint32_t)(i + 3); b[i] = ~a[i] * 7u; c[i] = 0u; }
    ProbeClock pc;
    pc.start();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < kProbeChains; ++i) {
#pragma unroll
            for (int l = 0; l < L; ++l) {
                uint32_t d;
                if (l & 1) asm("lop3.b32 %0, %1, %2, %3, 0xE8;" : "=r"(d) : "r"(a[i]), "r"(b[i]), "r"(s));
                else       asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(d) : "r"(a[i]), "r"(b[i]), "r"(s));
                b[i] = a[i]; a[i] = d;
            }
            c[i] = (uint32_t)__popc(a[i]) * weight + c[i];
            if (L == 0) a[i] = c[i];
        }
    }
    pc.stop(clk);
    uint32_t r = 0;
#pragma unroll
    for (int i = 0; i < kProbeChains; ++i) r += c[i] ^ a[i];
    if (r == 0xFFFFFFFFu && weight == 0u) sink[0] = r;   // keeps the loop alive
}

// Legacy one-bit tensor instruction: D = popc(A op B) + C on a 16 x 8 x 256 tile per warp, operands
// and accumulators in registers.  Four independent accumulator chains per warp; the operands
// never change, so there is no operand traffic at all: the figure is an upper bound on what a
// kernel built on this instruction could reach.
template <int AND_POPC>
__global__ void b1_mma_rate_kernel(uint32_t seed, int iters, uint32_t* sink, unsigned long long* clk) {
    constexpr int CH = 4;
    const uint32_t s = seed ^ (threadIdx.x * 0x9E3779B9u);
    uint32_t a[4] = {s, s * 3u, s * 5u, s * 7u}, b[2] = {~s, s * 11u};
    int c[CH][4];
#pragma unroll
    for (int i = 0; i < CH; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) c[i][j] = 0;
    ProbeClock pc;
    pc.start();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < CH; ++i) {
            if (AND_POPC)
                asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.and.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                             : "+r"(c[i][0]), "+r"(c[i][1]), "+r"(c[i][2]), "+r"(c[i][3])
                             : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
            else
                asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.xor.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                             : "+r"(c[i][0]), "+r"(c[i][1]), "+r"(c[i][2]), "+r"(c[i][3])
                             : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
        }
    }
    pc.stop(clk);
    int r = 0;
#pragma unroll
    for (int i = 0; i < CH; ++i) r += c[i][0] ^ c[i][1] ^ c[i][2] ^ c[i][3];
    if (r == 0x7FFFFFFF && iters < 0) sink[0] = (uint32_t)r;   // never true: keeps the loop alive
}

template <int L>
void launch_mix(int blocks, uint32_t seed, int iters, uint32_t* sink, unsigned long long* clk, cudaStream_t st) {
    mix_rate_kernel<L><<<blocks, kProbeThreads, 0, st>>>(seed, 1u, iters, sink, clk);
}

// Runs `launch(rep)` four times, keeps the fastest of the last three, and converts `work_per_thread`
// operations of every thread of the grid into a rate.
template <typename Launch>
int run_probe(Launch launch, double work_per_thread, double* rate, double* sm_mhz, int* sms, cudaStream_t st) {
    const int n_sm = sm_count();
    if (n_sm <= 0) return MPQ_ERR_CUDA;
    unsigned long long* d_clk = nullptr; uint32_t* d_sink = nullptr;
    if (cudaGetSymbolAddress((void**)&d_clk, probe_clk) != cudaSuccess) return MPQ_ERR_CUDA;
    if (cudaGetSymbolAddress((void**)&d_sink, probe_sink) != cudaSuccess) return MPQ_ERR_CUDA;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess) return MPQ_ERR_CUDA;
    if (cudaEventCreate(&e1) != cudaSuccess) { cudaEventDestroy(e0); return MPQ_ERR_CUDA; }
    float best_ms = 1e30f; unsigned long long h_clk[2] = {0, 0}, best_clk[2] = {1, 1};
    int rc = MPQ_OK;
    const int blocks = n_sm * kProbeBlocksPerSm;
    for (int rep = 0; rep < 4 && rc == MPQ_OK; ++rep) {
        cudaEventRecord(e0, st);
        launch(rep, blocks, d_sink, d_clk);
        cudaEventRecord(e1, st);
        if (cudaEventSynchronize(e1) != cudaSuccess || cudaGetLastError() != cudaSuccess) { rc = MPQ_ERR_CUDA; break; }
        float ms = 0; cudaEventElapsedTime(&ms, e0, e1);
        if (cudaMemcpy(h_clk, d_clk, sizeof(h_clk), cudaMemcpyDeviceToHost) != cudaSuccess) { rc = MPQ_ERR_CUDA; break; }
        if (rep > 0 && ms < best_ms) { best_ms = ms; best_clk[0] = h_clk[0]; best_clk[1] = h_clk[1]; }
    }
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    if (rc != MPQ_OK) return rc;
    if (rate) *rate = (double)blocks * kProbeThreads * work_per_thread / (best_ms * 1e-3);
    if (sm_mhz) *sm_mhz = (double)best_clk[0] / (double)best_clk[1] * 1e3;
    if (sms) *sms = n_sm;
    return MPQ_OK;
}
}  // namespace

extern "C" int mpq_measure_popc_peak(double* popc_per_s, double* sm_mhz, int* sms, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    const int iters = 20000;
    return run_probe([&](int rep, int blocks, uint32_t* sink, unsigned long long* clk) {
        popc_rate_kernel<<<blocks, kProbeThreads, 0, st>>>(12345u + rep, iters, sink, clk);
    }, (double)iters * kProbeChains, popc_per_s, sm_mhz, sms, st);
}

extern "C" int mpq_measure_mix_peak(int logic_per_popc, double* groups_per_s, double* sm_mhz, int* sms, void* stream) {
    if (logic_per_popc < 0 || logic_per_popc > 8) return MPQ_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    const int iters = 8000;
    return run_probe([&](int rep, int blocks, uint32_t* sink, unsigned long long* clk) {
        const uint32_t seed = 99u + rep;
        switch (logic_per_popc) {
            case 0: launch_mix<0>(blocks, seed, iters, sink, clk, st); break;
            case 1: launch_mix<1>(blocks, seed, iters, sink, clk, st); break;
            case 2: launch_mix<2>(blocks, seed, iters, sink, clk, st); break;
            case 3: launch_mix<3>(blocks, seed, iters, sink, clk, st); break;
            case 4: launch_mix<4>(blocks, seed, iters, sink, clk, st); break;
            case 5: launch_mix<5>(blocks, seed, iters, sink, clk, st); break;
            case 6: launch_mix<6>(blocks, seed, iters, sink, clk, st); break;
            case 7: launch_mix<7>(blocks, seed, iters, sink, clk, st); break;
            default: launch_mix<8>(blocks, seed, iters, sink, clk, st); break;
        }
    }, (double)iters * kProbeChains, groups_per_s, sm_mhz, sms, st);
}

extern "C" int mpq_measure_b1_mma_peak(int and_popc, double* warp_mma_per_s, double* sm_mhz, int* sms, void* stream) {
    if (and_popc != 0 && and_popc != 1) return MPQ_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    const int iters = 2000;
    double per_thread = 0.0;
    const int rc = run_probe([&](int rep, int blocks, uint32_t* sink, unsigned long long* clk) {
        if (and_popc) b1_mma_rate_kernel<1><<<blocks, kProbeThreads, 0, st>>>(7u + rep, iters, sink, clk);
        else          b1_mma_rate_kernel<0><<<blocks, kProbeThreads, 0, st>>>(7u + rep, iters, sink, clk);
    }, (double)iters * 4, &per_thread, sm_mhz, sms, st);
    // run_probe counts per thread; one warp-wide instruction is shared by 32 threads
    if (rc == MPQ_OK && warp_mma_per_s) *warp_mma_per_s = per_thread / 32.0;
    return rc;
}
