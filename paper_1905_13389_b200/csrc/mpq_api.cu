// Status strings, size queries, the host-buffer fully-connected layer and the POPC-rate probe.
#include <mutex>

#include "mpq_common.cuh"

using namespace mpq;

extern "C" const char* mpq_status_string(int status) {
    switch (status) {
        case MPQ_OK: return "ok";
        case MPQ_ERR_NULL: return "null pointer";
        case MPQ_ERR_BAD_SHAPE: return "bad shape";
        case MPQ_ERR_UNSUPPORTED: return "unsupported configuration";
        case MPQ_ERR_OVERFLOW: return "int32 accumulator would overflow";
        case MPQ_ERR_ALIGN: return "pointer not 16-byte aligned";
        case MPQ_ERR_CUDA: return "CUDA runtime error";
        case MPQ_ERR_WORKSPACE: return "workspace too small";
        case MPQ_ERR_STATIC_LIMIT: return "problem needs more scratch than MPQ_LINEAR_STATIC_BYTES";
    }
    return "unknown status";
}

extern "C" int64_t mpq_row_words(int64_t k) { return k > 0 ? row_words(k) : 0; }

extern "C" int64_t mpq_packed_words(int64_t rows, int64_t k, int bits) {
    if (rows <= 0 || k <= 0 || !bits_ok(bits)) return 0;
    return (int64_t)bits * rows * row_words(k);
}

// ---- whole fully-connected layer (Fig. 1): device buffers, then host buffers -------------------
namespace {
inline int64_t up256(int64_t v) { return (v + 255) / 256 * 256; }

// Scratch of one layer call: both ranges and both packed operands.
struct LinearScratch {
    int64_t s_a, s_w, a_planes, w_planes, total;
};
LinearScratch linear_scratch(int64_t m, int64_t n, int64_t k, int a_bits, int w_bits) {
    LinearScratch L;
    int64_t off = 0;
    L.s_a = off; off += 256;
    L.s_w = off; off += up256(n * 4);
    L.a_planes = off; off += up256(mpq_packed_words(m, k, a_bits) * 4);
    L.w_planes = off; off += up256(mpq_packed_words(n, k, w_bits) * 4);
    L.total = off;
    return L;
}

// Host staging of mpq_linear_host: fp32 operands and results, then the layer's own scratch.
struct HostLayout {
    int64_t x, w, out_i32, out_f32, scratch, total;
};
HostLayout host_layout(int64_t m, int64_t n, int64_t k, int a_bits, int w_bits) {
    HostLayout L;
    int64_t off = 0;
    L.x = off; off += up256(m * k * 4);
    L.w = off; off += up256(n * k * 4);
    L.out_i32 = off; off += up256(m * n * 4);
    L.out_f32 = off; off += up256(m * n * 4);
    L.scratch = off; off += linear_scratch(m, n, k, a_bits, w_bits).total;
    L.total = off;
    return L;
}

int linear_args_ok(int64_t m, int64_t n, int64_t k, int a_bits, int w_bits, int a_act, int w_mode) {
    if (m <= 0 || n <= 0 || k <= 0) return MPQ_ERR_BAD_SHAPE;
    if (!bits_ok(a_bits) || !bits_ok(w_bits) || (a_act != MPQ_ACT_HTANH && a_act != MPQ_ACT_HRELU) ||
        (w_mode != MPQ_SCALE_PER_TENSOR && w_mode != MPQ_SCALE_PER_ROW)) return MPQ_ERR_UNSUPPORTED;
    return MPQ_OK;
}

// range -> encode -> product with the scratch at `ws` (256-byte aligned device memory)
int linear_on_scratch(const float* x, const float* w, int64_t m, int64_t n, int64_t k,
                      int a_bits, int w_bits, int a_act, int w_mode,
                      int32_t* out_i32, float* out_f32, char* ws, cudaStream_t st) {
    const LinearScratch L = linear_scratch(m, n, k, a_bits, w_bits);
    float* s_a = reinterpret_cast<float*>(ws + L.s_a);
    float* s_w = reinterpret_cast<float*>(ws + L.s_w);
    uint32_t* ap = reinterpret_cast<uint32_t*>(ws + L.a_planes);
    uint32_t* wp = reinterpret_cast<uint32_t*>(ws + L.w_planes);
    int rc;
    if ((rc = mpq_absmax(x, m, k, k, MPQ_SCALE_PER_TENSOR, a_act, s_a, st)) != MPQ_OK) return rc;
    if ((rc = mpq_absmax(w, n, k, k, w_mode, MPQ_ACT_HTANH, s_w, st)) != MPQ_OK) return rc;
    if ((rc = mpq_encode(x, m, k, k, s_a, MPQ_SCALE_PER_TENSOR, a_act, a_bits, ap, st)) != MPQ_OK) return rc;
    if ((rc = mpq_encode(w, n, k, k, s_w, w_mode, MPQ_ACT_HTANH, w_bits, wp, st)) != MPQ_OK) return rc;
    return mpq_gemm(ap, a_bits, wp, w_bits, m, n, k, out_i32, out_f32, n, s_a, s_w, w_mode, st);
}
}  // namespace

extern "C" int64_t mpq_linear_workspace(int64_t m, int64_t n, int64_t k, int a_bits, int w_bits) {
    if (m <= 0 || n <= 0 || k <= 0 || !bits_ok(a_bits) || !bits_ok(w_bits)) return 0;
    return linear_scratch(m, n, k, a_bits, w_bits).total;
}

extern "C" int mpq_linear(const float* x, const float* w, int64_t m, int64_t n, int64_t k,
                          int a_bits, int w_bits, int a_act, int w_mode,
                          int32_t* out_i32, float* out_f32,
                          void* workspace, int64_t workspace_bytes, void* stream) {
    if (!x || !w || !workspace || (!out_i32 && !out_f32)) return MPQ_ERR_NULL;
    const int rc = linear_args_ok(m, n, k, a_bits, w_bits, a_act, w_mode);
    if (rc != MPQ_OK) return rc;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MPQ_ERR_ALIGN;
    if (workspace_bytes < linear_scratch(m, n, k, a_bits, w_bits).total) return MPQ_ERR_WORKSPACE;
    return linear_on_scratch(x, w, m, n, k, a_bits, w_bits, a_act, w_mode, out_i32, out_f32,
                             static_cast<char*>(workspace), (cudaStream_t)stream);
}

// ---- the layer on the library's own scratch: no allocation anywhere --------------------------
// The scratch is part of the loaded module: each GPU that loads the library carries these
// MPQ_LINEAR_STATIC_BYTES until the process exits.  In host code the array's name is only a
// handle for cudaGetSymbolAddress; kernels must be given the address that call returns.
static __device__ __align__(256) unsigned char g_linear_static_scratch[MPQ_LINEAR_STATIC_BYTES];

namespace {
std::mutex g_static_mutex;
unsigned char* g_static_ptr[kMaxDevices] = {};   // device address of the scratch, per device

// Looked up once per device, with that device current (the caller's current device).
int static_scratch_address(unsigned char** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MPQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_linear_static_scratch) != cudaSuccess || !ptr) return MPQ_ERR_CUDA;
        g_static_ptr[dev] = static_cast<unsigned char*>(ptr);
    }
    *out = g_static_ptr[dev];
    return MPQ_OK;
}
}  // namespace

extern "C" int mpq_linear_static(const float* x, const float* w, int64_t m, int64_t n, int64_t k,
                                 int a_bits, int w_bits, int a_act, int w_mode,
                                 int32_t* out_i32, float* out_f32, void* stream) {
    if (!x || !w || (!out_i32 && !out_f32)) return MPQ_ERR_NULL;
    int rc = linear_args_ok(m, n, k, a_bits, w_bits, a_act, w_mode);
    if (rc != MPQ_OK) return rc;
    if (linear_scratch(m, n, k, a_bits, w_bits).total > (int64_t)MPQ_LINEAR_STATIC_BYTES) return MPQ_ERR_STATIC_LIMIT;
    unsigned char* scratch = nullptr;
    if ((rc = static_scratch_address(&scratch)) != MPQ_OK) return rc;
    // Ranges are cleared by the range step on the stream; planes are fully rewritten by the encoders.
    return linear_on_scratch(x, w, m, n, k, a_bits, w_bits, a_act, w_mode, out_i32, out_f32,
                             reinterpret_cast<char*>(scratch), (cudaStream_t)stream);
}

extern "C" int64_t mpq_linear_host_workspace(int64_t m, int64_t n, int64_t k, int a_bits, int w_bits) {
    if (m <= 0 || n <= 0 || k <= 0 || !bits_ok(a_bits) || !bits_ok(w_bits)) return 0;
    return host_layout(m, n, k, a_bits, w_bits).total;
}

// Copy-out helper of mpq_linear_host: one extra stream and a few events per device, created on
// the first call on that device and kept until the process exits, so that finished row blocks
// travel to the host while the next block is still being computed.
namespace {
constexpr int kHostBlocks = 4;
struct HostPipe {
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t block_done[kHostBlocks] = {};
    cudaEvent_t copies_done = nullptr;
    bool ready = false;
};
HostPipe g_host_pipe[kMaxDevices];
std::mutex g_host_pipe_mutex;

int host_pipe(HostPipe** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MPQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_host_pipe_mutex);
    HostPipe& hp = g_host_pipe[dev];
    if (!hp.ready) {
        if (cudaStreamCreateWithFlags(&hp.copy_stream, cudaStreamNonBlocking) != cudaSuccess) return MPQ_ERR_CUDA;
        for (int i = 0; i < kHostBlocks; ++i)
            if (cudaEventCreateWithFlags(&hp.block_done[i], cudaEventDisableTiming) != cudaSuccess) return MPQ_ERR_CUDA;
        if (cudaEventCreateWithFlags(&hp.copies_done, cudaEventDisableTiming) != cudaSuccess) return MPQ_ERR_CUDA;
        hp.ready = true;
    }
    *out = &hp;
    return MPQ_OK;
}
}  // namespace

extern "C" int mpq_linear_host(const float* x_host, const float* w_host, int64_t m, int64_t n, int64_t k,
                               int a_bits, int w_bits, int a_act, int w_mode,
                               int32_t* out_i32_host, float* out_f32_host,
                               void* workspace, int64_t workspace_bytes, void* stream) {
    if (!x_host || !w_host || !workspace || (!out_i32_host && !out_f32_host)) return MPQ_ERR_NULL;
    int rc = linear_args_ok(m, n, k, a_bits, w_bits, a_act, w_mode);
    if (rc != MPQ_OK) return rc;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MPQ_ERR_ALIGN;
    const HostLayout L = host_layout(m, n, k, a_bits, w_bits);
    if (workspace_bytes < L.total) return MPQ_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char* ws = static_cast<char*>(workspace);
    float* x = reinterpret_cast<float*>(ws + L.x);
    float* w = reinterpret_cast<float*>(ws + L.w);
    int32_t* oi = out_i32_host ? reinterpret_cast<int32_t*>(ws + L.out_i32) : nullptr;
    float* of = out_f32_host ? reinterpret_cast<float*>(ws + L.out_f32) : nullptr;
    // weights first: their range and planes are computed while the activations are still in flight
    const LinearScratch S = linear_scratch(m, n, k, a_bits, w_bits);
    char* sc = ws + L.scratch;
    float* s_a = reinterpret_cast<float*>(sc + S.s_a);
    float* s_w = reinterpret_cast<float*>(sc + S.s_w);
    uint32_t* ap = reinterpret_cast<uint32_t*>(sc + S.a_planes);
    uint32_t* wp = reinterpret_cast<uint32_t*>(sc + S.w_planes);
    if (cudaMemcpyAsync(w, w_host, (size_t)n * k * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return MPQ_ERR_CUDA;
    if ((rc = mpq_absmax(w, n, k, k, w_mode, MPQ_ACT_HTANH, s_w, st)) != MPQ_OK) return rc;
    if ((rc = mpq_encode(w, n, k, k, s_w, w_mode, MPQ_ACT_HTANH, w_bits, wp, st)) != MPQ_OK) return rc;
    if (cudaMemcpyAsync(x, x_host, (size_t)m * k * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return MPQ_ERR_CUDA;
    if ((rc = mpq_absmax(x, m, k, k, MPQ_SCALE_PER_TENSOR, a_act, s_a, st)) != MPQ_OK) return rc;
    if ((rc = mpq_encode(x, m, k, k, s_a, MPQ_SCALE_PER_TENSOR, a_act, a_bits, ap, st)) != MPQ_OK) return rc;
    // the product in row blocks; each finished block is copied out on the helper stream
    HostPipe* hp = nullptr;
    if ((rc = host_pipe(&hp)) != MPQ_OK) return rc;
    const int blocks = m >= 1024 ? kHostBlocks : 1;
    const int64_t per = ((m + blocks - 1) / blocks + 63) / 64 * 64;
    for (int b = 0; b < blocks; ++b) {
        const int64_t r0 = (int64_t)b * per;
        if (r0 >= m) break;
        const int64_t rows = (r0 + per <= m) ? per : m - r0;
        if ((rc = gemm_rows(ap, a_bits, wp, w_bits, m, r0, rows, n, k, oi, of, n, s_a, s_w, w_mode, st)) != MPQ_OK) return rc;
        if (cudaEventRecord(hp->block_done[b], st) != cudaSuccess) return MPQ_ERR_CUDA;
        if (cudaStreamWaitEvent(hp->copy_stream, hp->block_done[b], 0) != cudaSuccess) return MPQ_ERR_CUDA;
        const size_t off = (size_t)r0 * n, bytes = (size_t)rows * n * 4;
        if (oi && cudaMemcpyAsync(out_i32_host + off, oi + off, bytes, cudaMemcpyDeviceToHost, hp->copy_stream) != cudaSuccess) return MPQ_ERR_CUDA;
        if (of && cudaMemcpyAsync(out_f32_host + off, of + off, bytes, cudaMemcpyDeviceToHost, hp->copy_stream) != cudaSuccess) return MPQ_ERR_CUDA;
    }
    if (cudaEventRecord(hp->copies_done, hp->copy_stream) != cudaSuccess) return MPQ_ERR_CUDA;
    if (cudaStreamWaitEvent(st, hp->copies_done, 0) != cudaSuccess) return MPQ_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? MPQ_OK : MPQ_ERR_CUDA;
}

// ---- POPC issue-rate probe ----------------------------------------------------------------
namespace {
constexpr int kProbeChains = 8;
// The probe's few result words live in the module so that the call needs no buffer from the caller.
__device__ unsigned long long probe_clk[2];
__device__ uint32_t probe_sink[1];
__global__ void popc_rate_kernel(uint32_t seed, int iters, uint32_t* sink, unsigned long long* clk) {
    uint32_t x[kProbeChains];
    const uint32_t s = seed ^ (threadIdx.x * 0x9E3779B9u);
#pragma unroll
    for (int i = 0; i < kProbeChains; ++i) x[i] = s * (uint32_t)(i + 3);
    unsigned long long g0, g1;
    const long long c0 = clock64();
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g0));
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < kProbeChains; ++i) x[i] = __popc(x[i]) + s;   // independent chains
    }
    const long long c1 = clock64();
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g1));
    uint32_t r = 0;
#pragma unroll
    for (int i = 0; i < kProbeChains; ++i) r += x[i];
    if (r == 0xFFFFFFFFu) sink[0] = r;          // never true: keeps the loop alive
    if (threadIdx.x == 0 && blockIdx.x == 0) { clk[0] = (unsigned long long)(c1 - c0); clk[1] = g1 - g0; }
}

// The instruction mix of the carry-save branch kernel in a register-only loop: per group L
// three-input logic operations, one population count and one integer multiply-add
// (L = 4 when one full adder is spent per two xor words: per word 1 xor + 1 adder half-pair).
template <int L>
__global__ void mix_rate_kernel(uint32_t seed, uint32_t weight, int iters, uint32_t* sink, unsigned long long* clk) {
    uint32_t a[kProbeChains], b[kProbeChains], c[kProbeChains];
    const uint32_t s = seed ^ (threadIdx.x * 0x9E3779B9u);
#pragma unroll
    for (int i = 0; i < kProbeChains; ++i) { a[i] = s * (uint32_t)(i + 3); b[i] = ~a[i] * 7u; c[i] = 0u; }
    unsigned long long g0, g1;
    const long long c0 = clock64();
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g0));
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
    const long long c1 = clock64();
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g1));
    uint32_t r = 0;
#pragma unroll
    for (int i = 0; i < kProbeChains; ++i) r += c[i] ^ a[i];
    if (r == 0xFFFFFFFFu && weight == 0u) sink[0] = r;   // keeps the loop alive
    if (threadIdx.x == 0 && blockIdx.x == 0) { clk[0] = (unsigned long long)(c1 - c0); clk[1] = g1 - g0; }
}

template <int L>
void launch_mix(int blocks, int threads, uint32_t seed, int iters, uint32_t* sink, unsigned long long* clk, cudaStream_t st) {
    mix_rate_kernel<L><<<blocks, threads, 0, st>>>(seed, 1u, iters, sink, clk);
}
}  // namespace

extern "C" int mpq_measure_popc_peak(double* popc_per_s, double* sm_mhz, int* sms, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MPQ_ERR_CUDA;
    if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return MPQ_ERR_CUDA;
    unsigned long long* d_clk = nullptr; uint32_t* d_sink = nullptr;
    if (cudaGetSymbolAddress((void**)&d_clk, probe_clk) != cudaSuccess) return MPQ_ERR_CUDA;
    if (cudaGetSymbolAddress((void**)&d_sink, probe_sink) != cudaSuccess) return MPQ_ERR_CUDA;
    const int threads = 512, blocks_per_sm = 2, iters = 20000;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return MPQ_ERR_CUDA;
    float best_ms = 1e30f; unsigned long long h_clk[2] = {0, 0}, best_clk[2] = {1, 1};
    int rc = MPQ_OK;
    for (int rep = 0; rep < 4 && rc == MPQ_OK; ++rep) {
        cudaEventRecord(e0, st);
        popc_rate_kernel<<<n_sm * blocks_per_sm, threads, 0, st>>>(12345u + rep, iters, d_sink, d_clk);
        cudaEventRecord(e1, st);
        if (cudaEventSynchronize(e1) != cudaSuccess || cudaGetLastError() != cudaSuccess) { rc = MPQ_ERR_CUDA; break; }
        float ms = 0; cudaEventElapsedTime(&ms, e0, e1);
        if (cudaMemcpy(h_clk, d_clk, sizeof(h_clk), cudaMemcpyDeviceToHost) != cudaSuccess) { rc = MPQ_ERR_CUDA; break; }
        if (rep > 0 && ms < best_ms) { best_ms = ms; best_clk[0] = h_clk[0]; best_clk[1] = h_clk[1]; }
    }
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    if (rc != MPQ_OK) return rc;
    const double popcs = (double)n_sm * blocks_per_sm * threads * (double)iters * kProbeChains;
    if (popc_per_s) *popc_per_s = popcs / (best_ms * 1e-3);
    if (sm_mhz) *sm_mhz = (double)best_clk[0] / (double)best_clk[1] * 1e3;
    if (sms) *sms = n_sm;
    return MPQ_OK;
}

extern "C" int mpq_measure_mix_peak(int logic_per_popc, double* groups_per_s, double* sm_mhz, int* sms, void* stream) {
    if (logic_per_popc < 0 || logic_per_popc > 8) return MPQ_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MPQ_ERR_CUDA;
    if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return MPQ_ERR_CUDA;
    unsigned long long* d_clk = nullptr; uint32_t* d_sink = nullptr;
    if (cudaGetSymbolAddress((void**)&d_clk, probe_clk) != cudaSuccess) return MPQ_ERR_CUDA;
    if (cudaGetSymbolAddress((void**)&d_sink, probe_sink) != cudaSuccess) return MPQ_ERR_CUDA;
    const int threads = 512, blocks_per_sm = 2, iters = 8000;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return MPQ_ERR_CUDA;
    float best_ms = 1e30f; unsigned long long h_clk[2] = {0, 0}, best_clk[2] = {1, 1};
    int rc = MPQ_OK;
    for (int rep = 0; rep < 4 && rc == MPQ_OK; ++rep) {
        cudaEventRecord(e0, st);
        const int blocks = n_sm * blocks_per_sm;
        switch (logic_per_popc) {
            case 0: launch_mix<0>(blocks, threads, 99u + rep, iters, d_sink, d_clk, st); break;
            case 1: launch_mix<1>(blocks, threads, 99u + rep, iters, d_sink, d_clk, st); break;
            case 2: launch_mix<2>(blocks, threads, 99u + rep, iters, d_sink, d_clk, st); break;
            case 3: launch_mix<3>(blocks, threads, 99u + rep, iters, d_sink, d_clk, st); break;
            case 4: launch_mix<4>(blocks, threads, 99u + rep, iters, d_sink, d_clk, st); break;
            case 5: launch_mix<5>(blocks, threads, 99u + rep, iters, d_sink, d_clk, st); break;
            case 6: launch_mix<6>(blocks, threads, 99u + rep, iters, d_sink, d_clk, st); break;
            case 7: launch_mix<7>(blocks, threads, 99u + rep, iters, d_sink, d_clk, st); break;
            default: launch_mix<8>(blocks, threads, 99u + rep, iters, d_sink, d_clk, st); break;
        }
        cudaEventRecord(e1, st);
        if (cudaEventSynchronize(e1) != cudaSuccess || cudaGetLastError() != cudaSuccess) { rc = MPQ_ERR_CUDA; break; }
        float ms = 0; cudaEventElapsedTime(&ms, e0, e1);
        if (cudaMemcpy(h_clk, d_clk, sizeof(h_clk), cudaMemcpyDeviceToHost) != cudaSuccess) { rc = MPQ_ERR_CUDA; break; }
        if (rep > 0 && ms < best_ms) { best_ms = ms; best_clk[0] = h_clk[0]; best_clk[1] = h_clk[1]; }
    }
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    if (rc != MPQ_OK) return rc;
    const double groups = (double)n_sm * blocks_per_sm * threads * (double)iters * kProbeChains;
    if (groups_per_s) *groups_per_s = groups / (best_ms * 1e-3);
    if (sm_mhz) *sm_mhz = (double)best_clk[0] / (double)best_clk[1] * 1e3;
    if (sms) *sms = n_sm;
    return MPQ_OK;
}
