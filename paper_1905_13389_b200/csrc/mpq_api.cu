// Status strings, size queries and the whole-layer entry points (device, built-in scratch, host buffers).
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

// Layout of mpq_linear_host_prepared's workspace: the activations' staging, the results, the
// activation range and the packed activations (the weights are already resident and packed).
struct PreparedLayout {
    int64_t x, out_i32, out_f32, s_a, a_planes, total;
};
PreparedLayout prepared_layout(int64_t m, int64_t n, int64_t k, int a_bits) {
    PreparedLayout L;
    int64_t off = 0;
    L.x = off; off += up256(m * k * 4);
    L.out_i32 = off; off += up256(m * n * 4);
    L.out_f32 = off; off += up256(m * n * 4);
    L.s_a = off; off += 256;
    L.a_planes = off; off += up256(mpq_packed_words(m, k, a_bits) * 4);
    L.total = off;
    return L;
}

// The product in row blocks; each finished block travels to the host on the helper stream while
// the next one is computed.  Returns after everything has drained.
int product_to_host(const uint32_t* ap, int a_bits, const uint32_t* wp, int w_bits, int64_t m, int64_t n, int64_t k,
                    int32_t* oi, float* of, int32_t* out_i32_host, float* out_f32_host,
                    const float* s_a, const float* s_w, int w_mode, cudaStream_t st) {
    int rc;
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
    return product_to_host(ap, a_bits, wp, w_bits, m, n, k, oi, of, out_i32_host, out_f32_host, s_a, s_w, w_mode, st);
}

extern "C" int64_t mpq_linear_host_prepared_workspace(int64_t m, int64_t n, int64_t k, int a_bits) {
    if (m <= 0 || n <= 0 || k <= 0 || !bits_ok(a_bits)) return 0;
    return prepared_layout(m, n, k, a_bits).total;
}

extern "C" int mpq_linear_host_prepared(const float* x_host, const uint32_t* w_planes, const float* w_scale,
                                        int64_t m, int64_t n, int64_t k,
                                        int a_bits, int w_bits, int a_act, int w_mode,
                                        int32_t* out_i32_host, float* out_f32_host,
                                        void* workspace, int64_t workspace_bytes, void* stream) {
    if (!x_host || !w_planes || !workspace || (!out_i32_host && !out_f32_host)) return MPQ_ERR_NULL;
    if (out_f32_host && !w_scale) return MPQ_ERR_NULL;
    int rc = linear_args_ok(m, n, k, a_bits, w_bits, a_act, w_mode);
    if (rc != MPQ_OK) return rc;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 || !aligned16(w_planes)) return MPQ_ERR_ALIGN;
    const PreparedLayout L = prepared_layout(m, n, k, a_bits);
    if (workspace_bytes < L.total) return MPQ_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char* ws = static_cast<char*>(workspace);
    float* x = reinterpret_cast<float*>(ws + L.x);
    int32_t* oi = out_i32_host ? reinterpret_cast<int32_t*>(ws + L.out_i32) : nullptr;
    float* of = out_f32_host ? reinterpret_cast<float*>(ws + L.out_f32) : nullptr;
    float* s_a = reinterpret_cast<float*>(ws + L.s_a);
    uint32_t* ap = reinterpret_cast<uint32_t*>(ws + L.a_planes);
    if (cudaMemcpyAsync(x, x_host, (size_t)m * k * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return MPQ_ERR_CUDA;
    if ((rc = mpq_absmax(x, m, k, k, MPQ_SCALE_PER_TENSOR, a_act, s_a, st)) != MPQ_OK) return rc;
    if ((rc = mpq_encode(x, m, k, k, s_a, MPQ_SCALE_PER_TENSOR, a_act, a_bits, ap, st)) != MPQ_OK) return rc;
    return product_to_host(ap, a_bits, w_planes, w_bits, m, n, k, oi, of, out_i32_host, out_f32_host, s_a, w_scale, w_mode, st);
}
