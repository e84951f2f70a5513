// C-ABI entry points of the layer product: argument checks, then dispatch on the bit-widths.
#include "mpq_branch_launch.cuh"
#include "mpq_pointwise_kernel.cuh"

namespace mpq {

template <int HB> int launch_gemm_hb(int sb, const BranchParams& p, cudaStream_t st);
template <int HB> int launch_conv_hb(int sb, const BranchParams& p, cudaStream_t st);

static int dispatch_gemm(int hb, int sb, const BranchParams& p, cudaStream_t st) {
    switch (hb) {
        case 1: return launch_gemm_hb<1>(sb, p, st);
        case 2: return launch_gemm_hb<2>(sb, p, st);
        case 3: return launch_gemm_hb<3>(sb, p, st);
        case 4: return launch_gemm_hb<4>(sb, p, st);
        case 5: return launch_gemm_hb<5>(sb, p, st);
        case 6: return launch_gemm_hb<6>(sb, p, st);
        case 7: return launch_gemm_hb<7>(sb, p, st);
        case 8: return launch_gemm_hb<8>(sb, p, st);
    }
    return MPQ_ERR_UNSUPPORTED;
}

static int dispatch_conv(int hb, int sb, const BranchParams& p, cudaStream_t st) {
    switch (hb) {
        case 1: return launch_conv_hb<1>(sb, p, st);
        case 2: return launch_conv_hb<2>(sb, p, st);
        case 3: return launch_conv_hb<3>(sb, p, st);
        case 4: return launch_conv_hb<4>(sb, p, st);
        case 5: return launch_conv_hb<5>(sb, p, st);
        case 6: return launch_conv_hb<6>(sb, p, st);
        case 7: return launch_conv_hb<7>(sb, p, st);
        case 8: return launch_conv_hb<8>(sb, p, st);
    }
    return MPQ_ERR_UNSUPPORTED;
}

static int dispatch_pointwise(int hb, int sb, const BranchParams& p, cudaStream_t st) {
    switch (hb) {
        case 1: return launch_pointwise_hb<1>(sb, p, st);
        case 2: return launch_pointwise_hb<2>(sb, p, st);
        case 3: return launch_pointwise_hb<3>(sb, p, st);
        case 4: return launch_pointwise_hb<4>(sb, p, st);
        case 5: return launch_pointwise_hb<5>(sb, p, st);
        case 6: return launch_pointwise_hb<6>(sb, p, st);
        case 7: return launch_pointwise_hb<7>(sb, p, st);
        case 8: return launch_pointwise_hb<8>(sb, p, st);
    }
    return MPQ_ERR_UNSUPPORTED;
}

static int dispatch_window3x3c64(int hb, int sb, const BranchParams& p, cudaStream_t st) {
    switch (hb) {
        case 1: return launch_window3x3c64_hb<1>(sb, p, st);
        case 2: return launch_window3x3c64_hb<2>(sb, p, st);
        case 3: return launch_window3x3c64_hb<3>(sb, p, st);
        case 4: return launch_window3x3c64_hb<4>(sb, p, st);
        case 5: return launch_window3x3c64_hb<5>(sb, p, st);
        case 6: return launch_window3x3c64_hb<6>(sb, p, st);
        case 7: return launch_window3x3c64_hb<7>(sb, p, st);
        case 8: return launch_window3x3c64_hb<8>(sb, p, st);
    }
    return MPQ_ERR_UNSUPPORTED;
}

static void fill_pow2(BranchParams& p) {
    for (int e = 0; e < 24; ++e) p.pow2[e] = 1u << e;
}

// k * L_a * L_w must stay below 2^31 so that every |acc| fits int32.
static bool int32_headroom(int64_t k, int a_bits, int w_bits) {
    const int64_t LL = (int64_t)((1 << a_bits) - 1) * ((1 << w_bits) - 1);
    return k < ((int64_t)1 << 31) && k * LL < ((int64_t)1 << 31);
}

}  // namespace mpq

using namespace mpq;

// Rows [row0, row0 + rows) of C = A * B^T, A holding m_total rows per plane.
int mpq::gemm_rows(const uint32_t* a_planes, int a_bits, const uint32_t* b_planes, int b_bits,
                   int64_t m_total, int64_t row0, int64_t rows, int64_t n, int64_t k,
                   int32_t* c_i32, float* c_f32, int64_t ldc,
                   const float* a_scale, const float* b_scale, int b_mode, cudaStream_t stream,
                   const GemmGlue& glue) {
    if (!a_planes || !b_planes || (!c_i32 && !c_f32)) return MPQ_ERR_NULL;
    if (c_f32 && (!a_scale || !b_scale)) return MPQ_ERR_NULL;
    if ((glue.bias || glue.residual || glue.relu) && !c_f32) return MPQ_ERR_NULL;
    if (m_total <= 0 || n <= 0 || k <= 0 || ldc < n || row0 < 0 || rows <= 0 || row0 + rows > m_total) return MPQ_ERR_BAD_SHAPE;
    if (!bits_ok(a_bits) || !bits_ok(b_bits) ||
        (b_mode != MPQ_SCALE_PER_TENSOR && b_mode != MPQ_SCALE_PER_ROW)) return MPQ_ERR_UNSUPPORTED;
    if (!int32_headroom(k, a_bits, b_bits)) return MPQ_ERR_OVERFLOW;
    if (!aligned16(a_planes) || !aligned16(b_planes)) return MPQ_ERR_ALIGN;
    BranchParams p = {};
    p.rw = row_words(k); p.k = k;
    p.held = a_planes + row0 * p.rw; p.streamed = b_planes;
    p.held_rows = rows; p.held_plane_rows = m_total; p.streamed_rows = n;
    p.out_i32 = c_i32 ? c_i32 + row0 * ldc : nullptr;
    p.out_f32 = c_f32 ? c_f32 + row0 * ldc : nullptr;
    p.ldc = ldc;
    p.a_scale = a_scale; p.w_scale = b_scale; p.w_per_row = b_mode == MPQ_SCALE_PER_ROW;
    p.bias = glue.bias;
    p.residual = glue.residual ? glue.residual + row0 * ldc : nullptr;
    p.relu = glue.relu;
    fill_pow2(p);
    return dispatch_gemm(a_bits, b_bits, p, stream);
}

extern "C" int mpq_gemm(const uint32_t* a_planes, int a_bits, const uint32_t* b_planes, int b_bits,
                        int64_t m, int64_t n, int64_t k,
                        int32_t* c_i32, float* c_f32, int64_t ldc,
                        const float* a_scale, const float* b_scale, int b_mode, void* stream) {
    return mpq::gemm_rows(a_planes, a_bits, b_planes, b_bits, m, 0, m, n, k, c_i32, c_f32, ldc,
                          a_scale, b_scale, b_mode, (cudaStream_t)stream);
}

extern "C" int mpq_gemm_fused(const uint32_t* a_planes, int a_bits, const uint32_t* b_planes, int b_bits,
                              int64_t m, int64_t n, int64_t k,
                              int32_t* c_i32, float* c_f32, int64_t ldc,
                              const float* a_scale, const float* b_scale, int b_mode,
                              const float* bias, const float* residual, int relu, void* stream) {
    GemmGlue glue;
    glue.bias = bias; glue.residual = residual; glue.relu = relu != 0;
    return mpq::gemm_rows(a_planes, a_bits, b_planes, b_bits, m, 0, m, n, k, c_i32, c_f32, ldc,
                          a_scale, b_scale, b_mode, (cudaStream_t)stream, glue);
}

extern "C" int mpq_conv(const uint32_t* x_planes, int a_bits, int N, int C, int H, int W,
                        const uint32_t* w_planes, int w_bits, const int32_t* tap_sums,
                        int O, int KH, int KW, int stride, int pad,
                        int32_t* y_i32, float* y_f32,
                        const float* x_scale, const float* w_scale, int w_mode, void* stream) {
    return mpq_conv_fused(x_planes, a_bits, N, C, H, W, w_planes, w_bits, tap_sums, O, KH, KW, stride, pad,
                          y_i32, y_f32, x_scale, w_scale, w_mode, nullptr, 0, nullptr, stream);
}

extern "C" int mpq_conv_fused(const uint32_t* x_planes, int a_bits, int N, int C, int H, int W,
                        const uint32_t* w_planes, int w_bits, const int32_t* tap_sums,
                        int O, int KH, int KW, int stride, int pad,
                        int32_t* y_i32, float* y_f32,
                        const float* x_scale, const float* w_scale, int w_mode,
                        const float* residual, int relu, float* out_max, void* stream) {
    return mpq_conv_encoded(x_planes, a_bits, N, C, H, W, w_planes, w_bits, tap_sums, O, KH, KW, stride, pad,
                            y_i32, y_f32, x_scale, w_scale, w_mode, residual, relu, out_max,
                            nullptr, 0, 0, nullptr, stream);
}

extern "C" int mpq_conv_encoded(const uint32_t* x_planes, int a_bits, int N, int C, int H, int W,
                        const uint32_t* w_planes, int w_bits, const int32_t* tap_sums,
                        int O, int KH, int KW, int stride, int pad,
                        int32_t* y_i32, float* y_f32,
                        const float* x_scale, const float* w_scale, int w_mode,
                        const float* residual, int relu, float* out_max,
                        const float* next_scale, int next_act, int next_bits, uint32_t* next_planes,
                        void* stream) {
    const bool want_f32 = y_f32 || next_planes;
    if ((residual || relu || out_max) && !want_f32) return MPQ_ERR_NULL;
    if (!x_planes || !w_planes || (!y_i32 && !want_f32)) return MPQ_ERR_NULL;
    if (want_f32 && (!x_scale || !w_scale)) return MPQ_ERR_NULL;
    if (next_planes) {
        if (!next_scale) return MPQ_ERR_NULL;
        if (!bits_ok(next_bits) || (next_act != MPQ_ACT_HTANH && next_act != MPQ_ACT_HRELU) || O % 32 != 0)
            return MPQ_ERR_UNSUPPORTED;
        if (!aligned16(next_planes)) return MPQ_ERR_ALIGN;
    }
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0 || O <= 0) return MPQ_ERR_BAD_SHAPE;
    if (!bits_ok(a_bits) || !bits_ok(w_bits) || !((KH == 1 && KW == 1) || (KH == 3 && KW == 3)) ||
        (stride != 1 && stride != 2) || pad < 0 || pad > 1 ||
        !(C == 32 || C == 64 || C % 128 == 0) ||
        (w_mode != MPQ_SCALE_PER_TENSOR && w_mode != MPQ_SCALE_PER_ROW)) return MPQ_ERR_UNSUPPORTED;
    if (pad > 0 && !tap_sums) return MPQ_ERR_NULL;
    if (H + 2 * pad < KH || W + 2 * pad < KW) return MPQ_ERR_BAD_SHAPE;
    const int64_t K = (int64_t)KH * KW * C;
    if (!int32_headroom(K, a_bits, w_bits)) return MPQ_ERR_OVERFLOW;
    if (!aligned16(x_planes) || !aligned16(w_planes)) return MPQ_ERR_ALIGN;
    BranchParams p = {};
    p.held = w_planes; p.streamed = x_planes;
    p.Ho = (H + 2 * pad - KH) / stride + 1;
    p.Wo = (W + 2 * pad - KW) / stride + 1;
    p.held_rows = O; p.held_plane_rows = O; p.streamed_rows = (int64_t)N * p.Ho * p.Wo;
    p.rw = row_words(K); p.k = K;
    p.out_i32 = y_i32; p.out_f32 = y_f32; p.ldc = 0;
    p.a_scale = x_scale; p.w_scale = w_scale; p.w_per_row = w_mode == MPQ_SCALE_PER_ROW;
    p.N = N; p.C = C; p.H = H; p.W = W; p.O = O; p.KH = KH; p.KW = KW; p.stride = stride; p.pad = pad;
    p.Cw = C / 32; p.granule = p.Cw >= 4 ? 4 : p.Cw;
    p.granule_shift = p.granule == 4 ? 0 : p.granule == 2 ? 1 : 2;
    p.tap_granules = p.Cw / p.granule;
    p.tap_magic = p.tap_granules > 1 ? (uint32_t)((((uint64_t)1 << 32) + p.tap_granules - 1) / p.tap_granules) : 0u;
    // the gather indexes pixels with 32-bit integers and divides copy indices below 2^16 exactly
    if ((int64_t)N * H * W >= ((int64_t)1 << 31) || (p.rw << p.granule_shift) >= 65536) return MPQ_ERR_UNSUPPORTED;
    p.tap_sums = tap_sums;
    p.residual = residual; p.relu = relu != 0; p.out_max = out_max;
    p.next_planes = next_planes; p.next_scale = next_scale; p.next_bits = next_bits; p.next_act = next_act;
    fill_pow2(p);
    p.half_tail = (ceil_div(K, 32) % 4 == 1 || ceil_div(K, 32) % 4 == 2) ? 1 : 0;
    for (int t = 0; t < 16; ++t) {
        const bool live = t < KH * KW;
        p.tap_dh[t] = (signed char)(live ? t / KW : 0);
        p.tap_dw[t] = (signed char)(live ? t % KW : 0);
        p.tap_offset[t] = p.tap_dh[t] * W + p.tap_dw[t];
    }
    p.sub_h = p.Ho; p.sub_w = p.Wo; p.in_step = stride; p.in_h0 = -pad; p.in_w0 = -pad;
    p.out_h0 = 0; p.out_w0 = 0; p.out_step = 1;
    p.window3x3 = KH == 3 ? 1 : 0;
    // held = weights (w_bits planes), streamed = activations (a_bits planes)
    if (pointwise_applies(p)) return dispatch_pointwise(w_bits, a_bits, p, (cudaStream_t)stream);
    if (window3x3c64_applies(p, a_bits)) return dispatch_window3x3c64(w_bits, a_bits, p, (cudaStream_t)stream);
    return dispatch_conv(w_bits, a_bits, p, (cudaStream_t)stream);
}

// Deconvolution: output pixel (oh, ow) receives x[ih][iw] * w[kh][kw] from every (ih, kh) with
// oh = ih * stride - pad + kh.  Outputs of one phase (oh mod stride, ow mod stride) all use the same
// taps, kh = r_h + stride * t_h with r_h = (oh + pad) mod stride, and ih = (oh + pad - r_h) / stride - t_h:
// per phase an ordinary gather over a T_h x T_w window that steps backwards through the image.  One
// launch of the branch kernel per phase, each over that phase's part of the output.
extern "C" int mpq_deconv(const uint32_t* x_planes, int a_bits, int N, int C, int H, int W,
                          const uint32_t* w_planes, int w_bits, const int32_t* tap_sums,
                          int O, int KH, int KW, int stride, int pad,
                          int32_t* y_i32, float* y_f32,
                          const float* x_scale, const float* w_scale, int w_mode,
                          const float* residual, int relu, float* out_max, void* stream) {
    if ((residual || relu || out_max) && !y_f32) return MPQ_ERR_NULL;
    if (!x_planes || !w_planes || !tap_sums || (!y_i32 && !y_f32)) return MPQ_ERR_NULL;
    if (y_f32 && (!x_scale || !w_scale)) return MPQ_ERR_NULL;
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0 || O <= 0 || KH <= 0 || KW <= 0) return MPQ_ERR_BAD_SHAPE;
    if (!bits_ok(a_bits) || !bits_ok(w_bits) || !deconv_filter_ok(KH, KW, stride) || pad < 0 || pad >= KH || pad >= KW ||
        !(C == 32 || C == 64 || C % 128 == 0) ||
        (w_mode != MPQ_SCALE_PER_TENSOR && w_mode != MPQ_SCALE_PER_ROW)) return MPQ_ERR_UNSUPPORTED;
    const int Ho = (H - 1) * stride - 2 * pad + KH, Wo = (W - 1) * stride - 2 * pad + KW;
    if (Ho <= 0 || Wo <= 0) return MPQ_ERR_BAD_SHAPE;
    if (!aligned16(x_planes) || !aligned16(w_planes)) return MPQ_ERR_ALIGN;
    // an output sums at most ceil(KH/stride) * ceil(KW/stride) * C products
    const int64_t k_max = (int64_t)ceil_div(KH, stride) * ceil_div(KW, stride) * C;
    if (!int32_headroom(k_max, a_bits, w_bits)) return MPQ_ERR_OVERFLOW;
    if ((int64_t)N * H * W >= ((int64_t)1 << 31) || (int64_t)N * Ho * Wo >= ((int64_t)1 << 31)) return MPQ_ERR_UNSUPPORTED;
    DeconvPhase phases[4];
    deconv_phases(O, C, KH, KW, stride, w_bits, phases);
    for (int out_ph = 0; out_ph < stride; ++out_ph) {
        for (int out_pw = 0; out_pw < stride; ++out_pw) {
            if (out_ph >= Ho || out_pw >= Wo) continue;                     // no output in this phase
            const int r_h = (out_ph + pad) % stride, r_w = (out_pw + pad) % stride;
            const DeconvPhase& g = phases[r_h * stride + r_w];
            BranchParams p = {};
            p.held = w_planes + g.word_offset; p.streamed = x_planes;
            p.Ho = Ho; p.Wo = Wo;
            p.sub_h = (int)ceil_div(Ho - out_ph, stride); p.sub_w = (int)ceil_div(Wo - out_pw, stride);
            p.held_rows = O; p.held_plane_rows = O; p.streamed_rows = (int64_t)N * p.sub_h * p.sub_w;
            p.k = (int64_t)g.T_h * g.T_w * C; p.rw = g.rw;
            p.out_i32 = y_i32; p.out_f32 = y_f32; p.ldc = 0;
            p.a_scale = x_scale; p.w_scale = w_scale; p.w_per_row = w_mode == MPQ_SCALE_PER_ROW;
            p.N = N; p.C = C; p.H = H; p.W = W; p.O = O; p.KH = g.T_h; p.KW = g.T_w; p.stride = stride; p.pad = pad;
            p.Cw = C / 32; p.granule = p.Cw >= 4 ? 4 : p.Cw;
            p.granule_shift = p.granule == 4 ? 0 : p.granule == 2 ? 1 : 2;
            p.tap_granules = p.Cw / p.granule;
            p.tap_magic = p.tap_granules > 1 ? (uint32_t)((((uint64_t)1 << 32) + p.tap_granules - 1) / p.tap_granules) : 0u;
            if ((p.rw << p.granule_shift) >= 65536) return MPQ_ERR_UNSUPPORTED;
            p.tap_sums = tap_sums + (int64_t)g.tap_start * O;
            p.residual = residual; p.relu = relu != 0; p.out_max = out_max;
            fill_pow2(p);
            const int64_t kw32 = ceil_div(p.k, 32);
            p.half_tail = (kw32 % 4 == 1 || kw32 % 4 == 2) ? 1 : 0;
            for (int t = 0; t < 16; ++t) {
                const bool live = t < g.T_h * g.T_w;
                p.tap_dh[t] = (signed char)(live ? -(t / g.T_w) : 0);
                p.tap_dw[t] = (signed char)(live ? -(t % g.T_w) : 0);
                p.tap_offset[t] = p.tap_dh[t] * W + p.tap_dw[t];
            }
            p.in_step = 1; p.in_h0 = (out_ph + pad - r_h) / stride; p.in_w0 = (out_pw + pad - r_w) / stride;
            p.out_h0 = out_ph; p.out_w0 = out_pw; p.out_step = stride;
            p.window3x3 = 0;
            const int rc = dispatch_conv(w_bits, a_bits, p, (cudaStream_t)stream);
            if (rc != MPQ_OK) return rc;
        }
    }
    return MPQ_OK;
}
