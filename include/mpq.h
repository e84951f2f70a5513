/*
 * mpq -- multi-precision quantized layers through the {-1,+1} encoding decomposition,
 * for NVIDIA B200 (sm_100a).  C ABI of libmpq.so.
 *
 * The method (Sun et al., "Multi-Precision Quantized Neural Networks via Encoding
 * Decomposition of {-1,+1}"): an activation of a_bits and a weight of w_bits are
 * quantized to odd integers, written as sum_p 2^p c_p with c_p in {-1,+1} (Eq. 10),
 * stored one bit per element in bit-planes, and every dot product of a layer becomes
 * a_bits x w_bits binary-branch dot products (Eq. 7-9), each computed with xor and
 * bitcount, weighted 2^(i+j), summed, and scaled back to a real number (Eq. 18).
 *
 * Conventions for every entry point
 *   - Pointers are DEVICE pointers unless the name ends in _host.  The caller owns and
 *     sizes every buffer; the library allocates no device memory and keeps no state between
 *     calls (mpq_linear and mpq_linear_host stage through a caller-provided device workspace).
 *     Documented exceptions: mpq_linear_static works on a buffer built into the library image;
 *     mpq_linear_host / mpq_linear_host_prepared keep one helper stream and a few events per
 *     device; and per device the library remembers the multiprocessor count and which kernels
 *     have had their shared-memory limit raised (facts that never change while the process lives).
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = the
 *     default stream) unless stated otherwise.  Outputs are fully overwritten.
 *   - Return value: an mpq_status.  Errors that the host can see (null pointers, bad
 *     sizes, unsupported widths, int32 headroom) are returned before anything is
 *     launched; a launch failure maps to MPQ_ERR_CUDA.  Nothing aborts or traps.
 *   - Bit-widths are 1..8 for both operands (the paper's 64 encoding choices, Section 5.1).
 *
 * Packed layout ("planes")
 *   planes[p][row][word], p = 0..bits-1, word = 0..mpq_row_words(k)-1, uint32.
 *   Bit t of word w of a row is element 32*w + t of that row.  Bit value 1 is +1, 0 is -1.
 *   Plane p holds bit p of the level index u = (q + 2^bits - 1)/2 and carries weight 2^p
 *   (plane 0 is the low bit: "x = x1 + 2 x2").  Bits past element k-1 and the words that
 *   pad a row to a multiple of 4 words are 0 in every operand.
 */
#ifndef MPQ_H_
#define MPQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MPQ_OK = 0,
    MPQ_ERR_NULL = 1,        /* a required pointer is NULL                                   */
    MPQ_ERR_BAD_SHAPE = 2,   /* a size is negative/zero where it may not be, or ld < extent  */
    MPQ_ERR_UNSUPPORTED = 3, /* bits outside 1..8; kernel not 1x1/3x3; stride not 1/2;
                                pad > 1; C not 32, 64 or a multiple of 128; unknown enum     */
    MPQ_ERR_OVERFLOW = 4,    /* k * (2^a_bits-1) * (2^w_bits-1) >= 2^31: int32 would overflow */
    MPQ_ERR_ALIGN = 5,       /* a plane pointer is not 16-byte aligned                       */
    MPQ_ERR_CUDA = 6,        /* the CUDA runtime reported an error (launch, copy)            */
    MPQ_ERR_WORKSPACE = 7,   /* caller-provided workspace is too small                       */
    MPQ_ERR_STATIC_LIMIT = 8 /* problem needs more than the library's built-in scratch       */
} mpq_status;

typedef enum { MPQ_SCALE_PER_TENSOR = 0, MPQ_SCALE_PER_ROW = 1 } mpq_scale_mode;

/* Range limiter applied before the quantizer (Table 1): HTanh clamps x/s to [-1,1],
 * HReLU clamps it to [0,1] (negative inputs land on the level just above zero). */
typedef enum { MPQ_ACT_HTANH = 0, MPQ_ACT_HRELU = 1 } mpq_act;

/* Form of the Encoder: the level-index route (quantizer of Eq. 15, the fast path) or the
 * trigonometric encoders of Section 3.2 (Eq. 11 and its family), one sine per bit. */
typedef enum { MPQ_ENC_LEVELS = 0, MPQ_ENC_TRIG = 1 } mpq_encoder;

const char* mpq_status_string(int status);

/* Words per packed row: ceil(k/32) rounded up to a multiple of 4 (rows are 16-byte multiples).
 * Storage is bits/32 of the fp32 tensor plus this padding (the paper's memory saving). */
int64_t mpq_row_words(int64_t k);
/* Words of a whole packed operand: bits * rows * mpq_row_words(k).  0 on invalid arguments. */
int64_t mpq_packed_words(int64_t rows, int64_t k, int bits);

/* ---- Range.  A generalisation of the paper's fixed [-1,1] / [0,1] ranges (Table 1) to data-dependent ones:
 * scale_out = max |x| (HTanh) or max of max(x,0) (HReLU), NaNs ignored; one value
 * (PER_TENSOR) or one per row (PER_ROW).  x is [rows x k] with row stride ldx (elements).
 * scale_out is overwritten (the call zeroes it first, on the stream). */
int mpq_absmax(const float* x, int64_t rows, int64_t k, int64_t ldx, int mode, int act,
               float* scale_out, void* stream);

/* ---- Encoder (Fig. 1 "Encoder"; quantizer Eq. 15 with round-half-up; code Table 2 / Eq. 10;
 * one bit per element, the bit-vector storage of Section 1).
 * Per element, in fp32: inv = 1/s (0 if s is not a finite positive number),
 * y = (x*inv) * ((2^bits-1)/2) as two rounded multiplies, NaN -> 0, HReLU: max(y,0),
 * clamp to [-2^(bits-1), 2^(bits-1)-1/2], u = floor(y) + 2^(bits-1).  Plane p gets bit p of u.
 * x: [rows x k], row stride ldx; scale: 1 value or `rows` values; planes: mpq_packed_words(). */
int mpq_encode(const float* x, int64_t rows, int64_t k, int64_t ldx,
               const float* scale, int mode, int act, int bits,
               uint32_t* planes, void* stream);

/* Range and Encoder of a matrix with ONE RANGE PER ROW in a single pass over memory (weights with a
 * range per output channel, encoded once when a layer is prepared): scale_out[r] = max |x[r][.]|
 * (HTanh) or max of max(x, 0) (HReLU), NaNs ignored, exactly as mpq_absmax gives it, and planes as
 * mpq_encode gives them with those ranges.  Rows of up to 49152 elements whose starts are 16-byte
 * aligned are staged in shared memory and read from memory once; other shapes run mpq_absmax and
 * mpq_encode one after the other (same results). */
int mpq_encode_ranged(const float* x, int64_t rows, int64_t k, int64_t ldx, int act, int bits,
                      float* scale_out, uint32_t* planes, void* stream);

/* The same call with the form of the Encoder selectable (Section 3.2 "M-bit Encoding Functions").
 * MPQ_ENC_LEVELS is mpq_encode.  MPQ_ENC_TRIG evaluates the paper's periodic encoders literally:
 * with y = x/s limited by `act` to [-1,1] (HTanh) or [0,1] (HReLU) and L = 2^bits - 1,
 *     bit bits-1 (highest)   = sign( sin(L/2^bits * pi * y)),
 *     bit m-1, 1 <= m < bits = sign(-sin(L/2^m * pi * y))
 * (Eq. 11 is the case bits = 2; other widths continue the family: the highest bit has half a period
 * on [-1,1], each lower bit doubles the frequency).  Each argument L/2^m * y is one rounded fp32
 * multiply.  At a zero of a sine -- a level boundary, a tie of Eq. 15 -- the sign is that of the
 * sine just above the zero, so ties go to the upper level as in mpq_encode and x = 0 lands on the
 * level above zero.  The two forms give the same planes except for inputs within one fp32 rounding
 * of a level boundary, where each takes its own decision.  A reference form, not tuned. */
int mpq_encode_with(int encoder, const float* x, int64_t rows, int64_t k, int64_t ldx,
                    const float* scale, int mode, int act, int bits,
                    uint32_t* planes, void* stream);

/* Activations for mpq_conv: x [N][C][H][W] fp32 -> planes[bits][N][H][W][C/32]
 * (channel innermost: bit t of word cw at a pixel is channel 32*cw + t).  One range value.
 * C must be 32, 64 or a multiple of 128. */
int mpq_encode_nchw(const float* x, int N, int C, int H, int W, const float* scale, int act,
                    int bits, uint32_t* planes, void* stream);

/* Weights for mpq_conv: w [O][C][KH][KW] fp32 -> planes[bits][O][mpq_row_words(KH*KW*C)], the
 * row of output channel o ordered (kh, kw, c) with c innermost.  scale: 1 value or O values.
 * tap_sums [KH*KW][O] int32 (required): sum over c of the decoded weight q_w[o][c][kh][kw];
 * mpq_conv uses it to make out-of-image taps contribute exactly 0.  KH*KW <= 16. */
int mpq_encode_oihw(const float* w, int O, int C, int KH, int KW, const float* scale, int mode,
                    int bits, uint32_t* planes, int32_t* tap_sums, void* stream);

/* ---- Layer product (Eq. 7-10 branches, xor + bitcount; Fig. 1 "Decoder"; scale Eq. 18).
 * C = A * B^T with A = a_planes [a_bits][m][rw], B = b_planes [b_bits][n][rw], rw = mpq_row_words(k):
 *   S        = sum_{i<a_bits, j<b_bits} 2^(i+j) * sum_w popcount(A_i[r][w] xor B_j[c][w])
 *   c_i32    = (2^a_bits-1)(2^b_bits-1) k - 2 S           (= sum_t q_a[r][t] q_b[c][t], exact)
 *   c_f32    = float(c_i32) * ((a_scale/(2^a_bits-1)) * (b_scale[c]/(2^b_bits-1)))
 * c_i32 and c_f32 are [m x n] row-major with row stride ldc; either may be NULL, not both.
 * a_scale: 1 value; b_scale: 1 value (PER_TENSOR) or n values (PER_ROW); both may be NULL
 * when c_f32 is NULL.  No bias term (Section 3.1 sets it aside). */
int mpq_gemm(const uint32_t* a_planes, int a_bits, const uint32_t* b_planes, int b_bits,
             int64_t m, int64_t n, int64_t k,
             int32_t* c_i32, float* c_f32, int64_t ldc,
             const float* a_scale, const float* b_scale, int b_mode, void* stream);

/* mpq_gemm with the glue of a chained layer folded into the store.  f = float(c_i32) * alpha[c]
 * (Eq. 18); if `bias` (n values, one per output column; the paper's layer has none, Section 3.1)
 * f = f + bias[c]; if `residual` ([m x n], row stride ldc) f = f + residual[r][c]; if `relu`
 * f = max(f, 0); c_f32 = f.  One rounded fp32 operation each, in that order.  bias, residual and
 * relu need c_f32; c_i32, when given, still receives the raw accumulators. */
int mpq_gemm_fused(const uint32_t* a_planes, int a_bits, const uint32_t* b_planes, int b_bits,
                   int64_t m, int64_t n, int64_t k,
                   int32_t* c_i32, float* c_f32, int64_t ldc,
                   const float* a_scale, const float* b_scale, int b_mode,
                   const float* bias, const float* residual, int relu, void* stream);

/* ---- Convolution by the same decomposition (Section 3.1 extends it to convolutions),
 * done as an implicit im2col on the packed planes: GEMM row = output pixel (n, oh, ow),
 * GEMM k = (kh, kw, c).  x_planes from mpq_encode_nchw, w_planes and tap_sums from
 * mpq_encode_oihw.  3x3 or 1x1, stride 1 or 2, pad 0 or 1, true zero padding (a tap outside
 * the image adds 0 to the integer sum).  y [N][O][Ho][Wo], Ho = (H + 2 pad - KH)/stride + 1.
 * y_i32 / y_f32: either may be NULL, not both.  w_scale: 1 or O values. */
int mpq_conv(const uint32_t* x_planes, int a_bits, int N, int C, int H, int W,
             const uint32_t* w_planes, int w_bits, const int32_t* tap_sums,
             int O, int KH, int KW, int stride, int pad,
             int32_t* y_i32, float* y_f32,
             const float* x_scale, const float* w_scale, int w_mode, void* stream);

/* mpq_conv with the glue of a chained network folded into the store (the arithmetic of the layer
 * itself is unchanged): f = float(acc) * alpha[o]; if `residual` (fp32, layout of y) f = f + residual
 * (one rounded add); if `relu` f = max(f, 0); y_f32 = f.  If `out_max` is given, the single float it
 * points to is raised to the largest stored max(f, 0) by an exact atomic maximum: it is the range
 * the next layer's HReLU encoder needs (Table 1), taken while the outputs are still in registers.
 * The caller zeroes *out_max beforehand (mpq_zero); the call never lowers it.  residual, relu and
 * out_max need y_f32.  y_i32, when given, still receives the raw accumulators. */
int mpq_conv_fused(const uint32_t* x_planes, int a_bits, int N, int C, int H, int W,
                   const uint32_t* w_planes, int w_bits, const int32_t* tap_sums,
                   int O, int KH, int KW, int stride, int pad,
                   int32_t* y_i32, float* y_f32,
                   const float* x_scale, const float* w_scale, int w_mode,
                   const float* residual, int relu, float* out_max, void* stream);

/* ---- Deconvolution (transposed convolution) by the same decomposition (Section 3.1 names the
 * deconvolution layer, next to the fully connected and the convolution layer, as one the method
 * applies to).  y[n][o][oh][ow] = sum over (c, kh, kw, ih, iw) with oh = ih*stride - pad + kh and
 * ow = iw*stride - pad + kw of q_x[n][c][ih][iw] * q_w[o][c][kh][kw]; y is [N][O][Ho][Wo] with
 * Ho = (H-1)*stride - 2*pad + KH.  Outputs that share (oh mod stride, ow mod stride) use the same
 * taps, so the layer runs as stride^2 gathers on the packed planes, one per output phase, each with
 * the branch kernel of mpq_conv; an output position that no input reaches gets 0.
 * Filters: stride 1 or 2, stride <= KH, KW <= 4, 0 <= pad < min(KH, KW); C as for mpq_conv.
 *
 * Weights: w [O][C][KH][KW] fp32 (OUTPUT channel first; a framework that stores transposed-
 * convolution filters input channel first swaps the two axes when it hands them over).
 * mpq_encode_deconv_weights writes mpq_deconv_weight_words() words: for each filter phase
 * (r_h, r_w) = (kh mod stride, kw mod stride), in the order r_h*stride + r_w, a matrix
 * [bits][O][mpq_row_words(T_h*T_w*C)] whose row o holds the taps kh = r_h + stride*t_h,
 * kw = r_w + stride*t_w ordered (t_h, t_w, c); and tap_sums [KH*KW][O] int32 (sum over c of the
 * decoded weight, taps counted phase by phase in that same order).  scale: 1 value or O values.
 * mpq_deconv_weight_words returns 0 for arguments outside the limits above. */
int64_t mpq_deconv_weight_words(int O, int C, int KH, int KW, int stride, int bits);
int mpq_encode_deconv_weights(const float* w, int O, int C, int KH, int KW, int stride,
                              const float* scale, int mode, int bits,
                              uint32_t* planes, int32_t* tap_sums, void* stream);
/* x_planes from mpq_encode_nchw.  y_i32 / y_f32: either may be NULL, not both.  residual, relu and
 * out_max as in mpq_conv_fused (they need y_f32). */
int mpq_deconv(const uint32_t* x_planes, int a_bits, int N, int C, int H, int W,
               const uint32_t* w_planes, int w_bits, const int32_t* tap_sums,
               int O, int KH, int KW, int stride, int pad,
               int32_t* y_i32, float* y_f32,
               const float* x_scale, const float* w_scale, int w_mode,
               const float* residual, int relu, float* out_max, void* stream);

/* mpq_conv_fused that also runs the CONSUMER's Encoder in its store (Fig. 1: the Decoder of one
 * layer feeding the Encoder of the next), for networks whose ranges are known before the layer
 * runs: the paper's fixed HReLU range [0,1] (Table 1), or a calibrated constant.  The value f
 * that mpq_conv_fused would store is quantized exactly as mpq_encode_nchw would quantize it with
 * range *next_scale, limiter next_act and next_bits bits, and written as
 * next_planes[next_bits][N][Ho][Wo][O/32] (the layout mpq_encode_nchw gives that tensor), so the
 * consumer needs neither the fp32 tensor nor an encode pass.  y_f32 may then be NULL (nothing is
 * stored in fp32); y_i32, residual, relu and out_max keep their meaning.  O must be a multiple of 32.
 * With next_planes NULL this is mpq_conv_fused. */
int mpq_conv_encoded(const uint32_t* x_planes, int a_bits, int N, int C, int H, int W,
                     const uint32_t* w_planes, int w_bits, const int32_t* tap_sums,
                     int O, int KH, int KW, int stride, int pad,
                     int32_t* y_i32, float* y_f32,
                     const float* x_scale, const float* w_scale, int w_mode,
                     const float* residual, int relu, float* out_max,
                     const float* next_scale, int next_act, int next_bits, uint32_t* next_planes,
                     void* stream);

/* Sets `bytes` bytes of device memory to zero on the stream (ranges that kernels raise by atomic maximum). */
int mpq_zero(void* p, int64_t bytes, void* stream);

/* ---- Glue for chained layers (not part of the paper's method): y = max(a + b, 0) elementwise,
 * b may be NULL (plain ReLU).  n elements, fp32, one rounded add. */
int mpq_add_relu(const float* a, const float* b, float* y, int64_t n, void* stream);

/* ---- Full-precision glue of a ResNet-shaped stack (not part of the paper's method; the first
 * layer of the network stays fp32).  Stem: x [N][3][H][W], w [64][3][7][7] -> y [N][64][Ho][Wo],
 * 7x7, stride 2, zero pad 3, Ho = (H - 1)/2 + 1; relu != 0 applies max(.,0) in the store.  Each
 * output is one chain of fused multiply-adds over (c, kh, kw) in that order.
 * Max-pool: 3x3, stride 2, pad 1: x [N][C][H][W] -> y [N][C][(H - 1)/2 + 1][(W - 1)/2 + 1]; out_max
 * (optional, zeroed by the caller) is raised to the largest max(y, 0), as in mpq_conv_fused. */
int mpq_stem_conv7x7(const float* x, const float* w, float* y, int N, int H, int W, int relu,
                     void* stream);
int mpq_maxpool3x3s2(const float* x, float* y, int N, int C, int H, int W, float* out_max, void* stream);

/* ---- Whole encoded fully-connected layer (Fig. 1 end to end: Encoder of both operands,
 * the a_bits x w_bits branches, Decoder): out = decode(encode(x) . encode(w)^T).
 * x [m x k] and w [n x k] are dense fp32 DEVICE tensors; activations take one range with `a_act`,
 * weights one range (PER_TENSOR) or one per output row (PER_ROW).  out_i32 / out_f32 [m x n],
 * dense; either may be NULL, not both.
 * workspace: device memory of at least mpq_linear_workspace() bytes, 256-byte aligned, holding the
 * two ranges and the two packed operands for the duration of the call (contents undefined after). */
int64_t mpq_linear_workspace(int64_t m, int64_t n, int64_t k, int a_bits, int w_bits);
int mpq_linear(const float* x, const float* w, int64_t m, int64_t n, int64_t k,
               int a_bits, int w_bits, int a_act, int w_mode,
               int32_t* out_i32, float* out_f32,
               void* workspace, int64_t workspace_bytes, void* stream);

/* ---- The same layer for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of mpq_linear, same arithmetic, same results.)
 * Some users of this library may not call cudaMalloc at the point where they need a layer:
 * an inference plug-in running inside a host framework that has already claimed the device's
 * memory for its own pool, a service whose start-up phase is the only place allocation is
 * allowed (cudaMalloc can block on the whole device and can fail late), or a small embedding
 * program that has no allocator to lend a workspace from.  For them the two ranges and the two
 * packed operands live in a buffer that is part of the library image itself: a file-scope
 * device array of MPQ_LINEAR_STATIC_BYTES bytes that every GPU which loads libmpq.so holds
 * until the process exits.  The caller passes only inputs and outputs (device pointers, as for
 * mpq_linear).  Nothing is allocated or freed, here or in anything this call uses.
 *   - Limit: mpq_linear_workspace(m, n, k, a_bits, w_bits) must not exceed
 *     MPQ_LINEAR_STATIC_BYTES, else MPQ_ERR_STATIC_LIMIT is returned and nothing is launched.
 *   - The first call on each device looks up the buffer's device address (with that device
 *     current) and remembers it; make that first call outside any stream capture.
 *   - All calls on a device share the one buffer, and it keeps whatever the previous call left.
 *     Nothing in it has to start at zero except the range words, which the range step clears on
 *     the stream itself.  Two calls that overlap on the GPU (different streams, or different
 *     host threads without ordering between their streams) race on the buffer: serialise them. */
#define MPQ_LINEAR_STATIC_BYTES (16 * 1024 * 1024)
int mpq_linear_static(const float* x, const float* w, int64_t m, int64_t n, int64_t k,
                      int a_bits, int w_bits, int a_act, int w_mode,
                      int32_t* out_i32, float* out_f32, void* stream);

/* The same layer from HOST buffers: copies x_host and w_host into the device workspace, runs
 * mpq_linear there, and copies out_i32_host / out_f32_host [m x n] back (either may be NULL, not
 * both).  Host buffers should be pinned for the copies to be asynchronous.  The weights are
 * copied and encoded first (that work overlaps the activations' copy), and the product runs in
 * row blocks whose results are copied back on a helper stream while the next block is computed
 * (one helper stream and five events per device, created by the first call on that device and
 * kept until exit; two calls on one device must not overlap).  The call returns after everything
 * has drained (it synchronizes `stream`).
 * workspace: device memory of at least mpq_linear_host_workspace() bytes, 256-byte aligned. */
int64_t mpq_linear_host_workspace(int64_t m, int64_t n, int64_t k, int a_bits, int w_bits);
int mpq_linear_host(const float* x_host, const float* w_host, int64_t m, int64_t n, int64_t k,
                    int a_bits, int w_bits, int a_act, int w_mode,
                    int32_t* out_i32_host, float* out_f32_host,
                    void* workspace, int64_t workspace_bytes, void* stream);

/* The deployed form of mpq_linear_host: the weights were encoded once (mpq_absmax + mpq_encode)
 * and stay on the device as w_planes [w_bits][n][mpq_row_words(k)] with their range(s) w_scale
 * (1 or n values); every call moves only the activations up (x_host, [m x k]) and the results
 * down.  Same pipeline as mpq_linear_host otherwise (row blocks copied back on the helper stream
 * while the next block is computed; synchronizes `stream`; two calls on one device must not
 * overlap).  workspace: at least mpq_linear_host_prepared_workspace() bytes, 256-byte aligned. */
int64_t mpq_linear_host_prepared_workspace(int64_t m, int64_t n, int64_t k, int a_bits);
int mpq_linear_host_prepared(const float* x_host, const uint32_t* w_planes, const float* w_scale,
                             int64_t m, int64_t n, int64_t k,
                             int a_bits, int w_bits, int a_act, int w_mode,
                             int32_t* out_i32_host, float* out_f32_host,
                             void* workspace, int64_t workspace_bytes, void* stream);

/* ---- Roofline denominator: measures this GPU's 32-bit population-count issue rate with a
 * register-only loop (no memory traffic) and the SM clock it ran at.  Synchronous.
 * popc_per_s: lane-level POPC results per second over the whole chip; sm_mhz: SM clock
 * observed inside the kernel; sms: multiprocessor count.  Any pointer may be NULL. */
int mpq_measure_popc_peak(double* popc_per_s, double* sm_mhz, int* sms, void* stream);

/* ---- Roofline denominator of the carry-save form of the branch products (Eq. 7-10 computed
 * with full adders on the xor words): issue rate of a register-only loop whose groups hold
 * `logic_per_popc` (0..8) three-input logic operations, one population count and one integer
 * multiply-add.  With one full adder per two xor words the kernel's mix is 4 logic operations
 * per population count and one group stands for two algorithmic word-popcounts.  Synchronous.
 * groups_per_s: lane-level groups per second over the whole chip. */
int mpq_measure_mix_peak(int logic_per_popc, double* groups_per_s, double* sm_mhz, int* sms, void* stream);

/* ---- Roofline denominator of the legacy one-bit tensor route for the binary branches (Eq. 7-10
 * with the bitcount done by mma.sync.m16n8k256 on b1 operands): issue rate of that instruction in
 * a register-only loop with constant operands, i.e. with no operand traffic at all.  and_popc = 0
 * measures the xor.popc form (the branch product itself), 1 the and.popc form.  One warp-wide
 * instruction stands for 16 * 8 * 256 / 32 = 1024 word-popcounts.  Synchronous.
 * warp_mma_per_s: warp-level instructions per second over the whole chip. */
int mpq_measure_b1_mma_peak(int and_popc, double* warp_mma_per_s, double* sm_mhz, int* sms, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MPQ_H_ */
