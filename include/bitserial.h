/*
 * bitserial.h -- C ABI of the bit-serial ultra-low-bit convolution library for NVIDIA B200 (sm_100a).
 *
 * Method (paper, Section V): weights (w bits) and activations (a bits) are split into bitplanes and
 * packed into machine words.  A dot product is then
 *       1-bit unipolar:   W . A = POPCOUNT(W & A)
 *       multi-bit:        W . A = sum_{i<w} sum_{j<a} POPCOUNT(W[i] & A[j]) << (i + j)
 * Extensions the paper leaves open and this library fixes:
 *   - two's-complement operands: the top plane carries weight -2^(b-1);
 *   - 1-bit bipolar operands {-1,+1} (stored bit 1 <-> +1): v = 2*bit - 1 is expanded algebraically,
 *     which for two bipolar operands is the identity dot = K - 2*POPCOUNT(a XOR w);
 *   - zero padding (value 0 has every plane 0, so out-of-image taps add nothing);
 *   - a fused per-output-channel requantisation epilogue (Section IV quantiser applied to
 *     scale*acc + bias), exact operation order documented at bs_conv_params.
 * The quantiser (paper, Section IV) is  code = round(clip(x / s, qmin, qmax)), round-to-nearest-even,
 * with [qmin, qmax] = [-2^(b-1), 2^(b-1)-1] (signed) or [0, 2^b-1] (unsigned).
 *
 * General conventions
 *   - Every function returns a bs_status.  Nothing throws, aborts or prints.
 *   - Every tensor pointer is DEVICE memory owned by the caller, 16-byte aligned, valid on the current
 *     device; `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls
 *     only enqueue work; they never synchronise and never allocate device memory.
 *   - bs_conv_params / scalar arguments are HOST values, read before the call returns.
 *   - Supported: bit-widths 1..4; sign BS_BIPOLAR only with 1 bit; square kernels R == S in
 *     {1, 3, 5, 7}; stride in {1, 2}; 0 <= pad < R.  Bipolar activations need pad == 0 (zero is not
 *     representable).  Shapes must keep |acc| < 2^31 (checked on the host).
 *
 * Packed storage (uint32 words, little-endian bit numbering):
 *   activations  [N][H][W][Cw][a_bits]      Cw = ceil(C / 32)
 *   weights      [O][R][S][Cw][w_bits]
 *   matrix rows  [rows][Kw][bits]           Kw = ceil(K / 32)
 *   Bit (c % 32) of word (c / 32) of plane j holds bit j of the stored pattern of channel c.  The
 *   stored pattern of an unsigned or two's-complement code is its low `bits` bits; a bipolar code
 *   stores 1 for +1 and 0 for -1.  Channels beyond C are stored as 0 in every plane.
 *   A 1x1 convolution over N*H*W pixels and a matrix product over M = N*H*W rows use identical bytes.
 */
#ifndef BITSERIAL_H_
#define BITSERIAL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BS_OK = 0,
    BS_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, bits outside 1..4, bad enum ...      */
    BS_ERR_UNSUPPORTED = 2, /* well-formed but outside the supported set listed above                 */
    BS_ERR_ALIGNMENT = 3,   /* a tensor pointer is not 16-byte aligned                                */
    BS_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed (launch error, no device, ...)       */
    BS_ERR_TIMEOUT = 5      /* a bounded device-side wait ran out (reported by bs_check_status)       */
} bs_status;

typedef enum { BS_UNSIGNED = 0, BS_SIGNED = 1, BS_BIPOLAR = 2 } bs_sign_t;
typedef enum { BS_NCHW = 0, BS_NHWC = 1 } bs_layout_t; /* for weights: OIHW = BS_NCHW, OHWI = BS_NHWC */

/* Bytes of a packed activation tensor / packed weight tensor / packed row matrix (0 on bad input). */
size_t bs_packed_act_bytes(int N, int C, int H, int W, int a_bits);
size_t bs_packed_wgt_bytes(int O, int C, int R, int S, int w_bits);
size_t bs_packed_rows_bytes(int rows, int K, int bits);

/*
 * bitpack_activations -- Section IV quantiser followed by the Section V bitplane split.
 *   x          device, [N][C][H][W] (BS_NCHW) or [N][H][W][C] (BS_NHWC); float32 when x_is_fp32 != 0,
 *              otherwise int8 codes already inside the code range of (a_bits, a_sign).
 *   act_scale  the step s of the quantiser (> 0, finite); ignored for int8 input.
 *              Bipolar: code = +1 when x >= 0 else -1.
 *   packed_out device, bs_packed_act_bytes(N, C, H, W, a_bits) bytes, fully overwritten.
 * The quantiser is evaluated in its comparison form (bs_quantiser_bounds), which takes the formula's decision for every
 * float32 input: +-inf clip to the limits, a NaN gets the lowest code.  One pass over x; bound by HBM bandwidth.
 */
int bitpack_activations(const void* x, int x_is_fp32, bs_layout_t layout, int N, int C, int H, int W,
                        float act_scale, int a_bits, bs_sign_t a_sign, uint32_t* packed_out, void* stream);

/*
 * bs_quantiser_bounds -- the comparison form of the Section IV quantiser that bitpack_activations evaluates.  Host call,
 * no device work.  Writes to bounds_out[k] (HOST memory, 2^a_bits - 1 floats; one for bipolar codes) the smallest
 * float32 input whose code is >= qmin + k + 1 under round_half_even(clip(x / act_scale, qmin, qmax)), found by bisection
 * with that very formula, so that  code = qmin + #{k : x >= bounds_out[k]}  for every float32 x (a NaN reaches no
 * level).  Returns BS_ERR_INVALID_ARG for a null pointer, a scale that is not positive and finite, or a bad width/sign.
 */
int bs_quantiser_bounds(float act_scale, int a_bits, bs_sign_t a_sign, float* bounds_out);

/* Inverse of the plane split (test and debugging aid): packed activations -> int8 codes in `layout`. */
int bitunpack_activations(const uint32_t* packed, int N, int C, int H, int W, int a_bits, bs_sign_t a_sign,
                          bs_layout_t layout, int8_t* codes_out, void* stream);

/*
 * pack_weights -- Section V bitplane split of quantised weights (done once per layer, off the hot loop).
 *   w_codes    device int8, [O][C][R][S] (BS_NCHW) or [O][R][S][C] (BS_NHWC), inside the code range.
 *   packed_out device, bs_packed_wgt_bytes(O, C, R, S, w_bits) bytes, fully overwritten.
 */
int pack_weights(const int8_t* w_codes, bs_layout_t layout, int O, int C, int R, int S, int w_bits,
                 bs_sign_t w_sign, uint32_t* packed_out, void* stream);

/* Plane split of a row-major int8 code matrix [rows][K] into [rows][Kw][bits] (operands of bitserial_gemm). */
int bs_pack_rows(const int8_t* codes, int rows, int K, int bits, bs_sign_t sign, uint32_t* packed_out,
                 void* stream);

/*
 * Convolution problem (host struct).  Output size P = (H + 2*pad - R)/stride + 1, Q likewise.
 *
 * Accumulator (exact int32):  acc[n][o][p][q] = sum_{c,r,s} a[n][c][p*stride-pad+r][q*stride-pad+s] * w[o][c][r][s]
 * evaluated as the Section V plane-pair popcount sum with the sign handling described at the top.
 *
 * Epilogue, applied when out_packed != NULL, in exactly this order in IEEE binary32:
 *     v = fmaf((float)acc, scale[o], bias[o]);
 *     if (residual) v = fmaf(res_scale, (float)res_code, v);
 *     if (relu)     v = fmaxf(v, 0.0f);
 *     v = fminf(fmaxf(v, qmin), qmax);            (clip, then round: order of the Section IV quantiser)
 *     code = (int) rintf(v);                      (ties to even; out_sign BS_BIPOLAR: code = v >= 0 ? +1 : -1)
 * and the codes are split into out_bits planes and stored as packed activations [N][P][Q][Ow][out_bits]
 * with Ow = ceil(out_c_total / 32), at channels [out_c_offset, out_c_offset + O) (concatenation for free).
 */
typedef struct {
    int N, C, H, W;          /* input: batch, channels, height, width                                 */
    int O, R, S;             /* filters and kernel size                                                */
    int stride, pad;
    int a_bits;  int a_sign; /* activation bits and bs_sign_t                                          */
    int w_bits;  int w_sign; /* weight bits and bs_sign_t (1-bit signed weights are BS_BIPOLAR)        */
    const float* scale;      /* device [O]; required iff out_packed != NULL                            */
    const float* bias;       /* device [O]; required iff out_packed != NULL                            */
    int relu;
    int out_bits; int out_sign;      /* code range of the packed output (the next layer's activations) */
    const uint32_t* residual;        /* device, packed activations [N][P][Q][ceil(res_c_total/32)][res_bits] or NULL */
    float res_scale;
    int res_bits; int res_sign;
    int res_c_offset, res_c_total;   /* the residual code of output channel o is channel res_c_offset + o */
    int out_c_offset, out_c_total;   /* out_c_offset is a multiple of 32; O is too unless the slice ends the tensor */
    int i32_layout;                  /* bs_layout_t of out_i32: [N][O][P][Q] or [N][P][Q][O]              */
} bs_conv_params;

/*
 * bitserial_conv2d -- Section V bit-serial convolution (implicit GEMM over packed bitplanes) with the
 * fused epilogue.
 *   act_packed  device, packed activations of shape (N, C, H, W, a_bits)
 *   wgt_packed  device, packed weights of shape (O, C, R, S, w_bits)
 *   out_i32     device or NULL: raw accumulators in p->i32_layout
 *   out_packed  device or NULL: requantised, packed output (see bs_conv_params); the channel range
 *               written is fully overwritten, other channels of a wider tensor are left untouched.
 * At least one output must be non-NULL.  Asynchronous on `stream`.
 */
int bitserial_conv2d(const uint32_t* act_packed, const uint32_t* wgt_packed, const bs_conv_params* p,
                     int32_t* out_i32, uint32_t* out_packed, void* stream);

/*
 * bitserial_gemm -- Section V bit-serial dot products on plain matrices:
 *     out[m][n] = sum_{k<K} a[m][k] * w[n][k]
 *   a_packed  device [M][Kw][a_bits], w_packed device [N][Kw][w_bits] (bs_pack_rows layout)
 *   out_i32   device or NULL, row-major [M][N]
 *   out_packed device or NULL, [M][ceil(N/32)][out_bits], epilogue as in bs_conv_params with
 *             scale/bias indexed by n (scale, bias may be NULL when out_packed is NULL)
 */
int bitserial_gemm(const uint32_t* a_packed, const uint32_t* w_packed, int M, int N, int K, int a_bits,
                   bs_sign_t a_sign, int w_bits, bs_sign_t w_sign, const float* scale, const float* bias,
                   int relu, int out_bits, bs_sign_t out_sign, int32_t* out_i32, uint32_t* out_packed,
                   void* stream);

/*
 * Reduction split over several thread blocks (for problems with few output tiles and a long reduction, e.g. a
 * 256 x 256 matrix product with K = 4608, or a 7 x 7 layer with 512 channels).  The Section V sum is associative,
 * so partial popcount sums of disjoint channel-word ranges are added in a caller-provided workspace and the last
 * block of a tile applies the epilogue; results are bit-identical to the unsplit entry points.
 *   workspace        device, 16-byte aligned, at least bs_*_workspace_bytes(...) bytes; it must be ZERO before the
 *                    first call and every call leaves it zero again, so one cudaMemset at allocation suffices.
 *                    Calls that share a workspace must not overlap on the GPU (use one stream, or one workspace
 *                    per stream).  A NULL or too small workspace falls back to the unsplit kernel.
 *   bs_*_workspace_bytes  bytes the planner wants for this shape on the CURRENT device (0: no split would be used).
 *                    Plans depend on the multiprocessor count, which is looked up per device: ask with the device
 *                    current on which the call will run.  No launch.
 */
size_t bs_conv_workspace_bytes(const bs_conv_params* p);
size_t bs_gemm_workspace_bytes(int M, int N, int K, int a_bits, bs_sign_t a_sign, int w_bits, bs_sign_t w_sign);
int bitserial_conv2d_ws(const uint32_t* act_packed, const uint32_t* wgt_packed, const bs_conv_params* p,
                        int32_t* out_i32, uint32_t* out_packed, void* workspace, size_t workspace_bytes, void* stream);
int bitserial_gemm_ws(const uint32_t* a_packed, const uint32_t* w_packed, int M, int N, int K, int a_bits,
                      bs_sign_t a_sign, int w_bits, bs_sign_t w_sign, const float* scale, const float* bias,
                      int relu, int out_bits, bs_sign_t out_sign, int32_t* out_i32, uint32_t* out_packed,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * bitserial_gemm_noalloc -- bitserial_gemm with the reduction split, for callers that must not allocate device
 * memory.  (The paper has no counterpart: this is a deployment convenience of this library, not part of the method.)
 *
 * Who needs it: host programs that hand all device memory to their own pool at start-up, inference loops that
 * are forbidden to call cudaMalloc/cudaFree after initialisation (those calls synchronise the whole device and
 * can fail late), and plugins that run inside another framework's stream and have no allocator of their own.
 * Such callers cannot provide the workspace bitserial_gemm_ws asks for, so the scratch for the partial sums is a
 * 2 MiB array built into the library image (bs_gemm_noalloc_max_scratch_bytes()); every GPU that loads the
 * library holds those 2 MiB until the process exits.  This call never calls cudaMalloc, cudaFree or any
 * allocating routine.
 *
 *   Arguments, outputs and results are exactly those of bitserial_gemm (bit-identical).
 *   Limit: shapes whose split plan needs more than the built-in scratch (roughly M*N above 400 thousand outputs
 *   when the planner splits) return BS_ERR_UNSUPPORTED and launch nothing; use bitserial_gemm or bitserial_gemm_ws.
 *   Shapes the planner does not split run the ordinary kernel and touch no scratch.
 *   First call on a device: looks up the device address of the built-in array (once per device, with that device
 *   current).  Make that first call before starting any stream capture.
 *   Sharing: all calls on a device use the same array, which keeps the previous call's contents.  A call that ran to
 *   completion leaves the part it used zero again (the last block of a tile restores it), so the clearing each call
 *   does on `stream` before its kernel is a guard against a predecessor that did NOT complete normally (one that ended
 *   with BS_ERR_TIMEOUT) and against a caller that wrote to the array.  Two calls that overlap on the GPU (different
 *   streams without ordering) race on the array and give wrong results; serialise them.
 */
size_t bs_gemm_noalloc_max_scratch_bytes(void);
/* Test aid (no counterpart in the paper): fills the built-in scratch with `byte_value` on `stream`, as a predecessor that
 * ended half-way would leave it.  A following bitserial_gemm_noalloc on the same stream must still be exact. */
int bs_selftest_dirty_noalloc_scratch(int byte_value, void* stream);
int bitserial_gemm_noalloc(const uint32_t* a_packed, const uint32_t* w_packed, int M, int N, int K, int a_bits,
                           bs_sign_t a_sign, int w_bits, bs_sign_t w_sign, const float* scale, const float* bias,
                           int relu, int out_bits, bs_sign_t out_sign, int32_t* out_i32, uint32_t* out_packed,
                           void* stream);

/*
 * Tensor-core formulation (exactly equivalent integer MMA).  The Section V plane-pair popcount sum is the integer
 * dot product of the unpacked codes, so the same int32 accumulators are produced by an int8 x int8 -> int32 matrix
 * product: activations stay bit-packed in memory and are expanded to int8 inside the kernel, filters are expanded
 * once by bs_tc_prepare_weights.  Results (accumulators and requantised codes) are bit-identical to
 * bitserial_conv2d / bitserial_gemm; the epilogue is the one documented at bs_conv_params.
 *   Supported subset (bs_tc_supported returns 1): C a multiple of 32 whose packed pixel record (C/32 * a_bits words)
 *   is a 16-byte multiple, or an 8-byte multiple when a packed image row (W records) is a 16-byte multiple and, for
 *   1x1 stride-1 layers, N*H*W is even; res_c_offset a multiple of 32; everything else as bitserial_conv2d.  Unsupported shapes return BS_ERR_UNSUPPORTED: use the
 *   popcount entry points.
 *   bs_tc_weights_bytes    bytes of the prepared int8 filter tensor (0 on bad input).
 *   bs_tc_prepare_weights  packed weights [O][R][S][Cw][w_bits] -> int8 tiles [C/32][ceil(O/128)*16][R*S][2][8][16]
 *                          (blocks of 32 channels; a_bits is accepted for forward compatibility).
 */
size_t bs_tc_weights_bytes(int O, int C, int R, int S);
int bs_tc_prepare_weights(const uint32_t* wgt_packed, int O, int C, int R, int S, int w_bits, bs_sign_t w_sign,
                          int a_bits, int8_t* wgt_tc_out, void* stream);
int bs_tc_supported(const bs_conv_params* p);
int bitserial_conv2d_tc(const uint32_t* act_packed, const int8_t* wgt_tc, const bs_conv_params* p, int32_t* out_i32,
                        uint32_t* out_packed, void* stream);
/*
 * bitserial_conv2d_tc_chained -- bitserial_conv2d_tc for a layer inside a chain of layers on one stream (the paper
 * runs a network layer by layer, Section V; overlapping consecutive layers is this library's addition).  The kernel
 * is launched so that its set-up (barriers, tensor memory, filter fetch, scale/bias fetch) may run while the
 * preceding kernel of `stream` is still finishing; activations and the residual are read, and outputs written,
 * only after that kernel has completed.  The CALLER PROMISES that wgt_tc, p->scale and p->bias were final before
 * the preceding kernel of the stream was launched (e.g. prepared at model load time, followed by a
 * synchronisation).  Results are identical to bitserial_conv2d_tc; errors likewise.  Works under stream capture.
 */
int bitserial_conv2d_tc_chained(const uint32_t* act_packed, const int8_t* wgt_tc, const bs_conv_params* p,
                                int32_t* out_i32, uint32_t* out_packed, void* stream);
/*
 * bitserial_conv2d_tc_chain -- 2 to 4 consecutive layers of a network in ONE launch (the paper runs a network layer by layer
 * and names tiling and parallelisation as the source of its speed, Section V; running several layers as one grid whose tiles
 * wait for the tiles they depend on, instead of one grid per layer, is this library's addition).  Every layer computes exactly
 * what bitserial_conv2d_tc computes for its bs_conv_params; results are identical.
 *   layers[l]        bs_conv_params of layer l.  All layers share N, C, H, W, O = C, R = S, pad = (R-1)/2, stride 1 (the output
 *                    is as large as the input), the activation and weight formats, and a packed output (out_bits > 0, no
 *                    channel offset: out_c_offset 0, out_c_total O) whose format is the next layer's activation format; a
 *                    residual, if any, has res_c_offset 0 and res_c_total O.  scale, bias and residual are DEVICE pointers.
 *   act_packed[l], wgt_tc[l], out_packed[l]   HOST arrays of `nlayers` DEVICE pointers: packed input, prepared filters
 *                    (bs_tc_prepare_weights) and packed output of layer l.  A layer may read -- as input or residual -- the
 *                    output of any EARLIER layer of the chain, or tensors that were final before the launch; an output must
 *                    not overlap a tensor the same chain reads unless that tensor is the output of an earlier layer or the
 *                    input of one.  Outputs of all layers are materialised in full.
 *   workspace        DEVICE, 16-byte aligned, at least bs_tc_chain_workspace_bytes(layers, nlayers) bytes, zero-filled by the
 *                    caller once before its first use (and again after a launch that ended with BS_ERR_TIMEOUT); the library
 *                    keeps per-tile progress counters in it from launch to launch.  One workspace serves one chain; launches
 *                    that share a workspace must not overlap on the GPU.
 *   chained          non-zero: launched like bitserial_conv2d_tc_chained (same promise by the caller, for every layer).
 * bs_tc_chain_workspace_bytes returns 0 when the layers cannot run as one chain (shapes differ, a layer does not take the
 * resident-filter plan, more than 4 layers); bitserial_conv2d_tc_chain then returns BS_ERR_UNSUPPORTED and launches nothing:
 * call bitserial_conv2d_tc per layer.  Other errors: BS_ERR_INVALID_ARG (null pointer, workspace too small),
 * BS_ERR_ALIGNMENT, BS_ERR_CUDA.  Every device-side wait is bounded (about a second); one that runs out sets the status
 * word read by bs_check_status.  Asynchronous on `stream`; works under stream capture.
 */
size_t bs_tc_chain_workspace_bytes(const bs_conv_params* layers, int nlayers);
int bitserial_conv2d_tc_chain(int nlayers, const uint32_t* const* act_packed, const int8_t* const* wgt_tc,
                              const bs_conv_params* layers, uint32_t* const* out_packed, void* workspace,
                              size_t workspace_bytes, int chained, void* stream);
int bitserial_gemm_tc(const uint32_t* a_packed, const int8_t* w_tc, int M, int N, int K, int a_bits, bs_sign_t a_sign,
                      int w_bits, bs_sign_t w_sign, const float* scale, const float* bias, int relu, int out_bits,
                      bs_sign_t out_sign, int32_t* out_i32, uint32_t* out_packed, void* stream);

/*
 * Layers kept in floating point.  The paper's mixed-precision networks keep "a few quantization-sensitive layers in FP32 and the
 * rest quantized down to 2 bits" (Section VII-D; the runtime of Section VI executes both kinds): in a residual classifier the
 * first convolution with its pooling, and the final pooling + fully connected layer.  The paper gives no arithmetic for them; this
 * library fixes it, because the quantiser behind the stem turns every rounding into a possible code change: IEEE binary32;
 *   bs_conv2d_f32       out[n][o][p][q] = chain of fused multiply-adds starting at bias[o] (0 when bias is NULL) over the taps in
 *                       the order c (outermost), r, s (innermost), all ascending; out-of-image taps add nothing; optional ReLU.
 *                       x [N][C][H][W], w [O][C][R][S], out [N][O][P][Q], device, 16-byte aligned.  Any R, S, stride >= 1, pad >= 0.
 *   bs_maxpool2d_f32    maximum over the k x k window positions inside the image (padding never wins); 2*pad <= k.
 *   bs_avgpool_codes_f32  global average pool of packed activation codes [N][H][W][Cw][a_bits] -> float [N][C]: the exact integer
 *                       sum of the H*W codes of a channel, converted to float and multiplied once by `inv` (code step / (H*W)).
 *   bs_fc_f32           out[n][j] = chain of fused multiply-adds starting at bias[j] over k ascending of x[n][k] * w[j][k];
 *                       x [N][K], w [J][K], out [N][J].
 * All asynchronous on `stream`; errors BS_ERR_INVALID_ARG / BS_ERR_ALIGNMENT / BS_ERR_UNSUPPORTED / BS_ERR_CUDA.
 */
int bs_conv2d_f32(const float* x, const float* w, const float* bias, int N, int C, int H, int W, int O, int R, int S, int stride,
                  int pad, int relu, float* out, void* stream);
int bs_maxpool2d_f32(const float* x, int N, int C, int H, int W, int k, int stride, int pad, float* out, void* stream);
int bs_avgpool_codes_f32(const uint32_t* packed, int N, int C, int H, int W, int a_bits, bs_sign_t a_sign, float inv, float* out,
                         void* stream);
int bs_fc_f32(const float* x, const float* w, const float* bias, int N, int K, int J, float* out, void* stream);

/*
 * bs_check_status -- synchronises `stream`, then reads and clears the device status word of the current
 * device.  Returns BS_ERR_TIMEOUT if any kernel since the last check gave up on a bounded wait (its
 * outputs are then undefined), BS_ERR_CUDA if the stream reports an error, else BS_OK.
 */
int bs_check_status(void* stream);

/*
 * bs_requant_bounds -- the comparison form of the requantisation epilogue for 1- and 2-bit outputs (the paper gives no
 * epilogue; this is the library's fixed order fma, residual fma, ReLU, clip, round-half-even).  Host call, no device
 * work.  With t = fmaf((float)acc, scale[o], bias[o]) the output code is  qmin + #{k : t >= bound[r][k]}  where r is
 * the stored pattern of the residual code (0 when there is none); writes bound[r][0..2] to bounds_out[3 r + k] (HOST
 * memory, 3 floats per residual pattern, 2^res_bits patterns; +inf for levels that do not exist).  Returns
 * BS_ERR_UNSUPPORTED for outputs wider than 2 bits (the kernels evaluate the formula there), BS_ERR_INVALID_ARG for a
 * null pointer or a bad width/sign.
 */
int bs_requant_bounds(int has_residual, float res_scale, int res_bits, bs_sign_t res_sign, int relu, int out_bits,
                      bs_sign_t out_sign, float* bounds_out);

/*
 * bs_selftest_wait_timeout -- exercises the failure path of the kernels' device-side waits without any fault (the paper
 * has no counterpart; Section V only describes the computation).  Launches, on `stream`, a one-warp kernel that waits
 * with the library's bounded wait on a barrier at which nothing ever arrives, gives up after `polls` polls (1..65536)
 * and sets the device status word like a convolution kernel whose staged tile never arrived.  The kernel always
 * returns; the next bs_check_status(stream) reports BS_ERR_TIMEOUT once and clears the word, and the device stays
 * usable.  Returns BS_ERR_INVALID_ARG for a poll count outside the range, BS_ERR_CUDA if the launch failed.
 */
int bs_selftest_wait_timeout(int polls, void* stream);

/*
 * bs_l2_prefetch -- asks the memory system to bring `count` device buffers into the L2 cache (bulk prefetches; the
 * kernel that issues them ends at once and the transfers overlap whatever runs next on `stream`).  Used at the start
 * of a forward pass for the prepared filters of all layers, which a layer otherwise fetches from HBM chunk by chunk
 * on its critical path (the paper keeps its weights in the CPU caches implicitly; it has no counterpart of this call).
 *   buffers  HOST array of `count` device pointers, 16-byte aligned;  bytes  HOST array of sizes (rounded down to 16).
 * Nothing is modified; a hint only.  Errors: BS_ERR_INVALID_ARG, BS_ERR_ALIGNMENT, BS_ERR_CUDA.
 */
int bs_l2_prefetch(const void* const* buffers, const size_t* bytes, int count, void* stream);

/*
 * bs_popc_rate -- register-only micro-benchmark of the SM population-count pipe: every thread runs
 * `iters` rounds of independent  acc += popc(x & y)  chains.  Writes the measured rate in
 * popc32(AND) word-operations per second to *wordops_per_s (HOST pointer).  Synchronises the device.
 * Used to state the arithmetic roofline of the convolution kernel beside its measured time.
 */
int bs_popc_rate(int iters, double* wordops_per_s);

/* Human-readable name of a bs_status (static storage). */
const char* bs_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* BITSERIAL_H_ */
