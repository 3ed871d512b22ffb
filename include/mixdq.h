/*
 * mixdq.h -- C ABI of the B200 (sm_100a) library for MixDQ's quantized inference path.
 *
 * The library runs the mixed-precision quantized linear and 3x3 convolution layers
 * of a diffusion UNet: every layer carries its own weight width (3, 4 or 8 bits) and
 * activation width (8 or 16 bits).  The bit-width table itself is an input: the
 * paper's sensitivity analysis and integer program (Sec. 3.2, 3.3) run offline.
 *
 * Conventions shared by every call
 *   - Return value: 0 on success, a negative MIXDQ_ERR_* code otherwise.  Argument
 *     errors are found on the host before anything is launched.
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer owned by the
 *     caller.  The library allocates and frees no memory that the caller sees.
 *   - `stream` is a cudaStream_t passed as void*.  Calls only enqueue work on it and
 *     never synchronize.
 *   - fp16 tensors are IEEE binary16, row-major, densely packed unless a stride is given.
 *   - Weight matrices are [N, K]: N output channels, K reduction length.  A 3x3 conv
 *     weight is passed flattened to [N, 9*Cin] in (kh, kw, cin) order.
 *   - `status` (optional, may be NULL) is a device int32 word.  A kernel whose bounded
 *     wait on a barrier runs out writes a non-zero code there and returns early; the
 *     host reads it after synchronizing.  A correct run leaves it untouched.
 *
 * Quantizer (paper Sec. 4.1 "Quantization Scheme": min-max uniform quantization with one
 * scale / zero-point per activation tensor and one per weight output channel):
 *   inv = fp32(1 / scale); code = clamp(round_half_even(v * inv) [+ zero]);
 *   symmetric codes lie in [-qmax, qmax], qmax = 2^(b-1) - 1, asymmetric ones in [0, 2^b - 1].
 */
#ifndef MIXDQ_H_
#define MIXDQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MIXDQ_OK 0
#define MIXDQ_ERR_INVALID_ARG (-1) /* NULL pointer, non-positive size, bad enum */
#define MIXDQ_ERR_UNSUPPORTED (-2) /* a width / shape combination the library does not run */
#define MIXDQ_ERR_ALIGNMENT (-3)   /* pointer or stride not aligned as documented */
#define MIXDQ_ERR_WORKSPACE (-4)   /* workspace missing or too small */
#define MIXDQ_ERR_CUDA (-5)        /* a CUDA runtime / driver call failed */
#define MIXDQ_ERR_TIMEOUT (-6)     /* written to `status` by a kernel whose wait ran out */

#define MIXDQ_LAYOUT_CANONICAL 0 /* documented, engine-independent byte layout */
#define MIXDQ_LAYOUT_DEVICE 1    /* layout the GEMM / conv kernels read */

#define MIXDQ_TOKENS_PER_PROMPT 77 /* text tokens per prompt; token 0 is BOS (Sec. 3.1) */

/* Library version as major*10000 + minor*100 + patch. */
int mixdq_version(void);

/* Number of kernels the layer calls (mixdq_linear, mixdq_conv3x3, mixdq_conv1x1,
 * mixdq_crossattn_kv and their variants) have launched, or recorded into a stream capture, in
 * this process so far: a measurement aid for counting launches per step. */
unsigned long long mixdq_kernel_launches(void);

/* Diagnostic (the paper has no counterpart): the output tile the W8A8 / W4A8 tensor-core GEMM uses, on the
 * current device and with a workspace, for a layer of M output rows, N output channels and k_blocks
 * reduction blocks of 128 (linear layer: ceil(K / 128); 3x3 convolution: 9 * ceil(Cin / 128)).
 * *tile_rows x *tile_cols (HOST pointers) is 256 x {160, 192, 224, 256} when two CTAs on neighbouring SMs
 * share a tile (tcgen05 cta_group::2), else 128 x {64, 96, 128, 256}.  The BOS-aware projection and the second branch
 * of a shortcut-split layer always run on 128-row tiles.  *reduction_splits (HOST): for 256-row tiles the number
 * of CTA pairs that share one tile's reduction (1: each pair walks whole tiles; 2 to 4: layers with few tiles and
 * a long reduction, partial sums added through distributed shared memory); 0 for 128-row tiles.  A linear layer for
 * which mixdq_linear_fused_quant_tile is positive runs as one kernel on 128-row tiles of that width instead, and a
 * shortcut-split layer (mixdq_linear_a8_split, mixdq_conv3x3_a8_split) takes the 256-row tiles reported for the sum of
 * its branches' reduction blocks, without a split reduction, or else 128-row tiles.  For tests and benchmarks: nothing
 * is launched. */
int mixdq_int8_tile_plan(int64_t M, int64_t N, int64_t k_blocks, int w_bits, int* tile_rows, int* tile_cols,
                         int* reduction_splits);

/* Diagnostic (the paper has no counterpart; its implementation runs the activation quantization as a kernel of
 * its own, Sec. 4.1 "Hardware Profiling"): width of the 128-row output tiles when mixdq_linear, called with a
 * workspace, 8-bit symmetric activations and a row-major X, runs a layer of M rows, N channels and K inputs as ONE
 * kernel that quantizes its activation tiles itself; 0 when the layer runs as quantization pass + GEMM (the
 * one-kernel form pays only for short reductions, K <= 640, on one wave of tiles).  Negative: an error code.
 * For tests and benchmarks: nothing is launched. */
int mixdq_linear_fused_quant_tile(int64_t M, int64_t N, int64_t K, int w_bits);

/* Static, NUL-terminated description of an error code (host pointer, never NULL). */
const char* mixdq_strerror(int code);

/*
 * Bytes of a packed [N, K] weight matrix.  `out` is a HOST pointer.
 * Canonical layout: row pitch K (8-bit), ceil(K/2) (4-bit, even k in the low nibble),
 * ceil(K/32)*12 (3-bit: per group of 32 codes three little-endian u32 bit-planes, bit j of
 * plane p = bit p of code 32g+j; a ragged last group is padded with the row's zero-point),
 * ceil(K/32)*8 (2-bit, the lowest candidate width of Sec. 3.3: the same with two planes).
 * Device layout: 8-bit rows padded to a multiple of 16 bytes; 4-bit rows padded to a
 * multiple of 32 codes with, inside every group of 8 codes, byte j holding code j in the
 * low nibble and code j+4 in the high nibble; 3-bit rows padded to a multiple of 128
 * codes, each block of 128 codes stored as three 16-byte bit-planes whose bits are
 * interleaved for the register decode (mixdq_unpack_weights undoes it); 2-bit rows alike with
 * two planes per block (32 bytes per 128 codes).
 */
int mixdq_packed_bytes(int64_t N, int64_t K, int bits, int layout, size_t* out);

/*
 * Per-output-channel min-max parameters of W (fp16 [N, K]) -- Sec. 4.1.
 * symmetric != 0: scale[n] = max_k |w| / qmax, zero[n] = 0.
 * symmetric == 0: lo = min(min_k w, 0), hi = max(max_k w, 0), L = 2^bits - 1,
 *                 scale[n] = (hi - lo) / L, zero[n] = clamp(rne(-lo * inv), 0, L).
 * A constant-zero row gets scale 1.  `zero_out` may be NULL when symmetric.
 */
int mixdq_weight_minmax_params(const void* W, int64_t N, int64_t K, int bits, int symmetric,
                               float* scale_out, int32_t* zero_out, void* stream);

/*
 * Quantize W (fp16 [N, K]) with the given per-channel scale (and zero-point) and pack the
 * codes.  bits in {2, 3, 4, 8}.  zero == NULL selects symmetric signed codes (not available
 * for 2 and 3 bits).  `packed_out` must hold mixdq_packed_bytes(N, K, bits, layout) bytes and be
 * 16-byte aligned.  This is the offline step of the path: it runs once per layer.
 */
int mixdq_pack_weights(const void* W, int64_t N, int64_t K, int bits, const float* scale,
                       const int32_t* zero, int layout, void* packed_out, void* stream);

/*
 * Parity hook: integer codes (int16 [N, K]) back out of a packed buffer in either layout.
 * is_signed tells how 4- and 8-bit fields are read.
 */
int mixdq_unpack_weights(const void* packed, int64_t N, int64_t K, int bits, int is_signed,
                         int layout, int16_t* codes_out, void* stream);

/*
 * max |x| over an fp16 matrix [rows, cols] with row stride `row_stride` elements, written to
 * amax_out[0] (fp32).  skip_rows_mod > 0 leaves out every row whose index is a multiple of
 * it: 77 removes the BOS token of every prompt from the range (Sec. 3.1).
 */
int mixdq_act_absmax(const void* X, int64_t rows, int64_t cols, int64_t row_stride,
                     int skip_rows_mod, float* amax_out, void* stream);

/* scale_out[0] = amax[0] / 127 (one fp32 division; 1 when amax is 0): the per-tensor
 * symmetric int8 activation scale of Sec. 4.1 computed on the device. */
int mixdq_act_scale_from_absmax(const float* amax, float* scale_out, void* stream);

/*
 * Range of an fp16 matrix [rows, cols] (row stride `row_stride` elements) with 0 included:
 * minmax_out[0] = min(min x, 0), minmax_out[1] = max(max x, 0) (device fp32 [2]).  The first step of the
 * asymmetric min-max activation quantizer (Sec. 4.1 "Quantization Scheme").
 */
int mixdq_act_minmax(const void* X, int64_t rows, int64_t cols, int64_t row_stride, float* minmax_out,
                     void* stream);

/* Asymmetric 8-bit parameters from that range, on the device: scale_out[0] = (hi - lo) / 255 (fp32),
 * zero_out[0] = clamp(rne(-lo / scale), 0, 255) (int32); scale 1 and zero 0 when hi == lo. */
int mixdq_act_asym_params_from_minmax(const float* minmax, float* scale_out, int32_t* zero_out,
                                      void* stream);

/* sums_out[n] = sum_k q[n, k] (device int32 [N]) of the signed codes of a MIXDQ_LAYOUT_DEVICE weight with
 * bits in {4, 8}: computed once per layer, it carries the activation zero-point through the int8 GEMM. */
int mixdq_weight_code_sums(const void* packed_W, int64_t N, int64_t K, int bits, int32_t* sums_out,
                           void* stream);

/*
 * Bytes of scratch memory the layer calls below need for a given problem (HOST `out`).
 * rows = output rows (tokens or output pixels), N, K as in the layer call.  The scratch
 * must be 256-byte aligned.  Nothing in it has to be initialised or to survive between calls
 * (a call clears what it needs cleared), so one buffer of the largest size can serve every
 * layer of a model -- as long as the calls that share it do not overlap on the GPU.
 * A result of 0 means the call runs without scratch.  The workspace is optional for every
 * call (NULL / 0 bytes): without it the int8 layers run as one fused kernel that quantizes
 * the activations while it feeds the tensor cores; with it, the activations are first
 * quantized once into the workspace and the GEMM is then fed entirely by TMA.  Weight-only
 * layers (act_bits = 16) on 256 rows or more use a workspace too: the layer's weights are
 * expanded once per call to fp16 integers (q - zero) there and the GEMM runs on fp16 tensor
 * cores with both operands fed by TMA (the paper's weight-only mode saves memory, not time:
 * Table 1 caption); without it, or on fewer rows, weight tiles are expanded inside the GEMM.
 */
int mixdq_workspace_bytes(int64_t rows, int64_t N, int64_t K, int w_bits, int act_bits,
                          size_t* out);

/* The same for mixdq_conv3x3 (its int8 path keeps a quantized copy of the input image). */
int mixdq_conv3x3_workspace_bytes(int64_t B, int64_t H, int64_t W, int64_t Cin, int64_t Cout,
                                  int stride, int w_bits, int act_bits, size_t* out);

/*
 * Constants of a layer.  packed_W, w_scale, w_zero, bias, the weight code sums and a stored BOS row are
 * constants of the layer (the paper quantizes weights offline, Sec. 4.1).  The layer kernels may load
 * them BEFORE they wait for earlier work on the stream, so that their start overlaps the previous
 * kernel's end; they must therefore be complete when a layer call that reads them is enqueued.  Buffers
 * written by mixdq_pack_weights, mixdq_weight_minmax_params and mixdq_weight_code_sums on the SAME stream
 * satisfy this by themselves (those calls end with a full stream dependency).  Constants produced any
 * other way (a copy, a kernel of the caller's, another stream) need a stream synchronization or an event
 * wait between their producer and the first layer call that uses them.  Everything else -- X, the
 * activation scale and zero-point, the workspace, Y -- follows ordinary stream order.
 */

/*
 * Quantized linear layer  Y[M, N] = X[M, K] * dequant(W)^T + bias   (paper Sec. 4.1, 4.3).
 *   act_bits == 8 : W8A8 / W4A8.  X is quantized per tensor with *act_scale (device fp32)
 *                   inside the kernel, multiplied with the integer weight codes in int32
 *                   and dequantized as  y = fp16(acc * act_scale * w_scale[n] + bias[n]).
 *                   Weights must be symmetric (w_zero == NULL), w_bits in {4, 8}.
 *   act_bits == 16: weight-only W2/W3/W4/W8-A16 (Table 1 "weight only" rows): X stays fp16,
 *                   y = fp16(w_scale[n] * sum_k x[k] * (q[n,k] - w_zero[n]) + bias[n]).
 *                   act_scale is ignored.  w_zero == NULL means signed codes, zero-point 0.
 * packed_W is in MIXDQ_LAYOUT_DEVICE.  ldx is the row stride of X in elements (>= K,
 * multiple of 8).  bias (fp16 [N]) may be NULL.  Y is dense [M, N].  X, Y 16-byte aligned.
 */
int mixdq_linear(const void* X, int64_t M, int64_t K, int64_t ldx, const void* packed_W, int64_t N,
                 int w_bits, const float* w_scale, const int32_t* w_zero, int act_bits,
                 const float* act_scale, const void* bias, void* Y, void* workspace,
                 size_t workspace_bytes, int32_t* status, void* stream);

/* Parity hook of the int8 path: the raw int32 accumulators acc[M, N] = sum_k qx * qw that
 * mixdq_linear(act_bits = 8) would dequantize. */
int mixdq_linear_acc_i32(const void* X, int64_t M, int64_t K, int64_t ldx, const void* packed_W,
                         int64_t N, int w_bits, const float* act_scale, int32_t* acc_out,
                         void* workspace, size_t workspace_bytes, int32_t* status, void* stream);

/*
 * W8A8 / W4A8 linear layer with ASYMMETRIC per-tensor activations, the quantizer the paper uses
 * (Sec. 4.1 "Quantization Scheme": asymmetric min-max): unsigned codes q = clamp(rne(x / s) + z, 0, 255),
 *   Y[m, n] = fp16( s * w_scale[n] * sum_k (q[m, k] - z) * qw[n, k] + bias[n] ).
 * The tensor cores multiply the re-centred int8 codes q - 128; the term (128 - z) * w_code_sums[n]
 * (mixdq_weight_code_sums) restores the zero-point in the epilogue.  act_scale (fp32) and act_zero (int32)
 * are device scalars, e.g. from mixdq_act_asym_params_from_minmax.  Other arguments as in mixdq_linear.
 * Unlike mixdq_linear this call NEEDS the workspace (mixdq_workspace_bytes(M, N, K, w_bits, 8)) and
 * K % 16 == 0, ldx % 8 == 0, K <= 66000; it returns MIXDQ_ERR_UNSUPPORTED otherwise.
 */
int mixdq_linear_a8_asym(const void* X, int64_t M, int64_t K, int64_t ldx, const void* packed_W, int64_t N,
                         int w_bits, const float* w_scale, const int32_t* w_code_sums,
                         const float* act_scale, const int32_t* act_zero, const void* bias, void* Y,
                         void* workspace, size_t workspace_bytes, int32_t* status, void* stream);

/* Parity hook: acc[M, N] = sum_k (q[m, k] - z) * qw[n, k] as int32. */
int mixdq_linear_a8_asym_acc_i32(const void* X, int64_t M, int64_t K, int64_t ldx, const void* packed_W,
                                 int64_t N, int w_bits, const int32_t* w_code_sums, const float* act_scale,
                                 const int32_t* act_zero, int32_t* acc_out, void* workspace,
                                 size_t workspace_bytes, int32_t* status, void* stream);

/*
 * Quantized 3x3 convolution as an implicit GEMM (all linear and conv layers are quantized,
 * Sec. 4.1 "Mixed Precision Allocation").  X fp16 NHWC [B, H, W, Cin], zero padding 1,
 * stride in {1, 2}; packed_W is the [Cout, 9*Cin] matrix in (kh, kw, cin) order; Y fp16 NHWC
 * [B, Ho, Wo, Cout] with Ho = (H - 1) / stride + 1.  Width arguments as in mixdq_linear.
 */
int mixdq_conv3x3(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin, const void* packed_W,
                  int64_t Cout, int stride, int w_bits, const float* w_scale, const int32_t* w_zero,
                  int act_bits, const float* act_scale, const void* bias, void* Y, void* workspace,
                  size_t workspace_bytes, int32_t* status, void* stream);

/*
 * The 3x3 convolution with asymmetric per-tensor activations (as mixdq_linear_a8_asym; Sec. 4.1).  The zero
 * padding is the real value 0, whose code is the zero-point: the call keeps the int8 image in the workspace
 * with a one-pixel border of that code, so border outputs need no special case.  w_code_sums =
 * mixdq_weight_code_sums(packed_W, Cout, 9 * Cin, w_bits).  NEEDS the workspace
 * (mixdq_conv3x3_workspace_bytes) and a geometry the two-kernel path takes (Cin % 32 == 0; Wo a multiple of
 * 128, or 128 / Wo a divisor or a multiple of Ho; stride 2 only on even H, W): MIXDQ_ERR_UNSUPPORTED otherwise.
 */
int mixdq_conv3x3_a8_asym(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin, const void* packed_W,
                          int64_t Cout, int stride, int w_bits, const float* w_scale,
                          const int32_t* w_code_sums, const float* act_scale, const int32_t* act_zero,
                          const void* bias, void* Y, void* workspace, size_t workspace_bytes, int32_t* status,
                          void* stream);

/* Parity hook: acc[B, Ho, Wo, Cout] = sum over the window of (q - z) * qw as int32. */
int mixdq_conv3x3_a8_asym_acc_i32(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin,
                                  const void* packed_W, int64_t Cout, int stride, int w_bits,
                                  const int32_t* w_code_sums, const float* act_scale, const int32_t* act_zero,
                                  int32_t* acc_out, void* workspace, size_t workspace_bytes, int32_t* status,
                                  void* stream);

/*
 * Activations stored as int8 between layers (the activation-memory saving of Sec. 4.3 / Table 2: an 8-bit
 * activation tensor is kept as its codes plus one scale).  The two steps of mixdq_linear with act_bits = 8
 * as calls of their own:
 *   mixdq_quantize_acts: Xq_out[r, k] = clamp(rne(X[r, k] / *act_scale), -127, 127) as a dense int8
 *     [rows, K] matrix (the symmetric per-tensor activation quantizer of Sec. 4.1; the paper's separate
 *     quantization kernel).  K % 16 == 0, ldx % 8 == 0 (MIXDQ_ERR_UNSUPPORTED otherwise), both pointers
 *     16-byte aligned.
 *   mixdq_linear_q8: Y = fp16(*act_scale * w_scale[n] * sum_k Xq[m, k] * qw[n, k] + bias[n]) on such codes
 *     (dense [M, K], 16-byte aligned, K % 16 == 0).  Several layers that read the same tensor (the q, k and v
 *     projections of self-attention) then share one quantization pass.  Needs no workspace.  Symmetric
 *     weights, w_bits in {4, 8}.
 */
int mixdq_quantize_acts(const void* X, int64_t rows, int64_t K, int64_t ldx, const float* act_scale, void* Xq_out,
                        void* stream);

int mixdq_linear_q8(const void* Xq, int64_t M, int64_t K, const void* packed_W, int64_t N, int w_bits,
                    const float* w_scale, const float* act_scale, const void* bias, void* Y, int32_t* status,
                    void* stream);

/*
 * The W8A8 / W4A8 linear layer of mixdq_linear as ONE kernel on 128 x tile_cols output tiles, whatever the planner
 * would choose: the GEMM kernel takes the fp16 activations by TMA and quantizes every tile itself (Sec. 4.1:
 * symmetric per-tensor 8-bit activations, the same codes as mixdq_quantize_acts), so no workspace is needed and
 * no quantization kernel runs; the output bits equal mixdq_linear's.  The paper runs the quantization as a kernel
 * of its own; this form trades that launch for arithmetic repeated in every tile column, and is faster only for
 * short reductions (mixdq_linear_fused_quant_tile).  tile_cols: a multiple of 32 in [32, 256]
 * (MIXDQ_ERR_INVALID_ARG otherwise).  X fp16 [M, K] with row stride ldx (K % 16 == 0, ldx % 8 == 0:
 * MIXDQ_ERR_UNSUPPORTED otherwise; 16-byte aligned), Y fp16 [M, N] with row stride ldy; symmetric weights,
 * w_bits in {4, 8}; bias may be NULL.  All pointers DEVICE except status (device, may be NULL) and stream.
 */
int mixdq_linear_a8_fused_quant(const void* X, int64_t M, int64_t K, int64_t ldx, const void* packed_W, int64_t N,
                                int w_bits, const float* w_scale, const float* act_scale, const void* bias, void* Y,
                                int64_t ldy, int tile_cols, int32_t* status, void* stream);

/* The 3x3 convolution on a stored int8 NHWC image [B, H, W, Cin] (codes from mixdq_quantize_acts on the
 * [B*H*W, Cin] pixel matrix); zero padding is code 0.  Geometry as for the two-kernel path of mixdq_conv3x3
 * (Cin % 32 == 0; Wo a multiple of 128, or 128 / Wo a divisor or a multiple of Ho; stride 2 only on even H, W):
 * MIXDQ_ERR_UNSUPPORTED otherwise.  Other arguments as in mixdq_linear_q8. */
int mixdq_conv3x3_q8(const void* Xq, int64_t B, int64_t H, int64_t W, int64_t Cin, const void* packed_W,
                     int64_t Cout, int stride, int w_bits, const float* w_scale, const float* act_scale,
                     const void* bias, void* Y, int32_t* status, void* stream);

/*
 * Self-test of the kernels' bounded waits (the paper has no counterpart).  Runs mixdq_linear_q8 on the given
 * operands, except that the weight tile of reduction block drop_k_block (1-based, blocks of 128) is announced
 * to its barrier and then never requested.  The warps that wait for it give up when their cycle budget (a few
 * hundred milliseconds) runs out: the kernel raises its abort flag, lets its copies in flight land, writes
 * MIXDQ_ERR_TIMEOUT to *status (required), releases its tensor memory and returns; nothing traps and the
 * context stays usable.  Y is written with unspecified values.  The call itself returns MIXDQ_OK (the launch
 * succeeded).  For tests: it shows that a lost transfer ends in a status word, not in a hung GPU.
 */
int mixdq_selftest_abandoned_wait(const void* Xq, int64_t M, int64_t K, const void* packed_W, int64_t N, int w_bits,
                                  const float* w_scale, const float* act_scale, void* Y, int drop_k_block,
                                  int32_t* status, void* stream);

/* Parity hook: int32 accumulators [M, N] of mixdq_linear_q8. */
int mixdq_linear_q8_acc_i32(const void* Xq, int64_t M, int64_t K, const void* packed_W, int64_t N, int w_bits,
                            int32_t* acc_out, int32_t* status, void* stream);

/*
 * Shortcut-splitting (Sec. 4.1, "Quantization Scheme"): a layer whose input is a concatenation of two
 * branches with different ranges (the skip connections of the UNet's up path) keeps one per-tensor
 * activation scale per branch.  Row elements [0, split_at) of X (channels, for a convolution) are
 * quantized with *act_scale_lo, elements [split_at, K) with *act_scale_hi; each part is multiplied with its
 * own part of the weights into an exact int32 sum, and
 *     y[m, n] = fp16( (s_lo * acc_lo[m, n] + s_hi * acc_hi[m, n]) * w_scale[n] + bias[n] ).
 * The weights arrive as two packed matrices made offline with mixdq_pack_weights from the two column
 * ranges of W and the SAME per-output-channel scale (taken over the whole row): packed_W_lo is
 * [N, split_at] and packed_W_hi [N, K - split_at]; for a convolution W[..., :split_at] and
 * W[..., split_at:] flattened to [Cout, 9 * split_at] and [Cout, 9 * (Cin - split_at)] in (kh, kw, cin) order.
 * Symmetric weights, w_bits in {4, 8}; symmetric activations.  NEEDS a workspace of
 * mixdq_split_workspace_bytes(in_rows, row_len, split_at, out_rows, N) bytes, where (in_rows, row_len,
 * out_rows) = (M, K, M) for a linear layer and (B*H*W, Cin, B*Ho*Wo) for a convolution; it holds the two
 * int8 copies and the first branch's int32 sums (the second branch's kernel reads them in its epilogue), must be
 * 16-byte aligned, needs no initial content, and calls sharing it must not overlap.
 * split_at and K - split_at (Cin - split_at) must suit the two-kernel path: multiples of 16 (convolution:
 * of 32, with an image geometry as for mixdq_conv3x3_a8_asym), ldx % 8 == 0, X 16-byte aligned;
 * MIXDQ_ERR_UNSUPPORTED otherwise, MIXDQ_ERR_WORKSPACE when the workspace is missing or too small.
 */
int mixdq_split_workspace_bytes(int64_t in_rows, int64_t row_len, int64_t split_at, int64_t out_rows, int64_t N,
                                size_t* out);

int mixdq_linear_a8_split(const void* X, int64_t M, int64_t K, int64_t ldx, int64_t split_at,
                          const void* packed_W_lo, const void* packed_W_hi, int64_t N, int w_bits,
                          const float* w_scale, const float* act_scale_lo, const float* act_scale_hi,
                          const void* bias, void* Y, void* workspace, size_t workspace_bytes, int32_t* status,
                          void* stream);

/* Parity hook: the two int32 sums [M, N] of a shortcut-split linear layer, before the epilogue. */
int mixdq_linear_a8_split_acc_i32(const void* X, int64_t M, int64_t K, int64_t ldx, int64_t split_at,
                                  const void* packed_W_lo, const void* packed_W_hi, int64_t N, int w_bits,
                                  const float* act_scale_lo, const float* act_scale_hi, int32_t* acc_lo_out,
                                  int32_t* acc_hi_out, void* workspace, size_t workspace_bytes, int32_t* status,
                                  void* stream);

/* Shortcut-splitting on a 3x3 convolution (NHWC input whose channels [0, split_at) and [split_at, Cin) come
 * from the two branches); other arguments as in mixdq_conv3x3 and mixdq_linear_a8_split. */
int mixdq_conv3x3_a8_split(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin, int64_t split_at,
                           const void* packed_W_lo, const void* packed_W_hi, int64_t Cout, int stride, int w_bits,
                           const float* w_scale, const float* act_scale_lo, const float* act_scale_hi,
                           const void* bias, void* Y, void* workspace, size_t workspace_bytes, int32_t* status,
                           void* stream);

/* Parity hook: the two int32 sums [B, Ho, Wo, Cout] of a shortcut-split convolution. */
int mixdq_conv3x3_a8_split_acc_i32(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin, int64_t split_at,
                                   const void* packed_W_lo, const void* packed_W_hi, int64_t Cout, int stride,
                                   int w_bits, const float* act_scale_lo, const float* act_scale_hi,
                                   int32_t* acc_lo_out, int32_t* acc_hi_out, void* workspace,
                                   size_t workspace_bytes, int32_t* status, void* stream);

/* Parity hook: int32 accumulators [B, Ho, Wo, Cout] of the int8 conv path. */
int mixdq_conv3x3_acc_i32(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin,
                          const void* packed_W, int64_t Cout, int stride, int w_bits,
                          const float* act_scale, int32_t* acc_out, void* workspace,
                          size_t workspace_bytes, int32_t* status, void* stream);

/* 1x1 convolution on NHWC = mixdq_linear on the [B*H*W, Cin] pixel matrix. */
int mixdq_conv1x1(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin, const void* packed_W,
                  int64_t Cout, int w_bits, const float* w_scale, const int32_t* w_zero, int act_bits,
                  const float* act_scale, const void* bias, void* Y, void* workspace,
                  size_t workspace_bytes, int32_t* status, void* stream);

/*
 * BOS-aware cross-attention K or V projection (Sec. 3.1).  text_emb fp16 [B, 77, Kt].
 * Token 0 of every prompt takes no part in the computation: Y[b, 0, :] is a bit-for-bit
 * copy of bos_out (fp16 [N], the floating-point projection of the BOS embedding computed
 * ahead of time), rows 1..76 run the W8A8 / W4A8 path with *act_scale (whose range the
 * caller takes over tokens 1..76 only, e.g. mixdq_act_absmax with skip_rows_mod = 77).
 * Y fp16 [B, 77, N].  No bias (to_k / to_v have none).
 */
int mixdq_crossattn_kv(const void* text_emb, int64_t B, int64_t Kt, const void* packed_W, int64_t N,
                       int w_bits, const float* w_scale, const float* act_scale,
                       const void* bos_out, void* Y, void* workspace, size_t workspace_bytes,
                       int32_t* status, void* stream);

/* Parity hook: int32 accumulators [B, 76, N] of the rows the int8 path computes. */
int mixdq_crossattn_kv_acc_i32(const void* text_emb, int64_t B, int64_t Kt, const void* packed_W,
                               int64_t N, int w_bits, const float* act_scale, int32_t* acc_out,
                               void* workspace, size_t workspace_bytes, int32_t* status,
                               void* stream);

/*
 * Measurement aid (the paper reports no kernel-level throughput): every SM issues
 * `batches` x 128 back-to-back 128x256 tensor-core MMAs on operands resident in shared
 * memory, with no loads and no epilogue.  kind 1 = int8 -> int32 (the W8A8 / W4A8 engine's
 * instruction), kind 0 = fp16 -> fp32.  *ops_out (HOST) receives 2 * multiply-adds issued by
 * the whole grid; dividing by the time of the call, measured by the caller with CUDA events,
 * gives the MMA-loop peak that benchmark fractions are quoted against.
 */
int mixdq_probe_mma_loop(int kind, int batches, double* ops_out, int32_t* status, void* stream);

/*
 * (No counterpart in the paper: an addition for hosts that cannot allocate.)
 * mixdq_linear with act_bits = 8 for callers that have no device memory to give as a
 * workspace -- a process whose memory manager owns the whole GPU, code embedded in another
 * framework's allocator, or a loop that cannot afford the device-wide synchronization of
 * cudaMalloc.  The layer's scratch -- the int8 copy of X that the quantization pass writes and
 * the GEMM reads, placed behind the region a split reduction would use -- is a fixed array of
 * mixdq_static_scratch_bytes() bytes (8 MiB) inside the library image; every GPU that loads
 * the library holds it until the process exits.  The call allocates and frees nothing.
 *   - A problem whose scratch need (mixdq_workspace_bytes) exceeds the array is rejected with
 *     MIXDQ_ERR_WORKSPACE; nothing is launched.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Make that first call outside any stream capture.
 *   - All calls share the one array, which keeps the previous call's contents; a call
 *     overwrites what it reads (and clears what it needs zeroed) itself, so two calls that can
 *     overlap on the GPU (different streams) race: serialize them.
 * Arguments as in mixdq_linear; weights symmetric, w_bits in {4, 8}.
 */
size_t mixdq_static_scratch_bytes(void);
int mixdq_linear_a8_static_scratch(const void* X, int64_t M, int64_t K, int64_t ldx,
                                   const void* packed_W, int64_t N, int w_bits, const float* w_scale,
                                   const float* act_scale, const void* bias, void* Y, int32_t* status,
                                   void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MIXDQ_H_ */
