/*
 * MixDQ reference oracle (test infrastructure, not product code).
 *
 * A plain, slow, obviously-correct CPU statement of what the quantized
 * linear / conv hot path of MixDQ computes.  It exists so that the CUDA
 * library can be checked against something written straight from the paper.
 * Only tests, the smoke check and the CPU-baseline leg of the benchmark may
 * call it; the CUDA library shares no code with it.
 *
 * Everything here works on host memory.  fp16 tensors travel as uint16_t
 * bit patterns so that no compiler half type is involved.
 *
 * What follows the paper, by passage:
 *   - Sec. 4.1 "Quantization Scheme": min-max uniform quantizer; one
 *     (scale, zero-point) per activation tensor, one per weight output
 *     channel.
 *   - Sec. 4.1 "Mixed Precision Allocation": every linear and conv layer is
 *     quantized with its own bit-widths; norms and non-linearities are not.
 *   - Sec. 3.1 (BOS-aware text embedding quantization): token 0 is left out
 *     of the activation range and of the computation; its output row is a
 *     stored floating-point vector.
 *   - Table 1 caption / Appendix "hardware experiments" (2): weight-only
 *     rows keep FP16 activations and FP16 compute.
 *   - Sec. 4.3 / Appendix (4): W8A8 and W4A8 both run 8-bit integer MACs.
 *
 * Readings taken where the paper is silent (each is listed in the design
 * notes of the repository):
 *   - rounding is round-half-to-even of the exact product v * inv, where
 *     inv = fp32(1 / scale) is one IEEE single-precision division;
 *   - symmetric codes use the restricted range [-qmax, +qmax],
 *     qmax = 2^(b-1) - 1; asymmetric codes use [0, 2^b - 1] with an integer
 *     zero-point and a range that always contains 0;
 *   - a constant-zero tensor/row gets scale 1 and all-zero codes.
 *
 * Parity pins live in tests/test_oracle_*.py: exhaustive fp16 conversion
 * against numpy, the |dequant - v| <= scale/2 bound, brute force dot
 * products, closed forms for conv tap counts, the W8A16 == fake-quant matmul
 * identity, hand-derived bit-plane words and Table 1's storage ratios.
 * Image-quality metrics of the paper (FID, CLIP score, ImageReward, SSIM at
 * the UNet output): parity unpinned -- they need the trained weights.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_OK 0
#define ORC_ERR_ARG (-1)
#define ORC_ERR_OVERFLOW (-2)

/* ------------------------------------------------------------------ */
/* fp16 <-> double, written out from the IEEE 754 binary16 definition. */
/* ------------------------------------------------------------------ */

static double half_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int expo = (h >> 10) & 0x1f;
    int frac = h & 0x3ff;
    double v;
    if (expo == 0) {
        v = ldexp((double)frac, -24); /* zero and subnormals: frac * 2^-24 */
    } else if (expo == 31) {
        v = frac ? NAN : INFINITY;
    } else {
        v = ldexp((double)(frac + 1024), expo - 25); /* (1 + frac/1024) * 2^(expo-15) */
    }
    return sign ? -v : v;
}

/* Round a double to the nearest binary16 (ties to even), overflow to inf. */
static uint16_t double_to_half(double d)
{
    uint16_t sign = 0;
    if (signbit(d)) {
        sign = 0x8000;
        d = -d;
    }
    if (isnan(d)) return (uint16_t)(sign | 0x7e00);
    if (isinf(d)) return (uint16_t)(sign | 0x7c00);
    if (d == 0.0) return sign;
    int e;
    (void)frexp(d, &e); /* d = m * 2^e with m in [0.5, 1) => exponent of d is e-1 */
    int expo = e - 1;
    if (expo < -14) expo = -14; /* subnormal range shares the spacing 2^-24 */
    /* spacing of binary16 numbers around d is 2^(expo-10) */
    double q = nearbyint(ldexp(d, 10 - expo)); /* default rounding mode: ties to even */
    /* q is in [0, 2048]; 2048 means the rounding carried into the next binade */
    if (q >= 2048.0) {
        q = 1024.0;
        expo += 1;
    }
    if (expo > 15) return (uint16_t)(sign | 0x7c00);
    uint16_t bits;
    if (q < 1024.0) {
        bits = (uint16_t)q; /* subnormal (expo == -14 here) */
    } else {
        bits = (uint16_t)(((expo + 15) << 10) | ((int)q - 1024));
    }
    return (uint16_t)(sign | bits);
}

double orc_half_to_double(uint16_t h) { return half_to_double(h); }
uint16_t orc_double_to_half(double d) { return double_to_half(d); }

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ */
/* Quantizer (Sec. 4.1, "Quantization Scheme").                         */
/* ------------------------------------------------------------------ */

/* inv = fp32(1 / scale): one IEEE single-precision division. */
static float inv_of_scale(float scale)
{
    volatile float one = 1.0f; /* volatile: keep this a run-time fp32 divide */
    volatile float s = scale;
    volatile float r = one / s;
    return r;
}

/* Round-half-even of the exact product v * inv.  v has an 11-bit
 * significand and inv a 24-bit one, so the double product is exact. */
static int64_t rne_product(double v, float inv)
{
    double p = v * (double)inv;
    if (p > 1e15) p = 1e15;
    if (p < -1e15) p = -1e15;
    return (int64_t)nearbyint(p);
}

static int64_t clamp_i64(int64_t x, int64_t lo, int64_t hi)
{
    return x < lo ? lo : (x > hi ? hi : x);
}

/* Per-output-channel min-max parameters of a weight matrix W[N,K].
 * symmetric: scale = max|w| / qmax, zero = 0.
 * asymmetric: lo = min(min w, 0), hi = max(max w, 0), L = 2^b - 1,
 *             scale = (hi - lo) / L, zero = clamp(rne(-lo * inv), 0, L).
 * Both divisions are single fp32 operations on exactly converted inputs. */
int orc_weight_minmax_params(const uint16_t *W, int64_t N, int64_t K, int bits, int symmetric,
                             float *scale_out, int32_t *zero_out)
{
    if (!W || !scale_out || N < 0 || K <= 0 || bits < 2 || bits > 8) return ORC_ERR_ARG;
    for (int64_t n = 0; n < N; ++n) {
        double lo = 0.0, hi = 0.0, amax = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            double w = half_to_double(W[n * K + k]);
            if (w < lo) lo = w;
            if (w > hi) hi = w;
            if (fabs(w) > amax) amax = fabs(w);
        }
        if (symmetric) {
            float qmax = (float)((1 << (bits - 1)) - 1);
            volatile float a = (float)amax; /* exact: a max of fp16 values */
            volatile float s = a / qmax;
            scale_out[n] = (amax == 0.0) ? 1.0f : s;
            if (zero_out) zero_out[n] = 0;
        } else {
            float L = (float)((1 << bits) - 1);
            volatile float fhi = (float)hi, flo = (float)lo; /* exact conversions */
            volatile float range = fhi - flo;                /* one fp32 subtraction */
            volatile float s = range / L;                    /* one fp32 division */
            float scale = (range == 0.0f) ? 1.0f : s;
            scale_out[n] = scale;
            if (zero_out) {
                int64_t z = rne_product(-lo, inv_of_scale(scale));
                zero_out[n] = (int32_t)clamp_i64(z, 0, (1 << bits) - 1);
            }
        }
    }
    return ORC_OK;
}

/* Weight codes.  zero == NULL: symmetric signed codes in [-qmax, qmax].
 * Otherwise unsigned codes q = clamp(rne(w * inv) + z, 0, 2^b - 1). */
int orc_quantize_weights(const uint16_t *W, int64_t N, int64_t K, int bits, const float *scale,
                         const int32_t *zero, int16_t *codes_out)
{
    if (!W || !scale || !codes_out || N < 0 || K <= 0 || bits < 2 || bits > 8) return ORC_ERR_ARG;
    for (int64_t n = 0; n < N; ++n) {
        float inv = inv_of_scale(scale[n]);
        for (int64_t k = 0; k < K; ++k) {
            double w = half_to_double(W[n * K + k]);
            int64_t r = rne_product(w, inv);
            int64_t q;
            if (zero) {
                q = clamp_i64(r + zero[n], 0, (1 << bits) - 1);
            } else {
                int64_t qmax = (1 << (bits - 1)) - 1;
                q = clamp_i64(r, -qmax, qmax);
            }
            codes_out[n * K + k] = (int16_t)q;
        }
    }
    return ORC_OK;
}

/* Dequantized weight value of a code, in double: s * (q - z). */
int orc_dequantize_weights(const int16_t *codes, int64_t N, int64_t K, const float *scale,
                           const int32_t *zero, double *w_out)
{
    if (!codes || !scale || !w_out) return ORC_ERR_ARG;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k)
            w_out[n * K + k] = (double)scale[n] * (double)(codes[n * K + k] - (zero ? zero[n] : 0));
    return ORC_OK;
}

/* max |x| over a row-major fp16 matrix; rows whose index is a multiple of
 * skip_rows_mod are left out when skip_rows_mod > 0 (Sec. 3.1: with 77 text
 * tokens per prompt, skip_rows_mod = 77 removes the BOS token of every
 * prompt from the range). */
int orc_act_absmax(const uint16_t *X, int64_t rows, int64_t cols, int64_t row_stride,
                   int skip_rows_mod, float *amax_out)
{
    if (!X || !amax_out || rows < 0 || cols < 0 || skip_rows_mod < 0) return ORC_ERR_ARG;
    double amax = 0.0;
    for (int64_t r = 0; r < rows; ++r) {
        if (skip_rows_mod > 0 && r % skip_rows_mod == 0) continue;
        for (int64_t c = 0; c < cols; ++c) {
            double v = fabs(half_to_double(X[r * row_stride + c]));
            if (v > amax) amax = v;
        }
    }
    *amax_out = (float)amax;
    return ORC_OK;
}

/* Per-tensor symmetric activation scale from the range: amax / qmax. */
int orc_act_scale(float amax, int bits, float *scale_out)
{
    if (!scale_out || bits < 2 || bits > 8) return ORC_ERR_ARG;
    volatile float a = amax;
    volatile float qmax = (float)((1 << (bits - 1)) - 1);
    volatile float s = a / qmax;
    *scale_out = (amax == 0.0f) ? 1.0f : s;
    return ORC_OK;
}

/* Per-tensor symmetric activation codes: clamp(rne(x * inv), -qmax, qmax). */
int orc_quantize_acts(const uint16_t *X, int64_t count, int bits, float scale, int8_t *codes_out)
{
    if (!X || !codes_out || count < 0 || bits < 2 || bits > 8) return ORC_ERR_ARG;
    float inv = inv_of_scale(scale);
    int64_t qmax = (1 << (bits - 1)) - 1;
    for (int64_t i = 0; i < count; ++i)
        codes_out[i] = (int8_t)clamp_i64(rne_product(half_to_double(X[i]), inv), -qmax, qmax);
    return ORC_OK;
}

/* Asymmetric per-tensor activation quantization (Sec. 4.1 "Quantization Scheme": the paper's scheme is
 * asymmetric min-max; used here for 8-bit activations of linear layers).
 * Range: lo = min(min x, 0), hi = max(max x, 0) over the tensor; scale = (hi - lo) / 255 (one fp32
 * division of exactly converted inputs); zero = clamp(rne(-lo * inv), 0, 255); hi == lo: scale 1, zero 0.
 * Same reading as for the asymmetric weights above. */
int orc_act_minmax_params(const uint16_t *X, int64_t count, float *scale_out, int32_t *zero_out)
{
    if (!X || !scale_out || !zero_out || count < 0) return ORC_ERR_ARG;
    double lo = 0.0, hi = 0.0;
    for (int64_t i = 0; i < count; ++i) {
        double v = half_to_double(X[i]);
        if (v < lo) lo = v;
        if (v > hi) hi = v;
    }
    if (hi == lo) {
        *scale_out = 1.0f;
        *zero_out = 0;
        return ORC_OK;
    }
    volatile float range = (float)hi - (float)lo; /* both exact in fp32; one fp32 subtraction */
    volatile float levels = 255.0f;
    volatile float s = range / levels;
    *scale_out = s;
    *zero_out = (int32_t)clamp_i64(rne_product(-lo, inv_of_scale(s)), 0, 255);
    return ORC_OK;
}

/* Centred codes of an asymmetrically quantized tensor: c = clamp(rne(x * inv) + zero, 0, 255) - zero,
 * i.e. what the integer GEMM multiplies (a value in [-255, 255], hence int16). */
int orc_quantize_acts_asym(const uint16_t *X, int64_t count, float scale, int32_t zero, int16_t *centred_out)
{
    if (!X || !centred_out || count < 0 || zero < 0 || zero > 255) return ORC_ERR_ARG;
    float inv = inv_of_scale(scale);
    for (int64_t i = 0; i < count; ++i) {
        int64_t q = clamp_i64(rne_product(half_to_double(X[i]), inv) + zero, 0, 255);
        centred_out[i] = (int16_t)(q - zero);
    }
    return ORC_OK;
}

/* acc[m,n] = sum_k cx[m,k] * qw[n,k] for centred activation codes, checked against int32 overflow. */
int orc_int_gemm_i16(const int16_t *cx, const int16_t *qw, int64_t M, int64_t N, int64_t K, int32_t *acc_out)
{
    if (!cx || !qw || !acc_out || M < 0 || N < 0 || K < 0) return ORC_ERR_ARG;
    int overflow = 0;
#pragma omp parallel for schedule(static) reduction(| : overflow)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            int64_t acc = 0;
            for (int64_t k = 0; k < K; ++k) acc += (int64_t)cx[m * K + k] * (int64_t)qw[n * K + k];
            if (acc > INT32_MAX || acc < INT32_MIN) overflow = 1;
            acc_out[m * N + n] = (int32_t)acc;
        }
    }
    return overflow ? ORC_ERR_OVERFLOW : ORC_OK;
}

/* ------------------------------------------------------------------ */
/* Canonical packed layouts.                                           */
/*   8-bit: one byte per code.                                         */
/*   4-bit: two codes per byte, even k in the low nibble (two's-       */
/*          complement nibble when signed); row pitch ceil(K/2).       */
/*   3-bit: unsigned codes only; per row, per group of 32 codes, three */
/*          little-endian u32 planes P0,P1,P2 with bit j of Pp = bit p */
/*          of code[32 g + j]; a ragged last group is padded with      */
/*          pad_code (the row's zero-point, so padding dequantizes to  */
/*          0); row pitch ceil(K/32) * 12.                             */
/*   2-bit: the same with two planes P0,P1 (four codes per byte: the   */
/*          paper's lowest candidate width, Sec. 3.3); pitch           */
/*          ceil(K/32) * 8.                                            */
/* ------------------------------------------------------------------ */

int64_t orc_packed_row_bytes(int64_t K, int bits)
{
    if (K <= 0) return -1;
    if (bits == 8) return K;
    if (bits == 4) return (K + 1) / 2;
    if (bits == 3 || bits == 2) return ((K + 31) / 32) * 4 * bits;
    return -1;
}

int orc_pack_codes(const int16_t *codes, int64_t N, int64_t K, int bits, const int32_t *pad_code,
                   uint8_t *packed_out)
{
    int64_t pitch = orc_packed_row_bytes(K, bits);
    if (!codes || !packed_out || pitch < 0 || N < 0) return ORC_ERR_ARG;
    memset(packed_out, 0, (size_t)(pitch * N));
    for (int64_t n = 0; n < N; ++n) {
        uint8_t *row = packed_out + n * pitch;
        if (bits == 8) {
            for (int64_t k = 0; k < K; ++k) row[k] = (uint8_t)(codes[n * K + k] & 0xff);
        } else if (bits == 4) {
            for (int64_t k = 0; k < K; ++k) {
                uint8_t nib = (uint8_t)(codes[n * K + k] & 0xf);
                row[k / 2] |= (uint8_t)((k % 2) ? (nib << 4) : nib);
            }
        } else {
            int64_t groups = (K + 31) / 32;
            for (int64_t g = 0; g < groups; ++g) {
                uint32_t plane[3] = {0u, 0u, 0u};
                for (int j = 0; j < 32; ++j) {
                    int64_t k = 32 * g + j;
                    int c = (k < K) ? codes[n * K + k] : (pad_code ? pad_code[n] : 0);
                    if (c < 0 || c >= (1 << bits)) return ORC_ERR_ARG;
                    for (int p = 0; p < bits; ++p)
                        if ((c >> p) & 1) plane[p] |= (1u << j);
                }
                for (int p = 0; p < bits; ++p)
                    for (int b = 0; b < 4; ++b)
                        row[g * 4 * bits + p * 4 + b] = (uint8_t)((plane[p] >> (8 * b)) & 0xff);
            }
        }
    }
    return ORC_OK;
}

int orc_unpack_codes(const uint8_t *packed, int64_t N, int64_t K, int bits, int is_signed,
                     int16_t *codes_out)
{
    int64_t pitch = orc_packed_row_bytes(K, bits);
    if (!packed || !codes_out || pitch < 0 || N < 0) return ORC_ERR_ARG;
    for (int64_t n = 0; n < N; ++n) {
        const uint8_t *row = packed + n * pitch;
        for (int64_t k = 0; k < K; ++k) {
            int c;
            if (bits == 8) {
                c = is_signed ? (int)(int8_t)row[k] : (int)row[k];
            } else if (bits == 4) {
                int nib = (k % 2) ? (row[k / 2] >> 4) : (row[k / 2] & 0xf);
                c = (is_signed && nib >= 8) ? nib - 16 : nib;
            } else {
                int64_t g = k / 32;
                int j = (int)(k % 32);
                c = 0;
                for (int p = 0; p < bits; ++p) {
                    uint32_t plane = 0;
                    for (int b = 0; b < 4; ++b) plane |= (uint32_t)row[g * 4 * bits + p * 4 + b] << (8 * b);
                    c |= (int)((plane >> j) & 1u) << p;
                }
            }
            codes_out[n * K + k] = (int16_t)c;
        }
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------ */
/* Integer GEMM and conv (Sec. 4.3: int8 kernels for W8A8 and W4A8).   */
/* ------------------------------------------------------------------ */

/* acc[m,n] = sum_k qx[m,k] * qw[n,k], checked against int32 overflow. */
int orc_int_gemm(const int8_t *qx, const int16_t *qw, int64_t M, int64_t N, int64_t K,
                 int32_t *acc_out)
{
    if (!qx || !qw || !acc_out || M < 0 || N < 0 || K < 0) return ORC_ERR_ARG;
    int overflow = 0;
#pragma omp parallel for schedule(static) reduction(| : overflow)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            int64_t acc = 0;
            for (int64_t k = 0; k < K; ++k) acc += (int64_t)qx[m * K + k] * (int64_t)qw[n * K + k];
            if (acc > INT32_MAX || acc < INT32_MIN) overflow = 1;
            acc_out[m * N + n] = (int32_t)acc;
        }
    }
    return overflow ? ORC_ERR_OVERFLOW : ORC_OK;
}

/* Direct 3x3 convolution on integer codes, NHWC input [B,H,W,C], weights
 * [N,3,3,C], zero padding 1, stride s in {1,2}:
 *   acc[b,ho,wo,n] = sum_{kh,kw,c} qx[b, ho*s+kh-1, wo*s+kw-1, c] * qw[n,kh,kw,c]
 * with out-of-image taps contributing 0.  Output [B,Ho,Wo,N],
 * Ho = (H + 2 - 3) / s + 1. */
int orc_int_conv3x3(const int8_t *qx, const int16_t *qw, int64_t B, int64_t H, int64_t W, int64_t C,
                    int64_t N, int stride, int32_t *acc_out)
{
    if (!qx || !qw || !acc_out || (stride != 1 && stride != 2)) return ORC_ERR_ARG;
    int64_t Ho = (H + 2 - 3) / stride + 1, Wo = (W + 2 - 3) / stride + 1;
    int overflow = 0;
#pragma omp parallel for collapse(2) schedule(static) reduction(| : overflow)
    for (int64_t b = 0; b < B; ++b) {
        for (int64_t ho = 0; ho < Ho; ++ho) {
            for (int64_t wo = 0; wo < Wo; ++wo) {
                for (int64_t n = 0; n < N; ++n) {
                    int64_t acc = 0;
                    for (int kh = 0; kh < 3; ++kh) {
                        int64_t hi = ho * stride + kh - 1;
                        if (hi < 0 || hi >= H) continue;
                        for (int kw = 0; kw < 3; ++kw) {
                            int64_t wi = wo * stride + kw - 1;
                            if (wi < 0 || wi >= W) continue;
                            const int8_t *xp = qx + ((b * H + hi) * W + wi) * C;
                            const int16_t *wp = qw + ((n * 3 + kh) * 3 + kw) * C;
                            for (int64_t c = 0; c < C; ++c) acc += (int64_t)xp[c] * (int64_t)wp[c];
                        }
                    }
                    if (acc > INT32_MAX || acc < INT32_MIN) overflow = 1;
                    acc_out[((b * Ho + ho) * Wo + wo) * N + n] = (int32_t)acc;
                }
            }
        }
    }
    return overflow ? ORC_ERR_OVERFLOW : ORC_OK;
}

/* The same direct convolution on centred codes of asymmetrically quantized activations (q - z, int16):
 * a padded position holds the real value 0, whose code is z, so it contributes (z - z) * w = 0 and is
 * skipped exactly as above. */
int orc_int_conv3x3_i16(const int16_t *cx, const int16_t *qw, int64_t B, int64_t H, int64_t W, int64_t C,
                        int64_t N, int stride, int32_t *acc_out)
{
    if (!cx || !qw || !acc_out || (stride != 1 && stride != 2)) return ORC_ERR_ARG;
    int64_t Ho = (H + 2 - 3) / stride + 1, Wo = (W + 2 - 3) / stride + 1;
    int overflow = 0;
#pragma omp parallel for collapse(2) schedule(static) reduction(| : overflow)
    for (int64_t b = 0; b < B; ++b) {
        for (int64_t ho = 0; ho < Ho; ++ho) {
            for (int64_t wo = 0; wo < Wo; ++wo) {
                for (int64_t n = 0; n < N; ++n) {
                    int64_t acc = 0;
                    for (int kh = 0; kh < 3; ++kh) {
                        int64_t hi = ho * stride + kh - 1;
                        if (hi < 0 || hi >= H) continue;
                        for (int kw = 0; kw < 3; ++kw) {
                            int64_t wi = wo * stride + kw - 1;
                            if (wi < 0 || wi >= W) continue;
                            const int16_t *xp = cx + ((b * H + hi) * W + wi) * C;
                            const int16_t *wp = qw + ((n * 3 + kh) * 3 + kw) * C;
                            for (int64_t c = 0; c < C; ++c) acc += (int64_t)xp[c] * (int64_t)wp[c];
                        }
                    }
                    if (acc > INT32_MAX || acc < INT32_MIN) overflow = 1;
                    acc_out[((b * Ho + ho) * Wo + wo) * N + n] = (int32_t)acc;
                }
            }
        }
    }
    return overflow ? ORC_ERR_OVERFLOW : ORC_OK;
}

/* Shortcut-splitting (Sec. 4.1, after Q-Diffusion): the reduction range of a layer fed by a concatenation
 * [hidden | skip] is cut at the seam, each part has its own per-tensor activation scale and its own int32
 * accumulator, and the two meet only after dequantization:
 *   y = fp16( (acc_lo * s_lo + acc_hi * s_hi) * s_w[n] + bias[n] ), in double. */
int orc_dequant_epilogue_split(const int32_t *acc_lo, const int32_t *acc_hi, int64_t M, int64_t N, float s_lo,
                               float s_hi, const float *w_scale, const uint16_t *bias, uint16_t *Y)
{
    if (!acc_lo || !acc_hi || !w_scale || !Y) return ORC_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double y = ((double)acc_lo[m * N + n] * (double)s_lo + (double)acc_hi[m * N + n] * (double)s_hi) *
                       (double)w_scale[n];
            if (bias) y += half_to_double(bias[n]);
            Y[m * N + n] = double_to_half(y);
        }
    return ORC_OK;
}

/* Dequantize + bias: y = fp16( acc * s_x * s_w[n] + bias[n] ), in double. */
int orc_dequant_epilogue(const int32_t *acc, int64_t M, int64_t N, float act_scale,
                         const float *w_scale, const uint16_t *bias, uint16_t *Y)
{
    if (!acc || !w_scale || !Y) return ORC_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double y = (double)acc[m * N + n] * (double)act_scale * (double)w_scale[n];
            if (bias) y += half_to_double(bias[n]);
            Y[m * N + n] = double_to_half(y);
        }
    return ORC_OK;
}

/* ------------------------------------------------------------------ */
/* Weight-only layers (FP16 activations, low-bit stored weights).       */
/* ------------------------------------------------------------------ */

/* y[m,n] = fp16( s_n * sum_k x[m,k] * (q[n,k] - z_n) + bias[n] ), in double. */
int orc_weight_only_linear(const uint16_t *X, const int16_t *codes, int64_t M, int64_t N, int64_t K,
                           const float *scale, const int32_t *zero, const uint16_t *bias,
                           uint16_t *Y)
{
    if (!X || !codes || !scale || !Y) return ORC_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            int z = zero ? zero[n] : 0;
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k)
                acc += half_to_double(X[m * K + k]) * (double)(codes[n * K + k] - z);
            double y = (double)scale[n] * acc;
            if (bias) y += half_to_double(bias[n]);
            Y[m * N + n] = double_to_half(y);
        }
    }
    return ORC_OK;
}

/* Weight-only 3x3 conv, same geometry as orc_int_conv3x3, in double. */
int orc_weight_only_conv3x3(const uint16_t *X, const int16_t *codes, int64_t B, int64_t H, int64_t W,
                            int64_t C, int64_t N, int stride, const float *scale,
                            const int32_t *zero, const uint16_t *bias, uint16_t *Y)
{
    if (!X || !codes || !scale || !Y || (stride != 1 && stride != 2)) return ORC_ERR_ARG;
    int64_t Ho = (H + 2 - 3) / stride + 1, Wo = (W + 2 - 3) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t b = 0; b < B; ++b) {
        for (int64_t ho = 0; ho < Ho; ++ho) {
            for (int64_t wo = 0; wo < Wo; ++wo) {
                for (int64_t n = 0; n < N; ++n) {
                    int z = zero ? zero[n] : 0;
                    double acc = 0.0;
                    for (int kh = 0; kh < 3; ++kh) {
                        int64_t hi = ho * stride + kh - 1;
                        if (hi < 0 || hi >= H) continue;
                        for (int kw = 0; kw < 3; ++kw) {
                            int64_t wi = wo * stride + kw - 1;
                            if (wi < 0 || wi >= W) continue;
                            const uint16_t *xp = X + ((b * H + hi) * W + wi) * C;
                            const int16_t *wp = codes + ((n * 3 + kh) * 3 + kw) * C;
                            for (int64_t c = 0; c < C; ++c)
                                acc += half_to_double(xp[c]) * (double)(wp[c] - z);
                        }
                    }
                    double y = (double)scale[n] * acc;
                    if (bias) y += half_to_double(bias[n]);
                    Y[((b * Ho + ho) * Wo + wo) * N + n] = double_to_half(y);
                }
            }
        }
    }
    return ORC_OK;
}

/* Plain fp16-in, double-accumulate matmul y = fp16(X W^T): used to build the
 * stored BOS row from the unquantized weight (Sec. 3.1: the floating-point
 * output of to_k / to_v for the BOS token is computed ahead of time). */
int orc_fp_linear(const uint16_t *X, const uint16_t *Wt, int64_t M, int64_t N, int64_t K, uint16_t *Y)
{
    if (!X || !Wt || !Y) return ORC_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k)
                acc += half_to_double(X[m * K + k]) * half_to_double(Wt[n * K + k]);
            Y[m * N + n] = double_to_half(acc);
        }
    return ORC_OK;
}
