// C ABI: argument validation and dispatch to the int8 and weight-only engines.
#include "common.cuh"
#include "engines.h"

using namespace mixdq;

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

int check_widths(int w_bits, int act_bits, const int32_t* w_zero)
{
    if (act_bits == 8) {
        if (w_bits != 4 && w_bits != 8) return MIXDQ_ERR_UNSUPPORTED;
        if (w_zero) return MIXDQ_ERR_UNSUPPORTED;  // the int8 path takes symmetric weights
        return MIXDQ_OK;
    }
    if (act_bits == 16) {
        if (w_bits != 2 && w_bits != 3 && w_bits != 4 && w_bits != 8) return MIXDQ_ERR_UNSUPPORTED;
        if (w_bits <= 3 && !w_zero) return MIXDQ_ERR_UNSUPPORTED;
        return MIXDQ_OK;
    }
    return MIXDQ_ERR_UNSUPPORTED;
}

bool fits_int(int64_t v) { return v > 0 && v <= 0x7fffffff; }

int linear_impl(const void* X, int64_t M, int64_t K, int64_t ldx, const void* packed_W, int64_t N,
                int w_bits, const float* w_scale, const int32_t* w_zero, int act_bits,
                const float* act_scale, const void* bias, void* Y, int32_t* acc_out, void* workspace,
                size_t ws_bytes, int32_t* status, void* stream, const int32_t* act_zero = nullptr,
                const int32_t* w_code_sums = nullptr)
{
    if (!X || !packed_W || (!Y && !acc_out)) return MIXDQ_ERR_INVALID_ARG;
    if (!fits_int(M) || !fits_int(K) || !fits_int(N) || ldx < K) return MIXDQ_ERR_INVALID_ARG;
    if (Y && !w_scale) return MIXDQ_ERR_INVALID_ARG;
    int rc = check_widths(w_bits, act_bits, w_zero);
    if (rc != MIXDQ_OK) return rc;
    if (!aligned16(packed_W)) return MIXDQ_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (act_bits == 8) {
        if (!act_scale) return MIXDQ_ERR_INVALID_ARG;
        i8::Params p;
        p.X = static_cast<const __half*>(X);
        p.ldx = ldx;
        p.M = static_cast<int>(M);
        p.N = static_cast<int>(N);
        p.K = static_cast<int>(K);
        p.act_scale = act_scale;
        p.act_zero = act_zero;
        p.w_code_sums = w_code_sums;
        p.w_scale = w_scale;
        p.bias = static_cast<const __half*>(bias);
        p.Y = static_cast<__half*>(Y);
        p.ldy = N;
        p.acc_out = acc_out;
        p.status = status;
        return i8::run(p, A_LINEAR, packed_W, w_bits, workspace, ws_bytes, st);
    }
    if (acc_out) return MIXDQ_ERR_UNSUPPORTED;
    wo::Params p;
    p.X = static_cast<const __half*>(X);
    p.ldx = ldx;
    p.M = static_cast<int>(M);
    p.N = static_cast<int>(N);
    p.K = static_cast<int>(K);
    p.w_scale = w_scale;
    p.w_zero = w_zero;
    p.bias = static_cast<const __half*>(bias);
    p.Y = static_cast<__half*>(Y);
    p.ldy = N;
    p.status = status;
    p.workspace = workspace;
    p.ws_bytes = ws_bytes;
    return wo::run(p, A_LINEAR, packed_W, w_bits, st);
}

int conv3_impl(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin, const void* packed_W,
               int64_t Cout, int stride, int w_bits, const float* w_scale, const int32_t* w_zero,
               int act_bits, const float* act_scale, const void* bias, void* Y, int32_t* acc_out,
               void* workspace, size_t ws_bytes, int32_t* status, void* stream,
               const int32_t* act_zero = nullptr, const int32_t* w_code_sums = nullptr)
{
    if (!X || !packed_W || (!Y && !acc_out)) return MIXDQ_ERR_INVALID_ARG;
    if (!fits_int(B) || !fits_int(H) || !fits_int(W) || !fits_int(Cin) || !fits_int(Cout))
        return MIXDQ_ERR_INVALID_ARG;
    if (stride != 1 && stride != 2) return MIXDQ_ERR_INVALID_ARG;
    if (Y && !w_scale) return MIXDQ_ERR_INVALID_ARG;
    int rc = check_widths(w_bits, act_bits, w_zero);
    if (rc != MIXDQ_OK) return rc;
    if (!aligned16(packed_W)) return MIXDQ_ERR_ALIGNMENT;
    const int64_t Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    if (!fits_int(B * Ho * Wo) || !fits_int(9 * Cin) || !fits_int(B * H * W * Cin)) return MIXDQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (act_bits == 8) {
        if (!act_scale) return MIXDQ_ERR_INVALID_ARG;
        i8::Params p;
        p.X = static_cast<const __half*>(X);
        p.ldx = 8;  // unused by the gather; keeps the alignment test of the dispatcher neutral
        p.M = static_cast<int>(B * Ho * Wo);
        p.N = static_cast<int>(Cout);
        p.K = static_cast<int>(9 * Cin);
        p.H = static_cast<int>(H);
        p.W = static_cast<int>(W);
        p.Cin = static_cast<int>(Cin);
        p.Ho = static_cast<int>(Ho);
        p.Wo = static_cast<int>(Wo);
        p.stride = stride;
        p.batch = static_cast<int>(B);
        p.act_scale = act_scale;
        p.act_zero = act_zero;
        p.w_code_sums = w_code_sums;
        p.w_scale = w_scale;
        p.bias = static_cast<const __half*>(bias);
        p.Y = static_cast<__half*>(Y);
        p.ldy = Cout;
        p.acc_out = acc_out;
        p.status = status;
        return i8::run(p, A_CONV3, packed_W, w_bits, workspace, ws_bytes, st);
    }
    if (acc_out) return MIXDQ_ERR_UNSUPPORTED;
    wo::Params p;
    p.X = static_cast<const __half*>(X);
    p.ldx = 8;
    p.M = static_cast<int>(B * Ho * Wo);
    p.N = static_cast<int>(Cout);
    p.K = static_cast<int>(9 * Cin);
    p.H = static_cast<int>(H);
    p.W = static_cast<int>(W);
    p.Cin = static_cast<int>(Cin);
    p.Ho = static_cast<int>(Ho);
    p.Wo = static_cast<int>(Wo);
    p.stride = stride;
    p.batch = static_cast<int>(B);
    p.w_scale = w_scale;
    p.w_zero = w_zero;
    p.bias = static_cast<const __half*>(bias);
    p.Y = static_cast<__half*>(Y);
    p.ldy = Cout;
    p.status = status;
    p.workspace = workspace;
    p.ws_bytes = ws_bytes;
    return wo::run(p, A_CONV3, packed_W, w_bits, st);
}

int kv_impl(const void* text_emb, int64_t B, int64_t Kt, const void* packed_W, int64_t N, int w_bits,
            const float* w_scale, const float* act_scale, const void* bos_out, void* Y, int32_t* acc_out,
            void* workspace, size_t ws_bytes, int32_t* status, void* stream)
{
    if (!text_emb || !packed_W || !act_scale || (!Y && !acc_out)) return MIXDQ_ERR_INVALID_ARG;
    if (Y && (!w_scale || !bos_out)) return MIXDQ_ERR_INVALID_ARG;
    if (!fits_int(B) || !fits_int(Kt) || !fits_int(N) || !fits_int(B * MIXDQ_TOKENS_PER_PROMPT))
        return MIXDQ_ERR_INVALID_ARG;
    if (w_bits != 4 && w_bits != 8) return MIXDQ_ERR_UNSUPPORTED;
    if (!aligned16(packed_W)) return MIXDQ_ERR_ALIGNMENT;
    i8::Params p;
    p.X = static_cast<const __half*>(text_emb);
    p.ldx = Kt;
    p.M = static_cast<int>(B * (MIXDQ_TOKENS_PER_PROMPT - 1));
    p.N = static_cast<int>(N);
    p.K = static_cast<int>(Kt);
    p.batch = static_cast<int>(B);
    p.act_scale = act_scale;
    p.w_scale = w_scale;
    p.bos_out = static_cast<const __half*>(bos_out);
    p.Y = static_cast<__half*>(Y);
    p.ldy = N;
    p.acc_out = acc_out;
    p.status = status;
    return i8::run(p, A_BOS, packed_W, w_bits, workspace, ws_bytes, static_cast<cudaStream_t>(stream));
}

}  // namespace

extern "C" int mixdq_version(void) { return 100; }

extern "C" unsigned long long mixdq_kernel_launches(void)
{
    return g_layer_kernel_launches.load(std::memory_order_relaxed);
}

extern "C" int mixdq_int8_tile_plan(int64_t M, int64_t N, int64_t k_blocks, int w_bits, int* tile_rows, int* tile_cols,
                                    int* reduction_splits)
{
    if (!tile_rows || !tile_cols || !reduction_splits || M <= 0 || N <= 0 || k_blocks <= 0 || M > 0x7fffffff || N > 0x7fffffff ||
        k_blocks > 0x7fffffff)
        return MIXDQ_ERR_INVALID_ARG;
    if (w_bits != 4 && w_bits != 8) return MIXDQ_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0) return MIXDQ_ERR_CUDA;
    int splits = 1;
    const int bn = i8::plan_pair_tile(static_cast<int>(M), static_cast<int>(N), static_cast<int>(k_blocks), w_bits == 4, sms,
                                      &splits);
    if (bn > 0) {
        *tile_rows = 256;
        *tile_cols = bn;
        *reduction_splits = splits;
    } else {
        *reduction_splits = 0;  // (decided at launch: a cluster of up to eight CTAs when the tiles are few)
        const bool wide = w_bits == 8 && (N >= 1024 || N % 256 == 0) && ceil_div(M, 128) * ceil_div(N, 256) >= 100;
        *tile_rows = 128;
        *tile_cols = wide ? 256 : i8::plan_narrow_tile(static_cast<int>(M), static_cast<int>(N), static_cast<int>(k_blocks), sms);
    }
    return MIXDQ_OK;
}

extern "C" int mixdq_linear_fused_quant_tile(int64_t M, int64_t N, int64_t K, int w_bits)
{
    if (M <= 0 || N <= 0 || K <= 0 || M > 0x7fffffff || N > 0x7fffffff || K > 0x7fffffff) return MIXDQ_ERR_INVALID_ARG;
    if (w_bits != 4 && w_bits != 8) return MIXDQ_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0) return MIXDQ_ERR_CUDA;
    if (K % 16 != 0) return 0;  // (the TMA-fed kernels need 16-byte rows of codes)
    return i8::plan_fq_tile(static_cast<int>(M), static_cast<int>(N), static_cast<int>(ceil_div(K, 128)), w_bits == 4, sms);
}

extern "C" const char* mixdq_strerror(int code)
{
    switch (code) {
        case MIXDQ_OK: return "success";
        case MIXDQ_ERR_INVALID_ARG: return "invalid argument";
        case MIXDQ_ERR_UNSUPPORTED: return "unsupported bit-width or shape";
        case MIXDQ_ERR_ALIGNMENT: return "misaligned pointer or stride";
        case MIXDQ_ERR_WORKSPACE: return "workspace missing or too small";
        case MIXDQ_ERR_CUDA: return "CUDA call failed";
        case MIXDQ_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown error";
    }
}

extern "C" int mixdq_workspace_bytes(int64_t rows, int64_t N, int64_t K, int w_bits, int act_bits, size_t* out)
{
    if (!out || rows <= 0 || N <= 0 || K <= 0) return MIXDQ_ERR_INVALID_ARG;
    if (act_bits != 8 && act_bits != 16) return MIXDQ_ERR_UNSUPPORTED;
    if (w_bits != 2 && w_bits != 3 && w_bits != 4 && w_bits != 8) return MIXDQ_ERR_UNSUPPORTED;
    // weight-only layers: room for the weights expanded to fp16, used on 256 rows or more
    *out = (act_bits == 8) ? i8::workspace_bytes(rows, N, rows, K) : (rows >= 256 ? wo::expanded_weight_bytes(N, K) : 0);
    return MIXDQ_OK;
}

extern "C" int mixdq_conv3x3_workspace_bytes(int64_t B, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int stride,
                                             int w_bits, int act_bits, size_t* out)
{
    if (!out || B <= 0 || H <= 0 || W <= 0 || Cin <= 0 || Cout <= 0) return MIXDQ_ERR_INVALID_ARG;
    if (stride != 1 && stride != 2) return MIXDQ_ERR_INVALID_ARG;
    if (act_bits != 8 && act_bits != 16) return MIXDQ_ERR_UNSUPPORTED;
    if (w_bits != 2 && w_bits != 3 && w_bits != 4 && w_bits != 8) return MIXDQ_ERR_UNSUPPORTED;
    const int64_t Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    // room for the int8 image with a one-pixel border, which the asymmetric-activation call keeps
    *out = (act_bits == 8) ? i8::workspace_bytes(B * Ho * Wo, Cout, B * (H + 2) * (W + 2), Cin)
                           : (B * Ho * Wo >= 256 ? wo::expanded_weight_bytes(Cout, 9 * Cin) : 0);
    return MIXDQ_OK;
}

extern "C" int mixdq_linear(const void* X, int64_t M, int64_t K, int64_t ldx, const void* packed_W, int64_t N,
                            int w_bits, const float* w_scale, const int32_t* w_zero, int act_bits,
                            const float* act_scale, const void* bias, void* Y, void* workspace,
                            size_t workspace_bytes, int32_t* status, void* stream)
{
    if (!Y) return MIXDQ_ERR_INVALID_ARG;
    return linear_impl(X, M, K, ldx, packed_W, N, w_bits, w_scale, w_zero, act_bits, act_scale, bias, Y,
                       nullptr, workspace, workspace_bytes, status, stream);
}

extern "C" int mixdq_linear_acc_i32(const void* X, int64_t M, int64_t K, int64_t ldx, const void* packed_W,
                                    int64_t N, int w_bits, const float* act_scale, int32_t* acc_out,
                                    void* workspace, size_t workspace_bytes, int32_t* status, void* stream)
{
    if (!acc_out) return MIXDQ_ERR_INVALID_ARG;
    return linear_impl(X, M, K, ldx, packed_W, N, w_bits, nullptr, nullptr, 8, act_scale, nullptr, nullptr,
                       acc_out, workspace, workspace_bytes, status, stream);
}

// |sum_k (q - z) qw| <= K * 255 * 127 must fit the int32 accumulator.
static bool asym_args_ok(int64_t K, const float* act_scale, const int32_t* act_zero, const int32_t* w_code_sums)
{
    return act_scale && act_zero && w_code_sums && K * 255 * 127 <= 0x7fffffffll;
}

extern "C" int mixdq_linear_a8_asym(const void* X, int64_t M, int64_t K, int64_t ldx, const void* packed_W,
                                    int64_t N, int w_bits, const float* w_scale, const int32_t* w_code_sums,
                                    const float* act_scale, const int32_t* act_zero, const void* bias, void* Y,
                                    void* workspace, size_t workspace_bytes, int32_t* status, void* stream)
{
    if (!Y || !asym_args_ok(K, act_scale, act_zero, w_code_sums)) return MIXDQ_ERR_INVALID_ARG;
    return linear_impl(X, M, K, ldx, packed_W, N, w_bits, w_scale, nullptr, 8, act_scale, bias, Y, nullptr,
                       workspace, workspace_bytes, status, stream, act_zero, w_code_sums);
}

extern "C" int mixdq_linear_a8_asym_acc_i32(const void* X, int64_t M, int64_t K, int64_t ldx,
                                            const void* packed_W, int64_t N, int w_bits,
                                            const int32_t* w_code_sums, const float* act_scale,
                                            const int32_t* act_zero, int32_t* acc_out, void* workspace,
                                            size_t workspace_bytes, int32_t* status, void* stream)
{
    if (!acc_out || !asym_args_ok(K, act_scale, act_zero, w_code_sums)) return MIXDQ_ERR_INVALID_ARG;
    return linear_impl(X, M, K, ldx, packed_W, N, w_bits, nullptr, nullptr, 8, act_scale, nullptr, nullptr,
                       acc_out, workspace, workspace_bytes, status, stream, act_zero, w_code_sums);
}

extern "C" int mixdq_conv3x3_a8_asym(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin,
                                     const void* packed_W, int64_t Cout, int stride, int w_bits,
                                     const float* w_scale, const int32_t* w_code_sums, const float* act_scale,
                                     const int32_t* act_zero, const void* bias, void* Y, void* workspace,
                                     size_t workspace_bytes, int32_t* status, void* stream)
{
    if (!Y || !asym_args_ok(9 * Cin, act_scale, act_zero, w_code_sums)) return MIXDQ_ERR_INVALID_ARG;
    return conv3_impl(X, B, H, W, Cin, packed_W, Cout, stride, w_bits, w_scale, nullptr, 8, act_scale, bias, Y,
                      nullptr, workspace, workspace_bytes, status, stream, act_zero, w_code_sums);
}

extern "C" int mixdq_conv3x3_a8_asym_acc_i32(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin,
                                             const void* packed_W, int64_t Cout, int stride, int w_bits,
                                             const int32_t* w_code_sums, const float* act_scale,
                                             const int32_t* act_zero, int32_t* acc_out, void* workspace,
                                             size_t workspace_bytes, int32_t* status, void* stream)
{
    if (!acc_out || !asym_args_ok(9 * Cin, act_scale, act_zero, w_code_sums)) return MIXDQ_ERR_INVALID_ARG;
    return conv3_impl(X, B, H, W, Cin, packed_W, Cout, stride, w_bits, nullptr, nullptr, 8, act_scale, nullptr,
                      nullptr, acc_out, workspace, workspace_bytes, status, stream, act_zero, w_code_sums);
}

// ---------------------------------------------------------------- int8 activations kept between layers

extern "C" int mixdq_quantize_acts(const void* X, int64_t rows, int64_t K, int64_t ldx, const float* act_scale,
                                   void* Xq_out, void* stream)
{
    if (!X || !act_scale || !Xq_out || !fits_int(rows) || !fits_int(K) || ldx < K) return MIXDQ_ERR_INVALID_ARG;
    if (K % 16 != 0 || ldx % 8 != 0) return MIXDQ_ERR_UNSUPPORTED;
    if (!aligned16(X) || !aligned16(Xq_out)) return MIXDQ_ERR_ALIGNMENT;
    return i8::run_quant(static_cast<const __half*>(X), ldx, rows, static_cast<int>(K), act_scale,
                         static_cast<int8_t*>(Xq_out), static_cast<cudaStream_t>(stream));
}

namespace {

int linear_q8_impl(const void* Xq, int64_t M, int64_t K, const void* packed_W, int64_t N, int w_bits,
                   const float* w_scale, const float* act_scale, const void* bias, void* Y, int32_t* acc_out,
                   int32_t* status, void* stream, int test_drop_b_kblock = 0)
{
    if (!Xq || !packed_W || (!Y && !acc_out)) return MIXDQ_ERR_INVALID_ARG;
    if (!fits_int(M) || !fits_int(K) || !fits_int(N)) return MIXDQ_ERR_INVALID_ARG;
    if (Y && (!w_scale || !act_scale)) return MIXDQ_ERR_INVALID_ARG;
    if (w_bits != 4 && w_bits != 8) return MIXDQ_ERR_UNSUPPORTED;
    if (K % 16 != 0) return MIXDQ_ERR_UNSUPPORTED;
    if (!aligned16(packed_W) || !aligned16(Xq)) return MIXDQ_ERR_ALIGNMENT;
    i8::Params p;
    p.ldx = K;
    p.M = static_cast<int>(M);
    p.N = static_cast<int>(N);
    p.K = static_cast<int>(K);
    p.act_scale = act_scale;
    p.w_scale = w_scale;
    p.bias = static_cast<const __half*>(bias);
    p.Y = static_cast<__half*>(Y);
    p.ldy = N;
    p.acc_out = acc_out;
    p.status = status;
    p.test_drop_b_kblock = test_drop_b_kblock;
    return i8::run_tma_prequantized(p, A_LINEAR, packed_W, w_bits, static_cast<const int8_t*>(Xq),
                                    static_cast<cudaStream_t>(stream));
}

}  // namespace

extern "C" int mixdq_linear_q8(const void* Xq, int64_t M, int64_t K, const void* packed_W, int64_t N, int w_bits,
                               const float* w_scale, const float* act_scale, const void* bias, void* Y,
                               int32_t* status, void* stream)
{
    if (!Y) return MIXDQ_ERR_INVALID_ARG;
    return linear_q8_impl(Xq, M, K, packed_W, N, w_bits, w_scale, act_scale, bias, Y, nullptr, status, stream);
}

extern "C" int mixdq_linear_a8_fused_quant(const void* X, int64_t M, int64_t K, int64_t ldx, const void* packed_W,
                                           int64_t N, int w_bits, const float* w_scale, const float* act_scale,
                                           const void* bias, void* Y, int64_t ldy, int tile_cols, int32_t* status,
                                           void* stream)
{
    if (!X || !packed_W || !Y || !w_scale || !act_scale) return MIXDQ_ERR_INVALID_ARG;
    if (!fits_int(M) || !fits_int(K) || !fits_int(N) || ldx < K || ldy < N) return MIXDQ_ERR_INVALID_ARG;
    if (tile_cols < 32 || tile_cols > 256 || tile_cols % 32 != 0) return MIXDQ_ERR_INVALID_ARG;
    if (w_bits != 4 && w_bits != 8) return MIXDQ_ERR_UNSUPPORTED;
    if (K % 16 != 0 || ldx % 8 != 0) return MIXDQ_ERR_UNSUPPORTED;
    if (!aligned16(packed_W) || !aligned16(X)) return MIXDQ_ERR_ALIGNMENT;
    i8::Params p;
    p.X = static_cast<const __half*>(X);
    p.ldx = ldx;
    p.M = static_cast<int>(M);
    p.N = static_cast<int>(N);
    p.K = static_cast<int>(K);
    p.act_scale = act_scale;
    p.w_scale = w_scale;
    p.bias = static_cast<const __half*>(bias);
    p.Y = static_cast<__half*>(Y);
    p.ldy = ldy;
    p.status = status;
    return i8::run_fq(p, packed_W, w_bits, tile_cols, static_cast<cudaStream_t>(stream));
}

extern "C" int mixdq_selftest_abandoned_wait(const void* Xq, int64_t M, int64_t K, const void* packed_W, int64_t N,
                                             int w_bits, const float* w_scale, const float* act_scale, void* Y,
                                             int drop_k_block, int32_t* status, void* stream)
{
    if (!Y || !status) return MIXDQ_ERR_INVALID_ARG;
    if (drop_k_block < 1 || drop_k_block > (K + 127) / 128) return MIXDQ_ERR_INVALID_ARG;
    return linear_q8_impl(Xq, M, K, packed_W, N, w_bits, w_scale, act_scale, nullptr, Y, nullptr, status, stream,
                          drop_k_block);
}

extern "C" int mixdq_linear_q8_acc_i32(const void* Xq, int64_t M, int64_t K, const void* packed_W, int64_t N,
                                       int w_bits, int32_t* acc_out, int32_t* status, void* stream)
{
    if (!acc_out) return MIXDQ_ERR_INVALID_ARG;
    return linear_q8_impl(Xq, M, K, packed_W, N, w_bits, nullptr, nullptr, nullptr, nullptr, acc_out, status, stream);
}

extern "C" int mixdq_conv3x3_q8(const void* Xq, int64_t B, int64_t H, int64_t W, int64_t Cin, const void* packed_W,
                                int64_t Cout, int stride, int w_bits, const float* w_scale, const float* act_scale,
                                const void* bias, void* Y, int32_t* status, void* stream)
{
    if (!Xq || !packed_W || !Y || !w_scale || !act_scale) return MIXDQ_ERR_INVALID_ARG;
    if (!fits_int(B) || !fits_int(H) || !fits_int(W) || !fits_int(Cin) || !fits_int(Cout))
        return MIXDQ_ERR_INVALID_ARG;
    if (stride != 1 && stride != 2) return MIXDQ_ERR_INVALID_ARG;
    if (w_bits != 4 && w_bits != 8) return MIXDQ_ERR_UNSUPPORTED;
    const int64_t Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    if (!fits_int(B * Ho * Wo) || !fits_int(9 * Cin) || !fits_int(B * H * W * Cin)) return MIXDQ_ERR_INVALID_ARG;
    if (!aligned16(packed_W) || !aligned16(Xq)) return MIXDQ_ERR_ALIGNMENT;
    i8::Params p;
    p.ldx = 8;
    p.M = static_cast<int>(B * Ho * Wo);
    p.N = static_cast<int>(Cout);
    p.K = static_cast<int>(9 * Cin);
    p.H = static_cast<int>(H);
    p.W = static_cast<int>(W);
    p.Cin = static_cast<int>(Cin);
    p.Ho = static_cast<int>(Ho);
    p.Wo = static_cast<int>(Wo);
    p.stride = stride;
    p.batch = static_cast<int>(B);
    p.act_scale = act_scale;
    p.w_scale = w_scale;
    p.bias = static_cast<const __half*>(bias);
    p.Y = static_cast<__half*>(Y);
    p.ldy = Cout;
    p.status = status;
    if (!i8::tma_path_ok(p, A_CONV3, w_bits)) return MIXDQ_ERR_UNSUPPORTED;
    return i8::run_tma_prequantized(p, A_CONV3, packed_W, w_bits, static_cast<const int8_t*>(Xq),
                                    static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------- shortcut-splitting (Sec. 4.1)

namespace {

int split_common(i8::Params& p, int amode, int64_t in_rows, int64_t row_len, int64_t split_at, const void* packed_lo,
                 const void* packed_hi, int w_bits, const float* act_scale_lo, const float* act_scale_hi,
                 int32_t* acc_lo_out, int32_t* acc_hi_out, void* workspace, size_t ws_bytes, void* stream)
{
    if (!p.X || !packed_lo || !packed_hi || !act_scale_lo || !act_scale_hi) return MIXDQ_ERR_INVALID_ARG;
    if (p.Y ? !p.w_scale : (!acc_lo_out || !acc_hi_out)) return MIXDQ_ERR_INVALID_ARG;
    if (split_at <= 0 || split_at >= row_len) return MIXDQ_ERR_INVALID_ARG;
    if (w_bits != 4 && w_bits != 8) return MIXDQ_ERR_UNSUPPORTED;
    if (!aligned16(packed_lo) || !aligned16(packed_hi) || !aligned16(workspace)) return MIXDQ_ERR_ALIGNMENT;
    if (!i8::split_path_ok(p, amode, static_cast<int>(split_at), w_bits)) return MIXDQ_ERR_UNSUPPORTED;
    if (!workspace || ws_bytes < i8::split_layer_scratch_bytes(in_rows, row_len, split_at, p.M, p.N))
        return MIXDQ_ERR_WORKSPACE;
    return i8::run_tma_split(p, amode, static_cast<int>(split_at), packed_lo, packed_hi, w_bits, act_scale_lo,
                             act_scale_hi, acc_lo_out, acc_hi_out, workspace, static_cast<cudaStream_t>(stream));
}

int linear_split_impl(const void* X, int64_t M, int64_t K, int64_t ldx, int64_t split_at, const void* packed_lo,
                      const void* packed_hi, int64_t N, int w_bits, const float* w_scale, const float* act_scale_lo,
                      const float* act_scale_hi, const void* bias, void* Y, int32_t* acc_lo_out,
                      int32_t* acc_hi_out, void* workspace, size_t ws_bytes, int32_t* status, void* stream)
{
    if (!fits_int(M) || !fits_int(K) || !fits_int(N) || ldx < K) return MIXDQ_ERR_INVALID_ARG;
    i8::Params p;
    p.X = static_cast<const __half*>(X);
    p.ldx = ldx;
    p.M = static_cast<int>(M);
    p.N = static_cast<int>(N);
    p.K = static_cast<int>(K);
    p.w_scale = w_scale;
    p.bias = static_cast<const __half*>(bias);
    p.Y = static_cast<__half*>(Y);
    p.ldy = N;
    p.status = status;
    return split_common(p, A_LINEAR, M, K, split_at, packed_lo, packed_hi, w_bits, act_scale_lo, act_scale_hi,
                        acc_lo_out, acc_hi_out, workspace, ws_bytes, stream);
}

int conv3_split_impl(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin, int64_t split_at,
                     const void* packed_lo, const void* packed_hi, int64_t Cout, int stride, int w_bits,
                     const float* w_scale, const float* act_scale_lo, const float* act_scale_hi, const void* bias,
                     void* Y, int32_t* acc_lo_out, int32_t* acc_hi_out, void* workspace, size_t ws_bytes,
                     int32_t* status, void* stream)
{
    if (!fits_int(B) || !fits_int(H) || !fits_int(W) || !fits_int(Cin) || !fits_int(Cout))
        return MIXDQ_ERR_INVALID_ARG;
    if (stride != 1 && stride != 2) return MIXDQ_ERR_INVALID_ARG;
    const int64_t Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    if (!fits_int(B * Ho * Wo) || !fits_int(9 * Cin) || !fits_int(B * H * W * Cin)) return MIXDQ_ERR_INVALID_ARG;
    i8::Params p;
    p.X = static_cast<const __half*>(X);
    p.ldx = 8;
    p.M = static_cast<int>(B * Ho * Wo);
    p.N = static_cast<int>(Cout);
    p.K = static_cast<int>(9 * Cin);
    p.H = static_cast<int>(H);
    p.W = static_cast<int>(W);
    p.Cin = static_cast<int>(Cin);
    p.Ho = static_cast<int>(Ho);
    p.Wo = static_cast<int>(Wo);
    p.stride = stride;
    p.batch = static_cast<int>(B);
    p.w_scale = w_scale;
    p.bias = static_cast<const __half*>(bias);
    p.Y = static_cast<__half*>(Y);
    p.ldy = Cout;
    p.status = status;
    return split_common(p, A_CONV3, B * H * W, Cin, split_at, packed_lo, packed_hi, w_bits, act_scale_lo,
                        act_scale_hi, acc_lo_out, acc_hi_out, workspace, ws_bytes, stream);
}

}  // namespace

extern "C" int mixdq_split_workspace_bytes(int64_t in_rows, int64_t row_len, int64_t split_at, int64_t out_rows,
                                           int64_t N, size_t* out)
{
    if (!out || in_rows <= 0 || out_rows <= 0 || N <= 0 || split_at <= 0 || split_at >= row_len)
        return MIXDQ_ERR_INVALID_ARG;
    *out = i8::split_layer_scratch_bytes(in_rows, row_len, split_at, out_rows, N);
    return MIXDQ_OK;
}

extern "C" int mixdq_linear_a8_split(const void* X, int64_t M, int64_t K, int64_t ldx, int64_t split_at,
                                     const void* packed_W_lo, const void* packed_W_hi, int64_t N, int w_bits,
                                     const float* w_scale, const float* act_scale_lo, const float* act_scale_hi,
                                     const void* bias, void* Y, void* workspace, size_t workspace_bytes,
                                     int32_t* status, void* stream)
{
    if (!Y) return MIXDQ_ERR_INVALID_ARG;
    return linear_split_impl(X, M, K, ldx, split_at, packed_W_lo, packed_W_hi, N, w_bits, w_scale, act_scale_lo,
                             act_scale_hi, bias, Y, nullptr, nullptr, workspace, workspace_bytes, status, stream);
}

extern "C" int mixdq_linear_a8_split_acc_i32(const void* X, int64_t M, int64_t K, int64_t ldx, int64_t split_at,
                                             const void* packed_W_lo, const void* packed_W_hi, int64_t N,
                                             int w_bits, const float* act_scale_lo, const float* act_scale_hi,
                                             int32_t* acc_lo_out, int32_t* acc_hi_out, void* workspace,
                                             size_t workspace_bytes, int32_t* status, void* stream)
{
    return linear_split_impl(X, M, K, ldx, split_at, packed_W_lo, packed_W_hi, N, w_bits, nullptr, act_scale_lo,
                             act_scale_hi, nullptr, nullptr, acc_lo_out, acc_hi_out, workspace, workspace_bytes,
                             status, stream);
}

extern "C" int mixdq_conv3x3_a8_split(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin, int64_t split_at,
                                      const void* packed_W_lo, const void* packed_W_hi, int64_t Cout, int stride,
                                      int w_bits, const float* w_scale, const float* act_scale_lo,
                                      const float* act_scale_hi, const void* bias, void* Y, void* workspace,
                                      size_t workspace_bytes, int32_t* status, void* stream)
{
    if (!Y) return MIXDQ_ERR_INVALID_ARG;
    return conv3_split_impl(X, B, H, W, Cin, split_at, packed_W_lo, packed_W_hi, Cout, stride, w_bits, w_scale,
                            act_scale_lo, act_scale_hi, bias, Y, nullptr, nullptr, workspace, workspace_bytes,
                            status, stream);
}

extern "C" int mixdq_conv3x3_a8_split_acc_i32(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin,
                                              int64_t split_at, const void* packed_W_lo, const void* packed_W_hi,
                                              int64_t Cout, int stride, int w_bits, const float* act_scale_lo,
                                              const float* act_scale_hi, int32_t* acc_lo_out, int32_t* acc_hi_out,
                                              void* workspace, size_t workspace_bytes, int32_t* status,
                                              void* stream)
{
    return conv3_split_impl(X, B, H, W, Cin, split_at, packed_W_lo, packed_W_hi, Cout, stride, w_bits, nullptr,
                            act_scale_lo, act_scale_hi, nullptr, nullptr, acc_lo_out, acc_hi_out, workspace,
                            workspace_bytes, status, stream);
}

extern "C" int mixdq_conv3x3(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin, const void* packed_W,
                             int64_t Cout, int stride, int w_bits, const float* w_scale,
                             const int32_t* w_zero, int act_bits, const float* act_scale, const void* bias,
                             void* Y, void* workspace, size_t workspace_bytes, int32_t* status, void* stream)
{
    if (!Y) return MIXDQ_ERR_INVALID_ARG;
    return conv3_impl(X, B, H, W, Cin, packed_W, Cout, stride, w_bits, w_scale, w_zero, act_bits, act_scale,
                      bias, Y, nullptr, workspace, workspace_bytes, status, stream);
}

extern "C" int mixdq_conv3x3_acc_i32(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin,
                                     const void* packed_W, int64_t Cout, int stride, int w_bits,
                                     const float* act_scale, int32_t* acc_out, void* workspace,
                                     size_t workspace_bytes, int32_t* status, void* stream)
{
    if (!acc_out) return MIXDQ_ERR_INVALID_ARG;
    return conv3_impl(X, B, H, W, Cin, packed_W, Cout, stride, w_bits, nullptr, nullptr, 8, act_scale, nullptr,
                      nullptr, acc_out, workspace, workspace_bytes, status, stream);
}

extern "C" int mixdq_conv1x1(const void* X, int64_t B, int64_t H, int64_t W, int64_t Cin, const void* packed_W,
                             int64_t Cout, int w_bits, const float* w_scale, const int32_t* w_zero,
                             int act_bits, const float* act_scale, const void* bias, void* Y, void* workspace,
                             size_t workspace_bytes, int32_t* status, void* stream)
{
    if (B <= 0 || H <= 0 || W <= 0) return MIXDQ_ERR_INVALID_ARG;
    return mixdq_linear(X, B * H * W, Cin, Cin, packed_W, Cout, w_bits, w_scale, w_zero, act_bits, act_scale,
                        bias, Y, workspace, workspace_bytes, status, stream);
}

extern "C" int mixdq_crossattn_kv(const void* text_emb, int64_t B, int64_t Kt, const void* packed_W, int64_t N,
                                  int w_bits, const float* w_scale, const float* act_scale,
                                  const void* bos_out, void* Y, void* workspace, size_t workspace_bytes,
                                  int32_t* status, void* stream)
{
    if (!Y) return MIXDQ_ERR_INVALID_ARG;
    return kv_impl(text_emb, B, Kt, packed_W, N, w_bits, w_scale, act_scale, bos_out, Y, nullptr, workspace,
                   workspace_bytes, status, stream);
}

extern "C" int mixdq_crossattn_kv_acc_i32(const void* text_emb, int64_t B, int64_t Kt, const void* packed_W,
                                          int64_t N, int w_bits, const float* act_scale, int32_t* acc_out,
                                          void* workspace, size_t workspace_bytes, int32_t* status,
                                          void* stream)
{
    if (!acc_out) return MIXDQ_ERR_INVALID_ARG;
    return kv_impl(text_emb, B, Kt, packed_W, N, w_bits, nullptr, act_scale, nullptr, nullptr, acc_out,
                   workspace, workspace_bytes, status, stream);
}
