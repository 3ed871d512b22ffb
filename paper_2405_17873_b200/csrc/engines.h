// Internal interface between the C ABI (api.cu) and the two engines.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace mixdq {

// How the rows of the A operand are found in memory.
enum : int {
    A_LINEAR = 0,  // row m of a [M, K] matrix with row stride ldx
    A_BOS = 1,     // row m = (prompt, token - 1): token 0 of every 77-token prompt is skipped
    A_CONV3 = 2,   // row m = (b, ho, wo): im2col gather of a 3x3 window, zero padding 1
};

namespace i8 {

struct Params {
    const __half* X = nullptr;
    long long ldx = 0;
    int M = 0, N = 0, K = 0, k_blocks = 0;
    int H = 0, W = 0, Cin = 0, Ho = 0, Wo = 0, stride = 1;  // conv geometry
    int batch = 0;                                          // prompts (BOS mode)
    const float* act_scale = nullptr;
    // asymmetric activations (two-kernel path; not the BOS-aware projection): zero-point and per-channel sums of
    // the weight codes; both nullptr for symmetric activations
    const int32_t* act_zero = nullptr;
    const int32_t* w_code_sums = nullptr;
    const float* w_scale = nullptr;
    const __half* bias = nullptr;
    const __half* bos_out = nullptr;
    __half* Y = nullptr;
    long long ldy = 0;
    int32_t* acc_out = nullptr;
    int32_t* status = nullptr;
    int32_t* ws_tickets = nullptr;  // split-K: one arrival counter per output tile
    int32_t* ws_acc = nullptr;      // split-K: int32 partial sums, padded to whole tiles
    // two-kernel path, second branch of a shortcut-split layer: the first branch's int32 sums [M, N] and its
    // activation scale; the epilogue adds addend * (*addend_scale) * w_scale[n]
    const int32_t* addend = nullptr;
    const float* addend_scale = nullptr;
    // self-test of the bounded waits (mixdq_selftest_abandoned_wait): > 0 = the weight tile of that k-block
    // (1-based) is announced to its barrier but never requested, so the waits on it run out
    int test_drop_b_kblock = 0;
};

// Scratch of the fused kernel's split reduction (tickets + int32 partial sums).
size_t split_scratch_bytes(int64_t rows, int64_t N);
// Scratch of the two-kernel path: the int8 copy of the activations.
size_t tma_scratch_bytes(int64_t in_rows, int64_t row_len);
// Whole workspace of a linear layer (conv: pass the input pixel count and Cin).
size_t workspace_bytes(int64_t out_rows, int64_t N, int64_t in_rows, int64_t row_len);
int run(Params p, int amode, const void* packed, int w_bits, void* workspace, size_t ws_bytes,
        cudaStream_t stream);
// Two-kernel path (quantize once, then a TMA-fed GEMM); see i8_tma.cu.
bool tma_path_ok(const Params& p, int amode, int w_bits);
int run_tma(const Params& p, int amode, const void* packed, int w_bits, void* scratch, cudaStream_t stream);
// Tile width of the pair form (two-CTA tiles of 256 x width) when the planner prefers it for an int8 GEMM of
// M x N over k_blocks k-blocks of 128, else 0 (the single-CTA kernels run).  *splits (optional): how many CTA
// pairs share one tile's reduction (1: persistent pairs; without the pointer only that form is considered).
int plan_pair_tile(int M, int N, int k_blocks, bool w4, int num_sms, int* splits = nullptr);
// Tile width of the fused-quantization kernel (one launch per layer, 128 x width tiles) when the planner prefers
// it for a linear layer with symmetric activations, else 0 (quantization pass + GEMM).
int plan_fq_tile(int M, int N, int k_blocks, bool w4, int num_sms);
// The one-kernel form itself on 128 x bn tiles (bn a multiple of 32, 32 .. 256): a linear layer with symmetric
// activations, K % 16 == 0, ldx % 8 == 0, X 16-byte aligned; p.Y and / or p.acc_out.
int run_fq(const Params& p, const void* packed, int w_bits, int bn, cudaStream_t stream);
// Tile width (128, 96 or 64) of the one-tile kernel on 128-wide slots.
int plan_narrow_tile(int M, int N, int k_blocks, int num_sms);
// The two steps as calls of their own, for activations that are stored as int8 between layers: the codes of
// X [rows, K] into a dense int8 matrix, and the GEMM / implicit-GEMM convolution on such codes (p.X unused).
int run_quant(const __half* X, long long ldx, long long rows, int K, const float* act_scale, int8_t* out,
              cudaStream_t stream);
int run_tma_prequantized(const Params& p, int amode, const void* packed, int w_bits, const int8_t* aq,
                         cudaStream_t stream);
// Shortcut-splitting (one activation scale per branch of a concatenated input): row elements [0, split_at)
// and [split_at, row_len) are quantized, multiplied and summed separately and meet in a two-scale epilogue.
// Linear layers and 3x3 convolutions whose halves both suit the two-kernel path.
size_t split_layer_scratch_bytes(int64_t in_rows, int64_t row_len, int64_t split_at, int64_t out_rows, int64_t N);
bool split_path_ok(const Params& p, int amode, int split_at, int w_bits);
int run_tma_split(const Params& p, int amode, int split_at, const void* packed_lo, const void* packed_hi, int w_bits,
                  const float* scale_lo, const float* scale_hi, int32_t* acc_lo_out, int32_t* acc_hi_out,
                  void* scratch, cudaStream_t stream);

}  // namespace i8

namespace wo {

struct Params {
    const __half* X = nullptr;
    long long ldx = 0;
    int M = 0, N = 0, K = 0;
    int H = 0, W = 0, Cin = 0, Ho = 0, Wo = 0, stride = 1;
    int batch = 0;  // images (conv)
    const float* w_scale = nullptr;
    const int32_t* w_zero = nullptr;  // nullptr: signed codes, zero-point 0
    const __half* bias = nullptr;
    __half* Y = nullptr;
    long long ldy = 0;
    int32_t* status = nullptr;
    // optional scratch for the layer's weights expanded to fp16 (many-token path); no initial content needed
    void* workspace = nullptr;
    size_t ws_bytes = 0;
};

int run(Params p, int amode, const void* packed, int w_bits, cudaStream_t stream);
// Many-token path with a workspace: the packed weights are expanded ONCE per call to fp16 (q - zero), then both
// operands reach a two-CTA tcgen05 kind::f16 GEMM by TMA; see wo_pair.cu.
size_t expanded_weight_bytes(int64_t N, int64_t K);
bool pair_path_ok(const Params& p, int amode, int w_bits);
int run_pair(const Params& p, int amode, const void* packed, int w_bits, cudaStream_t stream);
// Many-token path on tcgen05 (fp16 MMA, weights expanded into shared memory); see wo_tc.cu.
bool tc_path_ok(const Params& p, int amode, int w_bits);
int run_tc(const Params& p, int amode, const void* packed, int w_bits, int batch, cudaStream_t stream);

}  // namespace wo

}  // namespace mixdq
