// Pieces shared by the int8 GEMM kernels: launch parameters, the accumulator conversion and the
// 32-column epilogue passes (tensor memory -> registers -> fp16 -> staging tile -> global memory).
#pragma once

#include "common.cuh"
#include "engines.h"

namespace mixdq {
namespace i8 {

constexpr int BM = 128;  // rows of one CTA's share of an output tile = lanes of tensor memory
constexpr int BK = 128;  // reduction elements per k-block = one 128-byte swizzled row of int8

struct TmaParams {
    int M, N, k_blocks;
    int conv;     // 0: A is a [M, K] int8 matrix; 1: A is an int8 NHWC image gathered per filter tap
    int pad;      // conv: 1 when the int8 image carries its one-pixel border (asymmetric activations)
    int cblocks;  // conv: k-blocks per filter tap = ceil(Cin / 128)
    int Cin, HoWo, Wo;
    int stride;   // conv: input pixels per output pixel along H and W (1 or 2)
    int bos;      // output row m maps to row (m / 76) * 77 + m % 76 + 1 of Y
    int batch;
    const float* act_scale;
    const int32_t* act_zero;     // asymmetric activations: zero-point (the int8 operand holds q - 128) ...
    const int32_t* w_code_sums;  // ... and sum_k qw[n, k], so that sum_k (q - z) qw = acc + (128 - z) * sums[n]
    const float* w_scale;
    const __half* bias;
    const __half* bos_out;
    __half* Y;
    long long ldy;
    int32_t* acc_out;
    int32_t* status;
    // second branch of a shortcut-split layer: the first branch's int32 sums [M, N] and its activation scale;
    // the epilogue adds addend * (*addend_scale) * w_scale[n] to every output (ADD instances of the kernels)
    const int32_t* addend;
    const float* addend_scale;
    int tile_n;              // one-tile kernel with 128-wide slots: width of the tiles actually computed (0: 128)
    int test_drop_b_kblock;  // self-test: never request the weight tile of this k-block (1-based; 0: none)
    int small_acc;  // every |accumulator| (W4: after the >> 4) stays below 2^22
    int tma_store;  // Y is written through its tensor map (row-contiguous output, 16-byte aligned rows)
};

// int32 accumulator -> float.  W4 accumulators carry the factor 16 of the nibble placement, removed
// here by an exact shift.  SMALL: |v| < 2^22, so adding v to the bit pattern of 1.5 * 2^23 and
// subtracting that constant is exact -- two full-rate instructions instead of a quarter-rate convert.
template <bool W4, bool SMALL, bool F32 = false>
__device__ __forceinline__ float acc_to_float(uint32_t r)
{
    if (F32) return __uint_as_float(r);  // fp16 MMAs accumulate in fp32: the register already holds the sum
    const int32_t v = W4 ? (static_cast<int32_t>(r) >> 4) : static_cast<int32_t>(r);
    if (SMALL) return __int_as_float(0x4B400000 + v) - 12582912.f;
    return static_cast<float>(v);
}

// One warp's share of an output tile: 32 accumulator rows (one per lane, tensor-memory lanes of `acc`) x
// `ncols` columns, in passes of 32 columns: dequantize in registers (comb / bias: per-column factors of the
// tile in shared memory; acc2_off != 0: a second accumulator that many columns further on holds the other
// half of the sum), pass through the warp's staging tile, store.  The staging tile is 32 rows x 32 fp16, as
// dense 64-byte rows with the 64-byte swizzle when a TMA store (box 32 x 32) takes the tile, else rows 80 bytes apart.
constexpr int EPI32_ROW = 80;
constexpr int EPI32_TILE = 32 * EPI32_ROW;  // 2560: a multiple of 512, the period of the 64-byte swizzle

// TWO: the second accumulator holds the sums of the second branch of a shortcut-split layer (Sec. 4.1), with
// per-column factors comb2 of its own: y = acc2 * comb2[c] + (acc * comb[c] + bias[c]).
template <bool W4, bool SMALL, bool TMA, bool F32 = false, bool TWO = false>
__device__ __forceinline__ void store_rows32_from_tmem(uint32_t acc, uint32_t acc2_off, int ncols, const float* comb,
                                                       const float* bias, uint8_t* stage, const TmaParams& p,
                                                       const CUtensorMap* tmap_y, int m_first, int n0, int lane,
                                                       const float* comb2 = nullptr)
{
    const bool vec = ((p.ldy & 7) == 0) && ((p.N & 7) == 0);
    if (TMA && m_first >= p.M) return;  // uniform across the warp
    for (int c0 = 0; c0 < ncols; c0 += 32) {
        if (n0 + c0 >= p.N) break;  // uniform across the warp
        uint32_t r[32];
        uint32_t r2[TWO ? 32 : 1];
        tmem_ld_32x32(acc + c0, r);
        if (TWO) {
            tmem_ld_32x32(acc + acc2_off + c0, reinterpret_cast<uint32_t(&)[32]>(r2));
            tmem_ld_wait();
        } else if (acc2_off) {
            uint32_t rs[32];
            tmem_ld_32x32(acc + acc2_off + c0, rs);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) r[j] += rs[j];
        } else {
            tmem_ld_wait();
        }
        uint4 out[4];  // this lane's row of the pass as fp16
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
            const int c = c0 + j;
            const float4 ca = *reinterpret_cast<const float4*>(comb + c);
            const float4 cb = *reinterpret_cast<const float4*>(comb + c + 4);
            float4 ba = *reinterpret_cast<const float4*>(bias + c);
            float4 bb = *reinterpret_cast<const float4*>(bias + c + 4);
            if (TWO) {
                // the first branch's term joins the bias; the second branch's sums take the place of `r` below
                const float4 da = *reinterpret_cast<const float4*>(comb2 + c);
                const float4 db = *reinterpret_cast<const float4*>(comb2 + c + 4);
                ba.x = fmaf(acc_to_float<W4, SMALL, F32>(r[j]), ca.x, ba.x);
                ba.y = fmaf(acc_to_float<W4, SMALL, F32>(r[j + 1]), ca.y, ba.y);
                ba.z = fmaf(acc_to_float<W4, SMALL, F32>(r[j + 2]), ca.z, ba.z);
                ba.w = fmaf(acc_to_float<W4, SMALL, F32>(r[j + 3]), ca.w, ba.w);
                bb.x = fmaf(acc_to_float<W4, SMALL, F32>(r[j + 4]), cb.x, bb.x);
                bb.y = fmaf(acc_to_float<W4, SMALL, F32>(r[j + 5]), cb.y, bb.y);
                bb.z = fmaf(acc_to_float<W4, SMALL, F32>(r[j + 6]), cb.z, bb.z);
                bb.w = fmaf(acc_to_float<W4, SMALL, F32>(r[j + 7]), cb.w, bb.w);
                __half2 hv[4];
                hv[0] = __floats2half2_rn(fmaf(acc_to_float<W4, SMALL, F32>(r2[TWO ? j : 0]), da.x, ba.x),
                                          fmaf(acc_to_float<W4, SMALL, F32>(r2[TWO ? j + 1 : 0]), da.y, ba.y));
                hv[1] = __floats2half2_rn(fmaf(acc_to_float<W4, SMALL, F32>(r2[TWO ? j + 2 : 0]), da.z, ba.z),
                                          fmaf(acc_to_float<W4, SMALL, F32>(r2[TWO ? j + 3 : 0]), da.w, ba.w));
                hv[2] = __floats2half2_rn(fmaf(acc_to_float<W4, SMALL, F32>(r2[TWO ? j + 4 : 0]), db.x, bb.x),
                                          fmaf(acc_to_float<W4, SMALL, F32>(r2[TWO ? j + 5 : 0]), db.y, bb.y));
                hv[3] = __floats2half2_rn(fmaf(acc_to_float<W4, SMALL, F32>(r2[TWO ? j + 6 : 0]), db.z, bb.z),
                                          fmaf(acc_to_float<W4, SMALL, F32>(r2[TWO ? j + 7 : 0]), db.w, bb.w));
                out[j >> 3] = *reinterpret_cast<const uint4*>(hv);
                continue;
            }
            __half2 hv[4];
            hv[0] = __floats2half2_rn(fmaf(acc_to_float<W4, SMALL, F32>(r[j]), ca.x, ba.x),
                                      fmaf(acc_to_float<W4, SMALL, F32>(r[j + 1]), ca.y, ba.y));
            hv[1] = __floats2half2_rn(fmaf(acc_to_float<W4, SMALL, F32>(r[j + 2]), ca.z, ba.z),
                                      fmaf(acc_to_float<W4, SMALL, F32>(r[j + 3]), ca.w, ba.w));
            hv[2] = __floats2half2_rn(fmaf(acc_to_float<W4, SMALL, F32>(r[j + 4]), cb.x, bb.x),
                                      fmaf(acc_to_float<W4, SMALL, F32>(r[j + 5]), cb.y, bb.y));
            hv[3] = __floats2half2_rn(fmaf(acc_to_float<W4, SMALL, F32>(r[j + 6]), cb.z, bb.z),
                                      fmaf(acc_to_float<W4, SMALL, F32>(r[j + 7]), cb.w, bb.w));
            out[j >> 3] = *reinterpret_cast<const uint4*>(hv);
        }
        if (TMA) {
            // the previous bulk store must have read the staging tile; the conversion above hid that wait
            if (lane == 0) tma_store_wait_read();
            __syncwarp();
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint8_t* dst = TMA ? stage + lane * 64 + ((q ^ ((lane >> 1) & 3)) << 4) : stage + lane * EPI32_ROW + q * 16;
            *reinterpret_cast<uint4*>(dst) = out[q];
        }
        if (TMA) {
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                tma_store_2d(tmap_y, smem_u32(stage), n0 + c0, m_first);
                tma_store_commit();
            }
            continue;
        }
        __syncwarp();
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int rl = it * 8 + (lane >> 2), seg = lane & 3;
            const int mm = m_first + rl;
            const int n = n0 + c0 + seg * 8;
            if (mm >= p.M || n >= p.N) continue;
            long long orow = mm;
            if (p.bos) {
                const int prompt = mm / (MIXDQ_TOKENS_PER_PROMPT - 1);
                orow = static_cast<long long>(prompt) * MIXDQ_TOKENS_PER_PROMPT +
                       (mm - prompt * (MIXDQ_TOKENS_PER_PROMPT - 1) + 1);
            }
            const uint4 v = *reinterpret_cast<const uint4*>(stage + rl * EPI32_ROW + seg * 16);
            __half* dst = p.Y + orow * p.ldy + n;
            if (vec && n + 8 <= p.N) {
                *reinterpret_cast<uint4*>(dst) = v;
            } else {
                const __half* hs = reinterpret_cast<const __half*>(&v);
                for (int q = 0; q < 8; ++q)
                    if (n + q < p.N) dst[q] = hs[q];
            }
        }
        __syncwarp();
    }
}

// fp32 accumulators (weight-only layers on fp16 MMAs)
__device__ __forceinline__ void store_rows32_f32(uint32_t acc, int ncols, const float* comb, const float* bias,
                                                 uint8_t* stage, const TmaParams& p, const CUtensorMap* tmap_y,
                                                 int m_first, int n0, int lane);

// The two-scale form (see store_rows32_from_tmem, TWO).
template <bool W4>
__device__ __forceinline__ void store_rows32_two(uint32_t acc, uint32_t acc2_off, int ncols, const float* comb,
                                                 const float* comb2, const float* bias, uint8_t* stage, const TmaParams& p,
                                                 const CUtensorMap* tmap_y, int m_first, int n0, int lane)
{
    if (p.tma_store)
        store_rows32_from_tmem<W4, false, true, false, true>(acc, acc2_off, ncols, comb, bias, stage, p, tmap_y, m_first, n0,
                                                             lane, comb2);
    else
        store_rows32_from_tmem<W4, false, false, false, true>(acc, acc2_off, ncols, comb, bias, stage, p, tmap_y, m_first, n0,
                                                              lane, comb2);
}

template <bool W4>
__device__ __forceinline__ void store_rows32_dispatch(uint32_t acc, uint32_t acc2_off, int ncols, const float* comb,
                                                      const float* bias, uint8_t* stage, const TmaParams& p,
                                                      const CUtensorMap* tmap_y, int m_first, int n0, int lane)
{
    if (p.tma_store) {
        if (p.small_acc)
            store_rows32_from_tmem<W4, true, true>(acc, acc2_off, ncols, comb, bias, stage, p, tmap_y, m_first, n0, lane);
        else
            store_rows32_from_tmem<W4, false, true>(acc, acc2_off, ncols, comb, bias, stage, p, tmap_y, m_first, n0, lane);
    } else {
        if (p.small_acc)
            store_rows32_from_tmem<W4, true, false>(acc, acc2_off, ncols, comb, bias, stage, p, tmap_y, m_first, n0, lane);
        else
            store_rows32_from_tmem<W4, false, false>(acc, acc2_off, ncols, comb, bias, stage, p, tmap_y, m_first, n0, lane);
    }
}

__device__ __forceinline__ void store_rows32_f32(uint32_t acc, int ncols, const float* comb, const float* bias,
                                                 uint8_t* stage, const TmaParams& p, const CUtensorMap* tmap_y,
                                                 int m_first, int n0, int lane)
{
    if (p.tma_store)
        store_rows32_from_tmem<false, false, true, true>(acc, 0, ncols, comb, bias, stage, p, tmap_y, m_first, n0, lane);
    else
        store_rows32_from_tmem<false, false, false, true>(acc, 0, ncols, comb, bias, stage, p, tmap_y, m_first, n0, lane);
}

// Pair form (i8_pair.cu): persistent kernel of two-CTA clusters on 256 x bn tiles.  ta: activation map with a
// box of 128 rows (or pixels), tw: weight map with a box of bn / 2 rows, ty: output map with a 32 x 32 box.
// splits > 1: one tile per cluster of `splits` CTA pairs, each pair taking a share of the reduction (<= 4).
int launch_pair(const CUtensorMap& ta, const CUtensorMap& tw, const CUtensorMap& ty, const TmaParams& tp, bool w4, int bn,
                int splits, int num_sms, cudaStream_t stream);
// Clusters of `cluster_ctas` CTAs of that kernel the current device can hold at once (0 on error).
int pair_cluster_capacity(bool w4, int cluster_ctas);
// Two-branch form of the same kernel for a shortcut-split layer (Sec. 4.1: the input is a concatenation whose two
// parts keep an activation scale each): ONE launch, one pair per tile; the first `kb_first` k-blocks of a tile are the
// first branch (ta, tw, tp's convolution geometry and tp.act_scale) and accumulate in one accumulator, the others the
// second branch (the maps, geometry and scale below) in the other; the epilogue stores
// y = (s_first * acc_first + s_second * acc_second) * w_scale[n] + bias[n].  tp.acc_out / acc_out: the two branches'
// int32 sums (parity hook).  tp.k_blocks = k-blocks of both branches.
struct PairBranch {
    const CUtensorMap* ta;
    const CUtensorMap* tw;
    int kb_first;            // k-blocks of the FIRST branch
    int cblocks, Cin;        // convolution: k-blocks per filter tap and channels of the second branch
    const float* act_scale;  // activation scale of the second branch (device)
    int32_t* acc_out;        // its sums [M, N], or nullptr
};
int launch_pair_two(const CUtensorMap& ta, const CUtensorMap& tw, const CUtensorMap& ty, const TmaParams& tp, bool w4, int bn,
                    const PairBranch& second, int num_sms, cudaStream_t stream);

// The same kernel on fp16 operands (kind::f16, fp32 accumulators) for the weight-only layers: ta an fp16 map with a
// box of 128 rows x 64 elements, tw the map of the layer's weights expanded to fp16 (q - zero) with a box of
// bn / 2 rows x 64 elements; tp.k_blocks counts blocks of 64 elements and tp.act_scale is unused.
int launch_pair_f16(const CUtensorMap& ta, const CUtensorMap& tw, const CUtensorMap& ty, const TmaParams& tp, int bn,
                    int splits, int num_sms, cudaStream_t stream);

// The same kernel on fp16 activations and PACKED weights (2, 3 or 4 bits, device layout), expanded to fp16
// (code - zero: exact integers) in shared memory by each CTA for its half of the tile: no expanded copy of the
// weights exists in global memory and no expansion kernel runs.  ta as for launch_pair_f16; tw: byte map of the
// packed matrix with a box of bn / 2 rows x 16 * w_bits bytes (128 codes = two k-blocks); tp.k_blocks counts
// blocks of 64 elements; w_zero: per-channel zero-points (device), nullptr for signed codes.  The reduction is
// never split.
int launch_pair_wo(const CUtensorMap& ta, const CUtensorMap& tw, const CUtensorMap& ty, const TmaParams& tp, int bn,
                   int w_bits, const int32_t* w_zero, int num_sms, cudaStream_t stream);

// Fused-quantization form (i8_fq.cu): one kernel per linear layer, fp16 activations in.  tx: fp16 map of X with a
// box of 128 rows x 64 elements (128-byte swizzle), tw: weight map with a box of bn rows, ty: output map with a
// 32 x 32 box; tile 128 x bn (bn a multiple of 32, <= 256).
int launch_fq(const CUtensorMap& tx, const CUtensorMap& tw, const CUtensorMap& ty, const TmaParams& tp, bool w4, int bn,
              cudaStream_t stream);

}  // namespace i8
}  // namespace mixdq
