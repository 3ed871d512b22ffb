// Weight-only (W2 / W3 / W4 / W8, fp16 activations) layers on many tokens, with a workspace.
//
// With hundreds of tokens a layer is bound by the fp16 tensor pipe, not by its weight stream: the packed form
// then only has to save memory, not bandwidth.  The kernel that expands weight tiles inside the GEMM
// (wo_tc.cu) repeats the expansion for every 128-row block of the activations -- 32 times at 4096 tokens -- and
// its expansion warps cannot keep up with the MMAs.  Here the layer's weights are expanded ONCE per call into
// an fp16 matrix (q - zero, exact integers, so the weights still add no rounding of their own; the per-channel
// scale is applied to the fp32 sums) in the caller's workspace, which stays in L2 for all but the largest
// layers, and both operands then reach the two-CTA tcgen05 kernel (i8_pair.cu in its kind::f16 mode) by TMA.
#include <algorithm>
#include <cmath>

#include "codes.cuh"
#include "common.cuh"
#include "engines.h"
#include "i8_tiles.cuh"

namespace mixdq {
namespace wo {

namespace {

constexpr int BM = i8::BM;
constexpr int BKE = 64;  // fp16 elements of a k-block (128-byte rows)

// out[n, k] = half(code[n, k] - zero[n]) for k < K, 0 for K <= k < ldw.  One thread per eight elements.
template <int BITS, bool SIGNED>
__global__ void expand_weights_kernel(const uint8_t* __restrict__ packed, long long pitch, int N, int K, int ldw,
                                      const int32_t* __restrict__ w_zero, __half* __restrict__ out)
{
    pdl_launch_dependents();
    pdl_wait();  // the scratch may still be the weight operand of the previous layer's GEMM
    const int groups = ldw >> 3;
    const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    if (idx >= static_cast<long long>(N) * groups) return;
    const int n = static_cast<int>(idx / groups);
    const int k0 = static_cast<int>(idx - static_cast<long long>(n) * groups) * 8;
    const int z = SIGNED ? 0 : __ldg(w_zero + n);
    int c[8];
    codes8<BITS, SIGNED>(packed + n * pitch, k0, c);  // rows are padded to whole groups in the device layout
    __half2 h[4];
#pragma unroll
    for (int j = 0; j < 8; j += 2)
        h[j >> 1] = __halves2half2(k0 + j < K ? __int2half_rn(c[j] - z) : __half(0.f),
                                   k0 + j + 1 < K ? __int2half_rn(c[j + 1] - z) : __half(0.f));
    *reinterpret_cast<uint4*>(out + static_cast<long long>(n) * ldw + k0) = *reinterpret_cast<const uint4*>(h);
}

template <int BITS, bool SIGNED>
int launch_expand(const void* packed, long long pitch, int N, int K, int ldw, const int32_t* w_zero, __half* out,
                  cudaStream_t stream)
{
    const long long tasks = static_cast<long long>(N) * (ldw / 8);
    return launch_pdl(expand_weights_kernel<BITS, SIGNED>, dim3(static_cast<unsigned>(ceil_div(tasks, 256))), dim3(256), 0,
                      stream, 1, static_cast<const uint8_t*>(packed), pitch, N, K, ldw, w_zero, out);
}

bool conv_box(int Ho, int Wo, int* Wb, int* Hb, int* Bb)
{
    if (Wo >= BM) {
        if (Wo % BM) return false;
        *Wb = BM; *Hb = 1; *Bb = 1;
        return true;
    }
    if (BM % Wo) return false;
    const int rows = BM / Wo;
    if (Ho >= rows) {
        if (Ho % rows) return false;
        *Wb = Wo; *Hb = rows; *Bb = 1;
        return true;
    }
    if (rows % Ho) return false;
    *Wb = Wo; *Hb = Ho; *Bb = rows / Ho;
    return true;
}

// Tile width and reduction split: whole rounds of 256 x bn tiles over the SM pairs, the per-tile cost growing with
// the width; layers with few tiles and a long reduction give one tile to a cluster of two to four CTA pairs.
int pick_tile(int M, int N, int k_blocks, int num_sms, int* splits)
{
    double best = 0;
    int best_bn = 0;
    *splits = 1;
    const int pairs = num_sms / 2;
    for (int bn = 96; bn <= 256; bn += 32) {
        const int64_t tiles = ceil_div(M, 2 * BM) * ceil_div(N, bn);
        const double per_kb = 250.0 + 1.2 * bn;
        const double rounds = std::ceil(static_cast<double>(tiles) / pairs);
        const double t = rounds * (std::max(k_blocks * per_kb, 30.0 * bn) + 800.0) + 16.0 * bn;
        if (best_bn == 0 || t < best) {
            best = t;
            best_bn = bn;
            *splits = 1;
        }
        for (int sp = 2; sp <= 4 && tiles * sp <= pairs && k_blocks / sp >= 16; ++sp) {
            if (tiles > i8::pair_cluster_capacity(false, 2 * sp)) continue;
            const double ts = std::ceil(static_cast<double>(k_blocks) / sp) * per_kb + 16.0 * bn + 14000.0;
            if (ts < best) {
                best = ts;
                best_bn = bn;
                *splits = sp;
            }
        }
    }
    return best_bn;
}

}  // namespace

size_t expanded_weight_bytes(int64_t N, int64_t K) { return static_cast<size_t>(round_up(N * round_up(K, 8) * 2, 256)); }

bool pair_path_ok(const Params& p, int amode, int w_bits)
{
    if (!p.workspace || p.ws_bytes < expanded_weight_bytes(p.N, p.K) || (reinterpret_cast<uintptr_t>(p.workspace) & 15))
        return false;
    if (p.M < 2 * BM || p.N < 32) return false;  // below that the fused expansion is the better form
    if (w_bits <= 3 && !p.w_zero) return false;  // bit-plane codes are unsigned
    if (amode == A_CONV3) {
        int a, b, c;
        if (p.Cin % 8 != 0) return false;
        if (p.stride != 1 && !(p.stride == 2 && p.H % 2 == 0 && p.W % 2 == 0)) return false;
        return conv_box(p.Ho, p.Wo, &a, &b, &c);
    }
    return amode == A_LINEAR && p.K % 8 == 0 && p.ldx % 8 == 0 && (reinterpret_cast<uintptr_t>(p.X) & 15) == 0;
}

int run_pair(const Params& p, int amode, const void* packed, int w_bits, cudaStream_t stream)
{
    const int num_sms = sm_count();
    if (num_sms <= 0) return MIXDQ_ERR_CUDA;
    int rc = MIXDQ_OK;
    i8::TmaParams tp{};
    tp.M = p.M;
    tp.N = p.N;
    tp.w_scale = p.w_scale;
    tp.bias = p.bias;
    tp.Y = p.Y;
    tp.ldy = p.ldy;
    tp.status = p.status;
    tp.tma_store = p.Y && p.ldy % 8 == 0 && (reinterpret_cast<uintptr_t>(p.Y) & 15) == 0;
    CUtensorMap ta, tw, ty{};
    if (amode == A_CONV3) {
        int Wb, Hb, Bb;
        if (!conv_box(p.Ho, p.Wo, &Wb, &Hb, &Bb)) return MIXDQ_ERR_UNSUPPORTED;
        const uint64_t dims[4] = {static_cast<uint64_t>(p.Cin), static_cast<uint64_t>(p.W), static_cast<uint64_t>(p.H),
                                  static_cast<uint64_t>(p.batch)};
        const uint64_t strides[3] = {static_cast<uint64_t>(p.Cin) * 2, static_cast<uint64_t>(p.Cin) * p.W * 2,
                                     static_cast<uint64_t>(p.Cin) * p.W * p.H * 2};
        const uint32_t box[4] = {BKE, static_cast<uint32_t>(Wb), static_cast<uint32_t>(Hb), static_cast<uint32_t>(Bb)};
        rc = encode_tmap_4d_f16(&ta, p.X, dims, strides, box, static_cast<uint32_t>(p.stride));
        tp.conv = 1;
        tp.stride = p.stride;
        tp.cblocks = static_cast<int>(ceil_div(p.Cin, BKE));
        tp.Cin = p.Cin;
        tp.HoWo = p.Ho * p.Wo;
        tp.Wo = p.Wo;
        tp.batch = p.batch;
        tp.k_blocks = 9 * tp.cblocks;
    } else {
        rc = encode_tmap_2d_f16(&ta, p.X, static_cast<uint64_t>(p.K), static_cast<uint64_t>(p.M),
                                static_cast<uint64_t>(p.ldx), BKE, BM);
        tp.k_blocks = static_cast<int>(ceil_div(p.K, BKE));
    }
    if (rc != MIXDQ_OK) return rc;
    int splits = 1;
    const int bn = pick_tile(p.M, p.N, tp.k_blocks, num_sms, &splits);
    if (tp.tma_store) {
        rc = encode_tmap_2d_f16(&ty, p.Y, static_cast<uint64_t>(p.N), static_cast<uint64_t>(p.M),
                                static_cast<uint64_t>(p.ldy), 32, 32, true);
        if (rc != MIXDQ_OK) return rc;
    }
    const long long pitch = row_pitch_bytes(p.K, w_bits, MIXDQ_LAYOUT_DEVICE);
    // Unsplit reductions: the packed weights go to the GEMM kernel as they are and each CTA expands its half of a
    // weight tile in shared memory (a k-block of a convolution must be a whole block of the flattened reduction
    // index, i.e. Cin a multiple of 64).  Split reductions (few tiles, long reductions) and 8-bit weights (whose packed
    // tiles would take the shared memory of two activation slots) keep the expansion pass, and so do layers of more
    // than 2048 rows: every 256-row tile expands its weights again, and the in-kernel expansion makes the main loop
    // about 1.3 times slower (measured: 16384 x 640 x 5760 104 against 79 us, 4096 x 640 x 2560 19.0 against 15.6,
    // while 1024 x 1280 x 1280 gains 0.5 us and 1024 x 1280 x 5120 1.0 us from the launch it saves).
    if (splits == 1 && w_bits <= 4 && p.M <= 2048 && (amode != A_CONV3 || p.Cin % BKE == 0)) {
        rc = encode_tmap_2d_u8(&tw, packed, static_cast<uint64_t>(pitch), static_cast<uint64_t>(p.N), static_cast<uint64_t>(pitch),
                               static_cast<uint32_t>(16 * w_bits), static_cast<uint32_t>(bn / 2), false);
        if (rc != MIXDQ_OK) return rc;
        return i8::launch_pair_wo(ta, tw, ty, tp, bn, w_bits, p.w_zero, num_sms, stream);
    }
    // the layer's weights as fp16 integers, once per call
    __half* wexp = static_cast<__half*>(p.workspace);
    const int ldw = static_cast<int>(round_up(p.K, 8));
    const bool is_signed = p.w_zero == nullptr;
    rc = MIXDQ_ERR_UNSUPPORTED;
    if (w_bits == 8)
        rc = is_signed ? launch_expand<8, true>(packed, pitch, p.N, p.K, ldw, p.w_zero, wexp, stream)
                       : launch_expand<8, false>(packed, pitch, p.N, p.K, ldw, p.w_zero, wexp, stream);
    else if (w_bits == 4)
        rc = is_signed ? launch_expand<4, true>(packed, pitch, p.N, p.K, ldw, p.w_zero, wexp, stream)
                       : launch_expand<4, false>(packed, pitch, p.N, p.K, ldw, p.w_zero, wexp, stream);
    else if (w_bits == 3 && !is_signed)
        rc = launch_expand<3, false>(packed, pitch, p.N, p.K, ldw, p.w_zero, wexp, stream);
    else if (w_bits == 2 && !is_signed)
        rc = launch_expand<2, false>(packed, pitch, p.N, p.K, ldw, p.w_zero, wexp, stream);
    if (rc != MIXDQ_OK) return rc;

    rc = encode_tmap_2d_f16(&tw, wexp, static_cast<uint64_t>(p.K), static_cast<uint64_t>(p.N), static_cast<uint64_t>(ldw),
                            BKE, static_cast<uint32_t>(bn / 2));
    if (rc != MIXDQ_OK) return rc;
    return i8::launch_pair_f16(ta, tw, ty, tp, bn, splits, num_sms, stream);
}

}  // namespace wo
}  // namespace mixdq
