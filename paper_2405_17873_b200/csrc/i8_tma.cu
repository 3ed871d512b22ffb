// Two-kernel form of the W8A8 / W4A8 engine for layers large enough to be bound by the
// tensor cores or by on-chip bandwidth rather than by launch latency:
//   1. quant_kernel: the per-tensor fp16 -> int8 activation quantization, once per layer
//      (the fused engine in i8_gemm.cu repeats it for every tile column and, for a 3x3 conv,
//      for every filter tap);
//   2. tma_gemm_kernel: both operands arrive by TMA in the 128-byte-swizzled layout that
//      tcgen05.mma reads, so the main loop does no arithmetic of its own for int8 weights and
//      only the nibble expansion for int4 weights.  A 3x3 convolution is an implicit GEMM:
//      the A tile of filter tap (kh, kw) is a 4-D box of the int8 NHWC image shifted by
//      (kh - 1, kw - 1), and the zero padding is TMA's out-of-bounds fill.
// Output tile 128 x BN (BN = 128 or 256), 128-wide k-blocks, accumulators in tensor memory.
#include <algorithm>
#include <cmath>

#include "common.cuh"
#include "engines.h"
#include "i8_tiles.cuh"

namespace mixdq {
namespace i8 {

namespace {

constexpr float kMagic = 12582912.f;  // 1.5 * 2^23: fma(x, inv, magic) rounds x * inv to nearest even

// Four codes as bytes.  Symmetric: clamp(rne(x * inv), -127, 127).  Asymmetric (zoff = zero - 128):
// clamp(rne(x * inv) + zero, 0, 255) - 128, the unsigned code moved into int8 range; the rounding is done
// against the even magic constant before the offset is added, so that ties fall as they do without it.
__device__ __forceinline__ uint32_t q4(float a, float b, float c, float d, float inv, float lo, float hi, uint32_t zoff)
{
    const uint32_t qa = __float_as_uint(fminf(fmaxf(fmaf(a, inv, kMagic), lo), hi)) + zoff;
    const uint32_t qb = __float_as_uint(fminf(fmaxf(fmaf(b, inv, kMagic), lo), hi)) + zoff;
    const uint32_t qc = __float_as_uint(fminf(fmaxf(fmaf(c, inv, kMagic), lo), hi)) + zoff;
    const uint32_t qd = __float_as_uint(fminf(fmaxf(fmaf(d, inv, kMagic), lo), hi)) + zoff;
    return __byte_perm(__byte_perm(qa, qb, 0x0040), __byte_perm(qc, qd, 0x0040), 0x5410);
}

// 16 consecutive fp16 values (16-byte aligned) to 16 code bytes.
__device__ __forceinline__ uint4 quantize16(const __half* __restrict__ p, float inv, float lo, float hi, uint32_t zoff)
{
    const uint4* src = reinterpret_cast<const uint4*>(p);
    const uint4 v0 = __ldg(src), v1 = __ldg(src + 1);
    const __half2* h0 = reinterpret_cast<const __half2*>(&v0);
    const __half2* h1 = reinterpret_cast<const __half2*>(&v1);
    float2 f[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        f[j] = __half22float2(h0[j]);
        f[4 + j] = __half22float2(h1[j]);
    }
    uint4 o;
    o.x = q4(f[0].x, f[0].y, f[1].x, f[1].y, inv, lo, hi, zoff);
    o.y = q4(f[2].x, f[2].y, f[3].x, f[3].y, inv, lo, hi, zoff);
    o.z = q4(f[4].x, f[4].y, f[5].x, f[5].y, inv, lo, hi, zoff);
    o.w = q4(f[6].x, f[6].y, f[7].x, f[7].y, inv, lo, hi, zoff);
    return o;
}

// One thread per 16 consecutive elements of a row.  bos != 0: output row r reads input row
// (r / 76) * 77 + r % 76 + 1, i.e. the BOS token of every prompt is left out.
// act_zero != nullptr: asymmetric codes with that zero-point (see q4).
__global__ void quant_kernel(const __half* __restrict__ X, long long ldx, long long rows, int K, int bos,
                             const float* __restrict__ act_scale, const int32_t* __restrict__ act_zero,
                             int8_t* __restrict__ out)
{
    pdl_launch_dependents();
    pdl_wait();
    const int cpr = K >> 4;
    const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    if (idx >= rows * cpr) return;
    const long long r = idx / cpr;
    const int c = static_cast<int>(idx - r * cpr);
    long long src_row = r;
    if (bos) {
        const long long prompt = r / (MIXDQ_TOKENS_PER_PROMPT - 1);
        src_row = prompt * MIXDQ_TOKENS_PER_PROMPT + (r - prompt * (MIXDQ_TOKENS_PER_PROMPT - 1)) + 1;
    }
    const float inv = __fdiv_rn(1.f, __ldg(act_scale));
    float lo = kMagic - 127.f, hi = kMagic + 127.f;
    uint32_t zoff = 0;
    if (act_zero) {
        const int z = __ldg(act_zero);
        lo = kMagic - static_cast<float>(z);
        hi = kMagic + static_cast<float>(255 - z);
        zoff = static_cast<uint32_t>(z - 128);
    }
    *reinterpret_cast<uint4*>(out + r * K + c * 16) = quantize16(X + src_row * ldx + c * 16, inv, lo, hi, zoff);
}

// The int8 image of an asymmetrically quantized convolution input, with its padding written out: X fp16 NHWC
// [B, H, W, Cin] -> out int8 [B, H + 2, W + 2, Cin] whose one-pixel border holds the code of the real value
// 0 (the zero-point; stored re-centred, as zero - 128).  The GEMM's A tiles then never leave the image, and
// the padded positions cancel against the zero-point term like any other.  One thread per 16 channels.
__global__ void quant_pad_kernel(const __half* __restrict__ X, int B, int H, int W, int Cin,
                                 const float* __restrict__ act_scale, const int32_t* __restrict__ act_zero,
                                 int8_t* __restrict__ out)
{
    pdl_launch_dependents();
    pdl_wait();
    const int cpr = Cin >> 4;
    const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    if (idx >= static_cast<long long>(B) * (H + 2) * (W + 2) * cpr) return;
    const long long pix = idx / cpr;
    const int c = static_cast<int>(idx - pix * cpr);
    const int wp = static_cast<int>(pix % (W + 2));
    const long long t = pix / (W + 2);
    const int hp = static_cast<int>(t % (H + 2));
    const long long b = t / (H + 2);
    const int z = __ldg(act_zero);
    uint4 o;
    if (hp == 0 || hp == H + 1 || wp == 0 || wp == W + 1) {
        const uint32_t word = (static_cast<uint32_t>(z - 128) & 0xffu) * 0x01010101u;
        o = make_uint4(word, word, word, word);
    } else {
        const float inv = __fdiv_rn(1.f, __ldg(act_scale));
        const __half* src = X + ((b * H + (hp - 1)) * W + (wp - 1)) * Cin + c * 16;
        o = quantize16(src, inv, kMagic - static_cast<float>(z), kMagic + static_cast<float>(255 - z),
                       static_cast<uint32_t>(z - 128));
    }
    *reinterpret_cast<uint4*>(out + pix * Cin + c * 16) = o;
}

// Shortcut-splitting (Sec. 4.1): the input of a layer fed by a concatenation keeps one scale per branch.
// Columns [0, split) of every row are quantized with *scale_lo into the dense matrix out_lo [rows, split],
// columns [split, K) with *scale_hi into out_hi [rows, K - split].  split and K are multiples of 16, so a
// thread's 16 elements lie on one side.
__global__ void quant_split_kernel(const __half* __restrict__ X, long long ldx, long long rows, int K, int split,
                                   const float* __restrict__ scale_lo, const float* __restrict__ scale_hi,
                                   int8_t* __restrict__ out_lo, int8_t* __restrict__ out_hi)
{
    pdl_launch_dependents();
    pdl_wait();
    const int cpr = K >> 4;
    const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    if (idx >= rows * cpr) return;
    const long long r = idx / cpr;
    const int c = static_cast<int>(idx - r * cpr) * 16;
    const bool hi_side = c >= split;
    const float inv = __fdiv_rn(1.f, __ldg(hi_side ? scale_hi : scale_lo));
    const uint4 q = quantize16(X + r * ldx + c, inv, kMagic - 127.f, kMagic + 127.f, 0u);
    int8_t* dst = hi_side ? out_hi + r * (K - split) + (c - split) : out_lo + r * split + c;
    *reinterpret_cast<uint4*>(dst) = q;
}

// Barrier over all threads of all CTAs of the cluster (hardware barrier, not a spin).
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// 16 bytes from the shared memory of CTA `cta_rank` of this cluster, at this CTA's offset `addr`.
__device__ __forceinline__ int4 ld_cluster_v4(uint32_t addr, int cta_rank)
{
    // not volatile and no memory clobber: the data was published by the cluster barrier before,
    // and the compiler may then keep several of these loads in flight
    uint32_t remote;
    asm("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(addr), "r"(cta_rank));
    int4 v;
    asm("ld.shared::cluster.v4.s32 {%0, %1, %2, %3}, [%4];"
        : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
        : "r"(remote));
    return v;
}

// The 32-column passes for the second branch of a shortcut-split layer: y = acc * comb[c] + addend * ratio *
// comb[c] + bias[c], where comb[c] = s_hi * s_w and ratio = s_lo / s_hi.  The first branch's sums come in through
// the warp's staging tile, 16 columns at a time with four lanes along each row (coalesced), and the fp16 results
// leave through the same tile with two lanes along each row.
template <bool W4>
__device__ __forceinline__ void store_rows32_add_from_tmem(uint32_t acc, uint32_t acc2_off, int ncols, const float* comb,
                                                           const float* bias, uint8_t* stage, const TmaParams& p,
                                                           float ratio, int m_first, int n0, int lane)
{
    const bool yvec = ((p.ldy & 7) == 0) && ((p.N & 7) == 0);
    const bool avec = (p.N & 3) == 0;
    // The first branch's sums of one group of 16 columns: lane -> (row it * 8 + lane / 4, columns 4 * (lane % 4)...),
    // read through L2 (they are the previous kernel's output).  A group is fetched while the one before it is
    // converted and stored, so that its L2 round trip is not exposed.
    auto fetch = [&](int col, int4 (&pre)[4]) {
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int mm = m_first + it * 8 + (lane >> 2);
            const int n = n0 + col + (lane & 3) * 4;
            int4 a = make_int4(0, 0, 0, 0);
            if (col < ncols && mm < p.M && n < p.N) {
                const int32_t* ap = p.addend + static_cast<long long>(mm) * p.N + n;
                if (avec) {  // N % 4 == 0 and n % 4 == 0: four existing, 16-byte aligned columns
                    a = __ldcg(reinterpret_cast<const int4*>(ap));
                } else {
                    a.x = __ldcg(ap);
                    if (n + 1 < p.N) a.y = __ldcg(ap + 1);
                    if (n + 2 < p.N) a.z = __ldcg(ap + 2);
                    if (n + 3 < p.N) a.w = __ldcg(ap + 3);
                }
            }
            pre[it] = a;
        }
    };
    int4 pre[4];
    fetch(0, pre);
    for (int c0 = 0; c0 < ncols; c0 += 32) {
        if (n0 + c0 >= p.N) break;  // uniform across the warp
        uint32_t r[32];
        tmem_ld_32x32(acc + c0, r);
        if (acc2_off) {
            uint32_t r2[32];
            tmem_ld_32x32(acc + acc2_off + c0, r2);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) r[j] += r2[j];
        } else {
            tmem_ld_wait();
        }
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            __syncwarp();  // the tile's previous contents have been read out
#pragma unroll
            for (int it = 0; it < 4; ++it)
                *reinterpret_cast<int4*>(stage + (it * 8 + (lane >> 2)) * EPI32_ROW + (lane & 3) * 16) = pre[it];
            fetch(c0 + 16 * hh + 16, pre);  // the next group (nothing past the last column)
            __syncwarp();
            uint4 out[2];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int j = 16 * hh + 8 * q;  // column of the pass
                const int c = c0 + j;
                const int4 a0 = *reinterpret_cast<const int4*>(stage + lane * EPI32_ROW + q * 32);
                const int4 a1 = *reinterpret_cast<const int4*>(stage + lane * EPI32_ROW + q * 32 + 16);
                const float4 ca = *reinterpret_cast<const float4*>(comb + c);
                const float4 cb = *reinterpret_cast<const float4*>(comb + c + 4);
                const float4 ba = *reinterpret_cast<const float4*>(bias + c);
                const float4 bb = *reinterpret_cast<const float4*>(bias + c + 4);
                __half2 hv[4];
                hv[0] = __floats2half2_rn(
                    fmaf(acc_to_float<W4, false>(r[j]), ca.x, fmaf(static_cast<float>(a0.x), ca.x * ratio, ba.x)),
                    fmaf(acc_to_float<W4, false>(r[j + 1]), ca.y, fmaf(static_cast<float>(a0.y), ca.y * ratio, ba.y)));
                hv[1] = __floats2half2_rn(
                    fmaf(acc_to_float<W4, false>(r[j + 2]), ca.z, fmaf(static_cast<float>(a0.z), ca.z * ratio, ba.z)),
                    fmaf(acc_to_float<W4, false>(r[j + 3]), ca.w, fmaf(static_cast<float>(a0.w), ca.w * ratio, ba.w)));
                hv[2] = __floats2half2_rn(
                    fmaf(acc_to_float<W4, false>(r[j + 4]), cb.x, fmaf(static_cast<float>(a1.x), cb.x * ratio, bb.x)),
                    fmaf(acc_to_float<W4, false>(r[j + 5]), cb.y, fmaf(static_cast<float>(a1.y), cb.y * ratio, bb.y)));
                hv[3] = __floats2half2_rn(
                    fmaf(acc_to_float<W4, false>(r[j + 6]), cb.z, fmaf(static_cast<float>(a1.z), cb.z * ratio, bb.z)),
                    fmaf(acc_to_float<W4, false>(r[j + 7]), cb.w, fmaf(static_cast<float>(a1.w), cb.w * ratio, bb.w)));
                out[q] = *reinterpret_cast<const uint4*>(hv);
            }
            __syncwarp();  // every lane has read its row of sums
            *reinterpret_cast<uint4*>(stage + lane * EPI32_ROW) = out[0];
            *reinterpret_cast<uint4*>(stage + lane * EPI32_ROW + 16) = out[1];
            __syncwarp();
#pragma unroll
            for (int it = 0; it < 2; ++it) {
                const int rl = it * 16 + (lane >> 1), seg = lane & 1;
                const int mm = m_first + rl;
                const int n = n0 + c0 + 16 * hh + seg * 8;
                if (mm >= p.M || n >= p.N) continue;
                const uint4 v = *reinterpret_cast<const uint4*>(stage + rl * EPI32_ROW + seg * 16);
                __half* dst = p.Y + static_cast<long long>(mm) * p.ldy + n;
                if (yvec && n + 8 <= p.N) {
                    *reinterpret_cast<uint4*>(dst) = v;
                } else {
                    const __half* hs = reinterpret_cast<const __half*>(&v);
                    for (int q = 0; q < 8; ++q)
                        if (n + q < p.N) dst[q] = hs[q];
                }
            }
        }
        __syncwarp();
    }
}

// Rings of the pipeline and their barriers.  What bounds the k-block cadence of these kernels is neither the
// issue rate nor the tensor pipe but the bytes a CTA keeps in flight: a slot is away for about 1900 cycles
// (TMA request, L2 round trip, MMAs, commit, the producer noticing), so a ring of D tiles delivers one tile
// every 1900 / D cycles (measured with clock stamps: 6 stages of both operands -> 330 cycles per k-block,
// 4 activation stages -> 460), against 256 cycles of MMA work per 128 x 128 x 128 k-block.  Shared memory
// is the resource: everything not needed elsewhere goes into tiles that are in flight.
// W8: activation and weight tiles move in lockstep, STAGES deep.  W4 (128-wide tiles only): the packed int4
// rows have a ring of their own and are expanded into a short ring of int8 weight tiles, one slot per
// expansion group -- staging, not data in flight, so it is kept as small as the four groups allow.
template <int BN, int STAGES, bool W4, bool PERSIST>
struct Rings {
    static_assert(!W4 || BN == 128, "W4 runs on 128-wide tiles");
    static constexpr bool kW4 = W4;
    static constexpr int A_BYTES = BM * BK;
    static constexpr int B_BYTES = BN * BK;
    static constexpr int P_BYTES = BN * (BK / 2);
    // W4 needs an even number of int8 weight tiles: k-blocks alternate between the two MMA issuers by
    // the parity of their position in the CTA's sequence, so a weight slot always belongs to the same
    // issuer and its MMAs retire in order.  An expansion group reaches k-block i only after it has seen
    // the MMAs of k-block i - 4 - ES retire, which are the same issuer's as those of i - 2 ES: the
    // barrier of the slot can then never be a whole pair of phases behind what the group's parity wait
    // assumes.  (All rings of the W8 kernels are even for the same reason: an issuer must meet every
    // phase of the barriers it waits on.)
    static constexpr int AS = W4 ? 6 : STAGES;                  // activation tiles
    static constexpr int ES = W4 ? 4 : STAGES;                  // int8 weight tiles (W4: expanded, one per expansion group)
    static_assert(AS % 2 == 0 && ES % 2 == 0, "slots must keep their MMA issuer");
    static constexpr int PS = W4 ? (PERSIST ? 4 : 6) : 0;       // packed int4 weight tiles
    static constexpr int OFF_A = 0;
    static constexpr int OFF_B = OFF_A + AS * A_BYTES;
    static constexpr int OFF_P = OFF_B + ES * B_BYTES;
    static constexpr int RINGS_END = OFF_P + PS * P_BYTES;
    // barrier indices (8 bytes each)
    static constexpr int FULL_A = 0;                  // TMA bytes of the activation tile have landed
    static constexpr int EMPTY_A = FULL_A + AS;       // MMAs reading the tile have finished (W8: frees both tiles)
    static constexpr int READY_B = EMPTY_A + AS;      // W8: TMA bytes landed; W4: expansion finished
    static constexpr int EMPTY_B = READY_B + ES;      // W4: MMAs reading the int8 weight tile have finished
    static constexpr int FULL_P = EMPTY_B + ES;       // W4: TMA bytes of the packed tile have landed
    static constexpr int EMPTY_P = FULL_P + PS;       // W4: the packed tile has been read
    static constexpr int RING_BARS = EMPTY_P + PS;
};

template <class L>
__device__ __forceinline__ void init_ring_barriers(uint32_t bar0, bool w4)
{
    for (int s = 0; s < L::AS; ++s) {
        mbar_init(bar0 + 8 * (L::FULL_A + s), 1);
        mbar_init(bar0 + 8 * (L::EMPTY_A + s), 1);
    }
    for (int s = 0; s < L::ES; ++s) {
        mbar_init(bar0 + 8 * (L::READY_B + s), w4 ? 2 : 1);  // W4: the two warps of an expansion group
        mbar_init(bar0 + 8 * (L::EMPTY_B + s), 1);
    }
    for (int s = 0; s < L::PS; ++s) {
        mbar_init(bar0 + 8 * (L::FULL_P + s), 1);
        mbar_init(bar0 + 8 * (L::EMPTY_P + s), 2);
    }
}

// Activation tiles of one output tile, k-blocks kb_begin .. kb_begin + nkb - 1; seq0 = position of the
// first one in the CTA's running sequence of k-blocks (ring slot and phase follow from it).  Runs in a
// single thread; all indices are carried along instead of being recomputed.
template <class L>
__device__ __forceinline__ bool produce_a_tile(const CUtensorMap* tmap_a, const TmaParams& p, uint32_t seq0, int kb_begin,
                                               int nkb, int m0, uint32_t a0, uint32_t bar0, volatile int* s_abort)
{
    int img_b = 0, ho0 = 0, wo0 = 0, cb = 0, kh = 0, kw = 0;
    if (p.conv) {
        img_b = m0 / p.HoWo;
        const int rem = m0 - img_b * p.HoWo;
        ho0 = rem / p.Wo;
        wo0 = rem - ho0 * p.Wo;
        const int tap = kb_begin / p.cblocks;
        cb = kb_begin - tap * p.cblocks;
        kh = tap / 3;
        kw = tap - 3 * kh;
    }
    int xa = kb_begin * BK;
    uint32_t s = seq0 % L::AS, round = seq0 / L::AS;
    for (int i = 0; i < nkb; ++i) {
        // slots start out free
        if (round > 0 && !mbar_wait(bar0 + 8 * (L::EMPTY_A + s), (round & 1) ^ 1, s_abort)) return false;
        const uint32_t full = bar0 + 8 * (L::FULL_A + s);
        mbar_arrive_expect_tx(full, L::A_BYTES);
        if (p.conv) {
            tma_load_4d(a0 + s * L::A_BYTES, tmap_a, cb * BK, p.stride * wo0 + kw - 1 + p.pad,
                        p.stride * ho0 + kh - 1 + p.pad, img_b, full);
            if (++cb == p.cblocks) {
                cb = 0;
                if (++kw == 3) {
                    kw = 0;
                    ++kh;
                }
            }
        } else {
            tma_load_2d(a0 + s * L::A_BYTES, tmap_a, xa, m0, full);
            xa += BK;
        }
        if (++s == L::AS) {
            s = 0;
            ++round;
        }
    }
    return true;
}

// Weight tiles of one output tile: int8 tiles into the weight ring (W8) or packed int4 tiles into the
// packed ring (W4).  A thread of its own: one TMA issue costs a few hundred cycles of a single
// thread, and with both operands on one thread the issue rate sets the k-block cadence.
template <int BN, bool W4, class L>
__device__ __forceinline__ bool produce_b_tile(const CUtensorMap* tmap_w, const TmaParams& p, uint32_t seq0, int kb_begin,
                                               int nkb, int n0, uint32_t ring0, uint32_t bar0, volatile int* s_abort,
                                               int b_rows = BN)
{
    constexpr int ROW_BYTES = W4 ? BK / 2 : BK;
    constexpr int R = W4 ? L::PS : L::ES;
    constexpr int SLOT = W4 ? L::P_BYTES : L::B_BYTES;
    constexpr int FULL = W4 ? L::FULL_P : L::READY_B;
    constexpr int EMPTY = W4 ? L::EMPTY_P : L::EMPTY_A;  // W8: the MMA's commit frees both tiles of the slot
    int cb = 0, kx_tap = 0;
    if (p.conv) {
        const int tap = kb_begin / p.cblocks;
        cb = kb_begin - tap * p.cblocks;
        kx_tap = tap * p.Cin;  // first reduction index of the filter tap
    }
    int xb = kb_begin * ROW_BYTES;
    uint32_t s = seq0 % R, round = seq0 / R;
    for (int i = 0; i < nkb; ++i) {
        if (round > 0 && !mbar_wait(bar0 + 8 * (EMPTY + s), (round & 1) ^ 1, s_abort)) return false;
        const uint32_t full = bar0 + 8 * (FULL + s);
        mbar_arrive_expect_tx(full, static_cast<uint32_t>(b_rows * ROW_BYTES));  // the rows of the weight map's box
        // (self-test of the bounded waits: one announced tile is never requested)
        const bool drop = p.test_drop_b_kblock != 0 && kb_begin + i + 1 == p.test_drop_b_kblock;
        if (p.conv) {
            const int kx = kx_tap + cb * BK;
            if (!drop) tma_load_2d(ring0 + s * SLOT, tmap_w, W4 ? kx / 2 : kx, n0, full);
            if (++cb == p.cblocks) {
                cb = 0;
                kx_tap += p.Cin;
            }
        } else {
            if (!drop) tma_load_2d(ring0 + s * SLOT, tmap_w, xb, n0, full);
            xb += ROW_BYTES;
        }
        if (++s == R) {
            s = 0;
            ++round;
        }
    }
    return true;
}

// int4 -> int8 (x16) expansion of the weight tiles, run by four groups of two warps: group g takes
// the k-blocks g, g + 4, ... of the CTA's sequence, so four tiles are in the making at a time.  (A
// group's turn costs some 350 cycles of waits, fence and arrivals on top of its arithmetic, and a
// lone warp issues an instruction every four to five cycles: with two groups of four warps a tile
// took about 900 cycles per group against 620 for the two k-blocks' MMAs.)  A thread reads
// 16-byte runs of packed codes from the packed ring and writes them as two 16-byte chunks of the
// swizzled int8 tile: nibble -> high half of the byte (= 16 q), two ANDs and a shift per 8 codes.
template <int BN, class L>
__device__ __forceinline__ void expand_nibbles(int group, int gt, int lane, int total_kb, uint8_t* sB, const uint8_t* sP,
                                               uint32_t bar0, volatile int* s_abort, int b_rows = BN)
{
    const int runs = b_rows * 4;  // 16-byte packed runs of a tile
    constexpr int RUNS = (BN * 4) / 64;           // 16-byte packed runs per thread
    constexpr uint32_t PS = L::PS > 0 ? L::PS : 1;  // (instantiated, never run, for W8)
    for (int it = group; it < total_kb; it += 4) {
        const uint32_t sp = static_cast<uint32_t>(it) % PS, rp = static_cast<uint32_t>(it) / PS;
        const uint32_t se = static_cast<uint32_t>(it) % L::ES, re = static_cast<uint32_t>(it) / L::ES;
        bool ok = mbar_wait(bar0 + 8 * (L::FULL_P + sp), rp & 1, s_abort);
        if (ok && re > 0) ok = mbar_wait(bar0 + 8 * (L::EMPTY_B + se), (re & 1) ^ 1, s_abort);
        if (!__all_sync(0xffffffffu, ok)) break;  // the warp leaves together
        const uint8_t* stg = sP + sp * L::P_BYTES;
        uint8_t* b_stage = sB + se * L::B_BYTES;
        // all loads first: the compiler cannot move a load above a store to the other ring by itself
        uint4 wv[RUNS];
#pragma unroll
        for (int t = 0; t < RUNS; ++t) {
            const int task = gt + t * 64;
            wv[t] = task < runs ? *reinterpret_cast<const uint4*>(stg + (task >> 2) * (BK / 2) + (task & 3) * 16)
                                : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int t = 0; t < RUNS; ++t) {
            const int task = gt + t * 64;
            if (task >= runs) continue;
            const int r = task >> 2, j = task & 3;
            const uint4 w = wv[t];
            uint4 c0, c1;
            c0.x = (w.x << 4) & 0xF0F0F0F0u;
            c0.y = w.x & 0xF0F0F0F0u;
            c0.z = (w.y << 4) & 0xF0F0F0F0u;
            c0.w = w.y & 0xF0F0F0F0u;
            c1.x = (w.z << 4) & 0xF0F0F0F0u;
            c1.y = w.z & 0xF0F0F0F0u;
            c1.z = (w.w << 4) & 0xF0F0F0F0u;
            c1.w = w.w & 0xF0F0F0F0u;
            *reinterpret_cast<uint4*>(b_stage + sw128_offset(r, 2 * j)) = c0;
            *reinterpret_cast<uint4*>(b_stage + sw128_offset(r, 2 * j + 1)) = c1;
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
            mbar_arrive(bar0 + 8 * (L::READY_B + se));
            mbar_arrive(bar0 + 8 * (L::EMPTY_P + sp));
        }
    }
}

// The k-blocks first, first + step, ... of one output tile: wait for the tiles, issue the four MMAs
// into `acc`, hand the slots back.  Runs in a single thread; ring slots, phase parities and descriptors
// are carried along instead of recomputed.  seq0 as above; step <= 2.
template <int BN, bool W4, class L>
__device__ __forceinline__ bool issue_k_blocks(int first, int step, int nkb, uint32_t acc, uint32_t seq0, uint32_t a0,
                                               uint32_t b0, uint32_t bar0, volatile int* s_abort, int n_cols = BN)
{
    const uint32_t idesc = make_idesc(2, 1, BM, static_cast<uint32_t>(n_cols));
    static_assert(L::AS >= 2 && L::ES >= 2, "a step of two must stay inside one lap of a ring");
    if (first >= nkb) return true;
    const uint32_t q0 = seq0 + static_cast<uint32_t>(first);
    uint32_t sa = q0 % L::AS, pa = (q0 / L::AS) & 1, se = q0 % L::ES, pe = (q0 / L::ES) & 1;
    const uint64_t a_desc0 = smem_desc_sw128(a0), b_desc0 = smem_desc_sw128(b0);
    uint32_t accumulate = 0;
    for (int i = first; i < nkb; i += step) {
        if (!mbar_wait(bar0 + 8 * (L::FULL_A + sa), pa, s_abort)) return false;
        if (!mbar_wait(bar0 + 8 * (L::READY_B + se), pe, s_abort)) return false;
        tc_fence_after_sync();
        // (the start-address field counts 16-byte units and every tile lies below 256 KB: no carry out of it)
        const uint64_t a_desc = a_desc0 + sa * (L::A_BYTES >> 4);
        const uint64_t b_desc = b_desc0 + se * (L::B_BYTES >> 4);
        mma_i8_ss(acc, a_desc, b_desc, idesc, accumulate);
#pragma unroll
        for (int k = 1; k < BK / 32; ++k) mma_i8_ss(acc, a_desc + 2 * k, b_desc + 2 * k, idesc, 1u);
        accumulate = 1;
        tc_commit(bar0 + 8 * (L::EMPTY_A + sa));
        if (W4) tc_commit(bar0 + 8 * (L::EMPTY_B + se));
        sa += step;
        if (sa >= static_cast<uint32_t>(L::AS)) {
            sa -= L::AS;
            pa ^= 1;
        }
        se += step;
        if (se >= static_cast<uint32_t>(L::ES)) {
            se -= L::ES;
            pe ^= 1;
        }
    }
    return true;
}

template <int BN, int STAGES, bool W4>
struct TmaSmem : Rings<BN, STAGES, W4, false> {
    using R = Rings<BN, STAGES, W4, false>;
    static constexpr int OFF_BARS = R::RINGS_END;
    static constexpr int NUM_BARS = R::RING_BARS + 1;
    static constexpr int OFF_COMB = (OFF_BARS + NUM_BARS * 8 + 15) & ~15;  // read as float4
    static constexpr int OFF_BIAS = OFF_COMB + BN * 4;
    static constexpr int OFF_MISC = OFF_BIAS + BN * 4;
    static constexpr int TOTAL = OFF_MISC + 64 + 1024;
    static_assert(TOTAL <= 232448, "shared memory of one CTA");
    // warps: 0 activation producer, 1 MMA issuer, 2-5 per-column factors during the main loop, W4: 6-13
    // nibble expansion; then the weight producer and the second issuer.  An unsplit tile is dequantized and
    // stored by all sixteen warps (EPI_WARPS), each taking 32 rows x BN / 4 columns; a split tile is moved
    // to shared memory by warps 2-9.
    static constexpr int WORK_THREADS = W4 ? 448 : 320;
    static constexpr int B_WARP = WORK_THREADS / 32;      // TMA producer of the weight tiles
    // One thread issues a 128-wide MMA about every 68 cycles, the tensor core retires it in 64: a
    // lone issuer, which also waits and commits once per k-block, cannot keep the pipe busy.  Narrow
    // tiles therefore get a second issuer: even k-blocks accumulate into one accumulator, odd ones
    // into another, and the epilogue adds the two (integer adds: exact).
    static constexpr bool DUAL = BN == 128;
    static constexpr int MMA2_WARP = B_WARP + 1;
    static constexpr int EPI_WARPS = 16;
    static constexpr int THREADS = EPI_WARPS * 32;
    static_assert(WORK_THREADS + 32 + (DUAL ? 32 : 0) <= THREADS, "role warps");
    static_assert(EPI_WARPS * EPI32_TILE <= R::RINGS_END, "staging tiles lie in the drained pipeline buffers");
    static constexpr int TMEM_COLS = DUAL ? 2 * BN : BN;
};

template <int BN, int STAGES, bool W4, bool ADD = false>
__global__ void __maxnreg__(96)
tma_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                const __grid_constant__ CUtensorMap tmap_y, const TmaParams p)
{
    using L = TmaSmem<BN, STAGES, W4>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    uint8_t* sA = smem + L::OFF_A;
    uint8_t* sB = smem + L::OFF_B;
    uint8_t* sP = smem + L::OFF_P;  // W4: packed weight tiles
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BARS);
    float* s_comb = reinterpret_cast<float*>(smem + L::OFF_COMB);
    float* s_bias = reinterpret_cast<float*>(smem + L::OFF_BIAS);
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + L::OFF_MISC);
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + L::OFF_MISC + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // width of this launch's tiles: narrower than the template's 128 (96, 64 or 32) when that puts more CTAs on
    // the SMs in one wave; shared-memory slots and the accumulator keep the template's size
    const int bn = (BN == 128 && p.tile_n > 0) ? p.tile_n : BN;
    const int n0 = blockIdx.x * bn, m0 = blockIdx.y * BM;
    // the CTAs of a cluster (gridDim.z of them) share one output tile and split the reduction
    const int splits = gridDim.z, rank = blockIdx.z;
    const int kb_begin = static_cast<int>((static_cast<long long>(p.k_blocks) * rank) / splits);
    const int kb_end = static_cast<int>((static_cast<long long>(p.k_blocks) * (rank + 1)) / splits);
    const int nkb = kb_end - kb_begin;
    // an unsplit tile needs no pass through shared memory: its epilogue warps store it themselves
    // (nor does the second branch of a shortcut-split layer, whose epilogue reads the first branch's sums row-wise)
    const bool direct = splits == 1 && p.Y != nullptr && p.acc_out == nullptr && !ADD;
    const bool dual = L::DUAL && nkb >= 2;  // two MMA issuers, two accumulators

    const uint32_t bar0 = smem_u32(bars);  // ring barriers, see Rings
    const uint32_t bar_accum = smem_u32(bars + L::RING_BARS);

    pdl_launch_dependents();
    if (tid == 0) {
        init_ring_barriers<L>(bar0, W4);
        mbar_init(bar_accum, dual ? 2 : 1);
        *s_abort = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_w);
        if (p.tma_store) tma_prefetch_desc(&tmap_y);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(s_tmem), L::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    // everything above is independent of earlier kernels; global memory is not, except the packed
    // weights: no kernel that launches dependents early writes them, so their producer runs ahead
    // (nor do the warps that expand them, which touch shared memory only: the first weight tiles are expanded
    // while the previous kernel drains, and those warps wait before they turn to anything else)
    const bool expander = W4 && warp >= 6 && warp < L::B_WARP;
    if (warp != L::B_WARP && !expander) pdl_wait();
    const uint32_t tmem_base = *s_tmem;

    if (warp == 0) {
        // ------------------------------------------------------------ activation-tile producer
        if (lane == 0) produce_a_tile<L>(&tmap_a, p, 0, kb_begin, nkb, m0, smem_u32(sA), bar0, s_abort);
        __syncwarp();
    } else if (warp == L::B_WARP) {
        // ------------------------------------------------------------ weight-tile producer
        if (lane == 0)
            produce_b_tile<BN, W4, L>(&tmap_w, p, 0, kb_begin, nkb, n0, smem_u32(W4 ? sP : sB), bar0, s_abort, bn);
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const bool ok = issue_k_blocks<BN, W4, L>(0, dual ? 2 : 1, nkb, tmem_base, 0, smem_u32(sA), smem_u32(sB), bar0,
                                                      s_abort, bn);
            if (ok) tc_commit(bar_accum);
        }
        __syncwarp();
    } else if (warp < L::B_WARP) {
        if (warp < 6) {
            // -------------------------------------------------------- epilogue warps
            // while the main loop runs: per-column dequantization factors of this tile, and the
            // stored BOS rows
            const float sx = p.act_scale ? __ldg(p.act_scale) : 0.f;  // absent: accumulators only
            const int zshift = p.act_zero ? 128 - __ldg(p.act_zero) : 0;
            for (int j = tid - 64; j < bn; j += 128) {
                const int n = n0 + j;
                float comb = 0.f, b = 0.f;
                if (n < p.N && p.w_scale) {
                    comb = sx * __ldg(p.w_scale + n);
                    if (p.bias) b = __half2float(p.bias[n]);
                    // the zero-point term is constant along a column: it rides in the bias
                    if (p.act_zero) b = fmaf(static_cast<float>(zshift * __ldg(p.w_code_sums + n)), comb, b);
                }
                s_comb[j] = comb;
                s_bias[j] = b;
            }
            if (p.bos && p.Y && blockIdx.y == 0 && rank == 0) {
                // row 0 of every prompt: the stored floating-point BOS projection, copied as is
                for (int idx = tid - 64; idx < p.batch * BN; idx += 128) {
                    const int b = idx / BN, j = idx - b * BN;
                    if (j < bn && n0 + j < p.N)
                        p.Y[static_cast<long long>(b) * MIXDQ_TOKENS_PER_PROMPT * p.ldy + n0 + j] = p.bos_out[n0 + j];
                }
            }
        } else if (W4) {
            // -------------------------------------------------------- int4 -> int8 (x16) expansion
            const int group = (warp - 6) >> 1;  // warps 6-7, 8-9, 10-11, 12-13
            expand_nibbles<BN, L>(group, tid - 192 - group * 64, lane, nkb, sB, sP, bar0, s_abort, bn);
            pdl_wait();  // before these warps help with the epilogue
        }
        if (warp < 10 && !direct) {
            // -------------------------------------------------------- epilogue of a split tile, part 1
            // (or accumulator dump): warps 2-5 take the first half of the tile's columns, warps 6-9 the second
            // half; both read the 32 tensor-memory lanes their rank within a warpgroup gives access to
            asm volatile("bar.sync 1, 256;" ::: "memory");  // the factor tables above are complete
            bool ok = mbar_wait(bar_accum, 0, s_abort);
            tc_fence_after_sync();
            const bool go = __all_sync(0xffffffffu, ok && !*s_abort);
            const int lg = warp & 3;
            const int row = lg * 32 + lane;
            const int cbeg = warp < 6 ? 0 : BN / 2;
            const uint32_t acc = tmem_base + (static_cast<uint32_t>(lg * 32) << 16) + cbeg;
            if (go) {
                // tensor memory -> registers -> shared memory, 16-byte chunks XOR-swizzled by row
                uint8_t* prow = smem + row * (BN * 4);
                for (int c0 = 0; c0 < BN / 2; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld_32x32(acc + c0, r);
                    if (dual) {
                        uint32_t r2[32];
                        tmem_ld_32x32(acc + BN + c0, r2);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 32; ++j) r[j] += r2[j];
                    } else {
                        tmem_ld_wait();
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int chunk = ((cbeg + c0) >> 2) + j;
                        *reinterpret_cast<uint4*>(prow + ((chunk ^ (row & 7)) << 4)) =
                            make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
                    }
                }
            }
        }
    } else if (L::DUAL && warp == L::MMA2_WARP) {
        // ------------------------------------------------------------ second MMA issuer: odd k-blocks
        if (lane == 0 && dual) {
            const bool ok = issue_k_blocks<BN, W4, L>(1, 2, nkb, tmem_base + BN, 0, smem_u32(sA), smem_u32(sB), bar0,
                                                      s_abort, bn);
            if (ok) tc_commit(bar_accum);
        }
    }

    if (direct) {
        // ------------------------------------------------------------ epilogue of an unsplit tile
        // Every warp of the CTA, its main-loop role over, takes 32 rows (the tensor-memory lanes its rank
        // within a warpgroup gives access to) x BN / 4 columns: dequantize in registers, pass through a
        // staging tile in the drained pipeline buffers, store (TMA box 32 x 32, or coalesced).  With eight
        // warps the conversion, some six instructions per element, was issue-bound at about 2000 cycles.
        asm volatile("bar.sync 1, %0;" ::"n"(L::THREADS) : "memory");  // the factor tables are complete
        bool ok = mbar_wait(bar_accum, 0, s_abort);
        tc_fence_after_sync();
        constexpr int COLS = BN / (L::EPI_WARPS / 4);
        // (a column group past the tile's width has nothing to store)
        if (__all_sync(0xffffffffu, ok && !*s_abort) && (warp >> 2) * COLS < bn) {
            const int lg = warp & 3;
            const int cbeg = (warp >> 2) * COLS;
            const uint32_t acc = tmem_base + (static_cast<uint32_t>(lg * 32) << 16) + cbeg;
            uint8_t* stage = smem + warp * EPI32_TILE;
            store_rows32_dispatch<W4>(acc, dual ? BN : 0, COLS, s_comb + cbeg, s_bias + cbeg, stage, p, &tmap_y,
                                      m0 + lg * 32, n0 + cbeg, lane);
            if (p.tma_store && lane == 0) tma_store_wait_read();  // shared memory stays valid until then
        }
    }

    // ---------------------------------------------------------------- epilogue of a split tile, part 2
    // Every CTA of the cluster holds partial sums of the same tile in its shared memory.  CTA
    // `rank` adds up rows [rank * 128 / splits, ...) over all of them (integer adds: exact,
    // order-free), dequantizes and stores; threads run along a row so stores coalesce.
    __syncthreads();
    if (splits > 1) cluster_sync_all();
    if (!*s_abort && !direct) {
        // a thread keeps one group of four columns (its factors stay in registers) and walks
        // down the rows; consecutive threads take consecutive column groups
        const int rows_per = BM / splits;
        constexpr int CHUNKS = BN / 4;
        constexpr int RSTEP = L::WORK_THREADS / CHUNKS;
        static_assert(L::WORK_THREADS % CHUNKS == 0, "threads must tile the column groups");
        const int chunk = tid % CHUNKS;
        const int n = n0 + chunk * 4;
        const bool vec = ((p.ldy & 3) == 0) && n + 4 <= p.N;
        const float4 cb = *reinterpret_cast<const float4*>(s_comb + chunk * 4);
        const float4 bb = *reinterpret_cast<const float4*>(s_bias + chunk * 4);
        float4 cl = make_float4(0.f, 0.f, 0.f, 0.f);  // ADD: factors of the first branch's sums
        if (ADD && n < p.N && p.w_scale) {
            const float sl = __ldg(p.addend_scale);
            cl.x = sl * __ldg(p.w_scale + n);
            if (n + 1 < p.N) cl.y = sl * __ldg(p.w_scale + n + 1);
            if (n + 2 < p.N) cl.z = sl * __ldg(p.w_scale + n + 2);
            if (n + 3 < p.N) cl.w = sl * __ldg(p.w_scale + n + 3);
        }
        if (n < p.N && chunk * 4 < bn && tid < L::WORK_THREADS) {
#pragma unroll 2
            for (int rl = tid / CHUNKS; rl < rows_per; rl += RSTEP) {
                const int row = rank * rows_per + rl;
                const int m = m0 + row;
                if (m >= p.M) break;
                const uint8_t* src = smem + row * (BN * 4) + ((chunk ^ (row & 7)) << 4);
                int4 acc;
                if (splits == 1) {
                    acc = *reinterpret_cast<const int4*>(src);
                } else {
                    acc = make_int4(0, 0, 0, 0);
                    const uint32_t off = smem_u32(src);
                    int4 v[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) v[q] = (q < splits) ? ld_cluster_v4(off, q) : make_int4(0, 0, 0, 0);
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        acc.x += v[q].x;
                        acc.y += v[q].y;
                        acc.z += v[q].z;
                        acc.w += v[q].w;
                    }
                }
                if (p.acc_out) {
                    int32_t* dst = p.acc_out + static_cast<long long>(m) * p.N + n;
                    const int a[4] = {acc.x, acc.y, acc.z, acc.w};
                    const int zshift = p.act_zero ? 128 - __ldg(p.act_zero) : 0;
                    for (int j = 0; j < 4; ++j)
                        if (n + j < p.N)
                            dst[j] = (W4 ? (a[j] >> 4) : a[j]) + (p.act_zero ? zshift * __ldg(p.w_code_sums + n + j) : 0);
                }
                if (p.Y) {
                    long long out_row = m;
                    if (p.bos) {
                        const int prompt = m / (MIXDQ_TOKENS_PER_PROMPT - 1);
                        out_row = static_cast<long long>(prompt) * MIXDQ_TOKENS_PER_PROMPT +
                                  (m - prompt * (MIXDQ_TOKENS_PER_PROMPT - 1) + 1);
                    }
                    float4 b4 = bb;
                    if (ADD) {
                        const int32_t* ap = p.addend + static_cast<long long>(m) * p.N + n;
                        int4 a = make_int4(0, 0, 0, 0);
                        // (read through L2: the sums were written by the previous kernel of the stream)
                        if (((p.N & 3) == 0) && n + 4 <= p.N) {
                            a = __ldcg(reinterpret_cast<const int4*>(ap));
                        } else {
                            a.x = __ldcg(ap);
                            if (n + 1 < p.N) a.y = __ldcg(ap + 1);
                            if (n + 2 < p.N) a.z = __ldcg(ap + 2);
                            if (n + 3 < p.N) a.w = __ldcg(ap + 3);
                        }
                        b4.x = fmaf(static_cast<float>(a.x), cl.x, bb.x);
                        b4.y = fmaf(static_cast<float>(a.y), cl.y, bb.y);
                        b4.z = fmaf(static_cast<float>(a.z), cl.z, bb.z);
                        b4.w = fmaf(static_cast<float>(a.w), cl.w, bb.w);
                    }
                    __half2 h[2];
                    h[0] = __floats2half2_rn(fmaf(acc_to_float<W4, false>(acc.x), cb.x, b4.x),
                                             fmaf(acc_to_float<W4, false>(acc.y), cb.y, b4.y));
                    h[1] = __floats2half2_rn(fmaf(acc_to_float<W4, false>(acc.z), cb.z, b4.z),
                                             fmaf(acc_to_float<W4, false>(acc.w), cb.w, b4.w));
                    __half* dst = p.Y + out_row * p.ldy + n;
                    if (vec) {
                        *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(h);
                    } else {
                        const __half* hs = reinterpret_cast<const __half*>(h);
                        for (int j = 0; j < 4; ++j)
                            if (n + j < p.N) dst[j] = hs[j];
                    }
                }
            }
        }
    }
    if (*s_abort) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        if (tid == 0 && p.status) atomicExch(p.status, MIXDQ_ERR_TIMEOUT);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (splits > 1) cluster_sync_all();  // peers may still be reading this CTA's shared memory
    if (warp == 1) tmem_dealloc(tmem_base, L::TMEM_COLS);
}

// Persistent form for problems with at least as many output tiles as SMs: one CTA per SM
// walks over tiles (tile = blockIdx.x + i * gridDim.x, column-fastest so that concurrent CTAs
// share operands in L2).  Two accumulators in tensor memory alternate, so the epilogue of one
// tile (tensor memory -> registers -> fp16 stores) runs while the MMAs of the next tile are
// already being issued, and the TMA pipeline never drains between tiles.
template <int BN, int STAGES, bool W4>
struct PersistSmem : Rings<BN, STAGES, W4, true> {
    using R = Rings<BN, STAGES, W4, true>;
    static constexpr int OFF_BARS = R::RINGS_END;
    static constexpr int NUM_BARS = R::RING_BARS + 4;
    static constexpr int OFF_COMB = (OFF_BARS + NUM_BARS * 8 + 15) & ~15;  // [2][BN] floats
    static constexpr int OFF_BIAS = OFF_COMB + 2 * BN * 4;
    static constexpr int OFF_MISC = OFF_BIAS + 2 * BN * 4;
    static constexpr int OFF_EPI = (OFF_MISC + 64 + 1023) & ~1023;  // staging tiles of the eight epilogue warps
    static constexpr int TOTAL = OFF_EPI + 8 * EPI32_TILE + 1024;
    static_assert(TOTAL <= 232448, "shared memory of one CTA");
    // warps: 0 activation producer, 1 MMA issuer, 2-5 epilogue (first half of the tile's columns),
    // W4: 6-13 nibble expansion, then four epilogue helpers (second half of the columns)
    static constexpr int HELPER0 = W4 ? 14 : 6;
    static constexpr int WORK_THREADS = (HELPER0 + 4) * 32;
    static constexpr int B_WARP = WORK_THREADS / 32;      // TMA producer of the weight tiles
    static constexpr bool DUAL = BN == 128;               // second MMA issuer, as in the one-tile kernel
    static constexpr int MMA2_WARP = B_WARP + 1;
    static constexpr int THREADS = WORK_THREADS + 32 + (DUAL ? 32 : 0);
    static constexpr int ACC_COLS = DUAL ? 2 * BN : BN;   // tensor-memory columns of one tile's accumulator(s)
};

template <int BN, int STAGES, bool W4, bool ADD = false>
__global__ void __launch_bounds__(PersistSmem<BN, STAGES, W4>::THREADS, 1)
tma_gemm_persistent_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                           const __grid_constant__ CUtensorMap tmap_y, const TmaParams p, int n_tiles,
                           int total_tiles)
{
    using L = PersistSmem<BN, STAGES, W4>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    uint8_t* sA = smem + L::OFF_A;
    uint8_t* sB = smem + L::OFF_B;
    uint8_t* sP = smem + L::OFF_P;  // W4: packed weight tiles
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BARS);
    float* s_comb = reinterpret_cast<float*>(smem + L::OFF_COMB);
    float* s_bias = reinterpret_cast<float*>(smem + L::OFF_BIAS);
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + L::OFF_MISC);
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + L::OFF_MISC + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nkb = p.k_blocks;
    const bool dual = L::DUAL && nkb >= 2;  // two MMA issuers, two accumulators per tile
    const int my_tiles = (total_tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) /
                         static_cast<int>(gridDim.x);

    const uint32_t bar0 = smem_u32(bars);  // ring barriers, see Rings
    const uint32_t bar_acc_full = smem_u32(bars + L::RING_BARS);       // [2]: accumulator complete
    const uint32_t bar_acc_empty = smem_u32(bars + L::RING_BARS + 2);  // [2]: accumulator drained

    pdl_launch_dependents();
    if (tid == 0) {
        init_ring_barriers<L>(bar0, W4);
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_acc_full + 8 * b, dual ? 2 : 1);
            mbar_init(bar_acc_empty + 8 * b, 8);  // epilogue warps and their helpers
        }
        *s_abort = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_w);
        if (p.tma_store) tma_prefetch_desc(&tmap_y);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(s_tmem), 2 * L::ACC_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    // the weight producer runs ahead of earlier kernels, and so do the warps that expand int4 weight tiles
    if (warp != L::B_WARP && !(W4 && warp >= 6 && warp < L::HELPER0)) pdl_wait();
    const uint32_t tmem_base = *s_tmem;

    if (warp == 0) {
        // ------------------------------------------------------------ activation-tile producer
        if (lane == 0) {
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int tile = blockIdx.x + t * gridDim.x;
                ok = produce_a_tile<L>(&tmap_a, p, static_cast<uint32_t>(t * nkb), 0, nkb, (tile / n_tiles) * BM, smem_u32(sA),
                                       bar0, s_abort);
            }
        }
        __syncwarp();
    } else if (warp == L::B_WARP) {
        // ------------------------------------------------------------ weight-tile producer
        if (lane == 0) {
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int tile = blockIdx.x + t * gridDim.x;
                ok = produce_b_tile<BN, W4, L>(&tmap_w, p, static_cast<uint32_t>(t * nkb), 0, nkb, (tile % n_tiles) * BN,
                                               smem_u32(W4 ? sP : sB), bar0, s_abort);
            }
        }
        __syncwarp();
    } else if (warp == 1 || (L::DUAL && warp == L::MMA2_WARP)) {
        // ------------------------------------------------------------ MMA issuers
        // warp 1 (and, for narrow tiles, warp MMA2_WARP with the odd k-blocks and an accumulator of its own)
        if (lane == 0 && (warp == 1 || dual)) {
            const int which = warp == 1 ? 0 : 1;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int buf = t & 1;
                const uint32_t use = static_cast<uint32_t>(t >> 1);  // how often this accumulator was used before
                ok = mbar_wait(bar_acc_empty + 8 * buf, (use & 1) ^ 1, s_abort);
                if (!ok) break;
                tc_fence_after_sync();
                // k-blocks alternate between the issuers by the parity of their position in the CTA's
                // sequence (not in the tile: see Rings), so an issuer's first k-block of a tile is 0 or 1
                const int first = dual ? ((which + t * nkb) & 1) : 0;
                ok = issue_k_blocks<BN, W4, L>(first, dual ? 2 : 1, nkb, tmem_base + buf * L::ACC_COLS + which * BN,
                                               static_cast<uint32_t>(t * nkb), smem_u32(sA), smem_u32(sB), bar0, s_abort);
                if (ok) tc_commit(bar_acc_full + 8 * buf);
            }
        }
        __syncwarp();
    } else if (warp < 6 || (warp >= L::HELPER0 && warp < L::HELPER0 + 4)) {
        // ------------------------------------------------------------ epilogue warps and helpers
        const int lg = warp & 3;
        const int half = warp < 6 ? 0 : 1;
        const int et = tid - 64;  // epilogue warps only: 0..127
        const float sx = p.act_scale ? __ldg(p.act_scale) : 0.f;  // absent: accumulators only
        const int zshift = p.act_zero ? 128 - __ldg(p.act_zero) : 0;
        bool ok = true;
        for (int t = 0; t < my_tiles; ++t) {
            const int tile = blockIdx.x + t * gridDim.x;
            const int m0 = (tile / n_tiles) * BM, n0 = (tile % n_tiles) * BN;
            const int buf = t & 1;
            const uint32_t use = static_cast<uint32_t>(t >> 1);
            float* comb = s_comb + buf * BN;
            float* bias = s_bias + buf * BN;
            // this tile's per-column factors (the buffer was last read two tiles ago)
            for (int j = et; half == 0 && j < BN; j += 128) {
                const int n = n0 + j;
                float c = 0.f, b = 0.f;
                if (n < p.N && p.w_scale) {
                    c = sx * __ldg(p.w_scale + n);
                    if (p.bias) b = __half2float(p.bias[n]);
                    if (p.act_zero) b = fmaf(static_cast<float>(zshift * __ldg(p.w_code_sums + n)), c, b);
                }
                comb[j] = c;
                bias[j] = b;
            }
            if (half == 0 && p.bos && p.Y && m0 == 0) {
                for (int idx = et; idx < p.batch * BN; idx += 128) {
                    const int b = idx / BN, j = idx - b * BN;
                    if (n0 + j < p.N)
                        p.Y[static_cast<long long>(b) * MIXDQ_TOKENS_PER_PROMPT * p.ldy + n0 + j] = p.bos_out[n0 + j];
                }
            }
            if (ok) ok = mbar_wait(bar_acc_full + 8 * buf, use & 1, s_abort);
            tc_fence_after_sync();
            // the factor tables are complete; the same barrier carries the vote on whether every warp's
            // wait succeeded, so that all eight take the same path from here
            uint32_t go;
            asm volatile(
                "{\n\t"
                ".reg .pred p, q;\n\t"
                "setp.ne.u32 q, %1, 0;\n\t"
                "barrier.cta.red.and.pred p, 1, 256, q;\n\t"
                "selp.u32 %0, 1, 0, p;\n\t"
                "}\n"
                : "=r"(go)
                : "r"((ok && !*s_abort) ? 1u : 0u)
                : "memory");
            if (!go) {
                ok = false;
                continue;
            }
            const uint32_t acc = tmem_base + buf * L::ACC_COLS + (static_cast<uint32_t>(lg * 32) << 16);
            if (p.acc_out) {
                // raw int32 sums (parity hook; the branches of a shortcut-split layer): each half of the warps takes
                // its half of the columns, 16 at a time through the warp's staging tile (64-byte rows, 80 bytes
                // apart), so that four lanes store one row's 64 contiguous bytes
                const int cbeg = half * (BN / 2);
                uint8_t* stage = smem + L::OFF_EPI + (half * 4 + lg) * EPI32_TILE;
                const bool vec = ((p.N & 3) == 0) && ((reinterpret_cast<uintptr_t>(p.acc_out) & 15) == 0);
                if (p.tma_store && lane == 0) tma_store_wait_read();  // an output store may still read the tile
                for (int c0 = cbeg; c0 < cbeg + BN / 2; c0 += 32) {
                    if (n0 + c0 >= p.N) break;  // uniform across the warp
                    uint32_t r[32];
                    tmem_ld_32x32(acc + c0, r);
                    if (dual) {
                        uint32_t r2[32];
                        tmem_ld_32x32(acc + BN + c0, r2);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 32; ++j) r[j] += r2[j];
                    } else {
                        tmem_ld_wait();
                    }
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        int32_t v = W4 ? (static_cast<int32_t>(r[j]) >> 4) : static_cast<int32_t>(r[j]);
                        if (p.act_zero && n0 + c0 + j < p.N) v += zshift * __ldg(p.w_code_sums + n0 + c0 + j);
                        r[j] = static_cast<uint32_t>(v);
                    }
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        __syncwarp();  // the previous pass has been read out
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            *reinterpret_cast<uint4*>(stage + lane * EPI32_ROW + q * 16) =
                                make_uint4(r[16 * hh + 4 * q], r[16 * hh + 4 * q + 1], r[16 * hh + 4 * q + 2],
                                           r[16 * hh + 4 * q + 3]);
                        __syncwarp();
#pragma unroll
                        for (int it = 0; it < 4; ++it) {
                            const int rl = it * 8 + (lane >> 2), seg = lane & 3;
                            const int m = m0 + lg * 32 + rl;
                            const int n = n0 + c0 + 16 * hh + seg * 4;
                            if (m >= p.M || n >= p.N) continue;
                            const uint4 v = *reinterpret_cast<const uint4*>(stage + rl * EPI32_ROW + seg * 16);
                            int32_t* dst = p.acc_out + static_cast<long long>(m) * p.N + n;
                            if (vec) {  // n % 4 == 0 and N % 4 == 0: the four columns exist and are aligned
                                *reinterpret_cast<uint4*>(dst) = v;
                            } else {
                                const uint32_t a[4] = {v.x, v.y, v.z, v.w};
                                for (int j = 0; j < 4; ++j)
                                    if (n + j < p.N) dst[j] = static_cast<int32_t>(a[j]);
                            }
                        }
                    }
                }
                __syncwarp();
            }
            if (p.Y) {
                const int cbeg = half * (BN / 2);
                uint8_t* stage = smem + L::OFF_EPI + (half * 4 + lg) * EPI32_TILE;
                if (ADD)
                    store_rows32_add_from_tmem<W4>(acc + cbeg, dual ? BN : 0, BN / 2, comb + cbeg, bias + cbeg, stage, p,
                                                   __ldg(p.addend_scale) / sx, m0 + lg * 32, n0 + cbeg, lane);
                else
                    store_rows32_dispatch<W4>(acc + cbeg, dual ? BN : 0, BN / 2, comb + cbeg, bias + cbeg, stage, p,
                                              &tmap_y, m0 + lg * 32, n0 + cbeg, lane);
            }
            // the accumulator may be overwritten once every epilogue warp has read it
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acc_empty + 8 * buf);
        }
        if (p.tma_store && lane == 0) tma_store_wait_read();  // shared memory stays valid until then
    } else if (W4 && warp < L::HELPER0) {
        // ------------------------------------------------------------ int4 -> int8 (x16) expansion
        const int group = (warp - 6) >> 1;  // warps 6-7, 8-9, 10-11, 12-13
        expand_nibbles<BN, L>(group, tid - 192 - group * 64, lane, my_tiles * nkb, sB, sP, bar0, s_abort);
        pdl_wait();
    }

    if (*s_abort) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        if (tid == 0 && p.status) atomicExch(p.status, MIXDQ_ERR_TIMEOUT);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, 2 * L::ACC_COLS);
}

template <int BN, int STAGES, bool W4, bool ADD = false>
int launch_persistent(const CUtensorMap& ta, const CUtensorMap& tw, const CUtensorMap& ty, const TmaParams& tp, int num_sms,
                      cudaStream_t stream)
{
    using L = PersistSmem<BN, STAGES, W4>;
    auto kernel = tma_gemm_persistent_kernel<BN, STAGES, W4, ADD>;
    if (ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), L::TOTAL) != MIXDQ_OK) return MIXDQ_ERR_CUDA;
    const int n_tiles = static_cast<int>(ceil_div(tp.N, BN));
    const int total = n_tiles * static_cast<int>(ceil_div(tp.M, BM));
    const dim3 grid(static_cast<unsigned>(total < num_sms ? total : num_sms));
    return launch_pdl(kernel, grid, dim3(L::THREADS), L::TOTAL, stream, 1, ta, tw, ty, tp, n_tiles, total);
}

template <int BN, int STAGES, bool W4, bool ADD = false>
int launch_tma(const CUtensorMap& ta, const CUtensorMap& tw, const CUtensorMap& ty, const TmaParams& tp, int splits,
               cudaStream_t stream)
{
    using L = TmaSmem<BN, STAGES, W4>;
    auto kernel = tma_gemm_kernel<BN, STAGES, W4, ADD>;
    if (ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), L::TOTAL) != MIXDQ_OK) return MIXDQ_ERR_CUDA;
    const int bn = (BN == 128 && tp.tile_n > 0) ? tp.tile_n : BN;
    const dim3 grid(static_cast<unsigned>(ceil_div(tp.N, bn)), static_cast<unsigned>(ceil_div(tp.M, BM)),
                    static_cast<unsigned>(splits));
    return launch_pdl(kernel, grid, dim3(L::THREADS), L::TOTAL, stream, static_cast<unsigned>(splits), ta, tw, ty, tp);
}

// Reduction splits (cluster size): enough CTAs to cover the SMs, at least 4 k-blocks each.
int pick_splits(int64_t tiles, int k_blocks, int num_sms)
{
    int s = 1;
    while (s < 8 && tiles * (2 * s) <= num_sms && k_blocks / (2 * s) >= 2) s *= 2;
    return s;
}

}  // namespace

// Which kernel form runs an int8 GEMM of M x N over k_blocks k-blocks: 0 = the single-CTA kernels of this file,
// otherwise the tile width of the pair form.  Both are estimated in SM cycles from a model whose constants were
// fitted to timings of every layer shape of the SDXL-turbo-shaped UNet at image batch 1 and 4 on a B200 (each
// form at each width): rounds of tiles over the SMs (or SM pairs) times the cost of a tile -- the larger of its
// main loop, a per-k-block cost that grows with the tile width, and its epilogue -- plus fixed costs.
int plan_pair_tile(int M, int N, int k_blocks, bool w4, int num_sms, int* splits)
{
    if (splits) *splits = 1;
    if (M < 2 * BM || num_sms < 2) return 0;
    const double nkb = k_blocks;
    const int pairs = num_sms / 2;
    // pair form: 256 x bn tiles, widths below 160 never paid off
    double best = 0;
    int best_bn = 0, best_splits = 1;
    for (int bn = 160; bn <= 256; bn += 32) {
        const int64_t tiles = ceil_div(M, 2 * BM) * ceil_div(N, bn);
        const double per_kb = w4 ? 350.0 + 1.4 * bn : 250.0 + 1.2 * bn;
        const double rounds = std::ceil(static_cast<double>(tiles) / pairs);
        const double t = rounds * (std::max(nkb * per_kb, 30.0 * bn) + 800.0) + 16.0 * bn + 5000.0;
        if (best_bn == 0 || t < best) {
            best = t;
            best_bn = bn;
            best_splits = 1;
        }
        // few tiles, long reduction: one tile per cluster, the reduction split over up to four pairs; the
        // partial tiles meet through distributed shared memory at a fixed cost of some 14 000 cycles
        // (a cluster sits inside one GPC: the device holds fewer clusters of 4, 6 or 8 CTAs than SMs / size)
        for (int sp = 2; sp <= 4 && splits && tiles * sp <= pairs && k_blocks / sp >= 8; ++sp) {
            if (tiles > pair_cluster_capacity(w4, 2 * sp)) continue;
            const double ts = std::ceil(nkb / sp) * per_kb + 16.0 * bn + 14000.0 + 5000.0;
            if (ts < best) {
                best = ts;
                best_bn = bn;
                best_splits = sp;
            }
        }
    }
    // single-CTA kernels: 128 x 128 tiles (128 x 256 for wide int8 layers), persistent once the tiles cover the
    // SMs, else one tile per CTA with the reduction split over a cluster
    double old;
    const double c = w4 ? 580.0 : 420.0;
    const bool wide = !w4 && (N >= 1024 || N % 256 == 0) && ceil_div(M, BM) * ceil_div(N, 256) >= 100;
    if (wide) {
        const double tiles = static_cast<double>(ceil_div(M, BM) * ceil_div(N, 256));
        old = std::ceil(tiles / num_sms) * std::max(nkb * 620.0, 10000.0) + 3000.0;
    } else {
        const int64_t tiles = ceil_div(M, BM) * ceil_div(N, 128);
        if (tiles >= num_sms) {
            old = std::ceil(static_cast<double>(tiles) / num_sms) * std::max(nkb * c, 5000.0) + 3000.0;
        } else {
            const int s = pick_splits(tiles, k_blocks, num_sms);
            old = std::ceil(nkb / s) * c + 3000.0 + 3000.0 + (s > 1 ? 2500.0 : 0.0);
        }
    }
    if (best >= 1.05 * old) return 0;
    if (splits) *splits = best_splits;
    return best_bn;
}

// Fused-quantization kernel (i8_fq.cu) or the two-kernel forms.  The fused kernel's k-block costs three to four
// times the two-kernel main loop's (its converter warps' turn bounds it), and its fixed cost is one kernel's
// instead of two: it wins where the reduction is short (at most five k-blocks), the activations large enough for
// the quantization pass to matter, and the tiles fit the SMs in one wave.  Measured on B200, fused against
// two-kernel: 4096 x 640 x 640 W4 9.5 / 10.5 us, W8 7.8 / 9.2; 4096 x 640 x 320 7.5 / 9.9 and 6.5 / 8.7;
// 1024 x 640 x 640 W8 6.8 / 8.7, W4 8.3 / 8.7; losing: 1024 x 1280 x 640 (8.9 / 7.1), 16384 x 320 x 640 (two
// waves: 18.5 / 15.5), anything from ten k-blocks up (1024 x 1280 x 1280: 12.2 / 8.5).
// Width: the narrowest multiple of 32 whose tiles still fit one wave (less MMA and epilogue work per CTA).
int plan_fq_tile(int M, int N, int k_blocks, bool w4, int num_sms)
{
    (void)w4;
    if (k_blocks > 5 || N > 1024 || M < 1024) return 0;
    const int64_t row_tiles = ceil_div(M, BM);
    for (int bn = 64; bn <= 256; bn += 32)
        if (row_tiles * ceil_div(N, bn) <= num_sms) return bn;
    return 0;
}

// Width of the one-tile kernel's tiles for a layer the single-CTA kernels run on 128-wide slots: 128, or 96 / 64
// when that raises the number of CTAs while they still fit the SMs in one wave and the reduction is not split.
int plan_narrow_tile(int M, int N, int k_blocks, int num_sms)
{
    const int64_t row_tiles = ceil_div(M, BM);
    const int64_t t128 = row_tiles * ceil_div(N, 128);
    if (t128 >= num_sms || pick_splits(t128, k_blocks, num_sms) != 1) return 128;
    for (int cand : {64, 96}) {
        const int64_t t = row_tiles * ceil_div(N, cand);
        if (t < num_sms && t > t128) return cand;
    }
    return 128;
}

size_t tma_scratch_bytes(int64_t in_rows, int64_t K_row) { return static_cast<size_t>(round_up(in_rows * K_row, 256)); }

// Box of 128 consecutive output pixels as (Wb, Hb, Bb) in image coordinates; false when the
// image size does not tile that way.
static bool conv_box(int Ho, int Wo, int* Wb, int* Hb, int* Bb)
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

bool tma_path_ok(const Params& p, int amode, int w_bits)
{
    if (amode == A_CONV3) {
        int a, b, c;
        if (p.Cin % 32 != 0) return false;
        // stride 2: through the tensor map's element strides, for even images (Ho = H / 2, Wo = W / 2)
        if (p.stride != 1 && !(p.stride == 2 && p.H % 2 == 0 && p.W % 2 == 0)) return false;
        return conv_box(p.Ho, p.Wo, &a, &b, &c);
    }
    (void)w_bits;
    return p.K % 16 == 0 && p.ldx % 8 == 0 && (reinterpret_cast<uintptr_t>(p.X) & 15) == 0;
}

// Step 2 of the two-kernel path: the TMA-fed GEMM (or implicit-GEMM convolution) on int8 activations `aq`
// that an earlier kernel of the stream has written ([M, K] dense, or the NHWC image, padded when p.act_zero).
static int run_tma_gemm(const Params& p, int amode, const void* packed, int w_bits, int8_t* aq, cudaStream_t stream);

// One-kernel form: the GEMM kernel quantizes its own activation tiles (i8_fq.cu).
int run_fq(const Params& p, const void* packed, int w_bits, int bn, cudaStream_t stream)
{
    const bool w4 = w_bits == 4;
    const int64_t pitch = row_pitch_bytes(p.K, w_bits, MIXDQ_LAYOUT_DEVICE);
    CUtensorMap tx, tw, ty{};
    TmaParams tp{};
    tp.M = p.M;
    tp.N = p.N;
    tp.k_blocks = static_cast<int>(ceil_div(p.K, BK));
    tp.act_scale = p.act_scale;
    tp.w_scale = p.w_scale;
    tp.bias = p.bias;
    tp.Y = p.Y;
    tp.ldy = p.ldy;
    tp.acc_out = p.acc_out;
    tp.status = p.status;
    tp.small_acc = static_cast<long long>(p.K) * 127 * (w4 ? 7 : 127) < (1ll << 22);
    tp.tma_store = p.Y && p.ldy % 8 == 0 && (reinterpret_cast<uintptr_t>(p.Y) & 15) == 0;
    int rc = encode_tmap_2d_f16(&tx, p.X, static_cast<uint64_t>(p.K), static_cast<uint64_t>(p.M),
                                static_cast<uint64_t>(p.ldx), 64, BM, false);
    if (rc != MIXDQ_OK) return rc;
    if (w4)
        rc = encode_tmap_2d_u8(&tw, packed, static_cast<uint64_t>(pitch), p.N, pitch, BK / 2, static_cast<uint32_t>(bn), false);
    else
        rc = encode_tmap_2d_u8(&tw, packed, static_cast<uint64_t>(p.K), p.N, pitch, BK, static_cast<uint32_t>(bn), true);
    if (rc != MIXDQ_OK) return rc;
    if (tp.tma_store) {
        rc = encode_tmap_2d_f16(&ty, p.Y, static_cast<uint64_t>(p.N), static_cast<uint64_t>(p.M),
                                static_cast<uint64_t>(p.ldy), 32, 32, true);
        if (rc != MIXDQ_OK) return rc;
    }
    return launch_fq(tx, tw, ty, tp, w4, bn, stream);
}

int run_tma(const Params& p, int amode, const void* packed, int w_bits, void* scratch, cudaStream_t stream)
{
    int8_t* aq = static_cast<int8_t*>(scratch);
    if (amode == A_LINEAR && !p.act_zero && !p.addend && !p.test_drop_b_kblock) {
        const int num_sms = sm_count();
        const int fq_bn = num_sms > 0 ? plan_fq_tile(p.M, p.N, static_cast<int>(ceil_div(p.K, BK)), w_bits == 4, num_sms) : 0;
        if (fq_bn > 0) return run_fq(p, packed, w_bits, fq_bn, stream);
    }

    // 1. quantize the activations once
    const bool conv = amode == A_CONV3;
    const int pad = (conv && p.act_zero) ? 1 : 0;  // asymmetric conv input: the border is written out
    const long long in_rows = conv ? static_cast<long long>(p.batch) * (p.H + 2 * pad) * (p.W + 2 * pad) : p.M;
    const int row_len = conv ? p.Cin : p.K;
    const long long ldx = conv ? p.Cin : p.ldx;
    const long long tasks = in_rows * (row_len / 16);
    int rc;
    if (pad)
        rc = launch_pdl(quant_pad_kernel, dim3(static_cast<unsigned>(ceil_div(tasks, 256))), dim3(256), 0, stream, 1,
                        p.X, p.batch, p.H, p.W, p.Cin, p.act_scale, p.act_zero, aq);
    else
        rc = launch_pdl(quant_kernel, dim3(static_cast<unsigned>(ceil_div(tasks, 256))), dim3(256), 0, stream, 1,
                        p.X, ldx, in_rows, row_len, amode == A_BOS ? 1 : 0, p.act_scale, p.act_zero, aq);
    if (rc != MIXDQ_OK) return rc;
    return run_tma_gemm(p, amode, packed, w_bits, aq, stream);
}

static int run_tma_gemm(const Params& p, int amode, const void* packed, int w_bits, int8_t* aq, cudaStream_t stream)
{
    const bool w4 = w_bits == 4;
    const int64_t pitch = row_pitch_bytes(p.K, w_bits, MIXDQ_LAYOUT_DEVICE);
    const bool conv = amode == A_CONV3;
    const int pad = (conv && p.act_zero) ? 1 : 0;
    int rc;

    // 2. tensor maps
    CUtensorMap ta, tw, ty{};
    TmaParams tp{};
    tp.M = p.M;
    tp.N = p.N;
    tp.bos = amode == A_BOS;
    tp.batch = p.batch;
    tp.act_scale = p.act_scale;
    tp.act_zero = p.act_zero;
    tp.w_code_sums = p.w_code_sums;
    tp.w_scale = p.w_scale;
    tp.bias = p.bias;
    tp.bos_out = p.bos_out;
    tp.Y = p.Y;
    tp.ldy = p.ldy;
    tp.acc_out = p.acc_out;
    tp.status = p.status;
    // bound of any accumulator: K products of at most 127 * 127 (W4, after the shift: 127 * 7); the
    // re-centred codes of asymmetric activations reach -128
    tp.small_acc = static_cast<long long>(p.K) * (p.act_zero ? 128 : 127) * (w4 ? 7 : 127) < (1ll << 22);
    // output tiles leave through TMA stores when Y's rows are 16-byte aligned and consecutive output
    // rows are consecutive rows of Y (not so for the cross-attention K/V layout, which skips row 0)
    tp.addend = p.addend;
    tp.addend_scale = p.addend_scale;
    tp.test_drop_b_kblock = p.test_drop_b_kblock;
    tp.tma_store = p.Y && !p.addend && amode != A_BOS && p.ldy % 8 == 0 && (reinterpret_cast<uintptr_t>(p.Y) & 15) == 0;
    if (conv) {
        int Wb, Hb, Bb;
        if (!conv_box(p.Ho, p.Wo, &Wb, &Hb, &Bb)) return MIXDQ_ERR_UNSUPPORTED;
        const uint64_t Wi = static_cast<uint64_t>(p.W + 2 * pad), Hi = static_cast<uint64_t>(p.H + 2 * pad);
        const uint64_t dims[4] = {static_cast<uint64_t>(p.Cin), Wi, Hi, static_cast<uint64_t>(p.batch)};
        const uint64_t strides[3] = {static_cast<uint64_t>(p.Cin), static_cast<uint64_t>(p.Cin) * Wi,
                                     static_cast<uint64_t>(p.Cin) * Wi * Hi};
        const uint32_t box[4] = {BK, static_cast<uint32_t>(Wb), static_cast<uint32_t>(Hb), static_cast<uint32_t>(Bb)};
        rc = encode_tmap_4d_u8(&ta, aq, dims, strides, box, static_cast<uint32_t>(p.stride));
        tp.conv = 1;
        tp.pad = pad;
        tp.stride = p.stride;
        tp.cblocks = static_cast<int>(ceil_div(p.Cin, BK));
        tp.Cin = p.Cin;
        tp.HoWo = p.Ho * p.Wo;
        tp.Wo = p.Wo;
        tp.k_blocks = 9 * tp.cblocks;
    } else {
        rc = encode_tmap_2d_u8(&ta, aq, static_cast<uint64_t>(p.K), static_cast<uint64_t>(p.M),
                               static_cast<uint64_t>(p.K), BK, BM, true);
        tp.k_blocks = static_cast<int>(ceil_div(p.K, BK));
    }
    if (rc != MIXDQ_OK) return rc;
    const int num_sms = sm_count();
    if (num_sms <= 0) return MIXDQ_ERR_CUDA;
    // the pair form (two-CTA tiles of 256 x bn, i8_pair.cu) where its estimate beats the single-CTA kernels
    int pair_splits = 1;
    const int pair_bn = (!p.addend && amode != A_BOS && !p.test_drop_b_kblock)
                            ? plan_pair_tile(p.M, p.N, tp.k_blocks, w4, num_sms, &pair_splits) : 0;
    if (pair_bn > 0) {
        if (w4)
            rc = encode_tmap_2d_u8(&tw, packed, static_cast<uint64_t>(pitch), p.N, pitch, BK / 2, pair_bn / 2, false);
        else
            rc = encode_tmap_2d_u8(&tw, packed, static_cast<uint64_t>(p.K), p.N, pitch, BK, pair_bn / 2, true);
        if (rc != MIXDQ_OK) return rc;
        if (tp.tma_store) {
            rc = encode_tmap_2d_f16(&ty, p.Y, static_cast<uint64_t>(p.N), static_cast<uint64_t>(p.M),
                                    static_cast<uint64_t>(p.ldy), 32, 32, true);
            if (rc != MIXDQ_OK) return rc;
        }
        return launch_pair(ta, tw, ty, tp, w4, pair_bn, pair_splits, num_sms, stream);
    }
    // 256-wide tiles halve the A traffic per output but need enough tiles to cover the SMs
    // (W4 runs on 128-wide tiles only: its packed ring needs the room, and it measured no slower)
    const bool wide = !w4 && !p.addend && (p.N >= 1024 || p.N % 256 == 0) && ceil_div(p.M, BM) * ceil_div(p.N, 256) >= 100;
    uint32_t bn = wide ? 256 : 128;
    // Tile-count quantization of the one-tile kernel: a layer whose 128-wide tiles number between half the SMs
    // and all of them (1024 x 1280 outputs: 80 tiles on 148 SMs) leaves SMs idle and cannot split its reduction
    // either.  Narrower tiles (96 or 64 columns, multiples of the 32-column epilogue pass) in the same 128-wide
    // slots put more CTAs on the machine in one wave, each with proportionally less MMA, expansion and epilogue work.
    if (!wide && !p.addend) {
        bn = static_cast<uint32_t>(plan_narrow_tile(p.M, p.N, tp.k_blocks, num_sms));
        if (bn != 128) tp.tile_n = static_cast<int>(bn);
    }
    if (w4)
        rc = encode_tmap_2d_u8(&tw, packed, static_cast<uint64_t>(pitch), p.N, pitch, BK / 2, bn, false);
    else
        rc = encode_tmap_2d_u8(&tw, packed, static_cast<uint64_t>(p.K), p.N, pitch, BK, bn, true);
    if (rc != MIXDQ_OK) return rc;

    const int64_t tiles = ceil_div(p.M, BM) * ceil_div(p.N, bn);
    const bool persistent = tiles >= num_sms;
    if (tp.tma_store) {
        // store box: 32 columns x 32 rows (64-byte rows with the 64-byte swizzle), one per epilogue pass
        rc = encode_tmap_2d_f16(&ty, p.Y, static_cast<uint64_t>(p.N), static_cast<uint64_t>(p.M),
                                static_cast<uint64_t>(p.ldy), 32, 32, true);
        if (rc != MIXDQ_OK) return rc;
    }
    if (p.addend) {  // second branch of a shortcut-split layer: the instances with the two-scale epilogue
        if (persistent)
            return w4 ? launch_persistent<128, 6, true, true>(ta, tw, ty, tp, num_sms, stream)
                      : launch_persistent<128, 6, false, true>(ta, tw, ty, tp, num_sms, stream);
        const int sp = pick_splits(tiles, tp.k_blocks, num_sms);
        return w4 ? launch_tma<128, 6, true, true>(ta, tw, ty, tp, sp, stream)
                  : launch_tma<128, 6, false, true>(ta, tw, ty, tp, sp, stream);
    }
    if (persistent) {
        if (wide) return launch_persistent<256, 4, false>(ta, tw, ty, tp, num_sms, stream);
        return w4 ? launch_persistent<128, 6, true>(ta, tw, ty, tp, num_sms, stream)
                  : launch_persistent<128, 6, false>(ta, tw, ty, tp, num_sms, stream);
    }
    const int splits = pick_splits(tiles, tp.k_blocks, num_sms);
    if (wide) return launch_tma<256, 4, false>(ta, tw, ty, tp, splits, stream);
    return w4 ? launch_tma<128, 6, true>(ta, tw, ty, tp, splits, stream)
              : launch_tma<128, 6, false>(ta, tw, ty, tp, splits, stream);
}

// Step 1 alone: the int8 codes of X [rows, K] (row stride ldx) as a dense [rows, K] matrix.
int run_quant(const __half* X, long long ldx, long long rows, int K, const float* act_scale, int8_t* out,
              cudaStream_t stream)
{
    const long long tasks = rows * (K / 16);
    return launch_pdl(quant_kernel, dim3(static_cast<unsigned>(ceil_div(tasks, 256))), dim3(256), 0, stream, 1, X, ldx,
                      rows, K, 0, act_scale, static_cast<const int32_t*>(nullptr), out);
}

// Step 2 alone, on int8 activations the caller keeps (the stored form of an activation tensor).
int run_tma_prequantized(const Params& p, int amode, const void* packed, int w_bits, const int8_t* aq,
                         cudaStream_t stream)
{
    return run_tma_gemm(p, amode, packed, w_bits, const_cast<int8_t*>(aq), stream);
}

// Layout of the shortcut-split scratch: [int8 lo | int8 hi | int32 sums of the lo branch], each 256-byte aligned.
size_t split_layer_scratch_bytes(int64_t in_rows, int64_t row_len, int64_t split_at, int64_t out_rows, int64_t N)
{
    return static_cast<size_t>(round_up(in_rows * split_at, 256) + round_up(in_rows * (row_len - split_at), 256) +
                               round_up(out_rows * N * 4, 256));
}

bool split_path_ok(const Params& p, int amode, int split_at, int w_bits)
{
    if (amode != A_LINEAR && amode != A_CONV3) return false;
    const int row_len = amode == A_CONV3 ? p.Cin : p.K;
    if (split_at <= 0 || split_at >= row_len || split_at % 16 != 0 || row_len % 16 != 0) return false;
    if ((reinterpret_cast<uintptr_t>(p.X) & 15) != 0) return false;
    Params lo = p, hi = p;
    if (amode == A_CONV3) {
        lo.Cin = split_at;
        hi.Cin = row_len - split_at;
        lo.K = 9 * lo.Cin;
        hi.K = 9 * hi.Cin;
    } else {
        if (p.ldx % 8 != 0) return false;
        lo.K = split_at;
        hi.K = row_len - split_at;
    }
    return tma_path_ok(lo, amode, w_bits) && tma_path_ok(hi, amode, w_bits);
}

// Shortcut-splitting (Sec. 4.1): one quantization pass with a scale per branch, then one int8 GEMM (or
// implicit-GEMM convolution) per branch.  The first writes its exact int32 sums; the second is the instance with
// the two-scale epilogue, which reads those sums and stores y = fp16((s_lo * acc_lo + s_hi * acc_hi) * s_w[n] +
// bias[n]).  acc_lo_out / acc_hi_out given (parity hook, p.Y == nullptr): both kernels write their sums there.
int run_tma_split(const Params& p, int amode, int split_at, const void* packed_lo, const void* packed_hi, int w_bits,
                  const float* scale_lo, const float* scale_hi, int32_t* acc_lo_out, int32_t* acc_hi_out,
                  void* scratch, cudaStream_t stream)
{
    const bool conv = amode == A_CONV3;
    const long long in_rows = conv ? static_cast<long long>(p.batch) * p.H * p.W : p.M;
    const int row_len = conv ? p.Cin : p.K;
    const long long ldx = conv ? p.Cin : p.ldx;
    uint8_t* base = static_cast<uint8_t*>(scratch);
    int8_t* aq_lo = reinterpret_cast<int8_t*>(base);
    base += round_up(in_rows * split_at, 256);
    int8_t* aq_hi = reinterpret_cast<int8_t*>(base);
    base += round_up(in_rows * (row_len - split_at), 256);
    int32_t* acc_lo = p.Y ? reinterpret_cast<int32_t*>(base) : acc_lo_out;

    const long long tasks = in_rows * (row_len / 16);
    int rc = launch_pdl(quant_split_kernel, dim3(static_cast<unsigned>(ceil_div(tasks, 256))), dim3(256), 0, stream, 1,
                        p.X, ldx, in_rows, row_len, split_at, scale_lo, scale_hi, aq_lo, aq_hi);
    if (rc != MIXDQ_OK) return rc;

    // One launch where the two-CTA form suits the layer: both branches' k-blocks in one kernel, an accumulator per
    // branch in tensor memory, the two-scale epilogue straight from there (no int32 round trip through memory).
    const int num_sms = sm_count();
    if (num_sms <= 0) return MIXDQ_ERR_CUDA;
    const bool w4 = w_bits == 4;
    const int c_lo = split_at, c_hi = row_len - split_at;
    const int kb_lo = static_cast<int>(conv ? 9 * ceil_div(c_lo, BK) : ceil_div(c_lo, BK));
    const int kb_hi = static_cast<int>(conv ? 9 * ceil_div(c_hi, BK) : ceil_div(c_hi, BK));
    const int pair_bn = plan_pair_tile(p.M, p.N, kb_lo + kb_hi, w4, num_sms, nullptr);
    if (pair_bn > 0) {
        CUtensorMap ta[2], tw[2], ty{};
        const int8_t* aq[2] = {aq_lo, aq_hi};
        const void* pk[2] = {packed_lo, packed_hi};
        const int cin[2] = {c_lo, c_hi};
        for (int b = 0; b < 2; ++b) {
            const int64_t kb = conv ? 9ll * cin[b] : cin[b];
            const int64_t pitch = row_pitch_bytes(kb, w_bits, MIXDQ_LAYOUT_DEVICE);
            if (conv) {
                int Wb, Hb, Bb;
                if (!conv_box(p.Ho, p.Wo, &Wb, &Hb, &Bb)) return MIXDQ_ERR_UNSUPPORTED;
                const uint64_t dims[4] = {static_cast<uint64_t>(cin[b]), static_cast<uint64_t>(p.W), static_cast<uint64_t>(p.H),
                                          static_cast<uint64_t>(p.batch)};
                const uint64_t strides[3] = {static_cast<uint64_t>(cin[b]), static_cast<uint64_t>(cin[b]) * p.W,
                                             static_cast<uint64_t>(cin[b]) * p.W * p.H};
                const uint32_t box[4] = {BK, static_cast<uint32_t>(Wb), static_cast<uint32_t>(Hb), static_cast<uint32_t>(Bb)};
                rc = encode_tmap_4d_u8(&ta[b], aq[b], dims, strides, box, static_cast<uint32_t>(p.stride));
            } else {
                rc = encode_tmap_2d_u8(&ta[b], aq[b], static_cast<uint64_t>(cin[b]), static_cast<uint64_t>(p.M),
                                       static_cast<uint64_t>(cin[b]), BK, BM, true);
            }
            if (rc != MIXDQ_OK) return rc;
            if (w4)
                rc = encode_tmap_2d_u8(&tw[b], pk[b], static_cast<uint64_t>(pitch), p.N, pitch, BK / 2, pair_bn / 2, false);
            else
                rc = encode_tmap_2d_u8(&tw[b], pk[b], static_cast<uint64_t>(kb), p.N, pitch, BK, pair_bn / 2, true);
            if (rc != MIXDQ_OK) return rc;
        }
        TmaParams tp{};
        tp.M = p.M;
        tp.N = p.N;
        tp.k_blocks = kb_lo + kb_hi;
        tp.act_scale = scale_lo;
        tp.w_scale = p.w_scale;
        tp.bias = p.bias;
        tp.Y = p.Y;
        tp.ldy = p.ldy;
        tp.acc_out = p.Y ? nullptr : acc_lo_out;
        tp.status = p.status;
        tp.small_acc = 0;
        tp.tma_store = p.Y && p.ldy % 8 == 0 && (reinterpret_cast<uintptr_t>(p.Y) & 15) == 0;
        if (conv) {
            tp.conv = 1;
            tp.stride = p.stride;
            tp.cblocks = static_cast<int>(ceil_div(c_lo, BK));
            tp.Cin = c_lo;
            tp.HoWo = p.Ho * p.Wo;
            tp.Wo = p.Wo;
        }
        if (tp.tma_store) {
            rc = encode_tmap_2d_f16(&ty, p.Y, static_cast<uint64_t>(p.N), static_cast<uint64_t>(p.M),
                                    static_cast<uint64_t>(p.ldy), 32, 32, true);
            if (rc != MIXDQ_OK) return rc;
        }
        PairBranch second{};
        second.ta = &ta[1];
        second.tw = &tw[1];
        second.kb_first = kb_lo;
        second.cblocks = conv ? static_cast<int>(ceil_div(c_hi, BK)) : 0;
        second.Cin = conv ? c_hi : 0;
        second.act_scale = scale_hi;
        second.acc_out = p.Y ? nullptr : acc_hi_out;
        return launch_pair_two(ta[0], tw[0], ty, tp, w4, pair_bn, second, num_sms, stream);
    }

    Params q = p;
    q.Y = nullptr;
    q.bias = nullptr;
    q.act_zero = nullptr;
    q.w_code_sums = nullptr;
    q.acc_out = acc_lo;
    q.act_scale = scale_lo;
    q.Cin = conv ? split_at : 0;
    q.K = conv ? 9 * split_at : split_at;
    rc = run_tma_gemm(q, amode, packed_lo, w_bits, aq_lo, stream);
    if (rc != MIXDQ_OK) return rc;
    q.act_scale = scale_hi;
    q.Cin = conv ? row_len - split_at : 0;
    q.K = conv ? 9 * (row_len - split_at) : row_len - split_at;
    if (p.Y) {
        q.acc_out = nullptr;
        q.Y = p.Y;
        q.bias = p.bias;
        q.addend = acc_lo;
        q.addend_scale = scale_lo;
    } else {
        q.acc_out = acc_hi_out;
    }
    return run_tma_gemm(q, amode, packed_hi, w_bits, aq_hi, stream);
}

}  // namespace i8
}  // namespace mixdq
