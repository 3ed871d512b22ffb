// One-kernel form of a W8A8 / W4A8 linear layer: the per-tensor fp16 -> int8 activation quantization (Sec. 4.1)
// runs inside the GEMM kernel, so the layer is one launch instead of two and its activations make one trip from
// L2 instead of three (read fp16, write int8, read int8).
//
//   * the fp16 activation tile of a k-block arrives by TMA as two half-tiles (128 rows x 64 elements, 128-byte
//     swizzle); two groups of eight warps each turn one half into the 128-byte-swizzled int8 tile tcgen05.mma
//     reads, with the arithmetic of the stand-alone quantization kernel (fma against 1.5 * 2^23: one rounding);
//   * the same groups expand int4 weights (W4), half of the tile's rows each;
//   * output tile 128 x bn, bn a multiple of 32 up to 256: every tile column quantizes its 128 activation rows
//     again, so wide tiles keep the repeated arithmetic down.
// Measured on B200, this form is bound by the converter warps' turn (waits, some 3.3 instructions per element,
// proxy fence, arrival: 1500 cycles per k-block and more against 420 to 580 for the two-kernel path's main loop),
// so it pays only where the reduction is short and the quantization pass large: at most five k-blocks and one
// wave of tiles (the 4096 x 640 x 640 attention projections of the 32 x 32 level: 9.5 against 10.5 us with int4
// weights, 7.8 against 9.2 us with int8).  plan_fq_tile() selects those; everything else, and asymmetric
// activations, convolutions and the BOS-aware projection, stay on the two-kernel path.
#include "common.cuh"
#include "engines.h"
#include "i8_tiles.cuh"

namespace mixdq {
namespace i8 {

namespace {

constexpr int FQ_BN = 256;        // widest tile = tensor-memory columns of the accumulator
constexpr float kMagic = 12582912.f;  // 1.5 * 2^23

template <bool W4>
struct FqSmem {
    static constexpr int X_BYTES = BM * 64 * 2;   // fp16 half-tile: 128 rows x 64 elements
    static constexpr int A_BYTES = BM * BK;       // int8 activation tile
    static constexpr int B_BYTES = FQ_BN * BK;    // int8 weight tile
    static constexpr int P_BYTES = B_BYTES / 2;   // packed int4 weight tile
    // Half-tiles alternate between the two converter groups, so a group owns the ring slots of its parity and
    // meets every phase of their barriers; the int8 rings have one slot per MMA issuer for the same reason.
    static constexpr int XU = 6;
    static constexpr int QS = W4 ? 2 : 4;  // (a multiple of two: k-blocks alternate between the issuers)
    static constexpr int ES = 2;
    static constexpr int PS = W4 ? 2 : 0;
    static constexpr int OFF_X = 0;
    static constexpr int OFF_A = OFF_X + XU * X_BYTES;
    static constexpr int OFF_B = OFF_A + QS * A_BYTES;
    static constexpr int OFF_P = OFF_B + ES * B_BYTES;
    static constexpr int RINGS_END = OFF_P + PS * P_BYTES;
    static constexpr int FULL_X = 0;               // TMA bytes of the fp16 half-tile have landed
    static constexpr int EMPTY_X = FULL_X + XU;    // its converter group has read it
    static constexpr int FULL_A = EMPTY_X + XU;    // both halves of the int8 tile are written
    static constexpr int EMPTY_A = FULL_A + QS;    // the MMAs reading it have finished
    static constexpr int READY_B = EMPTY_A + QS;   // W8: TMA bytes landed; W4: expanded
    static constexpr int EMPTY_B = READY_B + ES;   // the MMAs reading the int8 weight tile have finished
    static constexpr int FULL_P = EMPTY_B + ES;    // W4: TMA bytes of the packed tile have landed
    static constexpr int EMPTY_P = FULL_P + (W4 ? PS : 0);  // W4: both groups have read it
    static constexpr int ACC_FULL = EMPTY_P + (W4 ? PS : 0);
    static constexpr int TILE_GO = ACC_FULL + 1;   // the first issuer has issued the overwriting MMA
    static constexpr int NUM_BARS = TILE_GO + 1;
    static constexpr int OFF_BARS = RINGS_END;
    static constexpr int OFF_COMB = (OFF_BARS + NUM_BARS * 8 + 15) & ~15;
    static constexpr int OFF_BIAS = OFF_COMB + FQ_BN * 4;
    static constexpr int OFF_MISC = OFF_BIAS + FQ_BN * 4;
    static constexpr int TOTAL = OFF_MISC + 64;  // the rings start at the (1024-byte aligned) base: no slack to round up in
    static_assert(TOTAL <= 232448, "shared memory of one CTA");
    // warps: 0 activation producer, 1 first MMA issuer and tensor-memory allocation, 2 second issuer, 3 weight
    // producer, 4-19 the two converter groups (4-11, 12-19), which are also the epilogue warps
    static constexpr int ALU0 = 4;
    static constexpr int GROUP_WARPS = 8;
    static constexpr int THREADS = (ALU0 + 2 * GROUP_WARPS) * 32;
    static_assert(2 * GROUP_WARPS * EPI32_TILE <= RINGS_END, "staging tiles lie in the drained pipeline buffers");
    static_assert(BM * FQ_BN * 4 <= RINGS_END, "the accumulator dump lies in the drained pipeline buffers");
};

// Largest fp16 value c with c * inv < 127.5, i.e. the largest input whose code needs no clamping, provided the code
// of c itself is 127 (true whenever fp16 is finer than the quantization step around 127 steps, which fails only for
// scales below about 1e-7 or above 500): then clamping the fp16 input to [-c, c] -- one packed min and one packed max
// per two elements -- gives the same codes as clamping the rounded product to [-127, 127] (rounding is monotonic:
// inputs beyond c round to at least 127.5 -> 128 -> 127, and c rounds to 127).  The products are exact in double
// (11 x 24 significant bits).  false: no such value; the caller clamps the rounded product instead.
__device__ __forceinline__ bool fp16_clamp_bound(float inv, __half* c_out)
{
    const float t = 127.5f / inv;
    if (!(t > 0.f) || !(t < 65000.f)) return false;
    const double dinv = static_cast<double>(inv);
    unsigned short bits = __half_as_ushort(__float2half_rz(t));
    for (int it = 0; it < 4 && bits > 0 && static_cast<double>(__half2float(__ushort_as_half(bits))) * dinv >= 127.5; ++it) --bits;
    for (int it = 0; it < 4 && bits < 0x7bfe &&
                     static_cast<double>(__half2float(__ushort_as_half(static_cast<unsigned short>(bits + 1)))) * dinv < 127.5;
         ++it)
        ++bits;
    const double prod = static_cast<double>(__half2float(__ushort_as_half(bits))) * dinv;
    const double next = static_cast<double>(__half2float(__ushort_as_half(static_cast<unsigned short>(bits + 1)))) * dinv;
    if (!(prod > 126.5 && prod < 127.5 && next >= 127.5)) return false;
    *c_out = __ushort_as_half(bits);
    return true;
}

// Two products rounded to nearest even by one packed fma against 1.5 * 2^23 each.
__device__ __forceinline__ float2 fma2_magic(float2 v, float inv)
{
    uint64_t a, b, c, d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(a) : "f"(v.x), "f"(v.y));
    asm("mov.b64 %0, {%1, %1};" : "=l"(b) : "f"(inv));
    asm("mov.b64 %0, {%1, %1};" : "=l"(c) : "f"(kMagic));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    float2 r;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(r.x), "=f"(r.y) : "l"(d));
    return r;
}

// 16 fp16 values (two 16-byte chunks) to 16 code bytes: clamp(rne(x * inv), -127, 127), the arithmetic of the
// stand-alone quantization kernel (one rounding, by an fma against 1.5 * 2^23).  FAST: the input is clamped as
// fp16 (see fp16_clamp_bound), so the low byte of the fma's result is the code.
template <bool FAST>
__device__ __forceinline__ uint4 quantize_chunks(const uint4& v0, const uint4& v1, float inv, __half2 c2)
{
    const __half2* h0 = reinterpret_cast<const __half2*>(&v0);
    const __half2* h1 = reinterpret_cast<const __half2*>(&v1);
    const float lo = kMagic - 127.f, hi = kMagic + 127.f;
    uint32_t w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        __half2 ha = j < 2 ? h0[2 * j] : h1[2 * j - 4];
        __half2 hb = j < 2 ? h0[2 * j + 1] : h1[2 * j - 3];
        uint32_t qa, qb, qc, qd;
        if (FAST) {
            ha = __hmin2(__hmax2(ha, __hneg2(c2)), c2);
            hb = __hmin2(__hmax2(hb, __hneg2(c2)), c2);
            const float2 ra = fma2_magic(__half22float2(ha), inv), rb = fma2_magic(__half22float2(hb), inv);
            qa = __float_as_uint(ra.x);
            qb = __float_as_uint(ra.y);
            qc = __float_as_uint(rb.x);
            qd = __float_as_uint(rb.y);
        } else {
            const float2 a = __half22float2(ha), b = __half22float2(hb);
            qa = __float_as_uint(fminf(fmaxf(fmaf(a.x, inv, kMagic), lo), hi));
            qb = __float_as_uint(fminf(fmaxf(fmaf(a.y, inv, kMagic), lo), hi));
            qc = __float_as_uint(fminf(fmaxf(fmaf(b.x, inv, kMagic), lo), hi));
            qd = __float_as_uint(fminf(fmaxf(fmaf(b.y, inv, kMagic), lo), hi));
        }
        w[j] = __byte_perm(__byte_perm(qa, qb, 0x0040), __byte_perm(qc, qd, 0x0040), 0x5410);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// Grid (tiles along N, tiles along M); tile 128 x bn.
template <bool W4>
__global__ void __launch_bounds__(FqSmem<W4>::THREADS, 1)
fq_gemm_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
               const __grid_constant__ CUtensorMap tmap_y, const TmaParams p, const int bn)
{
    using L = FqSmem<W4>;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = smem_raw;
    if ((smem_u32(smem) & 1023u) != 0) {
        // the swizzled tiles need a 1024-byte aligned base and the rings leave no room to round up
        if (threadIdx.x == 0 && p.status) atomicExch(p.status, MIXDQ_ERR_CUDA);
        return;
    }
    uint8_t* sX = smem + L::OFF_X;
    uint8_t* sA = smem + L::OFF_A;
    uint8_t* sB = smem + L::OFF_B;
    uint8_t* sP = smem + L::OFF_P;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BARS);
    float* s_comb = reinterpret_cast<float*>(smem + L::OFF_COMB);
    float* s_bias = reinterpret_cast<float*>(smem + L::OFF_BIAS);
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + L::OFF_MISC);
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + L::OFF_MISC + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = blockIdx.x * bn, m0 = blockIdx.y * BM;
    const int kb_begin = 0, nkb = p.k_blocks;
    // the accumulator dump (parity hook) leaves through shared memory; outputs alone are stored from tensor memory
    const bool direct = p.Y != nullptr && p.acc_out == nullptr;
    const uint32_t bar0 = smem_u32(bars);

    pdl_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < L::XU; ++s) {
            mbar_init(bar0 + 8 * (L::FULL_X + s), 1);
            mbar_init(bar0 + 8 * (L::EMPTY_X + s), L::GROUP_WARPS);
        }
        for (int s = 0; s < L::QS; ++s) {
            mbar_init(bar0 + 8 * (L::FULL_A + s), 2 * L::GROUP_WARPS);
            mbar_init(bar0 + 8 * (L::EMPTY_A + s), 1);
        }
        for (int s = 0; s < L::ES; ++s) {
            mbar_init(bar0 + 8 * (L::READY_B + s), W4 ? 2 * L::GROUP_WARPS : 1);
            mbar_init(bar0 + 8 * (L::EMPTY_B + s), 1);
        }
        for (int s = 0; s < L::PS; ++s) {
            mbar_init(bar0 + 8 * (L::FULL_P + s), 1);
            mbar_init(bar0 + 8 * (L::EMPTY_P + s), 2 * L::GROUP_WARPS);
        }
        mbar_init(bar0 + 8 * L::ACC_FULL, 2);
        mbar_init(bar0 + 8 * L::TILE_GO, 1);
        *s_abort = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmap_x);
        tma_prefetch_desc(&tmap_w);
        if (p.tma_store) tma_prefetch_desc(&tmap_y);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(s_tmem), FQ_BN);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *s_tmem;
    // the packed weights are written by no kernel that launches dependents early: their producer runs ahead of
    // the dependency wait; everything else that reads global memory waits first
    if (warp != 3) pdl_wait();

    if (warp == 0) {
        // ------------------------------------------------------------ fp16 activation half-tiles
        if (lane == 0) {
            const uint32_t x0 = smem_u32(sX);
            int xa = kb_begin * BK;
            uint32_t s = 0, round = 0;
            for (int u = 0; u < 2 * nkb; ++u) {
                if (round > 0 && !mbar_wait(bar0 + 8 * (L::EMPTY_X + s), (round & 1) ^ 1, s_abort)) break;
                const uint32_t full = bar0 + 8 * (L::FULL_X + s);
                mbar_arrive_expect_tx(full, L::X_BYTES);
                tma_load_2d(x0 + s * L::X_BYTES, &tmap_x, xa, m0, full);
                xa += 64;
                if (++s == L::XU) {
                    s = 0;
                    ++round;
                }
            }
        }
        __syncwarp();
    } else if (warp == 3) {
        // ------------------------------------------------------------ weight tiles (int8, or packed int4)
        if (lane == 0) {
            constexpr int ROW_BYTES = W4 ? BK / 2 : BK;
            constexpr int R = W4 ? L::PS : L::ES;
            constexpr int SLOT = W4 ? L::P_BYTES : L::B_BYTES;
            constexpr int FULL = W4 ? L::FULL_P : L::READY_B;
            constexpr int EMPTY = W4 ? L::EMPTY_P : L::EMPTY_B;
            const uint32_t ring0 = smem_u32(W4 ? sP : sB);
            int xb = kb_begin * ROW_BYTES;
            uint32_t s = 0, round = 0;
            for (int i = 0; i < nkb; ++i) {
                if (round > 0 && !mbar_wait(bar0 + 8 * (EMPTY + s), (round & 1) ^ 1, s_abort)) break;
                const uint32_t full = bar0 + 8 * (FULL + s);
                mbar_arrive_expect_tx(full, static_cast<uint32_t>(bn * ROW_BYTES));
                tma_load_2d(ring0 + s * SLOT, &tmap_w, xb, n0, full);
                xb += ROW_BYTES;
                if (++s == R) {
                    s = 0;
                    ++round;
                }
            }
        }
        __syncwarp();
    } else if (warp == 1 || warp == 2) {
        // ------------------------------------------------------------ MMA issuers
        // Issuer w takes the k-blocks w, w + 2, ... and so always slot w of both int8 rings; both add into one
        // accumulator (integer sums: the order is immaterial), after the first issuer's overwriting MMA.
        if (lane == 0) {
            const int which = warp - 1;
            const uint32_t idesc = make_idesc(2, 1, BM, static_cast<uint32_t>(bn));
            const uint64_t a_desc0 = smem_desc_sw128(smem_u32(sA));
            const uint64_t b_desc = smem_desc_sw128(smem_u32(sB) + which * L::B_BYTES);
            bool ok = true;
            uint32_t par = 0;  // of the weight slot (one per issuer)
            for (int i = which; i < nkb; i += 2, par ^= 1) {
                const uint32_t sa = static_cast<uint32_t>(i) % L::QS, pa = (static_cast<uint32_t>(i) / L::QS) & 1u;
                const uint64_t a_desc = a_desc0 + sa * (L::A_BYTES >> 4);
                if (!mbar_wait(bar0 + 8 * (L::FULL_A + sa), pa, s_abort) ||
                    !mbar_wait(bar0 + 8 * (L::READY_B + which), par, s_abort)) {
                    ok = false;
                    break;
                }
                if (i == 1 && !mbar_wait(bar0 + 8 * L::TILE_GO, 0, s_abort)) {
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                mma_i8_ss(tmem_base, a_desc, b_desc, idesc, i == 0 ? 0u : 1u);
#pragma unroll
                for (int k = 1; k < BK / 32; ++k) mma_i8_ss(tmem_base, a_desc + 2 * k, b_desc + 2 * k, idesc, 1u);
                if (i == 0) {
                    // the overwriting MMA is in the pipe's queue: the other thread may add to the accumulator
                    tc_fence_before_sync();
                    mbar_arrive(bar0 + 8 * L::TILE_GO);
                }
                tc_commit(bar0 + 8 * (L::EMPTY_A + sa));
                tc_commit(bar0 + 8 * (L::EMPTY_B + which));
            }
            // (an issuer without k-blocks still arrives: the barrier counts both)
            if (ok) tc_commit(bar0 + 8 * L::ACC_FULL);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ converter groups
        const int group = (warp - L::ALU0) / L::GROUP_WARPS;
        const int gt = tid - (L::ALU0 + group * L::GROUP_WARPS) * 32;  // 0..255 within the group
        // per-column dequantization factors of the tile (read by the epilogue)
        {
            const float sx = p.act_scale ? __ldg(p.act_scale) : 0.f;
            for (int j = tid - L::ALU0 * 32; j < bn; j += 2 * L::GROUP_WARPS * 32) {
                const int n = n0 + j;
                float comb = 0.f, b = 0.f;
                if (n < p.N && p.w_scale) {
                    comb = sx * __ldg(p.w_scale + n);
                    if (p.bias) b = __half2float(p.bias[n]);
                }
                s_comb[j] = comb;
                s_bias[j] = b;
            }
        }
        const float inv = __fdiv_rn(1.f, p.act_scale ? __ldg(p.act_scale) : 1.f);
        __half cbound = __ushort_as_half(0);
        const bool fast = fp16_clamp_bound(inv, &cbound);  // (uniform over the grid)
        const __half2 c2 = __half2half2(cbound);
        const int row = gt & 127, c = gt >> 7;  // this thread's row and the first of its two 16-element runs
        const uint32_t swz = static_cast<uint32_t>(row & 7);
        bool ok = true;
        for (int i = 0; i < nkb && ok; ++i) {
            const uint32_t es = static_cast<uint32_t>(i) & 1u, lap_e = static_cast<uint32_t>(i) >> 1;
            const uint32_t qs = static_cast<uint32_t>(i) % L::QS, lap = static_cast<uint32_t>(i) / L::QS;
            if (W4) {
                // this group's half of the weight tile's rows: int4 -> int8 (x16)
                const uint32_t ps = static_cast<uint32_t>(i) % (L::PS > 0 ? L::PS : 1), rp = static_cast<uint32_t>(i) / (L::PS > 0 ? L::PS : 1);
                // (one lane polls; the warp's reads are ordered behind its wait by the warp barrier)
                if (lane == 0) {
                    ok = mbar_wait(bar0 + 8 * (L::FULL_P + ps), rp & 1, s_abort);
                    if (ok && lap_e > 0) ok = mbar_wait(bar0 + 8 * (L::EMPTY_B + es), (lap_e & 1) ^ 1, s_abort);
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                __syncwarp();
                if (!ok) break;
                const uint8_t* stg = sP + ps * L::P_BYTES;
                uint8_t* b_stage = sB + es * L::B_BYTES;
                const int runs = bn * 4;  // 16-byte packed runs of the tile; the groups take alternate blocks of 256
                uint4 wv[2];
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const int task = gt + (2 * t + group) * 256;
                    wv[t] = task < runs ? *reinterpret_cast<const uint4*>(stg + task * 16) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const int task = gt + (2 * t + group) * 256;
                    if (task < runs) {
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
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(bar0 + 8 * (L::READY_B + es));
                    mbar_arrive(bar0 + 8 * (L::EMPTY_P + ps));
                }
            }
            // this group's half (64 reduction elements) of the activation tile: fp16 -> int8 codes
            const uint32_t u = 2u * static_cast<uint32_t>(i) + static_cast<uint32_t>(group);
            const uint32_t xs = u % L::XU, rx = u / L::XU;
            if (lane == 0) {
                ok = mbar_wait(bar0 + 8 * (L::FULL_X + xs), rx & 1, s_abort);
                if (ok && lap > 0) ok = mbar_wait(bar0 + 8 * (L::EMPTY_A + qs), (lap & 1) ^ 1, s_abort);
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            __syncwarp();
            if (!ok) break;
            const uint8_t* xrow = sX + xs * L::X_BYTES + row * 128;
            uint8_t* a_tile = sA + qs * L::A_BYTES;
            uint4 v[4];
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const uint32_t cc = static_cast<uint32_t>(c + 2 * t);  // 16-element run 0..3 of the half-tile's row
                v[2 * t] = *reinterpret_cast<const uint4*>(xrow + (((2 * cc) ^ swz) << 4));
                v[2 * t + 1] = *reinterpret_cast<const uint4*>(xrow + (((2 * cc + 1) ^ swz) << 4));
            }
            // (a branch, not a select: only one of the two forms runs)
            if (fast) {
#pragma unroll
                for (int t = 0; t < 2; ++t)
                    *reinterpret_cast<uint4*>(a_tile + sw128_offset(row, 4 * group + static_cast<uint32_t>(c + 2 * t))) =
                        quantize_chunks<true>(v[2 * t], v[2 * t + 1], inv, c2);
            } else {
#pragma unroll
                for (int t = 0; t < 2; ++t)
                    *reinterpret_cast<uint4*>(a_tile + sw128_offset(row, 4 * group + static_cast<uint32_t>(c + 2 * t))) =
                        quantize_chunks<false>(v[2 * t], v[2 * t + 1], inv, c2);
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar0 + 8 * (L::FULL_A + qs));
                mbar_arrive(bar0 + 8 * (L::EMPTY_X + xs));
            }
        }
    }

    // ---------------------------------------------------------------- epilogue
    const int ew = warp - L::ALU0;  // 0..15 for the converter warps
    if (direct) {
        // every converter warp takes 32 rows (the tensor-memory lanes its rank in a warpgroup reaches) x 64 columns
        asm volatile("bar.sync 1, %0;" ::"n"(L::THREADS) : "memory");  // the factor tables are complete
        if (ew >= 0) {
            bool ok = mbar_wait(bar0 + 8 * L::ACC_FULL, 0, s_abort);
            tc_fence_after_sync();
            const int lg = warp & 3, cbeg = (ew >> 2) * 64;
            if (__all_sync(0xffffffffu, ok && !*s_abort) && cbeg < bn) {
                const int ncols = bn - cbeg < 64 ? bn - cbeg : 64;
                const uint32_t acc = tmem_base + (static_cast<uint32_t>(lg * 32) << 16) + cbeg;
                uint8_t* stage = smem + ew * EPI32_TILE;
                store_rows32_dispatch<W4>(acc, 0, ncols, s_comb + cbeg, s_bias + cbeg, stage, p, &tmap_y, m0 + lg * 32,
                                          n0 + cbeg, lane);
                if (p.tma_store && lane == 0) tma_store_wait_read();
            }
        }
    } else {
        // accumulator dump: tensor memory -> shared memory, rows FQ_BN * 4 bytes apart, 16-byte chunks
        // XOR-swizzled by row
        asm volatile("bar.sync 1, %0;" ::"n"(L::THREADS) : "memory");
        if (ew >= 0) {
            bool ok = mbar_wait(bar0 + 8 * L::ACC_FULL, 0, s_abort);
            tc_fence_after_sync();
            const int lg = warp & 3, cbeg = (ew >> 2) * 64;
            if (__all_sync(0xffffffffu, ok && !*s_abort)) {
                const int rowl = lg * 32 + lane;
                uint8_t* prow = smem + rowl * (FQ_BN * 4);
                const uint32_t acc = tmem_base + (static_cast<uint32_t>(lg * 32) << 16);
                for (int c0 = cbeg; c0 < cbeg + 64 && c0 < bn; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld_32x32(acc + c0, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int chunk = (c0 >> 2) + j;
                        *reinterpret_cast<uint4*>(prow + ((chunk ^ (rowl & 7)) << 4)) =
                            make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
                    }
                }
            }
        }
    }

    __syncthreads();
    if (!*s_abort && !direct) {
        // consecutive threads take consecutive groups of four columns of a row, so the stores coalesce
        const int chunks = bn >> 2;
        const int total = BM * chunks;
        for (int idx = tid; idx < total; idx += L::THREADS) {
            const int rl = idx / chunks, chunk = idx % chunks;
            const int m = m0 + rl, n = n0 + chunk * 4;
            if (m >= p.M || n >= p.N) continue;
            const int4 v = *reinterpret_cast<const int4*>(smem + rl * (FQ_BN * 4) + ((chunk ^ (rl & 7)) << 4));
            const int a[4] = {v.x, v.y, v.z, v.w};
            if (p.acc_out) {
                int32_t* dst = p.acc_out + static_cast<long long>(m) * p.N + n;
                for (int j = 0; j < 4; ++j)
                    if (n + j < p.N) dst[j] = W4 ? (a[j] >> 4) : a[j];
            }
            if (p.Y) {
                __half h[4];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    h[j] = __float2half_rn(fmaf(acc_to_float<W4, false>(static_cast<uint32_t>(a[j])), s_comb[chunk * 4 + j],
                                                s_bias[chunk * 4 + j]));
                __half* dst = p.Y + static_cast<long long>(m) * p.ldy + n;
                if ((p.ldy & 3) == 0 && n + 4 <= p.N) {
                    *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(h);
                } else {
                    for (int j = 0; j < 4; ++j)
                        if (n + j < p.N) dst[j] = h[j];
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
    if (warp == 1) tmem_dealloc(tmem_base, FQ_BN);
}

template <bool W4>
int launch_fq_t(const CUtensorMap& tx, const CUtensorMap& tw, const CUtensorMap& ty, const TmaParams& tp, int bn,
                cudaStream_t stream)
{
    using L = FqSmem<W4>;
    auto kernel = fq_gemm_kernel<W4>;
    if (ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), L::TOTAL) != MIXDQ_OK) return MIXDQ_ERR_CUDA;
    const dim3 grid(static_cast<unsigned>(ceil_div(tp.N, bn)), static_cast<unsigned>(ceil_div(tp.M, BM)), 1u);
    return launch_pdl(kernel, grid, dim3(L::THREADS), L::TOTAL, stream, 1u, tx, tw, ty, tp, bn);
}

}  // namespace

int launch_fq(const CUtensorMap& tx, const CUtensorMap& tw, const CUtensorMap& ty, const TmaParams& tp, bool w4, int bn,
              cudaStream_t stream)
{
    if (bn < 32 || bn > FQ_BN || bn % 32 != 0 || tp.k_blocks < 1 || tp.conv || tp.bos || tp.act_zero || tp.addend)
        return MIXDQ_ERR_UNSUPPORTED;
    return w4 ? launch_fq_t<true>(tx, tw, ty, tp, bn, stream) : launch_fq_t<false>(tx, tw, ty, tp, bn, stream);
}

}  // namespace i8
}  // namespace mixdq
