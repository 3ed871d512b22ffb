// W8A8 / W4A8 engine: int8 x int8 -> int32 GEMM on the 5th-generation tensor cores
// (tcgen05.mma kind::i8, accumulators in tensor memory) for linear layers, the BOS-aware
// K/V projection and 3x3 convolution as an implicit GEMM.
//
// One CTA computes a 128 x BN output tile over a range of 128-wide k-blocks:
//   warp 0      TMA producer: weight tiles, global -> shared (128-byte swizzle for int8;
//               packed int4 goes to a staging buffer)
//   warp 1      owns tensor memory and issues the MMAs
//   warps 2..9  feed the A operand: read fp16 activations (plain rows, rows that skip the BOS
//               token, or the im2col gather of a 3x3 conv), quantize them to int8 with the
//               per-tensor scale and write them in the swizzled layout the MMA reads; for
//               W4 they also expand the staged nibbles to int8.  Afterwards the same warps
//               run the epilogue: tensor memory -> registers -> dequantize + bias -> fp16.
// Stages are handed over with mbarriers; every wait is bounded.
//
// int4 weights are expanded to (16 * q) by placing the nibble in the high half of the
// byte, which needs no sign extension; the factor 16 is divided out exactly afterwards.
#include <cstdlib>
#include <cstring>

#include "common.cuh"
#include "engines.h"

namespace mixdq {
namespace i8 {

constexpr int BM = 128;
constexpr int BK = 128;  // int8 elements per k-block = one 128-byte swizzled row
constexpr int kFeedWarps = 8;
constexpr int kFeedThreads = 32 * kFeedWarps;
constexpr int kThreads = 64 + kFeedThreads;
constexpr int A_STAGE_BYTES = BM * BK;

template <int BN, int STAGES, bool W4>
struct SmemLayout {
    static constexpr int B_STAGE_BYTES = BN * BK;
    static constexpr int STG_STAGE_BYTES = W4 ? BN * (BK / 2) : 0;
    static constexpr int OFF_A = 0;
    static constexpr int OFF_B = OFF_A + STAGES * A_STAGE_BYTES;
    static constexpr int OFF_STG = OFF_B + STAGES * B_STAGE_BYTES;
    static constexpr int OFF_BARS = OFF_STG + STAGES * STG_STAGE_BYTES;
    static constexpr int NUM_BARS = 3 * STAGES + 1;
    static constexpr int OFF_COMB = OFF_BARS + NUM_BARS * 8;
    static constexpr int OFF_BIAS = OFF_COMB + BN * 4;
    static constexpr int OFF_MISC = OFF_BIAS + BN * 4;
    static constexpr int TOTAL = OFF_MISC + 64 + 1024;  // + slack to align the base to 1024
};

// Magic-number rounding: fma(x, inv, 1.5 * 2^23) rounds the exact product x * inv to the
// nearest integer (ties to even) in one operation; the integer sits in the low mantissa bits.
constexpr float kMagic = 12582912.f;

__device__ __forceinline__ uint32_t quant4(float a, float b, float c, float d, float inv)
{
    const float lo = kMagic - 127.f, hi = kMagic + 127.f;
    const uint32_t qa = __float_as_uint(fminf(fmaxf(fmaf(a, inv, kMagic), lo), hi));
    const uint32_t qb = __float_as_uint(fminf(fmaxf(fmaf(b, inv, kMagic), lo), hi));
    const uint32_t qc = __float_as_uint(fminf(fmaxf(fmaf(c, inv, kMagic), lo), hi));
    const uint32_t qd = __float_as_uint(fminf(fmaxf(fmaf(d, inv, kMagic), lo), hi));
    const uint32_t ab = __byte_perm(qa, qb, 0x0040);  // bytes: a0 b0 . .
    const uint32_t cd = __byte_perm(qc, qd, 0x0040);
    return __byte_perm(ab, cd, 0x5410);               // a0 b0 c0 d0
}

// 16 fp16 values (two 16-byte loads) -> 16 int8 codes.
__device__ __forceinline__ uint4 quant16(const uint4& v0, const uint4& v1, float inv)
{
    const __half2* h0 = reinterpret_cast<const __half2*>(&v0);
    const __half2* h1 = reinterpret_cast<const __half2*>(&v1);
    float2 f[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        f[j] = __half22float2(h0[j]);
        f[4 + j] = __half22float2(h1[j]);
    }
    uint4 out;
    out.x = quant4(f[0].x, f[0].y, f[1].x, f[1].y, inv);
    out.y = quant4(f[2].x, f[2].y, f[3].x, f[3].y, inv);
    out.z = quant4(f[4].x, f[4].y, f[5].x, f[5].y, inv);
    out.w = quant4(f[6].x, f[6].y, f[7].x, f[7].y, inv);
    return out;
}

__device__ __forceinline__ void named_barrier_sync(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

template <int BN, int STAGES, bool W4, int AMODE>
__global__ void __launch_bounds__(kThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmap_w, const Params p)
{
    using L = SmemLayout<BN, STAGES, W4>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    uint8_t* sA = smem + L::OFF_A;
    uint8_t* sB = smem + L::OFF_B;
    uint8_t* sStg = smem + L::OFF_STG;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BARS);
    float* s_comb = reinterpret_cast<float*>(smem + L::OFF_COMB);
    float* s_bias = reinterpret_cast<float*>(smem + L::OFF_BIAS);
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + L::OFF_MISC);
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + L::OFF_MISC + 4);
    volatile int* s_last = reinterpret_cast<volatile int*>(smem + L::OFF_MISC + 8);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const int n0 = blockIdx.x * BN;
    const int m0 = blockIdx.y * BM;
    const int kb_begin = static_cast<int>((static_cast<long long>(p.k_blocks) * blockIdx.z) / gridDim.z);
    const int kb_end = static_cast<int>((static_cast<long long>(p.k_blocks) * (blockIdx.z + 1)) / gridDim.z);
    const int nkb = kb_end - kb_begin;

    const uint32_t bar_full_a = smem_u32(bars);
    const uint32_t bar_full_b = smem_u32(bars + STAGES);
    const uint32_t bar_empty = smem_u32(bars + 2 * STAGES);
    const uint32_t bar_accum = smem_u32(bars + 3 * STAGES);

    pdl_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full_a + 8 * s, kFeedWarps);
            mbar_init(bar_full_b + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_accum, 1);
        *s_abort = 0;
        *s_last = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmap_w);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(s_tmem), BN);
        tmem_relinquish();
    }
    pdl_wait();  // set-up above overlaps the previous kernel; global memory is touched only from here
    const float sx = __ldg(p.act_scale);
    if (tid >= 64) {
        // per-column epilogue factors of this tile
        for (int j = tid - 64; j < BN; j += kFeedThreads) {
            const int n = n0 + j;
            float comb = 0.f, b = 0.f;
            if (n < p.N && p.w_scale) {
                comb = sx * __ldg(p.w_scale + n);
                if (W4) comb *= 0.0625f;
                if (p.bias) b = __half2float(p.bias[n]);
            }
            s_comb[j] = comb;
            s_bias[j] = b;
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *s_tmem;

    if (warp == 0) {
        // ------------------------------------------------------------ weight producer
        if (lane == 0) {
            constexpr int ROW_BYTES = W4 ? BK / 2 : BK;
            for (int i = 0; i < nkb; ++i) {
                const int s = i % STAGES;
                const uint32_t round = static_cast<uint32_t>(i / STAGES);
                if (!mbar_wait(bar_empty + 8 * s, (round & 1) ^ 1, s_abort)) break;
                mbar_arrive_expect_tx(bar_full_b + 8 * s, BN * ROW_BYTES);
                const uint32_t dst = W4 ? smem_u32(sStg + s * L::STG_STAGE_BYTES)
                                        : smem_u32(sB + s * L::B_STAGE_BYTES);
                tma_load_2d(dst, &tmap_w, (kb_begin + i) * ROW_BYTES, n0, bar_full_b + 8 * s);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(2, 1, BM, BN);
            bool ok = true;
            for (int i = 0; i < nkb && ok; ++i) {
                const int s = i % STAGES;
                const uint32_t round = static_cast<uint32_t>(i / STAGES);
                ok = mbar_wait(bar_full_a + 8 * s, round & 1, s_abort);
                if (ok && !W4) ok = mbar_wait(bar_full_b + 8 * s, round & 1, s_abort);
                if (!ok) break;
                tc_fence_after_sync();
                const uint64_t a_desc = smem_desc_sw128(smem_u32(sA + s * A_STAGE_BYTES));
                const uint64_t b_desc = smem_desc_sw128(smem_u32(sB + s * L::B_STAGE_BYTES));
#pragma unroll
                for (int k = 0; k < BK / 32; ++k)  // 32 int8 per MMA = 32 bytes = 2 address units
                    mma_i8_ss(tmem_base, a_desc + 2 * k, b_desc + 2 * k, idesc, (i | k) != 0);
                tc_commit(bar_empty + 8 * s);
            }
            if (ok) tc_commit(bar_accum);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ A feeders, then epilogue
        const int ft = tid - 64;
        const int chunk = ft & 7;   // 16-element chunk inside the 128-wide k-block
        const int rbase = ft >> 3;  // rows rbase + 32 i, i = 0..3
        const float inv = __fdiv_rn(1.f, sx);

        long long row_off[4];
        int row_hi[4], row_wi[4];
        bool row_ok[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int m = m0 + rbase + 32 * i;
            row_ok[i] = m < p.M;
            row_hi[i] = row_wi[i] = 0;
            row_off[i] = 0;
            if (!row_ok[i]) continue;
            if (AMODE == A_LINEAR) {
                row_off[i] = static_cast<long long>(m) * p.ldx;
            } else if (AMODE == A_BOS) {
                const int prompt = m / (MIXDQ_TOKENS_PER_PROMPT - 1);
                const int t = m - prompt * (MIXDQ_TOKENS_PER_PROMPT - 1) + 1;
                row_off[i] = (static_cast<long long>(prompt) * MIXDQ_TOKENS_PER_PROMPT + t) * p.ldx;
            } else {
                const int hw = p.Ho * p.Wo;
                const int b = m / hw;
                const int rem = m - b * hw;
                const int ho = rem / p.Wo;
                const int wo = rem - ho * p.Wo;
                row_hi[i] = ho * p.stride - 1;
                row_wi[i] = wo * p.stride - 1;
                row_off[i] = static_cast<long long>(b) * p.H * p.W * p.Cin;
            }
        }

        if (AMODE == A_BOS && p.Y && blockIdx.y == 0 && blockIdx.z == 0) {
            // row 0 of every prompt: the stored floating-point BOS projection, copied as is
            for (int idx = ft; idx < p.batch * BN; idx += kFeedThreads) {
                const int b = idx / BN, j = idx - b * BN;
                if (n0 + j < p.N)
                    p.Y[static_cast<long long>(b) * MIXDQ_TOKENS_PER_PROMPT * p.ldy + n0 + j] =
                        p.bos_out[n0 + j];
            }
        }

        // position of this thread's chunk in the (kh, kw, cin) reduction order of a conv
        int tap = 0, ch = 0;
        if (AMODE == A_CONV3) {
            const int k0 = kb_begin * BK + chunk * 16;
            tap = k0 / p.Cin;
            ch = k0 - tap * p.Cin;
        }

        bool ok = true;
        for (int it = 0; it < nkb; ++it) {
            const int s = it % STAGES;
            const uint32_t round = static_cast<uint32_t>(it / STAGES);
            const int k0 = (kb_begin + it) * BK + chunk * 16;
            const bool k_ok = k0 < p.K;

            uint4 v[4][2];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const __half* src = nullptr;
                if (row_ok[i] && k_ok) {
                    if (AMODE == A_CONV3) {
                        const int kh = tap / 3, kw = tap - 3 * kh;
                        const int hi = row_hi[i] + kh, wi = row_wi[i] + kw;
                        if (hi >= 0 && hi < p.H && wi >= 0 && wi < p.W)
                            src = p.X + row_off[i] + (static_cast<long long>(hi) * p.W + wi) * p.Cin + ch;
                    } else {
                        src = p.X + row_off[i] + k0;
                    }
                }
                if (src) {
                    v[i][0] = __ldg(reinterpret_cast<const uint4*>(src));
                    v[i][1] = __ldg(reinterpret_cast<const uint4*>(src) + 1);
                } else {
                    v[i][0] = make_uint4(0, 0, 0, 0);
                    v[i][1] = make_uint4(0, 0, 0, 0);
                }
            }
            if (AMODE == A_CONV3) {
                ch += BK;
                while (ch >= p.Cin) {
                    ch -= p.Cin;
                    ++tap;
                }
            }

            ok = mbar_wait(bar_empty + 8 * s, (round & 1) ^ 1, s_abort);
            if (!ok) break;

            uint8_t* a_stage = sA + s * A_STAGE_BYTES;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int r = rbase + 32 * i;
                *reinterpret_cast<uint4*>(a_stage + sw128_offset(r, chunk)) = quant16(v[i][0], v[i][1], inv);
            }

            if (W4) {
                ok = mbar_wait(bar_full_b + 8 * s, round & 1, s_abort);
                if (!ok) break;
                const uint8_t* stg = sStg + s * L::STG_STAGE_BYTES;
                uint8_t* b_stage = sB + s * L::B_STAGE_BYTES;
#pragma unroll
                for (int t = 0; t < (BN * 4) / kFeedThreads; ++t) {
                    const int task = ft + t * kFeedThreads;
                    const int r = task >> 2, j = task & 3;
                    const uint4 w = *reinterpret_cast<const uint4*>(stg + r * (BK / 2) + j * 16);
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
            if (lane == 0) mbar_arrive(bar_full_a + 8 * s);
        }

        // ------------------------------------------------------------ epilogue
        if (ok && nkb > 0) ok = mbar_wait(bar_accum, 0, s_abort);
        tc_fence_after_sync();
        const int lg = warp & 3;           // tensor-memory lane group this warp may read
        const int half = (warp - 2) >> 2;  // which half of the tile's columns
        const int row = lg * 32 + lane;
        const int m = m0 + row;
        const bool m_ok = m < p.M;
        long long out_row = m;
        if (AMODE == A_BOS && m_ok) {
            const int prompt = m / (MIXDQ_TOKENS_PER_PROMPT - 1);
            out_row = static_cast<long long>(prompt) * MIXDQ_TOKENS_PER_PROMPT +
                      (m - prompt * (MIXDQ_TOKENS_PER_PROMPT - 1) + 1);
        }
        const bool split = gridDim.z > 1;
        int32_t* ws_acc = nullptr;
        if (split) {
            const long long n_pad = static_cast<long long>(gridDim.x) * BN;
            ws_acc = p.ws_acc + static_cast<long long>(m) * n_pad + n0;
        }

        // one decision per warp: the tensor-memory loads below must be executed by all 32 lanes
        const bool go = __all_sync(0xffffffffu, ok && !*s_abort);
        uint32_t r[32];
        if (split) {
            // add this CTA's partial sums to the int32 scratch tile (integer adds commute,
            // so the total does not depend on the order of arrival)
            if (go) {
                for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32) {
                    tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(lg * 32) << 16) + c0, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (r[j]) atomicAdd(ws_acc + c0 + j, static_cast<int32_t>(r[j]));
                }
            }
            __threadfence();
            named_barrier_sync(1, kFeedThreads);
            if (ft == 0) {
                const int tile = blockIdx.y * gridDim.x + blockIdx.x;
                const int ticket = atomicAdd(p.ws_tickets + tile, 1);
                const int last = ticket == static_cast<int>(gridDim.z) - 1;
                if (last) p.ws_tickets[tile] = 0;
                __threadfence();
                *s_last = last;
            }
            named_barrier_sync(1, kFeedThreads);
        }
        const bool do_out = !split || *s_last;
        if (do_out && go) {
            for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32) {
                if (split) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const int4 t = __ldcg(reinterpret_cast<const int4*>(ws_acc + c0 + j));
                        r[j] = t.x;
                        r[j + 1] = t.y;
                        r[j + 2] = t.z;
                        r[j + 3] = t.w;
                        *reinterpret_cast<int4*>(ws_acc + c0 + j) = make_int4(0, 0, 0, 0);
                    }
                } else {
                    tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(lg * 32) << 16) + c0, r);
                    tmem_ld_wait();
                }
                if (!m_ok) continue;
                const int n = n0 + c0;
                if (p.acc_out) {
                    int32_t* dst = p.acc_out + static_cast<long long>(m) * p.N + n;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (n + j < p.N) dst[j] = W4 ? (static_cast<int32_t>(r[j]) >> 4) : static_cast<int32_t>(r[j]);
                }
                if (p.Y) {
                    __half* dst = p.Y + out_row * p.ldy + n;
                    const bool vec = ((p.ldy & 7) == 0) && ((p.N & 7) == 0);
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        __half2 h[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const int c = c0 + j + 2 * q;
                            const float y0 = fmaf(static_cast<float>(static_cast<int32_t>(r[j + 2 * q])),
                                                  s_comb[c], s_bias[c]);
                            const float y1 = fmaf(static_cast<float>(static_cast<int32_t>(r[j + 2 * q + 1])),
                                                  s_comb[c + 1], s_bias[c + 1]);
                            h[q] = __floats2half2_rn(y0, y1);
                        }
                        if (vec && n + j + 8 <= p.N) {
                            *reinterpret_cast<uint4*>(dst + j) = *reinterpret_cast<const uint4*>(h);
                        } else {
                            const __half* hs = reinterpret_cast<const __half*>(h);
                            for (int q = 0; q < 8; ++q)
                                if (n + j + q < p.N) dst[j + q] = hs[q];
                        }
                    }
                }
            }
        }
    }

    if (*s_abort) {
        // give copies that may still be in flight time to land before shared memory goes away
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        if (tid == 0 && p.status) atomicExch(p.status, MIXDQ_ERR_TIMEOUT);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, BN);
}

// Plain kernel for shapes the tensor-core tiles do not cover (a reduction length or channel
// count that is not a multiple of 16, fewer than 16 output channels): one thread per output.
template <bool W4>
__global__ void simple_kernel(const uint8_t* __restrict__ packed, long long pitch, const Params p, int amode)
{
    pdl_launch_dependents();
    pdl_wait();
    const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    if (idx >= static_cast<long long>(p.M) * p.N) return;
    const int m = static_cast<int>(idx / p.N);
    const int n = static_cast<int>(idx - static_cast<long long>(m) * p.N);
    const float sx = __ldg(p.act_scale);
    const float inv = __fdiv_rn(1.f, sx);
    const uint8_t* wrow = packed + n * pitch;
    long long xoff = 0, out_row = m;
    int hi0 = 0, wi0 = 0;
    if (amode == A_LINEAR) {
        xoff = static_cast<long long>(m) * p.ldx;
    } else if (amode == A_BOS) {
        const int prompt = m / (MIXDQ_TOKENS_PER_PROMPT - 1);
        out_row = static_cast<long long>(prompt) * MIXDQ_TOKENS_PER_PROMPT +
                  (m - prompt * (MIXDQ_TOKENS_PER_PROMPT - 1) + 1);
        xoff = out_row * p.ldx;
    } else {
        const int hw = p.Ho * p.Wo;
        const int b = m / hw, rem = m - b * hw;
        const int ho = rem / p.Wo, wo = rem - ho * p.Wo;
        hi0 = ho * p.stride - 1;
        wi0 = wo * p.stride - 1;
        xoff = static_cast<long long>(b) * p.H * p.W * p.Cin;
    }
    int acc = 0;
    for (int k = 0; k < p.K; ++k) {
        float x;
        if (amode == A_CONV3) {
            const int tap = k / p.Cin, c = k - tap * p.Cin;
            const int hi = hi0 + tap / 3, wi = wi0 + tap % 3;
            if (hi < 0 || hi >= p.H || wi < 0 || wi >= p.W) continue;
            x = __half2float(p.X[xoff + (static_cast<long long>(hi) * p.W + wi) * p.Cin + c]);
        } else {
            x = __half2float(p.X[xoff + k]);
        }
        const float y = fminf(fmaxf(fmaf(x, inv, kMagic), kMagic - 127.f), kMagic + 127.f);
        const int qx = static_cast<int>(__float_as_uint(y)) - 0x4B400000;
        int qw;
        if (W4) {
            const int g = k >> 3, j = k & 7;
            const uint8_t b = wrow[4 * g + (j & 3)];
            const int nib = (j >= 4) ? (b >> 4) : (b & 0xf);
            qw = nib >= 8 ? nib - 16 : nib;
        } else {
            qw = static_cast<int8_t>(wrow[k]);
        }
        acc += qx * qw;
    }
    if (p.acc_out) p.acc_out[static_cast<long long>(m) * p.N + n] = acc;
    if (p.Y) {
        const float comb = sx * __ldg(p.w_scale + n);
        const float b = p.bias ? __half2float(p.bias[n]) : 0.f;
        p.Y[out_row * p.ldy + n] = __float2half_rn(fmaf(static_cast<float>(acc), comb, b));
    }
    if (amode == A_BOS && p.Y && m < p.batch)
        p.Y[static_cast<long long>(m) * MIXDQ_TOKENS_PER_PROMPT * p.ldy + n] = p.bos_out[n];
}

// Short reductions (K <= 64, int8 weights): the first convolution of the UNet has 4 input
// channels, i.e. K = 36.  A CTA quantizes the gathered inputs of 32 output rows into shared
// memory once; each thread then keeps one weight row in registers and produces that channel
// for all 32 rows with dp4a, so the stores of a row are contiguous across threads.
constexpr int kSmallKRows = 32;

__global__ void __launch_bounds__(128)
small_k_kernel(const uint8_t* __restrict__ packed, long long pitch, const Params p, int amode)
{
    __shared__ __align__(16) int8_t xq[kSmallKRows][64];
    pdl_launch_dependents();
    pdl_wait();
    const int tid = threadIdx.x;
    const int m0 = blockIdx.x * kSmallKRows;
    const float sx = __ldg(p.act_scale);
    const float inv = __fdiv_rn(1.f, sx);
    for (int idx = tid; idx < kSmallKRows * 64; idx += 128) {
        const int r = idx >> 6, k = idx & 63;
        const int m = m0 + r;
        int q = 0;
        if (m < p.M && k < p.K) {
            float x = 0.f;
            bool in = true;
            if (amode == A_CONV3) {
                const int hw = p.Ho * p.Wo;
                const int b = m / hw, rem = m - b * hw;
                const int ho = rem / p.Wo, wo = rem - ho * p.Wo;
                const int tap = k / p.Cin, c = k - tap * p.Cin;
                const int hi = ho * p.stride - 1 + tap / 3, wi = wo * p.stride - 1 + tap % 3;
                in = hi >= 0 && hi < p.H && wi >= 0 && wi < p.W;
                if (in) x = __half2float(p.X[((static_cast<long long>(b) * p.H + hi) * p.W + wi) * p.Cin + c]);
            } else {
                long long row = m;
                if (amode == A_BOS) {
                    const int prompt = m / (MIXDQ_TOKENS_PER_PROMPT - 1);
                    row = static_cast<long long>(prompt) * MIXDQ_TOKENS_PER_PROMPT +
                          (m - prompt * (MIXDQ_TOKENS_PER_PROMPT - 1) + 1);
                }
                x = __half2float(p.X[row * p.ldx + k]);
            }
            if (in) {
                const float y = fminf(fmaxf(fmaf(x, inv, kMagic), kMagic - 127.f), kMagic + 127.f);
                q = static_cast<int>(__float_as_uint(y)) - 0x4B400000;
            }
        }
        xq[r][k] = static_cast<int8_t>(q);
    }
    __syncthreads();
    const int words = (p.K + 3) >> 2;
    for (int n = tid; n < p.N; n += 128) {
        int w[16];
        const uint8_t* wrow = packed + static_cast<long long>(n) * pitch;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            w[j] = 0;
            if (j < words) {
                // bytes beyond K inside the last word are padding of the packed row (zero codes)
                const int byte0 = 4 * j;
                uint32_t v = 0;
                for (int b = 0; b < 4; ++b)
                    if (byte0 + b < p.K) v |= static_cast<uint32_t>(wrow[byte0 + b]) << (8 * b);
                w[j] = static_cast<int>(v);
            }
        }
        const float comb = p.w_scale ? sx * __ldg(p.w_scale + n) : 0.f;
        const float bias = p.bias ? __half2float(p.bias[n]) : 0.f;
        for (int r = 0; r < kSmallKRows; ++r) {
            const int m = m0 + r;
            if (m >= p.M) break;
            const int4* xr = reinterpret_cast<const int4*>(xq[r]);
            int acc = 0;
#pragma unroll
            for (int j4 = 0; j4 < 4; ++j4) {
                const int4 xv = xr[j4];
                acc = __dp4a(xv.x, w[4 * j4], acc);
                acc = __dp4a(xv.y, w[4 * j4 + 1], acc);
                acc = __dp4a(xv.z, w[4 * j4 + 2], acc);
                acc = __dp4a(xv.w, w[4 * j4 + 3], acc);
            }
            if (p.acc_out) p.acc_out[static_cast<long long>(m) * p.N + n] = acc;
            if (p.Y) {
                long long orow = m;
                if (amode == A_BOS) {
                    const int prompt = m / (MIXDQ_TOKENS_PER_PROMPT - 1);
                    orow = static_cast<long long>(prompt) * MIXDQ_TOKENS_PER_PROMPT +
                           (m - prompt * (MIXDQ_TOKENS_PER_PROMPT - 1) + 1);
                }
                p.Y[orow * p.ldy + n] = __float2half_rn(fmaf(static_cast<float>(acc), comb, bias));
            }
        }
        if (amode == A_BOS && p.Y && blockIdx.x == 0)
            for (int b = 0; b < p.batch; ++b)
                p.Y[static_cast<long long>(b) * MIXDQ_TOKENS_PER_PROMPT * p.ldy + n] = p.bos_out[n];
    }
}

template <int BN, int STAGES, bool W4, int AMODE>
int launch_tc(const Params& p, const void* packed, int64_t pitch, int splits, cudaStream_t stream)
{
    using L = SmemLayout<BN, STAGES, W4>;
    CUtensorMap tmap;
    int rc;
    if (W4)
        rc = encode_tmap_2d_u8(&tmap, packed, static_cast<uint64_t>(pitch), p.N, pitch, BK / 2, BN, false);
    else
        rc = encode_tmap_2d_u8(&tmap, packed, static_cast<uint64_t>(p.K), p.N, pitch, BK, BN, true);
    if (rc != MIXDQ_OK) return rc;
    auto kernel = gemm_kernel<BN, STAGES, W4, AMODE>;
    if (ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), L::TOTAL) != MIXDQ_OK) return MIXDQ_ERR_CUDA;
    dim3 grid(static_cast<unsigned>(ceil_div(p.N, BN)), static_cast<unsigned>(ceil_div(p.M, BM)),
              static_cast<unsigned>(splits));
    return launch_pdl(kernel, grid, dim3(kThreads), L::TOTAL, stream, 1, tmap, p);
}

template <bool W4, int AMODE>
int launch_mode(const Params& p, const void* packed, int64_t pitch, int splits, cudaStream_t stream)
{
    return launch_tc<128, 4, W4, AMODE>(p, packed, pitch, splits, stream);
}

size_t split_scratch_bytes(int64_t rows, int64_t N)
{
    const int64_t tiles = ceil_div(rows, BM) * ceil_div(N, 128);
    return static_cast<size_t>(round_up(tiles * 4, 256) + round_up(rows, BM) * round_up(N, 128) * 4);
}

size_t workspace_bytes(int64_t out_rows, int64_t N, int64_t in_rows, int64_t row_len)
{
    return split_scratch_bytes(out_rows, N) + tma_scratch_bytes(in_rows, row_len);
}

int run(Params p, int amode, const void* packed, int w_bits, void* workspace, size_t ws_bytes,
        cudaStream_t stream)
{
    const bool w4 = w_bits == 4;
    const int64_t pitch = row_pitch_bytes(p.K, w_bits, MIXDQ_LAYOUT_DEVICE);
    p.k_blocks = static_cast<int>(ceil_div(p.K, BK));
    const bool tc_ok = (amode == A_CONV3 ? (p.Cin % 16 == 0) : (p.K % 16 == 0)) && p.N >= 16 &&
                       (p.ldx % 8 == 0) && ((reinterpret_cast<uintptr_t>(p.X) & 15) == 0);

    // two-kernel path: needs room for the int8 activations behind the split-reduction scratch
    const size_t split_bytes = split_scratch_bytes(p.M, p.N);
    // an asymmetric convolution input is kept with its one-pixel border
    const int pad = (amode == A_CONV3 && p.act_zero) ? 2 : 0;
    const int64_t in_rows = amode == A_CONV3 ? static_cast<int64_t>(p.batch) * (p.H + pad) * (p.W + pad) : p.M;
    const int64_t row_len = amode == A_CONV3 ? p.Cin : p.K;
    const bool tma_room = workspace && ws_bytes >= split_bytes + tma_scratch_bytes(in_rows, row_len);
    if (p.act_zero) {
        // asymmetric activations exist in the two-kernel form only
        if (amode == A_BOS || !p.w_code_sums || !tma_room || !tma_path_ok(p, amode, w_bits)) return MIXDQ_ERR_UNSUPPORTED;
        return run_tma(p, amode, packed, w_bits, static_cast<uint8_t*>(workspace) + split_bytes, stream);
    }
    if (tma_room && tma_path_ok(p, amode, w_bits))
        return run_tma(p, amode, packed, w_bits, static_cast<uint8_t*>(workspace) + split_bytes, stream);

    if (!tc_ok && !w4 && p.K <= 64) {
        const unsigned grid = static_cast<unsigned>(ceil_div(p.M, kSmallKRows));
        const long long pitch_ll = pitch;
        return launch_pdl(small_k_kernel, dim3(grid), dim3(128), 0, stream, 1, static_cast<const uint8_t*>(packed),
                          pitch_ll, p, amode);
    }
    if (!tc_ok) {
        const long long total = static_cast<long long>(p.M) * p.N;
        const unsigned grid = static_cast<unsigned>(ceil_div(total, 128));
        const long long pitch_ll = pitch;
        if (w4)
            return launch_pdl(simple_kernel<true>, dim3(grid), dim3(128), 0, stream, 1,
                              static_cast<const uint8_t*>(packed), pitch_ll, p, amode);
        return launch_pdl(simple_kernel<false>, dim3(grid), dim3(128), 0, stream, 1,
                          static_cast<const uint8_t*>(packed), pitch_ll, p, amode);
    }
    // split the reduction across CTAs when the output tiles alone cannot fill the GPU
    const int64_t tiles = ceil_div(p.M, BM) * ceil_div(p.N, 128);
    int splits = 1;
    const bool split_room = workspace && ws_bytes >= split_bytes;
    const int num_sms = sm_count();
    if (num_sms <= 0) return MIXDQ_ERR_CUDA;
    if (split_room && tiles < 96 && p.k_blocks >= 8) {
        splits = static_cast<int>(num_sms / tiles);
        if (splits > p.k_blocks / 4) splits = p.k_blocks / 4;
        if (splits < 1) splits = 1;
    }
    if (splits > 1) {
        // a workspace shared between layers may hold another layer's int8 activations here, so the
        // counters and partial sums of the split reduction are cleared, not assumed zero
        uint8_t* region = static_cast<uint8_t*>(workspace);
        MIXDQ_CUDA_TRY(cudaMemsetAsync(region, 0, split_bytes, stream));
        p.ws_tickets = reinterpret_cast<int32_t*>(region);
        p.ws_acc = reinterpret_cast<int32_t*>(region + round_up(tiles * 4, 256));
    }
#define MIXDQ_DISPATCH(W4V)                                                                    \
    switch (amode) {                                                                           \
        case A_LINEAR: return launch_mode<W4V, A_LINEAR>(p, packed, pitch, splits, stream);    \
        case A_BOS: return launch_mode<W4V, A_BOS>(p, packed, pitch, splits, stream);          \
        case A_CONV3: return launch_mode<W4V, A_CONV3>(p, packed, pitch, splits, stream);      \
        default: return MIXDQ_ERR_INVALID_ARG;                                                 \
    }
    if (w4) {
        MIXDQ_DISPATCH(true)
    } else {
        MIXDQ_DISPATCH(false)
    }
#undef MIXDQ_DISPATCH
}

}  // namespace i8
}  // namespace mixdq
