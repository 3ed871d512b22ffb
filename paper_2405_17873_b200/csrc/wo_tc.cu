// Weight-only engine for many tokens (W3 / W4 / W8 with fp16 activations, M >= 64): the
// layer is then bound by the fp16 tensor pipe and by on-chip bandwidth, not by the weight
// stream, so it runs on tcgen05.mma kind::f16 with fp32 accumulators in tensor memory.
//   warp 0      TMA producer: fp16 activation tiles (128 rows x 64 k), 128-byte swizzle; a 3x3
//               convolution reads a 4-D box of the NHWC image shifted by the filter tap
//   warp 1      tensor-memory owner and MMA issuer (128 x 128 x 16 per instruction)
//   warps 2..9  epilogue: tensor memory -> registers -> y = fp16(scale[n] * acc + bias[n])
//   warps 10..17 weight feeders: packed codes straight from global memory into registers,
//               expanded to the exact fp16 integers (q - z) and written as the swizzled
//               K-major B tile
// One CTA per SM walks over output tiles; two accumulators alternate so that the epilogue of
// a tile overlaps the main loop of the next.
#include "common.cuh"
#include "engines.h"

namespace mixdq {
namespace wo {

namespace {

constexpr int BM = 128;
constexpr int BN = 128;
constexpr int BKE = 64;  // fp16 elements per k-block = one 128-byte swizzled row
constexpr int STAGES = 6;
constexpr int A_BYTES = BM * 128;
constexpr int B_BYTES = BN * 128;
constexpr int OFF_A = 0;
constexpr int OFF_B = STAGES * A_BYTES;
constexpr int OFF_BARS = OFF_B + STAGES * B_BYTES;
constexpr int NUM_BARS = 3 * STAGES + 4;
constexpr int OFF_COMB = (OFF_BARS + NUM_BARS * 8 + 15) & ~15;  // [2][BN] scales
constexpr int OFF_BIAS = OFF_COMB + 2 * BN * 4;                 // [2][BN] biases
constexpr int OFF_MISC = OFF_BIAS + 2 * BN * 4;
constexpr int OFF_EPI = OFF_MISC + 64;  // per epilogue warp: 32 rows x 32 fp16, rows 80 bytes apart
constexpr int EPI_ROW = 80;
constexpr int EPI_WARP_BYTES = 32 * EPI_ROW;
constexpr int SMEM_TOTAL = OFF_EPI + 8 * EPI_WARP_BYTES + 1024;
constexpr int THREADS = 576;
constexpr int kFeedWarps = 8;

struct TcParams {
    int M, N, K, k_blocks;
    int conv, cblocks, Cin, HoWo, Wo;
    const float* w_scale;
    const int32_t* w_zero;
    const __half* bias;
    __half* Y;
    long long ldy;
    int32_t* status;
    const uint8_t* packed;
    long long pitch;
};

__device__ __forceinline__ uint32_t h2u(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ __forceinline__ __half2 u2h(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }

// Eight 4-bit (FIELD = 0xF) or 3-bit (0x7) fields of a device-layout word -> (q - z) as eight
// fp16 values in reduction order.  Field n holds code n/2 (n even) or 4 + n/2 (n odd).
template <uint32_t FIELD>
__device__ __forceinline__ uint4 decode_word(uint32_t w, __half2 z_lo, __half2 z_hi)
{
    constexpr uint32_t MLO = FIELD * 0x00010001u, MHI = MLO << 4, MAGIC = 0x64006400u;
    const uint32_t w8 = w >> 8;
    const __half2 sixteenth = __float2half2_rn(0.0625f);
    const uint32_t c02 = h2u(__hsub2(u2h((w & MLO) | MAGIC), z_lo));
    const uint32_t c13 = h2u(__hsub2(u2h((w8 & MLO) | MAGIC), z_lo));
    const uint32_t c46 = h2u(__hfma2(u2h((w & MHI) | MAGIC), sixteenth, z_hi));
    const uint32_t c57 = h2u(__hfma2(u2h((w8 & MHI) | MAGIC), sixteenth, z_hi));
    return make_uint4(__byte_perm(c02, c13, 0x5410), __byte_perm(c02, c13, 0x7632),
                      __byte_perm(c46, c57, 0x5410), __byte_perm(c46, c57, 0x7632));
}

// Packed words of 32 consecutive codes of one row.
template <int BITS>
struct Codes32 {
    static constexpr int WORDS = BITS == 8 ? 8 : (BITS == 4 ? 4 : 3);
    uint32_t w[WORDS];
};

// k32: index of the 32-code run inside the row (reduction index / 32).
template <int BITS>
__device__ __forceinline__ void load_codes32(Codes32<BITS>& c, const uint8_t* __restrict__ row, long long pitch, int k32,
                                             bool ok)
{
#pragma unroll
    for (int i = 0; i < Codes32<BITS>::WORDS; ++i) c.w[i] = 0;
    if (!ok) return;
    if (BITS == 4) {
        const long long off = static_cast<long long>(k32) * 16;
        if (off < pitch) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(row + off));
            c.w[0] = v.x; c.w[1] = v.y; c.w[2] = v.z; c.w[3] = v.w;
        }
    } else if (BITS == 8) {
        const long long off = static_cast<long long>(k32) * 32;
        if (off < pitch) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(row + off));
            c.w[0] = v.x; c.w[1] = v.y; c.w[2] = v.z; c.w[3] = v.w;
        }
        if (off + 16 < pitch) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(row + off + 16));
            c.w[4] = v.x; c.w[5] = v.y; c.w[6] = v.z; c.w[7] = v.w;
        }
    } else {
        // 128-code blocks of three 16-byte planes; word (k32 % 4) of each plane holds this run
        // (two planes for 2-bit codes: the decode reads the absent top plane as zeros)
        const long long off = static_cast<long long>(k32 >> 2) * (16 * BITS) + (k32 & 3) * 4;
        if (off < pitch) {
#pragma unroll
            for (int p = 0; p < BITS; ++p) c.w[p] = __ldg(reinterpret_cast<const uint32_t*>(row + off + 16 * p));
        }
    }
}

// Eight fp16 values (q - z) of codes 8 s .. 8 s + 7 of the run.
template <int BITS, bool SIGNED>
__device__ __forceinline__ uint4 decode8(const Codes32<BITS>& c, int s, __half2 z_lo, __half2 z_hi)
{
    if (BITS == 4) {
        uint32_t w = c.w[s];
        if (SIGNED) w ^= 0x88888888u;
        return decode_word<0xFu>(w, z_lo, z_hi);
    } else if (BITS <= 3) {
        const uint32_t a = c.w[0] >> s;
        const uint32_t b = (s == 0) ? (c.w[1] << 1) : (c.w[1] >> (s - 1));
        const uint32_t d = (s <= 1) ? (c.w[2] << (2 - s)) : (c.w[2] >> (s - 2));
        const uint32_t ab = (a & 0x11111111u) | (b & ~0x11111111u);
        return decode_word<0x7u>((ab & 0x33333333u) | (d & ~0x33333333u), z_lo, z_hi);
    } else {
        uint32_t w0 = c.w[2 * s], w1 = c.w[2 * s + 1];
        if (SIGNED) {
            w0 ^= 0x80808080u;
            w1 ^= 0x80808080u;
        }
        return make_uint4(h2u(__hsub2(u2h(__byte_perm(w0, 0x64646464u, 0x4140)), z_lo)),
                          h2u(__hsub2(u2h(__byte_perm(w0, 0x64646464u, 0x4342)), z_lo)),
                          h2u(__hsub2(u2h(__byte_perm(w1, 0x64646464u, 0x4140)), z_lo)),
                          h2u(__hsub2(u2h(__byte_perm(w1, 0x64646464u, 0x4342)), z_lo)));
    }
}

template <int BITS, bool SIGNED>
__global__ void __launch_bounds__(THREADS, 1)
wo_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const TcParams p, int n_tiles, int total_tiles)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    uint8_t* sA = smem + OFF_A;
    uint8_t* sB = smem + OFF_B;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BARS);
    float* s_comb = reinterpret_cast<float*>(smem + OFF_COMB);
    float* s_bias = reinterpret_cast<float*>(smem + OFF_BIAS);
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + OFF_MISC);
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + OFF_MISC + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nkb = p.k_blocks;
    const int my_tiles = (total_tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) /
                         static_cast<int>(gridDim.x);

    const uint32_t bar_full_a = smem_u32(bars);
    const uint32_t bar_full_b = smem_u32(bars + STAGES);
    const uint32_t bar_empty = smem_u32(bars + 2 * STAGES);
    const uint32_t bar_acc_full = smem_u32(bars + 3 * STAGES);
    const uint32_t bar_acc_empty = smem_u32(bars + 3 * STAGES + 2);

    pdl_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full_a + 8 * s, 1);
            mbar_init(bar_full_b + 8 * s, kFeedWarps);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_acc_full + 8 * b, 1);
            mbar_init(bar_acc_empty + 8 * b, 8);
        }
        *s_abort = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmap_x);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(s_tmem), 2 * BN);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_wait();
    const uint32_t tmem_base = *s_tmem;

    if (warp == 0) {
        // ------------------------------------------------------------ activation producer
        if (lane == 0) {
            int it = 0;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int tile = blockIdx.x + t * gridDim.x;
                const int m0 = (tile / n_tiles) * BM;
                int img_b = 0, ho0 = 0, wo0 = 0;
                if (p.conv) {
                    img_b = m0 / p.HoWo;
                    const int rem = m0 - img_b * p.HoWo;
                    ho0 = rem / p.Wo;
                    wo0 = rem - ho0 * p.Wo;
                }
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t round = static_cast<uint32_t>(it / STAGES);
                    ok = mbar_wait(bar_empty + 8 * s, (round & 1) ^ 1, s_abort);
                    if (!ok) break;
                    mbar_arrive_expect_tx(bar_full_a + 8 * s, A_BYTES);
                    const uint32_t dst = smem_u32(sA + s * A_BYTES);
                    if (p.conv) {
                        const int tap = kb / p.cblocks, cb = kb - tap * p.cblocks;
                        const int kh = tap / 3, kw = tap - 3 * kh;
                        tma_load_4d(dst, &tmap_x, cb * BKE, wo0 + kw - 1, ho0 + kh - 1, img_b, bar_full_a + 8 * s);
                    } else {
                        tma_load_2d(dst, &tmap_x, kb * BKE, m0, bar_full_a + 8 * s);
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(1, 0, BM, BN);
            int it = 0;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int buf = t & 1;
                const uint32_t use = static_cast<uint32_t>(t >> 1);
                ok = mbar_wait(bar_acc_empty + 8 * buf, (use & 1) ^ 1, s_abort);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t acc = tmem_base + buf * BN;
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t round = static_cast<uint32_t>(it / STAGES);
                    ok = mbar_wait(bar_full_a + 8 * s, round & 1, s_abort);
                    if (ok) ok = mbar_wait(bar_full_b + 8 * s, round & 1, s_abort);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint64_t a_desc = smem_desc_sw128(smem_u32(sA + s * A_BYTES));
                    const uint64_t b_desc = smem_desc_sw128(smem_u32(sB + s * B_BYTES));
#pragma unroll
                    for (int k = 0; k < BKE / 16; ++k)  // 16 fp16 per MMA = 32 bytes = 2 address units
                        mma_f16_ss(acc, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0);
                    tc_commit(bar_empty + 8 * s);
                }
                if (ok) tc_commit(bar_acc_full + 8 * buf);
            }
        }
        __syncwarp();
    } else if (warp < 10) {
        // ------------------------------------------------------------ epilogue
        const int lg = warp & 3;
        const int chalf = (warp - 2) >> 2;  // which half of the tile's columns this warp handles
        const int et = tid - 64;
        const bool vec = ((p.ldy & 7) == 0) && ((p.N & 7) == 0);
        bool ok = true;
        for (int t = 0; t < my_tiles; ++t) {
            const int tile = blockIdx.x + t * gridDim.x;
            const int m0 = (tile / n_tiles) * BM, n0 = (tile % n_tiles) * BN;
            const int buf = t & 1;
            const uint32_t use = static_cast<uint32_t>(t >> 1);
            float* comb = s_comb + buf * BN;
            float* bias = s_bias + buf * BN;
            if (et < BN) {
                const int n = n0 + et;
                comb[et] = n < p.N ? __ldg(p.w_scale + n) : 0.f;
                bias[et] = (n < p.N && p.bias) ? __half2float(p.bias[n]) : 0.f;
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (ok) ok = mbar_wait(bar_acc_full + 8 * buf, use & 1, s_abort);
            tc_fence_after_sync();
            const bool go = __all_sync(0xffffffffu, ok && !*s_abort);
            if (!go) {
                ok = false;
                continue;
            }
            const uint32_t acc = tmem_base + buf * BN + (static_cast<uint32_t>(lg * 32) << 16);
            // 32 columns at a time: scale in registers (one row per thread), pass through a small
            // shared-memory tile, and store with four lanes along each row so that every store
            // instruction writes whole 32-byte sectors of eight rows
            uint8_t* stage = smem + OFF_EPI + (warp - 2) * EPI_WARP_BYTES;
            const int row_base = m0 + lg * 32;
            for (int c0 = chalf * (BN / 2); c0 < (chalf + 1) * (BN / 2); c0 += 32) {
                if (n0 + c0 >= p.N) break;  // uniform across the warp
                uint32_t r[32];
                tmem_ld_32x32(acc + c0, r);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; j += 8) {
                    const int c = c0 + j;
                    const float4 ca = *reinterpret_cast<const float4*>(comb + c);
                    const float4 cb = *reinterpret_cast<const float4*>(comb + c + 4);
                    const float4 ba = *reinterpret_cast<const float4*>(bias + c);
                    const float4 bb = *reinterpret_cast<const float4*>(bias + c + 4);
                    uint4 o;
                    o.x = h2u(__floats2half2_rn(fmaf(__uint_as_float(r[j]), ca.x, ba.x),
                                                fmaf(__uint_as_float(r[j + 1]), ca.y, ba.y)));
                    o.y = h2u(__floats2half2_rn(fmaf(__uint_as_float(r[j + 2]), ca.z, ba.z),
                                                fmaf(__uint_as_float(r[j + 3]), ca.w, ba.w)));
                    o.z = h2u(__floats2half2_rn(fmaf(__uint_as_float(r[j + 4]), cb.x, bb.x),
                                                fmaf(__uint_as_float(r[j + 5]), cb.y, bb.y)));
                    o.w = h2u(__floats2half2_rn(fmaf(__uint_as_float(r[j + 6]), cb.z, bb.z),
                                                fmaf(__uint_as_float(r[j + 7]), cb.w, bb.w)));
                    *reinterpret_cast<uint4*>(stage + lane * EPI_ROW + j * 2) = o;
                }
                __syncwarp();
                const int seg = lane & 3;
                const int n = n0 + c0 + seg * 8;
#pragma unroll
                for (int it4 = 0; it4 < 4; ++it4) {
                    const int rl = it4 * 8 + (lane >> 2);
                    const int mm = row_base + rl;
                    if (mm >= p.M || n >= p.N) continue;
                    const uint4 v = *reinterpret_cast<const uint4*>(stage + rl * EPI_ROW + seg * 16);
                    __half* dst = p.Y + static_cast<long long>(mm) * p.ldy + n;
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
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acc_empty + 8 * buf);
        }
    } else {
        // ------------------------------------------------------------ weight feeders
        // thread -> (row of the tile, which 32-code half of the 64-wide k-block)
        const int ft = tid - 320;
        const int half = ft & 1;
        const int r = ft >> 1;
        int it = 0;
        bool ok = true;
        for (int t = 0; t < my_tiles && ok; ++t) {
            const int tile = blockIdx.x + t * gridDim.x;
            const int n = (tile % n_tiles) * BN + r;
            const bool row_ok = n < p.N;
            const uint8_t* row = p.packed + static_cast<long long>(row_ok ? n : 0) * p.pitch;
            float z = SIGNED ? (BITS == 8 ? 128.f : 8.f) : 0.f;
            if (!SIGNED && p.w_zero && row_ok) z = static_cast<float>(__ldg(p.w_zero + n));
            const __half2 z_lo = __float2half2_rn(1024.f + z), z_hi = __float2half2_rn(-(64.f + z));
            // reduction index (in 32-code runs) of k-block kb: conv k-blocks restart per filter tap
            auto k32_of = [&](int kb) {
                if (p.conv) {
                    const int tap = kb / p.cblocks, cb = kb - tap * p.cblocks;
                    return (tap * p.Cin + cb * BKE) / 32 + half;
                }
                return kb * 2 + half;
            };
            // packed words two k-blocks ahead of the one being expanded
            Codes32<BITS> c0, c1, c2;
            load_codes32<BITS>(c0, row, p.pitch, k32_of(0), row_ok);
            load_codes32<BITS>(c1, row, p.pitch, k32_of(nkb > 1 ? 1 : 0), row_ok && nkb > 1);
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const int s = it % STAGES;
                const uint32_t round = static_cast<uint32_t>(it / STAGES);
                load_codes32<BITS>(c2, row, p.pitch, k32_of(kb + 2 < nkb ? kb + 2 : 0), row_ok && kb + 2 < nkb);
                ok = mbar_wait(bar_empty + 8 * s, (round & 1) ^ 1, s_abort);
                if (!ok) break;
                uint8_t* b_stage = sB + s * B_BYTES;
#pragma unroll
                for (int sub = 0; sub < 4; ++sub)
                    *reinterpret_cast<uint4*>(b_stage + sw128_offset(r, 4 * half + sub)) =
                        decode8<BITS, SIGNED>(c0, sub, z_lo, z_hi);
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_full_b + 8 * s);
                c0 = c1;
                c1 = c2;
            }
        }
    }

    if (*s_abort) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        if (tid == 0 && p.status) atomicExch(p.status, MIXDQ_ERR_TIMEOUT);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, 2 * BN);
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

template <int BITS, bool SIGNED>
int launch_tc(const CUtensorMap& tx, const TcParams& tp, cudaStream_t stream)
{
    auto kernel = wo_tc_kernel<BITS, SIGNED>;
    if (ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), SMEM_TOTAL) != MIXDQ_OK) return MIXDQ_ERR_CUDA;
    const int num_sms = sm_count();
    if (num_sms <= 0) return MIXDQ_ERR_CUDA;
    const int n_tiles = static_cast<int>(ceil_div(tp.N, BN));
    const int total = n_tiles * static_cast<int>(ceil_div(tp.M, BM));
    const dim3 grid(static_cast<unsigned>(total < num_sms ? total : num_sms));
    return launch_pdl(kernel, grid, dim3(THREADS), SMEM_TOTAL, stream, 1, tx, tp, n_tiles, total);
}

}  // namespace

bool tc_path_ok(const Params& p, int amode, int w_bits)
{
    if (p.M < 64) return false;
    if (amode == A_CONV3) {
        int a, b, c;
        // whole 32-code runs per k-block: channel count a multiple of 64
        if (p.stride != 1 || p.Cin % 64 != 0) return false;
        return conv_box(p.Ho, p.Wo, &a, &b, &c);
    }
    (void)w_bits;
    return amode == A_LINEAR && p.K % 8 == 0 && p.ldx % 8 == 0 && (reinterpret_cast<uintptr_t>(p.X) & 15) == 0;
}

int run_tc(const Params& p, int amode, const void* packed, int w_bits, int batch, cudaStream_t stream)
{
    TcParams tp{};
    tp.M = p.M;
    tp.N = p.N;
    tp.K = p.K;
    tp.w_scale = p.w_scale;
    tp.w_zero = p.w_zero;
    tp.bias = p.bias;
    tp.Y = p.Y;
    tp.ldy = p.ldy;
    tp.status = p.status;
    tp.packed = static_cast<const uint8_t*>(packed);
    tp.pitch = row_pitch_bytes(p.K, w_bits, MIXDQ_LAYOUT_DEVICE);
    CUtensorMap tx;
    int rc;
    if (amode == A_CONV3) {
        int Wb, Hb, Bb;
        if (!conv_box(p.Ho, p.Wo, &Wb, &Hb, &Bb)) return MIXDQ_ERR_UNSUPPORTED;
        const uint64_t dims[4] = {static_cast<uint64_t>(p.Cin), static_cast<uint64_t>(p.W),
                                  static_cast<uint64_t>(p.H), static_cast<uint64_t>(batch)};
        const uint64_t strides[3] = {static_cast<uint64_t>(p.Cin) * 2, static_cast<uint64_t>(p.Cin) * p.W * 2,
                                     static_cast<uint64_t>(p.Cin) * p.W * p.H * 2};
        const uint32_t box[4] = {BKE, static_cast<uint32_t>(Wb), static_cast<uint32_t>(Hb), static_cast<uint32_t>(Bb)};
        rc = encode_tmap_4d_f16(&tx, p.X, dims, strides, box);
        tp.conv = 1;
        tp.cblocks = p.Cin / BKE;
        tp.Cin = p.Cin;
        tp.HoWo = p.Ho * p.Wo;
        tp.Wo = p.Wo;
        tp.k_blocks = 9 * tp.cblocks;
    } else {
        rc = encode_tmap_2d_f16(&tx, p.X, static_cast<uint64_t>(p.K), static_cast<uint64_t>(p.M),
                                static_cast<uint64_t>(p.ldx), BKE, BM);
        tp.k_blocks = static_cast<int>(ceil_div(p.K, BKE));
    }
    if (rc != MIXDQ_OK) return rc;
    const bool is_signed = p.w_zero == nullptr;
    if (w_bits == 3) return is_signed ? MIXDQ_ERR_UNSUPPORTED : launch_tc<3, false>(tx, tp, stream);
    if (w_bits == 2) return is_signed ? MIXDQ_ERR_UNSUPPORTED : launch_tc<2, false>(tx, tp, stream);
    if (w_bits == 4) return is_signed ? launch_tc<4, true>(tx, tp, stream) : launch_tc<4, false>(tx, tp, stream);
    if (w_bits == 8) return is_signed ? launch_tc<8, true>(tx, tp, stream) : launch_tc<8, false>(tx, tp, stream);
    return MIXDQ_ERR_UNSUPPORTED;
}

}  // namespace wo
}  // namespace mixdq
