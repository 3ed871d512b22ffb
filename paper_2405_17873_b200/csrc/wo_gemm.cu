// Weight-only engine (W3 / W4 / W8 with fp16 activations): the packed weights are streamed
// from memory once, expanded to fp16 integers (q - z) in registers and multiplied with the
// fp16 activations on the tensor cores (mma.sync m16n8k16, fp32 accumulate); the per-channel
// scale and the bias are applied to the fp32 sums.  Keeping (q - z) an exact small integer
// in fp16 means the weights add no rounding error of their own.
//
// The weights are the M-side operand of the MMA (16 output channels per tile) and the
// tokens the N-side (8 per tile), so that a packed row is read by the four threads of a
// quad as one contiguous run and never passes through shared memory.  The activations of
// the CTA's token block are staged in shared memory once, in the order in which the
// register decode produces the weights.
//
// CTA = 8 warps = 2 channel tiles x 4 slices of the reduction; slices are summed through
// shared memory before the epilogue.
#include "common.cuh"
#include "engines.h"

namespace mixdq {
namespace wo {

constexpr int kThreads = 256;
constexpr int kTilesPerCta = 2;
constexpr int kSlices = 4;
constexpr int kChanPerCta = 16 * kTilesPerCta;
constexpr int kUnit = 128;       // reduction elements per unit: 32 codes per thread of a quad
constexpr int kChunkMax = 2048;  // reduction elements staged in shared memory at a time
constexpr int kSmallKMax = 5120; // longest reduction the small-token kernel keeps in shared memory

__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ int round_up_dev(int v) { return (v + kUnit - 1) / kUnit * kUnit; }

__device__ __forceinline__ uint32_t h2u(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ __forceinline__ __half2 u2h(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }

// Eight 4-bit (or 3-bit) fields of a device-layout word -> (q - z) as four half2.
// Field n of the word holds code n/2 (n even) or 4 + n/2 (n odd).  Output pairs:
// out[0] = (c0, c2), out[1] = (c1, c3), out[2] = (c4, c6), out[3] = (c5, c7).
template <uint32_t FIELD>
__device__ __forceinline__ void decode_fields(uint32_t w, __half2 z_lo, __half2 z_hi, uint32_t (&out)[4])
{
    constexpr uint32_t MLO = FIELD * 0x00010001u;
    constexpr uint32_t MHI = MLO << 4;
    constexpr uint32_t MAGIC = 0x64006400u;  // fp16 1024: the field lands in the low mantissa bits
    const uint32_t w8 = w >> 8;
    const __half2 sixteenth = __float2half2_rn(0.0625f);
    out[0] = h2u(__hsub2(u2h((w & MLO) | MAGIC), z_lo));
    out[1] = h2u(__hsub2(u2h((w8 & MLO) | MAGIC), z_lo));
    out[2] = h2u(__hfma2(u2h((w & MHI) | MAGIC), sixteenth, z_hi));
    out[3] = h2u(__hfma2(u2h((w8 & MHI) | MAGIC), sixteenth, z_hi));
}

// Packed weights of one unit (32 codes) of one row, as loaded by one thread.
template <int BITS>
struct UnitRegs {
    static constexpr int WORDS = BITS == 8 ? 8 : (BITS == 4 ? 4 : 3);
    uint32_t w[WORDS];
};

template <int BITS>
__device__ __forceinline__ void load_unit(UnitRegs<BITS>& u, const uint8_t* __restrict__ row, long long pitch,
                                          int unit, int t, bool row_ok)
{
#pragma unroll
    for (int i = 0; i < UnitRegs<BITS>::WORDS; ++i) u.w[i] = 0;
    if (!row_ok) return;
    if (BITS == 4) {
        const long long off = static_cast<long long>(unit) * 64 + t * 16;
        if (off < pitch) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(row + off));
            u.w[0] = v.x; u.w[1] = v.y; u.w[2] = v.z; u.w[3] = v.w;
        }
    } else if (BITS == 8) {
        const long long off = static_cast<long long>(unit) * 128 + t * 32;
        if (off < pitch) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(row + off));
            u.w[0] = v.x; u.w[1] = v.y; u.w[2] = v.z; u.w[3] = v.w;
        }
        if (off + 16 < pitch) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(row + off + 16));
            u.w[4] = v.x; u.w[5] = v.y; u.w[6] = v.z; u.w[7] = v.w;
        }
    } else {
        // bit-planes (3 or 2 of them; the decode reads an absent top plane as zeros)
        const long long off = static_cast<long long>(unit) * (16 * BITS) + t * 4;
        if (off < pitch) {
#pragma unroll
            for (int p = 0; p < BITS; ++p) u.w[p] = __ldg(reinterpret_cast<const uint32_t*>(row + off + 16 * p));
        }
    }
}

// Expand sub-step s (8 codes) of a unit into the A-fragment halves of two MMAs:
// f[0], f[1] feed the first MMA (k columns 2t.. and 2t+8..), f[2], f[3] the second.
template <int BITS, bool SIGNED>
__device__ __forceinline__ void decode_substep(const UnitRegs<BITS>& u, int s, __half2 z_lo, __half2 z_hi,
                                               uint32_t (&f)[4])
{
    if (BITS == 4) {
        uint32_t w = u.w[s];
        if (SIGNED) w ^= 0x88888888u;
        decode_fields<0xFu>(w, z_lo, z_hi, f);
    } else if (BITS <= 3) {
        // bit 4n + s of plane p is bit p of field n of sub-step s: gather the three planes
        // into one word of 4-bit-spaced fields (bit 3 of each field is ignored by the mask)
        const uint32_t a = u.w[0] >> s;
        const uint32_t b = (s == 0) ? (u.w[1] << 1) : (u.w[1] >> (s - 1));
        const uint32_t c = (s <= 1) ? (u.w[2] << (2 - s)) : (u.w[2] >> (s - 2));
        const uint32_t ab = (a & 0x11111111u) | (b & ~0x11111111u);
        const uint32_t w = (ab & 0x33333333u) | (c & ~0x33333333u);
        decode_fields<0x7u>(w, z_lo, z_hi, f);
    } else {
        uint32_t w0 = u.w[2 * s], w1 = u.w[2 * s + 1];
        if (SIGNED) {
            w0 ^= 0x80808080u;
            w1 ^= 0x80808080u;
        }
        // byte -> fp16 (1024 + byte) by placing it under the exponent byte 0x64
        f[0] = h2u(__hsub2(u2h(__byte_perm(w0, 0x64646464u, 0x4140)), z_lo));
        f[1] = h2u(__hsub2(u2h(__byte_perm(w0, 0x64646464u, 0x4342)), z_lo));
        f[2] = h2u(__hsub2(u2h(__byte_perm(w1, 0x64646464u, 0x4140)), z_lo));
        f[3] = h2u(__hsub2(u2h(__byte_perm(w1, 0x64646464u, 0x4342)), z_lo));
    }
}

// Source of 8 consecutive reduction elements k8*8.. of output row m (zeros when outside).
__device__ __forceinline__ uint4 load_x8(const Params& p, int amode, int m, int k)
{
    if (m >= p.M || k >= p.K) return make_uint4(0, 0, 0, 0);
    const __half* src;
    if (amode == A_CONV3) {
        const int hw = p.Ho * p.Wo;
        const int b = m / hw, rem = m - b * hw;
        const int ho = rem / p.Wo, wo = rem - ho * p.Wo;
        const long long img = static_cast<long long>(b) * p.H * p.W * p.Cin;
        if (p.Cin % 8 != 0) {
            // a run of eight may straddle filter taps: gather element by element
            __align__(16) __half tmp[8];
            for (int j = 0; j < 8; ++j) {
                tmp[j] = __float2half(0.f);
                const int kk = k + j;
                if (kk >= p.K) continue;
                const int tap = kk / p.Cin, c = kk - tap * p.Cin;
                const int hi = ho * p.stride - 1 + tap / 3, wi = wo * p.stride - 1 + tap % 3;
                if (hi < 0 || hi >= p.H || wi < 0 || wi >= p.W) continue;
                tmp[j] = p.X[img + (static_cast<long long>(hi) * p.W + wi) * p.Cin + c];
            }
            return *reinterpret_cast<uint4*>(tmp);
        }
        const int tap = k / p.Cin, c = k - tap * p.Cin;
        const int hi = ho * p.stride - 1 + tap / 3, wi = wo * p.stride - 1 + tap % 3;
        if (hi < 0 || hi >= p.H || wi < 0 || wi >= p.W) return make_uint4(0, 0, 0, 0);
        src = p.X + img + (static_cast<long long>(hi) * p.W + wi) * p.Cin + c;
    } else {
        src = p.X + static_cast<long long>(m) * p.ldx + k;
    }
    if (k + 8 <= p.K) return __ldg(reinterpret_cast<const uint4*>(src));
    // ragged end of the reduction (only when K is not a multiple of 8)
    __align__(16) __half tmp[8];
    for (int j = 0; j < 8; ++j) tmp[j] = (k + j < p.K) ? src[j] : __float2half(0.f);
    return *reinterpret_cast<uint4*>(tmp);
}

template <int BITS, bool SIGNED, int NT>
__global__ void __launch_bounds__(kThreads)
wo_kernel(const uint8_t* __restrict__ packed, long long pitch, const Params p, int amode, int chunk_len)
{
    pdl_launch_dependents();
    pdl_wait();
    extern __shared__ __align__(16) uint8_t smem[];
    constexpr int MB = 8 * NT;                       // tokens per CTA
    const int x_stride = chunk_len * 2 + 64;         // bytes per token row (64 mod 128: no bank conflicts)
    uint8_t* sX = smem;
    float* sRed = reinterpret_cast<float*>(smem + MB * x_stride);  // [kSlices][kChanPerCta][MB]

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    const int tile = warp % kTilesPerCta;
    const int slice = warp / kTilesPerCta;
    const int n_base = blockIdx.x * kChanPerCta + tile * 16;
    const int m_base = blockIdx.y * MB;

    const int n_lo = n_base + g, n_hi = n_base + g + 8;
    const bool lo_ok = n_lo < p.N, hi_ok = n_hi < p.N;
    const uint8_t* row_lo = packed + static_cast<long long>(lo_ok ? n_lo : 0) * pitch;
    const uint8_t* row_hi = packed + static_cast<long long>(hi_ok ? n_hi : 0) * pitch;

    // zero-points as fp16 offsets: low fields decode to 1024 + q, high fields to 64 + q
    float z_a = SIGNED ? (BITS == 8 ? 128.f : 8.f) : 0.f, z_b = z_a;
    if (!SIGNED && p.w_zero) {
        if (lo_ok) z_a = static_cast<float>(__ldg(p.w_zero + n_lo));
        if (hi_ok) z_b = static_cast<float>(__ldg(p.w_zero + n_hi));
    }
    const __half2 zlo_a = __float2half2_rn(1024.f + z_a), zhi_a = __float2half2_rn(-(64.f + z_a));
    const __half2 zlo_b = __float2half2_rn(1024.f + z_b), zhi_b = __float2half2_rn(-(64.f + z_b));

    float acc[NT][4];
#pragma unroll
    for (int i = 0; i < NT; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    constexpr int GROUP = BITS == 8 ? 2 : 4;  // units whose loads are issued together

    for (int kc0 = 0; kc0 < p.K; kc0 += chunk_len) {
        const int len = min(chunk_len, round_up_dev(p.K - kc0));
        const int units = len / kUnit;
        const int u_begin = (units * slice) / kSlices, u_end = (units * (slice + 1)) / kSlices;
        const int unit0 = kc0 / kUnit;

        // first group of weight loads goes out before the activations are staged
        UnitRegs<BITS> ra[GROUP], rb[GROUP];
#pragma unroll
        for (int i = 0; i < GROUP; ++i) {
            const bool in = u_begin + i < u_end;
            load_unit<BITS>(ra[i], row_lo, pitch, unit0 + u_begin + i, t, lo_ok && in);
            load_unit<BITS>(rb[i], row_hi, pitch, unit0 + u_begin + i, t, hi_ok && in);
        }

        if (kc0 > 0) __syncthreads();  // everyone is done reading the previous chunk
        // stage X[m_base .. m_base+MB) x [kc0, kc0+len) in decode order
        // (loads are issued eight at a time so that their latencies overlap)
        const int per_row = len / 8, total16 = MB * per_row;
        for (int base = tid; base < total16; base += kThreads * 8) {
            uint4 v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int idx = base + i * kThreads;
                if (idx < total16) {
                    const int r = idx / per_row, j = idx - r * per_row;
                    v[i] = load_x8(p, amode, m_base + r, kc0 + j * 8);
                }
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int idx = base + i * kThreads;
                if (idx >= total16) break;
                const int r = idx / per_row, j = idx - r * per_row;
                uint4 x = v[i];
                if (BITS != 8) {
                    // decode order inside each run of four: (0, 2, 1, 3)
                    const uint32_t a = __byte_perm(x.x, x.y, 0x5410), b = __byte_perm(x.x, x.y, 0x7632);
                    const uint32_t c = __byte_perm(x.z, x.w, 0x5410), d = __byte_perm(x.z, x.w, 0x7632);
                    x = make_uint4(a, b, c, d);
                }
                // 16-byte slot of (unit U, quad thread tt, sub-step s): 16 U + 4 s + tt
                const int U = j >> 4, tt = (j >> 2) & 3, sub = j & 3;
                *reinterpret_cast<uint4*>(sX + r * x_stride + (16 * U + 4 * sub + tt) * 16) = x;
            }
        }
        __syncthreads();

        for (int u0 = u_begin; u0 < u_end; u0 += GROUP) {
            // loads of the next group are issued before this group is consumed
            UnitRegs<BITS> na[GROUP], nb[GROUP];
#pragma unroll
            for (int i = 0; i < GROUP; ++i) {
                const bool in = u0 + GROUP + i < u_end;
                load_unit<BITS>(na[i], row_lo, pitch, unit0 + u0 + GROUP + i, t, lo_ok && in);
                load_unit<BITS>(nb[i], row_hi, pitch, unit0 + u0 + GROUP + i, t, hi_ok && in);
            }
#pragma unroll
            for (int i = 0; i < GROUP; ++i) {
                if (u0 + i >= u_end) break;
#pragma unroll
                for (int s = 0; s < 4; ++s) {
                    uint32_t fa[4], fb[4];
                    decode_substep<BITS, SIGNED>(ra[i], s, zlo_a, zhi_a, fa);
                    decode_substep<BITS, SIGNED>(rb[i], s, zlo_b, zhi_b, fb);
                    const uint32_t a1[4] = {fa[0], fb[0], fa[1], fb[1]};
                    const uint32_t a2[4] = {fa[2], fb[2], fa[3], fb[3]};
                    const int slot = (16 * (u0 + i) + 4 * s + t) * 16;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const uint4 xb = *reinterpret_cast<const uint4*>(sX + (g + 8 * nt) * x_stride + slot);
                        mma_16816(acc[nt], a1, xb.x, xb.y);
                        mma_16816(acc[nt], a2, xb.z, xb.w);
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < GROUP; ++i) {
                ra[i] = na[i];
                rb[i] = nb[i];
            }
        }
    }

    // sum the reduction slices: sRed[slice][channel][token]
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        float* base = sRed + (slice * kChanPerCta + tile * 16) * MB + nt * 8 + 2 * t;
        base[g * MB] = acc[nt][0];
        base[g * MB + 1] = acc[nt][1];
        base[(g + 8) * MB] = acc[nt][2];
        base[(g + 8) * MB + 1] = acc[nt][3];
    }
    __syncthreads();
    for (int idx = tid; idx < kChanPerCta * MB; idx += kThreads) {
        const int ch = idx % kChanPerCta, tok = idx / kChanPerCta;
        const int n = blockIdx.x * kChanPerCta + ch, m = m_base + tok;
        if (n >= p.N || m >= p.M) continue;
        float s = 0.f;
#pragma unroll
        for (int sl = 0; sl < kSlices; ++sl) s += sRed[(sl * kChanPerCta + ch) * MB + tok];
        const float b = p.bias ? __half2float(p.bias[n]) : 0.f;
        p.Y[static_cast<long long>(m) * p.ldy + n] = __float2half_rn(fmaf(__ldg(p.w_scale + n), s, b));
    }
}

// Small-token form (linear layers, at most 16 tokens): the layer is a single stream over the
// packed weights, so the kernel is built around that stream.  The first weight loads go out
// before the wait on the previous kernel -- weights and their parameters are constants of the
// layer, only the activations can come from the kernel before -- so consecutive layers keep
// the memory system busy across the kernel boundary.  The token rows come into shared memory
// by bulk copies (one per row, issued by one thread right after the wait): the load/store
// units are full of weight loads by then, and a staging pass through registers queued behind
// them took 2 to 6 us.  The rows stay in their natural order; the decode's pair order is
// applied to the fragments as they are read.
// CTA = 8 warps = TILES channel tiles x (8 / TILES) slices of the reduction.
template <int BITS, bool SIGNED, int NT, int TILES>
__global__ void __launch_bounds__(kThreads, 3)
wo_small_kernel(const uint8_t* __restrict__ packed, long long pitch, const Params p, int groups, int k_pad)
{
    constexpr int SLICES = 8 / TILES;
    constexpr int MB = 8 * NT;
    constexpr int GROUP = BITS == 8 ? 2 : 4;
    extern __shared__ __align__(16) uint8_t smem[];
    const int x_stride = k_pad * 2 + 16;  // token rows 16 bytes off a multiple of 128
    uint8_t* sX = smem;
    float* sRed = reinterpret_cast<float*>(smem + MB * x_stride);  // [SLICES][TILES * 16][MB]
    __shared__ __align__(8) uint64_t x_bar;
    __shared__ int x_abort;

    pdl_launch_dependents();
    const int tid = threadIdx.x;
    if (tid == 0) {
        mbar_init(smem_u32(&x_bar), 1);
        x_abort = 0;
        fence_barrier_init();
    }
    const int warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    const int tile = warp % TILES, slice = warp / TILES;
    const int units = k_pad / kUnit;
    const int u_begin = (units * slice) / SLICES, u_end = (units * (slice + 1)) / SLICES;

    // state of the channel-tile group being worked on (a CTA walks groups blockIdx.x,
    // blockIdx.x + gridDim.x, ...)
    const uint8_t *row_lo, *row_hi;
    bool lo_ok, hi_ok;
    float z_a, z_b;
    UnitRegs<BITS> ra[GROUP], rb[GROUP];

    auto load_group_units = [&](int u0) {
#pragma unroll
        for (int i = 0; i < GROUP; ++i) {
            const bool in = u0 + i < u_end;
            load_unit<BITS>(ra[i], row_lo, pitch, u0 + i, t, lo_ok && in);
            load_unit<BITS>(rb[i], row_hi, pitch, u0 + i, t, hi_ok && in);
        }
    };
    // weight side of a group: zero-points and the first packed words of this warp's slice
    auto begin_group = [&](int grp) {
        const int n_lo = (grp * TILES + tile) * 16 + g, n_hi = n_lo + 8;
        lo_ok = n_lo < p.N;
        hi_ok = n_hi < p.N;
        row_lo = packed + static_cast<long long>(lo_ok ? n_lo : 0) * pitch;
        row_hi = packed + static_cast<long long>(hi_ok ? n_hi : 0) * pitch;
        z_a = z_b = SIGNED ? (BITS == 8 ? 128.f : 8.f) : 0.f;
        if (!SIGNED && p.w_zero) {
            if (lo_ok) z_a = static_cast<float>(__ldg(p.w_zero + n_lo));
            if (hi_ok) z_b = static_cast<float>(__ldg(p.w_zero + n_hi));
        }
        load_group_units(u_begin);
    };

    int grp = blockIdx.x;
    if (grp < groups) begin_group(grp);  // issued before the wait: weights are constants of the layer
    pdl_wait();                          // the activations may be the previous kernel's output

    // the token rows, once per CTA: bulk copies of the rows that exist, zeros elsewhere
    __syncthreads();  // the barrier is initialised
    {
        const int rows = p.M < MB ? p.M : MB;
        if (tid == 0) {
            mbar_arrive_expect_tx(smem_u32(&x_bar), static_cast<uint32_t>(rows) * p.K * 2);
            for (int r = 0; r < rows; ++r)
                bulk_load(smem_u32(sX + r * x_stride), p.X + static_cast<long long>(r) * p.ldx, p.K * 2, smem_u32(&x_bar));
        }
        const int pad16 = (k_pad - p.K) / 8;  // 16-byte chunks past the end of a row
        for (int idx = tid; idx < rows * pad16; idx += kThreads) {
            const int r = idx / pad16, c = idx - r * pad16;
            *reinterpret_cast<uint4*>(sX + r * x_stride + (p.K + c * 8) * 2) = make_uint4(0, 0, 0, 0);
        }
        const int per_row = k_pad / 8;
        for (int idx = tid; idx < (MB - rows) * per_row; idx += kThreads) {
            const int r = rows + idx / per_row, c = idx % per_row;
            *reinterpret_cast<uint4*>(sX + r * x_stride + c * 16) = make_uint4(0, 0, 0, 0);
        }
    }
    __syncthreads();
    const bool x_ok = mbar_wait(smem_u32(&x_bar), 0, &x_abort);
    if (!x_ok && tid == 0 && p.status) atomicExch(p.status, MIXDQ_ERR_TIMEOUT);

    for (; grp < groups; grp += gridDim.x) {
        const __half2 zlo_a = __float2half2_rn(1024.f + z_a), zhi_a = __float2half2_rn(-(64.f + z_a));
        const __half2 zlo_b = __float2half2_rn(1024.f + z_b), zhi_b = __float2half2_rn(-(64.f + z_b));
        float acc[NT][4];
#pragma unroll
        for (int i = 0; i < NT; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

        for (int u0 = u_begin; u0 < u_end; u0 += GROUP) {
            if (u0 != u_begin) load_group_units(u0);
#pragma unroll
            for (int i = 0; i < GROUP; ++i) {
                if (u0 + i >= u_end) break;
#pragma unroll
                for (int sub = 0; sub < 4; ++sub) {
                    uint32_t fa[4], fb[4];
                    decode_substep<BITS, SIGNED>(ra[i], sub, zlo_a, zhi_a, fa);
                    decode_substep<BITS, SIGNED>(rb[i], sub, zlo_b, zhi_b, fb);
                    const uint32_t a1[4] = {fa[0], fb[0], fa[1], fb[1]};
                    const uint32_t a2[4] = {fa[2], fb[2], fa[3], fb[3]};
                    // the thread's eight reduction indices of this substep are one 16-byte chunk of the row
                    const int slot = (16 * (u0 + i) + 4 * t + sub) * 16;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        uint4 x = *reinterpret_cast<const uint4*>(sX + (g + 8 * nt) * x_stride + slot);
                        if (BITS != 8)  // the decode yields pairs (0, 2), (1, 3) of each run of four
                            x = make_uint4(__byte_perm(x.x, x.y, 0x5410), __byte_perm(x.x, x.y, 0x7632),
                                           __byte_perm(x.z, x.w, 0x5410), __byte_perm(x.z, x.w, 0x7632));
                        mma_16816(acc[nt], a1, x.x, x.y);
                        mma_16816(acc[nt], a2, x.z, x.w);
                    }
                }
            }
        }

        // the next group's weights start streaming while this one is reduced and stored
        const int out_grp = grp;
        if (grp + static_cast<int>(gridDim.x) < groups) begin_group(grp + gridDim.x);

        // sum the reduction slices: sRed[slice][channel][token]
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            float* base = sRed + (slice * TILES * 16 + tile * 16) * MB + nt * 8 + 2 * t;
            base[g * MB] = acc[nt][0];
            base[g * MB + 1] = acc[nt][1];
            base[(g + 8) * MB] = acc[nt][2];
            base[(g + 8) * MB + 1] = acc[nt][3];
        }
        __syncthreads();
        for (int idx = tid; idx < TILES * 16 * MB; idx += kThreads) {
            const int ch = idx % (TILES * 16), tok = idx / (TILES * 16);
            const int n = out_grp * TILES * 16 + ch;
            if (n >= p.N || tok >= p.M) continue;
            float sum = 0.f;
#pragma unroll
            for (int sl = 0; sl < SLICES; ++sl) sum += sRed[(sl * TILES * 16 + ch) * MB + tok];
            const float b = p.bias ? __half2float(p.bias[n]) : 0.f;
            p.Y[static_cast<long long>(tok) * p.ldy + n] = __float2half_rn(fmaf(__ldg(p.w_scale + n), sum, b));
        }
        __syncthreads();  // sRed is reused by the next group
    }
}

template <int BITS, bool SIGNED, int NT, int TILES>
int launch_small_tiles(const Params& p, const void* packed, long long pitch, cudaStream_t stream)
{
    constexpr int MB = 8 * NT;
    const int k_pad = static_cast<int>(round_up(p.K, kUnit));
    const size_t smem = static_cast<size_t>(MB) * (k_pad * 2 + 16) + 8 * 16 * MB * sizeof(float);
    auto kernel = wo_small_kernel<BITS, SIGNED, NT, TILES>;
    if (ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), 16 * (kSmallKMax * 2 + 64) + 8 * 16 * 16 * 4) != MIXDQ_OK) return MIXDQ_ERR_CUDA;
    // groups of TILES channel tiles are dealt to CTAs in equal rounds of at most three CTAs per SM
    const int groups = static_cast<int>(ceil_div(p.N, 16 * TILES));
    const int rounds = static_cast<int>(ceil_div(groups, 3 * (sm_count() > 0 ? sm_count() : 1)));
    const dim3 grid(static_cast<unsigned>(ceil_div(groups, rounds)));
    return launch_pdl(kernel, grid, dim3(kThreads), smem, stream, 1, static_cast<const uint8_t*>(packed), pitch, p,
                      groups, k_pad);
}

template <int BITS, bool SIGNED, int NT>
int launch_small(const Params& p, const void* packed, long long pitch, cudaStream_t stream)
{
    // one channel tile per CTA (more reduction slices) when two per CTA would leave SMs idle
    if (ceil_div(p.N, 32) < sm_count()) return launch_small_tiles<BITS, SIGNED, NT, 1>(p, packed, pitch, stream);
    return launch_small_tiles<BITS, SIGNED, NT, 2>(p, packed, pitch, stream);
}

template <int BITS, bool SIGNED, int NT>
int launch(const Params& p, int amode, const void* packed, long long pitch, cudaStream_t stream)
{
    constexpr int MB = 8 * NT;
    const int chunk_len = static_cast<int>(p.K > kChunkMax ? kChunkMax : round_up(p.K, kUnit));
    const size_t smem = static_cast<size_t>(MB) * (chunk_len * 2 + 64) + kSlices * kChanPerCta * MB * sizeof(float);
    auto kernel = wo_kernel<BITS, SIGNED, NT>;
    if (ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), 32 * (kChunkMax * 2 + 64) + kSlices * kChanPerCta * 32 * 4) != MIXDQ_OK) return MIXDQ_ERR_CUDA;
    dim3 grid(static_cast<unsigned>(ceil_div(p.N, kChanPerCta)), static_cast<unsigned>(ceil_div(p.M, MB)));
    return launch_pdl(kernel, grid, dim3(kThreads), smem, stream, 1, static_cast<const uint8_t*>(packed), pitch, p,
                      amode, chunk_len);
}

template <int BITS, bool SIGNED>
int launch_nt(const Params& p, int amode, const void* packed, long long pitch, cudaStream_t stream)
{
    if (amode == A_LINEAR && p.M <= 16 && p.K % 8 == 0 && p.K <= kSmallKMax) {
        if (p.M <= 8) return launch_small<BITS, SIGNED, 1>(p, packed, pitch, stream);
        return launch_small<BITS, SIGNED, 2>(p, packed, pitch, stream);
    }
    if (p.M <= 8) return launch<BITS, SIGNED, 1>(p, amode, packed, pitch, stream);
    if (p.M <= 16) return launch<BITS, SIGNED, 2>(p, amode, packed, pitch, stream);
    return launch<BITS, SIGNED, 4>(p, amode, packed, pitch, stream);
}

int run(Params p, int amode, const void* packed, int w_bits, cudaStream_t stream)
{
    if (amode != A_LINEAR && amode != A_CONV3) return MIXDQ_ERR_INVALID_ARG;
    if (amode == A_LINEAR && ((p.ldx % 8 != 0) || (reinterpret_cast<uintptr_t>(p.X) & 15)))
        return MIXDQ_ERR_ALIGNMENT;
    const long long pitch = row_pitch_bytes(p.K, w_bits, MIXDQ_LAYOUT_DEVICE);
    const bool is_signed = p.w_zero == nullptr;
    if (pair_path_ok(p, amode, w_bits)) return run_pair(p, amode, packed, w_bits, stream);
    if (tc_path_ok(p, amode, w_bits) && !(w_bits <= 3 && is_signed)) return run_tc(p, amode, packed, w_bits, p.batch, stream);
    if (w_bits == 3) return is_signed ? MIXDQ_ERR_UNSUPPORTED : launch_nt<3, false>(p, amode, packed, pitch, stream);
    if (w_bits == 2) return is_signed ? MIXDQ_ERR_UNSUPPORTED : launch_nt<2, false>(p, amode, packed, pitch, stream);
    if (w_bits == 4)
        return is_signed ? launch_nt<4, true>(p, amode, packed, pitch, stream)
                         : launch_nt<4, false>(p, amode, packed, pitch, stream);
    if (w_bits == 8)
        return is_signed ? launch_nt<8, true>(p, amode, packed, pitch, stream)
                         : launch_nt<8, false>(p, amode, packed, pitch, stream);
    return MIXDQ_ERR_UNSUPPORTED;
}

}  // namespace wo
}  // namespace mixdq
