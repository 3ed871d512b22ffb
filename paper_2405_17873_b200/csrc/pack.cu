// Offline side of the path: per-channel min-max parameters, weight quantization and
// packing (3 / 4 / 8 bits, canonical and device layouts), the unpack parity hook, and the
// per-tensor activation range helpers.  None of this is on the per-step hot path, so the
// kernels favour exactness (products in double, one IEEE divide per scale) over speed.
#include "common.cuh"
#include "codes.cuh"

namespace mixdq {

namespace {

// round-half-even of the exact product w * inv (11-bit x 24-bit significands fit a double)
__device__ __forceinline__ long long rne_product(float w, float inv)
{
    double p = static_cast<double>(w) * static_cast<double>(inv);
    p = fmin(fmax(p, -1e15), 1e15);
    return __double2ll_rn(p);
}

__device__ __forceinline__ int clampi(long long v, int lo, int hi)
{
    return v < lo ? lo : (v > hi ? hi : static_cast<int>(v));
}

// One block per output channel: min / max of the row, then scale and zero-point.
__global__ void weight_minmax_kernel(const __half* __restrict__ W, int64_t K, int bits, int symmetric,
                                     float* __restrict__ scale_out, int32_t* __restrict__ zero_out)
{
    const int64_t n = blockIdx.x;
    const __half* row = W + n * K;
    float lo = 0.f, hi = 0.f;
    for (int64_t k = threadIdx.x; k < K; k += blockDim.x) {
        float w = __half2float(row[k]);
        lo = fminf(lo, w);
        hi = fmaxf(hi, w);
    }
    __shared__ float s_lo[32], s_hi[32];
    for (int o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if ((threadIdx.x & 31) == 0) {
        s_lo[threadIdx.x >> 5] = lo;
        s_hi[threadIdx.x >> 5] = hi;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const int nw = (blockDim.x + 31) >> 5;
        for (int i = 1; i < nw; ++i) {
            lo = fminf(lo, s_lo[i]);
            hi = fmaxf(hi, s_hi[i]);
        }
        if (symmetric) {
            const float amax = fmaxf(-lo, hi);
            const float qmax = static_cast<float>((1 << (bits - 1)) - 1);
            scale_out[n] = (amax == 0.f) ? 1.f : __fdiv_rn(amax, qmax);
            if (zero_out) zero_out[n] = 0;
        } else {
            const int L = (1 << bits) - 1;
            const float range = __fsub_rn(hi, lo);
            const float scale = (range == 0.f) ? 1.f : __fdiv_rn(range, static_cast<float>(L));
            scale_out[n] = scale;
            if (zero_out) zero_out[n] = clampi(rne_product(-lo, __fdiv_rn(1.f, scale)), 0, L);
        }
    }
}

// Code of element (n, k); positions beyond K hold the pad code (0 signed, zero-point unsigned).
__device__ __forceinline__ int code_at(const __half* __restrict__ W, int64_t n, int64_t k, int64_t K,
                                       int bits, float inv, bool has_zero, int z)
{
    if (k >= K) return has_zero ? z : 0;
    const long long r = rne_product(__half2float(W[n * K + k]), inv);
    if (has_zero) return clampi(r + z, 0, (1 << bits) - 1);
    const int qmax = (1 << (bits - 1)) - 1;
    return clampi(r, -qmax, qmax);
}

// One thread per 32-bit output word of a packed row.
__global__ void pack_kernel(const __half* __restrict__ W, int64_t N, int64_t K, int bits,
                            const float* __restrict__ scale, const int32_t* __restrict__ zero,
                            int layout, int64_t pitch, uint8_t* __restrict__ out)
{
    const int64_t words_per_row = (pitch + 3) / 4;
    const int64_t idx = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x;
    if (idx >= N * words_per_row) return;
    const int64_t n = idx / words_per_row;
    const int64_t w = idx - n * words_per_row;
    const float inv = __fdiv_rn(1.f, scale[n]);
    const bool hz = zero != nullptr;
    const int z = hz ? zero[n] : 0;
    uint8_t* row = out + n * pitch;
    uint32_t word = 0;

    if (bits == 8) {
        for (int j = 0; j < 4; ++j)
            word |= static_cast<uint32_t>(code_at(W, n, 4 * w + j, K, 8, inv, hz, z) & 0xff) << (8 * j);
    } else if (bits == 4) {
        if (layout == MIXDQ_LAYOUT_CANONICAL) {
            // an odd K leaves the last high nibble empty (0) in the canonical layout
            for (int j = 0; j < 8; ++j)
                if (8 * w + j < K)
                    word |= static_cast<uint32_t>(code_at(W, n, 8 * w + j, K, 4, inv, hz, z) & 0xf)
                            << (4 * j);
        } else {
            // byte j of the word: code j in the low nibble, code j + 4 in the high nibble
            for (int j = 0; j < 4; ++j) {
                const uint32_t lo = code_at(W, n, 8 * w + j, K, 4, inv, hz, z) & 0xf;
                const uint32_t hi = code_at(W, n, 8 * w + 4 + j, K, 4, inv, hz, z) & 0xf;
                word |= (lo | (hi << 4)) << (8 * j);
            }
        }
    } else {  // bit-planes: `bits` (3 or 2) planes per group
        if (layout == MIXDQ_LAYOUT_CANONICAL) {
            const int64_t k0 = 32 * (w / bits);  // group g: words bits*g .. are planes 0..bits-1
            const int plane = static_cast<int>(w % bits);
            for (int j = 0; j < 32; ++j)
                word |= static_cast<uint32_t>((code_at(W, n, k0 + j, K, bits, inv, hz, z) >> plane) & 1) << j;
        } else {
            // block of 128 codes: planes in order, 4 words each; word t of a plane covers codes
            // 32t .. 32t+31 with bit 4f + s = code 8s + (f even ? f/2 : 4 + f/2), which is the
            // field order of the 4-bit device layout spread over four shifts of the word
            const int64_t blk = w / (4 * bits);
            const int r = static_cast<int>(w % (4 * bits));
            const int plane = r / 4;
            const int64_t k0 = 128 * blk + 32 * (r % 4);
            for (int pos = 0; pos < 32; ++pos) {
                const int f = pos >> 2, sft = pos & 3;
                const int j = 8 * sft + ((f & 1) ? 4 + (f >> 1) : (f >> 1));
                word |= static_cast<uint32_t>((code_at(W, n, k0 + j, K, bits, inv, hz, z) >> plane) & 1) << pos;
            }
        }
    }
    // the last word of an odd-sized canonical row may be partial
    const int64_t byte0 = 4 * w;
    for (int b = 0; b < 4 && byte0 + b < pitch; ++b) row[byte0 + b] = (word >> (8 * b)) & 0xff;
}

// One thread per code.
__global__ void unpack_kernel(const uint8_t* __restrict__ packed, int64_t N, int64_t K, int bits,
                              int is_signed, int layout, int64_t pitch, int16_t* __restrict__ codes)
{
    const int64_t idx = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x;
    if (idx >= N * K) return;
    const int64_t n = idx / K;
    const int64_t k = idx - n * K;
    codes[idx] = static_cast<int16_t>(decode_code(packed + n * pitch, k, bits, is_signed, layout));
}

// One CTA of 128 threads per output channel: sum over k of its signed codes.
__global__ void code_sums_kernel(const uint8_t* __restrict__ packed, int64_t K, int bits, int64_t pitch,
                                 int32_t* __restrict__ sums)
{
    __shared__ int part[4];
    const uint8_t* row = packed + blockIdx.x * pitch;
    int s = 0;
    for (int64_t k = threadIdx.x; k < K; k += blockDim.x) s += decode_code(row, k, bits, 1, MIXDQ_LAYOUT_DEVICE);
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) sums[blockIdx.x] = part[0] + part[1] + part[2] + part[3];
}

// Range of a tensor with 0 included: floats ordered through a monotone map to unsigned integers.
__device__ __forceinline__ unsigned int ordered_bits(float f)
{
    const unsigned int u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// range_bits[0]: ordered bits of the running minimum, [1]: of the running maximum.
__global__ void minmax_kernel(const __half* __restrict__ X, int64_t rows, int64_t cols, int64_t row_stride,
                              unsigned int* __restrict__ range_bits)
{
    float lo = 0.f, hi = 0.f;
    const int64_t chunks_per_row = (cols + 7) / 8;
    const int64_t total = rows * chunks_per_row;
    const bool vec_ok = (cols % 8 == 0) && (row_stride % 8 == 0) &&
                        ((reinterpret_cast<uintptr_t>(X) & 15) == 0);
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t r = i / chunks_per_row;
        const int64_t c = (i - r * chunks_per_row) * 8;
        const __half* p = X + r * row_stride + c;
        if (vec_ok) {
            const uint4 v = *reinterpret_cast<const uint4*>(p);
            const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 f = __half22float2(h[j]);
                lo = fminf(lo, fminf(f.x, f.y));
                hi = fmaxf(hi, fmaxf(f.x, f.y));
            }
        } else {
            for (int j = 0; j < 8 && c + j < cols; ++j) {
                const float f = __half2float(p[j]);
                lo = fminf(lo, f);
                hi = fmaxf(hi, f);
            }
        }
    }
    for (int o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if ((threadIdx.x & 31) == 0) {
        if (lo < 0.f) atomicMin(range_bits, ordered_bits(lo));
        if (hi > 0.f) atomicMax(range_bits + 1, ordered_bits(hi));
    }
}

// Both accumulators start at the ordered bits of +0.
__global__ void minmax_init_kernel(unsigned int* __restrict__ range_bits)
{
    range_bits[0] = 0x80000000u;
    range_bits[1] = 0x80000000u;
}

// Ordered bits back to the bit patterns of {lo, hi}.
__global__ void minmax_finish_kernel(unsigned int* __restrict__ range_bits)
{
    for (int i = 0; i < 2; ++i) {
        const unsigned int o = range_bits[i];
        range_bits[i] = (o & 0x80000000u) ? (o & 0x7fffffffu) : ~o;
    }
}

// scale = (hi - lo) / 255, zero = clamp(rne(-lo / scale), 0, 255); an all-zero tensor: scale 1, zero 0.
__global__ void act_asym_params_kernel(const float* __restrict__ minmax, float* __restrict__ scale_out,
                                       int32_t* __restrict__ zero_out)
{
    const float lo = minmax[0], hi = minmax[1];
    if (hi == lo) {
        scale_out[0] = 1.f;
        zero_out[0] = 0;
        return;
    }
    const float s = __fdiv_rn(__fsub_rn(hi, lo), 255.f);
    const float inv = __fdiv_rn(1.f, s);
    // -lo * inv <= 255 * (1 + 2^-22): the magic-number addition rounds the exact product to nearest even
    const float t = __fmaf_rn(-lo, inv, 12582912.f);
    int z = static_cast<int>(__float_as_uint(t)) - 0x4B400000;
    z = z < 0 ? 0 : (z > 255 ? 255 : z);
    scale_out[0] = s;
    zero_out[0] = z;
}

// max |x| as an atomic max on the bit pattern (non-negative floats order like integers).
__global__ void absmax_kernel(const __half* __restrict__ X, int64_t rows, int64_t cols,
                              int64_t row_stride, int skip_mod, unsigned int* __restrict__ amax_bits)
{
    float m = 0.f;
    const int64_t chunks_per_row = (cols + 7) / 8;
    const int64_t total = rows * chunks_per_row;
    const bool vec_ok = (cols % 8 == 0) && (row_stride % 8 == 0) &&
                        ((reinterpret_cast<uintptr_t>(X) & 15) == 0);
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t r = i / chunks_per_row;
        const int64_t c = (i - r * chunks_per_row) * 8;
        if (skip_mod > 0 && r % skip_mod == 0) continue;
        const __half* p = X + r * row_stride + c;
        if (vec_ok) {
            const uint4 v = *reinterpret_cast<const uint4*>(p);
            const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 f = __half22float2(h[j]);
                m = fmaxf(m, fmaxf(fabsf(f.x), fabsf(f.y)));
            }
        } else {
            for (int j = 0; j < 8 && c + j < cols; ++j) m = fmaxf(m, fabsf(__half2float(p[j])));
        }
    }
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0 && m > 0.f) atomicMax(amax_bits, __float_as_uint(m));
}

__global__ void act_scale_kernel(const float* __restrict__ amax, float* __restrict__ scale_out)
{
    const float a = amax[0];
    scale_out[0] = (a == 0.f) ? 1.f : __fdiv_rn(a, 127.f);
}

bool width_ok(int bits) { return bits == 2 || bits == 3 || bits == 4 || bits == 8; }

}  // namespace

}  // namespace mixdq

using namespace mixdq;

// The layer kernels load a layer's constants (packed weights, scales, zero-points, code sums) before they
// wait for earlier kernels of the stream, so a kernel that WRITES such constants must be complete, not merely
// finishing, when the next layer call is enqueued behind it.  The entry points below that produce constants
// therefore end with this empty kernel: launched plainly, it starts only after everything before it on the
// stream has completed and its writes are visible, and whatever follows it overlaps nothing but it.
__global__ void constants_complete_kernel() {}

static int finish_constants(cudaStream_t st)
{
    if (cudaGetLastError() != cudaSuccess) return MIXDQ_ERR_CUDA;
    constants_complete_kernel<<<1, 32, 0, st>>>();
    return check_launch();
}

extern "C" int mixdq_packed_bytes(int64_t N, int64_t K, int bits, int layout, size_t* out)
{
    if (!out || N <= 0 || K <= 0) return MIXDQ_ERR_INVALID_ARG;
    if (layout != MIXDQ_LAYOUT_CANONICAL && layout != MIXDQ_LAYOUT_DEVICE) return MIXDQ_ERR_INVALID_ARG;
    if (!width_ok(bits)) return MIXDQ_ERR_UNSUPPORTED;
    if (layout == MIXDQ_LAYOUT_CANONICAL) {
        *out = static_cast<size_t>(N * row_pitch_bytes(K, bits, layout));
    } else {
        // device buffers are read in whole 16-byte units
        *out = static_cast<size_t>(round_up(N * row_pitch_bytes(K, bits, layout), 16));
    }
    return MIXDQ_OK;
}

extern "C" int mixdq_weight_minmax_params(const void* W, int64_t N, int64_t K, int bits, int symmetric,
                                          float* scale_out, int32_t* zero_out, void* stream)
{
    if (!W || !scale_out || N <= 0 || K <= 0) return MIXDQ_ERR_INVALID_ARG;
    if (bits < 2 || bits > 8) return MIXDQ_ERR_UNSUPPORTED;
    if (!symmetric && !zero_out) return MIXDQ_ERR_INVALID_ARG;
    weight_minmax_kernel<<<static_cast<unsigned>(N), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const __half*>(W), K, bits, symmetric, scale_out, zero_out);
    return finish_constants(static_cast<cudaStream_t>(stream));
}

extern "C" int mixdq_pack_weights(const void* W, int64_t N, int64_t K, int bits, const float* scale,
                                  const int32_t* zero, int layout, void* packed_out, void* stream)
{
    if (!W || !scale || !packed_out || N <= 0 || K <= 0) return MIXDQ_ERR_INVALID_ARG;
    if (layout != MIXDQ_LAYOUT_CANONICAL && layout != MIXDQ_LAYOUT_DEVICE) return MIXDQ_ERR_INVALID_ARG;
    if (!width_ok(bits)) return MIXDQ_ERR_UNSUPPORTED;
    if (bits <= 3 && !zero) return MIXDQ_ERR_UNSUPPORTED;  // bit-plane codes are unsigned only
    if (reinterpret_cast<uintptr_t>(packed_out) & 15) return MIXDQ_ERR_ALIGNMENT;
    const int64_t pitch = row_pitch_bytes(K, bits, layout);
    const int64_t words = N * ((pitch + 3) / 4);
    pack_kernel<<<static_cast<unsigned>(ceil_div(words, 256)), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const __half*>(W), N, K, bits, scale, zero, layout, pitch,
        static_cast<uint8_t*>(packed_out));
    return finish_constants(static_cast<cudaStream_t>(stream));
}

extern "C" int mixdq_unpack_weights(const void* packed, int64_t N, int64_t K, int bits, int is_signed,
                                    int layout, int16_t* codes_out, void* stream)
{
    if (!packed || !codes_out || N <= 0 || K <= 0) return MIXDQ_ERR_INVALID_ARG;
    if (layout != MIXDQ_LAYOUT_CANONICAL && layout != MIXDQ_LAYOUT_DEVICE) return MIXDQ_ERR_INVALID_ARG;
    if (!width_ok(bits)) return MIXDQ_ERR_UNSUPPORTED;
    if (bits <= 3 && is_signed) return MIXDQ_ERR_UNSUPPORTED;
    const int64_t pitch = row_pitch_bytes(K, bits, layout);
    unpack_kernel<<<static_cast<unsigned>(ceil_div(N * K, 256)), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint8_t*>(packed), N, K, bits, is_signed, layout, pitch, codes_out);
    return check_launch();
}

extern "C" int mixdq_act_absmax(const void* X, int64_t rows, int64_t cols, int64_t row_stride,
                                int skip_rows_mod, float* amax_out, void* stream)
{
    if (!X || !amax_out || rows <= 0 || cols <= 0 || row_stride < cols || skip_rows_mod < 0)
        return MIXDQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    MIXDQ_CUDA_TRY(cudaMemsetAsync(amax_out, 0, sizeof(float), st));
    const int64_t chunks = rows * ((cols + 7) / 8);
    const unsigned grid = static_cast<unsigned>(chunks < 256 * 1184 ? ceil_div(chunks, 256) : 1184);
    absmax_kernel<<<grid, 256, 0, st>>>(static_cast<const __half*>(X), rows, cols, row_stride,
                                        skip_rows_mod, reinterpret_cast<unsigned int*>(amax_out));
    return check_launch();
}

extern "C" int mixdq_act_scale_from_absmax(const float* amax, float* scale_out, void* stream)
{
    if (!amax || !scale_out) return MIXDQ_ERR_INVALID_ARG;
    act_scale_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(amax, scale_out);
    return check_launch();
}

extern "C" int mixdq_act_minmax(const void* X, int64_t rows, int64_t cols, int64_t row_stride,
                                float* minmax_out, void* stream)
{
    if (!X || !minmax_out || rows <= 0 || cols <= 0 || row_stride < cols) return MIXDQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned int* bits = reinterpret_cast<unsigned int*>(minmax_out);
    minmax_init_kernel<<<1, 1, 0, st>>>(bits);
    int rc = check_launch();
    if (rc != MIXDQ_OK) return rc;
    const int64_t chunks = rows * ((cols + 7) / 8);
    const unsigned grid = static_cast<unsigned>(chunks < 256 * 1184 ? ceil_div(chunks, 256) : 1184);
    minmax_kernel<<<grid, 256, 0, st>>>(static_cast<const __half*>(X), rows, cols, row_stride, bits);
    rc = check_launch();
    if (rc != MIXDQ_OK) return rc;
    minmax_finish_kernel<<<1, 1, 0, st>>>(bits);
    return check_launch();
}

extern "C" int mixdq_act_asym_params_from_minmax(const float* minmax, float* scale_out, int32_t* zero_out,
                                                 void* stream)
{
    if (!minmax || !scale_out || !zero_out) return MIXDQ_ERR_INVALID_ARG;
    act_asym_params_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(minmax, scale_out, zero_out);
    return check_launch();
}

extern "C" int mixdq_weight_code_sums(const void* packed_W, int64_t N, int64_t K, int bits, int32_t* sums_out,
                                      void* stream)
{
    if (!packed_W || !sums_out || N <= 0 || K <= 0) return MIXDQ_ERR_INVALID_ARG;
    if (bits != 4 && bits != 8) return MIXDQ_ERR_UNSUPPORTED;
    const int64_t pitch = row_pitch_bytes(K, bits, MIXDQ_LAYOUT_DEVICE);
    code_sums_kernel<<<static_cast<unsigned>(N), 128, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint8_t*>(packed_W), K, bits, pitch, sums_out);
    return finish_constants(static_cast<cudaStream_t>(stream));
}
