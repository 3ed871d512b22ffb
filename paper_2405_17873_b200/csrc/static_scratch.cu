// W8A8 / W4A8 linear layer for callers that cannot hand the library any scratch memory.
//
// Some hosts of this library may not allocate device memory at all: a serving process whose
// memory manager has already claimed the whole GPU, a plug-in that runs inside another
// framework's allocator and must not go around it, or a latency-critical loop where the
// implicit device-wide synchronization of cudaMalloc / cudaFree is not acceptable.  For them
// the scratch of the int8 linear layer -- above all the int8 copy of the activations that the
// quantization pass writes and the GEMM kernel reads, behind the region reserved for a split
// reduction -- lives in a fixed array inside the library image instead of a caller-provided
// workspace.
#include <mutex>

#include "common.cuh"
#include "engines.h"

namespace {

// Held by every GPU that loads the library, from module load until the process exits.
constexpr size_t kStaticScratchBytes = 8u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the array on the current device.  In host code the symbol's name is only
// a handle; the address a kernel can use comes from cudaGetSymbolAddress, looked up once per
// device with that device current.
int scratch_address(void** out)
{
    int dev = -1;
    MIXDQ_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return MIXDQ_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_ptr[dev]) {
        void* ptr = nullptr;
        MIXDQ_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return MIXDQ_OK;
}

}  // namespace

extern "C" size_t mixdq_static_scratch_bytes(void) { return kStaticScratchBytes; }

extern "C" int mixdq_linear_a8_static_scratch(const void* X, int64_t M, int64_t K, int64_t ldx,
                                              const void* packed_W, int64_t N, int w_bits,
                                              const float* w_scale, const float* act_scale, const void* bias,
                                              void* Y, int32_t* status, void* stream)
{
    using namespace mixdq;
    if (!X || !packed_W || !w_scale || !act_scale || !Y) return MIXDQ_ERR_INVALID_ARG;
    if (M <= 0 || K <= 0 || N <= 0 || M > 0x7fffffff || K > 0x7fffffff || N > 0x7fffffff || ldx < K)
        return MIXDQ_ERR_INVALID_ARG;
    if (w_bits != 4 && w_bits != 8) return MIXDQ_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(packed_W) & 15) return MIXDQ_ERR_ALIGNMENT;
    const size_t need = i8::workspace_bytes(M, N, M, K);
    if (need > kStaticScratchBytes) return MIXDQ_ERR_WORKSPACE;  // problem too large for the fixed array
    void* scratch = nullptr;
    int rc = scratch_address(&scratch);
    if (rc != MIXDQ_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The array keeps whatever the previous call left behind.  Nothing in it has to start at zero for
    // the kernels reached from here: the quantization pass overwrites every byte of the int8 copy that
    // the GEMM reads, and the one user of counters that start at zero (the split reduction of the
    // single-kernel form) clears its region itself before it launches.
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
    p.ldy = N;
    p.status = status;
    return i8::run(p, A_LINEAR, packed_W, w_bits, scratch, kStaticScratchBytes, st);
}
