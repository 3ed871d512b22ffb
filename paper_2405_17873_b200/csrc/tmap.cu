// Tensor-map (TMA descriptor) encoding.  The driver entry point is looked up through the
// runtime so that the library has no link-time dependency on libcuda and still loads on
// a machine without a GPU driver.
#include <mutex>
#include <unordered_set>

#include "common.cuh"

namespace mixdq {

namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            (void)cudaGetLastError();
    });
    return fn;
}

}  // namespace

int encode_tmap_2d_u8(CUtensorMap* map, const void* base, uint64_t row_bytes, uint64_t rows,
                      uint64_t pitch_bytes, uint32_t box_bytes, uint32_t box_rows, bool swizzle128)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return MIXDQ_ERR_CUDA;
    if ((reinterpret_cast<uintptr_t>(base) & 15) || (pitch_bytes & 15)) return MIXDQ_ERR_ALIGNMENT;
    cuuint64_t dims[2] = {row_bytes, rows};
    cuuint64_t strides[1] = {pitch_bytes};
    cuuint32_t box[2] = {box_bytes, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE,
                    swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? MIXDQ_OK : MIXDQ_ERR_CUDA;
}

int encode_tmap_2d_f16(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows,
                       uint64_t pitch_elems, uint32_t box_cols, uint32_t box_rows, bool swizzle64)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return MIXDQ_ERR_CUDA;
    if ((reinterpret_cast<uintptr_t>(base) & 15) || ((pitch_elems * 2) & 15)) return MIXDQ_ERR_ALIGNMENT;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {pitch_elems * 2};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? MIXDQ_OK : MIXDQ_ERR_CUDA;
}


static int encode_tmap_4d(CUtensorMap* map, CUtensorMapDataType dtype, const void* base, const uint64_t dims[4],
                          const uint64_t strides_bytes[3], const uint32_t box[4], uint32_t hw_step);

int encode_tmap_4d_u8(CUtensorMap* map, const void* base, const uint64_t dims[4], const uint64_t strides_bytes[3],
                      const uint32_t box[4], uint32_t hw_step)
{
    return encode_tmap_4d(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, base, dims, strides_bytes, box, hw_step);
}

int encode_tmap_4d_f16(CUtensorMap* map, const void* base, const uint64_t dims[4], const uint64_t strides_bytes[3],
                       const uint32_t box[4], uint32_t hw_step)
{
    return encode_tmap_4d(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, base, dims, strides_bytes, box, hw_step);
}

static int encode_tmap_4d(CUtensorMap* map, CUtensorMapDataType dtype, const void* base, const uint64_t dims[4],
                          const uint64_t strides_bytes[3], const uint32_t box[4], uint32_t hw_step)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return MIXDQ_ERR_CUDA;
    if (reinterpret_cast<uintptr_t>(base) & 15) return MIXDQ_ERR_ALIGNMENT;
    cuuint64_t d[4], st[3];
    // hw_step > 1 (strided convolution): the box takes every hw_step-th pixel along W and H; the
    // encoder wants the traversed extent, of which it loads ceil(extent / step) elements
    cuuint32_t b[4], estr[4] = {1, hw_step, hw_step, 1};
    for (int i = 0; i < 4; ++i) {
        d[i] = dims[i];
        b[i] = (i == 1 || i == 2) ? box[i] * hw_step : box[i];
        if (b[i] > 256) return MIXDQ_ERR_UNSUPPORTED;
    }
    for (int i = 0; i < 3; ++i) {
        if (strides_bytes[i] & 15) return MIXDQ_ERR_ALIGNMENT;
        st[i] = strides_bytes[i];
    }
    CUresult r = fn(map, dtype, 4, const_cast<void*>(base), d, st, b, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? MIXDQ_OK : MIXDQ_ERR_CUDA;
}

namespace {

constexpr int kMaxDevices = 64;

// Function attributes and device properties belong to a device: everything cached here is keyed by it.
int current_device()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return -1;
    }
    return (dev >= 0 && dev < kMaxDevices) ? dev : -1;
}

}  // namespace

int prefer_max_shared_carveout(const void* kernel)
{
    static std::mutex mu;
    static std::unordered_set<const void*> done[kMaxDevices];
    const int dev = current_device();
    if (dev < 0) return MIXDQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (done[dev].count(kernel)) return MIXDQ_OK;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return MIXDQ_ERR_CUDA;
    }
    done[dev].insert(kernel);
    return MIXDQ_OK;
}

int ensure_dynamic_smem(const void* kernel, int bytes)
{
    static std::mutex mu;
    static std::unordered_set<const void*> done[kMaxDevices];
    const int dev = current_device();
    if (dev < 0) return MIXDQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (done[dev].count(kernel)) return MIXDQ_OK;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return MIXDQ_ERR_CUDA;
    }
    done[dev].insert(kernel);
    return MIXDQ_OK;
}

int sm_count()
{
    static std::mutex mu;
    static int count[kMaxDevices] = {};
    const int dev = current_device();
    if (dev < 0) return 0;
    std::lock_guard<std::mutex> lock(mu);
    if (!count[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            (void)cudaGetLastError();
            return 0;
        }
        count[dev] = n;
    }
    return count[dev];
}

}  // namespace mixdq
