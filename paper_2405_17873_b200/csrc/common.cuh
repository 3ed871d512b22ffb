// Shared helpers for the sm_100a kernels: PTX wrappers for mbarriers, TMA and tcgen05,
// plus small host-side utilities.  Internal to the library.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/mixdq.h"

namespace mixdq {

// ---------------------------------------------------------------- host utilities

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline int64_t round_up(int64_t a, int64_t b) { return ceil_div(a, b) * b; }

// Row pitch in bytes of the layouts documented in mixdq.h (-1: unsupported width).
inline int64_t row_pitch_bytes(int64_t K, int bits, int layout)
{
    if (layout == MIXDQ_LAYOUT_CANONICAL) {
        if (bits == 8) return K;
        if (bits == 4) return (K + 1) / 2;
        if (bits == 3 || bits == 2) return ceil_div(K, 32) * 4 * bits;
    } else if (layout == MIXDQ_LAYOUT_DEVICE) {
        if (bits == 8) return round_up(K, 16);
        if (bits == 4) return round_up(K, 32) / 2;
        if (bits == 3 || bits == 2) return ceil_div(K, 128) * 16 * bits;
    }
    return -1;
}

#define MIXDQ_CUDA_TRY(expr)                \
    do {                                    \
        cudaError_t err__ = (expr);         \
        if (err__ != cudaSuccess) {         \
            (void)cudaGetLastError();       \
            return MIXDQ_ERR_CUDA;          \
        }                                   \
    } while (0)

// Kernels of the layer calls launched (or captured into a graph) by this process so far.
inline std::atomic<unsigned long long> g_layer_kernel_launches{0};

inline int check_launch() { return cudaGetLastError() == cudaSuccess ? MIXDQ_OK : MIXDQ_ERR_CUDA; }

// 2-D byte tensor map (rows x row_bytes, pitch in bytes) for TMA tile loads.
int encode_tmap_2d_u8(CUtensorMap* map, const void* base, uint64_t row_bytes, uint64_t rows,
                      uint64_t pitch_bytes, uint32_t box_bytes, uint32_t box_rows, bool swizzle128);
// 2-D fp16 tensor map (rows x cols elements, pitch in elements), 128-byte swizzle (64-byte for
// boxes of 32 columns when swizzle64 is set).
int encode_tmap_2d_f16(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows,
                       uint64_t pitch_elems, uint32_t box_cols, uint32_t box_rows, bool swizzle64 = false);

// 4-D byte tensor map with the 128-byte swizzle (NHWC int8 image: dims {C, W, H, B}).  box: elements
// loaded per dimension; hw_step > 1 takes every hw_step-th pixel along W and H (strided convolution).
int encode_tmap_4d_u8(CUtensorMap* map, const void* base, const uint64_t dims[4], const uint64_t strides_bytes[3],
                      const uint32_t box[4], uint32_t hw_step = 1);
// The same for an fp16 NHWC image (box extents in elements, strides in bytes).
int encode_tmap_4d_f16(CUtensorMap* map, const void* base, const uint64_t dims[4], const uint64_t strides_bytes[3],
                       const uint32_t box[4], uint32_t hw_step = 1);

// Once per kernel: ask for the largest shared-memory carve-out.  An SM changes its L1 / shared
// split only when idle, so kernels with different preferences cannot share an SM and the change
// itself costs time at every kernel boundary; with one preference everywhere, a small kernel's
// tail and the next GEMM's set-up overlap.  Returns MIXDQ_OK or MIXDQ_ERR_CUDA.
int prefer_max_shared_carveout(const void* kernel);

// Once per (device, kernel): raise the kernel's dynamic shared-memory limit to `bytes`.
int ensure_dynamic_smem(const void* kernel, int bytes);

// Streaming multiprocessors of the current device (looked up once per device; 0 on error).
int sm_count();

#ifdef __CUDACC__

// Launch with programmatic dependent launch enabled (and an optional cluster along z): the
// grid may start while the previous kernel of the stream is still draining, so its set-up
// (barrier init, tensor-memory allocation, descriptor prefetch) overlaps that tail.  Every
// kernel launched this way calls pdl_wait() before it touches global memory.
template <typename... KArgs, typename... Args>
inline int launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              unsigned cluster_x, unsigned cluster_z, Args&&... args);

template <typename... KArgs, typename... Args>
inline int launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                      unsigned cluster_z, Args&&... args)
{
    return launch_pdl_cluster(kernel, grid, block, smem, stream, 1u, cluster_z, static_cast<Args&&>(args)...);
}

// The same with a cluster of cluster_x x 1 x cluster_z CTAs (kernels whose CTA pairs share tensor-core
// instructions need their pairs adjacent along x).
template <typename... KArgs, typename... Args>
inline int launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              unsigned cluster_x, unsigned cluster_z, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster_x;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = cluster_z;
    cfg.attrs = attr;
    cfg.numAttrs = (cluster_z > 1 || cluster_x > 1) ? 2 : 1;
    if (prefer_max_shared_carveout(reinterpret_cast<const void*>(kernel)) != MIXDQ_OK) return MIXDQ_ERR_CUDA;
    g_layer_kernel_launches.fetch_add(1, std::memory_order_relaxed);
    cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
    if (err != cudaSuccess) {
        (void)cudaGetLastError();
        return MIXDQ_ERR_CUDA;
    }
    return MIXDQ_OK;
}

// ---------------------------------------------------------------- device helpers

// Let the next kernel of the stream begin launching (it still waits for this grid to finish
// before reading memory).
__device__ __forceinline__ void pdl_launch_dependents()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Wait until every kernel this grid depends on has completed and its writes are visible.
__device__ __forceinline__ void pdl_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}


// Spin budget of every bounded wait, in SM clock cycles (a few hundred ms).
constexpr long long kWaitBudgetCycles = 400000000LL;

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// Make generic-proxy shared-memory writes visible to the async proxy (TMA, tcgen05.mma).
__device__ __forceinline__ void fence_proxy_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Non-blocking probe of a phase.  Measured on B200: about 35 cycles, against about 170 for a
// try_wait that succeeds at once -- so every wait below asks this way first.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait: returns false (and raises *abort_flag) when the budget runs out or when
// another thread of the CTA has already given up.  The polling loop is kept out of line: with
// the loop inlined behind the probe, a wait that succeeds at once still cost about 100 cycles
// more in the single-thread pipeline loops (measured), presumably for the reconvergence code
// around a loop inside a one-lane branch.
static __device__ __noinline__ bool mbar_wait_poll(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    const long long start = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*abort_flag) return false;
        if (clock64() - start > kWaitBudgetCycles) {
            *abort_flag = 1;
            return false;
        }
    }
    return true;
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    if (mbar_test_wait(bar, parity)) return true;
    return mbar_wait_poll(bar, parity, abort_flag);
}

// Tile store shared -> global through a tensor map (elements outside the tensor are dropped).
// x times the element size must be a multiple of 16 bytes and no coordinate may be negative.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(
                     reinterpret_cast<uint64_t>(map)),
                 "r"(src), "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Until every bulk store this thread has committed has finished reading its shared-memory source.
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

// Untiled bulk copy global -> shared (both addresses 16-byte aligned, size a multiple of 16 bytes);
// completion is counted in bytes on the mbarrier.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y,
                                            uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, "
        "%3}], [%4];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, "
        "%3, %4, %5}], [%6];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

// ---- tcgen05 / tensor memory

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst),
                 "r"(ncols)
                 : "memory");
}

__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
                 : "memory");
}

__device__ __forceinline__ void tc_fence_before_sync()
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}

__device__ __forceinline__ void tc_fence_after_sync()
{
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// Arrive on an mbarrier once every MMA this thread issued so far has completed.
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}

// Shared-memory matrix descriptor of a K-major tile stored as 128-byte rows with the
// 128-byte swizzle (what a SWIZZLE_128B tensor map writes): 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((addr & 0x3FFFFu) >> 4);  // start address, 16-byte units
    d |= static_cast<uint64_t>(1) << 16;                 // leading byte offset (unused here)
    d |= static_cast<uint64_t>(1024 >> 4) << 32;         // stride between 8-row groups
    d |= static_cast<uint64_t>(1) << 46;                 // descriptor version of sm_100
    d |= static_cast<uint64_t>(2) << 61;                 // layout: 128-byte swizzle
    return d;
}

// D[tmem] (+)= A[smem] * B[smem]^T, signed 8-bit inputs, int32 accumulate.
__device__ __forceinline__ void mma_i8_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                          uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t"
        "}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Same with fp16 inputs and fp32 accumulate.
__device__ __forceinline__ void mma_f16_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                           uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t"
        "}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Instruction descriptor: dense, K-major A and B, M x N tile.
// c_format: 1 = f32, 2 = s32.  ab_format: kind::i8 -> 1 = signed 8-bit; kind::f16 -> 0 = f16.
__host__ __device__ constexpr uint32_t make_idesc(uint32_t c_format, uint32_t ab_format, uint32_t M,
                                                  uint32_t N)
{
    return (c_format << 4) | (ab_format << 7) | (ab_format << 10) | ((N >> 3) << 17) |
           ((M >> 4) << 24);
}

// 32 consecutive 32-bit columns of this warp's 32 TMEM lanes: thread i gets lane base+i.
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
          "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
          "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
          "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_ld_wait()
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Byte offset of 16-byte chunk `chunk` (0..7) of row `row` inside a 128-byte-swizzled tile.
__device__ __forceinline__ uint32_t sw128_offset(uint32_t row, uint32_t chunk)
{
    return row * 128u + ((chunk ^ (row & 7u)) << 4);
}

#endif  // __CUDACC__

}  // namespace mixdq
