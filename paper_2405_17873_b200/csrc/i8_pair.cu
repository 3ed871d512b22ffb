// Pair form of the W8A8 / W4A8 GEMM for the large layers: two CTAs on neighbouring SMs (a cluster of two)
// share one 256 x BN output tile and one stream of tensor-core instructions (tcgen05.mma.cta_group::2).
//
// Why: the single-CTA kernels in i8_tma.cu are bound by the bytes a CTA can keep in flight, not by the tensor
// pipe.  A 128 x 128 x 128 k-block needs 32 KB of operands (24 KB with int4 weights) for 256 cycles of MMA
// work, a ring slot is away for about 1900 cycles, and shared memory holds six such k-blocks: one k-block per
// 330 cycles at best.  In the pair form each CTA still loads its own 128 rows of activations per k-block but
// only HALF of the weight tile (BN / 2 rows), and one instruction covers 256 x BN x 32: at BN = 256 the same
// 32 KB per CTA feed 512 cycles of MMA work, so the rings run ahead of the tensor pipe instead of behind it,
// and the tensor pipe, not the operand delivery, sets the pace.
//
// Roles.  Both CTAs run the same program.  Activation and weight producers of BOTH CTAs load into their own
// shared memory and signal the barriers of the pair's first CTA (the leader) -- plain TMA loads of this GPU's
// memory with the cta_group::2 qualifier, which is what lets the barrier live in the peer CTA; nothing is
// multicast.  Two threads of the leader issue the MMAs, which read both CTAs' shared memory and write both
// CTAs' tensor memory (each CTA holds the 128 accumulator rows of its own activations), and hands slots back
// with commits that arrive on the barriers of both CTAs.  int4 weights are expanded by each CTA's own warps
// into its own half of the int8 weight tile; the peer's expansion warps arrive on the leader's barrier.  Each
// CTA's epilogue warps dequantize and store its own 128 rows.  Tiles are walked persistently with two
// accumulators of 256 columns each, so a tile's epilogue overlaps the next tile's main loop.
//
// BN is a run-time value (a multiple of 32 up to 256) chosen per layer so that the tiles fill whole rounds of
// the SM pairs; shared-memory slots have the size of the widest tile.
#include <mutex>

#include "i8_tiles.cuh"

namespace mixdq {
namespace i8 {

namespace {

// ---------------------------------------------------------------- PTX of the pair (cta_group::2) forms

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

// Address of this CTA's shared-memory location `addr` as seen in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank)
{
    uint32_t out;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(addr), "r"(rank));
    return out;
}

__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// D[tmem of both CTAs] (+)= A[both CTAs' smem, 128 rows each] * B[both CTAs' smem, N / 2 rows each]^T.
__device__ __forceinline__ void mma_i8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t"
        "}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// The same with fp16 operands and fp32 accumulation.
__device__ __forceinline__ void mma_f16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t"
        "}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
template <bool F16>
__device__ __forceinline__ void mma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate)
{
    if (F16)
        mma_f16_pair(d_tmem, a_desc, b_desc, idesc, accumulate);
    else
        mma_i8_pair(d_tmem, a_desc, b_desc, idesc, accumulate);
}

// Once every MMA this thread issued so far has completed: arrive on the barrier at this shared-memory offset
// in both CTAs of the pair (`both`: their bits in the cluster's CTA mask).
__device__ __forceinline__ void tc_commit_pair(uint32_t bar, uint16_t both)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
                 "h"(both)
                 : "memory");
}

// TMA tile loads into this CTA's shared memory whose completion is counted on a barrier of the leader CTA
// (`bar` is an address in the cluster's shared window).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                                 uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
        : "memory");
}

// Arrive on a barrier that may belong to the other CTA of the cluster (address in the cluster's shared
// window).  Default semantics, as for a local arrive: a release at cluster scope was measured to cost the
// arriving thread some 2000 cycles per call (it turned a 550-cycle expansion turn into a 2600-cycle one).
// What the arrival publishes are shared-memory tiles for the tensor core, and those are ordered by the
// fence.proxy.async that every writer executes before its warp's arrival.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}

// ---------------------------------------------------------------- shared memory of one CTA of the pair

constexpr int PAIR_BN_MAX = 256;
constexpr int ACC_COLS = 256;  // tensor-memory columns of one accumulator (the widest tile)

// MODE: 0 = int8 weights, 1 = int4 weights (expanded in shared memory), 2 = fp16 operands (kind::f16), 3 = fp16
// activations and packed 2- / 3- / 4-bit weights expanded to fp16 (code - zero) in shared memory; 4 / 5 = modes 0 / 1
// with two branches of k-blocks and an accumulator each (instances of their own, so that the one-branch kernels
// carry none of that code)
template <int MODE>
struct PairSmem {
    static constexpr bool W4 = MODE == 1 || MODE == 5;
    static constexpr bool TWO = MODE >= 4;  // two-branch instances (shortcut-splitting): 4 = int8, 5 = int4 weights
    static constexpr bool F16 = MODE == 2 || MODE == 3;
    static constexpr bool WO = MODE == 3;
    static constexpr bool PACKED = W4 || WO;  // a ring of packed weight tiles and expansion warps
    static constexpr int BKE = F16 ? BK / 2 : BK;           // elements of a k-block (its rows are 128 bytes either way)
    static constexpr int A_BYTES = BM * BK;                 // this CTA's 128 activation rows of a k-block
    static constexpr int B_BYTES = (PAIR_BN_MAX / 2) * BK;  // this CTA's half of the int8 weight tile
    // packed tiles.  int4 -> int8: one per k-block.  Weight-only: one per TWO k-blocks (128 codes: the bit-plane
    // formats store blocks of 128), 16 bytes per bit and row, at most 4 bits (8-bit weights keep the expansion pass).
    static constexpr int P_BYTES = B_BYTES / 2;
    // Depths: everything that is in flight from L2 as deep as shared memory allows; the expanded int8 tiles of
    // the W4 form are staging, one per expansion group.
    // W4: the packed ring must be deeper than the number of expansion groups, or the request for a group's
    // next tile goes out only when its last one has been expanded and the groups stall together once per lap.
    // Weight-only: a packed tile serves two consecutive k-blocks, i.e. two of the four expansion groups; with an
    // even number of packed slots a slot always belongs to the same two groups, which then meet every phase of its
    // barrier.
    static constexpr int AS = W4 ? 4 : 6;
    static constexpr int ES = PACKED ? 4 : 6;
    static constexpr int PS = W4 ? 8 : (WO ? 4 : 0);
    // Rings of equal depth move in lockstep: the commit that frees the activation slot of a k-block frees its weight
    // slot too (one commit per k-block instead of two; measured 4 to 7 % on the large int4 convolutions).
    static constexpr bool ONE_COMMIT = !PACKED || AS == ES;
    static constexpr int OFF_A = 0;
    static constexpr int OFF_B = OFF_A + AS * A_BYTES;
    static constexpr int OFF_P = OFF_B + ES * B_BYTES;
    static constexpr int RINGS_END = OFF_P + PS * P_BYTES;
    // barriers (8 bytes each).  FULL_A, READY_B, ACC_EMPTY are used in the leader only (both CTAs signal them);
    // the others exist in both CTAs and are signalled by the leader's commits or by local producers.
    static constexpr int FULL_A = 0;              // activation tiles of both CTAs have landed
    static constexpr int EMPTY_A = FULL_A + AS;   // MMAs reading the k-block's activation tiles (W8: and weights) have finished
    static constexpr int READY_B = EMPTY_A + AS;  // W8: weight halves of both CTAs have landed; W4: both expanded
    static constexpr int EMPTY_B = READY_B + ES;  // W4: MMAs reading the int8 weight tiles have finished
    static constexpr int FULL_P = EMPTY_B + ES;   // W4: this CTA's packed half has landed
    static constexpr int EMPTY_P = FULL_P + PS;   // W4: this CTA's packed half has been read
    static constexpr int ACC_FULL = EMPTY_P + PS;     // [2]
    static constexpr int ACC_EMPTY = ACC_FULL + 2;    // [2]
    static constexpr int TILE_GO = ACC_EMPTY + 2;     // leader: the first issuer has issued k-block 0 of a tile
    static constexpr int TILE_GO2 = TILE_GO + 1;      // leader, two-branch mode: the second branch's first k-block is issued
    static constexpr int NUM_BARS = TILE_GO2 + 1;
    static constexpr int OFF_BARS = RINGS_END;
    static constexpr int OFF_COMB = (OFF_BARS + NUM_BARS * 8 + 15) & ~15;  // [2][PAIR_BN_MAX] floats
    static constexpr int OFF_BIAS = OFF_COMB + 2 * PAIR_BN_MAX * 4;
    static constexpr int OFF_MISC = OFF_BIAS + 2 * PAIR_BN_MAX * 4;
    static constexpr int OFF_EPI = (OFF_MISC + 64 + 1023) & ~1023;  // staging tiles of the eight epilogue warps
    static constexpr int TOTAL = OFF_EPI + 8 * EPI32_TILE + 1024;
    static_assert(TOTAL <= 232448, "shared memory of one CTA");
    // warps: 0 activation producer, 1 MMA issuer (leader) and tensor-memory allocation, 2-5 epilogue (first part
    // of the columns), W4: 6-13 nibble expansion, then four epilogue helpers (the other columns), then the weight
    // producer
    static constexpr int HELPER0 = PACKED ? 14 : 6;
    static constexpr int B_WARP = HELPER0 + 4;
    static constexpr int MMA2_WARP = B_WARP + 1;  // second MMA issuer (leader)
    static constexpr int THREADS = (MMA2_WARP + 1) * 32;
};

struct PairArgs {
    int bn;           // tile width (multiple of 32, <= 256); each CTA holds bn / 2 weight rows
    int n_tiles;      // tiles along N
    int total_tiles;  // pair tiles in all
    int splits;       // > 1: one tile per cluster of 2 * splits CTAs, the reduction split over its CTA pairs
    // weight-only mode: width of the packed codes (2, 3, 4, 8), whether they are signed, per-channel zero-points
    // (nullptr for signed codes)
    int w_bits;
    int w_signed;
    const int32_t* w_zero;
    // two-branch mode (shortcut-splitting, Sec. 4.1; int8 modes, one tile per pair): kb_lo > 0 = the first kb_lo
    // k-blocks are the first branch (tmap_a / tmap_w, TmaParams' geometry and act_scale, accumulator 0), the others
    // the second branch (tmap_a2 / tmap_w2, the geometry below and *act_scale2, accumulator 1); the epilogue
    // stores (s_lo * acc_lo + s_hi * acc_hi) * s_w[n] + bias[n].  acc_out2: the second branch's sums (parity hook).
    int kb_lo;
    int cblocks2, Cin2;
    const float* act_scale2;
    int32_t* acc_out2;
};

// Grid (2 * splits * (pairs or tiles), 1, 1) with clusters of 2 * splits CTAs along x: CTAs 2 i and 2 i + 1 of a
// cluster are an MMA pair (a cluster of this kernel must be even along x: the launch is refused otherwise).  splits == 1: the pairs walk the tiles persistently.  splits > 1 (layers with too few tiles to fill
// the machine): one tile per cluster, pair i takes the i-th share of the reduction, every CTA leaves its 128 x bn
// partial sums in shared memory, and after a cluster barrier each CTA adds up its share of the rows over the
// pairs through distributed shared memory (integer adds: exact and order-free), dequantizes and stores.
template <int MODE>
__global__ void __launch_bounds__(PairSmem<MODE>::THREADS, 1)
pair_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                 const __grid_constant__ CUtensorMap tmap_y, const __grid_constant__ CUtensorMap tmap_a2,
                 const __grid_constant__ CUtensorMap tmap_w2, const TmaParams p, const PairArgs g)
{
    using L = PairSmem<MODE>;
    constexpr bool W4 = L::W4;
    constexpr bool F16 = L::F16;
    constexpr bool WO = L::WO;
    constexpr bool PACKED = L::PACKED;
    constexpr int BKE = L::BKE;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    uint8_t* sB = smem + L::OFF_B;
    const uint8_t* sP = smem + L::OFF_P;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BARS);
    float* s_comb = reinterpret_cast<float*>(smem + L::OFF_COMB);
    float* s_bias = reinterpret_cast<float*>(smem + L::OFF_BIAS);
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + L::OFF_MISC);
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + L::OFF_MISC + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t crank = cluster_ctarank();  // rank in the cluster: pair crank / 2, CTA crank % 2 of the pair
    const uint32_t rank = crank & 1u;          // 0: the pair's leader
    const uint32_t leader_rank = crank & ~1u;
    const bool leader = rank == 0;
    const int splits = g.splits, slice = static_cast<int>(crank >> 1);
    // (non-split: index of this pair and number of pairs; split: index of this cluster's tile)
    const int pair = static_cast<int>(blockIdx.x) / (2 * splits), npairs = static_cast<int>(gridDim.x) / (2 * splits);
    // this pair's share of the reduction (all of it unless the tile is split over the cluster)
    const int kb_begin = static_cast<int>((static_cast<long long>(p.k_blocks) * slice) / splits);
    const int nkb = static_cast<int>((static_cast<long long>(p.k_blocks) * (slice + 1)) / splits) - kb_begin;
    const int bn = g.bn, bh = g.bn >> 1;
    const int my_tiles = splits > 1 ? 1 : (g.total_tiles - pair + npairs - 1) / npairs;
    const uint16_t pair_mask = static_cast<uint16_t>(3u << leader_rank);  // the two CTAs of this pair
    const int kb_lo = L::TWO ? g.kb_lo : 0;  // > 0: two branches, two accumulators, one tile per pair

    const uint32_t bar0 = smem_u32(bars);
    const uint32_t a0 = smem_u32(smem + L::OFF_A), b0 = smem_u32(sB), p0 = smem_u32(smem + L::OFF_P);
    // the same barriers as seen in the leader CTA (for the leader: its own)
    const uint32_t lead_bar0 = map_to_cta(bar0, leader_rank);

    pdl_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < L::AS; ++s) {
            mbar_init(bar0 + 8 * (L::FULL_A + s), 1);   // the leader's producer arms it with the bytes of both CTAs
            mbar_init(bar0 + 8 * (L::EMPTY_A + s), 1);  // one commit
        }
        for (int s = 0; s < L::ES; ++s) {
            mbar_init(bar0 + 8 * (L::READY_B + s), PACKED ? 4 : 1);  // packed: two expansion warps of each CTA
            mbar_init(bar0 + 8 * (L::EMPTY_B + s), 1);
        }
        for (int s = 0; s < L::PS; ++s) {
            mbar_init(bar0 + 8 * (L::FULL_P + s), 1);
            mbar_init(bar0 + 8 * (L::EMPTY_P + s), WO ? 4 : 2);  // the warps of the group(s) that read the tile
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar0 + 8 * (L::ACC_FULL + b), 2);    // one commit of each issuer
            mbar_init(bar0 + 8 * (L::ACC_EMPTY + b), 16);  // eight epilogue warps of each CTA
        }
        mbar_init(bar0 + 8 * L::TILE_GO, 1);
        mbar_init(bar0 + 8 * L::TILE_GO2, 1);
        *s_abort = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_w);
        if (p.tma_store) tma_prefetch_desc(&tmap_y);
        if (kb_lo > 0) {
            tma_prefetch_desc(&tmap_a2);
            tma_prefetch_desc(&tmap_w2);
        }
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(s_tmem), 2 * ACC_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    // no CTA signals a barrier of its peer before that barrier exists
    cluster_sync();
    tc_fence_after_sync();
    // everything above is independent of earlier kernels; global memory is not, except the packed weights
    // (constants of the layer), whose producer runs ahead
    // (and the warps that expand them, which touch shared memory only)
    // (fp16 mode: the weight operand is the output of the expansion kernel launched just before: everyone waits)
    if ((MODE == 2 || warp != L::B_WARP) && !(PACKED && warp >= 6 && warp < L::HELPER0)) pdl_wait();
    const uint32_t tmem_base = *s_tmem;

    if (warp == 0) {
        // ------------------------------------------------------------ activation-tile producer (own 128 rows)
        if (lane == 0) {
            uint32_t s = 0, par = 1;  // slots start out free: the first lap waits on the phase "before" phase 0
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int tile = pair + t * npairs;
                const int m0 = (tile / g.n_tiles) * (2 * BM) + static_cast<int>(rank) * BM;
                int img_b = 0, ho0 = 0, wo0 = 0, cb = 0, kh = 0, kw = 0, xa = kb_begin * BKE;
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
                const CUtensorMap* map = &tmap_a;
                int cblocks = p.cblocks;
                for (int i = 0; i < nkb; ++i) {
                    if (kb_lo > 0 && i == kb_lo) {  // second branch: its own map, from its first k-block
                        map = &tmap_a2;
                        cblocks = g.cblocks2;
                        cb = kh = kw = 0;
                        xa = 0;
                    }
                    if (!mbar_wait(bar0 + 8 * (L::EMPTY_A + s), par, s_abort)) {
                        ok = false;
                        break;
                    }
                    if (leader) mbar_arrive_expect_tx(bar0 + 8 * (L::FULL_A + s), 2 * L::A_BYTES);
                    const uint32_t full = lead_bar0 + 8 * (L::FULL_A + s);
                    if (p.conv) {
                        tma_load_4d_pair(a0 + s * L::A_BYTES, map, cb * BKE, p.stride * wo0 + kw - 1 + p.pad,
                                         p.stride * ho0 + kh - 1 + p.pad, img_b, full);
                        if (++cb == cblocks) {
                            cb = 0;
                            if (++kw == 3) {
                                kw = 0;
                                ++kh;
                            }
                        }
                    } else {
                        tma_load_2d_pair(a0 + s * L::A_BYTES, map, xa, m0, full);
                        xa += BKE;
                    }
                    if (++s == L::AS) {
                        s = 0;
                        par ^= 1;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == L::B_WARP) {
        // ------------------------------------------------------------ weight-tile producer (own half of the rows)
        if (lane == 0 && WO) {
            // packed tiles of 128 codes (two k-blocks), this CTA's half of the tile's rows; the reduction is never
            // split in this mode, so a tile's k-blocks start at 0
            constexpr uint32_t PS = L::PS > 0 ? L::PS : 1;
            const int unit_bytes = 16 * g.w_bits;
            const int units = (nkb + 1) >> 1;
            uint32_t s = 0, par = 1;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int tile = pair + t * npairs;
                const int n0 = (tile % g.n_tiles) * bn + static_cast<int>(rank) * bh;
                for (int u = 0; u < units; ++u) {
                    if (!mbar_wait(bar0 + 8 * (L::EMPTY_P + s), par, s_abort)) {
                        ok = false;
                        break;
                    }
                    const uint32_t full = bar0 + 8 * (L::FULL_P + s);
                    mbar_arrive_expect_tx(full, static_cast<uint32_t>(bh * unit_bytes));
                    tma_load_2d(p0 + s * L::P_BYTES, &tmap_w, u * unit_bytes, n0, full);
                    if (++s == PS) {
                        s = 0;
                        par ^= 1;
                    }
                }
            }
        } else if (lane == 0) {
            constexpr int R = W4 ? L::PS : L::ES;
            constexpr int ROW_BYTES = W4 ? BK / 2 : BK;   // bytes of a k-block of one weight row
            constexpr int ROW_STEP = F16 ? BKE : ROW_BYTES;  // the same in units of the weight map's element
            uint32_t s = 0, par = 1;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int tile = pair + t * npairs;
                const int n0 = (tile % g.n_tiles) * bn + static_cast<int>(rank) * bh;
                int cb = 0, kx_tap = 0, xb = kb_begin * ROW_STEP;
                if (p.conv) {
                    const int tap = kb_begin / p.cblocks;
                    cb = kb_begin - tap * p.cblocks;
                    kx_tap = tap * p.Cin;  // first reduction index of the filter tap
                }
                const CUtensorMap* map = &tmap_w;
                int cblocks = p.cblocks, cin = p.Cin;
                for (int i = 0; i < nkb; ++i) {
                    if (kb_lo > 0 && i == kb_lo) {  // second branch: its own packed matrix, from its first k-block
                        map = &tmap_w2;
                        cblocks = g.cblocks2;
                        cin = g.Cin2;
                        cb = kx_tap = 0;
                        xb = 0;
                    }
                    // W8: the commit that frees the activation slot frees the weight slot (the rings move in lockstep)
                    if (!mbar_wait(bar0 + 8 * ((W4 ? L::EMPTY_P : L::EMPTY_A) + s), par, s_abort)) {
                        ok = false;
                        break;
                    }
                    int x = xb;
                    if (p.conv) {
                        const int kx = kx_tap + cb * BKE;
                        x = W4 ? kx / 2 : kx;
                        if (++cb == cblocks) {
                            cb = 0;
                            kx_tap += cin;
                        }
                    }
                    xb += ROW_STEP;
                    if (W4) {
                        // packed rows are consumed inside this CTA: a barrier of its own
                        const uint32_t full = bar0 + 8 * (L::FULL_P + s);
                        mbar_arrive_expect_tx(full, static_cast<uint32_t>(bh * ROW_BYTES));
                        tma_load_2d(p0 + s * L::P_BYTES, map, x, n0, full);
                    } else {
                        if (leader) mbar_arrive_expect_tx(bar0 + 8 * (L::READY_B + s), static_cast<uint32_t>(bn * ROW_BYTES));
                        tma_load_2d_pair(b0 + s * L::B_BYTES, map, x, n0, lead_bar0 + 8 * (L::READY_B + s));
                    }
                    if (++s == R) {
                        s = 0;
                        par ^= 1;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1 || warp == L::MMA2_WARP) {
        // ------------------------------------------------------------ MMA issuers (two threads of the leader)
        // One thread needs some 650 cycles per k-block (four MMAs at about 62 cycles each, two waits, a commit
        // whose cost to its thread is several times an MMA's, the loop) against 512 cycles of tensor-pipe work,
        // and the pipe idles whenever its queue runs dry in between.  Two threads therefore alternate: warp 1
        // takes the even k-blocks of a tile, the second issuer the odd ones, both into the SAME accumulator --
        // the sums are integers, so the order in which the pipe adds the k-blocks does not matter, except that
        // the MMA that overwrites the accumulator (the first of k-block 0) must come first: the second issuer
        // starts a tile only after the first has issued k-block 0 (TILE_GO, with the tcgen05 fences that order
        // the two threads' instructions).  A tile is complete when both threads' commits have arrived.
        if (lane == 0 && leader) {
            const int which = warp == 1 ? 0 : 1;
            const uint32_t idesc = F16 ? make_idesc(1, 0, 2 * BM, static_cast<uint32_t>(bn))
                                       : make_idesc(2, 1, 2 * BM, static_cast<uint32_t>(bn));
            const uint64_t a_desc0 = smem_desc_sw128(a0), b_desc0 = smem_desc_sw128(b0);
            const uint32_t tile_go = bar0 + 8 * L::TILE_GO;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int buf = t & 1;
                const uint32_t use = static_cast<uint32_t>(t >> 1);  // how often this accumulator was used before
                ok = mbar_wait(bar0 + 8 * (L::ACC_EMPTY + buf), (use & 1) ^ 1, s_abort);
                if (!ok) break;
                if (which == 1 && nkb > 1) {
                    ok = mbar_wait(tile_go, t & 1, s_abort);
                    if (!ok) break;
                }
                tc_fence_after_sync();
                const uint32_t acc = tmem_base + buf * ACC_COLS;
                // position of this thread's first k-block of the tile in the CTA's running sequence
                uint32_t q = static_cast<uint32_t>(t) * static_cast<uint32_t>(nkb) + which;
                uint32_t sa = q % L::AS, pa = (q / L::AS) & 1, se = q % L::ES, pe = (q / L::ES) & 1;
                for (int i = which; i < nkb; i += 2) {
                    if (!mbar_wait(bar0 + 8 * (L::FULL_A + sa), pa, s_abort) ||
                        !mbar_wait(bar0 + 8 * (L::READY_B + se), pe, s_abort)) {
                        ok = false;
                        break;
                    }
                    // two-branch mode: the second branch's k-blocks go to the other accumulator, whose overwriting
                    // MMA (first of k-block kb_lo) must precede the other thread's first addition to it
                    const bool second = kb_lo > 0 && i >= kb_lo;
                    if (second && i == kb_lo + 1 && !mbar_wait(bar0 + 8 * L::TILE_GO2, 0, s_abort)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint64_t a_desc = a_desc0 + sa * (L::A_BYTES >> 4);
                    const uint64_t b_desc = b_desc0 + se * (L::B_BYTES >> 4);
                    const uint32_t acc_i = second ? tmem_base + ACC_COLS : acc;
                    // four instructions of 32 bytes along the reduction: 32 int8 or 16 fp16 elements each
                    mma_pair<F16>(acc_i, a_desc, b_desc, idesc, i != 0 && !(second && i == kb_lo));
#pragma unroll
                    for (int k = 1; k < BK / 32; ++k) mma_pair<F16>(acc_i, a_desc + 2 * k, b_desc + 2 * k, idesc, 1u);
                    if (i == 0 && nkb > 1) {
                        // the overwriting MMA is in the pipe's queue: the other thread may add to the accumulator
                        tc_fence_before_sync();
                        mbar_arrive(tile_go);
                    }
                    if (second && i == kb_lo) {
                        tc_fence_before_sync();
                        mbar_arrive(bar0 + 8 * L::TILE_GO2);
                    }
                    tc_commit_pair(bar0 + 8 * (L::EMPTY_A + sa), pair_mask);
                    if (!L::ONE_COMMIT) tc_commit_pair(bar0 + 8 * (L::EMPTY_B + se), pair_mask);
                    sa += 2;
                    if (sa >= static_cast<uint32_t>(L::AS)) {
                        sa -= L::AS;
                        pa ^= 1;
                    }
                    se += 2;
                    if (se >= static_cast<uint32_t>(L::ES)) {
                        se -= L::ES;
                        pe ^= 1;
                    }
                }
                // (a thread without a k-block in this tile still arrives: its commit has nothing to wait for)
                if (ok) tc_commit_pair(bar0 + 8 * (L::ACC_FULL + buf), pair_mask);
            }
        }
        __syncwarp();
    } else if (warp < 6 || (warp >= L::HELPER0 && warp < L::HELPER0 + 4)) {
        // ------------------------------------------------------------ epilogue warps and helpers (own 128 rows)
        const int lg = warp & 3;
        const int half = warp < 6 ? 0 : 1;
        const int et = tid - 64;  // epilogue warps only: 0..127
        // (fp16 mode: the activations are not quantized, the factor of a column is its weight scale)
        const float sx = F16 ? 1.f : (p.act_scale ? __ldg(p.act_scale) : 0.f);  // absent: accumulators only
        const int zshift = p.act_zero ? 128 - __ldg(p.act_zero) : 0;
        // the 32-column passes of a tile are dealt to the two halves of the warps
        const int passes = bn >> 5;
        const int c_begin = half == 0 ? 0 : ((passes + 1) >> 1) * 32;
        const int c_count = half == 0 ? ((passes + 1) >> 1) * 32 : (passes >> 1) * 32;
        uint8_t* stage = smem + L::OFF_EPI + (half * 4 + lg) * EPI32_TILE;
        const uint32_t lead_acc_empty = lead_bar0 + 8 * L::ACC_EMPTY;
        bool ok = true;
        for (int t = 0; t < my_tiles; ++t) {
            const int tile = pair + t * npairs;
            const int m0 = (tile / g.n_tiles) * (2 * BM) + static_cast<int>(rank) * BM, n0 = (tile % g.n_tiles) * bn;
            const int buf = t & 1;
            const uint32_t use = static_cast<uint32_t>(t >> 1);
            float* comb = s_comb + buf * PAIR_BN_MAX;
            float* bias = s_bias + buf * PAIR_BN_MAX;
            // this tile's per-column factors (the buffer was last read two tiles ago)
            for (int j = et; half == 0 && j < bn; j += 128) {
                const int n = n0 + j;
                float c = 0.f, b = 0.f;
                if (n < p.N && p.w_scale) {
                    c = sx * __ldg(p.w_scale + n);
                    if (p.bias) b = __half2float(p.bias[n]);
                    if (p.act_zero) b = fmaf(static_cast<float>(zshift * __ldg(p.w_code_sums + n)), c, b);
                }
                comb[j] = c;
                bias[j] = b;
                // two-branch mode (one tile): the second table holds the second branch's factors
                if (kb_lo > 0) s_comb[PAIR_BN_MAX + j] = (n < p.N && p.w_scale) ? __ldg(g.act_scale2) * __ldg(p.w_scale + n) : 0.f;
            }
            if (ok) ok = mbar_wait(bar0 + 8 * (L::ACC_FULL + buf), use & 1, s_abort);
            tc_fence_after_sync();
            // the factor tables are complete; the same barrier carries the vote on whether every warp's wait
            // succeeded, so that all eight take the same path from here
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
            const uint32_t acc = tmem_base + buf * ACC_COLS + (static_cast<uint32_t>(lg * 32) << 16);
            if (splits > 1) {
                // this pair's share of the sums: tensor memory -> registers -> shared memory (the drained pipeline
                // buffers), rows bn * 4 bytes apart, 16-byte chunks XOR-swizzled by row; reduced below
                const int row = lg * 32 + lane;
                uint8_t* prow = smem + row * (bn * 4);
                for (int c0 = c_begin; c0 < c_begin + c_count; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld_32x32(acc + c0, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int chunk = (c0 >> 2) + j;
                        *reinterpret_cast<uint4*>(prow + ((chunk ^ (row & 7)) << 4)) =
                            make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
                    }
                }
            } else if (!F16 && p.acc_out) {
                // raw int32 sums (parity hook): a lane owns a row, 32 columns of it at a time
                const int m = m0 + lg * 32 + lane;
                for (int c0 = c_begin; c0 < c_begin + c_count; c0 += 32) {
                    if (n0 + c0 >= p.N) break;  // uniform across the warp
                    uint32_t r[32];
                    tmem_ld_32x32(acc + c0, r);
                    tmem_ld_wait();
                    if (m < p.M) {
                        int32_t* dst = p.acc_out + static_cast<long long>(m) * p.N + n0 + c0;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (n0 + c0 + j < p.N) {
                                int32_t v = W4 ? (static_cast<int32_t>(r[j]) >> 4) : static_cast<int32_t>(r[j]);
                                if (p.act_zero) v += zshift * __ldg(p.w_code_sums + n0 + c0 + j);
                                dst[j] = v;
                            }
                        }
                    }
                    if (kb_lo > 0 && g.acc_out2) {
                        tmem_ld_32x32(acc + ACC_COLS + c0, r);
                        tmem_ld_wait();
                        if (m < p.M) {
                            int32_t* dst = g.acc_out2 + static_cast<long long>(m) * p.N + n0 + c0;
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (n0 + c0 + j < p.N) dst[j] = W4 ? (static_cast<int32_t>(r[j]) >> 4) : static_cast<int32_t>(r[j]);
                        }
                    }
                }
            }
            if (splits == 1 && p.Y && c_count > 0) {
                if (F16)
                    store_rows32_f32(acc + c_begin, c_count, comb + c_begin, bias + c_begin, stage, p, &tmap_y,
                                     m0 + lg * 32, n0 + c_begin, lane);
                else if (kb_lo > 0)
                    store_rows32_two<W4>(acc + c_begin, ACC_COLS, c_count, comb + c_begin, s_comb + PAIR_BN_MAX + c_begin,
                                         bias + c_begin, stage, p, &tmap_y, m0 + lg * 32, n0 + c_begin, lane);
                else
                    store_rows32_dispatch<W4>(acc + c_begin, 0, c_count, comb + c_begin, bias + c_begin, stage, p, &tmap_y,
                                              m0 + lg * 32, n0 + c_begin, lane);
            }
            // the accumulator may be overwritten once every epilogue warp of both CTAs has read it
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(lead_acc_empty + 8 * buf);
        }
        if (p.tma_store && lane == 0) tma_store_wait_read();  // shared memory stays valid until then
    } else if (WO && warp >= 6 && warp < L::HELPER0) {
        // ------------------------------------------------------------ packed codes -> fp16 (code - zero), own half
        // Four groups of two warps as below; group g takes the k-blocks g, g + 4, ... of the CTA's sequence and owns
        // slot g of the fp16 weight ring.  A thread turns eight codes of a row into one 16-byte chunk of the
        // swizzled tile: 1024 + u is the fp16 bit pattern 0x6400 | u for an integer u < 1024, so the difference
        // (1024 + u) - (1024 + zero) is exact and the weights enter the MMA as exact integers.
        const int group = (warp - 6) >> 1;
        const int gt = tid - 192 - group * 64;  // 0..63 within the group
        const int total_kb = my_tiles * nkb;
        const int units = (nkb + 1) >> 1;
        const int unit_bytes = 16 * g.w_bits;
        constexpr uint32_t PS = L::PS > 0 ? L::PS : 1;
        const uint32_t lead_ready = lead_bar0 + 8 * (L::READY_B + group);
        uint8_t* b_stage = sB + group * L::B_BYTES;
        uint32_t n = 0;
        int z_tile = -1;
        __half2 z2r[2] = {__half2half2(__ushort_as_half(0x6400)), __half2half2(__ushort_as_half(0x6400))};
        for (int it = group; it < total_kb; it += 4, ++n) {
            const int t = it / nkb, kbi = it - t * nkb;
            const uint32_t useq = static_cast<uint32_t>(t * units + (kbi >> 1));  // packed tile in the CTA's sequence
            const uint32_t sp = useq % PS, rp = useq / PS;
            const uint8_t* stg = sP + sp * L::P_BYTES;
            bool ok = mbar_wait(bar0 + 8 * (L::FULL_P + sp), rp & 1, s_abort);
            if (ok && n > 0) ok = mbar_wait(bar0 + 8 * ((L::ONE_COMMIT ? L::EMPTY_A : L::EMPTY_B) + group), (n & 1) ^ 1, s_abort);
            if (!__all_sync(0xffffffffu, ok)) break;  // the warp leaves together
            const int kofs = (kbi & 1) * 64;  // which half of the packed tile's 128 codes
            if (t != z_tile) {
                // zero-points of this thread's rows (rows gt and gt + 64 of the CTA's half tile), as fp16 1024 + zero
                // (+ the offset that moved signed codes into the unsigned range)
                z_tile = t;
                const int tile = pair + t * npairs;
                const int n_first = (tile % g.n_tiles) * bn + static_cast<int>(rank) * bh;
                const int code_bias = g.w_signed ? 8 : 0;
#pragma unroll
                for (int rr = 0; rr < 2; ++rr) {
                    const int nrow = n_first + gt + 64 * rr;
                    const int z = (g.w_zero && nrow < p.N) ? __ldg(g.w_zero + nrow) : 0;
                    z2r[rr] = __half2half2(__ushort_as_half(static_cast<unsigned short>(0x6400 + z + code_bias)));
                }
            }
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                const int r = gt + 64 * rr;
                if (r >= bh) break;
                const uint8_t* prow = stg + r * unit_bytes;
                // the row's 64 codes as eight pairs of byte words (codes 8 j .. 8 j + 3, 8 j + 4 .. 8 j + 7)
                uint32_t lo4[8], hi4[8];
                {
                    uint32_t w[8];  // eight codes per word, byte i = code i (low nibble) | code i + 4 (high nibble)
                    if (g.w_bits == 4) {
                        const uint4* src = reinterpret_cast<const uint4*>(prow + (kofs >> 1));
                        const uint4 v0 = src[0], v1 = src[1];
                        const uint32_t flip = g.w_signed ? 0x88888888u : 0u;
                        w[0] = v0.x ^ flip; w[1] = v0.y ^ flip; w[2] = v0.z ^ flip; w[3] = v0.w ^ flip;
                        w[4] = v1.x ^ flip; w[5] = v1.y ^ flip; w[6] = v1.z ^ flip; w[7] = v1.w ^ flip;
                    } else {
                        // bit planes: 16 bytes per bit and 128 codes; the two words of each plane that hold this half
                        const uint8_t* base = prow + (kofs >> 5) * 4;
                        const uint2 p0 = *reinterpret_cast<const uint2*>(base);
                        const uint2 p1 = *reinterpret_cast<const uint2*>(base + 16);
                        uint2 p2 = make_uint2(0u, 0u);
                        if (g.w_bits == 3) p2 = *reinterpret_cast<const uint2*>(base + 32);
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const int sft = j & 3;
                            const uint32_t a0 = j < 4 ? p0.x : p0.y, a1 = j < 4 ? p1.x : p1.y, a2 = j < 4 ? p2.x : p2.y;
                            w[j] = ((a0 >> sft) & 0x11111111u) | (((a1 >> sft) & 0x11111111u) << 1) |
                                   (((a2 >> sft) & 0x11111111u) << 2);
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        lo4[j] = w[j] & 0x0F0F0F0Fu;
                        hi4[j] = (w[j] >> 4) & 0x0F0F0F0Fu;
                    }
                }
                const __half2 z2 = z2r[rr];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    // byte u -> fp16 bits 0x64uu = 1024 + u, two at a time; minus 1024 + zero: exact
                    uint32_t h[4] = {__byte_perm(lo4[j], 0x64646464u, 0x5140), __byte_perm(lo4[j], 0x64646464u, 0x7362),
                                     __byte_perm(hi4[j], 0x64646464u, 0x5140), __byte_perm(hi4[j], 0x64646464u, 0x7362)};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const __half2 d = __hsub2(*reinterpret_cast<const __half2*>(&h[q]), z2);
                        h[q] = *reinterpret_cast<const uint32_t*>(&d);
                    }
                    *reinterpret_cast<uint4*>(b_stage + sw128_offset(r, j)) = make_uint4(h[0], h[1], h[2], h[3]);
                }
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive_cluster(lead_ready);
                // the packed tile is free once both of its k-blocks are expanded (four warps); the lone k-block of
                // a tile with an odd number arrives for the missing one too
                mbar_arrive(bar0 + 8 * (L::EMPTY_P + sp));
                if ((kbi & 1) == 0 && kbi == nkb - 1) mbar_arrive(bar0 + 8 * (L::EMPTY_P + sp));
            }
        }
    } else if (W4 && warp >= 6 && warp < L::HELPER0) {
        // ------------------------------------------------------------ int4 -> int8 (x16) expansion, own half
        // Four groups of two warps; group g takes the k-blocks g, g + 4, ... of the CTA's sequence and owns slot g
        // of the packed ring and of the int8 ring.  Nibble -> high half of the byte (= 16 q): two ANDs and a
        // shift per 8 codes; the factor 16 leaves in the epilogue by an exact shift.
        const int group = (warp - 6) >> 1;
        const int gt = tid - 192 - group * 64;  // 0..63 within the group
        const int total_kb = my_tiles * nkb;
        const int runs = bh * 4;  // 16-byte packed runs of this CTA's half tile
        constexpr uint32_t PS = L::PS > 0 ? L::PS : 1;
        const uint32_t lead_ready = lead_bar0 + 8 * (L::READY_B + group);
        uint8_t* b_stage = sB + group * L::B_BYTES;
        static_assert(!W4 || L::ES == 4, "one int8 slot per expansion group");
        uint32_t n = 0;  // turns taken
        for (int it = group; it < total_kb; it += 4, ++n) {
            const uint32_t sp = static_cast<uint32_t>(it) % PS, rp = static_cast<uint32_t>(it) / PS;
            const uint8_t* stg = sP + sp * L::P_BYTES;
            bool ok = mbar_wait(bar0 + 8 * (L::FULL_P + sp), rp & 1, s_abort);
            if (ok && n > 0) ok = mbar_wait(bar0 + 8 * ((L::ONE_COMMIT ? L::EMPTY_A : L::EMPTY_B) + group), (n & 1) ^ 1, s_abort);
            if (!__all_sync(0xffffffffu, ok)) break;  // the warp leaves together
            // all loads first: the compiler cannot move a load above a store to the other ring by itself
            uint4 wv[8];
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const int task = gt + t * 64;
                wv[t] = task < runs ? *reinterpret_cast<const uint4*>(stg + task * 16) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const int task = gt + t * 64;
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
                mbar_arrive_cluster(lead_ready);
                mbar_arrive(bar0 + 8 * (L::EMPTY_P + sp));
            }
        }
    }

    if (splits > 1) {
        // ------------------------------------------------------------ reduction over the pairs of the cluster
        // CTA (pair `slice`, rank r) adds up rows [slice * ceil(128 / splits), ...) of the rank-r halves of all
        // pairs; consecutive threads take consecutive groups of four columns, so stores coalesce.
        __syncthreads();
        cluster_sync();
        if (!*s_abort) {
            const int tile = pair;
            const int m_base = (tile / g.n_tiles) * (2 * BM) + static_cast<int>(rank) * BM, n0 = (tile % g.n_tiles) * bn;
            const int rows_per = (BM + splits - 1) / splits;
            const int r0 = slice * rows_per;
            const int r1 = r0 + rows_per < BM ? r0 + rows_per : BM;
            const int chunks = bn >> 2;
            const float* comb = s_comb;  // accumulator 0's tables
            const float* bias = s_bias;
            const int zshift = p.act_zero ? 128 - __ldg(p.act_zero) : 0;
            const uint32_t base = smem_u32(smem);
            for (int idx = tid; idx < (r1 - r0) * chunks; idx += L::THREADS) {
                const int row = r0 + idx / chunks, chunk = idx % chunks;
                const int m = m_base + row, n = n0 + chunk * 4;
                if (m >= p.M || n >= p.N) continue;
                const uint32_t off = base + row * (bn * 4) + ((chunk ^ (row & 7)) << 4);
                int4 acc = make_int4(0, 0, 0, 0);
                float4 facc = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int q = 0; q < splits; ++q) {
                    uint32_t remote;
                    asm("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(off), "r"(2 * q + static_cast<int>(rank)));
                    int4 v;
                    asm volatile("ld.shared::cluster.v4.s32 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                                 : "r"(remote));
                    if (F16) {
                        facc.x += __int_as_float(v.x);
                        facc.y += __int_as_float(v.y);
                        facc.z += __int_as_float(v.z);
                        facc.w += __int_as_float(v.w);
                    } else {
                        acc.x += v.x;
                        acc.y += v.y;
                        acc.z += v.z;
                        acc.w += v.w;
                    }
                }
                const int a[4] = {acc.x, acc.y, acc.z, acc.w};
                const float f[4] = {facc.x, facc.y, facc.z, facc.w};
                if (!F16 && p.acc_out) {
                    int32_t* dst = p.acc_out + static_cast<long long>(m) * p.N + n;
                    for (int j = 0; j < 4; ++j)
                        if (n + j < p.N)
                            dst[j] = (W4 ? (a[j] >> 4) : a[j]) + (p.act_zero ? zshift * __ldg(p.w_code_sums + n + j) : 0);
                }
                if (p.Y) {
                    __half h[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float v = F16 ? f[j] : acc_to_float<W4, false>(static_cast<uint32_t>(a[j]));
                        h[j] = __float2half_rn(fmaf(v, comb[chunk * 4 + j], bias[chunk * 4 + j]));
                    }
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
    }

    if (*s_abort) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        if (tid == 0 && p.status) atomicExch(p.status, MIXDQ_ERR_TIMEOUT);
    }
    // neither CTA leaves (or frees tensor memory) while its peer may still read its shared memory, signal its
    // barriers or run instructions that write its tensor memory
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync();
    if (warp == 1) tmem_dealloc_pair(tmem_base, 2 * ACC_COLS);
}

template <int MODE>
int launch_pair_t(const CUtensorMap& ta, const CUtensorMap& tw, const CUtensorMap& ty, const TmaParams& tp, int bn, int splits,
                  int num_sms, cudaStream_t stream, int w_bits = 0, const int32_t* w_zero = nullptr,
                  const PairBranch* second = nullptr)
{
    using L = PairSmem<MODE>;
    auto kernel = pair_gemm_kernel<MODE>;
    if (ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), L::TOTAL) != MIXDQ_OK) return MIXDQ_ERR_CUDA;
    PairArgs g;
    g.bn = bn;
    g.n_tiles = static_cast<int>(ceil_div(tp.N, bn));
    g.total_tiles = g.n_tiles * static_cast<int>(ceil_div(tp.M, 2 * BM));
    g.splits = splits;
    g.w_bits = w_bits;
    g.w_signed = w_zero ? 0 : 1;
    g.w_zero = w_zero;
    g.kb_lo = 0;
    g.cblocks2 = g.Cin2 = 0;
    g.act_scale2 = nullptr;
    g.acc_out2 = nullptr;
    if (second) {
        g.kb_lo = second->kb_first;
        g.cblocks2 = second->cblocks;
        g.Cin2 = second->Cin;
        g.act_scale2 = second->act_scale;
        g.acc_out2 = second->acc_out;
    }
    // persistent pairs; one cluster of `splits` pairs per tile; two-branch mode: one pair per tile (both
    // accumulators belong to the tile)
    const int pairs = (splits > 1 || second) ? g.total_tiles : (g.total_tiles < num_sms / 2 ? g.total_tiles : num_sms / 2);
    return launch_pdl_cluster(kernel, dim3(static_cast<unsigned>(2 * splits * pairs)), dim3(L::THREADS), L::TOTAL, stream,
                              static_cast<unsigned>(2 * splits), 1u, ta, tw, ty, second ? *second->ta : ta,
                              second ? *second->tw : tw, tp, g);
}

}  // namespace

// How many clusters of `cluster_ctas` CTAs of the pair kernel the device holds at once (a cluster lives inside one
// GPC, so this is well below SMs / cluster_ctas for the larger clusters); asked of the occupancy calculator once per
// device, width and cluster size.  0 on error.
int pair_cluster_capacity(bool w4, int cluster_ctas)
{
    static std::mutex mu;
    static int cache[64][2][9] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64 || cluster_ctas < 2 || cluster_ctas > 8) return 0;
    std::lock_guard<std::mutex> lock(mu);
    int& slot = cache[dev][w4 ? 1 : 0][cluster_ctas];
    if (slot == 0) {
        const void* kernel = w4 ? reinterpret_cast<const void*>(pair_gemm_kernel<1>) : reinterpret_cast<const void*>(pair_gemm_kernel<0>);
        const int smem = w4 ? PairSmem<1>::TOTAL : PairSmem<0>::TOTAL;
        const int threads = w4 ? PairSmem<1>::THREADS : PairSmem<0>::THREADS;
        if (ensure_dynamic_smem(kernel, smem) != MIXDQ_OK) return 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(cluster_ctas) * 64);
        cfg.blockDim = dim3(static_cast<unsigned>(threads));
        cfg.dynamicSmemBytes = static_cast<size_t>(smem);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = static_cast<unsigned>(cluster_ctas);
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess) {
            (void)cudaGetLastError();
            return 0;
        }
        slot = n > 0 ? n : -1;
    }
    return slot > 0 ? slot : 0;
}

int launch_pair(const CUtensorMap& ta, const CUtensorMap& tw, const CUtensorMap& ty, const TmaParams& tp, bool w4, int bn,
                int splits, int num_sms, cudaStream_t stream)
{
    if (bn < 32 || bn > PAIR_BN_MAX || bn % 32 != 0 || num_sms < 2 || splits < 1 || splits > 4 || splits > tp.k_blocks)
        return MIXDQ_ERR_INVALID_ARG;
    return w4 ? launch_pair_t<1>(ta, tw, ty, tp, bn, splits, num_sms, stream)
              : launch_pair_t<0>(ta, tw, ty, tp, bn, splits, num_sms, stream);
}

int launch_pair_two(const CUtensorMap& ta, const CUtensorMap& tw, const CUtensorMap& ty, const TmaParams& tp, bool w4, int bn,
                    const PairBranch& second, int num_sms, cudaStream_t stream)
{
    // tp.k_blocks counts both branches' k-blocks; a split reduction and asymmetric activations are not supported
    if (bn < 32 || bn > PAIR_BN_MAX || bn % 32 != 0 || num_sms < 2 || second.kb_first < 1 || second.kb_first >= tp.k_blocks ||
        !second.ta || !second.tw || !second.act_scale || tp.act_zero || tp.addend || tp.bos)
        return MIXDQ_ERR_INVALID_ARG;
    return w4 ? launch_pair_t<5>(ta, tw, ty, tp, bn, 1, num_sms, stream, 0, nullptr, &second)
              : launch_pair_t<4>(ta, tw, ty, tp, bn, 1, num_sms, stream, 0, nullptr, &second);
}

int launch_pair_f16(const CUtensorMap& ta, const CUtensorMap& tw, const CUtensorMap& ty, const TmaParams& tp, int bn,
                    int splits, int num_sms, cudaStream_t stream)
{
    if (bn < 32 || bn > PAIR_BN_MAX || bn % 32 != 0 || num_sms < 2 || tp.acc_out || splits < 1 || splits > 4 ||
        splits > tp.k_blocks)
        return MIXDQ_ERR_INVALID_ARG;
    return launch_pair_t<2>(ta, tw, ty, tp, bn, splits, num_sms, stream);
}

int launch_pair_wo(const CUtensorMap& ta, const CUtensorMap& tw, const CUtensorMap& ty, const TmaParams& tp, int bn,
                   int w_bits, const int32_t* w_zero, int num_sms, cudaStream_t stream)
{
    if (bn < 32 || bn > PAIR_BN_MAX || bn % 32 != 0 || num_sms < 2 || tp.acc_out || tp.k_blocks < 1)
        return MIXDQ_ERR_INVALID_ARG;
    if (w_bits != 2 && w_bits != 3 && w_bits != 4) return MIXDQ_ERR_UNSUPPORTED;
    if (w_bits <= 3 && !w_zero) return MIXDQ_ERR_UNSUPPORTED;  // bit-plane codes are unsigned
    return launch_pair_t<3>(ta, tw, ty, tp, bn, 1, num_sms, stream, w_bits, w_zero);
}

}  // namespace i8
}  // namespace mixdq
