// libmars: LM-head projection fused with the top-2 epilogue and the verification tail.
//
// z = H W^T (+ b)  (Eq. 2 of the paper: z_t = W_o h_t + b_o), H bf16 [M, d], W bf16 [V, d],
// fp32 accumulation in tensor memory.  The logits are never written to HBM: each epilogue
// thread owns one logits row (one TMEM lane) and keeps that row's running top-2 across the
// vocabulary tiles it sees; 16-byte records go to the workspace and a small second kernel
// merges them per row and runs the verification tail.
//
// Kernel 1 comes in two forms with the same pipeline (192 threads, warp-specialised):
//   lmhead_top2_kernel_pair  (default) clusters of two blocks sharing tcgen05.mma.cta_group::2,
//                            M = 256 per pair; see the comment above that kernel.
//   lmhead_top2_kernel       one block per SM, cta_group::1, M = 128 (test hook / fallback).
//   warp 0      TMA producer: H tile [128 x 64] and W tile [256 x 64] (128-byte swizzle) per
//               k-block into a shared-memory ring, completion on mbarriers.
//   warp 1      allocates the 512 TMEM columns and issues tcgen05.mma (N=256, K=16, kind::f16
//               with bf16 operands, fp32 accumulate); tcgen05.commit releases the ring stage /
//               publishes the accumulator.
//   warps 2..5  epilogue: tcgen05.ld of the finished accumulator (double-buffered, so the next
//               tile's MMAs overlap), bias, per-row running top-2.
// Work item = (vocabulary chunk of a few N-tiles, M-tile or pair of M-tiles); items are dealt
// round-robin with the M index fastest, so the blocks that run together share W tiles through
// L2 and W crosses HBM about once.
//
// Every wait on an mbarrier is bounded (clock64 budget).  A wait that gives up raises a
// block-wide abort flag and a status word in the workspace; all roles then fall through to
// the common exit, which drains outstanding copies (bounded), frees TMEM and returns.
#include "mars_common.cuh"
#include "mars_hooks.cuh"

#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdlib>
#include <mutex>

#include "mars.h"

namespace mars {

constexpr int kBM = 128;          // rows of H per tile = TMEM lanes
constexpr int kBN = 256;          // vocabulary entries per tile = TMEM columns per accumulator
constexpr int kBK = 64;           // k-block: 64 bf16 = one 128-byte swizzle row
constexpr int kUmmaK = 16;
constexpr int kStages = 4;
constexpr int kMaxChunkTiles = 16; // upper bound on N-tiles per work item
constexpr int kLmThreads = 192;
constexpr uint32_t kABytes = kBM * kBK * 2;   // 16 KB
constexpr uint32_t kBBytes = kBN * kBK * 2;   // 32 KB
constexpr uint32_t kStageBytes = kABytes + kBBytes;
constexpr uint32_t kTmemCols = 512;
constexpr long long kWaitCycles = 2000000000ll;   // about a second at B200 clocks
constexpr size_t kLmSmemBytes = (size_t)kStages * kStageBytes + 1024 /*align*/ + 256 /*barriers*/;

struct LmParams {
    int M, V, d;
    int n_mtiles, n_ntiles, n_chunks, n_items;
    int chunk_tiles;     // N-tiles per work item
    const float *bias;   // [V] or null
    Rec *partial;        // [M, n_chunks]
    unsigned *status;    // workspace word: 0 ok, else MARS_SEQ_TIMEOUT
};

// ----------------------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false if the budget ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          unsigned *status, long long budget = kWaitCycles)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > budget) {
            *abort_flag = 1;
            atomicExch(status, (unsigned)MARS_SEQ_TIMEOUT);
            return false;
        }
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// 32 lanes x 32 columns of 32-bit: thread t of the warp gets row (lane base + t), 32 columns.
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float (&v)[32])
{
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes,
// 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_k_sw128(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);   // start address, 16-byte units
    d |= (uint64_t)1 << 16;                         // leading byte offset (unused with swizzle)
    d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                         // descriptor version (sm_100)
    d |= (uint64_t)2 << 61;                         // layout: 128-byte swizzle
    return d;
}

// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = 256.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) |
                            ((uint32_t)(kBM >> 4) << 24);

// ----------------------------------------------------------------------------- GEMM + top-2

__global__ void __launch_bounds__(kLmThreads, 1)
lmhead_top2_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w,
                   const LmParams p)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;                 // 1024-byte aligned ring
    const uint32_t bars = tiles + kStages * kStageBytes;           // barriers after the ring
    const uint32_t full0 = bars, empty0 = bars + 8 * kStages;
    const uint32_t tfull0 = bars + 16 * kStages, tempty0 = tfull0 + 16, drain = tempty0 + 16;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kblocks = p.d / kBK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull0 + 8 * a, 1); mbar_init(tempty0 + 8 * a, 4); }
        mbar_init(drain, 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&s_tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int *abort_flag = &s_abort;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            uint32_t armed = 0, armed_parity = 0;     // per-stage bit: a load is outstanding
            bool ok = true;
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                const int mt = item % p.n_mtiles, chunk = item / p.n_mtiles;
                const int nt_end = min((chunk + 1) * p.chunk_tiles, p.n_ntiles);
                for (int nt = chunk * p.chunk_tiles; nt < nt_end && ok; ++nt) {
                    for (int kb = 0; kb < kblocks; ++kb) {
                        if (!mbar_wait(empty0 + 8 * stage, phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
                        const uint32_t fb = full0 + 8 * stage;
                        mbar_expect_tx(fb, kStageBytes);
                        const uint32_t a_dst = tiles + stage * kStageBytes;
                        tma_load_2d(a_dst, &map_h, kb * kBK, mt * kBM, fb);
                        tma_load_2d(a_dst + kABytes, &map_w, kb * kBK, nt * kBN, fb);
                        armed |= 1u << stage;
                        armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                }
            }
            if (*abort_flag) {
                // give this block's own outstanding copies a bounded time to land
                for (int s = 0; s < kStages; ++s) {
                    if (!(armed >> s & 1u)) continue;
                    const long long t0 = clock64();
                    while (!mbar_try_wait(full0 + 8 * s, (armed_parity >> s) & 1u) && clock64() - t0 < 20000000ll) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                const int chunk = item / p.n_mtiles;
                const int nt_end = min((chunk + 1) * p.chunk_tiles, p.n_ntiles);
                for (int nt = chunk * p.chunk_tiles; nt < nt_end && ok; ++nt) {
                    if (!mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + acc * kBN;
                    for (int kb = 0; kb < kblocks; ++kb) {
                        if (!mbar_wait(full0 + 8 * stage, phase, abort_flag, p.status)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t a_addr = tiles + stage * kStageBytes;
                        const uint64_t adesc = umma_desc_k_sw128(a_addr);
                        const uint64_t bdesc = umma_desc_k_sw128(a_addr + kABytes);
#pragma unroll
                        for (int k = 0; k < kBK / kUmmaK; ++k)   // 32 bytes along K per step
                            tc_mma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, kIdesc, (kb | k) != 0 ? 1u : 0u);
                        tc_commit(empty0 + 8 * stage);           // stage reusable once these MMAs retire
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                    if (!ok) break;
                    tc_commit(tfull0 + 8 * acc);                 // accumulator complete
                    if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
                }
            }
            // all MMAs issued by this thread must retire before TMEM is freed
            tc_commit(drain);
            const long long t0 = clock64();
            while (!mbar_try_wait(drain, 0) && clock64() - t0 < kWaitCycles) {}
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int quarter = warp & 3;                 // TMEM lanes this warp may read
        const int row_in_tile = quarter * 32 + lane;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
            const int mt = item % p.n_mtiles, chunk = item / p.n_mtiles;
            const int nt_end = min((chunk + 1) * p.chunk_tiles, p.n_ntiles);
            const int row = mt * kBM + row_in_tile;
            Rec rec = empty_rec();
            for (int nt = chunk * p.chunk_tiles; nt < nt_end && ok; ++nt) {
                // warp-uniform outcome: the TMEM loads below are warp-collective
                ok = __all_sync(0xffffffffu, mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag, p.status));
                if (!ok) break;
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * kBN;
#pragma unroll 1
                for (int c = 0; c < kBN / 32; ++c) {
                    float v[32];
                    tc_ld32(taddr + c * 32, v);
                    const int col0 = nt * kBN + c * 32;
                    if (p.bias) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] += (col0 + j < p.V) ? __ldg(p.bias + col0 + j) : 0.0f;
                    }
                    float m = v[0];
#pragma unroll
                    for (int j = 1; j < 32; ++j) m = fmaxf(m, v[j]);
                    if (m > rec.z2) {   // columns come in increasing token id: equality never displaces
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float x = v[j];
                            if (x > rec.z2 && col0 + j < p.V) {
                                if (x > rec.z1) { rec.z2 = rec.z1; rec.id2 = rec.id1; rec.z1 = x; rec.id1 = col0 + j; }
                                else { rec.z2 = x; rec.id2 = col0 + j; }
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty0 + 8 * acc);   // accumulator free for the next tile
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
            if (ok && row < p.M) p.partial[(size_t)row * p.n_chunks + chunk] = rec;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}


// ----------------------------------------------------------------------------- 2-CTA variant
//
// Same pipeline with tcgen05 `cta_group::2`: two thread blocks of a cluster (two SMs) share one
// MMA of M = 256 x N = 256.  Block r of the pair owns M-tile 2*pair + r: it loads its own
// 128 x 64 slice of H and HALF of the W tile (128 of the 256 vocabulary rows) per k-block, the
// leader block (rank 0) issues the MMAs, which read both blocks' shared memory and write each
// block's 128 accumulator rows into that block's TMEM.  Per block and k-block 32 KB instead of
// 48 KB come out of L2, and the ring has 6 stages instead of 4.
//
// Barriers (all in each block's own shared memory at identical offsets):
//   full[s]    leader's copy only is used: armed by the leader's producer with the bytes of
//              BOTH blocks; both producers' TMA loads complete on it.
//   empty[s]   each block's own copy, released for both blocks by one multicast tcgen05.commit.
//   tfull[a]   each block's own copy, published for both by one multicast tcgen05.commit.
//   tempty[a]  leader's copy: 8 arrivals (4 epilogue warps of each block; the peer's warps
//              arrive remotely).

constexpr int kStages2 = 6;
constexpr uint32_t kB2Bytes = (kBN / 2) * kBK * 2;          // 16 KB: this block's half of the W tile
constexpr uint32_t kStage2Bytes = kABytes + kB2Bytes;        // 32 KB
constexpr size_t kLm2SmemBytes = (size_t)kStages2 * kStage2Bytes + 1024 + 256;
constexpr uint32_t kIdesc2 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) |
                             ((uint32_t)((2 * kBM) >> 4) << 24);

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t cluster_addr, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t leader_bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(leader_bar)
        : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar)   // same offset in both blocks
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"((unsigned short)3)
        : "memory");
}
__device__ __forceinline__ void tc_commit_pair_local(uint32_t bar)   // this block's barrier only
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kLmThreads, 1)
lmhead_top2_kernel_pair(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w,
                        const LmParams p)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    const uint32_t bars = tiles + kStages2 * kStage2Bytes;
    const uint32_t full0 = bars, empty0 = bars + 8 * kStages2;
    const uint32_t tfull0 = bars + 16 * kStages2, tempty0 = tfull0 + 16, drain = tempty0 + 16;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();            // 0 = leader
    const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int kblocks = p.d / kBK;
    const int n_mpairs = (p.n_mtiles + 1) / 2;
    const int n_items = n_mpairs * p.n_chunks;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages2; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull0 + 8 * a, 1); mbar_init(tempty0 + 8 * a, 8); }
        mbar_init(drain, 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&s_tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    cluster_sync_all();            // both blocks' barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int *abort_flag = &s_abort;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both blocks)
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int item = pair_id; item < n_items && ok; item += n_pairs) {
                const int mt = 2 * (item % n_mpairs) + (int)rank, chunk = item / n_mpairs;
                const int nt_end = min((chunk + 1) * p.chunk_tiles, p.n_ntiles);
                for (int nt = chunk * p.chunk_tiles; nt < nt_end && ok; ++nt) {
                    for (int kb = 0; kb < kblocks; ++kb) {
                        if (!mbar_wait(empty0 + 8 * stage, phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
                        const uint32_t leader_full = mapa_shared(full0 + 8 * stage, 0);
                        if (rank == 0) mbar_expect_tx_cluster(leader_full, 2 * kStage2Bytes);
                        const uint32_t a_dst = tiles + stage * kStage2Bytes;
                        tma_load_2d_pair(a_dst, &map_h, kb * kBK, mt * kBM, leader_full);
                        tma_load_2d_pair(a_dst + kABytes, &map_w, kb * kBK, nt * kBN + (int)rank * (kBN / 2),
                                         leader_full);
                        if (++stage == kStages2) { stage = 0; phase ^= 1u; }
                    }
                }
            }
            if (*abort_flag) {     // let copies already issued by this block land (bounded)
                const long long t0 = clock64();
                while (clock64() - t0 < 20000000ll) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader only)
        if (lane == 0 && rank == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (int item = pair_id; item < n_items && ok; item += n_pairs) {
                const int chunk = item / n_mpairs;
                const int nt_end = min((chunk + 1) * p.chunk_tiles, p.n_ntiles);
                for (int nt = chunk * p.chunk_tiles; nt < nt_end && ok; ++nt) {
                    if (!mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + acc * kBN;
                    for (int kb = 0; kb < kblocks; ++kb) {
                        if (!mbar_wait(full0 + 8 * stage, phase, abort_flag, p.status)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t a_addr = tiles + stage * kStage2Bytes;
                        const uint64_t adesc = umma_desc_k_sw128(a_addr);
                        const uint64_t bdesc = umma_desc_k_sw128(a_addr + kABytes);
#pragma unroll
                        for (int k = 0; k < kBK / kUmmaK; ++k)
                            tc_mma_bf16_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, kIdesc2, (kb | k) != 0 ? 1u : 0u);
                        tc_commit_pair(empty0 + 8 * stage);      // frees the stage in both blocks
                        if (++stage == kStages2) { stage = 0; phase ^= 1u; }
                    }
                    if (!ok) break;
                    tc_commit_pair(tfull0 + 8 * acc);            // accumulator complete in both blocks
                    if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
                }
            }
            tc_commit_pair_local(drain);
        }
    } else {
        // ------------------------------------------------------------------ epilogue (both blocks)
        const int quarter = warp & 3;
        const int row_in_tile = quarter * 32 + lane;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int item = pair_id; item < n_items && ok; item += n_pairs) {
            const int mt = 2 * (item % n_mpairs) + (int)rank, chunk = item / n_mpairs;
            const int nt_end = min((chunk + 1) * p.chunk_tiles, p.n_ntiles);
            const int row = mt * kBM + row_in_tile;
            Rec rec = empty_rec();
            for (int nt = chunk * p.chunk_tiles; nt < nt_end && ok; ++nt) {
                ok = __all_sync(0xffffffffu, mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag, p.status));
                if (!ok) break;
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * kBN;
#pragma unroll 1
                for (int c = 0; c < kBN / 32; ++c) {
                    float v[32];
                    tc_ld32(taddr + c * 32, v);
                    const int col0 = nt * kBN + c * 32;
                    if (p.bias) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] += (col0 + j < p.V) ? __ldg(p.bias + col0 + j) : 0.0f;
                    }
                    float m = v[0];
#pragma unroll
                    for (int j = 1; j < 32; ++j) m = fmaxf(m, v[j]);
                    if (m > rec.z2) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float x = v[j];
                            if (x > rec.z2 && col0 + j < p.V) {
                                if (x > rec.z1) { rec.z2 = rec.z1; rec.id2 = rec.id1; rec.z1 = x; rec.id1 = col0 + j; }
                                else { rec.z2 = x; rec.id2 = col0 + j; }
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(mapa_shared(tempty0 + 8 * acc, 0));   // leader's barrier
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
            if (ok && row < p.M) p.partial[(size_t)row * p.n_chunks + chunk] = rec;
        }
    }

    // The leader's MMAs write both blocks' TMEM: wait for them to retire, then meet the peer.
    if (warp == 1 && lane == 0 && rank == 0) {
        const long long t0 = clock64();
        while (!mbar_try_wait(drain, 0) && clock64() - t0 < kWaitCycles) {}
    }
    tc_fence_before();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ----------------------------------------------------------------------------- wait self-test
//
// One block waits, with the pipeline's own bounded-wait routine, on an mbarrier that nothing
// ever arrives on.  The wait must give up after `budget` cycles, raise the status word and let
// the kernel return normally.  Used by mars_selftest_bounded_wait.
__global__ void bounded_wait_selftest_kernel(unsigned *status, long long budget, long long *cycles_waited)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        s_abort = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const long long t0 = clock64();
        const bool ok = mbar_wait(smem_u32(&bar), 0, &s_abort, status, budget);
        cycles_waited[0] = clock64() - t0;
        cycles_waited[1] = ok ? 1 : 0;
    }
}

// ----------------------------------------------------------------------------- tail kernel

__global__ void __launch_bounds__(128) lmhead_tail_kernel(const LmParams p, const TailArgs t)
{
    extern __shared__ __align__(16) unsigned char smem_dyn[];
    const int b = blockIdx.x;
    if (*(volatile unsigned *)p.status != 0) {
        // a device-side wait gave up: no valid result for any sequence
        if (threadIdx.x == 0) {
            t.accept_len[b] = 0;
            t.out_len[b] = 0;
            if (t.seq_status) t.seq_status[b] = MARS_SEQ_TIMEOUT;
        }
        for (int k = threadIdx.x; k <= t.Dcap; k += blockDim.x) {
            t.out_tokens[(size_t)b * (t.Dcap + 1) + k] = -1;
            if (t.path_nodes) t.path_nodes[(size_t)b * (t.Dcap + 1) + k] = -1;
        }
        return;
    }
    // Merge every row's per-chunk records first: a warp per row, lanes across the chunks, so that
    // the loads are coalesced and independent (one thread per row walking its chunks one load
    // after the other took 250 us at 66 chunks); the rows' records go to shared memory.
    const int nch = p.n_chunks;
    const Rec *base = p.partial + (size_t)b * t.N * nch;
    Rec *s_rec = reinterpret_cast<Rec *>(smem_dyn + (tail_smem_bytes(t.N) + 15) / 16 * 16);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int row = warp; row < t.N; row += nwarps) {
        Rec acc = empty_rec();
        for (int k = lane; k < nch; k += 32) {
            const int4 w = __ldcg(reinterpret_cast<const int4 *>(base + (size_t)row * nch + k));
            Rec r;
            r.z1 = __int_as_float(w.x); r.id1 = w.y; r.z2 = __int_as_float(w.z); r.id2 = w.w;
            acc = merge(acc, r);
        }
#pragma unroll
        for (int m = 16; m > 0; m >>= 1) acc = merge(acc, shfl_xor_rec(acc, m));
        if (lane == 0) s_rec[row] = acc;
    }
    __syncthreads();
    verify_tail(t, b, smem_dyn, [&](int i) { return finish_record(s_rec[i]); });
}

// Vocabulary shard: merge a row's per-chunk records into one record with global token ids
// (local id + id_offset), left unfinished for mars_verify_records.  One warp per row, lanes
// across the chunks.
__global__ void __launch_bounds__(128) lmhead_records_kernel(const LmParams p, int id_offset, Rec *records)
{
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= p.M) return;          // warp-uniform
    Rec acc = empty_rec();
    if (*(volatile unsigned *)p.status == 0) {
        const Rec *base = p.partial + (size_t)row * p.n_chunks;
        for (int k = lane; k < p.n_chunks; k += 32) {
            const int4 w = __ldcg(reinterpret_cast<const int4 *>(base + k));
            Rec r;
            r.z1 = __int_as_float(w.x); r.id1 = w.y; r.z2 = __int_as_float(w.z); r.id2 = w.w;
            acc = merge(acc, r);
        }
#pragma unroll
        for (int m = 16; m > 0; m >>= 1) acc = merge(acc, shfl_xor_rec(acc, m));
        if (acc.id1 != kNoId) acc.id1 += id_offset;
        if (acc.id2 != kNoId) acc.id2 += id_offset;
    }
    if (lane == 0) records[row] = acc;     // after a device-side timeout every record stays empty
}

// ----------------------------------------------------------------------------- host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)sym;
    });
    return fn;
}

// bf16 [rows, d] row-major -> boxes of [box_rows x 64] elements, 128-byte swizzle, zero fill.
static bool make_map(CUtensorMap *map, const void *ptr, uint64_t rows, uint64_t d, uint32_t box_rows)
{
    EncodeTiledFn enc = encode_tiled();
    if (!enc) return false;
    cuuint64_t dims[2] = {d, rows};
    cuuint64_t strides[1] = {d * 2};
    cuuint32_t box[2] = {(cuuint32_t)kBK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct LmShape { int n_mtiles, n_ntiles, n_chunks, n_items, chunk_tiles; };

// Work items are (vocabulary chunk, M-tile) pairs dealt round-robin to `blocks` persistent
// blocks.  The chunk length is the one that wastes the least of the last round: cost =
// rounds x (tiles per item + half a tile of per-item overhead); ties go to the longer chunk
// (fewer records per row to merge).  Host-only and independent of the
// device so that the workspace size is a pure function of the shapes.
static bool lm_pair_mode()
{
    return hook(kHookLmheadSingleBlock) != 1;      // test hook: force the single-block MMA kernel
}

static LmShape lm_shape(long long M, int V)
{
    const bool pair = lm_pair_mode();
    LmShape s;
    s.n_mtiles = (int)((M + kBM - 1) / kBM);
    s.n_ntiles = (V + kBN - 1) / kBN;
    const int blocks = pair ? 74 : 148;                          // schedulable units on a B200
    const int m_units = pair ? (s.n_mtiles + 1) / 2 : s.n_mtiles;
    long long best_cost = -1;
    s.chunk_tiles = 1;
    for (int c = 1; c <= kMaxChunkTiles && c <= s.n_ntiles; ++c) {
        const long long items = (long long)m_units * ((s.n_ntiles + c - 1) / c);
        // in half tiles: every item also costs about half a tile (accumulator hand-over, records),
        // and every chunk is one more record per row for the tail to merge -- without this term a
        // tie in rounds x tiles could pick one-tile chunks (594 records per row)
        const long long cost = ((items + blocks - 1) / blocks) * (2 * c + 1);
        if (best_cost < 0 || cost <= best_cost) { best_cost = cost; s.chunk_tiles = c; }
    }
    s.n_chunks = (s.n_ntiles + s.chunk_tiles - 1) / s.chunk_tiles;
    s.n_items = m_units * s.n_chunks;
    return s;
}

static bool lm_supported(int B, int N, int V, int d)
{
    if (B < 1 || N < 1 || N > MARS_MAX_NODES || V < 2 || V > (1 << 30)) return false;
    if (d < kBK || d % kBK != 0 || d > (1 << 20)) return false;
    if ((long long)B * N > (1ll << 24)) return false;
    return true;
}

// Per-device launch state: the opt-in to more than 48 KB of dynamic shared memory is a function
// attribute of the device that is current when it is set, and so is the number of 2-block
// clusters that can be resident at once.
struct LmDeviceState { int ready; int sms; int max_pairs; };
constexpr int kLmMaxDevices = 64;
static std::mutex g_lm_mu;
static LmDeviceState g_lm_state[kLmMaxDevices] = {};

static bool lm_device_state(LmDeviceState *out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kLmMaxDevices) return false;
    std::lock_guard<std::mutex> lock(g_lm_mu);
    LmDeviceState &d = g_lm_state[dev];
    if (!d.ready) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 2)
            return false;
        if (cudaFuncSetAttribute(lmhead_top2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kLmSmemBytes) != cudaSuccess)
            return false;
        if (cudaFuncSetAttribute(lmhead_top2_kernel_pair, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kLm2SmemBytes) != cudaSuccess)
            return false;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(sms / 2 * 2); cfg.blockDim = dim3(kLmThreads);
        cfg.dynamicSmemBytes = kLm2SmemBytes;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, lmhead_top2_kernel_pair, &cfg) == cudaSuccess && n > 0)
            d.max_pairs = n;
        else
            d.max_pairs = sms / 2;
        (void)cudaGetLastError();
        d.sms = sms;
        d.ready = 1;
    }
    *out = d;
    return true;
}

// Shapes, tensor maps and launch of the GEMM + top-2 kernel; fills *pout for the kernels that
// consume the per-chunk records.
static mars_status_t lm_launch_gemm(const void *hidden, const void *w_vocab, const float *bias, int d,
                                    int B, int N, int V, void *workspace, cudaStream_t st, LmParams *pout)
{
    const long long M = (long long)B * N;
    const LmShape s = lm_shape(M, V);
    LmParams p;
    p.M = (int)M; p.V = V; p.d = d;
    p.n_mtiles = s.n_mtiles; p.n_ntiles = s.n_ntiles; p.n_chunks = s.n_chunks; p.n_items = s.n_items;
    p.chunk_tiles = s.chunk_tiles;
    p.bias = bias;
    p.status = (unsigned *)workspace;
    p.partial = (Rec *)((char *)workspace + 256);

    CUtensorMap map_h, map_w;
    if (!make_map(&map_h, hidden, (uint64_t)M, (uint64_t)d, kBM)) return MARS_ERR_CUDA;
    if (!make_map(&map_w, w_vocab, (uint64_t)V, (uint64_t)d, lm_pair_mode() ? kBN / 2 : kBN)) return MARS_ERR_CUDA;

    // Function attributes and occupancy belong to a device: set them up once for each device
    // that this process calls from, with that device current.
    LmDeviceState dstate;
    if (!lm_device_state(&dstate)) return MARS_ERR_CUDA;
    const int sms = dstate.sms;

    if (cudaMemsetAsync(p.status, 0, 256, st) != cudaSuccess) return MARS_ERR_CUDA;
    if (lm_pair_mode()) {
        // persistent pairs: never launch more clusters than can be resident together
        const int max_pairs = dstate.max_pairs;
        int pairs = max_pairs < sms / 2 ? max_pairs : sms / 2;
        if (s.n_items < pairs) pairs = s.n_items;
        lmhead_top2_kernel_pair<<<2 * pairs, kLmThreads, kLm2SmemBytes, st>>>(map_h, map_w, p);
    } else {
        const int grid = s.n_items < sms ? s.n_items : sms;
        lmhead_top2_kernel<<<grid, kLmThreads, kLmSmemBytes, st>>>(map_h, map_w, p);
    }
    if (cudaGetLastError() != cudaSuccess) return MARS_ERR_CUDA;
    *pout = p;
    return MARS_OK;
}

}  // namespace mars

extern "C" {

size_t mars_lmhead_workspace_bytes(int B, int N, int V, int d)
{
    if (!mars::lm_supported(B, N, V, d)) return 0;
    const mars::LmShape s = mars::lm_shape((long long)B * N, V);
    return 256 + (size_t)B * N * s.n_chunks * sizeof(mars::Rec);
}

mars_status_t mars_lmhead_top2_shard(const void *hidden, const void *w_shard, const float *bias_shard, int d,
                                     int B, int N, int V_local, int32_t id_offset, void *records,
                                     void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    using namespace mars;
    if (!hidden || !w_shard || !records || ((uintptr_t)records & 15) || id_offset < 0) return MARS_ERR_INVALID_ARG;
    if (B < 1 || N < 1 || V_local < 2 || d < 1) return MARS_ERR_INVALID_ARG;
    if (((uintptr_t)hidden & 15) || ((uintptr_t)w_shard & 15)) return MARS_ERR_INVALID_ARG;
    if (!lm_supported(B, N, V_local, d)) return MARS_ERR_UNSUPPORTED;
    const size_t need = mars_lmhead_workspace_bytes(B, N, V_local, d);
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return MARS_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    LmParams p;
    const mars_status_t gs = lm_launch_gemm(hidden, w_shard, bias_shard, d, B, N, V_local, workspace, st, &p);
    if (gs != MARS_OK) return gs;
    lmhead_records_kernel<<<(p.M + 3) / 4, 128, 0, st>>>(p, id_offset, (Rec *)records);
    return cudaGetLastError() == cudaSuccess ? MARS_OK : MARS_ERR_CUDA;
}

mars_status_t mars_selftest_bounded_wait(int64_t budget_cycles, void *scratch32, void *cuda_stream)
{
    if (!scratch32 || ((uintptr_t)scratch32 & 7) || budget_cycles < 1 || budget_cycles > 2000000000ll)
        return MARS_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(scratch32, 0, 32, st) != cudaSuccess) return MARS_ERR_CUDA;
    mars::bounded_wait_selftest_kernel<<<1, 32, 0, st>>>((unsigned *)scratch32, (long long)budget_cycles,
                                                         (long long *)((char *)scratch32 + 8));
    return cudaGetLastError() == cudaSuccess ? MARS_OK : MARS_ERR_CUDA;
}

mars_status_t mars_lmhead_verify(const void *hidden, const void *w_vocab, const float *bias, int d,
                                 const int32_t *tok, const int32_t *parent, int B, int N, int V, float theta,
                                 uint32_t flags, int32_t *accept_len, int32_t *out_tokens, int32_t *path_nodes,
                                 int32_t *out_len, int Dcap, int32_t *seq_status, const mars_debug_out_t *dbg,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    using namespace mars;
    if (!hidden || !w_vocab || !tok || !parent || !accept_len || !out_tokens || !out_len) return MARS_ERR_INVALID_ARG;
    if (B < 1 || N < 1 || V < 2 || d < 1 || Dcap < 0 || theta != theta) return MARS_ERR_INVALID_ARG;
    if (((uintptr_t)hidden & 15) || ((uintptr_t)w_vocab & 15)) return MARS_ERR_INVALID_ARG;
    if (flags & ~(MARS_SIGN_LITERAL | MARS_SHARED_PARENT | MARS_RULE_MARGIN | MARS_RULE_PROB_RATIO))
        return MARS_ERR_UNSUPPORTED;
    if ((flags & MARS_RULE_MARGIN) && (flags & MARS_RULE_PROB_RATIO)) return MARS_ERR_INVALID_ARG;
    rule_threshold(&theta, &flags);
    if (!lm_supported(B, N, V, d)) return MARS_ERR_UNSUPPORTED;
    const size_t need = mars_lmhead_workspace_bytes(B, N, V, d);
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return MARS_ERR_WORKSPACE;

    cudaStream_t st = (cudaStream_t)cuda_stream;
    LmParams p;
    const mars_status_t gs = lm_launch_gemm(hidden, w_vocab, bias, d, B, N, V, workspace, st, &p);
    if (gs != MARS_OK) return gs;

    TailArgs t;
    t.tok = tok; t.parent = parent; t.accept_len = accept_len; t.out_tokens = out_tokens;
    t.path_nodes = path_nodes; t.out_len = out_len; t.seq_status = seq_status;
    t.dbg_val = dbg ? dbg->top2_val : nullptr;
    t.dbg_id = dbg ? dbg->top2_id : nullptr;
    t.dbg_flags = dbg ? dbg->node_flags : nullptr;
    t.N = N; t.Dcap = Dcap; t.theta = theta; t.flags = flags; t.chain = 0;

    lmhead_tail_kernel<<<B, 128, (tail_smem_bytes(N) + 15) / 16 * 16 + (size_t)N * sizeof(Rec), st>>>(p, t);
    return cudaGetLastError() == cudaSuccess ? MARS_OK : MARS_ERR_CUDA;
}

}  // extern "C"
