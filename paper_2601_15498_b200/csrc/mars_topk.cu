// libmars: exact top-k (k <= 32) of logits rows with token ids, the selection a drafter needs
// when it expands a token tree with the k best continuations of every frontier node (the paper
// builds its trees as EAGLE-3 does, with top-k = 10; Sec. 4.1, implementation details).
//
// Same streaming structure as the top-2 kernel: a block owns a slice of a row and reads it once
// with 16-byte loads; a batch of 8 vectors per thread is reduced to its maximum with packed max
// instructions and skipped unless it reaches the floor, a lower bound on the slice's k-th value.
// Two forms of the slice selection follow: an optimistic one that only collects candidates
// while streaming (topk_slice_kernel), and an exact one with per-warp ordered lists that the
// optimistic one falls back to (topk_slice_exact).  A second small kernel merges the slices of
// a row, completes rows that have fewer than k entries above -inf, and writes best first.
//
// Total order as everywhere in the library: larger value first, lower token id first among
// equal values, NaN counts as -inf, -0 is reported as +0.
#include "mars_common.cuh"
#include "mars_hooks.cuh"
#include "mars_stream.cuh"

#include <cstdlib>

#include "mars.h"

namespace mars {

constexpr int kTkThreads = 256;
constexpr int kTkU = 8;
constexpr int kTkMaxK = 32;
constexpr int kTkTargetBlocks = 148 * 4;
constexpr int kTkMinSliceBytes = kTkThreads * kTkU * 16;
constexpr int kTkCap = 2048;       // candidate slots of the optimistic collection

struct Cand {
    float z;
    int id;
};

struct TopkParams {
    const void *logits;
    long long ld;
    int V, S, L, k;
    Cand *partial;   // [R*S, k] unused entries {-inf, kNoId}
    int *redo;       // [R*S] 1: the optimistic pass ran out of candidate slots for this slice
    long long nslices;
};

// Order-preserving float <-> uint encoding for the block-wide bound (atomicMax on shared memory).
__device__ __forceinline__ unsigned tk_enc(float x)
{
    unsigned b = __float_as_uint(x + 0.0f);
    return b ^ ((unsigned)((int)b >> 31) | 0x80000000u);
}
__device__ __forceinline__ float tk_dec(unsigned e)
{
    return __uint_as_float(e ^ ((e & 0x80000000u) ? 0x80000000u : 0xffffffffu));
}

// A warp keeps its k best elements so far spread over its lanes: lane i < k holds the i-th best
// (value wz, token id wid), the other lanes hold {-inf, kNoId}.  Inserting one candidate is a
// ballot (how many entries beat it) and one shuffle; the candidate is the same in all lanes.
__device__ __forceinline__ void warp_list_insert(float &wz, int &wid, int lane, int k, float x, int id)
{
    const unsigned ahead = __ballot_sync(0xffffffffu, beats(wz, wid, x, id));
    const int pos = __popc(ahead);              // entries are sorted: exactly lanes 0..pos-1 beat it
    const float uz = __shfl_up_sync(0xffffffffu, wz, 1);
    const int uid = __shfl_up_sync(0xffffffffu, wid, 1);
    if (pos < k) {
        if (lane == pos) { wz = x; wid = id; }
        else if (lane > pos && lane < k) { wz = uz; wid = uid; }
    }
}

// Exact slice selection with per-warp lists; always correct, used when the optimistic collection
// below runs out of room.  Called by all threads of the block.
template <int DT>
__device__ void topk_slice_exact(const TopkParams &p, const long long blk)
{
    typedef Elem<DT> E;
    constexpr int kWarps = kTkThreads / 32;
    __shared__ Cand s_queue[kWarps][32 * 8];     // per warp: candidates of one vector step
    __shared__ int s_qn[kWarps];
    __shared__ unsigned s_bound;                 // block-wide lower bound on the slice's k-th value
    __shared__ Cand s_list[kWarps * kTkMaxK];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, k = p.k;
    const long long row = blk / p.S;
    const int slice = (int)(blk - row * p.S);
    const int lo = slice * p.L;
    const int hi = min(p.V, lo + p.L);
    const char *rowp = (const char *)p.logits + (size_t)row * (size_t)p.ld * E::kBytes;

    const uintptr_t a0 = (uintptr_t)(rowp + (size_t)lo * E::kBytes);
    int nhead = (int)(((16 - (a0 & 15)) & 15) / E::kBytes);
    nhead = min(nhead, max(hi - lo, 0));
    const int vlo = lo + nhead;
    const int nvec = max(hi - vlo, 0) / E::kVec;
    const int tlo = vlo + nvec * E::kVec;
    const int ntail = max(hi - tlo, 0);
    const uint4 *vbase = (const uint4 *)(rowp + (size_t)vlo * E::kBytes);

    __syncthreads();             // shared arrays may still be in use from a previous slice
    if (tid == 0) s_bound = tk_enc(-INFINITY);
    if (lane == 0) s_qn[warp] = 0;
    __syncthreads();

    float wz = -INFINITY;       // this lane's entry of the warp's list
    int wid = kNoId;
    float kth = -INFINITY;      // value / id of the warp's k-th best (entry of lane k-1)
    int kth_id = kNoId;
    float warp_floor = -INFINITY;   // value-only bound from the warp's first batch
    Cand *queue = s_queue[warp];

    // Drain the warp's queue into its list (all lanes), then publish the warp's k-th value.
    auto drain = [&]() {
        __syncwarp();
        const int n = s_qn[warp];
        for (int i = 0; i < n; ++i) {
            const Cand c = queue[i];
            if (beats(c.z, c.id, kth, kth_id)) {
                warp_list_insert(wz, wid, lane, k, c.z, c.id);
                kth = __shfl_sync(0xffffffffu, wz, k - 1);
                kth_id = __shfl_sync(0xffffffffu, wid, k - 1);
            }
        }
        __syncwarp();
        if (lane == 0) {
            s_qn[warp] = 0;
            if (kth > -INFINITY) atomicMax(&s_bound, tk_enc(kth));
        }
        __syncwarp();
    };
    // One element of this lane: queue it if it can still be among the slice's k best.
    auto offer = [&](float x, int idx, float floor_v) {
        if (x >= floor_v && x > -INFINITY && beats(x, idx, kth, kth_id)) {
            const int pos = atomicAdd(&s_qn[warp], 1);
            queue[pos].z = x;
            queue[pos].id = idx;
        }
    };

    // head and tail scalars (at most 15 elements) go through the same queue
    if (nhead > 0 || ntail > 0) {
        if (warp == 0) {
            if (lane < nhead) offer(E::scalar(rowp, lo + lane), lo + lane, -INFINITY);
            if (lane < ntail) offer(E::scalar(rowp, tlo + lane), tlo + lane, -INFINITY);
            drain();
        }
    }

    constexpr int kBatchVecs = kTkThreads * kTkU;
    const int nbatches = (nvec + kBatchVecs - 1) / kBatchVecs;
    for (int bi = 0; bi < nbatches; ++bi) {
        uint4 v[kTkU];
        typename E::packed_t q[kTkU];
        const int v0 = bi * kBatchVecs + tid;
#pragma unroll
        for (int u = 0; u < kTkU; ++u) {
            int vi = v0 + u * kTkThreads;
            v[u] = vi < nvec ? ld_stream(vbase + vi) : E::neg_inf();
        }
        typename E::packed_t m = E::vred(v[0]);
        q[0] = m;
#pragma unroll
        for (int u = 1; u < kTkU; ++u) { q[u] = E::vred(v[u]); m = E::pmax(m, q[u]); }
        const float bm = E::to_float(m);
        if (bi == 0) {
            // value-only bound for the warp: the k-th largest of its lanes' first-batch maxima
            // (maxima of distinct elements); rank by (value, lane).
            const float mine = (bm == bm) ? bm : -INFINITY;
            int rank = 0;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float o = __shfl_sync(0xffffffffu, mine, j);
                rank += (o > mine || (o == mine && j < lane)) ? 1 : 0;
            }
            const unsigned who = __ballot_sync(0xffffffffu, rank == k - 1);
            warp_floor = __shfl_sync(0xffffffffu, mine, __ffs(who) - 1);
        }
        float floor_v = fmaxf(warp_floor, tk_dec(*(volatile unsigned *)&s_bound));
        floor_v = fmaxf(floor_v, kth);
        if (__any_sync(0xffffffffu, bm >= floor_v)) {
#pragma unroll
            for (int u = 0; u < kTkU; ++u) {
                const float qf = E::to_float(q[u]);
                if (__any_sync(0xffffffffu, qf >= floor_v)) {
                    if (qf >= floor_v) {
                        const int base = vlo + (v0 + u * kTkThreads) * E::kVec;
#pragma unroll
                        for (int e = 0; e < E::kVec; ++e) offer(E::elem(v[u], e), base + e, floor_v);
                    }
                    drain();
                    floor_v = fmaxf(floor_v, kth);
                }
            }
        }
    }

    // ---- block: the k best of the warps' lists by rank counting ----
    if (lane < kTkMaxK) { s_list[warp * kTkMaxK + lane].z = lane < k ? wz : -INFINITY;
                          s_list[warp * kTkMaxK + lane].id = lane < k ? wid : kNoId; }
    Cand *out = p.partial + (size_t)blk * k;
    for (int i = tid; i < k; i += kTkThreads) { out[i].z = -INFINITY; out[i].id = kNoId; }
    __syncthreads();
    constexpr int kAll = kWarps * kTkMaxK;
    for (int i = tid; i < kAll; i += kTkThreads) {
        const Cand c = s_list[i];
        if (c.id == kNoId) continue;
        int rank = 0;
        for (int j = 0; j < kAll; ++j)
            rank += (s_list[j].id != kNoId && beats(s_list[j].z, s_list[j].id, c.z, c.id)) ? 1 : 0;
        if (rank < k) out[rank] = c;
    }
}

// Slice selection, optimistic form: nothing is ordered while the row streams by.  Elements that
// reach the current floor -- a valid lower bound on the slice's k-th value -- are appended to a
// block-wide candidate buffer (one shared-memory atomicAdd each); the floor starts as the k-th
// largest of the threads' first-batch maxima and is raised once per batch by one warp from the
// candidates collected so far.  The k best of the buffer are rank-counted at the end.  If the
// buffer ever fills up (adversarially ordered rows), the block redoes its slice with
// topk_slice_exact.
template <int DT>
__global__ void __launch_bounds__(kTkThreads, 4) topk_slice_kernel(const TopkParams p)
{
    typedef Elem<DT> E;
    constexpr int kWarps = kTkThreads / 32;
    __shared__ __align__(8) Cand s_cand[kTkCap];
    __shared__ float s_max[kTkThreads];
    __shared__ unsigned s_floor;
    __shared__ int s_n, s_overflow, s_seen;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, k = p.k;
    const long long blk = blockIdx.x;
    const long long row = blk / p.S;
    const int slice = (int)(blk - row * p.S);
    const int lo = slice * p.L;
    const int hi = min(p.V, lo + p.L);
    const char *rowp = (const char *)p.logits + (size_t)row * (size_t)p.ld * E::kBytes;
    const uintptr_t a0 = (uintptr_t)(rowp + (size_t)lo * E::kBytes);
    int nhead = (int)(((16 - (a0 & 15)) & 15) / E::kBytes);
    nhead = min(nhead, max(hi - lo, 0));
    const int vlo = lo + nhead;
    const int nvec = max(hi - vlo, 0) / E::kVec;
    const int tlo = vlo + nvec * E::kVec;
    const int ntail = max(hi - tlo, 0);
    const uint4 *vbase = (const uint4 *)(rowp + (size_t)vlo * E::kBytes);

    {   // empty slots carry kNoId so that a reader can tell a reserved slot from a written one
        Cand e; e.z = -INFINITY; e.id = kNoId;
        for (int i = tid; i < kTkCap; i += kTkThreads) s_cand[i] = e;
    }
    if (tid == 0) { s_floor = tk_enc(-INFINITY); s_n = 0; s_overflow = 0; s_seen = 0; }
    __syncthreads();

    auto append = [&](float x, int idx) {
        const int pos = atomicAdd(&s_n, 1);
        if (pos < kTkCap) {
            Cand e; e.z = x; e.id = idx;     // one 8-byte store: value and id become visible together
            *reinterpret_cast<volatile unsigned long long *>(&s_cand[pos]) = *reinterpret_cast<unsigned long long *>(&e);
        } else {
            s_overflow = 1;
        }
    };
    // One warp: k-th best of (up to 256 of) the candidates so far -> floor.  Slots that are
    // reserved but not written yet still hold kNoId and are skipped; every written slot is a
    // distinct element, so the k-th best of any subset is a valid bound.
    auto raise_floor = [&]() {
        const int n = min(*(volatile int *)&s_n, min(kTkCap, 8 * 32));
        Cand mine[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int i = j * 32 + lane;
            unsigned long long raw = *reinterpret_cast<volatile unsigned long long *>(&s_cand[i < n ? i : 0]);
            mine[j] = *reinterpret_cast<Cand *>(&raw);
            if (i >= n) mine[j].id = kNoId;
        }
        Cand win; win.z = -INFINITY; win.id = kNoId;
        for (int r = 0; r < k; ++r) {
            Cand b; b.z = -INFINITY; b.id = kNoId;
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (mine[j].id != kNoId && beats(mine[j].z, mine[j].id, b.z, b.id)) b = mine[j];
#pragma unroll
            for (int msk = 16; msk > 0; msk >>= 1) {
                float oz = __shfl_xor_sync(0xffffffffu, b.z, msk);
                int oi = __shfl_xor_sync(0xffffffffu, b.id, msk);
                if (oi != kNoId && beats(oz, oi, b.z, b.id)) { b.z = oz; b.id = oi; }
            }
            win = b;
            if (win.id == kNoId) break;
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (mine[j].id == win.id) mine[j].id = kNoId;
        }
        if (lane == 0 && win.id != kNoId) atomicMax(&s_floor, tk_enc(win.z));
        __syncwarp();
    };

    if (tid < nhead) { float x = E::scalar(rowp, lo + tid); if (x > -INFINITY) append(x, lo + tid); }
    if (tid < ntail) { float x = E::scalar(rowp, tlo + tid); if (x > -INFINITY) append(x, tlo + tid); }

    constexpr int kBatchVecs = kTkThreads * kTkU;
    const int nbatches = (nvec + kBatchVecs - 1) / kBatchVecs;
    for (int bi = 0; bi < nbatches; ++bi) {
        uint4 v[kTkU];
        typename E::packed_t q[kTkU];
        const int v0 = bi * kBatchVecs + tid;
#pragma unroll
        for (int u = 0; u < kTkU; ++u) {
            int vi = v0 + u * kTkThreads;
            v[u] = vi < nvec ? ld_stream(vbase + vi) : E::neg_inf();
        }
        typename E::packed_t m = E::vred(v[0]);
        q[0] = m;
#pragma unroll
        for (int u = 1; u < kTkU; ++u) { q[u] = E::vred(v[u]); m = E::pmax(m, q[u]); }
        const float bm = E::to_float(m);
        if (bi == 0) {
            // floor = k-th largest of the threads' first-batch maxima (values of distinct
            // elements).  Two levels: a lane can only be among the block's k largest if it is
            // among its warp's k largest, so only those lanes (at most 8k) are ranked block-wide.
            const float mine = (bm == bm) ? bm : -INFINITY;
            int wrank = 0;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float o = __shfl_sync(0xffffffffu, mine, j);
                wrank += (o > mine || (o == mine && j < lane)) ? 1 : 0;
            }
            s_max[tid] = wrank < k ? mine : -INFINITY;     // slot = warp * 32 + lane
            __syncthreads();
            if (wrank < k && mine > -INFINITY) {
                int rank = 0;
                for (int j = 0; j < kTkThreads; ++j) {
                    const float o = s_max[j];
                    rank += (o > mine || (o == mine && j < tid)) ? 1 : 0;
                }
                if (rank == k - 1) atomicMax(&s_floor, tk_enc(mine));
            }
            __syncthreads();
        } else if ((bi & (kWarps - 1)) == warp) {
            // raise the floor when enough new candidates have come in to move the k-th best
            const int n_now = *(volatile int *)&s_n;
            if (n_now - *(volatile int *)&s_seen >= max(2, k / 4)) {
                raise_floor();
                if (lane == 0) s_seen = n_now;
            }
        }
        const float floor_v = tk_dec(*(volatile unsigned *)&s_floor);
        if (bm >= floor_v) {
#pragma unroll
            for (int u = 0; u < kTkU; ++u) {
                if (E::to_float(q[u]) >= floor_v) {
                    const int base = vlo + (v0 + u * kTkThreads) * E::kVec;
#pragma unroll
                    for (int e = 0; e < E::kVec; ++e) {
                        const float x = E::elem(v[u], e);
                        if (x >= floor_v && x > -INFINITY) append(x, base + e);
                    }
                }
            }
        }
    }
    __syncthreads();
    if (tid == 0) p.redo[blk] = s_overflow;      // flagged slices are redone by topk_redo_kernel
    if (s_overflow) return;
    const int n = s_n;
    Cand *out = p.partial + (size_t)blk * k;
    for (int i = tid; i < k; i += kTkThreads) { out[i].z = -INFINITY; out[i].id = kNoId; }
    __syncthreads();
    for (int i = tid; i < n; i += kTkThreads) {
        const Cand c = s_cand[i];
        int rank = 0;
        for (int j = 0; j < n && rank < k; ++j) rank += beats(s_cand[j].z, s_cand[j].id, c.z, c.id) ? 1 : 0;
        if (rank < k) out[rank] = c;
    }
}

// Slices whose optimistic pass overflowed are redone exactly.  A small persistent grid scans the
// flags; without flagged slices this kernel only reads them.
template <int DT>
__global__ void __launch_bounds__(kTkThreads) topk_redo_kernel(const TopkParams p)
{
    for (long long blk = blockIdx.x; blk < p.nslices; blk += gridDim.x)
        if (p.redo[blk]) topk_slice_exact<DT>(p, blk);      // block-uniform condition
}

// Merge the S sorted slice lists of a row, complete and write it.  One block per row.
__global__ void __launch_bounds__(128) topk_merge_kernel(const TopkParams p, float *out_val, int32_t *out_id)
{
    extern __shared__ Cand s_c[];
    __shared__ int s_found;
    const int k = p.k, n = p.S * k;
    const long long row = blockIdx.x;
    const Cand *src = p.partial + (size_t)row * n;
    if (threadIdx.x == 0) s_found = 0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) s_c[i] = src[i];
    __syncthreads();
    float *ov = out_val + (size_t)row * k;
    int32_t *oi = out_id + (size_t)row * k;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const Cand c = s_c[i];
        if (c.id == kNoId) continue;
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += (s_c[j].id != kNoId && beats(s_c[j].z, s_c[j].id, c.z, c.id)) ? 1 : 0;
        if (rank < k) { ov[rank] = c.z + 0.0f; oi[rank] = c.id; atomicAdd(&s_found, 1); }
    }
    __syncthreads();
    // Fewer than k entries above -inf: the remaining places go to the lowest unused ids at -inf
    // (every -inf / NaN entry ties, lowest id first).
    if (threadIdx.x == 0 && s_found < k) {
        int found = s_found, next = 0;
        while (found < k) {
            bool used = false;
            for (int j = 0; j < found; ++j) used |= (oi[j] == next);
            if (!used) { ov[found] = -INFINITY; oi[found] = next; ++found; }
            ++next;
        }
    }
}

struct TkSplit { int S, L; };

static TkSplit topk_split(long long R, int V, int dt)
{
    const int es = dt == MARS_BF16 ? 2 : 4;
    long long S = 1;
    const int force = hook(kHookForceSplit);          // test hook shared with the top-2 kernel
    int min_elems = kTkMinSliceBytes / es;
    if (force >= 1) { S = force; min_elems = 64; }
    else if (R < kTkTargetBlocks) S = kTkTargetBlocks / R;
    long long smax = V / min_elems;
    if (smax < 1) smax = 1;
    if (S > smax) S = smax;
    if (S > 64) S = 64;
    long long L = (V + S - 1) / S;
    L = (L + 15) / 16 * 16;
    TkSplit sp;
    sp.L = (int)L;
    sp.S = (int)((V + L - 1) / L);
    return sp;
}

static bool topk_supported(long long R, int V, int dt, int k)
{
    if (R < 1 || R > (1ll << 30) || V < 1 || V > (1 << 30)) return false;
    if (dt != MARS_BF16 && dt != MARS_FP32) return false;
    return k >= 1 && k <= kTkMaxK && k <= V;
}

}  // namespace mars

extern "C" {

size_t mars_topk_workspace_bytes(int64_t rows, int V, mars_dtype_t dt, int k)
{
    if (!mars::topk_supported(rows, V, (int)dt, k)) return 0;
    const mars::TkSplit sp = mars::topk_split(rows, V, (int)dt);
    return (size_t)rows * sp.S * (k * sizeof(mars::Cand) + sizeof(int));
}

mars_status_t mars_topk_rows(const void *logits, int64_t ld, mars_dtype_t dt, int64_t rows, int V, int k,
                             float *out_val, int32_t *out_id, void *workspace, size_t workspace_bytes,
                             void *cuda_stream)
{
    using namespace mars;
    if (!logits || !out_val || !out_id || rows < 1 || V < 1 || ld < V || k < 1) return MARS_ERR_INVALID_ARG;
    if (!topk_supported(rows, V, (int)dt, k)) return k > V ? MARS_ERR_INVALID_ARG : MARS_ERR_UNSUPPORTED;
    const int es = dt == MARS_BF16 ? 2 : 4;
    if ((uintptr_t)logits % es) return MARS_ERR_INVALID_ARG;
    const TkSplit sp = topk_split(rows, V, (int)dt);
    if (rows * sp.S > 0x7fffffffll) return MARS_ERR_UNSUPPORTED;
    const size_t need = (size_t)rows * sp.S * (k * sizeof(Cand) + sizeof(int));
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return MARS_ERR_WORKSPACE;
    TopkParams p;
    p.logits = logits; p.ld = ld; p.V = V; p.S = sp.S; p.L = sp.L; p.k = k;
    p.partial = (Cand *)workspace;
    p.nslices = rows * sp.S;
    p.redo = (int *)((char *)workspace + (size_t)p.nslices * k * sizeof(Cand));
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const unsigned grid = (unsigned)(rows * sp.S);
    if (dt == MARS_BF16) topk_slice_kernel<MARS_BF16><<<grid, kTkThreads, 0, st>>>(p);
    else topk_slice_kernel<MARS_FP32><<<grid, kTkThreads, 0, st>>>(p);
    if (cudaGetLastError() != cudaSuccess) return MARS_ERR_CUDA;
    const unsigned redo_grid = (unsigned)(p.nslices < 148 * 2 ? p.nslices : 148 * 2);
    if (dt == MARS_BF16) topk_redo_kernel<MARS_BF16><<<redo_grid, kTkThreads, 0, st>>>(p);
    else topk_redo_kernel<MARS_FP32><<<redo_grid, kTkThreads, 0, st>>>(p);
    if (cudaGetLastError() != cudaSuccess) return MARS_ERR_CUDA;
    topk_merge_kernel<<<(unsigned)rows, 128, (size_t)sp.S * k * sizeof(Cand), st>>>(p, out_val, out_id);
    return cudaGetLastError() == cudaSuccess ? MARS_OK : MARS_ERR_CUDA;
}

}  // extern "C"
