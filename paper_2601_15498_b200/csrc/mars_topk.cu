// libmars: exact top-k (k <= 32) of logits rows with token ids, the selection a drafter needs
// when it expands a token tree with the k best continuations of every frontier node (the paper
// builds its trees as EAGLE-3 does, with top-k = 10; Sec. 4.1, implementation details).
//
// Same streaming structure as the top-2 kernel: a block owns a slice of a row and reads it once
// with 16-byte loads; a batch of 8 vectors per thread is reduced to its maximum with packed max
// instructions and skipped unless it reaches the floor, a lower bound on the slice's k-th value.
// Two forms of the slice selection follow: the streaming one with a queue and one ordered list
// per block that no warp ever waits for (topk_slice_kernel), and one with per-warp ordered lists
// that a block falls back to when its queue fills up (topk_slice_exact).  A block that streamed
// a whole row writes the row's result itself (one launch per call); only rows split over several
// blocks take a second small kernel that merges the slices' lists.  Either one completes rows
// that have fewer than k entries above -inf and writes best first.
//
// Total order as everywhere in the library: larger value first, lower token id first among
// equal values, NaN counts as -inf, -0 is reported as +0.
#include "mars_common.cuh"
#include "mars_hooks.cuh"
#include "mars_top2_stream.cuh"

#include <cstdlib>

#include "mars.h"

namespace mars {

constexpr int kTkThreads = 256;
constexpr int kTkU = 8;
constexpr int kTkMaxK = 32;
constexpr int kTkDenseMinRows = 148 * 24;   // rows from which the 6-blocks-per-SM shape is considered
constexpr int kTkMergeThreads = 512;   // merge kernel: one entry per thread for most rows
constexpr int kTkTargetBlocks = 148 * 4;
constexpr int kTkMinSliceBytes = kTkThreads * kTkU * 16;
constexpr int kTkCap = kTkThreads * 8;   // slots of the slice kernel's queue of elements at or above the floor
                                         // (the exact fallback reuses them: one vector step per thread)

struct Cand {
    float z;
    int id;
};

struct TopkParams {
    const void *logits;
    long long ld;
    int V, S, L, k;
    Cand *partial;   // [R*S, k] unused entries {-inf, kNoId}
    long long nslices;
    float *out_val;      // [R, k] final values, best first
    int32_t *out_id;     // [R, k] final token ids
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

// Exact slice selection with per-warp lists; always correct, used when the streaming kernel below
// runs out of room.  Called by all threads of the block.  The caller lends its shared memory:
//   queue_mem  kTkThreads * 8 candidates (per warp: the candidates of one vector step)
//   s_list     (kTkThreads / 32) * kTkMaxK candidates (the warps' lists for the final ranking)
//   s_qn       kTkThreads / 32 counters;  s_bound  block-wide lower bound on the slice's k-th value
template <int DT>
__device__ __noinline__ void topk_slice_exact(const char *rowp, const int lo, const int hi, const int k,
                                              Cand *out, Cand *queue_mem, Cand *s_list, int *s_qn,
                                              unsigned *s_bound_p)
{
    typedef Elem<DT> E;
    constexpr int kWarps = kTkThreads / 32;
    unsigned &s_bound = *s_bound_p;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

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
    Cand *queue = queue_mem + warp * (32 * 8);

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

// Fewer than k entries above -inf in a row: the remaining places go to the lowest unused ids at
// -inf (every -inf / NaN entry ties, lowest id first).  One thread.
__device__ void complete_row(float *ov, int32_t *oi, int found, int k)
{
    int next = 0;
    while (found < k) {
        bool used = false;
        for (int j = 0; j < found; ++j) used |= (oi[j] == next);
        if (!used) { ov[found] = -INFINITY; oi[found] = next; ++found; }
        ++next;
    }
}

// Slice selection.  A block streams its slice once, like the top-2 kernel (batches of 8 vectors
// per thread reduced with packed max instructions).  A batch is looked at more closely only if
// its maximum reaches the floor, a lower bound on the slice's k-th value:
//   - the floor starts as the k-th largest of the threads' first-batch maxima (values of distinct
//     elements): every warp orders its lanes' maxima, the k best of each warp go to a small
//     table, and the table's k-th entry is found by rank counting;
//   - a thread whose batch reaches the floor appends the elements that do to a queue in shared
//     memory (one atomicAdd each), nothing more;
//   - the slice's k best so far live in one ordered list in shared memory.  After appending, a
//     warp TRIES to take the list (one compare-and-swap, no waiting): if it gets it, it holds
//     the list in its lanes (lane i = entry i), feeds the queued elements into it one by one (a
//     ballot and a shuffle each), stores it back and publishes the k-th entry's value as the new
//     floor; if another warp has it, that warp or a later one will pick the elements up.
// So nobody ever waits, the floor trails the stream by at most a few elements, about
// k (1 + ln(batches)) elements reach the queue on unordered data, and the list is the result.
// If the queue fills up (adversarially ordered rows), the block redoes its slice with
// topk_slice_exact.
template <int DT, int U, int MINB>
__global__ void __launch_bounds__(kTkThreads, MINB) topk_slice_kernel(const TopkParams p)
{
    typedef Elem<DT> E;
    constexpr int kWarps = kTkThreads / 32;
    __shared__ __align__(8) Cand s_cand[kTkCap];
    __shared__ __align__(8) Cand s_list[kTkMaxK];
    __shared__ __align__(8) Cand s_xlist[kWarps * kTkMaxK];    // exact fallback only
    __shared__ float s_top[kWarps * kTkMaxK];
    __shared__ unsigned s_floor;
    __shared__ int s_tail, s_head, s_lock, s_overflow;
    __shared__ int s_xqn[kWarps];

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
    constexpr int kBatchVecs = kTkThreads * U;
    const int nfull = nvec / kBatchVecs;

    pdl_launch_dependents();    // the next call's kernel may be scheduled; it waits for this one first thing
    pdl_wait();     // scheduled early itself (behind the previous call's last kernel), reads nothing before that is done
    uint4 v[U];
    typename E::packed_t q[U];
    // batch 0: issue its loads first, so that the set-up below overlaps their latency
    float bm = (nfull > 0) ? load_batch<DT, U, false>(vbase, tid, nvec, v, q)
                           : load_batch<DT, U, true>(vbase, tid, nvec, v, q);
    {   // empty slots carry kNoId so that a reader can tell a reserved slot from a written one
        Cand e; e.z = -INFINITY; e.id = kNoId;
        for (int i = tid; i < kTkCap; i += kTkThreads) s_cand[i] = e;
        if (tid < kTkMaxK) s_list[tid] = e;
    }
    if (tid == 0) { s_floor = tk_enc(-INFINITY); s_tail = 0; s_head = 0; s_lock = 0; s_overflow = 0; }
    __syncthreads();

    auto append = [&](float x, int idx) {
        const int pos = atomicAdd(&s_tail, 1);
        if (pos < kTkCap) {
            Cand e; e.z = x; e.id = idx;     // one 8-byte store: value and id become visible together
            *reinterpret_cast<volatile unsigned long long *>(&s_cand[pos]) = *reinterpret_cast<unsigned long long *>(&e);
        } else {
            s_overflow = 1;
        }
    };
    // Feed the queued elements into the list.  Called by whole warps; `force` skips the
    // compare-and-swap (used once at the end, when no other warp can be in here).
    auto drain = [&](bool force) {
        int got = 1;
        if (!force) {
            if (lane == 0) got = atomicCAS(&s_lock, 0, 1) == 0 ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
        }
        if (!got) return;
        __threadfence_block();
        // one lane reads the queue's bounds for all: the tail moves while other warps append
        int i = 0, tail = 0;
        if (lane == 0) { i = *(volatile int *)&s_head; tail = min(*(volatile int *)&s_tail, kTkCap); }
        i = __shfl_sync(0xffffffffu, i, 0);
        tail = __shfl_sync(0xffffffffu, tail, 0);
        unsigned long long raw = *reinterpret_cast<volatile unsigned long long *>(&s_list[lane]);
        Cand mine = *reinterpret_cast<Cand *>(&raw);
        // 32 slots at a time, one per lane.  Lanes do not read at the same instant, so what is
        // "written" is settled by a ballot: every decision below is the same in all lanes.
        while (i < tail) {
            Cand c; c.z = -INFINITY; c.id = kNoId;
            if (i + lane < tail) {
                raw = *reinterpret_cast<volatile unsigned long long *>(&s_cand[i + lane]);
                c = *reinterpret_cast<Cand *>(&raw);
            }
            const unsigned written = __ballot_sync(0xffffffffu, c.id != kNoId);
            const int n = written == 0xffffffffu ? 32 : __ffs(~written) - 1;    // leading written slots
            for (int t = 0; t < n; ++t) {
                const float cz = __shfl_sync(0xffffffffu, c.z, t);
                const int cid = __shfl_sync(0xffffffffu, c.id, t);
                warp_list_insert(mine.z, mine.id, lane, k, cz, cid);
            }
            i += n;
            if (n < 32) break;       // a slot that is reserved but not written yet: a later round takes it
        }
        *reinterpret_cast<volatile unsigned long long *>(&s_list[lane]) = *reinterpret_cast<unsigned long long *>(&mine);
        if (lane == k - 1 && mine.id != kNoId) atomicMax(&s_floor, tk_enc(mine.z));
        __syncwarp();
        if (lane == 0) {
            *(volatile int *)&s_head = i;
            __threadfence_block();
            if (!force) atomicExch(&s_lock, 0);
        }
    };

    if (tid < nhead) { float x = E::scalar(rowp, lo + tid); if (x > -INFINITY) append(x, lo + tid); }
    if (tid < ntail) { float x = E::scalar(rowp, tlo + tid); if (x > -INFINITY) append(x, tlo + tid); }

    // First floor: the k-th largest of the threads' first-batch maxima, or a value just below it.
    // Each warp enters its m = min(k, 4 + k/4) largest maxima, ordered, into a table and the
    // k-th largest table entry is taken: the table is a subset of the maxima (8 m >= k entries),
    // so its k-th largest never exceeds theirs, and it falls short of it only when one warp
    // holds more than m of the block's k largest (k = 32: 12 of 32 in one of 8 warps).
    {
        const int m = min(k, 4 + (k >> 2));
        const float mine = (bm == bm) ? bm : -INFINITY;
        int wrank = 0;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            const float o = __shfl_sync(0xffffffffu, mine, j);
            wrank += (o > mine || (o == mine && j < lane)) ? 1 : 0;
        }
        if (wrank < m) s_top[warp * m + wrank] = mine;
        __syncthreads();
        const int nt = kWarps * m;
        if (tid < nt) {
            const float t = s_top[tid];
            int rank = 0;
            for (int j = 0; j < nt; ++j) {
                const float o = s_top[j];
                rank += (o > t || (o == t && j < tid)) ? 1 : 0;
            }
            if (rank == k - 1 && t > -INFINITY) atomicMax(&s_floor, tk_enc(t));
        }
        __syncthreads();
    }

    auto scan = [&](int v0) {
        const float floor_v = tk_dec(*(volatile unsigned *)&s_floor);
        bool appended = false;
        if (bm >= floor_v) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (E::to_float(q[u]) >= floor_v) {
                    unsigned em = 0;
#pragma unroll
                    for (int e = 0; e < E::kVec; ++e) {
                        const float x = E::elem(v[u], e);
                        em |= (x >= floor_v && x > -INFINITY) ? (1u << e) : 0u;
                    }
                    const int base = vlo + (v0 + u * kTkThreads) * E::kVec;
                    while (em) {
                        const int e = __ffs(em) - 1;
                        em &= em - 1;
                        append(E::elem(v[u], e), base + e);
                        appended = true;
                    }
                }
            }
        }
        if (__any_sync(0xffffffffu, appended)) drain(false);
    };

    scan(tid);
    for (int bi = 1; bi < nfull; ++bi) {
        bm = load_batch<DT, U, false>(vbase, bi * kBatchVecs + tid, nvec, v, q);
        scan(bi * kBatchVecs + tid);
    }
    if (nfull > 0 && nfull * kBatchVecs < nvec) {
        bm = load_batch<DT, U, true>(vbase, nfull * kBatchVecs + tid, nvec, v, q);
        scan(nfull * kBatchVecs + tid);
    }
    __syncthreads();
    if (s_overflow) {
        // The queue ran out of room (adversarially ordered data): redo the slice with the exact
        // per-warp lists, which leave the slice's ordered list in the workspace.
        const long long xrow = (long long)blockIdx.x / p.S;
        const int xlo = (int)((long long)blockIdx.x - xrow * p.S) * p.L;
        topk_slice_exact<DT>((const char *)p.logits + (size_t)xrow * (size_t)p.ld * E::kBytes, xlo,
                             min(p.V, xlo + p.L), p.k, p.partial + (size_t)blockIdx.x * p.k, s_cand,
                             s_xlist, s_xqn, &s_floor);
        __threadfence_block();
        __syncthreads();
    }
    if (warp == 0) {
        Cand c; c.z = -INFINITY; c.id = kNoId;   // ordered; unused entries are {-inf, kNoId}
        if (s_overflow) {
            if (lane < k) c = p.partial[(size_t)blk * k + lane];
        } else {
            drain(true);                         // whatever is still queued
            __syncwarp();
            c = s_list[lane];
        }
        if (p.S > 1) {
            if (!s_overflow && lane < k) p.partial[(size_t)blk * k + lane] = c;
        } else {
            // a whole row: the list is the row's result, write it out here
            float *ov = p.out_val + (size_t)row * k;
            int32_t *oi = p.out_id + (size_t)row * k;
            const bool real = lane < k && c.id != kNoId;
            if (real) { ov[lane] = c.z + 0.0f; oi[lane] = c.id; }
            const int found = __popc(__ballot_sync(0xffffffffu, real));
            __syncwarp();
            if (lane == 0 && found < k) complete_row(ov, oi, found, k);
        }
    }
}

// Rows that were split over several blocks: merge the S ordered slice lists of a row, complete the
// row if it has fewer than k entries above -inf, and write it best first.  One block per row.
// (Rows that one block streamed whole are written by that block; this kernel is not launched.)
// The lists prove lower bounds on the row's k-th value (see below); only entries at or above
// the largest bound can be in the result or ahead of one that is, so only they are kept and
// ranked against each other (of up to S k entries, k plus a few dozen).
__global__ void __launch_bounds__(kTkMergeThreads) topk_merge_kernel(const TopkParams p)
{
    extern __shared__ Cand s_c[];            // [n] the slices' lists, then [n] the entries kept
    __shared__ int s_found, s_nkeep;
    __shared__ unsigned s_thr;
    pdl_launch_dependents();     // the next call's slice kernel may be scheduled (it waits for this one)
    const int k = p.k, n = p.S * k;
    Cand *s_keep = s_c + n;
    const long long row = blockIdx.x;
    const Cand *src = p.partial + (size_t)row * n;
    if (threadIdx.x == 0) { s_found = 0; s_nkeep = 0; s_thr = tk_enc(-INFINITY); }
    pdl_wait();                  // scheduled while the slice kernel runs: its lists are complete after this
    for (int i = threadIdx.x; i < n; i += blockDim.x) s_c[i] = src[i];
    __syncthreads();
    // Two lower bounds on the row's k-th value: the last entry of any full list, and, with
    // pp + 1 = ceil(k / S) and m = ceil(k / (pp + 1)), the m-th largest of the lists' entries at
    // position pp (m lists hold pp + 1 entries each at or above it: k or more in all).
    const int pp = (k + p.S - 1) / p.S - 1, m = (k + pp) / (pp + 1);
    for (int sl = threadIdx.x; sl < p.S; sl += blockDim.x) {
        const Cand last = s_c[sl * k + k - 1];
        if (last.id != kNoId) atomicMax(&s_thr, tk_enc(last.z));
        const Cand a = s_c[sl * k + pp];
        if (a.id != kNoId) {
            int ahead = 0;
            for (int s2 = 0; s2 < p.S; ++s2) {
                const Cand b = s_c[s2 * k + pp];
                ahead += (b.id != kNoId && (b.z > a.z || (b.z == a.z && s2 < sl))) ? 1 : 0;
            }
            if (ahead == m - 1) atomicMax(&s_thr, tk_enc(a.z));
        }
    }
    __syncthreads();
    const float thr = tk_dec(s_thr);
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const Cand c = s_c[i];
        if (c.id != kNoId && c.z >= thr) s_keep[atomicAdd(&s_nkeep, 1)] = c;
    }
    __syncthreads();
    const int nk = s_nkeep;
    float *ov = p.out_val + (size_t)row * k;
    int32_t *oi = p.out_id + (size_t)row * k;
    for (int i = threadIdx.x; i < nk; i += blockDim.x) {
        const Cand c = s_keep[i];
        int rank = 0;
#pragma unroll 8
        for (int j = 0; j < nk; ++j) {
            const Cand o = s_keep[j];
            rank += beats(o.z, o.id, c.z, c.id) ? 1 : 0;
        }
        if (rank < k) { ov[rank] = c.z + 0.0f; oi[rank] = c.id; atomicAdd(&s_found, 1); }
    }
    __syncthreads();
    if (threadIdx.x == 0 && s_found < k) complete_row(ov, oi, s_found, k);
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
    return (size_t)rows * sp.S * (k * sizeof(mars::Cand));
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
    const size_t need = (size_t)rows * sp.S * (k * sizeof(Cand));
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return MARS_ERR_WORKSPACE;
    TopkParams p;
    p.logits = logits; p.ld = ld; p.V = V; p.S = sp.S; p.L = sp.L; p.k = k;
    p.partial = (Cand *)workspace;
    p.nslices = rows * sp.S;
    p.out_val = out_val; p.out_id = out_id;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const unsigned grid = (unsigned)(rows * sp.S);
    {
        const bool overlap = hook(kHookNoOverlap) == 0;
        // Two shapes of the same kernel.  8 vectors per batch and 4 blocks per SM is the faster
        // one nearly everywhere; with k above 16 on many long bf16 rows the kernel is bound by
        // instruction issue in its list and queue code, and 4 vectors per batch with 6 blocks per
        // SM (40 registers) gives the schedulers more warps to choose from (k = 32: 6-12 % faster
        // from 3 552 rows of 151 936 on; 15-20 % slower on rows of 32 000, slower at k = 10).
        const int variant = hook(kHookTopkVariant);
        const bool dense = variant ? variant == 2
                                   : (dt == MARS_BF16 && sp.S == 1 && k > 16 && V >= 65536 &&
                                      rows >= kTkDenseMinRows);
        const cudaError_t le =
            dense ? ((dt == MARS_BF16)
                         ? launch_pdl(overlap, topk_slice_kernel<MARS_BF16, 4, 6>, dim3(grid), dim3(kTkThreads), 0, st, p)
                         : launch_pdl(overlap, topk_slice_kernel<MARS_FP32, 4, 6>, dim3(grid), dim3(kTkThreads), 0, st, p))
                  : ((dt == MARS_BF16)
                         ? launch_pdl(overlap, topk_slice_kernel<MARS_BF16, kTkU, 4>, dim3(grid), dim3(kTkThreads), 0, st, p)
                         : launch_pdl(overlap, topk_slice_kernel<MARS_FP32, kTkU, 4>, dim3(grid), dim3(kTkThreads), 0, st, p));
        if (le != cudaSuccess) { (void)cudaGetLastError(); return MARS_ERR_CUDA; }
    }
    if (sp.S > 1) {
        const bool overlap = hook(kHookNoOverlap) == 0;
        const cudaError_t le = launch_pdl(overlap, topk_merge_kernel, dim3((unsigned)rows), dim3(kTkMergeThreads),
                                          2 * (size_t)sp.S * k * sizeof(Cand), st, p);
        if (le != cudaSuccess) { (void)cudaGetLastError(); return MARS_ERR_CUDA; }
    }
    return cudaGetLastError() == cudaSuccess ? MARS_OK : MARS_ERR_CUDA;
}

}  // extern "C"
