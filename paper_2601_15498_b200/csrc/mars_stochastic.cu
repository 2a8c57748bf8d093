// libmars: stochastic (temperature T > 0) verification.
//
// Sec. 2.2 of the paper: a drafted token is accepted with probability min(1, P_target/P_draft)
// (Eq. 1), a rejection draws the correction from the residual distribution, and tree methods
// apply the same logic to a token tree; P is the softmax of the logits (Eq. 3).  Draft trees are
// top-k expansions (Sec. 4.1), so a candidate's draft distribution is a point mass and Eq. 1
// reads "accept x with probability P(x)" under the running residual (P with the rejected
// siblings removed).  How the margin rule composes with Eq. 1 is a reading of this library,
// selected by flags (see mars.h).
//
// Two kernels per call:
//
//   stoch_stream_kernel   one pass over every logits row, as in the deterministic path (16-byte
//       streaming loads, filtered exact top-2 in registers), that also accumulates the softmax
//       denominator online: every thread keeps a reference `ref` (its largest batch maximum
//       times c = log2(e)/T) and sum = SUM 2^(z*c - ref); the reference only moves when a
//       batch maximum exceeds it, which the top-2 filter computes anyway.  One 32-byte record
//       {z1, id1, z2, id2, ref, sum} per slice.
//   stoch_tail_kernel     one thread-block cluster (1 to 8 blocks) per sequence: merges slice
//       records, gathers the logit of every node's token from its parent's row (one scalar load
//       per node, all in parallel), walks the tree (Eq. 1 on the running residual, or the margin
//       rule), then draws the next token from the residual of the row where the walk stopped by
//       inverting its CDF in token-id order: per-tile sums spread over the cluster's shared
//       memories, an fp64 prefix over them by the leader, then one tile and one element.
//
// A template flag of the tail covers chains whose drafts were sampled from a drafter's
// distribution Q (Eq. 1 in its general form): the test carries Q(x) and the residual is
// max(0, P - Q), read from the target's and the drafter's row of the rejected position.
#include "mars_top2_stream.cuh"

#include <cooperative_groups.h>

#include <cmath>

#include "mars.h"

namespace mars {

struct __align__(16) SRec {
    float z1; int id1; float z2; int id2;
    float ref;   // scaled reference: weights are 2^(z*c - ref)
    float sum;   // SUM of those weights over the slice
    int pad0, pad1;
};

__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// (ref, sum) of the union of two disjoint element sets.
__device__ __forceinline__ void soft_merge(float &ref, float &sum, float ref_b, float sum_b)
{
    const float r = fmaxf(ref, ref_b);
    if (r == -INFINITY) { ref = r; sum = 0.0f; return; }
    sum = sum * ex2f(ref - r) + sum_b * ex2f(ref_b - r);
    ref = r;
}

// One element joins (ref, sum); NaN counts as -inf (weight 0), +inf makes the sum infinite.
__device__ __forceinline__ void soft_add_scalar(float &ref, float &sum, float x, float c)
{
    if (!(x == x)) return;
    const float xc = x * c;
    if (xc > ref) { sum *= ex2f(ref - xc); ref = xc; }
    if (ref > -INFINITY) {
        const float t = fmaf(x, c, -ref);
        sum += (t == t) ? ex2f(t) : INFINITY;
    }
}

// ---- packed fp32 pairs (one instruction for two lanes of work) ----------------------------
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c)
{
    float2 d;
    asm("{ .reg .b64 ra, rb, rc, rd; mov.b64 ra, {%2,%3}; mov.b64 rb, {%4,%5}; mov.b64 rc, {%6,%7};\n"
        "fma.rn.f32x2 rd, ra, rb, rc; mov.b64 {%0,%1}, rd; }"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
    return d;
}
__device__ __forceinline__ float2 add2(float2 a, float2 b)
{
    float2 d;
    asm("{ .reg .b64 ra, rb, rd; mov.b64 ra, {%2,%3}; mov.b64 rb, {%4,%5};\n"
        "add.rn.f32x2 rd, ra, rb; mov.b64 {%0,%1}, rd; }"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}

// Rare path of soft_batch: the batch's sum of weights came out NaN, i.e. the batch holds a NaN
// logit (which counts as -inf: weight 0) or a +inf logit against an infinite reference (the
// row has no softmax; the sum is made infinite so that the tail reports it).  Re-reads the
// thread's elements one by one; kept out of line so that the fast path carries none of it.
template <int DT>
__device__ __noinline__ float soft_batch_slow(const uint4 *vbase, int v0, int nvec, int U, float c, float nref)
{
    typedef Elem<DT> E;
    float bs = 0.0f;
    for (int u = 0; u < U; ++u) {
        const int vi = v0 + u * kThreads;
        if (vi >= nvec) continue;
        for (int k = 0; k < E::kVec; ++k) {
            const float x = E::scalar(vbase, vi * E::kVec + k);
            if (x == x) {
                const float t = fmaf(x, c, nref);
                bs += (t == t) ? ex2f(t) : INFINITY;
            }
        }
    }
    return bs;
}

// A batch joins (ref, sum).  bm is the batch maximum (NaN operands ignored by the packed max).
// Elements are handled in pairs with packed fp32 instructions (one FMA and one add per pair);
// the 2^t themselves come from the exponential unit, 16 results per clock and SM, which is the
// tightest limit for bf16 rows at HBM speed.  (Moving a share of them to a polynomial on the
// FMA pipe was measured and lost: the extra issue slots cost more than the unit gained.)  The
// fast loop carries no per-element NaN test: a NaN shows in the batch's sum and sends the
// batch to the slow path.  (Also measured and dropped: a reference that moves only when a batch
// maximum exceeds it by a slack of 64, through an out-of-line call, to save the rescaling
// exponential per batch -- 19 % more cycles on bf16 rows at full clock.)
template <int DT, int U>
__device__ __forceinline__ void soft_batch(const uint4 (&v)[U], float bm, float c, float &ref, float &sum,
                                           const uint4 *vbase, int v0, int nvec)
{
    typedef Elem<DT> E;
    const float bmc = bm * c;
    if (bmc > ref) { sum *= ex2f(ref - bmc); ref = bmc; }
    if (!(ref > -INFINITY)) return;          // nothing above -inf seen so far: all weights are 0
    const float2 nref2 = make_float2(-ref, -ref), c2 = make_float2(c, c);
    float2 a0 = make_float2(0.0f, 0.0f), a1 = a0;
#pragma unroll
    for (int u = 0; u < U; ++u) {
#pragma unroll
        for (int k = 0; k < E::kVec; k += 2) {
            const int pair = u * (E::kVec / 2) + k / 2;
            const float2 t = fma2(make_float2(E::elem(v[u], k), E::elem(v[u], k + 1)), c2, nref2);
            float2 e;
            e.x = ex2f(t.x);
            e.y = ex2f(t.y);
            if (pair & 1) a1 = add2(a1, e); else a0 = add2(a0, e);
        }
    }
    a0 = add2(a0, a1);
    float bs = a0.x + a0.y;
    if (!(bs == bs)) bs = soft_batch_slow<DT>(vbase, v0, nvec, U, c, -ref);
    sum += bs;
}

// Batch load split in two, so that the next batch's loads can be in flight while the current
// batch is worked on: issue the 16-byte loads, and later reduce the vectors to their maxima.
template <int U>
__device__ __forceinline__ void issue_batch(const uint4 *vbase, int v0, uint4 (&v)[U])
{
#pragma unroll
    for (int u = 0; u < U; ++u) v[u] = ld_stream(vbase + v0 + u * kThreads);
}

template <int DT, int U>
__device__ __forceinline__ float reduce_batch(const uint4 (&v)[U], typename Elem<DT>::packed_t (&q)[U])
{
    typedef Elem<DT> E;
#pragma unroll
    for (int u = 0; u < U; ++u) q[u] = E::vred(v[u]);
    typename E::packed_t m[U / 2];
#pragma unroll
    for (int u = 0; u < U / 2; ++u) m[u] = E::pmax(q[2 * u], q[2 * u + 1]);
#pragma unroll
    for (int w = U / 4; w > 0; w >>= 1)
#pragma unroll
        for (int u = 0; u < w; ++u) m[u] = E::pmax(m[u], m[u + w]);
    return E::to_float(m[0]);
}

// ------------------------------------------------------------------- per-sequence tail

struct StochTailParams {
    const void *logits;
    long long ld;
    int V, N, S;
    float c, theta;
    uint32_t flags;
    int chain;
    int Dcap;
    const SRec *partial;     // [B*N*S]
    const int32_t *tok;      // tree [B,N]; chain: draft [B,N-1]
    const int32_t *parent;   // tree [B,N] or [N]
    const float *uniform;    // [B,N]
    // vocabulary-sharded form (mode 2): `logits` is this rank's column range [id_offset, id_offset+V)
    const SRec *records_all;      // [G_shards, B*N] records of all shards, global token ids
    const float *node_logit_all;  // [G_shards, B*N] logit of tok[i] in its parent's row where the shard holds it, else NaN
    int shards, my_shard, id_offset;
    int32_t *token_part;          // [B] the drawn token (global id) if this shard owns it, else -1
    const float *qx;         // sampled chains: [B,N-1] probability with which each draft was drawn
    const void *qlogits;     // sampled chains: drafter rows [B*(N-1), ldq], same dtype as logits
    long long ldq;
    float cq;                // log2(e) / T_draft
    int32_t *accept_len, *out_tokens, *path_nodes, *out_len, *seq_status;
    float *node_prob;        // [B,N] or null
    uint8_t *node_how;       // [B,N] or null
};

__host__ __device__ inline size_t stoch_tail_smem_bytes(int N)
{
    return (size_t)N * (9 * 4 + 3) + 64;
}

// The kVec logits that `lane` owns in 32-lane tile `tile` of a row (element j0 = (tile*32 +
// lane)*kVec onwards) as one 16-byte vector; elements beyond V read as -inf.  Rows that are not
// 16-byte aligned, and the last partial vector, are gathered element by element.
template <int DT>
__device__ __forceinline__ uint4 tile_load(const char *rowp, bool aligned, int V, long long tile, int lane)
{
    typedef Elem<DT> E;
    const long long j0 = (tile * 32 + lane) * E::kVec;
    if (aligned && j0 + E::kVec <= V) return __ldg(reinterpret_cast<const uint4 *>(rowp + (size_t)j0 * E::kBytes));
    uint32_t wds[4];
    if (DT == MARS_BF16) {
        const unsigned short *r = reinterpret_cast<const unsigned short *>(rowp);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t lo = (j0 + 2 * k < V) ? r[j0 + 2 * k] : 0xff80u;
            const uint32_t hi = (j0 + 2 * k + 1 < V) ? r[j0 + 2 * k + 1] : 0xff80u;
            wds[k] = lo | (hi << 16);
        }
    } else {
        const uint32_t *r = reinterpret_cast<const uint32_t *>(rowp);
#pragma unroll
        for (int k = 0; k < 4; ++k) wds[k] = (j0 + k < V) ? r[j0 + k] : 0xff800000u;
    }
    return make_uint4(wds[0], wds[1], wds[2], wds[3]);
}

// Weights 2^(z*c - ref) of those elements, zero for NaN / -inf logits and for removed tokens.
template <int DT>
__device__ __forceinline__ void tile_weights(const uint4 &raw, long long tile, int lane, float c, float nref,
                                             const int32_t *removed, int nrem, float (&w)[Elem<DT>::kVec])
{
    typedef Elem<DT> E;
    const long long j0 = (tile * 32 + lane) * E::kVec;
#pragma unroll
    for (int k = 0; k < E::kVec; ++k) {
        // NaN -> -inf with one max (weight 0); the reference of a row that is drawn from is finite
        // and at least every z*c, so the exponent is never NaN or positive beyond rounding
        const float x = fmaxf(E::elem(raw, k), -INFINITY);
        w[k] = ex2f(fmaf(x, c, nref));
    }
    for (int r = 0; r < nrem; ++r) {
        const int d = removed[r] - (int)j0;
        if (d >= 0 && d < E::kVec) {
#pragma unroll
            for (int k = 0; k < E::kVec; ++k) if (k == (int)d) w[k] = 0.0f;
        }
    }
}

// ---- the per-sequence tail kernel ---------------------------------------------------------
//
// One thread-block cluster per sequence: a single block when the batch alone fills the GPU, up to
// eight blocks when it does not, so that a lone sequence's draw still reads its row with eight
// SMs.  Every block of a cluster prepares and walks the tree redundantly (the walk is
// deterministic and cheap); the draw's pass over the row is shared: block r sums tiles
// [r*tpc, (r+1)*tpc) into per-tile sums in ITS shared memory, and after a cluster barrier the
// leader scans all of them through distributed shared memory, finds the tile that holds u*W
// and resolves the element.  Rows with more tiles than the per-block table holds (|V| above
// 262 144 bf16 / 131 072 fp32 logits) take the table-free multi-level search in one block.
constexpr int kTailThreads = 512;
constexpr int kTailWarps = kTailThreads / 32;
constexpr int kMaxTilesPerBlock = 1024;   // per-tile sums kept in shared memory (8 KB)
constexpr int kTailCluster = 8;

struct TailShared {
    double tile[kMaxTilesPerBlock];
    double part[kTailWarps];
    double wtot[kTailWarps];
    int whit[kTailWarps];
    float2 qwarp[kTailWarps];
    float2 qstat;
    double target;
    long long range[2];
    int ctl[8];       // 0 cur, 1 accept_len, 2 status, 3 nrem, 4 draw?, 5 picked token, 6 last tile with mass,
                      // 7 node of the rejected draft (sampled chains) or -1
    int pick_tile;
    int gstar;            // sharded form: the shard that owns the drawn token
    double target_abs;    // ... and the mass that lies before it inside that shard
};

// static + dynamic shared memory of the tail stay within the 48 KB that need no opt-in, up to the node cap
static_assert(sizeof(TailShared) + MARS_MAX_NODES * (9 * 4 + 3) + 64 + 256 <= 48 * 1024,
              "tail kernel: shared memory above 48 KB at MARS_MAX_NODES");

// ---- what a lane's elements of a tile weigh in the draw ----
// One row: 2^(z*c - ref), removed tokens at zero (the residual of point-mass drafts).
template <int DT>
struct ResidualOfRow {
    const char *rowp; bool aligned; int V; float c, nref; const int32_t *removed; int nrem;
    struct Raw { uint4 a; };
    __device__ __forceinline__ Raw load(long long tile, int lane) const
    {
        Raw r;
        r.a = tile_load<DT>(rowp, aligned, V, tile, lane);
        return r;
    }
    __device__ __forceinline__ void weights(const Raw &r, long long tile, int lane, float (&w)[Elem<DT>::kVec]) const
    {
        tile_weights<DT>(r.a, tile, lane, c, nref, removed, nrem, w);
    }
};

// A target row and the drafter's row: max(0, P - Q) on normalised probabilities (the residual of
// Eq. 1 for sampled drafts).
template <int DT>
struct ResidualOfPair {
    const char *rowp, *rowq; bool aligned_p, aligned_q; int V;
    float c, nref, inv_s, cq, nrefq, inv_sq;
    struct Raw { uint4 a, b; };
    __device__ __forceinline__ Raw load(long long tile, int lane) const
    {
        Raw r;
        r.a = tile_load<DT>(rowp, aligned_p, V, tile, lane);
        r.b = tile_load<DT>(rowq, aligned_q, V, tile, lane);
        return r;
    }
    __device__ __forceinline__ void weights(const Raw &r, long long, int, float (&w)[Elem<DT>::kVec]) const
    {
        typedef Elem<DT> E;
#pragma unroll
        for (int k = 0; k < E::kVec; ++k) {
            const float x = E::elem(r.a, k), y = E::elem(r.b, k);
            const float tp = fmaf(x, c, nref), tq = fmaf(y, cq, nrefq);
            const float pp = (x == x && tp == tp) ? ex2f(tp) * inv_s : 0.0f;
            const float qq = (y == y && tq == tq) ? ex2f(tq) * inv_sq : 0.0f;
            w[k] = fmaxf(pp - qq, 0.0f);
        }
    }
};

template <int DT, class WF>
__device__ __forceinline__ float lane_sum(const WF &wf, const typename WF::Raw &raw, long long tile, int lane)
{
    float w[Elem<DT>::kVec];
    wf.weights(raw, tile, lane, w);
    float ls = 0.0f;
#pragma unroll
    for (int k = 0; k < Elem<DT>::kVec; ++k) ls += w[k];
    return ls;
}

// Element inside one tile (warp-wide): lane prefix, then the element inside the lane.  `target` is
// the mass that lies before the wanted element within the tile, or, with whole_row, the tile is the
// whole row and the target is u * (its total).  Returns false if the tile holds no mass.
template <int DT, class WF>
__device__ __forceinline__ bool draw_in_tile(const WF &wf, long long t0, int lane, double target, bool whole_row,
                                             float u, int *picked)
{
    typedef Elem<DT> E;
    float w[E::kVec];
    wf.weights(wf.load(t0, lane), t0, lane, w);
    double ls = 0.0;
#pragma unroll
    for (int k = 0; k < E::kVec; ++k) ls += (double)w[k];
    double inc = ls;
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) {
        const double o = __shfl_up_sync(0xffffffffu, inc, m);
        if (lane >= m) inc += o;
    }
    const double total = __shfl_sync(0xffffffffu, inc, 31);
    bool good = true;
    if (whole_row) {
        good = (total > 0.0 && total < (double)INFINITY);
        if (u >= 0.0f) target = (double)u * total;      // u < 0: `target` is already absolute
    }
    // the first lane WITH mass whose inclusive prefix passes the target (a warp scan of floating-
    // point numbers need not be monotone to the last bit, hence the explicit conditions)
    const unsigned hit = __ballot_sync(0xffffffffu, inc > target && ls > 0.0);
    const unsigned pos = __ballot_sync(0xffffffffu, ls > 0.0);
    const int src = hit ? (__ffs(hit) - 1) : (pos ? 31 - __clz(pos) : -1);
    if (!good || src < 0) return false;
    if (lane == src) {
        const double tl = fmax(target - (inc - ls), 0.0);
        int pick = -1, lastpos = -1;
        double cum = 0.0;
#pragma unroll
        for (int k = 0; k < E::kVec; ++k) {
            if (w[k] > 0.0f) lastpos = k;
            cum += (double)w[k];
            if (pick < 0 && cum > tl) pick = k;
        }
        if (pick < 0) pick = lastpos;
        *picked = (int)((t0 * 32 + lane) * E::kVec) + pick;
    }
    return true;
}

// CDF inversion over the weights `wf` of one row of V elements with the uniform u0, by every thread
// of every block of the cluster (the condition to call it is the same in all of them).  On return
// the leader's sh.ctl[5] holds the drawn token, or sh.ctl[2] == 4 if the weights have no mass.
template <int DT, class WF>
__device__ void draw_token(cooperative_groups::cluster_group &cluster, TailShared &sh, const WF &wf, int V, float u0,
                           const double *target_abs = nullptr)
{
    typedef Elem<DT> E;
    const int G = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
    const bool leader = rank == 0;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long ntiles = ((long long)V + 32 * E::kVec - 1) / (32 * E::kVec);
    const long long tpc = (ntiles + G - 1) / G;          // tiles per block of the cluster
    if (tpc <= kMaxTilesPerBlock) {                       // the host launches clusters only if this holds
        // (1) every block: per-tile sums of its share of the row
        const long long t_lo = min(ntiles, (long long)rank * tpc), t_hi = min(ntiles, t_lo + tpc);
        // up to eight tiles per warp at a time, fewer when the block's share is small, so that all
        // warps take part
        const int per = (int)min(8ll, max(1ll, (t_hi - t_lo + kTailWarps - 1) / kTailWarps));
        for (long long t = t_lo + warp * per; t < t_hi; t += kTailWarps * per) {
            typename WF::Raw raw[8];
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (i < per && t + i < t_hi) raw[i] = wf.load(t + i, lane);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (i < per && t + i < t_hi) {
                    float ls = lane_sum<DT>(wf, raw[i], t + i, lane);
#pragma unroll
                    for (int m = 16; m > 0; m >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, m);
                    if (lane == 0) sh.tile[t + i - t_lo] = (double)ls;
                }
            }
        }
        cluster.sync();
        // (2) the leader: prefix over all tile sums (its own and, through distributed shared
        // memory, the other blocks'), a contiguous chunk of tiles per thread
        if (leader) {
            const int chunk = (int)((ntiles + kTailThreads - 1) / kTailThreads);
            const long long c_lo = min(ntiles, (long long)tid * chunk), c_hi = min(ntiles, c_lo + chunk);
            auto tile_sum = [&](long long t) -> double {
                const int owner = (int)(t / tpc);
                const double *base = (owner == 0) ? sh.tile : cluster.map_shared_rank(sh.tile, owner);
                return base[t - owner * tpc];
            };
            double mine = 0.0;
            int lastpos = -1;
            for (long long t = c_lo; t < c_hi; ++t) {
                const double v = tile_sum(t);
                if (v > 0.0) lastpos = (int)t;
                mine += v;
            }
            double inc = mine;
#pragma unroll
            for (int m = 1; m < 32; m <<= 1) {
                const double o = __shfl_up_sync(0xffffffffu, inc, m);
                if (lane >= m) inc += o;
            }
            if (lane == 31) sh.wtot[warp] = inc;
            if (lastpos >= 0) atomicMax(&sh.ctl[6], lastpos);
            __syncthreads();
            double before = 0.0, Wt = 0.0;
            for (int k = 0; k < kTailWarps; ++k) { if (k < warp) before += sh.wtot[k]; Wt += sh.wtot[k]; }
            inc += before;
            const double target = target_abs ? *target_abs : (double)u0 * Wt;
            const bool good = (Wt > 0.0 && Wt < (double)INFINITY);
            // the first thread WITH mass whose inclusive prefix passes the target
            const unsigned hits = __ballot_sync(0xffffffffu, good && inc > target && mine > 0.0);
            const double prev = __shfl_up_sync(0xffffffffu, inc, 1);
            if (lane == 0) sh.whit[warp] = hits ? (__ffs(hits) - 1) : -1;
            if (tid == 0) { sh.pick_tile = -1; sh.target = 0.0; if (!good) sh.ctl[2] = 4; }
            __syncthreads();
            int wsel = -1;
            for (int k = kTailWarps - 1; k >= 0; --k) if (sh.whit[k] >= 0) wsel = k;
            if (warp == wsel && lane == sh.whit[wsel]) {
                double cum = (lane == 0) ? before : prev;
                int last_in_chunk = -1;
                for (long long t = c_lo; t < c_hi; ++t) {
                    const double v = tile_sum(t);
                    if (v > 0.0) last_in_chunk = (int)t;
                    if (v > 0.0 && cum + v > target) { sh.pick_tile = (int)t; sh.target = fmax(target - cum, 0.0); break; }
                    cum += v;
                }
                if (sh.pick_tile < 0) { sh.pick_tile = last_in_chunk; sh.target = (double)INFINITY; }
            }
            __syncthreads();
            if (good && warp == 0) {
                long long t0 = sh.pick_tile;
                double target_in = sh.target;
                if (t0 < 0) { t0 = sh.ctl[6]; target_in = (double)INFINITY; }   // rounding: the last tile with mass
                int picked = -1;
                bool ok = t0 >= 0;
                if (ok) ok = draw_in_tile<DT>(wf, t0, lane, target_in, false, 0.0f, &picked);
                ok = __all_sync(0xffffffffu, ok);
                const int all = __reduce_max_sync(0xffffffffu, picked);   // the resolving lane's element
                if (lane == 0) { if (!ok || all < 0) sh.ctl[2] = 4; else sh.ctl[5] = all; }
            }
            __syncthreads();
        }
        cluster.sync();     // the other blocks' tables stay alive until the leader has read them
    } else {
        // table-free search (one block): sum contiguous warp segments, descend into the segment that
        // holds the target, repeat down to one tile
        long long t0 = 0, t1 = ntiles;
        bool first = true, ok = true;
        while (t1 - t0 > 1) {
            const long long len = (t1 - t0 + kTailWarps - 1) / kTailWarps;
            const long long w0 = min(t1, t0 + warp * len), w1 = min(t1, w0 + len);
            double acc = 0.0;
            long long t = w0;
            for (; t + 8 <= w1; t += 8) {   // eight independent loads in flight per lane
                typename WF::Raw raw[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) raw[i] = wf.load(t + i, lane);
#pragma unroll
                for (int i = 0; i < 8; ++i) acc += (double)lane_sum<DT>(wf, raw[i], t + i, lane);
            }
            for (; t < w1; ++t) acc += (double)lane_sum<DT>(wf, wf.load(t, lane), t, lane);
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, m);
            if (lane == 0) sh.part[warp] = acc;
            __syncthreads();
            if (tid == 0) {
                double target;
                bool good = true;
                if (first) {
                    double Wt = 0.0;
                    for (int k = 0; k < kTailWarps; ++k) Wt += sh.part[k];
                    good = (Wt > 0.0 && Wt < (double)INFINITY);
                    target = target_abs ? *target_abs : (double)u0 * Wt;
                } else target = sh.target;
                int pick = -1, lastpos = -1;
                double cum = 0.0, before = 0.0;
                for (int k = 0; k < kTailWarps && pick < 0; ++k) {
                    if (sh.part[k] > 0.0) lastpos = k;
                    before = cum;
                    cum += sh.part[k];
                    if (cum > target) pick = k;
                }
                if (pick < 0) {   // rounding pushed the target past the total: the last part with mass
                    pick = lastpos;
                    before = 0.0;
                    for (int k = 0; k < pick; ++k) before += sh.part[k];
                }
                if (!good || pick < 0) { sh.ctl[2] = 4; sh.range[0] = 0; sh.range[1] = 0; }
                else {
                    sh.target = fmax(target - before, 0.0);
                    sh.range[0] = min(t1, t0 + pick * len);
                    sh.range[1] = min(t1, sh.range[0] + len);
                }
            }
            __syncthreads();
            t0 = sh.range[0]; t1 = sh.range[1];
            first = false;
            if (t1 <= t0) { ok = false; break; }
        }
        if (ok && warp == 0) {
            int picked = -1;
            bool fine = draw_in_tile<DT>(wf, t0, lane, first ? (target_abs ? *target_abs : 0.0) : sh.target, first,
                                         target_abs ? -1.0f : u0, &picked);
            fine = __all_sync(0xffffffffu, fine);
            const int all = __reduce_max_sync(0xffffffffu, picked);
            if (lane == 0) { if (!fine || all < 0) sh.ctl[2] = 4; else sh.ctl[5] = all; }
        }
        __syncthreads();
    }
}

// (ref, sum) of 2^(z*c - ref) over one row, by the whole cluster: every block covers its share of
// the tiles, the per-block results meet through distributed shared memory and every block ends up
// with the row's total (merged in rank order, so all blocks hold the same bits).
template <int DT>
__device__ void row_softmax_cluster(cooperative_groups::cluster_group &cluster, TailShared &sh, const char *rowp,
                                    bool aligned, int V, float c, float *ref_out, float *sum_out)
{
    typedef Elem<DT> E;
    const int G = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long ntiles = ((long long)V + 32 * E::kVec - 1) / (32 * E::kVec);
    const long long tpc = (ntiles + G - 1) / G;
    const long long t_lo = min(ntiles, (long long)rank * tpc), t_hi = min(ntiles, t_lo + tpc);
    float ref = -INFINITY, sum = 0.0f;
    for (long long t = t_lo + warp * 4; t < t_hi; t += kTailWarps * 4) {
        uint4 raw[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (t + i < t_hi) raw[i] = tile_load<DT>(rowp, aligned, V, t + i, lane);
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (t + i < t_hi) {
#pragma unroll
                for (int k = 0; k < E::kVec; ++k) soft_add_scalar(ref, sum, E::elem(raw[i], k), c);
            }
    }
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) {
        const float rb = __shfl_xor_sync(0xffffffffu, ref, m), sb = __shfl_xor_sync(0xffffffffu, sum, m);
        soft_merge(ref, sum, rb, sb);
    }
    if (lane == 0) sh.qwarp[warp] = make_float2(ref, sum);
    __syncthreads();
    if (tid == 0) {
        float r = sh.qwarp[0].x, q = sh.qwarp[0].y;
        for (int k = 1; k < kTailWarps; ++k) soft_merge(r, q, sh.qwarp[k].x, sh.qwarp[k].y);
        sh.qstat = make_float2(r, q);
    }
    cluster.sync();
    float r = -INFINITY, q = 0.0f;
    for (int g = 0; g < G; ++g) {
        const float2 v = (g == rank) ? sh.qstat : *cluster.map_shared_rank(&sh.qstat, g);
        soft_merge(r, q, v.x, v.y);
    }
    cluster.sync();     // no block may move on (and possibly exit) while another still reads its result
    *ref_out = r;
    *sum_out = q;
}

// MODE 1 (sampled): chains whose drafts were sampled from a drafter's distribution (general
// Eq. 1): the acceptance test carries the draft's own probability and the residual is max(0, P - Q).
// MODE 2 (sharded): the vocabulary is split over ranks; the rows' records and the candidates'
// logits of all shards have been gathered, every rank walks the tree identically, works out from
// the shards' masses which shard holds the drawn token, and only that rank reads its part of the
// row; the token is left in token_part for a last exchange.
template <int DT, int MODE>
__global__ void __launch_bounds__(kTailThreads, MODE == 1 ? 1 : 2) stoch_tail_kernel(const StochTailParams p)
{
    constexpr bool SAMPLED = MODE == 1;
    constexpr bool SHARDED = MODE == 2;
    typedef Elem<DT> E;
    namespace cg = cooperative_groups;
    extern __shared__ __align__(16) unsigned char smem_dyn[];
    __shared__ TailShared sh;
    cg::cluster_group cluster = cg::this_cluster();
    const int G = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const bool leader = rank == 0;
    (void)rank;
    const int b = (int)(blockIdx.x / G);
    const int N = p.N, V = p.V, S = p.S;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // The next call's streaming kernel may be scheduled while this kernel runs (and, if its caller
    // set MARS_LOGITS_READY, read its logits); it waits for this kernel before it writes records.
    pdl_launch_dependents();

    int32_t *s_id1 = reinterpret_cast<int32_t *>(smem_dyn);
    int32_t *s_id2 = s_id1 + N;
    int32_t *s_par = s_id2 + N;
    int32_t *s_tok = s_par + N;
    int32_t *s_removed = s_tok + N;
    float *s_ref = reinterpret_cast<float *>(s_removed + N);
    float *s_sum = s_ref + N;
    float *s_e = s_sum + N;
    float *s_u = s_e + N;
    unsigned char *s_relax = reinterpret_cast<unsigned char *>(s_u + N);
    unsigned char *s_how = s_relax + N;
    unsigned char *s_own = s_how + N;      // sharded form: the shard that holds the node's token (255: none)

    // ---- rows: merge the slice records (four records' loads in flight at a time) ----
    const int32_t *par_g = p.chain ? nullptr : ((p.flags & MARS_SHARED_PARENT) ? p.parent : p.parent + (size_t)b * N);
    int bad = 0;
    for (int i = tid; i < N; i += kTailThreads) {
        // slices of the row (contiguous records), or in the sharded form the row's record of every shard
        const int4 *src = SHARDED ? reinterpret_cast<const int4 *>(p.records_all + ((size_t)b * N + i))
                                  : reinterpret_cast<const int4 *>(p.partial + ((size_t)b * N + i) * S);
        const size_t step = SHARDED ? (size_t)2 * gridDim.x / G * N : 2;      // in int4 units (a record is two)
        Rec acc = empty_rec();
        float ref = -INFINITY, sum = 0.0f;
        for (int k0 = 0; k0 < S; k0 += 4) {
            int4 a[4], q[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (k0 + j < S) { a[j] = __ldcg(src + step * (k0 + j)); q[j] = __ldcg(src + step * (k0 + j) + 1); }
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (k0 + j < S) {
                    Rec r;
                    r.z1 = __int_as_float(a[j].x); r.id1 = a[j].y; r.z2 = __int_as_float(a[j].z); r.id2 = a[j].w;
                    acc = merge(acc, r);
                    soft_merge(ref, sum, __int_as_float(q[j].x), __int_as_float(q[j].y));
                }
        }
        acc = finish_record(acc);
        s_id1[i] = acc.id1;
        s_id2[i] = acc.id2;
        s_relax[i] = relax_bit(acc.z1, acc.z2, p.theta, p.flags) ? 1 : 0;
        s_ref[i] = ref;
        s_sum[i] = sum;
        int pa, tk;
        if (p.chain) {
            pa = i - 1;
            tk = i > 0 ? p.tok[(size_t)b * (N - 1) + (i - 1)] : -1;
        } else {
            pa = par_g[i];
            tk = p.tok[(size_t)b * N + i];
            if (i == 0 ? (pa != -1) : (pa >= i || pa < -1)) bad = 1;
        }
        s_par[i] = pa;
        s_tok[i] = tk;
        s_u[i] = p.uniform[(size_t)b * N + i];
        s_how[i] = 0;
    }
    bad = __syncthreads_or(bad);

    // every node's token under its parent's row: unnormalised mass, plain softmax probability
    for (int i = tid; i < N; i += kTailThreads) {
        float e = 0.0f, prob = 0.0f;
        const int pa = s_par[i], tk = s_tok[i];
        unsigned char own = 255;
        float xs = __int_as_float(0x7fc00000);
        if (SHARDED && !bad && i > 0 && pa >= 0 && tk >= 0) {
            // the one shard whose column range holds the token reported its logit, the others NaN
            const size_t R = (size_t)(gridDim.x / G) * N;
            for (int g = 0; g < S; ++g) {
                const float z = __ldcg(p.node_logit_all + (size_t)g * R + (size_t)b * N + i);
                if (z == z && own == 255) { xs = z; own = (unsigned char)g; }
            }
        }
        if (SHARDED) s_own[i] = own;
        if (!bad && i > 0 && pa >= 0 && tk >= 0 && (SHARDED ? own != 255 : tk < V)) {
            const float ref = s_ref[pa], sum = s_sum[pa];
            if (ref > -INFINITY && ref < INFINITY && sum > 0.0f && sum < INFINITY) {
                const char *rowp = (const char *)p.logits + ((size_t)b * N + pa) * (size_t)p.ld * E::kBytes;
                const float x = SHARDED ? xs : E::scalar(rowp, tk);
                const float t = fmaf(x, p.c, -ref);
                e = (x == x && t == t) ? ex2f(t) : 0.0f;
                prob = __fdiv_rn(e, sum);
            }
        }
        s_e[i] = e;
        if (leader && p.node_prob) p.node_prob[(size_t)b * N + i] = prob;
    }
    __syncthreads();

    // ---- the walk: warp 0; the children of the current node are found 32 nodes at a time with a
    // ballot and judged in node order; every lane carries the same state ----
    const int Wd = p.Dcap + 1;
    int32_t *o_tok = p.out_tokens + (size_t)b * Wd;
    int32_t *o_path = p.path_nodes ? p.path_nodes + (size_t)b * Wd : nullptr;
    if (warp == 0) {
        int cur = 0, a = 0, status = bad ? 1 : 0, nrem = 0, draw = 0, rejected = -1;
        if (leader) {
            for (int k = lane; k < Wd; k += 32) { o_tok[k] = -1; if (o_path) o_path[k] = (k == 0) ? 0 : -1; }
        }
        while (status == 0) {
            const float ref = s_ref[cur], sum = s_sum[cur];
            nrem = 0;
            if (SHARDED) {      // mass removed from each shard's part of this row (the tile table is idle here)
                for (int g = lane; g < S; g += 32) sh.tile[g] = 0.0;
                __syncwarp();
            }
            if (!(ref > -INFINITY && ref < INFINITY && sum > 0.0f && sum < INFINITY)) { status = 4; break; }
            float rem = sum;
            int next = -1;
            const int id1 = s_id1[cur], id2 = s_id2[cur], rlx = s_relax[cur];
            for (int base = cur + 1; base < N && next < 0; base += 32) {
                const int i = base + lane;
                unsigned kids = __ballot_sync(0xffffffffu, i < N && s_par[i] == cur && s_tok[i] >= 0);
                while (kids && next < 0) {
                    const int j = base + __ffs(kids) - 1;
                    kids &= kids - 1;
                    const int x = s_tok[j];
                    bool gone = false;
                    for (int k = 0; k < nrem; ++k) gone |= (s_removed[k] == x);
                    const float ex = gone ? 0.0f : s_e[j];
                    int how = 0;
                    if (!(p.flags & MARS_STOCH_PLAIN)) {
                        if (x == id1) how = (p.flags & MARS_STOCH_RELAX_ONLY) ? 0 : 1;
                        else if (x == id2 && rlx) how = 2;
                    }
                    if (how == 0) {
                        float lhs = s_u[j];
                        if (SAMPLED) lhs = __fmul_rn(lhs, p.qx[(size_t)b * (N - 1) + (j - 1)]);   // u * Q(x) < P(x)
                        how = (__fmul_rn(lhs, rem) < ex) ? 3 : 4;    // Eq. 1 on the running residual
                    }
                    if (lane == 0) s_how[j] = (unsigned char)how;
                    if (how == 4) {
                        if (SAMPLED) rejected = j;     // the residual needs the drafter's row, not a removal
                        else if (ex > 0.0f) {
                            rem = fmaxf(__fsub_rn(rem, ex), 0.0f);
                            if (SHARDED && lane == 0) sh.tile[s_own[j]] += (double)ex;
                            if (lane == 0) s_removed[nrem] = x;
                            ++nrem;
                            __syncwarp();
                        }
                    } else next = j;
                }
            }
            if (next < 0) { draw = 1; break; }
            cur = next; ++a;
            if (leader && lane == 0 && a <= p.Dcap) { o_tok[a - 1] = s_tok[cur]; if (o_path) o_path[a] = cur; }
        }
        if ((status == 0 || status == 4) && a > p.Dcap) status = 2;
        if (status == 1 || status == 2) {
            __syncwarp();
            if (leader)
                for (int k = lane; k < Wd; k += 32) { o_tok[k] = -1; if (o_path) o_path[k] = (k == 0) ? 0 : -1; }
            for (int i = lane; i < N; i += 32) s_how[i] = 0;
            cur = 0; a = 0; draw = 0; nrem = 0; rejected = -1;
        }
        if (lane == 0) {
            sh.ctl[0] = cur; sh.ctl[1] = a; sh.ctl[2] = status; sh.ctl[3] = nrem; sh.ctl[4] = draw;
            sh.ctl[5] = s_id1[cur]; sh.ctl[6] = -1; sh.ctl[7] = rejected;
        }
    }
    __syncthreads();

    // ---- the next token: CDF inversion over the residual of row `cur` ----
    const int cur = sh.ctl[0];
    if (sh.ctl[4]) {
        const char *rowp = (const char *)p.logits + ((size_t)b * N + cur) * (size_t)p.ld * E::kBytes;
        const bool aligned = (((uintptr_t)rowp) & 15) == 0;
        const int rejected = sh.ctl[7];
        if (SAMPLED && rejected >= 0) {
            // draft `rejected - 1` failed Eq. 1: draw from max(0, P - Q) with Q the drafter's row
            const char *rowq = (const char *)p.qlogits + ((size_t)b * (N - 1) + (rejected - 1)) * (size_t)p.ldq * E::kBytes;
            const bool aligned_q = (((uintptr_t)rowq) & 15) == 0;
            float refq, sumq;
            row_softmax_cluster<DT>(cluster, sh, rowq, aligned_q, V, p.cq, &refq, &sumq);
            if (!(refq > -INFINITY && refq < INFINITY && sumq > 0.0f && sumq < INFINITY)) {
                if (tid == 0) sh.ctl[2] = 4;      // the drafter's row has no softmax (same in every block)
            } else {
                ResidualOfPair<DT> wf;
                wf.rowp = rowp; wf.rowq = rowq; wf.aligned_p = aligned; wf.aligned_q = aligned_q; wf.V = V;
                wf.c = p.c; wf.nref = -s_ref[cur]; wf.inv_s = __fdiv_rn(1.0f, s_sum[cur]);
                wf.cq = p.cq; wf.nrefq = -refq; wf.inv_sq = __fdiv_rn(1.0f, sumq);
                draw_token<DT>(cluster, sh, wf, V, s_u[0]);
            }
        } else if (SHARDED) {
            // Which shard holds the drawn token follows from the shards' records: shard g's part of
            // the row weighs sum_g * 2^(ref_g - ref) minus what the walk removed from it.
            if (tid == 0) {
                const size_t R = (size_t)(gridDim.x / G) * N;
                const float ref = s_ref[cur];
                double Wt = 0.0;
                for (int g = 0; g < S; ++g) {
                    const SRec *r = p.records_all + (size_t)g * R + (size_t)b * N + cur;
                    const float rg = __ldcg(&r->ref), sg = __ldcg(&r->sum);
                    double m = (rg > -INFINITY) ? (double)(sg * ex2f(rg - ref)) - sh.tile[g] : 0.0;
                    if (!(m > 0.0)) m = 0.0;
                    sh.tile[g] = m;
                    Wt += m;
                }
                int pick = -1, lastpos = -1;
                double cum = 0.0, before = 0.0;
                const double target = (double)s_u[0] * Wt;
                for (int g = 0; g < S && pick < 0; ++g) {
                    if (sh.tile[g] > 0.0) lastpos = g;
                    before = cum;
                    cum += sh.tile[g];
                    if (sh.tile[g] > 0.0 && cum > target) pick = g;
                }
                if (pick < 0) {
                    pick = lastpos;
                    before = 0.0;
                    for (int g = 0; g < pick; ++g) before += sh.tile[g];
                }
                if (!(Wt > 0.0 && Wt < (double)INFINITY) || pick < 0) { sh.ctl[2] = 4; sh.gstar = -1; }
                else { sh.gstar = pick; sh.target_abs = fmax(target - before, 0.0); }
            }
            __syncthreads();
            // removed tokens as local column indices (those of other shards fall outside every tile)
            for (int k = tid; k < sh.ctl[3]; k += kTailThreads) {
                const int x = s_removed[k] - p.id_offset;
                s_removed[k] = (x >= 0 && x < V) ? x : -0x40000000;
            }
            __syncthreads();
            if (sh.gstar == p.my_shard) {        // the same decision in every block of the cluster
                ResidualOfRow<DT> wf;
                wf.rowp = rowp; wf.aligned = aligned; wf.V = V; wf.c = p.c; wf.nref = -s_ref[cur];
                wf.removed = s_removed; wf.nrem = sh.ctl[3];
                if (tid == 0) sh.ctl[5] = -1;
                __syncthreads();
                draw_token<DT>(cluster, sh, wf, V, s_u[0], &sh.target_abs);
                __syncthreads();
                if (tid == 0) {
                    if (sh.ctl[2] == 4 || sh.ctl[5] < 0) { sh.ctl[2] = 0; sh.ctl[5] = -1; }   // rounding left this shard empty
                    else sh.ctl[5] += p.id_offset;
                }
            } else if (tid == 0 && sh.gstar >= 0) sh.ctl[5] = -1;
        } else {
            ResidualOfRow<DT> wf;
            wf.rowp = rowp; wf.aligned = aligned; wf.V = V; wf.c = p.c; wf.nref = -s_ref[cur];
            wf.removed = s_removed; wf.nrem = sh.ctl[3];
            draw_token<DT>(cluster, sh, wf, V, s_u[0]);
        }
        __syncthreads();
    }

    if (SHARDED && leader && tid == 0) {
        // the drawn token travels separately: every rank reports the fallback (the row's top-1) for
        // sequences without a draw, the owning rank the drawn token, the others -1
        const int status = sh.ctl[2];
        p.token_part[b] = (status != 0 || !sh.ctl[4]) ? s_id1[cur] : sh.ctl[5];
        sh.ctl[5] = s_id1[cur];
    }
    if (leader && tid == 0) {
        const int a = sh.ctl[1], status = sh.ctl[2];
        p.out_tokens[(size_t)b * (p.Dcap + 1) + a] = (status == 4) ? s_id1[cur] : sh.ctl[5];
        p.accept_len[b] = a;
        p.out_len[b] = a + 1;
        if (p.seq_status) p.seq_status[b] = status;
    }
    if (leader && p.node_how)
        for (int i = tid; i < N; i += kTailThreads) p.node_how[(size_t)b * N + i] = s_how[i];
}

// ------------------------------------------------------------------------ streaming kernel

struct StreamParams {
    const void *logits;
    long long ld;
    int V;
    int S;       // slices per row
    int L;       // elements per slice (multiple of 16)
    float c;     // log2(e) / T
    SRec *partial;   // [R*S]
    int early;   // MARS_LOGITS_READY: stream the logits before waiting for the predecessor
};

template <int DT, int U, int MINB>
__global__ void __launch_bounds__(kThreads, MINB) stoch_stream_kernel(const StreamParams p)
{
    typedef Elem<DT> E;
    __shared__ unsigned sT[2];
    __shared__ Rec s_warp[kThreads / 32];
    __shared__ float2 s_soft[kThreads / 32];

    if (!p.early) pdl_wait();        // by default nothing is read before the predecessor is done
    const int tid = threadIdx.x;
    const long long blk = blockIdx.x;
    const long long row = blk / p.S;
    const int slice = (int)(blk - row * p.S);
    const float c = p.c;

    const int lo = slice * p.L;
    const int hi = min(p.V, lo + p.L);
    const char *rowp = (const char *)p.logits + (size_t)row * (size_t)p.ld * E::kBytes;

    // [lo, hi) = head scalars | 16-byte vectors | tail scalars
    const uintptr_t a0 = (uintptr_t)(rowp + (size_t)lo * E::kBytes);
    int nhead = (int)(((16 - (a0 & 15)) & 15) / E::kBytes);
    nhead = min(nhead, max(hi - lo, 0));
    const int vlo = lo + nhead;
    const int nvec = max(hi - vlo, 0) / E::kVec;
    const int tlo = vlo + nvec * E::kVec;
    const int ntail = max(hi - tlo, 0);
    const uint4 *vbase = (const uint4 *)(rowp + (size_t)vlo * E::kBytes);

    constexpr int kBatchVecs = kThreads * U;
    const int nfull = nvec / kBatchVecs;
    uint4 v[U];
    typename E::packed_t q[U];

    float bm = (nfull > 0) ? load_batch<DT, U, false>(vbase, tid, nvec, v, q)
                           : load_batch<DT, U, true>(vbase, tid, nvec, v, q);
    if (tid == 0) { sT[0] = enc(-INFINITY); sT[1] = enc(-INFINITY); }
    __syncthreads();

    Rec s = empty_rec();
    float ref = -INFINITY, sum = 0.0f;
    if (tid < nhead) {
        const float x = E::scalar(rowp, lo + tid);
        insert<false>(s, x, lo + tid, sT);
        soft_add_scalar(ref, sum, x, c);
    }
    {   // bootstrap of the shared runner-up bound from the first batch's maxima
        float a1 = (bm == bm) ? bm : -INFINITY, a2 = -INFINITY;
#pragma unroll
        for (int m = 16; m > 0; m >>= 1) {
            float b1 = __shfl_xor_sync(0xffffffffu, a1, m), b2 = __shfl_xor_sync(0xffffffffu, a2, m);
            a2 = fmaxf(fminf(a1, b1), fmaxf(a2, b2));
            a1 = fmaxf(a1, b1);
        }
        if ((tid & 31) == 0) { publish(sT, a1); publish(sT, a2); }
        __syncwarp();
    }
    float T2 = dec(*(volatile unsigned *)&sT[1]);
    soft_batch<DT, U>(v, bm, c, ref, sum, vbase, tid, nvec);
    process_batch<DT, U, false>(v, q, bm, T2, vlo + tid * E::kVec, s, sT);

    // ---- steady state: two register buffers; the loads of batch bi+1 are issued before batch
    // bi is worked on, so memory latency overlaps the exponentials ----
    {
        uint4 vb[U];
        auto consume = [&](const uint4 (&x)[U], int bi) {
            const float m = reduce_batch<DT, U>(x, q);
            const float t2 = dec(*(volatile unsigned *)&sT[1]);
            soft_batch<DT, U>(x, m, c, ref, sum, vbase, bi * kBatchVecs + tid, nvec);
            process_batch<DT, U, true>(x, q, m, t2, vlo + (bi * kBatchVecs + tid) * E::kVec, s, sT);
        };
        int bi = 1;
        if (bi < nfull) issue_batch<U>(vbase, bi * kBatchVecs + tid, vb);
        while (bi < nfull) {
            if (bi + 1 < nfull) issue_batch<U>(vbase, (bi + 1) * kBatchVecs + tid, v);
            consume(vb, bi);
            if (++bi >= nfull) break;
            if (bi + 1 < nfull) issue_batch<U>(vbase, (bi + 1) * kBatchVecs + tid, vb);
            consume(v, bi);
            ++bi;
        }
    }
    if (nfull > 0 && nfull * kBatchVecs < nvec) {
        bm = load_batch<DT, U, true>(vbase, nfull * kBatchVecs + tid, nvec, v, q);
        T2 = dec(*(volatile unsigned *)&sT[1]);
        soft_batch<DT, U>(v, bm, c, ref, sum, vbase, nfull * kBatchVecs + tid, nvec);
        process_batch<DT, U, true>(v, q, bm, T2, vlo + (nfull * kBatchVecs + tid) * E::kVec, s, sT);
    }
    if (tid < ntail) {
        const float x = E::scalar(rowp, tlo + tid);
        insert<false>(s, x, tlo + tid, sT);
        soft_add_scalar(ref, sum, x, c);
    }

    // ---- block merge: top-2 under the total order, (ref, sum) by rescaling ----
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) {
        s = merge(s, shfl_xor_rec(s, m));
        const float rb = __shfl_xor_sync(0xffffffffu, ref, m), sb = __shfl_xor_sync(0xffffffffu, sum, m);
        soft_merge(ref, sum, rb, sb);
    }
    if ((tid & 31) == 0) { s_warp[tid >> 5] = s; s_soft[tid >> 5] = make_float2(ref, sum); }
    // Up to here only this call's logits were read.  The records below go to the workspace, which
    // the previous call's tail kernel may still be reading: wait for it (see pdl_wait).
    pdl_wait();
    __syncthreads();
    if (tid == 0) {
        Rec r = s_warp[0];
        float rr = s_soft[0].x, ss = s_soft[0].y;
#pragma unroll
        for (int w = 1; w < kThreads / 32; ++w) {
            r = merge(r, s_warp[w]);
            soft_merge(rr, ss, s_soft[w].x, s_soft[w].y);
        }
        SRec o;
        o.z1 = r.z1; o.id1 = r.id1; o.z2 = r.z2; o.id2 = r.id2; o.ref = rr; o.sum = ss; o.pad0 = 0; o.pad1 = 0;
        p.partial[blk] = o;
    }
}

// (Running the tail inside the streaming kernel, by the block that delivers a sequence's last
// record as the deterministic path does, was measured and lost 20 %: the tail's registers and its
// latency-bound work do not fit a kernel tuned to keep 64 registers and four blocks per SM
// streaming.  It is a kernel of its own, launched behind the streaming kernel on the same stream.)

// ---- vocabulary-sharded form: step 1 and step 3 kernels --------------------------------------

struct ShardRecordsParams {
    const void *logits;      // this rank's columns [id_offset, id_offset + V) of every row
    long long ld;
    int V, N, S, id_offset;
    long long R;
    uint32_t flags;
    const SRec *partial;     // [R*S] from the streaming kernel
    const int32_t *tok, *parent;
    SRec *records;           // [R] out: the row's record over this shard, global token ids
    float *node_logit;       // [R] out: logit of tok[i] in its parent's row if this shard holds it, else NaN
};

template <int DT>
__global__ void stoch_shard_records_kernel(const ShardRecordsParams p)
{
    typedef Elem<DT> E;
    const long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= p.R) return;
    const int4 *src = reinterpret_cast<const int4 *>(p.partial + (size_t)r * p.S);
    Rec acc = empty_rec();
    float ref = -INFINITY, sum = 0.0f;
    for (int k = 0; k < p.S; ++k) {
        const int4 a = __ldcg(src + 2 * k), q = __ldcg(src + 2 * k + 1);
        Rec x;
        x.z1 = __int_as_float(a.x); x.id1 = a.y; x.z2 = __int_as_float(a.z); x.id2 = a.w;
        acc = merge(acc, x);
        soft_merge(ref, sum, __int_as_float(q.x), __int_as_float(q.y));
    }
    SRec o;
    o.z1 = acc.z1; o.id1 = acc.id1 == kNoId ? kNoId : acc.id1 + p.id_offset;
    o.z2 = acc.z2; o.id2 = acc.id2 == kNoId ? kNoId : acc.id2 + p.id_offset;
    o.ref = ref; o.sum = sum; o.pad0 = 0; o.pad1 = 0;
    p.records[r] = o;
    const long long b = r / p.N;
    const int i = (int)(r - b * p.N);
    float z = __int_as_float(0x7fc00000);
    if (i > 0) {
        const int pa = ((p.flags & MARS_SHARED_PARENT) ? p.parent : p.parent + (size_t)b * p.N)[i];
        const int x = p.tok[r] - p.id_offset;
        if (pa >= 0 && pa < i && p.tok[r] >= 0 && x >= 0 && x < p.V) {
            const char *rowp = (const char *)p.logits + ((size_t)b * p.N + pa) * (size_t)p.ld * E::kBytes;
            const float v = E::scalar(rowp, x);
            z = (v == v) ? v : -INFINITY;       // a NaN logit counts as -inf; NaN means "not in this shard"
        }
    }
    p.node_logit[r] = z;
}

// Step 3: the drawn token of every sequence is the one entry >= 0 among the ranks' reports (or
// the fallback that all ranks report alike); a sequence nobody could draw for keeps the fallback
// already in place and gets MARS_SEQ_BAD_DISTRIBUTION.
__global__ void stoch_shard_finish_kernel(const int32_t *token_all, int shards, int B, int W, const int32_t *accept_len,
                                          int32_t *out_tokens, int32_t *seq_status)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    int t = -1;
    for (int g = 0; g < shards; ++g) t = max(t, token_all[(size_t)g * B + b]);
    const int a = accept_len[b];
    if (t >= 0) out_tokens[(size_t)b * W + a] = t;
    else if (seq_status) seq_status[b] = MARS_SEQ_BAD_DISTRIBUTION;
}

// ------------------------------------------------------------------------------- host

static size_t stoch_ws_bytes(long long R, int S) { return ((size_t)R * S * sizeof(SRec) + 255) / 256 * 256; }

static bool stoch_sizes_supported(int B, int N, int V, int dt)
{
    if (B < 1 || N < 1 || V < 2) return false;
    if (dt != MARS_BF16 && dt != MARS_FP32) return false;
    if (N > MARS_MAX_NODES || V > (1 << 30)) return false;
    if ((long long)B * N > (1ll << 40)) return false;
    return true;
}

struct SampledDrafts {        // chains whose drafts were sampled from a drafter (general Eq. 1)
    const void *qlogits;
    int64_t ldq;
    const float *qx;
    float draft_temperature;
};

static mars_status_t run_stochastic(const void *logits, int64_t ld, mars_dtype_t dt, const int32_t *tok,
                                    const int32_t *parent, const float *uniform, const SampledDrafts *sd,
                                    int chain, int B, int N,
                                    int V, float theta, float temperature, uint32_t flags,
                                    int32_t *accept_len, int32_t *out_tokens, int32_t *path_nodes,
                                    int32_t *out_len, int Dcap, int32_t *seq_status, float *node_prob,
                                    uint8_t *node_how, void *workspace, size_t workspace_bytes,
                                    void *cuda_stream)
{
    if (B < 1 || N < 1 || V < 2 || !logits || !uniform) return MARS_ERR_INVALID_ARG;
    if (ld < V || Dcap < 0 || theta != theta) return MARS_ERR_INVALID_ARG;
    if (!(temperature > 0.0f) || !(temperature < INFINITY)) return MARS_ERR_INVALID_ARG;
    double cqd = 0.0;
    if (sd) {
        if (!chain) return MARS_ERR_INVALID_ARG;
        if (N > 1 && (!sd->qlogits || !sd->qx || sd->ldq < V)) return MARS_ERR_INVALID_ARG;
        if (!(sd->draft_temperature > 0.0f) || !(sd->draft_temperature < INFINITY)) return MARS_ERR_INVALID_ARG;
        if ((uintptr_t)sd->qlogits % (dt == MARS_BF16 ? 2 : 4)) return MARS_ERR_INVALID_ARG;
        cqd = 1.4426950408889634074 / (double)sd->draft_temperature;
        if (!(cqd < 3.0e38)) return MARS_ERR_INVALID_ARG;
    }
    if (!accept_len || !out_tokens || !out_len) return MARS_ERR_INVALID_ARG;
    if (!chain && (!tok || !parent)) return MARS_ERR_INVALID_ARG;
    if (chain && N > 1 && !tok) return MARS_ERR_INVALID_ARG;
    if (flags & ~(MARS_SIGN_LITERAL | MARS_SHARED_PARENT | MARS_RULE_MARGIN | MARS_RULE_PROB_RATIO |
                  MARS_STOCH_PLAIN | MARS_STOCH_RELAX_ONLY | MARS_LOGITS_READY))
        return MARS_ERR_UNSUPPORTED;
    if ((flags & MARS_RULE_MARGIN) && (flags & MARS_RULE_PROB_RATIO)) return MARS_ERR_INVALID_ARG;
    if ((flags & MARS_STOCH_PLAIN) && (flags & MARS_STOCH_RELAX_ONLY)) return MARS_ERR_INVALID_ARG;
    rule_threshold(&theta, &flags);
    if (!stoch_sizes_supported(B, N, V, (int)dt)) return MARS_ERR_UNSUPPORTED;
    const int es = dt == MARS_BF16 ? 2 : 4;
    if ((uintptr_t)logits % es) return MARS_ERR_INVALID_ARG;
    const double cd = 1.4426950408889634074 / (double)temperature;   // log2(e) / T
    if (!(cd < 3.0e38)) return MARS_ERR_INVALID_ARG;
    const long long R = (long long)B * N;
    const Split sp = choose_split(R, V, (int)dt);
    if (R * sp.S > 0x7fffffffll) return MARS_ERR_UNSUPPORTED;
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < stoch_ws_bytes(R, sp.S))
        return MARS_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    StreamParams sp1;
    sp1.logits = logits; sp1.ld = ld; sp1.V = V; sp1.S = sp.S; sp1.L = sp.L; sp1.c = (float)cd;
    sp1.partial = (SRec *)workspace;
    sp1.early = (flags & MARS_LOGITS_READY) ? 1 : 0;
    const unsigned grid = (unsigned)(R * sp.S);
    // 4 vectors per batch in two register buffers, 4 blocks per SM (64 registers): measured
    // best for both dtypes; 5 or 6 blocks per SM spill the second buffer and run at half speed,
    // and 2 vectors per batch at 5 to 8 blocks per SM lose 10 to 50 %.
    {
        const bool overlap = hook(kHookNoOverlap) == 0;
        const cudaError_t le = (dt == MARS_BF16)
            ? launch_pdl(overlap, stoch_stream_kernel<MARS_BF16, 4, 4>, dim3(grid), dim3(kThreads), 0, st, sp1)
            : launch_pdl(overlap, stoch_stream_kernel<MARS_FP32, 4, 4>, dim3(grid), dim3(kThreads), 0, st, sp1);
        if (le != cudaSuccess) { (void)cudaGetLastError(); return MARS_ERR_CUDA; }
    }

    StochTailParams tp;
    tp.logits = logits; tp.ld = ld; tp.V = V; tp.N = N; tp.S = sp.S; tp.c = (float)cd; tp.theta = theta;
    tp.flags = flags; tp.chain = chain; tp.Dcap = Dcap; tp.partial = sp1.partial;
    tp.tok = tok; tp.parent = parent; tp.uniform = uniform;
    tp.qx = sd ? sd->qx : nullptr; tp.qlogits = sd ? sd->qlogits : nullptr; tp.ldq = sd ? sd->ldq : 0;
    tp.cq = (float)cqd;
    tp.accept_len = accept_len; tp.out_tokens = out_tokens; tp.path_nodes = path_nodes;
    tp.out_len = out_len; tp.seq_status = seq_status; tp.node_prob = node_prob; tp.node_how = node_how;
    const size_t smem = stoch_tail_smem_bytes(N);
    // The largest cluster (8, 4, 2 blocks per sequence) that still fits the GPU in one wave (two
    // blocks of 512 threads per SM; one for sampled chains, whose draw holds two rows in registers) and leaves each block a share of the row that fits its tile
    // table; rows too long for the table of a single block take the table-free search (G = 1).
    const int kv = dt == MARS_BF16 ? 8 : 4;
    const long long ntiles = ((long long)V + 32 * kv - 1) / (32 * kv);
    int G = 1;
    for (int g = kTailCluster; g > 1; g >>= 1)
        if ((long long)B * g <= (sd ? 1 : 2) * 148 && (ntiles + g - 1) / g <= kMaxTilesPerBlock) { G = g; break; }
    if (const int g = hook(kHookStochTailCluster)) {         // test hook: 1, 2, 4 or 8
        if ((g == 1 || g == 2 || g == 4 || g == 8) && (g == 1 || (ntiles + g - 1) / g <= kMaxTilesPerBlock)) G = g;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((long long)B * G));
    cfg.blockDim = dim3(kTailThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)G;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t err;
    if (sd)
        err = (dt == MARS_BF16) ? cudaLaunchKernelEx(&cfg, stoch_tail_kernel<MARS_BF16, 1>, tp)
                                : cudaLaunchKernelEx(&cfg, stoch_tail_kernel<MARS_FP32, 1>, tp);
    else
        err = (dt == MARS_BF16) ? cudaLaunchKernelEx(&cfg, stoch_tail_kernel<MARS_BF16, 0>, tp)
                                : cudaLaunchKernelEx(&cfg, stoch_tail_kernel<MARS_FP32, 0>, tp);
    if (err != cudaSuccess) { cudaGetLastError(); return MARS_ERR_CUDA; }
    return MARS_OK;
}

}  // namespace mars

extern "C" {

size_t mars_stochastic_workspace_bytes(int B, int N, int V, mars_dtype_t dt)
{
    if (!mars::stoch_sizes_supported(B, N, V, (int)dt)) return 0;
    const long long R = (long long)B * N;
    return mars::stoch_ws_bytes(R, mars::choose_split(R, V, (int)dt).S);
}

mars_status_t mars_verify_tree_stochastic(const void *logits, int64_t ld, mars_dtype_t dt, const int32_t *tok,
                                          const int32_t *parent, const float *uniform, int B, int N, int V,
                                          float theta, float temperature, uint32_t flags,
                                          int32_t *accept_len, int32_t *out_tokens, int32_t *path_nodes,
                                          int32_t *out_len, int Dcap, int32_t *seq_status, float *node_prob,
                                          uint8_t *node_how, void *workspace, size_t workspace_bytes,
                                          void *cuda_stream)
{
    return mars::run_stochastic(logits, ld, dt, tok, parent, uniform, nullptr, 0, B, N, V, theta, temperature, flags,
                                accept_len, out_tokens, path_nodes, out_len, Dcap, seq_status, node_prob,
                                node_how, workspace, workspace_bytes, cuda_stream);
}

mars_status_t mars_verify_chain_stochastic(const void *logits, int64_t ld, mars_dtype_t dt, const int32_t *draft,
                                           const float *uniform, int B, int K, int V, float theta,
                                           float temperature, uint32_t flags, int32_t *accept_len,
                                           int32_t *out_tokens, int32_t *out_len, int32_t *seq_status,
                                           float *node_prob, uint8_t *node_how, void *workspace,
                                           size_t workspace_bytes, void *cuda_stream)
{
    if (flags & MARS_SHARED_PARENT) return MARS_ERR_INVALID_ARG;
    return mars::run_stochastic(logits, ld, dt, draft, nullptr, uniform, nullptr, 1, B, K, V, theta, temperature,
                                flags, accept_len, out_tokens, nullptr, out_len, K - 1, seq_status, node_prob,
                                node_how, workspace, workspace_bytes, cuda_stream);
}

mars_status_t mars_verify_chain_sampled(const void *logits, int64_t ld, mars_dtype_t dt, const void *draft_logits,
                                        int64_t ld_draft, const int32_t *draft, const float *draft_prob,
                                        const float *uniform, int B, int K, int V, float theta, float temperature,
                                        float draft_temperature, uint32_t flags, int32_t *accept_len,
                                        int32_t *out_tokens, int32_t *out_len, int32_t *seq_status,
                                        float *node_prob, uint8_t *node_how, void *workspace,
                                        size_t workspace_bytes, void *cuda_stream)
{
    if (flags & MARS_SHARED_PARENT) return MARS_ERR_INVALID_ARG;
    mars::SampledDrafts sd;
    sd.qlogits = draft_logits; sd.ldq = ld_draft; sd.qx = draft_prob; sd.draft_temperature = draft_temperature;
    return mars::run_stochastic(logits, ld, dt, draft, nullptr, uniform, &sd, 1, B, K, V, theta, temperature, flags,
                                accept_len, out_tokens, nullptr, out_len, K - 1, seq_status, node_prob, node_how,
                                workspace, workspace_bytes, cuda_stream);
}

// ---- vocabulary-sharded stochastic verification ----------------------------------------------

mars_status_t mars_stochastic_shard_records(const void *logits_local, int64_t ld, mars_dtype_t dt,
                                            const int32_t *tok, const int32_t *parent, int B, int N,
                                            int V_local, int32_t id_offset, float temperature, uint32_t flags,
                                            void *records, float *node_logit, void *workspace,
                                            size_t workspace_bytes, void *cuda_stream)
{
    using namespace mars;
    if (B < 1 || N < 1 || V_local < 2 || !logits_local || !tok || !parent || !records || !node_logit)
        return MARS_ERR_INVALID_ARG;
    if (ld < V_local || id_offset < 0 || ((uintptr_t)records & 15)) return MARS_ERR_INVALID_ARG;
    if (!(temperature > 0.0f) || !(temperature < INFINITY)) return MARS_ERR_INVALID_ARG;
    if (flags & ~(MARS_SHARED_PARENT | MARS_LOGITS_READY)) return MARS_ERR_UNSUPPORTED;
    if (!stoch_sizes_supported(B, N, V_local, (int)dt)) return MARS_ERR_UNSUPPORTED;
    if ((uintptr_t)logits_local % (dt == MARS_BF16 ? 2 : 4)) return MARS_ERR_INVALID_ARG;
    const double cd = 1.4426950408889634074 / (double)temperature;
    if (!(cd < 3.0e38)) return MARS_ERR_INVALID_ARG;
    const long long R = (long long)B * N;
    const Split sp = choose_split(R, V_local, (int)dt);
    if (R * sp.S > 0x7fffffffll) return MARS_ERR_UNSUPPORTED;
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < stoch_ws_bytes(R, sp.S)) return MARS_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    StreamParams sp1;
    sp1.logits = logits_local; sp1.ld = ld; sp1.V = V_local; sp1.S = sp.S; sp1.L = sp.L; sp1.c = (float)cd;
    sp1.partial = (SRec *)workspace;
    sp1.early = (flags & MARS_LOGITS_READY) ? 1 : 0;
    const unsigned grid = (unsigned)(R * sp.S);
    {
        const bool overlap = hook(kHookNoOverlap) == 0;
        const cudaError_t le = (dt == MARS_BF16)
            ? launch_pdl(overlap, stoch_stream_kernel<MARS_BF16, 4, 4>, dim3(grid), dim3(kThreads), 0, st, sp1)
            : launch_pdl(overlap, stoch_stream_kernel<MARS_FP32, 4, 4>, dim3(grid), dim3(kThreads), 0, st, sp1);
        if (le != cudaSuccess) { (void)cudaGetLastError(); return MARS_ERR_CUDA; }
    }
    ShardRecordsParams rp;
    rp.logits = logits_local; rp.ld = ld; rp.V = V_local; rp.N = N; rp.S = sp.S; rp.id_offset = id_offset; rp.R = R;
    rp.flags = flags; rp.partial = sp1.partial; rp.tok = tok; rp.parent = parent;
    rp.records = (SRec *)records; rp.node_logit = node_logit;
    const unsigned g2 = (unsigned)((R + 255) / 256);
    if (dt == MARS_BF16) stoch_shard_records_kernel<MARS_BF16><<<g2, 256, 0, st>>>(rp);
    else stoch_shard_records_kernel<MARS_FP32><<<g2, 256, 0, st>>>(rp);
    return cudaGetLastError() == cudaSuccess ? MARS_OK : MARS_ERR_CUDA;
}

mars_status_t mars_stochastic_shard_verify(const void *logits_local, int64_t ld, mars_dtype_t dt,
                                           const void *records_all, const float *node_logit_all, int shards,
                                           int my_shard, const int32_t *tok, const int32_t *parent,
                                           const float *uniform, int B, int N, int V_local, int32_t id_offset,
                                           float theta, float temperature, uint32_t flags, int32_t *accept_len,
                                           int32_t *out_tokens, int32_t *path_nodes, int32_t *out_len, int Dcap,
                                           int32_t *seq_status, float *node_prob, uint8_t *node_how,
                                           int32_t *token_part, void *cuda_stream)
{
    using namespace mars;
    if (B < 1 || N < 1 || V_local < 2 || !logits_local || !records_all || !node_logit_all || !tok || !parent ||
        !uniform || !accept_len || !out_tokens || !out_len || !token_part)
        return MARS_ERR_INVALID_ARG;
    if (shards < 1 || shards > 254 || my_shard < 0 || my_shard >= shards || ld < V_local || Dcap < 0 || id_offset < 0 ||
        theta != theta || ((uintptr_t)records_all & 15))
        return MARS_ERR_INVALID_ARG;
    if (!(temperature > 0.0f) || !(temperature < INFINITY)) return MARS_ERR_INVALID_ARG;
    if (flags & ~(MARS_SIGN_LITERAL | MARS_SHARED_PARENT | MARS_RULE_MARGIN | MARS_RULE_PROB_RATIO | MARS_STOCH_PLAIN |
                  MARS_STOCH_RELAX_ONLY))
        return MARS_ERR_UNSUPPORTED;
    if ((flags & MARS_RULE_MARGIN) && (flags & MARS_RULE_PROB_RATIO)) return MARS_ERR_INVALID_ARG;
    if ((flags & MARS_STOCH_PLAIN) && (flags & MARS_STOCH_RELAX_ONLY)) return MARS_ERR_INVALID_ARG;
    rule_threshold(&theta, &flags);
    if (!stoch_sizes_supported(B, N, V_local, (int)dt)) return MARS_ERR_UNSUPPORTED;
    if ((uintptr_t)logits_local % (dt == MARS_BF16 ? 2 : 4)) return MARS_ERR_INVALID_ARG;
    const double cd = 1.4426950408889634074 / (double)temperature;
    if (!(cd < 3.0e38)) return MARS_ERR_INVALID_ARG;
    StochTailParams tp = {};
    tp.logits = logits_local; tp.ld = ld; tp.V = V_local; tp.N = N; tp.S = shards; tp.c = (float)cd; tp.theta = theta;
    tp.flags = flags; tp.chain = 0; tp.Dcap = Dcap; tp.partial = nullptr;
    tp.tok = tok; tp.parent = parent; tp.uniform = uniform;
    tp.records_all = (const SRec *)records_all; tp.node_logit_all = node_logit_all;
    tp.shards = shards; tp.my_shard = my_shard; tp.id_offset = id_offset; tp.token_part = token_part;
    tp.accept_len = accept_len; tp.out_tokens = out_tokens; tp.path_nodes = path_nodes;
    tp.out_len = out_len; tp.seq_status = seq_status; tp.node_prob = node_prob; tp.node_how = node_how;
    const int kv = dt == MARS_BF16 ? 8 : 4;
    const long long ntiles = ((long long)V_local + 32 * kv - 1) / (32 * kv);
    int G = 1;
    for (int g = kTailCluster; g > 1; g >>= 1)
        if ((long long)B * g <= 2 * 148 && (ntiles + g - 1) / g <= kMaxTilesPerBlock) { G = g; break; }
    if (const int g = hook(kHookStochTailCluster)) {         // test hook: 1, 2, 4 or 8
        if ((g == 1 || g == 2 || g == 4 || g == 8) && (g == 1 || (ntiles + g - 1) / g <= kMaxTilesPerBlock)) G = g;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((long long)B * G));
    cfg.blockDim = dim3(kTailThreads);
    cfg.dynamicSmemBytes = stoch_tail_smem_bytes(N);
    cfg.stream = (cudaStream_t)cuda_stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)G;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t err = (dt == MARS_BF16) ? cudaLaunchKernelEx(&cfg, stoch_tail_kernel<MARS_BF16, 2>, tp)
                                              : cudaLaunchKernelEx(&cfg, stoch_tail_kernel<MARS_FP32, 2>, tp);
    if (err != cudaSuccess) { cudaGetLastError(); return MARS_ERR_CUDA; }
    return MARS_OK;
}

mars_status_t mars_stochastic_shard_finish(const int32_t *token_all, int shards, int B, int Dcap,
                                           const int32_t *accept_len, int32_t *out_tokens, int32_t *seq_status,
                                           void *cuda_stream)
{
    if (!token_all || !accept_len || !out_tokens || shards < 1 || B < 1 || Dcap < 0) return MARS_ERR_INVALID_ARG;
    mars::stoch_shard_finish_kernel<<<(unsigned)((B + 255) / 256), 256, 0, (cudaStream_t)cuda_stream>>>(
        token_all, shards, B, Dcap + 1, accept_len, out_tokens, seq_status);
    return cudaGetLastError() == cudaSuccess ? MARS_OK : MARS_ERR_CUDA;
}


}  // extern "C"
