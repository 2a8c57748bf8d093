// Shared device-side pieces of libmars: the 16-byte top-2 record, its merge operator
// under the row's total order, and the per-sequence verification tail (margin test,
// node match, accepted-subtree propagation, longest accepted path, emit).
#pragma once

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

namespace mars {

constexpr int kNoId = 0x7fffffff;  // "no element yet": loses against every real element

// Top-2 of a set of elements: (z1,id1) best, (z2,id2) second best.  Elements equal to
// -inf (and NaN, which counts as -inf) are never stored; rows with fewer than two
// stored elements are completed by finish_record().
struct __align__(16) Rec {
    float z1;
    int id1;
    float z2;
    int id2;
};

__device__ __forceinline__ Rec empty_rec()
{
    Rec r;
    r.z1 = -INFINITY; r.id1 = kNoId; r.z2 = -INFINITY; r.id2 = kNoId;
    return r;
}

// Total order of Sec. 3.3 (z(1) >= z(2)) completed with "lower token id first".
__device__ __forceinline__ bool beats(float ax, int ai, float bx, int bi)
{
    return ax > bx || (ax == bx && ai < bi);
}

// Merge is associative and commutative under the total order, so any reduction tree
// (lanes, warps, slices, vocabulary shards) gives the same record.
__device__ __forceinline__ Rec merge(const Rec &a, const Rec &b)
{
    Rec o;
    if (beats(b.z1, b.id1, a.z1, a.id1)) {
        o.z1 = b.z1; o.id1 = b.id1;
        if (beats(a.z1, a.id1, b.z2, b.id2)) { o.z2 = a.z1; o.id2 = a.id1; }
        else { o.z2 = b.z2; o.id2 = b.id2; }
    } else {
        o.z1 = a.z1; o.id1 = a.id1;
        if (beats(b.z1, b.id1, a.z2, a.id2)) { o.z2 = b.z1; o.id2 = b.id1; }
        else { o.z2 = a.z2; o.id2 = a.id2; }
    }
    return o;
}

__device__ __forceinline__ Rec shfl_xor_rec(const Rec &r, int mask)
{
    Rec o;
    o.z1 = __shfl_xor_sync(0xffffffffu, r.z1, mask);
    o.id1 = __shfl_xor_sync(0xffffffffu, r.id1, mask);
    o.z2 = __shfl_xor_sync(0xffffffffu, r.z2, mask);
    o.id2 = __shfl_xor_sync(0xffffffffu, r.id2, mask);
    return o;
}

// A finished row record: rows with fewer than two elements above -inf take the lowest
// unused token ids with value -inf (every -inf / NaN element ties, lowest id first);
// -0 is reported as +0.
__device__ __forceinline__ Rec finish_record(Rec r)
{
    if (r.id1 == kNoId) { r.id1 = 0; r.z1 = -INFINITY; r.id2 = 1; r.z2 = -INFINITY; }
    else if (r.id2 == kNoId) { r.id2 = (r.id1 == 0) ? 1 : 0; r.z2 = -INFINITY; }
    r.z1 += 0.0f;
    r.z2 += 0.0f;
    return r;
}

// Adaptive-relaxation bit of one row.  Default: sign guard, then r = z2/z1 > theta with one
// IEEE round-to-nearest division (Eq. 4; strict comparison as in Sec. 3.4 / Algorithm 1).
// With flag bit 3 (fixed-margin variant) the test is Delta = z1 - z2 < theta instead, one fp32
// subtraction (Delta as defined with Eq. 5); the probability-ratio variant is mapped onto it
// on the host, see rule_threshold().
__device__ __forceinline__ bool relax_bit(float z1, float z2, float theta, uint32_t flags)
{
    if (flags & 8u) return __fsub_rn(z1, z2) < theta;
    bool guard = (flags & 1u) ? true : (z1 > 0.0f);
    return guard && (__fdiv_rn(z2, z1) > theta);
}

// Host: p2/p1 = exp(z2 - z1) > theta  <=>  z1 - z2 < -ln(theta)  (Sec. 3.3: the probability
// ratio is the exponentiated logit difference).  Rewrites the probability-ratio variant
// (flag bit 4) as a fixed margin c = -ln(theta), computed in double and rounded once;
// theta <= 0 accepts every runner-up (c = +inf).
inline void rule_threshold(float *theta, uint32_t *flags)
{
    if (*flags & 16u) {
        const double t = (double)*theta;
        *theta = t > 0.0 ? (float)(-log(t)) : INFINITY;
        *flags = (*flags & ~16u) | 8u;
    }
}

struct TailArgs {
    const int32_t *tok;     // tree: [B,N]; chain: draft [B,N-1]
    const int32_t *parent;  // tree: [B,N] or [N]; chain: unused
    int32_t *accept_len;
    int32_t *out_tokens;    // [B, Dcap+1]
    int32_t *path_nodes;    // [B, Dcap+1] or null
    int32_t *out_len;
    int32_t *seq_status;    // or null
    float *dbg_val;         // [R,2] or null
    int32_t *dbg_id;        // [R,2] or null
    uint8_t *dbg_flags;     // [B,N] or null
    int N;
    int Dcap;
    float theta;
    uint32_t flags;         // bit0 sign literal, bit1 shared parent
    int chain;              // 1: implicit parent[i] = i-1, tok[i] = draft[i-1]
};

// Shared-memory footprint of the tail for N nodes.
__host__ __device__ inline size_t tail_smem_bytes(int N)
{
    return (size_t)N * (4 * sizeof(int32_t) + 2) + 16;
}

// Verification tail for sequence b, run by ALL threads of one thread block.
//   load_rec(i) returns the finished record of row (b, i); called once per node.
// smem must provide tail_smem_bytes(N) bytes, 4-byte aligned.
template <class LoadRec>
__device__ void verify_tail(const TailArgs &t, int b, unsigned char *smem, LoadRec load_rec)
{
    const int N = t.N;
    const int tid = threadIdx.x, nthr = blockDim.x;
    int32_t *s_id1 = reinterpret_cast<int32_t *>(smem);
    int32_t *s_id2 = s_id1 + N;
    int32_t *s_par = s_id2 + N;
    int32_t *s_tok = s_par + N;
    unsigned char *s_relax = reinterpret_cast<unsigned char *>(s_tok + N);
    unsigned char *s_flag = s_relax + N;

    const int32_t *par_g = t.chain ? nullptr
                                   : ((t.flags & 2u) ? t.parent : t.parent + (size_t)b * N);
    int bad = 0;
    for (int i = tid; i < N; i += nthr) {
        Rec r = load_rec(i);
        s_id1[i] = r.id1;
        s_id2[i] = r.id2;
        s_relax[i] = relax_bit(r.z1, r.z2, t.theta, t.flags) ? 1 : 0;
        size_t row = (size_t)b * N + i;
        if (t.dbg_val) { t.dbg_val[2 * row] = r.z1; t.dbg_val[2 * row + 1] = r.z2; }
        if (t.dbg_id) { t.dbg_id[2 * row] = r.id1; t.dbg_id[2 * row + 1] = r.id2; }
        int p, tk;
        if (t.chain) {
            p = i - 1;
            tk = i > 0 ? t.tok[(size_t)b * (N - 1) + (i - 1)] : -1;
        } else {
            p = par_g[i];
            tk = t.tok[(size_t)b * N + i];
            if (i == 0 ? (p != -1) : (p >= i || p < -1)) bad = 1;
        }
        s_par[i] = p;
        s_tok[i] = tk;
    }
    bad = __syncthreads_or(bad);

    // three-way rule per node against the parent's row (Sec. 3.4)
    for (int i = tid; i < N; i += nthr) {
        int how = 0;
        int p = s_par[i], tk = s_tok[i];
        if (!bad && i > 0 && p >= 0 && tk >= 0) {
            if (tk == s_id1[p]) how = 1;
            else if (tk == s_id2[p] && s_relax[p]) how = 2;
        }
        s_flag[i] = (unsigned char)how;
    }
    __syncthreads();
    if (tid >= 32) return;

    // ---- one warp: accepted-subtree propagation and the deepest accepted node ----
    const int lane = tid;
    int best = 0, a = 0;
    int status = bad ? 1 : 0;
    if (!bad) {
        if (N <= 64) {
            // Nodes `lane` and `lane+32`.  Jacobi rounds over a 64-bit accepted mask: a node
            // turns accepted in the round equal to its depth, so the first fresh bit of
            // the last productive round is the deepest accepted node of lowest index.
            int p0 = lane < N ? s_par[lane] : -1, p1 = lane + 32 < N ? s_par[lane + 32] : -1;
            bool h0 = lane < N && s_flag[lane] != 0, h1 = lane + 32 < N && s_flag[lane + 32] != 0;
            unsigned long long acc = 1ull;
            for (int round = 1; round < N; ++round) {
                bool a0 = h0 && p0 >= 0 && ((acc >> (p0 & 63)) & 1ull);
                bool a1 = h1 && p1 >= 0 && ((acc >> (p1 & 63)) & 1ull);
                unsigned long long nacc = acc | (unsigned long long)__ballot_sync(0xffffffffu, a0) |
                                          ((unsigned long long)__ballot_sync(0xffffffffu, a1) << 32);
                unsigned long long fresh = nacc & ~acc;
                if (fresh == 0ull) break;
                best = __ffsll((long long)fresh) - 1;
                a = round;
                acc = nacc;
            }
            if (lane < N && ((acc >> lane) & 1ull)) s_flag[lane] |= 4;
            if (lane + 32 < N && ((acc >> (lane + 32)) & 1ull)) s_flag[lane + 32] |= 4;
        } else {
            // Larger trees: one pass in node order (parent[i] < i) by one lane.  Depths go
            // where the runner-up ids were; those are dead once the match flags exist.
            if (lane == 0) {
                int32_t *s_depth = s_id2;
                s_depth[0] = 0;
                s_flag[0] |= 4;
                for (int i = 1; i < N; ++i) {
                    int p = s_par[i];
                    int d = p >= 0 ? s_depth[p] + 1 : 0;
                    s_depth[i] = d;
                    bool ok = p >= 0 && (s_flag[p] & 4) && (s_flag[i] & 3);
                    if (ok) {
                        s_flag[i] |= 4;
                        if (d > a) { a = d; best = i; }
                    }
                }
            }
            best = __shfl_sync(0xffffffffu, best, 0);
            a = __shfl_sync(0xffffffffu, a, 0);
        }
        if (a > t.Dcap) status = 2;
    }
    __syncwarp();

    const int W = t.Dcap + 1;
    int32_t *o_tok = t.out_tokens + (size_t)b * W;
    int32_t *o_path = t.path_nodes ? t.path_nodes + (size_t)b * W : nullptr;
    for (int k = lane; k < W; k += 32) {
        o_tok[k] = -1;
        if (o_path) o_path[k] = -1;
    }
    __syncwarp();
    if (status != 0) {
        a = 0;
        best = 0;
        for (int i = lane; i < N; i += 32) s_flag[i] = (i == 0) ? 4 : 0;
        __syncwarp();
    }
    if (lane == 0) {
        int n = best;
        for (int d = a; d >= 0; --d) {
            if (d > 0) o_tok[d - 1] = s_tok[n];
            if (o_path) o_path[d] = n;
            s_flag[n] |= 8;
            n = s_par[n];
        }
        o_tok[a] = s_id1[best];  // correction token, or the bonus token at a leaf
        t.accept_len[b] = a;
        t.out_len[b] = a + 1;
        if (t.seq_status) t.seq_status[b] = status;
    }
    __syncwarp();
    if (t.dbg_flags)
        for (int i = lane; i < N; i += 32) t.dbg_flags[(size_t)b * N + i] = s_flag[i];
}

}  // namespace mars
