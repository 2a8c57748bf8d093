// Streaming top-2 building blocks shared by the row-scanning kernels of libmars: launch
// constants, the block-wide runner-up bound, the exact per-thread insert, the filtered batch
// step and the batch load, plus the host-side choice of how many slices a row is split into.
#pragma once

#include <cstdlib>

#include "mars_common.cuh"
#include "mars_hooks.cuh"
#include "mars_stream.cuh"

namespace mars {

constexpr int kThreads = 256;  // threads per block
constexpr int kU = 8;          // 16-byte vectors per thread per batch (128 B in flight each)
// Large bf16 batches run a second instantiation with 4 vectors per batch and 8 resident blocks
// per SM (32 registers): the same bytes in flight from twice the threads measured 1-1.5 %
// faster there, and slower for fp32 and for batches of a few hundred rows.
constexpr int kUDense = 4;
constexpr int kDenseMinRows = 148 * 16;
constexpr int kTargetBlocks = 148 * 4;      // resident blocks of this kernel on a B200
constexpr int kMinSliceBytes = kThreads * kU * 12;   // a slice is at least three quarters of a batch (24 KB):
                                                     // one round of loads per block measured best for a handful of rows

// ---- order-preserving float <-> uint encoding for the shared bound ----------------------
__device__ __forceinline__ unsigned enc(float x)
{
    unsigned b = __float_as_uint(x + 0.0f);
    return b ^ ((unsigned)((int)b >> 31) | 0x80000000u);
}
__device__ __forceinline__ float dec(unsigned e)
{
    return __uint_as_float(e ^ ((e & 0x80000000u) ? 0x80000000u : 0xffffffffu));
}

// Insert one element's value into the block-wide multiset top-2 {T1 >= T2}.  Every element
// is published at most once, so T2 never exceeds the slice's true runner-up value.
__device__ __forceinline__ void publish(unsigned *sT, float x)
{
    unsigned e = enc(x);
    if (e > *(volatile unsigned *)&sT[1]) {
        unsigned old = atomicMax(&sT[0], e);
        unsigned y = min(old, e);
        if (y > *(volatile unsigned *)&sT[1]) atomicMax(&sT[1], y);
    }
}

// Exact insert of one element into the thread's top-2.  Valid because a thread sees its
// elements in increasing token id: equality never displaces.
template <bool PUBLISH>
__device__ __forceinline__ void insert(Rec &s, float x, int idx, unsigned *sT)
{
    if (x > s.z2) {
        if (x > s.z1) { s.z2 = s.z1; s.id2 = s.id1; s.z1 = x; s.id1 = idx; }
        else { s.z2 = x; s.id2 = idx; }
        if (PUBLISH) publish(sT, x);
    }
}

template <int DT, int U, bool PUBLISH>
__device__ __forceinline__ void process_batch(const uint4 (&v)[U], const typename Elem<DT>::packed_t (&q)[U],
                                              float bm, float T2, int idx0, Rec &s, unsigned *sT)
{
    typedef Elem<DT> E;
    if (bm > s.z2 && bm >= T2) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            float qf = E::to_float(q[u]);
            if (qf > s.z2 && qf >= T2) {
                int base = idx0 + u * kThreads * E::kVec;
#pragma unroll
                for (int k = 0; k < E::kVec; ++k) insert<PUBLISH>(s, E::elem(v[u], k), base + k, sT);
            }
        }
    }
}

template <int DT, int U, bool GUARD>
__device__ __forceinline__ float load_batch(const uint4 *vbase, int v0, int nvec, uint4 (&v)[U],
                                            typename Elem<DT>::packed_t (&q)[U])
{
    typedef Elem<DT> E;
    static_assert(U >= 4 && (U & (U - 1)) == 0, "U must be a power of two >= 4");
#pragma unroll
    for (int u = 0; u < U; ++u) {
        int vi = v0 + u * kThreads;
        if (!GUARD || vi < nvec) v[u] = ld_stream(vbase + vi);
        else v[u] = E::neg_inf();
    }
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

// ---- host: slices per row ----------------------------------------------------------------

struct Split { int S; int L; };

inline Split choose_split(long long R, int V, int dt)
{
    const int es = dt == MARS_BF16 ? 2 : 4;
    long long S = 1;
    const int force = hook(kHookForceSplit);         // test hook: force slices per row
    int min_elems = kMinSliceBytes / es;
    if (force >= 1) { S = force; min_elems = 64; }
    else if (R < kTargetBlocks) S = kTargetBlocks / R;   // never more blocks than fit at once
    long long smax = V / min_elems;
    if (smax < 1) smax = 1;
    if (S > smax) S = smax;
    long long L = (V + S - 1) / S;
    L = (L + 15) / 16 * 16;
    Split sp;
    sp.L = (int)L;
    sp.S = (int)((V + L - 1) / L);
    return sp;
}

}  // namespace mars
