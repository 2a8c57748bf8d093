// Streaming pieces shared by the row-scanning kernels of libmars: the 16-byte streaming load,
// the packed bf16 maximum, and per-dtype helpers to reduce a 16-byte vector to its maximum and
// to pull single elements out of it.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "mars.h"

namespace mars {

__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 v;
    asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
        : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
        : "l"(p));
    return v;
}

__device__ __forceinline__ uint32_t bmax2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));  // NaN operand -> the other one
    return d;
}

// Programmatic dependent launch (back-to-back calls on one stream).  A kernel that is launched
// with programmatic stream serialisation may begin while its predecessor still runs, provided
// the predecessor lets it: pdl_launch_dependents() does that, and is a no-op otherwise.  Such a
// kernel must call pdl_wait() before its first access to anything the predecessor may produce or
// still use; it returns once the predecessor has completed and its writes are visible.  The
// streaming kernels wait first thing, unless the caller vouched (MARS_LOGITS_READY) that the
// logits do not come from the predecessor: then only workspaces and outputs are at stake, and the
// wait moves behind the streaming loop.  Without the launch attribute, or without a predecessor
// that triggers early, both calls do nothing.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Launch with programmatic stream serialisation allowed (see above); `allow` = false gives the
// plain stream order (a measurement aid: the cost of a call without any overlap).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(bool allow, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                              cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = allow ? 1 : 0;
    cfg.attrs = at; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

template <int DT> struct Elem;

template <> struct Elem<MARS_BF16> {
    static constexpr int kBytes = 2;
    static constexpr int kVec = 8;
    typedef uint32_t packed_t;  // two bf16 lanes
    static __device__ __forceinline__ uint4 neg_inf() { return make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u); }
    static __device__ __forceinline__ packed_t vred(const uint4 &v) { return bmax2(bmax2(v.x, v.y), bmax2(v.z, v.w)); }
    static __device__ __forceinline__ packed_t pmax(packed_t a, packed_t b) { return bmax2(a, b); }
    static __device__ __forceinline__ float to_float(packed_t m)
    {
        return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xffff0000u));
    }
    static __device__ __forceinline__ float elem(const uint4 &v, int k)
    {
        uint32_t w = (k >> 1) == 0 ? v.x : (k >> 1) == 1 ? v.y : (k >> 1) == 2 ? v.z : v.w;
        return (k & 1) ? __uint_as_float(w & 0xffff0000u) : __uint_as_float(w << 16);
    }
    static __device__ __forceinline__ float scalar(const void *row, int j)
    {
        return __uint_as_float((uint32_t)((const unsigned short *)row)[j] << 16);
    }
};

template <> struct Elem<MARS_FP32> {
    static constexpr int kBytes = 4;
    static constexpr int kVec = 4;
    typedef float packed_t;
    static __device__ __forceinline__ uint4 neg_inf() { return make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u); }
    static __device__ __forceinline__ packed_t vred(const uint4 &v)
    {
        return fmaxf(fmaxf(__uint_as_float(v.x), __uint_as_float(v.y)),
                     fmaxf(__uint_as_float(v.z), __uint_as_float(v.w)));
    }
    static __device__ __forceinline__ packed_t pmax(packed_t a, packed_t b) { return fmaxf(a, b); }
    static __device__ __forceinline__ float to_float(packed_t m) { return m; }
    static __device__ __forceinline__ float elem(const uint4 &v, int k)
    {
        return __uint_as_float(k == 0 ? v.x : k == 1 ? v.y : k == 2 ? v.z : v.w);
    }
    static __device__ __forceinline__ float scalar(const void *row, int j) { return ((const float *)row)[j]; }
};

}  // namespace mars
