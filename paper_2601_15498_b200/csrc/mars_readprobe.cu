// libmars: a read-only streaming probe.  It reads a buffer once with the same 16-byte streaming
// loads and the same launch shape as the verification kernel (256 threads, 8 vectors in flight
// per thread, 4 blocks per SM, one contiguous chunk per block) and keeps only a running maximum,
// so its rate is the ceiling that a kernel which must read every logit can reach on this GPU.
// The benchmark reports it next to the copy bandwidth that serves as the roofline's denominator.
#include "mars_stream.cuh"

#include "mars.h"

namespace mars {

__global__ void __launch_bounds__(256, 4) read_probe_kernel(const uint4 *buf, long long nvec, long long chunk,
                                                            unsigned *out)
{
    const long long lo = (long long)blockIdx.x * chunk;
    const long long hi = lo + chunk < nvec ? lo + chunk : nvec;
    uint32_t m = 0;
    for (long long v0 = lo + threadIdx.x; v0 < hi; v0 += 256 * 8) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = (v0 + u * 256 < hi) ? ld_stream(buf + v0 + u * 256) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int u = 0; u < 8; ++u) m = max(m, max(max(v[u].x, v[u].y), max(v[u].z, v[u].w)));
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, s));
    if ((threadIdx.x & 31) == 0) atomicMax(out, m);
}

}  // namespace mars

extern "C" mars_status_t mars_selftest_stream_read(const void *buffer, size_t bytes, size_t chunk_bytes,
                                                   uint32_t *out_max, void *cuda_stream)
{
    if (!buffer || !out_max || bytes < 16 || chunk_bytes < 16 || ((uintptr_t)buffer & 15)) return MARS_ERR_INVALID_ARG;
    const long long nvec = (long long)(bytes / 16), chunk = (long long)(chunk_bytes / 16);
    const long long blocks = (nvec + chunk - 1) / chunk;
    if (blocks > 0x7fffffffll) return MARS_ERR_UNSUPPORTED;
    mars::read_probe_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)cuda_stream>>>(
        (const uint4 *)buffer, nvec, chunk, out_max);
    return cudaGetLastError() == cudaSuccess ? MARS_OK : MARS_ERR_CUDA;
}
