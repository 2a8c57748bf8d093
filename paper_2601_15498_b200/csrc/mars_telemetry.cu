// libmars: histograms of the per-row top-2 statistics that the paper plots for its target
// models -- the top-1 logit, the logit ratio z2/z1 and the probability ratio p2/p1 (Fig. 1,
// Fig. 3) -- computed from the [rows, 2] top-2 values that the verification calls can emit.
//
// Every bin decision is a short fixed sequence of IEEE fp32 operations, so the counts are
// reproducible bit for bit: the probability-ratio bins are decided in the logit-difference
// domain against edges -ln(k/n) that the host evaluates once in double.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "mars.h"

namespace mars {

constexpr int kMaxBins = 256;

struct HistParams {
    const float *val;   // [R, 2]
    long long R;
    float lo, hi, inv_w;
    int nbins;
    unsigned *hist;      // [3, nbins]
    unsigned *outliers;  // [3]
    float edge[kMaxBins];   // edge[k] = (float)(-ln(k / nbins)), k = 1 .. nbins-1
};

__global__ void __launch_bounds__(256) histogram_kernel(const HistParams p)
{
    __shared__ unsigned s_hist[3 * kMaxBins];
    __shared__ unsigned s_out[3];
    for (int i = threadIdx.x; i < 3 * p.nbins; i += blockDim.x) s_hist[i] = 0;
    if (threadIdx.x < 3) s_out[threadIdx.x] = 0;
    __syncthreads();
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x; r < p.R; r += stride) {
        const float2 z = reinterpret_cast<const float2 *>(p.val)[r];
        const float z1 = z.x, z2 = z.y;
        // top-1 logit
        if (z1 >= p.lo && z1 < p.hi) {
            int b = (int)floorf(__fmul_rn(__fsub_rn(z1, p.lo), p.inv_w));
            b = min(max(b, 0), p.nbins - 1);
            atomicAdd(&s_hist[b], 1u);
        } else {
            atomicAdd(&s_out[0], 1u);
        }
        // logit ratio, defined for a positive top-1 logit (Sec. 3.3)
        const float ratio = __fdiv_rn(z2, z1);
        if (z1 > 0.0f && ratio >= 0.0f && ratio <= 1.0f) {
            int b = min((int)floorf(__fmul_rn(ratio, (float)p.nbins)), p.nbins - 1);
            atomicAdd(&s_hist[p.nbins + b], 1u);
        } else {
            atomicAdd(&s_out[1], 1u);
        }
        // probability ratio p2/p1 = exp(-(z1 - z2)): bin k holds k/n <= p2/p1 < (k+1)/n
        const float delta = __fsub_rn(z1, z2);
        if (delta >= 0.0f) {
            int b = 0;
            for (int k = 1; k < p.nbins; ++k) b += (delta <= p.edge[k]) ? 1 : 0;
            atomicAdd(&s_hist[2 * p.nbins + b], 1u);
        } else {
            atomicAdd(&s_out[2], 1u);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 3 * p.nbins; i += blockDim.x)
        if (s_hist[i]) atomicAdd(&p.hist[i], s_hist[i]);
    if (threadIdx.x < 3 && s_out[threadIdx.x]) atomicAdd(&p.outliers[threadIdx.x], s_out[threadIdx.x]);
}

}  // namespace mars

extern "C" mars_status_t mars_top2_histograms(const float *top2_val, int64_t rows, float z1_lo, float z1_hi,
                                              int nbins, uint32_t *hist, uint32_t *outliers, void *cuda_stream)
{
    using namespace mars;
    if (!hist || !outliers || rows < 0) return MARS_ERR_INVALID_ARG;
    if (rows > 0 && (!top2_val || ((uintptr_t)top2_val & 7))) return MARS_ERR_INVALID_ARG;
    if (!(z1_hi > z1_lo) || nbins < 1) return MARS_ERR_INVALID_ARG;
    if (nbins > kMaxBins) return MARS_ERR_UNSUPPORTED;
    HistParams p;
    p.val = top2_val; p.R = rows; p.lo = z1_lo; p.hi = z1_hi; p.nbins = nbins;
    p.inv_w = (float)nbins / (z1_hi - z1_lo);
    p.hist = hist; p.outliers = outliers;
    p.edge[0] = INFINITY;
    for (int k = 1; k < kMaxBins; ++k) p.edge[k] = k < nbins ? (float)(-log((double)k / (double)nbins)) : 0.0f;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(hist, 0, sizeof(uint32_t) * 3 * (size_t)nbins, st) != cudaSuccess) return MARS_ERR_CUDA;
    if (cudaMemsetAsync(outliers, 0, sizeof(uint32_t) * 3, st) != cudaSuccess) return MARS_ERR_CUDA;
    if (rows == 0) return MARS_OK;
    long long blocks = (rows + 255) / 256;
    if (blocks > 148 * 8) blocks = 148 * 8;
    histogram_kernel<<<(unsigned)blocks, 256, 0, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? MARS_OK : MARS_ERR_CUDA;
}
