// Effective-sample-size floor on the calibration weights: mean-normalise the raw sensitivities of every
// (layer, head, component) row, measure their squared coefficient of variation, and shrink them toward uniform
// just enough that the Kish effective sample size stays at or above min(n, 2 p).  HBM-bound: the row is read
// three times (mean, spread, output) and written once; sums are fp64 in a fixed order.
#include "cb_internal.cuh"

namespace cb {

static constexpr int ESS_THREADS = 512;

// Block-wide sum with a fixed association order (independent of timing); every thread gets the result.
__device__ __forceinline__ double ess_block_sum(double v, double *scratch /* [ESS_THREADS / 32] */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        int lo = __double2loint(v), hi = __double2hiint(v);
        lo = __shfl_xor_sync(0xffffffffu, lo, o);
        hi = __shfl_xor_sync(0xffffffffu, hi, o);
        v += __hiloint2double(hi, lo);
    }
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    double s = 0.0;
#pragma unroll
    for (int w = 0; w < ESS_THREADS / 32; ++w) s += scratch[w];
    return s;
}

__global__ void __launch_bounds__(ESS_THREADS) k_ess_weights(const float *__restrict__ r_raw, long long n, long long r_stride,
                                                            long long p_width, float *__restrict__ w, long long w_stride,
                                                            float *__restrict__ alpha_out)
{
    __shared__ double scratch[ESS_THREADS / 32];
    const float *r = r_raw + (long long)blockIdx.x * r_stride;
    float *wo = w + (long long)blockIdx.x * w_stride;
    double s = 0.0;
    for (long long i = threadIdx.x; i < n; i += ESS_THREADS) s += (double)r[i];
    const double mean = ess_block_sum(s, scratch) / (double)n;
    if (!(mean > 0.0)) {                                   // no sensitivity at all: uniform weights
        for (long long i = threadIdx.x; i < n; i += ESS_THREADS) wo[i] = 1.f;
        if (threadIdx.x == 0 && alpha_out) alpha_out[blockIdx.x] = 1.f;
        return;
    }
    const double inv = 1.0 / mean;
    double q = 0.0;
    for (long long i = threadIdx.x; i < n; i += ESS_THREADS) {
        const double d = (double)r[i] * inv - 1.0;
        q += d * d;
    }
    const double cv2 = ess_block_sum(q, scratch) / (double)n;
    const double tau = (double)((n < 2 * p_width) ? n : 2 * p_width);
    double alpha = 1.0;
    if (cv2 > 0.0) {
        const double a = sqrt(((double)n / tau - 1.0) / cv2);
        alpha = a < 1.0 ? a : 1.0;
    }
    for (long long i = threadIdx.x; i < n; i += ESS_THREADS) wo[i] = (float)(1.0 + alpha * ((double)r[i] * inv - 1.0));
    if (threadIdx.x == 0 && alpha_out) alpha_out[blockIdx.x] = (float)alpha;
}

cudaError_t launch_ess(const float *r_raw, int n_rows, long long n, long long r_stride, long long p_width, float *w,
                       long long w_stride, float *alpha_out, cudaStream_t st)
{
    k_ess_weights<<<n_rows, ESS_THREADS, 0, st>>>(r_raw, n, r_stride, p_width, w, w_stride, alpha_out);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

}  // namespace cb

extern "C" cb_status cb_ess_weights(const float *r_raw, int32_t n_rows, int64_t n_tokens, int64_t r_row_stride,
                                    int64_t p_width, float *w, int64_t w_row_stride, float *alpha_out, void *stream)
{
    if (!r_raw || !w || n_rows < 0 || n_tokens <= 0 || p_width <= 0) return CB_ERR_INVALID_ARG;
    if (r_row_stride < n_tokens || w_row_stride < n_tokens) return CB_ERR_INVALID_ARG;
    if (n_rows == 0) return CB_OK;
    if (const cudaError_t ce = cb::launch_ess(r_raw, n_rows, n_tokens, r_row_stride, p_width, w, w_row_stride, alpha_out,
                       static_cast<cudaStream_t>(stream)); ce != cudaSuccess) return cb::cuda_failed(ce);
    return CB_OK;
}
