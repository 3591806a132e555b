// Layer selector (Section 3.1, first paragraph): held-in R^2 of single-source-layer probes from statistics that the
// path produces anyway.  For a probe with statistics G, C (bias-column form), fitted map Theta = [W; b] and the
// target's sum of squares:
//     B   = C[0:d] - s_x s_y^T / s_w                  (centred cross statistics)
//     SST = sum_c (sum w y_c^2 - s_y,c^2 / s_w)
//     R^2 = (tr(B^T W) + lambda_eff ||W||_F^2) / SST
// which equals 1 - SSE/SST for the ridge solution W = (A + lambda_eff I)^-1 B (A W = B - lambda_eff W turns the
// quadratic term of SSE into the two traces); lambda = 0 is the ordinary least-squares probe of the paper.
#include "cb_internal.cuh"

namespace cb {

__global__ void __launch_bounds__(256) k_probe_r2(const float *__restrict__ G, const float *__restrict__ C,
                                                  const float *__restrict__ Wb, const float *__restrict__ syy,
                                                  int d, double lambda, double inv_n, int raw_lambda, float *__restrict__ r2)
{
    __shared__ double part[2][8];
    const int m = blockIdx.x, p = d + 1, tid = threadIdx.x;
    const float *Gm = G + (size_t)m * p * p;
    const float *Cm = C + (size_t)m * p * d;
    const float *Wm = Wb + (size_t)m * p * d;
    const double s_w = (double)Gm[(size_t)d * p + d];
    const double lam = raw_lambda ? lambda : lambda * s_w * inv_n;
    const double inv_sw = s_w > 0.0 ? 1.0 / s_w : 0.0;
    double num = 0.0, sst = 0.0;
    for (int e = tid; e < d * d; e += 256) {
        const int i = e / d, j = e % d;
        const double b = (double)Cm[e] - (double)Gm[(size_t)d * p + i] * (double)Cm[(size_t)d * d + j] * inv_sw;
        const double w = (double)Wm[e];
        num += b * w + lam * w * w;
    }
    for (int c = tid; c < d; c += 256) {
        const double sy = (double)Cm[(size_t)d * d + c];
        sst += (double)syy[(size_t)m * d + c] - sy * sy * inv_sw;
    }
    // fixed-order block sum: lanes by shuffle, warps in index order
    for (int o = 16; o > 0; o >>= 1) {
        num += __shfl_down_sync(0xffffffffu, num, o);
        sst += __shfl_down_sync(0xffffffffu, sst, o);
    }
    if ((tid & 31) == 0) { part[0][tid >> 5] = num; part[1][tid >> 5] = sst; }
    __syncthreads();
    if (tid == 0) {
        double a = 0.0, b = 0.0;
        for (int w = 0; w < 8; ++w) { a += part[0][w]; b += part[1][w]; }
        r2[m] = b > 0.0 ? (float)(a / b) : 0.f;
    }
}

cudaError_t launch_probe_r2(const float *G, const float *C, const float *Wb, const float *syy, int n_maps, int d,
                            double lambda, double inv_n, int raw_lambda, float *r2, cudaStream_t st)
{
    k_probe_r2<<<n_maps, 256, 0, st>>>(G, C, Wb, syy, d, lambda, inv_n, raw_lambda, r2);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

struct ScoreArgs {
    int src_layer[128];
};

// scores[l][src_layer[l]] += mean over (component, head) of r2; one thread per target layer, fixed order
__global__ void k_probe_scores(const float *__restrict__ r2, int Lt, int Ht, ScoreArgs sa, int Ls, float *__restrict__ scores)
{
    const int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l >= Lt) return;
    double acc = 0.0;
    for (int comp = 0; comp < 2; ++comp)
        for (int h = 0; h < Ht; ++h) acc += (double)r2[((size_t)comp * Lt + l) * Ht + h];
    scores[(size_t)l * Ls + sa.src_layer[l]] += (float)(acc / (2.0 * Ht));
}

cudaError_t launch_probe_scores(const float *r2, int Lt, int Ht, const int *src_layer_host, int Ls, float *scores, cudaStream_t st)
{
    ScoreArgs sa;
    for (int l = 0; l < 128; ++l) sa.src_layer[l] = l < Lt ? src_layer_host[l] : 0;
    k_probe_scores<<<(Lt + 63) / 64, 64, 0, st>>>(r2, Lt, Ht, sa, Ls, scores);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

}  // namespace cb
