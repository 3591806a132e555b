// Two-pass centred construction (Section 3.4): the pieces that the one-pass path does not have.
//
//   k_means            first pass: per map, sum w x, sum w y, sum w (and sum w y^2, which the layer selector needs)
//                      over a chunk, added to fp64 partial sums.
//                      Pure streaming (every source/target element and weight is read once per map that uses it),
//                      bound by HBM; the reduction order is fixed: a thread sums its rows in token order, the row
//                      groups of a block are combined in index order, the block adds to its own (split, map) entry.
//   k_means_rope_keys  the same for key maps whose rows are first turned back by the rotary angles of their positions.
//   k_means_finalize   sums the splits in index order (fp64) and divides by s_w.
//   k_reduce_centered  second-pass reduction: the accumulate kernel multiplies the ROUNDED centred operand
//                      a_t = bf16(w_t (x_t - mu_x)) with the uncentred [x_t | y_t]; with r = sum_t a_t (kept in the
//                      slot's s_x entries) the centred statistics are exactly
//                          A = sum_t a_t (x_t - mu_x)^T = D_xx - r mu_x^T,   B = D_xy - r mu_y^T.
#include "cb_internal.cuh"
#include "cb_rope.cuh"
#include "cb_math.cuh"

namespace cb {

template <int D>
__global__ void __launch_bounds__(256) k_means(const MeansArgs a, const int map_base)
{
    constexpr int CC = D / 8;            // 16-byte chunks per head row
    constexpr int RG = 256 / CC;         // row groups of the block
    constexpr int UN = 4;                // rows in flight per thread
    __shared__ float red[RG][3 * D + 1];
    const int n_maps = 2 * a.Lt * a.Ht;
    const int m = map_base + blockIdx.x, split = blockIdx.y;
    const int comp = m / (a.Lt * a.Ht), l = (m / a.Ht) % a.Lt, h = m % a.Ht;
    const int t0 = (int)(((long long)a.n_tokens * split) / gridDim.y);
    const int t1 = (int)(((long long)a.n_tokens * (split + 1)) / gridDim.y);
    const int cc = threadIdx.x % CC, rg = threadIdx.x / CC;
    const __nv_bfloat16 *xs = (comp ? a.src.v : a.src.k) + (long long)a.src_layer[l] * a.src.sl + (long long)a.src_head[h] * a.src.sh + cc * 8;
    const __nv_bfloat16 *ys = (comp ? a.tgt.v : a.tgt.k) + (long long)l * a.tgt.sl + (long long)h * a.tgt.sh + cc * 8;
    const float *ws = (comp ? a.w_v : a.w_k) + (long long)l * a.w_sl + (long long)h * a.w_sh;

    float sx[8], sy[8], sq[8], sw = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) sx[e] = sy[e] = sq[e] = 0.f;
    for (int r0 = t0 + rg; r0 < t1; r0 += UN * RG) {
        uint4 xv[UN], yv[UN];
        float wt[UN];
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const int r = r0 + u * RG;
            const bool in = r < t1;
            const int rr = in ? r : t0;
            xv[u] = __ldg(reinterpret_cast<const uint4 *>(xs + (long long)rr * a.src.st));
            yv[u] = __ldg(reinterpret_cast<const uint4 *>(ys + (long long)rr * a.tgt.st));
            wt[u] = in ? __ldg(ws + rr) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const unsigned xu[4] = {xv[u].x, xv[u].y, xv[u].z, xv[u].w};
            const unsigned yu[4] = {yv[u].x, yv[u].y, yv[u].z, yv[u].w};
            float fx[8], fy[8];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                fx[2 * e] = __uint_as_float(xu[e] << 16); fx[2 * e + 1] = __uint_as_float(xu[e] & 0xffff0000u);
                fy[2 * e] = __uint_as_float(yu[e] << 16); fy[2 * e + 1] = __uint_as_float(yu[e] & 0xffff0000u);
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                sx[e] = fmaf(wt[u], fx[e], sx[e]);
                const float wy = wt[u] * fy[e];
                sy[e] += wy;
                sq[e] = fmaf(wy, fy[e], sq[e]);
            }
            sw += wt[u];
        }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) { red[rg][cc * 8 + e] = sx[e]; red[rg][D + cc * 8 + e] = sy[e]; red[rg][2 * D + 1 + cc * 8 + e] = sq[e]; }
    if (cc == 0) red[rg][2 * D] = sw;
    __syncthreads();
    double *dst = a.msum + ((size_t)split * n_maps + m) * means_stride(D);
    for (int v = threadIdx.x; v < 3 * D + 1; v += 256) {
        double sum = 0.0;
#pragma unroll 4
        for (int g = 0; g < RG; ++g) sum += (double)red[g][v];
        dst[v] += sum;
    }
}

__device__ __forceinline__ void bf16x8_to_f32(const uint4 v, float (&f)[8])
{
    const unsigned u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) { f[2 * e] = __uint_as_float(u[e] << 16); f[2 * e + 1] = __uint_as_float(u[e] & 0xffff0000u); }
}

// Key maps with the rotary embedding removed (Section 3.1): the sums are those of the de-rotated rows, turned back in
// fp32 (nothing is rounded before it is summed).  Channel i pairs with i + D/2, so a thread takes chunk j of the lower
// half AND chunk j + CC/2 of the upper half of its rows: the eight angles are evaluated once for the sixteen channels
// they turn.  The two threads that share a chunk pair take alternate rows; their sums are added (lane exchange) before
// the block's row groups are combined as in k_means.
template <int D>
__global__ void __launch_bounds__(256, 2) k_means_rope_keys(const MeansArgs a, const RopeDev rope)
{
    constexpr int CC = D / 8, HC = CC / 2;
    constexpr int RG = 256 / CC;         // row groups of the block; each covers two rows per step
    constexpr int UN = 2;                // rows in flight per thread
    __shared__ float red[RG][3 * D + 1];
    const int n_maps = 2 * a.Lt * a.Ht;
    const int m = blockIdx.x, split = blockIdx.y;            // key maps are maps 0 .. Lt * Ht - 1
    const int l = m / a.Ht, h = m % a.Ht;
    const int t0 = (int)(((long long)a.n_tokens * split) / gridDim.y);
    const int t1 = (int)(((long long)a.n_tokens * (split + 1)) / gridDim.y);
    const int cc = threadIdx.x % CC, rg = threadIdx.x / CC, j = cc % HC, odd = cc / HC;
    const __nv_bfloat16 *xs = a.src.k + (long long)a.src_layer[l] * a.src.sl + (long long)a.src_head[h] * a.src.sh + j * 8;
    const __nv_bfloat16 *ys = a.tgt.k + (long long)l * a.tgt.sl + (long long)h * a.tgt.sh + j * 8;
    const float *ws = a.w_k + (long long)l * a.w_sl + (long long)h * a.w_sh;
    uint32_t fs[8], ft[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) { fs[e] = rope.f_src[j * 8 + e]; ft[e] = rope.f_tgt[j * 8 + e]; }

    float sxl[8], sxu[8], syl[8], syu[8], sql[8], squ[8], sw = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) sxl[e] = sxu[e] = syl[e] = syu[e] = sql[e] = squ[e] = 0.f;
    // the trip count is the same for every thread of the block
    for (int rb = t0; rb < t1; rb += UN * 2 * RG) {
        uint4 xl[UN], xu[UN], yl[UN], yu[UN];
        float wt[UN];
        int pv[UN];
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const int r = rb + 2 * rg + odd + u * 2 * RG;
            const bool in = r < t1;
            const int rr = in ? r : t0;
            xl[u] = __ldg(reinterpret_cast<const uint4 *>(xs + (long long)rr * a.src.st));
            xu[u] = __ldg(reinterpret_cast<const uint4 *>(xs + (long long)rr * a.src.st + D / 2));
            yl[u] = __ldg(reinterpret_cast<const uint4 *>(ys + (long long)rr * a.tgt.st));
            yu[u] = __ldg(reinterpret_cast<const uint4 *>(ys + (long long)rr * a.tgt.st + D / 2));
            wt[u] = in ? __ldg(ws + rr) : 0.f;
            pv[u] = __ldg(rope.pos + rr);
        }
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            float a0[8], a1[8], b0[8], b1[8];
            bf16x8_to_f32(xl[u], a0); bf16x8_to_f32(xu[u], a1);
            bf16x8_to_f32(yl[u], b0); bf16x8_to_f32(yu[u], b1);
            const float w = wt[u];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                // x~_i = x_i c + x_{i+D/2} s;  x~_{i+D/2} = x_{i+D/2} c - x_i s
                float c, s, ct, st;
                rope_cs_poly(fs[e], pv[u], c, s);
                if (rope.same) { ct = c; st = s; } else rope_cs_poly(ft[e], pv[u], ct, st);
                const float x0 = fmaf(a0[e], c, a1[e] * s), x1 = fmaf(a1[e], c, -a0[e] * s);
                const float y0 = fmaf(b0[e], ct, b1[e] * st), y1 = fmaf(b1[e], ct, -b0[e] * st);
                sxl[e] = fmaf(w, x0, sxl[e]); sxu[e] = fmaf(w, x1, sxu[e]);
                const float wy0 = w * y0, wy1 = w * y1;
                syl[e] += wy0; syu[e] += wy1;
                sql[e] = fmaf(wy0, y0, sql[e]); squ[e] = fmaf(wy1, y1, squ[e]);
            }
            sw += w;
        }
    }
    // even rows + odd rows of the row group (the sum of two floats does not depend on which lane forms it)
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        sxl[e] += __shfl_xor_sync(0xffffffffu, sxl[e], HC); sxu[e] += __shfl_xor_sync(0xffffffffu, sxu[e], HC);
        syl[e] += __shfl_xor_sync(0xffffffffu, syl[e], HC); syu[e] += __shfl_xor_sync(0xffffffffu, syu[e], HC);
        sql[e] += __shfl_xor_sync(0xffffffffu, sql[e], HC); squ[e] += __shfl_xor_sync(0xffffffffu, squ[e], HC);
    }
    sw += __shfl_xor_sync(0xffffffffu, sw, HC);
    const int c0 = odd ? D / 2 + j * 8 : j * 8;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        red[rg][c0 + e] = odd ? sxu[e] : sxl[e];
        red[rg][D + c0 + e] = odd ? syu[e] : syl[e];
        red[rg][2 * D + 1 + c0 + e] = odd ? squ[e] : sql[e];
    }
    if (cc == 0) red[rg][2 * D] = sw;
    __syncthreads();
    double *dst = a.msum + ((size_t)split * n_maps + m) * means_stride(D);
    for (int v = threadIdx.x; v < 3 * D + 1; v += 256) {
        double sum = 0.0;
#pragma unroll 4
        for (int g = 0; g < RG; ++g) sum += (double)red[g][v];
        dst[v] += sum;
    }
}

cudaError_t launch_means(const MeansArgs &a, int d, cudaStream_t st)
{
    const int half = a.Lt * a.Ht;
    if (a.rope_pos) {
        // key maps through the de-rotating kernel, value maps through the plain one
        RopeDev rope = RopeDev{};
        rope.pos = a.rope_pos;
        rope_frequencies(a.rope_base_src, d, rope.f_src);
        rope_frequencies(a.rope_base_tgt, d, rope.f_tgt);
        rope.same = (a.rope_base_src == a.rope_base_tgt) ? 1 : 0;
        dim3 grid(half, MEANS_SPLITS);
        if (d == 128) { k_means_rope_keys<128><<<grid, 256, 0, st>>>(a, rope); k_means<128><<<grid, 256, 0, st>>>(a, half); }
        else { k_means_rope_keys<64><<<grid, 256, 0, st>>>(a, rope); k_means<64><<<grid, 256, 0, st>>>(a, half); }
        cudaError_t e = cudaGetLastError();
        if (e == cudaSuccess) { count_launch(); count_launch(); }
        return e;
    }
    dim3 grid(2 * half, MEANS_SPLITS);
    if (d == 128) k_means<128><<<grid, 256, 0, st>>>(a, 0);
    else k_means<64><<<grid, 256, 0, st>>>(a, 0);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

// mu [n_maps][2d + 1]: mu_x, mu_y, s_w.  A map without weight gets zero means.
__global__ void k_means_finalize(const double *__restrict__ msum, int n_maps, int d, float *__restrict__ mu)
{
    const int m = blockIdx.x, ms = means_stride(d);
    double sw = 0.0;
    for (int s = 0; s < MEANS_SPLITS; ++s) sw += msum[((size_t)s * n_maps + m) * ms + 2 * d];
    for (int v = threadIdx.x; v < 2 * d + 1; v += blockDim.x) {
        double sum = 0.0;
        for (int s = 0; s < MEANS_SPLITS; ++s) sum += msum[((size_t)s * n_maps + m) * ms + v];
        mu[(size_t)m * (2 * d + 1) + v] = (v == 2 * d) ? (float)sw : (sw > 0.0 ? (float)(sum / sw) : 0.f);
    }
}

// syy [n_maps][d] = sum over the calibration rows of w y^2 per target channel (splits summed in index order)
__global__ void k_means_energy(const double *__restrict__ msum, int n_maps, int d, float *__restrict__ syy)
{
    const int m = blockIdx.x, ms = means_stride(d);
    for (int c = threadIdx.x; c < d; c += blockDim.x) {
        double sum = 0.0;
        for (int s = 0; s < MEANS_SPLITS; ++s) sum += msum[((size_t)s * n_maps + m) * ms + 2 * d + 1 + c];
        syy[(size_t)m * d + c] = (float)sum;
    }
}

cudaError_t launch_means_energy(const double *msum, int n_maps, int d, float *syy, cudaStream_t st)
{
    k_means_energy<<<n_maps, 128, 0, st>>>(msum, n_maps, d, syy);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

cudaError_t launch_means_finalize(const double *msum, int n_maps, int d, float *mu, cudaStream_t st)
{
    k_means_finalize<<<n_maps, 288, 0, st>>>(msum, n_maps, d, mu);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

// Same split summation as the one-pass reduction, then the rank-one corrections and the symmetrisation of A.
template <int d>
__global__ void __launch_bounds__(1024) k_reduce_centered(const float *__restrict__ slots, int n_splits, int n_maps,
                                                         const float *__restrict__ mu, float *__restrict__ A,
                                                         float *__restrict__ B, int k_operands_centred)
{
    extern __shared__ __align__(16) float rs[];       // [d][2d + 1] sums of D, then [2d + 4] sums of r, -, s_w; then mu_x, mu_y
    const int m = blockIdx.x, n2 = 2 * d, pitch = 2 * d + 1;
    const int sf = slot_floats(d);
    const float *base = slots + (size_t)m * sf;
    const size_t sstride = (size_t)n_maps * sf;
    float *mus = rs + (size_t)d * pitch + 2 * d + 4;
    // key maps accumulated with the rotary boundary have both operands centred already: nothing to correct
    const bool no_corr = k_operands_centred && m < n_maps / 2;
    for (int v = threadIdx.x; v < 2 * d; v += blockDim.x) mus[v] = no_corr ? 0.f : mu[(size_t)m * (2 * d + 1) + v];
    for (int e4 = threadIdx.x; e4 < sf / 4; e4 += blockDim.x) {
        double v[4] = {0.0, 0.0, 0.0, 0.0};
        for (int s = 0; s < n_splits; ++s) {
            const float4 f = *reinterpret_cast<const float4 *>(base + s * sstride + 4 * e4);
            v[0] += (double)f.x; v[1] += (double)f.y; v[2] += (double)f.z; v[3] += (double)f.w;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int e = 4 * e4 + q;
            if (e < d * n2) rs[(e / n2) * pitch + (e % n2)] = (float)v[q];
            else rs[d * pitch + (e - d * n2)] = (float)v[q];
        }
    }
    __syncthreads();
    const float *r = rs + d * pitch;                                // sum of the rounded centred operand, per channel
    float *Am = A + (size_t)m * d * d;
    float *Bm = B + (size_t)m * d * d;
    for (int e = threadIdx.x; e < d * d; e += blockDim.x) {
        const int i = e / d, j = e % d;
        const double aij = (double)rs[i * pitch + j] - (double)r[i] * (double)mus[j];
        const double aji = (double)rs[j * pitch + i] - (double)r[j] * (double)mus[i];
        Am[e] = (float)(0.5 * (aij + aji));                          // a + b == b + a: exactly symmetric
        Bm[e] = (float)((double)rs[i * pitch + d + j] - (double)r[i] * (double)mus[d + j]);
    }
}

cudaError_t launch_reduce_centered(const float *slots, int n_splits, int n_maps, int d, const float *mu, float *A, float *B,
                                   int k_operands_centred, cudaStream_t st)
{
    const size_t smem = sizeof(float) * ((size_t)d * (2 * d + 1) + 2 * d + 4 + 2 * d);
    static bool attr[MAX_DEVICES] = {};
    static bool attr64[MAX_DEVICES] = {};
    if (d == 128) {
        cudaError_t e = opt_in_smem(k_reduce_centered<128>, (size_t)(140 * 1024), attr);
        if (e != cudaSuccess) return e;
        k_reduce_centered<128><<<n_maps, 1024, smem, st>>>(slots, n_splits, n_maps, mu, A, B, k_operands_centred);
    } else {
        cudaError_t e = opt_in_smem(k_reduce_centered<64>, (size_t)(140 * 1024), attr64);
        if (e != cudaSuccess) return e;
        k_reduce_centered<64><<<n_maps, 1024, smem, st>>>(slots, n_splits, n_maps, mu, A, B, k_operands_centred);
    }
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

}  // namespace cb
