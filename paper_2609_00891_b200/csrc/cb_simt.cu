// CUDA-core kernels: fp32 statistics accumulation and affine apply (selected with CB_FLAG_SIMT, and used for
// bring-up of the tensor-core kernels), the deterministic split reduction, and the batched fp64 ridge solve.
#include "cb_internal.cuh"

namespace cb {

__device__ __forceinline__ float bf16_bits_to_f32(unsigned short b) { return __uint_as_float(((unsigned)b) << 16); }

__device__ __forceinline__ void unpack8(const uint4 &v, float *f)
{
    const unsigned u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(u[i] << 16);
        f[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
    }
}

// ======================================================================================================
// Statistics, CUDA cores.  Grid (n_maps, n_splits), 256 threads.  Each block owns slot (split, map).
// Tokens are staged 2048/D at a time in shared memory as fp32: xw = w*x  [TT][D], xy = [x | y]  [TT][2D].
// Thread (ty, tx) of a 16x16 layout accumulates rows ty*RI..+RI and columns q*64 + tx*4 + e of D = xw^T xy.
// ======================================================================================================
template <int D>
__global__ void __launch_bounds__(256) k_accum_simt(const AccumArgs a)
{
    constexpr int TT = 2048 / D;   // keeps the staging buffers under 48 KB of static shared memory
    constexpr int RI = D / 16;
    constexpr int Q = D / 32;  // column groups of 64
    __shared__ __align__(16) float xw[TT][D];
    __shared__ __align__(16) float xy[TT][2 * D];
    __shared__ float ws[TT];

    const int m = blockIdx.x, split = blockIdx.y;
    const int n_maps = 2 * a.Lt * a.Ht;
    const int comp = m / (a.Lt * a.Ht), l = (m / a.Ht) % a.Lt, h = m % a.Ht;
    const int j = a.src_layer[l], g = a.src_head[h];
    const __nv_bfloat16 *X = (comp ? a.src.v : a.src.k) + (long long)j * a.src.sl + (long long)g * a.src.sh;
    const __nv_bfloat16 *Y = (comp ? a.tgt.v : a.tgt.k) + (long long)l * a.tgt.sl + (long long)h * a.tgt.sh;
    const float *w = (comp ? a.w_v : a.w_k) + (long long)l * a.w_sl + (long long)h * a.w_sh;

    const int n_tiles = (a.n_tokens + TT - 1) / TT;
    const int tile0 = (int)(((long long)n_tiles * split) / a.n_splits);
    const int tile1 = (int)(((long long)n_tiles * (split + 1)) / a.n_splits);
    if (tile0 >= tile1) return;

    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    float acc[RI][Q * 4];
#pragma unroll
    for (int r = 0; r < RI; ++r)
#pragma unroll
        for (int c = 0; c < Q * 4; ++c) acc[r][c] = 0.f;
    float bias = 0.f, sw = 0.f;   // tid < D: s_x[tid]; D <= tid < 2D: s_y[tid - D]

    for (int tile = tile0; tile < tile1; ++tile) {
        const int t0 = tile * TT;
        if (tid < TT) ws[tid] = (t0 + tid < a.n_tokens) ? w[t0 + tid] : 0.f;
        __syncthreads();
        // stage: TT*D/8 16-byte pieces per array
        for (int c = tid; c < TT * D / 8; c += 256) {
            const int t = c / (D / 8), c8 = (c % (D / 8)) * 8;
            float fx[8], fy[8];
            if (t0 + t < a.n_tokens) {
                unpack8(*reinterpret_cast<const uint4 *>(X + (long long)(t0 + t) * a.src.st + c8), fx);
                unpack8(*reinterpret_cast<const uint4 *>(Y + (long long)(t0 + t) * a.tgt.st + c8), fy);
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) fx[e] = fy[e] = 0.f;
            }
            const float wt = ws[t];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                xw[t][c8 + e] = wt * fx[e];
                xy[t][c8 + e] = fx[e];
                xy[t][D + c8 + e] = fy[e];
            }
        }
        __syncthreads();
#pragma unroll 4
        for (int t = 0; t < TT; ++t) {
            float av[RI];
#pragma unroll
            for (int r = 0; r < RI; ++r) av[r] = xw[t][ty * RI + r];
#pragma unroll
            for (int q = 0; q < Q; ++q) {
                const float4 b = *reinterpret_cast<const float4 *>(&xy[t][q * 64 + tx * 4]);
#pragma unroll
                for (int r = 0; r < RI; ++r) {
                    acc[r][q * 4 + 0] = fmaf(av[r], b.x, acc[r][q * 4 + 0]);
                    acc[r][q * 4 + 1] = fmaf(av[r], b.y, acc[r][q * 4 + 1]);
                    acc[r][q * 4 + 2] = fmaf(av[r], b.z, acc[r][q * 4 + 2]);
                    acc[r][q * 4 + 3] = fmaf(av[r], b.w, acc[r][q * 4 + 3]);
                }
            }
            if (tid < D) bias += xw[t][tid];
            else if (tid < 2 * D) bias = fmaf(ws[t], xy[t][tid], bias);   // xy[t][D + (tid - D)]
            if (tid == 0) sw += ws[t];
        }
        __syncthreads();
    }

    float *slot = a.slots + ((size_t)split * n_maps + m) * slot_floats(D);
#pragma unroll
    for (int r = 0; r < RI; ++r)
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            float4 *ptr = reinterpret_cast<float4 *>(slot + (size_t)(ty * RI + r) * 2 * D + q * 64 + tx * 4);
            float4 v = *ptr;
            v.x += acc[r][q * 4 + 0];
            v.y += acc[r][q * 4 + 1];
            v.z += acc[r][q * 4 + 2];
            v.w += acc[r][q * 4 + 3];
            *ptr = v;
        }
    if (tid < 2 * D) slot[slot_sx(D) + tid] += bias;   // s_x then s_y are adjacent
    if (tid == 0) slot[slot_sw(D)] += sw;
}

cudaError_t launch_accum_simt(const AccumArgs &a, int d, cudaStream_t st)
{
    dim3 grid(2 * a.Lt * a.Ht, a.n_splits);
    if (d == 128) k_accum_simt<128><<<grid, 256, 0, st>>>(a);
    else k_accum_simt<64><<<grid, 256, 0, st>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

// ======================================================================================================
// Deterministic reduction of the splits: fixed index order, fp64 sums, symmetrised G.
// Grid n_maps, 1024 threads.  The splits are summed with coalesced reads into a shared-memory image of D
// (fp32, padded rows); G and C are then written from that image, the transpose needed for the
// symmetrisation being a shared-memory access.
// ======================================================================================================
// The head width is a template parameter: every index of the two output loops is a division by d, 2 d or d + 1, and
// with run-time divisors those divisions were most of the kernel's instructions.
template <int d>
__global__ void __launch_bounds__(1024) k_reduce(const float *__restrict__ slots, int n_splits, int n_maps,
                                                float *__restrict__ G, float *__restrict__ C)
{
    extern __shared__ __align__(16) float rs[];       // [d][2d + 1] sums of D, then [2d + 1] sums of s_x, s_y, s_w
    constexpr int p = d + 1, n2 = 2 * d, pitch = 2 * d + 1;
    const int m = blockIdx.x;
    constexpr int sf = slot_floats(d);
    const float *base = slots + (size_t)m * sf;
    const size_t sstride = (size_t)n_maps * sf;
    // sum the splits four floats at a time (slots are 16-byte aligned and sf is a multiple of 4); the slot's last
    // three floats are padding and land in unused tail entries
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
    const float *bs = rs + d * pitch;                               // s_x [d], s_y [d], s_w
    float *Gm = G + (size_t)m * p * p;
    float *Cm = C + (size_t)m * p * d;
    for (int e = threadIdx.x; e < p * p; e += blockDim.x) {
        const int i = e / p, j = e % p;
        float v;
        if (i < d && j < d) v = 0.5f * (rs[i * pitch + j] + rs[j * pitch + i]);     // a + b == b + a: exactly symmetric
        else if (i == d && j == d) v = bs[2 * d];
        else v = bs[(i == d) ? j : i];
        Gm[e] = v;
    }
    for (int e = threadIdx.x; e < p * d; e += blockDim.x) {
        const int i = e / d, j = e % d;
        Cm[e] = (i < d) ? rs[i * pitch + d + j] : bs[d + j];
    }
}

cudaError_t launch_reduce(const float *slots, int n_splits, int n_maps, int d, float *G, float *C, cudaStream_t st)
{
    const size_t smem = sizeof(float) * ((size_t)d * (2 * d + 1) + 2 * d + 4);
    static bool attr[MAX_DEVICES] = {};
    static bool attr64[MAX_DEVICES] = {};
    if (d == 128) {
        cudaError_t e = opt_in_smem(k_reduce<128>, (size_t)(140 * 1024), attr);
        if (e != cudaSuccess) return e;
        k_reduce<128><<<n_maps, 1024, smem, st>>>(slots, n_splits, n_maps, G, C);
    } else {
        cudaError_t e = opt_in_smem(k_reduce<64>, (size_t)(140 * 1024), attr64);
        if (e != cudaSuccess) return e;
        k_reduce<64><<<n_maps, 1024, smem, st>>>(slots, n_splits, n_maps, G, C);
    }
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

// ======================================================================================================
// Affine apply, CUDA cores.  Grid (n_maps, token splits), 256 threads; W (fp32) stays in shared memory while
// the block walks its token tiles of 32.
// ======================================================================================================
template <int D>
__global__ void __launch_bounds__(256) k_apply_simt(const ApplyArgs a)
{
    constexpr int TT = 32;
    extern __shared__ __align__(16) float smf[];
    float *W = smf;                   // [D+1][D]
    float *xs = smf + (D + 1) * D;    // [TT][D]
    const int m = blockIdx.x;
    const int comp = m / (a.Lt * a.Ht), l = (m / a.Ht) % a.Lt, h = m % a.Ht;
    const __nv_bfloat16 *X = (comp ? a.src.v : a.src.k) + (long long)a.src_layer[l] * a.src.sl + (long long)a.src_head[h] * a.src.sh;
    const float *Wm = a.Wb + (size_t)m * (D + 1) * D;
    const int tid = threadIdx.x;
    for (int e = tid; e < (D + 1) * D; e += 256) W[e] = Wm[e];

    const int n_tiles = (a.n_tokens + TT - 1) / TT;
    const int tile0 = (int)(((long long)n_tiles * blockIdx.y) / gridDim.y);
    const int tile1 = (int)(((long long)n_tiles * (blockIdx.y + 1)) / gridDim.y);
    constexpr int CG = D / 4;         // channel groups of 4
    constexpr int TG = 256 / CG;      // token groups
    constexpr int TPT = TT / TG;      // tokens per thread
    const int cg = tid % CG, tg = tid / CG;

    for (int tile = tile0; tile < tile1; ++tile) {
        const int t0 = tile * TT;
        __syncthreads();
        for (int c = tid; c < TT * D / 8; c += 256) {
            const int t = c / (D / 8), c8 = (c % (D / 8)) * 8;
            float fx[8];
            if (t0 + t < a.n_tokens) unpack8(*reinterpret_cast<const uint4 *>(X + (long long)(t0 + t) * a.src.st + c8), fx);
            else {
#pragma unroll
                for (int e = 0; e < 8; ++e) fx[e] = 0.f;
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) xs[t * D + c8 + e] = fx[e];
        }
        __syncthreads();
        float acc[TPT][4];
        const float4 bb = *reinterpret_cast<const float4 *>(&W[D * D + cg * 4]);
#pragma unroll
        for (int r = 0; r < TPT; ++r) { acc[r][0] = bb.x; acc[r][1] = bb.y; acc[r][2] = bb.z; acc[r][3] = bb.w; }
#pragma unroll 4
        for (int i = 0; i < D; ++i) {
            const float4 wv = *reinterpret_cast<const float4 *>(&W[i * D + cg * 4]);
#pragma unroll
            for (int r = 0; r < TPT; ++r) {
                const float x = xs[(tg * TPT + r) * D + i];
                acc[r][0] = fmaf(x, wv.x, acc[r][0]);
                acc[r][1] = fmaf(x, wv.y, acc[r][1]);
                acc[r][2] = fmaf(x, wv.z, acc[r][2]);
                acc[r][3] = fmaf(x, wv.w, acc[r][3]);
            }
        }
#pragma unroll
        for (int r = 0; r < TPT; ++r) {
            const int t = t0 + tg * TPT + r;
            if (t >= a.n_tokens) continue;
            const long long off = (long long)l * a.o_sl + (long long)t * a.o_st + (long long)h * a.o_sh + cg * 4;
            if (a.out_dtype == CB_DTYPE_F32) {
                float *o = reinterpret_cast<float *>(comp ? a.out_v : a.out_k) + off;
                *reinterpret_cast<float4 *>(o) = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
            } else {
                __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(comp ? a.out_v : a.out_k) + off;
                __nv_bfloat162 p0 = __floats2bfloat162_rn(acc[r][0], acc[r][1]);
                __nv_bfloat162 p1 = __floats2bfloat162_rn(acc[r][2], acc[r][3]);
                uint2 pk;
                pk.x = *reinterpret_cast<unsigned *>(&p0);
                pk.y = *reinterpret_cast<unsigned *>(&p1);
                *reinterpret_cast<uint2 *>(o) = pk;
            }
        }
    }
}

cudaError_t launch_apply_simt(const ApplyArgs &a, int d, cudaStream_t st)
{
    const int n_maps = 2 * a.Lt * a.Ht;
    const int n_tiles = (a.n_tokens + 31) / 32;
    int splits = (4 * 148 + n_maps - 1) / n_maps;
    if (splits > n_tiles) splits = n_tiles;
    if (splits < 1) splits = 1;
    const size_t smem = sizeof(float) * ((size_t)(d + 1) * d + 32 * d);
    cudaError_t e;
    if (d == 128) {
        e = cudaFuncSetAttribute(k_apply_simt<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k_apply_simt<128><<<dim3(n_maps, splits), 256, smem, st>>>(a);
    } else {
        e = cudaFuncSetAttribute(k_apply_simt<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k_apply_simt<64><<<dim3(n_maps, splits), 256, smem, st>>>(a);
    }
    e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

}  // namespace cb
