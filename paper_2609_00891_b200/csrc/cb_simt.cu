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
__global__ void __launch_bounds__(1024) k_reduce(const float *__restrict__ slots, int n_splits, int n_maps, int d,
                                                float *__restrict__ G, float *__restrict__ C)
{
    extern __shared__ __align__(16) float rs[];       // [d][2d + 1] sums of D, then [2d + 1] sums of s_x, s_y, s_w
    const int m = blockIdx.x, p = d + 1, n2 = 2 * d, pitch = 2 * d + 1;
    const int sf = slot_floats(d);
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
    {
        cudaError_t e = opt_in_smem(k_reduce, (size_t)(140 * 1024), attr);
        if (e != cudaSuccess) return e;
    }
    k_reduce<<<n_maps, 1024, smem, st>>>(slots, n_splits, n_maps, d, G, C);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

// ======================================================================================================
// Batched ridge solve, fp64, one block per (map, lambda).
//   A = G + lambda_eff * diag(1,..,1,0);  A = L L^T (packed lower triangle, rows padded to even length);
//   L Z = C, L^T Theta = Z.
// ======================================================================================================
struct SolveArgs {
    const float *G, *C;    // augmented: G [p][p], C [p][d];  centred: A [d][d], B [d][d]
    const float *mu;       // centred form only: [n_maps][2d + 1] = mu_x, mu_y, s_w; null for the augmented form
    float *Wb;
    int *info;
    int n_maps, d;
    double inv_n;
    unsigned flags;
    int n_lambda;
    float lambdas[16];
};

__host__ __device__ inline int tri_row_start(int i)
{
    // sum_{r<i} roundup2(r+1):  rows 0..i-1 have lengths 1..i, each padded to even
    const int h = i / 2;            // pairs (1,2),(3,4),.. padded to (2,2),(4,4),..
    return 2 * h * (h + 1) + ((i & 1) ? (i + 1) : 0);
}

// shuffle of a double between lane pairs
__device__ __forceinline__ double shfl_xor_f64(double v, int mask)
{
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_xor_sync(0xffffffffu, lo, mask);
    hi = __shfl_xor_sync(0xffffffffu, hi, mask);
    return __hiloint2double(hi, lo);
}

// Cholesky by block columns of 8 (left-looking): thread i owns row i of L; thread n + c owns right-hand-side column c,
// whose forward substitution obeys the same recurrence as a row of L below the diagonal block and rides along.  For
// a block column a thread pulls its 8 entries into registers, subtracts the contributions of all finished columns
// (its own row times the 8 rows of the diagonal block, read as broadcasts), the 8 diagonal-block rows publish theirs,
// one otherwise idle thread factors that 8 x 8 block in registers while the others already work on the next block
// column, and every thread solves its own row against the block.  Three block barriers per block column.
// The backward substitution gives every right-hand-side column to a pair of lanes that split the inner sums; eight
// rows are kept in registers at a time, so each loaded L entry feeds one FMA and each loaded Z entry feeds eight.
#ifdef CB_SOLVE_TIMING
__device__ long long g_solve_t[8];
extern "C" int cb_debug_solve_t(long long *h) { return (int)cudaMemcpyFromSymbol(h, g_solve_t, sizeof(g_solve_t)); }
#define ST(i) do { if (blockIdx.x == 0 && threadIdx.x == 0) g_solve_t[i] = clock64(); } while (0)
#else
#define ST(i) do {} while (0)
#endif
constexpr int SOLVE_THREADS = 320;     // 129 rows of L + 128 right-hand-side columns, and a warp for the thread that
constexpr int SOLVE_FACTOR_THREAD = 288;   // factors the diagonal blocks
#ifndef CB_SOLVE_AHEAD
#define CB_SOLVE_AHEAD 148
#endif
__global__ void __launch_bounds__(SOLVE_THREADS, 1) k_ridge_solve(const SolveArgs a)
{
    ST(0);
    extern __shared__ __align__(16) double sm[];
    constexpr int NB = 8;
    const int d = a.d, p = d + 1;
    const bool centred = a.mu != nullptr;
    const int n = centred ? d : p;                     // order of the system: the centred form has no bias row
    // blocks of one map's lambdas are neighbours in launch order: the second and third read G and C from L2
    const int m = blockIdx.x / a.n_lambda, li = blockIdx.x % a.n_lambda;
    double *Lp = sm;                                   // packed lower triangle, rows padded to even length
    double *Z = sm + tri_row_start(n);                 // [n][d]
    __shared__ double diag[NB][NB];
    __shared__ double rdiag[136];                      // reciprocals of the diagonal of L
    __shared__ int s_fail;
    const int tid = threadIdx.x;

    const float *Gm = a.G + (size_t)m * n * n;
    const float *Cm = a.C + (size_t)m * n * d;
    const double s_w = centred ? (double)a.mu[(size_t)m * (2 * d + 1) + 2 * d] : (double)Gm[(size_t)d * p + d];
    const double lam = (a.flags & CB_FLAG_RAW_LAMBDA) ? (double)a.lambdas[li] : (double)a.lambdas[li] * s_w * a.inv_n;
    if (tid == 0) s_fail = 0;
    {
        // The block that will follow this one on the SM is, to a good guess, gridDim-resident blocks further on (one
        // block per SM): ask L2 for its statistics now, so that its load phase does not wait for DRAM.
        const int nb = blockIdx.x + CB_SOLVE_AHEAD;
        if (nb < (int)gridDim.x && nb / a.n_lambda != m) {
            const int m2 = nb / a.n_lambda;
            const char *g2 = reinterpret_cast<const char *>(a.G + (size_t)m2 * n * n);
            const char *c2 = reinterpret_cast<const char *>(a.C + (size_t)m2 * n * d);
            for (int o = tid * 128; o < n * n * 4; o += blockDim.x * 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(g2 + o));
            for (int o = tid * 128; o < n * d * 4; o += blockDim.x * 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(c2 + o));
        }
    }
    {
        const int lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
        // one warp per row (coalesced, no divisions); the global loads of a row are issued together before any
        // shared-memory store so that they overlap
        constexpr int MAXV = 5;                            // ceil(129 / 32)
        // four rows in flight per warp (36 loads per lane): the phase is bound by load latency, L2 or DRAM
#pragma unroll 4
        for (int i = warp; i < n; i += nwarps) {
            const int rsi = tri_row_start(i);
            float gv[MAXV], cv[MAXV];
#pragma unroll
            for (int v = 0; v < MAXV; ++v) {
                const int k = lane + 32 * v;
                gv[v] = (k <= i) ? __ldg(Gm + (size_t)i * n + k) : 0.f;
                cv[v] = (k < d) ? __ldg(Cm + (size_t)i * d + k) : 0.f;
            }
#pragma unroll
            for (int v = 0; v < MAXV; ++v) {
                const int k = lane + 32 * v;
                if (k <= i) Lp[rsi + k] = (double)gv[v] + ((i == k && i < d) ? lam : 0.0);
                if (k < d) Z[(size_t)i * d + k] = (double)cv[v];
            }
        }
    }
    __syncthreads();

    ST(1);
    // ---------------- Cholesky, with the forward substitution riding along ----------------
    // Z^T = (L^-1 C)^T obeys the same recurrence as the rows of L below the diagonal block:
    //     Z[j][c] = (C[j][c] - sum_{k<j} Z[k][c] L[j][k]) / L[j][j],
    // so thread n + c treats right-hand-side column c as one more row of the matrix being factored (it never
    // contributes to a diagonal block).  All 257 threads work through the block columns together and no separate
    // forward pass is needed.
    // While one otherwise idle thread factors the 8 x 8 diagonal block of block column j0 (a serial chain of eight
    // reciprocal square roots), the row threads already subtract the finished columns k < j0 from their entries of
    // block column j0 + 8; the eight columns of block j0 itself are subtracted at the top of the next iteration.
    const int row = tid;
    const bool is_rhs = tid >= n && tid < n + d;
    const int col = tid - n;                           // right-hand-side column of an extra row
    const int rs = tri_row_start(row < n ? row : 0);
    // entries of block column jb owned by this thread, before any subtraction
    auto init_block = [&](double (&ac)[NB], int jb) {
        const int nbb = min(NB, n - jb);
        if (is_rhs) {
#pragma unroll
            for (int c = 0; c < NB; ++c) ac[c] = (c < nbb) ? Z[(size_t)(jb + c) * d + col] : 0.0;
        } else {
#pragma unroll
            for (int c = 0; c < NB; ++c) ac[c] = (c < nbb && jb + c <= row) ? Lp[rs + jb + c] : 0.0;
        }
    };
    // ac[c] -= sum_{k0 <= k < k1} (own row)[k] * L[jb + c][k]; k0, k1 multiples of 8: aligned pairs
    auto subtract_columns = [&](double (&ac)[NB], int jb, int k0, int k1) {
        int drs[NB];
#pragma unroll
        for (int c = 0; c < NB; ++c) drs[c] = tri_row_start(min(jb + c, n - 1));
        for (int k = k0; k < k1; k += 2) {
            double2 mine;
            if (is_rhs) mine = make_double2(Z[(size_t)k * d + col], Z[(size_t)(k + 1) * d + col]);
            else mine = *reinterpret_cast<const double2 *>(&Lp[rs + k]);
#pragma unroll
            for (int c = 0; c < NB; ++c) {
                const double2 o = *reinterpret_cast<const double2 *>(&Lp[drs[c] + k]);
                ac[c] -= mine.x * o.x;
                ac[c] -= mine.y * o.y;
            }
        }
    };
    double acc[NB];
#pragma unroll
    for (int c = 0; c < NB; ++c) acc[c] = 0.0;
    if (row < n || is_rhs) init_block(acc, 0);
    for (int j0 = 0; j0 < n; j0 += NB) {
        const int nb = min(NB, n - j0);
        const bool active = (row < n && row >= j0) || is_rhs;
        if (active) {
            if (j0 > 0) subtract_columns(acc, j0, j0 - NB, j0);
            if (!is_rhs && row < j0 + nb) {
#pragma unroll
                for (int c = 0; c < NB; ++c) diag[row - j0][c] = acc[c];
            }
        }
        __syncthreads();
        double accn[NB];
#pragma unroll
        for (int c = 0; c < NB; ++c) accn[c] = 0.0;
        if (tid == SOLVE_FACTOR_THREAD) {
            // one thread factors the nb x nb diagonal block (sqrt and reciprocal are long fp64 sequences: doing
            // them once and broadcasting beats doing them in every thread); the block is held in registers
            double Ld[NB][NB];
#pragma unroll
            for (int r = 0; r < NB; ++r)
#pragma unroll
                for (int c = 0; c < NB; ++c)
                    if (c <= r) Ld[r][c] = (r < nb) ? diag[r][c] : (r == c ? 1.0 : 0.0);
            int fail = 0;
#pragma unroll
            for (int c = 0; c < NB; ++c) {
                double v = Ld[c][c];
#pragma unroll
                for (int q = 0; q < NB; ++q)
                    if (q < c) v -= Ld[c][q] * Ld[c][q];
                if (!(v > 0.0)) { if (!fail) fail = j0 + c + 1; v = 1.0; }
                const double ri = rsqrt(v);
                Ld[c][c] = v * ri;
                if (c < nb) rdiag[j0 + c] = ri;
#pragma unroll
                for (int r = 0; r < NB; ++r)
                    if (r > c) {
                        double u = Ld[r][c];
#pragma unroll
                        for (int q = 0; q < NB; ++q)
                            if (q < c) u -= Ld[r][q] * Ld[c][q];
                        Ld[r][c] = u * ri;
                    }
            }
            if (fail) s_fail = fail;
#pragma unroll
            for (int r = 0; r < NB; ++r)
#pragma unroll
                for (int c = 0; c < NB; ++c)
                    if (c <= r) diag[r][c] = Ld[r][c];
        } else if (j0 + NB < n && ((row < n && row >= j0 + NB) || is_rhs)) {
            init_block(accn, j0 + NB);
            subtract_columns(accn, j0 + NB, 0, j0);
        }
        __syncthreads();
        if (active) {
            if (is_rhs || row >= j0 + nb) {
                // own row against the block: x_c = (acc_c - sum_{q<c} x_q L[c][q]) / L[c][c]
#pragma unroll
                for (int c = 0; c < NB; ++c)
                    if (c < nb) {
                        double v = acc[c];
#pragma unroll
                        for (int q = 0; q < NB; ++q)
                            if (q < c) v -= acc[q] * diag[c][q];
                        acc[c] = v * rdiag[j0 + c];
                        if (is_rhs) Z[(size_t)(j0 + c) * d + col] = acc[c];
                        else Lp[rs + j0 + c] = acc[c];
                    }
            } else {
                for (int c = 0; c <= row - j0; ++c) Lp[rs + j0 + c] = diag[row - j0][c];
            }
        }
        __syncthreads();
        if (s_fail) break;
#pragma unroll
        for (int c = 0; c < NB; ++c) acc[c] = accn[c];
    }

    float *Wm = a.Wb + ((size_t)li * a.n_maps + m) * p * d;
    if (s_fail) {
        for (int e = tid; e < p * d; e += blockDim.x) Wm[e] = 0.f;
        if (tid == 0) a.info[(size_t)li * a.n_maps + m] = s_fail;
        return;
    }

    ST(2);
    // ---------------- backward substitution: column c = tid / 2, the two lanes of a pair split the inner sums ----------------
    constexpr int RB = 8;
    if (tid < 2 * d) {
        const int c = tid >> 1, half = tid & 1;
        ST(3);
        // backward: L^T Theta = Z, row blocks bottom-up
        const int last = ((n - 1) / RB) * RB;
        for (int i0 = last; i0 >= 0; i0 -= RB) {
            double acc[RB];
#pragma unroll
            for (int r = 0; r < RB; ++r) acc[r] = (half == 0 && i0 + r < n) ? Z[(size_t)(i0 + r) * d + c] : 0.0;
            for (int k = i0 + RB + half; k < n; k += 2) {
                const double xk = Z[(size_t)k * d + c];
                const int rsk = tri_row_start(k) + i0;   // even offset: aligned pairs
#pragma unroll
                for (int r = 0; r < RB; r += 2) {
                    const double2 lv = *reinterpret_cast<const double2 *>(&Lp[rsk + r]);
                    acc[r] -= lv.x * xk;
                    acc[r + 1] -= lv.y * xk;
                }
            }
#pragma unroll
            for (int r = 0; r < RB; ++r) acc[r] += shfl_xor_f64(acc[r], 1);
#pragma unroll
            for (int r = RB - 1; r >= 0; --r)
                if (i0 + r < n) {
                    double v = acc[r];
#pragma unroll
                    for (int q = RB - 1; q >= 0; --q)
                        if (q > r && i0 + q < n) v -= Lp[tri_row_start(i0 + q) + i0 + r] * acc[q];
                    v *= rdiag[i0 + r];
                    acc[r] = v;
                    if (half == 0) Z[(size_t)(i0 + r) * d + c] = v;
                }
            __syncwarp();
        }
    }
    __syncthreads();
    ST(4);
    for (int e = tid; e < n * d; e += blockDim.x) Wm[e] = (float)Z[e];
    if (centred && tid < d) {
        // b = mu_y - mu_x W (Section 3.4, last display)
        const float *mup = a.mu + (size_t)m * (2 * d + 1);
        double v = (double)mup[d + tid];
        for (int i = 0; i < d; ++i) v -= (double)mup[i] * Z[(size_t)i * d + tid];
        Wm[(size_t)d * d + tid] = (float)v;
    }
    if (tid == 0) a.info[(size_t)li * a.n_maps + m] = 0;
    ST(5);
}

static cudaError_t launch_solve_any(const float *G, const float *C, const float *mu, int n_maps, int d, long long n_tokens,
                                    const float *lambdas, int n_lambda, unsigned flags, float *Wb, int *info, cudaStream_t st)
{
    SolveArgs a;
    a.G = G; a.C = C; a.mu = mu; a.Wb = Wb; a.info = info; a.n_maps = n_maps; a.d = d;
    a.inv_n = n_tokens > 0 ? 1.0 / (double)n_tokens : 0.0;
    a.flags = flags; a.n_lambda = n_lambda;
    for (int i = 0; i < 16; ++i) a.lambdas[i] = i < n_lambda ? lambdas[i] : 0.f;
    const int p = d + 1;
    const size_t smem = sizeof(double) * ((size_t)tri_row_start(p) + (size_t)p * d);
    static bool attr[MAX_DEVICES] = {};
    {
        cudaError_t e = opt_in_smem(k_ridge_solve, (size_t)(220 * 1024), attr);
        if (e != cudaSuccess) return e;
    }
    k_ridge_solve<<<n_maps * n_lambda, SOLVE_THREADS, smem, st>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

cudaError_t launch_solve(const float *G, const float *C, int n_maps, int d, long long n_tokens,
                         const float *lambdas, int n_lambda, unsigned flags, float *Wb, int *info, cudaStream_t st)
{
    return launch_solve_any(G, C, nullptr, n_maps, d, n_tokens, lambdas, n_lambda, flags, Wb, info, st);
}

cudaError_t launch_solve_centered(const float *A, const float *B, const float *mu, int n_maps, int d, long long n_tokens,
                                  const float *lambdas, int n_lambda, unsigned flags, float *Wb, int *info, cudaStream_t st)
{
    return launch_solve_any(A, B, mu, n_maps, d, n_tokens, lambdas, n_lambda, flags, Wb, info, st);
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
