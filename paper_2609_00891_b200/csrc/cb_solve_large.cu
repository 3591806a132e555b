// Batched ridge solve for regressors wider than one head (head-local support over k > 1 selected layers, Section 3.2:
// P = k*d + 1 up to a few thousand), where a system no longer fits in shared memory.  Blocked left-looking Cholesky
// and blocked substitutions in fp64 on a padded copy of every system in a caller-provided workspace:
//   per block column J (64 wide): subtract the products of the finished block columns from column J (one block per
//   64 x 64 tile and system, the tile held in registers over all products), factor the diagonal block, solve the
//   panel below it;
//   forward and backward substitution alternate a diagonal-block solve with tile updates of the remaining rows.
// Padding rows/columns carry an identity block, so every block step has the same shape.
#include "cb_internal.cuh"

namespace cb {

static constexpr int LNB = 64;                 // block size
static constexpr int LPAD = LNB + 2;           // shared-memory row pitch (doubles) of transposed tiles

struct LgArgs {
    double *A;        // [nsys][Pp][Pp] row-major; lower triangle becomes L
    double *Z;        // [nsys][Pp][d]
    int *fail;        // [nsys] first non-positive pivot (1-based) or 0
    int Pp, P, d, nsys;
};

// ---- copy in: A = G + lambda_eff J (fp32 -> fp64), identity on the padding; Z = C -----------------------------------
struct LgLoadArgs {
    const float *G, *C;
    int n_maps, sys0;
    double inv_n;
    unsigned flags;
    float lambdas[16];
};

constexpr int LG_LOAD_ROWS = 8;               // rows per block of the copy-in

__global__ void __launch_bounds__(256) k_lg_load(LgArgs a, LgLoadArgs la)
{
    const int s = blockIdx.y;                                 // system in the batch
    const int sys = la.sys0 + s, li = sys / la.n_maps, m = sys % la.n_maps;
    const float *Gm = la.G + (size_t)m * a.P * a.P;
    const float *Cm = la.C + (size_t)m * a.P * a.d;
    const double s_w = (double)Gm[(size_t)(a.P - 1) * a.P + (a.P - 1)];
    const double lam = (la.flags & CB_FLAG_RAW_LAMBDA) ? (double)la.lambdas[li] : (double)la.lambdas[li] * s_w * la.inv_n;
    for (int q = 0; q < LG_LOAD_ROWS; ++q) {
        const int i = blockIdx.x * LG_LOAD_ROWS + q;          // row
        if (i >= a.Pp) break;
        double *Ar = a.A + ((size_t)s * a.Pp + i) * a.Pp;
        double *Zr = a.Z + ((size_t)s * a.Pp + i) * a.d;
        for (int j = threadIdx.x; j < a.Pp; j += blockDim.x) {
            double v;
            if (i < a.P && j < a.P) v = (double)__ldg(Gm + (size_t)i * a.P + j) + ((i == j && i < a.P - 1) ? lam : 0.0);
            else v = (i == j) ? 1.0 : 0.0;
            Ar[j] = v;
        }
        for (int c = threadIdx.x; c < a.d; c += blockDim.x) Zr[c] = (i < a.P) ? (double)__ldg(Cm + (size_t)i * a.d + c) : 0.0;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) a.fail[s] = 0;
}

// ---- block column J, part 1: factor the 64 x 64 diagonal block A_JJ in place ---------------------------------------
// A chain of 64 dependent pivots: latency-bound, so the block is small (128 threads, 33 KB) and many systems share an SM.
__global__ void __launch_bounds__(128) k_lg_factor(LgArgs a, int J)
{
    __shared__ double Ld[LNB][LNB + 1];
    __shared__ double rinv[LNB];
    __shared__ int s_fail;
    const int s = blockIdx.x, tid = threadIdx.x;
    double *A = a.A + (size_t)s * a.Pp * a.Pp;
    const int j0 = J * LNB;
    if (tid == 0) s_fail = 0;
    for (int e = tid; e < LNB * LNB; e += 128) {
        const int r = e / LNB, c = e % LNB;
        Ld[r][c] = (c <= r) ? A[(size_t)(j0 + r) * a.Pp + j0 + c] : 0.0;
    }
    __syncthreads();
    for (int j = 0; j < LNB; ++j) {                            // unblocked right-looking Cholesky of the 64 x 64 block
        if (tid == 0) {
            double v = Ld[j][j];
            if (!(v > 0.0)) { if (!s_fail) s_fail = j0 + j + 1; v = 1.0; }
            const double ri = rsqrt(v);
            Ld[j][j] = v * ri;
            rinv[j] = ri;
        }
        __syncthreads();
        const double ri = rinv[j];
        for (int i = j + 1 + tid; i < LNB; i += 128) Ld[i][j] *= ri;
        __syncthreads();
        for (int e = tid; e < (LNB - j - 1) * (LNB - j - 1); e += 128) {
            const int i = j + 1 + e / (LNB - j - 1), k = j + 1 + e % (LNB - j - 1);
            if (k <= i) Ld[i][k] -= Ld[i][j] * Ld[k][j];
        }
        __syncthreads();
    }
    for (int e = tid; e < LNB * LNB; e += 128) {
        const int r = e / LNB, c = e % LNB;
        if (c <= r) A[(size_t)(j0 + r) * a.Pp + j0 + c] = Ld[r][c];
    }
    if (tid == 0 && s_fail && a.fail[s] == 0) a.fail[s] = s_fail;
}

// ---- block column J, part 2: L_IJ = A_IJ L_JJ^-T for the rows below; grid (row chunks of 128, systems) -------------
__global__ void __launch_bounds__(128) k_lg_panel(LgArgs a, int J)
{
    __shared__ double Ld[LNB][LNB + 1];
    __shared__ double rinv[LNB];
    const int s = blockIdx.y, tid = threadIdx.x;
    double *A = a.A + (size_t)s * a.Pp * a.Pp;
    const int j0 = J * LNB;
    for (int e = tid; e < LNB * LNB; e += 128) {
        const int r = e / LNB, c = e % LNB;
        Ld[r][c] = (c <= r) ? A[(size_t)(j0 + r) * a.Pp + j0 + c] : 0.0;
    }
    __syncthreads();
    if (tid < LNB) rinv[tid] = 1.0 / Ld[tid][tid];
    __syncthreads();
    // x L_JJ^T = a, one row per thread, the row held in registers
    const int i = j0 + LNB + blockIdx.x * 128 + tid;
    if (i >= a.Pp) return;
    double *row = A + (size_t)i * a.Pp + j0;
    double x[LNB];
#pragma unroll
    for (int c = 0; c < LNB; c += 2) {
        const double2 v = *reinterpret_cast<const double2 *>(row + c);
        x[c] = v.x;
        x[c + 1] = v.y;
    }
#pragma unroll
    for (int c = 0; c < LNB; ++c) {
        double v = x[c];
#pragma unroll
        for (int q = 0; q < c; ++q) v -= x[q] * Ld[c][q];
        x[c] = v * rinv[c];
    }
#pragma unroll
    for (int c = 0; c < LNB; c += 2) *reinterpret_cast<double2 *>(row + c) = make_double2(x[c], x[c + 1]);
}

// ---- tile products: Ctile[64 x NT] -= sum_K At_K[64 x 64] * Bt_K[64 x NT] --------------------------------------------
// MODE 0 (left-looking update of block column J before it is factored):
//                                     C = A[I][J],  At_K = L[I][K], Bt_K^T = L[J][K], K = 0 .. J-1   (I >= J, NT = 64)
// MODE 1 (forward substitution):      C = Z[I],     At = L[I][J],   Bt = Z[J]                        (I > J,  NT = d)
// MODE 2 (backward substitution):     C = Z[I],     At = L[J][I]^T, Bt = Z[J]                        (I < J,  NT = d)
// The left-looking form keeps the output tile in registers over all K: every tile of A is read and written once
// (the right-looking form re-read and re-wrote the whole trailing matrix at every step).
template <int MODE, int NT>
__global__ void __launch_bounds__(256, 2) k_lg_tile(LgArgs a, int J)
{
    extern __shared__ __align__(16) double lg_sm[];
    double (*Ats)[LPAD] = reinterpret_cast<double (*)[LPAD]>(lg_sm);                       // [k][row]
    double (*Bts)[NT + 2] = reinterpret_cast<double (*)[NT + 2]>(lg_sm + LNB * LPAD);      // [k][col]
    const int s = blockIdx.y, tid = threadIdx.x;
    double *A = a.A + (size_t)s * a.Pp * a.Pp;
    double *Z = a.Z + (size_t)s * a.Pp * a.d;
    int I;
    if (MODE == 0) I = J + blockIdx.x;
    else if (MODE == 1) I = J + 1 + blockIdx.x;
    else I = blockIdx.x;
    const int Kb = (MODE == 0) ? 0 : J, Ke = (MODE == 0) ? J : J + 1;
    // Thread (ty, tx) owns rows ty*4 .. ty*4+3 and the column pairs {32 jj + 2 tx, 32 jj + 2 tx + 1}, jj < NT/32: the 16
    // threads of a row group read 16 consecutive 16-byte pairs of Bts per access (no bank conflicts; a thread owning
    // NT/16 consecutive columns would put all 16 on two bank groups) and write 256 contiguous bytes per output row.
    constexpr int CJ = NT / 32;               // column pairs per thread
    const int ty = tid >> 4, tx = tid & 15;
    double acc[4][2 * CJ];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 2 * CJ; ++j) acc[i][j] = 0.0;
    for (int K = Kb; K < Ke; ++K) {
        if (K > Kb) __syncthreads();                              // the previous product has been read
        // All global loads of the iteration are issued before the first shared-memory store (16-byte loads, fixed
        // trip counts), so their latencies overlap instead of adding up.
        {
            // At transposed into Ats[k][r]: thread -> (row r, column pair k2) of a 64 x 64 tile, 8 pairs per thread
            double2 va[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const int e = tid + q * 256, r = e / (LNB / 2), k = (e % (LNB / 2)) * 2;
                if (MODE == 2) {                                   // L[K][I]^T: rows k, k+1 of block (K, I), column r
                    va[q].x = A[(size_t)(K * LNB + k) * a.Pp + I * LNB + r];
                    va[q].y = A[(size_t)(K * LNB + k + 1) * a.Pp + I * LNB + r];
                } else {
                    va[q] = *reinterpret_cast<const double2 *>(&A[(size_t)(I * LNB + r) * a.Pp + K * LNB + k]);
                }
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const int e = tid + q * 256, r = e / (LNB / 2), k = (e % (LNB / 2)) * 2;
                Ats[k][r] = va[q].x;
                Ats[k + 1][r] = va[q].y;
            }
            constexpr int NB2 = LNB * NT / 2 / 256;                // column pairs of Bt per thread, in batches of 8
#pragma unroll
            for (int q0 = 0; q0 < NB2; q0 += 8) {
                double2 vb[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const int e = tid + (q0 + q) * 256;
                    if (MODE == 0) {
                        const int c = e / (LNB / 2), k = (e % (LNB / 2)) * 2;
                        vb[q] = *reinterpret_cast<const double2 *>(&A[(size_t)(J * LNB + c) * a.Pp + K * LNB + k]);
                    } else {
                        const int k = e / (NT / 2), c = (e % (NT / 2)) * 2;
                        vb[q] = *reinterpret_cast<const double2 *>(&Z[(size_t)(K * LNB + k) * a.d + c]);
                    }
                }
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const int e = tid + (q0 + q) * 256;
                    if (MODE == 0) {
                        const int c = e / (LNB / 2), k = (e % (LNB / 2)) * 2;
                        Bts[k][c] = vb[q].x;
                        Bts[k + 1][c] = vb[q].y;
                    } else {
                        const int k = e / (NT / 2), c = (e % (NT / 2)) * 2;
                        *reinterpret_cast<double2 *>(&Bts[k][c]) = vb[q];
                    }
                }
            }
        }
        __syncthreads();
#pragma unroll 4
        for (int k = 0; k < LNB; ++k) {
            double av[4], bv[2 * CJ];
#pragma unroll
            for (int i = 0; i < 4; i += 2) {
                const double2 v = *reinterpret_cast<const double2 *>(&Ats[k][ty * 4 + i]);
                av[i] = v.x; av[i + 1] = v.y;
            }
#pragma unroll
            for (int jj = 0; jj < CJ; ++jj) {
                const double2 v = *reinterpret_cast<const double2 *>(&Bts[k][jj * 32 + tx * 2]);
                bv[2 * jj] = v.x; bv[2 * jj + 1] = v.y;
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 2 * CJ; ++j) acc[i][j] += av[i] * bv[j];
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = I * LNB + ty * 4 + i;
        double *crow = (MODE == 0) ? A + (size_t)r * a.Pp + J * LNB : Z + (size_t)r * a.d;
#pragma unroll
        for (int jj = 0; jj < CJ; ++jj) {
            const int c = jj * 32 + tx * 2;
            double2 v = *reinterpret_cast<double2 *>(crow + c);
            // MODE 0, diagonal tile: keep it lower-triangular
            if (!(MODE == 0 && I == J && c > ty * 4 + i)) v.x -= acc[i][2 * jj];
            if (!(MODE == 0 && I == J && c + 1 > ty * 4 + i)) v.y -= acc[i][2 * jj + 1];
            *reinterpret_cast<double2 *>(crow + c) = v;
        }
    }
}

// ---- diagonal-block solves of the substitutions: Z_J <- L_JJ^-1 Z_J (FWD) or L_JJ^-T Z_J ---------------------------
template <bool FWD>
__global__ void __launch_bounds__(128) k_lg_diag(LgArgs a, int J)
{
    extern __shared__ __align__(16) double lg_zs[];          // [LNB][d]: the block of right-hand sides being solved
    __shared__ double Ld[LNB][LNB + 1];
    __shared__ double rinv[LNB];
    const int s = blockIdx.x, tid = threadIdx.x;
    const double *A = a.A + (size_t)s * a.Pp * a.Pp;
    double *Z = a.Z + (size_t)s * a.Pp * a.d;
    const int j0 = J * LNB, d = a.d;
    for (int e = tid; e < LNB * LNB; e += 128) {
        const int r = e / LNB, c = e % LNB;
        Ld[r][c] = (c <= r) ? A[(size_t)(j0 + r) * a.Pp + j0 + c] : 0.0;
    }
    for (int e = tid; e < LNB * d; e += 128) lg_zs[e] = Z[(size_t)j0 * d + e];
    __syncthreads();
    if (tid < LNB) rinv[tid] = 1.0 / Ld[tid][tid];
    __syncthreads();
    for (int c = tid; c < d; c += 128) {                   // one column per thread; only its own column is touched
        if (FWD) {
            for (int r = 0; r < LNB; ++r) {
                double v0 = lg_zs[r * d + c], v1 = 0.0;
                int q = 0;
                for (; q + 1 < r; q += 2) { v0 -= Ld[r][q] * lg_zs[q * d + c]; v1 -= Ld[r][q + 1] * lg_zs[(q + 1) * d + c]; }
                if (q < r) v0 -= Ld[r][q] * lg_zs[q * d + c];
                lg_zs[r * d + c] = (v0 + v1) * rinv[r];
            }
        } else {
            for (int r = LNB - 1; r >= 0; --r) {
                double v0 = lg_zs[r * d + c], v1 = 0.0;
                int q = LNB - 1;
                for (; q - 1 > r; q -= 2) { v0 -= Ld[q][r] * lg_zs[q * d + c]; v1 -= Ld[q - 1][r] * lg_zs[(q - 1) * d + c]; }
                if (q > r) v0 -= Ld[q][r] * lg_zs[q * d + c];
                lg_zs[r * d + c] = (v0 + v1) * rinv[r];
            }
        }
    }
    __syncthreads();
    for (int e = tid; e < LNB * d; e += 128) Z[(size_t)j0 * d + e] = lg_zs[e];
}

// ---- copy out: Wb = Z (fp32), info; failed systems are zero-filled -------------------------------------------------
__global__ void __launch_bounds__(256) k_lg_store(LgArgs a, float *Wb, int *info, int sys0)
{
    const int s = blockIdx.y, i = blockIdx.x;
    const int sys = sys0 + s;
    const int f = a.fail[s];
    const double *Zr = a.Z + ((size_t)s * a.Pp + i) * a.d;
    float *Wr = Wb + ((size_t)sys * a.P + i) * a.d;
    for (int c = threadIdx.x; c < a.d; c += blockDim.x) Wr[c] = f ? 0.f : (float)Zr[c];
    if (i == 0 && threadIdx.x == 0) info[sys] = f;
}

template <int MODE, int NT>
static cudaError_t launch_tile(const LgArgs &a, int J, dim3 grid, cudaStream_t st)
{
    constexpr size_t smem = sizeof(double) * (LNB * LPAD + LNB * (NT + 2));
    static bool attr[MAX_DEVICES] = {};
    {
        cudaError_t e = opt_in_smem(k_lg_tile<MODE, NT>, (size_t)((int)smem), attr);
        if (e != cudaSuccess) return e;
    }
    k_lg_tile<MODE, NT><<<grid, 256, smem, st>>>(a, J);
    return cudaSuccess;
}

size_t solve_large_bytes_per_system(int P, int d)
{
    const size_t Pp = ((size_t)P + LNB - 1) / LNB * LNB;
    return sizeof(double) * (Pp * Pp + Pp * (size_t)d) + 256;
}

template <bool FWD>
static void launch_diag(const LgArgs &a, int J, cudaStream_t st)
{
    const size_t smem = sizeof(double) * LNB * (size_t)a.d;
    static bool attr[MAX_DEVICES] = {};
    opt_in_smem(k_lg_diag<FWD>, sizeof(double) * LNB * 128, attr);
    k_lg_diag<FWD><<<a.nsys, 128, smem, st>>>(a, J);
}

template <int NT>
static void launch_subst_tiles(const LgArgs &a, int nblk, cudaStream_t st)
{
    for (int J = 0; J < nblk; ++J) {
        launch_diag<true>(a, J, st);
        if (J + 1 < nblk) launch_tile<1, NT>(a, J, dim3(nblk - 1 - J, a.nsys), st);
    }
    for (int J = nblk - 1; J >= 0; --J) {
        launch_diag<false>(a, J, st);
        if (J > 0) launch_tile<2, NT>(a, J, dim3(J, a.nsys), st);
    }
}

cudaError_t launch_solve_large(const float *G, const float *C, int n_maps, int P, int d, long long n_tokens,
                               const float *lambdas, int n_lambda, unsigned flags, float *Wb, int *info,
                               void *workspace, size_t workspace_bytes, cudaStream_t st)
{
    const int Pp = (P + LNB - 1) / LNB * LNB, nblk = Pp / LNB;
    const size_t per = solve_large_bytes_per_system(P, d);
    const long long total = (long long)n_maps * n_lambda;
    long long batch = (long long)(workspace_bytes / per);
    if (batch < 1) return cudaErrorInvalidValue;
    if (batch > total) batch = total;
    if (batch > 65535) batch = 65535;
    LgLoadArgs la;
    la.G = G; la.C = C; la.n_maps = n_maps;
    la.inv_n = n_tokens > 0 ? 1.0 / (double)n_tokens : 0.0;
    la.flags = flags;
    for (int i = 0; i < 16; ++i) la.lambdas[i] = i < n_lambda ? lambdas[i] : 0.f;
    char *ws = static_cast<char *>(workspace);
    int launches = 0;
    for (long long sys0 = 0; sys0 < total; sys0 += batch) {
        LgArgs a;
        a.nsys = (int)((total - sys0 < batch) ? total - sys0 : batch);
        a.A = reinterpret_cast<double *>(ws);
        a.Z = a.A + (size_t)batch * Pp * Pp;
        a.fail = reinterpret_cast<int *>(a.Z + (size_t)batch * Pp * d);
        a.Pp = Pp; a.P = P; a.d = d;
        la.sys0 = (int)sys0;
        k_lg_load<<<dim3((Pp + LG_LOAD_ROWS - 1) / LG_LOAD_ROWS, a.nsys), 256, 0, st>>>(a, la);
        for (int J = 0; J < nblk; ++J) {
            if (J > 0) launch_tile<0, LNB>(a, J, dim3(nblk - J, a.nsys), st);      // column J -= L[:, <J] L[J, <J]^T
            k_lg_factor<<<a.nsys, 128, 0, st>>>(a, J);
            const int r = nblk - 1 - J;
            if (r > 0) k_lg_panel<<<dim3((r * LNB + 127) / 128, a.nsys), 128, 0, st>>>(a, J);
        }
        if (d == 128) launch_subst_tiles<128>(a, nblk, st);
        else launch_subst_tiles<64>(a, nblk, st);
        k_lg_store<<<dim3(P, a.nsys), 256, 0, st>>>(a, Wb, info, (int)sys0);
        launches += 2 + 3 * nblk + 4 * nblk - 4;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    count_launch(launches);
    return cudaSuccess;
}

}  // namespace cb
