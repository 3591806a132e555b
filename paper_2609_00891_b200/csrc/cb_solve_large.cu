// Batched ridge solve for regressors wider than one head (head-local support over k > 1 selected layers, Section 3.2:
// P = k*d + 1 up to a few thousand), where a system no longer fits in shared memory.  Blocked left-looking Cholesky
// and blocked LEFT-LOOKING substitutions in fp64 on a padded copy of every system in a caller-provided workspace
// (padding rows/columns carry an identity block, so every block step has the same shape).  64 x 64 blocks.
//   per block column J:  column J -= (finished block columns) x (block row J)^T, one thread block per 64 x 64 tile and
//                        system, the tile kept in registers over all products;
//                        a small block per system factors the diagonal block AND inverts its factor;
//                        the panel below becomes a product with that inverse (L_IJ = T_IJ L_JJ^-T).
//   substitutions:       per block row J one thread block per system sums the products of the solved block rows in
//                        registers and multiplies by the inverse diagonal block: every block of Z is written once
//                        (the right-looking form re-read and re-wrote all remaining rows at every step).
// All products run on the fp64 tensor-core instruction (mma.sync m8n8k4); tiles travel global -> shared memory by
// 16-byte asynchronous copies into a two-stage ring, so the loads of the next product overlap the current one.
#include "cb_internal.cuh"

namespace cb {

// D (8 x 8) += A (8 x 4, row) * B (4 x 8, col): lane T holds a = A[T / 4][T % 4], b = B[T % 4][T / 4] and
// c0 / c1 = C[T / 4][2 (T % 4)], C[T / 4][2 (T % 4) + 1].
__device__ __forceinline__ void lg_dmma(double &c0, double &c1, double a, double b)
{
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                 : "+d"(c0), "+d"(c1) : "d"(a), "d"(b));
}
__device__ __forceinline__ void lg_cp16(void *dst_smem, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((unsigned)__cvta_generic_to_shared(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void lg_cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void lg_cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

static constexpr int LNB = 64;                 // block size
static constexpr int LPA = LNB + 4;            // shared-memory pitch (doubles) of a 64-wide tile: = 4 mod 16, so the four
                                               // rows a half-warp reads together fall into four 32-byte bank groups

struct LgArgs {
    double *A;        // [nsys][Pp][Pp] row-major; lower triangle becomes L (diagonal blocks stay factored)
    double *Z;        // [nsys][Pp][d]
    double *Li;       // [nsys][nblk][64][64] inverses of the factored diagonal blocks (lower triangular, row-major)
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
        // only the lower block triangle is ever read
        const int jend = min(a.Pp, (i / LNB + 1) * LNB);
        for (int j = threadIdx.x; j < jend; j += blockDim.x) {
            double v;
            if (i < a.P && j < a.P) v = (double)__ldg(Gm + (size_t)i * a.P + j) + ((i == j && i < a.P - 1) ? lam : 0.0);
            else v = (i == j) ? 1.0 : 0.0;
            Ar[j] = v;
        }
        for (int c = threadIdx.x; c < a.d; c += blockDim.x) Zr[c] = (i < a.P) ? (double)__ldg(Cm + (size_t)i * a.d + c) : 0.0;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) a.fail[s] = 0;
}

// ---- block column J, part 2: factor the 64 x 64 diagonal block A_JJ in place and invert the factor ------------------
// A chain of 64 dependent pivots: latency-bound, so the block is small (128 threads, 66 KB) and several systems share an SM.
__global__ void __launch_bounds__(128) k_lg_factor(LgArgs a, int J)
{
    extern __shared__ __align__(16) double fs[];
    double (*Ld)[LNB + 1] = reinterpret_cast<double (*)[LNB + 1]>(fs);                       // the block, then its factor
    double (*Xi)[LNB + 1] = reinterpret_cast<double (*)[LNB + 1]>(fs + LNB * (LNB + 1));    // the inverse of the factor
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
        // trailing update, thread (ti, tk) of a 16 x 8 grid over (row, column): no index divisions in the loop
        for (int i = j + 1 + (tid >> 3); i < LNB; i += 16) {
            const double lij = Ld[i][j];
            for (int k = j + 1 + (tid & 7); k <= i; k += 8) Ld[i][k] -= lij * Ld[k][j];
        }
        __syncthreads();
    }
    for (int e = tid; e < LNB * LNB; e += 128) {
        const int r = e / LNB, c = e % LNB;
        if (c <= r) A[(size_t)(j0 + r) * a.Pp + j0 + c] = Ld[r][c];
    }
    // inverse of the lower-triangular factor, one column per thread by forward substitution:
    //   x_c = 1 / L_cc,  x_r = -(sum_{c <= k < r} L_rk x_k) / L_rr;  rows above the diagonal are zero
    if (tid < LNB) {
        const int c = tid;
        for (int r = 0; r < LNB; ++r) {
            double v0 = 0.0, v1 = 0.0;
            int k = 0;
            for (; k + 1 < r; k += 2) { v0 -= Ld[r][k] * Xi[k][c]; v1 -= Ld[r][k + 1] * Xi[k + 1][c]; }
            if (k < r) v0 -= Ld[r][k] * Xi[k][c];
            Xi[r][c] = (r < c) ? 0.0 : (r == c ? rinv[r] : (v0 + v1) * rinv[r]);
        }
    }
    __syncthreads();
    double *Li = a.Li + ((size_t)s * (a.Pp / LNB) + J) * LNB * LNB;
    for (int e = tid; e < LNB * LNB; e += 128) Li[e] = Xi[e / LNB][e % LNB];
    if (tid == 0 && s_fail && a.fail[s] == 0) a.fail[s] = s_fail;
}

// ---- tile products ---------------------------------------------------------------------------------------------------
// One thread block of 8 warps computes a 64 x NT tile; warp w owns rows 8 w .. 8 w + 7 and all NT columns (NT / 8
// accumulator fragments of the 8 x 8 x 4 product).
//   UPDATE (left-looking update of block column J before it is factored; NT = 64):
//            A[I][J] -= sum_{K < J} L[I][K] L[J][K]^T                       grid (nblk - J, systems), I = J + x
//   PANEL    L[I][J] = A[I][J] (L_JJ^-1)^T                                   grid (nblk - 1 - J, systems), I = J + 1 + x
//   FWD      Z[J] = L_JJ^-1 (Z[J] - sum_{K < J} L[J][K] Z[K])                grid (systems)
//   BWD      Z[J] = L_JJ^-T (Z[J] - sum_{K > J} L[K][J]^T Z[K])              grid (systems)
// The first operand's tile sits in shared memory as it sits in global memory (64 rows of 64 doubles, pitch LPA) and
// is read row-wise (AT = false) or column-wise (AT = true: the operand is the transpose of the stored tile); the
// second operand's tile is either 64 rows n of 64 doubles k (BT = true: L[J][K] and the inverse diagonal block of
// PANEL) or 64 rows k of NT doubles (Z).  With pitches = 4 mod 16 doubles every fragment load is conflict-free.
enum { LG_UPDATE = 0, LG_PANEL = 1, LG_FWD = 2, LG_BWD = 3 };

template <int KIND, int NT>
struct LgTile {
    static constexpr bool ZB = KIND >= LG_FWD;                 // second operand = rows of Z
    static constexpr int LDB = ZB ? NT + 4 : LPA;              // shared-memory pitch of the second operand
    static constexpr int BW = ZB ? NT : LNB;                   // doubles per row of the second operand's tile
    static constexpr int STAGE = LNB * LPA + LNB * LDB;        // doubles per stage
    static constexpr size_t SMEM = sizeof(double) * 2 * STAGE;
};

template <int KIND, int NT>
__global__ void __launch_bounds__(256, 1) k_lg_gemm(LgArgs a, int J)
{
    using T = LgTile<KIND, NT>;
    constexpr int NF = NT / 8;
    constexpr bool AT = KIND == LG_BWD;
    extern __shared__ __align__(16) double lg_sm[];
    const int s = (KIND <= LG_PANEL) ? blockIdx.y : blockIdx.x, tid = threadIdx.x;
    const int wp = tid >> 5, lane = tid & 31, g = lane >> 2, q = lane & 3;
    const int nblk = a.Pp / LNB;
    double *A = a.A + (size_t)s * a.Pp * a.Pp;
    double *Z = a.Z + (size_t)s * a.Pp * a.d;
    const double *Li = a.Li + ((size_t)s * nblk + J) * LNB * LNB;
    int I = J;
    if (KIND == LG_UPDATE) I = J + blockIdx.x;
    if (KIND == LG_PANEL) I = J + 1 + blockIdx.x;
    const int Kb = (KIND == LG_BWD) ? J + 1 : (KIND == LG_PANEL ? J : 0);
    const int Ke = (KIND == LG_BWD) ? nblk : (KIND == LG_PANEL ? J + 1 : J);

    // asynchronous copies of the two tiles of product K into stage `buf`
    auto issue = [&](int K, int buf) {
        double *As = lg_sm + buf * T::STAGE, *Bs = As + LNB * LPA;
        const double *ag;
        if (KIND == LG_UPDATE) ag = A + (size_t)(I * LNB) * a.Pp + K * LNB;          // L[I][K]
        else if (KIND == LG_PANEL) ag = A + (size_t)(I * LNB) * a.Pp + J * LNB;      // A[I][J]
        else if (KIND == LG_FWD) ag = A + (size_t)(J * LNB) * a.Pp + K * LNB;        // L[J][K]
        else ag = A + (size_t)(K * LNB) * a.Pp + J * LNB;                            // L[K][J] (read column-wise)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int ch = tid + 256 * i, r = ch >> 5, c2 = (ch & 31) * 2;
            lg_cp16(As + r * LPA + c2, ag + (size_t)r * a.Pp + c2);
        }
        const double *bg;
        size_t ldg;
        if (KIND == LG_UPDATE) { bg = A + (size_t)(J * LNB) * a.Pp + K * LNB; ldg = a.Pp; }   // L[J][K]: rows n
        else if (KIND == LG_PANEL) { bg = Li; ldg = LNB; }                                     // L_JJ^-1: rows n
        else { bg = Z + (size_t)(K * LNB) * a.d; ldg = a.d; }                                  // Z[K]: rows k
        constexpr int CPR = T::BW / 2;                                                         // 16-byte chunks per row
#pragma unroll
        for (int i = 0; i < LNB * CPR / 256; ++i) {
            const int ch = tid + 256 * i, r = ch / CPR, c2 = (ch % CPR) * 2;
            lg_cp16(Bs + r * T::LDB + c2, bg + (size_t)r * ldg + c2);
        }
        lg_cp_commit();
    };
    // acc += (first operand) x (second operand) from one stage
    auto product = [&](double (&acc)[NF][2], const double *As, const double *Bs, bool at) {
#pragma unroll 4
        for (int k = 0; k < LNB; k += 4) {
            const double av = at ? As[(k + q) * LPA + wp * 8 + g] : As[(wp * 8 + g) * LPA + k + q];
#pragma unroll
            for (int j = 0; j < NF; ++j) {
                const double bv = T::ZB ? Bs[(k + q) * T::LDB + j * 8 + g] : Bs[(j * 8 + g) * T::LDB + k + q];
                lg_dmma(acc[j][0], acc[j][1], av, bv);
            }
        }
    };

    double acc[NF][2];
#pragma unroll
    for (int j = 0; j < NF; ++j) acc[j][0] = acc[j][1] = 0.0;
    const int nK = Ke - Kb;
    if (nK > 0) issue(Kb, 0);
    for (int it = 0; it < nK; ++it) {
        if (it + 1 < nK) { issue(Kb + it + 1, (it + 1) & 1); lg_cp_wait<1>(); }
        else lg_cp_wait<0>();
        __syncthreads();
        const double *As = lg_sm + (it & 1) * T::STAGE;
        product(acc, As, As + LNB * LPA, AT);
        __syncthreads();                                    // the stage is refilled by the next iteration's copies
    }

    const int rl = wp * 8 + g;                              // this lane's row inside the tile
    if (KIND == LG_UPDATE) {
        double *crow = A + (size_t)(I * LNB + rl) * a.Pp + J * LNB;
#pragma unroll
        for (int j = 0; j < NF; ++j) {
            const int c = j * 8 + 2 * q;
            double2 v = *reinterpret_cast<double2 *>(crow + c);
            if (!(I == J && c > rl)) v.x -= acc[j][0];      // diagonal tile: keep it lower-triangular
            if (!(I == J && c + 1 > rl)) v.y -= acc[j][1];
            *reinterpret_cast<double2 *>(crow + c) = v;
        }
    } else if (KIND == LG_PANEL) {
        double *crow = A + (size_t)(I * LNB + rl) * a.Pp + J * LNB;
#pragma unroll
        for (int j = 0; j < NF; ++j) *reinterpret_cast<double2 *>(crow + j * 8 + 2 * q) = make_double2(acc[j][0], acc[j][1]);
    } else {
        // V = Z[J] - acc goes to shared memory as the second operand of the product with the inverse diagonal block
        double *As = lg_sm, *Bs = lg_sm + LNB * LPA;
        double *zrow = Z + (size_t)(J * LNB + rl) * a.d;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int ch = tid + 256 * i, r = ch >> 5, c2 = (ch & 31) * 2;
            lg_cp16(As + r * LPA + c2, Li + (size_t)r * LNB + c2);
        }
        lg_cp_commit();
#pragma unroll
        for (int j = 0; j < NF; ++j) {
            const int c = j * 8 + 2 * q;
            const double2 v = *reinterpret_cast<const double2 *>(zrow + c);
            *reinterpret_cast<double2 *>(Bs + rl * T::LDB + c) = make_double2(v.x - acc[j][0], v.y - acc[j][1]);
            acc[j][0] = acc[j][1] = 0.0;
        }
        lg_cp_wait<0>();
        __syncthreads();
        product(acc, As, Bs, KIND == LG_BWD);               // forward: L_JJ^-1 V;  backward: (L_JJ^-1)^T V
#pragma unroll
        for (int j = 0; j < NF; ++j) *reinterpret_cast<double2 *>(zrow + j * 8 + 2 * q) = make_double2(acc[j][0], acc[j][1]);
    }
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

template <int KIND, int NT>
static cudaError_t launch_gemm(const LgArgs &a, int J, dim3 grid, cudaStream_t st)
{
    using T = LgTile<KIND, NT>;
    static bool attr[MAX_DEVICES] = {};
    cudaError_t e = opt_in_smem(k_lg_gemm<KIND, NT>, T::SMEM, attr);
    if (e != cudaSuccess) return e;
    k_lg_gemm<KIND, NT><<<grid, 256, T::SMEM, st>>>(a, J);
    return cudaSuccess;
}

size_t solve_large_bytes_per_system(int P, int d)
{
    const size_t Pp = ((size_t)P + LNB - 1) / LNB * LNB;
    return sizeof(double) * (Pp * Pp + Pp * (size_t)d + (Pp / LNB) * LNB * LNB) + 256;
}

template <int NT>
static cudaError_t launch_substitutions(const LgArgs &a, int nblk, cudaStream_t st)
{
    cudaError_t e = cudaSuccess;
    for (int J = 0; J < nblk && e == cudaSuccess; ++J) e = launch_gemm<LG_FWD, NT>(a, J, dim3(a.nsys), st);
    for (int J = nblk - 1; J >= 0 && e == cudaSuccess; --J) e = launch_gemm<LG_BWD, NT>(a, J, dim3(a.nsys), st);
    return e;
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
    const size_t factor_smem = sizeof(double) * 2 * LNB * (LNB + 1);
    static bool fattr[MAX_DEVICES] = {};
    cudaError_t e = opt_in_smem(k_lg_factor, factor_smem, fattr);
    if (e != cudaSuccess) return e;
    int launches = 0;
    for (long long sys0 = 0; sys0 < total; sys0 += batch) {
        LgArgs a;
        a.nsys = (int)((total - sys0 < batch) ? total - sys0 : batch);
        a.A = reinterpret_cast<double *>(ws);
        a.Z = a.A + (size_t)batch * Pp * Pp;
        a.Li = a.Z + (size_t)batch * Pp * d;
        a.fail = reinterpret_cast<int *>(a.Li + (size_t)batch * nblk * LNB * LNB);
        a.Pp = Pp; a.P = P; a.d = d;
        la.sys0 = (int)sys0;
        k_lg_load<<<dim3((Pp + LG_LOAD_ROWS - 1) / LG_LOAD_ROWS, a.nsys), 256, 0, st>>>(a, la);
        for (int J = 0; J < nblk && e == cudaSuccess; ++J) {
            if (J > 0) e = launch_gemm<LG_UPDATE, LNB>(a, J, dim3(nblk - J, a.nsys), st);      // column J -= L[:, <J] L[J, <J]^T
            if (e != cudaSuccess) break;
            k_lg_factor<<<a.nsys, 128, factor_smem, st>>>(a, J);
            if (J + 1 < nblk) e = launch_gemm<LG_PANEL, LNB>(a, J, dim3(nblk - 1 - J, a.nsys), st);
        }
        if (e == cudaSuccess) e = (d == 128) ? launch_substitutions<128>(a, nblk, st) : launch_substitutions<64>(a, nblk, st);
        if (e != cudaSuccess) return e;
        k_lg_store<<<dim3(P, a.nsys), 256, 0, st>>>(a, Wb, info, (int)sys0);
        launches += 2 + 3 * nblk - 2 + 2 * nblk;
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    count_launch(launches);
    return cudaSuccess;
}

}  // namespace cb
