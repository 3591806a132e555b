// Batched closed-form ridge solve (Section 3.1, Eq. "closedform"; Section 3.4, last display), fp64, one block per
// (map, lambda), on the fp64 tensor-core instruction (mma.sync m8n8k4).
//
//   A = G + lambda_eff * diag(1,..,1,0);  A = L L^T;  L Z = C;  L^T Theta = Z.
//
// The system is padded to a multiple of 8 (identity on the padding) and cut into 8 x 8 blocks.  L lives in shared memory
// as a packed lower triangle OF BLOCKS (each block 64 contiguous doubles), the right-hand sides as rows of Z with a
// padded stride; both layouts are chosen so that every fragment load of the 8 x 8 x 4 product is free of bank
// conflicts.  A warp owns fixed tiles: right-hand-side column groups (8 columns of C, handled as tiles of Z^T, which
// obey the same recurrence as rows of L, so the forward substitution rides along with the factorization) and block
// rows of L.  Per block column: the finished tiles of the column go to shared memory; ONE warp factors the 8 x 8
// diagonal block and inverts it (the serial chain of pivots) while the eight worker warps already
// subtract all earlier block columns from their tiles of the NEXT column; then every tile of the column is multiplied
// by the inverse of the diagonal block (a product instead of eight dependent substitution steps), and the workers
// subtract the column just finished from their look-ahead tiles.  The backward substitution needs no block-wide
// barrier at all: a warp's column groups depend on nobody else's.
// Each product of 8 x 8 x 4 is one warp instruction with two 8-byte loads; the CUDA-core version it replaces issued
// one shared-memory load per 1.8 fp64 multiply-adds and was bound by shared-memory wavefronts.
#include "cb_internal.cuh"

namespace cb {

namespace {

struct SolveArgs {
    const float *G, *C;    // augmented: G [p][p], C [p][d];  centred: A [d][d], B [d][d]
    const float *mu;       // centred form only: [n_maps][2d + 1] = mu_x, mu_y, s_w; null for the augmented form
    float *Wb;
    int *info;
    int n_maps, d;
    double inv_n;
    unsigned flags;
    int n_lambda;
    int ahead;             // blocks resident at a time (one per SM): whose statistics to ask L2 for
    int c_vec;             // C is 16-byte aligned: vector loads
    float lambdas[16];
};

constexpr int SV_WORKERS = 8;                       // worker warps
constexpr int SV_THREADS = (SV_WORKERS + 1) * 32;   // + the warp that factors the diagonal blocks
constexpr int SV_LDZ = 132;                         // row stride of Z in doubles: 4 consecutive rows hit 4 distinct 32-byte bank groups
constexpr int SV_MAXBLK = 17;                       // (128 + 1 + 7) / 8

// Element (r, c) of block (ib, jb), jb <= ib.  Inside a block the two halves of a row are swapped when bit 1 of the
// row is set: the four rows that a half-warp reads together then fall into four distinct 32-byte bank groups, for
// row-wise and for column-wise fragments alike.
__device__ __forceinline__ int lidx(int ib, int jb, int r, int c)
{
    return (((ib * (ib + 1)) >> 1) + jb) * 64 + r * 8 + (c ^ ((r & 2) << 1));
}

// D (8 x 8) = A (8 x 4, row) * B (4 x 8, col) + C; lane T holds a = A[T / 4][T % 4], b = B[T % 4][T / 4],
// c0 / c1 = C[T / 4][2 (T % 4)], C[T / 4][2 (T % 4) + 1].
__device__ __forceinline__ void dmma(double &c0, double &c1, double a, double b)
{
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                 : "+d"(c0), "+d"(c1) : "d"(a), "d"(b));
}

// 1 / sqrt(v) for v > 0 on the critical path of the factorization (one pivot depends on the previous one through it):
// the single-precision reciprocal square root as a seed and two Newton steps in fp64 (relative error 2^-22 -> 2^-43 ->
// rounding level), a shorter dependent chain than the library routine.  Values outside the single-precision range take
// the library routine.
__device__ __forceinline__ double pivot_rsqrt(double v)
{
    const float vf = (float)v;
    if (!(vf > 1e-30f && vf < 1e30f)) return rsqrt(v);
    double y = (double)rsqrtf(vf);
    const double h = 0.5 * v;
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        const double e = fma(-(h * y), y, 0.5);
        y = fma(y, e, y);
    }
    return y;
}

// 1 / v the same way, with ONE Newton step (relative error 2^-23 -> 2^-45): it sits on the chain from one pivot to the
// next, where every dependent fp64 operation costs 25 to 30 cycles; the error is a relative perturbation of the
// pivots eight orders of magnitude below the precision of the fp32 statistics that are being factored.
__device__ __forceinline__ double pivot_rcp(double v)
{
    const float vf = (float)v;
    if (!(vf > 1e-30f && vf < 1e30f)) return 1.0 / v;
    float yf;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(yf) : "f"(vf));
    const double y = (double)yf;
    return fma(y, fma(-v, y, 1.0), y);
}

__global__ void __launch_bounds__(SV_THREADS, 1) k_ridge_solve(const SolveArgs a)
{
    extern __shared__ __align__(16) double sm[];
    const int d = a.d, p = d + 1;
    const bool centred = a.mu != nullptr;
    const int n = centred ? d : p;                     // order of the system: the centred form has no bias row
    const int nblk = (n + 7) >> 3, np = nblk * 8;
    const int ncg = d >> 3;                            // right-hand-side column groups
    // blocks of one map's lambdas are neighbours in launch order: the second and third read G and C from L2
    const int m = blockIdx.x / a.n_lambda, li = blockIdx.x % a.n_lambda;
    double *Ls = sm;                                   // lower triangle of 8 x 8 blocks
    double *Zs = sm + ((nblk * (nblk + 1)) >> 1) * 64; // [np][SV_LDZ]
    __shared__ int s_fail;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, q = lane & 3;

    const float *Gm = a.G + (size_t)m * n * n;
    const float *Cm = a.C + (size_t)m * n * d;
    const double s_w = centred ? (double)a.mu[(size_t)m * (2 * d + 1) + 2 * d] : (double)Gm[(size_t)d * p + d];
    const double lam = (a.flags & CB_FLAG_RAW_LAMBDA) ? (double)a.lambdas[li] : (double)a.lambdas[li] * s_w * a.inv_n;
    if (tid == 0) s_fail = 0;
    {
        // The block that will follow this one on the SM is, to a good guess, one wave of resident blocks further on
        // (one block per SM): ask L2 for its statistics now, so that its load phase does not wait for device memory.
        const int nb = blockIdx.x + a.ahead;
        if (nb < (int)gridDim.x && nb / a.n_lambda != m) {
            const int m2 = nb / a.n_lambda;
            const char *g2 = reinterpret_cast<const char *>(a.G + (size_t)m2 * n * n);
            const char *c2 = reinterpret_cast<const char *>(a.C + (size_t)m2 * n * d);
            for (int o = tid * 128; o < n * n * 4; o += SV_THREADS * 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(g2 + o));
            for (int o = tid * 128; o < n * d * 4; o += SV_THREADS * 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(c2 + o));
        }
    }
    // ---------------- load: padding first (identity on the diagonal, zero right-hand sides), then the statistics ----------------
    if (np > n) {
        const int lb = nblk - 1;
        for (int e = tid; e < nblk * 64; e += SV_THREADS) {          // last block row
            const int jb = e >> 6, r = (e >> 3) & 7, c = e & 7;
            Ls[lidx(lb, jb, r, c)] = (jb == lb && r == c) ? 1.0 : 0.0;
        }
        for (int e = tid; e < (np - n) * SV_LDZ; e += SV_THREADS) Zs[n * SV_LDZ + e] = 0.0;
        __syncthreads();
    }
    {
        // The phase is bound by load latency, so every thread keeps twelve loads in flight.  G: scalar loads (a map's G
        // starts on a 4-byte boundary only), flat over the matrix, entries above the diagonal block skipped.
        constexpr int NF = 12;
        const unsigned inv_n = (unsigned)(0x100000000ull / (unsigned)n) + 1u;      // e / n for e < 2^16 by one multiply
        for (int e0 = tid; e0 < n * n; e0 += NF * SV_THREADS) {
            float gv[NF];
#pragma unroll
            for (int v = 0; v < NF; ++v) {
                const int e = e0 + v * SV_THREADS;
                const int i = (int)__umulhi((unsigned)e, inv_n), k = e - i * n;
                gv[v] = (e < n * n && (k >> 3) <= (i >> 3)) ? __ldg(Gm + e) : 0.f;
            }
#pragma unroll
            for (int v = 0; v < NF; ++v) {
                const int e = e0 + v * SV_THREADS;
                const int i = (int)__umulhi((unsigned)e, inv_n), k = e - i * n;
                if (e < n * n && (k >> 3) <= (i >> 3))
                    Ls[lidx(i >> 3, k >> 3, i & 7, k & 7)] = (double)gv[v] + ((i == k && i < d) ? lam : 0.0);
            }
        }
        // C: 16-byte loads when the map's C is aligned for them (d is a multiple of 4, so every row then is)
        if (a.c_vec) {
            const int dq = d >> 2, sh = (d == 128) ? 5 : 4;
            for (int e0 = tid; e0 < n * dq; e0 += NF * SV_THREADS) {
                float4 cv[NF];
#pragma unroll
                for (int v = 0; v < NF; ++v) {
                    const int e = e0 + v * SV_THREADS;
                    cv[v] = (e < n * dq) ? __ldg(reinterpret_cast<const float4 *>(Cm) + e) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int v = 0; v < NF; ++v) {
                    const int e = e0 + v * SV_THREADS;
                    if (e < n * dq) {
                        double *z = Zs + (e >> sh) * SV_LDZ + (e & (dq - 1)) * 4;
                        *reinterpret_cast<double2 *>(z) = make_double2((double)cv[v].x, (double)cv[v].y);
                        *reinterpret_cast<double2 *>(z + 2) = make_double2((double)cv[v].z, (double)cv[v].w);
                    }
                }
            }
        } else {
            for (int e = tid; e < n * d; e += SV_THREADS) {
                const int i = e / d;
                Zs[i * SV_LDZ + (e - i * d)] = (double)__ldg(Cm + e);
            }
        }
    }
    __syncthreads();

    // ---------------- tiles of this warp ----------------
    // slots 0, 1: right-hand-side column groups warp, warp + 8 (tiles of Z^T); slots 2..4: block rows warp, warp + 8, warp + 16 of L
    const bool worker = warp < SV_WORKERS;
    auto z_ok = [&](int s) { return worker && warp + 8 * s < ncg; };
    auto l_ok = [&](int s, int jb) { return worker && warp + 8 * (s - 2) < nblk && warp + 8 * (s - 2) >= jb; };
    // entries of block column jb owned by this warp, before any subtraction (accumulator layout)
    auto init_tiles = [&](double (&t)[5][2], int jb) {
#pragma unroll
        for (int s = 0; s < 2; ++s)
            if (z_ok(s)) {
                const double *z = Zs + (jb * 8 + 2 * q) * SV_LDZ + (warp + 8 * s) * 8 + g;
                t[s][0] = z[0]; t[s][1] = z[SV_LDZ];
            }
#pragma unroll
        for (int s = 2; s < 5; ++s)
            if (l_ok(s, jb)) {
                const int ib = warp + 8 * (s - 2);
                t[s][0] = Ls[lidx(ib, jb, g, 2 * q)]; t[s][1] = Ls[lidx(ib, jb, g, 2 * q + 1)];
            }
    };
    auto store_tiles = [&](const double (&t)[5][2], int jb, int lmin) {      // L tiles with block row >= lmin
#pragma unroll
        for (int s = 0; s < 2; ++s)
            if (z_ok(s)) {
                double *z = Zs + (jb * 8 + 2 * q) * SV_LDZ + (warp + 8 * s) * 8 + g;
                z[0] = t[s][0]; z[SV_LDZ] = t[s][1];
            }
#pragma unroll
        for (int s = 2; s < 5; ++s)
            if (l_ok(s, lmin)) {
                const int ib = warp + 8 * (s - 2);
                Ls[lidx(ib, jb, g, 2 * q)] = t[s][0]; Ls[lidx(ib, jb, g, 2 * q + 1)] = t[s][1];
            }
    };
    // t -= (own rows)[:, block columns kb0..kb1) * (block row jb)[:, same columns]^T
    auto sub_cols = [&](double (&t)[5][2], int jb, int kb0, int kb1) {
        for (int kb = kb0; kb < kb1; ++kb) {
#pragma unroll
            for (int kh = 0; kh < 2; ++kh) {
                const double b = Ls[lidx(jb, kb, g, kh * 4 + q)];
#pragma unroll
                for (int s = 0; s < 2; ++s)
                    if (z_ok(s)) dmma(t[s][0], t[s][1], -Zs[(kb * 8 + kh * 4 + q) * SV_LDZ + (warp + 8 * s) * 8 + g], b);
#pragma unroll
                for (int s = 2; s < 5; ++s)
                    if (l_ok(s, jb)) dmma(t[s][0], t[s][1], -Ls[lidx(warp + 8 * (s - 2), kb, g, kh * 4 + q)], b);
            }
        }
    };

    // ---------------- Cholesky by block columns, the forward substitution riding along ----------------
    double acc[5][2], accn[5][2];
#pragma unroll
    for (int s = 0; s < 5; ++s) { acc[s][0] = acc[s][1] = 0.0; accn[s][0] = accn[s][1] = 0.0; }
    init_tiles(acc, 0);
    for (int jb = 0; jb < nblk; ++jb) {
        // acc holds this warp's tiles of block column jb with every earlier column subtracted
        store_tiles(acc, jb, jb);
        __syncthreads();
        if (!worker) {
            // ---- one warp turns the diagonal block into the inverse of its Cholesky factor ----
            // Pivot c + 1 depends on pivot c, and this warp shares the fp64 pipe with workers that keep it full (measured:
            // 300 cycles per pivot alone, a fifth of that speed while the workers' products run): what counts is the
            // number of fp64 instructions, most of all between two pivots.  Lane r owns row r of the block and of an identity carried through the
            // same row operations (four copies of the eight rows run side by side; values travel by shuffles, which
            // do not touch the fp64 pipe).  The block is eliminated in the root-free form A = L~ D L~^T: the next pivot
            // is one multiply and one multiply-add after the reciprocal of the current one, whose seed is the
            // single-precision reciprocal.  At the end row r of the identity part is row r of L~^-1, and
            // L^-1 = D^-1/2 L~^-1 needs one reciprocal square root per lane.
            const int r = lane & 7;
            double ar[8], xr[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                ar[k] = (k <= r) ? Ls[lidx(jb, jb, r, k)] : 0.0;
                xr[k] = (k == r) ? 1.0 : 0.0;
            }
            auto bcast = [&](double v, int src) {            // value of lane `src` of this group of eight
                const int lo = __shfl_sync(0xffffffffu, __double2loint(v), src, 8);
                const int hi = __shfl_sync(0xffffffffu, __double2hiint(v), src, 8);
                return __hiloint2double(hi, lo);
            };
            double vown = 1.0;
            int fail = 0;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                double v = bcast(ar[c], c);                  // the pivot
                if (!(v > 0.0)) { if (!fail) fail = jb * 8 + c + 1; v = 1.0; }
                if (r == c) vown = v;
                const double mrc = (r > c) ? ar[c] * pivot_rcp(v) : 0.0;
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (k > c) {                             // A[r][k] -= m_rc A[k][c]   (k <= r; the rest is never read)
                        const double akc = bcast(ar[c], k);
                        ar[k] = fma(-mrc, akc, ar[k]);
                    }
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (k <= c) {                            // the same row operation on the identity part
                        const double xck = bcast(xr[k], c);
                        xr[k] = fma(-mrc, xck, xr[k]);
                    }
            }
            if (fail && lane == 0) s_fail = fail;
            const double ri = pivot_rsqrt(vown);
            if (lane < 8) {
#pragma unroll
                for (int k = 0; k < 8; ++k) Ls[lidx(jb, jb, r, k)] = (k <= r) ? xr[k] * ri : 0.0;   // the diagonal slot now holds L_jj^-1
            }
        } else if (jb + 1 < nblk) {
            // ---- meanwhile the workers subtract all finished block columns from their tiles of the next one ----
            init_tiles(accn, jb + 1);
            sub_cols(accn, jb + 1, 0, jb);
        }
        __syncthreads();
        if (worker) {
            // ---- every tile of the column times the transposed inverse of the diagonal block ----
            const double b0 = Ls[lidx(jb, jb, g, q)], b1 = Ls[lidx(jb, jb, g, 4 + q)];
            double x[5][2];
#pragma unroll
            for (int s = 0; s < 5; ++s) {
                x[s][0] = x[s][1] = 0.0;
                if (s < 2 ? z_ok(s) : l_ok(s, jb + 1)) {
                    double a0, a1;
                    if (s < 2) {
                        const double *z = Zs + (jb * 8 + q) * SV_LDZ + (warp + 8 * s) * 8 + g;
                        a0 = z[0]; a1 = z[4 * SV_LDZ];
                    } else {
                        a0 = Ls[lidx(warp + 8 * (s - 2), jb, g, q)]; a1 = Ls[lidx(warp + 8 * (s - 2), jb, g, 4 + q)];
                    }
                    dmma(x[s][0], x[s][1], a0, b0);
                    dmma(x[s][0], x[s][1], a1, b1);
                }
            }
            __syncwarp();
            store_tiles(x, jb, jb + 1);
        }
        __syncthreads();
        if (s_fail) break;
        if (worker && jb + 1 < nblk) {
            sub_cols(accn, jb + 1, jb, jb + 1);
#pragma unroll
            for (int s = 0; s < 5; ++s) { acc[s][0] = accn[s][0]; acc[s][1] = accn[s][1]; }
        }
    }

    float *Wm = a.Wb + ((size_t)li * a.n_maps + m) * p * d;
    if (s_fail) {
        for (int e = tid; e < p * d; e += SV_THREADS) Wm[e] = 0.f;
        if (tid == 0) a.info[(size_t)li * a.n_maps + m] = s_fail;
        return;
    }

    // ---------------- backward substitution: a warp's column groups depend on nobody else's ----------------
    if (worker) {
        for (int jb = nblk - 1; jb >= 0; --jb) {
            double t[2][2];
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                t[s][0] = t[s][1] = 0.0;
                if (z_ok(s)) {
                    const double *z = Zs + (jb * 8 + 2 * q) * SV_LDZ + (warp + 8 * s) * 8 + g;
                    t[s][0] = z[0]; t[s][1] = z[SV_LDZ];
                }
            }
            // the two halves of every 8-wide step go to separate accumulators: four independent chains of products per warp
            double u[2][2];
#pragma unroll
            for (int s = 0; s < 2; ++s) u[s][0] = u[s][1] = 0.0;
            for (int ib = nblk - 1; ib > jb; --ib) {
                const double b0 = Ls[lidx(ib, jb, q, g)], b1 = Ls[lidx(ib, jb, 4 + q, g)];
#pragma unroll
                for (int s = 0; s < 2; ++s)
                    if (z_ok(s)) {
                        const double *z = Zs + (ib * 8 + q) * SV_LDZ + (warp + 8 * s) * 8 + g;
                        dmma(t[s][0], t[s][1], -z[0], b0);
                        dmma(u[s][0], u[s][1], -z[4 * SV_LDZ], b1);
                    }
            }
#pragma unroll
            for (int s = 0; s < 2; ++s) { t[s][0] += u[s][0]; t[s][1] += u[s][1]; }
            // times the inverse of the diagonal block: through shared memory into the first-operand layout
            const double b0 = Ls[lidx(jb, jb, q, g)], b1 = Ls[lidx(jb, jb, 4 + q, g)];
#pragma unroll
            for (int s = 0; s < 2; ++s)
                if (z_ok(s)) {
                    double *z = Zs + (jb * 8 + 2 * q) * SV_LDZ + (warp + 8 * s) * 8 + g;
                    z[0] = t[s][0]; z[SV_LDZ] = t[s][1];
                }
            __syncwarp();
            double x[2][2];
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                x[s][0] = x[s][1] = 0.0;
                if (z_ok(s)) {
                    const double *z = Zs + (jb * 8 + q) * SV_LDZ + (warp + 8 * s) * 8 + g;
                    dmma(x[s][0], x[s][1], z[0], b0);
                    dmma(x[s][0], x[s][1], z[4 * SV_LDZ], b1);
                }
            }
            __syncwarp();
#pragma unroll
            for (int s = 0; s < 2; ++s)
                if (z_ok(s)) {
                    double *z = Zs + (jb * 8 + 2 * q) * SV_LDZ + (warp + 8 * s) * 8 + g;
                    z[0] = x[s][0]; z[SV_LDZ] = x[s][1];
                }
            __syncwarp();
        }
    }
    __syncthreads();
    for (int e = tid; e < n * d; e += SV_THREADS) {
        const int i = e / d, c = e - i * d;
        Wm[e] = (float)Zs[i * SV_LDZ + c];
    }
    if (centred && tid < d) {
        // b = mu_y - mu_x W (Section 3.4, last display)
        const float *mup = a.mu + (size_t)m * (2 * d + 1);
        double v = (double)mup[d + tid];
        for (int i = 0; i < d; ++i) v -= (double)mup[i] * Zs[i * SV_LDZ + tid];
        Wm[(size_t)d * d + tid] = (float)v;
    }
    if (tid == 0) a.info[(size_t)li * a.n_maps + m] = 0;
}

cudaError_t launch_solve_any(const float *G, const float *C, const float *mu, int n_maps, int d, long long n_tokens,
                             const float *lambdas, int n_lambda, unsigned flags, float *Wb, int *info, cudaStream_t st)
{
    SolveArgs a;
    a.G = G; a.C = C; a.mu = mu; a.Wb = Wb; a.info = info; a.n_maps = n_maps; a.d = d;
    a.inv_n = n_tokens > 0 ? 1.0 / (double)n_tokens : 0.0;
    a.flags = flags; a.n_lambda = n_lambda;
    a.ahead = device_sm_count();
    a.c_vec = (((uintptr_t)C & 15) == 0 && (d & 3) == 0) ? 1 : 0;
    for (int i = 0; i < 16; ++i) a.lambdas[i] = i < n_lambda ? lambdas[i] : 0.f;
    const int n = mu ? d : d + 1, nblk = (n + 7) / 8;
    const size_t smem = sizeof(double) * ((size_t)(nblk * (nblk + 1) / 2) * 64 + (size_t)nblk * 8 * SV_LDZ);
    static bool attr[MAX_DEVICES] = {};
    {
        cudaError_t e = opt_in_smem(k_ridge_solve, sizeof(double) * ((size_t)(SV_MAXBLK * (SV_MAXBLK + 1) / 2) * 64 + (size_t)SV_MAXBLK * 8 * SV_LDZ), attr);
        if (e != cudaSuccess) return e;
    }
    k_ridge_solve<<<n_maps * n_lambda, SV_THREADS, smem, st>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

}  // namespace

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

}  // namespace cb
