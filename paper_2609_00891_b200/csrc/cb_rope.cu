// Stand-alone rotary embedding of a strided bf16 key tensor, in place (Section 2.2, Section 3.1): removes (inverse) or
// restores the position-dependent rotation outside the fused paths.  Pure streaming: one read and one write of K.
#include "cb_internal.cuh"
#include "cb_rope.cuh"

namespace cb {

struct RopeArgs {
    __nv_bfloat16 *k;
    long long sl, st, sh;
    int L, H, T, d;
    const int *pos;
    int inverse;
    uint32_t f[ROPE_MAX_FREQ];
};

// grid (token blocks, L * H); 256 threads = (d / 16 chunk pairs) x rows
__global__ void __launch_bounds__(256) k_rope_rotate(const RopeArgs a)
{
    const int HC = a.d / 16;                      // 16-byte chunk pairs per row
    const int rows = 256 / HC;
    const int lc = threadIdx.x % HC, r = threadIdx.x / HC;
    const int t = blockIdx.x * rows + r;
    if (t >= a.T) return;
    const int l = blockIdx.y / a.H, h = blockIdx.y % a.H;
    __nv_bfloat16 *row = a.k + (long long)l * a.sl + (long long)t * a.st + (long long)h * a.sh;
    uint4 *plo = reinterpret_cast<uint4 *>(row + lc * 8);
    uint4 *phi = reinterpret_cast<uint4 *>(row + a.d / 2 + lc * 8);
    const uint4 vlo = *plo, vhi = *phi;
    const unsigned ulo[4] = {vlo.x, vlo.y, vlo.z, vlo.w}, uhi[4] = {vhi.x, vhi.y, vhi.z, vhi.w};
    unsigned olo[4], ohi[4];
    const int pos = a.pos[t];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        float lo[2] = {__uint_as_float(ulo[e] << 16), __uint_as_float(ulo[e] & 0xffff0000u)};
        float hi[2] = {__uint_as_float(uhi[e] << 16), __uint_as_float(uhi[e] & 0xffff0000u)};
        float nl[2], nh[2];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            float c, s;
            rope_cs_poly(a.f[lc * 8 + 2 * e + q], pos, c, s);
            if (a.inverse) s = -s;
            nl[q] = lo[q] * c - hi[q] * s;
            nh[q] = lo[q] * s + hi[q] * c;
        }
        __nv_bfloat162 bl = __floats2bfloat162_rn(nl[0], nl[1]), bh = __floats2bfloat162_rn(nh[0], nh[1]);
        olo[e] = *reinterpret_cast<unsigned *>(&bl);
        ohi[e] = *reinterpret_cast<unsigned *>(&bh);
    }
    *plo = make_uint4(olo[0], olo[1], olo[2], olo[3]);
    *phi = make_uint4(ohi[0], ohi[1], ohi[2], ohi[3]);
}

cudaError_t launch_rope_rotate(void *k, int L, int H, int d, long long T, long long sl, long long st, long long sh,
                               const int *pos, double base, int inverse, cudaStream_t stream)
{
    RopeArgs a;
    a.k = static_cast<__nv_bfloat16 *>(k);
    a.sl = sl; a.st = st; a.sh = sh; a.L = L; a.H = H; a.T = (int)T; a.d = d; a.pos = pos; a.inverse = inverse;
    rope_frequencies(base, d, a.f);
    const int rows = 256 / (d / 16);
    dim3 grid((unsigned)((T + rows - 1) / rows), (unsigned)(L * H));
    k_rope_rotate<<<grid, 256, 0, stream>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

}  // namespace cb
