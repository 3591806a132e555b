// Rotary position embedding at the cache boundary (Section 2.2, Section 3.1): device-side angle arithmetic shared by
// the kernels that remove or restore the embedding.
//
// Rotate-half convention: channel i < d/2 pairs with channel i + d/2, angle phi_i(pos) = pos * base^(-2i/d).
// Angles are carried in TURNS as 0.32 fixed point: f_i = round(base^(-2i/d) / (2 pi) * 2^32), and pos * f_i in 32-bit
// unsigned arithmetic is the angle modulo one turn, exact up to pos * 2^-33 turns (2.4e-5 rad at position 32768).  The
// wrapped angle, read as a signed integer, lies in [-pi, pi), where the fast sine and cosine are accurate to ~2^-21.
#pragma once

#include <math.h>
#include <stdint.h>

namespace cb {

constexpr int ROPE_MAX_FREQ = 64;    // d / 2 for d = 128

struct RopeDev {
    const int *pos;                  // device [n_tokens]
    uint32_t f_src[ROPE_MAX_FREQ];   // source model's frequencies (turns, 0.32 fixed point)
    uint32_t f_tgt[ROPE_MAX_FREQ];   // target model's
    int same;                        // f_src == f_tgt: one sine/cosine pair serves both
};

inline void rope_frequencies(double base, int d, uint32_t *f)
{
    for (int i = 0; i < ROPE_MAX_FREQ; ++i) {
        if (i >= d / 2) { f[i] = 0; continue; }
        const double turns = pow(base, -2.0 * (double)i / (double)d) / 6.283185307179586476925286766559;
        f[i] = (uint32_t)llround((turns - floor(turns)) * 4294967296.0);
    }
}

#ifdef __CUDACC__
// cos and sin of pos * f turns.  The top 23 bits of the wrapped product become the mantissa of a float u in [1, 2):
// (u - 1.5) 2 pi, in one fused multiply-add, is the angle minus half a turn, in [-pi, pi), without an integer-to-float
// conversion (which would share the special-function unit with the sine and cosine); the half turn is undone by the
// signs.
__device__ __forceinline__ void rope_cs(uint32_t f, int pos, float &c, float &s)
{
    const uint32_t wrapped = (uint32_t)pos * f;
    const float ang = fmaf(__uint_as_float(0x3f800000u | (wrapped >> 9)), 6.283185307179586f, -9.42477796076938f);
    c = -__cosf(ang);
    s = -__sinf(ang);
}

// The same on the FMA pipe only (measured: the special-function unit delivers ~4 sine or cosine results per clock per
// SM, the FMA pipe 128 operations): quadrant by the magic-number rounding of 4 t, then degree-7 / degree-8 polynomials
// on [-pi/4, pi/4] (error ~1e-7), then the quadrant's swap and signs.  ~21 operations for the pair.
__device__ __forceinline__ void rope_cs_poly(uint32_t f, int pos, float &c, float &s)
{
    const uint32_t wrapped = (uint32_t)pos * f;
    const float t = __uint_as_float(0x3f800000u | (wrapped >> 9)) - 1.5f;      // angle - 1/2 turn, in [-0.5, 0.5) turns
    const float m = fmaf(t, 4.f, 12582912.f);                                   // 1.5 * 2^23: rounds 4 t to an integer
    const int q = __float_as_int(m);                                            // low bits = quadrant (two's complement)
    const float r = fmaf(m - 12582912.f, -0.25f, t);                            // [-1/8, 1/8] turns
    const float x = r * 6.283185307179586f;
    const float x2 = x * x;
    float sp = fmaf(x2, -1.9840874e-4f, 8.3333310e-3f);
    sp = fmaf(x2, sp, -1.6666667e-1f);
    const float sx = fmaf(x * x2, sp, x);
    float cp = fmaf(x2, 2.4760495e-5f, -1.3888378e-3f);
    cp = fmaf(x2, cp, 4.1666638e-2f);
    cp = fmaf(x2, cp, -0.5f);
    const float cx = fmaf(x2, cp, 1.f);
    // angle = (q/4 + r) turns - 1/2 turn:  quadrant q + 2
    const bool odd = q & 1;
    const float cb = odd ? sx : cx, sb = odd ? cx : sx;
    // q mod 4 -> (cos, sin) of (x + q pi/2): 0: (c, s)  1: (-s, c)  2: (-c, -s)  3: (s, -c); then the half turn flips both
    const uint32_t cneg = ((uint32_t)((q + 1) & 2) << 30) ^ 0x80000000u;
    const uint32_t sneg = ((uint32_t)(q & 2) << 30) ^ 0x80000000u;
    c = __uint_as_float(__float_as_uint(cb) ^ cneg);
    s = __uint_as_float(__float_as_uint(sb) ^ sneg);
}
#endif

}  // namespace cb
