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
// cos and sin of pos * f turns.  The top 23 bits of the wrapped product become the mantissa of a float in [1, 2):
// subtracting 1.5 gives the angle minus half a turn, in [-0.5, 0.5) turns, without an integer-to-float conversion
// (which would share the special-function unit with the sine and cosine); the half turn is undone by the signs.
__device__ __forceinline__ void rope_cs(uint32_t f, int pos, float &c, float &s)
{
    const uint32_t wrapped = (uint32_t)pos * f;
    const float t = __uint_as_float(0x3f800000u | (wrapped >> 9)) - 1.5f;
    const float ang = t * 6.283185307179586f;
    c = -__cosf(ang);
    s = -__sinf(ang);
}
#endif

}  // namespace cb
