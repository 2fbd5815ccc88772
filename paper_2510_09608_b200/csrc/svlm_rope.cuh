// Rotation factors (cos, sin)(c * theta_i) from a three-level table instead of per-element sincos.
// The table holds, for every pair i and k in [0,256): (cos, sin)(k * 256^level * theta_i), built on
// the host in fp64 and rounded to fp32.  Any |c| < 2^24 is the product of at most three entries
// (the angle-addition identity as a complex product in fp32, relative error ~2e-7).  Contiguous RoPE
// keeps positions below the retained size plus one chunk, so the third level is almost never read.
// Larger |c| (native positions of a very long stream) fall back to fp64 sincos.
#pragma once
#include <cuda_runtime.h>

#define SVLM_ROPE_LEVELS 3
#define SVLM_ROPE_RADIX 256

__device__ __forceinline__ float2 svlm_cmul(float2 a, float2 b) {
    return make_float2(a.x * b.x - a.y * b.y, a.x * b.y + a.y * b.x);
}

// Positions beyond the table's range: fp64 sincos, kept out of line (its argument reduction is a lot of code
// that the callers' instruction stream should not have to carry).
static __device__ __noinline__ float2 svlm_rope_cs_far(double angle) {
    double s, co;
    sincos(angle, &s, &co);
    return make_float2((float)co, (float)s);
}

// tab: [3][256][half] float2.  Returns (cos, sin) of c * theta where theta belongs to `pair`.
__device__ __forceinline__ float2 svlm_rope_cs(const float2* __restrict__ tab, int half, int pair, long long c,
                                               double theta) {
    const unsigned long long a = c < 0 ? (unsigned long long)(-c) : (unsigned long long)c;
    float2 r;
    if (a < (1ull << 24)) {
        const unsigned u = (unsigned)a;
        r = __ldg(tab + (size_t)(u & 255u) * half + pair);
        if (u >> 8) {
            r = svlm_cmul(r, __ldg(tab + (size_t)(256 + ((u >> 8) & 255u)) * half + pair));
            if (u >> 16) r = svlm_cmul(r, __ldg(tab + (size_t)(512 + (u >> 16)) * half + pair));
        }
    } else {
        r = svlm_rope_cs_far((double)a * theta);
    }
    if (c < 0) r.y = -r.y;
    return r;
}
