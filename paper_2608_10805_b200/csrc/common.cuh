// Shared device helpers of the WTConv CUDA library: activation load/store in the three
// storage types (arithmetic is always fp32), the Haar butterfly of Eq. 5, and the sign /
// address arithmetic of Proposition 2.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace wt {

__device__ __forceinline__ float ldf(const float *p) { return __ldg(p); }
__device__ __forceinline__ float ldf(const __half *p) { return __half2float(__ldg(p)); }
__device__ __forceinline__ float ldf(const __nv_bfloat16 *p) { return __bfloat162float(__ldg(p)); }
__device__ __forceinline__ void stf(float *p, float v) { *p = v; }
__device__ __forceinline__ void stf(__half *p, float v) { *p = __float2half_rn(v); }
__device__ __forceinline__ void stf(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

// Eq. 5: block [a b; c d] -> (LL, LH, HL, HH).
struct Haar4 {
    float ll, lh, hl, hh;
};
__device__ __forceinline__ Haar4 haar_butterfly(float a, float b, float c, float d) {
    float s0 = a + b, s1 = c + d, d0 = a - b, d1 = c - d;
    Haar4 r;
    r.ll = 0.5f * (s0 + s1);
    r.lh = 0.5f * (s0 - s1);
    r.hl = 0.5f * (d0 + d1);
    r.hh = 0.5f * (d0 - d1);
    return r;
}

// One level's term of Proposition 2 at pixel (y, x): 2^-l (LL + sy LH + sx HL + sy sx HH) with
// sy = (-1)^bit(l-1) of y.  `scale` is 2^-l.
__device__ __forceinline__ float synth_term(float ll, float lh, float hl, float hh, int by, int bx, float scale) {
    float p = by ? (ll - lh) : (ll + lh);  // LL + sy LH
    float q = by ? (hl - hh) : (hl + hh);  // HL + sy HH
    return scale * (bx ? (p - q) : (p + q));
}

static inline int host_half_up(int n) { return (n + 1) / 2; }

}  // namespace wt
