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

// Block containing unit v when `units` are split into `nb` contiguous ranges [iU/nb, (i+1)U/nb).
__host__ __device__ inline int block_of_unit(long long v, int nb, int units) {
    return (int)(((v + 1) * nb - 1) / units);
}

// ---- Launch overlap (programmatic dependent launch).  A kernel started with launch_overlapped() may begin while the
// kernel before it on the stream is still draining: its blocks take the SM resources the finished blocks of the
// predecessor gave back, run their set-up (shared memory and registers only), and stop at
// wait_for_predecessor(), which returns once the predecessor has completed and its writes are visible.  Every
// access to global memory comes after that call.  dependents_may_start() lets the next kernel on the stream do the
// same with respect to this one; both are no-ops in a kernel that was launched the ordinary way.  When to release the
// dependents matters: a persistent kernel's blocks must all become resident together (each owns a fixed share of the
// work), so nothing small may be let in early that would occupy part of an SM when they arrive.  Measured on B200 over
// the four-stage training step: forward kernels releasing at their start and backward kernels (followed by the small
// parameter-gradient epilogue) at their end gained 3 %; releasing the epilogue early cost 4 %.
__device__ __forceinline__ void dependents_may_start() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void wait_for_predecessor() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... P, typename... A>
inline cudaError_t launch_overlapped(void (*kern)(P...), unsigned grid, unsigned block, size_t smem, cudaStream_t st,
                                     A &&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<P>(args)...);
}

// ---- Status words at the start of a workspace whose kernels wait for bulk copies.  No launch clears them: every
// call carries a fresh non-zero tag; block 0 of each kernel of the call stores it in STATUS_LAUNCH, a block whose
// bounded wait ran out stores it in STATUS_TIMEOUT.  The last call timed out iff the two words are equal (and
// non-zero); a timeout of an earlier call leaves a different tag behind and reads as clean.
constexpr int STATUS_TIMEOUT = 0, STATUS_LAUNCH = 1, STATUS_RESOLVED = 2;

}  // namespace wt
