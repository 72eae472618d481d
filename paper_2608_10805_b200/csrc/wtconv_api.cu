// C ABI of the WTConv library: validation, workspace planning and kernel dispatch.
// Declarations and the full contract are in include/wtconv.h.  The kernels themselves are compiled in the
// per-dtype instantiation units (inst_*.cu); this unit only declares those instantiations.
#include "../../include/wtconv.h"

#include "common.cuh"
#include "tiled_kernels.cuh"
#include "plane_kernels.cuh"
#include "team_kernels.cuh"
#include "window_kernels.cuh"
#include "tiled_host.cuh"
#include "reference_chain.cuh"

#include <atomic>
#include <chrono>
#include <mutex>

namespace wt {
namespace plane {
WT_PLANE_INSTANTIATE(float, extern)
WT_PLANE_INSTANTIATE(__half, extern)
WT_PLANE_INSTANTIATE(__nv_bfloat16, extern)
}  // namespace plane
namespace team {
WT_TEAM_INSTANTIATE(float, extern)
WT_TEAM_INSTANTIATE(__half, extern)
WT_TEAM_INSTANTIATE(__nv_bfloat16, extern)
}  // namespace team
namespace window {
WT_WINDOW_INSTANTIATE(float, extern)
WT_WINDOW_INSTANTIATE(__half, extern)
WT_WINDOW_INSTANTIATE(__nv_bfloat16, extern)
}  // namespace window
namespace host {
WT_TILED_INSTANTIATE(float, 3, extern)
WT_TILED_INSTANTIATE(float, 5, extern)
WT_TILED_INSTANTIATE(float, 7, extern)
WT_TILED_INSTANTIATE(__half, 3, extern)
WT_TILED_INSTANTIATE(__half, 5, extern)
WT_TILED_INSTANTIATE(__half, 7, extern)
WT_TILED_INSTANTIATE(__nv_bfloat16, 3, extern)
WT_TILED_INSTANTIATE(__nv_bfloat16, 5, extern)
WT_TILED_INSTANTIATE(__nv_bfloat16, 7, extern)
}  // namespace host
namespace refchain {
WT_REFCHAIN_INSTANTIATE(float, 3, extern)
WT_REFCHAIN_INSTANTIATE(float, 5, extern)
WT_REFCHAIN_INSTANTIATE(float, 7, extern)
WT_REFCHAIN_INSTANTIATE(__half, 3, extern)
WT_REFCHAIN_INSTANTIATE(__half, 5, extern)
WT_REFCHAIN_INSTANTIATE(__half, 7, extern)
WT_REFCHAIN_INSTANTIATE(__nv_bfloat16, 3, extern)
WT_REFCHAIN_INSTANTIATE(__nv_bfloat16, 5, extern)
WT_REFCHAIN_INSTANTIATE(__nv_bfloat16, 7, extern)
}  // namespace refchain
}  // namespace wt

namespace {

using namespace wt::host;

wtconv_status validate_desc(const wtconv_desc *d) {
    if (!d) return WTCONV_ERR_NULL;
    if (d->B < 1 || d->C < 1 || d->H < 1 || d->W < 1) return WTCONV_ERR_SHAPE;
    if ((int64_t)d->B * d->C > 0x7fffffffLL || (int64_t)d->H * d->W > 0x3fffffffLL) return WTCONV_ERR_SHAPE;
    if (d->k != 3 && d->k != 5 && d->k != 7) return WTCONV_ERR_KERNEL_SIZE;
    if (d->L < 0 || d->L > WTCONV_MAX_LEVELS) return WTCONV_ERR_LEVELS;
    if (d->dtype != WTCONV_F32 && d->dtype != WTCONV_F16 && d->dtype != WTCONV_BF16) return WTCONV_ERR_DTYPE;
    return WTCONV_OK;
}

bool overlaps(const void *a, size_t na, const void *b, size_t nb) {
    const char *pa = (const char *)a, *pb = (const char *)b;
    return pa < pb + nb && pb < pa + na;
}

wtconv_status check_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return WTCONV_ERR_CUDA;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return WTCONV_ERR_CUDA;
    return major == 10 ? WTCONV_OK : WTCONV_ERR_ARCH;
}

// ------------------------------------------------------------------ status tags
// Every call that launches kernels with bounded waits carries a fresh non-zero tag (see the status words in
// common.cuh).  The sequence starts at a clock-derived value, so that tags left in a workspace by another process or
// an earlier load of the library are unlikely to repeat.
unsigned next_status_tag() {
    static std::atomic<unsigned> counter{
        (unsigned)std::chrono::steady_clock::now().time_since_epoch().count() * 2654435761u};
    unsigned t = counter.fetch_add(1u, std::memory_order_relaxed) + 1u;
    if (t == 0u) t = counter.fetch_add(1u, std::memory_order_relaxed) + 1u;
    return t;
}

// 1 if the last call on this workspace recorded a timeout, else 0, into the third status word.
__global__ void resolve_status_kernel(int *status) {
    const int timeout = status[wt::STATUS_TIMEOUT], launch = status[wt::STATUS_LAUNCH];
    status[wt::STATUS_RESOLVED] = (launch != 0 && timeout == launch) ? 1 : 0;
}

// ------------------------------------------------------------------ dispatch
int team_force_g(const wtconv_desc *d) { return (int)((d->flags >> 16) & 63u); }  // "planes per work unit" override
bool use_ref_chain(const wtconv_desc *d) { return (d->flags & WTCONV_FLAG_REFERENCE_CHAIN) != 0; }
bool use_team_path(const wtconv_desc *d) {
    if (d->flags & (WTCONV_FLAG_TILED_ONLY | WTCONV_FLAG_NO_TEAM | WTCONV_FLAG_REFERENCE_CHAIN)) return false;
    if ((d->flags >> 8) & ~(63u << 8)) return false;  // other launch-plan overrides address the block-per-plane kernels
    return wt::team::supported(d->B, d->C, d->H, d->W, d->k, d->L, d->dtype, team_force_g(d));
}
bool use_plane_path(const wtconv_desc *d) {  // any kernel family that keeps whole planes on chip (and a status word)
    if (d->flags & (WTCONV_FLAG_TILED_ONLY | WTCONV_FLAG_REFERENCE_CHAIN)) return false;
    return use_team_path(d) || wt::plane::supported(d->H, d->W, d->k, d->L, d->dtype);
}

// Large planes (k = 5): windows with levels 1-2 on chip, deeper levels on the whole-plane kernels over a carrier.
bool use_window_path(const wtconv_desc *d) {
    if (d->flags & (WTCONV_FLAG_TILED_ONLY | WTCONV_FLAG_NO_WINDOW | WTCONV_FLAG_REFERENCE_CHAIN)) return false;
    if (d->flags >> 8) return false;
    if (use_plane_path(d)) return false;
    // Measured on B200: with 16-byte aligned rows the per-level tiled kernels are as fast or faster (they stream whole
    // rows), with unaligned rows (225-wide 16-bit planes) they fall to element loads and the window kernels win.
    if (((size_t)d->W * elem_bytes(d->dtype)) % 16 == 0 && !(d->flags & WTCONV_FLAG_PREFER_WINDOW)) return false;
    return wt::window::supported(d->B, d->C, d->H, d->W, d->k, d->L, d->dtype);
}

// k = 3 through the k = 5 kernels.  A 3 x 3 depthwise kernel is a 5 x 5 kernel with a border of zeros, so wherever the
// kernels that keep planes on chip (k = 5 only) serve the shape, the parameters are copied into 5 x 5 tables at the
// head of the workspace, the k = 5 path runs on them, and the backward copies the inner 3 x 3 of the 5 x 5 weight
// gradients out (the border's gradients are dropped; the scale and bias gradients are unaffected, since the border
// weights are zero).  16 of 25 taps multiply zeros, and it is still 2-3 x faster than the per-level kernels.
wtconv_desc as_k5(const wtconv_desc *d) {
    wtconv_desc d5 = *d;
    d5.k = 5;
    return d5;
}
bool use_k3_embedding(const wtconv_desc *d) {
    if (d->k != 3 || (d->flags & (WTCONV_FLAG_TILED_ONLY | WTCONV_FLAG_REFERENCE_CHAIN))) return false;
    const wtconv_desc d5 = as_k5(d);
    return use_plane_path(&d5) || use_window_path(&d5);
}
// Workspace head of the embedding: w0 [C][25], wl [L][C][4][25], then the same two for the gradients; the k = 5
// path's own workspace follows.
struct EmbedLayout {
    size_t w0, wl, gw0, gwl, inner;  // byte offsets
    size_t nf0, nfl;                 // filters in w0 / wl
};
EmbedLayout embed_layout(const wtconv_desc *d) {
    EmbedLayout e;
    e.nf0 = (size_t)d->C;
    e.nfl = (size_t)d->L * d->C * 4;
    e.w0 = 0;
    e.wl = align_up(e.w0 + e.nf0 * 25 * sizeof(float));
    e.gw0 = align_up(e.wl + e.nfl * 25 * sizeof(float));
    e.gwl = align_up(e.gw0 + e.nf0 * 25 * sizeof(float));
    e.inner = align_up(e.gwl + e.nfl * 25 * sizeof(float));
    return e;
}
// filters [nf0] of a and [nfl] of b, 3 x 3 -> 5 x 5 with a zero border
__global__ void embed_k3_kernel(const float *__restrict__ a, const float *__restrict__ b, float *__restrict__ ae,
                                float *__restrict__ be, size_t nf0, size_t nfl) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (nf0 + nfl) * 25) return;
    const size_t f = i / 25;
    const int t = (int)(i - f * 25), u = t / 5, v = t - u * 5;
    const bool inner = u >= 1 && u <= 3 && v >= 1 && v <= 3;
    const int t3 = (u - 1) * 3 + (v - 1);
    if (f < nf0) ae[f * 25 + t] = inner ? a[f * 9 + t3] : 0.f;
    else be[(f - nf0) * 25 + t] = inner ? b[(f - nf0) * 9 + t3] : 0.f;
}
// the inner 3 x 3 of 5 x 5 gradients
__global__ void extract_k3_kernel(const float *__restrict__ ae, const float *__restrict__ be, float *__restrict__ a,
                                  float *__restrict__ b, size_t nf0, size_t nfl) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (nf0 + nfl) * 9) return;
    const size_t f = i / 9;
    const int t = (int)(i - f * 9), u = t / 3 + 1, v = t - (t / 3) * 3 + 1;
    if (f < nf0) a[f * 9 + t] = ae[f * 25 + u * 5 + v];
    else b[(f - nf0) * 9 + t] = be[(f - nf0) * 25 + u * 5 + v];
}

// `taps` (k = 5 only): 3 when the tables hold 3 x 3 kernels with a zero border; the block-per-plane kernels then
// leave the border out of their loops, the other kernel families multiply through it.
template <typename T, int K>
wtconv_status forward_tk(const wtconv_desc *d, const void *x, const float *w0, const float *s0, const float *b0,
                         const float *wl, const float *sl, void *out, char *ws, cudaStream_t st, int taps = 5) {
    if (use_ref_chain(d)) return wt::refchain::forward<T, K>(d, (const T *)x, w0, s0, b0, wl, sl, (T *)out, ws, st);
    if constexpr (K == 3) {
        if (use_k3_embedding(d)) {
            const wtconv_desc d5 = as_k5(d);
            const EmbedLayout e = embed_layout(d);
            float *w0e = (float *)(ws + e.w0), *wle = (float *)(ws + e.wl);
            const size_t n = (e.nf0 + e.nfl) * 25;
            embed_k3_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(w0, wl, w0e, wle, e.nf0, e.nfl);
            if (launch_status() != WTCONV_OK) return WTCONV_ERR_CUDA;
            return forward_tk<T, 5>(&d5, x, w0e, s0, b0, wle, sl, out, ws + e.inner, st, 3);
        }
    }
    if constexpr (K == 5) {
        if (use_team_path(d))
            return wt::team::forward<T>(d->B, d->C, d->H, d->W, d->L, (const T *)x, w0, s0, b0, wl, sl, (T *)out, ws, st,
                                        next_status_tag(), (d->flags & WTCONV_FLAG_TEST_NO_COPY) != 0,
                                        team_force_g(d)) == cudaSuccess
                       ? WTCONV_OK
                       : WTCONV_ERR_CUDA;
    }
    if constexpr (K == 5) {
        if (use_window_path(d))
            return wt::window::forward<T>(d->B, d->C, d->H, d->W, d->L, (const T *)x, w0, s0, b0, wl, sl, (T *)out, ws, st,
                                          next_status_tag()) == cudaSuccess
                       ? WTCONV_OK
                       : WTCONV_ERR_CUDA;
    }
    if (use_plane_path(d)) {
        if constexpr (K == 5)
            return wt::plane::forward<T>(d->B, d->C, d->H, d->W, d->L, (const T *)x, w0, s0, b0, wl, sl, (T *)out, ws,
                                         st, next_status_tag(), d->flags >> 8,
                                         (d->flags & WTCONV_FLAG_TEST_NO_COPY) != 0, taps) == cudaSuccess
                       ? WTCONV_OK
                       : WTCONV_ERR_CUDA;
    }
    return tiled_forward<T, K>(d, (const T *)x, w0, s0, b0, wl, sl, (T *)out, ws, st);
}

template <typename T, int K>
wtconv_status backward_tk(const wtconv_desc *d, const void *x, const void *g, const float *w0, const float *s0,
                          const float *b0, const float *wl, const float *sl, void *gx, float *gw0, float *gs0,
                          float *gb0, float *gwl, float *gsl, char *ws, cudaStream_t st, int taps = 5) {
    if (use_ref_chain(d))
        return wt::refchain::backward<T, K>(d, (const T *)x, (const T *)g, w0, s0, b0, wl, sl, (T *)gx, gw0, gs0, gb0, gwl, gsl,
                                            ws, st);
    if constexpr (K == 3) {
        if (use_k3_embedding(d)) {
            const wtconv_desc d5 = as_k5(d);
            const EmbedLayout e = embed_layout(d);
            float *w0e = (float *)(ws + e.w0), *wle = (float *)(ws + e.wl), *gw0e = (float *)(ws + e.gw0), *gwle = (float *)(ws + e.gwl);
            const size_t n = (e.nf0 + e.nfl) * 25, n3 = (e.nf0 + e.nfl) * 9;
            embed_k3_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(w0, wl, w0e, wle, e.nf0, e.nfl);
            if (launch_status() != WTCONV_OK) return WTCONV_ERR_CUDA;
            const wtconv_status st5 = backward_tk<T, 5>(&d5, x, g, w0e, s0, b0, wle, sl, gx, gw0e, gs0, gb0, gwle, gsl, ws + e.inner, st, 3);
            if (st5 != WTCONV_OK) return st5;
            extract_k3_kernel<<<(unsigned)((n3 + 255) / 256), 256, 0, st>>>(gw0e, gwle, gw0, gwl, e.nf0, e.nfl);
            return launch_status();
        }
    }
    if constexpr (K == 5) {
        if (use_team_path(d)) {
            wt::EpiloguePtrs ep = {};
            if (wt::team::backward<T>(d->B, d->C, d->H, d->W, d->L, (const T *)x, (const T *)g, w0, s0, wl, sl, (T *)gx,
                                      ws, &ep, st, next_status_tag(), (d->flags & WTCONV_FLAG_TEST_NO_COPY) != 0,
                                      team_force_g(d)) != cudaSuccess)
                return WTCONV_ERR_CUDA;
            return launch_epilogue(d, ep, w0, s0, b0, wl, sl, gw0, gs0, gb0, gwl, gsl, st);
        }
    }
    if constexpr (K == 5) {
        if (use_window_path(d)) {
            wt::EpiloguePtrs ep = {};
            if (wt::window::backward<T>(d->B, d->C, d->H, d->W, d->L, (const T *)x, (const T *)g, w0, s0, wl, sl, (T *)gx, ws, &ep,
                                        st, next_status_tag()) != cudaSuccess)
                return WTCONV_ERR_CUDA;
            return launch_epilogue(d, ep, w0, s0, b0, wl, sl, gw0, gs0, gb0, gwl, gsl, st);
        }
    }
    if (use_plane_path(d)) {
        if constexpr (K == 5) {
            wt::EpiloguePtrs ep = {};
            if (wt::plane::backward<T>(d->B, d->C, d->H, d->W, d->L, (const T *)x, (const T *)g, w0, s0, wl, sl,
                                       (T *)gx, ws, &ep, st, next_status_tag(), d->flags >> 8,
                                       (d->flags & WTCONV_FLAG_TEST_NO_COPY) != 0, taps) != cudaSuccess)
                return WTCONV_ERR_CUDA;
            return launch_epilogue(d, ep, w0, s0, b0, wl, sl, gw0, gs0, gb0, gwl, gsl, st);
        }
    }
    return tiled_backward<T, K>(d, (const T *)x, (const T *)g, w0, s0, b0, wl, sl, (T *)gx, gw0, gs0, gb0, gwl, gsl,
                                ws, st);
}

#define WT_DISPATCH(FN, ...)                                                                   \
    do {                                                                                       \
        switch (d->dtype * 8 + d->k) {                                                         \
            case WTCONV_F32 * 8 + 3: return FN<float, 3>(__VA_ARGS__);                         \
            case WTCONV_F32 * 8 + 5: return FN<float, 5>(__VA_ARGS__);                         \
            case WTCONV_F32 * 8 + 7: return FN<float, 7>(__VA_ARGS__);                         \
            case WTCONV_F16 * 8 + 3: return FN<__half, 3>(__VA_ARGS__);                        \
            case WTCONV_F16 * 8 + 5: return FN<__half, 5>(__VA_ARGS__);                        \
            case WTCONV_F16 * 8 + 7: return FN<__half, 7>(__VA_ARGS__);                        \
            case WTCONV_BF16 * 8 + 3: return FN<__nv_bfloat16, 3>(__VA_ARGS__);                \
            case WTCONV_BF16 * 8 + 5: return FN<__nv_bfloat16, 5>(__VA_ARGS__);                \
            case WTCONV_BF16 * 8 + 7: return FN<__nv_bfloat16, 7>(__VA_ARGS__);                \
        }                                                                                      \
        return WTCONV_ERR_DTYPE;                                                               \
    } while (0)

size_t fwd_ws_bytes(const wtconv_desc *d) {
    if (use_k3_embedding(d)) {
        const wtconv_desc d5 = as_k5(d);
        return embed_layout(d).inner + fwd_ws_bytes(&d5);
    }
    if (use_ref_chain(d)) return wt::refchain::make_plan(d).fwd_bytes;
    if (use_plane_path(d)) return align_up(wt::plane::forward_workspace_bytes(d->B, d->C, d->H, d->W, d->L));
    if (use_window_path(d)) return align_up(wt::window::ws_plan(d->B, d->C, d->H, d->W, d->L, (int)elem_bytes(d->dtype)).fwd_bytes);
    return make_tiled_plan(d).fwd_bytes;
}
size_t bwd_ws_bytes(const wtconv_desc *d) {
    if (use_k3_embedding(d)) {
        const wtconv_desc d5 = as_k5(d);
        return embed_layout(d).inner + bwd_ws_bytes(&d5);
    }
    if (use_ref_chain(d)) return wt::refchain::make_plan(d).bwd_bytes;
    if (use_team_path(d)) return align_up(wt::team::backward_workspace_bytes(d->B, d->C, d->H, d->W, d->L, (int)elem_bytes(d->dtype), team_force_g(d)));
    if (use_window_path(d)) return align_up(wt::window::ws_plan(d->B, d->C, d->H, d->W, d->L, (int)elem_bytes(d->dtype)).bwd_bytes);
    if (use_plane_path(d)) return align_up(wt::plane::backward_workspace_bytes(d->B, d->C, d->H, d->W, d->L, (int)elem_bytes(d->dtype), d->flags >> 8));
    return make_tiled_plan(d).bwd_bytes;
}

struct ParamSizes {
    size_t w0, s0, wl, sl;
};
ParamSizes param_sizes(const wtconv_desc *d) {
    size_t KK = (size_t)d->k * d->k, C = d->C, L = d->L;
    return {C * KK * 4, C * 4, L * C * 4 * KK * 4, L * C * 4 * 4};
}

// ------------------------------------------------------------------ allocation-free backward
// Scratch for wtconv_backward_static: lives in the library image, so every GPU that loads the library holds
// these bytes until the process exits.  Its name is only a host-side handle; the device address is looked
// up once per device with cudaGetSymbolAddress (see static_scratch_for_current_device).
static __device__ __align__(256) unsigned char wt_static_scratch[WTCONV_STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
std::mutex g_scratch_mutex;
void *g_scratch_ptr[MAX_DEVICES] = {};

// Device address of wt_static_scratch on the current device; resolved on the first call per device.
wtconv_status static_scratch_for_current_device(void **out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return WTCONV_ERR_CUDA;
    if (dev < 0 || dev >= MAX_DEVICES) return WTCONV_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, wt_static_scratch) != cudaSuccess || !p) return WTCONV_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return WTCONV_OK;
}

// wtconv_step_host splits the batch into chunks so that uploads, kernels and downloads of different chunks overlap.
constexpr int STEP_MAX_CHUNKS = 8;
int pick_step_chunks(const wtconv_desc *d) {
    const size_t per_image = (size_t)d->C * d->H * d->W * elem_bytes(d->dtype);
    for (int n = STEP_MAX_CHUNKS; n >= 2; n /= 2)
        if (d->B % n == 0 && d->B / n >= 4 && ((size_t)(d->B / n) * per_image) % 16 == 0 &&
            (size_t)(d->B / n) * per_image >= ((size_t)4 << 20))
            return n;
    return 1;
}
// dst[i] = sum over chunks of src[c * stride + i], in chunk order (deterministic).
__global__ void sum_chunks_kernel(float *__restrict__ dst, const float *__restrict__ src, size_t n, int nch, size_t stride) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float a = src[i];
    for (int c = 1; c < nch; ++c) a += src[(size_t)c * stride + i];
    dst[i] = a;
}

// Internal copy stream of wtconv_step_host, one per device, created on first use and kept for the process.
std::mutex g_side_mutex;
cudaStream_t g_side_stream[MAX_DEVICES][2] = {};  // [0] downloads, [1] uploads
wtconv_status side_stream_for_current_device(cudaStream_t *out, int which = 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return WTCONV_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_side_mutex);
    if (!g_side_stream[dev][which] &&
        cudaStreamCreateWithFlags(&g_side_stream[dev][which], cudaStreamNonBlocking) != cudaSuccess)
        return WTCONV_ERR_CUDA;
    *out = g_side_stream[dev][which];
    return WTCONV_OK;
}

// Events of wtconv_step_host, per device, created on first use and kept for the process (calls on one device
// must not overlap in time, so they can share them; creating and destroying twenty events per call costs more
// host time than a small layer's kernels take).
constexpr int STEP_EVENTS = 2 * STEP_MAX_CHUNKS + 4;
cudaEvent_t g_step_events[MAX_DEVICES][STEP_EVENTS] = {};
wtconv_status step_events_for_current_device(cudaEvent_t **out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return WTCONV_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_side_mutex);
    for (int i = 0; i < STEP_EVENTS; ++i)
        if (!g_step_events[dev][i] &&
            cudaEventCreateWithFlags(&g_step_events[dev][i], cudaEventDisableTiming) != cudaSuccess)
            return WTCONV_ERR_CUDA;
    *out = g_step_events[dev];
    return WTCONV_OK;
}

}  // namespace

extern "C" {

const char *wtconv_status_string(wtconv_status st) {
    switch (st) {
        case WTCONV_OK: return "ok";
        case WTCONV_ERR_NULL: return "a required pointer is NULL";
        case WTCONV_ERR_SHAPE: return "invalid shape";
        case WTCONV_ERR_KERNEL_SIZE: return "kernel size must be 3, 5 or 7";
        case WTCONV_ERR_LEVELS: return "level count out of range";
        case WTCONV_ERR_DTYPE: return "unknown dtype";
        case WTCONV_ERR_ALIGNMENT: return "pointer not sufficiently aligned";
        case WTCONV_ERR_WORKSPACE: return "workspace missing or too small";
        case WTCONV_ERR_ALIAS: return "an output overlaps an input";
        case WTCONV_ERR_ARCH: return "device is not compute capability 10.x";
        case WTCONV_ERR_CUDA: return "CUDA runtime error";
        case WTCONV_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

wtconv_status wtconv_level_shape(const wtconv_desc *d, int level, int32_t *Hl, int32_t *Wl) {
    if (!d || !Hl || !Wl) return WTCONV_ERR_NULL;
    if (d->H < 1 || d->W < 1) return WTCONV_ERR_SHAPE;
    if (level < 0 || level > WTCONV_MAX_LEVELS) return WTCONV_ERR_LEVELS;
    Shapes s = level_shapes(d);
    *Hl = s.Hs[level];
    *Wl = s.Ws[level];
    return WTCONV_OK;
}

wtconv_status wtconv_workspace_bytes(const wtconv_desc *d, size_t *fwd_bytes, size_t *bwd_bytes) {
    wtconv_status st = validate_desc(d);
    if (st != WTCONV_OK) return st;
    if (fwd_bytes) *fwd_bytes = fwd_ws_bytes(d);
    if (bwd_bytes) *bwd_bytes = bwd_ws_bytes(d);
    return WTCONV_OK;
}

const char *wtconv_plan_name(const wtconv_desc *d) {
    if (validate_desc(d) != WTCONV_OK) return nullptr;
    if (use_k3_embedding(d)) {  // the kernels that run: the k = 5 path's
        const wtconv_desc d5 = as_k5(d);
        return wtconv_plan_name(&d5);
    }
    return use_ref_chain(d) ? "reference-chain" : use_team_path(d) ? "team" : use_plane_path(d) ? "plane" : use_window_path(d) ? "window" : "tiled";
}

wtconv_status wtconv_plan_describe(const wtconv_desc *d, char *buf, size_t n) {
    wtconv_status st = validate_desc(d);
    if (st != WTCONV_OK) return st;
    if (!buf || n == 0) return WTCONV_ERR_NULL;
    buf[0] = 0;
    if (use_k3_embedding(d)) {
        const wtconv_desc d5 = as_k5(d);
        const int o = snprintf(buf, n, "3x3 kernels in 5x5 tables: ");
        return o > 0 && (size_t)o < n ? wtconv_plan_describe(&d5, buf + o, n - o) : WTCONV_OK;
    }
    if (use_ref_chain(d))
        snprintf(buf, n, "reference-chain (separate operators, intermediates in HBM)%s%s",
                 (d->flags & WTCONV_FLAG_ABLATE_FUSED_ANALYSIS) ? " +fused-analysis" : "",
                 (d->flags & WTCONV_FLAG_ABLATE_COLLAPSED_SYNTHESIS) ? " +collapsed-synthesis" : "");
    else if (use_team_path(d))
        wt::team::describe(d->B, d->C, d->H, d->W, d->L, (int)elem_bytes(d->dtype), buf, n, team_force_g(d));
    else if (use_window_path(d)) {
        wt::window::WGeom wf, wb;
        wt::window::make_plan(d->B, d->C, d->H, d->W, d->L, (int)elem_bytes(d->dtype), false, wf);
        wt::window::make_plan(d->B, d->C, d->H, d->W, d->L, (int)elem_bytes(d->dtype), true, wb);
        snprintf(buf, n, "window fwd[%dx%d px, %d thr x %d/SM, buffers=%d, %s] bwd[%dx%d px, %d thr x %d/SM, buffers=%d, np=%d]%s",
                 wf.WH, wf.WW, wf.g.nthreads, wf.g.blocks_per_sm, wf.nbuf, wf.aligned ? "aligned rows" : "unaligned rows", wb.WH, wb.WW,
                 wb.g.nthreads, wb.g.blocks_per_sm, wb.nbuf, wb.g.np, d->L > 2 ? " + whole-plane kernels on the level-2 carrier" : "");
    } else if (use_plane_path(d))
        wt::plane::describe(d->B, d->C, d->H, d->W, d->L, (int)elem_bytes(d->dtype), d->flags >> 8, buf, n);
    else
        snprintf(buf, n, "tiled fwd[%d launches] bwd[%d launches]", d->L + 1, d->L + 2);
    return WTCONV_OK;
}

wtconv_status wtconv_launch_count(const wtconv_desc *d, int32_t *fwd, int32_t *bwd) {
    wtconv_status st = validate_desc(d);
    if (st != WTCONV_OK) return st;
    if (use_k3_embedding(d)) {  // the k = 5 path's launches + the table kernel (+ the gradient copy in the backward)
        const wtconv_desc d5 = as_k5(d);
        st = wtconv_launch_count(&d5, fwd, bwd);
        if (st == WTCONV_OK && fwd) *fwd += 1;
        if (st == WTCONV_OK && bwd) *bwd += 2;
        return st;
    }
    if (use_ref_chain(d)) {
        const bool fa = d->flags & WTCONV_FLAG_ABLATE_FUSED_ANALYSIS, cs = d->flags & WTCONV_FLAG_ABLATE_COLLAPSED_SYNTHESIS;
        const int nf = (fa ? 1 : 0) + d->L * (fa ? 2 : 3) + (d->L > 1 && !fa ? d->L - 1 : 0) + 2 + (cs ? 1 : 2 * d->L + 1);
        if (fwd) *fwd = nf;
        if (bwd) *bwd = (4 * d->L + 3) + 7 + 9 * d->L;  // plain forward chain + gradient launches (approximate for L > 1 slices)
    } else if (use_window_path(d)) {
        // window kernel (+ carrier, scale fill and the whole-plane kernel when L > 2); backward: + second carrier, epilogue
        if (fwd) *fwd = d->L > 2 ? 4 : 1;
        if (bwd) *bwd = d->L > 2 ? 7 : 2;
    } else if (use_team_path(d)) {
        if (fwd) *fwd = 1;
        if (bwd) *bwd = 2;  // fused backward + epilogue (and nothing else on the stream)
    } else if (use_plane_path(d)) {
        if (fwd) *fwd = 1;
        if (bwd) {
            wt::plane::Geom gq;
            /* fused backward + epilogue, or weight-gradient + input-gradient + epilogue (and nothing else on the stream) */
            *bwd = wt::plane::plan_bwd_fused(d->B, d->C, d->H, d->W, d->L, (int)elem_bytes(d->dtype), gq, d->flags >> 8) ? 2 : 3;
        }
    } else {
        if (fwd) *fwd = d->L + 1;
        if (bwd) *bwd = d->L + 2;
    }
    return WTCONV_OK;
}

wtconv_status wtconv_forward(const wtconv_desc *d, const void *x, const float *w0, const float *s0, const float *b0,
                             const float *wl, const float *sl, void *out, void *workspace, size_t workspace_bytes,
                             void *stream) {
    wtconv_status st = validate_desc(d);
    if (st != WTCONV_OK) return st;
    if (!x || !w0 || !s0 || !out || (d->L > 0 && (!wl || !sl))) return WTCONV_ERR_NULL;
    if (((uintptr_t)x | (uintptr_t)out) & 15) return WTCONV_ERR_ALIGNMENT;
    const size_t need = fwd_ws_bytes(d);
    if (need > 0 && (!workspace || workspace_bytes < need)) return WTCONV_ERR_WORKSPACE;
    if (need > 0 && ((uintptr_t)workspace & (ALIGN - 1))) return WTCONV_ERR_ALIGNMENT;
    const size_t nbytes = (size_t)d->B * d->C * d->H * d->W * elem_bytes(d->dtype);
    if (overlaps(x, nbytes, out, nbytes)) return WTCONV_ERR_ALIAS;
    if ((st = check_device()) != WTCONV_OK) return st;
    char *ws = (char *)workspace;
    cudaStream_t cs = (cudaStream_t)stream;
    WT_DISPATCH(forward_tk, d, x, w0, s0, b0, wl, sl, out, ws, cs);
}

wtconv_status wtconv_backward(const wtconv_desc *d, const void *x, const void *grad_out, const float *w0,
                              const float *s0, const float *b0, const float *wl, const float *sl, void *grad_x,
                              float *grad_w0, float *grad_s0, float *grad_b0, float *grad_wl, float *grad_sl,
                              void *workspace, size_t workspace_bytes, void *stream) {
    wtconv_status st = validate_desc(d);
    if (st != WTCONV_OK) return st;
    if (!x || !grad_out || !w0 || !s0 || !grad_x || !grad_w0 || !grad_s0) return WTCONV_ERR_NULL;
    if (d->L > 0 && (!wl || !sl || !grad_wl || !grad_sl)) return WTCONV_ERR_NULL;
    if ((b0 == nullptr) != (grad_b0 == nullptr)) return WTCONV_ERR_NULL;
    if (((uintptr_t)x | (uintptr_t)grad_out | (uintptr_t)grad_x) & 15) return WTCONV_ERR_ALIGNMENT;
    const size_t need = bwd_ws_bytes(d);
    if (!workspace || workspace_bytes < need) return WTCONV_ERR_WORKSPACE;
    if ((uintptr_t)workspace & (ALIGN - 1)) return WTCONV_ERR_ALIGNMENT;
    const size_t nbytes = (size_t)d->B * d->C * d->H * d->W * elem_bytes(d->dtype);
    if (overlaps(x, nbytes, grad_x, nbytes) || overlaps(grad_out, nbytes, grad_x, nbytes)) return WTCONV_ERR_ALIAS;
    if ((st = check_device()) != WTCONV_OK) return st;
    char *ws = (char *)workspace;
    cudaStream_t cs = (cudaStream_t)stream;
    WT_DISPATCH(backward_tk, d, x, grad_out, w0, s0, b0, wl, sl, grad_x, grad_w0, grad_s0, grad_b0, grad_wl, grad_sl,
                ws, cs);
}

// Device staging layout of wtconv_step_host: x, g, out, gx (activation dtype), then the
// parameters, then the parameter gradients, then the kernels' own workspace.
wtconv_status wtconv_step_host_workspace_bytes(const wtconv_desc *d, size_t *bytes) {
    wtconv_status st = validate_desc(d);
    if (st != WTCONV_OK) return st;
    if (!bytes) return WTCONV_ERR_NULL;
    const size_t act = align_up((size_t)d->B * d->C * d->H * d->W * elem_bytes(d->dtype));
    ParamSizes ps = param_sizes(d);
    const size_t par = align_up(ps.w0) + 2 * align_up(ps.s0) + align_up(ps.wl) + align_up(ps.sl);
    size_t f = fwd_ws_bytes(d), b = bwd_ws_bytes(d);
    size_t scratch = f > b ? f : b;
    const int nch = pick_step_chunks(d);
    if (nch > 1) {  // the pipelined step runs the kernels on B / nch images: their scratch need not be smaller
        wtconv_desc dc = *d;
        dc.B = d->B / nch;
        f = fwd_ws_bytes(&dc);
        b = bwd_ws_bytes(&dc);
        if (f > scratch) scratch = f;
        if (b > scratch) scratch = b;
    }
    // parameters, their gradients, and one more gradient set per batch chunk of the pipelined step
    *bytes = 4 * act + (2 + STEP_MAX_CHUNKS) * par + align_up(scratch);
    return WTCONV_OK;
}

wtconv_status wtconv_step_host(const wtconv_desc *d, const void *h_x, const void *h_g, const float *h_w0,
                               const float *h_s0, const float *h_b0, const float *h_wl, const float *h_sl, void *h_out,
                               void *h_gx, float *h_gw0, float *h_gs0, float *h_gb0, float *h_gwl, float *h_gsl,
                               void *workspace, size_t workspace_bytes, void *stream) {
    wtconv_status st = validate_desc(d);
    if (st != WTCONV_OK) return st;
    if (!h_x || !h_g || !h_w0 || !h_s0 || !h_out || !h_gx || !h_gw0 || !h_gs0) return WTCONV_ERR_NULL;
    if (d->L > 0 && (!h_wl || !h_sl || !h_gwl || !h_gsl)) return WTCONV_ERR_NULL;
    if ((h_b0 == nullptr) != (h_gb0 == nullptr)) return WTCONV_ERR_NULL;
    size_t need = 0;
    wtconv_step_host_workspace_bytes(d, &need);
    if (!workspace || workspace_bytes < need) return WTCONV_ERR_WORKSPACE;
    if ((uintptr_t)workspace & (ALIGN - 1)) return WTCONV_ERR_ALIGNMENT;
    cudaStream_t cs = (cudaStream_t)stream;
    const size_t act_raw = (size_t)d->B * d->C * d->H * d->W * elem_bytes(d->dtype), act = align_up(act_raw);
    ParamSizes ps = param_sizes(d);
    char *p = (char *)workspace;
    char *dx_ = p, *dg = p + act, *dout = p + 2 * act, *dgx = p + 3 * act;
    p += 4 * act;
    auto take = [&](size_t n) { char *q = p; p += align_up(n); return q; };
    float *w0 = (float *)take(ps.w0), *s0 = (float *)take(ps.s0), *b0 = (float *)take(ps.s0);
    float *wl = (float *)take(ps.wl), *sl = (float *)take(ps.sl);
    float *gw0 = (float *)take(ps.w0), *gs0 = (float *)take(ps.s0), *gb0 = (float *)take(ps.s0);
    float *gwl = (float *)take(ps.wl), *gsl = (float *)take(ps.sl);
    const size_t rest = workspace_bytes - (size_t)(p - (char *)workspace);
    bool ok = true;
    auto h2d = [&](void *dst, const void *src, size_t n) {
        if (n) ok = ok && cudaMemcpyAsync(dst, src, n, cudaMemcpyHostToDevice, cs) == cudaSuccess;
    };
    auto d2h = [&](void *dst, const void *src, size_t n) {
        if (n) ok = ok && cudaMemcpyAsync(dst, src, n, cudaMemcpyDeviceToHost, cs) == cudaSuccess;
    };
    // The forward needs only x: its result travels back on an internal stream while grad_out is still on its
    // way up (the link is full duplex), and `stream` waits for that copy before it reaches the end of the step.
    cudaStream_t side = nullptr;
    if ((st = side_stream_for_current_device(&side)) != WTCONV_OK) return st;
    cudaEvent_t *pool = nullptr;
    if ((st = step_events_for_current_device(&pool)) != WTCONV_OK) return st;
    cudaEvent_t fwd_done = pool[STEP_EVENTS - 2], out_home = pool[STEP_EVENTS - 1];
    const float *b0p = h_b0 ? b0 : nullptr;
    const int nch = pick_step_chunks(d);
    if (nch > 1) {
        // Pipelined step: chunk c's upload and kernels run on `stream`, its results travel back on the internal
        // stream while chunk c+1 is uploaded.  Every chunk leaves its own parameter gradients; they are added
        // in chunk order at the end.
        const size_t par_bytes = (size_t)((char *)gsl + align_up(ps.sl) - (char *)gw0);  // one gradient set
        char *chunk_grads = p;
        p += (size_t)STEP_MAX_CHUNKS * par_bytes;
        const size_t rest_c = workspace_bytes - (size_t)(p - (char *)workspace);
        wtconv_desc dc = *d;
        dc.B = d->B / nch;
        const size_t cb = act_raw / nch;
        h2d(w0, h_w0, ps.w0);
        h2d(s0, h_s0, ps.s0);
        if (h_b0) h2d(b0, h_b0, ps.s0);
        h2d(wl, h_wl, ps.wl);
        h2d(sl, h_sl, ps.sl);
        // events: [0..nch) chunk computed, [nch] downloads done, [nch+1] stream position at entry,
        // [nch+2 .. 2 nch+2) chunk uploaded
        cudaEvent_t *ev = pool;
        cudaStream_t up = nullptr;
        if (ok && side_stream_for_current_device(&up, 1) != WTCONV_OK) ok = false;
        if (!ok) return WTCONV_ERR_CUDA;
        // uploads run on their own stream (behind whatever `stream` holds at entry), so that chunk c+1 arrives
        // while chunk c is being computed
        ok = ok && cudaEventRecord(ev[nch + 1], cs) == cudaSuccess && cudaStreamWaitEvent(up, ev[nch + 1], 0) == cudaSuccess;
        for (int c = 0; c < nch && ok; ++c) {
            const size_t o = (size_t)c * cb;
            ok = ok && cudaMemcpyAsync(dx_ + o, (const char *)h_x + o, cb, cudaMemcpyHostToDevice, up) == cudaSuccess;
            ok = ok && cudaMemcpyAsync(dg + o, (const char *)h_g + o, cb, cudaMemcpyHostToDevice, up) == cudaSuccess;
            ok = ok && cudaEventRecord(ev[nch + 2 + c], up) == cudaSuccess;
        }
        if (!ok) {  // nothing of this step may outlive the caller's stream position
            if (cudaEventRecord(ev[nch], up) == cudaSuccess) cudaStreamWaitEvent(cs, ev[nch], 0);
            return WTCONV_ERR_CUDA;
        }
        for (int c = 0; c < nch; ++c) {
            const size_t o = (size_t)c * cb;
            ok = ok && cudaStreamWaitEvent(cs, ev[nch + 2 + c], 0) == cudaSuccess;
            if (!ok) break;
            char *gq = chunk_grads + (size_t)c * par_bytes;  // same layout as the final gradient set
            float *cgw0 = (float *)gq, *cgs0 = (float *)(gq + ((char *)gs0 - (char *)gw0)),
                  *cgb0 = (float *)(gq + ((char *)gb0 - (char *)gw0)), *cgwl = (float *)(gq + ((char *)gwl - (char *)gw0)),
                  *cgsl = (float *)(gq + ((char *)gsl - (char *)gw0));
            st = wtconv_forward(&dc, dx_ + o, w0, s0, b0p, wl, sl, dout + o, p, rest_c, stream);
            if (st == WTCONV_OK)
                st = wtconv_backward(&dc, dx_ + o, dg + o, w0, s0, b0p, wl, sl, dgx + o, cgw0, cgs0, h_b0 ? cgb0 : nullptr,
                                     cgwl, cgsl, p, rest_c, stream);
            if (st != WTCONV_OK) break;
            ok = ok && cudaEventRecord(ev[c], cs) == cudaSuccess;
            ok = ok && cudaStreamWaitEvent(side, ev[c], 0) == cudaSuccess;
            if (ok) ok = cudaMemcpyAsync((char *)h_out + o, dout + o, cb, cudaMemcpyDeviceToHost, side) == cudaSuccess;
            if (ok) ok = cudaMemcpyAsync((char *)h_gx + o, dgx + o, cb, cudaMemcpyDeviceToHost, side) == cudaSuccess;
        }
        // join first, so that `stream` ends after both internal streams whatever happened above (every upload
        // event has either been waited for by `stream` or precedes the last one, which is waited for here)
        bool joined = cudaStreamWaitEvent(cs, ev[nch + 2 + nch - 1], 0) == cudaSuccess &&
                      cudaEventRecord(ev[nch], side) == cudaSuccess && cudaStreamWaitEvent(cs, ev[nch], 0) == cudaSuccess;
        if (st != WTCONV_OK) return st;
        if (!ok || !joined) return WTCONV_ERR_CUDA;
        const size_t nfl = par_bytes / sizeof(float);
        sum_chunks_kernel<<<(unsigned)((nfl + 255) / 256), 256, 0, cs>>>(gw0, (const float *)chunk_grads, nfl, nch, nfl);
        if (launch_status() != WTCONV_OK) return WTCONV_ERR_CUDA;
        d2h(h_gw0, gw0, ps.w0);
        d2h(h_gs0, gs0, ps.s0);
        if (h_b0) d2h(h_gb0, gb0, ps.s0);
        d2h(h_gwl, gwl, ps.wl);
        d2h(h_gsl, gsl, ps.sl);
        return ok ? WTCONV_OK : WTCONV_ERR_CUDA;
    }
    h2d(dx_, h_x, act_raw);
    h2d(w0, h_w0, ps.w0);
    h2d(s0, h_s0, ps.s0);
    if (h_b0) h2d(b0, h_b0, ps.s0);
    h2d(wl, h_wl, ps.wl);
    h2d(sl, h_sl, ps.sl);
    if (!ok) return WTCONV_ERR_CUDA;
    st = wtconv_forward(d, dx_, w0, s0, b0p, wl, sl, dout, p, rest, stream);
    if (st != WTCONV_OK) return st;
    ok = ok && cudaEventRecord(fwd_done, cs) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(side, fwd_done, 0) == cudaSuccess;
    if (ok) ok = cudaMemcpyAsync(h_out, dout, act_raw, cudaMemcpyDeviceToHost, side) == cudaSuccess;
    ok = ok && cudaEventRecord(out_home, side) == cudaSuccess;
    h2d(dg, h_g, act_raw);
    if (!ok) return WTCONV_ERR_CUDA;
    st = wtconv_backward(d, dx_, dg, w0, s0, b0p, wl, sl, dgx, gw0, gs0, h_b0 ? gb0 : nullptr, gwl, gsl, p, rest,
                         stream);
    if (st != WTCONV_OK) {
        cudaStreamWaitEvent(cs, out_home, 0);
        return st;
    }
    d2h(h_gx, dgx, act_raw);
    d2h(h_gw0, gw0, ps.w0);
    d2h(h_gs0, gs0, ps.s0);
    if (h_b0) d2h(h_gb0, gb0, ps.s0);
    d2h(h_gwl, gwl, ps.wl);
    d2h(h_gsl, gsl, ps.sl);
    ok = ok && cudaStreamWaitEvent(cs, out_home, 0) == cudaSuccess;  // join: the step ends when `out` is home too
    return ok ? WTCONV_OK : WTCONV_ERR_CUDA;
}

wtconv_status wtconv_read_status(const wtconv_desc *d, void *workspace, int32_t *h_flag, void *stream) {
    wtconv_status st = validate_desc(d);
    if (st != WTCONV_OK) return st;
    if (!h_flag) return WTCONV_ERR_NULL;
    if (!workspace) {  // the scratch array built into the library (wtconv_backward_static)
        void *scratch = nullptr;
        if ((st = check_device()) != WTCONV_OK) return st;
        if ((st = static_scratch_for_current_device(&scratch)) != WTCONV_OK) return st;
        workspace = scratch;
    }
    if ((uintptr_t)workspace & (ALIGN - 1)) return WTCONV_ERR_ALIGNMENT;
    wtconv_desc d5;
    if (use_k3_embedding(d)) {  // the status words belong to the k = 5 path, behind the parameter tables
        workspace = (char *)workspace + embed_layout(d).inner;
        d5 = as_k5(d);
        d = &d5;
    }
    if (use_window_path(d) && d->L > 2)  // the carrier's whole-plane kernels keep the only status word of this path
        workspace = (char *)workspace + wt::window::ws_plan(d->B, d->C, d->H, d->W, d->L, (int)elem_bytes(d->dtype)).deep;
    else if (!use_plane_path(d)) {  // the tiled, window (L <= 2) and reference kernels wait for nothing and keep no status word
        *h_flag = 0;
        return WTCONV_OK;
    }
    // the status words open every workspace the plane kernels use: compare the timeout tag with the tag of the
    // last launch on the device, then fetch the result
    int *words = (int *)workspace;
    resolve_status_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(words);
    if (launch_status() != WTCONV_OK) return WTCONV_ERR_CUDA;
    return cudaMemcpyAsync(h_flag, words + wt::STATUS_RESOLVED, sizeof(int32_t), cudaMemcpyDeviceToHost,
                           (cudaStream_t)stream) == cudaSuccess
               ? WTCONV_OK
               : WTCONV_ERR_CUDA;
}

wtconv_status wtconv_backward_static(const wtconv_desc *d, const void *x, const void *grad_out, const float *w0,
                                     const float *s0, const float *b0, const float *wl, const float *sl, void *grad_x,
                                     float *grad_w0, float *grad_s0, float *grad_b0, float *grad_wl, float *grad_sl,
                                     void *stream) {
    wtconv_status st = validate_desc(d);
    if (st != WTCONV_OK) return st;
    if (bwd_ws_bytes(d) > (size_t)WTCONV_STATIC_SCRATCH_BYTES) return WTCONV_ERR_WORKSPACE;  // shape needs more scratch than is built in
    if ((st = check_device()) != WTCONV_OK) return st;
    void *scratch = nullptr;
    if ((st = static_scratch_for_current_device(&scratch)) != WTCONV_OK) return st;
    // wtconv_backward never depends on what it finds in its workspace, so the contents a previous call left in
    // the shared array do not matter.
    return wtconv_backward(d, x, grad_out, w0, s0, b0, wl, sl, grad_x, grad_w0, grad_s0, grad_b0, grad_wl, grad_sl,
                           scratch, (size_t)WTCONV_STATIC_SCRATCH_BYTES, stream);
}

}  // extern "C"
