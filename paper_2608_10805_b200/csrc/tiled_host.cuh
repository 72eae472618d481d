// Host side of the tiled kernels and of the shared epilogue: workspace plan and launches.  Included by the API
// translation unit (declarations, explicit-instantiation declarations) and by the per-dtype instantiation units.
#pragma once
#include "../../include/wtconv.h"

#include "common.cuh"
#include "tiled_kernels.cuh"

namespace wt {
namespace host {

using wt::host_half_up;

constexpr size_t ALIGN = 256;
inline size_t align_up(size_t v) { return (v + ALIGN - 1) / ALIGN * ALIGN; }
inline int cdiv(int a, int b) { return (a + b - 1) / b; }

struct Shapes {
    int Hs[WTCONV_MAX_LEVELS + 1], Ws[WTCONV_MAX_LEVELS + 1];
};

inline Shapes level_shapes(const wtconv_desc *d) {
    Shapes s;
    s.Hs[0] = d->H;
    s.Ws[0] = d->W;
    for (int l = 1; l <= WTCONV_MAX_LEVELS; ++l) {
        s.Hs[l] = host_half_up(s.Hs[l - 1]);
        s.Ws[l] = host_half_up(s.Ws[l - 1]);
    }
    return s;
}

inline size_t elem_bytes(int dtype) { return dtype == WTCONV_F32 ? 4 : 2; }

// ------------------------------------------------------------------ tiled-path workspace plan
struct TiledPlan {
    Shapes sh;
    int P, KK;
    // forward
    size_t z_off[WTCONV_MAX_LEVELS], xc_off[WTCONV_MAX_LEVELS];  // Z^l / dY^l and carrier X^l (index l-1)
    size_t fwd_bytes;
    // backward extras
    size_t gc_off[WTCONV_MAX_LEVELS];
    size_t part0_off, partl_off[WTCONV_MAX_LEVELS];
    int bsplit0, np0, bsplitl[WTCONV_MAX_LEVELS], npl[WTCONV_MAX_LEVELS];
    int tx0, ty0, txl[WTCONV_MAX_LEVELS], tyl[WTCONV_MAX_LEVELS];
    size_t bwd_bytes;
};

inline int pick_bsplit(int B, long long blocks_per_batchloop) {
    // enough blocks to fill 148 SMs several times over, but never more than one batch per block
    long long want = (4LL * 148 * 2 + blocks_per_batchloop - 1) / blocks_per_batchloop;
    if (want < 1) want = 1;
    if (want > B) want = B;
    return (int)want;
}

inline TiledPlan make_tiled_plan(const wtconv_desc *d) {
    TiledPlan p;
    p.sh = level_shapes(d);
    p.P = d->B * d->C;
    p.KK = d->k * d->k;
    size_t off = 0;
    for (int l = 1; l <= d->L; ++l) {
        size_t S = (size_t)p.sh.Hs[l] * p.sh.Ws[l];
        p.z_off[l - 1] = off;
        off = align_up(off + sizeof(float) * 4 * S * p.P);
        p.xc_off[l - 1] = off;
        if (l < d->L) off = align_up(off + sizeof(float) * S * p.P);
    }
    p.fwd_bytes = off;
    for (int l = 1; l < d->L; ++l) {
        size_t S = (size_t)p.sh.Hs[l] * p.sh.Ws[l];
        p.gc_off[l - 1] = off;
        off = align_up(off + sizeof(float) * S * p.P);
    }
    p.tx0 = cdiv(d->W, wt::tiled::STW);
    p.ty0 = cdiv(d->H, wt::tiled::STH);
    p.bsplit0 = pick_bsplit(d->B, (long long)p.tx0 * p.ty0 * d->C);
    p.np0 = p.tx0 * p.ty0 * p.bsplit0;
    p.part0_off = off;
    off = align_up(off + sizeof(float) * (size_t)d->C * p.np0 * (p.KK + 1));
    for (int l = 1; l <= d->L; ++l) {
        p.txl[l - 1] = cdiv(p.sh.Ws[l], wt::tiled::TW);
        p.tyl[l - 1] = cdiv(p.sh.Hs[l], wt::tiled::TH);
        p.bsplitl[l - 1] = pick_bsplit(d->B, (long long)p.txl[l - 1] * p.tyl[l - 1] * d->C);
        p.npl[l - 1] = p.txl[l - 1] * p.tyl[l - 1] * p.bsplitl[l - 1];
        p.partl_off[l - 1] = off;
        off = align_up(off + sizeof(float) * (size_t)d->C * p.npl[l - 1] * 4 * p.KK);
    }
    p.bwd_bytes = off;
    return p;
}

inline wtconv_status launch_status() { return cudaGetLastError() == cudaSuccess ? WTCONV_OK : WTCONV_ERR_CUDA; }

// ------------------------------------------------------------------ tiled forward / backward
template <typename T, int K>
wtconv_status tiled_forward(const wtconv_desc *d, const T *x, const float *w0, const float *s0, const float *b0,
                            const float *wl, const float *sl, T *out, char *ws, cudaStream_t st) {
    using namespace wt::tiled;
    TiledPlan pl = make_tiled_plan(d);
    wt::tiled::LevelPtrs lv = {};
    const int C = d->C, KK = K * K;
    for (int l = 1; l <= d->L; ++l) {
        const int Hp = pl.sh.Hs[l - 1], Wp = pl.sh.Ws[l - 1], Hl = pl.sh.Hs[l], Wl = pl.sh.Ws[l];
        float *Z = (float *)(ws + pl.z_off[l - 1]);
        float *Xl = (l < d->L) ? (float *)(ws + pl.xc_off[l - 1]) : nullptr;
        dim3 grid((unsigned)((size_t)pl.P * cdiv(Wl, TW) * cdiv(Hl, TH)));  // plane-major
        const float *wq = wl + (size_t)(l - 1) * C * 4 * KK, *sq = sl + (size_t)(l - 1) * C * 4;
        if (l == 1)
            level_fwd_kernel<T, K><<<grid, NTHREADS, 0, st>>>(x, Hp, Wp, Hl, Wl, C, wq, sq, Z, Xl);
        else
            level_fwd_kernel<float, K><<<grid, NTHREADS, 0, st>>>((const float *)(ws + pl.xc_off[l - 2]), Hp, Wp, Hl,
                                                                   Wl, C, wq, sq, Z, Xl);
        lv.z[l - 1] = Z;
        lv.Hl[l - 1] = Hl;
        lv.Wl[l - 1] = Wl;
    }
    dim3 grid((unsigned)((size_t)pl.P * cdiv(d->W, STW) * cdiv(d->H, STH)));  // plane-major
    synth_fwd_kernel<T, K><<<grid, NTHREADS, 0, st>>>(x, d->H, d->W, C, d->L, w0, s0, b0, lv, out);
    return launch_status();
}

inline wtconv_status launch_epilogue(const wtconv_desc *d, const wt::EpiloguePtrs &ep, const float *w0, const float *s0,
                              const float *b0, const float *wl, const float *sl, float *gw0, float *gs0, float *gb0,
                              float *gwl, float *gsl, cudaStream_t st) {
    const int KK = d->k * d->k;
    size_t smem = sizeof(double) * (KK + 1 + (size_t)d->L * 4 * KK);
    // an ordinary launch: it starts when the kernels that produced the partial sums have completed
    // released by the last block of the kernel before it (or at that kernel's completion); waits for it itself
    if (wt::launch_overlapped(wt::unfold_epilogue_kernel<0>, (unsigned)d->C, 128u, smem, st, d->C, d->k, d->L, ep, w0, s0, b0,
                              wl, sl, gw0, gs0, gb0, gwl, gsl) != cudaSuccess)
        return WTCONV_ERR_CUDA;
    return launch_status();
}

template <typename T, int K>
wtconv_status tiled_backward(const wtconv_desc *d, const T *x, const T *g, const float *w0, const float *s0,
                             const float *b0, const float *wl, const float *sl, T *gx, float *gw0, float *gs0,
                             float *gb0, float *gwl, float *gsl, char *ws, cudaStream_t st) {
    using namespace wt::tiled;
    TiledPlan pl = make_tiled_plan(d);
    wt::tiled::LevelPtrs lv = {};
    wt::EpiloguePtrs ep = {};
    const int C = d->C, KK = K * K;
    for (int l = 1; l <= d->L; ++l) {
        const int Hp = pl.sh.Hs[l - 1], Wp = pl.sh.Ws[l - 1], Hl = pl.sh.Hs[l], Wl = pl.sh.Ws[l];
        float *dY = (float *)(ws + pl.z_off[l - 1]);
        float *Xl = (l < d->L) ? (float *)(ws + pl.xc_off[l - 1]) : nullptr;
        float *Gl = (l < d->L) ? (float *)(ws + pl.gc_off[l - 1]) : nullptr;
        float *part = (float *)(ws + pl.partl_off[l - 1]);
        dim3 grid((unsigned)((size_t)C * pl.bsplitl[l - 1] * pl.txl[l - 1] * pl.tyl[l - 1]));  // (channel, part)-major
        const float *wq = wl + (size_t)(l - 1) * C * 4 * KK, *sq = sl + (size_t)(l - 1) * C * 4;
        constexpr size_t lsmem = level_bwd_smem_bytes<K>();  // above 48 KB for k = 7: opt in
        if (l == 1) {
            auto kern = level_bwd_kernel<T, K>;
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lsmem) != cudaSuccess)
                return WTCONV_ERR_CUDA;
            kern<<<grid, NTHREADS, lsmem, st>>>(x, g, Hp, Wp, Hl, Wl, d->B, C, pl.bsplitl[l - 1], wq, sq, dY, Xl, Gl, part);
        } else {
            auto kern = level_bwd_kernel<float, K>;
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lsmem) != cudaSuccess)
                return WTCONV_ERR_CUDA;
            kern<<<grid, NTHREADS, lsmem, st>>>((const float *)(ws + pl.xc_off[l - 2]), (const float *)(ws + pl.gc_off[l - 2]),
                                                Hp, Wp, Hl, Wl, d->B, C, pl.bsplitl[l - 1], wq, sq, dY, Xl, Gl, part);
        }
        lv.z[l - 1] = dY;
        lv.Hl[l - 1] = Hl;
        lv.Wl[l - 1] = Wl;
        ep.partl[l - 1] = part;
        ep.npl[l - 1] = pl.npl[l - 1];
    }
    float *part0 = (float *)(ws + pl.part0_off);
    dim3 grid((unsigned)((size_t)C * pl.bsplit0 * pl.tx0 * pl.ty0));  // (channel, part)-major
    synth_bwd_kernel<T, K><<<grid, NTHREADS, 0, st>>>(x, g, d->H, d->W, d->B, C, d->L, pl.bsplit0, w0, s0, lv, gx,
                                                      part0);
    ep.part0 = part0;
    ep.np0 = pl.np0;
    if (launch_status() != WTCONV_OK) return WTCONV_ERR_CUDA;
    return launch_epilogue(d, ep, w0, s0, b0, wl, sl, gw0, gs0, gb0, gwl, gsl, st);
}

#define WT_TILED_INSTANTIATE(T, K, EXTERN)                                                                              \
    EXTERN template wtconv_status tiled_forward<T, K>(const wtconv_desc *, const T *, const float *, const float *,      \
                                                      const float *, const float *, const float *, T *, char *,          \
                                                      cudaStream_t);                                                     \
    EXTERN template wtconv_status tiled_backward<T, K>(const wtconv_desc *, const T *, const T *, const float *,         \
                                                       const float *, const float *, const float *, const float *, T *,  \
                                                       float *, float *, float *, float *, float *, char *, cudaStream_t);

}  // namespace host
}  // namespace wt
