// Reference-style comparator: the WTConv layer as the chain of separate operators of Sec. 3.1, every intermediate
// tensor materialised in HBM, written as plain CUDA kernels (no library calls).  It exists to re-measure, on this
// GPU, what the fused kernels are compared with in the paper: the traffic model of Eq. 2 against Eq. 10 (Table 1),
// the latency ratios of Tables 2-3 and the cumulative ablation of Table 8.
//
// Forward chain (one launch per arrow):
//   for l = 1..L:  Y^l = A X^(l-1)            analysis          (Eq. 5; reads N_l, writes N_l)
//                  T^l = Y^l *dw W^l           depthwise conv    (reads N_l, writes N_l)
//                  U^l = s^l (.) T^l           scale pass        (reads N_l, writes N_l)
//                  X^l = [Y^l]_LL              slice             (reads N_l/4, writes N_l/4)
//   for l = L..1:  V^l = U^l, V^l_LL += R^(l+1)  add + concatenate (reads N_l + N_l/4, writes N_l)
//                  R^l = A^T V^l               synthesis         (reads N_l, writes N_l)
//   P = x *dw W^0;  Q = s^0 (.) (P + b);  out = Q + R^1        base conv, scale pass, add
// Ablation steps of Table 8 (cumulative; forward only): FUSED_ANALYSIS replaces analysis + conv + slice by one
// kernel per level that runs the butterfly on chip (Sec. 4.1); COLLAPSED_SYNTHESIS replaces the per-level add /
// concatenate / synthesis launches and the final add by the single closed-form pass of Proposition 2 (Sec. 4.2);
// adding scale folding (Sec. 4.3) on top gives the paper's fused design, which is this library's tiled path.
//
// Backward chain: the forward chain is run first (its intermediates are the autograd tape: Y^l, T^l and P), then
// every operator's gradient as its own launch: scale (two kernels: input gradient, and the per-channel reduction
// for the scale gradient), depthwise conv (input gradient = conv with the rotated kernel; weight gradient = tap-wise
// correlation, per-block partials finished in a fixed order), slice / concatenate / add (copies and adds), analysis
// (its adjoint is the synthesis) and synthesis (adjoint = analysis), Sec. 2.2.  The wtconv_backward call in this
// mode therefore costs one reference training step (forward + backward).
//
// Intermediates are fp32 whatever the activation type (the element counts of Eq. 2 are what is compared).
#pragma once
#include "tiled_host.cuh"

namespace wt {
namespace refchain {

constexpr int RT = 256;
inline unsigned nblk(size_t n, int per = RT) { size_t b = (n + per - 1) / per; return (unsigned)(b > 1u << 20 ? 1u << 20 : b); }

// ---------------------------------------------------------------- element-wise / copy kernels (grid-stride)
template <typename Tin>
__global__ void analysis_kernel(const Tin *__restrict__ X, int Hp, int Wp, int Hl, int Wl, size_t P, float *__restrict__ Y) {
    const size_t S = (size_t)Hl * Wl, n = P * S;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const size_t p = e / S;
        const int r = (int)(e - p * S), i = r / Wl, j = r - i * Wl;
        const Tin *q = X + p * Hp * Wp + (size_t)(2 * i) * Wp + 2 * j;
        const bool x1 = 2 * j + 1 < Wp, y1 = 2 * i + 1 < Hp;
        const float a = ldf(q), b = x1 ? ldf(q + 1) : 0.f, c = y1 ? ldf(q + Wp) : 0.f, d = (x1 && y1) ? ldf(q + Wp + 1) : 0.f;
        const Haar4 h = haar_butterfly(a, b, c, d);
        float *y = Y + p * 4 * S + r;
        y[0] = h.ll; y[S] = h.lh; y[2 * S] = h.hl; y[3 * S] = h.hh;
    }
}
// out = A^T V cropped to Hp x Wp (Appendix A sign table); V [P][4][Hl][Wl]
static __global__ void synthesis_kernel(const float *__restrict__ V, int Hp, int Wp, int Hl, int Wl, size_t P, float *__restrict__ R) {
    const size_t S = (size_t)Hl * Wl, SP = (size_t)Hp * Wp, n = P * SP;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const size_t p = e / SP;
        const int r = (int)(e - p * SP), y = r / Wp, x = r - y * Wp;
        const float *v = V + p * 4 * S + (size_t)(y >> 1) * Wl + (x >> 1);
        R[e] = synth_term(v[0], v[S], v[2 * S], v[3 * S], y & 1, x & 1, 0.5f);
    }
}
// dst[p][plane 0 of 4][...] etc.: copy the LL band of Y [P][4][S] to X [P][S]
static __global__ void slice_ll_kernel(const float *__restrict__ Y, size_t S, size_t P, float *__restrict__ X) {
    const size_t n = P * S;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const size_t p = e / S;
        X[e] = Y[p * 4 * S + (e - p * S)];
    }
}
// V = U with R added to the LL band (R may be null: deepest level) - the add and the concatenate of the reference
static __global__ void add_cat_kernel(const float *__restrict__ U, const float *__restrict__ Rn, size_t S, size_t P, float *__restrict__ V) {
    const size_t n = P * 4 * S;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const size_t p = e / (4 * S), r = e - p * 4 * S;
        float v = U[e];
        if (Rn && r < S) v += Rn[p * S + r];
        V[e] = v;
    }
}
// dst[e] = scale[channel(e)] * (src[e] + bias[channel]);  channel = (e / S) % nch
static __global__ void scale_kernel(const float *__restrict__ src, const float *__restrict__ s, const float *__restrict__ bias, size_t S, int nch,
                             size_t n, float *__restrict__ dst) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const int ch = (int)((e / S) % nch);
        dst[e] = __ldg(s + ch) * (src[e] + (bias ? __ldg(bias + ch) : 0.f));
    }
}
template <typename T>
__global__ void add_out_kernel(const float *__restrict__ Q, const float *__restrict__ R1, size_t n, T *__restrict__ out) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x)
        stf(out + e, Q[e] + (R1 ? R1[e] : 0.f));
}
// dst[p][band 0] += src[p]  (gradient of the slice into the LL band of dY)
static __global__ void add_ll_kernel(float *__restrict__ dY, const float *__restrict__ dX, size_t S, size_t P) {
    const size_t n = P * S;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const size_t p = e / S;
        dY[p * 4 * S + (e - p * S)] += dX[e];
    }
}
template <typename T>
__global__ void cast_in_kernel(const T *__restrict__ src, size_t n, float *__restrict__ dst) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) dst[e] = ldf(src + e);
}
template <typename T>
__global__ void add_cast_out_kernel(const float *__restrict__ a, const float *__restrict__ b, size_t n, T *__restrict__ dst) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x)
        stf(dst + e, a[e] + (b ? b[e] : 0.f));
}

// ---------------------------------------------------------------- depthwise convolution and its gradients
// out[p] = in[p] (*) w[p % nch] (cross-correlation, zero padding K/2); flip: kernel rotated by 180 degrees (input
// gradient).  64 x 64 pixel tiles in shared memory, a 4 x 4 output block per thread.
template <typename Tin, int K>
__global__ void __launch_bounds__(tiled::NTHREADS)
dwconv_kernel(const Tin *__restrict__ in, int H, int W, int nch, size_t P, const float *__restrict__ w, int flip, float *__restrict__ out) {
    using S = tiled::SynthTile<K>;
    __shared__ __align__(16) float Xs[S::XH][S::XP];
    __shared__ float Ws[K * K];
    const int ntx = tiled::tiles_of(W, tiled::STW), ntile = ntx * tiled::tiles_of(H, tiled::STH);
    const size_t p = blockIdx.x / ntile;
    const int tile = (int)(blockIdx.x - p * ntile), c = (int)(p % nch);
    const int x0 = (tile % ntx) * tiled::STW, y0 = (tile / ntx) * tiled::STH;
    tiled::stage_pixels<Tin, K, true>(in, p, P * H * W, H, W, y0, x0, Xs);
    if (threadIdx.x < K * K) Ws[threadIdx.x] = __ldg(w + (size_t)c * K * K + (flip ? K * K - 1 - threadIdx.x : threadIdx.x));
    __syncthreads();
    float wr[K * K];
#pragma unroll
    for (int t = 0; t < K * K; ++t) wr[t] = Ws[t];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int X0 = x0 + 4 * tx, Y0 = y0 + 4 * ty;
    if (X0 >= W || Y0 >= H) return;
    float acc[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) acc[r][cc] = 0.f;
    tiled::block_conv<K, S::XP>(Xs, 4 * ty, 4 * tx, wr, acc);
    tiled::store_block<float>(out + p * H * W, H, W, Y0, X0, acc);
}

// Weight gradient partials: part[ch][split][K*K] = sum over the block's batches and pixels of g * shifted in.
// grid = nch * bsplit * tiles; block (ch, split, tile) loops over images b = split, split + bsplit, ...
template <typename Tin, int K>
__global__ void __launch_bounds__(tiled::NTHREADS)
wgrad_kernel(const Tin *__restrict__ in, const float *__restrict__ g, int H, int W, int nch, int B, int bsplit,
             float *__restrict__ part /* [nch][bsplit * ntile][K*K] */) {
    using S = tiled::SynthTile<K>;
    constexpr int R = K / 2, KK = K * K;
    __shared__ __align__(16) float Xs[S::XH][S::XP];
    __shared__ __align__(16) float Gs[S::XH][S::XP];
    __shared__ float red[8][KK];
    const int ntx = tiled::tiles_of(W, tiled::STW), ntile = ntx * tiled::tiles_of(H, tiled::STH);
    const int cp = blockIdx.x / ntile, tile = blockIdx.x - cp * ntile;
    const int c = cp / bsplit, split = cp - c * bsplit;
    const int x0 = (tile % ntx) * tiled::STW, y0 = (tile / ntx) * tiled::STH;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool live = x0 + 4 * tx < W && y0 + 4 * ty < H;
    float gw[KK];
#pragma unroll
    for (int t = 0; t < KK; ++t) gw[t] = 0.f;
    const size_t total = (size_t)B * nch * H * W;
    for (int b = split; b < B; b += bsplit) {
        const size_t p = (size_t)b * nch + c;
        __syncthreads();
        tiled::stage_pixels<Tin, K, false>(in, p, total, H, W, y0, x0, Xs);
        tiled::stage_pixels<float, K, false>(g, p, total, H, W, y0, x0, Gs);
        __syncthreads();
        if (!live) continue;
        float d[4][4];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) d[r][cc] = Gs[4 * ty + R + r][4 * tx + R + cc];
        tiled::block_wgrad<K, S::XP>(Xs, 4 * ty, 4 * tx, d, gw);
    }
#pragma unroll
    for (int t = 0; t < KK; ++t) {
        const float v = tiled::warp_sum(gw[t]);
        if (lane == 0) red[warp][t] = v;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < KK; e += tiled::NTHREADS) {
        float v = 0.f;
#pragma unroll
        for (int wi = 0; wi < 8; ++wi) v += red[wi][e];
        part[((size_t)c * bsplit * ntile + (size_t)split * ntile + tile) * KK + e] = v;
    }
}
// per-channel dot product partials: part[ch][split] = sum_{b = split, split + bsplit, ..} sum_pixels a * (b_ ? b_ : 1)
static __global__ void __launch_bounds__(RT)
chdot_kernel(const float *__restrict__ a, const float *__restrict__ b_, size_t S, int nch, int B, int bsplit, float *__restrict__ part) {
    __shared__ float red[RT / 32];
    const int c = blockIdx.x / bsplit, split = blockIdx.x - c * bsplit;
    float acc = 0.f;
    for (int b = split; b < B; b += bsplit) {
        const size_t o = ((size_t)b * nch + c) * S;
        for (size_t e = threadIdx.x; e < S; e += RT) acc += a[o + e] * (b_ ? b_[o + e] : 1.f);
    }
    acc = tiled::warp_sum(acc);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        float v = 0.f;
        for (int i = 0; i < RT / 32; ++i) v += red[i];
        part[(size_t)c * bsplit + split] = v;
    }
}
// dst[i] = scale(i) * sum_j part[i][j]   (fixed order, fp64); scale from s[i / per] when given
static __global__ void finish_kernel(const float *__restrict__ part, int n, int nparts, const float *__restrict__ s, int per, float *__restrict__ dst) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    double a = 0.0;
    for (int j = 0; j < nparts; ++j) a += (double)part[(size_t)i * nparts + j];
    dst[i] = (float)(s ? (double)s[i / per] * a : a);
}

// out[c][t] = sum_j part[c][j][t]   (fixed order, fp64)
static __global__ void sum_parts_kernel(const float *__restrict__ part, int nch, int nparts, int KK, float *__restrict__ dst) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nch * KK) return;
    const int c = i / KK, t = i - c * KK;
    double a = 0.0;
    for (int j = 0; j < nparts; ++j) a += (double)part[((size_t)c * nparts + j) * KK + t];
    dst[i] = (float)a;
}
// bias terms of the base scale pass: ds0 += b sum(g), db0 = s0 sum(g)
static __global__ void bias_grads_kernel(const float *__restrict__ sumg, const float *__restrict__ s0, const float *__restrict__ b0, int C,
                                         float *__restrict__ gs0, float *__restrict__ gb0) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    gs0[c] += b0[c] * sumg[c];
    gb0[c] = s0[c] * sumg[c];
}
static __global__ void fill_kernel(float *__restrict__ p, float v, size_t n) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) p[e] = v;
}
// out = Q + sum_l (Proposition 2 term of U^l): the collapsed synthesis of the ablation, one pass over the output;
// a 4 x 4 pixel block per thread, 64 x 64 pixel tiles per block (the layout of the fused synthesis kernel)
template <typename T>
__global__ void __launch_bounds__(tiled::NTHREADS)
closed_form_add_kernel(const float *__restrict__ Q, int H, int W, int L, tiled::LevelPtrs lv, T *__restrict__ out) {
    const int ntx = tiled::tiles_of(W, tiled::STW), ntile = ntx * tiled::tiles_of(H, tiled::STH);
    const size_t p = blockIdx.x / ntile;
    const int tile = (int)(blockIdx.x - p * ntile);
    const int X0 = (tile % ntx) * tiled::STW + 4 * (threadIdx.x & 15), Y0 = (tile / ntx) * tiled::STH + 4 * (threadIdx.x >> 4);
    if (X0 >= W || Y0 >= H) return;
    const tiled::Z12 z = tiled::load_z12(lv, L, p, Y0, X0);
    float a[4][4];
    const float *q = Q + p * H * W;
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) a[r][c] = (Y0 + r < H && X0 + c < W) ? __ldg(q + (size_t)(Y0 + r) * W + X0 + c) : 0.f;
    tiled::block_synthesis(lv, L, p, Y0, X0, z, a);
    tiled::store_block<T>(out + p * H * W, H, W, Y0, X0, a);
}

// ---------------------------------------------------------------- workspace plan
struct RefPlan {
    host::Shapes sh;
    size_t P, N;
    // forward tape / intermediates, per level (index l - 1)
    size_t Y[WTCONV_MAX_LEVELS], T[WTCONV_MAX_LEVELS], U[WTCONV_MAX_LEVELS], X[WTCONV_MAX_LEVELS], V[WTCONV_MAX_LEVELS],
        Rl[WTCONV_MAX_LEVELS];
    size_t Pb, Qb, ones;  // base conv result, scaled base result, a vector of ones (ablation)
    size_t fwd_bytes;
    // backward
    size_t gf, dP, dxb, dV[WTCONV_MAX_LEVELS], dT[WTCONV_MAX_LEVELS], dY[WTCONV_MAX_LEVELS], dX[WTCONV_MAX_LEVELS];
    size_t part, gfold;  // partial sums (largest user), scale-gradient staging
    int bsplit;
    size_t bwd_bytes;
};

inline RefPlan make_plan(const wtconv_desc *d) {
    RefPlan p = {};
    p.sh = host::level_shapes(d);
    p.P = (size_t)d->B * d->C;
    p.N = p.P * d->H * d->W;
    size_t off = 0;
    auto take = [&](size_t floats) { size_t o = off; off = host::align_up(off + floats * sizeof(float)); return o; };
    for (int l = 1; l <= d->L; ++l) {
        const size_t S = (size_t)p.sh.Hs[l] * p.sh.Ws[l] * p.P, Sp = (size_t)p.sh.Hs[l - 1] * p.sh.Ws[l - 1] * p.P;
        p.Y[l - 1] = take(4 * S); p.T[l - 1] = take(4 * S); p.U[l - 1] = take(4 * S); p.X[l - 1] = take(S);
        p.V[l - 1] = take(4 * S); p.Rl[l - 1] = take(Sp);
    }
    p.Pb = take(p.N); p.Qb = take(p.N); p.ones = take((size_t)4 * d->C);
    p.fwd_bytes = off;
    p.gf = take(p.N); p.dP = take(p.N); p.dxb = take(p.N);
    for (int l = 1; l <= d->L; ++l) {
        const size_t S = (size_t)p.sh.Hs[l] * p.sh.Ws[l] * p.P, Sp = (size_t)p.sh.Hs[l - 1] * p.sh.Ws[l - 1] * p.P;
        p.dV[l - 1] = take(4 * S); p.dT[l - 1] = take(4 * S); p.dY[l - 1] = take(4 * S); p.dX[l - 1] = take(Sp);
    }
    p.bsplit = d->B < 8 ? d->B : 8;
    const int ntile0 = host::cdiv(d->W, tiled::STW) * host::cdiv(d->H, tiled::STH);
    p.part = take((size_t)4 * d->C * p.bsplit * ntile0 * d->k * d->k + 16);
    p.gfold = take((size_t)4 * d->C * d->k * d->k + 16);
    p.bwd_bytes = off;
    return p;
}

// ---------------------------------------------------------------- the chains
template <typename T, int K>
wtconv_status forward(const wtconv_desc *d, const T *x, const float *w0, const float *s0, const float *b0, const float *wl,
                      const float *sl, T *out, char *ws, cudaStream_t st) {
    const RefPlan pl = make_plan(d);
    const int C = d->C, L = d->L, KK = K * K;
    const size_t P = pl.P;
    auto F = [&](size_t o) { return reinterpret_cast<float *>(ws + o); };
    const bool fused_analysis = d->flags & WTCONV_FLAG_ABLATE_FUSED_ANALYSIS, collapsed = d->flags & WTCONV_FLAG_ABLATE_COLLAPSED_SYNTHESIS;
    // unit scales for the fused-analysis kernel (it folds whatever scale it is given): a vector of ones
    float *ones = F(pl.ones);
    if (fused_analysis) {
        fill_kernel<<<nblk((size_t)4 * C), RT, 0, st>>>(ones, 1.f, (size_t)4 * C);
    }
    for (int l = 1; l <= L; ++l) {
        const int Hp = pl.sh.Hs[l - 1], Wp = pl.sh.Ws[l - 1], Hl = pl.sh.Hs[l], Wl = pl.sh.Ws[l];
        const size_t S = (size_t)Hl * Wl;
        const float *wq = wl + (size_t)(l - 1) * C * 4 * KK, *sq = sl + (size_t)(l - 1) * C * 4;
        if (fused_analysis) {
            // one kernel: butterfly on chip + depthwise conv (un-scaled), raw LL carrier written alongside
            dim3 grid((unsigned)(P * host::cdiv(Wl, tiled::TW) * host::cdiv(Hl, tiled::TH)));
            float *Xl = l < L ? F(pl.X[l - 1]) : nullptr;
            if (l == 1) tiled::level_fwd_kernel<T, K><<<grid, tiled::NTHREADS, 0, st>>>(x, Hp, Wp, Hl, Wl, C, wq, ones, F(pl.T[0]), Xl);
            else tiled::level_fwd_kernel<float, K><<<grid, tiled::NTHREADS, 0, st>>>(F(pl.X[l - 2]), Hp, Wp, Hl, Wl, C, wq, ones, F(pl.T[l - 1]), Xl);
        } else {
            if (l == 1) analysis_kernel<T><<<nblk(P * S), RT, 0, st>>>(x, Hp, Wp, Hl, Wl, P, F(pl.Y[0]));
            else analysis_kernel<float><<<nblk(P * S), RT, 0, st>>>(F(pl.X[l - 2]), Hp, Wp, Hl, Wl, P, F(pl.Y[l - 1]));
            const unsigned nb = (unsigned)(P * 4 * host::cdiv(Wl, tiled::STW) * host::cdiv(Hl, tiled::STH));
            dwconv_kernel<float, K><<<nb, tiled::NTHREADS, 0, st>>>(F(pl.Y[l - 1]), Hl, Wl, 4 * C, P * 4, wq, 0, F(pl.T[l - 1]));
            if (l < L) slice_ll_kernel<<<nblk(P * S), RT, 0, st>>>(F(pl.Y[l - 1]), S, P, F(pl.X[l - 1]));
        }
        scale_kernel<<<nblk(P * 4 * S), RT, 0, st>>>(F(pl.T[l - 1]), sq, nullptr, S, 4 * C, P * 4 * S, F(pl.U[l - 1]));
    }
    const unsigned nb0 = (unsigned)(P * host::cdiv(d->W, tiled::STW) * host::cdiv(d->H, tiled::STH));
    dwconv_kernel<T, K><<<nb0, tiled::NTHREADS, 0, st>>>(x, d->H, d->W, C, P, w0, 0, F(pl.Pb));
    scale_kernel<<<nblk(pl.N), RT, 0, st>>>(F(pl.Pb), s0, b0, (size_t)d->H * d->W, C, pl.N, F(pl.Qb));
    if (collapsed) {
        // one pass: Proposition 2 over all U^l plus the base result, straight into out
        tiled::LevelPtrs lv = {};
        for (int l = 1; l <= L; ++l) { lv.z[l - 1] = F(pl.U[l - 1]); lv.Hl[l - 1] = pl.sh.Hs[l]; lv.Wl[l - 1] = pl.sh.Ws[l]; }
        closed_form_add_kernel<T><<<nb0, tiled::NTHREADS, 0, st>>>(F(pl.Qb), d->H, d->W, L, lv, out);
    } else {
        for (int l = L; l >= 1; --l) {
            const int Hp = pl.sh.Hs[l - 1], Wp = pl.sh.Ws[l - 1], Hl = pl.sh.Hs[l], Wl = pl.sh.Ws[l];
            const size_t S = (size_t)Hl * Wl;
            add_cat_kernel<<<nblk(P * 4 * S), RT, 0, st>>>(F(pl.U[l - 1]), l < L ? F(pl.Rl[l]) : nullptr, S, P, F(pl.V[l - 1]));
            synthesis_kernel<<<nblk(P * Hp * Wp), RT, 0, st>>>(F(pl.V[l - 1]), Hp, Wp, Hl, Wl, P, F(pl.Rl[l - 1]));
        }
        add_out_kernel<T><<<nblk(pl.N), RT, 0, st>>>(F(pl.Qb), L >= 1 ? F(pl.Rl[0]) : nullptr, pl.N, out);
    }
    return host::launch_status();
}

template <typename T, int K>
wtconv_status backward(const wtconv_desc *d, const T *x, const T *g, const float *w0, const float *s0, const float *b0,
                       const float *wl, const float *sl, T *gx, float *gw0, float *gs0, float *gb0, float *gwl, float *gsl,
                       char *ws, cudaStream_t st) {
    // the tape: run the plain forward chain (its result goes to gx, which is overwritten at the end)
    wtconv_desc df = *d;
    df.flags &= ~(WTCONV_FLAG_ABLATE_FUSED_ANALYSIS | WTCONV_FLAG_ABLATE_COLLAPSED_SYNTHESIS);
    wtconv_status stt = forward<T, K>(&df, x, w0, s0, b0, wl, sl, gx, ws, st);
    if (stt != WTCONV_OK) return stt;
    const RefPlan pl = make_plan(d);
    const int C = d->C, L = d->L, KK = K * K, B = d->B, bs = pl.bsplit;
    const size_t P = pl.P, HW = (size_t)d->H * d->W;
    auto F = [&](size_t o) { return reinterpret_cast<float *>(ws + o); };
    float *part = F(pl.part), *gfold = F(pl.gfold);
    // out = Q + R^1: both get g.  Scale pass Q = s0 (P + b): dP = s0 g; ds0 = sum g (P + b); db0 = s0 sum g
    cast_in_kernel<T><<<nblk(pl.N), RT, 0, st>>>(g, pl.N, F(pl.gf));
    scale_kernel<<<nblk(pl.N), RT, 0, st>>>(F(pl.gf), s0, nullptr, HW, C, pl.N, F(pl.dP));
    chdot_kernel<<<C * bs, RT, 0, st>>>(F(pl.gf), F(pl.Pb), HW, C, B, bs, part);
    finish_kernel<<<host::cdiv(C, 128), 128, 0, st>>>(part, C, bs, nullptr, 1, gs0);
    if (b0) {
        chdot_kernel<<<C * bs, RT, 0, st>>>(F(pl.gf), nullptr, HW, C, B, bs, part);
        finish_kernel<<<host::cdiv(C, 128), 128, 0, st>>>(part, C, bs, nullptr, 1, gfold);       // sum g
        bias_grads_kernel<<<host::cdiv(C, 128), 128, 0, st>>>(gfold, s0, b0, C, gs0, gb0);   // ds0 += b sum g; db0 = s0 sum g
    }
    // base conv: input gradient and weight gradient
    const int ntile0 = host::cdiv(d->W, tiled::STW) * host::cdiv(d->H, tiled::STH);
    dwconv_kernel<float, K><<<(unsigned)(P * ntile0), tiled::NTHREADS, 0, st>>>(F(pl.dP), d->H, d->W, C, P, w0, 1, F(pl.dxb));
    wgrad_kernel<T, K><<<(unsigned)(C * bs * ntile0), tiled::NTHREADS, 0, st>>>(x, F(pl.dP), d->H, d->W, C, B, bs, part);
    sum_parts_kernel<<<host::cdiv(C * KK, 128), 128, 0, st>>>(part, C, bs * ntile0, KK, gw0);
    // downward: dR^1 = g; dV^l = A dR^l (adjoint of the synthesis); dR^(l+1) = dV^l_LL; dU^l = dV^l
    for (int l = 1; l <= L; ++l) {
        const int Hp = pl.sh.Hs[l - 1], Wp = pl.sh.Ws[l - 1], Hl = pl.sh.Hs[l], Wl = pl.sh.Ws[l];
        const size_t S = (size_t)Hl * Wl;
        if (l == 1) analysis_kernel<float><<<nblk(P * S), RT, 0, st>>>(F(pl.gf), Hp, Wp, Hl, Wl, P, F(pl.dV[0]));
        else {
            slice_ll_kernel<<<nblk(P * (size_t)Hp * Wp), RT, 0, st>>>(F(pl.dV[l - 2]), (size_t)Hp * Wp, P, F(pl.dX[l - 1]));  // dR^l (scratch)
            analysis_kernel<float><<<nblk(P * S), RT, 0, st>>>(F(pl.dX[l - 1]), Hp, Wp, Hl, Wl, P, F(pl.dV[l - 1]));
        }
    }
    // upward: scale pass and conv gradients per level, slice gradient into LL, analysis adjoint (= synthesis)
    for (int l = L; l >= 1; --l) {
        const int Hp = pl.sh.Hs[l - 1], Wp = pl.sh.Ws[l - 1], Hl = pl.sh.Hs[l], Wl = pl.sh.Ws[l];
        const size_t S = (size_t)Hl * Wl;
        const float *wq = wl + (size_t)(l - 1) * C * 4 * KK, *sq = sl + (size_t)(l - 1) * C * 4;
        float *gwq = gwl + (size_t)(l - 1) * C * 4 * KK, *gsq = gsl + (size_t)(l - 1) * C * 4;
        scale_kernel<<<nblk(P * 4 * S), RT, 0, st>>>(F(pl.dV[l - 1]), sq, nullptr, S, 4 * C, P * 4 * S, F(pl.dT[l - 1]));
        chdot_kernel<<<4 * C * bs, RT, 0, st>>>(F(pl.dV[l - 1]), F(pl.T[l - 1]), S, 4 * C, B, bs, part);
        finish_kernel<<<host::cdiv(4 * C, 128), 128, 0, st>>>(part, 4 * C, bs, nullptr, 1, gsq);
        const int ntl = host::cdiv(Wl, tiled::STW) * host::cdiv(Hl, tiled::STH);
        dwconv_kernel<float, K><<<(unsigned)(P * 4 * ntl), tiled::NTHREADS, 0, st>>>(F(pl.dT[l - 1]), Hl, Wl, 4 * C, P * 4, wq, 1, F(pl.dY[l - 1]));
        wgrad_kernel<float, K><<<(unsigned)(4 * C * bs * ntl), tiled::NTHREADS, 0, st>>>(F(pl.Y[l - 1]), F(pl.dT[l - 1]), Hl, Wl, 4 * C, B, bs, part);
        sum_parts_kernel<<<host::cdiv(4 * C * KK, 128), 128, 0, st>>>(part, 4 * C, bs * ntl, KK, gwq);
        if (l < L) add_ll_kernel<<<nblk(P * S), RT, 0, st>>>(F(pl.dY[l - 1]), F(pl.dX[l]), S, P);  // slice: X^l = Y^l_LL
        synthesis_kernel<<<nblk(P * (size_t)Hp * Wp), RT, 0, st>>>(F(pl.dY[l - 1]), Hp, Wp, Hl, Wl, P, F(pl.dX[l - 1]));
    }
    add_cast_out_kernel<T><<<nblk(pl.N), RT, 0, st>>>(F(pl.dxb), L >= 1 ? F(pl.dX[0]) : nullptr, pl.N, gx);
    return host::launch_status();
}

#define WT_REFCHAIN_INSTANTIATE(T, K, EXTERN)                                                                             \
    EXTERN template wtconv_status forward<T, K>(const wtconv_desc *, const T *, const float *, const float *, const float *, \
                                                const float *, const float *, T *, char *, cudaStream_t);                \
    EXTERN template wtconv_status backward<T, K>(const wtconv_desc *, const T *, const T *, const float *, const float *,  \
                                                 const float *, const float *, const float *, T *, float *, float *,     \
                                                 float *, float *, float *, char *, cudaStream_t);

}  // namespace refchain
}  // namespace wt
