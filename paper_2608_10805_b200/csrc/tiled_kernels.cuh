// Tiled WTConv kernels: one launch per decomposition level plus one synthesis launch, for
// planes of any size.  Subband tensors Z^l (forward) / dL/dY^l (backward) and the raw low-pass
// carriers live in the caller's workspace in fp32; the analysis butterfly (Eq. 5) is recomputed
// on chip per tile with a coefficient-space halo of R = k/2 (Sec. 4.1), scales are folded into
// the weights when they are loaded (Eq. 8), and the synthesis is the single bit-indexed pass of
// Proposition 2 with the base convolution fused into the final store (Sec. 4.2).
//
// Thread layout of every kernel here: 256 threads = 8 warps; lane = column inside a 32-wide
// tile.  In the level kernels warp w owns subband (w & 3) and the upper or lower half (w >> 2)
// of a 16-row coefficient tile, so a thread only ever sees one subband and can keep that
// subband's k*k weights and k*k weight-gradient accumulators in registers across a whole
// batch loop.
#pragma once
#include "common.cuh"

namespace wt {
namespace tiled {

constexpr int TW = 32;       // tile width (coefficients or pixels)
constexpr int TH = 16;       // tile height
constexpr int NTHREADS = 256;
constexpr int ROWS_PER_THREAD = 8;  // level kernels: TH / 2 halves

// Stage the four subbands of the level grid (Hl x Wl) around tile origin (i0, j0), with halo R,
// from the previous carrier plane `xp` (Hp x Wp).  Positions outside the level grid are zero
// (the depthwise conv's zero padding); pixels outside the carrier are zero (odd-size padding).
template <typename Tin, int K>
__device__ __forceinline__ void stage_subbands(const Tin *__restrict__ xp, int Hp, int Wp, int Hl, int Wl, int i0,
                                               int j0, float (*Ys)[TH + K - 1][TW + K] /* [4] */) {
    constexpr int R = K / 2, SW = TW + 2 * R, SH = TH + 2 * R;
    for (int e = threadIdx.x; e < SH * SW; e += NTHREADS) {
        int li = e / SW, lj = e - li * SW;
        int i = i0 + li - R, j = j0 + lj - R;
        Haar4 h = {0.f, 0.f, 0.f, 0.f};
        if (i >= 0 && i < Hl && j >= 0 && j < Wl) {
            int y = 2 * i, x = 2 * j;
            bool x1 = (x + 1 < Wp), y1 = (y + 1 < Hp);
            const Tin *q = xp + (size_t)y * Wp + x;
            float a = ldf(q);
            float b = x1 ? ldf(q + 1) : 0.f;
            float c = y1 ? ldf(q + Wp) : 0.f;
            float d = (x1 && y1) ? ldf(q + Wp + 1) : 0.f;
            h = haar_butterfly(a, b, c, d);
        }
        Ys[0][li][lj] = h.ll;
        Ys[1][li][lj] = h.lh;
        Ys[2][li][lj] = h.hl;
        Ys[3][li][lj] = h.hh;
    }
}

// Column conv: 8 vertically adjacent outputs at column `lx` (tile coords, halo-shifted), rows
// r0..r0+7, of S (one subband, with halo) against register weights w[K*K].
template <int K>
__device__ __forceinline__ void column_conv(const float (*S)[TW + K], int r0, int lx, const float *w, float *acc) {
#pragma unroll
    for (int r = 0; r < ROWS_PER_THREAD; ++r) acc[r] = 0.f;
#pragma unroll
    for (int rr = 0; rr < ROWS_PER_THREAD + K - 1; ++rr) {
        float in[K];
#pragma unroll
        for (int v = 0; v < K; ++v) in[v] = S[r0 + rr][lx + v];
#pragma unroll
        for (int u = 0; u < K; ++u) {
            int r = rr - u;
            if (r >= 0 && r < ROWS_PER_THREAD) {
#pragma unroll
                for (int v = 0; v < K; ++v) acc[r] = fmaf(w[u * K + v], in[v], acc[r]);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Forward level kernel: Z^l = Wfold^l (*) A(X^(l-1)), X^l = raw LL.   grid (P, tiles_x, tiles_y)
// ---------------------------------------------------------------------------------------------
template <typename Tin, int K>
__global__ void __launch_bounds__(NTHREADS)
level_fwd_kernel(const Tin *__restrict__ Xprev, int Hp, int Wp, int Hl, int Wl, int C,
                 const float *__restrict__ w /* [C][4][K][K] */, const float *__restrict__ s /* [C][4] */,
                 float *__restrict__ Z /* [P][4][Hl][Wl] */, float *__restrict__ Xl /* [P][Hl][Wl] or null */) {
    constexpr int R = K / 2;
    __shared__ float Ys[4][TH + K - 1][TW + K];
    const int p = blockIdx.x, c = p % C;
    const int j0 = blockIdx.y * TW, i0 = blockIdx.z * TH;
    stage_subbands<Tin, K>(Xprev + (size_t)p * Hp * Wp, Hp, Wp, Hl, Wl, i0, j0, Ys);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = warp & 3, r0 = (warp >> 2) * ROWS_PER_THREAD;
    float wr[K * K];
    const float sc = __ldg(s + c * 4 + sub);
#pragma unroll
    for (int t = 0; t < K * K; ++t) wr[t] = sc * __ldg(w + ((size_t)c * 4 + sub) * K * K + t);  // Eq. 8
    __syncthreads();
    float acc[ROWS_PER_THREAD];
    column_conv<K>(Ys[sub], r0, lane, wr, acc);
    const int j = j0 + lane;
    if (j < Wl) {
        float *zp = Z + ((size_t)p * 4 + sub) * Hl * Wl;
#pragma unroll
        for (int r = 0; r < ROWS_PER_THREAD; ++r) {
            int i = i0 + r0 + r;
            if (i < Hl) {
                zp[(size_t)i * Wl + j] = acc[r];
                if (sub == 0 && Xl) Xl[((size_t)p * Hl + i) * Wl + j] = Ys[0][r0 + r + R][lane + R];
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Forward synthesis kernel: out = Wfold^0 (*) x + bfold + sum_l (Prop. 2 term of Z^l).
// grid (P, tiles_x, tiles_y); thread = column lane, rows 2*warp, 2*warp+1 of the tile.
// ---------------------------------------------------------------------------------------------
struct LevelPtrs {
    const float *z[8];  // per level l (index l-1): [P][4][Hl][Wl]
    int Hl[8], Wl[8];
};

template <typename T, int K>
__global__ void __launch_bounds__(NTHREADS)
synth_fwd_kernel(const T *__restrict__ x, int H, int W, int C, int L, const float *__restrict__ w0,
                 const float *__restrict__ s0, const float *__restrict__ b0, LevelPtrs lv, T *__restrict__ out) {
    constexpr int R = K / 2, SW = TW + 2 * R, SH = TH + 2 * R;
    __shared__ float Xs[SH][SW + 1];
    const int p = blockIdx.x, c = p % C;
    const int x0 = blockIdx.y * TW, y0 = blockIdx.z * TH;
    const T *xp = x + (size_t)p * H * W;
    for (int e = threadIdx.x; e < SH * SW; e += NTHREADS) {
        int ly = e / SW, lx = e - ly * SW;
        int yy = y0 + ly - R, xx = x0 + lx - R;
        Xs[ly][lx] = (yy >= 0 && yy < H && xx >= 0 && xx < W) ? ldf(xp + (size_t)yy * W + xx) : 0.f;
    }
    float wr[K * K];
    const float sc = __ldg(s0 + c);
#pragma unroll
    for (int t = 0; t < K * K; ++t) wr[t] = sc * __ldg(w0 + (size_t)c * K * K + t);
    const float bias = b0 ? sc * __ldg(b0 + c) : 0.f;
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int xx = x0 + lane;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int ly = warp * 2 + r, yy = y0 + ly;
        if (yy >= H || xx >= W) continue;
        float acc = bias;
#pragma unroll
        for (int u = 0; u < K; ++u)
#pragma unroll
            for (int v = 0; v < K; ++v) acc = fmaf(wr[u * K + v], Xs[ly + u][lane + v], acc);
        float scale = 1.f;
        for (int l = 1; l <= L; ++l) {
            scale *= 0.5f;
            const int Hl = lv.Hl[l - 1], Wl = lv.Wl[l - 1];
            const size_t S = (size_t)Hl * Wl;
            const float *zp = lv.z[l - 1] + (size_t)p * 4 * S + (size_t)(yy >> l) * Wl + (xx >> l);
            acc += synth_term(__ldg(zp), __ldg(zp + S), __ldg(zp + 2 * S), __ldg(zp + 3 * S), (yy >> (l - 1)) & 1,
                              (xx >> (l - 1)) & 1, scale);
        }
        stf(out + (size_t)p * H * W + (size_t)yy * W + xx, acc);
    }
}

// Sum v over the 32 lanes; result valid in lane 0.
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;
}

// ---------------------------------------------------------------------------------------------
// Backward level kernel.  For the level-l grid:
//   D^l = A(G^(l-1)), Y^l = A(X^(l-1))            (staged with halo; Sec. 2.2: d/dR through synthesis is analysis)
//   dY^l = flip(Wfold^l) (*) D^l                  -> workspace
//   dWfold^l[u,v] += sum D^l[i,j] Y^l[i+u-R, j+v-R]   (register accumulators, batch loop, one partial per block)
//   carriers X^l = Y^l_LL, G^l = D^l_LL           -> workspace (if not the deepest level)
// grid (C * bsplit, tiles_x, tiles_y): block x = c * bsplit + part loops over batches
// b = part, part + bsplit, ...  Partials: [C][nparts][4][K*K], nparts = tiles_x*tiles_y*bsplit.
// ---------------------------------------------------------------------------------------------
template <typename Tin, int K>
__global__ void __launch_bounds__(NTHREADS)
level_bwd_kernel(const Tin *__restrict__ Xprev, const Tin *__restrict__ Gprev, int Hp, int Wp, int Hl, int Wl, int B,
                 int C, int bsplit, const float *__restrict__ w, const float *__restrict__ s,
                 float *__restrict__ dY /* [P][4][Hl][Wl] */, float *__restrict__ Xl, float *__restrict__ Gl,
                 float *__restrict__ partials) {
    constexpr int R = K / 2, KK = K * K;
    __shared__ float Ys[4][TH + K - 1][TW + K];
    __shared__ float Ds[4][TH + K - 1][TW + K];
    __shared__ float red[8][KK];
    const int c = blockIdx.x / bsplit, part = blockIdx.x - c * bsplit;
    const int j0 = blockIdx.y * TW, i0 = blockIdx.z * TH;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = warp & 3, r0 = (warp >> 2) * ROWS_PER_THREAD;
    float wf[KK], gw[KK];
    const float sc = __ldg(s + c * 4 + sub);
#pragma unroll
    for (int t = 0; t < KK; ++t) {
        wf[t] = sc * __ldg(w + ((size_t)c * 4 + sub) * KK + (KK - 1 - t));  // folded and rotated by 180 degrees
        gw[t] = 0.f;
    }
    const int j = j0 + lane;
    for (int b = part; b < B; b += bsplit) {
        const size_t p = (size_t)b * C + c;
        __syncthreads();
        stage_subbands<Tin, K>(Xprev + p * Hp * Wp, Hp, Wp, Hl, Wl, i0, j0, Ys);
        stage_subbands<Tin, K>(Gprev + p * Hp * Wp, Hp, Wp, Hl, Wl, i0, j0, Ds);
        __syncthreads();
        float acc[ROWS_PER_THREAD];
        column_conv<K>(Ds[sub], r0, lane, wf, acc);
        // weight gradient: this thread's 8 D values against the shifted Y window
        float dcol[ROWS_PER_THREAD];
#pragma unroll
        for (int r = 0; r < ROWS_PER_THREAD; ++r) dcol[r] = Ds[sub][r0 + r + R][lane + R];
#pragma unroll
        for (int rr = 0; rr < ROWS_PER_THREAD + K - 1; ++rr) {
            float in[K];
#pragma unroll
            for (int v = 0; v < K; ++v) in[v] = Ys[sub][r0 + rr][lane + v];
#pragma unroll
            for (int u = 0; u < K; ++u) {
                int r = rr - u;
                if (r >= 0 && r < ROWS_PER_THREAD) {
#pragma unroll
                    for (int v = 0; v < K; ++v) gw[u * K + v] = fmaf(dcol[r], in[v], gw[u * K + v]);
                }
            }
        }
        if (j < Wl) {
            float *yp = dY + (p * 4 + sub) * Hl * Wl;
#pragma unroll
            for (int r = 0; r < ROWS_PER_THREAD; ++r) {
                int i = i0 + r0 + r;
                if (i < Hl) {
                    yp[(size_t)i * Wl + j] = acc[r];
                    if (sub == 0 && Xl) {
                        Xl[(p * Hl + i) * Wl + j] = Ys[0][r0 + r + R][lane + R];
                        Gl[(p * Hl + i) * Wl + j] = Ds[0][r0 + r + R][lane + R];
                    }
                }
            }
        }
    }
    // block reduction: lanes by shuffle, the two row halves of a subband through shared memory
#pragma unroll
    for (int t = 0; t < KK; ++t) {
        float v = warp_sum(gw[t]);
        if (lane == 0) red[warp][t] = v;
    }
    __syncthreads();
    const int nparts = gridDim.y * gridDim.z * bsplit;
    const int pidx = (blockIdx.z * gridDim.y + blockIdx.y) * bsplit + part;
    for (int e = threadIdx.x; e < 4 * KK; e += NTHREADS) {
        int sb = e / KK, t = e - sb * KK;
        partials[(((size_t)c * nparts + pidx) * 4 + sb) * KK + t] = red[sb][t] + red[sb + 4][t];
    }
}

// ---------------------------------------------------------------------------------------------
// Backward synthesis kernel:
//   dx = flip(Wfold^0) (*) G + sum_l (Prop. 2 term of dY^l)       (Sec. 2.2 + Prop. 2)
//   dWfold^0[u,v] += sum G[y,x] x[y+u-R, x+v-R],  dbfold += sum G
// grid (C * bsplit, tiles_x, tiles_y).  Partials: [C][nparts][K*K + 1].
// ---------------------------------------------------------------------------------------------
template <typename T, int K>
__global__ void __launch_bounds__(NTHREADS)
synth_bwd_kernel(const T *__restrict__ x, const T *__restrict__ g, int H, int W, int B, int C, int L, int bsplit,
                 const float *__restrict__ w0, const float *__restrict__ s0, LevelPtrs lv, T *__restrict__ dx,
                 float *__restrict__ partials) {
    constexpr int R = K / 2, SW = TW + 2 * R, SH = TH + 2 * R, KK = K * K;
    __shared__ float Xs[SH][SW + 1];
    __shared__ float Gs[SH][SW + 1];
    __shared__ float red[8][KK + 1];
    const int c = blockIdx.x / bsplit, part = blockIdx.x - c * bsplit;
    const int x0 = blockIdx.y * TW, y0 = blockIdx.z * TH;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float wf[KK], gw[KK], gb = 0.f;
    const float sc = __ldg(s0 + c);
#pragma unroll
    for (int t = 0; t < KK; ++t) {
        wf[t] = sc * __ldg(w0 + (size_t)c * KK + (KK - 1 - t));
        gw[t] = 0.f;
    }
    const int xx = x0 + lane;
    for (int b = part; b < B; b += bsplit) {
        const size_t p = (size_t)b * C + c;
        const T *xp = x + p * H * W, *gp = g + p * H * W;
        __syncthreads();
        for (int e = threadIdx.x; e < SH * SW; e += NTHREADS) {
            int ly = e / SW, lx = e - ly * SW;
            int yy = y0 + ly - R, xc = x0 + lx - R;
            bool in = (yy >= 0 && yy < H && xc >= 0 && xc < W);
            Xs[ly][lx] = in ? ldf(xp + (size_t)yy * W + xc) : 0.f;
            Gs[ly][lx] = in ? ldf(gp + (size_t)yy * W + xc) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int ly = warp * 2 + r, yy = y0 + ly;
            if (yy >= H || xx >= W) continue;
            float acc = 0.f;
            const float gv = Gs[ly + R][lane + R];
            gb += gv;
#pragma unroll
            for (int u = 0; u < K; ++u)
#pragma unroll
                for (int v = 0; v < K; ++v) {
                    acc = fmaf(wf[u * K + v], Gs[ly + u][lane + v], acc);
                    gw[u * K + v] = fmaf(gv, Xs[ly + u][lane + v], gw[u * K + v]);
                }
            float scale = 1.f;
            for (int l = 1; l <= L; ++l) {
                scale *= 0.5f;
                const int Hl = lv.Hl[l - 1], Wl = lv.Wl[l - 1];
                const size_t S = (size_t)Hl * Wl;
                const float *zp = lv.z[l - 1] + p * 4 * S + (size_t)(yy >> l) * Wl + (xx >> l);
                acc += synth_term(__ldg(zp), __ldg(zp + S), __ldg(zp + 2 * S), __ldg(zp + 3 * S), (yy >> (l - 1)) & 1,
                                  (xx >> (l - 1)) & 1, scale);
            }
            stf(dx + p * H * W + (size_t)yy * W + xx, acc);
        }
    }
#pragma unroll
    for (int t = 0; t < KK; ++t) {
        float v = warp_sum(gw[t]);
        if (lane == 0) red[warp][t] = v;
    }
    {
        float v = warp_sum(gb);
        if (lane == 0) red[warp][KK] = v;
    }
    __syncthreads();
    const int nparts = gridDim.y * gridDim.z * bsplit;
    const int pidx = (blockIdx.z * gridDim.y + blockIdx.y) * bsplit + part;
    for (int t = threadIdx.x; t < KK + 1; t += NTHREADS) {
        float v = 0.f;
#pragma unroll
        for (int wi = 0; wi < 8; ++wi) v += red[wi][t];
        partials[((size_t)c * nparts + pidx) * (KK + 1) + t] = v;
    }
}

}  // namespace tiled

// ---------------------------------------------------------------------------------------------
// Parameter-gradient epilogue (Eq. 9), shared by every kernel family.  One block per channel:
// sums the per-block partials in a fixed order in fp64 (deterministic), then un-folds:
//   dW = s dWfold,  db = s dbfold,  ds = <dWfold, W> (+ dbfold b on the base path).
// Base partials [C][np0][KK+1]; level-l partials [C][npl[l]][4][KK].
// ---------------------------------------------------------------------------------------------
struct EpiloguePtrs {
    const float *part0;
    int np0;
    const float *partl[8];
    int npl[8];
};

__global__ void __launch_bounds__(128)
unfold_epilogue_kernel(int C, int K, int L, EpiloguePtrs ep, const float *__restrict__ w0,
                       const float *__restrict__ s0, const float *__restrict__ b0, const float *__restrict__ wl,
                       const float *__restrict__ sl, float *__restrict__ dw0, float *__restrict__ ds0,
                       float *__restrict__ db0, float *__restrict__ dwl, float *__restrict__ dsl) {
    extern __shared__ double folded[];  // [KK+1] base, then [L][4][KK]
    const int c = blockIdx.x, KK = K * K;
    const int n0 = KK + 1, nl = 4 * KK;
    for (int e = threadIdx.x; e < n0 + L * nl; e += blockDim.x) {
        double acc = 0.0;
        if (e < n0) {
            const float *q = ep.part0 + (size_t)c * ep.np0 * n0 + e;
            for (int i = 0; i < ep.np0; ++i) acc += (double)q[(size_t)i * n0];
        } else {
            int l = (e - n0) / nl, t = (e - n0) - l * nl;
            const float *q = ep.partl[l] + (size_t)c * ep.npl[l] * nl + t;
            for (int i = 0; i < ep.npl[l]; ++i) acc += (double)q[(size_t)i * nl];
        }
        folded[e] = acc;
    }
    __syncthreads();
    const double s0c = (double)s0[c];
    for (int t = threadIdx.x; t < KK; t += blockDim.x) dw0[(size_t)c * KK + t] = (float)(s0c * folded[t]);
    for (int e = threadIdx.x; e < L * nl; e += blockDim.x) {
        int l = e / nl, r = e - l * nl, sub = r / KK;
        dwl[((size_t)l * C + c) * nl + r] = (float)((double)sl[((size_t)l * C + c) * 4 + sub] * folded[n0 + e]);
    }
    if (threadIdx.x == 0) {
        double a = 0.0;
        for (int t = 0; t < KK; ++t) a += folded[t] * (double)w0[(size_t)c * KK + t];
        if (b0) {
            a += folded[KK] * (double)b0[c];
            db0[c] = (float)(s0c * folded[KK]);
        }
        ds0[c] = (float)a;
    }
    for (int e = threadIdx.x + 1; e < 1 + L * 4; e += blockDim.x) {
        int l = (e - 1) / 4, sub = (e - 1) & 3;
        double a = 0.0;
        const float *wq = wl + (((size_t)l * C + c) * 4 + sub) * KK;
        for (int t = 0; t < KK; ++t) a += folded[n0 + l * nl + sub * KK + t] * (double)wq[t];
        dsl[((size_t)l * C + c) * 4 + sub] = (float)a;
    }
}

}  // namespace wt
