// Tiled WTConv kernels: one launch per decomposition level plus one synthesis launch, for
// planes of any size.  Subband tensors Z^l (forward) / dL/dY^l (backward) and the raw low-pass
// carriers live in the caller's workspace in fp32; the analysis butterfly (Eq. 5) is recomputed
// on chip per tile with a coefficient-space halo of R = k/2 (Sec. 4.1), scales are folded into
// the weights when they are loaded (Eq. 8), and the synthesis is the single bit-indexed pass of
// Proposition 2 with the base convolution fused into the final store (Sec. 4.2).
//
// Thread layout of every kernel here: 256 threads, a 4 x 4 block of outputs per thread (register tile, window
// rows read as aligned float4 loads).  In the level kernels 64 threads own each subband of a 32 x 32
// coefficient tile, so a thread only ever sees one subband and can keep that subband's k*k weights and k*k
// weight-gradient accumulators in registers across a whole batch loop; the synthesis kernels work on
// 64 x 64 pixel tiles.
#pragma once
#include "common.cuh"

namespace wt {
namespace tiled {

constexpr int TW = 32;       // level kernels: tile width in coefficients
constexpr int TH = 32;       // level kernels: tile height in coefficients
constexpr int NTHREADS = 256;

// Grids are one-dimensional and plane-major: the tiles of one plane (or of one channel's batch slice) are
// neighbours in launch order, so the halo a tile shares with the next one is still in L2 when that one runs.
__host__ __device__ inline int tiles_of(int n, int t) { return (n + t - 1) / t; }

// Shared-memory tile of TWc x THc outputs with halo R = K/2.  Every thread computes a 4 x 4 output block; its
// window starts at a multiple of four floats, so window rows are read as NQ aligned float4 loads, and the pitch
// P leaves room for the last thread's last load.
template <int K, int TWc, int THc> struct TileDims {
    static constexpr int R = K / 2;
    static constexpr int NQ = (4 + K - 1 + 3) / 4;
    static constexpr int W = TWc + 2 * R, H = THc + 2 * R;
    static constexpr int P = TWc - 4 + 4 * NQ;
};
template <int K> using LevelTile = TileDims<K, TW, TH>;

// Four consecutive activations as floats (16-byte / 8-byte aligned vector load).
__device__ __forceinline__ float4 load_vec4(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }
__device__ __forceinline__ float4 load_vec4(const __half *p) {
    const uint2 q = __ldg(reinterpret_cast<const uint2 *>(p));
    const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&q.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2 *>(&q.y));
    return make_float4(a.x, a.y, b.x, b.y);
}
__device__ __forceinline__ float4 load_vec4(const __nv_bfloat16 *p) {
    const uint2 q = __ldg(reinterpret_cast<const uint2 *>(p));
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&q.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&q.y));
    return make_float4(a.x, a.y, b.x, b.y);
}

// Two horizontally adjacent activations as floats (the pair starts at an even column of an even-length row, so
// it is aligned to its own size).
__device__ __forceinline__ float2 load_pair(const float *p) { return __ldg(reinterpret_cast<const float2 *>(p)); }
__device__ __forceinline__ float2 load_pair(const __half *p) {
    const unsigned q = __ldg(reinterpret_cast<const unsigned *>(p));
    return __half22float2(*reinterpret_cast<const __half2 *>(&q));
}
__device__ __forceinline__ float2 load_pair(const __nv_bfloat16 *p) {
    const unsigned q = __ldg(reinterpret_cast<const unsigned *>(p));
    return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&q));
}

// Stage the four subbands of the level grid (Hl x Wl) around tile origin (i0, j0), with halo R,
// from the previous carrier plane `xp` (Hp x Wp).  Positions outside the level grid are zero
// (the depthwise conv's zero padding); pixels outside the carrier are zero (odd-size padding).
template <typename Tin, int K>
__device__ __forceinline__ void stage_subbands_batched(const Tin *__restrict__ xp, int Hp, int Wp, int Hl, int Wl, int i0,
                                               int j0, float (*Ys)[LevelTile<K>::H][LevelTile<K>::P] /* [4] */) {
    using D = LevelTile<K>;
    if ((D::R & 1) == 0 && (Wp & 3) == 0) {
        // two coefficients per step from one 4-pixel vector load per row: with an even halo and rows that are
        // multiples of four pixels a pair (j even) is aligned and lies wholly inside or wholly outside the grid
        constexpr int NIT = (D::H * (D::P / 2) + NTHREADS - 1) / NTHREADS;
        float4 t[NIT], u[NIT];  // all loads of a thread are issued before the first butterfly
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            const int e = threadIdx.x + it * NTHREADS;
            const int li = e / (D::P / 2), lj = 2 * (e - li * (D::P / 2));
            const int i = i0 + li - D::R, j = j0 + lj - D::R;
            t[it] = u[it] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (e < D::H * (D::P / 2) && lj < D::W && i >= 0 && i < Hl && j >= 0 && j < Wl) {
                const Tin *q = xp + (size_t)(2 * i) * Wp + 2 * j;
                t[it] = load_vec4(q);
                if (2 * i + 1 < Hp) u[it] = load_vec4(q + Wp);
            }
        }
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            const int e = threadIdx.x + it * NTHREADS;
            if (e < D::H * (D::P / 2)) {
                const int li = e / (D::P / 2), lj = 2 * (e - li * (D::P / 2));
                const Haar4 h0 = haar_butterfly(t[it].x, t[it].y, u[it].x, u[it].y);
                const Haar4 h1 = haar_butterfly(t[it].z, t[it].w, u[it].z, u[it].w);
                *reinterpret_cast<float2 *>(&Ys[0][li][lj]) = make_float2(h0.ll, h1.ll);
                *reinterpret_cast<float2 *>(&Ys[1][li][lj]) = make_float2(h0.lh, h1.lh);
                *reinterpret_cast<float2 *>(&Ys[2][li][lj]) = make_float2(h0.hl, h1.hl);
                *reinterpret_cast<float2 *>(&Ys[3][li][lj]) = make_float2(h0.hh, h1.hh);
            }
        }
        return;
    }
    const bool even = (Wp & 1) == 0;
    constexpr int NIT = (D::H * D::P + NTHREADS - 1) / NTHREADS;
    float px[NIT][4];  // the 2 x 2 pixels of each of this thread's coefficients: all loads before the first butterfly
#pragma unroll
    for (int it = 0; it < NIT; ++it) {
        const int e = threadIdx.x + it * NTHREADS;
        const int li = e / D::P, lj = e - li * D::P;
        const int i = i0 + li - D::R, j = j0 + lj - D::R;
        px[it][0] = px[it][1] = px[it][2] = px[it][3] = 0.f;
        if (e < D::H * D::P && lj < D::W && i >= 0 && i < Hl && j >= 0 && j < Wl) {
            const int y = 2 * i, x = 2 * j;
            const bool y1 = (y + 1 < Hp);
            const Tin *q = xp + (size_t)y * Wp + x;
            if (even) {
                const float2 t = load_pair(q);
                px[it][0] = t.x; px[it][1] = t.y;
                if (y1) { const float2 u = load_pair(q + Wp); px[it][2] = u.x; px[it][3] = u.y; }
            } else {
                const bool x1 = (x + 1 < Wp);
                px[it][0] = ldf(q);
                if (x1) px[it][1] = ldf(q + 1);
                if (y1) { px[it][2] = ldf(q + Wp); if (x1) px[it][3] = ldf(q + Wp + 1); }
            }
        }
    }
#pragma unroll
    for (int it = 0; it < NIT; ++it) {
        const int e = threadIdx.x + it * NTHREADS;
        if (e < D::H * D::P) {
            const int li = e / D::P, lj = e - li * D::P;
            const Haar4 h = haar_butterfly(px[it][0], px[it][1], px[it][2], px[it][3]);
            Ys[0][li][lj] = h.ll;
            Ys[1][li][lj] = h.lh;
            Ys[2][li][lj] = h.hl;
            Ys[3][li][lj] = h.hh;
        }
    }
}

template <typename Tin, int K>
__device__ __forceinline__ void stage_subbands_looped(const Tin *__restrict__ xp, int Hp, int Wp, int Hl, int Wl, int i0,
                                               int j0, float (*Ys)[LevelTile<K>::H][LevelTile<K>::P] /* [4] */) {
    using D = LevelTile<K>;
    if ((D::R & 1) == 0 && (Wp & 3) == 0) {
        // two coefficients per step from one 4-pixel vector load per row: with an even halo and rows that are
        // multiples of four pixels a pair (j even) is aligned and lies wholly inside or wholly outside the grid
        for (int e = threadIdx.x; e < D::H * (D::P / 2); e += NTHREADS) {
            const int li = e / (D::P / 2), lj = 2 * (e - li * (D::P / 2));
            const int i = i0 + li - D::R, j = j0 + lj - D::R;
            Haar4 h0 = {0.f, 0.f, 0.f, 0.f}, h1 = {0.f, 0.f, 0.f, 0.f};
            if (lj < D::W && i >= 0 && i < Hl && j >= 0 && j < Wl) {
                const Tin *q = xp + (size_t)(2 * i) * Wp + 2 * j;
                const float4 t = load_vec4(q);
                float4 u = make_float4(0.f, 0.f, 0.f, 0.f);
                if (2 * i + 1 < Hp) u = load_vec4(q + Wp);
                h0 = haar_butterfly(t.x, t.y, u.x, u.y);
                h1 = haar_butterfly(t.z, t.w, u.z, u.w);
            }
            *reinterpret_cast<float2 *>(&Ys[0][li][lj]) = make_float2(h0.ll, h1.ll);
            *reinterpret_cast<float2 *>(&Ys[1][li][lj]) = make_float2(h0.lh, h1.lh);
            *reinterpret_cast<float2 *>(&Ys[2][li][lj]) = make_float2(h0.hl, h1.hl);
            *reinterpret_cast<float2 *>(&Ys[3][li][lj]) = make_float2(h0.hh, h1.hh);
        }
        return;
    }
    const bool even = (Wp & 1) == 0;
    for (int e = threadIdx.x; e < D::H * D::P; e += NTHREADS) {
        const int li = e / D::P, lj = e - li * D::P;
        const int i = i0 + li - D::R, j = j0 + lj - D::R;
        Haar4 h = {0.f, 0.f, 0.f, 0.f};
        if (lj < D::W && i >= 0 && i < Hl && j >= 0 && j < Wl) {
            const int y = 2 * i, x = 2 * j;
            const bool y1 = (y + 1 < Hp);
            const Tin *q = xp + (size_t)y * Wp + x;
            float a, b, c = 0.f, d = 0.f;
            if (even) {
                const float2 t = load_pair(q);
                a = t.x; b = t.y;
                if (y1) { const float2 u = load_pair(q + Wp); c = u.x; d = u.y; }
            } else {
                const bool x1 = (x + 1 < Wp);
                a = ldf(q);
                b = x1 ? ldf(q + 1) : 0.f;
                if (y1) { c = ldf(q + Wp); d = x1 ? ldf(q + Wp + 1) : 0.f; }
            }
            h = haar_butterfly(a, b, c, d);
        }
        Ys[0][li][lj] = h.ll;
        Ys[1][li][lj] = h.lh;
        Ys[2][li][lj] = h.hl;
        Ys[3][li][lj] = h.hh;
    }
}

// BATCH = true issues all of a thread's loads before the first use (hides the load latency, costs registers:
// used where the kernel has them to spare); BATCH = false is the plain loop.
template <typename Tin, int K, bool BATCH>
__device__ __forceinline__ void stage_subbands(const Tin *__restrict__ xp, int Hp, int Wp, int Hl, int Wl, int i0,
                                               int j0, float (*Ys)[LevelTile<K>::H][LevelTile<K>::P] /* [4] */) {
    if (BATCH) stage_subbands_batched<Tin, K>(xp, Hp, Wp, Hl, Wl, i0, j0, Ys);
    else stage_subbands_looped<Tin, K>(xp, Hp, Wp, Hl, Wl, i0, j0, Ys);
}

// 4 x 4 outputs of the k x k correlation with register weights; `Xs` has pitch P and the window starts at
// (ly0, lx0), lx0 a multiple of 4, so its rows come as aligned float4 loads.
template <int K, int P>
__device__ __forceinline__ void block_conv(const float (*Xs)[P], int ly0, int lx0, const float *w, float (&acc)[4][4]) {
    constexpr int NQ = (4 + K - 1 + 3) / 4;
#pragma unroll
    for (int rr = 0; rr < 4 + K - 1; ++rr) {
        float in[4 * NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
            const float4 v = *reinterpret_cast<const float4 *>(&Xs[ly0 + rr][lx0 + 4 * q]);
            in[4 * q] = v.x; in[4 * q + 1] = v.y; in[4 * q + 2] = v.z; in[4 * q + 3] = v.w;
        }
#pragma unroll
        for (int u = 0; u < K; ++u) {
            const int r = rr - u;
            if (r >= 0 && r < 4) {
#pragma unroll
                for (int v = 0; v < K; ++v)
#pragma unroll
                    for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(w[u * K + v], in[c + v], acc[r][c]);
            }
        }
    }
}

// Weight-gradient taps of a 4 x 4 block: gw[u,v] += sum_{r,c} d[r][c] * Xs[ly0 + r + u][lx0 + c + v].
template <int K, int P>
__device__ __forceinline__ void block_wgrad(const float (*Xs)[P], int ly0, int lx0, const float (&d)[4][4], float *gw) {
    constexpr int NQ = (4 + K - 1 + 3) / 4;
#pragma unroll
    for (int rr = 0; rr < 4 + K - 1; ++rr) {
        float in[4 * NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
            const float4 v = *reinterpret_cast<const float4 *>(&Xs[ly0 + rr][lx0 + 4 * q]);
            in[4 * q] = v.x; in[4 * q + 1] = v.y; in[4 * q + 2] = v.z; in[4 * q + 3] = v.w;
        }
#pragma unroll
        for (int u = 0; u < K; ++u) {
            const int r = rr - u;
            if (r >= 0 && r < 4) {
#pragma unroll
                for (int v = 0; v < K; ++v)
#pragma unroll
                    for (int c = 0; c < 4; ++c) gw[u * K + v] = fmaf(d[r][c], in[c + v], gw[u * K + v]);
            }
        }
    }
}

// Store rows of four fp32 coefficients of a level grid (vector store where the row length allows).
__device__ __forceinline__ void store_coeff_block(float *__restrict__ plane, int Hl, int Wl, int I0, int J0,
                                                  const float (&a)[4][4]) {
    const bool vec = (Wl & 3) == 0 && J0 + 3 < Wl;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        if (I0 + r >= Hl) break;
        float *q = plane + (size_t)(I0 + r) * Wl + J0;
        if (vec) {
            *reinterpret_cast<float4 *>(q) = make_float4(a[r][0], a[r][1], a[r][2], a[r][3]);
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (J0 + c < Wl) q[c] = a[r][c];
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
    using D = LevelTile<K>;
    constexpr int KK = K * K;
    __shared__ __align__(16) float Ys[4][D::H][D::P];
    __shared__ float Ws[4][KK];
    const int ntx = tiles_of(Wl, TW), ntile = ntx * tiles_of(Hl, TH);
    const int p = blockIdx.x / ntile, tile = blockIdx.x - p * ntile, c = p % C;
    const int j0 = (tile % ntx) * TW, i0 = (tile / ntx) * TH;
    stage_subbands<Tin, K, true>(Xprev + (size_t)p * Hp * Wp, Hp, Wp, Hl, Wl, i0, j0, Ys);
    if (threadIdx.x < 4 * KK)  // Eq. 8
        Ws[threadIdx.x / KK][threadIdx.x % KK] = __ldg(s + c * 4 + threadIdx.x / KK) * __ldg(w + (size_t)c * 4 * KK + threadIdx.x);
    __syncthreads();
    const int sub = threadIdx.x >> 6, tx = threadIdx.x & 7, ty = (threadIdx.x >> 3) & 7;
    const int I0 = i0 + 4 * ty, J0 = j0 + 4 * tx;
    if (I0 >= Hl || J0 >= Wl) return;
    float wr[KK];
#pragma unroll
    for (int t = 0; t < KK; ++t) wr[t] = Ws[sub][t];
    float acc[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) acc[r][cc] = 0.f;
    block_conv<K, D::P>(Ys[sub], 4 * ty, 4 * tx, wr, acc);
    store_coeff_block(Z + ((size_t)p * 4 + sub) * Hl * Wl, Hl, Wl, I0, J0, acc);
    if (sub == 0 && Xl) {
        float ll[4][4];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) ll[r][cc] = Ys[0][4 * ty + D::R + r][4 * tx + D::R + cc];
        store_coeff_block(Xl + (size_t)p * Hl * Wl, Hl, Wl, I0, J0, ll);
    }
}

// ---------------------------------------------------------------------------------------------
// Forward synthesis kernel: out = Wfold^0 (*) x + bfold + sum_l (Prop. 2 term of Z^l).
// grid (P, tiles_x, tiles_y) over STW x STH pixel tiles; one 4 x 4 pixel block per thread.
// ---------------------------------------------------------------------------------------------
struct LevelPtrs {
    const float *z[8];  // per level l (index l-1): [P][4][Hl][Wl]
    int Hl[8], Wl[8];
};

// Pixel tile of the synthesis kernels: STW x STH pixels per block, a 4 x 4 pixel block per thread
// (16 x 16 threads).  The x tile sits in shared memory with halo R and a pitch that keeps every
// thread's window start 16-byte aligned.
constexpr int STW = 64, STH = 64;
template <int K> struct SynthTile : TileDims<K, STW, STH> {
    static constexpr int XW = TileDims<K, STW, STH>::W, XH = TileDims<K, STW, STH>::H, XP = TileDims<K, STW, STH>::P;
};

// Stage the STW x STH pixel tile at (y0, x0) of plane p of tensor `base` ([P][H][W], 16-byte aligned) with halo
// R; zero outside the image.  When the row length is a multiple of 4 the tile's own columns come as vector loads
// of 4 pixels (they are then either all inside the image or all outside) and only the 2R halo columns go element
// by element.  Otherwise rows start at arbitrary element offsets: the tile is zeroed and then filled from the
// aligned 4-element chunks of the whole tensor that overlap each tile row, every element placed on its own
// (chunks may begin in the previous row or end in the next one; `total` = elements in the tensor bounds them).
template <typename T, int K>
__device__ __forceinline__ void stage_pixels_batched(const T *__restrict__ base, size_t p, size_t total, int H, int W, int y0,
                                             int x0, float (*Xs)[SynthTile<K>::XP]) {
    using S = SynthTile<K>;
    const size_t plane0 = p * (size_t)H * W;
    const T *xp = base + plane0;
    if ((W & 3) == 0) {
        // all of a thread's vector loads are issued before the first one is used
        constexpr int NIT = (S::XH * (STW / 4) + NTHREADS - 1) / NTHREADS;
        float4 v[NIT];
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            const int e = threadIdx.x + it * NTHREADS;
            const int ly = e / (STW / 4), j = e - ly * (STW / 4);
            const int yy = y0 + ly - S::R, xx = x0 + 4 * j;
            v[it] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (e < S::XH * (STW / 4) && yy >= 0 && yy < H && xx < W) v[it] = load_vec4(xp + (size_t)yy * W + xx);
        }
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            const int e = threadIdx.x + it * NTHREADS;
            if (e < S::XH * (STW / 4)) {
                const int ly = e / (STW / 4), j = e - ly * (STW / 4);
                float *q = &Xs[ly][S::R + 4 * j];
                q[0] = v[it].x; q[1] = v[it].y; q[2] = v[it].z; q[3] = v[it].w;
            }
        }
        for (int e = threadIdx.x; e < S::XH * (S::XP - STW); e += NTHREADS) {
            const int ly = e / (S::XP - STW), h = e - ly * (S::XP - STW);
            const int lx = h < S::R ? h : STW + h;  // left halo, then right halo and the pitch padding
            const int yy = y0 + ly - S::R, xx = x0 + lx - S::R;
            Xs[ly][lx] = (yy >= 0 && yy < H && xx >= 0 && xx < W) ? ldf(xp + (size_t)yy * W + xx) : 0.f;
        }
        return;
    }
    float4 *z = reinterpret_cast<float4 *>(&Xs[0][0]);
    for (int e = threadIdx.x; e < S::XH * S::XP / 4; e += NTHREADS) z[e] = make_float4(0.f, 0.f, 0.f, 0.f);
    __syncthreads();
    constexpr int CH = (S::XW + 3) / 4 + 1;  // aligned chunks that can overlap one tile row
    const int xa = x0 - S::R < 0 ? 0 : x0 - S::R;                    // first image column the tile needs
    const int xb = x0 + STW + S::R > W ? W : x0 + STW + S::R;        // one past the last
    constexpr int NIT = (S::XH * CH + NTHREADS - 1) / NTHREADS;
    float v[NIT][4];
    long long col0[NIT];  // image column of the chunk's first element; a huge value marks "nothing to place"
#pragma unroll
    for (int it = 0; it < NIT; ++it) {  // all loads first
        const int e = threadIdx.x + it * NTHREADS;
        const int ly = e / CH, k = e - ly * CH;
        const int yy = y0 + ly - S::R;
        col0[it] = (long long)1 << 40;
        v[it][0] = v[it][1] = v[it][2] = v[it][3] = 0.f;
        if (e >= S::XH * CH || yy < 0 || yy >= H || xa >= xb) continue;
        const size_t row0 = plane0 + (size_t)yy * W;               // tensor-wide index of the row's first element
        const size_t c = ((row0 + xa) >> 2) + k;                    // aligned chunk
        if (4 * c >= row0 + xb) continue;
        if (4 * c + 3 < total) {
            const float4 t = load_vec4(base + 4 * c);
            v[it][0] = t.x; v[it][1] = t.y; v[it][2] = t.z; v[it][3] = t.w;
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) v[it][i] = 4 * c + i < total ? ldf(base + 4 * c + i) : 0.f;
        }
        col0[it] = (long long)(4 * c) - (long long)row0;
    }
#pragma unroll
    for (int it = 0; it < NIT; ++it) {
        const int ly = (threadIdx.x + it * NTHREADS) / CH;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const long long col = col0[it] + i;
            if (col >= xa && col < xb) Xs[ly][(int)col - x0 + S::R] = v[it][i];
        }
    }
}

template <typename T, int K>
__device__ __forceinline__ void stage_pixels_looped(const T *__restrict__ base, size_t p, size_t total, int H, int W, int y0,
                                             int x0, float (*Xs)[SynthTile<K>::XP]) {
    using S = SynthTile<K>;
    const size_t plane0 = p * (size_t)H * W;
    const T *xp = base + plane0;
    if ((W & 3) == 0) {
        for (int e = threadIdx.x; e < S::XH * (STW / 4); e += NTHREADS) {
            const int ly = e / (STW / 4), j = e - ly * (STW / 4);
            const int yy = y0 + ly - S::R, xx = x0 + 4 * j;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (yy >= 0 && yy < H && xx < W) v = load_vec4(xp + (size_t)yy * W + xx);
            float *q = &Xs[ly][S::R + 4 * j];
            q[0] = v.x; q[1] = v.y; q[2] = v.z; q[3] = v.w;
        }
        for (int e = threadIdx.x; e < S::XH * (S::XP - STW); e += NTHREADS) {
            const int ly = e / (S::XP - STW), h = e - ly * (S::XP - STW);
            const int lx = h < S::R ? h : STW + h;  // left halo, then right halo and the pitch padding
            const int yy = y0 + ly - S::R, xx = x0 + lx - S::R;
            Xs[ly][lx] = (yy >= 0 && yy < H && xx >= 0 && xx < W) ? ldf(xp + (size_t)yy * W + xx) : 0.f;
        }
        return;
    }
    float4 *z = reinterpret_cast<float4 *>(&Xs[0][0]);
    for (int e = threadIdx.x; e < S::XH * S::XP / 4; e += NTHREADS) z[e] = make_float4(0.f, 0.f, 0.f, 0.f);
    __syncthreads();
    constexpr int CH = (S::XW + 3) / 4 + 1;  // aligned chunks that can overlap one tile row
    const int xa = x0 - S::R < 0 ? 0 : x0 - S::R;                    // first image column the tile needs
    const int xb = x0 + STW + S::R > W ? W : x0 + STW + S::R;        // one past the last
    for (int e = threadIdx.x; e < S::XH * CH; e += NTHREADS) {
        const int ly = e / CH, k = e - ly * CH;
        const int yy = y0 + ly - S::R;
        if (yy < 0 || yy >= H || xa >= xb) continue;
        const size_t row0 = plane0 + (size_t)yy * W;               // tensor-wide index of the row's first element
        const size_t c = ((row0 + xa) >> 2) + k;                    // aligned chunk
        if (4 * c >= row0 + xb) continue;
        float v[4];
        if (4 * c + 3 < total) {
            const float4 t = load_vec4(base + 4 * c);
            v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) v[i] = 4 * c + i < total ? ldf(base + 4 * c + i) : 0.f;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const long long col = (long long)(4 * c + i) - (long long)row0;  // image column of this element
            if (col >= xa && col < xb) Xs[ly][(int)col - x0 + S::R] = v[i];
        }
    }
}

template <typename T, int K, bool BATCH>
__device__ __forceinline__ void stage_pixels(const T *__restrict__ base, size_t p, size_t total, int H, int W, int y0,
                                             int x0, float (*Xs)[SynthTile<K>::XP]) {
    if (BATCH) stage_pixels_batched<T, K>(base, p, total, H, W, y0, x0, Xs);
    else stage_pixels_looped<T, K>(base, p, total, H, W, y0, x0, Xs);
}

// Proposition 2 for the 4 x 4 pixel block with origin (Y0, X0), both multiples of 4, of plane p: level 1
// contributes 2 x 2 coefficients per subband, level 2 one coefficient whose signs vary inside the block, every
// deeper level one coefficient with a block-wide sign.  The level-1 and level-2 coefficients are fetched first
// (load_z12) so that their global-memory latency runs behind the block's convolution.
struct Z12 {
    float z1[2][2][4];  // [ci][cj][subband]
    float z2[4];
};
__device__ __forceinline__ Z12 load_z12(const LevelPtrs &lv, int L, size_t p, int Y0, int X0) {
    Z12 z;
#pragma unroll
    for (int ci = 0; ci < 2; ++ci)
#pragma unroll
        for (int cj = 0; cj < 2; ++cj)
#pragma unroll
            for (int sb = 0; sb < 4; ++sb) z.z1[ci][cj][sb] = 0.f;
#pragma unroll
    for (int sb = 0; sb < 4; ++sb) z.z2[sb] = 0.f;
    if (L >= 1) {
        const int Hl = lv.Hl[0], Wl = lv.Wl[0];
        const size_t S = (size_t)Hl * Wl;
        const float *zp = lv.z[0] + p * 4 * S;
#pragma unroll
        for (int ci = 0; ci < 2; ++ci)
#pragma unroll
            for (int cj = 0; cj < 2; ++cj) {
                const int i = (Y0 >> 1) + ci, j = (X0 >> 1) + cj;
                if (i < Hl && j < Wl) {  // coefficients beyond the grid only feed pixels beyond the image
                    const float *q = zp + (size_t)i * Wl + j;
#pragma unroll
                    for (int sb = 0; sb < 4; ++sb) z.z1[ci][cj][sb] = __ldg(q + sb * S);
                }
            }
    }
    if (L >= 2) {
        const int Wl = lv.Wl[1];
        const size_t S = (size_t)lv.Hl[1] * Wl;
        const float *q = lv.z[1] + p * 4 * S + (size_t)(Y0 >> 2) * Wl + (X0 >> 2);
#pragma unroll
        for (int sb = 0; sb < 4; ++sb) z.z2[sb] = __ldg(q + sb * S);
    }
    return z;
}
__device__ __forceinline__ void block_synthesis(const LevelPtrs &lv, int L, size_t p, int Y0, int X0, const Z12 &z,
                                                float (&a)[4][4]) {
    if (L >= 1) {
#pragma unroll
        for (int ci = 0; ci < 2; ++ci)
#pragma unroll
            for (int cj = 0; cj < 2; ++cj) {
                const float ll = z.z1[ci][cj][0], lh = z.z1[ci][cj][1], hl = z.z1[ci][cj][2], hh = z.z1[ci][cj][3];
                const float pp = ll + lh, pm = ll - lh, qp = hl + hh, qm = hl - hh;
                a[2 * ci][2 * cj] = fmaf(0.5f, pp + qp, a[2 * ci][2 * cj]);
                a[2 * ci][2 * cj + 1] = fmaf(0.5f, pp - qp, a[2 * ci][2 * cj + 1]);
                a[2 * ci + 1][2 * cj] = fmaf(0.5f, pm + qm, a[2 * ci + 1][2 * cj]);
                a[2 * ci + 1][2 * cj + 1] = fmaf(0.5f, pm - qm, a[2 * ci + 1][2 * cj + 1]);
            }
    }
    if (L >= 2) {
        float deep = 0.f, scale = 0.25f;
        for (int l = 3; l <= L; ++l) {
            scale *= 0.5f;
            const int Wl = lv.Wl[l - 1];
            const size_t S = (size_t)lv.Hl[l - 1] * Wl;
            const float *q = lv.z[l - 1] + p * 4 * S + (size_t)(Y0 >> l) * Wl + (X0 >> l);
            deep += synth_term(__ldg(q), __ldg(q + S), __ldg(q + 2 * S), __ldg(q + 3 * S), (Y0 >> (l - 1)) & 1,
                               (X0 >> (l - 1)) & 1, scale);
        }
        const float ll = z.z2[0], lh = z.z2[1], hl = z.z2[2], hh = z.z2[3];
        const float pp = ll + lh, pm = ll - lh, qp = hl + hh, qm = hl - hh;
        float t2[2][2];
        t2[0][0] = fmaf(0.25f, pp + qp, deep);
        t2[0][1] = fmaf(0.25f, pp - qp, deep);
        t2[1][0] = fmaf(0.25f, pm + qm, deep);
        t2[1][1] = fmaf(0.25f, pm - qm, deep);
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) a[r][c] += t2[r >> 1][c >> 1];
    }
}

// Store the block's rows that lie inside the image; whole aligned rows go out as one vector store.
__device__ __forceinline__ void store4(float *p, const float *v) { *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]); }
__device__ __forceinline__ void store4(__half *p, const float *v) {
    const __half2 a = __floats2half2_rn(v[0], v[1]), b = __floats2half2_rn(v[2], v[3]);
    uint2 q;
    q.x = *reinterpret_cast<const unsigned *>(&a);
    q.y = *reinterpret_cast<const unsigned *>(&b);
    *reinterpret_cast<uint2 *>(p) = q;
}
__device__ __forceinline__ void store4(__nv_bfloat16 *p, const float *v) {
    const __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
    uint2 q;
    q.x = *reinterpret_cast<const unsigned *>(&a);
    q.y = *reinterpret_cast<const unsigned *>(&b);
    *reinterpret_cast<uint2 *>(p) = q;
}
template <typename T>
__device__ __forceinline__ void store_block(T *__restrict__ plane, int H, int W, int Y0, int X0, const float (&a)[4][4]) {
    const bool vec = (W & 3) == 0 && X0 + 3 < W;  // base pointers are 16-byte aligned and the row pitch keeps it
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        if (Y0 + r >= H) break;
        T *q = plane + (size_t)(Y0 + r) * W + X0;
        if (vec) {
            store4(q, a[r]);
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (X0 + c < W) stf(q + c, a[r][c]);
        }
    }
}

template <typename T, int K>
__global__ void __launch_bounds__(NTHREADS)
synth_fwd_kernel(const T *__restrict__ x, int H, int W, int C, int L, const float *__restrict__ w0,
                 const float *__restrict__ s0, const float *__restrict__ b0, LevelPtrs lv, T *__restrict__ out) {
    using S = SynthTile<K>;
    __shared__ __align__(16) float Xs[S::XH][S::XP];
    const int ntx = tiles_of(W, STW), ntile = ntx * tiles_of(H, STH);
    const int p = blockIdx.x / ntile, tile = blockIdx.x - p * ntile, c = p % C;
    const int x0 = (tile % ntx) * STW, y0 = (tile / ntx) * STH;
    stage_pixels<T, K, true>(x, (size_t)p, (size_t)(gridDim.x / ntile) * H * W, H, W, y0, x0, Xs);
    // folded weights (Eq. 8) go through shared memory once, then live in registers
    __shared__ float Ws[K * K + 1];
    const float sc = __ldg(s0 + c);
    if (threadIdx.x < K * K) Ws[threadIdx.x] = sc * __ldg(w0 + (size_t)c * K * K + threadIdx.x);
    if (threadIdx.x == K * K) Ws[K * K] = b0 ? sc * __ldg(b0 + c) : 0.f;
    __syncthreads();
    float wr[K * K];
#pragma unroll
    for (int t = 0; t < K * K; ++t) wr[t] = Ws[t];
    const float bias = Ws[K * K];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int X0 = x0 + 4 * tx, Y0 = y0 + 4 * ty;
    if (X0 >= W || Y0 >= H) return;
    float acc[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) acc[r][cc] = bias;
    const Z12 z = load_z12(lv, L, (size_t)p, Y0, X0);
    block_conv<K, S::XP>(Xs, 4 * ty, 4 * tx, wr, acc);
    block_synthesis(lv, L, (size_t)p, Y0, X0, z, acc);
    store_block<T>(out + (size_t)p * H * W, H, W, Y0, X0, acc);
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
template <int K> constexpr size_t level_bwd_smem_bytes() {
    return sizeof(float) * (2 * 4 * LevelTile<K>::H * LevelTile<K>::P + 8 * K * K + 4 * K * K);
}

template <typename Tin, int K>
__global__ void __launch_bounds__(NTHREADS, K <= 5 ? 3 : 1)
level_bwd_kernel(const Tin *__restrict__ Xprev, const Tin *__restrict__ Gprev, int Hp, int Wp, int Hl, int Wl, int B,
                 int C, int bsplit, const float *__restrict__ w, const float *__restrict__ s,
                 float *__restrict__ dY /* [P][4][Hl][Wl] */, float *__restrict__ Xl, float *__restrict__ Gl,
                 float *__restrict__ partials) {
    using D = LevelTile<K>;
    constexpr int KK = K * K;
    extern __shared__ __align__(16) float lsm[];  // Ys[4][H][P], Ds[4][H][P], red[8][KK], Ws[4][KK]
    float (*Ys)[D::H][D::P] = reinterpret_cast<float (*)[D::H][D::P]>(lsm);
    float (*Ds)[D::H][D::P] = reinterpret_cast<float (*)[D::H][D::P]>(lsm + 4 * D::H * D::P);
    float (*red)[KK] = reinterpret_cast<float (*)[KK]>(lsm + 8 * D::H * D::P);
    float (*Ws)[KK] = reinterpret_cast<float (*)[KK]>(lsm + 8 * D::H * D::P + 8 * KK);
    const int ntx = tiles_of(Wl, TW), ntile = ntx * tiles_of(Hl, TH);
    const int cp = blockIdx.x / ntile, tile = blockIdx.x - cp * ntile;
    const int c = cp / bsplit, part = cp - c * bsplit;
    const int j0 = (tile % ntx) * TW, i0 = (tile / ntx) * TH;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = threadIdx.x >> 6, tx = threadIdx.x & 7, ty = (threadIdx.x >> 3) & 7;
    const int I0 = i0 + 4 * ty, J0 = j0 + 4 * tx;
    const bool live = I0 < Hl && J0 < Wl;
    if (threadIdx.x < 4 * KK) {  // folded (Eq. 8) and rotated by 180 degrees
        const int sb = threadIdx.x / KK, t = threadIdx.x % KK;
        Ws[sb][t] = __ldg(s + c * 4 + sb) * __ldg(w + ((size_t)c * 4 + sb) * KK + (KK - 1 - t));
    }
    __syncthreads();
    float wf[KK], gw[KK];
#pragma unroll
    for (int t = 0; t < KK; ++t) {
        wf[t] = Ws[sub][t];
        gw[t] = 0.f;
    }
    for (int b = part; b < B; b += bsplit) {
        const size_t p = (size_t)b * C + c;
        __syncthreads();
        // (three resident blocks at k <= 5 leave 80 registers: no room for batched loads)
        stage_subbands<Tin, K, (K > 5)>(Xprev + p * Hp * Wp, Hp, Wp, Hl, Wl, i0, j0, Ys);
        stage_subbands<Tin, K, (K > 5)>(Gprev + p * Hp * Wp, Hp, Wp, Hl, Wl, i0, j0, Ds);
        __syncthreads();
        if (!live) continue;
        // weight gradient: the block's 16 D values (zero outside the grid) against the shifted Y window
        float d[4][4];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) d[r][cc] = Ds[sub][4 * ty + D::R + r][4 * tx + D::R + cc];
        block_wgrad<K, D::P>(Ys[sub], 4 * ty, 4 * tx, d, gw);
        float acc[4][4];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) acc[r][cc] = 0.f;
        block_conv<K, D::P>(Ds[sub], 4 * ty, 4 * tx, wf, acc);
        store_coeff_block(dY + (p * 4 + sub) * Hl * Wl, Hl, Wl, I0, J0, acc);
        if (sub == 0 && Xl) {
            float ll[4][4];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) ll[r][cc] = Ys[0][4 * ty + D::R + r][4 * tx + D::R + cc];
            store_coeff_block(Xl + p * Hl * Wl, Hl, Wl, I0, J0, ll);
            store_coeff_block(Gl + p * Hl * Wl, Hl, Wl, I0, J0, d);
        }
    }
    // block reduction: lanes by shuffle, the two warps of a subband through shared memory
#pragma unroll
    for (int t = 0; t < KK; ++t) {
        float v = warp_sum(gw[t]);
        if (lane == 0) red[warp][t] = v;
    }
    __syncthreads();
    const int nparts = ntile * bsplit;
    const int pidx = tile * bsplit + part;
    for (int e = threadIdx.x; e < 4 * KK; e += NTHREADS) {
        int sb = e / KK, t = e - sb * KK;
        partials[(((size_t)c * nparts + pidx) * 4 + sb) * KK + t] = red[2 * sb][t] + red[2 * sb + 1][t];
    }
}

// ---------------------------------------------------------------------------------------------
// Backward synthesis kernel:
//   dx = flip(Wfold^0) (*) G + sum_l (Prop. 2 term of dY^l)       (Sec. 2.2 + Prop. 2)
//   dWfold^0[u,v] += sum G[y,x] x[y+u-R, x+v-R],  dbfold += sum G
// grid (C * bsplit, tiles_x, tiles_y).  Partials: [C][nparts][K*K + 1].
// ---------------------------------------------------------------------------------------------
template <typename T, int K>
__global__ void __launch_bounds__(NTHREADS, K <= 5 ? 3 : 1)
synth_bwd_kernel(const T *__restrict__ x, const T *__restrict__ g, int H, int W, int B, int C, int L, int bsplit,
                 const float *__restrict__ w0, const float *__restrict__ s0, LevelPtrs lv, T *__restrict__ dx,
                 float *__restrict__ partials) {
    using S = SynthTile<K>;
    constexpr int R = K / 2, KK = K * K;
    __shared__ __align__(16) float Xs[S::XH][S::XP];
    __shared__ __align__(16) float Gs[S::XH][S::XP];
    __shared__ float red[8][KK + 1];
    const int ntx = tiles_of(W, STW), ntile = ntx * tiles_of(H, STH);
    const int cp = blockIdx.x / ntile, tile = blockIdx.x - cp * ntile;
    const int c = cp / bsplit, part = cp - c * bsplit;
    const int x0 = (tile % ntx) * STW, y0 = (tile / ntx) * STH;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int X0 = x0 + 4 * tx, Y0 = y0 + 4 * ty;
    const bool live = X0 < W && Y0 < H;
    float wf[KK], gw[KK], gb = 0.f;
    const float sc = __ldg(s0 + c);
#pragma unroll
    for (int t = 0; t < KK; ++t) {
        wf[t] = sc * __ldg(w0 + (size_t)c * KK + (KK - 1 - t));  // folded and rotated by 180 degrees
        gw[t] = 0.f;
    }
    for (int b = part; b < B; b += bsplit) {
        const size_t p = (size_t)b * C + c;
        __syncthreads();
        stage_pixels<T, K, (K > 5)>(x, p, (size_t)B * C * H * W, H, W, y0, x0, Xs);
        stage_pixels<T, K, (K > 5)>(g, p, (size_t)B * C * H * W, H, W, y0, x0, Gs);
        __syncthreads();
        if (!live) continue;
        // weight gradient: the block's 16 upstream values (zero outside the image) against the shifted x window
        float d[4][4];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                d[r][cc] = Gs[4 * ty + R + r][4 * tx + R + cc];
                gb += d[r][cc];
            }
        block_wgrad<K, S::XP>(Xs, 4 * ty, 4 * tx, d, gw);
        // input gradient: rotated-kernel correlation of the upstream tile plus the Proposition 2 terms of dL/dY^l
        float acc[4][4];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) acc[r][cc] = 0.f;
        block_conv<K, S::XP>(Gs, 4 * ty, 4 * tx, wf, acc);
        const Z12 z = load_z12(lv, L, p, Y0, X0);  // (fetching these ahead of the conv costs spills at 80 registers)
        block_synthesis(lv, L, p, Y0, X0, z, acc);
        store_block<T>(dx + p * H * W, H, W, Y0, X0, acc);
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
    const int nparts = ntile * bsplit;
    const int pidx = tile * bsplit + part;
    for (int e = threadIdx.x; e < KK + 1; e += NTHREADS) {
        float v = 0.f;
#pragma unroll
        for (int wi = 0; wi < 8; ++wi) v += red[wi][e];
        partials[((size_t)c * nparts + pidx) * (KK + 1) + e] = v;
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
    // Which of a channel's slots hold sums.  grp == 0: all of them (the producer cleared the rest).  grp > 0: the
    // producer was a persistent kernel whose `nblocks` blocks split `units` = (C / grp) x B work units (grp channels
    // of one image each, channel-group major) into contiguous ranges; slot i of a channel belongs to the i-th block
    // whose range meets the channel's group, later slots were never written and are not read.
    int grp, B, units, nblocks;
};

template <int UNUSED>  // a template only so that every translation unit may include this header
__global__ void __launch_bounds__(128)
unfold_epilogue_kernel(int C, int K, int L, EpiloguePtrs ep, const float *__restrict__ w0,
                       const float *__restrict__ s0, const float *__restrict__ b0, const float *__restrict__ wl,
                       const float *__restrict__ sl, float *__restrict__ dw0, float *__restrict__ ds0,
                       float *__restrict__ db0, float *__restrict__ dwl, float *__restrict__ dsl) {
    extern __shared__ double prod[];  // dWfold[e] * W[e]: [KK+1] base (tap products, then dbfold * b), then [L][4][KK]
    const int c = blockIdx.x, KK = K * K;
    const int n0 = KK + 1, nl = 4 * KK;
    dependents_may_start();  // the next kernel on the stream may run its set-up beside this one
    wait_for_predecessor();  // the partial sums come from the kernels before this one
    int written = 0x7fffffff;  // slots of this channel that hold sums
    if (ep.grp > 0) {
        const long long first_unit = (long long)(c / ep.grp) * ep.B;
        written = block_of_unit(first_unit + ep.B - 1, ep.nblocks, ep.units) - block_of_unit(first_unit, ep.nblocks, ep.units) + 1;
    }
    // One entry per thread and pass: its partial sums, the parameter it meets in the scale gradient and its scale are
    // all requested before the first is used, so the block pays one memory round trip.
    for (int e = threadIdx.x; e < n0 + L * nl; e += blockDim.x) {
        const float *q;
        size_t stride;
        int n;
        float wv, sv;
        float *dst;
        if (e < n0) {
            q = ep.part0 + (size_t)c * ep.np0 * n0 + e;
            stride = n0;
            n = ep.np0 < written ? ep.np0 : written;
            wv = e < KK ? w0[(size_t)c * KK + e] : (b0 ? b0[c] : 0.f);
            sv = s0[c];
            dst = e < KK ? dw0 + (size_t)c * KK + e : (b0 ? db0 + c : nullptr);
        } else {
            const int l = (e - n0) / nl, t = (e - n0) - l * nl;
            q = ep.partl[l] + (size_t)c * ep.npl[l] * nl + t;
            stride = nl;
            n = ep.npl[l] < written ? ep.npl[l] : written;
            wv = wl[((size_t)l * C + c) * nl + t];
            sv = sl[((size_t)l * C + c) * 4 + t / KK];
            dst = dwl + ((size_t)l * C + c) * nl + t;
        }
        double acc = 0.0;  // fixed slot order, fp64: the batch sum does not depend on the launch geometry's timing
        for (int i = 0; i < n; ++i) acc += (double)q[(size_t)i * stride];
        prod[e] = acc * (double)wv;
        if (dst) *dst = (float)((double)sv * acc);  // Eq. 9: dW = s dWfold, db = s dbfold
    }
    __syncthreads();
    // Eq. 9: ds = <dWfold, W> per class (+ dbfold b on the base class), terms added in index order
    for (int cls = threadIdx.x; cls < 1 + 4 * L; cls += blockDim.x) {
        double a = 0.0;
        if (cls == 0) {
            for (int t = 0; t < KK; ++t) a += prod[t];
            if (b0) a += prod[KK];
            ds0[c] = (float)a;
        } else {
            const double *pq = prod + n0 + (cls - 1) * KK;
            for (int t = 0; t < KK; ++t) a += pq[t];
            dsl[((size_t)((cls - 1) >> 2) * C + c) * 4 + ((cls - 1) & 3)] = (float)a;
        }
    }
}

}  // namespace wt
