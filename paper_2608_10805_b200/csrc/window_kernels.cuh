// Window kernels for planes too large to keep whole in shared memory (k = 5): a plane is cut into windows of
// WH x WW output pixels; one block computes one window at a time with levels 1 and 2 entirely on chip, and levels
// >= 3 come from a 16 times smaller carrier tensor that the whole-plane kernels process.
//
// Dataflow (forward; the backward pass is the same dataflow on grad_out with rotated kernels, Sec. 2.2, plus the
// weight-gradient correlations):
//   carrier kernel   X2 = raw low-pass band of level 2 (one value per 4 x 4 pixel block, fp32)      N -> N/16
//   whole-plane kernel on X2 with levels 3..L (base weights zero)   ->  R3 (fp32, per 4 x 4 block)   N/16 -> N/16
//   window kernel    for every window: fetch the window of x with a halo of 8 pixels (the level-2 conv needs 2
//                    coefficients = 8 pixels; what lies outside the plane is zero), run the butterfly of Eq. 5 for
//                    levels 1 and 2 on chip (Sec. 4.1), convolve register tiles with folded weights (Eq. 8), add the
//                    closed-form synthesis of Proposition 2 for levels 1-2 and a quarter of R3 (levels >= 3 of
//                    Proposition 2 are constant over a 4 x 4 block), store.                          N (+halo) -> N
// HBM traffic: about (2 + 3/16 (+ halo re-reads that hit L2)) N elements instead of the (Q_fused - 2) N of
// per-level kernels; no Z^l ever reaches HBM.
//
// A window's pixels are fetched by 16-byte cp.async copies of whole aligned chunks of the rows it needs (a row may
// start at any 2-byte offset: 225-wide fp16 rows do), double buffered, so the next window's rows travel while this
// one is computed; rows outside the plane are zero-filled by the copy, columns outside it are masked in staging.
#pragma once
#include "plane_kernels.cuh"

namespace wt {
namespace plane {
WT_PLANE_INSTANTIATE(float, extern)  // the carrier runs on the fp32 whole-plane kernels, compiled in their own unit
}
namespace window {

using plane::Geom;
using plane::KK;
using plane::WT_STRIDE;

constexpr int TH = 8;

struct WGeom {
    Geom g;              // geometry of one window seen as a small plane (H = WH, W = WW, L = on-chip levels), NPL = 1
    int H, W, L;         // the real plane and level count
    int WH, WW, nwy, nwx, hp;   // window size, windows per plane, pixel halo of the fetch (4 or 8)
    int RH, RW, rawp;    // fetched rows / columns per window, bytes per raw row (16-byte multiple incl. shift slack)
    int nbuf, raw_bytes; // raw buffers (1 or 2), bytes per buffer (both tensors in the backward)
    int npy, npx;        // 4 x 4 staging patches per window
    int aligned;         // 1: every fetched row starts on a 16-byte boundary (vector staging)
    int H2, W2;          // carrier grid (ceil(H/4), ceil(W/4)); used when L > 2
    int esz;
    long long units;     // C * B * nwy * nwx, channel-major
    int raw_off;         // float offset of the raw buffers
};

__device__ __forceinline__ void cp_async16(void *dst, const void *src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(plane::smem_addr(dst)), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Enqueue the copies of one window of one tensor: rows oy - hp .. oy + WH + hp of plane p, columns ox - hp ..; whole
// 16-byte chunks starting at the aligned address below each row's first element.
template <typename T>
__device__ __forceinline__ void fetch_window(char *raw, const WGeom &w, const T *__restrict__ base, size_t plane, int oy, int ox,
                                             size_t total_bytes) {
    const int nchunk = w.rawp / 16;
    const char *b0 = reinterpret_cast<const char *>(base);
    for (int e = threadIdx.x; e < w.RH * nchunk; e += blockDim.x) {
        const int r = e / nchunk, k = e - r * nchunk;
        const int y = oy - w.hp + r;
        // address of the row's first fetched element (may lie left of the plane row: masked later) and its aligned chunk
        const long long first = ((long long)plane * w.H * w.W + (long long)y * w.W + (ox - w.hp)) * (long long)sizeof(T);
        const long long a = (first & ~15LL) + 16LL * k;
        int nbytes = 0;
        if (y >= 0 && y < w.H && a >= 0 && a < (long long)total_bytes) {
            const long long left = (long long)total_bytes - a;
            nbytes = left < 16 ? (int)left : 16;
        }
        cp_async16(raw + r * w.rawp + 16 * k, b0 + (nbytes ? a : 0), nbytes);
    }
}

// Per-thread staging patch (4 x 4 pixels): offsets into the raw buffer and the arrays, and which parts are kept.
struct WPatch {
    int rrow, rcol;   // raw row of the patch's first pixel row, element column of its first pixel
    int xi, y1, y2;   // float indices of its first x element / level-1 coefficient / level-2 coefficient (A side)
    int meta;         // bit 31 valid; bits 0-3 x rows kept; bits 4-5 x column pairs kept; bit 6 level-1 block kept;
                      // bit 7 level-2 coefficient kept; bits 8-15 patch column (for the plane-edge column mask)
};
__device__ __forceinline__ WPatch decode_wpatch(const WGeom &w, int e) {
    WPatch p;
    p.rrow = p.rcol = p.xi = p.y1 = p.y2 = p.meta = 0;
    if (e >= w.npy * w.npx) return p;
    const Geom &g = w.g;
    const int pi = e / w.npx, pj = e - pi * w.npx, L = g.L;
    p.rrow = 4 * pi;
    p.rcol = 4 * pj;
    int meta = (int)0x80000000u | (pj << 8);
    const int ly0 = 4 * pi - w.hp + 2, lx0 = 4 * pj - w.hp + 2;  // array coordinates of the patch's first pixel
    for (int rr = 0; rr < 4; ++rr)
        if (ly0 + rr >= 0 && ly0 + rr < w.WH + 4) meta |= 1 << rr;
    for (int cp = 0; cp < 2; ++cp)
        if (lx0 + 2 * cp >= 0 && lx0 + 2 * cp + 1 < w.WW + 4) meta |= 16 << cp;
    p.xi = g.offA[0] + ly0 * g.pitch[0] + lx0;
    if (L >= 1) {
        const int i1 = 2 * pi - w.hp / 2 + 2, j1 = 2 * pj - w.hp / 2 + 2;
        if (i1 >= 0 && i1 + 1 < w.WH / 2 + 4 && j1 >= 0 && j1 + 1 < w.WW / 2 + 4) meta |= 64;
        p.y1 = g.offA[1] + i1 * g.pitch[1] + j1;
    }
    if (L >= 2) {
        const int i2 = pi - w.hp / 4 + 2, j2 = pj - w.hp / 4 + 2;
        if (i2 >= 0 && i2 < w.WH / 4 + 4 && j2 >= 0 && j2 < w.WW / 4 + 4) meta |= 128;
        p.y2 = g.offA[2] + i2 * g.pitch[2] + j2;
    }
    p.meta = meta;
    return p;
}

// The 4 x 4 pixels of a patch from the raw buffer.  shift = byte offset of the fetched row's first element inside its
// first chunk (the same for every row when `aligned`); cmask = which of the four columns lie inside the plane.
template <typename T>
__device__ __forceinline__ void load_wpatch(const char *raw, const WGeom &w, const WPatch &p, int y0, long long plane_elem0, int ox,
                                            int cmask, float (&a)[4][4]) {
    if (w.aligned) {
#pragma unroll
        for (int rr = 0; rr < 4; ++rr) {
            const T *q = reinterpret_cast<const T *>(raw + (p.rrow + rr) * w.rawp) + p.rcol;
            plane::load4s(q, a[rr]);
        }
    } else {
#pragma unroll
        for (int rr = 0; rr < 4; ++rr) {
            const int y = y0 + p.rrow + rr;
            const long long first = (plane_elem0 + (long long)y * w.W + (ox - w.hp)) * (long long)sizeof(T);
            const T *q = reinterpret_cast<const T *>(raw + (p.rrow + rr) * w.rawp + (int)(first & 15LL)) + p.rcol;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) a[rr][cc] = plane::ldf_plain(q + cc);
        }
    }
#pragma unroll
    for (int rr = 0; rr < 4; ++rr)
#pragma unroll
        for (int cc = 0; cc < 4; ++cc)
            if (!((cmask >> cc) & 1)) a[rr][cc] = 0.f;
}

// x, level 1 and level 2 of one patch into the arrays (d0/d1/d2: offsets to the grad_out side).
__device__ __forceinline__ void store_wpatch(float *sm, const Geom &g, const WPatch &p, const float (&a)[4][4], int d0, int d1, int d2) {
    const int p0 = g.pitch[0];
#pragma unroll
    for (int rr = 0; rr < 4; ++rr) {
        if ((p.meta >> rr) & 1) {
            if (p.meta & 16) *reinterpret_cast<float2 *>(&sm[p.xi + d0 + rr * p0]) = make_float2(a[rr][0], a[rr][1]);
            if (p.meta & 32) *reinterpret_cast<float2 *>(&sm[p.xi + d0 + rr * p0 + 2]) = make_float2(a[rr][2], a[rr][3]);
        }
    }
    if (g.L < 1) return;
    Haar4 h[2][2];
#pragma unroll
    for (int bi = 0; bi < 2; ++bi)
#pragma unroll
        for (int bj = 0; bj < 2; ++bj)
            h[bi][bj] = haar_butterfly(a[2 * bi][2 * bj], a[2 * bi][2 * bj + 1], a[2 * bi + 1][2 * bj], a[2 * bi + 1][2 * bj + 1]);
    if (p.meta & 64) {
        const int p1 = g.pitch[1], sub1 = g.rows[1] * p1;
#pragma unroll
        for (int bi = 0; bi < 2; ++bi) {
            *reinterpret_cast<float2 *>(&sm[p.y1 + d1 + bi * p1]) = make_float2(h[bi][0].ll, h[bi][1].ll);
            *reinterpret_cast<float2 *>(&sm[p.y1 + d1 + bi * p1 + sub1]) = make_float2(h[bi][0].lh, h[bi][1].lh);
            *reinterpret_cast<float2 *>(&sm[p.y1 + d1 + bi * p1 + 2 * sub1]) = make_float2(h[bi][0].hl, h[bi][1].hl);
            *reinterpret_cast<float2 *>(&sm[p.y1 + d1 + bi * p1 + 3 * sub1]) = make_float2(h[bi][0].hh, h[bi][1].hh);
        }
    }
    if (g.L >= 2 && (p.meta & 128)) {
        const int sub2 = g.rows[2] * g.pitch[2];
        const Haar4 h2 = haar_butterfly(h[0][0].ll, h[0][1].ll, h[1][0].ll, h[1][1].ll);
        sm[p.y2 + d2] = h2.ll;
        sm[p.y2 + d2 + sub2] = h2.lh;
        sm[p.y2 + d2 + 2 * sub2] = h2.hl;
        sm[p.y2 + d2 + 3 * sub2] = h2.hh;
    }
}

// Carrier: X2[p][i][j] = raw level-2 low-pass band = 1/4 of the sum over the 4 x 4 pixel block (zero beyond the plane).
template <typename T>
__global__ void carrier_kernel(const T *__restrict__ x, int H, int W, int H2, int W2, size_t P, float *__restrict__ X2) {
    const size_t S2 = (size_t)H2 * W2, n = P * S2;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const size_t p = e / S2;
        const int r = (int)(e - p * S2), i = r / W2, j = r - i * W2;
        const T *q = x + p * H * W;
        // two butterflies' worth of low-pass sums in the order the on-chip analysis uses: (a + b) + (c + d) per 2 x 2 block
        float ll[2][2];
#pragma unroll
        for (int bi = 0; bi < 2; ++bi)
#pragma unroll
            for (int bj = 0; bj < 2; ++bj) {
                const int y = 4 * i + 2 * bi, xx = 4 * j + 2 * bj;
                const bool y0 = y < H, y1 = y + 1 < H, x0 = xx < W, x1 = xx + 1 < W;
                const float a = (y0 && x0) ? ldf(q + (size_t)y * W + xx) : 0.f, b = (y0 && x1) ? ldf(q + (size_t)y * W + xx + 1) : 0.f;
                const float c = (y1 && x0) ? ldf(q + (size_t)(y + 1) * W + xx) : 0.f, d = (y1 && x1) ? ldf(q + (size_t)(y + 1) * W + xx + 1) : 0.f;
                ll[bi][bj] = haar_butterfly(a, b, c, d).ll;
            }
        X2[e] = haar_butterfly(ll[0][0], ll[0][1], ll[1][0], ll[1][1]).ll;
    }
}

// BWD = false: out = WTConv(x) restricted to levels <= 2, plus add / 4 (levels >= 3).  BWD = true: out = grad_x likewise,
// and the weight-gradient partial sums of the base class and of levels 1-2 go to part0 / partl.
template <typename T, bool BWD, int MINB>
__global__ void __launch_bounds__(256, MINB)
window_kernel(const __grid_constant__ WGeom w, const T *__restrict__ x, const T *__restrict__ go, const float *__restrict__ w0,
              const float *__restrict__ s0, const float *__restrict__ b0, const float *__restrict__ wl, const float *__restrict__ sl,
              const float *__restrict__ add /* [P][H2][W2] or null */, T *__restrict__ out, float *__restrict__ part0,
              float *__restrict__ partl /* level l at l*C*np*100 */, size_t total_bytes) {
    extern __shared__ __align__(16) float sm[];
    const Geom &g = w.g;
    const int tid = threadIdx.x, nthr = blockDim.x;
    float *wtab = sm + g.wtab_off;
    char *raw = reinterpret_cast<char *>(sm + w.raw_off);
    const int L = g.L, nlv = g.lvl_start[L + 1], ncls = 1 + 4 * L;
    const int nitems = nlv + g.nbase;
    const int nwin = w.nwy * w.nwx;
    const long long u_begin = (long long)blockIdx.x * w.units / gridDim.x, u_end = (long long)(blockIdx.x + 1) * w.units / gridDim.x;
    int bslot = 0, tyy = 0, txx = 0;
    bool has_base = false;
    const plane::ItemD item = plane::decode_item(g, tid, nlv, nitems, bslot, tyy, txx, has_base);
    const int cls = (item.meta >> 24) & 0x3f;
    // the coefficients of this tile that belong to this window (tiles of a level grid may be padded beyond it)
    int rlim = TH, clim = 4;
    if (item.meta < 0 && !has_base) {
        int l, sb, ty2, tx2;
        plane::decode_level_item(g, tid, l, sb, ty2, tx2);
        rlim = (w.WH >> l) - TH * ty2;
        clim = (w.WW >> l) - 4 * tx2;
    }
    const WPatch patch0 = decode_wpatch(w, tid), patch1 = decode_wpatch(w, tid + nthr);
    const int dA0 = g.offG[0] - g.offA[0], dA1 = L >= 1 ? g.offG[1] - g.offA[1] : 0, dA2 = L >= 2 ? g.offG[2] - g.offA[2] : 0;
    const int tensor_bytes = w.RH * w.rawp;

    // unit -> (channel, image, window row, window column), carried along
    long long u = u_begin;
    int c, b, wy, wx;
    {
        long long r = u;
        wx = (int)(r % w.nwx); r /= w.nwx;
        wy = (int)(r % w.nwy); r /= w.nwy;
        b = (int)(r % g.B);
        c = (int)(r / g.B);
    }
    auto fetch = [&](int buf, int cc, int bb, int wyy, int wxx) {
        const size_t plane_idx = (size_t)bb * g.C + cc;
        char *dst = raw + buf * w.raw_bytes;
        fetch_window<T>(dst, w, x, plane_idx, wyy * w.WH, wxx * w.WW, total_bytes);
        if (BWD) fetch_window<T>(dst + tensor_bytes, w, go, plane_idx, wyy * w.WH, wxx * w.WW, total_bytes);
        cp_async_commit();
    };
    if (u < u_end) fetch(0, c, b, wy, wx);
    // Array rows and columns beyond a window's own grids (tile padding) are never staged: they must hold finite values
    // (they meet zero gradient entries or feed outputs nobody reads), so the arrays start as zeros.
    for (int i = tid; i < w.raw_off / 4; i += nthr) reinterpret_cast<float4 *>(sm)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    float accw[KK], gsum = 0.f;
#pragma unroll
    for (int t = 0; t < KK; ++t) accw[t] = 0.f;
    int c_prev = -1, buf = 0;
    for (; u < u_end; ++u) {
        // the next unit's coordinates (for the prefetch and the end-of-channel test)
        int cn = c, bn = b, wyn = wy, wxn = wx + 1;
        if (wxn == w.nwx) { wxn = 0; if (++wyn == w.nwy) { wyn = 0; if (++bn == g.B) { bn = 0; ++cn; } } }
        if (c != c_prev) {
            __syncthreads();  // the previous unit's tiles may still read the old table
            plane::build_weight_table(wtab, g, c, BWD, w0, s0, BWD ? nullptr : b0, wl, sl);
            c_prev = c;
        }
        if (w.nbuf == 2) {
            if (u + 1 < u_end) { fetch(buf ^ 1, cn, bn, wyn, wxn); cp_async_wait<1>(); } else cp_async_wait<0>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();  // this window's rows have landed for every thread; the table is complete
        const int oy = wy * w.WH, ox = wx * w.WW;
        const char *rx = raw + (w.nbuf == 2 ? buf : 0) * w.raw_bytes;
        {
            const long long plane0 = ((long long)b * g.C + c) * (long long)w.H * w.W;
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const WPatch &p = k ? patch1 : patch0;
                if (p.meta >= 0) continue;
                // columns of the patch inside the plane
                const int x0 = ox - w.hp + p.rcol;
                int cmask = 0;
#pragma unroll
                for (int cc = 0; cc < 4; ++cc)
                    if (x0 + cc >= 0 && x0 + cc < w.W) cmask |= 1 << cc;
                float a[4][4];
                load_wpatch<T>(rx, w, p, oy - w.hp, plane0, ox, cmask, a);
                store_wpatch(sm, g, p, a, 0, 0, 0);
                if (BWD) {
                    load_wpatch<T>(rx + tensor_bytes, w, p, oy - w.hp, plane0, ox, cmask, a);
                    store_wpatch(sm, g, p, a, dA0, dA1, dA2);
                }
            }
        }
        __syncthreads();
        if (w.nbuf == 1 && u + 1 < u_end) fetch(0, cn, bn, wyn, wxn);  // single buffer: refill behind the math
        float acc[TH][4];
        if (item.meta < 0) {
            const int pitch = item.meta & 0x3ff;
            const float *asrc = sm + item.src;
            if (BWD) {
                const float *gsrc = asrc + item.dg;
                float d[TH][4];
#pragma unroll
                for (int rr = 0; rr < TH; ++rr) {
                    const float2 q0 = *reinterpret_cast<const float2 *>(gsrc + (rr + 2) * pitch + 2);
                    const float2 q1 = *reinterpret_cast<const float2 *>(gsrc + (rr + 2) * pitch + 4);
                    d[rr][0] = q0.x; d[rr][1] = q0.y; d[rr][2] = q1.x; d[rr][3] = q1.y;
                }
                if (rlim < TH || clim < 4) {  // padded tile: what lies beyond this window's grid belongs to its neighbour
#pragma unroll
                    for (int rr = 0; rr < TH; ++rr)
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc)
                            if (rr >= rlim || cc >= clim) d[rr][cc] = 0.f;
                }
                if (cls == 0) {
#pragma unroll
                    for (int rr = 0; rr < TH; ++rr)
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) gsum += d[rr][cc];
                }
                float4 n0 = *reinterpret_cast<const float4 *>(asrc);
                float4 n1 = *reinterpret_cast<const float4 *>(asrc + 4);
#pragma unroll
                for (int rr = 0; rr < TH + 4; ++rr) {
                    const float in[8] = {n0.x, n0.y, n0.z, n0.w, n1.x, n1.y, n1.z, n1.w};
                    if (rr + 1 < TH + 4) {
                        n0 = *reinterpret_cast<const float4 *>(asrc + (rr + 1) * pitch);
                        n1 = *reinterpret_cast<const float4 *>(asrc + (rr + 1) * pitch + 4);
                    }
#pragma unroll
                    for (int uu = 0; uu < 5; ++uu) {
                        const int dr = rr - uu;
                        if (dr >= 0 && dr < TH) {
#pragma unroll
                            for (int v = 0; v < 5; ++v)
#pragma unroll
                                for (int cc = 0; cc < 4; ++cc) accw[uu * 5 + v] = fmaf(d[dr][cc], in[cc + v], accw[uu * 5 + v]);
                        }
                    }
                }
                float wr[KK];
                plane::load_weights(sm + item.wt, wr);
                plane::conv_tile<TH>(gsrc, pitch, wr, acc);
            } else {
                float wr[KK];
                plane::load_weights(sm + item.wt, wr);
                plane::conv_tile<TH>(asrc, pitch, wr, acc);
            }
            if (item.z >= 0) {
                const int zp = (item.meta >> 10) & 0x3ff, zleft = (item.meta >> 20) & 0xf;
                float *z = sm + item.z;
#pragma unroll
                for (int r = 0; r < TH; ++r)
                    if (r < zleft) *reinterpret_cast<float4 *>(z + r * zp) = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
            }
        }
        const float bias = BWD ? 0.f : wtab[KK];
        __syncthreads();
        if (has_base) {
            const size_t plane_idx = (size_t)b * g.C + c;
            T *oplane = out + plane_idx * w.H * w.W;
#pragma unroll
            for (int hb = 0; hb < TH / 4; ++hb) {
                const int t4 = (TH / 4) * tyy + hb;
                const int Y0 = oy + 4 * t4, X0 = ox + 4 * txx;
                float deep = bias;
                if (add && Y0 < w.H && X0 < w.W) deep += 0.25f * __ldg(add + plane_idx * w.H2 * w.W2 + (size_t)(Y0 >> 2) * w.W2 + (X0 >> 2));
                plane::synth_block(sm, g, t4, txx, deep, &acc[4 * hb]);
                const bool vec = (w.W & 3) == 0 && X0 + 3 < w.W;
#pragma unroll
                for (int r = 0; r < 4; ++r)
                    if (Y0 + r < w.H && X0 < w.W) plane::store_row4(oplane + (size_t)(Y0 + r) * w.W + X0, X0, w.W, vec, acc[4 * hb + r]);
            }
        }
        const bool last_of_channel = BWD && ((u + 1 == u_end) || cn != c);
        if (last_of_channel) {
            // block tree through shared memory (the arrays are idle): park every thread's sums, then one thread per
            // (class, tap) adds the threads of its class in index order
            __syncthreads();
            float *scr = sm;
#pragma unroll
            for (int t = 0; t < KK; ++t) scr[tid * (KK + 2) + t] = accw[t];
            scr[tid * (KK + 2) + KK] = gsum;
            scr[tid * (KK + 2) + KK + 1] = __int_as_float(item.meta < 0 ? cls : -1);
            __syncthreads();
            const long long first_unit = (long long)c * g.B * nwin;
            const int slotp = blockIdx.x - (int)(((first_unit + 1) * gridDim.x - 1) / w.units);
            for (int e = tid; e < ncls * (KK + 1); e += nthr) {
                const int c2 = e / (KK + 1), t = e - c2 * (KK + 1);
                if (c2 > 0 && t == KK) continue;
                float sacc = 0.f;
                for (int th = 0; th < nthr; ++th)
                    if (__float_as_int(scr[th * (KK + 2) + KK + 1]) == c2) sacc += scr[th * (KK + 2) + t];
                if (c2 == 0) {
                    part0[((size_t)c * g.np + slotp) * (KK + 1) + t] = sacc;
                } else {
                    const int l = (c2 - 1) >> 2, sb_ = (c2 - 1) & 3;
                    partl[(size_t)l * g.C * g.np * 4 * KK + (((size_t)c * g.np + slotp) * 4 + sb_) * KK + t] = sacc;
                }
            }
#pragma unroll
            for (int t = 0; t < KK; ++t) accw[t] = 0.f;
            gsum = 0.f;
            __syncthreads();  // the scratch is overwritten by the next window's staging only after everybody has read it
        }
        c = cn; b = bn; wy = wyn; wx = wxn;
        buf ^= 1;
    }
    cp_async_wait<0>();
}

// ------------------------------------------------------------------ host side
inline bool make_plan(int B, int C, int H, int W, int L, int esz, bool bwd, WGeom &w) {
    w = WGeom{};
    const int Lc = L < 2 ? L : 2;
    w.H = H; w.W = W; w.L = L; w.esz = esz;
    w.hp = Lc == 2 ? 8 : 4;
    // windows: as few as possible per plane, every level tile its own thread (<= 256 tiles), rows a multiple of 8
    bool found = false;
    double best = 1e30;
    for (int WH = 16; WH <= 64; WH += 8)
        for (int WW = 16; WW <= 64; WW += 16) {
            Geom g = {};
            plane::fill_common(g, B, C, WH, WW, Lc, esz, TH);
            const int slot = plane::layout_slot(g, bwd, true);
            const int ntiles = g.lvl_start[Lc + 1] + g.nbase;
            if (ntiles > 256) continue;
            const int nwy = (H + WH - 1) / WH, nwx = (W + WW - 1) / WW;
            const int RH = WH + 2 * w.hp, RW = WW + 2 * w.hp;
            const int rawp = ((RW * esz + 15) / 16 + 1) * 16;
            const int tensors = bwd ? 2 : 1;
            const int wtab = (1 + 4 * Lc) * WT_STRIDE;
            long long scratch = (long long)256 * (KK + 2);
            long long arrays = slot > scratch ? slot : scratch;
            for (int nbuf = 2; nbuf >= 1; --nbuf) {
                const long long floats = plane::pad4((int)arrays) + plane::pad4(wtab) + (long long)nbuf * tensors * RH * rawp / 4 + 16;
                const long long bytes = floats * 4;
                if (2 * (bytes + 1024) > plane::SMEM_PER_SM && !(nbuf == 1 && bytes <= plane::SMEM_LIMIT)) continue;
                int bps = 2 * (bytes + 1024) <= plane::SMEM_PER_SM ? 2 : 1;
                if (!bwd && 3 * (bytes + 1024) <= plane::SMEM_PER_SM) bps = 3;
                // cost: tile slots issued per useful pixel, the halo's share of staging, idle threads, resident blocks
                const double cover = (double)nwy * WH * nwx * WW / ((double)H * W);
                const double halo = (double)RH * RW / ((double)WH * WW);
                const double thr = 256.0 / ntiles;
                const double cost = cover * (1.0 + 0.15 * halo) * (0.7 + 0.3 * thr) * (bps >= 2 ? 1.0 : 1.6) * (nbuf == 2 ? 1.0 : 1.1);
                if (cost < best) {
                    best = cost;
                    found = true;
                    w.g = g;
                    w.g.NPL = 1; w.g.slot_stride = slot; w.g.bulk = 0;
                    w.g.wtab_off = plane::pad4((int)arrays);
                    w.raw_off = w.g.wtab_off + plane::pad4(wtab);
                    w.g.smem_floats = (int)floats;
                    w.g.nthreads = (ntiles + 31) & ~31;
                    w.g.blocks_per_sm = bps;
                    w.WH = WH; w.WW = WW; w.nwy = nwy; w.nwx = nwx;
                    w.RH = RH; w.RW = RW; w.rawp = rawp; w.nbuf = nbuf; w.raw_bytes = tensors * RH * rawp;
                    w.npy = RH / 4; w.npx = RW / 4;
                }
                break;  // two buffers fit: no need to look at one
            }
        }
    if (!found) return false;
    if (w.npy * w.npx > 2 * w.g.nthreads) return false;  // two staging patches per thread
    // every fetched row starts at element (plane, y, ox - hp): on a 16-byte boundary if all four strides are
    w.aligned = ((long long)W * esz) % 16 == 0 && ((long long)H * W * esz) % 16 == 0 && (w.WW * esz) % 16 == 0 && (w.hp * esz) % 16 == 0;
    w.H2 = (H + 3) / 4; w.W2 = (W + 3) / 4;
    w.units = (long long)C * B * w.nwy * w.nwx;
    long long nb = (long long)plane::NUM_SMS * w.g.blocks_per_sm;
    if (nb > w.units) nb = w.units;
    w.g.nblocks = (int)nb;
    // partial slots: blocks that share a channel
    const long long per_ch = (long long)B * w.nwy * w.nwx;
    int np = 1;
    for (int ch = 0; ch < C; ++ch) {
        const int first = (int)((((long long)ch * per_ch + 1) * nb - 1) / w.units);
        const int last = (int)((((long long)(ch + 1) * per_ch) * nb - 1) / w.units);
        if (last - first + 1 > np) np = last - first + 1;
    }
    w.g.np = np;
    return true;
}

// The deep part (levels >= 3) runs on the whole-plane kernels over the carrier; it must be supported there.
inline bool supported(int B, int C, int H, int W, int k, int L, int dtype) {
    if (k != 5) return false;
    WGeom w;
    const int esz = plane::dtype_bytes(dtype);
    if (!make_plan(B, C, H, W, L, esz, false, w) || !make_plan(B, C, H, W, L, esz, true, w)) return false;
    if (L > 2 && !plane::supported((H + 3) / 4, (W + 3) / 4, 5, L - 2, 0)) return false;
    return true;
}

// Workspace layout (both directions): [window partials: base + levels 1-2][X2][R3 / gX2][zero base weights][unit
// scales][G2][workspace of the whole-plane kernels, whose first word is their status word]
struct WsPlan {
    size_t part0, partl, X2, G2, R3, zeros, ones, deep, parts_end, fwd_bytes, bwd_bytes;
    int np;
};
inline size_t al(size_t v) { return (v + 255) / 256 * 256; }
inline WsPlan ws_plan(int B, int C, int H, int W, int L, int esz) {
    WsPlan p = {};
    WGeom wb;
    make_plan(B, C, H, W, L, esz, true, wb);
    const int Lc = L < 2 ? L : 2, H2 = (H + 3) / 4, W2 = (W + 3) / 4;
    const size_t S2 = (size_t)B * C * H2 * W2 * sizeof(float);
    size_t off = 0;
    p.np = wb.g.np;
    p.part0 = off; off = al(off + sizeof(float) * (size_t)C * wb.g.np * (KK + 1));
    p.partl = off; off = al(off + sizeof(float) * (size_t)Lc * C * wb.g.np * 4 * KK);
    p.parts_end = off;
    if (L > 2) {
        p.X2 = off; off = al(off + S2);
        p.R3 = off; off = al(off + S2);
        p.zeros = off; off = al(off + sizeof(float) * (size_t)C * KK);
        p.ones = off; off = al(off + sizeof(float) * (size_t)C);
        p.G2 = off; off = al(off + S2);
        p.deep = off;
        p.fwd_bytes = off + al(plane::forward_workspace_bytes(B, C, H2, W2, L - 2));
        p.bwd_bytes = off + al(plane::backward_workspace_bytes(B, C, H2, W2, L - 2, 4));
    } else {
        p.fwd_bytes = 256;
        p.bwd_bytes = off > 256 ? off : 256;
    }
    return p;
}

static __global__ void fill_f32_kernel(float *p, float v, size_t n) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) p[e] = v;
}

template <typename T, bool BWD>
cudaError_t launch_window(const WGeom &w, const T *x, const T *go, const float *w0, const float *s0, const float *b0, const float *wl,
                          const float *sl, const float *add, T *out, float *part0, float *partl, cudaStream_t st) {
    cudaError_t e;
    const size_t total = (size_t)w.g.B * w.g.C * w.H * w.W * sizeof(T);
    if (!BWD && w.g.blocks_per_sm >= 3) {
        constexpr auto kern = window_kernel<T, BWD, 3>;
        if ((e = plane::opt_in_smem<kern>()) != cudaSuccess) return e;
        kern<<<w.g.nblocks, w.g.nthreads, (size_t)w.g.smem_floats * 4, st>>>(w, x, go, w0, s0, b0, wl, sl, add, out, part0, partl, total);
    } else {
        constexpr auto kern = window_kernel<T, BWD, 2>;
        if ((e = plane::opt_in_smem<kern>()) != cudaSuccess) return e;
        kern<<<w.g.nblocks, w.g.nthreads, (size_t)w.g.smem_floats * 4, st>>>(w, x, go, w0, s0, b0, wl, sl, add, out, part0, partl, total);
    }
    return cudaGetLastError();
}

template <typename T>
cudaError_t forward(int B, int C, int H, int W, int L, const T *x, const float *w0, const float *s0, const float *b0,
                    const float *wl, const float *sl, T *out, char *ws, cudaStream_t st, unsigned tag) {
    WGeom w;
    if (!make_plan(B, C, H, W, L, (int)sizeof(T), false, w)) return cudaErrorInvalidValue;
    const WsPlan p = ws_plan(B, C, H, W, L, (int)sizeof(T));
    const float *add = nullptr;
    cudaError_t e;
    if (L > 2) {
        const size_t P = (size_t)B * C, n2 = P * w.H2 * w.W2;
        float *X2 = reinterpret_cast<float *>(ws + p.X2), *R3 = reinterpret_cast<float *>(ws + p.R3);
        float *zeros = reinterpret_cast<float *>(ws + p.zeros), *ones = reinterpret_cast<float *>(ws + p.ones);
        carrier_kernel<T><<<(unsigned)((n2 + 255) / 256), 256, 0, st>>>(x, H, W, w.H2, w.W2, P, X2);
        if ((e = cudaMemsetAsync(zeros, 0, sizeof(float) * (size_t)C * KK, st)) != cudaSuccess) return e;
        fill_f32_kernel<<<(C + 255) / 256, 256, 0, st>>>(ones, 1.f, (size_t)C);
        // levels 3..L of x are levels 1..L-2 of the carrier; its base path is switched off by zero weights
        if ((e = plane::forward<float>(B, C, w.H2, w.W2, L - 2, X2, zeros, ones, nullptr, wl + (size_t)2 * C * 4 * KK, sl + (size_t)2 * C * 4,
                                       R3, ws + p.deep, st, tag, 0, false)) != cudaSuccess)
            return e;
        add = R3;
    }
    return launch_window<T, false>(w, x, nullptr, w0, s0, b0, wl, sl, add, out, nullptr, nullptr, st);
}

template <typename T>
cudaError_t backward(int B, int C, int H, int W, int L, const T *x, const T *go, const float *w0, const float *s0,
                     const float *wl, const float *sl, T *gx, char *ws, EpiloguePtrs *ep, cudaStream_t st, unsigned tag) {
    WGeom w;
    if (!make_plan(B, C, H, W, L, (int)sizeof(T), true, w)) return cudaErrorInvalidValue;
    const WsPlan p = ws_plan(B, C, H, W, L, (int)sizeof(T));
    const int Lc = L < 2 ? L : 2;
    float *part0 = reinterpret_cast<float *>(ws + p.part0), *partl = reinterpret_cast<float *>(ws + p.partl);
    cudaError_t e;
    if ((e = cudaMemsetAsync(ws + p.part0, 0, p.parts_end, st)) != cudaSuccess) return e;  // unwritten partial slots read as zero
    const float *add = nullptr;
    if (L > 2) {
        const size_t P = (size_t)B * C, n2 = P * w.H2 * w.W2;
        float *X2 = reinterpret_cast<float *>(ws + p.X2), *G2 = reinterpret_cast<float *>(ws + p.G2), *gX2 = reinterpret_cast<float *>(ws + p.R3);
        float *zeros = reinterpret_cast<float *>(ws + p.zeros), *ones = reinterpret_cast<float *>(ws + p.ones);
        carrier_kernel<T><<<(unsigned)((n2 + 255) / 256), 256, 0, st>>>(x, H, W, w.H2, w.W2, P, X2);
        carrier_kernel<T><<<(unsigned)((n2 + 255) / 256), 256, 0, st>>>(go, H, W, w.H2, w.W2, P, G2);
        if ((e = cudaMemsetAsync(zeros, 0, sizeof(float) * (size_t)C * KK, st)) != cudaSuccess) return e;
        fill_f32_kernel<<<(C + 255) / 256, 256, 0, st>>>(ones, 1.f, (size_t)C);
        EpiloguePtrs deep = {};
        char *deep_ws = ws + p.deep;
        // the epilogue reads every slot of the merged partial sums: the slots the carrier's kernels do not write are zero
        if ((e = cudaMemsetAsync(deep_ws, 0, plane::backward_workspace_bytes(B, C, w.H2, w.W2, L - 2, 4), st)) != cudaSuccess) return e;
        if ((e = plane::backward<float>(B, C, w.H2, w.W2, L - 2, X2, G2, zeros, ones, wl + (size_t)2 * C * 4 * KK, sl + (size_t)2 * C * 4, gX2,
                                        deep_ws, &deep, st, tag, 0, false)) != cudaSuccess)
            return e;
        for (int l = 2; l < L; ++l) { ep->partl[l] = deep.partl[l - 2]; ep->npl[l] = deep.npl[l - 2]; }
        add = gX2;
    }
    if ((e = launch_window<T, true>(w, x, go, w0, s0, nullptr, wl, sl, add, gx, part0, partl, st)) != cudaSuccess) return e;
    ep->part0 = part0;
    ep->np0 = w.g.np;
    for (int l = 0; l < Lc; ++l) { ep->partl[l] = partl + (size_t)l * C * w.g.np * 4 * KK; ep->npl[l] = w.g.np; }
    return cudaSuccess;
}

#define WT_WINDOW_INSTANTIATE(T, EXTERN)                                                                                   \
    EXTERN template cudaError_t forward<T>(int, int, int, int, int, const T *, const float *, const float *, const float *, \
                                           const float *, const float *, T *, char *, cudaStream_t, unsigned);             \
    EXTERN template cudaError_t backward<T>(int, int, int, int, int, const T *, const T *, const float *, const float *,    \
                                            const float *, const float *, T *, char *, EpiloguePtrs *, cudaStream_t,       \
                                            unsigned);

}  // namespace window
}  // namespace wt
