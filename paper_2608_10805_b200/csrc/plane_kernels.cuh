// Whole-plane WTConv kernels for sm_100a (k = 5): every (b, c) plane's entire decomposition lives
// in shared memory, so the only HBM traffic is the compulsory one (read x, write out).
//
// Design
//  * A block works on PAIRS of planes (channels 2cp and 2cp+1 of the same image).  Every shared
//    array holds float2 {plane A, plane B} per element and every multiply-add is a packed
//    fma.rn.f32x2 whose weight operand is {w_A, w_B}: the FP32 pipe takes two FMAs per issued
//    instruction, which leaves issue slots for the shared-memory loads.
//  * Per work unit (a channel pair and a group of NPP images): stage x into a zero-haloed array
//    and run the Haar butterfly of Eq. 5 on chip (Sec. 4.1), level by level from the raw LL band;
//    then every thread convolves 4x4 output tiles straight out of shared memory with weights that
//    already carry the scale (Eq. 8); a thread keeps its base-conv tile in registers across one
//    barrier and then adds the bit-indexed closed-form synthesis of Proposition 2 (Sec. 4.2)
//    before the only global store.
//  * Backward = two kernels.  grad_x is the same kernel run on grad_out with the kernels rotated
//    by 180 degrees (Sec. 2.2: the adjoint of analysis is synthesis and vice versa, so the adjoint
//    of the whole operator has the operator's own structure).  The weight-gradient kernel stages
//    the decompositions of x and grad_out and correlates them tile by tile; each thread only ever
//    works on one (level, subband) class, so its 25 packed accumulators stay in registers across
//    all images of a channel pair and are reduced once (block tree through shared memory, then
//    fixed-order fp64 in the epilogue).
#pragma once
#include "common.cuh"
#include "tiled_kernels.cuh"

namespace wt {
namespace plane {

typedef unsigned long long u64;
constexpr int MAXL = 8;
constexpr int KK = 25;
constexpr int MAX_THREADS = 512;
constexpr int NUM_SMS = 148;                 // planning constant (B200); plans must not depend on the device
constexpr int SMEM_LIMIT = 227 * 1024;       // opt-in dynamic shared memory per block
constexpr int SMEM_PER_SM = 228 * 1024;      // per SM, 1 KB reserved per resident block

// ------------------------------------------------------------------ packed fp32x2 helpers
__device__ __forceinline__ u64 pk(float lo, float hi) {
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void upk(u64 v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 fma2(u64 a, u64 b, u64 c) {
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ u64 add2(u64 a, u64 b) {
    u64 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ u64 sub2(u64 a, u64 b) {
    u64 d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ u64 mul2(u64 a, u64 b) {
    u64 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// Packed Eq. 5 on {A,B} pairs.
struct Haar4x2 {
    u64 ll, lh, hl, hh;
};
__device__ __forceinline__ Haar4x2 haar2(u64 a, u64 b, u64 c, u64 d) {
    const u64 half = pk(0.5f, 0.5f);
    u64 s0 = add2(a, b), s1 = add2(c, d), d0 = sub2(a, b), d1 = sub2(c, d);
    Haar4x2 r;
    r.ll = mul2(half, add2(s0, s1));
    r.lh = mul2(half, sub2(s0, s1));
    r.hl = mul2(half, add2(d0, d1));
    r.hh = mul2(half, sub2(d0, d1));
    return r;
}

// ------------------------------------------------------------------ geometry (host-planned, passed by value)
// Division by a launch-invariant divisor as multiply-high: exact while dividend * divisor < 2^32.
struct FastDiv {
    unsigned mul, d;
};
inline FastDiv make_fastdiv(int d) {
    FastDiv f;
    f.d = (unsigned)(d < 1 ? 1 : d);
    f.mul = (unsigned)(0x100000000ULL / f.d) + 1u;
    return f;
}
__device__ __forceinline__ int fdiv(int e, const FastDiv &f) { return f.d == 1 ? e : (int)__umulhi((unsigned)e, f.mul); }

struct Geom {
    int B, C, H, W, L;
    int Hl[MAXL + 1], Wl[MAXL + 1];        // level grids, index 0 = input
    int rows[MAXL + 1], pitch[MAXL + 1];   // haloed arrays: pad4(Hl)+4 rows, pitch pad4(Wl)+4 (units of float2)
    int offA[MAXL + 1];                    // slot-relative offset of x (l=0) / Y^l subband 0 (subband stride rows*pitch)
    int offG[MAXL + 1];                    // same for grad_out / D^l (weight-gradient kernel only)
    int zrows[MAXL + 1], zpitch[MAXL + 1]; // conv outputs Z^l (forward kernel only)
    int offZ[MAXL + 1];
    int slot_stride;                       // float2 per plane-pair slot
    int NPP;                               // plane-pair slots per work unit
    int tx[MAXL + 1], ty[MAXL + 1];        // 4x4 tiles per level grid (index 0 = base)
    int lvl_start[MAXL + 2];               // per pair: first level-item of level l (1..L); [L+1] = count
    int nbase;                             // base tiles per pair
    int wtab_off;                          // offset of the folded weight table [(1+4L)][26] float2 (+ bias entry)
    int smem_u64;                          // shared memory in float2 units
    int bgroups, ncp, units;               // work units = ncp channel pairs x bgroups image groups
    int nthreads, nblocks, blocks_per_sm;
    int vec;                               // 1: W % 4 == 0, rows can be staged with 4-element vector loads
    int npatch;                            // staging work items per pair (vec: 2x4 pixel patches, else 2x2 blocks)
    FastDiv d_npatch, d_prow;              // / npatch, / (patches per patch-row)
    FastDiv d_lvl[MAXL + 1], d_lvlw[MAXL + 1];  // / (Hl*Wl), / Wl   (levels >= 2 staging)
    FastDiv d_nlv, d_nt[MAXL + 1], d_tx[MAXL + 1], d_nbase;
    // weight-gradient kernel: class-major thread allocation and partial-sum slots
    int thr_start[4 * MAXL + 2];
    int np;
    double score;
};

__host__ __device__ inline int pad4(int n) { return (n + 3) & ~3; }

// Block containing unit v when `units` are split into `nb` contiguous ranges [iU/nb, (i+1)U/nb).
__host__ __device__ inline int block_of_unit(long long v, int nb, int units) {
    return (int)(((v + 1) * nb - 1) / units);
}

// Shared-memory layout of a haloed array row (pitch float2, pitch % 4 == 0): the 16-byte chunks
// (two float2) of a row are de-interleaved, even chunks in the first half of the row and odd chunks in
// the second.  A thread's 4x4 tile window starts at column 4*tx, so lanes of a warp read chunk
// 2*tx + j: for fixed j consecutive lanes hit consecutive 16-byte words - no bank conflicts.
__device__ __forceinline__ int phys_col(int col, int half) {
    return ((col >> 1) & 1) * half + ((col >> 2) << 1) + (col & 1);
}

constexpr int WT_STRIDE = 26;  // float2 per class in the weight table (25 taps, padded to 16 bytes)

// ------------------------------------------------------------------ shared device pieces
__device__ __forceinline__ void build_weight_table(u64 *wtab, const Geom &g, int cA, bool hasB, bool flip,
                                                   const float *__restrict__ w0, const float *__restrict__ s0,
                                                   const float *__restrict__ b0, const float *__restrict__ wl,
                                                   const float *__restrict__ sl) {
    const int ncls = 1 + 4 * g.L, cB = cA + 1;
    for (int e = threadIdx.x; e < ncls * KK; e += blockDim.x) {
        const int cls = e / KK, t = e - cls * KK, src = flip ? (KK - 1 - t) : t;
        float wa, wb = 0.f;
        if (cls == 0) {
            wa = __ldg(w0 + cA * KK + src) * __ldg(s0 + cA);
            if (hasB) wb = __ldg(w0 + cB * KK + src) * __ldg(s0 + cB);
        } else {
            const int l = (cls - 1) >> 2, sub = (cls - 1) & 3;
            const size_t ia = ((size_t)l * g.C + cA) * 4 + sub, ib = ((size_t)l * g.C + cB) * 4 + sub;
            wa = __ldg(wl + ia * KK + src) * __ldg(sl + ia);
            if (hasB) wb = __ldg(wl + ib * KK + src) * __ldg(sl + ib);
        }
        wtab[cls * WT_STRIDE + t] = pk(wa, wb);  // Eq. 8: scale folded into the weight
    }
    if (threadIdx.x == 0) {
        float ba = 0.f, bb = 0.f;
        if (b0) {
            ba = __ldg(s0 + cA) * __ldg(b0 + cA);
            if (hasB) bb = __ldg(s0 + cB) * __ldg(b0 + cB);
        }
        wtab[KK] = pk(ba, bb);  // the spare 26th entry of class 0
    }
}

__device__ __forceinline__ void load_weights(const u64 *wt, u64 (&w)[KK]) {
    const ulonglong2 *q = reinterpret_cast<const ulonglong2 *>(wt);
#pragma unroll
    for (int t = 0; t < 12; ++t) {
        const ulonglong2 v = q[t];
        w[2 * t] = v.x;
        w[2 * t + 1] = v.y;
    }
    w[24] = wt[24];
}

template <typename T>
__device__ __forceinline__ void load4(const T *p, float (&v)[4]);
template <>
__device__ __forceinline__ void load4<float>(const float *p, float (&v)[4]) {
    const float4 q = __ldg(reinterpret_cast<const float4 *>(p));
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}
template <>
__device__ __forceinline__ void load4<__half>(const __half *p, float (&v)[4]) {
    const uint2 q = __ldg(reinterpret_cast<const uint2 *>(p));
    const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&q.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2 *>(&q.y));
    v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
}
template <>
__device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16 *p, float (&v)[4]) {
    const uint2 q = __ldg(reinterpret_cast<const uint2 *>(p));
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&q.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&q.y));
    v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
}

// Stage the planes of one unit: x into the haloed array `off[0]` and its level-1 Haar subbands (Eq. 5)
// into `off[1]`, both planes of each pair interleaved.  Pixels beyond H x W are never written and stay
// zero (odd-size padding and conv halo); images beyond the batch are written as zeros.
template <typename T>
__device__ __forceinline__ void stage_input(u64 *sm, const Geom &g, const int *off, const T *__restrict__ x, int cA,
                                            bool hasB, int bg) {
    const int H = g.H, W = g.W;
    const size_t HW = (size_t)H * W;
    const int p0 = g.pitch[0], h0 = p0 >> 1;
    if (g.L == 0) {
        for (int e = threadIdx.x; e < g.NPP * H * W; e += blockDim.x) {
            const int slot = e / (H * W), r = e - slot * (H * W), y = r / W, xx = r - y * W;
            const int b = bg * g.NPP + slot;
            float va = 0.f, vb = 0.f;
            if (b < g.B) {
                const T *pa = x + ((size_t)b * g.C + cA) * HW + r;
                va = ldf(pa);
                if (hasB) vb = ldf(pa + HW);
            }
            sm[(size_t)slot * g.slot_stride + off[0] + (y + 2) * p0 + phys_col(xx + 2, h0)] = pk(va, vb);
        }
        return;
    }
    const int p1 = g.pitch[1], h1 = p1 >> 1, sub1 = g.rows[1] * p1;
    if (g.vec) {
        // work item = 2 rows x 4 columns of both planes: two Haar blocks, whole 16-byte chunks everywhere
        for (int e = threadIdx.x; e < g.NPP * g.npatch; e += blockDim.x) {
            const int slot = fdiv(e, g.d_npatch), r = e - slot * g.npatch;
            const int i = fdiv(r, g.d_prow), q = r - i * (int)g.d_prow.d;
            const int b = bg * g.NPP + slot, y = 2 * i;
            const bool y1 = y + 1 < H;
            float a0[4] = {0.f, 0.f, 0.f, 0.f}, a1[4] = {0.f, 0.f, 0.f, 0.f}, b0[4] = {0.f, 0.f, 0.f, 0.f},
                  b1[4] = {0.f, 0.f, 0.f, 0.f};
            if (b < g.B) {
                const T *pa = x + ((size_t)b * g.C + cA) * HW + (size_t)y * W + 4 * q;
                load4<T>(pa, a0);
                if (y1) load4<T>(pa + W, a1);
                if (hasB) {
                    load4<T>(pa + HW, b0);
                    if (y1) load4<T>(pa + HW + W, b1);
                }
            }
            u64 *S = sm + (size_t)slot * g.slot_stride;
            u64 r0v[4], r1v[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                r0v[c] = pk(a0[c], b0[c]);
                r1v[c] = pk(a1[c], b1[c]);
            }
            // columns 4q+2 .. 4q+5 = chunk 2q+1 (odd half, index q) and chunk 2q+2 (even half, index q+1)
            u64 *X = S + off[0] + (y + 2) * p0;
            *reinterpret_cast<ulonglong2 *>(X + h0 + 2 * q) = make_ulonglong2(r0v[0], r0v[1]);
            *reinterpret_cast<ulonglong2 *>(X + 2 * q + 2) = make_ulonglong2(r0v[2], r0v[3]);
            if (y1) {
                *reinterpret_cast<ulonglong2 *>(X + p0 + h0 + 2 * q) = make_ulonglong2(r1v[0], r1v[1]);
                *reinterpret_cast<ulonglong2 *>(X + p0 + 2 * q + 2) = make_ulonglong2(r1v[2], r1v[3]);
            }
            const Haar4x2 ha = haar2(r0v[0], r0v[1], r1v[0], r1v[1]), hb = haar2(r0v[2], r0v[3], r1v[2], r1v[3]);
            // level-1 columns 2q+2, 2q+3 = chunk q+1
            u64 *Y = S + off[1] + (i + 2) * p1 + ((q + 1) & 1) * h1 + ((q + 1) >> 1) * 2;
            *reinterpret_cast<ulonglong2 *>(Y) = make_ulonglong2(ha.ll, hb.ll);
            *reinterpret_cast<ulonglong2 *>(Y + sub1) = make_ulonglong2(ha.lh, hb.lh);
            *reinterpret_cast<ulonglong2 *>(Y + 2 * sub1) = make_ulonglong2(ha.hl, hb.hl);
            *reinterpret_cast<ulonglong2 *>(Y + 3 * sub1) = make_ulonglong2(ha.hh, hb.hh);
        }
        return;
    }
    // general path: one 2x2 block per work item, scalar loads
    const int W1 = g.Wl[1];
    for (int e = threadIdx.x; e < g.NPP * g.npatch; e += blockDim.x) {
        const int slot = fdiv(e, g.d_npatch), r = e - slot * g.npatch;
        const int i = fdiv(r, g.d_prow), j = r - i * W1;
        const int b = bg * g.NPP + slot, y = 2 * i, xx = 2 * j;
        const bool x1 = xx + 1 < W, y1 = y + 1 < H;
        float aA = 0.f, bA = 0.f, cA_ = 0.f, dA = 0.f, aB = 0.f, bB = 0.f, cB_ = 0.f, dB = 0.f;
        if (b < g.B) {
            const T *pa = x + ((size_t)b * g.C + cA) * HW + (size_t)y * W + xx;
            aA = ldf(pa);
            if (x1) bA = ldf(pa + 1);
            if (y1) cA_ = ldf(pa + W);
            if (x1 && y1) dA = ldf(pa + W + 1);
            if (hasB) {
                const T *pb = pa + HW;
                aB = ldf(pb);
                if (x1) bB = ldf(pb + 1);
                if (y1) cB_ = ldf(pb + W);
                if (x1 && y1) dB = ldf(pb + W + 1);
            }
        }
        u64 *S = sm + (size_t)slot * g.slot_stride;
        u64 *X = S + off[0] + (y + 2) * p0 + phys_col(xx + 2, h0);  // xx even: xx+2, xx+3 share a chunk
        const u64 a = pk(aA, aB), bq = pk(bA, bB), c = pk(cA_, cB_), d = pk(dA, dB);
        X[0] = a;
        if (x1) X[1] = bq;
        if (y1) X[p0] = c;
        if (x1 && y1) X[p0 + 1] = d;
        const Haar4x2 h = haar2(a, bq, c, d);
        u64 *Y = S + off[1] + (i + 2) * p1 + phys_col(j + 2, h1);
        Y[0] = h.ll;
        Y[sub1] = h.lh;
        Y[2 * sub1] = h.hl;
        Y[3 * sub1] = h.hh;
    }
}

// Level l >= 2 from the raw LL band of level l-1 (already in shared memory).  Reads one element past
// an odd grid land in the zero padding.
__device__ __forceinline__ void stage_level(u64 *sm, const Geom &g, const int *off, int l) {
    const int Wl = g.Wl[l], n = (int)g.d_lvl[l].d;
    const int pp = g.pitch[l - 1], hp = pp >> 1, pl = g.pitch[l], hl = pl >> 1, subl = g.rows[l] * pl;
    for (int e = threadIdx.x; e < g.NPP * n; e += blockDim.x) {
        const int slot = fdiv(e, g.d_lvl[l]), r = e - slot * n, i = fdiv(r, g.d_lvlw[l]), j = r - i * Wl;
        u64 *S = sm + (size_t)slot * g.slot_stride;
        const u64 *src = S + off[l - 1] + (2 * i + 2) * pp + phys_col(2 * j + 2, hp);  // even column: one chunk
        const ulonglong2 top = *reinterpret_cast<const ulonglong2 *>(src);
        const ulonglong2 bot = *reinterpret_cast<const ulonglong2 *>(src + pp);
        const Haar4x2 h = haar2(top.x, top.y, bot.x, bot.y);
        u64 *Y = S + off[l] + (i + 2) * pl + phys_col(j + 2, hl);
        Y[0] = h.ll;
        Y[subl] = h.lh;
        Y[2 * subl] = h.hl;
        Y[3 * subl] = h.hh;
    }
}

// 4x4 output tile of a 5x5 correlation.  `src` = array + (4*ty)*pitch + 2*tx points at the even-half
// word of the window's first chunk (the array's halo of 2 makes window row rr = output row + tap row);
// the window's four chunks per row are src[0..1], src[half..], src[2..3], src[half+2..].
__device__ __forceinline__ void conv_tile(const u64 *__restrict__ src, int pitch, const u64 (&w)[KK],
                                          u64 (&acc)[4][4]) {
    const int half = pitch >> 1;
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = 0ull;
#pragma unroll
    for (int rr = 0; rr < 8; ++rr) {
        const u64 *rp = src + rr * pitch;
        const ulonglong2 q0 = *reinterpret_cast<const ulonglong2 *>(rp);
        const ulonglong2 q1 = *reinterpret_cast<const ulonglong2 *>(rp + half);
        const ulonglong2 q2 = *reinterpret_cast<const ulonglong2 *>(rp + 2);
        const ulonglong2 q3 = *reinterpret_cast<const ulonglong2 *>(rp + half + 2);
        const u64 in[8] = {q0.x, q0.y, q1.x, q1.y, q2.x, q2.y, q3.x, q3.y};
#pragma unroll
        for (int u = 0; u < 5; ++u) {
            const int r = rr - u;
            if (r >= 0 && r < 4) {
#pragma unroll
                for (int v = 0; v < 5; ++v)
#pragma unroll
                    for (int c = 0; c < 4; ++c) acc[r][c] = fma2(w[u * 5 + v], in[c + v], acc[r][c]);
            }
        }
    }
}

// Decode a level item of one pair: r in [0, lvl_start[L+1]) -> (level, subband, tile row, tile col).
__device__ __forceinline__ void decode_level_item(const Geom &g, int r, int &l, int &sub, int &tyy, int &txx) {
    l = 1;
    while (r >= g.lvl_start[l + 1]) ++l;
    r -= g.lvl_start[l];
    sub = fdiv(r, g.d_nt[l]);
    r -= sub * (int)g.d_nt[l].d;
    tyy = fdiv(r, g.d_tx[l]);
    txx = r - tyy * g.tx[l];
}

template <typename T>
__device__ __forceinline__ void store_row4(T *__restrict__ p, int x0, int W, bool vec, float v0, float v1, float v2,
                                           float v3);
template <>
__device__ __forceinline__ void store_row4<float>(float *__restrict__ p, int x0, int W, bool vec, float v0, float v1,
                                                  float v2, float v3) {
    if (vec) {
        *reinterpret_cast<float4 *>(p) = make_float4(v0, v1, v2, v3);
    } else {
        if (x0 < W) p[0] = v0;
        if (x0 + 1 < W) p[1] = v1;
        if (x0 + 2 < W) p[2] = v2;
        if (x0 + 3 < W) p[3] = v3;
    }
}
template <>
__device__ __forceinline__ void store_row4<__half>(__half *__restrict__ p, int x0, int W, bool vec, float v0, float v1,
                                                   float v2, float v3) {
    if (vec) {
        __half2 a = __floats2half2_rn(v0, v1), b = __floats2half2_rn(v2, v3);
        uint2 q;
        q.x = *reinterpret_cast<unsigned *>(&a);
        q.y = *reinterpret_cast<unsigned *>(&b);
        *reinterpret_cast<uint2 *>(p) = q;
    } else {
        if (x0 < W) p[0] = __float2half_rn(v0);
        if (x0 + 1 < W) p[1] = __float2half_rn(v1);
        if (x0 + 2 < W) p[2] = __float2half_rn(v2);
        if (x0 + 3 < W) p[3] = __float2half_rn(v3);
    }
}
template <>
__device__ __forceinline__ void store_row4<__nv_bfloat16>(__nv_bfloat16 *__restrict__ p, int x0, int W, bool vec,
                                                          float v0, float v1, float v2, float v3) {
    if (vec) {
        __nv_bfloat162 a = __floats2bfloat162_rn(v0, v1), b = __floats2bfloat162_rn(v2, v3);
        uint2 q;
        q.x = *reinterpret_cast<unsigned *>(&a);
        q.y = *reinterpret_cast<unsigned *>(&b);
        *reinterpret_cast<uint2 *>(p) = q;
    } else {
        if (x0 < W) p[0] = __float2bfloat16_rn(v0);
        if (x0 + 1 < W) p[1] = __float2bfloat16_rn(v1);
        if (x0 + 2 < W) p[2] = __float2bfloat16_rn(v2);
        if (x0 + 3 < W) p[3] = __float2bfloat16_rn(v3);
    }
}

// ------------------------------------------------------------------ forward / input-gradient kernel
// FLIP = false: out = WTConv(x).  FLIP = true: the same dataflow on grad_out with every kernel rotated
// by 180 degrees and no bias gives grad_x.
template <typename T, bool FLIP>
__global__ void __launch_bounds__(MAX_THREADS, 1)
plane_fwd_kernel(const __grid_constant__ Geom g, const T *__restrict__ x, const float *__restrict__ w0,
                 const float *__restrict__ s0, const float *__restrict__ b0, const float *__restrict__ wl,
                 const float *__restrict__ sl, T *__restrict__ out) {
    extern __shared__ __align__(16) u64 sm[];
    const int tid = threadIdx.x, nthr = blockDim.x;
    for (int i = tid; i < g.smem_u64; i += nthr) sm[i] = 0ull;
    u64 *wtab = sm + g.wtab_off;
    const int L = g.L, nlv = g.lvl_start[L + 1];
    const size_t HW = (size_t)g.H * g.W;
    const int u_begin = (int)((long long)blockIdx.x * g.units / gridDim.x);
    const int u_end = (int)((long long)(blockIdx.x + 1) * g.units / gridDim.x);
    // this thread's base tile never changes: decode it once
    const int bi = nthr - 1 - tid;
    const bool has_base = bi < g.NPP * g.nbase;
    int bslot = 0, tyy = 0, txx = 0;
    if (has_base) {
        bslot = fdiv(bi, g.d_nbase);
        const int r = bi - bslot * g.nbase;
        tyy = fdiv(r, g.d_tx[0]);
        txx = r - tyy * g.tx[0];
    }
    const u64 *base_src = sm + (size_t)bslot * g.slot_stride + g.offA[0] + 4 * tyy * g.pitch[0] + 2 * txx;
    int cp_prev = -1;
    __syncthreads();
    for (int u = u_begin; u < u_end; ++u) {
        const int cp = u / g.bgroups, bg = u - cp * g.bgroups;
        const int cA = 2 * cp;
        const bool hasB = cA + 1 < g.C;
        if (cp != cp_prev) {  // units are channel-pair major: the table survives all images of a pair
            build_weight_table(wtab, g, cA, hasB, FLIP, w0, s0, FLIP ? nullptr : b0, wl, sl);
            cp_prev = cp;
        }
        stage_input<T>(sm, g, g.offA, x, cA, hasB, bg);
        __syncthreads();
        for (int l = 2; l <= L; ++l) {
            stage_level(sm, g, g.offA, l);
            __syncthreads();
        }
        // ---- level tiles: Z^l = Wfold^l (*) Y^l
        for (int it = tid; it < g.NPP * nlv; it += nthr) {
            const int slot = fdiv(it, g.d_nlv);
            int l, sub, ty2, tx2;
            decode_level_item(g, it - slot * nlv, l, sub, ty2, tx2);
            u64 *S = sm + (size_t)slot * g.slot_stride;
            const int pl = g.pitch[l];
            u64 w[KK];
            load_weights(wtab + (1 + (l - 1) * 4 + sub) * WT_STRIDE, w);
            u64 acc[4][4];
            conv_tile(S + g.offA[l] + sub * g.rows[l] * pl + 4 * ty2 * pl + 2 * tx2, pl, w, acc);
            const int zp = g.zpitch[l];
            u64 *z = S + g.offZ[l] + sub * g.zrows[l] * zp + 4 * ty2 * zp + 4 * tx2;
            const int zr_left = g.zrows[l] - 4 * ty2;
            const bool c0 = 4 * tx2 < zp, c1 = 4 * tx2 + 2 < zp;
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                if (r < zr_left) {
                    ulonglong2 *zr = reinterpret_cast<ulonglong2 *>(z + r * zp);
                    if (c0) zr[0] = make_ulonglong2(acc[r][0], acc[r][1]);
                    if (c1) zr[1] = make_ulonglong2(acc[r][2], acc[r][3]);
                }
            }
        }
        // ---- base tile (at most one per thread), kept in registers across the barrier
        u64 acc[4][4];
        u64 bias2 = 0ull;
        if (has_base) {
            u64 w[KK];
            load_weights(wtab, w);
            conv_tile(base_src, g.pitch[0], w, acc);
            bias2 = wtab[KK];
        }
        __syncthreads();
        if (has_base) {
            const u64 *S = sm + (size_t)bslot * g.slot_stride;
            // Proposition 2, level 1: coefficient (2ty+ci, 2tx+cj) feeds pixels (2ci+by, 2cj+bx) of the tile
            if (L >= 1) {
                const u64 half = pk(0.5f, 0.5f);
                const int zp = g.zpitch[1], zs = g.zrows[1] * zp;
                const u64 *z = S + g.offZ[1] + (2 * tyy) * zp + 2 * txx;
#pragma unroll
                for (int ci = 0; ci < 2; ++ci) {
                    const ulonglong2 ll = *reinterpret_cast<const ulonglong2 *>(z + ci * zp);
                    const ulonglong2 lh = *reinterpret_cast<const ulonglong2 *>(z + zs + ci * zp);
                    const ulonglong2 hl = *reinterpret_cast<const ulonglong2 *>(z + 2 * zs + ci * zp);
                    const ulonglong2 hh = *reinterpret_cast<const ulonglong2 *>(z + 3 * zs + ci * zp);
#pragma unroll
                    for (int cj = 0; cj < 2; ++cj) {
                        const u64 LLv = cj ? ll.y : ll.x, LHv = cj ? lh.y : lh.x, HLv = cj ? hl.y : hl.x,
                                  HHv = cj ? hh.y : hh.x;
                        const u64 pp = add2(LLv, LHv), pm = sub2(LLv, LHv), qp = add2(HLv, HHv), qm = sub2(HLv, HHv);
                        acc[2 * ci][2 * cj] = fma2(half, add2(pp, qp), acc[2 * ci][2 * cj]);
                        acc[2 * ci][2 * cj + 1] = fma2(half, sub2(pp, qp), acc[2 * ci][2 * cj + 1]);
                        acc[2 * ci + 1][2 * cj] = fma2(half, add2(pm, qm), acc[2 * ci + 1][2 * cj]);
                        acc[2 * ci + 1][2 * cj + 1] = fma2(half, sub2(pm, qm), acc[2 * ci + 1][2 * cj + 1]);
                    }
                }
            }
            if (L >= 2) {
                // levels >= 3: the whole tile sits in one quadrant of the coefficient's block
                u64 deep = bias2;
                float scale = 0.25f;
                for (int l = 3; l <= L; ++l) {
                    scale *= 0.5f;
                    const int zp = g.zpitch[l], zs = g.zrows[l] * zp;
                    const u64 *z = S + g.offZ[l] + (tyy >> (l - 2)) * zp + (txx >> (l - 2));
                    const float sy = ((tyy >> (l - 3)) & 1) ? -1.f : 1.f, sx = ((txx >> (l - 3)) & 1) ? -1.f : 1.f;
                    const u64 sy2 = pk(sy, sy), sx2 = pk(sx, sx);
                    const u64 p = fma2(sy2, z[zs], z[0]), q = fma2(sy2, z[3 * zs], z[2 * zs]);
                    deep = fma2(pk(scale, scale), fma2(sx2, q, p), deep);
                }
                // level 2: coefficient (ty, tx); pixel (r, c) of the tile takes signs from (r>>1, c>>1)
                const int zp = g.zpitch[2], zs = g.zrows[2] * zp;
                const u64 *z = S + g.offZ[2] + tyy * zp + txx;
                const u64 LLv = z[0], LHv = z[zs], HLv = z[2 * zs], HHv = z[3 * zs];
                const u64 pp = add2(LLv, LHv), pm = sub2(LLv, LHv), qp = add2(HLv, HHv), qm = sub2(HLv, HHv);
                const u64 quarter = pk(0.25f, 0.25f);
                u64 t2[2][2];
                t2[0][0] = fma2(quarter, add2(pp, qp), deep);
                t2[0][1] = fma2(quarter, sub2(pp, qp), deep);
                t2[1][0] = fma2(quarter, add2(pm, qm), deep);
                t2[1][1] = fma2(quarter, sub2(pm, qm), deep);
#pragma unroll
                for (int r = 0; r < 4; ++r)
#pragma unroll
                    for (int c = 0; c < 4; ++c) acc[r][c] = add2(acc[r][c], t2[r >> 1][c >> 1]);
            } else {
#pragma unroll
                for (int r = 0; r < 4; ++r)
#pragma unroll
                    for (int c = 0; c < 4; ++c) acc[r][c] = add2(acc[r][c], bias2);
            }
            const int b = bg * g.NPP + bslot;
            if (b < g.B) {
                T *oa = out + ((size_t)b * g.C + cA) * HW + (size_t)(4 * tyy) * g.W + 4 * txx;
                const bool vec = g.vec && (4 * txx + 3 < g.W);
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    if (4 * tyy + r < g.H) {
                        float a0, a1, a2, a3, b0_, b1, b2, b3;
                        upk(acc[r][0], a0, b0_);
                        upk(acc[r][1], a1, b1);
                        upk(acc[r][2], a2, b2);
                        upk(acc[r][3], a3, b3);
                        store_row4<T>(oa + (size_t)r * g.W, 4 * txx, g.W, vec, a0, a1, a2, a3);
                        if (hasB) store_row4<T>(oa + HW + (size_t)r * g.W, 4 * txx, g.W, vec, b0_, b1, b2, b3);
                    }
                }
            }
        }
        // The next unit's staging overwrites x / Y (last read before the barrier above) and possibly the
        // weight table (bias already copied to a register); Z is next written after the staging barriers.
    }
}

// ------------------------------------------------------------------ weight-gradient kernel
// dWfold^l[u,v] += sum_{i,j} D^l[i,j] Y^l[i+u-2, j+v-2] (and the base class with grad_out and x), Sec. 2.2.
// Thread t serves class cls(t) only (class-major allocation thr_start[]); accumulators persist over all
// units of a channel pair and are flushed to `part0` / `partl` when the pair changes.
template <typename T>
__global__ void __launch_bounds__(MAX_THREADS, 1)
plane_wgrad_kernel(const __grid_constant__ Geom g, const T *__restrict__ x, const T *__restrict__ go,
                   float *__restrict__ part0, float *__restrict__ partl /* level l at l*C*np*100 */) {
    extern __shared__ __align__(16) u64 sm[];
    const int tid = threadIdx.x, nthr = blockDim.x;
    for (int i = tid; i < g.smem_u64; i += nthr) sm[i] = 0ull;
    const int L = g.L, ncls = 1 + 4 * L;
    int cls = 0;
    while (cls < ncls && tid >= g.thr_start[cls + 1]) ++cls;
    const bool active = cls < ncls;
    const int lvl = active ? (cls == 0 ? 0 : 1 + ((cls - 1) >> 2)) : 0, sub = (cls - 1) & 3;
    const int kth = active ? tid - g.thr_start[cls] : 0, nth = active ? g.thr_start[cls + 1] - g.thr_start[cls] : 1;
    const int ntile = g.tx[lvl] * g.ty[lvl];
    const int pl = g.pitch[lvl], hl = pl >> 1;
    const int suboff = (lvl == 0 ? 0 : sub * g.rows[lvl] * pl);
    u64 acc[KK], gsum = 0ull;
#pragma unroll
    for (int t = 0; t < KK; ++t) acc[t] = 0ull;
    const int u_begin = (int)((long long)blockIdx.x * g.units / gridDim.x);
    const int u_end = (int)((long long)(blockIdx.x + 1) * g.units / gridDim.x);
    __syncthreads();
    for (int u = u_begin; u < u_end; ++u) {
        const int cp = u / g.bgroups, bg = u - cp * g.bgroups;
        const int cA = 2 * cp;
        const bool hasB = cA + 1 < g.C;
        stage_input<T>(sm, g, g.offA, x, cA, hasB, bg);
        stage_input<T>(sm, g, g.offG, go, cA, hasB, bg);
        __syncthreads();
        for (int l = 2; l <= L; ++l) {
            stage_level(sm, g, g.offA, l);
            stage_level(sm, g, g.offG, l);
            __syncthreads();
        }
        if (active) {
            for (int it = kth; it < g.NPP * ntile; it += nth) {
                const int slot = fdiv(it, g.d_nt[lvl]), r = it - slot * ntile;
                const int tyy = fdiv(r, g.d_tx[lvl]), txx = r - tyy * g.tx[lvl];
                const u64 *S = sm + (size_t)slot * g.slot_stride;
                const u64 *ysrc = S + g.offA[lvl] + suboff + 4 * tyy * pl + 2 * txx;
                // D tile = columns 4tx+2..4tx+5 of rows 4ty+2..: chunk 2tx+1 (odd half) and chunk 2tx+2 (even half)
                const u64 *dsrc = S + g.offG[lvl] + suboff + (4 * tyy + 2) * pl + 2 * txx;
                u64 d[4][4];
#pragma unroll
                for (int rr = 0; rr < 4; ++rr) {
                    const ulonglong2 q0 = *reinterpret_cast<const ulonglong2 *>(dsrc + rr * pl + hl);
                    const ulonglong2 q1 = *reinterpret_cast<const ulonglong2 *>(dsrc + rr * pl + 2);
                    d[rr][0] = q0.x; d[rr][1] = q0.y; d[rr][2] = q1.x; d[rr][3] = q1.y;
                }
                if (cls == 0) {
#pragma unroll
                    for (int rr = 0; rr < 4; ++rr)
#pragma unroll
                        for (int c = 0; c < 4; ++c) gsum = add2(gsum, d[rr][c]);
                }
#pragma unroll
                for (int rr = 0; rr < 8; ++rr) {
                    const u64 *rp = ysrc + rr * pl;
                    const ulonglong2 q0 = *reinterpret_cast<const ulonglong2 *>(rp);
                    const ulonglong2 q1 = *reinterpret_cast<const ulonglong2 *>(rp + hl);
                    const ulonglong2 q2 = *reinterpret_cast<const ulonglong2 *>(rp + 2);
                    const ulonglong2 q3 = *reinterpret_cast<const ulonglong2 *>(rp + hl + 2);
                    const u64 in[8] = {q0.x, q0.y, q1.x, q1.y, q2.x, q2.y, q3.x, q3.y};
#pragma unroll
                    for (int uu = 0; uu < 5; ++uu) {
                        const int dr = rr - uu;
                        if (dr >= 0 && dr < 4) {
#pragma unroll
                            for (int v = 0; v < 5; ++v)
#pragma unroll
                                for (int c = 0; c < 4; ++c) acc[uu * 5 + v] = fma2(d[dr][c], in[c + v], acc[uu * 5 + v]);
                        }
                    }
                }
            }
        }
        __syncthreads();
        const bool last_of_pair = (u + 1 == u_end) || ((u + 1) / g.bgroups != cp);
        if (last_of_pair) {
            // block tree through shared memory: every thread parks its 26 packed sums, then one thread
            // per (class, tap) adds its class's threads in index order
            u64 *scr = sm;
#pragma unroll
            for (int t = 0; t < KK; ++t) scr[(size_t)tid * (KK + 1) + t] = acc[t];
            scr[(size_t)tid * (KK + 1) + KK] = gsum;
            __syncthreads();
            const int slotp = blockIdx.x - block_of_unit((long long)cp * g.bgroups, gridDim.x, g.units);
            for (int e = tid; e < ncls * (KK + 1); e += nthr) {
                const int c2 = e / (KK + 1), t = e - c2 * (KK + 1);
                if (c2 > 0 && t == KK) continue;
                u64 s = 0ull;
                for (int th = g.thr_start[c2]; th < g.thr_start[c2 + 1]; ++th) s = add2(s, scr[(size_t)th * (KK + 1) + t]);
                float sa, sb;
                upk(s, sa, sb);
                if (c2 == 0) {
                    part0[((size_t)cA * g.np + slotp) * (KK + 1) + t] = sa;
                    if (hasB) part0[((size_t)(cA + 1) * g.np + slotp) * (KK + 1) + t] = sb;
                } else {
                    const int l = (c2 - 1) >> 2, sb_ = (c2 - 1) & 3;
                    float *pl_ = partl + (size_t)l * g.C * g.np * 4 * KK;
                    pl_[(((size_t)cA * g.np + slotp) * 4 + sb_) * KK + t] = sa;
                    if (hasB) pl_[(((size_t)(cA + 1) * g.np + slotp) * 4 + sb_) * KK + t] = sb;
                }
            }
            __syncthreads();
            for (int i = tid; i < g.smem_u64; i += nthr) sm[i] = 0ull;  // restore the zero halos
#pragma unroll
            for (int t = 0; t < KK; ++t) acc[t] = 0ull;
            gsum = 0ull;
            __syncthreads();
        }
    }
}

// ------------------------------------------------------------------ host-side planning
inline void fill_common(Geom &g, int B, int C, int H, int W, int L) {
    g.B = B; g.C = C; g.H = H; g.W = W; g.L = L;
    g.Hl[0] = H; g.Wl[0] = W;
    for (int l = 1; l <= MAXL; ++l) { g.Hl[l] = (g.Hl[l - 1] + 1) / 2; g.Wl[l] = (g.Wl[l - 1] + 1) / 2; }
    for (int l = 0; l <= L; ++l) {
        g.rows[l] = pad4(g.Hl[l]) + 4;
        g.pitch[l] = pad4(g.Wl[l]) + 4;
        g.ty[l] = pad4(g.Hl[l]) / 4;
        g.tx[l] = pad4(g.Wl[l]) / 4;
    }
    g.nbase = g.tx[0] * g.ty[0];
    g.lvl_start[0] = 0; g.lvl_start[1] = 0;
    for (int l = 1; l <= L; ++l) g.lvl_start[l + 1] = g.lvl_start[l] + 4 * g.tx[l] * g.ty[l];
    g.ncp = (C + 1) / 2;
    g.vec = (L >= 1 && (W & 3) == 0) ? 1 : 0;
    if (L >= 1) {
        const int prow = g.vec ? W / 4 : g.Wl[1];
        g.npatch = g.Hl[1] * prow;
        g.d_npatch = make_fastdiv(g.npatch);
        g.d_prow = make_fastdiv(prow);
    } else {
        g.npatch = H * W;
        g.d_npatch = make_fastdiv(g.npatch);
        g.d_prow = make_fastdiv(W);
    }
    for (int l = 0; l <= L; ++l) {
        g.d_lvl[l] = make_fastdiv(g.Hl[l] * g.Wl[l]);
        g.d_lvlw[l] = make_fastdiv(g.Wl[l]);
        g.d_nt[l] = make_fastdiv(g.tx[l] * g.ty[l]);
        g.d_tx[l] = make_fastdiv(g.tx[l]);
    }
    g.d_nlv = make_fastdiv(g.lvl_start[L + 1]);
    g.d_nbase = make_fastdiv(g.nbase);
}

// Slot layout; returns float2 count per slot.  with_g: second copy of the input pyramid (grad_out);
// with_z: the conv-output arrays.
inline int layout_slot(Geom &g, bool with_g, bool with_z) {
    int off = 0;
    for (int l = 0; l <= g.L; ++l) { g.offA[l] = off; off += (l == 0 ? 1 : 4) * g.rows[l] * g.pitch[l]; }
    for (int l = 0; l <= g.L; ++l) { g.offG[l] = off; if (with_g) off += (l == 0 ? 1 : 4) * g.rows[l] * g.pitch[l]; }
    for (int l = 1; l <= g.L; ++l) {
        // only the coefficients the (padded) 4x4 pixel tiles read in the synthesis are kept
        const int zr = ((pad4(g.H) - 1) >> l) + 1;
        const int zc = ((((pad4(g.W) - 1) >> l) + 1) + 1) & ~1;
        g.zrows[l] = zr; g.zpitch[l] = zc; g.offZ[l] = off;
        if (with_z) off += 4 * zr * zc;
    }
    return (off + 1) & ~1;
}

inline double partition_eff(int units, int nblocks) {
    const int per = (units + nblocks - 1) / nblocks;
    return (double)units / ((double)per * nblocks);
}

// Forward plan: maximise (tile-slot use) x (threads resident) x (phase overlap) x (tail) over NPP, T, blocks/SM.
// `tune` (0 = automatic): bits 0-5 threads/32, bits 6-7 blocks per SM, bits 8-14 plane pairs per unit.
inline bool plan_forward(int B, int C, int H, int W, int L, Geom &best, unsigned tune = 0) {
    const int fT = (tune & 63) * 32, fBps = (tune >> 6) & 3, fNpp = (tune >> 8) & 127;
    Geom g = {};
    fill_common(g, B, C, H, W, L);
    const int slot = layout_slot(g, false, true);
    const int M = g.lvl_start[L + 1] + g.nbase;
    const int wtab = (1 + 4 * L) * WT_STRIDE;
    bool found = false;
    best.score = -1.0;
    for (int npp = 1; npp <= 64; ++npp) {
        if (npp > 1 && npp > B) break;
        if (fNpp && npp != fNpp) continue;
        const long long smem_u64 = (long long)npp * slot + ((wtab + 1) & ~1);
        const long long bytes = smem_u64 * 8;
        if (bytes > SMEM_LIMIT) break;
        for (int T = 64; T <= MAX_THREADS; T += 32) {
            if (npp * g.nbase > T) continue;
            if (fT && T != fT) continue;
            for (int bps = 1; bps <= 4; ++bps) {
                if (bps * T > 512) continue;
                if (fBps && bps != fBps) continue;
                if (bps * (bytes + 1024) > SMEM_PER_SM) continue;
                const int rounds = (npp * M + T - 1) / T;
                const double eff = (double)npp * M / ((double)T * rounds);
                const int bgroups = (B + npp - 1) / npp, units = g.ncp * bgroups;
                int nblocks = NUM_SMS * bps;
                if (nblocks > units) nblocks = units;
                const double sc = eff * ((double)bps * T / 512.0) * (bps >= 2 ? 1.0 : 0.9) *
                                  partition_eff(units, nblocks) * ((double)B / ((double)bgroups * npp)) *
                                  (rounds <= 3 ? 1.0 : 0.97);
                if (sc > best.score + 1e-9) {
                    best = g;
                    best.NPP = npp; best.slot_stride = slot; best.wtab_off = npp * slot;
                    best.smem_u64 = (int)smem_u64; best.bgroups = bgroups; best.units = units;
                    best.nthreads = T; best.nblocks = nblocks; best.blocks_per_sm = bps; best.score = sc;
                    found = true;
                }
            }
        }
    }
    return found;
}

// Weight-gradient plan: one block per SM; per class c with n_c tiles (x NPP) allocate ceil(n_c NPP / rounds)
// threads, smallest `rounds` that fits 512 threads.
inline bool plan_wgrad(int B, int C, int H, int W, int L, Geom &best, unsigned tune = 0) {
    const int fNpp = (tune >> 15) & 127;
    Geom g = {};
    fill_common(g, B, C, H, W, L);
    const int slot = layout_slot(g, true, false);
    const int ncls = 1 + 4 * L;
    bool found = false;
    best.score = -1.0;
    for (int npp = 1; npp <= 64; ++npp) {
        if (npp > 1 && npp > B) break;
        if (fNpp && npp != fNpp) continue;
        for (int rounds = 1; rounds <= 64; ++rounds) {
            int thr[4 * MAXL + 2];
            int tot = 0, work = 0;
            for (int c = 0; c < ncls; ++c) {
                const int l = c == 0 ? 0 : 1 + ((c - 1) >> 2);
                const int n = g.tx[l] * g.ty[l] * npp;
                thr[c] = tot;
                tot += (n + rounds - 1) / rounds;
                work += n;
            }
            thr[ncls] = tot;
            if (tot > MAX_THREADS) continue;
            const int T = (tot + 31) & ~31;
            long long smem_u64 = (long long)npp * slot;
            const long long scratch = (long long)T * (KK + 1);
            if (scratch > smem_u64) smem_u64 = scratch;
            smem_u64 = (smem_u64 + 1) & ~1LL;
            if (smem_u64 * 8 > SMEM_LIMIT) break;
            const int bgroups = (B + npp - 1) / npp, units = g.ncp * bgroups;
            int nblocks = NUM_SMS;
            if (nblocks > units) nblocks = units;
            const double sc = ((double)work / ((double)T * rounds)) * ((double)T / 512.0) *
                              partition_eff(units, nblocks) * ((double)B / ((double)bgroups * npp));
            if (sc > best.score + 1e-9) {
                best = g;
                best.NPP = npp; best.slot_stride = slot; best.wtab_off = 0; best.smem_u64 = (int)smem_u64;
                best.bgroups = bgroups; best.units = units; best.nthreads = T; best.nblocks = nblocks;
                best.blocks_per_sm = 1; best.score = sc;
                for (int c = 0; c <= ncls; ++c) best.thr_start[c] = thr[c];
                int np = 1;
                for (int cp = 0; cp < g.ncp; ++cp) {
                    const int first = block_of_unit((long long)cp * bgroups, nblocks, units);
                    const int last = block_of_unit((long long)(cp + 1) * bgroups - 1, nblocks, units);
                    if (last - first + 1 > np) np = last - first + 1;
                }
                best.np = np;
                found = true;
            }
            break;  // more rounds with the same NPP only lowers thread use
        }
    }
    return found;
}

inline bool supported(int H, int W, int k, int L, int dtype) {
    (void)dtype;
    if (k != 5) return false;
    Geom g;
    return plan_forward(2, 2, H, W, L, g) && plan_wgrad(2, 2, H, W, L, g);
}

inline size_t forward_workspace_bytes(int, int, int, int, int) { return 0; }

// Backward workspace: base partials [C][np][26] then level partials [L][C][np][4][25] (float).
inline size_t backward_workspace_bytes(int B, int C, int H, int W, int L, unsigned tune = 0) {
    Geom g;
    if (!plan_wgrad(B, C, H, W, L, g, tune)) return 0;
    return sizeof(float) * ((size_t)C * g.np * (KK + 1) + (size_t)L * C * g.np * 4 * KK);
}

template <typename T>
cudaError_t forward(int B, int C, int H, int W, int L, const T *x, const float *w0, const float *s0, const float *b0,
                    const float *wl, const float *sl, T *out, char *, cudaStream_t st, unsigned tune = 0) {
    Geom g;
    if (!plan_forward(B, C, H, W, L, g, tune)) return cudaErrorInvalidValue;
    auto kern = plane_fwd_kernel<T, false>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT);
    if (e != cudaSuccess) return e;
    kern<<<g.nblocks, g.nthreads, (size_t)g.smem_u64 * 8, st>>>(g, x, w0, s0, b0, wl, sl, out);
    return cudaGetLastError();
}

template <typename T>
cudaError_t backward(int B, int C, int H, int W, int L, const T *x, const T *go, const float *w0, const float *s0,
                     const float *wl, const float *sl, T *gx, char *ws, EpiloguePtrs *ep, cudaStream_t st, unsigned tune = 0) {
    Geom gw, gf;
    if (!plan_wgrad(B, C, H, W, L, gw, tune) || !plan_forward(B, C, H, W, L, gf, tune)) return cudaErrorInvalidValue;
    float *part0 = reinterpret_cast<float *>(ws);
    float *partl = part0 + (size_t)C * gw.np * (KK + 1);
    const size_t pbytes = backward_workspace_bytes(B, C, H, W, L, tune);
    cudaError_t e = cudaMemsetAsync(ws, 0, pbytes, st);  // slots no block writes must read as zero
    if (e != cudaSuccess) return e;
    auto kw = plane_wgrad_kernel<T>;
    e = cudaFuncSetAttribute(kw, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT);
    if (e != cudaSuccess) return e;
    kw<<<gw.nblocks, gw.nthreads, (size_t)gw.smem_u64 * 8, st>>>(gw, x, go, part0, partl);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    auto kf = plane_fwd_kernel<T, true>;
    e = cudaFuncSetAttribute(kf, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT);
    if (e != cudaSuccess) return e;
    kf<<<gf.nblocks, gf.nthreads, (size_t)gf.smem_u64 * 8, st>>>(gf, go, w0, s0, nullptr, wl, sl, gx);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    ep->part0 = part0;
    ep->np0 = gw.np;
    for (int l = 0; l < L; ++l) {
        ep->partl[l] = partl + (size_t)l * C * gw.np * 4 * KK;
        ep->npl[l] = gw.np;
    }
    return cudaSuccess;
}

}  // namespace plane
}  // namespace wt
