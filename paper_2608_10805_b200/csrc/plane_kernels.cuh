// Whole-plane WTConv kernels for sm_100a (k = 5, and k = 3 as the inner taps of 5 x 5 tables: KT = 3 builds of the
// kernels leave the zero border out of the tap loops): every (b, c) plane's entire decomposition lives
// in shared memory, so the only HBM traffic is the compulsory one (read x, write out; in the backward
// read x and grad_out, write grad_x).
//
// Design
//  * A block is persistent and walks a contiguous range of units.  A unit is NPL consecutive channels of
//    one image (contiguous in NCHW, so one aligned bulk copy fetches it); units are ordered channel-group
//    major, so a block keeps its folded weight table (Eq. 8) over all images of a group.  A plane's
//    footprint (x with a zero halo, the four Haar subbands of every level with halos, the conv outputs
//    Z^l) is about 58 KB for 56x56, so three blocks are resident per SM: while one block is in a
//    latency-bound phase (staging, synthesis, stores) the others keep the FP32 pipe busy.
//  * Units arrive through a ring of raw buffers filled by cp.async.bulk and watched by mbarriers (bounded
//    waits that raise a status word instead of spinning for ever); where no ring fits, the next unit is
//    warmed in L2.  Per unit: stage x into the haloed array and run the Haar butterfly of Eq. 5 on chip
//    (Sec. 4.1), levels 1 and 2 in the same pass, deeper levels from the raw LL band; then every thread
//    convolves 4-column x TH-row register tiles (TH = 4 or 8, chosen per plan) straight out of shared
//    memory (two aligned 16-byte loads per window row) with weights that already carry the scale.  Level
//    tiles and base tiles are one item list and one rolled copy of the tile code; a thread keeps its base
//    tile in registers across one barrier and then adds the bit-indexed closed-form synthesis of
//    Proposition 2 (Sec. 4.2) before the only store.
//  * Backward.  grad_x is the forward dataflow run on grad_out with the kernels rotated by 180 degrees
//    (Sec. 2.2: the adjoint of analysis is synthesis and vice versa, so the adjoint of the whole operator
//    has the operator's own structure).  The fused kernel stages the decompositions of x and grad_out
//    once; every thread owns one tile, first correlates it into the 25 weight-gradient accumulators of
//    its (level, subband) class - kept in registers across all images of a channel and reduced once by a
//    block tree through shared memory, then in fixed-order fp64 in the epilogue - and then runs the
//    rotated-kernel convolution, synthesis and store on the same window.  Shapes whose tiles do not fit
//    one pass of 256 threads take the split pair instead: a weight-gradient kernel with class-major
//    thread allocation plus the FLIP instantiation of the forward kernel.
//  * Launches overlap: every kernel here is started with programmatic stream serialisation (common.cuh), does its
//    set-up in shared memory and registers beside the tail of the kernel before it and only then waits for that
//    kernel; no call puts a clearing operation between two kernels (status words are tagged per call, the epilogue
//    is told which partial-sum slots the blocks write).
//  * Host side: plans (threads, blocks per SM, planes per unit, tile height, ring depth) come from a
//    search over a small cost model and are cached per shape.
#pragma once
#include <atomic>
#include <cmath>
#include <cstdio>
#include <mutex>
#include <vector>
#include "common.cuh"
#include "tiled_kernels.cuh"

namespace wt {
namespace plane {

constexpr int MAXL = 8;
constexpr int KK = 25;
constexpr int MAX_THREADS = 256;
constexpr int NUM_SMS = 148;                 // planning constant (B200); plans must not depend on the device
constexpr int SMEM_LIMIT = 227 * 1024;       // opt-in dynamic shared memory per block
constexpr int SMEM_PER_SM = 228 * 1024;      // per SM, 1 KB reserved per resident block
constexpr int WT_STRIDE = 28;                // floats per class in the weight table (25 taps, 16-byte padded)
constexpr int MAX_STAGES = 4;               // deepest prefetch ring (units in flight per block)
constexpr unsigned WAIT_LIMIT = 1u << 20;    // bounded number of (suspending) waits on the copy barrier: never an endless loop
constexpr unsigned WAIT_LIMIT_TEST = 64;     // the same under WTCONV_FLAG_TEST_NO_COPY (no copy is ever issued: every wait runs out)

// ------------------------------------------------------------------ bulk-copy (TMA, untiled) helpers
__device__ __forceinline__ unsigned smem_addr(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long *bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long *bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
// global -> shared, 16-byte aligned both sides, size a multiple of 16; completion counted on `bar`
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, unsigned bytes, unsigned long long *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(dst)),
                 "l"(src), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}
// Bounded wait for phase `parity` of `bar`: try_wait suspends the thread for a hardware-limited time per call, so
// waiting costs few instructions; false if the phase did not complete within `limit` calls.
__device__ __forceinline__ bool mbar_wait(unsigned long long *bar, unsigned parity, unsigned limit) {
    const unsigned a = smem_addr(bar);
    for (unsigned i = 0; i < limit; ++i) {
        unsigned ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok)
                     : "r"(a), "r"(parity)
                     : "memory");
        if (ok) return true;
    }
    return false;
}
// shared -> global bulk store (same alignment rules); completion is tracked per thread in bulk groups
__device__ __forceinline__ void bulk_s2g(void *gdst, const void *src, unsigned bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_addr(src)), "r"(bytes)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// wait until every bulk store this thread issued has finished READING its shared-memory source
__device__ __forceinline__ void bulk_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// order earlier generic-proxy accesses of shared memory before later async-proxy (bulk copy) writes
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ------------------------------------------------------------------ geometry (host-planned, passed by value)
// Division by a launch-invariant divisor as multiply-high: exact while dividend * divisor < 2^32.  Every use divides
// an index inside one work unit (tiles, staging patches or coefficients of at most 64 planes: below 2^18) by a
// per-plane count (below 2^13); indices over the whole tensor (units, images) are never divided this way.
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
    int rows[MAXL + 1], pitch[MAXL + 1];   // haloed arrays: ty*TH+4 rows, pitch pad4(Wl)+4 floats; element (y,x) at (y+2, x+2)
    int offA[MAXL + 1];                    // slot-relative offset of x (l=0) / Y^l subband 0 (subband stride rows*pitch)
    int offG[MAXL + 1];                    // same for grad_out / D^l (weight-gradient kernel only)
    int zrows[MAXL + 1], zpitch[MAXL + 1]; // conv outputs Z^l (forward kernel only)
    int offZ[MAXL + 1];
    int slot_stride;                       // floats per plane slot
    int th;                                // register tile height: tiles are 4 columns x th rows (4 or 8)
    int NPL;                               // plane slots per work unit: NPL consecutive channels of one image (contiguous in memory)
    int tx[MAXL + 1], ty[MAXL + 1];        // 4 x TH tiles per level grid (index 0 = base)
    int lvl_start[MAXL + 2];               // per plane: first level-item of level l (1..L); [L+1] = count
    int nbase;                             // base tiles per plane
    int wtab_off;                          // offset of the folded weight table [(1+4L)][WT_STRIDE] (bias at [0][25])
    int smem_floats;
    int ngroups, units;                    // work units = ngroups channel groups x B images, group-major (a block keeps a group's
                                           // weights and gradient accumulators while it walks through the images)
    int nthreads, nblocks, blocks_per_sm;
    int vec;                               // 1: W % 4 == 0, rows are staged with 4-element vector loads
    int no_copy;                           // test mode: bulk copies are never issued and waits give up quickly (the timeout path)
    unsigned tag;                          // non-zero tag of the call this launch belongs to (status words, see common.cuh)
    int taps;                              // taps per side in use: 5, or 3 for 3 x 3 kernels in the middle of 5 x 5 tables
    int bulk;                              // 1: planes are fetched ahead with cp.async.bulk into a ring of raw buffers at raw_off
    int nstage, stage_bytes;               // ring depth (units in flight) and bytes per ring entry
    int raw_off, raw_slot_bytes, plane_bytes;  // raw staging buffer (float offset), bytes per plane slot / per plane
    int bar_off;                           // float offset of the ring's mbarriers (8-byte aligned, one per entry)
    int bulk_out, out_off;                 // 1: results are assembled in shared memory (out_off) and leave with one bulk store
    int npatch4;                           // 4x4 pixel patches per plane (vec staging of levels 1 and 2 in one pass)
    FastDiv d_npatch4;
    int npatch;                            // staging work items per plane (vec: 2x4 pixel patches, else 2x2 blocks)
    FastDiv d_npatch, d_prow;              // / npatch, / (patches per patch-row)
    FastDiv d_lvl[MAXL + 1], d_lvlw[MAXL + 1];  // / (Hl*Wl), / Wl   (levels >= 2 staging)
    FastDiv d_nlv, d_nt[MAXL + 1], d_tx[MAXL + 1], d_nbase;
    // weight-gradient kernel: class-major thread allocation and partial-sum slots
    int thr_start[4 * MAXL + 2];
    int np;
    double score;
};

__host__ __device__ inline int pad4(int n) { return (n + 3) & ~3; }

using wt::block_of_unit;

// ------------------------------------------------------------------ shared device pieces
__device__ __forceinline__ void build_weight_table(float *wtab, const Geom &g, int c0, bool flip,
                                                   const float *__restrict__ w0, const float *__restrict__ s0,
                                                   const float *__restrict__ b0, const float *__restrict__ wl,
                                                   const float *__restrict__ sl) {
    // one table per plane slot (channel c0 + slot): [slot][class][WT_STRIDE], folded bias at [slot][0][25]
    const int ncls = 1 + 4 * g.L, n = g.NPL * ncls * KK;
    constexpr int WB = 4;
    // four entries per step, all eight loads issued before the first product: a 16-plane unit's table has 2000
    // entries and every block builds it, so the loads must overlap
    for (int e0 = threadIdx.x; e0 < n; e0 += WB * blockDim.x) {
        float wv[WB], sv[WB];
        int dst[WB];
#pragma unroll
        for (int k = 0; k < WB; ++k) {
            const int e = e0 + k * blockDim.x;
            wv[k] = sv[k] = 0.f;
            dst[k] = -1;
            if (e < n) {
                const int sc = e / KK, t = e - sc * KK, slot = sc / ncls, cls = sc - slot * ncls;
                const int c = c0 + slot, src = flip ? (KK - 1 - t) : t;
                dst[k] = sc * WT_STRIDE + t;
                if (c < g.C) {
                    if (cls == 0) {
                        wv[k] = __ldg(w0 + c * KK + src);
                        sv[k] = __ldg(s0 + c);
                    } else {
                        const int l = (cls - 1) >> 2, sub = (cls - 1) & 3;
                        const size_t i = ((size_t)l * g.C + c) * 4 + sub;
                        wv[k] = __ldg(wl + i * KK + src);
                        sv[k] = __ldg(sl + i);
                    }
                }
            }
        }
#pragma unroll
        for (int k = 0; k < WB; ++k)
            if (dst[k] >= 0) wtab[dst[k]] = wv[k] * sv[k];  // Eq. 8: scale folded into the weight
    }
    for (int slot = threadIdx.x; slot < g.NPL; slot += blockDim.x)
        wtab[slot * ncls * WT_STRIDE + KK] = (b0 && c0 + slot < g.C) ? __ldg(s0 + c0 + slot) * __ldg(b0 + c0 + slot) : 0.f;
}

__device__ __forceinline__ void load_weights(const float *wt, float (&w)[KK]) {
    const float4 *q = reinterpret_cast<const float4 *>(wt);
#pragma unroll
    for (int t = 0; t < 6; ++t) {
        const float4 v = q[t];
        w[4 * t] = v.x; w[4 * t + 1] = v.y; w[4 * t + 2] = v.z; w[4 * t + 3] = v.w;
    }
    w[24] = wt[24];
}

// four consecutive activations (16-byte aligned for float, 8-byte for the 16-bit types)
__device__ __forceinline__ void load4(const float *p, float (&v)[4]) {
    const float4 q = __ldg(reinterpret_cast<const float4 *>(p));
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}
__device__ __forceinline__ void load4(const __half *p, float (&v)[4]) {
    const uint2 q = __ldg(reinterpret_cast<const uint2 *>(p));
    const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&q.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2 *>(&q.y));
    v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
}
__device__ __forceinline__ void load4(const __nv_bfloat16 *p, float (&v)[4]) {
    const uint2 q = __ldg(reinterpret_cast<const uint2 *>(p));
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&q.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&q.y));
    v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
}

// the same from shared memory (a raw plane a bulk copy landed there)
__device__ __forceinline__ void load4s(const float *p, float (&v)[4]) {
    const float4 q = *reinterpret_cast<const float4 *>(p);
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}
__device__ __forceinline__ void load4s(const __half *p, float (&v)[4]) {
    const uint2 q = *reinterpret_cast<const uint2 *>(p);
    const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&q.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2 *>(&q.y));
    v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
}
__device__ __forceinline__ void load4s(const __nv_bfloat16 *p, float (&v)[4]) {
    const uint2 q = *reinterpret_cast<const uint2 *>(p);
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&q.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&q.y));
    v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
}
__device__ __forceinline__ float ldf_plain(const float *p) { return *p; }
__device__ __forceinline__ float ldf_plain(const __half *p) { return __half2float(*p); }
__device__ __forceinline__ float ldf_plain(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
template <typename T, bool RAW>
__device__ __forceinline__ float ld1(const T *p) { return RAW ? ldf_plain(p) : ldf(p); }
template <typename T, bool RAW>
__device__ __forceinline__ void ld4(const T *p, float (&v)[4]) {
    if (RAW) load4s(p, v); else load4(p, v);
}

__device__ __forceinline__ void decode_level_item(const Geom &g, int r, int &l, int &sub, int &tyy, int &txx);

// ---- per-thread work descriptors.  A thread's tiles and staging patches are the same for every unit, so
// ---- they are decoded once, before the unit loop, and live in registers.
struct PatchD {   // 4x4 pixel staging patch (vector path, L >= 2)
    int so;       // element offset of the patch inside its plane: y*W + 4q
    int xi, yi, y2;  // float indices of its first x / level-1 / level-2 element in shared memory
    int meta;     // bit 31 valid, bits 0-7 plane slot, bits 8-10 rows inside the image (1..4)
};
__device__ __forceinline__ PatchD decode_patch(const Geom &g, const int *off, int e) {
    PatchD p;
    p.meta = 0;
    p.so = p.xi = p.yi = p.y2 = 0;
    if (e < g.NPL * g.npatch4) {
        const int slot = fdiv(e, g.d_npatch4), r = e - slot * g.npatch4;
        const int i2 = fdiv(r, g.d_prow), q = r - i2 * (int)g.d_prow.d;
        const int y = 4 * i2, S = slot * g.slot_stride;
        int nrows = g.H - y;
        if (nrows > 4) nrows = 4;
        p.so = y * g.W + 4 * q;
        p.xi = S + off[0] + (y + 2) * g.pitch[0] + 4 * q + 2;
        p.yi = S + off[1] + (2 * i2 + 2) * g.pitch[1] + 2 * q + 2;
        p.y2 = S + off[2] + (i2 + 2) * g.pitch[2] + q + 2;
        p.meta = (int)(0x80000000u | (unsigned)slot | ((unsigned)nrows << 8));
    }
    return p;
}
// The 4 x 4 pixels of a patch (zero where the patch leaves the image or the plane slot is not in use).
template <typename T, bool RAW>
__device__ __forceinline__ void load_patch(const Geom &g, const PatchD &p, const T *__restrict__ gsrc, int nvalid,
                                           float (&a)[4][4]) {
    const int slot = p.meta & 0xff, nrows = (p.meta >> 8) & 7;
#pragma unroll
    for (int rr = 0; rr < 4; ++rr)
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) a[rr][cc] = 0.f;
    if (slot < nvalid) {
        const T *pa = gsrc + slot * (g.H * g.W) + p.so;  // the unit's planes are contiguous
#pragma unroll
        for (int rr = 0; rr < 4; ++rr)
            if (rr < nrows) ld4<T, RAW>(pa + rr * g.W, a[rr]);
    }
}
// x, level 1 and level 2 of one patch into the haloed arrays; d0/d1/d2 shift the targets to another set of
// arrays (grad_out side).
__device__ __forceinline__ void store_patch(float *sm, const Geom &g, const PatchD &p0_, const float (&a)[4][4], int d0,
                                            int d1, int d2) {
    PatchD p = p0_;
    p.xi += d0;
    p.yi += d1;
    p.y2 += d2;
    const int nrows = (p.meta >> 8) & 7;
    const int p0 = g.pitch[0], p1 = g.pitch[1], sub1 = g.rows[1] * p1, sub2 = g.rows[2] * g.pitch[2];
#pragma unroll
    for (int rr = 0; rr < 4; ++rr) {
        if (rr < nrows) {
            *reinterpret_cast<float2 *>(&sm[p.xi + rr * p0]) = make_float2(a[rr][0], a[rr][1]);
            *reinterpret_cast<float2 *>(&sm[p.xi + rr * p0 + 2]) = make_float2(a[rr][2], a[rr][3]);
        }
    }
    Haar4 h[2][2];
#pragma unroll
    for (int bi = 0; bi < 2; ++bi)
#pragma unroll
        for (int bj = 0; bj < 2; ++bj)
            h[bi][bj] = haar_butterfly(a[2 * bi][2 * bj], a[2 * bi][2 * bj + 1], a[2 * bi + 1][2 * bj], a[2 * bi + 1][2 * bj + 1]);
#pragma unroll
    for (int bi = 0; bi < 2; ++bi) {
        *reinterpret_cast<float2 *>(&sm[p.yi + bi * p1]) = make_float2(h[bi][0].ll, h[bi][1].ll);
        *reinterpret_cast<float2 *>(&sm[p.yi + bi * p1 + sub1]) = make_float2(h[bi][0].lh, h[bi][1].lh);
        *reinterpret_cast<float2 *>(&sm[p.yi + bi * p1 + 2 * sub1]) = make_float2(h[bi][0].hl, h[bi][1].hl);
        *reinterpret_cast<float2 *>(&sm[p.yi + bi * p1 + 3 * sub1]) = make_float2(h[bi][0].hh, h[bi][1].hh);
    }
    const Haar4 h2 = haar_butterfly(h[0][0].ll, h[0][1].ll, h[1][0].ll, h[1][1].ll);
    sm[p.y2] = h2.ll;
    sm[p.y2 + sub2] = h2.lh;
    sm[p.y2 + 2 * sub2] = h2.hl;
    sm[p.y2 + 3 * sub2] = h2.hh;
}
template <typename T, bool RAW>
__device__ __forceinline__ void run_patch(float *sm, const Geom &g, const PatchD &p, const T *__restrict__ gsrc,
                                          int nvalid, int d0 = 0, int d1 = 0, int d2 = 0) {
    if (p.meta >= 0) return;
    float a[4][4];
    load_patch<T, RAW>(g, p, gsrc, nvalid, a);
    store_patch(sm, g, p, a, d0, d1, d2);
}
// The same patch of two tensors (x and grad_out): both sets of loads are issued before either is used, so
// their global-memory latencies overlap.
template <typename T, bool RAW>
__device__ __forceinline__ void run_patch_pair(float *sm, const Geom &g, const PatchD &p, const T *__restrict__ xsrc,
                                               const T *__restrict__ gsrc, int nvalid, int d0, int d1, int d2) {
    if (p.meta >= 0) return;
    float a[4][4], b[4][4];
    load_patch<T, RAW>(g, p, xsrc, nvalid, a);
    load_patch<T, RAW>(g, p, gsrc, nvalid, b);
    store_patch(sm, g, p, a, 0, 0, 0);
    store_patch(sm, g, p, b, d0, d1, d2);
}

struct ItemD {    // one 4 x TH conv tile
    int src;      // float index of the window's top-left element
    int wt;       // float index of its 25 folded weights
    int z;        // level tile: float index of its output in Z^l, or -2 if the tile lies outside what the synthesis reads;
                  // base tile: -1
    int meta;     // bit 31 valid; bits 0-9 window pitch; bits 10-19 Z pitch; bits 20-23 rows to store (0..TH);
                  // bits 24-29 parameter class (0 = base, 1 + 4(l-1) + sub = level l subband sub)
    int slot;     // plane slot of the tile
    int dg;       // float offset from this tile's x-side array to the matching grad_out-side array (backward kernel)
};
__device__ __forceinline__ ItemD decode_item(const Geom &g, int it, int nlevel_items, int nitems, int &bslot, int &tyy,
                                             int &txx, bool &is_base) {
    ItemD d;
    d.src = d.wt = d.dg = d.slot = 0;
    d.z = -2;
    d.meta = 0;
    if (it >= nitems) return d;
    const int nlv = g.lvl_start[g.L + 1];
    if (it < nlevel_items) {
        int l, sub, ty2, tx2;
        const int slot = fdiv(it, g.d_nlv);
        decode_level_item(g, it - slot * nlv, l, sub, ty2, tx2);
        const int pitch = g.pitch[l], zp = g.zpitch[l];
        d.src = slot * g.slot_stride + g.offA[l] + sub * g.rows[l] * pitch + g.th * ty2 * pitch + 4 * tx2;
        d.wt = g.wtab_off + (slot * (1 + 4 * g.L) + 1 + (l - 1) * 4 + sub) * WT_STRIDE;
        int zleft = g.zrows[l] - g.th * ty2;
        if (zleft > g.th) zleft = g.th;
        if (4 * tx2 < zp && zleft > 0) d.z = slot * g.slot_stride + g.offZ[l] + sub * g.zrows[l] * zp + g.th * ty2 * zp + 4 * tx2;
        if (zleft < 0) zleft = 0;
        d.meta = (int)(0x80000000u | (unsigned)pitch | ((unsigned)zp << 10) | ((unsigned)zleft << 20) |
                       ((unsigned)(1 + (l - 1) * 4 + sub) << 24));
        d.dg = g.offG[l] - g.offA[l];
        d.slot = slot;
    } else {
        const int bi = it - nlevel_items;
        bslot = fdiv(bi, g.d_nbase);
        const int r = bi - bslot * g.nbase;
        tyy = fdiv(r, g.d_tx[0]);
        txx = r - tyy * g.tx[0];
        const int pitch = g.pitch[0];
        d.src = bslot * g.slot_stride + g.offA[0] + g.th * tyy * pitch + 4 * txx;
        d.wt = g.wtab_off + bslot * (1 + 4 * g.L) * WT_STRIDE;
        d.z = -1;
        d.meta = (int)(0x80000000u | (unsigned)pitch);
        d.dg = g.offG[0] - g.offA[0];
        d.slot = bslot;
        is_base = true;
    }
    return d;
}

// Stage the planes of one unit (channel c, images bg*NPL ..): x into the haloed array `off[0]`, its
// level-1 Haar subbands (Eq. 5) into `off[1]` and, on the vector path with L >= 2, the level-2 subbands
// into `off[2]` in the same pass (returns the first level that still has to be staged).  RAW = true reads
// plane slot s from the raw shared buffer at src + s * slot_elems (a bulk copy put it there); RAW = false
// reads global memory.  Pixels beyond H x W are never written and stay zero (odd-size padding and conv
// halo); images beyond the batch are written as zeros.
template <typename T, bool RAW>
__device__ __forceinline__ int stage_input(float *sm, const Geom &g, const int *off, const T *__restrict__ src, int c,
                                           int b, int srank, int nstagers) {
    const int H = g.H, W = g.W, HW = H * W;
    const int p0 = g.pitch[0];
    const T *gsrc = RAW ? src : src + ((size_t)b * g.C + c) * HW;  // channel c (first of the unit) of image b
    const int img_stride = HW;                                     // the unit's planes are contiguous
    const int nvalid = g.C - c < g.NPL ? g.C - c : g.NPL;
    if (g.L == 0) {
        for (int e = srank; e < g.NPL * HW; e += nstagers) {
            const int slot = fdiv(e, g.d_npatch), r = e - slot * HW, y = fdiv(r, g.d_prow), xx = r - y * W;
            const bool valid = slot < nvalid;
            sm[slot * g.slot_stride + off[0] + (y + 2) * p0 + xx + 2] =
                valid ? ld1<T, RAW>(gsrc + (size_t)slot * img_stride + r) : 0.f;
        }
        return 1;
    }
    const int p1 = g.pitch[1], sub1 = g.rows[1] * p1;
    if (g.vec && g.L >= 2) {
        // work item = 4 rows x 4 columns: four level-1 blocks and the level-2 block above them
        const int p2 = g.pitch[2], sub2 = g.rows[2] * p2;
        for (int e = srank; e < g.NPL * g.npatch4; e += nstagers) {
            const int slot = fdiv(e, g.d_npatch4), r = e - slot * g.npatch4;
            const int i2 = fdiv(r, g.d_prow), q = r - i2 * (int)g.d_prow.d;
            const int y = 4 * i2;
            float a[4][4];
#pragma unroll
            for (int rr = 0; rr < 4; ++rr)
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) a[rr][cc] = 0.f;
            if (slot < nvalid) {
                const T *pa = gsrc + (size_t)slot * img_stride + y * W + 4 * q;
#pragma unroll
                for (int rr = 0; rr < 4; ++rr)
                    if (y + rr < H) ld4<T, RAW>(pa + rr * W, a[rr]);
            }
            const int S = slot * g.slot_stride;
            const int xi = S + off[0] + (y + 2) * p0 + 4 * q + 2;  // 8-byte aligned
#pragma unroll
            for (int rr = 0; rr < 4; ++rr) {
                if (y + rr < H) {
                    *reinterpret_cast<float2 *>(&sm[xi + rr * p0]) = make_float2(a[rr][0], a[rr][1]);
                    *reinterpret_cast<float2 *>(&sm[xi + rr * p0 + 2]) = make_float2(a[rr][2], a[rr][3]);
                }
            }
            Haar4 h[2][2];
#pragma unroll
            for (int bi = 0; bi < 2; ++bi)
#pragma unroll
                for (int bj = 0; bj < 2; ++bj)
                    h[bi][bj] = haar_butterfly(a[2 * bi][2 * bj], a[2 * bi][2 * bj + 1], a[2 * bi + 1][2 * bj],
                                               a[2 * bi + 1][2 * bj + 1]);
            const int yi = S + off[1] + (2 * i2 + 2) * p1 + 2 * q + 2;
#pragma unroll
            for (int bi = 0; bi < 2; ++bi) {
                *reinterpret_cast<float2 *>(&sm[yi + bi * p1]) = make_float2(h[bi][0].ll, h[bi][1].ll);
                *reinterpret_cast<float2 *>(&sm[yi + bi * p1 + sub1]) = make_float2(h[bi][0].lh, h[bi][1].lh);
                *reinterpret_cast<float2 *>(&sm[yi + bi * p1 + 2 * sub1]) = make_float2(h[bi][0].hl, h[bi][1].hl);
                *reinterpret_cast<float2 *>(&sm[yi + bi * p1 + 3 * sub1]) = make_float2(h[bi][0].hh, h[bi][1].hh);
            }
            const Haar4 h2 = haar_butterfly(h[0][0].ll, h[0][1].ll, h[1][0].ll, h[1][1].ll);
            const int y2 = S + off[2] + (i2 + 2) * p2 + q + 2;
            sm[y2] = h2.ll;
            sm[y2 + sub2] = h2.lh;
            sm[y2 + 2 * sub2] = h2.hl;
            sm[y2 + 3 * sub2] = h2.hh;
        }
        return 3;
    }
    if (g.vec) {
        // work item = 2 rows x 4 columns: two Haar blocks
        for (int e = srank; e < g.NPL * g.npatch; e += nstagers) {
            const int slot = fdiv(e, g.d_npatch), r = e - slot * g.npatch;
            const int i = fdiv(r, g.d_prow), q = r - i * (int)g.d_prow.d;
            const int y = 2 * i;
            const bool y1 = y + 1 < H;
            float a0[4] = {0.f, 0.f, 0.f, 0.f}, a1[4] = {0.f, 0.f, 0.f, 0.f};
            if (slot < nvalid) {
                const T *pa = gsrc + (size_t)slot * img_stride + y * W + 4 * q;
                ld4<T, RAW>(pa, a0);
                if (y1) ld4<T, RAW>(pa + W, a1);
            }
            const int S = slot * g.slot_stride;
            const int xi = S + off[0] + (y + 2) * p0 + 4 * q + 2;  // 8-byte aligned
            *reinterpret_cast<float2 *>(&sm[xi]) = make_float2(a0[0], a0[1]);
            *reinterpret_cast<float2 *>(&sm[xi + 2]) = make_float2(a0[2], a0[3]);
            if (y1) {
                *reinterpret_cast<float2 *>(&sm[xi + p0]) = make_float2(a1[0], a1[1]);
                *reinterpret_cast<float2 *>(&sm[xi + p0 + 2]) = make_float2(a1[2], a1[3]);
            }
            const Haar4 ha = haar_butterfly(a0[0], a0[1], a1[0], a1[1]), hb = haar_butterfly(a0[2], a0[3], a1[2], a1[3]);
            const int yi = S + off[1] + (i + 2) * p1 + 2 * q + 2;
            *reinterpret_cast<float2 *>(&sm[yi]) = make_float2(ha.ll, hb.ll);
            *reinterpret_cast<float2 *>(&sm[yi + sub1]) = make_float2(ha.lh, hb.lh);
            *reinterpret_cast<float2 *>(&sm[yi + 2 * sub1]) = make_float2(ha.hl, hb.hl);
            *reinterpret_cast<float2 *>(&sm[yi + 3 * sub1]) = make_float2(ha.hh, hb.hh);
        }
        return 2;
    }
    // general path: one 2x2 block per work item, scalar loads
    const int W1 = g.Wl[1];
    for (int e = srank; e < g.NPL * g.npatch; e += nstagers) {
        const int slot = fdiv(e, g.d_npatch), r = e - slot * g.npatch;
        const int i = fdiv(r, g.d_prow), j = r - i * W1;
        const int y = 2 * i, xx = 2 * j;
        const bool x1 = xx + 1 < W, y1 = y + 1 < H;
        float a = 0.f, bq = 0.f, cq = 0.f, d = 0.f;
        if (slot < nvalid) {
            const T *pa = gsrc + (size_t)slot * img_stride + y * W + xx;
            a = ld1<T, RAW>(pa);
            if (x1) bq = ld1<T, RAW>(pa + 1);
            if (y1) cq = ld1<T, RAW>(pa + W);
            if (x1 && y1) d = ld1<T, RAW>(pa + W + 1);
        }
        const int S = slot * g.slot_stride;
        const int xi = S + off[0] + (y + 2) * p0 + xx + 2;
        sm[xi] = a;
        if (x1) sm[xi + 1] = bq;
        if (y1) sm[xi + p0] = cq;
        if (x1 && y1) sm[xi + p0 + 1] = d;
        const Haar4 h = haar_butterfly(a, bq, cq, d);
        const int yi = S + off[1] + (i + 2) * p1 + j + 2;
        sm[yi] = h.ll;
        sm[yi + sub1] = h.lh;
        sm[yi + 2 * sub1] = h.hl;
        sm[yi + 3 * sub1] = h.hh;
    }
    return 2;
}

// Zero the haloed arrays, the weight table and the output image; the prefetch ring and its barriers, which
// the first bulk copies may already be writing, are left alone.
__device__ __forceinline__ void zero_fill(float *sm, const Geom &g) {
    float4 *v = reinterpret_cast<float4 *>(sm);
    for (int i = threadIdx.x; i < g.raw_off / 4; i += blockDim.x) v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int i = g.out_off / 4 + threadIdx.x; i < g.bar_off / 4; i += blockDim.x) v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
}

// Without room for a raw prefetch buffer the next unit is at least pulled into L2: every thread touches some of
// the unit's 128-byte lines (prefetch only; no registers or shared memory are tied up).
template <typename T>
__device__ __forceinline__ void prefetch_unit_l2(const Geom &g, const T *__restrict__ src, int c0, int b) {
    const char *base = reinterpret_cast<const char *>(src + ((size_t)b * g.C + c0) * g.H * g.W);
    const int bytes = g.NPL * g.plane_bytes;
    for (int o = threadIdx.x * 128; o < bytes; o += blockDim.x * 128)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(base + o));
}

// Issue the bulk copy of one unit's planes into the raw buffer (one thread); a second tensor (grad_out) goes
// right behind the first on the same barrier.
template <typename T>
__device__ __forceinline__ void issue_unit_copies(unsigned long long *bar, char *raw, const Geom &g,
                                                  const T *__restrict__ src, const T *__restrict__ src2, int c0, int b) {
    // the unit (NPL consecutive channels of image b) is one contiguous, 16-byte aligned chunk
    const unsigned bytes = (unsigned)g.NPL * g.plane_bytes;
    if (g.no_copy) return;  // test mode: the barrier is never armed, nothing is in flight
    mbar_expect_tx(bar, bytes * (src2 ? 2u : 1u));
    const size_t po = ((size_t)b * g.C + c0) * g.H * g.W;
    bulk_g2s(raw, src + po, bytes, bar);
    if (src2) bulk_g2s(raw + bytes, src2 + po, bytes, bar);
}

// Start of a block: one thread arms the ring's barriers and sends the first `nstage` units on their way, so
// that the DRAM round trip runs behind the zero fill, the descriptor set-up and the weight table.
template <typename T>
__device__ __forceinline__ void start_prefetch(unsigned long long *bar, char *raw, const Geom &g, const T *__restrict__ src,
                                               const T *__restrict__ src2, int u_begin, int u_end) {
    if (threadIdx.x != 0) return;
    for (int s = 0; s < g.nstage; ++s) mbar_init(bar + s, 1);
    fence_async_smem();
    for (int s = 0; s < g.nstage && u_begin + s < u_end; ++s) {
        const int cgs = (u_begin + s) / g.B;
        issue_unit_copies<T>(bar + s, raw + s * g.stage_bytes, g, src, src2, cgs * g.NPL, u_begin + s - cgs * g.B);
    }
}

// A bounded wait ran out: the block records it in the status word and stops working (its outputs are invalid
// anyway).  Before it leaves, every thread waits - again with the limit - for the copies that are still on
// their way into the ring (the entries of the next nstage - 1 units and the one that was late), so that no
// copy lands in shared memory the block has already given back.
__device__ __forceinline__ void give_up_after_timeout(unsigned long long *bar, const Geom &g, int ring, unsigned parity, int u,
                                                      int u_end, int *status) {
    if (threadIdx.x == 0) atomicExch(status + STATUS_TIMEOUT, (int)g.tag);
    const unsigned limit = g.no_copy ? WAIT_LIMIT_TEST : WAIT_LIMIT;
    for (int s = 0; s < g.nstage && u + s < u_end; ++s) {
        mbar_wait(bar + ring, parity, limit);
        if (++ring == g.nstage) { ring = 0; parity ^= 1u; }
    }
}

// Level l >= 2 from the raw LL band of level l-1 (already in shared memory).  Reads one element past
// an odd grid land in the zero padding.
__device__ __forceinline__ void stage_level(float *sm, const Geom &g, const int *off, int l) {
    const int Wl = g.Wl[l], n = (int)g.d_lvl[l].d;
    const int pp = g.pitch[l - 1], pl = g.pitch[l], subl = g.rows[l] * pl;
    for (int e = threadIdx.x; e < g.NPL * n; e += blockDim.x) {
        const int slot = fdiv(e, g.d_lvl[l]), r = e - slot * n, i = fdiv(r, g.d_lvlw[l]), j = r - i * Wl;
        const int S = slot * g.slot_stride;
        const int si = S + off[l - 1] + (2 * i + 2) * pp + 2 * j + 2;  // even column: 8-byte aligned
        const float2 top = *reinterpret_cast<const float2 *>(&sm[si]);
        const float2 bot = *reinterpret_cast<const float2 *>(&sm[si + pp]);
        const Haar4 h = haar_butterfly(top.x, top.y, bot.x, bot.y);
        const int yi = S + off[l] + (i + 2) * pl + j + 2;
        sm[yi] = h.ll;
        sm[yi + subl] = h.lh;
        sm[yi + 2 * subl] = h.hl;
        sm[yi + 3 * subl] = h.hh;
    }
}

// 4-column x TH-row output tile of a 5x5 correlation.  `src` = array + (TH*ty)*pitch + 4*tx is the
// window's top-left element (the array's halo of 2 makes window row rr = output row + tap row), 16-byte
// aligned; eight floats per window row.
// KEEP: the window's interior (rows 2 .. TH+1, columns 2 .. 5: the tile's own elements) is copied to `keep` on the
// way through the registers.  KT: taps per side that are in use, 5 or 3 - a 3 x 3 kernel sits in the middle of the
// 5 x 5 table and of the 5 x 5 window, its zero border is neither read nor multiplied.
template <int TH, bool KEEP = false, int KT = 5>
__device__ __forceinline__ void conv_tile(const float *__restrict__ src, int pitch, const float (&w)[KK],
                                          float (&acc)[TH][4], float (*keep)[4] = nullptr) {
    constexpr int T0 = (5 - KT) / 2, T1 = 5 - T0;  // taps T0 .. T1-1 per side; window rows T0 .. TH+3-T0
#pragma unroll
    for (int r = 0; r < TH; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;
    // the next window row is fetched while the current one is being used (software pipelining by hand)
    float4 n0 = *reinterpret_cast<const float4 *>(src + T0 * pitch);
    float4 n1 = *reinterpret_cast<const float4 *>(src + T0 * pitch + 4);
#pragma unroll
    for (int rr = T0; rr < TH + 4 - T0; ++rr) {
        const float in[8] = {n0.x, n0.y, n0.z, n0.w, n1.x, n1.y, n1.z, n1.w};
        if (KEEP && rr >= 2 && rr < TH + 2) {
#pragma unroll
            for (int c = 0; c < 4; ++c) keep[rr - 2][c] = in[c + 2];
        }
        if (rr + 1 < TH + 4 - T0) {
            n0 = *reinterpret_cast<const float4 *>(src + (rr + 1) * pitch);
            n1 = *reinterpret_cast<const float4 *>(src + (rr + 1) * pitch + 4);
        }
#pragma unroll
        for (int u = T0; u < T1; ++u) {
            const int r = rr - u;
            if (r >= 0 && r < TH) {
#pragma unroll
                for (int v = T0; v < T1; ++v)
#pragma unroll
                    for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(w[u * 5 + v], in[c + v], acc[r][c]);
            }
        }
    }
}

// The weight-gradient taps of one tile: accw[u][v] += sum over the tile of D[r][c] * Y[r + u][c + v] (window
// coordinates; `d` = the tile's D values, `ysrc` = the window's top-left element).
template <int TH, int KT>
__device__ __forceinline__ void wgrad_taps(const float *__restrict__ ysrc, int pitch, const float (&d)[TH][4], float (&accw)[KK]) {
    constexpr int T0 = (5 - KT) / 2, T1 = 5 - T0;
    // the next window row is fetched while the current one is used
    float4 n0 = *reinterpret_cast<const float4 *>(ysrc + T0 * pitch);
    float4 n1 = *reinterpret_cast<const float4 *>(ysrc + T0 * pitch + 4);
#pragma unroll
    for (int rr = T0; rr < TH + 4 - T0; ++rr) {
        const float in[8] = {n0.x, n0.y, n0.z, n0.w, n1.x, n1.y, n1.z, n1.w};
        if (rr + 1 < TH + 4 - T0) {
            n0 = *reinterpret_cast<const float4 *>(ysrc + (rr + 1) * pitch);
            n1 = *reinterpret_cast<const float4 *>(ysrc + (rr + 1) * pitch + 4);
        }
#pragma unroll
        for (int uu = T0; uu < T1; ++uu) {
            const int dr = rr - uu;
            if (dr >= 0 && dr < TH) {
#pragma unroll
                for (int v = T0; v < T1; ++v)
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) accw[uu * 5 + v] = fmaf(d[dr][cc], in[cc + v], accw[uu * 5 + v]);
            }
        }
    }
}

// Decode a level item of one plane: r in [0, lvl_start[L+1]) -> (level, subband, tile row, tile col).
__device__ __forceinline__ void decode_level_item(const Geom &g, int r, int &l, int &sub, int &tyy, int &txx) {
    l = 1;
    while (r >= g.lvl_start[l + 1]) ++l;
    r -= g.lvl_start[l];
    sub = fdiv(r, g.d_nt[l]);
    r -= sub * (int)g.d_nt[l].d;
    tyy = fdiv(r, g.d_tx[l]);
    txx = r - tyy * g.tx[l];
}

__device__ __forceinline__ void store_row4(float *__restrict__ p, int x0, int W, bool vec, const float *v) {
    if (vec) {
        *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
    } else {
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (x0 + c < W) p[c] = v[c];
    }
}
__device__ __forceinline__ void store_row4(__half *__restrict__ p, int x0, int W, bool vec, const float *v) {
    if (vec) {
        __half2 a = __floats2half2_rn(v[0], v[1]), b = __floats2half2_rn(v[2], v[3]);
        uint2 q;
        q.x = *reinterpret_cast<unsigned *>(&a);
        q.y = *reinterpret_cast<unsigned *>(&b);
        *reinterpret_cast<uint2 *>(p) = q;
    } else {
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (x0 + c < W) p[c] = __float2half_rn(v[c]);
    }
}
__device__ __forceinline__ void store_row4(__nv_bfloat16 *__restrict__ p, int x0, int W, bool vec, const float *v) {
    if (vec) {
        __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
        uint2 q;
        q.x = *reinterpret_cast<unsigned *>(&a);
        q.y = *reinterpret_cast<unsigned *>(&b);
        *reinterpret_cast<uint2 *>(p) = q;
    } else {
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (x0 + c < W) p[c] = __float2bfloat16_rn(v[c]);
    }
}

// Store one finished 4 x TH tile: straight to global memory (vector rows where the width allows), or, in
// bulk-out mode, element by element into the unit's shared-memory image that one bulk store sends out.
template <typename T, int TH>
__device__ __forceinline__ void store_tile(const Geom &g, float *sm, T *__restrict__ gplane, int bslot, int tyy, int txx,
                                           float (&acc)[TH][4]) {
    if (g.bulk_out) {
        T *ob = reinterpret_cast<T *>(sm + g.out_off) + bslot * (g.H * g.W) + (TH * tyy) * g.W + 4 * txx;
#pragma unroll
        for (int r = 0; r < TH; ++r) {
            if (TH * tyy + r < g.H) {
#pragma unroll
                for (int cc = 0; cc < 4; ++cc)
                    if (4 * txx + cc < g.W) stf(ob + r * g.W + cc, acc[r][cc]);
            }
        }
    } else {
        T *oa = gplane + (size_t)(TH * tyy) * g.W + 4 * txx;
        const bool vec = g.vec && (4 * txx + 3 < g.W);
#pragma unroll
        for (int r = 0; r < TH; ++r)
            if (TH * tyy + r < g.H) store_row4(oa + (size_t)r * g.W, 4 * txx, g.W, vec, acc[r]);
    }
}

// ------------------------------------------------------------------ forward / input-gradient kernel
// Adds the Proposition 2 terms of all levels to one 4x4 pixel block (block row t4, block column tx of
// the plane) held in a[0..3][0..3]; `bias` is the folded bias.
__device__ __forceinline__ void synth_block(const float *S, const Geom &g, int t4, int txx, float bias, float (*a)[4]) {
    const int L = g.L;
    // level 1: coefficient (2*t4+ci, 2*tx+cj) feeds pixels (2ci+by, 2cj+bx) of the block
    if (L >= 1) {
        const int zp = g.zpitch[1], zs = g.zrows[1] * zp;
        const float *z = S + g.offZ[1] + (2 * t4) * zp + 2 * txx;
#pragma unroll
        for (int ci = 0; ci < 2; ++ci) {
            const float2 ll = *reinterpret_cast<const float2 *>(z + ci * zp);
            const float2 lh = *reinterpret_cast<const float2 *>(z + zs + ci * zp);
            const float2 hl = *reinterpret_cast<const float2 *>(z + 2 * zs + ci * zp);
            const float2 hh = *reinterpret_cast<const float2 *>(z + 3 * zs + ci * zp);
#pragma unroll
            for (int cj = 0; cj < 2; ++cj) {
                const float LLv = cj ? ll.y : ll.x, LHv = cj ? lh.y : lh.x, HLv = cj ? hl.y : hl.x,
                            HHv = cj ? hh.y : hh.x;
                const float pp = LLv + LHv, pm = LLv - LHv, qp = HLv + HHv, qm = HLv - HHv;
                a[2 * ci][2 * cj] = fmaf(0.5f, pp + qp, a[2 * ci][2 * cj]);
                a[2 * ci][2 * cj + 1] = fmaf(0.5f, pp - qp, a[2 * ci][2 * cj + 1]);
                a[2 * ci + 1][2 * cj] = fmaf(0.5f, pm + qm, a[2 * ci + 1][2 * cj]);
                a[2 * ci + 1][2 * cj + 1] = fmaf(0.5f, pm - qm, a[2 * ci + 1][2 * cj + 1]);
            }
        }
    }
    if (L >= 2) {
        // levels >= 3: the whole block sits in one quadrant of the coefficient's 2^l x 2^l block
        float deep = bias, scale = 0.25f;
        for (int l = 3; l <= L; ++l) {
            scale *= 0.5f;
            const int zp = g.zpitch[l], zs = g.zrows[l] * zp;
            const float *z = S + g.offZ[l] + (t4 >> (l - 2)) * zp + (txx >> (l - 2));
            const float sy = ((t4 >> (l - 3)) & 1) ? -1.f : 1.f, sx = ((txx >> (l - 3)) & 1) ? -1.f : 1.f;
            const float p = fmaf(sy, z[zs], z[0]), q = fmaf(sy, z[3 * zs], z[2 * zs]);
            deep = fmaf(scale, fmaf(sx, q, p), deep);
        }
        // level 2: coefficient (t4, tx); pixel (r, c) of the block takes its signs from (r>>1, c>>1)
        const int zp = g.zpitch[2], zs = g.zrows[2] * zp;
        const float *z = S + g.offZ[2] + t4 * zp + txx;
        const float LLv = z[0], LHv = z[zs], HLv = z[2 * zs], HHv = z[3 * zs];
        const float pp = LLv + LHv, pm = LLv - LHv, qp = HLv + HHv, qm = HLv - HHv;
        float t2[2][2];
        t2[0][0] = fmaf(0.25f, pp + qp, deep);
        t2[0][1] = fmaf(0.25f, pp - qp, deep);
        t2[1][0] = fmaf(0.25f, pm + qm, deep);
        t2[1][1] = fmaf(0.25f, pm - qm, deep);
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) a[r][c] += t2[r >> 1][c >> 1];
    } else {
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) a[r][c] += bias;
    }
}

// FLIP = false: out = WTConv(x).  FLIP = true: the same dataflow on grad_out with every kernel rotated
// by 180 degrees and no bias gives grad_x.  MINB = resident blocks per SM the register budget is sized for.
template <typename T, bool FLIP, int MAXT, int MINB, int TH, int KT>
__global__ void __launch_bounds__(MAXT, MINB)
plane_fwd_kernel(const __grid_constant__ Geom g, const T *__restrict__ x, const float *__restrict__ w0,
                 const float *__restrict__ s0, const float *__restrict__ b0, const float *__restrict__ wl,
                 const float *__restrict__ sl, T *__restrict__ out, int *__restrict__ status) {
    extern __shared__ __align__(16) float sm[];
    const int tid = threadIdx.x, nthr = blockDim.x;
    float *wtab = sm + g.wtab_off;
    unsigned long long *bar = reinterpret_cast<unsigned long long *>(sm + g.bar_off);
    char *raw = reinterpret_cast<char *>(sm + g.raw_off);
    const int u_begin = (int)((long long)blockIdx.x * g.units / gridDim.x);
    const int u_end = (int)((long long)(blockIdx.x + 1) * g.units / gridDim.x);
    zero_fill(sm, g);
    unsigned parity = 0;
    int ring = 0;  // ring entry the current unit arrives in
    const unsigned wait_limit = g.no_copy ? WAIT_LIMIT_TEST : WAIT_LIMIT;
    const int L = g.L, nlv = g.lvl_start[L + 1];
    const int nlevel_items = g.NPL * nlv, nitems = nlevel_items + g.NPL * g.nbase;
    const size_t HW = (size_t)g.H * g.W;
    int c_prev = -1;
    // Staging order: the threads that hold a base tile (the last `nbase_thr` items of the list) are busy with
    // the synthesis of the previous unit when the next one is staged, so the others stage, two patches each
    // if need be; only if they are too few does every thread take part.
    // Staging is done by whole warps that hold level tiles only (threads below the first base tile, rounded
    // down to a warp) while the others run the previous unit's synthesis; if those are too few, by everybody.
    int nstagers = (nlevel_items / 32) * 32;
    if (nstagers > nthr) nstagers = nthr;
    {   // staging work items of one unit; more than two per stager: everybody stages
        const int nwork = g.NPL * (L == 0 ? g.H * g.W : ((g.vec && L >= 2) ? g.npatch4 : g.npatch));
        if (nstagers * 4 < nthr || nwork > 2 * nstagers) nstagers = nthr;
    }
    const int srank = tid < nstagers ? tid : 0x3fffffff;
    // hoisted descriptors: two tiles and two staging patches per thread cover the plans in use
    constexpr int MAXI = 2;
    const bool hoist_items = nitems <= MAXI * nthr;
    const bool hoist_patch = g.vec && L >= 2 && g.NPL * g.npatch4 <= 2 * nstagers;
    ItemD items[MAXI];
    int bslot = 0, tyy = 0, txx = 0;
    bool has_base = false;
#pragma unroll
    for (int k = 0; k < MAXI; ++k)
        items[k] = decode_item(g, hoist_items ? tid + k * nthr : 0x3fffffff, nlevel_items, nitems, bslot, tyy, txx, has_base);
    PatchD patch0 = decode_patch(g, g.offA, hoist_patch ? srank : 0x3fffffff);
    PatchD patch1 = decode_patch(g, g.offA, hoist_patch && srank < nstagers ? srank + nstagers : 0x3fffffff);
    // Everything above touched shared memory and registers only and may have run beside the tail of the kernel
    // before this one; global memory is used from here on.  The input-gradient instantiation is followed by the small
    // epilogue and releases it at the end (see plane_bwd_kernel).
    if (!FLIP) dependents_may_start();
    wait_for_predecessor();
    if (blockIdx.x == 0 && tid == 0) status[STATUS_LAUNCH] = (int)g.tag;
    if (g.bulk) start_prefetch<T>(bar, raw, g, x, nullptr, u_begin, u_end);
    __syncthreads();
    // (channel group, image) of the current unit, carried along instead of divided out per unit
    int cg = u_begin / g.B, b = u_begin - cg * g.B;
    for (int u = u_begin; u < u_end; ++u, (++b == g.B ? (b = 0, ++cg) : 0)) {
        const int c = cg * g.NPL;
        const int nvalid = g.C - c < g.NPL ? g.C - c : g.NPL;
        if (c != c_prev) {  // units are group-major: the tables survive all images of a channel group
            build_weight_table(wtab, g, c, FLIP, w0, s0, FLIP ? nullptr : b0, wl, sl);
            c_prev = c;
        }
        int lnext;
        bool late = false;
        if (g.bulk) {
            // every thread polls the copy barrier itself (bounded); a copy that never lands is noticed by the
            // whole block at the staging barrier below
            late = !mbar_wait(bar + ring, parity, wait_limit);
            const T *rx = reinterpret_cast<const T *>(raw + ring * g.stage_bytes);
            if (hoist_patch) {
                run_patch<T, true>(sm, g, patch0, rx, nvalid);
                run_patch<T, true>(sm, g, patch1, rx, nvalid);
                lnext = 3;
            } else {
                lnext = stage_input<T, true>(sm, g, g.offA, rx, c, b, srank, nstagers);
            }
        } else if (hoist_patch) {
            const T *gsrc = x + ((size_t)b * g.C + c) * HW;
            run_patch<T, false>(sm, g, patch0, gsrc, nvalid);
            run_patch<T, false>(sm, g, patch1, gsrc, nvalid);
            lnext = 3;
        } else {
            lnext = stage_input<T, false>(sm, g, g.offA, x, c, b, srank, nstagers);
        }
        if (g.bulk) {
            if (__syncthreads_or(late)) {
                give_up_after_timeout(bar, g, ring, parity, u, u_end, status);
                break;
            }
        } else {
            __syncthreads();
        }
        if (g.bulk) {
            // this ring entry is free again: refill it with the unit `nstage` ahead, behind the math
            if (tid == 0 && u + g.nstage < u_end) {
                fence_async_smem();
                const int cgn = (u + g.nstage) / g.B;
                issue_unit_copies<T>(bar + ring, raw + ring * g.stage_bytes, g, x, nullptr, cgn * g.NPL,
                                     (u + g.nstage) - cgn * g.B);
            }
            if (++ring == g.nstage) { ring = 0; parity ^= 1u; }
        } else if (u + 1 < u_end) {  // no room for a raw buffer: at least warm the next unit in L2
            const int cgn = b + 1 == g.B ? cg + 1 : cg;
            if (cgn * g.NPL + g.NPL <= g.C) prefetch_unit_l2<T>(g, x, cgn * g.NPL, (u + 1) - cgn * g.B);
        }
        for (int l = lnext; l <= L; ++l) {
            stage_level(sm, g, g.offA, l);
            __syncthreads();
        }
        // ---- one item list: level tiles (Z^l = Wfold^l (*) Y^l) first, base tiles last; a thread's last
        //      item may be a base tile, which stays in registers across the barrier
        float acc[TH][4];
        {
            // one copy of the (large, fully unrolled) tile code serves every item: the loop is kept rolled and
            // the descriptor is either one of the two hoisted ones or decoded on the spot
            const int nmine = hoist_items ? MAXI : (nitems - tid + nthr - 1) / nthr;
            if (!hoist_items) has_base = false;
#pragma unroll 1
            for (int k = 0; k < nmine; ++k) {
                ItemD d;
                if (hoist_items) {
                    d = k == 0 ? items[0] : items[1];
                } else {
                    bool isb = false;
                    d = decode_item(g, tid + k * nthr, nlevel_items, nitems, bslot, tyy, txx, isb);
                    has_base = isb;
                }
                if (d.meta < 0) {
                    float w[KK];
                    load_weights(sm + d.wt, w);
                    conv_tile<TH, false, KT>(sm + d.src, d.meta & 0x3ff, w, acc);
                    if (d.z >= 0) {
                        const int zp = (d.meta >> 10) & 0x3ff, zleft = (d.meta >> 20) & 0xf;
                        float *z = sm + d.z;
#pragma unroll
                        for (int r = 0; r < TH; ++r)
                            if (r < zleft) *reinterpret_cast<float4 *>(z + r * zp) = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
                    }
                }
            }
        }
        const float bias = wtab[bslot * (1 + 4 * L) * WT_STRIDE + KK];
        if (g.bulk_out && tid == 0) bulk_store_wait_read();  // the previous unit's store has drained the output image
        __syncthreads();
        if (has_base) {
            const float *S = sm + bslot * g.slot_stride;
#pragma unroll
            for (int hb = 0; hb < TH / 4; ++hb) synth_block(S, g, (TH / 4) * tyy + hb, txx, bias, &acc[4 * hb]);
            if (bslot < nvalid) store_tile<T, TH>(g, sm, out + ((size_t)b * g.C + c + bslot) * HW, bslot, tyy, txx, acc);
        }
        if (g.bulk_out) {  // the unit is contiguous in global memory: one bulk store once every tile is in place
            fence_async_smem();  // every writer orders its shared-memory writes before the async proxy's reads
            __syncthreads();
            if (tid == 0) bulk_s2g(out + ((size_t)b * g.C + c) * HW, sm + g.out_off, (unsigned)g.NPL * g.plane_bytes);
        }
        // The next unit's staging overwrites x / Y (last read before the barrier above) and possibly the
        // weight table (bias already in a register); Z is next written after the staging barriers.
    }
    if (FLIP) dependents_may_start();
    if (g.bulk_out && tid == 0) bulk_store_wait_read();  // shared memory must outlive the last bulk store's reads
}

// ------------------------------------------------------------------ weight-gradient kernel
// dWfold^l[u,v] += sum_{i,j} D^l[i,j] Y^l[i+u-2, j+v-2] (and the base class with grad_out and x), Sec. 2.2.
// Thread t serves class cls(t) only (class-major allocation thr_start[]); accumulators persist over all
// units of a channel and are flushed to `part0` / `partl` when the channel changes.
template <typename T, int MAXT, int MINB, int TH, int KT>
__global__ void __launch_bounds__(MAXT, MINB)
plane_wgrad_kernel(const __grid_constant__ Geom g, const T *__restrict__ x, const T *__restrict__ go,
                   float *__restrict__ part0, float *__restrict__ partl /* level l at l*C*np*100 */,
                   int *__restrict__ status) {
    extern __shared__ __align__(16) float sm[];
    const int tid = threadIdx.x, nthr = blockDim.x;
    unsigned long long *bar = reinterpret_cast<unsigned long long *>(sm + g.bar_off);
    char *raw = reinterpret_cast<char *>(sm + g.raw_off);
    const int u_begin = (int)((long long)blockIdx.x * g.units / gridDim.x);
    const int u_end = (int)((long long)(blockIdx.x + 1) * g.units / gridDim.x);
    zero_fill(sm, g);
    const int arrays_floats = g.raw_off;  // haloed arrays (and reduction scratch) end where the raw buffer starts
    unsigned parity = 0;
    const int L = g.L, ncls = 1 + 4 * L;
    int cls = 0;
    while (cls < ncls && tid >= g.thr_start[cls + 1]) ++cls;
    const bool active = cls < ncls;
    const int lvl = active ? (cls == 0 ? 0 : 1 + ((cls - 1) >> 2)) : 0, sub = (cls - 1) & 3;
    const int kth = active ? tid - g.thr_start[cls] : 0, nth = active ? g.thr_start[cls + 1] - g.thr_start[cls] : 1;
    const int ntile = g.tx[lvl] * g.ty[lvl];
    const int pl = g.pitch[lvl];
    const int suboff = (lvl == 0 ? 0 : sub * g.rows[lvl] * pl);
    float acc[KK], gsum = 0.f;
#pragma unroll
    for (int t = 0; t < KK; ++t) acc[t] = 0.f;
    int ring = 0;
    dependents_may_start();
    wait_for_predecessor();  // shared memory and registers only up to here
    if (blockIdx.x == 0 && tid == 0) status[STATUS_LAUNCH] = (int)g.tag;
    if (g.bulk) start_prefetch<T>(bar, raw, g, x, go, u_begin, u_end);
    __syncthreads();
    int c = u_begin / g.B, b = u_begin - c * g.B;  // this kernel is planned with one plane per unit: group = channel
    for (int u = u_begin; u < u_end; ++u, (++b == g.B ? (b = 0, ++c) : 0)) {
        int lnext;
        if (g.bulk) {
            const bool late = !mbar_wait(bar + ring, parity, g.no_copy ? WAIT_LIMIT_TEST : WAIT_LIMIT);
            const T *rx = reinterpret_cast<const T *>(raw + ring * g.stage_bytes);
            const T *rg = reinterpret_cast<const T *>(raw + ring * g.stage_bytes + (size_t)g.NPL * g.plane_bytes);
            lnext = stage_input<T, true>(sm, g, g.offA, rx, c, b, tid, nthr);
            stage_input<T, true>(sm, g, g.offG, rg, c, b, tid, nthr);
            if (__syncthreads_or(late)) {
                give_up_after_timeout(bar, g, ring, parity, u, u_end, status);
                break;
            }
        } else {
            lnext = stage_input<T, false>(sm, g, g.offA, x, c, b, tid, nthr);
            stage_input<T, false>(sm, g, g.offG, go, c, b, tid, nthr);
            __syncthreads();
        }
        if (g.bulk) {
            if (tid == 0 && u + g.nstage < u_end) {
                fence_async_smem();
                const int cgn = (u + g.nstage) / g.B;
                issue_unit_copies<T>(bar + ring, raw + ring * g.stage_bytes, g, x, go, cgn * g.NPL,
                                     (u + g.nstage) - cgn * g.B);
            }
            if (++ring == g.nstage) { ring = 0; parity ^= 1u; }
        } else if (u + 1 < u_end) {
            const int cn = b + 1 == g.B ? c + 1 : c, bn = (u + 1) - cn * g.B;
            prefetch_unit_l2<T>(g, x, cn, bn);
            prefetch_unit_l2<T>(g, go, cn, bn);
        }
        for (int l = lnext; l <= L; ++l) {
            stage_level(sm, g, g.offA, l);
            stage_level(sm, g, g.offG, l);
            __syncthreads();
        }
        if (active) {
            for (int it = kth; it < g.NPL * ntile; it += nth) {
                const int slot = fdiv(it, g.d_nt[lvl]), r = it - slot * ntile;
                const int tyy = fdiv(r, g.d_tx[lvl]), txx = r - tyy * g.tx[lvl];
                const float *S = sm + slot * g.slot_stride;
                const float *ysrc = S + g.offA[lvl] + suboff + TH * tyy * pl + 4 * txx;
                // D tile = columns 4tx+2..4tx+5 of rows TH*ty+2.. (8-byte aligned)
                const float *dsrc = S + g.offG[lvl] + suboff + (TH * tyy + 2) * pl + 4 * txx + 2;
                float d[TH][4];
#pragma unroll
                for (int rr = 0; rr < TH; ++rr) {
                    const float2 q0 = *reinterpret_cast<const float2 *>(dsrc + rr * pl);
                    const float2 q1 = *reinterpret_cast<const float2 *>(dsrc + rr * pl + 2);
                    d[rr][0] = q0.x; d[rr][1] = q0.y; d[rr][2] = q1.x; d[rr][3] = q1.y;
                }
                if (cls == 0) {
#pragma unroll
                    for (int rr = 0; rr < TH; ++rr)
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) gsum += d[rr][cc];
                }
                wgrad_taps<TH, KT>(ysrc, pl, d, acc);
            }
        }
        __syncthreads();
        const bool last_of_channel = (u + 1 == u_end) || (b + 1 == g.B);
        if (last_of_channel) {
            // block tree through shared memory: every thread parks its 26 sums in the (now idle) array
            // region, then one thread per (class, tap) adds its class's threads in index order
            float *scr = sm;
#pragma unroll
            for (int t = 0; t < KK; ++t) scr[(size_t)tid * (KK + 1) + t] = acc[t];
            scr[(size_t)tid * (KK + 1) + KK] = gsum;
            __syncthreads();
            const int slotp = blockIdx.x - block_of_unit((long long)c * g.B, gridDim.x, g.units);
            for (int e = tid; e < ncls * (KK + 1); e += nthr) {
                const int c2 = e / (KK + 1), t = e - c2 * (KK + 1);
                if (c2 > 0 && t == KK) continue;
                float s = 0.f;
                for (int th = g.thr_start[c2]; th < g.thr_start[c2 + 1]; ++th) s += scr[(size_t)th * (KK + 1) + t];
                if (c2 == 0) {
                    part0[((size_t)c * g.np + slotp) * (KK + 1) + t] = s;
                } else {
                    const int l = (c2 - 1) >> 2, sb_ = (c2 - 1) & 3;
                    partl[(size_t)l * g.C * g.np * 4 * KK + (((size_t)c * g.np + slotp) * 4 + sb_) * KK + t] = s;
                }
            }
            __syncthreads();
            for (int i = tid; i < arrays_floats; i += nthr) sm[i] = 0.f;  // restore the zero halos (raw buffer untouched)
#pragma unroll
            for (int t = 0; t < KK; ++t) acc[t] = 0.f;
            gsum = 0.f;
            __syncthreads();
        }
    }
}

// ------------------------------------------------------------------ fused backward kernel
// One pass over x and grad_out gives grad_x and the weight-gradient partial sums.  Both decompositions are
// staged (x -> X, Y^l; grad_out -> G, D^l).  Each thread owns exactly one tile of the item list (so its
// parameter class never changes) and does two things with it:
//   weight gradient  dWfold[u,v] += sum_tile D[i,j] * Y[i+u-2, j+v-2]          (Sec. 2.2; 25 register accumulators
//                                                                              that live across all images of a channel)
//   input gradient   the forward dataflow on grad_out with rotated kernels: conv of the D window, then the
//                    closed-form synthesis of Proposition 2 and the store of grad_x.
// Used when a unit's item list fits one round of the block (<= 256 tiles); otherwise the separate weight-
// gradient and input-gradient kernels run.
template <typename T, int TH, int BULK, int KT>  // BULK: tensors prefetched by bulk copy (0 none, 2 x and grad_out)
__global__ void __launch_bounds__(256, 2)
plane_bwd_kernel(const __grid_constant__ Geom g, const T *__restrict__ x, const T *__restrict__ go,
                 const float *__restrict__ w0, const float *__restrict__ s0, const float *__restrict__ wl,
                 const float *__restrict__ sl, T *__restrict__ gx, float *__restrict__ part0,
                 float *__restrict__ partl /* level l at l*C*np*100 */, int *__restrict__ status) {
    extern __shared__ __align__(16) float sm[];
    const int tid = threadIdx.x, nthr = blockDim.x;
    float *wtab = sm + g.wtab_off;
    unsigned long long *bar = reinterpret_cast<unsigned long long *>(sm + g.bar_off);
    char *raw = reinterpret_cast<char *>(sm + g.raw_off);
    const int u_begin = (int)((long long)blockIdx.x * g.units / gridDim.x);
    const int u_end = (int)((long long)(blockIdx.x + 1) * g.units / gridDim.x);
    zero_fill(sm, g);
    unsigned parity = 0;
    const int L = g.L, nlv = g.lvl_start[L + 1], ncls = 1 + 4 * L;
    const int nlevel_items = g.NPL * nlv, nitems = nlevel_items + g.NPL * g.nbase;
    const size_t HW = (size_t)g.H * g.W;
    int bslot = 0, tyy = 0, txx = 0;
    bool has_base = false;
    const ItemD item = decode_item(g, tid, nlevel_items, nitems, bslot, tyy, txx, has_base);
    const int cls = (item.meta >> 24) & 0x3f;
    // No barrier separates a unit's synthesis (which reads only Z and registers) from the next unit's staging.
    // With the planes already in shared memory (BULK == 2) the staging is left to the whole warps that hold
    // level tiles only while the base-tile threads finish the synthesis - as long as one patch each covers the
    // unit.  Otherwise every thread takes part: two patches per thread make the exposed load-to-store chain twice
    // as long (measured slower at 56 x 56, from global memory as well as from the ring).
    int nstagers = (nlevel_items / 32) * 32;
    if (nstagers > nthr) nstagers = nthr;
    if (BULK != 2 || nstagers * 4 < nthr || g.NPL * g.npatch4 > nstagers) nstagers = nthr;
    const int srank = tid < nstagers ? tid : 0x3fffffff;
    const bool hoist_patch = g.vec && L >= 2 && g.NPL * g.npatch4 <= 2 * nstagers;
    const PatchD patch0 = decode_patch(g, g.offA, hoist_patch ? srank : 0x3fffffff);
    const PatchD patch1 = decode_patch(g, g.offA, hoist_patch && srank < nstagers ? srank + nstagers : 0x3fffffff);
    const int dA0 = g.offG[0] - g.offA[0], dA1 = L >= 1 ? g.offG[1] - g.offA[1] : 0, dA2 = L >= 2 ? g.offG[2] - g.offA[2] : 0;
    float accw[KK], gsum = 0.f;
#pragma unroll
    for (int t = 0; t < KK; ++t) accw[t] = 0.f;
    int c_prev = -1;
    int ring = 0;
    wait_for_predecessor();  // shared memory and registers only up to here (dependents are released at the end)
    if (blockIdx.x == 0 && tid == 0) status[STATUS_LAUNCH] = (int)g.tag;
    if (BULK) start_prefetch<T>(bar, raw, g, x, go, u_begin, u_end);
    __syncthreads();
    int cg = u_begin / g.B, b = u_begin - cg * g.B;
    for (int u = u_begin; u < u_end; ++u, (++b == g.B ? (b = 0, ++cg) : 0)) {
        const int c = cg * g.NPL;
        const int nvalid = g.C - c < g.NPL ? g.C - c : g.NPL;
        if (c != c_prev) {
            build_weight_table(wtab, g, c, true, w0, s0, nullptr, wl, sl);
            c_prev = c;
        }
        int lnext;
        bool late = false;
        if (BULK) {
            late = !mbar_wait(bar + ring, parity, g.no_copy ? WAIT_LIMIT_TEST : WAIT_LIMIT);
            const T *rx = reinterpret_cast<const T *>(raw + ring * g.stage_bytes);
            const T *rg = reinterpret_cast<const T *>(raw + ring * g.stage_bytes + (size_t)g.NPL * g.plane_bytes);
            if (hoist_patch) {
                run_patch<T, true>(sm, g, patch0, rx, nvalid);
                run_patch<T, true>(sm, g, patch0, rg, nvalid, dA0, dA1, dA2);
                run_patch<T, true>(sm, g, patch1, rx, nvalid);
                run_patch<T, true>(sm, g, patch1, rg, nvalid, dA0, dA1, dA2);
                lnext = 3;
            } else {
                lnext = stage_input<T, true>(sm, g, g.offA, rx, c, b, tid, nthr);
                stage_input<T, true>(sm, g, g.offG, rg, c, b, tid, nthr);
            }
        } else if (hoist_patch) {
            const size_t po = ((size_t)b * g.C + c) * HW;
            run_patch_pair<T, false>(sm, g, patch0, x + po, go + po, nvalid, dA0, dA1, dA2);
            run_patch_pair<T, false>(sm, g, patch1, x + po, go + po, nvalid, dA0, dA1, dA2);
            lnext = 3;
        } else {
            lnext = stage_input<T, false>(sm, g, g.offA, x, c, b, tid, nthr);
            stage_input<T, false>(sm, g, g.offG, go, c, b, tid, nthr);
        }
        if (BULK) {
            if (__syncthreads_or(late)) {
                give_up_after_timeout(bar, g, ring, parity, u, u_end, status);
                break;
            }
        } else {
            __syncthreads();
        }
        if (BULK) {
            if (tid == 0 && u + g.nstage < u_end) {
                fence_async_smem();
                const int cgn = (u + g.nstage) / g.B;
                issue_unit_copies<T>(bar + ring, raw + ring * g.stage_bytes, g, x, go, cgn * g.NPL,
                                     (u + g.nstage) - cgn * g.B);
            }
            if (++ring == g.nstage) { ring = 0; parity ^= 1u; }
        }
        if (!BULK && u + 1 < u_end) {  // no ring: the next unit is warmed in L2 behind this unit's math
            const int cgn = b + 1 == g.B ? cg + 1 : cg, bn = (u + 1) - cgn * g.B;
            if (cgn * g.NPL + g.NPL <= g.C) {
                prefetch_unit_l2<T>(g, x, cgn * g.NPL, bn);
                prefetch_unit_l2<T>(g, go, cgn * g.NPL, bn);
            }
        }
        for (int l = lnext; l <= L; ++l) {
            stage_level(sm, g, g.offA, l);
            stage_level(sm, g, g.offG, l);
            __syncthreads();
        }
        float acc[TH][4];
        if (item.meta < 0) {
            const int pitch = item.meta & 0x3ff;
            const float *ysrc = sm + item.src;            // Y window (x side)
            const float *gsrc = sm + item.src + item.dg;  // D window (grad_out side)
            // With 4-row tiles the registers allow the rotated convolution to go first and to hand the tile's D values
            // (the interior of the window it reads anyway) to the weight-gradient taps; with 8-row tiles the D values
            // are loaded on their own.
            float d[TH][4];
            if (TH == 4) {
                float w[KK];
                load_weights(sm + item.wt, w);
                conv_tile<TH, true, KT>(gsrc, pitch, w, acc, d);
            } else {
#pragma unroll
                for (int rr = 0; rr < TH; ++rr) {
                    const float2 q0 = *reinterpret_cast<const float2 *>(gsrc + (rr + 2) * pitch + 2);
                    const float2 q1 = *reinterpret_cast<const float2 *>(gsrc + (rr + 2) * pitch + 4);
                    d[rr][0] = q0.x; d[rr][1] = q0.y; d[rr][2] = q1.x; d[rr][3] = q1.y;
                }
            }
            {
                // weight gradient: the tile's D values are the window's interior
                if (cls == 0) {
#pragma unroll
                    for (int rr = 0; rr < TH; ++rr)
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) gsum += d[rr][cc];
                }
                wgrad_taps<TH, KT>(ysrc, pitch, d, accw);
            }
            if (TH != 4) {  // input gradient: rotated-kernel conv of the D window
                float w[KK];
                load_weights(sm + item.wt, w);
                conv_tile<TH, false, KT>(gsrc, pitch, w, acc);
            }
            if (item.z >= 0) {
                const int zp = (item.meta >> 10) & 0x3ff, zleft = (item.meta >> 20) & 0xf;
                float *z = sm + item.z;
#pragma unroll
                for (int r = 0; r < TH; ++r)
                    if (r < zleft) *reinterpret_cast<float4 *>(z + r * zp) = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
            }
        }
        if (BULK && g.bulk_out && tid == 0) bulk_store_wait_read();  // the previous unit's store has drained the output image
        __syncthreads();
        if (has_base) {
            const float *S = sm + bslot * g.slot_stride;
#pragma unroll
            for (int hb = 0; hb < TH / 4; ++hb) synth_block(S, g, (TH / 4) * tyy + hb, txx, 0.f, &acc[4 * hb]);
            if (bslot < nvalid) store_tile<T, TH>(g, sm, gx + ((size_t)b * g.C + c + bslot) * HW, bslot, tyy, txx, acc);
        }
        if (BULK && g.bulk_out) {
            fence_async_smem();  // every writer orders its shared-memory writes before the async proxy's reads
            __syncthreads();
            if (tid == 0) bulk_s2g(gx + ((size_t)b * g.C + c) * HW, sm + g.out_off, (unsigned)g.NPL * g.plane_bytes);
        }
        const bool last_of_channel = (u + 1 == u_end) || (b + 1 == g.B);
        if (last_of_channel) {
            // block tree through shared memory: park the 26 sums and the class of every thread in the array
            // region (idle now), then one thread per (class, tap) adds its class's threads in index order
            __syncthreads();
            float *scr = sm;
#pragma unroll
            for (int t = 0; t < KK; ++t) scr[tid * (KK + 2) + t] = accw[t];
            scr[tid * (KK + 2) + KK] = gsum;
            const int mytag = item.meta < 0 ? item.slot * 64 + cls : -1;
            scr[tid * (KK + 2) + KK + 1] = __int_as_float(mytag);
            __syncthreads();
            // the threads of one (plane, class) are neighbours in the item list: note where each run starts and ends
            int *run_start = reinterpret_cast<int *>(scr + nthr * (KK + 2)), *run_end = run_start + g.NPL * ncls;
            if (mytag >= 0) {
                if (tid == 0 || __float_as_int(scr[(tid - 1) * (KK + 2) + KK + 1]) != mytag) run_start[item.slot * ncls + cls] = tid;
                if (tid == nthr - 1 || __float_as_int(scr[(tid + 1) * (KK + 2) + KK + 1]) != mytag) run_end[item.slot * ncls + cls] = tid + 1;
            }
            __syncthreads();
            const int slotp = blockIdx.x - block_of_unit((long long)cg * g.B, gridDim.x, g.units);
            for (int e = tid; e < nvalid * ncls * (KK + 1); e += nthr) {
                const int sc = e / (KK + 1), t = e - sc * (KK + 1), slot = sc / ncls, c2 = sc - slot * ncls;
                if (c2 > 0 && t == KK) continue;
                const int ch = c + slot;
                float sacc = 0.f;
                const int th1 = run_end[sc];  // known trip count: the loads of the sum do not wait for one another
                for (int th = run_start[sc]; th < th1; ++th) sacc += scr[th * (KK + 2) + t];
                if (c2 == 0) {
                    part0[((size_t)ch * g.np + slotp) * (KK + 1) + t] = sacc;
                } else {
                    const int l = (c2 - 1) >> 2, sb_ = (c2 - 1) & 3;
                    partl[(size_t)l * g.C * g.np * 4 * KK + (((size_t)ch * g.np + slotp) * 4 + sb_) * KK + t] = sacc;
                }
            }
            __syncthreads();
            {   // restore the zero halos under the scratch (the rest of the arrays was not touched)
                int nz = (nthr * (KK + 2) + 2 * g.NPL * ncls + 3) / 4;
                if (nz > g.wtab_off / 4) nz = g.wtab_off / 4;
                for (int i = tid; i < nz; i += nthr) reinterpret_cast<float4 *>(sm)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int t = 0; t < KK; ++t) accw[t] = 0.f;
            gsum = 0.f;
            __syncthreads();  // the arrays are zeroed again before anybody stages into them
        }
        // No barrier here: the next unit's staging overwrites x / Y / D (last read before the barrier that
        // follows the tile phase) while the base-tile threads may still run this unit's synthesis, which
        // reads only Z (next written after the staging barriers) and registers.
    }
    // The kernel behind this one is the small parameter-gradient epilogue: released any earlier, its blocks would sit
    // on the SMs whose blocks finish first and keep the next persistent kernel from spreading over all SMs at once.
    dependents_may_start();
    if (BULK && g.bulk_out && tid == 0) bulk_store_wait_read();
}

// ------------------------------------------------------------------ host-side planning
inline void fill_common(Geom &g, int B, int C, int H, int W, int L, int elem_bytes, int TH) {
    g.B = B; g.C = C; g.H = H; g.W = W; g.L = L; g.th = TH;
    g.Hl[0] = H; g.Wl[0] = W;
    for (int l = 1; l <= MAXL; ++l) { g.Hl[l] = (g.Hl[l - 1] + 1) / 2; g.Wl[l] = (g.Wl[l - 1] + 1) / 2; }
    for (int l = 0; l <= L; ++l) {
        g.ty[l] = (g.Hl[l] + TH - 1) / TH;
        g.tx[l] = pad4(g.Wl[l]) / 4;
        g.rows[l] = g.ty[l] * TH + 4;
        g.pitch[l] = pad4(g.Wl[l]) + 4;
    }
    g.nbase = g.tx[0] * g.ty[0];
    g.lvl_start[0] = 0; g.lvl_start[1] = 0;
    for (int l = 1; l <= L; ++l) g.lvl_start[l + 1] = g.lvl_start[l] + 4 * g.tx[l] * g.ty[l];
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
    g.npatch4 = ((H + 3) / 4) * (W / 4 > 0 ? W / 4 : 1);
    g.d_npatch4 = make_fastdiv(g.npatch4);
    g.plane_bytes = H * W * elem_bytes;
    g.bulk = 0;  // decided per plan: a unit of NPL planes must be a 16-byte multiple and C a multiple of NPL
    g.raw_slot_bytes = g.plane_bytes;
}

// Tail of the shared-memory layout: [arrays][weight table][ring of raw units (bulk only)][output image]
// [mbarriers].  Returns floats.
inline long long finish_layout(Geom &g, long long arrays_floats, int wtab_floats, int raw_tensors, bool use_bulk,
                               int nstage = 1) {
    long long off = pad4((int)arrays_floats);
    g.wtab_off = (int)off;
    off += pad4(wtab_floats);
    g.raw_off = (int)off;
    g.nstage = use_bulk ? nstage : 1;
    g.stage_bytes = raw_tensors * g.NPL * g.plane_bytes;  // a multiple of 16 whenever bulk copies are allowed
    if (use_bulk) off += ((long long)g.nstage * g.stage_bytes + 3) / 4;
    off = pad4((int)off);
    g.out_off = (int)off;
    g.bulk_out = (use_bulk && !g.vec) ? 1 : 0;  // rows that are not 16-byte multiples: assemble the unit on chip
    if (g.bulk_out) off += ((long long)g.NPL * g.plane_bytes + 3) / 4;
    off = pad4((int)off);
    g.bar_off = (int)off;
    return off + 2 * MAX_STAGES;
}

// Deepen the prefetch ring of a finished plan as far as the shared memory left beside its resident blocks
// allows: short units (small planes) finish faster than one DRAM round trip, so one unit of look-ahead
// leaves the block waiting for its copy.
inline void deepen_prefetch(Geom &g) {
    if (!g.bulk) return;
    // the layout up to the ring is kept: [0, wtab_off) arrays, [wtab_off, raw_off) weight table
    const int raw_tensors = g.stage_bytes / (g.NPL * g.plane_bytes);
    for (int ns = 2; ns <= MAX_STAGES; ++ns) {
        if ((long long)(ns - 1) * g.nblocks >= g.units) break;  // deeper than the units a block has
        Geom t = g;
        const long long fl = finish_layout(t, g.wtab_off, g.raw_off - g.wtab_off, raw_tensors, true, ns);
        const long long bytes = fl * 4;
        if (bytes > SMEM_LIMIT || (long long)g.blocks_per_sm * (bytes + 1024) > SMEM_PER_SM) break;
        t.smem_floats = (int)fl;
        g = t;
    }
}

// Slot layout; returns floats per slot.  with_g: second copy of the input pyramid (grad_out); with_z:
// the conv-output arrays.
inline int layout_slot(Geom &g, bool with_g, bool with_z) {
    int off = 0;
    for (int l = 0; l <= g.L; ++l) { g.offA[l] = off; off += (l == 0 ? 1 : 4) * g.rows[l] * g.pitch[l]; }
    for (int l = 0; l <= g.L; ++l) { g.offG[l] = off; if (with_g) off += (l == 0 ? 1 : 4) * g.rows[l] * g.pitch[l]; }
    const int padH = g.ty[0] * g.th, padW = g.tx[0] * 4;  // pixels the base tiles cover
    for (int l = 1; l <= g.L; ++l) {
        // only the coefficients the (padded) base tiles read in the synthesis are kept
        const int zr = ((padH - 1) >> l) + 1;
        const int zc = pad4(((padW - 1) >> l) + 1);
        g.zrows[l] = zr; g.zpitch[l] = zc; g.offZ[l] = off;
        if (with_z) off += 4 * zr * zc;
    }
    return pad4(off);
}

inline double partition_eff(int units, int nblocks) {
    const int per = (units + nblocks - 1) / nblocks;
    return (double)units / ((double)per * nblocks);
}

// Useful conv outputs over tile slots issued, times `short_tiles` for 4-row tiles: below 1 where their per-tile
// overhead counts (forward), above 1 in the fused backward, whose unrolled tile code (weight-gradient taps plus the
// rotated convolution) is half as long with 4-row tiles and measured 3 % faster at equal tile efficiency (28 x 28).
inline double tile_score(const Geom &g, double short_tiles = 0.93) {
    double useful = (double)g.H * g.W, slots = (double)g.nbase * 4 * g.th;
    for (int l = 1; l <= g.L; ++l) {
        useful += 4.0 * g.Hl[l] * g.Wl[l];
        slots += 4.0 * g.tx[l] * g.ty[l] * 4 * g.th;
    }
    return useful / slots * (g.th == 8 ? 1.0 : short_tiles);
}

// Forward plan.  `tune` (0 = automatic): bits 0-4 threads/32, bits 5-7 blocks per SM, bits 8-13 planes per unit.
inline bool plan_forward_th(int B, int C, int H, int W, int L, int elem_bytes, Geom &best, unsigned tune, int th) {
    const int fT = (tune & 31) * 32, fBps = (tune >> 5) & 7, fNpl = (tune >> 8) & 63;
    const bool no_bulk = (tune >> 20) & 1;
    Geom g = {};
    fill_common(g, B, C, H, W, L, elem_bytes, th);
    const int slot = layout_slot(g, false, true);
    const int M = g.lvl_start[L + 1] + g.nbase;
    const double teff = tile_score(g);
    bool found = false;
    for (int npl = 1; npl <= 64; ++npl) {
        if (npl > 1 && npl > C) break;
        if (fNpl && npl != fNpl) continue;
        const int wtab = npl * (1 + 4 * L) * WT_STRIDE;
        const bool can_bulk = (C % npl == 0) && (((long long)npl * g.plane_bytes) % 16 == 0) && !no_bulk;
        for (int use_bulk = can_bulk ? 1 : 0; use_bulk >= 0; --use_bulk) {
        Geom cg = g;
        cg.NPL = npl; cg.slot_stride = slot; cg.bulk = use_bulk;
        const long long smem_floats = finish_layout(cg, (long long)npl * slot, wtab, 1, use_bulk);
        const long long bytes = smem_floats * 4;
        if (bytes > SMEM_LIMIT) continue;
        for (int T = 64; T <= MAX_THREADS; T += 32) {
            if (npl * g.nbase > T) continue;  // at most one base tile per thread
            if (fT && T != fT) continue;
            for (int bps = 1; bps <= 6; ++bps) {
                if (bps * T > 768) continue;  // register file: kernels are built for 128 / 84 registers
                if (fBps && bps != fBps) continue;
                if (bps * (bytes + 1024) > SMEM_PER_SM) continue;
                const int rounds = (npl * M + T - 1) / T;
                const double eff = (double)npl * M / ((double)T * rounds);
                const int ngroups = (C + npl - 1) / npl, units = ngroups * B;
                int nblocks = NUM_SMS * bps;
                if (nblocks > units) nblocks = units;
                // thread-slot use x resident warps (about 16 hide the latency-bound phases) x phase overlap
                double occ = (double)bps * T / 512.0;
                if (occ > 1.0) occ = 1.0;
                const double overlap = bps >= 4 ? 1.0 : (bps == 3 ? 0.95 : (bps == 2 ? 0.8 : 0.55));
                // more than 512 resident threads run the 80-register build, which spills with 8-row tiles and
                // measured slower than four blocks of 128 threads on the smallest planes
                const double regs = bps * T > 512 ? (th == 8 ? 0.75 : (T <= 128 ? 0.9 : 1.0)) : 1.0;
                // small planes are bound by per-unit fixed costs: what counts is how many pixels are resident per SM
                double inflight = (double)bps * npl * H * W / 8192.0;
                inflight = inflight >= 1.0 ? 1.0 : pow(inflight, 0.3);
                const double sc = teff * sqrt(eff) * (0.5 + 0.5 * occ) * overlap * (use_bulk ? 1.0 : 0.8) * (rounds <= 2 ? 1.0 : 0.9) *
                                  partition_eff(units, nblocks) * ((double)C / ((double)ngroups * npl)) *
                                  (1.0 - 1e-4 * T / 32.0) * regs * inflight;
                if (sc > best.score + 1e-9) {
                    best = cg;
                    best.smem_floats = (int)smem_floats; best.ngroups = ngroups; best.units = units;
                    best.nthreads = T; best.nblocks = nblocks; best.blocks_per_sm = bps; best.score = sc;
                    found = true;
                }
            }
        }
        }
    }
    return found;
}

// Weight-gradient plan: per class c with n_c tiles (x NPL) allocate ceil(n_c NPL / rounds) threads, smallest
// `rounds` that fits the thread limit.  tune bits 14-19: planes per unit.
inline bool plan_wgrad_th(int B, int C, int H, int W, int L, int elem_bytes, Geom &best, unsigned tune, int th) {
    const int fNpl = (tune >> 14) & 63, fBps = 0;
    const bool no_bulk = (tune >> 20) & 1;
    Geom g = {};
    fill_common(g, B, C, H, W, L, elem_bytes, th);
    const int slot = layout_slot(g, true, false);
    const int ncls = 1 + 4 * L;
    const double teff = tile_score(g);
    bool found = false;
    for (int npl = 1; npl <= 1; ++npl) {  // one plane per unit: a thread's class must map to one channel
        (void)fNpl;
        for (int rounds = 1; rounds <= 64; ++rounds) {
            int thr[4 * MAXL + 2];
            int tot = 0, work = 0;
            for (int c = 0; c < ncls; ++c) {
                const int l = c == 0 ? 0 : 1 + ((c - 1) >> 2);
                const int n = g.tx[l] * g.ty[l] * npl;
                thr[c] = tot;
                tot += (n + rounds - 1) / rounds;
                work += n;
            }
            thr[ncls] = tot;
            if (tot > MAX_THREADS) continue;
            const int T = (tot + 31) & ~31;
            long long arrays = (long long)npl * slot;
            const long long scratch = (long long)T * (KK + 1);
            if (scratch > arrays) arrays = scratch;
            bool any = false;
            const bool can_bulk = (g.plane_bytes % 16 == 0) && !no_bulk;
            for (int use_bulk = can_bulk ? 1 : 0; use_bulk >= 0; --use_bulk) {
                Geom cg = g;
                cg.NPL = npl; cg.slot_stride = slot; cg.bulk = use_bulk;
                const long long smem_floats = finish_layout(cg, arrays, 0, 2, use_bulk);
                const long long bytes = smem_floats * 4;
                if (bytes > SMEM_LIMIT) continue;
                any = true;
                for (int bps = 1; bps <= 4; ++bps) {
                    if (bps * T > 512) continue;  // 128 registers per thread
                    if (fBps && bps != fBps) continue;
                    if (bps * (bytes + 1024) > SMEM_PER_SM) continue;
                    const int units = C * B;
                    int nblocks = NUM_SMS * bps;
                    if (nblocks > units) nblocks = units;
                    double occ = (double)bps * T / 512.0;
                    if (occ > 1.0) occ = 1.0;
                    const double overlap = bps >= 3 ? 1.0 : (bps == 2 ? 0.85 : 0.55);
                    const double sc = teff * ((double)work / ((double)T * rounds)) * (0.5 + 0.5 * occ) * overlap *
                                      (use_bulk ? 1.0 : 0.8) * partition_eff(units, nblocks);
                    if (sc > best.score + 1e-9) {
                        best = cg;
                        best.smem_floats = (int)smem_floats;
                        best.ngroups = C; best.units = units;
                        best.nthreads = T; best.nblocks = nblocks; best.blocks_per_sm = bps; best.score = sc;
                        for (int k = 0; k <= ncls; ++k) best.thr_start[k] = thr[k];
                        int np = 1;
                        for (int ch = 0; ch < C; ++ch) {
                            const int first = block_of_unit((long long)ch * B, nblocks, units);
                            const int last = block_of_unit((long long)(ch + 1) * B - 1, nblocks, units);
                            if (last - first + 1 > np) np = last - first + 1;
                        }
                        best.np = np;
                        found = true;
                    }
                }
            }
            if (!any) break;
            break;  // more rounds with the same NPL only lowers thread use
        }
    }
    return found;
}

// Fused-backward plan: one round (every tile its own thread), both input pyramids plus Z in shared memory, no
// bulk prefetch unless it fits.  tune bits 14-19: planes per unit (shared with the weight-gradient plan).
inline bool plan_bwd_fused_th(int B, int C, int H, int W, int L, int elem_bytes, Geom &best, unsigned tune, int th) {
    const int fNpl = (tune >> 14) & 63, fBps = 0;
    Geom g = {};
    fill_common(g, B, C, H, W, L, elem_bytes, th);
    const int slot = layout_slot(g, true, true);
    const int M = g.lvl_start[L + 1] + g.nbase;
    const double teff = tile_score(g, 1.03);
    bool found = false;
    for (int npl = 1; npl <= 63; ++npl) {
        if (npl > 1 && npl > C) break;
        if (fNpl && npl != fNpl) continue;
        if (npl * M > 256) break;
        const int wtab = npl * (1 + 4 * L) * WT_STRIDE;
        const int T = (npl * M + 31) & ~31;
        long long arrays = (long long)npl * slot;
        const long long scratch = (long long)T * (KK + 2) + 2LL * npl * (1 + 4 * L);  // flush scratch: sums, tags, run starts and ends
        if (scratch > arrays) arrays = scratch;
        const bool can_bulk = (C % npl == 0) && (((long long)npl * g.plane_bytes) % 16 == 0) && !((tune >> 20) & 1);
        bool any = false;
        // use_bulk = tensors that arrive by bulk copy: both or none (x only, with grad_out read by plain loads,
        // measured slower than no prefetch at 56 x 56 fp32)
        for (int use_bulk = can_bulk ? 2 : 0; use_bulk >= 0; use_bulk -= 2) {
        Geom cg = g;
        cg.NPL = npl; cg.slot_stride = slot; cg.bulk = use_bulk;
        const long long smem_floats = finish_layout(cg, arrays, wtab, use_bulk ? use_bulk : 1, use_bulk > 0);
        const long long bytes = smem_floats * 4;
        if (bytes > SMEM_LIMIT) continue;
        any = true;
        for (int bps = 1; bps <= 4; ++bps) {
            if (bps * T > 512) continue;  // 128 registers per thread
            if (fBps && bps != fBps) continue;
            if (bps * (bytes + 1024) > SMEM_PER_SM) continue;
            const int ngroups = (C + npl - 1) / npl, units = ngroups * B;
            int nblocks = NUM_SMS * bps;
            if (nblocks > units) nblocks = units;
            double occ = (double)bps * T / 512.0;
            if (occ > 1.0) occ = 1.0;
            const double overlap = bps >= 3 ? 1.0 : (bps == 2 ? 0.85 : 0.55);
            const double sc = teff * ((double)npl * M / (double)T) * (0.5 + 0.5 * occ) * overlap *
                              (use_bulk == 2 ? 1.0 : 0.85) *
                              partition_eff(units, nblocks) * ((double)C / ((double)ngroups * npl));
            if (sc > best.score + 1e-9) {
                best = cg;
                best.smem_floats = (int)smem_floats;
                best.ngroups = ngroups; best.units = units;
                best.nthreads = T; best.nblocks = nblocks; best.blocks_per_sm = bps; best.score = sc;
                int np = 1;
                for (int ch = 0; ch < ngroups; ++ch) {
                    const int first = block_of_unit((long long)ch * B, nblocks, units);
                    const int last = block_of_unit((long long)(ch + 1) * B - 1, nblocks, units);
                    if (last - first + 1 > np) np = last - first + 1;
                }
                best.np = np;
                found = true;
            }
        }
        }
        if (!any) break;
    }
    return found;
}

// Each plan is searched for both tile heights; tune bit 22 forces 8 rows, bit 23 forces 4 rows.
inline bool search_forward(int B, int C, int H, int W, int L, int elem_bytes, Geom &best, unsigned tune) {
    best.score = -1.0;
    bool ok = false;
    if (!((tune >> 23) & 1)) ok |= plan_forward_th(B, C, H, W, L, elem_bytes, best, tune, 8);
    if (!((tune >> 22) & 1)) ok |= plan_forward_th(B, C, H, W, L, elem_bytes, best, tune, 4);
    if (ok) deepen_prefetch(best);
    return ok;
}
inline bool search_wgrad(int B, int C, int H, int W, int L, int elem_bytes, Geom &best, unsigned tune) {
    best.score = -1.0;
    bool ok = false;
    if (!((tune >> 23) & 1)) ok |= plan_wgrad_th(B, C, H, W, L, elem_bytes, best, tune, 8);
    if (!((tune >> 22) & 1)) ok |= plan_wgrad_th(B, C, H, W, L, elem_bytes, best, tune, 4);
    if (ok) deepen_prefetch(best);
    return ok;
}
inline bool search_bwd_fused(int B, int C, int H, int W, int L, int elem_bytes, Geom &best, unsigned tune) {
    if ((tune >> 21) & 1) return false;  // bit 21: never fuse
    best.score = -1.0;
    bool ok = false;
    if (!((tune >> 23) & 1)) ok |= plan_bwd_fused_th(B, C, H, W, L, elem_bytes, best, tune, 8);
    if (!((tune >> 22) & 1)) ok |= plan_bwd_fused_th(B, C, H, W, L, elem_bytes, best, tune, 4);
    if (ok) deepen_prefetch(best);
    return ok;
}

// The searches above walk a few thousand candidates (tens of microseconds of host time), more than a small
// layer's kernels take on the GPU, so every entry point looks its plan up in a small process-wide cache first.
struct PlanKey {
    int kind, B, C, H, W, L, elem_bytes;
    unsigned tune;
    bool operator==(const PlanKey &o) const {
        return kind == o.kind && B == o.B && C == o.C && H == o.H && W == o.W && L == o.L && elem_bytes == o.elem_bytes &&
               tune == o.tune;
    }
};
struct PlanEntry {
    PlanKey key;
    bool ok;
    Geom g;
};
inline bool cached_plan(int kind, int B, int C, int H, int W, int L, int elem_bytes, Geom &best, unsigned tune) {
    static std::mutex mu;
    static std::vector<PlanEntry> cache;
    const PlanKey key = {kind, B, C, H, W, L, elem_bytes, tune};
    {
        std::lock_guard<std::mutex> lock(mu);
        for (const PlanEntry &e : cache)
            if (e.key == key) {
                if (e.ok) best = e.g;
                return e.ok;
            }
    }
    PlanEntry e;
    e.key = key;
    e.g = Geom{};
    e.ok = kind == 0   ? search_forward(B, C, H, W, L, elem_bytes, e.g, tune)
           : kind == 1 ? search_wgrad(B, C, H, W, L, elem_bytes, e.g, tune)
                       : search_bwd_fused(B, C, H, W, L, elem_bytes, e.g, tune);
    {
        std::lock_guard<std::mutex> lock(mu);
        if (cache.size() >= 256) cache.clear();  // bounded: a process cycling through more shapes just searches again
        cache.push_back(e);
    }
    if (e.ok) best = e.g;
    return e.ok;
}
inline bool plan_forward(int B, int C, int H, int W, int L, int elem_bytes, Geom &best, unsigned tune = 0) {
    return cached_plan(0, B, C, H, W, L, elem_bytes, best, tune);
}
inline bool plan_wgrad(int B, int C, int H, int W, int L, int elem_bytes, Geom &best, unsigned tune = 0) {
    return cached_plan(1, B, C, H, W, L, elem_bytes, best, tune);
}
inline bool plan_bwd_fused(int B, int C, int H, int W, int L, int elem_bytes, Geom &best, unsigned tune = 0) {
    return cached_plan(2, B, C, H, W, L, elem_bytes, best, tune);
}

inline int dtype_bytes(int dtype) { return dtype == 0 ? 4 : 2; }

// Human-readable launch plan of a descriptor (threads, blocks per SM, planes per unit, tile rows, ring depth).
inline void describe(int B, int C, int H, int W, int L, int elem_bytes, unsigned tune, char *buf, size_t n) {
    Geom f, b;
    int o = 0;
    if (plan_forward(B, C, H, W, L, elem_bytes, f, tune))
        o += snprintf(buf + o, n - o, "plane fwd[T=%d bps=%d npl=%d th=%d ring=%d]", f.nthreads, f.blocks_per_sm, f.NPL, f.th,
                      f.bulk ? f.nstage : 0);
    if (o < (int)n && plan_bwd_fused(B, C, H, W, L, elem_bytes, b, tune))
        snprintf(buf + o, n - o, " bwd[fused T=%d bps=%d npl=%d th=%d ring=%d np=%d]", b.nthreads, b.blocks_per_sm, b.NPL, b.th,
                 b.bulk ? b.nstage : 0, b.np);
    else if (o < (int)n && plan_wgrad(B, C, H, W, L, elem_bytes, b, tune))
        snprintf(buf + o, n - o, " bwd[split wgrad T=%d bps=%d th=%d ring=%d np=%d]", b.nthreads, b.blocks_per_sm, b.th,
                 b.bulk ? b.nstage : 0, b.np);
}

inline bool supported(int H, int W, int k, int L, int dtype) {
    if (k != 5) return false;
    Geom g;
    return plan_forward(2, 2, H, W, L, dtype_bytes(dtype), g) && plan_wgrad(2, 2, H, W, L, dtype_bytes(dtype), g);
}

// Workspace: the status words (256 bytes reserved; see common.cuh), then for backward the base partials
// [C][np][26] and the level partials [L][C][np][4][25] (float).
constexpr size_t STATUS_BYTES = 256;
inline size_t forward_workspace_bytes(int, int, int, int, int) { return STATUS_BYTES; }
inline size_t backward_workspace_bytes(int B, int C, int H, int W, int L, int elem_bytes, unsigned tune = 0) {
    Geom g;
    if (!plan_bwd_fused(B, C, H, W, L, elem_bytes, g, tune) && !plan_wgrad(B, C, H, W, L, elem_bytes, g, tune)) return 0;
    return STATUS_BYTES + sizeof(float) * ((size_t)C * g.np * (KK + 1) + (size_t)L * C * g.np * 4 * KK);
}

// Opt a kernel in to the large dynamic shared-memory carve-out once per device (the attribute is sticky; asking
// for it on every launch costs host time that shows on the small layers).
template <auto Kern>
cudaError_t opt_in_smem() {
    static std::atomic<unsigned long long> done{0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const unsigned long long bit = dev >= 0 && dev < 64 ? 1ull << dev : 0ull;
    if (bit && (done.load(std::memory_order_acquire) & bit)) return cudaSuccess;
    e = cudaFuncSetAttribute(Kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT);
    if (e == cudaSuccess && bit) done.fetch_or(bit, std::memory_order_release);
    return e;
}

template <typename T, bool FLIP>
cudaError_t launch_fwd(const Geom &g, const T *x, const float *w0, const float *s0, const float *b0, const float *wl,
                       const float *sl, T *out, int *status, cudaStream_t st) {
    cudaError_t e;
    const size_t smem = (size_t)g.smem_floats * 4;
#define WT_LAUNCH_FWD_KT(MAXT_, MINB_, TH_, KT_)                                                    \
    {                                                                                               \
        constexpr auto kern = plane_fwd_kernel<T, FLIP, MAXT_, MINB_, TH_, KT_>;                    \
        if ((e = opt_in_smem<kern>()) != cudaSuccess) return e;                                     \
        if ((e = launch_overlapped(kern, (unsigned)g.nblocks, (unsigned)g.nthreads, smem, st, g, x, w0, s0, b0, wl, sl, \
                                   out, status)) != cudaSuccess)                                    \
            return e;                                                                               \
    }
#define WT_LAUNCH_FWD_TH(MAXT_, MINB_, TH_) { if (g.taps == 3) WT_LAUNCH_FWD_KT(MAXT_, MINB_, TH_, 3) else WT_LAUNCH_FWD_KT(MAXT_, MINB_, TH_, 5) }
#define WT_LAUNCH_FWD(MAXT_, MINB_) { if (g.th == 8) WT_LAUNCH_FWD_TH(MAXT_, MINB_, 8) else WT_LAUNCH_FWD_TH(MAXT_, MINB_, 4) }
    if (g.nthreads <= 128 && g.blocks_per_sm <= 3) {
        WT_LAUNCH_FWD(128, 3)
    } else if (g.nthreads * g.blocks_per_sm <= 512) {
        if (g.nthreads <= 128) WT_LAUNCH_FWD(128, 4) else WT_LAUNCH_FWD(256, 2)
    } else {
        if (g.nthreads <= 128) WT_LAUNCH_FWD(128, 6) else WT_LAUNCH_FWD(256, 3)
    }
#undef WT_LAUNCH_FWD
#undef WT_LAUNCH_FWD_TH
#undef WT_LAUNCH_FWD_KT
    return cudaGetLastError();
}

// `tag`: the call's status tag (non-zero, fresh per call).  Nothing is cleared and no other stream operation is
// enqueued besides the kernel, so that the launch can overlap the tail of the kernel before it.
template <typename T>
cudaError_t forward(int B, int C, int H, int W, int L, const T *x, const float *w0, const float *s0, const float *b0,
                    const float *wl, const float *sl, T *out, char *ws, cudaStream_t st, unsigned tag, unsigned tune = 0,
                    bool no_copy = false, int taps = 5) {
    Geom g;
    if (!plan_forward(B, C, H, W, L, (int)sizeof(T), g, tune)) return cudaErrorInvalidValue;
    g.no_copy = no_copy;
    g.tag = tag;
    g.taps = taps;
    return launch_fwd<T, false>(g, x, w0, s0, b0, wl, sl, out, reinterpret_cast<int *>(ws), st);
}

// The epilogue learns from `ep` which partial slots the blocks wrote (EpiloguePtrs::grp), so nothing is cleared here
// either.
template <typename T>
cudaError_t backward(int B, int C, int H, int W, int L, const T *x, const T *go, const float *w0, const float *s0,
                     const float *wl, const float *sl, T *gx, char *ws, EpiloguePtrs *ep, cudaStream_t st, unsigned tag,
                     unsigned tune = 0, bool no_copy = false, int taps = 5) {
    Geom gw, gf;
    cudaError_t e;
    if (plan_bwd_fused(B, C, H, W, L, (int)sizeof(T), gw, tune)) {
        gw.no_copy = no_copy;
        gw.tag = tag;
        gw.taps = taps;
        float *part0 = reinterpret_cast<float *>(ws + STATUS_BYTES);
        float *partl = part0 + (size_t)C * gw.np * (KK + 1);
#define WT_LAUNCH_BWD_KT(TH_, BULK_, KT_)                                                                  \
    {                                                                                                      \
        constexpr auto kb = plane_bwd_kernel<T, TH_, BULK_, KT_>;                                          \
        if ((e = opt_in_smem<kb>()) != cudaSuccess) return e;                                              \
        if ((e = launch_overlapped(kb, (unsigned)gw.nblocks, (unsigned)gw.nthreads, (size_t)gw.smem_floats * 4, st, gw, \
                                   x, go, w0, s0, wl, sl, gx, part0, partl, reinterpret_cast<int *>(ws))) !=  \
            cudaSuccess)                                                                                   \
            return e;                                                                                      \
    }
#define WT_LAUNCH_BWD(TH_, BULK_) { if (taps == 3) WT_LAUNCH_BWD_KT(TH_, BULK_, 3) else WT_LAUNCH_BWD_KT(TH_, BULK_, 5) }
        if (gw.th == 8) {
            if (gw.bulk == 2) WT_LAUNCH_BWD(8, 2) else WT_LAUNCH_BWD(8, 0)
        } else {
            if (gw.bulk == 2) WT_LAUNCH_BWD(4, 2) else WT_LAUNCH_BWD(4, 0)
        }
#undef WT_LAUNCH_BWD
#undef WT_LAUNCH_BWD_KT
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        ep->part0 = part0;
        ep->np0 = gw.np;
        for (int l = 0; l < L; ++l) {
            ep->partl[l] = partl + (size_t)l * C * gw.np * 4 * KK;
            ep->npl[l] = gw.np;
        }
        ep->grp = gw.NPL; ep->B = B; ep->units = gw.units; ep->nblocks = gw.nblocks;
        return cudaSuccess;
    }
    if (!plan_wgrad(B, C, H, W, L, (int)sizeof(T), gw, tune) || !plan_forward(B, C, H, W, L, (int)sizeof(T), gf, tune))
        return cudaErrorInvalidValue;
    gw.no_copy = gf.no_copy = no_copy;
    gw.tag = gf.tag = tag;
    gw.taps = gf.taps = taps;
    int *status = reinterpret_cast<int *>(ws);
    float *part0 = reinterpret_cast<float *>(ws + STATUS_BYTES);
    float *partl = part0 + (size_t)C * gw.np * (KK + 1);
    const size_t smem = (size_t)gw.smem_floats * 4;
#define WT_LAUNCH_WG_KT(MAXT_, MINB_, TH_, KT_)                                                    \
    {                                                                                              \
        constexpr auto kw = plane_wgrad_kernel<T, MAXT_, MINB_, TH_, KT_>;                         \
        if ((e = opt_in_smem<kw>()) != cudaSuccess) return e;                                      \
        if ((e = launch_overlapped(kw, (unsigned)gw.nblocks, (unsigned)gw.nthreads, smem, st, gw, x, go, part0, partl, \
                                   status)) != cudaSuccess)                                        \
            return e;                                                                              \
    }
#define WT_LAUNCH_WG(MAXT_, MINB_, TH_) { if (taps == 3) WT_LAUNCH_WG_KT(MAXT_, MINB_, TH_, 3) else WT_LAUNCH_WG_KT(MAXT_, MINB_, TH_, 5) }
    if (gw.nthreads <= 128) {
        if (gw.th == 8) WT_LAUNCH_WG(128, 4, 8) else WT_LAUNCH_WG(128, 4, 4)
    } else {
        if (gw.th == 8) WT_LAUNCH_WG(256, 2, 8) else WT_LAUNCH_WG(256, 2, 4)
    }
#undef WT_LAUNCH_WG
#undef WT_LAUNCH_WG_KT
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if ((e = launch_fwd<T, true>(gf, go, w0, s0, nullptr, wl, sl, gx, status, st)) != cudaSuccess) return e;
    ep->part0 = part0;
    ep->np0 = gw.np;
    for (int l = 0; l < L; ++l) {
        ep->partl[l] = partl + (size_t)l * C * gw.np * 4 * KK;
        ep->npl[l] = gw.np;
    }
    ep->grp = gw.NPL; ep->B = B; ep->units = gw.units; ep->nblocks = gw.nblocks;
    return cudaSuccess;
}

// Explicit instantiation (EXTERN empty) or its declaration (EXTERN = extern) of the host entry points for one
// activation type: the kernels are compiled once, in the instantiation unit of that type.
#define WT_PLANE_INSTANTIATE(T, EXTERN)                                                                                    \
    EXTERN template cudaError_t forward<T>(int, int, int, int, int, const T *, const float *, const float *, const float *, \
                                           const float *, const float *, T *, char *, cudaStream_t, unsigned, unsigned,    \
                                           bool, int);                                                                     \
    EXTERN template cudaError_t backward<T>(int, int, int, int, int, const T *, const T *, const float *, const float *,    \
                                            const float *, const float *, T *, char *, EpiloguePtrs *, cudaStream_t,       \
                                            unsigned, unsigned, bool, int);

}  // namespace plane
}  // namespace wt
