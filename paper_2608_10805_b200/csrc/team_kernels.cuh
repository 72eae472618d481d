// Team kernels for small planes (7 x 7, 14 x 14 and the like; k = 5): many planes are in flight per SM and the
// threads that work on one group of planes synchronise among themselves only.
//
// Design
//  * A unit is G consecutive channels of one image (contiguous in NCHW: one aligned bulk copy in, one out).  A
//    team of G x T threads (32 to 128) owns a unit at a time; thread t G + q of the team always works on tile t of
//    plane q (neighbouring lanes = the same tile of neighbouring planes: with the plane slots an odd number of
//    16-byte chunks apart their window loads fall into different banks), so its tile geometry, its folded weights (Eq. 8) and - in the backward pass - its 25 weight-gradient
//    accumulators live in registers across all images of a channel group.  Up to 15 teams share a block; they
//    meet only at hardware named barriers of their own (one warp: __syncwarp), never at a block barrier, so
//    while one team stages or stores another one convolves.  One persistent block per SM.
//  * The block walks a contiguous range of units in channel-group-major order.  Inside one channel group (a
//    segment) the teams take the images round robin; the folded weight table of the group is shared.  Block
//    barriers happen at segment boundaries only (weight table, gradient flush).
//  * Per unit: the raw planes arrive through a two-deep ring of bulk copies (bounded waits on mbarriers); 2 x 2
//    pixel blocks are staged into the haloed x array and butterflied (Eq. 5, without the factor 1/2: the powers
//    of two are folded into the weights, which is exact) into the level-1 subbands, deeper levels from the
//    low-pass band on chip (Sec. 4.1); every thread convolves its 4 x TH register tile (in the backward pass it
//    first correlates the tile of D^l with the window of Y^l into its weight-gradient registers, Sec. 2.2, then
//    runs the rotated-kernel convolution); the results overwrite the arrays they came from; then 4 x 4 pixel
//    blocks add the bit-indexed closed-form synthesis of Proposition 2 (Sec. 4.2) to the base convolution and
//    the finished unit leaves with one bulk store.
//  * Weight-gradient partial sums are reduced at the end of a segment in a fixed order (teams, then tiles)
//    through shared memory; one partial per block and channel goes to the workspace and the common epilogue
//    finishes the batch sum in fp64 and applies Eq. 9.
#pragma once
#include "plane_kernels.cuh"

namespace wt {
namespace team {

using plane::FastDiv;
using plane::fdiv;
using plane::make_fastdiv;
using plane::pad4;

constexpr int MAXL = 8;
constexpr int KK = 25;
constexpr int WT_STRIDE = 28;
constexpr int MAX_TEAMS = 15;   // named barriers 1..15 (0 is the block barrier)
constexpr int NSTAGE = 2;       // raw units in flight per team
constexpr int MAX_TEAM_THREADS = 128;

struct TGeom {
    int B, C, H, W, L;
    int Hl[MAXL + 1], Wl[MAXL + 1];
    int tx[MAXL + 1], ty[MAXL + 1];         // 4 x TH tiles per level grid (index 0 = base)
    int rows[MAXL + 1], pitch[MAXL + 1];    // haloed arrays: element (y, x) at (y + 2, x + 2)
    int sub[MAXL + 1];                      // rows * pitch (stride between the four subbands of a level)
    int offA[MAXL + 1], offG[MAXL + 1];     // per plane slot: x / Y^l (A side) and grad_out / D^l (G side, backward only)
    int slot_floats;
    int nbase, ntiles, T, G, team;          // tiles per plane, lanes per plane (>= ntiles), planes per unit, threads per team
    int lvl_start[MAXL + 2];                // first level tile of level l, relative to the first level tile
    FastDiv d_G;
    int HW, plane_bytes, unit_bytes, stage_bytes;
    int team_floats, raw_off, out_off;      // per-team shared-memory region
    int wtab_off, stg_off, bar_off, smem_bytes;
    int nby, nbx, nstg;                     // 2 x 2 staging blocks per plane, staging items per unit
    int nbh, nbx4;                          // synthesis items per plane (two per 4 x 4 pixel block), blocks per block row
    FastDiv d_nbh, d_nbx4;
    FastDiv d_lv[MAXL + 1], d_cl[MAXL + 1]; // deeper-level staging: / (padded coefficients per plane), / (padded columns)
    int vec2;                               // W even: pixel pairs are loaded and stored as one word
    int nteams, nthreads, nblocks, units, ngroups, np;
    int th;
    int no_copy;
    unsigned tag;                           // non-zero tag of the call this launch belongs to (status words)
    double score;
};

// ------------------------------------------------------------------ team synchronisation
__device__ __forceinline__ void team_sync(int tw, int id) {
    if (tw == 1) __syncwarp();
    else asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(tw * 32) : "memory");
}
// barrier + OR of `pred` over the team
__device__ __forceinline__ bool team_sync_or(int tw, int id, bool pred) {
    if (tw == 1) {
        __syncwarp();
        return __any_sync(0xffffffffu, pred);
    }
    unsigned r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\tbar.red.or.pred q, %2, %3, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                 : "=r"(r)
                 : "r"((unsigned)pred), "r"(id), "r"(tw * 32)
                 : "memory");
    return r != 0;
}

// ------------------------------------------------------------------ raw-plane access (shared memory)
__device__ __forceinline__ float px1(const float *p, int i) { return p[i]; }
__device__ __forceinline__ float px1(const __half *p, int i) { return __half2float(p[i]); }
__device__ __forceinline__ float px1(const __nv_bfloat16 *p, int i) { return __bfloat162float(p[i]); }
__device__ __forceinline__ float2 px2(const float *p, int i) { return *reinterpret_cast<const float2 *>(p + i); }
__device__ __forceinline__ float2 px2(const __half *p, int i) { return __half22float2(*reinterpret_cast<const __half2 *>(p + i)); }
__device__ __forceinline__ float2 px2(const __nv_bfloat16 *p, int i) {
    return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(p + i));
}
__device__ __forceinline__ void st2(float *p, float a, float b) { *reinterpret_cast<float2 *>(p) = make_float2(a, b); }
__device__ __forceinline__ void st2(__half *p, float a, float b) { *reinterpret_cast<__half2 *>(p) = __floats2half2_rn(a, b); }
__device__ __forceinline__ void st2(__nv_bfloat16 *p, float a, float b) {
    *reinterpret_cast<__nv_bfloat162 *>(p) = __floats2bfloat162_rn(a, b);
}

// The 2 x 2 pixel block a staging item covers (zero where it leaves the image).  meta bits: 0 column 2j inside,
// 1 column 2j + 1 inside, 2 row 2i inside, 3 row 2i + 1 inside.
template <typename T>
__device__ __forceinline__ void load_block(const T *raw, int src, int W, int m, bool vec2, float &a, float &b, float &c, float &d) {
    a = b = c = d = 0.f;
    if (vec2) {  // W even: both columns are inside together and the pair is aligned to its own size
        if ((m & 5) == 5) { const float2 v = px2(raw, src); a = v.x; b = v.y; }
        if ((m & 9) == 9) { const float2 v = px2(raw, src + W); c = v.x; d = v.y; }
    } else {
        if ((m & 5) == 5) a = px1(raw, src);
        if ((m & 6) == 6) b = px1(raw, src + 1);
        if ((m & 9) == 9) c = px1(raw, src + W);
        if ((m & 10) == 10) d = px1(raw, src + W + 1);
    }
}

// Un-normalised Haar butterfly of Eq. 5 (sums and differences only; the factor 1/2 per level sits in the weights).
__device__ __forceinline__ void butterfly_raw(float a, float b, float c, float d, float &ll, float &lh, float &hl, float &hh) {
    const float s0 = a + b, s1 = c + d, d0 = a - b, d1 = c - d;
    ll = s0 + s1;
    lh = s0 - s1;
    hl = d0 + d1;
    hh = d0 - d1;
}

// Folded weight table of channel group c0: [plane q][class][WT_STRIDE]; level-l weights carry s^l and 4^-l (the
// analysis and the synthesis are evaluated without their factors 2^-l), the base class carries s^0; the folded
// bias sits at [q][0][25].  flip: rotated by 180 degrees (backward).
__device__ __forceinline__ void build_table(float *wtab, const TGeom &g, int c0, bool flip, const float *__restrict__ w0,
                                            const float *__restrict__ s0, const float *__restrict__ b0,
                                            const float *__restrict__ wl, const float *__restrict__ sl) {
    const int ncls = 1 + 4 * g.L, n = g.G * ncls * KK;
    for (int e = threadIdx.x; e < n; e += blockDim.x) {
        const int sc = e / KK, t = e - sc * KK, q = sc / ncls, cls = sc - q * ncls;
        const int c = c0 + q, src = flip ? (KK - 1 - t) : t;
        float v;
        if (cls == 0) {
            v = __ldg(w0 + c * KK + src) * __ldg(s0 + c);
        } else {
            const int l = (cls - 1) >> 2, sb = (cls - 1) & 3;
            const size_t i = ((size_t)l * g.C + c) * 4 + sb;
            v = __ldg(wl + i * KK + src) * __ldg(sl + i) * __uint_as_float((unsigned)(127 - 2 * (l + 1)) << 23);  // 4^-(level)
        }
        wtab[sc * WT_STRIDE + t] = v;
    }
    for (int q = threadIdx.x; q < g.G; q += blockDim.x)
        wtab[q * ncls * WT_STRIDE + KK] = b0 ? __ldg(s0 + c0 + q) * __ldg(b0 + c0 + q) : 0.f;
}

// Level l >= 2 of one side (A or G) of all planes of the unit, from the low-pass band of level l - 1.
__device__ __forceinline__ void stage_deeper(float *A, const TGeom &g, const int *off, int l, int lt, int team) {
    const int cl = (int)g.d_cl[l].d, n = (int)g.d_lv[l].d;
    const int Hp = g.Hl[l - 1], Wp = g.Wl[l - 1], pp = g.pitch[l - 1], pl = g.pitch[l], sl = g.sub[l];
    for (int e = lt; e < g.G * n; e += team) {
        const int q = fdiv(e, g.d_lv[l]), r = e - q * n, i = fdiv(r, g.d_cl[l]), j = r - i * cl;
        const float *s = A + q * g.slot_floats + off[l - 1] + (2 * i + 2) * pp + 2 * j + 2;
        const bool y0 = 2 * i < Hp, y1 = 2 * i + 1 < Hp, x0 = 2 * j < Wp, x1 = 2 * j + 1 < Wp;
        const float a = (y0 && x0) ? s[0] : 0.f, b = (y0 && x1) ? s[1] : 0.f;
        const float c = (y1 && x0) ? s[pp] : 0.f, d = (y1 && x1) ? s[pp + 1] : 0.f;
        float ll, lh, hl, hh;
        butterfly_raw(a, b, c, d, ll, lh, hl, hh);
        float *y = A + q * g.slot_floats + off[l] + (i + 2) * pl + j + 2;
        y[0] = ll;
        y[sl] = lh;
        y[2 * sl] = hl;
        y[3 * sl] = hh;
    }
}

// Proposition 2 on two pixel rows (rows 2h, 2h + 1) of one 4 x 4 pixel block (block row t4, block column t4x of the
// plane): a[][] = base result + bias + every level's term.  S = the plane slot, off = the side the convolution
// results were written to (in place: element (i, j) of subband s of level l at off[l] + s sub[l] + (i + 2) pitch[l]
// + j + 2; the base result at off[0]).  The weights already carry 4^-l, so the terms are pure sums and differences.
// All loads are issued before the first addition.
__device__ __forceinline__ void synth_half(const float *S, const TGeom &g, const int *off, int t4, int t4x, int h, float bias,
                                           float (*a)[4]) {
    const int L = g.L, p0 = g.pitch[0];
    const float *sb0 = S + off[0] + (4 * t4 + 2 * h + 2) * p0 + 4 * t4x + 2;
    // rows beyond the image may lie outside the array: they are never stored, read the block's first row instead
    const int r1 = (4 * t4 + 2 * h + 1 < g.H) ? p0 : 0;
    const float2 b00 = *reinterpret_cast<const float2 *>(sb0), b01 = *reinterpret_cast<const float2 *>(sb0 + 2);
    const float2 b10 = *reinterpret_cast<const float2 *>(sb0 + r1), b11 = *reinterpret_cast<const float2 *>(sb0 + r1 + 2);
    float2 ll = make_float2(0.f, 0.f), lh = ll, hl = ll, hh = ll;
    if (L >= 1) {
        const int p1 = g.pitch[1], s1 = g.sub[1];
        const float *z = S + off[1] + (2 * t4 + h + 2) * p1 + 2 * t4x + 2;
        ll = *reinterpret_cast<const float2 *>(z);
        lh = *reinterpret_cast<const float2 *>(z + s1);
        hl = *reinterpret_cast<const float2 *>(z + 2 * s1);
        hh = *reinterpret_cast<const float2 *>(z + 3 * s1);
    }
    float z2[4] = {0.f, 0.f, 0.f, 0.f};
    if (L >= 2) {
        const int p2 = g.pitch[2], s2 = g.sub[2];
        const float *z = S + off[2] + (t4 + 2) * p2 + t4x + 2;
        z2[0] = z[0]; z2[1] = z[s2]; z2[2] = z[2 * s2]; z2[3] = z[3 * s2];
    }
    float deep = bias;
    for (int l = 3; l <= L; ++l) {  // the whole block sits in one quadrant of the coefficient's 2^l x 2^l block
        const int pl = g.pitch[l], sl = g.sub[l];
        const float *z = S + off[l] + ((t4 >> (l - 2)) + 2) * pl + (t4x >> (l - 2)) + 2;
        const bool by = (t4 >> (l - 3)) & 1, bx = (t4x >> (l - 3)) & 1;
        const float p = by ? z[0] - z[sl] : z[0] + z[sl];
        const float q = by ? z[2 * sl] - z[3 * sl] : z[2 * sl] + z[3 * sl];
        deep += bx ? p - q : p + q;
    }
    // level 2: the two rows share the row sign (h), the column sign changes between columns 1 and 2
    const float p2v = h ? z2[0] - z2[1] : z2[0] + z2[1], q2v = h ? z2[2] - z2[3] : z2[2] + z2[3];
    const float t2l = deep + (p2v + q2v), t2r = deep + (p2v - q2v);
    a[0][0] = b00.x + t2l; a[0][1] = b00.y + t2l; a[0][2] = b01.x + t2r; a[0][3] = b01.y + t2r;
    a[1][0] = b10.x + t2l; a[1][1] = b10.y + t2l; a[1][2] = b11.x + t2r; a[1][3] = b11.y + t2r;
    // level 1: coefficient row 2 t4 + h, columns 2 t4x + {0, 1}; pixel row r carries the row sign, pixel column parity the column sign
#pragma unroll
    for (int cj = 0; cj < 2; ++cj) {
        const float LLv = cj ? ll.y : ll.x, LHv = cj ? lh.y : lh.x, HLv = cj ? hl.y : hl.x, HHv = cj ? hh.y : hh.x;
        const float pp = LLv + LHv, pm = LLv - LHv, qp = HLv + HHv, qm = HLv - HHv;
        a[0][2 * cj] += pp + qp;
        a[0][2 * cj + 1] += pp - qp;
        a[1][2 * cj] += pm + qm;
        a[1][2 * cj + 1] += pm - qm;
    }
}

// BWD = false: out = WTConv(x) (go unused).  BWD = true: out = grad_x, and the weight-gradient partial sums of every
// channel the block touched go to part0 / partl (slot = block index relative to the channel group's first block).
template <typename T, int TH, bool BWD>
__global__ void __launch_bounds__(BWD ? (TH == 7 ? 384 : 512) : 640, 1)
team_kernel(const __grid_constant__ TGeom g, const T *__restrict__ x, const T *__restrict__ go,
            const float *__restrict__ w0, const float *__restrict__ s0, const float *__restrict__ b0,
            const float *__restrict__ wl, const float *__restrict__ sl, T *__restrict__ out, float *__restrict__ part0,
            float *__restrict__ partl, int *__restrict__ status) {
    extern __shared__ __align__(16) float sm[];
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int TEAM = g.team, tw = TEAM >> 5;
    const int team_id = tid / TEAM, lt = tid - team_id * TEAM, nteams = g.nteams;
    float *A = sm + team_id * g.team_floats;
    char *raw = reinterpret_cast<char *>(A + g.raw_off);
    T *outst = reinterpret_cast<T *>(A + g.out_off);
    unsigned long long *bar = reinterpret_cast<unsigned long long *>(sm + g.bar_off) + team_id * NSTAGE;
    float *wtab = sm + g.wtab_off;
    int4 *stg = reinterpret_cast<int4 *>(sm + g.stg_off);
    const int bar_id = 1 + team_id;
    const int L = g.L, ncls = 1 + 4 * L;
    const unsigned wait_limit = g.no_copy ? plane::WAIT_LIMIT_TEST : plane::WAIT_LIMIT;
    const int *offS = BWD ? g.offG : g.offA;  // the side whose arrays receive the convolution results

    // ---- this thread's tile: plane q of the unit, tile t of the plane (fixed for the whole launch)
    const int t = fdiv(lt, g.d_G), q = lt - t * g.G;
    const bool has_tile = t < g.ntiles;
    int lvl = 0, sb = 0, tyy = 0, txx = 0;
    if (has_tile) {
        if (t < g.nbase) {
            tyy = t / g.tx[0];
            txx = t - tyy * g.tx[0];
        } else {
            int r = t - g.nbase;
            lvl = 1;
            while (lvl < L && r >= g.lvl_start[lvl + 1]) ++lvl;
            r -= g.lvl_start[lvl];
            const int nt = g.tx[lvl] * g.ty[lvl];
            sb = r / nt;
            r -= sb * nt;
            tyy = r / g.tx[lvl];
            txx = r - tyy * g.tx[lvl];
        }
    }
    const int pitch = g.pitch[lvl];
    const int win = q * g.slot_floats + g.offA[lvl] + sb * g.sub[lvl] + TH * tyy * pitch + 4 * txx;  // window top-left, A side
    const int dG = BWD ? g.offG[lvl] - g.offA[lvl] : 0;
    const int cls = lvl == 0 ? 0 : 1 + 4 * (lvl - 1) + sb;
    const int dG0 = g.offG[0] - g.offA[0], dG1 = L >= 1 ? g.offG[1] - g.offA[1] : 0;

    // ---- block set-up: zero the arrays (halos stay zero for the whole launch), staging table, barriers
    {
        float4 *v = reinterpret_cast<float4 *>(sm);
        for (int i = tid; i < nteams * g.team_floats / 4; i += nthr) v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        const int nblk = g.nby * g.nbx, p0 = g.pitch[0], p1 = L >= 1 ? g.pitch[1] : 0;
        for (int e = tid; e < g.nstg; e += nthr) {
            const int qq = e / nblk, r = e - qq * nblk, i = r / g.nbx, j = r - i * g.nbx;
            int m = 0;
            if (2 * j < g.W) m |= 1;
            if (2 * j + 1 < g.W) m |= 2;
            if (2 * i < g.H) m |= 4;
            if (2 * i + 1 < g.H) m |= 8;
            if (L >= 1 && i < g.ty[1] * TH && j < g.tx[1] * 4) m |= 16;   // the coefficient lies in the level-1 tile area
            if (2 * i < g.ty[0] * TH && 2 * j < g.tx[0] * 4) m |= 32;     // the pixels lie in the base tile area
            int4 d;
            d.x = qq * g.HW + 2 * i * g.W + 2 * j;
            d.y = qq * g.slot_floats + g.offA[0] + (2 * i + 2) * p0 + 2 * j + 2;
            d.z = L >= 1 ? qq * g.slot_floats + g.offA[1] + (i + 2) * p1 + j + 2 : 0;
            d.w = m;
            stg[e] = d;
        }
        if (lt == 0)
            for (int s = 0; s < NSTAGE; ++s) plane::mbar_init(bar + s, 1);
        plane::fence_async_smem();  // the zero fill (generic proxy) is ordered before the first bulk copies into the ring
    }
    __syncthreads();
    // The set-up above touched shared memory and registers only and may have run beside the tail of the kernel
    // before this one; global memory is used from here on.
    if (!BWD) dependents_may_start();  // backward: at the end (the kernel behind it is the small epilogue, see plane_bwd_kernel)
    wait_for_predecessor();
    if (blockIdx.x == 0 && tid == 0) status[STATUS_LAUNCH] = (int)g.tag;

    const int u_begin = (int)((long long)blockIdx.x * g.units / gridDim.x);
    const int u_end = (int)((long long)(blockIdx.x + 1) * g.units / gridDim.x);
    const size_t unit_elems = (size_t)g.G * g.HW;
    unsigned it = 0;  // units this team has started: ring entry it & 1, phase (it >> 1) & 1
    bool dead = false;
    float w[KK], accw[KK], gsum = 0.f;
#pragma unroll
    for (int k = 0; k < KK; ++k) w[k] = accw[k] = 0.f;

    auto issue = [&](int u, int cgu, unsigned slot_it) {  // one thread: bulk copies of unit u (channel group cgu) into ring entry slot_it & 1
        if (g.no_copy) return;
        const int bu = u - cgu * g.B;
        const size_t po = ((size_t)bu * g.C + (size_t)cgu * g.G) * g.HW;
        unsigned long long *bq = bar + (slot_it & 1);
        char *dst = raw + (slot_it & 1) * g.stage_bytes;
        plane::mbar_expect_tx(bq, (unsigned)g.unit_bytes * (BWD ? 2u : 1u));
        plane::bulk_g2s(dst, x + po, (unsigned)g.unit_bytes, bq);
        if (BWD) plane::bulk_g2s(dst + g.unit_bytes, go + po, (unsigned)g.unit_bytes, bq);
    };

    for (int seg = u_begin; seg < u_end;) {
        const int cg = seg / g.B, c0 = cg * g.G;
        int seg_end = (cg + 1) * g.B;
        if (seg_end > u_end) seg_end = u_end;
        if (lt == 0 && !dead)
            for (int s = 0; s < NSTAGE; ++s)
                if (seg + team_id + s * nteams < seg_end) issue(seg + team_id + s * nteams, cg, it + s);
        build_table(wtab, g, c0, BWD, w0, s0, BWD ? nullptr : b0, wl, sl);
        __syncthreads();
        if (has_tile) plane::load_weights(wtab + (q * ncls + cls) * WT_STRIDE, w);

        for (int u = seg + team_id; u < seg_end && !dead; u += nteams, ++it) {
            const int b = u - cg * g.B;
            const unsigned st = it & 1u;
            const bool late = !plane::mbar_wait(bar + st, (it >> 1) & 1u, wait_limit);
            const T *rx = reinterpret_cast<const T *>(raw + st * g.stage_bytes);
            const T *rg = rx + unit_elems;
            // ---- staging: x (and grad_out) into the haloed arrays, level-1 subbands by the butterfly of Eq. 5.  Four
            //      items per thread and pass, all loads issued before the first butterfly, so that the shared-memory
            //      round trips of the items overlap instead of queueing behind one another
            for (int e0 = lt; e0 < g.nstg; e0 += 4 * TEAM) {
                int4 d[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) d[k] = e0 + k * TEAM < g.nstg ? stg[e0 + k * TEAM] : make_int4(0, 0, 0, 0);
                float xa[4][4], ga[4][4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    load_block<T>(rx, d[k].x, g.W, d[k].w, g.vec2 != 0, xa[k][0], xa[k][1], xa[k][2], xa[k][3]);
                    if (BWD) load_block<T>(rg, d[k].x, g.W, d[k].w, g.vec2 != 0, ga[k][0], ga[k][1], ga[k][2], ga[k][3]);
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    float ll, lh, hl, hh;
                    if (d[k].w & 32) {
                        *reinterpret_cast<float2 *>(A + d[k].y) = make_float2(xa[k][0], xa[k][1]);
                        *reinterpret_cast<float2 *>(A + d[k].y + g.pitch[0]) = make_float2(xa[k][2], xa[k][3]);
                        if (BWD) {
                            *reinterpret_cast<float2 *>(A + d[k].y + dG0) = make_float2(ga[k][0], ga[k][1]);
                            *reinterpret_cast<float2 *>(A + d[k].y + dG0 + g.pitch[0]) = make_float2(ga[k][2], ga[k][3]);
                        }
                    }
                    if (d[k].w & 16) {
                        butterfly_raw(xa[k][0], xa[k][1], xa[k][2], xa[k][3], ll, lh, hl, hh);
                        float *y = A + d[k].z;
                        y[0] = ll; y[g.sub[1]] = lh; y[2 * g.sub[1]] = hl; y[3 * g.sub[1]] = hh;
                        if (BWD) {
                            butterfly_raw(ga[k][0], ga[k][1], ga[k][2], ga[k][3], ll, lh, hl, hh);
                            y += dG1;
                            y[0] = ll; y[g.sub[1]] = lh; y[2 * g.sub[1]] = hl; y[3 * g.sub[1]] = hh;
                        }
                    }
                }
            }
            if (team_sync_or(tw, bar_id, late)) {  // a copy never landed: record it and stop working (see the end of the kernel)
                dead = true;
                if (lt == 0) atomicExch(status + STATUS_TIMEOUT, (int)g.tag);
                break;
            }
            if (lt == 0 && u + NSTAGE * nteams < seg_end) {  // the ring entry is free again: fetch the unit two rounds ahead
                plane::fence_async_smem();
                issue(u + NSTAGE * nteams, cg, it);
            }
            for (int l = 2; l <= L; ++l) {
                stage_deeper(A, g, g.offA, l, lt, TEAM);
                if (BWD) stage_deeper(A, g, g.offG, l, lt, TEAM);
                team_sync(tw, bar_id);
            }
            // ---- every thread's tile
            float acc[TH][4];
            if (has_tile) {
                const float *asrc = A + win;
                if (BWD) {
                    const float *gsrc = asrc + dG;
                    float d[TH][4];
#pragma unroll
                    for (int rr = 0; rr < TH; ++rr) {
                        const float2 q0 = *reinterpret_cast<const float2 *>(gsrc + (rr + 2) * pitch + 2);
                        const float2 q1 = *reinterpret_cast<const float2 *>(gsrc + (rr + 2) * pitch + 4);
                        d[rr][0] = q0.x; d[rr][1] = q0.y; d[rr][2] = q1.x; d[rr][3] = q1.y;
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
                    plane::conv_tile<TH>(gsrc, pitch, w, acc);
                } else {
                    plane::conv_tile<TH>(asrc, pitch, w, acc);
                }
            }
            team_sync(tw, bar_id);  // every window has been read: the results may overwrite the arrays
            if (has_tile) {
                float *z = A + win + dG + 2 * pitch + 2;
#pragma unroll
                for (int r = 0; r < TH; ++r) {
                    *reinterpret_cast<float2 *>(z + r * pitch) = make_float2(acc[r][0], acc[r][1]);
                    *reinterpret_cast<float2 *>(z + r * pitch + 2) = make_float2(acc[r][2], acc[r][3]);
                }
            }
            if (lt == 0) plane::bulk_store_wait_read();  // the previous unit's store has drained the output image
            team_sync(tw, bar_id);
            // ---- Proposition 2 + base result, two pixel rows of a 4 x 4 block per item, into the unit's output image
            for (int e = lt; e < g.G * g.nbh; e += TEAM) {
                const int qq = fdiv(e, g.d_nbh), r = e - qq * g.nbh, h = r & 1, blk = r >> 1;
                const int t4 = fdiv(blk, g.d_nbx4), t4x = blk - t4 * g.nbx4;
                const float *S = A + qq * g.slot_floats;
                const float bq = BWD ? 0.f : wtab[qq * ncls * WT_STRIDE + KK];
                float a[2][4];
                synth_half(S, g, offS, t4, t4x, h, bq, a);
                const int y0 = 4 * t4 + 2 * h;
                T *o = outst + qq * g.HW + y0 * g.W + 4 * t4x;
#pragma unroll
                for (int r2 = 0; r2 < 2; ++r2) {
                    if (y0 + r2 < g.H) {
                        if (g.vec2) {
                            if (4 * t4x < g.W) st2(o + r2 * g.W, a[r2][0], a[r2][1]);
                            if (4 * t4x + 2 < g.W) st2(o + r2 * g.W + 2, a[r2][2], a[r2][3]);
                        } else {
#pragma unroll
                            for (int cc = 0; cc < 4; ++cc)
                                if (4 * t4x + cc < g.W) stf(o + r2 * g.W + cc, a[r2][cc]);
                        }
                    }
                }
            }
            plane::fence_async_smem();  // every writer orders its shared-memory writes before the async proxy's reads
            team_sync(tw, bar_id);
            if (lt == 0) plane::bulk_s2g(out + ((size_t)b * g.C + c0) * g.HW, outst, (unsigned)g.unit_bytes);
            // The next unit's staging rewrites every array position a tile or the synthesis touched; the barrier above
            // separates it from this unit's last reads.
        }

        if (BWD) {
            // ---- flush the channel group's weight-gradient sums: park every thread's 26 sums in the (idle) array area,
            //      then one thread per (plane, class, tap) adds teams and tiles in a fixed order
            if (lt == 0) plane::bulk_store_wait_read();
            __syncthreads();
            float *scr = sm;
#pragma unroll
            for (int k = 0; k < KK; ++k) scr[tid * (KK + 1) + k] = accw[k];
            scr[tid * (KK + 1) + KK] = gsum;
            __syncthreads();
            const int slotp = blockIdx.x - plane::block_of_unit((long long)cg * g.B, gridDim.x, g.units);
            for (int e = tid; e < g.G * ncls * (KK + 1); e += nthr) {
                const int qc = e / (KK + 1), k = e - qc * (KK + 1), qq = qc / ncls, c2 = qc - qq * ncls;
                if (c2 > 0 && k == KK) continue;
                int t0 = 0, t1 = g.nbase, lv = 0;
                if (c2 > 0) {
                    lv = 1 + ((c2 - 1) >> 2);
                    const int nt = g.tx[lv] * g.ty[lv];
                    t0 = g.nbase + g.lvl_start[lv] + ((c2 - 1) & 3) * nt;
                    t1 = t0 + nt;
                }
                float s = 0.f;
                for (int tm = 0; tm < nteams; ++tm)
                    for (int tt = t0; tt < t1; ++tt) s += scr[(tm * TEAM + tt * g.G + qq) * (KK + 1) + k];
                const int ch = c0 + qq;
                if (c2 == 0) {
                    part0[((size_t)ch * g.np + slotp) * (KK + 1) + k] = s;
                } else {
                    s *= __uint_as_float((unsigned)(127 - 2 * lv) << 23);  // both factors were staged without their 2^-l
                    partl[(size_t)(lv - 1) * g.C * g.np * 4 * KK + (((size_t)ch * g.np + slotp) * 4 + ((c2 - 1) & 3)) * KK + k] = s;
                }
            }
            __syncthreads();
            float4 *v = reinterpret_cast<float4 *>(sm);
            for (int i = tid; i < nteams * g.team_floats / 4; i += nthr) v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int k = 0; k < KK; ++k) accw[k] = 0.f;
            gsum = 0.f;
            plane::fence_async_smem();  // scratch and zero fill touched the ring: order them before the next bulk copies
            __syncthreads();
        }
        seg = seg_end;
    }
    if (BWD) dependents_may_start();
    if (lt == 0) plane::bulk_store_wait_read();  // shared memory must outlive the last bulk store's reads
    if (dead) {
        // a wait ran out: wait once more, with the limit, for whatever may still be on its way into the ring, so that
        // no copy lands in shared memory the block has given back
        for (unsigned s = 0; s < NSTAGE; ++s) plane::mbar_wait(bar + ((it + s) & 1u), ((it + s) >> 1) & 1u, wait_limit);
    }
}

// ------------------------------------------------------------------ host-side planning
inline bool plan_th(int B, int C, int H, int W, int L, int eb, bool bwd, int TH, int forceG, TGeom &best) {
    TGeom g = {};
    g.B = B; g.C = C; g.H = H; g.W = W; g.L = L; g.th = TH;
    g.Hl[0] = H; g.Wl[0] = W;
    for (int l = 1; l <= MAXL; ++l) { g.Hl[l] = (g.Hl[l - 1] + 1) / 2; g.Wl[l] = (g.Wl[l - 1] + 1) / 2; }
    double useful = (double)H * W;
    for (int l = 0; l <= L; ++l) {
        g.tx[l] = pad4(g.Wl[l]) / 4;
        g.ty[l] = (g.Hl[l] + TH - 1) / TH;
        g.rows[l] = g.ty[l] * TH + 4;
        g.pitch[l] = g.tx[l] * 4 + 4;
        if (l) useful += 4.0 * g.Hl[l] * g.Wl[l];
    }
    g.nbase = g.tx[0] * g.ty[0];
    g.lvl_start[0] = g.lvl_start[1] = 0;
    for (int l = 1; l <= L; ++l) g.lvl_start[l + 1] = g.lvl_start[l] + 4 * g.tx[l] * g.ty[l];
    g.ntiles = g.nbase + g.lvl_start[L + 1];
    if (g.ntiles > 64) return false;
    // Array layout of one plane slot.  With fewer than 8 planes per unit a quarter-warp holds several tiles of one
    // plane, and the subbands are put 2 chunks (mod 8) apart so that neighbouring subband tiles hit different banks;
    // with 8 or more it holds the same tile of 8 planes and only the slot stride matters (no padding: more teams fit).
    auto layout = [&](TGeom &t, bool pad_subbands) {
        for (int l = 0; l <= L; ++l) {
            t.sub[l] = t.rows[l] * t.pitch[l];
            while (pad_subbands && (t.sub[l] / 4) % 8 != 2) t.sub[l] += 4;
        }
        int off = 0;
        for (int l = 0; l <= L; ++l) { t.offA[l] = off; off += (l ? 4 : 1) * t.sub[l]; }
        for (int l = 0; l <= L; ++l) { t.offG[l] = off; if (bwd) off += (l ? 4 : 1) * t.sub[l]; }
        return pad4(off);
    };
    g.HW = H * W;
    g.plane_bytes = H * W * eb;
    g.vec2 = (W % 2 == 0) ? 1 : 0;
    // staging blocks cover the base tile area and the level-1 tile area
    int hs = g.ty[0] * TH, ws = g.tx[0] * 4;
    if (L >= 1) { hs = hs > 2 * g.ty[1] * TH ? hs : 2 * g.ty[1] * TH; ws = ws > 2 * g.tx[1] * 4 ? ws : 2 * g.tx[1] * 4; }
    g.nby = (hs + 1) / 2; g.nbx = (ws + 1) / 2;
    g.nbx4 = (W + 3) / 4; g.nbh = 2 * ((H + 3) / 4) * g.nbx4;
    g.d_nbh = make_fastdiv(g.nbh); g.d_nbx4 = make_fastdiv(g.nbx4);
    for (int l = 2; l <= L; ++l) { g.d_lv[l] = make_fastdiv(g.ty[l] * TH * g.tx[l] * 4); g.d_cl[l] = make_fastdiv(g.tx[l] * 4); }
    const int ncls = 1 + 4 * L;
    const int max_threads = bwd ? (TH == 7 ? 384 : 512) : 640;
    bool found = false;
    for (int G = 1; G <= 16; ++G) {
        if (C % G || ((long long)G * g.plane_bytes) % 16) continue;
        if (forceG && G != forceG) continue;
        // lanes per plane: the smallest T >= ntiles that makes the team a whole number of warps
        int T = g.ntiles;
        while ((G * T) % 32) ++T;
        const int team = G * T;
        if (team > MAX_TEAM_THREADS) continue;
        TGeom c = g;
        c.G = G; c.T = T; c.team = team; c.d_G = make_fastdiv(G);
        // plane slots 8 / min(G, 8) chunks (mod 8) apart: a quarter-warp = the same tiles of min(G, 8) planes, bank-conflict free
        c.slot_floats = layout(c, G < 8);
        const int want = G >= 8 ? 1 : 8 / G;
        while (G > 1 && (c.slot_floats / 4) % 8 != want % 8) c.slot_floats += 4;
        c.unit_bytes = G * g.plane_bytes;
        c.stage_bytes = c.unit_bytes * (bwd ? 2 : 1);
        c.nstg = G * g.nby * g.nbx;
        int tf = pad4(G * c.slot_floats);
        c.raw_off = tf; tf += pad4((NSTAGE * c.stage_bytes + 3) / 4);
        c.out_off = tf; tf += pad4((c.unit_bytes + 3) / 4);
        c.team_floats = tf;
        const int block_floats = pad4(G * ncls * WT_STRIDE) + 4 * c.nstg + 2 * NSTAGE * MAX_TEAMS + 8;
        int nteams = (plane::SMEM_LIMIT / 4 - block_floats) / tf;
        if (nteams > MAX_TEAMS) nteams = MAX_TEAMS;
        if (nteams * team > max_threads) nteams = max_threads / team;
        const int units = (C / G) * B;
        int nblocks = plane::NUM_SMS < units ? plane::NUM_SMS : units;
        const int per_block = (units + nblocks - 1) / nblocks;
        if (nteams > per_block) nteams = per_block;
        if (nteams < 1) continue;
        if (bwd && (long long)nteams * team * (KK + 1) > (long long)nteams * tf) continue;  // flush scratch must fit the array area
        c.nteams = nteams; c.nthreads = nteams * team; c.nblocks = nblocks; c.units = units; c.ngroups = C / G;
        c.wtab_off = nteams * tf;
        c.stg_off = c.wtab_off + pad4(G * ncls * WT_STRIDE);
        c.bar_off = c.stg_off + 4 * c.nstg;
        c.smem_bytes = (c.bar_off + 2 * NSTAGE * nteams + 8) * 4;
        if (c.smem_bytes > plane::SMEM_LIMIT) continue;
        int np = 1;
        for (int ch = 0; ch < c.ngroups; ++ch) {
            const int first = plane::block_of_unit((long long)ch * B, nblocks, units);
            const int last = plane::block_of_unit((long long)(ch + 1) * B - 1, nblocks, units);
            if (last - first + 1 > np) np = last - first + 1;
        }
        c.np = np;
        // lanes that carry useful outputs x resident warps (about 12 hide the staging and synthesis phases) x how evenly
        // the teams of a block share its units
        const double lanes = useful / ((double)T * TH * 4);
        double occ = (double)c.nthreads / 384.0;
        if (occ > 1.0) occ = 1.0;
        const int rounds = (per_block + nteams - 1) / nteams;
        const double balance = (double)per_block / ((double)rounds * nteams);
        c.score = lanes * (0.4 + 0.6 * occ) * balance;
        if (c.score > best.score + 1e-9) { best = c; found = true; }
    }
    return found;
}

struct TeamKey {
    int B, C, H, W, L, eb, bwd, forceG;
    bool operator==(const TeamKey &o) const {
        return B == o.B && C == o.C && H == o.H && W == o.W && L == o.L && eb == o.eb && bwd == o.bwd && forceG == o.forceG;
    }
};
struct TeamEntry {
    TeamKey key;
    bool ok;
    TGeom g;
};
// forceG (0 = automatic): planes per unit, for tuning experiments.
inline bool plan(int B, int C, int H, int W, int L, int eb, bool bwd, TGeom &out, int forceG = 0) {
    static std::mutex mu;
    static std::vector<TeamEntry> cache;
    const TeamKey key = {B, C, H, W, L, eb, bwd ? 1 : 0, forceG};
    {
        std::lock_guard<std::mutex> lock(mu);
        for (const TeamEntry &e : cache)
            if (e.key == key) {
                if (e.ok) out = e.g;
                return e.ok;
            }
    }
    TeamEntry e;
    e.key = key;
    e.g = TGeom{};
    e.g.score = -1.0;
    e.ok = false;
    // tiny planes only (7 x 7 and the like): from 14 x 14 on the block-per-plane kernels measured as fast or faster
    if (H * W <= 100 && H <= 16 && W <= 16) {
        e.ok |= plan_th(B, C, H, W, L, eb, bwd, 7, forceG, e.g);
        e.ok |= plan_th(B, C, H, W, L, eb, bwd, 4, forceG, e.g);
    }
    {
        std::lock_guard<std::mutex> lock(mu);
        if (cache.size() >= 256) cache.clear();
        cache.push_back(e);
    }
    if (e.ok) out = e.g;
    return e.ok;
}

inline bool supported(int B, int C, int H, int W, int k, int L, int dtype, int forceG = 0) {
    if (k != 5) return false;
    TGeom g;
    const int eb = plane::dtype_bytes(dtype);
    return plan(B, C, H, W, L, eb, false, g, forceG) && plan(B, C, H, W, L, eb, true, g, forceG);
}

inline size_t backward_workspace_bytes(int B, int C, int H, int W, int L, int eb, int forceG = 0) {
    TGeom g;
    if (!plan(B, C, H, W, L, eb, true, g, forceG)) return 0;
    return plane::STATUS_BYTES + sizeof(float) * ((size_t)C * g.np * (KK + 1) + (size_t)L * C * g.np * 4 * KK);
}

inline void describe(int B, int C, int H, int W, int L, int eb, char *buf, size_t n, int forceG = 0) {
    TGeom f, b;
    int o = 0;
    if (plan(B, C, H, W, L, eb, false, f, forceG))
        o += snprintf(buf + o, n - o, "team fwd[teams=%d x %d thr G=%d T=%d th=%d ring=%d]", f.nteams, f.team, f.G, f.T, f.th, NSTAGE);
    if (o < (int)n && plan(B, C, H, W, L, eb, true, b, forceG))
        snprintf(buf + o, n - o, " bwd[teams=%d x %d thr G=%d T=%d th=%d ring=%d np=%d]", b.nteams, b.team, b.G, b.T, b.th, NSTAGE, b.np);
}

template <typename T, bool BWD>
cudaError_t launch(const TGeom &g, const T *x, const T *go, const float *w0, const float *s0, const float *b0,
                   const float *wl, const float *sl, T *out, float *part0, float *partl, int *status, cudaStream_t st) {
    cudaError_t e;
    if (g.th == 7) {
        constexpr auto kern = team_kernel<T, 7, BWD>;
        if ((e = plane::opt_in_smem<kern>()) != cudaSuccess) return e;
        e = launch_overlapped(kern, (unsigned)g.nblocks, (unsigned)g.nthreads, (size_t)g.smem_bytes, st, g, x, go, w0, s0, b0, wl,
                              sl, out, part0, partl, status);
    } else {
        constexpr auto kern = team_kernel<T, 4, BWD>;
        if ((e = plane::opt_in_smem<kern>()) != cudaSuccess) return e;
        e = launch_overlapped(kern, (unsigned)g.nblocks, (unsigned)g.nthreads, (size_t)g.smem_bytes, st, g, x, go, w0, s0, b0, wl,
                              sl, out, part0, partl, status);
    }
    return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename T>
cudaError_t forward(int B, int C, int H, int W, int L, const T *x, const float *w0, const float *s0, const float *b0,
                    const float *wl, const float *sl, T *out, char *ws, cudaStream_t st, unsigned tag, bool no_copy,
                    int forceG) {
    TGeom g;
    if (!plan(B, C, H, W, L, (int)sizeof(T), false, g, forceG)) return cudaErrorInvalidValue;
    g.no_copy = no_copy;
    g.tag = tag;  // nothing is cleared: see the status words in common.cuh
    return launch<T, false>(g, x, nullptr, w0, s0, b0, wl, sl, out, nullptr, nullptr, reinterpret_cast<int *>(ws), st);
}

template <typename T>
cudaError_t backward(int B, int C, int H, int W, int L, const T *x, const T *go, const float *w0, const float *s0,
                     const float *wl, const float *sl, T *gx, char *ws, EpiloguePtrs *ep, cudaStream_t st, unsigned tag,
                     bool no_copy, int forceG) {
    TGeom g;
    if (!plan(B, C, H, W, L, (int)sizeof(T), true, g, forceG)) return cudaErrorInvalidValue;
    g.no_copy = no_copy;
    g.tag = tag;
    float *part0 = reinterpret_cast<float *>(ws + plane::STATUS_BYTES);
    float *partl = part0 + (size_t)C * g.np * (KK + 1);
    cudaError_t e;  // nothing is cleared: the epilogue is told which partial slots the blocks write
    if ((e = launch<T, true>(g, x, go, w0, s0, nullptr, wl, sl, gx, part0, partl, reinterpret_cast<int *>(ws), st)) != cudaSuccess)
        return e;
    ep->part0 = part0;
    ep->np0 = g.np;
    for (int l = 0; l < L; ++l) {
        ep->partl[l] = partl + (size_t)l * C * g.np * 4 * KK;
        ep->npl[l] = g.np;
    }
    ep->grp = g.G; ep->B = B; ep->units = g.units; ep->nblocks = g.nblocks;
    return cudaSuccess;
}

#define WT_TEAM_INSTANTIATE(T, EXTERN)                                                                                     \
    EXTERN template cudaError_t forward<T>(int, int, int, int, int, const T *, const float *, const float *, const float *, \
                                           const float *, const float *, T *, char *, cudaStream_t, unsigned, bool, int);  \
    EXTERN template cudaError_t backward<T>(int, int, int, int, int, const T *, const T *, const float *, const float *,    \
                                            const float *, const float *, T *, char *, EpiloguePtrs *, cudaStream_t,       \
                                            unsigned, bool, int);

}  // namespace team
}  // namespace wt
