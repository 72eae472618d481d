/*
 * WTConv oracle: a plain, slow, fp64 CPU statement of the operator of Algorithm 1
 * (downward decomposition loop, upward reconstruction loop, base path) and of its
 * analytic gradient.
 *
 * THIS IS TEST INFRASTRUCTURE. It is not part of the product path. Only the test
 * suite, the smoke check and the benchmark's CPU-baseline leg may load it. It shares
 * no code, header, table or helper with the CUDA library.
 *
 * What it deliberately does NOT do (so that the CUDA path's reformulations stay real
 * tests): no scale folding (the scale multiplies the convolution result, as in line 4
 * of Algorithm 1 and Sec. 4.3's "reference" form), no closed-form synthesis (the
 * reconstruction is the level-by-level cascade of Algorithm 1 lines 7-10), no tiling,
 * no fusion. The scale gradient is the direct derivative of "scale times conv result",
 * not Eq. 9.
 *
 * Readings of points the paper leaves open (identical to the library's contract):
 *  - "depthwise convolution, zero-padded to preserve resolution" (Sec. 2.1) is a
 *    cross-correlation: out[y,x] = sum_{u,v} w[u,v] * in[y+u-R, x+v-R], R = k/2,
 *    zero outside the grid.
 *  - An odd height or width is zero-padded on the bottom/right to even before each
 *    Haar level; the level grid is ceil(H/2) x ceil(W/2); each synthesis result is
 *    cropped back to the size it came from. This is the only padding compatible with
 *    the origin-anchored bit indexing of Proposition 2.
 *  - Subband order (LL, LH, HL, HH) with the butterfly of Eq. 5; LH carries the
 *    row (y) sign and HL the column (x) sign, as in the sign table of Appendix A.
 *  - The carrier into the next level is the RAW low-pass band (Algorithm 1 line 5).
 *  - Bias b is optional (NULL means zero); only the base path has one.
 *
 * Layouts (all C-contiguous double):
 *   x, out, g, dx : [B][C][H][W]
 *   w0, dw0       : [C][k][k]        s0, ds0, b0, db0 : [C]
 *   wl, dwl       : [L][C][4][k][k]  sl, dsl          : [L][C][4]
 *
 * Parity pins live in tests/test_oracle_*.py: brute force from explicit Haar basis
 * functions, perfect reconstruction, closed form vs cascade, scale folding, torch
 * fp64 library convolutions + autograd, central finite differences, adjoint identity.
 */
#include <stdlib.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define MAXL 16

int wtoracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ceil(n / 2) */
static int half_up(int n) { return (n + 1) / 2; }

/* level shape: H_0 = H, H_l = ceil(H_{l-1} / 2) */
void wtoracle_level_shape(int H, int W, int level, int *Hl, int *Wl) {
    for (int l = 0; l < level; ++l) { H = half_up(H); W = half_up(W); }
    *Hl = H; *Wl = W;
}

static double at0(const double *p, int H, int W, int y, int x) {
    return (y >= 0 && y < H && x >= 0 && x < W) ? p[(size_t)y * W + x] : 0.0;
}

/* One Haar analysis level (Eq. 5). X: [H][W]; Y: [4][Hh][Wh], Hh=ceil(H/2). */
void wtoracle_haar_analysis(const double *X, int H, int W, double *Y) {
    int Hh = half_up(H), Wh = half_up(W);
    size_t S = (size_t)Hh * Wh;
    for (int i = 0; i < Hh; ++i)
        for (int j = 0; j < Wh; ++j) {
            double a = at0(X, H, W, 2 * i, 2 * j);
            double b = at0(X, H, W, 2 * i, 2 * j + 1);
            double c = at0(X, H, W, 2 * i + 1, 2 * j);
            double d = at0(X, H, W, 2 * i + 1, 2 * j + 1);
            size_t o = (size_t)i * Wh + j;
            Y[0 * S + o] = 0.5 * (a + b + c + d); /* LL */
            Y[1 * S + o] = 0.5 * (a + b - c - d); /* LH */
            Y[2 * S + o] = 0.5 * (a - b + c - d); /* HL */
            Y[3 * S + o] = 0.5 * (a - b - c + d); /* HH */
        }
}

/* One Haar synthesis level (sign table of Appendix A), cropped to H x W.
 * T: [4][Hh][Wh] with Hh=ceil(H/2); R: [H][W]. */
void wtoracle_haar_synthesis(const double *T, int H, int W, double *R) {
    int Hh = half_up(H), Wh = half_up(W);
    size_t S = (size_t)Hh * Wh;
    for (int y = 0; y < H; ++y)
        for (int x = 0; x < W; ++x) {
            int i = y / 2, j = x / 2, ry = y % 2, rx = x % 2;
            size_t o = (size_t)i * Wh + j;
            double sy = ry ? -1.0 : 1.0, sx = rx ? -1.0 : 1.0;
            R[(size_t)y * W + x] =
                0.5 * (T[0 * S + o] + sy * T[1 * S + o] + sx * T[2 * S + o] + sy * sx * T[3 * S + o]);
        }
}

/* Zero-padded "same" cross-correlation of one plane with one k x k kernel. */
void wtoracle_corr2d_same(const double *in, int H, int W, const double *w, int k, double *out) {
    int R = k / 2;
    for (int y = 0; y < H; ++y)
        for (int x = 0; x < W; ++x) {
            double acc = 0.0;
            for (int u = 0; u < k; ++u)
                for (int v = 0; v < k; ++v)
                    acc += w[u * k + v] * at0(in, H, W, y + u - R, x + v - R);
            out[(size_t)y * W + x] = acc;
        }
}

/* Same, with the kernel rotated by 180 degrees (the adjoint of the map above). */
static void corr2d_same_flipped(const double *in, int H, int W, const double *w, int k, double *out) {
    int R = k / 2;
    for (int y = 0; y < H; ++y)
        for (int x = 0; x < W; ++x) {
            double acc = 0.0;
            for (int u = 0; u < k; ++u)
                for (int v = 0; v < k; ++v)
                    acc += w[u * k + v] * at0(in, H, W, y - u + R, x - v + R);
            out[(size_t)y * W + x] = acc;
        }
}

/* The upward loop of Algorithm 1 for one plane: given Z^l (l=1..L, each [4][H_l][W_l]),
 * return R^1 [H][W].  R^{L+1}=0;  R^l = synth( (Z^l_LL + R^{l+1}) || Z^l_H ), cropped. */
void wtoracle_synthesis_cascade(const double *const *Z, int H, int W, int L, double *R1) {
    int Hs[MAXL + 1], Ws[MAXL + 1];
    for (int l = 0; l <= L; ++l) wtoracle_level_shape(H, W, l, &Hs[l], &Ws[l]);
    if (L == 0) { memset(R1, 0, sizeof(double) * (size_t)H * W); return; }
    double *Rnext = NULL; /* R^{l+1}, size H_l x W_l */
    for (int l = L; l >= 1; --l) {
        size_t S = (size_t)Hs[l] * Ws[l];
        double *T = (double *)malloc(sizeof(double) * 4 * S);
        memcpy(T, Z[l - 1], sizeof(double) * 4 * S);
        if (Rnext) for (size_t o = 0; o < S; ++o) T[o] += Rnext[o];
        double *Rl = (l == 1) ? R1 : (double *)malloc(sizeof(double) * (size_t)Hs[l - 1] * Ws[l - 1]);
        wtoracle_haar_synthesis(T, Hs[l - 1], Ws[l - 1], Rl);
        free(T);
        free(Rnext);
        Rnext = (l == 1) ? NULL : Rl;
    }
}

/* Forward of one (b,c) plane. If Zkeep != NULL, Zkeep[l-1] receives a malloc'd copy of Z^l. */
static void forward_plane(const double *x, int H, int W, int k, int L,
                          const double *w0, double s0, double b0,
                          const double *wl /* [L][4][k][k] via stride */, size_t wl_stride,
                          const double *sl /* [L][4] via stride */, size_t sl_stride,
                          double *out) {
    int Hs[MAXL + 1], Ws[MAXL + 1];
    for (int l = 0; l <= L; ++l) wtoracle_level_shape(H, W, l, &Hs[l], &Ws[l]);
    double *Z[MAXL];
    /* downward loop */
    double *carrier = (double *)malloc(sizeof(double) * (size_t)H * W);
    memcpy(carrier, x, sizeof(double) * (size_t)H * W);
    for (int l = 1; l <= L; ++l) {
        size_t S = (size_t)Hs[l] * Ws[l];
        double *Y = (double *)malloc(sizeof(double) * 4 * S);
        wtoracle_haar_analysis(carrier, Hs[l - 1], Ws[l - 1], Y);
        double *Zl = (double *)malloc(sizeof(double) * 4 * S);
        for (int sub = 0; sub < 4; ++sub) {
            wtoracle_corr2d_same(Y + sub * S, Hs[l], Ws[l], wl + (l - 1) * wl_stride + sub * k * k, k, Zl + sub * S);
            double s = sl[(l - 1) * sl_stride + sub];
            for (size_t o = 0; o < S; ++o) Zl[sub * S + o] *= s; /* filter, then scale */
        }
        Z[l - 1] = Zl;
        free(carrier);
        carrier = (double *)malloc(sizeof(double) * S);
        memcpy(carrier, Y, sizeof(double) * S); /* raw LL */
        free(Y);
    }
    free(carrier);
    /* upward loop */
    double *R1 = (double *)malloc(sizeof(double) * (size_t)H * W);
    wtoracle_synthesis_cascade((const double *const *)Z, H, W, L, R1);
    /* base path + reconstruction */
    wtoracle_corr2d_same(x, H, W, w0, k, out);
    for (size_t o = 0; o < (size_t)H * W; ++o) out[o] = s0 * (out[o] + b0) + R1[o];
    free(R1);
    for (int l = 0; l < L; ++l) free(Z[l]);
}

void wtoracle_forward(int B, int C, int H, int W, int k, int L,
                      const double *x, const double *w0, const double *s0, const double *b0,
                      const double *wl, const double *sl, double *out) {
    size_t plane = (size_t)H * W;
    int kk = k * k;
#pragma omp parallel for schedule(dynamic)
    for (int p = 0; p < B * C; ++p) {
        int c = p % C;
        forward_plane(x + p * plane, H, W, k, L, w0 + (size_t)c * kk, s0[c], b0 ? b0[c] : 0.0,
                      wl ? wl + (size_t)c * 4 * kk : NULL, (size_t)C * 4 * kk,
                      sl ? sl + (size_t)c * 4 : NULL, (size_t)C * 4, out + p * plane);
    }
}

/* Gradient of one plane. Parameter gradients are written to this plane's own slots:
 * pdw0[k*k], pds0, pdb0, pdwl[L][4][k*k], pdsl[L][4]. */
static void backward_plane(const double *x, const double *g, int H, int W, int k, int L,
                           const double *w0, double s0, double b0,
                           const double *wl, size_t wl_stride, const double *sl, size_t sl_stride,
                           double *dx, double *pdw0, double *pds0, double *pdb0, double *pdwl, double *pdsl) {
    int R = k / 2, kk = k * k;
    int Hs[MAXL + 1], Ws[MAXL + 1];
    for (int l = 0; l <= L; ++l) wtoracle_level_shape(H, W, l, &Hs[l], &Ws[l]);
    size_t plane = (size_t)H * W;

    /* ---- base path: out_base = s0 * (corr(x, w0) + b0) ---- */
    double *cx = (double *)malloc(sizeof(double) * plane);
    wtoracle_corr2d_same(x, H, W, w0, k, cx);
    double ds = 0.0, db = 0.0;
    for (size_t o = 0; o < plane; ++o) { ds += g[o] * (cx[o] + b0); db += g[o] * s0; }
    *pds0 = ds; *pdb0 = db;
    free(cx);
    for (int u = 0; u < k; ++u)
        for (int v = 0; v < k; ++v) {
            double acc = 0.0;
            for (int y = 0; y < H; ++y)
                for (int xx = 0; xx < W; ++xx)
                    acc += s0 * g[(size_t)y * W + xx] * at0(x, H, W, y + u - R, xx + v - R);
            pdw0[u * k + v] = acc;
        }
    double *sg = (double *)malloc(sizeof(double) * plane);
    for (size_t o = 0; o < plane; ++o) sg[o] = s0 * g[o];
    corr2d_same_flipped(sg, H, W, w0, k, dx);
    free(sg);
    if (L == 0) return;

    /* ---- recompute the decomposition Y^l (downward loop, forward values) ---- */
    double *Y[MAXL];
    {
        double *carrier = (double *)malloc(sizeof(double) * plane);
        memcpy(carrier, x, sizeof(double) * plane);
        for (int l = 1; l <= L; ++l) {
            size_t S = (size_t)Hs[l] * Ws[l];
            Y[l - 1] = (double *)malloc(sizeof(double) * 4 * S);
            wtoracle_haar_analysis(carrier, Hs[l - 1], Ws[l - 1], Y[l - 1]);
            free(carrier);
            carrier = (double *)malloc(sizeof(double) * S);
            memcpy(carrier, Y[l - 1], sizeof(double) * S);
        }
        free(carrier);
    }

    /* ---- backward through the upward loop: dZ^l.  R^l = crop(synth(T^l)) so
     * dT^l = analysis(pad(dR^l)) (Sec. 2.2: backward through synthesis is analysis);
     * dZ^l = dT^l, dR^{l+1} = dT^l_LL. ---- */
    double *dZ[MAXL];
    {
        double *dR = (double *)malloc(sizeof(double) * plane);
        memcpy(dR, g, sizeof(double) * plane);
        for (int l = 1; l <= L; ++l) {
            size_t S = (size_t)Hs[l] * Ws[l];
            dZ[l - 1] = (double *)malloc(sizeof(double) * 4 * S);
            wtoracle_haar_analysis(dR, Hs[l - 1], Ws[l - 1], dZ[l - 1]);
            free(dR);
            dR = (double *)malloc(sizeof(double) * S);
            memcpy(dR, dZ[l - 1], sizeof(double) * S);
        }
        free(dR);
    }

    /* ---- per level: Z = s * corr(Y, W).  dW, ds, and dY (through the conv). ---- */
    double *dY[MAXL];
    for (int l = 1; l <= L; ++l) {
        int Hl = Hs[l], Wl = Ws[l];
        size_t S = (size_t)Hl * Wl;
        dY[l - 1] = (double *)malloc(sizeof(double) * 4 * S);
        double *cy = (double *)malloc(sizeof(double) * S);
        double *sd = (double *)malloc(sizeof(double) * S);
        for (int sub = 0; sub < 4; ++sub) {
            const double *w = wl + (l - 1) * wl_stride + sub * kk;
            double s = sl[(l - 1) * sl_stride + sub];
            const double *Ys = Y[l - 1] + sub * S;
            const double *dZs = dZ[l - 1] + sub * S;
            wtoracle_corr2d_same(Ys, Hl, Wl, w, k, cy);
            double a = 0.0;
            for (size_t o = 0; o < S; ++o) a += dZs[o] * cy[o];
            pdsl[(l - 1) * 4 + sub] = a;
            for (int u = 0; u < k; ++u)
                for (int v = 0; v < k; ++v) {
                    double acc = 0.0;
                    for (int i = 0; i < Hl; ++i)
                        for (int j = 0; j < Wl; ++j)
                            acc += s * dZs[(size_t)i * Wl + j] * at0(Ys, Hl, Wl, i + u - R, j + v - R);
                    pdwl[((l - 1) * 4 + sub) * kk + u * k + v] = acc;
                }
            for (size_t o = 0; o < S; ++o) sd[o] = s * dZs[o];
            corr2d_same_flipped(sd, Hl, Wl, w, k, dY[l - 1] + sub * S);
        }
        free(cy); free(sd);
    }

    /* ---- backward through the downward loop: Y^l = analysis(pad(X^{l-1})), X^l = Y^l_LL.
     * dX^L = 0; dX^{l-1} = crop(synth(dY^l with dX^l added to its LL band)). ---- */
    {
        double *dXl = NULL; /* dX^l, size H_l x W_l */
        for (int l = L; l >= 1; --l) {
            size_t S = (size_t)Hs[l] * Ws[l];
            if (dXl) for (size_t o = 0; o < S; ++o) dY[l - 1][o] += dXl[o];
            double *dXprev = (double *)malloc(sizeof(double) * (size_t)Hs[l - 1] * Ws[l - 1]);
            wtoracle_haar_synthesis(dY[l - 1], Hs[l - 1], Ws[l - 1], dXprev);
            free(dXl);
            dXl = dXprev;
        }
        for (size_t o = 0; o < plane; ++o) dx[o] += dXl[o];
        free(dXl);
    }
    for (int l = 0; l < L; ++l) { free(Y[l]); free(dZ[l]); free(dY[l]); }
}

/* g = dLoss/d out.  db0/ b0 may be NULL together. Parameter gradients are summed over
 * the batch in index order (deterministic). */
void wtoracle_backward(int B, int C, int H, int W, int k, int L,
                       const double *x, const double *g,
                       const double *w0, const double *s0, const double *b0,
                       const double *wl, const double *sl,
                       double *dx, double *dw0, double *ds0, double *db0, double *dwl, double *dsl) {
    size_t plane = (size_t)H * W;
    int kk = k * k, P = B * C;
    size_t per = (size_t)kk + 2 + (size_t)L * 4 * kk + (size_t)L * 4; /* one plane's parameter-gradient slots */
    double *part = (double *)calloc((size_t)P * per, sizeof(double));
#pragma omp parallel for schedule(dynamic)
    for (int p = 0; p < P; ++p) {
        int c = p % C;
        double *q = part + (size_t)p * per;
        backward_plane(x + p * plane, g + p * plane, H, W, k, L, w0 + (size_t)c * kk, s0[c], b0 ? b0[c] : 0.0,
                       wl ? wl + (size_t)c * 4 * kk : NULL, (size_t)C * 4 * kk,
                       sl ? sl + (size_t)c * 4 : NULL, (size_t)C * 4,
                       dx + p * plane, q, q + kk, q + kk + 1, q + kk + 2, q + kk + 2 + (size_t)L * 4 * kk);
    }
    for (int c = 0; c < C; ++c) {
        for (int t = 0; t < kk; ++t) dw0[(size_t)c * kk + t] = 0.0;
        ds0[c] = 0.0;
        if (db0) db0[c] = 0.0;
        for (int l = 0; l < L; ++l)
            for (int sub = 0; sub < 4; ++sub) {
                for (int t = 0; t < kk; ++t) dwl[(((size_t)l * C + c) * 4 + sub) * kk + t] = 0.0;
                dsl[((size_t)l * C + c) * 4 + sub] = 0.0;
            }
    }
    for (int b = 0; b < B; ++b)
        for (int c = 0; c < C; ++c) {
            const double *q = part + (size_t)(b * C + c) * per;
            for (int t = 0; t < kk; ++t) dw0[(size_t)c * kk + t] += q[t];
            ds0[c] += q[kk];
            if (db0) db0[c] += q[kk + 1];
            const double *qw = q + kk + 2, *qs = qw + (size_t)L * 4 * kk;
            for (int l = 0; l < L; ++l)
                for (int sub = 0; sub < 4; ++sub) {
                    for (int t = 0; t < kk; ++t)
                        dwl[(((size_t)l * C + c) * 4 + sub) * kk + t] += qw[(l * 4 + sub) * kk + t];
                    dsl[((size_t)l * C + c) * 4 + sub] += qs[l * 4 + sub];
                }
        }
    free(part);
}
