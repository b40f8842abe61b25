/*
 * Sali-Cache pre-attention filter + mixed-precision K/V store: CPU ORACLE.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow statement of what the
 * hot path computes.  It shares no code, table or constant generator with the
 * CUDA library; only tests, the smoke check and the benchmark's CPU-baseline leg
 * may call it.  Scores are computed in double; the decision rule and the
 * quantisers use single IEEE-754 binary32 operations in a fixed order
 * (compile with -ffp-contract=off, no fast-math).
 *
 * Every function names the passage of the paper it follows.  Where the paper
 * is silent the reading taken is stated next to the code.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_*.py against
 * closed forms, brute force or library routines.  The paper's aggregate numbers
 * (2.20x compression, 26.7 % reuse, per-frame latency) are "parity unpinned":
 * they need the authors' videos, thresholds and model.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define EXPORT __attribute__((visibility("default")))

static int clampi(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }

EXPORT int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------- */
/* Gray level.  The paper does not say how colour becomes intensity; reading:  */
/* integer luma g = (77 R + 150 G + 29 B + 128) >> 8 so that the edge branch   */
/* is exact integer work.                                                      */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_gray(const uint8_t* rgb, int h, int w, uint8_t* g) {
    for (int i = 0; i < h * w; ++i) {
        int R = rgb[3 * i], G = rgb[3 * i + 1], B = rgb[3 * i + 2];
        g[i] = (uint8_t)((77 * R + 150 * G + 29 * B + 128) >> 8);
    }
}

/* Anyres base image: exact 2x2 integer box mean (a+b+c+d+2)>>2 per channel.   */
/* (The paper only mentions dynamic-resolution encoding, Sec. II-A.)           */
EXPORT void oracle_box_down2(const uint8_t* rgb, int h, int w, uint8_t* out) {
    int h2 = h / 2, w2 = w / 2;
    for (int y = 0; y < h2; ++y)
        for (int x = 0; x < w2; ++x)
            for (int c = 0; c < 3; ++c) {
                int s = rgb[((2 * y) * w + 2 * x) * 3 + c] + rgb[((2 * y) * w + 2 * x + 1) * 3 + c] +
                        rgb[((2 * y + 1) * w + 2 * x) * 3 + c] + rgb[((2 * y + 1) * w + 2 * x + 1) * 3 + c];
                out[(y * w2 + x) * 3 + c] = (uint8_t)((s + 2) >> 2);
            }
}

/* ------------------------------------------------------------------------- */
/* Pyramid, scale 0.5 (Sec. IV-B "pyramid scale of 0.5 and 3 pyramid levels"). */
/* Reading: 5x5 binomial smoothing [1 4 6 4 1]/16, sample at (2y, 2x), clamp.  */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_pyr_down(const double* src, int h, int w, double* dst) {
    static const double k[5] = {1.0 / 16, 4.0 / 16, 6.0 / 16, 4.0 / 16, 1.0 / 16};
    int h2 = h / 2, w2 = w / 2;
    for (int y = 0; y < h2; ++y)
        for (int x = 0; x < w2; ++x) {
            double acc = 0.0;
            for (int a = -2; a <= 2; ++a)
                for (int b = -2; b <= 2; ++b)
                    acc += k[a + 2] * k[b + 2] *
                           src[clampi(2 * y + a, 0, h - 1) * w + clampi(2 * x + b, 0, w - 1)];
            dst[y * w2 + x] = acc;
        }
}

/* ------------------------------------------------------------------------- */
/* Polynomial expansion (Farneback's method, named in Sec. IV-B).              */
/* f(x+d) ~ r1 + r2 dx + r3 dy + r4 dx^2 + r5 dy^2 + r6 dx dy, fitted by       */
/* least squares with separable Gaussian weights g(dx) g(dy) on a              */
/* (2n+1)^2 neighbourhood.  Because g is even the normal equations decouple:   */
/*   r2 = m10/mu2, r3 = m01/mu2, r6 = m11/mu2^2,                               */
/*   r4 = (m20 - mu2 m00)/(mu4 - mu2^2), r5 = (m02 - mu2 m00)/(mu4 - mu2^2),   */
/* with m_pq = sum g(dx) g(dy) dx^p dy^q f(x+d).  Output planes: r2 r3 r4 r5 r6*/
/* Reading (paper silent): n = 2, sigma = 1.2, clamp-to-edge.                  */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_poly_exp(const double* f, int h, int w, int n, double sigma, double* r) {
    double g[33];
    double Z = 0.0, mu2 = 0.0, mu4 = 0.0;
    for (int k = -n; k <= n; ++k) { g[k + n] = exp(-(double)(k * k) / (2.0 * sigma * sigma)); Z += g[k + n]; }
    for (int k = -n; k <= n; ++k) {
        g[k + n] /= Z;
        mu2 += g[k + n] * k * k;
        mu4 += g[k + n] * k * k * (double)(k * k);
    }
    double den = mu4 - mu2 * mu2;
    size_t P = (size_t)h * w;
    for (int y = 0; y < h; ++y)
        for (int x = 0; x < w; ++x) {
            double m00 = 0, m10 = 0, m01 = 0, m20 = 0, m02 = 0, m11 = 0;
            for (int dy = -n; dy <= n; ++dy)
                for (int dx = -n; dx <= n; ++dx) {
                    double v = g[dy + n] * g[dx + n] * f[clampi(y + dy, 0, h - 1) * w + clampi(x + dx, 0, w - 1)];
                    m00 += v;
                    m10 += v * dx;
                    m01 += v * dy;
                    m20 += v * dx * dx;
                    m02 += v * dy * dy;
                    m11 += v * dx * dy;
                }
            size_t i = (size_t)y * w + x;
            r[0 * P + i] = m10 / mu2;
            r[1 * P + i] = m01 / mu2;
            r[2 * P + i] = (m20 - mu2 * m00) / den;
            r[3 * P + i] = (m02 - mu2 * m00) / den;
            r[4 * P + i] = m11 / (mu2 * mu2);
        }
}

/* Bilinear sample of one plane at a clamped continuous position. */
static double bilin(const double* p, int h, int w, double y, double x) {
    if (x < 0) x = 0;
    if (x > w - 1) x = w - 1;
    if (y < 0) y = 0;
    if (y > h - 1) y = h - 1;
    int x0 = (int)floor(x), y0 = (int)floor(y);
    int x1 = x0 + 1 < w ? x0 + 1 : w - 1, y1 = y0 + 1 < h ? y0 + 1 : h - 1;
    double fx = x - x0, fy = y - y0;
    double top = p[y0 * w + x0] * (1.0 - fx) + p[y0 * w + x1] * fx;
    double bot = p[y1 * w + x0] * (1.0 - fx) + p[y1 * w + x1] * fx;
    return top * (1.0 - fy) + bot * fy;
}

/* ------------------------------------------------------------------------- */
/* One displacement update at one pyramid level (Farneback's estimate with an  */
/* a-priori displacement).  Convention: I_cur(x + d) ~ I_prev(x); d = (u, v),  */
/* u along x.  c1, c2: expansion planes of the previous and current frame.     */
/*   xt   = clamp(x + d~)                                                      */
/*   A    = (A1(x) + A2(xt))/2,      A = [[r4, r6/2],[r6/2, r5]]               */
/*   db   = -(b2(xt) - b1(x))/2 + A d~,   b = (r2, r3)                          */
/*   G    = A^T A,  hv = A^T db; both summed over the in-image part of the     */
/*   win x win box centred on x (uniform weights);                             */
/*   d    = adj(G) hv / (det G + eps)                                          */
/* Reading (paper silent): bilinear fetch, box window 15, eps = 1e-3.          */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_flow_iter(const double* c1, const double* c2, int h, int w, const double* d_in,
                             int win, double eps, double* d_out) {
    size_t P = (size_t)h * w;
    double* t = (double*)malloc(5 * P * sizeof(double));
    for (int y = 0; y < h; ++y)
        for (int x = 0; x < w; ++x) {
            size_t i = (size_t)y * w + x;
            double du = d_in[i], dv = d_in[P + i];
            double xt = x + du, yt = y + dv;
            double b2x = bilin(c2 + 0 * P, h, w, yt, xt), b2y = bilin(c2 + 1 * P, h, w, yt, xt);
            double a2xx = bilin(c2 + 2 * P, h, w, yt, xt), a2yy = bilin(c2 + 3 * P, h, w, yt, xt);
            double a2xy = 0.5 * bilin(c2 + 4 * P, h, w, yt, xt);
            double axx = 0.5 * (c1[2 * P + i] + a2xx);
            double ayy = 0.5 * (c1[3 * P + i] + a2yy);
            double axy = 0.5 * (0.5 * c1[4 * P + i] + a2xy);
            double dbx = -0.5 * (b2x - c1[0 * P + i]) + (axx * du + axy * dv);
            double dby = -0.5 * (b2y - c1[1 * P + i]) + (axy * du + ayy * dv);
            t[0 * P + i] = axx * axx + axy * axy;       /* g11 */
            t[1 * P + i] = axx * axy + axy * ayy;       /* g12 */
            t[2 * P + i] = axy * axy + ayy * ayy;       /* g22 */
            t[3 * P + i] = axx * dbx + axy * dby;       /* h1  */
            t[4 * P + i] = axy * dbx + ayy * dby;       /* h2  */
        }
    int rad = win / 2;
    for (int y = 0; y < h; ++y)
        for (int x = 0; x < w; ++x) {
            double s[5] = {0, 0, 0, 0, 0};
            for (int yy = y - rad; yy <= y + rad; ++yy) {
                if (yy < 0 || yy >= h) continue;
                for (int xx = x - rad; xx <= x + rad; ++xx) {
                    if (xx < 0 || xx >= w) continue;
                    size_t j = (size_t)yy * w + xx;
                    for (int c = 0; c < 5; ++c) s[c] += t[c * P + j];
                }
            }
            double det = s[0] * s[2] - s[1] * s[1] + eps;
            size_t i = (size_t)y * w + x;
            d_out[i] = (s[2] * s[3] - s[1] * s[4]) / det;
            d_out[P + i] = (s[0] * s[4] - s[1] * s[3]) / det;
        }
    free(t);
}

/* Coarse-to-fine transfer: d_fine(y,x) = 2 * bilinear(d_coarse) sampled at    */
/* ((x+1/2)/2 - 1/2, (y+1/2)/2 - 1/2), clamped (pixel-centre alignment).       */
EXPORT void oracle_flow_upsample(const double* dc, int hc, int wc, double* df, int hf, int wf) {
    size_t Pc = (size_t)hc * wc, Pf = (size_t)hf * wf;
    for (int y = 0; y < hf; ++y)
        for (int x = 0; x < wf; ++x) {
            double xs = (x + 0.5) / 2.0 - 0.5, ys = (y + 0.5) / 2.0 - 0.5;
            df[(size_t)y * wf + x] = 2.0 * bilin(dc, hc, wc, ys, xs);
            df[Pf + (size_t)y * wf + x] = 2.0 * bilin(dc + Pc, hc, wc, ys, xs);
        }
}

/* ------------------------------------------------------------------------- */
/* Dense flow between two RGB frames (Sec. III-A; Farneback, scale 0.5,        */
/* `levels` pyramid levels, Sec. IV-B).  Coarse to fine, `iters` updates per   */
/* level, zero prior at the coarsest level.  flow = [2][h][w] (u then v).      */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_flow(const uint8_t* prev, const uint8_t* cur, int h, int w, int levels, int poly_n,
                        double poly_sigma, int win, int iters, double eps, double* flow) {
    const uint8_t* fr[2] = {prev, cur};
    double* pyr[2][8];
    double* coef[2][8];
    int hs[8], ws[8];
    for (int l = 0; l < levels; ++l) { hs[l] = h >> l; ws[l] = w >> l; }
    for (int f = 0; f < 2; ++f) {
        uint8_t* g = (uint8_t*)malloc((size_t)h * w);
        oracle_gray(fr[f], h, w, g);
        pyr[f][0] = (double*)malloc((size_t)h * w * sizeof(double));
        for (int i = 0; i < h * w; ++i) pyr[f][0][i] = (double)g[i];
        free(g);
        for (int l = 1; l < levels; ++l) {
            pyr[f][l] = (double*)malloc((size_t)hs[l] * ws[l] * sizeof(double));
            oracle_pyr_down(pyr[f][l - 1], hs[l - 1], ws[l - 1], pyr[f][l]);
        }
        for (int l = 0; l < levels; ++l) {
            coef[f][l] = (double*)malloc((size_t)5 * hs[l] * ws[l] * sizeof(double));
            oracle_poly_exp(pyr[f][l], hs[l], ws[l], poly_n / 2, poly_sigma, coef[f][l]);
        }
    }
    double* d = NULL;
    for (int l = levels - 1; l >= 0; --l) {
        size_t P = (size_t)hs[l] * ws[l];
        double* dl = (double*)calloc(2 * P, sizeof(double));
        if (d) {
            oracle_flow_upsample(d, hs[l + 1], ws[l + 1], dl, hs[l], ws[l]);
            free(d);
        }
        double* tmp = (double*)malloc(2 * P * sizeof(double));
        for (int it = 0; it < iters; ++it) {
            oracle_flow_iter(coef[0][l], coef[1][l], hs[l], ws[l], dl, win, eps, tmp);
            memcpy(dl, tmp, 2 * P * sizeof(double));
        }
        free(tmp);
        d = dl;
    }
    memcpy(flow, d, (size_t)2 * h * w * sizeof(double));
    free(d);
    for (int f = 0; f < 2; ++f)
        for (int l = 0; l < levels; ++l) { free(pyr[f][l]); free(coef[f][l]); }
}

/* ------------------------------------------------------------------------- */
/* Patch temporal score (Eq. 5).  Reading: F in Eq. 5 is the displacement      */
/* field (the text, Alg. 1 and Sec. IV-B all say optical flow); the L2 norm    */
/* over the patch is normalised by its area, so dP is an RMS in pixels:        */
/*   dP_i = sqrt( (1/|P_i|) sum_{P_i} (u^2 + v^2) ).                            */
/* Patches row-major on the (h/patch) x (w/patch) grid.                        */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_delta_p(const double* flow, int h, int w, int patch, double* dP) {
    int gh = h / patch, gw = w / patch;
    size_t P = (size_t)h * w;
    for (int py = 0; py < gh; ++py)
        for (int px = 0; px < gw; ++px) {
            double acc = 0.0;
            for (int y = py * patch; y < (py + 1) * patch; ++y)
                for (int x = px * patch; x < (px + 1) * patch; ++x) {
                    double u = flow[(size_t)y * w + x], v = flow[P + (size_t)y * w + x];
                    acc += u * u + v * v;
                }
            dP[py * gw + px] = sqrt(acc / (double)(patch * patch));
        }
}

/* ------------------------------------------------------------------------- */
/* Eq. 5 exactly as printed: dP_i = || F^N_i - F^{N-1}_i ||_2 over the pixels   */
/* (all three channels) of patch i.  Reading: divided by sqrt(3 patch^2), so    */
/* that it is an RMS difference in grey levels (the paper gives no scale).      */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_diff_score(const uint8_t* prev, const uint8_t* cur, int h, int w, int patch, double* dP) {
    int gh = h / patch, gw = w / patch;
    for (int py = 0; py < gh; ++py)
        for (int px = 0; px < gw; ++px) {
            double acc = 0.0;
            for (int y = py * patch; y < (py + 1) * patch; ++y)
                for (int x = px * patch; x < (px + 1) * patch; ++x)
                    for (int c = 0; c < 3; ++c) {
                        double d = (double)cur[((size_t)y * w + x) * 3 + c] - (double)prev[((size_t)y * w + x) * 3 + c];
                        acc += d * d;
                    }
            dP[py * gw + px] = sqrt(acc / (3.0 * patch * patch));
        }
}

/* Frame pairs -> dP, B pairs in parallel over host threads.  dP: [B][n_patches]. */
EXPORT void oracle_flow_score_batch(const uint8_t* prev, const uint8_t* cur, int B, int h, int w, int patch,
                                    int levels, int poly_n, double poly_sigma, int win, int iters, double eps,
                                    double* dP, double* flow_or_null) {
    size_t fb = (size_t)h * w * 3;
    int np = (h / patch) * (w / patch);
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        double* fl = flow_or_null ? flow_or_null + (size_t)b * 2 * h * w : (double*)malloc((size_t)2 * h * w * sizeof(double));
        oracle_flow(prev + b * fb, cur + b * fb, h, w, levels, poly_n, poly_sigma, win, iters, eps, fl);
        oracle_delta_p(fl, h, w, patch, dP + (size_t)b * np);
        if (!flow_or_null) free(fl);
    }
}

/* ------------------------------------------------------------------------- */
/* Edge map E (Canny, Sec. III-B / IV-B), all integer.  Reading of the steps   */
/* the paper leaves open:                                                      */
/*  (i)  blur  Bl = (sum k(a) k(b) g + 128) >> 8, k = [1 4 6 4 1], clamp;      */
/*  (ii) Sobel 3x3 on Bl, clamp;  (iii) m = gx^2 + gy^2;                       */
/*  (iv) non-maximum suppression along the gradient sector: |gy|/|gx| <=       */
/*       13573/32768 (tan 22.5 deg) -> x; the transposed test -> y; else the   */
/*       diagonal picked by the sign of gx*gy.  Keep when m > m(n-) and        */
/*       m >= m(n+), n- the neighbour that comes first in (y, x) order;        */
/*       neighbours outside the image count as 0;                              */
/*  (v)  strong: m >= hi^2, weak: m >= lo^2;                                   */
/*  (vi) hysteresis: kept strong pixels, plus kept weak pixels 8-connected     */
/*       through kept weak/strong pixels to a strong one (flood fill).         */
/* cls_or_null receives 0 / 1 (kept weak) / 2 (kept strong) before hysteresis. */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_canny(const uint8_t* g, int h, int w, int lo, int hi, uint8_t* E, uint8_t* cls_or_null) {
    static const int k[5] = {1, 4, 6, 4, 1};
    size_t P = (size_t)h * w;
    int* Bl = (int*)malloc(P * sizeof(int));
    int* gx = (int*)malloc(P * sizeof(int));
    int* gy = (int*)malloc(P * sizeof(int));
    int* m = (int*)malloc(P * sizeof(int));
    uint8_t* cls = (uint8_t*)calloc(P, 1);
    for (int y = 0; y < h; ++y)
        for (int x = 0; x < w; ++x) {
            int acc = 0;
            for (int a = -2; a <= 2; ++a)
                for (int b = -2; b <= 2; ++b)
                    acc += k[a + 2] * k[b + 2] * g[clampi(y + a, 0, h - 1) * w + clampi(x + b, 0, w - 1)];
            Bl[y * w + x] = (acc + 128) >> 8;
        }
#define BL(yy, xx) Bl[clampi((yy), 0, h - 1) * w + clampi((xx), 0, w - 1)]
    for (int y = 0; y < h; ++y)
        for (int x = 0; x < w; ++x) {
            int sx = (BL(y - 1, x + 1) + 2 * BL(y, x + 1) + BL(y + 1, x + 1)) -
                     (BL(y - 1, x - 1) + 2 * BL(y, x - 1) + BL(y + 1, x - 1));
            int sy = (BL(y + 1, x - 1) + 2 * BL(y + 1, x) + BL(y + 1, x + 1)) -
                     (BL(y - 1, x - 1) + 2 * BL(y - 1, x) + BL(y - 1, x + 1));
            gx[y * w + x] = sx;
            gy[y * w + x] = sy;
            m[y * w + x] = sx * sx + sy * sy;
        }
#undef BL
#define M(yy, xx) (((yy) < 0 || (yy) >= h || (xx) < 0 || (xx) >= w) ? 0 : m[(yy) * w + (xx)])
    for (int y = 0; y < h; ++y)
        for (int x = 0; x < w; ++x) {
            int sx = gx[y * w + x], sy = gy[y * w + x], mm = m[y * w + x];
            long ax = labs((long)sx), ay = labs((long)sy);
            int mneg, mpos;
            if (32768 * ay <= 13573 * ax) { mneg = M(y, x - 1); mpos = M(y, x + 1); }
            else if (32768 * ax <= 13573 * ay) { mneg = M(y - 1, x); mpos = M(y + 1, x); }
            else if ((sx > 0) == (sy > 0)) { mneg = M(y - 1, x - 1); mpos = M(y + 1, x + 1); }
            else { mneg = M(y - 1, x + 1); mpos = M(y + 1, x - 1); }
            int keep = (mm > mneg) && (mm >= mpos);
            if (keep && mm >= hi * hi) cls[y * w + x] = 2;
            else if (keep && mm >= lo * lo) cls[y * w + x] = 1;
        }
#undef M
    memset(E, 0, P);
    int* stack = (int*)malloc(P * sizeof(int));
    size_t top = 0;
    for (size_t i = 0; i < P; ++i)
        if (cls[i] == 2) { E[i] = 1; stack[top++] = (int)i; }
    while (top) {
        int i = stack[--top];
        int y = i / w, x = i % w;
        for (int dy = -1; dy <= 1; ++dy)
            for (int dx = -1; dx <= 1; ++dx) {
                int yy = y + dy, xx = x + dx;
                if (yy < 0 || yy >= h || xx < 0 || xx >= w) continue;
                int j = yy * w + xx;
                if (cls[j] && !E[j]) { E[j] = 1; stack[top++] = j; }
            }
    }
    if (cls_or_null) memcpy(cls_or_null, cls, P);
    free(stack); free(cls); free(m); free(gy); free(gx); free(Bl);
}

/* ------------------------------------------------------------------------- */
/* sRGB (8-bit) -> CIE L*a*b*, D65.  IEC 61966-2-1 transfer curve, sRGB        */
/* primaries, white (0.95047, 1, 1.08883).  lab = [3] per pixel.               */
/* ------------------------------------------------------------------------- */
static double srgb_to_linear(int c) {
    double v = c / 255.0;
    return v <= 0.04045 ? v / 12.92 : pow((v + 0.055) / 1.055, 2.4);
}
static double lab_f(double t) {
    const double d = 6.0 / 29.0;
    return t > d * d * d ? cbrt(t) : t / (3.0 * d * d) + 4.0 / 29.0;
}
EXPORT void oracle_rgb_to_lab(const uint8_t* rgb, int n, double* lab) {
    for (int i = 0; i < n; ++i) {
        double r = srgb_to_linear(rgb[3 * i]), g = srgb_to_linear(rgb[3 * i + 1]), b = srgb_to_linear(rgb[3 * i + 2]);
        double X = 0.4124564 * r + 0.3575761 * g + 0.1804375 * b;
        double Y = 0.2126729 * r + 0.7151522 * g + 0.0721750 * b;
        double Zv = 0.0193339 * r + 0.1191920 * g + 0.9503041 * b;
        double fx = lab_f(X / 0.95047), fy = lab_f(Y / 1.0), fz = lab_f(Zv / 1.08883);
        lab[3 * i] = 116.0 * fy - 16.0;
        lab[3 * i + 1] = 500.0 * (fx - fy);
        lab[3 * i + 2] = 200.0 * (fy - fz);
    }
}

/* ------------------------------------------------------------------------- */
/* Colour branch C (Sec. III-B "color variance analysis in the LAB color       */
/* space", Sec. IV-B "adaptive thresholding based on the local color           */
/* variance").  Reading: V = sum over L, a, b of the population variance in    */
/* the (2r+1)^2 clamp-to-edge window; C = min(1, sqrt(V)/sigma_ref).           */
/* ------------------------------------------------------------------------- */
/* V alone: the summed population variance of L, a, b in the window, per pixel. */
EXPORT void oracle_color_variance(const uint8_t* rgb, int h, int w, int radius, double* V) {
    size_t P = (size_t)h * w;
    double* lab = (double*)malloc(3 * P * sizeof(double));
    oracle_rgb_to_lab(rgb, (int)P, lab);
    int n = (2 * radius + 1) * (2 * radius + 1);
    for (int y = 0; y < h; ++y)
        for (int x = 0; x < w; ++x) {
            double v = 0.0;
            for (int c = 0; c < 3; ++c) {
                double mean = 0.0;
                for (int dy = -radius; dy <= radius; ++dy)
                    for (int dx = -radius; dx <= radius; ++dx)
                        mean += lab[3 * ((size_t)clampi(y + dy, 0, h - 1) * w + clampi(x + dx, 0, w - 1)) + c];
                mean /= n;
                double var = 0.0;
                for (int dy = -radius; dy <= radius; ++dy)
                    for (int dx = -radius; dx <= radius; ++dx) {
                        double dv = lab[3 * ((size_t)clampi(y + dy, 0, h - 1) * w + clampi(x + dx, 0, w - 1)) + c] - mean;
                        var += dv * dv;
                    }
                v += var / n;
            }
            V[(size_t)y * w + x] = v;
        }
    free(lab);
}

EXPORT void oracle_color_contrast(const uint8_t* rgb, int h, int w, int radius, double sigma_ref, double* C) {
    size_t P = (size_t)h * w;
    oracle_color_variance(rgb, h, w, radius, C);
    for (size_t i = 0; i < P; ++i) {
        double c01 = sqrt(C[i]) / sigma_ref;
        C[i] = c01 < 1.0 ? c01 : 1.0;
    }
}

/* ------------------------------------------------------------------------- */
/* Colour branch, frame-adaptive reading of "adaptive thresholding based on    */
/* the local color variance" (Sec. IV-B): the local contrast sqrt(V) is        */
/* measured against the frame's own contrast level instead of a fixed          */
/* sigma_ref:                                                                  */
/*   sigma_frame = max( sqrt( mean over the frame of V ), sigma_min ),         */
/*   C = min(1, sqrt(V) / (kappa * sigma_frame)),                              */
/* so a dim or low-contrast frame keeps the same share of salient pixels as a  */
/* vivid one.  sigma_min (LAB units) keeps a frame without any contrast from   */
/* having its rounding noise promoted to saliency; with sigma_min = 0 a frame  */
/* whose V vanishes everywhere gets C = 0.  The normalisation is a function of */
/* the V map alone.                                                            */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_color_normalise_global(const double* V, size_t n, double kappa, double sigma_min, double* C) {
    double sum = 0.0;
    for (size_t i = 0; i < n; ++i) sum += V[i];
    double sigma = sqrt(sum / (double)n);
    if (sigma < sigma_min) sigma = sigma_min;
    for (size_t i = 0; i < n; ++i) {
        double c01 = sigma > 0.0 ? sqrt(V[i]) / (kappa * sigma) : 0.0;
        C[i] = c01 < 1.0 ? c01 : 1.0;
    }
}

EXPORT void oracle_color_contrast_global(const uint8_t* rgb, int h, int w, int radius, double kappa, double sigma_min,
                                         double* C) {
    size_t P = (size_t)h * w;
    double* V = (double*)malloc(P * sizeof(double));
    oracle_color_variance(rgb, h, w, radius, V);
    oracle_color_normalise_global(V, P, kappa, sigma_min, C);
    free(V);
}

/* ------------------------------------------------------------------------- */
/* Saliency map S in [0,1] and patch score s_i (Eq. 7):                        */
/*   S = clamp(w_edge E + w_color C, 0, 1),  s_i = mean over patch i of S.      */
/* S_or_null receives the per-pixel map.                                       */
/* ------------------------------------------------------------------------- */
static void saliency_impl(const uint8_t* rgb, int h, int w, int patch, int lo, int hi, int radius, int global_norm,
                          double sigma_ref_or_kappa, double sigma_min, double w_edge, double w_color, double* s,
                          double* S_or_null) {
    size_t P = (size_t)h * w;
    uint8_t* g = (uint8_t*)malloc(P);
    uint8_t* E = (uint8_t*)malloc(P);
    double* C = (double*)malloc(P * sizeof(double));
    oracle_gray(rgb, h, w, g);
    oracle_canny(g, h, w, lo, hi, E, NULL);
    if (global_norm) oracle_color_contrast_global(rgb, h, w, radius, sigma_ref_or_kappa, sigma_min, C);
    else oracle_color_contrast(rgb, h, w, radius, sigma_ref_or_kappa, C);
    int gh = h / patch, gw = w / patch;
    for (size_t i = 0; i < P; ++i) {
        double v = w_edge * E[i] + w_color * C[i];
        C[i] = v < 0.0 ? 0.0 : (v > 1.0 ? 1.0 : v);
    }
    for (int py = 0; py < gh; ++py)
        for (int px = 0; px < gw; ++px) {
            double acc = 0.0;
            for (int y = py * patch; y < (py + 1) * patch; ++y)
                for (int x = px * patch; x < (px + 1) * patch; ++x) acc += C[(size_t)y * w + x];
            s[py * gw + px] = acc / (double)(patch * patch);
        }
    if (S_or_null) memcpy(S_or_null, C, P * sizeof(double));
    free(C); free(E); free(g);
}

EXPORT void oracle_saliency(const uint8_t* rgb, int h, int w, int patch, int lo, int hi, int radius,
                            double sigma_ref, double w_edge, double w_color, double* s, double* S_or_null) {
    saliency_impl(rgb, h, w, patch, lo, hi, radius, 0, sigma_ref, 0.0, w_edge, w_color, s, S_or_null);
}

/* The same with the frame-adaptive colour term (kappa and sigma_min in place of sigma_ref). */
EXPORT void oracle_saliency_global(const uint8_t* rgb, int h, int w, int patch, int lo, int hi, int radius,
                                   double kappa, double sigma_min, double w_edge, double w_color, double* s,
                                   double* S_or_null) {
    saliency_impl(rgb, h, w, patch, lo, hi, radius, 1, kappa, sigma_min, w_edge, w_color, s, S_or_null);
}

EXPORT void oracle_saliency_batch(const uint8_t* frames, int B, int h, int w, int patch, int lo, int hi, int radius,
                                  double sigma_ref, double w_edge, double w_color, double* s) {
    size_t fb = (size_t)h * w * 3;
    int np = (h / patch) * (w / patch);
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b)
        oracle_saliency(frames + b * fb, h, w, patch, lo, hi, radius, sigma_ref, w_edge, w_color,
                        s + (size_t)b * np, NULL);
}

/* ------------------------------------------------------------------------- */
/* Decision rule for one frame (Eq. 6, Eq. 8, Alg. 1).  Scores are binary32.   */
/*   static_i = dP_i < tau_t (strict, Eq. 6);  R = count / N_tok (binary32);   */
/*   has_prev && R > theta_R  -> frame redundant: every token REUSE (Alg. 1    */
/*   lines 6-8), saliency not consulted;                                       */
/*   else, per token: patch_reuse && has_prev && static_i -> REUSE (reading:   */
/*   Fig. 3 counts skipped *patches*), else Eq. 8 as printed.                  */
/* Codes: 0 REUSE, 1 PRUNE, 2 INT4, 3 INT8, 4 FP16.  idx = [3][n_tok] lists    */
/* (FP16, INT8, INT4) of ascending token ids; counts[5] by code.               */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_select(const float* dP, const float* s, int n_tok, int has_prev, int patch_reuse, float tau_t,
                          float theta_R, float tau_high, float tau_med, float tau_low, uint8_t* decision,
                          int32_t* idx, int32_t* counts, uint8_t* frame_redundant, float* R_out) {
    int n_static = 0;
    if (has_prev)
        for (int i = 0; i < n_tok; ++i) n_static += (dP[i] < tau_t);
    float R = has_prev ? (float)n_static / (float)n_tok : 0.0f;
    int redundant = has_prev && (R > theta_R);
    for (int c = 0; c < 5; ++c) counts[c] = 0;
    int n16 = 0, n8 = 0, n4 = 0;
    for (int i = 0; i < n_tok; ++i) {
        uint8_t d;
        if (redundant) d = 0;
        else if (patch_reuse && has_prev && dP[i] < tau_t) d = 0;
        else if (s[i] > tau_high) d = 4;
        else if (s[i] > tau_med) d = 3;
        else if (s[i] > tau_low) d = 2;
        else d = 1;
        decision[i] = d;
        counts[d]++;
        if (d == 4) idx[0 * n_tok + n16++] = i;
        else if (d == 3) idx[1 * n_tok + n8++] = i;
        else if (d == 2) idx[2 * n_tok + n4++] = i;
    }
    for (int i = n16; i < n_tok; ++i) idx[0 * n_tok + i] = -1;
    for (int i = n8; i < n_tok; ++i) idx[1 * n_tok + i] = -1;
    for (int i = n4; i < n_tok; ++i) idx[2 * n_tok + i] = -1;
    *frame_redundant = (uint8_t)redundant;
    if (R_out) *R_out = R;
}

/* ------------------------------------------------------------------------- */
/* Adaptive tier thresholds (a variant: the paper's thresholds are fixed and it */
/* names their adaptation to the content as future work, Sec. V).  Reading: the */
/* temporal test is unchanged (Eq. 6, and patch reuse); among the tokens of a   */
/* frame that are not reused, the tiers of Eq. 8 are given out by rank of s_i   */
/* instead of by fixed thresholds, so that fixed shares of them are kept at     */
/* each precision whatever the frame's saliency level: with n_live such tokens, */
/*   q16 = (n_live * pm16 + 500) / 1000 (integer division), likewise q8, q4,     */
/*   each clipped to what is left of n_live;                                     */
/* the q16 most salient are FP16, the next q8 INT8, the next q4 INT4, the rest   */
/* pruned.  Ties in s go to the lower token id.  The thresholds of Eq. 8 thus     */
/* become order statistics of the frame's own scores.                            */
/* ------------------------------------------------------------------------- */
typedef struct { float s; int32_t i; } oracle_ranked_t;
static int oracle_ranked_cmp(const void* a, const void* b) {
    const oracle_ranked_t* x = (const oracle_ranked_t*)a;
    const oracle_ranked_t* y = (const oracle_ranked_t*)b;
    if (x->s > y->s) return -1;
    if (x->s < y->s) return 1;
    return x->i < y->i ? -1 : (x->i > y->i ? 1 : 0);
}
EXPORT void oracle_select_ranked(const float* dP, const float* s, int n_tok, int has_prev, int patch_reuse, float tau_t,
                                 float theta_R, int pm16, int pm8, int pm4, uint8_t* decision, int32_t* idx,
                                 int32_t* counts, uint8_t* frame_redundant) {
    int n_static = 0;
    if (has_prev)
        for (int i = 0; i < n_tok; ++i) n_static += (dP[i] < tau_t);
    float R = has_prev ? (float)n_static / (float)n_tok : 0.0f;
    int redundant = has_prev && (R > theta_R);
    oracle_ranked_t* live = (oracle_ranked_t*)malloc((size_t)n_tok * sizeof(oracle_ranked_t));
    int n_live = 0;
    for (int i = 0; i < n_tok; ++i) {
        if (redundant || (patch_reuse && has_prev && dP[i] < tau_t)) decision[i] = 0;
        else {
            live[n_live].s = s[i];
            live[n_live].i = i;
            ++n_live;
        }
    }
    qsort(live, (size_t)n_live, sizeof(oracle_ranked_t), oracle_ranked_cmp);
    long left = n_live;
    long q16 = ((long)n_live * pm16 + 500) / 1000; if (q16 > left) q16 = left; left -= q16;
    long q8 = ((long)n_live * pm8 + 500) / 1000;   if (q8 > left) q8 = left;   left -= q8;
    long q4 = ((long)n_live * pm4 + 500) / 1000;   if (q4 > left) q4 = left;
    for (int r = 0; r < n_live; ++r)
        decision[live[r].i] = r < q16 ? 4 : (r < q16 + q8 ? 3 : (r < q16 + q8 + q4 ? 2 : 1));
    free(live);
    for (int c = 0; c < 5; ++c) counts[c] = 0;
    int n16 = 0, n8 = 0, n4 = 0;
    for (int i = 0; i < n_tok; ++i) {
        uint8_t d = decision[i];
        counts[d]++;
        if (d == 4) idx[0 * n_tok + n16++] = i;
        else if (d == 3) idx[1 * n_tok + n8++] = i;
        else if (d == 2) idx[2 * n_tok + n4++] = i;
    }
    for (int i = n16; i < n_tok; ++i) idx[0 * n_tok + i] = -1;
    for (int i = n8; i < n_tok; ++i) idx[1 * n_tok + i] = -1;
    for (int i = n4; i < n_tok; ++i) idx[2 * n_tok + i] = -1;
    *frame_redundant = (uint8_t)redundant;
}

/* ------------------------------------------------------------------------- */
/* Anchor-frame mode of the temporal test (a variant: the paper compares        */
/* consecutive frames, Sec. III-A, which lets a slow pan or a slow fade stay    */
/* "static" forever because every single step is below tau_t).  Here token i of */
/* frame t is compared with the patch its cache entry was computed from: the    */
/* patch of the last frame in which token i was not REUSE (the frame Alg. 1's   */
/* pointer chain resolves to).  `anchor` is that composite image, [h][w][3],     */
/* read and updated in frame order:                                             */
/*   dP[t][i]  = Eq. 5 read literally between anchor and frame t (RMS grey-level */
/*               difference over patch i); 0 for a frame without predecessor;   */
/*   decisions = Eq. 6 / Eq. 8 on (dP[t], s[t]) exactly as oracle_select;        */
/*   anchor    <- frame t on every patch whose token is not REUSE.               */
/* The flow score is not used in this mode: each token has its own reference     */
/* frame, so it would need one flow field per (frame, anchor) pair.              */
/* Frames depend on their predecessors' decisions: a scan, not a map.            */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_select_anchored(const uint8_t* frames, const float* s, int T, int h, int w, int patch,
                                   int first_has_no_prev, int patch_reuse, float tau_t, float theta_R, float tau_high,
                                   float tau_med, float tau_low, uint8_t* anchor, float* dP, uint8_t* decision,
                                   int32_t* idx, int32_t* counts, uint8_t* frame_redundant) {
    int gw = w / patch, n_tok = (h / patch) * gw;
    size_t fb = (size_t)h * w * 3;
    double* d = (double*)malloc((size_t)n_tok * sizeof(double));
    for (int t = 0; t < T; ++t) {
        const uint8_t* f = frames + (size_t)t * fb;
        int has_prev = !(first_has_no_prev && t == 0);
        float* dp = dP + (size_t)t * n_tok;
        if (has_prev) {
            oracle_diff_score(anchor, f, h, w, patch, d);
            for (int i = 0; i < n_tok; ++i) dp[i] = (float)d[i];
        } else {
            for (int i = 0; i < n_tok; ++i) dp[i] = 0.0f;
        }
        uint8_t* dec = decision + (size_t)t * n_tok;
        oracle_select(dp, s + (size_t)t * n_tok, n_tok, has_prev, patch_reuse, tau_t, theta_R, tau_high, tau_med, tau_low,
                      dec, idx + (size_t)t * 3 * n_tok, counts + (size_t)t * 5, frame_redundant + t, NULL);
        for (int i = 0; i < n_tok; ++i) {
            if (dec[i] == 0) continue;
            int py = i / gw, px = i % gw;
            for (int y = py * patch; y < (py + 1) * patch; ++y)
                memcpy(anchor + ((size_t)y * w + (size_t)px * patch) * 3, f + ((size_t)y * w + (size_t)px * patch) * 3,
                       (size_t)patch * 3);
        }
    }
    free(d);
}

/* ------------------------------------------------------------------------- */
/* Source-frame table (Alg. 1 line 7: C[t] <- Pointer(C[t-1]); Fig. 3 counts    */
/* reuse per patch).  src[t][i] = src[t-1][i] when token i of frame t is REUSE, */
/* else t: every token names the frame whose entry it uses, chains resolved.   */
/* prev = sources of the frame before frame `first` (unused for tokens that do */
/* not reuse).                                                                 */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_source_frames(const uint8_t* decision, int T, int n_tok, int first, const int32_t* prev, int32_t* src) {
    for (int i = 0; i < n_tok; ++i)
        for (int t = 0; t < T; ++t) {
            int32_t before = t == 0 ? prev[i] : src[(size_t)(t - 1) * n_tok + i];
            src[(size_t)t * n_tok + i] = decision[(size_t)t * n_tok + i] == 0 ? before : first + t;
        }
}

/* ------------------------------------------------------------------------- */
/* binary16 <-> binary32, written out on the bits (round to nearest even).     */
/* ------------------------------------------------------------------------- */
EXPORT float oracle_half_to_float(uint16_t hbits) {
    int sign = (hbits >> 15) & 1, e = (hbits >> 10) & 31, mant = hbits & 1023;
    float v;
    if (e == 0) v = ldexpf((float)mant, -24);
    else if (e == 31) v = mant ? NAN : INFINITY;
    else v = ldexpf((float)(mant | 1024), e - 25);
    return sign ? -v : v;
}

EXPORT uint16_t oracle_float_to_half(float f) {
    uint32_t x;
    memcpy(&x, &f, 4);
    uint16_t sign = (uint16_t)((x >> 16) & 0x8000u);
    uint32_t a = x & 0x7fffffffu;
    if (a > 0x7f800000u) return (uint16_t)(sign | 0x7e00u);      /* NaN */
    if (a >= 0x477ff000u) return (uint16_t)(sign | 0x7c00u);     /* >= 65520 rounds to inf */
    if (a <= 0x33000000u) return sign;                           /* <= 2^-25 rounds to 0 */
    int e = (int)(a >> 23) - 127;
    uint32_t mant = (a & 0x7fffffu) | 0x800000u;                 /* 24-bit significand */
    int shift = e >= -14 ? 13 : 13 + (-14 - e);                  /* bits dropped */
    uint32_t kept = mant >> shift;
    uint32_t rem = mant & ((1u << shift) - 1u), half = 1u << (shift - 1);
    if (rem > half || (rem == half && (kept & 1u))) kept++;
    uint32_t out;
    if (e >= -14) out = ((uint32_t)(e + 14) << 10) + kept;        /* kept carries the implicit 1 (1<<10) */
    else out = kept;                                             /* subnormal; a carry lands on 2^-14 */
    return (uint16_t)(sign | out);
}

/* ------------------------------------------------------------------------- */
/* Quantisers (Sec. IV-B: symmetric min-max INT8, asymmetric INT4), one group  */
/* of G consecutive fp16 elements.  Reading of what the paper leaves open:     */
/* scale and zero are stored as fp16 and quantisation uses the STORED scale;   */
/* q = rint(x * (1/s)) with a multiply (not a divide, not an FMA), rint =      */
/* round half to even; a zero range takes s = 1.                               */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_quant_int8_group(const uint16_t* x, int G, int8_t* q, uint16_t* scale16) {
    float amax = 0.0f;
    for (int i = 0; i < G; ++i) {
        float v = fabsf(oracle_half_to_float(x[i]));
        if (v > amax) amax = v;
    }
    uint16_t s16 = oracle_float_to_half(amax / 127.0f);
    if ((s16 & 0x7fffu) == 0) s16 = 0x3c00u;
    float s = oracle_half_to_float(s16);
    float inv = 1.0f / s;
    for (int i = 0; i < G; ++i) {
        volatile float p = oracle_half_to_float(x[i]) * inv;
        float r = rintf(p);
        if (r > 127.0f) r = 127.0f;
        if (r < -127.0f) r = -127.0f;
        q[i] = (int8_t)r;
    }
    *scale16 = s16;
}

EXPORT void oracle_dequant_int8_group(const int8_t* q, int G, uint16_t scale16, uint16_t* xh) {
    float s = oracle_half_to_float(scale16);
    for (int i = 0; i < G; ++i) {
        volatile float p = (float)q[i] * s;
        xh[i] = oracle_float_to_half(p);
    }
}

/* INT4 asymmetric: s = fp16((max - min)/15), zero point = the group minimum    */
/* kept as fp16; q = clamp(rint((x - z) * (1/s)), 0, 15); element 2j in the    */
/* low nibble of byte j, 2j+1 in the high nibble.                              */
EXPORT void oracle_quant_int4_group(const uint16_t* x, int G, uint8_t* packed, uint16_t* scale16, uint16_t* zero16) {
    float mn = INFINITY, mx = -INFINITY;
    uint16_t mn16 = 0;
    for (int i = 0; i < G; ++i) {
        float v = oracle_half_to_float(x[i]);
        if (v < mn) { mn = v; mn16 = x[i]; }
        if (v > mx) mx = v;
    }
    if (mn == 0.0f) mn16 = 0; /* -0 and +0 compare equal: store +0 */
    volatile float range = mx - mn;
    uint16_t s16 = oracle_float_to_half(range / 15.0f);
    if ((s16 & 0x7fffu) == 0) s16 = 0x3c00u;
    float s = oracle_half_to_float(s16);
    float inv = 1.0f / s;
    float z = oracle_half_to_float(mn16);
    for (int i = 0; i < G; i += 2) {
        uint8_t qq[2];
        for (int j = 0; j < 2; ++j) {
            volatile float dlt = oracle_half_to_float(x[i + j]) - z;
            volatile float p = dlt * inv;
            float r = rintf(p);
            if (r > 15.0f) r = 15.0f;
            if (r < 0.0f) r = 0.0f;
            qq[j] = (uint8_t)r;
        }
        packed[i / 2] = (uint8_t)(qq[0] | (qq[1] << 4));
    }
    *scale16 = s16;
    *zero16 = mn16;
}

EXPORT void oracle_dequant_int4_group(const uint8_t* packed, int G, uint16_t scale16, uint16_t zero16, uint16_t* xh) {
    float s = oracle_half_to_float(scale16), z = oracle_half_to_float(zero16);
    for (int i = 0; i < G; ++i) {
        int q = (i & 1) ? (packed[i / 2] >> 4) : (packed[i / 2] & 15);
        volatile float p = (float)q * s;
        volatile float r = p + z;
        xh[i] = oracle_float_to_half(r);
    }
}

/* ------------------------------------------------------------------------- */
/* Mixed-precision store of one frame's K/V (Alg. 1 line 16).                  */
/* K, V: fp16 bits [L][n_tok][HD].  Pools (per tier, shared by all frames):    */
/*   fp16_pool  u16 [L][2][cap16][HD]                                          */
/*   int8_codes i8  [L][2][cap8][HD],   int8_scale u16 [L][2][cap8][HD/G]      */
/*   int4_codes u8  [L][2][cap4][HD/2], int4_sz    u16 [L][2][cap4][HD/G][2]   */
/* The j-th token of a tier list goes to row (off + j) mod cap of that tier    */
/* (ring != 0) or row off + j (ring == 0; rows past cap are dropped and the    */
/* return value is -1).  Index 0 of the second axis is K, 1 is V.              */
/* ------------------------------------------------------------------------- */
static int64_t pool_row(int64_t off, int64_t j, int64_t cap, int ring) {
    int64_t r = off + j;
    if (ring) return cap > 0 ? r % cap : -1;
    return r < cap ? r : -1;
}

EXPORT int oracle_pack_frame(const uint16_t* K, const uint16_t* V, int L, int n_tok, int HD, int G,
                             const int32_t* idx, const int32_t* counts, const int64_t* off, int ring,
                             uint16_t* fp16_pool, int64_t cap16, int8_t* int8_codes, uint16_t* int8_scale,
                             int64_t cap8, uint8_t* int4_codes, uint16_t* int4_sz, int64_t cap4) {
    int status = 0;
    int ng = HD / G;
    int n16 = counts[4], n8 = counts[3], n4 = counts[2];
#pragma omp parallel for schedule(static) reduction(min : status)
    for (int l = 0; l < L; ++l)
        for (int kv = 0; kv < 2; ++kv) {
            const uint16_t* src = (kv ? V : K) + (size_t)l * n_tok * HD;
            size_t plane = (size_t)l * 2 + kv;
            for (int j = 0; j < n16; ++j) {
                int64_t r = pool_row(off[0], j, cap16, ring);
                if (r < 0) { status = -1; continue; }
                memcpy(fp16_pool + (plane * cap16 + r) * HD, src + (size_t)idx[0 * n_tok + j] * HD, (size_t)HD * 2);
            }
            for (int j = 0; j < n8; ++j) {
                int64_t r = pool_row(off[1], j, cap8, ring);
                if (r < 0) { status = -1; continue; }
                const uint16_t* row = src + (size_t)idx[1 * n_tok + j] * HD;
                for (int g = 0; g < ng; ++g)
                    oracle_quant_int8_group(row + g * G, G, int8_codes + (plane * cap8 + r) * HD + g * G,
                                            int8_scale + (plane * cap8 + r) * ng + g);
            }
            for (int j = 0; j < n4; ++j) {
                int64_t r = pool_row(off[2], j, cap4, ring);
                if (r < 0) { status = -1; continue; }
                const uint16_t* row = src + (size_t)idx[2 * n_tok + j] * HD;
                for (int g = 0; g < ng; ++g)
                    oracle_quant_int4_group(row + g * G, G, int4_codes + (plane * cap4 + r) * (HD / 2) + g * (G / 2),
                                            int4_sz + ((plane * cap4 + r) * ng + g) * 2,
                                            int4_sz + ((plane * cap4 + r) * ng + g) * 2 + 1);
            }
        }
    return status;
}

/* ------------------------------------------------------------------------- */
/* Just-in-time dequantisation of one frame (Sec. III-C) into dense fp16       */
/* K^, V^ [L][n_tok][HD].  FP16 rows are bit copies.  PRUNE rows are zeroed    */
/* when zero_fill_pruned; REUSE rows are left untouched (the caller resolves   */
/* them through the source-frame table).                                       */
/* ------------------------------------------------------------------------- */
/* Ring pools under a budget: row r (absolute position) of a tier is still in the pool while          */
/* fill - cap <= r, fill being the tier's running fill (rows ever stored).  With fill_or_null given,  */
/* a row that has been overwritten since (oldest-first eviction) is not read: its output row is       */
/* zeroed and the return value is -9.                                                                 */
static int row_evicted(int64_t off, int64_t j, int64_t cap, int ring, const int64_t* fill_or_null, int tier) {
    return ring && fill_or_null && off + j < fill_or_null[tier] - cap;
}

EXPORT int oracle_unpack_frame(int L, int n_tok, int HD, int G, const int32_t* idx, const int32_t* counts,
                               const uint8_t* decision, const int64_t* off, int ring, const uint16_t* fp16_pool,
                               int64_t cap16, const int8_t* int8_codes, const uint16_t* int8_scale, int64_t cap8,
                               const uint8_t* int4_codes, const uint16_t* int4_sz, int64_t cap4,
                               int zero_fill_pruned, const int64_t* fill_or_null, uint16_t* K_out, uint16_t* V_out) {
    int status = 0;
    int ng = HD / G;
    int n16 = counts[4], n8 = counts[3], n4 = counts[2];
#pragma omp parallel for schedule(static) reduction(min : status)
    for (int l = 0; l < L; ++l)
        for (int kv = 0; kv < 2; ++kv) {
            uint16_t* dst = (kv ? V_out : K_out) + (size_t)l * n_tok * HD;
            size_t plane = (size_t)l * 2 + kv;
            for (int j = 0; j < n16; ++j) {
                int64_t r = pool_row(off[0], j, cap16, ring);
                if (r < 0) { status = -1; continue; }
                if (row_evicted(off[0], j, cap16, ring, fill_or_null, 0)) {
                    memset(dst + (size_t)idx[0 * n_tok + j] * HD, 0, (size_t)HD * 2);
                    status = -9;
                    continue;
                }
                memcpy(dst + (size_t)idx[0 * n_tok + j] * HD, fp16_pool + (plane * cap16 + r) * HD, (size_t)HD * 2);
            }
            for (int j = 0; j < n8; ++j) {
                int64_t r = pool_row(off[1], j, cap8, ring);
                if (r < 0) { status = -1; continue; }
                uint16_t* row = dst + (size_t)idx[1 * n_tok + j] * HD;
                if (row_evicted(off[1], j, cap8, ring, fill_or_null, 1)) { memset(row, 0, (size_t)HD * 2); status = -9; continue; }
                for (int g = 0; g < ng; ++g)
                    oracle_dequant_int8_group(int8_codes + (plane * cap8 + r) * HD + g * G, G,
                                              int8_scale[(plane * cap8 + r) * ng + g], row + g * G);
            }
            for (int j = 0; j < n4; ++j) {
                int64_t r = pool_row(off[2], j, cap4, ring);
                if (r < 0) { status = -1; continue; }
                uint16_t* row = dst + (size_t)idx[2 * n_tok + j] * HD;
                if (row_evicted(off[2], j, cap4, ring, fill_or_null, 2)) { memset(row, 0, (size_t)HD * 2); status = -9; continue; }
                for (int g = 0; g < ng; ++g)
                    oracle_dequant_int4_group(int4_codes + (plane * cap4 + r) * (HD / 2) + g * (G / 2), G,
                                              int4_sz[((plane * cap4 + r) * ng + g) * 2],
                                              int4_sz[((plane * cap4 + r) * ng + g) * 2 + 1], row + g * G);
            }
            if (zero_fill_pruned)
                for (int i = 0; i < n_tok; ++i)
                    if (decision[i] == 1) memset(dst + (size_t)i * HD, 0, (size_t)HD * 2);
        }
    return status;
}

/* ------------------------------------------------------------------------- */
/* Decode attention over the mixed-precision store with just-in-time           */
/* dequantisation (Eq. 2; Sec. III-C: dequantisation happens inside the        */
/* attention computation).  One query vector per layer and head; the keys and  */
/* values are the rows the store holds: rows [0, n16) of the FP16 pool, [0, n8)*/
/* of the INT8 pool, [0, n4) of the INT4 pool (pruned tokens have no row).     */
/*   score_j = q_h . K^_{j,h} / sqrt(D),  p = softmax_j(score),                */
/*   out_h   = sum_j p_j V^_{j,h}                                              */
/* with K^, V^ the dequantised values in exact arithmetic (q * s, q * s + z:   */
/* no rounding to binary16 in between, as in a fused kernel), everything in    */
/* double.  q: fp16 bits [L][H][D]; out: double [L][H][D]; zero rows -> zeros. */
/* ------------------------------------------------------------------------- */
static double pool_value(int tier, size_t prow, int h, int d, int HD, int D, int G, const uint16_t* fp16_pool,
                         const int8_t* int8_codes, const uint16_t* int8_scale, const uint8_t* int4_codes,
                         const uint16_t* int4_sz) {
    int e = h * D + d, ng = HD / G;
    if (tier == 0) return (double)oracle_half_to_float(fp16_pool[prow * HD + e]);
    if (tier == 1)
        return (double)int8_codes[prow * HD + e] * (double)oracle_half_to_float(int8_scale[prow * ng + e / G]);
    uint8_t byte = int4_codes[prow * (HD / 2) + e / 2];
    int q = (e & 1) ? (byte >> 4) : (byte & 15);
    return (double)q * (double)oracle_half_to_float(int4_sz[(prow * ng + e / G) * 2]) +
           (double)oracle_half_to_float(int4_sz[(prow * ng + e / G) * 2 + 1]);
}

EXPORT void oracle_attend(const uint16_t* q, int L, int H, int D, int G, const uint16_t* fp16_pool, int64_t cap16,
                          int64_t n16, const int8_t* int8_codes, const uint16_t* int8_scale, int64_t cap8, int64_t n8,
                          const uint8_t* int4_codes, const uint16_t* int4_sz, int64_t cap4, int64_t n4, double* out) {
    int HD = H * D;
    int64_t caps[3] = {cap16, cap8, cap4}, ns[3] = {n16, n8, n4};
    int64_t R = n16 + n8 + n4;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int l = 0; l < L; ++l)
        for (int h = 0; h < H; ++h) {
            double* o = out + ((size_t)l * H + h) * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            if (R == 0) continue;
            double* sc = (double*)malloc((size_t)R * sizeof(double));
            double mx = -INFINITY;
            int64_t j = 0;
            for (int t = 0; t < 3; ++t)
                for (int64_t r = 0; r < ns[t]; ++r, ++j) {
                    size_t prow = (size_t)(2 * l) * caps[t] + r;            /* K plane of layer l */
                    double dot = 0.0;
                    for (int d = 0; d < D; ++d)
                        dot += (double)oracle_half_to_float(q[((size_t)l * H + h) * D + d]) *
                               pool_value(t, prow, h, d, HD, D, G, fp16_pool, int8_codes, int8_scale, int4_codes, int4_sz);
                    sc[j] = dot / sqrt((double)D);
                    if (sc[j] > mx) mx = sc[j];
                }
            double den = 0.0;
            for (j = 0; j < R; ++j) { sc[j] = exp(sc[j] - mx); den += sc[j]; }
            j = 0;
            for (int t = 0; t < 3; ++t)
                for (int64_t r = 0; r < ns[t]; ++r, ++j) {
                    size_t prow = (size_t)(2 * l + 1) * caps[t] + r;        /* V plane */
                    double p = sc[j] / den;
                    for (int d = 0; d < D; ++d)
                        o[d] += p * pool_value(t, prow, h, d, HD, D, G, fp16_pool, int8_codes, int8_scale, int4_codes, int4_sz);
                }
            free(sc);
        }
}

/* Grouped-query form (the paper's evaluation model, LLaVA-1.6 Mistral-7B, has 8 key/value heads serving 32 query   */
/* heads, Sec. IV-A): query head hq attends to the rows of key/value head hq / q_per_kv; everything else as above.   */
/* q, out: [L][H * q_per_kv][D].                                                                                     */
EXPORT void oracle_attend_gqa(const uint16_t* q, int L, int H, int q_per_kv, int D, int G, const uint16_t* fp16_pool,
                              int64_t cap16, int64_t n16, const int8_t* int8_codes, const uint16_t* int8_scale, int64_t cap8,
                              int64_t n8, const uint8_t* int4_codes, const uint16_t* int4_sz, int64_t cap4, int64_t n4,
                              double* out) {
    int HD = H * D, HQ = H * q_per_kv;
    int64_t caps[3] = {cap16, cap8, cap4}, ns[3] = {n16, n8, n4};
    int64_t R = n16 + n8 + n4;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int l = 0; l < L; ++l)
        for (int hq = 0; hq < HQ; ++hq) {
            int h = hq / q_per_kv;
            const uint16_t* qv = q + ((size_t)l * HQ + hq) * D;
            double* o = out + ((size_t)l * HQ + hq) * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            if (R == 0) continue;
            double* sc = (double*)malloc((size_t)R * sizeof(double));
            double mx = -INFINITY;
            int64_t j = 0;
            for (int t = 0; t < 3; ++t)
                for (int64_t r = 0; r < ns[t]; ++r, ++j) {
                    size_t prow = (size_t)(2 * l) * caps[t] + r;
                    double dot = 0.0;
                    for (int d = 0; d < D; ++d)
                        dot += (double)oracle_half_to_float(qv[d]) *
                               pool_value(t, prow, h, d, HD, D, G, fp16_pool, int8_codes, int8_scale, int4_codes, int4_sz);
                    sc[j] = dot / sqrt((double)D);
                    if (sc[j] > mx) mx = sc[j];
                }
            double den = 0.0;
            for (j = 0; j < R; ++j) { sc[j] = exp(sc[j] - mx); den += sc[j]; }
            j = 0;
            for (int t = 0; t < 3; ++t)
                for (int64_t r = 0; r < ns[t]; ++r, ++j) {
                    size_t prow = (size_t)(2 * l + 1) * caps[t] + r;
                    double p = sc[j] / den;
                    for (int d = 0; d < D; ++d)
                        o[d] += p * pool_value(t, prow, h, d, HD, D, G, fp16_pool, int8_codes, int8_scale, int4_codes, int4_sz);
                }
            free(sc);
        }
}

/* ------------------------------------------------------------------------- */
/* Token order of a dynamic-resolution frame (Sec. II-A mentions the encoding  */
/* only; reading): a frame of 2x2 tiles of tg x tg patches plus one base image */
/* of tg x tg patches has (1 + 4) tg^2 tokens: the base image first, then tile */
/* (0,0), (0,1), (1,0), (1,1), each row-major.  full = per-patch values on the */
/* (2 tg) x (2 tg) grid of the whole frame (row-major), base = on the base     */
/* image's grid.                                                               */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_anyres_tokens(const double* full, const double* base, int tg, double* out) {
    int k = 0;
    for (int i = 0; i < tg * tg; ++i) out[k++] = base[i];
    for (int r = 0; r < 2; ++r)
        for (int c = 0; c < 2; ++c)
            for (int y = 0; y < tg; ++y)
                for (int x = 0; x < tg; ++x) out[k++] = full[(size_t)(r * tg + y) * (2 * tg) + (c * tg + x)];
}

/* ------------------------------------------------------------------------- */
/* Pool rows of a run of frames (the store step of Alg. 1, line 16): frame t's */
/* rows of a tier follow those of the frames before it, so its first row is    */
/* the running fill of that tier; the fill then grows by the frame's count.    */
/* counts [T][5] by code; off [T][3] and fill [3] in the order FP16, INT8,     */
/* INT4.  Offsets are absolute: a ring pool takes them modulo its capacity.    */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_row_offsets(const int32_t* counts, int T, int64_t* fill, int64_t* off) {
    const int code[3] = {4, 3, 2};
    for (int t = 0; t < T; ++t)
        for (int k = 0; k < 3; ++k) {
            off[(size_t)t * 3 + k] = fill[k];
            fill[k] += counts[(size_t)t * 5 + code[k]];
        }
}

/* ------------------------------------------------------------------------- */
/* Memory accounting (Eq. 3: M = 2 n_l L d sizeof(dtype), applied per tier).   */
/* raw: T frames of n_tok tokens, K and V, L layers, HD = heads x head_dim     */
/* fp16 elements per token.  stored: the pools' payload for the per-code       */
/* counts [T][5] (FP16 rows 2 HD bytes, INT8 rows HD + 2 HD/G, INT4 rows       */
/* HD/2 + 4 HD/G per layer and tensor) plus the metadata kept per frame (one   */
/* decision byte per token, an 8-byte pointer-table entry, three 8-byte row    */
/* offsets, five 4-byte counts) and a 4-byte index-list entry per stored token.*/
/* ------------------------------------------------------------------------- */
EXPORT int64_t oracle_raw_bytes(int64_t T, int L, int HD, int n_tok) { return 2 * (int64_t)L * T * n_tok * HD * 2; }

EXPORT int64_t oracle_stored_bytes(const int64_t* counts, int64_t T, int L, int HD, int G, int n_tok) {
    int64_t n4 = 0, n8 = 0, n16 = 0, ng = HD / G;
    for (int64_t t = 0; t < T; ++t) {
        n4 += counts[t * 5 + 2];
        n8 += counts[t * 5 + 3];
        n16 += counts[t * 5 + 4];
    }
    int64_t payload = (int64_t)L * 2 * (n16 * HD * 2 + n8 * (HD + 2 * ng) + n4 * (HD / 2 + 4 * ng));
    int64_t meta = T * ((int64_t)n_tok + 8 + 24 + 20) + 4 * (n4 + n8 + n16);
    return payload + meta;
}

/* ------------------------------------------------------------------------- */
/* Which stored frames a budgeted cache still holds (the paper runs its        */
/* baselines under a fixed memory budget, Sec. IV-A; reading for this store:   */
/* per-tier ring pools, oldest rows overwritten first).  Frame t is resident   */
/* in tier k when it stored no row there, or when its first row has not been   */
/* overwritten and the frame fits the ring at all:                             */
/*   n_tk == 0  or  (n_tk <= cap_k and off_tk >= fill_k - cap_k)               */
/* (linear pools, ring == 0: off_tk + n_tk <= cap_k).  A frame's record is     */
/* evicted as a whole: resident[t] = 1 only if that holds in all three tiers.  */
/* counts [T][5] by code, off [T][3] / cap [3] / fill [3] in the order FP16,   */
/* INT8, INT4.                                                                 */
/* ------------------------------------------------------------------------- */
EXPORT void oracle_frames_resident(const int32_t* counts, const int64_t* off, int T, const int64_t* cap, int ring,
                                   const int64_t* fill, uint8_t* resident) {
    const int code[3] = {4, 3, 2};
    for (int t = 0; t < T; ++t) {
        int ok = 1;
        for (int k = 0; k < 3; ++k) {
            int64_t n = counts[(size_t)t * 5 + code[k]], o = off[(size_t)t * 3 + k];
            if (n == 0) continue;
            if (ring) ok = ok && n <= cap[k] && o >= fill[k] - cap[k];
            else ok = ok && o + n <= cap[k];
        }
        resident[t] = (uint8_t)ok;
    }
}

/* A reused token lives as long as the frame that holds its entry: live[t][i] = */
/* resident[src[t][i] - first] (0 when the source frame precedes the table),    */
/* src being the source-frame table of oracle_source_frames: a root is evicted  */
/* together with every alias that points to it.  Pruned tokens have no entry;   */
/* they are reported live when their own frame is resident.                      */
EXPORT void oracle_tokens_live(const int32_t* src, int T, int n_tok, int first, const uint8_t* resident, int n_table,
                               uint8_t* live) {
    for (size_t i = 0; i < (size_t)T * n_tok; ++i) {
        int64_t k = (int64_t)src[i] - first;
        live[i] = (k >= 0 && k < n_table) ? resident[k] : 0;
    }
}
