// Temporal branch (Sec. III-A, Eq. 5): gray pyramid, polynomial expansion, coarse-to-fine
// displacement updates and the per-patch RMS flow magnitude.  Arithmetic in double.
#include <math.h>

#include "common.cuh"

namespace {

__device__ __forceinline__ int clampi(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }

// ---- level 0: integer luma g = (77R + 150G + 29B + 128) >> 8 as float; 16 pixels per thread,
// three 16-byte loads of the interleaved RGB bytes.
__global__ void k_gray(const uint8_t* __restrict__ frames, size_t frame_bytes, int n_px, int n_frames,
                       float* __restrict__ out) {
    int groups = n_px / 16;
    long long gid = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (gid >= (long long)groups * n_frames) return;
    int f = (int)(gid / groups), gidx = (int)(gid % groups);
    const uint4* src = reinterpret_cast<const uint4*>(frames + (size_t)f * frame_bytes) + (size_t)gidx * 3;
    uint4 v0 = __ldg(src), v1 = __ldg(src + 1), v2 = __ldg(src + 2);
    uint32_t w[12] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w, v2.x, v2.y, v2.z, v2.w};
    float* dst = out + (size_t)f * n_px + (size_t)gidx * 16;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        int b0 = 3 * i, b1 = b0 + 1, b2 = b0 + 2;
        int R = (w[b0 >> 2] >> ((b0 & 3) * 8)) & 255;
        int G = (w[b1 >> 2] >> ((b1 & 3) * 8)) & 255;
        int Bc = (w[b2 >> 2] >> ((b2 & 3) * 8)) & 255;
        dst[i] = (float)((77 * R + 150 * G + 29 * Bc + 128) >> 8);
    }
}

// ---- half-scale level: 5x5 binomial [1 4 6 4 1]/16 sampled at (2y, 2x), clamp-to-edge.  Level values are
// dyadic rationals with at most 24 significant bits, so float holds them exactly.
__global__ void k_pyr_down(const float* __restrict__ src, int h, int w, int n_frames, float* __restrict__ dst) {
    int h2 = h / 2, w2 = w / 2;
    long long gid = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (gid >= (long long)h2 * w2 * n_frames) return;
    int f = (int)(gid / (h2 * w2)), r = (int)(gid % (h2 * w2));
    int y = r / w2, x = r % w2;
    const float* s = src + (size_t)f * h * w;
    const float k[5] = {1.f, 4.f, 6.f, 4.f, 1.f};
    float acc = 0.f;
#pragma unroll
    for (int a = -2; a <= 2; ++a) {
        const float* row = s + (size_t)clampi(2 * y + a, 0, h - 1) * w;
        float ra = 0.f;
#pragma unroll
        for (int b = -2; b <= 2; ++b) ra += k[b + 2] * row[clampi(2 * x + b, 0, w - 1)];
        acc += k[a + 2] * ra;
    }
    dst[(size_t)f * h2 * w2 + r] = acc * (1.0f / 256.0f);
}

struct PolyW {
    double g[5];     // normalised Gaussian applicability
    double inv_mu2, inv_mu2sq, inv_den, mu2;
};

// ---- polynomial expansion, 5x5: planes r2 r3 r4 r5 r6 (b_x, b_y, A_xx, A_yy, 2 A_xy).
__global__ void k_poly_exp(const float* __restrict__ img, int h, int w, int n_frames, PolyW pw,
                           double* __restrict__ coef) {
    long long gid = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    size_t P = (size_t)h * w;
    if (gid >= (long long)P * n_frames) return;
    int f = (int)(gid / P);
    int r = (int)(gid % P);
    int y = r / w, x = r % w;
    const float* s = img + (size_t)f * P;
    int xs[5];
#pragma unroll
    for (int b = 0; b < 5; ++b) xs[b] = clampi(x + b - 2, 0, w - 1);
    double m00 = 0, m10 = 0, m01 = 0, m20 = 0, m02 = 0, m11 = 0;
#pragma unroll
    for (int a = -2; a <= 2; ++a) {
        const float* row = s + (size_t)clampi(y + a, 0, h - 1) * w;
        double s0 = 0, s1 = 0, s2 = 0;
#pragma unroll
        for (int b = -2; b <= 2; ++b) {
            double v = pw.g[b + 2] * (double)row[xs[b + 2]];
            s0 += v;
            s1 += v * b;
            s2 += v * (b * b);
        }
        double ga = pw.g[a + 2];
        m00 += ga * s0;
        m10 += ga * s1;
        m20 += ga * s2;
        m01 += ga * a * s0;
        m11 += ga * a * s1;
        m02 += ga * (a * a) * s0;
    }
    double* c = coef + (size_t)f * 5 * P + r;
    c[0 * P] = m10 * pw.inv_mu2;
    c[1 * P] = m01 * pw.inv_mu2;
    c[2 * P] = (m20 - pw.mu2 * m00) * pw.inv_den;
    c[3 * P] = (m02 - pw.mu2 * m00) * pw.inv_den;
    c[4 * P] = m11 * pw.inv_mu2sq;
}

// Bilinear corner set of a clamped continuous position.
struct Bilin {
    int i00, i01, i10, i11;
    double fx, fy;
};
__device__ __forceinline__ Bilin bilin_at(double y, double x, int h, int w) {
    x = fmin(fmax(x, 0.0), (double)(w - 1));
    y = fmin(fmax(y, 0.0), (double)(h - 1));
    int x0 = (int)floor(x), y0 = (int)floor(y);
    int x1 = min(x0 + 1, w - 1), y1 = min(y0 + 1, h - 1);
    Bilin b;
    b.fx = x - x0;
    b.fy = y - y0;
    b.i00 = y0 * w + x0;
    b.i01 = y0 * w + x1;
    b.i10 = y1 * w + x0;
    b.i11 = y1 * w + x1;
    return b;
}
__device__ __forceinline__ double bilin_fetch(const double* __restrict__ p, const Bilin& b) {
    double top = p[b.i00] * (1.0 - b.fx) + p[b.i01] * b.fx;
    double bot = p[b.i10] * (1.0 - b.fx) + p[b.i11] * b.fx;
    return top * (1.0 - b.fy) + bot * b.fy;
}

// ---- coarse-to-fine transfer: d_fine = 2 * bilinear(d_coarse) at ((x+1/2)/2 - 1/2, (y+1/2)/2 - 1/2).
__global__ void k_flow_upsample(const double* __restrict__ dc, int hc, int wc, double* __restrict__ df, int hf, int wf,
                                int n_pairs, size_t stride_c, size_t stride_f) {
    long long gid = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    size_t Pf = (size_t)hf * wf, Pc = (size_t)hc * wc;
    if (gid >= (long long)Pf * n_pairs) return;
    int f = (int)(gid / Pf), r = (int)(gid % Pf);
    int y = r / wf, x = r % wf;
    Bilin b = bilin_at((y + 0.5) * 0.5 - 0.5, (x + 0.5) * 0.5 - 0.5, hc, wc);
    const double* c = dc + (size_t)f * stride_c;
    double* o = df + (size_t)f * stride_f;
    o[r] = 2.0 * bilin_fetch(c, b);
    o[Pf + r] = 2.0 * bilin_fetch(c + Pc, b);
}

// ---- one displacement update (Farneback's estimate with a prior d~), one 32x32 tile per CTA.
// Phase 1: G = A^T A and h = A^T db at every in-image pixel of the tile grown by the 7-pixel window
// radius (zero outside the image: the box sum runs over the in-image part of the window only).
// Phase 2: 15-tap horizontal sums.  Phase 3: 15-tap vertical sums, 2x2 solve with det + eps.
constexpr int FT = 32;            // tile side
constexpr int FR = 7;             // window radius (window 15)
constexpr int FE = FT + 2 * FR;   // 46
constexpr int FEP = FE + 1;       // padded row
constexpr int FLOW_THREADS = 512;

__global__ void __launch_bounds__(FLOW_THREADS)
k_flow_iter(const double* __restrict__ coef1, const double* __restrict__ coef2, size_t coef_stride, int h, int w,
            const double* __restrict__ d_in, double* __restrict__ d_out, size_t flow_stride, int zero_prior,
            double eps) {
    extern __shared__ double sm[];
    double* T = sm;                          // [5][FE][FEP]
    double* Hs = sm + 5 * FE * FEP;          // [5][FE][FT]
    const int f = blockIdx.z;
    const int x0 = blockIdx.x * FT, y0 = blockIdx.y * FT;
    const size_t P = (size_t)h * w;
    const double* c1 = coef1 + (size_t)f * coef_stride;
    const double* c2 = coef2 + (size_t)f * coef_stride;
    const double* din = d_in + (size_t)f * flow_stride;
    for (int i = threadIdx.x; i < FE * FE; i += FLOW_THREADS) {
        int ry = i / FE, rx = i % FE;
        int y = y0 - FR + ry, x = x0 - FR + rx;
        double g11 = 0, g12 = 0, g22 = 0, h1 = 0, h2 = 0;
        if (y >= 0 && y < h && x >= 0 && x < w) {
            int p = y * w + x;
            double du = 0.0, dv = 0.0;
            if (!zero_prior) { du = din[p]; dv = din[P + p]; }
            Bilin b = bilin_at(y + dv, x + du, h, w);
            double b2x = bilin_fetch(c2, b), b2y = bilin_fetch(c2 + P, b);
            double a2xx = bilin_fetch(c2 + 2 * P, b), a2yy = bilin_fetch(c2 + 3 * P, b);
            double a2xy = 0.5 * bilin_fetch(c2 + 4 * P, b);
            double axx = 0.5 * (c1[2 * P + p] + a2xx);
            double ayy = 0.5 * (c1[3 * P + p] + a2yy);
            double axy = 0.5 * (0.5 * c1[4 * P + p] + a2xy);
            double dbx = -0.5 * (b2x - c1[p]) + (axx * du + axy * dv);
            double dby = -0.5 * (b2y - c1[P + p]) + (axy * du + ayy * dv);
            g11 = axx * axx + axy * axy;
            g12 = axx * axy + axy * ayy;
            g22 = axy * axy + ayy * ayy;
            h1 = axx * dbx + axy * dby;
            h2 = axy * dbx + ayy * dby;
        }
        int o = ry * FEP + rx;
        T[0 * FE * FEP + o] = g11;
        T[1 * FE * FEP + o] = g12;
        T[2 * FE * FEP + o] = g22;
        T[3 * FE * FEP + o] = h1;
        T[4 * FE * FEP + o] = h2;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 5 * FE * FT; i += FLOW_THREADS) {
        int c = i / (FE * FT), r = i % (FE * FT);
        int ry = r / FT, ox = r % FT;
        const double* row = T + c * FE * FEP + ry * FEP + ox;
        double s = 0.0;
#pragma unroll
        for (int k = 0; k < 2 * FR + 1; ++k) s += row[k];
        Hs[i] = s;
    }
    __syncthreads();
    double* dout = d_out + (size_t)f * flow_stride;
    for (int i = threadIdx.x; i < FT * FT; i += FLOW_THREADS) {
        int oy = i / FT, ox = i % FT;
        int y = y0 + oy, x = x0 + ox;
        if (y >= h || x >= w) continue;
        double s[5];
#pragma unroll
        for (int c = 0; c < 5; ++c) {
            const double* col = Hs + c * FE * FT + oy * FT + ox;
            double a = 0.0;
#pragma unroll
            for (int k = 0; k < 2 * FR + 1; ++k) a += col[k * FT];
            s[c] = a;
        }
        double det = s[0] * s[2] - s[1] * s[1] + eps;
        int p = y * w + x;
        dout[p] = (s[2] * s[3] - s[1] * s[4]) / det;
        dout[P + p] = (s[0] * s[4] - s[1] * s[3]) / det;
    }
}

// ---- Eq. 5 (flow reading): dP_i = sqrt(mean over the patch of u^2 + v^2); one warp per patch.
__global__ void k_delta_p(const double* __restrict__ flow, size_t flow_stride, PlaneGeom g, int patch, int n_pairs,
                          float* __restrict__ dP) {
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    int np = g.gh * g.gw;
    if (warp >= np * n_pairs) return;
    int f = warp / np, pi = warp % np;
    int py = pi / g.gw, px = pi % g.gw;
    size_t P = (size_t)g.H * g.W;
    const double* u = flow + (size_t)f * flow_stride;
    double acc = 0.0;
    for (int i = lane; i < patch * patch; i += 32) {
        int y = py * patch + i / patch, x = px * patch + i % patch;
        double a = u[(size_t)y * g.W + x], b = u[P + (size_t)y * g.W + x];
        acc += a * a + b * b;
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) dP[(size_t)f * g.n_tok + patch_token(g, py, px)] = (float)sqrt(acc / (double)(patch * patch));
}

inline unsigned blocks_for(long long n, int threads) { return (unsigned)((n + threads - 1) / threads); }

}  // namespace

size_t sc_flow_iter_smem() { return (size_t)(5 * FE * FEP + 5 * FE * FT) * sizeof(double); }

int sc_flow_init() {
    SC_CHECK(cudaFuncSetAttribute(k_flow_iter, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sc_flow_iter_smem()));
    return SALICACHE_OK;
}

int sc_flow_score(salicache_ctx* c, const PlaneGeom& g, const uint8_t* d_prev, const uint8_t* d_cur, size_t frame_bytes,
                  int B, bool sequence, float* d_deltaP, double* d_flow_or_null, cudaStream_t st) {
    const salicache_params& p = c->p;
    PolyW pw;
    {
        double Z = 0, mu2 = 0, mu4 = 0;
        for (int k = -2; k <= 2; ++k) { pw.g[k + 2] = exp(-(double)(k * k) / (2.0 * p.poly_sigma * p.poly_sigma)); Z += pw.g[k + 2]; }
        for (int k = -2; k <= 2; ++k) {
            pw.g[k + 2] /= Z;
            mu2 += pw.g[k + 2] * k * k;
            mu4 += pw.g[k + 2] * k * k * (double)(k * k);
        }
        pw.mu2 = mu2;
        pw.inv_mu2 = 1.0 / mu2;
        pw.inv_mu2sq = 1.0 / (mu2 * mu2);
        pw.inv_den = 1.0 / (mu4 - mu2 * mu2);
    }
    const int T = 256;
    int hs[3], ws[3];
    for (int l = 0; l < 3; ++l) { hs[l] = g.H >> l; ws[l] = g.W >> l; }
    const size_t P0 = (size_t)g.H * g.W;
    for (int b0 = 0; b0 < B; b0 += c->chunk) {
        int nb = B - b0 < c->chunk ? B - b0 : c->chunk;    // pairs in this pass
        // frames to expand: a video shares frame b+1 between pairs b and b+1
        int nf = sequence ? nb + 1 : 2 * nb;
        // slot s of the scratch holds: sequence -> frame b0+s ; otherwise slots [0,nb) = prev, [nb,2nb) = cur
        for (int part = 0; part < (sequence ? 1 : 2); ++part) {
            const uint8_t* src = (part == 0 ? d_prev : d_cur) + (size_t)b0 * frame_bytes;
            int n = sequence ? nf : nb;
            float* dst = c->pyr[0] + (size_t)part * nb * P0;
            k_gray<<<blocks_for((long long)(P0 / 16) * n, T), T, 0, st>>>(src, frame_bytes, (int)P0, n, dst);
            c->launches++;
        }
        c->launches += 6;   // two pyramid levels, three expansions
        for (int l = 1; l < 3; ++l)
            k_pyr_down<<<blocks_for((long long)hs[l] * ws[l] * nf, T), T, 0, st>>>(c->pyr[l - 1], hs[l - 1], ws[l - 1], nf,
                                                                                   c->pyr[l]);
        for (int l = 0; l < 3; ++l)
            k_poly_exp<<<blocks_for((long long)hs[l] * ws[l] * nf, T), T, 0, st>>>(c->pyr[l], hs[l], ws[l], nf, pw,
                                                                                   c->coef[l]);
        double* cur = c->flow_a;
        double* nxt = c->flow_b;
        for (int l = 2; l >= 0; --l) {
            size_t Pl = (size_t)hs[l] * ws[l];
            size_t cstride = 5 * Pl;
            const double* c1 = c->coef[l];
            const double* c2 = c->coef[l] + (sequence ? cstride : (size_t)nb * cstride);
            if (l < 2) {
                k_flow_upsample<<<blocks_for((long long)Pl * nb, T), T, 0, st>>>(cur, hs[l + 1], ws[l + 1], nxt, hs[l],
                                                                                 ws[l], nb, 2 * P0, 2 * P0);
                double* t = cur; cur = nxt; nxt = t;
                c->launches++;
            }
            dim3 grid((ws[l] + FT - 1) / FT, (hs[l] + FT - 1) / FT, nb);
            for (int it = 0; it < p.iters; ++it) {
                int zero_prior = (l == 2 && it == 0);
                double* out = nxt;
                size_t ostride = 2 * P0;
                if (l == 0 && it == p.iters - 1 && d_flow_or_null) { out = d_flow_or_null + (size_t)b0 * 2 * P0; }
                k_flow_iter<<<grid, FLOW_THREADS, sc_flow_iter_smem(), st>>>(c1, c2, cstride, hs[l], ws[l], cur, out,
                                                                             ostride, zero_prior, p.eps_det);
                c->launches++;
                if (out == nxt) { double* t = cur; cur = nxt; nxt = t; }
                else cur = out;
            }
        }
        int np = g.gh * g.gw;
        const double* fin = cur;
        k_delta_p<<<blocks_for((long long)np * nb * 32, T), T, 0, st>>>(fin, 2 * P0, g, p.patch, nb,
                                                                        d_deltaP + (size_t)b0 * g.n_tok);
        c->launches++;
    }
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}
