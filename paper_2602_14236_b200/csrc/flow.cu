// Temporal branch (Sec. III-A, Eq. 5): gray pyramid, polynomial expansion, coarse-to-fine
// displacement updates and the per-patch RMS flow magnitude.
//
// Arithmetic is double; only storage is single precision where that provably costs nothing or very
// little: pyramid levels are exact in float, expansion coefficients and the per-pixel normal-equation
// terms (G, h) are rounded to float between kernels (their effect on dP stays below 1 % of the 1e-4
// relative tolerance on every workload; the cancellation b2(x~) - b1(x) itself is done in double).
//
// One displacement update = box sums of (G, h) over the 15x15 window + a 2x2 solve.  k_flow_box does
// that on a 28x28 tile (2x2 patches) with a double-precision integral image of the tile grown by the
// window radius, and, fused behind the solve, the (G, h) of the NEXT update at the same pixels (which
// needs no halo), or the patch scores after the last update.
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
    float4* dst = reinterpret_cast<float4*>(out + (size_t)f * n_px + (size_t)gidx * 16);
    float o[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        int b0 = 3 * i, b1 = b0 + 1, b2 = b0 + 2;
        int R = (w[b0 >> 2] >> ((b0 & 3) * 8)) & 255;
        int G = (w[b1 >> 2] >> ((b1 & 3) * 8)) & 255;
        int Bc = (w[b2 >> 2] >> ((b2 & 3) * 8)) & 255;
        o[i] = (float)((77 * R + 150 * G + 29 * Bc + 128) >> 8);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) dst[i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
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

// ---- polynomial expansion, 5x5: planes r2 r3 r4 r5 r6 (b_x, b_y, A_xx, A_yy, 2 A_xy), stored as float.
__global__ void k_poly_exp(const float* __restrict__ img, int h, int w, int n_frames, PolyW pw,
                           float* __restrict__ coef) {
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
    float* c = coef + (size_t)f * 5 * P + r;
    c[0 * P] = (float)(m10 * pw.inv_mu2);
    c[1 * P] = (float)(m01 * pw.inv_mu2);
    c[2 * P] = (float)((m20 - pw.mu2 * m00) * pw.inv_den);
    c[3 * P] = (float)((m02 - pw.mu2 * m00) * pw.inv_den);
    c[4 * P] = (float)(m11 * pw.inv_mu2sq);
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
template <typename T>
__device__ __forceinline__ double bilin_fetch(const T* __restrict__ p, const Bilin& b) {
    double top = (double)p[b.i00] * (1.0 - b.fx) + (double)p[b.i01] * b.fx;
    double bot = (double)p[b.i10] * (1.0 - b.fx) + (double)p[b.i11] * b.fx;
    return top * (1.0 - b.fy) + bot * b.fy;
}

// Normal-equation terms of one pixel for the prior (du, dv): G = A^T A (g11 g12 g22), hv = A^T db,
//   A = (A1(x) + A2(x~))/2,  db = -(b2(x~) - b1(x))/2 + A d~,  x~ = clamp(x + d~), bilinear fetch.
__device__ __forceinline__ void normal_terms(const float* __restrict__ c1, const float* __restrict__ c2, size_t P,
                                             int h, int w, int y, int x, double du, double dv, double out[5]) {
    const int p = y * w + x;
    Bilin b = bilin_at(y + dv, x + du, h, w);
    double b2x = bilin_fetch(c2, b), b2y = bilin_fetch(c2 + P, b);
    double a2xx = bilin_fetch(c2 + 2 * P, b), a2yy = bilin_fetch(c2 + 3 * P, b);
    double a2xy = 0.5 * bilin_fetch(c2 + 4 * P, b);
    double axx = 0.5 * ((double)c1[2 * P + p] + a2xx);
    double ayy = 0.5 * ((double)c1[3 * P + p] + a2yy);
    double axy = 0.5 * (0.5 * (double)c1[4 * P + p] + a2xy);
    double dbx = -0.5 * (b2x - (double)c1[p]) + (axx * du + axy * dv);
    double dby = -0.5 * (b2y - (double)c1[P + p]) + (axy * du + ayy * dv);
    out[0] = axx * axx + axy * axy;
    out[1] = axx * axy + axy * ayy;
    out[2] = axy * axy + ayy * ayy;
    out[3] = axx * dbx + axy * dby;
    out[4] = axy * dbx + ayy * dby;
}

// ---- (G, h) of the first update of a level.  Prior: zero at the coarsest level, else the coarser
// level's field carried over as d = 2 * bilinear(d_coarse) at ((x+1/2)/2 - 1/2, (y+1/2)/2 - 1/2).
__global__ void __launch_bounds__(256)
k_flow_gh(const float* __restrict__ coef1, const float* __restrict__ coef2, size_t coef_stride, int h, int w,
          const double* __restrict__ d_coarse, size_t flow_stride, float* __restrict__ gh, size_t gh_stride,
          int n_pairs) {
    const size_t P = (size_t)h * w;
    long long gid = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (gid >= (long long)P * n_pairs) return;
    const int f = (int)(gid / P), r = (int)(gid % P);
    const int y = r / w, x = r % w;
    double du = 0.0, dv = 0.0;
    if (d_coarse) {
        const int hc = h / 2, wc = w / 2;
        Bilin b = bilin_at((y + 0.5) * 0.5 - 0.5, (x + 0.5) * 0.5 - 0.5, hc, wc);
        const double* c = d_coarse + (size_t)f * flow_stride;
        du = 2.0 * bilin_fetch(c, b);
        dv = 2.0 * bilin_fetch(c + (size_t)hc * wc, b);
    }
    double t[5];
    normal_terms(coef1 + (size_t)f * coef_stride, coef2 + (size_t)f * coef_stride, P, h, w, y, x, du, dv, t);
    float* o = gh + (size_t)f * gh_stride + r;
#pragma unroll
    for (int c = 0; c < 5; ++c) o[c * P] = (float)t[c];
}

// ---- one displacement update on a 28x28 tile.
constexpr int BT = 28;            // tile side = 2 patches of 14
constexpr int BR = 7;             // window radius (window 15)
constexpr int BE = BT + 2 * BR;   // 42
constexpr int BEP = BE + 1;       // padded row (odd stride in 8-byte words: conflict-free row scans)
constexpr int BOX_THREADS = 256;
constexpr int EMIT_NEXT = 1, EMIT_D = 2, EMIT_DP = 4;

__global__ void __launch_bounds__(BOX_THREADS)
k_flow_box(const float* __restrict__ gh_in, size_t gh_stride, int h, int w, double eps,
           const float* __restrict__ coef1, const float* __restrict__ coef2, size_t coef_stride,
           float* __restrict__ gh_out, double* __restrict__ d_out, size_t flow_stride, float* __restrict__ dP,
           PlaneGeom g, int flags) {
    extern __shared__ double I[];                 // [5][BE][BEP] -> integral images
    __shared__ double psum[BOX_THREADS / 32][4];
    const int f = blockIdx.z;
    const int x0 = blockIdx.x * BT, y0 = blockIdx.y * BT;
    const size_t P = (size_t)h * w;
    const float* in = gh_in + (size_t)f * gh_stride;
    // the in-image part of the window only: zeros outside the image
    for (int i = threadIdx.x; i < BE * BE; i += BOX_THREADS) {
        int ry = i / BE, rx = i % BE;
        int y = y0 - BR + ry, x = x0 - BR + rx;
        bool inside = y >= 0 && y < h && x >= 0 && x < w;
        int p = y * w + x;
#pragma unroll
        for (int c = 0; c < 5; ++c) I[(c * BE + ry) * BEP + rx] = inside ? (double)in[c * P + p] : 0.0;
    }
    __syncthreads();
    if (threadIdx.x < 5 * BE) {                   // inclusive scan along each row
        double* row = I + threadIdx.x * BEP;
        double run = 0.0;
#pragma unroll 6
        for (int rx = 0; rx < BE; ++rx) { run += row[rx]; row[rx] = run; }
    }
    __syncthreads();
    if (threadIdx.x < 5 * BE) {                   // then down each column
        int c = threadIdx.x / BE, rx = threadIdx.x % BE;
        double* col = I + c * BE * BEP + rx;
        double run = 0.0;
#pragma unroll 6
        for (int ry = 0; ry < BE; ++ry) { run += col[ry * BEP]; col[ry * BEP] = run; }
    }
    __syncthreads();
    double acc0 = 0.0, acc1 = 0.0, acc2 = 0.0, acc3 = 0.0;
    for (int i = threadIdx.x; i < BT * BT; i += BOX_THREADS) {
        int oy = i / BT, ox = i % BT;
        // window rows oy .. oy+14 and columns ox .. ox+14 of the grown tile
        double s[5];
#pragma unroll
        for (int c = 0; c < 5; ++c) {
            const double* Ic = I + c * BE * BEP;
            double a = Ic[(oy + 14) * BEP + ox + 14];
            double b = oy > 0 ? Ic[(oy - 1) * BEP + ox + 14] : 0.0;
            double cc = ox > 0 ? Ic[(oy + 14) * BEP + ox - 1] : 0.0;
            double d = (oy > 0 && ox > 0) ? Ic[(oy - 1) * BEP + ox - 1] : 0.0;
            s[c] = (a - b) - (cc - d);
        }
        const double det = s[0] * s[2] - s[1] * s[1] + eps;
        const double du = (s[2] * s[3] - s[1] * s[4]) / det;
        const double dv = (s[0] * s[4] - s[1] * s[3]) / det;
        const int y = y0 + oy, x = x0 + ox, p = y * w + x;
        if (flags & EMIT_D) {
            double* o = d_out + (size_t)f * flow_stride;
            o[p] = du;
            o[P + p] = dv;
        }
        if (flags & EMIT_NEXT) {
            double t[5];
            normal_terms(coef1 + (size_t)f * coef_stride, coef2 + (size_t)f * coef_stride, P, h, w, y, x, du, dv, t);
            float* o = gh_out + (size_t)f * gh_stride + p;
#pragma unroll
            for (int c = 0; c < 5; ++c) o[c * P] = (float)t[c];
        }
        if (flags & EMIT_DP) {
            const double m = du * du + dv * dv;
            const bool lower = oy >= BT / 2, right = ox >= BT / 2;
            acc0 += (!lower && !right) ? m : 0.0;
            acc1 += (!lower && right) ? m : 0.0;
            acc2 += (lower && !right) ? m : 0.0;
            acc3 += (lower && right) ? m : 0.0;
        }
    }
    if (flags & EMIT_DP) {     // Eq. 5 (flow reading): dP_i = sqrt(mean over the patch of u^2 + v^2)
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            acc0 += __shfl_xor_sync(0xffffffffu, acc0, o);
            acc1 += __shfl_xor_sync(0xffffffffu, acc1, o);
            acc2 += __shfl_xor_sync(0xffffffffu, acc2, o);
            acc3 += __shfl_xor_sync(0xffffffffu, acc3, o);
        }
        if ((threadIdx.x & 31) == 0) {
            double* ps = psum[threadIdx.x >> 5];
            ps[0] = acc0; ps[1] = acc1; ps[2] = acc2; ps[3] = acc3;
        }
        __syncthreads();
        if (threadIdx.x < 4) {
            double tot = 0.0;
            for (int wp = 0; wp < BOX_THREADS / 32; ++wp) tot += psum[wp][threadIdx.x];
            int py = blockIdx.y * 2 + threadIdx.x / 2, px = blockIdx.x * 2 + threadIdx.x % 2;
            dP[(size_t)f * g.n_tok + patch_token(g, py, px)] = (float)sqrt(tot / (double)((BT / 2) * (BT / 2)));
        }
    }
}

inline unsigned blocks_for(long long n, int threads) { return (unsigned)((n + threads - 1) / threads); }

}  // namespace

static size_t flow_box_smem() { return (size_t)5 * BE * BEP * sizeof(double); }

int sc_flow_init() {
    SC_CHECK(cudaFuncSetAttribute(k_flow_box, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)flow_box_smem()));
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
        const int nb = B - b0 < c->chunk ? B - b0 : c->chunk;    // pairs in this pass
        // frames to expand: a video shares frame b+1 between pairs b and b+1
        const int nf = sequence ? nb + 1 : 2 * nb;
        // scratch slot s holds: video -> frame b0+s ; otherwise slots [0,nb) = prev, [nb,2nb) = cur
        for (int part = 0; part < (sequence ? 1 : 2); ++part) {
            const uint8_t* src = (part == 0 ? d_prev : d_cur) + (size_t)b0 * frame_bytes;
            int n = sequence ? nf : nb;
            float* dst = c->pyr[0] + (size_t)part * nb * P0;
            k_gray<<<blocks_for((long long)(P0 / 16) * n, T), T, 0, st>>>(src, frame_bytes, (int)P0, n, dst);
            c->launches++;
        }
        for (int l = 1; l < 3; ++l)
            k_pyr_down<<<blocks_for((long long)hs[l] * ws[l] * nf, T), T, 0, st>>>(c->pyr[l - 1], hs[l - 1], ws[l - 1], nf,
                                                                                   c->pyr[l]);
        for (int l = 0; l < 3; ++l)
            k_poly_exp<<<blocks_for((long long)hs[l] * ws[l] * nf, T), T, 0, st>>>(c->pyr[l], hs[l], ws[l], nf, pw,
                                                                                   c->coef[l]);
        c->launches += 5;
        const size_t fstride = 2 * P0, gstride = 5 * P0;
        double* d_lvl[2] = {c->flow_a, c->flow_b};
        const double* coarse = nullptr;
        for (int l = 2; l >= 0; --l) {
            const size_t Pl = (size_t)hs[l] * ws[l];
            const size_t cstride = 5 * Pl;
            const float* c1 = c->coef[l];
            const float* c2 = c->coef[l] + (sequence ? cstride : (size_t)nb * cstride);
            k_flow_gh<<<blocks_for((long long)Pl * nb, 256), 256, 0, st>>>(c1, c2, cstride, hs[l], ws[l], coarse, fstride,
                                                                           c->gh_a, gstride, nb);
            c->launches++;
            float* gin = c->gh_a;
            float* gout = c->gh_b;
            double* dl = d_lvl[l & 1];
            dim3 grid(ws[l] / BT, hs[l] / BT, nb);
            for (int it = 0; it < p.iters; ++it) {
                const bool last = it == p.iters - 1;
                int flags = last ? 0 : EMIT_NEXT;
                double* dout = dl;
                if (last && l > 0) flags |= EMIT_D;
                if (last && l == 0) {
                    flags |= EMIT_DP;
                    if (d_flow_or_null) { flags |= EMIT_D; dout = d_flow_or_null + (size_t)b0 * fstride; }
                }
                k_flow_box<<<grid, BOX_THREADS, flow_box_smem(), st>>>(gin, gstride, hs[l], ws[l], p.eps_det, c1, c2,
                                                                       cstride, gout, dout, fstride,
                                                                       d_deltaP + (size_t)b0 * g.n_tok, g, flags);
                c->launches++;
                float* t = gin; gin = gout; gout = t;
            }
            coarse = dl;
        }
    }
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}
