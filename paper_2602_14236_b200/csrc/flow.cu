// Temporal branch (Sec. III-A, Eq. 5): gray pyramid, polynomial expansion, coarse-to-fine
// displacement updates and the per-patch RMS flow magnitude.
//
// Precision: everything but the patch reduction (double) runs in single precision.  Pyramid levels are exact in
// float; the expansion takes its moments through zero-sum kernels and differences from the window centre, so
// that its coefficients carry a relative error of a few 1e-7; the per-pixel normal-equation terms (G, h), their
// 15x15 window sums and the 2x2 solve sum without any subtraction and solve with compensated products; sampling
// positions are exact.  The effect on dP stays more than an order of
// magnitude below the 1e-4 relative tolerance on every workload.
//
// One displacement update = the terms (G, h) of every pixel at the current field (k_flow_terms, one pixel
// per thread) + window sums and a 2x2 solve (k_flow_update, on a 56x28 or 28x28 tile with separable sums:
// columns from registers, rows from shared memory), which leaves the new field or, after the last update,
// the patch scores.
#include <math.h>

#include <algorithm>

#include "common.cuh"

namespace {

__device__ __forceinline__ int clampi(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }

// ---- level 0: integer luma g = (77R + 150G + 29B + 128) >> 8 as float; 16 pixels per thread,
// three 16-byte loads of the interleaved RGB bytes.
__global__ void k_gray(const uint8_t* __restrict__ frames, size_t frame_bytes, int n_px, int n_frames,
                       float* __restrict__ out) {
    const int groups = n_px / 16;
    const int f = blockIdx.y, gidx = blockIdx.x * blockDim.x + threadIdx.x;      // grid: (groups of a frame, frames)
    if (gidx >= groups || f >= n_frames) return;
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
// One thread per 2x2 block of outputs: its 7x7 source neighbourhood is read once, five-tap sums along the rows
// first, then down the columns (the sums are exact, so their order does not matter).
__global__ void __launch_bounds__(256)
k_pyr_down(const float* __restrict__ src, int h, int w, int n_frames, float* __restrict__ dst) {
    const int h2 = h / 2, w2 = w / 2;
    const int bw = (w2 + 1) / 2, bh = (h2 + 1) / 2;
    const int f = blockIdx.y, r = blockIdx.x * blockDim.x + threadIdx.x;        // grid: (2x2 blocks of a level, frames)
    if (r >= bh * bw || f >= n_frames) return;
    const int by = r / bw, bx = r - by * bw;
    const int oy = 2 * by, ox = 2 * bx;
    const float* s = src + (size_t)f * h * w;
    int cx[7];
#pragma unroll
    for (int b = 0; b < 7; ++b) cx[b] = clampi(2 * ox - 2 + b, 0, w - 1);
    const bool inner = ox >= 1 && 2 * ox + 4 <= w - 1 && (w & 3) == 0;      // rows are then 16-byte aligned as well
    float hs[7][2];                                 // row sums of source rows 2 oy - 2 .. 2 oy + 4 for the two output columns
#pragma unroll
    for (int a = 0; a < 7; ++a) {
        const float* row = s + (size_t)clampi(2 * oy - 2 + a, 0, h - 1) * w;
        float v[7];
        if (inner) {                                // columns 4 bx - 2 .. 4 bx + 4 unclamped: 8 + 16 + 4 aligned bytes
            const float2 a2 = *reinterpret_cast<const float2*>(row + 2 * ox - 2);
            const float4 a4 = *reinterpret_cast<const float4*>(row + 2 * ox);
            v[0] = a2.x; v[1] = a2.y; v[2] = a4.x; v[3] = a4.y; v[4] = a4.z; v[5] = a4.w;
            v[6] = row[2 * ox + 4];
        } else {
#pragma unroll
            for (int b = 0; b < 7; ++b) v[b] = row[cx[b]];
        }
        hs[a][0] = (v[0] + v[4]) + 4.f * (v[1] + v[3]) + 6.f * v[2];
        hs[a][1] = (v[2] + v[6]) + 4.f * (v[3] + v[5]) + 6.f * v[4];
    }
    float* d = dst + (size_t)f * h2 * w2;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        if (oy + j >= h2) break;
        float o[2];
#pragma unroll
        for (int i = 0; i < 2; ++i)
            o[i] = ((hs[2 * j][i] + hs[2 * j + 4][i]) + 4.f * (hs[2 * j + 1][i] + hs[2 * j + 3][i]) + 6.f * hs[2 * j + 2][i]) * (1.0f / 256.0f);
        float* q = d + (size_t)(oy + j) * w2 + ox;
        if ((w2 & 1) == 0) {                        // even rows: the pair is inside and 8-byte aligned
            *reinterpret_cast<float2*>(q) = make_float2(o[0], o[1]);
        } else {
            q[0] = o[0];
            if (ox + 1 < w2) q[1] = o[1];
        }
    }
}

// ---- polynomial expansion, 5x5: r2 r3 r4 r5 r6 = (b_x, b_y, A_xx, A_yy, 2 A_xy), stored as float in the form the
// displacement updates read: (r2, r3, r4, r5) / 2 as one 16-byte record per pixel and r6 / 4 in a plane of its own.
// A 32x32 tile grown by 2 is staged in shared memory.
constexpr int PX = 32, PY = 32, PH = 2;          // tile and halo
constexpr int PEW = PX + 2 * PH, PEH = PY + 2 * PH;

// Single precision.  Every moment is taken through a kernel that sums to zero or
// through differences from the window's centre value, so that what gets multiplied and added are local
// differences of the image (exact in float: the levels are dyadic rationals) and never the image values
// themselves; the coefficients then carry a relative error of a few 1e-7 instead of an absolute one of 1e-5:
//   H1 = sum_b g(b) b f            = g1 (f[+1] - f[-1]) + 2 g2 (f[+2] - f[-2])            along a row
//   H2 = sum_b g(b) (b^2 - mu2) f  = k1 (f[+1] + f[-1] - 2 f[0]) + k2 (f[+2] + f[-2] - 2 f[0])
//   V1, V2 the same down a column;  S[q] = sum_a g(a) q[a] = q[0] + g1 ((q[1]-q[0]) + (q[-1]-q[0])) + g2 (...)
//   m10 = S_rows[H1], m20 - mu2 m00 = S_rows[H2], m11 = g1 (H1[+1] - H1[-1]) + 2 g2 (H1[+2] - H1[-2]) down the rows,
//   m01 = S_cols[V1], m02 - mu2 m00 = S_cols[V2].
struct PolyW32 {
    float g1, g2, k1, k2;            // g(1), g(2); g(1) (1 - mu2), g(2) (4 - mu2)
    float s2, s3, s45, s6;           // output scalings: 1/(2 mu2), 1/(2 mu2), 1/(2 (mu4 - mu2^2)), 1/(4 mu2^2)
};

__device__ __forceinline__ float smooth5(float qm2, float qm1, float q0, float qp1, float qp2, float g1, float g2) {
    return q0 + (g1 * ((qp1 - q0) + (qm1 - q0)) + g2 * ((qp2 - q0) + (qm2 - q0)));
}

// Block (32, 8): thread (tx, ty) owns column tx of rows 4 ty .. 4 ty + 3 (of rows ty, ty + 8, ... while staging and in
// the row pass): every loop below has a compile-time trip count, every shared-memory access is a base plus a constant,
// and the five-tap windows of a thread's four rows share their loads.
__global__ void __launch_bounds__(256)
k_poly_exp32(const float* __restrict__ img, int h, int w, int n_frames, PolyW32 pw, float4* __restrict__ cq,
             float* __restrict__ cr) {
    __shared__ float tile[PEH][PEW + 1];
    __shared__ float H1[PEH][PX], H2[PEH][PX];
    __shared__ float V1[PY][PEW + 1], V2[PY][PEW + 1];
    const int tx = threadIdx.x, ty = threadIdx.y;
    const int f = blockIdx.z, x0 = blockIdx.x * PX, y0 = blockIdx.y * PY;
    const size_t P = (size_t)h * w;
    const float* s = img + (size_t)f * P;
    const int xa = clampi(x0 - PH + tx, 0, w - 1), xb = clampi(x0 - PH + tx + 32, 0, w - 1);
#pragma unroll
    for (int k = 0; k < 5; ++k) {
        const int ry = ty + 8 * k;
        if (ry < PEH) {
            const float* row = s + (size_t)clampi(y0 - PH + ry, 0, h - 1) * w;
            tile[ry][tx] = row[xa];
            if (tx < PEW - 32) tile[ry][tx + 32] = row[xb];
        }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 5; ++k) {                      // along the rows of the grown tile
        const int ry = ty + 8 * k;
        if (ry < PEH) {
            const float* t = &tile[ry][tx];
            const float c = t[2];
            H1[ry][tx] = pw.g1 * (t[3] - t[1]) + 2.0f * pw.g2 * (t[4] - t[0]);
            H2[ry][tx] = pw.k1 * ((t[3] - c) + (t[1] - c)) + pw.k2 * ((t[4] - c) + (t[0] - c));
        }
    }
    auto down = [&](int oy, int rx) {                  // down the columns of the grown tile
        const float c = tile[oy + 2][rx];
        const float a1 = tile[oy + 1][rx], b1 = tile[oy + 3][rx], a2 = tile[oy][rx], b2 = tile[oy + 4][rx];
        V1[oy][rx] = pw.g1 * (b1 - a1) + 2.0f * pw.g2 * (b2 - a2);
        V2[oy][rx] = pw.k1 * ((b1 - c) + (a1 - c)) + pw.k2 * ((b2 - c) + (a2 - c));
    };
#pragma unroll
    for (int k = 0; k < 4; ++k) down(4 * ty + k, tx);              // four consecutive rows: their taps overlap
    if (ty < 4) down(8 * ty + (tx >> 2), 32 + (tx & 3));          // the four columns past the 32nd: 128 items, four warps
    __syncthreads();
    const int x = x0 + tx;
    if (x >= w) return;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int oy = 4 * ty + k, y = y0 + oy;                       // the rows of the column pass above: the windows overlap
        if (y >= h) break;
        const float h1a = H1[oy][tx], h1b = H1[oy + 1][tx], h1c = H1[oy + 2][tx], h1d = H1[oy + 3][tx], h1e = H1[oy + 4][tx];
        const float m10 = smooth5(h1a, h1b, h1c, h1d, h1e, pw.g1, pw.g2);
        const float m11 = pw.g1 * (h1d - h1b) + 2.0f * pw.g2 * (h1e - h1a);
        const float m20 = smooth5(H2[oy][tx], H2[oy + 1][tx], H2[oy + 2][tx], H2[oy + 3][tx], H2[oy + 4][tx], pw.g1, pw.g2);
        const float* v1 = &V1[oy][tx];
        const float* v2 = &V2[oy][tx];
        const float m01 = smooth5(v1[0], v1[1], v1[2], v1[3], v1[4], pw.g1, pw.g2);
        const float m02 = smooth5(v2[0], v2[1], v2[2], v2[3], v2[4], pw.g1, pw.g2);
        const size_t o = (size_t)f * P + (size_t)y * w + x;
        cq[o] = make_float4(m10 * pw.s2, m01 * pw.s3, m20 * pw.s45, m02 * pw.s45);
        cr[o] = m11 * pw.s6;
    }
}

// Expansion coefficients of one frame at one level, as the displacement updates read them:
//   q[p] = (b_x, b_y, A_xx, A_yy) / 2 as one 16-byte record per pixel,  r[p] = A_xy / 2.
// Halving is exact, so (A1 + A2)/2 and -(b2 - b1)/2 become plain sums and differences of stored values.
struct CoefView {
    const float4* __restrict__ q;
    const float* __restrict__ r;
};

__device__ __forceinline__ float lerp2(float a, float b, float c, float d, float gx, float fx, float gy, float fy) {
    const float top = a * gx + b * fx;
    const float bot = c * gx + d * fx;
    return top * gy + bot * fy;
}

// floor(v) as a float and as an int without the conversion unit, for |v| < 2^22: adding 1.5 * 2^23 rounds to the
// nearest integer, whose value sits in the low mantissa bits; one compare steps down where that rounded up.
__device__ __forceinline__ void floor_fi(float v, float& f, int& i) {
    const float t = v + 12582912.0f;
    float r = t - 12582912.0f;
    int k = __float_as_int(t) - 0x4B400000;
    if (r > v) { r -= 1.0f; k -= 1; }
    f = r;
    i = k;
}

// Normal-equation terms of one pixel for the prior (du, dv): G = A^T A (g11 g12 g22), hv = A^T db,
//   A = (A1(x) + A2(x~))/2,  db = -(b2(x~) - b1(x))/2 + A d~,  x~ = clamp(x + d~), bilinear fetch.
// The sampling position is exact: the displacement is clamped to [-x, w-1-x] (integers, exact in single
// precision), its floor and fraction are taken on the displacement itself and the integer part is added to the
// pixel index (x + d~ in single precision would move the sample by up to 2e-5 px at x ~ 300); the interpolation
// and the products run in single precision on the single-precision coefficients, whose rounding already bounds
// what they can deliver.  xlo = -x, xhi = w-1-x, ylo = -y, yhi = h-1-y as floats.
// The four taps are read at i, i+1, i+w, i+w+1 without clamping the far ones: where the position is
// clamped to the last column or row the fraction is zero, so the far tap is multiplied by zero, and it
// is a finite number (the next row, the next frame's plane, or the zeroed pad behind the last plane).
__device__ __forceinline__ void normal_terms(const float4 u, const float ur, const CoefView& c2, int w, int p, float xlo,
                                             float xhi, float ylo, float yhi, float du, float dv, float out[5]) {
    const float su = fminf(fmaxf(du, xlo), xhi), sv = fminf(fmaxf(dv, ylo), yhi);
    float fdu, fdv;
    int iu, iv;
    floor_fi(su, fdu, iu);
    floor_fi(sv, fdv, iv);
    const float fx = su - fdu, fy = sv - fdv;
    const float gx = 1.0f - fx, gy = 1.0f - fy;
    const int i0 = p + iv * w + iu;
    const float4 a = __ldg(c2.q + i0), b = __ldg(c2.q + i0 + 1), c = __ldg(c2.q + i0 + w), d = __ldg(c2.q + i0 + w + 1);
    const float ra = __ldg(c2.r + i0), rb = __ldg(c2.r + i0 + 1), rc = __ldg(c2.r + i0 + w), rd = __ldg(c2.r + i0 + w + 1);
    const float vbx = lerp2(a.x, b.x, c.x, d.x, gx, fx, gy, fy);
    const float vby = lerp2(a.y, b.y, c.y, d.y, gx, fx, gy, fy);
    const float vxx = lerp2(a.z, b.z, c.z, d.z, gx, fx, gy, fy);
    const float vyy = lerp2(a.w, b.w, c.w, d.w, gx, fx, gy, fy);
    const float vxy = lerp2(ra, rb, rc, rd, gx, fx, gy, fy);
    const float axx = u.z + vxx, ayy = u.w + vyy, axy = ur + vxy;
    const float dbx = (u.x - vbx) + (axx * du + axy * dv);
    const float dby = (u.y - vby) + (axy * du + ayy * dv);
    out[0] = axx * axx + axy * axy;
    out[1] = axx * axy + axy * ayy;
    out[2] = axy * axy + ayy * ayy;
    out[3] = axx * dbx + axy * dby;
    out[4] = axy * dbx + ayy * dby;
}

// a*d - b*c with one rounding error of each product recovered by a fused multiply-add (Kahan): good to
// about 1.5 ulp even when the products cancel.
__device__ __forceinline__ float det2(float a, float b, float c, float d) {
    const float w = b * c;
    const float e = fmaf(-b, c, w);
    const float f = fmaf(a, d, -w);
    return f + e;
}

// ---- (G, h) of the next update from the current field d (zero when there is none: the first update of the
// coarsest level).  One pixel per thread and no state shared between threads, so the kernel runs at full occupancy,
// which hides the latency of its gathers; fused behind the solve of the update kernel it ran at a quarter of the
// warps and took longer than the two kernels apart.  What streams from DRAM (the pixel's own record and field
// value, 28 bytes) is fetched one block ahead by asynchronous copies into a slot of shared memory that only the
// thread itself reads: the next block's bytes are in flight while this block's gathers wait for the L2.
constexpr int TERMS_THREADS = 256;
constexpr int TERMS_BLOCKS_PER_CTA = 8;      // at most

__device__ __forceinline__ void async_copy16(void* dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void async_copy8(void* dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void async_copy4(void* dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}

// PRIOR: `d` is the COARSER level's field (h/2 x w/2) and the pixel's value is the prior of the level,
//   d = 2 * bilinear(d_coarse) at ((x+1/2)/2 - 1/2, (y+1/2)/2 - 1/2), clamped to the coarse image:
// for a fine coordinate x that position is x/2 - 1/4, and at x = 0 and at the last fine pixel the clamp puts it on a
// tap itself.  It is formed here from its four taps (they come from the L2: every coarse value serves a dozen fine
// pixels), so that the first update of a level neither writes nor reads a prior field.
template <bool PRIOR>
__global__ void __launch_bounds__(TERMS_THREADS)
k_flow_terms(const float4* __restrict__ q1, const float* __restrict__ r1, const float4* __restrict__ q2,
             const float* __restrict__ r2, int h, int w, unsigned w_inv, const float2* __restrict__ d, size_t d_stride,
             float* __restrict__ gh, size_t gh_stride, int n_pairs) {
    __shared__ float4 sq[2][TERMS_THREADS];
    __shared__ float2 sd[2][TERMS_THREADS];
    __shared__ float sr[2][TERMS_THREADS];
    const int P = h * w;
    const int f = blockIdx.y;                                   // grid: (blocks of pixels / TERMS_BLOCKS_PER_CTA, pairs)
    if (f >= n_pairs) return;
    const int t = threadIdx.x;
    const int step = gridDim.x * TERMS_THREADS;
    const float4* qf = q1 + (size_t)f * P;
    const float* rf = r1 + (size_t)f * P;
    const float2* df = d ? d + (size_t)f * d_stride : nullptr;
    const CoefView c2{q2 + (size_t)f * P, r2 + (size_t)f * P};
    auto fetch = [&](int r, int slot) {
        if (r < P) {
            async_copy16(&sq[slot][t], qf + r);
            async_copy4(&sr[slot][t], rf + r);
            if (!PRIOR && df) async_copy8(&sd[slot][t], df + r);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    int r = blockIdx.x * TERMS_THREADS + t;
    fetch(r, 0);
    for (int n = 0; r < P; r += step, ++n) {
        fetch(r + step, (n + 1) & 1);
        asm volatile("cp.async.wait_group 1;" ::: "memory");       // this block's copies have landed, the next block's fly
        const int slot = n & 1;
        const float4 u = sq[slot][t];
        const float ur = sr[slot][t];
        const int y = (int)__umulhi((unsigned)r, w_inv), x = r - y * w;         // w_inv = ceil(2^32 / w): exact for r < 2^32 / w
        float2 dd = make_float2(0.0f, 0.0f);
        if (PRIOR) {
            // fine x = 2 xc takes taps (xc - 1, xc) with weight 3/4 on the right one, x = 2 xc + 1 taps (xc, xc + 1)
            // with weight 1/4 on the right one; a tap that the clamp moved carries weight zero.  Rows alike.
            const int wc = w >> 1, hc = h >> 1, xc = x >> 1, yc = y >> 1;
            const bool xo = x & 1, yo = y & 1;
            const bool xin = xo ? xc < wc - 1 : xc > 0, yin = yo ? yc < hc - 1 : yc > 0;
            const int c0 = xc - ((!xo && xin) ? 1 : 0), c1 = xc + ((xo && xin) ? 1 : 0);
            const int r0 = yc - ((!yo && yin) ? 1 : 0), r1c = yc + ((yo && yin) ? 1 : 0);
            const float fx = xin ? (xo ? 0.25f : 0.75f) : 0.0f, fy = yin ? (yo ? 0.25f : 0.75f) : 0.0f;
            const float2 p00 = __ldg(df + r0 * wc + c0), p01 = __ldg(df + r0 * wc + c1);
            const float2 p10 = __ldg(df + r1c * wc + c0), p11 = __ldg(df + r1c * wc + c1);
            const float gx = 1.0f - fx, gy = 1.0f - fy;
            dd.x = 2.0f * lerp2(p00.x, p01.x, p10.x, p11.x, gx, fx, gy, fy);
            dd.y = 2.0f * lerp2(p00.y, p01.y, p10.y, p11.y, gx, fx, gy, fy);
        } else if (df) {
            dd = sd[slot][t];
        }
        float o5[5];
        normal_terms(u, ur, c2, w, r, (float)-x, (float)(w - 1 - x), (float)-y, (float)(h - 1 - y), dd.x, dd.y, o5);
        float* o = gh + (size_t)f * gh_stride + r;
#pragma unroll
        for (int c = 0; c < 5; ++c) o[c * P] = o5[c];
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// ---- one displacement update on a tile of TW x 28 pixels (TW / 14 x 2 patches).
//   phase 1  one thread per (term, pair of columns of the tile grown by 8 columns each side): 42 8-byte
//            loads down the columns in three blocks of 14 rows; the 15-row sums of the 28 tile rows are a
//            suffix sum of one block plus a prefix sum of the next (no subtraction) -> shared memory
//   phase 2  one thread per (row, run of RUN columns): 15-column sums of the row sums the same way,
//            2x2 solve -> d in shared memory
//   phase 3  one thread per pixel: d itself (for k_flow_terms and for the next finer level), and / or the
//            patch scores after the last update
// The window covers the in-image part only: terms outside the image count as zero.
constexpr int TH = 28;             // tile height = 2 patches
constexpr int BR = 7;              // window radius (window 15)
constexpr int BLK = 2 * BR;        // rows per block of the suffix / prefix scheme
constexpr int UPD_THREADS = 224;
constexpr int EMIT_D = 2, EMIT_DP = 4, EMIT_D64 = 8;

template <int TW>
struct UpdGeom {
    static constexpr int RUN = TW % 8 == 0 ? 8 : 4;    // pixels per phase-2 thread
    static constexpr int EW = TW + 16;                 // columns loaded: x0 - 8 .. x0 + TW + 7 (8-byte aligned pairs)
    static constexpr int S = EW % 8 == 4 ? EW : EW + 4; // row stride in floats, = 4 (mod 8): the 16-byte loads of 8
                                                       // consecutive rows fall on distinct banks
    static constexpr int NQ = 2 * BR + RUN + 2;        // row sums read per run, starting one column early (16-byte aligned)
    static constexpr int DPITCH = TW + 1;              // (du, dv) row pitch: odd, spreads phase 2's stores over the banks
    static_assert(TW % 14 == 0 && (RUN == 4 || RUN == 8) && S % 8 == 4 && NQ % 4 == 0 && 5 * (EW / 2) <= UPD_THREADS &&
                      TH * (TW / RUN) <= UPD_THREADS && UPD_THREADS % TW == 0,
                  "tile geometry");
};

template <int TW, int FLAGS>
__global__ void __launch_bounds__(UPD_THREADS, 4)
k_flow_update(const float* __restrict__ gh_in, size_t gh_stride, int h, int w, float eps, float2* __restrict__ d_out,
              size_t d_stride, double* __restrict__ d_out64, size_t flow_stride, float* __restrict__ dP, PlaneGeom g) {
    using G = UpdGeom<TW>;
    constexpr int RUN = G::RUN, EW = G::EW, S = G::S, NQ = G::NQ, DPITCH = G::DPITCH;
    extern __shared__ __align__(16) float upd_smem[];
    float (*vs)[TH][S] = reinterpret_cast<float (*)[TH][S]>(upd_smem);                       // [5] 15-row sums
    float2 (*dsm)[DPITCH] = reinterpret_cast<float2 (*)[DPITCH]>(upd_smem + 5 * TH * S);     // [TH] (du, dv)
    const int f = blockIdx.z;
    const int x0 = blockIdx.x * TW, y0 = blockIdx.y * TH;
    const int P = h * w;
    const int t = threadIdx.x;
    if (t < 5 * (EW / 2)) {
        const int c = t / (EW / 2), cp = t - c * (EW / 2);
        const int x = x0 - 8 + 2 * cp;                  // even, and w is even: the pair is inside or outside together
        const bool xin = x >= 0 && x < w;
        const float* src = gh_in + (size_t)f * gh_stride + c * P + (xin ? x : 0) + (y0 - BR) * w;
        // rows y0 - 7 + r, r in [0, 42): those inside the image are r in [r_lo, r_hi)
        const unsigned r_lo = y0 >= BR ? 0u : (unsigned)(BR - y0);
        const unsigned r_n = (xin ? (unsigned)min(TH + 2 * BR, h - y0 + BR) : r_lo) - r_lo;
        auto load = [&](int r) {
            return ((unsigned)r - r_lo < r_n) ? __ldg(reinterpret_cast<const float2*>(src + r * w)) : make_float2(0.0f, 0.0f);
        };
        float2 a[BLK], b[BLK];
#pragma unroll
        for (int r = 0; r < BLK; ++r) a[r] = load(r);
#pragma unroll
        for (int r = 0; r < BLK; ++r) b[r] = load(BLK + r);
        // window of tile row r = rows r .. r+14 = (suffix of the block it starts in) + (prefix of the next block):
        // at most 14 roundings per sum and no subtraction (a sliding window would leave the rounding residue of a
        // strong edge in the flat region behind it)
#pragma unroll
        for (int r = BLK - 2; r >= 0; --r) { a[r].x += a[r + 1].x; a[r].y += a[r + 1].y; }
        float2* dst = reinterpret_cast<float2*>(&vs[c][0][2 * cp]);
        float2 pre = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int r = 0; r < BLK; ++r) {
            pre.x += b[r].x; pre.y += b[r].y;
            dst[r * (S / 2)] = make_float2(a[r].x + pre.x, a[r].y + pre.y);
        }
#pragma unroll
        for (int r = 0; r < BLK; ++r) a[r] = load(2 * BLK + r);
#pragma unroll
        for (int r = BLK - 2; r >= 0; --r) { b[r].x += b[r + 1].x; b[r].y += b[r + 1].y; }
        pre = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int r = 0; r < BLK; ++r) {
            pre.x += a[r].x; pre.y += a[r].y;
            dst[(BLK + r) * (S / 2)] = make_float2(b[r].x + pre.x, b[r].y + pre.y);
        }
    }
    __syncthreads();
    if (t < TH * (TW / RUN)) {
        const int row = t % TH, run = t / TH;      // a quarter warp reads 8 rows of one run: conflict-free 16-byte loads
        const int col0 = RUN * run;                // output columns col0 .. col0+RUN-1; their windows start at col0 + 1
        float s[5][RUN];
#pragma unroll
        for (int c = 0; c < 5; ++c) {
            const float4* src = reinterpret_cast<const float4*>(&vs[c][row][col0]);
            float q[NQ];
#pragma unroll
            for (int i = 0; i < NQ / 4; ++i) {
                float4 pr = src[i];
                q[4 * i] = pr.x;
                q[4 * i + 1] = pr.y;
                q[4 * i + 2] = pr.z;
                q[4 * i + 3] = pr.w;
            }
            // windows q[k+1 .. k+15], k = 0..RUN-1, again without subtraction: suffix sums ending at q[15],
            // prefix sums starting at q[16]
            float suf = q[RUN];
#pragma unroll
            for (int i = RUN + 1; i <= 2 * BR + 1; ++i) suf += q[i];
            s[c][RUN - 1] = suf;
#pragma unroll
            for (int k = RUN - 2; k >= 0; --k) {      // suf = q[k+1] + ... + q[15]
                suf += q[k + 1];
                s[c][k] = suf;
            }
            float pre = 0.0f;
#pragma unroll
            for (int k = 1; k < RUN; ++k) {            // pre = q[16] + ... + q[15+k]
                pre += q[2 * BR + 1 + k];
                s[c][k] += pre;
            }
        }
        // the 2x2 solve: determinant and numerators cancel, so each is formed with compensated products
#pragma unroll
        for (int k = 0; k < RUN; ++k) {
            const float g11 = s[0][k], g12 = s[1][k], g22 = s[2][k], h1 = s[3][k], h2 = s[4][k];
            const float inv = __frcp_rn(det2(g11, g12, g12, g22) + eps);
            dsm[row][col0 + k] = make_float2(det2(g22, g12, h2, h1) * inv, det2(g11, g12, h1, h2) * inv);
        }
    }
    __syncthreads();
    // UPD_THREADS is a multiple of TW: a thread keeps its column, hence its patch column, over its pixels
    constexpr int PER = (TH * TW + UPD_THREADS - 1) / UPD_THREADS, RSTEP = UPD_THREADS / TW;
    const int ox = t % TW, oyb = t / TW;
    const int x = x0 + ox;
    double acc_up = 0.0, acc_lo = 0.0;                 // upper / lower patch of the tile
    int p = (y0 + oyb) * w + x;
#pragma unroll
    for (int j = 0; j < PER; ++j, p += RSTEP * w) {
        const int oy = oyb + j * RSTEP;
        if ((TH * TW) % UPD_THREADS != 0 && oy >= TH) break;
        const float2 d = dsm[oy][ox];
        if (FLAGS & EMIT_D) d_out[(size_t)f * d_stride + p] = d;
        if (FLAGS & EMIT_D64) {
            double* o = d_out64 + (size_t)f * flow_stride;
            o[p] = (double)d.x;
            o[P + p] = (double)d.y;
        }
        if (FLAGS & EMIT_DP) {
            const double m = (double)d.x * (double)d.x + (double)d.y * (double)d.y;
            if (oy < 14) acc_up += m; else acc_lo += m;
        }
    }
    if (FLAGS & EMIT_DP) {     // Eq. 5 (flow reading): dP_i = sqrt(mean over the patch of u^2 + v^2)
        double* part = reinterpret_cast<double*>(upd_smem);     // the row sums are no longer needed
        part[t] = acc_up;                                       // t = oyb * TW + ox
        part[UPD_THREADS + t] = acc_lo;
        __syncthreads();
        if (t < 2 * TW) {                          // column totals, then 14 columns per patch: fixed order, deterministic
            const int half = t / TW, col = t - half * TW;
            double tot = 0.0;
#pragma unroll
            for (int k = 0; k < RSTEP; ++k) tot += part[half * UPD_THREADS + k * TW + col];
            part[2 * UPD_THREADS + t] = tot;
        }
        __syncthreads();
        if (t < 2 * (TW / 14)) {
            const int half = t / (TW / 14), pc = t - half * (TW / 14);
            double tot = 0.0;
#pragma unroll
            for (int q = 0; q < 14; ++q) tot += part[2 * UPD_THREADS + half * TW + 14 * pc + q];
            const int py = 2 * blockIdx.y + half, px = blockIdx.x * (TW / 14) + pc;
            dP[(size_t)f * g.n_tok + patch_token(g, py, px)] = (float)sqrt(tot / 196.0);
        }
    }
}

template <int TW>
constexpr size_t upd_smem_bytes() {
    // the row sums (reused as 2 * UPD_THREADS + 2 * TW doubles by the patch reduction), then (du, dv) as float2
    return (size_t)5 * TH * UpdGeom<TW>::S * sizeof(float) + (size_t)TH * UpdGeom<TW>::DPITCH * sizeof(float2);
}
static_assert((2 * UPD_THREADS + 2 * 56) * sizeof(double) <= 5 * TH * UpdGeom<28>::S * sizeof(float), "patch reduction fits");

template <int TW>
int init_update() {
#define SC_UPD(F) SC_CHECK(cudaFuncSetAttribute(k_flow_update<TW, F>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)upd_smem_bytes<TW>()));
    SC_UPD(EMIT_D) SC_UPD(EMIT_DP) SC_UPD(EMIT_DP | EMIT_D64)
#undef SC_UPD
    return SALICACHE_OK;
}

struct UpdArgs {
    const float* gin; size_t gstride; int h, w; float eps;
    float2* dout; size_t dstride; double* dout64; size_t fstride; float* dP;
};

template <int TW>
void launch_update(dim3 grid, cudaStream_t st, int flags, const UpdArgs& a, const PlaneGeom& g) {
#define SC_UPD(F)                                                                                                   \
    case F:                                                                                                         \
        k_flow_update<TW, F><<<grid, UPD_THREADS, upd_smem_bytes<TW>(), st>>>(a.gin, a.gstride, a.h, a.w, a.eps, a.dout, a.dstride, \
                                                                               a.dout64, a.fstride, a.dP, g);     \
        break;
    switch (flags) {
        SC_UPD(EMIT_D)
        SC_UPD(EMIT_DP)
        SC_UPD(EMIT_DP | EMIT_D64)
        default: break;
    }
#undef SC_UPD
}

// ---- Eq. 5 read literally: dP_i = L2 norm of the pixel difference over patch i, normalised by the patch's
// 3 * 14 * 14 values so that it is an RMS in grey levels.  One CTA per (band of 14 image rows, frame pair):
// both bands are read once with 16-byte loads, squared byte differences are summed exactly in integers
// (a 16-byte chunk straddles at most two patches: 42 bytes per patch row), one shared-memory counter per patch.
constexpr int DIFF_THREADS = 256;
__global__ void __launch_bounds__(DIFF_THREADS)
k_diff_score(const uint8_t* __restrict__ prev, const uint8_t* __restrict__ cur, size_t frame_bytes, PlaneGeom g,
             float* __restrict__ dP) {
    __shared__ unsigned int acc[64];                          // patches per band (<= 48)
    const int f = blockIdx.y, py = blockIdx.x;
    const int row_bytes = g.W * 3, chunks = row_bytes / 16;   // W is a multiple of 16
    for (int i = threadIdx.x; i < g.gw; i += DIFF_THREADS) acc[i] = 0;
    __syncthreads();
    const uint8_t* a = prev + (size_t)f * frame_bytes + (size_t)py * 14 * row_bytes;
    const uint8_t* b = cur + (size_t)f * frame_bytes + (size_t)py * 14 * row_bytes;
    for (int i = threadIdx.x; i < 14 * chunks; i += DIFF_THREADS) {
        const int r = i / chunks, k = i - r * chunks;
        const uint4 va = __ldg(reinterpret_cast<const uint4*>(a + (size_t)r * row_bytes) + k);
        const uint4 vb = __ldg(reinterpret_cast<const uint4*>(b + (size_t)r * row_bytes) + k);
        const int b0 = 16 * k, p0 = b0 / 42;
        const int m = 42 * (p0 + 1) - b0;                     // bytes of this chunk that belong to patch p0 (>= 1)
        const uint32_t wa[4] = {va.x, va.y, va.z, va.w}, wb[4] = {vb.x, vb.y, vb.z, vb.w};
        unsigned int lo = 0, hi = 0;
#pragma unroll
        for (int w4 = 0; w4 < 4; ++w4) {
            const uint32_t d = __vabsdiffu4(wa[w4], wb[w4]);
            const int n = m - 4 * w4;                         // bytes of this word in patch p0
            const uint32_t mask = n >= 4 ? 0xffffffffu : (n <= 0 ? 0u : ((1u << (8 * n)) - 1u));
            const uint32_t dl = d & mask, dh = d & ~mask;
            lo = __dp4a(dl, dl, lo);
            hi = __dp4a(dh, dh, hi);
        }
        atomicAdd(&acc[p0], lo);
        if (hi) atomicAdd(&acc[p0 + 1], hi);
    }
    __syncthreads();
    for (int px = threadIdx.x; px < g.gw; px += DIFF_THREADS)
        dP[(size_t)f * g.n_tok + patch_token(g, py, px)] = (float)sqrt((double)acc[px] / (double)(3 * 14 * 14));
}

inline unsigned blocks_for(long long n, int threads) { return (unsigned)((n + threads - 1) / threads); }

}  // namespace

int sc_flow_init() {
    int rc = init_update<56>();
    return rc != SALICACHE_OK ? rc : init_update<28>();
}

int sc_diff_score(salicache_ctx* c, const PlaneGeom& g, const uint8_t* d_prev, const uint8_t* d_cur, size_t frame_bytes,
                  int B, float* d_deltaP, cudaStream_t st) {
    if (B == 0) return SALICACHE_OK;
    dim3 grid(g.gh, B);
    k_diff_score<<<grid, DIFF_THREADS, 0, st>>>(d_prev, d_cur, frame_bytes, g, d_deltaP);
    c->launches++;
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}

int sc_flow_score(salicache_ctx* c, const PlaneGeom& g, const uint8_t* d_prev, const uint8_t* d_cur, size_t frame_bytes,
                  int B, bool sequence, float* d_deltaP, double* d_flow_or_null, cudaStream_t st) {
    const salicache_params& p = c->p;
    PolyW32 pw32;
    {
        double g[5], Z = 0, mu2 = 0, mu4 = 0;
        for (int k = -2; k <= 2; ++k) { g[k + 2] = exp(-(double)(k * k) / (2.0 * p.poly_sigma * p.poly_sigma)); Z += g[k + 2]; }
        for (int k = -2; k <= 2; ++k) {
            g[k + 2] /= Z;
            mu2 += g[k + 2] * k * k;
            mu4 += g[k + 2] * k * k * (double)(k * k);
        }
        pw32 = PolyW32{(float)g[3], (float)g[4], (float)(g[3] * (1.0 - mu2)), (float)(g[4] * (4.0 - mu2)),
                       (float)(0.5 / mu2), (float)(0.5 / mu2), (float)(0.5 / (mu4 - mu2 * mu2)), (float)(0.25 / (mu2 * mu2))};
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
            k_gray<<<dim3(blocks_for((long long)(P0 / 16), T), n), T, 0, st>>>(src, frame_bytes, (int)P0, n, dst);
            c->launches++;
        }
        for (int l = 1; l < 3; ++l)
            k_pyr_down<<<dim3(blocks_for((long long)((hs[l] + 1) / 2) * ((ws[l] + 1) / 2), T), nf), T, 0, st>>>(
                c->pyr[l - 1], hs[l - 1], ws[l - 1], nf, c->pyr[l]);
        const size_t slots = (size_t)2 * c->chunk;
        float4* cq[3];
        float* cr[3];
        for (int l = 0; l < 3; ++l) {      // the records, a pad of one row + 2, then the A_xy plane (and its pad)
            cq[l] = reinterpret_cast<float4*>(c->coef[l]);
            cr[l] = c->coef[l] + 4 * (slots * hs[l] * ws[l] + ws[l] + 2);
            dim3 gp((ws[l] + PX - 1) / PX, (hs[l] + PY - 1) / PY, nf);
            k_poly_exp32<<<gp, dim3(32, 8), 0, st>>>(c->pyr[l], hs[l], ws[l], nf, pw32, cq[l], cr[l]);
        }
        c->launches += 5;
        // Coarse to fine.  Per level `iters` times (terms of every pixel from the current field, the first time from the
        // coarser level's field; window sums + solve -> the new field), each launch over all pairs of the pass.  (Sub-batches sized for the L2 cache were measured and are slower: the kernels are bound by issue
        // slots and load latency, not by DRAM, and small launches add ramp-up and tail time.)
        const size_t fstride = 2 * P0, dstride = P0;      // caller's double field; float2 fields of the scratch
        float2* d_lvl[2] = {reinterpret_cast<float2*>(c->flow_a), reinterpret_cast<float2*>(c->flow_b)};
        for (int l = 2; l >= 0; --l) {
            const size_t Pl = (size_t)hs[l] * ws[l];
            const size_t gstride = 5 * Pl;
            float2* dl = d_lvl[l & 1];
            const int tw = ws[l] % 56 == 0 ? 56 : 28;
            const size_t second = sequence ? Pl : (size_t)nb * Pl;      // the pair's second frame, in pixels
            const float4* q1 = cq[l];
            const float* r1 = cr[l];
            const unsigned w_inv = (unsigned)((0x100000000ull + ws[l] - 1) / ws[l]);
            dim3 grid(ws[l] / tw, hs[l] / TH, nb);
            // blocks of pixels per CTA of the terms kernel: up to 8 (so that the copies ahead pay), fewer while the
            // launch would otherwise leave SMs without a full set of CTAs
            const long long terms_blocks = (long long)blocks_for((long long)Pl, TERMS_THREADS) * nb;
            const int terms_per_cta = (int)std::max(1ll, std::min((long long)TERMS_BLOCKS_PER_CTA, terms_blocks / (16ll * c->sm_count)));
            for (int it = 0; it < p.iters; ++it) {
                const bool last = it == p.iters - 1;
                // the first update of a finer level starts from the coarser level's field, transferred inside the kernel
                const dim3 tgrid(blocks_for((long long)Pl, TERMS_THREADS * terms_per_cta), nb);
                if (it == 0 && l < 2)
                    k_flow_terms<true><<<tgrid, TERMS_THREADS, 0, st>>>(q1, r1, q1 + second, r1 + second, hs[l], ws[l], w_inv,
                                                                        d_lvl[(l + 1) & 1], dstride, c->gh_a, gstride, nb);
                else
                    k_flow_terms<false><<<tgrid, TERMS_THREADS, 0, st>>>(q1, r1, q1 + second, r1 + second, hs[l], ws[l], w_inv,
                                                                         (l == 2 && it == 0) ? nullptr : dl, dstride, c->gh_a,
                                                                         gstride, nb);
                int flags = EMIT_D;
                double* dout64 = nullptr;
                if (last && l == 0) {      // the field goes to the caller's buffer if there is one
                    flags = EMIT_DP;
                    if (d_flow_or_null) {
                        flags |= EMIT_D64;
                        dout64 = d_flow_or_null + (size_t)b0 * fstride;
                    }
                }
                UpdArgs a{c->gh_a, gstride, hs[l], ws[l], (float)p.eps_det, dl, dstride, dout64, fstride,
                          d_deltaP + (size_t)b0 * g.n_tok};
                if (tw == 56) launch_update<56>(grid, st, flags, a, g);
                else launch_update<28>(grid, st, flags, a, g);
                c->launches += 2;
            }
        }
    }
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}
