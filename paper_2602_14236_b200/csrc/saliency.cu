// Spatial branch (Sec. III-B, Eq. 7): integer Canny edge map, LAB local colour variance,
// S = clamp(w_edge E + w_color C, 0, 1), per-patch mean.
#include <math.h>

#include "common.cuh"

namespace {

__device__ __forceinline__ int clampi(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }

__device__ __forceinline__ int gray_at(const uint8_t* __restrict__ fr, int w, int y, int x) {
    const uint8_t* p = fr + ((size_t)y * w + x) * 3;
    return (77 * p[0] + 150 * p[1] + 29 * p[2] + 128) >> 8;
}

// ---- anyres base image: 2x2 integer box mean (a+b+c+d+2)>>2 per channel.
__global__ void k_box_down2(const uint8_t* __restrict__ src, int H, int W, int n_frames, uint8_t* __restrict__ dst) {
    int h2 = H / 2, w2 = W / 2;
    long long gid = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (gid >= (long long)h2 * w2 * n_frames) return;
    int f = (int)(gid / (h2 * w2)), r = (int)(gid % (h2 * w2));
    int y = r / w2, x = r % w2;
    const uint8_t* s = src + (size_t)f * H * W * 3;
    const uint8_t* a = s + ((size_t)(2 * y) * W + 2 * x) * 3;
    const uint8_t* b = a + (size_t)W * 3;
    uint8_t* o = dst + ((size_t)f * h2 * w2 + r) * 3;
#pragma unroll
    for (int c = 0; c < 3; ++c) o[c] = (uint8_t)((a[c] + a[3 + c] + b[c] + b[3 + c] + 2) >> 2);
}

// ---- Canny up to the double threshold.  Tile 32x32, halo 4 (blur 2 + Sobel 1 + NMS 1).
// Writes two bit planes (bit i of word wx = pixel 32*wx + i): kept = NMS-kept with m >= lo^2,
// strong = kept with m >= hi^2.
// The frame's bytes are staged with 16-byte loads (a row of W pixels is 3 W bytes, a multiple of 16), gray is
// derived once from the staged bytes, and the 5x5 binomial blur runs as two passes of five taps: its integer sum
// is the same whichever way it is bracketed.
constexpr int CT = 32;
constexpr int CG = CT + 8;   // gray tile
constexpr int CB = CT + 4;   // blur tile
constexpr int CM = CT + 2;   // magnitude tile
constexpr int GRAY_ROWS = 7, GRAY_GROUPS = (CG + GRAY_ROWS - 1) / GRAY_ROWS;   // 6 groups of 40 columns: 240 threads
constexpr int BLUR_ROWS = 6, BLUR_GROUPS = (CG + BLUR_ROWS - 1) / BLUR_ROWS;   // 7 groups of 36 columns: 252 threads
constexpr int MAG_ROWS = 5, MAG_GROUPS = (CM + MAG_ROWS - 1) / MAG_ROWS;   // rows of the magnitude tile per thread; 7 groups
constexpr int CRAW = 9;      // 16-byte chunks staged per row: 40 pixels = 120 bytes starting up to 12 bytes into a chunk

__global__ void __launch_bounds__(256)
k_canny_classify(const uint8_t* __restrict__ frames, size_t frame_bytes, int h, int w, int words, int lo2, int hi2,
                 uint32_t* __restrict__ bits_kept, uint32_t* __restrict__ bits_strong, const uint8_t* __restrict__ skip) {
    __shared__ uint4 sraw[CG][CRAW];
    __shared__ uint8_t sg[CG][CG];
    __shared__ uint16_t sh[CG][CB];      // horizontal pass of the blur, at most 16 * 255
    __shared__ uint8_t sb[CB][CB];
    __shared__ int smag[CM][CM];
    const int f = blockIdx.z, x0 = blockIdx.x * CT, y0 = blockIdx.y * CT;
    if (skip && skip[f]) return;
    const uint8_t* fr = frames + (size_t)f * frame_bytes;
    const int row_bytes = 3 * w;
    // bytes of the clamped columns x0-4 .. x0+35: from the chunk that holds the first one
    const int xa = x0 >= 4 ? x0 - 4 : 0;
    const int byte0 = (3 * xa) & ~15;
    for (int i = threadIdx.x; i < CG * CRAW; i += blockDim.x) {
        const int ry = i / CRAW, ch = i - ry * CRAW;
        const int y = clampi(y0 - 4 + ry, 0, h - 1);
        const int off = byte0 + 16 * ch;
        if (off < row_bytes) sraw[ry][ch] = __ldg(reinterpret_cast<const uint4*>(fr + (size_t)y * row_bytes + off));
    }
    __syncthreads();
    // gray: thread -> column rx of seven rows (the column's clamp and byte offset once)
    if (threadIdx.x < CG * GRAY_GROUPS) {
        const int rx = threadIdx.x % CG, r0 = GRAY_ROWS * (threadIdx.x / CG);
        const int x = clampi(x0 - 4 + rx, 0, w - 1);
        const uint8_t* col = reinterpret_cast<const uint8_t*>(&sraw[0][0]) + (3 * x - byte0);
#pragma unroll
        for (int k = 0; k < GRAY_ROWS; ++k) {
            const int ry = r0 + k;
            if (ry >= CG) break;
            const uint8_t* p = col + ry * (int)(CRAW * sizeof(uint4));
            sg[ry][rx] = (uint8_t)((77 * p[0] + 150 * p[1] + 29 * p[2] + 128) >> 8);
        }
    }
    __syncthreads();
    // blur at the clamped position, so that the Sobel taps read Bl(clamp(y), clamp(x)): column map first;
    // thread -> column rx of six rows
    if (threadIdx.x < CB * BLUR_GROUPS) {
        const int rx = threadIdx.x % CB, r0 = BLUR_ROWS * (threadIdx.x / CB);
        const int gx0 = clampi(x0 - 2 + rx, 0, w - 1) - (x0 - 4);
#pragma unroll
        for (int k = 0; k < BLUR_ROWS; ++k) {
            const int gy = r0 + k;
            if (gy >= CG) break;
            const uint8_t* g = &sg[gy][gx0];
            sh[gy][rx] = (uint16_t)(g[-2] + 4 * g[-1] + 6 * g[0] + 4 * g[1] + g[2]);
        }
    }
    __syncthreads();
    // down the columns: thread -> column rx of six consecutive rows; away from the image's top and bottom their
    // five-tap windows are rows r0 .. r0 + 9 of the row sums, each read once
    if (threadIdx.x < CB * BLUR_GROUPS) {
        const int rx = threadIdx.x % CB, r0 = BLUR_ROWS * (threadIdx.x / CB);
        if (y0 >= 2 && y0 + CT + 1 <= h - 1) {               // no row of the blur tile is clamped: gy0 = ry + 2
            int v[BLUR_ROWS + 4];
#pragma unroll
            for (int k = 0; k < BLUR_ROWS + 4; ++k) v[k] = sh[r0 + k < CG ? r0 + k : CG - 1][rx];
#pragma unroll
            for (int k = 0; k < BLUR_ROWS; ++k) {
                const int ry = r0 + k;
                if (ry >= CB) break;
                const int acc = v[k] + 4 * v[k + 1] + 6 * v[k + 2] + 4 * v[k + 3] + v[k + 4];
                sb[ry][rx] = (uint8_t)((acc + 128) >> 8);
            }
        } else {
#pragma unroll
            for (int k = 0; k < BLUR_ROWS; ++k) {
                const int ry = r0 + k;
                if (ry >= CB) break;
                const int gy0 = clampi(y0 - 2 + ry, 0, h - 1) - (y0 - 4);
                const int acc = sh[gy0 - 2][rx] + 4 * sh[gy0 - 1][rx] + 6 * sh[gy0][rx] + 4 * sh[gy0 + 1][rx] + sh[gy0 + 2][rx];
                sb[ry][rx] = (uint8_t)((acc + 128) >> 8);
            }
        }
    }
    __syncthreads();
    // magnitude and direction sector of the tile grown by 1: thread -> column rx of five consecutive rows (their 3x3
    // neighbourhoods share rows), the sector in the four bits above the magnitude (at most 2 * 1020^2 < 2^21)
    if (threadIdx.x < CM * MAG_GROUPS) {
        const int rx = threadIdx.x % CM, r0 = MAG_ROWS * (threadIdx.x / CM);
        const int x = x0 - 1 + rx;
        const bool xin = x >= 0 && x < w;
#pragma unroll
        for (int k = 0; k < MAG_ROWS; ++k) {
            const int ry = r0 + k;
            if (ry >= CM) break;
            const int y = y0 - 1 + ry;
            uint32_t mv = 0;
            if (xin && y >= 0 && y < h) {
                const int by = ry + 1, bx = rx + 1;   // position in the blur tile
                const int gx = (sb[by - 1][bx + 1] + 2 * sb[by][bx + 1] + sb[by + 1][bx + 1]) -
                               (sb[by - 1][bx - 1] + 2 * sb[by][bx - 1] + sb[by + 1][bx - 1]);
                const int gy = (sb[by + 1][bx - 1] + 2 * sb[by + 1][bx] + sb[by + 1][bx + 1]) -
                               (sb[by - 1][bx - 1] + 2 * sb[by - 1][bx] + sb[by - 1][bx + 1]);
                const int ax = abs(gx), ay = abs(gy);
                // sector: 0 along the row, 1 down the column, 2 the diagonal (-1,-1)/(+1,+1), 3 the other one
                uint32_t sec;
                if (32768 * ay <= 13573 * ax) sec = 0;
                else if (32768 * ax <= 13573 * ay) sec = 1;
                else sec = ((gx > 0) == (gy > 0)) ? 2 : 3;
                mv = (uint32_t)(gx * gx + gy * gy) | (sec << 28);
            }
            smag[ry][rx] = (int)mv;
        }
    }
    __syncthreads();
    // a warp covers one row of the tile (the ballots), a thread four consecutive rows
    {
        const int ox = threadIdx.x & 31, x = x0 + ox;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int oy = 4 * (threadIdx.x >> 5) + k, y = y0 + oy;
            int cls = 0;
            if (y < h && x < w) {
                const int my = oy + 1, mx = ox + 1;
                const uint32_t mc = (uint32_t)smag[my][mx];
                const int mm = (int)(mc & 0x0fffffffu);
                const uint32_t sec = mc >> 28;
                const int dy = sec != 0 ? 1 : 0;
                const int dx = (sec == 0 || sec == 2) ? 1 : (sec == 3 ? -1 : 0);
                const int mneg = smag[my - dy][mx - dx] & 0x0fffffff, mpos = smag[my + dy][mx + dx] & 0x0fffffff;
                const bool keep = (mm > mneg) && (mm >= mpos);
                if (keep && mm >= hi2) cls = 2;
                else if (keep && mm >= lo2) cls = 1;
            }
            const uint32_t kept = __ballot_sync(0xffffffffu, cls > 0);
            const uint32_t strong = __ballot_sync(0xffffffffu, cls == 2);
            if (ox == 0 && y < h) {
                const size_t o = ((size_t)f * h + y) * words + blockIdx.x;
                bits_kept[o] = kept;
                bits_strong[o] = strong;
            }
        }
    }
}

// ---- hysteresis to the fixed point: one CTA per frame, both bit planes in shared memory.
// E starts as the strong plane and grows through 8-neighbours restricted to the kept plane; the closure is unique, so
// the order of the updates does not matter.  Every warp owns a strip of rows and sweeps it until nothing in it
// changes (at most HYST_INNER sweeps, synchronised inside the warp only), reading its neighbours' border rows as they
// stand (updates are monotone, so a stale read only delays); a round ends with a CTA-wide vote, and the fixed
// point is reached when a whole round changed nothing.  `max_iters` bounds the rounds.
constexpr int HYST_INNER = 64;
__global__ void __launch_bounds__(1024)
k_hysteresis(const uint32_t* __restrict__ bits_kept, uint32_t* __restrict__ bits_edge, int h, int words, int max_iters,
             int* __restrict__ status, const uint8_t* __restrict__ skip) {
    extern __shared__ uint32_t sh[];
    uint32_t* K = sh;                               // [h][words]
    volatile uint32_t* E = sh + (size_t)h * words;  // [h][words]
    const int f = blockIdx.x, n = h * words;
    if (skip && skip[f]) return;
    const uint32_t* gk = bits_kept + (size_t)f * n;
    uint32_t* ge = bits_edge + (size_t)f * n;
    for (int i = threadIdx.x; i < n; i += blockDim.x) { K[i] = gk[i]; E[i] = ge[i]; }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const int rows_per = (h + n_warps - 1) / n_warps;
    const int ya = min(h, warp * rows_per), yb = min(h, ya + rows_per);
    int it = 0;
    for (;;) {
        int changed = 0;
        for (int inner = 0; inner < HYST_INNER; ++inner) {
            int ch = 0;
            for (int i = ya * words + lane; i < yb * words; i += 32) {
                const uint32_t k = K[i], e = E[i];
                if (k == e) continue;
                const int y = i / words, wx = i - y * words;
                uint32_t acc = 0;
#pragma unroll
                for (int dy = -1; dy <= 1; ++dy) {
                    const int yy = y + dy;
                    if (yy < 0 || yy >= h) continue;
                    const volatile uint32_t* row = E + yy * words;
                    const uint32_t v = row[wx];
                    const uint32_t l = wx > 0 ? row[wx - 1] : 0u;
                    const uint32_t r = wx + 1 < words ? row[wx + 1] : 0u;
                    acc |= v | (v << 1) | (v >> 1) | (l >> 31) | (r << 31);
                }
                uint32_t ne = (e | acc) & k;
                for (;;) {   // run along the row inside the word
                    const uint32_t g = (ne | (ne << 1) | (ne >> 1)) & k;
                    if (g == ne) break;
                    ne = g;
                }
                if (ne != e) { E[i] = ne; ch = 1; }
            }
            if (!__any_sync(0xffffffffu, ch)) break;
            changed = 1;
        }
        if (!__syncthreads_or(changed)) break;
        if (++it >= max_iters) {
            if (threadIdx.x == 0) atomicMin(status, SALICACHE_E_NOCONVERGE);
            break;
        }
    }
    for (int i = threadIdx.x; i < n; i += blockDim.x) ge[i] = E[i];
}

// ---- sRGB -> CIE L*a*b* (D65) in double.  Cube root: a hardware log2 / exp2 seed in single precision
// (relative error below 1e-6) and one Newton step in double, y - (y^3 - t) / (3 y^2); the divisor only
// scales a 1e-6 correction, so its single-precision reciprocal is enough and the result is good to ~1e-12.
__device__ __forceinline__ double lab_f(double t) {
    const double d = 6.0 / 29.0;
    const float tf = fmaxf((float)t, 1e-6f);
    float y0;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y0) : "f"(__log2f(tf) * (1.0f / 3.0f)));
    const float r = __frcp_rn(3.0f * y0 * y0);
    const double y = (double)y0;
    const double cube = y - (y * y * y - t) * (double)r;
    const double lin = t * (1.0 / (3.0 * d * d)) + 4.0 / 29.0;
    return t > d * d * d ? cube : lin;
}
__device__ __forceinline__ void rgb_to_lab(const double* __restrict__ lut, int R, int G, int B, double& L, double& a,
                                           double& b) {
    double r = lut[R], g = lut[G], bl = lut[B];
    double X = 0.4124564 * r + 0.3575761 * g + 0.1804375 * bl;
    double Y = 0.2126729 * r + 0.7151522 * g + 0.0721750 * bl;
    double Z = 0.0193339 * r + 0.1191920 * g + 0.9503041 * bl;
    double fx = lab_f(X * (1.0 / 0.95047)), fy = lab_f(Y), fz = lab_f(Z * (1.0 / 1.08883));
    L = 116.0 * fy - 16.0;
    a = 500.0 * (fx - fy);
    b = 200.0 * (fy - fz);
}

// ---- colour branch + blend + patch mean.  One CTA per 2x2 patches (28x28 pixels), halo 3.
// Variances are taken about the LAB value of the tile's first pixel (variance is shift invariant),
// which keeps flat regions exactly zero and small contrasts accurate; the window sums stay in double
// because mean(x^2) - mean(x)^2 cancels.  With x = (dL, da, db) the sum of the three variances is
//   V = W[|x|^2] / n - (W[dL]^2 + W[da]^2 + W[db]^2) / n^2,    W[.] = 7x7 window sum,
// so four planes are summed, not six.
//   stage    the tile's bytes by 16-byte loads and the sRGB table into shared memory; warp 0 converts the
//            tile's first pixel (the shift)
//   convert  LAB of the 34x34 grown tile, minus the shift, and |x|^2 -> shared memory
//   then two planes at a time (the second plane's row sums lie over the staging area, dead by then, which keeps
//   four CTAs on an SM):
//   phase 2  one thread per (row, run of 4 columns): 7-column sums
//   phase 3  one thread per (column, run of 4 rows): 7-row sums
//   last     C, blend with the edge bit, patch partial sums
// Window sums of a run share their terms: the middle four once, then suffix sums to the left and prefix
// sums to the right (11 additions for 4 windows).
constexpr int ST = 28;
constexpr int SR = 3;
constexpr int SE = ST + 2 * SR;   // 34
constexpr int SLP = SE;           // row pitch of the planes: 17 16-byte units, odd, so the 16-byte loads that eight lanes
                                  // issue down eight rows fall on distinct banks
constexpr int HSP = ST + 2;       // row pitch of the row sums: 15 16-byte units, odd, for the same reason
constexpr int CRUN = 4;
constexpr int CNQ = 2 * SR + CRUN;   // 10 values feed 4 windows
constexpr int CROWS = 256 / SE;     // rows of the grown tile converted per sweep of the 256 threads (7)
constexpr int SRAW = 8;           // 16-byte chunks staged per row: 34 pixels = 102 bytes starting up to 15 bytes into a chunk

// w[k] = q[k] + ... + q[k+6], k = 0..3
__device__ __forceinline__ void window4(const double q[CNQ], double w[CRUN]) {
    double mid = (q[3] + q[4]) + (q[5] + q[6]);
    double s2 = q[2] + mid, s1 = q[1] + s2, s0 = q[0] + s1;
    double p8 = q[7] + q[8], p9 = p8 + q[9];
    w[0] = s0;
    w[1] = s1 + q[7];
    w[2] = s2 + p8;
    w[3] = mid + p9;
}

struct ColorStage {               // what the LAB stage reads; dead once the planes are filled
    double lut[256];
    uint4 raw[SE][SRAW];
};
struct ColorSmem {
    double plane[4][SE][SLP];     // dL, da, db, |x|^2
    double hs0[SE][HSP];          // 7-column sums of two planes at a time; the second set lies over the staging area
    union {
        ColorStage st;
        double hs1[SE][HSP];
    } u;
    double shift[3];
    double psum[8][4];
};

// ADAPTIVE = false: C = min(1, sqrt(V) * inv_sigma), blended and reduced to the patch scores here.
// ADAPTIVE = true:  the frame-adaptive colour term needs the image's mean V first: this kernel leaves sqrt(V) per
//                   pixel in `sqrt_v` and the tile's sum of V in `v_part`; k_color_adaptive finishes.
template <bool ADAPTIVE>
__global__ void __launch_bounds__(256, 4)
k_color_patch(const uint8_t* __restrict__ frames, size_t frame_bytes, PlaneGeom g, int patch,
              const double* __restrict__ lut, const uint32_t* __restrict__ bits_edge, int words, double inv_sigma,
              double w_edge, double w_color, float* __restrict__ s_out, const uint8_t* __restrict__ skip,
              float* __restrict__ sqrt_v, double* __restrict__ v_part) {
    extern __shared__ __align__(16) unsigned char cs_raw[];
    ColorSmem& sm = *reinterpret_cast<ColorSmem*>(cs_raw);
    const int f = blockIdx.z, x0 = blockIdx.x * ST, y0 = blockIdx.y * ST;
    if (skip && skip[f]) return;
    const int h = g.H, w = g.W;
    const uint8_t* fr = frames + (size_t)f * frame_bytes;
    const int row_bytes = 3 * w;
    const int xa = x0 >= SR ? x0 - SR : 0;
    const int byte0 = (3 * xa) & ~15;
    sm.u.st.lut[threadIdx.x] = __ldg(lut + threadIdx.x);
    for (int i = threadIdx.x; i < SE * SRAW; i += blockDim.x) {
        const int ry = i / SRAW, ch = i - ry * SRAW;
        const int y = clampi(y0 - SR + ry, 0, h - 1);
        const int off = byte0 + 16 * ch;
        if (off < row_bytes) sm.u.st.raw[ry][ch] = __ldg(reinterpret_cast<const uint4*>(fr + (size_t)y * row_bytes + off));
    }
    if (threadIdx.x >= 224) {          // the last warp: the shift, straight from global memory
        const uint8_t* p = fr + ((size_t)y0 * w + x0) * 3;
        double L0, a0, b0;
        rgb_to_lab(lut, p[0], p[1], p[2], L0, a0, b0);
        if (threadIdx.x == 224) { sm.shift[0] = L0; sm.shift[1] = a0; sm.shift[2] = b0; }
    }
    __syncthreads();
    {
        // thread -> column rx of rows r0, r0 + 7, ...: the column's clamp and byte offset are taken once
        const double L0 = sm.shift[0], a0 = sm.shift[1], b0 = sm.shift[2];
        const int rx = threadIdx.x % SE, r0 = threadIdx.x / SE;
        if (r0 < CROWS) {
            const int x = clampi(x0 - SR + rx, 0, w - 1);
            const uint8_t* col = reinterpret_cast<const uint8_t*>(&sm.u.st.raw[0][0]) + (3 * x - byte0);
#pragma unroll
            for (int k = 0; k < (SE + CROWS - 1) / CROWS; ++k) {
                const int ry = r0 + CROWS * k;
                if (ry < SE) {
                    const uint8_t* p = col + ry * (int)(SRAW * sizeof(uint4));
                    double L, a, b;
                    rgb_to_lab(sm.u.st.lut, p[0], p[1], p[2], L, a, b);
                    L -= L0; a -= a0; b -= b0;
                    sm.plane[0][ry][rx] = L;
                    sm.plane[1][ry][rx] = a;
                    sm.plane[2][ry][rx] = b;
                    sm.plane[3][ry][rx] = L * L + a * a + b * b;
                }
            }
        }
    }
    __syncthreads();
    const double inv_n = 1.0 / (double)((2 * SR + 1) * (2 * SR + 1));
    double acc0 = 0.0, acc1 = 0.0, acc2 = 0.0, acc3 = 0.0;   // the four patches of the tile
    // phase 3: (column, run of 4 rows); a warp holds the 28 columns of one run of rows (its last four lanes idle), so
    // that its 8-byte loads are consecutive
    const int ox = threadIdx.x & 31, oy0 = CRUN * (threadIdx.x >> 5);
    const bool owner = ox < ST && oy0 < ST;
    double M[CRUN] = {0.0, 0.0, 0.0, 0.0}, S2[CRUN] = {0.0, 0.0, 0.0, 0.0};
    for (int cp = 0; cp < 2; ++cp) {                            // two planes' row sums in shared memory at a time
        if (threadIdx.x < SE * (ST / CRUN)) {
            const int ry = threadIdx.x % SE, run = threadIdx.x / SE;   // lanes run down the rows: conflict-free 16-byte accesses
            const int cx = CRUN * run;                          // windows cx .. cx+3 read columns cx .. cx+9 of the grown tile
#pragma unroll
            for (int pl = 0; pl < 2; ++pl) {
                const double2* src = reinterpret_cast<const double2*>(&sm.plane[2 * cp + pl][ry][cx]);
                double q[CNQ];
#pragma unroll
                for (int k = 0; k < CNQ / 2; ++k) {
                    double2 v = src[k];
                    q[2 * k] = v.x;
                    q[2 * k + 1] = v.y;
                }
                double w1[CRUN];
                window4(q, w1);
                double2* dst = reinterpret_cast<double2*>(pl ? &sm.u.hs1[ry][cx] : &sm.hs0[ry][cx]);
                dst[0] = make_double2(w1[0], w1[1]);
                dst[1] = make_double2(w1[2], w1[3]);
            }
        }
        __syncthreads();
        if (owner) {
#pragma unroll
            for (int pl = 0; pl < 2; ++pl) {
                double q[CNQ];
#pragma unroll
                for (int k = 0; k < CNQ; ++k) q[k] = pl ? sm.u.hs1[oy0 + k][ox] : sm.hs0[oy0 + k][ox];
                double w1[CRUN];
                window4(q, w1);
#pragma unroll
                for (int k = 0; k < CRUN; ++k) {
                    if (2 * cp + pl < 3) M[k] += w1[k] * w1[k];
                    else S2[k] = w1[k];
                }
            }
        }
        __syncthreads();
    }
    if (owner) {
        const int x = x0 + ox;
#pragma unroll
        for (int k = 0; k < CRUN; ++k) {
            const int oy = oy0 + k, y = y0 + oy;
            const double V = fmax(S2[k] * inv_n - M[k] * (inv_n * inv_n), 0.0);
            if (ADAPTIVE) {
                sqrt_v[((size_t)f * h + y) * w + x] = sqrtf((float)V);
                acc0 += V;
                continue;
            }
            double C = (double)sqrtf((float)V) * inv_sigma;      // a rounding of 6e-8 relative: far inside the tolerance of s
            C = fmin(C, 1.0);
            uint32_t e = (bits_edge[((size_t)f * h + y) * words + (x >> 5)] >> (x & 31)) & 1u;
            double S = w_edge * (double)e + w_color * C;
            S = fmin(fmax(S, 0.0), 1.0);
            bool lower = oy >= patch, right = ox >= patch;
            acc0 += (!lower && !right) ? S : 0.0;
            acc1 += (!lower && right) ? S : 0.0;
            acc2 += (lower && !right) ? S : 0.0;
            acc3 += (lower && right) ? S : 0.0;
        }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        acc0 += __shfl_xor_sync(0xffffffffu, acc0, o);
        acc1 += __shfl_xor_sync(0xffffffffu, acc1, o);
        acc2 += __shfl_xor_sync(0xffffffffu, acc2, o);
        acc3 += __shfl_xor_sync(0xffffffffu, acc3, o);
    }
    if ((threadIdx.x & 31) == 0) {
        double* ps = sm.psum[threadIdx.x >> 5];
        ps[0] = acc0; ps[1] = acc1; ps[2] = acc2; ps[3] = acc3;
    }
    __syncthreads();
    if (ADAPTIVE) {
        if (threadIdx.x == 0) {
            double tot = 0.0;
            for (int wp = 0; wp < 8; ++wp) tot += sm.psum[wp][0];                 // fixed order: deterministic
            v_part[((size_t)f * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x] = tot;
        }
        return;
    }
    if (threadIdx.x < 4) {
        double tot = 0.0;
        for (int wp = 0; wp < 8; ++wp) tot += sm.psum[wp][threadIdx.x];      // fixed order: deterministic
        int py = blockIdx.y * 2 + threadIdx.x / 2, px = blockIdx.x * 2 + threadIdx.x % 2;
        s_out[(size_t)f * g.n_tok + patch_token(g, py, px)] = (float)(tot / (double)(patch * patch));
    }
}

// ---- frame-adaptive colour term, second pass.  One CTA per 2x2 patches: the image's mean V from the tile sums
// (every CTA adds them in the same fixed order), sigma = max(sqrt(mean V), sigma_min), then
// C = min(1, sqrt(V) / (kappa sigma)), the blend with the edge bit and the patch means.
__global__ void __launch_bounds__(256)
k_color_adaptive(const float* __restrict__ sqrt_v, const double* __restrict__ v_part, PlaneGeom g, int patch,
                 const uint32_t* __restrict__ bits_edge, int words, double kappa, double sigma_min, double w_edge,
                 double w_color, float* __restrict__ s_out, const uint8_t* __restrict__ skip) {
    __shared__ double red[256];
    __shared__ double psum[8][4];
    const int f = blockIdx.z, x0 = blockIdx.x * ST, y0 = blockIdx.y * ST;
    if (skip && skip[f]) return;
    const int h = g.H, w = g.W, n_tiles = gridDim.x * gridDim.y;
    double part = 0.0;
    for (int i = threadIdx.x; i < n_tiles; i += 256) part += v_part[(size_t)f * n_tiles + i];
    red[threadIdx.x] = part;
    __syncthreads();
    for (int o = 128; o; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    double sigma = sqrt(red[0] / ((double)h * (double)w));
    sigma = fmax(sigma, sigma_min);
    const double inv = sigma > 0.0 ? 1.0 / (kappa * sigma) : 0.0;
    double acc0 = 0.0, acc1 = 0.0, acc2 = 0.0, acc3 = 0.0;
    for (int i = threadIdx.x; i < ST * ST; i += 256) {
        const int oy = i / ST, ox = i - oy * ST;
        const int y = y0 + oy, x = x0 + ox;
        const double C = fmin((double)sqrt_v[((size_t)f * h + y) * w + x] * inv, 1.0);
        const uint32_t e = (bits_edge[((size_t)f * h + y) * words + (x >> 5)] >> (x & 31)) & 1u;
        double S = w_edge * (double)e + w_color * C;
        S = fmin(fmax(S, 0.0), 1.0);
        const bool lower = oy >= patch, right = ox >= patch;
        acc0 += (!lower && !right) ? S : 0.0;
        acc1 += (!lower && right) ? S : 0.0;
        acc2 += (lower && !right) ? S : 0.0;
        acc3 += (lower && right) ? S : 0.0;
    }
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
        for (int wp = 0; wp < 8; ++wp) tot += psum[wp][threadIdx.x];
        int py = blockIdx.y * 2 + threadIdx.x / 2, px = blockIdx.x * 2 + threadIdx.x % 2;
        s_out[(size_t)f * g.n_tok + patch_token(g, py, px)] = (float)(tot / (double)(patch * patch));
    }
}

inline unsigned blocks_for(long long n, int threads) { return (unsigned)((n + threads - 1) / threads); }

}  // namespace

static size_t color_smem() { return sizeof(ColorSmem); }

int sc_saliency_init(int max_h, int max_words) {
    SC_CHECK(cudaFuncSetAttribute(k_color_patch<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)color_smem()));
    SC_CHECK(cudaFuncSetAttribute(k_color_patch<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)color_smem()));
    size_t smem = (size_t)2 * max_h * max_words * sizeof(uint32_t);
    if (smem > 227 * 1024) return SALICACHE_E_SHAPE;
    // always the full opt-in limit: the attribute belongs to the function, not to a context, so a
    // later context with smaller frames must not lower it under an earlier context with larger ones
    SC_CHECK(cudaFuncSetAttribute(k_hysteresis, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    return SALICACHE_OK;
}

int sc_box_down2(const uint8_t* d_src, int H, int W, int B, uint8_t* d_dst, cudaStream_t st) {
    k_box_down2<<<blocks_for((long long)(H / 2) * (W / 2) * B, 256), 256, 0, st>>>(d_src, H, W, B, d_dst);
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}

int sc_saliency(salicache_ctx* c, const PlaneGeom& g, const uint8_t* d_frames, size_t frame_bytes, int B, float* d_s,
                const uint8_t* d_skip, cudaStream_t st) {
    const salicache_params& p = c->p;
    const int words = (g.W + 31) / 32;
    for (int b0 = 0; b0 < B; b0 += c->chunk) {
        int nb = B - b0 < c->chunk ? B - b0 : c->chunk;
        const uint8_t* fr = d_frames + (size_t)b0 * frame_bytes;
        const uint8_t* skip = d_skip ? d_skip + b0 : nullptr;
        dim3 gc((g.W + CT - 1) / CT, (g.H + CT - 1) / CT, nb);
        k_canny_classify<<<gc, 256, 0, st>>>(fr, frame_bytes, g.H, g.W, words, p.canny_lo * p.canny_lo,
                                             p.canny_hi * p.canny_hi, c->bits_kept, c->bits_edge, skip);
        size_t smem = (size_t)2 * g.H * words * sizeof(uint32_t);
        k_hysteresis<<<nb, 1024, smem, st>>>(c->bits_kept, c->bits_edge, g.H, words, p.hyst_max_iters, c->d_status, skip);
        dim3 gs(g.W / ST, g.H / ST, nb);
        float* s_dst = d_s + (size_t)b0 * g.n_tok;
        if (p.color_norm == 0) {
            k_color_patch<false><<<gs, 256, color_smem(), st>>>(fr, frame_bytes, g, p.patch, c->lut, c->bits_edge, words,
                                                                1.0 / p.sigma_ref, p.w_edge, p.w_color, s_dst, skip, nullptr, nullptr);
        } else {
            k_color_patch<true><<<gs, 256, color_smem(), st>>>(fr, frame_bytes, g, p.patch, c->lut, c->bits_edge, words, 0.0,
                                                               p.w_edge, p.w_color, s_dst, skip, c->sqrt_v, c->v_part);
            k_color_adaptive<<<gs, 256, 0, st>>>(c->sqrt_v, c->v_part, g, p.patch, c->bits_edge, words, p.color_kappa,
                                                 p.color_sigma_min, p.w_edge, p.w_color, s_dst, skip);
            c->launches++;
        }
        c->launches += 3;
    }
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}
