// Decode attention over the mixed-precision store with the dequantisation fused in (Eq. 2; Sec. III-C:
// "just-in-time" dequantisation inside the attention computation).  One query per layer and head attends
// to every row the three pools hold; codes are expanded in registers and never written back.
//
//   score_j = q_h . K^_{j,h} / sqrt(D),   p = softmax_j(score),   out_h = sum_j p_j V^_{j,h}
//
// Split over the rows: per layer and head a few dozen partial results of each of three kernels (one per tier),
// merged by a fourth.  All three walk 16 rows per warp at a time through matrix instructions: the FP16 rows as
// they are, the INT8 and INT4 rows after expanding the codes to binary16 in registers; with grouped queries up to
// 4 query heads of a key/value head are the columns of those instructions.  Online softmax and single precision
// accumulation in all.
#include <cuda_fp16.h>

#include <algorithm>
#include <math.h>

#include "common.cuh"

namespace {

constexpr int AT_D = 128;           // head size = threads per CTA = quantisation group
constexpr int AT_WARPS = AT_D / 32;
constexpr int AT_CHUNKS = 64;       // partial results of the INT4 kernel per (layer, head)
constexpr int AT_CH16 = 32;         // ... of the FP16 kernel (at most), and
constexpr int AT_CH8 = 32;          // ... of the INT8 kernel
constexpr int AT_REC = AT_D + 2;    // partial record: 128 sums, running maximum, running denominator
constexpr int AT_RECS = AT_CH16 + AT_CH8 + AT_CHUNKS;   // records per (layer, head): FP16, then INT8, then INT4 chunks
constexpr int AT_REC8 = AT_CH16, AT_REC4 = AT_CH16 + AT_CH8;      // first record of the INT8 and of the INT4 kernel

struct AtPools {
    const uint8_t* fp16_pool;
    const uint8_t* int8_codes;
    const uint8_t* int8_scale;
    const uint8_t* int4_codes;
    const uint8_t* int4_sz;
    long long cap16, cap8, cap4;
};

__device__ __forceinline__ float h2f(uint16_t b) { return __half2float(__ushort_as_half(b)); }
__device__ __forceinline__ float2 w2f(uint32_t w) { return __half22float2(*reinterpret_cast<const __half2*>(&w)); }

__device__ __forceinline__ uint32_t hsub2u(uint32_t a, uint32_t b) {
    __half2 r = __hsub2(*reinterpret_cast<const __half2*>(&a), *reinterpret_cast<const __half2*>(&b));
    return *reinterpret_cast<const uint32_t*>(&r);
}
__device__ __forceinline__ float block_max(float v, float* red) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
#pragma unroll
    for (int k = 1; k < AT_WARPS; ++k) r = fmaxf(r, red[k]);
    __syncthreads();
    return r;
}
__device__ __forceinline__ float block_sum(float v, float* red) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = 0.0f;
#pragma unroll
    for (int k = 0; k < AT_WARPS; ++k) r += red[k];      // fixed order: deterministic
    __syncthreads();
    return r;
}

// ---- INT4 rows on the tensor cores.  A single query is a matrix-vector product, but forming it with
// 16x8x16 matrix instructions (most of the 8 columns idle) still costs far fewer instructions per multiply-add
// than scalar code, which is what this stage is short of: it is bound by instruction issue, not by arithmetic.
//   scores  A = 16 key rows x 16 dimensions (codes expanded to binary16), B = the query in column 0
//   values  A = 16 dimensions x 16 value rows (codes, transposed), B = the 16 softmax weights (times the
//           value scale) in column 0 (high half) and column 1 (low half of a two-term binary16 split, so that
//           the weights keep 22 bits)
// One warp walks 16-row tiles with its own online softmax; the four warps of a CTA are merged at the end.
// The k index of a matrix instruction may be permuted freely as long as A and B agree, and so may the
// assignment of the 16 rows of A to dimensions; both are chosen so that a lane reads contiguous bytes.
__device__ __forceinline__ uint4 ld_stream16(const uint8_t* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ld_stream8(const uint8_t* p) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
// (a & b) | c in one instruction.  The compiler splits the expression into two when b and c are both literals
// (a logic instruction takes one immediate), so the masks and magic numbers below live in registers.
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// Codes to binary16 pairs.  A nibble in bits 0..3 of each half is OR-ed into the mantissa of 1024 (0x6400, unit in
// the last place 1), one in bits 4..7 into that of 64 (0x5400, unit 1/16): either adds exactly its value.
struct NibConst {
    uint32_t mask_lo, mask_hi, magic_lo, magic_hi;
    __device__ __forceinline__ void init() {        // opaque to the compiler, so that they stay in registers
        asm volatile("mov.b32 %0, 0x000f000f;" : "=r"(mask_lo));
        asm volatile("mov.b32 %0, 0x00f000f0;" : "=r"(mask_hi));
        asm volatile("mov.b32 %0, 0x64006400;" : "=r"(magic_lo));
        asm volatile("mov.b32 %0, 0x54005400;" : "=r"(magic_hi));
    }
    __device__ __forceinline__ uint32_t lo(uint32_t t) const { return hsub2u(and_or(t, mask_lo, magic_lo), magic_lo); }
    __device__ __forceinline__ uint32_t hi(uint32_t t) const { return hsub2u(and_or(t, mask_hi, magic_hi), magic_hi); }
    // the four pairs (e0,e4) (e1,e5) (e2,e6) (e3,e7) of a word of 8 nibbles
    __device__ __forceinline__ void word(uint32_t x, uint32_t out[4]) const {
        const uint32_t y = x >> 8;
        out[0] = lo(x);
        out[1] = hi(x);
        out[2] = lo(y);
        out[3] = hi(y);
    }
};

// What one lane loads of a tile of 16 INT4 rows: the keys of rows g8 and g8 + 8 (32 dimensions at 32 * c4), the
// values of rows 2 c4, 2 c4 + 1, 2 c4 + 8, 2 c4 + 9 (16 dimensions at 16 * g8) and the (scale, zero) pairs of
// the one row whose softmax weight it computes: g8 + 8 * (c4 & 1).
struct I4Tile {
    uint4 ka, kb;
    uint2 v0, v1, v2, v3;
    uint32_t ks, vs;
};
// The lane's addresses in its warp's first tile.  PITCH (bytes per row of codes) and NG ((scale, zero) pairs per
// row) are compile-time constants for the common shapes, so that the row offsets fold into the loads.
template <int PITCH, int NG>
struct I4Addr {
    const uint8_t* k;        // key codes of row g8
    const uint8_t* v;        // value codes of row 2 c4
    const uint32_t* ks;      // key (scale, zero) of the lane's own row
    const uint32_t* vs;      // value (scale, zero) of the lane's own row
    size_t pitch_rt, ng_rt;
    __device__ __forceinline__ size_t pitch() const { return PITCH ? (size_t)PITCH : pitch_rt; }
    __device__ __forceinline__ size_t ng() const { return NG ? (size_t)NG : ng_rt; }
};
// FULL: all 16 rows exist.  Otherwise rows at or beyond r1 read as zero codes and are not touched.
template <bool FULL, int PITCH, int NG>
__device__ __forceinline__ void i4_load(I4Tile& x, const I4Addr<PITCH, NG>& a, long long tile, long long t0, long long r1, int g8,
                                        int c4) {
    const size_t d = (size_t)(tile - t0);
    const size_t P = a.pitch();
    const uint8_t* k = a.k + d * P;
    const uint8_t* v = a.v + d * P;
    const uint32_t* ks = a.ks + d * a.ng();
    const uint32_t* vs = a.vs + d * a.ng();
    if (FULL) {
        x.ka = ld_stream16(k);
        x.kb = ld_stream16(k + 8 * P);
        x.v0 = ld_stream8(v);
        x.v1 = ld_stream8(v + P);
        x.v2 = ld_stream8(v + 8 * P);
        x.v3 = ld_stream8(v + 9 * P);
        x.ks = __ldg(ks);
        x.vs = __ldg(vs);
    } else {
        x.ka = x.kb = make_uint4(0, 0, 0, 0);
        x.v0 = x.v1 = x.v2 = x.v3 = make_uint2(0, 0);
        x.ks = x.vs = 0;
        const long long ra = tile + g8, rv = tile + 2 * c4;
        if (ra < r1) x.ka = ld_stream16(k);
        if (ra + 8 < r1) x.kb = ld_stream16(k + 8 * P);
        if (ra + 8 * (c4 & 1) < r1) {
            x.ks = __ldg(ks);
            x.vs = __ldg(vs);
        }
        if (rv < r1) x.v0 = ld_stream8(v);
        if (rv + 1 < r1) x.v1 = ld_stream8(v + P);
        if (rv + 8 < r1) x.v2 = ld_stream8(v + 8 * P);
        if (rv + 9 < r1) x.v3 = ld_stream8(v + 9 * P);
    }
}
template <int PITCH, int NG>
__device__ __forceinline__ void i4_fetch(I4Tile& x, const I4Addr<PITCH, NG>& a, long long tile, long long t0, long long r1, int g8,
                                         int c4) {
    if (tile + 16 <= r1) i4_load<true>(x, a, tile, t0, r1, g8, c4);
    else i4_load<false>(x, a, tile, t0, r1, g8, c4);      // loads nothing at all once tile >= r1
}

// Running state of a warp: m is its maximum (the same in every lane); den and zacc are per-lane partial sums;
// acc[b] holds, in the lanes with c4 == 0, dimensions 16 g8 + 2 b (.x high, .y low) and 16 g8 + 2 b + 1 (.z, .w).
struct I4State {
    float acc[8][4];
    float m, den, zacc, F;
};

__device__ __forceinline__ void i4_tile(I4State& st, const I4Tile& x, const uint32_t (&qf)[8][2], const NibConst& nc, long long tile,
                                        long long r1, float rs, float qsum, int g8, int c4) {
    // ---- scores: the query sits in columns 0 and 2 of B, so that the lanes with c4 == 0 receive the products
    // of rows g8 and g8 + 8 in column 0 and the lanes with c4 == 1 the same two in column 2
    float sc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    {
        const uint32_t wa[4] = {x.ka.x, x.ka.y, x.ka.z, x.ka.w}, wb[4] = {x.kb.x, x.kb.y, x.kb.z, x.kb.w};
#pragma unroll
        for (int w4 = 0; w4 < 4; ++w4) {
            uint32_t pa[4], pb[4];
            nc.word(wa[w4], pa);
            nc.word(wb[w4], pb);
            mma16816(sc, pa[0], pb[0], pa[1], pb[1], qf[2 * w4][0], qf[2 * w4][1]);
            mma16816(sc, pa[2], pb[2], pa[3], pb[3], qf[2 * w4 + 1][0], qf[2 * w4 + 1][1]);
        }
    }
    // one row per lane: c4 == 0 takes row g8, c4 == 1 takes row g8 + 8; the other lanes have none
    const bool own = c4 < 2 && tile + g8 + 8 * c4 < r1;
    const float2 kz = w2f(x.ks), vz = w2f(x.vs);    // (scale, zero); both 0 for an absent row
    const float s = own ? rs * ((c4 ? sc[2] : sc[0]) * kz.x + qsum * kz.y) : -INFINITY;
    const float sv = own ? vz.x : 0.0f;
    // ---- online softmax of this warp.  The maximum rarely moves after the first tiles and the scale F
    // almost never: one vote decides whether the reductions and the rescaling of the sums are needed.
    if (__any_sync(0xffffffffu, s > st.m || sv * st.F >= 32768.0f)) {
        const float m_new = fmaxf(st.m, warp_max(s));
        const float corr = st.m == -INFINITY ? 0.0f : __expf(st.m - m_new);
        st.m = m_new;
        // keep weight * scale * F below 32768 (binary16): F only ever shrinks, by powers of two
        const float smax = warp_max(sv);
        float Fn = st.F;
        for (int k = 0; k < 40 && smax * Fn >= 32768.0f; ++k) Fn *= 0.5f;
        const float rescale = corr * (Fn / st.F);
        st.F = Fn;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
#pragma unroll
            for (int i = 0; i < 4; ++i) st.acc[b][i] *= rescale;
        }
        st.den *= corr;
        st.zacc *= corr;
    }
    const float pr = __expf(s - st.m);              // 0 for a lane without a row
    st.den += pr;
    st.zacc += pr * vz.y;
    // the weight as a two-term binary16 split (high, low)
    uint32_t pack;
    {
        const float w = pr * sv * st.F;
        const __half hi = __float2half_rn(w);
        const __half lo = __float2half_rn(w - __half2float(hi));
        pack = (uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16);
    }
    // B fragment of the second product: column 0 = high halves, column 1 = low halves, k = tile rows as loaded.
    // Row r of the tile was weighted by lane 4 * (r % 8) + r / 8.
    const uint32_t x1 = __shfl_sync(0xffffffffu, pack, 8 * c4), x2 = __shfl_sync(0xffffffffu, pack, 8 * c4 + 4);
    const uint32_t y1 = __shfl_sync(0xffffffffu, pack, 8 * c4 + 1), y2 = __shfl_sync(0xffffffffu, pack, 8 * c4 + 5);
    const uint32_t psel = g8 == 0 ? 0x5410u : 0x7632u;
    const uint32_t b0 = g8 < 2 ? __byte_perm(x1, x2, psel) : 0u, b1 = g8 < 2 ? __byte_perm(y1, y2, psel) : 0u;
    // ---- values: instruction b takes byte b of the lane's 8 bytes of each row: dimensions 16 g8 + 2 b (A row g8)
    // and 16 g8 + 2 b + 1 (A row g8 + 8)
    {
        const uint32_t w0[2] = {x.v0.x, x.v0.y}, w1[2] = {x.v1.x, x.v1.y}, w2[2] = {x.v2.x, x.v2.y}, w3[2] = {x.v3.x, x.v3.y};
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            const uint32_t sel = (uint32_t)((b & 3) | ((b & 3) << 4) | ((4 + (b & 3)) << 8) | ((4 + (b & 3)) << 12));
            const uint32_t t1 = __byte_perm(w0[b >> 2], w1[b >> 2], sel);      // bytes (row 2 c4: b, -, row 2 c4 + 1: b, -)
            const uint32_t t2 = __byte_perm(w2[b >> 2], w3[b >> 2], sel);
            mma16816(st.acc[b], nc.lo(t1), nc.hi(t1), nc.lo(t2), nc.hi(t2), b0, b1);
        }
    }
}

template <int PITCH, int NG>
__global__ void __launch_bounds__(AT_D)
k_attend_int4(const __half* __restrict__ q, AtPools pp, const long long* __restrict__ fill, int H, int gq, int ng, int min_rows,
              float* __restrict__ ws) {
    __shared__ __align__(16) float qs[AT_D];
    __shared__ __align__(16) __half qp[AT_D];       // every 8 elements ordered 0 4 1 5 2 6 3 7
    __shared__ float red[AT_WARPS];
    __shared__ float wpart[AT_WARPS][AT_D];
    __shared__ float wstat[AT_WARPS][2];
    const int hq = blockIdx.x, c = blockIdx.y, l = blockIdx.z, t = threadIdx.x;
    const int h = hq / gq, Hq = H * gq;          // query head hq reads key/value head h
    const int lane = t & 31, wid = t >> 5, g8 = lane >> 2, c4 = lane & 3;
    const int HD = H * AT_D;
    const long long n4 = min(fill[2], pp.cap4);
    // whole tiles per chunk, and at least min_rows rows: a cache that is not huge is spread over fewer CTAs (the
    // rest leave at once), so that the fixed cost of a CTA, staging the query and merging its warps, is paid less often
    const long long per = max((long long)min_rows, ((n4 + gridDim.y - 1) / gridDim.y + 15) / 16 * 16);
    const long long r0 = (long long)c * per, r1 = min(n4, r0 + per);
    if (r0 >= r1) {                                 // nothing in this chunk: a record the merge skips
        if (t == 0) {
            float* rec = ws + (((size_t)l * Hq + hq) * AT_RECS + AT_REC4 + c) * AT_REC;
            rec[AT_D] = -INFINITY;
            rec[AT_D + 1] = 0.0f;
        }
        return;
    }
    {
        const __half qv = q[((size_t)l * Hq + hq) * AT_D + t];
        const int e = t & 7;
        qs[t] = __half2float(qv);
        qp[(t & ~7) | ((e & 3) * 2 + (e >> 2))] = qv;
    }
    __syncthreads();
    const float rs = rsqrtf((float)AT_D);
    const float qsum = block_sum(qs[t], red);
    const int g = ng == 1 ? 0 : h;
    // the query as B fragments: instruction j = 2 * word + u of a lane's 32 dimensions takes the pairs
    // (e[2u], e[2u+4]) and (e[2u+1], e[2u+5]) of octet 4 * c4 + word; columns 0 and 2 (lanes 0..3 and 8..11)
    uint32_t qf[8][2];
    {
        const uint32_t* qp32 = reinterpret_cast<const uint32_t*>(qp);
        const bool has = g8 == 0 || g8 == 2;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int oct = 4 * c4 + (j >> 1), u = j & 1;
            qf[j][0] = has ? qp32[oct * 4 + 2 * u] : 0u;
            qf[j][1] = has ? qp32[oct * 4 + 2 * u + 1] : 0u;
        }
    }
    const long long t0 = r0 + 16 * wid;             // this warp's first tile
    I4Addr<PITCH, NG> ad;
    ad.pitch_rt = (size_t)(HD / 2);
    ad.ng_rt = (size_t)ng;
    const size_t own_row = (size_t)(t0 + g8 + 8 * (c4 & 1));
    ad.k = pp.int4_codes + ((size_t)(2 * l) * pp.cap4 + (size_t)(t0 + g8)) * ad.pitch() + (size_t)h * (AT_D / 2) + 16 * c4;
    ad.v = pp.int4_codes + ((size_t)(2 * l + 1) * pp.cap4 + (size_t)(t0 + 2 * c4)) * ad.pitch() + (size_t)h * (AT_D / 2) + 8 * g8;
    ad.ks = reinterpret_cast<const uint32_t*>(pp.int4_sz) + ((size_t)(2 * l) * pp.cap4 + own_row) * ad.ng() + g;
    ad.vs = reinterpret_cast<const uint32_t*>(pp.int4_sz) + ((size_t)(2 * l + 1) * pp.cap4 + own_row) * ad.ng() + g;
    NibConst nc;
    nc.init();
    I4State st;
#pragma unroll
    for (int b = 0; b < 8; ++b) st.acc[b][0] = st.acc[b][1] = st.acc[b][2] = st.acc[b][3] = 0.0f;
    st.m = -INFINITY;
    st.den = st.zacc = 0.0f;
    st.F = 4096.0f;                                 // the weights are scaled by a power of two before the binary16 split
    constexpr long long STEP = 16 * AT_WARPS;
    I4Tile xa, xb;                                  // two tiles in turn: one is consumed while the other is in flight
    long long tile = t0;
    if (tile < r1) {
        i4_fetch(xa, ad, tile, t0, r1, g8, c4);
        for (;;) {
            i4_fetch(xb, ad, tile + STEP, t0, r1, g8, c4);
            i4_tile(st, xa, qf, nc, tile, r1, rs, qsum, g8, c4);
            tile += STEP;
            if (tile >= r1) break;
            i4_fetch(xa, ad, tile + STEP, t0, r1, g8, c4);
            i4_tile(st, xb, qf, nc, tile, r1, rs, qsum, g8, c4);
            tile += STEP;
            if (tile >= r1) break;
        }
    }
    // ---- this warp's result
    const float den = warp_sum(st.den);
    const float zs = warp_sum(st.zacc);
    if (c4 == 0) {
        const float invF = 1.0f / st.F;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            wpart[wid][16 * g8 + 2 * b] = (st.acc[b][0] + st.acc[b][1]) * invF + zs;
            wpart[wid][16 * g8 + 2 * b + 1] = (st.acc[b][2] + st.acc[b][3]) * invF + zs;
        }
    }
    if (lane == 0) {
        wstat[wid][0] = st.m;
        wstat[wid][1] = den;
    }
    __syncthreads();
    float M = wstat[0][0];
#pragma unroll
    for (int k = 1; k < AT_WARPS; ++k) M = fmaxf(M, wstat[k][0]);
    float sum = 0.0f, dsum = 0.0f;
    if (M != -INFINITY) {
#pragma unroll
        for (int k = 0; k < AT_WARPS; ++k) {
            const float e = wstat[k][0] == -INFINITY ? 0.0f : __expf(wstat[k][0] - M);
            sum += e * wpart[k][t];
            dsum += e * wstat[k][1];
        }
    }
    float* rec = ws + (((size_t)l * Hq + hq) * AT_RECS + AT_REC4 + c) * AT_REC;
    rec[t] = sum;
    if (t == 0) {
        rec[AT_D] = M;
        rec[AT_D + 1] = dsum;
    }
}

// ---- INT4 rows, grouped queries: up to 4 of the query heads that share a key/value head (queries q0 .. q0 + gqn - 1
// of each group; larger groups take several launches) are the columns of the matrix instructions, so the codes of a
// tile are expanded once for all of them.  Query j sits in column 2 j of
// the score product; lane (g8, c4) therefore finds the products of query c4 with rows g8 and g8 + 8 in its own
// accumulator, and keeps that query's softmax statistics (shared by the 8 lanes with the same c4).  In the value
// product the weights of query j fill columns 2 j (high halves) and 2 j + 1 (low halves), so every lane's
// accumulators belong to query c4: dimensions 16 g8 + 2 b and 16 g8 + 2 b + 1.
constexpr int GQ_MAX = 4;

struct G4Tile {
    uint4 ka, kb;                  // keys of rows g8 and g8 + 8: 32 dimensions at 32 * c4
    uint2 v0, v1, v2, v3;          // values of rows 2 c4, 2 c4 + 1, 2 c4 + 8, 2 c4 + 9: 16 dimensions at 16 * g8
    uint32_t ksa, ksb, vsa, vsb;   // (scale, zero) of the keys and values of rows g8 and g8 + 8
};
struct G4Addr {
    const uint8_t* k;
    const uint8_t* v;
    const uint32_t* ks;
    const uint32_t* vs;
    size_t pitch, ng;
};
__device__ __forceinline__ void g4_fetch(G4Tile& x, const G4Addr& a, long long tile, long long t0, long long r1, int g8, int c4) {
    const size_t d = (size_t)(tile - t0), P = a.pitch;
    const uint8_t* k = a.k + d * P;
    const uint8_t* v = a.v + d * P;
    const uint32_t* ks = a.ks + d * a.ng;
    const uint32_t* vs = a.vs + d * a.ng;
    if (tile + 16 <= r1) {
        x.ka = ld_stream16(k);
        x.kb = ld_stream16(k + 8 * P);
        x.v0 = ld_stream8(v);
        x.v1 = ld_stream8(v + P);
        x.v2 = ld_stream8(v + 8 * P);
        x.v3 = ld_stream8(v + 9 * P);
        x.ksa = __ldg(ks);
        x.ksb = __ldg(ks + 8 * a.ng);
        x.vsa = __ldg(vs);
        x.vsb = __ldg(vs + 8 * a.ng);
    } else {                                        // rows at or beyond r1 read as zero codes and are not touched
        x.ka = x.kb = make_uint4(0, 0, 0, 0);
        x.v0 = x.v1 = x.v2 = x.v3 = make_uint2(0, 0);
        x.ksa = x.ksb = x.vsa = x.vsb = 0;
        const long long ra = tile + g8, rv = tile + 2 * c4;
        if (ra < r1) { x.ka = ld_stream16(k); x.ksa = __ldg(ks); x.vsa = __ldg(vs); }
        if (ra + 8 < r1) { x.kb = ld_stream16(k + 8 * P); x.ksb = __ldg(ks + 8 * a.ng); x.vsb = __ldg(vs + 8 * a.ng); }
        if (rv < r1) x.v0 = ld_stream8(v);
        if (rv + 1 < r1) x.v1 = ld_stream8(v + P);
        if (rv + 8 < r1) x.v2 = ld_stream8(v + 8 * P);
        if (rv + 9 < r1) x.v3 = ld_stream8(v + 9 * P);
    }
}
// max / sum over the 8 lanes that share c4 (one query)
__device__ __forceinline__ float group_max(float v) {
#pragma unroll
    for (int o = 16; o >= 4; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float group_sum(float v) {
#pragma unroll
    for (int o = 16; o >= 4; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ void g4_tile(I4State& st, const G4Tile& x, const uint32_t (&qf)[8][2], const NibConst& nc, long long tile,
                                        long long r1, float rs, float qsum, int g8, int c4) {
    float sc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    {
        const uint32_t wa[4] = {x.ka.x, x.ka.y, x.ka.z, x.ka.w}, wb[4] = {x.kb.x, x.kb.y, x.kb.z, x.kb.w};
#pragma unroll
        for (int w4 = 0; w4 < 4; ++w4) {
            uint32_t pa[4], pb[4];
            nc.word(wa[w4], pa);
            nc.word(wb[w4], pb);
            mma16816(sc, pa[0], pb[0], pa[1], pb[1], qf[2 * w4][0], qf[2 * w4][1]);
            mma16816(sc, pa[2], pb[2], pa[3], pb[3], qf[2 * w4 + 1][0], qf[2 * w4 + 1][1]);
        }
    }
    // this lane: query c4 against rows g8 (sc[0]) and g8 + 8 (sc[2])
    const bool va = tile + g8 < r1, vb = tile + g8 + 8 < r1;
    const float2 kza = w2f(x.ksa), kzb = w2f(x.ksb), vza = w2f(x.vsa), vzb = w2f(x.vsb);
    const float sa = va ? rs * (sc[0] * kza.x + qsum * kza.y) : -INFINITY;
    const float sb = vb ? rs * (sc[2] * kzb.x + qsum * kzb.y) : -INFINITY;
    const float sm = fmaxf(sa, sb), sv = fmaxf(va ? vza.x : 0.0f, vb ? vzb.x : 0.0f);
    if (__any_sync(0xffffffffu, sm > st.m || sv * st.F >= 32768.0f)) {
        const float m_new = fmaxf(st.m, group_max(sm));                 // of this lane's query
        const float corr = st.m == -INFINITY ? 0.0f : __expf(st.m - m_new);
        st.m = m_new;
        const float smax = warp_max(sv);                                // F is shared by the whole warp
        float Fn = st.F;
        for (int k = 0; k < 40 && smax * Fn >= 32768.0f; ++k) Fn *= 0.5f;
        const float rescale = corr * (Fn / st.F);
        st.F = Fn;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
#pragma unroll
            for (int i = 0; i < 4; ++i) st.acc[b][i] *= rescale;
        }
        st.den *= corr;
        st.zacc *= corr;
    }
    const float pa_ = __expf(sa - st.m), pb_ = __expf(sb - st.m);
    st.den += pa_ + pb_;
    st.zacc += pa_ * vza.y + pb_ * vzb.y;
    uint32_t packa, packb;                          // weights of (row g8, query c4) and (row g8 + 8, query c4): high | low
    {
        const float wa_ = pa_ * vza.x * st.F, wb_ = pb_ * vzb.x * st.F;
        const __half ha = __float2half_rn(wa_), hb = __float2half_rn(wb_);
        const __half la = __float2half_rn(wa_ - __half2float(ha)), lb = __float2half_rn(wb_ - __half2float(hb));
        packa = (uint32_t)__half_as_ushort(ha) | ((uint32_t)__half_as_ushort(la) << 16);
        packb = (uint32_t)__half_as_ushort(hb) | ((uint32_t)__half_as_ushort(lb) << 16);
    }
    // B fragment of the value product: this lane supplies column g8 = high (even) or low (odd) halves of query g8 / 2,
    // for the rows 2 c4, 2 c4 + 1 (b0) and 2 c4 + 8, 2 c4 + 9 (b1); the weight of (row r, query j) is in lane 4 (r % 8) + j
    const int la = 8 * c4 + (g8 >> 1);
    const uint32_t x1 = __shfl_sync(0xffffffffu, packa, la), x2 = __shfl_sync(0xffffffffu, packa, la + 4);
    const uint32_t y1 = __shfl_sync(0xffffffffu, packb, la), y2 = __shfl_sync(0xffffffffu, packb, la + 4);
    const uint32_t psel = (g8 & 1) ? 0x7632u : 0x5410u;
    const uint32_t b0 = __byte_perm(x1, x2, psel), b1 = __byte_perm(y1, y2, psel);
    {
        const uint32_t w0[2] = {x.v0.x, x.v0.y}, w1[2] = {x.v1.x, x.v1.y}, w2[2] = {x.v2.x, x.v2.y}, w3[2] = {x.v3.x, x.v3.y};
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            const uint32_t sel = (uint32_t)((b & 3) | ((b & 3) << 4) | ((4 + (b & 3)) << 8) | ((4 + (b & 3)) << 12));
            const uint32_t t1 = __byte_perm(w0[b >> 2], w1[b >> 2], sel);      // bytes (row 2 c4: b, -, row 2 c4 + 1: b, -)
            const uint32_t t2 = __byte_perm(w2[b >> 2], w3[b >> 2], sel);
            mma16816(st.acc[b], nc.lo(t1), nc.hi(t1), nc.lo(t2), nc.hi(t2), b0, b1);
        }
    }
}

__global__ void __launch_bounds__(AT_D)
k_attend_int4_gqa(const __half* __restrict__ q, AtPools pp, const long long* __restrict__ fill, int H, int gq, int q0, int gqn, int ng,
                  int min_rows,
                  float* __restrict__ ws) {
    __shared__ __align__(16) __half qp[GQ_MAX][AT_D];       // per query, every 8 elements ordered 0 4 1 5 2 6 3 7
    __shared__ float qsum_s[GQ_MAX];
    __shared__ float wpart[AT_WARPS][GQ_MAX][AT_D];
    __shared__ float wstat[AT_WARPS][GQ_MAX][2];
    const int h = blockIdx.x, c = blockIdx.y, l = blockIdx.z, t = threadIdx.x;
    const int lane = t & 31, wid = t >> 5, g8 = lane >> 2, c4 = lane & 3;
    const int Hq = H * gq;
    const size_t HD2 = (size_t)H * (AT_D / 2);
    const long long n4 = min(fill[2], pp.cap4);
    const long long per = max((long long)min_rows, ((n4 + gridDim.y - 1) / gridDim.y + 15) / 16 * 16);
    const long long r0 = (long long)c * per, r1 = min(n4, r0 + per);
    float* rec0 = ws + (((size_t)l * Hq + (size_t)h * gq + q0) * AT_RECS + AT_REC4 + c) * AT_REC;      // of the group's first query
    if (r0 >= r1) {                                 // nothing in this chunk: records the merge skips
        if (t < gqn) {
            float* rec = rec0 + (size_t)t * AT_RECS * AT_REC;
            rec[AT_D] = -INFINITY;
            rec[AT_D + 1] = 0.0f;
        }
        return;
    }
    // warp w stages query w of the group and sums it
    if (wid < GQ_MAX) {
        float part = 0.0f;
#pragma unroll
        for (int k = 0; k < AT_D / 32; ++k) {
            const int e = lane + 32 * k;
            const __half qv = wid < gqn ? q[((size_t)l * Hq + (size_t)h * gq + q0 + wid) * AT_D + e] : __float2half(0.0f);
            const int e8 = e & 7;
            qp[wid][(e & ~7) | ((e8 & 3) * 2 + (e8 >> 2))] = qv;
            part += __half2float(qv);
        }
        part = warp_sum(part);
        if (lane == 0) qsum_s[wid] = part;
    }
    __syncthreads();
    const float rs = rsqrtf((float)AT_D);
    const float qsum = qsum_s[c4];                  // this lane's query
    const int g = ng == 1 ? 0 : h;
    // B fragments of the score product: the lanes with g8 = 2 j hold query j (column 2 j), the others zeros
    uint32_t qf[8][2];
    {
        const uint32_t* qp32 = reinterpret_cast<const uint32_t*>(qp[(g8 >> 1) & (GQ_MAX - 1)]);
        const bool has = (g8 & 1) == 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int oct = 4 * c4 + (j >> 1), u = j & 1;
            qf[j][0] = has ? qp32[oct * 4 + 2 * u] : 0u;
            qf[j][1] = has ? qp32[oct * 4 + 2 * u + 1] : 0u;
        }
    }
    const long long t0 = r0 + 16 * wid;             // this warp's first tile
    G4Addr ad;
    ad.pitch = HD2;
    ad.ng = (size_t)ng;
    ad.k = pp.int4_codes + ((size_t)(2 * l) * pp.cap4 + (size_t)(t0 + g8)) * HD2 + (size_t)h * (AT_D / 2) + 16 * c4;
    ad.v = pp.int4_codes + ((size_t)(2 * l + 1) * pp.cap4 + (size_t)(t0 + 2 * c4)) * HD2 + (size_t)h * (AT_D / 2) + 8 * g8;
    ad.ks = reinterpret_cast<const uint32_t*>(pp.int4_sz) + ((size_t)(2 * l) * pp.cap4 + (size_t)(t0 + g8)) * ng + g;
    ad.vs = reinterpret_cast<const uint32_t*>(pp.int4_sz) + ((size_t)(2 * l + 1) * pp.cap4 + (size_t)(t0 + g8)) * ng + g;
    NibConst nc;
    nc.init();
    I4State st;
#pragma unroll
    for (int b = 0; b < 8; ++b) st.acc[b][0] = st.acc[b][1] = st.acc[b][2] = st.acc[b][3] = 0.0f;
    st.m = -INFINITY;
    st.den = st.zacc = 0.0f;
    st.F = 4096.0f;
    constexpr long long STEP = 16 * AT_WARPS;
    G4Tile xa, xb;                                  // two tiles in turn: one is consumed while the other is in flight
    long long tile = t0;
    if (tile < r1) {
        g4_fetch(xa, ad, tile, t0, r1, g8, c4);
        for (;;) {
            g4_fetch(xb, ad, tile + STEP, t0, r1, g8, c4);
            g4_tile(st, xa, qf, nc, tile, r1, rs, qsum, g8, c4);
            tile += STEP;
            if (tile >= r1) break;
            g4_fetch(xa, ad, tile + STEP, t0, r1, g8, c4);
            g4_tile(st, xb, qf, nc, tile, r1, rs, qsum, g8, c4);
            tile += STEP;
            if (tile >= r1) break;
        }
    }
    // ---- this warp's results, one per query
    {
        const float den = group_sum(st.den), zs = group_sum(st.zacc);
        const float invF = 1.0f / st.F;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            wpart[wid][c4][16 * g8 + 2 * b] = (st.acc[b][0] + st.acc[b][1]) * invF + zs;
            wpart[wid][c4][16 * g8 + 2 * b + 1] = (st.acc[b][2] + st.acc[b][3]) * invF + zs;
        }
        if (g8 == 0) {
            wstat[wid][c4][0] = st.m;
            wstat[wid][c4][1] = den;
        }
    }
    __syncthreads();
    for (int j = 0; j < gqn; ++j) {
        float M = wstat[0][j][0];
#pragma unroll
        for (int k = 1; k < AT_WARPS; ++k) M = fmaxf(M, wstat[k][j][0]);
        float sum = 0.0f, dsum = 0.0f;
        if (M != -INFINITY) {
#pragma unroll
            for (int k = 0; k < AT_WARPS; ++k) {
                const float e = wstat[k][j][0] == -INFINITY ? 0.0f : __expf(wstat[k][j][0] - M);
                sum += e * wpart[k][j][t];
                dsum += e * wstat[k][j][1];
            }
        }
        float* rec = rec0 + (size_t)j * AT_RECS * AT_REC;
        rec[t] = sum;
        if (t == 0) {
            rec[AT_D] = M;
            rec[AT_D + 1] = dsum;
        }
    }
}

// ---- INT8 rows on the matrix instructions, the same plan as for INT4: scores = 16 key rows x 16 dimensions
// times the query in columns 0 and 2; values = 16 dimensions x 16 value rows times the split weights.  A code
// byte becomes binary16 by a byte permute with 0x64 above it (1024 + (code + 128) after flipping its sign bit)
// and one subtraction of 1152.  Symmetric quantiser: no zero point.
struct I8Tile {
    uint4 ka0, ka1, kb0, kb1;      // keys of rows g8 and g8 + 8: dimensions 16 c4 .. + 15 and 64 + 16 c4 .. + 15
    uint4 v0, v1, v2, v3;          // values of rows c4, c4 + 4, c4 + 8, c4 + 12: dimensions 16 g8 .. + 15
    uint32_t ks, vs;               // binary16 scales of the row whose weight this lane computes: g8 + 8 * (c4 & 1)
};
struct I8Addr {
    const uint8_t* k;
    const uint8_t* v;
    const uint16_t* ks;
    const uint16_t* vs;
    size_t pitch, ng;
};
__device__ __forceinline__ void i8_fetch(I8Tile& x, const I8Addr& a, long long tile, long long t0, long long r1, int g8, int c4) {
    const size_t d = (size_t)(tile - t0), P = a.pitch;
    const uint8_t* k = a.k + d * P;
    const uint8_t* v = a.v + d * P;
    const uint16_t* ks = a.ks + d * a.ng;
    const uint16_t* vs = a.vs + d * a.ng;
    if (tile + 16 <= r1) {
        x.ka0 = ld_stream16(k);
        x.ka1 = ld_stream16(k + 64);
        x.kb0 = ld_stream16(k + 8 * P);
        x.kb1 = ld_stream16(k + 8 * P + 64);
        x.v0 = ld_stream16(v);
        x.v1 = ld_stream16(v + 4 * P);
        x.v2 = ld_stream16(v + 8 * P);
        x.v3 = ld_stream16(v + 12 * P);
        x.ks = __ldg(ks);
        x.vs = __ldg(vs);
    } else {                                        // rows at or beyond r1 read as zero codes and are not touched
        const uint4 z = make_uint4(0, 0, 0, 0);
        x.ka0 = x.ka1 = x.kb0 = x.kb1 = x.v0 = x.v1 = x.v2 = x.v3 = z;
        x.ks = x.vs = 0;
        const long long ra = tile + g8, rv = tile + c4;
        if (ra < r1) { x.ka0 = ld_stream16(k); x.ka1 = ld_stream16(k + 64); }
        if (ra + 8 < r1) { x.kb0 = ld_stream16(k + 8 * P); x.kb1 = ld_stream16(k + 8 * P + 64); }
        if (ra + 8 * (c4 & 1) < r1) { x.ks = __ldg(ks); x.vs = __ldg(vs); }
        if (rv < r1) x.v0 = ld_stream16(v);
        if (rv + 4 < r1) x.v1 = ld_stream16(v + 4 * P);
        if (rv + 8 < r1) x.v2 = ld_stream16(v + 8 * P);
        if (rv + 12 < r1) x.v3 = ld_stream16(v + 12 * P);
    }
}
struct ByteConst {
    uint32_t hi64, magic;           // 0x64 in every byte; binary16 pair (1152, 1152)
    __device__ __forceinline__ void init() {        // opaque to the compiler, so that they stay in registers
        asm volatile("mov.b32 %0, 0x64646464;" : "=r"(hi64));
        asm volatile("mov.b32 %0, 0x64806480;" : "=r"(magic));
    }
    // bytes i and j (0..3) of a word of sign-flipped codes as a binary16 pair
    template <int I, int J>
    __device__ __forceinline__ uint32_t pair(uint32_t u) const { return hsub2u(__byte_perm(u, hi64, 0x4040 | I | (J << 8)), magic); }
};

__device__ __forceinline__ void i8_tile(I4State& st, const I8Tile& x, const uint32_t (&qf)[8][2], const ByteConst& bc, long long tile,
                                        long long r1, float rs, int g8, int c4) {
    float sc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    {
        const uint32_t wa[8] = {x.ka0.x, x.ka0.y, x.ka0.z, x.ka0.w, x.ka1.x, x.ka1.y, x.ka1.z, x.ka1.w};
        const uint32_t wb[8] = {x.kb0.x, x.kb0.y, x.kb0.z, x.kb0.w, x.kb1.x, x.kb1.y, x.kb1.z, x.kb1.w};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t ua = wa[j] ^ 0x80808080u, ub = wb[j] ^ 0x80808080u;
            mma16816(sc, bc.pair<0, 1>(ua), bc.pair<0, 1>(ub), bc.pair<2, 3>(ua), bc.pair<2, 3>(ub), qf[j][0], qf[j][1]);
        }
    }
    // one row per lane: c4 == 0 takes row g8 (column 0), c4 == 1 takes row g8 + 8 (column 2)
    const bool own = c4 < 2 && tile + g8 + 8 * c4 < r1;
    const float s = own ? rs * (c4 ? sc[2] : sc[0]) * h2f((uint16_t)x.ks) : -INFINITY;
    const float sv = own ? h2f((uint16_t)x.vs) : 0.0f;
    if (__any_sync(0xffffffffu, s > st.m || sv * st.F >= 32768.0f)) {
        const float m_new = fmaxf(st.m, warp_max(s));
        const float corr = st.m == -INFINITY ? 0.0f : __expf(st.m - m_new);
        st.m = m_new;
        const float smax = warp_max(sv);
        float Fn = st.F;
        for (int k = 0; k < 40 && smax * Fn >= 32768.0f; ++k) Fn *= 0.5f;
        const float rescale = corr * (Fn / st.F);
        st.F = Fn;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
#pragma unroll
            for (int i = 0; i < 4; ++i) st.acc[b][i] *= rescale;
        }
        st.den *= corr;
    }
    const float pr = __expf(s - st.m);
    st.den += pr;
    uint32_t pack;
    {
        const float w = pr * sv * st.F;
        const __half hi = __float2half_rn(w);
        const __half lo = __float2half_rn(w - __half2float(hi));
        pack = (uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16);
    }
    // B fragment: column 0 = high halves, column 1 = low halves; k = tile rows c4, c4 + 4, c4 + 8, c4 + 12.
    // Row r of the tile was weighted by lane 4 * (r % 8) + r / 8.
    const uint32_t x1 = __shfl_sync(0xffffffffu, pack, 4 * c4), x2 = __shfl_sync(0xffffffffu, pack, 4 * c4 + 16);
    const uint32_t y1 = __shfl_sync(0xffffffffu, pack, 4 * c4 + 1), y2 = __shfl_sync(0xffffffffu, pack, 4 * c4 + 17);
    const uint32_t psel = g8 == 0 ? 0x5410u : 0x7632u;
    const uint32_t b0 = g8 < 2 ? __byte_perm(x1, x2, psel) : 0u, b1 = g8 < 2 ? __byte_perm(y1, y2, psel) : 0u;
    {
        const uint32_t w0[4] = {x.v0.x, x.v0.y, x.v0.z, x.v0.w}, w1[4] = {x.v1.x, x.v1.y, x.v1.z, x.v1.w};
        const uint32_t w2[4] = {x.v2.x, x.v2.y, x.v2.z, x.v2.w}, w3[4] = {x.v3.x, x.v3.y, x.v3.z, x.v3.w};
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            // bytes 2 b and 2 b + 1 (dimensions 16 g8 + 2 b, + 1) of two rows in one word: (r.d, r.d+1, r'.d, r'.d+1)
            const uint32_t sel = (b & 1) ? 0x7632u : 0x5410u;
            const uint32_t t1 = __byte_perm(w0[b >> 1], w1[b >> 1], sel) ^ 0x80808080u;
            const uint32_t t2 = __byte_perm(w2[b >> 1], w3[b >> 1], sel) ^ 0x80808080u;
            mma16816(st.acc[b], bc.pair<0, 2>(t1), bc.pair<1, 3>(t1), bc.pair<0, 2>(t2), bc.pair<1, 3>(t2), b0, b1);
        }
    }
}

// ---- INT8 rows, grouped queries: as k_attend_int4_gqa, with the byte expansion of k_attend_int8.
struct G8Tile {
    uint4 ka0, ka1, kb0, kb1;      // keys of rows g8 and g8 + 8: dimensions 16 c4 .. + 15 and 64 + 16 c4 .. + 15
    uint4 v0, v1, v2, v3;          // values of rows c4, c4 + 4, c4 + 8, c4 + 12: dimensions 16 g8 .. + 15
    uint32_t ksa, ksb, vsa, vsb;   // binary16 scales of the keys and values of rows g8 and g8 + 8
};
__device__ __forceinline__ void g8_fetch(G8Tile& x, const I8Addr& a, long long tile, long long t0, long long r1, int g8, int c4) {
    const size_t d = (size_t)(tile - t0), P = a.pitch;
    const uint8_t* k = a.k + d * P;
    const uint8_t* v = a.v + d * P;
    const uint16_t* ks = a.ks + d * a.ng;
    const uint16_t* vs = a.vs + d * a.ng;
    const uint4 z = make_uint4(0, 0, 0, 0);
    const long long ra = tile + g8, rv = tile + c4;
    const bool full = tile + 16 <= r1;
    const bool pa = full || ra < r1, pb = full || ra + 8 < r1;
    x.ka0 = pa ? ld_stream16(k) : z;
    x.ka1 = pa ? ld_stream16(k + 64) : z;
    x.kb0 = pb ? ld_stream16(k + 8 * P) : z;
    x.kb1 = pb ? ld_stream16(k + 8 * P + 64) : z;
    x.v0 = full || rv < r1 ? ld_stream16(v) : z;
    x.v1 = full || rv + 4 < r1 ? ld_stream16(v + 4 * P) : z;
    x.v2 = full || rv + 8 < r1 ? ld_stream16(v + 8 * P) : z;
    x.v3 = full || rv + 12 < r1 ? ld_stream16(v + 12 * P) : z;
    x.ksa = pa ? (uint32_t)__ldg(ks) : 0u;
    x.vsa = pa ? (uint32_t)__ldg(vs) : 0u;
    x.ksb = pb ? (uint32_t)__ldg(ks + 8 * a.ng) : 0u;
    x.vsb = pb ? (uint32_t)__ldg(vs + 8 * a.ng) : 0u;
}

__device__ __forceinline__ void g8_tile(I4State& st, const G8Tile& x, const uint32_t (&qf)[8][2], const ByteConst& bc, long long tile,
                                        long long r1, float rs, int g8, int c4) {
    float sc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    {
        const uint32_t wa[8] = {x.ka0.x, x.ka0.y, x.ka0.z, x.ka0.w, x.ka1.x, x.ka1.y, x.ka1.z, x.ka1.w};
        const uint32_t wb[8] = {x.kb0.x, x.kb0.y, x.kb0.z, x.kb0.w, x.kb1.x, x.kb1.y, x.kb1.z, x.kb1.w};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t ua = wa[j] ^ 0x80808080u, ub = wb[j] ^ 0x80808080u;
            mma16816(sc, bc.pair<0, 1>(ua), bc.pair<0, 1>(ub), bc.pair<2, 3>(ua), bc.pair<2, 3>(ub), qf[j][0], qf[j][1]);
        }
    }
    // this lane: query c4 against rows g8 (sc[0]) and g8 + 8 (sc[2])
    const bool va = tile + g8 < r1, vb = tile + g8 + 8 < r1;
    const float sa = va ? rs * sc[0] * h2f((uint16_t)x.ksa) : -INFINITY;
    const float sb = vb ? rs * sc[2] * h2f((uint16_t)x.ksb) : -INFINITY;
    const float sva = va ? h2f((uint16_t)x.vsa) : 0.0f, svb = vb ? h2f((uint16_t)x.vsb) : 0.0f;
    const float sm = fmaxf(sa, sb), sv = fmaxf(sva, svb);
    if (__any_sync(0xffffffffu, sm > st.m || sv * st.F >= 32768.0f)) {
        const float m_new = fmaxf(st.m, group_max(sm));
        const float corr = st.m == -INFINITY ? 0.0f : __expf(st.m - m_new);
        st.m = m_new;
        const float smax = warp_max(sv);
        float Fn = st.F;
        for (int k = 0; k < 40 && smax * Fn >= 32768.0f; ++k) Fn *= 0.5f;
        const float rescale = corr * (Fn / st.F);
        st.F = Fn;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
#pragma unroll
            for (int i = 0; i < 4; ++i) st.acc[b][i] *= rescale;
        }
        st.den *= corr;
    }
    const float pa_ = __expf(sa - st.m), pb_ = __expf(sb - st.m);
    st.den += pa_ + pb_;
    uint32_t packa, packb;
    {
        const float wa_ = pa_ * sva * st.F, wb_ = pb_ * svb * st.F;
        const __half ha = __float2half_rn(wa_), hb = __float2half_rn(wb_);
        const __half la = __float2half_rn(wa_ - __half2float(ha)), lb = __float2half_rn(wb_ - __half2float(hb));
        packa = (uint32_t)__half_as_ushort(ha) | ((uint32_t)__half_as_ushort(la) << 16);
        packb = (uint32_t)__half_as_ushort(hb) | ((uint32_t)__half_as_ushort(lb) << 16);
    }
    // column g8 of the value product = high (even) or low (odd) halves of query g8 / 2; k = rows c4, c4 + 4 (b0) and
    // c4 + 8, c4 + 12 (b1); the weight of (row r, query j) is in lane 4 (r % 8) + j, in packa for r < 8, else packb
    const int la = 4 * c4 + (g8 >> 1);
    const uint32_t x1 = __shfl_sync(0xffffffffu, packa, la), x2 = __shfl_sync(0xffffffffu, packa, la + 16);
    const uint32_t y1 = __shfl_sync(0xffffffffu, packb, la), y2 = __shfl_sync(0xffffffffu, packb, la + 16);
    const uint32_t psel = (g8 & 1) ? 0x7632u : 0x5410u;
    const uint32_t b0 = __byte_perm(x1, x2, psel), b1 = __byte_perm(y1, y2, psel);
    {
        const uint32_t w0[4] = {x.v0.x, x.v0.y, x.v0.z, x.v0.w}, w1[4] = {x.v1.x, x.v1.y, x.v1.z, x.v1.w};
        const uint32_t w2[4] = {x.v2.x, x.v2.y, x.v2.z, x.v2.w}, w3[4] = {x.v3.x, x.v3.y, x.v3.z, x.v3.w};
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            const uint32_t sel = (b & 1) ? 0x7632u : 0x5410u;
            const uint32_t t1 = __byte_perm(w0[b >> 1], w1[b >> 1], sel) ^ 0x80808080u;
            const uint32_t t2 = __byte_perm(w2[b >> 1], w3[b >> 1], sel) ^ 0x80808080u;
            mma16816(st.acc[b], bc.pair<0, 2>(t1), bc.pair<1, 3>(t1), bc.pair<0, 2>(t2), bc.pair<1, 3>(t2), b0, b1);
        }
    }
}

__global__ void __launch_bounds__(AT_D)
k_attend_int8_gqa(const __half* __restrict__ q, AtPools pp, const long long* __restrict__ fill, int H, int gq, int q0, int gqn, int ng,
                  int min_rows,
                  float* __restrict__ ws) {
    __shared__ __align__(16) __half qn[GQ_MAX][AT_D];
    __shared__ float wpart[AT_WARPS][GQ_MAX][AT_D];
    __shared__ float wstat[AT_WARPS][GQ_MAX][2];
    const int h = blockIdx.x, c = blockIdx.y, l = blockIdx.z, t = threadIdx.x;
    const int lane = t & 31, wid = t >> 5, g8 = lane >> 2, c4 = lane & 3;
    const int Hq = H * gq;
    const size_t HD = (size_t)H * AT_D;
    const long long n8 = min(fill[1], pp.cap8);
    const long long per = max((long long)min_rows, ((n8 + gridDim.y - 1) / gridDim.y + 15) / 16 * 16);
    const long long r0 = (long long)c * per, r1 = min(n8, r0 + per);
    float* rec0 = ws + (((size_t)l * Hq + (size_t)h * gq + q0) * AT_RECS + AT_REC8 + c) * AT_REC;      // of the group's first query
    if (r0 >= r1) {
        if (t < gqn) {
            float* rec = rec0 + (size_t)t * AT_RECS * AT_REC;
            rec[AT_D] = -INFINITY;
            rec[AT_D + 1] = 0.0f;
        }
        return;
    }
#pragma unroll
    for (int j = 0; j < GQ_MAX; ++j) qn[j][t] = j < gqn ? q[((size_t)l * Hq + (size_t)h * gq + q0 + j) * AT_D + t] : __float2half(0.0f);
    __syncthreads();
    const float rs = rsqrtf((float)AT_D);
    const int g = ng == 1 ? 0 : h;
    uint32_t qf[8][2];                              // the lanes with g8 = 2 j hold query j (column 2 j)
    {
        const uint32_t* q32 = reinterpret_cast<const uint32_t*>(qn[(g8 >> 1) & (GQ_MAX - 1)]);
        const bool has = (g8 & 1) == 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int base = (j < 4 ? 16 * c4 + 4 * j : 64 + 16 * c4 + 4 * (j - 4)) / 2;
            qf[j][0] = has ? q32[base] : 0u;
            qf[j][1] = has ? q32[base + 1] : 0u;
        }
    }
    const long long t0 = r0 + 16 * wid;
    I8Addr ad;
    ad.pitch = HD;
    ad.ng = (size_t)ng;
    ad.k = pp.int8_codes + ((size_t)(2 * l) * pp.cap8 + (size_t)(t0 + g8)) * HD + (size_t)h * AT_D + 16 * c4;
    ad.v = pp.int8_codes + ((size_t)(2 * l + 1) * pp.cap8 + (size_t)(t0 + c4)) * HD + (size_t)h * AT_D + 16 * g8;
    ad.ks = reinterpret_cast<const uint16_t*>(pp.int8_scale) + ((size_t)(2 * l) * pp.cap8 + (size_t)(t0 + g8)) * ng + g;
    ad.vs = reinterpret_cast<const uint16_t*>(pp.int8_scale) + ((size_t)(2 * l + 1) * pp.cap8 + (size_t)(t0 + g8)) * ng + g;
    ByteConst bc;
    bc.init();
    I4State st;
#pragma unroll
    for (int b = 0; b < 8; ++b) st.acc[b][0] = st.acc[b][1] = st.acc[b][2] = st.acc[b][3] = 0.0f;
    st.m = -INFINITY;
    st.den = st.zacc = 0.0f;
    st.F = 4096.0f;
    constexpr long long STEP = 16 * AT_WARPS;
    G8Tile xa, xb;
    long long tile = t0;
    if (tile < r1) {
        g8_fetch(xa, ad, tile, t0, r1, g8, c4);
        for (;;) {
            g8_fetch(xb, ad, tile + STEP, t0, r1, g8, c4);
            g8_tile(st, xa, qf, bc, tile, r1, rs, g8, c4);
            tile += STEP;
            if (tile >= r1) break;
            g8_fetch(xa, ad, tile + STEP, t0, r1, g8, c4);
            g8_tile(st, xb, qf, bc, tile, r1, rs, g8, c4);
            tile += STEP;
            if (tile >= r1) break;
        }
    }
    {
        const float den = group_sum(st.den);
        const float invF = 1.0f / st.F;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            wpart[wid][c4][16 * g8 + 2 * b] = (st.acc[b][0] + st.acc[b][1]) * invF;
            wpart[wid][c4][16 * g8 + 2 * b + 1] = (st.acc[b][2] + st.acc[b][3]) * invF;
        }
        if (g8 == 0) {
            wstat[wid][c4][0] = st.m;
            wstat[wid][c4][1] = den;
        }
    }
    __syncthreads();
    for (int j = 0; j < gqn; ++j) {
        float M = wstat[0][j][0];
#pragma unroll
        for (int k = 1; k < AT_WARPS; ++k) M = fmaxf(M, wstat[k][j][0]);
        float sum = 0.0f, dsum = 0.0f;
        if (M != -INFINITY) {
#pragma unroll
            for (int k = 0; k < AT_WARPS; ++k) {
                const float e = wstat[k][j][0] == -INFINITY ? 0.0f : __expf(wstat[k][j][0] - M);
                sum += e * wpart[k][j][t];
                dsum += e * wstat[k][j][1];
            }
        }
        float* rec = rec0 + (size_t)j * AT_RECS * AT_REC;
        rec[t] = sum;
        if (t == 0) {
            rec[AT_D] = M;
            rec[AT_D + 1] = dsum;
        }
    }
}

// ---- FP16 rows, grouped queries: the rows need no expansion, so a tile is 16 loads of 16 bytes per lane, two
// byte permutes per value operand and 16 matrix instructions for up to 4 queries.  One query per key/value
// head is the group of one: it runs this kernel too, close to the memory bandwidth.
struct G16Tile {
    uint4 ka[4], kb[4];            // keys of rows g8 and g8 + 8: dimensions 32 c4 .. + 31
    uint4 v[4][2];                 // values of rows c4, c4 + 4, c4 + 8, c4 + 12: dimensions 16 g8 .. + 15
};
__device__ __forceinline__ void g16_fetch(G16Tile& x, const uint8_t* k, const uint8_t* v, size_t P, long long tile, long long r1,
                                          int g8, int c4) {
    const uint4 z = make_uint4(0, 0, 0, 0);
    const bool full = tile + 16 <= r1;
    const long long ra = tile + g8, rv = tile + c4;
    const bool pa = full || ra < r1, pb = full || ra + 8 < r1;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x.ka[i] = pa ? ld_stream16(k + 16 * i) : z;
        x.kb[i] = pb ? ld_stream16(k + 8 * P + 16 * i) : z;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const bool pv = full || rv + 4 * j < r1;
        x.v[j][0] = pv ? ld_stream16(v + 4 * j * P) : z;
        x.v[j][1] = pv ? ld_stream16(v + 4 * j * P + 16) : z;
    }
}

__global__ void __launch_bounds__(AT_D)
k_attend_fp16_gqa(const __half* __restrict__ q, AtPools pp, const long long* __restrict__ fill, int H, int gq, int q0, int gqn,
                  int min_rows,
                  float* __restrict__ ws) {
    __shared__ __align__(16) __half qn[GQ_MAX][AT_D];
    __shared__ float wpart[AT_WARPS][GQ_MAX][AT_D];
    __shared__ float wstat[AT_WARPS][GQ_MAX][2];
    const int h = blockIdx.x, c = blockIdx.y, l = blockIdx.z, t = threadIdx.x;
    const int lane = t & 31, wid = t >> 5, g8 = lane >> 2, c4 = lane & 3;
    const int Hq = H * gq;
    const size_t P = (size_t)H * AT_D * 2;          // bytes per row
    const long long n16 = min(fill[0], pp.cap16);
    const long long per = max((long long)min_rows, ((n16 + gridDim.y - 1) / gridDim.y + 15) / 16 * 16);
    const long long r0 = (long long)c * per, r1 = min(n16, r0 + per);
    float* rec0 = ws + (((size_t)l * Hq + (size_t)h * gq + q0) * AT_RECS + c) * AT_REC;       // of the group's first query
    if (r0 >= r1) {
        if (t < gqn) {
            float* rec = rec0 + (size_t)t * AT_RECS * AT_REC;
            rec[AT_D] = -INFINITY;
            rec[AT_D + 1] = 0.0f;
        }
        return;
    }
#pragma unroll
    for (int j = 0; j < GQ_MAX; ++j) qn[j][t] = j < gqn ? q[((size_t)l * Hq + (size_t)h * gq + q0 + j) * AT_D + t] : __float2half(0.0f);
    __syncthreads();
    const float rs = rsqrtf((float)AT_D);
    uint32_t qf[8][2];                              // the lanes with g8 = 2 j hold query j (column 2 j)
    {
        const uint32_t* q32 = reinterpret_cast<const uint32_t*>(qn[(g8 >> 1) & (GQ_MAX - 1)]);
        const bool has = (g8 & 1) == 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            qf[j][0] = has ? q32[16 * c4 + 2 * j] : 0u;               // dimensions 32 c4 + 4 j, + 1
            qf[j][1] = has ? q32[16 * c4 + 2 * j + 1] : 0u;           //            32 c4 + 4 j + 2, + 3
        }
    }
    const long long t0 = r0 + 16 * wid;
    const uint8_t* kbase = pp.fp16_pool + ((size_t)(2 * l) * pp.cap16 + (size_t)(t0 + g8)) * P + (size_t)h * AT_D * 2 + 64 * c4;
    const uint8_t* vbase = pp.fp16_pool + ((size_t)(2 * l + 1) * pp.cap16 + (size_t)(t0 + c4)) * P + (size_t)h * AT_D * 2 + 32 * g8;
    float acc[8][4];
#pragma unroll
    for (int b = 0; b < 8; ++b) acc[b][0] = acc[b][1] = acc[b][2] = acc[b][3] = 0.0f;
    float m = -INFINITY, den = 0.0f;
    constexpr float F = 4096.0f;                    // the weights are scaled by a power of two before the binary16 split
    constexpr long long STEP = 16 * AT_WARPS;
    for (long long tile = t0; tile < r1; tile += STEP) {
        G16Tile x;
        g16_fetch(x, kbase + (size_t)(tile - t0) * P, vbase + (size_t)(tile - t0) * P, P, tile, r1, g8, c4);
        float sc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            mma16816(sc, x.ka[i].x, x.kb[i].x, x.ka[i].y, x.kb[i].y, qf[2 * i][0], qf[2 * i][1]);
            mma16816(sc, x.ka[i].z, x.kb[i].z, x.ka[i].w, x.kb[i].w, qf[2 * i + 1][0], qf[2 * i + 1][1]);
        }
        // this lane: query c4 against rows g8 (sc[0]) and g8 + 8 (sc[2])
        const float sa = tile + g8 < r1 ? rs * sc[0] : -INFINITY;
        const float sb = tile + g8 + 8 < r1 ? rs * sc[2] : -INFINITY;
        const float sm = fmaxf(sa, sb);
        if (__any_sync(0xffffffffu, sm > m)) {
            const float m_new = fmaxf(m, group_max(sm));
            const float corr = m == -INFINITY ? 0.0f : __expf(m - m_new);
            m = m_new;
#pragma unroll
            for (int b = 0; b < 8; ++b) {
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[b][i] *= corr;
            }
            den *= corr;
        }
        const float pa_ = __expf(sa - m), pb_ = __expf(sb - m);
        den += pa_ + pb_;
        uint32_t packa, packb;
        {
            const float wa_ = pa_ * F, wb_ = pb_ * F;
            const __half ha = __float2half_rn(wa_), hb = __float2half_rn(wb_);
            const __half la = __float2half_rn(wa_ - __half2float(ha)), lb = __float2half_rn(wb_ - __half2float(hb));
            packa = (uint32_t)__half_as_ushort(ha) | ((uint32_t)__half_as_ushort(la) << 16);
            packb = (uint32_t)__half_as_ushort(hb) | ((uint32_t)__half_as_ushort(lb) << 16);
        }
        const int la = 4 * c4 + (g8 >> 1);
        const uint32_t x1 = __shfl_sync(0xffffffffu, packa, la), x2 = __shfl_sync(0xffffffffu, packa, la + 16);
        const uint32_t y1 = __shfl_sync(0xffffffffu, packb, la), y2 = __shfl_sync(0xffffffffu, packb, la + 16);
        const uint32_t psel = (g8 & 1) ? 0x7632u : 0x5410u;
        const uint32_t b0 = __byte_perm(x1, x2, psel), b1 = __byte_perm(y1, y2, psel);
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            // word b of a row's 32 bytes holds dimensions 16 g8 + 2 b and + 1: pair the same dimension of two rows
            const uint32_t w0 = b < 4 ? (&x.v[0][0].x)[b] : (&x.v[0][1].x)[b - 4], w1 = b < 4 ? (&x.v[1][0].x)[b] : (&x.v[1][1].x)[b - 4];
            const uint32_t w2 = b < 4 ? (&x.v[2][0].x)[b] : (&x.v[2][1].x)[b - 4], w3 = b < 4 ? (&x.v[3][0].x)[b] : (&x.v[3][1].x)[b - 4];
            mma16816(acc[b], __byte_perm(w0, w1, 0x5410), __byte_perm(w0, w1, 0x7632), __byte_perm(w2, w3, 0x5410),
                     __byte_perm(w2, w3, 0x7632), b0, b1);
        }
    }
    {
        const float dsum = group_sum(den);
        constexpr float invF = 1.0f / F;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            wpart[wid][c4][16 * g8 + 2 * b] = (acc[b][0] + acc[b][1]) * invF;
            wpart[wid][c4][16 * g8 + 2 * b + 1] = (acc[b][2] + acc[b][3]) * invF;
        }
        if (g8 == 0) {
            wstat[wid][c4][0] = m;
            wstat[wid][c4][1] = dsum;
        }
    }
    __syncthreads();
    for (int j = 0; j < gqn; ++j) {
        float M = wstat[0][j][0];
#pragma unroll
        for (int k = 1; k < AT_WARPS; ++k) M = fmaxf(M, wstat[k][j][0]);
        float sum = 0.0f, dsum = 0.0f;
        if (M != -INFINITY) {
#pragma unroll
            for (int k = 0; k < AT_WARPS; ++k) {
                const float e = wstat[k][j][0] == -INFINITY ? 0.0f : __expf(wstat[k][j][0] - M);
                sum += e * wpart[k][j][t];
                dsum += e * wstat[k][j][1];
            }
        }
        float* rec = rec0 + (size_t)j * AT_RECS * AT_REC;
        rec[t] = sum;
        if (t == 0) {
            rec[AT_D] = M;
            rec[AT_D + 1] = dsum;
        }
    }
}

// Merge the four warps of a CTA of the matrix-instruction kernels and write its partial record.
__device__ __forceinline__ void mma_finish(const I4State& st, float (*wpart)[AT_D], float (*wstat)[2], float* rec, int g8, int c4) {
    const int t = threadIdx.x, lane = t & 31, wid = t >> 5;
    const float den = warp_sum(st.den);
    const float zs = warp_sum(st.zacc);
    if (c4 == 0) {
        const float invF = 1.0f / st.F;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            wpart[wid][16 * g8 + 2 * b] = (st.acc[b][0] + st.acc[b][1]) * invF + zs;
            wpart[wid][16 * g8 + 2 * b + 1] = (st.acc[b][2] + st.acc[b][3]) * invF + zs;
        }
    }
    if (lane == 0) {
        wstat[wid][0] = st.m;
        wstat[wid][1] = den;
    }
    __syncthreads();
    float M = wstat[0][0];
#pragma unroll
    for (int k = 1; k < AT_WARPS; ++k) M = fmaxf(M, wstat[k][0]);
    float sum = 0.0f, dsum = 0.0f;
    if (M != -INFINITY) {
#pragma unroll
        for (int k = 0; k < AT_WARPS; ++k) {
            const float e = wstat[k][0] == -INFINITY ? 0.0f : __expf(wstat[k][0] - M);
            sum += e * wpart[k][t];
            dsum += e * wstat[k][1];
        }
    }
    rec[t] = sum;
    if (t == 0) {
        rec[AT_D] = M;
        rec[AT_D + 1] = dsum;
    }
}

__global__ void __launch_bounds__(AT_D)
k_attend_int8(const __half* __restrict__ q, AtPools pp, const long long* __restrict__ fill, int H, int gq, int ng, int min_rows,
              float* __restrict__ ws) {
    __shared__ __align__(16) __half qn[AT_D];
    __shared__ float wpart[AT_WARPS][AT_D];
    __shared__ float wstat[AT_WARPS][2];
    const int hq = blockIdx.x, c = blockIdx.y, l = blockIdx.z, t = threadIdx.x;
    const int h = hq / gq, Hq = H * gq;          // query head hq reads key/value head h
    const int lane = t & 31, wid = t >> 5, g8 = lane >> 2, c4 = lane & 3;
    const size_t HD = (size_t)H * AT_D;
    const long long n8 = min(fill[1], pp.cap8);
    const long long per = max((long long)min_rows, ((n8 + gridDim.y - 1) / gridDim.y + 15) / 16 * 16);
    const long long r0 = (long long)c * per, r1 = min(n8, r0 + per);
    float* rec = ws + (((size_t)l * Hq + hq) * AT_RECS + AT_REC8 + c) * AT_REC;
    if (r0 >= r1) {                                 // nothing in this chunk: a record the merge skips
        if (t == 0) {
            rec[AT_D] = -INFINITY;
            rec[AT_D + 1] = 0.0f;
        }
        return;
    }
    qn[t] = q[((size_t)l * Hq + hq) * AT_D + t];
    __syncthreads();
    const float rs = rsqrtf((float)AT_D);
    const int g = ng == 1 ? 0 : h;
    // the query as B fragments: instruction j takes dimensions base .. base + 3 of the lane's key bytes, base =
    // 16 c4 + 4 j for j < 4 and 64 + 16 c4 + 4 (j - 4) after; columns 0 and 2 (lanes 0..3 and 8..11)
    uint32_t qf[8][2];
    {
        const uint32_t* q32 = reinterpret_cast<const uint32_t*>(qn);
        const bool has = g8 == 0 || g8 == 2;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int base = (j < 4 ? 16 * c4 + 4 * j : 64 + 16 * c4 + 4 * (j - 4)) / 2;
            qf[j][0] = has ? q32[base] : 0u;
            qf[j][1] = has ? q32[base + 1] : 0u;
        }
    }
    const long long t0 = r0 + 16 * wid;             // this warp's first tile
    I8Addr ad;
    ad.pitch = HD;
    ad.ng = (size_t)ng;
    const size_t own_row = (size_t)(t0 + g8 + 8 * (c4 & 1));
    ad.k = pp.int8_codes + ((size_t)(2 * l) * pp.cap8 + (size_t)(t0 + g8)) * HD + (size_t)h * AT_D + 16 * c4;
    ad.v = pp.int8_codes + ((size_t)(2 * l + 1) * pp.cap8 + (size_t)(t0 + c4)) * HD + (size_t)h * AT_D + 16 * g8;
    ad.ks = reinterpret_cast<const uint16_t*>(pp.int8_scale) + ((size_t)(2 * l) * pp.cap8 + own_row) * ng + g;
    ad.vs = reinterpret_cast<const uint16_t*>(pp.int8_scale) + ((size_t)(2 * l + 1) * pp.cap8 + own_row) * ng + g;
    ByteConst bc;
    bc.init();
    I4State st;
#pragma unroll
    for (int b = 0; b < 8; ++b) st.acc[b][0] = st.acc[b][1] = st.acc[b][2] = st.acc[b][3] = 0.0f;
    st.m = -INFINITY;
    st.den = st.zacc = 0.0f;
    st.F = 4096.0f;
    constexpr long long STEP = 16 * AT_WARPS;
    I8Tile xa, xb;                                  // two tiles in turn: one is consumed while the other is in flight
    long long tile = t0;
    if (tile < r1) {
        i8_fetch(xa, ad, tile, t0, r1, g8, c4);
        for (;;) {
            i8_fetch(xb, ad, tile + STEP, t0, r1, g8, c4);
            i8_tile(st, xa, qf, bc, tile, r1, rs, g8, c4);
            tile += STEP;
            if (tile >= r1) break;
            i8_fetch(xa, ad, tile + STEP, t0, r1, g8, c4);
            i8_tile(st, xb, qf, bc, tile, r1, rs, g8, c4);
            tile += STEP;
            if (tile >= r1) break;
        }
    }
    mma_finish(st, wpart, wstat, rec, g8, c4);
}

// Merge the partial results of one (layer, head): out = sum_c e^(m_c - M) acc_c / sum_c e^(m_c - M) den_c.
__global__ void __launch_bounds__(AT_D)
k_attend_merge(const float* __restrict__ ws, int H, int nch16, int nch8, int nch4, float* __restrict__ out) {
    __shared__ float ew[AT_RECS];                   // e^(m_c - M), 0 for a record that is empty or was not written
    __shared__ float red[AT_WARPS];
    static_assert(AT_RECS == AT_D, "one record per thread in the statistics pass");
    const int h = blockIdx.x, l = blockIdx.y, t = threadIdx.x;
    const float* rec = ws + ((size_t)l * H + h) * AT_RECS * AT_REC;
    // the first nch16, nch8, nch4 records of the FP16, INT8, INT4 ranges were written by this call's kernels
    const bool written = t < nch16 || (t >= AT_REC8 && t < AT_REC8 + nch8) || (t >= AT_REC4 && t < AT_REC4 + nch4);
    const float mc = written ? rec[t * AT_REC + AT_D] : -INFINITY;
    const float dc = written ? rec[t * AT_REC + AT_D + 1] : 0.0f;
    const float M = block_max(mc, red);
    const float e = mc == -INFINITY ? 0.0f : __expf(mc - M);
    ew[t] = e;
    const float den = block_sum(e * dc, red);       // (its barriers also publish ew)
    float num = 0.0f;
#pragma unroll 8
    for (int c = 0; c < AT_RECS; ++c) {
        const float w = ew[c];
        if (w != 0.0f) num += w * rec[c * AT_REC + t];
    }
    out[((size_t)l * H + h) * AT_D + t] = den > 0.0f ? num / den : 0.0f;
}

}  // namespace

// The workspace holds the partial records of up to max(H, 64) query heads per layer: grouped-query attention has
// more query heads than key/value heads.
static int attend_max_query_heads(int H) { return H > 64 ? H : 64; }
size_t sc_attend_workspace_bytes(int L, int H) { return (size_t)L * attend_max_query_heads(H) * AT_RECS * AT_REC * sizeof(float); }

int sc_attend(salicache_ctx* c, const void* d_q, int q_per_kv, const salicache_pools* pools, const int64_t* d_fill, float* d_out,
              cudaStream_t st) {
    const salicache_params& p = c->p;
    if (p.head_dim != AT_D || (p.group != AT_D && p.group != p.heads * p.head_dim)) return SALICACHE_E_PARAM;
    if (q_per_kv < 1 || (long long)p.heads * q_per_kv > attend_max_query_heads(p.heads)) return SALICACHE_E_SHAPE;
    AtPools pp{(const uint8_t*)pools->fp16_pool, (const uint8_t*)pools->int8_codes, (const uint8_t*)pools->int8_scale,
               (const uint8_t*)pools->int4_codes, (const uint8_t*)pools->int4_sz, pools->cap_fp16, pools->cap_int8,
               pools->cap_int4};
    if (pp.cap16 >= (1ll << 28) || pp.cap8 >= (1ll << 28) || pp.cap4 >= (1ll << 28)) return SALICACHE_E_SHAPE;
    const int ng = p.group == AT_D ? p.heads : 1;
    const int gq = q_per_kv, Hq = p.heads * gq;     // query heads; query head hq reads key/value head hq / gq
    const __half* qh = (const __half*)d_q;
    const long long* fl = (const long long*)d_fill;
    // chunks of the FP16 kernel: as many as its pool can fill with four tiles each, 32 at most
    const int nch = (int)std::min<long long>(AT_CH16, std::max<long long>(1, (pp.cap16 + 4 * AT_D - 1) / (4 * AT_D)));
    // rows per chunk: up to 4096 of the quantised tiers, 1024 of FP16 (64 tiles per warp) when there are many (layer,
    // head) pairs to fill the GPU with, fewer when there are few
    const int min_rows = (int)std::min<long long>(4096, std::max<long long>(256, 8ll * p.L * Hq)) / 16 * 16;
    const int min_rows16 = (int)std::min<long long>(1024, std::max<long long>(64, 2ll * p.L * p.heads)) / 16 * 16;
    // chunks of the quantised kernels: no more than their pools can fill with min_rows rows each
    const int nch8 = (int)std::min<long long>(AT_CH8, std::max<long long>(1, (pp.cap8 + min_rows - 1) / min_rows));
    const int nch4 = (int)std::min<long long>(AT_CHUNKS, std::max<long long>(1, (pp.cap4 + min_rows - 1) / min_rows));
    int launches = 0;
    if (gq == 1) {
        // one query per head: the FP16 kernel with a single column; INT8 and INT4 with a softmax row per lane
        k_attend_fp16_gqa<<<dim3(p.heads, nch, p.L), AT_D, 0, st>>>(qh, pp, fl, p.heads, 1, 0, 1, min_rows16, c->attend_ws);
        k_attend_int8<<<dim3(p.heads, nch8, p.L), AT_D, 0, st>>>(qh, pp, fl, p.heads, 1, ng, min_rows, c->attend_ws);
        dim3 grid(p.heads, nch4, p.L);
        if (p.heads == 32 && ng == 32) k_attend_int4<32 * AT_D / 2, 32><<<grid, AT_D, 0, st>>>(qh, pp, fl, p.heads, 1, ng, min_rows, c->attend_ws);
        else if (p.heads == 32 && ng == 1) k_attend_int4<32 * AT_D / 2, 1><<<grid, AT_D, 0, st>>>(qh, pp, fl, p.heads, 1, ng, min_rows, c->attend_ws);
        else k_attend_int4<0, 0><<<grid, AT_D, 0, st>>>(qh, pp, fl, p.heads, 1, ng, min_rows, c->attend_ws);
        launches = 3;
    } else {
        // grouped queries: up to GQ_MAX queries of every key/value head per launch share one pass over its rows
        for (int q0 = 0; q0 < gq; q0 += GQ_MAX) {
            const int gqn = std::min(GQ_MAX, gq - q0);
            k_attend_fp16_gqa<<<dim3(p.heads, nch, p.L), AT_D, 0, st>>>(qh, pp, fl, p.heads, gq, q0, gqn, min_rows16, c->attend_ws);
            k_attend_int8_gqa<<<dim3(p.heads, nch8, p.L), AT_D, 0, st>>>(qh, pp, fl, p.heads, gq, q0, gqn, ng, min_rows, c->attend_ws);
            k_attend_int4_gqa<<<dim3(p.heads, nch4, p.L), AT_D, 0, st>>>(qh, pp, fl, p.heads, gq, q0, gqn, ng, min_rows, c->attend_ws);
            launches += 3;
        }
    }
    dim3 gm(Hq, p.L);
    k_attend_merge<<<gm, AT_D, 0, st>>>(c->attend_ws, Hq, nch, nch8, nch4, d_out);
    c->launches += launches + 1;
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}
