// Mixed-precision K/V store (Alg. 1 line 16; quantisers of Sec. IV-B) and its just-in-time
// dequantisation (Sec. III-C).  HBM-bound.  One warp moves one token row (HD fp16, 8 KiB at HD = 4096):
// all 16-byte loads of the row are issued before any arithmetic, one quantisation group (128 elements)
// is reduced per half warp, each lane then owns one group's scale, and codes leave as packed stores.
#include <cuda_fp16.h>

#include "common.cuh"

namespace {

constexpr int KV_THREADS = 256;
constexpr int KV_WARPS = KV_THREADS / 32;
constexpr int MAX_PREFIX = 4096;   // frames per call whose row prefix fits the shared-memory table

struct KvGeom {
    int L, n_tok, HD, ng;          // ng = groups per row: HD / 128, or 1 when the whole row is one group
    long long frame_stride;        // fp16 elements between frames
    int B;
    int row_group;                 // 1: one quantisation group per row (ng == 1)
};

struct PoolPtrs {
    uint8_t* fp16_pool;
    uint8_t* int8_codes;
    uint8_t* int8_scale;
    uint8_t* int4_codes;
    uint8_t* int4_sz;
    long long cap0, cap1, cap2;
    int ring;
    const long long* fill;         // running fill per tier, or null
};

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ld_stream(const uint2* p) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ uint32_t ld_stream(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void st_stream(uint2* p, uint2 v) {
    asm volatile("st.global.cs.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(v.x), "r"(v.y) : "memory");
}
__device__ __forceinline__ void st_stream(uint32_t* p, uint32_t v) {
    asm volatile("st.global.cs.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

__device__ __forceinline__ __half2 as_h2(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }
__device__ __forceinline__ uint32_t as_u32(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }

// d = (c << 16) | (sat_s8(a) << 8) | sat_s8(b)   (saturation to [-128, 127])
__device__ __forceinline__ uint32_t pack_s8(int a, int b, uint32_t c) {
    uint32_t d;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// Both halves of a word minus z, in binary32: the mixed-precision subtract converts the binary16 operand
// exactly and rounds once, so it equals convert-then-subtract.
__device__ __forceinline__ float2 sub_h2_f32(uint32_t w, float z) {
    float2 r;
    asm("{ .reg .b16 lo, hi; mov.b32 {lo, hi}, %2; sub.rn.f32.f16 %0, lo, %3; sub.rn.f32.f16 %1, hi, %3; }"
        : "=f"(r.x), "=f"(r.y)
        : "r"(w), "f"(z));
    return r;
}
// rint(d * inv) clamped to at most 15: multiply and round to nearest even as separate operations.
__device__ __forceinline__ int quant4(float d, float inv) { return __float2int_rn(fminf(__fmul_rn(d, inv), 15.0f)); }
// fl(d * inv) + 1.5 * 2^23 as bits: for |product| < 2^22 the sum is the product rounded to the nearest integer (ties to
// even), held in the low mantissa bits as a two's complement number.  Multiply and add round separately.
__device__ __forceinline__ uint32_t rint_bits(float d, float inv) {
    return __float_as_uint(__fadd_rn(__fmul_rn(d, inv), 12582912.0f));
}
// Bytes (q0 q1 q2 q3), (q4 q5 q6 q7), each 0..15 -> nibbles q0 | q1 << 4 | ... | q7 << 28.
__device__ __forceinline__ uint32_t nibbles(uint32_t lo, uint32_t hi) {
    lo |= lo >> 4;
    hi |= hi >> 4;
    return __byte_perm(lo, hi, 0x6420);
}

// Rows stored before each frame of the batch, built by every CTA in shared memory from the counts.
__device__ __forceinline__ void build_prefix(const int32_t* __restrict__ counts, int B, int* pre) {
    __shared__ int wsum[KV_WARPS];
    int carry = 0;
    for (int base = 0; base < B; base += KV_THREADS) {
        int b = base + threadIdx.x;
        int v = 0;
        if (b < B) v = counts[b * 5 + SALICACHE_FP16] + counts[b * 5 + SALICACHE_INT8] + counts[b * 5 + SALICACHE_INT4];
        int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, incl, o);
            if ((threadIdx.x & 31) >= o) incl += t;
        }
        if ((threadIdx.x & 31) == 31) wsum[threadIdx.x >> 5] = incl;
        __syncthreads();
        int woff = 0;
        for (int k = 0; k < (threadIdx.x >> 5); ++k) woff += wsum[k];
        if (b < B) pre[b] = carry + woff + incl - v;
        int tot = 0;
        for (int k = 0; k < KV_WARPS; ++k) tot += wsum[k];
        carry += tot;
        __syncthreads();
    }
    if (threadIdx.x == 0) pre[B] = carry;
    __syncthreads();
}

// Work unit u -> (frame b, plane = layer*2 + kv, tier, token, pool row).  Units of one frame are ordered
// plane-major, position-minor, so neighbouring warps read neighbouring token rows and write neighbouring
// pool rows.
struct Unit {
    int b, plane, tier, tok;
    long long row;   // pool row, or -1 when dropped
    long long cap;
};

// lim[tier] (ring pools): rows at an absolute position below it are gone: overwritten by a later row of the same
// call when storing, by newer frames when reading back.  Such rows come back as row -2; rows past the capacity of
// a linear pool as row -1.
__device__ __forceinline__ Unit decode_unit(uint32_t u, const int* pre, int B, uint32_t planes,
                                            const int32_t* __restrict__ counts, const int32_t* __restrict__ idx,
                                            const long long* __restrict__ row_offset, int n_tok, const PoolPtrs& pp,
                                            const long long* lim) {
    Unit r;
    const uint32_t q = u / planes;      // lies in [pre[b], pre[b+1]) of exactly one frame
    int lo = 0, hi = B;                 // largest b with pre[b] <= q
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if ((uint32_t)pre[mid] <= q) lo = mid; else hi = mid;
    }
    r.b = lo;
    const uint32_t stored = (uint32_t)(pre[lo + 1] - pre[lo]);
    const uint32_t local = u - (uint32_t)pre[lo] * planes;
    r.plane = (int)(local / stored);
    int j = (int)(local - (uint32_t)r.plane * stored);
    int n16 = counts[lo * 5 + SALICACHE_FP16], n8 = counts[lo * 5 + SALICACHE_INT8];
    if (j < n16) { r.tier = 0; r.cap = pp.cap0; }
    else if (j < n16 + n8) { r.tier = 1; j -= n16; r.cap = pp.cap1; }
    else { r.tier = 2; j -= n16 + n8; r.cap = pp.cap2; }
    r.tok = idx[((size_t)lo * 3 + r.tier) * n_tok + j];
    long long row = row_offset[(size_t)lo * 3 + r.tier] + j;
    if (pp.ring) row = r.cap <= 0 ? -1 : (row < lim[r.tier] ? -2 : row % r.cap);
    else if (row >= r.cap) row = -1;
    r.row = row;
    return r;
}

// The limits above, into shared memory (3 values), behind the prefix table.
//   storing: the call ends at absolute row end = row_offset of its last frame + that frame's count; a row
//            below end - cap is overwritten by a later row of this call;
//   reading: rows below fill - cap have been overwritten since (no limit when the caller gave no fill).
__device__ __forceinline__ void build_limits(bool storing, const int32_t* __restrict__ counts,
                                             const long long* __restrict__ row_offset, int B, const PoolPtrs& pp,
                                             long long* lim) {
    if (threadIdx.x < 3) {
        const int t = threadIdx.x;
        const int code = t == 0 ? SALICACHE_FP16 : (t == 1 ? SALICACHE_INT8 : SALICACHE_INT4);
        const long long cap = t == 0 ? pp.cap0 : (t == 1 ? pp.cap1 : pp.cap2);
        long long v = -0x7fffffffffffffffll;
        if (pp.ring) {
            if (storing) v = row_offset[(size_t)(B - 1) * 3 + t] + counts[(B - 1) * 5 + code] - cap;
            else if (pp.fill) v = pp.fill[t] - cap;
        }
        lim[t] = v;
    }
    __syncthreads();
}

// ---- pack ---------------------------------------------------------------------------------------
template <int N> struct ILog2 { static constexpr int v = 1 + ILog2<N / 2>::v; };
template <> struct ILog2<1> { static constexpr int v = 0; };

// m[i] holds this lane's partial (a half2, reduced with max) of the group that the lane's half warp reads
// in iteration i.  Reduces every m[i] over the 16 lanes of the half warp with a transposing butterfly:
// each step a lane hands half of its values to its partner and keeps the other half, so ITERS values
// cost ITERS - 1 exchanges instead of 4 * ITERS.  On return the lane whose low four bits are
// i << (4 - log2 ITERS) (and its neighbours above it) holds the reduced value of iteration i.
template <int ITERS>
__device__ __forceinline__ uint32_t half_warp_max_transpose(uint32_t (&m)[ITERS], int lane) {
    int s = 8;
#pragma unroll
    for (int n = ITERS; n > 1; n >>= 1, s >>= 1) {
        const bool up = lane & s;
#pragma unroll
        for (int j = 0; j < n / 2; ++j) {
            const uint32_t send = up ? m[j] : m[j + n / 2];
            const uint32_t keep = up ? m[j + n / 2] : m[j];
            m[j] = as_u32(__hmax2(as_h2(keep), as_h2(__shfl_xor_sync(0xffffffffu, send, s))));
        }
    }
#pragma unroll
    for (; s >= 1; s >>= 1) m[0] = as_u32(__hmax2(as_h2(m[0]), as_h2(__shfl_xor_sync(0xffffffffu, m[0], s))));
    return m[0];
}
// One row (or piece `part` of a row): ITERS 16-byte words per lane = 256 * ITERS elements = 2 * ITERS
// quantisation groups (<= 32, one per lane), or one group for the whole row when RG.
template <int ITERS, bool RG>
__device__ __forceinline__ void pack_piece(const uint4 (&v)[ITERS], const Unit& un, int part, const KvGeom& g,
                                           const PoolPtrs& pp, int lane) {
    // after the transposing reduction the lanes with low bits (i << SH) of each half warp hold iteration i's group
    constexpr int SH = 4 - ILog2<ITERS>::v;
    const bool owns = (lane & ((1 << SH) - 1)) == 0;
    const int my_group = 2 * ((lane & 15) >> SH) + (lane >> 4);
    const size_t prow = (size_t)un.plane * un.cap + un.row;
    if (un.tier == 0) {
        uint4* dst = reinterpret_cast<uint4*>(pp.fp16_pool + prow * (size_t)g.HD * 2) + part * (ITERS * 32) + lane;
#pragma unroll
        for (int i = 0; i < ITERS; ++i) st_stream(dst + i * 32, v[i]);
    } else if (un.tier == 1) {
        // INT8 symmetric: s = fp16(max|x| / 127), q = rint(x * (1/s)) clamped to [-127, 127]
        // (this tier runs at the memory limit: the plain butterfly, whose result every lane of the half warp
        // sees, then one pick per iteration by the lane that will own the group)
        uint32_t mine = 0;
        if (RG) {                         // one group: every lane ends with the row's maximum
            __half2 m = __floats2half2_rn(0.0f, 0.0f);
#pragma unroll
            for (int i = 0; i < ITERS; ++i)
                m = __hmax2(m, __hmax2(__hmax2(__habs2(as_h2(v[i].x)), __habs2(as_h2(v[i].y))),
                                       __hmax2(__habs2(as_h2(v[i].z)), __habs2(as_h2(v[i].w)))));
#pragma unroll
            for (int o = 16; o; o >>= 1) m = __hmax2(m, as_h2(__shfl_xor_sync(0xffffffffu, as_u32(m), o)));
            mine = as_u32(m);
        } else {
#pragma unroll
            for (int i = 0; i < ITERS; ++i) {
                __half2 m = __hmax2(__hmax2(__habs2(as_h2(v[i].x)), __habs2(as_h2(v[i].y))),
                                    __hmax2(__habs2(as_h2(v[i].z)), __habs2(as_h2(v[i].w))));
#pragma unroll
                for (int o = 8; o; o >>= 1) m = __hmax2(m, as_h2(__shfl_xor_sync(0xffffffffu, as_u32(m), o)));
                if (((lane & 15) >> SH) == i) mine = as_u32(m);
            }
        }
        float amax = fmaxf(__low2float(as_h2(mine)), __high2float(as_h2(mine)));
        __half s16 = __float2half_rn(__fdiv_rn(amax, 127.0f));
        if ((__half_as_ushort(s16) & 0x7fff) == 0) s16 = __ushort_as_half(0x3c00);
        const float my_inv = __fdiv_rn(1.0f, __half2float(s16));
        if (RG ? lane == 0 : owns)
            reinterpret_cast<uint16_t*>(pp.int8_scale + prow * (size_t)g.ng * 2)[RG ? 0 : part * 2 * ITERS + my_group] =
                __half_as_ushort(s16);
        uint2* dst = reinterpret_cast<uint2*>(pp.int8_codes + prow * (size_t)g.HD) + part * (ITERS * 32) + lane;
#pragma unroll
        for (int i = 0; i < ITERS; ++i) {
            const float inv = RG ? my_inv : __shfl_sync(0xffffffffu, my_inv, (lane & 16) | (i << SH));
            float2 f0 = __half22float2(as_h2(v[i].x)), f1 = __half22float2(as_h2(v[i].y));
            float2 f2 = __half22float2(as_h2(v[i].z)), f3 = __half22float2(as_h2(v[i].w));
            int q0 = __float2int_rn(__fmul_rn(f0.x, inv)), q1 = __float2int_rn(__fmul_rn(f0.y, inv));
            int q2 = __float2int_rn(__fmul_rn(f1.x, inv)), q3 = __float2int_rn(__fmul_rn(f1.y, inv));
            int q4 = __float2int_rn(__fmul_rn(f2.x, inv)), q5 = __float2int_rn(__fmul_rn(f2.y, inv));
            int q6 = __float2int_rn(__fmul_rn(f3.x, inv)), q7 = __float2int_rn(__fmul_rn(f3.y, inv));
            uint2 o;
            o.x = __vmaxs4(pack_s8(q1, q0, pack_s8(q3, q2, 0)), 0x81818181u);
            o.y = __vmaxs4(pack_s8(q5, q4, pack_s8(q7, q6, 0)), 0x81818181u);
            st_stream(dst + i * 32, o);
        }
    } else {
        // INT4 asymmetric: zero = min, s = fp16((max - min) / 15), q = rint((x - zero) * (1/s)) in [0, 15].
        // One half2 carries (max, -min) so a single max-reduction serves both.
        uint32_t ext[ITERS];
#pragma unroll
        for (int i = 0; i < ITERS; ++i) {
            __half2 a = as_h2(v[i].x), b = as_h2(v[i].y), c = as_h2(v[i].z), d = as_h2(v[i].w);
            __half2 mx = __hmax2(__hmax2(a, b), __hmax2(c, d));
            __half2 nmn = __hneg2(__hmin2(__hmin2(a, b), __hmin2(c, d)));
            ext[i] = as_u32(__hmax2(as_h2(__byte_perm(as_u32(mx), as_u32(nmn), 0x5410)),
                                     as_h2(__byte_perm(as_u32(mx), as_u32(nmn), 0x7632))));   // (max, -min)
        }
        uint32_t mine;
        if (RG) {
            __half2 m = as_h2(ext[0]);
#pragma unroll
            for (int i = 1; i < ITERS; ++i) m = __hmax2(m, as_h2(ext[i]));
#pragma unroll
            for (int o = 16; o; o >>= 1) m = __hmax2(m, as_h2(__shfl_xor_sync(0xffffffffu, as_u32(m), o)));
            mine = as_u32(m);
        } else {
            mine = half_warp_max_transpose<ITERS>(ext, lane);
        }
        const float fmx = __low2float(as_h2(mine));
        float fmn = -__high2float(as_h2(mine));
        __half z16 = __float2half_rn(fmn);                       // exact: fmn is an fp16 value
        if (fmn == 0.0f) z16 = __ushort_as_half(0);              // a zero minimum is stored as +0
        __half s16 = __float2half_rn(__fdiv_rn(__fsub_rn(fmx, fmn), 15.0f));
        if ((__half_as_ushort(s16) & 0x7fff) == 0) s16 = __ushort_as_half(0x3c00);
        const float my_inv = __fdiv_rn(1.0f, __half2float(s16));
        const float my_z = __half2float(z16);
        if (RG ? lane == 0 : owns)
            reinterpret_cast<uint32_t*>(pp.int4_sz + prow * (size_t)g.ng * 4)[RG ? 0 : part * 2 * ITERS + my_group] =
                (uint32_t)__half_as_ushort(s16) | ((uint32_t)__half_as_ushort(z16) << 16);
        uint32_t* dst = reinterpret_cast<uint32_t*>(pp.int4_codes + prow * (size_t)(g.HD / 2)) + part * (ITERS * 32) + lane;
        // x >= zero, so the product is >= 0.  It exceeds 15.5 only when the stored scale was rounded down by more than
        // 3 %, which binary16 does to subnormal scales alone (a normal one is within 2^-11 of (max - min) / 15): the
        // upper clamp is compiled in only for rows that have such a group.
        const bool tiny = (__half_as_ushort(s16) & 0x7fff) < 0x0400;
        // every lane's (1/s, zero) through shared memory: one 8-byte broadcast read per iteration
        __shared__ float2 sz_of[KV_WARPS][32];
        float2* sz = sz_of[threadIdx.x >> 5];
        if (!RG) {
            __syncwarp();
            sz[lane] = make_float2(my_inv, my_z);
            __syncwarp();
        }
        if (__any_sync(0xffffffffu, tiny)) {
#pragma unroll
            for (int i = 0; i < ITERS; ++i) {
                const int owner = (lane & 16) | (i << SH);
                const float2 iz = RG ? make_float2(my_inv, my_z) : sz[owner];
                const float inv = iz.x, z = iz.y;
                const float2 f0 = sub_h2_f32(v[i].x, z), f1 = sub_h2_f32(v[i].y, z), f2 = sub_h2_f32(v[i].z, z), f3 = sub_h2_f32(v[i].w, z);
                int q0 = quant4(f0.x, inv), q1 = quant4(f0.y, inv), q2 = quant4(f1.x, inv), q3 = quant4(f1.y, inv);
                int q4 = quant4(f2.x, inv), q5 = quant4(f2.y, inv), q6 = quant4(f3.x, inv), q7 = quant4(f3.y, inv);
                st_stream(dst + i * 32, nibbles(pack_s8(q1, q0, pack_s8(q3, q2, 0)), pack_s8(q5, q4, pack_s8(q7, q6, 0))));
            }
        } else {
#pragma unroll
            for (int i = 0; i < ITERS; ++i) {
                const int owner = (lane & 16) | (i << SH);
                const float2 iz = RG ? make_float2(my_inv, my_z) : sz[owner];
                const float inv = iz.x, z = iz.y;
                const float2 f0 = sub_h2_f32(v[i].x, z), f1 = sub_h2_f32(v[i].y, z), f2 = sub_h2_f32(v[i].z, z), f3 = sub_h2_f32(v[i].w, z);
                // 0 <= product < 15.5: adding 1.5 * 2^23 rounds it to nearest even and leaves the code in the low bits
                const uint32_t a = rint_bits(f0.x, inv) + (rint_bits(f0.y, inv) << 4), b = rint_bits(f1.x, inv) + (rint_bits(f1.y, inv) << 4);
                const uint32_t c = rint_bits(f2.x, inv) + (rint_bits(f2.y, inv) << 4), d = rint_bits(f3.x, inv) + (rint_bits(f3.y, inv) << 4);
                st_stream(dst + i * 32, __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410));
            }
        }
    }
}

template <int ITERS>
__device__ __forceinline__ void load_piece(uint4 (&v)[ITERS], const __half* K, const __half* V, const Unit& un, int part,
                                           const KvGeom& g, int lane) {
    const int layer = un.plane >> 1, kv = un.plane & 1;
    const __half* src_h = (kv ? V : K) + (size_t)un.b * g.frame_stride + ((size_t)layer * g.n_tok + un.tok) * g.HD;
    const uint4* src = reinterpret_cast<const uint4*>(src_h) + part * (ITERS * 32) + lane;
#pragma unroll
    for (int i = 0; i < ITERS; ++i) v[i] = ld_stream(src + i * 32);
}

// One warp per stored row: all 16-byte loads of the row are issued before any arithmetic, and the next
// row's lookups (index list, row offset) run while they are in flight.
template <int ITERS, bool RG>
__global__ void __launch_bounds__(KV_THREADS, 2)
k_pack(const __half* __restrict__ K, const __half* __restrict__ V, KvGeom g, const int32_t* __restrict__ idx,
       const int32_t* __restrict__ counts, const long long* __restrict__ row_offset, PoolPtrs pp,
       int* __restrict__ status) {
    extern __shared__ int pre[];
    __shared__ long long lim[3];
    build_prefix(counts, g.B, pre);
    build_limits(true, counts, row_offset, g.B, pp, lim);
    const uint32_t planes = 2u * (uint32_t)g.L;
    const uint32_t n_units = (uint32_t)pre[g.B] * planes;      // < 2^31: checked on the host
    const int lane = threadIdx.x & 31;
    const uint32_t warp0 = blockIdx.x * KV_WARPS + (threadIdx.x >> 5);
    const uint32_t wstride = gridDim.x * KV_WARPS;
    if (warp0 >= n_units) return;
    Unit un = decode_unit(warp0, pre, g.B, planes, counts, idx, row_offset, g.n_tok, pp, lim);
    uint4 v[ITERS];
    if (un.row >= 0) load_piece<ITERS>(v, K, V, un, 0, g, lane);
    for (uint32_t u = warp0; u < n_units; u += wstride) {
        const bool more = u + wstride < n_units;
        Unit nxt = un;
        if (more) nxt = decode_unit(u + wstride, pre, g.B, planes, counts, idx, row_offset, g.n_tok, pp, lim);
        if (un.row >= 0) pack_piece<ITERS, RG>(v, un, 0, g, pp, lane);
        else if (un.row == -1 && lane == 0) atomicMin(status, SALICACHE_E_CAPACITY);
        if (more && nxt.row >= 0) load_piece<ITERS>(v, K, V, nxt, 0, g, lane);
        un = nxt;
    }
}

// ---- unpack -------------------------------------------------------------------------------------
template <int ITERS>
__global__ void __launch_bounds__(KV_THREADS, 2)
k_unpack(__half* __restrict__ K, __half* __restrict__ V, KvGeom g, const int32_t* __restrict__ idx,
         const int32_t* __restrict__ counts, const long long* __restrict__ row_offset, PoolPtrs pp,
         int* __restrict__ status) {
    extern __shared__ int pre[];
    __shared__ long long lim[3];
    build_prefix(counts, g.B, pre);
    build_limits(false, counts, row_offset, g.B, pp, lim);
    const uint32_t planes = 2u * (uint32_t)g.L;
    const uint32_t n_units = (uint32_t)pre[g.B] * planes;      // < 2^31: checked on the host
    const int lane = threadIdx.x & 31;
    const uint32_t warp0 = blockIdx.x * KV_WARPS + (threadIdx.x >> 5);
    const uint32_t wstride = gridDim.x * KV_WARPS;
    for (uint32_t u = warp0; u < n_units; u += wstride) {
        Unit un = decode_unit(u, pre, g.B, planes, counts, idx, row_offset, g.n_tok, pp, lim);
        if (un.row == -1) {
            if (lane == 0) atomicMin(status, SALICACHE_E_CAPACITY);
            continue;
        }
        const int layer = un.plane >> 1, kv = un.plane & 1;
        __half* dst_h = (kv ? V : K) + (size_t)un.b * g.frame_stride + ((size_t)layer * g.n_tok + un.tok) * g.HD;
        uint4* dst = reinterpret_cast<uint4*>(dst_h) + lane;
        if (un.row < 0) {                  // overwritten since by a newer frame: zeros, never another frame's row
#pragma unroll
            for (int i = 0; i < ITERS; ++i) st_stream(dst + i * 32, make_uint4(0, 0, 0, 0));
            if (lane == 0) atomicMin(status, SALICACHE_E_EVICTED);
            continue;
        }
        const size_t prow = (size_t)un.plane * un.cap + un.row;
        if (un.tier == 0) {
            const uint4* src = reinterpret_cast<const uint4*>(pp.fp16_pool + prow * (size_t)g.HD * 2) + lane;
            uint4 v[ITERS];
#pragma unroll
            for (int i = 0; i < ITERS; ++i) v[i] = ld_stream(src + i * 32);
#pragma unroll
            for (int i = 0; i < ITERS; ++i) st_stream(dst + i * 32, v[i]);
        } else if (un.tier == 1) {
            const uint2* src = reinterpret_cast<const uint2*>(pp.int8_codes + prow * (size_t)g.HD) + lane;
            uint2 c[ITERS];
#pragma unroll
            for (int i = 0; i < ITERS; ++i) c[i] = ld_stream(src + i * 32);
            uint32_t my_scale = 0;
            if (lane < g.ng) my_scale = reinterpret_cast<const uint16_t*>(pp.int8_scale + prow * (size_t)g.ng * 2)[lane];
            const float my_s = __half2float(__ushort_as_half((uint16_t)my_scale));
#pragma unroll
            for (int i = 0; i < ITERS; ++i) {
                const float s = __shfl_sync(0xffffffffu, my_s, g.row_group ? 0 : 2 * i + (lane >> 4));
                const uint32_t w[2] = {c[i].x, c[i].y};
                uint32_t o[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    // code -> float without the conversion unit: the sign-flipped byte under the exponent of 2^23 is
                    // 8388608 + code + 128 exactly; one subtraction gives the code
                    const uint32_t u = w[k >> 1] ^ 0x80808080u;
                    const float qa = __uint_as_float(__byte_perm(u, 0x4b000000u, (k & 1) ? 0x7652 : 0x7650)) - 8388736.0f;
                    const float qb = __uint_as_float(__byte_perm(u, 0x4b000000u, (k & 1) ? 0x7653 : 0x7651)) - 8388736.0f;
                    o[k] = as_u32(__floats2half2_rn(__fmul_rn(qa, s), __fmul_rn(qb, s)));
                }
                st_stream(dst + i * 32, make_uint4(o[0], o[1], o[2], o[3]));
            }
        } else {
            const uint32_t* src = reinterpret_cast<const uint32_t*>(pp.int4_codes + prow * (size_t)(g.HD / 2)) + lane;
            uint32_t c[ITERS];
#pragma unroll
            for (int i = 0; i < ITERS; ++i) c[i] = ld_stream(src + i * 32);
            uint32_t my_sz = 0;
            if (lane < g.ng) my_sz = reinterpret_cast<const uint32_t*>(pp.int4_sz + prow * (size_t)g.ng * 4)[lane];
            const float my_s = __half2float(__ushort_as_half((uint16_t)(my_sz & 0xffff)));
            const float my_z = __half2float(__ushort_as_half((uint16_t)(my_sz >> 16)));
#pragma unroll
            for (int i = 0; i < ITERS; ++i) {
                const int owner = g.row_group ? 0 : 2 * i + (lane >> 4);
                const float s = __shfl_sync(0xffffffffu, my_s, owner);
                const float z = __shfl_sync(0xffffffffu, my_z, owner);
                uint32_t o[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    // code -> float without the conversion unit: the nibble under the exponent of 2^23 is 8388608 + code
                    const float qa = __uint_as_float(((c[i] >> (8 * k)) & 15u) | 0x4b000000u) - 8388608.0f;
                    const float qb = __uint_as_float(((c[i] >> (8 * k + 4)) & 15u) | 0x4b000000u) - 8388608.0f;
                    o[k] = as_u32(__floats2half2_rn(__fadd_rn(__fmul_rn(qa, s), z), __fadd_rn(__fmul_rn(qb, s), z)));
                }
                st_stream(dst + i * 32, make_uint4(o[0], o[1], o[2], o[3]));
            }
        }
    }
}

// Zero the rows of pruned tokens: one CTA per (frame, plane).
__global__ void __launch_bounds__(KV_THREADS)
k_zero_pruned(__half* __restrict__ K, __half* __restrict__ V, KvGeom g, const uint8_t* __restrict__ decision) {
    const int b = blockIdx.y, plane = blockIdx.x, layer = plane >> 1, kv = plane & 1;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    __half* base = (kv ? V : K) + (size_t)b * g.frame_stride + (size_t)layer * g.n_tok * g.HD;
    const int iters = g.HD / 8 / 32;
    for (int t = wid; t < g.n_tok; t += KV_WARPS) {
        if (decision[(size_t)b * g.n_tok + t] != SALICACHE_PRUNE) continue;
        uint4* dst = reinterpret_cast<uint4*>(base + (size_t)t * g.HD);
        for (int i = 0; i < iters; ++i) st_stream(dst + i * 32 + lane, make_uint4(0, 0, 0, 0));
    }
}

PoolPtrs make_pools(const salicache_pools* p) {
    PoolPtrs pp;
    pp.fp16_pool = (uint8_t*)p->fp16_pool;
    pp.int8_codes = (uint8_t*)p->int8_codes;
    pp.int8_scale = (uint8_t*)p->int8_scale;
    pp.int4_codes = (uint8_t*)p->int4_codes;
    pp.int4_sz = (uint8_t*)p->int4_sz;
    pp.cap0 = p->cap_fp16;
    pp.cap1 = p->cap_int8;
    pp.cap2 = p->cap_int4;
    pp.ring = p->ring;
    pp.fill = (const long long*)p->d_fill;
    return pp;
}

template <int ITERS>
void launch_pack(int grid, size_t smem, cudaStream_t st, const __half* K, const __half* V, const KvGeom& g,
                 const int32_t* idx, const int32_t* counts, const long long* off, const PoolPtrs& pp, int* status) {
    if (g.row_group) k_pack<ITERS, true><<<grid, KV_THREADS, smem, st>>>(K, V, g, idx, counts, off, pp, status);
    else k_pack<ITERS, false><<<grid, KV_THREADS, smem, st>>>(K, V, g, idx, counts, off, pp, status);
}
template <int ITERS>
void launch_unpack(int grid, size_t smem, cudaStream_t st, __half* K, __half* V, const KvGeom& g, const int32_t* idx,
                   const int32_t* counts, const long long* off, const PoolPtrs& pp, int* status) {
    k_unpack<ITERS><<<grid, KV_THREADS, smem, st>>>(K, V, g, idx, counts, off, pp, status);
}

}  // namespace

int sc_kv_max_batch() { return MAX_PREFIX; }

// Row lengths the kernels are instantiated for (HD = 256 * ITERS).
bool sc_kv_supported_hd(int HD) { return HD == 4096 || HD == 2048 || HD == 1024 || HD == 512 || HD == 256; }

// Work units of one call are counted in 32 bits on the device.
static bool units_fit(const salicache_ctx* c, int B) { return (long long)B * c->n_tok * 2 * c->p.L < (1ll << 31); }

int sc_pack(salicache_ctx* c, const void* d_K, const void* d_V, int64_t frame_stride, const int32_t* d_idx,
            const int32_t* d_counts, const int64_t* d_row_offset, int B, const salicache_pools* pools, cudaStream_t st) {
    if (B == 0) return SALICACHE_OK;
    if (!units_fit(c, B)) return SALICACHE_E_SHAPE;
    const int HD = c->p.heads * c->p.head_dim;
    const int row_group = c->p.group == HD ? 1 : 0;
    KvGeom g{c->p.L, c->n_tok, HD, row_group ? 1 : HD / 128, frame_stride, B, row_group};
    const int grid = c->sm_count * 2;
    const size_t smem = (size_t)(B + 1) * sizeof(int);
    const __half* K = (const __half*)d_K;
    const __half* V = (const __half*)d_V;
    const long long* off = (const long long*)d_row_offset;
    PoolPtrs pp = make_pools(pools);
    switch (HD / 256) {
        case 16: launch_pack<16>(grid, smem, st, K, V, g, d_idx, d_counts, off, pp, c->d_status); break;
        case 8: launch_pack<8>(grid, smem, st, K, V, g, d_idx, d_counts, off, pp, c->d_status); break;
        case 4: launch_pack<4>(grid, smem, st, K, V, g, d_idx, d_counts, off, pp, c->d_status); break;
        case 2: launch_pack<2>(grid, smem, st, K, V, g, d_idx, d_counts, off, pp, c->d_status); break;
        case 1: launch_pack<1>(grid, smem, st, K, V, g, d_idx, d_counts, off, pp, c->d_status); break;
        default: return SALICACHE_E_PARAM;
    }
    c->launches++;
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}

int sc_unpack(salicache_ctx* c, const salicache_pools* pools, const int32_t* d_idx, const int32_t* d_counts,
              const uint8_t* d_decision, const int64_t* d_row_offset, int B, int zero_fill_pruned, void* d_K_out,
              void* d_V_out, int64_t frame_stride, cudaStream_t st) {
    if (B == 0) return SALICACHE_OK;
    if (!units_fit(c, B)) return SALICACHE_E_SHAPE;
    const int HD = c->p.heads * c->p.head_dim;
    const int row_group = c->p.group == HD ? 1 : 0;
    KvGeom g{c->p.L, c->n_tok, HD, row_group ? 1 : HD / 128, frame_stride, B, row_group};
    const int grid = c->sm_count * 2;
    const size_t smem = (size_t)(B + 1) * sizeof(int);
    __half* K = (__half*)d_K_out;
    __half* V = (__half*)d_V_out;
    const long long* off = (const long long*)d_row_offset;
    PoolPtrs pp = make_pools(pools);
    switch (HD / 256) {
        case 16: launch_unpack<16>(grid, smem, st, K, V, g, d_idx, d_counts, off, pp, c->d_status); break;
        case 8: launch_unpack<8>(grid, smem, st, K, V, g, d_idx, d_counts, off, pp, c->d_status); break;
        case 4: launch_unpack<4>(grid, smem, st, K, V, g, d_idx, d_counts, off, pp, c->d_status); break;
        case 2: launch_unpack<2>(grid, smem, st, K, V, g, d_idx, d_counts, off, pp, c->d_status); break;
        case 1: launch_unpack<1>(grid, smem, st, K, V, g, d_idx, d_counts, off, pp, c->d_status); break;
        default: return SALICACHE_E_PARAM;
    }
    c->launches++;
    if (zero_fill_pruned) {
        dim3 gz(2 * g.L, B);
        k_zero_pruned<<<gz, KV_THREADS, 0, st>>>(K, V, g, d_decision);
        c->launches++;
    }
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}
