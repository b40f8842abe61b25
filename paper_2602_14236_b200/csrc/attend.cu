// Decode attention over the mixed-precision store with the dequantisation fused in (Eq. 2; Sec. III-C:
// "just-in-time" dequantisation inside the attention computation).  One query per layer and head attends
// to every row the three pools hold; codes are expanded in registers and never written back.
//
//   score_j = q_h . K^_{j,h} / sqrt(D),   p = softmax_j(score),   out_h = sum_j p_j V^_{j,h}
//
// Split over the rows (AT_CHUNKS partial results per layer and head, merged by a second kernel).  Within a
// CTA the scores are computed one row per thread (the thread walks the head's 128 key elements of its row:
// no cross-lane reduction), the softmax statistics are kept online, and the values are accumulated four
// dimensions per lane, one row per warp at a time.  Single precision throughout.
#include <cuda_fp16.h>
#include <math.h>

#include "common.cuh"

namespace {

constexpr int AT_D = 128;           // head size = threads per CTA = quantisation group
constexpr int AT_WARPS = AT_D / 32;
constexpr int AT_CHUNKS = 64;       // partial results per (layer, head)
constexpr int AT_REC = AT_D + 2;    // partial record: 128 sums, running maximum, running denominator

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

// c + a.lo * b.lo + a.hi * b.hi with a, b pairs of binary16: the mixed-precision multiply-add forms each
// product exactly and rounds the sum once to binary32.
__device__ __forceinline__ float dot2(uint32_t a, uint32_t b, float c) {
    float d;
    asm("{ .reg .b16 al, ah, bl, bh; .reg .f32 t; mov.b32 {al, ah}, %1; mov.b32 {bl, bh}, %2;\n\t"
        "fma.rn.f32.f16 t, al, bl, %3; fma.rn.f32.f16 %0, ah, bh, t; }"
        : "=f"(d)
        : "r"(a), "r"(b), "f"(c));
    return d;
}
__device__ __forceinline__ uint32_t hsub2u(uint32_t a, uint32_t b) {
    __half2 r = __hsub2(*reinterpret_cast<const __half2*>(&a), *reinterpret_cast<const __half2*>(&b));
    return *reinterpret_cast<const uint32_t*>(&r);
}
// Codes to binary16 without integer-to-float conversions: OR the code into the mantissa of 1024 (binary16
// 0x6400, unit in the last place 1) and subtract 1024 again; both steps are exact.
// Four INT4 code pairs of a word of 8 nibbles e0..e7: (e0,e4) (e1,e5) (e2,e6) (e3,e7).
__device__ __forceinline__ void nibbles_to_h2(uint32_t x, uint32_t out[4]) {
#pragma unroll
    for (int k = 0; k < 4; ++k) out[k] = hsub2u(((x >> (4 * k)) & 0x000f000fu) | 0x64006400u, 0x64006400u);
}
// Two INT8 code pairs of a word of 4 bytes b0..b3: (b0,b1) (b2,b3).  The bytes are biased by 128 first.
__device__ __forceinline__ void bytes_to_h2(uint32_t w, uint32_t out[2]) {
    const uint32_t u = w ^ 0x80808080u;
    out[0] = hsub2u(__byte_perm(u, 0x64646464u, 0x4140), 0x64806480u);
    out[1] = hsub2u(__byte_perm(u, 0x64646464u, 0x4342), 0x64806480u);
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

__global__ void __launch_bounds__(AT_D)
k_attend_partial(const __half* __restrict__ q, AtPools pp, const long long* __restrict__ fill, int H, int ng,
                 float* __restrict__ ws) {
    __shared__ __align__(16) float qs[AT_D];        // the query as binary32 (for sum(q))
    __shared__ __align__(16) __half qn[AT_D];       // the query in natural order
    __shared__ __align__(16) __half qp[AT_D];       // the query with every 8 elements ordered 0 4 1 5 2 6 3 7 (INT4 pairs)
    __shared__ float4 rowrec[AT_D];                 // per row of the tile: weight * value scale, weight * value zero,
                                                    // pool row (as an integer)
    __shared__ float red[AT_WARPS];
    __shared__ float part[AT_WARPS][AT_D];
    // heads vary fastest over the grid: the CTAs that read the 32 slices of one row run at about the same time
    const int h = blockIdx.x, c = blockIdx.y, l = blockIdx.z, t = threadIdx.x;
    const int lane = t & 31, wid = t >> 5;
    const int HD = H * AT_D;
    const long long n16 = min(fill[0], pp.cap16), n8 = min(fill[1], pp.cap8), n4 = min(fill[2], pp.cap4);
    const long long R = n16 + n8 + n4;
    const long long per = (R + AT_CHUNKS - 1) / AT_CHUNKS;
    const long long r0 = (long long)c * per, r1 = min(R, r0 + per);
    {
        const __half qv = q[((size_t)l * H + h) * AT_D + t];
        const int e = t & 7;
        qs[t] = __half2float(qv);
        qn[t] = qv;
        qp[(t & ~7) | ((e & 3) * 2 + (e >> 2))] = qv;      // element e of its octet goes to slot 2 (e mod 4) + e div 4
    }
    __syncthreads();
    const float rs = rsqrtf((float)AT_D);
    float qsum = block_sum(qs[t], red);             // the INT4 zero point adds z * sum(q) to a score
    const int g = ng == 1 ? 0 : h;                  // group of this head's elements in a row's scale array
    float m = -INFINITY, den = 0.0f;
    float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    float zacc = 0.0f;                              // sum of p * zero over this warp's INT4 rows: the same for every dimension
    // this lane's slice of the head's values in row 0 of each pool's V plane of layer l
    const uint8_t* vbase16 = pp.fp16_pool + (((size_t)(2 * l + 1) * pp.cap16) * HD + (size_t)h * AT_D) * 2 + lane * 8;
    const uint8_t* vbase8 = pp.int8_codes + ((size_t)(2 * l + 1) * pp.cap8) * HD + (size_t)h * AT_D + lane * 4;
    const uint8_t* vbase4 = pp.int4_codes + ((size_t)(2 * l + 1) * pp.cap4) * (HD / 2) + (size_t)h * (AT_D / 2) + lane * 2;
    const uint4* qn4 = reinterpret_cast<const uint4*>(qn);
    const uint4* qp4 = reinterpret_cast<const uint4*>(qp);
    for (long long tile = r0; tile < r1; tile += AT_D) {
        const long long r = tile + t;
        float s = -INFINITY;
        int vrow = 0;
        float vsc = 1.0f, vzr = 0.0f;               // scale and zero of the row's VALUE slice (its key has its own)
        if (r < r1) {
            float dot = 0.0f;
            if (r < n16) {
                const size_t prow = (size_t)(2 * l) * pp.cap16 + r;
                const uint4* kp = reinterpret_cast<const uint4*>(pp.fp16_pool + (prow * HD + (size_t)h * AT_D) * 2);
                vrow = (int)r;
#pragma unroll 4
                for (int i = 0; i < AT_D / 8; ++i) {
                    const uint4 w = __ldg(kp + i), qq = qn4[i];
                    dot = dot2(w.x, qq.x, dot);
                    dot = dot2(w.y, qq.y, dot);
                    dot = dot2(w.z, qq.z, dot);
                    dot = dot2(w.w, qq.w, dot);
                }
                s = dot * rs;
            } else if (r < n16 + n8) {
                const long long row = r - n16;
                const size_t prow = (size_t)(2 * l) * pp.cap8 + row;
                const uint4* kp = reinterpret_cast<const uint4*>(pp.int8_codes + prow * HD + (size_t)h * AT_D);
                vrow = (int)row;
                vsc = h2f(reinterpret_cast<const uint16_t*>(pp.int8_scale)[((size_t)(2 * l + 1) * pp.cap8 + row) * ng + g]);
#pragma unroll 2
                for (int i = 0; i < AT_D / 16; ++i) {
                    const uint4 w = __ldg(kp + i);
                    const uint4 qa = qn4[2 * i], qb = qn4[2 * i + 1];
                    uint32_t c[2];
                    bytes_to_h2(w.x, c); dot = dot2(c[0], qa.x, dot); dot = dot2(c[1], qa.y, dot);
                    bytes_to_h2(w.y, c); dot = dot2(c[0], qa.z, dot); dot = dot2(c[1], qa.w, dot);
                    bytes_to_h2(w.z, c); dot = dot2(c[0], qb.x, dot); dot = dot2(c[1], qb.y, dot);
                    bytes_to_h2(w.w, c); dot = dot2(c[0], qb.z, dot); dot = dot2(c[1], qb.w, dot);
                }
                s = dot * (rs * h2f(reinterpret_cast<const uint16_t*>(pp.int8_scale)[prow * ng + g]));
            } else {
                const long long row = r - n16 - n8;
                const size_t prow = (size_t)(2 * l) * pp.cap4 + row;
                const uint4* kp = reinterpret_cast<const uint4*>(pp.int4_codes + prow * (HD / 2) + (size_t)h * (AT_D / 2));
                float d4[4] = {0.0f, 0.0f, 0.0f, 0.0f};      // four partial sums: shorter dependency chains
                vrow = (int)row;
                {
                    const uint32_t vz = reinterpret_cast<const uint32_t*>(pp.int4_sz)[((size_t)(2 * l + 1) * pp.cap4 + row) * ng + g];
                    vsc = h2f((uint16_t)(vz & 0xffff));
                    vzr = h2f((uint16_t)(vz >> 16));
                }
#pragma unroll 2
                for (int i = 0; i < AT_D / 32; ++i) {
                    const uint4 w = __ldg(kp + i);
                    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint4 qq = qp4[4 * i + k];
                        uint32_t c[4];
                        nibbles_to_h2(ww[k], c);
                        d4[0] = dot2(c[0], qq.x, d4[0]);
                        d4[1] = dot2(c[1], qq.y, d4[1]);
                        d4[2] = dot2(c[2], qq.z, d4[2]);
                        d4[3] = dot2(c[3], qq.w, d4[3]);
                    }
                }
                dot = (d4[0] + d4[1]) + (d4[2] + d4[3]);
                const uint32_t sz = reinterpret_cast<const uint32_t*>(pp.int4_sz)[prow * ng + g];
                s = rs * (dot * h2f((uint16_t)(sz & 0xffff)) + qsum * h2f((uint16_t)(sz >> 16)));
            }
        }
        // online softmax: new running maximum, rescale what has been accumulated so far
        const float mt = block_max(s, red);
        const float m_new = fmaxf(m, mt);
        const float corr = m == -INFINITY ? 0.0f : __expf(m - m_new);
        const float p = r < r1 ? __expf(s - m_new) : 0.0f;
        rowrec[t] = make_float4(p * vsc, p * vzr, __int_as_float(vrow), 0.0f);
        den = den * corr + block_sum(p, red);       // (its barriers also publish rowrec)
        m = m_new;
#pragma unroll
        for (int k = 0; k < 4; ++k) acc[k] *= corr;
        zacc *= corr;
        // values: warp w takes the tile's rows w, w + 4, ...; a lane owns dimensions 4 * lane .. 4 * lane + 3
        const int n_tile = (int)min((long long)AT_D, r1 - tile);
        // the rows of a tile are ordered by tier (FP16, INT8, INT4): three loops without a per-row branch
        const int e16 = (int)max(0ll, min((long long)n_tile, n16 - tile));
        const int e8 = (int)max(0ll, min((long long)n_tile, n16 + n8 - tile));
        int rr = wid;
        for (; rr < e16; rr += AT_WARPS) {
            const float4 rec = rowrec[rr];
            const uint2 w = __ldg(reinterpret_cast<const uint2*>(vbase16 + (size_t)__float_as_int(rec.z) * ((size_t)HD * 2)));
            const float2 a = w2f(w.x), b = w2f(w.y);
            acc[0] += rec.x * a.x; acc[1] += rec.x * a.y; acc[2] += rec.x * b.x; acc[3] += rec.x * b.y;
        }
        for (; rr < e8; rr += AT_WARPS) {
            const float4 rec = rowrec[rr];
            const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(vbase8 + (size_t)__float_as_int(rec.z) * (size_t)HD));
            uint32_t cw[2];
            bytes_to_h2(w, cw);
            const float2 a = w2f(cw[0]), b = w2f(cw[1]);
            acc[0] += rec.x * a.x; acc[1] += rec.x * a.y; acc[2] += rec.x * b.x; acc[3] += rec.x * b.y;
        }
#pragma unroll 4
        for (; rr < n_tile; rr += AT_WARPS) {
            const float4 rec = rowrec[rr];
            const uint32_t w = __ldg(reinterpret_cast<const uint16_t*>(vbase4 + (size_t)__float_as_int(rec.z) * (size_t)(HD / 2)));
            const uint32_t y = __byte_perm(w, 0u, 0x4140);      // bytes (e1 e0) 0 (e3 e2) 0: pairs (e0,e2), (e1,e3) by one mask
            const float2 a = w2f(hsub2u((y & 0x000f000fu) | 0x64006400u, 0x64006400u));
            const float2 b = w2f(hsub2u(((y >> 4) & 0x000f000fu) | 0x64006400u, 0x64006400u));
            acc[0] += rec.x * a.x; acc[1] += rec.x * b.x; acc[2] += rec.x * a.y; acc[3] += rec.x * b.y;
            zacc += rec.y;
        }
        __syncthreads();                            // rowrec is rewritten by the next tile
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) part[wid][4 * lane + k] = acc[k] + zacc;
    __syncthreads();
    float* rec = ws + (((size_t)l * H + h) * AT_CHUNKS + c) * AT_REC;
    float sum = 0.0f;
#pragma unroll
    for (int k = 0; k < AT_WARPS; ++k) sum += part[k][t];
    rec[t] = sum;
    if (t == 0) {
        rec[AT_D] = m;
        rec[AT_D + 1] = den;
    }
}

// Merge the partial results of one (layer, head): out = sum_c e^(m_c - M) acc_c / sum_c e^(m_c - M) den_c.
__global__ void __launch_bounds__(AT_D)
k_attend_merge(const float* __restrict__ ws, int H, float* __restrict__ out) {
    const int h = blockIdx.x, l = blockIdx.y, t = threadIdx.x;
    const float* rec = ws + ((size_t)l * H + h) * AT_CHUNKS * AT_REC;
    float M = -INFINITY;
    for (int c = 0; c < AT_CHUNKS; ++c) M = fmaxf(M, rec[c * AT_REC + AT_D]);
    float num = 0.0f, den = 0.0f;
    if (M != -INFINITY)
        for (int c = 0; c < AT_CHUNKS; ++c) {
            const float mc = rec[c * AT_REC + AT_D];
            if (mc == -INFINITY) continue;
            const float e = __expf(mc - M);
            num += e * rec[c * AT_REC + t];
            den += e * rec[c * AT_REC + AT_D + 1];
        }
    out[((size_t)l * H + h) * AT_D + t] = den > 0.0f ? num / den : 0.0f;
}

}  // namespace

size_t sc_attend_workspace_bytes(int L, int H) { return (size_t)L * H * AT_CHUNKS * AT_REC * sizeof(float); }

int sc_attend(salicache_ctx* c, const void* d_q, const salicache_pools* pools, const int64_t* d_fill, float* d_out,
              cudaStream_t st) {
    const salicache_params& p = c->p;
    if (p.head_dim != AT_D || (p.group != AT_D && p.group != p.heads * p.head_dim)) return SALICACHE_E_PARAM;
    AtPools pp{(const uint8_t*)pools->fp16_pool, (const uint8_t*)pools->int8_codes, (const uint8_t*)pools->int8_scale,
               (const uint8_t*)pools->int4_codes, (const uint8_t*)pools->int4_sz, pools->cap_fp16, pools->cap_int8,
               pools->cap_int4};
    if (pp.cap16 >= (1ll << 28) || pp.cap8 >= (1ll << 28) || pp.cap4 >= (1ll << 28)) return SALICACHE_E_SHAPE;
    const int ng = p.group == AT_D ? p.heads : 1;
    dim3 grid(p.heads, AT_CHUNKS, p.L);
    k_attend_partial<<<grid, AT_D, 0, st>>>((const __half*)d_q, pp, (const long long*)d_fill, p.heads, ng, c->attend_ws);
    dim3 gm(p.heads, p.L);
    k_attend_merge<<<gm, AT_D, 0, st>>>(c->attend_ws, p.heads, d_out);
    c->launches += 2;
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}
