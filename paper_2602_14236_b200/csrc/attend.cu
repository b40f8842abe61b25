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
    __shared__ __align__(16) float qs[AT_D];        // the query, scaled by 1 / sqrt(D)
    __shared__ float pw[AT_D];                      // softmax weights of the tile's rows
    __shared__ int rinfo[AT_D];                     // tier << 28 | pool row
    __shared__ float red[AT_WARPS];
    __shared__ float part[AT_WARPS][AT_D];
    const int c = blockIdx.x, h = blockIdx.y, l = blockIdx.z, t = threadIdx.x;
    const int lane = t & 31, wid = t >> 5;
    const int HD = H * AT_D;
    const long long n16 = min(fill[0], pp.cap16), n8 = min(fill[1], pp.cap8), n4 = min(fill[2], pp.cap4);
    const long long R = n16 + n8 + n4;
    const long long per = (R + AT_CHUNKS - 1) / AT_CHUNKS;
    const long long r0 = (long long)c * per, r1 = min(R, r0 + per);
    qs[t] = __half2float(q[((size_t)l * H + h) * AT_D + t]) * rsqrtf((float)AT_D);
    __syncthreads();
    float qsum = block_sum(qs[t], red);             // the INT4 zero point adds z * sum(q) to a score
    const int g = ng == 1 ? 0 : h;                  // group of this head's elements in a row's scale array
    float m = -INFINITY, den = 0.0f;
    float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    const float4* q4 = reinterpret_cast<const float4*>(qs);
    for (long long tile = r0; tile < r1; tile += AT_D) {
        const long long r = tile + t;
        float s = -INFINITY;
        int info = 0;
        if (r < r1) {
            float dot = 0.0f;
            if (r < n16) {
                const size_t prow = (size_t)(2 * l) * pp.cap16 + r;
                const uint4* kp = reinterpret_cast<const uint4*>(pp.fp16_pool + (prow * HD + (size_t)h * AT_D) * 2);
                info = (int)r;
#pragma unroll 4
                for (int i = 0; i < AT_D / 8; ++i) {
                    const uint4 w = __ldg(kp + i);
                    const float4 qa = q4[2 * i], qb = q4[2 * i + 1];
                    const float2 a = w2f(w.x), b = w2f(w.y), cc = w2f(w.z), d = w2f(w.w);
                    dot += a.x * qa.x + a.y * qa.y + b.x * qa.z + b.y * qa.w + cc.x * qb.x + cc.y * qb.y + d.x * qb.z + d.y * qb.w;
                }
                s = dot;
            } else if (r < n16 + n8) {
                const long long row = r - n16;
                const size_t prow = (size_t)(2 * l) * pp.cap8 + row;
                const uint4* kp = reinterpret_cast<const uint4*>(pp.int8_codes + prow * HD + (size_t)h * AT_D);
                info = (1 << 28) | (int)row;
#pragma unroll 2
                for (int i = 0; i < AT_D / 16; ++i) {
                    const uint4 w = __ldg(kp + i);
                    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float4 qa = q4[4 * i + k];
                        dot += (float)(int8_t)(ww[k] & 255) * qa.x + (float)(int8_t)((ww[k] >> 8) & 255) * qa.y +
                               (float)(int8_t)((ww[k] >> 16) & 255) * qa.z + (float)(int8_t)(ww[k] >> 24) * qa.w;
                    }
                }
                s = dot * h2f(reinterpret_cast<const uint16_t*>(pp.int8_scale)[prow * ng + g]);
            } else {
                const long long row = r - n16 - n8;
                const size_t prow = (size_t)(2 * l) * pp.cap4 + row;
                const uint4* kp = reinterpret_cast<const uint4*>(pp.int4_codes + prow * (HD / 2) + (size_t)h * (AT_D / 2));
                info = (2 << 28) | (int)row;
#pragma unroll 2
                for (int i = 0; i < AT_D / 32; ++i) {
                    const uint4 w = __ldg(kp + i);
                    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float4 qa = q4[8 * i + 2 * k], qb = q4[8 * i + 2 * k + 1];
                        const uint32_t x = ww[k];
                        dot += (float)(x & 15) * qa.x + (float)((x >> 4) & 15) * qa.y + (float)((x >> 8) & 15) * qa.z +
                               (float)((x >> 12) & 15) * qa.w + (float)((x >> 16) & 15) * qb.x + (float)((x >> 20) & 15) * qb.y +
                               (float)((x >> 24) & 15) * qb.z + (float)(x >> 28) * qb.w;
                    }
                }
                const uint32_t sz = reinterpret_cast<const uint32_t*>(pp.int4_sz)[prow * ng + g];
                s = dot * h2f((uint16_t)(sz & 0xffff)) + qsum * h2f((uint16_t)(sz >> 16));
            }
        }
        // online softmax: new running maximum, rescale what has been accumulated so far
        const float mt = block_max(s, red);
        const float m_new = fmaxf(m, mt);
        const float corr = m == -INFINITY ? 0.0f : __expf(m - m_new);
        const float p = r < r1 ? __expf(s - m_new) : 0.0f;
        pw[t] = p;
        rinfo[t] = info;
        den = den * corr + block_sum(p, red);       // (its barriers also publish pw and rinfo)
        m = m_new;
#pragma unroll
        for (int k = 0; k < 4; ++k) acc[k] *= corr;
        // values: warp w takes the tile's rows w, w + 4, ...; a lane owns dimensions 4 * lane .. 4 * lane + 3
        const int n_tile = (int)min((long long)AT_D, r1 - tile);
        for (int rr = wid; rr < n_tile; rr += AT_WARPS) {
            const float pr = pw[rr];
            const int inf = rinfo[rr], tier = inf >> 28, row = inf & 0x0fffffff;
            if (tier == 0) {
                const size_t prow = (size_t)(2 * l + 1) * pp.cap16 + row;
                const uint2 w = __ldg(reinterpret_cast<const uint2*>(pp.fp16_pool + (prow * HD + (size_t)h * AT_D) * 2) + lane);
                const float2 a = w2f(w.x), b = w2f(w.y);
                acc[0] += pr * a.x; acc[1] += pr * a.y; acc[2] += pr * b.x; acc[3] += pr * b.y;
            } else if (tier == 1) {
                const size_t prow = (size_t)(2 * l + 1) * pp.cap8 + row;
                const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(pp.int8_codes + prow * HD + (size_t)h * AT_D) + lane);
                const float ps = pr * h2f(reinterpret_cast<const uint16_t*>(pp.int8_scale)[prow * ng + g]);
                acc[0] += ps * (float)(int8_t)(w & 255); acc[1] += ps * (float)(int8_t)((w >> 8) & 255);
                acc[2] += ps * (float)(int8_t)((w >> 16) & 255); acc[3] += ps * (float)(int8_t)(w >> 24);
            } else {
                const size_t prow = (size_t)(2 * l + 1) * pp.cap4 + row;
                const uint32_t w = __ldg(reinterpret_cast<const uint16_t*>(pp.int4_codes + prow * (HD / 2) + (size_t)h * (AT_D / 2)) + lane);
                const uint32_t sz = reinterpret_cast<const uint32_t*>(pp.int4_sz)[prow * ng + g];
                const float ps = pr * h2f((uint16_t)(sz & 0xffff)), pz = pr * h2f((uint16_t)(sz >> 16));
                acc[0] += ps * (float)(w & 15) + pz; acc[1] += ps * (float)((w >> 4) & 15) + pz;
                acc[2] += ps * (float)((w >> 8) & 15) + pz; acc[3] += ps * (float)((w >> 12) & 15) + pz;
            }
        }
        __syncthreads();                            // pw / rinfo are rewritten by the next tile
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) part[wid][4 * lane + k] = acc[k];
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
    dim3 grid(AT_CHUNKS, p.heads, p.L);
    k_attend_partial<<<grid, AT_D, 0, st>>>((const __half*)d_q, pp, (const long long*)d_fill, p.heads, ng, c->attend_ws);
    dim3 gm(p.heads, p.L);
    k_attend_merge<<<gm, AT_D, 0, st>>>(c->attend_ws, p.heads, d_out);
    c->launches += 2;
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}
