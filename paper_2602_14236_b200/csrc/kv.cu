// Mixed-precision K/V store (Alg. 1 line 16; quantisers of Sec. IV-B) and its just-in-time
// dequantisation (Sec. III-C).  HBM-bound: one warp moves one 8 KiB token row (HD = 4096 fp16) with
// 16-byte loads, one quantisation group (128 elements) per half warp, packed stores.
#include <cuda_fp16.h>

#include "common.cuh"

namespace {

constexpr int KV_THREADS = 256;
constexpr int KV_WARPS = KV_THREADS / 32;
constexpr int MAX_PREFIX = 4096;   // frames per call whose row prefix fits the shared-memory table

struct KvGeom {
    int L, n_tok, HD, ng;          // ng = HD / 128
    long long frame_stride;        // fp16 elements between frames
    int B;
};

struct PoolPtrs {
    uint8_t* fp16_pool;
    uint8_t* int8_codes;
    uint8_t* int8_scale;
    uint8_t* int4_codes;
    uint8_t* int4_sz;
    long long cap[3];
    int ring;
};

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
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

// Rows stored before each frame of the batch, built by every CTA in shared memory from the counts.
__device__ __forceinline__ void build_prefix(const int32_t* __restrict__ counts, int B, int* pre) {
    // pre[b] = sum_{b' < b} (n16 + n8 + n4); B <= MAX_PREFIX
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

// Work unit u -> (frame b, plane = layer*2 + kv, position j in the frame's stored-row list).
struct Unit {
    int b, plane, tier, j, tok;
    long long row;   // pool row, or -1 when dropped
};

__device__ __forceinline__ Unit decode_unit(long long u, const int* pre, int B, int planes,
                                            const int32_t* __restrict__ counts, const int32_t* __restrict__ idx,
                                            const long long* __restrict__ row_offset, int n_tok, const long long* cap,
                                            int ring) {
    Unit r;
    int q = (int)(u / planes);          // lies in [pre[b], pre[b+1]) of exactly one frame
    int lo = 0, hi = B;                 // largest b with pre[b] <= q
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (pre[mid] <= q) lo = mid; else hi = mid;
    }
    r.b = lo;
    int stored = pre[lo + 1] - pre[lo];
    long long local = u - (long long)pre[lo] * planes;
    r.plane = (int)(local / stored);
    int j = (int)(local % stored);
    int n16 = counts[lo * 5 + SALICACHE_FP16], n8 = counts[lo * 5 + SALICACHE_INT8];
    if (j < n16) r.tier = 0;
    else if (j < n16 + n8) { r.tier = 1; j -= n16; }
    else { r.tier = 2; j -= n16 + n8; }
    r.j = j;
    r.tok = idx[((size_t)lo * 3 + r.tier) * n_tok + j];
    long long row = row_offset[(size_t)lo * 3 + r.tier] + j;
    long long cp = cap[r.tier];
    if (ring) row = cp > 0 ? row % cp : -1;
    else if (row >= cp) row = -1;
    r.row = row;
    return r;
}

// ---- pack ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(KV_THREADS)
k_pack(const __half* __restrict__ K, const __half* __restrict__ V, KvGeom g, const int32_t* __restrict__ idx,
       const int32_t* __restrict__ counts, const long long* __restrict__ row_offset, PoolPtrs pp,
       int* __restrict__ status) {
    extern __shared__ int pre[];
    build_prefix(counts, g.B, pre);
    const int planes = 2 * g.L;
    const long long n_units = (long long)pre[g.B] * planes;
    const int lane = threadIdx.x & 31;
    const int half_id = lane >> 4;
    const long long warp0 = (long long)blockIdx.x * KV_WARPS + (threadIdx.x >> 5);
    const long long wstride = (long long)gridDim.x * KV_WARPS;
    const int vec_per_row = g.HD / 8;             // uint4 per row (512)
    const int iters = vec_per_row / 32;           // 16
    for (long long u = warp0; u < n_units; u += wstride) {
        Unit un = decode_unit(u, pre, g.B, planes, counts, idx, row_offset, g.n_tok, pp.cap, pp.ring);
        if (un.row < 0) {
            if (lane == 0) atomicMin(status, SALICACHE_E_CAPACITY);
            continue;
        }
        const int layer = un.plane >> 1, kv = un.plane & 1;
        const __half* src_h = (kv ? V : K) + (size_t)un.b * g.frame_stride + ((size_t)layer * g.n_tok + un.tok) * g.HD;
        const uint4* src = reinterpret_cast<const uint4*>(src_h);
        const size_t prow = (size_t)un.plane * pp.cap[un.tier] + un.row;
        if (un.tier == 0) {
            uint4* dst = reinterpret_cast<uint4*>(pp.fp16_pool + prow * (size_t)g.HD * 2);
#pragma unroll 8
            for (int i = 0; i < iters; ++i) st_stream(dst + i * 32 + lane, ld_stream(src + i * 32 + lane));
        } else if (un.tier == 1) {
            uint2* dst = reinterpret_cast<uint2*>(pp.int8_codes + prow * (size_t)g.HD);
            uint32_t my_scale = 0;
#pragma unroll 8
            for (int i = 0; i < iters; ++i) {
                uint4 v = ld_stream(src + i * 32 + lane);
                __half2 h0 = as_h2(v.x), h1 = as_h2(v.y), h2 = as_h2(v.z), h3 = as_h2(v.w);
                __half2 m = __hmax2(__hmax2(__habs2(h0), __habs2(h1)), __hmax2(__habs2(h2), __habs2(h3)));
#pragma unroll
                for (int o = 8; o; o >>= 1) m = __hmax2(m, as_h2(__shfl_xor_sync(0xffffffffu, as_u32(m), o)));
                float amax = fmaxf(__low2float(m), __high2float(m));
                __half s16 = __float2half_rn(__fdiv_rn(amax, 127.0f));
                if (__half_as_ushort(s16) == 0) s16 = __ushort_as_half(0x3c00);
                float inv = __fdiv_rn(1.0f, __half2float(s16));
                float2 f0 = __half22float2(h0), f1 = __half22float2(h1), f2 = __half22float2(h2), f3 = __half22float2(h3);
                int q0 = __float2int_rn(__fmul_rn(f0.x, inv)), q1 = __float2int_rn(__fmul_rn(f0.y, inv));
                int q2 = __float2int_rn(__fmul_rn(f1.x, inv)), q3 = __float2int_rn(__fmul_rn(f1.y, inv));
                int q4 = __float2int_rn(__fmul_rn(f2.x, inv)), q5 = __float2int_rn(__fmul_rn(f2.y, inv));
                int q6 = __float2int_rn(__fmul_rn(f3.x, inv)), q7 = __float2int_rn(__fmul_rn(f3.y, inv));
                q0 = max(-127, min(127, q0)); q1 = max(-127, min(127, q1));
                q2 = max(-127, min(127, q2)); q3 = max(-127, min(127, q3));
                q4 = max(-127, min(127, q4)); q5 = max(-127, min(127, q5));
                q6 = max(-127, min(127, q6)); q7 = max(-127, min(127, q7));
                uint2 o;
                o.x = (q0 & 255) | ((q1 & 255) << 8) | ((q2 & 255) << 16) | ((uint32_t)(q3 & 255) << 24);
                o.y = (q4 & 255) | ((q5 & 255) << 8) | ((q6 & 255) << 16) | ((uint32_t)(q7 & 255) << 24);
                st_stream(dst + i * 32 + lane, o);
                // group 2i + half_id: lane (2i + h) collects it for one coalesced scale store
                uint32_t sv = __shfl_sync(0xffffffffu, (uint32_t)__half_as_ushort(s16), (lane & 1) << 4);
                if ((lane >> 1) == i) my_scale = sv;
            }
            reinterpret_cast<uint16_t*>(pp.int8_scale + prow * (size_t)g.ng * 2)[lane] = (uint16_t)my_scale;
        } else {
            uint32_t* dst = reinterpret_cast<uint32_t*>(pp.int4_codes + prow * (size_t)(g.HD / 2));
            uint32_t my_sz = 0;
#pragma unroll 8
            for (int i = 0; i < iters; ++i) {
                uint4 v = ld_stream(src + i * 32 + lane);
                __half2 h0 = as_h2(v.x), h1 = as_h2(v.y), h2 = as_h2(v.z), h3 = as_h2(v.w);
                __half2 mx = __hmax2(__hmax2(h0, h1), __hmax2(h2, h3));
                __half2 mn = __hmin2(__hmin2(h0, h1), __hmin2(h2, h3));
#pragma unroll
                for (int o = 8; o; o >>= 1) {
                    mx = __hmax2(mx, as_h2(__shfl_xor_sync(0xffffffffu, as_u32(mx), o)));
                    mn = __hmin2(mn, as_h2(__shfl_xor_sync(0xffffffffu, as_u32(mn), o)));
                }
                float fmx = fmaxf(__low2float(mx), __high2float(mx));
                float fmn = fminf(__low2float(mn), __high2float(mn));
                __half z16 = __float2half_rn(fmn);                      // exact: fmn is an fp16 value
                if (fmn == 0.0f) z16 = __ushort_as_half(0);             // a zero minimum is stored as +0
                __half s16 = __float2half_rn(__fdiv_rn(__fsub_rn(fmx, fmn), 15.0f));
                if ((__half_as_ushort(s16) & 0x7fff) == 0) s16 = __ushort_as_half(0x3c00);
                float inv = __fdiv_rn(1.0f, __half2float(s16));
                float z = __half2float(z16);
                float2 f0 = __half22float2(h0), f1 = __half22float2(h1), f2 = __half22float2(h2), f3 = __half22float2(h3);
                float e[8] = {f0.x, f0.y, f1.x, f1.y, f2.x, f2.y, f3.x, f3.y};
                uint32_t o = 0;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    float r = rintf(__fmul_rn(__fsub_rn(e[k], z), inv));
                    r = fminf(fmaxf(r, 0.0f), 15.0f);
                    o |= (uint32_t)(int)r << (4 * k);
                }
                st_stream(dst + i * 32 + lane, o);
                uint32_t pair = (uint32_t)__half_as_ushort(s16) | ((uint32_t)__half_as_ushort(z16) << 16);
                uint32_t sv = __shfl_sync(0xffffffffu, pair, (lane & 1) << 4);
                if ((lane >> 1) == i) my_sz = sv;
            }
            reinterpret_cast<uint32_t*>(pp.int4_sz + prow * (size_t)g.ng * 4)[lane] = my_sz;
        }
    }
}

// ---- unpack -------------------------------------------------------------------------------------
__global__ void __launch_bounds__(KV_THREADS)
k_unpack(__half* __restrict__ K, __half* __restrict__ V, KvGeom g, const int32_t* __restrict__ idx,
         const int32_t* __restrict__ counts, const long long* __restrict__ row_offset, PoolPtrs pp,
         int* __restrict__ status) {
    extern __shared__ int pre[];
    build_prefix(counts, g.B, pre);
    const int planes = 2 * g.L;
    const long long n_units = (long long)pre[g.B] * planes;
    const int lane = threadIdx.x & 31;
    const long long warp0 = (long long)blockIdx.x * KV_WARPS + (threadIdx.x >> 5);
    const long long wstride = (long long)gridDim.x * KV_WARPS;
    const int iters = g.HD / 8 / 32;
    for (long long u = warp0; u < n_units; u += wstride) {
        Unit un = decode_unit(u, pre, g.B, planes, counts, idx, row_offset, g.n_tok, pp.cap, pp.ring);
        if (un.row < 0) {
            if (lane == 0) atomicMin(status, SALICACHE_E_CAPACITY);
            continue;
        }
        const int layer = un.plane >> 1, kv = un.plane & 1;
        __half* dst_h = (kv ? V : K) + (size_t)un.b * g.frame_stride + ((size_t)layer * g.n_tok + un.tok) * g.HD;
        uint4* dst = reinterpret_cast<uint4*>(dst_h);
        const size_t prow = (size_t)un.plane * pp.cap[un.tier] + un.row;
        if (un.tier == 0) {
            const uint4* src = reinterpret_cast<const uint4*>(pp.fp16_pool + prow * (size_t)g.HD * 2);
#pragma unroll 8
            for (int i = 0; i < iters; ++i) st_stream(dst + i * 32 + lane, ld_stream(src + i * 32 + lane));
        } else if (un.tier == 1) {
            const uint2* src = reinterpret_cast<const uint2*>(pp.int8_codes + prow * (size_t)g.HD);
            uint32_t my_scale = reinterpret_cast<const uint16_t*>(pp.int8_scale + prow * (size_t)g.ng * 2)[lane];
#pragma unroll 8
            for (int i = 0; i < iters; ++i) {
                uint2 c = __ldg(src + i * 32 + lane);
                float s = __half2float(__ushort_as_half((uint16_t)__shfl_sync(0xffffffffu, my_scale, 2 * i + (lane >> 4))));
                uint32_t w[2] = {c.x, c.y};
                uint32_t o[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    int qa = (int)(int8_t)((w[k >> 1] >> (16 * (k & 1))) & 255);
                    int qb = (int)(int8_t)((w[k >> 1] >> (16 * (k & 1) + 8)) & 255);
                    __half2 h = __floats2half2_rn(__fmul_rn((float)qa, s), __fmul_rn((float)qb, s));
                    o[k] = as_u32(h);
                }
                st_stream(dst + i * 32 + lane, make_uint4(o[0], o[1], o[2], o[3]));
            }
        } else {
            const uint32_t* src = reinterpret_cast<const uint32_t*>(pp.int4_codes + prow * (size_t)(g.HD / 2));
            uint32_t my_sz = reinterpret_cast<const uint32_t*>(pp.int4_sz + prow * (size_t)g.ng * 4)[lane];
#pragma unroll 8
            for (int i = 0; i < iters; ++i) {
                uint32_t c = __ldg(src + i * 32 + lane);
                uint32_t pair = __shfl_sync(0xffffffffu, my_sz, 2 * i + (lane >> 4));
                float s = __half2float(__ushort_as_half((uint16_t)(pair & 0xffff)));
                float z = __half2float(__ushort_as_half((uint16_t)(pair >> 16)));
                uint32_t o[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    float qa = (float)((c >> (8 * k)) & 15), qb = (float)((c >> (8 * k + 4)) & 15);
                    __half2 h = __floats2half2_rn(__fadd_rn(__fmul_rn(qa, s), z), __fadd_rn(__fmul_rn(qb, s), z));
                    o[k] = as_u32(h);
                }
                st_stream(dst + i * 32 + lane, make_uint4(o[0], o[1], o[2], o[3]));
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
    pp.cap[0] = p->cap_fp16;
    pp.cap[1] = p->cap_int8;
    pp.cap[2] = p->cap_int4;
    pp.ring = p->ring;
    return pp;
}

}  // namespace

int sc_kv_max_batch() { return MAX_PREFIX; }

int sc_pack(salicache_ctx* c, const void* d_K, const void* d_V, int64_t frame_stride, const int32_t* d_idx,
            const int32_t* d_counts, const int64_t* d_row_offset, int B, const salicache_pools* pools, cudaStream_t st) {
    if (B == 0) return SALICACHE_OK;
    KvGeom g{c->p.L, c->n_tok, c->p.heads * c->p.head_dim, c->p.heads * c->p.head_dim / 128, frame_stride, B};
    int grid = c->sm_count * 4;
    k_pack<<<grid, KV_THREADS, (size_t)(B + 1) * sizeof(int), st>>>((const __half*)d_K, (const __half*)d_V, g, d_idx,
                                                                    d_counts, (const long long*)d_row_offset,
                                                                    make_pools(pools), c->d_status);
    c->launches++;
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}

int sc_unpack(salicache_ctx* c, const salicache_pools* pools, const int32_t* d_idx, const int32_t* d_counts,
              const uint8_t* d_decision, const int64_t* d_row_offset, int B, int zero_fill_pruned, void* d_K_out,
              void* d_V_out, int64_t frame_stride, cudaStream_t st) {
    if (B == 0) return SALICACHE_OK;
    KvGeom g{c->p.L, c->n_tok, c->p.heads * c->p.head_dim, c->p.heads * c->p.head_dim / 128, frame_stride, B};
    int grid = c->sm_count * 4;
    k_unpack<<<grid, KV_THREADS, (size_t)(B + 1) * sizeof(int), st>>>((__half*)d_K_out, (__half*)d_V_out, g, d_idx,
                                                                      d_counts, (const long long*)d_row_offset,
                                                                      make_pools(pools), c->d_status);
    c->launches++;
    if (zero_fill_pruned) {
        dim3 gz(2 * g.L, B);
        k_zero_pruned<<<gz, KV_THREADS, 0, st>>>((__half*)d_K_out, (__half*)d_V_out, g, d_decision);
        c->launches++;
    }
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}
