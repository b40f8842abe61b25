// Decision rule (Eq. 6, Eq. 8, Alg. 1): per frame, the redundancy ratio, one code per token and the
// stable per-tier index lists; then the pool row offsets of the batch.
#include "common.cuh"

namespace {

constexpr int SEL_THREADS = 256;

__global__ void __launch_bounds__(SEL_THREADS)
k_select(const float* __restrict__ dP, const float* __restrict__ s, int n_tok, int first_has_no_prev, int patch_reuse,
         float tau_t, float theta_R, float tau_high, float tau_med, float tau_low, uint8_t* __restrict__ decision,
         int32_t* __restrict__ idx, int32_t* __restrict__ counts, uint8_t* __restrict__ frame_redundant) {
    __shared__ int s_red[SEL_THREADS / 32];
    __shared__ int s_static;
    __shared__ int s_warp[3][SEL_THREADS / 32];
    __shared__ int s_base[3];
    __shared__ int s_cnt[5];
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const bool has_prev = dP != nullptr && !(first_has_no_prev && b == 0);
    const float* dp = has_prev ? dP + (size_t)b * n_tok : nullptr;
    const float* sb = s + (size_t)b * n_tok;
    // Eq. 6: R = (1/N) sum [dP_i < tau_t]
    int n_static = 0;
    if (has_prev)
        for (int i = tid; i < n_tok; i += SEL_THREADS) n_static += (dp[i] < tau_t) ? 1 : 0;
#pragma unroll
    for (int o = 16; o; o >>= 1) n_static += __shfl_xor_sync(0xffffffffu, n_static, o);
    if (lane == 0) s_red[wid] = n_static;
    if (tid < 3) s_base[tid] = 0;
    if (tid < 5) s_cnt[tid] = 0;
    __syncthreads();
    if (tid == 0) {
        int t = 0;
        for (int k = 0; k < SEL_THREADS / 32; ++k) t += s_red[k];
        s_static = t;
    }
    __syncthreads();
    const float R = has_prev ? __fdiv_rn((float)s_static, (float)n_tok) : 0.0f;
    const bool redundant = has_prev && (R > theta_R);
    int my_cnt[5] = {0, 0, 0, 0, 0};
    for (int base = 0; base < n_tok; base += SEL_THREADS) {
        int i = base + tid;
        int d = -1;
        if (i < n_tok) {
            if (redundant) d = SALICACHE_REUSE;
            else if (patch_reuse && has_prev && dp[i] < tau_t) d = SALICACHE_REUSE;
            else {
                float sv = sb[i];
                d = sv > tau_high ? SALICACHE_FP16 : (sv > tau_med ? SALICACHE_INT8 : (sv > tau_low ? SALICACHE_INT4 : SALICACHE_PRUNE));
            }
            decision[(size_t)b * n_tok + i] = (uint8_t)d;
        }
        unsigned m[3];
        m[0] = __ballot_sync(0xffffffffu, d == SALICACHE_FP16);
        m[1] = __ballot_sync(0xffffffffu, d == SALICACHE_INT8);
        m[2] = __ballot_sync(0xffffffffu, d == SALICACHE_INT4);
        if (lane == 0) {
#pragma unroll
            for (int t = 0; t < 3; ++t) s_warp[t][wid] = __popc(m[t]);
        }
        __syncthreads();
        int tier = d == SALICACHE_FP16 ? 0 : (d == SALICACHE_INT8 ? 1 : (d == SALICACHE_INT4 ? 2 : -1));
        if (tier >= 0) {
            int pos = s_base[tier];
            for (int k = 0; k < wid; ++k) pos += s_warp[tier][k];
            pos += __popc(m[tier] & ((1u << lane) - 1u));
            idx[((size_t)b * 3 + tier) * n_tok + pos] = i;
        }
        if (d >= 0) my_cnt[d]++;
        __syncthreads();
        if (tid < 3) {
            int t = 0;
            for (int k = 0; k < SEL_THREADS / 32; ++k) t += s_warp[tid][k];
            s_base[tid] += t;
        }
        __syncthreads();
    }
#pragma unroll
    for (int c = 0; c < 5; ++c) {
        int v = my_cnt[c];
#pragma unroll
        for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0 && v) atomicAdd(&s_cnt[c], v);
    }
    __syncthreads();
    if (tid < 5) counts[(size_t)b * 5 + tid] = s_cnt[tid];
    if (tid == 0) frame_redundant[b] = redundant ? 1 : 0;
    // pad the lists with -1
    for (int t = 0; t < 3; ++t)
        for (int i = s_base[t] + tid; i < n_tok; i += SEL_THREADS) idx[((size_t)b * 3 + t) * n_tok + i] = -1;
}

// Eq. 6 alone: R = (1/N) sum [dP_i < tau_t], redundant when the frame has a predecessor and R > theta_R.
// The same arithmetic as k_select, so that both agree on every frame.
__global__ void __launch_bounds__(SEL_THREADS)
k_frame_redundancy(const float* __restrict__ dP, int n_tok, int first_has_no_prev, float tau_t, float theta_R,
                   uint8_t* __restrict__ frame_redundant) {
    __shared__ int s_red[SEL_THREADS / 32];
    const int b = blockIdx.x, tid = threadIdx.x;
    const bool has_prev = dP != nullptr && !(first_has_no_prev && b == 0);
    int n_static = 0;
    if (has_prev)
        for (int i = tid; i < n_tok; i += SEL_THREADS) n_static += (dP[(size_t)b * n_tok + i] < tau_t) ? 1 : 0;
#pragma unroll
    for (int o = 16; o; o >>= 1) n_static += __shfl_xor_sync(0xffffffffu, n_static, o);
    if ((tid & 31) == 0) s_red[tid >> 5] = n_static;
    __syncthreads();
    if (tid == 0) {
        int t = 0;
        for (int k = 0; k < SEL_THREADS / 32; ++k) t += s_red[k];
        const float R = has_prev ? __fdiv_rn((float)t, (float)n_tok) : 0.0f;
        frame_redundant[b] = (has_prev && R > theta_R) ? 1 : 0;
    }
}

// Source-frame table (Alg. 1 line 7, C[t] <- Pointer(C[t-1]), extended to patches): one thread per token
// walks the batch in frame order; a REUSE token inherits its predecessor's source, any other token is its
// own source.  `carry` holds the sources of the frame before the batch and receives those of its last frame.
__global__ void k_sources(const uint8_t* __restrict__ decision, int n_tok, int B, int first_frame, int32_t* __restrict__ carry,
                          int32_t* __restrict__ src) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_tok) return;
    int cur = carry[i];
    for (int b = 0; b < B; ++b) {
        if (decision[(size_t)b * n_tok + i] != SALICACHE_REUSE) cur = first_frame + b;
        src[(size_t)b * n_tok + i] = cur;
    }
    carry[i] = cur;
}

// Pool row offsets: exclusive scan over the frames of the batch, continuing from the running fill.  One CTA:
// a frame per thread, its three tier counts scanned together (warp scans, then the warps' totals), 1024 frames per
// sweep.  Sums within a sweep stay in 32 bits (a frame has fewer than 2^13 tokens: the edge planes of a frame must
// fit shared memory, which bounds its pixels); the running fill is 64-bit.
constexpr int OFF_THREADS = 1024;
__global__ void __launch_bounds__(OFF_THREADS)
k_row_offsets(const int32_t* __restrict__ counts, int B, int64_t* __restrict__ row_offset, int64_t* __restrict__ fill) {
    __shared__ int wtot[OFF_THREADS / 32][3];
    const int t = threadIdx.x, lane = t & 31, wp = t >> 5;
    const int code[3] = {SALICACHE_FP16, SALICACHE_INT8, SALICACHE_INT4};
    int64_t carry[3] = {fill[0], fill[1], fill[2]};
    for (int base = 0; base < B; base += OFF_THREADS) {
        const int b = base + t;
        int v[3] = {0, 0, 0}, incl[3];
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            if (b < B) v[k] = counts[(size_t)b * 5 + code[k]];
            incl[k] = v[k];
        }
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
            for (int k = 0; k < 3; ++k) {
                const int up = __shfl_up_sync(0xffffffffu, incl[k], o);
                if (lane >= o) incl[k] += up;
            }
        }
        if (lane == 31) { wtot[wp][0] = incl[0]; wtot[wp][1] = incl[1]; wtot[wp][2] = incl[2]; }
        __syncthreads();
        int below[3] = {0, 0, 0}, total[3] = {0, 0, 0};
        for (int w = 0; w < OFF_THREADS / 32; ++w) {
#pragma unroll
            for (int k = 0; k < 3; ++k) {
                const int x = wtot[w][k];
                if (w < wp) below[k] += x;
                total[k] += x;
            }
        }
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            if (b < B) row_offset[(size_t)b * 3 + k] = carry[k] + (int64_t)(below[k] + incl[k] - v[k]);
            carry[k] += total[k];
        }
        __syncthreads();
    }
    if (t < 3) fill[t] = carry[t];
}

// Residency of stored frames in budgeted pools: one thread per frame.
__global__ void k_frames_resident(const int32_t* __restrict__ counts, const int64_t* __restrict__ row_offset, int B,
                                  long long cap0, long long cap1, long long cap2, int ring, const int64_t* __restrict__ fill,
                                  uint8_t* __restrict__ resident) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int code[3] = {SALICACHE_FP16, SALICACHE_INT8, SALICACHE_INT4};
    const long long cap[3] = {cap0, cap1, cap2};
    bool ok = true;
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        const long long n = counts[(size_t)b * 5 + code[k]], o = row_offset[(size_t)b * 3 + k];
        if (n == 0) continue;
        if (ring) ok = ok && n <= cap[k] && o >= fill[k] - cap[k];
        else ok = ok && o + n <= cap[k];
    }
    resident[b] = ok ? 1 : 0;
}

__global__ void k_tokens_live(const int32_t* __restrict__ src, long long n, int first, const uint8_t* __restrict__ table,
                              int n_table, uint8_t* __restrict__ live) {
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (i >= n) return;
    const long long k = (long long)src[i] - first;
    live[i] = (k >= 0 && k < n_table) ? table[k] : 0;
}

}  // namespace

int sc_frames_resident(salicache_ctx* c, const int32_t* d_counts, const int64_t* d_row_offset, int B,
                       const salicache_pools* pools, uint8_t* d_resident, cudaStream_t st) {
    if (B == 0) return SALICACHE_OK;
    k_frames_resident<<<(B + 127) / 128, 128, 0, st>>>(d_counts, d_row_offset, B, pools->cap_fp16, pools->cap_int8,
                                                       pools->cap_int4, pools->ring, pools->d_fill, d_resident);
    c->launches++;
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}

int sc_tokens_live(salicache_ctx* c, const int32_t* d_src, int B, int first_frame, const uint8_t* d_table, int n_table,
                   uint8_t* d_live, cudaStream_t st) {
    const long long n = (long long)B * c->n_tok;
    if (n == 0) return SALICACHE_OK;
    k_tokens_live<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(d_src, n, first_frame, d_table, n_table, d_live);
    c->launches++;
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}

int sc_frame_redundancy(salicache_ctx* c, const float* d_deltaP, int B, int first_has_no_prev, uint8_t* d_frame_redundant,
                        cudaStream_t st) {
    if (B == 0) return SALICACHE_OK;
    k_frame_redundancy<<<B, SEL_THREADS, 0, st>>>(d_deltaP, c->n_tok, first_has_no_prev, c->p.tau_t, c->p.theta_R,
                                                  d_frame_redundant);
    c->launches++;
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}

int sc_sources(salicache_ctx* c, const uint8_t* d_decision, int B, int first_frame, int32_t* d_carry, int32_t* d_src,
               cudaStream_t st) {
    if (B == 0) return SALICACHE_OK;
    k_sources<<<(c->n_tok + 255) / 256, 256, 0, st>>>(d_decision, c->n_tok, B, first_frame, d_carry, d_src);
    c->launches++;
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}

int sc_select(salicache_ctx* c, const float* d_deltaP, const float* d_s, int B, int first_has_no_prev,
              uint8_t* d_decision, int32_t* d_idx, int32_t* d_counts, uint8_t* d_frame_redundant,
              int64_t* d_row_offset, int64_t* d_fill, cudaStream_t st) {
    const salicache_params& p = c->p;
    if (B == 0) return SALICACHE_OK;
    k_select<<<B, SEL_THREADS, 0, st>>>(d_deltaP, d_s, c->n_tok, first_has_no_prev, p.patch_reuse, p.tau_t, p.theta_R,
                                        p.tau_high, p.tau_med, p.tau_low, d_decision, d_idx, d_counts,
                                        d_frame_redundant);
    k_row_offsets<<<1, OFF_THREADS, 0, st>>>(d_counts, B, d_row_offset, d_fill);
    c->launches += 2;
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}
