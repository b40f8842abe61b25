// Adaptive tier thresholds (a variant: the paper's thresholds are fixed; it names their adaptation to the content as
// future work, Sec. V).  The temporal test is k_select's (Eq. 6 and patch reuse).  Among the tokens of a frame that are
// not reused, the tiers of Eq. 8 are given out by rank of s_i, in fixed shares: with n_live such tokens,
//   q16 = (n_live * pm16 + 500) / 1000, likewise q8 and q4, each clipped to what is left of n_live;
// the q16 most salient are FP16, the next q8 INT8, the next q4 INT4, the rest pruned; ties go to the lower token id.
// Eq. 8's thresholds thus become order statistics of the frame's own scores.
//
// One CTA per frame.  A token's rank is counted directly (how many live tokens come before it): n_tok^2 comparisons
// per frame out of shared memory, 0.3 M for 576 tokens, which is less work than a sort's bookkeeping at this size.
#include "common.cuh"

namespace {

constexpr int RK_THREADS = 256;

__global__ void __launch_bounds__(RK_THREADS)
k_select_ranked(const float* __restrict__ dP, const float* __restrict__ s, int n_tok, int first_has_no_prev, int patch_reuse,
                float tau_t, float theta_R, int pm16, int pm8, int pm4, uint8_t* __restrict__ decision,
                int32_t* __restrict__ idx, int32_t* __restrict__ counts, uint8_t* __restrict__ frame_redundant) {
    extern __shared__ float ss[];                   // [n_tok] scores; then [n_tok] bytes: 1 = live, later the decision
    uint8_t* flag = reinterpret_cast<uint8_t*>(ss + n_tok);
    __shared__ int s_red[RK_THREADS / 32];
    __shared__ int s_tot[2];                        // static patches, live tokens
    __shared__ int s_warp[3][RK_THREADS / 32];
    __shared__ int s_base[3];
    __shared__ int s_cnt[5];
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const bool has_prev = dP != nullptr && !(first_has_no_prev && b == 0);
    const float* dp = has_prev ? dP + (size_t)b * n_tok : nullptr;
    const float* sb = s + (size_t)b * n_tok;
    // Eq. 6: R = (1/N) sum [dP_i < tau_t]
    int n_static = 0;
    if (has_prev)
        for (int i = tid; i < n_tok; i += RK_THREADS) n_static += (dp[i] < tau_t) ? 1 : 0;
#pragma unroll
    for (int o = 16; o; o >>= 1) n_static += __shfl_xor_sync(0xffffffffu, n_static, o);
    if (lane == 0) s_red[wid] = n_static;
    if (tid < 3) s_base[tid] = 0;
    if (tid < 5) s_cnt[tid] = 0;
    __syncthreads();
    if (tid == 0) {
        int t = 0;
        for (int k = 0; k < RK_THREADS / 32; ++k) t += s_red[k];
        s_tot[0] = t;
    }
    __syncthreads();
    const float R = has_prev ? __fdiv_rn((float)s_tot[0], (float)n_tok) : 0.0f;
    const bool redundant = has_prev && (R > theta_R);
    // the tokens that are not reused
    int n_live = 0;
    for (int i = tid; i < n_tok; i += RK_THREADS) {
        const bool live = !redundant && !(patch_reuse && has_prev && dp[i] < tau_t);
        ss[i] = sb[i];
        flag[i] = live ? 1 : 0;
        n_live += live ? 1 : 0;
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) n_live += __shfl_xor_sync(0xffffffffu, n_live, o);
    __syncthreads();                                // s_red has been read
    if (lane == 0) s_red[wid] = n_live;
    __syncthreads();
    if (tid == 0) {
        int t = 0;
        for (int k = 0; k < RK_THREADS / 32; ++k) t += s_red[k];
        s_tot[1] = t;
    }
    __syncthreads();
    n_live = s_tot[1];
    long long left = n_live;
    long long q16 = ((long long)n_live * pm16 + 500) / 1000; if (q16 > left) q16 = left; left -= q16;
    long long q8 = ((long long)n_live * pm8 + 500) / 1000;   if (q8 > left) q8 = left;   left -= q8;
    long long q4 = ((long long)n_live * pm4 + 500) / 1000;   if (q4 > left) q4 = left;
    // ranks -> codes (kept in registers until every thread has finished reading the flags)
    constexpr int PER = 12;                         // tokens per thread: n_tok <= 12 * 256
    uint8_t code[PER];
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        const int i = tid + k * RK_THREADS;
        code[k] = 255;
        if (i < n_tok) {
            if (!flag[i]) code[k] = SALICACHE_REUSE;
            else {
                const float si = ss[i];
                int rank = 0;
                for (int j = 0; j < n_tok; ++j) {
                    const float sj = ss[j];
                    rank += (flag[j] && (sj > si || (sj == si && j < i))) ? 1 : 0;
                }
                code[k] = rank < q16 ? SALICACHE_FP16 : (rank < q16 + q8 ? SALICACHE_INT8 : (rank < q16 + q8 + q4 ? SALICACHE_INT4 : SALICACHE_PRUNE));
            }
        }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        const int i = tid + k * RK_THREADS;
        if (i < n_tok) flag[i] = code[k];
    }
    __syncthreads();
    // decisions, stable per-tier lists, counts (as k_select)
    int my_cnt[5] = {0, 0, 0, 0, 0};
    for (int base = 0; base < n_tok; base += RK_THREADS) {
        const int i = base + tid;
        int d = -1;
        if (i < n_tok) {
            d = flag[i];
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
        const int tier = d == SALICACHE_FP16 ? 0 : (d == SALICACHE_INT8 ? 1 : (d == SALICACHE_INT4 ? 2 : -1));
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
            for (int k = 0; k < RK_THREADS / 32; ++k) t += s_warp[tid][k];
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
    for (int t = 0; t < 3; ++t)
        for (int i = s_base[t] + tid; i < n_tok; i += RK_THREADS) idx[((size_t)b * 3 + t) * n_tok + i] = -1;
}

// Pool row offsets: exclusive scan over the frames of the batch, continuing from the running fill.
__global__ void k_ranked_row_offsets(const int32_t* __restrict__ counts, int B, int64_t* __restrict__ row_offset,
                                     int64_t* __restrict__ fill) {
    const int t = threadIdx.x;
    if (t >= 3) return;
    const int code = t == 0 ? SALICACHE_FP16 : (t == 1 ? SALICACHE_INT8 : SALICACHE_INT4);
    int64_t acc = fill[t];
    for (int b = 0; b < B; ++b) {
        row_offset[(size_t)b * 3 + t] = acc;
        acc += counts[(size_t)b * 5 + code];
    }
    fill[t] = acc;
}

}  // namespace

int sc_select_ranked(salicache_ctx* c, const float* d_deltaP, const float* d_s, int B, int first_has_no_prev, int pm16,
                     int pm8, int pm4, uint8_t* d_decision, int32_t* d_idx, int32_t* d_counts, uint8_t* d_frame_redundant,
                     int64_t* d_row_offset, int64_t* d_fill, cudaStream_t st) {
    const salicache_params& p = c->p;
    if (c->n_tok > 12 * RK_THREADS) return SALICACHE_E_PARAM;
    if (B == 0) return SALICACHE_OK;
    const size_t smem = (size_t)c->n_tok * (sizeof(float) + 1);
    k_select_ranked<<<B, RK_THREADS, smem, st>>>(d_deltaP, d_s, c->n_tok, first_has_no_prev, p.patch_reuse, p.tau_t, p.theta_R,
                                                 pm16, pm8, pm4, d_decision, d_idx, d_counts, d_frame_redundant);
    k_ranked_row_offsets<<<1, 32, 0, st>>>(d_counts, B, d_row_offset, d_fill);
    c->launches += 2;
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}
