// Anchor-frame mode of the temporal test (a variant: the paper compares consecutive frames, Sec. III-A, so a
// slow pan or fade whose every step stays below tau_t is "static" forever).  Here token i of frame t is
// compared with the patch its cache entry was computed from: the patch of the last frame in which token i was
// not REUSE, i.e. the frame Alg. 1's pointer chain resolves to.  The `anchor` image is that composite.  Per frame:
//
//   dP[t][i]  = Eq. 5 read literally between anchor and frame t (RMS grey-level difference over patch i)
//   decisions = Eq. 6 / Eq. 8 on (dP[t], s[t]), the arithmetic of k_select
//   anchor   <- frame t on every patch whose token is not REUSE
//
// Frame t needs the decisions of frame t-1: a scan over the frames, not a map.  To keep the scan's step short
// the frame is spread over a thread-block cluster of 8 CTAs that own contiguous bands of patch rows (so their
// tokens are contiguous in token order); what a step has to share, the number of static patches (Eq. 6) and
// the per-tier counts that place each CTA's tokens in the index lists, crosses the cluster through distributed
// shared memory, one cluster barrier per frame.  A CTA reads and writes only its own bands of the anchor image,
// so the image needs no synchronisation beyond the CTA's own barrier.  Several videos are several clusters of one
// launch; they share nothing.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int AN_CLUSTER = 8;       // CTAs per video
constexpr int AN_THREADS = 1024;    // a step is a few dependent memory round trips: every thread gets two or three chunks
constexpr int AN_WARPS = AN_THREADS / 32;
constexpr int AN_MAX_OWN = 288;     // tokens one CTA may own: ceil(48 / 8) bands of up to 48 patches
constexpr int AN_XCH = 6;           // shared per frame and CTA: static patches, then counts of REUSE PRUNE INT4 INT8 FP16

struct AnchorArgs {
    const uint8_t* frames;   // [B][H][W][3]
    const float* s;          // [B][n_tok]
    uint8_t* anchor;         // [H][W][3], read and written
    float* dP;               // [B][n_tok]
    uint8_t* decision;       // [B][n_tok]
    int32_t* idx;            // [B][3][n_tok]
    int32_t* counts;         // [B][5]
    uint8_t* redundant;      // [B]
    int64_t* row_offset;     // [B][3]
    int64_t* fill;           // [3]
    int B, H, W, gh, gw, first_has_no_prev, patch_reuse;
    float tau_t, theta_R, tau_high, tau_med, tau_low;
};

// Byte mask of the first n bytes of word w4 of a 16-byte chunk (n counted from the chunk's start).
__device__ __forceinline__ uint32_t head_mask(int n, int w4) {
    const int k = n - 4 * w4;
    return k >= 4 ? 0xffffffffu : (k <= 0 ? 0u : ((1u << (8 * k)) - 1u));
}

static_assert(AN_MAX_OWN <= AN_THREADS, "one owned token per thread");

__global__ void __cluster_dims__(AN_CLUSTER, 1, 1) __launch_bounds__(AN_THREADS)
k_select_anchored(AnchorArgs a) {
    cg::cluster_group cluster = cg::this_cluster();
    __shared__ unsigned int acc[2][AN_MAX_OWN];     // squared differences per owned patch; the other half is cleared meanwhile
    __shared__ uint8_t dec_l[AN_MAX_OWN];           // this frame's decisions of the owned tokens
    __shared__ int xch[2][AN_CLUSTER][AN_XCH];      // by frame parity and source CTA; written by every CTA of the cluster
    __shared__ int s_cnt[2][AN_XCH];
    __shared__ int s_warp[3][AN_WARPS];
    const int rank = (int)cluster.block_rank(), tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int n_tok = a.gh * a.gw;
    {   // one cluster per video: every array has a leading video dimension
        const size_t vid = blockIdx.x / AN_CLUSTER, vb = vid * (size_t)a.B;
        const size_t frame = (size_t)a.H * a.W * 3;
        a.frames += vb * frame;
        a.s += vb * n_tok;
        a.anchor += vid * frame;
        a.dP += vb * n_tok;
        a.decision += vb * n_tok;
        a.idx += vb * 3 * n_tok;
        a.counts += vb * 5;
        a.redundant += vb;
        a.row_offset += vb * 3;
        a.fill += vid * 3;
    }
    const int nb = (a.gh + AN_CLUSTER - 1) / AN_CLUSTER;                // bands per CTA
    const int band0 = min(a.gh, rank * nb), band1 = min(a.gh, band0 + nb);
    const int tok0 = band0 * a.gw, n_own = (band1 - band0) * a.gw;
    const int row_bytes = a.W * 3, chunks = row_bytes / 16;             // W is a multiple of 16
    const int rows = (band1 - band0) * 14;
    const size_t fb = (size_t)a.H * row_bytes;
    const bool owner = tid < n_own;                                     // thread tid owns token tok0 + tid
    uint8_t* anc = a.anchor + (size_t)band0 * 14 * row_bytes;           // plain loads and stores: this CTA rewrites it
    // the index lists start as all -1; the frames' steps then write the entries that exist
    for (size_t i = (size_t)rank * AN_THREADS + tid; i < (size_t)a.B * 3 * n_tok; i += (size_t)AN_CLUSTER * AN_THREADS) a.idx[i] = -1;
    if (owner) acc[0][tid] = 0;
    if (tid < AN_XCH) s_cnt[0][tid] = 0;
    cluster.sync();                                 // orders the fill before any CTA's entries, and the shared arrays
    for (int t = 0; t < a.B; ++t) {
        const bool has_prev = !(a.first_has_no_prev && t == 0);
        const uint8_t* fr = a.frames + (size_t)t * fb + (size_t)band0 * 14 * row_bytes;
        const int par = t & 1;
        // pull the next frame's bands into the L2 while this one is worked on; fetch this token's spatial score early
        if (t + 1 < a.B)
            for (int i = tid; i < (rows * row_bytes + 127) / 128; i += AN_THREADS)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(fr + fb + (size_t)i * 128));
        const float sv = owner ? __ldg(a.s + (size_t)t * n_tok + tok0 + tid) : 0.0f;
        // ---- Eq. 5 read literally, against the anchor: exact integer sums per patch
        if (has_prev)
            for (int i = tid; i < rows * chunks; i += AN_THREADS) {
                const int r = i / chunks, k = i - r * chunks;
                const uint4 va = *(reinterpret_cast<const uint4*>(anc + (size_t)r * row_bytes) + k);
                const uint4 vb = __ldg(reinterpret_cast<const uint4*>(fr + (size_t)r * row_bytes) + k);
                const int b0 = 16 * k, p0 = b0 / 42;
                const int m = 42 * (p0 + 1) - b0;                       // bytes of this chunk that belong to patch p0 (>= 1)
                const uint32_t wa[4] = {va.x, va.y, va.z, va.w}, wb[4] = {vb.x, vb.y, vb.z, vb.w};
                unsigned int lo = 0, hi = 0;
#pragma unroll
                for (int w4 = 0; w4 < 4; ++w4) {
                    const uint32_t d = __vabsdiffu4(wa[w4], wb[w4]);
                    const uint32_t mask = head_mask(m, w4);
                    const uint32_t dl = d & mask, dh = d & ~mask;
                    lo = __dp4a(dl, dl, lo);
                    hi = __dp4a(dh, dh, hi);
                }
                const int pl = (r / 14) * a.gw + p0;
                atomicAdd(&acc[par][pl], lo);
                if (hi) atomicAdd(&acc[par][pl + 1], hi);
            }
        __syncthreads();
        // ---- the score, the code the token would get in a frame that is not redundant, the CTA's counts
        int code = -1;
        bool is_static = false;
        if (owner) {
            const float d = has_prev ? (float)sqrt((double)acc[par][tid] / (double)(3 * 14 * 14)) : 0.0f;
            a.dP[(size_t)t * n_tok + tok0 + tid] = d;
            is_static = has_prev && d < a.tau_t;
            if (a.patch_reuse && is_static) code = SALICACHE_REUSE;
            else code = sv > a.tau_high ? SALICACHE_FP16 : (sv > a.tau_med ? SALICACHE_INT8 : (sv > a.tau_low ? SALICACHE_INT4 : SALICACHE_PRUNE));
            acc[par ^ 1][tid] = 0;                                      // for the next frame
        }
        if (tid < AN_XCH) s_cnt[par ^ 1][tid] = 0;
        unsigned m3[3];                                                 // lanes of this warp with an FP16, INT8, INT4 code
        {
            const unsigned ms = __ballot_sync(0xffffffffu, is_static);
            const unsigned m0 = __ballot_sync(0xffffffffu, code == SALICACHE_REUSE);
            const unsigned m1 = __ballot_sync(0xffffffffu, code == SALICACHE_PRUNE);
            m3[2] = __ballot_sync(0xffffffffu, code == SALICACHE_INT4);
            m3[1] = __ballot_sync(0xffffffffu, code == SALICACHE_INT8);
            m3[0] = __ballot_sync(0xffffffffu, code == SALICACHE_FP16);
            if (lane == 0) {
                s_warp[0][wid] = __popc(m3[0]);
                s_warp[1][wid] = __popc(m3[1]);
                s_warp[2][wid] = __popc(m3[2]);
                if (ms) atomicAdd(&s_cnt[par][0], __popc(ms));
                if (m0) atomicAdd(&s_cnt[par][1 + SALICACHE_REUSE], __popc(m0));
                if (m1) atomicAdd(&s_cnt[par][1 + SALICACHE_PRUNE], __popc(m1));
                if (m3[2]) atomicAdd(&s_cnt[par][1 + SALICACHE_INT4], __popc(m3[2]));
                if (m3[1]) atomicAdd(&s_cnt[par][1 + SALICACHE_INT8], __popc(m3[1]));
                if (m3[0]) atomicAdd(&s_cnt[par][1 + SALICACHE_FP16], __popc(m3[0]));
            }
        }
        __syncthreads();
        // ---- every CTA of the cluster receives this CTA's six numbers
        if (tid < AN_CLUSTER * AN_XCH) {
            const int dst = tid / AN_XCH, c = tid - dst * AN_XCH;
            int* remote = cluster.map_shared_rank(&xch[par][rank][c], dst);
            *remote = s_cnt[par][c];
        }
        cluster.sync();
        int n_static = 0, before[3] = {0, 0, 0}, total[5] = {0, 0, 0, 0, 0};
        for (int r = 0; r < AN_CLUSTER; ++r) {
            n_static += xch[par][r][0];
#pragma unroll
            for (int c = 0; c < 5; ++c) total[c] += xch[par][r][1 + c];
            if (r < rank) {
                before[0] += xch[par][r][1 + SALICACHE_FP16];
                before[1] += xch[par][r][1 + SALICACHE_INT8];
                before[2] += xch[par][r][1 + SALICACHE_INT4];
            }
        }
        // Eq. 6, as k_select computes it
        const float R = has_prev ? __fdiv_rn((float)n_static, (float)n_tok) : 0.0f;
        const bool redundant = has_prev && (R > a.theta_R);
        // ---- decisions and the stable per-tier index lists (FP16, INT8, INT4) of the owned tokens
        if (owner) {
            const int d = redundant ? SALICACHE_REUSE : code;
            dec_l[tid] = (uint8_t)d;
            a.decision[(size_t)t * n_tok + tok0 + tid] = (uint8_t)d;
            const int tier = d == SALICACHE_FP16 ? 0 : (d == SALICACHE_INT8 ? 1 : (d == SALICACHE_INT4 ? 2 : -1));
            if (tier >= 0) {
                int pos = before[tier];
                for (int k = 0; k < wid; ++k) pos += s_warp[tier][k];
                pos += __popc(m3[tier] & ((1u << lane) - 1u));
                a.idx[((size_t)t * 3 + tier) * n_tok + pos] = tok0 + tid;
            }
        }
        if (rank == 0) {
            if (tid < 5) a.counts[(size_t)t * 5 + tid] = redundant ? (tid == SALICACHE_REUSE ? n_tok : 0) : total[tid];
            if (tid == 0) a.redundant[t] = redundant ? 1 : 0;
        }
        __syncthreads();
        // ---- the anchor takes the pixels of every owned patch whose token is not REUSE
        if (!redundant)
            for (int i = tid; i < rows * chunks; i += AN_THREADS) {
                const int r = i / chunks, k = i - r * chunks;
                const int b0 = 16 * k, p0 = b0 / 42;
                const int m = 42 * (p0 + 1) - b0;
                const int pl = (r / 14) * a.gw + p0;
                const bool st0 = dec_l[pl] != SALICACHE_REUSE;
                const bool st1 = m >= 16 ? st0 : dec_l[pl + 1] != SALICACHE_REUSE;
                if (!st0 && !st1) continue;
                uint4* dst = reinterpret_cast<uint4*>(anc + (size_t)r * row_bytes) + k;
                const uint4 vf = __ldg(reinterpret_cast<const uint4*>(fr + (size_t)r * row_bytes) + k);
                if (st0 && st1) {
                    *dst = vf;
                } else {
                    const uint4 va = *dst;
                    const uint32_t wf[4] = {vf.x, vf.y, vf.z, vf.w}, wa[4] = {va.x, va.y, va.z, va.w};
                    uint32_t o[4];
#pragma unroll
                    for (int w4 = 0; w4 < 4; ++w4) {
                        const uint32_t head = head_mask(m, w4);                 // bytes of patch p0
                        const uint32_t take = st0 ? head : ~head;               // bytes that come from the frame
                        o[w4] = (wf[w4] & take) | (wa[w4] & ~take);
                    }
                    *dst = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
        __syncthreads();                            // the next frame reads the anchor and reuses the shared arrays
    }
    // ---- pool row offsets: exclusive scan over the frames, continuing from the running fill (as k_row_offsets)
    if (rank == 0 && tid < 3) {
        const int code = tid == 0 ? SALICACHE_FP16 : (tid == 1 ? SALICACHE_INT8 : SALICACHE_INT4);
        int64_t run = a.fill[tid];
        for (int t = 0; t < a.B; ++t) {
            a.row_offset[(size_t)t * 3 + tid] = run;
            run += a.counts[(size_t)t * 5 + code];
        }
        a.fill[tid] = run;
    }
    cluster.sync();                                 // no CTA leaves while another may still write into its shared memory
}

}  // namespace

int sc_select_anchored(salicache_ctx* c, const uint8_t* d_frames, const float* d_s, int n_videos, int B, int first_has_no_prev,
                       uint8_t* d_anchor, float* d_deltaP, uint8_t* d_decision, int32_t* d_idx, int32_t* d_counts,
                       uint8_t* d_frame_redundant, int64_t* d_row_offset, int64_t* d_fill, cudaStream_t st) {
    const salicache_params& p = c->p;
    const PlaneGeom& g = c->plane[0];
    if (c->n_planes != 1 || g.layout != 0 || p.patch != 14 || g.gh > 48 || g.gw > 48) return SALICACHE_E_PARAM;
    if (B == 0 || n_videos == 0) return SALICACHE_OK;
    AnchorArgs a{d_frames, d_s, d_anchor, d_deltaP, d_decision, d_idx, d_counts, d_frame_redundant, d_row_offset, d_fill,
                 B, g.H, g.W, g.gh, g.gw, first_has_no_prev, p.patch_reuse, p.tau_t, p.theta_R, p.tau_high, p.tau_med, p.tau_low};
    k_select_anchored<<<AN_CLUSTER * n_videos, AN_THREADS, 0, st>>>(a);
    c->launches++;
    SC_CHECK(cudaGetLastError());
    return SALICACHE_OK;
}
