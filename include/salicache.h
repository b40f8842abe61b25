/*
 * salicache.h -- C ABI of the B200 (sm_100a) Sali-Cache pre-attention filter and
 * mixed-precision K/V store.
 *
 * The hot path every video frame takes before its visual tokens reach attention
 * (paper Sec. III, Alg. 1):
 *     flow_score  ->  saliency  ->  select  ->  pack_kv        (+ unpack_kv)
 *
 * Conventions
 *   - Pointers named d_* are DEVICE pointers owned by the caller; h_* are HOST
 *     pointers.  The library never frees or reallocates caller memory.
 *   - A context owns only its scratch memory, sized at salicache_create.  No hot
 *     call allocates.
 *   - Every hot call is asynchronous on `cuda_stream` (a cudaStream_t passed as
 *     void*; NULL = the default stream) and does not synchronise the host.
 *   - Return value: 0 on success, a negative SALICACHE_E_* code otherwise.  No
 *     exceptions, no abort, no device trap.  Conditions only the device can see
 *     (pool overflow, hysteresis iteration cap) are recorded in a device status
 *     word and returned by salicache_poll_status.
 *   - Frames are uint8 HWC (R,G,B), 16-byte aligned, W a multiple of 16.
 *   - K/V are IEEE binary16, finite; NaN/Inf inputs give unspecified codes.
 *   - One context is used by one host thread at a time; contexts are independent.
 */
#ifndef SALICACHE_H
#define SALICACHE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define SALICACHE_API __attribute__((visibility("default")))
#else
#define SALICACHE_API
#endif

#define SALICACHE_OK            0
#define SALICACHE_E_NULL       -1   /* a required pointer is NULL                          */
#define SALICACHE_E_SHAPE      -2   /* sizes inconsistent with the context                 */
#define SALICACHE_E_ALIGN      -3   /* a pointer is not 16-byte aligned                    */
#define SALICACHE_E_PARAM      -4   /* unsupported parameter value                         */
#define SALICACHE_E_CUDA       -5   /* a CUDA runtime call failed                          */
#define SALICACHE_E_CAPACITY   -6   /* a tier pool is too small (rows dropped, ring == 0)  */
#define SALICACHE_E_NOCONVERGE -7   /* edge hysteresis hit hyst_max_iters                  */
#define SALICACHE_E_NOMEM      -8   /* scratch allocation failed at create                 */
#define SALICACHE_E_EVICTED    -9   /* rows asked for have been overwritten in a ring pool */

/* Decision code per token (Fig. 3 categories; Eq. 8 tiers). */
#define SALICACHE_REUSE 0   /* "skipped": K/V of the previous frame's token is reused       */
#define SALICACHE_PRUNE 1
#define SALICACHE_INT4  2
#define SALICACHE_INT8  3
#define SALICACHE_FP16  4

typedef struct salicache_ctx salicache_ctx;

/* Parameters.  The paper fixes: Farneback flow with pyramid scale 0.5 and 3 levels,
 * Canny + LAB colour variance, Eq. 5-8, symmetric INT8 and asymmetric INT4 (Sec. IV-B).
 * It prints no value for any threshold (Alg. 1 input); the other fields are the
 * readings this library takes where the paper is silent. */
typedef struct salicache_params {
    int32_t H, W;            /* frame size; multiples of `patch`, W % 16 == 0 (336 or 672)          */
    int32_t patch;           /* 14 (Sec. II-A)                                                       */
    int32_t n_images;        /* 1, or 5 = anyres: 336x336 base (2x2 box mean of the frame) followed  */
                             /* by the 2x2 grid of 336x336 tiles; H = W = 672 then                   */
    int32_t max_batch;       /* largest B accepted by any call                                       */
    int32_t chunk_frames;    /* frames per internal pass of flow/saliency (scratch size); 0 = 16     */
    /* temporal branch */
    int32_t pyr_levels;      /* 3 (only value supported)                                             */
    int32_t poly_n;          /* 5 (only value supported)                                             */
    double  poly_sigma;      /* 1.2                                                                  */
    int32_t win;             /* 15 (only value supported)                                            */
    int32_t iters;           /* updates per level, 3                                                 */
    double  eps_det;         /* regulariser added to det G, 1e-3                                     */
    /* spatial branch */
    int32_t canny_lo, canny_hi;   /* 50, 150 on the Sobel magnitude                                  */
    int32_t var_radius;      /* 3 (7x7 window; only value supported)                                 */
    double  sigma_ref;       /* 16.0: C = min(1, sqrt(V)/sigma_ref)                                  */
    double  w_edge, w_color; /* 0.5, 0.5                                                             */
    int32_t hyst_max_iters;  /* 4096                                                                 */
    /* decisions (Alg. 1 input) */
    float   tau_t, theta_R, tau_high, tau_med, tau_low;
    int32_t patch_reuse;     /* 1: static patches of a non-redundant frame are REUSE (Fig. 3)        */
    /* K/V shape and quantiser */
    int32_t L, heads, head_dim;   /* layers, heads, head size; heads*head_dim = row length HD        */
    int32_t group;           /* elements per quantisation group: 128 (one head), or heads*head_dim    */
                             /* (one scale, and zero, per token row)                                  */
    /* colour term, frame-adaptive reading of Sec. IV-B's "adaptive thresholding based on the local   */
    /* color variance" (a variant; 0 = the fixed sigma_ref above)                                     */
    int32_t color_norm;      /* 1: C = min(1, sqrt(V) / (color_kappa * sigma_frame)) with             */
                             /* sigma_frame = max(sqrt(mean over the image of V), color_sigma_min)    */
    double  color_kappa;     /* 1.0                                                                   */
    double  color_sigma_min; /* 0.5 (LAB units): an image without contrast stays without saliency     */
} salicache_params;

/* Fills *p with the defaults listed above for a 336x336, L=32, 32x128 configuration. */
SALICACHE_API int salicache_default_params(salicache_params* p);

/* Allocates a context and its scratch on the current CUDA device.  Errors: E_NULL, E_PARAM
 * (unsupported value), E_SHAPE (sizes not multiples), E_NOMEM, E_CUDA. */
SALICACHE_API int salicache_create(salicache_ctx** out, const salicache_params* p);
SALICACHE_API int salicache_destroy(salicache_ctx* ctx);
SALICACHE_API const char* salicache_strerror(int status);

/* Tokens per frame: n_images * (336/patch)^2 for anyres, else (H/patch)*(W/patch). */
SALICACHE_API int salicache_tokens_per_frame(const salicache_ctx* ctx);

/* Number of CUDA kernels this context has launched since it was created (host-side count). */
SALICACHE_API int64_t salicache_launch_count(const salicache_ctx* ctx);

/*
 * Temporal score (Sec. III-A, Eq. 5; Farneback flow, Sec. IV-B).
 * For b in [0,B): dense flow from d_prev[b] to d_cur[b] (frames of H*W*3 bytes, consecutive),
 * reduced to d_deltaP[b][i] = RMS flow magnitude (pixels) over patch i, i in token order.
 * d_cur == d_prev + H*W*3 (a video: pair b is frames b, b+1) is recognised and each frame is
 * expanded once.  d_flow_or_null, if given, receives the level-0 flow as double [B][2][H][W]
 * (u along x, then v); anyres contexts write only the full-resolution field.
 * Device arithmetic (Sec. III-A, Eq. 5): single precision throughout, arranged so that it holds the
 * tolerance: the polynomial expansion takes its moments through zero-sum kernels and differences from the
 * window centre (coefficients good to a few 1e-7 relative); the normal-equation terms, their 15x15 window sums (sums of their own
 * terms only, no running subtraction) and the 2x2 solve (compensated products) run in single precision;
 * sampling positions are exact; the patch reduction is double.  Tested bound: d_deltaP within 1e-4
 * relative (floor 1e-6) of the double-precision definition, the dense field within 2e-5 px.
 * Errors: E_NULL, E_SHAPE (B < 0 or > max_batch), E_ALIGN, E_CUDA.
 */
SALICACHE_API int salicache_flow_score(salicache_ctx* ctx, const uint8_t* d_prev, const uint8_t* d_cur, int B,
                         float* d_deltaP, double* d_flow_or_null, void* cuda_stream);

/*
 * Temporal score, Eq. 5 read literally (no optical flow): d_deltaP[b][i] = L2 norm of the pixel difference
 * d_cur[b] - d_prev[b] over patch i, divided by sqrt(3 * patch * patch): the RMS difference in grey levels,
 * summed exactly in integers.  A cheap alternative to salicache_flow_score (one pass over the two frames);
 * tau_t is then a grey-level threshold instead of pixels of motion.  Same arguments and errors as
 * salicache_flow_score (no flow field).
 */
SALICACHE_API int salicache_diff_score(salicache_ctx* ctx, const uint8_t* d_prev, const uint8_t* d_cur, int B,
                                       float* d_deltaP, void* cuda_stream);

/*
 * Spatial score (Sec. III-B, Eq. 7): Canny edge map E and LAB local colour variance C give
 * S = clamp(w_edge E + w_color C, 0, 1); d_s[b][i] = mean of S over patch i.
 * d_frames: B frames.  d_skip_or_null: DEVICE u8 [B] or NULL; frames with a non-zero entry are not
 * scored and their rows of d_s are left untouched (Alg. 1 skips the spatial branch of a temporally
 * redundant frame: pass the flags of salicache_frame_redundancy).  Edge hysteresis runs to its
 * fixed point on the device in rounds (in a round every strip of rows is swept until it is stable, at
 * most 64 times, then the whole frame votes); if it needs more than hyst_max_iters rounds the status
 * word records E_NOCONVERGE (see salicache_poll_status).
 */
SALICACHE_API int salicache_saliency(salicache_ctx* ctx, const uint8_t* d_frames, int B, float* d_s,
                                     const uint8_t* d_skip_or_null, void* cuda_stream);

/*
 * Frame redundancy alone (Eq. 6; Alg. 1 lines 4-8): d_frame_redundant[b] = 1 when frame b has a
 * predecessor and R_frame = (1/N) sum_i [dP_i < tau_t] exceeds theta_R, else 0.  Same arithmetic as
 * salicache_select, which recomputes it; this call exists so that the spatial branch can skip the
 * redundant frames.  d_deltaP: f32 [B][N_tok] or NULL (no frame has a predecessor);
 * first_has_no_prev as for salicache_select.  Errors: E_NULL, E_SHAPE, E_CUDA.
 */
SALICACHE_API int salicache_frame_redundancy(salicache_ctx* ctx, const float* d_deltaP, int B, int first_has_no_prev,
                                             uint8_t* d_frame_redundant, void* cuda_stream);

/*
 * Decisions (Eq. 6, Eq. 8, Alg. 1) for B frames, one row of d_deltaP / d_s per frame.
 * d_deltaP may be NULL (no frame has a predecessor).  If first_has_no_prev != 0, frame 0 is the
 * first frame of the video: its d_deltaP row is ignored and it is never REUSE (Alg. 1 line 4).
 * Outputs (all device):
 *   d_decision        u8  [B][N_tok]     SALICACHE_* code per token
 *   d_idx             i32 [B][3][N_tok]  ascending token ids kept as FP16 / INT8 / INT4; -1 padded
 *   d_counts          i32 [B][5]         tokens per code (indexed by code)
 *   d_frame_redundant u8  [B]            1 when R_frame > theta_R (whole frame points at t-1)
 *   d_row_offset      i64 [B][3]         first pool row of the frame in the FP16 / INT8 / INT4 pool
 *   d_fill            i64 [3]            running rows written per pool; read, used as the offset of
 *                                        frame 0 and advanced by the batch totals (zero it once)
 * pack_kv / unpack_kv consume these from device memory: no host round trip is needed.
 */
SALICACHE_API int salicache_select(salicache_ctx* ctx, const float* d_deltaP, const float* d_s, int B, int first_has_no_prev,
                     uint8_t* d_decision, int32_t* d_idx, int32_t* d_counts, uint8_t* d_frame_redundant,
                     int64_t* d_row_offset, int64_t* d_fill, void* cuda_stream);

/*
 * Source-frame table (Alg. 1 line 7: a reused entry is a pointer to the previous frame's entry; Fig. 3
 * counts reuse per patch).  For the B frames first_frame .. first_frame+B-1 of a video:
 *   d_src[b][i] = d_src[b-1][i] if decision[b][i] == SALICACHE_REUSE, else first_frame + b,
 * chains resolved, so that every token names the frame whose stored (or pruned) entry it uses.
 *   d_decision  DEVICE u8  [B][N_tok]  from salicache_select
 *   d_carry     DEVICE i32 [N_tok]     in: sources of frame first_frame-1 (ignored where frame 0 cannot
 *                                      reuse); out: sources of the batch's last frame, for the next call
 *   d_src       DEVICE i32 [B][N_tok]  written
 * Errors: E_NULL, E_SHAPE, E_CUDA.
 */
SALICACHE_API int salicache_source_frames(salicache_ctx* ctx, const uint8_t* d_decision, int B, int first_frame,
                                          int32_t* d_carry, int32_t* d_src, void* cuda_stream);

/* Per-tier pools of the mixed-precision store (device memory, caller-owned).  Axis 2 of the
 * second dimension: 0 = K, 1 = V.  ng = HD / group.
 *   fp16_pool   f16 [L][2][cap_fp16][HD]
 *   int8_codes  i8  [L][2][cap_int8][HD]      int8_scale f16 [L][2][cap_int8][ng]
 *   int4_codes  u8  [L][2][cap_int4][HD/2]    int4_sz    f16 [L][2][cap_int4][ng][2]  (scale, zero)
 * The j-th token of a frame's tier list lives in row (row_offset + j) % cap when ring != 0
 * (row offsets are absolute positions; the oldest rows are overwritten: oldest-first eviction
 * under a fixed budget; when one call stores more than cap rows in a pool, the rows that a later
 * row of the same call lands on are skipped, so that the newest cap rows are what the pool
 * holds), else in row row_offset + j, and rows at or past cap are dropped with E_CAPACITY in
 * the status word.
 *   d_fill      optional (NULL = no check): DEVICE i64 [3], the running fill salicache_select
 *               maintains (rows ever stored per tier: FP16, INT8, INT4).  With ring != 0 it tells
 *               salicache_unpack_kv which rows still exist: a row with row_offset + j <
 *               fill - cap has been overwritten by a newer frame; it is not read, the output row
 *               is zeroed, and E_EVICTED is recorded in the status word. */
typedef struct salicache_pools {
    void* fp16_pool;
    void* int8_codes;
    void* int8_scale;
    void* int4_codes;
    void* int4_sz;
    int64_t cap_fp16, cap_int8, cap_int4;
    int32_t ring;
    const int64_t* d_fill;
} salicache_pools;

/*
 * Mixed-precision store (Alg. 1 line 16; quantisers of Sec. IV-B).  d_K, d_V: f16
 * [B][L][N_tok][HD] with `frame_stride` elements between frames (L*N_tok*HD when dense).
 * FP16 rows are copied; INT8: s = fp16(max|x|/127), q = rint(x * (1/s)); INT4: s =
 * fp16((max-min)/15), zero = min (fp16), q = rint((x - zero) * (1/s)), element 2j in the low
 * nibble; s == 0 -> 1.  All binary32, round-to-nearest-even, no fused multiply-add.
 * PRUNE and REUSE tokens move no bytes.  Errors: E_NULL, E_SHAPE, E_ALIGN, E_CUDA; deferred
 * E_CAPACITY.
 */
SALICACHE_API int salicache_pack_kv(salicache_ctx* ctx, const void* d_K, const void* d_V, int64_t frame_stride,
                      const int32_t* d_idx, const int32_t* d_counts, const int64_t* d_row_offset, int B,
                      const salicache_pools* pools, void* cuda_stream);

/*
 * Just-in-time dequantisation (Sec. III-C) into dense f16 d_K_out, d_V_out [B][L][N_tok][HD].
 * INT8: fp16(q*s); INT4: fp16(q*s + zero) (multiply, then add); FP16 rows are bit copies;
 * PRUNE rows are zeroed when zero_fill_pruned != 0, otherwise untouched; REUSE rows are left
 * untouched (the caller resolves them through its source-frame table).  With ring pools and
 * pools->d_fill given, rows that have been overwritten are zeroed instead of read (deferred
 * E_EVICTED).  Errors: E_NULL, E_SHAPE, E_ALIGN, E_CUDA; deferred E_CAPACITY, E_EVICTED.
 */
SALICACHE_API int salicache_unpack_kv(salicache_ctx* ctx, const salicache_pools* pools, const int32_t* d_idx,
                        const int32_t* d_counts, const uint8_t* d_decision, const int64_t* d_row_offset, int B,
                        int zero_fill_pruned, void* d_K_out, void* d_V_out, int64_t frame_stride,
                        void* cuda_stream);

/*
 * Which stored frames a budgeted cache still holds (fixed memory budget, Sec. IV-A; ring pools with
 * oldest-first eviction).  d_resident[b] = 1 when every row frame b stored is still in the pools at the
 * running fill pools->d_fill (required): per tier, the frame stored nothing, or it fits the ring and
 * row_offset >= fill - cap (linear pools: row_offset + count <= cap).  A frame's record is evicted as a
 * whole: one overwritten tier makes it non-resident.
 *   d_counts i32 [B][5], d_row_offset i64 [B][3] as written by salicache_select; d_resident u8 [B] written.
 * Errors: E_NULL, E_SHAPE, E_CUDA.
 */
SALICACHE_API int salicache_frames_resident(salicache_ctx* ctx, const int32_t* d_counts, const int64_t* d_row_offset, int B,
                                            const salicache_pools* pools, uint8_t* d_resident, void* cuda_stream);

/*
 * A reused token lives as long as the frame that holds its entry (Alg. 1 line 7: a pointer; a root is
 * evicted together with every alias that points to it): d_live[b][i] = d_resident_table[d_src[b][i] -
 * first_frame], and 0 when the source frame lies outside the table.
 *   d_src i32 [B][N_tok] from salicache_source_frames; d_resident_table u8 [n_table] describes frames
 *   first_frame .. first_frame + n_table - 1; d_live u8 [B][N_tok] written.
 * Errors: E_NULL, E_SHAPE, E_CUDA.
 */
SALICACHE_API int salicache_tokens_live(salicache_ctx* ctx, const int32_t* d_src, int B, int first_frame,
                                        const uint8_t* d_resident_table, int n_table, uint8_t* d_live, void* cuda_stream);

/*
 * The spatial score without any allocation.  (The paper has no counterpart: this entry point
 * exists for the way the library is embedded, not for the method.)
 *
 * For callers that cannot allocate device memory while they run -- a serving process whose memory
 * pool already owns the whole GPU, a plug-in that may not grow the process, code under an
 * allocator lock -- and therefore cannot create a context.  It computes exactly what
 * salicache_saliency computes (same kernels, same bits), but keeps the edge bit planes, the sRGB
 * table and the status word in one fixed array inside the library's device image
 * (about 233 KB, held by every GPU that loads the library until the process exits).  It calls no
 * cudaMalloc / cudaFree and no allocating library routine.
 *
 *   p           HOST pointer; the fields read are H, W, patch, n_images, canny_lo, canny_hi,
 *               var_radius, sigma_ref, w_edge, w_color, hyst_max_iters, color_norm.  n_images must
 *               be 1, color_norm 0 (the frame-adaptive colour term needs a context's scratch) and
 *               H, W at most SALICACHE_NOALLOC_MAX_SIDE (multiples of 112 as for a context).
 *   d_frames    DEVICE, u8 [B][H][W][3], 16-byte aligned, caller-owned
 *   B           0 .. SALICACHE_NOALLOC_MAX_FRAMES; larger batches are rejected with E_SHAPE and
 *               nothing is launched (split them into several calls on the same stream)
 *   d_s         DEVICE, f32 [B][(H/patch)*(W/patch)], caller-owned, written
 *   d_status_or_null  DEVICE int32 the caller zeroed: receives SALICACHE_E_NOCONVERGE if edge
 *               hysteresis hits hyst_max_iters.  With NULL the condition is recorded in the
 *               library's own word, which this call clears first and nobody reads.
 *
 * The first call on each device resolves the array's device address, sets two kernel attributes
 * and copies the 2 KB sRGB table with a blocking copy; make that call once per device with that
 * device current before capturing a stream or entering a latency-critical section.  Later calls
 * are asynchronous on `cuda_stream`.
 * All calls on one device share the array and it keeps the previous call's contents (each call
 * overwrites what it reads, and clears the status word).  Two calls that overlap on the GPU --
 * different streams, or different host threads without ordering -- race on it: serialise them.
 * Errors: E_NULL, E_PARAM, E_SHAPE, E_ALIGN, E_CUDA, as for salicache_saliency.
 */
#define SALICACHE_NOALLOC_MAX_FRAMES 8
#define SALICACHE_NOALLOC_MAX_SIDE   336
SALICACHE_API int salicache_saliency_noalloc(const salicache_params* p, const uint8_t* d_frames, int B, float* d_s,
                                             int32_t* d_status_or_null, void* cuda_stream);

/*
 * Decisions with adaptive tier thresholds (a variant; the paper's thresholds are fixed and Sec. V names their
 * adaptation to the content as future work).  The temporal test is salicache_select's (Eq. 6, patch reuse).  Among
 * the n_live tokens of a frame that are not reused, Eq. 8's tiers are given out by rank of s_i in fixed shares:
 *   q16 = (n_live * share_fp16_permille + 500) / 1000 (integer division), likewise q8 and q4, each clipped to what
 *   is left of n_live; the q16 most salient tokens are FP16, the next q8 INT8, the next q4 INT4, the rest PRUNE;
 *   equal scores go to the lower token id first.
 * tau_high, tau_med and tau_low of the context are not used.  All other arguments, outputs and errors as for
 * salicache_select; shares outside [0, 1000]: E_PARAM; contexts with more than 3072 tokens per frame: E_PARAM.
 */
SALICACHE_API int salicache_select_ranked(salicache_ctx* ctx, const float* d_deltaP, const float* d_s, int B,
                                          int first_has_no_prev, int share_fp16_permille, int share_int8_permille,
                                          int share_int4_permille, uint8_t* d_decision, int32_t* d_idx, int32_t* d_counts,
                                          uint8_t* d_frame_redundant, int64_t* d_row_offset, int64_t* d_fill,
                                          void* cuda_stream);

/*
 * Temporal test and decisions in anchor-frame mode (a variant; the paper's test compares consecutive frames,
 * Sec. III-A, under which a slow pan or fade whose every step stays below tau_t is reused forever).  Token i of
 * frame b is compared with the patch its cache entry was computed from, i.e. patch i of the last frame in which
 * token i was not SALICACHE_REUSE (the frame Alg. 1's pointers resolve to).  d_anchor holds that composite image.
 * For b = 0 .. B-1 in order:
 *   d_deltaP[b][i] = Eq. 5 read literally (as salicache_diff_score) between d_anchor and frame b; 0 for a first
 *                    frame without predecessor;
 *   decisions, index lists, counts, redundancy flag = salicache_select's rule (Eq. 6, Eq. 8) on that row;
 *   d_anchor <- frame b on every patch whose token is not SALICACHE_REUSE;
 * then row offsets and d_fill as salicache_select.  tau_t is a grey-level threshold here.  Each frame depends on
 * the decisions of the one before: the frames of one call are processed in sequence by one cluster of CTAs.
 *   d_frames  DEVICE u8 [B][H][W][3], 16-byte aligned;  d_s DEVICE f32 [B][N_tok] (salicache_saliency)
 *   d_anchor  DEVICE u8 [H][W][3], 16-byte aligned, caller-owned, read and written: pass the same buffer to the
 *             next call (first_has_no_prev = 0) to continue the video; its content is ignored, and replaced, when
 *             first_has_no_prev != 0 (frame 0 then stores every token)
 *   d_deltaP  DEVICE f32 [B][N_tok], written;  the remaining arguments as for salicache_select
 * Contexts with an anyres token layout, a patch size other than 14 or more than 48 x 48 patches: E_PARAM.
 * Errors: E_NULL, E_SHAPE (B < 0 or > max_batch), E_ALIGN, E_PARAM, E_CUDA.
 */
SALICACHE_API int salicache_select_anchored(salicache_ctx* ctx, const uint8_t* d_frames, const float* d_s, int B,
                                            int first_has_no_prev, uint8_t* d_anchor, float* d_deltaP, uint8_t* d_decision,
                                            int32_t* d_idx, int32_t* d_counts, uint8_t* d_frame_redundant,
                                            int64_t* d_row_offset, int64_t* d_fill, void* cuda_stream);

/*
 * salicache_select_anchored for n_videos independent videos of B frames each in one launch (one cluster of CTAs per
 * video, so that a GPU works on many streams at once; a single video occupies 8 of its SMs).  Every array has a
 * leading video dimension: d_frames [n_videos][B][H][W][3], d_s and d_deltaP [n_videos][B][N_tok], d_anchor
 * [n_videos][H][W][3], d_decision [n_videos][B][N_tok], d_idx [n_videos][B][3][N_tok], d_counts [n_videos][B][5],
 * d_frame_redundant [n_videos][B], d_row_offset [n_videos][B][3], d_fill [n_videos][3] (each video fills pools of its
 * own); first_has_no_prev applies to every video.  n_videos < 0 or > 4096: E_SHAPE; otherwise as salicache_select_anchored.
 */
SALICACHE_API int salicache_select_anchored_batch(salicache_ctx* ctx, const uint8_t* d_frames, const float* d_s, int n_videos,
                                                  int B, int first_has_no_prev, uint8_t* d_anchor, float* d_deltaP,
                                                  uint8_t* d_decision, int32_t* d_idx, int32_t* d_counts,
                                                  uint8_t* d_frame_redundant, int64_t* d_row_offset, int64_t* d_fill,
                                                  void* cuda_stream);

/*
 * Decode attention straight from the mixed-precision store (Eq. 2 with the just-in-time dequantisation of
 * Sec. III-C fused in): for every layer l and head h,
 *   score_j = q[l][h] . K^_j / sqrt(head_dim),  p = softmax_j(score),  out[l][h] = sum_j p_j V^_j,
 * over the rows j the pools hold: rows [0, min(fill, cap)) of the FP16, INT8 and INT4 pool (pruned tokens
 * have no row; a reused token is attended through the row it points to, once).  K^, V^ are the dequantised
 * values q*s and q*s + zero in single precision, not rounded to binary16 in between.
 *   d_q     DEVICE f16 [L][heads][head_dim], 16-byte aligned
 *   pools   as for salicache_pack_kv;  d_fill DEVICE i64 [3]: rows written per pool (salicache_select's d_fill)
 *   d_out   DEVICE f32 [L][heads][head_dim], written; zeros when the store is empty
 * Needs head_dim == 128 and group == 128 or heads*head_dim (E_PARAM otherwise); pool capacities below 2^28
 * rows.  Errors: E_NULL, E_ALIGN, E_PARAM, E_SHAPE, E_CUDA.
 */
SALICACHE_API int salicache_attend(salicache_ctx* ctx, const void* d_q, const salicache_pools* pools, const int64_t* d_fill,
                                   float* d_out, void* cuda_stream);

/*
 * The same attention for grouped-query models (the paper's evaluation model, LLaVA-1.6 Mistral-7B, has 8 key/value
 * heads that serve 32 query heads, Sec. IV-A): query head hq, 0 <= hq < heads * q_per_kv, attends to the rows of
 * key/value head hq / q_per_kv of the store (heads = the context's heads, the store's key/value heads).
 *   d_q, d_out   DEVICE f16 / f32 [L][heads * q_per_kv][head_dim], 16-byte aligned
 * q_per_kv = 1 is salicache_attend.  q_per_kv < 1 or heads * q_per_kv > max(heads, 64): E_SHAPE.  Up to 4 queries
 * per key/value head share one pass over its rows (the store is read once for the whole group); larger groups take
 * one pass per 4 queries.  Other arguments and errors as for salicache_attend.
 */
SALICACHE_API int salicache_attend_gqa(salicache_ctx* ctx, const void* d_q, int q_per_kv, const salicache_pools* pools,
                                       const int64_t* d_fill, float* d_out, void* cuda_stream);

/* Synchronises `cuda_stream`, returns the deferred device status (0, E_CAPACITY or
 * E_NOCONVERGE; E_CUDA if the stream reports an error) and clears it. */
SALICACHE_API int salicache_poll_status(salicache_ctx* ctx, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SALICACHE_H */
