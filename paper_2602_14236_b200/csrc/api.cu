// C ABI of libsalicache.so: parameter validation, scratch ownership, dispatch to the stage launchers.
#include <math.h>
#include <new>
#include <string.h>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"

int sc_flow_init();
int sc_saliency_init(int max_h, int max_words);
int sc_kv_max_batch();
bool sc_kv_supported_hd(int HD);

namespace {

// A named range around the launches of one call, for timelines (costs nothing when no tool is attached).
struct Range {
    explicit Range(const char* name) { nvtxRangePushA(name); }
    ~Range() { nvtxRangePop(); }
};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

void free_scratch(salicache_ctx* c) {
    for (int l = 0; l < 3; ++l) {
        if (c->pyr[l]) cudaFree(c->pyr[l]);
        if (c->coef[l]) cudaFree(c->coef[l]);
    }
    if (c->gh_a) cudaFree(c->gh_a);
    if (c->flow_a) cudaFree(c->flow_a);
    if (c->flow_b) cudaFree(c->flow_b);
    if (c->bits_kept) cudaFree(c->bits_kept);
    if (c->bits_edge) cudaFree(c->bits_edge);
    if (c->lut) cudaFree(c->lut);
    if (c->sqrt_v) cudaFree(c->sqrt_v);
    if (c->v_part) cudaFree(c->v_part);
    if (c->base_frames) cudaFree(c->base_frames);
    if (c->row_prefix) cudaFree(c->row_prefix);
    if (c->attend_ws) cudaFree(c->attend_ws);
    if (c->d_status) cudaFree(c->d_status);
}

}  // namespace

extern "C" {

int salicache_default_params(salicache_params* p) {
    if (!p) return SALICACHE_E_NULL;
    memset(p, 0, sizeof(*p));
    p->H = 336; p->W = 336; p->patch = 14; p->n_images = 1; p->max_batch = 64; p->chunk_frames = 16;
    p->pyr_levels = 3; p->poly_n = 5; p->poly_sigma = 1.2; p->win = 15; p->iters = 3; p->eps_det = 1e-3;
    p->canny_lo = 50; p->canny_hi = 150; p->var_radius = 3; p->sigma_ref = 16.0; p->w_edge = 0.5; p->w_color = 0.5;
    p->hyst_max_iters = 4096;
    p->tau_t = 0.5f; p->theta_R = 0.90f; p->tau_high = 0.40f; p->tau_med = 0.36f; p->tau_low = 0.25f;
    p->patch_reuse = 1;
    p->L = 32; p->heads = 32; p->head_dim = 128; p->group = 128;
    p->color_norm = 0; p->color_kappa = 1.0; p->color_sigma_min = 0.5;
    return SALICACHE_OK;
}

const char* salicache_strerror(int status) {
    switch (status) {
        case SALICACHE_OK: return "ok";
        case SALICACHE_E_NULL: return "a required pointer is NULL";
        case SALICACHE_E_SHAPE: return "sizes inconsistent with the context";
        case SALICACHE_E_ALIGN: return "pointer not 16-byte aligned";
        case SALICACHE_E_PARAM: return "unsupported parameter value";
        case SALICACHE_E_CUDA: return "CUDA runtime error";
        case SALICACHE_E_CAPACITY: return "tier pool too small; rows were dropped";
        case SALICACHE_E_NOCONVERGE: return "edge hysteresis hit its iteration cap";
        case SALICACHE_E_NOMEM: return "scratch allocation failed";
        case SALICACHE_E_EVICTED: return "rows asked for have been overwritten in a ring pool; zeros were returned";
        default: return "unknown status";
    }
}

int salicache_create(salicache_ctx** out, const salicache_params* p) {
    if (!out || !p) return SALICACHE_E_NULL;
    *out = nullptr;
    if (p->pyr_levels != 3 || p->poly_n != 5 || p->win != 15 || p->var_radius != 3 || p->patch != 14 ||
        (p->group != 128 && p->group != p->heads * p->head_dim) || p->iters < 1 || p->iters > 64 || !(p->poly_sigma > 0) || !(p->sigma_ref > 0) ||
        p->canny_lo < 0 || p->canny_hi < p->canny_lo || p->canny_hi > 1442 || p->hyst_max_iters < 1 ||
        (p->n_images != 1 && p->n_images != 5) || p->L < 1 || p->heads < 1 || p->head_dim < 1 ||
        (p->color_norm != 0 && p->color_norm != 1) || (p->color_norm == 1 && (!(p->color_kappa > 0) || !(p->color_sigma_min >= 0))))
        return SALICACHE_E_PARAM;
    const int HD = p->heads * p->head_dim;
    if (!sc_kv_supported_hd(HD)) return SALICACHE_E_PARAM;
    if (p->H <= 0 || p->W <= 0 || p->H % 112 != 0 || p->W % 112 != 0) return SALICACHE_E_SHAPE;  // 28-px tiles at 1/4 scale, 16 | W
    if (p->n_images == 5 && (p->H != 672 || p->W != 672)) return SALICACHE_E_SHAPE;
    if (p->max_batch < 1 || p->max_batch > sc_kv_max_batch()) return SALICACHE_E_SHAPE;
    salicache_ctx* c = new (std::nothrow) salicache_ctx();
    if (!c) return SALICACHE_E_NOMEM;
    memset(c, 0, sizeof(*c));
    c->p = *p;
    c->chunk = p->chunk_frames > 0 ? p->chunk_frames : 16;
    if (c->chunk > p->max_batch) c->chunk = p->max_batch;
    const int gh = p->H / p->patch, gw = p->W / p->patch;
    if (p->n_images == 1) {
        c->n_planes = 1;
        c->n_tok = gh * gw;
        c->plane[0] = PlaneGeom{p->H, p->W, gh, gw, 0, 0, c->n_tok};
    } else {
        c->n_planes = 2;
        c->n_tok = 5 * 576;
        c->plane[0] = PlaneGeom{p->H, p->W, gh, gw, 1, 576, c->n_tok};
        c->plane[1] = PlaneGeom{p->H / 2, p->W / 2, gh / 2, gw / 2, 0, 0, c->n_tok};
    }
    int dev = 0;
    cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
        delete c;
        return SALICACHE_E_CUDA;
    }
    c->sm_count = prop.multiProcessorCount;
    const size_t P0 = (size_t)p->H * p->W;
    const size_t slots = (size_t)2 * c->chunk;   // independent pairs need prev and cur; a video needs chunk+1
    const int words = (p->W + 31) / 32;
    bool ok = true;
    for (int l = 0; l < 3 && ok; ++l) {
        size_t Pl = P0 >> (2 * l);
        ok = ok && cudaMalloc(&c->pyr[l], slots * Pl * sizeof(float)) == cudaSuccess;
        // 16-byte records then one plane, each zeroed and followed by a pad of one row + 2: the flow kernels read
        // (and multiply by zero) the tap after the last column / row
        const size_t cbytes = (slots * 5 * Pl + 5 * ((size_t)(p->W >> l) + 2)) * sizeof(float);
        ok = ok && cudaMalloc(&c->coef[l], cbytes) == cudaSuccess;
        ok = ok && cudaMemset(c->coef[l], 0, cbytes) == cudaSuccess;
    }
    ok = ok && cudaMalloc(&c->gh_a, (size_t)c->chunk * 5 * P0 * sizeof(float)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->flow_a, (size_t)c->chunk * 2 * P0 * sizeof(float)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->flow_b, (size_t)c->chunk * 2 * P0 * sizeof(float)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->bits_kept, (size_t)c->chunk * p->H * words * sizeof(uint32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->bits_edge, (size_t)c->chunk * p->H * words * sizeof(uint32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->lut, 256 * sizeof(double)) == cudaSuccess;
    if (p->color_norm == 1) {
        ok = ok && cudaMalloc(&c->sqrt_v, (size_t)c->chunk * P0 * sizeof(float)) == cudaSuccess;
        ok = ok && cudaMalloc(&c->v_part, (size_t)c->chunk * (p->H / 28) * (p->W / 28) * sizeof(double)) == cudaSuccess;
    }
    ok = ok && cudaMalloc(&c->row_prefix, ((size_t)p->max_batch + 1) * sizeof(int64_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_status, sizeof(int)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->attend_ws, sc_attend_workspace_bytes(p->L, p->heads)) == cudaSuccess;
    if (ok && p->n_images == 5)
        ok = cudaMalloc(&c->base_frames, ((size_t)p->max_batch + 1) * (P0 / 4) * 3) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        free_scratch(c);
        delete c;
        return SALICACHE_E_NOMEM;
    }
    double lut[256];
    for (int i = 0; i < 256; ++i) {   // IEC 61966-2-1 transfer curve
        double v = i / 255.0;
        lut[i] = v <= 0.04045 ? v / 12.92 : pow((v + 0.055) / 1.055, 2.4);
    }
    int st = SALICACHE_OK;
    if (cudaMemcpy(c->lut, lut, sizeof(lut), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemset(c->d_status, 0, sizeof(int)) != cudaSuccess ||
        cudaDeviceSynchronize() != cudaSuccess)      // the table and the zeroed scratch are in place before any stream uses them
        st = SALICACHE_E_CUDA;
    if (st == SALICACHE_OK) st = sc_flow_init();
    if (st == SALICACHE_OK) st = sc_saliency_init(p->H, words);
    if (st != SALICACHE_OK) {
        free_scratch(c);
        delete c;
        return st;
    }
    *out = c;
    return SALICACHE_OK;
}

int salicache_destroy(salicache_ctx* c) {
    if (!c) return SALICACHE_E_NULL;
    free_scratch(c);
    delete c;
    return SALICACHE_OK;
}

int salicache_tokens_per_frame(const salicache_ctx* c) { return c ? c->n_tok : SALICACHE_E_NULL; }

int64_t salicache_launch_count(const salicache_ctx* c) { return c ? (int64_t)c->launches : (int64_t)SALICACHE_E_NULL; }

int salicache_flow_score(salicache_ctx* c, const uint8_t* d_prev, const uint8_t* d_cur, int B, float* d_deltaP,
                         double* d_flow_or_null, void* cuda_stream) {
    Range range__("salicache_flow_score");
    if (!c || !d_prev || !d_cur || !d_deltaP) return SALICACHE_E_NULL;
    if (B < 0 || B > c->p.max_batch) return SALICACHE_E_SHAPE;
    if (!aligned16(d_prev) || !aligned16(d_cur) || !aligned16(d_deltaP) || !aligned16(d_flow_or_null))
        return SALICACHE_E_ALIGN;
    if (B == 0) return SALICACHE_OK;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t fb = (size_t)c->p.H * c->p.W * 3;
    const bool sequence = d_cur == d_prev + fb;
    int rc = sc_flow_score(c, c->plane[0], d_prev, d_cur, fb, B, sequence, d_deltaP, d_flow_or_null, st);
    if (rc != SALICACHE_OK || c->n_planes == 1) return rc;
    // anyres base image: 2x2 box mean of the frames, then the same path at 336x336
    const size_t fbb = fb / 4;
    uint8_t* base = c->base_frames;
    if (sequence) {
        rc = sc_box_down2(d_prev, c->p.H, c->p.W, B + 1, base, st);
        c->launches++;
        if (rc != SALICACHE_OK) return rc;
        return sc_flow_score(c, c->plane[1], base, base + fbb, fbb, B, true, d_deltaP, nullptr, st);
    }
    // independent pairs: process prev then cur halves in passes that fit the base buffer
    for (int b0 = 0; b0 < B;) {
        int nb = (c->p.max_batch + 1) / 2;
        if (nb > B - b0) nb = B - b0;
        rc = sc_box_down2(d_prev + (size_t)b0 * fb, c->p.H, c->p.W, nb, base, st);
        if (rc == SALICACHE_OK) rc = sc_box_down2(d_cur + (size_t)b0 * fb, c->p.H, c->p.W, nb, base + (size_t)nb * fbb, st);
        c->launches += 2;
        if (rc == SALICACHE_OK)
            rc = sc_flow_score(c, c->plane[1], base, base + (size_t)nb * fbb, fbb, nb, false,
                               d_deltaP + (size_t)b0 * c->n_tok, nullptr, st);
        if (rc != SALICACHE_OK) return rc;
        b0 += nb;
    }
    return SALICACHE_OK;
}

int salicache_diff_score(salicache_ctx* c, const uint8_t* d_prev, const uint8_t* d_cur, int B, float* d_deltaP,
                         void* cuda_stream) {
    Range range__("salicache_diff_score");
    if (!c || !d_prev || !d_cur || !d_deltaP) return SALICACHE_E_NULL;
    if (B < 0 || B > c->p.max_batch) return SALICACHE_E_SHAPE;
    if (!aligned16(d_prev) || !aligned16(d_cur) || !aligned16(d_deltaP)) return SALICACHE_E_ALIGN;
    if (B == 0) return SALICACHE_OK;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t fb = (size_t)c->p.H * c->p.W * 3;
    int rc = sc_diff_score(c, c->plane[0], d_prev, d_cur, fb, B, d_deltaP, st);
    if (rc != SALICACHE_OK || c->n_planes == 1) return rc;
    // anyres base image: 2x2 box mean of both frames of every pair, in passes that fit the base buffer
    const size_t fbb = fb / 4;
    uint8_t* base = c->base_frames;
    for (int b0 = 0; b0 < B;) {
        int nb = (c->p.max_batch + 1) / 2;
        if (nb > B - b0) nb = B - b0;
        rc = sc_box_down2(d_prev + (size_t)b0 * fb, c->p.H, c->p.W, nb, base, st);
        if (rc == SALICACHE_OK) rc = sc_box_down2(d_cur + (size_t)b0 * fb, c->p.H, c->p.W, nb, base + (size_t)nb * fbb, st);
        c->launches += 2;
        if (rc == SALICACHE_OK)
            rc = sc_diff_score(c, c->plane[1], base, base + (size_t)nb * fbb, fbb, nb, d_deltaP + (size_t)b0 * c->n_tok, st);
        if (rc != SALICACHE_OK) return rc;
        b0 += nb;
    }
    return SALICACHE_OK;
}

int salicache_frame_redundancy(salicache_ctx* c, const float* d_deltaP, int B, int first_has_no_prev,
                               uint8_t* d_frame_redundant, void* cuda_stream) {
    if (!c || !d_frame_redundant) return SALICACHE_E_NULL;
    if (B < 0 || B > c->p.max_batch) return SALICACHE_E_SHAPE;
    return sc_frame_redundancy(c, d_deltaP, B, first_has_no_prev, d_frame_redundant, (cudaStream_t)cuda_stream);
}

int salicache_saliency(salicache_ctx* c, const uint8_t* d_frames, int B, float* d_s, const uint8_t* d_skip_or_null,
                       void* cuda_stream) {
    Range range__("salicache_saliency");
    if (!c || !d_frames || !d_s) return SALICACHE_E_NULL;
    if (B < 0 || B > c->p.max_batch) return SALICACHE_E_SHAPE;
    if (!aligned16(d_frames) || !aligned16(d_s)) return SALICACHE_E_ALIGN;
    if (B == 0) return SALICACHE_OK;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t fb = (size_t)c->p.H * c->p.W * 3;
    int rc = sc_saliency(c, c->plane[0], d_frames, fb, B, d_s, d_skip_or_null, st);
    if (rc != SALICACHE_OK || c->n_planes == 1) return rc;
    rc = sc_box_down2(d_frames, c->p.H, c->p.W, B, c->base_frames, st);
    c->launches++;
    if (rc != SALICACHE_OK) return rc;
    return sc_saliency(c, c->plane[1], c->base_frames, fb / 4, B, d_s, d_skip_or_null, st);
}

int salicache_select(salicache_ctx* c, const float* d_deltaP, const float* d_s, int B, int first_has_no_prev,
                     uint8_t* d_decision, int32_t* d_idx, int32_t* d_counts, uint8_t* d_frame_redundant,
                     int64_t* d_row_offset, int64_t* d_fill, void* cuda_stream) {
    Range range__("salicache_select");
    if (!c || !d_s || !d_decision || !d_idx || !d_counts || !d_frame_redundant || !d_row_offset || !d_fill)
        return SALICACHE_E_NULL;
    if (B < 0 || B > c->p.max_batch) return SALICACHE_E_SHAPE;
    return sc_select(c, d_deltaP, d_s, B, first_has_no_prev, d_decision, d_idx, d_counts, d_frame_redundant,
                     d_row_offset, d_fill, (cudaStream_t)cuda_stream);
}

int salicache_select_ranked(salicache_ctx* c, const float* d_deltaP, const float* d_s, int B, int first_has_no_prev,
                            int share_fp16_permille, int share_int8_permille, int share_int4_permille, uint8_t* d_decision,
                            int32_t* d_idx, int32_t* d_counts, uint8_t* d_frame_redundant, int64_t* d_row_offset,
                            int64_t* d_fill, void* cuda_stream) {
    Range range__("salicache_select_ranked");
    if (!c || !d_s || !d_decision || !d_idx || !d_counts || !d_frame_redundant || !d_row_offset || !d_fill)
        return SALICACHE_E_NULL;
    if (B < 0 || B > c->p.max_batch) return SALICACHE_E_SHAPE;
    if (share_fp16_permille < 0 || share_int8_permille < 0 || share_int4_permille < 0 || share_fp16_permille > 1000 ||
        share_int8_permille > 1000 || share_int4_permille > 1000)
        return SALICACHE_E_PARAM;
    return sc_select_ranked(c, d_deltaP, d_s, B, first_has_no_prev, share_fp16_permille, share_int8_permille,
                            share_int4_permille, d_decision, d_idx, d_counts, d_frame_redundant, d_row_offset, d_fill,
                            (cudaStream_t)cuda_stream);
}

int salicache_select_anchored(salicache_ctx* c, const uint8_t* d_frames, const float* d_s, int B, int first_has_no_prev,
                              uint8_t* d_anchor, float* d_deltaP, uint8_t* d_decision, int32_t* d_idx, int32_t* d_counts,
                              uint8_t* d_frame_redundant, int64_t* d_row_offset, int64_t* d_fill, void* cuda_stream) {
    Range range__("salicache_select_anchored");
    if (!c || !d_frames || !d_s || !d_anchor || !d_deltaP || !d_decision || !d_idx || !d_counts || !d_frame_redundant ||
        !d_row_offset || !d_fill)
        return SALICACHE_E_NULL;
    if (B < 0 || B > c->p.max_batch) return SALICACHE_E_SHAPE;
    if (!aligned16(d_frames) || !aligned16(d_anchor)) return SALICACHE_E_ALIGN;
    return sc_select_anchored(c, d_frames, d_s, 1, B, first_has_no_prev, d_anchor, d_deltaP, d_decision, d_idx, d_counts,
                              d_frame_redundant, d_row_offset, d_fill, (cudaStream_t)cuda_stream);
}

int salicache_select_anchored_batch(salicache_ctx* c, const uint8_t* d_frames, const float* d_s, int n_videos, int B,
                                    int first_has_no_prev, uint8_t* d_anchor, float* d_deltaP, uint8_t* d_decision,
                                    int32_t* d_idx, int32_t* d_counts, uint8_t* d_frame_redundant, int64_t* d_row_offset,
                                    int64_t* d_fill, void* cuda_stream) {
    if (!c || !d_frames || !d_s || !d_anchor || !d_deltaP || !d_decision || !d_idx || !d_counts || !d_frame_redundant ||
        !d_row_offset || !d_fill)
        return SALICACHE_E_NULL;
    if (B < 0 || B > c->p.max_batch || n_videos < 0 || n_videos > 4096) return SALICACHE_E_SHAPE;
    if (!aligned16(d_frames) || !aligned16(d_anchor)) return SALICACHE_E_ALIGN;
    return sc_select_anchored(c, d_frames, d_s, n_videos, B, first_has_no_prev, d_anchor, d_deltaP, d_decision, d_idx, d_counts,
                              d_frame_redundant, d_row_offset, d_fill, (cudaStream_t)cuda_stream);
}

int salicache_source_frames(salicache_ctx* c, const uint8_t* d_decision, int B, int first_frame, int32_t* d_carry,
                            int32_t* d_src, void* cuda_stream) {
    if (!c || !d_decision || !d_carry || !d_src) return SALICACHE_E_NULL;
    if (B < 0 || B > c->p.max_batch || first_frame < 0) return SALICACHE_E_SHAPE;
    return sc_sources(c, d_decision, B, first_frame, d_carry, d_src, (cudaStream_t)cuda_stream);
}

static int check_pools(const salicache_pools* p) {
    if (!p) return SALICACHE_E_NULL;
    if (p->cap_fp16 < 0 || p->cap_int8 < 0 || p->cap_int4 < 0) return SALICACHE_E_SHAPE;
    if ((p->cap_fp16 > 0 && !p->fp16_pool) || (p->cap_int8 > 0 && (!p->int8_codes || !p->int8_scale)) ||
        (p->cap_int4 > 0 && (!p->int4_codes || !p->int4_sz)))
        return SALICACHE_E_NULL;
    if (!aligned16(p->fp16_pool) || !aligned16(p->int8_codes) || !aligned16(p->int8_scale) ||
        !aligned16(p->int4_codes) || !aligned16(p->int4_sz))
        return SALICACHE_E_ALIGN;
    return SALICACHE_OK;
}

int salicache_pack_kv(salicache_ctx* c, const void* d_K, const void* d_V, int64_t frame_stride, const int32_t* d_idx,
                      const int32_t* d_counts, const int64_t* d_row_offset, int B, const salicache_pools* pools,
                      void* cuda_stream) {
    Range range__("salicache_pack_kv");
    if (!c || !d_K || !d_V || !d_idx || !d_counts || !d_row_offset) return SALICACHE_E_NULL;
    int rc = check_pools(pools);
    if (rc != SALICACHE_OK) return rc;
    if (B < 0 || B > c->p.max_batch) return SALICACHE_E_SHAPE;
    const int64_t dense = (int64_t)c->p.L * c->n_tok * c->p.heads * c->p.head_dim;
    if (frame_stride < 0 || (B > 1 && frame_stride < dense) || frame_stride % 8 != 0) return SALICACHE_E_SHAPE;
    if (!aligned16(d_K) || !aligned16(d_V)) return SALICACHE_E_ALIGN;
    return sc_pack(c, d_K, d_V, frame_stride, d_idx, d_counts, d_row_offset, B, pools, (cudaStream_t)cuda_stream);
}

int salicache_unpack_kv(salicache_ctx* c, const salicache_pools* pools, const int32_t* d_idx, const int32_t* d_counts,
                        const uint8_t* d_decision, const int64_t* d_row_offset, int B, int zero_fill_pruned,
                        void* d_K_out, void* d_V_out, int64_t frame_stride, void* cuda_stream) {
    Range range__("salicache_unpack_kv");
    if (!c || !d_K_out || !d_V_out || !d_idx || !d_counts || !d_row_offset) return SALICACHE_E_NULL;
    if (zero_fill_pruned && !d_decision) return SALICACHE_E_NULL;
    int rc = check_pools(pools);
    if (rc != SALICACHE_OK) return rc;
    if (B < 0 || B > c->p.max_batch) return SALICACHE_E_SHAPE;
    const int64_t dense = (int64_t)c->p.L * c->n_tok * c->p.heads * c->p.head_dim;
    if (frame_stride < 0 || (B > 1 && frame_stride < dense) || frame_stride % 8 != 0) return SALICACHE_E_SHAPE;
    if (!aligned16(d_K_out) || !aligned16(d_V_out)) return SALICACHE_E_ALIGN;
    return sc_unpack(c, pools, d_idx, d_counts, d_decision, d_row_offset, B, zero_fill_pruned, d_K_out, d_V_out,
                     frame_stride, (cudaStream_t)cuda_stream);
}

int salicache_frames_resident(salicache_ctx* c, const int32_t* d_counts, const int64_t* d_row_offset, int B,
                              const salicache_pools* pools, uint8_t* d_resident, void* cuda_stream) {
    if (!c || !d_counts || !d_row_offset || !d_resident || !pools) return SALICACHE_E_NULL;
    if (pools->ring && !pools->d_fill) return SALICACHE_E_NULL;
    if (pools->cap_fp16 < 0 || pools->cap_int8 < 0 || pools->cap_int4 < 0 || B < 0) return SALICACHE_E_SHAPE;
    return sc_frames_resident(c, d_counts, d_row_offset, B, pools, d_resident, (cudaStream_t)cuda_stream);
}

int salicache_tokens_live(salicache_ctx* c, const int32_t* d_src, int B, int first_frame, const uint8_t* d_resident_table,
                          int n_table, uint8_t* d_live, void* cuda_stream) {
    if (!c || !d_src || !d_resident_table || !d_live) return SALICACHE_E_NULL;
    if (B < 0 || n_table < 0 || first_frame < 0) return SALICACHE_E_SHAPE;
    return sc_tokens_live(c, d_src, B, first_frame, d_resident_table, n_table, d_live, (cudaStream_t)cuda_stream);
}

int salicache_attend(salicache_ctx* c, const void* d_q, const salicache_pools* pools, const int64_t* d_fill, float* d_out,
                     void* cuda_stream) {
    Range range__("salicache_attend");
    if (!c || !d_q || !d_fill || !d_out) return SALICACHE_E_NULL;
    int rc = check_pools(pools);
    if (rc != SALICACHE_OK) return rc;
    if (!aligned16(d_q) || !aligned16(d_out)) return SALICACHE_E_ALIGN;
    return sc_attend(c, d_q, 1, pools, d_fill, d_out, (cudaStream_t)cuda_stream);
}

int salicache_attend_gqa(salicache_ctx* c, const void* d_q, int q_per_kv, const salicache_pools* pools, const int64_t* d_fill,
                         float* d_out, void* cuda_stream) {
    Range range__("salicache_attend_gqa");
    if (!c || !d_q || !d_fill || !d_out) return SALICACHE_E_NULL;
    int rc = check_pools(pools);
    if (rc != SALICACHE_OK) return rc;
    if (!aligned16(d_q) || !aligned16(d_out)) return SALICACHE_E_ALIGN;
    return sc_attend(c, d_q, q_per_kv, pools, d_fill, d_out, (cudaStream_t)cuda_stream);
}

int salicache_poll_status(salicache_ctx* c, void* cuda_stream) {
    if (!c) return SALICACHE_E_NULL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int h = 0;
    if (cudaMemcpyAsync(&h, c->d_status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SALICACHE_E_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SALICACHE_E_CUDA;
    if (h != 0 && cudaMemsetAsync(c->d_status, 0, sizeof(int), st) != cudaSuccess) return SALICACHE_E_CUDA;
    return h;
}

}  // extern "C"
