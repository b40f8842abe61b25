// Internal declarations shared by the translation units of libsalicache.so (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "salicache.h"

#define SC_CHECK(call)                                   \
    do {                                                 \
        cudaError_t e__ = (call);                        \
        if (e__ != cudaSuccess) return SALICACHE_E_CUDA; \
    } while (0)

// One image plane the pixel stages run on: the frame itself, or the anyres base image.
struct PlaneGeom {
    int H, W;        // pixels
    int gh, gw;      // patch grid
    int layout;      // 0: token = tok_base + py*gw + px ; 1: anyres tiles of 24x24 patches after the base image
    int tok_base;    // first token of this plane
    int n_tok;       // tokens per frame (row stride of the score arrays)
};

// Token id of patch (py, px) of a plane.
__host__ __device__ inline int patch_token(const PlaneGeom& g, int py, int px) {
    if (g.layout == 0) return g.tok_base + py * g.gw + px;
    const int tg = 24;                              // patches per tile side (336 / 14)
    int r = py / tg, c = px / tg;
    return g.tok_base + (r * (g.gw / tg) + c) * tg * tg + (py % tg) * tg + (px % tg);
}

struct salicache_ctx {
    salicache_params p;
    int n_tok;
    int chunk;                 // frames per internal pass
    int n_planes;              // 1, or 2 for anyres (full frame + base image)
    PlaneGeom plane[2];
    // flow scratch (sized for the largest plane)
    float* pyr[3];             // [chunk+1][h_l*w_l]
    float* coef[3];            // expansion coefficients: float4 [2*chunk][h_l*w_l] + pad, then float [2*chunk][h_l*w_l] + pad
    float* gh_a;               // [chunk][5][H*W] normal-equation terms of the current update
    float* flow_a;             // [chunk][H*W] (du, dv) records: the field of the level at work and of the coarser one
    float* flow_b;
    // saliency scratch
    uint32_t* bits_kept;       // [chunk][H][Ww]  NMS-kept weak or strong pixels
    uint32_t* bits_edge;       // [chunk][H][Ww]  strong pixels, grown to the edge map E
    double* lut;               // 256 entries sRGB -> linear
    float* sqrt_v;             // frame-adaptive colour term only: [chunk][H*W] local contrast sqrt(V)
    double* v_part;            //                                  [chunk][tiles] per-tile sums of V
    uint8_t* base_frames;      // anyres only: [chunk+1][336*336*3]
    // select / pack scratch
    int64_t* row_prefix;       // [max_batch+1] stored rows before each frame of the batch
    float* attend_ws;          // partial attention results [L][max(heads, 64)][128][head_dim + 2]
    int* d_status;             // deferred status word
    int sm_count;
    long long launches;        // kernels launched through this context so far
};

// flow.cu
int sc_flow_score(salicache_ctx* c, const PlaneGeom& g, const uint8_t* d_prev, const uint8_t* d_cur, size_t frame_bytes,
                  int B, bool sequence, float* d_deltaP, double* d_flow_or_null, cudaStream_t st);
int sc_diff_score(salicache_ctx* c, const PlaneGeom& g, const uint8_t* d_prev, const uint8_t* d_cur, size_t frame_bytes,
                  int B, float* d_deltaP, cudaStream_t st);
// saliency.cu
int sc_saliency(salicache_ctx* c, const PlaneGeom& g, const uint8_t* d_frames, size_t frame_bytes, int B, float* d_s,
                const uint8_t* d_skip, cudaStream_t st);
int sc_box_down2(const uint8_t* d_src, int H, int W, int B, uint8_t* d_dst, cudaStream_t st);
// select.cu
int sc_select(salicache_ctx* c, const float* d_deltaP, const float* d_s, int B, int first_has_no_prev,
              uint8_t* d_decision, int32_t* d_idx, int32_t* d_counts, uint8_t* d_frame_redundant,
              int64_t* d_row_offset, int64_t* d_fill, cudaStream_t st);
int sc_sources(salicache_ctx* c, const uint8_t* d_decision, int B, int first_frame, int32_t* d_carry, int32_t* d_src,
               cudaStream_t st);
int sc_frame_redundancy(salicache_ctx* c, const float* d_deltaP, int B, int first_has_no_prev, uint8_t* d_frame_redundant,
                        cudaStream_t st);
int sc_frames_resident(salicache_ctx* c, const int32_t* d_counts, const int64_t* d_row_offset, int B,
                       const salicache_pools* pools, uint8_t* d_resident, cudaStream_t st);
int sc_tokens_live(salicache_ctx* c, const int32_t* d_src, int B, int first_frame, const uint8_t* d_table, int n_table,
                   uint8_t* d_live, cudaStream_t st);
// ranked.cu
int sc_select_ranked(salicache_ctx* c, const float* d_deltaP, const float* d_s, int B, int first_has_no_prev, int pm16,
                     int pm8, int pm4, uint8_t* d_decision, int32_t* d_idx, int32_t* d_counts, uint8_t* d_frame_redundant,
                     int64_t* d_row_offset, int64_t* d_fill, cudaStream_t st);
// anchor.cu
int sc_select_anchored(salicache_ctx* c, const uint8_t* d_frames, const float* d_s, int n_videos, int B, int first_has_no_prev,
                       uint8_t* d_anchor, float* d_deltaP, uint8_t* d_decision, int32_t* d_idx, int32_t* d_counts,
                       uint8_t* d_frame_redundant, int64_t* d_row_offset, int64_t* d_fill, cudaStream_t st);
// attend.cu
size_t sc_attend_workspace_bytes(int L, int H);
int sc_attend(salicache_ctx* c, const void* d_q, int q_per_kv, const salicache_pools* pools, const int64_t* d_fill, float* d_out,
              cudaStream_t st);
// kv.cu
int sc_pack(salicache_ctx* c, const void* d_K, const void* d_V, int64_t frame_stride, const int32_t* d_idx,
            const int32_t* d_counts, const int64_t* d_row_offset, int B, const salicache_pools* pools, cudaStream_t st);
int sc_unpack(salicache_ctx* c, const salicache_pools* pools, const int32_t* d_idx, const int32_t* d_counts,
              const uint8_t* d_decision, const int64_t* d_row_offset, int B, int zero_fill_pruned, void* d_K_out,
              void* d_V_out, int64_t frame_stride, cudaStream_t st);
