// Declarations shared by the translation units of libavggt (not part of the ABI).
#pragma once

#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

#include "plan.h"

namespace avggt {

// ---- shared host helpers (api.cu)
struct DeviceInfo { int sm_count; int cc_major; };
// Properties of the current device.  AVGGT_OK only on an sm_100 device.
int device_info(DeviceInfo* out);
// Map a CUDA error to an AVGGT_* code, keeping its text for avggt_last_cuda_error.
int record_cuda(cudaError_t e);
// Keep `text` for avggt_last_cuda_error; returns AVGGT_ERR_CUDA.
int record_message(const char* text);

// ---- K/V compaction (build_kv.cu)
int build_kv_grid(const Plan& pl, int sm_count);
size_t build_kv_ws_bytes(const Plan& pl, int sm_count);
// caller_idx / slot_of_token: both null for the window rule of Sec. 4.3; for a caller-chosen retained set,
// the M retained token indices (device) and the [n_tok] map the call fills (device).
// kc_rows: rows per head of Kc / Vc (0 = M; larger when they are one rank's slot of an exchange buffer).
// sums_only: kmean / vmean receive the un-normalised sums over the dropped rows instead of the means.
cudaError_t launch_build_kv(const Plan& pl, int sm_count, const void* K, const void* V, void* Kc, void* Vc,
                            int32_t* idx, float* kmean, float* vmean, void* ws, cudaStream_t st,
                            const int32_t* caller_idx = nullptr, int32_t* slot_of_token = nullptr,
                            int64_t kc_rows = 0, bool sums_only = false);

// Frame-sharded layer: the ranks' slots of the exchange buffer -> one compact K/V pair, and the mean
// pair from the all-reduced sums.
constexpr int kMaxShardRanks = 64;
cudaError_t launch_assemble_shards(const void* gathered, int n_ranks, const int64_t* kept, int H, int d, int64_t slot_rows,
                                   void* Kc, void* Vc, const float* sums, int64_t n_dropped_total, float* kmean,
                                   float* vmean, cudaStream_t st);

// ---- attention (global_attn.cu)
constexpr size_t kAttnStatusBytes = 256;   // status block at the start of the attention workspace
size_t global_attn_ws_bytes(const Plan& pl, int sm_count);
// Returns cudaSuccess, or an error; *tmap_failed is set when a tensor map could not be encoded.
// slot_of_token: null for the window rule; else the map written by the indexed compaction.
cudaError_t launch_global_attn(const Plan& pl, int sm_count, const void* Q, const void* K, const void* V,
                               const void* Kc, const void* Vc, const float* kmean, const float* vmean, void* O,
                               float* lse, void* ws, cudaStream_t st, bool* tmap_failed,
                               const int32_t* slot_of_token = nullptr);

// Frame attention (Sec. 4.2): the same kernel, one independent dense problem per frame.
cudaError_t launch_frame_attn(const Plan& pl, int sm_count, const void* Q, const void* K, const void* V, void* O, float* lse,
                              void* ws, cudaStream_t st, bool* tmap_failed);

// ---- K/V projection with the compaction in its epilogue (project_kv.cu)
size_t project_kv_ws_bytes(const Plan& pl, int sm_count);
// X [n_tok, model_dim], Wk / Wv [H * d, model_dim] (the layout of a linear layer's weight), bias_k / bias_v [H * d] or
// null; K / V [n_tok, H, d] or null (written when given); the other outputs as for launch_build_kv.
cudaError_t launch_project_kv(const Plan& pl, int sm_count, int model_dim, const void* X, const void* Wk, const void* Wv,
                              const float* bias_k, const float* bias_v, void* K, void* V, void* Kc, void* Vc, int32_t* idx,
                              float* kmean, float* vmean, void* ws, cudaStream_t st, bool* tmap_failed);

}  // namespace avggt
