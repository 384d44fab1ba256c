// Declarations shared by the translation units of libavggt (not part of the ABI).
#pragma once

#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

#include "plan.h"

namespace avggt {

// ---- K/V compaction (build_kv.cu)
int build_kv_grid(const Plan& pl, int sm_count);
size_t build_kv_ws_bytes(const Plan& pl, int sm_count);
// caller_idx / slot_of_token: both null for the window rule of Sec. 4.3; for a caller-chosen retained set,
// the M retained token indices (device) and the [n_tok] map the call fills (device).
cudaError_t launch_build_kv(const Plan& pl, int sm_count, const void* K, const void* V, void* Kc, void* Vc,
                            int32_t* idx, float* kmean, float* vmean, void* ws, cudaStream_t st,
                            const int32_t* caller_idx = nullptr, int32_t* slot_of_token = nullptr);

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
cudaError_t launch_frame_attn(const Plan& pl, const void* Q, const void* K, const void* V, void* O, float* lse, void* ws,
                              cudaStream_t st, bool* tmap_failed);

}  // namespace avggt
