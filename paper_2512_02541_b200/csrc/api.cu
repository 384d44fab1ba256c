// C ABI of libavggt: argument validation, the problem plan, and the launchers'
// entry points.  Nothing here touches the data; every step of the path runs in
// the kernels of build_kv.cu and global_attn.cu.
#include <cmath>
#include <cstring>
#include <mutex>

#include "internal.h"

namespace avggt {

namespace {

thread_local char g_cuda_error[256] = "";

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

// Properties of the current device (queried once per device index).
int device_info(DeviceInfo* out) {
  static std::mutex mu;
  static DeviceInfo cache[64];
  static bool have[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return record_cuda(e);
  std::lock_guard<std::mutex> lock(mu);
  if (dev < 0 || dev >= 64) return AVGGT_ERR_UNSUPPORTED;
  if (!have[dev]) {
    DeviceInfo di;
    e = cudaDeviceGetAttribute(&di.sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return record_cuda(e);
    e = cudaDeviceGetAttribute(&di.cc_major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return record_cuda(e);
    cache[dev] = di;
    have[dev] = true;
  }
  *out = cache[dev];
  return out->cc_major == 10 ? AVGGT_OK : AVGGT_ERR_UNSUPPORTED;
}

int record_message(const char* text) {
  std::strncpy(g_cuda_error, text, sizeof(g_cuda_error) - 1);
  g_cuda_error[sizeof(g_cuda_error) - 1] = 0;
  return AVGGT_ERR_CUDA;
}

int record_cuda(cudaError_t e) {
  if (e == cudaSuccess) return AVGGT_OK;
  (void)cudaGetLastError();   // clear the non-sticky error state
  return record_message(cudaGetErrorString(e));
}

int make_plan(const avggt_params* p, Plan* pl) {
  if (p == nullptr || pl == nullptr) return AVGGT_ERR_INVALID_ARG;
  if (p->n_frames < 1 || p->grid_h < 1 || p->grid_w < 1 || p->n_special < 0 || p->n_heads < 1 || p->head_dim < 1)
    return AVGGT_ERR_INVALID_ARG;
  if (p->diag != 0 && p->diag != 1) return AVGGT_ERR_INVALID_ARG;
  if (p->mean_fill < AVGGT_MEAN_OFF || p->mean_fill > AVGGT_MEAN_FILL) return AVGGT_ERR_INVALID_ARG;
  if (p->flags & ~AVGGT_FLAG_KEEP_FIRST_FRAME) return AVGGT_ERR_INVALID_ARG;
  if (!(p->softmax_scale == p->softmax_scale) || std::isinf(p->softmax_scale)) return AVGGT_ERR_INVALID_ARG;
  const int64_t patches = static_cast<int64_t>(p->grid_h) * p->grid_w;
  if (patches + p->n_special != p->tokens_per_frame) return AVGGT_ERR_INVALID_ARG;
  if (p->batch != 1) return AVGGT_ERR_UNSUPPORTED;
  if (p->head_dim != 64) return AVGGT_ERR_UNSUPPORTED;
  if (p->n_heads > 32) return AVGGT_ERR_UNSUPPORTED;
  int s_h, s_w;
  switch (p->sigma) {   // Sec. 4.3, Subsampling Strategy
    case 1: s_h = 1; s_w = 1; break;
    case 2: s_h = 1; s_w = 2; break;
    case 4: s_h = 2; s_w = 2; break;
    case 6: s_h = 2; s_w = 3; break;
    case 9: s_h = 3; s_w = 3; break;
    default: return AVGGT_ERR_UNSUPPORTED;
  }
  const int64_t n_tok = static_cast<int64_t>(p->n_frames) * p->tokens_per_frame;
  if (n_tok > 0x7fffffffll - 256) return AVGGT_ERR_UNSUPPORTED;
  pl->n_frames = p->n_frames;
  pl->L = p->tokens_per_frame;
  pl->grid_h = p->grid_h;
  pl->grid_w = p->grid_w;
  pl->n_special = p->n_special;
  pl->H = p->n_heads;
  pl->d = p->head_dim;
  pl->s_h = s_h;
  pl->s_w = s_w;
  pl->kept_w = (p->grid_w + s_w - 1) / s_w;
  pl->kept_patches = ((p->grid_h + s_h - 1) / s_h) * pl->kept_w;
  pl->Lc = p->n_special + pl->kept_patches;
  pl->keep_first = (p->flags & AVGGT_FLAG_KEEP_FIRST_FRAME) ? 1 : 0;
  pl->diag = p->diag;
  pl->mean_fill = p->mean_fill;
  pl->n_tok = n_tok;
  pl->M = static_cast<int64_t>(p->n_frames) * pl->Lc + (pl->keep_first ? (patches - pl->kept_patches) : 0);
  pl->n_dropped = n_tok - pl->M;
  pl->scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / std::sqrt(static_cast<float>(p->head_dim));
  if (pl->M < 1) return AVGGT_ERR_INVALID_ARG;
  return AVGGT_OK;
}

}  // namespace avggt

using namespace avggt;

extern "C" {

int avggt_kv_count(const avggt_params* p, int64_t* n_kept, int64_t* n_dropped) {
  Plan pl;
  int rc = make_plan(p, &pl);
  if (rc != AVGGT_OK) return rc;
  if (n_kept) *n_kept = pl.M;
  if (n_dropped) *n_dropped = pl.n_dropped;
  return AVGGT_OK;
}

int avggt_workspace_bytes(const avggt_params* p, size_t* build_ws_bytes, size_t* attn_ws_bytes) {
  Plan pl;
  int rc = make_plan(p, &pl);
  if (rc != AVGGT_OK) return rc;
  DeviceInfo di;
  rc = device_info(&di);
  if (rc != AVGGT_OK) return rc;
  if (build_ws_bytes) *build_ws_bytes = build_kv_ws_bytes(pl, di.sm_count);
  if (attn_ws_bytes) *attn_ws_bytes = global_attn_ws_bytes(pl, di.sm_count);
  return AVGGT_OK;
}

int avggt_build_kv(const avggt_params* p, const void* K, const void* V, void* Kc, void* Vc, int32_t* idx,
                   float* kmean, float* vmean, void* ws, size_t ws_bytes, void* cuda_stream) {
  Plan pl;
  int rc = make_plan(p, &pl);
  if (rc != AVGGT_OK) return rc;
  if (!K || !V || !Kc || !Vc || !ws) return AVGGT_ERR_INVALID_ARG;
  if (pl.mean_fill != 0 && (!kmean || !vmean)) return AVGGT_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(Kc) || !aligned16(Vc) || !aligned16(ws) ||
      (reinterpret_cast<uintptr_t>(idx) & 3u) || !aligned16(kmean) || !aligned16(vmean))
    return AVGGT_ERR_ALIGNMENT;
  DeviceInfo di;
  rc = device_info(&di);
  if (rc != AVGGT_OK) return rc;
  if (ws_bytes < build_kv_ws_bytes(pl, di.sm_count)) return AVGGT_ERR_WORKSPACE_TOO_SMALL;
  return record_cuda(launch_build_kv(pl, di.sm_count, K, V, Kc, Vc, idx, kmean, vmean, ws, static_cast<cudaStream_t>(cuda_stream)));
}

// One attention call: which buffers, on which stream.
struct AttnCall {
  const void *Q, *K, *V, *Kc, *Vc;
  const float *kmean, *vmean;
  void* O;
  float* lse;
  void* ws;
  size_t ws_bytes;
  void* stream;
  const int32_t* slot_of_token;   // caller-chosen retained set, else null
  bool frame_mode;                // frame attention (Sec. 4.2): Kc, Vc, kmean, vmean play no part
};

// Validation and launch shared by every attention entry point.  Everything that can be rejected on the
// host is rejected before anything is enqueued.
static int run_attn(const Plan& pl, const AttnCall& c) {
  const bool need_diag = !c.frame_mode && pl.diag != 0 && pl.n_dropped > 0;
  const bool need_mean = !c.frame_mode && pl.mean_fill != 0 && pl.n_dropped > 0;
  if (!c.Q || !c.O || !c.ws) return AVGGT_ERR_INVALID_ARG;
  if (c.frame_mode ? (!c.K || !c.V) : (pl.M > 0 && (!c.Kc || !c.Vc))) return AVGGT_ERR_INVALID_ARG;
  if (need_diag && (!c.K || !c.V)) return AVGGT_ERR_INVALID_ARG;
  if (need_mean && (!c.kmean || !c.vmean)) return AVGGT_ERR_INVALID_ARG;
  if (!aligned16(c.Q) || !aligned16(c.K) || !aligned16(c.V) || !aligned16(c.Kc) || !aligned16(c.Vc) || !aligned16(c.O) ||
      !aligned16(c.ws) || !aligned16(c.kmean) || !aligned16(c.vmean) || (reinterpret_cast<uintptr_t>(c.lse) & 3u) ||
      (reinterpret_cast<uintptr_t>(c.slot_of_token) & 3u))
    return AVGGT_ERR_ALIGNMENT;
  DeviceInfo di;
  int rc = device_info(&di);
  if (rc != AVGGT_OK) return rc;
  if (c.ws_bytes < global_attn_ws_bytes(pl, di.sm_count)) return AVGGT_ERR_WORKSPACE_TOO_SMALL;
  bool tmap_failed = false;
  const cudaStream_t st = static_cast<cudaStream_t>(c.stream);
  const cudaError_t e = c.frame_mode
      ? launch_frame_attn(pl, di.sm_count, c.Q, c.K, c.V, c.O, c.lse, c.ws, st, &tmap_failed)
      : launch_global_attn(pl, di.sm_count, c.Q, c.K, c.V, c.Kc, c.Vc, c.kmean, c.vmean, c.O, c.lse, c.ws, st,
                           &tmap_failed, c.slot_of_token);
  if (tmap_failed) return record_message("cuTensorMapEncodeTiled failed");
  return record_cuda(e);
}

int avggt_global_attn(const avggt_params* p, const void* Q, const void* K, const void* V, const void* Kc,
                      const void* Vc, const float* kmean, const float* vmean, void* O, float* lse, void* ws,
                      size_t ws_bytes, void* cuda_stream) {
  Plan pl;
  int rc = make_plan(p, &pl);
  if (rc != AVGGT_OK) return rc;
  return run_attn(pl, AttnCall{Q, K, V, Kc, Vc, kmean, vmean, O, lse, ws, ws_bytes, cuda_stream, nullptr, false});
}

// Plan of a problem whose retained set is a caller-supplied list of n_kept tokens.
static int make_indexed_plan(const avggt_params* p, int64_t n_kept, Plan* pl) {
  int rc = make_plan(p, pl);
  if (rc != AVGGT_OK) return rc;
  if (n_kept < 0 || n_kept > pl->n_tok) return AVGGT_ERR_INVALID_ARG;
  // nothing retained (the G2M variant of Sec. 5.4): some column must remain for the softmax
  if (n_kept == 0 && pl->diag == 0 && pl->mean_fill == 0) return AVGGT_ERR_INVALID_ARG;
  pl->M = n_kept;
  pl->n_dropped = pl->n_tok - n_kept;
  pl->keep_first = 0;
  return AVGGT_OK;
}

int avggt_build_kv_indexed(const avggt_params* p, const int32_t* idx, int64_t n_kept, const void* K, const void* V,
                           void* Kc, void* Vc, int32_t* slot_of_token, float* kmean, float* vmean, void* ws,
                           size_t ws_bytes, void* cuda_stream) {
  Plan pl;
  int rc = make_indexed_plan(p, n_kept, &pl);
  if (rc != AVGGT_OK) return rc;
  if (!slot_of_token || !K || !V || !ws) return AVGGT_ERR_INVALID_ARG;
  if (n_kept > 0 && (!idx || !Kc || !Vc)) return AVGGT_ERR_INVALID_ARG;
  if (pl.mean_fill != 0 && (!kmean || !vmean)) return AVGGT_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(Kc) || !aligned16(Vc) || !aligned16(ws) ||
      (reinterpret_cast<uintptr_t>(idx) & 3u) || (reinterpret_cast<uintptr_t>(slot_of_token) & 3u) ||
      !aligned16(kmean) || !aligned16(vmean))
    return AVGGT_ERR_ALIGNMENT;
  DeviceInfo di;
  rc = device_info(&di);
  if (rc != AVGGT_OK) return rc;
  if (ws_bytes < build_kv_ws_bytes(pl, di.sm_count)) return AVGGT_ERR_WORKSPACE_TOO_SMALL;
  return record_cuda(launch_build_kv(pl, di.sm_count, K, V, Kc, Vc, nullptr, kmean, vmean, ws,
                                     static_cast<cudaStream_t>(cuda_stream), idx, slot_of_token));
}

int avggt_global_attn_indexed(const avggt_params* p, int64_t n_kept, const int32_t* slot_of_token, const void* Q,
                              const void* K, const void* V, const void* Kc, const void* Vc, const float* kmean,
                              const float* vmean, void* O, float* lse, void* ws, size_t ws_bytes, void* cuda_stream) {
  Plan pl;
  int rc = make_indexed_plan(p, n_kept, &pl);
  if (rc != AVGGT_OK) return rc;
  if (!slot_of_token) return AVGGT_ERR_INVALID_ARG;
  return run_attn(pl, AttnCall{Q, K, V, Kc, Vc, kmean, vmean, O, lse, ws, ws_bytes, cuda_stream, slot_of_token, false});
}

int avggt_global_attn_shard(const avggt_params* p, int64_t n_kept_total, int64_t n_dropped_total, const void* Q,
                            const void* K, const void* V, const void* Kc, const void* Vc, const float* kmean,
                            const float* vmean, void* O, float* lse, void* ws, size_t ws_bytes, void* cuda_stream) {
  Plan pl;
  int rc = make_plan(p, &pl);
  if (rc != AVGGT_OK) return rc;
  // the shard's own frames cannot hold more retained or dropped tokens than the whole sequence
  if (n_kept_total < pl.M || n_dropped_total < pl.n_dropped) return AVGGT_ERR_INVALID_ARG;
  pl.M = n_kept_total;
  pl.n_dropped = n_dropped_total;
  return run_attn(pl, AttnCall{Q, K, V, Kc, Vc, kmean, vmean, O, lse, ws, ws_bytes, cuda_stream, nullptr, false});
}

int avggt_project_workspace_bytes(const avggt_params* p, int32_t model_dim, size_t* ws_bytes) {
  Plan pl;
  int rc = make_plan(p, &pl);
  if (rc != AVGGT_OK) return rc;
  if (model_dim < 64 || model_dim % 64 != 0) return AVGGT_ERR_UNSUPPORTED;
  DeviceInfo di;
  rc = device_info(&di);
  if (rc != AVGGT_OK) return rc;
  if (ws_bytes) *ws_bytes = project_kv_ws_bytes(pl, di.sm_count);
  return AVGGT_OK;
}

int avggt_project_build_kv(const avggt_params* p, int32_t model_dim, const void* X, const void* Wk, const void* Wv,
                           const float* bias_k, const float* bias_v, void* K, void* V, void* Kc, void* Vc, int32_t* idx,
                           float* kmean, float* vmean, void* ws, size_t ws_bytes, void* cuda_stream) {
  Plan pl;
  int rc = make_plan(p, &pl);
  if (rc != AVGGT_OK) return rc;
  if (model_dim < 64 || model_dim % 64 != 0) return AVGGT_ERR_UNSUPPORTED;
  if (!X || !Wk || !Wv || !Kc || !Vc || !ws) return AVGGT_ERR_INVALID_ARG;
  if ((K == nullptr) != (V == nullptr)) return AVGGT_ERR_INVALID_ARG;
  if (pl.mean_fill != 0 && (!kmean || !vmean)) return AVGGT_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(Wk) || !aligned16(Wv) || !aligned16(K) || !aligned16(V) || !aligned16(Kc) ||
      !aligned16(Vc) || !aligned16(ws) || (reinterpret_cast<uintptr_t>(idx) & 3u) || !aligned16(kmean) ||
      !aligned16(vmean) || (reinterpret_cast<uintptr_t>(bias_k) & 3u) || (reinterpret_cast<uintptr_t>(bias_v) & 3u))
    return AVGGT_ERR_ALIGNMENT;
  DeviceInfo di;
  rc = device_info(&di);
  if (rc != AVGGT_OK) return rc;
  if (ws_bytes < project_kv_ws_bytes(pl, di.sm_count)) return AVGGT_ERR_WORKSPACE_TOO_SMALL;
  bool tmap_failed = false;
  const cudaError_t e = launch_project_kv(pl, di.sm_count, model_dim, X, Wk, Wv, bias_k, bias_v, K, V, Kc, Vc, idx, kmean,
                                          vmean, ws, static_cast<cudaStream_t>(cuda_stream), &tmap_failed);
  if (tmap_failed) return record_message("cuTensorMapEncodeTiled failed");
  return record_cuda(e);
}

int avggt_build_kv_shard(const avggt_params* p, const void* K, const void* V, void* slot, int64_t slot_rows,
                         int32_t* idx, float* sums, void* ws, size_t ws_bytes, void* cuda_stream) {
  Plan pl;
  int rc = make_plan(p, &pl);
  if (rc != AVGGT_OK) return rc;
  if (!K || !V || !slot || !ws) return AVGGT_ERR_INVALID_ARG;
  if (slot_rows < pl.M) return AVGGT_ERR_INVALID_ARG;
  if (pl.mean_fill != 0 && !sums) return AVGGT_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(slot) || !aligned16(ws) || (reinterpret_cast<uintptr_t>(idx) & 3u) ||
      !aligned16(sums))
    return AVGGT_ERR_ALIGNMENT;
  DeviceInfo di;
  rc = device_info(&di);
  if (rc != AVGGT_OK) return rc;
  if (ws_bytes < build_kv_ws_bytes(pl, di.sm_count)) return AVGGT_ERR_WORKSPACE_TOO_SMALL;
  const size_t part = static_cast<size_t>(pl.H) * static_cast<size_t>(slot_rows) * pl.d;   // elements of the K part of a slot
  void* Vc = static_cast<char*>(slot) + part * 2;
  float* vsum = sums ? sums + static_cast<size_t>(pl.H) * pl.d : nullptr;
  return record_cuda(launch_build_kv(pl, di.sm_count, K, V, slot, Vc, idx, sums, vsum, ws,
                                     static_cast<cudaStream_t>(cuda_stream), nullptr, nullptr, slot_rows, true));
}

int avggt_shard_assemble(const avggt_params* p, const void* gathered, int32_t n_ranks, const int64_t* kept,
                         int64_t slot_rows, const float* sums, int64_t n_dropped_total, void* Kc, void* Vc,
                         float* kmean, float* vmean, void* cuda_stream) {
  Plan pl;
  int rc = make_plan(p, &pl);
  if (rc != AVGGT_OK) return rc;
  if (!gathered || !kept || !Kc || !Vc || n_ranks < 1 || n_ranks > kMaxShardRanks || n_dropped_total < 0)
    return AVGGT_ERR_INVALID_ARG;
  for (int r = 0; r < n_ranks; ++r)
    if (kept[r] < 0 || kept[r] > slot_rows) return AVGGT_ERR_INVALID_ARG;
  const bool need_mean = pl.mean_fill != 0 && n_dropped_total > 0;
  if (need_mean && (!sums || !kmean || !vmean)) return AVGGT_ERR_INVALID_ARG;
  if (!aligned16(gathered) || !aligned16(Kc) || !aligned16(Vc) || !aligned16(sums) || !aligned16(kmean) || !aligned16(vmean))
    return AVGGT_ERR_ALIGNMENT;
  DeviceInfo di;
  rc = device_info(&di);
  if (rc != AVGGT_OK) return rc;
  return record_cuda(launch_assemble_shards(gathered, n_ranks, kept, pl.H, pl.d, slot_rows, Kc, Vc, need_mean ? sums : nullptr,
                                            n_dropped_total, kmean, vmean, static_cast<cudaStream_t>(cuda_stream)));
}

int avggt_frame_attn(const avggt_params* p, const void* Q, const void* K, const void* V, void* O, float* lse, void* ws,
                     size_t ws_bytes, void* cuda_stream) {
  Plan pl;
  int rc = make_plan(p, &pl);
  if (rc != AVGGT_OK) return rc;
  // one work item per pair of 128-row query tiles, head and frame; their number is a 32-bit count in the kernel
  if ((static_cast<int64_t>(pl.L) + 255) / 256 * pl.H * pl.n_frames > 2147483647LL) return AVGGT_ERR_UNSUPPORTED;
  return run_attn(pl, AttnCall{Q, K, V, nullptr, nullptr, nullptr, nullptr, O, lse, ws, ws_bytes, cuda_stream, nullptr, true});
}

int avggt_check_status(const void* attn_ws, uint32_t* detail) {
  if (!attn_ws) return AVGGT_ERR_INVALID_ARG;
  uint32_t st[4] = {0, 0, 0, 0};
  cudaError_t e = cudaMemcpy(st, attn_ws, sizeof(st), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return record_cuda(e);
  if (detail) std::memcpy(detail, st, sizeof(st));
  return st[0] == 0 ? AVGGT_OK : AVGGT_ERR_DEVICE_TIMEOUT;
}

const char* avggt_strerror(int code) {
  switch (code) {
    case AVGGT_OK: return "success";
    case AVGGT_ERR_INVALID_ARG: return "invalid argument";
    case AVGGT_ERR_UNSUPPORTED: return "unsupported configuration or device";
    case AVGGT_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case AVGGT_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
    case AVGGT_ERR_CUDA: return "CUDA call failed";
    case AVGGT_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    case AVGGT_ERR_STATIC_SCRATCH: return "problem exceeds the fixed scratch of avggt_build_kv_noalloc (n_heads * head_dim <= 1024)";
    default: return "unknown error code";
  }
}

const char* avggt_last_cuda_error(void) { return g_cuda_error; }

const char* avggt_version(void) { return "0.1.0"; }

}  // extern "C"
