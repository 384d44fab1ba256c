// Host-side problem plan: everything derived from avggt_params that the
// launchers and kernels need (Sec. 4.1 notation, Sec. 4.3 subsampling rule).
#pragma once

#include <cstdint>

#include "../../include/avggt.h"

namespace avggt {

// Plain data handed to the kernels by value.
struct Plan {
  int32_t n_frames;     // N
  int32_t L;            // tokens per frame
  int32_t grid_h, grid_w;
  int32_t n_special;
  int32_t H, d;
  int32_t s_h, s_w;     // strides of the window rule
  int32_t kept_w;       // ceil(grid_w / s_w): retained patch columns per row
  int32_t kept_patches; // ceil(grid_h / s_h) * kept_w: retained patches of a subsampled frame
  int32_t Lc;           // n_special + kept_patches: compact tokens of a subsampled frame
  int32_t keep_first;   // 1: frame 0 keeps every patch
  int32_t diag;
  int32_t mean_fill;
  int64_t n_tok;        // N * L
  int64_t M;            // compact keys
  int64_t n_dropped;    // |D|
  float   scale;        // softmax scale
};

// Validates p and fills plan.  Returns an AVGGT_* code.  Pure host arithmetic.
int make_plan(const avggt_params* p, Plan* plan);

// The window rule, shared by host and device code of the CUDA path.
//   slot u of frame f  ->  compact slot within the frame's compact block, or -1 if dropped
#if defined(__CUDACC__)
#define AVGGT_HD __host__ __device__ __forceinline__
#else
#define AVGGT_HD inline
#endif

AVGGT_HD int32_t compact_slot(const Plan& pl, int32_t f, int32_t u) {
  if (u < pl.n_special) return u;
  if (pl.keep_first && f == 0) return u;
  const int32_t patch = u - pl.n_special;
  const int32_t r = patch / pl.grid_w;
  const int32_t c = patch - r * pl.grid_w;
  if ((r % pl.s_h) != 0 || (c % pl.s_w) != 0) return -1;
  return pl.n_special + (r / pl.s_h) * pl.kept_w + (c / pl.s_w);
}

// first compact index of frame f
AVGGT_HD int64_t compact_frame_base(const Plan& pl, int32_t f) {
  if (pl.keep_first) return f == 0 ? 0 : static_cast<int64_t>(pl.L) + static_cast<int64_t>(f - 1) * pl.Lc;
  return static_cast<int64_t>(f) * pl.Lc;
}

}  // namespace avggt
