// K/V compaction and mean-fill reduction (Sec. 4.3 of the AVGGT paper):
// one pass over K and V that copies the retained rows into the head-major
// compact arrays and sums the dropped patch rows for the mean Key/Value pair.
//
// Memory-bound: every row of K and V is read once with 16-byte loads (a warp
// covers 512 contiguous bytes per load instruction), retained rows are written
// once as full 128-byte lines.  Sums are kept in registers per lane (a lane owns
// fixed columns), reduced across the warps of a block in shared memory in a
// fixed order, written as one partial row per block, and reduced across blocks
// by a second small kernel with a fixed shuffle tree: no floating-point
// atomics, so the result does not change from run to run.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "internal.h"

namespace avggt {

namespace {

constexpr int kBuildThreads = 256;
constexpr int kBuildWarps = kBuildThreads / 32;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ void add_bf16x8(float (&acc)[8], const uint4& v) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    acc[2 * i] += __uint_as_float(w[i] << 16);            // low half: even element
    acc[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);  // high half: odd element
  }
}

// PASSES = ceil(H * 8 / 32): 16-byte chunks of one row handled per lane.
// kc_rows: rows per head of the compact arrays (M, or more when the caller's arrays are a slot of a
// larger exchange buffer).
template <int PASSES>
__global__ void __launch_bounds__(kBuildThreads)
build_kv_kernel(const Plan pl, const uint4* __restrict__ K, const uint4* __restrict__ V, uint4* __restrict__ Kc,
                uint4* __restrict__ Vc, const int64_t kc_rows, int32_t* __restrict__ idx, float* __restrict__ partials,
                const int do_mean, const int32_t* __restrict__ slot_of_token) {
  extern __shared__ float red[];   // [kBuildWarps][PASSES * 256]
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const uint32_t chunks_per_row = static_cast<uint32_t>(pl.H) * 8u;   // 16-byte chunks (d = 64 bf16 = 8 chunks per head)
  const uint32_t n_tok = static_cast<uint32_t>(pl.n_tok);
  const uint32_t warps_total = gridDim.x * kBuildWarps;

  float acc_k[PASSES][8], acc_v[PASSES][8];
#pragma unroll
  for (int p = 0; p < PASSES; ++p)
#pragma unroll
    for (int e = 0; e < 8; ++e) { acc_k[p][e] = 0.f; acc_v[p][e] = 0.f; }

  for (uint32_t row = blockIdx.x * kBuildWarps + warp; row < n_tok; row += warps_total) {
    const int32_t f = static_cast<int32_t>(row / static_cast<uint32_t>(pl.L));
    const int32_t u = static_cast<int32_t>(row - static_cast<uint32_t>(f) * static_cast<uint32_t>(pl.L));
    // compact position within the frame's block by the window rule, or, for a caller-chosen retained set,
    // the global compact position from the caller's map
    const int32_t cs = slot_of_token != nullptr ? slot_of_token[row] : compact_slot(pl, f, u);
    if (cs < 0 && !do_mean) continue;
    const uint4* krow = K + static_cast<size_t>(row) * chunks_per_row;
    const uint4* vrow = V + static_cast<size_t>(row) * chunks_per_row;
    uint4 kv[PASSES], vv[PASSES];
#pragma unroll
    for (int p = 0; p < PASSES; ++p) {
      const uint32_t c = p * 32 + lane;
      if (c < chunks_per_row) { kv[p] = ld_stream(krow + c); vv[p] = ld_stream(vrow + c); }
      else { kv[p] = make_uint4(0, 0, 0, 0); vv[p] = make_uint4(0, 0, 0, 0); }
    }
    if (cs >= 0) {
      const int64_t m = slot_of_token != nullptr ? cs : compact_frame_base(pl, f) + cs;
      if (lane == 0 && idx != nullptr) idx[m] = static_cast<int32_t>(row);
#pragma unroll
      for (int p = 0; p < PASSES; ++p) {
        const uint32_t c = p * 32 + lane;
        if (c < chunks_per_row) {
          const size_t dst = (static_cast<size_t>(c >> 3) * static_cast<size_t>(kc_rows) + static_cast<size_t>(m)) * 8u + (c & 7u);
          Kc[dst] = kv[p];
          Vc[dst] = vv[p];
        }
      }
    } else {
#pragma unroll
      for (int p = 0; p < PASSES; ++p) { add_bf16x8(acc_k[p], kv[p]); add_bf16x8(acc_v[p], vv[p]); }
    }
  }

  if (!do_mean) return;
  // block reduction, K then V, fixed order over warps
  const int cols = pl.H * pl.d;   // = chunks_per_row * 8
#pragma unroll
  for (int which = 0; which < 2; ++which) {
    float* mine = red + warp * (PASSES * 256);
#pragma unroll
    for (int p = 0; p < PASSES; ++p)
#pragma unroll
      for (int e = 0; e < 8; ++e) mine[(p * 32 + lane) * 8 + e] = which == 0 ? acc_k[p][e] : acc_v[p][e];
    __syncthreads();
    for (int col = threadIdx.x; col < cols; col += kBuildThreads) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < kBuildWarps; ++w) s += red[w * (PASSES * 256) + col];
      partials[static_cast<size_t>(blockIdx.x) * (2 * cols) + which * cols + col] = s;
    }
    __syncthreads();
  }
}

// out[col] = (sum over blocks of partials[b][col]) / n_dropped, col in [0, 2*cols)
// block = 32 columns x 32 block-groups; the cross-group sum is a warp shuffle tree.
__global__ void __launch_bounds__(1024)
mean_finalize_kernel(const float* __restrict__ partials, int n_blocks, int cols2, float inv_count,
                     float* __restrict__ kmean, float* __restrict__ vmean) {
  __shared__ float tile[32][33];
  const int c = threadIdx.x & 31, g = threadIdx.x >> 5;
  const int col = blockIdx.x * 32 + c;
  float s = 0.f;
  if (col < cols2)
    for (int b = g; b < n_blocks; b += 32) s += partials[static_cast<size_t>(b) * cols2 + col];
  tile[c][g] = s;
  __syncthreads();
  // warp g now owns column blockIdx.x*32 + g; lane c holds the partial of group c
  float v = tile[g][c];
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  const int ocol = blockIdx.x * 32 + g;
  if (c == 0 && ocol < cols2) {
    const int cols = cols2 / 2;
    if (ocol < cols) kmean[ocol] = v * inv_count;
    else vmean[ocol - cols] = v * inv_count;
  }
}

// slot_of_token[t] = -1 for every token, then m for the m-th retained token.  Entries of idx outside
// [0, n_tok) are skipped.
__global__ void fill_slots_kernel(int32_t* __restrict__ slot_of_token, int64_t n_tok) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < n_tok) slot_of_token[i] = -1;
}
__global__ void scatter_slots_kernel(const int32_t* __restrict__ idx, int64_t M, int32_t* __restrict__ slot_of_token,
                                     int64_t n_tok) {
  const int64_t m = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (m < M) {
    const int32_t t = idx[m];
    if (t >= 0 && t < n_tok) slot_of_token[t] = static_cast<int32_t>(m);
  }
}

template <int PASSES>
cudaError_t launch_build(const Plan& pl, int grid, const void* K, const void* V, void* Kc, void* Vc, int64_t kc_rows,
                         int32_t* idx, float* partials, int do_mean, const int32_t* slot_of_token, cudaStream_t st) {
  const size_t smem = do_mean ? static_cast<size_t>(kBuildWarps) * PASSES * 256 * sizeof(float) : 0;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(build_kv_kernel<PASSES>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
  }
  build_kv_kernel<PASSES><<<grid, kBuildThreads, smem, st>>>(pl, static_cast<const uint4*>(K), static_cast<const uint4*>(V),
                                                           static_cast<uint4*>(Kc), static_cast<uint4*>(Vc), kc_rows, idx, partials,
                                                           do_mean, slot_of_token);
  return cudaGetLastError();
}

// Exchange buffer [n_ranks][2][H][slot_rows][d] (every rank's compact K then V, padded to slot_rows rows per
// head) -> Kc, Vc [H][M_total][d] with the ranks' rows one after the other.  One thread per 16-byte chunk.
struct ShardOffsets {
  int32_t n_ranks;
  int64_t first[kMaxShardRanks + 1];   // first compact row of rank r; first[n_ranks] = M_total
};
__global__ void __launch_bounds__(256)
assemble_shards_kernel(const uint4* __restrict__ gathered, const ShardOffsets off, const int H, const int64_t slot_rows,
                       uint4* __restrict__ Kc, uint4* __restrict__ Vc) {
  const int64_t m_total = off.first[off.n_ranks];
  const int64_t chunks = 2 * static_cast<int64_t>(H) * m_total * 8;   // 8 chunks of 16 bytes per row of 64 bf16
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < chunks;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t c = i & 7;
    int64_t row = i >> 3;                       // (which, head, m)
    const int64_t m = row % m_total;
    row /= m_total;
    const int64_t h = row % H;
    const int64_t which = row / H;
    int r = 0;
    while (r + 1 < off.n_ranks && m >= off.first[r + 1]) ++r;
    const int64_t src = ((((static_cast<int64_t>(r) * 2 + which) * H + h) * slot_rows) + (m - off.first[r])) * 8 + c;
    const uint4 v = gathered[src];
    (which == 0 ? Kc : Vc)[(h * m_total + m) * 8 + c] = v;
  }
}

}  // namespace

cudaError_t launch_assemble_shards(const void* gathered, int n_ranks, const int64_t* kept, int H, int d, int64_t slot_rows,
                                   void* Kc, void* Vc, const float* sums, int64_t n_dropped_total, float* kmean,
                                   float* vmean, cudaStream_t st) {
  ShardOffsets off;
  off.n_ranks = n_ranks;
  off.first[0] = 0;
  for (int r = 0; r < n_ranks; ++r) off.first[r + 1] = off.first[r] + kept[r];
  const int64_t chunks = 2 * static_cast<int64_t>(H) * off.first[n_ranks] * 8;
  if (chunks > 0) {
    int64_t blocks = (chunks + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    assemble_shards_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(static_cast<const uint4*>(gathered), off, H, slot_rows,
                                                                         static_cast<uint4*>(Kc), static_cast<uint4*>(Vc));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  if (sums != nullptr && n_dropped_total > 0) {
    const int cols2 = 2 * H * d;
    mean_finalize_kernel<<<(cols2 + 31) / 32, 1024, 0, st>>>(sums, 1, cols2, 1.0f / static_cast<float>(n_dropped_total), kmean, vmean);
    return cudaGetLastError();
  }
  return cudaSuccess;
}

int build_kv_grid(const Plan& pl, int sm_count) {
  const int64_t by_rows = (pl.n_tok + kBuildWarps - 1) / kBuildWarps;
  int64_t g = static_cast<int64_t>(sm_count) * 4;
  if (g > by_rows) g = by_rows;
  if (g < 1) g = 1;
  return static_cast<int>(g);
}

size_t build_kv_ws_bytes(const Plan& pl, int sm_count) {
  return static_cast<size_t>(build_kv_grid(pl, sm_count)) * 2 * pl.H * pl.d * sizeof(float);
}

cudaError_t launch_build_kv(const Plan& pl, int sm_count, const void* K, const void* V, void* Kc, void* Vc,
                            int32_t* idx, float* kmean, float* vmean, void* ws, cudaStream_t st,
                            const int32_t* caller_idx, int32_t* slot_of_token, int64_t kc_rows, bool sums_only) {
  if (kc_rows <= 0) kc_rows = pl.M;
  if (slot_of_token != nullptr) {
    // caller-chosen retained set: build the token -> compact position map first
    fill_slots_kernel<<<static_cast<unsigned>((pl.n_tok + 255) / 256), 256, 0, st>>>(slot_of_token, pl.n_tok);
    if (pl.M > 0 && caller_idx != nullptr)
      scatter_slots_kernel<<<static_cast<unsigned>((pl.M + 255) / 256), 256, 0, st>>>(caller_idx, pl.M, slot_of_token, pl.n_tok);
    cudaError_t e0 = cudaGetLastError();
    if (e0 != cudaSuccess) return e0;
    idx = nullptr;
  }
  const int grid = build_kv_grid(pl, sm_count);
  const int do_mean = (pl.mean_fill != 0 && pl.n_dropped > 0) ? 1 : 0;
  float* partials = static_cast<float*>(ws);
  const int passes = (pl.H * 8 + 31) / 32;
  cudaError_t e;
  switch (passes) {
    case 1: e = launch_build<1>(pl, grid, K, V, Kc, Vc, kc_rows, idx, partials, do_mean, slot_of_token, st); break;
    case 2: e = launch_build<2>(pl, grid, K, V, Kc, Vc, kc_rows, idx, partials, do_mean, slot_of_token, st); break;
    case 3: e = launch_build<3>(pl, grid, K, V, Kc, Vc, kc_rows, idx, partials, do_mean, slot_of_token, st); break;
    case 4: e = launch_build<4>(pl, grid, K, V, Kc, Vc, kc_rows, idx, partials, do_mean, slot_of_token, st); break;
    case 5: e = launch_build<5>(pl, grid, K, V, Kc, Vc, kc_rows, idx, partials, do_mean, slot_of_token, st); break;
    case 6: e = launch_build<6>(pl, grid, K, V, Kc, Vc, kc_rows, idx, partials, do_mean, slot_of_token, st); break;
    case 7: e = launch_build<7>(pl, grid, K, V, Kc, Vc, kc_rows, idx, partials, do_mean, slot_of_token, st); break;
    case 8: e = launch_build<8>(pl, grid, K, V, Kc, Vc, kc_rows, idx, partials, do_mean, slot_of_token, st); break;
    default: return cudaErrorInvalidValue;
  }
  if (e != cudaSuccess) return e;
  if (pl.mean_fill != 0) {
    const int cols2 = 2 * pl.H * pl.d;
    if (do_mean) {
      const float inv_count = sums_only ? 1.0f : 1.0f / static_cast<float>(pl.n_dropped);
      mean_finalize_kernel<<<(cols2 + 31) / 32, 1024, 0, st>>>(partials, grid, cols2, inv_count, kmean, vmean);
      e = cudaGetLastError();
    } else {
      e = cudaMemsetAsync(kmean, 0, static_cast<size_t>(pl.H) * pl.d * sizeof(float), st);
      if (e == cudaSuccess) e = cudaMemsetAsync(vmean, 0, static_cast<size_t>(pl.H) * pl.d * sizeof(float), st);
    }
  }
  return e;
}

}  // namespace avggt
