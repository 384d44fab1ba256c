// K/V projection with the compaction of Sec. 4.3 fused into its epilogue:
//   K = X Wk^T + bk,  V = X Wv^T + bv        (bf16 operands, fp32 accumulation)
// and, while a tile of the result is still in tensor memory, the retained rows go to the
// head-major compact arrays, the dropped rows are added to the sums behind the mean pair, and
// (optionally) every row is written to the full K / V arrays.  The paper's remark that diagonal
// preservation and mean-fill cost "only O(N)" holds here without a second pass over K and V.
//
// A dense contraction, so it runs on the tensor cores: a persistent kernel, one CTA per SM slot,
// three roles.
//   warp 0      TMA producer: X tiles (128 tokens x 64 channels) and W tiles (256 output columns x
//               64 channels) through a four-stage shared-memory ring (128-byte swizzle)
//   warp 1      MMA issuer: tcgen05.mma, M 128 x N 256 x K 16, fp32 accumulators in tensor memory;
//               two accumulators of 256 columns, so the next tile's products run under this
//               tile's epilogue
//   warps 2-5   epilogue, one token row per thread: accumulator -> registers, bias, bf16, stores;
//               the sums over dropped rows are taken across the 32 rows of a warp with a
//               transposing shuffle reduction (lane c ends up with column c) and kept in
//               registers for all the tiles of the CTA
// A CTA keeps one block of 256 output columns (four heads of K or of V) for its whole life and
// walks over token tiles; CTAs with the same token tile run side by side, so an X tile is
// fetched from HBM once and from L2 by the others.  Per-CTA partial sums go to the workspace and
// a small second kernel adds them in a fixed order: no floating-point atomics, results identical
// from run to run.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "internal.h"
#include "ptx.cuh"
#include "tmap.h"

namespace avggt {

namespace {

constexpr int kTileTok = 128;     // token rows per tile (M of the MMA)
constexpr int kTileCol = 256;     // output columns per tile (N of the MMA): four heads of 64
constexpr int kBlockK = 64;       // channels per ring stage: one 128-byte swizzle row
constexpr int kProjStages = 4;
constexpr uint32_t kBytesA = kTileTok * kBlockK * 2;   // 16 KiB
constexpr uint32_t kBytesB = kTileCol * kBlockK * 2;   // 32 KiB
constexpr int kProjThreads = 192;   // warps 2..5 are the epilogue: warp % 4 covers the four lane quarters of tensor memory
constexpr uint32_t kProjTmemCols = 512;

struct ProjArgs {
  Plan pl;
  int32_t C;              // model dimension (channels of X)
  int32_t n_col_tiles;    // column tiles of one projection: ceil(H * d / 256)
  int32_t n_tok_tiles;    // ceil(n_tok / 128)
  int32_t tok_stride;     // token tiles a CTA advances by: gridDim.x / (2 * n_col_tiles)
  const float* bias_k;    // [H * d] or null
  const float* bias_v;
  uint4* K_full;          // [n_tok, H, d] or null
  uint4* V_full;
  uint4* Kc;              // [H, M, d]
  uint4* Vc;
  int32_t* idx;           // [M] or null
  float* partials;        // [gridDim.x][4 warps][256]: sums over the dropped rows this warp has seen
  uint32_t* status;       // 4 words, as in the attention kernel
  int32_t do_mean;
};

struct __align__(8) ProjBarriers {
  uint64_t full[kProjStages], empty[kProjStages];
  uint64_t acc_full[2], acc_empty[2];
  uint64_t mma_idle;      // MMA issuer -> itself: every product it issued has completed
  uint32_t tmem_base;
  uint32_t abort_flag;
};

__device__ __forceinline__ void proj_report(const ProjArgs& a, ProjBarriers* bars, uint32_t where, uint32_t iter) {
  if (atomicCAS(a.status, 0u, 1u) == 0u) {
    a.status[1] = blockIdx.x;
    a.status[2] = where;
    a.status[3] = iter;
  }
  *reinterpret_cast<volatile uint32_t*>(&bars->abort_flag) = 1u;
}

// Bounded wait; false when the limit ran out or another role of the CTA gave up.
__device__ __forceinline__ bool proj_wait(uint64_t* bar, uint32_t parity, ProjBarriers* bars, const ProjArgs& a,
                                          uint32_t where, uint32_t iter, bool check_abort = true) {
  const uint32_t b = smem_u32(bar);
  if (mbar_try_wait(b, parity)) return true;
  const uint64_t t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (true) {
    if (mbar_try_wait(b, parity)) return true;
    if ((++spins & 0xffu) == 0) {
      if (check_abort && *reinterpret_cast<volatile uint32_t*>(&bars->abort_flag)) return false;
      if (globaltimer_ns() - t0 > AVGGT_WAIT_LIMIT_NS) {
        proj_report(a, bars, where, iter);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool proj_wait_warp(uint64_t* bar, uint32_t parity, ProjBarriers* bars, const ProjArgs& a,
                                               uint32_t where, uint32_t iter, bool check_abort = true) {
  return __all_sync(0xffffffffu, proj_wait(bar, parity, bars, a, where, iter, check_abort));
}

// v[i] of lane l  ->  lane c returns sum over l of v[c] (of lane l): 31 shuffles for 32 columns.
__device__ __forceinline__ float warp_column_sums(float (&v)[32], int lane) {
#pragma unroll
  for (int half = 16; half >= 1; half >>= 1) {
    // lanes with the bit set keep the upper `half` entries, the others the lower ones
    const bool upper = (lane & half) != 0;
#pragma unroll
    for (int i = 0; i < half; ++i) {
      const float mine = upper ? v[i + half] : v[i];
      const float theirs = upper ? v[i] : v[i + half];
      v[i] = mine + __shfl_xor_sync(0xffffffffu, theirs, half);
    }
  }
  return v[0];
}

__global__ void __launch_bounds__(kProjThreads, 1)
project_kv_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_wk,
                  const __grid_constant__ CUtensorMap tm_wv, const ProjArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;                               // kProjStages tiles of X
  uint8_t* sB = smem + kProjStages * kBytesA;       // kProjStages tiles of W
  __shared__ ProjBarriers bars;

  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0);
  const int lane = threadIdx.x & 31;
  // this CTA's block of output columns, for its whole life
  const int col_tile_all = blockIdx.x % (2 * a.n_col_tiles);
  const int which = col_tile_all / a.n_col_tiles;                 // 0: K, 1: V
  const int col_tile = col_tile_all - which * a.n_col_tiles;
  const int tok0 = blockIdx.x / (2 * a.n_col_tiles);              // first token tile
  const int n_kb = a.C / kBlockK;

  if (__syncthreads_or(*reinterpret_cast<volatile uint32_t*>(a.status) != 0u)) return;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kProjStages; ++s) {
      mbar_init(smem_u32(&bars.full[s]), 1);
      mbar_init(smem_u32(&bars.empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars.acc_full[b]), 1);
      mbar_init(smem_u32(&bars.acc_empty[b]), 4);
    }
    mbar_init(smem_u32(&bars.mma_idle), 1);
    bars.abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&bars.tmem_base), kProjTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars.tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    const CUtensorMap* tm_w = which == 0 ? &tm_wk : &tm_wv;
    if (elect_one()) {
      prefetch_tensormap(&tm_x);
      prefetch_tensormap(tm_w);
    }
    int stage = 0, issued = 0;
    uint32_t parity = 1;   // a fresh barrier passes the wait on the "previous" phase at once
    bool ok = true;
    for (int tt = tok0; tt < a.n_tok_tiles && ok; tt += a.tok_stride) {
      for (int kb = 0; kb < n_kb; ++kb) {
        ok = proj_wait_warp(&bars.empty[stage], parity, &bars, a, 10, issued);
        if (!ok) break;
        if (elect_one()) {
          const uint32_t fb = smem_u32(&bars.full[stage]);
          mbar_arrive_expect_tx(fb, kBytesA + kBytesB);
          tma_load_2d(smem_u32(sA + stage * kBytesA), &tm_x, kb * kBlockK, tt * kTileTok, fb);
          tma_load_2d(smem_u32(sB + stage * kBytesB), tm_w, kb * kBlockK, col_tile * kTileCol, fb);
        }
        __syncwarp();
        ++issued;
        if (++stage == kProjStages) { stage = 0; parity ^= 1; }
      }
    }
    if (!ok) {   // let the copies in flight land before the CTA gives up its shared memory
      for (int back = 1; back <= kProjStages; ++back) {
        const int jt = issued - back;
        if (jt >= 0) (void)proj_wait_warp(&bars.full[jt % kProjStages], (jt / kProjStages) & 1, &bars, a, 12, jt, false);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    constexpr uint32_t idesc = umma_idesc_bf16(kTileTok, kTileCol, false);
    int stage = 0, it = 0;
    uint32_t parity = 0;
    bool ok = true;
    for (int tt = tok0; tt < a.n_tok_tiles && ok; tt += a.tok_stride, ++it) {
      const int buf = it & 1;
      // the epilogue has emptied this accumulator (first use of either buffer: passes at once)
      ok = proj_wait_warp(&bars.acc_empty[buf], ((it >> 1) & 1) ^ 1, &bars, a, 20, it);
      if (!ok) break;
      tc_fence_after();
      for (int kb = 0; kb < n_kb; ++kb) {
        ok = proj_wait_warp(&bars.full[stage], parity, &bars, a, 21, kb);
        if (!ok) break;
        tc_fence_after();
        if (elect_one()) {
          const uint64_t da = umma_desc_sw128(smem_u32(sA + stage * kBytesA));
          const uint64_t db = umma_desc_sw128(smem_u32(sB + stage * kBytesB));
#pragma unroll
          for (int k = 0; k < kBlockK / 16; ++k)
            umma_ss(tmem + buf * kTileCol, da + (k * 32 >> 4), db + (k * 32 >> 4), idesc, (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit(smem_u32(&bars.empty[stage]));
          if (kb == n_kb - 1) umma_commit(smem_u32(&bars.acc_full[buf]));
        }
        __syncwarp();
        if (++stage == kProjStages) { stage = 0; parity ^= 1; }
      }
    }
    // every product this warp issued has completed before tensor memory is freed (also on a wait that ran out)
    __syncwarp();
    if (elect_one()) umma_commit(smem_u32(&bars.mma_idle));
    __syncwarp();
    (void)proj_wait_warp(&bars.mma_idle, 0, &bars, a, 22, it, false);
  } else {
    // ------------------------------------------------------------ epilogue: one token row per thread
    const Plan& pl = a.pl;
    const int quarter = warp & 3;                       // tensor-memory lanes [32 quarter, 32 quarter + 32)
    const float* bias = which == 0 ? a.bias_k : a.bias_v;
    uint4* full = which == 0 ? a.K_full : a.V_full;
    uint4* compact = which == 0 ? a.Kc : a.Vc;
    const int cols_total = pl.H * pl.d;
    float colsum[kTileCol / 32];                        // lane c: column 32 i + c of this CTA's block, over dropped rows
#pragma unroll
    for (int i = 0; i < kTileCol / 32; ++i) colsum[i] = 0.f;
    int it = 0;
    bool ok = true;
    for (int tt = tok0; tt < a.n_tok_tiles; tt += a.tok_stride, ++it) {
      const int buf = it & 1;
      ok = proj_wait_warp(&bars.acc_full[buf], (it >> 1) & 1, &bars, a, 30, it);
      if (!ok) break;
      tc_fence_after();
      const int64_t row = static_cast<int64_t>(tt) * kTileTok + quarter * 32 + lane;
      const bool row_valid = row < pl.n_tok;
      int32_t cs = -1;
      int64_t m = 0;
      if (row_valid) {
        const int32_t f = static_cast<int32_t>(row / pl.L);
        cs = compact_slot(pl, f, static_cast<int32_t>(row - static_cast<int64_t>(f) * pl.L));
        if (cs >= 0) m = compact_frame_base(pl, f) + cs;
      }
      const bool kept = row_valid && cs >= 0;
      const bool dropped = row_valid && cs < 0;
      if (kept && which == 0 && col_tile == 0 && a.idx != nullptr) a.idx[m] = static_cast<int32_t>(row);
      const uint32_t t_acc = tmem + buf * kTileCol + (static_cast<uint32_t>(32 * quarter) << 16);
#pragma unroll
      for (int c = 0; c < kTileCol / 32; ++c) {
        uint32_t raw[32];
        tmem_ld32(t_acc + c * 32, raw);
        tmem_wait_ld();
        const int col0 = col_tile * kTileCol + c * 32;            // first column of the chunk within K (or V)
        if (col0 < cols_total) {                                    // warp-uniform: a chunk is half a head
          float v[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(raw[i]) + (bias != nullptr ? __ldg(bias + col0 + i) : 0.f);
          uint4 out[4];
          uint32_t* o32 = reinterpret_cast<uint32_t*>(out);
#pragma unroll
          for (int i = 0; i < 16; ++i) o32[i] = pack_bf16x2(v[2 * i], v[2 * i + 1]);
          const int head = col0 >> 6, dchunk = (col0 & 63) >> 3;    // 16-byte chunk within the head's 64 values
          if (row_valid && full != nullptr) {
            uint4* dst = full + (static_cast<size_t>(row) * pl.H + head) * 8 + dchunk;
#pragma unroll
            for (int i = 0; i < 4; ++i) dst[i] = out[i];
          }
          if (kept) {
            uint4* dst = compact + (static_cast<size_t>(head) * static_cast<size_t>(pl.M) + static_cast<size_t>(m)) * 8 + dchunk;
#pragma unroll
            for (int i = 0; i < 4; ++i) dst[i] = out[i];
          }
          if (a.do_mean) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = dropped ? v[i] : 0.f;
            colsum[c] += warp_column_sums(v, lane);
          }
        }
      }
      // this warp is done with the accumulator
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars.acc_empty[buf]));
    }
    if (ok && a.do_mean) {
      float* dst = a.partials + (static_cast<size_t>(blockIdx.x) * 4 + quarter) * kTileCol;
#pragma unroll
      for (int i = 0; i < kTileCol / 32; ++i) dst[32 * i + lane] = colsum[i];
    }
  }

  tmem_wait_ld();
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kProjTmemCols);
}

// kmean[col] = (sum over the CTAs that own col's block, and their four epilogue warps, in a fixed order) / n_dropped
__global__ void __launch_bounds__(256)
project_mean_kernel(const float* __restrict__ partials, int grid, int n_col_tiles, int cols_total, float inv_count,
                    float* __restrict__ kmean, float* __restrict__ vmean) {
  const int g = blockIdx.x * blockDim.x + threadIdx.x;     // column of [K | V]
  if (g >= 2 * cols_total) return;
  const int which = g / cols_total, col = g - which * cols_total;
  const int col_tile_all = which * n_col_tiles + col / kTileCol, in_tile = col % kTileCol;
  float s = 0.f;
  for (int cta = col_tile_all; cta < grid; cta += 2 * n_col_tiles)
    for (int w = 0; w < 4; ++w) s += partials[(static_cast<size_t>(cta) * 4 + w) * kTileCol + in_tile];
  (which == 0 ? kmean : vmean)[col] = s * inv_count;
}

constexpr size_t kProjSmemBytes = static_cast<size_t>(kProjStages) * (kBytesA + kBytesB) + 1024;

int project_grid(const Plan& pl, int sm_count) {
  const int per_tok = 2 * ((pl.H * pl.d + kTileCol - 1) / kTileCol);
  int g = (sm_count / per_tok) * per_tok;
  if (g < per_tok) g = per_tok;
  const int64_t tok_tiles = (pl.n_tok + kTileTok - 1) / kTileTok;
  if (g / per_tok > tok_tiles) g = static_cast<int>(tok_tiles) * per_tok;
  return g;
}

}  // namespace

size_t project_kv_ws_bytes(const Plan& pl, int sm_count) {
  return kAttnStatusBytes + static_cast<size_t>(project_grid(pl, sm_count)) * 4 * kTileCol * sizeof(float);
}

cudaError_t launch_project_kv(const Plan& pl, int sm_count, int model_dim, const void* X, const void* Wk, const void* Wv,
                              const float* bias_k, const float* bias_v, void* K, void* V, void* Kc, void* Vc, int32_t* idx,
                              float* kmean, float* vmean, void* ws, cudaStream_t st, bool* tmap_failed) {
  *tmap_failed = false;
  const int cols_total = pl.H * pl.d;
  ProjArgs a;
  a.pl = pl;
  a.C = model_dim;
  a.n_col_tiles = (cols_total + kTileCol - 1) / kTileCol;
  a.n_tok_tiles = static_cast<int32_t>((pl.n_tok + kTileTok - 1) / kTileTok);
  const int grid = project_grid(pl, sm_count);
  a.tok_stride = grid / (2 * a.n_col_tiles);
  a.bias_k = bias_k;
  a.bias_v = bias_v;
  a.K_full = static_cast<uint4*>(K);
  a.V_full = static_cast<uint4*>(V);
  a.Kc = static_cast<uint4*>(Kc);
  a.Vc = static_cast<uint4*>(Vc);
  a.idx = idx;
  a.status = static_cast<uint32_t*>(ws);
  a.partials = reinterpret_cast<float*>(static_cast<char*>(ws) + kAttnStatusBytes);
  a.do_mean = (pl.mean_fill != 0 && pl.n_dropped > 0) ? 1 : 0;

  CUtensorMap tm_x, tm_wk, tm_wv;
  const uint64_t x_dims[2] = {static_cast<uint64_t>(model_dim), static_cast<uint64_t>(pl.n_tok)};
  const uint64_t w_dims[2] = {static_cast<uint64_t>(model_dim), static_cast<uint64_t>(cols_total)};
  const uint64_t row_bytes[1] = {static_cast<uint64_t>(model_dim) * 2};
  const uint32_t x_box[2] = {kBlockK, kTileTok};
  const uint32_t w_box[2] = {kBlockK, kTileCol};
  bool good = make_tmap_bf16(&tm_x, X, 2, x_dims, row_bytes, x_box);
  good = good && make_tmap_bf16(&tm_wk, Wk, 2, w_dims, row_bytes, w_box);
  good = good && make_tmap_bf16(&tm_wv, Wv, 2, w_dims, row_bytes, w_box);
  if (!good) { *tmap_failed = true; return cudaSuccess; }

  cudaError_t e = cudaFuncSetAttribute(project_kv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kProjSmemBytes));
  if (e != cudaSuccess) return e;
  e = cudaMemsetAsync(ws, 0, kAttnStatusBytes, st);
  if (e != cudaSuccess) return e;
  project_kv_kernel<<<grid, kProjThreads, kProjSmemBytes, st>>>(tm_x, tm_wk, tm_wv, a);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (pl.mean_fill != 0) {
    if (a.do_mean) {
      project_mean_kernel<<<(2 * cols_total + 255) / 256, 256, 0, st>>>(a.partials, grid, a.n_col_tiles, cols_total,
                                                                      1.0f / static_cast<float>(pl.n_dropped), kmean, vmean);
      e = cudaGetLastError();
    } else {
      e = cudaMemsetAsync(kmean, 0, static_cast<size_t>(cols_total) * sizeof(float), st);
      if (e == cudaSuccess) e = cudaMemsetAsync(vmean, 0, static_cast<size_t>(cols_total) * sizeof(float), st);
    }
  }
  return e;
}

}  // namespace avggt
