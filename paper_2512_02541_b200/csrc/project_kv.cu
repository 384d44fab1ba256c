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
//   warps 2-9   epilogue, one token row and half of the tile's columns per thread: accumulator -> registers, bias, bf16; a head's
//               64 values of the warp's 32 rows are staged in shared memory (128-byte swizzle),
//               from where one TMA store writes them to the full K / V array and the retained
//               rows are copied, 128 contiguous bytes at a time, to the compact arrays (a thread
//               storing its own row 16 bytes at a time kept the store path busy for longer than
//               the products of the tile take);
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
constexpr uint32_t kStageBytes = 32 * 128;   // epilogue staging: 32 rows x one head (64 bf16), one per epilogue warp
constexpr int kEpiWarps = 8;        // warps 2..9: warp % 4 is the lane quarter of tensor memory, (warp - 2) / 4 the half of
                                    // the tile's 256 columns (two heads each)
constexpr int kProjThreads = 64 + 32 * kEpiWarps;
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
                  const __grid_constant__ CUtensorMap tm_wv, const __grid_constant__ CUtensorMap tm_kfull,
                  const __grid_constant__ CUtensorMap tm_vfull, const ProjArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;                               // kProjStages tiles of X
  uint8_t* sB = smem + kProjStages * kBytesA;       // kProjStages tiles of W
  uint8_t* sStage = sB + kProjStages * kBytesB;     // one staging tile per epilogue warp
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
      mbar_init(smem_u32(&bars.acc_empty[b]), kEpiWarps);
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
    const int col_half = (warp - 2) >> 2;               // columns [128 col_half, 128 col_half + 128) of the tile
    uint8_t* sbuf = sStage + (warp - 2) * kStageBytes;
    const float* bias = which == 0 ? a.bias_k : a.bias_v;
    const bool write_full = (which == 0 ? a.K_full : a.V_full) != nullptr;
    const CUtensorMap* tm_full = which == 0 ? &tm_kfull : &tm_vfull;
    uint4* compact = which == 0 ? a.Kc : a.Vc;
    const int cols_total = pl.H * pl.d;
    float colsum[4];                                    // lane c: column 128 col_half + 32 i + c of this CTA's block, over dropped rows
#pragma unroll
    for (int i = 0; i < 4; ++i) colsum[i] = 0.f;
    int it = 0;
    bool ok = true;
    for (int tt = tok0; tt < a.n_tok_tiles; tt += a.tok_stride, ++it) {
      const int buf = it & 1;
      ok = proj_wait_warp(&bars.acc_full[buf], (it >> 1) & 1, &bars, a, 30, it);
      if (!ok) break;
      tc_fence_after();
      const int64_t row0 = static_cast<int64_t>(tt) * kTileTok + quarter * 32;   // first row of this warp
      const int64_t row = row0 + lane;
      const bool row_valid = row < pl.n_tok;
      int32_t cs = -1;
      int32_t m = 0;
      if (row_valid) {
        const int32_t f = static_cast<int32_t>(row / pl.L);
        cs = compact_slot(pl, f, static_cast<int32_t>(row - static_cast<int64_t>(f) * pl.L));
        if (cs >= 0) m = static_cast<int32_t>(compact_frame_base(pl, f) + cs);
      }
      const bool kept = row_valid && cs >= 0;
      const bool dropped = row_valid && cs < 0;
      if (kept && which == 0 && col_tile == 0 && col_half == 0 && a.idx != nullptr) a.idx[m] = static_cast<int32_t>(row);
      const uint32_t kept_mask = __ballot_sync(0xffffffffu, kept);
      const int n_kept = __popc(kept_mask);
      const uint32_t t_acc = tmem + buf * kTileCol + (static_cast<uint32_t>(32 * quarter) << 16);
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {                              // one head (64 columns) at a time
        const int hg = 2 * col_half + hh;                           // head within the tile
        const int col0 = col_tile * kTileCol + hg * 64;             // first column within K (or V)
        if (col0 >= cols_total) break;                              // warp-uniform: H * d is a multiple of 64
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t raw[32];
          tmem_ld32(t_acc + hg * 64 + half * 32, raw);
          tmem_wait_ld();
          float v[32];
#pragma unroll
          for (int i = 0; i < 32; ++i)
            v[i] = __uint_as_float(raw[i]) + (bias != nullptr ? __ldg(bias + col0 + half * 32 + i) : 0.f);
          if (half == 0) {
            // the store of the previous head has finished reading the staging tile
            if (lane == 0) bulk_wait_read<0>();
            __syncwarp();
          }
          // row `lane` of the staging tile, 16-byte chunks 4 half .. 4 half + 3, swizzled as TMA expects them
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 o;
            o.x = pack_bf16x2(v[8 * i], v[8 * i + 1]);
            o.y = pack_bf16x2(v[8 * i + 2], v[8 * i + 3]);
            o.z = pack_bf16x2(v[8 * i + 4], v[8 * i + 5]);
            o.w = pack_bf16x2(v[8 * i + 6], v[8 * i + 7]);
            *reinterpret_cast<uint4*>(sbuf + lane * 128 + (((4 * half + i) ^ (lane & 7)) << 4)) = o;
          }
          if (a.do_mean) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = dropped ? v[i] : 0.f;
            colsum[2 * hh + half] += warp_column_sums(v, lane);
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        // every row of the tile to the full array (rows beyond the last token are clipped by the tensor map)
        if (write_full && lane == 0) {
          tma_store_2d(tm_full, smem_u32(sbuf), col0, static_cast<int>(row0));
          bulk_commit();
        }
        // retained rows to the compact array: four rows per pass, eight lanes x 16 bytes per row
        const int head = col0 >> 6;
        for (int k0 = 0; k0 < n_kept; k0 += 4) {
          const int k = k0 + (lane >> 3);
          const bool have = k < n_kept;
          const int r = have ? static_cast<int>(__fns(kept_mask, 0, k + 1)) : 0;
          const int32_t m_r = __shfl_sync(0xffffffffu, m, r);
          if (have) {
            const uint4 val = *reinterpret_cast<const uint4*>(sbuf + r * 128 + (((lane & 7) ^ (r & 7)) << 4));
            compact[(static_cast<size_t>(head) * static_cast<size_t>(pl.M) + static_cast<size_t>(m_r)) * 8 + (lane & 7)] = val;
          }
        }
      }
      // this warp is done with the accumulator
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars.acc_empty[buf]));
    }
    if (lane == 0) bulk_wait<0>();   // the staging tiles stay put until the last store has read them
    __syncwarp();
    if (ok && a.do_mean) {
      float* dst = a.partials + (static_cast<size_t>(blockIdx.x) * 4 + quarter) * kTileCol + 128 * col_half;
#pragma unroll
      for (int i = 0; i < 4; ++i) dst[32 * i + lane] = colsum[i];
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

constexpr size_t kProjSmemBytes = static_cast<size_t>(kProjStages) * (kBytesA + kBytesB) + 8 * kStageBytes + 1024;

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

  CUtensorMap tm_x, tm_wk, tm_wv, tm_kfull, tm_vfull;
  const uint64_t x_dims[2] = {static_cast<uint64_t>(model_dim), static_cast<uint64_t>(pl.n_tok)};
  const uint64_t w_dims[2] = {static_cast<uint64_t>(model_dim), static_cast<uint64_t>(cols_total)};
  const uint64_t row_bytes[1] = {static_cast<uint64_t>(model_dim) * 2};
  const uint32_t x_box[2] = {kBlockK, kTileTok};
  const uint32_t w_box[2] = {kBlockK, kTileCol};
  bool good = make_tmap_bf16(&tm_x, X, 2, x_dims, row_bytes, x_box);
  good = good && make_tmap_bf16(&tm_wk, Wk, 2, w_dims, row_bytes, w_box);
  good = good && make_tmap_bf16(&tm_wv, Wv, 2, w_dims, row_bytes, w_box);
  // the full K / V arrays as [n_tok, H * d], written 32 rows x one head at a time (any valid map stands in for an
  // array that is not wanted; the kernel does not use it then)
  const uint64_t f_dims[2] = {static_cast<uint64_t>(cols_total), static_cast<uint64_t>(pl.n_tok)};
  const uint64_t f_row_bytes[1] = {static_cast<uint64_t>(cols_total) * 2};
  const uint32_t f_box[2] = {64, 32};
  if (K != nullptr) good = good && make_tmap_bf16(&tm_kfull, K, 2, f_dims, f_row_bytes, f_box);
  else tm_kfull = tm_x;
  if (V != nullptr) good = good && make_tmap_bf16(&tm_vfull, V, 2, f_dims, f_row_bytes, f_box);
  else tm_vfull = tm_x;
  if (!good) { *tmap_failed = true; return cudaSuccess; }

  cudaError_t e = cudaFuncSetAttribute(project_kv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kProjSmemBytes));
  if (e != cudaSuccess) return e;
  e = cudaMemsetAsync(ws, 0, kAttnStatusBytes, st);
  if (e != cudaSuccess) return e;
  project_kv_kernel<<<grid, kProjThreads, kProjSmemBytes, st>>>(tm_x, tm_wk, tm_wv, tm_kfull, tm_vfull, a);
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
