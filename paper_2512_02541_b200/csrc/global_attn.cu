// Subsampled global attention (Sec. 4.3 of the AVGGT paper) as one fused
// flash-style kernel for sm_100a.
//
// One CTA owns a tile of 128 query rows of one head.  It streams the compacted
// K/V of that head through shared memory with TMA (128-byte swizzle), computes
// S = Q Kc^T and O += P Vc with tcgen05.mma (bf16 operands, fp32 accumulators
// in tensor memory), and keeps the online softmax (running max and sum, fp32,
// base-2 exponentials) in registers, one query row per thread.  The last tile
// of the stream is the K/V of the query rows themselves: its diagonal gives the
// preserved self term.  The epilogue folds the diagonal and the mean-fill
// column into the same normalisation:
//   O = (a_S O_S + p_d v_i + p_m vmean) / (a_S l_S + p_d + p_m).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "internal.h"
#include "ptx.cuh"
#include "tmap.h"

namespace avggt {

namespace {

constexpr int kTileQ = 128;      // query rows per CTA
constexpr int kTileKV = 128;     // keys per step
constexpr int kHeadDim = 64;
constexpr uint32_t kTileBytes = kTileKV * kHeadDim * 2;   // 16 KiB: one 128 x 64 bf16 tile
constexpr int kStages = 2;
constexpr int kThreads = 128;
constexpr uint32_t kTmemCols = 256;  // S: 128, P: 64 (bf16 pairs), O: 64
constexpr float kLog2e = 1.4426950408889634f;

struct AttnArgs {
  Plan pl;
  const float* kmean;   // [H, d] or null
  const float* vmean;
  __nv_bfloat16* O;     // [n_tok, H, d]
  float* lse;           // [n_tok, H] or null
  uint32_t* status;     // 4 words
  int32_t n_kv_tiles;   // ceil(M / 128)
  int32_t use_diag;     // diag on and |D| > 0
  int32_t use_mean;     // mean_fill on and |D| > 0
  float scale_log2;     // softmax scale * log2(e)
};

struct __align__(8) Barriers {
  uint64_t q_full;
  uint64_t k_full[kStages];
  uint64_t v_full[kStages];
  uint64_t s_done;
  uint64_t o_done;
  uint32_t tmem_base;
  uint32_t abort_flag;
};

__device__ __forceinline__ void report_timeout(const AttnArgs& a, Barriers* bars, uint32_t where, uint32_t iter) {
  if (atomicCAS(a.status, 0u, 1u) == 0u) {
    a.status[1] = blockIdx.x + blockIdx.y * gridDim.x;
    a.status[2] = where;
    a.status[3] = iter;
  }
  *reinterpret_cast<volatile uint32_t*>(&bars->abort_flag) = 1u;
}

// bounded wait that also gives up when another thread of the CTA has aborted
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, Barriers* bars, bool check_abort = true) {
  const uint32_t b = smem_u32(bar);
  if (mbar_try_wait(b, parity)) return true;
  const uint64_t t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (true) {
    if (mbar_try_wait(b, parity)) return true;
    if ((++spins & 0xffu) == 0) {
      if (check_abort && *reinterpret_cast<volatile uint32_t*>(&bars->abort_flag)) return false;
      if (globaltimer_ns() - t0 > AVGGT_WAIT_LIMIT_NS) return false;
    }
  }
}

// 16-byte chunk c (0..7) of row r of a 128-byte-swizzled tile
__device__ __forceinline__ uint4 ld_swizzled(const uint8_t* tile, int r, int c) {
  return *reinterpret_cast<const uint4*>(tile + r * 128 + ((c ^ (r & 7)) << 4));
}

__device__ __forceinline__ float dot_bf16x8(const uint4& a, const uint4& b, float acc) {
  const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    acc = fmaf(__uint_as_float(aw[i] << 16), __uint_as_float(bw[i] << 16), acc);
    acc = fmaf(__uint_as_float(aw[i] & 0xffff0000u), __uint_as_float(bw[i] & 0xffff0000u), acc);
  }
  return acc;
}

__global__ void __launch_bounds__(kThreads, 2)
global_attn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_kc,
                   const __grid_constant__ CUtensorMap tm_vc, const AttnArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = smem + kTileBytes;                       // kStages tiles
  uint8_t* sV = smem + kTileBytes * (1 + kStages);       // kStages tiles
  __shared__ Barriers bars;

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int head = blockIdx.y;
  const int q0 = blockIdx.x * kTileQ;
  const Plan& pl = a.pl;

  if (tid == 0) {
    mbar_init(smem_u32(&bars.q_full), 1);
    for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&bars.k_full[s]), 1); mbar_init(smem_u32(&bars.v_full[s]), 1); }
    mbar_init(smem_u32(&bars.s_done), 1);
    mbar_init(smem_u32(&bars.o_done), 1);
    bars.abort_flag = 0;
    fence_mbar_init();
    prefetch_tensormap(&tm_q);
    prefetch_tensormap(&tm_kc);
    prefetch_tensormap(&tm_vc);
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&bars.tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars.tmem_base;
  const uint32_t lane_off = static_cast<uint32_t>(warp * 32) << 16;
  const uint32_t tS = tmem + lane_off;          // 128 fp32 columns
  const uint32_t tP = tmem + 128 + lane_off;    // 64 columns of bf16 pairs
  const uint32_t tO = tmem + 192 + lane_off;    // 64 fp32 columns

  // tiles 0 .. n_kv_tiles-1 come from the compact K/V; tile n_kv_tiles (only with
  // the diagonal switch) is the K/V of this CTA's own query rows.
  const int n_kv = a.n_kv_tiles;
  const int n_tiles = n_kv + (a.use_diag ? 1 : 0);

  auto issue_tile = [&](int t) {   // thread 0 only
    const int s = t % kStages;
    const uint32_t kb = smem_u32(&bars.k_full[s]), vb = smem_u32(&bars.v_full[s]);
    mbar_arrive_expect_tx(kb, kTileBytes);
    mbar_arrive_expect_tx(vb, kTileBytes);
    if (t < n_kv) {
      tma_load_3d(smem_u32(sK + s * kTileBytes), &tm_kc, 0, t * kTileKV, head, kb);
      tma_load_3d(smem_u32(sV + s * kTileBytes), &tm_vc, 0, t * kTileKV, head, vb);
    } else {
      tma_load_2d(smem_u32(sK + s * kTileBytes), &tm_k, head * kHeadDim, q0, kb);
      tma_load_2d(smem_u32(sV + s * kTileBytes), &tm_v, head * kHeadDim, q0, vb);
    }
  };

  int issued = 0;
  if (tid == 0) {
    mbar_arrive_expect_tx(smem_u32(&bars.q_full), kTileBytes);
    tma_load_2d(smem_u32(sQ), &tm_q, head * kHeadDim, q0, smem_u32(&bars.q_full));
    for (; issued < kStages && issued < n_tiles; ++issued) issue_tile(issued);
  }

  const uint32_t idesc_qk = umma_idesc_bf16(kTileQ, kTileKV, false);
  const uint32_t idesc_pv = umma_idesc_bf16(kTileQ, kHeadDim, true);
  const uint64_t desc_q = umma_desc_sw128(smem_u32(sQ));

  float m_run = -INFINITY;   // running max of scale_log2 * s
  float l_run = 0.f;         // running sum of 2^(scale_log2 * s - m_run)
  bool ok = true;

  if (tid == 0) {
    ok = wait_or_abort(&bars.q_full, 0, &bars);
    if (!ok) report_timeout(a, &bars, 1, 0);
  }

  for (int j = 0; j < n_kv; ++j) {
    const int s = j % kStages;
    const uint32_t ld_parity = (j / kStages) & 1;
    // ---- S = Q Kc_j^T
    if (tid == 0 && ok) {
      ok = wait_or_abort(&bars.k_full[s], ld_parity, &bars);
      if (!ok) report_timeout(a, &bars, 2, j);
      else {
        tc_fence_after();
        const uint64_t desc_k = umma_desc_sw128(smem_u32(sK + s * kTileBytes));
#pragma unroll
        for (int k = 0; k < kHeadDim / 16; ++k) umma_ss(tmem, desc_q + (k * 32 >> 4), desc_k + (k * 32 >> 4), idesc_qk, k > 0);
        umma_commit(smem_u32(&bars.s_done));
      }
    }
    if (!wait_or_abort(&bars.s_done, j & 1, &bars)) {
      if (!*reinterpret_cast<volatile uint32_t*>(&bars.abort_flag)) report_timeout(a, &bars, 3, j);
      ok = false;
    }
    // every thread leaves the loop together: the abort flag is CTA-wide
    if (__syncthreads_or(!ok)) { ok = false; break; }
    tc_fence_after();

    // ---- online softmax on this thread's row
    uint32_t sreg[4][32];
#pragma unroll
    for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, sreg[c]);
    tmem_wait_ld();
    const int valid = static_cast<int>(pl.M - static_cast<int64_t>(j) * kTileKV);   // columns of this tile that exist
    if (valid < kTileKV) {
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (c * 32 + i >= valid) sreg[c][i] = __float_as_uint(-INFINITY);
    }
    float mx = -INFINITY;
#pragma unroll
    for (int c = 0; c < 4; ++c)
#pragma unroll
      for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(sreg[c][i]));
    const float m_new = fmaxf(m_run, mx * a.scale_log2);
    const float alpha = ex2_approx(m_run - m_new);   // 0 on the first tile
    float sum = 0.f;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      uint32_t pk[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const float p0 = ex2_approx(fmaf(__uint_as_float(sreg[c][2 * i]), a.scale_log2, -m_new));
        const float p1 = ex2_approx(fmaf(__uint_as_float(sreg[c][2 * i + 1]), a.scale_log2, -m_new));
        sum += p0 + p1;
        pk[i] = pack_bf16x2(p0, p1);
      }
      tmem_st16(tP + c * 16, pk);
    }
    l_run = fmaf(l_run, alpha, sum);
    m_run = m_new;
    // rescale the accumulator (the previous P V product has completed: o_done was waited on)
    if (j > 0 && __any_sync(0xffffffffu, alpha != 1.0f)) {
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t o[32];
        tmem_ld32(tO + c * 32, o);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
        tmem_st32(tO + c * 32, o);
      }
    }
    tmem_wait_st();
    tc_fence_before();
    __syncthreads();

    // ---- O += P Vc_j
    if (tid == 0) {
      tc_fence_after();
      ok = wait_or_abort(&bars.v_full[s], ld_parity, &bars);
      if (!ok) report_timeout(a, &bars, 4, j);
      else {
        tc_fence_after();
        const uint64_t desc_v = umma_desc_sw128(smem_u32(sV + s * kTileBytes));
#pragma unroll
        for (int k = 0; k < kTileKV / 16; ++k)
          umma_ts(tmem + 192, tmem + 128 + k * 8, desc_v + (k * 2048 >> 4), idesc_pv, (j > 0 || k > 0) ? 1u : 0u);
        umma_commit(smem_u32(&bars.o_done));
      }
    }
    if (!wait_or_abort(&bars.o_done, j & 1, &bars)) {
      if (!*reinterpret_cast<volatile uint32_t*>(&bars.abort_flag)) report_timeout(a, &bars, 5, j);
      ok = false;
    }
    if (__syncthreads_or(!ok)) { ok = false; break; }
    tc_fence_after();
    // both MMAs that read stage s have completed: refill it
    if (tid == 0 && issued < n_tiles) { issue_tile(issued); ++issued; }
  }

  // ---- epilogue: diagonal and mean-fill terms, normalisation, store
  const int row = q0 + tid;                 // this thread's query token
  const bool row_valid = row < pl.n_tok;
  bool is_dropped = false;
  if (row_valid && pl.n_dropped > 0) {
    const int32_t f = row / pl.L;
    is_dropped = compact_slot(pl, f, row - f * pl.L) < 0;
  }
  float l_d = -INFINITY, l_m = -INFINITY;   // base-2 logits of the two extra columns
  const uint8_t* sKd = sK + (n_kv % kStages) * kTileBytes;
  const uint8_t* sVd = sV + (n_kv % kStages) * kTileBytes;
  if (ok && !wait_or_abort(&bars.q_full, 0, &bars)) ok = false;   // completed long ago: makes the Q tile visible to this thread
  if (ok && a.use_diag) {
    const uint32_t par = (n_kv / kStages) & 1;
    if (!wait_or_abort(&bars.k_full[n_kv % kStages], par, &bars) || !wait_or_abort(&bars.v_full[n_kv % kStages], par, &bars)) {
      if (!*reinterpret_cast<volatile uint32_t*>(&bars.abort_flag)) report_timeout(a, &bars, 6, n_kv);
      ok = false;
    }
  }
  if (__syncthreads_or(!ok)) ok = false;

  if (ok) {
    if (a.use_diag && is_dropped) {
      float acc = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) acc = dot_bf16x8(ld_swizzled(sQ, tid, c), ld_swizzled(sKd, tid, c), acc);
      l_d = acc * a.scale_log2;
    }
    const int64_t count = pl.n_dropped - ((a.use_diag && is_dropped) ? 1 : 0);
    const bool has_mean = a.use_mean && count > 0;
    if (has_mean) {
      const float4* km = reinterpret_cast<const float4*>(a.kmean + head * kHeadDim);
      float acc = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint4 q = ld_swizzled(sQ, tid, c);
        const float4 k0 = __ldg(km + 2 * c), k1 = __ldg(km + 2 * c + 1);
        acc = fmaf(__uint_as_float(q.x << 16), k0.x, acc);
        acc = fmaf(__uint_as_float(q.x & 0xffff0000u), k0.y, acc);
        acc = fmaf(__uint_as_float(q.y << 16), k0.z, acc);
        acc = fmaf(__uint_as_float(q.y & 0xffff0000u), k0.w, acc);
        acc = fmaf(__uint_as_float(q.z << 16), k1.x, acc);
        acc = fmaf(__uint_as_float(q.z & 0xffff0000u), k1.y, acc);
        acc = fmaf(__uint_as_float(q.w << 16), k1.z, acc);
        acc = fmaf(__uint_as_float(q.w & 0xffff0000u), k1.w, acc);
      }
      l_m = acc * a.scale_log2;
      if (pl.mean_fill == AVGGT_MEAN_FILL) l_m += log2f(static_cast<float>(count));
    }
    const float m_fin = fmaxf(m_run, fmaxf(l_d, l_m));
    const float a_s = exp2f(m_run - m_fin);
    const float p_d = exp2f(l_d - m_fin);      // 0 when the term is absent
    const float p_m = exp2f(l_m - m_fin);
    const float z = fmaf(l_run, a_s, p_d + p_m);
    const float inv_z = 1.0f / z;
    const float w_s = a_s * inv_z, w_d = p_d * inv_z, w_m = p_m * inv_z;

    uint32_t o[2][32];
    tmem_ld32(tO, o[0]);
    tmem_ld32(tO + 32, o[1]);
    tmem_wait_ld();
    if (row_valid) {
      uint4* dst = reinterpret_cast<uint4*>(a.O + (static_cast<size_t>(row) * pl.H + head) * kHeadDim);
      const float4* vm = reinterpret_cast<const float4*>(a.vmean + head * kHeadDim);
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        float v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(o[c >> 2][(c & 3) * 8 + e]) * w_s;
        if (w_d != 0.f) {
          const uint4 vd = ld_swizzled(sVd, tid, c);
          const uint32_t w[4] = {vd.x, vd.y, vd.z, vd.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            v[2 * e] = fmaf(w_d, __uint_as_float(w[e] << 16), v[2 * e]);
            v[2 * e + 1] = fmaf(w_d, __uint_as_float(w[e] & 0xffff0000u), v[2 * e + 1]);
          }
        }
        if (has_mean) {
          const float4 m0 = __ldg(vm + 2 * c), m1 = __ldg(vm + 2 * c + 1);
          v[0] = fmaf(w_m, m0.x, v[0]); v[1] = fmaf(w_m, m0.y, v[1]); v[2] = fmaf(w_m, m0.z, v[2]); v[3] = fmaf(w_m, m0.w, v[3]);
          v[4] = fmaf(w_m, m1.x, v[4]); v[5] = fmaf(w_m, m1.y, v[5]); v[6] = fmaf(w_m, m1.z, v[6]); v[7] = fmaf(w_m, m1.w, v[7]);
        }
        uint4 out;
        out.x = pack_bf16x2(v[0], v[1]);
        out.y = pack_bf16x2(v[2], v[3]);
        out.z = pack_bf16x2(v[4], v[5]);
        out.w = pack_bf16x2(v[6], v[7]);
        dst[c] = out;
      }
      if (a.lse != nullptr) a.lse[static_cast<size_t>(row) * pl.H + head] = (m_fin + log2f(z)) * 0.6931471805599453f;
    }
  } else if (tid == 0) {
    // a wait gave up: let the copies this CTA still has in flight land before its shared memory is released
    for (int t = 0; t < issued; ++t) {
      (void)wait_or_abort(&bars.k_full[t % kStages], (t / kStages) & 1, &bars, false);
      (void)wait_or_abort(&bars.v_full[t % kStages], (t / kStages) & 1, &bars, false);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

constexpr size_t kAttnSmemBytes = static_cast<size_t>(kTileBytes) * (1 + 2 * kStages) + 1024;

}  // namespace

size_t global_attn_ws_bytes(const Plan&, int) { return kAttnStatusBytes; }

cudaError_t launch_global_attn(const Plan& pl, int /*sm_count*/, const void* Q, const void* K, const void* V,
                               const void* Kc, const void* Vc, const float* kmean, const float* vmean, void* O,
                               float* lse, void* ws, cudaStream_t st, bool* tmap_failed) {
  *tmap_failed = false;
  AttnArgs a;
  a.pl = pl;
  a.kmean = kmean;
  a.vmean = vmean;
  a.O = static_cast<__nv_bfloat16*>(O);
  a.lse = lse;
  a.status = static_cast<uint32_t*>(ws);
  a.n_kv_tiles = static_cast<int32_t>((pl.M + kTileKV - 1) / kTileKV);
  a.use_diag = (pl.diag != 0 && pl.n_dropped > 0) ? 1 : 0;
  a.use_mean = (pl.mean_fill != 0 && pl.n_dropped > 0) ? 1 : 0;
  a.scale_log2 = pl.scale * kLog2e;

  // token-major [n_tok, H*d] maps for Q and (diagonal tile) K, V; head-major [H, M, d] maps for Kc, Vc
  CUtensorMap tm_q, tm_k, tm_v, tm_kc, tm_vc;
  const uint64_t tok_dims[2] = {static_cast<uint64_t>(pl.H) * pl.d, static_cast<uint64_t>(pl.n_tok)};
  const uint64_t tok_str[1] = {static_cast<uint64_t>(pl.H) * pl.d * 2};
  const uint32_t tok_box[2] = {kHeadDim, kTileQ};
  const uint64_t c_dims[3] = {static_cast<uint64_t>(pl.d), static_cast<uint64_t>(pl.M), static_cast<uint64_t>(pl.H)};
  const uint64_t c_str[2] = {static_cast<uint64_t>(pl.d) * 2, static_cast<uint64_t>(pl.M) * pl.d * 2};
  const uint32_t c_box[3] = {kHeadDim, kTileKV, 1};
  bool good = make_tmap_bf16(&tm_q, Q, 2, tok_dims, tok_str, tok_box);
  good = good && make_tmap_bf16(&tm_k, a.use_diag ? K : Q, 2, tok_dims, tok_str, tok_box);
  good = good && make_tmap_bf16(&tm_v, a.use_diag ? V : Q, 2, tok_dims, tok_str, tok_box);
  good = good && make_tmap_bf16(&tm_kc, Kc, 3, c_dims, c_str, c_box);
  good = good && make_tmap_bf16(&tm_vc, Vc, 3, c_dims, c_str, c_box);
  if (!good) { *tmap_failed = true; return cudaSuccess; }

  cudaError_t e = cudaMemsetAsync(ws, 0, kAttnStatusBytes, st);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(global_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kAttnSmemBytes));
  if (e != cudaSuccess) return e;
  const dim3 grid(static_cast<unsigned>((pl.n_tok + kTileQ - 1) / kTileQ), static_cast<unsigned>(pl.H));
  global_attn_kernel<<<grid, kThreads, kAttnSmemBytes, st>>>(tm_q, tm_k, tm_v, tm_kc, tm_vc, a);
  return cudaGetLastError();
}

}  // namespace avggt
