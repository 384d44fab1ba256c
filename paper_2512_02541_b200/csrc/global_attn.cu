// Subsampled global attention (Sec. 4.3 of the AVGGT paper) as one fused,
// warp-specialised flash-style kernel for sm_100a.
//
// One CTA owns two tiles of 128 query rows of one head.  Roles:
//   warps 0-3   softmax of tile 0 (one query row per thread)
//   warps 4-7   softmax of tile 1
//   warp  8     TMA producer: Q tiles once, then the compacted K/V of the head
//               through a ring of shared-memory stages (128-byte swizzle); the
//               last two ring items are the K/V rows of the CTA's own queries
//               (the preserved diagonal)
//   warp  9     MMA issuer: S_t = Q_t Kc_j^T and O_t += P_t Vc_j with tcgen05.mma,
//               bf16 operands, fp32 accumulators in tensor memory
//   warps 10-11 idle (they complete the third warpgroup so that registers can
//               be moved to the softmax warpgroups)
// Tensor memory per tile: S 128 columns (fp32), P 64 columns (bf16 pairs),
// O 64 columns (fp32); 512 columns in all.  A softmax thread pulls its row of
// S into registers and frees S at once, so the next Q K^T runs under the
// exponentials; P V of step j runs under the softmax of step j+1.  The
// accumulator is rescaled lazily: only when the running maximum grew by more
// than 2^8 since the last rescale.  The epilogue folds the diagonal and the
// mean-fill column into the same normalisation:
//   O = (a_S O_S + p_d v_i + p_m vmean) / (a_S l_S + p_d + p_m).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "internal.h"
#include "ptx.cuh"
#include "tmap.h"

namespace avggt {

namespace {

constexpr int kTileQ = 128;      // query rows per tile
constexpr int kQTiles = 2;       // tiles per CTA
constexpr int kTileKV = 128;     // keys per step
constexpr int kHeadDim = 64;
constexpr uint32_t kTileBytes = kTileKV * kHeadDim * 2;   // 16 KiB: one 128 x 64 bf16 tile
constexpr int kStages = 3;       // K ring and V ring depth
constexpr int kThreads = 384;
constexpr int kSoftmaxWarps = 8;
constexpr int kTmaWarp = 8;
constexpr int kMmaWarp = 9;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemTileStride = 256;   // columns per query tile: S [0,128) P [128,192) O [192,256)
constexpr uint32_t kColP = 128, kColO = 192;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;   // log2 units

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
  uint64_t k_full[kStages], k_empty[kStages];
  uint64_t v_full[kStages], v_empty[kStages];
  uint64_t s_full[kQTiles];    // MMA -> softmax: S_t(j) is in tensor memory
  uint64_t s_free[kQTiles];    // softmax -> MMA: S_t(j) has been read into registers
  uint64_t p_full[kQTiles];    // softmax -> MMA: P_t(j) stored (and O_t rescaled)
  uint64_t o_done[kQTiles];    // MMA -> softmax: P_t(j) V_j has completed
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

// Bounded wait.  Returns false when the time limit ran out (the failure is
// recorded and the CTA-wide abort flag raised) or when another role aborted.
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, Barriers* bars, const AttnArgs& a,
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
        report_timeout(a, bars, where, iter);
        return false;
      }
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

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

// Optional per-phase cycle counters of the softmax loop (a tuning aid; compiled out by default).
#ifdef AVGGT_PHASE_TIMERS
__device__ unsigned long long g_phase_cycles[2][8];
struct PhaseTimers {
  unsigned long long acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  long long last = 0;
  __device__ __forceinline__ void start() { last = clock64(); }
  __device__ __forceinline__ void lap(int i) { const long long now = clock64(); acc[i] += now - last; last = now; }
};
#else
struct PhaseTimers {
  __device__ __forceinline__ void start() {}
  __device__ __forceinline__ void lap(int) {}
};
#endif

struct SmemLayout {
  uint8_t* q[kQTiles];
  uint8_t* k;   // kStages tiles
  uint8_t* v;   // kStages tiles
};

// ------------------------------------------------------------------ TMA producer (one thread)
__device__ __forceinline__ void producer_role(const CUtensorMap* tm_q, const CUtensorMap* tm_k, const CUtensorMap* tm_v,
                                              const CUtensorMap* tm_kc, const CUtensorMap* tm_vc, const AttnArgs& a,
                                              Barriers* bars, const SmemLayout& sm, int head, int q0) {
  const int n_kv = a.n_kv_tiles;
  const int n_items = n_kv + (a.use_diag ? kQTiles : 0);
  mbar_arrive_expect_tx(smem_u32(&bars->q_full), kQTiles * kTileBytes);
#pragma unroll
  for (int t = 0; t < kQTiles; ++t)
    tma_load_2d(smem_u32(sm.q[t]), tm_q, head * kHeadDim, q0 + t * kTileQ, smem_u32(&bars->q_full));
  int it = 0;
  bool ok = true;
  for (; it < n_items; ++it) {
    const int s = it % kStages;
    const uint32_t round = static_cast<uint32_t>(it / kStages);
    // a fresh barrier passes the wait on the "previous" phase at once
    ok = wait_bar(&bars->k_empty[s], (round & 1) ^ 1, bars, a, 10, it);
    if (!ok) break;
    const uint32_t kb = smem_u32(&bars->k_full[s]);
    mbar_arrive_expect_tx(kb, kTileBytes);
    if (it < n_kv) tma_load_3d(smem_u32(sm.k + s * kTileBytes), tm_kc, 0, it * kTileKV, head, kb);
    else tma_load_2d(smem_u32(sm.k + s * kTileBytes), tm_k, head * kHeadDim, q0 + (it - n_kv) * kTileQ, kb);
    ok = wait_bar(&bars->v_empty[s], (round & 1) ^ 1, bars, a, 11, it);
    if (!ok) break;
    const uint32_t vb = smem_u32(&bars->v_full[s]);
    mbar_arrive_expect_tx(vb, kTileBytes);
    if (it < n_kv) tma_load_3d(smem_u32(sm.v + s * kTileBytes), tm_vc, 0, it * kTileKV, head, vb);
    else tma_load_2d(smem_u32(sm.v + s * kTileBytes), tm_v, head * kHeadDim, q0 + (it - n_kv) * kTileQ, vb);
  }
  if (!ok) {
    // let the copies still in flight land before the CTA gives up its shared memory
    (void)wait_bar(&bars->q_full, 0, bars, a, 12, 0, false);
    for (int back = 1; back <= kStages && it - back >= 0; ++back) {
      const int jt = it - back;
      (void)wait_bar(&bars->k_full[jt % kStages], (jt / kStages) & 1, bars, a, 12, jt, false);
      (void)wait_bar(&bars->v_full[jt % kStages], (jt / kStages) & 1, bars, a, 12, jt, false);
    }
  }
}

// ------------------------------------------------------------------ MMA issuer (one thread)
__device__ __forceinline__ void mma_role(const AttnArgs& a, Barriers* bars, const SmemLayout& sm, uint32_t tmem) {
  const int n_kv = a.n_kv_tiles;
  const uint32_t idesc_qk = umma_idesc_bf16(kTileQ, kTileKV, false);
  const uint32_t idesc_pv = umma_idesc_bf16(kTileQ, kHeadDim, true);
  uint64_t desc_q[kQTiles];
#pragma unroll
  for (int t = 0; t < kQTiles; ++t) desc_q[t] = umma_desc_sw128(smem_u32(sm.q[t]));

  auto issue_qk = [&](int t, int j) {
    const uint64_t desc_k = umma_desc_sw128(smem_u32(sm.k + (j % kStages) * kTileBytes));
#pragma unroll
    for (int k = 0; k < kHeadDim / 16; ++k)
      umma_ss(tmem + t * kTmemTileStride, desc_q[t] + (k * 32 >> 4), desc_k + (k * 32 >> 4), idesc_qk, k > 0);
    umma_commit(smem_u32(&bars->s_full[t]));
  };
  auto issue_pv = [&](int t, int j) {
    const uint64_t desc_v = umma_desc_sw128(smem_u32(sm.v + (j % kStages) * kTileBytes));
#pragma unroll
    for (int k = 0; k < kTileKV / 16; ++k)
      umma_ts(tmem + t * kTmemTileStride + kColO, tmem + t * kTmemTileStride + kColP + k * 8, desc_v + (k * 2048 >> 4),
              idesc_pv, (j > 0 || k > 0) ? 1u : 0u);
    umma_commit(smem_u32(&bars->o_done[t]));
  };

  if (!wait_bar(&bars->q_full, 0, bars, a, 20, 0)) return;
  if (!wait_bar(&bars->k_full[0], 0, bars, a, 21, 0)) return;
  tc_fence_after();
#pragma unroll
  for (int t = 0; t < kQTiles; ++t) issue_qk(t, 0);
  umma_commit(smem_u32(&bars->k_empty[0]));

  // Event loop: issue whichever product has its operands ready.  Per tile, Q K^T of step j
  // needs S_t free (softmax read step j-1) and K_j; P V of step j needs P_t(j) and V_j.
  // No barrier polled here can be more than one phase ahead of the step it is polled for.
  static_assert(kQTiles == 2, "the issue loop below is written for two query tiles");
  int qk0 = 1, qk1 = 1, pv0 = 0, pv1 = 0;   // next step to issue, per tile
  uint64_t t_idle = 0;
  uint32_t idle_polls = 0;
  bool progressed;
  auto poll_tile = [&](int t, int& qk_mine, int& pv_mine, const int& qk_other, const int& pv_other) {
    const int jq = qk_mine;
    if (jq < n_kv && mbar_test_wait(smem_u32(&bars->s_free[t]), (jq - 1) & 1) &&
        mbar_test_wait(smem_u32(&bars->k_full[jq % kStages]), (jq / kStages) & 1)) {
      tc_fence_after();
      issue_qk(t, jq);
      qk_mine = jq + 1;
      if (qk_other > jq) umma_commit(smem_u32(&bars->k_empty[jq % kStages]));   // both tiles have read K_jq
      progressed = true;
    }
    const int jp = pv_mine;
    if (jp < n_kv && mbar_test_wait(smem_u32(&bars->p_full[t]), jp & 1) &&
        mbar_test_wait(smem_u32(&bars->v_full[jp % kStages]), (jp / kStages) & 1)) {
      tc_fence_after();
      issue_pv(t, jp);
      pv_mine = jp + 1;
      if (pv_other > jp) umma_commit(smem_u32(&bars->v_empty[jp % kStages]));   // both tiles have read V_jp
      progressed = true;
    }
  };
  while (true) {
    progressed = false;
    poll_tile(0, qk0, pv0, qk1, pv1);
    poll_tile(1, qk1, pv1, qk0, pv0);
    const bool finished = pv0 >= n_kv && pv1 >= n_kv;
    if (finished) break;
    if (progressed) { idle_polls = 0; continue; }
    if ((++idle_polls & 0xffu) == 0) {
      if (*reinterpret_cast<volatile uint32_t*>(&bars->abort_flag)) return;
      const uint64_t now = globaltimer_ns();
      if (idle_polls == 0x100u) t_idle = now;
      else if (now - t_idle > AVGGT_WAIT_LIMIT_NS) { report_timeout(a, bars, 26, pv0); return; }
    }
  }
}

// ------------------------------------------------------------------ softmax warpgroup (128 threads per tile)
// kLse: also keep the sum of the unrounded exponentials, for the log-sum-exp output.
template <bool kMasked, bool kLse>
__device__ __forceinline__ void softmax_step(uint32_t tS, uint32_t tP, uint32_t tO, int j, int valid, float scale_log2,
                                             float& m_used, float& l_run, float& l_exact, Barriers* bars,
                                             const AttnArgs& a, int t, int lane, bool& ok, PhaseTimers& pt) {
  uint32_t s[4][32];
  tmem_ld32(tS, s[0]);
  tmem_ld32(tS + 32, s[1]);
  tmem_ld32(tS + 64, s[2]);
  tmem_ld32(tS + 96, s[3]);
  tmem_wait_ld();
  tc_fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive(smem_u32(&bars->s_free[t]));
  pt.lap(1);

  if (kMasked) {
#pragma unroll
    for (int i = 0; i < 128; ++i)
      if (i >= valid) s[i >> 5][i & 31] = __float_as_uint(-INFINITY);
  }
  float mx[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    mx[c] = fmaxf(__uint_as_float(s[c][0]), __uint_as_float(s[c][1]));
#pragma unroll
    for (int i = 2; i < 32; i += 2) mx[c] = max3(mx[c], __uint_as_float(s[c][i]), __uint_as_float(s[c][i + 1]));
  }
  const float tile_max = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * scale_log2;
  // lazy rescale: keep the old reference maximum unless the new one is far above it
  const bool jump = tile_max > m_used + kRescaleThreshold;
  float alpha = 1.0f;
  if (jump) {
    alpha = ex2_approx(m_used - tile_max);   // 0 on the first tile (m_used = -inf)
    m_used = tile_max;
    l_run *= alpha;
    if (kLse) l_exact *= alpha;
  }
  const bool rescale = (j > 0) && __any_sync(0xffffffffu, jump);
  pt.lap(2);

  // exponentials, rounded to bf16 for the value product; the normaliser sums the
  // rounded values so that numerator and denominator carry the same weights
  const float neg_m = -m_used;
  float sum0 = 0.f, sum1 = 0.f, sum_exact = 0.f;
  uint32_t pk[4][16];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float p0 = ex2_approx(fmaf(__uint_as_float(s[c][2 * i]), scale_log2, neg_m));
      const float p1 = ex2_approx(fmaf(__uint_as_float(s[c][2 * i + 1]), scale_log2, neg_m));
      const uint32_t w = pack_bf16x2(p0, p1);
      pk[c][i] = w;
      if (kLse) sum_exact += p0 + p1;
      sum0 += __uint_as_float(w << 16);
      sum1 += __uint_as_float(w & 0xffff0000u);
    }
  }

  pt.lap(3);
  // P_t(j-1) must have been consumed, and O_t be at rest, before either is written
  if (j > 0) {
    if (!wait_bar(&bars->o_done[t], (j - 1) & 1, bars, a, 30 + t, j)) { ok = false; return; }
    tc_fence_after();
  }
  pt.lap(4);
  if (rescale) {
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
#pragma unroll
  for (int c = 0; c < 4; ++c) tmem_st16(tP + c * 16, pk[c]);
  l_run += sum0 + sum1;
  if (kLse) l_exact += sum_exact;
  tmem_wait_st();
  tc_fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive(smem_u32(&bars->p_full[t]));
  pt.lap(5);
}

__device__ __forceinline__ void softmax_role(const AttnArgs& a, Barriers* bars, const SmemLayout& sm, uint32_t tmem,
                                             int t, int wg_tid, int head, int q0) {
  const Plan& pl = a.pl;
  const int n_kv = a.n_kv_tiles;
  const int lane = wg_tid & 31;
  const uint32_t lane_off = static_cast<uint32_t>(wg_tid & ~31) << 16;   // TMEM lane = row within the tile
  const uint32_t tS = tmem + t * kTmemTileStride + lane_off;
  const uint32_t tP = tS + kColP, tO = tS + kColO;
  float m_used = -INFINITY;   // reference maximum of the stored exponentials (log2 units)
  float l_run = 0.f;          // sum of the bf16-rounded 2^(scale_log2 * s - m_used): normaliser of O
  float l_exact = 0.f;        // the same sum without the rounding: log-sum-exp output only
  const bool want_lse = a.lse != nullptr;
  bool ok = true;
  PhaseTimers pt;
  pt.start();

  for (int j = 0; j < n_kv && ok; ++j) {
    if (!wait_bar(&bars->s_full[t], j & 1, bars, a, 40 + t, j)) { ok = false; break; }
    tc_fence_after();
    pt.lap(0);
    const int valid = static_cast<int>(pl.M - static_cast<int64_t>(j) * kTileKV);
    if (valid < kTileKV) softmax_step<true, true>(tS, tP, tO, j, valid, a.scale_log2, m_used, l_run, l_exact, bars, a, t, lane, ok, pt);
    else if (want_lse) softmax_step<false, true>(tS, tP, tO, j, valid, a.scale_log2, m_used, l_run, l_exact, bars, a, t, lane, ok, pt);
    else softmax_step<false, false>(tS, tP, tO, j, valid, a.scale_log2, m_used, l_run, l_exact, bars, a, t, lane, ok, pt);
  }
  if (!ok) return;
#ifdef AVGGT_PHASE_TIMERS
  if (blockIdx.x == 0 && blockIdx.y == 0 && wg_tid == 0)
    for (int i = 0; i < 8; ++i) g_phase_cycles[t][i] = pt.acc[i];
#endif

  // ---- epilogue: diagonal and mean-fill terms, normalisation, store
  const int r = wg_tid;                              // row within the tile
  const int row = q0 + t * kTileQ + r;               // query token
  const bool row_valid = row < pl.n_tok;
  bool is_dropped = false;
  if (row_valid && pl.n_dropped > 0) {
    const int32_t f = row / pl.L;
    is_dropped = compact_slot(pl, f, row - f * pl.L) < 0;
  }
  if (!wait_bar(&bars->o_done[t], (n_kv - 1) & 1, bars, a, 50 + t, n_kv)) return;
  tc_fence_after();
  if (!wait_bar(&bars->q_full, 0, bars, a, 52, 0)) return;   // completed long ago: makes the Q tile visible to this thread
  const int item = n_kv + t;                         // ring item holding this tile's own K/V rows
  const uint8_t* sKd = sm.k + (item % kStages) * kTileBytes;
  const uint8_t* sVd = sm.v + (item % kStages) * kTileBytes;
  if (a.use_diag) {
    const uint32_t par = (item / kStages) & 1;
    if (!wait_bar(&bars->k_full[item % kStages], par, bars, a, 53, item)) return;
    if (!wait_bar(&bars->v_full[item % kStages], par, bars, a, 54, item)) return;
  }
  const uint8_t* sQ = sm.q[t];
  float l_d = -INFINITY, l_m = -INFINITY;            // base-2 logits of the two extra columns
  if (a.use_diag && is_dropped) {
    float acc = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) acc = dot_bf16x8(ld_swizzled(sQ, r, c), ld_swizzled(sKd, r, c), acc);
    l_d = acc * a.scale_log2;
  }
  const int64_t count = pl.n_dropped - ((a.use_diag && is_dropped) ? 1 : 0);
  const bool has_mean = a.use_mean && count > 0;
  if (has_mean) {
    const float4* km = reinterpret_cast<const float4*>(a.kmean + head * kHeadDim);
    float acc = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const uint4 q = ld_swizzled(sQ, r, c);
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
  const float m_fin = fmaxf(m_used, fmaxf(l_d, l_m));
  const float a_s = exp2f(m_used - m_fin);
  const float p_d = exp2f(l_d - m_fin);              // 0 when the term is absent
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
        const uint4 vd = ld_swizzled(sVd, r, c);
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
    if (want_lse) {
      const float z_exact = fmaf(l_exact, a_s, p_d + p_m);
      a.lse[static_cast<size_t>(row) * pl.H + head] = (m_fin + log2f(z_exact)) * 0.6931471805599453f;
    }
  }
}

__global__ void __launch_bounds__(kThreads, 1)
global_attn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_kc,
                   const __grid_constant__ CUtensorMap tm_vc, const AttnArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  SmemLayout sm;
  sm.q[0] = smem;
  sm.q[1] = smem + kTileBytes;
  sm.k = smem + kQTiles * kTileBytes;
  sm.v = sm.k + kStages * kTileBytes;
  __shared__ Barriers bars;

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int head = blockIdx.y;
  const int q0 = blockIdx.x * (kQTiles * kTileQ);

  if (tid == 0) {
    mbar_init(smem_u32(&bars.q_full), 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&bars.k_full[s]), 1);
      mbar_init(smem_u32(&bars.k_empty[s]), 1);
      mbar_init(smem_u32(&bars.v_full[s]), 1);
      mbar_init(smem_u32(&bars.v_empty[s]), 1);
    }
    for (int t = 0; t < kQTiles; ++t) {
      mbar_init(smem_u32(&bars.s_full[t]), 1);
      mbar_init(smem_u32(&bars.s_free[t]), 4);
      mbar_init(smem_u32(&bars.p_full[t]), 4);
      mbar_init(smem_u32(&bars.o_done[t]), 1);
    }
    bars.abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == kTmaWarp) {
    tmem_alloc(smem_u32(&bars.tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars.tmem_base;

  if (warp < kSoftmaxWarps) {
    reg_inc<224>();
    const int t = warp >> 2;
    softmax_role(a, &bars, sm, tmem, t, tid & 127, head, q0);
  } else {
    reg_dec<56>();
    if (warp == kTmaWarp) {
      if ((tid & 31) == 0) {
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_kc);
        prefetch_tensormap(&tm_vc);
        producer_role(&tm_q, &tm_k, &tm_v, &tm_kc, &tm_vc, a, &bars, sm, head, q0);
      }
    } else if (warp == kMmaWarp) {
      if ((tid & 31) == 0) mma_role(a, &bars, sm, tmem);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kTmaWarp) tmem_dealloc(tmem, kTmemCols);
}

constexpr size_t kAttnSmemBytes = static_cast<size_t>(kTileBytes) * (kQTiles + 2 * kStages) + 1024;

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

  // token-major [n_tok, H*d] maps for Q and (diagonal tiles) K, V; head-major [H, M, d] maps for Kc, Vc
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
  const int rows_per_cta = kQTiles * kTileQ;
  const dim3 grid(static_cast<unsigned>((pl.n_tok + rows_per_cta - 1) / rows_per_cta), static_cast<unsigned>(pl.H));
  global_attn_kernel<<<grid, kThreads, kAttnSmemBytes, st>>>(tm_q, tm_k, tm_v, tm_kc, tm_vc, a);
  return cudaGetLastError();
}

}  // namespace avggt
