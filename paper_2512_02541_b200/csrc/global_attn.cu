// Subsampled global attention (Sec. 4.3 of the AVGGT paper) as one fused,
// warp-specialised flash-style kernel for sm_100a; the same kernel runs frame
// attention (Sec. 4.2) as many small dense problems.
//
// A work item is two tiles of 128 query rows of one head.  In the subsampled
// layer a CTA has one work item (hundreds of key steps); in frame attention one
// CTA per SM walks over many (a dozen key steps each), so that the next item's
// loads and first product run under the current item's epilogue.
// Roles (20 warps):
//   warps 0-15  softmax.  Warp 8 t + 4 h + q works on query tile t, rows
//               [32 q + 16 h, 32 q + 16 h + 16), all 128 columns of a key step.
//               It reads tensor memory in the 16-lane shapes, which spread a row
//               over the four threads of a quad (two rows per thread): a row's
//               maximum and sums are two shuffles away and every row lives in one
//               warp.  Four softmax warps per scheduler keep the exponential unit
//               busy while others wait on tensor memory or barriers.
//   warp  16    TMA producer: Q tiles once per work item, then the compacted K/V
//               of the head through a ring of shared-memory stages (128-byte
//               swizzle); in the subsampled layer the last two ring items are the
//               K/V rows of the CTA's own queries (the preserved diagonal)
//   warps 17-18 MMA issuers, one per query tile: S_t = Q_t Kc_j^T and
//               O_t += P_t Vc_j with tcgen05.mma, bf16 operands, fp32
//               accumulators in tensor memory
//   warp  19    idle (it completes the fifth warpgroup so that registers can
//               be moved to the softmax warpgroups)
// Tensor memory per tile: S 128 columns (fp32), P 64 columns (bf16 pairs),
// O 64 columns (fp32); 512 columns in all.  A softmax thread pulls its 64 scores
// of S into registers and the warp frees its rows at once, so the next Q K^T runs
// under the exponentials; P V of step j runs under the softmax of step j+1.  One
// block of 8 key columns in eight takes its exponentials from a polynomial on
// the FMA pipe.  The accumulator is rescaled lazily: only when the running
// maximum grew by more than 2^8 since the last rescale.  The epilogue folds the
// diagonal and the mean-fill column into the same normalisation:
//   O = (a_S O_S + p_d v_i + p_m vmean) / (a_S l_S + p_d + p_m).
#include <mutex>

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
// K ring and V ring depth.  The subsampled layer runs the same at 2 to 5; frame attention, whose strided key
// tiles take longer to arrive, gained 6 % from the fourth stage and nothing from a fifth.
#ifndef AVGGT_STAGES
#define AVGGT_STAGES 4
#endif
constexpr int kStages = AVGGT_STAGES;
constexpr int kThreads = 640;
constexpr int kSoftmaxWarps = 16;
constexpr int kTmaWarp = 16;
constexpr int kMmaWarp = 17;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemTileStride = 256;   // columns per query tile: S [0,128) P [128,192) O [192,256)
constexpr uint32_t kColP = 128, kColO = 192;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;   // log2 units

// Of every 8 blocks of 8 key columns, this many take their exponentials from a polynomial on the FMA pipe instead of
// the special-function unit (which, at 16 results per clock per SM, is the scarcest arithmetic unit of the softmax at
// head dimension 64).  One in eight measured best: 723 ms on the 800-frame layer against 768 ms with none and 767 ms
// with two in eight.
#ifndef AVGGT_POLY_EIGHTHS
#define AVGGT_POLY_EIGHTHS 1
#endif
constexpr int kPolyEighths = AVGGT_POLY_EIGHTHS;

struct AttnArgs {
  Plan pl;
  const float* kmean;   // [H, d] or null
  const float* vmean;
  __nv_bfloat16* O;     // [n_tok, H, d]
  float* lse;           // [n_tok, H] or null
  const int32_t* slot_of_token;   // caller-chosen retained set: compact position of every token, -1 = dropped; else null
  uint32_t* status;     // 4 words
  int32_t frame_mode;   // 0: subsampled global attention over the compact keys.  1: frame attention (Sec. 4.2):
                        //    every frame is a problem of its own, keys and values are the frame's own rows of K and V
  int64_t n_keys;       // keys of one problem: M, or the tokens of a frame
  int32_t n_kv_tiles;   // ceil(n_keys / 128)
  int32_t n_work;       // work items (pairs of query tiles x heads x problems) of the launch; a CTA takes the items
                        // blockIdx.x, blockIdx.x + gridDim.x, ...  (more than one per CTA only in frame attention)
  int32_t pairs;        // pairs of query tiles of one problem
  int32_t use_diag;     // diag on and |D| > 0
  int32_t use_mean;     // mean_fill on and |D| > 0
  float scale_log2;     // softmax scale * log2(e)
};

struct __align__(8) Barriers {
  uint64_t q_full;             // producer -> all: the work item's Q tiles are in shared memory
  uint64_t q_empty;            // MMA issuers -> producer: every Q K^T of the work item has completed, Q may be overwritten
  uint64_t o_free[kQTiles];    // softmax -> MMA: O_t of the finished work item has been read out
  uint64_t k_full[kStages], k_empty[kStages];
  uint64_t v_full[kStages], v_empty[kStages];
  uint64_t s_full[kQTiles];    // MMA -> softmax: S_t(j) is in tensor memory
  uint64_t s_free[kQTiles];    // softmax -> MMA: S_t(j) has been read into registers
  uint64_t p_full[kQTiles];    // softmax -> MMA: P_t(j) stored (and O_t rescaled)
  uint64_t o_done[kQTiles];    // MMA -> softmax: P_t(j) V_j has completed
  uint64_t mma_idle[kQTiles];  // MMA issuer t -> itself: every tcgen05.mma it issued has completed
  uint32_t tmem_base;
  uint32_t abort_flag;
};

__device__ __forceinline__ void report_timeout(const AttnArgs& a, Barriers* bars, uint32_t where, uint32_t iter) {
  if (atomicCAS(a.status, 0u, 1u) == 0u) {
    a.status[1] = blockIdx.x;
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

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Register budget per thread after the roles have split.  The sum over all warps must not
// exceed what the launch allocated (96 x 640): a setmaxnreg.inc that asks for more than the
// pool can ever hold waits for ever, and that wait has no time limit.
constexpr int kRegsLaunch = 96;   // 65536 / 640 threads, rounded down to the allocation unit
constexpr int kRegsSoftmax = 112, kRegsOther = 32;
static_assert(kRegsSoftmax * kSoftmaxWarps + kRegsOther * (kThreads / 32 - kSoftmaxWarps) <= kRegsLaunch * (kThreads / 32),
              "register budget after setmaxnreg exceeds the launch allocation");
template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

// What one CTA works on.
struct CtaProblem {
  int head;
  int q0;             // first query row (token index) of the CTA's two tiles
  int64_t row_end;    // query rows at or beyond this token index are not stored
  int key_row0;       // frame attention: token index of the frame's first key
};

// Work item -> problem.  Items are numbered with the pair of query tiles fastest, then the head, then (frame
// attention) the frame, so that the CTAs running side by side share one head's keys in L2.
__device__ __forceinline__ CtaProblem work_item(const AttnArgs& a, int item) {
  CtaProblem c;
  const int qp = item % a.pairs;
  const int rest = item / a.pairs;
  c.head = rest % a.pl.H;
  if (a.frame_mode) {
    c.key_row0 = (rest / a.pl.H) * a.pl.L;
    c.q0 = c.key_row0 + qp * (kQTiles * kTileQ);
    c.row_end = static_cast<int64_t>(c.key_row0) + a.pl.L;
  } else {
    c.key_row0 = 0;
    c.q0 = qp * (kQTiles * kTileQ);
    c.row_end = a.pl.n_tok;
  }
  return c;
}

struct SmemLayout {
  uint8_t* q[kQTiles];
  uint8_t* k;   // kStages tiles
  uint8_t* v;   // kStages tiles
};

// The producer and the MMA issuers run with all 32 lanes of their warp in step (every branch
// condition is made warp-uniform with a vote) and issue the TMA / tcgen05 instructions from one
// elected lane.  Those instructions take their operands from the uniform datapath; issued from
// divergent single-lane code they fall on a slow path that costs on the order of 100 clocks each.
constexpr uint32_t kFullMask = 0xffffffffu;

__device__ __forceinline__ bool wait_bar_warp(uint64_t* bar, uint32_t parity, Barriers* bars, const AttnArgs& a,
                                              uint32_t where, uint32_t iter, bool check_abort = true) {
  return __all_sync(kFullMask, wait_bar(bar, parity, bars, a, where, iter, check_abort));
}

// ------------------------------------------------------------------ TMA producer (one warp)
__device__ __forceinline__ void producer_role(const CUtensorMap* tm_q, const CUtensorMap* tm_k, const CUtensorMap* tm_v,
                                              const CUtensorMap* tm_kc, const CUtensorMap* tm_vc, const AttnArgs& a,
                                              Barriers* bars, const SmemLayout& sm) {
  const int n_kv = a.n_kv_tiles;
  const int n_ring = n_kv + (a.use_diag ? kQTiles : 0);   // ring items of one work item
  if (elect_one()) {
    prefetch_tensormap(tm_q);
    prefetch_tensormap(tm_kc);
    prefetch_tensormap(tm_vc);
  }
  int k_issued = 0, v_issued = 0;   // K / V copies issued so far, over all work items
  int stage = 0;
  uint32_t empty_parity = 1;   // a fresh barrier passes the wait on the "previous" phase at once
  bool ok = true;
  int n_done = 0;              // work items completed by this role
  int q_issued = 0;            // work items whose Q copies have been issued
  for (int item = blockIdx.x; item < a.n_work && ok; item += gridDim.x, ++n_done) {
    const CtaProblem cta = work_item(a, item);
    const int head = cta.head, q0 = cta.q0;
    // the Q tiles of the previous work item are no longer read by any Q K^T
    if (n_done > 0) {
      ok = wait_bar_warp(&bars->q_empty, (n_done - 1) & 1, bars, a, 14, n_done);
      if (!ok) break;
    }
    if (elect_one()) {
      mbar_arrive_expect_tx(smem_u32(&bars->q_full), kQTiles * kTileBytes);
#pragma unroll
      for (int t = 0; t < kQTiles; ++t)
        tma_load_2d(smem_u32(sm.q[t]), tm_q, head * kHeadDim, q0 + t * kTileQ, smem_u32(&bars->q_full));
    }
    __syncwarp();
    ++q_issued;
    for (int it = 0; it < n_ring; ++it) {
      ok = wait_bar_warp(&bars->k_empty[stage], empty_parity, bars, a, 10, it);
      if (!ok) break;
#ifdef AVGGT_TEST_SKIP_K_LOAD
      // Build for the wait-limit test only (never part of libavggt.so): the first thread block leaves out one K
      // tile, so that the waits on it run out, the block reports the time-out and every role leaves in order.
      const bool skip_load = it == AVGGT_TEST_SKIP_K_LOAD && n_done == 0 && blockIdx.x == 0;
#else
      constexpr bool skip_load = false;
#endif
      if (elect_one() && !skip_load) {
        const uint32_t kb = smem_u32(&bars->k_full[stage]);
        mbar_arrive_expect_tx(kb, kTileBytes);
        if (a.frame_mode) tma_load_2d(smem_u32(sm.k + stage * kTileBytes), tm_k, head * kHeadDim, cta.key_row0 + it * kTileKV, kb);
        else if (it < n_kv) tma_load_3d(smem_u32(sm.k + stage * kTileBytes), tm_kc, 0, it * kTileKV, head, kb);
        else tma_load_2d(smem_u32(sm.k + stage * kTileBytes), tm_k, head * kHeadDim, q0 + (it - n_kv) * kTileQ, kb);
      }
      __syncwarp();
      ++k_issued;
      ok = wait_bar_warp(&bars->v_empty[stage], empty_parity, bars, a, 11, it);
      if (!ok) break;
      if (elect_one()) {
        const uint32_t vb = smem_u32(&bars->v_full[stage]);
        mbar_arrive_expect_tx(vb, kTileBytes);
        if (a.frame_mode) tma_load_2d(smem_u32(sm.v + stage * kTileBytes), tm_v, head * kHeadDim, cta.key_row0 + it * kTileKV, vb);
        else if (it < n_kv) tma_load_3d(smem_u32(sm.v + stage * kTileBytes), tm_vc, 0, it * kTileKV, head, vb);
        else tma_load_2d(smem_u32(sm.v + stage * kTileBytes), tm_v, head * kHeadDim, q0 + (it - n_kv) * kTileQ, vb);
      }
      __syncwarp();
      ++v_issued;
      if (++stage == kStages) { stage = 0; empty_parity ^= 1; }
    }
  }
  if (!ok) {
    // let the copies still in flight land before the CTA gives up its shared memory: the Q tiles of the last work
    // item begun, and the last kStages issued into either ring (earlier ones completed before their stage was reused)
    if (q_issued > 0) (void)wait_bar_warp(&bars->q_full, (q_issued - 1) & 1, bars, a, 12, 0, false);
    for (int back = 1; back <= kStages; ++back) {
      const int jk = k_issued - back, jv = v_issued - back;
      if (jk >= 0) (void)wait_bar_warp(&bars->k_full[jk % kStages], (jk / kStages) & 1, bars, a, 12, jk, false);
      if (jv >= 0) (void)wait_bar_warp(&bars->v_full[jv % kStages], (jv / kStages) & 1, bars, a, 13, jv, false);
    }
  }
}

// ------------------------------------------------------------------ MMA issuer (one warp per query tile)
// Per tile the order of events is fixed: S_t(j) is read by the softmax (s_free) before P_t(j) is
// stored (p_full), which precedes the read of S_t(j+1).  The issuer of tile t therefore waits, in
// turn, for "S_t free and K_{j+1} loaded" -> Q K^T of step j+1, then "P_t(j) stored and V_j
// loaded" -> P V of step j.  A K or V stage is released when both tiles' issuers have committed
// their product on it (the empty barriers count two arrivals).
template <int t>
__device__ __forceinline__ void issue_qk(const AttnArgs& a, Barriers* bars, uint32_t tmem, uint64_t desc_q, uint32_t k_base,
                                         int stage, int j) {
  if (elect_one()) {
    constexpr uint32_t idesc = umma_idesc_bf16(kTileQ, kTileKV, false);
    const uint64_t desc_k = umma_desc_sw128(k_base + stage * kTileBytes);
#pragma unroll
    for (int k = 0; k < kHeadDim / 16; ++k)
      umma_ss(tmem + t * kTmemTileStride, desc_q + (k * 32 >> 4), desc_k + (k * 32 >> 4), idesc, k > 0);
    umma_commit(smem_u32(&bars->s_full[t]));
    umma_commit(smem_u32(&bars->k_empty[stage]));
  }
  __syncwarp();
}

template <int t>
__device__ __forceinline__ void issue_pv(const AttnArgs& a, Barriers* bars, uint32_t tmem, uint32_t v_base, int stage, int j) {
  if (elect_one()) {
    constexpr uint32_t idesc = umma_idesc_bf16(kTileQ, kHeadDim, true);
    const uint64_t desc_v = umma_desc_sw128(v_base + stage * kTileBytes);
#pragma unroll
    for (int k = 0; k < kTileKV / 16; ++k)
      umma_ts(tmem + t * kTmemTileStride + kColO, tmem + t * kTmemTileStride + kColP + k * 8, desc_v + (k * 2048 >> 4),
              idesc, (j > 0 || k > 0) ? 1u : 0u);
    umma_commit(smem_u32(&bars->o_done[t]));
    umma_commit(smem_u32(&bars->v_empty[stage]));
  }
  __syncwarp();
}

template <int t>
__device__ __forceinline__ void mma_issue_loop(const AttnArgs& a, Barriers* bars, const SmemLayout& sm, uint32_t tmem) {
  static_assert(kStages >= 2, "the K ring must hold the tile in use and the next one");
  const int n_kv = a.n_kv_tiles;
  const uint64_t desc_q = umma_desc_sw128(smem_u32(sm.q[t]));
  const uint32_t k_base = smem_u32(sm.k), v_base = smem_u32(sm.v);
  if (n_kv == 0) return;   // no retained keys: the epilogue's two extra columns are the whole layer

  // Running over all work items of the CTA: the ring positions of the next K and V tile, and g, the number of key
  // steps of this tile so far (the phase of the per-step barriers).  The rings carry the work item's own rows
  // (the diagonal) only in the subsampled layer, where a CTA has one work item.
  int k_stage = 0, v_stage = 0;
  uint32_t k_parity = 0, v_parity = 0;   // parity of their "full" phase
  int g = 0;
  int n_done = 0;
  for (int item = blockIdx.x; item < a.n_work; item += gridDim.x, ++n_done, g += n_kv) {
    if (!wait_bar_warp(&bars->q_full, n_done & 1, bars, a, 20, n_done)) return;
    // first product of the work item: S_t must have been read by the softmax of the previous item's last step
    if (n_done > 0 && !wait_bar_warp(&bars->s_free[t], (g - 1) & 1, bars, a, 22 + t, g - 1)) return;
    if (!wait_bar_warp(&bars->k_full[k_stage], k_parity, bars, a, 21, g)) return;
    tc_fence_after();
    issue_qk<t>(a, bars, tmem, desc_q, k_base, k_stage, 0);
    if (++k_stage == kStages) { k_stage = 0; k_parity ^= 1; }
    for (int j = 0; j < n_kv; ++j) {
      if (j + 1 < n_kv) {
        if (!wait_bar_warp(&bars->s_free[t], (g + j) & 1, bars, a, 22 + t, g + j)) return;
        if (!wait_bar_warp(&bars->k_full[k_stage], k_parity, bars, a, 24 + t, g + j)) return;
        tc_fence_after();
        issue_qk<t>(a, bars, tmem, desc_q, k_base, k_stage, j + 1);
        if (++k_stage == kStages) { k_stage = 0; k_parity ^= 1; }
      } else {
        // every Q K^T of this work item has been issued: when they have completed, Q may be overwritten
        if (elect_one()) umma_commit(smem_u32(&bars->q_empty));
        __syncwarp();
      }
      if (!wait_bar_warp(&bars->p_full[t], (g + j) & 1, bars, a, 26 + t, g + j)) return;
      if (!wait_bar_warp(&bars->v_full[v_stage], v_parity, bars, a, 28 + t, g + j)) return;
      // the first P V of a work item overwrites O_t: the previous item's epilogue must have read it out
      if (j == 0 && n_done > 0 && !wait_bar_warp(&bars->o_free[t], (n_done - 1) & 1, bars, a, 29, n_done)) return;
      tc_fence_after();
      issue_pv<t>(a, bars, tmem, v_base, v_stage, j);
      if (++v_stage == kStages) { v_stage = 0; v_parity ^= 1; }
    }
    // ring positions of the work item's own K/V rows (read by the softmax epilogue, not by any product)
    if (a.use_diag) {
      for (int i = 0; i < kQTiles; ++i) {
        if (++k_stage == kStages) { k_stage = 0; k_parity ^= 1; }
        if (++v_stage == kStages) { v_stage = 0; v_parity ^= 1; }
      }
    }
  }
}

// The issue loop, then (on every path out of it, a wait that ran out included) a wait until the
// tensor core has finished everything this warp issued: the CTA must not free its tensor memory
// or leave its shared memory while a tcgen05.mma still reads or writes them.
template <int t>
__device__ __forceinline__ void mma_role(const AttnArgs& a, Barriers* bars, const SmemLayout& sm, uint32_t tmem) {
  mma_issue_loop<t>(a, bars, sm, tmem);
  __syncwarp();
  if (elect_one()) umma_commit(smem_u32(&bars->mma_idle[t]));
  __syncwarp();
  (void)wait_bar_warp(&bars->mma_idle[t], 0, bars, a, 70 + t, 0, false);
}

// ------------------------------------------------------------------ softmax warpgroup (128 threads per tile)
// 2^x for a pair of values on the FMA pipe.  x = n + r with n = round(x), |r| <= 1/2: adding
// 1.5 * 2^23 leaves n in the low mantissa bits of the sum; 2^r is a degree-3 minimax polynomial
// (relative error 7.5e-5, a twenty-sixth of the bf16 rounding step the result goes through);
// 2^n is applied by adding n to the exponent field.  Valid for x <= 100; x is clamped at -125.
__device__ __forceinline__ void exp2_poly_pair(uint64_t x2, float& p0, float& p1) {
  float x0, x1;
  unpack_f32x2(x2, x0, x1);
  x2 = pack_f32x2(fmaxf(x0, -125.0f), fmaxf(x1, -125.0f));
  const uint64_t magic = pack_f32x2(12582912.0f, 12582912.0f);
  const uint64_t t = add_f32x2(x2, magic);
  const uint64_t r = sub_f32x2(x2, sub_f32x2(t, magic));
  uint64_t q = fma_f32x2(pack_f32x2(0x1.c3f76p-5f, 0x1.c3f76p-5f), r, pack_f32x2(0x1.f0de1ap-3f, 0x1.f0de1ap-3f));
  q = fma_f32x2(q, r, pack_f32x2(0x1.62f31ap-1f, 0x1.62f31ap-1f));
  q = fma_f32x2(q, r, pack_f32x2(0x1.fff692p-1f, 0x1.fff692p-1f));
  float t0, t1, q0, q1;
  unpack_f32x2(t, t0, t1);
  unpack_f32x2(q, q0, q1);
  p0 = __uint_as_float(__float_as_uint(q0) + (__float_as_uint(t0) << 23));
  p1 = __uint_as_float(__float_as_uint(q1) + (__float_as_uint(t1) << 23));
}

// Block b of 8 key columns (0..15 within a step) goes to the polynomial when kPoly of eight blocks do.  The choice
// depends on the column alone, so a query row's result does not depend on where in a tile the row sits.
template <int kPoly>
__device__ __forceinline__ constexpr bool block_uses_poly(int b) { return (((b & 7) + 1) * kPoly) / 8 != ((b & 7) * kPoly) / 8; }

// What a softmax thread knows about itself.  A softmax warp works on 16 query rows of its tile, all 128 columns
// of a key step: the tensor-memory lanes [32 q + 16 h, 32 q + 16 h + 16) of the tile.  Its tensor-memory
// accesses use the 16-lane shapes, which spread a row over the four threads of a quad: thread `lane` holds,
// of every block of 8 columns, columns 2 i and 2 i + 1 (i = lane % 4) of the rows lane / 4 and lane / 4 + 8.
// A row's maximum and sums therefore take two shuffles within the quad and no shared memory, and every row
// is handled inside one warp.
struct SoftmaxThread {
  int t;        // query tile of the CTA
  int h;        // which 16 of the 32 lanes of the warp's tensor-memory quarter
  int q;        // tensor-memory quarter (and scheduler): lanes [32 q, 32 q + 32)
  int lane;
  int i;        // position in the quad: columns 2 i, 2 i + 1 of every 8
  int r[2];     // the thread's two rows within the tile
  uint32_t tS, tP, tO;   // tensor-memory addresses (first lane of the warp's 16) of S, P and O of the tile
};

// tensor memory <-> registers in the 16-lane shapes (layout above): S (128 columns) and O (64 columns) as 32-bit
// columns, P as 64 columns of bf16 pairs
__device__ __forceinline__ void tmem_ld_rows16_c128(uint32_t taddr, uint32_t (&r)[64]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, "
      "%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, "
      "%48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]),
        "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]),
        "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]),
        "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]),
        "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_rows16_c64(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x8.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st_rows16_c64(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.16x256b.x8.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
// bf16 pairs of 4 blocks of 8 keys: register 2 n + hi -> row hi of the thread, pair column 4 n + i
__device__ __forceinline__ void tmem_st_rows16_p16(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.16x128b.x4.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}

// value over the four threads of a quad
__device__ __forceinline__ float quad_max(float v) {
  v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
  return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
}
__device__ __forceinline__ float quad_sum(float v) {
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  return v + __shfl_xor_sync(0xffffffffu, v, 2);
}

// 4 x 4 transpose over a quad: thread i gives word b and ends with the four words that the threads 0..3 held in
// their place i (two exchanges, with the neighbour at distance 1 and then 2; every lane of the warp takes part)
__device__ __forceinline__ void quad_transpose(uint32_t& w0, uint32_t& w1, uint32_t& w2, uint32_t& w3, int i) {
  const bool odd = (i & 1) != 0, upper = (i & 2) != 0;
  uint32_t got;
  got = __shfl_xor_sync(0xffffffffu, odd ? w0 : w1, 1);
  if (odd) w0 = got; else w1 = got;
  got = __shfl_xor_sync(0xffffffffu, odd ? w2 : w3, 1);
  if (odd) w2 = got; else w3 = got;
  got = __shfl_xor_sync(0xffffffffu, upper ? w0 : w2, 2);
  if (upper) w0 = got; else w2 = got;
  got = __shfl_xor_sync(0xffffffffu, upper ? w1 : w3, 2);
  if (upper) w1 = got; else w3 = got;
}

// Running state of the thread's two rows (the same in all four threads of a quad, except the partial sums).
struct RowState {
  float m_used[2];    // reference maximum of the stored exponentials (log2 units)
  float l_run[2];     // this thread's part of the sum of the bf16-rounded 2^(scale_log2 * s - m_used): normaliser of O
  float l_exact[2];   // the same sum without the rounding: log-sum-exp output only
};

// The thread's 64 scores of a key step (register 4 b + 2 hi + e: row hi, column 8 b + 2 i + e) -> bf16
// probabilities, stored to tensor memory at tP, relative to the rows' reference maxima folded into neg_m2; adds
// to the sums for the normaliser (of the rounded values) and for the log-sum-exp (unrounded).  Written pair by
// pair in dependency order; the instruction scheduler interleaves the pairs.
template <bool kMasked, bool kLse, int kPoly>
__device__ __forceinline__ void softmax_rows(const uint32_t (&s)[64], uint64_t scale2, const uint64_t (&neg_m2)[2],
                                             float (&sum_lo)[2], float (&sum_hi)[2], uint64_t (&sum_exact2)[2], uint32_t tP,
                                             int n_blocks) {
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    uint32_t pk[8];   // P of 32 keys x 2 rows as bf16 pairs
#pragma unroll
    for (int n = 0; n < 4; ++n) {
      // ragged last step: a block of 8 columns with no key in it gives zeros without any arithmetic
      if (kMasked && 4 * g + n >= n_blocks) {
        pk[2 * n] = 0u;
        pk[2 * n + 1] = 0u;
        continue;
      }
#pragma unroll
      for (int hi = 0; hi < 2; ++hi) {
        const int c = 4 * (4 * g + n) + 2 * hi;
        const uint64_t x2 = fma_f32x2(pack_f32x2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), scale2, neg_m2[hi]);
        float p0, p1;
        if (block_uses_poly<kPoly>(4 * g + n)) {
          exp2_poly_pair(x2, p0, p1);
        } else {
          float x0, x1;
          unpack_f32x2(x2, x0, x1);
          p0 = ex2_approx(x0);
          p1 = ex2_approx(x1);
        }
        const uint32_t w = pack_bf16x2(p0, p1);
        pk[2 * n + hi] = w;
        if (kLse) sum_exact2[hi] = add_f32x2(sum_exact2[hi], pack_f32x2(p0, p1));
        add_bf16x2_to_f32(w, sum_lo[hi], sum_hi[hi]);
      }
    }
    tmem_st_rows16_p16(tP + g * 16, pk);
  }
}

// One step of the online softmax of the thread's two rows: S_t(j) in tensor memory -> P_t(j) in tensor
// memory, running reference maxima and partial sums updated.
//
// The 64 scores are pulled into registers at once and the warp's share of S_t is released, so that the next
// Q K^T runs under this step's exponentials.  The row maxima (two shuffles within the quad) decide whether a
// reference maximum moves (lazy rescale).
// j: step within the work item; g: the tile's steps in the CTA's earlier work items.  kPoly: blocks of 8 columns per eight
// whose exponentials are polynomials.  kLse: also keep the sum of the unrounded exponentials, for the
// log-sum-exp output.  kMasked: columns >= valid are excluded (valid may be <= 0).
template <bool kMasked, bool kLse, int kPoly>
__device__ __forceinline__ bool softmax_step(const SoftmaxThread& me, int j, int g, int valid, float scale_log2,
                                             RowState& st, Barriers* bars, const AttnArgs& a) {
  const int gj = g + j;   // this tile's key steps so far, over all work items of the CTA: the phase of the per-step barriers
  uint32_t s[64];
  tmem_ld_rows16_c128(me.tS, s);
  tmem_wait_ld();
  tc_fence_before();
  __syncwarp();
  if (me.lane == 0) mbar_arrive(smem_u32(&bars->s_free[me.t]));

  if (kMasked) {
#pragma unroll
    for (int c = 0; c < 64; ++c)
      if (8 * (c >> 2) + 2 * me.i + (c & 1) >= valid) s[c] = __float_as_uint(-INFINITY);
  }
  float alpha[2];
  bool jump_any = false;
#pragma unroll
  for (int hi = 0; hi < 2; ++hi) {
    float mx = fmaxf(__uint_as_float(s[2 * hi]), __uint_as_float(s[2 * hi + 1]));
#pragma unroll
    for (int b = 1; b < 16; ++b) mx = max3(mx, __uint_as_float(s[4 * b + 2 * hi]), __uint_as_float(s[4 * b + 2 * hi + 1]));
    const float tile_max = quad_max(mx) * scale_log2;
    // lazy rescale: keep the old reference maximum unless the new one is far above it
    const bool jump = tile_max > st.m_used[hi] + kRescaleThreshold;
    alpha[hi] = 1.0f;
    if (jump) {
      alpha[hi] = ex2_approx(st.m_used[hi] - tile_max);   // 0 on the first tile (m_used = -inf)
      st.m_used[hi] = tile_max;
      st.l_run[hi] *= alpha[hi];
      if (kLse) st.l_exact[hi] *= alpha[hi];
    }
    jump_any = jump_any || jump;
  }
  const bool rescale = (j > 0) && __any_sync(0xffffffffu, jump_any);

  // P_t(j-1) must have been consumed, and O_t be at rest, before either is written
  if (j > 0) {
    if (!wait_bar(&bars->o_done[me.t], (gj - 1) & 1, bars, a, 30 + me.t, gj)) return false;
    tc_fence_after();
  }
  if (rescale) {   // the warp's 16 rows of the accumulator: register 4 b + 2 hi + e is row hi
    uint32_t o[32];
    tmem_ld_rows16_c64(me.tO, o);
    tmem_wait_ld();
#pragma unroll
    for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha[(c >> 1) & 1]);
    tmem_st_rows16_c64(me.tO, o);
  }

  // exponentials, rounded to bf16 for the value product; the normaliser sums the
  // rounded values so that numerator and denominator carry the same weights
  const uint64_t scale2 = pack_f32x2(scale_log2, scale_log2);
  const uint64_t neg_m2[2] = {pack_f32x2(-st.m_used[0], -st.m_used[0]), pack_f32x2(-st.m_used[1], -st.m_used[1])};
  float sum_lo[2] = {0.f, 0.f}, sum_hi[2] = {0.f, 0.f};   // even and odd columns
  uint64_t sum_exact2[2] = {pack_f32x2(0.f, 0.f), pack_f32x2(0.f, 0.f)};
  const int n_blocks = kMasked ? (valid + 7) >> 3 : 16;   // blocks of 8 columns that hold a key
  softmax_rows<kMasked, kLse, kPoly>(s, scale2, neg_m2, sum_lo, sum_hi, sum_exact2, me.tP, n_blocks);
#pragma unroll
  for (int hi = 0; hi < 2; ++hi) {
    st.l_run[hi] += sum_lo[hi] + sum_hi[hi];
    if (kLse) {
      float sum_a, sum_b;
      unpack_f32x2(sum_exact2[hi], sum_a, sum_b);
      st.l_exact[hi] += sum_a + sum_b;
    }
  }
  tmem_wait_st();
  tc_fence_before();
  __syncwarp();
  if (me.lane == 0) mbar_arrive(smem_u32(&bars->p_full[me.t]));
  return true;
}

// 4-byte word (two bf16) number w (0..31) of row r of a 128-byte-swizzled tile
__device__ __forceinline__ uint32_t ld_swizzled_word(const uint8_t* tile, int r, int w) {
  return *reinterpret_cast<const uint32_t*>(tile + r * 128 + (((w >> 2) ^ (r & 7)) << 4) + ((w & 3) << 2));
}

// One work item of a softmax thread: the key steps, then the epilogue.  g: this tile's key steps in the CTA's earlier
// work items; n_done: work items before this one.
__device__ __forceinline__ bool softmax_item(const AttnArgs& a, Barriers* bars, const SmemLayout& sm, const SoftmaxThread& me,
                                             const CtaProblem& cta, int g, int n_done) {
  const Plan& pl = a.pl;
  const int n_kv = a.n_kv_tiles;
  const int t = me.t, lane = me.lane;
  RowState st;
#pragma unroll
  for (int hi = 0; hi < 2; ++hi) { st.m_used[hi] = -INFINITY; st.l_run[hi] = 0.f; st.l_exact[hi] = 0.f; }
  const bool want_lse = a.lse != nullptr;

#pragma unroll 1
  for (int j = 0; j < n_kv; ++j) {
    if (!wait_bar(&bars->s_full[t], (g + j) & 1, bars, a, 40 + t, g + j)) return false;
    tc_fence_after();
    const int valid = static_cast<int>(a.n_keys - static_cast<int64_t>(j) * kTileKV);
    bool ok;
    // the masked (last, ragged) tile keeps every exponential on the special-function unit, where -inf gives an exact 0
    if (valid < kTileKV) ok = want_lse ? softmax_step<true, true, 0>(me, j, g, valid, a.scale_log2, st, bars, a)
                                       : softmax_step<true, false, 0>(me, j, g, valid, a.scale_log2, st, bars, a);
    else if (want_lse) ok = softmax_step<false, true, kPolyEighths>(me, j, g, valid, a.scale_log2, st, bars, a);
    else ok = softmax_step<false, false, kPolyEighths>(me, j, g, valid, a.scale_log2, st, bars, a);
    if (!ok) return false;
  }

  // ---- epilogue: diagonal and mean-fill terms, normalisation, store of this thread's 16 output dimensions of two rows
  const int head = cta.head;
  if (n_kv > 0) {
    if (!wait_bar(&bars->o_done[t], (g + n_kv - 1) & 1, bars, a, 50 + t, g + n_kv)) return false;
    tc_fence_after();
  }
  // completed long ago: makes the Q tile visible to this thread.  Only the two extra columns read Q here, and a CTA
  // that has them has one work item (a later item's Q may already be on its way otherwise).
  if ((a.use_diag || a.use_mean) && !wait_bar(&bars->q_full, n_done & 1, bars, a, 52, 0)) return false;
  const int item = n_kv + t;                         // ring item holding this tile's own K/V rows
  const uint8_t* sKd = sm.k + (item % kStages) * kTileBytes;
  const uint8_t* sVd = sm.v + (item % kStages) * kTileBytes;
  if (a.use_diag) {
    const uint32_t par = (item / kStages) & 1;
    if (!wait_bar(&bars->k_full[item % kStages], par, bars, a, 53, item)) return false;
    if (!wait_bar(&bars->v_full[item % kStages], par, bars, a, 54, item)) return false;
  }
  const uint8_t* sQ = sm.q[t];

  uint32_t o[32];   // register 4 b + 2 hi + e: row hi, output dimension 8 b + 2 i + e
  if (n_kv > 0) {
    tmem_ld_rows16_c64(me.tO, o);
    tmem_wait_ld();
    // O_t is in registers: the next work item's first P V may overwrite it
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&bars->o_free[t]));
  } else {   // no retained keys at all: the accumulator was never written
#pragma unroll
    for (int c = 0; c < 32; ++c) o[c] = 0u;
  }

#pragma unroll
  for (int hi = 0; hi < 2; ++hi) {
    const int r = me.r[hi];
    const int row = cta.q0 + t * kTileQ + r;           // query token
    const bool row_valid = row < cta.row_end;
    bool is_dropped = false;   // only the diagonal term asks
    if (a.use_diag && row_valid) {
      const int32_t f = row / pl.L;
      is_dropped = (a.slot_of_token != nullptr ? a.slot_of_token[row] : compact_slot(pl, f, row - f * pl.L)) < 0;
    }
    // the row's sums over its four threads
    const float l_run = quad_sum(st.l_run[hi]);
    const float l_exact = want_lse ? quad_sum(st.l_exact[hi]) : 0.f;
    const float m_used = st.m_used[hi];
    // base-2 logits of the two extra columns: each thread of the quad takes its 16 dimensions, then the quad adds up
    // (every thread runs the shuffles; rows without the term carry zeros)
    const bool has_diag = a.use_diag && is_dropped;
    const int64_t count = pl.n_dropped - (has_diag ? 1 : 0);
    const bool has_mean = a.use_mean && count > 0;
    float acc_d = 0.f, acc_m = 0.f;
    if (a.use_diag || a.use_mean) {
#pragma unroll
      for (int b = 0; b < 8; ++b) {
        const uint32_t qw = ld_swizzled_word(sQ, r, 4 * b + me.i);
        const float q0 = __uint_as_float(qw << 16), q1 = __uint_as_float(qw & 0xffff0000u);
        if (has_diag) {
          const uint32_t kw = ld_swizzled_word(sKd, r, 4 * b + me.i);
          acc_d = fmaf(q0, __uint_as_float(kw << 16), acc_d);
          acc_d = fmaf(q1, __uint_as_float(kw & 0xffff0000u), acc_d);
        }
        if (has_mean) {
          const float2 km = __ldg(reinterpret_cast<const float2*>(a.kmean + head * kHeadDim + 8 * b + 2 * me.i));
          acc_m = fmaf(q0, km.x, acc_m);
          acc_m = fmaf(q1, km.y, acc_m);
        }
      }
      acc_d = quad_sum(acc_d);
      acc_m = quad_sum(acc_m);
    }
    float m_fin = m_used, a_s = 1.0f, p_d = 0.f, p_m = 0.f;
    if (a.use_diag || a.use_mean) {   // the same for every row of the launch; frame attention has neither
      float l_d = -INFINITY, l_m = -INFINITY;
      if (has_diag) l_d = acc_d * a.scale_log2;
      if (has_mean) {
        l_m = acc_m * a.scale_log2;
        if (pl.mean_fill == AVGGT_MEAN_FILL) l_m += log2f(static_cast<float>(count));
      }
      m_fin = fmaxf(m_used, fmaxf(l_d, l_m));
      a_s = exp2f(m_used - m_fin);
      p_d = exp2f(l_d - m_fin);              // 0 when the term is absent
      p_m = exp2f(l_m - m_fin);
    }
    const float z = fmaf(l_run, a_s, p_d + p_m);
    const float inv_z = __fdividef(1.0f, z);   // z is at least one exponential of a row maximum, far from the ends of the range
    const float w_s = a_s * inv_z, w_d = p_d * inv_z, w_m = p_m * inv_z;
    // the thread's 8 words of the output row: word 4 b + i (dimensions 8 b + 2 i, 8 b + 2 i + 1)
    uint32_t w[8];
#pragma unroll
    for (int b = 0; b < 8; ++b) {
      float v0 = __uint_as_float(o[4 * b + 2 * hi]) * w_s, v1 = __uint_as_float(o[4 * b + 2 * hi + 1]) * w_s;
      if (w_d != 0.f) {
        const uint32_t vw = ld_swizzled_word(sVd, r, 4 * b + me.i);
        v0 = fmaf(w_d, __uint_as_float(vw << 16), v0);
        v1 = fmaf(w_d, __uint_as_float(vw & 0xffff0000u), v1);
      }
      if (has_mean) {
        const float2 vm = __ldg(reinterpret_cast<const float2*>(a.vmean + head * kHeadDim + 8 * b + 2 * me.i));
        v0 = fmaf(w_m, vm.x, v0);
        v1 = fmaf(w_m, vm.y, v1);
      }
      w[b] = pack_bf16x2(v0, v1);
    }
    // Transposed within the quad, a thread holds 16 contiguous bytes of each half of the row: 4 stores of 16 bytes
    // per thread instead of 16 of 4 bytes (whose 8 rows x 16 bytes per warp instruction kept the store path of the
    // SM busy for thousands of clocks per work item).
    quad_transpose(w[0], w[1], w[2], w[3], me.i);
    quad_transpose(w[4], w[5], w[6], w[7], me.i);
    if (row_valid) {
      uint4* dst = reinterpret_cast<uint4*>(a.O + (static_cast<size_t>(row) * pl.H + head) * kHeadDim);
      dst[me.i] = make_uint4(w[0], w[1], w[2], w[3]);
      dst[4 + me.i] = make_uint4(w[4], w[5], w[6], w[7]);
      if (want_lse && me.i == 0) {
        const float z_exact = fmaf(l_exact, a_s, p_d + p_m);
        a.lse[static_cast<size_t>(row) * pl.H + head] = (m_fin + log2f(z_exact)) * 0.6931471805599453f;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void softmax_role(const AttnArgs& a, Barriers* bars, const SmemLayout& sm, uint32_t tmem, int warp,
                                             int lane) {
  SoftmaxThread me;
  me.t = warp >> 3;
  me.h = (warp >> 2) & 1;
  me.q = warp & 3;
  me.lane = lane;
  me.i = lane & 3;
  me.r[0] = 32 * me.q + 16 * me.h + (lane >> 2);
  me.r[1] = me.r[0] + 8;
  const uint32_t tile_base = tmem + me.t * kTmemTileStride + (static_cast<uint32_t>(32 * me.q + 16 * me.h) << 16);   // TMEM lane = row
  me.tS = tile_base;
  me.tP = tile_base + kColP;
  me.tO = tile_base + kColO;
  const int n_kv = a.n_kv_tiles;
  int g = 0, n_done = 0;
#pragma unroll 1
  for (int item = blockIdx.x; item < a.n_work; item += gridDim.x) {
    if (!softmax_item(a, bars, sm, me, work_item(a, item), g, n_done)) return;
    g += n_kv;
    ++n_done;
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
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);   // warp-uniform by construction
  // a launch in which a wait has already run out is abandoned: the remaining CTAs leave at once
  if (__syncthreads_or(*reinterpret_cast<volatile uint32_t*>(a.status) != 0u)) return;

  if (tid == 0) {
    mbar_init(smem_u32(&bars.q_full), 1);
    mbar_init(smem_u32(&bars.q_empty), kQTiles);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&bars.k_full[s]), 1);
      mbar_init(smem_u32(&bars.k_empty[s]), kQTiles);
      mbar_init(smem_u32(&bars.v_full[s]), 1);
      mbar_init(smem_u32(&bars.v_empty[s]), kQTiles);
    }
    for (int t = 0; t < kQTiles; ++t) {
      mbar_init(smem_u32(&bars.s_full[t]), 1);
      mbar_init(smem_u32(&bars.s_free[t]), kSoftmaxWarps / kQTiles);
      mbar_init(smem_u32(&bars.p_full[t]), kSoftmaxWarps / kQTiles);
      mbar_init(smem_u32(&bars.o_done[t]), 1);
      mbar_init(smem_u32(&bars.mma_idle[t]), 1);
      mbar_init(smem_u32(&bars.o_free[t]), kSoftmaxWarps / kQTiles);
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
    reg_inc<kRegsSoftmax>();
    softmax_role(a, &bars, sm, tmem, warp, tid & 31);
  } else {
    reg_dec<kRegsOther>();
    if (warp == kTmaWarp) producer_role(&tm_q, &tm_k, &tm_v, &tm_kc, &tm_vc, a, &bars, sm);
    else if (warp == kMmaWarp) mma_role<0>(a, &bars, sm, tmem);
    else if (warp == kMmaWarp + 1) mma_role<1>(a, &bars, sm, tmem);
  }

  // a role that left on a wait that ran out may have tensor-memory loads or stores in flight
  tmem_wait_ld();
  tmem_wait_st();
  tc_fence_before();
  __syncthreads();
  if (warp == kTmaWarp) tmem_dealloc(tmem, kTmemCols);
}

constexpr size_t kAttnSmemBytes = static_cast<size_t>(kTileBytes) * (kQTiles + 2 * kStages) + 1024;

}  // namespace

size_t global_attn_ws_bytes(const Plan&, int) { return kAttnStatusBytes; }

namespace {

// Once per device: the dynamic shared-memory limit of the kernel, and a check that the launch allocates the
// registers the role split hands out.  setmaxnreg.inc waits, without a time limit, for registers that other
// warps release; if the compiler gave the kernel fewer than kRegsLaunch registers per thread the pool could
// never cover the softmax warps' share and the kernel would hang, so such a build refuses to launch.
cudaError_t prepare_kernel() {
  static std::mutex mu;
  static bool ready[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  if (ready[dev]) return cudaSuccess;
  cudaFuncAttributes fa;
  e = cudaFuncGetAttributes(&fa, global_attn_kernel);
  if (e != cudaSuccess) return e;
  if (fa.numRegs * (kThreads / 32) < kRegsSoftmax * kSoftmaxWarps + kRegsOther * (kThreads / 32 - kSoftmaxWarps))
    return cudaErrorLaunchOutOfResources;
  e = cudaFuncSetAttribute(global_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kAttnSmemBytes));
  if (e != cudaSuccess) return e;
  ready[dev] = true;
  return cudaSuccess;
}

// Tensor maps and launch shared by the two entry points.  frame_mode: see AttnArgs.
cudaError_t launch_attn(const Plan& pl, int sm_count, bool frame_mode, const void* Q, const void* K, const void* V, const void* Kc,
                        const void* Vc, const float* kmean, const float* vmean, void* O, float* lse, void* ws,
                        cudaStream_t st, bool* tmap_failed, const int32_t* slot_of_token) {
  *tmap_failed = false;
  AttnArgs a;
  a.pl = pl;
  a.slot_of_token = slot_of_token;
  a.kmean = kmean;
  a.vmean = vmean;
  a.O = static_cast<__nv_bfloat16*>(O);
  a.lse = lse;
  a.status = static_cast<uint32_t*>(ws);
  a.frame_mode = frame_mode ? 1 : 0;
  a.n_keys = frame_mode ? pl.L : pl.M;
  a.n_kv_tiles = static_cast<int32_t>((a.n_keys + kTileKV - 1) / kTileKV);
  a.use_diag = (!frame_mode && pl.diag != 0 && pl.n_dropped > 0) ? 1 : 0;
  a.use_mean = (!frame_mode && pl.mean_fill != 0 && pl.n_dropped > 0) ? 1 : 0;
  a.scale_log2 = pl.scale * kLog2e;
  const int64_t rows = frame_mode ? pl.L : pl.n_tok;
  a.pairs = static_cast<int32_t>((rows + kQTiles * kTileQ - 1) / (kQTiles * kTileQ));
  a.n_work = a.pairs * pl.H * (frame_mode ? pl.n_frames : 1);

  // token-major [n_tok, H*d] maps for Q and for K, V (the diagonal tiles; all tiles of frame attention);
  // head-major [H, M, d] maps for Kc, Vc
  CUtensorMap tm_q, tm_k, tm_v, tm_kc, tm_vc;
  const uint64_t tok_dims[2] = {static_cast<uint64_t>(pl.H) * pl.d, static_cast<uint64_t>(pl.n_tok)};
  const uint64_t tok_str[1] = {static_cast<uint64_t>(pl.H) * pl.d * 2};
  const uint32_t tok_box[2] = {kHeadDim, kTileQ};
  const bool reads_kv = frame_mode || a.use_diag;
  bool good = make_tmap_bf16(&tm_q, Q, 2, tok_dims, tok_str, tok_box);
  good = good && make_tmap_bf16(&tm_k, reads_kv ? K : Q, 2, tok_dims, tok_str, tok_box);
  good = good && make_tmap_bf16(&tm_v, reads_kv ? V : Q, 2, tok_dims, tok_str, tok_box);
  if (frame_mode || pl.M == 0) {
    tm_kc = tm_k;   // not read
    tm_vc = tm_v;
  } else {
    const uint64_t c_dims[3] = {static_cast<uint64_t>(pl.d), static_cast<uint64_t>(pl.M), static_cast<uint64_t>(pl.H)};
    const uint64_t c_str[2] = {static_cast<uint64_t>(pl.d) * 2, static_cast<uint64_t>(pl.M) * pl.d * 2};
    const uint32_t c_box[3] = {kHeadDim, kTileKV, 1};
    good = good && make_tmap_bf16(&tm_kc, Kc, 3, c_dims, c_str, c_box);
    good = good && make_tmap_bf16(&tm_vc, Vc, 3, c_dims, c_str, c_box);
  }
  if (!good) { *tmap_failed = true; return cudaSuccess; }

  cudaError_t e = prepare_kernel();
  if (e != cudaSuccess) return e;
  e = cudaMemsetAsync(ws, 0, kAttnStatusBytes, st);
  if (e != cudaSuccess) return e;
  // The subsampled layer: one work item per CTA (hundreds of key steps each).  Frame attention: a dozen key steps
  // per work item, so one CTA per SM walks over many of them and the next item's loads and first product run
  // under the current item's epilogue.
  const unsigned grid = frame_mode ? static_cast<unsigned>(a.n_work < sm_count ? a.n_work : sm_count)
                                   : static_cast<unsigned>(a.n_work);
  global_attn_kernel<<<grid, kThreads, kAttnSmemBytes, st>>>(tm_q, tm_k, tm_v, tm_kc, tm_vc, a);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_global_attn(const Plan& pl, int sm_count, const void* Q, const void* K, const void* V,
                               const void* Kc, const void* Vc, const float* kmean, const float* vmean, void* O,
                               float* lse, void* ws, cudaStream_t st, bool* tmap_failed, const int32_t* slot_of_token) {
  return launch_attn(pl, sm_count, false, Q, K, V, Kc, Vc, kmean, vmean, O, lse, ws, st, tmap_failed, slot_of_token);
}

cudaError_t launch_frame_attn(const Plan& pl, int sm_count, const void* Q, const void* K, const void* V, void* O, float* lse,
                              void* ws, cudaStream_t st, bool* tmap_failed) {
  return launch_attn(pl, sm_count, true, Q, K, V, nullptr, nullptr, nullptr, nullptr, O, lse, ws, st, tmap_failed, nullptr);
}

}  // namespace avggt
