/*
 * avggt.h - C ABI of libavggt: subsampled global self-attention for
 * VGGT / pi^3 style alternating frame/global transformers on NVIDIA B200
 * (sm_100a).
 *
 * The library implements one layer of the AVGGT paper, "Subsampling Global
 * Attention" (Sec. 4.3): every token of all N frames is a query; the keys and
 * values are (i) all special tokens plus the first patch token of every
 * s_h x s_w window of each frame's patch grid, (ii) the query's own key/value
 * (diagonal preservation) and (iii) one mean key/value pair standing for all
 * dropped patch tokens (mean-fill), normalised by one shared softmax.
 *
 * Conventions that hold for every entry point
 *   - Plain C types only.  Pointers marked "device" are CUDA device pointers
 *     on the current device; pointers marked "host" are ordinary host memory.
 *   - The library never allocates or frees memory the caller can see.  All
 *     buffers, including the workspace, are owned by the caller and must stay
 *     valid until the work enqueued on the stream has finished.
 *   - Device buffers must be 16-byte aligned (AVGGT_ERR_ALIGNMENT otherwise).
 *   - Calls that take a stream only enqueue work on it and return without
 *     synchronising.  `cuda_stream` is a cudaStream_t passed as void*
 *     (NULL = the legacy default stream).
 *   - Return value: 0 on success, a negative AVGGT_ERR_* code otherwise.
 *     Arguments are validated on the host before anything is launched; after an
 *     argument error nothing has been enqueued.  (If the launch itself fails with
 *     AVGGT_ERR_CUDA, the clearing of the status block may already be on the
 *     stream; no kernel is.)  No exception crosses this boundary.
 *   - Size limits: head_dim == 64; n_heads <= 32; batch == 1;
 *     N * L <= 2^31 - 257 tokens; frame attention: ceil(L / 256) * H * N < 2^31.  Anything
 *     beyond them is rejected with AVGGT_ERR_UNSUPPORTED.
 *   - Only sm_100 devices are supported (AVGGT_ERR_UNSUPPORTED elsewhere).
 *     There is no CPU fallback.
 *   - Calls on distinct streams with distinct output/workspace buffers may be
 *     made from different host threads.
 *
 * Token layout (Sec. 4.1 notation): a frame has L = n_special + n_h*n_w
 * tokens; slots [0, n_special) of a frame are its special tokens (camera and
 * register tokens), followed by the patch grid in row-major order.  Token t
 * of the sequence is slot t % L of frame t / L.  Q, K, V and O are
 * [N*L, H, d] arrays, d contiguous, i.e. what a fused QKV projection
 * produces for the (B, N*L, C) global layout of Sec. 4.2 with C = H*d.
 */
#ifndef AVGGT_H_
#define AVGGT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AVGGT_OK                        0
#define AVGGT_ERR_INVALID_ARG          -1   /* NULL pointer, non-positive size, inconsistent sizes   */
#define AVGGT_ERR_UNSUPPORTED          -2   /* sigma, head_dim, batch, device not supported           */
#define AVGGT_ERR_WORKSPACE_TOO_SMALL  -3
#define AVGGT_ERR_ALIGNMENT            -4   /* a device pointer is not 16-byte aligned                */
#define AVGGT_ERR_CUDA                 -5   /* a CUDA runtime/driver call failed; see avggt_last_cuda_error */
#define AVGGT_ERR_DEVICE_TIMEOUT       -6   /* a bounded device-side wait ran out (avggt_check_status) */
#define AVGGT_ERR_STATIC_SCRATCH       -7   /* problem exceeds the fixed scratch of avggt_build_kv_noalloc */

/* flags */
#define AVGGT_FLAG_KEEP_FIRST_FRAME    1u   /* frame 0 keeps all patch K/V (VGGT variant, Sec. 4.3)   */

/* mean_fill modes */
#define AVGGT_MEAN_OFF     0
#define AVGGT_MEAN_UNIT    1   /* the mean pair is one extra column of weight 1                       */
#define AVGGT_MEAN_FILL    2   /* every dropped column is filled with the mean pair: the single mean  */
                               /* column carries the count of columns it stands for                   */

/*
 * Problem statement (Sec. 4.1 and 4.3).  Plain data, passed by pointer (host).
 */
typedef struct avggt_params {
  int32_t batch;             /* B; must be 1 (independent problems are separate calls)                */
  int32_t n_frames;          /* N >= 1                                                                */
  int32_t tokens_per_frame;  /* L; must equal n_special + grid_h * grid_w                             */
  int32_t grid_h, grid_w;    /* n_h, n_w: patch grid of one frame                                     */
  int32_t n_special;         /* special tokens per frame (5 for VGGT and pi^3), >= 0                  */
  int32_t n_heads;           /* H, 1 <= H <= 32                                                       */
  int32_t head_dim;          /* d; must be 64                                                         */
  int32_t sigma;             /* subsampling factor: 1 (dense), 2, 4, 6, 9 -> (s_h, s_w) =
                                (1,1), (1,2), (2,2), (2,3), (3,3)  (Sec. 4.3, Subsampling Strategy)   */
  int32_t diag;              /* 0/1: diagonal preservation                                            */
  int32_t mean_fill;         /* AVGGT_MEAN_*                                                          */
  float   softmax_scale;     /* <= 0 selects 1/sqrt(d)                                                */
  uint32_t flags;            /* AVGGT_FLAG_*; unknown bits are rejected                               */
} avggt_params;

/*
 * Number of compacted keys M and of dropped patch tokens |D| for a problem
 * (Sec. 4.3: special tokens are always kept; a partial window at the grid
 * edge keeps its first token).  Host-only, pure.
 */
int avggt_kv_count(const avggt_params* p, int64_t* n_kept, int64_t* n_dropped);

/*
 * Workspace sizes in bytes needed by avggt_build_kv and avggt_global_attn for
 * this problem on the current device.  Either output may be NULL.
 * Host-only apart from a device-property query.
 */
int avggt_workspace_bytes(const avggt_params* p, size_t* build_ws_bytes, size_t* attn_ws_bytes);

/*
 * K/V compaction and mean-fill reduction (Sec. 4.3, Subsampling Strategy and
 * Enhanced Subsampling).  One pass over K and V:
 *   Kc[h][m][:] = K[idx[m]][h][:],  Vc likewise      (bit copies)
 *   kmean[h][:] = mean over dropped patch tokens j of K[j][h][:]   (fp32), vmean likewise
 * where idx[m] is the global token index of the m-th retained key in ascending
 * order.
 *
 *   K, V    device, bf16 [N*L, H, d]             read only
 *   Kc, Vc  device, bf16 [H, M, d]  (head-major) written
 *   idx     device, int32 [M], may be NULL       written
 *   kmean, vmean  device, float [H, d]           written when mean_fill != 0 and |D| > 0
 *                                                (zero-filled when |D| == 0); may be NULL when
 *                                                mean_fill == 0
 *   ws      device scratch of at least build_ws_bytes; holds per-block partial sums and is
 *           fully rewritten by each call, so it needs no initialisation.  The reduction order is
 *           fixed: results are identical from run to run.
 */
int avggt_build_kv(const avggt_params* p, const void* K, const void* V,
                   void* Kc, void* Vc, int32_t* idx, float* kmean, float* vmean,
                   void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * avggt_build_kv for callers that cannot allocate.  (The paper has no counterpart to this
 * entry point; it exists for the sake of the library's users.)
 *
 * Who needs it: a program whose memory manager owns every byte of device memory before this
 * library is loaded, a plugin that lives under another process's fixed memory budget, or a
 * latency-critical loop that must not call cudaMalloc because it synchronises the device.
 * Such a caller has no workspace to lend.  Here the scratch of the mean reduction (the
 * per-block partial sums) is a fixed array inside the library image: about 2.3 MiB that every
 * GPU which loads the library holds until the process exits.
 *
 * Same inputs, outputs and results as avggt_build_kv (the mean pair may differ in the last
 * bits, because the partial sums are grouped over fewer blocks), with these differences:
 *   - no ws / ws_bytes arguments; the call makes no cudaMalloc, cudaFree or other allocating
 *     call, on any path;
 *   - limit: n_heads * head_dim <= 1024.  Larger problems are rejected with
 *     AVGGT_ERR_STATIC_SCRATCH before anything is enqueued;
 *   - the first call on each device looks up the array's device address (and the device's
 *     properties) with that device current; make that first call before any stream capture
 *     begins.  Later calls only enqueue kernels.  The address is kept for the life of the
 *     process: after a cudaDeviceReset it is stale and this entry point must not be used again;
 *   - all calls on one device share the one array.  Each call rewrites every element it later
 *     reads, so the previous call's contents do no harm and nothing needs clearing; but two
 *     calls whose kernels overlap on the GPU (different streams, or different host threads)
 *     race on it and give wrong means.  Serialise them on one stream.
 */
int avggt_build_kv_noalloc(const avggt_params* p, const void* K, const void* V,
                           void* Kc, void* Vc, int32_t* idx, float* kmean, float* vmean,
                           void* cuda_stream);

/*
 * Subsampled global attention (Sec. 4.3): for every query token i and head h
 *   O[i][h][:] = ( sum_{m<M} e^{l_m} Vc[h][m] + [i in D, diag] e^{l_d} V[i][h] + [c_i>0, mean] e^{l_mu} vmean[h] ) / Z
 * with l_m = scale q.Kc[h][m], l_d = scale q.K[i][h], l_mu = scale q.kmean[h] (+ ln c_i in
 * AVGGT_MEAN_FILL mode), c_i = |D| - [i in D and diag], and Z the sum of the same exponentials
 * (one shared softmax over the three disjoint components).  A query whose own column is
 * retained has no separate diagonal term.  With |D| = 0 the result is dense softmax attention.
 * Arithmetic: bf16 operands, fp32 accumulation and softmax, probabilities rounded to bf16 for
 * the value product, output rounded to bf16 (nearest even).
 *
 *   Q             device, bf16 [N*L, H, d]
 *   K, V          device, bf16 [N*L, H, d]; read only when diag != 0 (may be NULL otherwise)
 *   Kc, Vc        device, bf16 [H, M, d] from avggt_build_kv
 *   kmean, vmean  device, float [H, d]; read only when mean_fill != 0 and |D| > 0
 *   O             device, bf16 [N*L, H, d]       written
 *   lse           device, float [N*L, H] or NULL: natural-log normaliser ln(Z) + max-shift
 *   ws            device scratch of at least attn_ws_bytes.  It starts with a 256-byte status
 *                 block that the call clears on the stream and whose first 16 bytes
 *                 avggt_check_status reads.  The kernel looks at the block when it starts (a
 *                 launch in which a wait has run out is abandoned by its remaining thread
 *                 blocks), so one workspace serves one attention launch at a time: launches that
 *                 may be in flight together need a workspace each.
 */
int avggt_global_attn(const avggt_params* p, const void* Q, const void* K, const void* V,
                      const void* Kc, const void* Vc, const float* kmean, const float* vmean,
                      void* O, float* lse, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The same layer with a retained set chosen by the caller instead of the window rule (the
 * alternative selectors of the supplement, "Comparison with other subsampling strategies":
 * random, norm-ranked or feature-based picks).  `idx` lists the n_kept retained tokens; every
 * other token is in D, whatever its kind (list the special tokens to keep them).  Diagonal
 * preservation, the mean pair over D and the shared softmax are as in Sec. 4.3.  Of `p`, sigma
 * and flags play no part but must be valid.  n_kept = 0 is allowed when diag or mean_fill is on: it
 * is the G2M variant of Sec. 5.4 ("Effect of the Early Global Attention Layers"), in which one mean
 * pair over the whole sequence stands for every Key/Value (idx, Kc and Vc may then be NULL).
 *
 * avggt_build_kv_indexed
 *   idx            device, int32 [n_kept], strictly ascending token indices in [0, N*L).  The list
 *                  is not checked on the host: entries out of range are skipped, a repeated entry
 *                  leaves one compact row unwritten; neither reads or writes out of bounds.
 *   K, V, Kc, Vc, kmean, vmean, ws   as for avggt_build_kv, with M = n_kept
 *   slot_of_token  device, int32 [N*L]              written: compact position of a retained
 *                  token, -1 for a dropped one.  Pass it on to avggt_global_attn_indexed.
 * avggt_global_attn_indexed
 *   as avggt_global_attn with M = n_kept and the map from avggt_build_kv_indexed.
 */
int avggt_build_kv_indexed(const avggt_params* p, const int32_t* idx, int64_t n_kept,
                           const void* K, const void* V, void* Kc, void* Vc,
                           int32_t* slot_of_token, float* kmean, float* vmean,
                           void* ws, size_t ws_bytes, void* cuda_stream);
int avggt_global_attn_indexed(const avggt_params* p, int64_t n_kept, const int32_t* slot_of_token,
                              const void* Q, const void* K, const void* V,
                              const void* Kc, const void* Vc, const float* kmean, const float* vmean,
                              void* O, float* lse, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Subsampled global attention for a shard of the frames (one rank of a frame-sharded run): the
 * queries are the tokens of the n_frames frames that `p` describes (this rank's), the compact keys
 * and the mean pair are those of the WHOLE sequence (Sec. 4.3 defines S and the mean over all
 * frames).  The caller gathers Kc/Vc of all ranks into one [H, n_kept_total, d] array in this
 * GPU's memory and combines the ranks' means before the call; the library does no communication.
 *
 *   n_kept_total     compact keys of the whole sequence (>= this shard's own)
 *   n_dropped_total  dropped tokens of the whole sequence (the count behind the mean pair)
 *   Q, K, V, O, lse  this shard's rows only, [n_frames*L, H, d] / [n_frames*L, H]
 *   Kc, Vc           device, bf16 [H, n_kept_total, d]
 *   other arguments as for avggt_global_attn.  AVGGT_FLAG_KEEP_FIRST_FRAME refers to the first
 *   frame of the shard: set it only on the rank that owns frame 0 of the sequence.
 */
int avggt_global_attn_shard(const avggt_params* p, int64_t n_kept_total, int64_t n_dropped_total,
                            const void* Q, const void* K, const void* V,
                            const void* Kc, const void* Vc, const float* kmean, const float* vmean,
                            void* O, float* lse, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The K/V projection with the compaction of avggt_build_kv fused into its epilogue (Sec. 4.3: the
 * diagonal and mean-fill terms add "only O(N)" work; here that work needs no second pass over K
 * and V, because every tile of the projection is compacted while it is still on chip):
 *   K = X Wk^T + bias_k,  V = X Wv^T + bias_v       bf16 operands, fp32 accumulation on the tensor cores
 *   Kc, Vc, idx   as avggt_build_kv would produce them from the bf16-rounded K and V
 *   kmean, vmean  mean over the dropped patch tokens of the projections BEFORE the rounding to bf16
 *                 (fp32; the accumulators are at hand), with a fixed summation order
 *
 *   model_dim     C, channels of X: a multiple of 64
 *   X             device, bf16 [N*L, C]
 *   Wk, Wv        device, bf16 [H*d, C]  (the layout of a linear layer's weight: one row per output)
 *   bias_k/_v     device, float [H*d], or NULL
 *   K, V          device, bf16 [N*L, H, d], written; both NULL when the caller does not need the
 *                 full arrays (avggt_global_attn reads them only when diag != 0)
 *   Kc, Vc, idx, kmean, vmean   as for avggt_build_kv
 *   ws            device scratch of at least the size avggt_project_workspace_bytes returns; it starts
 *                 with a status block like the attention workspace (avggt_check_status reads it)
 */
int avggt_project_workspace_bytes(const avggt_params* p, int32_t model_dim, size_t* ws_bytes);
int avggt_project_build_kv(const avggt_params* p, int32_t model_dim,
                           const void* X, const void* Wk, const void* Wv,
                           const float* bias_k, const float* bias_v,
                           void* K, void* V, void* Kc, void* Vc, int32_t* idx,
                           float* kmean, float* vmean,
                           void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The exchange step of a frame-sharded run, in two library calls around the caller's two collectives
 * (Sec. 4.3 defines S and the mean pair over all frames, so the ranks exchange their compact K/V and
 * the sums behind the mean once per layer; the library itself does no communication).
 *
 * avggt_build_kv_shard: avggt_build_kv for this rank's frames (`p` describes them), writing straight
 * into this rank's slot of the exchange buffer and leaving the mean un-normalised.
 *   slot        device, bf16 [2][H][slot_rows][d]: compact K, then compact V, head-major; rows
 *               [M, slot_rows) of every head are left untouched (zero the buffer once: the rows are
 *               never read as keys, but they travel)
 *   slot_rows   rows per head in a slot, >= M of this shard (use the largest shard's M on every rank)
 *   idx         as for avggt_build_kv (token indices local to the shard), may be NULL
 *   sums        device, float [2][H][d]: sums of K, then of V, over this shard's dropped tokens
 *               (zero-filled when the shard drops none); may be NULL when mean_fill == 0
 *   ws          as for avggt_build_kv
 * The caller then all-gathers the slots into [n_ranks][2][H][slot_rows][d] (in place when `slot`
 * already lies inside that buffer) and all-reduces `sums`.
 *
 * avggt_shard_assemble: the gathered slots -> one compact K/V pair in ascending token order (ranks own
 * ascending frame ranges), and the mean pair = reduced sums / n_dropped_total.
 *   gathered         device, bf16 [n_ranks][2][H][slot_rows][d]
 *   kept             host, int64 [n_ranks]: M of every rank's shard (a pure function of the split)
 *   sums             device, float [2][H][d], after the all-reduce; read when mean_fill != 0 and
 *                    n_dropped_total > 0
 *   Kc, Vc           device, bf16 [H][sum of kept][d]            written
 *   kmean, vmean     device, float [H][d]                        written (same condition as sums)
 *   1 <= n_ranks <= 64.  Of `p` the call uses n_heads, head_dim and mean_fill.
 * Cost of the assembly: one read and one write of the compact K/V (0.57 GB at 800 frames, s = 9).
 */
int avggt_build_kv_shard(const avggt_params* p, const void* K, const void* V,
                         void* slot, int64_t slot_rows, int32_t* idx, float* sums,
                         void* ws, size_t ws_bytes, void* cuda_stream);
int avggt_shard_assemble(const avggt_params* p, const void* gathered, int32_t n_ranks,
                         const int64_t* kept, int64_t slot_rows, const float* sums,
                         int64_t n_dropped_total, void* Kc, void* Vc,
                         float* kmean, float* vmean, void* cuda_stream);

/*
 * Frame attention of a converted early global block (Sec. 4.2, "Global-to-Frame Attention
 * Conversion"): the (B, N L, C) rearrangement is skipped, so every token attends to the L tokens
 * of its own frame only, special tokens included, with plain softmax attention:
 *   O[i][h][:] = sum_{j in frame(i)} softmax_j(scale q_i.k_j) V[j][h][:].
 * N independent dense problems in one launch of the same kernel; keys and values are read
 * straight from K and V (nothing is compacted), so avggt_build_kv is not needed.  Of `p` the
 * call uses n_frames, tokens_per_frame, n_heads, head_dim and softmax_scale; sigma, diag,
 * mean_fill and flags play no part but must be valid.  ceil(L / 256) * H * N < 2^31.
 *
 *   Q, K, V       device, bf16 [N*L, H, d]; must be finite (a tile of keys may reach into the
 *                 next frame's rows, whose products are masked to zero weight)
 *   O             device, bf16 [N*L, H, d]       written
 *   lse           device, float [N*L, H] or NULL
 *   ws            device scratch of at least attn_ws_bytes (avggt_workspace_bytes); status
 *                 block as for avggt_global_attn
 */
int avggt_frame_attn(const avggt_params* p, const void* Q, const void* K, const void* V,
                     void* O, float* lse, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * After the caller has synchronised the stream: reads the status block at the start of an
 * attention workspace (a 16-byte device-to-host copy) and returns AVGGT_OK or
 * AVGGT_ERR_DEVICE_TIMEOUT if a bounded wait inside the kernel gave up (the output is then
 * undefined; the context stays usable).  `detail`, if not NULL, receives the raw status words
 * (host, 4 x uint32: code, block, role/stage, iteration).
 */
int avggt_check_status(const void* attn_ws, uint32_t* detail);

/* Static description of an error code. */
const char* avggt_strerror(int code);

/* Text of the last CUDA error seen by this thread inside the library ("" if none). */
const char* avggt_last_cuda_error(void);

/* Library version, "major.minor.patch". */
const char* avggt_version(void);

#ifdef __cplusplus
}
#endif
#endif /* AVGGT_H_ */
