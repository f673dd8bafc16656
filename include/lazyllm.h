/*
 * lazyllm.h — C ABI of the token-pruned prefill / decode library (sm_100a).
 *
 * The library runs the prefill forward of a Llama-style decoder with dynamic token
 * pruning, and the decode step that can revive pruned tokens from an Aux Cache.
 * Paper passages are cited per entry point ("Section 3.2", "Eq. 1", ...).
 *
 * Conventions that hold for every call
 *   - Return value: 0 (LAZY_OK) or a negative lazy_status. Nothing throws, aborts or traps.
 *   - "device" pointers are CUDA global-memory addresses of the current device; "host"
 *     pointers are ordinary process memory.  The library never allocates or frees device
 *     memory: weights, ids, logits and one workspace blob are caller-owned and must outlive
 *     the context.  The context itself (host metadata only) is owned by the library.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Work
 *     is enqueued asynchronously unless stated otherwise; device-side problems (a bounded
 *     wait that ran out, an index out of range) are written to a per-device status word and
 *     surface through lazy_sync_status() / lazy_device_status().
 *   - Matrices are row-major [out_features, in_features] (K-contiguous), activations are
 *     row-major [rows, features].  dtype LAZY_BF16: bf16 storage, fp32 accumulation;
 *     LAZY_F32: fp32 storage and arithmetic (CUDA cores; small models only).
 *   - A context holds ONE generation state; it is not thread-safe.
 */
#ifndef LAZYLLM_H_
#define LAZYLLM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LAZY_OK = 0,
  LAZY_E_BADARG = -1,      /* null pointer, non-positive size, unsupported shape            */
  LAZY_E_BADSCHEDULE = -2, /* schedule not strictly increasing / keep fractions increasing  */
  LAZY_E_CAPACITY = -3,    /* more tokens, sequences or workspace than the context was sized for */
  LAZY_E_NOT_IN_AUX = -4,  /* a position asked from an Aux Cache is not held there          */
  LAZY_E_TIMEOUT = -5,     /* a bounded device-side wait ran out                            */
  LAZY_E_CUDA = -6,        /* a CUDA runtime / driver call failed                           */
  LAZY_E_STATE = -7        /* call out of order (decode before prefill, ...)                */
} lazy_status;

enum { LAZY_BF16 = 0, LAZY_F32 = 1 };

typedef struct lazy_ctx lazy_ctx;

/* Model shape (Section 1: Llama 2 7B = 32 layers, model dimension 4096) and capacities. */
typedef struct {
  int32_t n_layers, d_model, n_heads, head_dim, d_ffn, vocab;
  float rms_eps, rope_theta;
  int32_t dtype;             /* LAZY_BF16 or LAZY_F32                                         */
  int32_t max_seqs;          /* sequences per batch                                          */
  int32_t max_prompt_tokens; /* packed total over the batch                                  */
  int32_t max_new_tokens;    /* decode steps per sequence the caches leave room for          */
  int32_t n_kv_heads;        /* key/value heads (grouped-query attention); 0 = n_heads.  Must divide
                              * n_heads: query head h reads key/value head h / (n_heads / n_kv_heads) */
} lazy_model_cfg;

/* Weights, all device memory except the per-layer pointer arrays themselves (host arrays of
 * n_layers device pointers).  w_qkv = [d + 2 d_kv, d] with the d query rows first, then the d_kv key rows,
 * then the d_kv value rows, d_kv = n_kv_heads * head_dim (= d without grouped-query attention).  K / V
 * cache rows (lazy_get_kv) are d_kv wide. */
typedef struct {
  const void *tok_embed;          /* [vocab, d]                */
  const void *const *w_qkv;       /* n_layers x [d + 2 d_kv, d] */
  const void *const *w_o;         /* n_layers x [d, d]         */
  const void *const *w_gate;      /* n_layers x [d_ffn, d]     */
  const void *const *w_up;        /* n_layers x [d_ffn, d]     */
  const void *const *w_down;      /* n_layers x [d, d_ffn]     */
  const void *const *g_attn;      /* n_layers x [d] RMSNorm gain before attention */
  const void *const *g_mlp;       /* n_layers x [d] RMSNorm gain before the MLP   */
  const void *g_final;            /* [d]                       */
  const void *w_lm_head;          /* [vocab, d]                */
} lazy_weights;

/* Layer-wise keep schedule (Section 3.2, progressive token pruning; the three knobs of
 * Section 4.2: how many pruning layers, where, how many tokens).  Point i says: the set that
 * ENTERS layer layer_entered[i] holds ceil(keep_bp[i]/10000 * N) tokens of the N-token
 * prompt, chosen by the Eq. 1 score of layer layer_entered[i]-1.  Layer 0 sees everything.
 * layer_entered strictly increasing in (0, n_layers); keep_bp in 1..10000, non-increasing. */
typedef struct {
  int32_t n_points;
  const int32_t *layer_entered; /* host */
  const uint32_t *keep_bp;      /* host */
} lazy_schedule;

/* Counters of the latest prefill / decode call (Section 4.3 "% of prompt tokens computed",
 * Section 4.5 cumulative token usage = KV-cache size per layer). Host struct, filled by
 * lazy_get_stats. Arrays are indexed by layer, up to LAZY_MAX_LAYERS. */
#define LAZY_MAX_LAYERS 128
typedef struct {
  int32_t n_layers;
  int32_t rows_computed[LAZY_MAX_LAYERS]; /* rows that went through each layer in the latest call */
  int32_t kv_rows[LAZY_MAX_LAYERS];       /* tokens whose K/V exist at each layer (all sequences)  */
  int32_t aux_rows[LAZY_MAX_LAYERS];      /* tokens held by the Aux Cache that follows each layer  */
  int32_t revived[LAZY_MAX_LAYERS];       /* rows revived into each layer in the latest call       */
  int64_t kernel_launches;                /* kernels enqueued by the latest call                   */
} lazy_stats;

/* ---- context ------------------------------------------------------------------------- */

/* Bytes of device workspace a context of this shape and schedule needs (0 on bad args).
 * Plumbing: no counterpart in the paper. */
size_t lazy_prefill_workspace_bytes(const lazy_model_cfg *cfg, const lazy_schedule *sched);

/* Validates cfg and schedule, records the weight pointers and carves `d_workspace`
 * (256-byte aligned, at least lazy_prefill_workspace_bytes).  Enqueues a few small set-up
 * kernels (RoPE table) on the default stream and synchronises before returning.  On success
 * *out owns host memory only.  Plumbing: no counterpart in the paper (the schedule it records
 * is Section 3.2's; the weights must stay unmodified while the context lives). */
int lazy_prefill_init(const lazy_model_cfg *cfg, const lazy_weights *w, const lazy_schedule *sched,
                      void *d_workspace, size_t workspace_bytes, lazy_ctx **out);

/* Token-pruned prefill (Section 3.1 prefilling stage; Section 3.2 progressive token pruning,
 * Eq. 1, Aux Cache).  d_prompt_ids: device int32, the prompts packed back to back;
 * h_cu_seqlens: host int32[n_seqs+1], cumulative lengths (h_cu_seqlens[0] = 0).
 * Writes fp32 next-token logits [n_seqs, vocab] to d_logits (device) and leaves per-layer KV
 * caches and Aux Caches in the workspace for decode.  Resets any earlier generation state.
 * Row counts follow from (lengths, schedule) alone, so nothing is read back: the call only
 * enqueues work on `stream`.  `stream` must not be capturing into a CUDA graph: the call copies small
 * index tables from host memory that does not outlive it, and a replay would read that memory again. */
int lazy_prefill_run(lazy_ctx *ctx, void *stream, const int32_t *d_prompt_ids,
                     const int32_t *h_cu_seqlens, int32_t n_seqs, float *d_logits);

/* One decode step for every sequence of the batch (Section 3.1 decoding stage; Section 3.2:
 * each step re-selects its context set by the new token's Eq. 1 score and may revive pruned
 * tokens from the Aux Cache instead of recomputing them).  d_new_ids: device int32[n_seqs],
 * the token appended to each sequence.  d_logits: device fp32 [n_seqs, vocab].  d_next_ids:
 * device int32[n_seqs] greedy argmax (lowest id on ties) or NULL.  How many rows are revived
 * depends on the data: at every scheduled layer the call reads a few counters back
 * (a stream synchronisation), so it returns with the step's selection already decided. */
int lazy_decode_step(lazy_ctx *ctx, void *stream, const int32_t *d_new_ids, float *d_logits,
                     int32_t *d_next_ids);

/* Reads hidden states of pruned tokens from the Aux Cache that follows `layer` (Section 3.2,
 * Aux Cache: hidden states of tokens whose KV is absent from the next layer's cache).
 * d_positions: device int32[n] original token positions of sequence `seq`; d_hidden_out:
 * device [n, d_model] in the context's dtype.  This is a NON-CONSUMING read for inspection and
 * for callers that drive their own decode loop: the entries stay in the cache.  lazy_decode_step
 * does not go through this call; it revives inside its own kernels (same look-up, same rows) and
 * there an entry leaves the Aux Cache the moment its token gets K/V in the next layer.
 * Synchronises the stream; a position not held there gives LAZY_E_NOT_IN_AUX (rows of found
 * positions are still written). */
int aux_cache_revive(lazy_ctx *ctx, void *stream, int32_t layer, int32_t seq,
                     const int32_t *d_positions, int32_t n, void *d_hidden_out);

/* ---- introspection (parity checks, replay of another implementation's kept sets) ------- */

/* Kept set entering `layer_entered` (a schedule point) of sequence `seq` in the latest call
 * (after a decode step: the context re-selected there, the new token included), as
 * original token positions ascending; d_pos: device int32 with room for the count (may be NULL
 * to query the count only).  Synchronises the stream. */
int lazy_get_kept(lazy_ctx *ctx, void *stream, int32_t layer_entered, int32_t seq, int32_t *d_pos,
                  int32_t *h_count);
/* Eq. 1 scores of `layer` for sequence `seq` in the latest call, one per candidate row in
 * ascending position order (prefill: the rows present at that layer; decode: the context the new
 * token attended at that layer, itself last). */
int lazy_get_scores(lazy_ctx *ctx, void *stream, int32_t layer, int32_t seq, float *d_scores,
                    int32_t *h_count);
/* Test hook (no counterpart in the paper): the NEXT prefill (decode step) takes this kept set (positions, ascending, device
 * int32[n]; the last token is kept regardless) at the schedule point instead of selecting by
 * score.  n = 0 clears the hook for that point.  The array must stay valid until that call
 * has run. */
int lazy_set_forced_keep(lazy_ctx *ctx, int32_t layer_entered, int32_t seq, const int32_t *d_pos,
                         int32_t n);
/* With capture on, every prefill also keeps the residual stream after each layer
 * (workspace must have been sized with capture in mind: see lazy_prefill_workspace_bytes_ex). */
size_t lazy_prefill_workspace_bytes_ex(const lazy_model_cfg *cfg, const lazy_schedule *sched,
                                       int32_t debug_capture);
int lazy_set_debug_capture(lazy_ctx *ctx, int32_t on);
/* Residual stream after layer `layer` of the latest PREFILL, all sequences packed:
 * d_out [rows, d_model] (context dtype; may be NULL to query rows).  LAZY_E_STATE if capture
 * was off. */
int lazy_get_hidden(lazy_ctx *ctx, void *stream, int32_t layer, void *d_out, int32_t *h_rows);
/* KV-cache / Aux-Cache contents of a layer for sequence `seq`: positions in order of insertion
 * and the rows.  Any of the device outputs may be NULL. */
int lazy_get_kv(lazy_ctx *ctx, void *stream, int32_t layer, int32_t seq, int32_t *d_pos, void *d_k,
                void *d_v, int32_t *h_count);
int lazy_get_aux(lazy_ctx *ctx, void *stream, int32_t layer, int32_t seq, int32_t *d_pos,
                 void *d_hidden, int32_t *h_count);
/* Positions (ascending) of the tokens of sequence `seq` that the latest decode step revived from
 * the Aux Cache into `layer_entered` (Section 3.2: hidden states fetched from the Aux Cache of the
 * previous layer instead of being recomputed).  Zero after a prefill. */
int lazy_get_revived(lazy_ctx *ctx, void *stream, int32_t layer_entered, int32_t seq, int32_t *d_pos,
                     int32_t *h_count);
int lazy_get_stats(lazy_ctx *ctx, lazy_stats *out);
/* Rows kept at a schedule point (Section 3.2, top-percentile selection as a count): ceil(keep_bp / 10000 *
 * n_total) in integer arithmetic, clamped to [1, n_present]; n_total = tokens of the sequence the
 * percentage refers to, n_present = rows still present before the cut.  The same function sizes every
 * buffer inside the library; 0 on bad arguments. */
int32_t lazy_keep_count(int32_t n_total, uint32_t keep_bp, int32_t n_present);
/* Per-step device times.  With timing on, every kernel launch of lazy_prefill_run is bracketed by
 * CUDA events on the caller's stream; lazy_get_kernel_times synchronises the stream and returns,
 * per kind of step, the summed event time of the latest run together with the ALGORITHMIC work of
 * those launches (floating-point operations for the tensor-core steps, bytes that must move for
 * the memory-bound ones).  Event creation happens inside lazy_set_kernel_timing.  `on`: 0 = off,
 * 1 = every kind, otherwise a bit set shifted left by one ((1 << LAZY_K_x) << 1 per wanted kind), so
 * that a single kernel family can be timed without the events of all the small kernels around it. */
enum {
  LAZY_K_GEMM_QKV = 0, LAZY_K_GEMM_O, LAZY_K_GEMM_GATE_UP, LAZY_K_GEMM_DOWN, LAZY_K_ATTENTION,
  LAZY_K_SCORE, LAZY_K_SELECT, LAZY_K_COMPACT, LAZY_K_RMSNORM, LAZY_K_ROPE_KV, LAZY_K_EMBED,
  LAZY_K_LM_HEAD, LAZY_K_OTHER, LAZY_N_KERNEL_KINDS
};
typedef struct {
  float ms[LAZY_N_KERNEL_KINDS];
  int32_t launches[LAZY_N_KERNEL_KINDS];
  double flops[LAZY_N_KERNEL_KINDS];
  double bytes[LAZY_N_KERNEL_KINDS];
} lazy_kernel_times;
int lazy_set_kernel_timing(lazy_ctx *ctx, int32_t on);
int lazy_get_kernel_times(lazy_ctx *ctx, void *stream, lazy_kernel_times *out);
/* The same measurements launch by launch, in launch order: kind, device time and algorithmic work of
 * every timed launch of the latest run (host arrays with room for `cap` entries; *count receives the
 * number of timed launches, which may exceed cap).  Lets a caller see how a kind's rate depends on the
 * number of surviving rows (the row count follows from the work: flops / flops per row). */
int lazy_get_kernel_events(lazy_ctx *ctx, void *stream, int32_t cap, int32_t *kinds, float *ms, double *flops,
                           double *bytes, int32_t *count);
/* How the scheduled percentile selects (Section 3.2, token pruning).  mode 0 (default): as a count, exactly
 * lazy_keep_count() tokens survive a point, ties going to the lower position, so every row count follows
 * from lengths and schedule and lazy_prefill_run never synchronises.  mode 1: as a threshold, a token is
 * pruned iff its score is smaller than the score at that rank (the last token counting as the largest), so
 * tokens tied with the threshold all survive and later layers may see more rows than scheduled; the kept
 * count of every sequence is then read back from the device at each point (one stream synchronisation per
 * point in lazy_prefill_run, one more per point in lazy_decode_step).  Without ties both modes select the
 * same sets.  Takes effect with the next lazy_prefill_run / lazy_decode_step. */
int lazy_set_selection(lazy_ctx *ctx, int32_t mode);
/* 8-bit projections (no counterpart in the paper, which runs 16-bit weights; a deployment option for the
 * "linear layers" of Section 3.1).  With fp8 weights set, lazy_prefill_run computes the four projections of
 * every layer (QKV, output, gate/up, down) on e4m3 operands with fp32 accumulation: the weights are the e4m3
 * codes given here times one scale per matrix, the activations are quantised per row on the way in (scale =
 * max|x| / 448, nearest-even e4m3 code of x / scale, decided in fp32).  Everything else (normalisation,
 * attention, scores, selection, the LM head, every lazy_decode_step) stays in the context's bf16 arithmetic
 * and bf16 weights.  bf16 contexts only.  Arrays: host arrays of n_layers entries; code matrices: device,
 * same [out, in] shapes as their 16-bit counterparts, one byte per element, 16-byte aligned, in-features a
 * multiple of 16.  The pointers must stay valid while set; NULL switches back to the 16-bit weights. */
typedef struct {
  const void *const *w_qkv, *const *w_o, *const *w_gate, *const *w_up, *const *w_down;
  const float *s_qkv, *s_o, *s_gate, *s_up, *s_down;
} lazy_fp8_weights;
int lazy_set_fp8_weights(lazy_ctx *ctx, const lazy_fp8_weights *w);
/* Where the scoring layer is cut (Section 3.2, Aux Cache paragraph).  after_layer = 0 (default): between
 * the layer's attention half and its MLP, so that MLP already runs on the kept rows, the Aux Cache holds
 * post-attention hidden states and a revived token first gets that layer's MLP.  after_layer = 1: after
 * the whole layer, as the paragraph is worded: the MLP runs on every row and the Aux Cache holds layer
 * outputs.  The MLP is row-wise, so logits, kept sets and revivals are the same either way; what changes
 * is the Aux Cache content and the number of MLP rows.  Call before lazy_prefill_run: a change of the
 * setting invalidates the caches of an earlier prefill (decode then returns LAZY_E_STATE). */
int lazy_set_aux_point(lazy_ctx *ctx, int32_t after_layer);
/* Synchronises `stream` and returns the first device-side error recorded since the last call
 * of this function (LAZY_OK if none), clearing it.  Plumbing: no counterpart in the paper.  After a
 * LAZY_E_TIMEOUT the context stays usable: the next lazy_prefill_run / lazy_decode_step starts by
 * clearing the arrival counters an aborted GEMM may have left behind. */
int lazy_sync_status(lazy_ctx *ctx, void *stream);
/* Same, for the context-free calls below. */
int lazy_device_status(void *stream);
/* Where the latest non-OK device status taken by this process came from: *where = code of the wait or
 * check that failed (1..4 GEMM roles, 5 gather index, 6 Aux look-up, 7 token id, 8 selection, 9 decode
 * planning, 10 RoPE position, 11..13 attention roles, 14 split-wave counter wait, 15 wait self-test),
 * *a / *b two integers of context (CTA and parity for a wait, row and value for a check).  Any pointer
 * may be NULL.  Plumbing: no counterpart in the paper. */
int lazy_status_detail(int32_t *where, int32_t *a, int32_t *b);
/* Self-test of the bounded device-side waits (no counterpart in the paper).  Enqueues a one-warp kernel
 * that waits, for at most limit_us microseconds (1..100000), on something that is never signalled:
 * which = 0 an mbarrier phase (the wait every tensor-core role uses), which = 1 the arrival counter of
 * the split last GEMM wave.  No copy, MMA or tensor-memory allocation is in flight, so the wait simply
 * runs out: the kernel records LAZY_E_TIMEOUT in the status word and returns, and the device stays
 * usable.  The status surfaces through lazy_device_status(). */
int lazy_k_wait_selftest(void *stream, int32_t which, uint32_t limit_us);
void lazy_destroy(lazy_ctx *ctx);
const char *lazy_strerror(int status);

/* ---- single-layer pruning op ------------------------------------------------------------ */

/* One layer's attention half followed by the cut (Section 3.2): RMSNorm, QKV projection, RoPE,
 * causal attention, output projection + residual, Eq. 1 score of the last row, top-percentile
 * selection, then gather of the kept hidden / K / V / position rows and scatter of the pruned
 * hidden rows into an Aux Cache.  All pointers device, bf16 (dtype LAZY_BF16) or fp32.
 *   x [n, d] hidden states entering the layer; pos int32[n] ascending positions;
 *   w_qkv [3d, d], w_o [d, d], g_attn [d]; keep_bp: keep ceil(keep_bp/10000*n) rows;
 *   max_pos: every position is < max_pos (sizes the RoPE table kept in the workspace).
 * Outputs: scores fp32[n]; keep_idx int32[n_keep], drop_idx int32[n-n_keep] (row indices,
 * ascending); hidden_kept [n_keep, d], k_kept / v_kept [n_keep, d] (k rotated),
 * pos_kept int32[n_keep]; aux_hidden [n-n_keep, d], aux_pos int32[n-n_keep].
 * d_workspace: lazy_prune_op_workspace_bytes(...) bytes.  forced_keep_idx (device, may be NULL):
 * n_forced row indices ascending that replace the score-based choice (test hook). */
size_t lazy_prune_op_workspace_bytes(int32_t n, int32_t d_model, int32_t n_heads, int32_t head_dim,
                                     int32_t dtype, int32_t max_pos);
int lazy_prune_op(void *stream, int32_t dtype, int32_t n, int32_t d_model, int32_t n_heads,
                  int32_t head_dim, int32_t max_pos, float rms_eps, float rope_theta, uint32_t keep_bp,
                  const void *x, const int32_t *pos, const void *w_qkv, const void *w_o,
                  const void *g_attn, const int32_t *forced_keep_idx, int32_t n_forced,
                  float *scores, int32_t *keep_idx, int32_t *drop_idx, void *hidden_kept,
                  void *k_kept, void *v_kept, int32_t *pos_kept, void *aux_hidden,
                  int32_t *aux_pos, void *d_workspace, size_t workspace_bytes);

/* ---- individual steps of the path (each also used inside the calls above) ----------------- */

/* y[r,:] = x[r,:] * rsqrt(mean(x[r,:]^2) + eps) * g  (Llama-2 pre-norm). x, y [n, d]. */
int lazy_k_rmsnorm(void *stream, int32_t dtype, const void *x, const void *g, void *y, int32_t n,
                   int32_t d, float eps);
/* C[M,N] = A[M,K] * B[N,K]^T (+ R[M,N] if R != NULL): the dense products of the layers of
 * Section 3.1 / 3.2. bf16: tcgen05 tensor cores, TMA-fed;
 * fp32: CUDA cores. lda = K, ldc = N (dense).  K and N multiples of 8.  impl: 0 = the
 * dtype's production kernel (bf16: weight streaming for M <= 4; tensor cores above, with one CTA
 * per 128x256 tile or a CTA pair per 256x256 tile, whichever measured faster for the shape),
 * 1 = the CUDA-core kernel (cross-check), 2 / 3 = bf16 tensor cores with one CTA per tile / with
 * CTA pairs at every M > 128 (cross-checks of one against the other). */
int lazy_k_gemm(void *stream, int32_t dtype, int32_t impl, const void *A, const void *B,
                const void *R, void *C, int32_t M, int32_t N, int32_t K);
/* The same product with a device scratch of lazy_k_gemm_scratch_bytes() bytes that the bf16
 * tensor-core kernels use to split the last, partial wave of output tiles along K (partial sums and
 * arrival counters).  The scratch must be zero before its first use, is left zero by every call,
 * and must not be shared by calls running at the same time.  Results do not depend on it being
 * given (the parts of a tile are added in a fixed order).  The paper has no counterpart: this is
 * scheduling of the dense products of Section 3.2's layers.  NULL scratch = lazy_k_gemm.  If a call
 * ended in LAZY_E_TIMEOUT, zero the first 2048 bytes of the scratch before using it again. */
size_t lazy_k_gemm_scratch_bytes(void);
int lazy_k_gemm_ws(void *stream, int32_t dtype, int32_t impl, const void *A, const void *B,
                   const void *R, void *C, int32_t M, int32_t N, int32_t K, void *d_scratch,
                   size_t scratch_bytes);
/* C[M,F] = silu(A Bg^T) * (A Bu^T), Bg, Bu [F, K] (SwiGLU, first half of the MLP). */
int lazy_k_gemm_swiglu(void *stream, int32_t dtype, int32_t impl, const void *A, const void *Bg,
                       const void *Bu, void *C, int32_t M, int32_t F, int32_t K);
int lazy_k_gemm_swiglu_ws(void *stream, int32_t dtype, int32_t impl, const void *A, const void *Bg,
                          const void *Bu, void *C, int32_t M, int32_t F, int32_t K, void *d_scratch,
                          size_t scratch_bytes);
/* Per-row e4m3 quantisation of bf16 activations x [M, K] (K a multiple of 16): q [M, K] receives the codes
 * (bytes), scale [M] (device fp32) the row scales max|x| / 448 (1 for an all-zero row). */
int lazy_k_quant_rows_e4m3(void *stream, const void *x, void *q, float *scale, int32_t M, int32_t K);
/* C[M,N] = (A8 B8^T) * a_scale[row] * w_scale (+ R) in bf16, A8 [M,K] / B8 [N,K] e4m3 codes, tcgen05
 * kind::f8f6f4 with fp32 accumulation.  With B8u != NULL: C[M,N] = silu(A8 B8^T * s) * (A8 B8u^T * s_up), the
 * first half of the MLP (R must be NULL).  M > 0, K a multiple of 16, N a multiple of 8. */
int lazy_k_gemm_fp8(void *stream, const void *A8, const float *a_scale, const void *B8, float w_scale,
                    const void *B8u, float w_scale_up, const void *R, void *C, int32_t M, int32_t N, int32_t K);
/* In-place RoPE of q and k inside qkv [n, 3*H*dh] by positions pos[n]; rotated k and v are
 * also written to kcache / vcache [n, H*dh].  rope_table: device fp32[max_pos*head_dim] scratch
 * that the call fills first. */
int lazy_k_rope_kv(void *stream, int32_t dtype, void *qkv, const int32_t *pos, float *rope_table,
                   void *kcache, void *vcache, int32_t n, int32_t n_heads, int32_t head_dim,
                   int32_t max_pos, float theta);
/* Causal multi-head attention over packed sequences. q: rows of stride ldq elements, k/v rows of
 * stride ldkv; o [n, H*dh] dense. d_cu_seqlens: device int32[n_seqs+1]. */
int lazy_k_attention(void *stream, int32_t dtype, const void *q, int32_t ldq, const void *k,
                     const void *v, int32_t ldkv, void *o, const int32_t *d_cu_seqlens,
                     int32_t n_seqs, int32_t max_len, int32_t n_total, int32_t n_heads,
                     int32_t head_dim);
/* Eq. 1: s[j] = (1/H) sum_h softmax_j(q_last,h . k_j,h / sqrt(dh)) per sequence, q_last = the
 * sequence's last row. scratch: device fp32[lazy_k_score_scratch_floats(...)]. */
size_t lazy_k_score_scratch_floats(int32_t n_seqs, int32_t n_total, int32_t n_heads);
int lazy_k_score(void *stream, int32_t dtype, const void *q, int32_t ldq, const void *k,
                 int32_t ldkv, const int32_t *d_cu_seqlens, int32_t n_seqs, int32_t n_total,
                 int32_t n_heads, int32_t head_dim, float *scratch, float *scores);
/* Same result as lazy_k_score, for callers that cannot allocate device memory (no counterpart in
 * the paper: this is a deployment convenience).  Such callers exist: a plugin inside a host
 * application that owns all device memory, a latency-critical callback where cudaMalloc would
 * stall the device, a process that has already handed its memory to another owner.  The scratch
 * (per-head logits and softmax statistics) lives in a fixed array inside the library that every
 * GPU loading it holds until exit (about 1.04 MB).  Limits: n_heads * n_total <= 262144 and
 * 2 * n_heads * n_seqs <= 4096; anything larger returns LAZY_E_CAPACITY and runs nothing.  The
 * call allocates and frees nothing.  The first call on each device looks up the array's device
 * address (a synchronous runtime query), so make that first call outside any stream capture; the
 * address is remembered per device for the life of the process, so do not call this on a device
 * after a cudaDeviceReset of it.
 * All calls share the one array, which simply keeps what the last call left there (nothing needs
 * clearing: every value read is written earlier by the same call); two calls whose kernels may
 * overlap on the GPU (different streams, different threads) race on it, so serialise them. */
int lazy_k_score_static(void *stream, int32_t dtype, const void *q, int32_t ldq, const void *k,
                        int32_t ldkv, const int32_t *d_cu_seqlens, int32_t n_seqs, int32_t n_total,
                        int32_t n_heads, int32_t head_dim, float *scores);
/* Top-percentile selection per sequence (Section 3.2): keeps n_keep[s] rows with the largest
 * score, the last row always, ties to the lower index.  d_cu_in / d_cu_keep: device
 * int32[n_seqs+1] prefix sums of rows in / rows kept.  keep_idx / drop_idx receive packed row
 * indices (global, ascending within a sequence); drop rows of sequence s start at
 * d_cu_in[s]-d_cu_keep[s]. */
int lazy_k_select(void *stream, const float *scores, const int32_t *d_cu_in,
                  const int32_t *d_cu_keep, int32_t n_seqs, int32_t *keep_idx, int32_t *drop_idx);
/* The same selection read as a threshold (Section 3.2: a token is pruned if its score is smaller than the
 * k-th percentile among the input tokens): per sequence of n rows, tau = the order statistic with
 * index floor((n-1) * prune_bp / 10000) from below (prune_bp = percentile in basis points, 0..9999; the
 * "lower" percentile definition, no interpolation), every row with score >= tau is kept, the last row
 * always.  Ties at tau are all kept, so the count depends on the data: keep_idx / drop_idx (device
 * int32[n_total]) are packed per sequence from d_cu_in[s], ascending, and d_counts[s] (device
 * int32[n_seqs]) receives the number kept.  A step-level call: the prefill and decode calls above use
 * the count-based form, whose counts the host knows before launching. */
int lazy_k_select_threshold(void *stream, const float *scores, const int32_t *d_cu_in, int32_t n_seqs,
                            uint32_t prune_bp, int32_t *keep_idx, int32_t *drop_idx, int32_t *d_counts);
/* dst[i,:] = src[idx[i],:] for i < n (row gather), rows of `row_bytes` bytes (multiple of 16);
 * src has src_rows rows (indices outside are reported, not dereferenced). */
int lazy_k_gather_rows(void *stream, const void *src, const int32_t *idx, void *dst, int32_t n,
                       int32_t row_bytes, int32_t src_rows);

#ifdef __cplusplus
}
#endif
#endif /* LAZYLLM_H_ */
