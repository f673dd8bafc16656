// Context-free entry points: the individual steps of the path and the single-layer pruning op.
#include "gemm_epilogue.cuh"
#include "runtime.cuh"

using namespace lazy;

namespace {
inline bool bad_dtype(int dtype) { return dtype != LAZY_BF16 && dtype != LAZY_F32; }
}  // namespace

extern "C" {

int lazy_k_rmsnorm(void *stream, int32_t dtype, const void *x, const void *g, void *y, int32_t n,
                   int32_t d, float eps) {
  if (bad_dtype(dtype) || !x || !g || !y || n < 0 || d < 1 || d % 8) return LAZY_E_BADARG;
  return launch_rmsnorm((cudaStream_t)stream, dtype, x, g, y, n, d, eps);
}

size_t lazy_k_gemm_scratch_bytes(void) { return gemm_scratch_bytes(); }

int lazy_k_gemm(void *stream, int32_t dtype, int32_t impl, const void *A, const void *B, const void *R,
                void *C, int32_t M, int32_t N, int32_t K) {
  return lazy_k_gemm_ws(stream, dtype, impl, A, B, R, C, M, N, K, nullptr, 0);
}

int lazy_k_gemm_ws(void *stream, int32_t dtype, int32_t impl, const void *A, const void *B, const void *R,
                   void *C, int32_t M, int32_t N, int32_t K, void *d_scratch, size_t scratch_bytes) {
  if (bad_dtype(dtype) || M < 0 || N < 1 || K < 1 || N % 8 || K % 8) return LAZY_E_BADARG;
  if (M == 0) return LAZY_OK;  // nothing to compute; an empty matrix may have no address
  if (!A || !B || !C) return LAZY_E_BADARG;
  DevStatus *status = dev_status_ptr();
  if (!status) return LAZY_E_CUDA;
  if (impl == 1) return launch_gemm_simt((cudaStream_t)stream, dtype, A, B, nullptr, R, C, M, N, K, 0);
  return launch_gemm((cudaStream_t)stream, dtype, A, B, R, C, M, N, K, status, d_scratch, scratch_bytes,
                     impl == 2 ? 1 : (impl == 3 ? 2 : 0));
}

int lazy_k_gemm_swiglu(void *stream, int32_t dtype, int32_t impl, const void *A, const void *Bg,
                       const void *Bu, void *C, int32_t M, int32_t F, int32_t K) {
  return lazy_k_gemm_swiglu_ws(stream, dtype, impl, A, Bg, Bu, C, M, F, K, nullptr, 0);
}

int lazy_k_gemm_swiglu_ws(void *stream, int32_t dtype, int32_t impl, const void *A, const void *Bg,
                          const void *Bu, void *C, int32_t M, int32_t F, int32_t K, void *d_scratch,
                          size_t scratch_bytes) {
  if (bad_dtype(dtype) || M < 0 || F < 1 || K < 1 || F % 8 || K % 8) return LAZY_E_BADARG;
  if (M == 0) return LAZY_OK;
  if (!A || !Bg || !Bu || !C) return LAZY_E_BADARG;
  DevStatus *status = dev_status_ptr();
  if (!status) return LAZY_E_CUDA;
  if (impl == 1) return launch_gemm_simt((cudaStream_t)stream, dtype, A, Bg, Bu, nullptr, C, M, F, K, 1);
  return launch_gemm_swiglu((cudaStream_t)stream, dtype, A, Bg, Bu, C, M, F, K, status, d_scratch, scratch_bytes,
                            impl == 2 ? 1 : (impl == 3 ? 2 : 0));
}

int lazy_k_quant_rows_e4m3(void *stream, const void *x, void *q, float *scale, int32_t M, int32_t K) {
  if (M < 0 || K < 16 || K % 16) return LAZY_E_BADARG;
  if (M == 0) return LAZY_OK;
  if (!x || !q || !scale) return LAZY_E_BADARG;
  return launch_quant_rows_e4m3((cudaStream_t)stream, x, q, scale, M, K);
}

int lazy_k_gemm_fp8(void *stream, const void *A8, const float *a_scale, const void *B8, float w_scale,
                    const void *B8u, float w_scale_up, const void *R, void *C, int32_t M, int32_t N, int32_t K) {
  if (M < 0 || N < 8 || K < 16 || N % 8 || K % 16) return LAZY_E_BADARG;
  if (M == 0) return LAZY_OK;
  if (!A8 || !a_scale || !B8 || !C || (B8u && R)) return LAZY_E_BADARG;
  DevStatus *status = dev_status_ptr();
  if (!status) return LAZY_E_CUDA;
  const int epi = B8u ? EPI_SWIGLU : (R ? EPI_RESIDUAL : EPI_PLAIN);
  return launch_gemm_fp8((cudaStream_t)stream, epi, A8, a_scale, B8, w_scale, B8u, w_scale_up, R, C, M, N, K, status,
                         RopeArgs(), nullptr, 0);
}

int lazy_k_rope_kv(void *stream, int32_t dtype, void *qkv, const int32_t *pos, float *rope_table,
                   void *kcache, void *vcache, int32_t n, int32_t n_heads, int32_t head_dim,
                   int32_t max_pos, float theta) {
  const int v = dtype == LAZY_F32 ? 4 : 8;
  if (bad_dtype(dtype) || !qkv || !pos || !rope_table || !kcache || !vcache || n < 0 || n_heads < 1 ||
      head_dim < 2 || (head_dim / 2) % v || max_pos < 1)
    return LAZY_E_BADARG;
  DevStatus *status = dev_status_ptr();
  if (!status) return LAZY_E_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  LAZY_TRY(launch_rope_table(st, rope_table, max_pos, head_dim, theta));
  return launch_rope_kv(st, dtype, qkv, pos, rope_table, kcache, vcache, nullptr, nullptr, n, n_heads,
                        head_dim, max_pos, status);
}

int lazy_k_attention(void *stream, int32_t dtype, const void *q, int32_t ldq, const void *k,
                     const void *v, int32_t ldkv, void *o, const int32_t *d_cu_seqlens, int32_t n_seqs,
                     int32_t max_len, int32_t n_total, int32_t n_heads, int32_t head_dim) {
  if (bad_dtype(dtype) || !q || !k || !v || !o || !d_cu_seqlens || n_seqs < 0 || n_total < 0 ||
      max_len < 0 || n_heads < 1 || head_dim < 32 || head_dim % 32)
    return LAZY_E_BADARG;
  if (attention_tc_eligible(dtype, head_dim, ldq, ldkv)) {
    DevStatus *status = dev_status_ptr();
    if (!status) return LAZY_E_CUDA;
    return launch_attention_tc((cudaStream_t)stream, q, ldq, n_total, k, v, ldkv, n_total, o, n_heads,
                               d_cu_seqlens, nullptr, n_seqs, max_len, 0, 0, 0, status);
  }
  return launch_attention((cudaStream_t)stream, dtype, q, ldq, k, v, ldkv, o, d_cu_seqlens, nullptr,
                          n_seqs, max_len, n_total, n_heads, head_dim);
}

size_t lazy_k_score_scratch_floats(int32_t n_seqs, int32_t n_total, int32_t n_heads) {
  if (n_seqs < 0 || n_total < 0 || n_heads < 0) return 0;
  return score_scratch_floats(n_seqs, n_total, n_heads);
}

int lazy_k_score(void *stream, int32_t dtype, const void *q, int32_t ldq, const void *k, int32_t ldkv,
                 const int32_t *d_cu_seqlens, int32_t n_seqs, int32_t n_total, int32_t n_heads,
                 int32_t head_dim, float *scratch, float *scores) {
  if (bad_dtype(dtype) || !q || !k || !d_cu_seqlens || !scratch || !scores || n_seqs < 0 || n_total < 0 ||
      n_heads < 1)
    return LAZY_E_BADARG;
  // the longest sequence is not known here: size the key grid for the whole batch
  return launch_score((cudaStream_t)stream, dtype, q, ldq, k, ldkv, d_cu_seqlens, nullptr, n_seqs, n_total,
                      n_total, n_heads, head_dim, scratch, scores);
}

int lazy_k_select(void *stream, const float *scores, const int32_t *d_cu_in, const int32_t *d_cu_keep,
                  int32_t n_seqs, int32_t *keep_idx, int32_t *drop_idx) {
  if (!scores || !d_cu_in || !d_cu_keep || !keep_idx || !drop_idx || n_seqs < 0) return LAZY_E_BADARG;
  DevStatus *status = dev_status_ptr();
  if (!status) return LAZY_E_CUDA;
  return launch_select((cudaStream_t)stream, scores, d_cu_in, d_cu_keep, n_seqs, keep_idx, drop_idx, status);
}

int lazy_k_select_threshold(void *stream, const float *scores, const int32_t *d_cu_in, int32_t n_seqs,
                            uint32_t prune_bp, int32_t *keep_idx, int32_t *drop_idx, int32_t *d_counts) {
  if (!scores || !d_cu_in || !keep_idx || !drop_idx || !d_counts || n_seqs < 0 || prune_bp > 9999)
    return LAZY_E_BADARG;
  return launch_select_threshold((cudaStream_t)stream, scores, d_cu_in, n_seqs, prune_bp, keep_idx, drop_idx,
                                 d_counts);
}

int lazy_k_gather_rows(void *stream, const void *src, const int32_t *idx, void *dst, int32_t n,
                       int32_t row_bytes, int32_t src_rows) {
  if (n < 0 || row_bytes < 16 || row_bytes % 16 || src_rows < 0) return LAZY_E_BADARG;
  if (n == 0) return LAZY_OK;
  if (!src || !dst) return LAZY_E_BADARG;
  DevStatus *status = dev_status_ptr();
  if (!status) return LAZY_E_CUDA;
  return launch_gather_rows((cudaStream_t)stream, src, idx, dst, n, row_bytes, src_rows, status);
}

// ---- single-layer pruning op ----------------------------------------------------------------------
// workspace: h [n,d] | qkv [n,3d] | attn [n,d] | y [n,d] | K [n,d] | V [n,d] | rope table |
//            score scratch | sel scores [n] | cu_in[2] cu_keep[2]
namespace {
struct PruneWs {
  char *h, *qkv, *attn, *y, *k, *v;
  float *rope, *sscratch, *sel;
  int32_t *cu;
  size_t bytes;
};
PruneWs prune_carve(char *base, int n, int d, int H, int dh, int dtype, int max_pos) {
  PruneWs w;
  size_t off = 0;
  const size_t rb = (size_t)d * elem_bytes(dtype);
  auto take = [&](size_t b) {
    char *p = base ? base + off : nullptr;
    off += align_up(b ? b : 1, 256);
    return p;
  };
  w.h = take((size_t)n * rb);
  w.qkv = take((size_t)n * rb * 3);
  w.attn = take((size_t)n * rb);
  w.y = take((size_t)n * rb);
  w.k = take((size_t)n * rb);
  w.v = take((size_t)n * rb);
  w.rope = (float *)take((size_t)max_pos * dh * 4);
  w.sscratch = (float *)take(score_scratch_floats(1, n, H) * 4);
  w.sel = (float *)take((size_t)n * 4);
  w.cu = (int32_t *)take(16 * 4);
  w.bytes = off;
  return w;
}
}  // namespace

size_t lazy_prune_op_workspace_bytes(int32_t n, int32_t d_model, int32_t n_heads, int32_t head_dim,
                                     int32_t dtype, int32_t max_pos) {
  if (n < 1 || d_model < 1 || n_heads < 1 || head_dim < 1 || bad_dtype(dtype) || max_pos < 1) return 0;
  return prune_carve(nullptr, n, d_model, n_heads, head_dim, dtype, max_pos).bytes;
}

int lazy_prune_op(void *stream, int32_t dtype, int32_t n, int32_t d_model, int32_t n_heads,
                  int32_t head_dim, int32_t max_pos, float rms_eps, float rope_theta, uint32_t keep_bp,
                  const void *x,
                  const int32_t *pos, const void *w_qkv, const void *w_o, const void *g_attn,
                  const int32_t *forced_keep_idx, int32_t n_forced, float *scores, int32_t *keep_idx,
                  int32_t *drop_idx, void *hidden_kept, void *k_kept, void *v_kept, int32_t *pos_kept,
                  void *aux_hidden, int32_t *aux_pos, void *d_workspace, size_t workspace_bytes) {
  lazy_model_cfg cfg = {1, d_model, n_heads, head_dim, 8, 8, rms_eps, rope_theta, dtype, 1, n > 0 ? n : 1, 0};
  LAZY_TRY(validate_cfg(&cfg));
  if (n < 1 || max_pos < 1 || keep_bp < 1 || keep_bp > 10000) return LAZY_E_BADARG;
  if (!x || !pos || !w_qkv || !w_o || !g_attn || !scores || !keep_idx || !drop_idx || !hidden_kept ||
      !k_kept || !v_kept || !pos_kept || !aux_hidden || !aux_pos || !d_workspace)
    return LAZY_E_BADARG;
  if (((uintptr_t)d_workspace & 255)) return LAZY_E_BADARG;
  PruneWs w = prune_carve((char *)d_workspace, n, d_model, n_heads, head_dim, dtype, max_pos);
  if (workspace_bytes < w.bytes) return LAZY_E_CAPACITY;
  int n_keep = keep_count(n, keep_bp, n);
  if (forced_keep_idx) {
    if (n_forced < 1 || n_forced > n) return LAZY_E_BADARG;
    n_keep = n_forced;
  }
  const int n_drop = n - n_keep;
  cudaStream_t st = (cudaStream_t)stream;
  DevStatus *status = dev_status_ptr();
  if (!status) return LAZY_E_CUDA;
  const int d = d_model;
  const int rb = d * elem_bytes(dtype);
  const int32_t h_cu[4] = {0, n, 0, n_keep};
  LAZY_CUDA_OK(cudaMemcpyAsync(w.cu, h_cu, sizeof(h_cu), cudaMemcpyHostToDevice, st));
  LAZY_TRY(launch_rope_table(st, w.rope, max_pos, head_dim, rope_theta));
  LAZY_TRY(launch_rmsnorm(st, dtype, x, g_attn, w.h, n, d, rms_eps));
  LAZY_TRY(launch_gemm(st, dtype, w.h, w_qkv, nullptr, w.qkv, n, 3 * d, d, status));
  LAZY_TRY(launch_rope_kv(st, dtype, w.qkv, pos, w.rope, w.k, w.v, nullptr, nullptr, n, n_heads, head_dim,
                          max_pos, status));
  if (attention_tc_eligible(dtype, head_dim, 3 * d, d))
    LAZY_TRY(launch_attention_tc(st, w.qkv, 3 * d, n, w.k, w.v, d, n, w.attn, n_heads, nullptr, nullptr, 1, n,
                                 0, n, 0, status));
  else
    LAZY_TRY(launch_attention(st, dtype, w.qkv, 3 * d, w.k, w.v, d, w.attn, w.cu, nullptr, 1, n, n, n_heads,
                              head_dim));
  LAZY_TRY(launch_score(st, dtype, w.qkv, 3 * d, w.k, d, w.cu, nullptr, 1, n, n, n_heads, head_dim,
                        w.sscratch, scores));
  LAZY_TRY(launch_gemm(st, dtype, w.attn, w_o, x, w.y, n, d, d, status));
  const float *sel = scores;
  if (forced_keep_idx) {
    // forced rows get score 2, the rest 0: the selection then reproduces exactly that set.
    // Row indices double as "positions" of an identity position list here.
    LAZY_TRY(launch_iota_pos(st, (int32_t *)w.h, w.cu, 1, n));
    LAZY_TRY(launch_forced_scores(st, (const int32_t *)w.h, 0, n, forced_keep_idx, n_forced, w.sel));
    sel = w.sel;
  }
  LAZY_TRY(launch_select(st, sel, w.cu, w.cu + 2, 1, keep_idx, drop_idx, status));
  LAZY_TRY(launch_gather_rows(st, w.y, keep_idx, hidden_kept, n_keep, rb, n, status));
  LAZY_TRY(launch_gather_rows(st, w.k, keep_idx, k_kept, n_keep, rb, n, status));
  LAZY_TRY(launch_gather_rows(st, w.v, keep_idx, v_kept, n_keep, rb, n, status));
  LAZY_TRY(launch_gather_i32(st, pos, keep_idx, pos_kept, n_keep));
  LAZY_TRY(launch_gather_rows(st, w.y, drop_idx, aux_hidden, n_drop, rb, n, status));
  LAZY_TRY(launch_gather_i32(st, pos, drop_idx, aux_pos, n_drop));
  return LAZY_OK;
}

}  // extern "C"
