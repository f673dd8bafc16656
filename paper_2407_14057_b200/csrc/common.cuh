// Shared declarations of the CUDA side: status word, launch helpers, storage-type traits.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "lazyllm.h"

namespace lazy {

// ---- device status word -------------------------------------------------------------------
// First error wins.  `where` identifies the wait or check that failed.
struct DevStatus {
  int code;
  int where;
  int a;
  int b;
};

enum DevWhere {
  W_GEMM_PRODUCER = 1,
  W_GEMM_MMA_FULL = 2,
  W_GEMM_MMA_TMEM = 3,
  W_GEMM_EPILOGUE = 4,
  W_GATHER_INDEX = 5,
  W_AUX_LOOKUP = 6,
  W_EMBED_ID = 7,
  W_SELECT = 8,
  W_DECODE = 9,
  W_ROPE_POS = 10,
  W_ATTN_PRODUCER = 11,
  W_ATTN_MMA = 12,
  W_ATTN_SOFTMAX = 13,
  W_GEMM_TAIL = 14,
  W_WAIT_SELFTEST = 15,
};

__device__ __forceinline__ void dev_fail(DevStatus *st, int code, int where, int a = 0, int b = 0) {
  if (atomicCAS(&st->code, 0, code) == 0) {
    st->where = where;
    st->a = a;
    st->b = b;
  }
}

// Address of this device's status word (a __device__ global of the library); NULL on failure.
DevStatus *dev_status_ptr();
// Synchronises the stream, returns and clears the status word.  The detail fields of the latest
// non-OK status taken by this process stay readable through last_status_detail().
int sync_and_take_status(cudaStream_t stream, int *where_out);
void last_status_detail(int *where, int *a, int *b);

// ---- storage types --------------------------------------------------------------------------
typedef __nv_bfloat16 bf16;

template <typename T>
struct Elem;
template <>
struct Elem<float> {
  static constexpr int kPerVec = 4;  // elements per 16-byte vector
  __device__ static __forceinline__ float to_f(float v) { return v; }
  __device__ static __forceinline__ float from_f(float v) { return v; }
};
template <>
struct Elem<bf16> {
  static constexpr int kPerVec = 8;
  __device__ static __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
  __device__ static __forceinline__ bf16 from_f(float v) { return __float2bfloat16_rn(v); }
};

__device__ __forceinline__ void bf16x2_unpack(uint32_t u, float &lo, float &hi) {
  lo = __uint_as_float(u << 16);
  hi = __uint_as_float(u & 0xffff0000u);
}
__device__ __forceinline__ uint32_t bf16x2_pack(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

// 16-byte vector of T, unpacked to floats and back.
template <typename T>
struct Vec16 {
  uint4 raw;
  __device__ __forceinline__ void load(const T *p) { raw = *reinterpret_cast<const uint4 *>(p); }
  __device__ __forceinline__ void store(T *p) const { *reinterpret_cast<uint4 *>(p) = raw; }
  __device__ __forceinline__ void unpack(float *f) const;
  __device__ __forceinline__ void pack(const float *f);
};
template <>
__device__ __forceinline__ void Vec16<float>::unpack(float *f) const {
  f[0] = __uint_as_float(raw.x);
  f[1] = __uint_as_float(raw.y);
  f[2] = __uint_as_float(raw.z);
  f[3] = __uint_as_float(raw.w);
}
template <>
__device__ __forceinline__ void Vec16<float>::pack(const float *f) {
  raw = make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]),
                   __float_as_uint(f[3]));
}
template <>
__device__ __forceinline__ void Vec16<bf16>::unpack(float *f) const {
  bf16x2_unpack(raw.x, f[0], f[1]);
  bf16x2_unpack(raw.y, f[2], f[3]);
  bf16x2_unpack(raw.z, f[4], f[5]);
  bf16x2_unpack(raw.w, f[6], f[7]);
}
template <>
__device__ __forceinline__ void Vec16<bf16>::pack(const float *f) {
  raw = make_uint4(bf16x2_pack(f[0], f[1]), bf16x2_pack(f[2], f[3]), bf16x2_pack(f[4], f[5]),
                   bf16x2_pack(f[6], f[7]));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

inline int elem_bytes(int dtype) { return dtype == LAZY_F32 ? 4 : 2; }
inline int cdiv(int a, int b) { return (a + b - 1) / b; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Number of SMs of the current device (cached).
int sm_count();
// Counts kernels enqueued by this library (per process); used for the launch statistics.
extern long long g_launches;
#define LAZY_COUNT_LAUNCH() (++::lazy::g_launches)

#define LAZY_CUDA_OK(expr)                      \
  do {                                          \
    cudaError_t e__ = (expr);                   \
    if (e__ != cudaSuccess) return LAZY_E_CUDA; \
  } while (0)
#define LAZY_TRY(expr)                \
  do {                                \
    int rc__ = (expr);                \
    if (rc__ != LAZY_OK) return rc__; \
  } while (0)

// Programmatic dependent launch, used along the chain of small kernels of a decode step: the grid may be
// set up while the kernel before it in the stream drains.  Such a kernel starts with LAZY_PDL_ENTER(): it
// releases its own dependent right away and then waits for the grid before it to complete and flush (which,
// that grid having waited in its turn, covers everything earlier in the stream).  Launched the ordinary
// way the two instructions do nothing.
#define LAZY_PDL_ENTER()                                                  \
  do {                                                                    \
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");       \
    asm volatile("griddepcontrol.wait;" ::: "memory");                    \
  } while (0)

template <typename... KArgs, typename... Args>
inline int launch_pdl(void (*kfn)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kfn, static_cast<KArgs>(args)...) == cudaSuccess ? LAZY_OK : LAZY_E_CUDA;
}

inline int launch_ok() { return cudaPeekAtLastError() == cudaSuccess ? LAZY_OK : LAZY_E_CUDA; }

// ---- launchers (one per step of the path); all enqueue on `st` and return a lazy_status ----
int launch_embed(cudaStream_t st, int dtype, const void *table, const int32_t *ids, void *x, int n,
                 int d, int vocab, DevStatus *status);
int launch_rmsnorm(cudaStream_t st, int dtype, const void *x, const void *g, void *y, int n, int d,
                   float eps);
// rows listed in row_idx (or rows 0..n-1 if NULL) of x -> y rows 0..n-1
int launch_rmsnorm_rows(cudaStream_t st, int dtype, const void *x, const int32_t *row_idx,
                        const void *g, void *y, int n, int d, float eps);
int launch_rope_table(cudaStream_t st, float *table, int max_pos, int head_dim, float theta);
// Per-row e4m3 quantisation of bf16 activations x [M, K]: q [M, K] codes (bytes), scale [M]; K multiple of 16.
int launch_quant_rows_e4m3(cudaStream_t st, const void *x, void *q, float *scale, int M, int K);
// q rotated in place inside qkv; rotated k and v written to the caches at row kv_row[r]
// (or r if kv_row is NULL) together with the position tag.  Grouped-query attention: n_kv_heads key/value
// heads (0 = n_heads); a row of qkv is [q: n_heads*dh | k: n_kv_heads*dh | v: n_kv_heads*dh], a cache row
// n_kv_heads*dh wide.  Every attention / score launcher below takes the same n_kv_heads: query head h reads
// key/value head h / (n_heads / n_kv_heads).
int launch_rope_kv(cudaStream_t st, int dtype, void *qkv, const int32_t *pos, const float *table,
                   void *kcache, void *vcache, int32_t *kv_pos, const int32_t *kv_row, int n,
                   int n_heads, int head_dim, int max_pos, DevStatus *status, int n_kv_heads = 0);
// scratch (gemm_scratch_bytes() bytes, zeroed once, private to the stream) lets the tensor-core kernels
// split the last partial wave of tiles along K; without it they run a plain tile loop.
size_t gemm_scratch_bytes();
// force_kernel (cross-checks): 0 = chosen by shape, 1 = one CTA per tile, 2 = CTA pairs.
// b_const: the caller guarantees that B (the weights) is not written by earlier work still in flight on
// the stream; only then may the weight-streaming kernel (M <= 4) start fetching B while the kernel before
// it drains.
// res_rows (device int32[M], optional, bf16 tensor-core path with R only): the addend of output row r is
// R[res_rows[r]] instead of R[r]; R and C must then be different buffers.
int launch_gemm(cudaStream_t st, int dtype, const void *A, const void *B, const void *R, void *C,
                int M, int N, int K, DevStatus *status, void *scratch = nullptr, size_t scratch_bytes = 0,
                int force_kernel = 0, bool b_const = false, const int32_t *res_rows = nullptr);
int launch_gemm_swiglu(cudaStream_t st, int dtype, const void *A, const void *Bg, const void *Bu,
                       void *C, int M, int F, int K, DevStatus *status, void *scratch = nullptr,
                       size_t scratch_bytes = 0, int force_kernel = 0, bool b_const = false);
// QKV projection with the rotary embedding and the K/V cache write in its epilogue (bf16,
// head_dim 128, d_model a multiple of 256): qkv [M, 3d] receives the rotated q (its k and v thirds
// are left untouched), rotated k and v go to cache rows kv_row[r] (or r) with their position tag.
bool gemm_qkv_rope_eligible(int dtype, int d_model, int head_dim, int d_kv = 0);
bool gemm_res_rows_supported(int dtype, int M, int K);
int launch_gemm_qkv_rope(cudaStream_t st, const void *h, const void *w_qkv, void *qkv, const int32_t *pos,
                         const float *table, void *kcache, void *vcache, int32_t *kv_pos,
                         const int32_t *kv_row, int M, int d_model, int max_pos, DevStatus *status,
                         void *scratch = nullptr, size_t scratch_bytes = 0, int d_kv = 0, int kv_rows = 0);
// Weight-streaming kernel for M <= 4 rows (decode); same results as the tensor-core GEMM.  With gain the
// rows of A are RMS-normalised on the way in; with c_f32 the output is fp32 (LM head).
bool gemv_small_m_eligible(int dtype, int M, int K);
// b_const: B is not being written by earlier work on the stream, so the launch may be a programmatic
// dependent whose first weight loads are issued before the preceding kernel has completed.
int launch_gemv_small_m(cudaStream_t st, const void *A, const void *B0, const void *B1, const void *R,
                        void *C, int M, int N, int K, int swiglu, const void *gain = nullptr,
                        float eps = 0.f, int c_f32 = 0, bool b_const = false);
int launch_gemv_qkv_rope(cudaStream_t st, const void *x, const void *w_qkv, void *qkv, const void *gain, float eps,
                         const int32_t *pos, const float *table, void *kcache, void *vcache, int32_t *kv_pos,
                         const int32_t *kv_row, int M, int d_model, int max_pos, DevStatus *status, int d_kv = 0);
int launch_gemm_simt(cudaStream_t st, int dtype, const void *A, const void *B0, const void *B1,
                     const void *R, void *C, int M, int N, int K, int swiglu);
// Attention over packed sequences. Sequence s: query rows [cu_q[s], cu_q[s+1]) of q, key rows
// kv_base[s] + j of k/v (kv_base NULL: same rows as q). Query row i sees keys j <= i (prefill).
int launch_attention(cudaStream_t st, int dtype, const void *q, int ldq, const void *k,
                     const void *v, int ldkv, void *o, const int32_t *cu_q, const int32_t *kv_base,
                     int n_seqs, int max_len, int n_total, int n_heads, int head_dim, int n_kv_heads = 0);
// Query heads per key/value head (1 without grouping); 0 if n_kv_heads does not divide n_heads.
inline int kv_group_of(int n_heads, int n_kv_heads) {
  if (n_kv_heads <= 0) return 1;
  return n_heads % n_kv_heads ? 0 : n_heads / n_kv_heads;
}
// General form (decode): sequence s has query rows [cu_q[s], cu_q[s+1]) and a key LIST
// kv_idx[cu_kv[s] .. cu_kv[s+1]) of cache rows in ascending position order; query row r sees the
// first q_kvlen[r] entries of its sequence's list.
int launch_attention_ex(cudaStream_t st, int dtype, const void *q, int ldq, const void *k,
                        const void *v, int ldkv, void *o, const int32_t *cu_q, const int32_t *kv_base,
                        const int32_t *cu_kv, const int32_t *kv_idx, const int32_t *q_kvlen, int n_seqs,
                        int max_len, int n_total, int n_heads, int head_dim, int n_kv_heads = 0);
// Prefill attention, bf16 / head_dim 128, on tcgen05 (see attention_tc.cu).  Sequences either come
// from device arrays (cu_q, kv_base) or one sequence is given by scalars; q_rows / kv_rows bound
// the tensor maps (reads beyond them give zeros).
int launch_attention_tc(cudaStream_t st, const void *q, int ldq, long long q_rows, const void *k,
                        const void *v, int ldkv, long long kv_rows, void *o, int n_heads,
                        const int32_t *cu_q, const int32_t *kv_base, int n_seqs, int max_len, int q_start,
                        int n, int kv_start, DevStatus *status, float *score_scratch = nullptr,
                        int max_tiles = 0, int n_seqs_total = 0, int seq_id = 0, int n_kv_heads = 0);
// With score_scratch (attn_score_scratch_floats floats) the attention kernel also leaves the last
// row's softmax numerators there; launch_score_from_attention turns them into the Eq. 1 scores, for
// n_layers consecutive layers over the same rows in one launch (layer y: by-product at scratch +
// y * scratch_stride, scores to scores + y * scores_stride).
// max_tiles = ceil(longest sequence / 64), the same value in both calls.
size_t attn_score_scratch_floats(int n_seqs, int n_heads, int max_tiles);
int launch_score_from_attention(cudaStream_t st, const float *scratch, size_t scratch_stride, int n_layers,
                                const int32_t *cu_q, int n_seqs, int n_total, int n_heads, int max_tiles,
                                float *scores, size_t scores_stride);
// True when the tensor-core prefill attention applies.
bool attention_tc_eligible(int dtype, int head_dim, int ldq, int ldkv);
size_t score_scratch_floats(int n_seqs, int n_total, int n_heads);
int launch_score(cudaStream_t st, int dtype, const void *q, int ldq, const void *k, int ldkv,
                 const int32_t *cu_q, const int32_t *kv_base, int n_seqs, int n_total, int max_len,
                 int n_heads, int head_dim, float *scratch, float *scores, int n_kv_heads = 0);
// General form (decode): sequence s scores the key LIST key_rows[cu_q[s] .. cu_q[s+1]) (cache rows)
// with the query in row q_rows[s].
int launch_score_mean(cudaStream_t st, const float *logits, const float *stats, const int32_t *cu_q,
                      int n_seqs, int n_total, int n_heads, float *scores, int n_layers = 1,
                      size_t layer_stride = 0, size_t scores_stride = 0);
// Split-key attention for one to eight query rows over key lists (decode); leaves the score row's
// logits and softmax statistics for launch_score_mean.
bool attention_decode_eligible(int dtype, int head_dim, int n_rows, int max_ctx);
size_t attention_decode_scratch_floats(int n_rows, int n_heads, int max_ctx);
int launch_attention_decode(cudaStream_t st, const void *q, int ldq, const void *k, const void *v,
                            int ldkv, void *o, int ldo, const int32_t *cu_x, const int32_t *cu_ctx,
                            const int32_t *ctx_rows, const int32_t *q_kvlen, const int32_t *score_row,
                            int n_seqs, int n_rows, int n_ctx_total, int max_ctx, int n_heads,
                            float *part, float *logits, float *stats, int n_kv_heads = 0);
int launch_attention_combine(cudaStream_t st, const float *part_o, const float *part_ml, int n_splits,
                             const int32_t *cu_x, const int32_t *score_row, int n_seqs, int n_rows, int n_heads,
                             void *o, int ldo, float *stats);
// Key-list attention for many query rows with the key tiles cut into slices (see attention.cu).
bool attention_list_split_eligible(int dtype, int head_dim);
int attention_list_splits(int n_seqs, int max_rows, int n_heads, int max_ctx);
int launch_attention_list_split(cudaStream_t st, const void *q, int ldq, const void *k, const void *v, int ldkv,
                                void *o, const int32_t *cu_q, const int32_t *cu_kv, const int32_t *kv_idx,
                                const int32_t *q_kvlen, const int32_t *score_row, int n_seqs, int max_rows,
                                int n_total, int n_heads, int n_splits, float *part, float *stats,
                                int n_kv_heads = 0);
int launch_score_ex(cudaStream_t st, int dtype, const void *q, int ldq, const void *k, int ldkv,
                    const int32_t *cu_q, const int32_t *kv_base, const int32_t *key_rows,
                    const int32_t *q_rows, int n_seqs, int n_total, int max_len, int n_heads,
                    int head_dim, float *scratch, float *scores, int n_kv_heads = 0);
int launch_select_threshold(cudaStream_t st, const float *scores, const int32_t *cu_in, int n_seqs,
                            uint32_t prune_bp, int32_t *keep_idx, int32_t *drop_idx, int32_t *counts);
// counts[s] = rows of sequence s whose score is not smaller than its (cu_keep[s+1] - cu_keep[s])-th largest
// score, the last row counting as the largest: the kept count of the threshold reading (ties all kept).
int launch_select_tie_count(cudaStream_t st, const float *scores, const int32_t *cu_in, const int32_t *cu_keep,
                            int n_seqs, int32_t *counts, DevStatus *status);
// With pos_in (position of every input row) the kernel also writes the kept rows' positions to pos_keep
// (packed like keep_idx) and the dropped rows' positions to aux_pos[aux_dst[j]] (j = slot in drop_idx).
int launch_select(cudaStream_t st, const float *scores, const int32_t *cu_in,
                  const int32_t *cu_keep, int n_seqs, int32_t *keep_idx, int32_t *drop_idx,
                  DevStatus *status, const int32_t *pos_in = nullptr, int32_t *pos_keep = nullptr,
                  const int32_t *aux_dst = nullptr, int32_t *aux_pos = nullptr);
// scores[r] = 2 if pos[r] is in the ascending list forced[0..n_forced), else 0 (rows r0..r0+n)
int launch_forced_scores(cudaStream_t st, const int32_t *pos, int r0, int n, const int32_t *forced,
                         int n_forced, float *scores);
int launch_gather_rows(cudaStream_t st, const void *src, const int32_t *idx, void *dst, int n,
                       int row_bytes, int src_rows, DevStatus *status);
int launch_gather_i32(cudaStream_t st, const int32_t *src, const int32_t *idx, int32_t *dst, int n);
int launch_lm_head(cudaStream_t st, int dtype, const void *h, const void *w, float *logits,
                   int n_rows, int d, int vocab, bool w_const = false);
int launch_argmax(cudaStream_t st, const float *logits, int32_t *out, int n_rows, int vocab);
int launch_fill_i32(cudaStream_t st, int32_t *p, int32_t v, size_t n);
int launch_iota_pos(cudaStream_t st, int32_t *pos, const int32_t *cu, int n_seqs, int n_total);

}  // namespace lazy
