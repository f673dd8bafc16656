// Attention for a handful of query rows over long key lists (decode: the new token, plus at most
// a few revived rows).  With one to eight query rows there is nothing for the tensor cores to chew
// on: the step is a read of the selected K and V rows, so the keys are split across many CTAs
// (64 keys each), every CTA produces a partial softmax (max, sum, unnormalised output) and a small
// second kernel merges the partials.  The row of the new token also leaves its logits and final
// softmax statistics behind, from which the Eq. 1 score is averaged without reading K again.
// bf16, head_dim 128.  Keys come through a list of cache rows (ascending positions); query row r
// sees the first q_kvlen[r] entries of its sequence's list.
#include "common.cuh"

namespace lazy {

namespace {

constexpr int DK_SPLIT = 64;    // keys per CTA
constexpr int DK_THREADS = 128; // 4 warps; thread t owns output column t
constexpr int DK_HD = 128;
static_assert(DK_SPLIT == 64 && DK_THREADS == 128 && DK_HD == 128, "the partial kernel maps 4 warps x 16 keys and 8 groups x 8 keys");
constexpr float LOG2E = 1.4426950408889634f, LN2 = 0.6931471805599453f;

__device__ __forceinline__ float ex2f_fast(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ int seq_of_row(const int32_t *cu, int n_seqs, int r) {
  int lo = 0, hi = n_seqs;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (cu[mid] <= r) lo = mid; else hi = mid;
  }
  return lo;
}

// grid (n_splits, H, M).  part_o [M, H, n_splits, 128] fp32, part_ml [M, H, n_splits, 2] (max in log2
// units, sum).  logits (score rows only): [H, n_ctx_total] natural-log units.
// Every load of a phase is issued before the first use, so one CTA keeps 8 x 16 bytes per thread in
// flight; 64 keys per CTA put a few thousand CTAs on the machine at a 4096-token context.
__global__ void __launch_bounds__(DK_THREADS)
attn_decode_partial_kernel(const bf16 *__restrict__ q, int ldq, const bf16 *__restrict__ k,
                           const bf16 *__restrict__ v, int ldkv, const int32_t *__restrict__ cu_x,
                           const int32_t *__restrict__ cu_ctx, const int32_t *__restrict__ ctx_rows,
                           const int32_t *__restrict__ q_kvlen, const int32_t *__restrict__ score_row,
                           int n_seqs, int n_ctx_total, float *__restrict__ part_o,
                           float *__restrict__ part_ml, float *__restrict__ logits, int kv_group) {
  __shared__ int32_t srow[DK_SPLIT];
  __shared__ float sl[DK_SPLIT];
  __shared__ float so[DK_THREADS / 16][DK_HD];
  LAZY_PDL_ENTER();
  const int split = blockIdx.x, h = blockIdx.y, r = blockIdx.z;
  const int n_splits = gridDim.x, H = gridDim.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int s = seq_of_row(cu_x, n_seqs, r);
  const int c0 = cu_ctx[s];
  const int vis = q_kvlen[r];
  const int k0 = split * DK_SPLIT;
  const int cnt = min(DK_SPLIT, vis - k0);
  const size_t pidx = ((size_t)r * H + h) * n_splits + split;
  if (cnt <= 0) {  // nothing visible in this split: an empty partial
    if (threadIdx.x == 0) {
      part_ml[pidx * 2] = -INFINITY;
      part_ml[pidx * 2 + 1] = 0.f;
    }
    return;
  }
  if (threadIdx.x < DK_SPLIT) {
    srow[threadIdx.x] = threadIdx.x < cnt ? ctx_rows[c0 + k0 + threadIdx.x] : -1;
    sl[threadIdx.x] = -INFINITY;
  }
  const int sub = lane & 15, half = lane >> 4;
  float qf[8];
  {
    Vec16<bf16> qv;
    qv.load(q + (size_t)r * ldq + h * DK_HD + sub * 8);
    qv.unpack(qf);
    const float sc = rsqrtf((float)DK_HD) * LOG2E;
#pragma unroll
    for (int i = 0; i < 8; ++i) qf[i] *= sc;
  }
  const bool is_score = score_row[s] == r;
  __syncthreads();
  // ---- logits: 16 lanes per key; warp w owns keys w*16 .. w*16+15, two per instruction
  {
    Vec16<bf16> kv[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int row = srow[warp * 16 + i * 2 + half];
      if (row >= 0) kv[i].load(k + (size_t)row * ldkv + (h / kv_group) * DK_HD + sub * 8);
      else kv[i].raw = make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float kf[8], dot = 0.f;
      kv[i].unpack(kf);
#pragma unroll
      for (int e = 0; e < 8; ++e) dot = fmaf(qf[e], kf[e], dot);
      dot += __shfl_xor_sync(0xffffffffu, dot, 1);
      dot += __shfl_xor_sync(0xffffffffu, dot, 2);
      dot += __shfl_xor_sync(0xffffffffu, dot, 4);
      dot += __shfl_xor_sync(0xffffffffu, dot, 8);
      const int j = warp * 16 + i * 2 + half;
      if (sub == 0 && j < cnt) {
        sl[j] = dot;
        if (is_score) logits[(size_t)h * n_ctx_total + c0 + k0 + j] = dot * LN2;
      }
    }
  }
  __syncthreads();
  // ---- partial softmax over the split (every warp computes the same max and sum)
  const float l0 = sl[lane], l1 = sl[lane + 32];
  const float m = warp_max(fmaxf(l0, l1));
  const float sum = warp_sum(ex2f_fast(l0 - m) + ex2f_fast(l1 - m));  // ex2(-inf) = 0 past the tail
  // ---- unnormalised output: group g (16 lanes) takes keys g*8 .. g*8+7, lane takes 8 columns
  const int g = threadIdx.x >> 4;
  float acc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) acc[e] = 0.f;
  {
    Vec16<bf16> vv[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int row = srow[g * 8 + i];
      if (row >= 0) vv[i].load(v + (size_t)row * ldkv + (h / kv_group) * DK_HD + sub * 8);
      else vv[i].raw = make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float p = ex2f_fast(sl[g * 8 + i] - m);
      float vf[8];
      vv[i].unpack(vf);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = fmaf(p, vf[e], acc[e]);
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) so[g][sub * 8 + e] = acc[e];
  __syncthreads();
  float o = 0.f;
#pragma unroll
  for (int gg = 0; gg < DK_THREADS / 16; ++gg) o += so[gg][threadIdx.x];
  part_o[pidx * DK_HD + threadIdx.x] = o;
  if (threadIdx.x == 0) {
    part_ml[pidx * 2] = m;
    part_ml[pidx * 2 + 1] = sum;
  }
}

// grid (H, M): merges the splits of one (row, head).  512 threads: thread (g, t) adds the splits i = g mod 4
// of output column t (four chains of loads in flight per column: with 32 CTAs on the whole GPU the kernel is
// a latency chain), then the four groups are summed through shared memory.  For a score row the final
// (max, 1/sum) pair goes to stats[(seq*H + h)*2], max in natural-log units.
constexpr int DK_MAX_SPLITS = 2048;  // 131072 keys
constexpr int DK_CGROUPS = 4;
constexpr int DK_CTHREADS = DK_CGROUPS * DK_HD;
__global__ void __launch_bounds__(DK_CTHREADS)
attn_decode_combine_kernel(const float *__restrict__ part_o, const float *__restrict__ part_ml,
                           int n_splits, const int32_t *__restrict__ cu_x,
                           const int32_t *__restrict__ score_row, int n_seqs, bf16 *__restrict__ o,
                           int ldo, float *__restrict__ stats) {
  __shared__ float sw[DK_MAX_SPLITS];  // weight of each split: 2^(m_i - m), 0 for an empty one
  __shared__ float red[DK_CTHREADS / 32];
  __shared__ float sacc[DK_CGROUPS][DK_HD];
  LAZY_PDL_ENTER();
  const int h = blockIdx.x, r = blockIdx.y, H = gridDim.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = threadIdx.x / DK_HD, t = threadIdx.x - g * DK_HD;
  const size_t base = ((size_t)r * H + h) * n_splits;
  const float2 *ml = reinterpret_cast<const float2 *>(part_ml) + base;
  float m = -INFINITY;
  for (int i = threadIdx.x; i < n_splits; i += DK_CTHREADS) m = fmaxf(m, ml[i].x);
  m = warp_max(m);
  if (lane == 0) red[warp] = m;
  __syncthreads();
  m = red[0];
#pragma unroll
  for (int w = 1; w < DK_CTHREADS / 32; ++w) m = fmaxf(m, red[w]);
  __syncthreads();
  float l = 0.f;
  for (int i = threadIdx.x; i < n_splits; i += DK_CTHREADS) {
    const float2 v = ml[i];
    const float w = v.y > 0.f ? ex2f_fast(v.x - m) : 0.f;
    sw[i] = w;
    l = fmaf(v.y, w, l);
  }
  l = warp_sum(l);
  if (lane == 0) red[warp] = l;
  __syncthreads();
  l = 0.f;
#pragma unroll
  for (int w = 0; w < DK_CTHREADS / 32; ++w) l += red[w];  // fixed order: the same in every thread
  const float *po = part_o + base * DK_HD + t;
  float acc0 = 0.f, acc1 = 0.f;
  int i = g;
  for (; i + DK_CGROUPS < n_splits; i += 2 * DK_CGROUPS) {  // an empty split never wrote its slot: do not touch it
    const float w0 = sw[i], w1 = sw[i + DK_CGROUPS];
    const float v0 = w0 > 0.f ? po[(size_t)i * DK_HD] : 0.f;
    const float v1 = w1 > 0.f ? po[(size_t)(i + DK_CGROUPS) * DK_HD] : 0.f;
    acc0 = fmaf(v0, w0, acc0);
    acc1 = fmaf(v1, w1, acc1);
  }
  if (i < n_splits) {
    const float w = sw[i];
    if (w > 0.f) acc0 = fmaf(po[(size_t)i * DK_HD], w, acc0);
  }
  sacc[g][t] = acc0 + acc1;
  __syncthreads();
  if (g == 0) {
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const float acc = (sacc[0][t] + sacc[1][t]) + (sacc[2][t] + sacc[3][t]);
    o[(size_t)r * ldo + h * DK_HD + t] = __float2bfloat16(acc * inv);
    if (t == 0) {
      const int s = seq_of_row(cu_x, n_seqs, r);
      if (score_row[s] == r) {
        stats[((size_t)s * H + h) * 2] = m * LN2;
        stats[((size_t)s * H + h) * 2 + 1] = inv;
      }
    }
  }
}

}  // namespace

// The merge step alone: partials [n_rows, n_heads, n_splits] x (128 fp32 | max in log2 units, sum).
int launch_attention_combine(cudaStream_t st, const float *part_o, const float *part_ml, int n_splits,
                             const int32_t *cu_x, const int32_t *score_row, int n_seqs, int n_rows, int n_heads,
                             void *o, int ldo, float *stats) {
  if (n_rows == 0) return LAZY_OK;
  if (n_splits < 1 || n_splits > DK_MAX_SPLITS) return LAZY_E_CAPACITY;
  attn_decode_combine_kernel<<<dim3(n_heads, n_rows), DK_CTHREADS, 0, st>>>(part_o, part_ml, n_splits, cu_x, score_row,
                                                                        n_seqs, (bf16 *)o, ldo, stats);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

bool attention_decode_eligible(int dtype, int head_dim, int n_rows, int max_ctx) {
  return dtype == LAZY_BF16 && head_dim == DK_HD && n_rows >= 1 && n_rows <= 8 &&
         max_ctx <= DK_MAX_SPLITS * DK_SPLIT;
}

size_t attention_decode_scratch_floats(int n_rows, int n_heads, int max_ctx) {
  const size_t n_splits = (size_t)cdiv(max_ctx > 0 ? max_ctx : 1, DK_SPLIT);
  return (size_t)n_rows * n_heads * n_splits * (DK_HD + 2);
}

// q/o: [n_rows, ld] bf16 with head h at columns h*128; k/v: cache rows addressed through ctx_rows.
// cu_x [n_seqs+1] query rows per sequence, cu_ctx [n_seqs+1] key-list offsets, q_kvlen [n_rows] visible
// keys per row, score_row [n_seqs] the row whose probabilities feed Eq. 1.  logits [H, n_ctx_total] and
// stats [n_seqs, H, 2] are outputs for launch_score_mean.  part: attention_decode_scratch_floats().
int launch_attention_decode(cudaStream_t st, const void *q, int ldq, const void *k, const void *v,
                            int ldkv, void *o, int ldo, const int32_t *cu_x, const int32_t *cu_ctx,
                            const int32_t *ctx_rows, const int32_t *q_kvlen, const int32_t *score_row,
                            int n_seqs, int n_rows, int n_ctx_total, int max_ctx, int n_heads,
                            float *part, float *logits, float *stats, int n_kv_heads) {
  if (n_rows == 0) return LAZY_OK;
  const int kv_group = kv_group_of(n_heads, n_kv_heads);
  if (kv_group < 1) return LAZY_E_BADARG;
  if (!q || !k || !v || !o || !cu_x || !cu_ctx || !ctx_rows || !q_kvlen || !score_row || !part ||
      !logits || !stats)
    return LAZY_E_BADARG;
  if (n_rows > 8 || n_seqs < 1 || n_heads < 1 || max_ctx < 1) return LAZY_E_BADARG;
  const int n_splits = cdiv(max_ctx, DK_SPLIT);
  if (n_splits > DK_MAX_SPLITS) return LAZY_E_CAPACITY;
  float *part_o = part;
  float *part_ml = part + (size_t)n_rows * n_heads * n_splits * DK_HD;
  LAZY_TRY(launch_pdl(attn_decode_partial_kernel, dim3(n_splits, n_heads, n_rows), dim3(DK_THREADS), 0, st,
                      (const bf16 *)q, ldq, (const bf16 *)k, (const bf16 *)v, ldkv, cu_x, cu_ctx, ctx_rows, q_kvlen,
                      score_row, n_seqs, n_ctx_total, part_o, part_ml, logits, kv_group));
  LAZY_COUNT_LAUNCH();
  LAZY_TRY(launch_pdl(attn_decode_combine_kernel, dim3(n_heads, n_rows), dim3(DK_CTHREADS), 0, st,
                      (const float *)part_o, (const float *)part_ml, n_splits, cu_x, score_row, n_seqs, (bf16 *)o,
                      ldo, stats));
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

}  // namespace lazy
