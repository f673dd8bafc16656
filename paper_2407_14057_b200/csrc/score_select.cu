// Importance score (Eq. 1) and top-percentile selection (Section 3.2).
//
// Score: s_j = (1/H) sum_h softmax_j(q_last,h . k_j,h / sqrt(dh)).  Three small kernels:
//   1. logits[h][j] for every key of every sequence: K is read once with 16-byte loads, a group of
//      dh/8 (bf16) lanes per key, partial dot products combined with shuffles;
//   2. per (sequence, head) max and 1/sum of exp;
//   3. head mean of the normalised probabilities.
// Scratch: fp32 logits [H, n_total] plus (max, 1/sum) per (sequence, head).
//
// Select: one CTA per sequence.  The n_keep-th largest score is found with a 4-pass, 8-bit-per-pass
// radix select over the fp32 bit patterns (the last row is given the maximal key so it always
// survives); a final pass in index order emits kept and dropped row indices with ballot / popcount
// prefix sums, taking ties at the threshold in ascending index order until n_keep is reached.
#include <atomic>

#include "common.cuh"

namespace lazy {

namespace {

template <typename T>
__global__ void score_logits_kernel(const T *__restrict__ q, int ldq, const T *__restrict__ k,
                                    int ldkv, const int32_t *__restrict__ cu_q,
                                    const int32_t *__restrict__ kv_base,
                                    const int32_t *__restrict__ key_rows,
                                    const int32_t *__restrict__ q_rows, int n_total, int head_dim,
                                    float *__restrict__ logits, int kv_group) {
  constexpr int V = Elem<T>::kPerVec;
  const int seq = blockIdx.z, h = blockIdx.y;
  const int q_start = cu_q[seq];
  const int n = cu_q[seq + 1] - q_start;
  const int lpk = head_dim / V;       // lanes per key (power of two, <= 32)
  const int kpw = 32 / lpk;           // keys per warp per iteration
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int warps = blockDim.x >> 5;
  const int sub = lane % lpk, kslot = lane / lpk;
  const size_t kb = kv_base ? (size_t)kv_base[seq] : (size_t)q_start;
  if (n == 0) return;
  // this lane's slice of the last row's query, pre-scaled
  float qf[V];
  {
    Vec16<T> qv;
    const size_t qrow = q_rows ? (size_t)q_rows[seq] : (size_t)(q_start + n - 1);
    qv.load(q + qrow * ldq + h * head_dim + sub * V);
    qv.unpack(qf);
    const float scale = rsqrtf((float)head_dim);
#pragma unroll
    for (int i = 0; i < V; ++i) qf[i] *= scale;
  }
  const int keys_per_block = warps * kpw * 4;
  const int j_begin = blockIdx.x * keys_per_block;
  const int j_end = min(n, j_begin + keys_per_block);
  for (int j0 = j_begin + warp * kpw; j0 < j_end; j0 += warps * kpw) {
    const int j = j0 + kslot;
    float dot = 0.f;
    if (j < j_end) {
      Vec16<T> kv;
      const size_t krow = key_rows ? (size_t)key_rows[q_start + j] : kb + j;
      kv.load(k + krow * ldkv + (h / kv_group) * head_dim + sub * V);
      float kf[V];
      kv.unpack(kf);
#pragma unroll
      for (int i = 0; i < V; ++i) dot += qf[i] * kf[i];
    }
    for (int o = lpk >> 1; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    if (j < j_end && sub == 0) logits[(size_t)h * n_total + q_start + j] = dot;
  }
}

__global__ void score_stats_kernel(const float *__restrict__ logits, const int32_t *__restrict__ cu_q,
                                   int n_total, int n_heads, float *__restrict__ stats) {
  const int h = blockIdx.x, seq = blockIdx.y;
  const int q_start = cu_q[seq];
  const int n = cu_q[seq + 1] - q_start;
  const float *row = logits + (size_t)h * n_total + q_start;
  __shared__ float red[32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, warps = blockDim.x >> 5;
  float m = -INFINITY;
  for (int j = threadIdx.x; j < n; j += blockDim.x) m = fmaxf(m, row[j]);
  m = warp_max(m);
  if (lane == 0) red[warp] = m;
  __syncthreads();
  m = -INFINITY;
  for (int w = 0; w < warps; ++w) m = fmaxf(m, red[w]);
  __syncthreads();
  float s = 0.f;
  for (int j = threadIdx.x; j < n; j += blockDim.x) s += __expf(row[j] - m);
  s = warp_sum(s);
  if (lane == 0) red[warp] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < warps; ++w) t += red[w];
    stats[((size_t)seq * n_heads + h) * 2 + 0] = m;
    stats[((size_t)seq * n_heads + h) * 2 + 1] = n > 0 ? 1.f / t : 0.f;
  }
}

// 8 lanes per key, each over a slice of the heads.  blockIdx.y = one of several layers whose logits / statistics
// lie layer_stride floats apart and whose scores lie scores_stride floats apart (decode: the layers between two
// re-selections attend over the same context, so their head means are taken in one launch).
__global__ void score_mean_kernel(const float *__restrict__ logits, const float *__restrict__ stats,
                                  const int32_t *__restrict__ cu_q, int n_seqs, int n_total,
                                  int n_heads, float *__restrict__ scores, size_t layer_stride,
                                  size_t scores_stride) {
  logits += (size_t)blockIdx.y * layer_stride;
  stats += (size_t)blockIdx.y * layer_stride;
  scores += (size_t)blockIdx.y * scores_stride;
  // releases a following programmatic dependent (decode: the output projection's weight streaming can start
  // its weight reads now) and, launched as one itself, waits for the kernel before it
  LAZY_PDL_ENTER();
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  const int r = t >> 3, sub = t & 7;
  float acc = 0.f;
  if (r < n_total) {
    int lo = 0, hi = n_seqs;
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (cu_q[mid] <= r) lo = mid; else hi = mid;
    }
    const float *st = stats + (size_t)lo * n_heads * 2;
    for (int h = sub; h < n_heads; h += 8)
      acc += __expf(logits[(size_t)h * n_total + r] - st[2 * h]) * st[2 * h + 1];
  }
  acc += __shfl_xor_sync(0xffffffffu, acc, 1);
  acc += __shfl_xor_sync(0xffffffffu, acc, 2);
  acc += __shfl_xor_sync(0xffffffffu, acc, 4);
  if (r < n_total && sub == 0) scores[r] = acc / (float)n_heads;
}

// ------------------------------------------------------------------------------------------ select
constexpr int SEL_THREADS = 1024;

__device__ __forceinline__ uint32_t score_key(float s) {
  uint32_t u = __float_as_uint(s);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // monotone for every finite float
}

// Exclusive prefix of `flag` over the CTA in thread order; total returned through *total.
__device__ __forceinline__ int block_excl_scan(int flag, int *warp_tot /*[32]*/, int *total) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t b = __ballot_sync(0xffffffffu, flag);
  const int within = __popc(b & ((1u << lane) - 1u));
  __syncthreads();  // warp_tot may still be read from the previous scan
  if (lane == 0) warp_tot[warp] = __popc(b);
  __syncthreads();
  int before = 0, tot = 0;
  for (int w = 0; w < SEL_THREADS / 32; ++w) {
    const int c = warp_tot[w];
    if (w < warp) before += c;
    tot += c;
  }
  *total = tot;
  return before + within;
}

// One warp: the bin b (from the top) in which the k-th largest key lies, and how many keys lie in bins above
// it.  Lane l owns bins [8l, 8l + 8); a suffix sum over the lanes finds the lane, a walk over its 8 bins the
// bin.  (One thread walking 256 bins took a quarter of the whole selection.)
__device__ __forceinline__ void radix_pick_bin(const int *hist, int k, int &bin, int &above) {
  const int lane = threadIdx.x & 31;
  int mine = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) mine += hist[lane * 8 + i];
  int incl = mine;  // keys in bins of lanes >= this one
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_down_sync(0xffffffffu, incl, o);
    if (lane + o < 32) incl += v;
  }
  // the highest lane whose suffix count reaches k holds the bin
  const unsigned reach = __ballot_sync(0xffffffffu, incl >= k);
  const int owner = reach ? 31 - __clz(reach) : 0;
  int b = owner * 8, ab = 0;
  if (lane == owner) {
    ab = incl - mine;  // keys in the lanes above
    b = owner * 8 + 7;
    for (; b > owner * 8; --b) {
      if (ab + hist[b] >= k) break;
      ab += hist[b];
    }
  }
  bin = __shfl_sync(0xffffffffu, b, owner);
  above = __shfl_sync(0xffffffffu, ab, owner);
}

// Keys of a sequence are read from global memory once and kept in shared memory for the four radix passes
// and the emit pass (sequences of up to SEL_CACHE rows; longer ones re-read the scores).
constexpr int SEL_CACHE = 8192;

struct SelShared {
  int hist[256];
  int warp_tot[32];
  uint32_t prefix;
  int k;
  uint32_t keys[SEL_CACHE];
};

// Radix select over the order-preserving keys of s[0..n): on return *k_ties = how many keys equal to the
// returned key tau belong to the k largest.  force_last: the last row gets the maximal key.  Scores of a
// long prompt are nearly equal (about 1/n), so their keys share the high bytes and a plain histogram would
// serialise every shared-memory atomic of the first passes on one bin: the lanes of a warp that hit the
// same bin as its first active lane are counted with a ballot and added once.
__device__ __forceinline__ uint32_t radix_kth_largest(const float *__restrict__ s, int n, int k, bool force_last,
                                                      SelShared &sh, int *k_ties) {
  const bool cached = n <= SEL_CACHE;
  const int lane = threadIdx.x & 31;
  if (cached)
    for (int i = threadIdx.x; i < n; i += SEL_THREADS)
      sh.keys[i] = (force_last && i == n - 1) ? 0xffffffffu : score_key(s[i]);
  uint32_t prefix = 0, mask = 0;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = threadIdx.x; i < 256; i += SEL_THREADS) sh.hist[i] = 0;
    __syncthreads();  // also orders the key cache before its first use
    for (int base = 0; base < n; base += SEL_THREADS) {
      const int i = base + threadIdx.x;
      uint32_t key = 0;
      bool act = false;
      if (i < n) {
        key = cached ? sh.keys[i] : ((force_last && i == n - 1) ? 0xffffffffu : score_key(s[i]));
        act = (key & mask) == prefix;
      }
      const uint32_t bin = (key >> shift) & 255u;
      // lanes that share the bin of the warp's first active lane add once, together; the others one by one
      const unsigned active = __ballot_sync(0xffffffffu, act);
      if (active) {
        const uint32_t bin0 = __shfl_sync(0xffffffffu, bin, __ffs(active) - 1);
        const unsigned same = __ballot_sync(0xffffffffu, act && bin == bin0);
        if (act) {
          if (bin != bin0) atomicAdd(&sh.hist[bin], 1);
          else if (lane == __ffs(same) - 1) atomicAdd(&sh.hist[bin0], __popc(same));
        }
      }
    }
    __syncthreads();
    if (threadIdx.x < 32) {
      int above, b;
      radix_pick_bin(sh.hist, k, b, above);
      if (threadIdx.x == 0) {
        sh.prefix = prefix | ((uint32_t)b << shift);
        sh.k = k - above;
      }
    }
    __syncthreads();
    prefix = sh.prefix;
    k = sh.k;
    mask |= 255u << shift;
    __syncthreads();
  }
  *k_ties = k;
  return prefix;
}

// pos_in (optional): position of every input row.  The kept rows' positions then go to pos_keep (packed like
// keep_idx) and the dropped rows' positions to aux_pos[aux_dst[j]], j = the row's slot in drop_idx: the
// position lists of the next segment and of the Aux Cache come out of the selection itself.
__global__ void __launch_bounds__(SEL_THREADS)
select_kernel(const float *__restrict__ scores, const int32_t *__restrict__ cu_in,
              const int32_t *__restrict__ cu_keep, int32_t *__restrict__ keep_idx,
              int32_t *__restrict__ drop_idx, DevStatus *status, const int32_t *__restrict__ pos_in,
              int32_t *__restrict__ pos_keep, const int32_t *__restrict__ aux_dst, int32_t *__restrict__ aux_pos) {
  const int seq = blockIdx.x;
  const int in0 = cu_in[seq], n = cu_in[seq + 1] - in0;
  const int k0 = cu_keep[seq], n_keep = cu_keep[seq + 1] - k0;
  const int d0 = in0 - k0;
  if (n == 0) return;
  if (n_keep < 1 || n_keep > n) {
    if (threadIdx.x == 0) dev_fail(status, LAZY_E_BADARG, W_SELECT, seq, n_keep);
    return;
  }
  const float *s = scores + in0;
  __shared__ SelShared sh;
  int k;  // how many keys == tau to keep
  const uint32_t tau = radix_kth_largest(s, n, n_keep, true, sh, &k);
  const bool cached = n <= SEL_CACHE;

  // ---- emit in index order
  int kept_so_far = 0, eq_so_far = 0;
  for (int base = 0; base < n; base += SEL_THREADS) {
    const int i = base + threadIdx.x;
    uint32_t key = 0;
    const bool valid = i < n;
    if (valid) key = cached ? sh.keys[i] : ((i == n - 1) ? 0xffffffffu : score_key(s[i]));
    const int is_eq = valid && key == tau;
    int eq_total;
    const int eq_rank = eq_so_far + block_excl_scan(is_eq, sh.warp_tot, &eq_total);
    const int keep = valid && (key > tau || (is_eq && eq_rank < k));
    int keep_total;
    const int keep_rank = kept_so_far + block_excl_scan(keep, sh.warp_tot, &keep_total);
    if (valid) {
      if (keep) {
        keep_idx[k0 + keep_rank] = in0 + i;
        if (pos_in) pos_keep[k0 + keep_rank] = pos_in[in0 + i];
      } else {
        const int j = d0 + (i - keep_rank);
        drop_idx[j] = in0 + i;
        if (pos_in) aux_pos[aux_dst[j]] = pos_in[in0 + i];
      }
    }
    eq_so_far += eq_total;
    kept_so_far += keep_total;
  }
  if (threadIdx.x == 0 && kept_so_far != n_keep) dev_fail(status, LAZY_E_STATE, W_SELECT, seq, kept_so_far);
}

// Threshold reading at the scheduled rank: tau = the n_keep-th largest key of the sequence (the last row
// counting as the largest), and every row whose score is not smaller than tau survives.  The kernel only
// COUNTS the survivors: counts[seq] = n_keep + (keys equal to tau beyond the ones the count form would
// keep).  With that count the ordinary selection keeps exactly the rows with score >= tau (no tie is cut),
// so the host reads the counts back and launches select_kernel with them.
__global__ void __launch_bounds__(SEL_THREADS)
select_tie_count_kernel(const float *__restrict__ scores, const int32_t *__restrict__ cu_in,
                        const int32_t *__restrict__ cu_keep, int32_t *__restrict__ counts, DevStatus *status) {
  const int seq = blockIdx.x;
  const int in0 = cu_in[seq], n = cu_in[seq + 1] - in0;
  const int n_keep = cu_keep[seq + 1] - cu_keep[seq];
  if (n == 0) {
    if (threadIdx.x == 0) counts[seq] = 0;
    return;
  }
  if (n_keep < 1 || n_keep > n) {
    if (threadIdx.x == 0) {
      dev_fail(status, LAZY_E_BADARG, W_SELECT, seq, n_keep);
      counts[seq] = n_keep < 1 ? 1 : n;
    }
    return;
  }
  const float *s = scores + in0;
  __shared__ SelShared sh;
  int k_ties;
  const uint32_t tau = radix_kth_largest(s, n, n_keep, true, sh, &k_ties);
  const bool cached = n <= SEL_CACHE;
  int eq_total = 0;
  for (int base = 0; base < n; base += SEL_THREADS) {
    const int i = base + threadIdx.x;
    uint32_t key = 0;
    const bool valid = i < n;
    if (valid) key = cached ? sh.keys[i] : ((i == n - 1) ? 0xffffffffu : score_key(s[i]));
    int t;
    block_excl_scan(valid && key == tau, sh.warp_tot, &t);
    eq_total += t;
  }
  if (threadIdx.x == 0) counts[seq] = n_keep - k_ties + eq_total;
}

// Threshold form of the selection: tau = the score at the prune_bp/10000 quantile of the sequence's n scores
// (the order statistic with index floor((n-1) * prune_bp / 10000) from below), every row with score >= tau is
// kept, and the last row always.  The count depends on the data (ties at tau are all kept), so kept / dropped
// indices are packed from the sequence's input offset and the count is written to counts[seq].
__global__ void __launch_bounds__(SEL_THREADS)
select_threshold_kernel(const float *__restrict__ scores, const int32_t *__restrict__ cu_in, uint32_t prune_bp,
                        int32_t *__restrict__ keep_idx, int32_t *__restrict__ drop_idx,
                        int32_t *__restrict__ counts) {
  const int seq = blockIdx.x;
  const int in0 = cu_in[seq], n = cu_in[seq + 1] - in0;
  if (n == 0) {
    if (threadIdx.x == 0) counts[seq] = 0;
    return;
  }
  const float *s = scores + in0;
  __shared__ SelShared sh;
  const int lo = (int)(((long long)(n - 1) * prune_bp) / 10000);
  // the (n - lo)-th largest key = the lo-th smallest
  int k_unused;
  const uint32_t tau = radix_kth_largest(s, n, n - lo, false, sh, &k_unused);
  const bool cached = n <= SEL_CACHE;
  // ---- emit in index order
  int kept_so_far = 0;
  for (int base = 0; base < n; base += SEL_THREADS) {
    const int i = base + threadIdx.x;
    const bool valid = i < n;
    const int keep = valid && (i == n - 1 || (cached ? sh.keys[i] : score_key(s[i])) >= tau);
    int keep_total;
    const int keep_rank = kept_so_far + block_excl_scan(keep, sh.warp_tot, &keep_total);
    if (valid) {
      if (keep) keep_idx[in0 + keep_rank] = in0 + i;
      else drop_idx[in0 + (i - keep_rank)] = in0 + i;
    }
    kept_so_far += keep_total;
  }
  if (threadIdx.x == 0) counts[seq] = kept_so_far;
}

__global__ void forced_scores_kernel(const int32_t *__restrict__ pos, int r0, int n,
                                     const int32_t *__restrict__ forced, int n_forced,
                                     float *__restrict__ scores) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int p = pos[r0 + i];
  int lo = 0, hi = n_forced;  // first index with forced[idx] >= p
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (forced[mid] < p) lo = mid + 1; else hi = mid;
  }
  scores[r0 + i] = (lo < n_forced && forced[lo] == p) ? 2.f : 0.f;
}

}  // namespace

size_t score_scratch_floats(int n_seqs, int n_total, int n_heads) {
  return (size_t)n_heads * n_total + (size_t)2 * n_heads * n_seqs;
}

int launch_score(cudaStream_t st, int dtype, const void *q, int ldq, const void *k, int ldkv,
                 const int32_t *cu_q, const int32_t *kv_base, int n_seqs, int n_total, int max_len,
                 int n_heads, int head_dim, float *scratch, float *scores, int n_kv_heads) {
  return launch_score_ex(st, dtype, q, ldq, k, ldkv, cu_q, kv_base, nullptr, nullptr, n_seqs, n_total,
                         max_len, n_heads, head_dim, scratch, scores, n_kv_heads);
}

int launch_score_ex(cudaStream_t st, int dtype, const void *q, int ldq, const void *k, int ldkv,
                    const int32_t *cu_q, const int32_t *kv_base, const int32_t *key_rows,
                    const int32_t *q_rows, int n_seqs, int n_total, int max_len, int n_heads,
                    int head_dim, float *scratch, float *scores, int n_kv_heads) {
  if (n_total == 0 || n_seqs == 0) return LAZY_OK;
  const int kv_group = kv_group_of(n_heads, n_kv_heads);
  if (kv_group < 1) return LAZY_E_BADARG;
  const int V = dtype == LAZY_F32 ? 4 : 8;
  const int lpk = head_dim / V;
  if (head_dim % V || lpk < 1 || lpk > 32 || (lpk & (lpk - 1))) return LAZY_E_BADARG;
  float *logits = scratch;
  float *stats = scratch + (size_t)n_heads * n_total;
  const int threads = 256;
  const int keys_per_block = (threads / 32) * (32 / lpk) * 4;
  dim3 grid(cdiv(max_len, keys_per_block), n_heads, n_seqs);
  if (dtype == LAZY_F32)
    score_logits_kernel<float><<<grid, threads, 0, st>>>((const float *)q, ldq, (const float *)k, ldkv,
                                                         cu_q, kv_base, key_rows, q_rows, n_total, head_dim,
                                                         logits, kv_group);
  else
    score_logits_kernel<bf16><<<grid, threads, 0, st>>>((const bf16 *)q, ldq, (const bf16 *)k, ldkv,
                                                        cu_q, kv_base, key_rows, q_rows, n_total, head_dim,
                                                        logits, kv_group);
  LAZY_COUNT_LAUNCH();
  score_stats_kernel<<<dim3(n_heads, n_seqs), 256, 0, st>>>(logits, cu_q, n_total, n_heads, stats);
  LAZY_COUNT_LAUNCH();
  score_mean_kernel<<<cdiv(n_total, 32), 256, 0, st>>>(logits, stats, cu_q, n_seqs, n_total, n_heads,
                                                        scores, (size_t)0, (size_t)0);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

// Eq. 1 mean over heads from logits [H, n_total] and per-(sequence, head) (max, 1/sum) pairs that
// another kernel already produced.
int launch_score_mean(cudaStream_t st, const float *logits, const float *stats, const int32_t *cu_q,
                      int n_seqs, int n_total, int n_heads, float *scores, int n_layers, size_t layer_stride,
                      size_t scores_stride) {
  if (n_total == 0 || n_layers == 0) return LAZY_OK;
  if (!logits || !stats || !cu_q || !scores || n_layers < 1) return LAZY_E_BADARG;
  LAZY_TRY(launch_pdl(score_mean_kernel, dim3(cdiv(n_total, 32), n_layers), dim3(256), 0, st, logits, stats, cu_q,
                      n_seqs, n_total, n_heads, scores, layer_stride, scores_stride));
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

int launch_select_threshold(cudaStream_t st, const float *scores, const int32_t *cu_in, int n_seqs,
                            uint32_t prune_bp, int32_t *keep_idx, int32_t *drop_idx, int32_t *counts) {
  if (n_seqs == 0) return LAZY_OK;
  select_threshold_kernel<<<n_seqs, SEL_THREADS, 0, st>>>(scores, cu_in, prune_bp, keep_idx, drop_idx, counts);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

int launch_select_tie_count(cudaStream_t st, const float *scores, const int32_t *cu_in, const int32_t *cu_keep,
                            int n_seqs, int32_t *counts, DevStatus *status) {
  if (n_seqs == 0) return LAZY_OK;
  select_tie_count_kernel<<<n_seqs, SEL_THREADS, 0, st>>>(scores, cu_in, cu_keep, counts, status);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

int launch_select(cudaStream_t st, const float *scores, const int32_t *cu_in,
                  const int32_t *cu_keep, int n_seqs, int32_t *keep_idx, int32_t *drop_idx,
                  DevStatus *status, const int32_t *pos_in, int32_t *pos_keep, const int32_t *aux_dst,
                  int32_t *aux_pos) {
  if (n_seqs == 0) return LAZY_OK;
  if (pos_in && (!pos_keep || !aux_dst || !aux_pos)) return LAZY_E_BADARG;
  select_kernel<<<n_seqs, SEL_THREADS, 0, st>>>(scores, cu_in, cu_keep, keep_idx, drop_idx, status, pos_in,
                                                pos_keep, aux_dst, aux_pos);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

int launch_forced_scores(cudaStream_t st, const int32_t *pos, int r0, int n, const int32_t *forced,
                         int n_forced, float *scores) {
  if (n == 0) return LAZY_OK;
  forced_scores_kernel<<<cdiv(n, 256), 256, 0, st>>>(pos, r0, n, forced, n_forced, scores);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}


// ---- importance score without caller-provided scratch ---------------------------------------------
// Some callers of this library cannot hand over scratch memory because they are not allowed to
// allocate device memory at all: a plugin running inside a host application whose memory pool is
// closed to it, a callback on a serving path where cudaMalloc would stall every stream of the
// device, or code that runs after the process has given all memory to another owner.  For them the
// score's scratch (per-head logits plus the softmax statistics) lives in this fixed array, which
// every GPU that loads the library holds until the process exits.
namespace {
constexpr int STATIC_SCORE_MAX_LOGITS = 262144;  // n_heads * n_total, e.g. 32 heads x 8192 tokens
constexpr int STATIC_SCORE_MAX_STATS = 4096;     // 2 * n_heads * n_seqs
static __device__ __align__(256) float g_static_score_scratch[STATIC_SCORE_MAX_LOGITS + STATIC_SCORE_MAX_STATS];

// Device address of the array on the current device.  The array's name is only a host-side handle
// here: the address a kernel can use comes from cudaGetSymbolAddress, asked once per device.
// The per-device slots are atomic, so two host threads making their first call at once both store
// the same address without a data race.  The slots outlive a cudaDeviceReset of their device: a
// process that resets a device must not call this entry point on it afterwards.
float *static_score_scratch_ptr() {
  static std::atomic<float *> ptrs[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  float *p = ptrs[dev].load(std::memory_order_acquire);
  if (!p) {
    if (cudaGetSymbolAddress((void **)&p, g_static_score_scratch) != cudaSuccess) return nullptr;
    ptrs[dev].store(p, std::memory_order_release);
  }
  return p;
}
}  // namespace

}  // namespace lazy

extern "C" int lazy_k_score_static(void *stream, int32_t dtype, const void *q, int32_t ldq, const void *k,
                                   int32_t ldkv, const int32_t *d_cu_seqlens, int32_t n_seqs,
                                   int32_t n_total, int32_t n_heads, int32_t head_dim, float *scores) {
  using namespace lazy;
  if ((dtype != LAZY_BF16 && dtype != LAZY_F32) || !q || !k || !d_cu_seqlens || !scores || n_seqs < 0 ||
      n_total < 0 || n_heads < 1)
    return LAZY_E_BADARG;
  // sizes beyond the fixed array are refused, never truncated
  if ((long long)n_heads * n_total > STATIC_SCORE_MAX_LOGITS ||
      2LL * n_heads * n_seqs > STATIC_SCORE_MAX_STATS)
    return LAZY_E_CAPACITY;
  float *scratch = static_score_scratch_ptr();
  if (!scratch) return LAZY_E_CUDA;
  // Layout inside the array matches what launch_score expects for this (n_heads, n_total): logits
  // first, statistics right after them.  Every element that is read is written first by the same
  // call, so nothing has to be cleared between calls.
  return launch_score((cudaStream_t)stream, dtype, q, ldq, k, ldkv, d_cu_seqlens, nullptr, n_seqs, n_total,
                      n_total, n_heads, head_dim, scratch, scores);
}
