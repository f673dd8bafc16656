// Decode step with dynamic re-selection and revival from the Aux Cache (Section 3.2).
//
// Per sequence the step carries a context list T (positions, ascending) and a set X of rows "in
// flight" (the new token plus tokens revived earlier in the step).  At each layer the in-flight
// rows get q/k/v, append their K/V to the layer's cache, attend over T + the new token (keys are
// looked up by position through the layer's position -> cache-row map) and the new token's Eq. 1
// score over that list is taken.  At a scheduled boundary the list is re-selected; selected
// positions without K/V in the next layer form the next in-flight set: they either are in flight
// already or are fetched from the Aux Cache; in-flight rows that fell out go to the Aux Cache.
// How many rows that is depends on the data, so each boundary reads two counters per sequence
// back (one stream synchronisation).
#include <string.h>

#include "runtime.cuh"

namespace lazy {

namespace {

constexpr int PLAN_THREADS = 1024;

__device__ __forceinline__ int seq_of(const int32_t *cu, int n_seqs, int r) {
  int lo = 0, hi = n_seqs;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (cu[mid] <= r) lo = mid; else hi = mid;
  }
  return lo;
}

__device__ __forceinline__ int block_scan_excl(int flag, int *warp_tot, int *total) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t b = __ballot_sync(0xffffffffu, flag);
  const int within = __popc(b & ((1u << lane) - 1u));
  __syncthreads();
  if (lane == 0) warp_tot[warp] = __popc(b);
  __syncthreads();
  int before = 0, tot = 0;
  for (int w = 0; w < PLAN_THREADS / 32; ++w) {
    const int c = warp_tot[w];
    if (w < warp) before += c;
    tot += c;
  }
  *total = tot;
  return before + within;
}

// map[base + tag[base + i]] = base + i for the first `count` rows of a sequence's region
__global__ void map_build_kernel(const int32_t *tags, int32_t *map, int base, int count) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) {
    const int p = tags[base + i];
    if (p >= 0) map[base + p] = base + i;
  }
}

// Per-layer bookkeeping in one launch.  Thread i < m (in-flight rows): the cache row it appends to, its
// position -> row map entry, and the number of context entries it may see (those with position <= its
// own).  Thread i < n (context list): the cache row of this layer holding that position.  A position
// that is in flight gets its row from xmap (the row is being appended by this very step), so no thread
// depends on a map entry another thread of this launch writes.
// blockIdx.y = layer within the segment (the layers up to the next re-selection run on the same in-flight rows
// and the same context list, so their bookkeeping is done in one launch): layer y appends at append_at +
// y * append_stride, owns the map kv_map + y * rows_stride and receives kv_row_new / ctx_rows + y * rows_stride;
// the visible lengths do not depend on the layer and are written by layer 0.
__global__ void dec_prepare_kernel(const int32_t *cu_x, const int32_t *cu_ctx, const int32_t *seq_base,
                                   const int32_t *append_at, const int32_t *xpos, const int32_t *ctx_pos,
                                   const int32_t *xmap, int n_seqs, int m, int n, int32_t *kv_row_new,
                                   int32_t *kv_map, int32_t *q_kvlen, int32_t *ctx_rows, DevStatus *status,
                                   int append_stride, size_t rows_stride) {
  // the projection that follows is a programmatic dependent: it may start fetching weights now and
  // still waits for this grid before it reads the rows computed here; this grid is one too
  LAZY_PDL_ENTER();
  append_at += (size_t)blockIdx.y * append_stride;
  kv_map += (size_t)blockIdx.y * rows_stride;
  kv_row_new += (size_t)blockIdx.y * rows_stride;
  ctx_rows += (size_t)blockIdx.y * rows_stride;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    const int s = seq_of(cu_ctx, n_seqs, i);
    const int p = ctx_pos[i];
    const int xr = xmap[seq_base[s] + p];
    int row = xr >= 0 ? append_at[s] + (xr - cu_x[s]) : kv_map[seq_base[s] + p];
    if (row < 0) {  // a selected token without K/V here would break the subset property
      dev_fail(status, LAZY_E_STATE, W_DECODE, i, p);
      row = seq_base[s];
    }
    ctx_rows[i] = row;
  }
  if (i < m) {
    const int s = seq_of(cu_x, n_seqs, i);
    const int row = append_at[s] + (i - cu_x[s]);
    const int p = xpos[i];
    kv_row_new[i] = row;
    kv_map[seq_base[s] + p] = row;
    const int32_t *list = ctx_pos + cu_ctx[s];
    int lo = 0, hi = cu_ctx[s + 1] - cu_ctx[s];  // first index with list[idx] > p
    if (hi > 0 && list[hi - 1] <= p) lo = hi;    // the new token sees the whole list
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (list[mid] <= p) lo = mid + 1; else hi = mid;
    }
    if (blockIdx.y == 0) q_kvlen[i] = lo;
  }
}

// xmap[base + pos] = row (or -1 to clear) for the in-flight rows.
__global__ void xmap_kernel(const int32_t *cu_x, const int32_t *seq_base, const int32_t *xpos, int n_seqs,
                            int m, int32_t *xmap, int set) {
  int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= m) return;
  const int s = seq_of(cu_x, n_seqs, r);
  xmap[seq_base[s] + xpos[r]] = set ? r : -1;
}

// One CTA per sequence.  Walks the re-selected context (ascending positions): every entry is marked
// selected; entries without K/V in the next layer form the next in-flight list, each with its source:
// >= 0: row of the current in-flight buffer, < 0: -(Aux row + 2).
__global__ void __launch_bounds__(PLAN_THREADS)
dec_plan_kernel(const int32_t *cu_ctx, const int32_t *seq_base, const int32_t *ctx_pos,
                const int32_t *kv_map_next, const int32_t *xmap, const int32_t *aux_map, int32_t *selmark,
                int tag, int32_t *new_pos, int32_t *new_src, int32_t *counts, DevStatus *status) {
  __shared__ int warp_tot[32];
  const int s = blockIdx.x;
  const int c0 = cu_ctx[s], n = cu_ctx[s + 1] - c0, base = seq_base[s];
  int done = 0;
  for (int b = 0; b < n; b += PLAN_THREADS) {
    const int i = b + threadIdx.x;
    int need = 0, p = 0;
    if (i < n) {
      p = ctx_pos[c0 + i];
      selmark[base + p] = tag;
      need = (kv_map_next == nullptr) ? 0 : (kv_map_next[base + p] < 0);
    }
    int tot;
    const int rank = done + block_scan_excl(need, warp_tot, &tot);
    if (need) {
      int src = xmap[base + p];
      if (src < 0) {
        const int a = aux_map[base + p];
        if (a < 0) {  // selected, no K/V ahead, not in flight, not in the Aux Cache: invariant broken
          dev_fail(status, LAZY_E_NOT_IN_AUX, W_DECODE, s, p);
          src = 0;
        } else {
          src = -(a + 2);
        }
      }
      new_pos[c0 + rank] = p;
      new_src[c0 + rank] = src;
    }
    done += tot;
  }
  if (threadIdx.x == 0) counts[2 * s] = done;
}

// One CTA per sequence.  In-flight rows that are no longer selected go to the Aux Cache: emits the
// (source row, Aux row) pairs, tags the Aux rows with their position and maps the position.
__global__ void __launch_bounds__(PLAN_THREADS)
dec_drop_kernel(const int32_t *cu_x, const int32_t *seq_base, const int32_t *xpos, const int32_t *selmark,
                int tag, const int32_t *aux_append_at, int32_t *aux_pos, int32_t *aux_map, int32_t *drop_src,
                int32_t *drop_dst, int32_t *counts) {
  __shared__ int warp_tot[32];
  const int s = blockIdx.x;
  const int x0 = cu_x[s], m = cu_x[s + 1] - x0, base = seq_base[s];
  int done = 0;
  for (int b = 0; b < m; b += PLAN_THREADS) {
    const int i = b + threadIdx.x;
    int drop = 0, p = 0;
    if (i < m) {
      p = xpos[x0 + i];
      drop = selmark[base + p] != tag;
    }
    int tot;
    const int rank = done + block_scan_excl(drop, warp_tot, &tot);
    if (drop) {
      const int dst = aux_append_at[s] + rank;
      drop_src[x0 + rank] = x0 + i;
      drop_dst[x0 + rank] = dst;
      aux_pos[dst] = p;
      aux_map[base + p] = dst;
    }
    done += tot;
  }
  if (threadIdx.x == 0) counts[2 * s + 1] = done;
}

// Builds the next in-flight buffer: row i of sequence s comes from the current buffer or from the
// Aux Cache (whose entry is then retired: the token is about to get K/V in the next layer).
__global__ void dec_build_kernel(const uint4 *__restrict__ x, const uint4 *__restrict__ aux_rows,
                                 uint4 *__restrict__ x_new, const int32_t *__restrict__ new_pos,
                                 const int32_t *__restrict__ new_src, int32_t *__restrict__ xpos_new,
                                 int32_t *__restrict__ revived_pos, const int32_t *cu_tmp,
                                 const int32_t *cu_new, const int32_t *seq_base, int32_t *aux_pos,
                                 int32_t *aux_map, int n_seqs, int m_new, int vec_per_row) {
  for (int r = blockIdx.x; r < m_new; r += gridDim.x) {
    const int s = seq_of(cu_new, n_seqs, r);
    const int t = cu_tmp[s] + (r - cu_new[s]);
    const int src = new_src[t], p = new_pos[t];
    const uint4 *sp;
    if (src >= 0) {
      sp = x + (size_t)src * vec_per_row;
    } else {
      const int a = -(src + 2);
      sp = aux_rows + (size_t)a * vec_per_row;
    }
    uint4 *dp = x_new + (size_t)r * vec_per_row;
    for (int i = threadIdx.x; i < vec_per_row; i += blockDim.x) dp[i] = sp[i];
    if (threadIdx.x == 0) {
      xpos_new[r] = p;
      revived_pos[r] = src >= 0 ? -1 : p;
      if (src < 0) {
        aux_pos[-(src + 2)] = -1;
        aux_map[seq_base[s] + p] = -1;
      }
    }
  }
}

__global__ void set_rows_pos_kernel(int32_t *xpos, const int32_t *p_of_seq, int n_seqs) {
  int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s < n_seqs) xpos[s] = p_of_seq[s];
}

}  // namespace

#define KLAUNCH_OK()  \
  do {                \
    LAZY_COUNT_LAUNCH(); \
    if (cudaPeekAtLastError() != cudaSuccess) return LAZY_E_CUDA; \
  } while (0)

static int build_maps(lazy_ctx *c, cudaStream_t st) {
  const int L = c->L, P = c->P;
  LAZY_TRY(launch_fill_i32(st, c->kv_map, -1, (size_t)L * c->cap_kv));
  LAZY_TRY(launch_fill_i32(st, c->aux_map, -1, (size_t)P * c->cap_kv));
  LAZY_TRY(launch_fill_i32(st, c->dec_i32, -1, (size_t)16 * c->cap_kv));
  for (int l = 0; l < L; ++l)
    for (int s = 0; s < c->n_seqs; ++s) {
      const int cnt = c->kv_count[l][s];
      if (!cnt) continue;
      map_build_kernel<<<cdiv(cnt, 256), 256, 0, st>>>(c->kv_pos + (size_t)l * c->cap_kv,
                                                       c->kv_map + (size_t)l * c->cap_kv, c->seq_base[s], cnt);
      KLAUNCH_OK();
    }
  for (int p = 0; p < P; ++p)
    for (int s = 0; s < c->n_seqs; ++s) {
      const int cnt = c->aux_count[p][s];
      if (!cnt) continue;
      map_build_kernel<<<cdiv(cnt, 256), 256, 0, st>>>(c->aux_pos + (size_t)p * c->cap_kv,
                                                       c->aux_map + (size_t)p * c->cap_kv, c->seq_base[s], cnt);
      KLAUNCH_OK();
    }
  c->maps_built = true;
  c->dec_tag = 0;
  return LAZY_OK;
}

int decode_step_impl(lazy_ctx *c, cudaStream_t st, const int32_t *d_new_ids, float *d_logits,
                     int32_t *d_next_ids) {
  DevStatus *status = dev_status_ptr();
  if (!status) return LAZY_E_CUDA;
  const long long launches0 = g_launches;
  const int S = c->n_seqs, L = c->L, d = c->d, dt = c->dtype, KV = c->cap_kv;
  const int dkv = c->dkv, qc = c->qkv_cols;
  const size_t rb = c->row_bytes();
  for (int s = 0; s < S; ++s) {
    if (c->n_tokens[s] + 1 > c->prompt_len[s] + c->cfg.max_new_tokens) return LAZY_E_CAPACITY;
    if (c->n_tokens[s] >= c->max_pos) return LAZY_E_CAPACITY;
  }
  if (!c->maps_built) LAZY_TRY(build_maps(c, st));
  c->ev_kind.clear();

  // ---- integer scratch
  int32_t *I = c->dec_i32;
  int32_t *ctx_pos = I, *ctx_pos2 = I + (size_t)KV;  // (slot 2 of the scratch is unused)
  int32_t *xpos = I + (size_t)3 * KV, *xpos2 = I + (size_t)4 * KV, *q_kvlen = I + (size_t)5 * KV;
  int32_t *new_src = I + (size_t)7 * KV, *xmap = I + (size_t)8 * KV;  // (slot 6 unused)
  // per layer: the cache rows the in-flight rows append to, and the cache rows of the context list
  auto kv_row_new_of = [&](int l) { return c->dec_seg + (size_t)l * KV; };
  auto ctx_rows_of = [&](int l) { return c->dec_seg + (size_t)(L + l) * KV; };
  int32_t *selmark = I + (size_t)9 * KV, *keep_idx = I + (size_t)10 * KV, *drop_idx = I + (size_t)11 * KV;
  int32_t *new_pos = I + (size_t)12 * KV, *drop_src = I + (size_t)13 * KV, *drop_dst = I + (size_t)14 * KV;
  int32_t *revived = I + (size_t)15 * KV;
  int32_t *tabs = I + (size_t)16 * KV;  // small per-sequence tables, (S+1) ints each
  const int W = c->S + 1;
  enum { T_CU_X = 0, T_CU_CTX, T_CU_KEEP, T_BASE, T_P, T_QROW, T_APPEND, T_AUXAPP, T_CU_NEWX, T_LAST, T_COUNTS = 14 /* two slots: 2 ints per sequence */, T_N = 16 };
  float *scores_sel = c->dec_f32;

  std::vector<int32_t> h((size_t)T_N * W, 0);
  auto tab = [&](int t) { return h.data() + (size_t)t * W; };
  auto dtab = [&](int t) { return tabs + (size_t)t * W; };
  auto upload = [&](int t) {
    return cudaMemcpyAsync(dtab(t), tab(t), (size_t)W * 4, cudaMemcpyHostToDevice, st) == cudaSuccess
               ? LAZY_OK : LAZY_E_CUDA;
  };

  std::vector<int> p_of(S), m_of(S, 1), ctx_n(S);
  int M = S, n_ctx = 0;
  for (int s = 0; s < S; ++s) {
    p_of[s] = c->n_tokens[s];
    ctx_n[s] = p_of[s] + 1;
    tab(T_CU_X)[s + 1] = s + 1;
    tab(T_CU_CTX)[s + 1] = tab(T_CU_CTX)[s] + ctx_n[s];
    tab(T_BASE)[s] = c->seq_base[s];
    tab(T_P)[s] = p_of[s];
    n_ctx += ctx_n[s];
  }
  if (n_ctx > KV) return LAZY_E_CAPACITY;
  LAZY_TRY(upload(T_CU_X));
  // Where each layer's cache appends this step is known up front (one table per layer, one copy); the
  // score row only moves when the in-flight set changes.
  std::vector<int32_t> h_append((size_t)L * W, 0);
  for (int l = 0; l < L; ++l)
    for (int s = 0; s < S; ++s) h_append[(size_t)l * W + s] = c->seq_base[s] + c->kv_count[l][s];
  int32_t *d_append = tabs + (size_t)2 * T_N * W;
  LAZY_CUDA_OK(cudaMemcpyAsync(d_append, h_append.data(), h_append.size() * 4, cudaMemcpyHostToDevice, st));
  for (int s = 0; s < S; ++s) tab(T_QROW)[s] = tab(T_CU_X)[s + 1] - 1;  // the new token: largest position
  LAZY_TRY(upload(T_QROW));
  LAZY_TRY(upload(T_CU_CTX));
  LAZY_TRY(upload(T_BASE));
  LAZY_TRY(upload(T_P));
  memset(c->stats.rows_computed, 0, sizeof(c->stats.rows_computed));
  memset(c->stats.revived, 0, sizeof(c->stats.revived));
  c->seg_cu.assign(c->P + 1, std::vector<int>(S + 1, 0));
  for (int s = 0; s <= S; ++s) c->seg_cu[0][s] = tab(T_CU_CTX)[s];
  c->dec_revived_cu.assign(c->P, std::vector<int>(S + 1, 0));

  // new token rows and the full context 0..p
  LAZY_TRY(launch_embed(st, dt, c->tok_embed, d_new_ids, c->x, S, d, c->V, status));
  set_rows_pos_kernel<<<cdiv(S, 128), 128, 0, st>>>(xpos, dtab(T_P), S);
  KLAUNCH_OK();
  LAZY_TRY(launch_iota_pos(st, ctx_pos, dtab(T_CU_CTX), S, n_ctx));
  LAZY_CUDA_OK(cudaMemcpyAsync(c->pos_seg[0], ctx_pos, (size_t)n_ctx * 4, cudaMemcpyDeviceToDevice, st));
  xmap_kernel<<<cdiv(M, 256), 256, 0, st>>>(dtab(T_CU_X), dtab(T_BASE), xpos, S, M, xmap, 1);
  KLAUNCH_OK();

  char *x = c->x, *x2 = c->x2;
  int seg_end = -1;        // last layer of the segment whose bookkeeping has been launched
  int score_from = -1;     // first layer of the segment whose head means are still to be taken (-1: none pending)
  size_t score_stride = 0; // floats between two layers' logits + statistics in the score scratch
  for (int l = 0; l < L; ++l) {
    int32_t *kv_row_new = kv_row_new_of(l), *ctx_rows = ctx_rows_of(l);
    char *kc = c->kcache + (size_t)l * KV * c->kv_row_bytes();
    char *vc = c->vcache + (size_t)l * KV * c->kv_row_bytes();
    int32_t *kvp = c->kv_pos + (size_t)l * KV;
    int32_t *kvm = c->kv_map + (size_t)l * KV;
    float *sc = c->scores + (size_t)l * KV;
    int max_m = 0;
    for (int s = 0; s < S; ++s) {
      if (c->kv_count[l][s] + m_of[s] > c->prompt_len[s] + c->cfg.max_new_tokens) return LAZY_E_CAPACITY;
      if (m_of[s] > max_m) max_m = m_of[s];
    }
    if (M > c->cap_rows) return LAZY_E_CAPACITY;
    c->stats.rows_computed[l] = M;

    if (l > seg_end) {
      // Bookkeeping first (the projection below may already write the rows' K/V into their cache rows), for
      // every layer up to the next re-selection at once: they all run on these in-flight rows and this context.
      seg_end = l;
      while (seg_end + 1 < L && c->point_at[seg_end + 1] < 0) ++seg_end;
      for (int ll = l + 1; ll <= seg_end; ++ll)
        for (int s = 0; s < S; ++s)
          if (c->kv_count[ll][s] + m_of[s] > c->prompt_len[s] + c->cfg.max_new_tokens) return LAZY_E_CAPACITY;
      const int n_thr = M > n_ctx ? M : n_ctx;
      LAZY_TRY(launch_pdl(dec_prepare_kernel, dim3(cdiv(n_thr, 256), seg_end - l + 1), dim3(256), 0, st,
                          (const int32_t *)dtab(T_CU_X), (const int32_t *)dtab(T_CU_CTX),
                          (const int32_t *)dtab(T_BASE), (const int32_t *)(d_append + (size_t)l * W),
                          (const int32_t *)xpos, (const int32_t *)ctx_pos, (const int32_t *)xmap, S, M, n_ctx,
                          kv_row_new, kvm, q_kvlen, ctx_rows, status, W, (size_t)KV));
      KLAUNCH_OK();
      // room for every layer's score logits and statistics side by side? then their head means wait for the
      // segment's last layer
      score_stride = align_up((size_t)c->H * n_ctx + (size_t)2 * S * c->H, 64);
      score_from = score_stride * (size_t)(seg_end - l + 1) <= c->score_scratch_cap ? l : -1;
    }
    if (gemv_small_m_eligible(dt, M, d) && c->dh == 128 && dkv % 128 == 0) {
      // one to four rows: one weight-streaming kernel does RMSNorm, the projection, RoPE and the cache write
      LAZY_TRY(launch_gemv_qkv_rope(st, x, c->w_qkv[l], c->qkv, c->g_attn[l], c->cfg.rms_eps, xpos, c->rope_table,
                                    kc, vc, kvp, kv_row_new, M, d, c->max_pos, status, dkv));
    } else {
      if (gemv_small_m_eligible(dt, M, d)) {
        LAZY_TRY(launch_gemv_small_m(st, x, c->w_qkv[l], nullptr, nullptr, c->qkv, M, qc, d, 0, c->g_attn[l],
                                     c->cfg.rms_eps, 0, true));
      } else {
        LAZY_TRY(launch_rmsnorm(st, dt, x, c->g_attn[l], c->h, M, d, c->cfg.rms_eps));
        LAZY_TRY(launch_gemm(st, dt, c->h, c->w_qkv[l], nullptr, c->qkv, M, qc, d, status, c->gemm_scratch,
                             c->gemm_scratch_bytes, 0, true));
      }
      LAZY_TRY(launch_rope_kv(st, dt, c->qkv, xpos, c->rope_table, kc, vc, kvp, kv_row_new, M, c->H, c->dh,
                              c->max_pos, status, c->Hkv));
    }
    for (int s = 0; s < S; ++s) c->kv_count[l][s] += m_of[s];
    int max_ctx = 0;
    for (int s = 0; s < S; ++s) max_ctx = ctx_n[s] > max_ctx ? ctx_n[s] : max_ctx;
    // the MLP activation buffer is idle during attention: it holds the split partials
    if (attention_decode_eligible(dt, c->dh, M, max_ctx) &&
        attention_decode_scratch_floats(M, c->H, max_ctx) * 4 <= (size_t)c->cap_rows * c->F * c->eb) {
      float *logits = c->score_scratch + (score_from >= 0 ? (size_t)(l - score_from) * score_stride : 0);
      float *stats = logits + (size_t)c->H * n_ctx;
      LAZY_TRY(launch_attention_decode(st, c->qkv, qc, kc, vc, dkv, c->attn, d, dtab(T_CU_X), dtab(T_CU_CTX),
                                       ctx_rows, q_kvlen, dtab(T_QROW), S, M, n_ctx, max_ctx, c->H,
                                       (float *)c->act, logits, stats, c->Hkv));
      if (score_from < 0) {
        LAZY_TRY(launch_score_mean(st, logits, stats, dtab(T_CU_CTX), S, n_ctx, c->H, sc));
      } else if (l == seg_end) {  // Eq. 1 head means of the whole segment, before its scores are needed
        LAZY_TRY(launch_score_mean(st, c->score_scratch, c->score_scratch + (size_t)c->H * n_ctx, dtab(T_CU_CTX), S,
                                   n_ctx, c->H, c->scores + (size_t)score_from * KV, seg_end - score_from + 1,
                                   score_stride, (size_t)KV));
      }
    } else {
      // many rows in flight: the tile kernel, with the key list cut into slices when there are too few
      // (query tile, head) pairs to fill the machine
      const int splits = attention_list_split_eligible(dt, c->dh) ? attention_list_splits(S, max_m, c->H, max_ctx) : 1;
      if (splits > 1 && (size_t)M * c->H * splits * 130 * 4 <= (size_t)c->cap_rows * c->F * c->eb) {
        LAZY_TRY(launch_attention_list_split(st, c->qkv, qc, kc, vc, dkv, c->attn, dtab(T_CU_X), dtab(T_CU_CTX),
                                             ctx_rows, q_kvlen, dtab(T_QROW), S, max_m, M, c->H, splits,
                                             (float *)c->act, c->score_scratch + (size_t)c->H * n_ctx, c->Hkv));
      } else {
        LAZY_TRY(launch_attention_ex(st, dt, c->qkv, qc, kc, vc, dkv, c->attn, dtab(T_CU_X), nullptr,
                                     dtab(T_CU_CTX), ctx_rows, q_kvlen, S, max_m, M, c->H, c->dh, c->Hkv));
      }
      LAZY_TRY(launch_score_ex(st, dt, c->qkv, qc, kc, dkv, dtab(T_CU_CTX), nullptr, ctx_rows, dtab(T_QROW), S,
                               n_ctx, max_ctx, c->H, c->dh, c->score_scratch, sc, c->Hkv));
    }
    LAZY_TRY(launch_gemm(st, dt, c->attn, c->w_o[l], x, x, M, d, d, status, c->gemm_scratch, c->gemm_scratch_bytes, 0,
                         true));

    const int pt = c->point_at[l + 1];
    // The layer's MLP on the rows in flight (revived rows included, under the default cut point).
    auto run_mlp = [&]() -> int {
      if (gemv_small_m_eligible(dt, M, d)) {
        LAZY_TRY(launch_gemv_small_m(st, x, c->w_gate[l], c->w_up[l], nullptr, c->act, M, c->F, d, 1, c->g_mlp[l],
                                     c->cfg.rms_eps, 0, true));
      } else {
        LAZY_TRY(launch_rmsnorm(st, dt, x, c->g_mlp[l], c->h, M, d, c->cfg.rms_eps));
        LAZY_TRY(launch_gemm_swiglu(st, dt, c->h, c->w_gate[l], c->w_up[l], c->act, M, c->F, d, status,
                                    c->gemm_scratch, c->gemm_scratch_bytes, 0, true));
      }
      LAZY_TRY(launch_gemm(st, dt, c->act, c->w_down[l], x, x, M, d, c->F, status, c->gemm_scratch,
                           c->gemm_scratch_bytes, 0, true));
      return LAZY_OK;
    };
    // cut after the whole layer: the MLP runs before the re-selection, and rows revived from the Aux Cache
    // (layer outputs under that reading) skip it
    const bool cut_after = pt >= 0 && c->aux_after_layer;
    if (cut_after) LAZY_TRY(run_mlp());
    if (pt >= 0) {
      // ---- re-select the context by the new token's score
      const float *sel = sc;
      bool any_forced = false;
      for (int s = 0; s < S; ++s) {
        int keep = keep_count(p_of[s] + 1, c->sched_bp[pt], ctx_n[s]);
        auto it = c->forced.find(std::make_pair(pt, s));
        if (it != c->forced.end()) {
          keep = it->second.second;
          if (keep < 1 || keep > ctx_n[s]) return LAZY_E_BADARG;
          any_forced = true;
        }
        tab(T_CU_KEEP)[s + 1] = tab(T_CU_KEEP)[s] + keep;
      }
      LAZY_TRY(upload(T_CU_KEEP));
      if (any_forced) {
        LAZY_CUDA_OK(cudaMemcpyAsync(scores_sel, sc, (size_t)n_ctx * 4, cudaMemcpyDeviceToDevice, st));
        for (int s = 0; s < S; ++s) {
          auto it = c->forced.find(std::make_pair(pt, s));
          if (it == c->forced.end()) continue;
          LAZY_TRY(launch_forced_scores(st, ctx_pos, tab(T_CU_CTX)[s], ctx_n[s], it->second.first,
                                        it->second.second, scores_sel));
        }
        sel = scores_sel;
      }
      if (c->select_threshold) {
        // threshold reading: ties at the scheduled rank all survive; the counts come back from the device
        // (one more stream synchronisation at this boundary)
        LAZY_TRY(launch_select_tie_count(st, sel, dtab(T_CU_CTX), dtab(T_CU_KEEP), S, dtab(T_COUNTS), status));
        LAZY_CUDA_OK(cudaMemcpyAsync(tab(T_COUNTS), dtab(T_COUNTS), (size_t)S * 4, cudaMemcpyDeviceToHost, st));
        LAZY_CUDA_OK(cudaStreamSynchronize(st));
        for (int s = 0; s < S; ++s) {
          const int keep = tab(T_COUNTS)[s];
          if (keep < 1 || keep > ctx_n[s]) return LAZY_E_STATE;
          tab(T_CU_KEEP)[s + 1] = tab(T_CU_KEEP)[s] + keep;
        }
        LAZY_TRY(upload(T_CU_KEEP));
      }
      LAZY_TRY(launch_select(st, sel, dtab(T_CU_CTX), dtab(T_CU_KEEP), S, keep_idx, drop_idx, status));
      const int n_keep = tab(T_CU_KEEP)[S];
      LAZY_TRY(launch_move_i32(st, ctx_pos, keep_idx, ctx_pos2, nullptr, n_keep));
      { int32_t *t = ctx_pos; ctx_pos = ctx_pos2; ctx_pos2 = t; }
      for (int s = 0; s <= S; ++s) tab(T_CU_CTX)[s] = tab(T_CU_KEEP)[s];
      for (int s = 0; s < S; ++s) ctx_n[s] = tab(T_CU_CTX)[s + 1] - tab(T_CU_CTX)[s];
      n_ctx = n_keep;
      LAZY_TRY(upload(T_CU_CTX));
      for (int s = 0; s <= S; ++s) c->seg_cu[pt + 1][s] = tab(T_CU_CTX)[s];
      LAZY_CUDA_OK(cudaMemcpyAsync(c->pos_seg[pt + 1], ctx_pos, (size_t)n_ctx * 4, cudaMemcpyDeviceToDevice, st));

      // ---- plan the next in-flight set, retire rows that fell out
      const int tag = ++c->dec_tag;
      int32_t *ap = c->aux_pos + (size_t)pt * KV;
      int32_t *am = c->aux_map + (size_t)pt * KV;
      char *ar = c->aux_rows + (size_t)pt * KV * rb;
      for (int s = 0; s < S; ++s) tab(T_AUXAPP)[s] = c->seq_base[s] + c->aux_count[pt][s];
      LAZY_TRY(upload(T_AUXAPP));
      dec_plan_kernel<<<S, PLAN_THREADS, 0, st>>>(dtab(T_CU_CTX), dtab(T_BASE), ctx_pos,
                                                  c->kv_map + (size_t)(l + 1) * KV, xmap, am, selmark, tag,
                                                  new_pos, new_src, dtab(T_COUNTS), status);
      KLAUNCH_OK();
      dec_drop_kernel<<<S, PLAN_THREADS, 0, st>>>(dtab(T_CU_X), dtab(T_BASE), xpos, selmark, tag,
                                                  dtab(T_AUXAPP), ap, am, drop_src, drop_dst, dtab(T_COUNTS));
      KLAUNCH_OK();
      LAZY_CUDA_OK(cudaMemcpyAsync(tab(T_COUNTS), dtab(T_COUNTS), (size_t)2 * S * 4, cudaMemcpyDeviceToHost, st));
      LAZY_CUDA_OK(cudaStreamSynchronize(st));
      int m_new = 0, n_drop = 0;
      for (int s = 0; s < S; ++s) {
        const int cn = tab(T_COUNTS)[2 * s], cd = tab(T_COUNTS)[2 * s + 1];
        if (c->aux_count[pt][s] + cd > c->prompt_len[s] + c->cfg.max_new_tokens) return LAZY_E_CAPACITY;
        tab(T_CU_NEWX)[s + 1] = tab(T_CU_NEWX)[s] + cn;
        m_new += cn;
        n_drop += cd;
      }
      if (m_new > c->cap_rows) return LAZY_E_CAPACITY;
      LAZY_TRY(upload(T_CU_NEWX));
      // rows that fell out -> Aux Cache (lists of sequence s sit at offset cu_x[s])
      for (int s = 0; s < S; ++s) {
        const int cd = tab(T_COUNTS)[2 * s + 1], x0 = tab(T_CU_X)[s];
        LAZY_TRY(launch_move_rows(st, x, drop_src + x0, ar, drop_dst + x0, cd, (int)rb, M, KV, status));
        c->aux_count[pt][s] += cd;
      }
      xmap_kernel<<<cdiv(M, 256), 256, 0, st>>>(dtab(T_CU_X), dtab(T_BASE), xpos, S, M, xmap, 0);
      KLAUNCH_OK();
      if (m_new > 0) {
        int blocks = m_new < sm_count() * 16 ? m_new : sm_count() * 16;
        dec_build_kernel<<<blocks, 128, 0, st>>>((const uint4 *)x, (const uint4 *)ar, (uint4 *)x2, new_pos,
                                                 new_src, xpos2, revived, dtab(T_CU_CTX), dtab(T_CU_NEWX),
                                                 dtab(T_BASE), ap, am, S, m_new, (int)(rb / 16));
        KLAUNCH_OK();
      }
      { char *t = x; x = x2; x2 = t; }
      { int32_t *t = xpos; xpos = xpos2; xpos2 = t; }
      int revived_total = 0;
      for (int s = 0; s < S; ++s) {
        const int carried = m_of[s] - tab(T_COUNTS)[2 * s + 1];
        const int rv = tab(T_COUNTS)[2 * s] - carried;
        revived_total += rv;
        c->aux_live[pt][s] += tab(T_COUNTS)[2 * s + 1] - rv;
        m_of[s] = tab(T_COUNTS)[2 * s];
        tab(T_CU_X)[s + 1] = tab(T_CU_NEWX)[s + 1];
        c->dec_revived_cu[pt][s + 1] = tab(T_CU_NEWX)[s + 1];
      }
      LAZY_CUDA_OK(cudaMemcpyAsync(c->revived_pos[pt], revived, (size_t)m_new * 4, cudaMemcpyDeviceToDevice, st));
      M = m_new;
      LAZY_TRY(upload(T_CU_X));
      for (int s = 0; s < S; ++s) tab(T_QROW)[s] = tab(T_CU_X)[s + 1] - 1;
      LAZY_TRY(upload(T_QROW));
      xmap_kernel<<<cdiv(M, 256), 256, 0, st>>>(dtab(T_CU_X), dtab(T_BASE), xpos, S, M, xmap, 1);
      KLAUNCH_OK();
      c->stats.revived[l + 1] = revived_total;
    }
    if (!cut_after) LAZY_TRY(run_mlp());
  }
  for (int s = 0; s < S; ++s) tab(T_LAST)[s] = tab(T_CU_X)[s + 1] - 1;
  LAZY_TRY(upload(T_LAST));
  LAZY_TRY(launch_rmsnorm_rows(st, dt, x, dtab(T_LAST), c->g_final, c->h_last, S, d, c->cfg.rms_eps));
  LAZY_TRY(launch_lm_head(st, dt, c->h_last, c->w_lm_head, d_logits, S, d, c->V, true));
  if (d_next_ids) LAZY_TRY(launch_argmax(st, d_logits, d_next_ids, S, c->V));
  xmap_kernel<<<cdiv(M, 256), 256, 0, st>>>(dtab(T_CU_X), dtab(T_BASE), xpos, S, M, xmap, 0);
  KLAUNCH_OK();
  // the small host tables above are read by asynchronous copies: finish them before they go away
  LAZY_CUDA_OK(cudaStreamSynchronize(st));
  for (int s = 0; s < S; ++s) c->n_tokens[s] += 1;
  for (int l = 0; l < L; ++l) {
    int tot = 0;
    for (int s = 0; s < S; ++s) tot += c->kv_count[l][s];
    c->stats.kv_rows[l] = tot;
    const int pt = l + 1 <= L ? c->point_at[l + 1] : -1;
    if (pt >= 0) {
      int a = 0;
      for (int s = 0; s < S; ++s) a += c->aux_live[pt][s];
      c->stats.aux_rows[l] = a;
    }
  }
  c->forced.clear();
  c->last_was_decode = true;
  c->stats.kernel_launches = g_launches - launches0;
  return LAZY_OK;
}

}  // namespace lazy
