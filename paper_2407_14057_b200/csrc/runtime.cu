// Context set-up, the token-pruned prefill, Aux-Cache reads and the introspection calls.
#include <string.h>

#include <new>

#include "gemm_epilogue.cuh"
#include "runtime.cuh"

namespace lazy {

// ---- small kernels used only by the runtime ---------------------------------------------------
__global__ void move_rows_kernel(const uint4 *__restrict__ src, const int32_t *__restrict__ src_idx,
                                 uint4 *__restrict__ dst, const int32_t *__restrict__ dst_idx, int n,
                                 int vec_per_row, int src_rows, int dst_rows, DevStatus *status) {
  for (int r = blockIdx.x; r < n; r += gridDim.x) {
    const int s = src_idx ? src_idx[r] : r;
    const int t = dst_idx ? dst_idx[r] : r;
    if (s < 0 || s >= src_rows || t < 0 || t >= dst_rows) {
      if (threadIdx.x == 0) dev_fail(status, LAZY_E_BADARG, W_GATHER_INDEX, s, t);
      continue;
    }
    const uint4 *sp = src + (size_t)s * vec_per_row;
    uint4 *dp = dst + (size_t)t * vec_per_row;
    for (int i = threadIdx.x; i < vec_per_row; i += blockDim.x) dp[i] = sp[i];
  }
}
int launch_move_rows(cudaStream_t st, const void *src, const int32_t *src_idx, void *dst,
                     const int32_t *dst_idx, int n, int row_bytes, int src_rows, int dst_rows,
                     DevStatus *status) {
  if (n == 0) return LAZY_OK;
  int blocks = n < sm_count() * 16 ? n : sm_count() * 16;
  move_rows_kernel<<<blocks, 128, 0, st>>>((const uint4 *)src, src_idx, (uint4 *)dst, dst_idx, n,
                                           row_bytes / 16, src_rows, dst_rows, status);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

__global__ void move_i32_kernel(const int32_t *src, const int32_t *src_idx, int32_t *dst,
                                const int32_t *dst_idx, int n) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[dst_idx ? dst_idx[i] : i] = src[src_idx ? src_idx[i] : i];
}
int launch_move_i32(cudaStream_t st, const int32_t *src, const int32_t *src_idx, int32_t *dst,
                    const int32_t *dst_idx, int n) {
  if (n == 0) return LAZY_OK;
  move_i32_kernel<<<cdiv(n, 256), 256, 0, st>>>(src, src_idx, dst, dst_idx, n);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

__global__ void seg_rows_kernel(const int32_t *cu, const int32_t *base, int n_seqs, int n_total,
                                int32_t *out) {
  int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= n_total) return;
  int lo = 0, hi = n_seqs;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (cu[mid] <= r) lo = mid; else hi = mid;
  }
  out[r] = base[lo] + (r - cu[lo]);
}
int launch_seg_rows(cudaStream_t st, const int32_t *cu, const int32_t *base, int n_seqs, int n_total,
                    int32_t *out) {
  if (n_total == 0) return LAZY_OK;
  seg_rows_kernel<<<cdiv(n_total, 256), 256, 0, st>>>(cu, base, n_seqs, n_total, out);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

// For each requested position: the Aux row that holds it (scan of the sequence's region), or -1.
__global__ void aux_find_kernel(const int32_t *__restrict__ aux_pos, int region0, int count,
                                const int32_t *__restrict__ want, int n, int32_t *__restrict__ found,
                                DevStatus *status) {
  const int i = blockIdx.x;
  if (i >= n) return;
  const int p = want[i];
  __shared__ int hit;
  if (threadIdx.x == 0) hit = -1;
  __syncthreads();
  for (int j = threadIdx.x; j < count; j += blockDim.x)
    if (aux_pos[region0 + j] == p) hit = region0 + j;
  __syncthreads();
  if (threadIdx.x == 0) {
    found[i] = hit;
    if (hit < 0) dev_fail(status, LAZY_E_NOT_IN_AUX, W_AUX_LOOKUP, i, p);
  }
}

// ---- validation ------------------------------------------------------------------------------------
int validate_cfg(const lazy_model_cfg *c) {
  if (!c) return LAZY_E_BADARG;
  if (c->n_layers < 1 || c->n_layers > LAZY_MAX_LAYERS || c->d_model < 1 || c->n_heads < 1 ||
      c->head_dim < 1 || c->d_ffn < 1 || c->vocab < 1)
    return LAZY_E_BADARG;
  if (c->n_heads * c->head_dim != c->d_model) return LAZY_E_BADARG;
  if (c->n_kv_heads < 0 || (c->n_kv_heads > 0 && c->n_heads % c->n_kv_heads)) return LAZY_E_BADARG;
  if (c->dtype != LAZY_BF16 && c->dtype != LAZY_F32) return LAZY_E_BADARG;
  // 16-byte vectors everywhere; RoPE pairs 16-byte vectors of the two halves of a head;
  // the generic attention kernel gives each lane head_dim/32 output columns.
  const int v = c->dtype == LAZY_F32 ? 4 : 8;
  if (c->d_model % 8 || c->d_ffn % 8 || (c->head_dim / 2) % v || c->head_dim % 32 || c->head_dim > 256)
    return LAZY_E_BADARG;
  const int lpk = c->head_dim / v;
  if (lpk > 32 || (lpk & (lpk - 1))) return LAZY_E_BADARG;
  if (c->max_seqs < 1 || c->max_prompt_tokens < 1 || c->max_new_tokens < 0) return LAZY_E_BADARG;
  if (!(c->rms_eps > 0.f) || !(c->rope_theta > 0.f)) return LAZY_E_BADARG;
  return LAZY_OK;
}

int validate_schedule(const lazy_model_cfg *c, const lazy_schedule *s) {
  if (!s || s->n_points < 0 || s->n_points >= LAZY_MAX_LAYERS) return LAZY_E_BADSCHEDULE;
  if (s->n_points > 0 && (!s->layer_entered || !s->keep_bp)) return LAZY_E_BADSCHEDULE;
  int prev_e = 0;
  uint32_t prev_bp = 10000;
  for (int i = 0; i < s->n_points; ++i) {
    const int e = s->layer_entered[i];
    const uint32_t bp = s->keep_bp[i];
    if (!(prev_e < e && e < c->n_layers)) return LAZY_E_BADSCHEDULE;
    if (bp < 1 || bp > 10000 || bp > prev_bp) return LAZY_E_BADSCHEDULE;
    prev_e = e;
    prev_bp = bp;
  }
  return LAZY_OK;
}

// ---- workspace carve-up -------------------------------------------------------------------------------
struct Carver {
  char *base;
  size_t off;
  explicit Carver(char *b) : base(b), off(0) {}
  char *take(size_t bytes) {
    char *p = base ? base + off : nullptr;
    off += align_up(bytes ? bytes : 1, 256);
    return p;
  }
};

// Fills the pointers of `c` (all NULL-based offsets when base is NULL) and returns the bytes needed.
static size_t carve(lazy_ctx *c, char *base, bool with_capture) {
  Carver k(base);
  const size_t rb = c->row_bytes();
  const size_t R = (size_t)c->cap_rows, KV = (size_t)c->cap_kv;
  const int P = c->P, L = c->L;
  c->x = k.take(R * rb);
  c->x2 = k.take(R * rb);
  c->h = k.take(R * rb);
  c->qkv = k.take(R * (size_t)c->qkv_cols * c->eb);
  c->attn = k.take(R * rb);
  c->act = k.take(R * (size_t)c->F * c->eb);
  c->h_last = k.take((size_t)c->S * rb);
  c->pos_seg.assign(P + 1, nullptr);
  c->kv_row.assign(P + 1, nullptr);
  for (int g = 0; g <= P; ++g) {
    c->pos_seg[g] = (int32_t *)k.take(KV * 4);
    c->kv_row[g] = (int32_t *)k.take(R * 4);
  }
  c->scores = (float *)k.take((size_t)L * KV * 4);
  c->sel_scores = (float *)k.take(R * 4);
  {
    // prefill keeps the attention kernel's score by-product of every layer (the head means of the layers
    // between two cuts are taken in one launch); decode uses the same memory for its per-step logits
    size_t a = score_scratch_floats(c->S, c->cap_kv, c->H);
    c->score_layer_stride = align_up(attn_score_scratch_floats(c->S, c->H, c->cap_rows / 64 + 1), 64);
    size_t b = c->score_layer_stride * (size_t)c->L;
    c->score_scratch_cap = a > b ? a : b;
    c->score_scratch = (float *)k.take(c->score_scratch_cap * 4);
  }
  c->keep_idx.assign(P, nullptr);
  c->drop_idx.assign(P, nullptr);
  c->aux_dst.assign(P, nullptr);
  for (int p = 0; p < P; ++p) {
    c->keep_idx[p] = (int32_t *)k.take(R * 4);
    c->drop_idx[p] = (int32_t *)k.take(R * 4);
    c->aux_dst[p] = (int32_t *)k.take(R * 4);
  }
  c->revived_pos.assign(P, nullptr);
  for (int p = 0; p < P; ++p) c->revived_pos[p] = (int32_t *)k.take(KV * 4);
  c->rope_table = (float *)k.take((size_t)c->max_pos * c->dh * 4);
  c->kcache = k.take((size_t)L * KV * c->kv_row_bytes());
  c->vcache = k.take((size_t)L * KV * c->kv_row_bytes());
  c->kv_pos = (int32_t *)k.take((size_t)L * KV * 4);
  c->aux_rows = k.take((size_t)P * KV * rb);
  c->aux_pos = (int32_t *)k.take((size_t)P * KV * 4);
  c->d_ints = (int32_t *)k.take((size_t)(2 * P + 8) * (c->S + 1) * 4);
  c->d_found = (int32_t *)k.take(KV * 4);
  c->kv_map = (int32_t *)k.take((size_t)L * KV * 4);
  c->aux_map = (int32_t *)k.take((size_t)P * KV * 4);
  c->dec_i32 = (int32_t *)k.take((size_t)16 * KV * 4 + (size_t)(16 * 2 + L) * (c->S + 1) * 4);
  c->dec_f32 = (float *)k.take((size_t)2 * KV * 4);
  c->dec_seg = (int32_t *)k.take((size_t)2 * L * KV * 4);
  c->a8 = (uint8_t *)k.take(c->dtype == LAZY_BF16 ? R * (size_t)(c->F > c->d ? c->F : c->d) : 0);
  c->a8_scale = (float *)k.take(c->dtype == LAZY_BF16 ? R * 4 : 0);
  c->gemm_scratch_bytes = c->dtype == LAZY_BF16 ? gemm_scratch_bytes() : 0;
  c->gemm_scratch = c->gemm_scratch_bytes ? k.take(c->gemm_scratch_bytes) : nullptr;
  c->capture = with_capture ? k.take((size_t)L * R * rb) : nullptr;
  return k.off;
}

static void fill_shape(lazy_ctx *c, const lazy_model_cfg *cfg, const lazy_schedule *s) {
  c->cfg = *cfg;
  c->L = cfg->n_layers;
  c->d = cfg->d_model;
  c->H = cfg->n_heads;
  c->dh = cfg->head_dim;
  c->Hkv = cfg->n_kv_heads > 0 ? cfg->n_kv_heads : cfg->n_heads;
  c->dkv = c->Hkv * cfg->head_dim;
  c->qkv_cols = cfg->d_model + 2 * c->dkv;
  c->F = cfg->d_ffn;
  c->V = cfg->vocab;
  c->dtype = cfg->dtype;
  c->eb = elem_bytes(cfg->dtype);
  c->S = cfg->max_seqs;
  c->P = s->n_points;
  c->sched_layer.assign(s->layer_entered, s->layer_entered + s->n_points);
  c->sched_bp.assign(s->keep_bp, s->keep_bp + s->n_points);
  c->point_at.assign(c->L + 1, -1);
  for (int p = 0; p < c->P; ++p) c->point_at[c->sched_layer[p]] = p;
  c->cap_rows = cfg->max_prompt_tokens;
  c->cap_kv = cfg->max_prompt_tokens + cfg->max_seqs * cfg->max_new_tokens;
  c->max_pos = cfg->max_prompt_tokens + cfg->max_new_tokens;
}

// The split-wave GEMMs leave their arrival counters at zero, except when a bounded wait ran out in the
// middle of a launch.  A run that follows such a failure must not inherit the stale counts, so every run
// starts by clearing the 2 KiB counter block (one tiny memset in a 27 ms prefill / 3 ms decode step).
static int reset_gemm_counters(lazy_ctx *c, cudaStream_t st) {
  if (!c->gemm_scratch) return LAZY_OK;
  return cudaMemsetAsync(c->gemm_scratch, 0, GEMM_TAIL_COUNTER_BYTES, st) == cudaSuccess ? LAZY_OK : LAZY_E_CUDA;
}

}  // namespace lazy

using namespace lazy;

lazy_ctx::~lazy_ctx() {
  for (cudaEvent_t e : ev_pool) cudaEventDestroy(e);
}
int lazy_ctx::time_begin(cudaStream_t st, int kind, double flops, double bytes) {
  if (!timing_on || !((timing_mask >> kind) & 1u)) return -1;
  k_flops[kind] += flops;
  k_bytes[kind] += bytes;
  const int slot = (int)ev_kind.size();
  while ((int)ev_pool.size() < 2 * (slot + 1)) {
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) return -1;
    ev_pool.push_back(e);
  }
  ev_kind.push_back(kind);
  ev_flops.push_back(flops);
  ev_bytes.push_back(bytes);
  cudaEventRecord(ev_pool[2 * slot], st);
  return slot;
}
void lazy_ctx::time_end(cudaStream_t st, int slot) {
  if (slot >= 0) cudaEventRecord(ev_pool[2 * slot + 1], st);
}
// Runs one launcher call bracketed by an event pair when timing is on.
#define TIMED(kind, flops, bytes, call)                                  \
  do {                                                                   \
    const int slot__ = c->time_begin(st, (kind), (double)(flops), (double)(bytes)); \
    const int rc__ = (call);                                             \
    c->time_end(st, slot__);                                             \
    if (rc__ != LAZY_OK) return rc__;                                    \
  } while (0)

// =====================================================================================================
extern "C" {

size_t lazy_prefill_workspace_bytes_ex(const lazy_model_cfg *cfg, const lazy_schedule *sched,
                                       int32_t debug_capture) {
  if (validate_cfg(cfg) != LAZY_OK || validate_schedule(cfg, sched) != LAZY_OK) return 0;
  lazy_ctx tmp;
  fill_shape(&tmp, cfg, sched);
  return carve(&tmp, nullptr, debug_capture != 0);
}
size_t lazy_prefill_workspace_bytes(const lazy_model_cfg *cfg, const lazy_schedule *sched) {
  return lazy_prefill_workspace_bytes_ex(cfg, sched, 0);
}

int lazy_prefill_init(const lazy_model_cfg *cfg, const lazy_weights *w, const lazy_schedule *sched,
                      void *d_workspace, size_t workspace_bytes, lazy_ctx **out) {
  if (!out) return LAZY_E_BADARG;
  *out = nullptr;
  LAZY_TRY(validate_cfg(cfg));
  int rc = validate_schedule(cfg, sched);
  if (rc != LAZY_OK) return rc;
  if (!w || !d_workspace || ((uintptr_t)d_workspace & 255)) return LAZY_E_BADARG;
  if (!w->tok_embed || !w->w_qkv || !w->w_o || !w->w_gate || !w->w_up || !w->w_down || !w->g_attn ||
      !w->g_mlp || !w->g_final || !w->w_lm_head)
    return LAZY_E_BADARG;
  for (int l = 0; l < cfg->n_layers; ++l) {
    const void *ps[7] = {w->w_qkv[l], w->w_o[l], w->w_gate[l], w->w_up[l], w->w_down[l], w->g_attn[l],
                         w->g_mlp[l]};
    for (const void *p : ps)
      if (!p || ((uintptr_t)p & 15)) return LAZY_E_BADARG;
  }
  lazy_ctx *c = new (std::nothrow) lazy_ctx();
  if (!c) return LAZY_E_BADARG;
  fill_shape(c, cfg, sched);
  const size_t need = carve(c, nullptr, false);
  const size_t need_cap = carve(c, nullptr, true);
  if (workspace_bytes < need) {
    delete c;
    return LAZY_E_CAPACITY;
  }
  c->capture_sized = workspace_bytes >= need_cap;
  carve(c, (char *)d_workspace, c->capture_sized);
  c->ws_base = (char *)d_workspace;
  c->ws_bytes = workspace_bytes;
  c->capture_on = false;
  c->tok_embed = w->tok_embed;
  c->g_final = w->g_final;
  c->w_lm_head = w->w_lm_head;
  c->w_qkv.assign(w->w_qkv, w->w_qkv + c->L);
  c->w_o.assign(w->w_o, w->w_o + c->L);
  c->w_gate.assign(w->w_gate, w->w_gate + c->L);
  c->w_up.assign(w->w_up, w->w_up + c->L);
  c->w_down.assign(w->w_down, w->w_down + c->L);
  c->g_attn.assign(w->g_attn, w->g_attn + c->L);
  c->g_mlp.assign(w->g_mlp, w->g_mlp + c->L);
  c->have_prefill = false;
  c->maps_built = false;
  c->n_seqs = 0;
  memset(&c->stats, 0, sizeof(c->stats));
  if (!dev_status_ptr()) {
    delete c;
    return LAZY_E_CUDA;
  }
  rc = launch_rope_table(0, c->rope_table, c->max_pos, c->dh, cfg->rope_theta);
  // the GEMMs' arrival counters start at zero and return to zero after every launch
  if (rc == LAZY_OK && c->gemm_scratch &&
      cudaMemsetAsync(c->gemm_scratch, 0, c->gemm_scratch_bytes, 0) != cudaSuccess)
    rc = LAZY_E_CUDA;
  if (rc == LAZY_OK && cudaStreamSynchronize(0) != cudaSuccess) rc = LAZY_E_CUDA;
  if (rc != LAZY_OK) {
    delete c;
    return rc;
  }
  *out = c;
  return LAZY_OK;
}

int32_t lazy_keep_count(int32_t n_total, uint32_t keep_bp, int32_t n_present) {
  if (n_total < 1 || keep_bp < 1 || keep_bp > 10000 || n_present < 1) return 0;
  return keep_count(n_total, keep_bp, n_present);
}

int lazy_set_fp8_weights(lazy_ctx *c, const lazy_fp8_weights *w) {
  if (!c) return LAZY_E_BADARG;
  if (!w) {
    c->fp8_on = false;
    return LAZY_OK;
  }
  if (c->dtype != LAZY_BF16 || c->d % 16 || c->F % 16) return LAZY_E_BADARG;
  if (!w->w_qkv || !w->w_o || !w->w_gate || !w->w_up || !w->w_down || !w->s_qkv || !w->s_o || !w->s_gate ||
      !w->s_up || !w->s_down)
    return LAZY_E_BADARG;
  for (int l = 0; l < c->L; ++l) {
    const void *ps[5] = {w->w_qkv[l], w->w_o[l], w->w_gate[l], w->w_up[l], w->w_down[l]};
    for (const void *p : ps)
      if (!p || ((uintptr_t)p & 15)) return LAZY_E_BADARG;
    const float ss[5] = {w->s_qkv[l], w->s_o[l], w->s_gate[l], w->s_up[l], w->s_down[l]};
    for (float s : ss)
      if (!(s > 0.f)) return LAZY_E_BADARG;
  }
  c->w8_qkv.assign(w->w_qkv, w->w_qkv + c->L);
  c->w8_o.assign(w->w_o, w->w_o + c->L);
  c->w8_gate.assign(w->w_gate, w->w_gate + c->L);
  c->w8_up.assign(w->w_up, w->w_up + c->L);
  c->w8_down.assign(w->w_down, w->w_down + c->L);
  c->s8_qkv.assign(w->s_qkv, w->s_qkv + c->L);
  c->s8_o.assign(w->s_o, w->s_o + c->L);
  c->s8_gate.assign(w->s_gate, w->s_gate + c->L);
  c->s8_up.assign(w->s_up, w->s_up + c->L);
  c->s8_down.assign(w->s_down, w->s_down + c->L);
  c->fp8_on = true;
  return LAZY_OK;
}

int lazy_set_selection(lazy_ctx *c, int32_t mode) {
  if (!c || (mode != 0 && mode != 1)) return LAZY_E_BADARG;
  c->select_threshold = mode == 1;
  return LAZY_OK;
}

int lazy_set_aux_point(lazy_ctx *c, int32_t after_layer) {
  if (!c || (after_layer != 0 && after_layer != 1)) return LAZY_E_BADARG;
  if (c->aux_after_layer != (after_layer != 0)) {
    c->aux_after_layer = after_layer != 0;
    c->have_prefill = false;  // caches filled under the other reading cannot be decoded from
  }
  return LAZY_OK;
}

void lazy_destroy(lazy_ctx *ctx) { delete ctx; }

const char *lazy_strerror(int status) {
  switch (status) {
    case LAZY_OK: return "ok";
    case LAZY_E_BADARG: return "bad argument";
    case LAZY_E_BADSCHEDULE: return "bad keep schedule";
    case LAZY_E_CAPACITY: return "capacity exceeded";
    case LAZY_E_NOT_IN_AUX: return "position not held by the Aux Cache";
    case LAZY_E_TIMEOUT: return "bounded device-side wait ran out";
    case LAZY_E_CUDA: return "CUDA call failed";
    case LAZY_E_STATE: return "call out of order";
    default: return "unknown status";
  }
}

int lazy_set_debug_capture(lazy_ctx *c, int32_t on) {
  if (!c) return LAZY_E_BADARG;
  if (on && !c->capture_sized) return LAZY_E_CAPACITY;
  c->capture_on = on != 0;
  return LAZY_OK;
}

int lazy_set_forced_keep(lazy_ctx *c, int32_t layer_entered, int32_t seq, const int32_t *d_pos,
                         int32_t n) {
  if (!c || layer_entered < 0 || layer_entered > c->L || seq < 0 || seq >= c->S || n < 0)
    return LAZY_E_BADARG;
  const int p = c->point_at[layer_entered];
  if (p < 0) return LAZY_E_BADARG;
  if (n == 0) {
    c->forced.erase(std::make_pair(p, (int)seq));
    return LAZY_OK;
  }
  if (!d_pos) return LAZY_E_BADARG;
  c->forced[std::make_pair(p, (int)seq)] = std::make_pair(d_pos, (int)n);
  return LAZY_OK;
}

// ---------------------------------------------------------------------------------------- prefill
int lazy_prefill_run(lazy_ctx *c, void *stream, const int32_t *d_prompt_ids,
                     const int32_t *h_cu_seqlens, int32_t n_seqs, float *d_logits) {
  if (!c || !d_prompt_ids || !h_cu_seqlens || !d_logits || n_seqs < 1) return LAZY_E_BADARG;
  if (n_seqs > c->S) return LAZY_E_CAPACITY;
  if (h_cu_seqlens[0] != 0) return LAZY_E_BADARG;
  for (int s = 0; s < n_seqs; ++s)
    if (h_cu_seqlens[s + 1] <= h_cu_seqlens[s]) return LAZY_E_BADARG;  // empty prompts not allowed
  const int N = h_cu_seqlens[n_seqs];
  if (N > c->cap_rows) return LAZY_E_CAPACITY;
  cudaStream_t st = (cudaStream_t)stream;
  DevStatus *status = dev_status_ptr();
  if (!status) return LAZY_E_CUDA;
  const long long launches0 = g_launches;
  const int P = c->P, L = c->L, d = c->d, dt = c->dtype;
  const int dkv = c->dkv, qc = c->qkv_cols;
  const size_t rb = c->row_bytes(), kvb = c->kv_row_bytes();
  LAZY_TRY(reset_gemm_counters(c, st));
  c->ev_kind.clear();
  c->ev_flops.clear();
  c->ev_bytes.clear();
  for (int i = 0; i < LAZY_N_KERNEL_KINDS; ++i) c->k_flops[i] = c->k_bytes[i] = 0.0;

  // ---- host bookkeeping: every row count follows from the lengths and the schedule
  c->have_prefill = false;
  c->maps_built = false;
  c->n_seqs = n_seqs;
  c->prompt_len.resize(n_seqs);
  c->n_tokens.resize(n_seqs);
  c->seq_base.resize(n_seqs);
  int max_len = 0;
  for (int s = 0; s < n_seqs; ++s) {
    c->prompt_len[s] = h_cu_seqlens[s + 1] - h_cu_seqlens[s];
    c->n_tokens[s] = c->prompt_len[s];
    c->seq_base[s] = h_cu_seqlens[s] + s * c->cfg.max_new_tokens;
    if (c->prompt_len[s] > max_len) max_len = c->prompt_len[s];
    if (c->prompt_len[s] + c->cfg.max_new_tokens > c->max_pos) return LAZY_E_CAPACITY;
  }
  c->seg_cu.assign(P + 1, std::vector<int>(n_seqs + 1, 0));
  for (int s = 0; s <= n_seqs; ++s) c->seg_cu[0][s] = h_cu_seqlens[s];
  std::vector<std::vector<int>> cu_drop(P, std::vector<int>(n_seqs + 1, 0));
  // Rows kept at points p_from.. from the rows present at p_from (count form: the scheduled count; under the
  // threshold reading these are the counts before ties, corrected point by point once the scores exist).
  auto plan_from = [&](int p_from) -> int {
    for (int p = p_from; p < P; ++p) {
      for (int s = 0; s < n_seqs; ++s) {
        const int present = c->seg_cu[p][s + 1] - c->seg_cu[p][s];
        int keep = keep_count(c->prompt_len[s], c->sched_bp[p], present);
        auto it = c->forced.find(std::make_pair(p, s));
        if (it != c->forced.end()) {
          keep = it->second.second;
          if (keep < 1 || keep > present) return LAZY_E_BADARG;
        }
        c->seg_cu[p + 1][s + 1] = c->seg_cu[p + 1][s] + keep;
        cu_drop[p][s + 1] = cu_drop[p][s] + (present - keep);
      }
    }
    return LAZY_OK;
  };
  LAZY_TRY(plan_from(0));
  c->kv_count.assign(L, std::vector<int>(n_seqs, 0));
  c->aux_count.assign(P, std::vector<int>(n_seqs, 0));
  c->aux_live.assign(P, std::vector<int>(n_seqs, 0));
  c->dec_revived_cu.assign(P, std::vector<int>(n_seqs + 1, 0));
  c->last_was_decode = false;
  memset(&c->stats, 0, sizeof(c->stats));
  c->stats.n_layers = L;

  // ---- integer tables to the device: segment cu arrays, drop cu arrays, bases, last rows
  const int W = c->S + 1;
  std::vector<int32_t> ints((size_t)(2 * P + 8) * W, 0);
  auto tab = [&](int i) { return ints.data() + (size_t)i * W; };
  auto d_cu = [&](int g) { return c->d_ints + (size_t)g * W; };
  auto d_cu_drop = [&](int p) { return c->d_ints + (size_t)(P + 1 + p) * W; };
  const int32_t *d_base = c->d_ints + (size_t)(2 * P + 1) * W;
  const int32_t *d_last = c->d_ints + (size_t)(2 * P + 2) * W;
  // Uploads the tables and rebuilds the cache-row lists of segments g_from.. and the Aux-row lists of
  // points p_from.. (everything, at the start of a run; the tail, after a cut whose count was read back).
  auto upload_tables = [&](int g_from, int p_from) -> int {
    for (int g = 0; g <= P; ++g)
      for (int s = 0; s <= n_seqs; ++s) tab(g)[s] = c->seg_cu[g][s];
    for (int p = 0; p < P; ++p)
      for (int s = 0; s <= n_seqs; ++s) tab(P + 1 + p)[s] = cu_drop[p][s];
    for (int s = 0; s < n_seqs; ++s) {
      tab(2 * P + 1)[s] = c->seq_base[s];
      tab(2 * P + 2)[s] = c->seg_cu[P][s + 1] - 1;  // last row of the sequence in the final segment
    }
    LAZY_CUDA_OK(cudaMemcpyAsync(c->d_ints, ints.data(), ints.size() * 4, cudaMemcpyHostToDevice, st));
    for (int g = g_from; g <= P; ++g)
      LAZY_TRY(launch_seg_rows(st, d_cu(g), d_base, n_seqs, c->seg_cu[g][n_seqs], c->kv_row[g]));
    for (int p = p_from; p < P; ++p)
      LAZY_TRY(launch_seg_rows(st, d_cu_drop(p), d_base, n_seqs, cu_drop[p][n_seqs], c->aux_dst[p]));
    return LAZY_OK;
  };
  LAZY_TRY(upload_tables(0, 0));

  // ---- embedding, positions
  TIMED(LAZY_K_EMBED, 0, 2.0 * N * rb, launch_embed(st, dt, c->tok_embed, d_prompt_ids, c->x, N, d, c->V, status));
  LAZY_TRY(launch_iota_pos(st, c->pos_seg[0], d_cu(0), n_seqs, N));

  char *x = c->x, *x2 = c->x2;
  int g = 0;
  int score_pending = 0;  // first layer whose Eq. 1 head mean has not been taken yet (tensor-core attention path)
  for (int l = 0; l < L; ++l) {
    const int n = c->seg_cu[g][n_seqs];
    const int32_t *pos = c->pos_seg[g];
    char *kc = c->kcache + (size_t)l * c->cap_kv * kvb;
    char *vc = c->vcache + (size_t)l * c->cap_kv * kvb;
    int32_t *kvp = c->kv_pos + (size_t)l * c->cap_kv;
    float *sc = c->scores + (size_t)l * c->cap_kv;
    int seg_max = 0;
    for (int s = 0; s < n_seqs; ++s) {
      const int ns = c->seg_cu[g][s + 1] - c->seg_cu[g][s];
      c->kv_count[l][s] = ns;
      if (ns > seg_max) seg_max = ns;
    }
    c->stats.rows_computed[l] = n;
    c->stats.kv_rows[l] = n;

    double attn_flops = 0.0;
    for (int s = 0; s < n_seqs; ++s) {
      const double ns = c->seg_cu[g][s + 1] - c->seg_cu[g][s];
      attn_flops += 2.0 * d * ns * (ns + 1.0);
    }
    TIMED(LAZY_K_RMSNORM, 0, 2.0 * n * rb, launch_rmsnorm(st, dt, x, c->g_attn[l], c->h, n, d, c->cfg.rms_eps));
    // 8-bit projections: the activation is quantised per row into the staging buffer, then multiplied as
    // e4m3 codes (products of up to four rows stay on the 16-bit weight-streaming kernel)
    const bool f8 = c->fp8_on && dt == LAZY_BF16 && n > 4;
    auto quant = [&](const void *src, int rows, int width) -> int {
      return launch_quant_rows_e4m3(st, src, c->a8, c->a8_scale, rows, width);
    };
    if (f8) {
      TIMED(LAZY_K_OTHER, 0, 3.0 * n * d, quant(c->h, n, d));
      RopeArgs r = {};
      const bool fused = gemm_qkv_rope_eligible(dt, d, c->dh, dkv);
      if (fused) {
        r.pos = pos;
        r.table = (const float2 *)c->rope_table;
        r.kcache = (bf16 *)kc;
        r.kv_rows = c->cap_kv;
        r.vcache = (bf16 *)vc;
        r.kv_pos = kvp;
        r.kv_row = c->kv_row[g];
        r.d_model = d;
        r.max_pos = c->max_pos;
        r.d_kv = dkv;
      }
      TIMED(LAZY_K_GEMM_QKV, 2.0 * n * qc * d, 0,
            launch_gemm_fp8(st, fused ? EPI_QKV_ROPE : EPI_PLAIN, c->a8, c->a8_scale, c->w8_qkv[l], c->s8_qkv[l], nullptr,
                            1.f, nullptr, c->qkv, n, qc, d, status, r, c->gemm_scratch, c->gemm_scratch_bytes));
      if (!fused)
        TIMED(LAZY_K_ROPE_KV, 0, 6.0 * n * rb,
              launch_rope_kv(st, dt, c->qkv, pos, c->rope_table, kc, vc, kvp, c->kv_row[g], n, c->H, c->dh,
                             c->max_pos, status, c->Hkv));
    } else if (gemm_qkv_rope_eligible(dt, d, c->dh, dkv)) {
      // rotary embedding and the K/V cache write ride in the projection's epilogue
      TIMED(LAZY_K_GEMM_QKV, 2.0 * n * qc * d, 0,
            launch_gemm_qkv_rope(st, c->h, c->w_qkv[l], c->qkv, pos, c->rope_table, kc, vc, kvp, c->kv_row[g], n,
                                 d, c->max_pos, status, c->gemm_scratch, c->gemm_scratch_bytes, dkv, c->cap_kv));
    } else {
      TIMED(LAZY_K_GEMM_QKV, 2.0 * n * qc * d, 0,
            launch_gemm(st, dt, c->h, c->w_qkv[l], nullptr, c->qkv, n, qc, d, status, c->gemm_scratch,
                        c->gemm_scratch_bytes));
      TIMED(LAZY_K_ROPE_KV, 0, 6.0 * n * rb,
            launch_rope_kv(st, dt, c->qkv, pos, c->rope_table, kc, vc, kvp, c->kv_row[g], n, c->H, c->dh,
                           c->max_pos, status, c->Hkv));
    }
    bool fused_score = false;
    if (attention_tc_eligible(dt, c->dh, qc, dkv)) {
      // Eq. 1 comes from the last row's softmax numerators, which the attention kernel leaves in this layer's
      // slice of the score scratch; the head means of all layers since the previous cut are taken in one
      // launch when the next cut (or the end of the prefill) needs them.
      // One attention launch per sequence: its tensor maps end at the sequence's last row, so rows beyond it
      // read as zeros instead of whatever the cache region holds.
      for (int s = 0; s < n_seqs; ++s) {
        const int q0 = c->seg_cu[g][s], ns = c->seg_cu[g][s + 1] - q0;
        const double fl = 2.0 * d * (double)ns * (ns + 1.0);
        TIMED(LAZY_K_ATTENTION, fl, 0,
              launch_attention_tc(st, c->qkv, qc, q0 + ns, kc, vc, dkv, c->seq_base[s] + ns, c->attn, c->H,
                                  nullptr, nullptr, 1, ns, q0, ns, c->seq_base[s], status,
                                  c->score_scratch + (size_t)l * c->score_layer_stride, cdiv(seg_max, 64), n_seqs, s,
                                  c->Hkv));
      }
      fused_score = true;
      const bool last_of_group = c->point_at[l + 1] >= 0 || l == L - 1;
      if (last_of_group) {  // layers score_pending..l ran on the same rows (segment g)
        const int nl = l - score_pending + 1;
        TIMED(LAZY_K_SCORE, 0, nl * (4.0 * c->H * n + 4.0 * n),
              launch_score_from_attention(st, c->score_scratch + (size_t)score_pending * c->score_layer_stride,
                                          c->score_layer_stride, nl, d_cu(g), n_seqs, n, c->H, cdiv(seg_max, 64),
                                          c->scores + (size_t)score_pending * c->cap_kv, (size_t)c->cap_kv));
        score_pending = l + 1;
      }
    } else {
      TIMED(LAZY_K_ATTENTION, attn_flops, 0,
            launch_attention(st, dt, c->qkv, qc, kc, vc, dkv, c->attn, d_cu(g), d_base, n_seqs, seg_max, n,
                             c->H, c->dh, c->Hkv));
    }
    if (!fused_score)
      TIMED(LAZY_K_SCORE, 0, (double)n * rb + 4.0 * n,
            launch_score(st, dt, c->qkv, qc, kc, dkv, d_cu(g), d_base, n_seqs, n, seg_max, c->H, c->dh,
                         c->score_scratch, sc, c->Hkv));
    if (f8) {
      TIMED(LAZY_K_OTHER, 0, 3.0 * n * d, quant(c->attn, n, d));
      TIMED(LAZY_K_GEMM_O, 2.0 * n * d * d, 0,
            launch_gemm_fp8(st, EPI_RESIDUAL, c->a8, c->a8_scale, c->w8_o[l], c->s8_o[l], nullptr, 1.f, x, x, n, d, d,
                            status, RopeArgs(), c->gemm_scratch, c->gemm_scratch_bytes));
    } else {
      TIMED(LAZY_K_GEMM_O, 2.0 * n * d * d, 0, launch_gemm(st, dt, c->attn, c->w_o[l], x, x, n, d, d, status,
                                                        c->gemm_scratch, c->gemm_scratch_bytes, 0, true));
    }

    const int p = c->point_at[l + 1];
    // Rows of the residual stream that survive a cut made in this layer, when they are still where they
    // were (x is then compacted on the way through the MLP instead of by a copy of its own): the MLP's
    // RMSNorm reads x[keep[r]], and the down projection adds x[keep[r]] and writes row r of the other buffer.
    const int32_t *via_keep = nullptr;
    // The layer's MLP, on the rows of the current segment.
    auto run_mlp = [&]() -> int {
      const int n2 = c->seg_cu[g][n_seqs];
      TIMED(LAZY_K_RMSNORM, 0, 2.0 * n2 * rb,
            launch_rmsnorm_rows(st, dt, x, via_keep, c->g_mlp[l], c->h, n2, d, c->cfg.rms_eps));
      if (c->fp8_on && dt == LAZY_BF16 && n2 > 4) {
        TIMED(LAZY_K_OTHER, 0, 3.0 * n2 * d, quant(c->h, n2, d));
        TIMED(LAZY_K_GEMM_GATE_UP, 4.0 * n2 * c->F * d, 0,
              launch_gemm_fp8(st, EPI_SWIGLU, c->a8, c->a8_scale, c->w8_gate[l], c->s8_gate[l], c->w8_up[l], c->s8_up[l],
                              nullptr, c->act, n2, c->F, d, status, RopeArgs(), c->gemm_scratch, c->gemm_scratch_bytes));
        TIMED(LAZY_K_OTHER, 0, 3.0 * n2 * c->F, quant(c->act, n2, c->F));
        RopeArgs rr = {};
        rr.res_rows = via_keep;
        TIMED(LAZY_K_GEMM_DOWN, 2.0 * n2 * d * c->F, 0,
              launch_gemm_fp8(st, EPI_RESIDUAL, c->a8, c->a8_scale, c->w8_down[l], c->s8_down[l], nullptr, 1.f, x,
                              via_keep ? x2 : x, n2, d, c->F, status, rr, c->gemm_scratch, c->gemm_scratch_bytes));
      } else {
        TIMED(LAZY_K_GEMM_GATE_UP, 4.0 * n2 * c->F * d, 0,
              launch_gemm_swiglu(st, dt, c->h, c->w_gate[l], c->w_up[l], c->act, n2, c->F, d, status, c->gemm_scratch,
                                 c->gemm_scratch_bytes, 0, true));
        TIMED(LAZY_K_GEMM_DOWN, 2.0 * n2 * d * c->F, 0,
              launch_gemm(st, dt, c->act, c->w_down[l], x, via_keep ? x2 : x, n2, d, c->F, status, c->gemm_scratch,
                          c->gemm_scratch_bytes, 0, true, via_keep));
      }
      if (via_keep) {
        char *t = x; x = x2; x2 = t;
        via_keep = nullptr;
      }
      return LAZY_OK;
    };
    // Default: the cut sits between attention and MLP, so the MLP of this layer already runs on the kept
    // rows.  With aux_after_layer the MLP runs on every row first and the Aux Cache receives layer outputs.
    const bool cut_after = p >= 0 && c->aux_after_layer;
    if (cut_after) LAZY_TRY(run_mlp());
    if (p >= 0) {
      const float *sel = sc;
      bool any_forced = false;
      for (int s = 0; s < n_seqs; ++s)
        if (c->forced.count(std::make_pair(p, s))) any_forced = true;
      if (any_forced) {
        LAZY_CUDA_OK(cudaMemcpyAsync(c->sel_scores, sc, (size_t)n * 4, cudaMemcpyDeviceToDevice, st));
        for (int s = 0; s < n_seqs; ++s) {
          auto it = c->forced.find(std::make_pair(p, s));
          if (it == c->forced.end()) continue;
          LAZY_TRY(launch_forced_scores(st, pos, c->seg_cu[g][s], c->seg_cu[g][s + 1] - c->seg_cu[g][s],
                                        it->second.first, it->second.second, c->sel_scores));
        }
        sel = c->sel_scores;
      }
      if (c->select_threshold) {
        // Threshold reading: a row is pruned iff its score is smaller than the score at the scheduled rank, so
        // ties at that rank all survive and the count depends on the data.  One count per sequence is read
        // back here (a stream synchronisation per cut); every later row count is re-planned from it.
        std::vector<int32_t> h_counts((size_t)n_seqs, 0);
        LAZY_TRY(launch_select_tie_count(st, sel, d_cu(g), d_cu(g + 1), n_seqs, c->d_found, status));
        LAZY_CUDA_OK(cudaMemcpyAsync(h_counts.data(), c->d_found, (size_t)n_seqs * 4, cudaMemcpyDeviceToHost, st));
        LAZY_CUDA_OK(cudaStreamSynchronize(st));
        bool changed = false;
        for (int s = 0; s < n_seqs; ++s) {
          const int present = c->seg_cu[g][s + 1] - c->seg_cu[g][s];
          const int keep = h_counts[s];
          if (keep < 1 || keep > present) return LAZY_E_STATE;
          if (keep != c->seg_cu[g + 1][s + 1] - c->seg_cu[g + 1][s]) changed = true;
          c->seg_cu[g + 1][s + 1] = c->seg_cu[g + 1][s] + keep;
          cu_drop[p][s + 1] = cu_drop[p][s] + (present - keep);
        }
        if (changed) {
          LAZY_TRY(plan_from(p + 1));
          LAZY_TRY(upload_tables(g + 1, p));
        }
      }
      const int n_keep = c->seg_cu[g + 1][n_seqs], n_drop = n - n_keep;
      char *ar = c->aux_rows + (size_t)p * c->cap_kv * rb;
      int32_t *ap = c->aux_pos + (size_t)p * c->cap_kv;
      // the selection also writes the position lists of the next segment and of the Aux Cache
      TIMED(LAZY_K_SELECT, 0, 8.0 * n + 8.0 * n,
            launch_select(st, sel, d_cu(g), d_cu(g + 1), n_seqs, c->keep_idx[p], c->drop_idx[p], status, pos,
                          c->pos_seg[g + 1], c->aux_dst[p], ap));
      // pruned rows to the Aux Cache (the one copy the method itself asks for)
      TIMED(LAZY_K_COMPACT, 0, 2.0 * n_drop * rb,
            launch_move_rows(st, x, c->drop_idx[p], ar, c->aux_dst[p], n_drop, (int)rb, n, c->cap_kv, status));
      if (!cut_after && gemm_res_rows_supported(dt, n_keep, c->F)) {
        via_keep = c->keep_idx[p];  // kept rows are gathered on load by the MLP that follows
      } else {
        TIMED(LAZY_K_COMPACT, 0, 2.0 * n_keep * rb,
              launch_move_rows(st, x, c->keep_idx[p], x2, nullptr, n_keep, (int)rb, n, c->cap_rows, status));
        char *t = x; x = x2; x2 = t;
      }
      for (int s = 0; s < n_seqs; ++s)
        c->aux_count[p][s] = c->aux_live[p][s] = cu_drop[p][s + 1] - cu_drop[p][s];
      c->stats.aux_rows[l] = n_drop;
      ++g;
    }
    if (!cut_after) LAZY_TRY(run_mlp());
    const int n2 = c->seg_cu[g][n_seqs];
    if (c->capture_on && c->capture)
      LAZY_CUDA_OK(cudaMemcpyAsync(c->capture + (size_t)l * c->cap_rows * rb, x, (size_t)n2 * rb,
                                   cudaMemcpyDeviceToDevice, st));
  }
  // ---- first-token logits from the last row of every sequence
  TIMED(LAZY_K_RMSNORM, 0, 2.0 * n_seqs * rb,
        launch_rmsnorm_rows(st, dt, x, d_last, c->g_final, c->h_last, n_seqs, d, c->cfg.rms_eps));
  TIMED(LAZY_K_LM_HEAD, 0, (double)c->V * rb,
        launch_lm_head(st, dt, c->h_last, c->w_lm_head, d_logits, n_seqs, d, c->V, true));
  // the residual stream may live in either ping-pong buffer; decode does not need it
  c->forced.clear();
  c->have_prefill = true;
  c->stats.kernel_launches = g_launches - launches0;
  return LAZY_OK;
}

// ---------------------------------------------------------------------------------------- Aux read
int aux_cache_revive(lazy_ctx *c, void *stream, int32_t layer, int32_t seq, const int32_t *d_positions,
                     int32_t n, void *d_hidden_out) {
  if (!c || layer < 0 || layer + 1 > c->L || seq < 0 || n < 0 || (n > 0 && (!d_positions || !d_hidden_out)))
    return LAZY_E_BADARG;
  if (!c->have_prefill) return LAZY_E_STATE;
  if (seq >= c->n_seqs) return LAZY_E_BADARG;
  const int p = c->point_at[layer + 1];
  if (p < 0) return n == 0 ? LAZY_OK : LAZY_E_NOT_IN_AUX;  // no Aux Cache follows this layer
  if (n > c->cap_kv) return LAZY_E_CAPACITY;
  cudaStream_t st = (cudaStream_t)stream;
  DevStatus *status = dev_status_ptr();
  if (!status) return LAZY_E_CUDA;
  if (n == 0) return LAZY_OK;
  const size_t rb = c->row_bytes();
  const int32_t *ap = c->aux_pos + (size_t)p * c->cap_kv;
  const char *ar = c->aux_rows + (size_t)p * c->cap_kv * rb;
  // a pending device error of an earlier call must not be mistaken for a miss of this one
  int rc = sync_and_take_status(st, nullptr);
  if (rc != LAZY_OK) return rc;
  aux_find_kernel<<<n, 128, 0, st>>>(ap, c->seq_base[seq], c->aux_count[p][seq], d_positions, n,
                                     c->d_found, status);
  LAZY_COUNT_LAUNCH();
  LAZY_TRY(launch_ok());
  // rows of found positions are copied; misses (index -1) are skipped and reported
  LAZY_TRY(launch_move_rows(st, ar, c->d_found, d_hidden_out, nullptr, n, (int)rb, c->cap_kv, n, status));
  rc = sync_and_take_status(st, nullptr);
  if (rc == LAZY_E_BADARG) rc = LAZY_E_NOT_IN_AUX;
  return rc;
}

int lazy_decode_step(lazy_ctx *c, void *stream, const int32_t *d_new_ids, float *d_logits,
                     int32_t *d_next_ids) {
  if (!c || !d_new_ids || !d_logits) return LAZY_E_BADARG;
  if (!c->have_prefill) return LAZY_E_STATE;
  LAZY_TRY(reset_gemm_counters(c, (cudaStream_t)stream));
  return decode_step_impl(c, (cudaStream_t)stream, d_new_ids, d_logits, d_next_ids);
}

// ---------------------------------------------------------------------------------------- introspection
int lazy_get_kept(lazy_ctx *c, void *stream, int32_t layer_entered, int32_t seq, int32_t *d_pos,
                  int32_t *h_count) {
  if (!c || layer_entered < 0 || layer_entered > c->L || seq < 0) return LAZY_E_BADARG;
  if (!c->have_prefill) return LAZY_E_STATE;
  if (seq >= c->n_seqs) return LAZY_E_BADARG;
  const int p = c->point_at[layer_entered];
  if (p < 0) return LAZY_E_BADARG;
  const int a = c->seg_cu[p + 1][seq], b = c->seg_cu[p + 1][seq + 1];
  if (h_count) *h_count = b - a;
  cudaStream_t st = (cudaStream_t)stream;
  if (d_pos)
    LAZY_CUDA_OK(cudaMemcpyAsync(d_pos, c->pos_seg[p + 1] + a, (size_t)(b - a) * 4, cudaMemcpyDeviceToDevice, st));
  LAZY_CUDA_OK(cudaStreamSynchronize(st));
  return LAZY_OK;
}

int lazy_get_scores(lazy_ctx *c, void *stream, int32_t layer, int32_t seq, float *d_scores,
                    int32_t *h_count) {
  if (!c || layer < 0 || layer >= c->L || seq < 0) return LAZY_E_BADARG;
  if (!c->have_prefill) return LAZY_E_STATE;
  if (seq >= c->n_seqs) return LAZY_E_BADARG;
  const int g = c->seg_of_layer(layer);
  const int a = c->seg_cu[g][seq], b = c->seg_cu[g][seq + 1];
  if (h_count) *h_count = b - a;
  cudaStream_t st = (cudaStream_t)stream;
  if (d_scores)
    LAZY_CUDA_OK(cudaMemcpyAsync(d_scores, c->scores + (size_t)layer * c->cap_kv + a, (size_t)(b - a) * 4,
                                 cudaMemcpyDeviceToDevice, st));
  LAZY_CUDA_OK(cudaStreamSynchronize(st));
  return LAZY_OK;
}

int lazy_get_hidden(lazy_ctx *c, void *stream, int32_t layer, void *d_out, int32_t *h_rows) {
  if (!c || layer < 0 || layer >= c->L) return LAZY_E_BADARG;
  if (!c->have_prefill || !c->capture_on || !c->capture) return LAZY_E_STATE;
  int g = c->seg_of_layer(layer);
  if (c->point_at[layer + 1] >= 0) g += 1;  // the layer's MLP already ran on the kept rows
  const int rows = c->seg_cu[g][c->n_seqs];
  if (h_rows) *h_rows = rows;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t rb = c->row_bytes();
  if (d_out)
    LAZY_CUDA_OK(cudaMemcpyAsync(d_out, c->capture + (size_t)layer * c->cap_rows * rb, (size_t)rows * rb,
                                 cudaMemcpyDeviceToDevice, st));
  LAZY_CUDA_OK(cudaStreamSynchronize(st));
  return LAZY_OK;
}

int lazy_get_kv(lazy_ctx *c, void *stream, int32_t layer, int32_t seq, int32_t *d_pos, void *d_k,
                void *d_v, int32_t *h_count) {
  if (!c || layer < 0 || layer >= c->L || seq < 0) return LAZY_E_BADARG;
  if (!c->have_prefill) return LAZY_E_STATE;
  if (seq >= c->n_seqs) return LAZY_E_BADARG;
  const int cnt = c->kv_count[layer][seq];
  const size_t rb = c->kv_row_bytes();  // K / V rows: n_kv_heads * head_dim wide
  const size_t row0 = (size_t)layer * c->cap_kv + c->seq_base[seq];
  if (h_count) *h_count = cnt;
  cudaStream_t st = (cudaStream_t)stream;
  if (d_pos) LAZY_CUDA_OK(cudaMemcpyAsync(d_pos, c->kv_pos + row0, (size_t)cnt * 4, cudaMemcpyDeviceToDevice, st));
  if (d_k) LAZY_CUDA_OK(cudaMemcpyAsync(d_k, c->kcache + row0 * rb, (size_t)cnt * rb, cudaMemcpyDeviceToDevice, st));
  if (d_v) LAZY_CUDA_OK(cudaMemcpyAsync(d_v, c->vcache + row0 * rb, (size_t)cnt * rb, cudaMemcpyDeviceToDevice, st));
  LAZY_CUDA_OK(cudaStreamSynchronize(st));
  return LAZY_OK;
}

// Live entries of a region of position tags (tag >= 0), as global rows, uploaded to d_list.
static int live_rows(lazy_ctx *c, cudaStream_t st, const int32_t *tags, int row0, int count,
                     int32_t *d_list, int *n_live, bool want_tag_value, std::vector<int32_t> *vals) {
  std::vector<int32_t> h((size_t)count);
  if (count) {
    LAZY_CUDA_OK(cudaMemcpyAsync(h.data(), tags + row0, (size_t)count * 4, cudaMemcpyDeviceToHost, st));
    LAZY_CUDA_OK(cudaStreamSynchronize(st));
  }
  std::vector<int32_t> rows;
  for (int i = 0; i < count; ++i)
    if (h[i] >= 0) {
      rows.push_back(row0 + i);
      if (want_tag_value && vals) vals->push_back(h[i]);
    }
  *n_live = (int)rows.size();
  if (d_list && !rows.empty()) {
    LAZY_CUDA_OK(cudaMemcpyAsync(d_list, rows.data(), rows.size() * 4, cudaMemcpyHostToDevice, st));
    LAZY_CUDA_OK(cudaStreamSynchronize(st));
  }
  (void)c;
  return LAZY_OK;
}

int lazy_get_aux(lazy_ctx *c, void *stream, int32_t layer, int32_t seq, int32_t *d_pos, void *d_hidden,
                 int32_t *h_count) {
  if (!c || layer < 0 || layer >= c->L || seq < 0) return LAZY_E_BADARG;
  if (!c->have_prefill) return LAZY_E_STATE;
  if (seq >= c->n_seqs) return LAZY_E_BADARG;
  const int p = c->point_at[layer + 1];
  if (p < 0) {
    if (h_count) *h_count = 0;
    return LAZY_OK;
  }
  cudaStream_t st = (cudaStream_t)stream;
  DevStatus *status = dev_status_ptr();
  if (!status) return LAZY_E_CUDA;
  const size_t rb = c->row_bytes();
  const int32_t *ap = c->aux_pos + (size_t)p * c->cap_kv;
  int n_live = 0;
  // entries revived during decode stay in place with tag -1: hand out the live ones only
  LAZY_TRY(live_rows(c, st, ap, c->seq_base[seq], c->aux_count[p][seq], c->d_found, &n_live, false, nullptr));
  if (h_count) *h_count = n_live;
  if (d_pos) LAZY_TRY(launch_move_i32(st, ap, c->d_found, d_pos, nullptr, n_live));
  if (d_hidden)
    LAZY_TRY(launch_move_rows(st, c->aux_rows + (size_t)p * c->cap_kv * rb, c->d_found, d_hidden, nullptr,
                              n_live, (int)rb, c->cap_kv, n_live > 0 ? n_live : 1, status));
  LAZY_CUDA_OK(cudaStreamSynchronize(st));
  return LAZY_OK;
}

int lazy_get_revived(lazy_ctx *c, void *stream, int32_t layer_entered, int32_t seq, int32_t *d_pos,
                     int32_t *h_count) {
  if (!c || layer_entered < 0 || layer_entered > c->L || seq < 0) return LAZY_E_BADARG;
  if (!c->have_prefill) return LAZY_E_STATE;
  if (seq >= c->n_seqs) return LAZY_E_BADARG;
  const int p = c->point_at[layer_entered];
  if (p < 0) return LAZY_E_BADARG;
  if (!c->last_was_decode) {  // prefill revives nothing
    if (h_count) *h_count = 0;
    return LAZY_OK;
  }
  cudaStream_t st = (cudaStream_t)stream;
  const int a = c->dec_revived_cu[p][seq], b = c->dec_revived_cu[p][seq + 1];
  std::vector<int32_t> vals;
  int n_live = 0;
  LAZY_TRY(live_rows(c, st, c->revived_pos[p], a, b - a, nullptr, &n_live, true, &vals));
  if (h_count) *h_count = n_live;
  if (d_pos && n_live) {
    LAZY_CUDA_OK(cudaMemcpyAsync(d_pos, vals.data(), vals.size() * 4, cudaMemcpyHostToDevice, st));
    LAZY_CUDA_OK(cudaStreamSynchronize(st));
  }
  return LAZY_OK;
}

int lazy_get_stats(lazy_ctx *c, lazy_stats *out) {
  if (!c || !out) return LAZY_E_BADARG;
  *out = c->stats;
  return LAZY_OK;
}

int lazy_set_kernel_timing(lazy_ctx *c, int32_t on) {
  if (!c) return LAZY_E_BADARG;
  c->timing_on = on != 0;
  c->timing_mask = on == 1 ? 0xffffffffu : (uint32_t)on >> 1;  // 1 = every kind, else (kind bits << 1)
  if (on) {  // create the events now so that the timed run itself creates none
    while (c->ev_pool.size() < 2048) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return LAZY_E_CUDA;
      c->ev_pool.push_back(e);
    }
  }
  return LAZY_OK;
}

int lazy_get_kernel_times(lazy_ctx *c, void *stream, lazy_kernel_times *out) {
  if (!c || !out) return LAZY_E_BADARG;
  LAZY_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
  memset(out, 0, sizeof(*out));
  for (size_t i = 0; i < c->ev_kind.size(); ++i) {
    float ms = 0.f;
    LAZY_CUDA_OK(cudaEventElapsedTime(&ms, c->ev_pool[2 * i], c->ev_pool[2 * i + 1]));
    out->ms[c->ev_kind[i]] += ms;
    out->launches[c->ev_kind[i]] += 1;
  }
  for (int k = 0; k < LAZY_N_KERNEL_KINDS; ++k) {
    out->flops[k] = c->k_flops[k];
    out->bytes[k] = c->k_bytes[k];
  }
  return LAZY_OK;
}

int lazy_get_kernel_events(lazy_ctx *c, void *stream, int32_t cap, int32_t *kinds, float *ms, double *flops,
                           double *bytes, int32_t *count) {
  if (!c || !count || cap < 0 || (cap > 0 && (!kinds || !ms || !flops || !bytes))) return LAZY_E_BADARG;
  LAZY_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
  *count = (int32_t)c->ev_kind.size();
  for (size_t i = 0; i < c->ev_kind.size() && (int32_t)i < cap; ++i) {
    float t = 0.f;
    LAZY_CUDA_OK(cudaEventElapsedTime(&t, c->ev_pool[2 * i], c->ev_pool[2 * i + 1]));
    kinds[i] = c->ev_kind[i];
    ms[i] = t;
    flops[i] = c->ev_flops[i];
    bytes[i] = c->ev_bytes[i];
  }
  return LAZY_OK;
}

int lazy_sync_status(lazy_ctx *c, void *stream) {
  if (!c) return LAZY_E_BADARG;
  return sync_and_take_status((cudaStream_t)stream, nullptr);
}
int lazy_device_status(void *stream) { return sync_and_take_status((cudaStream_t)stream, nullptr); }

}  // extern "C"
