// Host-side context of one generation state: shapes, weight pointers, the carved workspace and
// the bookkeeping that prefill leaves for decode.  No device memory is owned here.
#pragma once

#include <map>
#include <utility>
#include <vector>

#include "common.cuh"

struct lazy_ctx {
  lazy_model_cfg cfg;
  int L, d, H, dh, F, V, dtype, eb;
  int Hkv, dkv, qkv_cols;  // key/value heads, width of a K / V cache row, width of a row of the fused projection
  int P;  // schedule points
  std::vector<int> sched_layer;
  std::vector<uint32_t> sched_bp;
  std::vector<int> point_at;  // [L+1]: index of the schedule point entering that layer, or -1

  const void *tok_embed, *g_final, *w_lm_head;
  std::vector<const void *> w_qkv, w_o, w_gate, w_up, w_down, g_attn, g_mlp;

  // capacities
  int cap_rows;  // activation rows (packed prompt tokens; decode in-flight rows)
  int cap_kv;    // rows of every per-layer cache: prompt tokens + max_seqs * max_new_tokens
  int max_pos;   // positions per sequence the RoPE table covers
  int S;         // max_seqs

  // workspace carve-up (device)
  char *ws_base;
  size_t ws_bytes;
  char *x, *x2, *h, *qkv, *attn, *act, *h_last;
  std::vector<int32_t *> pos_seg;  // [P+1] positions of the rows of each segment
  float *scores;                   // [L, cap_rows]
  float *sel_scores;               // [cap_rows] scores handed to the selection when a set is forced
  float *score_scratch;
  size_t score_layer_stride;  // floats per layer of the attention kernels' score by-product
  std::vector<int32_t *> keep_idx, drop_idx;  // [P] x [cap_rows]
  std::vector<int32_t *> aux_dst;             // [P] x [cap_rows] Aux row of the i-th dropped row
  std::vector<int32_t *> kv_row;              // [P+1] x [cap_rows] cache row of packed row r
  float *rope_table;
  char *kcache, *vcache;  // [L, cap_kv, d]
  int32_t *kv_pos;        // [L, cap_kv]
  char *aux_rows;         // [P, cap_kv, d]
  int32_t *aux_pos;       // [P, cap_kv]
  int32_t *d_ints;        // small integer tables uploaded per call (cu arrays, bases, last rows)
  int32_t *d_found;       // [cap_rows] scratch for Aux lookups
  char *capture;          // [L, cap_rows, d] or NULL
  // decode-only buffers
  int32_t *kv_map;   // [L, cap_kv]: cache row of (sequence base + position), -1 if absent
  int32_t *aux_map;  // [P, cap_kv]: Aux row of (sequence base + position), -1 if absent
  std::vector<int32_t *> revived_pos;  // [P] x [cap_kv]: per in-flight row after a boundary, its
                                       // position if it came from the Aux Cache, else -1
  int32_t *dec_seg;  // [2][L][cap_kv]: per layer of a decode segment, the cache rows appended to and the context's rows
  size_t score_scratch_cap;  // floats in score_scratch
  int32_t *dec_i32;  // integer scratch of the decode step
  float *dec_f32;
  bool select_threshold = false;  // threshold reading of the selection: ties at the scheduled rank all survive
  bool aux_after_layer = false;  // cut after the whole scoring layer (Aux rows = layer output) instead of before its MLP
  // 8-bit projections: codes and scales per layer (empty = off), staging for the quantised activations
  std::vector<const void *> w8_qkv, w8_o, w8_gate, w8_up, w8_down;
  std::vector<float> s8_qkv, s8_o, s8_gate, s8_up, s8_down;
  bool fp8_on = false;
  uint8_t *a8;       // [cap_rows, max(d, F)] e4m3 codes of the activation entering a projection
  float *a8_scale;   // [cap_rows]
  void *gemm_scratch;  // split-wave partials and counters of the tensor-core GEMMs (bf16 only)
  size_t gemm_scratch_bytes;

  bool capture_on, capture_sized;

  // ---- state of the latest call (host)
  bool have_prefill;
  bool maps_built;
  int n_seqs;
  std::vector<int> prompt_len;             // [n_seqs]
  std::vector<int> n_tokens;               // [n_seqs] tokens so far (prompt + generated)
  std::vector<int> seq_base;               // [n_seqs] first cache row of the sequence's region
  std::vector<std::vector<int>> seg_cu;    // [P+1][n_seqs+1] packed row offsets per segment
  std::vector<std::vector<int>> kv_count;  // [L][n_seqs]
  std::vector<std::vector<int>> aux_count; // [P][n_seqs] rows appended (retired entries included)
  std::vector<std::vector<int>> aux_live;  // [P][n_seqs] entries currently held
  std::vector<std::vector<int>> dec_revived_cu;  // [P][n_seqs+1] in-flight rows after each boundary
  int dec_tag = 0;                         // tag of the latest selection mark
  bool last_was_decode = false;
  std::map<std::pair<int, int>, std::pair<const int32_t *, int>> forced;  // (point, seq) -> list
  lazy_stats stats;

  // ---- optional per-kernel event timing
  bool timing_on = false;
  uint32_t timing_mask = 0xffffffffu;  // kinds that get an event pair
  std::vector<cudaEvent_t> ev_pool;  // pairs: 2*i start, 2*i+1 stop
  std::vector<int> ev_kind;          // kind of each used pair
  std::vector<double> ev_flops, ev_bytes;  // algorithmic work of the launch each pair brackets
  double k_flops[LAZY_N_KERNEL_KINDS], k_bytes[LAZY_N_KERNEL_KINDS];
  // Returns the index of a fresh event pair (or -1) after recording its start.
  int time_begin(cudaStream_t st, int kind, double flops, double bytes);
  void time_end(cudaStream_t st, int slot);
  ~lazy_ctx();

  size_t row_bytes() const { return (size_t)d * eb; }
  size_t kv_row_bytes() const { return (size_t)dkv * eb; }
  int seg_of_layer(int l) const {  // segment whose rows enter layer l
    int g = 0;
    for (int p = 0; p < P; ++p)
      if (sched_layer[p] <= l) g = p + 1;
    return g;
  }
};

namespace lazy {

int validate_cfg(const lazy_model_cfg *cfg);
int validate_schedule(const lazy_model_cfg *cfg, const lazy_schedule *s);
inline int keep_count(long long n_total, long long bp, int n_present) {
  long long c = (n_total * bp + 9999) / 10000;
  if (c > n_present) c = n_present;
  if (c < 1) c = 1;
  return (int)c;
}

// rows moved with optional source and destination index lists
int launch_move_rows(cudaStream_t st, const void *src, const int32_t *src_idx, void *dst,
                     const int32_t *dst_idx, int n, int row_bytes, int src_rows, int dst_rows,
                     DevStatus *status);
int launch_move_i32(cudaStream_t st, const int32_t *src, const int32_t *src_idx, int32_t *dst,
                    const int32_t *dst_idx, int n);
// out[r] = base[s] + (r - cu[s]) for the sequence s owning packed row r
int launch_seg_rows(cudaStream_t st, const int32_t *cu, const int32_t *base, int n_seqs, int n_total,
                    int32_t *out);

int decode_step_impl(lazy_ctx *c, cudaStream_t st, const int32_t *d_new_ids, float *d_logits,
                     int32_t *d_next_ids);

}  // namespace lazy
