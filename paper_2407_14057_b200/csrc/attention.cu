// Causal attention over the rows that survive at a layer (packed sequences).
//
//  * attn_mma_kernel: bf16, head_dim 128.  Flash-style streaming softmax; 64 query rows per CTA
//    (4 warps x 16 rows), 64-key tiles of K and V double-buffered in shared memory with
//    cp.async 16-byte copies into an XOR-swizzled layout, ldmatrix + mma.sync m16n8k16 with fp32
//    accumulation, softmax statistics kept per row in registers with quad shuffles.
//  * attn_rowwarp_kernel: any storage type / head_dim (fp32 mode, small models): one warp per
//    (query row, head), one key per lane, streaming softmax with warp shuffles.
// The causal mask is by row order inside a sequence: rows are kept in ascending position order,
// so row order and position order coincide.
#include <stdlib.h>

#include "common.cuh"

namespace lazy {

namespace {

// ------------------------------------------------------------------------------------------------
// generic kernel
template <typename T>
__global__ void attn_rowwarp_kernel(const T *__restrict__ q, int ldq, const T *__restrict__ k,
                                    const T *__restrict__ v, int ldkv, T *__restrict__ o,
                                    const int32_t *__restrict__ cu_q,
                                    const int32_t *__restrict__ kv_base,
                                    const int32_t *__restrict__ cu_kv,
                                    const int32_t *__restrict__ kv_idx,
                                    const int32_t *__restrict__ q_kvlen, int n_seqs, int n_total,
                                    int n_heads, int head_dim, int kv_group) {
  extern __shared__ float qs_all[];  // [warps][head_dim]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = blockIdx.x * (blockDim.x >> 5) + warp;
  const int h = blockIdx.y;
  const int hk = h / kv_group;  // key/value head of this query head
  if (r >= n_total) return;
  int lo = 0, hi = n_seqs;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (cu_q[mid] <= r) lo = mid; else hi = mid;
  }
  // keys visible to this row: the first `vis` entries of the sequence's key list
  const int vis = q_kvlen ? q_kvlen[r] : r - cu_q[lo] + 1;
  const int i = vis - 1;
  const size_t kbase = kv_base ? (size_t)kv_base[lo] : (size_t)cu_q[lo];
  const int32_t *kidx = kv_idx ? kv_idx + cu_kv[lo] : nullptr;
  float *qs = qs_all + warp * head_dim;
  const float scale = rsqrtf((float)head_dim);
  for (int t = lane; t < head_dim; t += 32)
    qs[t] = Elem<T>::to_f(q[(size_t)r * ldq + h * head_dim + t]) * scale;
  __syncwarp();
  const int per_lane = head_dim / 32;  // output dims owned by a lane: lane + 32*t
  float acc[8];
#pragma unroll
  for (int t = 0; t < 8; ++t) acc[t] = 0.f;
  float m = -INFINITY, l = 0.f;
  for (int j0 = 0; j0 <= i; j0 += 32) {
    const int j = j0 + lane;
    float s = -INFINITY;
    if (j <= i) {
      const T *kr = k + (kidx ? (size_t)kidx[j] : kbase + j) * ldkv + hk * head_dim;
      float dot = 0.f;
      for (int t = 0; t < head_dim; ++t) dot += qs[t] * Elem<T>::to_f(kr[t]);
      s = dot;
    }
    const float m_new = fmaxf(m, warp_max(s));
    const float p = (j <= i) ? __expf(s - m_new) : 0.f;
    const float corr = __expf(m - m_new);
    l = l * corr + warp_sum(p);
    m = m_new;
#pragma unroll
    for (int t = 0; t < 8; ++t) acc[t] *= corr;
    const int cnt = min(32, i - j0 + 1);
    for (int jj = 0; jj < cnt; ++jj) {
      const float pj = __shfl_sync(0xffffffffu, p, jj);
      const T *vr = v + (kidx ? (size_t)kidx[j0 + jj] : kbase + j0 + jj) * ldkv + hk * head_dim;
#pragma unroll
      for (int t = 0; t < 8; ++t)
        if (t < per_lane) acc[t] += pj * Elem<T>::to_f(vr[lane + 32 * t]);
    }
  }
  const float inv = 1.f / l;
#pragma unroll
  for (int t = 0; t < 8; ++t)
    if (t < per_lane)
      o[(size_t)r * (n_heads * head_dim) + h * head_dim + lane + 32 * t] = Elem<T>::from_f(acc[t] * inv);
}

// ------------------------------------------------------------------------------------------------
// tensor-core kernel (bf16, head_dim = 128)
constexpr int FA_BM = 64, FA_BN = 64, FA_D = 128, FA_THREADS = 128;
constexpr int FA_ROW_BYTES = FA_D * 2;                    // 256 B = 16 chunks of 16 B
constexpr int FA_TILE_BYTES = FA_BN * FA_ROW_BYTES;       // 16 KiB
constexpr int FA_SMEM_BYTES = FA_TILE_BYTES * 5;          // Q + 2 x (K, V)

__device__ __forceinline__ uint32_t smem_addr(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
// byte offset of 16-byte chunk `c` of row `r` in a swizzled [rows][128] bf16 tile
__device__ __forceinline__ uint32_t sw_off(int r, int c) {
  return (uint32_t)(r * FA_ROW_BYTES + ((c ^ (r & 7)) << 4));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float *c, const uint32_t *a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Copies 64 rows x 256 B (one head's slice) into a swizzled tile.  Rows past `n_valid` re-read the
// last valid row so that shared memory never holds uninitialised (possibly non-finite) data.
// With `idx`, list entry j names the cache row to read (decode: keys picked by position).
__device__ __forceinline__ void load_tile(uint32_t tile, const bf16 *base, int ld, int row0, int n_valid,
                                          const int32_t *idx = nullptr) {
  for (int t = threadIdx.x; t < FA_BN * 16; t += FA_THREADS) {
    const int r = t >> 4, c = t & 15;
    int gr = row0 + r;
    if (gr > n_valid - 1) gr = n_valid - 1;
    const size_t src = idx ? (size_t)idx[gr] : (size_t)gr;
    cp_async16(tile + sw_off(r, c), base + src * ld + c * 8);
  }
}

__global__ void __launch_bounds__(FA_THREADS)
attn_mma_kernel(const bf16 *__restrict__ q, int ldq, const bf16 *__restrict__ k,
                const bf16 *__restrict__ v, int ldkv, bf16 *__restrict__ o,
                const int32_t *__restrict__ cu_q, const int32_t *__restrict__ kv_base,
                const int32_t *__restrict__ cu_kv, const int32_t *__restrict__ kv_idx,
                const int32_t *__restrict__ q_kvlen, int n_heads, int n_splits,
                float *__restrict__ part_o, float *__restrict__ part_ml, int kv_group) {
  extern __shared__ __align__(128) uint8_t fa_smem[];
  const int seq = blockIdx.z, h = blockIdx.y;
  const int q_start = cu_q[seq];
  const int n = cu_q[seq + 1] - q_start;
  const int q_tiles = (n + FA_BM - 1) / FA_BM;
  // n_splits > 1 (few query rows, long key lists: decode with revived rows): blockIdx.x also names a
  // slice of the key tiles; the CTA then leaves an unnormalised partial result per row for a merge kernel
  const int split = (int)blockIdx.x % n_splits, bx = (int)blockIdx.x / n_splits;
  if (bx >= q_tiles) return;
  const int qt = q_tiles - 1 - bx;  // longest rows first
  const int q0 = qt * FA_BM;
  // keys: either the sequence's contiguous cache rows, or the rows a list names (decode)
  const int32_t *kidx = kv_idx ? kv_idx + cu_kv[seq] : nullptr;
  const int n_kv = kv_idx ? cu_kv[seq + 1] - cu_kv[seq] : n;
  const size_t kb = kv_idx ? 0 : (kv_base ? (size_t)kv_base[seq] : (size_t)q_start);
  const bf16 *qg = q + (size_t)q_start * ldq + h * FA_D;
  const bf16 *kg = k + kb * ldkv + (h / kv_group) * FA_D;
  const bf16 *vg = v + kb * ldkv + (h / kv_group) * FA_D;

  const uint32_t sQ = smem_addr(fa_smem);
  const uint32_t sK = sQ + FA_TILE_BYTES;       // two buffers
  const uint32_t sV = sK + 2 * FA_TILE_BYTES;   // two buffers
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t4 = lane & 3;

  // Row i sees the first vis(i) keys; vis is non-decreasing in i (prefill: i + 1).
  const int last_row = min(q0 + FA_BM, n) - 1;
  const int vis_tile = q_kvlen ? min(q_kvlen[q_start + last_row], n_kv) : last_row + 1;
  const int n_kt_all = (vis_tile + FA_BN - 1) / FA_BN;  // key tiles up to the diagonal
  const int tiles_per_split = ((n_kv + FA_BN - 1) / FA_BN + n_splits - 1) / n_splits;
  const int kt0 = split * tiles_per_split;
  const int n_kt = min(n_kt_all, kt0 + tiles_per_split);  // this CTA walks key tiles [kt0, n_kt)
  if (kt0 >= n_kt) {  // nothing visible in this slice: empty partials (n_splits > 1 only)
    for (int r = threadIdx.x; r < FA_BM; r += FA_THREADS) {
      if (q0 + r < n) {
        const size_t pidx = ((size_t)(q_start + q0 + r) * n_heads + h) * n_splits + split;
        part_ml[pidx * 2] = -INFINITY;
        part_ml[pidx * 2 + 1] = 0.f;
      }
    }
    return;
  }
  const int wrow0 = min(q0 + warp * 16 + g, n - 1), wrow1 = min(q0 + warp * 16 + g + 8, n - 1);
  const int vis0 = q_kvlen ? q_kvlen[q_start + wrow0] : wrow0 + 1;
  const int vis1 = q_kvlen ? q_kvlen[q_start + wrow1] : wrow1 + 1;
  const int wfirst = min(q0 + warp * 16, n - 1);
  const int vis_first = q_kvlen ? q_kvlen[q_start + wfirst] : wfirst + 1;
  load_tile(sQ, qg, ldq, q0, n);
  load_tile(sK, kg, ldkv, kt0 * FA_BN, n_kv, kidx);
  load_tile(sV, vg, ldkv, kt0 * FA_BN, n_kv, kidx);
  cp_async_commit();

  uint32_t qf[8][4];
  float oacc[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) { oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  const float sl2 = rsqrtf((float)FA_D) * 1.4426950408889634f;  // softmax scale in log2 units

  for (int kt = kt0; kt < n_kt; ++kt) {
    const int buf = (kt - kt0) & 1;
    if (kt + 1 < n_kt) {  // prefetch the next K/V tile into the other buffer
      load_tile(sK + (buf ^ 1) * FA_TILE_BYTES, kg, ldkv, (kt + 1) * FA_BN, n_kv, kidx);
      load_tile(sV + (buf ^ 1) * FA_TILE_BYTES, vg, ldkv, (kt + 1) * FA_BN, n_kv, kidx);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    if (kt == kt0) {
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const int r = warp * 16 + (lane & 15);
        const int c = ks * 2 + (lane >> 4);
        ldsm_x4(sQ + sw_off(r, c), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
      }
    }
    const uint32_t kbuf = sK + buf * FA_TILE_BYTES, vbuf = sV + buf * FA_TILE_BYTES;
    float s[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        const int r = np * 16 + (lane & 7) + ((lane >> 4) << 3);
        const int c = ks * 2 + ((lane >> 3) & 1);
        uint32_t b0, b1, b2, b3;
        ldsm_x4(kbuf + sw_off(r, c), b0, b1, b2, b3);
        mma_bf16(s[2 * np], qf[ks], b0, b1);
        mma_bf16(s[2 * np + 1], qf[ks], b2, b3);
      }
    }
    // scale, causal mask (key index >= keys visible to the row), running max
    const int kcol0 = kt * FA_BN + 2 * t4;
    const bool diag = (kt + 1) * FA_BN > vis_first;  // tile may cross this warp's diagonal
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float val = s[i][e] * sl2;
        if (diag) {
          const int col = kcol0 + i * 8 + (e & 1);
          if (col >= ((e >> 1) ? vis1 : vis0)) val = -INFINITY;
        }
        s[i][e] = val;
        mx[e >> 1] = fmaxf(mx[e >> 1], val);
      }
    }
    float corr[2];
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      mx[rr] = fmaxf(mx[rr], __shfl_xor_sync(0xffffffffu, mx[rr], 1));
      mx[rr] = fmaxf(mx[rr], __shfl_xor_sync(0xffffffffu, mx[rr], 2));
      // finite from the first tile on when the walk starts at key 0 (visible to every row); a later slice
      // may show a row nothing yet: then everything stays zero and no exponent sees inf - inf
      const float m_new = fmaxf(m_run[rr], mx[rr]);
      corr[rr] = m_new == -INFINITY ? 1.f : exp2f(m_run[rr] - m_new);
      m_run[rr] = m_new;
    }
    const float mref[2] = {m_run[0] == -INFINITY ? 0.f : m_run[0], m_run[1] == -INFINITY ? 0.f : m_run[1]};
    float rs[2] = {0.f, 0.f};
    uint32_t pf[4][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float p0 = exp2f(s[i][0] - mref[0]), p1 = exp2f(s[i][1] - mref[0]);
      const float p2 = exp2f(s[i][2] - mref[1]), p3 = exp2f(s[i][3] - mref[1]);
      rs[0] += p0 + p1;
      rs[1] += p2 + p3;
      pf[i >> 1][(i & 1) * 2 + 0] = bf16x2_pack(p0, p1);
      pf[i >> 1][(i & 1) * 2 + 1] = bf16x2_pack(p2, p3);
    }
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) l_run[rr] = l_run[rr] * corr[rr] + rs[rr];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      oacc[i][0] *= corr[0];
      oacc[i][1] *= corr[0];
      oacc[i][2] *= corr[1];
      oacc[i][3] *= corr[1];
    }
#pragma unroll
    for (int kc = 0; kc < 4; ++kc) {
#pragma unroll
      for (int dp = 0; dp < 8; ++dp) {
        const int r = kc * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
        const int c = dp * 2 + (lane >> 4);
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(vbuf + sw_off(r, c), b0, b1, b2, b3);
        mma_bf16(oacc[2 * dp], pf[kc], b0, b1);
        mma_bf16(oacc[2 * dp + 1], pf[kc], b2, b3);
      }
    }
    __syncthreads();  // everyone is done with `buf` before the next prefetch overwrites it
  }

#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    l_run[rr] += __shfl_xor_sync(0xffffffffu, l_run[rr], 1);
    l_run[rr] += __shfl_xor_sync(0xffffffffu, l_run[rr], 2);
  }
  if (n_splits > 1) {  // unnormalised partials: [row, head, split] x (128 fp32 | max in log2 units, sum)
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int row = q0 + warp * 16 + g + rr * 8;
      if (row < n) {
        const size_t pidx = ((size_t)(q_start + row) * n_heads + h) * n_splits + split;
        float *po = part_o + pidx * FA_D + 2 * t4;
#pragma unroll
        for (int i = 0; i < 16; ++i)
          *reinterpret_cast<float2 *>(po + i * 8) = make_float2(oacc[i][rr * 2], oacc[i][rr * 2 + 1]);
        if (t4 == 0) {
          part_ml[pidx * 2] = m_run[rr];
          part_ml[pidx * 2 + 1] = l_run[rr];
        }
      }
    }
    return;
  }
  const int ldo = n_heads * FA_D;
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    const int row = q0 + warp * 16 + g + rr * 8;
    if (row < n) {
      const float inv = 1.f / l_run[rr];
      bf16 *orow = o + (size_t)(q_start + row) * ldo + h * FA_D + 2 * t4;
#pragma unroll
      for (int i = 0; i < 16; ++i)
        *reinterpret_cast<uint32_t *>(orow + i * 8) =
            bf16x2_pack(oacc[i][rr * 2] * inv, oacc[i][rr * 2 + 1] * inv);
    }
  }
}

}  // namespace

bool attention_tc_eligible(int dtype, int head_dim, int ldq, int ldkv) {
  return dtype == LAZY_BF16 && head_dim == 128 && (ldq % 8) == 0 && (ldkv % 8) == 0;
}

int launch_attention(cudaStream_t st, int dtype, const void *q, int ldq, const void *k,
                     const void *v, int ldkv, void *o, const int32_t *cu_q, const int32_t *kv_base,
                     int n_seqs, int max_len, int n_total, int n_heads, int head_dim, int n_kv_heads) {
  return launch_attention_ex(st, dtype, q, ldq, k, v, ldkv, o, cu_q, kv_base, nullptr, nullptr, nullptr,
                             n_seqs, max_len, n_total, n_heads, head_dim, n_kv_heads);
}

bool attention_list_split_eligible(int dtype, int head_dim) { return dtype == LAZY_BF16 && head_dim == FA_D; }

// Splits of the key list that put ~4 CTAs on every SM for n_rows query rows (1 = do not split).
int attention_list_splits(int n_seqs, int max_rows, int n_heads, int max_ctx) {
  const int ctas = cdiv(max_rows, FA_BM) * n_heads * n_seqs;
  int s = (4 * sm_count()) / (ctas > 0 ? ctas : 1);
  const int key_tiles = cdiv(max_ctx, FA_BN);
  if (s > key_tiles / 4) s = key_tiles / 4;  // at least four key tiles per slice
  if (s > 8) s = 8;
  return s < 2 ? 1 : s;
}

// Key-list attention (decode with many rows in flight) with the key tiles of every (query tile, head) cut
// into n_splits slices; part: n_total * n_heads * n_splits * 130 floats.  The merge kernel of the
// split-key decode attention finishes the rows (and leaves the score row's softmax statistics in stats).
int launch_attention_list_split(cudaStream_t st, const void *q, int ldq, const void *k, const void *v, int ldkv,
                                void *o, const int32_t *cu_q, const int32_t *cu_kv, const int32_t *kv_idx,
                                const int32_t *q_kvlen, const int32_t *score_row, int n_seqs, int max_rows,
                                int n_total, int n_heads, int n_splits, float *part, float *stats, int n_kv_heads) {
  if (n_total == 0 || n_seqs == 0) return LAZY_OK;
  const int kv_group = kv_group_of(n_heads, n_kv_heads);
  if (kv_group < 1) return LAZY_E_BADARG;
  if (!part || !stats || !score_row || n_splits < 2 || (ldq % 8) || (ldkv % 8)) return LAZY_E_BADARG;
  static bool attr_set = false;
  if (!attr_set) {
    LAZY_CUDA_OK(cudaFuncSetAttribute(attn_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FA_SMEM_BYTES));
    attr_set = true;
  }
  float *part_o = part;
  float *part_ml = part + (size_t)n_total * n_heads * n_splits * FA_D;
  dim3 grid(cdiv(max_rows, FA_BM) * n_splits, n_heads, n_seqs);
  attn_mma_kernel<<<grid, FA_THREADS, FA_SMEM_BYTES, st>>>((const bf16 *)q, ldq, (const bf16 *)k, (const bf16 *)v,
                                                           ldkv, (bf16 *)o, cu_q, nullptr, cu_kv, kv_idx, q_kvlen,
                                                           n_heads, n_splits, part_o, part_ml, kv_group);
  LAZY_COUNT_LAUNCH();
  if (launch_ok() != LAZY_OK) return LAZY_E_CUDA;
  return launch_attention_combine(st, part_o, part_ml, n_splits, cu_q, score_row, n_seqs, n_total, n_heads, o,
                                  n_heads * FA_D, stats);
}

int launch_attention_ex(cudaStream_t st, int dtype, const void *q, int ldq, const void *k,
                        const void *v, int ldkv, void *o, const int32_t *cu_q, const int32_t *kv_base,
                        const int32_t *cu_kv, const int32_t *kv_idx, const int32_t *q_kvlen, int n_seqs,
                        int max_len, int n_total, int n_heads, int head_dim, int n_kv_heads) {
  if (n_total == 0 || n_seqs == 0) return LAZY_OK;
  const int kv_group = kv_group_of(n_heads, n_kv_heads);
  if (kv_group < 1) return LAZY_E_BADARG;
  if (dtype == LAZY_BF16 && head_dim == FA_D && (ldq % 8) == 0 && (ldkv % 8) == 0) {
    static bool attr_set = false;
    if (!attr_set) {
      LAZY_CUDA_OK(cudaFuncSetAttribute(attn_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        FA_SMEM_BYTES));
      attr_set = true;
    }
    dim3 grid(cdiv(max_len, FA_BM), n_heads, n_seqs);
    attn_mma_kernel<<<grid, FA_THREADS, FA_SMEM_BYTES, st>>>((const bf16 *)q, ldq, (const bf16 *)k,
                                                             (const bf16 *)v, ldkv, (bf16 *)o, cu_q,
                                                             kv_base, cu_kv, kv_idx, q_kvlen, n_heads, 1, nullptr,
                                                             nullptr, kv_group);
    LAZY_COUNT_LAUNCH();
    return launch_ok();
  }
  if (head_dim % 32 || head_dim > 256) return LAZY_E_BADARG;
  const int warps = 4;
  dim3 grid(cdiv(n_total, warps), n_heads);
  size_t smem = (size_t)warps * head_dim * sizeof(float);
  if (dtype == LAZY_F32)
    attn_rowwarp_kernel<float><<<grid, warps * 32, smem, st>>>((const float *)q, ldq, (const float *)k,
                                                              (const float *)v, ldkv, (float *)o, cu_q,
                                                              kv_base, cu_kv, kv_idx, q_kvlen, n_seqs, n_total,
                                                              n_heads, head_dim, kv_group);
  else
    attn_rowwarp_kernel<bf16><<<grid, warps * 32, smem, st>>>((const bf16 *)q, ldq, (const bf16 *)k,
                                                             (const bf16 *)v, ldkv, (bf16 *)o, cu_q,
                                                             kv_base, cu_kv, kv_idx, q_kvlen, n_seqs, n_total,
                                                             n_heads, head_dim, kv_group);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

}  // namespace lazy
