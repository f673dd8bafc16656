// HBM-bound steps of the path: embedding gather, RMSNorm, RoPE + KV-cache write, row gathers,
// the LM head on the last rows, greedy argmax.
// All rows are moved with 16-byte vector accesses; reductions use warp shuffles.
#include "common.cuh"

namespace lazy {

long long g_launches = 0;

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  }
  return n;
}

// ---- status word ------------------------------------------------------------------------------
__device__ DevStatus g_dev_status;

DevStatus *dev_status_ptr() {
  static DevStatus *ptrs[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!ptrs[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_dev_status) != cudaSuccess) return nullptr;
    if (cudaMemset(p, 0, sizeof(DevStatus)) != cudaSuccess) return nullptr;
    ptrs[dev] = static_cast<DevStatus *>(p);
  }
  return ptrs[dev];
}

static DevStatus g_last_bad_status = {0, 0, 0, 0};
void last_status_detail(int *where, int *a, int *b) {
  if (where) *where = g_last_bad_status.where;
  if (a) *a = g_last_bad_status.a;
  if (b) *b = g_last_bad_status.b;
}

int sync_and_take_status(cudaStream_t stream, int *where_out) {
  DevStatus *p = dev_status_ptr();
  if (!p) return LAZY_E_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return LAZY_E_CUDA;
  DevStatus h;
  if (cudaMemcpy(&h, p, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return LAZY_E_CUDA;
  if (h.code != 0) {
    g_last_bad_status = h;
    if (cudaMemset(p, 0, sizeof(DevStatus)) != cudaSuccess) return LAZY_E_CUDA;
  }
  if (where_out) *where_out = h.where;
  return h.code;
}

// ---- small fills ------------------------------------------------------------------------------
__global__ void fill_i32_kernel(int32_t *p, int32_t v, size_t n) {
  size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
  size_t stride = (size_t)gridDim.x * blockDim.x;
  for (; i < n; i += stride) p[i] = v;
}
int launch_fill_i32(cudaStream_t st, int32_t *p, int32_t v, size_t n) {
  if (n == 0) return LAZY_OK;
  size_t blocks = (n + 255) / 256;
  if (blocks > (size_t)sm_count() * 8) blocks = (size_t)sm_count() * 8;
  fill_i32_kernel<<<(int)blocks, 256, 0, st>>>(p, v, n);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

// pos[r] = r - cu[s] for the sequence s that owns packed row r.
__global__ void iota_pos_kernel(int32_t *pos, const int32_t *cu, int n_seqs, int n_total) {
  int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= n_total) return;
  int lo = 0, hi = n_seqs;  // largest s with cu[s] <= r
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (cu[mid] <= r) lo = mid; else hi = mid;
  }
  pos[r] = r - cu[lo];
}
int launch_iota_pos(cudaStream_t st, int32_t *pos, const int32_t *cu, int n_seqs, int n_total) {
  if (n_total == 0) return LAZY_OK;
  iota_pos_kernel<<<cdiv(n_total, 256), 256, 0, st>>>(pos, cu, n_seqs, n_total);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

// ---- embedding gather ---------------------------------------------------------------------------
template <typename T>
__global__ void embed_kernel(const T *__restrict__ table, const int32_t *__restrict__ ids,
                             T *__restrict__ x, int d, int vocab, DevStatus *status) {
  const int r = blockIdx.x;
  int id = ids[r];
  const bool bad = (id < 0 || id >= vocab);
  if (bad) {
    if (threadIdx.x == 0) dev_fail(status, LAZY_E_BADARG, W_EMBED_ID, r, id);
    id = 0;
  }
  const int nvec = d / Elem<T>::kPerVec;
  const uint4 *src = reinterpret_cast<const uint4 *>(table + (size_t)id * d);
  uint4 *dst = reinterpret_cast<uint4 *>(x + (size_t)r * d);
  for (int i = threadIdx.x; i < nvec; i += blockDim.x) dst[i] = bad ? make_uint4(0, 0, 0, 0) : src[i];
}

int launch_embed(cudaStream_t st, int dtype, const void *table, const int32_t *ids, void *x, int n,
                 int d, int vocab, DevStatus *status) {
  if (n == 0) return LAZY_OK;
  if (dtype == LAZY_F32)
    embed_kernel<float><<<n, 128, 0, st>>>((const float *)table, ids, (float *)x, d, vocab, status);
  else
    embed_kernel<bf16><<<n, 128, 0, st>>>((const bf16 *)table, ids, (bf16 *)x, d, vocab, status);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

// ---- RMSNorm --------------------------------------------------------------------------------------
// One CTA per row.  fp32 sum of squares, warp shuffles + one smem exchange.
template <typename T, int THREADS>
__global__ void rmsnorm_kernel(const T *__restrict__ x, const int32_t *__restrict__ row_idx,
                               const T *__restrict__ g, T *__restrict__ y, int d, float eps) {
  constexpr int V = Elem<T>::kPerVec;
  const int r = blockIdx.x;
  const size_t src_row = row_idx ? (size_t)row_idx[r] : (size_t)r;
  const T *xr = x + src_row * d;
  T *yr = y + (size_t)r * d;
  const int nvec = d / V;
  float ss = 0.f;
  for (int i = threadIdx.x; i < nvec; i += THREADS) {
    Vec16<T> v;
    v.load(xr + i * V);
    float f[V];
    v.unpack(f);
#pragma unroll
    for (int j = 0; j < V; ++j) ss += f[j] * f[j];
  }
  __shared__ float part[THREADS / 32];
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < THREADS / 32; ++w) tot += part[w];
  const float scale = rsqrtf(tot / (float)d + eps);
  for (int i = threadIdx.x; i < nvec; i += THREADS) {
    Vec16<T> v, gv, o;
    v.load(xr + i * V);
    gv.load(g + i * V);
    float f[V], gf[V];
    v.unpack(f);
    gv.unpack(gf);
#pragma unroll
    for (int j = 0; j < V; ++j) f[j] = f[j] * scale * gf[j];
    o.pack(f);
    o.store(yr + i * V);
  }
}

// One WARP per row, the row held in registers between the sum of squares and the scaling: x is read
// once (VPL 16-byte vectors per lane, all requested before the first is used), no shared memory, no
// block barrier.  Rows of VPL * 32 vectors exactly (d = 4096 in bf16: VPL = 16).
template <typename T, int VPL>
__global__ void __launch_bounds__(256)
rmsnorm_warp_kernel(const T *__restrict__ x, const int32_t *__restrict__ row_idx, const T *__restrict__ g,
                    T *__restrict__ y, int n, int d, float eps) {
  constexpr int V = Elem<T>::kPerVec;
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= n) return;
  const size_t src_row = row_idx ? (size_t)row_idx[r] : (size_t)r;
  const uint4 *xr = reinterpret_cast<const uint4 *>(x + src_row * d);
  uint4 *yr = reinterpret_cast<uint4 *>(y + (size_t)r * d);
  const uint4 *gr = reinterpret_cast<const uint4 *>(g);
  Vec16<T> v[VPL];
#pragma unroll
  for (int u = 0; u < VPL; ++u) v[u].raw = xr[lane + 32 * u];
  float ss = 0.f;
#pragma unroll
  for (int u = 0; u < VPL; ++u) {
    float f[V];
    v[u].unpack(f);
#pragma unroll
    for (int j = 0; j < V; ++j) ss += f[j] * f[j];
  }
  ss = warp_sum(ss);
  const float scale = rsqrtf(ss / (float)d + eps);
  // Only the packed row stays in registers across the reduction: the values are unpacked again below
  // (the empty asm keeps the compiler from carrying the unpacked copy along, which costs occupancy).
#pragma unroll
  for (int u = 0; u < VPL; ++u)
    asm volatile("" : "+r"(v[u].raw.x), "+r"(v[u].raw.y), "+r"(v[u].raw.z), "+r"(v[u].raw.w));
#pragma unroll
  for (int u = 0; u < VPL; ++u) {
    Vec16<T> gv, o;
    gv.raw = gr[lane + 32 * u];
    float f[V], gf[V];
    v[u].unpack(f);
    gv.unpack(gf);
#pragma unroll
    for (int j = 0; j < V; ++j) f[j] = f[j] * scale * gf[j];
    o.pack(f);
    yr[lane + 32 * u] = o.raw;
  }
}

template <typename T>
static bool launch_rmsnorm_warp(cudaStream_t st, const T *x, const int32_t *row_idx, const T *g, T *y, int n, int d,
                                float eps) {
  const int nvec = d / Elem<T>::kPerVec;
  if (nvec % 32) return false;
  const int blocks = cdiv(n, 8);
  switch (nvec / 32) {
#define RW_CASE(v)                                                                                    \
  case v:                                                                                             \
    rmsnorm_warp_kernel<T, v><<<blocks, 256, 0, st>>>(x, row_idx, g, y, n, d, eps);                   \
    return true;
    RW_CASE(1) RW_CASE(2) RW_CASE(4) RW_CASE(8) RW_CASE(16)
#undef RW_CASE
    default: return false;
  }
}

int launch_rmsnorm_rows(cudaStream_t st, int dtype, const void *x, const int32_t *row_idx,
                        const void *g, void *y, int n, int d, float eps) {
  if (n == 0) return LAZY_OK;
  // The sum of squares is added in another order than in the one-CTA-per-row kernel below (per lane over
  // its vectors, then the shuffle tree): rows whose width the warp kernel covers always take it, so a
  // given shape is always normalised by the same kernel.
  const bool warp_ok = dtype == LAZY_F32
                           ? launch_rmsnorm_warp<float>(st, (const float *)x, row_idx, (const float *)g, (float *)y, n, d, eps)
                           : launch_rmsnorm_warp<bf16>(st, (const bf16 *)x, row_idx, (const bf16 *)g, (bf16 *)y, n, d, eps);
  if (warp_ok) {
    LAZY_COUNT_LAUNCH();
    return launch_ok();
  }
  if (dtype == LAZY_F32)
    rmsnorm_kernel<float, 128><<<n, 128, 0, st>>>((const float *)x, row_idx, (const float *)g,
                                                  (float *)y, d, eps);
  else
    rmsnorm_kernel<bf16, 128><<<n, 128, 0, st>>>((const bf16 *)x, row_idx, (const bf16 *)g,
                                                 (bf16 *)y, d, eps);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}
int launch_rmsnorm(cudaStream_t st, int dtype, const void *x, const void *g, void *y, int n, int d,
                   float eps) {
  return launch_rmsnorm_rows(st, dtype, x, nullptr, g, y, n, d, eps);
}

// ---- per-row e4m3 quantisation of activations ------------------------------------------------------------
// One CTA per row: scale = max|x| / 448 (1 for an all-zero row), code = e4m3(x / scale), both decided in
// fp32 with IEEE division and round-to-nearest-even conversion (the definition the CPU reference follows).
// The row is read twice (the second pass hits L1 / L2).
__global__ void __launch_bounds__(256)
quant_rows_e4m3_kernel(const bf16 *__restrict__ x, uint8_t *__restrict__ q, float *__restrict__ scale, int K) {
  const int r = blockIdx.x;
  const uint4 *xr = reinterpret_cast<const uint4 *>(x + (size_t)r * K);
  const int nvec = K >> 3;
  float amax = 0.f;
  for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
    Vec16<bf16> v;
    v.raw = xr[i];
    float f[8];
    v.unpack(f);
#pragma unroll
    for (int j = 0; j < 8; ++j) amax = fmaxf(amax, fabsf(f[j]));
  }
  __shared__ float part[8];
  amax = warp_max(amax);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = amax;
  __syncthreads();
  amax = part[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) amax = fmaxf(amax, part[w]);
  const float sc = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
  if (threadIdx.x == 0) scale[r] = sc;
  uint2 *qr = reinterpret_cast<uint2 *>(q + (size_t)r * K);
  for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
    Vec16<bf16> v;
    v.raw = xr[i];
    float f[8];
    v.unpack(f);
    uint32_t w[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      unsigned short lo, hi;  // each: two codes, the first operand of the conversion in the upper byte
      asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(__fdiv_rn(f[4 * h + 1], sc)), "f"(__fdiv_rn(f[4 * h], sc)));
      asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(__fdiv_rn(f[4 * h + 3], sc)), "f"(__fdiv_rn(f[4 * h + 2], sc)));
      w[h] = (uint32_t)lo | ((uint32_t)hi << 16);
    }
    qr[i] = make_uint2(w[0], w[1]);
  }
}
int launch_quant_rows_e4m3(cudaStream_t st, const void *x, void *q, float *scale, int M, int K) {
  if (M == 0) return LAZY_OK;
  if ((K % 16) || ((uintptr_t)x & 15) || ((uintptr_t)q & 15)) return LAZY_E_BADARG;
  quant_rows_e4m3_kernel<<<M, 256, 0, st>>>((const bf16 *)x, (uint8_t *)q, scale, K);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

// ---- RoPE table -----------------------------------------------------------------------------------
// table[pos][i] = (cos, sin)(pos * theta^(-2i/dh)), evaluated in double once at set-up.
__global__ void rope_table_kernel(float2 *table, int max_pos, int half, int head_dim, double theta) {
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= max_pos * half) return;
  int p = idx / half, i = idx % half;
  double inv_freq = pow(theta, -2.0 * (double)i / (double)head_dim);
  double s, c;
  sincos((double)p * inv_freq, &s, &c);
  table[idx] = make_float2((float)c, (float)s);
}
int launch_rope_table(cudaStream_t st, float *table, int max_pos, int head_dim, float theta) {
  int half = head_dim / 2;
  int n = max_pos * half;
  if (n == 0) return LAZY_OK;
  rope_table_kernel<<<cdiv(n, 256), 256, 0, st>>>((float2 *)table, max_pos, half, head_dim,
                                                  (double)theta);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

// ---- RoPE + KV-cache write ---------------------------------------------------------------------------
// gridDim.y CTAs per row of qkv = [q | k | v].  Pairs (i, i + dh/2) of every q and k head are rotated by
// the row's ORIGINAL position; q goes back in place, k and v go to the layer's cache rows.
template <typename T>
__global__ void rope_kv_kernel(T *__restrict__ qkv, const int32_t *__restrict__ pos,
                               const float2 *__restrict__ table, T *__restrict__ kcache,
                               T *__restrict__ vcache, int32_t *__restrict__ kv_pos,
                               const int32_t *__restrict__ kv_row, int n_heads, int n_kv_heads, int head_dim,
                               int max_pos, DevStatus *status) {
  constexpr int V = Elem<T>::kPerVec;
  const int r = blockIdx.x;
  const int d = n_heads * head_dim, dkv = n_kv_heads * head_dim;  // a row of qkv = [q: d | k: dkv | v: dkv]
  const int half = head_dim / 2;
  int p = pos[r];
  if (p < 0 || p >= max_pos) {
    if (threadIdx.x == 0) dev_fail(status, LAZY_E_CAPACITY, W_ROPE_POS, r, p);
    p = 0;
  }
  const size_t krow = kv_row ? (size_t)kv_row[r] : (size_t)r;
  T *row = qkv + (size_t)r * (d + 2 * dkv);
  const float2 *tab = table + (size_t)p * half;
  const int vec_per_half = half / V;
  const int pairs_q = n_heads * vec_per_half, pairs_k = n_kv_heads * vec_per_half;  // vector pairs of q, of k
  const int tid = blockIdx.y * blockDim.x + threadIdx.x, tstep = gridDim.y * blockDim.x;
  for (int t = tid; t < pairs_q + pairs_k; t += tstep) {
    const int which = t >= pairs_q;  // 0 = q, 1 = k
    const int u = t - which * pairs_q;
    const int h = u / vec_per_half;
    const int i0 = (u - h * vec_per_half) * V;
    T *base = row + which * d + h * head_dim;
    Vec16<T> a, b;
    a.load(base + i0);
    b.load(base + half + i0);
    float fa[V], fb[V], oa[V], ob[V];
    a.unpack(fa);
    b.unpack(fb);
#pragma unroll
    for (int j = 0; j < V; ++j) {
      const float2 cs = tab[i0 + j];
      oa[j] = fa[j] * cs.x - fb[j] * cs.y;
      ob[j] = fb[j] * cs.x + fa[j] * cs.y;
    }
    a.pack(oa);
    b.pack(ob);
    if (which == 0) {
      a.store(base + i0);
      b.store(base + half + i0);
    } else {
      T *kd = kcache + krow * dkv + h * head_dim;
      a.store(kd + i0);
      b.store(kd + half + i0);
    }
  }
  const uint4 *vs = reinterpret_cast<const uint4 *>(row + d + dkv);
  uint4 *vd = reinterpret_cast<uint4 *>(vcache + krow * dkv);
  for (int i = tid; i < dkv / V; i += tstep) vd[i] = vs[i];
  if (tid == 0 && kv_pos) kv_pos[krow] = p;
}

int launch_rope_kv(cudaStream_t st, int dtype, void *qkv, const int32_t *pos, const float *table,
                   void *kcache, void *vcache, int32_t *kv_pos, const int32_t *kv_row, int n,
                   int n_heads, int head_dim, int max_pos, DevStatus *status, int n_kv_heads) {
  if (n == 0) return LAZY_OK;
  if (n_kv_heads <= 0) n_kv_heads = n_heads;
  const dim3 grid(n, n <= 16 ? 8 : 1);  // a handful of rows (decode): spread each over several CTAs
  if (dtype == LAZY_F32)
    rope_kv_kernel<float><<<grid, 128, 0, st>>>((float *)qkv, pos, (const float2 *)table,
                                             (float *)kcache, (float *)vcache, kv_pos, kv_row,
                                             n_heads, n_kv_heads, head_dim, max_pos, status);
  else
    rope_kv_kernel<bf16><<<grid, 128, 0, st>>>((bf16 *)qkv, pos, (const float2 *)table, (bf16 *)kcache,
                                            (bf16 *)vcache, kv_pos, kv_row, n_heads, n_kv_heads, head_dim,
                                            max_pos, status);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

// ---- row gather (stream compaction of hidden / K / V rows, Aux-Cache reads) --------------------------
// dst[i] = src[idx[i]] (idx NULL: dst[i] = src[i]).
__global__ void gather_rows_kernel(const uint4 *__restrict__ src, const int32_t *__restrict__ idx,
                                   uint4 *__restrict__ dst, int n, int vec_per_row, int src_rows,
                                   DevStatus *status) {
  for (int r = blockIdx.x; r < n; r += gridDim.x) {
    int s = idx ? idx[r] : r;
    if (s < 0 || s >= src_rows) {
      if (threadIdx.x == 0) dev_fail(status, LAZY_E_BADARG, W_GATHER_INDEX, r, s);
      continue;
    }
    const uint4 *sp = src + (size_t)s * vec_per_row;
    uint4 *dp = dst + (size_t)r * vec_per_row;
    for (int i = threadIdx.x; i < vec_per_row; i += blockDim.x) dp[i] = sp[i];
  }
}
int launch_gather_rows(cudaStream_t st, const void *src, const int32_t *idx, void *dst, int n,
                       int row_bytes, int src_rows, DevStatus *status) {
  if (n == 0) return LAZY_OK;
  int blocks = n < sm_count() * 16 ? n : sm_count() * 16;
  gather_rows_kernel<<<blocks, 128, 0, st>>>((const uint4 *)src, idx, (uint4 *)dst, n,
                                             row_bytes / 16, src_rows, status);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

__global__ void gather_i32_kernel(const int32_t *src, const int32_t *idx, int32_t *dst, int n) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = src[idx[i]];
}
int launch_gather_i32(cudaStream_t st, const int32_t *src, const int32_t *idx, int32_t *dst, int n) {
  if (n == 0) return LAZY_OK;
  gather_i32_kernel<<<cdiv(n, 256), 256, 0, st>>>(src, idx, dst, n);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

// ---- LM head on the last rows ---------------------------------------------------------------------------
// logits[s, v] = sum_k h[s, k] * W[v, k].  One warp per vocabulary row streams W once (16-byte
// loads); the few hidden rows sit in shared memory as fp32.
template <typename T, int SEQ_CHUNK>
__global__ void lm_head_kernel(const T *__restrict__ h, const T *__restrict__ w,
                               float *__restrict__ logits, int n_rows, int d, int vocab) {
  constexpr int V = Elem<T>::kPerVec;
  extern __shared__ float hs[];  // [SEQ_CHUNK][d]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int warps = blockDim.x >> 5;
  for (int s0 = 0; s0 < n_rows; s0 += SEQ_CHUNK) {
    const int ns = min(SEQ_CHUNK, n_rows - s0);
    __syncthreads();
    for (int i = threadIdx.x; i < ns * d; i += blockDim.x)
      hs[i] = Elem<T>::to_f(h[(size_t)s0 * d + i]);
    __syncthreads();
    for (int v = blockIdx.x * warps + warp; v < vocab; v += gridDim.x * warps) {
      float acc[SEQ_CHUNK];
#pragma unroll
      for (int s = 0; s < SEQ_CHUNK; ++s) acc[s] = 0.f;
      const T *wr = w + (size_t)v * d;
      for (int i = lane * V; i < d; i += 32 * V) {
        Vec16<T> wv;
        wv.load(wr + i);
        float wf[V];
        wv.unpack(wf);
#pragma unroll
        for (int s = 0; s < SEQ_CHUNK; ++s) {
          if (s < ns) {
            const float *hp = hs + s * d + i;
#pragma unroll
            for (int j = 0; j < V; ++j) acc[s] += wf[j] * hp[j];
          }
        }
      }
#pragma unroll
      for (int s = 0; s < SEQ_CHUNK; ++s) {
        float t = warp_sum(acc[s]);
        if (lane == 0 && s < ns) logits[(size_t)(s0 + s) * vocab + v] = t;
      }
    }
  }
}

int launch_lm_head(cudaStream_t st, int dtype, const void *h, const void *w, float *logits,
                   int n_rows, int d, int vocab, bool w_const) {
  if (n_rows == 0) return LAZY_OK;
  if (gemv_small_m_eligible(dtype, 4, d)) {  // up to four rows per pass over the matrix
    for (int s0 = 0; s0 < n_rows; s0 += 4) {
      const int m = n_rows - s0 < 4 ? n_rows - s0 : 4;
      LAZY_TRY(launch_gemv_small_m(st, (const bf16 *)h + (size_t)s0 * d, w, nullptr, nullptr,
                                   logits + (size_t)s0 * vocab, m, vocab, d, 0, nullptr, 0.f, 1, w_const));
    }
    return LAZY_OK;
  }
  constexpr int SC = 4;
  size_t smem = (size_t)SC * d * sizeof(float);
  int blocks = sm_count() * 2;
  if (dtype == LAZY_F32) {
    auto kfn = lm_head_kernel<float, SC>;
    LAZY_CUDA_OK(cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kfn<<<blocks, 256, smem, st>>>((const float *)h, (const float *)w, logits, n_rows, d, vocab);
  } else {
    auto kfn = lm_head_kernel<bf16, SC>;
    LAZY_CUDA_OK(cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kfn<<<blocks, 256, smem, st>>>((const bf16 *)h, (const bf16 *)w, logits, n_rows, d, vocab);
  }
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

// ---- greedy argmax (ties -> lowest id) ----------------------------------------------------------------------
constexpr int ARGMAX_THREADS = 1024;
__global__ void __launch_bounds__(ARGMAX_THREADS)
argmax_kernel(const float *__restrict__ logits, int32_t *__restrict__ out, int vocab) {
  const float *row = logits + (size_t)blockIdx.x * vocab;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  auto take = [&](float v, int i) {
    if (v > best || (v == best && i < bi)) { best = v; bi = i; }
  };
  if ((((uintptr_t)row) & 15) == 0) {
    const int nv = vocab >> 2;
    for (int i = threadIdx.x; i < nv; i += ARGMAX_THREADS) {
      const float4 v = reinterpret_cast<const float4 *>(row)[i];
      take(v.x, 4 * i); take(v.y, 4 * i + 1); take(v.z, 4 * i + 2); take(v.w, 4 * i + 3);
    }
    for (int i = 4 * nv + threadIdx.x; i < vocab; i += ARGMAX_THREADS) take(row[i], i);
  } else {
    for (int i = threadIdx.x; i < vocab; i += ARGMAX_THREADS) take(row[i], i);
  }
  // warp, then CTA: larger value wins, equal values go to the lower id
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float v = __shfl_xor_sync(0xffffffffu, best, o);
    const int i = __shfl_xor_sync(0xffffffffu, bi, o);
    take(v, i);
  }
  __shared__ float sv[ARGMAX_THREADS / 32];
  __shared__ int si[ARGMAX_THREADS / 32];
  if ((threadIdx.x & 31) == 0) {
    sv[threadIdx.x >> 5] = best;
    si[threadIdx.x >> 5] = bi;
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    best = sv[threadIdx.x];
    bi = si[threadIdx.x];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float v = __shfl_xor_sync(0xffffffffu, best, o);
      const int i = __shfl_xor_sync(0xffffffffu, bi, o);
      take(v, i);
    }
    if (threadIdx.x == 0) out[blockIdx.x] = bi == 0x7fffffff ? 0 : bi;
  }
}
int launch_argmax(cudaStream_t st, const float *logits, int32_t *out, int n_rows, int vocab) {
  if (n_rows == 0) return LAZY_OK;
  argmax_kernel<<<n_rows, ARGMAX_THREADS, 0, st>>>(logits, out, vocab);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

}  // namespace lazy
