// Skinny GEMM for decode: C[M,N] = A[M,K] * B[N,K]^T with M <= 4 rows (bf16 storage, fp32
// accumulation).  At these sizes the step is pure weight streaming, so the kernel is laid out for
// HBM: every warp owns output columns, reads each weight row exactly once with 16-byte loads
// (several in flight per lane), keeps the few activation rows in shared memory, and reduces with
// shuffles.  Same epilogues as the tensor-core GEMM: plain, + residual, SiLU(gate) * up, and the QKV
// projection with the rotary embedding and the K/V cache write (a warp then owns the two columns i and
// i + 64 of a head that rotate together).
#include "common.cuh"

namespace lazy {

namespace {

constexpr int GV_MAX_M = 4;
constexpr int GV_THREADS = 256;

// Weights are read once: keep them out of L1.
__device__ __forceinline__ uint4 ld_stream(const uint4 *p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  return r;
}

enum { GV_PLAIN = 0, GV_SWIGLU = 1, GV_QKV_ROPE = 2 };

// Operands of the QKV mode (head_dim 128): positions and the (cos, sin) table, the layer's cache rows.
struct GemvRope {
  const int32_t *pos;     // [M] original positions
  const float2 *table;    // [max_pos][64]
  bf16 *kcache, *vcache;  // [rows, d_model]
  int32_t *kv_pos;        // position tag per cache row
  const int32_t *kv_row;  // cache row of input row m
  int d_model, max_pos;
  int d_kv;               // width of a K / V cache row (n_kv_heads * 128)
  DevStatus *status;
};

// The weight rows a warp streams for its n-th task.  Plain: output column n.  SwiGLU: gate row n and up
// row n.  QKV: task n = (section q/k/v, head, i < 64) -> rows of output columns i and i + 64 of that head.
template <int MODE>
__device__ __forceinline__ void gv_task_rows(int n, const bf16 *B0, const bf16 *B1, int K, int d_model, int d_kv,
                                             const uint4 *&w0, const uint4 *&w1, int &col0) {
  if (MODE == GV_QKV_ROPE) {
    // d_model / 2 tasks for q, then d_kv / 2 each for k and v
    const int tq = d_model >> 1, tk = d_kv >> 1;
    const int sect = n < tq ? 0 : (n < tq + tk ? 1 : 2);
    const int u = n - (sect == 0 ? 0 : (sect == 1 ? tq : tq + tk));
    col0 = (sect == 0 ? 0 : (sect == 1 ? d_model : d_model + d_kv)) + (u >> 6) * 128 + (u & 63);
    w0 = reinterpret_cast<const uint4 *>(B0 + (size_t)col0 * K);
    w1 = reinterpret_cast<const uint4 *>(B0 + (size_t)(col0 + 64) * K);
  } else {
    col0 = n;
    w0 = reinterpret_cast<const uint4 *>(B0 + (size_t)n * K);
    w1 = MODE == GV_SWIGLU ? reinterpret_cast<const uint4 *>(B1 + (size_t)n * K) : nullptr;
  }
}

template <int M_ROWS, int MODE>
__global__ void __launch_bounds__(GV_THREADS, 4)
gemv_small_m_kernel(const bf16 *__restrict__ A, const bf16 *__restrict__ B0, const bf16 *__restrict__ B1,
                    const bf16 *__restrict__ R, void *__restrict__ C, int N, int K,
                    const bf16 *__restrict__ gain, float eps, int c_f32, const GemvRope rope) {
  constexpr bool SWIGLU = MODE != GV_PLAIN;  // two weight rows per task
  extern __shared__ uint4 gv_smem[];  // [M_ROWS][K/8] activation rows as 16-byte vectors
  __shared__ float gv_red[M_ROWS][GV_THREADS / 32];
  const int kvec = K >> 3;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // When launched as a programmatic dependent (the caller vouches that the weights are not being written
  // by earlier work on the stream), this grid starts while the kernel before it drains: the first batch of
  // this warp's first column is requested before waiting for that kernel, and the kernel after this one is
  // released to do the same.  Activations, gains and residuals are touched only after the wait.  Launched
  // the ordinary way the grid starts after that kernel has completed and the two instructions do nothing.
  constexpr int U = SWIGLU ? 4 : 8;  // weight vectors per lane in flight (x2 matrices for SwiGLU)
  const int n_first = blockIdx.x * (GV_THREADS / 32) + warp;
  uint4 wr[U], ur[SWIGLU ? U : 1];  // the batch in flight
  if (n_first < N) {
    const uint4 *w0, *w1;
    int col0;
    gv_task_rows<MODE>(n_first, B0, B1, K, rope.d_model, rope.d_kv, w0, w1, col0);
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int v = lane + 32 * u;
      if (v < kvec) {
        wr[u] = ld_stream(w0 + v);
        if (SWIGLU) ur[u] = ld_stream(w1 + v);
      }
    }
  }
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  for (int i = threadIdx.x; i < M_ROWS * kvec; i += GV_THREADS)
    gv_smem[i] = reinterpret_cast<const uint4 *>(A)[i];
  __syncthreads();
  if (gain) {  // RMSNorm of the rows on the way in: a = bf16(x * rsqrt(mean(x^2) + eps) * gain)
    float ss[M_ROWS];
#pragma unroll
    for (int m = 0; m < M_ROWS; ++m) {
      ss[m] = 0.f;
      for (int v = threadIdx.x; v < kvec; v += GV_THREADS) {
        Vec16<bf16> xv;
        xv.raw = gv_smem[m * kvec + v];
        float f[8];
        xv.unpack(f);
#pragma unroll
        for (int i = 0; i < 8; ++i) ss[m] = fmaf(f[i], f[i], ss[m]);
      }
      ss[m] = warp_sum(ss[m]);
      if (lane == 0) gv_red[m][warp] = ss[m];
    }
    __syncthreads();
#pragma unroll
    for (int m = 0; m < M_ROWS; ++m) {
      float tot = 0.f;
#pragma unroll
      for (int w = 0; w < GV_THREADS / 32; ++w) tot += gv_red[m][w];
      const float scale = rsqrtf(tot / (float)K + eps);
      for (int v = threadIdx.x; v < kvec; v += GV_THREADS) {
        Vec16<bf16> xv, gv;
        xv.raw = gv_smem[m * kvec + v];
        gv.raw = reinterpret_cast<const uint4 *>(gain)[v];
        float f[8], gf[8];
        xv.unpack(f);
        gv.unpack(gf);
#pragma unroll
        for (int i = 0; i < 8; ++i) f[i] = f[i] * scale * gf[i];
        xv.pack(f);
        gv_smem[m * kvec + v] = xv.raw;
      }
    }
    __syncthreads();
  }
  const int warps_total = gridDim.x * (GV_THREADS / 32);
  bool have_first = true;
  for (int n = blockIdx.x * (GV_THREADS / 32) + warp; n < N; n += warps_total) {
    const uint4 *w0, *w1;
    int col0;
    gv_task_rows<MODE>(n, B0, B1, K, rope.d_model, rope.d_kv, w0, w1, col0);
    float acc0[M_ROWS], acc1[M_ROWS];
#pragma unroll
    for (int m = 0; m < M_ROWS; ++m) acc0[m] = acc1[m] = 0.f;
    // U weight vectors per lane are requested before the first is used: 8 x 16 bytes in flight
    for (int v0 = lane; v0 < kvec; v0 += 32 * U) {
      if (have_first) {  // on its way since before the wait
        have_first = false;
      } else {
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int v = v0 + 32 * u;
          if (v < kvec) {
            wr[u] = ld_stream(w0 + v);
            if (SWIGLU) ur[u] = ld_stream(w1 + v);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int v = v0 + 32 * u;
        if (v >= kvec) break;
        Vec16<bf16> wv;
        wv.raw = wr[u];
        float wf[8], uf[8];
        wv.unpack(wf);
        if (SWIGLU) {
          Vec16<bf16> uv;
          uv.raw = ur[u];
          uv.unpack(uf);
        }
#pragma unroll
        for (int m = 0; m < M_ROWS; ++m) {
          Vec16<bf16> av;
          av.raw = gv_smem[m * kvec + v];
          float af[8];
          av.unpack(af);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            acc0[m] = fmaf(af[i], wf[i], acc0[m]);
            if (SWIGLU) acc1[m] = fmaf(af[i], uf[i], acc1[m]);
          }
        }
      }
    }
#pragma unroll
    for (int m = 0; m < M_ROWS; ++m) {
      float g = warp_sum(acc0[m]);
      float u = SWIGLU ? warp_sum(acc1[m]) : 0.f;
      if (MODE == GV_QKV_ROPE) {
        if (lane == 0) {
          const int d = rope.d_model, dkv = rope.d_kv;
          const int sect = col0 < d ? 0 : (col0 < d + dkv ? 1 : 2);
          const int cin = col0 - (sect == 0 ? 0 : (sect == 1 ? d : d + dkv));  // column inside q, k or v
          int p = rope.pos[m];
          if (p < 0 || p >= rope.max_pos) {
            dev_fail(rope.status, LAZY_E_CAPACITY, W_ROPE_POS, m, p);
            p = 0;
          }
          float o0 = g, o1 = u;
          if (sect < 2) {  // q and k rotate by the row's original position
            const float2 cs = rope.table[(size_t)p * 64 + (cin & 63)];
            o0 = g * cs.x - u * cs.y;
            o1 = u * cs.x + g * cs.y;
          }
          const size_t krow = (size_t)rope.kv_row[m];
          bf16 *dst = sect == 0 ? reinterpret_cast<bf16 *>(C) + (size_t)m * (d + 2 * dkv) + cin
                                : (sect == 1 ? rope.kcache : rope.vcache) + krow * dkv + cin;
          dst[0] = __float2bfloat16_rn(o0);
          dst[64] = __float2bfloat16_rn(o1);
          if (n == 0) rope.kv_pos[krow] = p;
        }
      } else if (lane == 0) {
        float out = g;
        if (MODE == GV_SWIGLU) out = g / (1.f + __expf(-g)) * u;
        else if (R) out += __bfloat162float(R[(size_t)m * N + n]);
        if (c_f32) reinterpret_cast<float *>(C)[(size_t)m * N + n] = out;
        else reinterpret_cast<bf16 *>(C)[(size_t)m * N + n] = __float2bfloat16_rn(out);
      }
    }
  }
}

template <int M_ROWS, int MODE>
int launch_one(cudaStream_t st, const void *A, const void *B0, const void *B1, const void *R, void *C, int N,
               int K, const void *gain, float eps, int c_f32, bool pdl, const GemvRope &rope = GemvRope()) {
  const size_t smem = (size_t)M_ROWS * K * 2;
  auto kfn = gemv_small_m_kernel<M_ROWS, MODE>;
  LAZY_CUDA_OK(cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  int blocks = cdiv(N, GV_THREADS / 32);
  const int cap = sm_count() * 4;
  if (blocks > cap) blocks = cap;
  // programmatic dependent launch (pdl): this grid may start while the kernel before it in the stream drains
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks, 1, 1);
  cfg.blockDim = dim3(GV_THREADS, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = pdl ? 1 : 0;
  LAZY_CUDA_OK(cudaLaunchKernelEx(&cfg, kfn, (const bf16 *)A, (const bf16 *)B0, (const bf16 *)B1, (const bf16 *)R, C,
                                  N, K, (const bf16 *)gain, eps, c_f32, rope));
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

}  // namespace

bool gemv_small_m_eligible(int dtype, int M, int K) {
  return dtype == LAZY_BF16 && M >= 1 && M <= GV_MAX_M && (K % 8) == 0 && (size_t)M * K * 2 <= 200 * 1024;
}

// gain != NULL: the rows of A are RMS-normalised (gain, eps) before the product, with the rounding a
// separate normalisation kernel writing bf16 would have had.  c_f32: C holds fp32 instead of bf16.
int launch_gemv_small_m(cudaStream_t st, const void *A, const void *B0, const void *B1, const void *R,
                        void *C, int M, int N, int K, int swiglu, const void *gain, float eps, int c_f32,
                        bool b_const) {
  if (((uintptr_t)A & 15) || ((uintptr_t)B0 & 15) || ((uintptr_t)B1 & 15) || ((uintptr_t)gain & 15))
    return LAZY_E_BADARG;
#define GV_CASE(m)                                                                            \
  case m:                                                                                     \
    return swiglu ? launch_one<m, GV_SWIGLU>(st, A, B0, B1, nullptr, C, N, K, gain, eps, c_f32, b_const) \
                  : launch_one<m, GV_PLAIN>(st, A, B0, nullptr, R, C, N, K, gain, eps, c_f32, b_const);
  switch (M) {
    GV_CASE(1)
    GV_CASE(2)
    GV_CASE(3)
    GV_CASE(4)
    default: return LAZY_E_BADARG;
  }
#undef GV_CASE
}

// QKV projection of one to four rows (optionally RMS-normalised first) with the rotary embedding and the
// K/V cache write in its epilogue: qkv [M, 3d] receives the rotated q (its k and v thirds are left
// untouched), rotated k and v go to cache rows kv_row[m] with their position tag.  head_dim 128.  Only the
// decode step calls this, with the context's own (constant) weights: always a programmatic dependent.
int launch_gemv_qkv_rope(cudaStream_t st, const void *x, const void *w_qkv, void *qkv, const void *gain, float eps,
                         const int32_t *pos, const float *table, void *kcache, void *vcache, int32_t *kv_pos,
                         const int32_t *kv_row, int M, int d_model, int max_pos, DevStatus *status, int d_kv) {
  if (d_kv <= 0) d_kv = d_model;
  if (((uintptr_t)x & 15) || ((uintptr_t)w_qkv & 15) || ((uintptr_t)gain & 15) || !pos || !table || !kcache ||
      !vcache || !kv_pos || !kv_row || (d_model % 128) || (d_kv % 128))
    return LAZY_E_BADARG;
  GemvRope r;
  r.pos = pos;
  r.table = (const float2 *)table;
  r.kcache = (bf16 *)kcache;
  r.vcache = (bf16 *)vcache;
  r.kv_pos = kv_pos;
  r.kv_row = kv_row;
  r.d_model = d_model;
  r.d_kv = d_kv;
  r.max_pos = max_pos;
  r.status = status;
  const int tasks = (d_model + 2 * d_kv) / 2;
#define GV_CASE(m) \
  case m: return launch_one<m, GV_QKV_ROPE>(st, x, w_qkv, nullptr, nullptr, qkv, tasks, d_model, gain, eps, 0, true, r);
  switch (M) {
    GV_CASE(1)
    GV_CASE(2)
    GV_CASE(3)
    GV_CASE(4)
    default: return LAZY_E_BADARG;
  }
#undef GV_CASE
}

}  // namespace lazy
