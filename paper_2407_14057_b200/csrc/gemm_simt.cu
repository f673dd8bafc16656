// CUDA-core GEMM for the fp32 mode (small models): C = A B^T (+R), or the SwiGLU form
// C = silu(A B0^T) * (A B1^T).  64x64 tile, 16-deep k-slices in shared memory, 4x4 per thread,
// fp32 accumulation, plain FMA (no TF32).  Also instantiated for bf16 storage so the tensor-core
// kernel can be cross-checked on the device.
#include "common.cuh"

namespace lazy {

template <typename T, bool SWIGLU>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const T *__restrict__ A, const T *__restrict__ B0, const T *__restrict__ B1,
                 const T *__restrict__ R, T *__restrict__ C, int M, int N, int K) {
  constexpr int TM = 64, TN = 64, TK = 16;
  __shared__ float As[TK][TM + 1];
  __shared__ float B0s[TK][TN + 1];
  __shared__ float B1s[SWIGLU ? TK : 1][TN + 1];
  const int m0 = blockIdx.y * TM, n0 = blockIdx.x * TN;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc0[4][4] = {}, acc1[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += TK) {
    for (int i = threadIdx.x; i < TM * TK; i += 256) {
      const int r = i / TK, c = i % TK;
      const int gm = m0 + r, gn = n0 + r, gk = k0 + c;
      As[c][r] = (gm < M && gk < K) ? Elem<T>::to_f(A[(size_t)gm * K + gk]) : 0.f;
      B0s[c][r] = (gn < N && gk < K) ? Elem<T>::to_f(B0[(size_t)gn * K + gk]) : 0.f;
      if (SWIGLU) B1s[c][r] = (gn < N && gk < K) ? Elem<T>::to_f(B1[(size_t)gn * K + gk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float a[4], b0[4], b1[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        b0[j] = B0s[kk][tx * 4 + j];
        b1[j] = SWIGLU ? B1s[kk][tx * 4 + j] : 0.f;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc0[i][j] = fmaf(a[i], b0[j], acc0[i][j]);
          if (SWIGLU) acc1[i][j] = fmaf(a[i], b1[j], acc1[i][j]);
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tx * 4 + j;
      if (gn >= N) continue;
      float v = acc0[i][j];
      if (SWIGLU) {
        v = v / (1.f + expf(-v)) * acc1[i][j];
      } else if (R) {
        v += Elem<T>::to_f(R[(size_t)gm * N + gn]);
      }
      C[(size_t)gm * N + gn] = Elem<T>::from_f(v);
    }
  }
}

int launch_gemm_simt(cudaStream_t st, int dtype, const void *A, const void *B0, const void *B1,
                     const void *R, void *C, int M, int N, int K, int swiglu) {
  if (M == 0) return LAZY_OK;
  dim3 grid(cdiv(N, 64), cdiv(M, 64));
  if (dtype == LAZY_F32) {
    if (swiglu)
      gemm_simt_kernel<float, true><<<grid, 256, 0, st>>>((const float *)A, (const float *)B0,
                                                          (const float *)B1, nullptr, (float *)C, M, N, K);
    else
      gemm_simt_kernel<float, false><<<grid, 256, 0, st>>>((const float *)A, (const float *)B0, nullptr,
                                                           (const float *)R, (float *)C, M, N, K);
  } else {
    if (swiglu)
      gemm_simt_kernel<bf16, true><<<grid, 256, 0, st>>>((const bf16 *)A, (const bf16 *)B0,
                                                         (const bf16 *)B1, nullptr, (bf16 *)C, M, N, K);
    else
      gemm_simt_kernel<bf16, false><<<grid, 256, 0, st>>>((const bf16 *)A, (const bf16 *)B0, nullptr,
                                                          (const bf16 *)R, (bf16 *)C, M, N, K);
  }
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

}  // namespace lazy
