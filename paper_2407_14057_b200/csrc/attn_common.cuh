// Pieces shared by the tensor-core attention kernels: instruction descriptor, the score by-product's
// layout, and the few arithmetic instructions the softmax threads are written around.
#pragma once
#include "tc_common.cuh"

namespace lazy {

// kind::f16 instruction descriptor: D fp32, A/B bf16; major bits: 0 = K-major, 1 = MN-major.
__device__ __forceinline__ uint32_t idesc_bf16(int m, int n, int a_mn, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// Optional by-product: the last row's softmax numerators, for the Eq. 1 score.
// p[(seq*H + h)*max_tiles*64 + j] receives 2^(s - m_tile) for key j of the sequence,
// mtile[(seq*H + h)*max_tiles + t] the reference exponent used in tile t, stats[(seq*H + h)*2 ..] the
// final (m, 1/l).
struct AttnScoreOut {
  float *p, *mtile, *stats;
  int max_tiles, seq_id;
};

// 2^x on the special-function unit; ex2(-inf) = 0.
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Three-input maximum and two-wide fp32 arithmetic (one instruction each on this architecture): the
// softmax threads are bound by instruction issue, so halving the count of the plain ALU work matters.
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ unsigned long long f32x2_pack(float lo, float hi) {
  unsigned long long p;
  asm("mov.b64 %0, {%1, %2};" : "=l"(p) : "f"(lo), "f"(hi));
  return p;
}
__device__ __forceinline__ void f32x2_unpack(unsigned long long p, float &lo, float &hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p));
}
__device__ __forceinline__ unsigned long long f32x2_fma(unsigned long long a, unsigned long long b,
                                                        unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ unsigned long long f32x2_add(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

}  // namespace lazy
