// Epilogues of the bf16 tensor-core GEMMs: what a thread does with its row of a finished 128x256
// fp32 accumulator tile in tensor memory.  Shared by the one-CTA and the CTA-pair kernels.
#pragma once
#include "tc_common.cuh"

namespace lazy {

constexpr int GEMM_ACC_N = 256;  // accumulator columns per tile

enum { EPI_PLAIN = 0, EPI_RESIDUAL = 1, EPI_SWIGLU = 2, EPI_QKV_ROPE = 3 };

// Extra operands of the QKV epilogue: the rotary embedding is applied to the fp32 accumulators and
// the rotated k, and v, go straight to the layer's cache rows (head_dim 128: one 256-column tile is
// two whole heads of q, k or v, and a thread holds its row's full heads).
struct RopeArgs {
  const int32_t *pos;     // [M] original positions
  const float2 *table;    // [max_pos][64] (cos, sin)
  bf16 *kcache, *vcache;  // [rows, d_model]
  int32_t *kv_pos;        // position tag per cache row (may be NULL)
  const int32_t *kv_row;  // cache row of GEMM row r (NULL: r)
  int d_model, max_pos;
};

// One thread, one row.  taddr: TMEM address of the row's first accumulator column (lane field set);
// row: global output row; n0: first output column of the tile as the caller sees it.  C is [M, ldc];
// for EPI_SWIGLU accumulator columns [0,128) are gate features, [128,256) the matching up features and C
// receives 128 columns per tile.
template <int EPI>
__device__ __forceinline__ void gemm_epilogue_row(uint32_t taddr, int row, int n0, int M, int N, int ldc,
                                                  const bf16 *__restrict__ R, bf16 *__restrict__ C,
                                                  const RopeArgs &rope, DevStatus *status) {
  constexpr int BN = GEMM_ACC_N;
  constexpr int TILE_N = (EPI == EPI_SWIGLU) ? BN / 2 : BN;
  bf16 *crow = C + (size_t)row * ldc;
  const bf16 *rrow = (EPI == EPI_RESIDUAL) ? R + (size_t)row * ldc : nullptr;
  if (EPI == EPI_QKV_ROPE) {
    // section of the fused projection this tile belongs to: 0 = q, 1 = k, 2 = v
    const int sect = n0 / rope.d_model;
    const int col_in = n0 - sect * rope.d_model;
    int p = 0;
    size_t krow = 0;
    if (row < M) {
      p = rope.pos[row];
      if (p < 0 || p >= rope.max_pos) {
        dev_fail(status, LAZY_E_CAPACITY, W_ROPE_POS, row, p);
        p = 0;
      }
      krow = rope.kv_row ? (size_t)rope.kv_row[row] : (size_t)row;
    }
    bf16 *dst = sect == 0 ? crow + n0
                          : (sect == 1 ? rope.kcache : rope.vcache) + krow * rope.d_model + col_in;
    if (sect == 2) {
#pragma unroll 1
      for (int c = 0; c < BN; c += 32) {
        float v[32];
        tmem_ld_32x32(taddr + (uint32_t)c, v);
        if (row < M) {
#pragma unroll
          for (int j = 0; j < 32; j += 8) {
            Vec16<bf16> o;
            o.pack(v + j);
            o.store(dst + c + j);
          }
        }
      }
    } else {
      const float2 *tab = rope.table + (size_t)p * 64;
#pragma unroll 1
      for (int hc = 0; hc < BN; hc += 128) {  // the two heads of the tile
#pragma unroll 1
        for (int o = 0; o < 64; o += 32) {    // pairs (i, i + 64), 32 at a time
          float lo[32], hi[32];
          tmem_ld_32x32(taddr + (uint32_t)(hc + o), lo);
          tmem_ld_32x32(taddr + (uint32_t)(hc + o + 64), hi);
          if (row < M) {
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              const float4 cs = *reinterpret_cast<const float4 *>(tab + o + i);  // two (cos, sin)
              const float a0 = lo[i], b0 = hi[i], a1 = lo[i + 1], b1 = hi[i + 1];
              lo[i] = a0 * cs.x - b0 * cs.y;
              hi[i] = b0 * cs.x + a0 * cs.y;
              lo[i + 1] = a1 * cs.z - b1 * cs.w;
              hi[i + 1] = b1 * cs.z + a1 * cs.w;
            }
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
              Vec16<bf16> ol, oh;
              ol.pack(lo + j);
              oh.pack(hi + j);
              ol.store(dst + hc + o + j);
              oh.store(dst + hc + o + 64 + j);
            }
          }
        }
      }
      if (sect == 1 && col_in == 0 && row < M && rope.kv_pos) rope.kv_pos[krow] = p;
    }
  } else {
#pragma unroll 1
  for (int c = 0; c < TILE_N; c += 32) {
    float v[32];
    tmem_ld_32x32(taddr + (uint32_t)c, v);
    if (EPI == EPI_SWIGLU) {
      float u[32];
      tmem_ld_32x32(taddr + (uint32_t)(BN / 2 + c), u);
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = v[i] / (1.f + __expf(-v[i])) * u[i];
    }
    if (row < M) {
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        const int col = n0 + c + j;
        if (col < N) {  // N is a multiple of 8: a vector is entirely inside or outside
          float f[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) f[i] = v[j + i];
          if (EPI == EPI_RESIDUAL) {
            Vec16<bf16> rv;
            rv.load(rrow + col);
            float rf[8];
            rv.unpack(rf);
#pragma unroll
            for (int i = 0; i < 8; ++i) f[i] += rf[i];
          }
          Vec16<bf16> o;
          o.pack(f);
          o.store(crow + col);
        }
      }
    }
  }
  }  // epilogue kinds
}

// The same GEMM on CTA pairs (256x256 tiles, cta_group::2); epi is one of the EPI_* values.
int launch_gemm_pair(int epi, cudaStream_t st, const void *A, const void *B0, const void *B1, const void *R,
                     void *C, int M, int N, int K, DevStatus *status, const RopeArgs &rope);
// Clusters of two CTAs of that kernel the device can hold at once (-1: query failed).
int gemm_pair_max_clusters();

}  // namespace lazy
