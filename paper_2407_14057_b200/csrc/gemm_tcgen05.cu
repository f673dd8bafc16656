// bf16 GEMM on the 5th-generation tensor cores: C[M,N] = A[M,K] * B[N,K]^T with fp32
// accumulation in tensor memory (TMEM).
//
// One persistent CTA per SM walks 128x256 output tiles.  Warp roles:
//   warp 0      TMA producer: K-slices of A (128x64) and B (2 boxes of 128x64) into a 4-stage
//               ring of 128-byte-swizzled shared-memory tiles, completion on "full" mbarriers;
//   warp 1      owns TMEM (512 columns = two 128x256 fp32 accumulators) and issues
//               tcgen05.mma (M128 N256 K16) from one lane; tcgen05.commit releases ring stages
//               ("empty" barriers) and publishes finished accumulators ("tmem full");
//   warps 2-5   epilogue: tcgen05.ld their 32-lane quarter of the accumulator, apply the
//               epilogue (plain / + residual / SiLU(gate)*up / rotary), convert to bf16, stage 64-column
//               groups of the warp's 32 rows in shared memory and hand them to the TMA unit to store.
// The second accumulator lets the epilogue of tile i overlap the MMAs of tile i+1.
// Work items come from gemm_epilogue.cuh: whole tiles in a banded order, then, when it pays, K ranges
// of the last partial wave of tiles (a dumped partial accumulator, or the part that adds the dumps and
// finishes the tile).  The host side picks, per launch, this kernel or the CTA-pair kernel of
// gemm_tcgen05_pair.cu (gemm_use_pair), and the weight-streaming kernel for up to four rows.
// Ragged M, N, K rely on TMA zero fill for loads and on the TMA unit dropping what a store box holds
// beyond the matrix (row-by-row stores, where they remain, are predicated).
// Every mbarrier wait is bounded (wall-clock limit); on expiry the kernel records
// LAZY_E_TIMEOUT in the status word, every role leaves its loop, TMEM is released and the CTA
// exits.  No cluster launch, no multicast.
#include "gemm_epilogue.cuh"

namespace lazy {

namespace {

static_assert(GEMM_ACC_N == 256, "tile width");

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4, UMMA_K = 16;
constexpr int A_STAGE_BYTES = BM * BK * 2;       // 16 KiB
constexpr int B_STAGE_BYTES = BN * BK * 2;       // 32 KiB
constexpr int B_HALF_BYTES = B_STAGE_BYTES / 2;  // one 128-row TMA box
constexpr int NUM_ACC = 2;
constexpr int TMEM_COLS = 512;
constexpr int GEMM_THREADS = 192;

struct __align__(8) GemmBarriers {
  unsigned long long full[STAGES];
  unsigned long long empty[STAGES];
  unsigned long long tmem_full[NUM_ACC];
  unsigned long long tmem_empty[NUM_ACC];
  uint32_t tmem_base;
  int abort_flag;
};
constexpr int RING_BYTES = STAGES * (A_STAGE_BYTES + B_STAGE_BYTES);
// operand ring | output staging of the epilogue warps | barriers
constexpr int GEMM_SMEM_BYTES = RING_BYTES + GEMM_STG_PER_CTA + 1024 /*align slack*/ + (int)sizeof(GemmBarriers);
static_assert(GEMM_SMEM_BYTES <= 232448, "shared memory per CTA");

// C is [M, ldc]; for EPI_SWIGLU the accumulator's columns [0,128) are gate features and
// [128,256) the matching up features, and C receives 128 columns per tile.
// FP8: A and B hold e4m3 codes (one byte each): a stage is still 128-byte rows, now 128 elements of K, and the
// MMA is kind::f8f6f4 with K = 32 per instruction; the epilogue applies the operands' scales.
template <int EPI, bool FP8>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_bf16_tcgen05_kernel(const __grid_constant__ CUtensorMap map_a,
                         const __grid_constant__ CUtensorMap map_b0,
                         const __grid_constant__ CUtensorMap map_b1,
                         const __grid_constant__ CUtensorMap map_c,
                         const __grid_constant__ CUtensorMap map_k,
                         const __grid_constant__ CUtensorMap map_v, const bf16 *__restrict__ R,
                         bf16 *__restrict__ C, int M, int N, int K, int ldc, DevStatus *status,
                         const RopeArgs rope, const GemmTail tail) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t pad = ((raw_addr + 1023u) & ~1023u) - raw_addr;
  uint8_t *smem = smem_raw + pad;  // 1024-byte aligned: required by the 128B swizzle atoms
  uint8_t *smem_a = smem;
  uint8_t *smem_b = smem + STAGES * A_STAGE_BYTES;
  GemmBarriers *bars = reinterpret_cast<GemmBarriers *>(smem + RING_BYTES + GEMM_STG_PER_CTA);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Output tiles: columns per tile as seen by the caller.
  constexpr int TILE_N_OUT = (EPI == EPI_SWIGLU) ? BN / 2 : BN;
  const int m_tiles = (M + BM - 1) / BM;
  const int n_tiles = (N + TILE_N_OUT - 1) / TILE_N_OUT;
  const int num_tiles = m_tiles * n_tiles;
  constexpr int BKE = FP8 ? 2 * BK : BK;  // elements of K per stage (128 bytes per row either way)
  const int num_kb = (K + BKE - 1) / BKE;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bars->full[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), 1);
    }
    for (int a = 0; a < NUM_ACC; ++a) {
      mbar_init(smem_u32(&bars->tmem_full[a]), 1);
      mbar_init(smem_u32(&bars->tmem_empty[a]), 4);  // one arrival per epilogue warp
    }
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    tma_prefetch_desc(&map_a);
    tma_prefetch_desc(&map_b0);
    tma_prefetch_desc(&map_b1);
    tma_prefetch_desc(&map_c);
  }
  if (warp == 1) {  // TMEM allocation by one whole warp; the same warp frees it at the end
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&bars->tmem_base)),
                 "r"((uint32_t)TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(&bars->tmem_base);
  volatile int *abort_flag = &bars->abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      GemmWork w;
      for (int it = 0; ok && gemm_work_item(it, blockIdx.x, gridDim.x, num_tiles, num_kb, tail, w); ++it) {
        int m_idx, n_idx;
        gemm_tile_coords(w.tile, m_tiles, n_tiles, tail.m_band, m_idx, n_idx);
        const int m0 = m_idx * BM, n0 = n_idx * TILE_N_OUT;
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          ok = mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, abort_flag, status, W_GEMM_PRODUCER);
          if (!ok) break;
          const uint32_t full = smem_u32(&bars->full[stage]);
          mbar_expect_tx(full, A_STAGE_BYTES + B_STAGE_BYTES);
          tma_load_2d(smem_u32(smem_a + stage * A_STAGE_BYTES), &map_a, full, kb * BKE, m0);
          const uint32_t bdst = smem_u32(smem_b + stage * B_STAGE_BYTES);
          if (EPI == EPI_SWIGLU) {
            tma_load_2d(bdst, &map_b0, full, kb * BKE, n0);
            tma_load_2d(bdst + B_HALF_BYTES, &map_b1, full, kb * BKE, n0);
          } else {
            tma_load_2d(bdst, &map_b0, full, kb * BKE, n0);
            tma_load_2d(bdst + B_HALF_BYTES, &map_b0, full, kb * BKE, n0 + BN / 2);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = FP8 ? umma_idesc_e4m3(BM, BN) : umma_idesc_bf16(BM, BN);
      int stage = 0;
      uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      GemmWork w;
      for (; ok && gemm_work_item(local, blockIdx.x, gridDim.x, num_tiles, num_kb, tail, w); ++local) {
        const int acc = local & 1;
        const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
        ok = mbar_wait(smem_u32(&bars->tmem_empty[acc]), acc_phase ^ 1u, abort_flag, status, W_GEMM_MMA_TMEM);
        if (!ok) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * BN);
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          ok = mbar_wait(smem_u32(&bars->full[stage]), phase, abort_flag, status, W_GEMM_MMA_FULL);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem_a + stage * A_STAGE_BYTES);
          const uint32_t b_addr = smem_u32(smem_b + stage * B_STAGE_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t adesc = umma_smem_desc(a_addr + k * UMMA_K * 2);
            const uint64_t bdesc = umma_smem_desc(b_addr + k * UMMA_K * 2);
            if (FP8) umma_f8(tmem_d, adesc, bdesc, idesc, (kb > w.kb0 || k > 0) ? 1u : 0u);
            else umma_bf16(tmem_d, adesc, bdesc, idesc, (kb > w.kb0 || k > 0) ? 1u : 0u);
          }
          umma_commit(smem_u32(&bars->empty[stage]));  // stage reusable once these MMAs retire
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(smem_u32(&bars->tmem_full[acc]));
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int quarter = warp & 3;  // TMEM lanes [32*quarter, 32*quarter+32) belong to this warp
    int local = 0;
    bool ok = true;
    GemmWork w;
    EpiStore es = {&map_c, &map_k, &map_v, smem_u32(smem + RING_BYTES) + (uint32_t)(quarter * 2 * GEMM_STG_BYTES), 0, 0u};
    for (; ok && gemm_work_item(local, blockIdx.x, gridDim.x, num_tiles, num_kb, tail, w); ++local) {
      const int acc = local & 1;
      const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
      int m_idx, n_idx;
      gemm_tile_coords(w.tile, m_tiles, n_tiles, tail.m_band, m_idx, n_idx);
      const int m0 = m_idx * BM, n0 = n_idx * TILE_N_OUT;
      const int row = m0 + quarter * 32 + lane;
      uint4 res_first[GEMM_RES_AHEAD][4] = {};
      if (EPI == EPI_RESIDUAL && w.mode != 1)  // requested now, needed once the accumulator is complete
        gemm_residual_prefetch(res_first, R, rope, row, n0, M, N, ldc);
      ok = mbar_wait(smem_u32(&bars->tmem_full[acc]), acc_phase, abort_flag, status, W_GEMM_EPILOGUE);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
      const int row_in_tile = quarter * 32 + lane;
      if (w.mode == 1) {  // partial accumulator of a split tile: to this CTA's slot, then tell the finisher
        gemm_dump_row(taddr, tail.partials + (size_t)blockIdx.x * GEMM_SLOT_FLOATS, row_in_tile);
        __threadfence();
        __syncwarp();
        if (lane == 0) {
          __threadfence();
          atomicAdd(tail.flags + w.tail_idx, 1u);
        }
      } else {
        if (w.mode == 2) {  // first part of a split tile: the other parts' sums come first
          const int n_parts = gemm_tail_dumps(blockIdx.x, w.tail_idx, num_tiles, num_kb, tail);
          ok = gemm_tail_wait(tail.flags + w.tail_idx, 4u * (unsigned)n_parts, abort_flag, status);
          if (!ok) break;
          gemm_fixup_row(taddr, tail.partials + (size_t)(blockIdx.x + 1) * GEMM_SLOT_FLOATS, 1, n_parts, smem,
                         row_in_tile);
        }
        es.y0 = m0 + quarter * 32;
        gemm_epilogue_row<EPI>(taddr, row, n0, M, N, ldc, R, C, rope, status, res_first, es);
        if (w.mode == 2) {
          __syncwarp();
          if (lane == 0 && atomicAdd(tail.done + w.tail_idx, 1u) == 3u) {  // last warp through: clean for the next launch
            tail.flags[w.tail_idx] = 0u;
            tail.done[w.tail_idx] = 0u;
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->tmem_empty[acc]));
    }
    epi_stage_drain();  // the staging buffers must not go away under a store that still reads them
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"((uint32_t)TMEM_COLS)
                 : "memory");
  }
}

// ---- host side -----------------------------------------------------------------------------------
// Which kernel takes a product of more than one row tile: the one whose launch is estimated shorter.
// Both cover the same outputs per wave (148 tiles of 128 rows, or 74 pair tiles of 256 rows); what differs is
// how the row count pads to 128 / 256, how many waves that makes, what the split last wave recovers, and the
// pair kernel's measured ~6 % shorter wave on the plain / residual / QKV epilogues (none on SwiGLU, whose
// epilogue dominates the difference).  Measured against both kernels at 1013-23112 rows of the 7B widths the
// estimate picks the faster one except within ~2 %.  force: 1 = one CTA per tile, 2 = CTA pairs (the
// cross-check entry points), 0 = by the estimate.
bool gemm_use_pair(int epi, int M, int N, int K, void *scratch, size_t scratch_bytes, int force) {
  static int max_pairs = -1;
  if (max_pairs < 0) {
    int n = gemm_pair_max_clusters();
    if (n > sm_count() / 2) n = sm_count() / 2;
    max_pairs = n < 0 ? 0 : n;
  }
  if (M <= BM || force == 1 || max_pairs < 1) return false;
  if (force == 2) return true;
  const int tile_n = epi == EPI_SWIGLU ? BN / 2 : BN, extra = epi == EPI_SWIGLU ? 8 : 0, num_kb = cdiv(K, BK);
  double w_one = 0, w_pair = 0;
  plan_tail(cdiv(M, BM) * cdiv(N, tile_n), num_kb, sm_count(), 1, cdiv(M, BM), gemm_m_band(M, K, BM), M, K, extra,
            scratch, scratch_bytes, &w_one);
  plan_tail(cdiv(M, 2 * BM) * cdiv(N, tile_n), num_kb, max_pairs, 2, cdiv(M, 2 * BM), gemm_m_band(M, K, 2 * BM), M, K,
            extra, scratch, scratch_bytes, &w_pair);
  const double pair_wave = 0.95;
  return w_pair * pair_wave < w_one;  // a pair tile takes pair_wave x the time of a one-CTA tile
}

// FP8: A [M, K] and B0 / B1 [N, K] hold e4m3 codes (bytes), rope.a_scale / w_scale their scales; always the
// one-CTA kernel.
template <int EPI, bool FP8 = false>
int launch_tc(cudaStream_t st, const void *A, const void *B0, const void *B1, const void *R, void *C,
              int M, int N, int K, DevStatus *status, const RopeArgs &rope, void *scratch,
              size_t scratch_bytes, int force_kernel) {
  // TMA needs 16-byte aligned bases and row pitches; the epilogue stores 8 columns at a time.
  if ((K % (FP8 ? 16 : 8)) || (N % 8) || ((uintptr_t)A & 15) || ((uintptr_t)B0 & 15) || ((uintptr_t)B1 & 15) ||
      ((uintptr_t)C & 15) || ((uintptr_t)R & 15))
    return LAZY_E_BADARG;
  if (!FP8 && gemm_use_pair(EPI, M, N, K, scratch, scratch_bytes, force_kernel))
    return launch_gemm_pair(EPI, st, A, B0, B1, R, C, M, N, K, status, rope, scratch, scratch_bytes);
  constexpr int EB = FP8 ? 1 : 2, BKE = FP8 ? 2 * BK : BK;  // element bytes, elements of K per 128-byte stage row
  CUtensorMap ma, mb0, mb1;
  LAZY_TRY(tma_map_2d(&ma, A, M, K, K, BKE, BM, EB));
  LAZY_TRY(tma_map_2d(&mb0, B0, N, K, K, BKE, BN / 2, EB));
  LAZY_TRY(tma_map_2d(&mb1, B1, N, K, K, BKE, BN / 2, EB));
  CUtensorMap mc;  // the output: 64-column x 32-row boxes written from the epilogue's staging buffers
  LAZY_TRY(tma_map_2d_bf16(&mc, C, M, N, N, 64, 32));
  CUtensorMap mk = mc, mv = mc;  // QKV epilogue: rotated k and v go to the layer's cache rows
  if (EPI == EPI_QKV_ROPE && rope.kv_rows > 0) {
    if (((uintptr_t)rope.kcache & 15) || ((uintptr_t)rope.vcache & 15)) return LAZY_E_BADARG;
    LAZY_TRY(tma_map_2d_bf16(&mk, rope.kcache, rope.kv_rows, rope.d_kv, rope.d_kv, 64, 32));
    LAZY_TRY(tma_map_2d_bf16(&mv, rope.vcache, rope.kv_rows, rope.d_kv, rope.d_kv, 64, 32));
  }
  constexpr int TILE_N_OUT = (EPI == EPI_SWIGLU) ? BN / 2 : BN;
  const int tiles = cdiv(M, BM) * cdiv(N, TILE_N_OUT);
  const GemmTail tail = plan_tail(tiles, cdiv(K, BKE), sm_count(), 1, cdiv(M, BM), gemm_m_band(M, K, BM), M, K,
                                  EPI == EPI_SWIGLU ? 8 : 0, scratch,
                                  scratch_bytes);
  const int grid = (tiles < sm_count() && tail.tail_units == 0) ? tiles : sm_count();
  auto kfn = gemm_bf16_tcgen05_kernel<EPI, FP8>;
  static bool attr_set = false;
  if (!attr_set) {
    LAZY_CUDA_OK(cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_BYTES));
    attr_set = true;
  }
  kfn<<<grid, GEMM_THREADS, GEMM_SMEM_BYTES, st>>>(ma, mb0, mb1, mc, mk, mv, (const bf16 *)R, (bf16 *)C, M, N, K, N,
                                                  status, rope, tail);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

}  // namespace

// Sized for up to 160 persistent CTAs whatever the device (the size is asked for without one, too); with
// more SMs than that the kernels fall back to the plain tile loop.
size_t gemm_scratch_bytes() { return gemm_tail_scratch_bytes(GEMM_TAIL_MAX_CTAS); }

int launch_gemm(cudaStream_t st, int dtype, const void *A, const void *B, const void *R, void *C,
                int M, int N, int K, DevStatus *status, void *scratch, size_t scratch_bytes, int force_kernel,
                bool b_const, const int32_t *res_rows) {
  if (M == 0) return LAZY_OK;
  if (res_rows && (!gemm_res_rows_supported(dtype, M, K) || !R || R == C)) return LAZY_E_BADARG;
  if (dtype == LAZY_F32) return launch_gemm_simt(st, dtype, A, B, nullptr, R, C, M, N, K, 0);
  if (gemv_small_m_eligible(dtype, M, K))
    return launch_gemv_small_m(st, A, B, nullptr, R, C, M, N, K, 0, nullptr, 0.f, 0, b_const);
  if (R) {
    RopeArgs extra = {};
    extra.res_rows = res_rows;
    return launch_tc<EPI_RESIDUAL>(st, A, B, B, R, C, M, N, K, status, extra, scratch, scratch_bytes, force_kernel);
  }
  return launch_tc<EPI_PLAIN>(st, A, B, B, nullptr, C, M, N, K, status, RopeArgs(), scratch, scratch_bytes,
                              force_kernel);
}

// 8-bit products: A8 [M, K] and B8 [N, K] are e4m3 codes, a_scale [M] the per-row scales of A, w_scale the
// scale of B (w_scale_up of the second matrix of a SwiGLU product).  epi: EPI_PLAIN (R NULL) / EPI_RESIDUAL /
// EPI_SWIGLU (B8 = gate, B8u = up, N = features) / EPI_QKV_ROPE (extra carries the rotary operands).
int launch_gemm_fp8(cudaStream_t st, int epi, const void *A8, const float *a_scale, const void *B8, float w_scale,
                    const void *B8u, float w_scale_up, const void *R, void *C, int M, int N, int K, DevStatus *status,
                    RopeArgs extra, void *scratch, size_t scratch_bytes) {
  if (M == 0) return LAZY_OK;
  if (!a_scale) return LAZY_E_BADARG;
  extra.a_scale = a_scale;
  extra.w_scale = w_scale;
  extra.w_scale_up = w_scale_up;
  switch (epi) {
    case EPI_PLAIN:
      return launch_tc<EPI_PLAIN, true>(st, A8, B8, B8, nullptr, C, M, N, K, status, extra, scratch, scratch_bytes, 1);
    case EPI_RESIDUAL:
      return launch_tc<EPI_RESIDUAL, true>(st, A8, B8, B8, R, C, M, N, K, status, extra, scratch, scratch_bytes, 1);
    case EPI_SWIGLU:
      return launch_tc<EPI_SWIGLU, true>(st, A8, B8, B8u, nullptr, C, M, N, K, status, extra, scratch, scratch_bytes, 1);
    case EPI_QKV_ROPE:
      return launch_tc<EPI_QKV_ROPE, true>(st, A8, B8, B8, nullptr, C, M, N, K, status, extra, scratch, scratch_bytes, 1);
    default: return LAZY_E_BADARG;
  }
}

// The residual row list exists in the tensor-core epilogue only.
bool gemm_res_rows_supported(int dtype, int M, int K) {
  return dtype == LAZY_BF16 && !gemv_small_m_eligible(dtype, M, K);
}

bool gemm_qkv_rope_eligible(int dtype, int d_model, int head_dim, int d_kv) {
  if (d_kv <= 0) d_kv = d_model;
  return dtype == LAZY_BF16 && head_dim == 128 && d_model % BN == 0 && d_kv % BN == 0;
}

int launch_gemm_qkv_rope(cudaStream_t st, const void *h, const void *w_qkv, void *qkv, const int32_t *pos,
                         const float *table, void *kcache, void *vcache, int32_t *kv_pos,
                         const int32_t *kv_row, int M, int d_model, int max_pos, DevStatus *status,
                         void *scratch, size_t scratch_bytes, int d_kv, int kv_rows) {
  if (M == 0) return LAZY_OK;
  if (d_kv <= 0) d_kv = d_model;
  RopeArgs r;
  r.kv_rows = kv_rows > 0 ? kv_rows : 0;  // 0: extent unknown, k and v are stored row by row
  r.d_kv = d_kv;
  r.pos = pos;
  r.table = (const float2 *)table;
  r.kcache = (bf16 *)kcache;
  r.vcache = (bf16 *)vcache;
  r.kv_pos = kv_pos;
  r.kv_row = kv_row;
  r.d_model = d_model;
  r.max_pos = max_pos;
  return launch_tc<EPI_QKV_ROPE>(st, h, w_qkv, w_qkv, nullptr, qkv, M, d_model + 2 * d_kv, d_model, status, r, scratch,
                                 scratch_bytes, 0);
}

int launch_gemm_swiglu(cudaStream_t st, int dtype, const void *A, const void *Bg, const void *Bu,
                       void *C, int M, int F, int K, DevStatus *status, void *scratch, size_t scratch_bytes,
                       int force_kernel, bool b_const) {
  if (M == 0) return LAZY_OK;
  if (dtype == LAZY_F32) return launch_gemm_simt(st, dtype, A, Bg, Bu, nullptr, C, M, F, K, 1);
  if (gemv_small_m_eligible(dtype, M, K))
    return launch_gemv_small_m(st, A, Bg, Bu, nullptr, C, M, F, K, 1, nullptr, 0.f, 0, b_const);
  return launch_tc<EPI_SWIGLU>(st, A, Bg, Bu, nullptr, C, M, F, K, status, RopeArgs(), scratch, scratch_bytes,
                               force_kernel);
}

}  // namespace lazy
