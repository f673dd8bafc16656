// bf16 GEMM on CTA pairs: C[M,N] = A[M,K] * B[N,K]^T, one tcgen05.mma (cta_group::2, M256 N256 K16)
// spanning the tensor cores of two neighbouring SMs.
//
// A cluster of two persistent CTAs walks 256x256 output tiles.  CTA r of the pair owns rows
// [128 r, 128 r + 128) of the tile: it loads those rows of A and HALF of the B tile (128 of the 256
// weight rows) per K-slice, and ends up with its 128 x 256 fp32 accumulator in its own tensor memory.
// Against one CTA per 128x256 tile this halves the B bytes every SM pulls from L2 and reads from shared
// memory per MMA (32 KiB instead of 48 KiB per K-slice), and leaves room for a 6-stage ring.
//   warp 0      TMA producer in BOTH CTAs (own halves); all completion bytes of a stage are counted on
//               the leader's (rank 0) "full" barrier;
//   warp 1      allocates / frees TMEM in both CTAs (paired allocation); in the leader one lane issues the
//               MMAs and, by tcgen05.commit to the barrier of each CTA, releases ring stages ("empty") and
//               publishes finished accumulators ("tmem full");
//   warps 2-5   epilogue in both CTAs (same code as the one-CTA kernel); each warp reports a drained
//               accumulator to the leader's "tmem empty" barrier (8 arrivals).
// Every mbarrier wait is bounded; on expiry the CTA records LAZY_E_TIMEOUT, leaves its loops, meets its
// peer at the closing cluster barrier (which every path reaches) and frees its TMEM.
#include "gemm_epilogue.cuh"
#include "tc_pair.cuh"

namespace lazy {

namespace {

constexpr int PBM = 128;  // rows per CTA; 256 per pair
constexpr int PBN = GEMM_ACC_N, PBK = 64, PSTAGES = 6, PUMMA_K = 16;
constexpr int PA_BYTES = PBM * PBK * 2;        // 16 KiB: this CTA's rows of A
constexpr int PB_BYTES = (PBN / 2) * PBK * 2;  // 16 KiB: this CTA's half of the B tile
constexpr int PNUM_ACC = 2, PTMEM_COLS = 512, PTHREADS = 192;

struct __align__(8) PairBarriers {
  unsigned long long full[PSTAGES];        // used in the leader: bytes of both CTAs
  unsigned long long empty[PSTAGES];       // one per CTA, signalled by the leader's commits
  unsigned long long tmem_full[PNUM_ACC];  // one per CTA
  unsigned long long tmem_empty[PNUM_ACC]; // used in the leader: 4 epilogue warps x 2 CTAs
  uint32_t tmem_base;
  int abort_flag;
};
constexpr int PRING_BYTES = PSTAGES * (PA_BYTES + PB_BYTES);
// operand ring | output staging of the epilogue warps | barriers
constexpr int PAIR_SMEM_BYTES = PRING_BYTES + GEMM_STG_PER_CTA + 1024 /*align slack*/ + (int)sizeof(PairBarriers);
static_assert(PAIR_SMEM_BYTES <= 232448, "shared memory per CTA");

template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PTHREADS, 1)
gemm_bf16_tcgen05_pair_kernel(const __grid_constant__ CUtensorMap map_a,
                              const __grid_constant__ CUtensorMap map_b0,
                              const __grid_constant__ CUtensorMap map_b1,
                              const __grid_constant__ CUtensorMap map_c,
                         const __grid_constant__ CUtensorMap map_k,
                         const __grid_constant__ CUtensorMap map_v, const bf16 *__restrict__ R,
                              bf16 *__restrict__ C, int M, int N, int K, int ldc, DevStatus *status,
                              const RopeArgs rope, const GemmTail tail) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t pad = ((raw_addr + 1023u) & ~1023u) - raw_addr;  // same in both CTAs of the pair
  uint8_t *smem = smem_raw + pad;
  uint8_t *smem_a = smem;
  uint8_t *smem_b = smem + PSTAGES * PA_BYTES;
  PairBarriers *bars = reinterpret_cast<PairBarriers *>(smem + PRING_BYTES + GEMM_STG_PER_CTA);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_cta_rank();  // 0 = leader
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  constexpr int TILE_N_OUT = (EPI == EPI_SWIGLU) ? PBN / 2 : PBN;
  const int m_tiles = (M + 2 * PBM - 1) / (2 * PBM);
  const int n_tiles = (N + TILE_N_OUT - 1) / TILE_N_OUT;
  const int num_tiles = m_tiles * n_tiles;
  const int num_kb = (K + PBK - 1) / PBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < PSTAGES; ++s) {
      mbar_init(smem_u32(&bars->full[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), 1);
    }
    for (int a = 0; a < PNUM_ACC; ++a) {
      mbar_init(smem_u32(&bars->tmem_full[a]), 1);
      mbar_init(smem_u32(&bars->tmem_empty[a]), 8);
    }
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    tma_prefetch_desc(&map_a);
    tma_prefetch_desc(&map_b0);
    tma_prefetch_desc(&map_b1);
    tma_prefetch_desc(&map_c);
  }
  if (warp == 1) tmem_alloc_pair(smem_u32(&bars->tmem_base), PTMEM_COLS);  // same warp in both CTAs
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // both CTAs' barriers exist before anything signals across
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(&bars->tmem_base);
  volatile int *abort_flag = &bars->abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      GemmWork w;
      for (int it = 0; ok && gemm_work_item(it, pair, n_pairs, num_tiles, num_kb, tail, w); ++it) {
        int m_idx, n_idx;
        gemm_tile_coords(w.tile, m_tiles, n_tiles, tail.m_band, m_idx, n_idx);
        const int m0 = m_idx * (2 * PBM) + (int)rank * PBM, n0 = n_idx * TILE_N_OUT;
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          ok = mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, abort_flag, status, W_GEMM_PRODUCER);
          if (!ok) break;
          const uint32_t full_local = smem_u32(&bars->full[stage]);
          if (rank == 0) mbar_expect_tx(full_local, 2 * (PA_BYTES + PB_BYTES));
          const uint32_t full = cluster_map_shared(full_local, 0);
          tma_load_2d_pair(smem_u32(smem_a + stage * PA_BYTES), &map_a, full, kb * PBK, m0);
          const uint32_t bdst = smem_u32(smem_b + stage * PB_BYTES);
          if (EPI == EPI_SWIGLU) {  // leader holds the gate rows, its peer the matching up rows
            tma_load_2d_pair(bdst, rank == 0 ? &map_b0 : &map_b1, full, kb * PBK, n0);
          } else {
            tma_load_2d_pair(bdst, &map_b0, full, kb * PBK, n0 + (int)rank * (PBN / 2));
          }
          if (++stage == PSTAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = umma_idesc_bf16(2 * PBM, PBN);
      int stage = 0;
      uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      GemmWork w;
      for (; ok && gemm_work_item(local, pair, n_pairs, num_tiles, num_kb, tail, w); ++local) {
        const int acc = local & 1;
        const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
        ok = mbar_wait(smem_u32(&bars->tmem_empty[acc]), acc_phase ^ 1u, abort_flag, status, W_GEMM_MMA_TMEM);
        if (!ok) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * PBN);
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          ok = mbar_wait(smem_u32(&bars->full[stage]), phase, abort_flag, status, W_GEMM_MMA_FULL);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem_a + stage * PA_BYTES);
          const uint32_t b_addr = smem_u32(smem_b + stage * PB_BYTES);
#pragma unroll
          for (int k = 0; k < PBK / PUMMA_K; ++k) {
            const uint64_t adesc = umma_smem_desc(a_addr + k * PUMMA_K * 2);
            const uint64_t bdesc = umma_smem_desc(b_addr + k * PUMMA_K * 2);
            umma_bf16_pair(tmem_d, adesc, bdesc, idesc, (kb > w.kb0 || k > 0) ? 1u : 0u);
          }
          // the stage is reusable in both CTAs once these MMAs retire
          const uint32_t empty_local = smem_u32(&bars->empty[stage]);
          umma_commit_pair(cluster_map_shared(empty_local, 0));
          umma_commit_pair(cluster_map_shared(empty_local, 1));
          if (++stage == PSTAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) {
          const uint32_t tf_local = smem_u32(&bars->tmem_full[acc]);
          umma_commit_pair(cluster_map_shared(tf_local, 0));
          umma_commit_pair(cluster_map_shared(tf_local, 1));
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps (both CTAs)
    const int quarter = warp & 3;  // TMEM lanes [32*quarter, 32*quarter+32) belong to this warp
    int local = 0;
    bool ok = true;
    GemmWork w;
    EpiStore es = {&map_c, &map_k, &map_v, smem_u32(smem + PRING_BYTES) + (uint32_t)(quarter * 2 * GEMM_STG_BYTES), 0, 0u};
    for (; ok && gemm_work_item(local, pair, n_pairs, num_tiles, num_kb, tail, w); ++local) {
      const int acc = local & 1;
      const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
      int m_idx, n_idx;
      gemm_tile_coords(w.tile, m_tiles, n_tiles, tail.m_band, m_idx, n_idx);
      const int m0 = m_idx * (2 * PBM) + (int)rank * PBM, n0 = n_idx * TILE_N_OUT;
      const int row = m0 + quarter * 32 + lane;
      es.y0 = m0 + quarter * 32;
      uint4 res_first[GEMM_RES_AHEAD][4] = {};
      if (EPI == EPI_RESIDUAL && w.mode != 1)  // requested now, needed once the accumulator is complete
        gemm_residual_prefetch(res_first, R, rope, row, n0, M, N, ldc);
      ok = mbar_wait(smem_u32(&bars->tmem_full[acc]), acc_phase, abort_flag, status, W_GEMM_EPILOGUE);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * PBN);
      // split tiles: slot of pair p, rank r = CTA 2p + r; one arrival counter per (tail tile, rank)
      const int row_in_tile = quarter * 32 + lane;
      const int flag_idx = 2 * w.tail_idx + (int)rank;
      if (w.mode == 1) {
        gemm_dump_row(taddr, tail.partials + (size_t)(2 * pair + (int)rank) * GEMM_SLOT_FLOATS, row_in_tile);
        __threadfence();
        __syncwarp();
        if (lane == 0) {
          __threadfence();
          atomicAdd(tail.flags + flag_idx, 1u);
        }
      } else {
        if (w.mode == 2) {  // first part of a split tile: the other parts' sums come first
          const int n_parts = gemm_tail_dumps(pair, w.tail_idx, num_tiles, num_kb, tail);
          ok = gemm_tail_wait(tail.flags + flag_idx, 4u * (unsigned)n_parts, abort_flag, status);
          if (!ok) break;
          // the dumps of the following pairs, same rank: every second slot
          gemm_fixup_row(taddr, tail.partials + (size_t)(2 * (pair + 1) + (int)rank) * GEMM_SLOT_FLOATS, 2, n_parts,
                         smem, row_in_tile);
        }
        gemm_epilogue_row<EPI>(taddr, row, n0, M, N, ldc, R, C, rope, status, res_first, es);
        if (w.mode == 2) {
          __syncwarp();
          if (lane == 0 && atomicAdd(tail.done + flag_idx, 1u) == 3u) {
            tail.flags[flag_idx] = 0u;
            tail.done[flag_idx] = 0u;
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(cluster_map_shared(smem_u32(&bars->tmem_empty[acc]), 0));
    }
    epi_stage_drain();  // the staging buffers must not go away under a store that still reads them
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // neither CTA leaves (or frees TMEM) while its peer may still signal or compute into it
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, PTMEM_COLS);
  }
}

template <int EPI>
int launch_pair(cudaStream_t st, const void *A, const void *B0, const void *B1, const void *R, void *C, int M,
                int N, int K, DevStatus *status, const RopeArgs &rope, void *scratch, size_t scratch_bytes) {
  if ((K % 8) || (N % 8) || ((uintptr_t)A & 15) || ((uintptr_t)B0 & 15) || ((uintptr_t)B1 & 15) ||
      ((uintptr_t)C & 15) || ((uintptr_t)R & 15))
    return LAZY_E_BADARG;
  CUtensorMap ma, mb0, mb1;
  LAZY_TRY(tma_map_2d_bf16(&ma, A, M, K, K, PBK, PBM));
  LAZY_TRY(tma_map_2d_bf16(&mb0, B0, N, K, K, PBK, PBN / 2));
  LAZY_TRY(tma_map_2d_bf16(&mb1, B1, N, K, K, PBK, PBN / 2));
  CUtensorMap mc;  // the output: 64-column x 32-row boxes written from the epilogue's staging buffers
  LAZY_TRY(tma_map_2d_bf16(&mc, C, M, N, N, 64, 32));
  CUtensorMap mk = mc, mv = mc;  // QKV epilogue: rotated k and v go to the layer's cache rows
  if (EPI == EPI_QKV_ROPE && rope.kv_rows > 0) {
    if (((uintptr_t)rope.kcache & 15) || ((uintptr_t)rope.vcache & 15)) return LAZY_E_BADARG;
    LAZY_TRY(tma_map_2d_bf16(&mk, rope.kcache, rope.kv_rows, rope.d_kv, rope.d_kv, 64, 32));
    LAZY_TRY(tma_map_2d_bf16(&mv, rope.vcache, rope.kv_rows, rope.d_kv, rope.d_kv, 64, 32));
  }
  constexpr int TILE_N_OUT = (EPI == EPI_SWIGLU) ? PBN / 2 : PBN;
  const int tiles = cdiv(M, 2 * PBM) * cdiv(N, TILE_N_OUT);
  auto kfn = gemm_bf16_tcgen05_pair_kernel<EPI>;
  static int max_pairs = 0;  // co-resident clusters of two, asked once per kernel
  if (max_pairs == 0) {
    LAZY_CUDA_OK(cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, PAIR_SMEM_BYTES));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sm_count(), 1, 1);
    cfg.blockDim = dim3(PTHREADS, 1, 1);
    cfg.dynamicSmemBytes = PAIR_SMEM_BYTES;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kfn, &cfg) != cudaSuccess || n < 1) {
      cudaGetLastError();
      n = sm_count() / 2;
    }
    max_pairs = n < sm_count() / 2 ? n : sm_count() / 2;
  }
  const GemmTail tail = plan_tail(tiles, cdiv(K, PBK), max_pairs, 2, cdiv(M, 2 * PBM), gemm_m_band(M, K, 2 * PBM), M, K,
                                  EPI == EPI_SWIGLU ? 8 : 0, scratch, scratch_bytes);
  const int pairs = (tiles < max_pairs && tail.tail_units == 0) ? tiles : max_pairs;
  kfn<<<2 * pairs, PTHREADS, PAIR_SMEM_BYTES, st>>>(ma, mb0, mb1, mc, mk, mv, (const bf16 *)R, (bf16 *)C, M, N, K, N, status,
                                                    rope, tail);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

}  // namespace

int gemm_pair_max_clusters() {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(sm_count(), 1, 1);
  cfg.blockDim = dim3(PTHREADS, 1, 1);
  cfg.dynamicSmemBytes = PAIR_SMEM_BYTES;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  auto kfn = gemm_bf16_tcgen05_pair_kernel<EPI_PLAIN>;
  if (cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, PAIR_SMEM_BYTES) != cudaSuccess)
    return -1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kfn, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return n;
}

int launch_gemm_pair(int epi, cudaStream_t st, const void *A, const void *B0, const void *B1, const void *R,
                     void *C, int M, int N, int K, DevStatus *status, const RopeArgs &rope, void *scratch,
                     size_t scratch_bytes) {
  switch (epi) {
    case EPI_PLAIN: return launch_pair<EPI_PLAIN>(st, A, B0, B1, R, C, M, N, K, status, rope, scratch, scratch_bytes);
    case EPI_RESIDUAL: return launch_pair<EPI_RESIDUAL>(st, A, B0, B1, R, C, M, N, K, status, rope, scratch, scratch_bytes);
    case EPI_SWIGLU: return launch_pair<EPI_SWIGLU>(st, A, B0, B1, R, C, M, N, K, status, rope, scratch, scratch_bytes);
    case EPI_QKV_ROPE: return launch_pair<EPI_QKV_ROPE>(st, A, B0, B1, R, C, M, N, K, status, rope, scratch, scratch_bytes);
    default: return LAZY_E_BADARG;
  }
}

}  // namespace lazy
