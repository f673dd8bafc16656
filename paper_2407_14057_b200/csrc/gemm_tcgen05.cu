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
//               epilogue (plain / + residual / SiLU(gate)*up), convert to bf16, 16-byte stores.
// The second accumulator lets the epilogue of tile i overlap the MMAs of tile i+1.
// Ragged M, N, K rely on TMA zero fill for loads and on predicated stores.
// Every mbarrier wait is bounded (wall-clock limit); on expiry the kernel records
// LAZY_E_TIMEOUT in the status word, every role leaves its loop, TMEM is released and the CTA
// exits.  No cluster launch, no multicast.
#include <cuda.h>

#include "common.cuh"

namespace lazy {

namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4, UMMA_K = 16;
constexpr int A_STAGE_BYTES = BM * BK * 2;       // 16 KiB
constexpr int B_STAGE_BYTES = BN * BK * 2;       // 32 KiB
constexpr int B_HALF_BYTES = B_STAGE_BYTES / 2;  // one 128-row TMA box
constexpr int NUM_ACC = 2;
constexpr int TMEM_COLS = 512;
constexpr int GEMM_THREADS = 192;
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;  // 2 s per wait

struct __align__(8) GemmBarriers {
  unsigned long long full[STAGES];
  unsigned long long empty[STAGES];
  unsigned long long tmem_full[NUM_ACC];
  unsigned long long tmem_empty[NUM_ACC];
  uint32_t tmem_base;
  int abort_flag;
};
constexpr int GEMM_SMEM_BYTES = STAGES * (A_STAGE_BYTES + B_STAGE_BYTES) + 1024 /*align slack*/ +
                                (int)sizeof(GemmBarriers);

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false when the limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          DevStatus *status, int where) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_timer_ns();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (*abort_flag) return false;
      if (global_timer_ns() - t0 > WAIT_LIMIT_NS) {
        *abort_flag = 1;
        dev_fail(status, LAZY_E_TIMEOUT, where, (int)blockIdx.x, (int)parity);
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t smem_dst, const CUtensorMap *map, uint32_t bar,
                                            int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_dst), "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap *map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// Shared-memory matrix descriptor: K-major operand tile of 128-byte rows, 128B swizzle,
// 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);  // start address
  d |= (uint64_t)1 << 16;                        // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;              // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                        // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                        // 128-byte swizzle
  return d;
}
// Instruction descriptor, kind::f16: D fp32, A and B bf16, both K-major.
__device__ __forceinline__ uint32_t umma_idesc_bf16(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread i of the warp receives lane (base + i).
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, float *v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
        "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
        "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
        "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

enum { EPI_PLAIN = 0, EPI_RESIDUAL = 1, EPI_SWIGLU = 2 };

// C is [M, ldc]; for EPI_SWIGLU the accumulator's columns [0,128) are gate features and
// [128,256) the matching up features, and C receives 128 columns per tile.
template <int EPI>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_bf16_tcgen05_kernel(const __grid_constant__ CUtensorMap map_a,
                         const __grid_constant__ CUtensorMap map_b0,
                         const __grid_constant__ CUtensorMap map_b1, const bf16 *__restrict__ R,
                         bf16 *__restrict__ C, int M, int N, int K, int ldc, DevStatus *status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t pad = ((raw_addr + 1023u) & ~1023u) - raw_addr;
  uint8_t *smem = smem_raw + pad;  // 1024-byte aligned: required by the 128B swizzle atoms
  uint8_t *smem_a = smem;
  uint8_t *smem_b = smem + STAGES * A_STAGE_BYTES;
  GemmBarriers *bars = reinterpret_cast<GemmBarriers *>(smem + STAGES * (A_STAGE_BYTES + B_STAGE_BYTES));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Output tiles: columns per tile as seen by the caller.
  constexpr int TILE_N_OUT = (EPI == EPI_SWIGLU) ? BN / 2 : BN;
  const int m_tiles = (M + BM - 1) / BM;
  const int n_tiles = (N + TILE_N_OUT - 1) / TILE_N_OUT;
  const int num_tiles = m_tiles * n_tiles;
  const int num_kb = (K + BK - 1) / BK;

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
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile % m_tiles) * BM;
        const int n0 = (tile / m_tiles) * TILE_N_OUT;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, abort_flag, status, W_GEMM_PRODUCER);
          if (!ok) break;
          const uint32_t full = smem_u32(&bars->full[stage]);
          mbar_expect_tx(full, A_STAGE_BYTES + B_STAGE_BYTES);
          tma_load_2d(smem_u32(smem_a + stage * A_STAGE_BYTES), &map_a, full, kb * BK, m0);
          const uint32_t bdst = smem_u32(smem_b + stage * B_STAGE_BYTES);
          if (EPI == EPI_SWIGLU) {
            tma_load_2d(bdst, &map_b0, full, kb * BK, n0);
            tma_load_2d(bdst + B_HALF_BYTES, &map_b1, full, kb * BK, n0);
          } else {
            tma_load_2d(bdst, &map_b0, full, kb * BK, n0);
            tma_load_2d(bdst + B_HALF_BYTES, &map_b0, full, kb * BK, n0 + BN / 2);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(BM, BN);
      int stage = 0;
      uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++local) {
        const int acc = local & 1;
        const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
        ok = mbar_wait(smem_u32(&bars->tmem_empty[acc]), acc_phase ^ 1u, abort_flag, status, W_GEMM_MMA_TMEM);
        if (!ok) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = mbar_wait(smem_u32(&bars->full[stage]), phase, abort_flag, status, W_GEMM_MMA_FULL);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem_a + stage * A_STAGE_BYTES);
          const uint32_t b_addr = smem_u32(smem_b + stage * B_STAGE_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t adesc = umma_smem_desc(a_addr + k * UMMA_K * 2);
            const uint64_t bdesc = umma_smem_desc(b_addr + k * UMMA_K * 2);
            umma_bf16(tmem_d, adesc, bdesc, idesc, (kb | k) != 0 ? 1u : 0u);
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
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++local) {
      const int acc = local & 1;
      const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
      const int m0 = (tile % m_tiles) * BM;
      const int n0 = (tile / m_tiles) * TILE_N_OUT;
      ok = mbar_wait(smem_u32(&bars->tmem_full[acc]), acc_phase, abort_flag, status, W_GEMM_EPILOGUE);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int row = m0 + quarter * 32 + lane;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
      bf16 *crow = C + (size_t)row * ldc;
      const bf16 *rrow = (EPI == EPI_RESIDUAL) ? R + (size_t)row * ldc : nullptr;
#pragma unroll 1
      for (int c = 0; c < TILE_N_OUT; c += 32) {
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
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->tmem_empty[acc]));
    }
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
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Row-major bf16 matrix [rows, cols] (cols contiguous), box = 64 columns x box_rows rows.
int make_map(CUtensorMap *map, const void *base, int rows, int cols, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return LAZY_E_CUDA;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides,
                  box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? LAZY_OK : LAZY_E_CUDA;
}

template <int EPI>
int launch_tc(cudaStream_t st, const void *A, const void *B0, const void *B1, const void *R, void *C,
              int M, int N, int K, DevStatus *status) {
  // TMA needs 16-byte aligned bases and row pitches; the epilogue stores 8 columns at a time.
  if ((K % 8) || (N % 8) || ((uintptr_t)A & 15) || ((uintptr_t)B0 & 15) || ((uintptr_t)B1 & 15) ||
      ((uintptr_t)C & 15) || ((uintptr_t)R & 15))
    return LAZY_E_BADARG;
  CUtensorMap ma, mb0, mb1;
  LAZY_TRY(make_map(&ma, A, M, K, BM));
  LAZY_TRY(make_map(&mb0, B0, N, K, BN / 2));
  LAZY_TRY(make_map(&mb1, B1, N, K, BN / 2));
  constexpr int TILE_N_OUT = (EPI == EPI_SWIGLU) ? BN / 2 : BN;
  const int tiles = cdiv(M, BM) * cdiv(N, TILE_N_OUT);
  const int grid = tiles < sm_count() ? tiles : sm_count();
  auto kfn = gemm_bf16_tcgen05_kernel<EPI>;
  static bool attr_set = false;
  if (!attr_set) {
    LAZY_CUDA_OK(cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_BYTES));
    attr_set = true;
  }
  kfn<<<grid, GEMM_THREADS, GEMM_SMEM_BYTES, st>>>(ma, mb0, mb1, (const bf16 *)R, (bf16 *)C, M, N, K, N,
                                                  status);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

}  // namespace

int launch_gemm(cudaStream_t st, int dtype, const void *A, const void *B, const void *R, void *C,
                int M, int N, int K, DevStatus *status) {
  if (M == 0) return LAZY_OK;
  if (dtype == LAZY_F32) return launch_gemm_simt(st, dtype, A, B, nullptr, R, C, M, N, K, 0);
  if (R) return launch_tc<EPI_RESIDUAL>(st, A, B, B, R, C, M, N, K, status);
  return launch_tc<EPI_PLAIN>(st, A, B, B, nullptr, C, M, N, K, status);
}

int launch_gemm_swiglu(cudaStream_t st, int dtype, const void *A, const void *Bg, const void *Bu,
                       void *C, int M, int F, int K, DevStatus *status) {
  if (M == 0) return LAZY_OK;
  if (dtype == LAZY_F32) return launch_gemm_simt(st, dtype, A, Bg, Bu, nullptr, C, M, F, K, 1);
  return launch_tc<EPI_SWIGLU>(st, A, Bg, Bu, nullptr, C, M, F, K, status);
}

}  // namespace lazy
