// Epilogues of the bf16 tensor-core GEMMs: what a thread does with its row of a finished 128x256
// fp32 accumulator tile in tensor memory.  Shared by the one-CTA and the CTA-pair kernels.
#pragma once
#include "tc_common.cuh"

namespace lazy {

constexpr int GEMM_ACC_N = 256;  // accumulator columns per tile

enum { EPI_PLAIN = 0, EPI_RESIDUAL = 1, EPI_SWIGLU = 2, EPI_QKV_ROPE = 3 };

// Extra operands of the epilogues.  QKV: the rotary embedding is applied to the fp32 accumulators and
// the rotated k, and v, go straight to the layer's cache rows (head_dim 128: one 256-column tile is
// two whole heads of q, k or v, and a thread holds its row's full heads).  Residual: an optional row
// list for the addend, so that C[r] = acc[r] + R[res_rows[r]] compacts the residual stream on the way.
struct RopeArgs {
  const int32_t *res_rows = nullptr;  // [M] row of R added to output row r (NULL: r)
  const int32_t *pos;     // [M] original positions
  const float2 *table;    // [max_pos][64] (cos, sin)
  bf16 *kcache, *vcache;  // [kv_rows, d_kv]
  int kv_rows = 0;        // rows of the two caches (extent of their tensor maps)
  int32_t *kv_pos;        // position tag per cache row (may be NULL)
  const int32_t *kv_row;  // cache row of GEMM row r (NULL: r)
  int d_model, max_pos;
  int d_kv;               // width of a K / V cache row: n_kv_heads * head_dim (= d_model without grouping)
  // 8-bit operands: the accumulator of row r is the product of e4m3 codes and is multiplied by
  // a_scale[r] * w_scale on the way out (SwiGLU: gate columns by w_scale, up columns by w_scale_up)
  const float *a_scale = nullptr;
  float w_scale = 1.f, w_scale_up = 1.f;
};

// ---- the last, partial wave ------------------------------------------------------------------------------
// num_tiles is rarely a multiple of the number of persistent units (CTAs, or CTA pairs), so a plain
// tile loop ends with a wave in which most units idle for a whole tile time.  Instead the K loops of the
// last (num_tiles - first_tail) tiles are laid end to end and cut into tail_units equal ranges, one per
// unit.  A range touches at most two tiles: the end of one (a DUMP: the fp32 partial accumulator goes to
// the unit's slot of `partials`) and the start of the next (the FINISH part: it waits for the dumps of the
// units after it that cover the same tile, adds them in unit order - deterministic - and runs the normal
// epilogue).  A dump never waits, and every unit dumps before it finishes, so no wait is circular; all
// units are resident at once (persistent grid), and the wait is time-bounded anyway.
constexpr int GEMM_TAIL_MIN_KB = 8;               // shortest K range (in 64-wide slices) worth a part
constexpr int GEMM_SLOT_FLOATS = 128 * GEMM_ACC_N;  // one CTA's accumulator

struct GemmTail {
  float *partials;   // [CTAs][128][256] fp32
  unsigned *flags;   // [tail tiles x ranks] dump arrivals (one per epilogue warp); zero between launches
  unsigned *done;    // [tail tiles x ranks] finisher warps through; the last one re-zeroes both
  int first_tail;    // tiles [first_tail, num_tiles) are split along K; num_tiles: nothing is
  int tail_units;    // units that share them
  int m_band;        // row tiles per band of the tile order (see gemm_tile_coords); >= m_tiles: one band
};

// Tile order.  Consecutive tile numbers walk the row tiles of one column block, so the units of a wave
// share a B (weight) tile and read different A tiles.  With very many rows (packed batches, long prompts)
// one sweep over all row tiles no longer fits in L2 and A would come from HBM once per column block:
// the row tiles are therefore taken in bands of m_band, each band walking all column blocks before the
// next band starts (A band + one wave of B stay L2-resident; B is re-read once per band instead).
__device__ __forceinline__ void gemm_tile_coords(int tile, int m_tiles, int n_tiles, int m_band, int &m_idx,
                                                 int &n_idx) {
  if (m_band >= m_tiles) {
    m_idx = tile % m_tiles;
    n_idx = tile / m_tiles;
    return;
  }
  const int per_band = m_band * n_tiles;
  const int band = tile / per_band, r = tile - band * per_band;
  const int rows = min(m_band, m_tiles - band * m_band);  // the last band may be short
  n_idx = r / rows;
  m_idx = band * m_band + (r - n_idx * rows);
}

// Row tiles per band for tiles of tile_rows rows: one band while A (M x K bf16) is under 96 MiB, else
// about 64 MiB of A per band.
inline int gemm_m_band(long long M, long long K, int tile_rows) {
  if (M * K * 2 <= (96ll << 20)) return 1 << 30;
  const long long t = (64ll << 20) / (K * 2) / tile_rows;
  return (int)(t < 4 ? 4 : t);
}

// Scratch layout: 2 x GEMM_TAIL_MAX_CTAS counters (2 KiB), then one accumulator slot per persistent CTA.
constexpr int GEMM_TAIL_MAX_CTAS = 160;
constexpr size_t GEMM_TAIL_COUNTER_BYTES = 2048;
static_assert(2 * GEMM_TAIL_MAX_CTAS * sizeof(unsigned) <= GEMM_TAIL_COUNTER_BYTES, "counter block");
inline size_t gemm_tail_scratch_bytes(int ctas) {
  return GEMM_TAIL_COUNTER_BYTES + (size_t)ctas * GEMM_SLOT_FLOATS * 4;
}

struct GemmWork {
  int tile, kb0, kb1;
  int mode;      // 0: whole tile, 1: dump, 2: finish
  int tail_idx;  // index among the tail tiles
};

__device__ __forceinline__ int gemm_tail_start(int u, int tail_units, int total_kb) {
  return (int)(((long long)u * total_kb) / tail_units);
}

// i-th work item of unit u of `units`; false when the unit has no more.
__device__ __forceinline__ bool gemm_work_item(int i, int u, int units, int num_tiles, int num_kb,
                                               const GemmTail &t, GemmWork &w) {
  const int n_whole = u < t.first_tail ? (t.first_tail - u + units - 1) / units : 0;
  if (i < n_whole) {
    w.tile = u + i * units;
    w.kb0 = 0;
    w.kb1 = num_kb;
    w.mode = 0;
    w.tail_idx = 0;
    return true;
  }
  if (t.first_tail >= num_tiles || u >= t.tail_units) return false;
  const int total = (num_tiles - t.first_tail) * num_kb;
  const int s = gemm_tail_start(u, t.tail_units, total), e = gemm_tail_start(u + 1, t.tail_units, total);
  const int t0 = s / num_kb;
  const int e0 = min(e, (t0 + 1) * num_kb);
  int a, b, tt;
  if (i == n_whole) {
    a = s; b = e0; tt = t0;
  } else if (i == n_whole + 1) {
    a = e0; b = e; tt = t0 + 1;
  } else {
    return false;
  }
  if (b <= a) return false;
  w.tile = t.first_tail + tt;
  w.kb0 = a - tt * num_kb;
  w.kb1 = b - tt * num_kb;
  w.mode = w.kb0 != 0 ? 1 : (w.kb1 == num_kb ? 0 : 2);
  w.tail_idx = tt;
  return true;
}

// Units after u whose range starts inside tail tile tt: each holds one dump for it.
__device__ __forceinline__ int gemm_tail_dumps(int u, int tt, int num_tiles, int num_kb, const GemmTail &t) {
  const int total = (num_tiles - t.first_tail) * num_kb;
  int n = 0;
  for (int v = u + 1; v < t.tail_units && gemm_tail_start(v, t.tail_units, total) < (tt + 1) * num_kb; ++v) ++n;
  return n;
}

// A slot holds one CTA's 128 x 256 accumulator as [column quad q = col/4][row][4 floats]: a warp (32
// consecutive rows) then moves 512 contiguous bytes per instruction, in the dump and in the fix-up.
__device__ __forceinline__ void gemm_dump_row(uint32_t taddr, float *slot, int row_in_tile) {
#pragma unroll 1
  for (int c = 0; c < GEMM_ACC_N; c += 32) {
    float v[32];
    tmem_ld_32x32(taddr + (uint32_t)c, v);
#pragma unroll
    for (int j = 0; j < 8; ++j)
      *reinterpret_cast<float4 *>(slot + ((size_t)(c / 4 + j) * 128 + row_in_tile) * 4) =
          make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
  }
}

// Fix-up of a split tile, one thread per accumulator row: the n_parts dumps (slots slot0, slot0 +
// slot_step, ...) are added, in that order, into the row's accumulator in tensor memory, after which the
// ordinary epilogue runs as if the tile had been computed whole.  Each dump is first pulled into shared
// memory with cp.async (64 x 16 bytes per thread in flight at once, where plain loads into registers would
// leave the fix-up latency-bound); `stage` is 128 KiB of this CTA's operand ring, idle once the tile's last
// MMA has retired (which the accumulator-full barrier has already told the caller).  A thread reads back
// only what it copied itself, so no barrier is needed between the copy and the adds.
__device__ __forceinline__ void gemm_fixup_row(uint32_t taddr, const float *slot0, int slot_step, int n_parts,
                                               uint8_t *stage, int row_in_tile) {
  const uint32_t sbase = smem_u32(stage) + (uint32_t)row_in_tile * 16u;
  for (int p = 0; p < n_parts; ++p) {
    const float *src = slot0 + (size_t)p * slot_step * GEMM_SLOT_FLOATS + (size_t)row_in_tile * 4;
#pragma unroll 8
    for (int q = 0; q < GEMM_ACC_N / 4; ++q)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sbase + (uint32_t)q * 2048u),
                   "l"(src + (size_t)q * 512)
                   : "memory");
    asm volatile("cp.async.wait_all;" ::: "memory");
#pragma unroll 1
    for (int c = 0; c < GEMM_ACC_N; c += 32) {
      float v[32];
      tmem_ld_32x32(taddr + (uint32_t)c, v);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float4 x;
        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                     : "=f"(x.x), "=f"(x.y), "=f"(x.z), "=f"(x.w)
                     : "r"(sbase + (uint32_t)(c / 4 + j) * 2048u)
                     : "memory");
        v[4 * j] += x.x;
        v[4 * j + 1] += x.y;
        v[4 * j + 2] += x.z;
        v[4 * j + 3] += x.w;
      }
      tmem_st_32x32(taddr + (uint32_t)c, reinterpret_cast<const uint32_t *>(v));
    }
    tmem_st_wait();
  }
}

// Warp-level, bounded wait until *flag >= target.  False (and the abort flag set) on expiry.
__device__ __forceinline__ bool gemm_tail_wait(const unsigned *flag, unsigned target, volatile int *abort_flag,
                                               DevStatus *status, unsigned long long limit_ns = WAIT_LIMIT_NS) {
  int ok = 1;
  if ((threadIdx.x & 31) == 0) {
    const unsigned long long t0 = global_timer_ns();
    uint32_t spins = 0;
    for (;;) {
      unsigned v;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
      if (v >= target) break;
      if ((++spins & 63u) == 0) {
        if (*abort_flag) { ok = 0; break; }
        if (global_timer_ns() - t0 > limit_ns) {
          *abort_flag = 1;
          dev_fail(status, LAZY_E_TIMEOUT, W_GEMM_TAIL, (int)blockIdx.x, (int)v);
          ok = 0;
          break;
        }
      }
    }
  }
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// Residual addend of the 32 output columns [col0, col0 + 32) of a row, as four 16-byte vectors (a vector
// beyond N, or a row beyond M, is left as it is).  These reads are row-strided (a thread owns a row), and a
// group that is only asked for when the group before it is being worked on costs a full L2 round trip per
// group: measured, a 256-column tile then spent ~14 000 clocks in its residual epilogue, nearly all of it
// waiting.  So a thread keeps GEMM_RES_AHEAD groups in flight: the first ones are requested before it waits
// for the tile's accumulator, and each group consumed is replaced by the request GEMM_RES_AHEAD groups on.
constexpr int GEMM_RES_AHEAD = 8;
__device__ __forceinline__ void gemm_residual_load(uint4 (&r)[4], const bf16 *__restrict__ R, const RopeArgs &extra,
                                                   int row, int col0, int M, int N, int ldc) {
  if (row >= M) return;
  const bf16 *rrow = R + (size_t)(extra.res_rows ? extra.res_rows[row] : row) * ldc;
#pragma unroll
  for (int j = 0; j < 4; ++j)
    if (col0 + 8 * j < N) r[j] = *reinterpret_cast<const uint4 *>(rrow + col0 + 8 * j);
}
// The first GEMM_RES_AHEAD groups of a tile whose first output column is n0.
__device__ __forceinline__ void gemm_residual_prefetch(uint4 (&r)[GEMM_RES_AHEAD][4], const bf16 *__restrict__ R,
                                                       const RopeArgs &extra, int row, int n0, int M, int N, int ldc) {
#pragma unroll
  for (int g = 0; g < GEMM_RES_AHEAD; ++g) gemm_residual_load(r[g], R, extra, row, n0 + 32 * g, M, N, ldc);
}

// Output staging of an epilogue warp.  A thread owns a row, so storing straight from registers makes every
// warp-wide store touch 32 different rows with 16 bytes each: measured, a 256-column tile's stores then took
// 8 000-9 000 clocks (more when all CTAs end a launch together), most of a tile's epilogue.  Instead the
// warp writes 64-column groups of its 32 rows into a 4 KiB shared-memory buffer in the 128-byte-swizzled
// layout and one lane hands the buffer to the TMA unit, which writes whole 128-byte lines and drops what
// lies beyond M or N.  Two buffers alternate, so a group is staged while the one before it drains.
constexpr int GEMM_STG_BYTES = 4096;                       // 32 rows x 64 bf16
constexpr int GEMM_STG_PER_CTA = 4 * 2 * GEMM_STG_BYTES;   // four epilogue warps, two buffers each
struct EpiStore {
  const CUtensorMap *map;  // the output matrix: box 64 columns x 32 rows, 128-byte swizzle
  const CUtensorMap *map_k, *map_v;  // QKV epilogue: the layer's K and V caches (same box), else unused
  uint32_t stg;            // shared-memory address of this warp's two buffers (1024-byte aligned)
  int y0;                  // first output row of the warp's 32-row block of the current tile
  uint32_t n_out;          // groups handed over so far: the next group takes buffer n_out & 1
};
// Buffer for the next group, free to be written (the store that last read it has done so).
__device__ __forceinline__ uint32_t epi_stage_begin(const EpiStore &es) {
  if ((threadIdx.x & 31) == 0) bulk_wait_group_read<1>();
  __syncwarp();
  return es.stg + (es.n_out & 1u) * GEMM_STG_BYTES;
}
// 16-byte chunk j (columns 8j .. 8j+7 of the group) of this thread's row.
__device__ __forceinline__ void epi_stage_put(uint32_t buf, int j, const uint4 &v) {
  const uint32_t lane = threadIdx.x & 31;
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(buf + lane * 128u + (((uint32_t)j ^ (lane & 7u)) << 4)),
               "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
               : "memory");
}
// Hands the staged group to the TMA unit: columns [x, x + 64) of rows [y0, y0 + 32).
__device__ __forceinline__ void epi_stage_commit(EpiStore &es, uint32_t buf, const CUtensorMap *map, int x, int y) {
  fence_proxy_async_smem();
  __syncwarp();
  if ((threadIdx.x & 31) == 0) {
    tma_store_2d(map, buf, x, y);
    bulk_commit_group();
  }
  ++es.n_out;
}
__device__ __forceinline__ void epi_stage_commit(EpiStore &es, uint32_t buf, int x) {
  epi_stage_commit(es, buf, es.map, x, es.y0);
}
// Before the CTA exits: every store of this warp has completed.
__device__ __forceinline__ void epi_stage_drain() {
  if ((threadIdx.x & 31) == 0) bulk_wait_group_all();
  __syncwarp();
}

// One thread, one row.  taddr: TMEM address of the row's first accumulator column (lane field set);
// row: global output row; n0: first output column of the tile as the caller sees it.  C is [M, ldc];
// for EPI_SWIGLU accumulator columns [0,128) are gate features, [128,256) the matching up features and C
// receives 128 columns per tile.
template <int EPI>
__device__ __forceinline__ void gemm_epilogue_row(uint32_t taddr, int row, int n0, int M, int N, int ldc,
                                                  const bf16 *__restrict__ R, bf16 *__restrict__ C,
                                                  const RopeArgs &rope, DevStatus *status,
                                                  uint4 (&res_q)[GEMM_RES_AHEAD][4], EpiStore &es) {
  // res_q (EPI_RESIDUAL): the addends of the tile's first column groups, requested by the caller ahead of time
  constexpr int BN = GEMM_ACC_N;
  constexpr int TILE_N = (EPI == EPI_SWIGLU) ? BN / 2 : BN;
  bf16 *crow = C + (size_t)row * ldc;
  if (EPI == EPI_QKV_ROPE) {
    // section of the fused projection this tile belongs to: 0 = q, 1 = k, 2 = v
    // output columns are [q: d_model | k: d_kv | v: d_kv]
    const int sect = n0 < rope.d_model ? 0 : (n0 < rope.d_model + rope.d_kv ? 1 : 2);
    const int col_in = n0 - (sect == 0 ? 0 : (sect == 1 ? rope.d_model : rope.d_model + rope.d_kv));
    int p = 0;
    size_t krow = 0;
    bool kv_valid = true;  // false: the row's cache row lies outside the caches; its k / v are dropped
    if (row < M) {
      p = rope.pos[row];
      if (p < 0 || p >= rope.max_pos) {
        dev_fail(status, LAZY_E_CAPACITY, W_ROPE_POS, row, p);
        p = 0;
      }
      krow = rope.kv_row ? (size_t)rope.kv_row[row] : (size_t)row;
      // a cache row outside the caches (a corrupted row table) is reported, and the row's k / v are dropped
      // instead of being stored out of range (a box store must not start at such a row either)
      if (rope.kv_rows > 0 && krow >= (size_t)rope.kv_rows) {
        dev_fail(status, LAZY_E_CAPACITY, W_ROPE_POS, row, (int)krow);
        kv_valid = false;
        krow = 0;
      }
    }
    const float osc = (rope.a_scale && row < M) ? rope.a_scale[row] * rope.w_scale : 1.f;
    bf16 *dst = sect == 0 ? crow + n0
                          : (sect == 1 ? rope.kcache : rope.vcache) + krow * rope.d_kv + col_in;
    // Where the warp's 32 rows go as one box: q always (rows of C); k and v when all 32 rows are real and
    // their cache rows are consecutive (one sequence, or a block inside one sequence of a packed batch).
    // Otherwise k / v are stored row by row from registers.
    const size_t krow0 = __shfl_sync(0xffffffffu, krow, 0);
    const bool block_ok = rope.kv_rows > 0 && krow0 + 32 <= (size_t)rope.kv_rows &&
                          __all_sync(0xffffffffu, row < M && kv_valid && krow == krow0 + (size_t)(threadIdx.x & 31));
    const bool staged = sect == 0 || block_ok;
    const CUtensorMap *omap = sect == 0 ? es.map : (sect == 1 ? es.map_k : es.map_v);
    const int ox = sect == 0 ? n0 : col_in, oy = sect == 0 ? es.y0 : (int)krow0;
    if (sect == 2) {
#pragma unroll 1
      for (int c = 0; c < BN; c += 32) {
        float v[32];
        tmem_ld_32x32(taddr + (uint32_t)c, v);
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] *= osc;
        if (staged) {
          uint32_t buf = es.stg + (es.n_out & 1u) * GEMM_STG_BYTES;
          if ((c & 32) == 0) buf = epi_stage_begin(es);
#pragma unroll
          for (int j = 0; j < 32; j += 8) {
            Vec16<bf16> o;
            o.pack(v + j);
            epi_stage_put(buf, ((c & 32) >> 3) + (j >> 3), o.raw);
          }
          if (c & 32) epi_stage_commit(es, buf, omap, ox + c - 32, oy);
        } else if (row < M && kv_valid) {
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
        // a head goes out through both staging buffers: columns [0,64) in the first, [64,128) in the second
        if (staged) {
          if ((threadIdx.x & 31) == 0) bulk_wait_group_read<0>();
          __syncwarp();
        }
#pragma unroll 1
        for (int o = 0; o < 64; o += 32) {    // pairs (i, i + 64), 32 at a time
          float lo[32], hi[32];
          tmem_ld_32x32(taddr + (uint32_t)(hc + o), lo);
          tmem_ld_32x32(taddr + (uint32_t)(hc + o + 64), hi);
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float4 cs = *reinterpret_cast<const float4 *>(tab + o + i);  // two (cos, sin)
            const float a0 = lo[i] * osc, b0 = hi[i] * osc, a1 = lo[i + 1] * osc, b1 = hi[i + 1] * osc;
            lo[i] = a0 * cs.x - b0 * cs.y;
            hi[i] = b0 * cs.x + a0 * cs.y;
            lo[i + 1] = a1 * cs.z - b1 * cs.w;
            hi[i + 1] = b1 * cs.z + a1 * cs.w;
          }
          if (staged) {
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
              Vec16<bf16> ol, oh;
              ol.pack(lo + j);
              oh.pack(hi + j);
              epi_stage_put(es.stg, (o >> 3) + (j >> 3), ol.raw);
              epi_stage_put(es.stg + GEMM_STG_BYTES, (o >> 3) + (j >> 3), oh.raw);
            }
          } else if (row < M && kv_valid) {
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
        if (staged) {
          fence_proxy_async_smem();
          __syncwarp();
          if ((threadIdx.x & 31) == 0) {
            tma_store_2d(omap, es.stg, ox + hc, oy);
            tma_store_2d(omap, es.stg + GEMM_STG_BYTES, ox + hc + 64, oy);
            bulk_commit_group();
          }
          es.n_out += 2;
        }
      }
      if (sect == 1 && col_in == 0 && row < M && kv_valid && rope.kv_pos) rope.kv_pos[krow] = p;
    }
  } else {
  const float asc = (rope.a_scale && row < M) ? rope.a_scale[row] : 1.f;
  const float osc = asc * rope.w_scale, osc_up = asc * rope.w_scale_up;
  // fully unrolled with the residual epilogue, whose ring of requested groups is indexed statically
#pragma unroll(EPI == EPI_RESIDUAL ? TILE_N / 32 : 1)
  for (int c = 0; c < TILE_N; c += 32) {
    float v[32];
    tmem_ld_32x32(taddr + (uint32_t)c, v);
    if (rope.a_scale) {
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] *= osc;
    }
    if (EPI == EPI_SWIGLU) {
      float u[32];
      tmem_ld_32x32(taddr + (uint32_t)(BN / 2 + c), u);
      if (rope.a_scale) {
#pragma unroll
        for (int i = 0; i < 32; ++i) u[i] *= osc_up;
      }
#pragma unroll
      // SiLU(g) * u with the approximate reciprocal: the IEEE division cost ~100 clocks per element of a
      // thread's row here (a tile's epilogue was compute-bound at ~15 000 clocks), and the result is rounded
      // to bf16 anyway
      for (int i = 0; i < 32; ++i) v[i] = __fdividef(v[i], 1.f + __expf(-v[i])) * u[i];
    }
    uint4 res_cur[4];
    if (EPI == EPI_RESIDUAL) {
      constexpr int kGroups = TILE_N / 32;
      const int g = (c >> 5) % GEMM_RES_AHEAD;  // static after unrolling
#pragma unroll
      for (int j = 0; j < 4; ++j) res_cur[j] = res_q[g][j];
      if ((c >> 5) + GEMM_RES_AHEAD < kGroups)
        gemm_residual_load(res_q[g], R, rope, row, n0 + c + 32 * GEMM_RES_AHEAD, M, N, ldc);
    }
    // the 32 columns go to the staging buffer of their 64-column group (rows beyond M and columns beyond N
    // are staged too and dropped by the store)
    uint32_t buf = es.stg + (es.n_out & 1u) * GEMM_STG_BYTES;
    if ((c & 32) == 0) buf = epi_stage_begin(es);
#pragma unroll
    for (int j = 0; j < 32; j += 8) {
      float f[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) f[i] = v[j + i];
      if (EPI == EPI_RESIDUAL) {
        Vec16<bf16> rv;
        rv.raw = res_cur[j >> 3];
        float rf[8];
        rv.unpack(rf);
#pragma unroll
        for (int i = 0; i < 8; ++i) f[i] += rf[i];
      }
      Vec16<bf16> o;
      o.pack(f);
      epi_stage_put(buf, ((c & 32) >> 3) + (j >> 3), o.raw);
    }
    if (c & 32) epi_stage_commit(es, buf, n0 + c - 32);
  }
  }  // epilogue kinds
}

// Splits the last partial wave along K when that pays: `units` persistent units of `cta_per_unit` CTAs,
// m_tiles row tiles, M x K activations.  Costs are in K slices (one slice of MMAs ~ 0.4 us): a split tile
// is charged 3 slices for its dump and 4 for each part its finisher adds (extra_cost more for a heavy
// epilogue), tiles are cut into at most four parts, and only when the wave then ends earlier than 95 % of a
// whole tile.  (Swept on the four projections at 1013-3376 rows: with the charges at 6 / 10 and the bar at
// 80 % the output and down projections at 2364 rows ran whole waves and took 87 / 198 us instead of 78 /
// 176 us.)  The parts of
// the tiles of one column block run skewed in K, so the B rows of the tail must stay L2-resident (next to
// A) or they are re-read from HBM.  scratch NULL or too small, or no gain: plain tile loop.
inline GemmTail plan_tail(int num_tiles, int num_kb, int units, int cta_per_unit, int m_tiles, int m_band,
                          long long M, long long K, int extra_cost, void *scratch, size_t scratch_bytes,
                          double *waves = nullptr) {
  GemmTail t = {};
  t.first_tail = num_tiles;
  t.tail_units = 0;
  t.m_band = m_band;
  // *waves: the launch's length in whole-tile times (for the choice between the two kernels)
  if (waves) *waves = (double)((num_tiles + units - 1) / units);
  if (m_band < m_tiles) m_tiles = m_tiles % m_band ? m_tiles % m_band : m_band;  // the tail lies in the last band
  if (!scratch || units * cta_per_unit > GEMM_TAIL_MAX_CTAS ||
      scratch_bytes < gemm_tail_scratch_bytes(units * cta_per_unit))
    return t;
  const int first = (num_tiles / units) * units, rem = num_tiles - first;
  if (rem == 0) return t;
  const long long b_tail = (long long)((rem + m_tiles - 1) / m_tiles + 1) * GEMM_ACC_N * K * 2;
  const long long a_rows = M < (long long)m_tiles * 256 ? M : (long long)m_tiles * 256;  // rows of the tail's band
  if (m_tiles > 2 && b_tail + a_rows * K * 2 > 96ll << 20) return t;  // one or two row tiles: B is read once anyway
  int best_units = 0;
  long long best_cost = (long long)num_kb * 19 / 20;
  for (int parts = 2; parts <= 4; ++parts) {
    long long tu = (long long)rem * parts;
    if (tu > units) tu = units;
    if (tu <= rem) continue;
    const long long per_unit = ((long long)rem * num_kb + tu - 1) / tu;
    if (per_unit < GEMM_TAIL_MIN_KB) continue;
    const bool aligned = tu == (long long)rem * parts;  // ranges end on tile boundaries
    const long long pieces = aligned ? parts : (num_kb + per_unit - 1) / per_unit + 1;
    const long long cost = per_unit + 3 + 4 * (pieces - 1) + extra_cost;
    if (cost < best_cost) {
      best_cost = cost;
      best_units = (int)tu;
    }
  }
  if (best_units == 0) return t;
  if (waves) *waves = (double)(num_tiles / units) + (double)best_cost / (double)num_kb;
  t.flags = (unsigned *)scratch;
  t.done = t.flags + GEMM_TAIL_MAX_CTAS;
  t.partials = (float *)((char *)scratch + GEMM_TAIL_COUNTER_BYTES);
  t.first_tail = first;
  t.tail_units = best_units;
  return t;
}

// The same GEMM on CTA pairs (256x256 tiles, cta_group::2); epi is one of the EPI_* values.
int launch_gemm_pair(int epi, cudaStream_t st, const void *A, const void *B0, const void *B1, const void *R,
                     void *C, int M, int N, int K, DevStatus *status, const RopeArgs &rope, void *scratch,
                     size_t scratch_bytes);
// 8-bit products (e4m3 codes with scales; see gemm_tcgen05.cu).
int launch_gemm_fp8(cudaStream_t st, int epi, const void *A8, const float *a_scale, const void *B8, float w_scale,
                    const void *B8u, float w_scale_up, const void *R, void *C, int M, int N, int K, DevStatus *status,
                    RopeArgs extra, void *scratch, size_t scratch_bytes);
// Clusters of two CTAs of that kernel the device can hold at once (-1: query failed).
int gemm_pair_max_clusters();

}  // namespace lazy
