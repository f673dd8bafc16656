// Causal attention on the 5th-generation tensor cores (bf16, head_dim 128, prefill form: query
// row i of a sequence sees keys 0..i of the same sequence).
//
// One CTA = 128 query rows of one head; two CTAs share an SM (96 KiB of shared memory and 256
// TMEM columns each), so that one CTA's softmax overlaps the other's MMAs.  Warp roles:
//   warp 0     TMA: Q once (two 128x64 boxes), then 64-key tiles of K and of V (two 64x64 boxes
//              each) into two 2-stage rings with their own barriers (one lane per ring);
//   warp 1     owns TMEM and issues the S MMAs from one lane (warp 6 the P V MMAs):
//                S_j = Q K_j^T   (M128 N64 K16 x 8, operands in shared memory, both K-major)
//                O  += P_j V_j   (M128 N128 K16 x 4, A = P_j read from TMEM, B = V_j as an
//                                 MN-major shared-memory operand: V stays [key][dh] as loaded)
//              TMEM columns: S (64) | P of even tiles (32) | P of odd tiles (32) | O (128).  P has its
//              own columns, so the single S buffer is free again as soon as the softmax threads
//              have loaded S_j into registers ("s free"): S_{j+1} is then issued at once and is
//              computed underneath the exponentials of tile j, and P_j V_j is issued the moment P_j
//              arrives.  (With P written over a double-buffered S, S_{j+2} had to wait for
//              P_j V_j to retire, and the softmax threads sat waiting for S 38 % of the time.)
//   warp 6     issues P_j V_j from one lane (its own thread: a chain of MMAs blocks its issuer while
//              the pipe takes it, and S_{j+1} must not queue behind that);
//   warps 2-5  softmax: thread = query row (TMEM lane).  tcgen05.ld its 64 logits, mask the
//              diagonal tile, running max / sum in registers, P_j packed to bf16 pairs and written
//              to the tile's P columns with tcgen05.st (once P_{j-1} V_{j-1} has retired).  The running max is only raised when
//              it grows by more than 2^8 (then O is rescaled in TMEM after the previous P V
//              retired); otherwise P is allowed to exceed 1, which fp32/bf16 ranges absorb.
//              After the last tile: O / l -> bf16 -> global.
// Rows past the sequence end are read as zeros (the tensor maps end there) or as other rows'
// finite data and are never stored.  Every mbarrier wait is bounded and reports LAZY_E_TIMEOUT.
#include "attn_common.cuh"

namespace lazy {

namespace {

constexpr int TQ = 128, TK = 64, HD = 128, KV_STAGES = 2;
constexpr int Q_BYTES = TQ * HD * 2;       // 32 KiB: two [128][64] blocks
constexpr int KV_TILE_BYTES = TK * HD * 2; // 16 KiB: two [64][64] blocks
constexpr int Q_BLK = TQ * 64 * 2;         // 16 KiB
constexpr int KV_BLK = TK * 64 * 2;        // 8 KiB
constexpr int ATT_TMEM_COLS = 256;         // S (64) | P even (32) | P odd (32) | O (128 columns)
constexpr int ATT_THREADS = 224;          // TMA warp, S-issuing warp, 4 softmax warps, P V-issuing warp
constexpr float RESCALE_LOG2 = 8.f;

struct __align__(8) AttBarriers {
  unsigned long long q_full;
  unsigned long long k_full[KV_STAGES];
  unsigned long long k_empty[KV_STAGES];
  unsigned long long v_full[KV_STAGES];
  unsigned long long v_empty[KV_STAGES];
  unsigned long long s_full;   // S_j computed (phase j)
  unsigned long long s_free;   // S_j loaded into registers by all four softmax warps (phase j)
  unsigned long long p_full[2];
  // P_j V_j retired; one barrier per P buffer (tile parity), phase index j >> 1.  A parity wait can
  // only tell a phase from the one before it, so a waiter must never lag two phases: tile j+2 cannot
  // retire on pv_done[j & 1] before P_{j+2} exists, and the softmax threads await P_j V_j before they
  // write P_{j+2}, so every wait below is for the barrier's current or just-completed phase.
  unsigned long long pv_done[2];
  uint32_t tmem_base;
  int abort_flag;
};
constexpr int ATT_SMEM_BYTES = Q_BYTES + KV_STAGES * 2 * KV_TILE_BYTES + 1024 + (int)sizeof(AttBarriers);

}  // namespace

namespace {

__global__ void __launch_bounds__(ATT_THREADS, 2)
attn_tcgen05_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, bf16 *__restrict__ o, int ldo,
                    const int32_t *__restrict__ cu_q, const int32_t *__restrict__ kv_base, int q_start_arg,
                    int n_arg, int kv_start_arg, DevStatus *status, const AttnScoreOut sc, int kv_group) {
  extern __shared__ uint8_t att_smem_raw[];
  const uint32_t raw_addr = smem_u32(att_smem_raw);
  const uint32_t pad = ((raw_addr + 1023u) & ~1023u) - raw_addr;
  uint8_t *smem = att_smem_raw + pad;
  const uint32_t sQ = smem_u32(smem);
  const uint32_t sK = sQ + Q_BYTES;                          // stage s at + s * KV_TILE_BYTES
  const uint32_t sV = sK + KV_STAGES * KV_TILE_BYTES;
  AttBarriers *bars = reinterpret_cast<AttBarriers *>(smem + Q_BYTES + KV_STAGES * 2 * KV_TILE_BYTES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Heads are the fastest grid dimension and query tiles run from the longest to the shortest along y, so
  // CTAs are handed out longest first over ALL heads: the long tiles of the last head start with the first
  // wave instead of at the end of the launch.
  const int h = blockIdx.x;
  const int hk = h / kv_group;  // key/value head this query head reads (grouped-query attention)
  int q_start = q_start_arg, n = n_arg, kv_start = kv_start_arg;
  if (cu_q) {
    q_start = cu_q[blockIdx.z];
    n = cu_q[blockIdx.z + 1] - q_start;
    kv_start = kv_base ? kv_base[blockIdx.z] : q_start;
  }
  const int q_tiles = (n + TQ - 1) / TQ;
  if ((int)blockIdx.y >= q_tiles) return;          // before any barrier or TMEM use: safe to leave
  const int qt = q_tiles - 1 - blockIdx.y;         // longest rows first
  const int q0 = qt * TQ;
  const int n_kt = (min(q0 + TQ, n) + TK - 1) / TK;  // key tiles up to the diagonal

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bars->q_full), 1);
    for (int s = 0; s < KV_STAGES; ++s) {
      mbar_init(smem_u32(&bars->k_full[s]), 1);
      mbar_init(smem_u32(&bars->k_empty[s]), 1);
      mbar_init(smem_u32(&bars->v_full[s]), 1);
      mbar_init(smem_u32(&bars->v_empty[s]), 1);
    }
    mbar_init(smem_u32(&bars->s_full), 1);
    mbar_init(smem_u32(&bars->s_free), 4);       // one arrival per softmax warp
    for (int b = 0; b < 2; ++b) mbar_init(smem_u32(&bars->p_full[b]), 4);
    for (int b = 0; b < 2; ++b) mbar_init(smem_u32(&bars->pv_done[b]), 1);
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    tma_prefetch_desc(&map_q);
    tma_prefetch_desc(&map_k);
    tma_prefetch_desc(&map_v);
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&bars->tmem_base)),
                 "r"((uint32_t)ATT_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(&bars->tmem_base);
  volatile int *abort_flag = &bars->abort_flag;
  const uint32_t tmem_o = tmem_base + 128u;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producers
    // Lane 0 streams Q and the K tiles, lane 1 the V tiles.  A K stage is free as soon as S_j has
    // been computed, a V stage once P_j V_j has: K_{j+2} is then in flight long before it is needed.
    if (lane == 0) {
      const uint32_t qf = smem_u32(&bars->q_full);
      mbar_expect_tx(qf, Q_BYTES);
      tma_load_2d(sQ, &map_q, qf, h * HD, q_start + q0);
      tma_load_2d(sQ + Q_BLK, &map_q, qf, h * HD + 64, q_start + q0);
      for (int j = 0; j < n_kt; ++j) {
        const int st = j & 1;
        const uint32_t ph = (uint32_t)(j >> 1) & 1u;
        if (!mbar_wait(smem_u32(&bars->k_empty[st]), ph ^ 1u, abort_flag, status, W_ATTN_PRODUCER)) break;
        const uint32_t full = smem_u32(&bars->k_full[st]);
        mbar_expect_tx(full, KV_TILE_BYTES);
        const int row = kv_start + j * TK;
        tma_load_2d(sK + st * KV_TILE_BYTES, &map_k, full, hk * HD, row);
        tma_load_2d(sK + st * KV_TILE_BYTES + KV_BLK, &map_k, full, hk * HD + 64, row);
      }
    } else if (lane == 1) {
      for (int j = 0; j < n_kt; ++j) {
        const int st = j & 1;
        const uint32_t ph = (uint32_t)(j >> 1) & 1u;
        if (!mbar_wait(smem_u32(&bars->v_empty[st]), ph ^ 1u, abort_flag, status, W_ATTN_PRODUCER)) break;
        const uint32_t full = smem_u32(&bars->v_full[st]);
        mbar_expect_tx(full, KV_TILE_BYTES);
        const int row = kv_start + j * TK;
        tma_load_2d(sV + st * KV_TILE_BYTES, &map_v, full, hk * HD, row);
        tma_load_2d(sV + st * KV_TILE_BYTES + KV_BLK, &map_v, full, hk * HD + 64, row);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc_s = idesc_bf16(TQ, TK, 0, 0);
      bool ok = mbar_wait(smem_u32(&bars->q_full), 0, abort_flag, status, W_ATTN_MMA);
      auto issue_s = [&](int j) -> bool {
        const int st = j & 1;
        if (!mbar_wait(smem_u32(&bars->k_full[st]), (uint32_t)(j >> 1) & 1u, abort_flag, status, W_ATTN_MMA))
          return false;
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < HD / 16; ++k) {
          const uint64_t ad = umma_smem_desc(sQ + (k >> 2) * Q_BLK + (k & 3) * 32);
          const uint64_t bd = umma_smem_desc(sK + st * KV_TILE_BYTES + (k >> 2) * KV_BLK + (k & 3) * 32);
          umma_bf16(tmem_base, ad, bd, idesc_s, k != 0 ? 1u : 0u);
        }
        umma_commit(smem_u32(&bars->k_empty[st]));  // K_j is free once S_j is computed
        umma_commit(smem_u32(&bars->s_full));
        return true;
      };
      if (ok) ok = issue_s(0);
      for (int j = 0; j + 1 < n_kt && ok; ++j) {  // S_{j+1} as soon as the softmax threads hold S_j in registers
        ok = mbar_wait(smem_u32(&bars->s_free), (uint32_t)j & 1u, abort_flag, status, W_ATTN_MMA);
        if (!ok) break;
        ok = issue_s(j + 1);
      }
    }
  } else if (warp == 6) {
    // ---------------------------------------------------------------- P V issuer
    // A thread of its own: issuing a chain of MMAs blocks the issuing thread for as long as the pipe needs
    // to take them (both resident CTAs queue there), and one thread issuing S_{j+1} and then P_j V_j spent
    // nearly the whole tile period blocked while the softmax threads idled 30-40 % of it.
    if (lane == 0) {
      const uint32_t idesc_pv = idesc_bf16(TQ, HD, 0, 1);
      bool ok = true;
      for (int j = 0; j < n_kt && ok; ++j) {
        const int st = j & 1;
        ok = mbar_wait(smem_u32(&bars->p_full[st]), (uint32_t)(j >> 1) & 1u, abort_flag, status, W_ATTN_MMA);
        if (!ok) break;
        ok = mbar_wait(smem_u32(&bars->v_full[st]), (uint32_t)(j >> 1) & 1u, abort_flag, status, W_ATTN_MMA);
        if (!ok) break;
        tc_fence_after();
        const uint32_t tmem_p = tmem_base + 64u + (uint32_t)(st * 32);
#pragma unroll
        for (int k = 0; k < TK / 16; ++k) {
          const uint64_t vd = umma_smem_desc_mn(sV + st * KV_TILE_BYTES + k * 2048, KV_BLK, 1024);
          umma_bf16_a_tmem(tmem_o, tmem_p + (uint32_t)(k * 8), vd, idesc_pv, (j | k) != 0 ? 1u : 0u);
        }
        umma_commit(smem_u32(&bars->v_empty[st]));  // V_j is free once these MMAs retire
        umma_commit(smem_u32(&bars->pv_done[st]));
      }
    }
  } else {
    // ---------------------------------------------------------------- softmax warps
    const int quarter = warp & 3;
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const int row = q0 + quarter * 32 + lane;  // index inside the sequence
    const float sl2 = rsqrtf((float)HD) * 1.4426950408889634f;
    float m = -INFINITY, l = 0.f;
    bool ok = true;
    // the thread that owns the sequence's last row also records that row's softmax numerators
    const bool score_row = sc.p != nullptr && row == n - 1;
    const bool score_warp = __any_sync(0xffffffffu, score_row);
    const int seq_id = cu_q ? (int)blockIdx.z : sc.seq_id;
    // row (seq, h) of P: max_tiles * 64 floats, 16-byte aligned, so whole tiles are stored as float4
    float *sc_p = score_row ? sc.p + ((size_t)seq_id * gridDim.x + h) * sc.max_tiles * TK : nullptr;
    float *sc_m = score_row ? sc.mtile + ((size_t)seq_id * gridDim.x + h) * sc.max_tiles : nullptr;
    for (int j = 0; j < n_kt && ok; ++j) {
      const int b = j & 1;
      ok = mbar_wait(smem_u32(&bars->s_full), (uint32_t)j & 1u, abort_flag, status, W_ATTN_SOFTMAX);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t t_s = tmem_base + lane_base;
      uint32_t raw[64];
      tmem_ld_32x32_raw(t_s, raw);
      tmem_ld_32x32_raw(t_s + 32u, raw + 32);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->s_free));  // S's columns may take the next tile
      // running maximum on the raw logits (the softmax scale is positive); the mask only matters on
      // tiles that cross the row's diagonal, so the common tile takes the short path
      const int col0 = j * TK;
      if (col0 + TK - 1 > row) {
#pragma unroll
        for (int c = 0; c < 64; ++c)
          if (col0 + c > row) raw[c] = 0xff800000u;  // -inf
      }
      float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // four chains of three-input maxima
#pragma unroll
      for (int c = 0; c < 64; c += 8) {
        mx[0] = fmax3(mx[0], __uint_as_float(raw[c]), __uint_as_float(raw[c + 1]));
        mx[1] = fmax3(mx[1], __uint_as_float(raw[c + 2]), __uint_as_float(raw[c + 3]));
        mx[2] = fmax3(mx[2], __uint_as_float(raw[c + 4]), __uint_as_float(raw[c + 5]));
        mx[3] = fmax3(mx[3], __uint_as_float(raw[c + 6]), __uint_as_float(raw[c + 7]));
      }
      const float mj = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * sl2;  // log2 units
      float alpha = 1.f;
      if (j == 0) {
        m = mj;  // key 0 is visible to every row: finite
      } else {
        const bool need = mj - m > RESCALE_LOG2;
        if (need) {
          alpha = ex2_approx(m - mj);
          m = mj;
        }
        if (__any_sync(0xffffffffu, need)) {
          // O must be at rest: the previous P V has to retire before it is rescaled in place
          ok = mbar_wait(smem_u32(&bars->pv_done[(j - 1) & 1]), (uint32_t)((j - 1) >> 1) & 1u, abort_flag, status,
                         W_ATTN_SOFTMAX);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
#pragma unroll 1
          for (int c = 0; c < HD; c += 32) {
            uint32_t ov[32];
            tmem_ld_32x32_raw(tmem_o + lane_base + (uint32_t)c, ov);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
            tmem_st_32x32(tmem_o + lane_base + (uint32_t)c, ov);
          }
          tmem_st_wait();
        }
      }
      // p = 2^(s * scale - m): half a two-wide FMA, one ex2 and one add per element (two-wide sums as well
      // pushed the kernel over its register budget)
      float sm[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t pk[32];
      const float neg_m = -m;
      const unsigned long long sl2x2 = f32x2_pack(sl2, sl2), negmx2 = f32x2_pack(neg_m, neg_m);
#pragma unroll
      for (int c = 0; c < 64; c += 4) {
        float x0, x1, x2, x3;
        f32x2_unpack(f32x2_fma(f32x2_pack(__uint_as_float(raw[c]), __uint_as_float(raw[c + 1])), sl2x2, negmx2), x0, x1);
        f32x2_unpack(f32x2_fma(f32x2_pack(__uint_as_float(raw[c + 2]), __uint_as_float(raw[c + 3])), sl2x2, negmx2), x2, x3);
        const float p0 = ex2_approx(x0), p1 = ex2_approx(x1), p2 = ex2_approx(x2), p3 = ex2_approx(x3);
        sm[0] += p0;
        sm[1] += p1;
        sm[2] += p2;
        sm[3] += p3;
        pk[c >> 1] = bf16x2_pack(p0, p1);
        pk[(c >> 1) + 1] = bf16x2_pack(p2, p3);
      }
      l = l * alpha + ((sm[0] + sm[1]) + (sm[2] + sm[3]));
      if (score_warp) {  // warp-uniform: only the warp that owns the sequence's last row gets here
        if (score_row) {
          float4 *dst = reinterpret_cast<float4 *>(sc_p + col0);
#pragma unroll
          for (int c = 0; c < 64; c += 4) {
            float4 pv;
            pv.x = ex2_approx(fmaf(__uint_as_float(raw[c]), sl2, neg_m));
            pv.y = ex2_approx(fmaf(__uint_as_float(raw[c + 1]), sl2, neg_m));
            pv.z = ex2_approx(fmaf(__uint_as_float(raw[c + 2]), sl2, neg_m));
            pv.w = ex2_approx(fmaf(__uint_as_float(raw[c + 3]), sl2, neg_m));
            dst[c >> 2] = pv;  // keys past the row hold 0 (masked) and land in the row's padding
          }
          sc_m[j] = m;
        }
      }
      // P_j goes where P_{j-2} was.  P_{j-2} V_{j-2} is issued by another thread than the S MMAs, so S_j's
      // arrival says nothing about it: its own barrier does (phase (j-2) >> 1 of pv_done[b]).
      if (j >= 2) {
        ok = mbar_wait(smem_u32(&bars->pv_done[b]), (uint32_t)((j - 2) >> 1) & 1u, abort_flag, status,
                       W_ATTN_SOFTMAX);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      tmem_st_32x32(t_s + 64u + (uint32_t)(b * 32), pk);  // P_j: 64 bf16 = 32 columns of its own
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->p_full[b]));
    }
    // The last two P V products (one per barrier) may still be in flight.
    if (ok && n_kt >= 2) {
      ok = mbar_wait(smem_u32(&bars->pv_done[(n_kt - 2) & 1]), (uint32_t)((n_kt - 2) >> 1) & 1u, abort_flag, status,
                     W_ATTN_SOFTMAX);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      ok = mbar_wait(smem_u32(&bars->pv_done[(n_kt - 1) & 1]), (uint32_t)((n_kt - 1) >> 1) & 1u, abort_flag, status,
                     W_ATTN_SOFTMAX);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok && score_row) {
      float *stt = sc.stats + ((size_t)seq_id * gridDim.x + h) * 2;
      stt[0] = m;
      stt[1] = 1.f / l;
    }
    if (ok) {
      tc_fence_after();
      const float inv = 1.f / l;
      bf16 *orow = o + (size_t)(q_start + row) * ldo + h * HD;
#pragma unroll 1
      for (int c = 0; c < HD; c += 32) {
        float v[32];
        tmem_ld_32x32(tmem_o + lane_base + (uint32_t)c, v);
        if (row < n) {
#pragma unroll
          for (int i = 0; i < 32; i += 8) {
            float f[8];
#pragma unroll
            for (int t = 0; t < 8; ++t) f[t] = v[i + t] * inv;
            Vec16<bf16> ov;
            ov.pack(f);
            ov.store(orow + c + i);
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"((uint32_t)ATT_TMEM_COLS)
                 : "memory");
  }
}

}  // namespace

// q: rows of pitch ldq elements (heads side by side), k/v: rows of pitch ldkv.  Either the sequences
// come from device arrays (cu_q, kv_base; one launch, q_rows/kv_rows = extent of the buffers), or one
// sequence is described by scalars (q_start, n, kv_start).
int launch_attention_tc(cudaStream_t st, const void *q, int ldq, long long q_rows, const void *k,
                        const void *v, int ldkv, long long kv_rows, void *o, int n_heads,
                        const int32_t *cu_q, const int32_t *kv_base, int n_seqs, int max_len, int q_start,
                        int n, int kv_start, DevStatus *status, float *score_scratch, int max_tiles,
                        int n_seqs_total, int seq_id, int n_kv_heads) {
  if (n_seqs == 0 || max_len == 0) return LAZY_OK;
  const int kv_group = kv_group_of(n_heads, n_kv_heads);
  if (kv_group < 1) return LAZY_E_BADARG;
  if ((ldq % 8) || (ldkv % 8) || ((uintptr_t)q & 15) || ((uintptr_t)k & 15) || ((uintptr_t)v & 15) ||
      ((uintptr_t)o & 15))
    return LAZY_E_BADARG;
  CUtensorMap mq, mk, mv;
  LAZY_TRY(tma_map_2d_bf16(&mq, q, q_rows, n_heads * HD, ldq, 64, TQ));
  LAZY_TRY(tma_map_2d_bf16(&mk, k, kv_rows, n_heads / kv_group * HD, ldkv, 64, TK));
  LAZY_TRY(tma_map_2d_bf16(&mv, v, kv_rows, n_heads / kv_group * HD, ldkv, 64, TK));
  static bool attr_set = false;
  if (!attr_set) {
    LAZY_CUDA_OK(cudaFuncSetAttribute(attn_tcgen05_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      ATT_SMEM_BYTES));
    attr_set = true;
  }
  dim3 grid(n_heads, cdiv(max_len, TQ), n_seqs);
  AttnScoreOut sc = {nullptr, nullptr, nullptr, 0, 0};
  if (score_scratch) {  // layout: P [S, H, max_tiles*64] | mtile [S, H, max_tiles] | stats [S, H, 2]
    sc.p = score_scratch;
    sc.mtile = score_scratch + (size_t)n_seqs_total * n_heads * max_tiles * TK;
    sc.stats = sc.mtile + (size_t)n_seqs_total * n_heads * max_tiles;
    sc.max_tiles = max_tiles;
    sc.seq_id = seq_id;
  }
  attn_tcgen05_kernel<<<grid, ATT_THREADS, ATT_SMEM_BYTES, st>>>(mq, mk, mv, (bf16 *)o, n_heads * HD, cu_q,
                                                                 kv_base, q_start, n, kv_start, status, sc, kv_group);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

namespace {
// Eq. 1 from the attention kernel's by-product: s_r = (1/H) sum_h p[h][r] * 2^(m_tile - m_final) / l.
// Eight lanes share a key row, each summing every eighth head; a fixed shuffle tree adds them up.
// blockIdx.y = layer of a group of consecutive layers that share the same rows (cu_q): layer y reads the
// by-product at scratch + y * scratch_stride and writes scores + y * scores_stride, so that the head means
// of all layers between two cuts take one launch.
__global__ void score_from_attention_kernel(const float *__restrict__ scratch, size_t scratch_stride,
                                            const int32_t *__restrict__ cu_q, int n_seqs, int n_total, int n_heads,
                                            int max_tiles, float *__restrict__ scores, size_t scores_stride) {
  const float *p = scratch + (size_t)blockIdx.y * scratch_stride;
  const float *mtile = p + (size_t)n_seqs * n_heads * max_tiles * TK;
  const float *stats = mtile + (size_t)n_seqs * n_heads * max_tiles;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  const int r = t >> 3, part = t & 7;
  float acc = 0.f;
  if (r < n_total) {
    int lo = 0, hi = n_seqs;
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (cu_q[mid] <= r) lo = mid; else hi = mid;
    }
    const int j = r - cu_q[lo];
    const int tile = j / TK;
#pragma unroll 4
    for (int h = part; h < n_heads; h += 8) {
      const size_t sh = (size_t)lo * n_heads + h;
      acc += p[sh * max_tiles * TK + j] * ex2_approx(mtile[sh * max_tiles + tile] - stats[sh * 2]) * stats[sh * 2 + 1];
    }
  }
  acc += __shfl_xor_sync(0xffffffffu, acc, 1);
  acc += __shfl_xor_sync(0xffffffffu, acc, 2);
  acc += __shfl_xor_sync(0xffffffffu, acc, 4);
  if (r < n_total && part == 0) scores[(size_t)blockIdx.y * scores_stride + r] = acc / (float)n_heads;
}
}  // namespace

size_t attn_score_scratch_floats(int n_seqs, int n_heads, int max_tiles) {
  return (size_t)n_seqs * n_heads * max_tiles * (TK + 1) + (size_t)2 * n_seqs * n_heads;
}

// n_layers consecutive layers over the same rows: layer y's by-product at scratch + y * scratch_stride,
// its scores to scores + y * scores_stride.
int launch_score_from_attention(cudaStream_t st, const float *scratch, size_t scratch_stride, int n_layers,
                                const int32_t *cu_q, int n_seqs, int n_total, int n_heads, int max_tiles,
                                float *scores, size_t scores_stride) {
  if (n_total == 0 || n_layers == 0) return LAZY_OK;
  score_from_attention_kernel<<<dim3(cdiv(n_total * 8, 256), n_layers), 256, 0, st>>>(
      scratch, scratch_stride, cu_q, n_seqs, n_total, n_heads, max_tiles, scores, scores_stride);
  LAZY_COUNT_LAUNCH();
  return launch_ok();
}

}  // namespace lazy
