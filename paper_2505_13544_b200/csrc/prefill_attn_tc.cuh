// Tensor-core (tcgen05 / TMEM / TMA) prefill attention under the stride-aware causal mask of
// Section 4.2, in the un-absorbed form (Eq. 9-11 with the RoPE term of Eq. 17), bf16 operands,
// fp32 accumulation.
//
// Row m (0-based token) of a sequence attends to the closed slots j < floor(m / s), each
// represented by the running state and RoPE key of its last token j*s + s - 1, and to its own
// running state at column m: exactly the columns the mask admits, expressed as a predicate.
// The closed slots are read through a strided TMA view (row j of the view is token
// j*s + s - 1), so they form an ordinary dense key / value sequence of length floor(T / s), and
// the kernel is a flash-attention loop over that sequence with the predicate j < floor(m / s),
// followed by one "diagonal" pass over the query tile's own tokens with the predicate n == m.
//
// One CTA per (128-row query tile, head, sequence).  Per key tile of KT slots:
//   scores  S[128 x KT]  = Q_h K_h^T + Q^R K^R^T      A = Q (K-major), B = K tile (K-major), N = KT
//   values  O[128 x d_h] += P[128 x KT] V[KT x d_h]    A = P (K-major, written by the softmax
//                                                      threads), B = V tile (MN-major)
// Keys and values are kept as two bf16 halves (hi + lo, the up-projection's fp32 result split
// once).  The value halves sit side by side in the MMA's N, their products land in two column
// blocks of the accumulator and are added in the epilogue; the key remainders get their own
// score MMAs into the same accumulator.  A row with few visible slots is almost a copy of its
// values, and with outputs of magnitude 4-8 the bf16 rounding of the output alone uses most of
// the error budget, so a single rounding of keys or values would show.
// Accumulators live in TMEM (two score buffers, one output block of two halves); TMEM lane i is query row i,
// so each of the 128 softmax threads owns one row and its maximum and sum are thread-local.
// The reference maximum of a row is raised only when a tile exceeds it by more than 2^8; a warp
// rescales its 32 rows of O in TMEM only when one of them must.  On fully visible tiles the
// maximum is not even computed: the exponentials are taken against the current reference and
// the tile's sum tells whether the reference was outgrown.
//
// Warp roles: warp 0 = TMA producer, warp 1 = score MMA issuer and TMEM owner, warp 2 = value
// MMA issuer, warp 3 idle, warps 4-7 = softmax and epilogue.  Every wait is a bounded mbarrier
// wait (see sm100_ptx.cuh).
#pragma once

#include <math.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mtla {

struct PrefillAttnTcArgs {
  bf16* out;        // [B*T][2][n_h*d_h]: per-head outputs as bf16 hi halves, then remainders
  int* error_word;
  int n_heads, dr, stride, T;
};

namespace pft {

constexpr int kThreads = 256;
constexpr int kQTile = 128;
constexpr int kStages = 2;
constexpr int kTmemCols = 512;
constexpr int kColO = 256;
constexpr float kRescaleThreshold = 8.f;

__host__ __device__ constexpr int key_tile(int dh) { return dh == 64 ? 128 : 64; }
__host__ __device__ constexpr int q_bytes(int dh) { return (dh / 64 + 1) * kQTile * 128; }
__host__ __device__ constexpr int stage_bytes(int dh) {
  // K_h chunks (hi, then lo) + one RoPE-key chunk + V chunks (hi, then lo), each [KT rows x 128 B].
  return (4 * (dh / 64) + 1) * key_tile(dh) * 128;
}
__host__ __device__ constexpr int p_bytes(int dh) { return kQTile * key_tile(dh) * 2; }
__host__ __device__ constexpr int smem_bytes(int dh) {
  return q_bytes(dh) + kStages * stage_bytes(dh) + p_bytes(dh) + 256 + 1024;
}

struct Bars {
  unsigned long long q_full, k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  unsigned long long s_full[2], s_empty[2], p_full, p_empty;
  uint32_t tmem_base;
  int abort_word;
};
static_assert(sizeof(Bars) <= 256, "barrier block too large");

}  // namespace pft

// Tensor maps: q [B][T][n_h*(d_h+d_R)]; kv_closed / kv_self over [B*T][4*n_h*d_h] (keys, values,
// then the bf16 remainders of both), the first with row j = token j*s+s-1 of each sequence, the
// second dense; kr_closed /
// kr_self likewise over the RoPE keys [B*T][d_R].  Boxes: 64 columns x 128 (q) or KT rows.
template <int DH>
__global__ void __launch_bounds__(pft::kThreads, 1)
prefill_attn_tc_kernel(const __grid_constant__ CUtensorMap q_map,
                       const __grid_constant__ CUtensorMap kv_closed,
                       const __grid_constant__ CUtensorMap kv_self,
                       const __grid_constant__ CUtensorMap kr_closed,
                       const __grid_constant__ CUtensorMap kr_self, PrefillAttnTcArgs a) {
  using namespace pft;
  using namespace ptx;
  constexpr int KT = key_tile(DH);
  constexpr int CK = DH / 64;                       // 64-column chunks of a head's keys / values
  constexpr int SUB = KT * 128;                     // bytes of one [KT x 64] chunk
  constexpr int QSUB = kQTile * 128;                // bytes of one [128 x 64] chunk of Q
  constexpr int PSUB = kQTile * 128;                // bytes of one [128 rows x 64 keys] chunk of P
  constexpr uint32_t IDESC_QK = make_idesc_bf16(128, KT, 0, 0);
  constexpr uint32_t IDESC_PV = make_idesc_bf16(128, 2 * DH, 0, 1);   // N = [V hi | V lo]
  constexpr int kOffQ = 0;
  constexpr int kOffKv = q_bytes(DH);
  constexpr int kOffP = kOffKv + kStages * stage_bytes(DH);
  constexpr int kOffBars = kOffP + p_bytes(DH);
  constexpr int DIAG = kQTile / KT;                 // diagonal passes per query tile

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  Bars* bars = reinterpret_cast<Bars*>(sm + kOffBars);
  volatile int* abort_word = &bars->abort_word;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  auto bar = [&](unsigned long long* p) { return smem_u32(p); };

  if (threadIdx.x == 0) {
    mbar_init(bar(&bars->q_full), 1);
    for (int i = 0; i < kStages; ++i) {
      mbar_init(bar(&bars->k_full[i]), 1);
      mbar_init(bar(&bars->k_empty[i]), 1);         // score issuer
      mbar_init(bar(&bars->v_full[i]), 1);
      mbar_init(bar(&bars->v_empty[i]), 1);         // value issuer
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(&bars->s_full[i]), 1);
      mbar_init(bar(&bars->s_empty[i]), 128);
    }
    mbar_init(bar(&bars->p_full), 128);
    mbar_init(bar(&bars->p_empty), 1);
    bars->abort_word = 0;
    mbar_fence_init();
    prefetch_tensormap(&q_map);
    prefetch_tensormap(&kv_closed);
    prefetch_tensormap(&kv_self);
    prefetch_tensormap(&kr_closed);
    prefetch_tensormap(&kr_self);
  }
  if (warp == 1) tmem_alloc(smem_u32(&bars->tmem_base), kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;

  // Long query tiles (late rows, many key tiles) are scheduled first.
  const int qt = (int)(gridDim.x - 1 - blockIdx.x), h = blockIdx.y, b = blockIdx.z;
  const int q0 = qt * kQTile;
  const int last_row = min(a.T, q0 + kQTile) - 1;
  const int n_closed = last_row / a.stride;                // closed slots visible to the last row
  const int n_kv = (n_closed + KT - 1) / KT;               // key tiles over the closed slots
  const int n_tiles = n_kv + DIAG;                         // + the diagonal passes
  const int hd = a.n_heads * DH;

  const uint32_t q_u32 = base + kOffQ, kv_u32 = base + kOffKv, p_u32 = base + kOffP;

  if (warp == 0 && lane == 0) {
    // ------------------------------------------------------------------ TMA producer
    mbar_arrive_expect_tx(bar(&bars->q_full), q_bytes(DH));
    for (int c = 0; c <= CK; ++c)
      tma_load_3d(q_u32 + c * QSUB, &q_map, bar(&bars->q_full), h * (DH + a.dr) + c * 64, q0, b);
    // A stage's key part (K hi, K lo, RoPE keys) is free as soon as its score MMAs are done,
    // its value part only after the value MMAs: the keys of tile t + 1 are therefore requested
    // before the values of tile t, which keeps the score MMAs one load latency ahead.
    auto tile_source = [&](int t, const CUtensorMap*& kvm, const CUtensorMap*& krm, int& row) {
      const bool diag = t >= n_kv;
      kvm = diag ? &kv_self : &kv_closed;
      krm = diag ? &kr_self : &kr_closed;
      row = diag ? q0 + (t - n_kv) * KT : t * KT;   // token, or closed-slot index
    };
    // Stage layout in chunks: K hi [0, CK), K lo [CK, 2CK), RoPE keys 2CK, V hi, V lo.
    auto load_keys = [&](int t) {
      const int st = t % kStages;
      if (!mbar_wait(bar(&bars->k_empty[st]), ((t / kStages) & 1) ^ 1, abort_word, a.error_word, 21))
        return false;
      const CUtensorMap *kvm, *krm;
      int row;
      tile_source(t, kvm, krm, row);
      const uint32_t dst = kv_u32 + st * stage_bytes(DH);
      mbar_arrive_expect_tx(bar(&bars->k_full[st]), (2 * CK + 1) * SUB);
      for (int c = 0; c < CK; ++c)
        for (int half = 0; half < 2; ++half)       // remainders sit 2 n_h d_h columns further
          tma_load_3d(dst + (half * CK + c) * SUB, kvm, bar(&bars->k_full[st]),
                      half * 2 * hd + h * DH + c * 64, row, b);
      tma_load_3d(dst + 2 * CK * SUB, krm, bar(&bars->k_full[st]), 0, row, b);
      return true;
    };
    auto load_values = [&](int t) {
      const int st = t % kStages;
      if (!mbar_wait(bar(&bars->v_empty[st]), ((t / kStages) & 1) ^ 1, abort_word, a.error_word, 20))
        return false;
      const CUtensorMap *kvm, *krm;
      int row;
      tile_source(t, kvm, krm, row);
      const uint32_t dst = kv_u32 + st * stage_bytes(DH) + (2 * CK + 1) * SUB;
      mbar_arrive_expect_tx(bar(&bars->v_full[st]), 2 * CK * SUB);
      for (int c = 0; c < CK; ++c)
        for (int half = 0; half < 2; ++half)
          tma_load_3d(dst + (half * CK + c) * SUB, kvm, bar(&bars->v_full[st]),
                      hd + half * 2 * hd + h * DH + c * 64, row, b);
      return true;
    };
    bool ok = load_keys(0);
    for (int t = 0; t < n_tiles && ok; ++t) {
      if (t + 1 < n_tiles) ok = load_keys(t + 1);
      if (ok) ok = load_values(t);
    }
  } else if (warp == 1 && lane == 0) {
    // ------------------------------------------------------------------ score MMA issuer
    bool ok = mbar_wait(bar(&bars->q_full), 0, abort_word, a.error_word, 22);
    for (int t = 0; t < n_tiles && ok; ++t) {
      const int st = t % kStages;
      ok = mbar_wait(bar(&bars->s_empty[t & 1]), ((t >> 1) & 1) ^ 1, abort_word, a.error_word, 23) &&
           mbar_wait(bar(&bars->k_full[st]), (t / kStages) & 1, abort_word, a.error_word, 24);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t kbase = kv_u32 + st * stage_bytes(DH);
      const uint32_t d_tmem = tmem_base + (t & 1) * KT;
      // Key chunk kc of the stage against query chunk qc: K hi and K lo meet the same queries,
      // the last key chunk (RoPE keys) meets the RoPE queries.
#pragma unroll
      for (int kc = 0; kc <= 2 * CK; ++kc) {
        const int qc = kc == 2 * CK ? CK : kc % CK;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          const uint64_t ad = make_smem_desc(q_u32 + qc * QSUB + ks * 32, 16, 1024, kSwizzle128B);
          const uint64_t bd = make_smem_desc(kbase + kc * SUB + ks * 32, 16, 1024, kSwizzle128B);
          mma_bf16_ss(d_tmem, ad, bd, IDESC_QK, (kc > 0 || ks > 0) ? 1u : 0u);
        }
      }
      mma_commit(bar(&bars->s_full[t & 1]));
      mma_commit(bar(&bars->k_empty[st]));
    }
  } else if (warp == 2 && lane == 0) {
    // ------------------------------------------------------------------ value MMA issuer
    bool ok = true;
    for (int t = 0; t < n_tiles && ok; ++t) {
      const int st = t % kStages;
      ok = mbar_wait(bar(&bars->p_full), t & 1, abort_word, a.error_word, 25) &&
           mbar_wait(bar(&bars->v_full[st]), (t / kStages) & 1, abort_word, a.error_word, 19);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t vbase = kv_u32 + st * stage_bytes(DH) + (2 * CK + 1) * SUB;
      const uint32_t pbase = p_u32;
#pragma unroll
      for (int ks = 0; ks < KT / 16; ++ks) {
        // A = P [128 rows x KT keys], K-major, 64-key chunks of PSUB bytes.
        const uint64_t ad = make_smem_desc(pbase + (ks >> 2) * PSUB + (ks & 3) * 32, 16, 1024, kSwizzle128B);
        // B = V [d_h columns x KT keys], MN-major: 16 keys per k-step = 2048 bytes down the chunk.
        const uint64_t bd = make_smem_desc(vbase + ks * 2048, SUB, 1024, kSwizzle128B);
        mma_bf16_ss(tmem_base + kColO, ad, bd, IDESC_PV, (t > 0 || ks > 0) ? 1u : 0u);
      }
      mma_commit(bar(&bars->v_empty[st]));
      mma_commit(bar(&bars->p_empty));
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ softmax / epilogue warps
    const int q = warp & 3, row = q * 32 + lane;           // query row within the tile = TMEM lane
    const int m = q0 + row;                                 // token index of this thread's row
    const int closed = m / a.stride;                        // closed slots this row may see
    const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
    bool ok = true;
    float m_run = -INFINITY, l_run = 0.f;
    for (int t = 0; t < n_tiles; ++t) {
      if (ok) ok = mbar_wait(bar(&bars->s_full[t & 1]), (t >> 1) & 1, abort_word, a.error_word, 26);
      ok = __all_sync(0xffffffffu, ok);                    // TMEM accesses are whole-warp operations
      if (!ok) break;
      tc_fence_after_sync();
      const bool diag = t >= n_kv;
      const int col0 = diag ? (t - n_kv) * KT : t * KT;     // key index of column 0 (slot, or row offset)
      // The tile's scores of this row, then the mask as a predicate on the column index:
      // closed slots below `lim`, or the row's own column `own` in a diagonal pass.
      const int lim = diag ? 0 : closed - col0;
      const int own = (diag && m < a.T) ? row - col0 : -1;
      uint32_t sv[KT];
#pragma unroll
      for (int c0 = 0; c0 < KT; c0 += 32) {
        uint32_t(&v)[32] = *reinterpret_cast<uint32_t(*)[32]>(&sv[c0]);
        tmem_ld_x32(lane_base + (t & 1) * KT + c0, v);
      }
      tmem_wait_ld();
      tc_fence_before_sync();
      mbar_arrive(bar(&bars->s_empty[t & 1]));            // the scores are in registers now
      uint32_t pk[KT / 2];
      // Common case: the whole tile is visible to every row of the warp and every row has a
      // reference already.  Then the probabilities are formed at once, and the row maximum is
      // never computed: a tile that had outgrown a reference by 2^8 would show in its sum
      // (sum <= 2^15 guarantees every probability <= 2^15), in which case the careful path
      // below redoes the tile.  The comparison also catches an overflow to infinity.
      bool fast = __all_sync(0xffffffffu, lim >= KT && m_run != -INFINITY);
      if (fast) {
        float lsum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c = 0; c < KT; c += 2) {
          const float p0 = ex2_approx(__uint_as_float(sv[c]) - m_run);
          const float p1 = ex2_approx(__uint_as_float(sv[c + 1]) - m_run);
          lsum[(c >> 1) & 3] += p0 + p1;
          const __nv_bfloat162 two = __floats2bfloat162_rn(p0, p1);
          pk[c / 2] = *reinterpret_cast<const uint32_t*>(&two);
        }
        const float tile_sum = (lsum[0] + lsum[1]) + (lsum[2] + lsum[3]);
        fast = __all_sync(0xffffffffu, tile_sum <= 32768.f);
        if (fast) l_run += tile_sum;
      }
      if (!fast) {
        // Careful path: predicate, row maximum, lazy raise of the reference (by more than 2^8
        // only), rescale of this warp's O rows when one of them raised.
        float mt = -INFINITY;
#pragma unroll
        for (int c = 0; c < KT; ++c) {
          if (!(c < lim || c == own)) sv[c] = 0xff800000u;   // -inf
          mt = fmaxf(mt, __uint_as_float(sv[c]));
        }
        const bool raise = mt > m_run + kRescaleThreshold;
        const float m_new = raise ? mt : m_run;
        const float fac = (raise && m_run != -INFINITY) ? exp2f(m_run - m_new) : 1.f;
        if (__any_sync(0xffffffffu, raise && t > 0)) {
          // O rows are scaled to the old references: wait for the previous tile's value MMAs.
          ok = mbar_wait(bar(&bars->p_empty), (t & 1) ^ 1, abort_word, a.error_word, 27);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after_sync();
#pragma unroll
          for (int c0 = 0; c0 < 2 * DH; c0 += 32) {
            uint32_t ov[32];
            tmem_ld_x32(lane_base + kColO + c0, ov);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * fac);
            tmem_st_x32(lane_base + kColO + c0, ov);
          }
          tmem_wait_st();
          tc_fence_before_sync();
        }
        l_run *= fac;
        m_run = m_new;
        const float m_eff = m_run == -INFINITY ? 0.f : m_run;   // a row that has seen nothing yet
        float lsum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c = 0; c < KT; c += 2) {
          const float p0 = ex2_approx(__uint_as_float(sv[c]) - m_eff);
          const float p1 = ex2_approx(__uint_as_float(sv[c + 1]) - m_eff);
          lsum[(c >> 1) & 3] += p0 + p1;
          const __nv_bfloat162 two = __floats2bfloat162_rn(p0, p1);
          pk[c / 2] = *reinterpret_cast<const uint32_t*>(&two);
        }
        l_run += (lsum[0] + lsum[1]) + (lsum[2] + lsum[3]);
      }
      // The single probability buffer is free once the previous tile's value MMAs have completed.
      ok = mbar_wait(bar(&bars->p_empty), (t & 1) ^ 1, abort_word, a.error_word, 28);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      // P as the K-major, 128-byte-swizzled A operand: row r of a 64-key chunk at r*128, its
      // 16-byte piece c at position c ^ (r % 8).
      uint8_t* prow = sm + kOffP + row * 128;
#pragma unroll
      for (int c0 = 0; c0 < KT; c0 += 8) {
        const int chunk = c0 >> 6, piece = (c0 >> 3) & 7;
        *reinterpret_cast<uint4*>(prow + chunk * PSUB + ((piece ^ (row & 7)) << 4)) =
            make_uint4(pk[c0 / 2], pk[c0 / 2 + 1], pk[c0 / 2 + 2], pk[c0 / 2 + 3]);
      }
      fence_proxy_async_smem();
      tc_fence_before_sync();
      mbar_arrive(bar(&bars->p_full));
    }
    // Epilogue: wait for the last value MMAs, normalise this row and store hi / lo halves.
    if (ok) ok = mbar_wait(bar(&bars->p_empty), (n_tiles - 1) & 1, abort_word, a.error_word, 29);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after_sync();
      const float inv = 1.f / l_run;
      bf16* o_hi = a.out + ((long long)b * a.T + m) * 2 * hd + h * DH;
#pragma unroll
      for (int c0 = 0; c0 < DH; c0 += 32) {
        uint32_t ov[32], ol[32];
        tmem_ld_x32(lane_base + kColO + c0, ov);
        tmem_ld_x32(lane_base + kColO + DH + c0, ol);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) + __uint_as_float(ol[j]));
        if (m < a.T) {
#pragma unroll
          for (int j = 0; j < 32; j += 8) {
            uint32_t hi[4], lo[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float v0 = __uint_as_float(ov[j + 2 * e]) * inv, v1 = __uint_as_float(ov[j + 2 * e + 1]) * inv;
              const __nv_bfloat162 hh = __floats2bfloat162_rn(v0, v1);
              const __nv_bfloat162 ll = __floats2bfloat162_rn(v0 - __low2float(hh), v1 - __high2float(hh));
              hi[e] = *reinterpret_cast<const uint32_t*>(&hh);
              lo[e] = *reinterpret_cast<const uint32_t*>(&ll);
            }
            *reinterpret_cast<uint4*>(o_hi + c0 + j) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            *reinterpret_cast<uint4*>(o_hi + hd + c0 + j) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
          }
        }
      }
      tc_fence_before_sync();
    }
  }

  __syncthreads();
  if (*abort_word) {
    // Give copies that may still be in flight time to land before the CTA's memory is reused.
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 100000ull) __nanosleep(1000);
  }
  if (warp == 1) {
    __syncwarp();
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace mtla
