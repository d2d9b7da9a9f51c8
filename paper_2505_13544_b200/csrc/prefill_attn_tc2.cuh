// Prefill attention (Section 4.2 mask, un-absorbed form) with TWO query tiles per CTA, for
// d_h = 64.  Same mathematics, operands and mask-as-predicate as prefill_attn_tc.cuh; what
// changes is the schedule.  With one query tile per CTA the per-tile chain of hand-overs
// (score commit -> softmax wake-up -> TMEM load -> P store and proxy fence -> value-issuer
// wake-up -> value commit -> P buffer free) has nothing to overlap with and bounds the loop.
// Here a CTA owns 256 query rows as two tiles of 128 that share every key / value tile: each
// query tile has its own score issuer, its own softmax warpgroup, its own probability buffer and
// its own accumulators, so the two chains interleave, and a key / value tile is loaded once for
// twice the tensor work.  Key tiles are 64 slots, so that two query tiles, their probability
// buffers and a two-stage key / value ring fit shared memory, and two double-buffered score
// blocks plus two output blocks fit TMEM's 512 columns.
//
// A key tile beyond what query tile 0 may see (the pair's tile count follows its last row) and
// the diagonal passes over the other query tile's tokens hold nothing a query tile may attend
// to: that tile's issuer, softmax warps and value products skip them (`relevant` below), and
// each query tile counts its own tiles for the parities of its score and probability buffers.
//
// Warp roles: warp 0 = TMA producer, warps 1-2 = score issuers of query tile 0 / 1 (warp 1 owns
// TMEM), warp 3 = value issuer of both, warps 4-7 / 8-11 = softmax and epilogue of query tile
// 0 / 1.  Every wait is a bounded mbarrier wait (see sm100_ptx.cuh).
#pragma once

#include <math.h>

#include "common.cuh"
#include "prefill_attn_tc.cuh"
#include "sm100_ptx.cuh"

namespace mtla {

namespace pft2 {

constexpr int DH = 64;
constexpr int kThreads = 384;
constexpr int kQTile = 128, kQTiles = 2;
constexpr int KT = 64;                                  // slots per key tile
constexpr int kStages = 2;
constexpr int kTmemCols = 512;
constexpr int kColO = 256;                              // O of query tile u at kColO + u * 128
constexpr float kRescaleThreshold = 8.f;
constexpr int SUB = KT * 128;                           // bytes of one [KT x 64] chunk
constexpr int QSUB = kQTile * 128;                      // bytes of one [128 x 64] chunk of Q
constexpr int kQBytes = kQTiles * 2 * QSUB;             // per query tile: head chunk, RoPE chunk
constexpr int kKeyBytes = 3 * SUB;                      // K hi, K lo, RoPE keys
constexpr int kValBytes = 2 * SUB;                      // V hi, V lo
constexpr int kPBytes = kQTile * KT * 2;                // one query tile's probabilities
constexpr int kOffQ = 0;
constexpr int kOffKey = kOffQ + kQBytes;
constexpr int kOffVal = kOffKey + kStages * kKeyBytes;
constexpr int kOffP = kOffVal + kStages * kValBytes;
constexpr int kOffBars = kOffP + kQTiles * kPBytes;
constexpr int kSmemBytes = kOffBars + 512 + 1024;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

struct Bars {
  unsigned long long q_full, k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  unsigned long long s_full[kQTiles][2], s_empty[kQTiles][2], p_full[kQTiles], p_empty[kQTiles];
  uint32_t tmem_base;
  int abort_word;
};
static_assert(sizeof(Bars) <= 512, "barrier block too large");

}  // namespace pft2

// Tensor maps as for prefill_attn_tc_kernel, the key / value ones with boxes of 64 rows.
__global__ void __launch_bounds__(pft2::kThreads, 1)
prefill_attn_tc2_kernel(const __grid_constant__ CUtensorMap q_map,
                        const __grid_constant__ CUtensorMap kv_closed,
                        const __grid_constant__ CUtensorMap kv_self,
                        const __grid_constant__ CUtensorMap kr_closed,
                        const __grid_constant__ CUtensorMap kr_self, PrefillAttnTcArgs a) {
  using namespace pft2;
  using namespace ptx;
  constexpr uint32_t IDESC_QK = make_idesc_bf16(128, KT, 0, 0);
  constexpr uint32_t IDESC_PV = make_idesc_bf16(128, 2 * DH, 0, 1);   // N = [V hi | V lo]

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
      mbar_init(bar(&bars->k_empty[i]), kQTiles);     // both score issuers
      mbar_init(bar(&bars->v_full[i]), 1);
      mbar_init(bar(&bars->v_empty[i]), 1);           // value issuer
    }
    for (int u = 0; u < kQTiles; ++u) {
      for (int i = 0; i < 2; ++i) {
        mbar_init(bar(&bars->s_full[u][i]), 1);
        mbar_init(bar(&bars->s_empty[u][i]), 128);
      }
      mbar_init(bar(&bars->p_full[u]), 128);
      mbar_init(bar(&bars->p_empty[u]), 1);
    }
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

  // Long query pairs (late rows, many key tiles) are scheduled first.
  const int qp = (int)(gridDim.x - 1 - blockIdx.x), h = blockIdx.y, b = blockIdx.z;
  const int q0 = qp * kQTiles * kQTile;
  const int last_row = min(a.T, q0 + kQTiles * kQTile) - 1;
  const int n_closed = last_row / a.stride;                // closed slots visible to the last row
  const int n_kv = (n_closed + KT - 1) / KT;               // key tiles over the closed slots
  constexpr int DIAG = kQTiles * kQTile / KT;              // diagonal passes over the pair's own tokens
  const int n_tiles = n_kv + DIAG;
  const int hd = a.n_heads * DH;
  // Key tiles over the closed slots that query tile 0's last row can see.
  const int n_kv0 = ((min(a.T, q0 + kQTile) - 1) / a.stride + KT - 1) / KT;
  // Does key tile t hold anything query tile u may see?  Closed slots up to its last row's
  // count; of the diagonal passes, the two over its own 128 tokens.
  auto relevant = [&](int u, int t) {
    return t < n_kv ? (u == 1 || t < n_kv0) : (t - n_kv) * KT / kQTile == u;
  };
  const int n_rel[2] = {n_kv0 + kQTile / KT, n_kv + kQTile / KT};

  const uint32_t q_u32 = base + kOffQ, key_u32 = base + kOffKey, val_u32 = base + kOffVal;
  const uint32_t p_u32 = base + kOffP;

  if (warp == 0 && lane == 0) {
    // ------------------------------------------------------------------ TMA producer
    mbar_arrive_expect_tx(bar(&bars->q_full), kQBytes);
    for (int u = 0; u < kQTiles; ++u)
      for (int c = 0; c < 2; ++c)
        tma_load_3d(q_u32 + (u * 2 + c) * QSUB, &q_map, bar(&bars->q_full), h * (DH + a.dr) + c * 64,
                    q0 + u * kQTile, b);
    auto tile_source = [&](int t, const CUtensorMap*& kvm, const CUtensorMap*& krm, int& row) {
      const bool diag = t >= n_kv;
      kvm = diag ? &kv_self : &kv_closed;
      krm = diag ? &kr_self : &kr_closed;
      row = diag ? q0 + (t - n_kv) * KT : t * KT;   // token, or closed-slot index
    };
    auto load_keys = [&](int t) {
      const int st = t % kStages;
      if (!mbar_wait(bar(&bars->k_empty[st]), ((t / kStages) & 1) ^ 1, abort_word, a.error_word, 41))
        return false;
      const CUtensorMap *kvm, *krm;
      int row;
      tile_source(t, kvm, krm, row);
      const uint32_t dst = key_u32 + st * kKeyBytes;
      mbar_arrive_expect_tx(bar(&bars->k_full[st]), kKeyBytes);
      tma_load_3d(dst, kvm, bar(&bars->k_full[st]), h * DH, row, b);                    // K hi
      tma_load_3d(dst + SUB, kvm, bar(&bars->k_full[st]), 2 * hd + h * DH, row, b);     // K lo
      tma_load_3d(dst + 2 * SUB, krm, bar(&bars->k_full[st]), 0, row, b);               // RoPE keys
      return true;
    };
    auto load_values = [&](int t) {
      const int st = t % kStages;
      if (!mbar_wait(bar(&bars->v_empty[st]), ((t / kStages) & 1) ^ 1, abort_word, a.error_word, 40))
        return false;
      const CUtensorMap *kvm, *krm;
      int row;
      tile_source(t, kvm, krm, row);
      const uint32_t dst = val_u32 + st * kValBytes;
      mbar_arrive_expect_tx(bar(&bars->v_full[st]), kValBytes);
      tma_load_3d(dst, kvm, bar(&bars->v_full[st]), hd + h * DH, row, b);               // V hi
      tma_load_3d(dst + SUB, kvm, bar(&bars->v_full[st]), 3 * hd + h * DH, row, b);     // V lo
      return true;
    };
    bool ok = load_keys(0);
    for (int t = 0; t < n_tiles && ok; ++t) {
      if (t + 1 < n_tiles) ok = load_keys(t + 1);
      if (ok) ok = load_values(t);
    }
  } else if ((warp == 1 || warp == 2) && lane == 0) {
    // ------------------------------------------------------------------ score issuer of query tile u
    const int u = warp - 1;
    bool ok = mbar_wait(bar(&bars->q_full), 0, abort_word, a.error_word, 42);
    int c = 0;                                     // this query tile's tiles so far
    for (int t = 0; t < n_tiles && ok; ++t) {
      const int st = t % kStages;
      // (Also for a skipped tile: the stage's previous phase must be over before this arrival
      // may count towards the new one.)
      ok = mbar_wait(bar(&bars->k_full[st]), (t / kStages) & 1, abort_word, a.error_word, 44);
      if (!ok) break;
      if (!relevant(u, t)) {
        mbar_arrive(bar(&bars->k_empty[st]));
        continue;
      }
      ok = mbar_wait(bar(&bars->s_empty[u][c & 1]), ((c >> 1) & 1) ^ 1, abort_word, a.error_word, 43);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t kbase = key_u32 + st * kKeyBytes;
      const uint32_t d_tmem = tmem_base + (u * 2 + (c & 1)) * KT;
      // K hi and K lo meet the head's queries, the RoPE keys the RoPE queries.
#pragma unroll
      for (int kc = 0; kc < 3; ++kc) {
        const int qc = kc == 2 ? 1 : 0;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          const uint64_t ad = make_smem_desc(q_u32 + (u * 2 + qc) * QSUB + ks * 32, 16, 1024, kSwizzle128B);
          const uint64_t bd = make_smem_desc(kbase + kc * SUB + ks * 32, 16, 1024, kSwizzle128B);
          mma_bf16_ss(d_tmem, ad, bd, IDESC_QK, (kc > 0 || ks > 0) ? 1u : 0u);
        }
      }
      mma_commit(bar(&bars->s_full[u][c & 1]));
      mma_commit(bar(&bars->k_empty[st]));
      ++c;
    }
  } else if (warp == 3 && lane == 0) {
    // ------------------------------------------------------------------ value issuer (both query tiles)
    bool ok = true;
    int cu[kQTiles] = {0, 0};                      // each query tile's tiles so far
    for (int t = 0; t < n_tiles && ok; ++t) {
      const int st = t % kStages;
      ok = mbar_wait(bar(&bars->v_full[st]), (t / kStages) & 1, abort_word, a.error_word, 45);
      const uint32_t vbase = val_u32 + st * kValBytes;
      for (int u = 0; u < kQTiles && ok; ++u) {
        if (!relevant(u, t)) continue;
        const int c = cu[u]++;
        ok = mbar_wait(bar(&bars->p_full[u]), c & 1, abort_word, a.error_word, 46);
        if (!ok) break;
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < KT / 16; ++ks) {
          // A = P [128 rows x 64 keys], K-major; B = V [d_h columns x 64 keys], MN-major.
          const uint64_t ad = make_smem_desc(p_u32 + u * kPBytes + ks * 32, 16, 1024, kSwizzle128B);
          const uint64_t bd = make_smem_desc(vbase + ks * 2048, SUB, 1024, kSwizzle128B);
          mma_bf16_ss(tmem_base + kColO + u * 2 * DH, ad, bd, IDESC_PV, (c > 0 || ks > 0) ? 1u : 0u);
        }
        mma_commit(bar(&bars->p_empty[u]));
      }
      if (ok) mma_commit(bar(&bars->v_empty[st]));
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ softmax / epilogue of query tile u
    const int u = (warp - 4) >> 2;
    const int q = warp & 3, row = q * 32 + lane;           // query row within the tile = TMEM lane
    const int m = q0 + u * kQTile + row;                   // token index of this thread's row
    const int closed = m / a.stride;                       // closed slots this row may see
    const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
    const uint32_t o_base = lane_base + kColO + u * 2 * DH;
    bool ok = true;
    float m_run = -INFINITY, l_run = 0.f;
    int cnt = -1;                                  // this query tile's tiles so far
    for (int t = 0; t < n_tiles; ++t) {
      if (!relevant(u, t)) continue;
      ++cnt;
      if (ok) ok = mbar_wait(bar(&bars->s_full[u][cnt & 1]), (cnt >> 1) & 1, abort_word, a.error_word, 47);
      ok = __all_sync(0xffffffffu, ok);                    // TMEM accesses are whole-warp operations
      if (!ok) break;
      tc_fence_after_sync();
      const bool diag = t >= n_kv;
      // Key index of column 0: a closed slot, or an offset into the pair's own tokens, which this
      // row meets at column (its offset in the pair) - col0 if that falls inside the tile.
      const int col0 = diag ? (t - n_kv) * KT : t * KT;
      const int lim = diag ? 0 : closed - col0;
      const int own = (diag && m < a.T) ? u * kQTile + row - col0 : -1;
      uint32_t sv[KT];
#pragma unroll
      for (int c0 = 0; c0 < KT; c0 += 32) {
        uint32_t(&v)[32] = *reinterpret_cast<uint32_t(*)[32]>(&sv[c0]);
        tmem_ld_x32(lane_base + (u * 2 + (cnt & 1)) * KT + c0, v);
      }
      tmem_wait_ld();
      tc_fence_before_sync();
      mbar_arrive(bar(&bars->s_empty[u][cnt & 1]));       // the scores are in registers now
      uint32_t pk[KT / 2];
      // Fully visible tile and every row has a reference: probabilities at once, the tile's sum
      // tells whether a reference was outgrown (see prefill_attn_tc.cuh).
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
        if (__any_sync(0xffffffffu, raise && cnt > 0)) {
          // O rows are scaled to the old references: wait for the previous tile's value MMAs.
          ok = mbar_wait(bar(&bars->p_empty[u]), (cnt & 1) ^ 1, abort_word, a.error_word, 48);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after_sync();
#pragma unroll
          for (int c0 = 0; c0 < 2 * DH; c0 += 32) {
            uint32_t ov[32];
            tmem_ld_x32(o_base + c0, ov);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * fac);
            tmem_st_x32(o_base + c0, ov);
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
      // This query tile's probability buffer is free once its previous value MMAs have completed.
      ok = mbar_wait(bar(&bars->p_empty[u]), (cnt & 1) ^ 1, abort_word, a.error_word, 49);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      // P as the K-major, 128-byte-swizzled A operand: row r at r*128, its 16-byte piece c at
      // position c ^ (r % 8).
      uint8_t* prow = sm + kOffP + u * kPBytes + row * 128;
#pragma unroll
      for (int c0 = 0; c0 < KT; c0 += 8) {
        const int piece = c0 >> 3;
        *reinterpret_cast<uint4*>(prow + ((piece ^ (row & 7)) << 4)) =
            make_uint4(pk[c0 / 2], pk[c0 / 2 + 1], pk[c0 / 2 + 2], pk[c0 / 2 + 3]);
      }
      fence_proxy_async_smem();
      tc_fence_before_sync();
      mbar_arrive(bar(&bars->p_full[u]));
    }
    // Epilogue: wait for the last value MMAs, normalise this row and store hi / lo halves.
    if (ok) ok = mbar_wait(bar(&bars->p_empty[u]), (n_rel[u] - 1) & 1, abort_word, a.error_word, 50);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after_sync();
      const float inv = 1.f / l_run;
      bf16* o_hi = a.out + ((long long)b * a.T + m) * 2 * hd + h * DH;
#pragma unroll
      for (int c0 = 0; c0 < DH; c0 += 32) {
        uint32_t ov[32], ol[32];
        tmem_ld_x32(o_base + c0, ov);
        tmem_ld_x32(o_base + DH + c0, ol);
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
