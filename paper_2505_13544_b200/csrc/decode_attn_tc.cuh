// Tensor-core (tcgen05 / TMEM / TMA) split-K decode attention over the compressed cache in
// the absorbed form (Eq. 12 / Eq. 17), bf16 operands, fp32 accumulation.
//
// Work unit: one CTA per (split, sequence) streams its slot range in tiles of 128 slots.
// A tile is brought in by TMA as 64-column sub-tiles [128 slots x 128 B] with the 128-byte
// swizzle; the SAME shared-memory bytes feed both contractions, so every cache byte is read
// from HBM exactly once per step:
//   scores  S^T[128 slots x heads]  = tile[128 x (r+d_R)] . q~^T      A = tile, K-major
//   values  O^T[r x heads]         += tile[:, :r]^T . P^T[128 x heads] A = tile, MN-major
// Heads sit in the MMA's N dimension (16 or 32), slots / latent columns in M = 128, so no
// padding of heads up to M is paid for.  Accumulators live in TMEM: two score buffers and
// r/128 output blocks.  Warp roles: warp 0 = TMA producer (one thread), warp 1 = MMA issuer
// (one thread) and TMEM owner, warps 4-7 = softmax (one thread per slot of the tile).
//
// Shared memory: a ring of five 32 KB "pairs" (two adjacent 64-column sub-tiles = one
// 128-row MN-major operand block) + one 16 KB sub-tile for the RoPE-key columns + q~ as the
// K-major B operand + the bf16 probabilities P.  A tile needs r/128 pairs; with r = 512 the
// fifth pair lets the next tile's first loads overlap this tile's softmax and value MMAs.
//
// The online softmax rescales lazily: the reference maximum of a head is only raised when a
// tile exceeds it by more than 2^8, so the TMEM read-modify-write of O is rare.  Results are
// exact either way because the same reference enters numerator and denominator.
//
// Every wait is bounded (see sm100_ptx.cuh); on a timeout the CTA raises its abort word, all
// roles unwind, and the host sees MTLA_ERR_DEVICE_TIMEOUT from mtla_check.
#pragma once

#include <math.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mtla {

struct AttnTcArgs {
  const bf16* qt;      // [B][n_h][r + d_R] bf16, pre-scaled by log2(e)/sqrt(d_h)
  float* o_part;       // [B * n_split][n_h][r]
  float* ml_part;      // [B * n_split][n_h][2]
  int* error_word;
  int n_heads, r, dr, n_slots, slots_per_split, n_split;
};

namespace tc {

constexpr int kTile = 128;            // slots per tile
constexpr int kSubBytes = 128 * 128;  // one 64-column sub-tile
constexpr int kPairBytes = 2 * kSubBytes;
constexpr int kPairs = 5;
constexpr int kTmemCols = 256;
constexpr int kColS = 0;              // two score buffers at columns 0 and 32
constexpr int kColO = 64;             // output blocks at 64 + 32 * block
constexpr float kRescaleThreshold = 8.f;

constexpr int kOffPairs = 0;
constexpr int kOffKr = kPairs * kPairBytes;
constexpr int kOffQ = kOffKr + kSubBytes;
constexpr int kMaxQBytes = 32 * 576 * 2;
constexpr int kOffP = kOffQ + kMaxQBytes;
constexpr int kPBytes = 32 * kTile * 2;
constexpr int kOffMisc = kOffP + kPBytes;
constexpr int kMiscBytes = 2048;
constexpr int kSmemBytes = kOffMisc + kMiscBytes + 1024;  // + slack for 1024-byte alignment

struct Misc {
  unsigned long long full_pair[kPairs], empty_pair[kPairs];
  unsigned long long full_kr, empty_kr, s_full[2], s_empty[2], p_full, pv_done, group_sync;
  uint32_t tmem_base;
  int abort_word;
  int flag[2];
  float wmax[4][32];
  float cand_m[32], fac[32], m_cur[32];
  float lsum[4][32];
};
static_assert(sizeof(Misc) <= kMiscBytes, "misc region too small");

// Butterfly "transposed" reductions: every lane contributes 32 values; afterwards lane i
// holds the reduction over all lanes of value i (31 shuffles instead of 160).
template <typename Op>
__device__ __forceinline__ float transposed_reduce(float (&v)[32], int lane, Op op) {
#pragma unroll
  for (int off = 16, n = 32; off >= 1; off >>= 1, n >>= 1) {
    const bool upper = (lane & off) != 0;
#pragma unroll
    for (int i = 0; i < n / 2; ++i) {
      const float keep = upper ? v[i + n / 2] : v[i];
      const float send = upper ? v[i] : v[i + n / 2];
      v[i] = op(keep, __shfl_xor_sync(0xffffffffu, send, off));
    }
  }
  return v[0];
}

}  // namespace tc

// NHP: heads padded to the MMA's N (16 or 32).  RP: r / 128 (pairs per tile).
template <int NHP, int RP>
__global__ void __launch_bounds__(256, 1)
decode_attn_tc_kernel(const __grid_constant__ CUtensorMap cache_map, AttnTcArgs a) {
  using namespace tc;
  using namespace ptx;
  constexpr int WP = (2 * RP + 1) * 64;          // q~ width padded to whole 64-column chunks
  constexpr uint32_t SBOQ = (WP / 8) * 128;      // bytes between 8-head groups of q~
  constexpr uint32_t IDESC_QK = make_idesc_bf16(128, NHP, 0, 0);
  constexpr uint32_t IDESC_PV = make_idesc_bf16(128, NHP, 1, 0);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  Misc* misc = reinterpret_cast<Misc*>(sm + kOffMisc);
  volatile int* abort_word = &misc->abort_word;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  auto bar = [&](unsigned long long* p) { return smem_u32(p); };

  if (threadIdx.x == 0) {
    for (int i = 0; i < kPairs; ++i) {
      mbar_init(bar(&misc->full_pair[i]), 1);
      mbar_init(bar(&misc->empty_pair[i]), 1);
    }
    mbar_init(bar(&misc->full_kr), 1);
    mbar_init(bar(&misc->empty_kr), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(&misc->s_full[i]), 1);
      mbar_init(bar(&misc->s_empty[i]), 128);
    }
    mbar_init(bar(&misc->p_full), 128);
    mbar_init(bar(&misc->pv_done), 1);
    mbar_init(bar(&misc->group_sync), 128);
    misc->abort_word = 0;
    misc->flag[0] = 0;
    misc->flag[1] = 0;
    mbar_fence_init();
    prefetch_tensormap(&cache_map);
  }
  if (warp == 1) tmem_alloc(smem_u32(&misc->tmem_base), kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = misc->tmem_base;

  const int b = blockIdx.y, split = blockIdx.x;
  const int slot0 = split * a.slots_per_split;
  const int slot1 = min(a.n_slots, slot0 + a.slots_per_split);
  const int n_tiles = (slot1 - slot0 + kTile - 1) / kTile;
  const long long unit = (long long)b * a.n_split + split;
  const int W = a.r + a.dr;

  // q~ as the K-major, un-swizzled B operand: 8 x 16-byte core matrices, K-adjacent cores
  // 128 B apart, 8-head groups SBOQ apart.  Heads >= n_h and columns >= r + d_R are zero.
  {
    const bf16* q = a.qt + (long long)b * a.n_heads * W;
    for (int v = threadIdx.x; v < NHP * (WP / 8); v += 256) {
      const int n = v / (WP / 8), kc = v % (WP / 8);
      uint4 val = make_uint4(0, 0, 0, 0);
      if (n < a.n_heads && kc * 8 < W) val = *reinterpret_cast<const uint4*>(q + n * W + kc * 8);
      *reinterpret_cast<uint4*>(sm + kOffQ + (n >> 3) * SBOQ + kc * 128 + (n & 7) * 16) = val;
    }
    if (threadIdx.x >= 128 && threadIdx.x < 160) misc->m_cur[threadIdx.x - 128] = -INFINITY;
  }
  fence_proxy_async_smem();
  __syncthreads();

  const uint32_t pairs_u32 = base + kOffPairs, kr_u32 = base + kOffKr;
  const uint32_t q_u32 = base + kOffQ, p_u32 = base + kOffP;

  if (warp == 0 && lane == 0) {
    // ------------------------------------------------------------------ TMA producer
    bool ok = true;
    int pc = 0;
    for (int t = 0; t < n_tiles && ok; ++t) {
      const int slot = slot0 + t * kTile;
      ok = mbar_wait(bar(&misc->empty_kr), (t & 1) ^ 1, abort_word, a.error_word, 1);
      if (!ok) break;
      mbar_arrive_expect_tx(bar(&misc->full_kr), kSubBytes);
      tma_load_3d(kr_u32, &cache_map, bar(&misc->full_kr), a.r, slot, b);
      for (int c = 0; c < RP && ok; ++c, ++pc) {
        const int buf = pc % kPairs, use = pc / kPairs;
        ok = mbar_wait(bar(&misc->empty_pair[buf]), (use & 1) ^ 1, abort_word, a.error_word, 2);
        if (!ok) break;
        const uint32_t dst = pairs_u32 + buf * kPairBytes;
        mbar_arrive_expect_tx(bar(&misc->full_pair[buf]), kPairBytes);
        tma_load_3d(dst, &cache_map, bar(&misc->full_pair[buf]), c * 128, slot, b);
        tma_load_3d(dst + kSubBytes, &cache_map, bar(&misc->full_pair[buf]), c * 128 + 64, slot, b);
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ------------------------------------------------------------------ MMA issuer
    bool ok = true;
    // Score MMAs of one 64-column chunk held at `a_smem`; chunk index selects q~'s columns.
    auto qk_chunk = [&](uint32_t a_smem, int chunk, uint32_t d_tmem, bool first) {
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        const uint64_t ad = make_smem_desc(a_smem + ks * 32, 16, 1024, kSwizzle128B);
        const uint64_t bd = make_smem_desc(q_u32 + (chunk * 8 + ks * 2) * 128, 128, SBOQ, kSwizzleNone);
        mma_bf16_ss(d_tmem, ad, bd, IDESC_QK, (first && ks == 0) ? 0u : 1u);
      }
    };
    // Score phase for tile t, pairs [c_begin, c_end); the RoPE-key chunk goes first.
    auto qk_phase = [&](int t, int c_begin, int c_end) {
      const uint32_t d_tmem = tmem_base + kColS + (t & 1) * 32;
      if (c_begin == 0) {
        ok = mbar_wait(bar(&misc->s_empty[t & 1]), ((t >> 1) & 1) ^ 1, abort_word, a.error_word, 3);
        if (!ok) return;
        ok = mbar_wait(bar(&misc->full_kr), t & 1, abort_word, a.error_word, 4);
        if (!ok) return;
        tc_fence_after_sync();
        qk_chunk(kr_u32, 2 * RP, d_tmem, true);
        mma_commit(bar(&misc->empty_kr));
      }
      for (int c = c_begin; c < c_end; ++c) {
        const int pcn = t * RP + c, buf = pcn % kPairs, use = pcn / kPairs;
        ok = mbar_wait(bar(&misc->full_pair[buf]), use & 1, abort_word, a.error_word, 5);
        if (!ok) return;
        const uint32_t src = pairs_u32 + buf * kPairBytes;
        qk_chunk(src, 2 * c, d_tmem, false);
        qk_chunk(src + kSubBytes, 2 * c + 1, d_tmem, false);
      }
      if (c_end == RP) mma_commit(bar(&misc->s_full[t & 1]));
    };
    qk_phase(0, 0, RP);
    for (int t = 0; t < n_tiles && ok; ++t) {
      if (t + 1 < n_tiles) {
        qk_phase(t + 1, 0, 1);   // the spare pair: overlaps this tile's softmax
        if (!ok) break;
      }
      ok = mbar_wait(bar(&misc->p_full), t & 1, abort_word, a.error_word, 6);
      if (!ok) break;
      tc_fence_after_sync();
      for (int mb = 0; mb < RP; ++mb) {
        const int pcn = t * RP + mb, buf = pcn % kPairs;
        const uint32_t src = pairs_u32 + buf * kPairBytes;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t ad = make_smem_desc(src + ks * 2048, kSubBytes, 1024, kSwizzle128B);
          const uint64_t bd = make_smem_desc(p_u32 + ks * 256, 128, 2048, kSwizzleNone);
          mma_bf16_ss(tmem_base + kColO + mb * 32, ad, bd, IDESC_PV, (t == 0 && ks == 0) ? 0u : 1u);
        }
        mma_commit(bar(&misc->empty_pair[buf]));
      }
      mma_commit(bar(&misc->pv_done));
      if (RP > 1 && t + 1 < n_tiles) qk_phase(t + 1, 1, RP);
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ softmax warps
    const int q = warp - 4, row = q * 32 + lane, sidx = threadIdx.x - 128;
    const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
    bool ok = true;
    // Rendezvous of the 128 softmax threads on an mbarrier, so that it is bounded like
    // every other wait (a plain named barrier could not give up).
    int sync_phase = 0;
    auto group_sync = [&]() {
      mbar_arrive(bar(&misc->group_sync));
      ok = mbar_wait(bar(&misc->group_sync), sync_phase & 1, abort_word, a.error_word, 10);
      ++sync_phase;
      return ok;
    };
    float m_used[32], l_acc[32];
#pragma unroll
    for (int h = 0; h < 32; ++h) {
      m_used[h] = -INFINITY;
      l_acc[h] = 0.f;
    }
    for (int t = 0; t < n_tiles && ok; ++t) {
      ok = mbar_wait(bar(&misc->s_full[t & 1]), (t >> 1) & 1, abort_word, a.error_word, 7);
      if (!ok) break;
      tc_fence_after_sync();
      uint32_t sv[32];
      if (NHP == 32) tmem_ld_x32(lane_base + kColS + (t & 1) * 32, sv);
      else tmem_ld_x16(lane_base + kColS + (t & 1) * 32, sv);
      tmem_wait_ld();
      tc_fence_before_sync();
      mbar_arrive(bar(&misc->s_empty[t & 1]));

      const bool valid = slot0 + t * kTile + row < slot1;
      float s[32], red[32];
#pragma unroll
      for (int h = 0; h < 32; ++h) {
        s[h] = (valid && h < NHP) ? __uint_as_float(sv[h]) : -INFINITY;
        red[h] = s[h];
      }
      misc->wmax[q][lane] = transposed_reduce(red, lane, [](float x, float y) { return fmaxf(x, y); });
      if (!group_sync()) break;
      if (sidx < 32) {
        const float mt = fmaxf(fmaxf(misc->wmax[0][sidx], misc->wmax[1][sidx]),
                               fmaxf(misc->wmax[2][sidx], misc->wmax[3][sidx]));
        const float m_old = misc->m_cur[sidx];
        const float m_new = fmaxf(m_old, mt);
        misc->cand_m[sidx] = m_new;
        misc->fac[sidx] = (m_new == -INFINITY) ? 1.f : exp2f(m_old - m_new);
        if (mt > m_old + kRescaleThreshold) misc->flag[t & 1] = 1;
        if (sidx == 0) misc->flag[(t + 1) & 1] = 0;
      }
      if (!group_sync()) break;
      const bool rescale = misc->flag[t & 1] != 0;
      if (rescale) {
#pragma unroll
        for (int h = 0; h < 32; ++h) {
          m_used[h] = misc->cand_m[h];
          l_acc[h] *= misc->fac[h];
        }
        if (sidx < 32) misc->m_cur[sidx] = misc->cand_m[sidx];
      }
      uint32_t pb[16];
#pragma unroll
      for (int h = 0; h < NHP; h += 2) {
        const float p0 = exp2f(s[h] - m_used[h]), p1 = exp2f(s[h + 1] - m_used[h + 1]);
        const __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
        l_acc[h] += __low2float(pk);
        l_acc[h + 1] += __high2float(pk);
        pb[h / 2] = *reinterpret_cast<const uint32_t*>(&pk);
      }
      if (t > 0) {
        ok = mbar_wait(bar(&misc->pv_done), (t - 1) & 1, abort_word, a.error_word, 8);
        if (!ok) break;
        tc_fence_after_sync();
        if (rescale) {
          for (int mb = 0; mb < RP; ++mb) {
            uint32_t ov[32];
            const uint32_t addr = lane_base + kColO + mb * 32;
            if (NHP == 32) tmem_ld_x32(addr, ov); else tmem_ld_x16(addr, ov);
            tmem_wait_ld();
#pragma unroll
            for (int h = 0; h < NHP; ++h) ov[h] = __float_as_uint(__uint_as_float(ov[h]) * misc->fac[h]);
            if (NHP == 32) tmem_st_x32(addr, ov); else tmem_st_x16(addr, ov);
          }
          tmem_wait_st();
        }
      }
      // P^T as the K-major, un-swizzled B operand of the value MMA: element (head n, slot k)
      // at (n/8)*2048 + (k/8)*128 + (n%8)*16 + (k%8)*2.
      uint8_t* prow = sm + kOffP + (row >> 3) * 128 + (row & 7) * 2;
#pragma unroll
      for (int h = 0; h < NHP; ++h) {
        const uint16_t bits = (h & 1) ? (uint16_t)(pb[h / 2] >> 16) : (uint16_t)(pb[h / 2] & 0xffffu);
        *reinterpret_cast<uint16_t*>(prow + (h >> 3) * 2048 + (h & 7) * 16) = bits;
      }
      fence_proxy_async_smem();
      tc_fence_before_sync();
      mbar_arrive(bar(&misc->p_full));
    }
    if (ok && n_tiles > 0) {
      ok = mbar_wait(bar(&misc->pv_done), (n_tiles - 1) & 1, abort_word, a.error_word, 9);
    }
    if (ok && n_tiles > 0) {
      tc_fence_after_sync();
      float* o_part = a.o_part + unit * a.n_heads * a.r;
      for (int mb = 0; mb < RP; ++mb) {
        uint32_t ov[32];
        const uint32_t addr = lane_base + kColO + mb * 32;
        if (NHP == 32) tmem_ld_x32(addr, ov); else tmem_ld_x16(addr, ov);
        tmem_wait_ld();
#pragma unroll
        for (int h = 0; h < NHP; ++h)
          if (h < a.n_heads) o_part[h * a.r + mb * 128 + row] = __uint_as_float(ov[h]);
      }
      misc->lsum[q][lane] = transposed_reduce(l_acc, lane, [](float x, float y) { return x + y; });
      if (group_sync() && sidx < a.n_heads) {
        const float l = misc->lsum[0][sidx] + misc->lsum[1][sidx] + misc->lsum[2][sidx] +
                        misc->lsum[3][sidx];
        a.ml_part[(unit * a.n_heads + sidx) * 2] = misc->m_cur[sidx];
        a.ml_part[(unit * a.n_heads + sidx) * 2 + 1] = l;
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
