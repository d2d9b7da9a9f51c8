// Persistent tensor-core GEMM for the large bf16 products:
//     D[z][i][j] = alpha * sum_k A[z][i][k] * B[z][j][k]
// Same operands, tensor maps, output addressing and hi / lo conventions as gemm_tc_kernel
// (gemm_tc.cuh); what differs is the schedule.  One CTA per SM stays resident and walks a
// contiguous share of the product's k-block list (tile-major, 64 reduction columns per block):
//
//   * few tiles and a long reduction (the decode step's weight-streaming products: every weight
//     byte is read once, the batch sits in the MMA's N): the list is cut into equal shares
//     wherever the cut falls, so every SM streams the same number of weight bytes through one
//     deep TMA ring that never drains between tiles.  A share that ends inside a tile leaves a
//     partial accumulator in a workspace; the CTA that delivers a tile's last partial sums them
//     in share order (an atomic ticket per 32-row quarter, never a wait), so the result does
//     not depend on arrival order;
//   * many tiles (the prefill's projections): shares are cut at tile boundaries, nothing is
//     partial, and the CTA simply runs tile after tile.
//
// The accumulator is double-buffered in TMEM: while the four epilogue warps drain (and, for a
// partial, reduce) one buffer, the MMA issuer is already filling the other, so the epilogue of a
// segment overlaps the main loop of the next.  Warp roles: warp 0 = TMA producer, warp 1 = MMA
// issuer and TMEM owner, warps 2-5 = epilogue (one TMEM lane quarter each).  Every mbarrier wait
// is bounded (sm100_ptx.cuh).
#pragma once

#include "common.cuh"
#include "gemm_tc.cuh"
#include "sm100_ptx.cuh"

namespace mtla {

struct GemmStreamArgs {
  GemmTcArgs g;          // operands and output as for gemm_tc_kernel (n_split / kb_per_split unused)
  int batches;           // z extent
  int whole_tiles;       // 1: shares end at tile boundaries (no partials)
  float* parts;          // [gridDim.x + tiles][BN][128] fp32 partial accumulators
};

namespace gts {

using gtc::kBM;
using gtc::kBK;
using gtc::kABytes;

__host__ __device__ constexpr int stages_for(int nb) { return nb <= 64 ? 8 : nb <= 128 ? 6 : 4; }
__host__ __device__ constexpr int smem_bytes(int nb) {
  return stages_for(nb) * gtc::stage_bytes(nb) + 1024 /* alignment slack */ + 256 /* barriers */;
}

struct Bars {
  unsigned long long full[8], empty[8], acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int abort_word;
};
static_assert(sizeof(Bars) <= 256, "barrier block too large");

// First k-block of CTA c's share of a list of `total` k-blocks dealt to G CTAs.
__host__ __device__ inline long long share_begin(long long c, long long total, long long G) {
  return c * total / G;
}
// The CTA whose share contains k-block i.
__host__ __device__ inline long long share_owner(long long i, long long total, long long G) {
  return ((i + 1) * G - 1) / total;
}

// A CTA's share as a sequence of segments: (tile, first k-block, end k-block) within one tile.
struct Segments {
  long long pos, end;
  int kb_total;
  __device__ __forceinline__ bool next(long long& tile, int& kb0, int& kb1) {
    if (pos >= end) return false;
    tile = pos / kb_total;
    const long long tile_end = (tile + 1) * kb_total;
    const long long stop = tile_end < end ? tile_end : end;
    kb0 = (int)(pos - tile * kb_total);
    kb1 = (int)(stop - tile * kb_total);
    pos = stop;
    return true;
  }
};

}  // namespace gts

template <int BN, typename OutT, bool HILO>
__global__ void __launch_bounds__(192, 1)
gemm_tc_stream_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                      GemmStreamArgs s) {
  using namespace gts;
  using namespace ptx;
  static_assert(BN == 16 || BN == 32 || BN == 64 || BN == 128 || BN == 256, "BN");
  constexpr int CH = BN < 32 ? 16 : 32;             // TMEM columns per epilogue chunk
  constexpr int NB = HILO ? 2 * BN : BN;            // rows of the B tile = the MMA's N
  static_assert(NB <= 256, "stacked hi / lo halves exceed the MMA's N");
  constexpr int STAGES = stages_for(NB);
  constexpr int STAGE = gtc::stage_bytes(NB);
  constexpr uint32_t IDESC = make_idesc_bf16(128, NB, 0, 0);
  constexpr uint32_t TMEM_COLS = 2 * NB < 32 ? 32 : 2 * NB;   // two accumulator buffers
  static_assert(TMEM_COLS <= 512, "accumulators exceed tensor memory");
  const GemmTcArgs& g = s.g;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  Bars* bars = reinterpret_cast<Bars*>(sm + STAGES * STAGE);
  volatile int* abort_word = &bars->abort_word;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  auto bar = [&](unsigned long long* p) { return smem_u32(p); };

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) {
      mbar_init(bar(&bars->full[i]), 1);
      mbar_init(bar(&bars->empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(&bars->acc_full[i]), 1);
      mbar_init(bar(&bars->acc_empty[i]), 4);       // one arrival per epilogue warp
    }
    bars->abort_word = 0;
    mbar_fence_init();
    prefetch_tensormap(&map_a);
    prefetch_tensormap(&map_b);
  }
  if (warp == 1) tmem_alloc(smem_u32(&bars->tmem_base), TMEM_COLS);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;
  grid_launch_dependents();      // this CTA owns its TMEM columns: successors may start
  grid_dependency_wait();        // nothing before this line touches the previous kernel's data

  const int kb_total = (g.k + kBK - 1) / kBK;
  const long long tiles = (long long)g.m_tiles * g.n_tiles * s.batches;
  const long long total = tiles * kb_total, G = gridDim.x;
  long long g0, g1;
  if (s.whole_tiles) {
    g0 = share_begin(blockIdx.x, tiles, G) * kb_total;
    g1 = share_begin(blockIdx.x + 1, tiles, G) * kb_total;
  } else {
    g0 = share_begin(blockIdx.x, total, G);
    g1 = share_begin(blockIdx.x + 1, total, G);
  }
  const int passes = (!HILO && g.b_lo_col > 0) ? 2 : 1;
  // Tile index -> (A tile, B tile, z): A tiles fastest, so neighbouring shares meet one B panel.
  auto tile_coords = [&](long long tile, int& mt, int& nt, int& z) {
    mt = (int)(tile % g.m_tiles);
    const long long rest = tile / g.m_tiles;
    nt = (int)(rest % g.n_tiles);
    z = (int)(rest / g.n_tiles);
  };

  if (warp == 0 && lane == 0) {
    // ------------------------------------------------------------------ TMA producer
    Segments seg{g0, g1, kb_total};
    long long tile;
    int kb0, kb1, it = 0;
    bool ok = true;
    while (ok && seg.next(tile, kb0, kb1)) {
      int mt, nt, z;
      tile_coords(tile, mt, nt, z);
      const int a_row = z * g.a_row_z + mt * kBM, b_row = z * g.b_row_z + nt * BN;
      const int a_col = z * g.a_col_z, b_col = z * g.b_col_z;
      for (int kb = kb0; kb < kb1 && ok; ++kb)
        for (int lo = 0; lo < passes; ++lo, ++it) {
          const int st = it % STAGES, use = it / STAGES;
          ok = mbar_wait(bar(&bars->empty[st]), (use & 1) ^ 1, abort_word, g.error_word, 31);
          if (!ok) break;
          const uint32_t dst = base + st * STAGE;
          mbar_arrive_expect_tx(bar(&bars->full[st]), STAGE);
          tma_load_2d(dst, &map_a, bar(&bars->full[st]), a_col + kb * kBK, a_row);
          tma_load_2d(dst + kABytes, &map_b, bar(&bars->full[st]), b_col + lo * g.b_lo_col + kb * kBK,
                      b_row);
          if (HILO)
            tma_load_2d(dst + kABytes + gtc::b_bytes(BN), &map_b, bar(&bars->full[st]),
                        b_col + g.b_lo_col + kb * kBK, b_row);
        }
    }
  } else if (warp == 1 && lane == 0) {
    // ------------------------------------------------------------------ MMA issuer
    Segments seg{g0, g1, kb_total};
    long long tile;
    int kb0, kb1, it = 0, n_seg = 0;
    bool ok = true;
    while (ok && seg.next(tile, kb0, kb1)) {
      const int acc = n_seg & 1;
      // The buffer is free once the epilogue has drained the segment before last.
      ok = mbar_wait(bar(&bars->acc_empty[acc]), ((n_seg >> 1) & 1) ^ 1, abort_word, g.error_word, 32);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t d_tmem = tmem_base + acc * NB;
      const int n_it = (kb1 - kb0) * passes;
      for (int i = 0; i < n_it; ++i, ++it) {
        const int st = it % STAGES, use = it / STAGES;
        ok = mbar_wait(bar(&bars->full[st]), use & 1, abort_word, g.error_word, 33);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t a_smem = base + st * STAGE, b_smem = a_smem + kABytes;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          const uint64_t ad = make_smem_desc(a_smem + ks * 32, 16, 1024, kSwizzle128B);
          const uint64_t bd = make_smem_desc(b_smem + ks * 32, 16, 1024, kSwizzle128B);
          mma_bf16_ss(d_tmem, ad, bd, IDESC, (i > 0 || ks > 0) ? 1u : 0u);
        }
        mma_commit(bar(&bars->empty[st]));
      }
      if (ok) mma_commit(bar(&bars->acc_full[acc]));
      ++n_seg;
    }
  } else if (warp >= 2) {
    // ------------------------------------------------------------------ epilogue warps
    const int q = warp & 3;                        // TMEM lane quarter this warp may read
    const int row_local = q * 32 + lane;
    Segments seg{g0, g1, kb_total};
    long long tile;
    int kb0, kb1, n_seg = 0;
    while (seg.next(tile, kb0, kb1)) {
      const int acc = n_seg & 1;
      int ok = mbar_wait(bar(&bars->acc_full[acc]), (n_seg >> 1) & 1, abort_word, g.error_word, 34) ? 1 : 0;
      ok = __all_sync(0xffffffffu, ok);            // the warp proceeds or gives up as one
      if (!ok) break;
      tc_fence_after_sync();
      int mt, nt, z;
      tile_coords(tile, mt, nt, z);
      const int i_row = mt * kBM + row_local;      // A-row index of this thread
      const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16) + acc * NB;
      OutT* c = static_cast<OutT*>(g.c) + (long long)z * g.c_sz;
      const bool row_ok = i_row < g.m;
      auto put = [&](OutT* p, float val) {
        const OutT hi = Elem<OutT>::from_float(val);
        *p = hi;
        if (sizeof(OutT) == 2 && g.c_lo_off > 0)
          p[g.c_lo_off] = Elem<OutT>::from_float(val - Elem<OutT>::to_float(hi));
      };
      auto emit = [&](const uint32_t (&v)[32], int c0) {
        const int j0 = nt * BN + c0;
        if (!row_ok) return;
        if (g.c_sn == 1) {
          OutT* p = c + (long long)i_row * g.c_sm + j0;
          if (g.vec_ok && g.c_lo_off == 0 && j0 + CH <= g.n) {
            gtc::store_row32<OutT>(p, v, g.alpha, CH);
          } else {
#pragma unroll
            for (int j = 0; j < CH; ++j)
              if (j0 + j < g.n) put(p + j, gtc::finish(g, __uint_as_float(v[j]), i_row, j0 + j));
          }
        } else {
          OutT* p = c + (long long)i_row * g.c_sm;
#pragma unroll
          for (int j = 0; j < CH; ++j)
            if (j0 + j < g.n)
              put(p + (long long)(j0 + j) * g.c_sn, gtc::finish(g, __uint_as_float(v[j]), i_row, j0 + j));
        }
      };
      // Accumulator columns c0 .. c0 + CH of this thread's row (hi and lo products added).
      auto load_acc = [&](int c0, uint32_t (&v)[32]) {
        if (CH == 32) tmem_ld_x32(lane_base + c0, v); else tmem_ld_x16(lane_base + c0, v);
        if (HILO) {
          uint32_t w[32];
          if (CH == 32) tmem_ld_x32(lane_base + BN + c0, w); else tmem_ld_x16(lane_base + BN + c0, w);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < CH; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(w[j]));
        } else {
          tmem_wait_ld();
        }
      };
      const bool whole = kb0 == 0 && kb1 == kb_total;
      if (whole) {
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += CH) {
          uint32_t v[32];
          load_acc(c0, v);
          emit(v, c0);
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(&bars->acc_empty[acc]));
      } else {
        // A partial: to the workspace slot of (this CTA, this tile), then a ticket.  Slots of one
        // tile's parts are consecutive and in share order: first owner + tile, ...
        float* part = s.parts + ((long long)blockIdx.x + tile) * (long long)(BN * kBM);
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += CH) {
          uint32_t v[32];
          load_acc(c0, v);
#pragma unroll
          for (int j = 0; j < CH; ++j) part[(c0 + j) * kBM + row_local] = __uint_as_float(v[j]);
        }
        // The accumulator is in the workspace: the issuer may reuse the buffer while this warp
        // goes on to the ticket and, if it is the last, the sum.
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(&bars->acc_empty[acc]));
        const long long k_first = tile * kb_total;
        const long long c_first = share_owner(k_first, total, G);
        const int n_parts = (int)(share_owner(k_first + kb_total - 1, total, G) - c_first) + 1;
        __threadfence();
        __syncwarp();
        int last = 0;
        if (lane == 0) {
          int* ticket = g.tickets + tile * 4 + q;
          last = atomicAdd(ticket, 1) == n_parts - 1;
          if (last) *ticket = 0;               // every other part has already arrived
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
          __threadfence();
          // This warp sums its 32-row quarter over the parts, in share order.  Lane l owns rows
          // 4*(l%8)..+3 of column (l/8) in each group of four columns: every load is a 16-byte
          // vector and a warp instruction covers 512 contiguous bytes.  The sum is bound by the
          // L2 round trip, so as many loads as the registers hold are in flight: U column groups
          // of up to four parts at a time.
          const float* all = s.parts + (c_first + tile) * (long long)(BN * kBM) + q * 32;
          const int r4 = 4 * (lane & 7), cs = lane >> 3;
          constexpr int U = BN >= 32 ? 8 : 4;           // column groups per step (BN / 4 >= U)
#pragma unroll 1
          for (int jb = 0; jb < BN; jb += 4 * U) {
            float4 accv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) accv[u] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
            for (int sp0 = 0; sp0 < n_parts; sp0 += 4) {
              float4 t[4][U];
#pragma unroll
              for (int s4 = 0; s4 < 4; ++s4)
#pragma unroll
                for (int u = 0; u < U; ++u)
                  t[s4][u] = sp0 + s4 < n_parts
                                 ? __ldcg(reinterpret_cast<const float4*>(
                                       all + (long long)(sp0 + s4) * (BN * kBM) +
                                       (jb + u * 4 + cs) * kBM + r4))
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
              for (int s4 = 0; s4 < 4; ++s4)
#pragma unroll
                for (int u = 0; u < U; ++u) {
                  accv[u].x += t[s4][u].x; accv[u].y += t[s4][u].y;
                  accv[u].z += t[s4][u].z; accv[u].w += t[s4][u].w;
                }
            }
            const int i0 = mt * kBM + q * 32 + r4;
#pragma unroll
            for (int u = 0; u < U; ++u) {
              const int j = nt * BN + jb + u * 4 + cs;
              if (j >= g.n || i0 >= g.m) continue;
              const float sum[4] = {accv[u].x, accv[u].y, accv[u].z, accv[u].w};
              OutT* p = c + (long long)j * g.c_sn + (long long)i0 * g.c_sm;
              if (g.vec4_ok) {
                const float val[4] = {g.alpha * sum[0], g.alpha * sum[1], g.alpha * sum[2], g.alpha * sum[3]};
                gtc::store4(p, val, g.c_lo_off);
              } else {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                  if (i0 + e < g.m) put(p + (long long)e * g.c_sm, gtc::finish(g, sum[e], i0 + e, j));
              }
            }
          }
        }
      }
      ++n_seg;
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
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

}  // namespace mtla
