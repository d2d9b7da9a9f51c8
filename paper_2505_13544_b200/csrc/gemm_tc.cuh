// Tensor-core (tcgen05 / TMEM / TMA) GEMM for the bf16 projections:
//     D[z][i][j] = alpha * sum_k A[z][i][k] * B[z][j][k]
// Both operands are bf16 and K-contiguous, reached through 2-D tensor maps (128-byte
// swizzle, 64-column boxes).  A supplies the MMA's M = 128 rows per CTA, B its N = BN rows,
// the fp32 accumulator [128 x BN] lives in TMEM.  The output is addressed through two element
// strides, so either operand may be the weights.  The library puts the weights [out][in] on
// the A side and the activation rows on the B side (c_sm = 1, c_sn = leading dimension):
//   * decode (few activation rows): every weight byte is streamed from HBM exactly once and
//     split-K spreads one weight panel over several CTAs;
//   * prefill (many activation rows): neighbouring CTAs share one 128-row activation panel
//     and sweep the weight tiles, which stay in L2.
// Stores are coalesced across the warp (lane = output feature) in that orientation; the
// row-major orientation (c_sn = 1) stores 16-byte vectors per thread.
// Per-z offsets select a head's rows / K-columns for the per-head products (query absorption,
// Eq. 12; value up-projection, Eq. 10).
//
// Activations that were produced in fp32 by an earlier kernel can be passed as two bf16 halves
// (value = hi + lo), which keeps fp32-like precision of the intermediate.  With HILO the two
// halves of the BN activation rows are stacked as one B tile of 2 BN rows, so a single MMA per
// k-step multiplies the weight tile by both and the epilogue adds the two column halves of the
// accumulator; when 2 BN would exceed the MMA's N (BN = 256) each K block is run twice instead.
//
// Split-K partials go to a workspace; the last CTA (per 32-row quarter of a tile) to take a
// ticket sums them in split order, so results do not depend on arrival order and no CTA ever
// waits for another.  Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner,
// warps 2-5 = epilogue (one TMEM lane quarter each).  All mbarrier waits are bounded.
#pragma once

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mtla {

struct GemmTcArgs {
  void* c;                    // output base
  long long c_sm, c_sn, c_sz; // element strides of the output: A-row index, B-row index, z
  int m, n, k;                // per-z extents: A rows, B rows, reduction length
  int a_row_z, b_row_z;       // per-z row offsets into the A / B tensors
  int a_col_z, b_col_z;       // per-z K-column offsets into the A / B tensors
  int b_lo_col;               // > 0: B rows hold [hi | lo] bf16 halves of an fp32 activation, lo
                              // starting at this column; both halves are multiplied (2 passes
                              // over each K block), which keeps ~16 mantissa bits of B
  int b_k_wrap;               // K blocks after which B's K index starts over (A holds [hi | lo]
                              // halves of a weight along K, both multiplied by the same B columns);
                              // a value >= the K blocks of the product leaves B unwrapped
  long long c_lo_off;         // > 0 (bf16 output only): also store the rounding remainder
                              // bf16(val - bf16(val)) this many elements after each output
  int kb_per_split, n_split;  // K blocks (of 64) per split; number of splits
  int m_tiles, n_tiles;       // tiles along A / B rows: gridDim.x = m_tiles * n_tiles * n_split,
                              // A tiles fastest (neighbouring CTAs share the B panel)
  int vec_ok;                 // 1: c, c_sm, c_sz keep 16-byte alignment for the row-major path
  int vec4_ok;                // 1: c_sm == 1, m % 4 == 0 and every column start is 16-byte aligned,
                              // so the split-K reduction may store four rows at once
  float alpha;
  // Optional epilogue, applied to alpha * sum in this order (feed-forward block of a decoder
  // layer): + bias[i] (one value per A row = output feature), ReLU, + residual[i * r_sm + j * r_sn]
  // (fp32, may alias the output: every element is read and written by the same thread).
  const float* bias;
  const float* residual;
  long long r_sm, r_sn;
  int relu;
  // Optional second destination (the QSPLIT instantiations; the prefill's fused projection):
  // output features below q_rows are the queries; they go, scaled and rounded to bf16, straight
  // into the attention's query rows [token][head][q_dq] instead of the fp32 output.
  bf16* q_out;
  int q_rows, q_dh_shift, q_dq;   // d_h = 1 << q_dh_shift; q_dq = d_h + d_R
  long long q_sn;                 // elements between the query rows of consecutive tokens
  float q_scale;
  float* partial;             // [tiles][n_split][BN][128] fp32 (split-K only)
  int* tickets;               // [tiles][4], zero between launches (split-K only)
  int* error_word;
};

namespace gtc {

constexpr int kBM = 128, kBK = 64;
constexpr int kABytes = kBM * kBK * 2;

__host__ __device__ constexpr int b_bytes(int bn) { return bn * kBK * 2; }
// `nb` = rows of the B tile (BN, or 2 BN with stacked hi / lo halves).
__host__ __device__ constexpr int stage_bytes(int nb) { return kABytes + b_bytes(nb); }
__host__ __device__ constexpr int smem_bytes(int nb, int stages) {
  return stages * stage_bytes(nb) + 1024 /* alignment slack */ + 256 /* barriers */;
}

struct Bars {
  unsigned long long full[8], empty[8], acc_full;
  uint32_t tmem_base;
  int abort_word;
};
static_assert(sizeof(Bars) <= 256, "barrier block too large");

template <typename OutT>
__device__ __forceinline__ void store_row32(OutT* p, const uint32_t (&v)[32], float alpha, int count);

template <>
__device__ __forceinline__ void store_row32<float>(float* p, const uint32_t (&v)[32], float alpha,
                                                   int count) {
#pragma unroll
  for (int j = 0; j < 32; j += 4)
    if (j < count)
      *reinterpret_cast<float4*>(p + j) =
          make_float4(alpha * __uint_as_float(v[j]), alpha * __uint_as_float(v[j + 1]),
                      alpha * __uint_as_float(v[j + 2]), alpha * __uint_as_float(v[j + 3]));
}
template <>
__device__ __forceinline__ void store_row32<bf16>(bf16* p, const uint32_t (&v)[32], float alpha,
                                                  int count) {
#pragma unroll
  for (int j = 0; j < 32; j += 8)
    if (j < count) {
      uint32_t w[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const __nv_bfloat162 h = __floats2bfloat162_rn(alpha * __uint_as_float(v[j + 2 * e]),
                                                       alpha * __uint_as_float(v[j + 2 * e + 1]));
        w[e] = *reinterpret_cast<const uint32_t*>(&h);
      }
      *reinterpret_cast<uint4*>(p + j) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// Stores four consecutive outputs (and, for bf16 with lo_off > 0, their rounding remainders).
__device__ __forceinline__ void store4(float* p, const float (&v)[4], long long) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ void store4(bf16* p, const float (&v)[4], long long lo_off) {
  const __nv_bfloat162 h0 = __floats2bfloat162_rn(v[0], v[1]), h1 = __floats2bfloat162_rn(v[2], v[3]);
  *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<const uint32_t*>(&h0),
                                            *reinterpret_cast<const uint32_t*>(&h1));
  if (lo_off > 0) {
    const __nv_bfloat162 l0 = __floats2bfloat162_rn(v[0] - __low2float(h0), v[1] - __high2float(h0));
    const __nv_bfloat162 l1 = __floats2bfloat162_rn(v[2] - __low2float(h1), v[3] - __high2float(h1));
    *reinterpret_cast<uint2*>(p + lo_off) = make_uint2(*reinterpret_cast<const uint32_t*>(&l0),
                                                       *reinterpret_cast<const uint32_t*>(&l1));
  }
}

// The finished value of output (i, j): scale, then - in the instantiations that carry them - the
// optional bias / ReLU / residual.  (Run-time flags instead of the template parameter slowed
// the plain products' epilogue by a third.)
template <bool EXTRAS>
__device__ __forceinline__ float finish(const GemmTcArgs& g, float acc, int i, int j) {
  float v = g.alpha * acc;
  if constexpr (EXTRAS) {
    if (g.bias) v += g.bias[i];
    if (g.relu) v = fmaxf(v, 0.f);
    if (g.residual) v += g.residual[(long long)i * g.r_sm + (long long)j * g.r_sn];
  }
  return v;
}

}  // namespace gtc

template <int BN, int STAGES, typename OutT, bool HILO, bool EXTRAS = false, bool QSPLIT = false>
__global__ void __launch_bounds__(192, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               GemmTcArgs g) {
  using namespace gtc;
  using namespace ptx;
  static_assert(BN == 16 || BN == 32 || BN == 64 || BN == 128 || BN == 256, "BN");
  static_assert(STAGES >= 2 && STAGES <= 8, "STAGES");
  constexpr int CH = BN < 32 ? 16 : 32;             // TMEM columns per epilogue chunk
  constexpr int NB = HILO ? 2 * BN : BN;            // rows of the B tile = the MMA's N
  static_assert(NB <= 256, "stacked hi / lo halves exceed the MMA's N");
  constexpr uint32_t IDESC = make_idesc_bf16(128, NB, 0, 0);
  constexpr uint32_t TMEM_COLS = NB < 32 ? 32 : NB;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  Bars* bars = reinterpret_cast<Bars*>(sm + STAGES * stage_bytes(NB));
  volatile int* abort_word = &bars->abort_word;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  auto bar = [&](unsigned long long* p) { return smem_u32(p); };

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) {
      mbar_init(bar(&bars->full[i]), 1);
      mbar_init(bar(&bars->empty[i]), 1);
    }
    mbar_init(bar(&bars->acc_full), 1);
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
  // Only now may the next kernel's CTAs start: this CTA owns its TMEM columns, so a successor
  // that shares the SM cannot take them first and then sit in its dependency wait.
  grid_launch_dependents();
  grid_dependency_wait();        // nothing before this line touches the previous kernel's data

  const int mt = blockIdx.x % g.m_tiles, ny = blockIdx.x / g.m_tiles;
  const int nt = ny / g.n_split, split = ny % g.n_split;
  const int z = blockIdx.z;
  const int kb_total = (g.k + kBK - 1) / kBK;
  const int kb0 = split * g.kb_per_split;
  const int n_kb = min(kb_total, kb0 + g.kb_per_split) - kb0;   // >= 1 by construction
  const int passes = (!HILO && g.b_lo_col > 0) ? 2 : 1;
  const int n_it = n_kb * passes;

  if (warp == 0 && lane == 0) {
    // ------------------------------------------------------------------ TMA producer
    const int a_row = z * g.a_row_z + mt * kBM, b_row = z * g.b_row_z + nt * BN;
    const int a_col = z * g.a_col_z, b_col = z * g.b_col_z;
    for (int i = 0; i < n_it; ++i) {
      const int st = i % STAGES, use = i / STAGES;
      const int kb = kb0 + (passes == 2 ? i >> 1 : i), lo = passes == 2 ? (i & 1) : 0;
      if (!mbar_wait(bar(&bars->empty[st]), (use & 1) ^ 1, abort_word, g.error_word, 11)) break;
      const uint32_t dst = base + st * stage_bytes(NB);
      mbar_arrive_expect_tx(bar(&bars->full[st]), stage_bytes(NB));
      tma_load_2d(dst, &map_a, bar(&bars->full[st]), a_col + kb * kBK, a_row);
      const int kbb = kb - (kb >= g.b_k_wrap ? g.b_k_wrap : 0);
      tma_load_2d(dst + kABytes, &map_b, bar(&bars->full[st]), b_col + lo * g.b_lo_col + kbb * kBK,
                  b_row);
      if (HILO)
        tma_load_2d(dst + kABytes + b_bytes(BN), &map_b, bar(&bars->full[st]),
                    b_col + g.b_lo_col + kbb * kBK, b_row);
    }
  } else if (warp == 1 && lane == 0) {
    // ------------------------------------------------------------------ MMA issuer
    bool ok = true;
    for (int i = 0; i < n_it && ok; ++i) {
      const int st = i % STAGES, use = i / STAGES;
      ok = mbar_wait(bar(&bars->full[st]), use & 1, abort_word, g.error_word, 12);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t a_smem = base + st * stage_bytes(NB), b_smem = a_smem + kABytes;
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        const uint64_t ad = make_smem_desc(a_smem + ks * 32, 16, 1024, kSwizzle128B);
        const uint64_t bd = make_smem_desc(b_smem + ks * 32, 16, 1024, kSwizzle128B);
        mma_bf16_ss(tmem_base, ad, bd, IDESC, (i > 0 || ks > 0) ? 1u : 0u);
      }
      mma_commit(bar(&bars->empty[st]));
    }
    if (ok) mma_commit(bar(&bars->acc_full));
  } else if (warp >= 2) {
    // ------------------------------------------------------------------ epilogue warps
    const int q = warp & 3;                        // TMEM lane quarter this warp may read
    const int row_local = q * 32 + lane;
    const int i_row = mt * kBM + row_local;        // A-row index of this thread
    int ok = mbar_wait(bar(&bars->acc_full), 0, abort_word, g.error_word, 13) ? 1 : 0;
    ok = __all_sync(0xffffffffu, ok);              // the warp proceeds or gives up as one
    if (ok) {
      tc_fence_after_sync();
      const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
      OutT* c = static_cast<OutT*>(g.c) + (long long)z * g.c_sz;
      const long long tile = ((long long)z * g.m_tiles + mt) * g.n_tiles + nt;
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
        if constexpr (QSPLIT) {
          if (i_row < g.q_rows) {        // uniform over the CTA: q_rows is a multiple of 128
            bf16* p = g.q_out + (i_row >> g.q_dh_shift) * g.q_dq + (i_row & ((1 << g.q_dh_shift) - 1));
#pragma unroll
            for (int j = 0; j < CH; ++j)
              if (j0 + j < g.n)
                p[(long long)(j0 + j) * g.q_sn] = __float2bfloat16_rn(g.alpha * __uint_as_float(v[j]) * g.q_scale);
            return;
          }
        }
        if (g.c_sn == 1) {
          OutT* p = c + (long long)i_row * g.c_sm + j0;
          if (g.vec_ok && g.c_lo_off == 0 && j0 + CH <= g.n) {
            store_row32<OutT>(p, v, g.alpha, CH);
          } else {
#pragma unroll
            for (int j = 0; j < CH; ++j)
              if (j0 + j < g.n) put(p + j, finish<EXTRAS>(g, __uint_as_float(v[j]), i_row, j0 + j));
          }
        } else {
          OutT* p = c + (long long)i_row * g.c_sm;
#pragma unroll
          for (int j = 0; j < CH; ++j)
            if (j0 + j < g.n)
              put(p + (long long)(j0 + j) * g.c_sn, finish<EXTRAS>(g, __uint_as_float(v[j]), i_row, j0 + j));
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
      if (g.n_split == 1) {
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += CH) {
          uint32_t v[32];
          load_acc(c0, v);
          emit(v, c0);
        }
      } else {
        float* part = g.partial + (tile * g.n_split + split) * (long long)(BN * kBM);
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += CH) {
          uint32_t v[32];
          load_acc(c0, v);
#pragma unroll
          for (int j = 0; j < CH; ++j) part[(c0 + j) * kBM + row_local] = __uint_as_float(v[j]);
        }
        __threadfence();
        __syncwarp();
        int last = 0;
        if (lane == 0) {
          int* ticket = g.tickets + tile * 4 + q;
          last = atomicAdd(ticket, 1) == g.n_split - 1;
          if (last) *ticket = 0;               // every other split has already arrived
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
          __threadfence();
          // This warp sums its 32-row quarter over the splits, in split order.  Lane l owns
          // rows 4*(l%8)..+3 of column (l/8) in each group of four columns, so every load is
          // a 16-byte vector and a warp instruction covers 512 contiguous bytes; several
          // column groups and splits are in flight per thread to cover the L2 latency.
          const float* all = g.partial + tile * g.n_split * (long long)(BN * kBM) + q * 32;
          const int r4 = 4 * (lane & 7), cs = lane >> 3;
          constexpr int U = BN >= 16 ? 4 : 1;          // column groups per step (BN / 4 >= U)
#pragma unroll 1
          for (int jb = 0; jb < BN; jb += 4 * U) {
            float4 acc[U];
#pragma unroll
            for (int u = 0; u < U; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
            for (int sp0 = 0; sp0 < g.n_split; sp0 += 4) {
              float4 t[4][U];
#pragma unroll
              for (int s4 = 0; s4 < 4; ++s4)
#pragma unroll
                for (int u = 0; u < U; ++u)
                  t[s4][u] = sp0 + s4 < g.n_split
                                 ? __ldcg(reinterpret_cast<const float4*>(
                                       all + (long long)(sp0 + s4) * (BN * kBM) +
                                       (jb + u * 4 + cs) * kBM + r4))
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
              for (int s4 = 0; s4 < 4; ++s4)
#pragma unroll
                for (int u = 0; u < U; ++u) {
                  acc[u].x += t[s4][u].x; acc[u].y += t[s4][u].y;
                  acc[u].z += t[s4][u].z; acc[u].w += t[s4][u].w;
                }
            }
            const int i0 = mt * kBM + q * 32 + r4;
#pragma unroll
            for (int u = 0; u < U; ++u) {
              const int j = nt * BN + jb + u * 4 + cs;
              if (j >= g.n || i0 >= g.m) continue;
              const float sum[4] = {acc[u].x, acc[u].y, acc[u].z, acc[u].w};
              OutT* p = c + (long long)j * g.c_sn + (long long)i0 * g.c_sm;
              if (g.vec4_ok) {
                float val[4] = {g.alpha * sum[0], g.alpha * sum[1], g.alpha * sum[2], g.alpha * sum[3]};
                if constexpr (EXTRAS) {
                  // Four consecutive output features: bias and residual as 16-byte vectors too.
                  if (g.bias) {
                    const float4 b4 = *reinterpret_cast<const float4*>(g.bias + i0);
                    val[0] += b4.x; val[1] += b4.y; val[2] += b4.z; val[3] += b4.w;
                  }
                  if (g.relu) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) val[e] = fmaxf(val[e], 0.f);
                  }
                  if (g.residual) {
                    const float4 r4 = *reinterpret_cast<const float4*>(g.residual + i0 + (long long)j * g.r_sn);
                    val[0] += r4.x; val[1] += r4.y; val[2] += r4.z; val[3] += r4.w;
                  }
                }
                store4(p, val, g.c_lo_off);
              } else {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                  if (i0 + e < g.m) put(p + (long long)e * g.c_sm, finish<EXTRAS>(g, sum[e], i0 + e, j));
              }
            }
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
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

}  // namespace mtla
