// Kernels of the training path's backward pass (Section 4.2: the dense parallel form with the
// chunk-masked merge weights of Eq. 14-16 and the stride-aware causal mask), fp32 on the CUDA
// cores.  The forward pass is the parallel prefill, which computes exactly that form without
// materialising its T x T matrices; the backward pass reads what the prefill left in its
// workspace and does materialise the attention probabilities, one T x T matrix per (sequence,
// head), because every one of its products needs them twice.
#pragma once

#include <math.h>

#include "common.cuh"
#include "decode_kernels.cuh"

namespace mtla {

// C[z](i, j) = alpha * sum_k A[z](i, k) * B[z](k, j) + beta * C[z](i, j), every operand addressed
// through element strides, so one kernel serves the plain, the transposed-A (sums over rows,
// the weight gradients) and the transposed-B products of the backward pass.
struct GemmF32Args {
  const float* a;
  const float* b;
  float* c;
  int m, n, k;
  long long a_sm, a_sk, b_sk, b_sn, c_sm, c_sn;
  long long a_z, b_z, c_z;      // per-z element offsets
  int z_inner;                  // z = z_outer * z_inner + z_in: a second level of offsets
  long long a_z2, b_z2, c_z2;   //   applied to z_outer (e.g. sequence over head)
  float alpha, beta;
  int causal;                   // square products of the causal attention (row m sees columns n <= m):
                                // 1: output tiles wholly above the diagonal are skipped (their
                                //    consumers never read them); 2: A(i, k) is zero for k < i, the
                                //    reduction starts at the tile's first row; 3: A(i, k) is zero for
                                //    k > i, it ends after the tile's last row.  0: a full product.
  int c_vec;                    // 1: c_sn == 1 and every row start, z offset and n keep 16-byte alignment
                                // (the tiled kernel then stores four adjacent columns at once)
};

// 64 x 64 output tile per CTA of 256 threads, 16 reduction steps per stage, 4 x 4 outputs per
// thread.  Tile loads walk whichever index of the operand is contiguous, so they coalesce for
// both orientations.  The reduction runs in index order: results do not depend on the launch.
__global__ void __launch_bounds__(256) gemm_f32_kernel(GemmF32Args g) {
  __shared__ float as[16][64 + 4];
  __shared__ float bs[16][64 + 4];
  const int tid = threadIdx.x;
  const int z = blockIdx.z, zo = z / g.z_inner, zi = z % g.z_inner;
  const float* A = g.a + zi * g.a_z + zo * g.a_z2;
  const float* B = g.b + zi * g.b_z + zo * g.b_z2;
  float* C = g.c + zi * g.c_z + zo * g.c_z2;
  const int i0 = blockIdx.y * 64, j0 = blockIdx.x * 64;
  if (g.causal == 1 && j0 > i0 + 63) return;
  const int k_begin = g.causal == 2 ? i0 / 16 * 16 : 0;
  const int k_end = g.causal == 3 ? min(g.k, i0 + 64) : g.k;
  const int ti = (tid / 16) * 4, tj = (tid % 16) * 4;
  float acc[4][4];
#pragma unroll
  for (int x = 0; x < 4; ++x)
#pragma unroll
    for (int y = 0; y < 4; ++y) acc[x][y] = 0.f;
  const bool a_k_fast = g.a_sk == 1, b_n_fast = g.b_sn == 1;
  for (int k0 = k_begin; k0 < k_end; k0 += 16) {
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int idx = tid + t * 256;
      const int kk = a_k_fast ? idx % 16 : idx / 64, ii = a_k_fast ? idx / 16 : idx % 64;
      const int gi = i0 + ii, gk = k0 + kk;
      as[kk][ii] = (gi < g.m && gk < k_end) ? A[gi * g.a_sm + gk * g.a_sk] : 0.f;
      const int jj = b_n_fast ? idx % 64 : idx / 16, kb = b_n_fast ? idx / 64 : idx % 16;
      const int gj = j0 + jj, gkb = k0 + kb;
      bs[kb][jj] = (gj < g.n && gkb < k_end) ? B[gkb * g.b_sk + gj * g.b_sn] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      const float4 av = *reinterpret_cast<const float4*>(&as[kk][ti]);
      const float4 bv = *reinterpret_cast<const float4*>(&bs[kk][tj]);
      const float a4[4] = {av.x, av.y, av.z, av.w}, b4[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(a4[x], b4[y], acc[x][y]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int x = 0; x < 4; ++x)
#pragma unroll
    for (int y = 0; y < 4; ++y) {
      const int gi = i0 + ti + x, gj = j0 + tj + y;
      if (gi >= g.m || gj >= g.n) continue;
      float* p = C + gi * g.c_sm + gj * g.c_sn;
      *p = g.alpha * acc[x][y] + (g.beta != 0.f ? g.beta * *p : 0.f);
    }
}

// The same product on (16 TM) x (16 TN) output tiles, TM x TN outputs per thread (as two groups of
// TM / 2 rows and TN / 2 columns, 16 TM / 2 and 16 TN / 2 apart, so that shared-memory reads are
// 16-byte vectors without bank conflicts), the next 16 reduction steps fetched into registers
// while the current ones are multiplied.  One accumulator per output, reduction in index order:
// the same sums as gemm_f32_kernel.  For products with at least 16 TM rows and 16 TN columns.
template <int TM, int TN>
__global__ void __launch_bounds__(256) gemm_f32_tiled_kernel(GemmF32Args g) {
  constexpr int BM = 16 * TM, BN = 16 * TN, BK = 16, HM = TM / 2, HN = TN / 2;
  static_assert(HM == 2 || HM == 4, "row groups are float2 / float4 reads");
  static_assert(HN == 2 || HN == 4, "column groups are float2 / float4 reads");
  __shared__ __align__(16) float as[2][BK][BM + 4];
  __shared__ __align__(16) float bs[2][BK][BN + 4];
  const int tid = threadIdx.x;
  const int z = blockIdx.z, zo = z / g.z_inner, zi = z % g.z_inner;
  const float* A = g.a + zi * g.a_z + zo * g.a_z2;
  const float* B = g.b + zi * g.b_z + zo * g.b_z2;
  float* C = g.c + zi * g.c_z + zo * g.c_z2;
  const int i0 = blockIdx.y * BM, j0 = blockIdx.x * BN;
  if (g.causal == 1 && j0 > i0 + BM - 1) return;
  const int k_begin = g.causal == 2 ? i0 / BK * BK : 0;
  const int k_end = g.causal == 3 ? min(g.k, i0 + BM) : g.k;
  const int ty = tid / 16, tx = tid % 16;
  const bool a_k_fast = g.a_sk == 1, b_n_fast = g.b_sn == 1;
  float acc[TM][TN];
#pragma unroll
  for (int x = 0; x < TM; ++x)
#pragma unroll
    for (int y = 0; y < TN; ++y) acc[x][y] = 0.f;
  float ra[TM], rb[TN];
  // Tile element e of this thread: (k, i) for A, (k, j) for B, walking the contiguous index.
  auto fetch = [&](int k0) {
#pragma unroll
    for (int e = 0; e < TM; ++e) {
      const int idx = tid + e * 256;
      const int kk = a_k_fast ? idx % BK : idx / BM, ii = a_k_fast ? idx / BK : idx % BM;
      const int gi = i0 + ii, gk = k0 + kk;
      ra[e] = (gi < g.m && gk < k_end) ? A[gi * g.a_sm + gk * g.a_sk] : 0.f;
    }
#pragma unroll
    for (int e = 0; e < TN; ++e) {
      const int idx = tid + e * 256;
      const int jj = b_n_fast ? idx % BN : idx / BK, kk = b_n_fast ? idx / BN : idx % BK;
      const int gj = j0 + jj, gk = k0 + kk;
      rb[e] = (gj < g.n && gk < k_end) ? B[gk * g.b_sk + gj * g.b_sn] : 0.f;
    }
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int e = 0; e < TM; ++e) {
      const int idx = tid + e * 256;
      const int kk = a_k_fast ? idx % BK : idx / BM, ii = a_k_fast ? idx / BK : idx % BM;
      as[buf][kk][ii] = ra[e];
    }
#pragma unroll
    for (int e = 0; e < TN; ++e) {
      const int idx = tid + e * 256;
      const int jj = b_n_fast ? idx % BN : idx / BK, kk = b_n_fast ? idx / BN : idx % BK;
      bs[buf][kk][jj] = rb[e];
    }
  };
  fetch(k_begin);
  stash(0);
  __syncthreads();
  int buf = 0;
  for (int k0 = k_begin; k0 < k_end; k0 += BK) {
    const bool more = k0 + BK < k_end;
    if (more) fetch(k0 + BK);
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a8[TM], b8[TN];
#pragma unroll
      for (int hlf = 0; hlf < 2; ++hlf) {
#pragma unroll
        for (int x = 0; x < HM; ++x) a8[hlf * HM + x] = as[buf][kk][hlf * (BM / 2) + ty * HM + x];
#pragma unroll
        for (int y = 0; y < HN; ++y) b8[hlf * HN + y] = bs[buf][kk][hlf * (BN / 2) + tx * HN + y];
      }
#pragma unroll
      for (int x = 0; x < TM; ++x)
#pragma unroll
        for (int y = 0; y < TN; ++y) acc[x][y] = fmaf(a8[x], b8[y], acc[x][y]);
    }
    if (more) {
      stash(buf ^ 1);       // the other buffer was last read before the previous barrier
      __syncthreads();
      buf ^= 1;
    }
  }
#pragma unroll
  for (int x = 0; x < TM; ++x) {
    const int gi = i0 + (x / HM) * (BM / 2) + ty * HM + x % HM;
    if (gi >= g.m) continue;
    if (HN == 4 && g.c_vec) {
      // The thread's columns come in runs of four adjacent ones: one 16-byte access each.
#pragma unroll
      for (int yh = 0; yh < 2; ++yh) {
        const int gj = j0 + yh * (BN / 2) + tx * HN;
        if (gj >= g.n) continue;                       // n is a multiple of 4: whole runs only
        float4* p = reinterpret_cast<float4*>(C + gi * g.c_sm + gj);
        float4 v = make_float4(g.alpha * acc[x][yh * HN], g.alpha * acc[x][yh * HN + 1],
                               g.alpha * acc[x][yh * HN + 2], g.alpha * acc[x][yh * HN + 3]);
        if (g.beta != 0.f) {
          const float4 o = *p;
          v.x += g.beta * o.x; v.y += g.beta * o.y; v.z += g.beta * o.z; v.w += g.beta * o.w;
        }
        *p = v;
      }
      continue;
    }
#pragma unroll
    for (int y = 0; y < TN; ++y) {
      const int gj = j0 + (y / HN) * (BN / 2) + tx * HN + y % HN;
      if (gj >= g.n) continue;
      float* p = C + gi * g.c_sm + gj * g.c_sn;
      *p = g.alpha * acc[x][y] + (g.beta != 0.f ? g.beta * *p : 0.f);
    }
  }
}

// Row m of a score matrix S [T][T] (log2 units, one matrix per blockIdx.y): softmax under the
// stride-aware causal mask of Section 4.2 (column n allowed iff n == m, or n < m and
// (n + 1) mod s == 0 for 0-based m, n), in place.  One warp per row, 8 rows per CTA.
__global__ void __launch_bounds__(256) masked_softmax_kernel(float* s, int T, int stride) {
  const int lane = threadIdx.x & 31;
  const int m = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (m >= T) return;
  float* row = s + ((long long)blockIdx.y * T + m) * T;
  auto allowed = [&](int n) { return n == m || (n < m && (n + 1) % stride == 0); };
  float mx = -INFINITY;
  for (int n = lane; n <= m; n += 32)
    if (allowed(n)) mx = fmaxf(mx, row[n]);
  mx = warp_max(mx);
  float sum = 0.f;
  for (int n = lane; n < T; n += 32) {
    const float p = allowed(n) ? exp2f(row[n] - mx) : 0.f;
    row[n] = p;
    sum += p;
  }
  const float inv = 1.f / warp_sum(sum);
  for (int n = lane; n <= m; n += 32) row[n] *= inv;
}

// Backward of that softmax, in place on dP: dS = P o (dP - sum_n dP o P) * scale, where scale is
// 1 / sqrt(d_h), the derivative of the score's own scaling.
__global__ void __launch_bounds__(256) softmax_backward_kernel(const float* p, float* dp, int T,
                                                               float scale) {
  const int lane = threadIdx.x & 31;
  const int m = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (m >= T) return;
  const long long off = ((long long)blockIdx.y * T + m) * T;
  const float* prow = p + off;
  float* drow = dp + off;
  float dot = 0.f;
  for (int n = lane; n <= m; n += 32) dot += prow[n] * drow[n];
  dot = warp_sum(dot);
  for (int n = lane; n < T; n += 32) drow[n] = n <= m ? prow[n] * (drow[n] - dot) * scale : 0.f;
}

struct GateLnBackwardArgs {
  const float* p1;        // [rows][proj.width] forward projections (c_raw at proj.off_c)
  ProjLayout proj;
  const float* gamma;
  const float* beta;
  const float* hyp_c_w;   // [r][d_w]
  const float* hyp_c_wt;  // [d_w][r]: the same matrix transposed, so that the reverse product's reads
                          // (one thread per latent column) coalesce as the forward product's do
  const float* hyp_c_b;   // [d_w]
  const float* gate_pe;   // [max_slots][d_w]: Linear(pe_j) per chunk
  const float* dcprime;   // [rows][r] gradient of the running merge states (Eq. 14's sequence)
  float* dp1;             // [rows][proj.width]: receives the gradient of c_raw at proj.off_c
  float* c;               // [rows][r] normalised latents (for the hyper-network's weight gradient)
  float* xhat;            // [rows][r] normalised latents before gain and bias
  float* dc;              // [rows][r] gradient of the normalised latents
  float* dh;              // [rows][d_w] gradient of Linear(c)
  float* dg;              // [B * chunks][d_w] gradient of Linear(pe_j)
  int r, dw, stride, T, use_gate;
  float ln_eps;
};

// One CTA of 256 threads per (chunk, sequence): the reverse of the chunk's running merge, its
// gates (Eq. 13 / 16) and the LayerNorm of its <= s tokens.  Tokens are revisited from the last
// to the first, carrying the suffix sum of the states' gradients.
__global__ void __launch_bounds__(256) gate_ln_backward_kernel(GateLnBackwardArgs a) {
  __shared__ float c_s[512], xh_s[512], suf_s[512], dc_s[512];
  __shared__ float h_s[256], dh_s[256], dg_s[256];
  __shared__ float red_s[33];
  const int chunk = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
  const int tok0 = chunk * a.stride, tok1 = min(a.T, tok0 + a.stride);
  const int chunks = gridDim.x;
  const float* g = a.gate_pe + (long long)chunk * a.dw;
  for (int i = tid; i < a.r; i += 256) suf_s[i] = 0.f;
  for (int n = tid; n < a.dw; n += 256) dg_s[n] = 0.f;
  for (int tok = tok1 - 1; tok >= tok0; --tok) {
    const long long rowi = (long long)b * a.T + tok;
    const float* row = a.p1 + rowi * a.proj.width + a.proj.off_c;
    __syncthreads();
    // Forward values of this token again: LayerNorm, Linear(c), gate.
    float s = 0.f;
    for (int i = tid; i < a.r; i += 256) {
      c_s[i] = row[i];
      s += row[i];
    }
    const float mean = block_sum(s, red_s) / a.r;
    float sq = 0.f;
    for (int i = tid; i < a.r; i += 256) {
      const float d = c_s[i] - mean;
      sq += d * d;
    }
    __syncthreads();
    const float rstd = rsqrtf(block_sum(sq, red_s) / a.r + a.ln_eps);
    for (int i = tid; i < a.r; i += 256) {
      const float xh = (c_s[i] - mean) * rstd;
      xh_s[i] = xh;
      c_s[i] = xh * a.gamma[i] + a.beta[i];
      suf_s[i] += a.dcprime[rowi * a.r + i];        // every later state of the chunk holds w c
    }
    __syncthreads();
    float w = 1.f, dz = 0.f;
    if (a.use_gate) {
      // Linear(c): the r rows of A are cut into 256 / d_w ranges so that every thread works;
      // the ranges' sums are added in range order (part_s aliases dc_s, written only later).
      float prod = 0.f;
      const int parts = a.dw <= 128 ? 256 / a.dw : 1;
      if (parts > 1) {
        float* part_s = dc_s;                      // parts * d_w <= 256 floats
        const int n = tid % a.dw, pt = tid / a.dw;
        if (pt < parts) {
          const int per = (a.r + parts - 1) / parts, lo = pt * per, hi = min(a.r, lo + per);
          float hn = 0.f;
          for (int i = lo; i < hi; ++i) hn = fmaf(c_s[i], a.hyp_c_w[(long long)i * a.dw + n], hn);
          part_s[pt * a.dw + n] = hn;
        }
        __syncthreads();
        if (tid < a.dw) {
          float hn = a.hyp_c_b[tid];
          for (int pt2 = 0; pt2 < parts; ++pt2) hn += part_s[pt2 * a.dw + tid];
          h_s[tid] = hn;
          prod = hn * g[tid];
        }
      } else {
        for (int n = tid; n < a.dw; n += 256) {
          float hn = a.hyp_c_b[n];
          for (int i = 0; i < a.r; ++i) hn = fmaf(c_s[i], a.hyp_c_w[(long long)i * a.dw + n], hn);
          h_s[n] = hn;
          prod += hn * g[n];
        }
      }
      const float logit = block_sum(prod, red_s);
      w = 1.f / (1.f + expf(-logit));
      float dwp = 0.f;
      for (int i = tid; i < a.r; i += 256) dwp += suf_s[i] * c_s[i];
      const float dw_tok = block_sum(dwp, red_s);
      dz = dw_tok * w * (1.f - w);
      for (int n = tid; n < a.dw; n += 256) {
        dh_s[n] = dz * g[n];
        dg_s[n] += dz * h_s[n];
        a.dh[rowi * a.dw + n] = dh_s[n];
      }
      __syncthreads();
    }
    // dL/dc = w * suffix (+ the hyper-network's path), then the LayerNorm's reverse.
    float p1s = 0.f, p2s = 0.f;
    for (int i = tid; i < a.r; i += 256) {
      float d = w * suf_s[i];
      if (a.use_gate) {
        float t = 0.f;
        for (int n = 0; n < a.dw; ++n) t = fmaf(dh_s[n], a.hyp_c_wt[(long long)n * a.r + i], t);
        d += t;
      }
      dc_s[i] = d;
      const float dxh = d * a.gamma[i];
      p1s += dxh;
      p2s += dxh * xh_s[i];
    }
    const float m1 = block_sum(p1s, red_s) / a.r;
    __syncthreads();
    const float m2 = block_sum(p2s, red_s) / a.r;
    for (int i = tid; i < a.r; i += 256) {
      const float dxh = dc_s[i] * a.gamma[i];
      a.dp1[rowi * a.proj.width + a.proj.off_c + i] = (dxh - m1 - xh_s[i] * m2) * rstd;
      a.c[rowi * a.r + i] = c_s[i];
      a.xhat[rowi * a.r + i] = xh_s[i];
      a.dc[rowi * a.r + i] = dc_s[i];
    }
  }
  __syncthreads();
  if (a.use_gate)
    for (int n = tid; n < a.dw; n += 256) a.dg[((long long)b * chunks + chunk) * a.dw + n] = dg_s[n];
}

// out[j] = sum_i a[i][j] * (b ? b[i][j] : 1) over `rows` rows of width n: LayerNorm gain / bias
// and Linear bias gradients.  A CTA of 32 x 32 threads owns 32 columns: thread (x, y) adds rows
// y, y + 32, ... of column x in order, then thread (x, 0) adds the 32 partial sums in order, so
// the result does not depend on the launch.
__global__ void __launch_bounds__(1024) column_sum_kernel(const float* a, const float* b, float* out,
                                                          long long rows, int n, long long ld) {
  __shared__ float part[32][33];
  const int x = threadIdx.x, y = threadIdx.y;
  const int j = blockIdx.x * 32 + x;
  float s = 0.f;
  if (j < n)
    for (long long i = y; i < rows; i += 32) s += a[i * ld + j] * (b ? b[i * ld + j] : 1.f);
  part[y][x] = s;
  __syncthreads();
  if (y == 0 && j < n) {
    float total = 0.f;
#pragma unroll
    for (int k = 0; k < 32; ++k) total += part[k][x];
    out[j] = total;
  }
}

// out(i, j) = alpha * sum_s part[s][i * n + j] + beta * out(i, j), the partial products of a
// reduction that was split over `splits` launches' worth of CTAs, added in split order.
__global__ void __launch_bounds__(256) sum_splits_kernel(const float* part, int splits, long long count,
                                                         int n, float* out, long long c_sm, long long c_sn,
                                                         float alpha, float beta) {
  const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
  if (idx >= count) return;
  float s = 0.f;
  for (int k = 0; k < splits; ++k) s += part[k * count + idx];
  float* p = out + (idx / n) * c_sm + (idx % n) * c_sn;
  *p = alpha * s + (beta != 0.f ? beta * *p : 0.f);
}

// Sinusoidal positional embedding rows pe_{j+1} (dimension r) for chunk j of every sequence:
// out [B * chunks][r]; the input of Linear(pe_j) in Eq. 13 / Eq. 15.
__global__ void pe_rows_kernel(float* out, int chunks, int r, long long total) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int i = (int)(idx % r);
  const int j = (int)((idx / r) % chunks);
  const double angle = (double)(j + 1) / pow(10000.0, 2.0 * (double)(i / 2) / (double)r);
  out[idx] = (float)((i & 1) ? cos(angle) : sin(angle));
}

// Gradients of the query block back to the un-rotated projections: reads dqcat
// [rows][n_h][d_h + d_R] (gradient of the query | of the rotated RoPE query, both un-scaled) and
// dkr [rows][d_R] (gradient of the rotated RoPE key), writes dp1's q, q^R and k^R columns.
// A rotation's reverse is the rotation by the negative angle.
struct RopeBackwardArgs {
  const float* dqcat;
  const float* dkr;
  float* dp1;
  ProjLayout proj;
  const float* rope_cos;
  const float* rope_sin;
  int n_heads, head_dim, dr, T;
};
__global__ void __launch_bounds__(256) rope_backward_kernel(RopeBackwardArgs a) {
  const long long rowi = blockIdx.x;
  const int tok = (int)(rowi % a.T), tid = threadIdx.x, half = a.dr / 2, DQ = a.head_dim + a.dr;
  const float* cs = a.rope_cos + (long long)tok * half;
  const float* sn = a.rope_sin + (long long)tok * half;
  const float* dq = a.dqcat + rowi * a.n_heads * DQ;
  float* out = a.dp1 + rowi * a.proj.width;
  for (int i = tid; i < a.n_heads * a.head_dim; i += 256) {
    const int h = i / a.head_dim, e = i % a.head_dim;
    out[a.proj.off_q + i] = dq[h * DQ + e];
  }
  for (int i = tid; i < a.n_heads * half; i += 256) {
    const int h = i / half, k = i % half;
    const float g0 = dq[h * DQ + a.head_dim + 2 * k];
    const float g1 = dq[h * DQ + a.head_dim + 2 * k + 1];
    out[a.proj.off_qr + h * a.dr + 2 * k] = g0 * cs[k] + g1 * sn[k];
    out[a.proj.off_qr + h * a.dr + 2 * k + 1] = -g0 * sn[k] + g1 * cs[k];
  }
  for (int k = tid; k < half; k += 256) {
    const float g0 = a.dkr[rowi * a.dr + 2 * k], g1 = a.dkr[rowi * a.dr + 2 * k + 1];
    out[a.proj.off_kr + 2 * k] = g0 * cs[k] + g1 * sn[k];
    out[a.proj.off_kr + 2 * k + 1] = -g0 * sn[k] + g1 * cs[k];
  }
}

}  // namespace mtla
