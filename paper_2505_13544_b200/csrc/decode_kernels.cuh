// Decode-step kernels that are not GEMMs: the fused LayerNorm / hyper-network gate / slot
// update / RoPE kernel, the CUDA-core split-K attention over the compressed cache, and the
// cross-split combine.
#pragma once

#include <math.h>

#include "common.cuh"

namespace mtla {

// Column offsets of the fused input projection output row: [ q | q^R | c_raw | k^R | u_hi | u_lo ].
// The last two blocks (d_w columns each, off_u < 0 when absent) are the hyper-network's
// Linear(c_i) of Eq. 13 folded through the LayerNorm into the projection:
//   c A + a = rstd * (c_raw (gamma .* A) - mean * (gamma^T A)) + (beta^T A + a),
// and c_raw (gamma .* A) = x (W_r diag(gamma) A) = u, one more block of the fused product
// (its weights kept as bf16 hi + lo halves, so u carries fp32-like precision).
struct ProjLayout {
  int off_q, off_qr, off_c, off_kr, off_u, width;
};

struct PostArgs {
  const float* p1;        // [B][proj.width] fused projection of this step's tokens (fp32)
  ProjLayout proj;
  int absorbed;           // 1: the query block of p1 is the absorbed, pre-scaled query (layers that keep
                          // W_Q W_K^T pre-multiplied): n_h r columns from the weight's bf16 hi half,
                          // then n_h r from its lo half; their sum goes to qt
  const float* gamma;     // [r]
  const float* beta;      // [r]
  const float* hyp_c_w;   // [r][d_w] fp32
  const float* hyp_c_b;   // [d_w]
  const float* gate_pe;   // [max_slots][d_w]: row j0 is Linear(pe_{j0+1}) of Eq. 13
  const float* gate_s;    // [d_w]: gamma^T A        (folded gate only)
  const float* gate_t;    // [d_w]: beta^T A + a     (folded gate only)
  const float* rope_cos;  // [max_tokens][d_R/2]
  const float* rope_sin;  // [max_tokens][d_R/2]
  float* open_acc;        // [B][r] fp32 running sum of the open slot
  CacheView cache;
  int* seq_tokens;        // [B] tokens each sequence has consumed, advanced by this kernel; or
                          // nullptr when all sequences stand at `tokens`
  void* qt;               // [B][n_h][r + d_R] absorbed query; this kernel writes the RoPE tail
  bf16* q16;              // [B][2*n_h*d_h]: q as bf16 [hi | lo] halves (q = hi + lo) for the
                          // tensor-core absorption, or nullptr
  int n_heads, head_dim, r, dr, dw;
  int tokens;             // tokens consumed so far = 0-based index of this token (lock-step batch)
  int stride;             // s: slot tokens / s receives the token, opened when tokens mod s == 0
  int use_gate;           // 0 at s == 1 (w = 1)
  float ln_eps;
  float q_scale;          // log2(e) / sqrt(d_h), folded into the absorbed query
};

// Merge weight of Eq. 13 for one token, by a CTA of 256 threads: h = c A + a over the d_w
// hyper-network outputs, then sigmoid(<h, g>) with g = Linear(pe_j) from the table.  `c` is the
// normalised latent in shared memory; `part` holds 512 floats, `red` 33.  A [r][d_w] is read
// once per CTA: each thread owns two adjacent outputs and a slice of the r rows, with sixteen
// independent 8-byte loads in flight to cover the L2 latency (d_w even; a scalar loop otherwise).
// Every thread receives the weight.  Contains __syncthreads().
__device__ inline float gate_weight(const float* c, const float* hyp_w, const float* hyp_b,
                                    const float* gate_pe, int r, int dw, float* part, float* red) {
  const int tid = threadIdx.x;
  float prod = 0.f;
  if ((dw & 1) == 0) {
    const int pairs = dw >> 1, parts = 256 / pairs;      // pairs <= 128, so parts >= 2
    float h0 = 0.f, h1 = 0.f;
    if (tid < parts * pairs) {
      const int n2 = tid % pairs, part_i = tid / pairs;
      const int per = ceil_div(r, parts);
      const int lo = part_i * per, hi = min(r, lo + per);
      const float2* wp = reinterpret_cast<const float2*>(hyp_w) + n2;
#pragma unroll 16
      for (int i = lo; i < hi; ++i) {
        const float2 wv = __ldg(wp + (long long)i * pairs);
        h0 = fmaf(c[i], wv.x, h0);
        h1 = fmaf(c[i], wv.y, h1);
      }
    }
    part[2 * tid] = h0;
    part[2 * tid + 1] = h1;
    __syncthreads();
    if (tid < dw) {
      float hn = hyp_b[tid];
      for (int p = 0; p < parts; ++p) hn += part[2 * (p * pairs + (tid >> 1)) + (tid & 1)];
      prod = hn * gate_pe[tid];
    }
  } else {
    const int parts = 256 / dw > 0 ? 256 / dw : 1;
    float h = 0.f;
    if (tid < parts * dw) {
      const int n = tid % dw, part_i = tid / dw;
      const int per = ceil_div(r, parts);
      const int lo = part_i * per, hi = min(r, lo + per);
      for (int i = lo; i < hi; ++i) h = fmaf(c[i], hyp_w[(long long)i * dw + n], h);
    }
    part[tid] = h;
    __syncthreads();
    if (tid < dw) {
      float hn = hyp_b[tid];
      for (int p = 0; p < parts; ++p) hn += part[p * dw + tid];
      prod = hn * gate_pe[tid];
    }
  }
  const float logit = block_sum(prod, red);
  return 1.f / (1.f + expf(-logit));
}

// The same weight from the folded projection block u (see ProjLayout): no matrix is read.
__device__ inline float gate_weight_folded(const float* u, int dw, float mean, float rstd,
                                           const float* gate_s, const float* gate_t,
                                           const float* gate_pe, float* red) {
  const int tid = threadIdx.x;
  float prod = 0.f;
  if (tid < dw) {
    const float h = rstd * (u[tid] + u[dw + tid] - mean * gate_s[tid]) + gate_t[tid];
    prod = h * gate_pe[tid];
  }
  const float logit = block_sum(prod, red);
  return 1.f / (1.f + expf(-logit));
}

// One CTA of 256 threads per sequence.  Section 4.1: c_i = LayerNorm(x_i W_r); Eq. 13 gate;
// slot update (open: c_hat_j = w c, else c_hat_j += w c); Section 4.3: RoPE key replaces
// the slot's key, RoPE queries are rotated and written behind the absorbed query.
// T is the cache element type, TQ the element type of the absorbed-query buffer.
template <typename T, typename TQ>
__global__ void __launch_bounds__(256) decode_post_kernel(PostArgs a) {
  __shared__ float c_s[512];
  __shared__ float part_s[512];
  __shared__ float red_s[33];
  const int b = blockIdx.x, tid = threadIdx.x;
  const float* row = a.p1 + (long long)b * a.proj.width;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();   // the projection kernel's output is read from here on
  const int i0 = a.seq_tokens ? a.seq_tokens[b] : a.tokens;
  const int slot = i0 / a.stride;
  const bool new_slot = i0 % a.stride == 0;
  const float* gate_pe = a.gate_pe + (long long)slot * a.dw;
  const float* rope_cos = a.rope_cos + (long long)i0 * (a.dr / 2);
  const float* rope_sin = a.rope_sin + (long long)i0 * (a.dr / 2);

  // LayerNorm over r (two-pass variance).
  float s = 0.f;
  for (int i = tid; i < a.r; i += 256) {
    const float v = row[a.proj.off_c + i];
    c_s[i] = v;
    s += v;
  }
  const float mean = block_sum(s, red_s) / a.r;
  float sq = 0.f;
  for (int i = tid; i < a.r; i += 256) {
    const float dlt = c_s[i] - mean;
    sq += dlt * dlt;
  }
  __syncthreads();
  const float rstd = rsqrtf(block_sum(sq, red_s) / a.r + a.ln_eps);
  for (int i = tid; i < a.r; i += 256) c_s[i] = (c_s[i] - mean) * rstd * a.gamma[i] + a.beta[i];
  __syncthreads();

  // Hyper-network gate: w = sigmoid(<c A + a, Linear(pe_j)>).
  float w = 1.f;
  if (a.use_gate)
    w = a.proj.off_u >= 0
            ? gate_weight_folded(row + a.proj.off_u, a.dw, mean, rstd, a.gate_s, a.gate_t, gate_pe, red_s)
            : gate_weight(c_s, a.hyp_c_w, a.hyp_c_b, gate_pe, a.r, a.dw, part_s, red_s);

  // Slot update: fp32 running sum, stored to the cache in the storage type.
  const int W = a.r + a.dr;
  T* slot_row = static_cast<T*>(a.cache.base) + cache_row(a.cache, b, slot) * W;
  float* acc = a.open_acc + (long long)b * a.r;
  for (int i = tid; i < a.r; i += 256) {
    const float v = (new_slot ? 0.f : acc[i]) + w * c_s[i];
    acc[i] = v;
    slot_row[i] = Elem<T>::from_float(v);
  }
  // RoPE key of this token replaces the slot's key.
  for (int k = tid; k < a.dr / 2; k += 256) {
    const float x0 = row[a.proj.off_kr + 2 * k], x1 = row[a.proj.off_kr + 2 * k + 1];
    const float cs = rope_cos[k], sn = rope_sin[k];
    slot_row[a.r + 2 * k] = Elem<T>::from_float(x0 * cs - x1 * sn);
    slot_row[a.r + 2 * k + 1] = Elem<T>::from_float(x0 * sn + x1 * cs);
  }
  if (a.q16) {
    const int hd = a.n_heads * a.head_dim;
    for (int i = tid * 2; i < hd; i += 512) {
      const float q0 = row[a.proj.off_q + i], q1 = row[a.proj.off_q + i + 1];
      const __nv_bfloat162 hi = __floats2bfloat162_rn(q0, q1);
      bf16* dst = a.q16 + (long long)b * 2 * hd + i;
      *reinterpret_cast<__nv_bfloat162*>(dst) = hi;
      *reinterpret_cast<__nv_bfloat162*>(dst + hd) =
          __floats2bfloat162_rn(q0 - __low2float(hi), q1 - __high2float(hi));
    }
  }
  // Rotated, pre-scaled RoPE queries behind the (separately computed) absorbed query.
  TQ* qt = static_cast<TQ*>(a.qt) + (long long)b * a.n_heads * W;
  const int half = a.dr / 2;
  for (int i = tid; i < a.n_heads * half; i += 256) {
    const int h = i / half, k = i % half;
    const float x0 = row[a.proj.off_qr + h * a.dr + 2 * k];
    const float x1 = row[a.proj.off_qr + h * a.dr + 2 * k + 1];
    const float cs = rope_cos[k], sn = rope_sin[k];
    qt[h * W + a.r + 2 * k] = Elem<TQ>::from_float((x0 * cs - x1 * sn) * a.q_scale);
    qt[h * W + a.r + 2 * k + 1] = Elem<TQ>::from_float((x0 * sn + x1 * cs) * a.q_scale);
  }
  // Every thread read the position before the first block-wide reduction above.
  if (a.seq_tokens && tid == 0) a.seq_tokens[b] = i0 + 1;
}

// The same step for layers whose gate needs no matrix (the folded form, or s = 1 where w = 1),
// laid out for latency: warp 0 alone carries the dependent chain of a sequence (latent row ->
// LayerNorm by shuffles -> gate -> slot row), everything it touches moving as 16-byte vectors,
// while warps 1-7 convert the queries (bf16 hi / lo halves for the tensor-core absorption) and
// rotate the RoPE queries, which depend on nothing but the projection row.  No block-wide
// barrier is needed.  One CTA of 256 threads per sequence; r <= 512.
template <typename T, typename TQ>
__global__ void __launch_bounds__(256) decode_post_fast_kernel(PostArgs a) {
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* row = a.p1 + (long long)b * a.proj.width;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();   // the projection kernel's output is read from here on
  const int i0 = a.seq_tokens ? a.seq_tokens[b] : a.tokens;
  const int slot = i0 / a.stride;
  const bool new_slot = i0 % a.stride == 0;
  const int half = a.dr / 2, W = a.r + a.dr;
  const float* rope_cos = a.rope_cos + (long long)i0 * half;
  const float* rope_sin = a.rope_sin + (long long)i0 * half;
  if (warp == 0) {
    // Latent: lane l holds elements 128 v + 4 l .. + 3 of the row, v < ceil(r / 128).
    float c[4][4];
    float sum = 0.f;
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const int i = v * 128 + lane * 4;
      const float4 x4 = i < a.r ? *reinterpret_cast<const float4*>(row + a.proj.off_c + i)
                                : make_float4(0.f, 0.f, 0.f, 0.f);
      c[v][0] = x4.x; c[v][1] = x4.y; c[v][2] = x4.z; c[v][3] = x4.w;
      sum += (x4.x + x4.y) + (x4.z + x4.w);
    }
    // The other inputs of the chain are requested before the first reduction.
    float uu[8], gss[8], gtt[8], gpp[8];
    const float* gate_pe = a.gate_pe + (long long)slot * a.dw;
    if (a.use_gate) {
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int n = k * 32 + lane;
        const bool in = n < a.dw;
        uu[k] = in ? row[a.proj.off_u + n] + row[a.proj.off_u + a.dw + n] : 0.f;
        gss[k] = in ? a.gate_s[n] : 0.f;
        gtt[k] = in ? a.gate_t[n] : 0.f;
        gpp[k] = in ? gate_pe[n] : 0.f;
      }
    }
    float acc_old[4][4];
    float* acc = a.open_acc + (long long)b * a.r;
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const int i = v * 128 + lane * 4;
      const float4 o4 = (!new_slot && i < a.r) ? *reinterpret_cast<const float4*>(acc + i)
                                               : make_float4(0.f, 0.f, 0.f, 0.f);
      acc_old[v][0] = o4.x; acc_old[v][1] = o4.y; acc_old[v][2] = o4.z; acc_old[v][3] = o4.w;
    }
    const float mean = warp_sum(sum) / a.r;
    float sq = 0.f;
#pragma unroll
    for (int v = 0; v < 4; ++v)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float d = (v * 128 + lane * 4 + e < a.r) ? c[v][e] - mean : 0.f;
        sq += d * d;
      }
    const float rstd = rsqrtf(warp_sum(sq) / a.r + a.ln_eps);
    float w = 1.f;
    if (a.use_gate) {
      float prod = 0.f;
#pragma unroll
      for (int k = 0; k < 8; ++k) prod += (rstd * (uu[k] - mean * gss[k]) + gtt[k]) * gpp[k];
      w = 1.f / (1.f + expf(-warp_sum(prod)));
    }
    T* slot_row = static_cast<T*>(a.cache.base) + cache_row(a.cache, b, slot) * W;
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const int i = v * 128 + lane * 4;
      if (i >= a.r) continue;
      const float4 g4 = *reinterpret_cast<const float4*>(a.gamma + i);
      const float4 b4 = *reinterpret_cast<const float4*>(a.beta + i);
      const float gam[4] = {g4.x, g4.y, g4.z, g4.w}, bet[4] = {b4.x, b4.y, b4.z, b4.w};
      float val[4];
#pragma unroll
      for (int e = 0; e < 4; ++e)
        val[e] = acc_old[v][e] + w * ((c[v][e] - mean) * rstd * gam[e] + bet[e]);
      *reinterpret_cast<float4*>(acc + i) = make_float4(val[0], val[1], val[2], val[3]);
      if (sizeof(T) == 2) {
        const __nv_bfloat162 h0 = __floats2bfloat162_rn(val[0], val[1]), h1 = __floats2bfloat162_rn(val[2], val[3]);
        *reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(slot_row) + i) =
            make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
      } else {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(slot_row) + i) =
            make_float4(val[0], val[1], val[2], val[3]);
      }
    }
    // RoPE key of this token replaces the slot's key (pairs 2k, 2k + 1; d_R / 2 <= 32 pairs).
    if (lane < half) {
      const float2 x2 = *reinterpret_cast<const float2*>(row + a.proj.off_kr + 2 * lane);
      const float cs = rope_cos[lane], sn = rope_sin[lane];
      const float y0 = x2.x * cs - x2.y * sn, y1 = x2.x * sn + x2.y * cs;
      if (sizeof(T) == 2)
        *reinterpret_cast<__nv_bfloat162*>(reinterpret_cast<bf16*>(slot_row) + a.r + 2 * lane) =
            __floats2bfloat162_rn(y0, y1);
      else
        *reinterpret_cast<float2*>(reinterpret_cast<float*>(slot_row) + a.r + 2 * lane) = make_float2(y0, y1);
    }
    if (a.seq_tokens && lane == 0) a.seq_tokens[b] = i0 + 1;
    return;
  }
  // Warps 1-7: queries.  bf16 [hi | lo] halves of q, four elements per thread and step.
  const int t = tid - 32;
  if (a.absorbed) {
    // The projection already holds q~ (Eq. 12) in two parts: add them, narrow into the attention kernel's rows.
    TQ* qrow = static_cast<TQ*>(a.qt) + (long long)b * a.n_heads * W;
    for (int i = t * 4; i < a.n_heads * a.r; i += 224 * 4) {
      const int h = i / a.r, j = i % a.r;
      float4 q4 = *reinterpret_cast<const float4*>(row + a.proj.off_q + i);
      const float4 ql = *reinterpret_cast<const float4*>(row + a.proj.off_q + a.n_heads * a.r + i);
      q4.x += ql.x; q4.y += ql.y; q4.z += ql.z; q4.w += ql.w;
      if (sizeof(TQ) == 2) {
        const __nv_bfloat162 h0 = __floats2bfloat162_rn(q4.x, q4.y), h1 = __floats2bfloat162_rn(q4.z, q4.w);
        *reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(qrow) + h * W + j) =
            make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
      } else {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(qrow) + h * W + j) = q4;
      }
    }
  } else if (a.q16) {
    const int hd = a.n_heads * a.head_dim;
    bf16* dst = a.q16 + (long long)b * 2 * hd;
    for (int i = t * 4; i < hd; i += 224 * 4) {
      const float4 q4 = *reinterpret_cast<const float4*>(row + a.proj.off_q + i);
      const __nv_bfloat162 h0 = __floats2bfloat162_rn(q4.x, q4.y), h1 = __floats2bfloat162_rn(q4.z, q4.w);
      const __nv_bfloat162 l0 = __floats2bfloat162_rn(q4.x - __low2float(h0), q4.y - __high2float(h0));
      const __nv_bfloat162 l1 = __floats2bfloat162_rn(q4.z - __low2float(h1), q4.w - __high2float(h1));
      *reinterpret_cast<uint2*>(dst + i) =
          make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
      *reinterpret_cast<uint2*>(dst + hd + i) =
          make_uint2(*reinterpret_cast<const uint32_t*>(&l0), *reinterpret_cast<const uint32_t*>(&l1));
    }
  }
  // Rotated, pre-scaled RoPE queries behind the (separately computed) absorbed query.
  TQ* qt = static_cast<TQ*>(a.qt) + (long long)b * a.n_heads * W;
  for (int i = t; i < a.n_heads * half; i += 224) {
    const int h = i / half, k = i % half;
    const float2 x2 = *reinterpret_cast<const float2*>(row + a.proj.off_qr + h * a.dr + 2 * k);
    const float cs = rope_cos[k], sn = rope_sin[k];
    const float y0 = (x2.x * cs - x2.y * sn) * a.q_scale, y1 = (x2.x * sn + x2.y * cs) * a.q_scale;
    if (sizeof(TQ) == 2)
      *reinterpret_cast<__nv_bfloat162*>(reinterpret_cast<bf16*>(qt) + h * W + a.r + 2 * k) =
          __floats2bfloat162_rn(y0, y1);
    else
      *reinterpret_cast<float2*>(reinterpret_cast<float*>(qt) + h * W + a.r + 2 * k) = make_float2(y0, y1);
  }
}

struct AttnArgs {
  const void* qt;      // [B][n_h][r + d_R], pre-scaled by log2(e)/sqrt(d_h)
  CacheView cache;
  float* o_part;       // [B * n_split][n_h][r] un-normalised partial outputs
  float* ml_part;      // [B * n_split][n_h][2]: running max (log2 units), sum
  const int* seq_tokens;   // [B] tokens per sequence (this step's included), or nullptr: n_slots
  int n_heads, r, dr, stride, n_slots, slots_per_split, n_split;
};

constexpr int kAttnFmaTile = 16;

inline size_t attn_fma_smem_bytes(int nh_padded, int r, int dr) {
  const int W = r + dr;
  return sizeof(float) * ((size_t)nh_padded * W + (size_t)kAttnFmaTile * (W + 1) +
                          (size_t)kAttnFmaTile * nh_padded + 3 * nh_padded);
}

// CUDA-core split-K decode attention in the absorbed form (Eq. 12 / Eq. 17): one CTA per
// (split, sequence) streams its slot range once; every head reuses the staged tile.
// T = cache element type, TQ = absorbed-query element type, NH = head count padded to the
// template instance, RPT = latent columns per thread.
template <typename T, typename TQ, int NH, int RPT>
__global__ void __launch_bounds__(256) decode_attn_fma_kernel(AttnArgs a) {
  extern __shared__ float smem[];
  constexpr int TS = kAttnFmaTile;
  constexpr int V = Elem<T>::kVec, VQ = Elem<TQ>::kVec;
  const int W = a.r + a.dr, WS = W + 1;
  float* qs = smem;
  float* tile = qs + NH * W;
  float* ps = tile + TS * WS;
  float* m_s = ps + TS * NH;
  float* fac_s = m_s + NH;
  const int tid = threadIdx.x, b = blockIdx.y, split = blockIdx.x;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();   // the query and the cache row are the previous kernels' output
  const int slot0 = split * a.slots_per_split;
  // A split beyond a short sequence's end leaves an empty partial (maximum -inf, sum 0).
  const int n_slots = a.seq_tokens ? ceil_div(a.seq_tokens[b], a.stride) : a.n_slots;
  const int slot1 = min(n_slots, slot0 + a.slots_per_split);
  const TQ* qt = static_cast<const TQ*>(a.qt) + (long long)b * a.n_heads * W;
  const T* cache = static_cast<const T*>(a.cache.base);

  for (int v = tid; v < NH * (W / VQ); v += 256) {
    const int h = v / (W / VQ), kv = (v % (W / VQ)) * VQ;
    float tmp[VQ];
    if (h < a.n_heads) {
      load_vec(qt + h * W + kv, tmp);
    } else {
#pragma unroll
      for (int e = 0; e < VQ; ++e) tmp[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < VQ; ++e) qs[h * W + kv + e] = tmp[e];
  }
  if (tid < NH) m_s[tid] = -INFINITY;
  float acc[NH][RPT];
#pragma unroll
  for (int h = 0; h < NH; ++h)
#pragma unroll
    for (int q = 0; q < RPT; ++q) acc[h][q] = 0.f;
  float l_run = 0.f;  // threads < NH: running softmax denominator of head tid

  for (int t0 = slot0; t0 < slot1; t0 += TS) {
    __syncthreads();
    for (int v = tid; v < TS * (W / V); v += 256) {
      const int sl = v / (W / V), kv = (v % (W / V)) * V;
      float tmp[V];
      if (t0 + sl < slot1) {
        load_vec(cache + cache_row(a.cache, b, t0 + sl) * W + kv, tmp);
      } else {
#pragma unroll
        for (int e = 0; e < V; ++e) tmp[e] = 0.f;
      }
#pragma unroll
      for (int e = 0; e < V; ++e) tile[sl * WS + kv + e] = tmp[e];
    }
    __syncthreads();
    for (int idx = tid; idx < NH * TS; idx += 256) {
      const int sl = idx % TS, h = idx / TS;
      const float* qrow = qs + h * W;
      const float* trow = tile + sl * WS;
      float d0 = 0.f, d1 = 0.f;
      for (int k = 0; k < W; k += 2) {
        d0 = fmaf(qrow[k], trow[k], d0);
        d1 = fmaf(qrow[k + 1], trow[k + 1], d1);
      }
      ps[sl * NH + h] = (t0 + sl < slot1) ? d0 + d1 : -INFINITY;
    }
    __syncthreads();
    if (tid < NH) {
      float m_new = m_s[tid];
#pragma unroll
      for (int sl = 0; sl < TS; ++sl) m_new = fmaxf(m_new, ps[sl * NH + tid]);
      fac_s[tid] = exp2f(m_s[tid] - m_new);  // 0 on the first tile (m = -inf)
      m_s[tid] = m_new;
    }
    __syncthreads();
    for (int idx = tid; idx < NH * TS; idx += 256) {
      const int h = idx % NH;
      ps[idx] = exp2f(ps[idx] - m_s[h]);
    }
    __syncthreads();
#pragma unroll
    for (int h = 0; h < NH; ++h) {
      const float f = fac_s[h];
#pragma unroll
      for (int q = 0; q < RPT; ++q) acc[h][q] *= f;
    }
    for (int sl = 0; sl < TS; ++sl) {
      float cv[RPT];
#pragma unroll
      for (int q = 0; q < RPT; ++q) {
        const int col = tid + 256 * q;
        cv[q] = col < a.r ? tile[sl * WS + col] : 0.f;
      }
#pragma unroll
      for (int h = 0; h < NH; ++h) {
        const float p = ps[sl * NH + h];
#pragma unroll
        for (int q = 0; q < RPT; ++q) acc[h][q] = fmaf(p, cv[q], acc[h][q]);
      }
    }
    if (tid < NH) {
      float sum = 0.f;
#pragma unroll
      for (int sl = 0; sl < TS; ++sl) sum += ps[sl * NH + tid];
      l_run = l_run * fac_s[tid] + sum;
    }
  }

  const long long unit = (long long)b * a.n_split + split;
  float* o_part = a.o_part + unit * a.n_heads * a.r;
#pragma unroll
  for (int h = 0; h < NH; ++h) {
    if (h >= a.n_heads) break;
#pragma unroll
    for (int q = 0; q < RPT; ++q) {
      const int col = tid + 256 * q;
      if (col < a.r) o_part[h * a.r + col] = acc[h][q];
    }
  }
  if (tid < a.n_heads) {
    a.ml_part[(unit * a.n_heads + tid) * 2] = m_s[tid];
    a.ml_part[(unit * a.n_heads + tid) * 2 + 1] = l_run;
  }
}

struct CombineArgs {
  const float* o_part;   // [B * n_split][n_h][r]
  const float* ml_part;  // [B * n_split][n_h][2]
  void* o;               // [B][n_h][r] normalised attention output in latent space; for bf16
                         // rows are [2][n_h][r]: hi halves, then the rounding remainders
  int n_heads, r, n_split;
};

// Cross-split combine: rescales each split's partial by 2^(m_split - m) and normalises.
// Grid (n_h, B), 128 threads over r.
template <typename T>
__global__ void __launch_bounds__(128) decode_combine_kernel(CombineArgs a) {
  const int h = blockIdx.x, b = blockIdx.y;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();
  float m = -INFINITY;
  for (int sp = 0; sp < a.n_split; ++sp)
    m = fmaxf(m, a.ml_part[(((long long)b * a.n_split + sp) * a.n_heads + h) * 2]);
  float denom = 0.f;
  for (int sp = 0; sp < a.n_split; ++sp) {
    const float* ml = a.ml_part + (((long long)b * a.n_split + sp) * a.n_heads + h) * 2;
    denom += exp2f(ml[0] - m) * ml[1];
  }
  const float inv = 1.f / denom;
  constexpr bool kSplit = sizeof(T) == 2;
  const long long lo_off = (long long)a.n_heads * a.r;
  T* o = static_cast<T*>(a.o) + ((long long)b * (kSplit ? 2 : 1) * a.n_heads + h) * a.r;
  for (int col = threadIdx.x; col < a.r; col += 128) {
    float sum = 0.f;
    for (int sp = 0; sp < a.n_split; ++sp) {
      const long long unit = (long long)b * a.n_split + sp;
      const float wgt = exp2f(a.ml_part[(unit * a.n_heads + h) * 2] - m);
      sum = fmaf(wgt, a.o_part[(unit * a.n_heads + h) * a.r + col], sum);
    }
    const float val = sum * inv;
    const T hi = Elem<T>::from_float(val);
    o[col] = hi;
    if (kSplit) o[lo_off + col] = Elem<T>::from_float(val - Elem<T>::to_float(hi));
  }
}

}  // namespace mtla
