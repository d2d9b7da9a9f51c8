// Prefill kernels that are not GEMMs: the per-chunk LayerNorm / gate / running-merge kernel
// and the CUDA-core attention under the stride-aware causal mask (Section 4.2).
#pragma once

#include <math.h>

#include "common.cuh"
#include "decode_kernels.cuh"

namespace mtla {

struct PrefillPostArgs {
  const float* p1;        // [B*T][proj.width] fused input projection (fp32)
  ProjLayout proj;
  const float* gamma;
  const float* beta;
  const float* hyp_c_w;   // [r][d_w]
  const float* hyp_c_b;   // [d_w]
  const float* gate_pe;   // [max_slots][d_w]; row j0 is Linear(pe_{j0+1})
  const float* gate_s;    // [d_w], [d_w]: constants of the folded gate (see ProjLayout)
  const float* gate_t;
  const float* rope_cos;  // [max_tokens][d_R/2]
  const float* rope_sin;
  float* open_acc;        // [B][r]
  CacheView cache;
  int seq0;               // the call's sequences are seq0, seq0 + 1, ... of the cache
  void* qcat;             // [B*T][n_h][d_h + d_R]: scaled query and rotated RoPE query
  void* cprime;           // [B*T][r]: running merge state after each token (Eq. 14's sequence)
  void* kr;               // [B*T][d_R]: rotated RoPE key of each token (query element type)
  int n_heads, head_dim, r, dr, dw, stride, T, max_slots;
  int batch;              // sequences of the call (prefill_post_fast_kernel's grid is flat)
  int q_done;             // 1: the projection kernel has already written the scaled queries to qcat
  int use_gate;
  float ln_eps, q_scale;
};

// One CTA per (chunk, sequence): walks the chunk's <= s tokens in order so that the running
// sum is formed exactly as the decode steps would form it, and leaves the chunk's final
// state in the cache (the last chunk also leaves the fp32 accumulator for later decoding).
// T is the cache / state element type, TQ the element type of the query buffer.
template <typename T, typename TQ>
__global__ void __launch_bounds__(256) prefill_post_kernel(PrefillPostArgs a) {
  __shared__ float c_s[512];
  __shared__ float acc_s[512];
  __shared__ float part_s[512];
  __shared__ float red_s[33];
  const int chunk = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
  const int W = a.r + a.dr, DQ = a.head_dim + a.dr, half = a.dr / 2;
  const int tok0 = chunk * a.stride, tok1 = min(a.T, tok0 + a.stride);
  const float* gate_pe = a.gate_pe + (long long)chunk * a.dw;
  for (int i = tid; i < a.r; i += 256) acc_s[i] = 0.f;

  for (int tok = tok0; tok < tok1; ++tok) {
    const long long rowi = (long long)b * a.T + tok;
    const float* row = a.p1 + rowi * a.proj.width;
    __syncthreads();
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
    for (int i = tid; i < a.r; i += 256)
      c_s[i] = (c_s[i] - mean) * rstd * a.gamma[i] + a.beta[i];
    __syncthreads();

    float w = 1.f;
    if (a.use_gate)
      w = a.proj.off_u >= 0
              ? gate_weight_folded(row + a.proj.off_u, a.dw, mean, rstd, a.gate_s, a.gate_t, gate_pe, red_s)
              : gate_weight(c_s, a.hyp_c_w, a.hyp_c_b, gate_pe, a.r, a.dw, part_s, red_s);

    T* cp = static_cast<T*>(a.cprime) + rowi * a.r;
    for (int i = tid; i < a.r; i += 256) {
      const float v = acc_s[i] + w * c_s[i];
      acc_s[i] = v;
      cp[i] = Elem<T>::from_float(v);
    }
    const float* cs_row = a.rope_cos + (long long)tok * half;
    const float* sn_row = a.rope_sin + (long long)tok * half;
    // Keys are rounded to the cache type (what decoding would read back), held as TQ.
    TQ* kr = static_cast<TQ*>(a.kr) + rowi * a.dr;
    for (int k = tid; k < half; k += 256) {
      const float x0 = row[a.proj.off_kr + 2 * k], x1 = row[a.proj.off_kr + 2 * k + 1];
      const T k0 = Elem<T>::from_float(x0 * cs_row[k] - x1 * sn_row[k]);
      const T k1 = Elem<T>::from_float(x0 * sn_row[k] + x1 * cs_row[k]);
      kr[2 * k] = Elem<TQ>::from_float(Elem<T>::to_float(k0));
      kr[2 * k + 1] = Elem<TQ>::from_float(Elem<T>::to_float(k1));
    }
    TQ* qc = static_cast<TQ*>(a.qcat) + rowi * a.n_heads * DQ;
    for (int i = tid; i < a.n_heads * a.head_dim; i += 256) {
      const int h = i / a.head_dim, e = i % a.head_dim;
      qc[h * DQ + e] = Elem<TQ>::from_float(row[a.proj.off_q + i] * a.q_scale);
    }
    for (int i = tid; i < a.n_heads * half; i += 256) {
      const int h = i / half, k = i % half;
      const float x0 = row[a.proj.off_qr + h * a.dr + 2 * k];
      const float x1 = row[a.proj.off_qr + h * a.dr + 2 * k + 1];
      qc[h * DQ + a.head_dim + 2 * k] =
          Elem<TQ>::from_float((x0 * cs_row[k] - x1 * sn_row[k]) * a.q_scale);
      qc[h * DQ + a.head_dim + 2 * k + 1] =
          Elem<TQ>::from_float((x0 * sn_row[k] + x1 * cs_row[k]) * a.q_scale);
    }
  }
  __syncthreads();

  // The chunk's state after its last available token is what the cache holds.
  const long long last = (long long)b * a.T + (tok1 - 1);
  T* slot_row = static_cast<T*>(a.cache.base) + cache_row(a.cache, a.seq0 + b, chunk) * W;
  const TQ* kr = static_cast<const TQ*>(a.kr) + last * a.dr;
  for (int i = tid; i < a.r; i += 256) slot_row[i] = Elem<T>::from_float(acc_s[i]);
  for (int i = tid; i < a.dr; i += 256)
    slot_row[a.r + i] = Elem<T>::from_float(Elem<TQ>::to_float(kr[i]));
  if (tok1 == a.T)
    for (int i = tid; i < a.r; i += 256) a.open_acc[(long long)(a.seq0 + b) * a.r + i] = acc_s[i];
}

// Stores four / two consecutive values in the element type of the destination (16 / 8 bytes of
// fp32, 8 / 4 bytes of bf16; the address is aligned to the access).
__device__ __forceinline__ void put4(float* p, float v0, float v1, float v2, float v3) {
  *reinterpret_cast<float4*>(p) = make_float4(v0, v1, v2, v3);
}
__device__ __forceinline__ void put4(bf16* p, float v0, float v1, float v2, float v3) {
  const __nv_bfloat162 a = __floats2bfloat162_rn(v0, v1), b = __floats2bfloat162_rn(v2, v3);
  *reinterpret_cast<uint2*>(p) =
      make_uint2(*reinterpret_cast<const uint32_t*>(&a), *reinterpret_cast<const uint32_t*>(&b));
}
__device__ __forceinline__ void put2(float* p, float v0, float v1) {
  *reinterpret_cast<float2*>(p) = make_float2(v0, v1);
}
__device__ __forceinline__ void put2(bf16* p, float v0, float v1) {
  *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(v0, v1);
}

// The same work for layers whose gate needs no matrix (folded into the projection, or absent at
// s = 1) and whose stride is at most 8, laid out for bandwidth: ONE WARP per (chunk, sequence),
// eight chunks per CTA, no shared memory and no block-wide barrier.  The warp walks the chunk's
// tokens in order; lane l owns latent columns 128 k + 4 l .. + 3 (k < 4), so the projection row is
// read and the running state written 16 bytes at a time, the LayerNorm statistics are warp
// shuffles, and the running sum lives in registers and grows in the same fp32 order as the
// decode steps form it.  Queries and RoPE queries / keys move as 16- and 8-byte vectors too.
constexpr int kPostFastMaxStride = 8;

template <typename T, typename TQ>
__global__ void __launch_bounds__(256, 3) prefill_post_fast_kernel(PrefillPostArgs a) {
  const int lane = threadIdx.x & 31;
  const int chunks = (a.T + a.stride - 1) / a.stride;
  const long long unit = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);    // (sequence, chunk)
  if (unit >= (long long)a.batch * chunks) return;
  const int b = (int)(unit / chunks), chunk = (int)(unit % chunks);
  const int W = a.r + a.dr, DQ = a.head_dim + a.dr, half = a.dr / 2;
  const int tok0 = chunk * a.stride, ntok = min(a.T, tok0 + a.stride) - tok0;
  const long long row0 = (long long)b * a.T + tok0;
  const int hd = a.n_heads * a.head_dim, dh_shift = a.head_dim == 64 ? 6 : 7;   // d_h is 64 or 128
  T* slot_row = static_cast<T*>(a.cache.base) + cache_row(a.cache, a.seq0 + b, chunk) * W;

  float acc[16];
#pragma unroll
  for (int k = 0; k < 16; ++k) acc[k] = 0.f;
  for (int t = 0; t < ntok; ++t) {
    const long long rowi = row0 + t;
    const float* row = a.p1 + rowi * a.proj.width;
    // Latent: LayerNorm (two-pass variance over the registers), gate, running sum.
    float cv[16];
    float sum = 0.f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = 128 * k + 4 * lane;
      const float4 c4 = i < a.r ? *reinterpret_cast<const float4*>(row + a.proj.off_c + i)
                                : make_float4(0.f, 0.f, 0.f, 0.f);
      cv[4 * k] = c4.x; cv[4 * k + 1] = c4.y; cv[4 * k + 2] = c4.z; cv[4 * k + 3] = c4.w;
      sum += (c4.x + c4.y) + (c4.z + c4.w);
    }
    const float mean = warp_sum(sum) / a.r;
    float sq = 0.f;
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      const float dlt = 128 * (k / 4) + 4 * lane < a.r ? cv[k] - mean : 0.f;
      sq += dlt * dlt;
    }
    const float rstd = rsqrtf(warp_sum(sq) / a.r + a.ln_eps);
    float w = 1.f;
    if (a.use_gate) {
      const float* u = row + a.proj.off_u;
      const float* gate_pe = a.gate_pe + (long long)chunk * a.dw;
      float prod = 0.f;
      for (int n = lane; n < a.dw; n += 32) {
        const float h = rstd * (u[n] + u[a.dw + n] - mean * a.gate_s[n]) + a.gate_t[n];
        prod = fmaf(h, gate_pe[n], prod);
      }
      w = 1.f / (1.f + expf(-warp_sum(prod)));
    }
    T* cp = static_cast<T*>(a.cprime) + rowi * a.r;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = 128 * k + 4 * lane;
      if (i >= a.r) continue;
      const float4 g4 = *reinterpret_cast<const float4*>(a.gamma + i);
      const float4 b4 = *reinterpret_cast<const float4*>(a.beta + i);
      const float gam[4] = {g4.x, g4.y, g4.z, g4.w}, bet[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float c = (cv[4 * k + e] - mean) * rstd * gam[e] + bet[e];
        acc[4 * k + e] += w * c;
      }
      put4(cp + i, acc[4 * k], acc[4 * k + 1], acc[4 * k + 2], acc[4 * k + 3]);
    }
    // RoPE key (rounded to the cache type, which is what decoding reads back); the slot keeps
    // the key of the chunk's last token.
    const float* cs_row = a.rope_cos + (long long)(tok0 + t) * half;
    const float* sn_row = a.rope_sin + (long long)(tok0 + t) * half;
    if (lane < half) {
      const float2 x = *reinterpret_cast<const float2*>(row + a.proj.off_kr + 2 * lane);
      const float cs = cs_row[lane], sn = sn_row[lane];
      const float k0 = Elem<T>::to_float(Elem<T>::from_float(x.x * cs - x.y * sn));
      const float k1 = Elem<T>::to_float(Elem<T>::from_float(x.x * sn + x.y * cs));
      put2(static_cast<TQ*>(a.kr) + rowi * a.dr + 2 * lane, k0, k1);
      if (t == ntok - 1) put2(slot_row + a.r + 2 * lane, k0, k1);
    }
    // Scaled queries, four columns per lane and step (they never straddle a head).
    TQ* qrow = static_cast<TQ*>(a.qcat) + rowi * a.n_heads * DQ;
    // (Four loads are issued before the first store: the compiler cannot move a load over a
    // store to another buffer by itself.)
    for (int i0 = 4 * lane; i0 < hd && !a.q_done; i0 += 512) {
      float4 q4[4];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (i0 + 128 * j < hd) q4[j] = *reinterpret_cast<const float4*>(row + a.proj.off_q + i0 + 128 * j);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int i = i0 + 128 * j;
        if (i < hd)
          put4(qrow + (i >> dh_shift) * DQ + (i & (a.head_dim - 1)), q4[j].x * a.q_scale,
               q4[j].y * a.q_scale, q4[j].z * a.q_scale, q4[j].w * a.q_scale);
      }
    }
    // Rotated, scaled RoPE queries, one pair per lane and step.
    // Pair idx of the row = pair idx mod (d_R / 2) of head idx / (d_R / 2); the pairs of a row are
    // contiguous in the projection, so lane and step index them directly.
    const int half_shift = half == 16 ? 4 : 5;                      // d_R is 32 or 64
    for (int i0 = lane; i0 < a.n_heads * half; i0 += 128) {
      float2 x[4];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (i0 + 32 * j < a.n_heads * half)
          x[j] = *reinterpret_cast<const float2*>(row + a.proj.off_qr + 2 * (i0 + 32 * j));
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int idx = i0 + 32 * j;
        if (idx >= a.n_heads * half) continue;
        const int h = idx >> half_shift, k = idx & (half - 1);
        const float cs = cs_row[k], sn = sn_row[k];
        put2(qrow + h * DQ + a.head_dim + 2 * k, (x[j].x * cs - x[j].y * sn) * a.q_scale,
             (x[j].x * sn + x[j].y * cs) * a.q_scale);
      }
    }
  }
  // The chunk's final state is what the cache holds; the last, still open chunk also leaves its
  // fp32 sum for the decode steps that follow.
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int i = 128 * k + 4 * lane;
    if (i >= a.r) continue;
    put4(slot_row + i, acc[4 * k], acc[4 * k + 1], acc[4 * k + 2], acc[4 * k + 3]);
    if (tok0 + ntok == a.T)
      *reinterpret_cast<float4*>(a.open_acc + (long long)(a.seq0 + b) * a.r + i) =
          make_float4(acc[4 * k], acc[4 * k + 1], acc[4 * k + 2], acc[4 * k + 3]);
  }
}

struct PrefillAttnArgs {
  const void* qcat;   // [B*T][n_h][d_h + d_R], pre-scaled by log2(e)/sqrt(d_h)
  const void* kv;     // [B*T][2*n_h*d_h]: keys then values up-projected from cprime (Eq. 9-10)
  const void* kr;     // [B*T][d_R]
  void* out;          // [B*T][n_h*d_h] per-head attention outputs (input of W_O); bf16 rows
                      // are [2][n_h*d_h]: hi halves, then the rounding remainders
  int n_heads, dr, stride, T;
};

constexpr int kPfTile = 64;

inline size_t prefill_attn_fma_smem_bytes(int dh, int dr) {
  const int DQ = dh + dr;
  return sizeof(float) * ((size_t)2 * DQ * kPfTile + (size_t)kPfTile * dh +
                          (size_t)kPfTile * (kPfTile + 1));
}

// CUDA-core flash-style attention for the prefill.  Row m (0-based token) sees the closed
// slots j < floor(m/s), each represented by the state and RoPE key of its last token
// j*s + s - 1, plus its own running state at column m: exactly the columns the
// stride-aware mask of Section 4.2 admits.  The mask is a predicate on (m, j).
// Grid (ceil(T/64), n_h, B), 256 threads as 16 x 16, each owning a 4 x 4 score patch.
// TQ = element type of queries, keys, values and RoPE keys; TOut = element type of the outputs.
template <typename TQ, typename TOut, int DH>
__global__ void __launch_bounds__(256) prefill_attn_fma_kernel(PrefillAttnArgs a) {
  extern __shared__ float smem[];
  constexpr int BT = kPfTile, V = Elem<TQ>::kVec, OC = DH / 16;
  const int DQ = DH + a.dr;
  float* qs = smem;                 // [DQ][BT]  (transposed: k-major)
  float* ks = qs + DQ * BT;         // [DQ][BT]
  float* vs = ks + DQ * BT;         // [BT][DH]
  float* ps = vs + BT * DH;         // [BT][BT+1]
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int q0 = blockIdx.x * BT, h = blockIdx.y, b = blockIdx.z;
  const TQ* qcat = static_cast<const TQ*>(a.qcat);
  const TQ* kv = static_cast<const TQ*>(a.kv);
  const TQ* kr = static_cast<const TQ*>(a.kr);
  const long long base = (long long)b * a.T;
  const int kvw = 2 * a.n_heads * DH;

  for (int v = tid; v < BT * (DQ / V); v += 256) {
    const int row = v / (DQ / V), kk = (v % (DQ / V)) * V;
    float tmp[V];
    if (q0 + row < a.T) {
      load_vec(qcat + ((base + q0 + row) * a.n_heads + h) * DQ + kk, tmp);
    } else {
#pragma unroll
      for (int e = 0; e < V; ++e) tmp[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < V; ++e) qs[(kk + e) * BT + row] = tmp[e];
  }

  float m_run[4], l_run[4], o[4][OC];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m_run[i] = -INFINITY;
    l_run[i] = 0.f;
#pragma unroll
    for (int c = 0; c < OC; ++c) o[i][c] = 0.f;
  }

  const int last_row = min(a.T, q0 + BT) - 1;
  const int n_closed = last_row / a.stride;         // closed slots visible to the last row
  const int n_tiles = ceil_div(n_closed, BT);
  // Tiles 0..n_tiles-1 walk the closed slots; tile n_tiles is the diagonal (own state).
  for (int t = 0; t <= n_tiles; ++t) {
    const bool diag = (t == n_tiles);
    __syncthreads();
    for (int v = tid; v < BT * (DQ / V); v += 256) {
      const int col = v / (DQ / V), kk = (v % (DQ / V)) * V;
      const int j = t * BT + col;
      const long long tok = diag ? (long long)(q0 + col) : (long long)j * a.stride + a.stride - 1;
      const bool ok = diag ? (q0 + col < a.T) : (j < n_closed);
      float tmp[V];
      if (ok) {
        if (kk < DH) load_vec(kv + (base + tok) * kvw + h * DH + kk, tmp);
        else load_vec(kr + (base + tok) * a.dr + (kk - DH), tmp);
      } else {
#pragma unroll
        for (int e = 0; e < V; ++e) tmp[e] = 0.f;
      }
#pragma unroll
      for (int e = 0; e < V; ++e) ks[(kk + e) * BT + col] = tmp[e];
    }
    for (int v = tid; v < BT * (DH / V); v += 256) {
      const int col = v / (DH / V), kk = (v % (DH / V)) * V;
      const int j = t * BT + col;
      const long long tok = diag ? (long long)(q0 + col) : (long long)j * a.stride + a.stride - 1;
      const bool ok = diag ? (q0 + col < a.T) : (j < n_closed);
      float tmp[V];
      if (ok) {
        load_vec(kv + (base + tok) * kvw + a.n_heads * DH + h * DH + kk, tmp);
      } else {
#pragma unroll
        for (int e = 0; e < V; ++e) tmp[e] = 0.f;
      }
#pragma unroll
      for (int e = 0; e < V; ++e) vs[col * DH + kk + e] = tmp[e];
    }
    __syncthreads();

    float sc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) sc[i][j] = 0.f;
    for (int k = 0; k < DQ; ++k) {
      const float4 q4 = *reinterpret_cast<const float4*>(qs + k * BT + ty * 4);
      const float4 k4 = *reinterpret_cast<const float4*>(ks + k * BT + tx * 4);
      const float qv[4] = {q4.x, q4.y, q4.z, q4.w}, kv4[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) sc[i][j] = fmaf(qv[i], kv4[j], sc[i][j]);
    }
    // Stride-aware mask as a predicate, then the online softmax update per row.
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = q0 + ty * 4 + i;
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int col = tx * 4 + j;
        const bool allowed = diag ? (col == ty * 4 + i && row < a.T)
                                  : (t * BT + col < row / a.stride);
        sc[i][j] = allowed ? sc[i][j] : -INFINITY;
        mx = fmaxf(mx, sc[i][j]);
      }
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
      const float m_new = fmaxf(m_run[i], mx);
      const float fac = (m_new == -INFINITY) ? 1.f : exp2f(m_run[i] - m_new);
      float sum = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float p = (m_new == -INFINITY) ? 0.f : exp2f(sc[i][j] - m_new);
        ps[(ty * 4 + i) * (BT + 1) + tx * 4 + j] = p;
        sum += p;
      }
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
      l_run[i] = l_run[i] * fac + sum;
      m_run[i] = m_new;
#pragma unroll
      for (int c = 0; c < OC; ++c) o[i][c] *= fac;
    }
    __syncthreads();
    for (int k = 0; k < BT; ++k) {
      float vv[OC];
#pragma unroll
      for (int c = 0; c < OC; ++c) vv[c] = vs[k * DH + tx * OC + c];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float p = ps[(ty * 4 + i) * (BT + 1) + k];
#pragma unroll
        for (int c = 0; c < OC; ++c) o[i][c] = fmaf(p, vv[c], o[i][c]);
      }
    }
  }

  TOut* out = static_cast<TOut*>(a.out);
  constexpr bool kSplit = sizeof(TOut) == 2;
  const long long hdw = (long long)a.n_heads * DH;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = q0 + ty * 4 + i;
    if (row >= a.T) continue;
    const float inv = 1.f / l_run[i];
    TOut* orow = out + (base + row) * (kSplit ? 2 : 1) * hdw + h * DH + tx * OC;
#pragma unroll
    for (int c = 0; c < OC; ++c) {
      const float val = o[i][c] * inv;
      const TOut hi = Elem<TOut>::from_float(val);
      orow[c] = hi;
      if (kSplit) orow[hdw + c] = Elem<TOut>::from_float(val - Elem<TOut>::to_float(hi));
    }
  }
}

}  // namespace mtla
