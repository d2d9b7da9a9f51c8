// Kernels around the attention in a decoder layer (Section 5.2: MTLA self-attention plus a
// feed-forward block, pre-norm residual form): the LayerNorms on the fp32 residual stream and,
// for fp32 layers, the feed-forward epilogues that the tensor-core GEMM fuses for bf16 layers.
#pragma once

#include "common.cuh"

namespace mtla {

struct RowNormArgs {
  float* res;            // [rows][d] fp32 residual stream (read, and rewritten when `add` is set)
  const void* add;       // [rows][d] storage type, or nullptr
  int init;              // 1: res = add (the stream starts from the layer input), 0: res += add
  const float* gamma;    // [d]
  const float* beta;     // [d]
  void* out;             // [rows][d] storage type: LayerNorm(res)
  long long rows;
  int d;
  float eps;
};

// One warp per row, 8 rows per CTA.  res <- (init ? add : res + add) when add is given, then
// out = LayerNorm(res) in the storage type.  The row is walked three times (mean, variance,
// output) with 16-byte accesses; d is a multiple of 8, so every row start is 16-byte aligned.
// Two-pass variance in fp32, as the attention's own LayerNorm.
template <typename T>
__global__ void __launch_bounds__(256) row_norm_kernel(RowNormArgs a) {
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();   // the rows are the previous kernel's output
  if (row >= a.rows) return;
  float* res = a.res + row * a.d;
  const T* add = a.add ? static_cast<const T*>(a.add) + row * a.d : nullptr;
  constexpr int V = Elem<T>::kVec;          // elements per 16-byte access of the storage type
  float sum = 0.f;
  for (int i = lane * V; i < a.d; i += 32 * V) {
    float v[V];
#pragma unroll
    for (int e = 0; e < V; e += 4) {
      const float4 r4 = a.init ? make_float4(0.f, 0.f, 0.f, 0.f)
                               : *reinterpret_cast<const float4*>(res + i + e);
      v[e] = r4.x; v[e + 1] = r4.y; v[e + 2] = r4.z; v[e + 3] = r4.w;
    }
    if (add) {
      float w[V];
      load_vec(add + i, w);
#pragma unroll
      for (int e = 0; e < V; ++e) v[e] += w[e];
#pragma unroll
      for (int e = 0; e < V; e += 4)
        *reinterpret_cast<float4*>(res + i + e) = make_float4(v[e], v[e + 1], v[e + 2], v[e + 3]);
    }
#pragma unroll
    for (int e = 0; e < V; ++e) sum += v[e];
  }
  const float mean = warp_sum(sum) / a.d;
  __syncwarp();                                // this warp's own writes to res are read below
  float sq = 0.f;
  for (int i = lane * 4; i < a.d; i += 128) {
    const float4 r4 = *reinterpret_cast<const float4*>(res + i);
    const float d0 = r4.x - mean, d1 = r4.y - mean, d2 = r4.z - mean, d3 = r4.w - mean;
    sq += d0 * d0 + d1 * d1 + d2 * d2 + d3 * d3;
  }
  const float rstd = rsqrtf(warp_sum(sq) / a.d + a.eps);
  T* out = static_cast<T*>(a.out) + row * a.d;
  for (int i = lane * V; i < a.d; i += 32 * V) {
    float v[V];
#pragma unroll
    for (int e = 0; e < V; e += 4) {
      const float4 r4 = *reinterpret_cast<const float4*>(res + i + e);
      const float4 g4 = *reinterpret_cast<const float4*>(a.gamma + i + e);
      const float4 b4 = *reinterpret_cast<const float4*>(a.beta + i + e);
      v[e] = (r4.x - mean) * rstd * g4.x + b4.x;
      v[e + 1] = (r4.y - mean) * rstd * g4.y + b4.y;
      v[e + 2] = (r4.z - mean) * rstd * g4.z + b4.z;
      v[e + 3] = (r4.w - mean) * rstd * g4.w + b4.w;
    }
    store_vec(out + i, v);
  }
}

// fp32 layers: out[row][j] = (relu?)(acc[row][j] + bias[j]) (+ residual[row][j]), the epilogue the
// CUDA-core GEMM does not have.  acc and out may alias; residual may alias out.
__global__ void __launch_bounds__(256) bias_act_residual_kernel(const float* acc, const float* bias,
                                                                const float* residual, float* out,
                                                                long long rows, int n, int relu) {
  const long long idx = ((long long)blockIdx.x * 256 + threadIdx.x) * 4;
  if (idx >= rows * n) return;
  const int j = (int)(idx % n);
  const float4 v = *reinterpret_cast<const float4*>(acc + idx);
  const float4 b = *reinterpret_cast<const float4*>(bias + j);
  float o[4] = {v.x + b.x, v.y + b.y, v.z + b.z, v.w + b.w};
  if (relu) {
#pragma unroll
    for (int e = 0; e < 4; ++e) o[e] = fmaxf(o[e], 0.f);
  }
  if (residual) {
    const float4 r = *reinterpret_cast<const float4*>(residual + idx);
    o[0] += r.x; o[1] += r.y; o[2] += r.z; o[3] += r.w;
  }
  *reinterpret_cast<float4*>(out + idx) = make_float4(o[0], o[1], o[2], o[3]);
}

}  // namespace mtla
