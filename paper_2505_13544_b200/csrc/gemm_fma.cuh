// CUDA-core (fp32 FMA) GEMM used wherever a projection is not on the tensor-core path:
// the fp32 configuration (TF32 would break its 1e-4 bound), small batches, and as the
// shape-generic fallback.  Computes, for each batch index z,
//     C[z][m][n] = alpha * sum_k A[z][m][k] * Bt[z][n][k]
// with A and Bt both K-contiguous ("NT" form: weights are stored as [out][in]).
#pragma once

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mtla {

struct GemmArgs {
  const void* a;   // [M][lda]
  const void* bt;  // [N][ldb]
  void* c;         // [M][ldc]
  int m, n, k;
  int lda, ldb, ldc;           // in elements
  long long za, zb, zc;        // per-z element offsets
  float alpha;
};

// Tile: BM x 64 outputs per CTA of 256 threads, BK = 32.  Thread (ty, tx) of a 16 x 16
// grid owns rows ty + 16*i (i < BM/16) and columns tx*4 .. tx*4+3.
template <typename TA, typename TB, typename TOut, int BM>
__global__ void __launch_bounds__(256) gemm_nt_fma_kernel(GemmArgs g) {
  constexpr int BN = 64, BK = 32, TM = BM / 16, TN = 4;
  constexpr int VA = Elem<TA>::kVec, VB = Elem<TB>::kVec;
  __shared__ float as[BK][BM + 4];
  __shared__ float bs[BK][BN + 4];

  const TA* a = static_cast<const TA*>(g.a) + (long long)blockIdx.z * g.za;
  const TB* bt = static_cast<const TB*>(g.bt) + (long long)blockIdx.z * g.zb;
  TOut* c = static_cast<TOut*>(g.c) + (long long)blockIdx.z * g.zc;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();   // a no-op unless this is a programmatic dependent launch

  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < g.k; k0 += BK) {
    // Stage A and Bt tiles (transposed to [k][row]) as fp32.
    for (int v = tid; v < BM * (BK / VA); v += 256) {
      const int row = v / (BK / VA), kv = (v % (BK / VA)) * VA;
      float tmp[VA];
      if (m0 + row < g.m && k0 + kv < g.k) {
        load_vec(a + (long long)(m0 + row) * g.lda + k0 + kv, tmp);
      } else {
#pragma unroll
        for (int e = 0; e < VA; ++e) tmp[e] = 0.f;
      }
#pragma unroll
      for (int e = 0; e < VA; ++e) as[kv + e][row] = tmp[e];
    }
    for (int v = tid; v < BN * (BK / VB); v += 256) {
      const int row = v / (BK / VB), kv = (v % (BK / VB)) * VB;
      float tmp[VB];
      if (n0 + row < g.n && k0 + kv < g.k) {
        load_vec(bt + (long long)(n0 + row) * g.ldb + k0 + kv, tmp);
      } else {
#pragma unroll
        for (int e = 0; e < VB; ++e) tmp[e] = 0.f;
      }
#pragma unroll
      for (int e = 0; e < VB; ++e) bs[kv + e][row] = tmp[e];
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float av[TM], bv[TN];
#pragma unroll
      for (int i = 0; i < TM; ++i) av[i] = as[kk][ty + 16 * i];
      const float4 b4 = *reinterpret_cast<const float4*>(&bs[kk][tx * 4]);
      bv[0] = b4.x; bv[1] = b4.y; bv[2] = b4.z; bv[3] = b4.w;
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }

#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int row = m0 + ty + 16 * i;
    if (row >= g.m) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int col = n0 + tx * 4 + j;
      if (col < g.n)
        c[(long long)row * g.ldc + col] = Elem<TOut>::from_float(g.alpha * acc[i][j]);
    }
  }
}

// Launches the NT GEMM over `batches` z-slices.  K must be a multiple of the 16-byte
// vector widths of TA and TB and all row starts 16-byte aligned (guaranteed by the caller).
template <typename TA, typename TB, typename TOut>
inline cudaError_t launch_gemm_nt_fma(const GemmArgs& g, int batches, cudaStream_t st,
                                      bool dependent = false) {
  if (g.m <= 0 || g.n <= 0 || batches <= 0) return cudaSuccess;
  if (g.m <= 16) {
    dim3 grid(ceil_div(g.n, 64), ceil_div(g.m, 16), batches);
    return launch_kernel(gemm_nt_fma_kernel<TA, TB, TOut, 16>, grid, dim3(256), 0, st, dependent, g);
  } else if (g.m <= 64) {
    dim3 grid(ceil_div(g.n, 64), ceil_div(g.m, 64), batches);
    return launch_kernel(gemm_nt_fma_kernel<TA, TB, TOut, 64>, grid, dim3(256), 0, st, dependent, g);
  }
  dim3 grid(ceil_div(g.n, 64), ceil_div(g.m, 128), batches);
  return launch_kernel(gemm_nt_fma_kernel<TA, TB, TOut, 128>, grid, dim3(256), 0, st, dependent, g);
}

}  // namespace mtla
