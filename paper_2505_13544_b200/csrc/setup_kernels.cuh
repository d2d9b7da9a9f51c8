// One-time kernels run by mtla_create: weight repacking and the positional tables.
#pragma once

#include <math.h>

#include "common.cuh"

namespace mtla {

// dst[n][k] = src[k][n] for a row-major src [K][N] (leading dimension ld_src); dst has
// leading dimension ld_dst.  Grid (ceil(N/32), ceil(K/32)), block (32, 8).
template <typename T>
__global__ void transpose_kernel(const T* src, T* dst, int K, int N, int ld_src, int ld_dst) {
  __shared__ T tile[32][33];
  const int n0 = blockIdx.x * 32, k0 = blockIdx.y * 32;
  for (int i = threadIdx.y; i < 32; i += 8) {
    const int k = k0 + i, n = n0 + threadIdx.x;
    if (k < K && n < N) tile[i][threadIdx.x] = src[(long long)k * ld_src + n];
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += 8) {
    const int n = n0 + i, k = k0 + threadIdx.x;
    if (k < K && n < N) dst[(long long)n * ld_dst + k] = tile[threadIdx.x][i];
  }
}

// dst (fp32) = src (T); src == nullptr fills zeros.
template <typename T>
__global__ void widen_kernel(const T* src, float* dst, long long n) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = src ? Elem<T>::to_float(src[i]) : 0.f;
}

// Folding Linear(c_i) of Eq. 13 into the input projection (see ProjLayout).
// ga[n][i] = gamma[i] * A[i][n]: the [d_w][r] left operand of W_g^T = ga . W_r^T.
__global__ void gate_fold_scale_kernel(const float* a /*[r][d_w]*/, const float* gamma, float* ga,
                                       int r, int dw) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= r * dw) return;
  const int n = idx / r, i = idx % r;
  ga[idx] = gamma[i] * a[(long long)i * dw + n];
}

// Splits W_g^T [d_w][d] (fp32) into bf16 halves: rows [0, d_w) of dst receive the rounded
// values, rows [d_w, 2 d_w) the rounding remainders.
__global__ void gate_fold_pack_kernel(const float* wg, bf16* dst, int dw, long long d) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= dw * d) return;
  const bf16 hi = __float2bfloat16_rn(wg[idx]);
  dst[idx] = hi;
  dst[dw * d + idx] = __float2bfloat16_rn(wg[idx] - __bfloat162float(hi));
}

// Splits a rows x cols fp32 matrix (row pitch ld_src) into bf16 halves: `hi` receives the rounded
// values, `lo` the rounding remainders, both with row pitch ld_dst.
__global__ void split_hi_lo_kernel(const float* src, bf16* hi, bf16* lo, int rows, int cols,
                                   long long ld_src, long long ld_dst) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)rows * cols) return;
  const long long i = idx / cols, j = idx % cols;
  const float v = src[i * ld_src + j];
  const bf16 h = __float2bfloat16_rn(v);
  hi[i * ld_dst + j] = h;
  lo[i * ld_dst + j] = __float2bfloat16_rn(v - __bfloat162float(h));
}

// gate_s[n] = sum_i gamma[i] A[i][n];  gate_t[n] = sum_i beta[i] A[i][n] + a[n].
__global__ void gate_fold_vectors_kernel(const float* a /*[r][d_w]*/, const float* bias,
                                         const float* gamma, const float* beta, float* gate_s,
                                         float* gate_t, int r, int dw) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= dw) return;
  double s = 0.0, t = bias[n];
  for (int i = 0; i < r; ++i) {
    const double w = a[(long long)i * dw + n];
    s += gamma[i] * w;
    t += beta[i] * w;
  }
  gate_s[n] = (float)s;
  gate_t[n] = (float)t;
}

// Row j0 of the table is Linear(pe_j) of Eq. 13 for the 1-based slot number j = j0 + 1:
// pe_j is the sinusoidal embedding of dimension r (sin at even, cos at odd indices,
// wavelengths 10000^(2k/r)), evaluated in fp64.  One CTA per slot number.
__global__ void __launch_bounds__(256) gate_pe_table_kernel(const float* w /*[r][d_w]*/,
                                                            const float* bias /*[d_w]*/,
                                                            float* table /*[slots][d_w]*/,
                                                            int r, int dw) {
  __shared__ double pe[512];
  const int j = blockIdx.x + 1;
  for (int k = threadIdx.x; k < r / 2; k += blockDim.x) {
    const double angle = (double)j / pow(10000.0, 2.0 * k / r);
    pe[2 * k] = sin(angle);
    pe[2 * k + 1] = cos(angle);
  }
  __syncthreads();
  for (int n = threadIdx.x; n < dw; n += blockDim.x) {
    double acc = bias[n];
    for (int i = 0; i < r; ++i) acc += pe[i] * (double)w[(long long)i * dw + n];
    table[(long long)blockIdx.x * dw + n] = (float)acc;
  }
}

// cos/sin of pos * theta^(-2k/d_R) for every position and pair index (Section 4.3), fp64
// evaluation rounded to fp32.
__global__ void rope_table_kernel(float* cos_t, float* sin_t, int positions, int half,
                                  double theta) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long long)positions * half) return;
  const int pos = (int)(i / half), k = (int)(i % half);
  const double angle = (double)pos * pow(theta, -2.0 * k / (2.0 * half));
  cos_t[i] = (float)cos(angle);
  sin_t[i] = (float)sin(angle);
}

// Initialises the fp32 accumulator of the open slot of sequences seq0 + blockIdx.x from the
// stored cache row `slot`.
template <typename T>
__global__ void open_acc_from_cache_kernel(CacheView cache, float* open_acc, int r, int W,
                                           int seq0, int slot) {
  const int b = seq0 + blockIdx.x;
  const T* row = static_cast<const T*>(cache.base) + cache_row(cache, b, slot) * W;
  for (int i = threadIdx.x; i < r; i += blockDim.x)
    open_acc[(long long)b * r + i] = Elem<T>::to_float(row[i]);
}

}  // namespace mtla
