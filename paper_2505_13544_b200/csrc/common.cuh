// Shared device helpers for the MTLA kernels: element conversion, 128-bit loads, reductions.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

namespace mtla {

typedef __nv_bfloat16 bf16;

constexpr int kWarp = 32;

__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
__host__ __device__ inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Where the compressed cache keeps slot `slot` of sequence `b`, as a row index into `base`
// (rows of r + d_R elements).  Contiguous storage: [max_batch][max_slots] rows.  Paged storage
// (page_table != nullptr): a pool of 64-slot pages and, per sequence, the pages it holds.
struct CacheView {
  void* base;
  const int* page_table;   // [max_batch][max_pages] or nullptr
  int max_pages;
  int max_slots;
};
__device__ inline long long cache_row(const CacheView& v, int b, int slot) {
  if (v.page_table)
    return (long long)v.page_table[(long long)b * v.max_pages + (slot >> 6)] * 64 + (slot & 63);
  return (long long)b * v.max_slots + slot;
}

template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int kVec = 4;  // elements per 16-byte access
  __device__ static float to_float(float v) { return v; }
  __device__ static float from_float(float v) { return v; }
};
template <> struct Elem<bf16> {
  static constexpr int kVec = 8;
  __device__ static float to_float(bf16 v) { return __bfloat162float(v); }
  __device__ static bf16 from_float(float v) { return __float2bfloat16_rn(v); }
};

// Loads 16 bytes of T from a 16-byte aligned address and widens to fp32.
__device__ inline void load_vec(const float* p, float (&out)[4]) {
  float4 v = *reinterpret_cast<const float4*>(p);
  out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
__device__ inline void load_vec(const bf16* p, float (&out)[8]) {
  uint4 v = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    out[2 * i] = __uint_as_float(w[i] << 16);
    out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

// Narrows fp32 to T (round to nearest even) and stores 16 bytes to an aligned address.
__device__ inline void store_vec(float* p, const float (&in)[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(in[0], in[1], in[2], in[3]);
}
__device__ inline void store_vec(bf16* p, const float (&in)[8]) {
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(in[2 * i], in[2 * i + 1]);
    w[i] = *reinterpret_cast<uint32_t*>(&h);
  }
  *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ inline float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ inline float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Block-wide sum for blockDim.x a multiple of 32 (<= 1024); `scratch` holds >= 33 floats.
// Every thread receives the total.  Contains two __syncthreads().
__device__ inline float block_sum(float v, float* scratch) {
  v = warp_sum(v);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  if (warp == 0) {
    float t = lane < (int)(blockDim.x >> 5) ? scratch[lane] : 0.f;
    t = warp_sum(t);
    if (lane == 0) scratch[32] = t;
  }
  __syncthreads();
  return scratch[32];
}

// Launches `kernel`; with `dependent` it may start its prologue while the previous kernel on
// the stream is still running (programmatic dependent launch: the kernel itself waits, with
// griddepcontrol.wait, before it touches that kernel's data).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                          cudaStream_t st, bool dependent, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = dependent ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

}  // namespace mtla
