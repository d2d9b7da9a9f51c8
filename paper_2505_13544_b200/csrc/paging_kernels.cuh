// Device side of the paged cache and of per-sequence positions: small kernels that apply what
// the host-side page pool has decided (table entries, page copies, beam reordering) and that
// move whole sequences between the paged pool and a contiguous [sequence][slot] layout.
// Their operands travel as kernel parameters, so a call may return before the work has run
// without any host buffer having to stay alive.  The three kernels of a beam-search step are
// programmatic dependent launches (see sm100_ptx.cuh): they start while their predecessor drains
// and wait before they touch memory.
#pragma once

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mtla {

constexpr int kScatterOps = 448;
struct IntScatter {          // dst[idx[i]] = val[i]
  int n;
  int idx[kScatterOps];
  int val[kScatterOps];
};
__global__ void int_scatter_kernel(int* dst, IntScatter ops) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();
  if (i < ops.n) dst[ops.idx[i]] = ops.val[i];
}

constexpr int kPageCopyOps = 256;
struct PageCopies {          // rows [0, rows[i]) of page src[i] -> page dst[i]
  int n;
  int src[kPageCopyOps], dst[kPageCopyOps], rows[kPageCopyOps];
};
// One CTA per copy; row_bytes is a multiple of 16.
__global__ void __launch_bounds__(256) page_copy_kernel(char* pool, long long page_bytes, int row_bytes,
                                                         PageCopies ops) {
  const int i = blockIdx.x;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();
  const uint4* s = reinterpret_cast<const uint4*>(pool + ops.src[i] * page_bytes);
  uint4* d = reinterpret_cast<uint4*>(pool + ops.dst[i] * page_bytes);
  const int n = ops.rows[i] * (row_bytes / 16);
  for (int v = threadIdx.x; v < n; v += 256) d[v] = s[v];
}

constexpr int kBeamChunk = 768;
struct BeamParents {         // new sequence first + i continues old sequence parent[i]
  int n, first;
  int parent[kBeamChunk];
};
struct BeamArgs {
  const int* tokens_old;  int* tokens_new;       // [max_batch] tokens consumed per sequence
  const int* table_old;   int* table_new;        // [max_batch][max_pages]
  const float* acc_old;   float* acc_new;        // [max_batch][r] fp32 state of the open slot
  int max_pages, r, stride;
};
// Beam reordering on the device: one CTA per new sequence copies its parent's position, page
// table row (the pages in use) and open-slot accumulator from the old buffers to the new ones.
__global__ void __launch_bounds__(128) beam_gather_kernel(BeamArgs a, BeamParents p) {
  const int b = p.first + blockIdx.x, src = p.parent[blockIdx.x];
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();
  const int tokens = a.tokens_old[src];
  if (threadIdx.x == 0) a.tokens_new[b] = tokens;
  const int pages = ceil_div(ceil_div(tokens, a.stride), 64);
  for (int k = threadIdx.x; k < pages; k += 128)
    a.table_new[(long long)b * a.max_pages + k] = a.table_old[(long long)src * a.max_pages + k];
  for (int i = threadIdx.x; i < a.r; i += 128)
    a.acc_new[(long long)b * a.r + i] = a.acc_old[(long long)src * a.r + i];
}

// Copies slots [0, n_slots) of sequences seq0 + blockIdx.y between the cache and a contiguous
// buffer flat[blockIdx.y][n_slots][W]; grid.x covers the 64-slot pages.  row_bytes = W * elem
// is a multiple of 16, so are all addresses involved.
__global__ void __launch_bounds__(256) cache_rows_copy_kernel(CacheView view, int seq0, int n_slots,
                                                               int row_bytes, char* flat, int to_cache) {
  const int b = blockIdx.y, slot0 = blockIdx.x * 64;
  const int rows = min(64, n_slots - slot0);
  char* in_cache = static_cast<char*>(view.base) + cache_row(view, seq0 + b, slot0) * row_bytes;
  char* in_flat = flat + ((long long)b * n_slots + slot0) * row_bytes;
  const uint4* s = reinterpret_cast<const uint4*>(to_cache ? in_flat : in_cache);
  uint4* d = reinterpret_cast<uint4*>(to_cache ? in_cache : in_flat);
  const int n = rows * (row_bytes / 16);
  for (int v = threadIdx.x; v < n; v += 256) d[v] = s[v];
}

}  // namespace mtla
