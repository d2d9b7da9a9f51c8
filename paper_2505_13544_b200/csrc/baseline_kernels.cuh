// Kernels of the comparison attentions (Section 3: multi-head, multi-query and grouped-query
// attention with a key-value cache) that are not shared with the MTLA path.  The cache keeps,
// per sequence and key/value head ("group"), one row [value | key] of 2 d_h elements per
// token; with that layout the decode attention over the compressed cache serves unchanged:
// a (sequence, group) pair is one of its "sequences", the group's query heads are its heads,
// the row is its latent (values = the first d_h columns of the result) and the query is
// [0 | q_h / sqrt(d_h)], so the score is q_h . k and the zero half meets the value columns.
#pragma once

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mtla {

struct KvPostArgs {
  const float* p1;        // [B][(n_h + 2 g) d_h] fused projection of this step: [ q | k | v ]
  const float* rope_cos;  // [max_tokens][d_h / 2]
  const float* rope_sin;
  bf16* cache;            // [B * g][max_tokens][2 d_h]: value, then rotated key
  bf16* qt;               // [B * g][n_h / g][2 d_h]: zeros (set at create), then the rotated query
  int n_heads, n_groups, head_dim, max_tokens;
  int tokens;             // tokens consumed so far = position of this token
  float q_scale;          // log2(e) / sqrt(d_h)
};

// One CTA of 256 threads per sequence: standard rotary embedding of the queries and keys at the
// token's position, the key/value append, and the attention kernel's query rows.
__global__ void __launch_bounds__(256) kv_post_kernel(KvPostArgs a) {
  const int b = blockIdx.x, tid = threadIdx.x;
  const int dh = a.head_dim, half = dh / 2, W = 2 * dh, per = a.n_heads / a.n_groups;
  const int off_k = a.n_heads * dh, off_v = off_k + a.n_groups * dh;
  const float* row = a.p1 + (long long)b * (off_v + a.n_groups * dh);
  const float* cs = a.rope_cos + (long long)a.tokens * half;
  const float* sn = a.rope_sin + (long long)a.tokens * half;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();
  for (int i = tid; i < a.n_heads * half; i += 256) {
    const int h = i / half, k = i % half;
    const float x0 = row[h * dh + 2 * k], x1 = row[h * dh + 2 * k + 1];
    bf16* q = a.qt + (((long long)b * a.n_groups + h / per) * per + h % per) * W + dh;
    *reinterpret_cast<__nv_bfloat162*>(q + 2 * k) = __floats2bfloat162_rn(
        (x0 * cs[k] - x1 * sn[k]) * a.q_scale, (x0 * sn[k] + x1 * cs[k]) * a.q_scale);
  }
  for (int i = tid; i < a.n_groups * half; i += 256) {
    const int g = i / half, k = i % half;
    const float x0 = row[off_k + g * dh + 2 * k], x1 = row[off_k + g * dh + 2 * k + 1];
    bf16* dst = a.cache + (((long long)b * a.n_groups + g) * a.max_tokens + a.tokens) * W;
    *reinterpret_cast<__nv_bfloat162*>(dst + dh + 2 * k) =
        __floats2bfloat162_rn(x0 * cs[k] - x1 * sn[k], x0 * sn[k] + x1 * cs[k]);
    *reinterpret_cast<__nv_bfloat162*>(dst + 2 * k) =
        __floats2bfloat162_rn(row[off_v + g * dh + 2 * k], row[off_v + g * dh + 2 * k + 1]);
  }
}

// Gathers the value halves of the attention output, o [B * g][2][n_h / g][2 d_h] (bf16 hi
// halves, then remainders), into rows [B][2][n_h d_h] for the output projection.
__global__ void __launch_bounds__(256) kv_heads_gather_kernel(const bf16* o, bf16* out, int n_heads,
                                                              int n_groups, int head_dim) {
  const int b = blockIdx.x, dh = head_dim, W = 2 * dh, per = n_heads / n_groups;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();
  for (int i = threadIdx.x; i < 2 * n_heads * (dh / 2); i += 256) {
    const int c2 = i % (dh / 2), h = (i / (dh / 2)) % n_heads, part = i / (n_heads * (dh / 2));
    const bf16* src = o + ((((long long)b * n_groups + h / per) * 2 + part) * per + h % per) * W + 2 * c2;
    bf16* dst = out + ((long long)b * 2 + part) * n_heads * dh + h * dh + 2 * c2;
    *reinterpret_cast<__nv_bfloat162*>(dst) = *reinterpret_cast<const __nv_bfloat162*>(src);
  }
}

}  // namespace mtla
