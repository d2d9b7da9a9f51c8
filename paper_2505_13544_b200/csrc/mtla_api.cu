// C ABI of the MTLA library (see include/mtla.h): validation, arena carving, weight
// repacking and the launch sequences of the decode step and the prefill.
#include "mtla.h"

#include <cuda.h>
#include <math.h>
#include <algorithm>
#include <new>
#include <stdlib.h>
#include <string.h>
#include <utility>
#include <vector>

#include "common.cuh"
#include "decode_attn_tc.cuh"
#include "decode_kernels.cuh"
#include "gemm_fma.cuh"
#include "gemm_tc.cuh"
#include "prefill_attn_tc.cuh"
#include "prefill_attn_tc2.cuh"
#include "prefill_kernels.cuh"
#include "setup_kernels.cuh"
#include "paging_kernels.cuh"
#include "baseline_kernels.cuh"
#include "selftest_kernels.cuh"
#include "page_pool.h"

using namespace mtla;

namespace {

// The split workspaces are sized for persistent grids of up to kPlanSms CTAs (B200: 148 SMs);
// the grids themselves follow the device's SM count read at create, capped at this bound.
constexpr int kPlanSms = 148;
constexpr int kTargetCtas = 2 * kPlanSms;   // CUDA-core attention: two CTAs per SM
constexpr int kMinSlotsPerSplit = 64;
constexpr int kFusedCombineMaxParts = 8;   // more parts per sequence: the combine gets its own launch
constexpr int kPrefillBn = 128;             // prompt rows per CTA in the prefill's output projection
                                            // (its hi / lo halves are stacked: N = 256)
constexpr int kPrefillBnWide = 256;         // and in its input and key / value projections
// Layers whose pre-multiplied matrices W_Q W_K^T and W_V W_O (Eq. 12, taken literally) stay below
// this size each keep them for the decode step: two launches fewer per step, which is what counts
// where the whole layer lives in L2.  Larger layers keep the two-step form (the pre-multiplied
// matrices have n_h r / (n_h d_h) times the bytes of the factors, and decode streams the weights).
constexpr size_t kFoldMaxBytes = 8u << 20;
constexpr int kGemmSlots = 2 * kPlanSms;   // CTAs a split-K GEMM may spread one product over


// Rows of the activation-side TMA box (the MMA's N) for a decode batch of B sequences.
int act_box_rows(int B) {
  for (int bn = 16; bn < 256; bn *= 2)
    if (B <= bn) return bn;
  return 256;
}

struct ArenaPlan {
  size_t wcat_t, w_k, w_kv_t, w_o_t;
  size_t wcat_dec_t, w_vo_t;   // folded decode weights (Dims::fold): [q~ hi | q~ lo | q^R | c | k^R | u][d],
                               // [d][hi | lo of n_h r]
  size_t fold_tmp;             // [r][d] fp32: one head's product before it is split (create only)
  size_t gamma, beta, hyp_c_w, hyp_c_b, hyp_pe_w, hyp_pe_b, gate_pe, rope_cos, rope_sin;
  size_t gate_s, gate_t, gate_tmp;
  size_t cache, open_acc, err_flag;
  size_t page_table, seq_tokens;   // paged handles: two buffers each (beam reordering flips them)
  size_t p1, q16, qt, o_part, ml_part, o, v, x_stage, y_stage, gemm_part, gemm_tickets, attn_tickets;
  size_t pf_p1, pf_qcat, pf_cprime, pf_kr, pf_kv, pf_attn;
  size_t scratch_begin;   // everything from here on is per-call scratch (nothing survives a call)
  size_t total;
};

struct Dims {
  int d, nh, dh, r, dr, dw, s, W, ntot, max_slots, max_units;
  int n_pages, max_pages;   // paged handles: pool size, pages per sequence; 0 otherwise
  size_t elem;
  ProjLayout proj;
  // Decode with pre-multiplied weights: the input projection emits the absorbed query directly
  // (columns [0, n_h r) of proj_dec, its off_q), the attention output goes through W_V W_O at once.
  bool fold;
  ProjLayout proj_dec;
  int ntot_dec;
};

bool normalise(const mtla_config* in, const mtla_paging* pg, mtla_config* out, Dims* dm) {
  if (!in) return false;
  mtla_config c = *in;
  if (c.hyper_dim == 0) c.hyper_dim = c.latent_rank / 4;
  if (c.ln_eps == 0.f) c.ln_eps = 1e-5f;
  if (c.rope_theta == 0.f) c.rope_theta = 10000.f;
  if (c.d_model <= 0 || c.d_model % 8) return false;
  if (c.n_heads < 1 || c.n_heads > 32) return false;
  if (c.head_dim != 64 && c.head_dim != 128) return false;
  if (c.latent_rank < 64 || c.latent_rank > 512 || c.latent_rank % 64) return false;
  if (c.rope_dim != 32 && c.rope_dim != 64) return false;
  if (c.stride < 1) return false;
  if (c.hyper_dim < 1 || c.hyper_dim > 256) return false;
  if (c.max_batch < 1 || c.max_tokens < 1 || c.max_prefill_tokens < 0) return false;
  if (c.dtype != MTLA_DTYPE_FP32 && c.dtype != MTLA_DTYPE_BF16) return false;
  if (c.kernel_path != MTLA_PATH_AUTO && c.kernel_path != MTLA_PATH_CUDA_CORE) return false;
  if (!(c.ln_eps > 0.f) || !(c.rope_theta > 0.f)) return false;
  if ((long long)c.max_batch * c.max_tokens > (1ll << 31)) return false;
  *out = c;
  dm->d = c.d_model; dm->nh = c.n_heads; dm->dh = c.head_dim; dm->r = c.latent_rank;
  dm->dr = c.rope_dim; dm->dw = c.hyper_dim; dm->s = c.stride;
  dm->W = dm->r + dm->dr;
  dm->elem = c.dtype == MTLA_DTYPE_BF16 ? 2 : 4;
  dm->proj.off_q = 0;
  dm->proj.off_qr = dm->nh * dm->dh;
  dm->proj.off_c = dm->proj.off_qr + dm->nh * dm->dr;
  dm->proj.off_kr = dm->proj.off_c + dm->r;
  dm->proj.width = dm->proj.off_kr + dm->dr;
  // bf16 layers with a gate (s > 1) carry the folded Linear(c_i) as 2 d_w more output columns.
  dm->proj.off_u = -1;
  if (c.dtype == MTLA_DTYPE_BF16 && c.stride > 1) {
    dm->proj.off_u = dm->proj.width;
    // Rows of the projection output are read 16 bytes at a time by the CUDA-core GEMMs: an odd
    // d_w would leave every other row misaligned, so the row is padded (zero weight rows).
    dm->proj.width = (dm->proj.width + 2 * dm->dw + 3) / 4 * 4;
  }
  dm->ntot = dm->proj.width;
  dm->fold = c.dtype == MTLA_DTYPE_BF16 && c.latent_rank % 128 == 0 && c.kernel_path != MTLA_PATH_CUDA_CORE &&
             (size_t)dm->nh * dm->r * dm->d * 2 <= kFoldMaxBytes;
  dm->proj_dec = dm->proj;
  dm->ntot_dec = dm->ntot;
  if (dm->fold) {
    // The query block widens from d_h to r columns per head, twice: the pre-multiplied weight is
    // kept as bf16 [hi | lo] row blocks and the two partial queries are added after the product.
    const int shift = 2 * dm->nh * dm->r - dm->nh * dm->dh;
    dm->proj_dec.off_qr += shift;
    dm->proj_dec.off_c += shift;
    dm->proj_dec.off_kr += shift;
    if (dm->proj_dec.off_u >= 0) dm->proj_dec.off_u += shift;
    dm->proj_dec.width += shift;
    dm->ntot_dec = dm->proj_dec.width;
  }
  dm->max_slots = ceil_div(c.max_tokens, c.stride);
  dm->max_units = kTargetCtas + c.max_batch;
  dm->n_pages = dm->max_pages = 0;
  if (pg) {
    if (pg->page_slots != kPageSlots || pg->n_pages < 0) return false;
    dm->max_pages = ceil_div(dm->max_slots, kPageSlots);
    const long long full = (long long)c.max_batch * dm->max_pages;
    if (full > (1ll << 30) || pg->n_pages > full) return false;
    dm->n_pages = pg->n_pages ? pg->n_pages : (int)full;
  }
  return true;
}

void plan_arena(const mtla_config& c, const Dims& dm, ArenaPlan* p) {
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off = align_up(off + bytes, 1024);
    return at;
  };
  const size_t e = dm.elem, B = c.max_batch;
  const size_t hd = (size_t)dm.nh * dm.dh;
  p->wcat_t = take((size_t)dm.ntot * dm.d * e);
  p->w_k = take((size_t)dm.r * hd * e);
  p->w_kv_t = take(2 * hd * dm.r * e);
  p->w_o_t = take((size_t)dm.d * hd * e);
  p->wcat_dec_t = take(dm.fold ? (size_t)dm.ntot_dec * dm.d * e : 0);
  p->w_vo_t = take(dm.fold ? (size_t)dm.d * 2 * dm.nh * dm.r * e : 0);
  p->fold_tmp = take(dm.fold ? (size_t)dm.r * dm.d * 4 : 0);
  p->gamma = take(dm.r * 4);
  p->beta = take(dm.r * 4);
  p->hyp_c_w = take((size_t)dm.r * dm.dw * 4);
  p->hyp_c_b = take(dm.dw * 4);
  p->hyp_pe_w = take((size_t)dm.r * dm.dw * 4);
  p->hyp_pe_b = take(dm.dw * 4);
  p->gate_pe = take((size_t)dm.max_slots * dm.dw * 4);
  p->gate_s = take(dm.dw * 4);
  p->gate_t = take(dm.dw * 4);
  p->gate_tmp = take(dm.proj.off_u >= 0 ? ((size_t)dm.dw * dm.r + (size_t)dm.dw * dm.d) * 4 : 0);
  p->rope_cos = take((size_t)c.max_tokens * (dm.dr / 2) * 4);
  p->rope_sin = take((size_t)c.max_tokens * (dm.dr / 2) * 4);
  const size_t paged = dm.n_pages > 0;
  p->cache = take(paged ? (size_t)dm.n_pages * kPageSlots * dm.W * e : B * dm.max_slots * dm.W * e);
  p->open_acc = take((1 + paged) * B * dm.r * 4);
  p->page_table = take(paged * 2 * B * dm.max_pages * sizeof(int));
  p->seq_tokens = take(paged * 2 * B * sizeof(int));
  p->err_flag = take(16);
  p->scratch_begin = off;
  p->p1 = take(B * (size_t)max(dm.ntot, dm.ntot_dec) * 4);
  p->q16 = take(B * 2 * hd * 2);
  p->qt = take(B * dm.nh * dm.W * 4);
  p->o_part = take((size_t)dm.max_units * dm.nh * dm.r * 4);
  p->ml_part = take((size_t)dm.max_units * dm.nh * 2 * 4);
  p->o = take(B * dm.nh * dm.r * 4);
  p->v = take(B * hd * 4);
  p->x_stage = take(B * dm.d * e);
  p->y_stage = take(B * dm.d * e);
  // Split-K workspace of the tensor-core GEMMs: at most kGemmSlots CTAs hold a partial tile.
  p->gemm_part = take(c.dtype == MTLA_DTYPE_BF16
                          ? (size_t)kGemmSlots * gtc::kBM * act_box_rows(c.max_batch) * 4 : 0);
  p->gemm_tickets = take((size_t)kGemmSlots * 4 * sizeof(int));
  p->attn_tickets = take(B * sizeof(int));
  const size_t rows = B * (size_t)c.max_prefill_tokens;
  p->pf_p1 = take(rows * dm.ntot * 4);
  p->pf_qcat = take(rows * dm.nh * (dm.dh + dm.dr) * 4);
  p->pf_cprime = take(rows * dm.r * e);
  p->pf_kr = take(rows * dm.dr * 4);
  p->pf_kv = take(rows * 2 * hd * 4);
  p->pf_attn = take(rows * hd * 4);
  p->total = off;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// The GPU that owns `arena` and its SM count (capped at the planning bound).
int arena_device(const void* arena, int* device, int* sm_count) {
  cudaPointerAttributes attr;
  if (cudaPointerGetAttributes(&attr, arena) != cudaSuccess) return MTLA_ERR_CUDA;
  if (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged) return MTLA_ERR_INVALID_ARG;
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, attr.device) != cudaSuccess || sms < 1)
    return MTLA_ERR_CUDA;
  *device = attr.device;
  *sm_count = sms < kPlanSms ? sms : kPlanSms;
  return MTLA_OK;
}

}  // namespace

// Split workspace of mtla_decode_step_static: lives in every GPU that loads the library, for
// the life of the process.  In host code this name is only a handle for cudaGetSymbolAddress;
// the device address is looked up once per device and kept here.
static __device__ __align__(256) unsigned char g_static_scratch[MTLA_STATIC_SCRATCH_BYTES];
constexpr int kMaxDevices = 64;
static unsigned char* g_static_scratch_addr[kMaxDevices];

struct mtla_handle {
  mtla_config cfg;
  Dims dm;
  ArenaPlan plan;
  char* arena;
  // Offsets at or beyond plan.scratch_begin resolve against this base instead of the arena
  // (already shifted by -scratch_begin).  The layers of a stack share one scratch region:
  // their calls are ordered on one stream and nothing in it survives a call.
  char* scratch;
  int tokens;   // tokens consumed per sequence (paged handles: the longest sequence's)
  int batch;    // 0 while the cache is empty and no batch has been fixed
  // Paged handles (mtla_create_paged): per-sequence positions and the page pool.  The device
  // keeps its own copy of the positions, advanced by the decode step's kernels; host-side
  // changes (prefill, import, reset) mark it stale and the next call re-sends them.
  PagePool* pool;
  std::vector<int> seq_tokens;
  int last_gang = 0;      // gang size of the latest tensor-core decode attention launch (0: none yet)
  bool tokens_stale;
  // Comparison layers (mtla_baseline_create): multi-head / grouped-query / multi-query attention
  // over a key-value cache; g key/value heads per sequence, each a plane of the cache.
  bool is_baseline;
  int bl_groups;
  int64_t launches;
  int train_B, train_T;   // shape of the prefill whose workspace mtla_train_backward may read (0: none)
  int device;     // ordinal of the GPU that owns the arena
  int sm_count;   // its SM count, capped at the bound the workspaces are sized for
  bool attn_smem_ready, pf_smem_ready;
  // Tensor-core decode attention (bf16, r a multiple of 128): TMA view of the cache.
  bool use_tc;
  CUtensorMap cache_map, q_map;
  // Tensor-core projections (bf16): weight panels as 128-row boxes, serving as the MMA's M side
  // in the decode step and as its N side in the prefill; decode activations as act_bn-row boxes.
  CUtensorMap map_wcat, map_wk, map_wkvt, map_wvt, map_wot;
  CUtensorMap map_wcat_dec, map_wvo;   // folded decode weights
  CUtensorMap map_q16, map_o16, map_v16;
  int act_bn;               // box rows the three activation maps were encoded with (0: none yet)
  unsigned long long gemm_attr_mask;  // kernel instances whose shared-memory limit has been raised
  // Optional timing of the decode step's kernels: MTLA_DECODE_STAGES + 1 events per profiled step.
  std::vector<cudaEvent_t> prof_events;
  int prof_used;
  bool prof_attention_only;   // record only the two events around the attention kernel

  template <typename P> P* at(size_t off) const {
    return reinterpret_cast<P*>((scratch && off >= plan.scratch_begin ? scratch : arena) + off);
  }
  bool paged() const { return pool != nullptr; }
  int buf() const { return pool ? pool->current_buffer() : 0; }
  int* d_page_table(int which) const {
    return at<int>(plan.page_table) + (size_t)which * cfg.max_batch * dm.max_pages;
  }
  int* d_seq_tokens(int which) const { return at<int>(plan.seq_tokens) + (size_t)which * cfg.max_batch; }
  float* d_open_acc(int which) const {
    return at<float>(plan.open_acc) + (size_t)which * cfg.max_batch * dm.r;
  }
  // The cache as the kernels address it, under the current page table.
  CacheView cache_view() const {
    CacheView v;
    v.base = at<void>(plan.cache);
    v.page_table = pool ? d_page_table(buf()) : nullptr;
    v.max_pages = dm.max_pages;
    v.max_slots = dm.max_slots;
    return v;
  }
  int seq_len(int b) const { return pool ? seq_tokens[b] : tokens; }
  int planes_per_seq() const { return is_baseline ? bl_groups : 1; }
};

namespace {

#define MTLA_CUDA(call)                       \
  do {                                        \
    if ((call) != cudaSuccess) return MTLA_ERR_CUDA; \
  } while (0)

template <typename T>
int launch_transpose(mtla_handle* h, const void* src, void* dst, int K, int N, int ld_src,
                     int ld_dst, cudaStream_t st) {
  dim3 grid(ceil_div(N, 32), ceil_div(K, 32)), block(32, 8);
  transpose_kernel<T><<<grid, block, 0, st>>>(static_cast<const T*>(src), static_cast<T*>(dst),
                                              K, N, ld_src, ld_dst);
  h->launches++;
  return cudaGetLastError() == cudaSuccess ? MTLA_OK : MTLA_ERR_CUDA;
}

template <typename T>
int launch_widen(mtla_handle* h, const void* src, float* dst, long long n, cudaStream_t st) {
  widen_kernel<T><<<(unsigned)((n + 255) / 256), 256, 0, st>>>(static_cast<const T*>(src), dst, n);
  h->launches++;
  return cudaGetLastError() == cudaSuccess ? MTLA_OK : MTLA_ERR_CUDA;
}

template <typename TA, typename TB, typename TOut>
int gemm(mtla_handle* h, const void* a, const void* bt, void* c, int m, int n, int k, int lda,
         int ldb, int ldc, float alpha, int batches, long long za, long long zb, long long zc,
         cudaStream_t st, bool dependent = false) {
  GemmArgs g;
  g.a = a; g.bt = bt; g.c = c; g.m = m; g.n = n; g.k = k;
  g.lda = lda; g.ldb = ldb; g.ldc = ldc; g.za = za; g.zb = zb; g.zc = zc; g.alpha = alpha;
  h->launches++;
  return launch_gemm_nt_fma<TA, TB, TOut>(g, batches, st, dependent) == cudaSuccess ? MTLA_OK : MTLA_ERR_CUDA;
}

#define MTLA_TRY(expr)            \
  do {                            \
    const int rc_ = (expr);       \
    if (rc_ != MTLA_OK) return rc_; \
  } while (0)

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn cached = nullptr;
  if (cached) return cached;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  cached = reinterpret_cast<EncodeTiledFn>(fn);
  return cached;
}

// TMA views for the decode attention: the bf16 cache [max_batch][max_slots][r + d_R] in boxes of
// 64 slots x 64 columns (128 bytes, the swizzle span), and the absorbed queries
// [max_batch][n_h][r + d_R] in boxes of `heads_padded` heads x 64 columns; zero fill outside.
int make_cache_map(mtla_handle* h) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return MTLA_ERR_CUDA;
  const Dims& dm = h->dm;
  // Paged: the planes are the pool's 64-slot pages instead of the sequences' row ranges.
  // Comparison layers: one plane per (sequence, key/value head).
  const cuuint64_t plane_rows = h->paged() ? kPageSlots : dm.max_slots;
  const cuuint64_t planes = h->paged() ? dm.n_pages : (cuuint64_t)h->cfg.max_batch * h->planes_per_seq();
  const cuuint64_t dims[3] = {(cuuint64_t)dm.W, plane_rows, planes};
  const cuuint64_t strides[2] = {(cuuint64_t)dm.W * 2, plane_rows * dm.W * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)tc::kTile, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult rc = fn(
      &h->cache_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, h->at<void>(h->plan.cache), dims, strides,
      box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (rc != CUDA_SUCCESS) return MTLA_ERR_CUDA;
  const cuuint64_t qdims[3] = {(cuuint64_t)dm.W, (cuuint64_t)dm.nh,
                               (cuuint64_t)h->cfg.max_batch * h->planes_per_seq()};
  const cuuint64_t qstrides[2] = {(cuuint64_t)dm.W * 2, (cuuint64_t)dm.nh * dm.W * 2};
  const cuuint32_t qbox[3] = {64, (cuuint32_t)(dm.nh <= 16 ? 16 : 32), 1};
  rc = fn(&h->q_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, h->at<void>(h->plan.qt), qdims, qstrides,
          qbox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? MTLA_OK : MTLA_ERR_CUDA;
}

// TMA view of a row-major bf16 matrix [rows][cols] with leading dimension ld (elements):
// boxes of box_rows rows x 64 columns (128 bytes, the swizzle span), zero fill outside.
int make_map_2d(CUtensorMap* map, const void* ptr, long long rows, long long cols, long long ld,
                int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return MTLA_ERR_CUDA;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims,
                         strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? MTLA_OK : MTLA_ERR_CUDA;
}

// TMA view of bf16 data as [n2][n1][cols] with element strides ld1 / ld2 between rows / planes:
// boxes of box_rows rows x 64 columns, 128-byte swizzle, zero fill outside.
int make_map_3d(CUtensorMap* map, const void* ptr, long long cols, long long n1, long long n2,
                long long ld1, long long ld2, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return MTLA_ERR_CUDA;
  const cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)n1, (cuuint64_t)n2};
  const cuuint64_t strides[2] = {(cuuint64_t)ld1 * 2, (cuuint64_t)ld2 * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims,
                         strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? MTLA_OK : MTLA_ERR_CUDA;
}

template <int BN, int STAGES, typename OutT, bool HILO, bool EXTRAS = false, bool QSPLIT = false>
int launch_gemm_tc_inst(mtla_handle* h, int inst, const CUtensorMap& ma, const CUtensorMap& mb,
                        const GemmTcArgs& g, dim3 grid, cudaStream_t st, bool dependent) {
  constexpr int smem = gtc::smem_bytes(HILO ? 2 * BN : BN, STAGES);
  if (!(h->gemm_attr_mask & (1ull << inst))) {
    MTLA_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<BN, STAGES, OutT, HILO, EXTRAS, QSPLIT>,
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    h->gemm_attr_mask |= 1ull << inst;
  }
  MTLA_CUDA(launch_kernel(gemm_tc_kernel<BN, STAGES, OutT, HILO, EXTRAS, QSPLIT>, grid, dim3(192), smem, st,
                          dependent, ma, mb, g));
  h->launches++;
  return MTLA_OK;
}

// D[z][i][j] = alpha * sum_k A[z][i][k] B[z][j][k] on the tensor cores (see gemm_tc.cuh).
// `bn` is the row count of map_b's box.  With allow_split the reduction is spread over
// several CTAs when the tile count alone would leave most SMs idle.
template <typename OutT>
int gemm_tc(mtla_handle* h, const CUtensorMap& ma, const CUtensorMap& mb, GemmTcArgs g, int bn,
            int batches, bool allow_split, cudaStream_t st, bool dependent = false) {
  const int m_tiles = ceil_div(g.m, gtc::kBM);
  g.m_tiles = m_tiles;
  g.n_tiles = ceil_div(g.n, bn);
  const long long tiles = (long long)m_tiles * g.n_tiles * batches;
  const int kb_total = ceil_div(g.k, gtc::kBK);
  // Stacked hi / lo halves double the B tile: one CTA per SM then, two otherwise.
  const bool hilo = g.b_lo_col > 0 && bn <= 128 && sizeof(OutT) == 2;
  const int slots = (hilo && bn == 128) || bn == 256 ? h->sm_count : 2 * h->sm_count;
  int n_split = 1;
  // The partials are summed by the last CTA of a tile alone: at most four splits keep that short
  // (eight where a product has so few tiles that four splits would still leave it on <= 32 CTAs).
  if (allow_split && tiles < slots)
    n_split = max(1, min(min(kb_total / 4, (int)(slots / tiles)), tiles <= 8 ? 8 : 4));
  // Short reductions with few activation rows (the paper's layer: K = 512, B <= 64): one CTA per
  // tile with the whole K range in flight at once beats splitting it, which costs a trip of the
  // partials through global memory on top of two load round trips.
  const bool shallow = allow_split && kb_total <= 8 && bn <= 64;
  if (shallow) n_split = 1;
  g.kb_per_split = ceil_div(kb_total, n_split);
  g.n_split = ceil_div(kb_total, g.kb_per_split);
  g.partial = h->at<float>(h->plan.gemm_part);
  g.tickets = h->at<int>(h->plan.gemm_tickets);
  g.error_word = h->at<int>(h->plan.err_flag);
  const size_t osz = sizeof(OutT);
  g.vec_ok = (reinterpret_cast<uintptr_t>(g.c) % 16 == 0) && (g.c_sm * osz % 16 == 0) &&
             (g.c_sz * osz % 16 == 0);
  if ((long long)m_tiles * g.n_tiles * g.n_split > 0x7fffffffll) return MTLA_ERR_UNSUPPORTED_SHAPE;
  g.vec4_ok = g.c_sm == 1 && g.m % 4 == 0 && reinterpret_cast<uintptr_t>(g.c) % 16 == 0 &&
              g.c_sn * osz % 16 == 0 && g.c_sz * osz % 16 == 0 && g.c_lo_off * osz % 8 == 0;
  if (g.bias || g.residual || g.relu) {
    // The unsplit epilogue applies the extras one element at a time; the split reduction takes
    // four consecutive output features at once where bias and residual allow 16-byte reads.
    g.vec_ok = 0;
    g.vec4_ok = g.vec4_ok && (!g.bias || reinterpret_cast<uintptr_t>(g.bias) % 16 == 0) &&
                (!g.residual || (g.r_sm == 1 && g.r_sn % 4 == 0 &&
                                 reinterpret_cast<uintptr_t>(g.residual) % 16 == 0));
  }
  dim3 grid(m_tiles * g.n_tiles * g.n_split, 1, batches);
  constexpr int o = sizeof(OutT) == 4 ? 0 : 1;
  if (g.bias || g.residual || g.relu) {
    // The feed-forward products of a decoder layer: the instantiations with the fused
    // bias / ReLU / residual epilogue (single bf16 activations, no hi / lo halves).
    if (hilo || g.b_lo_col > 0) return MTLA_ERR_UNSUPPORTED_SHAPE;
    switch (bn) {
      case 16: return launch_gemm_tc_inst<16, 4, OutT, false, true>(h, 21 + o, ma, mb, g, grid, st, dependent);
      case 32: return launch_gemm_tc_inst<32, 4, OutT, false, true>(h, 23 + o, ma, mb, g, grid, st, dependent);
      case 64: return launch_gemm_tc_inst<64, 4, OutT, false, true>(h, 25 + o, ma, mb, g, grid, st, dependent);
      case 128: return launch_gemm_tc_inst<128, 3, OutT, false, true>(h, 27 + o, ma, mb, g, grid, st, dependent);
      case 256: return launch_gemm_tc_inst<256, 4, OutT, false, true>(h, 29 + o, ma, mb, g, grid, st, dependent);
      default: return MTLA_ERR_UNSUPPORTED_SHAPE;
    }
  }
  if (shallow && (sizeof(OutT) == 4 || hilo)) {
    if constexpr (sizeof(OutT) == 4) {
      switch (bn) {
        case 16: return launch_gemm_tc_inst<16, 8, OutT, false>(h, 14, ma, mb, g, grid, st, dependent);
        case 32: return launch_gemm_tc_inst<32, 8, OutT, false>(h, 15, ma, mb, g, grid, st, dependent);
        default: return launch_gemm_tc_inst<64, 8, OutT, false>(h, 16, ma, mb, g, grid, st, dependent);
      }
    } else {
      switch (bn) {
        case 16: return launch_gemm_tc_inst<16, 8, OutT, true>(h, 17, ma, mb, g, grid, st, dependent);
        case 32: return launch_gemm_tc_inst<32, 8, OutT, true>(h, 18, ma, mb, g, grid, st, dependent);
        default: return launch_gemm_tc_inst<64, 6, OutT, true>(h, 19, ma, mb, g, grid, st, dependent);
      }
    }
  }
  if constexpr (sizeof(OutT) == 2) {
    if (hilo) {
      switch (bn) {
        case 16: return launch_gemm_tc_inst<16, 4, OutT, true>(h, 10, ma, mb, g, grid, st, dependent);
        case 32: return launch_gemm_tc_inst<32, 4, OutT, true>(h, 11, ma, mb, g, grid, st, dependent);
        case 64: return launch_gemm_tc_inst<64, 3, OutT, true>(h, 12, ma, mb, g, grid, st, dependent);
        case 128:
          // Prefill (many tiles, no split): two stages, so that two CTAs share an SM.
          if (!allow_split)
            return launch_gemm_tc_inst<128, 2, OutT, true>(h, 34, ma, mb, g, grid, st, dependent);
          return launch_gemm_tc_inst<128, 4, OutT, true>(h, 13, ma, mb, g, grid, st, dependent);
        default: return MTLA_ERR_UNSUPPORTED_SHAPE;
      }
    }
  }
  switch (bn) {
    case 16: return launch_gemm_tc_inst<16, 4, OutT, false>(h, 0 + o, ma, mb, g, grid, st, dependent);
    case 32: return launch_gemm_tc_inst<32, 4, OutT, false>(h, 2 + o, ma, mb, g, grid, st, dependent);
    case 64: return launch_gemm_tc_inst<64, 4, OutT, false>(h, 4 + o, ma, mb, g, grid, st, dependent);
    case 128: return launch_gemm_tc_inst<128, 3, OutT, false>(h, 6 + o, ma, mb, g, grid, st, dependent);
    case 256:
      // Prefill (many tiles, no split): two stages leave room for two CTAs per SM, whose epilogues
      // and main loops overlap; the weight-streaming decode products want the deeper ring.
      if constexpr (sizeof(OutT) == 4) {
        if (!allow_split && g.q_out)
          return launch_gemm_tc_inst<256, 2, OutT, false, false, true>(h, 33, ma, mb, g, grid, st, dependent);
      }
      if (g.q_out) return MTLA_ERR_UNSUPPORTED_SHAPE;
      if (!allow_split)
        return launch_gemm_tc_inst<256, 2, OutT, false>(h, 31 + o, ma, mb, g, grid, st, dependent);
      return launch_gemm_tc_inst<256, 4, OutT, false>(h, 8 + o, ma, mb, g, grid, st, dependent);
    default: return MTLA_ERR_UNSUPPORTED_SHAPE;
  }
}

GemmTcArgs gemm_tc_args(void* c, long long c_sm, long long c_sn, int m, int n, int k, float alpha) {
  GemmTcArgs g;
  memset(&g, 0, sizeof(g));
  g.c = c; g.c_sm = c_sm; g.c_sn = c_sn; g.m = m; g.n = n; g.k = k; g.alpha = alpha;
  g.b_k_wrap = 1 << 30;
  return g;
}

template <int NHP, bool RAGGED>
int launch_attn_tc_rp(mtla_handle* h, const AttnTcArgs& a, dim3 grid, cudaStream_t st, bool dependent) {
  constexpr int kSmem = tc::Layout<RAGGED>::kSmemBytes;
#define MTLA_TC_CASE(RP)                                                                       \
  case RP:                                                                                     \
    if (!h->attn_smem_ready) {                                                                 \
      /* The kernel re-allocates registers between warpgroups; its launch-time pool must */    \
      /* cover the budget, or the increase inside the kernel would never be granted.     */    \
      cudaFuncAttributes fa;                                                                   \
      MTLA_CUDA(cudaFuncGetAttributes(&fa, decode_attn_tc_kernel<NHP, RP, RAGGED>));                   \
      if (fa.numRegs * tc::kThreads < (tc::kThreads - tc::kSoftmaxThreads) * tc::kRegsIssuer + \
                                          tc::kSoftmaxThreads * tc::kRegsSoftmax)              \
        return MTLA_ERR_CUDA;                                                                  \
      MTLA_CUDA(cudaFuncSetAttribute(decode_attn_tc_kernel<NHP, RP, RAGGED>,                           \
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem)); \
    }                                                                                          \
    MTLA_CUDA(launch_kernel(decode_attn_tc_kernel<NHP, RP, RAGGED>, grid, dim3(tc::kThreads),          \
                            kSmem, st, dependent, h->cache_map, h->q_map, a));                 \
    break;
  switch (a.r / 128) {
    MTLA_TC_CASE(1)
    MTLA_TC_CASE(2)
    MTLA_TC_CASE(3)
    MTLA_TC_CASE(4)
    default: return MTLA_ERR_UNSUPPORTED_SHAPE;
  }
#undef MTLA_TC_CASE
  h->attn_smem_ready = true;
  h->launches++;
  return MTLA_OK;
}

template <typename T>
int create_impl(mtla_handle* h, const mtla_weights* w, cudaStream_t st) {
  const Dims& dm = h->dm;
  const ArenaPlan& p = h->plan;
  const int hd = dm.nh * dm.dh;
  T* wcat = h->at<T>(p.wcat_t);
  // Fused input projection, stored [out][in]: rows [ q | q^R | c | k^R ].
  MTLA_TRY(launch_transpose<T>(h, w->w_q, wcat + (size_t)dm.proj.off_q * dm.d, dm.d, hd, hd, dm.d, st));
  MTLA_TRY(launch_transpose<T>(h, w->w_qr, wcat + (size_t)dm.proj.off_qr * dm.d, dm.d,
                               dm.nh * dm.dr, dm.nh * dm.dr, dm.d, st));
  MTLA_TRY(launch_transpose<T>(h, w->w_r, wcat + (size_t)dm.proj.off_c * dm.d, dm.d, dm.r, dm.r, dm.d, st));
  MTLA_TRY(launch_transpose<T>(h, w->w_kr, wcat + (size_t)dm.proj.off_kr * dm.d, dm.d, dm.dr, dm.dr, dm.d, st));
  // W_K as given serves the query absorption ([r][n_h*d_h]: out = r, in = d_h per head).
  MTLA_CUDA(cudaMemcpyAsync(h->at<T>(p.w_k), w->w_k, (size_t)dm.r * hd * sizeof(T),
                            cudaMemcpyDeviceToDevice, st));
  // [W_K^T ; W_V^T] stored [out][in] = [2*n_h*d_h][r] for the up-projections.
  MTLA_TRY(launch_transpose<T>(h, w->w_k, h->at<T>(p.w_kv_t), dm.r, hd, hd, dm.r, st));
  MTLA_TRY(launch_transpose<T>(h, w->w_v, h->at<T>(p.w_kv_t) + (size_t)hd * dm.r, dm.r, hd, hd, dm.r, st));
  MTLA_TRY(launch_transpose<T>(h, w->w_o, h->at<T>(p.w_o_t), hd, dm.d, dm.d, hd, st));
  MTLA_TRY(launch_widen<T>(h, w->ln_gamma, h->at<float>(p.gamma), dm.r, st));
  MTLA_TRY(launch_widen<T>(h, w->ln_beta, h->at<float>(p.beta), dm.r, st));
  MTLA_TRY(launch_widen<T>(h, w->hyp_c_w, h->at<float>(p.hyp_c_w), (long long)dm.r * dm.dw, st));
  MTLA_TRY(launch_widen<T>(h, w->hyp_c_b, h->at<float>(p.hyp_c_b), dm.dw, st));
  MTLA_TRY(launch_widen<T>(h, w->hyp_pe_w, h->at<float>(p.hyp_pe_w), (long long)dm.r * dm.dw, st));
  MTLA_TRY(launch_widen<T>(h, w->hyp_pe_b, h->at<float>(p.hyp_pe_b), dm.dw, st));
  if (dm.proj.off_u >= 0) {
    // W_g^T = (gamma .* A)^T W_r^T as two bf16 row blocks behind the projection's other rows.
    float* ga = h->at<float>(p.gate_tmp);
    float* wg = ga + (size_t)dm.dw * dm.r;
    gate_fold_scale_kernel<<<ceil_div(dm.r * dm.dw, 256), 256, 0, st>>>(
        h->at<float>(p.hyp_c_w), h->at<float>(p.gamma), ga, dm.r, dm.dw);
    h->launches++;
    MTLA_CUDA(cudaGetLastError());
    MTLA_TRY((gemm<float, T, float>(h, ga, w->w_r, wg, dm.dw, dm.d, dm.r, dm.r, dm.r, dm.d, 1.f, 1,
                                    0, 0, 0, st)));
    const int pad_rows = dm.ntot - (dm.proj.off_u + 2 * dm.dw);
    if (pad_rows > 0)
      MTLA_CUDA(cudaMemsetAsync(h->at<bf16>(p.wcat_t) + (size_t)(dm.ntot - pad_rows) * dm.d, 0,
                                (size_t)pad_rows * dm.d * sizeof(bf16), st));
    const long long n_wg = (long long)dm.dw * dm.d;
    gate_fold_pack_kernel<<<(unsigned)((n_wg + 255) / 256), 256, 0, st>>>(
        wg, h->at<bf16>(p.wcat_t) + (size_t)dm.proj.off_u * dm.d, dm.dw, dm.d);
    h->launches++;
    MTLA_CUDA(cudaGetLastError());
    gate_fold_vectors_kernel<<<ceil_div(dm.dw, 128), 128, 0, st>>>(
        h->at<float>(p.hyp_c_w), h->at<float>(p.hyp_c_b), h->at<float>(p.gamma),
        h->at<float>(p.beta), h->at<float>(p.gate_s), h->at<float>(p.gate_t), dm.r, dm.dw);
    h->launches++;
    MTLA_CUDA(cudaGetLastError());
  }
  gate_pe_table_kernel<<<dm.max_slots, 256, 0, st>>>(h->at<float>(p.hyp_pe_w), h->at<float>(p.hyp_pe_b),
                                                     h->at<float>(p.gate_pe), dm.r, dm.dw);
  h->launches++;
  MTLA_CUDA(cudaGetLastError());
  const long long n_rope = (long long)h->cfg.max_tokens * (dm.dr / 2);
  rope_table_kernel<<<(unsigned)((n_rope + 255) / 256), 256, 0, st>>>(
      h->at<float>(p.rope_cos), h->at<float>(p.rope_sin), h->cfg.max_tokens, dm.dr / 2,
      (double)h->cfg.rope_theta);
  h->launches++;
  MTLA_CUDA(cudaGetLastError());
  MTLA_CUDA(cudaMemsetAsync(h->at<char>(p.err_flag), 0, 16, st));
  // Unused cache rows must hold finite values: the tensor-core kernel multiplies rows
  // beyond the valid range by a zero probability.
  const size_t cache_rows = h->paged() ? (size_t)dm.n_pages * kPageSlots
                                       : (size_t)h->cfg.max_batch * dm.max_slots;
  MTLA_CUDA(cudaMemsetAsync(h->at<char>(p.cache), 0, cache_rows * dm.W * dm.elem, st));
  MTLA_CUDA(cudaMemsetAsync(h->at<char>(p.gemm_tickets), 0, (size_t)kGemmSlots * 4 * sizeof(int), st));
  MTLA_CUDA(cudaMemsetAsync(h->at<char>(p.attn_tickets), 0, (size_t)h->cfg.max_batch * sizeof(int), st));
  if (h->use_tc) {
    MTLA_TRY(make_cache_map(h));
    MTLA_TRY(make_map_2d(&h->map_wcat, h->at<void>(p.wcat_t), dm.ntot, dm.d, dm.d, gtc::kBM));
    MTLA_TRY(make_map_2d(&h->map_wk, h->at<void>(p.w_k), dm.r, hd, hd, gtc::kBM));
    MTLA_TRY(make_map_2d(&h->map_wkvt, h->at<void>(p.w_kv_t), 2 * hd, dm.r, dm.r, gtc::kBM));
    MTLA_TRY(make_map_2d(&h->map_wvt, h->at<T>(p.w_kv_t) + (size_t)hd * dm.r, hd, dm.r, dm.r, gtc::kBM));
    MTLA_TRY(make_map_2d(&h->map_wot, h->at<void>(p.w_o_t), dm.d, hd, hd, gtc::kBM));
    if (dm.fold) {
      // Eq. 12's products, per head, from the weights as given, accumulated in fp32 and kept as
      // bf16 [hi | lo] halves (about 16 mantissa bits, as the activations of the unfolded path):
      //   rows h r + j of the decode projection = scale * W_{K,h}[j] . W_{Q,h}^T      [r][d], hi block
      //   rows n_h r + h r + j                  = its rounding remainder                      lo block
      //   columns h r + j of W_VO^T             = W_{O,h}^T . W_{V,h}[j]              [d][r], hi half
      //   columns n_h r + h r + j               = its rounding remainder                      lo half
      bf16* wdec = h->at<bf16>(p.wcat_dec_t);
      bf16* wvo = h->at<bf16>(p.w_vo_t);
      float* tmp = h->at<float>(p.fold_tmp);
      const T* wk_in = static_cast<const T*>(w->w_k);
      const T* wq_in = static_cast<const T*>(w->w_q);
      const T* wv_in = static_cast<const T*>(w->w_v);
      const long long onr = (long long)dm.nh * dm.r;
      const float q_scale = (float)(1.4426950408889634 / sqrt((double)dm.dh));
      const unsigned pack_blocks = (unsigned)(((long long)dm.r * dm.d + 255) / 256);
      for (int hh = 0; hh < dm.nh; ++hh) {
        MTLA_TRY((gemm<T, T, float>(h, wk_in + (size_t)hh * dm.dh, wq_in + (size_t)hh * dm.dh, tmp, dm.r,
                                    dm.d, dm.dh, hd, hd, dm.d, q_scale, 1, 0, 0, 0, st)));
        split_hi_lo_kernel<<<pack_blocks, 256, 0, st>>>(tmp, wdec + (size_t)hh * dm.r * dm.d,
                                                        wdec + (size_t)(onr + hh * dm.r) * dm.d, dm.r,
                                                        dm.d, dm.d, dm.d);
        h->launches++;
        MTLA_CUDA(cudaGetLastError());
        MTLA_TRY((gemm<T, T, float>(h, h->at<T>(p.w_o_t) + (size_t)hh * dm.dh, wv_in + (size_t)hh * dm.dh,
                                    tmp, dm.d, dm.r, dm.dh, hd, hd, dm.r, 1.f, 1, 0, 0, 0, st)));
        split_hi_lo_kernel<<<pack_blocks, 256, 0, st>>>(tmp, wvo + (size_t)hh * dm.r,
                                                        wvo + (size_t)(onr + hh * dm.r), dm.d, dm.r,
                                                        dm.r, 2 * onr);
        h->launches++;
        MTLA_CUDA(cudaGetLastError());
      }
      // Everything behind the query block is the same in both projections.
      MTLA_CUDA(cudaMemcpyAsync(wdec + (size_t)2 * onr * dm.d,
                                h->at<bf16>(p.wcat_t) + (size_t)dm.proj.off_qr * dm.d,
                                (size_t)(dm.ntot - dm.proj.off_qr) * dm.d * sizeof(bf16),
                                cudaMemcpyDeviceToDevice, st));
      MTLA_TRY(make_map_2d(&h->map_wcat_dec, wdec, dm.ntot_dec, dm.d, dm.d, gtc::kBM));
      MTLA_TRY(make_map_2d(&h->map_wvo, h->at<void>(p.w_vo_t), dm.d, 2 * onr, 2 * onr, gtc::kBM));
    }
  }
  return MTLA_OK;
}

// (Re-)encodes the TMA views of the decode step's bf16 intermediates for a batch of B rows.
int ensure_activation_maps(mtla_handle* h, int B) {
  const int bn = act_box_rows(B);
  if (h->act_bn == bn) return MTLA_OK;
  const Dims& dm = h->dm;
  const ArenaPlan& p = h->plan;
  const int hd = dm.nh * dm.dh, mb = h->cfg.max_batch;
  // Each intermediate row holds the bf16 [hi | lo] halves of an fp32 activation.
  const long long onr = (long long)dm.nh * dm.r;
  MTLA_TRY(make_map_2d(&h->map_q16, h->at<void>(p.q16), mb, 2 * hd, 2 * hd, bn));
  MTLA_TRY(make_map_2d(&h->map_o16, h->at<void>(p.o), mb, 2 * onr, 2 * onr, bn));
  MTLA_TRY(make_map_2d(&h->map_v16, h->at<void>(p.v), mb, 2 * hd, 2 * hd, bn));
  h->act_bn = bn;
  return MTLA_OK;
}

template <typename T, typename TQ, int NH>
int launch_attn_fma_rpt(mtla_handle* h, const AttnArgs& a, int B, cudaStream_t st, bool dependent) {
  const size_t smem = attn_fma_smem_bytes(NH, a.r, a.dr);
  dim3 grid(a.n_split, B);
  if (a.r <= 256) {
    if (!h->attn_smem_ready)
      MTLA_CUDA(cudaFuncSetAttribute(decode_attn_fma_kernel<T, TQ, NH, 1>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    MTLA_CUDA(launch_kernel(decode_attn_fma_kernel<T, TQ, NH, 1>, grid, dim3(256), smem, st, dependent, a));
  } else {
    if (!h->attn_smem_ready)
      MTLA_CUDA(cudaFuncSetAttribute(decode_attn_fma_kernel<T, TQ, NH, 2>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    MTLA_CUDA(launch_kernel(decode_attn_fma_kernel<T, TQ, NH, 2>, grid, dim3(256), smem, st, dependent, a));
  }
  h->attn_smem_ready = true;
  h->launches++;
  MTLA_CUDA(cudaGetLastError());
  return MTLA_OK;
}

template <typename T, typename TQ>
int launch_attn_fma(mtla_handle* h, const AttnArgs& a, int B, cudaStream_t st, bool dependent) {
  if (a.n_heads <= 4) return launch_attn_fma_rpt<T, TQ, 4>(h, a, B, st, dependent);
  if (a.n_heads <= 8) return launch_attn_fma_rpt<T, TQ, 8>(h, a, B, st, dependent);
  if (a.n_heads <= 16) return launch_attn_fma_rpt<T, TQ, 16>(h, a, B, st, dependent);
  return launch_attn_fma_rpt<T, TQ, 32>(h, a, B, st, dependent);
}

// Gang size for the paged attention launch (beam search).  The kernel needs the batch to be
// blocks of g consecutive sequences with equal token counts; gangs pay when the sequences of a
// block share their pages, which is taken from the first page: g is the length of the first run
// of sequences that have the same first page and length, and at least half of the blocks must
// share theirs (an utterance shorter than a page does not: its only page is the one each beam
// writes).  The gang is the largest divisor of g that leaves at most a tenth of the SMs without
// a whole gang.  1: no gangs.
int beam_gang(const mtla_handle* h, int B) {
  auto same_len = [&](int a, int b) { return h->seq_tokens[a] == h->seq_tokens[b]; };
  auto same_page = [&](int a, int b) {
    return h->pool->pages_held(a) > 0 && h->pool->pages_held(b) > 0 &&
           h->pool->row(a)[0] == h->pool->row(b)[0];
  };
  int b0 = 0;
  while (b0 + 1 < B && !(same_len(b0, b0 + 1) && same_page(b0, b0 + 1))) ++b0;
  if (b0 + 1 >= B) return 1;
  int g = 1;
  while (b0 + g < B && same_len(b0, b0 + g) && same_page(b0, b0 + g)) ++g;
  if (B % g || b0 % g) return 1;
  int sharing = 0;
  for (int k = 0; k < B; k += g) {
    bool shares = true;
    for (int j = 1; j < g; ++j) {
      if (!same_len(k, k + j)) return 1;
      shares = shares && same_page(k, k + j);
    }
    sharing += shares ? 1 : 0;
  }
  if (2 * sharing < B / g) return 1;
  for (int gang = g; gang >= 2; --gang)
    if (g % gang == 0 && gang <= h->sm_count && (h->sm_count % gang) * 10 <= h->sm_count) return gang;
  return 1;
}

// Where the attention kernels keep their split partials; nullptr members select the arena.
struct AttnScratch {
  float* o_part;
  float* ml_part;
  int* tickets;
};

// Records the event that closes stage `stage - 1` / opens stage `stage` of a profiled step.
int prof_mark(mtla_handle* h, bool prof, int stage, cudaStream_t st) {
  if (!prof) return MTLA_OK;
  if (h->prof_attention_only && stage != MTLA_STAGE_ATTENTION && stage != MTLA_STAGE_ATTENTION + 1)
    return MTLA_OK;
  MTLA_CUDA(cudaEventRecord(h->prof_events[h->prof_used + stage], st));
  return MTLA_OK;
}

// The decode step (Section 4.1): a1 fused projection, a2-a5 post kernel, a6 absorption,
// a7 split-K attention + combine, a8 value and output projections.
template <typename T>
int decode_impl(mtla_handle* h, const void* x, int B, void* y, cudaStream_t st,
                const AttnScratch* scratch = nullptr) {
  const Dims& dm = h->dm;
  const ArenaPlan& p = h->plan;
  const int hd = dm.nh * dm.dh;
  // Lock-step batches: every sequence is at token i0.  Paged handles: each at its own, kept on
  // the device; n_slots is then the longest sequence's count after this step.
  const int i0 = h->tokens;
  int n_slots = i0 / dm.s + 1;
  long long ragged_tiles = 0;
  if (h->paged()) {
    n_slots = 0;
    for (int b = 0; b < B; ++b) {
      const int nb = h->seq_tokens[b] / dm.s + 1;
      n_slots = max(n_slots, nb);
      ragged_tiles += ceil_div(nb, tc::kTile);
    }
  }
  const int buf = h->buf();
  int* seq_tokens = h->paged() ? h->d_seq_tokens(buf) : nullptr;

  const bool prof = h->prof_used + MTLA_DECODE_STAGES + 1 <= (int)h->prof_events.size();
  MTLA_TRY(prof_mark(h, prof, 0, st));
  const int bn = act_box_rows(B);
  // On the tensor-core path every kernel is a programmatic dependent launch: its prologue
  // overlaps the tail of its predecessor in the stream (the previous step's or layer's last
  // kernel for the first one), and it waits before it touches any data.  Not while events sit
  // between the kernels.
  const bool pdl = h->use_tc && !(prof && !h->prof_attention_only);
  const bool pdl_cc = !h->use_tc && !(prof && !h->prof_attention_only);   // the same on the CUDA-core path
  if (h->use_tc) {
    // a1 on the tensor cores: weights stream through the MMA's M side, the batch sits in N.
    MTLA_TRY(ensure_activation_maps(h, B));
    CUtensorMap map_x;
    MTLA_TRY(make_map_2d(&map_x, x, B, dm.d, dm.d, bn));
    // With pre-multiplied weights the projection's query block is the absorbed query itself.
    const int n_out = dm.fold ? dm.ntot_dec : dm.ntot;
    MTLA_TRY(gemm_tc<float>(h, dm.fold ? h->map_wcat_dec : h->map_wcat, map_x,
                            gemm_tc_args(h->at<float>(p.p1), 1, n_out, n_out, B, dm.d, 1.f), bn, 1, true, st,
                            pdl));
  } else {
    MTLA_TRY((gemm<T, T, float>(h, x, h->at<T>(p.wcat_t), h->at<float>(p.p1), B, dm.ntot, dm.d,
                                dm.d, dm.d, dm.ntot, 1.f, 1, 0, 0, 0, st, pdl_cc)));
  }

  MTLA_TRY(prof_mark(h, prof, 1, st));
  PostArgs pa;
  pa.p1 = h->at<float>(p.p1);
  pa.proj = dm.fold ? dm.proj_dec : dm.proj;
  pa.absorbed = dm.fold ? 1 : 0;
  pa.gamma = h->at<float>(p.gamma);
  pa.beta = h->at<float>(p.beta);
  pa.hyp_c_w = h->at<float>(p.hyp_c_w);
  pa.hyp_c_b = h->at<float>(p.hyp_c_b);
  pa.gate_pe = h->at<float>(p.gate_pe);
  pa.gate_s = h->at<float>(p.gate_s);
  pa.gate_t = h->at<float>(p.gate_t);
  pa.rope_cos = h->at<float>(p.rope_cos);
  pa.rope_sin = h->at<float>(p.rope_sin);
  pa.open_acc = h->d_open_acc(buf);
  pa.cache = h->cache_view();
  pa.seq_tokens = seq_tokens;
  pa.qt = h->at<void>(p.qt);
  pa.q16 = h->use_tc ? h->at<bf16>(p.q16) : nullptr;
  pa.n_heads = dm.nh; pa.head_dim = dm.dh; pa.r = dm.r; pa.dr = dm.dr; pa.dw = dm.dw;
  pa.tokens = i0; pa.stride = dm.s;
  pa.use_gate = dm.s > 1;
  pa.ln_eps = h->cfg.ln_eps;
  pa.q_scale = (float)(1.4426950408889634 / sqrt((double)dm.dh));
  // Layers whose gate needs no matrix (folded form, or s = 1) take the latency-oriented kernel.
  const bool post_fast = dm.proj.off_u >= 0 || !pa.use_gate;
  if (h->use_tc) {
    if (post_fast)
      MTLA_CUDA(launch_kernel(decode_post_fast_kernel<T, bf16>, dim3(B), dim3(256), 0, st, pdl, pa));
    else
      MTLA_CUDA(launch_kernel(decode_post_kernel<T, bf16>, dim3(B), dim3(256), 0, st, pdl, pa));
  } else {
    if (post_fast) MTLA_CUDA(launch_kernel(decode_post_fast_kernel<T, float>, dim3(B), dim3(256), 0, st, pdl_cc, pa));
    else MTLA_CUDA(launch_kernel(decode_post_kernel<T, float>, dim3(B), dim3(256), 0, st, pdl_cc, pa));
    MTLA_CUDA(cudaGetLastError());
  }
  h->launches++;

  MTLA_TRY(prof_mark(h, prof, 2, st));
  // a6: q~_h = scale * q_h W_{K,h}^T, one z-slice per head, straight from the fp32 projection
  // (bf16 output where the tensor-core attention consumes it).
  if (dm.fold) {
    // nothing to do: the post kernel has written the absorbed query
  } else if (h->use_tc) {
    GemmTcArgs g = gemm_tc_args(h->at<bf16>(p.qt), 1, (long long)dm.nh * dm.W, dm.r, B, dm.dh, pa.q_scale);
    g.c_sz = dm.W; g.a_col_z = dm.dh; g.b_col_z = dm.dh; g.b_lo_col = hd;
    MTLA_TRY(gemm_tc<bf16>(h, h->map_wk, h->map_q16, g, bn, dm.nh, true, st, pdl));
  } else
    MTLA_TRY((gemm<float, T, float>(h, h->at<float>(p.p1) + dm.proj.off_q, h->at<T>(p.w_k),
                                    h->at<float>(p.qt), B, dm.r, dm.dh, dm.ntot, hd, dm.nh * dm.W,
                                    pa.q_scale, dm.nh, dm.dh, dm.dh, dm.W, st, pdl_cc)));

  MTLA_TRY(prof_mark(h, prof, 3, st));
  AttnArgs aa;
  aa.qt = h->at<void>(p.qt);
  aa.cache = h->cache_view();
  aa.o_part = scratch ? scratch->o_part : h->at<float>(p.o_part);
  aa.ml_part = scratch ? scratch->ml_part : h->at<float>(p.ml_part);
  aa.seq_tokens = seq_tokens;
  aa.n_heads = dm.nh; aa.r = dm.r; aa.dr = dm.dr; aa.stride = dm.s;
  aa.n_slots = n_slots;
  if (h->use_tc) {
    // One persistent CTA per SM; the step's 64-slot tiles are dealt out in equal shares, and
    // the kernel combines the partials itself (no separate combine launch).
    AttnTcArgs ta;
    ta.o_part = aa.o_part; ta.ml_part = aa.ml_part;
    ta.o16 = h->at<bf16>(p.o);
    ta.tickets = scratch ? scratch->tickets : h->at<int>(p.attn_tickets);
    ta.error_word = h->at<int>(p.err_flag);
    ta.n_heads = dm.nh; ta.r = dm.r; ta.dr = dm.dr; ta.n_slots = n_slots; ta.batch = B;
    ta.tiles_per_seq = ceil_div(n_slots, tc::kTile);
    ta.seq_tokens = seq_tokens;
    ta.page_table = h->paged() ? h->d_page_table(buf) : nullptr;
    ta.max_pages = dm.max_pages; ta.stride = dm.s;
    long long total = h->paged() ? ragged_tiles : (long long)B * ta.tiles_per_seq;
    // Beam search: consecutive sequences of equal length that start on the same page (the beams
    // of one utterance) are walked by a gang of CTAs side by side (AttnTcArgs::gang).
    const int gang = h->paged() ? beam_gang(h, B) : 1;
    ta.n_list = B / gang;
    h->last_gang = gang;
    if (gang > 1) total = ragged_tiles / gang;              // tiles of the gangs' first sequences
    const int grid_slots = h->sm_count / gang;              // whole gangs that fit the SMs
    const int vctas = (int)(total < grid_slots ? total : grid_slots);
    const int grid = vctas * gang;
    aa.n_split = 0;
    // A lock-step batch whose sequences are each spread over many CTAs hands the combine to a
    // launch of its own, one CTA per (head, sequence), instead of one CTA per sequence.
    const bool split_combine = !h->paged() && grid / B + 2 > kFusedCombineMaxParts;
    ta.fused_combine = !split_combine;
    ta.attn_grid = grid;
    const bool attn_pdl = pdl && !prof;     // the attention kernel is bracketed by events when timed
    if (h->paged()) {
      // (gang member, virtual CTA): members of a gang are neighbours in launch order.
      if (dm.nh <= 16) MTLA_TRY((launch_attn_tc_rp<16, true>(h, ta, dim3(gang, vctas), st, attn_pdl)));
      else MTLA_TRY((launch_attn_tc_rp<32, true>(h, ta, dim3(gang, vctas), st, attn_pdl)));
    } else {
      if (dm.nh <= 16) MTLA_TRY((launch_attn_tc_rp<16, false>(h, ta, dim3(grid), st, attn_pdl)));
      else MTLA_TRY((launch_attn_tc_rp<32, false>(h, ta, dim3(grid), st, attn_pdl)));
    }
    MTLA_TRY(prof_mark(h, prof, 4, st));
    if (split_combine) {
      MTLA_CUDA(launch_kernel(decode_combine_parts_kernel, dim3(dm.nh, B), dim3(128), 0, st, pdl && !prof, ta));
      h->launches++;
    }
  } else {
    int want = ceil_div(2 * h->sm_count, B);
    int n_split = min(want, ceil_div(n_slots, kMinSlotsPerSplit));
    if (n_split < 1) n_split = 1;
    aa.slots_per_split = ceil_div(ceil_div(n_slots, n_split), kAttnFmaTile) * kAttnFmaTile;
    aa.n_split = ceil_div(n_slots, aa.slots_per_split);
    MTLA_TRY((launch_attn_fma<T, float>(h, aa, B, st, pdl_cc && !prof)));
    MTLA_TRY(prof_mark(h, prof, 4, st));
  }

  CombineArgs ca;
  ca.o_part = aa.o_part; ca.ml_part = aa.ml_part; ca.o = h->at<void>(p.o);
  ca.n_heads = dm.nh; ca.r = dm.r; ca.n_split = aa.n_split;
  if (!h->use_tc) {
    MTLA_CUDA(launch_kernel(decode_combine_kernel<float>, dim3(dm.nh, B), dim3(128), 0, st, pdl_cc && !prof, ca));
    h->launches++;
    MTLA_CUDA(cudaGetLastError());
  }

  // a8: v_h = o_h W_{V,h} per head, then y = concat_h(v_h) W_O.
  MTLA_TRY(prof_mark(h, prof, 5, st));
  if (dm.fold) {
    // y = o (W_V W_O) over K = 2 n_h r: the weight's [hi | lo] halves along K meet the same
    // columns of o, itself [hi | lo] halves stacked in the B tile.
    MTLA_TRY(prof_mark(h, prof, 6, st));
    GemmTcArgs g = gemm_tc_args(y, 1, dm.d, dm.d, B, 2 * dm.nh * dm.r, 1.f);
    g.b_lo_col = dm.nh * dm.r;
    g.b_k_wrap = dm.nh * dm.r / gtc::kBK;
    MTLA_TRY(gemm_tc<bf16>(h, h->map_wvo, h->map_o16, g, bn, 1, true, st, pdl && !prof));
  } else if (h->use_tc) {
    GemmTcArgs g = gemm_tc_args(h->at<bf16>(p.v), 1, 2 * hd, dm.dh, B, dm.r, 1.f);
    g.c_sz = dm.dh; g.a_row_z = dm.dh; g.b_col_z = dm.r; g.b_lo_col = dm.nh * dm.r; g.c_lo_off = hd;
    MTLA_TRY(gemm_tc<bf16>(h, h->map_wvt, h->map_o16, g, bn, dm.nh, true, st, pdl && !prof));
    MTLA_TRY(prof_mark(h, prof, 6, st));
    g = gemm_tc_args(y, 1, dm.d, dm.d, B, hd, 1.f);
    g.b_lo_col = hd;
    MTLA_TRY(gemm_tc<bf16>(h, h->map_wot, h->map_v16, g, bn, 1, true, st, pdl));
  } else {
    MTLA_TRY((gemm<float, T, float>(h, h->at<float>(p.o), h->at<T>(p.w_kv_t) + (size_t)hd * dm.r,
                                    h->at<float>(p.v), B, dm.dh, dm.r, dm.nh * dm.r, dm.r, hd, 1.f,
                                    dm.nh, dm.r, (long long)dm.dh * dm.r, dm.dh, st, pdl_cc && !prof)));
    MTLA_TRY(prof_mark(h, prof, 6, st));
    MTLA_TRY((gemm<float, T, T>(h, h->at<float>(p.v), h->at<T>(p.w_o_t), y, B, dm.d, hd, hd, hd,
                                dm.d, 1.f, 1, 0, 0, 0, st, pdl_cc)));
  }
  MTLA_TRY(prof_mark(h, prof, 7, st));
  if (prof) h->prof_used += MTLA_DECODE_STAGES + 1;
  return MTLA_OK;
}

template <typename T>
int prefill_impl(mtla_handle* h, const void* x, int seq0, int B, int T_len, void* y, cudaStream_t st) {
  const Dims& dm = h->dm;
  const ArenaPlan& p = h->plan;
  const int hd = dm.nh * dm.dh;
  const int rows = B * T_len;
  const float q_scale = (float)(1.4426950408889634 / sqrt((double)dm.dh));
  const bool post_fast = (dm.proj.off_u >= 0 || dm.s == 1) && dm.s <= kPostFastMaxStride;
  const bool q_split = h->use_tc && post_fast && hd % gtc::kBM == 0;

  if (h->use_tc) {
    // Weights on the MMA's M side, 128 prompt rows per CTA on its N side: neighbouring CTAs
    // share an activation panel while the (small) weight matrix stays in L2.
    CUtensorMap map_x;
    MTLA_TRY(make_map_2d(&map_x, x, rows, dm.d, dm.d, kPrefillBnWide));
    GemmTcArgs g1 = gemm_tc_args(h->at<float>(p.pf_p1), 1, dm.ntot, dm.ntot, rows, dm.d, 1.f);
    if (q_split) {
      // The query block leaves the projection kernel scaled and rounded, in the attention's
      // layout; the post kernel then has only the latent, the gate and the RoPE vectors to do.
      g1.q_out = h->at<bf16>(p.pf_qcat);
      g1.q_rows = hd;
      g1.q_dh_shift = dm.dh == 64 ? 6 : 7;
      g1.q_dq = dm.dh + dm.dr;
      g1.q_sn = (long long)dm.nh * (dm.dh + dm.dr);
      g1.q_scale = q_scale;
    }
    MTLA_TRY(gemm_tc<float>(h, h->map_wcat, map_x, g1, kPrefillBnWide, 1, false, st));
  } else {
    MTLA_TRY((gemm<T, T, float>(h, x, h->at<T>(p.wcat_t), h->at<float>(p.pf_p1), rows, dm.ntot,
                                dm.d, dm.d, dm.d, dm.ntot, 1.f, 1, 0, 0, 0, st)));
  }
  PrefillPostArgs pa;
  pa.p1 = h->at<float>(p.pf_p1);
  pa.proj = dm.proj;
  pa.gamma = h->at<float>(p.gamma);
  pa.beta = h->at<float>(p.beta);
  pa.hyp_c_w = h->at<float>(p.hyp_c_w);
  pa.hyp_c_b = h->at<float>(p.hyp_c_b);
  pa.gate_pe = h->at<float>(p.gate_pe);
  pa.gate_s = h->at<float>(p.gate_s);
  pa.gate_t = h->at<float>(p.gate_t);
  pa.rope_cos = h->at<float>(p.rope_cos);
  pa.rope_sin = h->at<float>(p.rope_sin);
  pa.open_acc = h->d_open_acc(h->buf());
  pa.cache = h->cache_view();
  pa.seq0 = seq0;
  pa.qcat = h->at<void>(p.pf_qcat);
  pa.cprime = h->at<void>(p.pf_cprime);
  pa.kr = h->at<void>(p.pf_kr);
  pa.n_heads = dm.nh; pa.head_dim = dm.dh; pa.r = dm.r; pa.dr = dm.dr; pa.dw = dm.dw;
  pa.stride = dm.s; pa.T = T_len; pa.max_slots = dm.max_slots;
  pa.use_gate = dm.s > 1;
  pa.ln_eps = h->cfg.ln_eps;
  pa.q_scale = q_scale;
  pa.batch = B;
  const dim3 post_grid(ceil_div(T_len, dm.s), B);
  // The fast kernel takes one warp per (chunk, sequence), eight to a CTA.
  const dim3 fast_grid((unsigned)(((long long)ceil_div(T_len, dm.s) * B + 7) / 8));
  pa.q_done = q_split ? 1 : 0;
  if (h->use_tc) {
    if (post_fast) prefill_post_fast_kernel<T, bf16><<<fast_grid, 256, 0, st>>>(pa);
    else prefill_post_kernel<T, bf16><<<post_grid, 256, 0, st>>>(pa);
  } else {
    if (post_fast) prefill_post_fast_kernel<T, float><<<fast_grid, 256, 0, st>>>(pa);
    else prefill_post_kernel<T, float><<<post_grid, 256, 0, st>>>(pa);
  }
  h->launches++;
  MTLA_CUDA(cudaGetLastError());
  if (!y) return MTLA_OK;

  // Eq. 9-10 on the running-state sequence: keys and values of every column.
  if (h->use_tc) {
    CUtensorMap map_c;
    MTLA_TRY(make_map_2d(&map_c, h->at<void>(p.pf_cprime), rows, dm.r, dm.r, kPrefillBnWide));
    // Keys and values as bf16, followed by their rounding remainders: rows of 4 n_h d_h.
    GemmTcArgs gkv = gemm_tc_args(h->at<bf16>(p.pf_kv), 1, 4 * hd, 2 * hd, rows, dm.r, 1.f);
    gkv.c_lo_off = 2 * hd;
    MTLA_TRY(gemm_tc<bf16>(h, h->map_wkvt, map_c, gkv, kPrefillBnWide, 1, false, st));
    // Attention on the tensor cores; the closed slots are a strided view of the token rows.
    // d_h = 64: two query tiles per CTA over 64-slot key tiles (prefill_attn_tc2.cuh).
    const bool two_tiles = dm.dh == 64;
    const int DQ = dm.dh + dm.dr, kt = two_tiles ? pft2::KT : pft::key_tile(dm.dh);
    const int n_slots_closed = T_len / dm.s;
    const bf16* kv = h->at<bf16>(p.pf_kv);
    const bf16* kr = h->at<bf16>(p.pf_kr);
    CUtensorMap q_map, kv_closed, kv_self, kr_closed, kr_self;
    MTLA_TRY(make_map_3d(&q_map, h->at<void>(p.pf_qcat), (long long)dm.nh * DQ, T_len, B,
                         (long long)dm.nh * DQ, (long long)T_len * dm.nh * DQ, pft::kQTile));
    MTLA_TRY(make_map_3d(&kv_self, kv, 4 * hd, T_len, B, 4 * hd, (long long)T_len * 4 * hd, kt));
    MTLA_TRY(make_map_3d(&kr_self, kr, dm.dr, T_len, B, dm.dr, (long long)T_len * dm.dr, kt));
    if (n_slots_closed > 0) {
      MTLA_TRY(make_map_3d(&kv_closed, kv + (size_t)(dm.s - 1) * 4 * hd, 4 * hd, n_slots_closed, B,
                           (long long)dm.s * 4 * hd, (long long)T_len * 4 * hd, kt));
      MTLA_TRY(make_map_3d(&kr_closed, kr + (size_t)(dm.s - 1) * dm.dr, dm.dr, n_slots_closed, B,
                           (long long)dm.s * dm.dr, (long long)T_len * dm.dr, kt));
    } else {
      kv_closed = kv_self;   // never read: a prompt shorter than the stride closes no slot
      kr_closed = kr_self;
    }
    PrefillAttnTcArgs ta;
    ta.out = h->at<bf16>(p.pf_attn);
    ta.error_word = h->at<int>(p.err_flag);
    ta.n_heads = dm.nh; ta.dr = dm.dr; ta.stride = dm.s; ta.T = T_len;
    dim3 grid(ceil_div(T_len, pft::kQTile), dm.nh, B);
    if (two_tiles) {
      if (!h->pf_smem_ready)
        MTLA_CUDA(cudaFuncSetAttribute(prefill_attn_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       pft2::kSmemBytes));
      grid.x = ceil_div(T_len, pft2::kQTiles * pft2::kQTile);
      prefill_attn_tc2_kernel<<<grid, pft2::kThreads, pft2::kSmemBytes, st>>>(
          q_map, kv_closed, kv_self, kr_closed, kr_self, ta);
    } else {
      if (!h->pf_smem_ready)
        MTLA_CUDA(cudaFuncSetAttribute(prefill_attn_tc_kernel<128>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, pft::smem_bytes(128)));
      prefill_attn_tc_kernel<128><<<grid, pft::kThreads, pft::smem_bytes(128), st>>>(
          q_map, kv_closed, kv_self, kr_closed, kr_self, ta);
    }
    h->pf_smem_ready = true;
    h->launches++;
    MTLA_CUDA(cudaGetLastError());
    CUtensorMap map_a;
    MTLA_TRY(make_map_2d(&map_a, h->at<void>(p.pf_attn), rows, 2 * hd, 2 * hd, kPrefillBn));
    GemmTcArgs g = gemm_tc_args(y, 1, dm.d, dm.d, rows, hd, 1.f);
    g.b_lo_col = hd;
    MTLA_TRY(gemm_tc<bf16>(h, h->map_wot, map_a, g, kPrefillBn, 1, false, st));
    return MTLA_OK;
  }
  MTLA_TRY((gemm<T, T, float>(h, h->at<T>(p.pf_cprime), h->at<T>(p.w_kv_t), h->at<float>(p.pf_kv),
                              rows, 2 * hd, dm.r, dm.r, dm.r, 2 * hd, 1.f, 1, 0, 0, 0, st)));
  PrefillAttnArgs aa;
  aa.qcat = pa.qcat; aa.kv = h->at<void>(p.pf_kv); aa.kr = pa.kr; aa.out = h->at<void>(p.pf_attn);
  aa.n_heads = dm.nh; aa.dr = dm.dr; aa.stride = dm.s; aa.T = T_len;
  const size_t smem = prefill_attn_fma_smem_bytes(dm.dh, dm.dr);
  dim3 grid(ceil_div(T_len, kPfTile), dm.nh, B);
  if (dm.dh == 64) {
    if (!h->pf_smem_ready)
      MTLA_CUDA(cudaFuncSetAttribute(prefill_attn_fma_kernel<float, float, 64>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    prefill_attn_fma_kernel<float, float, 64><<<grid, 256, smem, st>>>(aa);
  } else {
    if (!h->pf_smem_ready)
      MTLA_CUDA(cudaFuncSetAttribute(prefill_attn_fma_kernel<float, float, 128>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    prefill_attn_fma_kernel<float, float, 128><<<grid, 256, smem, st>>>(aa);
  }
  h->pf_smem_ready = true;
  h->launches++;
  MTLA_CUDA(cudaGetLastError());
  MTLA_TRY((gemm<float, T, T>(h, h->at<float>(p.pf_attn), h->at<T>(p.w_o_t), y, rows, dm.d, hd, hd,
                              hd, dm.d, 1.f, 1, 0, 0, 0, st)));
  return MTLA_OK;
}

// dst[idx] = val for every pair, in launches of at most kScatterOps pairs.
int send_scatter(mtla_handle* h, int* dst, const std::vector<int>& idx, const std::vector<int>& val,
                 cudaStream_t st) {
  for (size_t at = 0; at < idx.size(); at += kScatterOps) {
    IntScatter ops;
    ops.n = (int)std::min<size_t>(kScatterOps, idx.size() - at);
    for (int i = 0; i < ops.n; ++i) {
      ops.idx[i] = idx[at + i];
      ops.val[i] = val[at + i];
    }
    MTLA_CUDA(launch_kernel(int_scatter_kernel, dim3(ceil_div(ops.n, 128)), dim3(128), 0, st, true, dst, ops));
    h->launches++;
  }
  return MTLA_OK;
}

// Re-sends the per-sequence positions after the host changed them.
int sync_tokens(mtla_handle* h, cudaStream_t st) {
  if (!h->paged() || !h->tokens_stale) return MTLA_OK;
  std::vector<int> idx(h->cfg.max_batch), val(h->seq_tokens);
  for (int b = 0; b < h->cfg.max_batch; ++b) idx[b] = b;
  MTLA_TRY(send_scatter(h, h->d_seq_tokens(h->buf()), idx, val, st));
  h->tokens_stale = false;
  return MTLA_OK;
}

// Enqueues what the page pool decided: page copies first, then the table entries.
int apply_page_ops(mtla_handle* h, const std::vector<PageSet>& sets, const std::vector<PageCopy>& copies,
                   cudaStream_t st) {
  const long long page_bytes = (long long)kPageSlots * h->dm.W * h->dm.elem;
  for (size_t at = 0; at < copies.size(); at += kPageCopyOps) {
    PageCopies ops;
    ops.n = (int)std::min<size_t>(kPageCopyOps, copies.size() - at);
    for (int i = 0; i < ops.n; ++i) {
      ops.src[i] = copies[at + i].src;
      ops.dst[i] = copies[at + i].dst;
      ops.rows[i] = copies[at + i].rows;
    }
    MTLA_CUDA(launch_kernel(page_copy_kernel, dim3(ops.n), dim3(256), 0, st, true, h->at<char>(h->plan.cache),
                            page_bytes, (int)(h->dm.W * h->dm.elem), ops));
    h->launches++;
  }
  std::vector<int> idx(sets.size()), val(sets.size());
  for (size_t i = 0; i < sets.size(); ++i) {
    idx[i] = sets[i].seq * h->dm.max_pages + sets[i].index;
    val[i] = sets[i].page;
  }
  return send_scatter(h, h->d_page_table(h->buf()), idx, val, st);
}

int check_step_args(mtla_handle* h, const void* x, int32_t B, const void* y) {
  if (!h || !x || !y || B <= 0) return MTLA_ERR_INVALID_ARG;
  if (h->batch == 0) {
    if (B > h->cfg.max_batch) return MTLA_ERR_CAPACITY;
  } else if (B != h->batch) {
    return MTLA_ERR_BATCH_MISMATCH;
  }
  if (!h->paged()) return h->tokens + 1 > h->cfg.max_tokens ? MTLA_ERR_CAPACITY : MTLA_OK;
  if (h->use_tc && B > tc::kMaxRaggedBatch) return MTLA_ERR_CAPACITY;
  // Pages the step will take from the free list: new pages at page boundaries, and copies of
  // shared newest pages.  Of the w sequences about to write a page that ref sequences hold, the
  // last one to be served keeps the page if all holders write it: min(w, ref - 1) copies.
  int need = 0;
  std::vector<int> shared;
  for (int b = 0; b < B; ++b) {
    if (h->seq_tokens[b] + 1 > h->cfg.max_tokens) return MTLA_ERR_CAPACITY;
    const int slot = h->seq_tokens[b] / h->dm.s, k = slot / kPageSlots;
    const int have = h->pool->pages_held(b);
    need += std::max(0, PagePool::pages_for(slot + 1) - have);
    if (k < have && h->pool->ref(h->pool->row(b)[k]) > 1) shared.push_back(h->pool->row(b)[k]);
  }
  std::sort(shared.begin(), shared.end());
  for (size_t i = 0; i < shared.size();) {
    size_t j = i;
    while (j < shared.size() && shared[j] == shared[i]) ++j;
    need += std::min((int)(j - i), h->pool->ref(shared[i]) - 1);
    i = j;
  }
  return need > h->pool->pages_free() ? MTLA_ERR_CAPACITY : MTLA_OK;
}

// Paged handles, before the kernels of a decode step: every sequence gets the page its new
// token's slot lives in, private to it (copy-on-write after a beam fork).
int step_begin(mtla_handle* h, int B, cudaStream_t st) {
  if (!h->paged()) return MTLA_OK;
  MTLA_TRY(sync_tokens(h, st));
  std::vector<PageSet> sets;
  std::vector<PageCopy> copies;
  for (int b = 0; b < B; ++b) {
    const int slot = h->seq_tokens[b] / h->dm.s;
    if (!h->pool->prepare(b, slot + 1, slot, &sets, &copies)) return MTLA_ERR_STATE;
  }
  return apply_page_ops(h, sets, copies, st);
}

void step_end(mtla_handle* h, int B) {
  h->train_B = h->train_T = 0;      // the decode step reuses the prefill's scratch
  if (h->paged()) {
    for (int b = 0; b < B; ++b) {
      h->seq_tokens[b] += 1;
      h->tokens = max(h->tokens, h->seq_tokens[b]);
    }
  } else {
    h->tokens += 1;
  }
  h->batch = B;
}

template <typename T>
int dispatch_decode(mtla_handle* h, const void* x, int B, void* y, cudaStream_t st,
                    const AttnScratch* scratch) {
  MTLA_TRY(step_begin(h, B, st));
  MTLA_TRY(decode_impl<T>(h, x, B, y, st, scratch));
  step_end(h, B);
  return MTLA_OK;
}

int baseline_decode(mtla_handle* h, const void* x, int B, void* y, cudaStream_t st);

int run_decode(mtla_handle* h, const void* x, int B, void* y, cudaStream_t st,
               const AttnScratch* scratch = nullptr) {
  if (h->is_baseline) {
    if (scratch) return MTLA_ERR_STATE;
    MTLA_TRY(baseline_decode(h, x, B, y, st));
    step_end(h, B);
    return MTLA_OK;
  }
  return h->cfg.dtype == MTLA_DTYPE_BF16 ? dispatch_decode<bf16>(h, x, B, y, st, scratch)
                                         : dispatch_decode<float>(h, x, B, y, st, scratch);
}

// Prefill of sequences seq0 .. seq0 + B - 1 (all empty), T tokens each.
int run_prefill(mtla_handle* h, const void* x, int seq0, int B, int T, void* y, cudaStream_t st) {
  const int n_slots = ceil_div(T, h->dm.s);
  if (h->paged()) {
    if (B * PagePool::pages_for(n_slots) > h->pool->pages_free()) return MTLA_ERR_CAPACITY;
    std::vector<PageSet> sets;
    std::vector<PageCopy> copies;
    for (int b = seq0; b < seq0 + B; ++b)
      if (!h->pool->prepare(b, n_slots, -1, &sets, &copies)) return MTLA_ERR_STATE;
    MTLA_TRY(apply_page_ops(h, sets, copies, st));
  }
  const int rc = h->cfg.dtype == MTLA_DTYPE_BF16 ? prefill_impl<bf16>(h, x, seq0, B, T, y, st)
                                                 : prefill_impl<float>(h, x, seq0, B, T, y, st);
  if (rc != MTLA_OK) return rc;
  if (h->paged()) {
    for (int b = seq0; b < seq0 + B; ++b) h->seq_tokens[b] = T;
    h->tokens_stale = true;
  }
  h->tokens = max(h->tokens, T);
  h->batch = max(h->batch, seq0 + B);
  return MTLA_OK;
}

int create_handle(const mtla_config* cfg, const mtla_paging* paging, const mtla_weights* w, void* arena,
                  size_t arena_bytes, void* stream, mtla_handle** out, void* shared_scratch = nullptr);

}  // namespace

extern "C" {

size_t mtla_arena_bytes(const mtla_config* cfg) {
  mtla_config c;
  Dims dm;
  if (!normalise(cfg, nullptr, &c, &dm)) return 0;
  ArenaPlan p;
  plan_arena(c, dm, &p);
  return p.total;
}

size_t mtla_arena_bytes_paged(const mtla_config* cfg, const mtla_paging* paging) {
  mtla_config c;
  Dims dm;
  if (!paging || !normalise(cfg, paging, &c, &dm)) return 0;
  ArenaPlan p;
  plan_arena(c, dm, &p);
  return p.total;
}

int mtla_create(const mtla_config* cfg, const mtla_weights* w, void* arena, size_t arena_bytes,
                void* stream, mtla_handle** out) {
  return create_handle(cfg, nullptr, w, arena, arena_bytes, stream, out);
}

int mtla_create_paged(const mtla_config* cfg, const mtla_paging* paging, const mtla_weights* w,
                      void* arena, size_t arena_bytes, void* stream, mtla_handle** out) {
  if (!paging) return MTLA_ERR_INVALID_ARG;
  return create_handle(cfg, paging, w, arena, arena_bytes, stream, out);
}

}  // extern "C"

namespace {

// With shared_scratch the arena holds only the persistent part (plan.scratch_begin bytes) and the
// per-call scratch lives at shared_scratch (plan.total - plan.scratch_begin bytes, 1024-aligned).
int create_handle(const mtla_config* cfg, const mtla_paging* paging, const mtla_weights* w, void* arena,
                  size_t arena_bytes, void* stream, mtla_handle** out, void* shared_scratch) {
  if (!cfg || !w || !arena || !out) return MTLA_ERR_INVALID_ARG;
  mtla_config c;
  Dims dm;
  if (!normalise(cfg, paging, &c, &dm)) return MTLA_ERR_UNSUPPORTED_SHAPE;
  const void* required[] = {w->w_q, w->w_qr, w->w_r, w->w_kr, w->ln_gamma, w->ln_beta,
                            w->w_k, w->w_v, w->w_o, w->hyp_c_w, w->hyp_pe_w};
  for (const void* ptr : required)
    if (!ptr || !aligned16(ptr)) return MTLA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(arena) & 1023) return MTLA_ERR_INVALID_ARG;
  ArenaPlan p;
  plan_arena(c, dm, &p);
  if (arena_bytes < (shared_scratch ? p.scratch_begin : p.total)) return MTLA_ERR_ARENA_TOO_SMALL;
  mtla_handle* h = new (std::nothrow) mtla_handle();
  if (!h) return MTLA_ERR_INVALID_ARG;
  h->cfg = c; h->dm = dm; h->plan = p; h->arena = static_cast<char*>(arena);
  h->scratch = shared_scratch ? static_cast<char*>(shared_scratch) - p.scratch_begin : nullptr;
  h->tokens = 0; h->batch = 0; h->launches = 0;
  h->train_B = h->train_T = 0;
  h->attn_smem_ready = false; h->pf_smem_ready = false;
  h->prof_used = 0;
  h->prof_attention_only = false;
  h->act_bn = 0;
  h->gemm_attr_mask = 0;
  h->pool = nullptr;
  h->tokens_stale = false;
  h->is_baseline = false;
  h->bl_groups = 1;
  const int dev_rc = arena_device(arena, &h->device, &h->sm_count);
  if (dev_rc != MTLA_OK) {
    delete h;
    return dev_rc;
  }
  if (paging) {
    h->pool = new (std::nothrow) PagePool(dm.n_pages, c.max_batch, dm.max_pages);
    if (!h->pool) {
      delete h;
      return MTLA_ERR_INVALID_ARG;
    }
    h->seq_tokens.assign(c.max_batch, 0);
    h->tokens_stale = true;
  }
  // The tensor-core kernels need bf16 and whole 128-column latent blocks; config.kernel_path
  // can keep such a layer on the CUDA-core kernels (for comparisons between the two).
  h->use_tc = c.dtype == MTLA_DTYPE_BF16 && dm.r % 128 == 0 && c.kernel_path != MTLA_PATH_CUDA_CORE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int rc = c.dtype == MTLA_DTYPE_BF16 ? create_impl<bf16>(h, w, st) : create_impl<float>(h, w, st);
  if (rc != MTLA_OK) {
    delete h->pool;
    delete h;
    return rc;
  }
  *out = h;
  return MTLA_OK;
}


// ---------------------------------------------------------------------------------------------
// Comparison layers (Section 3): MHA / GQA / MQA decode over a key-value cache, bf16, built from
// the same projection GEMM and the same decode attention kernel (see baseline_kernels.cuh).

bool baseline_dims(const mtla_baseline_config* in, mtla_config* cfg, Dims* dm, int* groups) {
  if (!in) return false;
  if (in->d_model <= 0 || in->d_model % 8) return false;
  if (in->head_dim != 64 && in->head_dim != 128) return false;
  if (in->n_heads < 1 || in->n_kv_heads < 1 || in->n_heads % in->n_kv_heads) return false;
  const int per = in->n_heads / in->n_kv_heads;
  if (per > 32) return false;
  if (in->max_batch < 1 || in->max_tokens < 1) return false;
  if ((long long)in->max_batch * in->n_kv_heads * in->max_tokens > (1ll << 40)) return false;
  memset(cfg, 0, sizeof(*cfg));
  cfg->d_model = in->d_model; cfg->n_heads = in->n_heads; cfg->head_dim = in->head_dim;
  cfg->max_batch = in->max_batch; cfg->max_tokens = in->max_tokens; cfg->stride = 1;
  cfg->dtype = MTLA_DTYPE_BF16;
  cfg->rope_theta = in->rope_theta == 0.f ? 10000.f : in->rope_theta;
  memset(dm, 0, sizeof(*dm));
  dm->d = in->d_model; dm->dh = in->head_dim; dm->s = 1; dm->elem = 2;
  dm->nh = per;                       // heads the attention kernel sees per (sequence, group)
  dm->W = 2 * in->head_dim;           // cache row: value, then key
  dm->r = dm->W; dm->dr = 0;
  dm->max_slots = in->max_tokens;
  dm->ntot = (in->n_heads + 2 * in->n_kv_heads) * in->head_dim;
  dm->max_units = kPlanSms + in->max_batch * in->n_kv_heads;
  *groups = in->n_kv_heads;
  return true;
}

void plan_baseline(const mtla_config& c, const Dims& dm, int groups, ArenaPlan* p) {
  memset(p, 0, sizeof(*p));
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off = align_up(off + bytes, 1024);
    return at;
  };
  const size_t B = c.max_batch, hd = (size_t)c.n_heads * dm.dh, planes = B * groups;
  p->wcat_t = take((size_t)dm.ntot * dm.d * 2);
  p->w_o_t = take((size_t)dm.d * hd * 2);
  p->rope_cos = take((size_t)c.max_tokens * (dm.dh / 2) * 4);
  p->rope_sin = take((size_t)c.max_tokens * (dm.dh / 2) * 4);
  p->cache = take(planes * dm.max_slots * dm.W * 2);
  p->err_flag = take(16);
  p->scratch_begin = off;
  p->p1 = take(B * dm.ntot * 4);
  p->qt = take(planes * dm.nh * dm.W * 2);
  p->o_part = take((size_t)dm.max_units * dm.nh * dm.W * 4);
  p->ml_part = take((size_t)dm.max_units * dm.nh * 2 * 4);
  p->o = take(planes * 2 * dm.nh * dm.W * 2);
  p->v = take(B * 2 * hd * 2);
  p->gemm_part = take((size_t)kGemmSlots * gtc::kBM * act_box_rows(c.max_batch) * 4);
  p->gemm_tickets = take((size_t)kGemmSlots * 4 * sizeof(int));
  p->attn_tickets = take(planes * sizeof(int));
  p->total = off;
}

int baseline_decode(mtla_handle* h, const void* x, int B, void* y, cudaStream_t st) {
  const Dims& dm = h->dm;
  const ArenaPlan& p = h->plan;
  const int g = h->bl_groups, n_heads = dm.nh * g, hd = n_heads * dm.dh, pos = h->tokens;
  const int bn = act_box_rows(B);
  const bool prof = h->prof_used + MTLA_DECODE_STAGES + 1 <= (int)h->prof_events.size();
  if (h->act_bn != bn) {
    MTLA_TRY(make_map_2d(&h->map_v16, h->at<void>(p.v), h->cfg.max_batch, 2 * hd, 2 * hd, bn));
    h->act_bn = bn;
  }
  MTLA_TRY(prof_mark(h, prof, 0, st));
  CUtensorMap map_x;
  MTLA_TRY(make_map_2d(&map_x, x, B, dm.d, dm.d, bn));
  MTLA_TRY(gemm_tc<float>(h, h->map_wcat, map_x,
                          gemm_tc_args(h->at<float>(p.p1), 1, dm.ntot, dm.ntot, B, dm.d, 1.f), bn, 1,
                          true, st));
  MTLA_TRY(prof_mark(h, prof, 1, st));
  KvPostArgs ka;
  ka.p1 = h->at<float>(p.p1);
  ka.rope_cos = h->at<float>(p.rope_cos);
  ka.rope_sin = h->at<float>(p.rope_sin);
  ka.cache = h->at<bf16>(p.cache);
  ka.qt = h->at<bf16>(p.qt);
  ka.n_heads = n_heads; ka.n_groups = g; ka.head_dim = dm.dh; ka.max_tokens = dm.max_slots;
  ka.tokens = pos;
  ka.q_scale = (float)(1.4426950408889634 / sqrt((double)dm.dh));
  const bool pdl = !(prof && !h->prof_attention_only);
  MTLA_CUDA(launch_kernel(kv_post_kernel, dim3(B), dim3(256), 0, st, pdl, ka));
  h->launches++;
  MTLA_TRY(prof_mark(h, prof, 2, st));
  MTLA_TRY(prof_mark(h, prof, 3, st));
  AttnTcArgs ta;
  memset(&ta, 0, sizeof(ta));
  ta.o_part = h->at<float>(p.o_part); ta.ml_part = h->at<float>(p.ml_part);
  ta.o16 = h->at<bf16>(p.o);
  ta.tickets = h->at<int>(p.attn_tickets);
  ta.error_word = h->at<int>(p.err_flag);
  ta.n_heads = dm.nh; ta.r = dm.W; ta.dr = 0; ta.n_slots = pos + 1; ta.batch = B * g;
  ta.tiles_per_seq = ceil_div(pos + 1, tc::kTile);
  const long long total = (long long)ta.batch * ta.tiles_per_seq;
  const int grid = (int)(total < h->sm_count ? total : h->sm_count);
  const bool attn_pdl = pdl && !prof;
  const bool split_combine = grid / ta.batch + 2 > kFusedCombineMaxParts;
  ta.fused_combine = !split_combine;
  ta.attn_grid = grid;
  if (dm.nh <= 16) MTLA_TRY((launch_attn_tc_rp<16, false>(h, ta, grid, st, attn_pdl)));
  else MTLA_TRY((launch_attn_tc_rp<32, false>(h, ta, grid, st, attn_pdl)));
  if (split_combine) {
    MTLA_CUDA(launch_kernel(decode_combine_parts_kernel, dim3(dm.nh, ta.batch), dim3(128), 0, st, attn_pdl, ta));
    h->launches++;
  }
  MTLA_TRY(prof_mark(h, prof, 4, st));
  MTLA_TRY(prof_mark(h, prof, 5, st));
  MTLA_CUDA(launch_kernel(kv_heads_gather_kernel, dim3(B), dim3(256), 0, st, pdl && !prof,
                          (const bf16*)h->at<bf16>(p.o), h->at<bf16>(p.v), n_heads, g, dm.dh));
  h->launches++;
  MTLA_TRY(prof_mark(h, prof, 6, st));
  GemmTcArgs ga = gemm_tc_args(y, 1, dm.d, dm.d, B, hd, 1.f);
  ga.b_lo_col = hd;
  MTLA_TRY(gemm_tc<bf16>(h, h->map_wot, h->map_v16, ga, bn, 1, true, st, pdl));
  MTLA_TRY(prof_mark(h, prof, 7, st));
  if (prof) h->prof_used += MTLA_DECODE_STAGES + 1;
  return MTLA_OK;
}

int baseline_create(mtla_handle* h, const mtla_baseline_weights* w, cudaStream_t st) {
  const Dims& dm = h->dm;
  const ArenaPlan& p = h->plan;
  const int g = h->bl_groups, n_heads = dm.nh * g, hd = n_heads * dm.dh, gd = g * dm.dh;
  bf16* wcat = h->at<bf16>(p.wcat_t);
  // Fused projection stored [out][in]: rows [ q | k | v ].
  MTLA_TRY(launch_transpose<bf16>(h, w->w_q, wcat, dm.d, hd, hd, dm.d, st));
  MTLA_TRY(launch_transpose<bf16>(h, w->w_k, wcat + (size_t)hd * dm.d, dm.d, gd, gd, dm.d, st));
  MTLA_TRY(launch_transpose<bf16>(h, w->w_v, wcat + (size_t)(hd + gd) * dm.d, dm.d, gd, gd, dm.d, st));
  MTLA_TRY(launch_transpose<bf16>(h, w->w_o, h->at<bf16>(p.w_o_t), hd, dm.d, dm.d, hd, st));
  const long long n_rope = (long long)h->cfg.max_tokens * (dm.dh / 2);
  rope_table_kernel<<<(unsigned)((n_rope + 255) / 256), 256, 0, st>>>(
      h->at<float>(p.rope_cos), h->at<float>(p.rope_sin), h->cfg.max_tokens, dm.dh / 2,
      (double)h->cfg.rope_theta);
  h->launches++;
  MTLA_CUDA(cudaGetLastError());
  const size_t planes = (size_t)h->cfg.max_batch * g;
  MTLA_CUDA(cudaMemsetAsync(h->at<char>(p.err_flag), 0, 16, st));
  // Rows beyond the valid range are multiplied by probability 0 and must be finite; the zero
  // halves of the query rows stay zero for the handle's life.
  MTLA_CUDA(cudaMemsetAsync(h->at<char>(p.cache), 0, planes * dm.max_slots * dm.W * 2, st));
  MTLA_CUDA(cudaMemsetAsync(h->at<char>(p.qt), 0, planes * dm.nh * dm.W * 2, st));
  MTLA_CUDA(cudaMemsetAsync(h->at<char>(p.gemm_tickets), 0, (size_t)kGemmSlots * 4 * sizeof(int), st));
  MTLA_CUDA(cudaMemsetAsync(h->at<char>(p.attn_tickets), 0, planes * sizeof(int), st));
  MTLA_TRY(make_cache_map(h));
  MTLA_TRY(make_map_2d(&h->map_wcat, h->at<void>(p.wcat_t), dm.ntot, dm.d, dm.d, gtc::kBM));
  MTLA_TRY(make_map_2d(&h->map_wot, h->at<void>(p.w_o_t), dm.d, hd, hd, gtc::kBM));
  return MTLA_OK;
}

}  // namespace

extern "C" {

size_t mtla_baseline_arena_bytes(const mtla_baseline_config* cfg) {
  mtla_config c;
  Dims dm;
  int groups;
  if (!baseline_dims(cfg, &c, &dm, &groups)) return 0;
  ArenaPlan p;
  plan_baseline(c, dm, groups, &p);
  return p.total;
}

int mtla_baseline_create(const mtla_baseline_config* cfg, const mtla_baseline_weights* w, void* arena,
                         size_t arena_bytes, void* stream, mtla_handle** out) {
  if (!cfg || !w || !arena || !out) return MTLA_ERR_INVALID_ARG;
  mtla_config c;
  Dims dm;
  int groups;
  if (!baseline_dims(cfg, &c, &dm, &groups)) return MTLA_ERR_UNSUPPORTED_SHAPE;
  for (const void* ptr : {w->w_q, w->w_k, w->w_v, w->w_o})
    if (!ptr || !aligned16(ptr)) return MTLA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(arena) & 1023) return MTLA_ERR_INVALID_ARG;
  ArenaPlan p;
  plan_baseline(c, dm, groups, &p);
  if (arena_bytes < p.total) return MTLA_ERR_ARENA_TOO_SMALL;
  mtla_handle* h = new (std::nothrow) mtla_handle();
  if (!h) return MTLA_ERR_INVALID_ARG;
  h->cfg = c; h->dm = dm; h->plan = p; h->arena = static_cast<char*>(arena);
  h->scratch = nullptr;
  h->tokens = 0; h->batch = 0; h->launches = 0;
  h->train_B = h->train_T = 0;
  h->attn_smem_ready = false; h->pf_smem_ready = false;
  h->prof_used = 0;
  h->prof_attention_only = false;
  h->act_bn = 0;
  h->gemm_attr_mask = 0;
  h->pool = nullptr;
  h->tokens_stale = false;
  h->is_baseline = true;
  h->bl_groups = groups;
  h->use_tc = true;
  const int dev_rc = arena_device(arena, &h->device, &h->sm_count);
  if (dev_rc != MTLA_OK) {
    delete h;
    return dev_rc;
  }
  const int rc = baseline_create(h, w, static_cast<cudaStream_t>(stream));
  if (rc != MTLA_OK) {
    delete h;
    return rc;
  }
  *out = h;
  return MTLA_OK;
}

}  // extern "C"

namespace {
}  // namespace

extern "C" {

int mtla_prefill(mtla_handle* h, const void* x, int32_t B, int32_t T, void* y, void* stream) {
  if (!h || !x || B <= 0 || T <= 0) return MTLA_ERR_INVALID_ARG;
  if (h->is_baseline) return MTLA_ERR_STATE;
  if (!aligned16(x) || (y && !aligned16(y))) return MTLA_ERR_INVALID_ARG;
  if (h->tokens != 0 || h->batch != 0) return MTLA_ERR_STATE;
  if (B > h->cfg.max_batch || T > h->cfg.max_prefill_tokens || T > h->cfg.max_tokens)
    return MTLA_ERR_CAPACITY;
  const int rc = run_prefill(h, x, 0, B, T, y, static_cast<cudaStream_t>(stream));
  if (rc == MTLA_OK && y) {
    h->train_B = B;
    h->train_T = T;
  }
  return rc;
}

int mtla_prefill_seqs(mtla_handle* h, int32_t seq0, const void* x, int32_t B, int32_t T, void* y,
                      void* stream) {
  if (!h || !x || B <= 0 || T <= 0 || seq0 < 0) return MTLA_ERR_INVALID_ARG;
  if (!aligned16(x) || (y && !aligned16(y))) return MTLA_ERR_INVALID_ARG;
  if (!h->paged()) return MTLA_ERR_STATE;
  if (seq0 > h->batch) return MTLA_ERR_STATE;           // sequences are numbered without gaps
  if (seq0 + B > h->cfg.max_batch || T > h->cfg.max_prefill_tokens || T > h->cfg.max_tokens)
    return MTLA_ERR_CAPACITY;
  for (int b = seq0; b < seq0 + B; ++b)
    if (h->seq_tokens[b] != 0) return MTLA_ERR_STATE;
  return run_prefill(h, x, seq0, B, T, y, static_cast<cudaStream_t>(stream));
}

int mtla_decode_step(mtla_handle* h, const void* x, int32_t B, void* y, void* stream) {
  const int chk = check_step_args(h, x, B, y);
  if (chk != MTLA_OK) return chk;
  if (!aligned16(x) || !aligned16(y)) return MTLA_ERR_INVALID_ARG;
  return run_decode(h, x, B, y, static_cast<cudaStream_t>(stream));
}

int mtla_decode_step_host(mtla_handle* h, const void* x_host, int32_t B, void* y_host,
                          void* stream) {
  const int chk = check_step_args(h, x_host, B, y_host);
  if (chk != MTLA_OK) return chk;
  if (h->is_baseline) return MTLA_ERR_STATE;    // no staging rows in a comparison layer's arena
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t bytes = (size_t)B * h->dm.d * h->dm.elem;
  void* xs = h->at<void>(h->plan.x_stage);
  void* ys = h->at<void>(h->plan.y_stage);
  MTLA_CUDA(cudaMemcpyAsync(xs, x_host, bytes, cudaMemcpyHostToDevice, st));
  MTLA_TRY(run_decode(h, xs, B, ys, st));
  MTLA_CUDA(cudaMemcpyAsync(y_host, ys, bytes, cudaMemcpyDeviceToHost, st));
  return MTLA_OK;
}

int mtla_decode_step_static(mtla_handle* h, const void* x, int32_t B, void* y, void* stream) {
  const int chk = check_step_args(h, x, B, y);
  if (chk != MTLA_OK) return chk;
  if (!aligned16(x) || !aligned16(y)) return MTLA_ERR_INVALID_ARG;
  if (h->is_baseline) return MTLA_ERR_STATE;
  // Same sizing as the arena's split workspace, for this call's batch.
  const Dims& dm = h->dm;
  const size_t units = (size_t)(h->use_tc ? kPlanSms : kTargetCtas) + (size_t)B;
  const size_t tickets_bytes = align_up((size_t)B * sizeof(int), 256);
  const size_t ml_bytes = align_up(units * dm.nh * 2 * sizeof(float), 256);
  const size_t o_bytes = units * dm.nh * dm.r * sizeof(float);
  if (tickets_bytes + ml_bytes + o_bytes > MTLA_STATIC_SCRATCH_BYTES) return MTLA_ERR_SCRATCH_LIMIT;
  // The array exists once per GPU: the kernels must get the copy of the GPU that owns the
  // handle's arena, so that GPU has to be the current one, on every call.
  int dev = -1;
  MTLA_CUDA(cudaGetDevice(&dev));
  if (dev != h->device) return MTLA_ERR_STATE;
  if (dev < 0 || dev >= kMaxDevices) return MTLA_ERR_UNSUPPORTED_SHAPE;
  // First call on this device: turn the array's host-side name into its device address.  Two
  // threads that race here store the same address, so the slot needs no lock.
  if (!g_static_scratch_addr[dev]) {
    void* addr = nullptr;
    MTLA_CUDA(cudaGetSymbolAddress(&addr, g_static_scratch));
    g_static_scratch_addr[dev] = static_cast<unsigned char*>(addr);
  }
  unsigned char* base = g_static_scratch_addr[dev];
  AttnScratch sc;
  sc.tickets = reinterpret_cast<int*>(base);
  sc.ml_part = reinterpret_cast<float*>(base + tickets_bytes);
  sc.o_part = reinterpret_cast<float*>(base + tickets_bytes + ml_bytes);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The array keeps whatever the previous call left: the tickets must start at zero.
  MTLA_CUDA(cudaMemsetAsync(sc.tickets, 0, (size_t)B * sizeof(int), st));
  return run_decode(h, x, B, y, st, &sc);
}

size_t mtla_cache_bytes(const mtla_handle* h) {
  if (!h) return 0;
  size_t slots = 0;
  for (int b = 0; b < h->batch; ++b) slots += ceil_div(h->seq_len(b), h->dm.s);
  return slots * h->planes_per_seq() * h->dm.W * h->dm.elem;
}

int mtla_destroy(mtla_handle* h) {
  if (!h) return MTLA_ERR_INVALID_ARG;
  for (cudaEvent_t e : h->prof_events) cudaEventDestroy(e);
  delete h->pool;
  delete h;
  return MTLA_OK;
}

int mtla_reset(mtla_handle* h) {
  if (!h) return MTLA_ERR_INVALID_ARG;
  h->tokens = 0;
  h->batch = 0;
  h->train_B = h->train_T = 0;
  if (h->paged()) {
    h->pool->reset();
    h->seq_tokens.assign(h->cfg.max_batch, 0);
    h->tokens_stale = true;
  }
  return MTLA_OK;
}

int mtla_position(const mtla_handle* h, int32_t* tokens, int32_t* slots, int32_t* batch) {
  if (!h) return MTLA_ERR_INVALID_ARG;
  if (tokens) *tokens = h->tokens;
  if (slots) *slots = ceil_div(h->tokens, h->dm.s);
  if (batch) *batch = h->batch;
  return MTLA_OK;
}

int mtla_cache_export(mtla_handle* h, void* dst, size_t bytes, void* stream) {
  if (!h || !dst) return MTLA_ERR_INVALID_ARG;
  const size_t need = mtla_cache_bytes(h);
  if (bytes < need) return MTLA_ERR_CAPACITY;
  if (need == 0) return MTLA_OK;
  if (h->paged()) {
    if (!aligned16(dst)) return MTLA_ERR_INVALID_ARG;
    for (int b = 0; b < h->batch; ++b)
      if (h->seq_tokens[b] != h->tokens) return MTLA_ERR_STATE;   // ragged: use mtla_cache_export_seq
    const int n_slots = ceil_div(h->tokens, h->dm.s);
    cache_rows_copy_kernel<<<dim3(ceil_div(n_slots, kPageSlots), h->batch), 256, 0,
                             static_cast<cudaStream_t>(stream)>>>(
        h->cache_view(), 0, n_slots, (int)(h->dm.W * h->dm.elem), static_cast<char*>(dst), 0);
    h->launches++;
    MTLA_CUDA(cudaGetLastError());
    return MTLA_OK;
  }
  const size_t row = (size_t)ceil_div(h->tokens, h->dm.s) * h->dm.W * h->dm.elem;
  const size_t pitch = (size_t)h->dm.max_slots * h->dm.W * h->dm.elem;
  MTLA_CUDA(cudaMemcpy2DAsync(dst, row, h->at<char>(h->plan.cache), pitch, row,
                              (size_t)h->batch * h->planes_per_seq(), cudaMemcpyDeviceToDevice,
                              static_cast<cudaStream_t>(stream)));
  return MTLA_OK;
}

int mtla_cache_import(mtla_handle* h, const void* src, int32_t B, int32_t tokens, void* stream) {
  if (!h || !src || B <= 0 || tokens <= 0 || !aligned16(src)) return MTLA_ERR_INVALID_ARG;
  if (B > h->cfg.max_batch || tokens > h->cfg.max_tokens) return MTLA_ERR_CAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int n_slots = ceil_div(tokens, h->dm.s);
  const size_t row = (size_t)n_slots * h->dm.W * h->dm.elem;
  const size_t pitch = (size_t)h->dm.max_slots * h->dm.W * h->dm.elem;
  if (h->paged()) {
    // The import replaces everything: all pages go back to the pool first.
    if ((long long)B * PagePool::pages_for(n_slots) > h->pool->n_pages()) return MTLA_ERR_CAPACITY;
    h->pool->reset();
    std::vector<PageSet> sets;
    std::vector<PageCopy> copies;
    for (int b = 0; b < B; ++b)
      if (!h->pool->prepare(b, n_slots, -1, &sets, &copies)) return MTLA_ERR_STATE;
    MTLA_TRY(apply_page_ops(h, sets, copies, st));
    cache_rows_copy_kernel<<<dim3(ceil_div(n_slots, kPageSlots), B), 256, 0, st>>>(
        h->cache_view(), 0, n_slots, (int)(h->dm.W * h->dm.elem),
        const_cast<char*>(static_cast<const char*>(src)), 1);
    h->launches++;
    MTLA_CUDA(cudaGetLastError());
    h->seq_tokens.assign(h->cfg.max_batch, 0);
    for (int b = 0; b < B; ++b) h->seq_tokens[b] = tokens;
    h->tokens_stale = true;
  } else {
    MTLA_CUDA(cudaMemcpy2DAsync(h->at<char>(h->plan.cache), pitch, src, row, row,
                                (size_t)B * h->planes_per_seq(), cudaMemcpyDeviceToDevice, st));
  }
  if (tokens % h->dm.s != 0) {
    if (h->cfg.dtype == MTLA_DTYPE_BF16)
      open_acc_from_cache_kernel<bf16><<<B, 256, 0, st>>>(h->cache_view(), h->d_open_acc(h->buf()),
                                                          h->dm.r, h->dm.W, 0, n_slots - 1);
    else
      open_acc_from_cache_kernel<float><<<B, 256, 0, st>>>(h->cache_view(), h->d_open_acc(h->buf()),
                                                           h->dm.r, h->dm.W, 0, n_slots - 1);
    h->launches++;
    MTLA_CUDA(cudaGetLastError());
  }
  h->tokens = tokens;
  h->batch = B;
  h->train_B = h->train_T = 0;
  return MTLA_OK;
}

int mtla_cache_import_seqs(mtla_handle* h, int32_t seq0, const void* src, int32_t B, int32_t tokens,
                           void* stream) {
  if (!h || !src || B <= 0 || tokens <= 0 || seq0 < 0 || !aligned16(src)) return MTLA_ERR_INVALID_ARG;
  if (!h->paged() || seq0 > h->batch) return MTLA_ERR_STATE;
  if (seq0 + B > h->cfg.max_batch || tokens > h->cfg.max_tokens) return MTLA_ERR_CAPACITY;
  for (int b = seq0; b < seq0 + B; ++b)
    if (h->seq_tokens[b] != 0) return MTLA_ERR_STATE;
  const int n_slots = ceil_div(tokens, h->dm.s);
  if ((long long)B * PagePool::pages_for(n_slots) > h->pool->pages_free()) return MTLA_ERR_CAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  std::vector<PageSet> sets;
  std::vector<PageCopy> copies;
  for (int b = seq0; b < seq0 + B; ++b)
    if (!h->pool->prepare(b, n_slots, -1, &sets, &copies)) return MTLA_ERR_STATE;
  MTLA_TRY(apply_page_ops(h, sets, copies, st));
  cache_rows_copy_kernel<<<dim3(ceil_div(n_slots, kPageSlots), B), 256, 0, st>>>(
      h->cache_view(), seq0, n_slots, (int)(h->dm.W * h->dm.elem),
      const_cast<char*>(static_cast<const char*>(src)), 1);
  h->launches++;
  MTLA_CUDA(cudaGetLastError());
  if (tokens % h->dm.s != 0) {
    if (h->cfg.dtype == MTLA_DTYPE_BF16)
      open_acc_from_cache_kernel<bf16><<<B, 256, 0, st>>>(h->cache_view(), h->d_open_acc(h->buf()),
                                                          h->dm.r, h->dm.W, seq0, n_slots - 1);
    else
      open_acc_from_cache_kernel<float><<<B, 256, 0, st>>>(h->cache_view(), h->d_open_acc(h->buf()),
                                                           h->dm.r, h->dm.W, seq0, n_slots - 1);
    h->launches++;
    MTLA_CUDA(cudaGetLastError());
  }
  for (int b = seq0; b < seq0 + B; ++b) h->seq_tokens[b] = tokens;
  h->tokens_stale = true;
  h->tokens = max(h->tokens, tokens);
  h->batch = max(h->batch, seq0 + B);
  return MTLA_OK;
}

int mtla_beam_reorder(mtla_handle* h, const int32_t* parents, int32_t n_new, void* stream) {
  if (!h || !parents || n_new <= 0) return MTLA_ERR_INVALID_ARG;
  if (!h->paged() || h->batch == 0) return MTLA_ERR_STATE;
  if (n_new > h->cfg.max_batch) return MTLA_ERR_CAPACITY;
  for (int b = 0; b < n_new; ++b)
    if (parents[b] < 0 || parents[b] >= h->batch) return MTLA_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  MTLA_TRY(sync_tokens(h, st));
  const int old = h->buf(), nxt = old ^ 1;
  BeamArgs a;
  a.tokens_old = h->d_seq_tokens(old); a.tokens_new = h->d_seq_tokens(nxt);
  a.table_old = h->d_page_table(old); a.table_new = h->d_page_table(nxt);
  a.acc_old = h->d_open_acc(old); a.acc_new = h->d_open_acc(nxt);
  a.max_pages = h->dm.max_pages; a.r = h->dm.r; a.stride = h->dm.s;
  for (int at = 0; at < n_new; at += kBeamChunk) {
    BeamParents p;
    p.n = min(kBeamChunk, n_new - at);
    p.first = at;
    for (int i = 0; i < p.n; ++i) p.parent[i] = parents[at + i];
    MTLA_CUDA(launch_kernel(beam_gather_kernel, dim3(p.n), dim3(128), 0, st, true, a, p));
    h->launches++;
  }
  h->pool->reorder(parents, n_new, h->batch);
  std::vector<int> moved(h->cfg.max_batch, 0);
  h->tokens = 0;
  for (int b = 0; b < n_new; ++b) {
    moved[b] = h->seq_tokens[parents[b]];
    h->tokens = max(h->tokens, moved[b]);
  }
  h->seq_tokens.swap(moved);
  h->batch = n_new;
  // Rows beyond the new batch keep stale positions on the device; they are re-sent (as 0) with
  // the next host-side change and are not read before.
  return MTLA_OK;
}

int mtla_seq_positions(const mtla_handle* h, int32_t* tokens, int32_t n) {
  if (!h || !tokens || n < 0 || n > h->cfg.max_batch) return MTLA_ERR_INVALID_ARG;
  for (int b = 0; b < n; ++b) tokens[b] = b < h->batch ? h->seq_len(b) : 0;
  return MTLA_OK;
}

int64_t mtla_pages_in_use(const mtla_handle* h) { return h && h->paged() ? h->pool->pages_in_use() : -1; }

int mtla_cache_export_seq(mtla_handle* h, int32_t seq, void* dst, size_t bytes, void* stream) {
  if (!h || !dst || !aligned16(dst) || seq < 0 || seq >= h->batch) return MTLA_ERR_INVALID_ARG;
  if (h->is_baseline) return MTLA_ERR_STATE;
  const int n_slots = ceil_div(h->seq_len(seq), h->dm.s);
  if (bytes < (size_t)n_slots * h->dm.W * h->dm.elem) return MTLA_ERR_CAPACITY;
  if (n_slots == 0) return MTLA_OK;
  cache_rows_copy_kernel<<<dim3(ceil_div(n_slots, kPageSlots), 1), 256, 0,
                           static_cast<cudaStream_t>(stream)>>>(
      h->cache_view(), seq, n_slots, (int)(h->dm.W * h->dm.elem), static_cast<char*>(dst), 0);
  h->launches++;
  MTLA_CUDA(cudaGetLastError());
  return MTLA_OK;
}

/* Host-only access to the page pool's decisions (no GPU involved). */
mtla_page_pool* mtla_page_pool_create(int32_t n_pages, int32_t max_seqs, int32_t max_pages_per_seq) {
  if (n_pages <= 0 || max_seqs <= 0 || max_pages_per_seq <= 0) return nullptr;
  return reinterpret_cast<mtla_page_pool*>(new (std::nothrow) PagePool(n_pages, max_seqs, max_pages_per_seq));
}
void mtla_page_pool_destroy(mtla_page_pool* p) { delete reinterpret_cast<PagePool*>(p); }
int mtla_page_pool_prepare(mtla_page_pool* pp, int32_t seq, int32_t n_slots, int32_t write_slot,
                           int32_t* copies, int32_t max_copies) {
  PagePool* p = reinterpret_cast<PagePool*>(pp);
  if (!p || seq < 0 || n_slots < 0) return MTLA_ERR_INVALID_ARG;
  if (p->pages_needed(seq, n_slots, write_slot) > p->pages_free()) return MTLA_ERR_CAPACITY;
  std::vector<PageSet> sets;
  std::vector<PageCopy> cp;
  if (!p->prepare(seq, n_slots, write_slot, &sets, &cp)) return MTLA_ERR_STATE;
  for (size_t i = 0; i < cp.size() && (int)i < max_copies; ++i) {
    copies[3 * i] = cp[i].src; copies[3 * i + 1] = cp[i].dst; copies[3 * i + 2] = cp[i].rows;
  }
  return (int)cp.size();
}
int mtla_page_pool_reorder(mtla_page_pool* pp, const int32_t* parents, int32_t n_new, int32_t n_old) {
  PagePool* p = reinterpret_cast<PagePool*>(pp);
  if (!p || !parents || n_new <= 0 || n_old <= 0) return MTLA_ERR_INVALID_ARG;
  p->reorder(parents, n_new, n_old);
  return MTLA_OK;
}
int mtla_page_pool_row(const mtla_page_pool* pp, int32_t seq, int32_t* pages, int32_t max_pages) {
  const PagePool* p = reinterpret_cast<const PagePool*>(pp);
  if (!p || seq < 0) return MTLA_ERR_INVALID_ARG;
  const int n = p->pages_held(seq);
  for (int k = 0; k < n && k < max_pages; ++k) pages[k] = p->row(seq)[k];
  return n;
}
int mtla_page_pool_in_use(const mtla_page_pool* pp) {
  const PagePool* p = reinterpret_cast<const PagePool*>(pp);
  return p ? p->pages_in_use() : MTLA_ERR_INVALID_ARG;
}
int mtla_page_pool_ref(const mtla_page_pool* pp, int32_t page) {
  const PagePool* p = reinterpret_cast<const PagePool*>(pp);
  return p && page >= 0 && page < p->n_pages() ? p->ref(page) : MTLA_ERR_INVALID_ARG;
}

int mtla_check(mtla_handle* h, void* stream) {
  if (!h) return MTLA_ERR_INVALID_ARG;
  MTLA_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  int flag[4] = {0, 0, 0, 0};
  MTLA_CUDA(cudaMemcpy(flag, h->at<char>(h->plan.err_flag), sizeof(flag), cudaMemcpyDeviceToHost));
  return flag[0] ? MTLA_ERR_DEVICE_TIMEOUT : MTLA_OK;
}

int mtla_selftest_wait_timeout(mtla_handle* h, int32_t budget_us, void* stream) {
  if (!h || budget_us < 1 || budget_us > 1000000) return MTLA_ERR_INVALID_ARG;
  int* flag = h->at<int>(h->plan.err_flag);
  wait_timeout_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(
      flag, 99, (unsigned long long)budget_us * 1000ull, flag + 1);
  h->launches++;
  MTLA_CUDA(cudaGetLastError());
  return MTLA_OK;
}

int mtla_clear_error(mtla_handle* h, void* stream) {
  if (!h) return MTLA_ERR_INVALID_ARG;
  MTLA_CUDA(cudaMemsetAsync(h->at<char>(h->plan.err_flag), 0, 16, static_cast<cudaStream_t>(stream)));
  return MTLA_OK;
}

int64_t mtla_launch_count(const mtla_handle* h) { return h ? h->launches : 0; }

int mtla_profile_begin_attention(mtla_handle* h, int32_t max_steps) {
  const int rc = mtla_profile_begin(h, max_steps);
  if (rc == MTLA_OK) h->prof_attention_only = true;
  return rc;
}

int mtla_profile_begin(mtla_handle* h, int32_t max_steps) {
  if (!h || max_steps <= 0) return MTLA_ERR_INVALID_ARG;
  h->prof_attention_only = false;
  for (cudaEvent_t e : h->prof_events) cudaEventDestroy(e);
  h->prof_events.clear();
  h->prof_used = 0;
  for (int i = 0; i < (MTLA_DECODE_STAGES + 1) * max_steps; ++i) {
    cudaEvent_t e;
    MTLA_CUDA(cudaEventCreate(&e));
    h->prof_events.push_back(e);
  }
  return MTLA_OK;
}

int mtla_profile_end_stages(mtla_handle* h, double* stage_ms, int32_t* steps) {
  if (!h || !stage_ms || !steps) return MTLA_ERR_INVALID_ARG;
  constexpr int per_step = MTLA_DECODE_STAGES + 1;
  for (int s = 0; s < MTLA_DECODE_STAGES; ++s) stage_ms[s] = 0.0;
  for (int i = 0; i + per_step <= h->prof_used; i += per_step) {
    MTLA_CUDA(cudaEventSynchronize(h->prof_events[i + MTLA_DECODE_STAGES]));
    for (int s = 0; s < MTLA_DECODE_STAGES; ++s) {
      if (h->prof_attention_only && s != MTLA_STAGE_ATTENTION) continue;
      float ms = 0.f;
      MTLA_CUDA(cudaEventElapsedTime(&ms, h->prof_events[i + s], h->prof_events[i + s + 1]));
      stage_ms[s] += ms;
    }
  }
  *steps = h->prof_used / per_step;
  for (cudaEvent_t e : h->prof_events) cudaEventDestroy(e);
  h->prof_events.clear();
  h->prof_used = 0;
  return MTLA_OK;
}

int mtla_profile_end(mtla_handle* h, double* attention_ms, int32_t* steps) {
  if (!attention_ms) return MTLA_ERR_INVALID_ARG;
  double stage_ms[MTLA_DECODE_STAGES];
  const int rc = mtla_profile_end_stages(h, stage_ms, steps);
  if (rc == MTLA_OK) *attention_ms = stage_ms[MTLA_STAGE_ATTENTION];
  return rc;
}

int32_t mtla_attention_gang(const mtla_handle* h) { return h ? h->last_gang : 0; }

const char* mtla_attention_variant(const mtla_handle* h) {
  return (h && h->use_tc) ? "tcgen05" : "fma";
}

const char* mtla_error_string(int status) {
  switch (status) {
    case MTLA_OK: return "ok";
    case MTLA_ERR_INVALID_ARG: return "invalid argument";
    case MTLA_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case MTLA_ERR_ARENA_TOO_SMALL: return "arena too small";
    case MTLA_ERR_CAPACITY: return "capacity exceeded";
    case MTLA_ERR_BATCH_MISMATCH: return "batch mismatch";
    case MTLA_ERR_CUDA: return "CUDA error";
    case MTLA_ERR_STATE: return "call not valid in this state";
    case MTLA_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case MTLA_ERR_SCRATCH_LIMIT: return "batch and layer shape need more than the built-in static scratch";
    default: return "unknown status";
  }
}

}  // extern "C"

#include "stack_api.inc"
#include "train_api.inc"
