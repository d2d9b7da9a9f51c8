// Tensor-core (tcgen05 / TMEM / TMA) split-K decode attention over the compressed cache in
// the absorbed form (Eq. 12 / Eq. 17), bf16 operands, fp32 accumulation, with the
// cross-split combine fused in.
//
// Work is cut into tiles of 64 slots.  The B * ceil(n_slots / 64) tiles of a step form one
// list (sequence-major) that is dealt out in equal contiguous shares to one persistent CTA per
// SM, so a CTA's share may end one sequence and start the next ("segments").  Each segment
// yields a partial (reference maximum, denominator, un-normalised output) and the CTA that
// delivers a sequence's last partial combines them (an atomic ticket, never a wait).
//
// A tile is brought in by TMA as 64-column sub-tiles [64 slots x 128 B] with the 128-byte
// swizzle; the SAME shared-memory bytes feed both contractions, so every cache byte is read
// from HBM exactly once per step:
//   scores  S^T[64 slots x heads]  = tile[64 x (r+d_R)] . q~^T        A = tile, K-major, M = 64
//   values  O^T[r x heads]        += tile[:, :r]^T . P^T[64 x heads]  A = tile, MN-major, M = 128
// Heads sit in the MMA's N dimension (16 or 32), so no padding of heads up to M is paid for.
// Accumulators live in TMEM: two score buffers and r/128 output blocks.  With M = 64 the score
// of slot i sits in TMEM lane 32*(i/16) + i%16, i.e. in the first 16 lanes of each warp's
// quarter; a softmax warp reads them with the two-half load shape (16x32bx2), so that its two
// half-warps own the same 16 slots and different heads and no lane idles.
//
// A score buffer is four partial accumulators: k-step ks (16 columns) of every 64-column chunk
// goes to partial ks, each partial has its own issuing thread (see below), and the softmax
// threads add the four when they read them.
//
// Shared memory: a ring of ten 16 KB "pairs" (two adjacent sub-tiles = a 128-row MN-major
// operand block) and two 8 KB sub-tiles for the RoPE-key columns (nine and three for ragged
// batches, see Layout), q~ as a K-major swizzled B operand (TMA-loaded per segment), and two
// bf16 probability buffers.  The ring holds a little more than two tiles, and a load can only
// be issued once its slot is free; to keep the DRAM
// latency off that path the producer also asks the tile after the one it is loading into L2
// (cp.async.bulk.prefetch), so the load proper is an L2 hit.
//
// The online softmax raises a head's reference maximum only when a tile exceeds it by more
// than 2^8.  The common tile therefore needs no cross-thread reduction: each thread compares
// its scores with the shared references, raises a flag if one is outgrown, and forms its
// probabilities at once; the flag is collected through a split mbarrier arrive / wait that
// overlaps that work, and only a raised flag (always at a sequence's first tile, otherwise
// rare) sends the softmax threads through the reduction, the TMEM rescale of O and a second
// exponentiation.  Results are exact either way because the same reference enters numerator
// and denominator.
//
// One thread can issue a tcgen05.mma only about every hundred cycles, far slower than these
// small-N MMAs execute, so issue is spread over eight single-thread issuers in eight warps:
// four for the scores (issuer k owns partial accumulator k) and four for the values (issuer j
// owns output block j and returns its pair to the ring as soon as its four MMAs are in).
// The softmax is instruction- and latency-bound too, so it runs on eight warps: two warps per
// TMEM quarter split the heads between them, and each warp's halves split them again.  Warp roles: warp 0 = TMA producer, warps 1-4 = score issuers,
// warps 5-8 = value issuers, warps 9-11 idle, warps 12-19 = softmax and epilogue.  The first
// three warpgroups give most of their registers to the other two (setmaxnreg).
//
// Ragged, paged batches (template parameter RAGGED): every sequence has its own length and its
// slots live in 64-slot pages of a pool, found through a per-sequence page table.  A page is a
// tile, so only the tile's TMA coordinate changes; the tile list is then B variable-length runs,
// whose prefix sums every CTA forms in shared memory before it locates its share, and the page
// numbers of the share's first tiles are staged in shared memory so that no load waits for a
// table lookup.  With a gang size (gridDim.x) above 1 the list is that of the gangs' first
// sequences, CTA (j, v) is member j of virtual CTA v and walks v's share on sequence
// entry * gang + j; partials and tickets are indexed so that each member's parts keep the
// order of the virtual CTAs.
//
// Every wait is a bounded mbarrier wait (see sm100_ptx.cuh), the rendezvous of the softmax
// threads included; on a timeout the CTA raises its abort word, all roles unwind, and the host
// sees MTLA_ERR_DEVICE_TIMEOUT from mtla_check.
#pragma once

#include <math.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mtla {

struct AttnTcArgs {
  float* o_part;       // [B + grid][n_h][r] un-normalised partial outputs
  float* ml_part;      // [B + grid][n_h][2]: reference maximum (log2 units), denominator
  bf16* o16;           // [B][2][n_h][r]: combined output as bf16 hi halves, then remainders
  int* tickets;        // [B], zero between launches
  int* error_word;
  int n_heads, r, dr, n_slots, batch;
  int tiles_per_seq;   // ceil(n_slots / 64)
  // Ragged, paged batches only (otherwise nullptr / unused):
  const int* seq_tokens;   // [B] tokens per sequence, this step's included
  const int* page_table;   // [B][max_pages] page of tile t of sequence b
  int max_pages, stride;
  // Ragged batches: `gang` consecutive sequences with equal tile counts (the beams of one
  // utterance, which share all pages but their newest) are walked by `gang` CTAs side by side,
  // one sequence each over the same tile range at the same time, so that a shared page is read
  // from DRAM once and served to the other CTAs by L2.  The ragged kernel is launched on a
  // grid (gang, virtual CTAs): blockIdx.x is the member, blockIdx.y the virtual CTA whose share
  // of the list of gangs it walks; gang 1 gives every CTA its own share of the whole list.
  int n_list;              // entries of the tile list: batch / gang
  // 0: the partials are combined by decode_combine_parts_kernel afterwards (lock-step batches
  // whose sequences are spread over many CTAs), 1: by the last CTA of each sequence.
  int fused_combine;
  int attn_grid;           // decode_combine_parts_kernel: grid size of the attention launch
};

namespace tc {

constexpr int kTile = 64;                  // slots per tile
constexpr int kThreads = 640;
constexpr int kQkIssuers = 4, kPvIssuers = 4;
constexpr int kFirstSoftmaxWarp = 12, kSoftmaxThreads = 256;
// setmaxnreg moves registers inside the pool the CTA was launched with (threads x the per-thread
// count the compiler settles on, which is the launch-bound cap rounded down to 8).  An increase
// that the pool cannot cover would block for ever, so the budget is checked here.
constexpr int kRegsIssuer = 40, kRegsSoftmax = 176;
constexpr int kRegsAtLaunch = 65536 / kThreads / 8 * 8;
static_assert((kThreads - kSoftmaxThreads) * kRegsIssuer + kSoftmaxThreads * kRegsSoftmax <=
                  kThreads * kRegsAtLaunch,
              "register re-allocation exceeds the CTA's pool");
static_assert(kFirstSoftmaxWarp % 4 == 0 && kThreads == kFirstSoftmaxWarp * 32 + kSoftmaxThreads,
              "softmax warps must start at a warpgroup boundary");
constexpr int kSubBytes = kTile * 128;     // one 64-column sub-tile
constexpr int kPairBytes = 2 * kSubBytes;
constexpr int kPrefetchAhead = 1;          // tiles asked into L2 ahead of the tile being loaded
constexpr int kTmemCols = 512;
constexpr int kSParts = 4;                 // independent partial score accumulators per buffer
constexpr int kColS = 0;                   // score buffer b, partial k at column (b * 4 + k) * 32
constexpr int kColO = 2 * kSParts * 32;    // output blocks at 256 + 32 * block
constexpr float kRescaleThreshold = 8.f;
constexpr int kSmCountMax = 256;           // upper bound on the attention grid (one CTA per SM)

constexpr int kMaxQBytes = 9 * 32 * 128;   // (2 * 4 + 1) chunks x 32 heads x 128 B
constexpr int kPBytes = 32 * kTile * 2;    // one probability buffer
constexpr int kMiscBytes = 4096;
// Ragged batches add the tile prefix sums of up to kMaxRaggedBatch sequences and the page
// numbers of the first kStagedPages tiles of the CTA's share.
constexpr int kMaxRaggedBatch = 1022;
constexpr int kStagedPages = 1024;
constexpr int kMaxPairs = 10, kMaxKrBufs = 3;

// Shared-memory layout.  The ring of latent pairs is what bounds the tiles in flight, and the time
// of a tile follows the ring's depth (measured at the largest workload: 8 / 9 / 10 pairs = 428 /
// 417 / 410 us), so lock-step batches spend the 8 KB that ragged ones need for their lists, and
// one of the three RoPE-key buffers (a RoPE-key buffer is free again as soon as its tile's first
// score MMA has been issued), on a tenth pair.
template <bool RAGGED>
struct Layout {
  static constexpr int kPairs = RAGGED ? 9 : 10;
  static constexpr int kKrBufs = RAGGED ? 3 : 2;
  static constexpr int kOffPairs = 0;
  static constexpr int kOffKr = kPairs * kPairBytes;
  static constexpr int kOffQ = kOffKr + kKrBufs * kSubBytes;
  static constexpr int kOffP = kOffQ + kMaxQBytes;
  static constexpr int kOffMisc = kOffP + 2 * kPBytes;
  static constexpr int kOffPrefix = kOffMisc + kMiscBytes;
  static constexpr int kOffStaged = kOffPrefix + (kMaxRaggedBatch + 2) * 4;
  // + slack for 1024-byte alignment
  static constexpr int kSmemBytes = (RAGGED ? kOffStaged + kStagedPages * 4 : kOffPrefix) + 1024;
  static_assert(kPairs <= kMaxPairs && kKrBufs <= kMaxKrBufs, "barrier arrays too small");
  static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
};

struct Misc {
  unsigned long long full_pair[kMaxPairs], empty_pair[kMaxPairs];
  unsigned long long full_kr[kMaxKrBufs], empty_kr[kMaxKrBufs];
  unsigned long long s_full[2], s_empty[2], p_full[2], p_empty[2], q_full, q_empty;
  unsigned long long flag_bar[2], group_sync;
  uint32_t tmem_base;
  int abort_word;
  int last_flag;
  int exceed_flag[2];      // raised by any softmax thread whose tile outgrew a reference
  float m_used[32];        // per-head reference maximum of the running segment (log2 units)
  float red[8][32];        // per-warp reductions (tile maxima / denominators) of the softmax warps
  float fac[32];
  float comb_m[32];
  float comb_w[8][32];     // combine: weight of part p for head h (first 8 parts cached)
  // Ragged batches: the tile list's length, and the segment the softmax warps are in (kept
  // here, written by one thread per segment, so that no thread carries a list position).
  long long total_tiles;
  int seg_b, seg_tiles, seg_tps, seg_start, seg_tail_rows;
  // Per-tile flags (1 = first of its segment, 2 = last) from the producer to the score issuers,
  // and "first of its segment" from the softmax warps to the value issuers, so that the issuers
  // carry no list position; both are written before the mbarrier arrival that the reader waits for.
  int tile_flags[16];
  int pv_first[2];
};
static_assert(sizeof(Misc) <= kMiscBytes, "misc region too small");

// Share of the tile list owned by CTA c of G: [c * total / G, (c + 1) * total / G).
__host__ __device__ inline long long share_begin(long long c, long long total, long long G) {
  return c * total / G;
}
// The CTA whose share contains tile g.
__host__ __device__ inline long long share_owner(long long g, long long total, long long G) {
  return ((g + 1) * G - 1) / total;
}

// Position in the tile list: tile t of sequence b, which has tps tiles.  Lock-step batches
// have tps tiles everywhere; ragged ones read the prefix sums.
template <bool RAGGED>
struct TileCursor {
  int b, t, tps;
  // `prefix` is the shared-memory address of the prefix sums (ragged batches only).
  // List index of the sequence's first tile.
  __device__ __forceinline__ long long start(uint32_t prefix) const {
    if constexpr (RAGGED) return ptx::lds_i32(prefix + 4 * b);
    else return (long long)b * tps;
  }
  __device__ __forceinline__ void locate(long long g, int tps_uniform, uint32_t prefix, int batch) {
    if constexpr (RAGGED) {
      int lo = 0, hi = batch;               // largest b with prefix[b] <= g
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (ptx::lds_i32(prefix + 4 * mid) <= g) lo = mid; else hi = mid;
      }
      b = lo;
      tps = ptx::lds_i32(prefix + 4 * b + 4) - ptx::lds_i32(prefix + 4 * b);
    } else {
      b = (int)(g / tps_uniform);
      tps = tps_uniform;
    }
    t = (int)(g - start(prefix));
  }
  __device__ __forceinline__ void next(uint32_t prefix) {
    if (++t == tps) {
      t = 0;
      ++b;
      if constexpr (RAGGED)                  // the array has one entry to spare past the batch
        tps = ptx::lds_i32(prefix + 4 * b + 4) - ptx::lds_i32(prefix + 4 * b);
    }
  }
  __device__ __forceinline__ bool seq_first() const { return t == 0; }
  __device__ __forceinline__ bool seq_last() const { return t + 1 == tps; }
};

}  // namespace tc

// NHP: heads padded to the MMA's N (16 or 32).  RP: r / 128 (pairs per tile).
template <int NHP, int RP, bool RAGGED>
__global__ void __launch_bounds__(tc::kThreads, 1)
decode_attn_tc_kernel(const __grid_constant__ CUtensorMap cache_map,
                      const __grid_constant__ CUtensorMap q_map, AttnTcArgs a) {
  using namespace tc;
  using L = Layout<RAGGED>;
  using namespace ptx;
  constexpr int NCH = 2 * RP + 1;                // 64-column chunks of q~ (latent + RoPE)
  constexpr uint32_t QCHUNK = NHP * 128;         // bytes of one q~ chunk
  constexpr uint32_t IDESC_QK = make_idesc_bf16(64, NHP, 0, 0);
  constexpr uint32_t IDESC_PV = make_idesc_bf16(128, NHP, 1, 0);
  constexpr uint32_t PSBO = (kTile / 8) * 128;   // bytes between 8-head groups of P^T

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  Misc* misc = reinterpret_cast<Misc*>(sm + L::kOffMisc);
  volatile int* abort_word = &misc->abort_word;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  auto bar = [&](unsigned long long* p) { return smem_u32(p); };

  if (threadIdx.x == 0) {
    for (int i = 0; i < L::kPairs; ++i) {
      mbar_init(bar(&misc->full_pair[i]), 1);
      mbar_init(bar(&misc->empty_pair[i]), 1);
    }
    for (int i = 0; i < L::kKrBufs; ++i) {
      mbar_init(bar(&misc->full_kr[i]), 1);
      mbar_init(bar(&misc->empty_kr[i]), kQkIssuers);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(&misc->s_full[i]), kQkIssuers);
      mbar_init(bar(&misc->s_empty[i]), kSoftmaxThreads);
      mbar_init(bar(&misc->p_full[i]), kSoftmaxThreads);
      mbar_init(bar(&misc->p_empty[i]), kPvIssuers);
    }
    mbar_init(bar(&misc->q_full), 1);
    mbar_init(bar(&misc->q_empty), kQkIssuers);
    mbar_init(bar(&misc->flag_bar[0]), kSoftmaxThreads);
    mbar_init(bar(&misc->flag_bar[1]), kSoftmaxThreads);
    mbar_init(bar(&misc->group_sync), kSoftmaxThreads);
    misc->abort_word = 0;
    misc->last_flag = 0;
    misc->exceed_flag[0] = 0;
    misc->exceed_flag[1] = 0;
    mbar_fence_init();
    prefetch_tensormap(&cache_map);
    prefetch_tensormap(&q_map);
  }
  if (warp == 1) tmem_alloc(smem_u32(&misc->tmem_base), kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = misc->tmem_base;
  // Only now may the next kernel's CTAs start: this CTA owns its TMEM columns, so a successor
  // that shares the SM cannot take them first and then sit in its dependency wait.
  grid_launch_dependents();
  grid_dependency_wait();        // nothing before this line touches the previous kernel's data

  // This CTA's share of the tile list.
  const uint32_t prefix_s = base + L::kOffPrefix, staged_s = base + L::kOffStaged;   // ragged only
  long long total = (long long)a.batch * a.tiles_per_seq;
  // Lock-step batches: a 1-D grid.  Ragged ones: (gang member, virtual CTA), all of them special
  // registers, so that no thread carries them through its loop.
  const int gang = RAGGED ? gridDim.x : 1;
  const int vcta = RAGGED ? blockIdx.y : blockIdx.x, member = RAGGED ? blockIdx.x : 0;
  const int n_list = RAGGED ? a.n_list : a.batch;   // entries of the tile list (sequences or gangs)
  if constexpr (RAGGED) {
    // prefix[b] = tiles of the sequences before b; prefix[batch + 1] repeats the total.
    int* prefix = reinterpret_cast<int*>(sm + L::kOffPrefix);
    for (int i = threadIdx.x; i < n_list; i += kThreads)
      prefix[i + 1] = ceil_div(ceil_div(a.seq_tokens[i * gang], a.stride), kTile);
    __syncthreads();
    if (warp == 0) {
      const int per = ceil_div(n_list, 32);
      const int lo = min(n_list, lane * per), hi = min(n_list, lo + per);
      int sum = 0;
      for (int i = lo; i < hi; ++i) sum += prefix[i + 1];
      int incl = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      int run = incl - sum;
      for (int i = lo; i < hi; ++i) {
        run += prefix[i + 1];
        prefix[i + 1] = run;
      }
      if (lane == 0) prefix[0] = 0;
    }
    __syncthreads();
    total = prefix[n_list];
    if (threadIdx.x == 0) {
      prefix[n_list + 1] = (int)total;
      misc->total_tiles = total;
    }
  }
  const long long G = RAGGED ? gridDim.y : gridDim.x;     // (virtual) CTAs that share the list
  const long long g0 = share_begin(vcta, total, G), g1 = share_begin(vcta + 1, total, G);
  const int n_tiles = (int)(g1 - g0);
  const int tps_u = a.tiles_per_seq;
  if constexpr (RAGGED) {
    int* staged = reinterpret_cast<int*>(sm + L::kOffStaged);
    for (int n = threadIdx.x; n < min(n_tiles, kStagedPages); n += kThreads) {
      TileCursor<true> c;
      c.locate(g0 + n, 0, prefix_s, n_list);
      staged[n] = a.page_table[(long long)(c.b * gang + member) * a.max_pages + c.t];
    }
    __syncthreads();
  }

  const uint32_t pairs_u32 = base + L::kOffPairs, kr_u32 = base + L::kOffKr;
  const uint32_t q_u32 = base + L::kOffQ, p_u32 = base + L::kOffP;

  if (warp < kFirstSoftmaxWarp) {
  // Register budget: the producer / issuer warpgroups keep 40 registers, the softmax ones get 176.
  reg_dealloc<kRegsIssuer>();
  if (warp == 0 && lane == 0) {
    // ------------------------------------------------------------------ TMA producer
    bool ok = true;
    int pc = 0, seg = 0;
    TileCursor<RAGGED> cur, ahead;
    cur.locate(g0, tps_u, prefix_s, n_list);
    ahead = cur;
    // TMA coordinates (slot, plane) of a tile: its place in the sequence's row range, or its page.
    auto tile_coords = [&](const TileCursor<RAGGED>& c, int n, int& c_slot, int& c_plane) {
      if constexpr (RAGGED) {
        c_slot = 0;
        c_plane = n < kStagedPages ? lds_i32(staged_s + 4 * n)
                                   : __ldg(a.page_table + (long long)(c.b * gang + member) * a.max_pages + c.t);
      } else {
        c_slot = c.t * kTile;
        c_plane = c.b;
      }
    };
    // The ring holds little more than two tiles, too few to cover the DRAM latency of a load
    // that can only be issued once its slot is free.  So tiles are first asked into L2, a few
    // tiles ahead; the load proper then finds them there.
    // Called for n_ahead = 0, 1, 2, ... in turn: `ahead` walks the list with it.
    auto prefetch_tile = [&](int n_ahead) {
      if (n_ahead >= n_tiles) return;
      int slot, plane;
      tile_coords(ahead, n_ahead, slot, plane);
      for (int c = 0; c < 2 * RP + 1; ++c) tma_prefetch_l2_3d(&cache_map, c * 64, slot, plane);
      ahead.next(prefix_s);
    };
    for (int n = 0; n < kPrefetchAhead; ++n) prefetch_tile(n);
    for (int n = 0; n < n_tiles && ok; ++n, cur.next(prefix_s)) {
      prefetch_tile(n + kPrefetchAhead);
      if (n == 0 || cur.seq_first()) {
        const int b = cur.b * gang + member;
        // A segment starts: q~ of sequence b, once the previous segment's score MMAs are done.
        ok = mbar_wait(bar(&misc->q_empty), (seg & 1) ^ 1, abort_word, a.error_word, 1);
        if (!ok) break;
        mbar_arrive_expect_tx(bar(&misc->q_full), NCH * QCHUNK);
        for (int ch = 0; ch < NCH; ++ch)
          tma_load_3d(q_u32 + ch * QCHUNK, &q_map, bar(&misc->q_full), ch * 64, 0, b);
        ++seg;
      }
      int slot, plane;
      tile_coords(cur, n, slot, plane);
      const int kb = n % L::kKrBufs;
      ok = mbar_wait(bar(&misc->empty_kr[kb]), ((n / L::kKrBufs) & 1) ^ 1, abort_word, a.error_word, 2);
      if (!ok) break;
      misc->tile_flags[n & 15] = ((n == 0 || cur.seq_first()) ? 1 : 0) |
                                 ((n + 1 == n_tiles || cur.seq_last()) ? 2 : 0);
      mbar_arrive_expect_tx(bar(&misc->full_kr[kb]), kSubBytes);
      tma_load_3d(kr_u32 + kb * kSubBytes, &cache_map, bar(&misc->full_kr[kb]), a.r, slot, plane);
      for (int c = 0; c < RP && ok; ++c, ++pc) {
        const int buf = pc % L::kPairs;
        ok = mbar_wait(bar(&misc->empty_pair[buf]), ((pc / L::kPairs) & 1) ^ 1, abort_word,
                       a.error_word, 3);
        if (!ok) break;
        const uint32_t dst = pairs_u32 + buf * kPairBytes;
        mbar_arrive_expect_tx(bar(&misc->full_pair[buf]), kPairBytes);
        tma_load_3d(dst, &cache_map, bar(&misc->full_pair[buf]), c * 128, slot, plane);
        tma_load_3d(dst + kSubBytes, &cache_map, bar(&misc->full_pair[buf]), c * 128 + 64, slot, plane);
      }
    }
  } else if (warp >= 1 && warp <= kQkIssuers && lane == 0) {
    // ------------------------------------------------------------------ score issuer k
    // Issuer k multiplies k-step k (16 columns) of every 64-column chunk into partial k.
    const int k = warp - 1;
    bool ok = true;
    int seg = 0;
    for (int n = 0; n < n_tiles && ok; ++n) {
      const uint32_t d_tmem = tmem_base + kColS + (n & 1) * (kSParts * 32) + k * 32;
      auto qk = [&](uint32_t a_smem, int chunk, uint32_t accumulate) {
        const uint64_t ad = make_smem_desc(a_smem + k * 32, 16, 1024, kSwizzle128B);
        const uint64_t bd = make_smem_desc(q_u32 + chunk * QCHUNK + k * 32, 16, 1024, kSwizzle128B);
        mma_bf16_ss(d_tmem, ad, bd, IDESC_QK, accumulate);
      };
      const int kb = n % L::kKrBufs;
      ok = mbar_wait(bar(&misc->s_empty[n & 1]), ((n >> 1) & 1) ^ 1, abort_word, a.error_word, 9) &&
           mbar_wait(bar(&misc->full_kr[kb]), (n / L::kKrBufs) & 1, abort_word, a.error_word, 10);
      if (!ok) break;
      const int flags = *reinterpret_cast<volatile int*>(&misc->tile_flags[n & 15]);
      const bool seg_last = flags & 2;
      if (flags & 1) {                   // a segment starts: its q~ must have landed
        ok = mbar_wait(bar(&misc->q_full), seg & 1, abort_word, a.error_word, 4);
        if (!ok) break;
        ++seg;
      }
      tc_fence_after_sync();
      qk(kr_u32 + kb * kSubBytes, 2 * RP, 0u);
      mma_commit(bar(&misc->empty_kr[kb]));
      for (int c = 0; c < RP && ok; ++c) {
        const int pcn = n * RP + c, buf = pcn % L::kPairs;
        ok = mbar_wait(bar(&misc->full_pair[buf]), (pcn / L::kPairs) & 1, abort_word, a.error_word, 11);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t src = pairs_u32 + buf * kPairBytes;
        qk(src, 2 * c, 1u);
        qk(src + kSubBytes, 2 * c + 1, 1u);
      }
      if (!ok) break;
      mma_commit(bar(&misc->s_full[n & 1]));
      if (seg_last) mma_commit(bar(&misc->q_empty));
    }
  } else if (warp > kQkIssuers && warp <= kQkIssuers + kPvIssuers && lane == 0) {
    // ------------------------------------------------------------------ value issuer j
    // Issuer j accumulates the output blocks mb = j, j + 2, ... once a tile's probabilities
    // are published, and hands the pairs it read back to the producer.
    const int j = warp - 1 - kQkIssuers;
    bool ok = true;
    for (int n = 0; n < n_tiles && ok; ++n) {
      ok = mbar_wait(bar(&misc->p_full[n & 1]), (n >> 1) & 1, abort_word, a.error_word, 12);
      if (!ok) break;
      tc_fence_after_sync();
      const bool seg_first = *reinterpret_cast<volatile int*>(&misc->pv_first[n & 1]) != 0;
      for (int mb = j; mb < RP; mb += kPvIssuers) {
        const int buf = (n * RP + mb) % L::kPairs;
        const uint32_t src = pairs_u32 + buf * kPairBytes;
#pragma unroll
        for (int ks = 0; ks < kTile / 16; ++ks) {
          const uint64_t bd = make_smem_desc(p_u32 + (n & 1) * kPBytes + ks * 256, 128, PSBO, kSwizzleNone);
          const uint64_t ad = make_smem_desc(src + ks * 2048, kSubBytes, 1024, kSwizzle128B);
          mma_bf16_ss(tmem_base + kColO + mb * 32, ad, bd, IDESC_PV, (seg_first && ks == 0) ? 0u : 1u);
        }
        mma_commit(bar(&misc->empty_pair[buf]));      // the pair goes back to the producer at once
      }
      mma_commit(bar(&misc->p_empty[n & 1]));
    }
  }
  } else {
    // ------------------------------------------------------------------ softmax / epilogue warps
    // Two groups of four warps; group g owns heads [g * NHH, (g + 1) * NHH) of every slot, i.e.
    // TMEM columns g * NHH .. of each score partial and of each output block.  The scores of a
    // tile sit in the first 16 lanes of each TMEM quarter (M = 64); the two halves of a warp
    // read the same 16 slots and split the group's heads again (NQ each), so all lanes work.
    reg_alloc<kRegsSoftmax>();
    constexpr int NHH = NHP / 2, NQ = NHH / 2;
    const int sw = warp - kFirstSoftmaxWarp;                // 0..7
    const int g = sw >> 2, q = warp & 3;                    // head group; TMEM lane quarter
    const int HO = g * NHH;
    const int HQ = HO + (lane >> 4) * NQ;                   // first head of this thread's scores
    const int sidx = sw * 32 + lane;                        // index among the 256
    const int row = q * 16 + (lane & 15);                   // slot within the tile
    const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16) + HO;
    bool ok = true;
    auto ld_cols = [&](uint32_t addr, uint32_t (&v)[16]) {
      if (NHH == 16) tmem_ld_x16(addr, v); else tmem_ld_x8(addr, v);
    };
    auto st_cols = [&](uint32_t addr, const uint32_t (&v)[16]) {
      if (NHH == 16) tmem_st_x16(addr, v); else tmem_st_x8(addr, v);
    };
    // Rendezvous of the 256 threads on an mbarrier, so that it is bounded like every other wait.
    int sync_phase = 0;
    auto group_sync = [&]() {
      mbar_arrive(bar(&misc->group_sync));
      if (ok) ok = mbar_wait(bar(&misc->group_sync), sync_phase & 1, abort_word, a.error_word, 13);
      ++sync_phase;
    };
    // Per-warp reduction of one value per owned head over the 16 slots of the warp (each half
    // of the warp holds NQ heads), left in misc->red[sw][i] for head HO + i.
    auto reduce_heads = [&](const float (&v)[NQ], bool is_max) {
#pragma unroll
      for (int i = 0; i < NQ; ++i) {
        float x = v[i];
#pragma unroll
        for (int o = 8; o >= 1; o >>= 1) {
          const float y = __shfl_xor_sync(0xffffffffu, x, o);
          x = is_max ? fmaxf(x, y) : x + y;
        }
        if ((lane & 15) == 0) misc->red[sw][(lane >> 4) * NQ + i] = x;
      }
    };
    // Head h's value combined over the four warps of the group that owns it.
    auto reduced = [&](int h, bool is_max) {
      const int gg = h / NHH, i = h % NHH;
      const float* r0 = &misc->red[gg * 4][i];
      return is_max ? fmaxf(fmaxf(r0[0], r0[32]), fmaxf(r0[64], r0[96])) : r0[0] + r0[32] + r0[64] + r0[96];
    };
    float l_acc[NQ];
    TileCursor<false> cur;             // lock-step batches: every thread walks the list
    if constexpr (!RAGGED) cur.locate(g0, tps_u, prefix_s, n_list);
    int seg_left = 0;                  // ragged batches: tiles left in the running segment
    for (int n = 0; n < n_tiles; ++n) {
      bool seg_first, seg_last;
      if constexpr (RAGGED) {
        seg_first = seg_left == 0;
        if (seg_first && sidx == 0) {
          // One thread finds the segment that starts at tile n and describes it in shared memory.
          TileCursor<true> c;
          c.locate(g0 + n, 0, prefix_s, n_list);
          const int tiles = min(n_tiles - n, c.tps - c.t);
          const int seq_slots = ceil_div(__ldg(a.seq_tokens + c.b * gang + member), a.stride);
          misc->seg_b = c.b;
          misc->seg_tiles = tiles;
          misc->seg_tps = c.tps;
          misc->seg_start = (int)c.start(prefix_s);
          misc->seg_tail_rows = c.t + tiles == c.tps ? seq_slots - (c.tps - 1) * kTile : kTile;
        }
      } else {
        seg_first = n == 0 || cur.seq_first();
      }
      if (seg_first) {
        // New sequence: empty references (shared by all threads) and denominators.
        if (sidx < 32) misc->m_used[sidx] = -INFINITY;
#pragma unroll
        for (int i = 0; i < NQ; ++i) l_acc[i] = 0.f;
        group_sync();
        if constexpr (RAGGED) seg_left = misc->seg_tiles;
      }
      int rows_valid;                  // slots of this tile that exist
      if constexpr (RAGGED) {
        seg_last = seg_left == 1;
        --seg_left;
        rows_valid = seg_last ? misc->seg_tail_rows : kTile;
      } else {
        seg_last = n + 1 == n_tiles || cur.seq_last();
        rows_valid = a.n_slots - cur.t * kTile;
        cur.next(prefix_s);
      }
      float s[NQ];
#pragma unroll
      for (int i = 0; i < NQ; ++i) s[i] = 0.f;
      if (ok) ok = mbar_wait(bar(&misc->s_full[n & 1]), (n >> 1) & 1, abort_word, a.error_word, 5);
      ok = __all_sync(0xffffffffu, ok);             // TMEM accesses are whole-warp operations
      if (ok) {
        tc_fence_after_sync();
        const uint32_t s_addr = lane_base + kColS + (n & 1) * (kSParts * 32);
        uint32_t sp[kSParts][8];
#pragma unroll
        for (int k = 0; k < kSParts; ++k) {
          if (NQ == 8) tmem_ld_16x2_x8<NQ>(s_addr + k * 32, sp[k]);
          else tmem_ld_16x2_x4<NQ>(s_addr + k * 32, sp[k]);
        }
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < NQ; ++i)                // the score is the sum of the partials
          s[i] = (__uint_as_float(sp[0][i]) + __uint_as_float(sp[1][i])) +
                 (__uint_as_float(sp[2][i]) + __uint_as_float(sp[3][i]));
        tc_fence_before_sync();
      }
      const bool valid = ok && row < rows_valid;
      float m_ref[NQ];
      bool exceed = false;
#pragma unroll
      for (int i = 0; i < NQ; ++i) {
        m_ref[i] = misc->m_used[HQ + i];
        s[i] = valid ? s[i] : -INFINITY;
        exceed |= s[i] > m_ref[i] + kRescaleThreshold;
      }
      // Tell the others (rarely) that a reference must rise; the answer is collected further
      // down, after the probabilities have been formed with the current references.
      if (exceed) misc->exceed_flag[n & 1] = 1;
      mbar_arrive(bar(&misc->flag_bar[n & 1]));
      if (ok) mbar_arrive(bar(&misc->s_empty[n & 1]));

      uint32_t pb[NQ / 2];
      auto probabilities = [&]() {
#pragma unroll
        for (int i = 0; i < NQ; i += 2) {
          const __nv_bfloat162 pk = __floats2bfloat162_rn(ex2_approx(s[i] - m_ref[i]),
                                                          ex2_approx(s[i + 1] - m_ref[i + 1]));
          pb[i / 2] = *reinterpret_cast<const uint32_t*>(&pk);
        }
      };
      // P^T as the K-major, un-swizzled B operand of the value MMA: element (head h, slot k)
      // at (h/8)*PSBO + (k/8)*128 + (h%8)*16 + (k%8)*2.
      auto store_probabilities = [&]() {
        uint8_t* prow = sm + L::kOffP + (n & 1) * kPBytes + (row >> 3) * 128 + (row & 7) * 2;
#pragma unroll
        for (int i = 0; i < NQ; ++i) {
          const int h = HQ + i;
          const uint16_t bits = (i & 1) ? (uint16_t)(pb[i / 2] >> 16) : (uint16_t)(pb[i / 2] & 0xffffu);
          *reinterpret_cast<uint16_t*>(prow + (h >> 3) * PSBO + (h & 7) * 16) = bits;
        }
      };
      probabilities();
      // The probability buffer is free once the value MMAs of tile n - 2 have completed.
      if (ok) ok = mbar_wait(bar(&misc->p_empty[n & 1]), ((n >> 1) & 1) ^ 1, abort_word, a.error_word, 7);
      if (ok && sidx == 0) misc->pv_first[n & 1] = seg_first;
      if (ok) store_probabilities();
      if (ok) ok = mbar_wait(bar(&misc->flag_bar[n & 1]), (n >> 1) & 1, abort_word, a.error_word, 14);
      if (ok && misc->exceed_flag[n & 1]) {
        // ---- rare: some head's scores rose more than 2^8 above its reference (always at
        // a sequence's first tile).  Everybody takes this branch: the flag is read after all
        // arrivals.  New references, rescaled denominators and accumulators, new P.
        reduce_heads(s, true);
        group_sync();
        if (sidx == 0) misc->exceed_flag[n & 1] = 0;
        if (sidx < NHP) {
          const float mt = reduced(sidx, true);
          const float m_old = misc->m_used[sidx];
          const float m_nw = mt > m_old + kRescaleThreshold ? mt : m_old;
          misc->m_used[sidx] = m_nw;
          misc->fac[sidx] = (m_nw == m_old) ? 1.f : exp2f(m_old - m_nw);   // 0 from -inf
        }
        group_sync();
#pragma unroll
        for (int i = 0; i < NQ; ++i) {
          m_ref[i] = misc->m_used[HQ + i];
          l_acc[i] *= misc->fac[HQ + i];
        }
        if (!seg_first) {
          // O holds contributions scaled to the old references: wait for the previous tile's
          // value MMAs, then rescale this group's accumulator columns in TMEM.
          if (ok) ok = mbar_wait(bar(&misc->p_empty[(n - 1) & 1]), ((n - 1) >> 1) & 1, abort_word,
                                 a.error_word, 6);
          ok = __all_sync(0xffffffffu, ok);
          if (ok) {
            tc_fence_after_sync();
            for (int mb = 0; mb < RP; ++mb) {
              uint32_t ov[16];
              const uint32_t addr = lane_base + kColO + mb * 32;
              ld_cols(addr, ov);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < NHH; ++i)
                ov[i] = __float_as_uint(__uint_as_float(ov[i]) * misc->fac[HO + i]);
              st_cols(addr, ov);
            }
            tmem_wait_st();
          }
        }
        probabilities();
        if (ok) store_probabilities();
        group_sync();                         // fac / red may be rewritten by the next rare tile
      }
#pragma unroll
      for (int i = 0; i < NQ; i += 2) {
        const __nv_bfloat162 pk = *reinterpret_cast<const __nv_bfloat162*>(&pb[i / 2]);
        l_acc[i] += __low2float(pk);
        l_acc[i + 1] += __high2float(pk);
      }
      if (ok) {
        fence_proxy_async_smem();
        tc_fence_before_sync();
        mbar_arrive(bar(&misc->p_full[n & 1]));
      }

      if (!seg_last) continue;
      // ---------------------------------------------------------------- end of a segment
      // Partial of sequence b: wait for the last value MMAs, read O^T from TMEM.
      int b, seq_tiles;                // b: list entry (the sequence, or its gang)
      long long seq_start;
      if constexpr (RAGGED) {          // read before the first rendezvous below
        b = misc->seg_b;
        seq_tiles = misc->seg_tps;
        seq_start = misc->seg_start;
      } else {                         // cur has already moved on to the next tile
        b = cur.t == 0 ? cur.b - 1 : cur.b;
        seq_tiles = tps_u;
        seq_start = (long long)b * tps_u;
      }
      const int seq = b * gang + member;
      // Unique per (CTA, sequence); a sequence's parts follow one another `gang` entries apart.
      const long long part = ((long long)vcta + b) * gang + member;
      if (ok) ok = mbar_wait(bar(&misc->p_empty[n & 1]), (n >> 1) & 1, abort_word, a.error_word, 8);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        tc_fence_after_sync();
        float* o_part = a.o_part + part * a.n_heads * a.r;
        for (int mb = 0; mb < RP; ++mb) {
          uint32_t ov[16];
          ld_cols(lane_base + kColO + mb * 32, ov);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < NHH; ++i)
            if (HO + i < a.n_heads) o_part[(HO + i) * a.r + mb * 128 + q * 32 + lane] = __uint_as_float(ov[i]);
        }
        tc_fence_before_sync();
      }
      reduce_heads(l_acc, false);
      __threadfence();
      group_sync();
      if (ok && sidx < a.n_heads) {
        a.ml_part[(part * a.n_heads + sidx) * 2] = misc->m_used[sidx];
        a.ml_part[(part * a.n_heads + sidx) * 2 + 1] = reduced(sidx, false);
        __threadfence();
      }
      // Ticket: the CTA that delivers the sequence's last partial combines them.
      const long long list_len = RAGGED ? misc->total_tiles : total;
      const long long c_first = share_owner(seq_start, list_len, G);
      const int n_parts = (int)(share_owner(seq_start + seq_tiles - 1, list_len, G) - c_first) + 1;
      group_sync();
      if (!a.fused_combine) continue;        // a separate launch combines (uniform over the CTA)
      if (sidx == 0) {
        int last = 0;
        if (ok) {
          const int old = atomicAdd(a.tickets + seq, 1);
          last = old == n_parts - 1;
          if (last) a.tickets[seq] = 0;
        }
        misc->last_flag = last;
      }
      group_sync();
      if (ok && misc->last_flag) {
        __threadfence();
        const long long part0 = (c_first + b) * gang + member;
        // Per head: global reference, each part's weight 2^(m_p - m) and the denominator.  All
        // loops over the parts keep kU loads in flight: a sequence spread over many CTAs (a small
        // batch with a long context) has tens of parts, and one load at a time would make this
        // the longest phase of the kernel.
        constexpr int kU = 8;
        if (sidx < a.n_heads) {
          const float* ml0 = a.ml_part + (part0 * a.n_heads + sidx) * 2;
          const long long ml_step = 2ll * a.n_heads * gang;
          float m = -INFINITY;
          for (int p0 = 0; p0 < n_parts; p0 += kU) {
            float mv[kU];
#pragma unroll
            for (int u = 0; u < kU; ++u) mv[u] = p0 + u < n_parts ? __ldcg(ml0 + (p0 + u) * ml_step) : -INFINITY;
#pragma unroll
            for (int u = 0; u < kU; ++u) m = fmaxf(m, mv[u]);
          }
          float denom = 0.f;
          for (int p0 = 0; p0 < n_parts; p0 += kU) {
            float mv[kU], lv[kU];
#pragma unroll
            for (int u = 0; u < kU; ++u) {
              const bool in = p0 + u < n_parts;
              mv[u] = in ? __ldcg(ml0 + (p0 + u) * ml_step) : -INFINITY;
              lv[u] = in ? __ldcg(ml0 + (p0 + u) * ml_step + 1) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < kU; ++u) {
              if (p0 + u >= n_parts) break;
              const float wgt = exp2f(mv[u] - m);
              denom += wgt * lv[u];
              if (p0 + u < 8) misc->comb_w[p0 + u][sidx] = wgt;
            }
          }
          misc->fac[sidx] = 1.f / denom;
          misc->comb_m[sidx] = m;
        }
        group_sync();
        // Thread (cg, hh): latent columns 4*cg .. 4*cg+3 of the heads hh, hh + lanes, ...
        const int col_groups = a.r >> 2, lanes = kSoftmaxThreads / col_groups;
        const int cg = sidx % col_groups, hh = sidx / col_groups;
        if (ok && hh < lanes) {
          bf16* o_hi = a.o16 + (long long)seq * 2 * a.n_heads * a.r + 4 * cg;
          bf16* o_lo = o_hi + (long long)a.n_heads * a.r;
          const long long o_step = (long long)a.n_heads * a.r * gang, ml_step = 2ll * a.n_heads * gang;
          for (int h = hh; h < a.n_heads; h += lanes) {
            const float* o0 = a.o_part + (part0 * a.n_heads + h) * a.r + 4 * cg;
            const float* ml0 = a.ml_part + (part0 * a.n_heads + h) * 2;
            const float m = misc->comb_m[h];
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int p0 = 0; p0 < n_parts; p0 += kU) {
              float4 v[kU];
              float wg[kU];
#pragma unroll
              for (int u = 0; u < kU; ++u) {
                const int pt = p0 + u;
                if (pt < n_parts) {
                  v[u] = __ldcg(reinterpret_cast<const float4*>(o0 + pt * o_step));
                  wg[u] = pt < 8 ? misc->comb_w[pt][h] : __ldcg(ml0 + pt * ml_step);
                } else {
                  v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                  wg[u] = -INFINITY;
                }
              }
#pragma unroll
              for (int u = 0; u < kU; ++u) {
                const int pt = p0 + u;
                if (pt >= n_parts) break;
                const float wgt = pt < 8 ? wg[u] : exp2f(wg[u] - m);
                acc.x = fmaf(wgt, v[u].x, acc.x); acc.y = fmaf(wgt, v[u].y, acc.y);
                acc.z = fmaf(wgt, v[u].z, acc.z); acc.w = fmaf(wgt, v[u].w, acc.w);
              }
            }
            const float inv = misc->fac[h];
            const float val[4] = {acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv};
            const __nv_bfloat162 h0 = __floats2bfloat162_rn(val[0], val[1]);
            const __nv_bfloat162 h1 = __floats2bfloat162_rn(val[2], val[3]);
            const __nv_bfloat162 l0 = __floats2bfloat162_rn(val[0] - __low2float(h0), val[1] - __high2float(h0));
            const __nv_bfloat162 l1 = __floats2bfloat162_rn(val[2] - __low2float(h1), val[3] - __high2float(h1));
            *reinterpret_cast<uint2*>(o_hi + (long long)h * a.r) =
                make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
            *reinterpret_cast<uint2*>(o_lo + (long long)h * a.r) =
                make_uint2(*reinterpret_cast<const uint32_t*>(&l0), *reinterpret_cast<const uint32_t*>(&l1));
          }
        }
        group_sync();   // comb_w / fac are reused by the next segment
      }
    }
  }

  __syncthreads();
  if (*abort_word) {
    // Give copies that may still be in flight time to land before the CTA's memory is reused.
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 100000ull) __nanosleep(1000);
  }
  if (warp == 1) {
    __syncwarp();
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// Combine of the attention partials as a launch of its own, grid (n_h, B), 128 threads: used
// for lock-step batches in which a sequence is spread over many CTAs (a small batch with a long
// context), where one CTA reading every part of a sequence would be the kernel's longest phase.
// Same arithmetic, in the same order, as the fused combine.
__global__ void __launch_bounds__(128) decode_combine_parts_kernel(AttnTcArgs a) {
  using namespace tc;
  __shared__ float w_s[kSmCountMax];
  __shared__ float red_s[33];
  const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();
  const long long tps = a.tiles_per_seq, total = (long long)a.batch * tps, G = a.attn_grid;
  const long long c_first = share_owner((long long)b * tps, total, G);
  const int n_parts = (int)(share_owner((long long)(b + 1) * tps - 1, total, G) - c_first) + 1;
  const long long part0 = c_first + b;
  const float* ml0 = a.ml_part + (part0 * a.n_heads + h) * 2;
  const long long ml_step = 2ll * a.n_heads, o_step = (long long)a.n_heads * a.r;
  // Reference maximum, weights and denominator of head h (n_parts <= grid size <= kSmCountMax).
  float m = -INFINITY;
  for (int pt = tid; pt < n_parts; pt += 128) m = fmaxf(m, __ldcg(ml0 + pt * ml_step));
  m = warp_max(m);
  if ((tid & 31) == 0) red_s[tid >> 5] = m;
  __syncthreads();
  m = fmaxf(fmaxf(red_s[0], red_s[1]), fmaxf(red_s[2], red_s[3]));
  for (int pt = tid; pt < n_parts; pt += 128) w_s[pt] = exp2f(__ldcg(ml0 + pt * ml_step) - m);
  __syncthreads();
  if (tid == 0) {
    float denom = 0.f;
    for (int pt = 0; pt < n_parts; ++pt) denom += w_s[pt] * __ldcg(ml0 + pt * ml_step + 1);   // part order
    red_s[32] = 1.f / denom;
  }
  __syncthreads();
  const float inv = red_s[32];
  if (4 * tid >= a.r) return;
  constexpr int kU = 8;
  const float* o0 = a.o_part + (part0 * a.n_heads + h) * a.r + 4 * tid;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int p0 = 0; p0 < n_parts; p0 += kU) {
    float4 v[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u)
      v[u] = p0 + u < n_parts ? __ldcg(reinterpret_cast<const float4*>(o0 + (p0 + u) * o_step))
                              : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      if (p0 + u >= n_parts) break;
      const float wgt = w_s[p0 + u];
      acc.x = fmaf(wgt, v[u].x, acc.x); acc.y = fmaf(wgt, v[u].y, acc.y);
      acc.z = fmaf(wgt, v[u].z, acc.z); acc.w = fmaf(wgt, v[u].w, acc.w);
    }
  }
  const float val[4] = {acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv};
  const __nv_bfloat162 h0 = __floats2bfloat162_rn(val[0], val[1]);
  const __nv_bfloat162 h1 = __floats2bfloat162_rn(val[2], val[3]);
  const __nv_bfloat162 l0 = __floats2bfloat162_rn(val[0] - __low2float(h0), val[1] - __high2float(h0));
  const __nv_bfloat162 l1 = __floats2bfloat162_rn(val[2] - __low2float(h1), val[3] - __high2float(h1));
  bf16* o_hi = a.o16 + ((long long)b * 2 * a.n_heads + h) * a.r + 4 * tid;
  bf16* o_lo = o_hi + (long long)a.n_heads * a.r;
  *reinterpret_cast<uint2*>(o_hi) =
      make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
  *reinterpret_cast<uint2*>(o_lo) =
      make_uint2(*reinterpret_cast<const uint32_t*>(&l0), *reinterpret_cast<const uint32_t*>(&l1));
}

}  // namespace mtla
