/*
 * mtla.h: C ABI of the B200 (sm_100a) Multi-head Temporal Latent Attention library.
 *
 * One handle is one MTLA attention layer (Section 4 of the paper) together with the
 * compressed temporal-latent cache of a batch of sequences that advance in lock-step.
 * Notation follows the paper: d (model dim), n_h heads of d_h, latent rank r, decoupled
 * RoPE dim d_h^R (written d_R here), temporal stride s, hyper-network width d_w.
 *
 * Conventions for every call
 *   - Returns MTLA_OK (0) or a negative mtla_status.  Argument errors are detected before
 *     anything is enqueued and leave the handle unchanged.
 *   - "device" pointers are CUDA device addresses, 16-byte aligned; "host" pointers are
 *     ordinary host addresses.  `stream` is a cudaStream_t passed as void* (NULL = the
 *     legacy default stream).  Calls enqueue work on `stream` and return; the caller
 *     synchronises.  Calls on one handle must be issued in order on one stream.  The
 *     kernels of a decode step are programmatic dependent launches: one may begin (its
 *     set-up only) while earlier work on the stream is still finishing, but none reads or
 *     writes memory before all earlier work on the stream, the caller's included, is complete,
 *     so stream order holds for every buffer.
 *   - Ownership: the caller owns x, y, the weight buffers (may be freed once mtla_create
 *     has completed on its stream) and the arena (must outlive the handle and must not be
 *     touched while the handle lives).  The library owns only the host-side handle.
 *     Nothing here calls cudaMalloc: all device memory is carved from the arena.
 *   - Element type of x, y, weights and cache is config.dtype (fp32 or bf16); reductions
 *     are fp32.  Matrices are row-major.
 */
#ifndef MTLA_H_
#define MTLA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mtla_handle mtla_handle;

typedef enum {
  MTLA_OK = 0,
  MTLA_ERR_INVALID_ARG = -1,      /* null pointer, misaligned pointer, non-positive size */
  MTLA_ERR_UNSUPPORTED_SHAPE = -2,/* dims outside what the kernels are built for (see mtla_create) */
  MTLA_ERR_ARENA_TOO_SMALL = -3,
  MTLA_ERR_CAPACITY = -4,         /* token count would exceed max_tokens / max_prefill_tokens */
  MTLA_ERR_BATCH_MISMATCH = -5,   /* B differs from the batch the cache currently holds */
  MTLA_ERR_CUDA = -6,             /* a CUDA runtime call or launch failed */
  MTLA_ERR_STATE = -7,            /* call not valid in the handle's current state */
  MTLA_ERR_DEVICE_TIMEOUT = -8,   /* a bounded device-side wait gave up (reported by mtla_check) */
  MTLA_ERR_SCRATCH_LIMIT = -9     /* mtla_decode_step_static: split workspace exceeds the static array */
} mtla_status;

enum { MTLA_DTYPE_FP32 = 0, MTLA_DTYPE_BF16 = 1 };
/* mtla_config.kernel_path: which kernels a bf16 layer with r a multiple of 128 runs on.  Every
 * other layer runs on the CUDA-core kernels whatever the setting. */
enum { MTLA_PATH_AUTO = 0, MTLA_PATH_CUDA_CORE = 1 };

/* Layer dimensions (paper's Section 4 and 4.3) and capacities. */
typedef struct {
  int32_t d_model;            /* d */
  int32_t n_heads;            /* n_h, 1..32 */
  int32_t head_dim;           /* d_h, 64 or 128 */
  int32_t latent_rank;        /* r, multiple of 64, <= 512 */
  int32_t rope_dim;           /* d_R, even, multiple of 32, <= 64 */
  int32_t stride;             /* s >= 1; s = 1 is plain multi-head latent attention (w = 1) */
  int32_t hyper_dim;          /* d_w <= 256; 0 selects r/4 (Appendix: 256 -> 64) */
  int32_t max_batch;          /* capacity in sequences */
  int32_t max_tokens;         /* capacity in tokens per sequence: ceil(max_tokens/s) slots */
  int32_t max_prefill_tokens; /* largest T of one mtla_prefill call; 0 = no prefill workspace */
  int32_t dtype;              /* MTLA_DTYPE_* */
  float ln_eps;               /* 0 selects 1e-5 */
  float rope_theta;           /* 0 selects 10000 */
  int32_t kernel_path;        /* MTLA_PATH_*: AUTO takes the tensor-core kernels where they apply */
} mtla_config;

/* Device pointers to the parameters, row-major [in][out], element type config.dtype.
 * They are repacked into the arena by mtla_create and not referenced afterwards.
 * Bias pointers may be NULL (treated as zero). */
typedef struct {
  const void* w_q;       /* [d][n_h*d_h]      Eq. 7 */
  const void* w_qr;      /* [d][n_h*d_R]      RoPE queries, Section 4.3 */
  const void* w_r;       /* [d][r]            Eq. 8 */
  const void* w_kr;      /* [d][d_R]          shared RoPE key, Section 4.3 */
  const void* ln_gamma;  /* [r]               LayerNorm after Eq. 8 */
  const void* ln_beta;   /* [r] */
  const void* w_k;       /* [r][n_h*d_h]      Eq. 9 */
  const void* w_v;       /* [r][n_h*d_h]      Eq. 10 */
  const void* w_o;       /* [n_h*d_h][d]      Eq. 11 */
  const void* hyp_c_w;   /* [r][d_w]          Eq. 13, Linear(c_i) */
  const void* hyp_c_b;   /* [d_w] or NULL */
  const void* hyp_pe_w;  /* [r][d_w]          Eq. 13, Linear(pe_j) */
  const void* hyp_pe_b;  /* [d_w] or NULL */
} mtla_weights;

/* Paged storage of the cache, for ragged batches and beam search (the paper decodes with beam
 * search over utterances of different lengths, Section 5 and the appendix on decoding
 * set-ups).  The slots live in a pool of pages of page_slots slots; every sequence has its own
 * token count and holds the pages of its slots.  Closed slots never change (Section 4.1 only
 * ever writes a sequence's newest slot), so beams that continue one hypothesis share its pages
 * and only the page of the newest slot is copied when a beam first writes to it. */
typedef struct {
  int32_t page_slots;   /* slots per page: 64 (one tile of the decode attention) */
  int32_t n_pages;      /* pages in the pool; 0 selects max_batch * ceil(ceil(max_tokens/s)/64),
                           enough for max_batch unshared sequences of max_tokens tokens */
} mtla_paging;

/* Device bytes mtla_create needs for this configuration (weights, tables, cache, decode
 * scratch and, if max_prefill_tokens > 0, the prefill workspace).  0 if cfg is invalid. */
size_t mtla_arena_bytes(const mtla_config* cfg);

/* Builds a layer (Section 4): validates cfg, repacks the weights into `arena` (device,
 * 1024-byte aligned, >= mtla_arena_bytes(cfg)), builds the positional tables (sinusoidal
 * pe_j pushed through Linear(pe_j) of Eq. 13; RoPE angles of Section 4.3) and starts with
 * an empty cache.  The packing kernels run on `stream`.  *out receives the handle. */
int mtla_create(const mtla_config* cfg, const mtla_weights* weights, void* arena,
                size_t arena_bytes, void* stream, mtla_handle** out);

/* The same layer with the cache in paged storage (see mtla_paging) and a token count per
 * sequence.  On such a handle mtla_decode_step advances every sequence from its own position
 * (the slot, the merge weight's pe_j and the RoPE angle of Section 4.1 / 4.3 are those of the
 * sequence), mtla_prefill_seqs fills chosen sequences, mtla_beam_reorder re-parents the batch,
 * and every other call keeps its meaning.  At most 1022 sequences on the tensor-core path.
 * mtla_arena_bytes_paged is the arena size for the pair (cfg, paging); 0 if invalid. */
size_t mtla_arena_bytes_paged(const mtla_config* cfg, const mtla_paging* paging);
int mtla_create_paged(const mtla_config* cfg, const mtla_paging* paging, const mtla_weights* weights,
                      void* arena, size_t arena_bytes, void* stream, mtla_handle** out);

/* Parallel prefill (Section 4.2 with the RoPE shortcut of Section 4.3): consumes T prompt
 * tokens for each of B sequences, x device [B][T][d], and reproduces what T decode steps
 * would have produced: y device [B][T][d] (may be NULL to skip the outputs), the
 * ceil(T/s) cache slots, and the open slot if T is not a multiple of s.  The stride-aware
 * causal mask is applied as a predicate, never materialised.  Requires an empty cache
 * (tokens == 0), B <= max_batch, T <= min(max_prefill_tokens, max_tokens). */
int mtla_prefill(mtla_handle* h, const void* x, int32_t B, int32_t T, void* y, void* stream);

/* Paged handles only: the prefill of mtla_prefill for sequences seq0 .. seq0 + B - 1, which must
 * be empty; x device [B][T][d], y device [B][T][d] or NULL.  seq0 may not exceed the current
 * batch (sequences are numbered without gaps); the batch becomes max(batch, seq0 + B).  Calls
 * with different T build a ragged batch.  MTLA_ERR_STATE on a handle without paging or a
 * non-empty sequence, MTLA_ERR_CAPACITY if the pool has too few free pages. */
int mtla_prefill_seqs(mtla_handle* h, int32_t seq0, const void* x, int32_t B, int32_t T, void* y,
                      void* stream);

/* One incremental decoding step (Section 4.1, Eq. 13, Eq. 17) for every sequence:
 * x device [B][d] is token number tokens+1; its latent is merged into slot
 * ceil((tokens+1)/s) (a new slot opens when tokens mod s == 0), the slot's RoPE key is
 * replaced by this token's, and y device [B][d] receives the attention output over all
 * slots in the absorbed form.  B is the batch fixed by the preceding prefill / import, or
 * by the first decode step on an empty cache. */
int mtla_decode_step(mtla_handle* h, const void* x, int32_t B, void* y, void* stream);

/* Same step with HOST buffers: copies x_host [B][d] to the device, runs the step and copies
 * y back to y_host [B][d], all enqueued on `stream` (pinned host memory keeps it async). */
int mtla_decode_step_host(mtla_handle* h, const void* x_host, int32_t B, void* y_host,
                          void* stream);

/* The same decode step as mtla_decode_step, for callers that must not depend on allocated
 * scratch.  (The paper has no counterpart to this call; it exists for integration reasons only.)
 * Who needs it: a host program that has handed all device memory to its own pool and sizes the
 * arena to the byte, an embedding that runs under a "no allocation after start-up" rule, or a
 * caller that wants to shrink the arena by leaving the attention split workspace out of it.  The
 * attention kernel's scratch - the per-split partial outputs, their (maximum, denominator) pairs
 * and the combine tickets - is taken from an array of MTLA_STATIC_SCRATCH_BYTES that is built
 * into the library image, so each GPU that loads the library carries it until the process
 * exits.  The call itself allocates nothing: no cudaMalloc, no cudaFree, no allocating library
 * routine.  x, y, B and stream mean what they mean for mtla_decode_step, and the result is the
 * same within rounding (the partials are summed in the same order).
 *   - Limit: (B + 148) * n_h * (r + 2) * 4 bytes (B + 296 units on the CUDA-core path) plus
 *     the tickets must fit the array; otherwise MTLA_ERR_SCRATCH_LIMIT is returned and nothing
 *     is enqueued.  The paper's layer (8 heads, r 256) fits up to B = 359.
 *   - Every GPU has its own copy of the array, so the GPU that owns the handle's arena must be
 *     the current device on every call (MTLA_ERR_STATE otherwise).  The first call on a device
 *     resolves the array's device address (cudaGetSymbolAddress, checked); make that first
 *     call before starting any stream capture.  The address cache is filled without a lock:
 *     concurrent first calls store the same value.
 *   - All handles and all calls on a device share the one array, and it keeps the previous
 *     call's contents.  The tickets are cleared on `stream` at the start of every call; the
 *     partials are fully rewritten before they are read.  Two calls whose kernels may overlap
 *     on the GPU (different streams, or different handles without ordering) race on it: keep
 *     calls of this entry point ordered on one stream per device. */
#define MTLA_STATIC_SCRATCH_BYTES (4u << 20)
int mtla_decode_step_static(mtla_handle* h, const void* x, int32_t B, void* y, void* stream);

/* ---- comparison layers: multi-head, grouped-query and multi-query attention (Section 3) ----
 *
 * The attentions the paper compares against, at the same boundary, so that its speed and
 * cache-size ratios can be restated on this hardware: q = x W_Q (n_h heads), k = x W_K and
 * v = x W_V (n_kv_heads heads, each shared by n_h / n_kv_heads query heads: n_kv_heads = n_h is
 * MHA, 1 is MQA), the ordinary rotary embedding of q and k at the token's position (what the
 * appendix on the training set-up states for MHA), softmax(q K^T / sqrt(d_h)) V over the cached keys and values
 * including the token's own, y = concat(heads) W_O.  bf16 only.  The cache keeps 2 n_kv_heads d_h
 * elements per token, laid out [sequence][kv head][token][value | key].
 * A handle made by mtla_baseline_create is used with mtla_decode_step, mtla_cache_bytes,
 * mtla_cache_export / mtla_cache_import (layout [B][n_kv_heads][tokens][2 d_h]), mtla_position,
 * mtla_reset, mtla_check, mtla_profile_* and mtla_destroy; every other call returns
 * MTLA_ERR_STATE.  Weights: device, row-major [in][out], bf16. */
typedef struct {
  int32_t d_model, n_heads, n_kv_heads;
  int32_t head_dim;           /* 64 or 128 */
  int32_t max_batch, max_tokens;
  float rope_theta;           /* 0 selects 10000 */
} mtla_baseline_config;
typedef struct {
  const void* w_q;            /* [d][n_h*d_h] */
  const void* w_k;            /* [d][n_kv_heads*d_h] */
  const void* w_v;            /* [d][n_kv_heads*d_h] */
  const void* w_o;            /* [n_h*d_h][d] */
} mtla_baseline_weights;
size_t mtla_baseline_arena_bytes(const mtla_baseline_config* cfg);
int mtla_baseline_create(const mtla_baseline_config* cfg, const mtla_baseline_weights* weights,
                         void* arena, size_t arena_bytes, void* stream, mtla_handle** out);

/* ---- decoder layers and stacks (Section 5.2; appendix on hyper-parameters) ----
 *
 * The paper's model is a Transformer decoder without cross-attention (the encoder output is
 * simply the first part of the input sequence): 9 layers of width 512 with 8 heads and a
 * feed-forward block of width 2048, every layer's self-attention being MTLA.  A stack is that
 * model's hot path: n_layers layers, each
 *     h = x + MTLA(LayerNorm_1(x));   y = h + W_2 relu(W_1 LayerNorm_2(h) + b_1) + b_2,
 * followed by one final LayerNorm.  Pre-norm placement and ReLU are the usual settings of the
 * toolkit the paper builds on (the paper states neither).  Every layer has the attention
 * dimensions of `cfg` and its own weights and cache; the residual stream between sub-layers is
 * kept in fp32, x and y are in cfg.dtype.  All layers advance in lock-step.
 * Weights: device pointers, row-major [in][out], element type cfg.dtype, repacked at create and
 * not referenced afterwards.  `layers` is a host array of n_layers entries. */
typedef struct {
  mtla_weights attn;                     /* the layer's self-attention (Section 4) */
  const void *ln1_gamma, *ln1_beta;      /* [d]  LayerNorm in front of the attention */
  const void *ln2_gamma, *ln2_beta;      /* [d]  LayerNorm in front of the feed-forward block */
  const void *w1, *b1;                   /* [d][d_ff], [d_ff] */
  const void *w2, *b2;                   /* [d_ff][d], [d] */
} mtla_layer_weights;
typedef struct {
  int32_t n_layers;                      /* 1..256; the paper: 9 */
  int32_t d_ff;                          /* feed-forward width, multiple of 8; the paper: 2048 */
  float ln_eps;                          /* eps of the layers' LayerNorms; 0 selects 1e-5 */
} mtla_stack_config;
typedef struct mtla_stack mtla_stack;

/* Device bytes mtla_stack_create needs (0 if the pair is invalid), and the constructor: arena
 * device, 1024-byte aligned; lnf_gamma / lnf_beta [d] are the final LayerNorm. */
size_t mtla_stack_arena_bytes(const mtla_config* cfg, const mtla_stack_config* scfg);
int mtla_stack_create(const mtla_config* cfg, const mtla_stack_config* scfg,
                      const mtla_layer_weights* layers, const void* lnf_gamma, const void* lnf_beta,
                      void* arena, size_t arena_bytes, void* stream, mtla_stack** out);

/* mtla_prefill / mtla_decode_step through every layer: x device [B][T][d] resp. [B][d], y the
 * stack's output of the same shape (required).  Errors as for the single-layer calls. */
int mtla_stack_prefill(mtla_stack* s, const void* x, int32_t B, int32_t T, void* y, void* stream);
int mtla_stack_decode_step(mtla_stack* s, const void* x, int32_t B, void* y, void* stream);

/* Cache bytes in use over all layers (n_layers times the per-layer count of Section 4.3). */
size_t mtla_stack_cache_bytes(const mtla_stack* s);

/* The attention handle of one layer, borrowed (valid until mtla_stack_destroy; do not destroy
 * it): for mtla_position, mtla_cache_export and the other inspection calls. */
mtla_handle* mtla_stack_layer(mtla_stack* s, int32_t layer);

int mtla_stack_reset(mtla_stack* s);                       /* empties every layer's cache */
int mtla_stack_check(mtla_stack* s, void* stream);          /* mtla_check over the layers */
int64_t mtla_stack_launch_count(const mtla_stack* s);
int mtla_stack_destroy(mtla_stack* s);

/* ---- training path (Section 4.2, Eq. 14-16) ----
 *
 * The paper trains with the parallel form: the merge weights of every chunk at once (Eq. 16 with
 * the chunk mask), the sequence of running states C' (Eq. 14), attention over C' and the
 * un-compressed RoPE keys under the stride-aware causal mask.  mtla_prefill computes exactly
 * that form (as per-chunk running sums and a mask predicate instead of T x T matrices), so it IS
 * the training forward pass; mtla_train_backward is its reverse.  Given dL/dY it returns dL/dX
 * and the gradient of every parameter, through the softmax and the mask, the key / value
 * up-projections, the running sums and their sigmoid gates (including both Linear layers of
 * the hyper-network), the LayerNorm, the rotations and the fused input projection.
 *
 * fp32 layers on contiguous storage only (MTLA_ERR_UNSUPPORTED_SHAPE otherwise).  The call must
 * follow mtla_prefill(h, x, B, T, y != NULL) on the same handle with nothing in between
 * (MTLA_ERR_STATE otherwise): it reads what that call left in the handle's prefill workspace.
 * x, dy, dx device [B][T][d] fp32; x is the prefill's input again.  The gradient buffers are
 * device fp32 arrays shaped like the weights of mtla_weights (row-major [in][out]); they are
 * overwritten, not accumulated, and hold sums over the batch.  At s = 1 the hyper-network's
 * gradients are zero.  `workspace` is device memory of at least
 * mtla_train_workspace_bytes(h, B, T) bytes, 256-byte aligned, owned by the caller; it holds,
 * among others, two T x T matrices per (sequence, head).  Results do not depend on the launch
 * configuration (every reduction runs in index order). */
typedef struct {
  void *w_q, *w_qr, *w_r, *w_kr, *ln_gamma, *ln_beta, *w_k, *w_v, *w_o;
  void *hyp_c_w, *hyp_c_b, *hyp_pe_w, *hyp_pe_b;
} mtla_grads;
size_t mtla_train_workspace_bytes(const mtla_handle* h, int32_t B, int32_t T);
int mtla_train_backward(mtla_handle* h, const void* x, const void* dy, int32_t B, int32_t T, void* dx,
                        const mtla_grads* grads, void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of cache in use: B * ceil(tokens/s) * (r + d_R) * sizeof(element)  (Sections 4, 4.3);
 * with per-sequence token counts, the sum over the sequences. */
size_t mtla_cache_bytes(const mtla_handle* h);

/* Releases the host-side handle.  The arena is the caller's. */
int mtla_destroy(mtla_handle* h);

/* ---- support calls (state inspection, cache checkpointing, diagnostics) ---- */

/* Empties the cache (tokens = 0, batch unset).  Nothing is enqueued. */
int mtla_reset(mtla_handle* h);

/* Current position: tokens consumed per sequence (the longest sequence's on a paged handle),
 * slots held (= ceil(tokens/s)), batch. */
int mtla_position(const mtla_handle* h, int32_t* tokens, int32_t* slots, int32_t* batch);

/* Copies the cache in use to dst (device), layout [B][slots][r + d_R], element type dtype;
 * `bytes` must be >= mtla_cache_bytes(h).  MTLA_ERR_STATE on a paged handle whose sequences
 * differ in length (use mtla_cache_export_seq). */
int mtla_cache_export(mtla_handle* h, void* dst, size_t bytes, void* stream);

/* Replaces the cache by src (device) [B][ceil(tokens/s)][r + d_R] and sets the position to
 * `tokens`.  If tokens is not a multiple of s the last slot is open and its fp32
 * accumulator is initialised from the stored value. */
int mtla_cache_import(mtla_handle* h, const void* src, int32_t B, int32_t tokens, void* stream);

/* Paged handles only: mtla_cache_import for the empty sequences seq0 .. seq0 + B - 1, leaving
 * the others as they are; src device [B][ceil(tokens/s)][r + d_R].  seq0 may not exceed the
 * current batch; the batch becomes max(batch, seq0 + B). */
int mtla_cache_import_seqs(mtla_handle* h, int32_t seq0, const void* src, int32_t B, int32_t tokens,
                           void* stream);

/* Beam reordering (paged handles): sequence b of the new batch continues old sequence
 * parents[b] (host array of n_new indices into the current batch; an index may repeat or be
 * absent).  Positions, page tables and the fp32 state of the open slot follow on `stream`;
 * pages are shared, not copied, and pages that no sequence holds any more return to the pool.
 * The batch becomes n_new.  The parents array is read before the call returns. */
int mtla_beam_reorder(mtla_handle* h, const int32_t* parents, int32_t n_new, void* stream);

/* Tokens consumed by sequences 0 .. n-1 (host array; 0 beyond the batch).  On a handle without
 * paging every sequence reports the common count. */
int mtla_seq_positions(const mtla_handle* h, int32_t* tokens, int32_t n);

/* Pages of the pool that some sequence holds (shared pages count once); -1 without paging.
 * Physical cache bytes = pages * 64 * (r + d_R) * sizeof(element), while mtla_cache_bytes
 * reports the logical sum over sequences of ceil(tokens/s) slots. */
int64_t mtla_pages_in_use(const mtla_handle* h);

/* Copies the slots of one sequence to dst (device) [ceil(tokens/s)][r + d_R]; works with and
 * without paging. */
int mtla_cache_export_seq(mtla_handle* h, int32_t seq, void* dst, size_t bytes, void* stream);

/* The page pool's bookkeeping on its own, host-only (no GPU is touched): the object a paged
 * handle uses to decide which pages to allocate, share and copy.  A scheduler can run it ahead
 * of the GPU to see whether a batch fits; the tests drive it against a model of the sharing
 * rules.  prepare(seq, n_slots, write_slot): make slots [0, n_slots) of seq addressable and,
 * if write_slot >= 0, the page holding it private to seq; returns the number of page copies
 * that implies and writes up to max_copies triples (source page, destination page, rows) to
 * `copies`, or MTLA_ERR_CAPACITY (state unchanged) if the pool has too few free pages.
 * reorder: as mtla_beam_reorder.  row: the pages seq holds, returns their count.  ref: how
 * many sequences hold a page. */
typedef struct mtla_page_pool mtla_page_pool;
mtla_page_pool* mtla_page_pool_create(int32_t n_pages, int32_t max_seqs, int32_t max_pages_per_seq);
void mtla_page_pool_destroy(mtla_page_pool* p);
int mtla_page_pool_prepare(mtla_page_pool* p, int32_t seq, int32_t n_slots, int32_t write_slot,
                           int32_t* copies, int32_t max_copies);
int mtla_page_pool_reorder(mtla_page_pool* p, const int32_t* parents, int32_t n_new, int32_t n_old);
int mtla_page_pool_row(const mtla_page_pool* p, int32_t seq, int32_t* pages, int32_t max_pages);
int mtla_page_pool_in_use(const mtla_page_pool* p);
int mtla_page_pool_ref(const mtla_page_pool* p, int32_t page);

/* Synchronises `stream` and reports a sticky device-side status (MTLA_ERR_DEVICE_TIMEOUT if
 * a bounded wait inside a kernel gave up; MTLA_ERR_CUDA if the stream is in error). */
int mtla_check(mtla_handle* h, void* stream);

/* Diagnostics of the bounded device-side waits.  Every wait inside the tensor-core kernels
 * gives up after a time budget, records a code and lets the kernel return, which is what
 * mtla_check reports as MTLA_ERR_DEVICE_TIMEOUT.  mtla_selftest_wait_timeout exercises that path
 * on purpose and harmlessly: it enqueues a one-CTA kernel whose only wait (on a barrier nobody
 * arrives at) has a budget of budget_us microseconds (1 .. 1000000); the kernel returns by
 * itself, and the next mtla_check on the stream reports the timeout.  The status is sticky
 * until mtla_clear_error, which zeroes it on `stream`. */
int mtla_selftest_wait_timeout(mtla_handle* h, int32_t budget_us, void* stream);
int mtla_clear_error(mtla_handle* h, void* stream);

/* Number of kernels the library has launched on behalf of this handle since creation. */
int64_t mtla_launch_count(const mtla_handle* h);

/* Kernel timing for benchmarks.  After mtla_profile_begin, each of the next max_steps decode
 * steps records CUDA events on its stream between its kernels, in the order of Section 4.1:
 * stage 0 input projections (Eq. 7, Eq. 8, RoPE projections), 1 LayerNorm + gate (Eq. 13) + slot
 * update + RoPE, 2 query absorption (Eq. 12), 3 attention over the cache (Eq. 17; the kernel
 * that streams the cache), 4 cross-split combine, 5 value up-projection (Eq. 10), 6 output
 * projection (Eq. 11).  mtla_profile_end_stages waits for those events, returns the summed
 * duration of every stage in milliseconds (stage_ms host [MTLA_DECODE_STAGES]) and the number
 * of steps covered, and releases the events; mtla_profile_end returns the attention stage only.
 * mtla_profile_begin_attention records only the two events around the attention kernel (the
 * other stages then read 0), which perturbs a timed loop least. */
enum { MTLA_DECODE_STAGES = 7, MTLA_STAGE_ATTENTION = 3 };
int mtla_profile_begin(mtla_handle* h, int32_t max_steps);
int mtla_profile_begin_attention(mtla_handle* h, int32_t max_steps);
int mtla_profile_end(mtla_handle* h, double* attention_ms, int32_t* steps);
int mtla_profile_end_stages(mtla_handle* h, double* stage_ms, int32_t* steps);

/* Beam search on paged handles: when the batch consists of blocks of consecutive sequences of
 * equal length that share their first page (the beams of one utterance after mtla_beam_reorder),
 * the tensor-core decode attention walks each block with a gang of CTAs side by side, one
 * sequence each over the same tiles at the same time, so that a shared page is read from DRAM
 * once.  Returns the gang size of the handle's latest decode step: 1 = every CTA on its own
 * share (lock-step batches, unrelated sequences), 0 = no tensor-core decode step has run yet
 * (or h is NULL).  Host query only; never fails. */
int32_t mtla_attention_gang(const mtla_handle* h);

/* Name of the decode-attention kernel variant the handle dispatches to ("fma" or "tcgen05"). */
const char* mtla_attention_variant(const mtla_handle* h);

const char* mtla_error_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* MTLA_H_ */
