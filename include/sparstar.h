/*
 * sparstar.h - C ABI of the B200 (sm_100a) library for SparSTAR's per-scale, per-head
 * dynamic block-sparse attention: block-mean pooling -> aggregated query-key block scores
 * -> selection of key blocks per query block -> forward-only sparse attention, plus a
 * dense attention for comparison.
 *
 * Conventions for every call
 *   - All data pointers are DEVICE pointers owned by the caller unless a parameter says
 *     "host".  Nothing is retained after the call returns except by the context.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     The operator calls only enqueue work; they neither allocate device memory nor
 *     synchronise - with one exception: the context keeps a device scratch buffer (work order
 *     and union lists of the sparse attention, pre-scores of SPARSTAR_SCORE_TCGEN05), and a call
 *     that needs more of it than the context holds allocates a larger buffer first (cudaMalloc).
 *     The outgrown buffer is kept until sparstar_destroy, never freed earlier: work already
 *     enqueued, and any CUDA graph captured from earlier calls, go on using the address they were
 *     given.  CUDA graphs: run every call once eagerly (or call sparstar_reserve_scratch) before
 *     capturing it; a call that would have to grow the scratch while `stream` is capturing
 *     returns SPARSTAR_ERR_CAPTURE and enqueues nothing.
 *   - The context's device must be the calling thread's current device for every call that
 *     takes a context and a stream (SPARSTAR_ERR_INVALID_ARG otherwise).
 *   - The int return value is a sparstar_status decided on the HOST before any launch
 *     (argument, shape, alignment and support checks).  Conditions found on the DEVICE
 *     (list entry out of range, capacity exceeded, a bounded wait that ran out) are
 *     recorded in the context's device status word and reported by sparstar_check().
 *   - Tensors are [B, H, L, D] with D contiguous and element strides sB, sH, sL.
 *     Rows must be 16-byte aligned (base pointer and every stride times the element size).
 *   - A context serves one device; calls that share a context must be stream-ordered.
 */
#ifndef SPARSTAR_H_
#define SPARSTAR_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sparstar_ctx sparstar_ctx;

typedef enum {
  SPARSTAR_OK = 0,
  SPARSTAR_ERR_INVALID_ARG = 1,  /* null pointer, non-positive size, misaligned pointer/stride */
  SPARSTAR_ERR_UNSUPPORTED = 2,  /* a shape/dtype/block combination no kernel covers */
  SPARSTAR_ERR_CAPACITY = 3,     /* device: a row needed more than `cap` list entries */
  SPARSTAR_ERR_BAD_INDEX = 4,    /* device: a list entry out of range or not ascending */
  SPARSTAR_ERR_TIMEOUT = 5,      /* device: a bounded wait expired; while it is on record the tensor-core attention
                                    kernel does no work (outputs unspecified) until sparstar_check clears it */
  SPARSTAR_ERR_CUDA = 6,         /* a CUDA runtime/driver call failed */
  SPARSTAR_ERR_TOO_LARGE = 7,    /* the problem exceeds a fixed built-in limit of the entry point */
  SPARSTAR_ERR_CAPTURE = 8       /* the context scratch would have to grow while `stream` is capturing */
} sparstar_status;

typedef enum { SPARSTAR_F32 = 0, SPARSTAR_BF16 = 1 } sparstar_dtype;

typedef enum {
  SPARSTAR_SEL_TOPK_RATIO = 0,   /* k from Eq. 5 with density `ratio` */
  SPARSTAR_SEL_TOPK_COUNT = 1,   /* k = min(n_sel, count) */
  SPARSTAR_SEL_MASS = 2          /* cumulative block-score mass >= `mass` (not in the paper) */
} sparstar_sel_mode;

typedef enum {
  SPARSTAR_ATTN_AUTO = 0,        /* tensor-core kernel when the shape allows, else SIMT */
  SPARSTAR_ATTN_SIMT = 1,        /* fp32 FFMA kernel (any supported shape) */
  SPARSTAR_ATTN_TCGEN05 = 2,     /* tcgen05/TMEM/TMA kernels (bf16, D in {64,128}, block in {32,64,128,256,512});
                                    three score tiles in flight, one accumulator; blocks of 64 / 32 tokens are
                                    gathered two / four to a 128-key tile */
  SPARSTAR_ATTN_TCGEN05_2STREAM = 3, /* same shapes on the older two-stream kernel (two score tiles, two accumulators
                                    merged at the end) - kept as a cross-check */
  SPARSTAR_ATTN_TCGEN05_PAIR = 4  /* same shapes; where two adjacent 128-row query tiles walk the same list (dense,
                                    blocks of 256 or 512 tokens) and D = 128, they run on a pair of CTAs that issue
                                    tcgen05.mma.cta_group::2 together, each holding half of every K and V tile;
                                    everything else as SPARSTAR_ATTN_TCGEN05 */
} sparstar_attn_impl;

typedef enum {
  SPARSTAR_SCORE_FP64 = 0,       /* score strip as an fp64 tensor-core GEMM inside the selection kernel (exact) */
  SPARSTAR_SCORE_TCGEN05 = 1     /* tcgen05 GEMM on 3-term bf16 splits (fp32-grade) + exact fp64 re-scoring of
                                    the blocks next to the cutoff; D in {64, 128} */
} sparstar_score_impl;

/* Half-open range [begin, end) of key-token positions. */
typedef struct { int64_t begin, end; } sparstar_range;

typedef struct {
  void*   ptr;            /* device */
  int32_t dtype;          /* sparstar_dtype */
  int32_t B, H, L, D;
  int64_t sB, sH, sL;     /* element strides; D has stride 1 */
} sparstar_tensor;

typedef struct {
  int32_t mode;                  /* sparstar_sel_mode */
  int32_t count;                 /* SEL_TOPK_COUNT */
  double  ratio;                 /* SEL_TOPK_RATIO: rho of Eq. 5 */
  double  mass;                  /* SEL_MASS: p in (0, 1] */
  const sparstar_range* forced;  /* HOST array: token ranges whose blocks stay dense (Eq. 3) */
  int32_t n_forced;              /* 0..16 */
} sparstar_select_params;

/* ---- context ---------------------------------------------------------------------------
 * sparstar_create allocates the context (host) and its device status word on `device`.
 * sparstar_check synchronises `stream`, returns the first device-side status recorded since
 * the last check (SPARSTAR_OK if none) and clears it; *site (nullable, host) receives an
 * implementation-defined code locating the condition.
 * sparstar_set_attn_impl selects the attention kernel family for later calls.
 * sparstar_set_score_impl selects how sparstar_score_select forms the block scores (see
 *   sparstar_score_impl); with SPARSTAR_SCORE_TCGEN05 the pre-scores go to `scores_out` when
 *   given, else to the context's scratch buffer (allocated on first use).
 * sparstar_launch_count returns how many kernels this context has launched so far.
 * sparstar_reserve_scratch grows the context scratch to at least `bytes` now (no-op if it is
 *   that large already), so that later calls - captured ones in particular - need not;
 *   sparstar_scratch_bytes returns its present size.
 * sparstar_set_debug (test aid, not for production use): work_order_on = 0 makes the sparse
 *   tensor-core attention walk the query tiles in index order instead of longest list first;
 *   drop_stage >= 0 makes its TMA producer arm the barrier of that list position and copy
 *   nothing, so that the consumer's bounded wait runs out after about a second, the launch ends
 *   with SPARSTAR_ERR_TIMEOUT on record and unspecified outputs (exercises the bounded waits
 *   without faulting anything); drop_stage < 0 switches it off.  Defaults: 1, -1.
 * sparstar_set_trace (profiling aid): `buf` = device array of 4 * capacity * 2 int64, or NULL to
 *   switch tracing off.  While set, the first CTA of the tensor-core attention kernel records
 *   (tag, SM clock modulo 2^26) pairs for its four roles (MMA issuer, softmax warpgroup 0,
 *   softmax warpgroup 1, TMA producer): events of list positions >= `skip`, at most
 *   min(capacity, 48) per role; unused pairs are written as zeros. */
int sparstar_create(sparstar_ctx** out, int device);
int sparstar_destroy(sparstar_ctx* ctx);
int sparstar_check(sparstar_ctx* ctx, void* stream, int32_t* site);
int sparstar_set_attn_impl(sparstar_ctx* ctx, int32_t impl);
int sparstar_set_score_impl(sparstar_ctx* ctx, int32_t impl);
int64_t sparstar_launch_count(const sparstar_ctx* ctx);
int sparstar_set_trace(sparstar_ctx* ctx, int64_t* buf, int32_t capacity, int32_t skip);
int sparstar_set_debug(sparstar_ctx* ctx, int32_t work_order_on, int32_t drop_stage);
int sparstar_reserve_scratch(sparstar_ctx* ctx, int64_t bytes, void* stream);
int64_t sparstar_scratch_bytes(const sparstar_ctx* ctx);
const char* sparstar_status_string(int status);

/* ---- host integer helpers ---------------------------------------------------------------
 * sparstar_num_blocks: n = ceil(L / block), the original-order partition into contiguous
 *   blocks from token 0, not aligned to segments (Sec. "Aggregated Query-Key Block
 *   Selector", block-partition paragraph).  Returns -1 on invalid arguments.
 * sparstar_budget: Eq. 5, k = min(n_sel, max(1, ceil(ratio * n_sel))); the product is formed
 *   in double with a 1e-9 guard below the ceiling.  n_sel <= 0 gives 0.
 * sparstar_forced_count: number of key blocks whose token set [j*block, min((j+1)*block, L_k))
 *   intersects one of the `n` host ranges (the intersection definition of J_text / J_ref,
 *   which covers blocks straddling a segment boundary).  Returns -1 on invalid arguments. */
int32_t sparstar_num_blocks(int64_t L, int32_t block);
int32_t sparstar_budget(int32_t n_sel, double ratio);
int32_t sparstar_forced_count(int64_t L_k, int32_t block, const sparstar_range* ranges, int32_t n);

/* ---- clip policy (host integers) ------------------------------------------------------------
 * sparstar_keep_ranges: the always-retained token ranges of Eq. 3 - clip 1 keeps the text range
 *   and the final image-pyramid (reference) range dense, every later clip keeps only the text
 *   range (reference blocks are then ranked jointly with the current-scale blocks, without a
 *   quota).  Writes 1 or 2 ranges to `out` (room for 2) and returns how many; empty input
 *   ranges are dropped; returns -1 on invalid arguments (clip < 1, out NULL).
 * sparstar_density_lookup: the scale-wise density schedule rho_c(L_q) of Sec. "Clip-Dependent
 *   Retained and Selectable Blocks": one table per clip group, indexed by the query length;
 *   scales with the same token count share a density.  Returns 1 and *rho when `L_q` is in the
 *   table (the scale is sparsified), 0 when it is not (the scale stays dense), -1 on invalid
 *   arguments.
 * sparstar_schedule_preset: fills `out` (room for 4) with a built-in table and returns its
 *   length.  SPARSTAR_SCHEDULE_480P: the four final scales printed in the paper's configuration
 *   table (5,040 / 11,520 / 20,640 / 31,800 query tokens -> 0.625, 0.1875, 0.1875, 0.09375),
 *   used for 480p clip 1 and clip 2 alike.  SPARSTAR_SCHEDULE_720P_PYRAMID: the same four
 *   densities at 4,800 / 18,400 / 40,800 / 72,000 tokens; the paper prints only the 72,000-token
 *   count for 720p, the other three are this library's benchmark pyramid. */
typedef struct { int64_t L_q; double rho; } sparstar_density_entry;
typedef enum { SPARSTAR_SCHEDULE_480P = 0, SPARSTAR_SCHEDULE_720P_PYRAMID = 1 } sparstar_schedule_id;
int32_t sparstar_keep_ranges(int32_t clip, sparstar_range text, sparstar_range ref, sparstar_range* out);
int32_t sparstar_density_lookup(const sparstar_density_entry* table, int32_t n, int64_t L_q, double* rho);
int32_t sparstar_schedule_preset(int32_t id, sparstar_density_entry* out);

/* ---- sparstar_pool_blocks ---------------------------------------------------------------
 * Block means xbar_i = (1/block) * sum of the block's tokens; the final partial block is
 * zero-padded and still divided by the nominal block length (block-partition and per-head
 * score paragraphs of Sec. "Aggregated Query-Key Block Selector").
 *   x       [B,H,L,D] f32 or bf16; D*elemsize a multiple of 16 and <= 4096 bytes
 *   pooled  [B,H,nb,D] fp32, contiguous, nb = ceil(L/block); written in full
 * fp32 accumulation in a fixed order (bit-reproducible). */
int sparstar_pool_blocks(sparstar_ctx* ctx, const sparstar_tensor* x, int32_t block,
                         float* pooled, void* stream);
/* Same, for blocks first_block .. first_block + n_blocks - 1 only: rows of `pooled` (the full
 * [B,H,nb,D] array) outside that range are left untouched.  Lets a caller keep the block means of
 * conditioning keys that do not change between the scales of a clip and refresh only the blocks
 * from the first one that holds a current-scale token. */
int sparstar_pool_blocks_range(sparstar_ctx* ctx, const sparstar_tensor* x, int32_t block,
                               int32_t first_block, int32_t n_blocks, float* pooled, void* stream);

/* ---- sparstar_score_select --------------------------------------------------------------
 * Block scores S_ij = scale * qbar_i . kbar_j per head (Eq. 2), then per query block the
 * retained key-block set A_i = J_keep U TopKIdx over J_sel (Eq. 3, 4, 6) written as the
 * forward BlockMask fields (Sec. "Forward-Only Sparse Execution").
 *   q_pooled [B,H,n_q,D], k_pooled [B,H,n_k,D]  fp32 contiguous (outputs of pool_blocks)
 *   block, L_k      key block length and key count (define the forced block set)
 *   scale           tau; the paper's value is D^(-1/2)
 *   params          HOST struct.  J_keep = blocks intersecting params->forced; the rest is
 *                   J_sel and is ranked.  TOPK_*: the k best by (score desc, index asc).
 *                   MASS: softmax of S over J_sel only; the shortest prefix of that order
 *                   whose mass is >= params->mass (benchmark-defined, absent from the paper).
 *   kv_num_blocks   [B,H,n_q] int32: |A_i| (written in full even if it exceeds cap)
 *   kv_indices      [B,H,n_q,cap] int32: A_i ascending, unique; entries past the count are
 *                   not written; a row longer than cap is truncated and ERR_CAPACITY recorded
 *   scores_out      nullable [B,H,n_q,n_k] fp32: S rounded to fp32 (diagnostic)
 * Scores are accumulated in fp64 and ranked in fp64. */
int sparstar_score_select(sparstar_ctx* ctx, const float* q_pooled, const float* k_pooled,
                          int32_t B, int32_t H, int32_t n_q, int32_t n_k, int32_t D,
                          int32_t block, int64_t L_k, double scale,
                          const sparstar_select_params* params,
                          int32_t* kv_num_blocks, int32_t* kv_indices, int32_t cap,
                          float* scores_out, void* stream);

/* ---- sparstar_select_fused -----------------------------------------------------------------
 * Pooling of Q and K, block scores and selection of one scale in ONE launch (the three steps of
 * Sec. "Aggregated Query-Key Block Selector" before the attention: block means, Eq. 2, Eq. 5-6),
 * with the lists sparstar_pool_blocks + sparstar_score_select give, bit for bit.
 *   q [B,H,L_q,D], k [B,H,L_k,D]   as for sparstar_pool_blocks
 *   k_cond_pooled / n_cond   nullable [B,H,n_cond,D] fp32: block means of the first n_cond key
 *       blocks, computed earlier (conditioning keys that do not change between the scales of a
 *       clip, Sec. "Preliminaries"); those blocks are copied, not pooled again.  Only blocks that
 *       lie wholly inside the unchanged part may be passed.
 *   q_pooled [B,H,n_q,D], k_pooled [B,H,n_k,D]   fp32 work arrays, written in full
 *   params, scale, kv_num_blocks, kv_indices, cap   as for sparstar_score_select
 * A cooperative launch: the grid is as large as the device holds at once and meets at a grid-wide
 * barrier between pooling and selection. */
int sparstar_select_fused(sparstar_ctx* ctx, const sparstar_tensor* q, const sparstar_tensor* k, int32_t block,
                          double scale, const sparstar_select_params* params, const float* k_cond_pooled,
                          int32_t n_cond, float* q_pooled, float* k_pooled, int32_t* kv_num_blocks,
                          int32_t* kv_indices, int32_t cap, void* stream);

/* ---- sparstar_sparse_attn_fwd -----------------------------------------------------------
 * O_t = sum_u softmax_u(scale * q_t . k_u) v_u over keys u < L_k whose block pi_k(u) is in
 * A_{pi_q(t)} (Eq. 7; the key tail is the padding mask).  Forward only.
 *   q [B,H,L_q,D], k, v [B,H,L_k,D], o [B,H,L_q,D]: one dtype; supported:
 *       bf16, D in {64, 128}, block in {32, 64, 128, 256, 512} (tensor-core kernel; a block is
 *         walked as tiles of 128 tokens; for blocks of 64 / 32 tokens the query blocks of a
 *         128-row tile are served over the union of their lists, which the call builds in the
 *         context scratch: ceil(L_q/128) * ceil(L_k/block) ints per (batch, head); blocks 64 and
 *         128 also on SIMT)
 *       f32 or bf16 with D in {64,128}, block in {64,128}, (f32: block*D <= 8192) (SIMT)
 *   kv_num_blocks / kv_indices / cap  as written by sparstar_score_select; every row must
 *       hold at least one block; entries must be ascending and < ceil(L_k/block), otherwise
 *       ERR_BAD_INDEX is recorded and that row's output is unspecified (no access leaves the
 *       tensors); a row with no block gives zeros and lse = -inf
 *   lse  nullable [B,H,L_q] fp32: log sum_u exp(scale * q_t . k_u) over the kept keys
 * Query rows >= L_q are neither computed nor written. */
int sparstar_sparse_attn_fwd(sparstar_ctx* ctx, const sparstar_tensor* q, const sparstar_tensor* k,
                             const sparstar_tensor* v, const sparstar_tensor* o, int32_t block,
                             float scale, const int32_t* kv_num_blocks, const int32_t* kv_indices,
                             int32_t cap, float* lse, void* stream);

/* ---- sparstar_attn_fwd ------------------------------------------------------------------
 * Dense softmax(scale * Q K^T) V over every key (Sec. "Complexity and Scope"): the
 * comparison the sparse path is measured against.  Same tensors and `block` (tile length)
 * as sparstar_sparse_attn_fwd. */
int sparstar_attn_fwd(sparstar_ctx* ctx, const sparstar_tensor* q, const sparstar_tensor* k,
                      const sparstar_tensor* v, const sparstar_tensor* o, int32_t block,
                      float scale, float* lse, void* stream);

/* ---- attention-mass analysis (Sec. "Analysis": retained attention mass of a selection) -------
 * sparstar_block_mass: exact post-softmax mass per (query block, key block),
 *   M_ij = mean over queries t of block i of sum over keys u of block j of softmax_u(scale q_t.k_u),
 *   from Q, K and the log-sum-exp of the dense attention (`lse_dense` [B,H,L_q], as written by
 *   sparstar_attn_fwd).  mass_out [B,H,n_q,n_k] fp32 (n = ceil(L / block)), rows sum to 1.  bf16, D in
 *   {64, 128}, block in {32, 64, 128, 256, 512}.
 * sparstar_select_from_scores: the selection stage of sparstar_score_select applied to a given
 *   score array [B,H,n_q,n_k] fp32 (e.g. the exact masses: the block-wise oracle selector of
 *   the paper's analysis) with the same params, tie rule, forced blocks and outputs.
 * sparstar_retained_mass: out[row] = sum over the row's kept list of mass[row][j] for
 *   rows = B*H*n_q rows; equals the mean over the block's queries of
 *   exp(lse_sparse - lse_dense). */
int sparstar_block_mass(sparstar_ctx* ctx, const sparstar_tensor* q, const sparstar_tensor* k, int32_t block,
                        float scale, const float* lse_dense, float* mass_out, void* stream);
int sparstar_select_from_scores(sparstar_ctx* ctx, const float* scores, int32_t B, int32_t H, int32_t n_q,
                                int32_t n_k, int32_t block, int64_t L_k, const sparstar_select_params* params,
                                int32_t* kv_num_blocks, int32_t* kv_indices, int32_t cap, void* stream);
int sparstar_retained_mass(sparstar_ctx* ctx, const float* mass, const int32_t* kv_num_blocks,
                           const int32_t* kv_indices, int32_t rows, int32_t n_k, int32_t cap, float* out,
                           void* stream);

/* ---- comparison selectors (the selection-strategy ablation: sliding window, random blocks,
 * cross-scale reuse; Table "selection strategies") ------------------------------------------------
 * The paper names these selectors but defines none of them; the definitions here are this
 * library's, made for analysis on synthetic inputs.  Each call writes a score array
 * [B,H,n_q,n_k] fp32 for sparstar_select_from_scores, which applies the same budget (Eq. 5), tie
 * rule and always-kept blocks (Eq. 3) as the method's own selector.
 *   sparstar_segment: one run of tokens; T > 0 means a raster (t, h, w) grid with T*H*W == length
 *     (token u sits at t = u / (H*W), h = (u / W) % H, w = u % W), T == 0 means tokens without a
 *     position (text), which count as sitting at the centre (1/2, 1/2, 1/2).  At most 8 segments.
 *   sparstar_block_centres (host): centres [n_blocks*3] of the blocks of `block` tokens over the
 *     concatenated segments: per coordinate the mean over the block's tokens of index/extent
 *     (integer index sums, one fp64 division per segment, segment order).  Returns n_blocks
 *     (also when `centres` is NULL), -1 on invalid arguments.
 *   sparstar_nearest_block_map (host): map[i] = the coarse block whose centre is nearest to fine
 *     block i (squared Euclidean distance in fp64, ties to the lower index).  Returns n_fine or -1.
 *   sparstar_window_scores: score[i][j] = -||centre_q(i) - centre_k(j)||, the same for every
 *     (batch, head); centres are formed on the device exactly as by sparstar_block_centres, the
 *     distance in fp64 with separately rounded operations, rounded once to fp32.
 *   sparstar_random_scores: score = u(seed, linear index over [B,H,n_q,n_k]) in [0, 1):
 *     z = seed + (index + 1) * 0x9E3779B97F4A7C15; z = (z ^ z >> 30) * 0xBF58476D1CE4E5B9;
 *     z = (z ^ z >> 27) * 0x94D049BB133111EB; z ^= z >> 31; u = (z >> 40) * 2^-24.
 *   sparstar_remap_scores: out[b][h][i][j] = coarse[b][h][q_map[i]][k_map[j]]: a coarser scale's
 *     scores (the scores_out of its sparstar_score_select) reused at a finer scale through
 *     nearest-position maps.  q_map [n_q], k_map [n_k]: DEVICE int32; an entry out of range is
 *     clamped and SPARSTAR_ERR_BAD_INDEX recorded. */
typedef struct { int64_t length; int32_t T, H, W; } sparstar_segment;
int32_t sparstar_block_centres(const sparstar_segment* segs, int32_t n_segs, int32_t block, double* centres);
int32_t sparstar_nearest_block_map(const double* fine, int32_t n_fine, const double* coarse, int32_t n_coarse,
                                   int32_t* map);
int sparstar_window_scores(sparstar_ctx* ctx, const sparstar_segment* q_segs, int32_t n_q_segs,
                           const sparstar_segment* k_segs, int32_t n_k_segs, int32_t block, int32_t B, int32_t H,
                           float* scores_out, void* stream);
int sparstar_random_scores(sparstar_ctx* ctx, uint64_t seed, int32_t B, int32_t H, int32_t n_q, int32_t n_k,
                           float* scores_out, void* stream);
int sparstar_remap_scores(sparstar_ctx* ctx, const float* coarse_scores, int32_t B, int32_t H, int32_t n_qc,
                          int32_t n_kc, const int32_t* q_map, const int32_t* k_map, int32_t n_q, int32_t n_k,
                          float* scores_out, void* stream);

/* ---- sparstar_sparse_attn_fwd_static -----------------------------------------------------
 * (The paper has no counterpart for this call; it exists for integration reasons only.)
 * The sparse forward for callers that must not allocate device memory - code running inside a
 * framework's memory plan, a real-time or serving loop with a frozen memory budget, or a host
 * that is not allowed to call cudaMalloc at all.  Such callers cannot even create a context
 * (sparstar_create allocates), so this call takes none: the work-order scratch and a status
 * word live in a fixed array inside the library's device image (about 257 KB, held by every
 * GPU that loads the library until the process exits).
 *   Same tensors, lists, scale and lse as sparstar_sparse_attn_fwd, with these limits:
 *     bf16, D = 128, block = 128 only (SPARSTAR_ERR_UNSUPPORTED otherwise);
 *     B * H * ceil(L_q / 128) <= 65536 work items and ceil(L_q / 128) <= 51200 query tiles per
 *     (batch, head), else SPARSTAR_ERR_TOO_LARGE and nothing is enqueued.
 *   status_out  nullable DEVICE pointer to two int32 {status, site}: zeroed by this call
 *     (stream-ordered) and then written by the kernel with the first device-side condition
 *     (bad list entry, expired wait).  If NULL the built-in word is used and cannot be read back.
 * It calls no cudaMalloc/cudaFree and no allocating library routine.  The first call on each
 * device looks up the array's device address (that device must be current, as for every later
 * call) and sets two kernel attributes; make that first call outside any stream capture.
 * All calls share the one array, which keeps the previous call's contents (this call rewrites
 * every entry it reads): two calls whose kernels can overlap on the GPU - different streams
 * without ordering - race on it; order them on one stream or with events. */
int sparstar_sparse_attn_fwd_static(const sparstar_tensor* q, const sparstar_tensor* k,
                                    const sparstar_tensor* v, const sparstar_tensor* o, int32_t block,
                                    float scale, const int32_t* kv_num_blocks, const int32_t* kv_indices,
                                    int32_t cap, float* lse, int32_t* status_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SPARSTAR_H_ */
