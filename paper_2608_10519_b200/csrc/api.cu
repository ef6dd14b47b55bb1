// C ABI entry points: argument validation, host integer work (block partition, forced block
// sets of Eq. 3-4, budget of Eq. 5) and dispatch to the kernels.  create / destroy / check
// allocate, free and synchronise; the operator calls only enqueue work, except that a call whose
// scratch need exceeds what the context holds allocates a larger buffer first (ensure_scratch;
// sparstar_reserve_scratch does it ahead of time).
#include <math.h>
#include <new>

#include "common.cuh"

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_tensor(const sparstar_tensor* t) {
  if (t == nullptr || t->ptr == nullptr) return SPARSTAR_ERR_INVALID_ARG;
  if (t->dtype != SPARSTAR_F32 && t->dtype != SPARSTAR_BF16) return SPARSTAR_ERR_INVALID_ARG;
  if (t->B <= 0 || t->H <= 0 || t->L <= 0 || t->D <= 0) return SPARSTAR_ERR_INVALID_ARG;
  if (t->sL < t->D || t->sH < 0 || t->sB < 0) return SPARSTAR_ERR_INVALID_ARG;
  const int esz = t->dtype == SPARSTAR_BF16 ? 2 : 4;
  if (!aligned16(t->ptr)) return SPARSTAR_ERR_INVALID_ARG;
  if ((t->sL * esz) % 16 || (t->sH * esz) % 16 || (t->sB * esz) % 16) return SPARSTAR_ERR_INVALID_ARG;
  return SPARSTAR_OK;
}

// Blocks intersecting the token ranges, as merged ascending block intervals.
int forced_intervals(int64_t L_k, int32_t block, const sparstar_range* ranges, int32_t n,
                     ForcedBlocks* out, int* count) {
  if (L_k <= 0 || block <= 0 || n < 0 || n > 16 || (n > 0 && ranges == nullptr))
    return SPARSTAR_ERR_INVALID_ARG;
  const int64_t n_k = (L_k + block - 1) / block;
  int64_t lo[16], hi[16];
  int m = 0;
  for (int i = 0; i < n; ++i) {
    int64_t b = ranges[i].begin < 0 ? 0 : ranges[i].begin;
    int64_t e = ranges[i].end > L_k ? L_k : ranges[i].end;
    if (b >= e) continue;                       // empty after clipping
    lo[m] = b / block;                          // first block holding a token of the range
    hi[m] = (e - 1) / block + 1;                // one past the last such block
    if (hi[m] > n_k) hi[m] = n_k;
    ++m;
  }
  for (int i = 1; i < m; ++i)                   // insertion sort by begin
    for (int j = i; j > 0 && lo[j] < lo[j - 1]; --j) {
      int64_t t = lo[j]; lo[j] = lo[j - 1]; lo[j - 1] = t;
      t = hi[j]; hi[j] = hi[j - 1]; hi[j - 1] = t;
    }
  out->n = 0;
  int total = 0;
  for (int i = 0; i < m; ++i) {
    if (out->n > 0 && lo[i] <= out->end[out->n - 1]) {
      if (hi[i] > out->end[out->n - 1]) {
        total += (int)(hi[i] - out->end[out->n - 1]);
        out->end[out->n - 1] = (int)hi[i];
      }
    } else {
      out->begin[out->n] = (int)lo[i];
      out->end[out->n] = (int)hi[i];
      total += (int)(hi[i] - lo[i]);
      out->n++;
    }
  }
  *count = total;
  return SPARSTAR_OK;
}

int check_attn(const sparstar_tensor* q, const sparstar_tensor* k, const sparstar_tensor* v,
               const sparstar_tensor* o, int block) {
  int st;
  if ((st = check_tensor(q)) || (st = check_tensor(k)) || (st = check_tensor(v)) || (st = check_tensor(o)))
    return st;
  if (block <= 0) return SPARSTAR_ERR_INVALID_ARG;
  if (q->dtype != k->dtype || q->dtype != v->dtype || q->dtype != o->dtype) return SPARSTAR_ERR_INVALID_ARG;
  if (k->B != q->B || v->B != q->B || o->B != q->B) return SPARSTAR_ERR_INVALID_ARG;
  if (k->H != q->H || v->H != q->H || o->H != q->H) return SPARSTAR_ERR_INVALID_ARG;
  if (k->D != q->D || v->D != q->D || o->D != q->D) return SPARSTAR_ERR_INVALID_ARG;
  if (v->L != k->L || o->L != q->L) return SPARSTAR_ERR_INVALID_ARG;
  return SPARSTAR_OK;
}

int dispatch_attn(sparstar_ctx* ctx, const AttnArgs& a, cudaStream_t s) {
  const int impl = ctx->attn_impl;
  if (impl == SPARSTAR_ATTN_TCGEN05 || impl == SPARSTAR_ATTN_TCGEN05_2STREAM || impl == SPARSTAR_ATTN_TCGEN05_PAIR) {
    if (!attn_tc_supported(a)) return SPARSTAR_ERR_UNSUPPORTED;
    return launch_attn_tc(ctx, a, s);
  }
  if (impl == SPARSTAR_ATTN_AUTO && attn_tc_supported(a)) return launch_attn_tc(ctx, a, s);
  return launch_attn_simt(ctx, a, s);
}

}  // namespace

int ensure_scratch(sparstar_ctx* ctx, size_t bytes, cudaStream_t s) {
  if (bytes <= ctx->scratch_bytes) return SPARSTAR_OK;
  // A stream that is capturing cannot allocate, and a graph captured earlier keeps the address it
  // was given: the old buffer is therefore never freed before sparstar_destroy, only retired.
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  SPARSTAR_CUDA_TRY(cudaStreamIsCapturing(s, &cap));
  if (cap != cudaStreamCaptureStatusNone) return SPARSTAR_ERR_CAPTURE;
  if (ctx->scratch != nullptr && ctx->n_retired >= 32) return SPARSTAR_ERR_TOO_LARGE;
  size_t want = bytes < (1u << 20) ? (1u << 20) : bytes;
  if (want < ctx->scratch_bytes + ctx->scratch_bytes / 2) want = ctx->scratch_bytes + ctx->scratch_bytes / 2;
  void* fresh = nullptr;
  SPARSTAR_CUDA_TRY(cudaMalloc(&fresh, want));
  if (ctx->scratch != nullptr) ctx->retired[ctx->n_retired++] = ctx->scratch;
  ctx->scratch = fresh;
  ctx->scratch_bytes = want;
  return SPARSTAR_OK;
}

int ctx_device_current(const sparstar_ctx* ctx) {
  int dev = -1;
  SPARSTAR_CUDA_TRY(cudaGetDevice(&dev));
  return dev == ctx->device ? SPARSTAR_OK : SPARSTAR_ERR_INVALID_ARG;
}

// Every operator call: a context, and its device current on the calling thread.
#define SPARSTAR_CTX_TRY(ctx)                                   \
  do {                                                          \
    if ((ctx) == nullptr) return SPARSTAR_ERR_INVALID_ARG;      \
    const int st__ = ctx_device_current(ctx);                   \
    if (st__ != SPARSTAR_OK) return st__;                       \
  } while (0)

extern "C" {

int sparstar_create(sparstar_ctx** out, int device) {
  if (out == nullptr || device < 0 || device >= 64) return SPARSTAR_ERR_INVALID_ARG;   // per-device launch state holds 64 slots
  *out = nullptr;
  int prev = 0;
  SPARSTAR_CUDA_TRY(cudaGetDevice(&prev));
  SPARSTAR_CUDA_TRY(cudaSetDevice(device));
  sparstar_ctx* c = new (std::nothrow) sparstar_ctx();
  if (c == nullptr) return SPARSTAR_ERR_CUDA;
  c->device = device;
  c->attn_impl = SPARSTAR_ATTN_AUTO;
  c->score_impl = SPARSTAR_SCORE_FP64;
  c->launches = 0;
  c->d_status = nullptr;
  c->trace = nullptr;
  c->scratch = nullptr;
  c->scratch_bytes = 0;
  c->n_retired = 0;
  c->debug_work_order = 1;
  c->debug_drop_stage = -1;
  c->trace_cap = 0;
  c->trace_skip = 0;
  c->h_status = nullptr;
  cudaError_t e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device);
  if (e == cudaSuccess) e = cudaMalloc(&c->d_status, sizeof(sparstar_devstatus));
  if (e == cudaSuccess) e = cudaMemset(c->d_status, 0, sizeof(sparstar_devstatus));
  if (e == cudaSuccess) e = cudaMallocHost(&c->h_status, sizeof(sparstar_devstatus));
  cudaSetDevice(prev);
  if (e != cudaSuccess) {
    if (c->d_status) cudaFree(c->d_status);
    if (c->h_status) cudaFreeHost(c->h_status);
    delete c;
    return SPARSTAR_ERR_CUDA;
  }
  *out = c;
  return SPARSTAR_OK;
}

int sparstar_destroy(sparstar_ctx* ctx) {
  if (ctx == nullptr) return SPARSTAR_ERR_INVALID_ARG;
  cudaFree(ctx->d_status);
  if (ctx->scratch != nullptr) cudaFree(ctx->scratch);
  for (int i = 0; i < ctx->n_retired; ++i) cudaFree(ctx->retired[i]);
  cudaFreeHost(ctx->h_status);
  delete ctx;
  return SPARSTAR_OK;
}

int sparstar_check(sparstar_ctx* ctx, void* stream, int32_t* site) {
  SPARSTAR_CTX_TRY(ctx);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  SPARSTAR_CUDA_TRY(cudaMemcpyAsync(ctx->h_status, ctx->d_status, sizeof(sparstar_devstatus),
                                    cudaMemcpyDeviceToHost, s));
  SPARSTAR_CUDA_TRY(cudaMemsetAsync(ctx->d_status, 0, sizeof(sparstar_devstatus), s));
  SPARSTAR_CUDA_TRY(cudaStreamSynchronize(s));
  if (site != nullptr) *site = ctx->h_status->site;
  return ctx->h_status->status;
}

int sparstar_set_attn_impl(sparstar_ctx* ctx, int32_t impl) {
  if (ctx == nullptr || impl < SPARSTAR_ATTN_AUTO || impl > SPARSTAR_ATTN_TCGEN05_PAIR)
    return SPARSTAR_ERR_INVALID_ARG;
  ctx->attn_impl = impl;
  return SPARSTAR_OK;
}

int sparstar_set_score_impl(sparstar_ctx* ctx, int32_t impl) {
  if (ctx == nullptr || (impl != SPARSTAR_SCORE_FP64 && impl != SPARSTAR_SCORE_TCGEN05)) return SPARSTAR_ERR_INVALID_ARG;
  ctx->score_impl = impl;
  return SPARSTAR_OK;
}

int sparstar_set_trace(sparstar_ctx* ctx, int64_t* buf, int32_t capacity, int32_t skip) {
  if (ctx == nullptr || capacity < 0 || skip < 0 || (buf == nullptr && capacity != 0)) return SPARSTAR_ERR_INVALID_ARG;
  ctx->trace = reinterpret_cast<long long*>(buf);
  ctx->trace_cap = buf == nullptr ? 0 : capacity;
  ctx->trace_skip = skip;
  return SPARSTAR_OK;
}

int sparstar_set_debug(sparstar_ctx* ctx, int32_t work_order_on, int32_t drop_stage) {
  if (ctx == nullptr) return SPARSTAR_ERR_INVALID_ARG;
  ctx->debug_work_order = work_order_on != 0 ? 1 : 0;
  ctx->debug_drop_stage = drop_stage < 0 ? -1 : drop_stage;
  return SPARSTAR_OK;
}

int sparstar_reserve_scratch(sparstar_ctx* ctx, int64_t bytes, void* stream) {
  SPARSTAR_CTX_TRY(ctx);
  if (bytes < 0) return SPARSTAR_ERR_INVALID_ARG;
  return ensure_scratch(ctx, (size_t)bytes, static_cast<cudaStream_t>(stream));
}

int64_t sparstar_scratch_bytes(const sparstar_ctx* ctx) { return ctx == nullptr ? -1 : (int64_t)ctx->scratch_bytes; }

int64_t sparstar_launch_count(const sparstar_ctx* ctx) { return ctx == nullptr ? -1 : ctx->launches; }

const char* sparstar_status_string(int status) {
  switch (status) {
    case SPARSTAR_OK: return "ok";
    case SPARSTAR_ERR_INVALID_ARG: return "invalid argument";
    case SPARSTAR_ERR_UNSUPPORTED: return "unsupported shape, dtype or block size";
    case SPARSTAR_ERR_CAPACITY: return "a row needed more list entries than cap";
    case SPARSTAR_ERR_BAD_INDEX: return "malformed key-block list entry";
    case SPARSTAR_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case SPARSTAR_ERR_CUDA: return "CUDA call failed";
    case SPARSTAR_ERR_TOO_LARGE: return "problem exceeds a fixed built-in limit of this entry point";
    case SPARSTAR_ERR_CAPTURE: return "the context scratch would have to grow while the stream is capturing";
    default: return "unknown status";
  }
}

int32_t sparstar_num_blocks(int64_t L, int32_t block) {
  if (L < 0 || block <= 0) return -1;
  const int64_t n = (L + block - 1) / block;
  return n > INT32_MAX ? -1 : (int32_t)n;
}

int32_t sparstar_budget(int32_t n_sel, double ratio) {
  if (n_sel <= 0) return 0;
  double k = ceil(ratio * (double)n_sel - 1e-9);
  if (!(k >= 1.0)) k = 1.0;
  if (k > (double)n_sel) k = (double)n_sel;
  return (int32_t)k;
}

int32_t sparstar_forced_count(int64_t L_k, int32_t block, const sparstar_range* ranges, int32_t n) {
  ForcedBlocks f;
  int count = 0;
  if (forced_intervals(L_k, block, ranges, n, &f, &count) != SPARSTAR_OK) return -1;
  return count;
}

int sparstar_pool_blocks(sparstar_ctx* ctx, const sparstar_tensor* x, int32_t block, float* pooled,
                         void* stream) {
  SPARSTAR_CTX_TRY(ctx);
  if (pooled == nullptr || block <= 0) return SPARSTAR_ERR_INVALID_ARG;
  int st = check_tensor(x);
  if (st != SPARSTAR_OK) return st;
  if (!aligned16(pooled)) return SPARSTAR_ERR_INVALID_ARG;
  const int nb = (int)((x->L + block - 1) / block);
  return launch_pool(ctx, x, block, 0, nb, pooled, static_cast<cudaStream_t>(stream));
}

int sparstar_pool_blocks_range(sparstar_ctx* ctx, const sparstar_tensor* x, int32_t block, int32_t first_block,
                               int32_t n_blocks, float* pooled, void* stream) {
  SPARSTAR_CTX_TRY(ctx);
  if (pooled == nullptr || block <= 0) return SPARSTAR_ERR_INVALID_ARG;
  int st = check_tensor(x);
  if (st != SPARSTAR_OK) return st;
  if (!aligned16(pooled)) return SPARSTAR_ERR_INVALID_ARG;
  return launch_pool(ctx, x, block, first_block, n_blocks, pooled, static_cast<cudaStream_t>(stream));
}

int32_t sparstar_keep_ranges(int32_t clip, sparstar_range text, sparstar_range ref, sparstar_range* out) {
  if (clip < 1 || out == nullptr) return -1;
  int32_t n = 0;
  if (text.end > text.begin) out[n++] = text;
  if (clip == 1 && ref.end > ref.begin) out[n++] = ref;
  return n;
}

int32_t sparstar_density_lookup(const sparstar_density_entry* table, int32_t n, int64_t L_q, double* rho) {
  if (n < 0 || (n > 0 && table == nullptr) || rho == nullptr || L_q <= 0) return -1;
  for (int32_t i = 0; i < n; ++i)
    if (table[i].L_q == L_q) {
      *rho = table[i].rho;
      return 1;
    }
  return 0;
}

int32_t sparstar_schedule_preset(int32_t id, sparstar_density_entry* out) {
  if (out == nullptr) return -1;
  static const double rho[4] = {0.625, 0.1875, 0.1875, 0.09375};
  static const int64_t tokens_480p[4] = {5040, 11520, 20640, 31800};
  static const int64_t tokens_720p[4] = {4800, 18400, 40800, 72000};
  const int64_t* t = id == SPARSTAR_SCHEDULE_480P ? tokens_480p : id == SPARSTAR_SCHEDULE_720P_PYRAMID ? tokens_720p : nullptr;
  if (t == nullptr) return -1;
  for (int i = 0; i < 4; ++i) { out[i].L_q = t[i]; out[i].rho = rho[i]; }
  return 4;
}

// Host part shared by the two selection entry points: forced block intervals (Eq. 3-4), budget
// (Eq. 5), mode decoding.
static int fill_select_args(SelectArgs* a, int32_t B, int32_t H, int32_t n_q, int32_t n_k, int32_t D, int32_t block,
                            int64_t L_k, const sparstar_select_params* params, int32_t* kv_num_blocks,
                            int32_t* kv_indices, int32_t cap) {
  if (params == nullptr || kv_num_blocks == nullptr || kv_indices == nullptr) return SPARSTAR_ERR_INVALID_ARG;
  if (B <= 0 || H <= 0 || n_q <= 0 || n_k <= 0 || D <= 0 || block <= 0 || cap <= 0 || L_k <= 0)
    return SPARSTAR_ERR_INVALID_ARG;
  if ((int64_t)n_k != (L_k + block - 1) / block) return SPARSTAR_ERR_INVALID_ARG;
  int n_forced = 0;
  int st = forced_intervals(L_k, block, params->forced, params->n_forced, &a->forced, &n_forced);
  if (st != SPARSTAR_OK) return st;
  a->B = B; a->H = H; a->n_q = n_q; a->n_k = n_k; a->D = D;
  a->n_sel = n_k - n_forced;
  a->k = 0; a->mass = 0.0;
  switch (params->mode) {
    case SPARSTAR_SEL_TOPK_RATIO:
      if (!(params->ratio >= 0.0)) return SPARSTAR_ERR_INVALID_ARG;
      a->mode = 0; a->k = sparstar_budget(a->n_sel, params->ratio);
      break;
    case SPARSTAR_SEL_TOPK_COUNT:
      if (params->count < 0) return SPARSTAR_ERR_INVALID_ARG;
      a->mode = 0; a->k = params->count < a->n_sel ? params->count : a->n_sel;
      break;
    case SPARSTAR_SEL_MASS:
      if (!(params->mass > 0.0)) return SPARSTAR_ERR_INVALID_ARG;
      a->mode = 2; a->mass = params->mass;
      break;
    default:
      return SPARSTAR_ERR_INVALID_ARG;
  }
  a->kv_num_blocks = kv_num_blocks; a->kv_indices = kv_indices; a->cap = cap;
  return SPARSTAR_OK;
}

int sparstar_score_select(sparstar_ctx* ctx, const float* q_pooled, const float* k_pooled,
                          int32_t B, int32_t H, int32_t n_q, int32_t n_k, int32_t D, int32_t block,
                          int64_t L_k, double scale, const sparstar_select_params* params,
                          int32_t* kv_num_blocks, int32_t* kv_indices, int32_t cap, float* scores_out,
                          void* stream) {
  SPARSTAR_CTX_TRY(ctx);
  if (q_pooled == nullptr || k_pooled == nullptr) return SPARSTAR_ERR_INVALID_ARG;
  if (!aligned16(q_pooled) || !aligned16(k_pooled)) return SPARSTAR_ERR_INVALID_ARG;
  SelectArgs a;
  int st = fill_select_args(&a, B, H, n_q, n_k, D, block, L_k, params, kv_num_blocks, kv_indices, cap);
  if (st != SPARSTAR_OK) return st;
  a.q_pooled = q_pooled; a.k_pooled = k_pooled; a.scores_in = nullptr; a.refine = 0;
  a.scale = scale;
  a.scores_out = scores_out;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (ctx->score_impl == SPARSTAR_SCORE_TCGEN05 && score_tc_supported(D, (long long)B * H)) {
    // tensor-core pre-score into scores_out (if given) or the context scratch, then selection
    // with exact re-scoring next to the cutoff
    float* pre = scores_out;
    if (pre == nullptr) {
      st = ensure_scratch(ctx, sizeof(float) * (size_t)B * H * n_q * n_k, s);
      if (st != SPARSTAR_OK) return st;
      pre = static_cast<float*>(ctx->scratch);
    }
    st = launch_score_tc(ctx, q_pooled, k_pooled, B * H, n_q, n_k, D, (float)scale, pre, s);
    if (st != SPARSTAR_OK) return st;
    a.scores_in = pre; a.refine = 1; a.scores_out = nullptr;
  }
  return launch_score_select(ctx, a, s);
}

int sparstar_select_fused(sparstar_ctx* ctx, const sparstar_tensor* q, const sparstar_tensor* k, int32_t block, double scale,
                          const sparstar_select_params* params, const float* k_cond_pooled, int32_t n_cond,
                          float* q_pooled, float* k_pooled, int32_t* kv_num_blocks, int32_t* kv_indices, int32_t cap,
                          void* stream) {
  SPARSTAR_CTX_TRY(ctx);
  if (q_pooled == nullptr || k_pooled == nullptr || block <= 0) return SPARSTAR_ERR_INVALID_ARG;
  int st;
  if ((st = check_tensor(q)) || (st = check_tensor(k))) return st;
  if (k->B != q->B || k->H != q->H || k->D != q->D || k->dtype != q->dtype) return SPARSTAR_ERR_INVALID_ARG;
  if (!aligned16(q_pooled) || !aligned16(k_pooled)) return SPARSTAR_ERR_INVALID_ARG;
  if (n_cond < 0 || (n_cond > 0 && (k_cond_pooled == nullptr || !aligned16(k_cond_pooled)))) return SPARSTAR_ERR_INVALID_ARG;
  const int n_q = (int)((q->L + block - 1) / block), n_k = (int)((k->L + block - 1) / block);
  // cached means are valid only for blocks that hold no token past the conditioning part; the caller
  // says how many such blocks it has
  if (n_cond > n_k) return SPARSTAR_ERR_INVALID_ARG;
  SelectArgs a;
  st = fill_select_args(&a, q->B, q->H, n_q, n_k, q->D, block, k->L, params, kv_num_blocks, kv_indices, cap);
  if (st != SPARSTAR_OK) return st;
  a.scale = scale;
  a.scores_out = nullptr;
  return launch_select_fused(ctx, a, *q, *k, block, n_cond, k_cond_pooled, n_cond, q_pooled, k_pooled,
                             static_cast<cudaStream_t>(stream));
}

int sparstar_select_from_scores(sparstar_ctx* ctx, const float* scores, int32_t B, int32_t H, int32_t n_q,
                                int32_t n_k, int32_t block, int64_t L_k, const sparstar_select_params* params,
                                int32_t* kv_num_blocks, int32_t* kv_indices, int32_t cap, void* stream) {
  SPARSTAR_CTX_TRY(ctx);
  if (scores == nullptr) return SPARSTAR_ERR_INVALID_ARG;
  SelectArgs a;
  int st = fill_select_args(&a, B, H, n_q, n_k, 4, block, L_k, params, kv_num_blocks, kv_indices, cap);
  if (st != SPARSTAR_OK) return st;
  a.q_pooled = nullptr; a.k_pooled = nullptr; a.scores_in = scores; a.refine = 0;
  a.scale = 1.0;
  a.scores_out = nullptr;
  return launch_score_select(ctx, a, static_cast<cudaStream_t>(stream));
}

int sparstar_block_mass(sparstar_ctx* ctx, const sparstar_tensor* q, const sparstar_tensor* k, int32_t block,
                        float scale, const float* lse_dense, float* mass_out, void* stream) {
  SPARSTAR_CTX_TRY(ctx);
  if (lse_dense == nullptr || mass_out == nullptr) return SPARSTAR_ERR_INVALID_ARG;
  int st;
  if ((st = check_tensor(q)) || (st = check_tensor(k))) return st;
  if (k->B != q->B || k->H != q->H || k->D != q->D || k->dtype != q->dtype) return SPARSTAR_ERR_INVALID_ARG;
  const bool block_ok = block == 32 || block == 64 || block == 128 || block == 256 || block == 512;
  if (q->dtype != SPARSTAR_BF16 || (q->D != 128 && q->D != 64) || !block_ok || q->H > 65535 || q->B > 65535)
    return SPARSTAR_ERR_UNSUPPORTED;
  return launch_block_mass_tc(ctx, *q, *k, block, scale, lse_dense, mass_out, static_cast<cudaStream_t>(stream));
}

int sparstar_retained_mass(sparstar_ctx* ctx, const float* mass, const int32_t* kv_num_blocks,
                           const int32_t* kv_indices, int32_t rows, int32_t n_k, int32_t cap, float* out,
                           void* stream) {
  SPARSTAR_CTX_TRY(ctx);
  if (mass == nullptr || kv_num_blocks == nullptr || kv_indices == nullptr || out == nullptr ||
      rows <= 0 || n_k <= 0 || cap <= 0)
    return SPARSTAR_ERR_INVALID_ARG;
  return launch_retained_mass(ctx, mass, kv_num_blocks, kv_indices, rows, n_k, cap, out,
                              static_cast<cudaStream_t>(stream));
}

int sparstar_sparse_attn_fwd(sparstar_ctx* ctx, const sparstar_tensor* q, const sparstar_tensor* k,
                             const sparstar_tensor* v, const sparstar_tensor* o, int32_t block,
                             float scale, const int32_t* kv_num_blocks, const int32_t* kv_indices,
                             int32_t cap, float* lse, void* stream) {
  SPARSTAR_CTX_TRY(ctx);
  if (kv_num_blocks == nullptr || kv_indices == nullptr || cap <= 0) return SPARSTAR_ERR_INVALID_ARG;
  int st = check_attn(q, k, v, o, block);
  if (st != SPARSTAR_OK) return st;
  AttnArgs a;
  a.q = *q; a.k = *k; a.v = *v; a.o = *o;
  a.block = block; a.scale = scale;
  a.kv_num_blocks = kv_num_blocks; a.kv_indices = kv_indices; a.cap = cap; a.lse = lse;
  return dispatch_attn(ctx, a, static_cast<cudaStream_t>(stream));
}

int sparstar_attn_fwd(sparstar_ctx* ctx, const sparstar_tensor* q, const sparstar_tensor* k,
                      const sparstar_tensor* v, const sparstar_tensor* o, int32_t block, float scale,
                      float* lse, void* stream) {
  SPARSTAR_CTX_TRY(ctx);
  int st = check_attn(q, k, v, o, block);
  if (st != SPARSTAR_OK) return st;
  AttnArgs a;
  a.q = *q; a.k = *k; a.v = *v; a.o = *o;
  a.block = block; a.scale = scale;
  a.kv_num_blocks = nullptr; a.kv_indices = nullptr; a.cap = 0; a.lse = lse;
  return dispatch_attn(ctx, a, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
