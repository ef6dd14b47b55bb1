// Shared declarations of the sm_100a library: context, device status word, launch plumbing.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/sparstar.h"

// Device status word: {status, site}.  The first condition recorded wins.
struct sparstar_devstatus {
  int status;
  int site;
};

struct sparstar_ctx {
  int device;
  int sm_count;
  int attn_impl;
  int score_impl;
  long long launches;
  sparstar_devstatus* d_status;   // device
  sparstar_devstatus* h_status;   // pinned host mirror used by sparstar_check
  void* scratch;                  // device scratch owned by the context, grown on first use
  size_t scratch_bytes;
  void* retired[32];              // outgrown scratch buffers: kept until destroy, because work already
  int n_retired;                  // enqueued (or a captured graph) may still name their addresses
  int debug_work_order;           // test switch: 0 = the sparse attention walks query tiles in index order
  int debug_drop_stage;           // test switch: >= 0 = the TMA producer skips the copy of this list position
  long long* trace;               // optional device buffer for clock stamps (caller-owned)
  int trace_cap;
  int trace_skip;
};

__device__ __forceinline__ void record_status(sparstar_devstatus* st, int status, int site) {
  if (atomicCAS(&st->status, 0, status) == 0) st->site = site;
}

// Up to 16 forced block intervals [begin, end), merged and ascending, passed by value.
struct ForcedBlocks {
  int n;
  int begin[16];
  int end[16];
};

__host__ __device__ __forceinline__ bool is_forced(const ForcedBlocks& f, int j) {
  bool r = false;
#pragma unroll 1
  for (int i = 0; i < f.n; ++i) r = r || (j >= f.begin[i] && j < f.end[i]);
  return r;
}

#define SPARSTAR_CUDA_TRY(expr)                     \
  do {                                              \
    cudaError_t e__ = (expr);                       \
    if (e__ != cudaSuccess) return SPARSTAR_ERR_CUDA; \
  } while (0)

// Grows the context's device scratch to at least `bytes` (allocates only when it must grow; the
// outgrown buffer is retired, not freed).  Fails with SPARSTAR_ERR_CAPTURE if `s` is capturing.
int ensure_scratch(sparstar_ctx* ctx, size_t bytes, cudaStream_t s);
// SPARSTAR_OK iff the context's device is the calling thread's current device.
int ctx_device_current(const sparstar_ctx* ctx);

// Launchers implemented in the kernel files; each returns a sparstar_status.
int launch_pool(sparstar_ctx* ctx, const sparstar_tensor* x, int block, int first_block, int n_blocks, float* pooled,
                cudaStream_t s);

struct SelectArgs {
  const float* q_pooled;
  const float* k_pooled;
  const float* scores_in;   // optional [B,H,n_q,n_k]: rank these instead of forming q.k scores
  int refine;               // scores_in are approximate: re-score blocks next to the cutoff exactly from q/k_pooled
  int B, H, n_q, n_k, D;
  double scale;
  int mode;        // 0 = top-k with budget k, 2 = mass
  int k;
  double mass;
  ForcedBlocks forced;
  int n_sel;
  int* kv_num_blocks;
  int* kv_indices;
  int cap;
  float* scores_out;
};
int launch_score_select(sparstar_ctx* ctx, const SelectArgs& a, cudaStream_t s);
int launch_select_fused(sparstar_ctx* ctx, const SelectArgs& a, const sparstar_tensor& q, const sparstar_tensor& k, int block,
                        int first_k_block, const float* k_cond_pooled, int n_cond, float* q_pooled, float* k_pooled,
                        cudaStream_t s);
bool score_tc_supported(int D, long long BH);
int launch_score_tc(sparstar_ctx* ctx, const float* q_pooled, const float* k_pooled, int BH, int n_q, int n_k, int D,
                    float scale, float* scores, cudaStream_t s);

struct AttnArgs {
  sparstar_tensor q, k, v, o;
  int block;
  float scale;
  const int* kv_num_blocks;   // null = dense
  const int* kv_indices;
  int cap;
  float* lse;
};
int launch_attn_simt(sparstar_ctx* ctx, const AttnArgs& a, cudaStream_t s);
int launch_attn_tc(sparstar_ctx* ctx, const AttnArgs& a, cudaStream_t s);
bool attn_tc_supported(const AttnArgs& a);
int launch_block_mass_tc(sparstar_ctx* ctx, const sparstar_tensor& q, const sparstar_tensor& k, int block, float scale,
                         const float* lse_dense, float* mass_out, cudaStream_t s);
int launch_retained_mass(sparstar_ctx* ctx, const float* mass, const int* kv_num_blocks, const int* kv_indices,
                         int rows, int n_k, int cap, float* out, cudaStream_t s);
