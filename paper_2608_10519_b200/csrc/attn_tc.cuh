// Declarations shared by the tensor-core attention kernels (attn_tc.cu: two-stream kernel, mass
// and gathered-block instances; attn_tc3.cu: three-tile pipeline): geometry constants, the kernel
// parameter block, the trace macro and the tensor-map builder.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace {

constexpr int kBlock = 128;
constexpr int kD = 128;                      // head dimension of the default instance (64 is the other)
constexpr int kThreads_ = 384;
constexpr int kThreads = kThreads_;          // three warpgroups: softmax 0, softmax 1, {producer, MMA, 2 idle}
constexpr int kStages = 3;
constexpr float kSumLimit = 1.152921504606846976e18f;   // 2^60: a tile's sum of exponentials above this raises the reference
// Register budget: the kernel is launched with kRegsLaunch per thread (what 384 threads allow);
// the softmax warpgroups then grow and the third warpgroup shrinks.  setmaxnreg.inc blocks until
// the CTA's pool holds enough registers, so the three budgets must fit the launch allocation.
constexpr int kRegsLaunch = 168, kRegsSoftmax = 224, kRegsOther = 56;
static_assert(2 * 128 * kRegsSoftmax + 128 * kRegsOther <= kThreads_ * kRegsLaunch, "register budgets exceed the CTA's pool");
constexpr uint32_t kTileBytes = kBlock * kD * 2;        // 32 KB
constexpr uint32_t kHalfBytes = kTileBytes / 2;         // one 64-column half

// shared memory map (offsets from the 1024-byte aligned base)
constexpr uint32_t kOffQ = 0;
constexpr uint32_t kOffK = kOffQ + kTileBytes;
constexpr uint32_t kOffV = kOffK + kStages * kTileBytes;
constexpr uint32_t kOffBar = kOffV + kStages * kTileBytes;
// barriers (8 bytes each)
enum {
  BAR_Q = 0,                             // Q, K_0, K_1
  BAR_STAGE = 1,                         // 3: {V_u, K_{u+2}} landed
  BAR_SFULL = BAR_STAGE + kStages,       // 4: S of tile t is complete (barrier t % 4), which is also the end of service t-2
  BAR_PFULL = BAR_SFULL + 4,             // 2: the stream's softmax warpgroup wrote P
  BAR_OFULL = BAR_PFULL + 2,             // 2: the stream's last P V completed
  BAR_COUNT = BAR_OFULL + 2
};
constexpr uint32_t kOffMisc = kOffBar + 8 * BAR_COUNT;   // tmem base, abort flag
constexpr uint32_t kOffStats = kOffMisc + 16;            // (m, l) per stream and row: 2 x 128 x float2
constexpr int kTraceSlots = 48;
constexpr uint32_t kOffTrace = kOffStats + 2 * 128 * 8;  // [4 roles][kTraceSlots] packed (tag, clock)
constexpr uint32_t kSmemBytes = kOffTrace + 4 * kTraceSlots * 4;
constexpr uint32_t smem_bytes_for(int hd) {
  return (1u + 2u * kStages) * (128u * (uint32_t)hd * 2u) + 8u * BAR_COUNT + 16u + 2u * 128u * 8u + 4u * kTraceSlots * 4u;
}
static_assert(smem_bytes_for(128) == kSmemBytes, "shared memory map");

}  // namespace

struct TcParams {
  void* o;
  long long osB, osH, osL;
  int H, L_q, L_k;
  int n_q, n_k;          // 128-token tiles along queries / keys
  int m, n_qb, n_kb;     // tiles per selection block (block = 128 * m) and block counts (the lists' domain)
  int gather;            // listed key blocks per 128-key tile: 1, or 2 / 4 for selection blocks of 64 / 32 tokens.
                         // Then a list belongs to a query TILE: entries (block << 4) | bits, bit s set if the
                         // block is kept by the tile's s-th query block (attn_union_kernel); m = 1, n_qb = n_q,
                         // K/V maps with boxes of 128/gather rows
  float scale;
  const int* kv_num_blocks;
  const int* kv_indices;
  int cap;
  const float* lse_in;   // mass mode: [B,H,L_q] log-sum-exp of the dense attention (natural log)
  float* mass_out;       // mass mode: [B,H,n_qb,n_kb] (per selection block)
  int mass_g;            // mass mode: selection blocks per 128-token tile (1, or 2 / 4 for blocks of 64 / 32 tokens)
  const int* order;      // optional [B*H][n_q]: query blocks of each head, longest list first
  float* lse;
  sparstar_devstatus* status;
  int debug_drop_stage;  // >= 0: the producer arms this stage's barrier but issues no copy (exercises the bounded waits)
  long long* trace;      // optional: clock stamps of CTA (0,0,0), [4 roles][trace_cap] pairs (tag, clock)
  int trace_cap;
  int trace_skip;
};

namespace {

// Appends (tag, SM clock) to the role's trace lane in shared memory: one leader thread per
// role, first CTA only, from list position trace_skip on, up to kTraceSlots events per role.
#define TRACE(role, tag, tile)                                                             \
  do {                                                                                     \
    if (tracing && (tile) >= p.trace_skip && trace_n < kTraceSlots) {                      \
      trace_smem[(role) * kTraceSlots + trace_n] =                                         \
          ((uint32_t)(tag) << 26) | ((uint32_t)clock() & 0x3FFFFFFu);                      \
      ++trace_n;                                                                           \
    }                                                                                      \
  } while (0)

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// [B,H,L,D] bf16 -> 4-D map {D, L, H, B}, box {64, box_rows, 1, 1}, 128-byte swizzle, zero fill.
int make_map(CUtensorMap* map, const sparstar_tensor& t, int box_rows = 128) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return SPARSTAR_ERR_CUDA;
  cuuint64_t dims[4] = {(cuuint64_t)t.D, (cuuint64_t)t.L, (cuuint64_t)t.H, (cuuint64_t)t.B};
  // a stride of 0 (size-1 dimension given as 0) is not accepted: give the natural value
  cuuint64_t sH = t.H > 1 ? (cuuint64_t)t.sH : (cuuint64_t)t.sL * t.L;
  cuuint64_t sB = t.B > 1 ? (cuuint64_t)t.sB : sH * t.H;
  cuuint64_t strides[3] = {(cuuint64_t)t.sL * 2, sH * 2, sB * 2};
  cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, t.ptr, dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SPARSTAR_OK : SPARSTAR_ERR_INVALID_ARG;
}

}  // namespace

// The three-tile pipeline (attn_tc3.cu): same parameters, lists of whole 128-token tiles or
// selection blocks that are multiples of a tile (p.gather == 1), attention only.
int launch_attn_tc3(sparstar_ctx* ctx, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                    const TcParams& p, int head_dim, dim3 grid, cudaStream_t s, bool pair = false, bool gathered = false);
