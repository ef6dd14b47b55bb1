// Block-score GEMM S = scale * qbar kbar^T (Eq. 2) on the sm_100a tensor cores, used as a
// pre-score: fp32-grade values that the selection kernel then makes exact next to the cutoff.
//
// fp32 operands cannot enter tcgen05.mma directly, and a single bf16 or tf32 pass is three
// orders of magnitude too coarse for a ranking, so every operand is split into three bf16 terms
// x = hi + mid + lo (24 mantissa bits in all) and the six products whose weight is above 2^-24
// are accumulated in fp32 in tensor memory:
//     hi*hi + hi*mid + mid*hi + mid*mid + hi*lo + lo*hi
// One CTA per 128 x 128 tile of S of one head.  The threads split the pooled fp32 rows while
// copying them into shared memory in the 128-byte-swizzled K-major layout the MMA reads (no TMA:
// the data must be converted on the way), one thread issues the 6 x D/16 MMAs, and the four
// warps read the accumulator back with tcgen05.ld and write fp32 scores.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace {

constexpr int kTile = 128;
constexpr int kScoreThreads = 128;

// three bf16 terms of an fp32 value
__device__ __forceinline__ void split3(float x, __nv_bfloat16& hi, __nv_bfloat16& mid, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(x);
  const float r1 = x - __bfloat162float(hi);
  mid = __float2bfloat16_rn(r1);
  const float r2 = r1 - __bfloat162float(mid);
  lo = __float2bfloat16_rn(r2);
}

// byte offset of element (row, col) of a 128 x HD bf16 tile stored as 64-column halves of
// 128-byte rows with the 128-byte swizzle (16-byte chunk index xor row mod 8)
__device__ __forceinline__ uint32_t swz_offset(int row, int col) {
  const int half = col >> 6, c = col & 63;
  const int chunk = (c >> 3) ^ (row & 7);
  return (uint32_t)half * (kTile * 128u) + (uint32_t)row * 128u + (uint32_t)chunk * 16u + (uint32_t)(c & 7) * 2u;
}

struct ScoreTcParams {
  const float* q_pooled;   // [BH, n_q, D]
  const float* k_pooled;   // [BH, n_k, D]
  float* scores;           // [BH, n_q, n_k]
  int n_q, n_k;
  float scale;
  sparstar_devstatus* status;
};

// Shared memory: A_hi | A_mid | A_lo | B_hi | B_mid | B_lo (each 128 x HD bf16), then the control words.
template <int HD>
__global__ void __launch_bounds__(kScoreThreads, 1)
score_tc_kernel(const ScoreTcParams p) {
  constexpr uint32_t kTileBytes = kTile * HD * 2u;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  if ((base & 1023u) != 0u) {
    if (threadIdx.x == 0) record_status(p.status, SPARSTAR_ERR_CUDA, 901);
    return;
  }
  // control words live behind the tiles so that the tiles keep their 1024-byte alignment
  uint64_t& mma_bar = *reinterpret_cast<uint64_t*>(smem_raw + 6u * kTileBytes);
  uint32_t& tmem_slot = *reinterpret_cast<uint32_t*>(smem_raw + 6u * kTileBytes + 8);
  volatile int& abort_flag = *reinterpret_cast<volatile int*>(smem_raw + 6u * kTileBytes + 12);
  const int tid = threadIdx.x, warp = tid >> 5;
  const int j0 = blockIdx.x * kTile, i0 = blockIdx.y * kTile, bh = blockIdx.z;

  if (tid == 0) {
    mbar_init(smem_u32(&mma_bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), 128);

  // split + swizzled copy: thread t converts 4 consecutive fp32 of one row per step (16-byte loads)
  const float* qg = p.q_pooled + ((size_t)bh * p.n_q + i0) * HD;
  const float* kg = p.k_pooled + ((size_t)bh * p.n_k + j0) * HD;
  constexpr int kVecPerRow = HD / 4;
  for (int e = tid; e < kTile * kVecPerRow; e += kScoreThreads) {
    const int row = e / kVecPerRow, c4 = (e % kVecPerRow) * 4;
#pragma unroll
    for (int which = 0; which < 2; ++which) {
      const bool valid = which == 0 ? (i0 + row < p.n_q) : (j0 + row < p.n_k);
      const float* src = (which == 0 ? qg : kg) + (size_t)row * HD + c4;
      const float4 x = valid ? *reinterpret_cast<const float4*>(src) : make_float4(0.f, 0.f, 0.f, 0.f);
      const float xs[4] = {x.x, x.y, x.z, x.w};
      __nv_bfloat16 h[4], m[4], l[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) split3(xs[i], h[i], m[i], l[i]);
      unsigned char* tile = smem_raw + (which == 0 ? 0u : 3u * kTileBytes);
      const uint32_t off = swz_offset(row, c4);          // 4 elements = 8 bytes inside one 16-byte chunk
      *reinterpret_cast<uint2*>(tile + off) =
          make_uint2(((uint32_t)__bfloat16_as_ushort(h[1]) << 16) | __bfloat16_as_ushort(h[0]),
                     ((uint32_t)__bfloat16_as_ushort(h[3]) << 16) | __bfloat16_as_ushort(h[2]));
      *reinterpret_cast<uint2*>(tile + kTileBytes + off) =
          make_uint2(((uint32_t)__bfloat16_as_ushort(m[1]) << 16) | __bfloat16_as_ushort(m[0]),
                     ((uint32_t)__bfloat16_as_ushort(m[3]) << 16) | __bfloat16_as_ushort(m[2]));
      *reinterpret_cast<uint2*>(tile + 2u * kTileBytes + off) =
          make_uint2(((uint32_t)__bfloat16_as_ushort(l[1]) << 16) | __bfloat16_as_ushort(l[0]),
                     ((uint32_t)__bfloat16_as_ushort(l[3]) << 16) | __bfloat16_as_ushort(l[2]));
    }
  }
  // the MMA reads shared memory through the async proxy: make the generic-proxy stores visible
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;

  if (tid < 32) {                                          // warp 0, converged: one elected lane issues
    constexpr uint32_t idesc = instr_desc(false, 128u);
    // (A term, B term) pairs, largest weight first
    const int pa[6] = {0, 0, 1, 1, 0, 2};
    const int pb[6] = {0, 1, 0, 1, 2, 0};
    uint32_t acc = 0u;
#pragma unroll
    for (int t = 0; t < 6; ++t) {
      const uint64_t ad = smem_desc(base + (uint32_t)pa[t] * kTileBytes, 16, 1024);
      const uint64_t bd = smem_desc(base + (3u + (uint32_t)pb[t]) * kTileBytes, 16, 1024);
#pragma unroll
      for (int kk = 0; kk < HD / 16; ++kk) {
        const uint64_t off = (uint64_t)((((uint32_t)kk >> 2) * (kTile * 128u) + ((uint32_t)kk & 3u) * 32u) >> 4);
        umma_ss(tmem, ad + off, bd + off, idesc, acc);
        acc = 1u;
      }
    }
    umma_commit(smem_u32(&mma_bar));
  }
  const bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&mma_bar), 0u, &abort_flag, 400));
  tc_fence_after();
  if (ok) {
    const int row = i0 + tid;                              // thread = accumulator row = TMEM lane
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    float* out = p.scores + ((size_t)bh * p.n_q + row) * p.n_k + j0;
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
      uint32_t r[32];
      tmem_ld32(tmem + lane_off + 32u * cc, r);
      tmem_wait_ld();
      if (row < p.n_q) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int col = j0 + cc * 32 + i;
          if (col < p.n_k) out[cc * 32 + i] = __uint_as_float(r[i]) * p.scale;
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0) tmem_dealloc(tmem, 128);
  if (tid == 0 && abort_flag != 0) record_status(p.status, SPARSTAR_ERR_TIMEOUT, abort_flag);
}

template <int HD>
int launch_hd(sparstar_ctx* ctx, const ScoreTcParams& p, int BH, cudaStream_t s) {
  constexpr size_t smem = 6u * kTile * HD * 2u + 64u;
  static bool attr_set[64] = {};
  if (!attr_set[ctx->device & 63]) {
    SPARSTAR_CUDA_TRY(cudaFuncSetAttribute(score_tc_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    attr_set[ctx->device & 63] = true;
  }
  dim3 grid((p.n_k + kTile - 1) / kTile, (p.n_q + kTile - 1) / kTile, BH);
  score_tc_kernel<HD><<<grid, kScoreThreads, smem, s>>>(p);
  ctx->launches++;
  SPARSTAR_CUDA_TRY(cudaGetLastError());
  return SPARSTAR_OK;
}

}  // namespace

bool score_tc_supported(int D, long long BH) { return (D == 128 || D == 64) && BH <= 65535; }

int launch_score_tc(sparstar_ctx* ctx, const float* q_pooled, const float* k_pooled, int BH, int n_q, int n_k, int D,
                    float scale, float* scores, cudaStream_t s) {
  ScoreTcParams p;
  p.q_pooled = q_pooled; p.k_pooled = k_pooled; p.scores = scores;
  p.n_q = n_q; p.n_k = n_k; p.scale = scale;
  p.status = ctx->d_status;
  if (D == 128) return launch_hd<128>(ctx, p, BH, s);
  if (D == 64) return launch_hd<64>(ctx, p, BH, s);
  return SPARSTAR_ERR_UNSUPPORTED;
}
