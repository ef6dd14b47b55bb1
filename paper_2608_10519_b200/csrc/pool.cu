// Block-mean pooling (block-partition and per-head score paragraphs of Sec. "Aggregated
// Query-Key Block Selector"): xbar_i = (1/b) * sum over the block's valid tokens; the final
// partial block counts as zero-padded, so the divisor stays the nominal b.
//
// HBM-bound: every input byte is read once with 16-byte loads, coalesced along D (a warp
// covers whole consecutive rows), fp32 accumulation in a fixed order, one fp32 row written
// per block.  One CTA per (batch, head, block).
#include "pool.cuh"

namespace {

template <typename T>
__global__ void __launch_bounds__(kPoolThreads, 8)
pool_kernel(const T* __restrict__ x, float* __restrict__ pooled, int H, int L, int D, int nb,
            long long sB, long long sH, long long sL, int block, int vl, int groups, int first_block) {
  extern __shared__ float part[];             // [groups][D]
  const int blk = first_block + blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  pool_block_body<T>(x + b * sB + h * sH, pooled + (((long long)b * H + h) * nb + blk) * D, L, D, sL, block, vl, groups,
                     blk, part);
}

}  // namespace

int launch_pool(sparstar_ctx* ctx, const sparstar_tensor* x, int block, int first_block, int n_blocks, float* pooled,
                cudaStream_t s) {
  const int esz = x->dtype == SPARSTAR_BF16 ? 2 : 4;
  const int row_bytes = x->D * esz;
  if (row_bytes % 16 != 0 || row_bytes > 4096) return SPARSTAR_ERR_UNSUPPORTED;
  const int vl = row_bytes / 16;
  const int groups = kPoolThreads / vl;
  const int nb = (int)((x->L + block - 1) / block);
  if (x->H > 65535 || x->B > 65535) return SPARSTAR_ERR_UNSUPPORTED;
  if (first_block < 0 || n_blocks <= 0 || first_block + n_blocks > nb) return SPARSTAR_ERR_INVALID_ARG;
  dim3 grid(n_blocks, x->H, x->B);
  const size_t smem = (size_t)groups * x->D * sizeof(float);
  if (x->dtype == SPARSTAR_BF16) {
    pool_kernel<__nv_bfloat16><<<grid, kPoolThreads, smem, s>>>(
        (const __nv_bfloat16*)x->ptr, pooled, x->H, x->L, x->D, nb, x->sB, x->sH, x->sL, block, vl, groups, first_block);
  } else {
    pool_kernel<float><<<grid, kPoolThreads, smem, s>>>(
        (const float*)x->ptr, pooled, x->H, x->L, x->D, nb, x->sB, x->sH, x->sL, block, vl, groups, first_block);
  }
  ctx->launches++;
  SPARSTAR_CUDA_TRY(cudaGetLastError());
  return SPARSTAR_OK;
}
