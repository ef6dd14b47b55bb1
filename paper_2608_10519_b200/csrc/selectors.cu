// Comparison selectors of the paper's selection-strategy ablation (the table that sets fresh
// aggregated-QK selection beside a sliding window, random blocks and cross-scale reuse), as score
// generators: each writes a [B,H,n_q,n_k] fp32 score array that sparstar_select_from_scores turns
// into lists with the same budget, tie rule and kept blocks as the method's own selector.  The
// paper names these selectors without defining them; the definitions below are this library's.
//   window  score = -(Euclidean distance between the normalised (t, h, w) centres of the query
//           block and the key block); tokens without a position (text) sit at (1/2, 1/2, 1/2)
//   random  score = a counter-based uniform number in [0, 1) per (batch, head, query block, key block)
//   remap   score of a coarser scale carried over by position: out[i][j] = coarse[q_map[i]][k_map[j]]
// Block centres and the nearest-centre maps are host integer / fp64 work (small: one value per block).
#include <math.h>

#include "common.cuh"

namespace {

constexpr int kMaxSegs = 8;
struct SegList {
  int n;
  long long length[kMaxSegs];
  int T[kMaxSegs], H[kMaxSegs], W[kMaxSegs];
};

// Centre of block `blk` (tokens [blk*block, min((blk+1)*block, L))) of a token sequence made of the
// segments in order.  Per segment the raster indices of the block's tokens are summed as integers
// and divided once by the grid extent; the partial sums are added in segment order and divided by
// the token count.  Host and device run the same operations in the same order in fp64.
__host__ __device__ inline void block_centre(const SegList& sl, int block, long long blk, double* c3) {
  const long long lo = blk * block, hi = lo + block;
  double st = 0.0, sh = 0.0, sw = 0.0;
  long long cnt = 0, pos = 0;
  for (int s = 0; s < sl.n; ++s) {
    const long long a = lo > pos ? lo : pos;
    const long long e = pos + sl.length[s];
    const long long b = hi < e ? hi : e;
    if (a < b) {
      const long long m = b - a;
      if (sl.T[s] <= 0) {
        st = st + 0.5 * (double)m; sh = sh + 0.5 * (double)m; sw = sw + 0.5 * (double)m;
      } else {
        const long long HW = (long long)sl.H[s] * sl.W[s];
        long long it = 0, ih = 0, iw = 0;
        for (long long u = a - pos; u < b - pos; ++u) {
          it += u / HW;
          ih += (u / sl.W[s]) % sl.H[s];
          iw += u % sl.W[s];
        }
        st = st + (double)it / (double)sl.T[s];
        sh = sh + (double)ih / (double)sl.H[s];
        sw = sw + (double)iw / (double)sl.W[s];
      }
      cnt += m;
    }
    pos = e;
  }
  const double d = cnt > 0 ? (double)cnt : 1.0;
  c3[0] = st / d; c3[1] = sh / d; c3[2] = sw / d;
}

int fill_segs(const sparstar_segment* segs, int32_t n, SegList* out, long long* total) {
  if (segs == nullptr || n <= 0 || n > kMaxSegs) return SPARSTAR_ERR_INVALID_ARG;
  out->n = n;
  long long L = 0;
  for (int i = 0; i < n; ++i) {
    if (segs[i].length <= 0) return SPARSTAR_ERR_INVALID_ARG;
    if (segs[i].T > 0 && (segs[i].H <= 0 || segs[i].W <= 0 ||
                          (long long)segs[i].T * segs[i].H * segs[i].W != segs[i].length))
      return SPARSTAR_ERR_INVALID_ARG;
    out->length[i] = segs[i].length;
    out->T[i] = segs[i].T > 0 ? segs[i].T : 0; out->H[i] = segs[i].H; out->W[i] = segs[i].W;
    L += segs[i].length;
  }
  *total = L;
  return SPARSTAR_OK;
}

__global__ void __launch_bounds__(128)
centres_kernel(const SegList q, const SegList k, int block, int n_q, int n_k, double* __restrict__ out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_q + n_k) return;
  if (i < n_q) block_centre(q, block, i, out + 3 * (size_t)i);
  else block_centre(k, block, i - n_q, out + 3 * (size_t)i);
}

__global__ void __launch_bounds__(256)
window_scores_kernel(const double* __restrict__ centres, int n_q, int n_k, int BH, float* __restrict__ out) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)n_q * n_k) return;
  const int i = (int)(idx / n_k), j = (int)(idx % n_k);
  const double* a = centres + 3 * (size_t)i;
  const double* b = centres + 3 * ((size_t)n_q + j);
  const double dt = __dsub_rn(a[0], b[0]), dh = __dsub_rn(a[1], b[1]), dw = __dsub_rn(a[2], b[2]);
  const double d2 = __dadd_rn(__dadd_rn(__dmul_rn(dt, dt), __dmul_rn(dh, dh)), __dmul_rn(dw, dw));
  const float s = __double2float_rn(-__dsqrt_rn(d2));
  for (int bh = 0; bh < BH; ++bh) out[(size_t)bh * n_q * n_k + idx] = s;
}

__host__ __device__ inline unsigned long long mix64(unsigned long long z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__global__ void __launch_bounds__(256)
random_scores_kernel(unsigned long long seed, long long total, float* __restrict__ out) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const unsigned long long z = mix64(seed + (unsigned long long)(idx + 1) * 0x9E3779B97F4A7C15ull);
  out[idx] = (float)(z >> 40) * 5.9604644775390625e-8f;              // 24 bits -> [0, 1)
}

__global__ void __launch_bounds__(256)
remap_scores_kernel(const float* __restrict__ coarse, int n_qc, int n_kc, const int* __restrict__ q_map,
                    const int* __restrict__ k_map, int n_q, int n_k, float* __restrict__ out,
                    sparstar_devstatus* status) {
  const int bh = blockIdx.y;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)n_q * n_k) return;
  const int i = (int)(idx / n_k), j = (int)(idx % n_k);
  int ic = q_map[i], jc = k_map[j];
  if (ic < 0 || ic >= n_qc || jc < 0 || jc >= n_kc) {                 // malformed map: flag it, stay in bounds
    record_status(status, SPARSTAR_ERR_BAD_INDEX, i);
    ic = min(max(ic, 0), n_qc - 1); jc = min(max(jc, 0), n_kc - 1);
  }
  out[(size_t)bh * n_q * n_k + idx] = coarse[((size_t)bh * n_qc + ic) * n_kc + jc];
}

}  // namespace

extern "C" {

int32_t sparstar_block_centres(const sparstar_segment* segs, int32_t n_segs, int32_t block, double* centres) {
  SegList sl;
  long long L = 0;
  if (block <= 0 || fill_segs(segs, n_segs, &sl, &L) != SPARSTAR_OK) return -1;
  const long long nb = (L + block - 1) / block;
  if (nb > INT32_MAX) return -1;
  if (centres != nullptr)
    for (long long i = 0; i < nb; ++i) block_centre(sl, block, i, centres + 3 * i);
  return (int32_t)nb;
}

int32_t sparstar_nearest_block_map(const double* fine, int32_t n_fine, const double* coarse, int32_t n_coarse,
                                   int32_t* map) {
  if (fine == nullptr || coarse == nullptr || map == nullptr || n_fine <= 0 || n_coarse <= 0) return -1;
  for (int32_t i = 0; i < n_fine; ++i) {
    int32_t best = 0;
    double bd = INFINITY;
    for (int32_t j = 0; j < n_coarse; ++j) {
      const double dt = fine[3 * i] - coarse[3 * j], dh = fine[3 * i + 1] - coarse[3 * j + 1],
                   dw = fine[3 * i + 2] - coarse[3 * j + 2];
      const double d2 = (dt * dt + dh * dh) + dw * dw;
      if (d2 < bd) { bd = d2; best = j; }                             // ties: the lower index stays
    }
    map[i] = best;
  }
  return n_fine;
}

int sparstar_window_scores(sparstar_ctx* ctx, const sparstar_segment* q_segs, int32_t n_q_segs,
                           const sparstar_segment* k_segs, int32_t n_k_segs, int32_t block, int32_t B, int32_t H,
                           float* scores_out, void* stream) {
  if (ctx == nullptr) return SPARSTAR_ERR_INVALID_ARG;
  int st = ctx_device_current(ctx);
  if (st != SPARSTAR_OK) return st;
  if (scores_out == nullptr || block <= 0 || B <= 0 || H <= 0) return SPARSTAR_ERR_INVALID_ARG;
  SegList q, k;
  long long L_q = 0, L_k = 0;
  if ((st = fill_segs(q_segs, n_q_segs, &q, &L_q)) || (st = fill_segs(k_segs, n_k_segs, &k, &L_k))) return st;
  const long long n_q = (L_q + block - 1) / block, n_k = (L_k + block - 1) / block;
  if (n_q + n_k > (1 << 24)) return SPARSTAR_ERR_TOO_LARGE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  st = ensure_scratch(ctx, sizeof(double) * 3 * (size_t)(n_q + n_k), s);
  if (st != SPARSTAR_OK) return st;
  double* centres = static_cast<double*>(ctx->scratch);
  centres_kernel<<<(unsigned)((n_q + n_k + 127) / 128), 128, 0, s>>>(q, k, block, (int)n_q, (int)n_k, centres);
  window_scores_kernel<<<(unsigned)((n_q * n_k + 255) / 256), 256, 0, s>>>(centres, (int)n_q, (int)n_k, B * H, scores_out);
  ctx->launches += 2;
  SPARSTAR_CUDA_TRY(cudaGetLastError());
  return SPARSTAR_OK;
}

int sparstar_random_scores(sparstar_ctx* ctx, uint64_t seed, int32_t B, int32_t H, int32_t n_q, int32_t n_k,
                           float* scores_out, void* stream) {
  if (ctx == nullptr) return SPARSTAR_ERR_INVALID_ARG;
  const int st = ctx_device_current(ctx);
  if (st != SPARSTAR_OK) return st;
  if (scores_out == nullptr || B <= 0 || H <= 0 || n_q <= 0 || n_k <= 0) return SPARSTAR_ERR_INVALID_ARG;
  const long long total = (long long)B * H * n_q * n_k;
  if ((total + 255) / 256 > 2147483647ll) return SPARSTAR_ERR_TOO_LARGE;
  random_scores_kernel<<<(unsigned)((total + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      (unsigned long long)seed, total, scores_out);
  ctx->launches++;
  SPARSTAR_CUDA_TRY(cudaGetLastError());
  return SPARSTAR_OK;
}

int sparstar_remap_scores(sparstar_ctx* ctx, const float* coarse_scores, int32_t B, int32_t H, int32_t n_qc,
                          int32_t n_kc, const int32_t* q_map, const int32_t* k_map, int32_t n_q, int32_t n_k,
                          float* scores_out, void* stream) {
  if (ctx == nullptr) return SPARSTAR_ERR_INVALID_ARG;
  const int st = ctx_device_current(ctx);
  if (st != SPARSTAR_OK) return st;
  if (coarse_scores == nullptr || q_map == nullptr || k_map == nullptr || scores_out == nullptr || B <= 0 || H <= 0 ||
      n_qc <= 0 || n_kc <= 0 || n_q <= 0 || n_k <= 0)
    return SPARSTAR_ERR_INVALID_ARG;
  if ((long long)B * H > 65535) return SPARSTAR_ERR_UNSUPPORTED;
  dim3 grid((unsigned)(((long long)n_q * n_k + 255) / 256), (unsigned)(B * H));
  remap_scores_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(coarse_scores, n_qc, n_kc, q_map, k_map,
                                                                           n_q, n_k, scores_out, ctx->d_status);
  ctx->launches++;
  SPARSTAR_CUDA_TRY(cudaGetLastError());
  return SPARSTAR_OK;
}

}  // extern "C"
