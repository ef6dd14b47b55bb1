// Aggregated query-key block scores (Eq. 2) fused with the per-row selection of key blocks
// (Eq. 3-6) and the write of the forward BlockMask fields (Sec. "Forward-Only Sparse
// Execution").
//
// One CTA owns R consecutive query blocks of one head.  Phase 1 forms the R x n_k score
// strip S = scale * qbar kbar^T with fp64 accumulation (fp32 pooled operands) and keeps it in
// shared memory: ranking is decided next to the cutoff, so the scores are kept at a precision
// where re-association cannot reorder neighbours.  Phase 2 gives each row to one warp, which
// finds the cutoff by a bitwise search on order-preserving keys (top-k: k-th largest score;
// mass: largest cutoff whose softmax mass still reaches p), then emits forced and selected
// blocks in ascending order by ballot compaction - sorted and unique by construction.
#include <cooperative_groups.h>

#include "pool.cuh"

namespace {

constexpr int kThreads = 256;
static_assert(kThreads == kPoolThreads, "the fused kernel runs the pooling routine with the selection kernel's threads");
constexpr int kWarps = kThreads / 32;
constexpr int kRegElems = 36;          // rows of up to 32 * 36 = 1,152 key blocks are searched in registers

__device__ __forceinline__ unsigned long long order_key(double s) {
  unsigned long long u = (unsigned long long)__double_as_longlong(s);
  return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}

__device__ __forceinline__ double key_to_score(unsigned long long key) {
  const unsigned long long u = (key >> 63) ? (key ^ 0x8000000000000000ull) : ~key;
  return __longlong_as_double((long long)u);
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_max(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ int warp_sum_int(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// D(8x8) += A(8x4) * B(4x8) in fp64 on the tensor cores.  Lane l holds A[l>>2][l&3], B[l&3][l>>2]
// and D[l>>2][2*(l&3) + {0,1}].
__device__ __forceinline__ void dmma_8x8x4(double& d0, double& d1, double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
               : "+d"(d0), "+d"(d1) : "d"(a), "d"(b));
}

struct Params {
  SelectArgs a;
  sparstar_devstatus* status;
  int R;          // query blocks per CTA
};

// Pooled vectors: through the read-only path when an earlier launch wrote them; through L2 when this
// very kernel wrote them before a grid-wide barrier (the fused kernel), where the read-only path
// would be allowed to return stale lines.
template <bool kSameKernel> __device__ __forceinline__ float4 ld_pooled4(const float4* ptr) {
  return kSameKernel ? __ldcg(ptr) : __ldg(ptr);
}
template <bool kSameKernel> __device__ __forceinline__ float ld_pooled(const float* ptr) {
  return kSameKernel ? __ldcg(ptr) : *ptr;
}

// The strip of R query blocks starting at i0 of (batch, head) bh: scores, then selection.
// Shared memory: qd [D][R] double | S [R][n_k] double | E [R][n_k] double (mass mode on approximate scores only)
template <int R, bool kSameKernel>
__device__ __forceinline__ void score_select_body(const Params& p, const int bh, const int i0, unsigned char* smem_raw) {
  const SelectArgs& a = p.a;
  const int D = a.D, n_k = a.n_k, n_q = a.n_q;
  double* qd = reinterpret_cast<double*>(smem_raw);
  double* S = qd + (size_t)D * R;
  double* E = S + (size_t)R * n_k;
  const int tid = threadIdx.x;

  if (a.scores_in != nullptr) {
    // given scores (e.g. exact block masses): widen them and go straight to the selection
    for (int e = tid; e < R * n_k; e += kThreads) {
      const int r = e / n_k, j = e % n_k;
      S[(size_t)r * n_k + j] = (i0 + r < n_q) ? (double)a.scores_in[((size_t)bh * n_q + i0 + r) * n_k + j] : 0.0;
    }
  } else {
  // qbar rows of this strip, widened, laid out [d][r] so one d gives R contiguous doubles
  for (int e = tid; e < R * D; e += kThreads) {
    const int r = e / D, d = e % D;
    const int i = i0 + r;
    qd[d * R + r] = (i < n_q) ? (double)ld_pooled<kSameKernel>(a.q_pooled + ((size_t)bh * n_q + i) * D + d) : 0.0;
  }
  __syncthreads();

  // ---- phase 1: score strip -----------------------------------------------------------
  const float* kb = a.k_pooled + (size_t)bh * n_k * D;
  if (R == 8 && (D == 128 || D == 64)) {
    // Tensor-core path: the strip is an 8 x n_k x D fp64 GEMM, done as m8n8k4 MMAs, one warp per
    // group of 8 key blocks.  The contraction index may be visited in any order as long as A and
    // B agree, so lane (g, t) takes d = 16 s + 4 t + e: one 16-byte load of kbar feeds four MMAs.
    const int warp_id = tid / 32, lane_id = tid % 32;
    const int g = lane_id >> 2, t4 = lane_id & 3;
    const int steps = D / 16;                              // s = 0 .. steps-1, e = 0 .. 3
    double qa[32];                                         // A fragments of the whole contraction
#pragma unroll
    for (int s_ = 0; s_ < 8; ++s_)
#pragma unroll
      for (int e = 0; e < 4; ++e)
        qa[s_ * 4 + e] = s_ < steps ? qd[(size_t)(16 * s_ + 4 * t4 + e) * R + g] : 0.0;
    for (int j0 = warp_id * 8; j0 < n_k; j0 += kWarps * 8) {
      const int col = j0 + g;
      const float4* kp = reinterpret_cast<const float4*>(kb + (size_t)min(col, n_k - 1) * D) + t4;
      float4 kv[8];
#pragma unroll
      for (int s_ = 0; s_ < 8; ++s_)
        kv[s_] = (s_ < steps && col < n_k) ? ld_pooled4<kSameKernel>(kp + 4 * s_) : make_float4(0.f, 0.f, 0.f, 0.f);
      double c0 = 0.0, c1 = 0.0;
#pragma unroll
      for (int s_ = 0; s_ < 8; ++s_) {
        if (s_ < steps) {
          dmma_8x8x4(c0, c1, qa[s_ * 4 + 0], (double)kv[s_].x);
          dmma_8x8x4(c0, c1, qa[s_ * 4 + 1], (double)kv[s_].y);
          dmma_8x8x4(c0, c1, qa[s_ * 4 + 2], (double)kv[s_].z);
          dmma_8x8x4(c0, c1, qa[s_ * 4 + 3], (double)kv[s_].w);
        }
      }
      // lane holds S[row g][j0 + 2 t + {0, 1}]
      const int jc = j0 + 2 * t4;
      const double s0 = a.scale * c0, s1 = a.scale * c1;
      if (jc < n_k) {
        S[(size_t)g * n_k + jc] = s0;
        if (a.scores_out != nullptr && i0 + g < n_q) a.scores_out[((size_t)bh * n_q + i0 + g) * n_k + jc] = (float)s0;
      }
      if (jc + 1 < n_k) {
        S[(size_t)g * n_k + jc + 1] = s1;
        if (a.scores_out != nullptr && i0 + g < n_q) a.scores_out[((size_t)bh * n_q + i0 + g) * n_k + jc + 1] = (float)s1;
      }
    }
  } else {
  // two key blocks per thread and pass: every qbar value read from shared memory feeds two FMAs
  for (int j = tid; j < n_k; j += 2 * kThreads) {
    const int j2 = j + kThreads;
    const bool two = j2 < n_k;
    double acc[R], acc2[R];
#pragma unroll
    for (int r = 0; r < R; ++r) { acc[r] = 0.0; acc2[r] = 0.0; }
    const float4* kp = reinterpret_cast<const float4*>(kb + (size_t)j * D);
    const float4* kp2 = reinterpret_cast<const float4*>(kb + (size_t)(two ? j2 : j) * D);
    for (int d4 = 0; d4 < D / 4; ++d4) {
      const float4 kv = ld_pooled4<kSameKernel>(kp + d4);
      const float4 kw = ld_pooled4<kSameKernel>(kp2 + d4);
      const double k0 = kv.x, k1 = kv.y, k2 = kv.z, k3 = kv.w;
      const double w0 = kw.x, w1 = kw.y, w2 = kw.z, w3 = kw.w;
      const double* q = qd + (size_t)d4 * 4 * R;
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const double q0 = q[r], q1 = q[R + r], q2 = q[2 * R + r], q3 = q[3 * R + r];
        acc[r] = fma(q0, k0, acc[r]);   acc2[r] = fma(q0, w0, acc2[r]);
        acc[r] = fma(q1, k1, acc[r]);   acc2[r] = fma(q1, w1, acc2[r]);
        acc[r] = fma(q2, k2, acc[r]);   acc2[r] = fma(q2, w2, acc2[r]);
        acc[r] = fma(q3, k3, acc[r]);   acc2[r] = fma(q3, w3, acc2[r]);
      }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const double s = a.scale * acc[r];
      S[(size_t)r * n_k + j] = s;
      if (a.scores_out != nullptr && i0 + r < n_q)
        a.scores_out[((size_t)bh * n_q + i0 + r) * n_k + j] = (float)s;
      if (two) {
        const double s2 = a.scale * acc2[r];
        S[(size_t)r * n_k + j2] = s2;
        if (a.scores_out != nullptr && i0 + r < n_q)
          a.scores_out[((size_t)bh * n_q + i0 + r) * n_k + j2] = (float)s2;
      }
    }
  }
  }  // FMA path
  }  // scores_in == nullptr
  __syncthreads();

  // ---- phase 2: one warp per row ------------------------------------------------------
  // The row's scores are replaced in place by order-preserving 64-bit keys split into two
  // 32-bit words (forced blocks get key 0, below every real key).  The cutoff is found by a
  // bitwise search on the high words (32 passes of cheap integer compares); only if several
  // blocks share the cutoff's high word does a second search on the low words run.
  const int warp = tid / 32, lane = tid % 32;
  for (int r = warp; r < R; r += kWarps) {
    const int i = i0 + r;
    if (i >= n_q) continue;
    double* Sr = S + (size_t)r * n_k;
    uint2* Kr = reinterpret_cast<uint2*>(Sr);       // .x = high word, .y = low word
    double* Er = E + (size_t)r * n_k;
    uint32_t Th = 0u, Tl = 0u;                       // cutoff key
    int need_eq = 0;                                 // blocks equal to the cutoff that are admitted
    bool none = false;                               // nothing selectable is taken
    double target = 0.0;
    double m = -INFINITY;                            // softmax reference of the mass mode

    // Mass mode with exact scores: exp is monotone, so the softmax numerators E_j order the
    // blocks as their scores do (and exactly as the normalised masses the selection is defined
    // on), and E_j's own bits serve as the key.  Key and mass are then one 8-byte word, the strip
    // needs no second array and every pass of the search reads half as much.
    const bool ekey = a.mode == 2 && !a.refine;
    auto mass_at = [&](const uint2& kk, int j) { return ekey ? __hiloint2double((int)kk.x, (int)kk.y) : Er[j]; };
    if (a.mode == 2 && a.n_sel > 0) {
      // softmax over selectable blocks only; E_j = exp(S_j - max)
      for (int j = lane; j < n_k; j += 32)
        if (!is_forced(a.forced, j)) m = fmax(m, Sr[j]);
      m = warp_max(m);
      double z = 0.0;
      for (int j = lane; j < n_k; j += 32) {
        const bool forced_j = is_forced(a.forced, j);
        double e = forced_j ? 0.0 : exp(Sr[j] - m);
        if (ekey) {
          // key 0 marks a forced block: a selectable block whose numerator underflows keeps the
          // smallest positive key (its mass is nil either way, ties go by index as in the definition)
          if (!forced_j && e == 0.0) e = __longlong_as_double(1ll);
          Kr[j] = make_uint2((uint32_t)__double2hiint(e), (uint32_t)__double2loint(e));
        } else {
          Er[j] = e;
        }
        z += e;
      }
      z = warp_sum(z);
      target = a.mass * z;
    }
    if (!ekey || a.n_sel == 0) {
      for (int j = lane; j < n_k; j += 32) {
        const unsigned long long key = is_forced(a.forced, j) ? 0ull : order_key(Sr[j]);
        Kr[j] = make_uint2((uint32_t)(key >> 32), (uint32_t)key);
      }
    }
    __syncwarp();

    // Search for the cutoff.  With approximate input scores (tensor-core pre-score) a second
    // pass follows if two or more blocks lie so close to the cutoff that their order is not
    // certain: those blocks are re-scored exactly in fp64 from the pooled vectors first.
    for (int pass = 0; pass < 2; ++pass) {
      Th = 0u; Tl = 0u; need_eq = 0;
      if (a.n_sel == 0 || (a.mode == 0 && a.k <= 0)) {
        none = true;
      } else if (a.mode == 0) {
        // (Th, Tl) = k-th largest key among selectable blocks
        if (n_k <= 32 * kRegElems) {
          // the row's high words fit in registers: the 32 passes touch no shared memory
          uint32_t kh[kRegElems];
#pragma unroll
          for (int i = 0; i < kRegElems; ++i) {
            const int j = lane + 32 * i;
            kh[i] = j < n_k ? Kr[j].x : 0u;               // 0 is below every candidate
          }
#pragma unroll 1
          for (int bit = 31; bit >= 0; --bit) {
            const uint32_t cand = Th | (1u << bit);
            int c = 0;
#pragma unroll
            for (int i = 0; i < kRegElems; ++i) c += kh[i] >= cand ? 1 : 0;
            if (warp_sum_int(c) >= a.k) Th = cand;
          }
        } else
        for (int bit = 31; bit >= 0; --bit) {
          const uint32_t cand = Th | (1u << bit);
          int c = 0;
          for (int j = lane; j < n_k; j += 32) c += Kr[j].x >= cand ? 1 : 0;
          if (warp_sum_int(c) >= a.k) Th = cand;
        }
        int gt = 0, eq = 0;
        for (int j = lane; j < n_k; j += 32) {
          const uint32_t hi = Kr[j].x;
          gt += hi > Th ? 1 : 0;
          eq += hi == Th ? 1 : 0;
        }
        gt = warp_sum_int(gt);
        eq = warp_sum_int(eq);
        const int need = a.k - gt;                     // 1 <= need <= eq
        if (need >= eq) {
          need_eq = eq;                                // every block of the group enters (Tl = 0)
        } else {
          for (int bit = 31; bit >= 0; --bit) {
            const uint32_t cand = Tl | (1u << bit);
            int c = 0;
            for (int j = lane; j < n_k; j += 32) {
              const uint2 kk = Kr[j];
              c += (kk.x == Th && kk.y >= cand) ? 1 : 0;
            }
            if (warp_sum_int(c) >= need) Tl = cand;
          }
          int g2 = 0;
          for (int j = lane; j < n_k; j += 32) {
            const uint2 kk = Kr[j];
            g2 += (kk.x == Th && kk.y > Tl) ? 1 : 0;
          }
          need_eq = need - warp_sum_int(g2);
        }
      } else {
        // largest cutoff with mass{key >= cutoff} >= p*Z; forced blocks carry E = 0
        if (ekey && n_k <= 32 * kRegElems) {
          // keys = masses fit in registers; four partial sums with a fixed grouping (the same in
          // every pass, so the masked sum stays monotone in the cutoff); entries past the row are 0
          double ev[kRegElems];
#pragma unroll
          for (int i = 0; i < kRegElems; ++i) {
            const int j = lane + 32 * i;
            const uint2 kk = j < n_k ? Kr[j] : make_uint2(0u, 0u);
            ev[i] = __hiloint2double((int)kk.x, (int)kk.y);
          }
#pragma unroll 1
          for (int bit = 31; bit >= 0; --bit) {
            const uint32_t cand = Th | (1u << bit);
            double f[4] = {0.0, 0.0, 0.0, 0.0};
#pragma unroll
            for (int i = 0; i < kRegElems; ++i)
              f[i & 3] += (uint32_t)__double2hiint(ev[i]) >= cand ? ev[i] : 0.0;
            if (warp_sum((f[0] + f[1]) + (f[2] + f[3])) >= target) Th = cand;
          }
        } else
        for (int bit = 31; bit >= 0; --bit) {
          const uint32_t cand = Th | (1u << bit);
          // four partial sums per lane: the additions of one pass do not wait on each other; the
          // grouping is the same in every pass, so the masked sum stays monotone in the cutoff
          double f0 = 0.0, f1 = 0.0, f2 = 0.0, f3 = 0.0;
          int j = lane;
          for (; j + 96 < n_k; j += 128) {
            const uint2 k0 = Kr[j], k1 = Kr[j + 32], k2 = Kr[j + 64], k3 = Kr[j + 96];
            f0 += k0.x >= cand ? mass_at(k0, j) : 0.0;
            f1 += k1.x >= cand ? mass_at(k1, j + 32) : 0.0;
            f2 += k2.x >= cand ? mass_at(k2, j + 64) : 0.0;
            f3 += k3.x >= cand ? mass_at(k3, j + 96) : 0.0;
          }
          for (; j < n_k; j += 32) {
            const uint2 k0 = Kr[j];
            f0 += k0.x >= cand ? mass_at(k0, j) : 0.0;
          }
          if (warp_sum((f0 + f1) + (f2 + f3)) >= target) Th = cand;
        }
        double fgt = 0.0;
        int eq = 0;
        uint32_t lo_seen = 0u;
        for (int j = lane; j < n_k; j += 32) {
          const uint2 kk = Kr[j];
          fgt += kk.x > Th ? mass_at(kk, j) : 0.0;
          if (kk.x == Th && (kk.x | kk.y) != 0u) { eq += 1; lo_seen = max(lo_seen, kk.y); }
        }
        fgt = warp_sum(fgt);
        eq = warp_sum_int(eq);
  #pragma unroll
        for (int o = 16; o > 0; o >>= 1) lo_seen = max(lo_seen, __shfl_xor_sync(0xffffffffu, lo_seen, o));
        if (eq <= 1) {
          Tl = lo_seen;                                // the single block at the cutoff
          need_eq = eq;
        } else {
          for (int bit = 31; bit >= 0; --bit) {
            const uint32_t cand = Tl | (1u << bit);
            double f = 0.0;
            for (int j = lane; j < n_k; j += 32) {
              const uint2 kk = Kr[j];
              f += (kk.x == Th && kk.y >= cand) ? mass_at(kk, j) : 0.0;
            }
            if (fgt + warp_sum(f) >= target) Tl = cand;
          }
          double f2 = 0.0, eq_e = 0.0;
          int eq_n = 0;
          for (int j = lane; j < n_k; j += 32) {
            const uint2 kk = Kr[j];
            f2 += (kk.x == Th && kk.y > Tl) ? mass_at(kk, j) : 0.0;
            if (kk.x == Th && kk.y == Tl && (kk.x | kk.y) != 0u) { eq_n += 1; eq_e = mass_at(kk, j); }
          }
          f2 = warp_sum(f2);
          eq_n = warp_sum_int(eq_n);
          eq_e = warp_max(eq_e);
          // equal-score blocks enter by ascending index until the mass is reached
          need_eq = eq_n;
          double run = fgt + f2;
          for (int t = 1; t <= eq_n; ++t) {
            run += eq_e;
            if (run >= target) { need_eq = t; break; }
          }
        }
      }

      if (!a.refine || pass == 1 || none) break;
      const double cut = key_to_score(((unsigned long long)Th << 32) | Tl);
      const double delta = 1e-4 * (1.0 + fabs(cut));   // far above the pre-score's error (about 1e-5)
      int near = 0;
      for (int j = lane; j < n_k; j += 32) {
        const uint2 kk = Kr[j];
        if ((kk.x | kk.y) != 0u && fabs(key_to_score(((unsigned long long)kk.x << 32) | kk.y) - cut) <= delta) ++near;
      }
      if (warp_sum_int(near) < 2) break;               // only the cutoff block itself: the order is certain
      const float* qrow = a.q_pooled + ((size_t)bh * n_q + i) * D;
      for (int j = lane; j < n_k; j += 32) {
        const uint2 kk = Kr[j];
        if ((kk.x | kk.y) == 0u) continue;
        if (fabs(key_to_score(((unsigned long long)kk.x << 32) | kk.y) - cut) > delta) continue;
        const float* krow = a.k_pooled + ((size_t)bh * n_k + j) * D;
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc = fma((double)ld_pooled<kSameKernel>(qrow + d), (double)ld_pooled<kSameKernel>(krow + d), acc);
        const double sx = a.scale * acc;
        const unsigned long long key = order_key(sx);
        Kr[j] = make_uint2((uint32_t)(key >> 32), (uint32_t)key);
        if (a.mode == 2) Er[j] = exp(sx - m);
      }
      __syncwarp();
    }

    // emission in ascending block order
    int* out = a.kv_indices + ((size_t)bh * n_q + i) * a.cap;
    int written = 0, eq_seen = 0;
    const unsigned lt = (1u << lane) - 1u;
    for (int j0 = 0; j0 < n_k; j0 += 32) {
      const int j = j0 + lane;
      bool take = false, eq = false;
      if (j < n_k) {
        const uint2 kk = Kr[j];
        if ((kk.x | kk.y) == 0u) {
          take = true;                               // forced block
        } else if (!none) {
          take = kk.x > Th || (kk.x == Th && kk.y > Tl);
          eq = kk.x == Th && kk.y == Tl;
        }
      }
      const unsigned eqb = __ballot_sync(0xffffffffu, eq);
      if (eq && eq_seen + __popc(eqb & lt) < need_eq) take = true;
      const unsigned tb = __ballot_sync(0xffffffffu, take);
      const int pos = written + __popc(tb & lt);
      if (take && pos < a.cap) out[pos] = j;
      written += __popc(tb);
      eq_seen += __popc(eqb);
    }
    if (lane == 0) {
      a.kv_num_blocks[(size_t)bh * n_q + i] = written;
      if (written > a.cap) record_status(p.status, SPARSTAR_ERR_CAPACITY, i);
    }
  }
}

template <int R>
__global__ void __launch_bounds__(kThreads)
score_select_kernel(const Params p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  score_select_body<R, false>(p, blockIdx.y, blockIdx.x * R, smem_raw);
}

// Pooling, scores and selection of one scale in ONE launch (cooperative: the grid is resident as a
// whole and meets at a grid-wide barrier).  Phase A: block means of Q (all blocks) and of K (blocks
// from first_k_block on; the means of the blocks before it - conditioning keys that do not change
// between the scales of a clip - are copied from k_cond_pooled), by the pooling kernel's own block
// routine, hence with its bits.  Phase B: the strips of the selection kernel, taken round-robin.
struct FusedParams {
  Params sel;
  const void* q; const void* k;          // [B,H,L,D] in the dtype T
  long long q_sB, q_sH, q_sL, k_sB, k_sH, k_sL;
  int L_q, L_k, block, vl, groups;
  int first_k_block;                     // K blocks below it come from k_cond_pooled
  const float* k_cond_pooled;            // [B,H,n_cond,D]
  int n_cond;
  float* q_pooled; float* k_pooled;      // written here, read by phase B
};

template <int R, typename T>
__global__ void __launch_bounds__(kThreads)
select_fused_kernel(const FusedParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const SelectArgs& a = p.sel.a;
  const int BH = a.B * a.H, D = a.D;
  float* part = reinterpret_cast<float*>(smem_raw);
  // ---- phase A -----------------------------------------------------------------------------
  const int kb_new = a.n_k - p.first_k_block;
  const long long n_items = (long long)BH * (a.n_q + kb_new);
  for (long long it = blockIdx.x; it < n_items; it += gridDim.x) {
    const int bh = (int)(it / (a.n_q + kb_new)), r = (int)(it % (a.n_q + kb_new));
    const int b = bh / a.H, h = bh % a.H;
    if (r < a.n_q)
      pool_block_body<T, true>(static_cast<const T*>(p.q) + b * p.q_sB + h * p.q_sH, p.q_pooled + ((size_t)bh * a.n_q + r) * D,
                         p.L_q, D, p.q_sL, p.block, p.vl, p.groups, r, part);
    else
      pool_block_body<T, true>(static_cast<const T*>(p.k) + b * p.k_sB + h * p.k_sH,
                         p.k_pooled + ((size_t)bh * a.n_k + p.first_k_block + (r - a.n_q)) * D, p.L_k, D, p.k_sL, p.block,
                         p.vl, p.groups, p.first_k_block + (r - a.n_q), part);
    __syncthreads();
  }
  if (p.first_k_block > 0) {                     // cached means of the conditioning blocks
    const long long n4 = (long long)BH * p.first_k_block * (D / 4);
    for (long long e = (long long)blockIdx.x * kThreads + threadIdx.x; e < n4; e += (long long)gridDim.x * kThreads) {
      const int d4 = (int)(e % (D / 4));
      const long long row = e / (D / 4);
      const int bh = (int)(row / p.first_k_block), j = (int)(row % p.first_k_block);
      reinterpret_cast<float4*>(p.k_pooled + ((size_t)bh * a.n_k + j) * D)[d4] =
          __ldg(reinterpret_cast<const float4*>(p.k_cond_pooled + ((size_t)bh * p.n_cond + j) * D) + d4);
    }
  }
  __threadfence();
  cooperative_groups::this_grid().sync();
  // ---- phase B -----------------------------------------------------------------------------
  const int strips = (a.n_q + R - 1) / R;
  for (long long it = blockIdx.x; it < (long long)BH * strips; it += gridDim.x) {
    score_select_body<R, true>(p.sel, (int)(it / strips), (int)(it % strips) * R, smem_raw);
    __syncthreads();
  }
}

size_t smem_bytes(const SelectArgs& a, int R) {
  const size_t strip = (size_t)R * a.n_k * sizeof(double);
  return (size_t)a.D * R * sizeof(double) + strip * (a.mode == 2 && a.refine ? 2 : 1);   // E array only beside score keys
}

template <int R>
int launch_R(sparstar_ctx* ctx, const SelectArgs& a, cudaStream_t s) {
  Params p;
  p.a = a;
  p.status = ctx->d_status;
  p.R = R;
  const size_t smem = smem_bytes(a, R);
  static bool attr_set[64] = {};   // per device
  if (!attr_set[ctx->device & 63]) {
    SPARSTAR_CUDA_TRY(cudaFuncSetAttribute(score_select_kernel<R>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    attr_set[ctx->device & 63] = true;
  }
  dim3 grid((a.n_q + R - 1) / R, a.B * a.H);
  score_select_kernel<R><<<grid, kThreads, smem, s>>>(p);
  ctx->launches++;
  SPARSTAR_CUDA_TRY(cudaGetLastError());
  return SPARSTAR_OK;
}

// Retained attention mass of every query block: sum of the block-mass row over the kept list.
__global__ void __launch_bounds__(256)
retained_mass_kernel(const float* __restrict__ mass, const int* __restrict__ num, const int* __restrict__ idx,
                     int rows, int n_k, int cap, float* __restrict__ out) {
  const int row = blockIdx.x * 8 + threadIdx.x / 32, lane = threadIdx.x % 32;
  if (row >= rows) return;
  const int c = min(num[row], cap);
  float s = 0.f;
  for (int t = lane; t < c; t += 32) {
    const int j = idx[(size_t)row * cap + t];
    if (j >= 0 && j < n_k) s += mass[(size_t)row * n_k + j];
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) out[row] = s;
}

}  // namespace

int launch_retained_mass(sparstar_ctx* ctx, const float* mass, const int* kv_num_blocks, const int* kv_indices,
                         int rows, int n_k, int cap, float* out, cudaStream_t s) {
  retained_mass_kernel<<<(rows + 7) / 8, 256, 0, s>>>(mass, kv_num_blocks, kv_indices, rows, n_k, cap, out);
  ctx->launches++;
  SPARSTAR_CUDA_TRY(cudaGetLastError());
  return SPARSTAR_OK;
}

int launch_score_select(sparstar_ctx* ctx, const SelectArgs& a, cudaStream_t s) {
  if (a.scores_in == nullptr && a.D % 4 != 0) return SPARSTAR_ERR_UNSUPPORTED;
  if ((long long)a.B * a.H > 65535) return SPARSTAR_ERR_UNSUPPORTED;
  const size_t limit = 200 * 1024;
  if (smem_bytes(a, 8) <= limit) return launch_R<8>(ctx, a, s);
  if (smem_bytes(a, 4) <= limit) return launch_R<4>(ctx, a, s);
  if (smem_bytes(a, 2) <= limit) return launch_R<2>(ctx, a, s);
  if (smem_bytes(a, 1) <= limit) return launch_R<1>(ctx, a, s);
  return SPARSTAR_ERR_UNSUPPORTED;
}


// ---- pooling + scores + selection in one cooperative launch ----------------------------------
namespace {

template <int R, typename T>
int launch_fused_RT(sparstar_ctx* ctx, FusedParams& p, size_t smem, cudaStream_t s) {
  static bool attr_set[64] = {};
  static int blocks_per_sm[64] = {};
  static size_t smem_seen[64] = {};
  const int dev = ctx->device & 63;
  if (!attr_set[dev]) {
    SPARSTAR_CUDA_TRY(cudaFuncSetAttribute(select_fused_kernel<R, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    attr_set[dev] = true;
  }
  if (blocks_per_sm[dev] == 0 || smem_seen[dev] != smem) {
    int nb = 0;
    SPARSTAR_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, select_fused_kernel<R, T>, kThreads, smem));
    if (nb <= 0) return SPARSTAR_ERR_UNSUPPORTED;
    blocks_per_sm[dev] = nb;
    smem_seen[dev] = smem;
  }
  p.sel.R = R;
  void* args[] = {&p};
  SPARSTAR_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)select_fused_kernel<R, T>, dim3(ctx->sm_count * blocks_per_sm[dev]),
                                                dim3(kThreads), args, smem, s));
  ctx->launches++;
  return SPARSTAR_OK;
}

template <typename T>
int launch_fused_T(sparstar_ctx* ctx, FusedParams& p, cudaStream_t s) {
  const SelectArgs& a = p.sel.a;
  const size_t pool_smem = (size_t)p.groups * a.D * sizeof(float);
  const size_t limit = 200 * 1024;
  auto need = [&](int R) { const size_t b = smem_bytes(a, R); return b > pool_smem ? b : pool_smem; };
  if (need(8) <= limit) return launch_fused_RT<8, T>(ctx, p, need(8), s);
  if (need(4) <= limit) return launch_fused_RT<4, T>(ctx, p, need(4), s);
  if (need(2) <= limit) return launch_fused_RT<2, T>(ctx, p, need(2), s);
  if (need(1) <= limit) return launch_fused_RT<1, T>(ctx, p, need(1), s);
  return SPARSTAR_ERR_UNSUPPORTED;
}

}  // namespace

int launch_select_fused(sparstar_ctx* ctx, const SelectArgs& a, const sparstar_tensor& q, const sparstar_tensor& k, int block,
                        int first_k_block, const float* k_cond_pooled, int n_cond, float* q_pooled, float* k_pooled,
                        cudaStream_t s) {
  if (a.D % 4 != 0 || (long long)a.B * a.H > 65535) return SPARSTAR_ERR_UNSUPPORTED;
  const int esz = q.dtype == SPARSTAR_BF16 ? 2 : 4;
  const int row_bytes = q.D * esz;
  if (row_bytes % 16 != 0 || row_bytes > 4096) return SPARSTAR_ERR_UNSUPPORTED;
  FusedParams p;
  p.sel.a = a;
  p.sel.a.q_pooled = q_pooled; p.sel.a.k_pooled = k_pooled; p.sel.a.scores_in = nullptr; p.sel.a.refine = 0;
  p.sel.status = ctx->d_status;
  p.q = q.ptr; p.k = k.ptr;
  p.q_sB = q.sB; p.q_sH = q.sH; p.q_sL = q.sL; p.k_sB = k.sB; p.k_sH = k.sH; p.k_sL = k.sL;
  p.L_q = q.L; p.L_k = k.L; p.block = block;
  p.vl = row_bytes / 16; p.groups = kThreads / p.vl;
  p.first_k_block = first_k_block; p.k_cond_pooled = k_cond_pooled; p.n_cond = n_cond;
  p.q_pooled = q_pooled; p.k_pooled = k_pooled;
  return q.dtype == SPARSTAR_BF16 ? launch_fused_T<__nv_bfloat16>(ctx, p, s) : launch_fused_T<float>(ctx, p, s);
}
