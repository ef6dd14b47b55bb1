// Block-mean pooling of one block, shared by the pooling kernel and the fused selection kernel
// (block-partition and per-head score paragraphs of Sec. "Aggregated Query-Key Block Selector").
#pragma once

#include "common.cuh"

namespace {

constexpr int kPoolThreads = 256;

template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int N = 4;
  __device__ static void add(float* acc, const uint4& u) {
    acc[0] += __uint_as_float(u.x); acc[1] += __uint_as_float(u.y);
    acc[2] += __uint_as_float(u.z); acc[3] += __uint_as_float(u.w);
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void add(float* acc, const uint4& u) {
    // bf16 -> fp32 is a 16-bit shift
    acc[0] += __uint_as_float(u.x << 16); acc[1] += __uint_as_float(u.x & 0xffff0000u);
    acc[2] += __uint_as_float(u.y << 16); acc[3] += __uint_as_float(u.y & 0xffff0000u);
    acc[4] += __uint_as_float(u.z << 16); acc[5] += __uint_as_float(u.z & 0xffff0000u);
    acc[6] += __uint_as_float(u.w << 16); acc[7] += __uint_as_float(u.w & 0xffff0000u);
  }
};

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// One block of one (batch, head): blk = block index, x already offset to the (batch, head) slice.
// vl = 16-byte vectors per row; groups = row groups that fit in the CTA (256 threads).  `part` =
// shared memory [groups][D] floats.  Fixed summation order: the result does not depend on which
// kernel calls this.  Ends with the output row written; the caller synchronises before `part` is
// reused.
template <typename T, bool kDeep = false>
__device__ __forceinline__ void pool_block_body(const T* __restrict__ xbh, float* __restrict__ out_row, int L, int D,
                                                long long sL, int block, int vl, int groups, int blk, float* part) {
  constexpr int N = Vec16<T>::N;
  const int lane = threadIdx.x % vl;
  const int grp = threadIdx.x / vl;
  const int r0 = blk * block;
  const int valid = min(block, L - r0);
  const T* base = xbh + (long long)r0 * sL;

  float acc[N];
#pragma unroll
  for (int i = 0; i < N; ++i) acc[i] = 0.f;
  if (grp < groups) {
    int r = grp;
    if (kDeep) {
      // eight loads in flight per thread (callers that run few threads per SM); the additions keep
      // the row order of the four-at-a-time loop, so the sum has the same bits
      for (; r + 7 * groups < valid; r += 8 * groups) {
        uint4 u[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) u[i] = ld_stream(reinterpret_cast<const uint4*>(base + (long long)(r + i * groups) * sL) + lane);
#pragma unroll
        for (int i = 0; i < 8; ++i) Vec16<T>::add(acc, u[i]);
      }
    }
    // four independent 16-byte loads in flight per thread
    for (; r + 3 * groups < valid; r += 4 * groups) {
      uint4 u0 = ld_stream(reinterpret_cast<const uint4*>(base + (long long)r * sL) + lane);
      uint4 u1 = ld_stream(reinterpret_cast<const uint4*>(base + (long long)(r + groups) * sL) + lane);
      uint4 u2 = ld_stream(reinterpret_cast<const uint4*>(base + (long long)(r + 2 * groups) * sL) + lane);
      uint4 u3 = ld_stream(reinterpret_cast<const uint4*>(base + (long long)(r + 3 * groups) * sL) + lane);
      Vec16<T>::add(acc, u0); Vec16<T>::add(acc, u1); Vec16<T>::add(acc, u2); Vec16<T>::add(acc, u3);
    }
    for (; r < valid; r += groups) {
      uint4 u = ld_stream(reinterpret_cast<const uint4*>(base + (long long)r * sL) + lane);
      Vec16<T>::add(acc, u);
    }
#pragma unroll
    for (int i = 0; i < N; ++i) part[grp * D + lane * N + i] = acc[i];
  }
  __syncthreads();
  const float inv = 1.0f / (float)block;
  for (int d = threadIdx.x; d < D; d += kPoolThreads) {
    float s = 0.f;
    for (int g = 0; g < groups; ++g) s += part[g * D + d];
    out_row[d] = s * inv;
  }
}

}  // namespace
