// Block-sparse / dense attention forward for bf16 on the sm_100a tensor cores, three-tile pipeline
// (Eq. 7: softmax over the keys of the retained blocks A_i, tiles outside A_i skipped).  Head
// dimension 128 or 64; selection blocks of 128, 256 or 512 tokens walked as tiles of 128 tokens, or of 64 /
// 32 tokens (template flag: the query blocks of a tile share the union of their lists, two / four listed key
// blocks are gathered into one tile, each row masks what its own query block does not keep).
//
// One CTA per (batch, head, 128-row query tile).  Tensor memory holds THREE score tiles and ONE
// output accumulator (S0 | S1 | S2 | O): tile t of the key-block list lives in score buffer t % 3
// and its softmax is done by warpgroup t % 2, so at any time two tiles are being exponentiated
// (two warps per scheduler keep the exponential pipe full) while the tensor pipe works on a third.
// P V products accumulate in list order into the one accumulator; nothing is merged at the end.
//
// Roles (384 threads; registers are moved from the third warpgroup to the softmax ones):
//   warps 0-3  softmax warpgroup 0 (tiles 0, 2, ...): thread r owns query row r (TMEM lane r)
//   warps 4-7  softmax warpgroup 1 (tiles 1, 3, ...)
//   warp  8    TMA producer (one lane)
//   warp  9    MMA issuer (whole warp converged, one elected lane issues)
//              "service u" = O += P_u V_u (P read from tensor memory, where the softmax wrote it as
//              bf16 over S) followed at once by S[u % 3] = Q K_{u+3}^T into the same columns (the
//              tensor pipe runs in order, so the overwrite of P_u needs no wait), then ONE commit
// Barriers:
//   STAGE[s]  {V_u, K_{u+3}} landed in slot s = u % 3 (transaction bytes)
//   SFULL[s]  phase 0 = prologue Q K_s^T complete; phase k >= 1 = service 3(k-1)+s complete.
//             "S of tile t is ready" = phase t/3 of SFULL[t%3]; "service u is complete" = phase
//             u/3 + 1 of SFULL[u%3]; the producer refills stage u after phase u/3 of SFULL[u%3]
//   PFULL[s]  the four warps that own the tile in buffer s have written P (one arrival per warp)
//
// Softmax reference.  One accumulator means one reference per query row, shared by the row's two
// threads (one per warpgroup) through a word in shared memory.  Scaling a row's P, O and
// denominator by a common power of two changes nothing in floating point, so the reference only
// has to keep the numbers away from overflow: it is the row maximum of the first tile and is raised
// only when a tile's exponentials leave the safe range.  The common tile therefore has no row
// maximum and no hand-over of references: exponentials against the thread's cached reference, one
// comparison on their sum, and, before P is released, a look at the shared word after the tile
// before (the other warpgroup's) has been released - the release of tile t-1 is the point at which
// its owner has decided whether it raised the reference.  If the word differs from the cached
// value, or the sum is out of range, or the row has no reference yet, the warp takes the slow
// path: adopt the published reference, take the tile's row maximum, raise the reference if needed
// (wait until every earlier P V has landed, scale O in place, publish), and redo the tile's P from
// the scores (lower half still in registers, upper half still in tensor memory).
//
// CTA pairs (template flag; opt-in).  Where two adjacent query tiles walk the same list (dense; selection
// blocks of 256 / 512 tokens), a cluster of two CTAs serves them: each CTA has the structure above in its
// own tensor memory, holds its own Q tile and HALF of every K tile (64 keys) and V tile (64 columns), and one
// thread of the first CTA issues tcgen05.mma.cta_group::2 with M = 256 for both, followed by one commit
// that arrives on both CTAs' SFULL barriers.  The second CTA's copies and P releases are counted on
// barriers of the first CTA (PEERQ, PEERSTAGE, PEERP).  It halves the L2 -> shared-memory bytes and is
// slower than single CTAs (P V of a tile has to wait for both CTAs' softmax), hence not the default.
//
// Every wait on an mbarrier is bounded (about a second); on expiry the CTA records
// SPARSTAR_ERR_TIMEOUT, all roles leave their loops, tensor memory is released and the kernel
// returns.
#include "attn_tc.cuh"

namespace {

enum {
  B3_Q = 0,                 // Q and the first (up to three) K tiles
  B3_STAGE = 1,             // 3
  B3_SFULL = B3_STAGE + 3,  // 3
  B3_PFULL = B3_SFULL + 3,  // 3
  // CTA pairs only, used in the first CTA: what the second CTA contributes is counted on barriers of its own
  B3_PEERP = B3_PFULL + 3,       // 3: the second CTA's warps have written their P
  B3_PEERQ = B3_PEERP + 3,       // the second CTA's Q and its halves of the first K tiles
  B3_PEERSTAGE = B3_PEERQ + 1,   // 3: the second CTA's halves of {V_u, K_{u+3}}
  B3_COUNT = B3_PEERSTAGE + 3
};
constexpr float kRaiseLog2 = 52.5f;   // a tile whose row maximum exceeds the reference by more than 2^52.5 raises it
                                      // (128 exponentials of at most 2^53 sum to at most kSumLimit = 2^60)

// Q, then kStages slots of K and of V; a CTA of a pair holds half of every K and V tile
constexpr uint32_t smem3_tiles(int hd, bool pair = false) {
  return (1u + (pair ? 1u : 2u) * kStages) * (128u * (uint32_t)hd * 2u);
}
constexpr uint32_t kOff3Misc = 8u * 24u;                         // after the barrier area (24 slots)
constexpr uint32_t kOff3Mref = kOff3Misc + 16u;                  // 128 floats: the rows' published references
constexpr uint32_t kOff3Trace = kOff3Mref + 128u * 4u;
constexpr uint32_t kTail3Bytes = kOff3Trace + 4u * kTraceSlots * 4u;
constexpr uint32_t smem3_bytes(int hd, bool pair = false) { return smem3_tiles(hd, pair) + kTail3Bytes; }
static_assert(B3_COUNT <= 24, "barrier area");
static_assert(smem3_bytes(128) <= 232448u, "shared memory per CTA");

template <int HD, bool kPair, bool kTrace, bool kGather>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc3_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const TcParams p) {
  static_assert(HD == 64 || HD == 128, "head dimension");
  static_assert(!kPair || HD == 128, "CTA pairs: head dimension 128");
  static_assert(!(kPair && kGather), "gathered blocks run on single CTAs");
  constexpr uint32_t kTileBytes = 128u * HD * 2u;
  constexpr uint32_t kKVBytes = kPair ? kTileBytes / 2u : kTileBytes;   // this CTA's share of a K or V tile
  constexpr uint32_t kOffK = kOffQ + kTileBytes;
  constexpr uint32_t kOffV = kOffK + kStages * kKVBytes;
  constexpr uint32_t kOffTail = kOffV + kStages * kKVBytes;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  unsigned char* tail = smem_raw + kOffTail;
  if ((base & 1023u) != 0u) {       // swizzled tiles need 1024-byte alignment (uniform exit)
    if (threadIdx.x == 0) record_status(p.status, SPARSTAR_ERR_CUDA, 902);
    return;
  }
  const uint32_t bar0 = base + kOffTail;
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail + kOff3Misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + kOff3Misc + 4);
  volatile float* mref = reinterpret_cast<volatile float*>(tail + kOff3Mref);
  volatile uint32_t* trace_smem = reinterpret_cast<volatile uint32_t*>(tail + kOff3Trace);

  const int h = blockIdx.y, b = blockIdx.z;
  // work item: a query tile, or (CTA pairs) two adjacent query tiles that walk the same list
  const uint32_t rank = kPair ? cluster_ctarank() : 0u;
  const int item = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int n_items = kPair ? (p.n_q + 1) / 2 : p.n_q;
  int wi = p.order != nullptr ? p.order[((size_t)b * p.H + h) * n_items + item] : item;
  if (wi < 0 || wi >= n_items) {    // a work order that is not this launch's (stale scratch): flag it, stay in bounds
    if (threadIdx.x == 0) record_status(p.status, SPARSTAR_ERR_BAD_INDEX, -1);
    wi = item;
  }
  // the second CTA of the last pair of an odd number of tiles gets a tile past the end: zero-filled Q, no output
  const int qi = kPair ? 2 * wi + (int)rank : wi;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const size_t row_id = ((size_t)b * p.H + h) * p.n_qb + (kPair ? 2 * wi : qi) / p.m;      // the query block's list
  // clock stamps cost registers in the softmax loop: they exist only in the instances launched with a trace buffer
  const bool tracing = kTrace && p.trace != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && lane == 0 &&
                       (warp == 0 || warp == 4 || warp >= 8);
  int trace_n = 0;
  const bool dense = p.kv_num_blocks == nullptr;
  const int* list = dense ? nullptr : p.kv_indices + row_id * (size_t)p.cap;
  const int cnt = dense ? 0 : max(min(p.kv_num_blocks[row_id], p.cap), 0);
  // tiles to walk: every listed block contributes m tiles, except that the last key block may hold fewer
  // kGather: selection blocks shorter than a tile.  The list then belongs to the query TILE (the union of its
  // query blocks' lists, entries (block << 4) | bits, bit s = kept by the tile's s-th query block) and
  // p.gather listed blocks are gathered into each 128-key tile; a row masks what its own block does not keep.
  const int gather = kGather ? p.gather : 1;
  const int sub_rows = kBlock / gather;           // tokens of a gathered block
  int n = dense ? p.n_k : (kGather ? (cnt + gather - 1) / gather : cnt * p.m);
  if (!kGather && !dense && p.m > 1 && cnt > 0 && list[cnt - 1] == p.n_kb - 1) n -= p.m * p.n_kb - p.n_k;
  const int q_row0 = qi * kBlock;

  if (threadIdx.x == 0) {
    mbar_init(bar(B3_Q), 1);
    for (int i = 0; i < 3; ++i) {
      mbar_init(bar(B3_STAGE + i), 1);
      mbar_init(bar(B3_SFULL + i), 1);
      mbar_init(bar(B3_PFULL + i), 4);
      if (kPair) {
        mbar_init(bar(B3_PEERP + i), 4);
        mbar_init(bar(B3_PEERSTAGE + i), 1);
      }
    }
    if (kPair) mbar_init(bar(B3_PEERQ), 1);
    // an expired wait already on record (this launch or an earlier one): do no work, so that a
    // failing launch ends after one timeout instead of one per wave of CTAs
    *abort_flag = *reinterpret_cast<volatile int*>(&p.status->status) == SPARSTAR_ERR_TIMEOUT ? 1 : 0;
    if (kTrace && p.trace != nullptr)
      for (int i = 0; i < 4 * kTraceSlots; ++i) trace_smem[i] = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (threadIdx.x < 128) mref[threadIdx.x] = -INFINITY;
  if (warp == 9) {
    if (kPair) tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
    else tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
  }
  tc_fence_before();
  __syncthreads();
  if (kPair) cluster_sync_all();     // both CTAs' barriers exist before either signals the other's
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tS[3] = {tmem + 0u, tmem + 128u, tmem + 256u};
  const uint32_t tO = tmem + 384u;
  const bool live = *abort_flag == 0;
  if (!live) n = 0;

  if (warp == 8) {
    // ================================ TMA producer ======================================
    reg_dec<kRegsOther>();
    if (kGather) {
      // Lane s < gather owns the tile's s-th listed block: it reads the entry and issues that block's copies, so a
      // tile's 4 * gather copies leave as four instructions; lane 0 also arms the barriers, copies Q and waits.
      if (n > 0) {
        const bool active = lane < gather;
        auto my_row = [&](int t) {                     // a missing entry repeats the tile's first
          int e = t * gather + lane;
          if (!active || e >= cnt) e = t * gather;
          return min(max(list[e] >> 4, 0), p.n_kb - 1) * sub_rows;
        };
        auto load_part = [&](const CUtensorMap* map, uint32_t dst, uint32_t barrier, int r) {
          const uint32_t d = dst + (uint32_t)(lane * sub_rows) * 128u;     // 128-byte rows inside a column half
          tma_load_4d(d, map, barrier, 0, r, h, b);
          if (HD == 128) tma_load_4d(d + kHalfBytes, map, barrier, 64, r, h, b);
        };
        int rt[3] = {0, 0, 0};
        const int n_pro = min(n, 3);
        for (int t = 0; t < n_pro; ++t) rt[t] = my_row(t);
        if (lane == 0) {
          mbar_expect_tx(bar(B3_Q), kTileBytes * (uint32_t)(1 + n_pro));
          tma_load_4d(base + kOffQ, &map_q, bar(B3_Q), 0, q_row0, h, b);
          if (HD == 128) tma_load_4d(base + kOffQ + kHalfBytes, &map_q, bar(B3_Q), 64, q_row0, h, b);
        }
        __syncwarp();
        if (active)
          for (int t = 0; t < n_pro; ++t) load_part(&map_k, base + kOffK + (uint32_t)t * kTileBytes, bar(B3_Q), rt[t]);
        bool ok = true;
        int st = 0;
        uint32_t ph = 0;
        for (int u = 0; u < n && ok; ++u) {
          const bool more = u + 3 < n;
          const int rk = more ? my_row(u + 3) : 0;
          int okk = 1;
          if (lane == 0) okk = mbar_wait(bar(B3_SFULL + st), ph, abort_flag, 100 + st) ? 1 : 0;
          ok = __shfl_sync(0xffffffffu, okk, 0) != 0;
          if (!ok) break;
          if (lane == 0) mbar_expect_tx(bar(B3_STAGE + st), more ? 2u * kTileBytes : kTileBytes);
          __syncwarp();
          if (active) {
            load_part(&map_v, base + kOffV + (uint32_t)st * kTileBytes, bar(B3_STAGE + st), rt[0]);
            if (more) load_part(&map_k, base + kOffK + (uint32_t)st * kTileBytes, bar(B3_STAGE + st), rk);
          }
          rt[0] = rt[1]; rt[1] = rt[2]; rt[2] = rk;
          if (++st == kStages) { st = 0; ph ^= 1u; }
        }
      }
    } else if (lane == 0 && n > 0) {
      int prev = -1;
      auto checked = [&](int j, bool first_of_block) {
        if (j < 0 || j >= p.n_kb || (first_of_block && j <= prev)) {   // malformed: flag it, stay in bounds
          record_status(p.status, SPARSTAR_ERR_BAD_INDEX, (int)row_id);
          j = min(max(j, 0), p.n_kb - 1);
        }
        prev = j;
        return j;
      };
      // first token row of key tile t
      auto block_at = [&](int t) {
        if (dense) return t * kBlock;
        const int sub = p.m == 1 ? 0 : t % p.m;
        const int j = checked(list[p.m == 1 ? t : t / p.m], sub == 0);
        return min(j * p.m + sub, p.n_k - 1) * kBlock;
      };
      // A CTA of a pair copies its own query tile, keys [64 rank, 64 rank + 64) of every K tile and columns
      // [64 rank, 64 rank + 64) of every V tile.  The first CTA's bytes are counted on its barriers Q / STAGE, the
      // second CTA's on the first CTA's barriers PEERQ / PEERSTAGE; the first CTA's producer arms both (the two
      // CTAs copy the same amounts).
      auto peer_of = [&](int i) { return i == B3_Q ? (int)B3_PEERQ : (int)B3_PEERSTAGE + (i - (int)B3_STAGE); };
      auto barrier_of = [&](int i) { return kPair && rank == 1u ? cluster_map(bar(peer_of(i)), 0u) : bar(i); };
      auto arm = [&](int i, uint32_t bytes) {          // `bytes`: what ONE CTA copies
        if (rank == 0u) {
          mbar_expect_tx(bar(i), bytes);
          if (kPair) mbar_expect_tx(bar(peer_of(i)), bytes);
        }
      };
      auto load_q = [&](int bi) {
        const uint32_t dst = base + kOffQ, bb = barrier_of(bi);
        if (kPair && rank == 1u) {
          tma_load_4d_pair(dst, &map_q, bb, 0, q_row0, h, b);
          tma_load_4d_pair(dst + kHalfBytes, &map_q, bb, 64, q_row0, h, b);
        } else {
          tma_load_4d(dst, &map_q, bb, 0, q_row0, h, b);
          if (HD == 128) tma_load_4d(dst + kHalfBytes, &map_q, bb, 64, q_row0, h, b);
        }
      };
      auto load_k = [&](int slot, int bi, int row) {
        const uint32_t dst = base + kOffK + (uint32_t)slot * kKVBytes, bb = barrier_of(bi);
        if (kPair && rank == 1u) {                         // 64 keys x D as two boxes of 64 x 64 (map with 64-row boxes)
          tma_load_4d_pair(dst, &map_k, bb, 0, row + 64, h, b);
          tma_load_4d_pair(dst + kKVBytes / 2u, &map_k, bb, 64, row + 64, h, b);
        } else if (kPair) {
          tma_load_4d(dst, &map_k, bb, 0, row, h, b);
          tma_load_4d(dst + kKVBytes / 2u, &map_k, bb, 64, row, h, b);
        } else {
          tma_load_4d(dst, &map_k, bb, 0, row, h, b);
          if (HD == 128) tma_load_4d(dst + kHalfBytes, &map_k, bb, 64, row, h, b);
        }
      };
      auto load_v = [&](int slot, int bi, int row) {
        const uint32_t dst = base + kOffV + (uint32_t)slot * kKVBytes, bb = barrier_of(bi);
        if (kPair && rank == 1u) {                         // 128 keys x 64 columns: one box
          tma_load_4d_pair(dst, &map_v, bb, 64, row, h, b);
        } else if (kPair) {
          tma_load_4d(dst, &map_v, bb, 0, row, h, b);
        } else {
          tma_load_4d(dst, &map_v, bb, 0, row, h, b);
          if (HD == 128) tma_load_4d(dst + kHalfBytes, &map_v, bb, 64, row, h, b);
        }
      };
      // Q with the first three score tiles' keys
      int jt[3] = {0, 0, 0};
      const int n_pro = min(n, 3);
      for (int t = 0; t < n_pro; ++t) jt[t] = block_at(t);
      arm(B3_Q, kTileBytes + kKVBytes * (uint32_t)n_pro);
      load_q(B3_Q);
      for (int t = 0; t < n_pro; ++t) load_k(t, B3_Q, jt[t]);
      // stage u = {V_u, K_{u+3}} into slot u % 3, free once phase u/3 of SFULL[u%3] has completed
      bool ok = true;
      int st = 0;
      uint32_t ph = 0;
      for (int u = 0; u < n && ok; ++u) {
        const bool more = u + 3 < n;
        const int jk = more ? block_at(u + 3) : 0;
        ok = mbar_wait(bar(B3_SFULL + st), ph, abort_flag, 100 + st);
        if (!ok) break;
        TRACE(3, 10, u);
        if (u == p.debug_drop_stage) {
          arm(B3_STAGE + st, kKVBytes);                                 // bytes that never arrive
        } else {
          arm(B3_STAGE + st, more ? 2u * kKVBytes : kKVBytes);
          load_v(st, B3_STAGE + st, jt[0]);
          if (more) load_k(st, B3_STAGE + st, jk);
        }
        jt[0] = jt[1]; jt[1] = jt[2]; jt[2] = jk;
        if (++st == kStages) { st = 0; ph ^= 1u; }
      }
    }
  } else if (warp == 9) {
    // ================================ MMA issuer ========================================
    reg_dec<kRegsOther>();
    // All 32 lanes run this loop converged (every value in it is warp-uniform); the MMA and commit
    // wrappers elect the one lane that issues.  Waits are made warp-uniform with a vote so that no
    // lane can leave the loop alone.
    auto wait_all = [&](uint32_t bb, uint32_t parity, int site) {
      return __all_sync(0xffffffffu, mbar_wait(bb, parity, abort_flag, site));
    };
    // CTA pairs: the first CTA's warp issues for both (M = 256: each CTA's tensor core takes its own 128 query
    // rows, from its own Q and P, against the key tile whose halves lie in the two CTAs' shared memories)
    if (n > 0 && (!kPair || rank == 0u)) {
      constexpr uint32_t kM = kPair ? 256u : 128u;
      constexpr uint32_t idesc_qk = instr_desc(false, 128u, kM);         // S: queries x 128 keys
      constexpr uint32_t idesc_pv = instr_desc(true, (uint32_t)HD, kM);  // O: queries x HD
      const uint64_t qdesc0 = smem_desc(base + kOffQ, 16, 1024);
      const uint64_t kdesc0 = smem_desc(base + kOffK, 16, 1024);
      const uint64_t vdesc0 = smem_desc(base + kOffV, kHalfBytes, 1024);
      auto commit = [&](int i) {
        if (kPair) umma_commit_pair(bar(i), (uint16_t)3);
        else umma_commit(bar(i));
      };
      auto issue_qk = [&](int slot) {                       // S[slot] = Q K^T with the K tile in `slot`
        const uint64_t kd = kdesc0 + (uint64_t)((uint32_t)slot * (kKVBytes >> 4));
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
          // 16 contraction elements = 32 bytes inside the swizzle atom; the second 64 columns lie behind the
          // first (Q: 16 KB on; K: half of this CTA's share of the tile on)
          const uint64_t off_q = (uint64_t)((((uint32_t)kk >> 2) * kHalfBytes + ((uint32_t)kk & 3u) * 32u) >> 4);
          const uint64_t off_k = (uint64_t)((((uint32_t)kk >> 2) * (kKVBytes / 2u) + ((uint32_t)kk & 3u) * 32u) >> 4);
          if (kPair) umma_ss_pair(tS[slot], qdesc0 + off_q, kd + off_k, idesc_qk, kk > 0 ? 1u : 0u);
          else umma_ss(tS[slot], qdesc0 + off_q, kd + off_k, idesc_qk, kk > 0 ? 1u : 0u);
        }
      };
      // P of the tile in buffer s written: by this CTA's four warps and, in a pair, by the other CTA's
      auto wait_p = [&](int sidx, uint32_t parity) {
        bool got = wait_all(bar(B3_PFULL + sidx), parity, 220 + sidx);
        if (kPair && got)
          got = __all_sync(0xffffffffu, mbar_wait_cluster(bar(B3_PEERP + sidx), parity, abort_flag, 230 + sidx));
        return got;
      };
      // the tiles of stage barrier i landed: this CTA's share and, in a pair, the other CTA's
      auto wait_tiles = [&](int i, int peer_i, uint32_t parity, int site) {
        bool got = wait_all(bar(i), parity, site);
        if (kPair && got) got = wait_all(bar(peer_i), parity, site + 40);
        return got;
      };
      bool ok = wait_tiles(B3_Q, B3_PEERQ, 0u, 200);
      if (ok) {
        tc_fence_after();
        TRACE(0, 20, 0);
        for (int t = 0; t < 3 && t < n; ++t) {
          issue_qk(t);
          commit(B3_SFULL + t);
        }
        TRACE(0, 21, 0);
        ok = wait_tiles(B3_STAGE + 0, B3_PEERSTAGE + 0, 0u, 210);
        if (ok) ok = wait_p(0, 0u);
        tc_fence_after();
      }
      int st = 0;
      uint32_t ph = 0;                                       // parity of the current lap over the three buffers
      for (int u = 0; u < n && ok; ++u) {
        const uint64_t vd = vdesc0 + (uint64_t)((uint32_t)st * (kKVBytes >> 4));
        TRACE(0, 22, u);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {                      // 16 keys = 16 rows of 128 B; P advances 8 columns
          const uint32_t pa = tS[st] + (uint32_t)kk * 8u;
          const uint64_t vk = vd + (uint64_t)((uint32_t)kk * (2048u >> 4));
          if (kPair) umma_ts_pair(tO, pa, vk, idesc_pv, (kk > 0 || u > 0) ? 1u : 0u);
          else umma_ts(tO, pa, vk, idesc_pv, (kk > 0 || u > 0) ? 1u : 0u);
        }
        if (u + 3 < n) issue_qk(st);
        commit(B3_SFULL + st);
        TRACE(0, 24, u);
        if (++st == kStages) { st = 0; ph ^= 1u; }
        if (u + 1 < n) {                                      // operands of the next service, while this one runs
          ok = wait_p(st, ph);
          if (ok) ok = wait_tiles(B3_STAGE + st, B3_PEERSTAGE + st, ph, 210 + st);
          tc_fence_after();
          TRACE(0, 25, u);
        }
      }
    }
  } else if (warp >= 10) {
    reg_dec<kRegsOther>();                                  // idle warps of the third warpgroup
  } else {
    // ================================ softmax warpgroups ================================
    reg_inc<kRegsSoftmax>();
    const int w = warp >> 2;                        // owner of tiles w, w + 2, ...
    const int row = (warp & 3) * 32 + lane;         // query row = TMEM lane
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const float c = p.scale * 1.4426950408889634f;  // logits in log2 units
    // valid key columns of the last tile: lists ascend, so only the final entry can be the partial last key block
    int last_valid = kBlock;
    if (!kGather && n > 0 && (dense || list[cnt - 1] == p.n_kb - 1)) last_valid = p.L_k - (p.n_k - 1) * kBlock;
    const int row_group = row / sub_rows;           // gathered blocks: which of the tile's query blocks owns this row
    const int tail_sub = p.L_k - (p.n_kb - 1) * sub_rows;     // keys of the last (possibly partial) gathered block
    float my_ref = -INFINITY;                       // the reference my P and partial denominator are expressed in
    float l = 0.f;
    bool ok = true;
    int sb = w;                                     // t % 3
    uint32_t sph = 0;                               // (t / 3) & 1
    for (int t = w; t < n && ok; t += 2) {
      // gathered blocks: this tile's union entries, fetched before the wait so that the loads are not on the
      // critical path (0 = no entry)
      int ent[4] = {0, 0, 0, 0};
      if (kGather) {
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          const int e = t * gather + g;
          if (g < gather && e < cnt) ent[g] = list[e];
        }
      }
      ok = __all_sync(0xffffffffu, mbar_wait(bar(B3_SFULL + sb), sph, abort_flag, 300 + w));
      if (!ok) break;
      tc_fence_after();
      TRACE(1 + w, 30, t);
      // Valid columns of the tile's four 32-column segments for this row.  Gathered blocks: an entry counts only
      // if this row's query block keeps it (rows of one warp share a query block, so all of this is warp-uniform).
      int c0 = 32, c1 = 32, c2 = 32, c3 = 32;
      if (kGather) {
        int vc[4];
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          vc[g] = 0;
          if ((ent[g] >> row_group) & 1) vc[g] = (ent[g] >> 4) == p.n_kb - 1 ? tail_sub : sub_rows;
        }
        if (gather == 4) {
          c0 = vc[0]; c1 = vc[1]; c2 = vc[2]; c3 = vc[3];
        } else {
          c0 = min(vc[0], 32); c1 = max(vc[0] - 32, 0); c2 = min(vc[1], 32); c3 = max(vc[1] - 32, 0);
        }
        if ((c0 | c1 | c2 | c3) == 0) {
          // nothing of this tile is kept by the row's query block: P = 0, no exponentials, the reference and the
          // denominator stay as they are (a later tile adopts whatever has been published meanwhile)
          uint32_t zero[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) zero[i] = 0u;
          tmem_st32(tS[sb] + lane_off, zero);
          tmem_st32(tS[sb] + lane_off + 32u, zero);
          tmem_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(B3_PFULL + sb));
          sb += 2;
          if (sb >= 3) { sb -= 3; sph ^= 1u; }
          continue;
        }
      } else if (t == n - 1 && last_valid < kBlock) {
        c0 = min(max(last_valid, 0), 32); c1 = min(max(last_valid - 32, 0), 32);
        c2 = min(max(last_valid - 64, 0), 32); c3 = min(max(last_valid - 96, 0), 32);
      }
      uint32_t sr[128];
      tmem_ld32(tS[sb] + lane_off + 0u, sr + 0);
      tmem_ld32(tS[sb] + lane_off + 32u, sr + 32);
      tmem_ld32(tS[sb] + lane_off + 64u, sr + 64);
      tmem_ld32(tS[sb] + lane_off + 96u, sr + 96);
      tmem_wait_ld();
      if ((c0 & c1 & c2 & c3) != 32) {                        // some segment is not full: -inf there
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          if (i >= c0) sr[i] = 0xff800000u;
          if (i >= c1) sr[32 + i] = 0xff800000u;
          if (i >= c2) sr[64 + i] = 0xff800000u;
          if (i >= c3) sr[96 + i] = 0xff800000u;
        }
      }
      TRACE(1 + w, 31, t);
      // exponentials of one half of the tile (64 keys) against my_ref, packed and stored as P over
      // the first 64 columns of the score buffer (a row that has no reference yet gives zeros)
      auto exp_half = [&](int cc) {
        const float nmc = my_ref > -INFINITY ? -(my_ref * c) : 0.f;
        float sum[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t pk[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          float a0, a1;
          fma2(a0, a1, __uint_as_float(sr[cc * 64 + 2 * i]), __uint_as_float(sr[cc * 64 + 2 * i + 1]), c, nmc);
          const float p0 = ex2(a0), p1 = ex2(a1);
          sum[i & 3] += p0 + p1;
          pk[i] = pack_bf16(p0, p1);
        }
        tmem_st32(tS[sb] + lane_off + 32u * cc, pk);
        return (sum[0] + sum[1]) + (sum[2] + sum[3]);
      };
      float tile_sum = 0.f;
      const bool fresh = __any_sync(0xffffffffu, my_ref == -INFINITY);
      if (!fresh) tile_sum = exp_half(0) + exp_half(1);
      // The tile before this one (the other warpgroup's) has been released, hence decided: its
      // owner published any raise of the reference before it arrived.
      float cur = my_ref;
      if (t > 0) {
        const int pb = sb == 0 ? 2 : sb - 1;
        ok = __all_sync(0xffffffffu, mbar_wait(bar(B3_PFULL + pb), sb == 0 ? sph ^ 1u : sph, abort_flag, 330 + w));
        if (!ok) break;
        cur = mref[row];
      }
      const bool slow = fresh || cur != my_ref || !(tile_sum < kSumLimit);     // the last also catches inf and NaN
      if (__any_sync(0xffffffffu, slow)) {
        if (cur != my_ref) {                         // adopt the published reference
          l *= my_ref > -INFINITY ? ex2((my_ref - cur) * c) : 0.f;
          my_ref = cur;
        }
        // the tile's scores again: lower 64 still in registers, upper 64 from tensor memory (P never covers them)
        tmem_ld32(tS[sb] + lane_off + 64u, sr + 64);
        tmem_ld32(tS[sb] + lane_off + 96u, sr + 96);
        tmem_wait_ld();
        if ((c2 & c3) != 32) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            if (i >= c2) sr[64 + i] = 0xff800000u;
            if (i >= c3) sr[96 + i] = 0xff800000u;
          }
        }
        float mxa[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) mxa[e] = fmaxf(__uint_as_float(sr[e]), __uint_as_float(sr[8 + e]));
#pragma unroll
        for (int i = 16; i < 128; i += 16)
#pragma unroll
          for (int e = 0; e < 8; ++e) mxa[e] = max3(mxa[e], __uint_as_float(sr[i + e]), __uint_as_float(sr[i + 8 + e]));
        const float mx = fmaxf(max3(mxa[0], mxa[1], mxa[2]), max3(mxa[3], mxa[4], max3(mxa[5], mxa[6], mxa[7])));
        float ref_new = my_ref;
        if (my_ref == -INFINITY || (mx - my_ref) * c > kRaiseLog2) ref_new = fmaxf(my_ref, mx);
        const bool changed = ref_new != my_ref;      // false when both are -inf (no valid key seen yet)
        if (t > 0 && __any_sync(0xffffffffu, changed)) {
          // every earlier P V must have landed in O: that is the completion of service t - 1
          const int pb = sb == 0 ? 2 : sb - 1;
          ok = __all_sync(0xffffffffu, mbar_wait(bar(B3_SFULL + pb), (sb == 0 ? sph ^ 1u : sph) ^ 1u, abort_flag, 310 + w));
          if (!ok) break;
          tc_fence_after();
          const float alpha = changed ? (my_ref > -INFINITY ? ex2((my_ref - ref_new) * c) : 0.f) : 1.f;
          tmem_wait_st();
#pragma unroll 1
          for (int cc = 0; cc < HD / 32; ++cc) {
            uint32_t orr[32];
            tmem_ld32(tO + lane_off + 32u * cc, orr);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * alpha);
            tmem_st32(tO + lane_off + 32u * cc, orr);
          }
          l *= alpha;
        }
        if (changed) mref[row] = ref_new;
        my_ref = ref_new;
        tile_sum = exp_half(0) + exp_half(1);
      }
      TRACE(1 + w, 32, t);
      l += tile_sum;
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar(B3_PFULL + sb));
        if (kPair && rank == 1u) mbar_arrive_cluster(cluster_map(bar(B3_PEERP + sb), 0u));
      }
      TRACE(1 + w, 33, t);
      sb += 2;
      if (sb >= 3) { sb -= 3; sph ^= 1u; }
    }
    // ---- normalise and write O --------------------------------------------------------------
    if (ok && n > 0) {                              // the completion of the last service
      // = phase (n-1)/3 + 1 of the last tile's barrier.  A parity wait is only right for a thread that is at most
      // one phase behind: the warpgroup that owns the last tile has consumed phase (n-1)/3 ("its scores are
      // ready"), the other one has not and must pass it first - otherwise, arriving while that phase is still
      // open, it would take the phase before it (same parity as the one it wants) for the end of the kernel.
      const int lb = (n - 1) % 3;
      const uint32_t kph = (uint32_t)((n - 1) / 3);
      if (((n - 1) & 1) != w)
        ok = __all_sync(0xffffffffu, mbar_wait(bar(B3_SFULL + lb), kph & 1u, abort_flag, 325 + w));
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(B3_SFULL + lb), (kph + 1u) & 1u, abort_flag, 320 + w));
      tc_fence_after();
    }
    // The V ring is dead now (every service is complete) and serves as scratch: the row's two partial results
    // meet there, and the output is staged there so that it leaves in whole 128-byte row pieces instead of 32
    // scattered 16-byte pieces per store instruction.
    unsigned char* vring = smem_raw + kOffV;
    volatile float* stats = reinterpret_cast<volatile float*>(vring + 32768);   // (reference, partial denominator)
    stats[2 * (w * 128 + row)] = my_ref;
    stats[2 * (w * 128 + row) + 1] = l;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    const int q_row = q_row0 + row;
    constexpr int kCols = HD / 2;                   // this warpgroup's half of D
    constexpr int kChunks = kCols / 32;
    if (*abort_flag == 0 && n > 0) {
      // references only rise, so the row's final reference is the larger of the two cached ones
      const float oref = stats[2 * ((w ^ 1) * 128 + row)], ol = stats[2 * ((w ^ 1) * 128 + row) + 1];
      const float ref = fmaxf(my_ref, oref);
      const float lt = (my_ref > -INFINITY ? l * ex2((my_ref - ref) * c) : 0.f) +
                       (oref > -INFINITY ? ol * ex2((oref - ref) * c) : 0.f);
      const float inv = lt > 0.f ? 1.0f / lt : 0.f;
      const uint32_t col0 = (uint32_t)w * (uint32_t)kCols;
      uint32_t oa[kChunks][32];
#pragma unroll
      for (int cc = 0; cc < kChunks; ++cc) tmem_ld32(tO + lane_off + col0 + 32u * cc, oa[cc]);
      tmem_wait_ld();
      // this warp's 32 rows x kCols columns, staged with the 16-byte pieces of a row rotated by the row number
      // (no bank conflicts either way), then stored row-contiguously
      constexpr int kRowBytes = kCols * 2;
      constexpr int kPieces = kRowBytes / 16;       // 8 (D = 128) or 4 (D = 64)
      unsigned char* stage = vring + warp * (32 * kRowBytes);
#pragma unroll
      for (int pc = 0; pc < kPieces; ++pc) {
        const uint32_t* src = &oa[pc / 4][8 * (pc % 4)];
        uint4 val;
        val.x = pack_bf16(__uint_as_float(src[0]) * inv, __uint_as_float(src[1]) * inv);
        val.y = pack_bf16(__uint_as_float(src[2]) * inv, __uint_as_float(src[3]) * inv);
        val.z = pack_bf16(__uint_as_float(src[4]) * inv, __uint_as_float(src[5]) * inv);
        val.w = pack_bf16(__uint_as_float(src[6]) * inv, __uint_as_float(src[7]) * inv);
        *reinterpret_cast<uint4*>(stage + lane * kRowBytes + ((pc ^ (lane & (kPieces - 1))) * 16)) = val;
      }
      __syncwarp();
      __nv_bfloat16* ob = reinterpret_cast<__nv_bfloat16*>(p.o) + b * p.osB + h * p.osH + col0;
      const int warp_row0 = q_row0 + (warp & 3) * 32;
#pragma unroll
      for (int i = 0; i < kPieces; ++i) {
        const int r = i * (32 / kPieces) + lane / kPieces, pc = lane % kPieces;
        const uint4 val = *reinterpret_cast<const uint4*>(stage + r * kRowBytes + ((pc ^ (r & (kPieces - 1))) * 16));
        if (warp_row0 + r < p.L_q) *reinterpret_cast<uint4*>(ob + (long long)(warp_row0 + r) * p.osL + pc * 8) = val;
      }
      if (q_row < p.L_q && p.lse != nullptr && w == 0)
        p.lse[((size_t)b * p.H + h) * p.L_q + q_row] = lt > 0.f ? ref * p.scale + logf(lt) : -INFINITY;
    } else if (n == 0 && live) {
      if (q_row < p.L_q) {
        __nv_bfloat16* og = reinterpret_cast<__nv_bfloat16*>(p.o) + b * p.osB + h * p.osH +
                            (long long)q_row * p.osL + w * kCols;
        uint4* dst = reinterpret_cast<uint4*>(og);
#pragma unroll
        for (int i = 0; i < HD / 16; ++i) dst[i] = make_uint4(0u, 0u, 0u, 0u);
        if (p.lse != nullptr && w == 0) p.lse[((size_t)b * p.H + h) * p.L_q + q_row] = -INFINITY;
      }
    }
  }

  // ---- teardown -----------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (kPair) cluster_sync_all();     // neither CTA's shared or tensor memory goes away while the other may still signal it
  tc_fence_after();
  if (warp == 9) {
    if (kPair) tmem_dealloc_pair(tmem, 512);
    else tmem_dealloc(tmem, 512);
  }
  if (kTrace && p.trace != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0)
    for (int i = threadIdx.x; i < 4 * kTraceSlots; i += kThreads) {
      const int role = i / kTraceSlots, k = i % kTraceSlots;
      if (k < p.trace_cap) {
        p.trace[(role * p.trace_cap + k) * 2] = trace_smem[i] >> 26;
        p.trace[(role * p.trace_cap + k) * 2 + 1] = trace_smem[i] & 0x3FFFFFFu;
      }
    }
  if (threadIdx.x == 0 && *abort_flag != 0) record_status(p.status, SPARSTAR_ERR_TIMEOUT, *abort_flag);
}

template <int HD, bool kPair, bool kTrace, bool kGather>
int launch3(sparstar_ctx* ctx, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const TcParams& p,
            dim3 grid, cudaStream_t s) {
  static bool attr_set[64] = {};
  if (!attr_set[ctx->device & 63]) {
    // the in-kernel register re-balancing needs the compiled allocation to be what it assumes
    cudaFuncAttributes fa;
    SPARSTAR_CUDA_TRY(cudaFuncGetAttributes(&fa, attn_tc3_kernel<HD, kPair, kTrace, kGather>));
    if (2 * 128 * kRegsSoftmax + 128 * kRegsOther > kThreads * fa.numRegs) return SPARSTAR_ERR_UNSUPPORTED;
    SPARSTAR_CUDA_TRY(cudaFuncSetAttribute(attn_tc3_kernel<HD, kPair, kTrace, kGather>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)smem3_bytes(HD, kPair)));
    attr_set[ctx->device & 63] = true;
  }
  if (kPair) {
    // two adjacent query tiles per work item, one CTA each, launched as a cluster of two
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2u * ((grid.x + 1u) / 2u), grid.y, grid.z);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem3_bytes(HD, true);
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    SPARSTAR_CUDA_TRY(cudaLaunchKernelEx(&cfg, attn_tc3_kernel<HD, kPair, kTrace, kGather>, mq, mk, mv, p));
  } else {
    attn_tc3_kernel<HD, kPair, kTrace, kGather><<<grid, kThreads, smem3_bytes(HD), s>>>(mq, mk, mv, p);
  }
  return SPARSTAR_OK;
}

}  // namespace

// `pair`: two adjacent query tiles per work item on a pair of CTAs (head dimension 128; the tiles of a pair must
// walk the same list: dense, or selection blocks of an even number of tiles); `mk` then has 64-row boxes and
// `p.order`, if given, orders the pairs.  `gathered`: selection blocks of 64 / 32 tokens (p.gather = 2 / 4, union
// lists per query tile, K/V maps with boxes of that many rows).  `grid.x` is the number of query tiles either way.
int launch_attn_tc3(sparstar_ctx* ctx, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                    const TcParams& p, int head_dim, dim3 grid, cudaStream_t s, bool pair, bool gathered) {
  const bool tr = p.trace != nullptr;
  if (pair) {
    if (head_dim != 128 || gathered) return SPARSTAR_ERR_UNSUPPORTED;
    return tr ? launch3<128, true, true, false>(ctx, mq, mk, mv, p, grid, s)
              : launch3<128, true, false, false>(ctx, mq, mk, mv, p, grid, s);
  }
  if (gathered) {
    if (head_dim == 64) return launch3<64, false, false, true>(ctx, mq, mk, mv, p, grid, s);
    return launch3<128, false, false, true>(ctx, mq, mk, mv, p, grid, s);
  }
  if (head_dim == 64)
    return tr ? launch3<64, false, true, false>(ctx, mq, mk, mv, p, grid, s)
              : launch3<64, false, false, false>(ctx, mq, mk, mv, p, grid, s);
  return tr ? launch3<128, false, true, false>(ctx, mq, mk, mv, p, grid, s)
            : launch3<128, false, false, false>(ctx, mq, mk, mv, p, grid, s);
}
