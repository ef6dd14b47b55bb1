// The older two-stream form of the attention kernel, kept as a cross-check of the three-tile kernel
// (attn_tc3.cu) and as the block-mass kernel, and the launcher of both.
// Block-sparse / dense attention forward for bf16 on the sm_100a tensor cores (Eq. 7: softmax
// over the keys of the retained blocks A_i, tiles outside A_i skipped).  Head dimension 128 or
// 64; selection blocks of 128, 256 or 512 tokens, always walked as tiles of 128 tokens, or of 64 /
// 32 tokens (the query blocks of a tile share the union of their lists, two / four listed key
// blocks are gathered into one tile, each row masks what its own query block does not keep).
//
// One CTA per (batch, head, 128-row query tile).  The key-block list of the query block is walked by
// two interleaved streams (even / odd list positions); each stream has its own score tile S
// and output accumulator O in tensor memory and its own softmax warpgroup with a private
// softmax reference and denominator, so while one warpgroup exponentiates tile t the tensor pipe
// runs the GEMMs of tile t+1.  The two partial results are merged once at the end (the usual
// log-sum-exp combination of two disjoint key sets).
//
// Roles (384 threads; registers are moved from the third warpgroup to the softmax ones):
//   warps 0-3  softmax warpgroup of stream 0: thread r owns query row r (TMEM lane r)
//   warps 4-7  softmax warpgroup of stream 1
//   warp  8    TMA producer
//   warp  9    MMA issuer (whole warp converged, one elected lane issues): "service u" = O += P_u V_u (P read from tensor memory, where the
//              softmax warpgroup wrote it as bf16 over S) followed at once by S = Q K_{u+2}^T
//              into the same columns; the tensor pipe runs its instructions in order, so the
//              overwrite of P_u needs no wait
// The issuing thread's own latency shows up as idle tensor-pipe time (the pipe runs little
// ahead of issue), so a service has the fewest possible synchronisations: one wait for its
// operands, one wait for P, one commit.
//   stage u (ring of 3) = {V_u, K_{u+2}}: one mbarrier, loaded once service u-3 is complete
//   S-full of tile t    = completion of the commit that ends service t-2: read by the softmax
//                         warpgroup (S_t is ready) and by the producer (stage t-2 is free).
//                         Four barriers, tile t on barrier t % 4: the producer may trail the
//                         issuing thread by a whole service, and with one barrier per stream the
//                         phase it waits for could then be two completions old, which a parity
//                         wait cannot tell from "not yet"; with four, the barrier it waits on
//                         cannot complete again before the stage it is about to load is used
// Shared memory (D = 128): Q 32 KB + 3 x K 32 KB + 3 x V 32 KB, all 128-byte-swizzled 64-column
// halves.  Tensor memory (512 columns): S0 | S1 (128 fp32 columns each) | O0 | O1 (D columns each).
//
// Every wait on an mbarrier is bounded (about a second); on expiry the CTA records
// SPARSTAR_ERR_TIMEOUT, all roles leave their loops, tensor memory is released and the kernel
// returns.
#include "attn_tc.cuh"

namespace {

template <int kMode, int HD>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, const TcParams p) {
  // geometry for head dimension HD (64 or 128): a tile is 128 rows x HD bf16 = HD/64 swizzled halves
  static_assert(HD == 64 || HD == 128, "head dimension");
  constexpr uint32_t kTileBytes = 128u * HD * 2u;
  constexpr uint32_t kOffK = kOffQ + kTileBytes;
  constexpr uint32_t kOffV = kOffK + kStages * kTileBytes;
  constexpr uint32_t kOffBar = kOffV + kStages * kTileBytes;
  constexpr uint32_t kOffMisc = kOffBar + 8 * BAR_COUNT;
  constexpr uint32_t kOffStats = kOffMisc + 16;
  constexpr uint32_t kOffTrace = kOffStats + 2 * 128 * 8;
  // kMode 0: attention.  1 = analysis mode: no P V; per tile the mean over the block's queries of
  // sum_u exp(s - lse) is written.  2 = attention with selection blocks shorter than a tile
  // (p.gather of them per key tile); a separate instance keeps that bookkeeping out of mode 0.
  constexpr bool kMass = kMode == 1;
  const int gather = kMode == 2 ? p.gather : 1;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  unsigned char* base_ptr = smem_raw;
  if ((base & 1023u) != 0u) {       // swizzled tiles need 1024-byte alignment (uniform exit)
    if (threadIdx.x == 0) record_status(p.status, SPARSTAR_ERR_CUDA, 900);
    return;
  }
  const uint32_t bar0 = base + kOffBar;
  auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + kOffMisc + 4);
  float2* stats = reinterpret_cast<float2*>(base_ptr + kOffStats);
  volatile uint32_t* trace_smem = reinterpret_cast<volatile uint32_t*>(base_ptr + kOffTrace);

  const int h = blockIdx.y, b = blockIdx.z;
  int qi = p.order != nullptr ? p.order[((size_t)b * p.H + h) * p.n_q + blockIdx.x] : (int)blockIdx.x;
  if (qi < 0 || qi >= p.n_q) {      // a work order that is not this launch's (stale scratch): flag it, stay in bounds
    if (threadIdx.x == 0) record_status(p.status, SPARSTAR_ERR_BAD_INDEX, -1);
    qi = (int)blockIdx.x;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const size_t row_id = ((size_t)b * p.H + h) * p.n_qb + qi / p.m;      // the query block's list
  const bool tracing = p.trace != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && lane == 0 &&
                       (warp == 0 || warp == 4 || warp >= 8);
  int trace_n = 0;
  const bool dense = p.kv_num_blocks == nullptr;
  const int* list = dense ? nullptr : p.kv_indices + row_id * (size_t)p.cap;
  const int cnt = dense ? 0 : max(min(p.kv_num_blocks[row_id], p.cap), 0);
  // tiles to walk: every listed block contributes m tiles, except that the last key block may
  // hold fewer
  int n = dense ? p.n_k : (gather > 1 ? (cnt + gather - 1) / gather : cnt * p.m);
  if (!dense && p.m > 1 && cnt > 0 && list[cnt - 1] == p.n_kb - 1) n -= p.m * p.n_kb - p.n_k;
  const int sub_rows = kBlock / gather;           // tokens of a gathered block
  const int q_row0 = qi * kBlock;

  if (threadIdx.x == 0) {
    mbar_init(bar(BAR_Q), 1);
    for (int st = 0; st < kStages; ++st) mbar_init(bar(BAR_STAGE + st), 1);
    for (int x = 0; x < 4; ++x) mbar_init(bar(BAR_SFULL + x), 1);
    for (int x = 0; x < 2; ++x) {
      mbar_init(bar(BAR_PFULL + x), 128);
      mbar_init(bar(BAR_OFULL + x), 1);
    }
    // an expired wait already on record (this launch or an earlier one): do no work, so that a
    // failing launch ends after one timeout instead of one per wave of CTAs
    *abort_flag = *reinterpret_cast<volatile int*>(&p.status->status) == SPARSTAR_ERR_TIMEOUT ? 1 : 0;
    if (p.trace != nullptr)
      for (int i = 0; i < 4 * kTraceSlots; ++i) trace_smem[i] = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 9) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tS[2] = {tmem + 0u, tmem + 128u};
  const uint32_t tO[2] = {tmem + 256u, tmem + 256u + (uint32_t)HD};
  const bool live = *abort_flag == 0;
  if (!live) n = 0;

  if (warp == 8) {
    // ================================ TMA producer ======================================
    reg_dec<kRegsOther>();
    if (kMode == 2) {
      // Gathered blocks: lane s < gather owns the tile's s-th listed block, reads its entry and
      // issues its copies, so a tile's 4 * gather copies go out as four instructions; lane 0
      // also arms the barriers, copies Q and does the waiting.
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
        const int r0 = my_row(0), r1 = n > 1 ? my_row(1) : r0;
        if (lane == 0) {
          mbar_expect_tx(bar(BAR_Q), kTileBytes * (n > 1 ? 3u : 2u));
          tma_load_4d(base + kOffQ, &map_q, bar(BAR_Q), 0, q_row0, h, b);
          if (HD == 128) tma_load_4d(base + kOffQ + kHalfBytes, &map_q, bar(BAR_Q), 64, q_row0, h, b);
        }
        __syncwarp();
        if (active) {
          load_part(&map_k, base + kOffK, bar(BAR_Q), r0);
          if (n > 1) load_part(&map_k, base + kOffK + kTileBytes, bar(BAR_Q), r1);
        }
        int rv = r0, rv1 = r1;
        bool ok = true;
        int st = 0;
        for (int u = 0; u < n && ok; ++u) {
          const bool more = u + 2 < n;
          const int rk = more ? my_row(u + 2) : rv;
          if (u >= 1) {
            int okk = 1;
            if (lane == 0)
              okk = mbar_wait(bar(BAR_SFULL + ((u - 1) & 3)), (uint32_t)((u - 1) >> 2) & 1u, abort_flag, 100 + st) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, okk, 0) != 0;
            if (!ok) break;
          }
          TRACE(3, 10, u);
          if (lane == 0) mbar_expect_tx(bar(BAR_STAGE + st), more ? 2u * kTileBytes : kTileBytes);
          __syncwarp();
          if (active) {
            load_part(&map_v, base + kOffV + (uint32_t)st * kTileBytes, bar(BAR_STAGE + st), rv);
            if (more) load_part(&map_k, base + kOffK + (uint32_t)(st == 0 ? 2 : st - 1) * kTileBytes, bar(BAR_STAGE + st), rk);
          }
          rv = rv1; rv1 = rk;
          if (++st == kStages) st = 0;
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
      auto load_tile = [&](const CUtensorMap* map, uint32_t dst, uint32_t barrier, int row) {
        tma_load_4d(dst, map, barrier, 0, row, h, b);
        if (HD == 128) tma_load_4d(dst + kHalfBytes, map, barrier, 64, row, h, b);
      };
      // Q with the first score tile of each stream
      const int j0 = block_at(0);
      const int j1 = n > 1 ? block_at(1) : j0;
      mbar_expect_tx(bar(BAR_Q), kTileBytes * (n > 1 ? 3u : 2u));
      load_tile(&map_q, base + kOffQ, bar(BAR_Q), q_row0);
      load_tile(&map_k, base + kOffK, bar(BAR_Q), j0);
      if (n > 1) load_tile(&map_k, base + kOffK + kTileBytes, bar(BAR_Q), j1);
      // stage u = {V_u, K_{u+2}}; its slots were last read by service u-3, whose end is the
      // completion of Q K_{u-1}^T
      int jv = j0, jv1 = j1;                          // first rows of V_u and V_{u+1}
      bool ok = true;
      int st = 0;
      for (int u = 0; u < n && ok; ++u) {
        const bool more = u + 2 < n;
        const int jk = more ? block_at(u + 2) : jv;
        if (u >= 1) {
          ok = mbar_wait(bar(BAR_SFULL + ((u - 1) & 3)), (uint32_t)((u - 1) >> 2) & 1u, abort_flag, 100 + st);
          if (!ok) break;
        }
        TRACE(3, 10, u);
        if (u == p.debug_drop_stage) {
          mbar_expect_tx(bar(BAR_STAGE + st), kTileBytes);                 // bytes that never arrive
          jv = jv1; jv1 = jk;
          if (++st == kStages) st = 0;
          continue;
        }
        if (kMass) {
          if (more) mbar_expect_tx(bar(BAR_STAGE + st), kTileBytes);       // no V in mass mode
        } else {
          mbar_expect_tx(bar(BAR_STAGE + st), more ? 2u * kTileBytes : kTileBytes);
          load_tile(&map_v, base + kOffV + (uint32_t)st * kTileBytes, bar(BAR_STAGE + st), jv);
        }
        if (more) {
          const int sk = st == 0 ? 2 : st - 1;         // (u + 2) % 3
          load_tile(&map_k, base + kOffK + (uint32_t)sk * kTileBytes, bar(BAR_STAGE + st), jk);
        }
        jv = jv1; jv1 = jk;
        if (++st == kStages) st = 0;
      }
    }
  } else if (warp == 9) {
    // ================================ MMA issuer ========================================
    reg_dec<kRegsOther>();
    // All 32 lanes run this loop converged (every value in it is warp-uniform); the MMA and commit
    // wrappers elect the one lane that issues.  Waits are made warp-uniform with a vote so that no
    // lane can leave the loop alone.
    auto wait_all = [&](uint32_t b, uint32_t parity, int site) {
      return __all_sync(0xffffffffu, mbar_wait(b, parity, abort_flag, site));
    };
    if (n > 0) {
      constexpr uint32_t idesc_qk = instr_desc(false, 128u);         // S: 128 queries x 128 keys
      constexpr uint32_t idesc_pv = instr_desc(true, (uint32_t)HD);  // O: 128 queries x HD
      const uint64_t qdesc0 = smem_desc(base + kOffQ, 16, 1024);
      const uint64_t kdesc0 = smem_desc(base + kOffK, 16, 1024);
      const uint64_t vdesc0 = smem_desc(base + kOffV, kHalfBytes, 1024);
      // S[t&1] = Q K_t^T, K_t in slot sk
      auto issue_qk = [&](int t, int sk) {
        const uint64_t kd = kdesc0 + (uint64_t)((uint32_t)sk * (kTileBytes >> 4));
        const uint32_t ts = tS[t & 1];
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
          // 16 contraction elements = 32 bytes inside the swizzle atom; second half 16 KB on
          const uint64_t off = (uint64_t)((((uint32_t)kk >> 2) * kHalfBytes + ((uint32_t)kk & 3u) * 32u) >> 4);
          umma_ss(ts, qdesc0 + off, kd + off, idesc_qk, kk > 0 ? 1u : 0u);
        }
      };
      bool ok = wait_all(bar(BAR_Q), 0, 200);
      if (ok) {
        tc_fence_after();
        TRACE(0, 20, 0);
        issue_qk(0, 0);
        umma_commit(bar(BAR_SFULL + 0));
        if (n > 1) {
          issue_qk(1, 1);
          umma_commit(bar(BAR_SFULL + 1));
        }
        TRACE(0, 21, 0);
        if (!kMass || n > 2) ok = wait_all(bar(BAR_STAGE + 0), 0u, 210);
      }
      int st = 0;
      uint32_t sph = 0;
      for (int u = 0; u < n && ok; ++u) {
        const int x = u & 1;
        const uint64_t vd = vdesc0 + (uint64_t)((uint32_t)st * (kTileBytes >> 4));
        const uint32_t to = tO[x], tp = tS[x];
        const uint32_t acc0 = u >= 2 ? 1u : 0u;
        ok = wait_all(bar(BAR_PFULL + x), (uint32_t)(u >> 1) & 1u, 220 + x);
        if (!ok) break;
        tc_fence_after();
        TRACE(0, 22, u);
        if (!kMass) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)             // 16 keys = 16 rows of 128 B; P advances 8 columns
            umma_ts(to, tp + (uint32_t)kk * 8u, vd + (uint64_t)((uint32_t)kk * (2048u >> 4)), idesc_pv,
                    kk > 0 ? 1u : acc0);
        }
        if (u + 2 < n) {
          issue_qk(u + 2, st == 0 ? 2 : st - 1);
          umma_commit(bar(BAR_SFULL + ((u + 2) & 3)));
        } else {
          umma_commit(bar(BAR_OFULL + x));           // the stream's last tile
        }
        TRACE(0, 24, u);
        if (++st == kStages) { st = 0; sph ^= 1u; }
        if (kMass ? (u + 3 < n) : (u + 1 < n)) {     // operands of the next service, while this one runs
          ok = wait_all(bar(BAR_STAGE + st), sph, 210 + st);
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
    const int x = warp >> 2;                        // stream
    const int row = (warp & 3) * 32 + lane;         // query row = TMEM lane
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const float c = p.scale * 1.4426950408889634f;  // logits in log2 units
    // valid key columns of the last tile: lists ascend, so only the final entry can be the
    // partial last key block (gathered blocks are masked per entry below)
    int last_valid = kBlock;
    if (n > 0 && gather == 1 && (dense || list[cnt - 1] == p.n_kb - 1)) last_valid = p.L_k - (p.n_k - 1) * kBlock;
    const int row_group = row / sub_rows;           // gathered blocks: which of the tile's query blocks owns this row
    const int tail_sub = p.L_k - (p.n_kb - 1) * sub_rows;     // keys of the last (possibly partial) gathered block
    float m_ref = -INFINITY;                        // reference maximum (raw score units)
    float l = 0.f;
    bool ok = true;
    const int n_mine = (n - x + 1) / 2;             // list positions x, x+2, ...
    float mass_lse2 = 0.f, mass_w = 0.f;
    // mass mode: the selection block this row belongs to (blocks of 128 * m tokens, or p.mass_g blocks
    // of 128 / mass_g tokens per tile; rows of one warp share a block) and its count of valid queries
    int mass_qb = 0;
    if (kMass) {
      const int q_row = qi * kBlock + row;
      const int blk_len = p.mass_g > 1 ? kBlock / p.mass_g : kBlock * p.m;
      mass_qb = q_row / blk_len;
      const int q_valid = min(blk_len, p.L_q - mass_qb * blk_len);
      if (q_row < p.L_q) {
        mass_lse2 = p.lse_in[((size_t)b * p.H + h) * p.L_q + q_row] * 1.4426950408889634f;
        mass_w = 1.0f / (float)q_valid;
      }
    }
    for (int it = 0; it < n_mine && ok; ++it) {
      const int t = 2 * it + x;
      // gathered blocks: this tile's union entries, fetched before the wait so that the loads
      // are not on the critical path (0 = no entry)
      int ent[4] = {0, 0, 0, 0};
      if (kMode == 2) {
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          const int e = t * gather + g;
          if (g < gather && e < cnt) ent[g] = list[e];
        }
      }
      ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_SFULL + (t & 3)), (uint32_t)(t >> 2) & 1u, abort_flag, 300 + x));
      if (!ok) break;
      tc_fence_after();
      TRACE(1 + x, 30, t);
      // Valid key columns of the tile's four 32-column segments for this row.  Gathered blocks:
      // an entry counts only if this row's query block keeps it (rows of one warp share a query
      // block, so all of this is warp-uniform).
      int c0 = 32, c1 = 32, c2 = 32, c3 = 32;
      if (gather > 1) {
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
      } else if (t == n - 1 && last_valid < kBlock) {
        c0 = min(max(last_valid, 0), 32); c1 = min(max(last_valid - 32, 0), 32);
        c2 = min(max(last_valid - 64, 0), 32); c3 = min(max(last_valid - 96, 0), 32);
      }
      if (kMode == 2 && (c0 | c1 | c2 | c3) == 0) {
        // nothing of this tile is kept by the row's query block: P = 0
        uint32_t zero[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) zero[i] = 0u;
        tmem_st32(tS[x] + lane_off, zero);
        tmem_st32(tS[x] + lane_off + 32u, zero);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(BAR_PFULL + x));
        continue;
      }
      uint32_t sr[128];
      auto load_s = [&]() {
        tmem_ld32(tS[x] + lane_off + 0u, sr + 0);
        tmem_ld32(tS[x] + lane_off + 32u, sr + 32);
        tmem_ld32(tS[x] + lane_off + 64u, sr + 64);
        tmem_ld32(tS[x] + lane_off + 96u, sr + 96);
        tmem_wait_ld();
        if ((c0 & c1 & c2 & c3) != 32) {                      // some segment is not full: -inf there
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            if (i >= c0) sr[i] = 0xff800000u;
            if (i >= c1) sr[32 + i] = 0xff800000u;
            if (i >= c2) sr[64 + i] = 0xff800000u;
            if (i >= c3) sr[96 + i] = 0xff800000u;
          }
        }
      };
      load_s();
      TRACE(1 + x, 31, t);
      if (kMass) {
        // p = exp(scale*s - lse_row): the dense softmax probability, summed over the keys of each 32-column
        // segment of the tile, then over the segments of one key block
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int sgm = 0; sgm < 4; ++sgm)
#pragma unroll
          for (int i = 0; i < 32; ++i) acc[sgm] += ex2(fmaf(__uint_as_float(sr[32 * sgm + i]), c, -mass_lse2));
        const int g = p.mass_g;                                          // key blocks per tile
        float rs[4];
        if (g == 1) { rs[0] = (acc[0] + acc[1]) + (acc[2] + acc[3]); rs[1] = rs[2] = rs[3] = 0.f; }
        else if (g == 2) { rs[0] = acc[0] + acc[1]; rs[1] = acc[2] + acc[3]; rs[2] = rs[3] = 0.f; }
        else { rs[0] = acc[0]; rs[1] = acc[1]; rs[2] = acc[2]; rs[3] = acc[3]; }
        const int tile = dense ? t : min(max(list[t], 0), p.n_k - 1);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (e < g) {
            float v_ = rs[e] * mass_w;                                   // rows past L_q weigh 0
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v_ += __shfl_xor_sync(0xffffffffu, v_, o);
            // one atomic per warp and key block into the zero-initialised output: no barrier inside the
            // loop, so a warp that abandons a wait can never leave the others of its warpgroup stranded
            const int kb = g > 1 ? tile * g + e : tile / p.m;
            if (lane == 0 && kb < p.n_kb && mass_qb < p.n_qb)
              atomicAdd(&p.mass_out[(((size_t)b * p.H + h) * p.n_qb + mass_qb) * (size_t)p.n_kb + kb], v_);
          }
        }
        mbar_arrive(bar(BAR_PFULL + x));                                 // S may be overwritten
        continue;
      }
      // Softmax against a lagging reference.  Scaling a row's P, O and denominator by a common
      // power of two changes nothing in floating point, so the reference only has to keep the
      // numbers far from overflow: it is the row maximum of the stream's first kept tile and is
      // raised only when a tile's sum of exponentials leaves the safe range (or is not finite).
      // The common tile therefore needs no row maximum at all: exponentials against the current
      // reference, one comparison on their sum.  P stays in registers until that check has passed;
      // otherwise (first tile, or the rare raise) the tile is redone from S, still intact in
      // tensor memory, against its own maximum after O and the denominator have been rescaled.
      // exponentials of one half of the tile (64 keys) against m_ref, packed and stored as P
      auto exp_half = [&](int cc) {
        const float nmc = -(m_ref * c);
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
        tmem_st32(tS[x] + lane_off + 32u * cc, pk);            // P (bf16) over the first 64 columns of S
        return (sum[0] + sum[1]) + (sum[2] + sum[3]);
      };
      // The first half's P overwrites S columns 0..31 before the check; a redo takes those scores
      // from the registers, which still hold them, and reloads only the upper 64 columns.
      float tile_sum = 0.f;
      const bool fresh = m_ref == -INFINITY;                   // no kept key seen yet
      if (!__any_sync(0xffffffffu, fresh)) tile_sum = exp_half(0) + exp_half(1);
      const bool redo = fresh || !(tile_sum < kSumLimit);      // also catches inf and NaN
      if (__any_sync(0xffffffffu, redo)) {
        tmem_ld32(tS[x] + lane_off + 64u, sr + 64);
        tmem_ld32(tS[x] + lane_off + 96u, sr + 96);
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
        const float m_new = fmaxf(m_ref, mx);
        if (it > 0) {
          // The stream's previous P V is complete: this S tile was issued after it and the
          // tensor pipe completes in order.  Scale O in place (rows whose reference stays: by 1).
          const float alpha = fresh ? 0.f : ex2((m_ref - m_new) * c);
          tmem_wait_st();
#pragma unroll 1
          for (int cc = 0; cc < HD / 32; ++cc) {
            uint32_t orr[32];
            tmem_ld32(tO[x] + lane_off + 32u * cc, orr);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * alpha);
            tmem_st32(tO[x] + lane_off + 32u * cc, orr);
          }
          l *= alpha;
        }
        m_ref = m_new;
        tile_sum = exp_half(0) + exp_half(1);
      }
      TRACE(1 + x, 32, t);
      l += tile_sum;
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar(BAR_PFULL + x));
      TRACE(1 + x, 33, t);
    }
    // ---- merge the two streams and write O ------------------------------------------------
    if (ok && n_mine > 0) {
      ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_OFULL + x), 0u, abort_flag, 320 + x));
      tc_fence_after();
    }
    if (!kMass) {
    stats[x * 128 + row] = make_float2(m_ref, l);
    tc_fence_before();
    asm volatile("bar.sync 1, 256;" ::: "memory");            // both streams' last PV have landed
    tc_fence_after();
    const int n1 = n / 2;                                     // tiles of stream 1
    const float m0 = stats[row].x, l0 = stats[row].y;
    const float m1 = stats[128 + row].x, l1 = stats[128 + row].y;
    if (*abort_flag == 0 && n > 0) {
      // a stream that saw no kept key for this row (gathered blocks) still has m = -inf, l = 0
      const float m = fmaxf(m0, n1 > 0 ? m1 : -INFINITY);
      const float w0 = m0 > -INFINITY ? ex2((m0 - m) * c) : 0.f;
      const float w1 = n1 > 0 && m1 > -INFINITY ? ex2((m1 - m) * c) : 0.f;
      const float lt = l0 * w0 + l1 * w1;
      const float inv = lt > 0.f ? 1.0f / lt : 0.f;          // a row whose query block keeps nothing gives zeros
      const int q_row = q_row0 + row;
      constexpr int kCols = HD / 2;                           // this warpgroup's half of D
      constexpr int kChunks = kCols / 32;
      const uint32_t col0 = (uint32_t)x * (uint32_t)kCols;
      uint32_t oa[kChunks][32], ob[kChunks][32];
#pragma unroll
      for (int cc = 0; cc < kChunks; ++cc) {
        tmem_ld32(tO[0] + lane_off + col0 + 32u * cc, oa[cc]);
        if (n1 > 0) tmem_ld32(tO[1] + lane_off + col0 + 32u * cc, ob[cc]);
      }
      tmem_wait_ld();
      if (q_row < p.L_q) {
        __nv_bfloat16* og = reinterpret_cast<__nv_bfloat16*>(p.o) + b * p.osB + h * p.osH +
                            (long long)q_row * p.osL + col0;
        const float s0 = w0 * inv, s1 = w1 * inv;
        uint32_t out[kChunks * 16];
#pragma unroll
        for (int cc = 0; cc < kChunks; ++cc)
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            float v0 = __uint_as_float(oa[cc][2 * i]) * s0, v1 = __uint_as_float(oa[cc][2 * i + 1]) * s0;
            if (n1 > 0) {
              v0 = fmaf(__uint_as_float(ob[cc][2 * i]), s1, v0);
              v1 = fmaf(__uint_as_float(ob[cc][2 * i + 1]), s1, v1);
            }
            out[cc * 16 + i] = pack_bf16(v0, v1);
          }
        uint4* dst = reinterpret_cast<uint4*>(og);
#pragma unroll
        for (int i = 0; i < kChunks * 4; ++i) dst[i] = make_uint4(out[4 * i], out[4 * i + 1], out[4 * i + 2], out[4 * i + 3]);
        if (p.lse != nullptr && x == 0)
          p.lse[((size_t)b * p.H + h) * p.L_q + q_row] = lt > 0.f ? m * p.scale + logf(lt) : -INFINITY;
      }
    } else if (n == 0 && live) {
      const int q_row = q_row0 + row;
      if (q_row < p.L_q) {
        __nv_bfloat16* og = reinterpret_cast<__nv_bfloat16*>(p.o) + b * p.osB + h * p.osH +
                            (long long)q_row * p.osL + x * (HD / 2);
        uint4* dst = reinterpret_cast<uint4*>(og);
#pragma unroll
        for (int i = 0; i < HD / 16; ++i) dst[i] = make_uint4(0u, 0u, 0u, 0u);
        if (p.lse != nullptr && x == 0) p.lse[((size_t)b * p.H + h) * p.L_q + q_row] = -INFINITY;
      }
    }
    }  // !kMass
  }

  // ---- teardown -----------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 9) tmem_dealloc(tmem, 512);
  if (p.trace != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0)
    for (int i = threadIdx.x; i < 4 * kTraceSlots; i += kThreads) {
      const int role = i / kTraceSlots, k = i % kTraceSlots;
      if (k < p.trace_cap) {
        p.trace[(role * p.trace_cap + k) * 2] = trace_smem[i] >> 26;
        p.trace[(role * p.trace_cap + k) * 2 + 1] = trace_smem[i] & 0x3FFFFFFu;
      }
    }
  if (threadIdx.x == 0 && *abort_flag != 0) record_status(p.status, SPARSTAR_ERR_TIMEOUT, *abort_flag);
}

}  // namespace

// Longest-list-first order of the query blocks of one head (one CTA per (batch, head)): the
// attention grid is walked head by head, so within a head the long rows start first and the
// short ones fill the tail.  rank = number of rows that are longer, or equally long and earlier.
__global__ void __launch_bounds__(256)
attn_order_kernel(const int* __restrict__ kv_num_blocks, int n_q, int m, int n_qb, int cap,
                  int* __restrict__ order) {
  // n_q = 128-row query tiles of the head; tile i belongs to query block i / m
  extern __shared__ int cnt[];
  const size_t base = (size_t)blockIdx.x * n_q;
  for (int i = threadIdx.x; i < n_q; i += blockDim.x)
    cnt[i] = min(kv_num_blocks[(size_t)blockIdx.x * n_qb + i / m], cap);
  __syncthreads();
  for (int i = threadIdx.x; i < n_q; i += blockDim.x) {
    const int c = cnt[i];
    int rank = 0;
    for (int j = 0; j < n_q; ++j) rank += (cnt[j] > c || (cnt[j] == c && j < i)) ? 1 : 0;
    order[base + rank] = i;
  }
}

// Selection blocks shorter than a tile: the g = 128 / block query blocks that share a 128-row
// query tile are served together over the UNION of their key-block lists.  One warp per query
// tile: the g lists are marked in a table of n_kb bytes (bit s = block is in the list of the
// tile's s-th query block), the table is compacted in ascending block order into entries
// (block << 4) | bits.  Entries out of range or not ascending are flagged and left out.
constexpr int kUnionWarps = 4;
__global__ void __launch_bounds__(kUnionWarps * 32)
attn_union_kernel(const int* __restrict__ kv_num_blocks, const int* __restrict__ kv_indices, int cap, int n_qb,
                  int n_kb, int g, int n_tiles, long long total_tiles, int* __restrict__ u_num,
                  int* __restrict__ u_idx, sparstar_devstatus* status) {
  extern __shared__ unsigned int tab_all[];             // kUnionWarps tables of n_kb bytes, word-aligned
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int words = (n_kb + 3) / 4;
  unsigned int* tab = tab_all + (size_t)warp * words;
  const long long tile = (long long)blockIdx.x * kUnionWarps + warp;   // (batch*head, query tile)
  if (tile >= total_tiles) return;
  const long long bh = tile / n_tiles;
  const int ti = (int)(tile % n_tiles);
  for (int w = lane; w < words; w += 32) tab[w] = 0u;
  __syncwarp();
  for (int sblk = 0; sblk < g; ++sblk) {
    const int qb = ti * g + sblk;
    if (qb >= n_qb) break;
    const size_t row = (size_t)bh * n_qb + qb;
    const int cnt = max(min(kv_num_blocks[row], cap), 0);
    const int* list = kv_indices + row * (size_t)cap;
    for (int e = lane; e < cnt; e += 32) {
      const int j = list[e];
      if (j < 0 || j >= n_kb || (e > 0 && list[e - 1] >= j)) {
        record_status(status, SPARSTAR_ERR_BAD_INDEX, (int)row);
        continue;
      }
      atomicOr(&tab[j >> 2], (1u << sblk) << ((j & 3) * 8));
    }
  }
  __syncwarp();
  int* out = u_idx + (size_t)tile * n_kb;
  int written = 0;
  const unsigned lt = (1u << lane) - 1u;
  for (int j0 = 0; j0 < n_kb; j0 += 32) {
    const int j = j0 + lane;
    const unsigned bits = j < n_kb ? (tab[j >> 2] >> ((j & 3) * 8)) & 0xffu : 0u;
    const unsigned present = __ballot_sync(0xffffffffu, bits != 0u);
    if (bits != 0u) out[written + __popc(present & lt)] = (j << 4) | (int)bits;
    written += __popc(present);
  }
  if (lane == 0) u_num[tile] = written;
}

template <int kMode, int HD = 128>
int launch_variant(sparstar_ctx* ctx, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                   const TcParams& p, dim3 grid, cudaStream_t s) {
  static bool attr_set[64] = {};
  if (!attr_set[ctx->device & 63]) {
    // the in-kernel register re-balancing needs the compiled allocation to be what it assumes
    cudaFuncAttributes fa;
    SPARSTAR_CUDA_TRY(cudaFuncGetAttributes(&fa, attn_tc_kernel<kMode, HD>));
    if (2 * 128 * kRegsSoftmax + 128 * kRegsOther > kThreads * fa.numRegs) return SPARSTAR_ERR_UNSUPPORTED;
    SPARSTAR_CUDA_TRY(cudaFuncSetAttribute(attn_tc_kernel<kMode, HD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)smem_bytes_for(HD)));
    attr_set[ctx->device & 63] = true;
  }
  attn_tc_kernel<kMode, HD><<<grid, kThreads, smem_bytes_for(HD), s>>>(mq, mk, mv, p);
  return SPARSTAR_OK;
}

bool attn_tc_supported(const AttnArgs& a) {
  // selection blocks of 128, 256 or 512 tokens are walked as 1, 2 or 4 tiles of 128; blocks of 64
  // or 32 tokens are gathered two or four to a tile (dense attention has no lists: any block size
  // runs as 128)
  const bool block_ok = a.block == 32 || a.block == 64 || a.block == 128 || a.block == 256 || a.block == 512;
  return a.q.dtype == SPARSTAR_BF16 && (a.q.D == 128 || a.q.D == 64) && (block_ok || a.kv_num_blocks == nullptr) &&
         a.q.H <= 65535 && a.q.B <= 65535;
}

int launch_attn_tc(sparstar_ctx* ctx, const AttnArgs& a, cudaStream_t s) {
  CUtensorMap mq, mk, mv;
  int st;
  const bool dense = a.kv_num_blocks == nullptr;
  const int gather = !dense && a.block < kBlock ? kBlock / a.block : 1;
  const int block = dense ? kBlock : a.block;
  const int kv_rows = kBlock / gather;
  // two adjacent query tiles on a pair of CTAs: they must walk the same list
  const bool pair = ctx->attn_impl == SPARSTAR_ATTN_TCGEN05_PAIR && gather == 1 && a.q.D == 128 &&
                    (dense || (block / kBlock) % 2 == 0);
  if ((st = make_map(&mq, a.q)) || (st = make_map(&mk, a.k, pair ? 64 : kv_rows)) || (st = make_map(&mv, a.v, kv_rows)))
    return st;
  TcParams p;
  p.o = a.o.ptr; p.osB = a.o.sB; p.osH = a.o.sH; p.osL = a.o.sL;
  p.H = a.q.H; p.L_q = a.q.L; p.L_k = a.k.L;
  p.gather = gather;
  p.n_q = (a.q.L + kBlock - 1) / kBlock;                 // query tiles = CTAs per head
  p.n_k = (a.k.L + kBlock - 1) / kBlock;
  p.n_qb = (a.q.L + block - 1) / block;
  p.n_kb = (a.k.L + block - 1) / block;
  p.m = gather > 1 ? 1 : block / kBlock;
  p.scale = a.scale;
  p.kv_num_blocks = a.kv_num_blocks; p.kv_indices = a.kv_indices; p.cap = a.cap;
  p.lse = a.lse;
  p.lse_in = nullptr; p.mass_out = nullptr; p.mass_g = 1;
  p.order = nullptr;
  const bool want_order = !dense && p.n_q > 1 && (size_t)p.n_q * sizeof(int) <= 200 * 1024 &&
                          ctx->debug_work_order != 0;
  // context scratch: [work order: one int per query tile] [union counts] [union lists]
  const size_t tiles = (size_t)a.q.B * a.q.H * p.n_q;
  const size_t order_bytes = (tiles * sizeof(int) + 255) / 256 * 256;
  size_t need = want_order ? order_bytes : 0;
  if (gather > 1) need = 2 * order_bytes + tiles * (size_t)p.n_kb * sizeof(int);
  if (need > 0) {
    const int st3 = ensure_scratch(ctx, need, s);
    if (st3 != SPARSTAR_OK) return st3;
  }
  char* scratch = static_cast<char*>(ctx->scratch);
  if (gather > 1) {
    // the query blocks of a tile are served together over the union of their lists
    int* u_num = reinterpret_cast<int*>(scratch + order_bytes);
    int* u_idx = reinterpret_cast<int*>(scratch + 2 * order_bytes);
    const size_t smem = (size_t)kUnionWarps * ((p.n_kb + 3) / 4) * sizeof(unsigned int);
    if (smem > 200 * 1024) return SPARSTAR_ERR_UNSUPPORTED;
    static bool union_attr[64] = {};
    if (!union_attr[ctx->device & 63]) {
      SPARSTAR_CUDA_TRY(cudaFuncSetAttribute(attn_union_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
      union_attr[ctx->device & 63] = true;
    }
    attn_union_kernel<<<(unsigned)((tiles + kUnionWarps - 1) / kUnionWarps), kUnionWarps * 32, smem, s>>>(
        a.kv_num_blocks, a.kv_indices, a.cap, p.n_qb, p.n_kb, gather, p.n_q, (long long)tiles, u_num, u_idx,
        ctx->d_status);
    ctx->launches++;
    p.kv_num_blocks = u_num; p.kv_indices = u_idx; p.cap = p.n_kb;
    p.n_qb = p.n_q;                                      // one (union) list per query tile
  }
  if (want_order) {
    int* order = reinterpret_cast<int*>(scratch);
    static bool order_attr[64] = {};
    if (!order_attr[ctx->device & 63]) {
      SPARSTAR_CUDA_TRY(cudaFuncSetAttribute(attn_order_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
      order_attr[ctx->device & 63] = true;
    }
    // work items: query tiles, or (CTA pairs) pairs of adjacent tiles of one selection block
    const int n_items = pair ? (p.n_q + 1) / 2 : p.n_q, per_block = pair ? p.m / 2 : p.m;
    attn_order_kernel<<<a.q.B * a.q.H, 256, (size_t)n_items * sizeof(int), s>>>(p.kv_num_blocks, n_items, per_block,
                                                                                 p.n_qb, p.cap, order);
    ctx->launches++;
    p.order = order;
  }
  p.status = ctx->d_status;
  p.trace = ctx->trace; p.trace_cap = ctx->trace_cap; p.trace_skip = ctx->trace_skip;
  p.debug_drop_stage = ctx->debug_drop_stage;
  dim3 grid(p.n_q, a.q.H, a.q.B);
  int st2;
  if (gather > 1 && ctx->attn_impl == SPARSTAR_ATTN_TCGEN05_2STREAM)
    st2 = a.q.D == 64 ? launch_variant<2, 64>(ctx, mq, mk, mv, p, grid, s) : launch_variant<2, 128>(ctx, mq, mk, mv, p, grid, s);
  else if (gather > 1)
    st2 = launch_attn_tc3(ctx, mq, mk, mv, p, a.q.D, grid, s, false, true);
  else if (ctx->attn_impl == SPARSTAR_ATTN_TCGEN05_2STREAM)
    st2 = a.q.D == 64 ? launch_variant<0, 64>(ctx, mq, mk, mv, p, grid, s) : launch_variant<0, 128>(ctx, mq, mk, mv, p, grid, s);
  else
    st2 = launch_attn_tc3(ctx, mq, mk, mv, p, a.q.D, grid, s, pair);
  if (st2 != SPARSTAR_OK) return st2;
  ctx->launches++;
  SPARSTAR_CUDA_TRY(cudaGetLastError());
  return SPARSTAR_OK;
}

// ---- block attention mass (analysis) --------------------------------------------------------
int launch_block_mass_tc(sparstar_ctx* ctx, const sparstar_tensor& q, const sparstar_tensor& k, int block, float scale,
                         const float* lse_dense, float* mass_out, cudaStream_t s) {
  CUtensorMap mq, mk;
  int st;
  if ((st = make_map(&mq, q)) || (st = make_map(&mk, k))) return st;
  TcParams p;
  p.o = nullptr; p.osB = p.osH = p.osL = 0;
  p.H = q.H; p.L_q = q.L; p.L_k = k.L;
  p.n_q = (q.L + kBlock - 1) / kBlock;                    // 128-token tiles: the kernel walks every (query tile, key tile)
  p.n_k = (k.L + kBlock - 1) / kBlock;
  p.n_qb = (q.L + block - 1) / block;                     // the output is per selection block
  p.n_kb = (k.L + block - 1) / block;
  p.m = block >= kBlock ? block / kBlock : 1;
  p.mass_g = block < kBlock ? kBlock / block : 1;
  p.gather = 1;
  p.scale = scale;
  p.kv_num_blocks = nullptr; p.kv_indices = nullptr; p.cap = 0;
  p.lse = nullptr;
  p.lse_in = lse_dense; p.mass_out = mass_out;
  p.order = nullptr;
  p.status = ctx->d_status;
  p.trace = nullptr; p.trace_cap = 0; p.trace_skip = 0;
  p.debug_drop_stage = -1;
  dim3 grid(p.n_q, q.H, q.B);
  SPARSTAR_CUDA_TRY(cudaMemsetAsync(mass_out, 0, sizeof(float) * (size_t)q.B * q.H * p.n_qb * p.n_kb, s));
  st = q.D == 64 ? launch_variant<1, 64>(ctx, mq, mk, mk, p, grid, s) : launch_variant<1, 128>(ctx, mq, mk, mk, p, grid, s);
  if (st != SPARSTAR_OK) return st;
  ctx->launches++;
  SPARSTAR_CUDA_TRY(cudaGetLastError());
  return SPARSTAR_OK;
}

// ---- allocation-free variant of the sparse forward -----------------------------------------
namespace {

// Work-order scratch and a status word for callers that cannot allocate.  Lives in the module's
// device image: every GPU that loads the library holds these 257 KB until the process exits.
constexpr int kStaticOrderItems = 65536;                 // B * H * ceil(L_q / 128) at most
struct StaticScratch {
  sparstar_devstatus status;                             // used when the caller passes no status word
  int pad[62];
  int order[kStaticOrderItems];
};
static __device__ __align__(256) StaticScratch g_static_scratch;

// Device address of the array above, looked up once per device with that device current.
// In host code the symbol's name is only a handle, never a pointer a kernel may be given.
StaticScratch* static_scratch_address(int device, cudaError_t* err) {
  static StaticScratch* addr[64] = {};
  *err = cudaSuccess;
  if (device < 0 || device >= 64) { *err = cudaErrorInvalidDevice; return nullptr; }
  if (addr[device] == nullptr) {
    void* ptr = nullptr;
    *err = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (*err != cudaSuccess) return nullptr;
    addr[device] = static_cast<StaticScratch*>(ptr);
  }
  return addr[device];
}

bool row_aligned(const sparstar_tensor* t) {
  return t != nullptr && t->ptr != nullptr && (reinterpret_cast<uintptr_t>(t->ptr) & 15u) == 0 &&
         t->B > 0 && t->H > 0 && t->L > 0 && t->D > 0 && t->sL >= t->D && (t->sL * 2) % 16 == 0 &&
         (t->sH * 2) % 16 == 0 && (t->sB * 2) % 16 == 0 && t->sH >= 0 && t->sB >= 0;
}

}  // namespace

extern "C" int sparstar_sparse_attn_fwd_static(const sparstar_tensor* q, const sparstar_tensor* k,
                                               const sparstar_tensor* v, const sparstar_tensor* o,
                                               int32_t block, float scale, const int32_t* kv_num_blocks,
                                               const int32_t* kv_indices, int32_t cap, float* lse,
                                               int32_t* status_out, void* stream) {
  if (kv_num_blocks == nullptr || kv_indices == nullptr || cap <= 0) return SPARSTAR_ERR_INVALID_ARG;
  if (!row_aligned(q) || !row_aligned(k) || !row_aligned(v) || !row_aligned(o)) return SPARSTAR_ERR_INVALID_ARG;
  if (k->B != q->B || v->B != q->B || o->B != q->B || k->H != q->H || v->H != q->H || o->H != q->H ||
      k->D != q->D || v->D != q->D || o->D != q->D || v->L != k->L || o->L != q->L)
    return SPARSTAR_ERR_INVALID_ARG;
  if (q->dtype != SPARSTAR_BF16 || k->dtype != SPARSTAR_BF16 || v->dtype != SPARSTAR_BF16 ||
      o->dtype != SPARSTAR_BF16 || q->D != kD || block != kBlock || q->H > 65535 || q->B > 65535)
    return SPARSTAR_ERR_UNSUPPORTED;
  const int n_q = (q->L + kBlock - 1) / kBlock;
  const long long items = (long long)q->B * q->H * n_q;
  if (items > kStaticOrderItems) return SPARSTAR_ERR_TOO_LARGE;      // the fixed scratch cannot hold the work order
  if ((size_t)n_q * sizeof(int) > 200 * 1024) return SPARSTAR_ERR_TOO_LARGE;   // the order kernel sorts a head in shared memory

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int device = 0;
  SPARSTAR_CUDA_TRY(cudaGetDevice(&device));
  cudaError_t err;
  StaticScratch* scratch = static_scratch_address(device, &err);
  if (scratch == nullptr) return SPARSTAR_ERR_CUDA;

  // The scratch keeps the previous call's contents.  The order array is rewritten in full for
  // the entries this call reads; the status word must start at zero.
  sparstar_devstatus* status = status_out != nullptr ? reinterpret_cast<sparstar_devstatus*>(status_out)
                                                      : &scratch->status;
  SPARSTAR_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(sparstar_devstatus), s));

  CUtensorMap mq, mk, mv;
  int st;
  if ((st = make_map(&mq, *q)) || (st = make_map(&mk, *k)) || (st = make_map(&mv, *v))) return st;
  TcParams p;
  p.o = o->ptr; p.osB = o->sB; p.osH = o->sH; p.osL = o->sL;
  p.H = q->H; p.L_q = q->L; p.L_k = k->L;
  p.n_q = n_q;
  p.n_k = (k->L + kBlock - 1) / kBlock;
  p.m = 1; p.n_qb = p.n_q; p.n_kb = p.n_k; p.gather = 1;
  p.scale = scale;
  p.kv_num_blocks = kv_num_blocks; p.kv_indices = kv_indices; p.cap = cap;
  p.lse = lse;
  p.lse_in = nullptr; p.mass_out = nullptr; p.mass_g = 1;
  p.order = scratch->order;
  p.status = status;
  p.trace = nullptr; p.trace_cap = 0; p.trace_skip = 0;
  p.debug_drop_stage = -1;
  static bool order_attr[64] = {};
  if (!order_attr[device]) {
    SPARSTAR_CUDA_TRY(cudaFuncSetAttribute(attn_order_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    order_attr[device] = true;
  }
  attn_order_kernel<<<q->B * q->H, 256, (size_t)n_q * sizeof(int), s>>>(kv_num_blocks, n_q, 1, n_q, cap, scratch->order);
  SPARSTAR_CUDA_TRY(cudaGetLastError());
  sparstar_ctx host_only;                       // plain host struct: names the device for the launcher
  host_only.device = device;
  dim3 grid(n_q, q->H, q->B);
  st = launch_attn_tc3(&host_only, mq, mk, mv, p, kD, grid, s);
  if (st != SPARSTAR_OK) return st;
  SPARSTAR_CUDA_TRY(cudaGetLastError());
  return SPARSTAR_OK;
}
