// Forward pass of block-sparse causal attention (paper Section 3.2: a FlashAttention-style
// kernel that never loads or computes a KV block whose mask is zero), with the log-sum-exp.
//
// One CTA owns a super-tile of 256 query rows of one head: two tiles ("slots") of 128 rows
// that share every K / V tile brought into shared memory.  It walks the ascending union of
// the slots' active KV blocks in steps of 128 keys (one 128-token block, or two 64-token
// blocks side by side), each step in two halves of 64 keys; a slot skips the halves none of
// its rows can see.  Roles:
//   warps 0-3 / 4-7 : softmax of slot 0 / 1 (thread = query row = TMEM lane)
//   warp 8          : TMA producer (Q once, then the K and V rings)
//   warps 9 / 10    : issue the tcgen05.mma of slot 0 / 1 (warp-uniform code, one elected lane;
//                     the two warps sit on different scheduler partitions of the SM)
// Tensor memory: S of slot s, half h at columns 128 s + 64 h (P is written as bf16 over the
// first 32 of them), O of slot s at 256 + 128 s.  Per slot the issue order is
//   S_0(0) S_1(0) | PV_0(0) S_0(1) | PV_1(0) S_1(1) | PV_0(1) S_0(2) | ...
// so the two halves of a slot form a double buffer: while the softmax works on one half the
// tensor pipe computes the other, and the second slot fills what is left.  The online softmax
// advances half by half.  A row's reference (the maximum its probabilities are expressed relative
// to) only moves, and O is only rescaled, when a half's probabilities sum to more than 2^8;
// until then they are relative to the older reference, which fp32 / bf16 hold easily, and the
// row maximum is not computed at all.
#pragma once
#include <cuda.h>
#include "lg_common.cuh"

namespace lg {

struct FwdArgs {
  const int32_t* tile_off;   // row_ptr (CSR): entries of super-tile t start at tile_off[(256 / block) * t]
  const int32_t* tile_cnt;   // [n_super_tiles]
  const int32_t* tile_ent;   // kb * 16 + member mask (bit r: pattern row r of the super-tile has the block)
  const int32_t* order;      // [n_super_tiles] launch rank -> super-tile
  __nv_bfloat16* o;
  float* lse;                // [B, Hq, L]
  unsigned int* error_word;  // first word of the workspace header
  unsigned long long expect_fp, expect_fp2;   // fingerprints of the lists this call was told the workspace holds (0: built by the call itself)
  int n_tiles, nB, n_list;   // sizes of the schedule arrays: tiles, pattern blocks, entries (bounds of the checked build)
  int64_t o_strides[3];      // batch, head, token (elements)
  int L, Hq, G;              // G = Hq / Hkv
  int q_start, Lq;           // queries exist for rows [q_start, q_start + Lq) of the L key positions only
                             // (a chunk served against a cache); Q, O, LSE are indexed by row - q_start
  int exact_w, ns;           // token-exact window (0: off) and number of sink blocks
  int win_block, win_phase;  // with exact_w: the window edge is block-aligned in shifted coordinates instead --
                             // row i keeps the keys j with (i + phase) / win_block - (j + phase) / win_block
                             // < exact_w / win_block (a chunk served against a ring whose first kept token
                             // is `phase` tokens into the sequence); win_block = 0: token-exact edge
  const int32_t* doc_start;  // [B, L] first position of each query's document, or null
  float scale_log2;          // scale * log2(e)
  int head_group;            // heads whose CTAs run side by side (cta_coords); >= gridDim.x: all of them
};

constexpr int kFwdTmaWarp = 8, kFwdMmaWarp0 = 9;
constexpr int kFwdThreads = 11 * 32;
constexpr float kFwdMaxProb = 256.0f;   // a half's probabilities may grow to this (relative to the row's reference) before the reference moves
template <int D>
struct FwdSmem {
  static constexpr int kBox = 128 * 128;               // one 64-column box of 128 rows
  static constexpr int kTile = (D / 64) * kBox;        // 128 rows x D bf16
  static constexpr int kKStages = 3, kVStages = 2;
  static constexpr int oQ = 0;                         // [2 slots]
  static constexpr int oK = 2 * kTile;
  static constexpr int oV = oK + kKStages * kTile;
  static constexpr int oBar = oV + kVStages * kTile;
  static constexpr int kTotal = oBar + 256;
};

template <int D, int BS>
__global__ void __launch_bounds__(kFwdThreads, 1)
fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
           const __grid_constant__ CUtensorMap tm_v, const FwdArgs a) {
  using SM = FwdSmem<D>;
  constexpr int R4 = 256 / BS;                  // pattern rows per super-tile (2 or 4)
  constexpr int RS = R4 / 2;                    // pattern rows per slot
  constexpr uint32_t kSlotMask = (1u << RS) - 1u;
  constexpr int kTile = SM::kTile;
  constexpr uint32_t kColS = 0, kColO = 256;
  // SF / PF / OD are indexed [slot * 2 + half].  A parity wait is only meaningful while the barrier
  // is at most one phase behind the waiter; per half buffer that holds by construction (the S
  // product that re-fills a half is queued behind the P V product that read it), which is why
  // "O is complete" is tracked per half as well.
  enum { B_Q = 0, B_KF = 1, B_KE = 4, B_VF = 7, B_VE = 9, B_SF = 11, B_PF = 15, B_OD = 19, B_DRAIN = 23, B_COUNT = 25 };

  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::oBar);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);
  static_assert(B_COUNT * 8 + 8 <= 256, "barrier area too small");
  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);   // same value, known to be warp-uniform
  if ((smem_u32(smem) & 1023u) != 0) {   // the swizzled tiles need 1024-byte alignment
    if (tid == 0) atomicCAS(a.error_word, 0u, (2u << 24) | 1u);
    return;
  }
  if (!lists_match(a.error_word, a.expect_fp, a.expect_fp2, 1u)) return;
  uint8_t* sQ = smem + SM::oQ;
  uint8_t* sK = smem + SM::oK;
  uint8_t* sV = smem + SM::oV;

  // has a wait already given up in this call?  (read now, so that it travels with the schedule loads below)
  unsigned int abort_word = 0;
  if (tid == 0) abort_word = *reinterpret_cast<volatile unsigned int*>(a.error_word);
  int cta_x, cta_y;   // (batch, query head) and launch rank of this CTA's super-tile
  cta_coords(static_cast<long long>(blockIdx.y) * gridDim.x + blockIdx.x, gridDim.x, gridDim.y, a.head_group, cta_x, cta_y);
  const int tile = checked(a.order[cta_y], 0, a.n_tiles - 1, a.error_word, 100);
  const int b = cta_x / a.Hq, h = cta_x % a.Hq, hk = h / a.G;
  const int ent_off = checked(a.tile_off[tile * R4], 0, a.n_list, a.error_word, 101);
  const int n_ent = checked(a.tile_cnt[tile], 0, a.n_list - ent_off, a.error_word, 102);
  const int32_t* ent = a.tile_ent + ent_off;
  const int row0 = tile * 256;
  const int n_steps = (BS == 128) ? n_ent : (n_ent + 1) / 2;
  if (row0 + 256 <= a.q_start) return;   // no query lives in this super-tile (uniform over the CTA)

  // entries of the two halves of step j (0: nobody's member, also past the end)
  auto load_ent = [&](int j, int& e0, int& e1) {
    if (j >= n_steps) { e0 = e1 = 0; return; }
    if (BS == 128) { e0 = e1 = ent[j]; return; }
    e0 = ent[2 * j];
    e1 = (2 * j + 1 < n_ent) ? ent[2 * j + 1] : 0;   // odd tail: no second block
  };

  if (tid == 0) {
    mbar_init(bars + B_Q, 1);
    for (int i = 0; i < 3; ++i) { mbar_init(bars + B_KF + i, 1); mbar_init(bars + B_KE + i, 2); }   // both issuers release
    for (int i = 0; i < 2; ++i) {
      mbar_init(bars + B_VF + i, 1); mbar_init(bars + B_VE + i, 2);
      mbar_init(bars + B_DRAIN + i, 1);
    }
    for (int i = 0; i < 4; ++i) { mbar_init(bars + B_SF + i, 1); mbar_init(bars + B_PF + i, 4); mbar_init(bars + B_OD + i, 1); }
    mbar_fence_init();
    tmem_slot[1] = abort_word;
  }
  if (warp == kFwdMmaWarp0) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  if (tmem_slot[1] != 0) {   // after a failed wait the rest of the grid does nothing: the call ends in seconds, not minutes
    if (warp == kFwdMmaWarp0) tmem_dealloc(tmem, 512);
    return;
  }

  if (warp == kFwdTmaWarp) {
    // ------------------------------ TMA producer ------------------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v);
      mbar_expect_tx(bars + B_Q, 2 * kTile);
#pragma unroll
      for (int s = 0; s < 2; ++s)
#pragma unroll
        for (int x = 0; x < D / 64; ++x)
          // rows before q_start lie outside the tensor and arrive as zeros (their results are never stored)
          tma_load_4d(sQ + s * kTile + x * SM::kBox, &tm_q, bars + B_Q, x * 64, row0 + s * 128 - a.q_start, h, b);
      auto load_step = [&](uint8_t* dst, const CUtensorMap* tm, uint64_t* bar, int kb0, int kb1) {
#pragma unroll
        for (int x = 0; x < D / 64; ++x) {
          tma_load_4d(dst + x * SM::kBox, tm, bar, x * 64, kb0 * BS, hk, b);
          if (BS == 64) tma_load_4d(dst + x * SM::kBox + 64 * 128, tm, bar, x * 64, kb1 * BS, hk, b);
        }
      };
      bool ok = true;
      int nk = 0, nv = 0;   // loads started
      int e_next = n_steps > 0 ? ent[0] : 0, e_next1 = (BS == 64 && n_ent > 1) ? ent[1] : e_next;
      for (int j = 0; j < n_steps; ++j) {
        const int sk = j % 3, sv = j & 1;
        const int kb0 = e_next >> 4, kb1 = e_next1 >> 4;
        if (j + 1 < n_steps) {   // fetch the next step's entries now; they are needed one step later
          const int i0 = (BS == 128) ? j + 1 : 2 * j + 2;
          e_next = ent[i0];
          e_next1 = (BS == 64) ? ent[min(i0 + 1, n_ent - 1)] : e_next;
        }
        if (j >= 3) ok = mbar_wait(bars + B_KE + sk, ((j / 3) - 1) & 1, a.error_word, 2);
        if (!ok) break;
        mbar_expect_tx(bars + B_KF + sk, kTile);
        load_step(sK + sk * kTile, &tm_k, bars + B_KF + sk, kb0, kb1);
        nk = j + 1;
        if (j >= 2) ok = mbar_wait(bars + B_VE + sv, ((j / 2) - 1) & 1, a.error_word, 3);
        if (!ok) break;
        mbar_expect_tx(bars + B_VF + sv, kTile);
        load_step(sV + sv * kTile, &tm_v, bars + B_VF + sv, kb0, kb1);
        nv = j + 1;
      }
      // every copy this thread started has landed before the CTA may exit
      mbar_wait(bars + B_Q, 0, a.error_word, 4);
      for (int j = max(nk - 3, 0); j < nk; ++j) mbar_wait(bars + B_KF + j % 3, (j / 3) & 1, a.error_word, 5);
      for (int j = max(nv - 2, 0); j < nv; ++j) mbar_wait(bars + B_VF + (j & 1), (j / 2) & 1, a.error_word, 6);
    }
  } else if (warp == kFwdMmaWarp0 || warp == kFwdMmaWarp0 + 1) {
    // ------------------------------ MMA issuer of one slot --------------------------------
    // The whole warp runs the loop (addresses and descriptors stay warp-uniform values); one
    // elected lane issues.  Both issuers arrive once per step on the K / V "empty" barriers,
    // whether or not their slot used the step, and only after having seen the step's tile
    // arrive: an idle issuer can then never be a whole ring turn ahead of the other one.
    const int s = warp - kFwdMmaWarp0;
    const bool lead = elect_one();
    constexpr uint32_t idesc_s = make_idesc_bf16(128, 64, 0, 0);
    constexpr uint32_t idesc_o = make_idesc_bf16(128, D, 0, 1);
    constexpr uint32_t kHalfRows = (64 * 128) >> 4;   // 64 rows of a box, in 16-byte units
    const uint32_t hi = desc_hi(1024);
    const uint32_t q_lo = desc_lo(smem_u32(sQ), 16) + s * (kTile >> 4), k_lo = desc_lo(smem_u32(sK), 16);
    const uint32_t v_mn_lo = desc_lo(smem_u32(sV), SM::kBox);
    const uint32_t t_s = tmem + kColS + s * 128, t_o = tmem + kColO + s * 128;
    bool ok = mbar_wait(bars + B_Q, 0, a.error_word, 7);
    int n_pv = 0;                 // P V products issued (accumulate flag)
    int pf0 = 0, pf1 = 0;         // uses of the two half buffers whose P V product was issued (barrier phases)
    int ce0 = 0, ce1 = 0, ne0, ne1, nn0, nn1;
    load_ent(0, ne0, ne1);
    load_ent(1, nn0, nn1);
#pragma unroll 1
    for (int j = -1; j < n_steps; ++j) {   // step -1 only issues the S products of step 0
      bool v_seen = false, k_seen = false;
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const int ce = hf ? ce1 : ce0, ne = hf ? ne1 : ne0;
        if ((static_cast<uint32_t>(ce) >> (s * RS)) & kSlotMask) {           // P V of half hf of step j
          const int sv = j & 1;
          if (!v_seen) { ok = ok && mbar_wait(bars + B_VF + sv, (j / 2) & 1, a.error_word, 9); v_seen = true; }
          ok = ok && mbar_wait(bars + B_PF + s * 2 + hf, (hf ? pf1 : pf0) & 1, a.error_word, 10);
          if (ok) {
            tc_fence_after();
            const uint32_t b_lo = v_mn_lo + sv * (kTile >> 4) + hf * 4 * (2048 >> 4);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              if (lead) mma_ts2(t_o, t_s + hf * 64 + kk * 8, b_lo + kk * (2048 >> 4), hi, idesc_o, (n_pv > 0) || (kk > 0));
          }
          if (lead) mma_commit(bars + B_OD + s * 2 + hf);
          ++n_pv;
          if (hf) ++pf1; else ++pf0;
        }
        if (hf == 1 && j >= 0) {
          if (!v_seen) ok = ok && mbar_wait(bars + B_VF + (j & 1), (j / 2) & 1, a.error_word, 9);
          if (lead) mma_commit(bars + B_VE + (j & 1));
        }
        if ((static_cast<uint32_t>(ne) >> (s * RS)) & kSlotMask) {           // S of half hf of step j + 1
          const int sk = (j + 1) % 3;
          if (!k_seen) { ok = ok && mbar_wait(bars + B_KF + sk, ((j + 1) / 3) & 1, a.error_word, 8); k_seen = true; }
          if (ok) {
            tc_fence_after();
            const uint32_t b_lo = k_lo + sk * (kTile >> 4) + hf * kHalfRows;
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
              constexpr int kB = SM::kBox >> 4;
              const uint32_t off = (k >> 2) * kB + (k & 3) * 2;
              if (lead) mma_ss2(t_s + hf * 64, q_lo + off, b_lo + off, hi, idesc_s, k > 0);
            }
          }
          if (lead) mma_commit(bars + B_SF + s * 2 + hf);
        }
        if (hf == 1 && j + 1 < n_steps) {
          if (!k_seen) ok = ok && mbar_wait(bars + B_KF + (j + 1) % 3, ((j + 1) / 3) & 1, a.error_word, 8);
          if (lead) mma_commit(bars + B_KE + (j + 1) % 3);
        }
      }
      ce0 = ne0; ce1 = ne1;
      ne0 = nn0; ne1 = nn1;
      load_ent(j + 3, nn0, nn1);   // read ahead: off the critical path
    }
    if (lead) mma_commit(bars + B_DRAIN + s);
    mbar_wait(bars + B_DRAIN + s, 0, a.error_word, 11);   // nothing of ours is still running at exit
  } else {
    // ------------------------------ softmax warps -----------------------------------------
    const int s = warp >> 2;                                 // slot
    const int r = (warp & 3) * 32 + lane;                    // row in the slot == TMEM lane
    const int qi = row0 + s * 128 + r;
    const int member = s * RS + (BS == 128 ? 0 : (r >> 6));  // pattern row of the super-tile
    const uint32_t lane_addr = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const uint32_t my_s = lane_addr + kColS + s * 128, my_o = lane_addr + kColO + s * 128;
    // lowest key position this row may see outside what the pattern already excludes: the start of its
    // document (0 without documents)
    const int dstart = (a.doc_start && qi < a.L && qi >= a.q_start) ? a.doc_start[static_cast<int64_t>(b) * a.L + qi] : 0;
    // oldest key position the window lets this row see (blocks outside the sink)
    const int win_lo = a.win_block > 0
                           ? ((qi + a.win_phase) / a.win_block - a.exact_w / a.win_block + 1) * a.win_block - a.win_phase
                           : qi - a.exact_w + 1;
    float m_ref = -INFINITY;   // reference maximum (scaled, log2 domain) the probabilities are relative to
    float l_run = 0.f;
    int p0 = 0, p1 = 0;        // P tiles published per half buffer (barrier phases)
    // every P V product issued so far has completed (at most one per half can still be running)
    auto wait_o = [&](uint32_t site) {
      bool w = true;
      if (p0 > 0) w = mbar_wait_warp(bars + B_OD + s * 2, (p0 - 1) & 1, a.error_word, site);
      if (w && p1 > 0) w = mbar_wait_warp(bars + B_OD + s * 2 + 1, (p1 - 1) & 1, a.error_word, site);
      return w;
    };
    bool ok = true;
    int ne0, ne1;
    load_ent(0, ne0, ne1);
#pragma unroll 1
    for (int j = 0; j < n_steps && ok; ++j) {
      const int e0 = ne0, e1 = ne1;
      load_ent(j + 1, ne0, ne1);
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const int e = hf ? e1 : e0;
        if (((static_cast<uint32_t>(e) >> (s * RS)) & kSlotMask) == 0) continue;   // uniform over the slot
        // visible columns of this half: lo <= c < lim (the lower bound only exists with a
        // token-exact window, on blocks outside the sink)
        const int key0 = (e >> 4) * BS + (BS == 128 ? 64 * hf : 0);
        const int lim = ((e >> member) & 1) ? min(max(qi - key0 + 1, 0), 64) : 0;
        const int lo_abs = (a.exact_w > 0 && (e >> 4) >= a.ns) ? max(dstart, win_lo) : dstart;
        const int lo = min(max(lo_abs - key0, 0), 64);

        const bool masked = __any_sync(0xffffffffu, lim < 64 || lo > 0);   // (voted before the wait: off the chain)
        ok = mbar_wait_warp(bars + B_SF + s * 2 + hf, (hf ? p1 : p0) & 1, a.error_word, 12);
        if (!ok) break;
        tc_fence_after();
        uint32_t v[64];
        tmem_ld32(my_s + hf * 64, v);
        tmem_ld32(my_s + hf * 64 + 32, v + 32);
        tmem_ld_wait();
        if (masked) {
#pragma unroll
          for (int x = 0; x < 64; ++x)
            v[x] = (x < lim && x >= lo) ? v[x] : 0xff800000u;   // -inf: the exponential below gives exactly 0
        }
        // Probabilities relative to the reference as it stands; the row maximum is only looked at when
        // that cannot be right: the row has no reference yet, or the sum of the half's probabilities
        // (an upper bound of each of them) passes 2^8.  Otherwise every probability is below 2^8 and the
        // reference stays -- the maximum, its 32 instructions per row and the vote are off the common path.
        uint32_t preg[32];
        float psum;
        auto exp_half = [&](float neg_m) {
          float q0 = 0.f, q1 = 0.f, q2 = 0.f, q3 = 0.f;   // independent partial sums
#pragma unroll
          for (int x = 0; x < 64; x += 4) {
            const float x0 = fmaf(__uint_as_float(v[x]), a.scale_log2, neg_m);
            const float x1 = fmaf(__uint_as_float(v[x + 1]), a.scale_log2, neg_m);
            const float x2 = fmaf(__uint_as_float(v[x + 2]), a.scale_log2, neg_m);
            const float x3 = fmaf(__uint_as_float(v[x + 3]), a.scale_log2, neg_m);
            const float e0 = fast_exp2(x0), e1 = fast_exp2(x1), e2 = fast_exp2(x2), e3 = fast_exp2(x3);
            q0 += e0; q1 += e1; q2 += e2; q3 += e3;
            preg[x >> 1] = pack_bf16(e0, e1);
            preg[(x >> 1) + 1] = pack_bf16(e2, e3);
          }
          psum = (q0 + q2) + (q1 + q3);
        };
        const bool unset = (m_ref == -INFINITY);
        exp_half(unset ? 0.f : -m_ref);
        // (an unset reference with every column masked gives zeros and stays unset; NaN compares false
        // and cannot appear: masked scores are -inf, whose exponential is 0)
        const bool look = unset ? (lim > lo) : !(psum <= kFwdMaxProb);
        if (__any_sync(0xffffffffu, look)) {
          float mx;
          {
            float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
            for (int x = 0; x < 64; x += 8) {
              m0 = max3(m0, __uint_as_float(v[x + 0]), __uint_as_float(v[x + 1]));
              m1 = max3(m1, __uint_as_float(v[x + 2]), __uint_as_float(v[x + 3]));
              m2 = max3(m2, __uint_as_float(v[x + 4]), __uint_as_float(v[x + 5]));
              m3 = max3(m3, __uint_as_float(v[x + 6]), __uint_as_float(v[x + 7]));
            }
            mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
          }
          // the rows that asked move their reference to the maximum seen so far (the others keep theirs)
          const float m_new = fmaxf(m_ref, mx * a.scale_log2);
          const bool raise = look && m_new > m_ref;
          const float alpha = raise ? fast_exp2(m_ref - m_new) : 1.f;   // m_ref = -inf -> 0
          if (raise) { m_ref = m_new; l_run *= alpha; }
          if (p0 + p1 > 0) {   // O already holds products: wait for them, then rescale my row
            ok = wait_o(13);
            if (!ok) break;
            tc_fence_after();
#pragma unroll 1
            for (int c = 0; c < D / 16; ++c) {
              uint32_t oreg[16];
              tmem_ld16(my_o + c * 16, oreg);
              tmem_ld_wait();
#pragma unroll
              for (int x = 0; x < 16; ++x) oreg[x] = __float_as_uint(__uint_as_float(oreg[x]) * alpha);
              tmem_st16(my_o + c * 16, oreg);
            }
          }
          exp_half((m_ref == -INFINITY) ? 0.f : -m_ref);
        }
        l_run += psum;
        tmem_st32(my_s + hf * 64, preg);   // P over the first columns of this half's S
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + B_PF + s * 2 + hf);
        if (hf) ++p1; else ++p0;
      }
    }
    // ---- epilogue: O / l -> bf16, LSE ------------------------------------------------------
    if (ok) ok = wait_o(14);
    // warp-uniform condition (the tensor-memory loads below need the whole warp): some row of the warp
    // is a real query; rows past L or before q_start load with the others and store nothing
    if (ok && p0 + p1 > 0 && qi - lane < a.L && qi - lane + 32 > a.q_start) {
      const bool mine = qi < a.L && qi >= a.q_start;
      tc_fence_after();
      const float inv_l = l_run > 0.f ? 1.f / l_run : 0.f;
      // rows leave through the slot's own Q tile (its last S product is done: it precedes the last P V in
      // the issuer's queue), 4 KB per warp, so that the stores cover whole rows (store_acc_64cols)
      uint8_t* stage = sQ + s * kTile + (warp & 3) * 4096;
      const int q_first = row0 + s * 128 + (warp & 3) * 32;        // the warp's first row
      __nv_bfloat16* obase = a.o + b * a.o_strides[0] + h * a.o_strides[1];
#pragma unroll
      for (int c = 0; c < D / 64; ++c)
        store_acc_64cols(my_o + c * 64, stage, inv_l, [&](int r2) -> __nv_bfloat16* {
          const int q2 = q_first + r2;
          return (q2 < a.L && q2 >= a.q_start) ? obase + static_cast<int64_t>(q2 - a.q_start) * a.o_strides[2] + c * 64 : nullptr;
        });
      if (mine)
        a.lse[(static_cast<int64_t>(b) * a.Hq + h) * a.Lq + qi - a.q_start] =
            l_run > 0.f ? (m_ref + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kFwdMmaWarp0) tmem_dealloc(tmem, 512);
}

}  // namespace lg
