// Backward pass of block-sparse causal attention (paper Section 3.2: masked blocks are
// skipped in the backward as in the forward; Table 1 counts both in the training FLOPs).
//
//   delta_i = dO_i . O_i                      P = exp(scale * S - LSE) on visible pairs
//   dV = P^T dO      dP = dO V^T      dS = P * (dP - delta)
//   dQ = scale * dS K                 dK = scale * dS^T Q      (dK, dV summed over a GQA group)
//
// Two passes, each with a single writer per output tile and a fixed accumulation order:
//   * dK/dV pass: one CTA per tile of 128 keys of one kv head; it walks the query blocks of
//     the tile's CSC column(s) for every query head of the group.  S^T = K Q^T and
//     dP^T = V dO^T land in tensor memory with one key per lane; P^T and dS^T are written
//     back as bf16 over them and feed dV += P^T dO and dK += dS^T Q as TMEM A operands.
//   * dQ pass: one CTA per tile of 128 queries of one head walks its CSR row(s):
//     S = Q K^T, dP = dO V^T, dS over S, dQ += dS K.
//
// Both kernels are warp-specialised: warps 0-15 do the element-wise work (four groups of four
// warps; thread = TMEM lane, each group owns a quarter of the columns in work), warp 16 feeds
// shared memory with TMA, warps 17 and 18 issue tcgen05.mma (the whole warp runs the loop with
// warp-uniform values, one elected lane issues).  The two issuing warps sit on different scheduler
// partitions of the SM: issuing an MMA is slowed by other warps' arithmetic on the issuer's
// partition, and two queues halve what each has to push through.  MMAs whose operands alias in
// tensor memory stay on one warp, so that the queue order is the only synchronisation they need.
// A step covers 128 streamed rows: one 128-token pattern block, or two 64-token blocks side by
// side; the dK/dV pass works it in two half-steps of 64 queries whose score buffers alternate.
//   dQ pass   : warp A: dQ(j) then S(j+2) (S double-buffered, dS over S)   warp B: dP(j+1) once dP(j) is read
//   dK/dV pass: warp A: dV(h) then S^T(h+2) (P^T over S^T)       warp B: dK(h) then dP^T(h+2)   (h: half-step)
// Options folded into the masks: a token-exact window edge, packed documents (no key of an earlier
// document), and a sequence length that ends inside a block.
#pragma once
#include <cuda.h>
#include "lg_common.cuh"

namespace lg {

struct BwdArgs {
  const int32_t* tile_off;   // dQ pass: CSR row_ptr (tile t starts at tile_off[R t]); dK/dV pass: start per tile
  const int32_t* tile_cols;  // dK/dV pass: pattern column of each member of a kv tile (-1: none)
  const int32_t* tile_cnt;
  const int32_t* tile_ent;   // idx * 4 + member mask
  const int32_t* order;
  const float* stat;         // two planes of [B, Hq, Lp] floats: -LSE * log2(e), then -delta; Lp = L rounded up
                             // to 128 (rows past L hold zeros, so that whole-tile copies stay inside a head)
  int64_t stat_plane;        // floats per plane
  int Lp;
  __nv_bfloat16* out0;       // dQ   | dK
  __nv_bfloat16* out1;       // unused | dV
  unsigned int* error_word;  // first word of the workspace header
  unsigned long long expect_fp, expect_fp2;   // fingerprints of the lists this call was told the workspace holds (0: built by the call itself)
  int n_tiles, nB, n_list;   // sizes of the schedule arrays: tiles, pattern blocks, entries (bounds of the checked build)
  int64_t s0[3], s1[3];      // strides of out0 / out1 (batch, head, token; elements)
  int L, Hq, Hkv, G;
  int exact_w, ns;           // token-exact window (0: off) and number of sink blocks
  const int32_t* doc_start;  // [B, L] first position of each token's document, or null
  const int32_t* doc_end;    // [B, L] end of each token's document (null together with doc_start)
  float scale, scale_log2;
  // dK/dV pass that also keeps dS (see bwd_dkdv_kernel): dS^T of every block of the pattern goes to ds_buf
  // in tiles of 64 queries x KT keys, KT = the block size: with p = the block's position in the column
  // lists (col_ptr[column] + rank of the query block in the column), a head's tiles are 2 p and 2 p + 1
  // (the block's two 64-query halves, 16 KB each) with 128-token blocks and p (8 KB) with 64-token
  // blocks; head (b, h) starts at tile (b * Hq + h) * ds_nnz * (block / 64).  The dQ pass reads them back.
  // Inside a tile the element (key k, query q) sits at byte (q / 8) * 16 KT + k * 16 + (q % 8) * 2: eight
  // queries of one key are 16 contiguous bytes, the KT keys of such a group follow one another -- the
  // un-swizzled core-matrix layout of a tensor-core operand whose M (query) index is the contiguous one,
  // and a layout in which the 32 key rows of a warp write 512 contiguous bytes per store instruction.
  int64_t ds_nnz;
  __nv_bfloat16* ds_buf;
  const int32_t* col_ptr;    // column lists of the pattern (dK/dV pass that keeps dS: positions of its blocks)
  int ahead;                 // dK/dV pass: CTAs that run at a time (see prefetch_successor), 0: no prefetch
  int head_group;            // dK/dV pass: kv heads whose CTAs run side by side (cta_coords); >= gridDim.x: all of them
  int descending;            // dK/dV pass: walk a tile's entries from the last query block down (see the producer)
  int n_long;                // dK/dV pass: launch ranks taken in head groups (cta_coords2); >= gridDim.y: all of them
};
template <int BS> constexpr int kDsTileBytes = BS * 64 * 2;

// ---- stat = -(LSE * log2 e) and -rowsum(dO * O), stored negated (they are only ever subtracted),
// each in a plane of its own: the dK/dV pass fetches four neighbouring queries' values of one kind
// with a single 16-byte shared-memory load ---------------------------------------------------------
constexpr int kDeltaRowsPerThread = 4;   // rows a thread works, their loads issued together
template <int D>
__global__ void delta_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ d_o,
                             const float* __restrict__ lse, float* __restrict__ stat, int64_t sb, int64_t sh,
                             int64_t sl, int Hq, int n_bh, int L, int Lp, int64_t plane) {
  // grid.x walks the padded rows of a head (rows i >= L exist only in `stat`, as zeros), grid.y the heads
  constexpr int TPR = D / 8;   // threads per row, 16 bytes each
  constexpr int U = kDeltaRowsPerThread;
  const int rows = blockDim.x / TPR;                       // rows per pass of the block
  const int i0 = blockIdx.x * (rows * U) + threadIdx.x / TPR;
  const int ch = threadIdx.x % TPR;
  for (int bh = blockIdx.y; bh < n_bh; bh += gridDim.y) {
    const int h = bh % Hq, b = bh / Hq;
    uint4 ov[U], dv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + u * rows;
      ov[u] = dv[u] = make_uint4(0, 0, 0, 0);
      if (i < L) {
        const int64_t off = b * sb + h * sh + static_cast<int64_t>(i) * sl + ch * 8;
        ov[u] = *reinterpret_cast<const uint4*>(o + off);
        dv[u] = *reinterpret_cast<const uint4*>(d_o + off);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + u * rows;
      const __nv_bfloat162* op = reinterpret_cast<const __nv_bfloat162*>(&ov[u]);
      const __nv_bfloat162* dp = reinterpret_cast<const __nv_bfloat162*>(&dv[u]);
      float acc = 0.f;
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const float2 a = __bfloat1622float2(op[x]), c = __bfloat1622float2(dp[x]);
        acc += a.x * c.x + a.y * c.y;
      }
#pragma unroll
      for (int s = TPR / 2; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
      if (i < Lp && ch == 0) {
        const int64_t row = static_cast<int64_t>(bh) * Lp + i;
        stat[row] = i < L ? -lse[static_cast<int64_t>(bh) * L + i] * 1.4426950408889634f : 0.f;
        stat[plane + row] = -acc;
      }
    }
  }
}

// Every tile in shared memory holds 128 rows of D bf16: D/64 column boxes of [128 rows x 128 B].
template <int D>
struct BwdTile {
  static constexpr int kBox = 128 * 128;            // bytes of one 64-column box of 128 rows
  static constexpr int kBytes = (D / 64) * kBox;
};

template <int D, int BS>
struct BwdSmem {
  static constexpr int kTile = BwdTile<D>::kBytes;
  static constexpr int kAStages = 3;   // operand read by the first and the last MMA of a step (K | Q)
  static constexpr int kBStages = 2;   // operand read by adjacent MMAs (V | dO)
  static constexpr int oFix0 = 0, oFix1 = kTile;
  static constexpr int oA = 2 * kTile;
  static constexpr int oB = oA + kAStages * kTile;
  static constexpr int oStat = oB + kBStages * kTile;            // dK/dV pass: [2 stages][2 planes][128] floats
  static constexpr int oBar = oStat + 2 * 128 * 8;
  static constexpr int kBarBytes = 512;                          // mbarriers, the TMEM slot and the step's schedule entries
  static constexpr int kTotal = oBar + kBarBytes;
};

// load one step (128 rows: one 128-row block, or two 64-row blocks) of a [.., L, D] tensor
template <int D, int BS>
__device__ __forceinline__ void tma_load_rows(uint8_t* dst, const CUtensorMap* tm, uint64_t* bar, int half,
                                              int row, int head, int batch) {
  // BS == 128: half is ignored (box = 128 rows); BS == 64: box = 64 rows placed at rows 64 * half
#pragma unroll
  for (int x = 0; x < D / 64; ++x)
    tma_load_4d(dst + x * BwdTile<D>::kBox + (BS == 64 ? half * (64 * 128) : 0), tm, bar, x * 64, row, head, batch);
}

// A warp of element-wise threads finished writing tensor memory: publish it to the MMA thread.
__device__ __forceinline__ void ew_publish(uint64_t* bar) {
  tmem_st_wait();
  tc_fence_before();
  __syncwarp();
  if (lane_id() == 0) mbar_arrive(bar);
}

// ================================== dQ pass =================================================
// TMEM columns: S[2] at 0 / 128 (dS of a step is written as bf16 over its own S), dP at 256,
// dQ at 384.  Sixteen element-wise warps (four column groups of 32) and TWO issuing threads on
// different scheduler partitions: thread A issues S and dQ (they alias the same columns, so their
// order must stay with one thread), thread B issues dP (its only hazard is the element-wise read
// of the previous dP, signalled by a barrier).  The two never have to wait for one another.
constexpr int kDqEwWarps = 16;
constexpr int kDqTmaWarp = 16, kDqMmaWarpA = 17, kDqMmaWarpB = 18;
constexpr int kDqThreads = 19 * 32;
constexpr int kDqCols = 128 / (kDqEwWarps / 4);   // columns of a step per element-wise thread

template <int D, int BS>
__global__ void __launch_bounds__(kDqThreads, 1)
bwd_dq_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
              const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
              const BwdArgs a) {
  using SM = BwdSmem<D, BS>;
  constexpr int R = 128 / BS;
  constexpr uint32_t kColS = 0, kColDP = 256, kColDQ = 384;
  constexpr int kTile = SM::kTile;
  enum { B_FIX = 0, B_KF = 1, B_KE = 4, B_VF = 7, B_VE = 9, B_SF = 11, B_DPF = 13, B_DSF = 14, B_DONE = 15,
         B_DRAIN = 16, B_DPR = 18, B_COUNT = 19 };

  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::oBar);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);
  static_assert(B_COUNT * 8 + 8 <= SM::kBarBytes, "barrier area too small");
  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);   // same value, known to be warp-uniform
  if ((smem_u32(smem) & 1023u) != 0) {   // the swizzled tiles need 1024-byte alignment
    if (tid == 0) atomicCAS(a.error_word, 0u, (2u << 24) | 20u);
    return;
  }
  if (!lists_match(a.error_word, a.expect_fp, a.expect_fp2, 20u)) return;
  uint8_t* sQ = smem + SM::oFix0;
  uint8_t* sDO = smem + SM::oFix1;
  uint8_t* sK = smem + SM::oA;
  uint8_t* sV = smem + SM::oB;

  // has a wait already given up in this call?  (read now, so that it travels with the schedule loads below)
  unsigned int abort_word = 0;
  if (tid == 0) abort_word = *reinterpret_cast<volatile unsigned int*>(a.error_word);
  int cta_x, cta_y;   // (batch, query head) and launch rank of this CTA's query tile
  cta_coords(static_cast<long long>(blockIdx.y) * gridDim.x + blockIdx.x, gridDim.x, gridDim.y, a.head_group, cta_x, cta_y);
  const int tile = checked(a.order[cta_y], 0, a.n_tiles - 1, a.error_word, 110);
  const int b = cta_x / a.Hq, h = cta_x % a.Hq, hk = h / a.G;
  const int ent_off = checked(a.tile_off[tile * R], 0, a.n_list, a.error_word, 111);
  const int n_ent = checked(a.tile_cnt[tile], 0, a.n_list - ent_off, a.error_word, 112);
  const int32_t* ent = a.tile_ent + ent_off;
  const int row0 = tile * 128;
  const int n_steps = (BS == 128) ? n_ent : (n_ent + 1) / 2;

  if (tid == 0) {
    mbar_init(bars + B_FIX, 1);
    for (int i = 0; i < 3; ++i) { mbar_init(bars + B_KF + i, 1); mbar_init(bars + B_KE + i, 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bars + B_VF + i, 1); mbar_init(bars + B_VE + i, 1); mbar_init(bars + B_SF + i, 1);
      mbar_init(bars + B_DRAIN + i, 1);
    }
    mbar_init(bars + B_DPF, 1);
    mbar_init(bars + B_DSF, kDqEwWarps);
    mbar_init(bars + B_DPR, kDqEwWarps);
    mbar_init(bars + B_DONE, 1);
    mbar_fence_init();
    tmem_slot[1] = abort_word;
  }
  if (warp == kDqMmaWarpA) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  if (tmem_slot[1] != 0) {   // after a failed wait the rest of the grid does nothing: the call ends in seconds, not minutes
    if (warp == kDqMmaWarpA) tmem_dealloc(tmem, 512);
    return;
  }

  if (warp == kDqTmaWarp) {
    // ------------------------------ TMA producer ------------------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v); tma_prefetch_desc(&tm_do);
      mbar_expect_tx(bars + B_FIX, 2 * kTile);
      tma_load_rows<D, 128>(sQ, &tm_q, bars + B_FIX, 0, row0, h, b);
      tma_load_rows<D, 128>(sDO, &tm_do, bars + B_FIX, 0, row0, h, b);
      bool ok = true;
      int nk = 0, nv = 0;   // loads started
      int e_cur0 = n_steps > 0 ? ent[0] : 0, e_cur1 = (BS == 64 && n_ent > 1) ? ent[1] : e_cur0;
      for (int j = 0; j < n_steps; ++j) {
        const int sk = j % 3, sv = j & 1;
        const int kb0 = e_cur0 >> 2, kb1 = e_cur1 >> 2;
        if (j + 1 < n_steps) {   // next step's entries: read now, used one step later
          const int i0 = (BS == 128) ? j + 1 : 2 * j + 2;
          e_cur0 = ent[i0];
          e_cur1 = (BS == 64) ? ent[min(i0 + 1, n_ent - 1)] : e_cur0;
        }
        if (j >= 3) ok = mbar_wait(bars + B_KE + sk, ((j / 3) - 1) & 1, a.error_word, 21);
        if (!ok) break;
        mbar_expect_tx(bars + B_KF + sk, kTile);
        tma_load_rows<D, BS>(sK + sk * kTile, &tm_k, bars + B_KF + sk, 0, kb0 * BS, hk, b);
        if (BS == 64) tma_load_rows<D, BS>(sK + sk * kTile, &tm_k, bars + B_KF + sk, 1, kb1 * BS, hk, b);
        nk = j + 1;
        if (j >= 2) ok = mbar_wait(bars + B_VE + sv, ((j / 2) - 1) & 1, a.error_word, 22);
        if (!ok) break;
        mbar_expect_tx(bars + B_VF + sv, kTile);
        tma_load_rows<D, BS>(sV + sv * kTile, &tm_v, bars + B_VF + sv, 0, kb0 * BS, hk, b);
        if (BS == 64) tma_load_rows<D, BS>(sV + sv * kTile, &tm_v, bars + B_VF + sv, 1, kb1 * BS, hk, b);
        nv = j + 1;
      }
      // Before leaving, make sure every copy this thread started has landed (they all have
      // when the kernel ran normally; after a failed wait this keeps shared memory ours).
      mbar_wait(bars + B_FIX, 0, a.error_word, 26);
      for (int j = max(nk - 3, 0); j < nk; ++j) mbar_wait(bars + B_KF + j % 3, (j / 3) & 1, a.error_word, 27);
      for (int j = max(nv - 2, 0); j < nv; ++j) mbar_wait(bars + B_VF + (j & 1), (j / 2) & 1, a.error_word, 28);
    }
  } else if (warp == kDqMmaWarpA) {
    // ------------------------------ MMA issuer A: S and dQ ---------------------------------
    {
      // The whole warp runs the loop (so that addresses and descriptors stay warp-uniform values);
      // one elected lane issues.
      const bool lead = elect_one();
      constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, 0, 0);
      constexpr uint32_t idesc_dq = make_idesc_bf16(128, D, 0, 1);
      const uint32_t hi = desc_hi(1024);
      const uint32_t q_lo = desc_lo(smem_u32(sQ), 16), k_lo = desc_lo(smem_u32(sK), 16);
      const uint32_t k_mn_lo = desc_lo(smem_u32(sK), BwdTile<D>::kBox);   // K tile as an MN-major operand
      bool ok = mbar_wait(bars + B_FIX, 0, a.error_word, 23);
      auto issue_s = [&](int j) {
        const int sk = j % 3;
        ok = ok && mbar_wait(bars + B_KF + sk, (j / 3) & 1, a.error_word, 24);
        if (ok) {
          tc_fence_after();
          const uint32_t b_lo = k_lo + sk * (kTile >> 4), d_s = tmem + kColS + (j & 1) * 128;
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            constexpr int kB = BwdTile<D>::kBox >> 4;
            const uint32_t off = (k >> 2) * kB + (k & 3) * 2;          // (bytes >> 4) of K slice k
            if (lead) mma_ss2(d_s, q_lo + off, b_lo + off, hi, idesc_s, k > 0);
          }
        }
        if (lead) mma_commit(bars + B_SF + (j & 1));
      };
#pragma unroll 1
      for (int j = -2; j < n_steps; ++j) {   // steps -2 and -1 only issue S(0) and S(1)
        if (j >= 0) {
          ok = ok && mbar_wait(bars + B_DSF, j & 1, a.error_word, 29);
          if (ok) {
            tc_fence_after();
            const uint32_t b_lo = k_mn_lo + (j % 3) * (kTile >> 4), a_t = tmem + kColS + (j & 1) * 128;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              if (lead) mma_ts2(tmem + kColDQ, a_t + (kk >> 1) * kDqCols + (kk & 1) * 8, b_lo + kk * (2048 >> 4), hi, idesc_dq,
                      (j > 0) || (kk > 0));
          }
          if (lead) mma_commit(bars + B_KE + j % 3);
        }
        if (j + 2 < n_steps) issue_s(j + 2);
      }
      if (lead) { mma_commit(bars + B_DONE); mma_commit(bars + B_DRAIN); }
      mbar_wait(bars + B_DRAIN, 0, a.error_word, 30);   // nothing of ours is still running at exit
    }
  } else if (warp == kDqMmaWarpB) {
    // ------------------------------ MMA issuer B: dP ---------------------------------------
    {
      const bool lead = elect_one();
      constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, 0, 0);
      const uint32_t hi = desc_hi(1024);
      const uint32_t do_lo = desc_lo(smem_u32(sDO), 16), v_lo = desc_lo(smem_u32(sV), 16);
      bool ok = mbar_wait(bars + B_FIX, 0, a.error_word, 35);
#pragma unroll 1
      for (int j = 0; j < n_steps; ++j) {
        const int sv = j & 1;
        if (j > 0) ok = ok && mbar_wait(bars + B_DPR, (j - 1) & 1, a.error_word, 34);   // dP(j-1) was read
        ok = ok && mbar_wait(bars + B_VF + sv, (j / 2) & 1, a.error_word, 25);
        if (ok) {
          tc_fence_after();
          const uint32_t b_lo = v_lo + sv * (kTile >> 4);
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            constexpr int kB = BwdTile<D>::kBox >> 4;
            const uint32_t off = (k >> 2) * kB + (k & 3) * 2;
            if (lead) mma_ss2(tmem + kColDP, do_lo + off, b_lo + off, hi, idesc_s, k > 0);
          }
        }
        if (lead) { mma_commit(bars + B_DPF); mma_commit(bars + B_VE + sv); }
      }
      if (lead) mma_commit(bars + B_DRAIN + 1);
      mbar_wait(bars + B_DRAIN + 1, 0, a.error_word, 36);
    }
  } else {
    // ------------------------------ element-wise warps ------------------------------------
    constexpr int C = kDqCols;
    const int g = warp >> 2;                                // column group of C columns
    const int r = (warp & 3) * 32 + lane;                   // query row in the tile == TMEM lane
    const int qi = row0 + r;
    const int member = (R == 1) ? 0 : (r / BS);
    const uint32_t lane_addr = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    float nlse2 = 0.f, ndlt = 0.f;   // -LSE2 and -delta of my row
    if (qi < a.L) {
      const int64_t row = (static_cast<int64_t>(b) * a.Hq + h) * a.Lp + qi;
      nlse2 = a.stat[row];
      ndlt = a.stat[a.stat_plane + row];
    }
    const int dstart = (a.doc_start && qi < a.L) ? a.doc_start[static_cast<int64_t>(b) * a.L + qi] : 0;   // start of my document
    // entry of the step: read one step ahead so that the load is off the critical path
    auto entry_of = [&](int j, bool& have) {
      int e = (BS == 128) ? j : 2 * j + (g >> 1);
      have = e < n_ent;
      return ent[min(e, n_ent - 1)];
    };
    bool have = false, have_next = false;
    int entry = n_steps > 0 ? entry_of(0, have) : 0;
    bool ok = true;
#pragma unroll 1
    for (int j = 0; j < n_steps; ++j) {
      const int entry_next = (j + 1 < n_steps) ? entry_of(j + 1, have_next) : 0;
      // which keys do my C columns hold, and how many of them may this row see
      const int key0 = (entry >> 2) * BS + (BS == 128 ? C * g : C * (g & 1));
      const bool on = have && ((entry >> member) & 1);
      const int lim = on ? min(max(qi - key0 + 1, 0), C) : 0;   // columns lo <= c < lim are visible
      const int lo_abs = (a.exact_w > 0 && (entry >> 2) >= a.ns) ? max(dstart, qi - a.exact_w + 1) : dstart;
      const int lo = min(max(lo_abs - key0, 0), C);
      const uint32_t s_addr = lane_addr + kColS + (j & 1) * 128 + g * C;

      ok = mbar_wait(bars + B_SF + (j & 1), (j >> 1) & 1, a.error_word, 31);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      float p[C];
      {
        uint32_t sreg[C];
        tmem_ld32(s_addr, sreg);
        tmem_ld_wait();
        if (__any_sync(0xffffffffu, lim < C || lo > 0)) {
#pragma unroll
          for (int c = 0; c < C; ++c) {
            const float v = fast_exp2(fmaf(__uint_as_float(sreg[c]), a.scale_log2, nlse2));
            p[c] = (c < lim && c >= lo) ? v : 0.f;
          }
        } else {
#pragma unroll
          for (int c = 0; c < C; ++c) p[c] = fast_exp2(fmaf(__uint_as_float(sreg[c]), a.scale_log2, nlse2));
        }
      }
      ok = mbar_wait(bars + B_DPF, j & 1, a.error_word, 32);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t dsreg[C / 2];
      {
        uint32_t dreg[C];
        tmem_ld32(lane_addr + kColDP + g * C, dreg);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + B_DPR);   // the dP columns may be overwritten
#pragma unroll
        for (int x = 0; x < C; x += 2)
          dsreg[x >> 1] = pack_bf16(p[x] * (__uint_as_float(dreg[x]) + ndlt),
                                    p[x + 1] * (__uint_as_float(dreg[x + 1]) + ndlt));
      }
      tmem_st16(s_addr, dsreg);   // dS over my own S columns
      ew_publish(bars + B_DSF);
      entry = entry_next;
      have = have_next;
    }
    // ---- epilogue: dQ * scale -> bf16 -------------------------------------------------------
    if (ok && n_steps > 0) {
      ok = mbar_wait(bars + B_DONE, 0, a.error_word, 33);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      if (g * 64 < D) {                            // warp-uniform: warp group g takes 64 output columns
        __nv_bfloat16* base = a.out0 + b * a.s0[0] + h * a.s0[1] + g * 64;
        if (n_steps > 0) {
          // through the K ring (every tile loaded into it has been consumed): whole rows per store instruction;
          // rows past L take part in the loads only
          const int q_first = qi - lane;
          store_acc_64cols(lane_addr + kColDQ + g * 64, smem + SM::oA + warp * 4096, a.scale, [&](int r2) -> __nv_bfloat16* {
            return q_first + r2 < a.L ? base + static_cast<int64_t>(q_first + r2) * a.s0[2] : nullptr;
          });
        } else if (qi < a.L) {
#pragma unroll
          for (int x = 0; x < 64; x += 8) *reinterpret_cast<uint4*>(base + static_cast<int64_t>(qi) * a.s0[2] + x) = make_uint4(0, 0, 0, 0);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kDqMmaWarpA) tmem_dealloc(tmem, 512);
}

// ============================== dK / dV pass ==================================================
// Items = (query head of the group, entry of the tile's CSC schedule) in a fixed order; a step
// streams 128 query rows (one item with 128-token blocks, two with 64-token blocks) and is
// worked in two half-steps of 64 queries.  TMEM columns: S^T of the even / odd half-step at
// 0 / 64 (P^T written as bf16 over it), dP^T at 128 / 192 (dS^T over it), dV at 256, dK at 384:
// both score tiles are double-buffered, so the S^T of the next half-step is computed while the
// exponentials of this one are evaluated.  Sixteen element-wise warps in two teams of eight: team t
// works the half-steps t, t + 2, ... (the t-th half of every step; its threads take 32 of the 64
// streamed queries each), so that on every scheduler partition two warps are in the arithmetic of one
// half-step while the other two sit in the loads, stores, fences and barrier round trips of the next
// -- with all sixteen warps on the same half-step those latencies were paid one after the other and
// the element-wise path, not the tensor pipe, set the pace.  Two issuing threads on different
// scheduler partitions: thread A issues S^T and dV (dV reads P^T from the S^T columns, so the S^T
// that overwrites them follows it in the same queue), thread B issues dP^T and dK likewise.
constexpr int kKvEwWarps = 16;
constexpr int kKvTeamWarps = kKvEwWarps / 2;
constexpr int kKvTmaWarp = kKvEwWarps, kKvMmaWarpA = kKvEwWarps + 1, kKvMmaWarpB = kKvEwWarps + 2;
constexpr int kKvThreads = (kKvEwWarps + 3) * 32;
constexpr int kKvHalf = 64;                                // queries of a half-step
constexpr int kKvNB = 128 / kKvHalf;                       // half-steps per step = score buffers in rotation = teams
constexpr int kKvCols = kKvHalf / (kKvTeamWarps / 4);      // queries of a half-step per element-wise thread

// kSpill: the pass also writes dS^T (bf16) of every half-step to global memory (BwdArgs::ds_buf), so
// that the dQ pass is one product per step, dQ += dS K, instead of recomputing S and dP
// (bwd_dq_from_ds_kernel).  Every element-wise thread stores the 64 bytes it holds (32 queries of its
// key) straight from its registers: in the tile layout described at BwdArgs::ds_buf a warp's store
// instruction covers 512 contiguous bytes.  (Staging the tiles in shared memory for a TMA store cost
// a shared-memory ring stage of Q, a proxy fence and two barrier round trips per half-step; storing
// rows of a [key][query] layout from registers touched 32 separate cache lines per instruction.)
template <int D, int BS, bool kSpill>
__global__ void __launch_bounds__(kKvThreads, 1)
bwd_dkdv_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do, const BwdArgs a) {
  using SM = BwdSmem<D, BS>;
  constexpr int kQS = SM::kAStages;
  constexpr int R = 128 / BS;
  constexpr uint32_t kColS = 0, kColDP = 128, kColDV = 256, kColDK = 384;
  constexpr int kTile = SM::kTile;
  enum { B_FIX = 0, B_QF = 1, B_QE = 4, B_OF = 7, B_OE = 9, B_SF = 11, B_DPF = 13, B_PF = 15, B_DSF = 17,
         B_DONE = 19, B_DRAIN = 20, B_STF = 22, B_STE = 24, B_COUNT = 26 };

  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::oBar);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);
  int32_t* sEnt = reinterpret_cast<int32_t*>(bars + B_COUNT + 1);   // [2][2]: entries of a step's items
  int64_t* sTile = reinterpret_cast<int64_t*>(bars + B_COUNT + 3);  // [2][2][2]: dS tile of (half-step, member) of a step (kSpill)
  static_assert((B_COUNT + 3) * 8 + 64 <= SM::kBarBytes, "barrier area too small");
  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);   // same value, known to be warp-uniform
  if ((smem_u32(smem) & 1023u) != 0) {
    if (tid == 0) atomicCAS(a.error_word, 0u, (2u << 24) | 10u);
    return;
  }
  if (!lists_match(a.error_word, a.expect_fp, a.expect_fp2, 10u)) return;
  uint8_t* sK = smem + SM::oFix0;
  uint8_t* sV = smem + SM::oFix1;
  uint8_t* sQ = smem + SM::oA;     // [3]
  uint8_t* sDO = smem + SM::oB;    // [2]
  float* sStat = reinterpret_cast<float*>(smem + SM::oStat);   // [2 stages][-LSE2 | -delta][128 queries]

  // has a wait already given up in this call?  (read now, so that it travels with the schedule loads below)
  unsigned int abort_word = 0;
  if (tid == 0) abort_word = *reinterpret_cast<volatile unsigned int*>(a.error_word);
  int cta_x, cta_y;   // (batch, kv head) and launch rank of this CTA's kv tile
  cta_coords2(static_cast<long long>(blockIdx.y) * gridDim.x + blockIdx.x, gridDim.x, gridDim.y, a.head_group, a.n_long, cta_x, cta_y);
  const int tile = checked(a.order[cta_y], 0, a.n_tiles - 1, a.error_word, 120);
  const int b = cta_x / a.Hkv, hk = cta_x % a.Hkv;
  const int ent_off = checked(a.tile_off[tile], 0, a.n_list, a.error_word, 121);
  const int n_ent = checked(a.tile_cnt[tile], 0, a.n_list - ent_off, a.error_word, 122);
  const int32_t* ent = a.tile_ent + ent_off;
  // key blocks of the tile's members (with 64-token blocks the two members need not be neighbours)
  const int kb_a = checked(a.tile_cols[R * tile], 0, a.nB - 1, a.error_word, 123);
  const int kb_b = (R == 2) ? checked(a.tile_cols[R * tile + 1], -1, a.nB - 1, a.error_word, 124) : -1;
  const int n_items = n_ent * a.G;
  const int n_hs = (BS == 128) ? kKvNB * n_items : (kKvNB == 2 ? n_items : (n_items + 1) / 2);    // half-steps
  const int n_steps = (n_hs + kKvNB - 1) / kKvNB;          // 128-row tiles streamed
  // half-step hs belongs to step hs / kKvNB and is its last one when:
  auto closes_step = [&](int hs) { return (hs % kKvNB == kKvNB - 1) || hs == n_hs - 1; };


  if (tid == 0) {
    mbar_init(bars + B_FIX, 1);
    for (int i = 0; i < 3; ++i) { mbar_init(bars + B_QF + i, 1); mbar_init(bars + B_QE + i, 1); }   // (kQS of them are used)
    for (int i = 0; i < 2; ++i) {
      mbar_init(bars + B_OF + i, 1);
      mbar_init(bars + B_OE + i, 2);      // dP^T (thread B) and dV (thread A) both read the dO tile
      mbar_init(bars + B_SF + i, 1);
      mbar_init(bars + B_DPF + i, 1);
      mbar_init(bars + B_PF + i, kKvTeamWarps);
      mbar_init(bars + B_DSF + i, kKvTeamWarps);
      mbar_init(bars + B_DRAIN + i, 1);
      mbar_init(bars + B_STF + i, 1);
      mbar_init(bars + B_STE + i, kKvEwWarps);   // every warp once per step, after its team's half
    }
    mbar_init(bars + B_DONE, 2);          // the last dV and the last dK
    mbar_fence_init();
    tmem_slot[1] = abort_word;
  }
  if (warp == kKvMmaWarpA) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  if (tmem_slot[1] != 0) {   // after a failed wait the rest of the grid does nothing: the call ends in seconds, not minutes
    if (warp == kKvMmaWarpA) tmem_dealloc(tmem, 512);
    return;
  }

  if (warp == kKvTmaWarp) {
    // ------------------------------ TMA producer ------------------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v); tma_prefetch_desc(&tm_do);
      mbar_expect_tx(bars + B_FIX, 2 * kTile);
      tma_load_rows<D, BS>(sK, &tm_k, bars + B_FIX, 0, kb_a * BS, hk, b);
      tma_load_rows<D, BS>(sV, &tm_v, bars + B_FIX, 0, kb_a * BS, hk, b);
      if (R == 2) {   // second member (a missing one re-loads the first; its rows are never stored)
        tma_load_rows<D, BS>(sK, &tm_k, bars + B_FIX, 1, (kb_b >= 0 ? kb_b : kb_a) * BS, hk, b);
        tma_load_rows<D, BS>(sV, &tm_v, bars + B_FIX, 1, (kb_b >= 0 ? kb_b : kb_a) * BS, hk, b);
      }
      // Besides the tiles, each step gets the softmax statistics of its 128 queries and the
      // schedule entries of its items, so that the element-wise warps read neither global memory
      // nor the schedule.
      bool ok = true;
      int nq = 0, no = 0, nst = 0;   // loads started
      // Items: the tile's entries in order, and for every entry the query heads of the group one after the
      // other.  The order is ascending (from the tile's own diagonal upwards) where the tiles of a head take
      // about the same time, and DESCENDING, from the last query block down, where they do not (a.descending:
      // strided combs, full causal attention): every tile of a comb column needs every later row of every
      // head, and walking down from the last row the kv tiles of a kv head that run at one time stream the
      // same Q / dO tiles at the same time, whatever their own first row is, and share them in the L2 (cfg 4:
      // 127 -> 92 GB of DRAM reads in the pass; its operands are 5 GB, but tiles that start later are on
      // rows of their own again).
      const int e_step = a.descending ? -1 : 1;
      int grp = 0, e = a.descending ? n_ent - 1 : 0;    // (query head within the group, entry) of the next item
      // positions, in the column lists, of the members' next blocks: the entries that carry a member's bit
      // are that column's query blocks in the same order
      auto col_first = [&](int kb) { return (!kSpill || kb < 0) ? 0 : (a.descending ? a.col_ptr[kb + 1] - 1 : a.col_ptr[kb]); };
      int pos_a = col_first(kb_a), pos_b = col_first(kb_b);
      auto next_item = [&](int& hq, int& qrow, int& entry, int64_t& ta, int64_t& tb) {
        entry = ent[e];
        hq = hk * a.G + grp;
        qrow = checked(entry >> 2, 0, a.nB - 1, a.error_word, 125) * BS;   // (also the address of the item's statistics)
        const int64_t head_base = (static_cast<int64_t>(b) * a.Hq + hq) * a.ds_nnz;
        ta = (head_base + pos_a) * (BS / 64);
        tb = (head_base + pos_b) * (BS / 64);
        if (++grp == a.G) { grp = 0; pos_a += e_step * (entry & 1); pos_b += e_step * ((entry >> 1) & 1); e += e_step; }
      };
      // Each load is started as soon as its ring slot is free, in the order in which the slots come
      // free: dO of step j (its slot is released when the dV and dP^T products of step j - 2 are done),
      // the statistics of step j (released by the element-wise warps at the end of step j - 2), then Q
      // of step j + 1 (three stages: the slot of step j - 2, released by its dK product).  Q is the first
      // operand a step needs -- S^T of step j + 1 is issued early in step j -- hence the step of lead.
      // CTAs start in launch order as SMs come free, and the tiles of a pattern's band take the same time:
      // the CTA `ahead` places after this one starts about when this one ends, on some SM.  Its K and V
      // tiles are first touched by it and would come from HBM at the head of its critical path; asked for
      // a few steps before this tile ends (earlier, the stream of dS stores has pushed them out of the L2
      // again by the time they are wanted: + 25 % of DRAM reads in the profile), they are in the L2 by then.
      // A hint only: nothing waits for it and a wrong guess costs two tile reads.
      auto prefetch_successor = [&]() {
        if (a.ahead <= 0) return;
        const int64_t w = static_cast<int64_t>(blockIdx.y) * gridDim.x + blockIdx.x + a.ahead;
        if (w >= static_cast<int64_t>(gridDim.x) * gridDim.y) return;
        int x2, y2;
        cta_coords2(w, gridDim.x, gridDim.y, a.head_group, a.n_long, x2, y2);
        const int t2 = checked(a.order[y2], 0, a.n_tiles - 1, a.error_word, 126);
        const int b2 = x2 / a.Hkv, hk2 = x2 % a.Hkv;
#pragma unroll
        for (int m = 0; m < R; ++m) {
          const int kb2 = checked(a.tile_cols[R * t2 + m], -1, a.nB - 1, a.error_word, 127);
          if (kb2 < 0) continue;
#pragma unroll
          for (int x = 0; x < D / 64; ++x) {
            tma_prefetch_l2_4d(&tm_k, x * 64, kb2 * BS, hk2, b2);
            tma_prefetch_l2_4d(&tm_v, x * 64, kb2 * BS, hk2, b2);
          }
        }
      };
      struct Item { int h, r, e; int64_t ta, tb; };
      auto step_items = [&](int j, Item& i0, Item& i1) {
        next_item(i0.h, i0.r, i0.e, i0.ta, i0.tb);
        i1 = i0; i1.e = i0.e & ~3; i1.ta = i0.ta + 1;           // a missing second item repeats the first block, as nobody's member
        if (BS == 64 && 2 * j + 1 < n_items) next_item(i1.h, i1.r, i1.e, i1.ta, i1.tb);
      };
      auto load_q = [&](int j, const Item& i0, const Item& i1) {
        const int sq = j % kQS;
        if (j >= kQS) ok = mbar_wait(bars + B_QE + sq, ((j / kQS) - 1) & 1, a.error_word, 11);
        if (!ok) return;
        mbar_expect_tx(bars + B_QF + sq, kTile);
        tma_load_rows<D, BS>(sQ + sq * kTile, &tm_q, bars + B_QF + sq, 0, i0.r, i0.h, b);
        if (BS == 64) tma_load_rows<D, BS>(sQ + sq * kTile, &tm_q, bars + B_QF + sq, 1, i1.r, i1.h, b);
        nq = j + 1;
      };
      Item c0, c1, n0, n1;   // items of step j and of step j + 1
      if (n_steps > 0) { step_items(0, n0, n1); load_q(0, n0, n1); }
      for (int j = 0; j < n_steps && ok; ++j) {
        const int so = j & 1;
        c0 = n0; c1 = n1;
        if (j + 1 < n_steps) step_items(j + 1, n0, n1);
        if (j >= 2) ok = mbar_wait(bars + B_OE + so, ((j / 2) - 1) & 1, a.error_word, 12);
        if (!ok) break;
        mbar_expect_tx(bars + B_OF + so, kTile);
        tma_load_rows<D, BS>(sDO + so * kTile, &tm_do, bars + B_OF + so, 0, c0.r, c0.h, b);
        if (BS == 64) tma_load_rows<D, BS>(sDO + so * kTile, &tm_do, bars + B_OF + so, 1, c1.r, c1.h, b);
        no = j + 1;
        if (j >= 2) ok = mbar_wait(bars + B_STE + so, ((j / 2) - 1) & 1, a.error_word, 40);
        if (!ok) break;
        sEnt[so * 2] = c0.e;
        sEnt[so * 2 + 1] = c1.e;
        if (kSpill) {   // (128-token blocks: the two halves of the one item are neighbouring tiles)
          sTile[so * 4] = c0.ta; sTile[so * 4 + 1] = c0.tb;
          sTile[so * 4 + 2] = c1.ta; sTile[so * 4 + 3] = c1.tb;
        }
        mbar_expect_tx(bars + B_STF + so, 2 * 128 * 4);         // (release: publishes the entries as well)
        {
          const float* st0 = a.stat + (static_cast<int64_t>(b) * a.Hq + c0.h) * a.Lp + c0.r;
          const float* st1 = a.stat + (static_cast<int64_t>(b) * a.Hq + c1.h) * a.Lp + c1.r;
#pragma unroll
          for (int pl = 0; pl < 2; ++pl) {
            float* dst = sStat + (so * 2 + pl) * 128;
            if (BS == 128) {
              bulk_load(dst, st0 + pl * a.stat_plane, 128 * 4, bars + B_STF + so);
            } else {
              bulk_load(dst, st0 + pl * a.stat_plane, 64 * 4, bars + B_STF + so);
              bulk_load(dst + 64, st1 + pl * a.stat_plane, 64 * 4, bars + B_STF + so);
            }
          }
        }
        nst = j + 1;
        if (j + 1 < n_steps) load_q(j + 1, n0, n1);
        if (j + 1 == (n_steps > 8 ? n_steps - 8 : 1)) prefetch_successor();   // a few steps before this tile ends
      }
      mbar_wait(bars + B_FIX, 0, a.error_word, 16);
      for (int j = max(nq - kQS, 0); j < nq; ++j) mbar_wait(bars + B_QF + j % kQS, (j / kQS) & 1, a.error_word, 17);
      for (int j = max(no - 2, 0); j < no; ++j) mbar_wait(bars + B_OF + (j & 1), (j / 2) & 1, a.error_word, 18);
      for (int j = max(nst - 2, 0); j < nst; ++j) mbar_wait(bars + B_STF + (j & 1), (j / 2) & 1, a.error_word, 41);
    }
  } else if (warp == kKvMmaWarpA) {
    // ------------------------------ MMA issuer A: S^T and dV -------------------------------
    {
      // The whole warp runs the loop (so that addresses and descriptors stay warp-uniform values);
      // one elected lane issues.
      const bool lead = elect_one();
      constexpr uint32_t idesc_st = make_idesc_bf16(128, kKvHalf, 0, 0);   // S^T: N = queries of a half-step
      constexpr uint32_t idesc_acc = make_idesc_bf16(128, D, 0, 1);        // dV: B = dO, MN-major
      constexpr uint32_t kHalfRows = (kKvHalf * 128) >> 4;                 // 64 rows of a box, in 16-byte units
      const uint32_t hi = desc_hi(1024);
      const uint32_t k_lo = desc_lo(smem_u32(sK), 16), q_lo = desc_lo(smem_u32(sQ), 16);
      const uint32_t do_mn_lo = desc_lo(smem_u32(sDO), BwdTile<D>::kBox);
      bool ok = mbar_wait(bars + B_FIX, 0, a.error_word, 13);
#pragma unroll 1
      for (int hs = -kKvNB; hs < n_hs; ++hs) {   // the first kKvNB rounds only issue S^T
        if (hs >= 0) {
          const int j = hs / kKvNB, half = hs % kKvNB, so = j & 1;
          if (half == 0) ok = ok && mbar_wait(bars + B_OF + so, (j / 2) & 1, a.error_word, 19);
          ok = ok && mbar_wait(bars + B_PF + half, j & 1, a.error_word, 9);
          if (ok) {
            tc_fence_after();
            const uint32_t b_lo = do_mn_lo + so * (kTile >> 4) + half * (kKvHalf / 16) * (2048 >> 4);
            const uint32_t a_t = tmem + kColS + half * kKvHalf;
#pragma unroll
            for (int kk = 0; kk < kKvHalf / 16; ++kk)
              if (lead) mma_ts2(tmem + kColDV, a_t + (kk * 16 / kKvCols) * kKvCols + (kk * 16 % kKvCols) / 2, b_lo + kk * (2048 >> 4), hi, idesc_acc, (hs > 0) || (kk > 0));
          }
          if (lead && closes_step(hs)) mma_commit(bars + B_OE + so);
        }
        const int hn = hs + kKvNB;
        if (hn < n_hs) {
          const int j = hn / kKvNB, half = hn % kKvNB, sq = j % kQS;
          if (half == 0) ok = ok && mbar_wait(bars + B_QF + sq, (j / kQS) & 1, a.error_word, 14);
          if (ok) {
            tc_fence_after();
            const uint32_t b_lo = q_lo + sq * (kTile >> 4) + half * kHalfRows;
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
              constexpr int kB = BwdTile<D>::kBox >> 4;
              const uint32_t off = (k >> 2) * kB + (k & 3) * 2;
              if (lead) mma_ss2(tmem + kColS + half * kKvHalf, k_lo + off, b_lo + off, hi, idesc_st, k > 0);
            }
          }
          if (lead) mma_commit(bars + B_SF + half);
        }
      }
      if (lead) { mma_commit(bars + B_DONE); mma_commit(bars + B_DRAIN); }
      mbar_wait(bars + B_DRAIN, 0, a.error_word, 8);
    }
  } else if (warp == kKvMmaWarpB) {
    // ------------------------------ MMA issuer B: dP^T and dK ------------------------------
    {
      const bool lead = elect_one();
      constexpr uint32_t idesc_st = make_idesc_bf16(128, kKvHalf, 0, 0);
      constexpr uint32_t idesc_acc = make_idesc_bf16(128, D, 0, 1);        // dK: B = Q, MN-major
      constexpr uint32_t kHalfRows = (kKvHalf * 128) >> 4;
      const uint32_t hi = desc_hi(1024);
      const uint32_t v_lo = desc_lo(smem_u32(sV), 16), do_lo = desc_lo(smem_u32(sDO), 16);
      const uint32_t q_mn_lo = desc_lo(smem_u32(sQ), BwdTile<D>::kBox);
      bool ok = mbar_wait(bars + B_FIX, 0, a.error_word, 5);
#pragma unroll 1
      for (int hs = -kKvNB; hs < n_hs; ++hs) {   // the first kKvNB rounds only issue dP^T
        if (hs >= 0) {
          const int j = hs / kKvNB, half = hs % kKvNB, sq = j % kQS;
          ok = ok && mbar_wait(bars + B_DSF + half, j & 1, a.error_word, 15);
          if (ok) {
            tc_fence_after();
            const uint32_t b_lo = q_mn_lo + sq * (kTile >> 4) + half * (kKvHalf / 16) * (2048 >> 4);
            const uint32_t a_t = tmem + kColDP + half * kKvHalf;
#pragma unroll
            for (int kk = 0; kk < kKvHalf / 16; ++kk)
              if (lead) mma_ts2(tmem + kColDK, a_t + (kk * 16 / kKvCols) * kKvCols + (kk * 16 % kKvCols) / 2, b_lo + kk * (2048 >> 4), hi, idesc_acc, (hs > 0) || (kk > 0));
          }
          if (lead && closes_step(hs)) mma_commit(bars + B_QE + sq);
        }
        const int hn = hs + kKvNB;
        if (hn < n_hs) {
          const int j = hn / kKvNB, half = hn % kKvNB, so = j & 1;
          if (half == 0) ok = ok && mbar_wait(bars + B_OF + so, (j / 2) & 1, a.error_word, 6);
          if (ok) {
            tc_fence_after();
            const uint32_t b_lo = do_lo + so * (kTile >> 4) + half * kHalfRows;
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
              constexpr int kB = BwdTile<D>::kBox >> 4;
              const uint32_t off = (k >> 2) * kB + (k & 3) * 2;
              if (lead) mma_ss2(tmem + kColDP + half * kKvHalf, v_lo + off, b_lo + off, hi, idesc_st, k > 0);
            }
          }
          if (lead) {
            mma_commit(bars + B_DPF + half);
            if (closes_step(hn)) mma_commit(bars + B_OE + so);
          }
        }
      }
      if (lead) { mma_commit(bars + B_DONE); mma_commit(bars + B_DRAIN + 1); }
      mbar_wait(bars + B_DRAIN + 1, 0, a.error_word, 7);
    }
  } else {
    // ------------------------------ element-wise warps ------------------------------------
    constexpr int C = kKvCols;
    const int half = warp / kKvTeamWarps;                   // team = the half of every step it works
    const int g = (warp >> 2) % (kKvTeamWarps / 4);         // group of C streamed queries within the half-step
    const int r = (warp & 3) * 32 + lane;                   // key row in the tile == TMEM lane
    const int member = (R == 1) ? 0 : (r / BS);
    const int kb_mine = (R == 2 && member) ? kb_b : kb_a;
    const int kj = kb_mine * BS + (R == 2 ? (r & (BS - 1)) : r);   // this thread's key (kb_mine < 0: none)
    // end of my key's document: queries from there on do not see it (no documents: the end of the sequence,
    // which also keeps the rows a partial last block lacks out of the sums)
    const int dend = (a.doc_end && kb_mine >= 0 && kj < a.L) ? a.doc_end[static_cast<int64_t>(b) * a.L + kj] : a.L;
    const uint32_t lane_addr = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const uint64_t scale2 = f32x2(a.scale_log2, a.scale_log2);
    uint64_t evict_first = 0;
    if (kSpill) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(evict_first));
    bool ok = true;
#pragma unroll 1
    for (int hs = half; hs < n_hs; hs += kKvNB) {
      const int j = hs / kKvNB;
      ok = mbar_wait(bars + B_STF + (j & 1), (j >> 1) & 1, a.error_word, 4);   // statistics and entries of step j
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      // -LSE2 and -delta of my C queries, four to a load
      const float4* st_l = reinterpret_cast<const float4*>(sStat + (j & 1) * 256 + half * kKvHalf + g * C);
      const float4* st_d = st_l + 128 / 4;
      // the queries my columns hold, and from which of them on this key may be seen
      const int col0 = half * kKvHalf + g * C;                 // my first column within the step's 128 queries
      const int entry = sEnt[(j & 1) * 2 + (BS == 64 ? col0 / 64 : 0)];
      const int q0 = (entry >> 2) * BS + (BS == 128 ? col0 : col0 % 64);
      const bool on = (entry >> member) & 1;
      const int xmin = on ? min(max(kj - q0, 0), C) : C;      // columns xmin <= c < xmax are visible
      const int hi_abs = (a.exact_w > 0 && kb_mine >= a.ns) ? min(dend, kj + a.exact_w) : dend;   // first query that no longer sees me
      const int xmax = min(max(hi_abs - q0, 0), C);
      const uint32_t s_addr = lane_addr + kColS + half * kKvHalf + g * C;
      const uint32_t dp_addr = lane_addr + kColDP + half * kKvHalf + g * C;

      ok = mbar_wait(bars + B_SF + half, j & 1, a.error_word, 1);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      float p[C];
      {
        uint32_t sreg[C];
#pragma unroll
        for (int c = 0; c < C; c += 32) tmem_ld32(s_addr + c, sreg + c);
        tmem_ld_wait();
        const bool masked = __any_sync(0xffffffffu, xmin > 0 || xmax < C);
#pragma unroll
        for (int c = 0; c < C; c += 4) {
          const float4 l4 = st_l[c >> 2];
          float x0, x1, x2, x3;
          f32x2_split(fma_f32x2(f32x2(__uint_as_float(sreg[c]), __uint_as_float(sreg[c + 1])), scale2,
                                f32x2(l4.x, l4.y)), x0, x1);
          f32x2_split(fma_f32x2(f32x2(__uint_as_float(sreg[c + 2]), __uint_as_float(sreg[c + 3])), scale2,
                                f32x2(l4.z, l4.w)), x2, x3);
          // (all on the exponential unit: with the two teams the element-wise warps have slack, and under
          // the power cap the instructions of a polynomial on the FMA pipe cost more than the unit's cycles)
          float v0 = fast_exp2(x0), v1 = fast_exp2(x1), v2 = fast_exp2(x2), v3 = fast_exp2(x3);
          if (masked) {
            v0 = (c >= xmin && c < xmax) ? v0 : 0.f;
            v1 = (c + 1 >= xmin && c + 1 < xmax) ? v1 : 0.f;
            v2 = (c + 2 >= xmin && c + 2 < xmax) ? v2 : 0.f;
            v3 = (c + 3 >= xmin && c + 3 < xmax) ? v3 : 0.f;
          }
          p[c] = v0;
          p[c + 1] = v1;
          p[c + 2] = v2;
          p[c + 3] = v3;
        }
        uint32_t preg[C / 2];
#pragma unroll
        for (int c = 0; c < C; c += 2) preg[c >> 1] = pack_bf16(p[c], p[c + 1]);
        if constexpr (C == 32) tmem_st16(s_addr, preg); else tmem_st32(s_addr, preg);   // P^T over my own S^T columns
        ew_publish(bars + B_PF + half);
      }
      ok = mbar_wait(bars + B_DPF + half, j & 1, a.error_word, 2);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t dsreg[C / 2];
      {
#pragma unroll
        for (int c0 = 0; c0 < C; c0 += 32) {   // 32 columns at a time: their dP^T leaves the registers before the next 32 arrive
          uint32_t dreg[32];
          tmem_ld32(dp_addr + c0, dreg);
          tmem_ld_wait();
#pragma unroll
          for (int y = 0; y < 32; y += 4) {
            const int x = c0 + y;
            const float4 d4 = st_d[x >> 2];
            float d0, d1, d2, d3;
            f32x2_split(mul_f32x2(f32x2(p[x], p[x + 1]),
                                  add_f32x2(f32x2(__uint_as_float(dreg[y]), __uint_as_float(dreg[y + 1])),
                                            f32x2(d4.x, d4.y))), d0, d1);
            f32x2_split(mul_f32x2(f32x2(p[x + 2], p[x + 3]),
                                  add_f32x2(f32x2(__uint_as_float(dreg[y + 2]), __uint_as_float(dreg[y + 3])),
                                            f32x2(d4.z, d4.w))), d2, d3);
            dsreg[x >> 1] = pack_bf16(d0, d1);
            dsreg[(x >> 1) + 1] = pack_bf16(d2, d3);
          }
        }
      }
      if constexpr (C == 32) tmem_st16(dp_addr, dsreg); else tmem_st32(dp_addr, dsreg);   // dS^T over my own dP^T columns
      if constexpr (kSpill) {
        static_assert(!kSpill || ((C == 32 || C == 64) && kKvNB == 2), "the kept tiles are laid out for half-steps of 64 queries");
        // ... and to this half-step's tile in global memory: my C queries are C / 8 16-byte groups of my
        // key.  (Written once, read once by the dQ pass: marked evict-first so that the stream does not
        // push the Q / dO tiles, which every kv tile of a window re-reads, out of the L2.)
        // (a member the entry does not list has no block, hence no tile: its dS is zero and stays unwritten)
        if (on) {
          uint8_t* dst = reinterpret_cast<uint8_t*>(a.ds_buf) + sTile[(j & 1) * 4 + half * 2 + member] * kDsTileBytes<BS> +
                         (C / 8 * g) * (16 * BS) + (r & (BS - 1)) * 16;
#pragma unroll
          for (int i = 0; i < C / 8; ++i)
            asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(dst + i * (16 * BS)),
                         "r"(dsreg[4 * i]), "r"(dsreg[4 * i + 1]), "r"(dsreg[4 * i + 2]), "r"(dsreg[4 * i + 3]), "l"(evict_first) : "memory");
        }
      }
      ew_publish(bars + B_DSF + half);
      __syncwarp();   // this warp is done with the statistics of step j
      if (lane == 0) mbar_arrive(bars + B_STE + (j & 1));
    }
    // ---- epilogue: dV, dK * scale -> bf16 ---------------------------------------------------
    if (ok && n_hs > 0) {
      ok = mbar_wait(bars + B_DONE, 0, a.error_word, 3);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      // The sixteen warps share the output: warp group ge takes 64 columns of one accumulator (dV first, then
      // dK) for its 32 keys.  The rows leave through the Q ring (every load into it has been consumed by the
      // products that are now done), 4 KB per warp, so that the stores cover whole rows (store_acc_64cols).
      constexpr int kParts = D / 64, kGroups = kKvEwWarps / 4;
      const int ge = warp >> 2;
      if (kb_mine >= 0) {
#pragma unroll
        for (int pi = ge; pi < 2 * kParts; pi += kGroups) {      // warp-uniform
          const bool is_dk = pi >= kParts;
          const int part = pi % kParts;
          const int64_t* st = is_dk ? a.s0 : a.s1;
          __nv_bfloat16* base = (is_dk ? a.out0 : a.out1) + b * st[0] + hk * st[1] + part * 64;
          const int64_t row_stride = st[2];
          if (n_hs > 0) {
            const int r_first = (warp & 3) * 32;
            store_acc_64cols(lane_addr + (is_dk ? kColDK : kColDV) + part * 64, sQ + warp * 4096, is_dk ? a.scale : 1.0f,
                             [&](int r2) -> __nv_bfloat16* {
                               const int rr = r_first + r2;
                               const int k2 = kb_mine * BS + (R == 2 ? (rr & (BS - 1)) : rr);   // keys past L take part in the loads only
                               return k2 < a.L ? base + static_cast<int64_t>(k2) * row_stride : nullptr;
                             });
          } else if (kj < a.L) {
#pragma unroll
            for (int x = 0; x < 64; x += 8) *reinterpret_cast<uint4*>(base + static_cast<int64_t>(kj) * row_stride + x) = make_uint4(0, 0, 0, 0);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kKvMmaWarpA) tmem_dealloc(tmem, 512);
}

// ============================== dQ from the kept dS ===========================================
// dQ(128 queries x D) = scale * sum over the kv tiles of the row of dS(128 queries x 128 keys) K(128 keys x D),
// with dS^T read back from the tiles the dK/dV pass left in global memory (per kv tile of the row the two
// tiles of 64 queries x 128 keys, or the four of 64 x 64, that make up the 128 x 128 product, in the
// core-matrix layout described at BwdArgs::ds_buf, copied as they are and used as an un-swizzled operand;
// where the pattern has no block the tile of zeros is read):
// one product per step, no exponentials, nothing recomputed.  The kernel is a plain pipelined
// contraction -- warp 4 loads (a ring of dS^T tile pairs and a ring of K tiles), warp 5 issues, warps
// 0-3 write the result -- and is bound by the HBM reads of dS.
template <int D>
struct DqDsSmem {
  static constexpr int kTile = BwdTile<D>::kBytes;
  static constexpr int kDs2 = 128 * 128 * 2;                   // dS^T of a step: [key half (64-token blocks)][query half][8 queries][keys][8 queries]
  static constexpr int kAStages = (D == 128) ? 3 : 5;          // dS^T comes from HBM: the deeper ring
  static constexpr int kKStages = 3;                           // K comes from the L2
  static constexpr int kStage = 4 * 4096;                      // the epilogue's rows, 4 KB per warp (store_acc_64cols)
  static constexpr int oA = 0;
  static constexpr int oK = kAStages * kDs2;
  static constexpr int oStage = oK + kKStages * kTile;
  static constexpr int oBar = oStage + kStage;
  static constexpr int kTotal = oBar + 256;
};
constexpr int kDq2Threads = 6 * 32;

// One CTA per SM, each working the (head, query tile) items  c, c + gridDim.x, ...  of the launch order (head
// fastest, tiles longest first).  The three roles run through the items on their own: the rings carry on from
// one item to the next and the accumulator alternates between two column ranges, so that the loads and the
// products of an item run while the rows of the one before leave -- with one item per CTA, the 2-4 us between
// an item's last load and the first load of the CTA that followed left the memory system idle for a seventh of
// the pass.
template <int D, int BS>
__global__ void __launch_bounds__(kDq2Threads, 1)
bwd_dq_from_ds_kernel(const __grid_constant__ CUtensorMap tm_k, const BwdArgs a, const int n_heads, const int n_ranks) {
  using SM = DqDsSmem<D>;
  constexpr int kAS = SM::kAStages, kKS = SM::kKStages;
  constexpr int R = 128 / BS;
  constexpr int kTile = SM::kTile;
  enum { B_AF = 0, B_AE = kAS, B_KF = 2 * kAS, B_KE = 2 * kAS + kKS, B_DONE = 2 * kAS + 2 * kKS, B_FREE = B_DONE + 2,
         B_ALL = B_FREE + 2, B_COUNT = B_ALL + 1 };
  static_assert(B_COUNT * 8 + 8 <= 256, "barrier area too small");
  static_assert(SM::kTotal <= 227 * 1024, "shared memory");
  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::oBar);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);
  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
  if ((smem_u32(smem) & 1023u) != 0) {
    if (tid == 0) atomicCAS(a.error_word, 0u, (2u << 24) | 80u);
    return;
  }
  if (!lists_match(a.error_word, a.expect_fp, a.expect_fp2, 80u)) return;
  unsigned int abort_word = 0;
  if (tid == 0) abort_word = *reinterpret_cast<volatile unsigned int*>(a.error_word);
  const long long n_items = static_cast<long long>(n_heads) * n_ranks;
  if (tid == 0) {
    for (int i = 0; i < kAS; ++i) { mbar_init(bars + B_AF + i, 1); mbar_init(bars + B_AE + i, 1); }
    for (int i = 0; i < kKS; ++i) { mbar_init(bars + B_KF + i, 1); mbar_init(bars + B_KE + i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bars + B_DONE + i, 1); mbar_init(bars + B_FREE + i, 4); }
    mbar_init(bars + B_ALL, 1);
    mbar_fence_init();
    tmem_slot[1] = abort_word;
  }
  if (warp == 5) {
    tmem_alloc(tmem_slot, 2 * D);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  if (tmem_slot[1] != 0) {
    if (warp == 5) tmem_dealloc(tmem, 2 * D);
    return;
  }
  // item w of the launch order: (batch entry, head), query tile and its schedule entries
  struct Item { int b, h, t, n_ent; const int32_t* ent; };
  auto item_of = [&](long long w) {
    Item it;
    const int x = static_cast<int>(w % n_heads), y = static_cast<int>(w / n_heads);
    it.b = x / a.Hq; it.h = x % a.Hq;
    it.t = checked(a.order[y], 0, a.n_tiles - 1, a.error_word, 130);   // query tile (128 rows)
    const int ent_off = checked(a.tile_off[R * it.t], 0, a.n_list, a.error_word, 131);
    it.n_ent = checked(a.tile_cnt[it.t], 0, a.n_list - ent_off, a.error_word, 132);
    it.ent = a.tile_ent + kDqEntInts * static_cast<int64_t>(ent_off);   // (kv tile, dS tiles of its quarters)
    return it;
  };
  if (warp == 4) {
    // ------------------------------ TMA producer ------------------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&tm_k);
      uint64_t evict_first;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(evict_first));   // dS tiles are read once
      constexpr int E = kDqEntInts, NT = (BS == 128) ? 2 : 4;   // tiles per step
      const int64_t zero_tile = static_cast<int64_t>(n_heads) * a.ds_nnz * (BS / 64);                // the tile after the last head's
      bool ok = true;
      int g = 0;   // steps loaded so far, over all items: ring slots and barrier phases follow it
      for (long long w = blockIdx.x; w < n_items && ok; w += gridDim.x) {
        const Item it = item_of(w);
        const int hk = it.h / a.G;
        const int64_t head_base = (static_cast<int64_t>(it.b) * a.Hq + it.h) * a.ds_nnz * (BS / 64);
        int e_next[E];
#pragma unroll
        for (int i = 0; i < E; ++i) e_next[i] = it.n_ent > 0 ? it.ent[i] : 0;
        for (int x = 0; x < it.n_ent; ++x) {
          int e_cur[E];
#pragma unroll
          for (int i = 0; i < E; ++i) e_cur[i] = e_next[i];
          const int T = checked(e_cur[0], 0, a.nB - 1, a.error_word, 133);   // (with 64-token blocks T indexes the tiles' column pairs; nB bounds it from above)
          if (x + 1 < it.n_ent) {   // read ahead
#pragma unroll
            for (int i = 0; i < E; ++i) e_next[i] = it.ent[E * (x + 1) + i];
          }
          const int sa = g % kAS, sk = g % kKS;
          if (g >= kAS) ok = mbar_wait(bars + B_AE + sa, ((g / kAS) - 1) & 1, a.error_word, 81);
          if (!ok) break;
          mbar_expect_tx(bars + B_AF + sa, SM::kDs2);
          uint8_t* dA = smem + SM::oA + sa * SM::kDs2;
#pragma unroll
          for (int i = 0; i < NT; ++i) {   // i = 2 * key half + query half: the order of the schedule entry and of the stage
            const int hx = checked(e_cur[1 + i], -1, static_cast<int>(a.ds_nnz * (BS / 64)) - 1, a.error_word, 134);
            const int64_t tile_idx = hx >= 0 ? head_base + hx : zero_tile;
            bulk_load_hint(dA + i * kDsTileBytes<BS>, reinterpret_cast<const uint8_t*>(a.ds_buf) + tile_idx * kDsTileBytes<BS>,
                           kDsTileBytes<BS>, bars + B_AF + sa, evict_first);
          }
          if (g >= kKS) ok = mbar_wait(bars + B_KE + sk, ((g / kKS) - 1) & 1, a.error_word, 86);
          if (!ok) {   // the dS tiles just asked for: let them land before the CTA leaves
            mbar_wait(bars + B_AF + sa, (g / kAS) & 1, a.error_word, 82);
            break;
          }
          mbar_expect_tx(bars + B_KF + sk, kTile);
          uint8_t* dK = smem + SM::oK + sk * kTile;
          if (BS == 128) {
            tma_load_rows<D, 128>(dK, &tm_k, bars + B_KF + sk, 0, T * 128, hk, it.b);
          } else {   // the tile's two pattern columns need not be neighbours (a missing one: its dS rows are zero)
            const int ca = a.tile_cols[2 * T], cb = a.tile_cols[2 * T + 1];
            tma_load_rows<D, 64>(dK, &tm_k, bars + B_KF + sk, 0, ca * 64, hk, it.b);
            tma_load_rows<D, 64>(dK, &tm_k, bars + B_KF + sk, 1, (cb >= 0 ? cb : ca) * 64, hk, it.b);
          }
          ++g;
        }
      }
      // every load asked for has landed before the CTA leaves
      for (int x = max(g - kAS, 0); x < g; ++x) mbar_wait(bars + B_AF + x % kAS, (x / kAS) & 1, a.error_word, 82);
      for (int x = max(g - kKS, 0); x < g; ++x) mbar_wait(bars + B_KF + x % kKS, (x / kKS) & 1, a.error_word, 87);
    }
  } else if (warp == 5) {
    // ------------------------------ MMA issuer ---------------------------------------------
    const bool lead = elect_one();
    constexpr uint32_t idesc = make_idesc_bf16(128, D, 1, 1);   // A = dS^T and B = K, both MN-major
    const uint32_t hi = desc_hi(1024);
    // A without swizzle: groups of 8 keys are 128 bytes apart (leading offset), groups of 8 queries 16 bytes x
    // the keys of a tile (stride offset); with 64-token blocks the key halves of a step are 16 KB apart
    const uint32_t a_hi = desc_hi(16 * BS, 0);
    const uint32_t a_lo0 = desc_lo(smem_u32(smem + SM::oA), 128), k_lo0 = desc_lo(smem_u32(smem + SM::oK), BwdTile<D>::kBox);
    bool ok = true;
    int g = 0, n_acc = 0;   // steps consumed and accumulators filled so far, over all items
#pragma unroll 1
    for (long long w = blockIdx.x; w < n_items && ok; w += gridDim.x) {
      const Item it = item_of(w);
      if (it.n_ent == 0) continue;
      const uint32_t acc = tmem + (n_acc & 1) * D;
      // the rows of the item that used this accumulator two items ago have been read
      if (n_acc >= 2) ok = mbar_wait(bars + B_FREE + (n_acc & 1), ((n_acc >> 1) - 1) & 1, a.error_word, 89);
#pragma unroll 1
      for (int x = 0; x < it.n_ent && ok; ++x, ++g) {
        const int sa = g % kAS, sk = g % kKS;
        ok = ok && mbar_wait(bars + B_AF + sa, (g / kAS) & 1, a.error_word, 83);
        ok = ok && mbar_wait(bars + B_KF + sk, (g / kKS) & 1, a.error_word, 88);
        if (ok) {
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + sa * (SM::kDs2 >> 4), b_lo = k_lo0 + sk * (kTile >> 4);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            if (lead)
              mma_ss2x(acc, a_lo + (BS == 128 ? kk * (256 >> 4) : (kk >> 2) * (16384 >> 4) + (kk & 3) * (256 >> 4)), a_hi,
                       b_lo + kk * (2048 >> 4), hi, idesc, (x > 0) || (kk > 0));
        }
        if (lead) { mma_commit(bars + B_AE + sa); mma_commit(bars + B_KE + sk); }
      }
      if (lead) mma_commit(bars + B_DONE + (n_acc & 1));
      ++n_acc;
    }
    if (lead) mma_commit(bars + B_ALL);
    mbar_wait(bars + B_ALL, 0, a.error_word, 84);           // nothing of mine is still running at exit
  } else {
    // ------------------------------ epilogue: dQ * scale -> bf16 ----------------------------
    bool ok = true;
    int n_acc = 0;
    for (long long w = blockIdx.x; w < n_items && ok; w += gridDim.x) {
      const Item it = item_of(w);
      const int qi = it.t * 128 + warp * 32 + lane;
      __nv_bfloat16* base = a.out0 + it.b * a.s0[0] + it.h * a.s0[1];
      if (it.n_ent > 0) {
        ok = mbar_wait_warp(bars + B_DONE + (n_acc & 1), (n_acc >> 1) & 1, a.error_word, 85);
        if (!ok) break;
        tc_fence_after();
        const uint32_t lane_addr = tmem + (n_acc & 1) * D + (static_cast<uint32_t>(warp * 32) << 16);
        // through 4 KB of shared memory per warp: whole rows per store instruction
#pragma unroll
        for (int c = 0; c < D / 64; ++c)
          store_acc_64cols(lane_addr + c * 64, smem + SM::oStage + warp * 4096, a.scale, [&](int r2) -> __nv_bfloat16* {
            const int q2 = it.t * 128 + warp * 32 + r2;
            return q2 < a.L ? base + static_cast<int64_t>(q2) * a.s0[2] + c * 64 : nullptr;
          });
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + B_FREE + (n_acc & 1));   // the accumulator may be filled again
        ++n_acc;
      } else if (qi < a.L) {
        __nv_bfloat16* dq_row = base + static_cast<int64_t>(qi) * a.s0[2];
#pragma unroll
        for (int x = 0; x < D; x += 8) *reinterpret_cast<uint4*>(dq_row + x) = make_uint4(0, 0, 0, 0);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem, 2 * D);
}

}  // namespace lg
