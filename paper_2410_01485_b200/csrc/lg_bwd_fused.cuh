// Backward pass in ONE sweep over the active blocks (paper Section 3.2: the masked blocks are
// skipped in the backward as in the forward; Table 1 counts forward and backward FLOPs).
//
// The two-pass backward (lg_bwd.cuh) computes S and dP twice, once per pass.  Here one CTA per
// kv tile (128 keys of one kv head) walks the tile's schedule exactly as the dK/dV pass does and
// produces, per half-step of 64 queries,
//   S^T = K Q^T,  dP^T = V dO^T          (tensor memory, one key per lane)
//   P^T, dS^T                            (element-wise warps; P^T back to tensor memory, dS^T to shared memory)
//   dV += P^T dO,  dK += dS^T Q          (accumulated in tensor memory over the whole schedule)
//   dQ^T(64 queries) = K^T dS^T          (a fresh [D x 64] product per half-step)
// and adds dQ^T into an fp32 copy of dQ in the workspace.  Several kv tiles add to the same query
// rows; to keep the result bitwise reproducible the parts of a 64-row group are added in a FIXED
// order, the launch order of the kv tiles: every schedule entry carries its rank, a counter per
// (head, 64-row group, quarter of the head dimension) says how many parts have arrived, and a part
// of rank r is added when the counter reads r (rank 0 stores instead of adding, so the buffer needs no clearing).  CTAs take
// their tile from a ticket counter, so a CTA only ever waits for CTAs that already run.
//
// Roles: warps 0-15 element-wise (four groups of 16 queries; thread = key = TMEM lane), warp 16 TMA,
// warps 17 / 18 issue tcgen05.mma, warps 19-22 move dQ^T from tensor memory to global memory.
//   issuer A: S^T(h+2) after dV(h)            (P^T is written over the S^T columns dV reads)
//   issuer B: dP^T(h+1), then dK(h), dQ^T(h)  (dQ^T(h) lands in the dP^T columns of its half, once
//                                               dP^T(h) has been read; dP^T(h+2) follows when dQ^T(h)
//                                               has been moved out)
// TMEM columns: S^T halves at 0 / 64, dP^T | dQ^T halves at 128 / 192, dV at 256, dK at 384.
#pragma once
#include <cuda.h>
#include "lg_bwd.cuh"

namespace lg {

struct FusedArgs {
  BwdArgs b;                  // schedule, statistics, outputs dK (out0) / dV (out1) as in the dK/dV pass
  const int32_t* tile_rank;   // parallel to tile_ent: rank of the tile's dQ part among the parts of that query block
  float* dq_acc;              // [B * Hq, Lp, D] fp32, Lp = L rounded up to 128 (b.Lp)
  unsigned int* sem;          // [0]: CTA ticket; [64 + ((b * Hq + h) * n64 + q64) * 4 + quarter]: parts of dQ added so far
  int n64;                    // 64-row groups per head = Lp / 64
  int n_tiles;
};

constexpr int kFuEwWarps = 16;
constexpr int kFuTmaWarp = 16, kFuMmaWarpA = 17, kFuMmaWarpB = 18, kFuRedWarp0 = 19, kFuRedWarps = 4;
constexpr int kFuThreads = (kFuRedWarp0 + kFuRedWarps) * 32;
constexpr int kFuCols = 64 / (kFuEwWarps / 4);   // queries of a half-step per element-wise thread (16)

template <int D, int BS>
struct FusedSmem {
  static constexpr int kTile = BwdTile<D>::kBytes;
  static constexpr int kDs = 128 * 128;                       // dS^T of one half-step: 128 keys x 64 queries bf16
  static constexpr int oK = 0, oV = kTile;
  static constexpr int oQ = 2 * kTile;                        // [2]
  static constexpr int oDO = oQ + 2 * kTile;                  // [2]
  static constexpr int oDS = oDO + 2 * kTile;                 // [2]
  static constexpr int oStat = oDS + 2 * kDs;                 // [2 stages][2 planes][128] floats
  static constexpr int oBar = oStat + 2 * 128 * 8;
  static constexpr int kTotal = oBar + 512;
};

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_add_u32(unsigned int* p, unsigned int v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_add_f32(float* p, float v) {
  asm volatile("red.relaxed.gpu.global.add.f32 [%0], %1;" ::"l"(p), "f"(v) : "memory");
}

template <int D, int BS>
__global__ void __launch_bounds__(kFuThreads, 1)
bwd_fused_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                 const FusedArgs fa) {
  static_assert(D == 128, "the dQ^T product puts the head dimension on the 128 TMEM lanes");
  const BwdArgs& a = fa.b;
  using SM = FusedSmem<D, BS>;
  constexpr int R = 128 / BS;
  constexpr uint32_t kColS = 0, kColDP = 128, kColDV = 256, kColDK = 384;
  constexpr int kTile = SM::kTile;
  enum { B_FIX = 0, B_QF = 1, B_QE = 3, B_OF = 5, B_OE = 7, B_SF = 9, B_DPF = 11, B_PF = 13, B_DSF = 15, B_DSE = 17,
         B_DQF = 19, B_DQR = 21, B_STF = 23, B_STE = 25, B_DONE = 27, B_DRAIN = 28, B_COUNT = 30 };

  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::oBar);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);       // [0] TMEM base, [1] abort word, [2] ticket
  int32_t* sInfo = reinterpret_cast<int32_t*>(bars + B_COUNT + 2);          // [2 stages][2 items][4]: entry, head, rank, -
  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
  if ((smem_u32(smem) & 1023u) != 0) {
    if (tid == 0) atomicCAS(a.error_word, 0u, (2u << 24) | 50u);
    return;
  }
  if (!lists_match(a.error_word, a.expect_fp, a.expect_fp2, 50u)) return;
  uint8_t* sK = smem + SM::oK;
  uint8_t* sV = smem + SM::oV;
  uint8_t* sQ = smem + SM::oQ;      // [2]
  uint8_t* sDO = smem + SM::oDO;    // [2]
  uint8_t* sDS = smem + SM::oDS;    // [2]
  float* sStat = reinterpret_cast<float*>(smem + SM::oStat);

  if (tid == 0) {
    tmem_slot[1] = *reinterpret_cast<volatile unsigned int*>(a.error_word);
    // Tiles are handed out in launch order through a ticket: a part of dQ only ever waits for parts of
    // tiles with a smaller ticket, and those CTAs are running (or done) by the time this one starts.
    tmem_slot[2] = atomicAdd(fa.sem, 1u);
    mbar_init(bars + B_FIX, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bars + B_QF + i, 1);
      mbar_init(bars + B_QE + i, 1);
      mbar_init(bars + B_OF + i, 1);
      mbar_init(bars + B_OE + i, 2);      // dP^T (issuer B) and dV (issuer A) both read the dO tile
      mbar_init(bars + B_SF + i, 1);
      mbar_init(bars + B_DPF + i, 1);
      mbar_init(bars + B_PF + i, kFuEwWarps);
      mbar_init(bars + B_DSF + i, kFuEwWarps);
      mbar_init(bars + B_DSE + i, 1);
      mbar_init(bars + B_DQF + i, 1);
      mbar_init(bars + B_DQR + i, kFuRedWarps);
      mbar_init(bars + B_STF + i, 1);
      mbar_init(bars + B_STE + i, kFuEwWarps + kFuRedWarps);
      mbar_init(bars + B_DRAIN + i, 1);
    }
    mbar_init(bars + B_DONE, 2);          // the last dV and the last dK / dQ^T
    mbar_fence_init();
  }
  if (warp == kFuMmaWarpA) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const unsigned int ticket = tmem_slot[2];
  const unsigned int n_heads_x = gridDim.x;
  if (tmem_slot[1] != 0 || ticket >= n_heads_x * static_cast<unsigned int>(fa.n_tiles)) {
    if (warp == kFuMmaWarpA) tmem_dealloc(tmem, 512);
    return;
  }
  const int tile = a.order[ticket / n_heads_x];
  const int bx = static_cast<int>(ticket % n_heads_x);
  const int b = bx / a.Hkv, hk = bx % a.Hkv;
  const int n_ent = a.tile_cnt[tile];
  const int32_t* ent = a.tile_ent + a.tile_off[tile];
  const int32_t* rnk = fa.tile_rank + a.tile_off[tile];
  const int kb_a = a.tile_cols[R * tile], kb_b = (R == 2) ? a.tile_cols[R * tile + 1] : -1;
  const int n_items = n_ent * a.G;
  const int n_hs = (BS == 128) ? 2 * n_items : n_items;     // half-steps of 64 queries
  const int n_steps = (n_hs + 1) / 2;
  auto closes_step = [&](int hs) { return (hs & 1) == 1 || hs == n_hs - 1; };

  if (warp == kFuTmaWarp) {
    // ------------------------------ TMA producer ------------------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v); tma_prefetch_desc(&tm_do);
      mbar_expect_tx(bars + B_FIX, 2 * kTile);
      tma_load_rows<D, BS>(sK, &tm_k, bars + B_FIX, 0, kb_a * BS, hk, b);
      tma_load_rows<D, BS>(sV, &tm_v, bars + B_FIX, 0, kb_a * BS, hk, b);
      if (R == 2) {
        tma_load_rows<D, BS>(sK, &tm_k, bars + B_FIX, 1, (kb_b >= 0 ? kb_b : kb_a) * BS, hk, b);
        tma_load_rows<D, BS>(sV, &tm_v, bars + B_FIX, 1, (kb_b >= 0 ? kb_b : kb_a) * BS, hk, b);
      }
      bool ok = true;
      int nq = 0, no = 0, nst = 0;
      int grp = 0, e = 0;
      auto next_item = [&](int& hq, int& qrow, int& entry, int& rank) {
        entry = ent[e];
        rank = rnk[e];
        hq = hk * a.G + grp;
        qrow = (entry >> 2) * BS;
        if (++e == n_ent) { e = 0; ++grp; }
      };
      for (int j = 0; j < n_steps; ++j) {
        const int st = j & 1;
        int h0, r0, e0, k0, h1, r1, e1, k1;
        next_item(h0, r0, e0, k0);
        h1 = h0; r1 = r0; e1 = e0 & ~3; k1 = -1;               // a missing second item: nobody's member, no dQ part
        if (BS == 64 && 2 * j + 1 < n_items) next_item(h1, r1, e1, k1);
        if (BS == 128) k1 = k0;
        if (j >= 2) ok = mbar_wait(bars + B_STE + st, ((j / 2) - 1) & 1, a.error_word, 51);
        if (!ok) break;
        int32_t* info = sInfo + st * 8;
        info[0] = e0; info[1] = h0; info[2] = k0; info[3] = r0;
        info[4] = e1; info[5] = h1; info[6] = k1; info[7] = (BS == 128) ? r0 + 64 : r1;
        mbar_expect_tx(bars + B_STF + st, 2 * 128 * 4);
        {
          const float* st0 = a.stat + (static_cast<int64_t>(b) * a.Hq + h0) * a.Lp + r0;
          const float* st1 = a.stat + (static_cast<int64_t>(b) * a.Hq + h1) * a.Lp + r1;
#pragma unroll
          for (int pl = 0; pl < 2; ++pl) {
            float* dst = sStat + (st * 2 + pl) * 128;
            if (BS == 128) {
              bulk_load(dst, st0 + pl * a.stat_plane, 128 * 4, bars + B_STF + st);
            } else {
              bulk_load(dst, st0 + pl * a.stat_plane, 64 * 4, bars + B_STF + st);
              bulk_load(dst + 64, st1 + pl * a.stat_plane, 64 * 4, bars + B_STF + st);
            }
          }
        }
        nst = j + 1;
        if (j >= 2) ok = mbar_wait(bars + B_QE + st, ((j / 2) - 1) & 1, a.error_word, 52);
        if (!ok) break;
        mbar_expect_tx(bars + B_QF + st, kTile);
        tma_load_rows<D, BS>(sQ + st * kTile, &tm_q, bars + B_QF + st, 0, r0, h0, b);
        if (BS == 64) tma_load_rows<D, BS>(sQ + st * kTile, &tm_q, bars + B_QF + st, 1, r1, h1, b);
        nq = j + 1;
        if (j >= 2) ok = mbar_wait(bars + B_OE + st, ((j / 2) - 1) & 1, a.error_word, 53);
        if (!ok) break;
        mbar_expect_tx(bars + B_OF + st, kTile);
        tma_load_rows<D, BS>(sDO + st * kTile, &tm_do, bars + B_OF + st, 0, r0, h0, b);
        if (BS == 64) tma_load_rows<D, BS>(sDO + st * kTile, &tm_do, bars + B_OF + st, 1, r1, h1, b);
        no = j + 1;
      }
      mbar_wait(bars + B_FIX, 0, a.error_word, 54);
      for (int j = max(nq - 2, 0); j < nq; ++j) mbar_wait(bars + B_QF + (j & 1), (j / 2) & 1, a.error_word, 55);
      for (int j = max(no - 2, 0); j < no; ++j) mbar_wait(bars + B_OF + (j & 1), (j / 2) & 1, a.error_word, 56);
      for (int j = max(nst - 2, 0); j < nst; ++j) mbar_wait(bars + B_STF + (j & 1), (j / 2) & 1, a.error_word, 57);
    }
  } else if (warp == kFuMmaWarpA) {
    // ------------------------------ MMA issuer A: S^T and dV -------------------------------
    const bool lead = elect_one();
    constexpr uint32_t idesc_st = make_idesc_bf16(128, 64, 0, 0);
    constexpr uint32_t idesc_acc = make_idesc_bf16(128, D, 0, 1);        // dV: B = dO, MN-major
    constexpr uint32_t kHalfRows = (64 * 128) >> 4;
    const uint32_t hi = desc_hi(1024);
    const uint32_t k_lo = desc_lo(smem_u32(sK), 16), q_lo = desc_lo(smem_u32(sQ), 16);
    const uint32_t do_mn_lo = desc_lo(smem_u32(sDO), BwdTile<D>::kBox);
    bool ok = mbar_wait(bars + B_FIX, 0, a.error_word, 58);
#pragma unroll 1
    for (int hs = -2; hs < n_hs; ++hs) {
      if (hs >= 0) {
        const int j = hs >> 1, half = hs & 1, st = j & 1;
        if (half == 0) ok = ok && mbar_wait(bars + B_OF + st, (j / 2) & 1, a.error_word, 59);
        ok = ok && mbar_wait(bars + B_PF + half, j & 1, a.error_word, 60);
        if (ok) {
          tc_fence_after();
          const uint32_t b_lo = do_mn_lo + st * (kTile >> 4) + half * 4 * (2048 >> 4);
          const uint32_t a_t = tmem + kColS + half * 64;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            if (lead) mma_ts2(tmem + kColDV, a_t + kk * kFuCols, b_lo + kk * (2048 >> 4), hi, idesc_acc, (hs > 0) || (kk > 0));   // P^T of query group kk sits in the first half of the group's own 16 columns
        }
        if (lead && closes_step(hs)) mma_commit(bars + B_OE + st);
      }
      const int hn = hs + 2;
      if (hn < n_hs) {
        const int j = hn >> 1, half = hn & 1, st = j & 1;
        if (half == 0) ok = ok && mbar_wait(bars + B_QF + st, (j / 2) & 1, a.error_word, 61);
        if (ok) {
          tc_fence_after();
          const uint32_t b_lo = q_lo + st * (kTile >> 4) + half * kHalfRows;
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            constexpr int kB = BwdTile<D>::kBox >> 4;
            const uint32_t off = (k >> 2) * kB + (k & 3) * 2;
            if (lead) mma_ss2(tmem + kColS + half * 64, k_lo + off, b_lo + off, hi, idesc_st, k > 0);
          }
        }
        if (lead) mma_commit(bars + B_SF + half);
      }
    }
    if (lead) { mma_commit(bars + B_DONE); mma_commit(bars + B_DRAIN); }
    mbar_wait(bars + B_DRAIN, 0, a.error_word, 62);
  } else if (warp == kFuMmaWarpB) {
    // ------------------------------ MMA issuer B: dP^T, dK and dQ^T ------------------------
    const bool lead = elect_one();
    constexpr uint32_t idesc_st = make_idesc_bf16(128, 64, 0, 0);
    constexpr uint32_t idesc_dk = make_idesc_bf16(128, D, 0, 1);         // dK: A = dS^T (K-major), B = Q (MN-major)
    constexpr uint32_t idesc_dq = make_idesc_bf16(D, 64, 1, 1);          // dQ^T: A = K^T (MN-major), B = dS^T (MN-major)
    constexpr uint32_t kHalfRows = (64 * 128) >> 4;
    const uint32_t hi = desc_hi(1024);
    const uint32_t v_lo = desc_lo(smem_u32(sV), 16), do_lo = desc_lo(smem_u32(sDO), 16);
    const uint32_t q_mn_lo = desc_lo(smem_u32(sQ), BwdTile<D>::kBox);
    const uint32_t k_mn_lo = desc_lo(smem_u32(sK), BwdTile<D>::kBox);
    const uint32_t ds_lo = desc_lo(smem_u32(sDS), 16);                    // as the K-major A operand of dK
    const uint32_t ds_mn_lo = desc_lo(smem_u32(sDS), SM::kDs);            // as the MN-major B operand of dQ^T (one column group)
    bool ok = mbar_wait(bars + B_FIX, 0, a.error_word, 63);
#pragma unroll 1
    for (int hs = -1; hs < n_hs; ++hs) {
      const int hn = hs + 1;
      if (hn < n_hs) {   // dP^T(hn) into its half's columns, once the dQ^T that sat there has been moved out
        const int j = hn >> 1, half = hn & 1, st = j & 1;
        if (j >= 1) ok = ok && mbar_wait(bars + B_DQR + half, (j - 1) & 1, a.error_word, 64);
        if (half == 0) ok = ok && mbar_wait(bars + B_OF + st, (j / 2) & 1, a.error_word, 65);
        if (ok) {
          tc_fence_after();
          const uint32_t b_lo = do_lo + st * (kTile >> 4) + half * kHalfRows;
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            constexpr int kB = BwdTile<D>::kBox >> 4;
            const uint32_t off = (k >> 2) * kB + (k & 3) * 2;
            if (lead) mma_ss2(tmem + kColDP + half * 64, v_lo + off, b_lo + off, hi, idesc_st, k > 0);
          }
        }
        if (lead) {
          mma_commit(bars + B_DPF + half);
          if (closes_step(hn)) mma_commit(bars + B_OE + st);
        }
      }
      if (hs >= 0) {
        const int j = hs >> 1, half = hs & 1, st = j & 1;
        ok = ok && mbar_wait(bars + B_DSF + half, j & 1, a.error_word, 66);
        if (ok) {
          tc_fence_after();
          const uint32_t ds_off = half * (SM::kDs >> 4);
          // dK += dS^T(128 keys x 64 queries) Q(64 queries x D)
          const uint32_t bq_lo = q_mn_lo + st * (kTile >> 4) + half * 4 * (2048 >> 4);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            if (lead) mma_ss2(tmem + kColDK, ds_lo + ds_off + kk * 2, bq_lo + kk * (2048 >> 4), hi, idesc_dk, (hs > 0) || (kk > 0));
          // dQ^T(D x 64 queries) = K^T(D x 128 keys) dS^T(128 keys x 64 queries)
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            if (lead) mma_ss2(tmem + kColDP + half * 64, k_mn_lo + kk * (2048 >> 4), ds_mn_lo + ds_off + kk * (2048 >> 4), hi, idesc_dq, kk > 0);
        }
        if (lead) {
          mma_commit(bars + B_DQF + half);
          mma_commit(bars + B_DSE + half);
          if (closes_step(hs)) mma_commit(bars + B_QE + st);
        }
      }
    }
    if (lead) { mma_commit(bars + B_DONE); mma_commit(bars + B_DRAIN + 1); }
    mbar_wait(bars + B_DRAIN + 1, 0, a.error_word, 67);
  } else if (warp >= kFuRedWarp0) {
    // ------------------------------ dQ^T: tensor memory -> fp32 dQ in global memory ---------
    const int rw = warp & 3;                                  // TMEM lane quarter this warp may read
    const int d = rw * 32 + lane;                             // head-dimension index of this thread
    const uint32_t lane_addr = tmem + (static_cast<uint32_t>(rw * 32) << 16);
    bool ok = true;
    // The count that lets the next part in may only rise once my adds have been performed, and finding
    // that out (a fence) takes a round trip to the L2 of a couple of thousand cycles.  The fence is
    // therefore paid once per step (two parts), after the next product has been taken out of tensor
    // memory, so that the tensor pipe never waits for it.
    unsigned int* rel0 = nullptr;                             // counters of the parts whose adds are not yet published
    unsigned int* rel1 = nullptr;
    auto publish = [&]() {
      if (rel0 || rel1) {
        __threadfence();                                      // my stores / adds come before ...
        __syncwarp();
        if (lane == 0) {                                      // ... the counts that let the next parts in
          if (rel0) red_release_add_u32(rel0, 1u);
          if (rel1) red_release_add_u32(rel1, 1u);
        }
        rel0 = rel1 = nullptr;
      }
    };
    auto counter_of = [&](int hq, int qrow0) {
      // one counter per (head, 64-row group, quarter of the head dimension): the four warps move disjoint
      // columns of dQ and never have to wait for one another
      return fa.sem + 64 + (((static_cast<int64_t>(b) * a.Hq + hq) * fa.n64 + (qrow0 >> 6)) << 2) + rw;
    };
    // wait (bounded) until `rank` parts are in; gives up at once if any CTA has reported a failure
    auto wait_turn = [&](const unsigned int* sp, int rank, unsigned int seen) {
      if (rank <= 0 || seen >= static_cast<unsigned int>(rank)) return true;
      const long long t0 = clock64();
      unsigned int it = 0;
      while (ld_acquire_u32(sp) < static_cast<unsigned int>(rank)) {
        if ((++it & 63u) == 0) {
          if (*reinterpret_cast<volatile unsigned int*>(a.error_word) != 0) return false;
          if (clock64() - t0 > kWaitLimitCycles) {
            atomicCAS(a.error_word, 0u, (1u << 24) | 70u);
            return false;
          }
        }
      }
      return true;
    };
#pragma unroll 1
    for (int j = 0; j < n_steps && ok; ++j) {
      const int st = j & 1;
      ok = mbar_wait(bars + B_STF + st, (j >> 1) & 1, a.error_word, 68);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const int32_t* info = sInfo + st * 8;
      const bool two = 2 * j + 1 < n_hs;
      const int hq0 = info[1], rank0 = info[2], row0 = info[3];
      const int hq1 = info[5], rank1 = two ? info[6] : -1, row1 = info[7];
      unsigned int* sp0 = counter_of(hq0, row0);
      unsigned int* sp1 = counter_of(hq1, row1);
      // is it my turn?  asked now, so that the answers travel while the products are still being computed
      const unsigned int seen0 = rank0 > 0 ? ld_acquire_u32(sp0) : 0u;
      const unsigned int seen1 = rank1 > 0 ? ld_acquire_u32(sp1) : 0u;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        if (half == 1 && !two) break;
        ok = mbar_wait(bars + B_DQF + half, j & 1, a.error_word, 69);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        uint32_t v[64];
        tmem_ld32(lane_addr + kColDP + half * 64, v);
        tmem_ld32(lane_addr + kColDP + half * 64 + 32, v + 32);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + B_DQR + half);      // the columns may take the next dP^T
        if (half == 1 || !two) {
          __syncwarp();
          if (lane == 0) mbar_arrive(bars + B_STE + st);
        }
        if (half == 0) publish();                             // the previous step's parts
        const int rank = half ? rank1 : rank0;
        if (rank < 0) continue;                               // a padding half-step: no part of dQ
        unsigned int* sp = half ? sp1 : sp0;
        float* dst = fa.dq_acc + ((static_cast<int64_t>(b) * a.Hq + (half ? hq1 : hq0)) * a.Lp + (half ? row1 : row0)) * D + d;
        if (rank == 0) {
#pragma unroll
          for (int c = 0; c < 64; ++c) dst[c * D] = __uint_as_float(v[c]);
        } else {
          ok = wait_turn(sp, rank, half ? seen1 : seen0);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
#pragma unroll
          for (int c = 0; c < 64; ++c) red_add_f32(dst + c * D, __uint_as_float(v[c]));
        }
        if (half) rel1 = sp; else rel0 = sp;
      }
    }
    if (ok) publish();
  } else {
    // ------------------------------ element-wise warps ------------------------------------
    constexpr int C = kFuCols;
    const int g = warp >> 2;
    const int r = (warp & 3) * 32 + lane;                   // key row in the tile == TMEM lane
    const int member = (R == 1) ? 0 : (r / BS);
    const int kb_mine = (R == 2 && member) ? kb_b : kb_a;
    const int kj = kb_mine * BS + (R == 2 ? (r & (BS - 1)) : r);
    const int dend = (a.doc_end && kb_mine >= 0 && kj < a.L) ? a.doc_end[static_cast<int64_t>(b) * a.L + kj] : a.L;
    const uint32_t lane_addr = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const uint64_t scale2 = f32x2(a.scale_log2, a.scale_log2);
    // my 16 queries of a half-step are two 16-byte chunks of my key's row of the dS^T tile (128-byte swizzle)
    const uint32_t ds_row = smem_u32(sDS) + r * 128;
    const uint32_t ds_c0 = static_cast<uint32_t>(((2 * g) ^ (r & 7)) * 16), ds_c1 = static_cast<uint32_t>(((2 * g + 1) ^ (r & 7)) * 16);
    bool ok = true;
#pragma unroll 1
    for (int hs = 0; hs < n_hs; ++hs) {
      const int j = hs >> 1, half = hs & 1, st = j & 1;
      if (half == 0) {
        ok = mbar_wait(bars + B_STF + st, (j >> 1) & 1, a.error_word, 71);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      const float4* st_l = reinterpret_cast<const float4*>(sStat + st * 256 + half * 64 + g * C);
      const float4* st_d = st_l + 128 / 4;
      const int col0 = half * 64 + g * C;
      const int entry = sInfo[st * 8 + (BS == 64 ? half * 4 : 0)];
      const int q0 = (entry >> 2) * BS + (BS == 128 ? col0 : col0 % 64);
      const bool on = (entry >> member) & 1;
      const int xmin = on ? min(max(kj - q0, 0), C) : C;
      const int hi_abs = (a.exact_w > 0 && kb_mine >= a.ns) ? min(dend, kj + a.exact_w) : dend;
      const int xmax = min(max(hi_abs - q0, 0), C);
      const uint32_t s_addr = lane_addr + kColS + half * 64 + g * C;
      const uint32_t dp_addr = lane_addr + kColDP + half * 64 + g * C;

      ok = mbar_wait(bars + B_SF + half, j & 1, a.error_word, 72);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      float p[C];
      {
        uint32_t sreg[C];
        tmem_ld16(s_addr, sreg);
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
          float v0 = fast_exp2(x0), v1 = fast_exp2(x1), v2 = fast_exp2(x2), v3 = fast_exp2(x3);
          if (masked) {
            v0 = (c >= xmin && c < xmax) ? v0 : 0.f;
            v1 = (c + 1 >= xmin && c + 1 < xmax) ? v1 : 0.f;
            v2 = (c + 2 >= xmin && c + 2 < xmax) ? v2 : 0.f;
            v3 = (c + 3 >= xmin && c + 3 < xmax) ? v3 : 0.f;
          }
          p[c] = v0; p[c + 1] = v1; p[c + 2] = v2; p[c + 3] = v3;
        }
        uint32_t preg[C / 2];
#pragma unroll
        for (int c = 0; c < C; c += 2) preg[c >> 1] = pack_bf16(p[c], p[c + 1]);
        tmem_st8(s_addr, preg);                               // P^T over my own S^T columns
        ew_publish(bars + B_PF + half);
      }
      ok = mbar_wait(bars + B_DPF + half, j & 1, a.error_word, 73);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t dsreg[C / 2];
      {
        uint32_t dreg[C];
        tmem_ld16(dp_addr, dreg);
        tmem_ld_wait();
#pragma unroll
        for (int x = 0; x < C; x += 4) {
          const float4 d4 = st_d[x >> 2];
          float d0, d1, d2, d3;
          f32x2_split(mul_f32x2(f32x2(p[x], p[x + 1]),
                                add_f32x2(f32x2(__uint_as_float(dreg[x]), __uint_as_float(dreg[x + 1])),
                                          f32x2(d4.x, d4.y))), d0, d1);
          f32x2_split(mul_f32x2(f32x2(p[x + 2], p[x + 3]),
                                add_f32x2(f32x2(__uint_as_float(dreg[x + 2]), __uint_as_float(dreg[x + 3])),
                                          f32x2(d4.z, d4.w))), d2, d3);
          dsreg[x >> 1] = pack_bf16(d0, d1);
          dsreg[(x >> 1) + 1] = pack_bf16(d2, d3);
        }
      }
      // dS^T goes to shared memory (the operand of both dK and dQ^T); the half's tile is free again once
      // the products of half-step hs - 2 have finished
      if (j >= 1) {
        ok = mbar_wait(bars + B_DSE + half, (j - 1) & 1, a.error_word, 74);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      {
        const uint32_t base = ds_row + half * SM::kDs;
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(base + ds_c0), "r"(dsreg[0]), "r"(dsreg[1]),
                     "r"(dsreg[2]), "r"(dsreg[3]) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(base + ds_c1), "r"(dsreg[4]), "r"(dsreg[5]),
                     "r"(dsreg[6]), "r"(dsreg[7]) : "memory");
      }
      tc_fence_before();                                      // my tcgen05.ld of dP^T is done before dQ^T may overwrite it
      fence_proxy_async_smem();                               // my stores are visible to the tensor core's reads
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + B_DSF + half);
      if (closes_step(hs)) {
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + B_STE + st);
      }
    }
    // ---- epilogue: dV, dK * scale -> bf16 ---------------------------------------------------
    if (ok && n_hs > 0) {
      ok = mbar_wait(bars + B_DONE, 0, a.error_word, 75);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      constexpr int kEpi = 32;
      const bool mine = kj < a.L;
      if (kb_mine >= 0 && g * kEpi < D) {
        __nv_bfloat16* dk_row = a.out0 + b * a.s0[0] + hk * a.s0[1] + static_cast<int64_t>(kj) * a.s0[2] + g * kEpi;
        __nv_bfloat16* dv_row = a.out1 + b * a.s1[0] + hk * a.s1[1] + static_cast<int64_t>(kj) * a.s1[2] + g * kEpi;
        if (n_hs > 0) {
          store_acc_cols<kEpi>(lane_addr + kColDV + g * kEpi, dv_row, 1.0f, mine);
          store_acc_cols<kEpi>(lane_addr + kColDK + g * kEpi, dk_row, a.scale, mine);
        } else if (mine) {
#pragma unroll
          for (int x = 0; x < kEpi; x += 8) {
            *reinterpret_cast<uint4*>(dk_row + x) = make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4*>(dv_row + x) = make_uint4(0, 0, 0, 0);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kFuMmaWarpA) tmem_dealloc(tmem, 512);
}

// dq = scale * (fp32 sum of the parts), rounded to bf16.  One thread per 8 elements.
template <int D>
__global__ void dq_convert_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dq, int64_t sb, int64_t sh,
                                  int64_t sl, int Hq, int L, int Lp, int64_t n_rows, float scale) {
  constexpr int TPR = D / 8;
  const int64_t gid = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t row = gid / TPR;
  const int ch = static_cast<int>(gid % TPR);
  if (row >= n_rows) return;
  const int i = static_cast<int>(row % L);
  const int64_t bh = row / L;
  const float4* src = reinterpret_cast<const float4*>(acc + (bh * Lp + i) * D + ch * 8);
  const float4 x = src[0], y = src[1];
  uint4 v;
  v.x = pack_bf16(x.x * scale, x.y * scale);
  v.y = pack_bf16(x.z * scale, x.w * scale);
  v.z = pack_bf16(y.x * scale, y.y * scale);
  v.w = pack_bf16(y.z * scale, y.w * scale);
  const int64_t b = bh / Hq, h = bh % Hq;
  *reinterpret_cast<uint4*>(dq + b * sb + h * sh + static_cast<int64_t>(i) * sl + ch * 8) = v;
}

}  // namespace lg
