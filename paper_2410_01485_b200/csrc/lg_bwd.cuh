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
#pragma once
#include <cuda.h>
#include "lg_common.cuh"

namespace lg {

struct BwdArgs {
  const int32_t* tile_off;   // CSR row_ptr (dQ pass) or CSC col_ptr (dK/dV pass)
  const int32_t* tile_cnt;
  const int32_t* tile_ent;   // idx * 4 + member mask
  const int32_t* order;
  const float* lse;          // [B, Hq, L]
  const float* delta;        // [B, Hq, L]
  __nv_bfloat16* out0;       // dQ   | dK
  __nv_bfloat16* out1;       // unused | dV
  unsigned int* error_word;
  int64_t s0[3], s1[3];      // strides of out0 / out1 (batch, head, token; elements)
  int L, Hq, Hkv, G;
  float scale, scale_log2;
};

// ---- delta = rowsum(dO * O) ---------------------------------------------------------------
template <int D>
__global__ void delta_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ d_o,
                             float* __restrict__ delta, int64_t sb, int64_t sh, int64_t sl, int Hq, int L,
                             int64_t total_rows) {
  constexpr int TPR = D / 8;   // threads per row, 16 bytes each
  const int64_t gid = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t row = gid / TPR;
  const int ch = static_cast<int>(gid % TPR);
  float acc = 0.f;
  if (row < total_rows) {
    const int i = static_cast<int>(row % L);
    const int64_t bh = row / L;
    const int h = static_cast<int>(bh % Hq);
    const int64_t b = bh / Hq;
    const int64_t off = b * sb + h * sh + static_cast<int64_t>(i) * sl + ch * 8;
    const uint4 ov = *reinterpret_cast<const uint4*>(o + off);
    const uint4 dv = *reinterpret_cast<const uint4*>(d_o + off);
    const __nv_bfloat162* op = reinterpret_cast<const __nv_bfloat162*>(&ov);
    const __nv_bfloat162* dp = reinterpret_cast<const __nv_bfloat162*>(&dv);
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const float2 a = __bfloat1622float2(op[x]), c = __bfloat1622float2(dp[x]);
      acc += a.x * c.x + a.y * c.y;
    }
  }
#pragma unroll
  for (int s = TPR / 2; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
  if (row < total_rows && ch == 0) delta[row] = acc;
}

template <int D, int BS>
struct BwdSmem {
  static constexpr int kFixBytes = 128 * D * 2;   // Q or K (and dO or V) tile of the CTA's own 128 rows
  static constexpr int kStgBytes = BS * D * 2;    // streamed operand tile
  static constexpr int kVecOff = 2 * kFixBytes + 4 * kStgBytes;   // [2 stages][lse2, delta][BS] floats
  static constexpr int kBarOff = kVecOff + 2 * 2 * BS * 4;
  static constexpr int kTotal = kBarOff + 128 + 1024;
};

// store one 128 x D fp32 accumulator tile from TMEM as bf16 rows (times `mul`)
template <int D>
__device__ __forceinline__ void store_acc_rows(uint32_t taddr, __nv_bfloat16* row_ptr, float mul, bool do_store) {
#pragma unroll
  for (int c = 0; c < D / 32; ++c) {
    uint32_t reg[32];
    tmem_ld32(taddr + c * 32, reg);
    tmem_ld_wait();
    if (do_store) {
#pragma unroll
      for (int x = 0; x < 32; x += 8) {
        uint4 v4;
        v4.x = pack_bf16(__uint_as_float(reg[x + 0]) * mul, __uint_as_float(reg[x + 1]) * mul);
        v4.y = pack_bf16(__uint_as_float(reg[x + 2]) * mul, __uint_as_float(reg[x + 3]) * mul);
        v4.z = pack_bf16(__uint_as_float(reg[x + 4]) * mul, __uint_as_float(reg[x + 5]) * mul);
        v4.w = pack_bf16(__uint_as_float(reg[x + 6]) * mul, __uint_as_float(reg[x + 7]) * mul);
        *reinterpret_cast<uint4*>(row_ptr + c * 32 + x) = v4;
      }
    }
  }
}

// ============================== dK / dV pass ==================================================
template <int D, int BS>
__global__ void __launch_bounds__(128, 1)
bwd_dkdv_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                const BwdArgs a) {
  using SM = BwdSmem<D, BS>;
  constexpr int R = 128 / BS;
  constexpr int NBOX = D / 64;
  constexpr uint32_t kColS = 0, kColDP = BS, kColDV = 2 * BS, kColDK = 2 * BS + D;
  constexpr uint32_t kTmemCols = (2 * BS + 2 * D) <= 256 ? 256 : 512;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sK = smem;
  uint8_t* sV = sK + SM::kFixBytes;
  uint8_t* sQ = sV + SM::kFixBytes;                 // [stage]
  uint8_t* sDO = sQ + 2 * SM::kStgBytes;            // [stage]
  float* sVec = reinterpret_cast<float*>(smem + SM::kVecOff);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::kBarOff);
  uint64_t* bar_fix = bars + 0;
  uint64_t* bar_ld = bars + 1;   // [2]
  uint64_t* bar_s = bars + 3;
  uint64_t* bar_o = bars + 4;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 5);
  volatile uint32_t* s_fail = tmem_slot + 1;

  const int tid = threadIdx.x, warp = tid >> 5;
  const int tile = a.order[blockIdx.y];
  const int b = blockIdx.x / a.Hkv, hk = blockIdx.x % a.Hkv;
  const int n_ent = a.tile_cnt[tile];
  const int32_t* ent = a.tile_ent + a.tile_off[tile * R];
  const int key0 = tile * 128;
  const int n_iter = n_ent * a.G;

  if (warp == 0) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  if (tid == 0) {
    *s_fail = 0;
    mbar_init(bar_fix, 1);
    mbar_init(bar_ld + 0, 1);
    mbar_init(bar_ld + 1, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_o, 1);
    mbar_fence_init();
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    tma_prefetch_desc(&tm_do);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t lane_addr = tmem + (static_cast<uint32_t>(warp * 32) << 16);

  auto issue_ld = [&](int it) {
    const int st = it & 1;
    const int g = it / n_ent, e = it - g * n_ent;
    const int qb = ent[e] >> 2;
    const int h = hk * a.G + g;
    mbar_expect_tx(bar_ld + st, 2 * SM::kStgBytes);
#pragma unroll
    for (int x = 0; x < NBOX; ++x) {
      tma_load_4d(sQ + st * SM::kStgBytes + x * (BS * 128), &tm_q, bar_ld + st, x * 64, qb * BS, h, b);
      tma_load_4d(sDO + st * SM::kStgBytes + x * (BS * 128), &tm_do, bar_ld + st, x * 64, qb * BS, h, b);
    }
  };

  if (tid == 0) {
    mbar_expect_tx(bar_fix, 2 * SM::kFixBytes);
#pragma unroll
    for (int x = 0; x < NBOX; ++x) {
      tma_load_4d(sK + x * (128 * 128), &tm_k, bar_fix, x * 64, key0, hk, b);
      tma_load_4d(sV + x * (128 * 128), &tm_v, bar_fix, x * 64, key0, hk, b);
    }
    if (n_iter > 0) issue_ld(0);
  }

  constexpr uint32_t idesc_st = make_idesc_bf16(128, BS, 0, 0);   // S^T, dP^T: N = query block
  constexpr uint32_t idesc_acc = make_idesc_bf16(128, D, 0, 1);   // dV, dK: B = dO / Q, MN-major
  const int r = tid;
  const int kj = key0 + r;                         // this thread's key
  const int member = (R == 1) ? 0 : (r / BS);
  bool fail = false;

  for (int it = 0; it < n_iter; ++it) {
    const int st = it & 1;
    const int g = it / n_ent, e = it - g * n_ent;
    const int entry = ent[e];
    const int qb = entry >> 2;
    const int h = hk * a.G + g;
    // stage the per-query statistics of this block
    if (tid < BS) {
      const int64_t off = (static_cast<int64_t>(b) * a.Hq + h) * a.L + qb * BS + tid;
      sVec[(st * 2 + 0) * BS + tid] = a.lse[off] * 1.4426950408889634f;
      sVec[(st * 2 + 1) * BS + tid] = a.delta[off];
    }
    if (tid == 0) {
      if (it == 0) fail |= !mbar_wait(bar_fix, 0, a.error_word, 11);
      if (it > 0) fail |= !mbar_wait(bar_o, (it - 1) & 1, a.error_word, 12);   // MMAs of it-1 done
      if (!fail && it + 1 < n_iter) issue_ld(it + 1);
      fail |= !mbar_wait(bar_ld + st, (it >> 1) & 1, a.error_word, 13);
      if (!fail) {
        tc_fence_after();
        const uint32_t k_base = smem_u32(sK), v_base = smem_u32(sV);
        const uint32_t q_base = smem_u32(sQ + st * SM::kStgBytes), do_base = smem_u32(sDO + st * SM::kStgBytes);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t fo = (k >> 2) * (128 * 128) + (k & 3) * 32, so = (k >> 2) * (BS * 128) + (k & 3) * 32;
          mma_ss(tmem + kColS, make_smem_desc(k_base + fo, 16, 1024), make_smem_desc(q_base + so, 16, 1024),
                 idesc_st, k > 0);
        }
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t fo = (k >> 2) * (128 * 128) + (k & 3) * 32, so = (k >> 2) * (BS * 128) + (k & 3) * 32;
          mma_ss(tmem + kColDP, make_smem_desc(v_base + fo, 16, 1024), make_smem_desc(do_base + so, 16, 1024),
                 idesc_st, k > 0);
        }
      }
      mma_commit(bar_s);
    }
    __syncthreads();   // sVec visible
    fail |= !mbar_wait(bar_s, it & 1, a.error_word, 14);
    tc_fence_after();

    const bool need_mask = ((entry & 3) != ((1 << R) - 1)) || (qb * BS < key0 + 127);
    const bool row_on = (entry >> member) & 1;
    const float* lse2 = sVec + (st * 2 + 0) * BS;
    const float* dlt = sVec + (st * 2 + 1) * BS;
    // visible iff row_on and key <= query, i.e. column x (query qb*BS + x) >= kj - qb*BS
    const int xmin = need_mask ? (row_on ? kj - qb * BS : BS) : 0;
#pragma unroll
    for (int c = 0; c < BS / 32; ++c) {
      uint32_t sreg[32], dreg[32], preg[16], dsreg[16];
      tmem_ld32(lane_addr + kColS + c * 32, sreg);
      tmem_ld32(lane_addr + kColDP + c * 32, dreg);
      tmem_ld_wait();
#pragma unroll
      for (int x = 0; x < 32; x += 2) {
        const int col = c * 32 + x;
        float p0 = fast_exp2(__uint_as_float(sreg[x]) * a.scale_log2 - lse2[col]);
        float p1 = fast_exp2(__uint_as_float(sreg[x + 1]) * a.scale_log2 - lse2[col + 1]);
        p0 = (col >= xmin) ? p0 : 0.f;
        p1 = (col + 1 >= xmin) ? p1 : 0.f;
        const float d0 = p0 * (__uint_as_float(dreg[x]) - dlt[col]);
        const float d1 = p1 * (__uint_as_float(dreg[x + 1]) - dlt[col + 1]);
        preg[x >> 1] = pack_bf16(p0, p1);
        dsreg[x >> 1] = pack_bf16(d0, d1);
      }
      tmem_st16(lane_addr + kColS + c * 16, preg);     // P^T over the S^T columns already read
      tmem_st16(lane_addr + kColDP + c * 16, dsreg);   // dS^T over dP^T
    }
    tmem_st_wait();
    tc_fence_before();
    if (fail) *s_fail = 1;
    __syncthreads();
    const bool cta_fail = *s_fail != 0;
    if (tid == 0) {
      tc_fence_after();
      if (!cta_fail) {
        const uint32_t q_base = smem_u32(sQ + st * SM::kStgBytes), do_base = smem_u32(sDO + st * SM::kStgBytes);
#pragma unroll
        for (int k = 0; k < BS / 16; ++k)
          mma_ts(tmem + kColDV, tmem + kColS + k * 8, make_smem_desc(do_base + k * 2048, BS * 128, 1024), idesc_acc,
                 (it > 0) || (k > 0));
#pragma unroll
        for (int k = 0; k < BS / 16; ++k)
          mma_ts(tmem + kColDK, tmem + kColDP + k * 8, make_smem_desc(q_base + k * 2048, BS * 128, 1024), idesc_acc,
                 (it > 0) || (k > 0));
      }
      mma_commit(bar_o);
    }
    if (cta_fail) { fail = true; break; }
  }

  if (n_iter > 0) {
    fail |= !mbar_wait(bar_o, (n_iter - 1) & 1, a.error_word, 15);
    tc_fence_after();
  }
  {
    const bool st_ok = !fail && kj < a.L;
    __nv_bfloat16* dk_row = a.out0 + b * a.s0[0] + hk * a.s0[1] + static_cast<int64_t>(kj) * a.s0[2];
    __nv_bfloat16* dv_row = a.out1 + b * a.s1[0] + hk * a.s1[1] + static_cast<int64_t>(kj) * a.s1[2];
    if (n_iter > 0) {
      store_acc_rows<D>(lane_addr + kColDV, dv_row, 1.0f, st_ok);
      store_acc_rows<D>(lane_addr + kColDK, dk_row, a.scale, st_ok);
    } else if (st_ok) {
      for (int x = 0; x < D; x += 8) {
        *reinterpret_cast<uint4*>(dk_row + x) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(dv_row + x) = make_uint4(0, 0, 0, 0);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// ================================== dQ pass =================================================
template <int D, int BS>
__global__ void __launch_bounds__(128, 1)
bwd_dq_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
              const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
              const BwdArgs a) {
  using SM = BwdSmem<D, BS>;
  constexpr int R = 128 / BS;
  constexpr int NBOX = D / 64;
  constexpr uint32_t kColS = 0, kColDP = BS, kColDQ = 2 * BS;
  constexpr uint32_t kTmemCols = (2 * BS + D) <= 256 ? 256 : 512;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sDO = sQ + SM::kFixBytes;
  uint8_t* sK = sDO + SM::kFixBytes;                // [stage]
  uint8_t* sV = sK + 2 * SM::kStgBytes;             // [stage]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::kBarOff);
  uint64_t* bar_fix = bars + 0;
  uint64_t* bar_ld = bars + 1;
  uint64_t* bar_s = bars + 3;
  uint64_t* bar_o = bars + 4;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 5);
  volatile uint32_t* s_fail = tmem_slot + 1;

  const int tid = threadIdx.x, warp = tid >> 5;
  const int tile = a.order[blockIdx.y];
  const int b = blockIdx.x / a.Hq, h = blockIdx.x % a.Hq, hk = h / a.G;
  const int n_ent = a.tile_cnt[tile];
  const int32_t* ent = a.tile_ent + a.tile_off[tile * R];
  const int row0 = tile * 128;

  if (warp == 0) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  if (tid == 0) {
    *s_fail = 0;
    mbar_init(bar_fix, 1);
    mbar_init(bar_ld + 0, 1);
    mbar_init(bar_ld + 1, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_o, 1);
    mbar_fence_init();
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    tma_prefetch_desc(&tm_do);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t lane_addr = tmem + (static_cast<uint32_t>(warp * 32) << 16);

  auto issue_ld = [&](int e) {
    const int st = e & 1;
    const int kb = ent[e] >> 2;
    mbar_expect_tx(bar_ld + st, 2 * SM::kStgBytes);
#pragma unroll
    for (int x = 0; x < NBOX; ++x) {
      tma_load_4d(sK + st * SM::kStgBytes + x * (BS * 128), &tm_k, bar_ld + st, x * 64, kb * BS, hk, b);
      tma_load_4d(sV + st * SM::kStgBytes + x * (BS * 128), &tm_v, bar_ld + st, x * 64, kb * BS, hk, b);
    }
  };

  if (tid == 0) {
    mbar_expect_tx(bar_fix, 2 * SM::kFixBytes);
#pragma unroll
    for (int x = 0; x < NBOX; ++x) {
      tma_load_4d(sQ + x * (128 * 128), &tm_q, bar_fix, x * 64, row0, h, b);
      tma_load_4d(sDO + x * (128 * 128), &tm_do, bar_fix, x * 64, row0, h, b);
    }
    if (n_ent > 0) issue_ld(0);
  }

  constexpr uint32_t idesc_s = make_idesc_bf16(128, BS, 0, 0);
  constexpr uint32_t idesc_dq = make_idesc_bf16(128, D, 0, 1);
  const int r = tid;
  const int qi = row0 + r;
  const int member = (R == 1) ? 0 : (r / BS);
  float lse2 = 0.f, dlt = 0.f;
  if (qi < a.L) {
    const int64_t off = (static_cast<int64_t>(b) * a.Hq + h) * a.L + qi;
    lse2 = a.lse[off] * 1.4426950408889634f;
    dlt = a.delta[off];
  }
  bool fail = false;

  for (int e = 0; e < n_ent; ++e) {
    const int st = e & 1;
    const int entry = ent[e];
    const int kb = entry >> 2;
    if (tid == 0) {
      if (e == 0) fail |= !mbar_wait(bar_fix, 0, a.error_word, 21);
      if (e > 0) fail |= !mbar_wait(bar_o, (e - 1) & 1, a.error_word, 22);
      if (!fail && e + 1 < n_ent) issue_ld(e + 1);
      fail |= !mbar_wait(bar_ld + st, (e >> 1) & 1, a.error_word, 23);
      if (!fail) {
        tc_fence_after();
        const uint32_t q_base = smem_u32(sQ), do_base = smem_u32(sDO);
        const uint32_t k_base = smem_u32(sK + st * SM::kStgBytes), v_base = smem_u32(sV + st * SM::kStgBytes);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t fo = (k >> 2) * (128 * 128) + (k & 3) * 32, so = (k >> 2) * (BS * 128) + (k & 3) * 32;
          mma_ss(tmem + kColS, make_smem_desc(q_base + fo, 16, 1024), make_smem_desc(k_base + so, 16, 1024),
                 idesc_s, k > 0);
        }
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t fo = (k >> 2) * (128 * 128) + (k & 3) * 32, so = (k >> 2) * (BS * 128) + (k & 3) * 32;
          mma_ss(tmem + kColDP, make_smem_desc(do_base + fo, 16, 1024), make_smem_desc(v_base + so, 16, 1024),
                 idesc_s, k > 0);
        }
      }
      mma_commit(bar_s);
    }
    fail |= !mbar_wait(bar_s, e & 1, a.error_word, 24);
    tc_fence_after();

    const bool need_mask = ((entry & 3) != ((1 << R) - 1)) || (kb * BS + BS - 1 > row0);
    const bool row_on = (entry >> member) & 1;
    const int jmax = need_mask ? (row_on ? qi - kb * BS : -1) : BS;   // columns <= jmax visible
#pragma unroll
    for (int c = 0; c < BS / 32; ++c) {
      uint32_t sreg[32], dreg[32], dsreg[16];
      tmem_ld32(lane_addr + kColS + c * 32, sreg);
      tmem_ld32(lane_addr + kColDP + c * 32, dreg);
      tmem_ld_wait();
#pragma unroll
      for (int x = 0; x < 32; x += 2) {
        const int col = c * 32 + x;
        float p0 = fast_exp2(__uint_as_float(sreg[x]) * a.scale_log2 - lse2);
        float p1 = fast_exp2(__uint_as_float(sreg[x + 1]) * a.scale_log2 - lse2);
        p0 = (col <= jmax) ? p0 : 0.f;
        p1 = (col + 1 <= jmax) ? p1 : 0.f;
        dsreg[x >> 1] = pack_bf16(p0 * (__uint_as_float(dreg[x]) - dlt), p1 * (__uint_as_float(dreg[x + 1]) - dlt));
      }
      tmem_st16(lane_addr + kColS + c * 16, dsreg);   // dS over the S columns already read
    }
    tmem_st_wait();
    tc_fence_before();
    if (fail) *s_fail = 1;
    __syncthreads();
    const bool cta_fail = *s_fail != 0;
    if (tid == 0) {
      tc_fence_after();
      if (!cta_fail) {
        const uint32_t k_base = smem_u32(sK + st * SM::kStgBytes);
#pragma unroll
        for (int k = 0; k < BS / 16; ++k)
          mma_ts(tmem + kColDQ, tmem + kColS + k * 8, make_smem_desc(k_base + k * 2048, BS * 128, 1024), idesc_dq,
                 (e > 0) || (k > 0));
      }
      mma_commit(bar_o);
    }
    if (cta_fail) { fail = true; break; }
  }

  if (n_ent > 0) {
    fail |= !mbar_wait(bar_o, (n_ent - 1) & 1, a.error_word, 25);
    tc_fence_after();
  }
  {
    const bool st_ok = !fail && qi < a.L;
    __nv_bfloat16* dq_row = a.out0 + b * a.s0[0] + h * a.s0[1] + static_cast<int64_t>(qi) * a.s0[2];
    if (n_ent > 0) store_acc_rows<D>(lane_addr + kColDQ, dq_row, a.scale, st_ok);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace lg
