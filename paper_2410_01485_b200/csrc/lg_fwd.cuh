// Forward pass of block-sparse causal attention (paper Section 3.2: a FlashAttention-style
// kernel that never loads or computes a KV block whose mask is zero), with the log-sum-exp.
//
// One CTA owns a tile of 128 query rows of one head and walks the tile's schedule of active
// KV blocks.  Per block: TMA brings K and V tiles into 128-byte-swizzled shared memory,
// tcgen05.mma computes S = Q K^T into tensor memory, the 128 softmax threads (one per query
// row = one TMEM lane) update the running max / sum, write P as bf16 back into tensor
// memory, and a second tcgen05.mma accumulates O += P V with P read from tensor memory and
// V as an MN-major shared-memory operand.
#pragma once
#include <cuda.h>
#include "lg_common.cuh"

namespace lg {

struct FwdArgs {
  const int32_t* tile_off;   // row_ptr (CSR): entries of tile t start at tile_off[R * t]
  const int32_t* tile_cnt;   // [n_tiles]
  const int32_t* tile_ent;   // kb * 4 + member mask
  const int32_t* order;      // [n_tiles] launch rank -> tile
  __nv_bfloat16* o;
  float* lse;                // [B, Hq, L]
  unsigned int* error_word;
  int64_t o_strides[3];      // batch, head, token (elements)
  int L, Hq, G;              // G = Hq / Hkv
  float scale_log2;          // scale * log2(e)
};

template <int D, int BS>
struct FwdSmem {
  static constexpr int kQBytes = 128 * D * 2;
  static constexpr int kKVBytes = BS * D * 2;
  static constexpr int kStages = 2;
  static constexpr int kBarOff = kQBytes + 2 * kStages * kKVBytes;
  static constexpr int kTotal = kBarOff + 128 + 1024;   // + barriers + alignment slack
};

template <int D, int BS>
__global__ void __launch_bounds__(128, 1)
fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
           const __grid_constant__ CUtensorMap tm_v, const FwdArgs a) {
  using SM = FwdSmem<D, BS>;
  constexpr int R = 128 / BS;                 // pattern rows per query tile
  constexpr int NBOX = D / 64;                // 64-column TMA boxes per operand row
  constexpr uint32_t kColS = 0, kColP = BS, kColO = BS + BS / 2;
  constexpr uint32_t kTmemCols = (BS + BS / 2 + D) <= 256 ? 256 : 512;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = sQ + SM::kQBytes;                       // [stage][box][BS rows][128 B]
  uint8_t* sV = sK + SM::kStages * SM::kKVBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM::kBarOff);
  uint64_t* bar_q = bars + 0;
  uint64_t* bar_kv = bars + 1;                          // [2]
  uint64_t* bar_s = bars + 3;
  uint64_t* bar_o = bars + 4;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 5);
  volatile uint32_t* s_fail = tmem_slot + 1;   // set by any thread whose bounded wait expired

  const int tid = threadIdx.x, warp = tid >> 5;
  const int tile = a.order[blockIdx.y];
  const int bh = blockIdx.x;
  const int b = bh / a.Hq, h = bh % a.Hq, hk = h / a.G;
  const int n_ent = a.tile_cnt[tile];
  const int32_t* ent = a.tile_ent + a.tile_off[tile * R];
  const int row0 = tile * 128;

  if (warp == 0) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  if (tid == 0) {
    *s_fail = 0;
    mbar_init(bar_q, 1);
    mbar_init(bar_kv + 0, 1);
    mbar_init(bar_kv + 1, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_o, 1);
    mbar_fence_init();
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t lane_addr = tmem + (static_cast<uint32_t>(warp * 32) << 16);

  auto issue_kv = [&](int e) {
    const int st = e & 1;
    const int kb = ent[e] >> 2;
    mbar_expect_tx(bar_kv + st, 2 * SM::kKVBytes);
#pragma unroll
    for (int x = 0; x < NBOX; ++x) {
      tma_load_4d(sK + st * SM::kKVBytes + x * (BS * 128), &tm_k, bar_kv + st, x * 64, kb * BS, hk, b);
      tma_load_4d(sV + st * SM::kKVBytes + x * (BS * 128), &tm_v, bar_kv + st, x * 64, kb * BS, hk, b);
    }
  };

  if (tid == 0) {
    mbar_expect_tx(bar_q, SM::kQBytes);
#pragma unroll
    for (int x = 0; x < NBOX; ++x) tma_load_4d(sQ + x * (128 * 128), &tm_q, bar_q, x * 64, row0, h, b);
    if (n_ent > 0) issue_kv(0);
    if (n_ent > 1) issue_kv(1);
  }

  constexpr uint32_t idesc_s = make_idesc_bf16(128, BS, 0, 0);
  constexpr uint32_t idesc_o = make_idesc_bf16(128, D, 0, 1);

  float m_run = -INFINITY;   // running max of scale*log2e*s
  float l_run = 0.f;
  const int r = tid;                       // query row inside the tile == TMEM lane
  const int qi = row0 + r;
  const int member = (R == 1) ? 0 : (r / BS);
  bool fail = false;

  for (int e = 0; e < n_ent; ++e) {
    const int st = e & 1;
    const int entry = ent[e];
    const int kb = entry >> 2;
    if (tid == 0) {
      if (e == 0) fail |= !mbar_wait(bar_q, 0, a.error_word, 1);
      fail |= !mbar_wait(bar_kv + st, (e >> 1) & 1, a.error_word, 2);
      if (!fail) {
        tc_fence_after();
        const uint32_t q_base = smem_u32(sQ), k_base = smem_u32(sK + st * SM::kKVBytes);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t da = make_smem_desc(q_base + (k >> 2) * (128 * 128) + (k & 3) * 32, 16, 1024);
          const uint64_t db = make_smem_desc(k_base + (k >> 2) * (BS * 128) + (k & 3) * 32, 16, 1024);
          mma_ss(tmem + kColS, da, db, idesc_s, k > 0);
        }
      }
      mma_commit(bar_s);   // always commit so the other threads' wait ends
    }
    fail |= !mbar_wait(bar_s, e & 1, a.error_word, 3);
    tc_fence_after();

    // ---- softmax on this thread's row -----------------------------------------------
    uint32_t sreg[BS];
#pragma unroll
    for (int c = 0; c < BS / 32; ++c) tmem_ld32(lane_addr + kColS + c * 32, sreg + c * 32);
    tmem_ld_wait();
    const bool need_mask = ((entry & 3) != ((1 << R) - 1)) || (kb * BS + BS - 1 > row0);
    float mx = -INFINITY;
    if (need_mask) {
      const bool row_on = (entry >> member) & 1;
      const int jmax = row_on ? (qi - kb * BS) : -1;   // columns c <= jmax are visible
#pragma unroll
      for (int c = 0; c < BS; ++c) {
        float s = __uint_as_float(sreg[c]) * a.scale_log2;
        s = (c <= jmax) ? s : -INFINITY;
        sreg[c] = __float_as_uint(s);
        mx = fmaxf(mx, s);
      }
    } else {
#pragma unroll
      for (int c = 0; c < BS; ++c) {
        const float s = __uint_as_float(sreg[c]) * a.scale_log2;
        sreg[c] = __float_as_uint(s);
        mx = fmaxf(mx, s);
      }
    }
    const float m_new = fmaxf(m_run, mx);
    const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
    const float alpha = fast_exp2(m_run - m_use);     // m_run = -inf -> 0
    float rs = 0.f;
    uint32_t preg[BS / 2];
#pragma unroll
    for (int c = 0; c < BS; c += 2) {
      const float p0 = fast_exp2(__uint_as_float(sreg[c]) - m_use);
      const float p1 = fast_exp2(__uint_as_float(sreg[c + 1]) - m_use);
      rs += p0 + p1;
      preg[c >> 1] = pack_bf16(p0, p1);
    }
    l_run = l_run * alpha + rs;
    m_run = m_new;
#pragma unroll
    for (int c = 0; c < BS / 64; ++c) tmem_st32(lane_addr + kColP + c * 32, preg + c * 32);

    // ---- rescale the running O (needs the previous P V product to have landed) --------
    if (e > 0) {
      fail |= !mbar_wait(bar_o, (e - 1) & 1, a.error_word, 4);
      tc_fence_after();
      if (tid == 0 && !fail && e + 1 < n_ent) issue_kv(e + 1);   // stage (e+1)&1 was freed by P V of e-1
      if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t oreg[32];
          tmem_ld32(lane_addr + kColO + c * 32, oreg);
          tmem_ld_wait();
#pragma unroll
          for (int x = 0; x < 32; ++x) oreg[x] = __float_as_uint(__uint_as_float(oreg[x]) * alpha);
          tmem_st32(lane_addr + kColO + c * 32, oreg);
        }
      }
    }
    tmem_st_wait();
    tc_fence_before();
    if (fail) *s_fail = 1;
    __syncthreads();
    const bool cta_fail = *s_fail != 0;   // uniform: every thread leaves the loop together
    if (tid == 0) {
      tc_fence_after();
      if (!cta_fail) {
        const uint32_t v_base = smem_u32(sV + st * SM::kKVBytes);
#pragma unroll
        for (int k = 0; k < BS / 16; ++k) {
          const uint64_t db = make_smem_desc(v_base + k * 2048, BS * 128, 1024);
          mma_ts(tmem + kColO, tmem + kColP + k * 8, db, idesc_o, (e > 0) || (k > 0));
        }
      }
      mma_commit(bar_o);
    }
    if (cta_fail) { fail = true; break; }
  }

  // ---- epilogue: O / l -> bf16, LSE ------------------------------------------------------
  if (n_ent > 0) {
    fail |= !mbar_wait(bar_o, (n_ent - 1) & 1, a.error_word, 5);
    tc_fence_after();
  }
  if (qi < a.L) {   // warp-uniform: L is a multiple of 64
    const float inv_l = l_run > 0.f ? 1.f / l_run : 0.f;
    __nv_bfloat16* orow = a.o + b * a.o_strides[0] + h * a.o_strides[1] + static_cast<int64_t>(qi) * a.o_strides[2];
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
      uint32_t oreg[32];
      tmem_ld32(lane_addr + kColO + c * 32, oreg);
      tmem_ld_wait();
#pragma unroll
      for (int x = 0; x < 32; x += 8) {
        uint4 v4;
        v4.x = pack_bf16(__uint_as_float(oreg[x + 0]) * inv_l, __uint_as_float(oreg[x + 1]) * inv_l);
        v4.y = pack_bf16(__uint_as_float(oreg[x + 2]) * inv_l, __uint_as_float(oreg[x + 3]) * inv_l);
        v4.z = pack_bf16(__uint_as_float(oreg[x + 4]) * inv_l, __uint_as_float(oreg[x + 5]) * inv_l);
        v4.w = pack_bf16(__uint_as_float(oreg[x + 6]) * inv_l, __uint_as_float(oreg[x + 7]) * inv_l);
        if (!fail) *reinterpret_cast<uint4*>(orow + c * 32 + x) = v4;
      }
    }
    if (!fail)
      a.lse[(static_cast<int64_t>(b) * a.Hq + h) * a.L + qi] =
          l_run > 0.f ? (m_run + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace lg
