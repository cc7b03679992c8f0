// Serving side of the paper's Section 3.2: a rolling-buffer KV cache for the sliding window
// with the sink kept beside it, and a single-token decode whose only job is to stream that
// cache from HBM as fast as possible.
//
// Decode layout: the 16-token tiles of all (sequence, kv head, head group of <= 8 query heads)
// units form one sequence that is cut into equal slices, one per CTA, so that a single wave of
// CTAs streams the whole cache whatever the mix of lengths.  Each of a CTA's warps owns a
// contiguous run of tiles and keeps a private cp.async pipeline of kDecStages tiles (16-byte
// copies into XOR-swizzled shared memory, so the HBM stream never waits on arithmetic).  Scores
// are S^T = K Q^T and the output is O^T = V^T P^T, both on mma.sync m16n8k16 (bf16 in, fp32
// accumulate) with the 8 query heads of the group as the N dimension, so all heads of a GQA group
// share every byte loaded.  The warps' (max, sum, O) are merged in warp order in shared memory; a
// CTA whose slice is a whole unit writes the result itself, otherwise the CTAs of a unit leave
// records in the workspace and the one that arrives last merges them in index order.  Either way
// the summation order is fixed, so results are bitwise reproducible.  (Batches of more than
// kDecFlatMaxB sequences use a per-unit split grid and a separate merge kernel.)
#include <math.h>

#include <mutex>

#include "lg_common.cuh"
#include "lg_host.h"

namespace lg {

#ifndef LG_DEC_WARPS
#define LG_DEC_WARPS 8
#endif
constexpr int kDecWarps = LG_DEC_WARPS;   // warps per CTA, each with its own pipeline of tiles
constexpr int kDecThreads = kDecWarps * 32;
constexpr int kDecStages = 3;
constexpr int kDecTile = 16;          // tokens per warp tile
constexpr int kDecHeads = 8;          // query heads per CTA (mma N)

struct DecodeArgs {
  const __nv_bfloat16* q;        // [B, Hq, D]
  const __nv_bfloat16* k_cache;  // [B, Hkv, C, D]
  const __nv_bfloat16* v_cache;
  const int64_t* n_tokens;       // [B]
  float* part;                   // [B, Hkv*HG, nsplit, 8 heads, (D + 2)] : O, m, l
  __nv_bfloat16* o;              // [B, Hq, D]
  float* lse;                    // [B, Hq] or null
  int Hq, Hkv, G, HG, C, nsplit;
  float scale_log2;
  int sink, block_tokens;        // sink slots; block of the block-aligned window (0: every held token is attended)
  int B;                         // sequences (flattened path)
  unsigned int* unit_count;      // [B * Hkv * HG] records delivered per unit (flattened path; zero between calls)
};

__device__ __forceinline__ void cp_async16(uint32_t smem_addr, const void* gptr, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_addr), "l"(gptr), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ uint32_t movmatrix_t(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
  return y;
}
__device__ __forceinline__ void mma16816(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// One segment of one (sequence, kv head, head group): warp w of the CTA streams tiles
// [t_begin, t_end) of the cache, the four warps' partials are merged in warp order and the
// CTA's (max, sum, O) record for its 8 heads is written to `out`.
template <int D>
__device__ __forceinline__ void decode_run_segment(const DecodeArgs& a, uint8_t* dsmem, int b, int kvh, int hg,
                                                   int nvalid, int t_begin, int t_end, float* out, bool direct) {
  constexpr int kRowBytes = D * 2;
  constexpr int kChunks = D / 8;                      // 16-byte chunks per row
  constexpr int kTileBytes = kDecTile * kRowBytes;    // K (or V) bytes of one tile
  constexpr int kCopiesPerLane = kDecTile * kChunks / 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = lane >> 2, c = lane & 3;
  uint8_t* wsm = dsmem + warp * (kDecStages * 2 * kTileBytes);
  const uint32_t wsm_u32 = smem_u32(wsm);
  const uint8_t* kbase = reinterpret_cast<const uint8_t*>(a.k_cache) +
                         (static_cast<int64_t>(b) * a.Hkv + kvh) * static_cast<int64_t>(a.C) * kRowBytes;
  const uint8_t* vbase = reinterpret_cast<const uint8_t*>(a.v_cache) +
                         (static_cast<int64_t>(b) * a.Hkv + kvh) * static_cast<int64_t>(a.C) * kRowBytes;

  // Block-aligned window (block_tokens = Bs > 0): the query at position n - 1 attends, besides the sink,
  // the tokens j with floor((n-1)/Bs) - floor(j/Bs) < W/Bs.  The ring holds the last W tokens, up to
  // Bs - 1 more: those oldest ones occupy ex_cnt consecutive (cyclic) ring slots from ring offset ex0
  // and are masked out of the scores (they are still streamed with their tiles).
  int ex0 = 0, ex_cnt = 0;
  const int ring_w = a.C - a.sink;
  if (a.block_tokens > 0) {
    const int64_t n = a.n_tokens[b];
    if (n > a.C) {                                  // before the ring has wrapped nothing is left out
      const int64_t first_held = n - ring_w;        // oldest window token in the ring (>= sink here)
      const int64_t first_kept = ((n - 1) / a.block_tokens - ring_w / a.block_tokens + 1) * a.block_tokens;
      if (first_kept > first_held) {
        ex_cnt = static_cast<int>(first_kept - first_held);
        ex0 = static_cast<int>((first_held - a.sink) % ring_w);
      }
    }
  }
  auto attended = [&](int slot) {
    if (slot >= nvalid) return false;
    if (ex_cnt == 0 || slot < a.sink) return true;
    int d = slot - a.sink - ex0;
    if (d < 0) d += ring_w;
    return d >= ex_cnt;
  };

  auto issue_tile = [&](int t) {
    const int stage = (t - t_begin) % kDecStages;
    const uint32_t sk = wsm_u32 + stage * 2 * kTileBytes, sv = sk + kTileBytes;
    const int slot0 = t * kDecTile;
#pragma unroll
    for (int it = 0; it < kCopiesPerLane; ++it) {
      const int ch = it * 32 + lane;
      const int row = ch / kChunks, cc = ch % kChunks;
      const bool valid = slot0 + row < nvalid;
      const int64_t goff = static_cast<int64_t>(valid ? slot0 + row : 0) * kRowBytes + cc * 16;
      const uint32_t soff = row * kRowBytes + ((cc ^ (row & 7)) * 16);
      cp_async16(sk + soff, kbase + goff, valid);
      cp_async16(sv + soff, vbase + goff, valid);
    }
  };

  // Q^T fragments: b0 = Q[head r][16k + 2c, +1], b1 = Q[head r][16k + 8 + 2c, +1]
  uint32_t qf[D / 16][2];
  {
    const int head = hg * kDecHeads + r;
    const bool on = head < a.G;
    const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
        a.q + (static_cast<int64_t>(b) * a.Hq + kvh * a.G + (on ? head : 0)) * D);
#pragma unroll
    for (int k = 0; k < D / 16; ++k) {
      qf[k][0] = on ? qrow[8 * k + c] : 0u;
      qf[k][1] = on ? qrow[8 * k + 4 + c] : 0u;
    }
  }

  float m_run[2] = {-INFINITY, -INFINITY};   // heads 2c, 2c+1 (scaled log2 domain), warp-uniform per head
  float l_run[2] = {0.f, 0.f};               // this thread's share of the row sums
  float oacc[D / 16][4];
#pragma unroll
  for (int i = 0; i < D / 16; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;

#pragma unroll
  for (int s = 0; s < kDecStages - 1; ++s) {
    if (t_begin + s < t_end) issue_tile(t_begin + s);
    cp_async_commit();
  }

  for (int t = t_begin; t < t_end; ++t) {
    cp_async_wait<kDecStages - 2>();
    __syncwarp();
    const int stage = (t - t_begin) % kDecStages;
    const uint32_t sk = wsm_u32 + stage * 2 * kTileBytes, sv = sk + kTileBytes;

    // ---- S^T[16 tokens, 8 heads] = K Q^T ------------------------------------------------
    float sacc[4] = {0.f, 0.f, 0.f, 0.f};
    {
      const int row = ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
      for (int k = 0; k < D / 16; ++k) {
        const int cc = 2 * k + (lane >> 4);
        uint32_t a0, a1, a2, a3;
        ldsm_x4(sk + row * kRowBytes + ((cc ^ (row & 7)) * 16), a0, a1, a2, a3);
        mma16816(sacc, a0, a1, a2, a3, qf[k][0], qf[k][1]);
      }
    }
    // sacc[0,1]: token r, heads 2c, 2c+1;  sacc[2,3]: token r + 8
    const int tok0 = t * kDecTile + r;
    const bool v0 = attended(tok0), v1 = attended(tok0 + 8);
    float s00 = v0 ? sacc[0] * a.scale_log2 : -INFINITY, s01 = v0 ? sacc[1] * a.scale_log2 : -INFINITY;
    float s10 = v1 ? sacc[2] * a.scale_log2 : -INFINITY, s11 = v1 ? sacc[3] * a.scale_log2 : -INFINITY;
    float mx0 = fmaxf(s00, s10), mx1 = fmaxf(s01, s11);
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
    }
    const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);
    const float mu0 = mn0 == -INFINITY ? 0.f : mn0, mu1 = mn1 == -INFINITY ? 0.f : mn1;
    const float al0 = fast_exp2(m_run[0] - mu0), al1 = fast_exp2(m_run[1] - mu1);
    m_run[0] = mn0; m_run[1] = mn1;
    const float p00 = fast_exp2(s00 - mu0), p01 = fast_exp2(s01 - mu1);
    const float p10 = fast_exp2(s10 - mu0), p11 = fast_exp2(s11 - mu1);
    l_run[0] = l_run[0] * al0 + p00 + p10;
    l_run[1] = l_run[1] * al1 + p01 + p11;
    if (__any_sync(0xffffffffu, al0 != 1.f || al1 != 1.f)) {
#pragma unroll
      for (int i = 0; i < D / 16; ++i) {
        oacc[i][0] *= al0; oacc[i][1] *= al1; oacc[i][2] *= al0; oacc[i][3] *= al1;
      }
    }
    // P^T as the B operand: transpose the two 8x8 (token x head) fragments across the warp
    const uint32_t pb0 = movmatrix_t(pack_bf16(p00, p01));   // tokens 2c, 2c+1 of head r
    const uint32_t pb1 = movmatrix_t(pack_bf16(p10, p11));   // tokens 8 + 2c, +1

    // ---- O^T[D, 8 heads] += V^T P^T ----------------------------------------------------
    {
      const int row = (lane >> 4) * 8 + (lane & 7);
#pragma unroll
      for (int i = 0; i < D / 16; ++i) {
        const int cc = 2 * i + ((lane >> 3) & 1);
        uint32_t a0, a1, a2, a3;
        ldsm_x4_t(sv + row * kRowBytes + ((cc ^ (row & 7)) * 16), a0, a1, a2, a3);
        mma16816(oacc[i], a0, a1, a2, a3, pb0, pb1);
      }
    }
    __syncwarp();
    if (t + kDecStages - 1 < t_end) issue_tile(t + kDecStages - 1);
    cp_async_commit();
  }
  cp_async_wait<0>();

  // ---- warp partial -> shared, then merge the warps in warp order.  `direct`: this segment is the
  // whole unit, so the merged result is final and goes straight to o / lse; otherwise it is the
  // CTA's record for the cross-CTA merge ------------------------------------------------------
#pragma unroll
  for (int o = 4; o < 32; o <<= 1) {
    l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], o);
    l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], o);
  }
  __syncthreads();                       // everyone is done with the pipeline buffers
  float* red = reinterpret_cast<float*>(dsmem);          // [warp][head 8][D + 2]
  constexpr int kRec = D + 2;
  {
    float* mine = red + warp * kDecHeads * kRec;
#pragma unroll
    for (int i = 0; i < D / 16; ++i) {
      mine[(2 * c) * kRec + 16 * i + r] = oacc[i][0];
      mine[(2 * c + 1) * kRec + 16 * i + r] = oacc[i][1];
      mine[(2 * c) * kRec + 16 * i + 8 + r] = oacc[i][2];
      mine[(2 * c + 1) * kRec + 16 * i + 8 + r] = oacc[i][3];
    }
    if (r == 0) {
      mine[(2 * c) * kRec + D] = m_run[0];
      mine[(2 * c) * kRec + D + 1] = l_run[0];
      mine[(2 * c + 1) * kRec + D] = m_run[1];
      mine[(2 * c + 1) * kRec + D + 1] = l_run[1];
    }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < kDecHeads * D; idx += blockDim.x) {
    const int head = idx / D, d = idx % D;
    float m = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) m = fmaxf(m, red[(w * kDecHeads + head) * kRec + D]);
    const float mu = m == -INFINITY ? 0.f : m;
    float acc = 0.f, l = 0.f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) {
      const float f = fast_exp2(red[(w * kDecHeads + head) * kRec + D] - mu);
      acc += f * red[(w * kDecHeads + head) * kRec + d];
      l += f * red[(w * kDecHeads + head) * kRec + D + 1];
    }
    if (direct) {
      const int gh = hg * kDecHeads + head;
      if (gh < a.G) {
        const int64_t qh = static_cast<int64_t>(b) * a.Hq + kvh * a.G + gh;
        a.o[qh * D + d] = __float2bfloat16(l > 0.f ? acc / l : 0.f);
        if (d == 0 && a.lse) a.lse[qh] = l > 0.f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
      }
    } else {
      out[head * kRec + d] = acc;
      if (d == 0) { out[head * kRec + D] = m; out[head * kRec + D + 1] = l; }
    }
  }
}

template <int D>
__global__ void __launch_bounds__(kDecWarps * 32) decode_split_kernel(const DecodeArgs a) {
  extern __shared__ __align__(128) uint8_t dsmem[];
  const int warp = threadIdx.x >> 5;
  const int split = blockIdx.x, kg = blockIdx.y, b = blockIdx.z;
  const int kvh = kg / a.HG, hg = kg % a.HG;
  const int64_t n = a.n_tokens[b];
  const int nvalid = static_cast<int>(n < a.C ? (n < 0 ? 0 : n) : a.C);
  const int ntile = (nvalid + kDecTile - 1) / kDecTile;
  const int wg = split * kDecWarps + warp, nw = a.nsplit * kDecWarps;
  const int t_begin = static_cast<int>(static_cast<int64_t>(ntile) * wg / nw);
  const int t_end = static_cast<int>(static_cast<int64_t>(ntile) * (wg + 1) / nw);
  constexpr int kRec = D + 2;
  float* out = a.part + ((static_cast<int64_t>(b) * gridDim.y + kg) * a.nsplit + split) * (kDecHeads * kRec);
  decode_run_segment<D>(a, dsmem, b, kvh, hg, nvalid, t_begin, t_end, out, false);
}

// ---- flattened schedule ---------------------------------------------------------------------
// The tiles of all (sequence, kv head, head group) units form one sequence, unit after unit
// (sequence-major); CTA c of N streams the slice [T c / N, T (c + 1) / N) of it, so every CTA
// moves the same number of bytes whatever the mix of sequence lengths, and one wave of CTAs
// covers the whole cache.  A slice that crosses a unit boundary is processed in segments; the
// record of (CTA c, unit u) lives at index c + u, which grows strictly along the sequence.
constexpr int kDecFlatMaxB = 2048;      // sequences the flattened path supports (prefix array in shared memory)
constexpr int kDecFlatMaxCtas = 320;    // upper bound of its grid (two CTAs per SM)

__device__ __forceinline__ int decode_tiles_of(const DecodeArgs& a, int b) {
  const int64_t n = a.n_tokens[b];
  const int nvalid = static_cast<int>(n < a.C ? (n < 0 ? 0 : n) : a.C);
  return (nvalid + kDecTile - 1) / kDecTile;
}

// cum[b] = tiles of the sequences before b, b = 0 .. B (block of kDecThreads threads; ends with a barrier)
__device__ __forceinline__ void decode_build_cum(const DecodeArgs& a, int* cum) {
  __shared__ int warp_sum[kDecWarps];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ipt = (a.B + kDecThreads - 1) / kDecThreads;
  const int b0 = tid * ipt;
  int local = 0;
  for (int i = 0; i < ipt; ++i)
    if (b0 + i < a.B) local += decode_tiles_of(a, b0 + i);
  int incl = local;
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) warp_sum[warp] = incl;
  __syncthreads();
  int run = incl - local;
  for (int w = 0; w < warp; ++w) run += warp_sum[w];
  for (int i = 0; i < ipt; ++i)
    if (b0 + i < a.B) { cum[b0 + i] = run; run += decode_tiles_of(a, b0 + i); }
  if (tid == kDecThreads - 1) cum[a.B] = run;   // the last thread's running total is the grand total
  __syncthreads();
}

// Merge the records of unit (b, k): CTAs first_cta .. first_cta + n_rec - 1, in that order
// (whichever CTA happens to run this, the summation order is the same).  kDecThreads threads.
template <int D>
__device__ __forceinline__ void decode_merge_unit(const DecodeArgs& a, int b, int k, int64_t u, int first_cta,
                                                  int n_rec, int64_t total, int n_cta) {
  constexpr int kRec = D + 2;
  const int kvh = k / a.HG, hg = k % a.HG;
  const float* recs = a.part + (static_cast<int64_t>(first_cta) + u) * (kDecHeads * kRec);
  // a CTA with an empty slice (possible only with fewer tiles than CTAs) wrote no record
  const bool sparse_slices = total < n_cta;
  auto empty_slice = [&](int c) { return total * c / n_cta == total * (c + 1) / n_cta; };
  // Each thread owns kOut outputs (all handled together so that the loads of one record are in
  // flight at once: the records sit in L2 and a dependent chain of loads would dominate).
  constexpr int kOut = kDecHeads * D / kDecThreads;
  int head[kOut], dd[kOut];
  float m[kOut], acc[kOut], l[kOut];
#pragma unroll
  for (int j = 0; j < kOut; ++j) {
    const int idx = threadIdx.x + j * kDecThreads;
    head[j] = idx / D;
    dd[j] = idx % D;
    m[j] = -INFINITY;
    acc[j] = 0.f;
    l[j] = 0.f;
  }
  for (int i = 0; i < n_rec; ++i) {
    if (sparse_slices && empty_slice(first_cta + i)) continue;
#pragma unroll
    for (int j = 0; j < kOut; ++j) m[j] = fmaxf(m[j], __ldcg(recs + (i * kDecHeads + head[j]) * kRec + D));
  }
  for (int i = 0; i < n_rec; ++i) {
    if (sparse_slices && empty_slice(first_cta + i)) continue;
    float rm[kOut], rl[kOut], ro[kOut];
#pragma unroll
    for (int j = 0; j < kOut; ++j) {
      const float* rec = recs + (i * kDecHeads + head[j]) * kRec;
      rm[j] = __ldcg(rec + D);
      rl[j] = __ldcg(rec + D + 1);
      ro[j] = __ldcg(rec + dd[j]);
    }
#pragma unroll
    for (int j = 0; j < kOut; ++j) {
      const float f = fast_exp2(rm[j] - (m[j] == -INFINITY ? 0.f : m[j]));
      acc[j] += f * ro[j];
      l[j] += f * rl[j];
    }
  }
#pragma unroll
  for (int j = 0; j < kOut; ++j) {
    const int gh = hg * kDecHeads + head[j];
    if (gh >= a.G) continue;
    const int64_t qh = static_cast<int64_t>(b) * a.Hq + kvh * a.G + gh;
    a.o[qh * D + dd[j]] = __float2bfloat16(l[j] > 0.f ? acc[j] / l[j] : 0.f);
    if (dd[j] == 0 && a.lse) a.lse[qh] = l[j] > 0.f ? (m[j] + log2f(l[j])) * 0.6931471805599453f : -INFINITY;
  }
}

template <int D>
__global__ void __launch_bounds__(kDecWarps * 32) decode_stream_kernel(const DecodeArgs a) {
  extern __shared__ __align__(128) uint8_t dsmem[];
  constexpr int kPipeBytes = kDecWarps * kDecStages * 2 * kDecTile * D * 2;
  constexpr int kRec = D + 2;
  int* cum = reinterpret_cast<int*>(dsmem + kPipeBytes);
  decode_build_cum(a, cum);
  const int ups = a.Hkv * a.HG;
  const int64_t total = static_cast<int64_t>(cum[a.B]) * ups;
  __shared__ int s_merge[3];
  auto start_of = [&](int64_t c) { return total * c / gridDim.x; };
  auto cta_of = [&](int64_t f) {           // the CTA whose slice holds tile f
    int64_t c = f * gridDim.x / total;
    while (c + 1 < gridDim.x && start_of(c + 1) <= f) ++c;
    while (c > 0 && start_of(c) > f) --c;
    return static_cast<int>(c);
  };
  // units of sequences without tokens get their (empty) result here, spread over the CTAs
  for (int e = 0; e < a.B; ++e) {
    if (cum[e + 1] != cum[e]) continue;
    for (int k = 0; k < ups; ++k) {
      const int64_t u = static_cast<int64_t>(e) * ups + k;
      if (u % gridDim.x == blockIdx.x) decode_merge_unit<D>(a, e, k, u, 0, 0, total, gridDim.x);
    }
  }
  const int64_t f0 = start_of(blockIdx.x), f1 = start_of(blockIdx.x + 1);
  if (f0 >= f1) return;
  int lo = 0, hi = a.B;   // cum[lo] * ups <= f0 < cum[hi] * ups
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (static_cast<int64_t>(cum[mid]) * ups <= f0) lo = mid; else hi = mid;
  }
  int b = lo;
  const int warp = threadIdx.x >> 5;
  int64_t pos = f0;
  while (pos < f1) {
    while (static_cast<int64_t>(cum[b + 1]) * ups <= pos) ++b;          // skip finished / empty sequences
    const int nt = cum[b + 1] - cum[b];
    const int64_t rel = pos - static_cast<int64_t>(cum[b]) * ups;
    const int k = static_cast<int>(rel / nt), t0 = static_cast<int>(rel - static_cast<int64_t>(k) * nt);
    const int n = static_cast<int>(min(static_cast<int64_t>(nt - t0), f1 - pos));
    const int64_t nn = a.n_tokens[b];
    const int nvalid = static_cast<int>(nn < a.C ? (nn < 0 ? 0 : nn) : a.C);
    const int tb = t0 + static_cast<int>(static_cast<int64_t>(n) * warp / kDecWarps);
    const int te = t0 + static_cast<int>(static_cast<int64_t>(n) * (warp + 1) / kDecWarps);
    const int64_t u = static_cast<int64_t>(b) * ups + k;
    __syncthreads();   // the previous segment's merge is done with shared memory
    const bool direct = (t0 == 0 && n == nt);   // my segment is the whole unit: no record, no ticket
    decode_run_segment<D>(a, dsmem, b, k / a.HG, k % a.HG, nvalid, tb, te,
                          a.part + (blockIdx.x + u) * (kDecHeads * kRec), direct);
    pos += n;
    if (direct) continue;
    // The CTA that delivers the last record of a unit merges it (records are read in index
    // order, so the result does not depend on which CTA that is) and re-arms the counter.
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
      const int64_t first = static_cast<int64_t>(cum[b]) * ups + static_cast<int64_t>(k) * nt;
      const int c_lo = (t0 == 0) ? static_cast<int>(blockIdx.x) : cta_of(first);
      const int c_hi = (t0 + n == nt) ? static_cast<int>(blockIdx.x) : cta_of(first + nt - 1);
      int pieces = c_hi - c_lo + 1;
      if (total < gridDim.x)
        for (int c = c_lo; c <= c_hi; ++c) pieces -= (start_of(c) == start_of(c + 1)) ? 1 : 0;
      const unsigned ticket = atomicAdd(a.unit_count + u, 1u);
      s_merge[0] = (ticket + 1u == static_cast<unsigned>(pieces)) ? 1 : 0;
      s_merge[1] = c_lo;
      s_merge[2] = c_hi - c_lo + 1;
    }
    __syncthreads();
    if (s_merge[0]) {
      __threadfence();
      decode_merge_unit<D>(a, b, k, u, s_merge[1], s_merge[2], total, gridDim.x);
      if (threadIdx.x == 0) a.unit_count[u] = 0u;
    }
  }
}

// grid = (B * Hkv * HG); 128 threads.  Merges the splits in ascending order.
template <int D>
__global__ void __launch_bounds__(128) decode_merge_kernel(const DecodeArgs a) {
  constexpr int kRec = D + 2;
  const int kg = blockIdx.x % (a.Hkv * a.HG), b = blockIdx.x / (a.Hkv * a.HG);
  const int kvh = kg / a.HG, hg = kg % a.HG;
  const float* part = a.part + (static_cast<int64_t>(b) * (a.Hkv * a.HG) + kg) * a.nsplit * (kDecHeads * kRec);
  for (int idx = threadIdx.x; idx < kDecHeads * D; idx += blockDim.x) {
    const int head = idx / D, d = idx % D;
    const int gh = hg * kDecHeads + head;
    if (gh >= a.G) continue;
    float m = -INFINITY;
    for (int s = 0; s < a.nsplit; ++s) m = fmaxf(m, part[(s * kDecHeads + head) * kRec + D]);
    const float mu = m == -INFINITY ? 0.f : m;
    float acc = 0.f, l = 0.f;
    for (int s = 0; s < a.nsplit; ++s) {
      const float f = fast_exp2(part[(s * kDecHeads + head) * kRec + D] - mu);
      acc += f * part[(s * kDecHeads + head) * kRec + d];
      l += f * part[(s * kDecHeads + head) * kRec + D + 1];
    }
    const int64_t qh = static_cast<int64_t>(b) * a.Hq + kvh * a.G + gh;
    a.o[qh * D + d] = __float2bfloat16(l > 0.f ? acc / l : 0.f);
    if (d == 0 && a.lse) a.lse[qh] = l > 0.f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
  }
}

// ---- ring append ------------------------------------------------------------------------
// slot(j) = j < sink ? j : sink + (j - sink) % window.  One group of D/8 threads copies one
// K row and one V row (16 bytes per thread per row).  A token that a later token of the same
// call would overwrite is skipped, so the outcome equals appending one at a time.
__global__ void ring_append_kernel(__nv_bfloat16* k_cache, __nv_bfloat16* v_cache, const __nv_bfloat16* k_new,
                                   const __nv_bfloat16* v_new, const int64_t* n_before, int B, int Hkv, int D, int T,
                                   int sink, int window) {
  const int per_row = D / 8;
  const int64_t gid = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t row_id = gid / per_row;
  const int ch = static_cast<int>(gid % per_row);
  const int64_t total_rows = static_cast<int64_t>(B) * Hkv * T;
  if (row_id >= total_rows) return;
  const int t = static_cast<int>(row_id % T);
  const int64_t bh = row_id / T;
  const int b = static_cast<int>(bh / Hkv);
  const int64_t n0 = n_before[b];
  if (n0 < 0) return;                                  // a negative count addresses nothing: the sequence is skipped
  const int64_t j = n0 + t, last = n0 + T - 1;
  if (j >= sink && j + window <= last) return;       // overwritten later in this call
  const int64_t slot = j < sink ? j : sink + (j - sink) % window;
  const int64_t C = static_cast<int64_t>(sink) + window;
  const uint4* ks = reinterpret_cast<const uint4*>(k_new + row_id * D) + ch;
  const uint4* vs = reinterpret_cast<const uint4*>(v_new + row_id * D) + ch;
  uint4* kd = reinterpret_cast<uint4*>(k_cache + (bh * C + slot) * D) + ch;
  uint4* vd = reinterpret_cast<uint4*>(v_cache + (bh * C + slot) * D) + ch;
  *kd = *ks;
  *vd = *vs;
}

static lg_status check_decode(const lg_decode_params* p) {
  if (!p) return LG_ERR_INVALID_ARG;
  if (p->B < 1 || p->Hq < 1 || p->Hkv < 1 || p->Hq % p->Hkv != 0) return LG_ERR_INVALID_ARG;
  if (p->sink_tokens < 0 || p->window_tokens < 1) return LG_ERR_INVALID_ARG;
  if (p->block_tokens < 0) return LG_ERR_INVALID_ARG;
  if (p->block_tokens > 0 && (p->window_tokens % p->block_tokens != 0 || p->sink_tokens % p->block_tokens != 0))
    return LG_ERR_INVALID_ARG;                         // the block-aligned window counts whole blocks
  if (!(p->scale >= 0.f) || isinf(p->scale)) return LG_ERR_INVALID_ARG;
  if (p->D != 64 && p->D != 128) return LG_ERR_UNSUPPORTED;
  if (static_cast<int64_t>(p->sink_tokens) + p->window_tokens > (1ll << 30)) return LG_ERR_UNSUPPORTED;
  return LG_OK;
}

// Number of KV splits: enough CTAs to fill the machine a few times over, but at least
// 4 tiles of work per warp.
static int choose_nsplit(const lg_decode_params* p) {
  const int C = p->sink_tokens + p->window_tokens;
  const int HG = (p->Hq / p->Hkv + kDecHeads - 1) / kDecHeads;
  const int64_t units = static_cast<int64_t>(p->B) * p->Hkv * HG;
  const int64_t tiles = (C + kDecTile - 1) / kDecTile;
  int64_t max_by_work = tiles / (kDecWarps * 4);
  if (max_by_work < 1) max_by_work = 1;
  int64_t want = (148 * 2 * 2 + units - 1) / units;    // about two waves of two CTAs per SM
  if (want < 1) want = 1;
  int64_t ns = want < max_by_work ? want : max_by_work;
  if (ns > 256) ns = 256;
  return static_cast<int>(ns);
}

// Batches of up to kDecFlatMaxB sequences take the flattened one-wave schedule.
static bool decode_is_flat(const lg_decode_params* p) { return p->B <= kDecFlatMaxB; }

// What a decode call needs to know about its device, looked up once per device: the SM count, and
// that the streaming kernels may use their large dynamic shared memory.  (A serving loop makes this call
// every 50 microseconds; the runtime queries cost a noticeable part of that on the host.)
namespace {
constexpr int kMaxDecodeDevices = 64;
struct DecodeDeviceInfo { int sms = 0; bool ready = false; };
DecodeDeviceInfo g_decode_dev[kMaxDecodeDevices];
std::mutex g_decode_dev_mutex;

lg_status decode_device_info(int* sms_out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return LG_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDecodeDevices) return LG_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_decode_dev_mutex);
  DecodeDeviceInfo& d = g_decode_dev[dev];
  if (!d.ready) {
    const lg_status arch = check_arch();                     // the kernels are built for sm_100a only
    if (arch != LG_OK) return arch;
    if (cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return LG_ERR_CUDA;
    // the most dynamic shared memory a launch of each kernel can ask for: the tile pipelines of the
    // warps, plus (flattened schedule) the prefix array of the largest batch it takes
    auto pipe = [](int D) { return kDecWarps * kDecStages * 2 * kDecTile * D * 2; };
    const int cum = (kDecFlatMaxB + 1) * static_cast<int>(sizeof(int));
    if (cudaFuncSetAttribute(decode_stream_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, pipe(128) + cum) != cudaSuccess ||
        cudaFuncSetAttribute(decode_stream_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, pipe(64) + cum) != cudaSuccess ||
        cudaFuncSetAttribute(decode_split_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, pipe(128)) != cudaSuccess ||
        cudaFuncSetAttribute(decode_split_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, pipe(64)) != cudaSuccess)
      return LG_ERR_CUDA;
    d.ready = true;
  }
  *sms_out = d.sms;
  return LG_OK;
}
}  // namespace

static size_t decode_part_bytes(const lg_decode_params* p, int nsplit) {
  const int HG = (p->Hq / p->Hkv + kDecHeads - 1) / kDecHeads;
  return static_cast<size_t>(p->B) * p->Hkv * HG * nsplit * kDecHeads * (p->D + 2) * sizeof(float);
}

}  // namespace lg

using namespace lg;

extern "C" {

lg_status lg_kv_ring_append(const lg_decode_params* p, void* k_cache, void* v_cache, const void* k_new,
                            const void* v_new, int32_t T_new, const int64_t* n_tokens_before, void* stream) {
  LG_RANGE("lg_kv_ring_append");
  lg_status s = check_decode(p);
  if (s != LG_OK) return s;
  if (T_new < 0) return LG_ERR_INVALID_ARG;
  if (T_new == 0) return LG_OK;
  if (!k_cache || !v_cache || !k_new || !v_new || !n_tokens_before) return LG_ERR_INVALID_ARG;
  if (!aligned16(k_cache) || !aligned16(v_cache) || !aligned16(k_new) || !aligned16(v_new) ||
      (reinterpret_cast<uintptr_t>(n_tokens_before) & 7))
    return LG_ERR_INVALID_ARG;
  const int64_t threads = static_cast<int64_t>(p->B) * p->Hkv * T_new * (p->D / 8);
  const int64_t blocks = (threads + 255) / 256;
  if (blocks > 0x7fffffff) return LG_ERR_UNSUPPORTED;
  ring_append_kernel<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<__nv_bfloat16*>(k_cache), static_cast<__nv_bfloat16*>(v_cache),
      static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new), n_tokens_before, p->B,
      p->Hkv, p->D, T_new, p->sink_tokens, p->window_tokens); note_launch();
  return cudaGetLastError() == cudaSuccess ? LG_OK : LG_ERR_CUDA;
}

size_t lg_sparse_decode_workspace_bytes(const lg_decode_params* p) {
  if (check_decode(p) != LG_OK) return 0;
  if (decode_is_flat(p)) {   // one record per (CTA, unit) pair that can occur: index CTA + unit
    const int HG = (p->Hq / p->Hkv + kDecHeads - 1) / kDecHeads;
    const size_t units = static_cast<size_t>(p->B) * p->Hkv * HG;
    const size_t records = static_cast<size_t>(kDecFlatMaxCtas) + units;
    return sizeof(WsHeader) + align_up(units * sizeof(unsigned int), 256) +
           align_up(records * kDecHeads * (p->D + 2) * sizeof(float), 256);
  }
  return sizeof(WsHeader) + align_up(decode_part_bytes(p, choose_nsplit(p)), 256);
}

lg_status lg_sparse_decode_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  LG_RANGE("lg_sparse_decode_workspace_init");
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255)) return LG_ERR_INVALID_ARG;
  return cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream)) == cudaSuccess ? LG_OK
                                                                                                           : LG_ERR_CUDA;
}

lg_status lg_sparse_decode(const lg_decode_params* p, const void* q, const void* k_cache, const void* v_cache,
                           const int64_t* n_tokens, void* o, float* lse, void* workspace, size_t workspace_bytes,
                           void* stream) {
  LG_RANGE("lg_sparse_decode");
  lg_status s = check_decode(p);
  if (s != LG_OK) return s;
  if (!q || !k_cache || !v_cache || !n_tokens || !o || !workspace) return LG_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(o) ||
      (reinterpret_cast<uintptr_t>(n_tokens) & 7) || (reinterpret_cast<uintptr_t>(lse) & 3) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255))
    return LG_ERR_INVALID_ARG;
  if (workspace_bytes < lg_sparse_decode_workspace_bytes(p)) return LG_ERR_WORKSPACE;
  int sms = 0;
  if ((s = decode_device_info(&sms)) != LG_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  DecodeArgs a;
  a.q = static_cast<const __nv_bfloat16*>(q);
  a.k_cache = static_cast<const __nv_bfloat16*>(k_cache);
  a.v_cache = static_cast<const __nv_bfloat16*>(v_cache);
  a.n_tokens = n_tokens;
  a.part = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + sizeof(WsHeader));
  a.o = static_cast<__nv_bfloat16*>(o);
  a.lse = lse;
  a.Hq = p->Hq; a.Hkv = p->Hkv; a.G = p->Hq / p->Hkv;
  a.HG = (a.G + kDecHeads - 1) / kDecHeads;
  a.C = p->sink_tokens + p->window_tokens;
  a.sink = p->sink_tokens;
  a.block_tokens = p->block_tokens;
  a.nsplit = choose_nsplit(p);
  const float scale = p->scale > 0.f ? p->scale : 1.0f / sqrtf(static_cast<float>(p->D));
  a.scale_log2 = scale * 1.4426950408889634f;
  a.B = p->B;
  if (decode_is_flat(p)) {
    // as many CTAs per SM as shared memory allows (at most two), fewer when the cache is too small to
    // give each warp a couple of tiles
    const int64_t units = static_cast<int64_t>(p->B) * a.Hkv * a.HG;
    const int64_t max_tiles = units * ((a.C + kDecTile - 1) / kDecTile);
    int64_t n_cta = (max_tiles + 2 * kDecWarps - 1) / (2 * kDecWarps);
    const int64_t pipe_bytes = static_cast<int64_t>(kDecWarps) * kDecStages * 2 * kDecTile * p->D * 2;
    const int per_sm = pipe_bytes * 2 + 4096 <= 227 * 1024 ? 2 : 1;
    if (n_cta > per_sm * sms) n_cta = per_sm * sms;
    if (n_cta > kDecFlatMaxCtas) n_cta = kDecFlatMaxCtas;
    // A whole number of CTAs per unit when that costs at most a quarter of the CTAs: with equal
    // lengths every slice then lies inside one unit (one pipeline fill, one record, one ticket per
    // CTA instead of two); with mixed lengths the slices fall where they fall, as before.
    if (units > 0 && n_cta > units && (n_cta / units) * units * 4 >= n_cta * 3) n_cta = (n_cta / units) * units;
    if (n_cta < 1) n_cta = 1;
    if (units > 0x7fffffff) return LG_ERR_UNSUPPORTED;
    // header word and per-unit counters are zero on entry (the caller zero-filled the workspace once,
    // and the CTA that merges a unit re-arms its counter); the records follow them
    const size_t count_bytes = align_up(static_cast<size_t>(units) * sizeof(unsigned int), 256);
    a.unit_count = reinterpret_cast<unsigned int*>(static_cast<uint8_t*>(workspace) + sizeof(WsHeader));
    a.part = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + sizeof(WsHeader) + count_bytes);
    const int smem_flat = kDecWarps * kDecStages * 2 * kDecTile * p->D * 2 + (p->B + 1) * static_cast<int>(sizeof(int));
    if (p->D == 128) {
      decode_stream_kernel<128><<<static_cast<unsigned>(n_cta), kDecWarps * 32, smem_flat, st>>>(a); note_launch();
    } else {
      decode_stream_kernel<64><<<static_cast<unsigned>(n_cta), kDecWarps * 32, smem_flat, st>>>(a); note_launch();
    }
    return cudaGetLastError() == cudaSuccess ? LG_OK : LG_ERR_CUDA;
  }
  if (a.Hkv * a.HG > 65535 || p->B > 65535) return LG_ERR_UNSUPPORTED;
  if (cudaMemsetAsync(workspace, 0, sizeof(WsHeader), st) != cudaSuccess) return LG_ERR_CUDA;
  dim3 grid(a.nsplit, a.Hkv * a.HG, p->B);
  const int smem = kDecWarps * kDecStages * 2 * kDecTile * p->D * 2;
  if (p->D == 128) {
    decode_split_kernel<128><<<grid, kDecWarps * 32, smem, st>>>(a); note_launch();
    decode_merge_kernel<128><<<p->B * a.Hkv * a.HG, 128, 0, st>>>(a); note_launch();
  } else {
    decode_split_kernel<64><<<grid, kDecWarps * 32, smem, st>>>(a); note_launch();
    decode_merge_kernel<64><<<p->B * a.Hkv * a.HG, 128, 0, st>>>(a); note_launch();
  }
  return cudaGetLastError() == cudaSuccess ? LG_OK : LG_ERR_CUDA;
}

// ---- decode without any allocation ------------------------------------------------------
// Scratch for lg_sparse_decode_static: lives in the library image, one copy per GPU that
// loads it.  In host code this name is only a handle; the device address comes from
// cudaGetSymbolAddress, looked up once per device below.
static __device__ __align__(256) unsigned char g_decode_static_scratch[LG_DECODE_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxStaticDevices = 64;
void* g_static_scratch_addr[kMaxStaticDevices];   // device address per device ordinal, 0 = not looked up yet
std::mutex g_static_scratch_mutex;

// Device address of the scratch array on the CURRENT device (looked up on first use).
lg_status static_scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return LG_ERR_CUDA;
  if (dev < 0 || dev >= kMaxStaticDevices) return LG_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (!g_static_scratch_addr[dev]) {
    void* addr = nullptr;
    if (cudaGetSymbolAddress(&addr, g_decode_static_scratch) != cudaSuccess || !addr) return LG_ERR_CUDA;
    g_static_scratch_addr[dev] = addr;
  }
  *out = g_static_scratch_addr[dev];
  return LG_OK;
}
}  // namespace

lg_status lg_sparse_decode_static(const lg_decode_params* p, const void* q, const void* k_cache,
                                  const void* v_cache, const int64_t* n_tokens, void* o, float* lse,
                                  void* stream) {
  LG_RANGE("lg_sparse_decode_static");
  lg_status s = check_decode(p);
  if (s != LG_OK) return s;
  // the split partials of this problem must fit the fixed array
  if (lg_sparse_decode_workspace_bytes(p) > static_cast<size_t>(LG_DECODE_STATIC_SCRATCH_BYTES))
    return LG_ERR_WORKSPACE;
  void* scratch = nullptr;
  if ((s = static_scratch_address(&scratch)) != LG_OK) return s;
  // Same kernels as lg_sparse_decode, with the array as their workspace: a static array starts
  // zero-filled, and every call leaves its counters at zero again.
  return lg_sparse_decode(p, q, k_cache, v_cache, n_tokens, o, lse, scratch, LG_DECODE_STATIC_SCRATCH_BYTES,
                          stream);
}

lg_status lg_sparse_decode_static_reset(void* stream) {
  LG_RANGE("lg_sparse_decode_static_reset");
  void* scratch = nullptr;
  lg_status s = static_scratch_address(&scratch);
  if (s != LG_OK) return s;
  return cudaMemsetAsync(scratch, 0, LG_DECODE_STATIC_SCRATCH_BYTES, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? LG_OK
             : LG_ERR_CUDA;
}

}  // extern "C"
