// Block-index builder: CSR / CSC lists of active blocks of the static pattern (paper
// Section 3.2: the mask lives in compressed-sparse-row form and is the same for all heads),
// plus the per-tile schedules the attention kernels walk.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "lg_pattern.h"

namespace lg {

// ---- pass 1: per-row and per-column counts -------------------------------------------
// grid = nB blocks of 128 threads; block b counts row b and column b.
__global__ void index_count_kernel(PatternDev p, int32_t* __restrict__ row_ptr, int32_t* __restrict__ col_ptr) {
  const int b = blockIdx.x;
  int rc = 0, cc = 0;
  for (int x = threadIdx.x; x < p.nB; x += blockDim.x) {
    rc += block_active(p, b, x) ? 1 : 0;
    cc += block_active(p, x, b) ? 1 : 0;
  }
  __shared__ int s_r[4], s_c[4];
  for (int o = 16; o > 0; o >>= 1) {
    rc += __shfl_xor_sync(0xffffffffu, rc, o);
    cc += __shfl_xor_sync(0xffffffffu, cc, o);
  }
  if ((threadIdx.x & 31) == 0) { s_r[threadIdx.x >> 5] = rc; s_c[threadIdx.x >> 5] = cc; }
  __syncthreads();
  if (threadIdx.x == 0) {
    row_ptr[b + 1] = s_r[0] + s_r[1] + s_r[2] + s_r[3];
    col_ptr[b + 1] = s_c[0] + s_c[1] + s_c[2] + s_c[3];
  }
}

// ---- pass 2: in-place inclusive scan of ptr[1..n], ptr[0] = 0 (one block, 1024 threads;
// blockIdx.x selects which of the two arrays) ---------------------------------------------
__global__ void index_scan_kernel(int32_t* __restrict__ row_ptr, int32_t* __restrict__ col_ptr, int n) {
  int32_t* ptr = blockIdx.x == 0 ? row_ptr : col_ptr;
  __shared__ int warp_tot[32];
  __shared__ int carry;
  if (threadIdx.x == 0) { carry = 0; ptr[0] = 0; }
  __syncthreads();
  for (int base = 0; base < n; base += 1024) {
    const int i = base + threadIdx.x;
    int v = i < n ? ptr[i + 1] : 0;
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(0xffffffffu, v, o);
      if ((threadIdx.x & 31) >= o) v += t;
    }
    if ((threadIdx.x & 31) == 31) warp_tot[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x < 32) {
      int w = warp_tot[threadIdx.x];
      for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, w, o);
        if (threadIdx.x >= o) w += t;
      }
      warp_tot[threadIdx.x] = w;
    }
    __syncthreads();
    const int prefix = carry + ((threadIdx.x >> 5) ? warp_tot[(threadIdx.x >> 5) - 1] : 0);
    if (i < n) ptr[i + 1] = v + prefix;
    __syncthreads();
    if (threadIdx.x == 0) carry += warp_tot[31];
    __syncthreads();
  }
}

// ---- pass 3: fill.  grid = nB blocks of 64 threads: warp 0 writes row b (ascending kb),
// warp 1 writes column b (ascending qb), by ordered ballot compaction. ---------------------
__global__ void index_fill_kernel(PatternDev p, const int32_t* __restrict__ row_ptr, int32_t* __restrict__ col_idx,
                                  const int32_t* __restrict__ col_ptr, int32_t* __restrict__ row_idx) {
  const int b = blockIdx.x;
  const int lane = threadIdx.x & 31;
  const bool is_row = (threadIdx.x >> 5) == 0;
  int32_t* out = is_row ? col_idx + row_ptr[b] : row_idx + col_ptr[b];
  int written = 0;
  for (int base = 0; base < p.nB; base += 32) {
    const int x = base + lane;
    const bool on = x < p.nB && (is_row ? block_active(p, b, x) : block_active(p, x, b));
    const unsigned m = __ballot_sync(0xffffffffu, on);
    if (on) out[written + __popc(m & ((1u << lane) - 1))] = x;
    written += __popc(m);
  }
}

// ---- tile schedules ---------------------------------------------------------------------
// A tile groups R consecutive pattern rows (or columns).  Its schedule is the ascending
// union of their lists; entry = idx * 4 + member_mask (bit r set: member r of the tile has
// the block).  Entries of tile t start at ptr[R * t]; cnt[t] says how many there are.
// One thread per tile.
__global__ void tile_merge_kernel(const int32_t* __restrict__ ptr, const int32_t* __restrict__ idx, int nB, int R,
                                  int n_tiles, int32_t* __restrict__ tile_cnt, int32_t* __restrict__ tile_ent) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n_tiles) return;
  const int r0 = t * R;
  int32_t* out = tile_ent + ptr[r0];
  int n = 0;
  if (R == 1 || r0 + 1 >= nB) {
    for (int e = ptr[r0]; e < ptr[r0 + 1]; ++e) out[n++] = idx[e] * 4 + 1;
  } else {  // R == 2: merge two ascending lists
    int a = ptr[r0], ae = ptr[r0 + 1], c = ptr[r0 + 1], ce = ptr[r0 + 2];
    while (a < ae || c < ce) {
      const int va = a < ae ? idx[a] : 0x7fffffff;
      const int vc = c < ce ? idx[c] : 0x7fffffff;
      if (va == vc) { out[n++] = va * 4 + 3; ++a; ++c; }
      else if (va < vc) { out[n++] = va * 4 + 1; ++a; }
      else { out[n++] = vc * 4 + 2; ++c; }
    }
  }
  tile_cnt[t] = n;
}

// The same for tiles of up to four pattern rows (the forward's super-tiles of 256 query rows):
// entry = idx * 16 + member mask.
__global__ void tile_merge4_kernel(const int32_t* __restrict__ ptr, const int32_t* __restrict__ idx, int nB, int R,
                                   int n_tiles, int32_t* __restrict__ tile_cnt, int32_t* __restrict__ tile_ent) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n_tiles) return;
  const int r0 = t * R;
  int32_t* out = tile_ent + ptr[r0];
  int cur[4], end[4];
  for (int r = 0; r < 4; ++r) {
    const bool have = r < R && r0 + r < nB;
    cur[r] = have ? ptr[r0 + r] : 0;
    end[r] = have ? ptr[r0 + r + 1] : 0;
  }
  int n = 0;
  for (;;) {
    int lo = 0x7fffffff;
    for (int r = 0; r < 4; ++r)
      if (cur[r] < end[r]) lo = min(lo, idx[cur[r]]);
    if (lo == 0x7fffffff) break;
    int mask = 0;
    for (int r = 0; r < 4; ++r)
      if (cur[r] < end[r] && idx[cur[r]] == lo) { mask |= 1 << r; ++cur[r]; }
    out[n++] = lo * 16 + mask;
  }
  tile_cnt[t] = n;
}

// Launch order: tiles with more work first.  order[rank] = tile; rank by (count desc, tile asc).
__global__ void tile_order_kernel(const int32_t* __restrict__ tile_cnt, int n_tiles, int32_t* __restrict__ order) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n_tiles) return;
  const int c = tile_cnt[t];
  int rank = 0;
  for (int u = 0; u < n_tiles; ++u) {
    const int cu = tile_cnt[u];
    rank += (cu > c || (cu == c && u < t)) ? 1 : 0;
  }
  order[rank] = t;
}

// ---- kv tiles of the dK/dV pass ------------------------------------------------------------
// A kv tile holds R pattern columns (R = 128 / block).  With R = 2 the two columns of a tile
// should have similar lists: a comb column of the strided pattern is attended by every later
// query block and its neighbour by a handful, so pairing neighbours would leave half of every
// MMA idle.  Columns are therefore ranked by list length (longest first, ties by index) and
// consecutive ranks share a tile.  cols[R * t + m] = pattern column of member m (-1: none).
__global__ void kv_tile_cols_kernel(const int32_t* __restrict__ col_ptr, int nB, int R, int n_tiles,
                                    int32_t* __restrict__ cols) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c < n_tiles * R && c >= nB) cols[c] = -1;          // padding member of the last tile
  if (c >= nB) return;
  if (R == 1) { cols[c] = c; return; }
  const int len = col_ptr[c + 1] - col_ptr[c];
  int rank = 0;
  for (int u = 0; u < nB; ++u) {
    const int lu = col_ptr[u + 1] - col_ptr[u];
    rank += (lu > len || (lu == len && u < c)) ? 1 : 0;
  }
  cols[rank] = c;
}

// upper bound of a tile's schedule length, written to off[t + 1] (off[0] = 0) for the scan
__global__ void kv_tile_len_kernel(const int32_t* __restrict__ col_ptr, const int32_t* __restrict__ cols, int R,
                                   int n_tiles, int32_t* __restrict__ off) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n_tiles) return;
  int n = 0;
  for (int m = 0; m < R; ++m) {
    const int c = cols[R * t + m];
    if (c >= 0) n += col_ptr[c + 1] - col_ptr[c];
  }
  off[t + 1] = n;
  if (t == 0) off[0] = 0;
}

// ascending union of the members' CSC lists; entry = query block * 4 + member mask
__global__ void kv_tile_merge_kernel(const int32_t* __restrict__ col_ptr, const int32_t* __restrict__ row_idx,
                                     const int32_t* __restrict__ cols, const int32_t* __restrict__ off, int R,
                                     int n_tiles, int32_t* __restrict__ tile_cnt, int32_t* __restrict__ tile_ent) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n_tiles) return;
  int32_t* out = tile_ent + off[t];
  const int ca = cols[R * t], cb = (R == 2) ? cols[R * t + 1] : -1;
  int a = ca >= 0 ? col_ptr[ca] : 0, ae = ca >= 0 ? col_ptr[ca + 1] : 0;
  int c = cb >= 0 ? col_ptr[cb] : 0, ce = cb >= 0 ? col_ptr[cb + 1] : 0;
  int n = 0;
  while (a < ae || c < ce) {
    const int va = a < ae ? row_idx[a] : 0x7fffffff;
    const int vc = c < ce ? row_idx[c] : 0x7fffffff;
    if (va == vc) { out[n++] = va * 4 + 3; ++a; ++c; }
    else if (va < vc) { out[n++] = va * 4 + 1; ++a; }
    else { out[n++] = vc * 4 + 2; ++c; }
  }
  tile_cnt[t] = n;
}

// tile_of[kb] = kv tile of pattern column kb
__global__ void kv_tile_of_kernel(const int32_t* __restrict__ cols, int R, int n_tiles, int32_t* __restrict__ tile_of) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= n_tiles * R) return;
  const int kb = cols[c];
  if (kb >= 0) tile_of[kb] = c / R;
}

// ---- schedule of the dQ pass that reads the kept dS tiles -------------------------------------
// The dK/dV pass leaves one dS tile per block of the pattern and 64-row half of its query block, numbered by
// the block's position p in the column lists (col_ptr[c] + rank of the query block in column c):
// 128-token blocks: tiles 2 p and 2 p + 1 (128 keys x 64 queries each); 64-token blocks: tile p (64 keys x
// 64 queries).  A query tile of 128 rows needs, for every kv tile T with an active column in the row(s) of
// its query block(s), the four quarters (64-row half m, 64-key half n) of its 128 x 128 product; entry =
// (T, tile of (m, n) at 1 + 2 n + m), -1 where the pattern has no block (that quarter of dS is zero).  With
// 128-token blocks only n = 0 is used: the tiles of the two halves.  One thread per query tile; entries at
// dq_ent[kDqEntInts * (row_ptr[R t] + i)], kv tiles ascending.
__global__ void dq_sched_kernel(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                                const int32_t* __restrict__ col_ptr, const int32_t* __restrict__ row_idx,
                                const int32_t* __restrict__ tile_of, const int32_t* __restrict__ cols, int R, int nB,
                                int n_qtiles, int32_t* __restrict__ dq_cnt, int32_t* __restrict__ dq_ent) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n_qtiles) return;
  constexpr int E = kDqEntInts;
  int32_t* out = dq_ent + E * static_cast<int64_t>(row_ptr[R * t]);
  int n = 0;
  for (int m = 0; m < R; ++m) {          // distinct kv tiles of the tile's query blocks, kept ascending
    const int qb = R * t + m;
    if (qb >= nB) break;
    for (int x = row_ptr[qb]; x < row_ptr[qb + 1]; ++x) {
      const int T = tile_of[col_idx[x]];
      int pos = 0;
      while (pos < n && out[E * pos] < T) ++pos;
      if (pos < n && out[E * pos] == T) continue;
      for (int y = n; y > pos; --y) out[E * y] = out[E * (y - 1)];
      out[E * pos] = T;
      ++n;
    }
  }
  auto find = [&](int c, int qb) {       // position of block (row qb, column c) in the column lists, or -1
    if (c < 0 || qb >= nB) return -1;
    int lo = col_ptr[c], hi = col_ptr[c + 1];
    const int end = hi;
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (row_idx[mid] < qb) lo = mid + 1; else hi = mid;
    }
    return (lo < end && row_idx[lo] == qb) ? lo : -1;
  };
  for (int i = 0; i < n; ++i) {
    const int T = out[E * i];
    if (R == 1) {
      const int p = find(cols[T], t);
      out[E * i + 1] = p >= 0 ? 2 * p : -1;
      out[E * i + 2] = p >= 0 ? 2 * p + 1 : -1;
      out[E * i + 3] = out[E * i + 4] = -1;
    } else {
      for (int nn = 0; nn < 2; ++nn)
        for (int m = 0; m < 2; ++m) out[E * i + 1 + 2 * nn + m] = find(cols[2 * T + nn], 2 * t + m);
    }
  }
  dq_cnt[t] = n;
}

// doc_end[b][j] = end (one past the last token) of the document token j belongs to, from
// doc_start[b][i] = first token of token i's document (non-decreasing): the first i > j whose
// document starts after j, found by bisection, or L.
__global__ void doc_end_kernel(const int32_t* __restrict__ doc_start, int32_t* __restrict__ doc_end, int B, int L) {
  const int64_t gid = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (gid >= static_cast<int64_t>(B) * L) return;
  const int j = static_cast<int>(gid % L);
  const int32_t* ds = doc_start + (gid - j);
  int lo = j, hi = L;            // ds[lo] <= j (its own document); ds[hi] > j, with ds[L] taken as +inf
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (ds[mid] > j) hi = mid; else lo = mid;
  }
  doc_end[gid] = hi;
}

}  // namespace lg
