// Launch of the backward attention kernels: delta pre-pass, dK/dV pass, dQ pass.
#include "lg_bwd.cuh"
#include "lg_host.h"

namespace lg {

template <int D, int BS>
static lg_status launch_bwd_t(const Resolved& r, const WsLayout& w, const void* q, const void* k, const void* v,
                              const void* o, const float* lse, const void* d_o, void* dq, void* dk, void* dv,
                              uint8_t* ws, cudaStream_t stream, cudaEvent_t* marks) {
  lg_status s;
  float* stat = reinterpret_cast<float*>(ws + w.delta);
  if (marks) cudaEventRecord(marks[0], stream);
  {
    const int Lp = static_cast<int>(align_up(r.L, 128));
    const int n_bh = r.B * r.Hq;
    const int rows_per_block = 256 / (D / 8) * kDeltaRowsPerThread;
    dim3 grid((Lp + rows_per_block - 1) / rows_per_block, n_bh < 65535 ? n_bh : 65535);
    delta_kernel<D><<<grid, 256, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(o), static_cast<const __nv_bfloat16*>(d_o), lse, stat, r.os[0], r.os[1],
        r.os[2], r.Hq, n_bh, r.L, Lp, static_cast<int64_t>(n_bh) * Lp); note_launch();
  }
  if (marks) cudaEventRecord(marks[1], stream);
  BwdArgs a;
  a.stat = stat;
  a.Lp = static_cast<int>(align_up(r.L, 128));
  a.stat_plane = static_cast<int64_t>(r.B) * r.Hq * a.Lp;
  a.error_word = r.error_word ? r.error_word : reinterpret_cast<unsigned int*>(ws);
  a.expect_fp = r.expect_fp;
  a.n_tiles = r.n_ktiles; a.nB = r.pat.nB; a.n_list = static_cast<int>(r.nnz);   // (all three kernels walk ceil(L / 128) tiles)
  a.expect_fp2 = r.expect_fp2;
  a.L = r.L; a.Hq = r.Hq; a.Hkv = r.Hkv; a.G = r.G;
  a.exact_w = r.exact_w; a.ns = r.pat.ns;
  a.doc_start = r.doc_start;
  a.doc_end = r.doc_start ? reinterpret_cast<const int32_t*>(ws + w.doc_end) : nullptr;
  a.scale = r.scale;
  a.scale_log2 = r.scale * 1.4426950408889634f;
  a.ds_nnz = r.nnz;
  a.ds_buf = reinterpret_cast<__nv_bfloat16*>(ws + w.ds_buf);
  a.col_ptr = reinterpret_cast<const int32_t*>(ws + w.col_ptr);
  constexpr int smem = BwdSmem<D, BS>::kTotal;
  const BwdVariant variant = bwd_variant(r);

  // ---- dK / dV pass -------------------------------------------------------------------
  {
    CUtensorMap tq, tk, tv, tdo;
    if ((s = make_tmap(&tq, q, r.B, r.Hq, r.L, D, r.qs, BS)) != LG_OK) return s;
    if ((s = make_tmap(&tdo, d_o, r.B, r.Hq, r.L, D, r.os, BS)) != LG_OK) return s;
    if ((s = make_tmap(&tk, k, r.B, r.Hkv, r.L, D, r.ks, BS)) != LG_OK) return s;
    if ((s = make_tmap(&tv, v, r.B, r.Hkv, r.L, D, r.vs, BS)) != LG_OK) return s;
    a.tile_off = reinterpret_cast<const int32_t*>(ws + w.kt_off);
    a.tile_cols = reinterpret_cast<const int32_t*>(ws + w.kt_cols);
    a.tile_cnt = reinterpret_cast<const int32_t*>(ws + w.kt_cnt);
    a.tile_ent = reinterpret_cast<const int32_t*>(ws + w.kt_ent);
    a.order = reinterpret_cast<const int32_t*>(ws + w.kt_order);
    a.out0 = static_cast<__nv_bfloat16*>(dk);
    a.out1 = static_cast<__nv_bfloat16*>(dv);
    for (int i = 0; i < 3; ++i) { a.s0[i] = r.ks[i]; a.s1[i] = r.vs[i]; }
    dim3 grid(r.B * r.Hkv, r.n_ktiles);
    a.ahead = sm_count();   // one CTA per SM
    a.head_group = head_group(r, r.B * r.Hkv);
    a.n_long = r.n_ktiles;
    a.descending = r.mode != LG_MODE_SINK_WINDOW;   // combs and full causal attention
    if (r.mode == LG_MODE_STRIDED_LOCAL && r.pat.stride > 1) {
      // the comb columns (every stride-th) are the longest and share kv tiles among themselves: those tiles,
      // a few heads at a time, walk down the same rows together; the short tiles follow with all heads side
      // by side (stride-64 setting, 32 heads, two at a time: dK/dV pass 6.3 -> 5.9 ms).  With grouped-query
      // attention a tile streams each row for all query heads of its group; four kv heads at a time were
      // measured best there (64 / 8 heads at 128K, dS kept: 40.5-41.7 -> 39.8-39.9 ms, two at a time 40.8-41.1;
      // recomputing dQ pass: 34.4-34.9 -> 33.9-35.2 ms, two at a time 34.9-35.7).
      const int n_comb = (r.pat.nB + r.pat.stride - 1) / r.pat.stride, per_tile = 128 / r.block;
      a.n_long = (n_comb + per_tile - 1) / per_tile;
      if (a.n_long > r.n_ktiles) a.n_long = r.n_ktiles;
      const int comb_group = r.Hq == r.Hkv ? kHeadGroupCombs : kHeadGroupCombsGqa;
      a.head_group = r.B * r.Hkv > comb_group ? comb_group : r.B * r.Hkv;
    }
    if (a.ahead < 0) return LG_ERR_CUDA;
    if (variant == kBwdKeepDs) {
      // the tile of zeros that stands in for a half of a query tile a kv tile has no entry for
      if (cudaMemsetAsync(ws + w.ds_buf + ds_buffer_bytes(r) - 128 * 64 * 2, 0, 128 * 64 * 2, stream) != cudaSuccess) return LG_ERR_CUDA;
      auto kern = bwd_dkdv_kernel<D, BS, true>;
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
        return LG_ERR_CUDA;
      kern<<<grid, kKvThreads, smem, stream>>>(tq, tk, tv, tdo, a); note_launch();
    } else {
      auto kern = bwd_dkdv_kernel<D, BS, false>;
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
        return LG_ERR_CUDA;
      kern<<<grid, kKvThreads, smem, stream>>>(tq, tk, tv, tdo, a); note_launch();
    }
    if (marks) cudaEventRecord(marks[2], stream);
  }
  if (variant == kBwdKeepDs) {
    // ---- dQ = scale * dS K from the kept tiles --------------------------------------------
    CUtensorMap tk;
    if ((s = make_tmap(&tk, k, r.B, r.Hkv, r.L, D, r.ks, BS)) != LG_OK) return s;
    a.tile_off = reinterpret_cast<const int32_t*>(ws + w.row_ptr);
    a.tile_ent = reinterpret_cast<const int32_t*>(ws + w.dq_ent);
    a.tile_cols = reinterpret_cast<const int32_t*>(ws + w.kt_cols);
    a.tile_cnt = reinterpret_cast<const int32_t*>(ws + w.dq_cnt);
    a.order = reinterpret_cast<const int32_t*>(ws + w.qt_order);
    a.out0 = static_cast<__nv_bfloat16*>(dq);
    a.out1 = nullptr;
    for (int i = 0; i < 3; ++i) { a.s0[i] = r.qs[i]; a.s1[i] = 0; }
    auto kern = bwd_dq_from_ds_kernel<D, BS>;
    constexpr int smem_q = DqDsSmem<D>::kTotal;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_q) != cudaSuccess)
      return LG_ERR_CUDA;
    const int n_sm = sm_count();
    if (n_sm <= 0) return LG_ERR_CUDA;
    const long long n_items = static_cast<long long>(r.B) * r.Hq * r.n_qtiles;
    const int n_cta = static_cast<int>(n_items < n_sm ? n_items : n_sm);   // one CTA per SM, each working every n_cta-th item
    kern<<<n_cta, kDq2Threads, smem_q, stream>>>(tk, a, r.B * r.Hq, r.n_qtiles); note_launch();
    if (marks) cudaEventRecord(marks[3], stream);
    return cudaGetLastError() == cudaSuccess ? LG_OK : LG_ERR_CUDA;
  }
  // ---- dQ pass ------------------------------------------------------------------------
  {
    CUtensorMap tq, tk, tv, tdo;
    if ((s = make_tmap(&tq, q, r.B, r.Hq, r.L, D, r.qs, 128)) != LG_OK) return s;
    if ((s = make_tmap(&tdo, d_o, r.B, r.Hq, r.L, D, r.os, 128)) != LG_OK) return s;
    if ((s = make_tmap(&tk, k, r.B, r.Hkv, r.L, D, r.ks, BS)) != LG_OK) return s;
    if ((s = make_tmap(&tv, v, r.B, r.Hkv, r.L, D, r.vs, BS)) != LG_OK) return s;
    a.tile_off = reinterpret_cast<const int32_t*>(ws + w.row_ptr);
    a.tile_cols = nullptr;
    a.tile_cnt = reinterpret_cast<const int32_t*>(ws + w.qt_cnt);
    a.tile_ent = reinterpret_cast<const int32_t*>(ws + w.qt_ent);
    a.order = reinterpret_cast<const int32_t*>(ws + w.qt_order);
    a.out0 = static_cast<__nv_bfloat16*>(dq);
    a.out1 = nullptr;
    for (int i = 0; i < 3; ++i) { a.s0[i] = r.qs[i]; a.s1[i] = 0; }
    a.head_group = head_group(r, r.B * r.Hq);
    auto kern = bwd_dq_kernel<D, BS>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
      return LG_ERR_CUDA;
    dim3 grid(r.B * r.Hq, r.n_qtiles);
    kern<<<grid, kDqThreads, smem, stream>>>(tq, tk, tv, tdo, a); note_launch();
    if (marks) cudaEventRecord(marks[3], stream);
  }
  return cudaGetLastError() == cudaSuccess ? LG_OK : LG_ERR_CUDA;
}

lg_status launch_bwd(const Resolved& r, const WsLayout& w, const void* q, const void* k, const void* v,
                     const void* o, const float* lse, const void* d_o, void* dq, void* dk, void* dv, uint8_t* ws,
                     cudaStream_t stream, cudaEvent_t* marks) {
  if (r.n_qtiles > 65535) return LG_ERR_UNSUPPORTED;
#define LG_BWD_CASE(DD, BB) \
  if (r.D == DD && r.block == BB) return launch_bwd_t<DD, BB>(r, w, q, k, v, o, lse, d_o, dq, dk, dv, ws, stream, marks);
  LG_BWD_CASE(128, 128)
  LG_BWD_CASE(128, 64)
  LG_BWD_CASE(64, 128)
  LG_BWD_CASE(64, 64)
#undef LG_BWD_CASE
  return LG_ERR_UNSUPPORTED;
}

}  // namespace lg
