// Launch of the forward attention kernel.
#include "lg_fwd.cuh"
#include "lg_host.h"

namespace lg {

template <int D, int BS>
static lg_status launch_fwd_t(const Resolved& r, const WsLayout& w, const void* q, const void* k, const void* v,
                              void* o, float* lse, uint8_t* ws, cudaStream_t stream) {
  CUtensorMap tq, tk, tv;
  lg_status s;
  if ((s = make_tmap(&tq, q, r.B, r.Hq, r.Lq, D, r.qs, 128)) != LG_OK) return s;
  if ((s = make_tmap(&tk, k, r.B, r.Hkv, r.L, D, r.ks, BS)) != LG_OK) return s;
  if ((s = make_tmap(&tv, v, r.B, r.Hkv, r.L, D, r.vs, BS)) != LG_OK) return s;
  FwdArgs a;
  a.tile_off = reinterpret_cast<const int32_t*>(ws + w.row_ptr);
  a.tile_cnt = reinterpret_cast<const int32_t*>(ws + w.sq_cnt);
  a.tile_ent = reinterpret_cast<const int32_t*>(ws + w.sq_ent);
  a.order = reinterpret_cast<const int32_t*>(ws + w.sq_order);
  a.o = static_cast<__nv_bfloat16*>(o);
  a.lse = lse;
  a.error_word = r.error_word ? r.error_word : reinterpret_cast<unsigned int*>(ws);
  a.expect_fp = r.expect_fp;
  a.n_tiles = r.n_stiles; a.nB = r.pat.nB; a.n_list = static_cast<int>(r.nnz);
  a.expect_fp2 = r.expect_fp2;
  for (int i = 0; i < 3; ++i) a.o_strides[i] = r.os[i];
  a.L = r.L; a.Hq = r.Hq; a.G = r.G;
  a.q_start = r.q_start; a.Lq = r.Lq;
  a.exact_w = r.exact_w; a.ns = r.pat.ns;
  a.win_block = r.win_block; a.win_phase = r.win_phase;
  a.doc_start = r.doc_start;
  a.scale_log2 = r.scale * 1.4426950408889634f;
  a.head_group = head_group(r, r.B * r.Hq);
  auto kern = fwd_kernel<D, BS>;
  constexpr int smem = FwdSmem<D>::kTotal;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return LG_ERR_CUDA;
  dim3 grid(r.B * r.Hq, r.n_stiles);
  kern<<<grid, kFwdThreads, smem, stream>>>(tq, tk, tv, a); note_launch();
  return cudaGetLastError() == cudaSuccess ? LG_OK : LG_ERR_CUDA;
}

lg_status launch_fwd(const Resolved& r, const WsLayout& w, const void* q, const void* k, const void* v, void* o,
                     float* lse, uint8_t* ws, cudaStream_t stream) {
  if (r.n_qtiles > 65535) return LG_ERR_UNSUPPORTED;
  if (r.D == 128 && r.block == 128) return launch_fwd_t<128, 128>(r, w, q, k, v, o, lse, ws, stream);
  if (r.D == 128 && r.block == 64) return launch_fwd_t<128, 64>(r, w, q, k, v, o, lse, ws, stream);
  if (r.D == 64 && r.block == 128) return launch_fwd_t<64, 128>(r, w, q, k, v, o, lse, ws, stream);
  if (r.D == 64 && r.block == 64) return launch_fwd_t<64, 64>(r, w, q, k, v, o, lse, ws, stream);
  return LG_ERR_UNSUPPORTED;
}

}  // namespace lg
