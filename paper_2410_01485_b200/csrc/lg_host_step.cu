// A whole training step (forward + backward) on HOST buffers: head groups pipelined over a
// copy-in stream, a compute stream and a copy-out stream.  Only copies, events and the two
// device entry points; no arithmetic of its own.
#include <cuda_runtime.h>

#include "lg_host.h"

namespace lg {
namespace {

struct GroupPlan {
  lg_attn_params pg;      // the group's problem: kv_per kv heads with their query heads, strides of the whole tensors
  int n_groups, kv_per, q_per;
  size_t ws_per;          // workspace slice of one group
};

lg_status plan_groups(const lg_attn_params* p, int head_groups, GroupPlan* g) {
  Resolved r;
  lg_status s = resolve(p, &r);
  if (s != LG_OK) return s;
  if (head_groups < 1 || r.Hkv % head_groups != 0) return LG_ERR_INVALID_ARG;
  g->n_groups = head_groups;
  g->kv_per = r.Hkv / head_groups;
  g->q_per = g->kv_per * r.G;
  g->pg = *p;
  g->pg.Hq = g->q_per;
  g->pg.Hkv = g->kv_per;
  g->pg.lists_prepared = 0;
  // contiguous [B, H, L, D] of the WHOLE tensors: a group is a slice of heads
  const int64_t ld = static_cast<int64_t>(r.L) * r.D;
  const int64_t sq[3] = {static_cast<int64_t>(r.Hq) * ld, ld, r.D}, sk[3] = {static_cast<int64_t>(r.Hkv) * ld, ld, r.D};
  for (int i = 0; i < 3; ++i) {
    g->pg.q_strides[i] = g->pg.o_strides[i] = sq[i];
    g->pg.k_strides[i] = g->pg.v_strides[i] = sk[i];
  }
  const size_t one = lg_sparse_attn_workspace_bytes(&g->pg, 1);
  if (one == 0) return LG_ERR_INVALID_ARG;
  g->ws_per = align_up(one, 256);
  return LG_OK;
}

// copy heads [h0, h0 + nh) of a contiguous [B, H, row_bytes-per-head] tensor between host and device
cudaError_t copy_heads(void* dst, const void* src, int B, int H, int h0, int nh, size_t head_bytes, cudaMemcpyKind kind,
                       cudaStream_t st) {
  uint8_t* d = static_cast<uint8_t*>(dst) + static_cast<size_t>(h0) * head_bytes;
  const uint8_t* s = static_cast<const uint8_t*>(src) + static_cast<size_t>(h0) * head_bytes;
  if (B == 1 || nh == H) return cudaMemcpyAsync(d, s, static_cast<size_t>(B == 1 ? nh : B * H) * head_bytes, kind, st);
  return cudaMemcpy2DAsync(d, static_cast<size_t>(H) * head_bytes, s, static_cast<size_t>(H) * head_bytes,
                           static_cast<size_t>(nh) * head_bytes, B, kind, st);
}

}  // namespace
}  // namespace lg

using namespace lg;

extern "C" {

size_t lg_sparse_attn_fwd_bwd_host_workspace_bytes(const lg_attn_params* p, int head_groups) {
  GroupPlan g;
  if (!p || plan_groups(p, head_groups, &g) != LG_OK) return 0;
  return g.ws_per * g.n_groups;
}

lg_status lg_sparse_attn_fwd_bwd_host(const lg_attn_params* p, const void* q_host, const void* k_host,
                                      const void* v_host, const void* d_o_host, void* o_host, float* lse_host,
                                      void* dq_host, void* dk_host, void* dv_host, const lg_device_step_buffers* dev,
                                      int head_groups, void* stream_in, void* stream_compute, void* stream_out) {
  LG_RANGE("lg_sparse_attn_fwd_bwd_host");
  if (!p || !dev) return LG_ERR_INVALID_ARG;
  GroupPlan g;
  lg_status s = plan_groups(p, head_groups, &g);
  if (s != LG_OK) return s;
  if (!q_host || !k_host || !v_host || !d_o_host || !o_host || !lse_host || !dq_host || !dk_host || !dv_host)
    return LG_ERR_INVALID_ARG;
  if (!dev->q || !dev->k || !dev->v || !dev->d_o || !dev->o || !dev->lse || !dev->dq || !dev->dk || !dev->dv ||
      !dev->workspace)
    return LG_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(dev->workspace) & 255) return LG_ERR_INVALID_ARG;
  if (dev->workspace_bytes < g.ws_per * g.n_groups) return LG_ERR_WORKSPACE;
  cudaStream_t s_in = static_cast<cudaStream_t>(stream_in), s_cmp = static_cast<cudaStream_t>(stream_compute),
               s_out = static_cast<cudaStream_t>(stream_out);
  const int B = p->B, Hq = p->Hq, Hkv = p->Hkv;
  const size_t head_bytes = static_cast<size_t>(p->L) * p->D * 2, lse_head_bytes = static_cast<size_t>(p->L) * 4;
  uint8_t* ws = static_cast<uint8_t*>(dev->workspace);
  lg_status result = LG_OK;
  bool cuda_ok = true;
  auto ck = [&](cudaError_t e) { if (e != cudaSuccess) cuda_ok = false; return e == cudaSuccess; };
  for (int grp = 0; grp < g.n_groups && cuda_ok && result == LG_OK; ++grp) {
    const int kv0 = grp * g.kv_per, q0 = grp * g.q_per;
    cudaEvent_t ev_in = nullptr, ev_cmp = nullptr;
    if (!ck(cudaEventCreateWithFlags(&ev_in, cudaEventDisableTiming))) break;
    if (!ck(cudaEventCreateWithFlags(&ev_cmp, cudaEventDisableTiming))) { cudaEventDestroy(ev_in); break; }
    // inputs of the group
    ck(copy_heads(dev->q, q_host, B, Hq, q0, g.q_per, head_bytes, cudaMemcpyHostToDevice, s_in));
    ck(copy_heads(dev->k, k_host, B, Hkv, kv0, g.kv_per, head_bytes, cudaMemcpyHostToDevice, s_in));
    ck(copy_heads(dev->v, v_host, B, Hkv, kv0, g.kv_per, head_bytes, cudaMemcpyHostToDevice, s_in));
    ck(copy_heads(dev->d_o, d_o_host, B, Hq, q0, g.q_per, head_bytes, cudaMemcpyHostToDevice, s_in));
    ck(cudaEventRecord(ev_in, s_in));
    ck(cudaStreamWaitEvent(s_cmp, ev_in, 0));
    if (cuda_ok) {
      auto off = [&](void* base, int h0, size_t hb) { return static_cast<void*>(static_cast<uint8_t*>(base) + static_cast<size_t>(h0) * hb); };
      void* qd = off(dev->q, q0, head_bytes);
      void* kd = off(dev->k, kv0, head_bytes);
      void* vd = off(dev->v, kv0, head_bytes);
      void* dod = off(dev->d_o, q0, head_bytes);
      void* od = off(dev->o, q0, head_bytes);
      // LSE of a group is not a slice with the group's own batch stride unless B == 1: with B > 1 the
      // group's LSE goes to a compact [B, q_per, L] block at the group's position of the staging buffer
      float* lsed = reinterpret_cast<float*>(static_cast<uint8_t*>(static_cast<void*>(dev->lse)) +
                                             static_cast<size_t>(B) * q0 * lse_head_bytes);
      uint8_t* wsg = ws + grp * g.ws_per;
      // every group reports through the first word of the caller's workspace (group 0's own header):
      // a failure of any group shows in lg_last_status(dev->workspace), and later groups then do nothing
      unsigned int* status = grp == 0 ? nullptr : reinterpret_cast<unsigned int*>(ws);
      result = attn_fwd_entry(&g.pg, qd, kd, vd, od, lsed, wsg, g.ws_per, s_cmp, status);
      if (result == LG_OK)
        result = attn_bwd_entry(&g.pg, qd, kd, vd, od, lsed, dod, off(dev->dq, q0, head_bytes),
                                off(dev->dk, kv0, head_bytes), off(dev->dv, kv0, head_bytes), wsg, g.ws_per, s_cmp,
                                nullptr, status);
    }
    ck(cudaEventRecord(ev_cmp, s_cmp));
    ck(cudaStreamWaitEvent(s_out, ev_cmp, 0));
    if (cuda_ok && result == LG_OK) {
      ck(copy_heads(o_host, dev->o, B, Hq, q0, g.q_per, head_bytes, cudaMemcpyDeviceToHost, s_out));
      ck(copy_heads(dq_host, dev->dq, B, Hq, q0, g.q_per, head_bytes, cudaMemcpyDeviceToHost, s_out));
      ck(copy_heads(dk_host, dev->dk, B, Hkv, kv0, g.kv_per, head_bytes, cudaMemcpyDeviceToHost, s_out));
      ck(copy_heads(dv_host, dev->dv, B, Hkv, kv0, g.kv_per, head_bytes, cudaMemcpyDeviceToHost, s_out));
      // LSE: compact [B, q_per, L] block of the group on the device -> rows (b, q0 .. q0 + q_per) of the host tensor
      const uint8_t* src = static_cast<const uint8_t*>(static_cast<const void*>(dev->lse)) + static_cast<size_t>(B) * q0 * lse_head_bytes;
      uint8_t* dst = static_cast<uint8_t*>(static_cast<void*>(lse_host)) + static_cast<size_t>(q0) * lse_head_bytes;
      ck(cudaMemcpy2DAsync(dst, static_cast<size_t>(Hq) * lse_head_bytes, src, static_cast<size_t>(g.q_per) * lse_head_bytes,
                           static_cast<size_t>(g.q_per) * lse_head_bytes, B, cudaMemcpyDeviceToHost, s_out));
    }
    // a destroyed event is released once the work that refers to it has passed it
    cudaEventDestroy(ev_in);
    cudaEventDestroy(ev_cmp);
  }
  if (result != LG_OK) return result;
  if (!cuda_ok) return LG_ERR_CUDA;
  return LG_OK;
}

}  // extern "C"
