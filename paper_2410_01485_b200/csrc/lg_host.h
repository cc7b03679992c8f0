// Host-side helpers shared by the C-ABI entry points: validation, workspace layout,
// tensor-map encoding.  Nothing here is exported.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/lg.h"
#include "lg_pattern.h"

// Optional NVTX ranges around every entry point (build with -DLG_NVTX; the NVTX headers are
// self-contained and cost nothing when no tool is attached).
#ifdef LG_NVTX
#include <nvtx3/nvToolsExt.h>
namespace lg {
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
};
}  // namespace lg
#define LG_RANGE(name) ::lg::NvtxRange lg_nvtx_range_(name)
#else
#define LG_RANGE(name) ((void)0)
#endif

namespace lg {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Diagnostic only: how many kernels the library has launched in this process (read through
// lg_debug_kernel_launches); nothing in the library depends on it.
void note_launch();

struct Resolved {          // validated, defaulted copy of lg_attn_params
  int B, Hq, Hkv, L, D, block, mode, G;
  PatternDev pat;
  float scale;
  int exact_w;             // token-exact window length in tokens (0: block-granular)
  int win_block, win_phase;  // forward only, with exact_w: block-aligned window edge in coordinates shifted by win_phase (0: off)
  int64_t qs[3], ks[3], vs[3], os[3];
  int n_qtiles, n_ktiles;  // ceil(L / 128)
  int n_stiles;            // ceil(L / 256): super-tiles of the forward
  int q_start, Lq;         // forward only: queries exist for rows [q_start, q_start + Lq) (0, L by default)
  const int32_t* doc_start;  // device [B, L] or null: first position of each token's document
  unsigned int* error_word;  // status word of the call when it is not the start of `ws` (null: it is)
  int lists_prepared;        // the caller says the workspace already holds this pattern's lists
  unsigned long long expect_fp, expect_fp2;   // fingerprints the kernels accept in the header (0: no check)
  int64_t nnz;
};

lg_status resolve(const lg_attn_params* p, Resolved* r);

// Layout of the attention workspace (all offsets 256-byte aligned).
struct WsLayout {
  size_t row_ptr, col_idx, col_ptr, row_idx;     // the CSR / CSC lists
  size_t qt_cnt, qt_ent, qt_order;               // query-tile schedules (dQ pass)
  size_t sq_cnt, sq_ent, sq_order;               // super-tile schedules (forward)
  size_t kt_cnt, kt_ent, kt_order;               // kv-tile schedules (dK/dV pass)
  size_t kt_cols, kt_off;                        // members of each kv tile, start of its schedule
  size_t doc_end;                                // int32 [B, L]: end of each token's document (bwd with documents only)
  size_t delta;                                  // 2 x float [B, Hq, L]: -LSE * log2 e, then -delta (bwd only)
  // backward that keeps dS only (0 otherwise): pattern column -> kv tile, the schedule of its dQ pass, the dS^T tiles
  size_t kt_tile_of, dq_cnt, dq_ent, ds_buf;
  size_t total;
};
WsLayout ws_layout(const Resolved& r, bool want_bwd);

// Build CSR/CSC on `stream` into the given device arrays.
lg_status launch_index_build(const Resolved& r, int32_t* row_ptr, int32_t* col_idx, int32_t* col_ptr,
                             int32_t* row_idx, cudaStream_t stream);
// Build lists + tile schedules inside a workspace.
// `what`: bit 0 = the forward's schedule, bit 1 = the backward's schedules.
lg_status prepare_workspace(const Resolved& r, const WsLayout& w, uint8_t* ws, int what, cudaStream_t stream);

// bf16 [B, H, L, D] tensor (element strides bs, hs, ls; D contiguous) as a 4-D tensor map with
// boxes of 64 columns x `box_rows` rows and the 128-byte swizzle.
lg_status make_tmap(CUtensorMap* out, const void* base, int B, int H, int L, int D, const int64_t strides[3],
                    int box_rows);

// Which backward runs for this problem.
enum BwdVariant {
  kBwdTwoPass = 0,   // dK/dV pass, then a dQ pass that recomputes S and dP
  kBwdKeepDs = 2     // dK/dV pass that also writes dS^T to the workspace, then a dQ pass that is one product: dQ = dS K
};
BwdVariant bwd_variant(const Resolved& r);
// bytes of the dS^T buffer of the kBwdKeepDs variant
int sm_count();   // SMs of the current device, < 0 on failure
int head_group(const Resolved& r, int n_x);
size_t ds_buffer_bytes(const Resolved& r);


lg_status check_arch();
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

lg_status launch_fwd(const Resolved& r, const WsLayout& w, const void* q, const void* k, const void* v, void* o,
                     float* lse, uint8_t* ws, cudaStream_t stream);
lg_status launch_bwd(const Resolved& r, const WsLayout& w, const void* q, const void* k, const void* v,
                     const void* o, const float* lse, const void* d_o, void* dq, void* dk, void* dv, uint8_t* ws,
                     cudaStream_t stream, cudaEvent_t* marks /* null, or 4 events recorded around the 3 kernels */);

// The forward / backward entry points with the status word of the call redirected (null: the start
// of `workspace`): a step that runs several calls on slices of one workspace reports through one word.
lg_status attn_fwd_entry(const lg_attn_params* p, const void* q, const void* k, const void* v, void* o, float* lse,
                         void* workspace, size_t workspace_bytes, void* stream, unsigned int* status_word);
lg_status attn_bwd_entry(const lg_attn_params* p, const void* q, const void* k, const void* v, const void* o,
                         const float* lse, const void* d_o, void* dq, void* dk, void* dv, void* workspace,
                         size_t workspace_bytes, void* stream, cudaEvent_t* marks, unsigned int* status_word);

}  // namespace lg
