"""Thin ctypes binding of the C-ABI library (argument marshalling only).

PyTorch supplies device memory and streams; every step of the attention path runs in
the library's CUDA kernels.  There is no CPU fallback: if the shared library is missing
or the device is not sm_100, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblg_sparse_attn.so")

LG_OK = 0
MODE_FULL_CAUSAL, MODE_SINK_WINDOW, MODE_STRIDED_LOCAL = 0, 1, 2


class LgError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__("%s failed: %s (%d)" % (what, status_string(code), code))
        self.code = code


class AttnParams(C.Structure):
    _fields_ = [("B", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("L", C.c_int32), ("D", C.c_int32),
                ("block", C.c_int32), ("mode", C.c_int32), ("sink_tokens", C.c_int32),
                ("window_tokens", C.c_int32), ("stride_blocks", C.c_int32), ("local_blocks", C.c_int32),
                ("window_exact", C.c_int32), ("lists_prepared", C.c_int32), ("scale", C.c_float),
                ("q_strides", C.c_int64 * 3), ("k_strides", C.c_int64 * 3), ("v_strides", C.c_int64 * 3),
                ("o_strides", C.c_int64 * 3), ("doc_start", C.c_void_p)]


class DeviceStepBuffers(C.Structure):
    _fields_ = [("q", C.c_void_p), ("k", C.c_void_p), ("v", C.c_void_p), ("d_o", C.c_void_p),
                ("o", C.c_void_p), ("lse", C.c_void_p), ("dq", C.c_void_p), ("dk", C.c_void_p), ("dv", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


class DecodeParams(C.Structure):
    _fields_ = [("B", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("D", C.c_int32),
                ("sink_tokens", C.c_int32), ("window_tokens", C.c_int32), ("block_tokens", C.c_int32),
                ("scale", C.c_float)]


_lib = None

# every symbol include/lg.h declares: (restype, argtypes)
_vp, _sz = C.c_void_p, C.c_size_t
SYMBOLS = {
    "lg_block_index_nnz": (C.c_int64, [C.POINTER(AttnParams)]),
    "lg_block_index_bytes": (_sz, [C.POINTER(AttnParams)]),
    "lg_build_block_index": (C.c_int, [C.POINTER(AttnParams), _vp, _vp, _vp, _vp, C.POINTER(C.c_int64), _vp]),
    "lg_sparse_attn_workspace_bytes": (_sz, [C.POINTER(AttnParams), C.c_int]),
    "lg_sparse_attn_prepare": (C.c_int, [C.POINTER(AttnParams), _vp, _sz, C.c_int, _vp]),
    "lg_sparse_attn_bwd_variant": (C.c_int32, [C.POINTER(AttnParams)]),
    "lg_sparse_attn_fwd": (C.c_int, [C.POINTER(AttnParams), _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "lg_sparse_attn_bwd": (C.c_int, [C.POINTER(AttnParams)] + [_vp] * 9 + [_vp, _sz, _vp]),
    "lg_sparse_attn_bwd_marked": (C.c_int, [C.POINTER(AttnParams)] + [_vp] * 9 + [_vp, _sz, _vp, C.POINTER(_vp)]),
    "lg_sparse_attn_fwd_bwd_host_workspace_bytes": (_sz, [C.POINTER(AttnParams), C.c_int]),
    "lg_sparse_attn_fwd_bwd_host": (C.c_int, [C.POINTER(AttnParams)] + [_vp] * 9 + [_vp, C.c_int, _vp, _vp, _vp]),
    "lg_kv_ring_append": (C.c_int, [C.POINTER(DecodeParams), _vp, _vp, _vp, _vp, C.c_int32, _vp, _vp]),
    "lg_sparse_decode_workspace_bytes": (_sz, [C.POINTER(DecodeParams)]),
    "lg_sparse_decode_workspace_init": (C.c_int, [_vp, _sz, _vp]),
    "lg_sparse_decode": (C.c_int, [C.POINTER(DecodeParams), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "lg_chunk_prefill_workspace_bytes": (_sz, [C.POINTER(DecodeParams), C.c_int32, C.c_int64]),
    "lg_chunk_prefill": (C.c_int, [C.POINTER(DecodeParams), _vp, _vp, _vp, _vp, _vp, C.c_int32, C.c_int64, _vp, _vp,
                                   _vp, _sz, _vp]),
    "lg_sparse_decode_static": (C.c_int, [C.POINTER(DecodeParams), _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "lg_sparse_decode_static_reset": (C.c_int, [_vp]),
    "lg_selftest_wait_timeout": (C.c_int, [_vp, _vp]),
    "lg_last_status": (C.c_int, [_vp, _vp]),
    "lg_status_string": (C.c_char_p, [C.c_int]),
    "lg_debug_kernel_launches": (C.c_int64, []),
}


def load_library() -> C.CDLL:
    """Load the in-tree shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("CUDA library %s is missing: run `python -m paper_2410_01485_b200.build` "
                               "(there is no CPU fallback)" % LIB_PATH)
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in SYMBOLS.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def status_string(code: int) -> str:
    return load_library().lg_status_string(code).decode()


def _check(code: int, what: str):
    if code != LG_OK:
        raise LgError(code, what)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _strides3(t: torch.Tensor):
    assert t.dim() == 4 and t.stride(3) == 1, "expect [B, H, L, D] with contiguous D"
    return (C.c_int64 * 3)(t.stride(0), t.stride(1), t.stride(2))


def attn_params(B, Hq, Hkv, L, D, block, mode, sink_tokens=0, window_tokens=0, stride_blocks=0, local_blocks=0,
                scale=0.0, window_exact=False, doc_start=None) -> AttnParams:
    """doc_start: optional CUDA int32 tensor [B, L] (first position of each token's document); the params
    object keeps a reference to it."""
    p = AttnParams()
    if doc_start is not None:
        assert doc_start.dtype == torch.int32 and doc_start.is_contiguous() and tuple(doc_start.shape) == (B, L)
        p.doc_start = doc_start.data_ptr()
        p._doc_start_ref = doc_start
    p.B, p.Hq, p.Hkv, p.L, p.D, p.block, p.mode = B, Hq, Hkv, L, D, block, mode
    p.sink_tokens, p.window_tokens, p.stride_blocks, p.local_blocks = sink_tokens, window_tokens, stride_blocks, local_blocks
    p.scale = scale
    p.window_exact = int(bool(window_exact))
    return p


def params_of(cfg, scale: float = 0.0, doc_start=None) -> AttnParams:
    """AttnParams from a synth.AttnConfig-like object."""
    return attn_params(cfg.B, cfg.Hq, cfg.Hkv, cfg.L, cfg.D, cfg.block, cfg.mode, cfg.sink_tokens,
                       cfg.window_tokens, cfg.stride_blocks, cfg.local_blocks, scale,
                       getattr(cfg, "window_exact", False), doc_start)


# ------------------------------------------------------------------------------ index

def lg_block_index_nnz(p: AttnParams) -> int:
    n = load_library().lg_block_index_nnz(C.byref(p))
    if n < 0:
        raise LgError(int(n), "lg_block_index_nnz")
    return int(n)


def lg_build_block_index(p: AttnParams, device="cuda") -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor, torch.Tensor]:
    """Returns device int32 tensors (row_ptr, col_idx, col_ptr, row_idx)."""
    lib = load_library()
    nnz = lg_block_index_nnz(p)
    nB = -(-p.L // p.block)
    assert lib.lg_block_index_bytes(C.byref(p)) == 4 * (2 * (nB + 1) + 2 * nnz)
    row_ptr = torch.empty(nB + 1, dtype=torch.int32, device=device)
    col_ptr = torch.empty(nB + 1, dtype=torch.int32, device=device)
    col_idx = torch.empty(max(nnz, 1), dtype=torch.int32, device=device)
    row_idx = torch.empty(max(nnz, 1), dtype=torch.int32, device=device)
    out = C.c_int64(-1)
    _check(lib.lg_build_block_index(C.byref(p), row_ptr.data_ptr(), col_idx.data_ptr(), col_ptr.data_ptr(),
                                    row_idx.data_ptr(), C.byref(out), _stream()), "lg_build_block_index")
    assert out.value == nnz
    return row_ptr, col_idx[:nnz], col_ptr, row_idx[:nnz]


# ------------------------------------------------------------------------- fwd / bwd

def attn_workspace(p: AttnParams, want_bwd: bool, device="cuda") -> torch.Tensor:
    n = load_library().lg_sparse_attn_workspace_bytes(C.byref(p), int(want_bwd))
    if n == 0:
        raise LgError(-1, "lg_sparse_attn_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def lg_sparse_attn_prepare(p: AttnParams, workspace: torch.Tensor, want_bwd: bool) -> AttnParams:
    """Build lists and schedules once into `workspace`; sets p.lists_prepared so that later forward /
    backward calls with this params object and workspace launch their attention kernels only."""
    p.lists_prepared = 0
    _check(load_library().lg_sparse_attn_prepare(C.byref(p), workspace.data_ptr(), workspace.numel(), int(want_bwd),
                                                 _stream()), "lg_sparse_attn_prepare")
    p.lists_prepared = 1
    return p


def bwd_variant_name(p: AttnParams) -> str:
    """Which backward variant lg_sparse_attn_bwd runs for these parameters."""
    v = load_library().lg_sparse_attn_bwd_variant(C.byref(p))
    if v < 0:
        raise LgError(int(v), "lg_sparse_attn_bwd_variant")
    return {0: "two_pass", 2: "keep_ds"}[int(v)]


def lg_sparse_attn_fwd(p: AttnParams, q, k, v, o=None, lse=None, workspace=None):
    """q [B,Hq,L,D], k, v [B,Hkv,L,D] bf16 CUDA tensors -> (o bf16, lse fp32 [B,Hq,L])."""
    lib = load_library()
    o = torch.empty_like(q) if o is None else o
    lse = torch.empty(q.shape[:3], dtype=torch.float32, device=q.device) if lse is None else lse
    ws = attn_workspace(p, False, q.device) if workspace is None else workspace
    p.q_strides, p.k_strides, p.v_strides, p.o_strides = _strides3(q), _strides3(k), _strides3(v), _strides3(o)
    _check(lib.lg_sparse_attn_fwd(C.byref(p), q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                  lse.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "lg_sparse_attn_fwd")
    return o, lse


def lg_sparse_attn_bwd(p: AttnParams, q, k, v, o, lse, d_o, dq=None, dk=None, dv=None, workspace=None):
    """Gradients (dq, dk, dv) bf16 of sum(O * dO)."""
    lib = load_library()
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    ws = attn_workspace(p, True, q.device) if workspace is None else workspace
    assert d_o.stride() == o.stride() and dq.stride() == q.stride()
    assert dk.stride() == k.stride() and dv.stride() == v.stride()
    p.q_strides, p.k_strides, p.v_strides, p.o_strides = _strides3(q), _strides3(k), _strides3(v), _strides3(o)
    _check(lib.lg_sparse_attn_bwd(C.byref(p), q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                  lse.data_ptr(), d_o.data_ptr(), dq.data_ptr(), dk.data_ptr(), dv.data_ptr(),
                                  ws.data_ptr(), ws.numel(), _stream()), "lg_sparse_attn_bwd")
    return dq, dk, dv


def lg_sparse_attn_bwd_marked(p: AttnParams, q, k, v, o, lse, d_o, dq, dk, dv, workspace, events):
    """As lg_sparse_attn_bwd; records the caller's four torch.cuda.Event objects (timing enabled, each
    recorded once before so that its handle exists) around the delta, dK/dV and dQ kernels.  Does not
    synchronise: read event durations after the stream has passed them."""
    p.q_strides, p.k_strides, p.v_strides, p.o_strides = _strides3(q), _strides3(k), _strides3(v), _strides3(o)
    assert len(events) == 4
    ev = (C.c_void_p * 4)(*[e.cuda_event for e in events])
    _check(load_library().lg_sparse_attn_bwd_marked(
        C.byref(p), q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), d_o.data_ptr(),
        dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), workspace.data_ptr(), workspace.numel(), _stream(), ev),
        "lg_sparse_attn_bwd_marked")


def timing_events(n: int = 4):
    """n CUDA events with timing, each recorded once so that the driver object behind it exists."""
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
    for e in evs:
        e.record()
    return evs


def host_step_workspace(p: AttnParams, head_groups: int, device="cuda") -> torch.Tensor:
    n = load_library().lg_sparse_attn_fwd_bwd_host_workspace_bytes(C.byref(p), head_groups)
    if n == 0:
        raise LgError(-1, "lg_sparse_attn_fwd_bwd_host_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def host_step_groups(p: AttnParams, head_groups: int) -> int:
    """The number of head groups a step can be cut into: `head_groups` if it divides Hkv, else 1."""
    return head_groups if (head_groups > 1 and p.Hkv % head_groups == 0) else 1


def sparse_attn_fwd_bwd_host(p: AttnParams, host_in, host_out, dev=None, head_groups: int = 4):
    """End-to-end training step with HOST buffers through lg_sparse_attn_fwd_bwd_host: pinned q, k, v, do
    go to the device, forward and backward run there, and o, lse, dq, dk, dv come back into the pinned
    tensors of `host_out`; head groups are pipelined over three streams inside the library call.
    `dev` optionally supplies preallocated device buffers (inputs dict, o, lse, dq, dk, dv, workspace of
    host_step_workspace(p, groups) bytes).  This wrapper only marshals pointers and streams."""
    n_groups = host_step_groups(p, head_groups)
    if dev is None:
        d_in = {k: torch.empty(v.shape, dtype=v.dtype, device="cuda") for k, v in host_in.items()}
        o = torch.empty_like(d_in["q"])
        lse = torch.empty(d_in["q"].shape[:3], dtype=torch.float32, device="cuda")
        dq, dk, dv = torch.empty_like(d_in["q"]), torch.empty_like(d_in["k"]), torch.empty_like(d_in["v"])
        ws = host_step_workspace(p, n_groups)
    else:
        d_in, o, lse, dq, dk, dv, ws = dev
    for t in list(host_in.values()) + list(host_out.values()) + list(d_in.values()) + [o, lse, dq, dk, dv]:
        assert t.is_contiguous()
    bufs = DeviceStepBuffers(d_in["q"].data_ptr(), d_in["k"].data_ptr(), d_in["v"].data_ptr(), d_in["do"].data_ptr(),
                             o.data_ptr(), lse.data_ptr(), dq.data_ptr(), dk.data_ptr(), dv.data_ptr(),
                             ws.data_ptr(), ws.numel())
    cur = torch.cuda.current_stream()
    s_in, s_cmp, s_out = (_side_stream(i) for i in range(3))
    for st in (s_in, s_cmp, s_out):
        st.wait_stream(cur)
    _check(load_library().lg_sparse_attn_fwd_bwd_host(
        C.byref(p), host_in["q"].data_ptr(), host_in["k"].data_ptr(), host_in["v"].data_ptr(), host_in["do"].data_ptr(),
        host_out["o"].data_ptr(), host_out["lse"].data_ptr(), host_out["dq"].data_ptr(), host_out["dk"].data_ptr(),
        host_out["dv"].data_ptr(), C.byref(bufs), n_groups, s_in.cuda_stream, s_cmp.cuda_stream, s_out.cuda_stream),
        "lg_sparse_attn_fwd_bwd_host")
    for st in (s_in, s_cmp, s_out):
        cur.wait_stream(st)
    return host_out


_side_streams = {}


def _side_stream(i: int) -> "torch.cuda.Stream":
    key = (torch.cuda.current_device(), i)
    if key not in _side_streams:
        _side_streams[key] = torch.cuda.Stream()
    return _side_streams[key]


# ---------------------------------------------------------------------- decode / ring

def decode_params(B, Hq, Hkv, D, sink_tokens, window_tokens, scale=0.0, block_tokens=0) -> DecodeParams:
    """block_tokens: 0 = attend every token the cache holds; Bs = the block-granular window of training."""
    p = DecodeParams()
    p.B, p.Hq, p.Hkv, p.D, p.sink_tokens, p.window_tokens, p.scale = B, Hq, Hkv, D, sink_tokens, window_tokens, scale
    p.block_tokens = block_tokens
    return p


def lg_kv_ring_append(p: DecodeParams, k_cache, v_cache, k_new, v_new, n_tokens_before):
    """Append k_new, v_new [B,Hkv,T,D] in place; n_tokens_before int64 device [B]."""
    assert k_cache.is_contiguous() and v_cache.is_contiguous() and k_new.is_contiguous() and v_new.is_contiguous()
    _check(load_library().lg_kv_ring_append(C.byref(p), k_cache.data_ptr(), v_cache.data_ptr(), k_new.data_ptr(),
                                            v_new.data_ptr(), k_new.shape[2], n_tokens_before.data_ptr(),
                                            _stream()), "lg_kv_ring_append")


def decode_workspace(p: DecodeParams, device="cuda") -> torch.Tensor:
    """A workspace ready for lg_sparse_decode (allocated and zero-filled through the library's own call)."""
    n = load_library().lg_sparse_decode_workspace_bytes(C.byref(p))
    if n == 0:
        raise LgError(-1, "lg_sparse_decode_workspace_bytes")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    _check(load_library().lg_sparse_decode_workspace_init(ws.data_ptr(), ws.numel(), _stream()),
           "lg_sparse_decode_workspace_init")
    return ws


def lg_sparse_decode(p: DecodeParams, q, k_cache, v_cache, n_tokens, o=None, lse=None, workspace=None,
                     want_lse: bool = True):
    """q [B,Hq,D] bf16 -> (o [B,Hq,D] bf16, lse [B,Hq] fp32 or None)."""
    assert q.is_contiguous() and k_cache.is_contiguous() and v_cache.is_contiguous()
    o = torch.empty_like(q) if o is None else o
    if lse is None and want_lse:
        lse = torch.empty(q.shape[:2], dtype=torch.float32, device=q.device)
    ws = decode_workspace(p, q.device) if workspace is None else workspace
    _check(load_library().lg_sparse_decode(C.byref(p), q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(),
                                           n_tokens.data_ptr(), o.data_ptr(), lse.data_ptr() if lse is not None else None,
                                           ws.data_ptr(), ws.numel(), _stream()), "lg_sparse_decode")
    return o, lse


def decode_call(p: DecodeParams, q, k_cache, v_cache, n_tokens, o, lse, workspace, stream=None):
    """lg_sparse_decode on fixed buffers (a serving loop's): every argument is marshalled once, the stream
    included (`stream`, default: the stream that is current now).  The returned function takes no arguments,
    launches on that stream and returns nothing (the results are in o, lse).  The tensors must stay alive
    and in place."""
    assert q.is_contiguous() and k_cache.is_contiguous() and v_cache.is_contiguous()
    fn = load_library().lg_sparse_decode
    handle = (torch.cuda.current_stream() if stream is None else stream).cuda_stream
    args = (C.byref(p), C.c_void_p(q.data_ptr()), C.c_void_p(k_cache.data_ptr()), C.c_void_p(v_cache.data_ptr()),
            C.c_void_p(n_tokens.data_ptr()), C.c_void_p(o.data_ptr()),
            C.c_void_p(lse.data_ptr() if lse is not None else None), C.c_void_p(workspace.data_ptr()),
            C.c_size_t(workspace.numel()), C.c_void_p(handle))
    keep = (p, q, k_cache, v_cache, n_tokens, o, lse, workspace)

    def call(_keep=keep):
        code = fn(*args)
        if code != LG_OK:
            raise LgError(code, "lg_sparse_decode")

    return call


def chunk_prefill_workspace(p: DecodeParams, T: int, n_tokens_before: int, device="cuda") -> torch.Tensor:
    n = load_library().lg_chunk_prefill_workspace_bytes(C.byref(p), T, n_tokens_before)
    if n == 0:
        raise LgError(-1, "lg_chunk_prefill_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def lg_chunk_prefill(p: DecodeParams, q_chunk, k_chunk, v_chunk, k_cache, v_cache, n_tokens_before: int,
                     o=None, lse=None, workspace=None):
    """q_chunk [B,Hq,T,D], k_chunk, v_chunk [B,Hkv,T,D] bf16 against the ring caches (None while empty);
    n_tokens_before is a host integer.  Returns (o [B,Hq,T,D] bf16, lse [B,Hq,T] fp32)."""
    assert q_chunk.is_contiguous() and k_chunk.is_contiguous() and v_chunk.is_contiguous()
    assert k_cache is None or (k_cache.is_contiguous() and v_cache.is_contiguous())
    T = q_chunk.shape[2]
    o = torch.empty_like(q_chunk) if o is None else o
    lse = torch.empty(q_chunk.shape[:3], dtype=torch.float32, device=q_chunk.device) if lse is None else lse
    ws = chunk_prefill_workspace(p, T, n_tokens_before, q_chunk.device) if workspace is None else workspace
    _check(load_library().lg_chunk_prefill(
        C.byref(p), q_chunk.data_ptr(), k_chunk.data_ptr(), v_chunk.data_ptr(),
        k_cache.data_ptr() if k_cache is not None else None, v_cache.data_ptr() if v_cache is not None else None,
        T, n_tokens_before, o.data_ptr(), lse.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "lg_chunk_prefill")
    return o, lse


DECODE_STATIC_SCRATCH_BYTES = 4 << 20   # LG_DECODE_STATIC_SCRATCH_BYTES of include/lg.h


def lg_sparse_decode_static(p: DecodeParams, q, k_cache, v_cache, n_tokens, o, lse=None):
    """lg_sparse_decode for callers that cannot allocate: no workspace argument, the split
    partials live in a fixed array inside the library (see include/lg.h).  `o` (and `lse`, if
    wanted) must be supplied by the caller, so this wrapper allocates nothing either."""
    assert q.is_contiguous() and k_cache.is_contiguous() and v_cache.is_contiguous() and o.is_contiguous()
    _check(load_library().lg_sparse_decode_static(C.byref(p), q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(),
                                                  n_tokens.data_ptr(), o.data_ptr(),
                                                  lse.data_ptr() if lse is not None else None, _stream()),
           "lg_sparse_decode_static")
    return o, lse


def lg_selftest_wait_timeout(workspace: torch.Tensor) -> None:
    """Launch the one-warp kernel whose bounded wait must expire (see include/lg.h)."""
    _check(load_library().lg_selftest_wait_timeout(workspace.data_ptr(), _stream()), "lg_selftest_wait_timeout")


def kernel_launches() -> int:
    """Kernels launched by the library in this process so far (diagnostic counter)."""
    return int(load_library().lg_debug_kernel_launches())


def lg_last_status(workspace: torch.Tensor) -> int:
    return int(load_library().lg_last_status(workspace.data_ptr(), _stream()))
