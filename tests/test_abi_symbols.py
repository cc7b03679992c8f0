"""The C-ABI library loads on a machine without a GPU and exports every symbol that
include/lg.h declares; host-side validation rejects bad arguments without launching."""
import ctypes as C
import os
import re

import pytest

from paper_2410_01485_b200 import binding, build


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(os.path.dirname(build.HERE), "include", "lg.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(lg_[a-z_0-9]+)\s*\(", header))
    assert declared, "no declarations parsed"
    assert declared == set(binding.SYMBOLS), (declared ^ set(binding.SYMBOLS))
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert binding.status_string(0) == "ok"
    for code in range(-6, 0):
        assert binding.status_string(code) not in ("ok", "unknown status")


def _good():
    return binding.attn_params(1, 4, 2, 512, 128, 64, binding.MODE_SINK_WINDOW, sink_tokens=64, window_tokens=128)


def test_nnz_and_sizes_on_host(lib):
    p = _good()
    assert binding.lg_block_index_nnz(p) == 21      # same pattern as the tiny config
    assert lib.lg_block_index_bytes(C.byref(p)) == 4 * (2 * 9 + 2 * 21)
    assert lib.lg_sparse_attn_workspace_bytes(C.byref(p), 1) > lib.lg_sparse_attn_workspace_bytes(C.byref(p), 0) > 256
    full = binding.attn_params(1, 1, 1, 32768, 128, 64, binding.MODE_FULL_CAUSAL)
    assert binding.lg_block_index_nnz(full) == 131328
    strided = binding.attn_params(1, 64, 8, 131072, 128, 64, binding.MODE_STRIDED_LOCAL, stride_blocks=16, local_blocks=4)
    assert binding.lg_block_index_nnz(strided) == 139770


def test_backward_variant_follows_the_ds_buffer_and_the_environment(lib, monkeypatch):
    """Which backward a call takes is host logic: dS is kept while its buffer (2 bytes per pair of the pattern's
    blocks and query head) is within the limit, and the workspace grows by that buffer."""
    cfg3 = binding.attn_params(1, 32, 32, 131072, 128, 128, binding.MODE_SINK_WINDOW, sink_tokens=128, window_tokens=4096)
    nnz = binding.lg_block_index_nnz(cfg3)
    ds_bytes = 32 * nnz * 128 * 128 * 2                       # 34.9e9
    assert 34.8e9 < ds_bytes < 35.0e9
    monkeypatch.delenv("LG_BWD_VARIANT", raising=False)
    sizes = {}
    for cap, want in (("34", 0), ("36", 2)):                  # just below and just above the buffer
        monkeypatch.setenv("LG_KEEP_DS_MAX_GB", cap)
        assert lib.lg_sparse_attn_bwd_variant(C.byref(cfg3)) == want
        sizes[want] = lib.lg_sparse_attn_workspace_bytes(C.byref(cfg3), 1)
    assert ds_bytes <= sizes[2] - sizes[0] < ds_bytes + (1 << 20)
    monkeypatch.setenv("LG_BWD_VARIANT", "two_pass")          # the explicit choice wins over the limit
    assert lib.lg_sparse_attn_bwd_variant(C.byref(cfg3)) == 0
    monkeypatch.setenv("LG_BWD_VARIANT", "keep_ds")
    monkeypatch.setenv("LG_KEEP_DS_MAX_GB", "1")
    assert lib.lg_sparse_attn_bwd_variant(C.byref(cfg3)) == 2
    # without either variable the limit is 40 % of the device's memory, 48 GB where there is no device:
    # the 34.9 GB of this config are kept either way
    monkeypatch.delenv("LG_BWD_VARIANT")
    monkeypatch.delenv("LG_KEEP_DS_MAX_GB")
    assert lib.lg_sparse_attn_bwd_variant(C.byref(cfg3)) == 2
    assert lib.lg_sparse_attn_bwd_variant(None) < 0


@pytest.mark.parametrize("mutate", [
    lambda p: setattr(p, "Hkv", 3),                 # Hq % Hkv != 0
    lambda p: setattr(p, "L", 0),                   # empty sequence
    lambda p: setattr(p, "block", 32),
    lambda p: setattr(p, "sink_tokens", 10),        # not a multiple of block
    lambda p: setattr(p, "window_tokens", 0),       # window < block
    lambda p: setattr(p, "mode", 7),
    lambda p: setattr(p, "scale", -1.0),
    lambda p: setattr(p, "B", 0),
    lambda p: setattr(p, "window_exact", 2),      # only 0 or 1
])
def test_invalid_params_rejected(lib, mutate):
    p = _good()
    mutate(p)
    assert lib.lg_block_index_nnz(C.byref(p)) == -1
    assert lib.lg_block_index_bytes(C.byref(p)) == 0
    assert lib.lg_sparse_attn_workspace_bytes(C.byref(p), 0) == 0
    # fwd with (fake but aligned) pointers: rejected before anything is touched
    assert lib.lg_sparse_attn_fwd(C.byref(p), 256, 256, 256, 256, 256, 256, 1 << 30, None) == -1


def test_header_compiles_as_c(tmp_path):
    """include/lg.h is a C header: a C translation unit that includes it and takes the address of an entry
    point compiles with the C compiler (no C++ construct has slipped in)."""
    import shutil
    import subprocess
    cc = shutil.which("gcc") or shutil.which("cc")
    if cc is None:
        pytest.skip("no C compiler")
    src = tmp_path / "use_lg.c"
    src.write_text('#include "lg.h"\n'
                   'lg_status (*fwd)(const lg_attn_params*, const void*, const void*, const void*, void*, float*,\n'
                   '                 void*, size_t, void*) = lg_sparse_attn_fwd;\n'
                   'int main(void) { lg_attn_params p; lg_decode_params d; lg_device_step_buffers b;\n'
                   '  (void)p; (void)d; (void)b; return sizeof(p) == 0; }\n')
    inc = os.path.join(os.path.dirname(build.HERE), "include")
    res = subprocess.run([cc, "-std=c99", "-Wall", "-Werror", "-pedantic", "-I", inc, "-c", str(src), "-o",
                          str(tmp_path / "use_lg.o")], capture_output=True, text=True)
    assert res.returncode == 0, res.stderr


def test_prepare_and_host_step_validation(lib):
    """The entry points added around the plain forward / backward reject bad arguments on the host."""
    p = _good()
    need = lib.lg_sparse_attn_workspace_bytes(C.byref(p), 1)
    assert lib.lg_sparse_attn_prepare(C.byref(p), None, need, 1, None) == -1
    assert lib.lg_sparse_attn_prepare(C.byref(p), 128, need, 1, None) == -1          # workspace alignment
    assert lib.lg_sparse_attn_prepare(C.byref(p), 256, need - 1, 1, None) == -3
    p.lists_prepared = 2
    assert lib.lg_sparse_attn_workspace_bytes(C.byref(p), 1) == 0                      # only 0 or 1
    p.lists_prepared = 0
    p.doc_start, p.B = 256, 2                                                          # lists per sequence: no prepare
    assert lib.lg_sparse_attn_prepare(C.byref(p), 256, 1 << 30, 1, None) == -2
    # host step: group count must divide Hkv; sizes grow with the number of groups
    p = _good()
    sz = lib.lg_sparse_attn_fwd_bwd_host_workspace_bytes
    assert sz(C.byref(p), 0) == 0 and sz(C.byref(p), 3) == 0
    assert 0 < sz(C.byref(p), 1) and sz(C.byref(p), 2) > 0
    bufs = binding.DeviceStepBuffers(*([256] * 10), sz(C.byref(p), 2) - 1)
    args = [C.byref(p)] + [256] * 9 + [C.byref(bufs), 2, None, None, None]
    assert lib.lg_sparse_attn_fwd_bwd_host(*args) == -3                               # workspace too small
    bufs.workspace_bytes = sz(C.byref(p), 2)
    bufs.dq = None
    assert lib.lg_sparse_attn_fwd_bwd_host(*args) == -1                               # a staging buffer is missing
    args[3] = None
    assert lib.lg_sparse_attn_fwd_bwd_host(*args) == -1                               # a host tensor is missing
    # marked backward: the four events are mandatory
    ev = (C.c_void_p * 4)(1, 2, 3, None)
    assert lib.lg_sparse_attn_bwd_marked(C.byref(p), *([256] * 9), 256, need, None, None) == -1
    assert lib.lg_sparse_attn_bwd_marked(C.byref(p), *([256] * 9), 256, need, None, ev) == -1
    assert lib.lg_debug_kernel_launches() >= 0


def test_unsupported_head_dim(lib):
    p = _good()
    p.D = 96
    assert lib.lg_block_index_nnz(C.byref(p)) == -2


def test_null_misaligned_and_small_workspace(lib):
    p = _good()
    need = lib.lg_sparse_attn_workspace_bytes(C.byref(p), 0)
    assert lib.lg_sparse_attn_fwd(C.byref(p), None, 256, 256, 256, 256, 256, need, None) == -1
    assert lib.lg_sparse_attn_fwd(C.byref(p), 264, 256, 256, 256, 256, 256, need, None) == -1   # 8-byte aligned only
    assert lib.lg_sparse_attn_fwd(C.byref(p), 256, 256, 256, 256, 256, 128, need, None) == -1   # workspace alignment
    assert lib.lg_sparse_attn_fwd(C.byref(p), 256, 256, 256, 256, 256, 256, need - 1, None) == -3
    assert lib.lg_sparse_attn_bwd(C.byref(p), *([256] * 9), 256, need, None) == -3              # bwd needs more
    p.q_strides[0], p.q_strides[1], p.q_strides[2] = 4 * 512 * 128, 512 * 128, 100              # stride < D
    assert lib.lg_sparse_attn_fwd(C.byref(p), 256, 256, 256, 256, 256, 256, need, None) == -1
    assert lib.lg_build_block_index(C.byref(_good()), None, 256, 256, 256, None, None) == -1
    assert lib.lg_last_status(None, None) == -1


def test_chunk_prefill_planning_on_host(lib):
    """Sizes and limits of a chunk served against the ring are decided on the host."""
    p = binding.decode_params(1, 4, 2, 128, 64, 128)
    sz = lib.lg_chunk_prefill_workspace_bytes
    assert sz(C.byref(p), 0, 0) == 0 and sz(C.byref(p), 64, -1) == 0
    assert sz(C.byref(p), 60, 0) > 0           # neither the chunk nor the fill level need be a multiple of 64
    assert sz(C.byref(p), 64, 100) > sz(C.byref(p), 64, 64)
    full, more = sz(C.byref(p), 64, 1000), sz(C.byref(p), 128, 1000)
    assert 0 < full < more                     # a full ring: any fill level; longer chunk, more room
    assert sz(C.byref(p), 64, 192) == full     # exactly full = full
    assert sz(C.byref(p), 64, 64) < full       # fewer kept tokens, smaller copy
    assert sz(C.byref(binding.decode_params(1, 4, 2, 128, 32, 128)), 64, 0) == 0    # sink not a multiple of 64
    assert sz(C.byref(binding.decode_params(1, 4, 2, 96, 64, 128)), 64, 0) == 0     # head dimension
    # argument checks come before any CUDA call
    assert lib.lg_chunk_prefill(C.byref(p), None, 256, 256, 256, 256, 64, 1000, 256, 256, 256, full, None) == -1
    assert lib.lg_chunk_prefill(C.byref(p), 256, 256, 256, 256, 256, 64, 1000, 256, 256, 128, full, None) == -1   # workspace alignment
    assert lib.lg_chunk_prefill(C.byref(p), 256, 256, 256, 256, 256, 64, 1000, 256, 256, 256, full - 1, None) == -3


def test_block_aligned_decode_params_are_validated(lib):
    ok = binding.decode_params(1, 8, 1, 128, 64, 256, block_tokens=64)
    assert lib.lg_sparse_decode_workspace_bytes(C.byref(ok)) > 0
    for bad in (binding.decode_params(1, 8, 1, 128, 64, 256, block_tokens=-1),
                binding.decode_params(1, 8, 1, 128, 64, 200, block_tokens=64),      # window not whole blocks
                binding.decode_params(1, 8, 1, 128, 32, 256, block_tokens=64)):     # sink not whole blocks
        assert lib.lg_sparse_decode_workspace_bytes(C.byref(bad)) == 0
        assert lib.lg_sparse_decode(C.byref(bad), 256, 256, 256, 256, 256, None, 256, 1 << 20, None) == -1
    assert lib.lg_chunk_prefill_workspace_bytes(C.byref(binding.decode_params(1, 4, 2, 128, 64, 128, block_tokens=48)), 64, 0) == 0


def test_decode_workspace_init_rejects_bad_pointers(lib):
    assert lib.lg_sparse_decode_workspace_init(None, 1024, None) == -1
    assert lib.lg_sparse_decode_workspace_init(128, 1024, None) == -1   # not 256-byte aligned


def test_document_array_must_be_aligned(lib):
    p = _good()
    need = lib.lg_sparse_attn_workspace_bytes(C.byref(p), 1)
    p.doc_start = 258                          # not 4-byte aligned
    assert lib.lg_sparse_attn_workspace_bytes(C.byref(p), 1) == 0
    p.doc_start = 256
    assert lib.lg_sparse_attn_workspace_bytes(C.byref(p), 1) > need      # the backward keeps the documents' ends
    assert lib.lg_sparse_attn_workspace_bytes(C.byref(p), 0) == lib.lg_sparse_attn_workspace_bytes(C.byref(_good()), 0)


def test_partial_last_block_is_accepted(lib):
    p = _good()
    full = lib.lg_block_index_nnz(C.byref(p))
    p.L = p.L - 37                              # last block partial: same number of blocks, same lists
    assert lib.lg_block_index_nnz(C.byref(p)) == full
    p.L = p.L - 64                              # one block fewer
    assert 0 < lib.lg_block_index_nnz(C.byref(p)) < full


def test_documents_with_several_sequences_take_a_workspace_slice_each(lib):
    p = _good()
    p.B = 1
    p.doc_start = 256
    one = lib.lg_sparse_attn_workspace_bytes(C.byref(p), 1)
    p.B = 3
    assert lib.lg_sparse_attn_workspace_bytes(C.byref(p), 1) == 3 * one
    p.doc_start = None
    assert lib.lg_sparse_attn_workspace_bytes(C.byref(p), 1) < 3 * one      # shared lists without documents


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    """There is no CPU path: without the built CUDA library every call raises, naming the build step."""
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nothing_here.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load_library()
    with pytest.raises(RuntimeError):
        binding.lg_block_index_nnz(_good())
