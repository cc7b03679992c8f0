"""lg_sparse_decode_static: the decode entry point for callers that cannot allocate.

Some users of this library run where device memory cannot be requested at call time (a
serving loop whose pool was handed out at start-up, a plug-in without its host's allocator,
a step that must not hit cudaMalloc's implicit synchronisation).  For them the library keeps
the split-KV partials in a fixed array of its own.  The checks here: the call rejects a
problem whose partials exceed that array, and on the GPU it returns what lg_sparse_decode
returns, twice in a row (the array is shared by all calls and keeps the previous call's
contents, so the second call must not be disturbed by what the first one left behind).

This file is named so that pytest collects it last.
"""
import ctypes as C

import pytest
import torch

from paper_2410_01485_b200 import binding as lg, build, synth

TOL_O = 1e-2      # max-abs on bf16 outputs, as in the parity tests
TOL_LSE = 1e-3


@pytest.fixture(scope="module")
def lib():
    build.build()
    return lg.load_library()


def test_static_decode_rejects_problems_beyond_the_fixed_array(lib):
    """Host-only: the size check comes before any CUDA call, so it runs without a GPU."""
    big = lg.decode_params(1024, 64, 8, 128, 128, 1 << 20)
    assert lib.lg_sparse_decode_workspace_bytes(C.byref(big)) > lg.DECODE_STATIC_SCRATCH_BYTES
    rc = lib.lg_sparse_decode_static(C.byref(big), 16, 16, 16, 16, 16, None, None)
    assert rc == -3 and "workspace" in lg.status_string(rc)
    # the headline decode shape fits
    c = synth.CFG5
    fits = lg.decode_params(c.B, c.Hq, c.Hkv, c.D, c.sink_tokens, c.window_tokens)
    assert 0 < lib.lg_sparse_decode_workspace_bytes(C.byref(fits)) <= lg.DECODE_STATIC_SCRATCH_BYTES
    # invalid parameters are still reported as such
    bad = lg.decode_params(1, 7, 2, 128, 0, 16)
    assert lib.lg_sparse_decode_static(C.byref(bad), 16, 16, 16, 16, 16, None, None) == -1


@pytest.mark.gpu
def test_static_decode_matches_workspace_decode_twice(lib):
    c = synth.CFG5
    B = 4
    p = lg.decode_params(B, c.Hq, c.Hkv, c.D, c.sink_tokens, c.window_tokens)
    cap = c.sink_tokens + c.window_tokens
    g = torch.Generator(device="cuda").manual_seed(7)
    calls = []
    for n_list in ([cap + 1000, cap, 777, 1], [5, cap + 3, 4000, 131072]):   # second call: other lengths, other data
        q = torch.randn(B, c.Hq, c.D, generator=g, device="cuda").to(torch.bfloat16)
        kc = torch.randn(B, c.Hkv, cap, c.D, generator=g, device="cuda").to(torch.bfloat16)
        vc = torch.randn(B, c.Hkv, cap, c.D, generator=g, device="cuda").to(torch.bfloat16)
        n_t = torch.tensor(n_list, dtype=torch.int64, device="cuda")
        calls.append((q, kc, vc, n_t))
    refs = [lg.lg_sparse_decode(p, q, kc, vc, n_t) for (q, kc, vc, n_t) in calls]
    torch.cuda.synchronize()
    for (q, kc, vc, n_t), (o_ref, lse_ref) in zip(calls, refs):
        o = torch.full_like(q, float("nan"))
        lse = torch.full((B, c.Hq), float("nan"), dtype=torch.float32, device="cuda")
        lg.lg_sparse_decode_static(p, q, kc, vc, n_t, o, lse)
        torch.cuda.synchronize()
        assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
        assert (o.float() - o_ref.float()).abs().max().item() <= TOL_O
        assert (lse - lse_ref).abs().max().item() <= TOL_LSE
        assert torch.equal(o, o_ref) and torch.equal(lse, lse_ref)   # same kernels, same order: same bits


@pytest.mark.gpu
def test_static_decode_second_shape_over_the_first_ones_leftovers_and_no_allocation(lib):
    """Two problems of different shape, one after the other, share the fixed array: the second (other batch,
    head counts, head dimension and lengths, hence other units, counters and record layout) must not be
    disturbed by what the first left there.  And the call requests no device memory: the bytes the driver
    reports free and the bytes torch has handed out are the same before and after it."""
    g = torch.Generator(device="cuda").manual_seed(11)
    shapes = [(4, 64, 8, 128, 128, 4096, [5000, 4224, 777, 131072]),   # the headline head layout, split units
              (3, 12, 4, 64, 64, 512, [600, 1, 300])]                   # other B / Hkv / G / D / capacity
    for B, Hq, Hkv, D, sink, W, n_list in shapes:
        p = lg.decode_params(B, Hq, Hkv, D, sink, W)
        cap = sink + W
        q = torch.randn(B, Hq, D, generator=g, device="cuda").to(torch.bfloat16)
        kc = torch.randn(B, Hkv, cap, D, generator=g, device="cuda").to(torch.bfloat16)
        vc = torch.randn(B, Hkv, cap, D, generator=g, device="cuda").to(torch.bfloat16)
        n_t = torch.tensor(n_list, dtype=torch.int64, device="cuda")
        o_ref, lse_ref = lg.lg_sparse_decode(p, q, kc, vc, n_t)
        o = torch.full_like(q, float("nan"))
        lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device="cuda")
        lg.lg_sparse_decode_static(p, q, kc, vc, n_t, o, lse)      # (first call of a shape: one-time set-up of the device's facts)
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        held0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
        o.fill_(float("nan")); lse.fill_(float("nan"))
        lg.lg_sparse_decode_static(p, q, kc, vc, n_t, o, lse)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0, "the call changed the device's free memory by %d bytes" % (free0 - free1)
        assert torch.cuda.memory_allocated() == held0 and torch.cuda.memory_reserved() == reserved0
        assert torch.equal(o, o_ref) and torch.equal(lse, lse_ref)
