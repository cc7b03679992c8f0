"""The checked build of the library (-DLG_DEBUG): every schedule value the kernels use as an index, an
offset or an address is bounds-checked and a value out of range is reported through the status word
instead of being used.  On a healthy workspace the checks are silent and change nothing: the checked
library returns, bit for bit, what the normal one returns, for both backward variants."""
import importlib.util
from dataclasses import replace

import pytest
import torch

from paper_2410_01485_b200 import binding, build, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def libs():
    build.build()
    path = build.build(debug=True)
    binding.load_library()
    spec = importlib.util.spec_from_file_location("lg_binding_checked", binding.__file__)
    checked = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(checked)
    checked.LIB_PATH = path
    checked.load_library()
    return binding, checked


@pytest.mark.parametrize("variant", ["two_pass", "keep_ds"])
@pytest.mark.parametrize("cfg", [
    replace(synth.CFG1, name="dbg_bs64_gqa", L=1024 + 40, D=128, Hq=4, Hkv=2),
    replace(synth.CFG1, name="dbg_bs128", block=128, sink_tokens=128, window_tokens=256, L=1536, D=128),
    replace(synth.CFG1, name="dbg_strided", mode=synth.MODE_STRIDED_LOCAL, stride_blocks=4, local_blocks=2, L=2048, D=64),
], ids=lambda c: c.name)
def test_checked_build_is_silent_and_identical(libs, cfg, variant, monkeypatch):
    monkeypatch.setenv("LG_BWD_VARIANT", variant)
    normal, checked = libs
    inp = synth.make_attn_inputs(cfg, "cuda", seed=5, with_do=True)
    outs = []
    for lg in (normal, checked):
        p = lg.params_of(cfg)
        ws = lg.attn_workspace(p, True)
        lg.lg_sparse_attn_prepare(p, ws, True)
        o, lse = lg.lg_sparse_attn_fwd(p, inp["q"], inp["k"], inp["v"], workspace=ws)
        dq, dk, dv = lg.lg_sparse_attn_bwd(p, inp["q"], inp["k"], inp["v"], o, lse, inp["do"], workspace=ws)
        assert lg.lg_last_status(ws) == 0
        outs.append((o, lse, dq, dk, dv))
    for x, y in zip(*outs):
        assert torch.equal(x, y)
