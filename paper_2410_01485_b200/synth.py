"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds no attention arithmetic.  It is the only code that both the
CUDA path's harness and the CPU oracle's tests use: it names the benchmark
configurations (Llama-2 7B / 70B attention shapes at 4K-128K, Section 4.1 of the
paper) and draws iid N(0,1) tensors rounded to bf16 from a seeded generator.

The paper trains on real activations of a language model; these tensors stand
in for them.  With N(0,1) entries and scale 1/sqrt(D) the scores are ~N(0,1),
so the softmax is diffuse and no row is dominated by one key.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Optional

import torch

MODE_FULL_CAUSAL = 0
MODE_SINK_WINDOW = 1
MODE_STRIDED_LOCAL = 2


@dataclass(frozen=True)
class AttnConfig:
    """Problem statement of one fwd/bwd workload (paper Section 3.1 patterns)."""
    name: str
    B: int
    Hq: int
    Hkv: int
    L: int
    D: int
    block: int
    mode: int
    sink_tokens: int = 0
    window_tokens: int = 0
    stride_blocks: int = 0
    local_blocks: int = 0
    backward: bool = True
    window_exact: bool = False   # sink + window: token-exact window edge (matches the decode's ring)

    def full_causal(self) -> "AttnConfig":
        return replace(self, name=self.name + "_full", mode=MODE_FULL_CAUSAL)


@dataclass(frozen=True)
class DecodeConfig:
    """One-token decode over a sink + rolling-window cache (paper Section 3.2)."""
    name: str
    B: int
    Hq: int
    Hkv: int
    D: int
    sink_tokens: int
    window_tokens: int
    n_tokens: int  # context position after the append


# The five benchmark configurations.
CFG1 = AttnConfig("cfg1_tiny_sink_window", B=1, Hq=2, Hkv=2, L=512, D=64, block=64,
                  mode=MODE_SINK_WINDOW, sink_tokens=64, window_tokens=128)
CFG2 = AttnConfig("cfg2_7b_prefill_32k", B=1, Hq=32, Hkv=32, L=32768, D=128, block=64,
                  mode=MODE_SINK_WINDOW, sink_tokens=64, window_tokens=4032, backward=False)
CFG3 = AttnConfig("cfg3_7b_train_128k", B=1, Hq=32, Hkv=32, L=131072, D=128, block=128,
                  mode=MODE_SINK_WINDOW, sink_tokens=128, window_tokens=4096)
CFG4 = AttnConfig("cfg4_70b_strided_128k", B=1, Hq=64, Hkv=8, L=131072, D=128, block=64,
                  mode=MODE_STRIDED_LOCAL, stride_blocks=16, local_blocks=4)
CFG5 = DecodeConfig("cfg5_70b_decode", B=16, Hq=64, Hkv=8, D=128, sink_tokens=128,
                    window_tokens=4096, n_tokens=131072)
# The paper's own pattern settings (Section 4.1): 64-token blocks, one sink block plus
# the 32 most recent blocks; or one retained block in every 64.
PAPER_SINK = AttnConfig("paper_sink_1p32", B=1, Hq=32, Hkv=32, L=131072, D=128, block=64,
                        mode=MODE_SINK_WINDOW, sink_tokens=64, window_tokens=32 * 64)
PAPER_STRIDED = AttnConfig("paper_stride64", B=1, Hq=32, Hkv=32, L=131072, D=128, block=64,
                           mode=MODE_STRIDED_LOCAL, stride_blocks=64, local_blocks=1)

ATTN_CONFIGS: Dict[str, AttnConfig] = {c.name: c for c in (CFG1, CFG2, CFG3, CFG4, PAPER_SINK, PAPER_STRIDED)}


def _randn_bf16(shape, gen: torch.Generator, device) -> torch.Tensor:
    # Draw in fp32 in chunks along the first axis to bound peak memory, round to bf16.
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    step = 1 << 26
    for s in range(0, flat.numel(), step):
        n = min(step, flat.numel() - s)
        flat[s:s + n] = torch.randn(n, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)
    return out


def make_attn_inputs(cfg: AttnConfig, device="cpu", seed: int = 0, with_do: Optional[bool] = None):
    """Q [B,Hq,L,D], K,V [B,Hkv,L,D], dO [B,Hq,L,D]: bf16, iid N(0,1), drawn in that
    order from one generator seeded with `seed` (inputs are taken as already rotated
    by RoPE).  Returns a dict of contiguous tensors on `device`."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    out = {
        "q": _randn_bf16((cfg.B, cfg.Hq, cfg.L, cfg.D), gen, dev),
        "k": _randn_bf16((cfg.B, cfg.Hkv, cfg.L, cfg.D), gen, dev),
        "v": _randn_bf16((cfg.B, cfg.Hkv, cfg.L, cfg.D), gen, dev),
    }
    if cfg.backward if with_do is None else with_do:
        out["do"] = _randn_bf16((cfg.B, cfg.Hq, cfg.L, cfg.D), gen, dev)
    return out


def make_decode_inputs(cfg: DecodeConfig, device="cpu", seed: int = 0, capacity: Optional[int] = None):
    """q [B,Hq,D] and cache K,V [B,Hkv,capacity,D] (bf16, iid N(0,1)).  `capacity`
    defaults to sink+window slots; pass n_tokens for the dense linear-cache comparator."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    cap = cfg.sink_tokens + cfg.window_tokens if capacity is None else capacity
    return {
        "q": _randn_bf16((cfg.B, cfg.Hq, cfg.D), gen, dev),
        "k_cache": _randn_bf16((cfg.B, cfg.Hkv, cap, cfg.D), gen, dev),
        "v_cache": _randn_bf16((cfg.B, cfg.Hkv, cap, cfg.D), gen, dev),
    }


def make_doc_start(L: int, seed: int = 0, mean_len: int = 700, device="cpu") -> torch.Tensor:
    """doc_start[i] (int32 [L]) for documents packed back to back into a sample of L tokens: lengths are
    drawn from a seeded exponential distribution with the given mean (a few long documents, many short
    ones, as in a web corpus), at least 1 token each; the last document is cut at L."""
    gen = torch.Generator().manual_seed(seed)
    out = torch.empty(L, dtype=torch.int32)
    pos = 0
    while pos < L:
        n = max(1, int(-mean_len * torch.log(1.0 - torch.rand(1, generator=gen)).item()))
        out[pos:pos + n] = pos
        pos += n
    return out.to(device)


def to_f64(t: torch.Tensor):
    """Exact widening of a bf16/fp32 tensor to a float64 numpy array (host)."""
    return t.detach().to("cpu").to(torch.float64).numpy()
