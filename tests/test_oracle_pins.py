"""Pins for the CPU oracle: each test ties it to something other than itself --
numbers the paper prints, closed forms, textbook/library special cases, brute force
on tiny inputs, finite differences.  No GPU needed."""
import math

import numpy as np
import pytest
import torch

from oracle import lg_oracle as O
from paper_2410_01485_b200 import synth


def _read_kv(path):
    out = {}
    with open(path) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = [s.strip() for s in line.split("=")]
                out[k] = float(v)
    return out


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


TINY_PATTERNS = [
    O.Pattern(L=32, block=4, mode=O.MODE_SINK_WINDOW, sink_tokens=4, window_tokens=8),
    O.Pattern(L=32, block=4, mode=O.MODE_SINK_WINDOW, sink_tokens=8, window_tokens=4),
    O.Pattern(L=48, block=8, mode=O.MODE_STRIDED_LOCAL, stride_blocks=2, local_blocks=1),
    O.Pattern(L=40, block=4, mode=O.MODE_STRIDED_LOCAL, stride_blocks=3, local_blocks=2),
    O.Pattern(L=24, block=8, mode=O.MODE_FULL_CAUSAL),
]


# ----------------------------------------------------------------- patterns / lists

def test_paper_retained_tokens_and_kv_budget(golden_dir):
    """Section 4.1 / 4.3: ~2K retained tokens per sparse layer at 128K; 69.2 GB -> 26.5 GB."""
    g = _read_kv(golden_dir + "/paper_arithmetic.txt")
    Bs, L = int(g["block_tokens"]), int(g["seq_len"])
    sink = O.Pattern(L=L, block=Bs, mode=O.MODE_SINK_WINDOW, sink_tokens=int(g["sink_blocks"]) * Bs,
                     window_tokens=int(g["local_blocks"]) * Bs)
    last = O.allowed(sink, L - 1, np.arange(L))
    assert last.sum() == (1 + 32) * 64 - 0  # last row of its block sees every retained token
    assert abs(last.sum() - g["retained_tokens_approx"]) / g["retained_tokens_approx"] < 0.05
    strided = O.Pattern(L=L, block=Bs, mode=O.MODE_STRIDED_LOCAL, stride_blocks=int(g["stride_blocks"]),
                        local_blocks=1)
    comb = O.allowed(strided, L - 1, np.arange(L))
    # 2048 blocks / 64 = 32 comb blocks (+ the query's own block)
    assert abs(comb.sum() - g["retained_tokens_approx"]) / g["retained_tokens_approx"] < 0.05
    # KV bytes: what decode keeps per sparse layer is what the last query may see.
    per_tok_layer = 2 * g["n_heads"] * g["head_dim"] * g["bytes_per_value"]
    full_gb = g["n_layers"] * per_tok_layer * L / 1e9
    assert abs(full_gb - g["kv_full_gb"]) / g["kv_full_gb"] < 0.01
    n_sparse = g["n_layers"] - g["n_full_layers"]
    kept = O.decode_valid(L, int(g["sink_blocks"]) * Bs, int(g["local_blocks"]) * Bs).sum()
    assert kept == last.sum()
    hybrid_gb = (g["n_full_layers"] * per_tok_layer * L + n_sparse * per_tok_layer * kept) / 1e9
    assert abs(hybrid_gb - g["kv_hybrid_gb"]) < 0.06
    assert abs(100 * (1 - hybrid_gb / full_gb) - g["kv_saving_pct"]) < 1.0


def _nnz_closed_form(cfg):
    nB = cfg.L // cfg.block
    if cfg.mode == synth.MODE_FULL_CAUSAL:
        return nB * (nB + 1) // 2
    if cfg.mode == synth.MODE_SINK_WINDOW:
        ns, nw = cfg.sink_tokens // cfg.block, cfg.window_tokens // cfg.block
        return sum(min(qb + 1, nw) + min(ns, max(qb + 1 - nw, 0)) for qb in range(nB))
    nl, s = cfg.local_blocks, cfg.stride_blocks
    return sum(min(qb + 1, nl) + -(-max(qb - nl + 1, 0) // s) for qb in range(nB))


@pytest.mark.parametrize("cfg", [synth.CFG1, synth.CFG2, synth.CFG2.full_causal()], ids=lambda c: c.name)
def test_block_counts_match_closed_form(cfg, golden_dir):
    g = _read_kv(golden_dir + "/block_counts.txt")
    row_ptr, col_idx, col_ptr, row_idx = O.block_lists(O.Pattern.of(cfg))
    assert int(row_ptr[-1]) == int(g[cfg.name]) == _nnz_closed_form(cfg)
    assert len(col_idx) == len(row_idx) == int(g[cfg.name])


def test_block_counts_golden_closed_forms_128k(golden_dir):
    """The 128K entries of the fixture agree with the hand-derived row formulas (the
    mask-derived lists at 128K are checked against the same numbers in the GPU tests)."""
    g = _read_kv(golden_dir + "/block_counts.txt")
    for cfg in (synth.CFG3, synth.CFG4, synth.PAPER_SINK):
        assert _nnz_closed_form(cfg) == int(g[cfg.name])


def test_block_counts_128k_scaled_down():
    """Same patterns as the 128K configs at 1/8 of the length: counted from the mask."""
    from dataclasses import replace
    for cfg in (synth.CFG3, synth.CFG4, synth.PAPER_SINK, synth.PAPER_STRIDED):
        small = replace(cfg, L=cfg.L // 8)
        assert int(O.block_lists(O.Pattern.of(small))[0][-1]) == _nnz_closed_form(small)


@pytest.mark.parametrize("p", TINY_PATTERNS)
def test_lists_structure(p):
    row_ptr, col_idx, col_ptr, row_idx = O.block_lists(p)
    nB = p.L // p.block
    dense = np.zeros((nB, nB), dtype=bool)
    for qb in range(nB):
        cols = col_idx[row_ptr[qb]:row_ptr[qb + 1]]
        assert (np.diff(cols) > 0).all()            # ascending, no duplicates
        assert cols[-1] == qb                       # diagonal block always active, nothing above it
        dense[qb, cols] = True
    # CSC is the exact transpose
    dense_t = np.zeros((nB, nB), dtype=bool)
    for kb in range(nB):
        rows = row_idx[col_ptr[kb]:col_ptr[kb + 1]]
        assert (np.diff(rows) > 0).all()
        dense_t[rows, kb] = True
    assert (dense == dense_t).all()
    # brute force over token pairs with python loops
    for qb in range(nB):
        for kb in range(nB):
            any_pair = any(bool(O.allowed(p, i, j)) for i in range(qb * p.block, (qb + 1) * p.block)
                           for j in range(kb * p.block, (kb + 1) * p.block))
            assert any_pair == dense[qb, kb]


def test_sink_window_rows_are_sink_plus_contiguous_run():
    """What a query sees under sink+window: the sink tokens and one contiguous run ending
    at itself whose length lies in ((nw-1)*Bs, nw*Bs] (block-granular window, own block
    counted) -- stated without the predicate's formula."""
    p = O.Pattern(L=96, block=8, mode=O.MODE_SINK_WINDOW, sink_tokens=8, window_tokens=24)
    M = O.token_mask(p)
    for i in range(p.L):
        seen = np.nonzero(M[i])[0]
        assert seen[-1] == i and (seen <= i).all()
        run = 1
        while run < len(seen) and seen[-run - 1] == seen[-run] - 1:
            run += 1
        rest = seen[:-run]
        if len(rest):                                  # the run does not reach the sink
            assert list(rest) == list(range(8))
            assert 16 < run <= 24
            assert (i - run + 1) % 8 == 0              # run starts on a block boundary
        else:
            assert run == i + 1                        # everything up to i


def test_strided_rows_keep_absolute_comb():
    p = O.Pattern(L=128, block=8, mode=O.MODE_STRIDED_LOCAL, stride_blocks=4, local_blocks=2)
    M = O.token_mask(p)
    far = M[:, :]
    for i in (40, 77, 127):
        seen_blocks = sorted(set(np.nonzero(far[i])[0] // 8))
        qb = i // 8
        comb = [b for b in seen_blocks if b < qb - 1]
        assert comb == [b for b in range(0, qb - 1) if b % 4 == 0]   # same comb for every query
        assert seen_blocks[-2:] == [qb - 1, qb]


def test_wide_window_is_full_causal():
    L = 64
    full = O.token_mask(O.Pattern(L=L, block=8, mode=O.MODE_FULL_CAUSAL))
    assert (full == np.tril(np.ones((L, L), dtype=bool))).all()
    assert (O.token_mask(O.Pattern(L=L, block=8, mode=O.MODE_SINK_WINDOW, sink_tokens=8, window_tokens=L)) == full).all()
    assert (O.token_mask(O.Pattern(L=L, block=8, mode=O.MODE_STRIDED_LOCAL, stride_blocks=1, local_blocks=1)) == full).all()
    assert (O.token_mask(O.Pattern(L=L, block=8, mode=O.MODE_STRIDED_LOCAL, stride_blocks=5, local_blocks=8)) == full).all()


def test_pair_count_ratio_cfg3_scaled():
    """Section 3.3: sparse-layer cost is a small fraction of dense when S << N.  For the
    128K sink+window setting the exact pair ratio is 0.0625; at 1/8 length it is 8x that
    minus edge effects -- compare the mask count with the closed form."""
    from dataclasses import replace
    cfg = replace(synth.CFG3, L=synth.CFG3.L // 8)
    Bs, nB = cfg.block, cfg.L // cfg.block
    ns, nw = 1, cfg.window_tokens // Bs
    blocks_full = sum(min(qb + 1, nw) - 1 + min(ns, max(qb + 1 - nw, 0)) for qb in range(nB))
    expect = blocks_full * Bs * Bs + nB * Bs * (Bs + 1) // 2
    assert O.count_pairs(O.Pattern.of(cfg)) == expect
    # the closed form at the full 128K length gives the 0.0625 of the measurement plan
    nB = synth.CFG3.L // Bs
    blocks_full = sum(min(qb + 1, nw) - 1 + min(ns, max(qb + 1 - nw, 0)) for qb in range(nB))
    pairs = blocks_full * Bs * Bs + nB * Bs * (Bs + 1) // 2
    assert pairs == 536674304
    assert abs(pairs / (synth.CFG3.L * (synth.CFG3.L + 1) // 2) - 0.0625) < 5e-4


# -------------------------------------------------------------------------- forward

def _brute_forward_row(q, k, v, p, scale, h, g, i):
    js = [j for j in range(p.L) if bool(O.allowed(p, i, j))]
    s = [scale * sum(q[h, i, d] * k[g, j, d] for d in range(q.shape[2])) for j in js]
    m = max(s)
    e = [math.exp(x - m) for x in s]
    z = sum(e)
    o = [sum(e[t] / z * v[g, js[t], d] for t in range(len(js))) for d in range(q.shape[2])]
    return o, m + math.log(z), e, z


@pytest.mark.parametrize("p", TINY_PATTERNS)
def test_forward_vs_bruteforce_rows(p):
    Hq, Hkv, D = 4, 2, 5
    q, k, v = _rand((Hq, p.L, D), 1), _rand((Hkv, p.L, D), 2), _rand((Hkv, p.L, D), 3)
    scale = 0.37
    Oo, LSE = O.attn_forward(q, k, v, p, scale)
    for h in range(Hq):
        for i in range(0, p.L, 3):
            o, lse, _, _ = _brute_forward_row(q, k, v, p, scale, h, h // 2, i)
            np.testing.assert_allclose(Oo[h, i], o, rtol=1e-12, atol=1e-13)
            assert abs(LSE[h, i] - lse) < 1e-12


def test_forward_full_causal_equals_torch_sdpa():
    """Special case that reduces to a library routine: dense causal attention in fp64."""
    Hq, Hkv, L, D = 4, 2, 48, 8
    q, k, v = _rand((Hq, L, D), 4), _rand((Hkv, L, D), 5), _rand((Hkv, L, D), 6)
    scale = 1 / math.sqrt(D)
    tq, tk, tv = (torch.from_numpy(x) for x in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(
        tq[None], tk.repeat_interleave(2, 0)[None], tv.repeat_interleave(2, 0)[None], is_causal=True, scale=scale)[0].numpy()
    for p in (O.Pattern(L=L, block=8, mode=O.MODE_FULL_CAUSAL),
              O.Pattern(L=L, block=8, mode=O.MODE_SINK_WINDOW, sink_tokens=8, window_tokens=L),
              O.Pattern(L=L, block=8, mode=O.MODE_STRIDED_LOCAL, stride_blocks=1, local_blocks=1)):
        got, lse = O.attn_forward(q, k, v, p, scale)
        np.testing.assert_allclose(got, ref, rtol=1e-11, atol=1e-12)
        # LSE against torch.logsumexp over the causal prefix
        for h in (0, 3):
            s = scale * (tq[h] @ tk[h // 2].T)
            s = s.masked_fill(~torch.ones(L, L, dtype=torch.bool).tril(), float("-inf"))
            np.testing.assert_allclose(lse[h], torch.logsumexp(s, dim=1).numpy(), rtol=1e-12)


@pytest.mark.parametrize("p", TINY_PATTERNS)
def test_forward_invariants(p):
    Hq, Hkv, D = 2, 1, 6
    q, k, v = _rand((Hq, p.L, D), 7), _rand((Hkv, p.L, D), 8), _rand((Hkv, p.L, D), 9)
    scale = 0.5
    Oo, LSE = O.attn_forward(q, k, v, p, scale)
    # row 0 sees only key 0
    np.testing.assert_allclose(Oo[:, 0], np.broadcast_to(v[0, 0], (Hq, D)), rtol=1e-13)
    np.testing.assert_allclose(LSE[:, 0], scale * q[:, 0] @ k[0, 0], rtol=1e-13)
    # LSE bounds: max <= LSE <= max + log(count)
    M = O.token_mask(p)
    for h in range(Hq):
        S = np.where(M, scale * q[h] @ k[0].T, -np.inf)
        assert (LSE[h] >= S.max(1) - 1e-12).all()
        assert (LSE[h] <= S.max(1) + np.log(M.sum(1)) + 1e-12).all()
        # rows of P = exp(S - LSE) sum to one
        np.testing.assert_allclose(np.exp(S - LSE[h][:, None]).sum(1), 1.0, rtol=1e-12)
    # all keys equal -> uniform weights -> O is the mean of the visible values
    k_same = np.broadcast_to(k[:, :1], k.shape).copy()
    O2, LSE2 = O.attn_forward(q, k_same, v, p, scale)
    for i in (0, p.L // 2, p.L - 1):
        np.testing.assert_allclose(O2[1, i], v[0, M[i]].mean(0), rtol=1e-12, atol=1e-13)
        assert abs(LSE2[1, i] - (scale * q[1, i] @ k[0, 0] + math.log(M[i].sum()))) < 1e-12
    # V = const vector -> O = that vector
    v_const = np.broadcast_to(v[:, :1], v.shape).copy()
    O3, _ = O.attn_forward(q, k, v_const, p, scale)
    np.testing.assert_allclose(O3, np.broadcast_to(v[0, 0], O3.shape), rtol=1e-12)


def test_masked_keys_do_not_influence_output():
    p = O.Pattern(L=64, block=8, mode=O.MODE_SINK_WINDOW, sink_tokens=8, window_tokens=16)
    q, k, v = _rand((1, 64, 4), 10), _rand((1, 64, 4), 11), _rand((1, 64, 4), 12)
    O1, L1 = O.attn_forward(q, k, v, p, 0.5)
    k2, v2 = k.copy(), v.copy()
    k2[0, 8:16] += 100.0   # block 1: invisible to queries of blocks >= 3
    v2[0, 8:16] -= 50.0
    O2, L2 = O.attn_forward(q, k2, v2, p, 0.5)
    assert (O1[0, 24:] == O2[0, 24:]).all() and (L1[0, 24:] == L2[0, 24:]).all()
    assert not np.allclose(O1[0, 8:24], O2[0, 8:24])


def test_slab_oracle_equals_dense_oracle():
    for p in TINY_PATTERNS:
        q, k, v, do = (_rand((4, p.L, 3), s) for s in (13, 14, 15, 16))
        k, v = k[:2], v[:2]
        a = O.attn_backward(q, k, v, do, p, 0.3)
        b = O.attn_backward(q, k, v, do, p, 0.3, rows_per_slab=p.block)
        c = O.attn_forward(q, k, v, p, 0.3, rows_per_slab=2 * p.block)
        for x, y in zip(a, b):
            np.testing.assert_allclose(x, y, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(a[3], c[0], rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(a[4], c[1], rtol=1e-12, atol=1e-13)


def test_subset_evaluators_equal_full_oracle():
    """attn_rows / attn_keys_grad (used at 128K, where only samples are affordable) give
    the same numbers as the pinned full evaluation."""
    for p in TINY_PATTERNS:
        q, k, v, do = (_rand((4, p.L, 3), s) for s in (17, 18, 19, 20))
        k, v = k[:2], v[:2]
        dQ, dK, dV, Oo, LSE = O.attn_backward(q, k, v, do, p, 0.3)
        for r0 in range(0, p.L, p.block):
            o, lse, dq = O.attn_rows(q, k, v, do, p, 0.3, r0, r0 + p.block)
            np.testing.assert_allclose(o, Oo[:, r0:r0 + p.block], rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(lse, LSE[:, r0:r0 + p.block], rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(dq, dQ[:, r0:r0 + p.block], rtol=1e-12, atol=1e-13)
            dk, dv = O.attn_keys_grad(q, k, v, do, p, 0.3, r0, r0 + p.block)
            np.testing.assert_allclose(dk, dK[:, r0:r0 + p.block], rtol=1e-11, atol=1e-12)
            np.testing.assert_allclose(dv, dV[:, r0:r0 + p.block], rtol=1e-11, atol=1e-12)
        dk, dv = O.attn_keys_grad(q, k, v, do, p, 0.3, 3, p.L - 5)
        np.testing.assert_allclose(dk, dK[:, 3:p.L - 5], rtol=1e-11, atol=1e-12)
    # a sequence that ends inside a block: the last slab of rows is shorter than a block
    for p in (O.Pattern(L=30, block=4, mode=O.MODE_SINK_WINDOW, sink_tokens=4, window_tokens=8),
              O.Pattern(L=43, block=8, mode=O.MODE_STRIDED_LOCAL, stride_blocks=2, local_blocks=1)):
        q, k, v, do = (_rand((4, p.L, 3), s) for s in (27, 28, 29, 30))
        k, v = k[:2], v[:2]
        dQ, dK, dV, Oo, LSE = O.attn_backward(q, k, v, do, p, 0.3)
        for j0, j1 in ((0, p.L), (p.L - 3, p.L), (5, p.L - 1)):
            dk, dv = O.attn_keys_grad(q, k, v, do, p, 0.3, j0, j1)
            np.testing.assert_allclose(dk, dK[:, j0:j1], rtol=1e-11, atol=1e-12)
            np.testing.assert_allclose(dv, dV[:, j0:j1], rtol=1e-11, atol=1e-12)
        o, lse, dq = O.attn_rows(q, k, v, do, p, 0.3, p.L - 5, p.L)
        np.testing.assert_allclose(o, Oo[:, p.L - 5:], rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(dq, dQ[:, p.L - 5:], rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------------- backward

def _loss(q, k, v, do, p, scale):
    return float((O.attn_forward(q, k, v, p, scale)[0] * do).sum())


@pytest.mark.parametrize("p", TINY_PATTERNS[:4])
def test_backward_finite_differences(p):
    Hq, Hkv, D = 2, 1, 3
    q, k, v, do = _rand((Hq, p.L, D), 20), _rand((Hkv, p.L, D), 21), _rand((Hkv, p.L, D), 22), _rand((Hq, p.L, D), 23)
    scale = 0.6
    dQ, dK, dV, _, _ = O.attn_backward(q, k, v, do, p, scale)
    rng = np.random.default_rng(0)
    eps = 1e-5
    for name, x, gx in (("q", q, dQ), ("k", k, dK), ("v", v, dV)):
        for _ in range(12):
            idx = tuple(rng.integers(0, s) for s in x.shape)
            old = x[idx]
            x[idx] = old + eps
            up = _loss(q, k, v, do, p, scale)
            x[idx] = old - eps
            dn = _loss(q, k, v, do, p, scale)
            x[idx] = old
            fd = (up - dn) / (2 * eps)
            assert abs(fd - gx[idx]) <= 1e-6 * max(1.0, abs(fd)), (name, idx, fd, gx[idx])


@pytest.mark.parametrize("p", TINY_PATTERNS)
def test_backward_equals_torch_autograd(p):
    """Library autodiff of masked softmax attention in fp64 (GQA by repeat_interleave)."""
    Hq, Hkv, D = 4, 2, 5
    q, k, v, do = _rand((Hq, p.L, D), 30), _rand((Hkv, p.L, D), 31), _rand((Hkv, p.L, D), 32), _rand((Hq, p.L, D), 33)
    scale = 0.45
    tq, tk, tv = (torch.from_numpy(x).requires_grad_(True) for x in (q, k, v))
    M = torch.from_numpy(O.token_mask(p))
    s = scale * torch.einsum("hid,hjd->hij", tq, tk.repeat_interleave(2, 0))
    pr = torch.softmax(s.masked_fill(~M, float("-inf")), dim=-1)
    out = torch.einsum("hij,hjd->hid", pr, tv.repeat_interleave(2, 0))
    (out * torch.from_numpy(do)).sum().backward()
    dQ, dK, dV, Oo, _ = O.attn_backward(q, k, v, do, p, scale)
    np.testing.assert_allclose(Oo, out.detach().numpy(), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(dQ, tq.grad.numpy(), rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(dK, tk.grad.numpy(), rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(dV, tv.grad.numpy(), rtol=1e-10, atol=1e-11)


def test_backward_masked_keys_get_exactly_zero():
    p = O.Pattern(L=64, block=8, mode=O.MODE_SINK_WINDOW, sink_tokens=8, window_tokens=16)
    q, k, v, do = (_rand((2, 64, 4), s) for s in (40, 41, 42, 43))
    do[:, :24] = 0.0      # only queries of blocks >= 3 carry gradient; they cannot see block 1
    dQ, dK, dV, _, _ = O.attn_backward(q, k, v, do, p, 0.5)
    assert (dK[:, 8:16] == 0).all() and (dV[:, 8:16] == 0).all()
    assert np.abs(dK[:, 0:8]).max() > 0 and np.abs(dV[:, 16:24]).max() > 0
    assert (dQ[:, :24] == 0).all()


@pytest.mark.parametrize("p", TINY_PATTERNS)
def test_backward_shift_invariances(p):
    """softmax is invariant to adding one vector to every key, so sum_j dK_j = 0 per kv
    head (a consequence of sum_j dS_ij = 0); and sum_j dV_j = sum_i dO_i per group."""
    Hq, Hkv, D = 4, 2, 3
    q, k, v, do = _rand((Hq, p.L, D), 50), _rand((Hkv, p.L, D), 51), _rand((Hkv, p.L, D), 52), _rand((Hq, p.L, D), 53)
    dQ, dK, dV, _, _ = O.attn_backward(q, k, v, do, p, 0.7)
    np.testing.assert_allclose(dK.sum(1), 0.0, atol=1e-11)
    np.testing.assert_allclose(dV.sum(1), do.reshape(Hkv, 2, p.L, D).sum((1, 2)), rtol=1e-11)


def test_backward_gqa_is_sum_of_mha_groups():
    p = TINY_PATTERNS[3]
    Hq, Hkv, D = 6, 2, 4
    q, k, v, do = _rand((Hq, p.L, D), 60), _rand((Hkv, p.L, D), 61), _rand((Hkv, p.L, D), 62), _rand((Hq, p.L, D), 63)
    dQ, dK, dV, _, _ = O.attn_backward(q, k, v, do, p, 0.5)
    kr, vr = np.repeat(k, 3, axis=0), np.repeat(v, 3, axis=0)
    dQm, dKm, dVm, _, _ = O.attn_backward(q, kr, vr, do, p, 0.5)
    np.testing.assert_allclose(dQ, dQm, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dK, dKm.reshape(Hkv, 3, p.L, D).sum(1), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dV, dVm.reshape(Hkv, 3, p.L, D).sum(1), rtol=1e-12, atol=1e-13)


# --------------------------------------------------------------------- decode / ring

def test_decode_dense_equals_full_causal_last_row():
    Hq, Hkv, n, D = 4, 2, 40, 8
    q, k, v = _rand((Hq, n, D), 70), _rand((Hkv, n, D), 71), _rand((Hkv, n, D), 72)
    Oo, LSE = O.attn_forward(q, k, v, O.Pattern(L=n, block=8, mode=O.MODE_FULL_CAUSAL), 0.35)
    o, lse = O.decode(q[:, n - 1], k, v, n, sink=0, window=n, scale=0.35)
    np.testing.assert_allclose(o, Oo[:, n - 1], rtol=1e-12)
    np.testing.assert_allclose(lse, LSE[:, n - 1], rtol=1e-12)


def test_decode_bruteforce_and_permutation_invariance():
    Hq, Hkv, D, sink, W = 4, 2, 4, 3, 5
    rng = np.random.default_rng(5)
    for n in (1, 2, 3, 4, 8, 9, 23):
        q, k, v = _rand((Hq, D), 80 + n), _rand((Hkv, n, D), 81 + n), _rand((Hkv, n, D), 82 + n)
        o, lse = O.decode(q, k, v, n, sink, W, 0.5)
        keep = [j for j in range(n) if j < sink or j >= n - W]
        assert len(keep) == min(n, sink + W) or n - W < sink
        for h in range(Hq):
            s = [0.5 * float(q[h] @ k[h // 2, j]) for j in keep]
            m = max(s)
            z = sum(math.exp(x - m) for x in s)
            ref = sum(math.exp(s[t] - m) / z * v[h // 2, keep[t]] for t in range(len(keep)))
            np.testing.assert_allclose(o[h], ref, rtol=1e-12)
            assert abs(lse[h] - (m + math.log(z))) < 1e-12
        # a set function of the surviving (k, v) pairs: shuffle them inside the history
        if n == 23:
            perm = np.array(keep)
            shuffled = rng.permutation(perm)
            k2, v2 = k.copy(), v.copy()
            k2[:, perm], v2[:, perm] = k[:, shuffled], v[:, shuffled]
            o2, lse2 = O.decode(q, k2, v2, n, sink, W, 0.5)
            np.testing.assert_allclose(o2, o, rtol=1e-12)
    o0, lse0 = O.decode(_rand((Hq, D), 1), np.zeros((Hkv, 0, D)), np.zeros((Hkv, 0, D)), 0, sink, W, 0.5)
    assert (o0 == 0).all() and np.isneginf(lse0).all()


def test_block_aligned_decode_is_the_training_masks_row():
    """With block_tokens the serving mask is the block-granular training mask (Section 4.1: the local
    context is counted in blocks): the decode at position n - 1 equals row n - 1 of the mask-based forward
    under the default (block-granular) pattern, for every n, and its keys are tokens the ring still holds."""
    Hq, Hkv, D, Bs, sink, W = 4, 2, 6, 4, 4, 12
    L = 61
    q, k, v = _rand((Hq, L, D), 90), _rand((Hkv, L, D), 91), _rand((Hkv, L, D), 92)
    pat = O.Pattern(L=L, block=Bs, mode=O.MODE_SINK_WINDOW, sink_tokens=sink, window_tokens=W)
    Oo, LSE = O.attn_forward(q, k, v, pat, 0.4)
    for n in range(1, L + 1):
        o, lse = O.decode(q[:, n - 1], k, v, n, sink, W, 0.4, block_tokens=Bs)
        np.testing.assert_allclose(o, Oo[:, n - 1], rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(lse, LSE[:, n - 1], rtol=1e-12, atol=1e-13)
        aligned, held = O.decode_valid(n, sink, W, Bs), O.decode_valid(n, sink, W)
        assert (aligned <= held).all()                       # a subset of what the cache holds
        assert held.sum() - aligned.sum() == (0 if n <= sink + W else Bs - 1 - (n - 1) % Bs)
        # written out with loops
        i = n - 1
        assert [j for j in range(n) if j < sink or i // Bs - j // Bs < W // Bs] == list(np.nonzero(aligned)[0])
    # the chunk function is T such steps
    n0, T = 23, 9
    oc, lc = O.chunk_prefill(q[:, n0:n0 + T], k, v, n0, sink, W, 0.4, block_tokens=Bs)
    np.testing.assert_allclose(oc, Oo[:, n0:n0 + T], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(lc, LSE[:, n0:n0 + T], rtol=1e-12, atol=1e-13)


def test_ring_replay_holds_exactly_the_surviving_tokens():
    sink, W = 3, 5
    for n0, T in ((0, 1), (0, 4), (2, 3), (0, 8), (5, 20), (7, 1), (0, 31)):
        cache = np.full((sink + W, 1), -1.0)
        # history before: tokens 0..n0-1 appended one by one
        O.ring_append_replay(cache, np.arange(n0, dtype=float)[:, None], 0, sink, W)
        O.ring_append_replay(cache, np.arange(n0, n0 + T, dtype=float)[:, None], n0, sink, W)
        n = n0 + T
        held = sorted(int(x) for x in cache[:, 0] if x >= 0)
        assert held == list(np.nonzero(O.decode_valid(n, sink, W))[0])
        # every surviving token sits where the slot rule says, each slot holds one token
        for j in held:
            assert cache[O.ring_slot(j, sink, W), 0] == j
        # sink slots never move; the ring holds the last W non-sink tokens
        assert all(cache[j, 0] == j for j in range(min(n, sink)))


# --------------------------------------------------------- token-exact window (window_exact)

def _exact(L=512, block=64, sink=64, window=128):
    return O.Pattern(L, block, O.MODE_SINK_WINDOW, sink_tokens=sink, window_tokens=window, window_exact=True)


def test_exact_window_predicate_bruteforce():
    """Plain loops over token pairs: j <= i and (j in a sink block or i - j < W)."""
    p = _exact(L=320, block=64, sink=64, window=128)
    m = O.token_mask(p)
    for i in range(p.L):
        for j in range(p.L):
            want = j <= i and (j < p.sink_tokens or i - j < p.window_tokens)
            assert bool(m[i, j]) == want, (i, j)


@pytest.mark.parametrize("block,sink,window", [(64, 64, 128), (128, 128, 256), (64, 0, 64), (64, 128, 64)])
def test_exact_window_row_counts_and_block_counts(block, sink, window):
    """Late rows see exactly sink + W keys; the exact window reaches one block further back than
    the block-granular one, so nnz follows the closed form with nw + 1 window blocks."""
    L = 16 * block
    p = _exact(L, block, sink, window)
    m = O.token_mask(p)
    for i in range(sink + window, L):
        assert m[i].sum() == sink + window
    nB, ns, nw1 = L // block, sink // block, window // block + 1
    nnz = sum(min(qb + 1, nw1) + min(ns, max(qb + 1 - nw1, 0)) for qb in range(nB))
    row_ptr, col_idx, col_ptr, row_idx = O.block_lists(p)
    assert row_ptr[-1] == nnz == len(col_idx) == len(row_idx)
    # it contains the block-granular pattern with the same sizes, and nothing older than W tokens
    coarse = O.token_mask(O.Pattern(L, block, O.MODE_SINK_WINDOW, sink_tokens=sink, window_tokens=window))
    i, j = np.nonzero(m & ~coarse)
    assert ((i - j) < window).all() and ((i // block) - (j // block) == window // block).all()
    i, j = np.nonzero(coarse & ~m)
    assert ((i - j) >= window).all()


def test_exact_window_wide_is_full_causal():
    p = _exact(L=256, block=64, sink=0, window=256)
    assert np.array_equal(O.token_mask(p), np.tril(np.ones((256, 256), dtype=bool)))


def test_exact_window_last_row_equals_decode():
    """The decode oracle (written separately: survivors of a linear history) attends exactly the keys
    the exact-window mask gives the last query row, so the two must agree on that row."""
    rng = np.random.default_rng(5)
    L, D, sink, window = 448, 32, 64, 128
    q = rng.standard_normal((2, L, D))
    k = rng.standard_normal((1, L, D))
    v = rng.standard_normal((1, L, D))
    p = _exact(L, 64, sink, window)
    scale = 1.0 / math.sqrt(D)
    o, lse = O.attn_forward(q, k, v, p, scale)
    for n in (L, L - 37, sink + window + 1):
        od, ld = O.decode(q[:, n - 1], k, v, n, sink, window, scale)
        np.testing.assert_allclose(od, o[:, n - 1], rtol=0, atol=1e-12)
        np.testing.assert_allclose(ld, lse[:, n - 1], rtol=0, atol=1e-12)


def test_exact_window_backward_finite_differences():
    rng = np.random.default_rng(6)
    L, D = 192, 8
    p = _exact(L, 64, 64, 64)
    q, k, v, do = (rng.standard_normal((1, L, D)) for _ in range(4))
    scale = 0.3
    dQ, dK, dV, _, _ = O.attn_backward(q, k, v, do, p, scale)
    f = lambda q_, k_, v_: float((O.attn_forward(q_, k_, v_, p, scale)[0] * do).sum())
    eps = 1e-6
    for arr, grad in ((q, dQ), (k, dK), (v, dV)):
        for idx in [(0, 3, 1), (0, 100, 5), (0, 191, 7), (0, 64, 0)]:
            a0 = arr[idx]
            arr[idx] = a0 + eps; fp = f(q, k, v)
            arr[idx] = a0 - eps; fm = f(q, k, v)
            arr[idx] = a0
            assert abs((fp - fm) / (2 * eps) - grad[idx]) < 1e-6


# --------------------------------------------------------------------- chunked prefill

def test_chunk_prefill_equals_exact_window_rows():
    """Serving a chunk against the cache gives the rows the token-exact sink + window mask gives those
    positions in one pass over the whole sequence (the mask-based forward shares no code with the
    decode-based chunk function): before the ring is full, exactly at the fill point, and long after."""
    rng = np.random.default_rng(11)
    L, D, sink, window = 640, 16, 64, 128
    q = rng.standard_normal((4, L, D))
    k = rng.standard_normal((2, L, D))
    v = rng.standard_normal((2, L, D))
    scale = 1.0 / math.sqrt(D)
    o, lse = O.attn_forward(q, k, v, _exact(L, 64, sink, window), scale)
    for n0, T in ((0, 64), (64, 128), (128, 64), (192, 128), (320, 192), (576, 64), (37, 5)):
        oc, lc = O.chunk_prefill(q[:, n0:n0 + T], k, v, n0, sink, window, scale)
        np.testing.assert_allclose(oc, o[:, n0:n0 + T], rtol=0, atol=1e-12)
        np.testing.assert_allclose(lc, lse[:, n0:n0 + T], rtol=0, atol=1e-12)


def test_chunk_prefill_bruteforce_tiny():
    """Written out with loops: token i sees the sink tokens and the last `window` tokens up to itself."""
    rng = np.random.default_rng(12)
    Hq, Hkv, D, sink, window, n0, T = 2, 1, 4, 2, 3, 7, 4
    q = rng.standard_normal((Hq, T, D))
    k = rng.standard_normal((Hkv, n0 + T, D))
    v = rng.standard_normal((Hkv, n0 + T, D))
    o, lse = O.chunk_prefill(q, k, v, n0, sink, window, 0.7)
    for h in range(Hq):
        for t in range(T):
            i = n0 + t
            js = [j for j in range(i + 1) if j < sink or i - j < window]
            w = [math.exp(0.7 * float(np.dot(q[h, t], k[0, j]))) for j in js]
            z = sum(w)
            ref = sum(wj / z * v[0, j] for wj, j in zip(w, js))
            np.testing.assert_allclose(o[h, t], ref, rtol=1e-12, atol=1e-12)
            assert abs(lse[h, t] - math.log(z)) < 1e-12


def test_chunk_prefill_ignores_evicted_tokens():
    """Tokens that fell out of the ring before the chunk arrived cannot influence it."""
    rng = np.random.default_rng(13)
    Hq, Hkv, D, sink, window, n0, T = 2, 2, 8, 4, 16, 40, 8
    q = rng.standard_normal((Hq, T, D))
    k = rng.standard_normal((Hkv, n0 + T, D))
    v = rng.standard_normal((Hkv, n0 + T, D))
    o, lse = O.chunk_prefill(q, k, v, n0, sink, window, 0.3)
    k2, v2 = k.copy(), v.copy()
    gone = slice(sink, n0 - window + 1)      # evicted before the chunk's first token attends
    k2[:, gone] = 99.0
    v2[:, gone] = -99.0
    o2, lse2 = O.chunk_prefill(q, k2, v2, n0, sink, window, 0.3)
    assert np.array_equal(o, o2) and np.array_equal(lse, lse2)
    k2[:, n0 - window + 1] += 1.0            # the oldest token the first chunk token still sees
    o3, _ = O.chunk_prefill(q, k2, v2, n0, sink, window, 0.3)
    assert not np.array_equal(o3[:, 0], o[:, 0]) and np.array_equal(o3[:, 1:], o[:, 1:])


# --------------------------------------------------------------------- packed documents

def _doc_bounds(L, cuts):
    ds = np.zeros(L, dtype=np.int32)
    for a, b in zip(cuts[:-1], cuts[1:]):
        ds[a:b] = a
    return ds


def test_documents_full_causal_equals_torch_per_document():
    """Full causal attention with the document option is plain causal attention run on every document by
    itself: forward and all three gradients against torch (fp64 SDPA / autograd), document by document."""
    rng = np.random.default_rng(21)
    L, D, cuts = 320, 16, [0, 37, 38, 130, 256, 320]      # one-token document, block-straddling cuts
    q = rng.standard_normal((2, L, D)); k = rng.standard_normal((1, L, D)); v = rng.standard_normal((1, L, D))
    do = rng.standard_normal((2, L, D))
    scale = 0.31
    p = O.Pattern(L, 64, O.MODE_FULL_CAUSAL, doc_start=_doc_bounds(L, cuts))
    dQ, dK, dV, Oo, LSE = O.attn_backward(q, k, v, do, p, scale)
    for a, b in zip(cuts[:-1], cuts[1:]):
        tq = torch.tensor(q[:, a:b], requires_grad=True); tk = torch.tensor(k[:, a:b], requires_grad=True)
        tv = torch.tensor(v[:, a:b], requires_grad=True)
        s = scale * tq @ tk.expand(2, -1, -1).transpose(1, 2)
        s = s.masked_fill(~torch.tril(torch.ones(b - a, b - a, dtype=torch.bool)), float("-inf"))
        out = torch.softmax(s, dim=-1) @ tv.expand(2, -1, -1)
        (out * torch.tensor(do[:, a:b])).sum().backward()
        np.testing.assert_allclose(Oo[:, a:b], out.detach().numpy(), rtol=0, atol=1e-12)
        np.testing.assert_allclose(LSE[:, a:b], torch.logsumexp(s, dim=-1).detach().numpy(), rtol=0, atol=1e-12)
        np.testing.assert_allclose(dQ[:, a:b], tq.grad.numpy(), rtol=0, atol=1e-11)
        np.testing.assert_allclose(dK[:, a:b], tk.grad.numpy(), rtol=0, atol=1e-11)
        np.testing.assert_allclose(dV[:, a:b], tv.grad.numpy(), rtol=0, atol=1e-11)


def test_documents_with_window_are_the_pattern_and_the_document_mask():
    """With a sparse pattern the option only removes pairs: allowed = pattern AND same document, written out
    with loops; and an exact window without sink is translation invariant, so each document by itself
    (positions restarting at 0) gives the same rows."""
    L, cuts = 256, [0, 100, 101, 256]
    ds = _doc_bounds(L, cuts)
    for base in (O.Pattern(L, 64, O.MODE_SINK_WINDOW, sink_tokens=64, window_tokens=128),
                 O.Pattern(L, 64, O.MODE_STRIDED_LOCAL, stride_blocks=2, local_blocks=1),
                 O.Pattern(L, 64, O.MODE_SINK_WINDOW, sink_tokens=0, window_tokens=64, window_exact=True)):
        withd = O.Pattern(base.L, base.block, base.mode, base.sink_tokens, base.window_tokens, base.stride_blocks,
                          base.local_blocks, base.window_exact, doc_start=ds)
        m0, m1 = O.token_mask(base), O.token_mask(withd)
        for i in range(L):
            for j in range(L):
                assert m1[i, j] == (m0[i, j] and j >= ds[i])
    rng = np.random.default_rng(22)
    D = 8
    q = rng.standard_normal((1, L, D)); k = rng.standard_normal((1, L, D)); v = rng.standard_normal((1, L, D))
    o, lse = O.attn_forward(q, k, v, withd, 0.4)[:2]
    for a, b in zip(cuts[:-1], cuts[1:]):
        n = b - a
        npad = (n + 63) // 64 * 64          # the per-document run needs a multiple of the block
        pad = lambda x: np.concatenate([x[:, a:b], np.zeros((1, npad - n, D))], axis=1)
        od, ld = O.attn_forward(pad(q), pad(k), pad(v), O.Pattern(npad, 64, O.MODE_SINK_WINDOW, 0, 64, window_exact=True), 0.4)[:2]
        np.testing.assert_allclose(o[:, a:b], od[:, :n], rtol=0, atol=1e-12)
        np.testing.assert_allclose(lse[:, a:b], ld[:, :n], rtol=0, atol=1e-12)


# --------------------------------------------------------------------- L not a multiple of the block

def test_partial_last_block_is_a_prefix_of_the_padded_problem():
    """Causal attention never looks ahead, so the first L rows of a longer, block-aligned problem are the
    answer for L (forward; and gradients when dO is zero past L); block lists are those of the aligned
    problem cut to ceil(L / block) blocks; full causal with a ragged L against torch."""
    rng = np.random.default_rng(31)
    L, Lp, D = 200, 256, 8
    q = rng.standard_normal((2, Lp, D)); k = rng.standard_normal((1, Lp, D)); v = rng.standard_normal((1, Lp, D))
    do = rng.standard_normal((2, Lp, D)); do[:, L:] = 0.0
    for mk in (lambda n: O.Pattern(n, 64, O.MODE_SINK_WINDOW, sink_tokens=64, window_tokens=64),
               lambda n: O.Pattern(n, 64, O.MODE_STRIDED_LOCAL, stride_blocks=2, local_blocks=1),
               lambda n: O.Pattern(n, 64, O.MODE_SINK_WINDOW, sink_tokens=0, window_tokens=64, window_exact=True),
               lambda n: O.Pattern(n, 64, O.MODE_FULL_CAUSAL)):
        dQ, dK, dV, Oo, LSE = O.attn_backward(q[:, :L], k[:, :L], v[:, :L], do[:, :L], mk(L), 0.5)
        dQp, dKp, dVp, Op, LSEp = O.attn_backward(q, k, v, do, mk(Lp), 0.5)
        for a, b in ((Oo, Op), (LSE, LSEp), (dQ, dQp), (dK, dKp), (dV, dVp)):
            np.testing.assert_allclose(a, b[:, :L], rtol=0, atol=1e-12)
        rp, ci, cp, ri = O.block_lists(mk(L))
        rpp, cip, cpp, rip = O.block_lists(mk(Lp))
        nB = 4
        assert len(rp) == nB + 1 and np.array_equal(rp, rpp[:nB + 1]) and np.array_equal(ci, cip[:rp[-1]])
        assert O.count_pairs(mk(L)) == int(O.token_mask(mk(Lp))[:L, :L].sum())
    tq = torch.tensor(q[:, :L]); tk = torch.tensor(k[:, :L]).expand(2, -1, -1); tv = torch.tensor(v[:, :L]).expand(2, -1, -1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=0.5)
    np.testing.assert_allclose(Oo, ref.numpy(), rtol=0, atol=1e-12)
