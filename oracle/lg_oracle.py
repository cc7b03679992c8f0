"""CPU fp64 oracle for LongGen's efficient attention layers.  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
module.  It shares no code with the CUDA library and imports nothing from it.

What it computes is masked softmax attention written out from its definition
(paper Section 3.2: the sparse kernel skips positions whose mask value is zero, so
the result IS masked attention, only cheaper), under the two static block
patterns of Section 3.1 / 4.1:

  * attention sink + sliding window: the first blocks plus the most recent blocks,
  * blockwise strided: every `stride`-th block plus a few local blocks,

and plain causal attention for the full-attention layers.  Every function
materialises the explicit token-level boolean mask; nothing here is blocked,
fused or reordered beyond "work on a slab of rows at a time", which changes no
value.  All arithmetic is float64.

Readings of points on which the paper is silent:
  - the window is block-granular and counts the query's own block
    (Section 4.1 keeps one sink block and the 32 latest blocks); with
    window_exact it is the token-exact window of the rolling-buffer cache
    (Section 3.2), i - j < window_tokens, which is what the decode attends;
  - the strided comb is absolute: KV block kb is retained iff kb % stride == 0;
  - LSE is the natural log of the sum of exp of the *scaled* scores;
  - the backward formulas are the derivatives of the definition (the paper
    inherits them from FlashAttention and prints none);
  - documents packed into one sample: the paper masks nothing across them; the
    optional doc_start array adds "no key of an earlier document" to the pattern.

Pins (tests/test_oracle_*.py): brute-force per-row softmax, torch's dense causal
attention and autograd in fp64, central finite differences, closed-form block
counts, the paper's KV-cache arithmetic; the chunk-against-cache function (T decode
steps) against the rows of the mask-based forward and against explicit loops; the
document option against torch attention run on each document separately.  Trained-model quality: parity unpinned
and out of scope.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import Optional, Tuple

import numpy as np

MODE_FULL_CAUSAL = 0
MODE_SINK_WINDOW = 1
MODE_STRIDED_LOCAL = 2


@dataclass(frozen=True)
class Pattern:
    """Static sparse pattern (Section 3.1).  Sink and window token counts are multiples of `block`;
    L need not be (the last block is then partial)."""
    L: int
    block: int
    mode: int
    sink_tokens: int = 0
    window_tokens: int = 0
    stride_blocks: int = 0
    local_blocks: int = 0
    window_exact: bool = False   # sink + window only: the window edge is token-exact (i - j < window_tokens)
    # packed documents (Section 4.1 packs documents, each opened by <bos>, into one training sample):
    # doc_start[i] = position of the first token of the document that token i belongs to; when given,
    # a query sees no key of an earlier document.  The paper describes no such masking; it is an
    # option on top of the static pattern, which itself stays in absolute positions.
    doc_start: Optional[np.ndarray] = None

    @staticmethod
    def of(cfg) -> "Pattern":
        return Pattern(cfg.L, cfg.block, cfg.mode, cfg.sink_tokens, cfg.window_tokens,
                       cfg.stride_blocks, cfg.local_blocks, bool(getattr(cfg, "window_exact", False)))


# --------------------------------------------------------------------------- masks

def allowed(p: Pattern, i, j):
    """Token-level predicate: may query i attend key j?  i, j broadcastable int arrays.

    Section 3.1 (patterns), Section 4.1 (block = 64 tokens, 1 sink block + 32 recent
    blocks; stride in blocks)."""
    i = np.asarray(i, dtype=np.int32)
    j = np.asarray(j, dtype=np.int32)
    causal = j <= i
    if p.doc_start is not None:
        causal = causal & (j >= np.asarray(p.doc_start, dtype=np.int32)[i])
    if p.mode == MODE_FULL_CAUSAL:
        return causal
    qb = i // p.block
    kb = j // p.block
    if p.mode == MODE_SINK_WINDOW:
        ns = p.sink_tokens // p.block
        nw = p.window_tokens // p.block
        if p.window_exact:
            # the Mistral-style window the paper cites for serving (Section 3.2): the last
            # window_tokens tokens, the query's own included; sink blocks as before
            return causal & ((kb < ns) | (i - j < p.window_tokens))
        return causal & ((kb < ns) | (qb - kb < nw))
    if p.mode == MODE_STRIDED_LOCAL:
        return causal & ((qb - kb < p.local_blocks) | (kb % p.stride_blocks == 0))
    raise ValueError("unknown mode")


def token_mask(p: Pattern, r0: int = 0, r1: Optional[int] = None) -> np.ndarray:
    """Explicit boolean mask for query rows [r0, r1) against all L keys."""
    r1 = p.L if r1 is None else r1
    return allowed(p, np.arange(r0, r1)[:, None], np.arange(p.L)[None, :])


def block_lists(p: Pattern):
    """CSR and CSC lists of active blocks, derived from the explicit token mask.

    Block (qb, kb) is active iff some allowed (i, j) lies inside it (Section 3.2: the
    mask is kept in compressed-sparse-row form, one list shared by all heads).
    Returns int32 arrays (row_ptr[nB+1], col_idx[nnz], col_ptr[nB+1], row_idx[nnz]);
    rows ascending in kb, columns ascending in qb."""
    Bs = p.block
    nB = -(-p.L // Bs)                 # the last block may be partial
    active = np.zeros((nB, nB), dtype=bool)

    def one_block_row(qb):
        m = token_mask(p, qb * Bs, min(p.L, (qb + 1) * Bs))        # [<= Bs, L]
        full = np.zeros((m.shape[0], nB * Bs), dtype=bool)
        full[:, :p.L] = m
        active[qb] = full.reshape(m.shape[0], nB, Bs).any(axis=(0, 2))

    # a plain parallel-for over block rows (numpy releases the GIL inside its loops)
    with ThreadPoolExecutor(max_workers=os.cpu_count() or 1) as pool:
        list(pool.map(one_block_row, range(nB)))
    row_ptr = np.zeros(nB + 1, dtype=np.int32)
    col_ptr = np.zeros(nB + 1, dtype=np.int32)
    row_ptr[1:] = np.cumsum(active.sum(axis=1))
    col_ptr[1:] = np.cumsum(active.sum(axis=0))
    qb_i, kb_i = np.nonzero(active)            # row-major order: ascending qb, then kb
    col_idx = kb_i.astype(np.int32)
    kb_t, qb_t = np.nonzero(active.T)          # ascending kb, then qb
    row_idx = qb_t.astype(np.int32)
    return row_ptr, col_idx, col_ptr, row_idx


def count_pairs(p: Pattern) -> int:
    """Number of allowed (i, j) pairs for one head, counted from the explicit mask."""
    Bs = p.block
    with ThreadPoolExecutor(max_workers=os.cpu_count() or 1) as pool:
        return sum(pool.map(lambda r0: int(token_mask(p, r0, min(p.L, r0 + Bs)).sum()), range(0, p.L, Bs)))


# ------------------------------------------------------------------------- forward

def _softmax_rows(S: np.ndarray, M: np.ndarray):
    """Masked softmax of score rows S under boolean mask M -> (P, LSE)."""
    Sm = np.where(M, S, -np.inf)
    mx = Sm.max(axis=1, keepdims=True)
    E = np.where(M, np.exp(Sm - mx), 0.0)
    Z = E.sum(axis=1, keepdims=True)
    return E / Z, (mx + np.log(Z))[:, 0]


def attn_forward(q, k, v, p: Pattern, scale: float, rows_per_slab: Optional[int] = None):
    """O = softmax(scale*Q K^T + mask) V and LSE_i = log sum_j exp(scale*q_i.k_j).

    q [Hq, L, D], k, v [Hkv, L, D] float64; query head h uses kv head h // (Hq/Hkv)
    (grouped-query attention, Llama-2 70B).  Returns O [Hq, L, D], LSE [Hq, L].
    rows_per_slab=None materialises the full L x L mask at once; otherwise rows are
    taken a slab at a time and keys no row of the slab may see are dropped."""
    Hq, L, D = q.shape
    G = Hq // k.shape[0]
    O = np.zeros_like(q)
    LSE = np.zeros((Hq, L))
    slab = L if rows_per_slab is None else rows_per_slab
    for r0 in range(0, L, slab):
        r1 = min(L, r0 + slab)
        M = token_mask(p, r0, r1)
        cols = np.nonzero(M.any(axis=0))[0]
        Mc = M[:, cols]
        for h in range(Hq):
            S = scale * (q[h, r0:r1] @ k[h // G, cols].T)
            P, lse = _softmax_rows(S, Mc)
            O[h, r0:r1] = P @ v[h // G, cols]
            LSE[h, r0:r1] = lse
    return O, LSE


def attn_backward(q, k, v, do, p: Pattern, scale: float, rows_per_slab: Optional[int] = None):
    """Gradients of sum(O * dO) w.r.t. Q, K, V from the definition:

      P = exp(S - LSE) on allowed pairs, 0 elsewhere;  dV_j = sum_i P_ij dO_i;
      dP_ij = dO_i . v_j;  delta_i = sum_j P_ij dP_ij;  dS = P * (dP - delta);
      dQ_i = scale * sum_j dS_ij k_j;  dK_j = scale * sum_i dS_ij q_i;
      dK, dV of a kv head sum over the query heads of its group.

    Returns (dQ [Hq,L,D], dK [Hkv,L,D], dV [Hkv,L,D], O, LSE)."""
    Hq, L, D = q.shape
    G = Hq // k.shape[0]
    dQ = np.zeros_like(q)
    dK = np.zeros_like(k)
    dV = np.zeros_like(v)
    O = np.zeros_like(q)
    LSE = np.zeros((Hq, L))
    slab = L if rows_per_slab is None else rows_per_slab
    for r0 in range(0, L, slab):
        r1 = min(L, r0 + slab)
        M = token_mask(p, r0, r1)
        cols = np.nonzero(M.any(axis=0))[0]
        Mc = M[:, cols]
        for h in range(Hq):
            g = h // G
            kc, vc = k[g, cols], v[g, cols]
            S = scale * (q[h, r0:r1] @ kc.T)
            P, lse = _softmax_rows(S, Mc)
            O[h, r0:r1] = P @ vc
            LSE[h, r0:r1] = lse
            dOh = do[h, r0:r1]
            dP = dOh @ vc.T
            delta = (P * dP).sum(axis=1, keepdims=True)
            dS = P * (dP - delta)
            dQ[h, r0:r1] = scale * (dS @ kc)
            dK[g, cols] += scale * (dS.T @ q[h, r0:r1])
            dV[g, cols] += P.T @ dOh
    return dQ, dK, dV, O, LSE


# ----------------------------------------------------- subsets of the outputs (large L)

def attn_rows(q, k, v, do, p: Pattern, scale: float, r0: int, r1: int):
    """The definition restricted to query rows [r0, r1): O, LSE and (if `do` is given) dQ
    of those rows for every head.  Row i of O, LSE and dQ depends on row i of Q and dO only,
    so this is attn_forward / attn_backward evaluated on one slab.
    Returns (O [Hq, r1-r0, D], LSE [Hq, r1-r0], dQ or None)."""
    Hq, L, D = q.shape
    G = Hq // k.shape[0]
    M = token_mask(p, r0, r1)
    cols = np.nonzero(M.any(axis=0))[0]
    Mc = M[:, cols]
    O = np.zeros((Hq, r1 - r0, D))
    LSE = np.zeros((Hq, r1 - r0))
    dQ = None if do is None else np.zeros((Hq, r1 - r0, D))
    for h in range(Hq):
        kc, vc = k[h // G, cols], v[h // G, cols]
        S = scale * (q[h, r0:r1] @ kc.T)
        P, lse = _softmax_rows(S, Mc)
        O[h] = P @ vc
        LSE[h] = lse
        if do is not None:
            dP = do[h, r0:r1] @ vc.T
            delta = (P * dP).sum(axis=1, keepdims=True)
            dQ[h] = scale * ((P * (dP - delta)) @ kc)
    return O, LSE, dQ


def attn_keys_grad(q, k, v, do, p: Pattern, scale: float, j0: int, j1: int):
    """The definition restricted to keys [j0, j1): dK and dV of those keys for every kv
    head.  Every query row that may see one of these keys is found from the explicit mask
    and taken a block of rows at a time; its softmax runs over ALL keys it may see.
    Returns (dK [Hkv, j1-j0, D], dV [Hkv, j1-j0, D])."""
    Hq, L, D = q.shape
    Hkv = k.shape[0]
    G = Hq // Hkv
    dK = np.zeros((Hkv, j1 - j0, D))
    dV = np.zeros((Hkv, j1 - j0, D))
    for r0 in range(0, L, p.block):
        r1 = min(L, r0 + p.block)          # the last block may be partial
        # does any row of this slab see one of the wanted keys?  (the explicit mask, on those columns only,
        # before the slab's whole mask is materialised)
        if not allowed(p, np.arange(r0, r1)[:, None], np.arange(j0, j1)[None, :]).any():
            continue
        M = token_mask(p, r0, r1)
        cols = np.nonzero(M.any(axis=0))[0]
        Mc = M[:, cols]
        sel = (cols >= j0) & (cols < j1)        # which of the slab's keys are the wanted ones
        for h in range(Hq):
            g = h // G
            kc, vc = k[g, cols], v[g, cols]
            S = scale * (q[h, r0:r1] @ kc.T)
            P, _ = _softmax_rows(S, Mc)
            dOh = do[h, r0:r1]
            dP = dOh @ vc.T
            delta = (P * dP).sum(axis=1, keepdims=True)
            dS = P * (dP - delta)
            dK[g, cols[sel] - j0] += scale * (dS[:, sel].T @ q[h, r0:r1])
            dV[g, cols[sel] - j0] += P[:, sel].T @ dOh
    return dK, dV


# -------------------------------------------------------------------------- decode

def decode_valid(n: int, sink: int, window: int, block_tokens: int = 0) -> np.ndarray:
    """Which of the first n tokens the query token n - 1 attends to in serving.

    block_tokens == 0: every token a sink + rolling-window cache still holds after n appends
    (Section 3.2: rolling buffer for the window, sink kept beside it): token j survives iff
    j < sink or it is among the last `window` tokens.
    block_tokens == Bs > 0: the block-granular window the sparse layers are trained with
    (Section 4.1 counts the local context in blocks, the query's own block included): token j
    is attended iff j < sink or floor((n-1)/Bs) - floor(j/Bs) < window/Bs.  These are tokens
    the cache holds (a subset: up to Bs - 1 of the oldest window tokens are left out)."""
    j = np.arange(n)
    if block_tokens:
        return (j < sink) | ((n - 1) // block_tokens - j // block_tokens < window // block_tokens)
    return (j < sink) | (n - 1 - j < window)


def decode(qv, k_lin, v_lin, n: int, sink: int, window: int, scale: float, block_tokens: int = 0):
    """One query token per head attends to the surviving tokens of a linear history
    (block_tokens: see decode_valid).

    qv [Hq, D]; k_lin, v_lin [Hkv, >=n, D] hold token j at index j (the oracle never
    sees the ring layout).  Returns o [Hq, D], lse [Hq]; n == 0 gives o = 0, lse = -inf."""
    Hq, D = qv.shape
    G = Hq // k_lin.shape[0]
    o = np.zeros((Hq, D))
    lse = np.full(Hq, -np.inf)
    if n == 0:
        return o, lse
    keep = np.nonzero(decode_valid(n, sink, window, block_tokens))[0]
    for h in range(Hq):
        s = scale * (k_lin[h // G, keep] @ qv[h])
        mx = s.max()
        e = np.exp(s - mx)
        z = e.sum()
        o[h] = (e / z) @ v_lin[h // G, keep]
        lse[h] = mx + np.log(z)
    return o, lse


def chunk_prefill(q_chunk, k_lin, v_lin, n_before: int, sink: int, window: int, scale: float, block_tokens: int = 0):
    """A chunk of T new tokens served against a sink + rolling-window cache (Section 3.2: in
    serving the sparse layers keep only the sink and the last `window` tokens).  By definition
    the result is what T successive decode steps give: token n_before + t is appended and then
    attends to whatever the cache holds at that moment.

    q_chunk [Hq, T, D]; k_lin, v_lin [Hkv, >= n_before + T, D] hold token j at index j (the
    oracle never sees the ring layout).  Returns o [Hq, T, D], lse [Hq, T]."""
    Hq, T, D = q_chunk.shape
    o = np.zeros((Hq, T, D))
    lse = np.full((Hq, T), -np.inf)
    for t in range(T):
        o[:, t], lse[:, t] = decode(q_chunk[:, t], k_lin, v_lin, n_before + t + 1, sink, window, scale, block_tokens)
    return o, lse


def ring_slot(j: int, sink: int, window: int) -> int:
    """Cache slot of token j: sink tokens stay put, later ones roll (Mistral's
    i mod W, offset past the sink)."""
    return j if j < sink else sink + (j - sink) % window


def ring_append_replay(cache: np.ndarray, new: np.ndarray, n_before: int, sink: int, window: int):
    """Write tokens n_before, n_before+1, ... one at a time into `cache`
    [sink+window, ...] in place; later writes overwrite earlier ones."""
    for t in range(new.shape[0]):
        cache[ring_slot(n_before + t, sink, window)] = new[t]
    return cache
