"""fp64 CPU oracle for Eigen Attention (rank-r attention) -- TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the GPU library must compute.
It is imported only by the tests, by the smoke check and by the benchmark's
CPU-baseline leg; the product path never routes through it.  It shares no code
with the CUDA sources and never sees a value produced by them.

Everything is numpy float64.  The result has a closed-form definition
(Eq. 7 of the paper), so the oracle is that definition written out: project,
score, ordinary three-pass softmax, weighted sum, lift.  No tiling, no
splitting of the key axis, no online softmax.

Notation follows the paper: d_h head dimension, r rank, U^K / U^V bases with
orthonormal columns (d_h x r), n cached length, per-head index i dropped where
one head is handled.

Parity pins (see tests): the functions here are pinned against an independent
library routine for softmax attention applied to the d_h-wide low-rank inputs
Q', K', V' of Eq. 6, brute-force Python loops on tiny inputs, closed-form
special cases, and the numbers the paper prints for cache sizes.  The ALiBi
bias is pinned by the same library routine given the bias as an additive
mask, by the geometric-series closed form for a zero query, and by loops.
Grouped-query decode is pinned by the library routine's own grouped mode and
by ordinary decode with the K/V heads repeated.
The RoPE variant (Section 4.3) is pinned by library attention on keys and
queries rotated with complex arithmetic, by its relative-position invariance,
by the zero-angle special case and by loops; its prompt form (prefill_head_rope)
by causal library attention on the same rotated tensors and by the generation
form row by row.
decode_quant is ordinary decode over the rows returned by kv_quant.quantized_view, which has its own pins.
paged_gather / paged_scatter (address arithmetic of a paged cache) are pinned by the identity "paged == contiguous"
for random page tables, by the identity table, and by a hand-written two-page example.
Nothing in this file is "parity unpinned".
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# Building blocks
# --------------------------------------------------------------------------

def softmax_rows(S: np.ndarray) -> np.ndarray:
    """Row-wise Softmax of Eq. 2/3: max, exp-sum, normalise (three passes)."""
    S = np.asarray(S, dtype=F64)
    m = S.max(axis=-1, keepdims=True)
    E = np.exp(S - m)
    return E / E.sum(axis=-1, keepdims=True)


def to_rank_space(X: np.ndarray, U: np.ndarray) -> np.ndarray:
    """Coordinates of the rows of X in the basis U: X U  (the r-wide factor of Eq. 6;
    the merged weights W U of Eq. 8 produce exactly these rows)."""
    return np.asarray(X, dtype=F64) @ np.asarray(U, dtype=F64)


def lift(Y: np.ndarray, U: np.ndarray) -> np.ndarray:
    """Back to d_h dimensions: Y U^T  (the trailing (U^V)^T of Eq. 7)."""
    return np.asarray(Y, dtype=F64) @ np.asarray(U, dtype=F64).T


# --------------------------------------------------------------------------
# One head, stateless: the definition
# --------------------------------------------------------------------------

def alibi_bias(slope: float, pos: int, n: int) -> np.ndarray:
    """Linear position bias of the MPT models (Section 5.1 names ALiBi as their position scheme; the
    paper prints no formula, this is the published one): the score of the query at position `pos`
    against key j gets -slope * (pos - j), j = 0..n-1.  The head's slope is an input."""
    return -float(slope) * (float(pos) - np.arange(n, dtype=F64))


def decode_head(q: np.ndarray, K: np.ndarray, V: np.ndarray,
                U_K: np.ndarray, U_V: np.ndarray, lowrank_out: bool = False,
                alibi_slope: float = 0.0) -> np.ndarray:
    """Generation-phase Eigen Attention for one head (Eq. 3 in the space of Eq. 7).

    q [d_h]; K, V [n, d_h] are the un-projected rows of the n cached tokens
    (the new token's row included: the cache is extended first, then attended,
    Section 2 "LLM Inference").  Returns [d_h] (or [r_V] with lowrank_out).
    The softmax scale is 1/sqrt(d_h) -- Eq. 7 keeps d_h although the vectors
    are r wide.  With alibi_slope the query (position n-1) adds alibi_bias to the scores.
    """
    d_h = U_K.shape[0]
    qp = to_rank_space(q, U_K)                    # [r_K]
    Kp = to_rank_space(K, U_K)                    # [n, r_K]
    Vp = to_rank_space(V, U_V)                    # [n, r_V]
    s = (Kp @ qp) / math.sqrt(d_h)                # [n]
    if alibi_slope:
        s = s + alibi_bias(alibi_slope, Kp.shape[0] - 1, Kp.shape[0])
    p = softmax_rows(s[None, :])[0]
    o = p @ Vp                                    # [r_V]
    return o if lowrank_out else lift(o, U_V)


def prefill_head(Q: np.ndarray, K: np.ndarray, V: np.ndarray,
                 U_K: np.ndarray, U_V: np.ndarray, len0: int = 0,
                 lowrank_out: bool = False, alibi_slope: float = 0.0) -> np.ndarray:
    """Causal Eigen Attention for one head over a prompt.

    Q [T, d_h] are the T new queries; K, V [len0+T, d_h] are all rows cached
    after the call (len0 earlier rows followed by the T new ones).  Query t
    attends rows 0..len0+t inclusive (decoder-only models; masked entries are
    excluded from the softmax).  Returns [T, d_h] (or [T, r_V]).
    """
    d_h = U_K.shape[0]
    T = Q.shape[0]
    Qp = to_rank_space(Q, U_K)
    Kp = to_rank_space(K, U_K)
    Vp = to_rank_space(V, U_V)
    O = np.zeros((T, Vp.shape[1]), dtype=F64)
    for t in range(T):
        n_t = len0 + t + 1
        s = (Kp[:n_t] @ Qp[t]) / math.sqrt(d_h)
        if alibi_slope:
            s = s + alibi_bias(alibi_slope, n_t - 1, n_t)
        p = softmax_rows(s[None, :])[0]
        O[t] = p @ Vp[:n_t]
    return O if lowrank_out else lift(O, U_V)


# --------------------------------------------------------------------------
# Section 4.3: Eigen Attention for models with rotary position embedding
# --------------------------------------------------------------------------

def rope_rotate(x: np.ndarray, pos, base: float = 10000.0, interleaved: bool = False) -> np.ndarray:
    """x R for the row(s) x [..., d_h] at position(s) `pos` (Section 4.3, first equation): coordinate
    pair i is turned by the angle pos * base^(-2i/d_h).  Pairs are (i, i + d_h/2) as in the Llama models the
    paper evaluates, or (2i, 2i+1) with interleaved=True (the original RoPE layout).  Built as an explicit
    block rotation: y_a = x_a cos - x_b sin, y_b = x_a sin + x_b cos."""
    x = np.asarray(x, dtype=F64)
    d = x.shape[-1]
    half = d // 2
    pos = np.asarray(pos, dtype=F64)
    ang = pos[..., None] * (float(base) ** (-2.0 * np.arange(half, dtype=F64) / d))   # [..., half]
    c, s_ = np.cos(ang), np.sin(ang)
    if interleaved:
        a, b = x[..., 0::2], x[..., 1::2]
    else:
        a, b = x[..., :half], x[..., half:]
    ya, yb = a * c - b * s_, a * s_ + b * c
    y = np.empty_like(x)
    if interleaved:
        y[..., 0::2], y[..., 1::2] = ya, yb
    else:
        y[..., :half], y[..., half:] = ya, yb
    return y


def decode_head_rope(q: np.ndarray, Kp: np.ndarray, Vp: np.ndarray, U_K: np.ndarray, U_V: np.ndarray,
                     base: float = 10000.0, interleaved: bool = False, pos0: int = 0,
                     lowrank_out: bool = False) -> np.ndarray:
    """Generation-phase Eigen Attention with RoPE for one head (Section 4.3, second equation, Fig. 6b).

    The query stays full rank.  The cache holds the low-dimensional keys Kp [n, r_K] (= K U^K of the
    un-rotated keys); each is taken back to d_h dimensions through (U^K)^T, rotated by its own position, and
    dotted with the rotated query.  Row j sits at position pos0 + j, the query at the last row's position.
    The value side is Eq. 7 unchanged.  q [d_h]; Vp [n, r_V]."""
    d_h = U_K.shape[0]
    n = Kp.shape[0]
    K_back = lift(Kp, U_K)                                         # [n, d_h]
    K_pos = rope_rotate(K_back, pos0 + np.arange(n), base, interleaved)
    q_pos = rope_rotate(np.asarray(q, dtype=F64), pos0 + n - 1, base, interleaved)
    s = (K_pos @ q_pos) / math.sqrt(d_h)
    p = softmax_rows(s[None, :])[0]
    o = p @ np.asarray(Vp, dtype=F64)
    return o if lowrank_out else lift(o, U_V)


def prefill_head_rope(Q: np.ndarray, Kp: np.ndarray, Vp: np.ndarray, U_K: np.ndarray, U_V: np.ndarray,
                      base: float = 10000.0, interleaved: bool = False, len0: int = 0,
                      lowrank_out: bool = False) -> np.ndarray:
    """Causal prompt attention of the RoPE variant for one head (Section 4.3 applied to the prefill phase of
    Section 2): Q [T, d_h] are the T new full-rank queries, Kp [len0+T, r_K], Vp [len0+T, r_V] the
    low-dimensional rows cached after the call.  Row j of the cache sits at position j, query t at position
    len0 + t and sees rows 0..len0+t.  Every cached key is lifted through (U^K)^T and rotated by its position,
    every query is rotated by its own; the value side is Eq. 7 unchanged."""
    d_h = U_K.shape[0]
    Q = np.asarray(Q, dtype=F64)
    T, n = Q.shape[0], Kp.shape[0]
    assert n == len0 + T
    K_pos = rope_rotate(lift(Kp, U_K), np.arange(n), base, interleaved)        # [n, d_h]
    Q_pos = rope_rotate(Q, len0 + np.arange(T), base, interleaved)             # [T, d_h]
    Vp = np.asarray(Vp, dtype=F64)
    O = np.zeros((T, Vp.shape[1]), dtype=F64)
    for t in range(T):
        n_t = len0 + t + 1
        s = (K_pos[:n_t] @ Q_pos[t]) / math.sqrt(d_h)
        p = softmax_rows(s[None, :])[0]
        O[t] = p @ Vp[:n_t]
    return O if lowrank_out else lift(O, U_V)


# --------------------------------------------------------------------------
# One decoder layer with a rank-r KV cache (stateful, mirrors the library calls)
# --------------------------------------------------------------------------

class LayerOracle:
    """Rank-r KV cache of one layer plus the calls of the library, in fp64.

    U_K[h] is d_h x r_K[h], U_V[h] is d_h x r_V[h]  (per layer and head,
    Section 4.1).  `tracked` optionally restricts the state to a list of
    (b, h) units so that very large workloads can be checked on a subset.
    """

    def __init__(self, batch: int, n_heads: int, d_head: int,
                 U_K: Sequence[np.ndarray], U_V: Sequence[np.ndarray],
                 tracked: Optional[Sequence[Tuple[int, int]]] = None,
                 alibi_slopes: Optional[Sequence[float]] = None,
                 storage=None, rope: Optional[dict] = None):
        """`storage`, if given, maps an array of freshly projected rows to what the cache keeps of them
        (e.g. rounding to the 16-bit format of Section 2, p = 16); None keeps fp64."""
        assert len(U_K) == n_heads and len(U_V) == n_heads
        self.storage = storage
        self.rope = rope          # None, or {"base": float, "interleaved": bool}: decode() follows Section 4.3
        self.alibi = [float(x) for x in alibi_slopes] if alibi_slopes is not None else [0.0] * n_heads
        assert len(self.alibi) == n_heads
        self.B, self.H, self.d_h = batch, n_heads, d_head
        self.U_K = [np.asarray(u, dtype=F64) for u in U_K]
        self.U_V = [np.asarray(u, dtype=F64) for u in U_V]
        for u in self.U_K + self.U_V:
            assert u.shape[0] == d_head
        self.units = list(tracked) if tracked is not None else [
            (b, h) for b in range(batch) for h in range(n_heads)]
        self.Kp = {u: np.zeros((0, self.U_K[u[1]].shape[1]), dtype=F64) for u in self.units}
        self.Vp = {u: np.zeros((0, self.U_V[u[1]].shape[1]), dtype=F64) for u in self.units}
        self.len = 0
        # counters for the closed forms of Table 1
        self.cache_elements = 0       # stored numbers, all tracked units
        self.projection_macs = 0      # run-time U multiplications
        self.attention_macs = 0       # q'K'^T and pV' of the last decode call

    # -- Section 2 "LLM Inference": K <- Concat(K, k), V <- Concat(V, v), in rank space (Eq. 6/8)
    def append_kv(self, k: np.ndarray, v: np.ndarray) -> None:
        """k, v: [B, T, H, d_h].  Projects each new row and extends the cache."""
        k = np.asarray(k, dtype=F64)
        v = np.asarray(v, dtype=F64)
        T = k.shape[1]
        for (b, h) in self.units:
            kp = to_rank_space(k[b, :, h, :], self.U_K[h])
            vp = to_rank_space(v[b, :, h, :], self.U_V[h])
            if self.storage is not None:
                kp, vp = self.storage(kp), self.storage(vp)
            self.Kp[(b, h)] = np.concatenate([self.Kp[(b, h)], kp], axis=0)
            self.Vp[(b, h)] = np.concatenate([self.Vp[(b, h)], vp], axis=0)
            self.cache_elements += kp.size + vp.size
            self.projection_macs += T * self.d_h * (kp.shape[1] + vp.shape[1])
        self.len += T

    def append_unit_rows(self, unit: Tuple[int, int], k_rows: np.ndarray, v_rows: np.ndarray) -> None:
        """Same as append_kv for one tracked unit given its rows [T, d_h] (large workloads
        hand the history over unit by unit); the caller advances `len` with set_len."""
        b, h = unit
        kp = to_rank_space(k_rows, self.U_K[h])
        vp = to_rank_space(v_rows, self.U_V[h])
        if self.storage is not None:
            kp, vp = self.storage(kp), self.storage(vp)
        self.Kp[unit] = np.concatenate([self.Kp[unit], kp], axis=0)
        self.Vp[unit] = np.concatenate([self.Vp[unit], vp], axis=0)
        self.cache_elements += kp.size + vp.size
        self.projection_macs += k_rows.shape[0] * self.d_h * (kp.shape[1] + vp.shape[1])

    def set_len(self, n: int) -> None:
        self.len = n

    # -- Eq. 3 in the rank-r space of Eq. 7
    def decode(self, q: np.ndarray, lowrank_out: bool = False) -> dict:
        """q: [B, 1, H, d_h] (or [B, H, d_h]).  Returns {(b,h): out[d_h]} for tracked units."""
        q = np.asarray(q, dtype=F64).reshape(self.B, self.H, self.d_h)
        out = {}
        self.attention_macs = 0
        for (b, h) in self.units:
            Kp, Vp = self.Kp[(b, h)], self.Vp[(b, h)]
            assert Kp.shape[0] == self.len and self.len > 0
            if self.rope is not None:
                assert not self.alibi[h]
                o = decode_head_rope(q[b, h], Kp, Vp, self.U_K[h], self.U_V[h], self.rope["base"],
                                     self.rope.get("interleaved", False), 0, lowrank_out)
                self.projection_macs += self.d_h * (Kp.size + (0 if lowrank_out else o.shape[0]))
                self.attention_macs += self.d_h * Kp.shape[0] + Vp.size
                out[(b, h)] = o
                continue
            qp = to_rank_space(q[b, h], self.U_K[h])
            self.projection_macs += self.d_h * qp.shape[0]
            s = (Kp @ qp) / math.sqrt(self.d_h)
            if self.alibi[h]:
                s = s + alibi_bias(self.alibi[h], self.len - 1, self.len)
            p = softmax_rows(s[None, :])[0]
            o = p @ Vp
            self.attention_macs += Kp.size + Vp.size
            if lowrank_out:
                out[(b, h)] = o
            else:
                out[(b, h)] = lift(o, self.U_V[h])
                self.projection_macs += self.d_h * o.shape[0]
        return out

    # -- grouped-query attention (Section 5.1: Llama-2-70b and Llama-3 share each K/V head among a group of
    #    query heads): the cache, U^K and U^V belong to the K/V head, every query head of its group uses them
    def decode_gqa(self, q: np.ndarray, group: int) -> np.ndarray:
        """q: [B, 1, H*group, d_h], query head hq belongs to K/V head hq // group.  Returns [B, 1, H*group, d_h].
        Each query head is Eq. 3 in the space of Eq. 7 against its K/V head's rank-r rows; with a rotary embedding
        each query head is the Section 4.3 form against its K/V head's rows and bases."""
        q = np.asarray(q, dtype=F64).reshape(self.B, self.H * group, self.d_h)
        out = np.zeros((self.B, 1, self.H * group, self.d_h), dtype=F64)
        for (b, h) in self.units:
            Kp, Vp = self.Kp[(b, h)], self.Vp[(b, h)]
            assert Kp.shape[0] == self.len and self.len > 0
            for i in range(group):
                hq = h * group + i
                if self.rope is not None:
                    assert not self.alibi[h]
                    out[b, 0, hq] = decode_head_rope(q[b, hq], Kp, Vp, self.U_K[h], self.U_V[h], self.rope["base"],
                                                     self.rope.get("interleaved", False), 0)
                    continue
                qp = to_rank_space(q[b, hq], self.U_K[h])
                s = (Kp @ qp) / math.sqrt(self.d_h)
                if self.alibi[h]:
                    s = s + alibi_bias(self.alibi[h], self.len - 1, self.len)
                p = softmax_rows(s[None, :])[0]
                out[b, 0, hq] = lift(p @ Vp, self.U_V[h])
        return out

    # -- Section 5.3: the same decode step over a cache whose complete groups of G rows are kept as b-bit codes
    def decode_quant(self, q: np.ndarray, bits: int, group: int, lowrank_out: bool = False) -> dict:
        """Eq. 3 in the space of Eq. 7 with K', V' replaced by what the quantised cache holds of them
        (oracle/kv_quant.py: keys per channel, values per token, the newest n mod G rows as stored)."""
        from .kv_quant import quantized_view
        q = np.asarray(q, dtype=F64).reshape(self.B, self.H, self.d_h)
        assert self.rope is None
        out = {}
        for (b, h) in self.units:
            Kq, Vq = quantized_view(self.Kp[(b, h)], self.Vp[(b, h)], bits, group)
            qp = to_rank_space(q[b, h], self.U_K[h])
            s = (Kq @ qp) / math.sqrt(self.d_h)
            if self.alibi[h]:
                s = s + alibi_bias(self.alibi[h], self.len - 1, self.len)
            o = softmax_rows(s[None, :])[0] @ Vq
            out[(b, h)] = o if lowrank_out else lift(o, self.U_V[h])
        return out

    def decode_dense(self, q: np.ndarray) -> np.ndarray:
        """decode() gathered into [B, 1, H, d_h] (all units must be tracked)."""
        res = self.decode(q)
        out = np.zeros((self.B, 1, self.H, self.d_h), dtype=F64)
        for (b, h), o in res.items():
            out[b, 0, h] = o
        return out

    # -- prefill: cache the prompt's rank-r K/V, causal attention of its queries
    def prefill(self, q: np.ndarray, k: np.ndarray, v: np.ndarray) -> dict:
        """q, k, v: [B, T, H, d_h].  Returns {(b,h): out[T, d_h]}."""
        q = np.asarray(q, dtype=F64)
        len0 = self.len
        self.append_kv(k, v)
        T = q.shape[1]
        out = {}
        if self.rope is not None:
            for (b, h) in self.units:
                assert not self.alibi[h]
                out[(b, h)] = prefill_head_rope(q[b, :, h, :], self.Kp[(b, h)], self.Vp[(b, h)], self.U_K[h], self.U_V[h],
                                                self.rope["base"], self.rope.get("interleaved", False), len0)
            return out
        for (b, h) in self.units:
            Qp = to_rank_space(q[b, :, h, :], self.U_K[h])
            Kp, Vp = self.Kp[(b, h)], self.Vp[(b, h)]
            O = np.zeros((T, Vp.shape[1]), dtype=F64)
            for t in range(T):
                n_t = len0 + t + 1
                s = (Kp[:n_t] @ Qp[t]) / math.sqrt(self.d_h)
                if self.alibi[h]:
                    s = s + alibi_bias(self.alibi[h], n_t - 1, n_t)
                p = softmax_rows(s[None, :])[0]
                O[t] = p @ Vp[:n_t]
            out[(b, h)] = lift(O, self.U_V[h])
        return out

    def prefill_dense(self, q, k, v) -> np.ndarray:
        res = self.prefill(q, k, v)
        T = np.asarray(q).shape[1]
        out = np.zeros((self.B, T, self.H, self.d_h), dtype=F64)
        for (b, h), o in res.items():
            out[b, :, h, :] = o
        return out


# --------------------------------------------------------------------------
# A paged cache: where a sequence's rows live, nothing else
# --------------------------------------------------------------------------

def paged_gather(pool: np.ndarray, table_row: Sequence[int], page_rows: int, n: int) -> np.ndarray:
    """Rows 0..n-1 of one sequence out of a pool of pages.  `pool` is [pages * page_rows, width] (physical page p =
    rows p*page_rows .. (p+1)*page_rows - 1); logical row r lives in physical page table_row[r // page_rows] at
    offset r % page_rows.  Paging changes addresses only: the paper's generation phase (Section 2) is stated on
    the rows K, V of a sequence, wherever they are kept, so attention over the gathered rows IS the paged result."""
    pool = np.asarray(pool)
    out = np.empty((n, pool.shape[1]), dtype=pool.dtype)
    for r in range(n):
        page = int(table_row[r // page_rows])
        assert page >= 0, "row in an unmapped page"
        out[r] = pool[page * page_rows + r % page_rows]
    return out


def paged_scatter(pool: np.ndarray, table_row: Sequence[int], page_rows: int, row0: int, rows: np.ndarray) -> None:
    """Writes `rows` at logical rows row0.. of one sequence into the pool (the append of Section 2, paged)."""
    for i in range(rows.shape[0]):
        r = row0 + i
        page = int(table_row[r // page_rows])
        assert page >= 0, "row in an unmapped page"
        pool[page * page_rows + r % page_rows] = rows[i]


# --------------------------------------------------------------------------
# Closed forms the paper states (Table 1, Section 2)
# --------------------------------------------------------------------------

def kv_cache_bits(b: int, n: int, d: int, L: int, p: int) -> int:
    """KV-cache size in bits: 2 * b * n * d * L * p with d the model width.

    Section 2 prints an extra factor h; since d = h * d_h already covers all
    heads, the paper's own worked example (batch 16, 32k context, 7B model,
    16 bit -> 256 GB, Section 1) fixes the formula without it.
    """
    return 2 * b * n * d * L * p


def table1_standard(n: int, d: int) -> dict:
    """Table 1, standard attention column (per token, per layer; FLOPs are multiply-accumulates)."""
    return {"kv_cache": 2 * n * d, "params": 4 * d * d, "flops": 4 * d * d + 2 * n * d}


def table1_eigen(n: int, d: int, r: int) -> dict:
    """Table 1, Eigen Attention column; r is the layer-wide rank (sum over heads)."""
    return {"kv_cache": 2 * n * r, "params": 4 * d * r, "flops": 4 * d * r + 2 * n * r}
