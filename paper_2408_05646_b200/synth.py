"""Seeded synthetic inputs for Eigen Attention workloads.

This module only *draws inputs*: orthonormal bases, low-rank-plus-noise K/V/Q
rows and per-head ranks.  It contains none of the method's arithmetic (no
projection into the rank-r space, no softmax, no attention) and is the one
module that both the CUDA path's callers and the CPU oracle's tests may share.

Recipe (shapes follow the 7B-class layers the paper evaluates: 32 heads,
d_head 128, 16-bit cache, ranks at 0.6x-0.8x of d_head):

* bases   U = Q factor of a Householder QR of a seeded N(0,1) d_head x r matrix,
          computed in fp64, signs fixed so diag(R) > 0, checked for
          max|U^T U - I| <= 1e-12, then rounded once to fp32.  Both the GPU
          library and the oracle receive those fp32 values.
* K, V, Q rows: per head a fixed mixing matrix W ~ N(0,1)^{rho x d_head}
          (a property of the layer, shared across the batch), per token a
          latent z ~ N(0,1)^rho;  x = z W / sqrt(rho) + sigma * N(0,1), which
          has roughly unit variance and the low-rank-plus-noise spectrum the
          paper reports for keys and values.  Rows are rounded once to the IO
          dtype (round-to-nearest-even for bf16); both sides get those values.
* ranks   per-head r drawn uniformly from a given set.

Streams: base seed 240805646 + config index; one sub-stream per tag below, so
that drawing one tensor never shifts another.
"""
from __future__ import annotations

import dataclasses
from typing import List, Sequence

import numpy as np
import torch

BASE_SEED = 240805646

TAGS = {
    "U_K": 1, "U_V": 2, "W_K": 3, "W_V": 4, "W_Q": 5,
    "z_K": 6, "z_V": 7, "z_Q": 8, "noise_K": 9, "noise_V": 10, "noise_Q": 11,
    "ranks": 12, "q": 13, "subset": 14,
}


def stream_seed(config: int, tag: str, extra: int = 0) -> int:
    """Seed of the sub-stream `tag` of workload `config` (`extra` separates chunks)."""
    return (BASE_SEED + config) * 1000003 + TAGS[tag] * 7919 + extra * 104729


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape of one synthetic workload (one decoder layer)."""
    index: int            # which of the five reference workloads (1-based)
    name: str
    batch: int
    n_heads: int
    d_head: int
    ranks: Sequence[int]  # candidate set; one value = uniform rank
    context: int          # cached rows before the new token (decode) or prompt length (prefill)
    dtype: str            # "bf16" | "fp32"
    rho: int              # rank of the low-rank signal
    sigma: float          # noise level
    q_scale: float        # q ~ N(0,1) * q_scale for decode workloads


WORKLOADS = {
    "tiny_fp32": Workload(1, "tiny_fp32", 1, 4, 64, (32,), 512, "fp32", 24, 0.05, 1.0 / 8.0),
    "llama2_7b_b16_n32k": Workload(2, "llama2_7b_b16_n32k", 16, 32, 128, (80,), 32768, "bf16", 64, 0.1, 1.0),
    "opt_6p7b_hetero": Workload(3, "opt_6p7b_hetero", 4, 32, 128, (48, 64, 80, 96, 112), 8192, "bf16", 64, 0.1, 1.0),
    "mpt_7b_long": Workload(4, "mpt_7b_long", 1, 32, 128, (64,), 131072, "bf16", 64, 0.1, 1.0),
    "prefill_b4_t4096": Workload(5, "prefill_b4_t4096", 4, 32, 128, (80,), 4096, "bf16", 64, 0.1, 1.0),
    # grouped-query layer of the 8B-class models: 8 K/V heads (n_heads), 4 query heads each
    "llama3_8b_gqa_b16_n32k": Workload(6, "llama3_8b_gqa_b16_n32k", 16, 8, 128, (80,), 32768, "bf16", 64, 0.1, 1.0),
}
GQA_GROUP = {"llama3_8b_gqa_b16_n32k": 4}


def torch_dtype(name: str) -> torch.dtype:
    return {"bf16": torch.bfloat16, "fp32": torch.float32}[name]


def draw_ranks(n_heads: int, choices: Sequence[int], config: int) -> List[int]:
    """Per-head ranks, uniform over `choices` (a single choice gives a uniform rank)."""
    if len(choices) == 1:
        return [int(choices[0])] * n_heads
    rng = np.random.default_rng(stream_seed(config, "ranks"))
    return [int(choices[i]) for i in rng.integers(0, len(choices), size=n_heads)]


def orthonormal_basis(d_head: int, r: int, seed: int) -> np.ndarray:
    """d_head x r matrix with orthonormal columns (fp64), from QR of a seeded Gaussian."""
    rng = np.random.default_rng(seed)
    G = rng.standard_normal((d_head, r))
    Q, R = np.linalg.qr(G, mode="reduced")          # LAPACK Householder QR, fp64
    sign = np.sign(np.diag(R))
    sign[sign == 0] = 1.0
    Q = Q * sign[None, :]
    err = np.abs(Q.T @ Q - np.eye(r)).max()
    if err > 1e-12:
        raise RuntimeError(f"basis not orthonormal: {err}")
    return Q


def make_bases(d_head: int, ranks: Sequence[int], config: int, tag: str) -> List[np.ndarray]:
    """One fp32 basis per head (d_head x r[h], columns = basis vectors)."""
    return [orthonormal_basis(d_head, int(r), stream_seed(config, tag, extra=h)).astype(np.float32)
            for h, r in enumerate(ranks)]


def mixing_matrices(n_heads: int, rho: int, d_head: int, config: int, tag: str,
                    device: str | torch.device = "cpu") -> torch.Tensor:
    """W[h] ~ N(0,1)^{rho x d_head}, fp32, drawn on the CPU so every device sees the same layer."""
    g = torch.Generator(device="cpu").manual_seed(stream_seed(config, tag))
    W = torch.randn((n_heads, rho, d_head), generator=g, dtype=torch.float32)
    return W.to(device)


def lowrank_rows(W: torch.Tensor, batch: int, tokens: int, sigma: float, config: int,
                 which: str, chunk: int = 0, dtype: torch.dtype = torch.bfloat16,
                 device: str | torch.device = "cpu") -> torch.Tensor:
    """[batch][tokens][n_heads][d_head] rows x = z W / sqrt(rho) + sigma * e, rounded to `dtype`.

    `which` is "K", "V" or "Q" (selects the latent and noise streams); `chunk`
    separates successive calls that fill one long context piece by piece.
    """
    n_heads, rho, d_head = W.shape
    dev = torch.device(device)
    gz = torch.Generator(device=dev).manual_seed(stream_seed(config, "z_" + which, extra=chunk))
    ge = torch.Generator(device=dev).manual_seed(stream_seed(config, "noise_" + which, extra=chunk))
    z = torch.randn((batch, tokens, n_heads, rho), generator=gz, dtype=torch.float32, device=dev)
    x = torch.einsum("bthp,hpd->bthd", z, W.to(dev)) / float(np.sqrt(rho))
    del z
    e = torch.randn((batch, tokens, n_heads, d_head), generator=ge, dtype=torch.float32, device=dev)
    x.add_(e, alpha=float(sigma))
    del e
    return x.to(dtype).contiguous()


def gaussian_query(batch: int, n_heads: int, d_head: int, scale: float, config: int,
                   step: int = 0, dtype: torch.dtype = torch.bfloat16,
                   device: str | torch.device = "cpu") -> torch.Tensor:
    """[batch][1][n_heads][d_head] query q ~ N(0,1) * scale, rounded to `dtype`."""
    dev = torch.device(device)
    g = torch.Generator(device=dev).manual_seed(stream_seed(config, "q", extra=step))
    q = torch.randn((batch, 1, n_heads, d_head), generator=g, dtype=torch.float32, device=dev) * scale
    return q.to(dtype).contiguous()


def alibi_slopes(n_heads: int) -> List[float]:
    """Per-head ALiBi slopes as published for a power-of-two head count: 2^(-8 (h+1) / H), h = 0..H-1;
    other head counts take the slopes of the next power of two, the even ones first then the odd ones."""
    def pow2(n):
        return [2.0 ** (-8.0 * (i + 1) / n) for i in range(n)]
    if n_heads & (n_heads - 1) == 0:
        return pow2(n_heads)
    lower = 1 << (n_heads.bit_length() - 1)
    return pow2(lower) + pow2(2 * lower)[0::2][: n_heads - lower]


def sample_units(batch: int, n_heads: int, ranks: Sequence[int], count: int, config: int):
    """Seeded subset of (b, h) units: always the two corners, every distinct rank and every batch index."""
    rng = np.random.default_rng(stream_seed(config, "subset"))
    chosen = [(0, 0), (batch - 1, n_heads - 1)]
    seen_r = set()
    for h, r in enumerate(ranks):
        if r not in seen_r:
            seen_r.add(r)
            chosen.append((int(rng.integers(0, batch)), h))
    for b in range(batch):
        chosen.append((b, int(rng.integers(0, n_heads))))
    while len(set(chosen)) < min(count, batch * n_heads):
        chosen.append((int(rng.integers(0, batch)), int(rng.integers(0, n_heads))))
    out, seen = [], set()
    for u in chosen:
        if u not in seen:
            seen.add(u)
            out.append(u)
    return out
