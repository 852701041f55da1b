"""Pins for the oracle's ALiBi bias (the MPT models' position scheme, Section 5.1): a library attention
routine given the bias as an additive mask, the geometric-series closed form for a zero query, Python
loops, and the consistency of decode with the last prefill row."""
import math

import numpy as np
import pytest
import torch

from oracle import eigen_attention as orc
from paper_2408_05646_b200 import synth


def case(seed, n, d_h, r_k, r_v):
    rng = np.random.default_rng(seed)
    U_K = synth.orthonormal_basis(d_h, r_k, seed + 1)
    U_V = synth.orthonormal_basis(d_h, r_v, seed + 2)
    return rng.standard_normal((n, d_h)), rng.standard_normal((n, d_h)), rng.standard_normal((n, d_h)), U_K, U_V


@pytest.mark.parametrize("d_h,r_k,r_v,n,slope", [(16, 5, 9, 23, 0.5), (64, 32, 32, 70, 0.0625), (128, 80, 48, 33, 2.0 ** -8)])
def test_bias_equals_library_attention_with_additive_mask(d_h, r_k, r_v, n, slope):
    Q, K, V, U_K, U_V = case(31 + d_h, n, d_h, r_k, r_v)
    Qp, Kp, Vp = Q @ U_K @ U_K.T, K @ U_K @ U_K.T, V @ U_V @ U_V.T        # Eq. 6
    i = torch.arange(n, dtype=torch.float64)
    mask = -slope * (i[:, None] - i[None, :])                              # query position minus key position
    mask = mask.masked_fill(i[None, :] > i[:, None], float("-inf"))       # causal
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Qp)[None, None], torch.from_numpy(Kp)[None, None], torch.from_numpy(Vp)[None, None],
        attn_mask=mask)[0, 0].numpy()
    got = orc.prefill_head(Q, K, V, U_K, U_V, alibi_slope=slope)
    assert np.abs(got - ref).max() < 1e-12
    got1 = orc.decode_head(Q[-1], K, V, U_K, U_V, alibi_slope=slope)       # the last query, all rows
    assert np.abs(got1 - ref[-1]).max() < 1e-12


@pytest.mark.parametrize("n,slope", [(1, 0.5), (7, 0.5), (200, 0.03125), (5000, 2.0 ** -8)])
def test_zero_query_gives_truncated_geometric_weights(n, slope):
    """q = 0: weights are rho^(n-1-j) (1-rho)/(1-rho^n) with rho = exp(-slope), so a value channel that
    holds j has mean (n-1) - [rho/(1-rho) - n rho^n/(1-rho^n)], and a constant channel stays constant."""
    d_h = 8
    U = np.eye(d_h)
    K = np.random.default_rng(5).standard_normal((n, d_h))
    V = np.zeros((n, d_h))
    V[:, 0] = 1.0
    V[:, 1] = np.arange(n)
    out = orc.decode_head(np.zeros(d_h), K, V, U, U, alibi_slope=slope)
    rho = math.exp(-slope)
    mean_back = rho / (1 - rho) - n * rho ** n / (1 - rho ** n)
    assert abs(out[0] - 1.0) < 1e-12
    assert abs(out[1] - ((n - 1) - mean_back)) < 1e-9 * max(1, n)
    # a wrong sign would favour the oldest rows instead
    assert out[1] > (n - 1) / 2 or n == 1


def test_bias_by_loops_and_zero_slope():
    n, d_h, r = 9, 6, 4
    Q, K, V, U_K, U_V = case(77, n, d_h, r, r)
    slope = 0.25
    qp = [sum(Q[-1][d] * U_K[d][c] for d in range(d_h)) for c in range(r)]
    s = []
    for j in range(n):
        kp = [sum(K[j][d] * U_K[d][c] for d in range(d_h)) for c in range(r)]
        s.append(sum(qp[c] * kp[c] for c in range(r)) / math.sqrt(d_h) - slope * ((n - 1) - j))
    m = max(s)
    e = [math.exp(x - m) for x in s]
    z = sum(e)
    o = [0.0] * r
    for j in range(n):
        vp = [sum(V[j][d] * U_V[d][c] for d in range(d_h)) for c in range(r)]
        for c in range(r):
            o[c] += e[j] / z * vp[c]
    out = [sum(o[c] * U_V[d][c] for c in range(r)) for d in range(d_h)]
    got = orc.decode_head(Q[-1], K, V, U_K, U_V, alibi_slope=slope)
    assert np.abs(got - np.array(out)).max() < 1e-12
    # slope 0 is the plain path
    assert np.array_equal(orc.decode_head(Q[-1], K, V, U_K, U_V, alibi_slope=0.0), orc.decode_head(Q[-1], K, V, U_K, U_V))


def test_layer_applies_per_head_slopes_and_decode_equals_last_prefill_row():
    B, H, d_h, T = 2, 4, 16, 12
    rng = np.random.default_rng(3)
    rk, rv = [4, 8, 16, 5], [8, 4, 3, 16]
    U_K = [synth.orthonormal_basis(d_h, r, 10 + h) for h, r in enumerate(rk)]
    U_V = [synth.orthonormal_basis(d_h, r, 20 + h) for h, r in enumerate(rv)]
    slopes = synth.alibi_slopes(H)
    q, k, v = (rng.standard_normal((B, T, H, d_h)) for _ in range(3))
    lay = orc.LayerOracle(B, H, d_h, U_K, U_V, alibi_slopes=slopes)
    out = lay.prefill_dense(q, k, v)
    for b in range(B):
        for h in range(H):
            ref = orc.prefill_head(q[b, :, h], k[b, :, h], v[b, :, h], U_K[h], U_V[h], alibi_slope=slopes[h])
            assert np.abs(out[b, :, h] - ref).max() < 1e-12
    lay2 = orc.LayerOracle(B, H, d_h, U_K, U_V, alibi_slopes=slopes)
    lay2.append_kv(k, v)
    dec = lay2.decode_dense(q[:, -1:])
    assert np.abs(dec[:, 0] - out[:, -1]).max() < 1e-12
    # chunked prefill: positions continue from the cached length
    lay3 = orc.LayerOracle(B, H, d_h, U_K, U_V, alibi_slopes=slopes)
    a = lay3.prefill_dense(q[:, :5], k[:, :5], v[:, :5])
    c = lay3.prefill_dense(q[:, 5:], k[:, 5:], v[:, 5:])
    assert np.abs(np.concatenate([a, c], axis=1) - out).max() < 1e-12


def test_published_slopes():
    s8 = synth.alibi_slopes(8)
    assert s8 == [2.0 ** -(i + 1) for i in range(8)]                      # 1/2, 1/4, ... 1/256
    s32 = synth.alibi_slopes(32)
    assert abs(s32[0] - 2.0 ** -0.25) < 1e-15 and abs(s32[-1] - 2.0 ** -8) < 1e-15
    s12 = synth.alibi_slopes(12)
    assert len(s12) == 12 and s12[:8] == s8 and s12[8:] == [2.0 ** -0.5, 2.0 ** -1.5, 2.0 ** -2.5, 2.0 ** -3.5]


def test_storage_hook_rounds_only_the_cached_rows():
    B, H, d_h, T = 1, 2, 16, 6
    rng = np.random.default_rng(9)
    U = [synth.orthonormal_basis(d_h, 8, 40 + h) for h in range(H)]
    k, v, q = (rng.standard_normal((B, T, H, d_h)) for _ in range(3))
    to_bf16 = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).double().numpy()
    plain = orc.LayerOracle(B, H, d_h, U, U)
    same = orc.LayerOracle(B, H, d_h, U, U, storage=lambda a: a)
    rounded = orc.LayerOracle(B, H, d_h, U, U, storage=to_bf16)
    for lay in (plain, same, rounded):
        lay.append_kv(k, v)
    assert np.array_equal(plain.decode_dense(q[:, -1:]), same.decode_dense(q[:, -1:]))
    for u in rounded.units:
        assert np.array_equal(rounded.Kp[u], to_bf16(plain.Kp[u])) and np.array_equal(rounded.Vp[u], to_bf16(plain.Vp[u]))
    # attention over the rounded rows equals the per-head definition given rows that are exact in the basis
    b, h = 0, 1
    K_exact = rounded.Kp[(b, h)] @ U[h].T           # rows whose coordinates are the stored ones
    V_exact = rounded.Vp[(b, h)] @ U[h].T
    ref = orc.decode_head(q[b, -1, h], K_exact, V_exact, U[h], U[h])
    assert np.abs(rounded.decode_dense(q[:, -1:])[b, 0, h] - ref).max() < 1e-12
