"""Pins for the oracle's grouped-query decode: the library attention routine in its grouped mode on the d_h-wide
low-rank inputs of Eq. 6, and ordinary multi-head decode with every K/V head repeated for its group."""
import numpy as np
import pytest
import torch

from oracle import eigen_attention as orc
from paper_2408_05646_b200 import synth


@pytest.mark.parametrize("H,g,d_h,n", [(2, 4, 16, 23), (3, 2, 32, 40), (1, 8, 64, 9)])
def test_gqa_equals_library_grouped_attention_and_repeated_heads(H, g, d_h, n):
    B = 2
    rng = np.random.default_rng(H * 10 + g)
    rk = [max(2, d_h // 2 - h) for h in range(H)]
    rv = [max(3, d_h // 2 + h) for h in range(H)]
    U_K = [synth.orthonormal_basis(d_h, r, 70 + h) for h, r in enumerate(rk)]
    U_V = [synth.orthonormal_basis(d_h, r, 80 + h) for h, r in enumerate(rv)]
    k, v = rng.standard_normal((2, B, n, H, d_h))
    q = rng.standard_normal((B, 1, H * g, d_h))
    lay = orc.LayerOracle(B, H, d_h, U_K, U_V)
    lay.append_kv(k, v)
    got = lay.decode_gqa(q, g)
    # (1) the library's grouped mode on Q', K', V' of Eq. 6 (d_h wide, so its default scale is 1/sqrt(d_h))
    Kp = np.stack([k[:, :, h] @ U_K[h] @ U_K[h].T for h in range(H)], axis=1)            # [B, H, n, d_h]
    Vp = np.stack([v[:, :, h] @ U_V[h] @ U_V[h].T for h in range(H)], axis=1)
    Qp = np.stack([q[:, :, hq] @ U_K[hq // g] @ U_K[hq // g].T for hq in range(H * g)], axis=1)   # [B, H*g, 1, d_h]
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Qp), torch.from_numpy(Kp), torch.from_numpy(Vp), enable_gqa=True).numpy()   # [B, H*g, 1, d_h]
    assert np.abs(got[:, 0] - ref[:, :, 0]).max() < 1e-12
    # (2) ordinary decode of a layer whose heads are the K/V heads repeated g times
    rep = orc.LayerOracle(B, H * g, d_h, [U_K[hq // g] for hq in range(H * g)], [U_V[hq // g] for hq in range(H * g)])
    rep.append_kv(np.repeat(k, g, axis=2), np.repeat(v, g, axis=2))
    assert np.abs(got - rep.decode_dense(q)).max() < 1e-12
    # group 1 is the multi-head path itself
    one = orc.LayerOracle(B, H, d_h, U_K, U_V)
    one.append_kv(k, v)
    assert np.array_equal(one.decode_gqa(q[:, :, ::g], 1), one.decode_dense(q[:, :, ::g]))


@pytest.mark.parametrize("interleaved", [False, True])
@pytest.mark.parametrize("H,g,d_h,n", [(2, 4, 16, 23), (1, 3, 32, 11)])
def test_gqa_with_rotary_embedding_equals_library_attention_on_rotated_lifted_keys(H, g, d_h, n, interleaved):
    """Section 4.3 for a group: every query head against its K/V head's keys taken back through (U^K)^T and rotated.
    The reference rotates with torch's complex arithmetic (its own cos/sin and pairing), lifts with plain matrix
    products and calls the library's grouped attention; a second reference is the (pinned) multi-head form of a
    layer whose heads are the K/V heads repeated."""
    B, base = 2, 10000.0
    rng = np.random.default_rng(100 + H * 10 + g)
    rk = [max(2, d_h // 2 - h) for h in range(H)]
    rv = [max(3, d_h // 2 + h) for h in range(H)]
    U_K = [synth.orthonormal_basis(d_h, r, 170 + h) for h, r in enumerate(rk)]
    U_V = [synth.orthonormal_basis(d_h, r, 180 + h) for h, r in enumerate(rv)]
    k, v = rng.standard_normal((2, B, n, H, d_h))
    q = rng.standard_normal((B, 1, H * g, d_h))
    lay = orc.LayerOracle(B, H, d_h, U_K, U_V, rope={"base": base, "interleaved": interleaved})
    lay.append_kv(k, v)
    got = lay.decode_gqa(q, g)

    def rotate(x, pos):                                              # x [..., d_h] at integer positions pos [...]
        t = torch.from_numpy(np.ascontiguousarray(x))
        freq = base ** (-torch.arange(0, d_h, 2, dtype=torch.float64) / d_h)
        ang = torch.tensor(np.array(pos), dtype=torch.float64)[..., None] * freq
        z = torch.polar(torch.ones_like(ang), ang)
        if interleaved:
            pairs = torch.view_as_complex(t.reshape(*t.shape[:-1], d_h // 2, 2).contiguous())
            return torch.view_as_real(pairs * z).reshape(t.shape).numpy()
        pairs = torch.complex(t[..., : d_h // 2], t[..., d_h // 2:]) * z
        return torch.cat([pairs.real, pairs.imag], dim=-1).numpy()

    pos = np.arange(n)
    K_back = np.stack([rotate(k[:, :, h] @ U_K[h] @ U_K[h].T, np.broadcast_to(pos, (B, n))) for h in range(H)], axis=1)
    V_back = np.stack([v[:, :, h] @ U_V[h] @ U_V[h].T for h in range(H)], axis=1)                   # [B, H, n, d_h]
    Q_rot = np.stack([rotate(q[:, :, hq], np.full((B, 1), n - 1)) for hq in range(H * g)], axis=1)   # [B, H*g, 1, d_h]
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q_rot), torch.from_numpy(K_back), torch.from_numpy(V_back), enable_gqa=True).numpy()
    assert np.abs(got[:, 0] - ref[:, :, 0]).max() < 1e-11
    rep = orc.LayerOracle(B, H * g, d_h, [U_K[hq // g] for hq in range(H * g)], [U_V[hq // g] for hq in range(H * g)],
                          rope={"base": base, "interleaved": interleaved})
    rep.append_kv(np.repeat(k, g, axis=2), np.repeat(v, g, axis=2))
    assert np.abs(got - rep.decode_dense(q)).max() < 1e-12
