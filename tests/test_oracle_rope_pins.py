"""Pins for the oracle's RoPE variant (Section 4.3): library attention on keys and queries rotated with complex
arithmetic (an independent route to the rotation), relative-position invariance, the zero-angle special case,
Python loops with explicit 2x2 rotations, and the layer against the per-head function."""
import math

import numpy as np
import pytest
import torch

from oracle import eigen_attention as orc
from paper_2408_05646_b200 import synth


def rotate_complex(x, pos, base, interleaved):
    """RoPE through complex multiplication (torch.polar), independent of the oracle's block rotation."""
    x = torch.from_numpy(np.asarray(x, dtype=np.float64))
    d = x.shape[-1]
    inv = torch.tensor([base ** (-2.0 * i / d) for i in range(d // 2)], dtype=torch.float64)
    ang = torch.as_tensor(pos, dtype=torch.float64)[..., None] * inv
    rot = torch.polar(torch.ones_like(ang), ang)
    if interleaved:
        z = torch.view_as_complex(x.reshape(*x.shape[:-1], d // 2, 2).contiguous()) * rot
        return torch.view_as_real(z).reshape(x.shape).numpy()
    z = torch.complex(x[..., : d // 2], x[..., d // 2:]) * rot
    return torch.cat([z.real, z.imag], dim=-1).numpy()


@pytest.mark.parametrize("interleaved", [False, True])
@pytest.mark.parametrize("d_h,r_k,r_v,n,base", [(16, 16, 16, 23, 10000.0), (64, 20, 32, 70, 500000.0), (128, 80, 48, 33, 10000.0)])
def test_rope_variant_equals_library_attention_on_rotated_lifted_keys(d_h, r_k, r_v, n, base, interleaved):
    rng = np.random.default_rng(d_h + n)
    U_K = synth.orthonormal_basis(d_h, r_k, 3)
    U_V = synth.orthonormal_basis(d_h, r_v, 4)
    q, K, V = rng.standard_normal(d_h), rng.standard_normal((n, d_h)), rng.standard_normal((n, d_h))
    Kp, Vp = K @ U_K, V @ U_V
    pos0 = 5
    K_back = Kp @ U_K.T                                   # the extra transformation of Fig. 6(b)
    k_rot = rotate_complex(K_back, np.arange(pos0, pos0 + n), base, interleaved)
    q_rot = rotate_complex(q[None], [pos0 + n - 1], base, interleaved)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q_rot)[None, None], torch.from_numpy(k_rot)[None, None],
        torch.from_numpy(Vp @ U_V.T)[None, None])[0, 0, 0].numpy()          # scale 1/sqrt(d_h)
    got = orc.decode_head_rope(q, Kp, Vp, U_K, U_V, base, interleaved, pos0)
    assert np.abs(got - ref).max() < 1e-12
    if r_k == d_h:      # full rank: standard attention with RoPE on the original keys
        k_rot_full = rotate_complex(K, np.arange(pos0, pos0 + n), base, interleaved)
        ref_full = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q_rot)[None, None], torch.from_numpy(k_rot_full)[None, None],
            torch.from_numpy(V)[None, None])[0, 0, 0].numpy()
        assert np.abs(got - ref_full).max() < 1e-11


def test_rotation_properties():
    rng = np.random.default_rng(1)
    x, y = rng.standard_normal((2, 7, 32))
    for inter in (False, True):
        pos = np.arange(7) * 13 + 2
        rx = orc.rope_rotate(x, pos, 10000.0, inter)
        assert np.abs(np.linalg.norm(rx, axis=-1) - np.linalg.norm(x, axis=-1)).max() < 1e-12     # an isometry
        assert np.abs(orc.rope_rotate(x, np.zeros(7), 10000.0, inter) - x).max() == 0              # position 0: identity
        # the dot product of two rotated rows depends on the position difference only
        a = (orc.rope_rotate(x[0], 40, 10000.0, inter) * orc.rope_rotate(y[0], 33, 10000.0, inter)).sum()
        b = (orc.rope_rotate(x[0], 1007, 10000.0, inter) * orc.rope_rotate(y[0], 1000, 10000.0, inter)).sum()
        assert abs(a - b) < 1e-10
        # first pair turns by pos radians (frequency 1), by hand
        a_i, b_i = (0, 1) if inter else (0, 16)
        r = orc.rope_rotate(x[0], 3, 10000.0, inter)
        assert abs(r[a_i] - (x[0][a_i] * math.cos(3) - x[0][b_i] * math.sin(3))) < 1e-14
        assert abs(r[b_i] - (x[0][a_i] * math.sin(3) + x[0][b_i] * math.cos(3))) < 1e-14


def test_shift_invariance_zero_angle_case_and_self_score():
    d_h, r_k, r_v, n = 32, 12, 20, 40
    rng = np.random.default_rng(8)
    U_K, U_V = synth.orthonormal_basis(d_h, r_k, 5), synth.orthonormal_basis(d_h, r_v, 6)
    q, Kp, Vp = rng.standard_normal(d_h), rng.standard_normal((n, r_k)), rng.standard_normal((n, r_v))
    a = orc.decode_head_rope(q, Kp, Vp, U_K, U_V, 10000.0, False, 0)
    b = orc.decode_head_rope(q, Kp, Vp, U_K, U_V, 10000.0, False, 12345)
    assert np.abs(a - b).max() < 1e-9                                 # only relative positions matter
    # an enormous base makes every angle but the first pair's vanish; a single row sees no rotation at all:
    # then Section 4.3 reduces to Eq. 7 with q' = q U^K
    one = orc.decode_head_rope(q, Kp[:1], Vp[:1], U_K, U_V, 10000.0, False, 77)
    assert np.abs(one - Vp[0] @ U_V.T).max() < 1e-12
    # the newest row's score is the plain dot product q . (U k'): R R^T = I at equal positions
    K_back = Kp @ U_K.T
    s_rot = orc.rope_rotate(K_back[-1], n - 1) @ orc.rope_rotate(q, n - 1)
    assert abs(s_rot - K_back[-1] @ q) < 1e-11
    assert abs(K_back[-1] @ q - Kp[-1] @ (q @ U_K)) < 1e-11


def test_rope_variant_by_loops():
    d_h, r, n, base = 8, 3, 6, 100.0
    rng = np.random.default_rng(2)
    U_K, U_V = synth.orthonormal_basis(d_h, r, 7), synth.orthonormal_basis(d_h, r, 8)
    q, Kp, Vp = rng.standard_normal(d_h), rng.standard_normal((n, r)), rng.standard_normal((n, r))

    def rot(x, pos):                                  # half-split pairs (i, i + d/2), explicit 2x2 rotations
        y = [0.0] * d_h
        for i in range(d_h // 2):
            ang = pos * base ** (-2.0 * i / d_h)
            y[i] = x[i] * math.cos(ang) - x[i + d_h // 2] * math.sin(ang)
            y[i + d_h // 2] = x[i] * math.sin(ang) + x[i + d_h // 2] * math.cos(ang)
        return y
    qr = rot(list(q), n - 1)
    s = []
    for j in range(n):
        kb = [sum(Kp[j][c] * U_K[d][c] for c in range(r)) for d in range(d_h)]
        kr = rot(kb, j)
        s.append(sum(qr[d] * kr[d] for d in range(d_h)) / math.sqrt(d_h))
    m = max(s)
    e = [math.exp(x - m) for x in s]
    z = sum(e)
    o = [sum(e[j] / z * Vp[j][c] for j in range(n)) for c in range(r)]
    out = [sum(o[c] * U_V[d][c] for c in range(r)) for d in range(d_h)]
    got = orc.decode_head_rope(q, Kp, Vp, U_K, U_V, base, False, 0)
    assert np.abs(got - np.array(out)).max() < 1e-12


def test_layer_decode_follows_the_per_head_function():
    B, H, d_h, n = 2, 3, 16, 9
    rng = np.random.default_rng(4)
    rk, rv = [4, 16, 7], [8, 5, 16]
    U_K = [synth.orthonormal_basis(d_h, r, 50 + h) for h, r in enumerate(rk)]
    U_V = [synth.orthonormal_basis(d_h, r, 60 + h) for h, r in enumerate(rv)]
    k, v = rng.standard_normal((2, B, n, H, d_h))
    q = rng.standard_normal((B, 1, H, d_h))
    lay = orc.LayerOracle(B, H, d_h, U_K, U_V, rope={"base": 10000.0, "interleaved": True})
    lay.append_kv(k, v)
    out = lay.decode_dense(q)
    for b in range(B):
        for h in range(H):
            ref = orc.decode_head_rope(q[b, 0, h], k[b, :, h] @ U_K[h], v[b, :, h] @ U_V[h], U_K[h], U_V[h], 10000.0, True)
            assert np.abs(out[b, 0, h] - ref).max() < 1e-12


@pytest.mark.parametrize("interleaved", [False, True])
@pytest.mark.parametrize("d_h,r_k,r_v,T,len0,base", [(16, 16, 16, 9, 0, 10000.0), (64, 20, 32, 17, 6, 500000.0), (128, 80, 48, 12, 30, 10000.0)])
def test_rope_prompt_form_equals_causal_library_attention_and_the_generation_form(d_h, r_k, r_v, T, len0, base, interleaved):
    # The prompt form of Section 4.3: causal library attention on lifted keys and queries rotated through complex
    # multiplication (another route to the rotation, another implementation of the softmax and of the mask), with
    # the queries aligned to the END of the key axis (query t sits at position len0 + t); and row t equals the
    # generation form over the first len0 + t + 1 rows.
    rng = np.random.default_rng(d_h + T)
    U_K, U_V = synth.orthonormal_basis(d_h, r_k, 13), synth.orthonormal_basis(d_h, r_v, 14)
    n = len0 + T
    Q, K, V = rng.standard_normal((T, d_h)), rng.standard_normal((n, d_h)), rng.standard_normal((n, d_h))
    Kp, Vp = K @ U_K, V @ U_V
    got = orc.prefill_head_rope(Q, Kp, Vp, U_K, U_V, base, interleaved, len0)
    k_rot = rotate_complex(Kp @ U_K.T, np.arange(n), base, interleaved)
    q_rot = rotate_complex(Q, len0 + np.arange(T), base, interleaved)
    mask = torch.from_numpy(np.arange(n)[None, :] <= (len0 + np.arange(T))[:, None])
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q_rot)[None, None], torch.from_numpy(k_rot)[None, None],
        torch.from_numpy(Vp @ U_V.T)[None, None], attn_mask=mask)[0, 0].numpy()
    assert np.abs(got - ref).max() < 1e-12
    for t in (0, T // 2, T - 1):
        n_t = len0 + t + 1
        row = orc.decode_head_rope(Q[t], Kp[:n_t], Vp[:n_t], U_K, U_V, base, interleaved, 0)
        assert np.abs(got[t] - row).max() < 1e-12
    low = orc.prefill_head_rope(Q, Kp, Vp, U_K, U_V, base, interleaved, len0, lowrank_out=True)
    assert np.abs(low @ U_V.T - got).max() < 1e-12
    # a mask off by one (query t seeing row len0 + t + 1) or positions that ignore len0 do not pass
    if len0:
        wrong = orc.prefill_head_rope(Q, Kp[len0:], Vp[len0:], U_K, U_V, base, interleaved, 0)
        assert np.abs(wrong - got).max() > 1e-6


def test_layer_prefill_with_rope_follows_the_per_head_function_in_chunks():
    B, H, d_h, T = 2, 3, 16, 11
    rng = np.random.default_rng(14)
    rk, rv = [4, 16, 7], [8, 5, 16]
    U_K = [synth.orthonormal_basis(d_h, r, 70 + h) for h, r in enumerate(rk)]
    U_V = [synth.orthonormal_basis(d_h, r, 80 + h) for h, r in enumerate(rv)]
    q, k, v = rng.standard_normal((3, B, T, H, d_h))
    rope = {"base": 10000.0, "interleaved": False}
    one = orc.LayerOracle(B, H, d_h, U_K, U_V, rope=rope).prefill_dense(q, k, v)
    lay = orc.LayerOracle(B, H, d_h, U_K, U_V, rope=rope)
    two = np.concatenate([lay.prefill_dense(q[:, :4], k[:, :4], v[:, :4]), lay.prefill_dense(q[:, 4:], k[:, 4:], v[:, 4:])], axis=1)
    assert np.abs(one - two).max() < 1e-12                              # chunked prompt = one prompt
    for b in range(B):
        for h in range(H):
            ref = orc.prefill_head_rope(q[b, :, h], k[b, :, h] @ U_K[h], v[b, :, h] @ U_V[h], U_K[h], U_V[h], 10000.0, False)
            assert np.abs(one[b, :, h] - ref).max() < 1e-12
    nxt = rng.standard_normal((3, B, 1, H, d_h))                        # the prompt's cache serves the generation phase
    lay.append_kv(nxt[1], nxt[2])
    full = orc.LayerOracle(B, H, d_h, U_K, U_V, rope=rope)
    last = full.prefill_dense(np.concatenate([q, nxt[0]], axis=1), np.concatenate([k, nxt[1]], axis=1), np.concatenate([v, nxt[2]], axis=1))
    assert np.abs(lay.decode_dense(nxt[0]) - last[:, -1:]).max() < 1e-12
