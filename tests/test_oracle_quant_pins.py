"""Pins for the oracle's quantised cache (Section 5.3, Table 8): the cache sizes the paper prints, the error
bound of a uniform grid, data that already lies on the grid, the axis of the groups (keys per channel, values
per token), Python loops, and the limit of many bits."""
import math
import os

import numpy as np
import pytest

from oracle import eigen_attention as orc
from oracle import kv_quant as kq
from paper_2408_05646_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table8_quant_cache_sizes.txt")


def golden_rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                label, d, L, ratio, bits, group, gib = line.split()
                rows.append((label, int(d), int(L), float(ratio), int(bits), int(group), float(gib)))
    return rows


@pytest.mark.parametrize("row", golden_rows(), ids=lambda r: r[0])
def test_cache_size_matches_table_8(row):
    """All fifteen printed sizes follow from b bits per element plus one 16-bit number per group; a 32-bit
    scale-and-zero pair per group, or no metadata at all, misses several rows by more than the print
    precision (checked below for the rows with small groups)."""
    _, d, L, ratio, bits, group, printed = row
    elements = round(2 * 2048 * d * L * ratio)
    gib = kq.quant_cache_bytes(elements, bits, group) / 2 ** 30
    assert abs(gib - printed) <= 0.0051, (gib, printed)
    if group <= 32:
        two_numbers = elements * (bits + 32.0 / group) / 8 / 2 ** 30
        nothing = elements * bits / 8 / 2 ** 30
        assert abs(two_numbers - printed) > 0.0051 and abs(nothing - printed) > 0.0051


def loops_quantize(x, bits, group):
    """One group at a time, one element at a time, in Python floats rounded through numpy scalars."""
    qmax = 2 ** (bits - 1) - 1
    codes, scales = [], []
    for g0 in range(0, len(x), group):
        seg = [np.float32(v) for v in x[g0:g0 + group]]
        amax = max(abs(v) for v in seg)
        s = np.float16(np.float32(amax) / np.float32(qmax))
        scales.append(s)
        for v in seg:
            if float(s) == 0.0:
                codes.append(0)
                continue
            t = float(np.float32(v) / np.float32(s))
            r = math.floor(t)
            frac = t - r
            c = r + 1 if frac > 0.5 or (frac == 0.5 and r % 2 != 0) else r      # round half to even
            codes.append(max(-qmax, min(qmax, c)))
    return np.array(codes), np.array(scales)


@pytest.mark.parametrize("bits,group,n", [(4, 16, 16), (4, 32, 77), (3, 8, 40), (8, 128, 300), (2, 4, 9)])
def test_codes_and_scales_match_python_loops(bits, group, n):
    rng = np.random.default_rng(100 + bits * n)
    x = (rng.standard_normal(n) * 3.0).astype(np.float32).astype(np.float64)
    c, s = kq.quantize_groups(x, bits, group, axis=0)
    lc, ls = loops_quantize(x, bits, group)
    assert np.array_equal(c, lc)
    assert np.array_equal(s, ls)


@pytest.mark.parametrize("bits,group", [(4, 32), (3, 16), (8, 64)])
def test_error_is_at_most_half_a_step_and_extremes_hit_the_end_codes(bits, group):
    rng = np.random.default_rng(7)
    x = (rng.standard_normal((5, 4 * group)) * np.array([[0.01], [1.0], [30.0], [1e3], [1e-3]])).astype(np.float32)
    c, s = kq.quantize_groups(x, bits, group, axis=1)
    xh = kq.dequantize_groups(c, s, group, axis=1)
    qmax = kq.qmax_of(bits)
    step = np.repeat(s.astype(np.float64), group, axis=1)
    # half a step, plus what rounding the scale to half precision moves the end of the grid (2^-11 relative)
    bound = 0.5 * step + qmax * step * 2.0 ** -11 + 1e-12
    assert np.all(np.abs(xh - x) <= bound)
    assert np.all(np.abs(c) <= qmax)
    for g in range(4):
        seg = np.abs(c[:, g * group:(g + 1) * group])
        assert np.all(seg.max(axis=1) == qmax)              # the largest magnitude of a group takes an end code


def test_data_on_the_grid_is_reproduced_exactly():
    rng = np.random.default_rng(3)
    for bits, group in [(4, 32), (3, 16), (5, 8)]:
        qmax = kq.qmax_of(bits)
        codes = rng.integers(-qmax, qmax + 1, size=(6, 3 * group))
        codes[:, ::group] = qmax                             # every group reaches its end code
        scale = np.array([0.125, 0.5, 1.0, 3.0, 0.0078125, 10.0])[:, None]     # exact in half precision
        x = codes * scale
        c, s = kq.quantize_groups(x, bits, group, axis=1)
        assert np.array_equal(c, codes)
        assert np.array_equal(s.astype(np.float64), np.broadcast_to(scale, s.shape))
        assert np.array_equal(kq.dequantize_groups(c, s, group, axis=1), x)


def test_keys_are_grouped_per_channel_and_values_per_token():
    """An outlier changes the scale of its own group only: for keys that group is G tokens of ONE channel,
    for values G channels of ONE token.  A transposed axis fails both halves."""
    rng = np.random.default_rng(11)
    G, n, r = 16, 48, 32
    K = rng.standard_normal((n, r))
    V = rng.standard_normal((n, r))
    kc0, ks0 = kq.quantize_keys(K, 4, G)
    vc0, vs0 = kq.quantize_values(V, 4, G)
    assert ks0.shape == (n // G, r) and vs0.shape == (n, r // G)
    K2, V2 = K.copy(), V.copy()
    K2[20, 5] = 500.0          # token 20 (token group 1), channel 5
    V2[20, 5] = 500.0          # token 20, channel 5 (channel group 0)
    kc1, _ = kq.quantize_keys(K2, 4, G)
    vc1, _ = kq.quantize_values(V2, 4, G)
    changed_k = np.argwhere(kc1 != kc0)
    changed_v = np.argwhere(vc1 != vc0)
    assert len(changed_k) > 0 and len(changed_v) > 0
    assert set(changed_k[:, 1]) == {5} and set(changed_k[:, 0]) <= set(range(16, 32))     # one channel, its 16 tokens
    assert set(changed_v[:, 0]) == {20} and set(changed_v[:, 1]) <= set(range(0, 16))      # one token, its 16 channels


def test_scale_saturates_at_the_largest_half_precision_number():
    x = np.array([1e6, -3e5, 2e4, 0.0])
    c, s = kq.quantize_groups(x, 4, 4, axis=0)
    assert float(s[0]) == 65504.0 and np.all(np.isfinite(kq.dequantize_groups(c, s, 4, 0)))
    assert list(c) == [7, -5, 0, 0]                      # 1e6 / 65504 = 15.3 clips to 7; -3e5 / 65504 = -4.58


def test_view_keeps_the_incomplete_group_as_stored():
    rng = np.random.default_rng(5)
    K, V = rng.standard_normal((70, 24)), rng.standard_normal((70, 24))
    Kq, Vq = kq.quantized_view(K, V, 4, 32)
    assert np.array_equal(Kq[64:], K[64:]) and np.array_equal(Vq[64:], V[64:])
    assert not np.array_equal(Kq[:64], K[:64])
    Kq2, Vq2 = kq.quantized_view(K[:31], V[:31], 4, 32)          # no complete group: nothing is quantised
    assert np.array_equal(Kq2, K[:31]) and np.array_equal(Vq2, V[:31])


def test_decode_quant_tends_to_decode_as_the_grid_gets_fine_and_equals_it_without_complete_groups():
    d_h, r, n = 32, 16, 80
    rng = np.random.default_rng(9)
    U_K = [synth.orthonormal_basis(d_h, r, 1)]
    U_V = [synth.orthonormal_basis(d_h, r, 2)]
    L = orc.LayerOracle(1, 1, d_h, U_K, U_V)
    L.append_kv(rng.standard_normal((1, n, 1, d_h)), rng.standard_normal((1, n, 1, d_h)))
    q = rng.standard_normal((1, 1, 1, d_h))
    ref = L.decode(q)[(0, 0)]
    err = [np.abs(L.decode_quant(q, bits, 16)[(0, 0)] - ref).max() for bits in (3, 5, 8)]
    assert err[0] > err[1] > err[2] and err[2] < 5e-3 and err[0] > 1e-2
    assert np.array_equal(L.decode_quant(q, 4, 128)[(0, 0)], ref)    # 80 rows < one group of 128


def test_decode_quant_equals_loops_over_dequantised_rows():
    d_h, r, n, G = 16, 8, 40, 16
    rng = np.random.default_rng(21)
    U_K = [synth.orthonormal_basis(d_h, r, 3)]
    U_V = [synth.orthonormal_basis(d_h, r, 4)]
    L = orc.LayerOracle(1, 1, d_h, U_K, U_V)
    L.append_kv(rng.standard_normal((1, n, 1, d_h)), rng.standard_normal((1, n, 1, d_h)))
    q = rng.standard_normal((1, 1, 1, d_h))
    got = L.decode_quant(q, 4, G, lowrank_out=True)[(0, 0)]
    Kp, Vp = L.Kp[(0, 0)], L.Vp[(0, 0)]
    qp = q[0, 0, 0] @ U_K[0]
    # rows 0..31 through the grid (keys: scale per channel and 16 tokens; values: scale per token and 16 channels)
    w, o = [], np.zeros(r)
    Kh, Vh = np.zeros((n, r)), np.zeros((n, r))
    for j in range(n):
        for c in range(r):
            if j < 32:
                g0 = (j // G) * G
                sk = float(np.float16(np.float32(np.abs(Kp[g0:g0 + G, c].astype(np.float32)).max()) / np.float32(7)))
                sv = float(np.float16(np.float32(np.abs(Vp[j, :].astype(np.float32)).max()) / np.float32(7)))
                Kh[j, c] = max(-7, min(7, float(np.rint(np.float32(Kp[j, c]) / np.float32(sk))))) * sk
                Vh[j, c] = max(-7, min(7, float(np.rint(np.float32(Vp[j, c]) / np.float32(sv))))) * sv
            else:
                Kh[j, c], Vh[j, c] = Kp[j, c], Vp[j, c]
        w.append(math.exp(sum(qp[c] * Kh[j, c] for c in range(r)) / math.sqrt(d_h)))
    for j in range(n):
        o += w[j] / sum(w) * Vh[j]
    assert np.abs(got - o).max() < 1e-12
