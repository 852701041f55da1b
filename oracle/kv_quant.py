"""CPU oracle for the quantised rank-r KV cache (Section 5.3, "Eigen Attention with Quantization";
Table 8) -- TEST INFRASTRUCTURE ONLY.

Imported only by the tests, the smoke check and the benchmark's CPU legs; shares no code with the CUDA
sources and never sees a value they produced.

What the paper fixes: integer quantisation of the compressed keys and values at a precision of b bits
and a group size G; keys per channel (a group is G consecutive tokens of one channel), values per
token (a group is G consecutive channels of one token); and, through the cache sizes of Table 8, the
storage cost: every printed size equals elements * (b + 16/G) / 8 bytes, i.e. ONE 16-bit number of
metadata per group.  The reading taken here: that number is a half-precision scale and there is no
zero point, hence symmetric codes

    s = fp16( min(max|x| / (2^(b-1) - 1), 65504) ),    c = clip( rint(x / s), -(2^(b-1)-1), 2^(b-1)-1 ),    x^ = c * s .

The code is an integer decided by floating point, so the precision of that decision is part of the
definition: x is the stored (16-bit) cache value, the quotient max|x| / qmax and x / s are single
precision divisions, rint rounds half to even.  Everything downstream (de-quantisation, attention) is
float64.

Tokens that do not fill a group of G yet cannot be quantised per channel; they stay in the storage
format of the cache (keys and values alike) until their group is complete.

Parity pins (tests/test_oracle_quant_pins.py): the sizes printed in Table 8, the half-step error
bound, exact reproduction of data that already lies on a group's grid, the group axis (an outlier
planted in one channel / one token changes only that channel's / token's codes), brute-force loops.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def qmax_of(bits: int) -> int:
    assert 2 <= bits <= 8
    return 2 ** (bits - 1) - 1


def quantize_groups(x: np.ndarray, bits: int, group: int, axis: int):
    """Symmetric integer codes of `x` in groups of `group` consecutive entries along `axis` (the last
    group may be shorter).  Returns (codes int8 with x's shape, scales float16 with the group count
    along `axis`)."""
    qmax = np.float32(qmax_of(bits))
    x32 = np.moveaxis(np.asarray(x, dtype=np.float32), axis, -1)
    n = x32.shape[-1]
    n_groups = (n + group - 1) // group
    codes = np.zeros(x32.shape, dtype=np.int8)
    scales = np.zeros(x32.shape[:-1] + (n_groups,), dtype=np.float16)
    for g in range(n_groups):
        seg = x32[..., g * group:(g + 1) * group]
        amax = np.max(np.abs(seg), axis=-1)
        # single-precision quotient (kept inside the half-precision range), then round to half
        s16 = np.minimum(amax / qmax, np.float32(65504.0)).astype(np.float16)
        s32 = s16.astype(np.float32)[..., None]
        with np.errstate(divide="ignore", invalid="ignore"):
            c = np.where(s32 > 0, np.rint(seg / s32), np.float32(0))
        codes[..., g * group:(g + 1) * group] = np.clip(c, -qmax, qmax).astype(np.int8)
        scales[..., g] = s16
    return np.moveaxis(codes, -1, axis), np.moveaxis(scales, -1, axis)


def dequantize_groups(codes: np.ndarray, scales: np.ndarray, group: int, axis: int) -> np.ndarray:
    """x^ = c * s in float64 (exact: a small integer times a half-precision number)."""
    c = np.moveaxis(np.asarray(codes, dtype=F64), axis, -1)
    s = np.moveaxis(np.asarray(scales, dtype=F64), axis, -1)
    out = c * np.repeat(s, group, axis=-1)[..., :c.shape[-1]]
    return np.moveaxis(out, -1, axis)


def quantize_keys(Kp: np.ndarray, bits: int, group: int):
    """Per-channel: Kp is [tokens, channels], a group is `group` consecutive tokens of one channel."""
    return quantize_groups(Kp, bits, group, axis=0)


def quantize_values(Vp: np.ndarray, bits: int, group: int):
    """Per-token: Vp is [tokens, channels], a group is `group` consecutive channels of one token."""
    return quantize_groups(Vp, bits, group, axis=1)


def quantized_view(Kp: np.ndarray, Vp: np.ndarray, bits: int, group: int):
    """What a decode step sees of a cache of n rows: the floor(n / G) * G oldest rows de-quantised,
    the remaining rows as stored."""
    n = Kp.shape[0]
    nq = (n // group) * group
    kc, ks = quantize_keys(Kp[:nq], bits, group)
    vc, vs = quantize_values(Vp[:nq], bits, group)
    Kq = np.concatenate([dequantize_groups(kc, ks, group, 0), np.asarray(Kp[nq:], dtype=F64)], axis=0)
    Vq = np.concatenate([dequantize_groups(vc, vs, group, 1), np.asarray(Vp[nq:], dtype=F64)], axis=0)
    return Kq, Vq


def quant_cache_bytes(elements: int, bits: int, group: int) -> float:
    """Storage of `elements` cached numbers at `bits` bits plus one 16-bit scale per `group` of them
    (the accounting behind Table 8)."""
    return elements * (bits + 16.0 / group) / 8.0
