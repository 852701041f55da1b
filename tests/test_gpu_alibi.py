"""GPU parity of the ALiBi position bias (MPT models, Section 5.1) against the fp64 oracle, through the C ABI:
decode (fused step, separate launches, several splits of the key axis), the no-scratch decode, and the prefill
kernels that carry the bias."""
import numpy as np
import pytest
import torch

from helpers import OraclePair, assert_close, make_case, oracle_layer, storage_model, to_np
from paper_2408_05646_b200 import synth

pytestmark = pytest.mark.gpu
BF16, FP32 = torch.bfloat16, torch.float32


@pytest.fixture(scope="module")
def B():
    from paper_2408_05646_b200 import build
    build.build_library()
    from paper_2408_05646_b200 import binding
    return binding


@pytest.mark.parametrize("dtype,H,d,rk,rv,n", [
    (FP32, 4, 64, [32, 20, 64, 8], [16, 40, 64, 24], 700),
    (BF16, 8, 128, [80] * 8, [80] * 8, 3000),
    (BF16, 4, 128, [48, 64, 112, 128], [96, 80, 48, 128], 1037),
])
def test_decode_with_alibi_matches_oracle(B, dtype, H, d, rk, rv, n):
    B_ = 2
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n + 3, dtype, seed_cfg=131, T_q=4)
    slopes = synth.alibi_slopes(H)
    lay = B.EigenAttnLayer(B_, H, d, n + 8, dtype, U_k, U_v)
    lay.set_alibi(slopes)
    ref = OraclePair(B_, H, d, U_k, U_v, dtype, alibi_slopes=slopes)   # steep slopes: few rows carry the softmax
    lay.append_kv(k[:, :n], v[:, :n])
    ref.append_kv(to_np(k[:, :n]), to_np(v[:, :n]))
    tol = dict(fp32_rel=2e-5) if dtype == FP32 else {}
    out = lay.decode(q[:, :1])                                     # cache only, separate append
    assert_close(out, ref.decode_dense(to_np(q[:, :1])), dtype, "decode", **tol, plain_within=True)
    for step in range(3):                                          # fused append + attend
        o = lay.decode_step(q[:, step + 1:step + 2], k[:, n + step:n + step + 1], v[:, n + step:n + step + 1])
        ref.append_kv(to_np(k[:, n + step:n + step + 1]), to_np(v[:, n + step:n + step + 1]))
        assert_close(o, ref.decode_dense(to_np(q[:, step + 1:step + 2])), dtype, f"decode_step {step}", **tol, plain_within=True)
    expect = ref.decode_dense(to_np(q[:, :1]))
    for ctas, fused in ((1, 1), (37, 0), (148, 1)):                # split of the key axis must not matter
        lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        lay.set_option(B.EA_OPT_DECODE_FUSED, fused)
        assert_close(lay.decode(q[:, :1]), expect, dtype, f"decode ctas={ctas} fused={fused}", **tol, plain_within=True)
    assert_close(lay.decode_static(q[:, :1]), expect, dtype, "decode_static", **tol, plain_within=True)
    lay.set_alibi(None)                                            # back to the plain path
    plain = OraclePair(B_, H, d, U_k, U_v, dtype)
    plain.append_kv(to_np(k[:, :n + 3]), to_np(v[:, :n + 3]))
    assert_close(lay.decode(q[:, :1]), plain.decode_dense(to_np(q[:, :1])), dtype, "bias off", **tol, plain_within=True)
    lay.poll_status()


def test_alibi_dominates_at_long_range(B):
    """With a steep slope only the newest rows count: the far end of a long context must vanish exactly as in
    the oracle (biases of thousands in the exponent, rows of the first tiles underflow to zero)."""
    B_, H, d, n = 1, 2, 128, 20000
    U_k, U_v, q, k, v = make_case(B_, H, d, [80, 64], [80, 64], n, BF16, seed_cfg=133)
    slopes = [0.5, 2.0 ** -8]
    lay = B.EigenAttnLayer(B_, H, d, n, BF16, U_k, U_v)
    lay.set_alibi(slopes)
    lay.append_kv(k, v)
    ref = OraclePair(B_, H, d, U_k, U_v, BF16, alibi_slopes=slopes)
    ref.append_kv(to_np(k), to_np(v))
    assert_close(lay.decode(q), ref.decode_dense(to_np(q)), BF16, "long range", plain_within=True)


@pytest.mark.parametrize("dtype,H,d,rk,rv,T", [
    (FP32, 2, 64, [32, 20], [16, 40], 75),
    (BF16, 4, 128, [80, 48, 128, 64], [80, 112, 8, 64], 300),
])
def test_prefill_with_alibi_matches_oracle(B, dtype, H, d, rk, rv, T):
    B_ = 2
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, T, dtype, seed_cfg=137, T_q=T)
    slopes = synth.alibi_slopes(H)
    ref = OraclePair(B_, H, d, U_k, U_v, dtype, alibi_slopes=slopes)
    expect = ref.prefill_dense(to_np(q), to_np(k), to_np(v))
    for impl in ((0, 1) if dtype == FP32 else (0, 3, 1)):          # auto, single-tile tcgen05, CUDA cores
        lay = B.EigenAttnLayer(B_, H, d, T, dtype, U_k, U_v, max_prefill_tokens=T)
        lay.set_alibi(slopes)
        lay.set_option(B.EA_OPT_PREFILL_IMPL, impl)
        half = T // 2 + 3                                          # two chunks: positions continue from the cached length
        a = lay.prefill(q[:, :half], k[:, :half], v[:, :half])
        c = lay.prefill(q[:, half:], k[:, half:], v[:, half:])
        lay.poll_status()
        assert_close(torch.cat([a, c], dim=1), expect, dtype, f"prefill impl {impl}", plain_within=True)


def test_set_alibi_rejects_bad_slopes(B):
    U_k, U_v, q, k, v = make_case(1, 2, 64, [16, 16], [16, 16], 8, FP32, seed_cfg=139)
    lay = B.EigenAttnLayer(1, 2, 64, 8, FP32, U_k, U_v)
    for bad in ([-0.5, 0.1], [float("nan"), 0.1], [float("inf"), 0.1]):
        with pytest.raises(B.EigenAttnError):
            lay.set_alibi(bad)
