"""GPU parity of grouped-query decode (the Section 5.1 models that share K/V heads) against the fp64 oracle,
through the C ABI; and against the library's own multi-head decode for group 1."""
import numpy as np
import pytest
import torch

from helpers import assert_close, make_case, oracle_layer, to_np
from paper_2408_05646_b200 import synth

pytestmark = pytest.mark.gpu
BF16, FP32 = torch.bfloat16, torch.float32


@pytest.fixture(scope="module")
def B():
    from paper_2408_05646_b200 import build
    build.build_library()
    from paper_2408_05646_b200 import binding
    return binding


def group_queries(B_, H, g, d, seed):
    W_q = synth.mixing_matrices(H * g, 16, d, seed, "W_Q")
    return synth.lowrank_rows(W_q, B_, 1, 0.1, seed, "Q", dtype=BF16, device="cuda:0")       # [B][1][H*g][d]


@pytest.mark.parametrize("H,g,d,rk,rv,n", [
    (2, 4, 128, [80, 80], [80, 80], 128),                           # exactly one tile
    (2, 4, 128, [80, 80], [80, 80], 1037),                          # several tiles, ragged tail
    (3, 8, 128, [48, 64, 128], [96, 80, 128], 700),                 # per-head ranks, widest rank
    (2, 2, 64, [24, 64], [56, 8], 517),                             # small d_head, ranks that are not multiples of 16
    (1, 16, 128, [80], [80], 17),                                   # largest group, shorter than a tile
    (2, 1, 128, [64, 64], [64, 64], 3000),                          # group 1 = multi-head attention
    (2, 5, 128, [80, 80], [80, 80], 9000),                          # a group that is not a power of two
    (3, 3, 64, [32, 64, 16], [16, 48, 64], 2100),                   # small d_head, ranks that are multiples of 16, per head
    (1, 12, 128, [128], [128], 1500),                               # more than 8 queries on the widest rank
])
@pytest.mark.parametrize("impl", [0, 1])               # 0: warp-level products where the ranks allow, 1: the tcgen05 kernel
def test_gqa_decode_matches_oracle(B, H, g, d, rk, rv, n, impl):
    B_ = 2
    U_k, U_v, _, k, v = make_case(B_, H, d, rk, rv, n, BF16, seed_cfg=161)
    q = group_queries(B_, H, g, d, 161)
    lay = B.EigenAttnLayer(B_, H, d, n + 4, BF16, U_k, U_v)
    lay.set_option(B.EA_OPT_GQA_IMPL, impl)
    lay.append_kv(k, v)
    ref = oracle_layer(B_, H, d, U_k, U_v)
    ref.append_kv(to_np(k), to_np(v))
    expect = ref.decode_gqa(to_np(q), g)
    assert_close(lay.decode_gqa(q, g), expect, BF16, "gqa decode")
    for ctas in (1, 7, 300, 1024):                                   # CTAs per unit must not matter
        lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        assert_close(lay.decode_gqa(q, g), expect, BF16, f"gqa decode ctas={ctas}")
    if g == 1:
        lay.set_option(B.EA_OPT_DECODE_CTAS, 0)
        assert float((lay.decode_gqa(q, 1).float() - lay.decode(q).float()).abs().max()) < 2e-2
    lay.poll_status()


@pytest.mark.parametrize("impl", [0, 1])
def test_gqa_peaked_attention_and_steps(B, impl):
    """Sharply peaked weights (queries scaled by 6) over several appended tokens: an error in a handful of rows
    or in one query of the group shows up here."""
    from helpers import OraclePair
    B_, H, g, d, n, steps = 2, 2, 4, 128, 300, 3
    rk, rv = [80, 48], [64, 80]
    U_k, U_v, _, k, v = make_case(B_, H, d, rk, rv, n + steps, BF16, seed_cfg=163)
    lay = B.EigenAttnLayer(B_, H, d, n + steps, BF16, U_k, U_v)
    lay.set_option(B.EA_OPT_GQA_IMPL, impl)
    lay.append_kv(k[:, :n], v[:, :n])
    ref = OraclePair(B_, H, d, U_k, U_v, BF16)
    ref.append_kv(to_np(k[:, :n]), to_np(v[:, :n]))
    for s in range(steps):
        q = (group_queries(B_, H, g, d, 170 + s).float() * 6.0).to(BF16)
        lay.append_kv(k[:, n + s:n + s + 1], v[:, n + s:n + s + 1])
        ref.append_kv(to_np(k[:, n + s:n + s + 1]), to_np(v[:, n + s:n + s + 1]))
        assert_close(lay.decode_gqa(q, g), ref.decode_gqa(to_np(q), g), BF16, f"gqa step {s}")
    lay.poll_status()


def test_gqa_rejections(B):
    U_k, U_v, q, k, v = make_case(1, 2, 64, [16, 16], [16, 16], 8, FP32, seed_cfg=165)
    lay32 = B.EigenAttnLayer(1, 2, 64, 8, FP32, U_k, U_v)
    lay32.append_kv(k, v)
    with pytest.raises(B.EigenAttnError):
        lay32.decode_gqa(q, 1)                                       # bf16 layers only
    U_k, U_v, q, k, v = make_case(1, 2, 64, [16, 16], [16, 16], 8, BF16, seed_cfg=165)
    lay = B.EigenAttnLayer(1, 2, 64, 8, BF16, U_k, U_v)
    with pytest.raises(B.EigenAttnError):
        lay.decode_gqa(q, 1)                                         # empty cache
    lay.append_kv(k, v)
    q17 = torch.zeros((1, 1, 2 * 17, 64), dtype=BF16, device="cuda")
    with pytest.raises(B.EigenAttnError):
        lay.decode_gqa(q17, 17)
    lay.set_alibi([0.5, 0.25])
    with pytest.raises(B.EigenAttnError):
        lay.decode_gqa(q, 1)


@pytest.mark.parametrize("H,g,d,rk,rv,n,base,interleaved", [
    (2, 4, 128, [80, 80], [80, 80], 1037, 10000.0, False),          # the 8B-class shape: several tiles, ragged tail
    (3, 2, 64, [24, 64, 40], [56, 8, 64], 517, 500000.0, True),     # small d_head, per-head ranks, interleaved pairs
    (1, 16, 128, [80], [80], 17, 10000.0, False),                   # largest group, shorter than a tile
    (2, 5, 128, [64, 112], [96, 48], 3000, 10000.0, True),          # a group that is not a power of two
])
def test_gqa_decode_with_rotary_embedding_matches_oracle(B, H, g, d, rk, rv, n, base, interleaved):
    """Section 4.3 for grouped queries (the Llama models that share K/V heads also rotate their keys): every query
    head against its K/V head's lifted, rotated keys."""
    from helpers import OraclePair
    B_ = 2
    U_k, U_v, _, k, v = make_case(B_, H, d, rk, rv, n + 1, BF16, seed_cfg=167)
    lay = B.EigenAttnLayer(B_, H, d, n + 4, BF16, U_k, U_v)
    lay.set_rope(base, interleaved)
    lay.append_kv(k[:, :n], v[:, :n])
    ref = OraclePair(B_, H, d, U_k, U_v, BF16, rope={"base": base, "interleaved": interleaved})
    ref.append_kv(to_np(k[:, :n]), to_np(v[:, :n]))
    for step, scale in enumerate((1.0, 4.0)):                        # the second step with peaked weights
        if step:
            lay.append_kv(k[:, n:n + 1], v[:, n:n + 1])
            ref.append_kv(to_np(k[:, n:n + 1]), to_np(v[:, n:n + 1]))
        q = (group_queries(B_, H, g, d, 180 + step).float() * scale).to(BF16)
        expect = ref.decode_gqa(to_np(q), g)
        for ctas in (0, 1, 7, 300):                                  # CTAs per unit must not matter
            lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
            assert_close(lay.decode_gqa(q, g), expect, BF16, f"gqa rope decode step {step} ctas={ctas}")
    lay.set_option(B.EA_OPT_DECODE_CTAS, 0)                          # one query head per K/V head: the multi-head call
    q1 = q[:, :, ::g].contiguous()
    assert torch.equal(lay.decode_gqa(q1, 1), lay.decode(q1))
    lay.poll_status()
