"""GPU parity of the RoPE variant of the generation phase (Section 4.3) against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from helpers import assert_close, make_case, oracle_layer, to_np
from oracle import eigen_attention as orc

pytestmark = pytest.mark.gpu
BF16, FP32 = torch.bfloat16, torch.float32


@pytest.fixture(scope="module")
def B():
    from paper_2408_05646_b200 import build
    build.build_library()
    from paper_2408_05646_b200 import binding
    return binding


def rope_oracle(B_, H, d, U_k, U_v, base, interleaved):
    return orc.LayerOracle(B_, H, d, U_k, U_v, rope={"base": base, "interleaved": interleaved})


@pytest.mark.parametrize("H,d,rk,rv,n,base,interleaved", [
    (2, 128, [80, 80], [80, 80], 128, 10000.0, False),              # exactly one tile
    (2, 128, [80, 80], [80, 80], 1037, 10000.0, False),             # several tiles, ragged tail
    (4, 128, [48, 64, 112, 128], [96, 80, 48, 128], 700, 10000.0, True),
    (3, 64, [24, 64, 40], [56, 8, 64], 517, 500000.0, False),       # small d_head, ranks that are not multiples of 16
    (1, 128, [80], [80], 17, 10000.0, True),                        # shorter than a tile
    (2, 128, [64, 64], [64, 64], 9000, 10000.0, False),             # positions in the thousands
])
def test_rope_decode_matches_oracle(B, H, d, rk, rv, n, base, interleaved):
    B_ = 2
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n, BF16, seed_cfg=151)
    lay = B.EigenAttnLayer(B_, H, d, n + 4, BF16, U_k, U_v)
    lay.set_rope(base, interleaved)
    lay.append_kv(k, v)
    ref = rope_oracle(B_, H, d, U_k, U_v, base, interleaved)
    ref.append_kv(to_np(k), to_np(v))
    expect = ref.decode_dense(to_np(q))
    assert_close(lay.decode(q), expect, BF16, "rope decode")
    for ctas in (1, 7, 300, 1024):                                   # CTAs per unit must not matter
        lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        assert_close(lay.decode(q), expect, BF16, f"rope decode ctas={ctas}")
    lay.poll_status()


@pytest.mark.parametrize("interleaved", [False, True])
def test_rope_decode_with_peaked_attention(B, interleaved):
    """Queries scaled by 4: a handful of positions carry the softmax, so one wrongly rotated or wrongly lifted row
    (a tile boundary, the ragged tail, a stale staging buffer) is not averaged away.  Heads of unequal widths are
    streamed one after the other; any number of CTAs per unit must agree."""
    from helpers import OraclePair
    B_, H, d, n = 2, 4, 128, 1037
    rk, rv = [48, 80, 64, 112], [96, 64, 80, 32]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n, BF16, seed_cfg=157, q_scale=4.0)
    lay = B.EigenAttnLayer(B_, H, d, n, BF16, U_k, U_v)
    lay.set_rope(10000.0, interleaved)
    lay.append_kv(k, v)
    ref = OraclePair(B_, H, d, U_k, U_v, BF16, rope={"base": 10000.0, "interleaved": interleaved})
    ref.append_kv(to_np(k), to_np(v))
    expect = ref.decode_dense(to_np(q))
    weights_on_few_rows = np.abs(expect.plain).max() > 0.5          # a diffuse average of ~1000 rows stays far below
    assert weights_on_few_rows
    for ctas in (0, 1, 9, 300):
        lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        assert_close(lay.decode(q), expect, BF16, f"peaked rope decode ctas={ctas}", plain_within=True)
    lay.poll_status()


def test_rope_decode_steps_lowrank_output_and_switching_off(B):
    B_, H, d, n, steps = 2, 2, 128, 300, 5
    rk, rv = [80, 48], [64, 80]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n + steps, BF16, seed_cfg=153, T_q=steps)
    lay = B.EigenAttnLayer(B_, H, d, n + steps, BF16, U_k, U_v)
    lay.set_rope(10000.0)
    lay.append_kv(k[:, :n], v[:, :n])
    ref = rope_oracle(B_, H, d, U_k, U_v, 10000.0, False)
    ref.append_kv(to_np(k[:, :n]), to_np(v[:, :n]))
    for s in range(steps):                                           # append + decode, positions advance by one
        o = lay.decode_step(q[:, s:s + 1], k[:, n + s:n + s + 1], v[:, n + s:n + s + 1])
        ref.append_kv(to_np(k[:, n + s:n + s + 1]), to_np(v[:, n + s:n + s + 1]))
        assert_close(o, ref.decode_dense(to_np(q[:, s:s + 1])), BF16, f"rope step {s}")
    low = lay.decode(q[:, :1], out_lowrank=True)
    res = ref.decode(to_np(q[:, :1]), lowrank_out=True)
    for b in range(B_):
        for h in range(H):
            assert_close(low[b, 0, lay.offs_v[h]:lay.offs_v[h] + rv[h]], res[(b, h)], BF16, "rope lowrank out")
    lay.set_rope(0.0)                                                # back to the plain path
    plain = oracle_layer(B_, H, d, U_k, U_v)
    plain.append_kv(to_np(k), to_np(v))
    assert_close(lay.decode(q[:, :1]), plain.decode_dense(to_np(q[:, :1])), BF16, "rope off")
    lay.poll_status()


@pytest.mark.parametrize("H,d,rk,rv,T,base,interleaved", [
    (2, 128, [80, 48], [64, 80], 300, 10000.0, False),
    (3, 64, [24, 64, 40], [56, 8, 64], 150, 500000.0, True),
    (1, 128, [128], [128], 77, 10000.0, False),
])
def test_rope_prefill_matches_oracle_and_feeds_decode(B, H, d, rk, rv, T, base, interleaved):
    """A layer with rotary embedding runs prompt -> generation through the library: the prompt in two chunks
    (positions continue from the cached length), then decode steps over the cache the prompt left."""
    B_, steps = 2, 2
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, T + steps, BF16, seed_cfg=159, T_q=T + steps)
    lay = B.EigenAttnLayer(B_, H, d, T + steps, BF16, U_k, U_v, max_prefill_tokens=T)
    lay.set_rope(base, interleaved)
    ref = rope_oracle(B_, H, d, U_k, U_v, base, interleaved)
    cut = T // 2 + 5
    a = lay.prefill(q[:, :cut].contiguous(), k[:, :cut].contiguous(), v[:, :cut].contiguous())
    c = lay.prefill(q[:, cut:T].contiguous(), k[:, cut:T].contiguous(), v[:, cut:T].contiguous())
    lay.poll_status()
    expect = ref.prefill_dense(to_np(q[:, :T]), to_np(k[:, :T]), to_np(v[:, :T]))
    assert_close(torch.cat([a, c], dim=1), expect, BF16, "rope prefill")
    low = lay_low = None
    for s in range(steps):
        t = T + s
        o = lay.decode_step(q[:, t:t + 1], k[:, t:t + 1], v[:, t:t + 1])
        ref.append_kv(to_np(k[:, t:t + 1]), to_np(v[:, t:t + 1]))
        assert_close(o, ref.decode_dense(to_np(q[:, t:t + 1])), BF16, f"decode step {s} after a rope prefill")
    # rank-space output of the prompt
    lay2 = B.EigenAttnLayer(B_, H, d, T, BF16, U_k, U_v, max_prefill_tokens=T)
    lay2.set_rope(base, interleaved)
    low = lay2.prefill(q[:, :T].contiguous(), k[:, :T].contiguous(), v[:, :T].contiguous(), out_lowrank=True)
    for b in range(B_):
        for h in range(H):
            back = to_np(low[b, :, lay2.offs_v[h]:lay2.offs_v[h] + rv[h]]) @ U_v[h].astype(np.float64).T
            assert_close(torch.from_numpy(back), expect[b, :, h], BF16, "rope prefill, rank-space output")
    lay.poll_status()


@pytest.mark.parametrize("H,d,rk,rv,T,base,interleaved", [
    (2, 128, [80, 48], [64, 80], 700, 10000.0, False),              # several query blocks and key tiles
    (3, 64, [24, 64, 40], [56, 8, 64], 150, 500000.0, True),
    (1, 128, [128], [128], 77, 10000.0, False),
    (2, 80, [40, 80], [80, 16], 333, 10000.0, True),                # d_head that is not a multiple of 64
])
def test_rope_prefill_on_the_tensor_cores(B, H, d, rk, rv, T, base, interleaved):
    """The same prompt path with the scratch for rotated queries and lifted, rotated keys (a descriptor flag): the
    warp-specialised tensor-core kernel, forced by option so that a silent fall back cannot pass.  Two chunks
    (positions and keys continue from the cached rows), batches of unequal lengths, then generation; and the
    CUDA-core kernel of a layer without the scratch must agree within the 16-bit roundings of the two."""
    B_, steps = 2, 2
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, T + steps, BF16, seed_cfg=191, T_q=T + steps)
    q = (q.float() * 0.5).to(BF16)
    lay = B.EigenAttnLayer(B_, H, d, T + steps, BF16, U_k, U_v, max_prefill_tokens=T, rope_prompt_scratch=True)
    lay.set_rope(base, interleaved)
    lay.set_option(B.EA_OPT_PREFILL_IMPL, 2)
    ref = rope_oracle(B_, H, d, U_k, U_v, base, interleaved)
    cut = T // 2 + 5
    a = lay.prefill(q[:, :cut].contiguous(), k[:, :cut].contiguous(), v[:, :cut].contiguous())
    c = lay.prefill(q[:, cut:T].contiguous(), k[:, cut:T].contiguous(), v[:, cut:T].contiguous())
    lay.poll_status()
    expect = ref.prefill_dense(to_np(q[:, :T]), to_np(k[:, :T]), to_np(v[:, :T]))
    got = torch.cat([a, c], dim=1)
    assert_close(got, expect, BF16, "rope prefill on the tensor cores")
    slow = B.EigenAttnLayer(B_, H, d, T + steps, BF16, U_k, U_v, max_prefill_tokens=T)
    slow.set_rope(base, interleaved)
    other = slow.prefill(q[:, :T].contiguous(), k[:, :T].contiguous(), v[:, :T].contiguous())
    assert float((other.float() - got.float()).abs().max()) < 2e-2
    lay.set_option(B.EA_OPT_PREFILL_IMPL, 0)
    for s in range(steps):
        t = T + s
        o = lay.decode_step(q[:, t:t + 1], k[:, t:t + 1], v[:, t:t + 1])
        ref.append_kv(to_np(k[:, t:t + 1]), to_np(v[:, t:t + 1]))
        assert_close(o, ref.decode_dense(to_np(q[:, t:t + 1])), BF16, f"decode step {s} after the prompt")
    # a prompt that does not fit the scratch any more falls back (automatic) or is refused (forced)
    lay.set_len(T)
    lay.set_option(B.EA_OPT_PREFILL_IMPL, 2)
    with pytest.raises(B.EigenAttnError) as e:
        lay.prefill(q[:, :2].contiguous(), k[:, :2].contiguous(), v[:, :2].contiguous())
    assert e.value.status == B.EA_ERR_UNSUPPORTED and lay.len == T
    lay.set_option(B.EA_OPT_PREFILL_IMPL, 0)
    tail = lay.prefill(q[:, T:T + 2].contiguous(), k[:, T:T + 2].contiguous(), v[:, T:T + 2].contiguous())
    full = rope_oracle(B_, H, d, U_k, U_v, base, interleaved)
    assert_close(tail, full.prefill_dense(to_np(q[:, :T + 2]), to_np(k[:, :T + 2]), to_np(v[:, :T + 2]))[:, T:], BF16,
                 "chunk past the scratch (CUDA-core kernel)")
    lay.poll_status()


def test_rope_rejections(B):
    U_k, U_v, q, k, v = make_case(1, 2, 64, [16, 16], [16, 16], 8, FP32, seed_cfg=155)
    lay32 = B.EigenAttnLayer(1, 2, 64, 8, FP32, U_k, U_v)
    with pytest.raises(B.EigenAttnError):
        lay32.set_rope(10000.0)                                      # bf16 layers only
    U_k, U_v, q, k, v = make_case(1, 2, 64, [16, 16], [16, 16], 8, BF16, seed_cfg=155)
    lay = B.EigenAttnLayer(1, 2, 64, 8, BF16, U_k, U_v, max_prefill_tokens=8)
    with pytest.raises(B.EigenAttnError):
        lay.set_rope(0.5)
    lay.set_rope(10000.0)
    lay.append_kv(k, v)
    with pytest.raises(B.EigenAttnError):
        lay.decode_static(q)
    with pytest.raises(B.EigenAttnError):
        lay.set_alibi([0.5, 0.25])
    qp = torch.zeros((1, 1, lay.offs_k[-1]), dtype=BF16, device="cuda")
    with pytest.raises(B.EigenAttnError):
        lay.decode(qp, q_preprojected=True)
