"""eigen_attn_decode_static: the decode call for users who cannot give it scratch memory.

Some callers of this library may not obtain device memory once they are running (an engine plugin
with a frozen memory plan, a latency-critical loop that cannot afford cudaMalloc's device-wide
synchronisation).  For them the library keeps the split-KV partial results in an array of its own.
This file checks, through the C ABI, that the variant returns what eigen_attn_decode returns, twice in
a row (the array is shared and keeps the previous call's contents), and that it refuses layers that
do not fit.  It is collected last on purpose, and must also pass when run alone."""
import pytest
import torch

from helpers import assert_close, make_case, oracle_layer, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2408_05646_b200 import build
    build.build_library()
    from paper_2408_05646_b200 import binding
    return binding


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_static_scratch_decode_matches_workspace_decode_twice(B, dtype):
    B_, H, d, n = 2, 6, 128, 5000
    rk, rv = [80, 64, 48, 112, 33, 128], [80, 96, 128, 24, 64, 8]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n, dtype, seed_cfg=120, T_q=2)
    lay = B.EigenAttnLayer(B_, H, d, n, dtype, U_k, U_v)
    lay.append_kv(k, v)
    ref = oracle_layer(B_, H, d, U_k, U_v)
    ref.append_kv(to_np(k), to_np(v))
    for call in range(2):                       # second call: the array still holds the first call's partials
        qq = q[:, call:call + 1]
        lay.set_len(n - 37 * call)              # a different split plan, so different slots are (re)used
        want = lay.decode(qq)
        out = torch.empty_like(want)
        got = lay.decode_static(qq, out=out)
        lay.poll_status()
        assert torch.equal(got, want), f"call {call}: differs from eigen_attn_decode"
        if call == 0:
            assert_close(got, ref.decode_dense(to_np(qq)), dtype, "static decode vs oracle")


def test_static_scratch_decode_with_peaked_attention(B):
    """Queries scaled by 6: a few rows carry the softmax, so a partial read from the wrong slot of the built-in
    array, or a slot left over from the previous call, would show.  Checked against the oracle, for several split
    plans in a row (each leaves its partials behind for the next)."""
    from helpers import OraclePair
    dtype = torch.bfloat16
    B_, H, d, n = 2, 6, 128, 1037
    rk, rv = [48, 64, 80, 96, 64, 48], [96, 80, 64, 48, 80, 96]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n, dtype, seed_cfg=122, q_scale=6.0)
    lay = B.EigenAttnLayer(B_, H, d, n, dtype, U_k, U_v)
    lay.append_kv(k, v)
    ref = OraclePair(B_, H, d, U_k, U_v, dtype)
    ref.append_kv(to_np(k), to_np(v))
    expect = ref.decode_dense(to_np(q))
    for ctas, fused in ((0, 1), (5, 1), (37, 0), (148, 1), (2, 1)):
        lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        lay.set_option(B.EA_OPT_DECODE_FUSED, fused)
        assert_close(lay.decode_static(q), expect, dtype, f"peaked static decode ctas={ctas} fused={fused}")
    lay.poll_status()


def test_static_scratch_rejects_layers_beyond_its_limit(B):
    # (batch*heads + CTAs) * (4 + widest rp_v) must stay within 270336 floats
    B_, H, d, n = 64, 32, 128, 4
    U_k, U_v, q, k, v = make_case(B_, H, d, [128] * H, [128] * H, n, torch.bfloat16, seed_cfg=121)
    lay = B.EigenAttnLayer(B_, H, d, n, torch.bfloat16, U_k, U_v)
    lay.append_kv(k, v)
    lay.decode(q)                               # the workspace path takes it
    with pytest.raises(B.EigenAttnError) as e:
        lay.decode_static(q)
    assert e.value.status == B.EA_ERR_CAPACITY and "built-in scratch" in str(e.value)
    lay.poll_status()
