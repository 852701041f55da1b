"""The failure path and the memory guards.

A device-side wait that exceeds its bound must end the launch cleanly (no copy in flight, no hang), surface as
EA_ERR_TIMEOUT through eigen_attn_poll_status exactly once, and leave the handle usable.  The wait is made to run
out by the library's own test hook (EA_OPT_TEST_WAIT_GIVES_UP): one warp reports its first wait as run out on an
otherwise correct launch, so nothing on the GPU hangs or faults.

The guard regions that tests/conftest.py puts around every device buffer are themselves checked here on the CPU:
a byte planted outside a buffer must be reported."""
import numpy as np
import pytest
import torch

from conftest import GUARD_BYTES, GuardedAllocator
from helpers import assert_close, make_case, oracle_layer, to_np


@pytest.fixture(scope="module")
def B():
    from paper_2408_05646_b200 import build
    build.build_library()
    from paper_2408_05646_b200 import binding
    return binding


def test_guard_regions_report_a_planted_overrun():
    alloc = GuardedAllocator()
    a = alloc(1000, "cpu")
    b = alloc(4096, "cpu")
    a.fill_(7)
    b.fill_(9)                                   # writes inside the buffers leave the guards alone
    assert alloc.check() == []
    c = alloc(1000, "cpu")
    outer, n = alloc.live[0]
    assert c.data_ptr() == outer.data_ptr() + GUARD_BYTES and n == 1000
    outer[GUARD_BYTES + 1000] = 0                # one byte past the end
    outer[GUARD_BYTES - 3] = 1                   # three bytes before the start
    v = alloc.check()
    assert len(v) == 2 and "after" in v[1] and "before" in v[0] and "offset 0 " in v[1]


@pytest.mark.gpu
@pytest.mark.parametrize("entry", ["decode", "decode_step", "decode_static"])
def test_wait_that_runs_out_is_reported_once_and_the_handle_recovers(B, entry):
    dtype = torch.bfloat16
    B_, H, d, n = 2, 8, 128, 6000                # 16 units over 148 CTAs: every unit is split, counters in use
    rk = [80, 64, 48, 112, 80, 96, 128, 72]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rk, n + 1, dtype, seed_cfg=130)
    lay = B.EigenAttnLayer(B_, H, d, n + 1, dtype, U_k, U_v)
    lay.append_kv(k[:, :n], v[:, :n])
    ref = oracle_layer(B_, H, d, U_k, U_v)
    ref.append_kv(to_np(k[:, :n]), to_np(v[:, :n]))

    def call():
        if entry == "decode":
            return lay.decode(q)
        if entry == "decode_static":
            return lay.decode_static(q)
        out = lay.decode_step(q, k[:, n:], v[:, n:])
        lay.set_len(n)
        return out

    good = call()
    lay.poll_status()
    lay.set_option(B.EA_OPT_TEST_WAIT_GIVES_UP, 1)
    call()                                       # completes; its output is undefined
    with pytest.raises(B.EigenAttnError) as e:
        lay.poll_status()
    assert e.value.status == B.EA_ERR_TIMEOUT
    lay.poll_status()                            # reported once; the status word is clear again
    again = call()                               # the hook was one-shot, the arrival counters were cleared
    lay.poll_status()
    assert torch.equal(again, good)
    if entry == "decode_step":
        ref.append_kv(to_np(k[:, n:]), to_np(v[:, n:]))
    assert_close(again, ref.decode_dense(to_np(q)), dtype, f"{entry} after a reported timeout")
