"""CPU-only checks of the C ABI: the library loads, exports every declared symbol, and its host-side
size arithmetic and argument validation behave as the header states (no GPU work is issued)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2408_05646_b200 import build
    build.build_library()
    from paper_2408_05646_b200 import binding as b
    return b


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "eigen_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(eigen_attn_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(binding):
    names = declared_symbols()
    assert len(names) >= 18
    raw = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), n
        assert n in binding.SYMBOLS, f"{n} is declared but not bound"
    assert set(binding.SYMBOLS) == set(names)
    assert binding.lib.eigen_attn_version() >= 100


def test_cache_bytes_matches_the_rank_r_cache_formula(binding):
    # Llama-2-7B-shaped layer, r = 80 of 128, bf16: 2 * B * n * sum(r) * 2 bytes (Table 1: 2.n.r per layer)
    B, H, n = 16, 32, 32768
    cb, wb = binding.cache_bytes(B, H, 128, n, binding.EA_BF16, [80] * H)
    assert cb == 2 * B * n * H * 80 * 2 == 5 * 2**30
    assert wb < 64 * 2**20
    # ranks are padded to multiples of 8; K and V ranks may differ
    cb2, _ = binding.cache_bytes(1, 2, 64, 100, binding.EA_FP32, [5, 9], [16, 3])
    assert cb2 >= 100 * 4 * (8 + 16 + 16 + 8)
    assert cb2 < 100 * 4 * (8 + 16 + 16 + 8) + 4 * 256


@pytest.mark.parametrize("kwargs,status", [
    (dict(batch=0), "EA_ERR_SHAPE"), (dict(d_head=12), "EA_ERR_SHAPE"), (dict(d_head=256), "EA_ERR_SHAPE"),
    (dict(n_heads=257), "EA_ERR_SHAPE"), (dict(dtype=7), "EA_ERR_INVALID_ARG"),
    (dict(r=0), "EA_ERR_SHAPE"), (dict(r=65), "EA_ERR_SHAPE"), (dict(max_prefill=1000), "EA_ERR_SHAPE"),
])
def test_bad_descriptors_are_rejected_on_the_host(binding, kwargs, status):
    a = dict(batch=1, n_heads=2, d_head=64, n_max=128, dtype=binding.EA_BF16, r=32, max_prefill=0)
    a.update(kwargs)
    with pytest.raises(binding.EigenAttnError) as e:
        binding.cache_bytes(a["batch"], a["n_heads"], a["d_head"], a["n_max"], a["dtype"],
                            [a["r"]] * max(a["n_heads"], 1), None, a["max_prefill"])
    assert binding.STATUS_NAMES[e.value.status] == status


def test_null_arguments(binding):
    lib = binding.lib
    assert lib.eigen_attn_cache_bytes(None, None, None) == binding.EA_ERR_INVALID_ARG
    assert lib.eigen_attn_get_len(None, None) == binding.EA_ERR_INVALID_ARG
    assert lib.eigen_attn_decode(None, None, 0, None, 0, 0, None) == binding.EA_ERR_INVALID_ARG
    assert lib.eigen_attn_last_error(None) == b"null handle"
    lib.eigen_attn_destroy(None)
