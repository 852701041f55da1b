"""GPU parity of the paged rank-r cache: a page table changes where a sequence's rows live and nothing else, so a
paged layer must return what the contiguous layer returns (bit for bit: same kernels, same tiles), its pool must hold
each sequence's rows where the oracle's address arithmetic says, and both must agree with the fp64 oracle."""
import numpy as np
import pytest
import torch

from helpers import OraclePair, assert_close, make_case, oracle_layer, to_np
from oracle import eigen_attention as orc
from paper_2408_05646_b200 import synth

pytestmark = pytest.mark.gpu
BF16, FP32 = torch.bfloat16, torch.float32


@pytest.fixture(scope="module")
def B():
    from paper_2408_05646_b200 import build
    build.build_library()
    from paper_2408_05646_b200 import binding
    return binding


def pool_of(lay, head, which):
    """A head's slab as the pool of physical rows [batch * n_max, rp]."""
    x = lay.cache_rows(head, which)
    return x.reshape(-1, x.shape[-1])


@pytest.mark.parametrize("dtype,page_rows", [(BF16, 128), (FP32, 256)])
def test_paged_layer_equals_contiguous_layer(B, dtype, page_rows):
    B_, H, d, n_max = 3, 4, 128, 1024
    rk, rv = [80, 48, 112, 64], [64, 96, 80, 128]
    n, steps = 700, 3
    U_k, U_v, qq, k, v = make_case(B_, H, d, rk, rv, n + steps, dtype, seed_cfg=181, q_scale=4.0, T_q=256 + steps + 1)
    q_prompt, q = (qq[:, :256].float() / 4.0).to(dtype), qq[:, 256:]   # peaked weights for the decode calls only
    flat = B.EigenAttnLayer(B_, H, d, n_max, dtype, U_k, U_v, max_prefill_tokens=256)
    paged = B.EigenAttnLayer(B_, H, d, n_max, dtype, U_k, U_v, max_prefill_tokens=256)
    pool_pages = B_ * n_max // page_rows
    per_seq = n_max // page_rows
    perm = np.random.default_rng(5).permutation(pool_pages)
    table = [[int(x) for x in perm[b * per_seq:(b + 1) * per_seq]] for b in range(B_)]   # pages shuffled across sequences
    paged.set_page_table(table, page_rows)
    flat.set_option(B.EA_OPT_PREFILL_IMPL, 1)         # the CUDA-core prefill, as the paged layer runs it: identical cache rows
    flat.set_option(B.EA_OPT_DECODE_MIN_COPY_BYTES, 0)   # one tile per ring slot, as with pages: the same rows meet in the same thread
    ref = OraclePair(B_, H, d, U_k, U_v, dtype)
    # prompt of 256 tokens through prefill (two chunks), the rest appended, then fused decode steps
    outs = []
    for lay in (flat, paged):
        a = lay.prefill(q_prompt[:, :200].contiguous(), k[:, :200].contiguous(), v[:, :200].contiguous())
        c = lay.prefill(q_prompt[:, 200:].contiguous(), k[:, 200:256].contiguous(), v[:, 200:256].contiguous())
        lay.append_kv(k[:, 256:n], v[:, 256:n])
        outs.append([a, c])
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])   # same kernels on both layers
    want_p = ref.prefill_dense(to_np(q_prompt), to_np(k[:, :256]), to_np(v[:, :256]))
    for o in outs:                                    # the prompt's outputs, both layers
        assert_close(torch.cat(o, dim=1), want_p, dtype, "prefill", **(dict(fp32_rel=2e-4) if dtype == FP32 else {}))
    ref.append_kv(to_np(k[:, 256:n]), to_np(v[:, 256:n]))
    tol = dict(fp32_rel=2e-4) if dtype == FP32 else {}
    for ctas, fused in ((0, 1), (1, 1), (7, 0), (148, 1)):
        for lay in (flat, paged):
            lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
            lay.set_option(B.EA_OPT_DECODE_FUSED, fused)
        want = flat.decode(q[:, :1])
        assert torch.equal(paged.decode(q[:, :1]), want), f"paged decode differs, ctas={ctas} fused={fused}"
        assert torch.equal(paged.decode_static(q[:, :1]), want)
        assert_close(want, ref.decode_dense(to_np(q[:, :1])), dtype, f"decode ctas={ctas}", **tol)
    for s in range(steps):
        t = n + s
        o_f = flat.decode_step(q[:, s + 1:s + 2], k[:, t:t + 1], v[:, t:t + 1])
        o_p = paged.decode_step(q[:, s + 1:s + 2], k[:, t:t + 1], v[:, t:t + 1])
        ref.append_kv(to_np(k[:, t:t + 1]), to_np(v[:, t:t + 1]))
        assert torch.equal(o_p, o_f), f"paged decode_step {s} differs"
        assert_close(o_p, ref.decode_dense(to_np(q[:, s + 1:s + 2])), dtype, f"paged decode_step {s}", **tol)
    paged.poll_status(); flat.poll_status()
    # the pool holds every sequence's rows where the oracle's address arithmetic puts them
    for h in (0, H - 1):
        for which in "kv":
            pool = to_np(pool_of(paged, h, which))
            rows = to_np(flat.cache_rows(h, which))
            for b in range(B_):
                got = orc.paged_gather(pool, table[b], page_rows, n + steps)
                assert np.array_equal(got, rows[b, :n + steps]), (h, which, b)


def test_a_sequence_can_outgrow_n_max_on_pages_others_leave_free(B):
    """Two sequences share a pool of 8 pages: the first maps 7 (896 rows, beyond n_max = 512), the second 1.  The
    second is rewound after every append so that it never needs a second page.  Both decode against the oracle."""
    B_, H, d, n_max = 2, 2, 128, 512
    rk, rv = [80, 64], [64, 80]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, 880, BF16, seed_cfg=183)
    lay = B.EigenAttnLayer(B_, H, d, n_max, BF16, U_k, U_v)
    lay.set_page_table([[3, 0, 6, 1, 7, 2, 5], [4, -1, -1, -1, -1, -1, -1]], 128)
    short = 20
    lay.append_kv(k[:, :short], v[:, :short])
    lens = [short, short]
    for c0 in range(short, 880, 100):
        c1 = min(880, c0 + 100)
        lay.set_lens([lens[0], short])                 # sequence 1 back to its first rows; the new rows land behind them
        lay.append_kv(k[:, c0:c1], v[:, c0:c1])
        lens = [lens[0] + (c1 - c0), short + (c1 - c0)]
    assert lay.lens() == lens and lens[0] == 880 > n_max
    out = lay.decode(q)
    lay.poll_status()
    for b, kk, vv in ((0, k[0, :880], v[0, :880]),
                      (1, torch.cat([k[1, :short], k[1, 820:880]]), torch.cat([v[1, :short], v[1, 820:880]]))):
        r = oracle_layer(1, H, d, U_k, U_v)
        r.append_kv(to_np(kk)[None], to_np(vv)[None])
        assert_close(out[b:b + 1], r.decode_dense(to_np(q[b:b + 1])), BF16, f"sequence {b}")
    with pytest.raises(B.EigenAttnError) as e:         # sequence 1 has one page: 128 rows
        lay.set_lens([880, 129])
    assert e.value.status == B.EA_ERR_CAPACITY
    lay.set_lens([880, 128])
    with pytest.raises(B.EigenAttnError) as e:         # its next row has no page
        lay.append_kv(k[:, :1], v[:, :1])
    assert e.value.status == B.EA_ERR_CAPACITY


def test_page_table_argument_checks(B):
    B_, H, d, n_max = 2, 1, 64, 256
    U_k, U_v, q, k, v = make_case(B_, H, d, [32], [32], 8, BF16, seed_cfg=185)
    lay = B.EigenAttnLayer(B_, H, d, n_max, BF16, U_k, U_v)
    for table, rows in (([[0, 1], [1, 2]], 128),       # a physical page mapped twice
                        ([[0, 4], [1, 2]], 128),       # outside the pool of 4 pages
                        ([[-1, 0], [1, 2]], 128),      # a mapped page behind an unmapped one
                        ([[0, 1], [2, 3]], 96),        # not a power of two
                        ([[0, 1], [2, 3]], 64)):       # smaller than a tile
        with pytest.raises(B.EigenAttnError):
            lay.set_page_table(table, rows)
    lay.set_page_table([[2, 3], [0, 1]], 128)
    lay.append_kv(k, v)
    with pytest.raises(B.EigenAttnError) as e:
        lay.quant_attach(4, 32)
    assert e.value.status == B.EA_ERR_UNSUPPORTED
    # grouped queries follow the page table in the warp-level kernel; the tcgen05 kernel reads contiguous slabs only
    assert float((lay.decode_gqa(q, 1).float() - lay.decode(q).float()).abs().max()) < 2e-2
    lay.set_option(B.EA_OPT_GQA_IMPL, 1)
    with pytest.raises(B.EigenAttnError) as e:
        lay.decode_gqa(q, 1)
    assert e.value.status == B.EA_ERR_UNSUPPORTED
    lay.set_option(B.EA_OPT_GQA_IMPL, 0)
    with pytest.raises(B.EigenAttnError) as e:         # the rows held must stay mapped
        lay.set_page_table([[2, -1], [-1, -1]], 128)
    assert e.value.status == B.EA_ERR_CAPACITY
    lay.set_page_table(None)                           # contiguous again
    lay.poll_status()


@pytest.mark.parametrize("interleaved", [False, True])
def test_paged_layer_with_rotary_embedding_equals_contiguous_layer(B, interleaved):
    """Section 4.3 over a paged cache: prompt, generation steps and grouped queries of a paged layer equal those of
    the contiguous layer bit for bit (same kernels, same tiles, other addresses) and both agree with the oracle."""
    B_, H, d, n_max, page_rows = 3, 3, 128, 1024, 256
    rk, rv = [80, 48, 112], [64, 96, 80]
    n, steps, g = 700, 2, 2
    U_k, U_v, qq, k, v = make_case(B_, H, d, rk, rv, n + steps, BF16, seed_cfg=187, T_q=200 + steps + 1)
    q_prompt, q = (qq[:, :200].float() / 4.0).to(BF16), qq[:, 200:]
    rope = {"base": 10000.0, "interleaved": interleaved}
    flat = B.EigenAttnLayer(B_, H, d, n_max, BF16, U_k, U_v, max_prefill_tokens=200)
    paged = B.EigenAttnLayer(B_, H, d, n_max, BF16, U_k, U_v, max_prefill_tokens=200)
    per_seq = n_max // page_rows
    perm = np.random.default_rng(7).permutation(B_ * per_seq)
    paged.set_page_table([[int(x) for x in perm[b * per_seq:(b + 1) * per_seq]] for b in range(B_)], page_rows)
    ref = OraclePair(B_, H, d, U_k, U_v, BF16, rope=rope)
    outs = []
    for lay in (flat, paged):
        lay.set_rope(rope["base"], interleaved)
        outs.append(lay.prefill(q_prompt, k[:, :200].contiguous(), v[:, :200].contiguous()))
        lay.append_kv(k[:, 200:n], v[:, 200:n])
    assert torch.equal(outs[0], outs[1])
    assert_close(outs[1], ref.prefill_dense(to_np(q_prompt), to_np(k[:, :200]), to_np(v[:, :200])), BF16, "rope prefill, paged")
    ref.append_kv(to_np(k[:, 200:n]), to_np(v[:, 200:n]))
    for ctas in (0, 1, 5):
        for lay in (flat, paged):
            lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        want = flat.decode(q[:, :1])
        assert torch.equal(paged.decode(q[:, :1]), want), f"paged rope decode differs, ctas={ctas}"
        assert_close(want, ref.decode_dense(to_np(q[:, :1])), BF16, f"rope decode ctas={ctas}")
    W_q = synth.mixing_matrices(H * g, 16, d, 188, "W_Q")
    qg = synth.lowrank_rows(W_q, B_, 1, 0.1, 188, "Q", dtype=BF16, device="cuda:0")
    want = flat.decode_gqa(qg, g)
    assert torch.equal(paged.decode_gqa(qg, g), want)
    assert_close(want, ref.decode_gqa(to_np(qg), g), BF16, "grouped queries, rope, paged")
    for s in range(steps):
        t = n + s
        o_f = flat.decode_step(q[:, s + 1:s + 2], k[:, t:t + 1], v[:, t:t + 1])
        o_p = paged.decode_step(q[:, s + 1:s + 2], k[:, t:t + 1], v[:, t:t + 1])
        ref.append_kv(to_np(k[:, t:t + 1]), to_np(v[:, t:t + 1]))
        assert torch.equal(o_p, o_f), f"paged rope decode_step {s} differs"
        assert_close(o_p, ref.decode_dense(to_np(q[:, s + 1:s + 2])), BF16, f"paged rope decode_step {s}")
    paged.poll_status(); flat.poll_status()
    # pages that straddle two sequences' slabs cannot be addressed by the rotary kernel's tiled copies
    odd = B.EigenAttnLayer(2, 1, 128, 384, BF16, [U_k[0]], [U_v[0]])
    odd.set_page_table([[0, 2], [1, -1]], 256)
    odd.set_rope(10000.0)
    odd.append_kv(k[:2, :8, :1].contiguous(), v[:2, :8, :1].contiguous())
    with pytest.raises(B.EigenAttnError) as e:
        odd.decode(q[:2, :1, :1].contiguous())
    assert e.value.status == B.EA_ERR_UNSUPPORTED


@pytest.mark.parametrize("g,rk,rv", [(4, [80, 80], [80, 80]), (12, [48, 128], [96, 64])])
def test_grouped_queries_over_a_paged_cache(B, g, rk, rv):
    """Grouped queries (no rotary embedding) of a paged layer: the warp-level kernel fetches every tile of 128 rows
    from the page that holds it and returns what the contiguous layer returns, bit for bit, through several CTA counts
    and a decode step; both agree with the oracle.  The tcgen05 kernel reads contiguous slabs only and is refused."""
    B_, H, d, n_max, page_rows = 3, 2, 128, 1536, 128
    n = 1100
    U_k, U_v, _, k, v = make_case(B_, H, d, rk, rv, n + 1, BF16, seed_cfg=191)
    W_q = synth.mixing_matrices(H * g, 16, d, 191, "W_Q")
    qg = synth.lowrank_rows(W_q, B_, 1, 0.1, 191, "Q", dtype=BF16, device="cuda:0")
    flat = B.EigenAttnLayer(B_, H, d, n_max, BF16, U_k, U_v)
    paged = B.EigenAttnLayer(B_, H, d, n_max, BF16, U_k, U_v)
    per_seq = n_max // page_rows
    perm = np.random.default_rng(11).permutation(B_ * per_seq)
    paged.set_page_table([[int(x) for x in perm[b * per_seq:(b + 1) * per_seq]] for b in range(B_)], page_rows)
    ref = oracle_layer(B_, H, d, U_k, U_v)
    for lay in (flat, paged):
        lay.append_kv(k[:, :n], v[:, :n])
    ref.append_kv(to_np(k[:, :n]), to_np(v[:, :n]))
    expect = ref.decode_gqa(to_np(qg), g)
    for ctas in (0, 1, 9, 300):
        for lay in (flat, paged):
            lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        want = flat.decode_gqa(qg, g)
        assert torch.equal(paged.decode_gqa(qg, g), want), f"paged grouped decode differs, ctas={ctas}"
        assert_close(want, expect, BF16, f"grouped queries, paged, ctas={ctas}")
    for lay in (flat, paged):
        lay.append_kv(k[:, n:], v[:, n:])
    ref.append_kv(to_np(k[:, n:]), to_np(v[:, n:]))
    want = flat.decode_gqa(qg, g)
    assert torch.equal(paged.decode_gqa(qg, g), want)
    assert_close(want, ref.decode_gqa(to_np(qg), g), BF16, "grouped queries, paged, after an append")
    paged.poll_status(); flat.poll_status()
    paged.set_option(B.EA_OPT_GQA_IMPL, 1)
    with pytest.raises(B.EigenAttnError):
        paged.decode_gqa(qg, g)
