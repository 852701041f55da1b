"""GPU parity for a batch whose sequences differ in length (eigen_attn_set_lens): every sequence attends its own
rows and grows at its own end.  The generation phase of Section 2 is stated per sequence, so the expected value
of sequence b is the oracle run on that sequence alone with its own history."""
import numpy as np
import pytest
import torch

from helpers import Expect, assert_close, make_case, oracle_layer, storage_model, to_np
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


class PerSequenceOracle:
    """One single-sequence oracle layer per sequence of the batch."""

    def __init__(self, H, d, U_k, U_v, k, v, lens, alibi_slopes=None, storage=None, rope=None):
        """With `storage` (the 16-bit cache model) a second set of layers keeps fp64 rows, and decode() returns
        an Expect carrying both results."""
        self.H, self.d = H, d
        self.refs, self.plain = [], []
        for b, n in enumerate(lens):
            for group, st in ((self.refs, storage),) + (((self.plain, None),) if storage is not None else ()):
                r = orc.LayerOracle(1, H, d, U_k, U_v, alibi_slopes=alibi_slopes, storage=st, rope=rope)
                if n > 0:
                    r.append_kv(to_np(k[b:b + 1, :n]), to_np(v[b:b + 1, :n]))
                group.append(r)

    def append(self, k, v):                       # k, v: [B, T, H, d]
        for group in (self.refs, self.plain):
            for b, r in enumerate(group):
                r.append_kv(to_np(k[b:b + 1]), to_np(v[b:b + 1]))

    def prefill(self, q, k, v):                   # q, k, v: [B, T, H, d] -> [B, T, H, d]; the rows are appended
        one = lambda group: np.concatenate([r.prefill_dense(to_np(q[b:b + 1]), to_np(k[b:b + 1]), to_np(v[b:b + 1]))
                                            for b, r in enumerate(group)], axis=0)
        return Expect(one(self.refs), one(self.plain)) if self.plain else one(self.refs)

    def decode(self, q):                          # q: [B, 1, H, d] -> [B, 1, H, d]
        one = lambda group: np.concatenate([r.decode_dense(to_np(q[b:b + 1])).reshape(1, 1, self.H, self.d)
                                            for b, r in enumerate(group)], axis=0)
        return Expect(one(self.refs), one(self.plain)) if self.plain else one(self.refs)


@pytest.mark.parametrize("dtype,d,rk,rv,n,lens", [
    (FP32, 64, [32, 20, 64], [16, 40, 8], 700, [700, 1, 77, 570]),
    (BF16, 128, [80, 48, 128], [80, 112, 64], 3000, [3000, 129, 1, 2871]),      # units split over many CTAs
    (BF16, 128, [80, 80, 80], [80, 80, 80], 2048, [5, 2048, 2047, 1024]),       # the first sequence is the short one
])
def test_decode_and_steps_with_unequal_lengths(B, dtype, d, rk, rv, n, lens):
    B_, H = 4, 3
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n + 8, dtype, seed_cfg=140, T_q=8)
    lay = B.EigenAttnLayer(B_, H, d, n + 8, dtype, U_k, U_v)
    lay.append_kv(k[:, :n], v[:, :n])             # every sequence holds n rows; each keeps its first lens[b]
    lay.set_lens(lens)
    assert lay.lens() == list(lens) and lay.len == max(lens)
    ref = PerSequenceOracle(H, d, U_k, U_v, k, v, lens)
    expect = ref.decode(q[:, :1])
    for ctas, fused in ((0, 1), (0, 0), (1, 1), (37, 0), (5, 1)):
        lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        lay.set_option(B.EA_OPT_DECODE_FUSED, fused)
        assert_close(lay.decode(q[:, :1]), expect, dtype, f"decode ctas={ctas} fused={fused}")
    lay.set_option(B.EA_OPT_DECODE_CTAS, 0)
    assert_close(lay.decode_static(q[:, :1]), expect, dtype, "decode_static")
    # generation: each sequence's new row goes behind its own end (fresh rows, not the ones cut off above)
    for step, fused in enumerate((1, 1, 0)):
        lay.set_option(B.EA_OPT_DECODE_FUSED, fused)
        kn, vn = k[:, n + step:n + step + 1], v[:, n + step:n + step + 1]
        o = lay.decode_step(q[:, step + 1:step + 2], kn, vn)
        ref.append(kn, vn)
        assert_close(o, ref.decode(q[:, step + 1:step + 2]), dtype, f"decode_step {step} fused={fused}")
    assert lay.lens() == [x + 3 for x in lens]
    # several rows at once behind each end
    lay.append_kv(k[:, n + 3:n + 8], v[:, n + 3:n + 8])
    ref.append(k[:, n + 3:n + 8], v[:, n + 3:n + 8])
    lay.set_option(B.EA_OPT_DECODE_FUSED, 1)
    assert_close(lay.decode(q[:, 4:5]), ref.decode(q[:, 4:5]), dtype, "decode after append_kv")
    lay.poll_status()


def test_sequence_with_no_rows_and_return_to_equal_lengths(B):
    B_, H, d, n = 3, 2, 64, 300
    rk, rv = [32, 24], [16, 40]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n + 1, FP32, seed_cfg=141, T_q=2)
    lay = B.EigenAttnLayer(B_, H, d, n + 1, FP32, U_k, U_v, max_prefill_tokens=16)
    lay.append_kv(k[:, :n], v[:, :n])
    uniform = lay.decode(q[:, :1]).clone()
    lens = [0, n, 150]
    lay.set_lens(lens)
    with pytest.raises(B.EigenAttnError) as e:    # a sequence without rows has nothing to attend
        lay.decode(q[:, :1])
    assert e.value.status == B.EA_ERR_SHAPE
    with pytest.raises(B.EigenAttnError) as e:
        lay.set_lens([0, n + 2, 1])
    assert e.value.status == B.EA_ERR_CAPACITY and lay.lens() == lens
    # with its new token the empty sequence attends exactly that token
    ref = PerSequenceOracle(H, d, U_k, U_v, k, v, lens)
    o = lay.decode_step(q[:, 1:2], k[:, n:n + 1], v[:, n:n + 1])
    ref.append(k[:, n:n + 1], v[:, n:n + 1])
    assert_close(o, ref.decode(q[:, 1:2]), FP32, "decode_step with an empty sequence")
    assert lay.lens() == [1, n + 1, 151]
    lay.set_len(n)                                # equal lengths again: rows [0, n) of every sequence
    assert lay.lens() == [n] * B_
    # the step above overwrote row 0 of sequence 0 and row 150 of sequence 2; sequence 1 is as before
    again = lay.decode(q[:, :1])
    assert torch.equal(again[1], uniform[1])
    lay.poll_status()


@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_alibi_positions_count_from_each_sequences_own_end(B, dtype):
    B_, H, d, n = 3, 4, 64, 900
    rk, rv = [32, 48, 64, 16], [32, 16, 64, 48]
    lens = [900, 333, 2]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n + 1, dtype, seed_cfg=142, T_q=2)
    slopes = synth.alibi_slopes(H)
    lay = B.EigenAttnLayer(B_, H, d, n + 1, dtype, U_k, U_v)
    lay.set_alibi(slopes)
    lay.append_kv(k[:, :n], v[:, :n])
    lay.set_lens(lens)
    ref = PerSequenceOracle(H, d, U_k, U_v, k, v, lens, alibi_slopes=slopes, storage=storage_model(dtype))
    tol = dict(fp32_rel=2e-5) if dtype == FP32 else {}
    assert_close(lay.decode(q[:, :1]), ref.decode(q[:, :1]), dtype, "decode", **tol, plain_within=True)
    o = lay.decode_step(q[:, 1:2], k[:, n:n + 1], v[:, n:n + 1])
    ref.append(k[:, n:n + 1], v[:, n:n + 1])
    assert_close(o, ref.decode(q[:, 1:2]), dtype, "decode_step", **tol, plain_within=True)
    lay.poll_status()


@pytest.mark.parametrize("rope", [None, {"base": 10000.0, "interleaved": False}])
@pytest.mark.parametrize("H,g,d,rk,rv,n,lens", [
    (2, 4, 128, [80, 80], [80, 80], 1037, [1037, 1, 500]),
    (3, 8, 128, [48, 64, 128], [96, 80, 128], 700, [129, 700, 128]),
])
def test_grouped_query_decode_with_unequal_lengths(B, H, g, d, rk, rv, n, lens, rope):
    """Every query head of a group attends the own rows of its sequence's K/V head; with a rotary embedding the
    queries of a sequence sit at that sequence's own last position (first case: the grouped rotary kernel on the
    tensor cores; second: a rank of 128 does not fit it, every query head is a unit of the multi-head kernel)."""
    B_ = len(lens)
    U_k, U_v, _, k, v = make_case(B_, H, d, rk, rv, n + 1, BF16, seed_cfg=143)
    W_q = synth.mixing_matrices(H * g, 16, d, 143, "W_Q")
    q = synth.lowrank_rows(W_q, B_, 1, 0.1, 143, "Q", dtype=BF16, device="cuda:0")        # [B][1][H*g][d]
    lay = B.EigenAttnLayer(B_, H, d, n + 1, BF16, U_k, U_v)
    if rope:
        lay.set_rope(rope["base"], rope["interleaved"])
    lay.append_kv(k[:, :n], v[:, :n])
    lay.set_lens(lens)
    refs = []
    for b, nb in enumerate(lens):
        r = orc.LayerOracle(1, H, d, U_k, U_v, rope=rope)
        r.append_kv(to_np(k[b:b + 1, :nb]), to_np(v[b:b + 1, :nb]))
        refs.append(r)
    expect = lambda: np.concatenate([r.decode_gqa(to_np(q[b:b + 1]), g) for b, r in enumerate(refs)], axis=0)
    for ctas in (0, 1, 7, 300):
        lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        assert_close(lay.decode_gqa(q, g), expect(), BF16, f"gqa decode ctas={ctas}")
    lay.append_kv(k[:, n:], v[:, n:])             # one more row behind every sequence's own end
    for b, r in enumerate(refs):
        r.append_kv(to_np(k[b:b + 1, n:]), to_np(v[b:b + 1, n:]))
    assert_close(lay.decode_gqa(q, g), expect(), BF16, "gqa decode after append")
    lay.poll_status()


def test_set_lens_argument_checks(B):
    B_, H, d, n = 2, 2, 128, 64
    U_k, U_v, q, k, v = make_case(B_, H, d, [64] * H, [64] * H, n, BF16, seed_cfg=144)
    lay = B.EigenAttnLayer(B_, H, d, n, BF16, U_k, U_v)
    lay.append_kv(k, v)
    lay.set_lens([n, 5])
    for call in (lambda: lay.set_lens([n, -1]), lambda: lay.set_lens([n + 1, 1])):
        with pytest.raises(B.EigenAttnError):
            call()
    assert lay.lens() == [n, 5]
    lay.set_lens([n, n])                          # equal again
    assert lay.lens() == [n, n]
    lay.poll_status()


@pytest.mark.parametrize("bits,G", [(4, 32), (3, 16), (4, 128)])
def test_quantised_cache_with_unequal_lengths(B, bits, G):
    """Section 5.3 per sequence: every sequence keeps the codes of its own complete blocks and attends them plus
    its own 16-bit tail.  The expected value is the oracle's quantised decode of each sequence alone.  Order of
    events: uniform fill and sync, then the true lengths (codes below each length are kept), decode; more rows
    behind every sequence's own end, sync with lengths in force, decode; a buffer attached while lengths differ;
    back to equal lengths."""
    from oracle import kv_quant as kq
    H, d, n = 3, 128, 1500
    rk, rv = [80, 48, 128], [80, 112, 64]
    lens = [1500, 700, 37, 1]                      # 37 < G for G = 128: that sequence has no codes at all
    B_ = len(lens)
    extra = 40
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n + extra, BF16, seed_cfg=146, T_q=3)
    lay = B.EigenAttnLayer(B_, H, d, n + extra, BF16, U_k, U_v)
    lay.append_kv(k[:, :n], v[:, :n])
    lay.quant_attach(bits, G)
    lay.quant_sync()
    assert lay.quant_len == n // G * G
    lay.set_lens(lens)
    assert lay.quant_lens() == [x // G * G for x in lens] and lay.quant_len == lens[0] // G * G

    store = storage_model(BF16)                    # the oracle quantises the 16-bit rows the cache holds
    def expect(qq, cur_lens, rows_of):
        outs = []
        for b, nb in enumerate(cur_lens):
            r = orc.LayerOracle(1, H, d, U_k, U_v, storage=store)
            kk, vv = rows_of(b, nb)
            r.append_kv(kk, vv)
            res = r.decode_quant(to_np(qq[b:b + 1]), bits, G)
            outs.append(np.stack([res[(0, h)] for h in range(H)])[None, None])
        return np.concatenate(outs, axis=0)

    first = lambda b, nb: (to_np(k[b:b + 1, :nb]), to_np(v[b:b + 1, :nb]))
    for ctas in (0, 1, 400):
        lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        assert_close(lay.decode_quant(q[:, :1]), expect(q[:, :1], lens, first), BF16, f"ragged quant decode ctas={ctas}")
    lay.set_option(B.EA_OPT_DECODE_CTAS, 0)
    # `extra` more rows behind each sequence's own end; some sequences complete new blocks, which the sync quantises
    lay.append_kv(k[:, n:], v[:, n:])
    lens2 = [x + extra for x in lens]
    grown = lambda b, nb: (np.concatenate([to_np(k[b:b + 1, :lens[b]]), to_np(k[b:b + 1, n:])], axis=1),
                           np.concatenate([to_np(v[b:b + 1, :lens[b]]), to_np(v[b:b + 1, n:])], axis=1))
    before = lay.quant_lens()
    out_unsynced = lay.decode_quant(q[:, 1:2])     # new rows still 16-bit: codes below the old counts only
    lay.quant_sync()
    assert lay.quant_lens() == [x // G * G for x in lens2] and lay.quant_lens() != before
    assert_close(lay.decode_quant(q[:, 1:2]), expect(q[:, 1:2], lens2, grown), BF16, "after a sync with lengths in force")
    assert float((out_unsynced.float() - lay.decode_quant(q[:, 1:2]).float()).abs().max()) < 0.25   # same rows, other precision
    # a fresh buffer attached while lengths differ starts without codes: the decode reads 16-bit rows only
    lay.quant_attach(bits, G)
    assert lay.quant_lens() == [0] * B_
    plain = lay.decode(q[:, 1:2])
    assert torch.equal(lay.decode_quant(q[:, 1:2]), plain) or float((lay.decode_quant(q[:, 1:2]).float() - plain.float()).abs().max()) < 2e-2
    lay.quant_sync()
    assert_close(lay.decode_quant(q[:, 1:2]), expect(q[:, 1:2], lens2, grown), BF16, "buffer attached while lengths differ")
    # back to equal lengths: the codes every sequence holds stay
    lay.set_len(min(lens2))
    assert lay.quant_len == min(lens2) // G * G
    lay.poll_status()


@pytest.mark.parametrize("interleaved,lens", [(False, [1037, 1, 300]), (True, [129, 1037, 128])])
def test_rope_decode_with_unequal_lengths(B, interleaved, lens):
    """Section 4.3 per sequence: row j of a sequence sits at position j, its query at its own last position."""
    B_, H, d, n = len(lens), 2, 128, 1037
    rk, rv = [80, 48], [64, 80]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n + 2, BF16, seed_cfg=145, T_q=3)
    lay = B.EigenAttnLayer(B_, H, d, n + 2, BF16, U_k, U_v)
    lay.set_rope(10000.0, interleaved)
    lay.append_kv(k[:, :n], v[:, :n])
    lay.set_lens(lens)
    ref = PerSequenceOracle(H, d, U_k, U_v, k, v, lens, storage=storage_model(BF16),    # few rows: model the 16-bit cache
                            rope={"base": 10000.0, "interleaved": interleaved})
    expect = ref.decode
    for ctas in (0, 1, 300):
        lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        assert_close(lay.decode(q[:, :1]), expect(q[:, :1]), BF16, f"rope decode ctas={ctas}", plain_within=True)
    for s_ in range(2):                           # each sequence's new row at its own next position
        kn, vn = k[:, n + s_:n + s_ + 1], v[:, n + s_:n + s_ + 1]
        o = lay.decode_step(q[:, s_ + 1:s_ + 2], kn, vn)
        ref.append(kn, vn)
        assert_close(o, expect(q[:, s_ + 1:s_ + 2]), BF16, f"rope step {s_}", plain_within=True)
    lay.poll_status()


def test_padded_prompt_batch_then_generation_at_the_true_lengths(B):
    """The serving pattern: prompts of different lengths are padded to a common T and prefilled in one call (causality
    keeps the padding out of every real token's result), then the layer is told the true lengths and generation
    appends behind each prompt's own end, over the padding rows."""
    B_, H, d, T = 3, 2, 128, 300
    rk, rv = [80, 48], [64, 80]
    lens = [300, 131, 7]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, T + 2, BF16, seed_cfg=146, T_q=T + 2)
    lay = B.EigenAttnLayer(B_, H, d, T + 2, BF16, U_k, U_v, max_prefill_tokens=T)
    out = lay.prefill(q[:, :T], k[:, :T], v[:, :T])
    refs = []
    for b, nb in enumerate(lens):
        r = oracle_layer(1, H, d, U_k, U_v)
        expect = r.prefill_dense(to_np(q[b:b + 1, :nb]), to_np(k[b:b + 1, :nb]), to_np(v[b:b + 1, :nb]))
        assert_close(out[b:b + 1, :nb], expect, BF16, f"prompt of sequence {b}")
        refs.append(r)
    lay.set_lens(lens)
    for s_ in range(2):
        qn, kn, vn = (x[:, T + s_:T + s_ + 1] for x in (q, k, v))
        o = lay.decode_step(qn, kn, vn)
        for b, r in enumerate(refs):
            r.append_kv(to_np(kn[b:b + 1]), to_np(vn[b:b + 1]))
        expect = np.concatenate([r.decode_dense(to_np(qn[b:b + 1])).reshape(1, 1, H, d) for b, r in enumerate(refs)], axis=0)
        assert_close(o, expect, BF16, f"generated token {s_}")
    assert lay.lens() == [x + 2 for x in lens]
    lay.poll_status()


def test_many_sequences_of_unequal_lengths(B):
    """More sequences than one step of the tile-count prefix handles (32): lengths 1 .. n in a fixed shuffle."""
    B_, H, d, n = 70, 1, 64, 200
    lens = [1 + (37 * b) % n for b in range(B_)]
    U_k, U_v, q, k, v = make_case(B_, H, d, [32], [24], n + 1, FP32, seed_cfg=147, T_q=2)
    lay = B.EigenAttnLayer(B_, H, d, n + 1, FP32, U_k, U_v)
    lay.append_kv(k[:, :n], v[:, :n])
    lay.set_lens(lens)
    ref = PerSequenceOracle(H, d, U_k, U_v, k, v, lens)
    for ctas in (0, 3):
        lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        assert_close(lay.decode(q[:, :1]), ref.decode(q[:, :1]), FP32, f"decode ctas={ctas}")
    o = lay.decode_step(q[:, 1:2], k[:, n:], v[:, n:])
    ref.append(k[:, n:], v[:, n:])
    assert_close(o, ref.decode(q[:, 1:2]), FP32, "decode_step")
    lay.poll_status()


@pytest.mark.parametrize("dtype,d,rk,rv,n,lens,T,variant", [
    (BF16, 128, [80, 48, 128], [80, 112, 64], 600, [600, 129, 0, 471], 300, "plain"),     # warp-specialised tcgen05 kernel
    (BF16, 128, [80, 80, 80], [80, 80, 80], 300, [5, 300, 299, 64], 130, "alibi"),
    (BF16, 128, [80, 64, 48], [64, 80, 96], 260, [260, 1, 77, 130], 70, "rope"),          # Section 4.3 prompt form
    (BF16, 128, [80, 64, 48], [64, 80, 96], 260, [260, 1, 77, 130], 70, "rope-tc"),       # ... on the tensor cores
    (FP32, 64, [32, 20, 64], [16, 40, 8], 200, [200, 1, 77, 0], 50, "plain"),             # CUDA-core kernel
    (BF16, 128, [80, 48, 128], [80, 112, 64], 400, [400, 129, 3, 271], 200, "single-tile"),
])
def test_prompt_chunk_behind_sequences_of_unequal_lengths(B, dtype, d, rk, rv, n, lens, T, variant):
    """A chunk of T prompt tokens for every sequence of a batch whose sequences hold different numbers of rows
    (continuous batching: chunked prompts of some sequences beside others further along): token t of sequence b
    sits at position lens[b] + t and sees that sequence's own rows only.  Then a generated token on top."""
    B_, H = 4, 3
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n + T + 1, dtype, seed_cfg=148, T_q=n + T + 1)
    if dtype == BF16:
        q = (q.float() * 0.25).to(dtype)                              # Q' is kept in 16 bits by the prompt kernels
    tc_rope = variant == "rope-tc"                 # the scratch must hold every row a sequence has after the call
    lay = B.EigenAttnLayer(B_, H, d, n + T + 1, dtype, U_k, U_v, max_prefill_tokens=n + T if tc_rope else T,
                           rope_prompt_scratch=tc_rope)
    slopes = [0.5, 0.0625, 0.25] if variant == "alibi" else None
    rope = {"base": 10000.0, "interleaved": False} if variant.startswith("rope") else None
    if slopes:
        lay.set_alibi(slopes)
    if rope:
        lay.set_rope(rope["base"], rope["interleaved"])
    if variant == "single-tile":
        lay.set_option(B.EA_OPT_PREFILL_IMPL, 3)
    if tc_rope:
        lay.set_option(B.EA_OPT_PREFILL_IMPL, 2)   # refuse rather than fall back to the CUDA-core kernel
    lay.append_kv(k[:, :n], v[:, :n])              # every sequence holds n rows; each keeps its first lens[b]
    lay.set_lens(lens)
    ref = PerSequenceOracle(H, d, U_k, U_v, k, v, lens, alibi_slopes=slopes, storage=storage_model(dtype), rope=rope)
    # the chunk of sequence b: rows n .. n + T - 1 of the drawn tensors (any rows would do)
    qc, kc, vc = (x[:, n:n + T].contiguous() for x in (q, k, v))
    out = lay.prefill(qc, kc, vc)
    assert_close(out, ref.prefill(qc, kc, vc), dtype, f"prompt chunk ({variant})")
    assert lay.lens() == [x + T for x in lens]
    qn, kn, vn = (x[:, n + T:n + T + 1] for x in (q, k, v))
    o = lay.decode_step(qn, kn, vn)
    ref.append(kn, vn)
    assert_close(o, ref.decode(qn), dtype, f"generated token after the chunk ({variant})")
    lay.poll_status()
