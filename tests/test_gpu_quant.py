"""GPU parity of the quantised rank-r cache (Section 5.3, Table 8) against the oracle, through the C ABI.

Codes and scales are integer / bit work and must match exactly: both sides start from the same 16-bit rows
(rank-space rows handed to the library as they are, so no projection arithmetic precedes the quantiser) and
take every rounding decision in single precision.  The decode over the codes is compared with the fp64 oracle
over the de-quantised rows within the bf16 tolerances of the other decode tests."""
import numpy as np
import pytest
import torch

from helpers import assert_close, make_case, oracle_layer, to_np
from oracle import kv_quant as kq
from paper_2408_05646_b200 import synth

pytestmark = pytest.mark.gpu
BF16 = torch.bfloat16


@pytest.fixture(scope="module")
def B():
    from paper_2408_05646_b200 import build
    build.build_library()
    from paper_2408_05646_b200 import binding
    return binding


def rank_space_case(B_, H, d, rk, rv, n, seed, q_scale=1.0):
    """Bases, a query, and the rank-space rows K' = K U^K, V' = V U^V rounded to bf16 on the host: the packed
    tensors for the library and the per-unit float64 arrays (the same values) for the oracle."""
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n, BF16, seed_cfg=seed, q_scale=q_scale)
    offs_k = np.concatenate([[0], np.cumsum([(r + 7) // 8 * 8 for r in rk])])
    offs_v = np.concatenate([[0], np.cumsum([(r + 7) // 8 * 8 for r in rv])])
    kp = torch.zeros((B_, n, int(offs_k[-1])), dtype=BF16)
    vp = torch.zeros((B_, n, int(offs_v[-1])), dtype=BF16)
    kn, vn = to_np(k), to_np(v)
    rows = {}
    for h in range(H):
        a = torch.from_numpy(kn[:, :, h, :] @ U_k[h].astype(np.float64)).to(BF16)
        c = torch.from_numpy(vn[:, :, h, :] @ U_v[h].astype(np.float64)).to(BF16)
        kp[:, :, offs_k[h]:offs_k[h] + rk[h]] = a
        vp[:, :, offs_v[h]:offs_v[h] + rv[h]] = c
        for b in range(B_):
            rows[(b, h)] = (a[b].double().numpy(), c[b].double().numpy())
    return U_k, U_v, q, kp.cuda(), vp.cuda(), rows


def fill_both(B, B_, H, d, rk, rv, n, n_max, seed, group, alibi=None, q_scale=1.0, bits=4):
    U_k, U_v, q, kp, vp, rows = rank_space_case(B_, H, d, rk, rv, n, seed, q_scale)
    lay = B.EigenAttnLayer(B_, H, d, n_max, BF16, U_k, U_v)
    lay.append_kv(kp, vp, preprojected=True)
    ref = oracle_layer(B_, H, d, U_k, U_v, alibi_slopes=alibi)
    for u, (a, c) in rows.items():
        ref.Kp[u], ref.Vp[u] = a, c
    ref.set_len(n)
    if alibi is not None:
        lay.set_alibi(alibi)
    lay.quant_attach(bits, group)
    return lay, ref, q, rows


def unpack_codes(area: np.ndarray, rp: int, G: int, bits: int, values: bool = False) -> np.ndarray:
    """A block's code area (bytes) -> codes [G][rp], each stored as code + 2^(bits-1).
    3-bit: unit j of row i holds channels 8j..8j+7 (channel 8j+k in bits 3k..); the low 16 bits of all units
    ([rp/8][G] halfwords), then their high 8 bits ([rp/8][G] bytes).
    4-bit keys: word j of row i (channel 8j+k in bits 4k..) sits at j G + ((i + 8 (j mod 4)) mod G).
    4-bit values: chunks of min(G, 32) rows, a chunk [rp][rows/8] words, word (c, o) = rows 8o..8o+7 of channel c."""
    nw = rp // 8
    out = np.zeros((G, rp), dtype=np.int64)
    if bits == 4 and values:
        rows = min(G, 32)
        words = area.view(np.uint32).reshape(G // rows, rp, rows // 8).astype(np.int64)
        for k in range(8):
            nib = ((words >> (4 * k)) & 15) - 8                     # [chunk][c][o] -> row 32 chunk + 8 o + k
            for qc in range(G // rows):
                for o in range(rows // 8):
                    out[qc * rows + 8 * o + k, :] = nib[qc, :, o]
        return out
    if bits == 4:
        stored = area.view(np.uint32).reshape(nw, G).astype(np.int64)
        units = np.zeros_like(stored)
        for j in range(nw):
            units[j, :] = stored[j, (np.arange(G) + 8 * (j % 4)) % G]
    else:
        lo = area[:2 * nw * G].view(np.uint16).reshape(nw, G).astype(np.int64)
        hi = area[2 * nw * G:3 * nw * G].reshape(nw, G).astype(np.int64)
        units = lo | (hi << 16)
    for k in range(8):
        out[:, k::8] = ((units.T >> (bits * k)) & ((1 << bits) - 1)) - (1 << (bits - 1))
    return out


def read_block(lay, head, b, blk, G, rp_k, rp_v, bits=4):
    _, bb, ks_off, vc_off, vs_off = lay.quant_layout(head)
    raw = lay.quant_blocks(head)[b, blk].cpu().numpy()
    assert ks_off == G * rp_k * bits // 8 and vs_off - vc_off == G * rp_v * bits // 8      # exactly `bits` per element
    kc = unpack_codes(raw[:ks_off], rp_k, G, bits)
    ks = raw[ks_off:vc_off].view(np.float16)
    vc = unpack_codes(raw[vc_off:vs_off], rp_v, G, bits, values=True)
    nvg = (rp_v + G - 1) // G
    vs = raw[vs_off:vs_off + 2 * G * nvg].view(np.float16).reshape(nvg, G).T       # -> [G][nvg]
    return kc, ks, vc, vs


@pytest.mark.parametrize("bits", [4, 3])
@pytest.mark.parametrize("G,H,d,rk,rv,n", [
    (32, 2, 128, [80, 80], [80, 80], 200),            # the headline rank; 6 blocks and 8 rows left over
    (16, 2, 128, [80, 48], [64, 80], 100),            # smallest group: five value groups per row
    (64, 3, 64, [24, 64, 37], [56, 8, 64], 300),      # ranks that are not multiples of 8 (zero padding inside a word)
    (128, 2, 128, [128, 80], [128, 96], 400),         # widest rank; one value group per row
])
def test_codes_and_scales_are_bit_exact(B, G, H, d, rk, rv, n, bits):
    B_ = 2
    lay, ref, q, rows = fill_both(B, B_, H, d, rk, rv, n, n + 5, 171, G, bits=bits)
    lay.quant_sync()
    torch.cuda.synchronize()
    assert lay.quant_len == n // G * G
    for h in range(H):
        rp_k, rp_v = (rk[h] + 7) // 8 * 8, (rv[h] + 7) // 8 * 8
        for b in range(B_):
            Kp, Vp = rows[(b, h)]
            nq = n // G * G
            kc_ref, ks_ref = kq.quantize_keys(Kp[:nq], bits, G)
            vc_ref, vs_ref = kq.quantize_values(Vp[:nq], bits, G)
            for blk in range(n // G):
                kc, ks, vc, vs = read_block(lay, h, b, blk, G, rp_k, rp_v, bits)
                sl = slice(blk * G, (blk + 1) * G)
                assert np.array_equal(kc[:, :rk[h]], kc_ref[sl]), (h, b, blk, "key codes")
                assert np.array_equal(ks[:rk[h]], ks_ref[blk]), (h, b, blk, "key scales")
                assert np.array_equal(vc[:, :rv[h]], vc_ref[sl]), (h, b, blk, "value codes")
                assert np.array_equal(vs[:, :vs_ref.shape[1]], vs_ref[sl]), (h, b, blk, "value scales")
                assert np.all(kc[:, rk[h]:] == 0) and np.all(vc[:, rv[h]:] == 0)      # padding columns hold zeros


@pytest.mark.parametrize("G,H,d,rk,rv,n", [
    (32, 2, 128, [80, 80], [80, 80], 128),            # exactly one stage, nothing left over
    (32, 2, 128, [80, 80], [80, 80], 1037),           # several stages, a partial last stage, 13 rows left over
    (16, 2, 128, [80, 48], [64, 80], 777),            # two blocks per warp
    (64, 3, 64, [24, 64, 37], [56, 8, 64], 2500),     # per-head ranks, small d_head
    (128, 2, 128, [128, 80], [128, 96], 1500),        # widest rank (the 16-word kernel)
    (32, 1, 128, [80], [80], 20),                     # shorter than one group: all rows come from the 16-bit cache
    (32, 4, 128, [80] * 4, [80] * 4, 9000),           # many stages per CTA, several splits
])
@pytest.mark.parametrize("bits", [4, 3])
def test_decode_quant_matches_oracle(B, G, H, d, rk, rv, n, bits):
    B_ = 2
    lay, ref, q, _ = fill_both(B, B_, H, d, rk, rv, n, n + 7 + G, 172, G, bits=bits)
    lay.quant_sync()
    out = lay.decode_quant(q)
    lay.poll_status()
    res = ref.decode_quant(to_np(q), bits, G)
    want = np.stack([np.stack([res[(b, h)] for h in range(H)]) for b in range(B_)])[:, None]
    assert_close(out, want, BF16, f"decode_quant G={G} n={n}")
    # the quantisation error itself is far above the tolerance: the test would notice codes that are ignored
    plain = ref.decode_dense(to_np(q))
    if n >= 4 * G:
        assert np.abs(plain - want).max() > 1e-3


def test_decode_quant_with_rows_that_are_not_synced_yet(B):
    """quant_sync is the caller's to schedule: rows appended after it are read from the 16-bit cache."""
    B_, H, d, G = 2, 2, 128, 32
    n0, n1 = 300, 420
    U_k, U_v, q, kp, vp, rows = rank_space_case(B_, H, d, [80, 64], [80, 72], n1, 173)
    lay = B.EigenAttnLayer(B_, H, d, n1, BF16, U_k, U_v)
    lay.quant_attach(4, G)
    lay.append_kv(kp[:, :n0].contiguous(), vp[:, :n0].contiguous(), preprojected=True)
    lay.quant_sync()
    assert lay.quant_len == 288
    lay.append_kv(kp[:, n0:].contiguous(), vp[:, n0:].contiguous(), preprojected=True)
    out = lay.decode_quant(q)
    lay.poll_status()
    # the oracle's view with 288 quantised rows: quantise the first 288, keep the rest
    ref = oracle_layer(B_, H, d, U_k, U_v)
    for u, (a, c) in rows.items():
        Kq, Vq = kq.quantized_view(a[:288], c[:288], 4, G)
        ref.Kp[u], ref.Vp[u] = np.concatenate([Kq, a[288:]]), np.concatenate([Vq, c[288:]])
    ref.set_len(n1)
    assert_close(out, ref.decode_dense(to_np(q)), BF16, "unsynced tail")
    # after the next sync the newer blocks are codes too
    lay.quant_sync()
    assert lay.quant_len == 416
    out2 = lay.decode_quant(q)
    ref2 = oracle_layer(B_, H, d, U_k, U_v)
    for u, (a, c) in rows.items():
        ref2.Kp[u], ref2.Vp[u] = a, c
    ref2.set_len(n1)
    res = ref2.decode_quant(to_np(q), 4, G)
    want = np.stack([np.stack([res[(b, h)] for h in range(H)]) for b in range(B_)])[:, None]
    assert_close(out2, want, BF16, "after the second sync")
    # rewinding below the quantised length forgets whole blocks
    lay.set_len(100)
    assert lay.quant_len == 96


@pytest.mark.parametrize("bits", [4, 3])
def test_decode_quant_with_peaked_attention_and_alibi(B, bits):
    """Few rows carry the softmax (scaled query, steep bias on one head): a wrong scale or code of a single row
    is not averaged away."""
    B_, H, d, G, n = 2, 4, 128, 32, 1500
    slopes = [0.25, 0.0, 2.0 ** -4, 2.0 ** -8]
    lay, ref, q, _ = fill_both(B, B_, H, d, [80] * H, [80] * H, n, n, 174, G, alibi=slopes, q_scale=3.0, bits=bits)
    lay.quant_sync()
    out = lay.decode_quant(q)
    lay.poll_status()
    res = ref.decode_quant(to_np(q), bits, G)
    want = np.stack([np.stack([res[(b, h)] for h in range(H)]) for b in range(B_)])[:, None]
    assert_close(out, want, BF16, "peaked + alibi")


def scaled_case(B, B_, H, d, r, n, seed, G, k_gain, v_gain, q_scale=1.0):
    """A layer whose rank-space rows are those of rank_space_case times per-channel key gains [r] and per-row
    value gains [n] (exact powers of two, so the 16-bit rows stay exact), on both sides."""
    U_k, U_v, q, kp, vp, _ = rank_space_case(B_, H, d, [r] * H, [r] * H, n, seed, q_scale)
    kg = torch.tensor(k_gain, dtype=torch.float32).cuda()
    vg = torch.tensor(v_gain, dtype=torch.float32).cuda()
    kp = (kp.float() * kg.repeat(H)[None, None, :]).to(BF16)
    vp = (vp.float() * vg[None, :, None]).to(BF16)
    lay = B.EigenAttnLayer(B_, H, d, n, BF16, U_k, U_v)
    lay.append_kv(kp, vp, preprojected=True)
    ref = oracle_layer(B_, H, d, U_k, U_v)
    for b in range(B_):
        for h in range(H):
            ref.Kp[(b, h)] = kp[b, :, h * r:(h + 1) * r].double().cpu().numpy()
            ref.Vp[(b, h)] = vp[b, :, h * r:(h + 1) * r].double().cpu().numpy()
    ref.set_len(n)
    lay.quant_attach(4, G)
    lay.quant_sync()
    return lay, ref, q


def test_decode_quant_scales_that_grow_and_spread(B):
    """Value scales that grow by 2^14 along the sequence (the fixed-point unit of the weights has to follow them,
    folding what was accumulated under the old unit) and key channels whose scales spread over 2^10 (the digits of
    q' s are taken relative to the largest channel of a block)."""
    B_, H, d, r, G, n = 2, 2, 128, 80, 32, 2048 + 64
    k_gain = [2.0 ** -(c // 8) for c in range(r)]
    v_gain = [2.0 ** (i // 150 - 14) for i in range(n)]          # the last rows, which carry the output, have gain 1
    lay, ref, q = scaled_case(B, B_, H, d, r, n, 177, G, k_gain, v_gain)
    out = lay.decode_quant(q)
    lay.poll_status()
    res = ref.decode_quant(to_np(q), 4, G)
    want = np.stack([np.stack([res[(b, h)] for h in range(H)]) for b in range(B_)])[:, None]
    assert_close(out, want, BF16, "growing value scales, spread key scales")


def test_decode_quant_one_cta_over_more_blocks_than_one_fold(B):
    """One CTA per unit over 140 000 rows: every warp meets more blocks than the integer accumulators may take
    before they are folded into fp32, so the periodic fold runs."""
    B_, H, d, r, G, n = 1, 1, 128, 80, 32, 140000
    lay, ref, q = scaled_case(B, B_, H, d, r, n, 178, G, [1.0] * r, [1.0] * n)
    lay.set_option(B.EA_OPT_DECODE_CTAS, 1)
    out = lay.decode_quant(q)
    lay.poll_status()
    res = ref.decode_quant(to_np(q), 4, G)
    want = np.stack([np.stack([res[(b, h)] for h in range(H)]) for b in range(B_)])[:, None]
    assert_close(out, want, BF16, "one CTA, 1094 stages")


def test_decode_quant_merged_weight_flags(B):
    B_, H, d, G, n = 2, 2, 128, 32, 500
    lay, ref, q, _ = fill_both(B, B_, H, d, [80, 56], [72, 80], n, n, 175, G)
    lay.quant_sync()
    low = lay.decode_quant(q, out_lowrank=True)
    res = ref.decode_quant(to_np(q), 4, G, lowrank_out=True)
    for b in range(B_):
        for h in range(H):
            r = res[(b, h)].shape[0]
            assert_close(low[b, 0, lay.offs_v[h]:lay.offs_v[h] + r], res[(b, h)], BF16, "lowrank out")
    # rank-space query: q U^K rounded to bf16 on the host; the oracle gets the same rounded q' lifted back
    qn = to_np(q)
    qp = torch.zeros((B_, 1, lay.offs_k[-1]), dtype=BF16)
    q_back = np.zeros_like(qn)
    for h in range(H):
        U = ref.U_K[h]
        y = torch.from_numpy(qn[:, 0, h, :] @ U).to(BF16)
        qp[:, 0, lay.offs_k[h]:lay.offs_k[h] + U.shape[1]] = y
        q_back[:, 0, h, :] = y.double().numpy() @ U.T          # U^T U = I: projecting this gives y again
    out = lay.decode_quant(qp.cuda(), q_preprojected=True)
    res2 = ref.decode_quant(q_back, 4, G)
    want = np.stack([np.stack([res2[(b, h)] for h in range(H)]) for b in range(B_)])[:, None]
    assert_close(out, want, BF16, "preprojected q")


def test_quant_argument_checks(B):
    U_k, U_v, q, k, v = make_case(1, 1, 64, [32], [32], 64, BF16, seed_cfg=176)
    lay = B.EigenAttnLayer(1, 1, 64, 64, BF16, U_k, U_v)
    with pytest.raises(B.EigenAttnError):
        lay.decode_quant(q)                                   # nothing attached
    with pytest.raises(B.EigenAttnError):
        lay.quant_bytes(2, 32)                                # 3- and 4-bit codes are built
    with pytest.raises(B.EigenAttnError):
        lay.quant_bytes(4, 48)                                # group must be 16, 32, 64 or 128
    lay.quant_attach(4, 32)
    with pytest.raises(B.EigenAttnError):
        lay.decode_quant(q)                                   # empty cache
    lay32 = B.EigenAttnLayer(1, 1, 64, 64, torch.float32, U_k, U_v)
    with pytest.raises(B.EigenAttnError):
        lay32.quant_bytes(4, 32)                              # 16-bit layers only
    # storage per element of whole blocks: bits + 16/G bits for keys (Table 8's accounting), both precisions
    _, bb, ks_off, vc_off, _ = lay.quant_layout(0)
    assert vc_off * 8 / (32 * 32) == 4 + 16 / 32
    for bits, G in ((3, 128), (3, 32), (3, 64), (4, 16), (4, 128), (4, 32)):       # the Eigen Attention rows of Table 8
        U_k, U_v, *_ = make_case(1, 2, 128, [80, 80], [80, 80], 256, BF16, seed_cfg=176)
        lay2 = B.EigenAttnLayer(1, 2, 128, 256, BF16, U_k, U_v)
        lay2.quant_attach(bits, G)
        _, bb, ks_off, vc_off, vs_off = lay2.quant_layout(0)
        assert vc_off == kq.quant_cache_bytes(G * 80, bits, G)                        # keys: bits + 16/G per element
        assert (bb - vc_off) * 8 == G * 80 * bits + 16 * G * -(-80 // G)               # values: one scale per started group
        table, blocks = 256, 256 // G                                                   # per-head table (padded), blocks per sequence
        assert lay2.quant_bytes(bits, G) == table + 2 * ((blocks * bb + 255) // 256 * 256)
