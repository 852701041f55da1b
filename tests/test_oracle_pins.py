"""Pins for the fp64 oracle: each test checks it against something other than itself --
a library attention routine applied to the paper's d_h-wide low-rank inputs, brute-force
Python loops, closed-form special cases, and the numbers the paper prints."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import eigen_attention as orc
from paper_2408_05646_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_case(seed, n, d_h, r_k, r_v, T=1):
    rng = np.random.default_rng(seed)
    U_K = synth.orthonormal_basis(d_h, r_k, seed + 1)
    U_V = synth.orthonormal_basis(d_h, r_v, seed + 2)
    Q = rng.standard_normal((T, d_h))
    K = rng.standard_normal((n, d_h))
    V = rng.standard_normal((n, d_h))
    return Q, K, V, U_K, U_V


def sdpa(Q, K, V, causal):
    """Library softmax attention in fp64 (default scale 1/sqrt(last dim of Q))."""
    q = torch.from_numpy(Q)[None, None]
    k = torch.from_numpy(K)[None, None]
    v = torch.from_numpy(V)[None, None]
    return torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=causal)[0, 0].numpy()


def brute_attention(q, K, V, scale):
    """Textbook softmax attention for one query with Python loops and math.exp."""
    n = len(K)
    s = [sum(q[c] * K[j][c] for c in range(len(q))) * scale for j in range(n)]
    m = max(s)
    e = [math.exp(x - m) for x in s]
    z = sum(e)
    return [sum(e[j] / z * V[j][c] for j in range(n)) for c in range(len(V[0]))]


# ---- P1: full rank reduces to standard attention (Eq. 2/3) -------------------------------

@pytest.mark.parametrize("basis", ["identity", "orthogonal"])
def test_full_rank_equals_standard_attention(basis):
    d_h, n = 8, 11
    Q, K, V, U_K, U_V = rand_case(3, n, d_h, d_h, d_h, T=n)
    if basis == "identity":
        U_K = np.eye(d_h)
        U_V = np.eye(d_h)
    # decode: brute-force loops
    got = orc.decode_head(Q[0], K, V, U_K, U_V)
    ref = brute_attention(Q[0].tolist(), K.tolist(), V.tolist(), 1.0 / math.sqrt(d_h))
    assert np.abs(got - np.array(ref)).max() < 1e-12
    # causal prefill: library routine
    got = orc.prefill_head(Q, K, V, U_K, U_V)
    assert np.abs(got - sdpa(Q, K, V, True)).max() < 1e-12


# ---- P2: rank-space form == Eq. 7 first line evaluated on the d_h-wide Q', K', V' of Eq. 6 ---

@pytest.mark.parametrize("d_h,r_k,r_v,n", [(16, 5, 9, 23), (64, 32, 32, 70), (128, 80, 48, 33)])
def test_rank_space_equals_library_attention_on_lowrank_inputs(d_h, r_k, r_v, n):
    Q, K, V, U_K, U_V = rand_case(7 + d_h, n, d_h, r_k, r_v, T=n)
    Qp = Q @ U_K @ U_K.T            # Eq. 6
    Kp = K @ U_K @ U_K.T
    Vp = V @ U_V @ U_V.T
    # causal, all queries
    ref = sdpa(Qp, Kp, Vp, True)    # scale 1/sqrt(d_h): the last dim of Q' is d_h
    got = orc.prefill_head(Q, K, V, U_K, U_V)
    assert np.abs(got - ref).max() < 1e-12
    # decode: one query against all n rows
    ref1 = sdpa(Qp[-1:], Kp, Vp, False)[0]
    got1 = orc.decode_head(Q[-1], K, V, U_K, U_V)
    assert np.abs(got1 - ref1).max() < 1e-12


def test_projected_scores_identity_and_orthonormality():
    d_h, r, n = 32, 12, 9
    Q, K, V, U_K, U_V = rand_case(11, n, d_h, r, r, T=4)
    assert np.abs(U_K.T @ U_K - np.eye(r)).max() <= 1e-12
    assert np.abs(U_V.T @ U_V - np.eye(r)).max() <= 1e-12
    lhs = orc.to_rank_space(Q, U_K) @ orc.to_rank_space(K, U_K).T
    rhs = Q @ (U_K @ U_K.T) @ K.T
    assert np.abs(lhs - rhs).max() < 1e-12


def test_scale_is_sqrt_d_head_not_sqrt_r():
    # With r < d_h a 1/sqrt(r) scale would change the result; the library routine on the
    # d_h-wide inputs uses 1/sqrt(d_h) by construction.
    d_h, r, n = 16, 4, 12
    Q, K, V, U_K, U_V = rand_case(5, n, d_h, r, r)
    Kp, Vp, qp = K @ U_K, V @ U_V, Q[0] @ U_K
    wrong = np.array(brute_attention(qp.tolist(), Kp.tolist(), Vp.tolist(), 1.0 / math.sqrt(r))) @ U_V.T
    right = np.array(brute_attention(qp.tolist(), Kp.tolist(), Vp.tolist(), 1.0 / math.sqrt(d_h))) @ U_V.T
    got = orc.decode_head(Q[0], K, V, U_K, U_V)
    assert np.abs(got - right).max() < 1e-12
    assert np.abs(got - wrong).max() > 1e-3


# ---- P3: softmax rows, Table 1 counters -----------------------------------------------------

def test_softmax_rows_sum_to_one_and_match_bruteforce():
    rng = np.random.default_rng(0)
    S = rng.standard_normal((7, 13)) * 30
    P = orc.softmax_rows(S)
    assert np.abs(P.sum(axis=1) - 1).max() < 1e-14
    for i in range(7):
        m = max(S[i])
        e = [math.exp(x - m) for x in S[i]]
        assert np.abs(P[i] - np.array(e) / sum(e)).max() < 1e-15


def read_table1():
    rows = {}
    with open(os.path.join(GOLDEN, "table1_closed_forms.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, std, eig = line.split()
            rows[name] = (std, eig)
    return rows


@pytest.mark.parametrize("wl", list(synth.WORKLOADS.values()), ids=lambda w: w.name)
def test_table1_closed_forms_hold_for_every_workload(wl):
    rows = read_table1()
    ranks = synth.draw_ranks(wl.n_heads, wl.ranks, wl.index)
    d = wl.n_heads * wl.d_head
    R = sum(ranks)
    n = wl.context + 1
    env = {"n": n, "d": d, "r": R}
    std = orc.table1_standard(n, d)
    eig = orc.table1_eigen(n, d, R)
    for name, (e_std, e_eig) in rows.items():
        assert std[name] == eval(e_std, {}, env)
        assert eig[name] == eval(e_eig, {}, env)
    # the counters of a (small) run of the stateful oracle reproduce the per-token closed forms
    n_small, B = 6, 2
    U_K = synth.make_bases(wl.d_head, ranks, wl.index, "U_K")
    U_V = synth.make_bases(wl.d_head, ranks, wl.index, "U_V")
    lay = orc.LayerOracle(B, wl.n_heads, wl.d_head, U_K, U_V)
    rng = np.random.default_rng(1)
    k = rng.standard_normal((B, n_small, wl.n_heads, wl.d_head))
    v = rng.standard_normal((B, n_small, wl.n_heads, wl.d_head))
    lay.append_kv(k, v)
    assert lay.cache_elements == B * eval(rows["kv_cache"][1], {}, {"n": n_small, "d": d, "r": R})
    pm0 = lay.projection_macs
    assert pm0 == B * n_small * 2 * wl.d_head * R            # K and V projections, un-merged form
    lay.decode(rng.standard_normal((B, 1, wl.n_heads, wl.d_head)))
    assert lay.attention_macs == B * 2 * n_small * R          # the 2.n.r term of Table 1
    # q projection + lift: with K/V projections this is 4 * d_h * r per head per token
    assert lay.projection_macs - pm0 == B * 2 * wl.d_head * R


# ---- P4: printed cache sizes ------------------------------------------------------------------

def test_kv_cache_sizes_printed_in_paper():
    with open(os.path.join(GOLDEN, "kv_cache_sizes.txt")) as f:
        lines = [l.split() for l in f if l.strip() and not l.startswith("#")]
    assert len(lines) >= 16
    for label, b, n, d, L, bits, ratio, printed, tol in lines:
        gib = orc.kv_cache_bits(int(b), int(n), int(d), int(L), int(bits)) / 8 / 2**30 * float(ratio)
        assert abs(gib - float(printed)) <= float(tol) + 1e-9, (label, gib, printed)
    # weights of the 7B model at 16 bit: ~14 GB (Section 1); 6.74e9 parameters
    assert abs(6.74e9 * 2 / 1e9 - 14) < 0.6
    # the Llama-2-7B-shaped decode workload: one layer at r = 80 of 128 is 5 GiB
    wl = synth.WORKLOADS["llama2_7b_b16_n32k"]
    per_layer = orc.kv_cache_bits(wl.batch, wl.context, wl.n_heads * wl.d_head, 1, 16) / 8
    assert per_layer == 8 * 2**30
    assert per_layer * 80 // 128 == 5 * 2**30


# ---- P5: closed-form special cases -----------------------------------------------------------

def test_special_cases():
    d_h, r_k, r_v, n = 16, 6, 7, 10
    Q, K, V, U_K, U_V = rand_case(21, n, d_h, r_k, r_v)
    q = Q[0]
    P_V = U_V @ U_V.T
    # n = 1: the output is the projection of v, whatever q is
    out = orc.decode_head(q, K[:1], V[:1], U_K, U_V)
    assert np.abs(out - V[0] @ P_V).max() < 1e-12
    # q = 0: uniform weights
    out = orc.decode_head(np.zeros(d_h), K, V, U_K, U_V)
    assert np.abs(out - V.mean(axis=0) @ P_V).max() < 1e-12
    # duplicating every cached row changes nothing
    a = orc.decode_head(q, K, V, U_K, U_V)
    b = orc.decode_head(q, np.concatenate([K, K]), np.concatenate([V, V]), U_K, U_V)
    assert np.abs(a - b).max() < 1e-12
    # adding a fixed vector to every key shifts all scores equally
    c = orc.decode_head(q, K + rand_case(22, 1, d_h, 1, 1)[1], V, U_K, U_V)
    assert np.abs(a - c).max() < 1e-11
    # one dominant key: the output tends to the projection of its value row
    j = 4
    kj = (K[j] @ U_K) @ U_K.T
    out = orc.decode_head(400.0 * kj / np.linalg.norm(kj) * 1.0, K, V, U_K, U_V)
    s = (K @ U_K) @ (U_K.T @ (400.0 * kj / np.linalg.norm(kj))) / math.sqrt(d_h)
    if s.argmax() == j and (np.sort(s)[-1] - np.sort(s)[-2]) > 40:
        assert np.abs(out - V[j] @ P_V).max() < 1e-9
    # a key orthogonal to span(U_K) is invisible to the scores
    w = np.linalg.svd(U_K, full_matrices=True)[0][:, -1]       # in the orthogonal complement
    assert np.abs(w @ U_K).max() < 1e-12
    K2 = K.copy()
    K2[3] += 5.0 * w
    d_out = orc.decode_head(q, K2, V, U_K, U_V)
    assert np.abs(a - d_out).max() < 1e-11


def test_one_hot_limit_is_reached():
    d_h, r, n = 8, 8, 6
    rng = np.random.default_rng(2)
    K = np.eye(n, d_h) * 10
    V = rng.standard_normal((n, d_h))
    U = np.eye(d_h)
    out = orc.decode_head(K[2] * 10, K, V, U, U)
    assert np.abs(out - V[2]).max() < 1e-9


# ---- P6: consistency of the stateful layer ------------------------------------------------------

def make_layer(seed, B, H, d_h, ranks_k, ranks_v, tracked=None):
    U_K = [synth.orthonormal_basis(d_h, r, seed + 10 + h) for h, r in enumerate(ranks_k)]
    U_V = [synth.orthonormal_basis(d_h, r, seed + 100 + h) for h, r in enumerate(ranks_v)]
    return orc.LayerOracle(B, H, d_h, U_K, U_V, tracked), U_K, U_V


def test_layer_matches_per_head_definition_and_append_splits():
    B, H, d_h, T = 2, 3, 16, 7
    rk, rv = [4, 9, 16], [7, 3, 12]
    rng = np.random.default_rng(9)
    q = rng.standard_normal((B, T, H, d_h))
    k = rng.standard_normal((B, T, H, d_h))
    v = rng.standard_normal((B, T, H, d_h))
    lay1, U_K, U_V = make_layer(1, B, H, d_h, rk, rv)
    lay1.append_kv(k, v)
    lay2, _, _ = make_layer(1, B, H, d_h, rk, rv)
    for t in range(T):
        lay2.append_kv(k[:, t:t + 1], v[:, t:t + 1])
    o1 = lay1.decode_dense(q[:, -1:])
    o2 = lay2.decode_dense(q[:, -1:])
    assert np.abs(o1 - o2).max() < 1e-13     # BLAS may block a T-row product differently
    for b in range(B):
        for h in range(H):
            ref = orc.decode_head(q[b, -1, h], k[b, :, h], v[b, :, h], U_K[h], U_V[h])
            assert np.abs(o1[b, 0, h] - ref).max() < 1e-13
    # prefill: last row == decode after append; row t == decode over the first t+1 rows
    lay3, _, _ = make_layer(1, B, H, d_h, rk, rv)
    P = lay3.prefill_dense(q, k, v)
    assert np.abs(P[:, -1:] - o1).max() < 1e-13
    for b in range(B):
        for h in range(H):
            ref = orc.prefill_head(q[b, :, h], k[b, :, h], v[b, :, h], U_K[h], U_V[h])
            assert np.abs(P[b, :, h] - ref).max() < 1e-13
    # chunked prefill (len0 > 0) equals one prefill
    lay4, _, _ = make_layer(1, B, H, d_h, rk, rv)
    Pa = lay4.prefill_dense(q[:, :3], k[:, :3], v[:, :3])
    Pb = lay4.prefill_dense(q[:, 3:], k[:, 3:], v[:, 3:])
    assert np.abs(np.concatenate([Pa, Pb], axis=1) - P).max() < 1e-13


def test_zero_padded_basis_columns_and_head_permutation():
    B, H, d_h, n = 1, 2, 8, 5
    rng = np.random.default_rng(4)
    q = rng.standard_normal((B, 1, H, d_h))
    k = rng.standard_normal((B, n, H, d_h))
    v = rng.standard_normal((B, n, H, d_h))
    lay, U_K, U_V = make_layer(2, B, H, d_h, [3, 5], [4, 2])
    lay.append_kv(k, v)
    o = lay.decode_dense(q)
    pad = lambda U, c: np.concatenate([U, np.zeros((d_h, c))], axis=1)
    layp = orc.LayerOracle(B, H, d_h, [pad(U_K[0], 5), pad(U_K[1], 3)], [pad(U_V[0], 4), pad(U_V[1], 6)])
    layp.append_kv(k, v)
    assert np.abs(layp.decode_dense(q) - o).max() < 1e-13
    perm = [1, 0]
    layq = orc.LayerOracle(B, H, d_h, [U_K[i] for i in perm], [U_V[i] for i in perm])
    layq.append_kv(k[:, :, perm], v[:, :, perm])
    assert np.abs(layq.decode_dense(q[:, :, perm]) - o[:, :, perm]).max() < 1e-13


def test_tracked_subset_equals_full_state():
    B, H, d_h, n = 3, 4, 8, 6
    rng = np.random.default_rng(6)
    q = rng.standard_normal((B, 1, H, d_h))
    k = rng.standard_normal((B, n, H, d_h))
    v = rng.standard_normal((B, n, H, d_h))
    full, _, _ = make_layer(3, B, H, d_h, [4] * H, [5] * H)
    full.append_kv(k, v)
    sub, _, _ = make_layer(3, B, H, d_h, [4] * H, [5] * H, tracked=[(0, 1), (2, 3)])
    sub.append_kv(k, v)
    of, os_ = full.decode(q), sub.decode(q)
    for u in [(0, 1), (2, 3)]:
        assert np.array_equal(of[u], os_[u])


def test_append_unit_rows_equals_append_kv_and_the_per_head_definition():
    # The unit-by-unit hand-over used for large workloads: same state, counters and outputs as append_kv on the
    # same rows, in chunks, with and without a storage rounding; and the outputs equal the stateless per-head
    # definition on the raw rows (itself pinned by library attention above), so a wrong basis, a skipped
    # storage hook or rows filed under another unit cannot pass.
    B, H, d_h, n = 3, 4, 16, 11
    rk, rv = [4, 9, 16, 7], [7, 3, 12, 5]          # every head its own ranks: a swapped basis changes shapes or values
    rng = np.random.default_rng(12)
    q = rng.standard_normal((B, 1, H, d_h))
    k = rng.standard_normal((B, n, H, d_h))
    v = rng.standard_normal((B, n, H, d_h))
    tracked = [(0, 1), (2, 3), (1, 0)]
    half = lambda a: a.astype(np.float16).astype(np.float64)      # a 16-bit storage format (Section 2, p = 16)
    for storage in (None, half):
        a, U_K, U_V = make_layer(5, B, H, d_h, rk, rv, tracked=tracked)
        b, _, _ = make_layer(5, B, H, d_h, rk, rv, tracked=tracked)
        a.storage = b.storage = storage
        a.append_kv(k, v)
        for (bb, hh) in tracked:                                   # two chunks per unit, units in another order
            b.append_unit_rows((bb, hh), k[bb, :4, hh], v[bb, :4, hh])
        for (bb, hh) in reversed(tracked):
            b.append_unit_rows((bb, hh), k[bb, 4:, hh], v[bb, 4:, hh])
        assert b.len == 0                                          # the caller advances the length
        b.set_len(n)
        assert a.cache_elements == b.cache_elements == sum(n * (rk[h] + rv[h]) for _, h in tracked)
        assert a.projection_macs == b.projection_macs
        oa, ob = a.decode(q), b.decode(q)
        for u in tracked:
            assert b.Kp[u].shape == (n, rk[u[1]]) and b.Vp[u].shape == (n, rv[u[1]])
            assert np.abs(a.Kp[u] - b.Kp[u]).max() < 1e-14 and np.abs(a.Vp[u] - b.Vp[u]).max() < 1e-14
            assert np.abs(oa[u] - ob[u]).max() < 1e-13
            if storage is None:
                ref = orc.decode_head(q[u[0], 0, u[1]], k[u[0], :, u[1]], v[u[0], :, u[1]], U_K[u[1]], U_V[u[1]])
                assert np.abs(ob[u] - ref).max() < 1e-13
            else:                                                  # the hook really rounded what the unit keeps
                assert np.array_equal(b.Kp[u], half(b.Kp[u])) and np.array_equal(b.Vp[u], half(b.Vp[u]))
                assert np.abs(b.Kp[u] - k[u[0], :, u[1]] @ U_K[u[1]]).max() > 1e-6


def test_paged_rows_equal_contiguous_rows():
    # Paging moves rows, nothing else: scatter through any page table then gather returns the rows, attention over the
    # gathered rows equals attention over the contiguous ones, pages of different sequences never mix, and a
    # two-page example written out by hand fixes the index arithmetic (page = r // page_rows, offset = r % page_rows).
    rng = np.random.default_rng(21)
    page_rows, pages, width, B = 4, 9, 3, 3
    pool = np.full((pages * page_rows, width), np.nan)
    perm = rng.permutation(pages)
    table = [list(perm[0:4]), list(perm[4:6]) + [-1, -1], list(perm[6:9]) + [-1]]
    lens = [14, 7, 9]
    rows = [rng.standard_normal((n, width)) for n in lens]
    for b in range(B):                                   # appended in chunks that straddle page boundaries
        cut = lens[b] // 2 + 1
        orc.paged_scatter(pool, table[b], page_rows, 0, rows[b][:cut])
        orc.paged_scatter(pool, table[b], page_rows, cut, rows[b][cut:])
    for b in range(B):
        assert np.array_equal(orc.paged_gather(pool, table[b], page_rows, lens[b]), rows[b])
    written = int(np.isfinite(pool[:, 0]).sum())
    assert written == sum(lens)                          # no row written twice, none outside the sequences' pages
    ident = list(range(pages))
    flat = rng.standard_normal((pages * page_rows, width))
    assert np.array_equal(orc.paged_gather(flat, ident, page_rows, 30), flat[:30])       # identity table = contiguous
    hand = np.arange(16, dtype=np.float64).reshape(8, 2)                                  # 2 pages of 4 rows
    got = orc.paged_gather(hand, [1, 0], 4, 6)                                            # logical rows 0..3 in page 1, 4..5 in page 0
    assert np.array_equal(got, hand[[4, 5, 6, 7, 0, 1]])
    with pytest.raises(AssertionError):
        orc.paged_gather(pool, table[1], page_rows, 9)                                    # row 8 is in an unmapped page
    # attention over rows kept in pages = attention over the same rows kept contiguously
    d_h, r = 8, 5
    U_K, U_V = synth.orthonormal_basis(d_h, r, 31), synth.orthonormal_basis(d_h, r, 32)
    K, V, q = rng.standard_normal((11, d_h)), rng.standard_normal((11, d_h)), rng.standard_normal(d_h)
    poolK, poolV = np.zeros((3 * 4, d_h)), np.zeros((3 * 4, d_h))
    orc.paged_scatter(poolK, [2, 0, 1], 4, 0, K)
    orc.paged_scatter(poolV, [2, 0, 1], 4, 0, V)
    a = orc.decode_head(q, orc.paged_gather(poolK, [2, 0, 1], 4, 11), orc.paged_gather(poolV, [2, 0, 1], 4, 11), U_K, U_V)
    assert np.array_equal(a, orc.decode_head(q, K, V, U_K, U_V))


# ---- P7: tiny brute force with explicit d_h x d_h projectors (Eq. 7, second line) ---------------

@pytest.mark.parametrize("n", [1, 2, 5])
def test_tiny_bruteforce_full_space(n):
    d_h, r = 4, 2
    Q, K, V, U_K, U_V = rand_case(40 + n, n, d_h, r, r, T=n)
    PK = (U_K @ U_K.T).tolist()
    PV = (U_V @ U_V.T).tolist()
    for t in range(n):
        qP = [sum(Q[t][a] * PK[a][c] for a in range(d_h)) for c in range(d_h)]        # q U U^T
        VP = [[sum(V[j][a] * PV[a][c] for a in range(d_h)) for c in range(d_h)] for j in range(t + 1)]
        ref = brute_attention(qP, K[:t + 1].tolist(), VP, 1.0 / math.sqrt(d_h))      # ... K^T, V U U^T
        got = orc.prefill_head(Q, K, V, U_K, U_V)[t]
        assert np.abs(got - np.array(ref)).max() < 1e-13


# ---- the seeded generator ----------------------------------------------------------------------

def test_generator_is_seeded_and_shaped():
    wl = synth.WORKLOADS["tiny_fp32"]
    W = synth.mixing_matrices(wl.n_heads, wl.rho, wl.d_head, wl.index, "W_K")
    a = synth.lowrank_rows(W, 1, 16, wl.sigma, wl.index, "K", dtype=torch.float32)
    b = synth.lowrank_rows(W, 1, 16, wl.sigma, wl.index, "K", dtype=torch.float32)
    c = synth.lowrank_rows(W, 1, 16, wl.sigma, wl.index, "K", chunk=1, dtype=torch.float32)
    assert a.shape == (1, 16, wl.n_heads, wl.d_head) and torch.equal(a, b) and not torch.equal(a, c)
    big = synth.lowrank_rows(W, 2, 2000, wl.sigma, wl.index, "V", dtype=torch.float32)
    assert abs(float(big.var()) - 1.0) < 0.1
    sv = torch.linalg.svdvals(big[0, :, 0, :].double())
    assert sv[wl.rho - 1] > 5 * sv[wl.rho]          # rank-rho signal over a small noise floor
    ranks = synth.draw_ranks(32, (48, 64, 80, 96, 112), 3)
    assert ranks == synth.draw_ranks(32, (48, 64, 80, 96, 112), 3) and len(set(ranks)) > 1
    U = synth.make_bases(128, ranks, 3, "U_K")
    assert all(u.dtype == np.float32 and u.shape == (128, r) for u, r in zip(U, ranks))
    units = synth.sample_units(16, 32, ranks, 64, 3)
    assert len(units) >= 64 and (0, 0) in units and (15, 31) in units and len(set(units)) == len(units)
