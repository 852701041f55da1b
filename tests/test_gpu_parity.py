"""GPU parity: the CUDA path (through the C ABI) against the fp64 oracle, element by element, on the
same seeded inputs.  Sizes span several shared-memory tiles, ragged tails and several CTAs' splits."""
import numpy as np
import pytest
import torch

from helpers import assert_close, make_case, oracle_layer, to_np

pytestmark = pytest.mark.gpu

BF16, FP32 = torch.bfloat16, torch.float32


@pytest.fixture(scope="module")
def B():
    from paper_2408_05646_b200 import build
    build.build_library()
    from paper_2408_05646_b200 import binding
    return binding


def run_decode_case(B_, bnd, H, d_head, rk, rv, n, dtype, seed=90, q_scale=1.0, opts=None):
    U_k, U_v, q, k, v = make_case(B_, H, d_head, rk, rv, n, dtype, seed_cfg=seed, q_scale=q_scale)
    lay = bnd.EigenAttnLayer(B_, H, d_head, n + 4, dtype, U_k, U_v)
    for o, val in (opts or {}).items():
        lay.set_option(o, val)
    lay.append_kv(k, v)
    out = lay.decode(q)
    lay.poll_status()
    ref = oracle_layer(B_, H, d_head, U_k, U_v)
    ref.append_kv(to_np(k), to_np(v))
    expect = ref.decode_dense(to_np(q))
    assert_close(out, expect, dtype, f"decode B{B_} H{H} d{d_head} n{n}")
    return lay, ref, (U_k, U_v, q, k, v), out


def test_tiny_fp32_workload(B):
    # the small reference workload: 1 x 4 heads, d_head 64, r 32, 512 cached rows + 1 new token
    from paper_2408_05646_b200 import synth
    wl = synth.WORKLOADS["tiny_fp32"]
    ranks = synth.draw_ranks(wl.n_heads, wl.ranks, wl.index)
    U_k = synth.make_bases(wl.d_head, ranks, wl.index, "U_K")
    U_v = synth.make_bases(wl.d_head, ranks, wl.index, "U_V")
    W_k = synth.mixing_matrices(wl.n_heads, wl.rho, wl.d_head, wl.index, "W_K")
    W_v = synth.mixing_matrices(wl.n_heads, wl.rho, wl.d_head, wl.index, "W_V")
    k = synth.lowrank_rows(W_k, wl.batch, wl.context + 1, wl.sigma, wl.index, "K", dtype=FP32, device="cuda:0")
    v = synth.lowrank_rows(W_v, wl.batch, wl.context + 1, wl.sigma, wl.index, "V", dtype=FP32, device="cuda:0")
    q = synth.gaussian_query(wl.batch, wl.n_heads, wl.d_head, wl.q_scale, wl.index, dtype=FP32, device="cuda:0")
    lay = B.EigenAttnLayer(wl.batch, wl.n_heads, wl.d_head, wl.context + 1, FP32, U_k, U_v)
    lay.append_kv(k[:, :wl.context], v[:, :wl.context])
    out = lay.decode_step(q, k[:, wl.context:], v[:, wl.context:])      # one new token appended, then attended
    assert lay.len == wl.context + 1
    ref = oracle_layer(wl.batch, wl.n_heads, wl.d_head, U_k, U_v)
    ref.append_kv(to_np(k), to_np(v))
    assert_close(out, ref.decode_dense(to_np(q)), FP32, "tiny fp32")
    # cache contents == the oracle's projected rows
    for h in range(wl.n_heads):
        Kc = lay.cache_rows(h, "k")[:, :wl.context + 1, :ranks[h]]
        Vc = lay.cache_rows(h, "v")[:, :wl.context + 1, :ranks[h]]
        for b in range(wl.batch):
            assert_close(Kc[b], ref.Kp[(b, h)], FP32, "K' rows")
            assert_close(Vc[b], ref.Vp[(b, h)], FP32, "V' rows")


@pytest.mark.parametrize("dtype", [BF16, FP32])
@pytest.mark.parametrize("r", [8, 16, 32, 48, 64, 80, 96, 112, 128])
def test_decode_uniform_ranks(B, dtype, r):
    # every lane-pair width class and both bank-rotation cases; n spans tiles with a ragged tail
    run_decode_case(2, B, 3, 128, [r] * 3, [r] * 3, 700, dtype)


@pytest.mark.parametrize("dtype", [BF16, FP32])
def test_decode_heterogeneous_and_unpadded_ranks(B, dtype):
    rk = [5, 48, 80, 33, 112, 64, 17, 96]
    rv = [9, 64, 80, 128, 40, 7, 100, 24]
    lay, ref, _, _ = run_decode_case(3, B, 8, 128, rk, rv, 1111, dtype)
    # padding columns of the cache hold zeros
    for h in (0, 6):
        assert float(lay.cache_rows(h, "k")[:, :1111, rk[h]:].abs().max()) == 0.0
        assert float(lay.cache_rows(h, "v")[:, :1111, rv[h]:].abs().max()) == 0.0


@pytest.mark.parametrize("n", [1, 2, 15, 16, 17, 127, 128, 129, 513])
def test_decode_short_contexts(B, n):
    run_decode_case(2, B, 4, 64, [32] * 4, [24] * 4, n, BF16)
    run_decode_case(1, B, 2, 64, [32] * 2, [32] * 2, n, FP32)


@pytest.mark.parametrize("d_head", [8, 64, 96, 128])
def test_decode_head_dims(B, d_head):
    r = max(8, d_head // 2)
    run_decode_case(2, B, 2, d_head, [r, d_head], [d_head, r], 300, FP32)


def test_long_context_split_over_all_ctas_matches_single_cta(B):
    # few units, long context: every unit is split over many CTAs and merged by the combine kernel
    B_, H, n = 1, 2, 40000
    lay, ref, (U_k, U_v, q, k, v), out = run_decode_case(B_, B, H, 128, [64, 64], [64, 64], n, BF16)
    for ctas, tile, stages in [(1, 0, 0), (7, 64, 2), (148, 32, 3), (300, 128, 0)]:
        lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        lay.set_option(B.EA_OPT_DECODE_TILE_ROWS, tile)
        lay.set_option(B.EA_OPT_DECODE_STAGES, stages)
        o2 = lay.decode(q)
        lay.poll_status()
        assert_close(o2, ref.decode_dense(to_np(q)), BF16, f"ctas={ctas}")
        assert float((o2.float() - out.float()).abs().max()) < 2e-2


def test_split_consistency_fp32(B):
    # the split-KV result is an exact re-association: in fp32 mode any CTA count agrees to 1e-5
    B_, H, n = 2, 3, 9000
    lay, ref, (U_k, U_v, q, k, v), out = run_decode_case(B_, B, H, 64, [32, 16, 48], [32, 64, 8], n, FP32)
    for ctas in (1, 2, 5, 33, 148, 512):
        lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        o2 = lay.decode(q)
        assert_close(o2, ref.decode_dense(to_np(q)), FP32, f"ctas={ctas}")


@pytest.mark.parametrize("fused", [1, 0])
def test_append_T_tokens_equals_T_single_appends_and_64_steps(B, fused):
    # long-context workload shape in miniature: 64 consecutive single-token append+decode steps,
    # as one fused launch per step and as separate append / attention / merge launches
    B_, H, d, r, n0, steps = 2, 4, 128, 64, 1000, 64
    U_k, U_v, q, k, v = make_case(B_, H, d, [r] * H, [r] * H, n0 + steps, BF16, seed_cfg=94, T_q=steps)
    a = B.EigenAttnLayer(B_, H, d, n0 + steps, BF16, U_k, U_v)
    a.set_option(B.EA_OPT_DECODE_FUSED, fused)
    b = B.EigenAttnLayer(B_, H, d, n0 + steps, BF16, U_k, U_v)
    a.append_kv(k[:, :n0], v[:, :n0])
    b.append_kv(k[:, :n0], v[:, :n0])
    ref = oracle_layer(B_, H, d, U_k, U_v)
    ref.append_kv(to_np(k[:, :n0]), to_np(v[:, :n0]))
    for t in range(steps):
        out = a.decode_step(q[:, t:t + 1], k[:, n0 + t:n0 + t + 1], v[:, n0 + t:n0 + t + 1])
        ref.append_kv(to_np(k[:, n0 + t:n0 + t + 1]), to_np(v[:, n0 + t:n0 + t + 1]))
        if t % 9 == 0 or t == steps - 1:
            assert_close(out, ref.decode_dense(to_np(q[:, t:t + 1])), BF16, f"step {t}")
    b.append_kv(k[:, n0:], v[:, n0:])
    assert a.len == b.len == n0 + steps
    assert torch.equal(a.cache, b.cache)          # identical cache bytes either way


@pytest.mark.parametrize("dtype", [BF16, FP32])
@pytest.mark.parametrize("fused", [1, 0])
def test_decode_step_from_empty_cache_and_hetero_ranks(B, dtype, fused):
    # steps starting at len = 0 (first token attends only to itself), per-head ranks, few and many CTAs
    B_, H, d, steps = 3, 5, 128, 40
    rk, rv = [80, 17, 128, 48, 64], [24, 96, 80, 128, 9]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, steps, dtype, seed_cfg=93, T_q=steps)
    lay = B.EigenAttnLayer(B_, H, d, steps, dtype, U_k, U_v)
    lay.set_option(B.EA_OPT_DECODE_FUSED, fused)
    ref = oracle_layer(B_, H, d, U_k, U_v)
    for t in range(steps):
        if t == 20:
            lay.set_option(B.EA_OPT_DECODE_CTAS, 3)
        out = lay.decode_step(q[:, t:t + 1], k[:, t:t + 1], v[:, t:t + 1])
        ref.append_kv(to_np(k[:, t:t + 1]), to_np(v[:, t:t + 1]))
        assert_close(out, ref.decode_dense(to_np(q[:, t:t + 1])), dtype, f"step {t}")
    assert lay.len == steps
    lay.poll_status()
    # every stored row equals the oracle's projected row
    for h in range(H):
        assert_close(lay.cache_rows(h, "k")[0, :steps, :rk[h]], ref.Kp[(0, h)], dtype, "K' rows")
        assert_close(lay.cache_rows(h, "v")[1, :steps, :rv[h]], ref.Vp[(1, h)], dtype, "V' rows")


def test_fused_and_unfused_steps_agree_on_split_units(B):
    # long context, few units: every unit is split over many CTAs; the last-arriving CTA merges
    B_, H, d, n = 1, 3, 128, 30000
    rk = [64, 80, 112]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rk, n + 1, BF16, seed_cfg=92)
    outs = []
    for fused in (1, 0):
        lay = B.EigenAttnLayer(B_, H, d, n + 1, BF16, U_k, U_v)
        lay.set_option(B.EA_OPT_DECODE_FUSED, fused)
        lay.append_kv(k[:, :n], v[:, :n])
        for rep in range(3):                      # counters must be clean again after every call
            lay.set_len(n)
            o = lay.decode_step(q, k[:, n:], v[:, n:])
        lay.poll_status()
        outs.append(o)
        plain = lay.decode(q)                     # same rows through the non-step entry point
        assert float((plain.float() - o.float()).abs().max()) < 1e-2
    ref = oracle_layer(B_, H, d, U_k, U_v)
    ref.append_kv(to_np(k), to_np(v))
    assert_close(outs[0], ref.decode_dense(to_np(q)), BF16, "fused")
    assert_close(outs[1], ref.decode_dense(to_np(q)), BF16, "unfused")


def test_adversarial_softmax_inputs(B):
    B_, H, d, r, n = 1, 2, 64, 32, 600
    U_k, U_v, q, k, v = make_case(B_, H, d, [r] * H, [r] * H, n, FP32, seed_cfg=95)
    Uk0 = torch.from_numpy(U_k[0]).cuda()
    cases = {}
    # scores increasing with position: a rescale of the running state at every row
    dirn = (Uk0 @ torch.ones(r, device="cuda")).float()
    dirn = dirn / dirn.norm()
    k_inc = k.clone()
    k_inc[0, :, 0, :] = dirn[None, :] * torch.linspace(-40, 40, n, device="cuda")[:, None]
    q_inc = q.clone()
    q_inc[0, 0, 0, :] = dirn * 8.0
    cases["increasing"] = (q_inc, k_inc)
    # one dominant key
    k_dom = k.clone()
    k_dom[0, 77, 1, :] = (Uk0 @ torch.ones(r, device="cuda")) * 3
    q_dom = q.clone()
    q_dom[0, 0, 1, :] = k_dom[0, 77, 1, :] * 4
    cases["dominant"] = (q_dom, k_dom)
    # all-equal scores (q = 0) and very large |scores| (~ +-80 before the softmax)
    cases["uniform"] = (torch.zeros_like(q), k)
    cases["large"] = (q * 60.0, k)
    for name, (qq, kk) in cases.items():
        lay = B.EigenAttnLayer(B_, H, d, n, FP32, U_k, U_v)
        lay.append_kv(kk, v)
        out = lay.decode(qq)
        ref = oracle_layer(B_, H, d, U_k, U_v)
        ref.append_kv(to_np(kk), to_np(v))
        # a score s carries an absolute fp32 error of about |s| * 2^-23 * sqrt(r), which the softmax turns
        # into the same relative error of a weight: with |s| up to ~300 here the bound is 2e-4, not 1e-5
        tol = 2e-4 if name in ("large", "increasing", "dominant") else 1e-5
        assert_close(out, ref.decode_dense(to_np(qq)), FP32, name, fp32_rel=tol)


def test_merged_weight_flags(B):
    # rank-space inputs/outputs for callers whose projection weights already contain U (Eq. 8)
    B_, H, d, n = 2, 3, 64, 257
    rk, rv = [16, 24, 30], [8, 40, 21]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n, FP32, seed_cfg=96)
    lay = B.EigenAttnLayer(B_, H, d, n, FP32, U_k, U_v)
    ref = oracle_layer(B_, H, d, U_k, U_v)
    ref.append_kv(to_np(k), to_np(v))
    # packed rank-space tensors built on the host from the same fp32 bases
    def pack(x, U, offs):
        out = torch.zeros((B_, x.shape[1], offs[-1]), dtype=torch.float32)
        xn = to_np(x)
        for h in range(H):
            y = xn[:, :, h, :] @ U[h].astype(np.float64)
            out[:, :, offs[h]:offs[h] + U[h].shape[1]] = torch.from_numpy(y).float()
        return out.cuda()
    kp, vp, qp = pack(k, U_k, lay.offs_k), pack(v, U_v, lay.offs_v), pack(q, U_k, lay.offs_k)
    lay.append_kv(kp, vp, preprojected=True)
    out = lay.decode(qp, q_preprojected=True)
    assert_close(out, ref.decode_dense(to_np(q)), FP32, "preprojected q,k,v")
    low = lay.decode(q, out_lowrank=True)
    res = ref.decode(to_np(q), lowrank_out=True)
    for b in range(B_):
        for h in range(H):
            got = low[b, 0, lay.offs_v[h]:lay.offs_v[h] + rv[h]]
            assert_close(got, res[(b, h)], FP32, "lowrank out")


def rank_space_inputs(lay, U_k, U_v, q, k, v, dtype):
    """What a layer with merged weights (Eq. 8) hands over: the packed rank-space tensors q U^K, k U^K, v U^V computed
    on the host and rounded to the IO dtype, and the d_head-wide tensors whose projections are exactly those rounded
    rows (x' U^T: since U^T U = I, projecting it returns x'), which is what the oracle receives."""
    def one(x, U, offs):
        xn = to_np(x)
        packed = torch.zeros((x.shape[0], x.shape[1], offs[-1]), dtype=dtype)
        back = np.zeros_like(xn)
        for h in range(len(U)):
            Uh = U[h].astype(np.float64)
            y = torch.from_numpy(xn[:, :, h, :] @ Uh).to(dtype)
            packed[:, :, offs[h]:offs[h] + Uh.shape[1]] = y
            back[:, :, h, :] = y.double().numpy() @ Uh.T
        return packed.cuda(), back
    (qp, q_b), (kp, k_b), (vp, v_b) = one(q, U_k, lay.offs_k), one(k, U_k, lay.offs_k), one(v, U_v, lay.offs_v)
    return qp, kp, vp, q_b, k_b, v_b


@pytest.mark.parametrize("dtype,H,d,rk,rv,T", [
    (FP32, 3, 64, [16, 24, 30], [8, 40, 21], 75),
    (BF16, 4, 128, [80, 48, 128, 64], [80, 112, 8, 64], 300),
])
def test_merged_weight_mode_end_to_end(B, dtype, H, d, rk, rv, T):
    """Eq. 8: a model whose W^Q, W^K, W^V, W^O carry the bases calls prefill and the decode step with rank-space
    q', k', v' and takes o' back in rank space.  Prompt (two chunks), then three generated tokens, all three flags;
    then each input flag alone."""
    B_, steps = 2, 3
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, T + steps, dtype, seed_cfg=98, T_q=T + steps)
    lay = B.EigenAttnLayer(B_, H, d, T + steps, dtype, U_k, U_v, max_prefill_tokens=T)
    qp, kp, vp, q_b, k_b, v_b = rank_space_inputs(lay, U_k, U_v, q, k, v, dtype)
    ref = oracle_layer(B_, H, d, U_k, U_v)
    want = ref.prefill(q_b[:, :T], k_b[:, :T], v_b[:, :T])
    cut = T // 2 + 1
    tol = dict(fp32_rel=2e-5) if dtype == FP32 else {}

    def check_lowrank(got, res, t_axis, what):
        for b in range(B_):
            for h in range(H):
                o = to_np(got[b, :, lay.offs_v[h]:lay.offs_v[h] + rv[h]])
                exp = res[(b, h)]                                   # [T, d_h] (prefill) or [d_h] (decode): back to rank space
                exp = (exp if t_axis else exp[None]) @ U_v[h].astype(np.float64)
                assert_close(torch.from_numpy(o), exp, dtype, f"{what} unit ({b},{h})", **tol)
                pad = got[b, :, lay.offs_v[h] + rv[h]:lay.offs_v[h + 1]]          # padding lanes of the packed output
                assert pad.numel() == 0 or float(pad.float().abs().max()) == 0.0

    a = lay.prefill(qp[:, :cut].contiguous(), kp[:, :cut].contiguous(), vp[:, :cut].contiguous(), out_lowrank=True,
                    q_preprojected=True, kv_preprojected=True)
    c = lay.prefill(qp[:, cut:T].contiguous(), kp[:, cut:T].contiguous(), vp[:, cut:T].contiguous(), out_lowrank=True,
                    q_preprojected=True, kv_preprojected=True)
    lay.poll_status()
    check_lowrank(torch.cat([a, c], dim=1), want, True, "merged prefill")
    for s in range(steps):
        t = T + s
        o = lay.decode_step(qp[:, t:t + 1].contiguous(), kp[:, t:t + 1].contiguous(), vp[:, t:t + 1].contiguous(),
                            q_preprojected=True, kv_preprojected=True, out_lowrank=True)
        ref.append_kv(k_b[:, t:t + 1], v_b[:, t:t + 1])
        check_lowrank(o, ref.decode(q_b[:, t:t + 1]), False, f"merged decode step {s}")
    assert lay.len == T + steps
    # the rows the merged calls stored are the packed rows themselves
    for h in (0, H - 1):
        assert torch.equal(lay.cache_rows(h, "k")[:, :T + steps, :rk[h]], kp[:, :, lay.offs_k[h]:lay.offs_k[h] + rk[h]])
        assert torch.equal(lay.cache_rows(h, "v")[:, :T + steps, :rv[h]], vp[:, :, lay.offs_v[h]:lay.offs_v[h] + rv[h]])
    # one input flag at a time, d_head-wide output
    for qf, kvf in ((True, False), (False, True)):
        lay2 = B.EigenAttnLayer(B_, H, d, T + 1, dtype, U_k, U_v, max_prefill_tokens=T)
        r2 = oracle_layer(B_, H, d, U_k, U_v)
        q_in = qp[:, :T].contiguous() if qf else torch.from_numpy(q_b[:, :T]).to(dtype).cuda()
        k_in = kp[:, :T].contiguous() if kvf else torch.from_numpy(k_b[:, :T]).to(dtype).cuda()
        v_in = vp[:, :T].contiguous() if kvf else torch.from_numpy(v_b[:, :T]).to(dtype).cuda()
        q_ref = q_b[:, :T] if qf else to_np(q_in)
        k_ref = k_b[:, :T] if kvf else to_np(k_in)
        v_ref = v_b[:, :T] if kvf else to_np(v_in)
        got = lay2.prefill(q_in, k_in, v_in, q_preprojected=qf, kv_preprojected=kvf)
        assert_close(got, r2.prefill_dense(q_ref, k_ref, v_ref), dtype, f"prefill q'={qf} kv'={kvf}", **tol)
        t = T
        q1 = qp[:, t:t + 1].contiguous() if qf else torch.from_numpy(q_b[:, t:t + 1]).to(dtype).cuda()
        k1 = kp[:, t:t + 1].contiguous() if kvf else torch.from_numpy(k_b[:, t:t + 1]).to(dtype).cuda()
        v1 = vp[:, t:t + 1].contiguous() if kvf else torch.from_numpy(v_b[:, t:t + 1]).to(dtype).cuda()
        o1 = lay2.decode_step(q1, k1, v1, q_preprojected=qf, kv_preprojected=kvf)
        r2.append_kv(k_b[:, t:t + 1] if kvf else to_np(k1), v_b[:, t:t + 1] if kvf else to_np(v1))
        assert_close(o1, r2.decode_dense(q_b[:, t:t + 1] if qf else to_np(q1)), dtype, f"step q'={qf} kv'={kvf}", **tol)
        lay2.set_option(B.EA_OPT_DECODE_FUSED, 0)                   # the separate-launch form of the same step
        lay2.set_len(T)
        o2 = lay2.decode_step(q1, k1, v1, q_preprojected=qf, kv_preprojected=kvf)
        assert_close(o2, r2.decode_dense(q_b[:, t:t + 1] if qf else to_np(q1)), dtype, f"unfused step q'={qf} kv'={kvf}", **tol)
        lay2.poll_status()


@pytest.mark.parametrize("dtype,H,d,rk,rv,T", [
    (FP32, 2, 64, [32, 20], [16, 40], 75),
    (BF16, 4, 128, [80, 48, 128, 64], [80, 112, 8, 64], 200),
    (BF16, 1, 128, [80], [80], 33),
])
def test_prefill_matches_oracle_and_feeds_decode(B, dtype, H, d, rk, rv, T):
    B_ = 2
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, T + 1, dtype, seed_cfg=97, T_q=T + 1)
    lay = B.EigenAttnLayer(B_, H, d, T + 1, dtype, U_k, U_v, max_prefill_tokens=T)
    out = lay.prefill(q[:, :T], k[:, :T], v[:, :T])
    ref = oracle_layer(B_, H, d, U_k, U_v)
    expect = ref.prefill_dense(to_np(q[:, :T]), to_np(k[:, :T]), to_np(v[:, :T]))
    assert_close(out, expect, dtype, "prefill")
    # the cache the prefill wrote serves the next decode step
    o1 = lay.decode_step(q[:, T:], k[:, T:], v[:, T:])
    ref.append_kv(to_np(k[:, T:]), to_np(v[:, T:]))
    assert_close(o1, ref.decode_dense(to_np(q[:, T:])), dtype, "decode after prefill")


@pytest.mark.parametrize("H,d,rk,rv,T", [
    (1, 128, [80], [80], 128),                       # exactly one query tile and one key tile
    (2, 128, [80, 64], [80, 96], 300),               # several tiles, ragged tail, K and V ranks differ
    (3, 64, [24, 64, 40], [56, 8, 64], 517),         # small d_head, ranks that are not multiples of 16
    (2, 128, [128, 16], [16, 128], 1000),            # widest and narrowest ranks
])
def test_tensor_core_prefill_matches_oracle_and_cuda_core_kernel(B, H, d, rk, rv, T):
    B_ = 2
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, T, BF16, seed_cfg=101, T_q=T)
    ref = oracle_layer(B_, H, d, U_k, U_v)
    expect = ref.prefill_dense(to_np(q), to_np(k), to_np(v))
    outs = {}
    for impl in (2, 3, 1):                           # 2 = tcgen05 (warp-specialised if it fits), 3 = single-tile tcgen05, 1 = CUDA cores
        lay = B.EigenAttnLayer(B_, H, d, T, BF16, U_k, U_v, max_prefill_tokens=T)
        lay.set_option(B.EA_OPT_PREFILL_IMPL, impl)
        outs[impl] = lay.prefill(q, k, v)
        lay.poll_status()
        assert_close(outs[impl], expect, BF16, f"prefill impl {impl}")
    assert float((outs[1].float() - outs[2].float()).abs().max()) < 3e-2
    assert float((outs[3].float() - outs[2].float()).abs().max()) < 3e-2


def test_tensor_core_prefill_chunked_and_lowrank(B):
    B_, H, d, T = 1, 2, 128, 700
    rk, rv = [80, 48], [64, 80]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, T, BF16, seed_cfg=102, T_q=T)
    ref = oracle_layer(B_, H, d, U_k, U_v)
    expect = ref.prefill_dense(to_np(q), to_np(k), to_np(v))
    lay = B.EigenAttnLayer(B_, H, d, T, BF16, U_k, U_v, max_prefill_tokens=400)
    lay.set_option(B.EA_OPT_PREFILL_IMPL, 2)
    cuts = [0, 130, 530, 700]                        # len0 > 0 and not a multiple of the tile
    parts = [lay.prefill(q[:, a:b_].contiguous(), k[:, a:b_].contiguous(), v[:, a:b_].contiguous())
             for a, b_ in zip(cuts[:-1], cuts[1:])]
    lay.poll_status()
    assert_close(torch.cat(parts, dim=1), expect, BF16, "chunked tensor-core prefill")
    lay.set_len(0)
    low = lay.prefill(q[:, :400].contiguous(), k[:, :400].contiguous(), v[:, :400].contiguous(), out_lowrank=True)
    for h in range(H):
        got = to_np(low[0, :, lay.offs_v[h]:lay.offs_v[h] + rv[h]]) @ U_v[h].astype(np.float64).T
        assert np.abs(got - expect[0, :400, h, :]).max() < 2e-2


def test_chunked_prefill_and_lowrank_output(B):
    B_, H, d, T = 1, 2, 64, 90
    rk, rv = [32, 24], [16, 32]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, T, FP32, seed_cfg=98, T_q=T)
    lay = B.EigenAttnLayer(B_, H, d, T, FP32, U_k, U_v, max_prefill_tokens=64)
    o1 = lay.prefill(q[:, :50].contiguous(), k[:, :50].contiguous(), v[:, :50].contiguous())
    o2 = lay.prefill(q[:, 50:].contiguous(), k[:, 50:].contiguous(), v[:, 50:].contiguous())
    ref = oracle_layer(B_, H, d, U_k, U_v)
    expect = ref.prefill_dense(to_np(q), to_np(k), to_np(v))
    assert_close(torch.cat([o1, o2], dim=1), expect, FP32, "chunked prefill")
    lay.set_len(0)
    low = lay.prefill(q[:, :64].contiguous(), k[:, :64].contiguous(), v[:, :64].contiguous(), out_lowrank=True)
    for h in range(H):
        got = to_np(low[0, :, lay.offs_v[h]:lay.offs_v[h] + rv[h]]) @ U_v[h].astype(np.float64).T
        assert np.abs(got - expect[0, :64, h, :]).max() < 1e-5


def test_strided_inputs_and_host_step(B):
    B_, H, d, n = 2, 2, 64, 100
    U_k, U_v, q, k, v = make_case(B_, H, d, [32] * H, [32] * H, n, BF16, seed_cfg=99)
    # q/k/v as slices of a fused [B][T][3][H][d] projection output (non-contiguous batch/token strides)
    fused = torch.stack([k, v, k], dim=2).contiguous()
    ks, vs = fused[:, :, 0], fused[:, :, 1]
    lay = B.EigenAttnLayer(B_, H, d, n + 1, BF16, U_k, U_v)
    lay.append_kv(ks[:, :n - 1], vs[:, :n - 1])
    hq, hk, hv = q.cpu().pin_memory(), k[:, n - 1:].cpu().contiguous().pin_memory(), v[:, n - 1:].cpu().contiguous().pin_memory()
    hout = torch.empty_like(hq).pin_memory()
    lay.decode_step_host(hq, hk, hv, hout)
    ref = oracle_layer(B_, H, d, U_k, U_v)
    ref.append_kv(to_np(k), to_np(v))
    assert_close(hout, ref.decode_dense(to_np(q)), BF16, "host step")
    assert lay.launch_count() == 2          # one append launch, one fused decode-step launch
    # q, k, v adjacent in one pinned buffer (they travel as one copy): same result.  (The three separate pinned
    # tensors above can come out adjacent too, from different allocations: the library must then fall back.)
    lay.set_len(n - 1)
    packed = torch.stack([hq, hk, hv]).pin_memory()
    hout2 = torch.empty_like(hq).pin_memory()
    lay.decode_step_host(packed[0], packed[1], packed[2], hout2)
    assert torch.equal(hout2, hout)


def test_errors_leave_state_unchanged(B):
    B_, H, d = 1, 2, 64
    U_k, U_v, q, k, v = make_case(B_, H, d, [32] * H, [32] * H, 8, BF16, seed_cfg=100)
    lay = B.EigenAttnLayer(B_, H, d, 8, BF16, U_k, U_v, max_prefill_tokens=4, check_orthonormal=True)
    with pytest.raises(B.EigenAttnError) as e:
        lay.decode(q)
    assert e.value.status == B.EA_ERR_SHAPE and "empty" in str(e.value)
    lay.append_kv(k, v)
    with pytest.raises(B.EigenAttnError) as e:
        lay.append_kv(k[:, :1], v[:, :1])
    assert e.value.status == B.EA_ERR_CAPACITY and lay.len == 8
    lay.set_len(0)
    with pytest.raises(B.EigenAttnError) as e:
        lay.prefill(q.expand(B_, 8, H, d).contiguous(), k, v)
    assert e.value.status == B.EA_ERR_CAPACITY and lay.len == 0
    with pytest.raises(B.EigenAttnError):
        lay.set_option(B.EA_OPT_DECODE_TILE_ROWS, 24)
    bad = [u.copy() for u in U_k]
    bad[1][:, 0] *= 1.5
    with pytest.raises(B.EigenAttnError) as e:
        B.EigenAttnLayer(B_, H, d, 8, BF16, bad, U_v, check_orthonormal=True)
    assert e.value.status == B.EA_ERR_NOT_ORTHONORMAL
    lay.poll_status()


@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_peaked_attention_over_heads_that_share_a_slot_size(B, dtype):
    """Heads whose K' and V' widths differ but add up to the same row size, streamed by the same CTA one after
    the other, with sharply peaked weights: an error in a handful of rows (a stale tile layout, a ragged tail)
    shows up here, whereas diffuse weights average it away."""
    B_, H, d, n = 2, 6, 128, 1037
    rk, rv = [48, 64, 80, 96, 64, 48], [96, 80, 64, 48, 80, 96]        # every head: 144 columns per row
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n, dtype, seed_cfg=141, q_scale=6.0)
    from helpers import OraclePair
    lay = B.EigenAttnLayer(B_, H, d, n, dtype, U_k, U_v)
    lay.append_kv(k, v)
    ref = OraclePair(B_, H, d, U_k, U_v, dtype)
    ref.append_kv(to_np(k), to_np(v))
    expect = ref.decode_dense(to_np(q))
    tol = dict(fp32_rel=2e-4) if dtype == FP32 else {}               # scores of a few tens: see the adversarial test
    for ctas, fused in ((0, 1), (1, 1), (2, 0), (5, 1), (12, 1), (37, 0), (148, 1)):
        lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        lay.set_option(B.EA_OPT_DECODE_FUSED, fused)
        assert_close(lay.decode(q), expect, dtype, f"ctas={ctas} fused={fused}", **tol)
    lay.poll_status()


@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_peaked_attention_with_several_tiles_per_ring_slot(B, dtype):
    """Narrow heads put up to four consecutive tiles into one ring slot (one bulk copy).  Pieces start and end at
    any tile, so a slot can hold 1..4 tiles and end with the unit's ragged tail; peaked weights make a row that is
    skipped, read twice or taken from the neighbouring tile visible.  Wide and narrow heads alternate, so the slot
    layout changes from piece to piece."""
    from helpers import OraclePair
    B_, H, d, n = 2, 5, 128, 2077
    rk, rv = [16, 112, 24, 48, 8], [24, 96, 16, 40, 128]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, n + 1, dtype, seed_cfg=147, q_scale=6.0, T_q=2)
    lay = B.EigenAttnLayer(B_, H, d, n + 1, dtype, U_k, U_v)
    lay.append_kv(k[:, :n], v[:, :n])
    ref = OraclePair(B_, H, d, U_k, U_v, dtype)
    ref.append_kv(to_np(k[:, :n]), to_np(v[:, :n]))
    expect = ref.decode_dense(to_np(q[:, :1]))
    tol = dict(fp32_rel=2e-4) if dtype == FP32 else {}
    for rows, min_copy, ctas in ((0, -1, 0), (16, 1 << 20, 3), (32, 1 << 20, 148), (128, 1 << 20, 7), (64, 0, 37), (16, 6000, 1)):
        lay.set_option(B.EA_OPT_DECODE_TILE_ROWS, rows)
        lay.set_option(B.EA_OPT_DECODE_MIN_COPY_BYTES, min_copy)
        lay.set_option(B.EA_OPT_DECODE_CTAS, ctas)
        assert_close(lay.decode(q[:, :1]), expect, dtype, f"tile_rows={rows} min_copy={min_copy} ctas={ctas}", **tol)
    o = lay.decode_step(q[:, 1:], k[:, n:], v[:, n:])               # the fused step over multi-tile slots
    ref.append_kv(to_np(k[:, n:]), to_np(v[:, n:]))
    assert_close(o, ref.decode_dense(to_np(q[:, 1:])), dtype, "decode_step", **tol)
    lay.poll_status()


@pytest.mark.parametrize("impl", [2, 3, 1])
def test_prefill_with_peaked_attention(B, impl):
    """Queries scaled by 3: the weights of a prompt row sit on a few keys, so an error in a few rows (a stale tile, a
    ragged tail, the diagonal mask) is not averaged away.  (Not more: the kernels keep Q' in bf16, and its rounding
    grows with the scores, about |s| * 2^-9 per score.)  All three prefill kernels, two chunks."""
    from helpers import OraclePair
    B_, H, d, T = 2, 4, 128, 700
    rk, rv = [80, 48, 128, 64], [64, 112, 16, 80]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, T, BF16, seed_cfg=143, T_q=T, q_scale=3.0)
    ref = OraclePair(B_, H, d, U_k, U_v, BF16)
    expect = ref.prefill_dense(to_np(q), to_np(k), to_np(v))
    lay = B.EigenAttnLayer(B_, H, d, T, BF16, U_k, U_v, max_prefill_tokens=T)
    lay.set_option(B.EA_OPT_PREFILL_IMPL, impl)
    a = lay.prefill(q[:, :300], k[:, :300], v[:, :300])
    c = lay.prefill(q[:, 300:], k[:, 300:], v[:, 300:])
    lay.poll_status()
    assert_close(torch.cat([a, c], dim=1), expect, BF16, f"peaked prefill impl {impl}")


@pytest.mark.parametrize("H,d,rk,rv,cuts", [
    (3, 128, [80, 48, 128], [80, 112, 8], [0, 128]),             # exactly one tile
    (2, 128, [80, 64], [64, 96], [0, 333, 1000]),                # ragged tiles, second chunk starts mid-cache
    (5, 64, [24, 64, 40, 8, 56], [56, 8, 64, 32, 16], [0, 700]), # one atom per row, more (head, tensor) pairs than a CTA keeps
])
def test_streaming_projection_equals_per_tile_projection(B, H, d, rk, rv, cuts):
    """Prefill's projections run either as a persistent kernel (token tiles by TMA, basis resident) or with
    one CTA per tile: the same products in the same order, so the cache rows and the outputs are bit-identical.
    Inputs are slices of a wider tensor (token stride larger than H * d_head) and of a longer one."""
    B_, T = 3, cuts[-1]
    U_k, U_v, q, k, v = make_case(B_, H, d, rk, rv, T + 5, BF16, seed_cfg=103, T_q=T + 5)
    wide = lambda x: torch.cat([x, torch.zeros_like(x)], dim=2)[:, :T, :H]      # views with padded strides
    q, k, v = wide(q), wide(k), wide(v)
    got = {}
    for mode in (0, 1, 2, 7):                        # 2 and 7 CTAs: every CTA walks through several bases
        lay = B.EigenAttnLayer(B_, H, d, T, BF16, U_k, U_v, max_prefill_tokens=T)
        lay.set_option(B.EA_OPT_PREFILL_PROJECT, mode)
        outs = [lay.prefill(q[:, a:b_], k[:, a:b_], v[:, a:b_]) for a, b_ in zip(cuts[:-1], cuts[1:])]
        lay.poll_status()
        got[mode] = (torch.cat(outs, dim=1), [lay.cache_rows(h, w).clone() for h in range(H) for w in "kv"])
    for mode in (0, 2, 7):
        assert torch.equal(got[mode][0], got[1][0])
        for a, b_ in zip(got[mode][1], got[1][1]):
            assert torch.equal(a, b_)
    ref = oracle_layer(B_, H, d, U_k, U_v)
    expect = ref.prefill_dense(to_np(q), to_np(k), to_np(v))
    assert_close(got[0][0], expect, BF16, "prefill with streamed projections")
