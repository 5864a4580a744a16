"""GPU parity: every stage of the CUDA path, called through the C ABI, against the CPU oracle on
the same seeded inputs.  Sizes span several 256-row tiles, ragged tails and thread-block clusters."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2503_07518_b200 import workloads as wl  # noqa: E402


@pytest.fixture(scope="module")
def H():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from oracle import tb_oracle
    tb_oracle.build()
    from paper_2503_07518_b200 import build
    build.build()
    import gpu_harness
    return gpu_harness


def tb():
    from paper_2503_07518_b200 import binding
    return binding


def full_pipeline_check(H, case, p, step=0, dense_too=False):
    """select (vs oracle, with the near-tie rule) then attention from the stored lists (vs oracle on
    the GPU's own list, and end to end when the sets agree).  Written over the case's lists and
    attention units, so it serves every selection scope."""
    w = case.w
    q, qi = H.queries(w, step)
    qi = qi[:, :, :case.Hl * case.gl]                     # one list per layer: a single importance query
    base_lists = None
    if p.radius > 0:
        # The GPU's own pre-expansion selection: the same launch with radius 0 (selection is bit-reproducible).
        # It is held to the oracle's with the near-tie rule; the expanded list must then be EXACTLY the
        # oracle's neighbour rule applied to it.  Taken first, so the lists left in the context are the expanded ones.
        assert p.step % p.interval == 0
        p0 = tb().select_params(p.budget, p.sinks, p.recent, 0, p.nmode, p.interval, p.step, p.reduce, p.score_scale)
        base_lists = H.gpu_select(case, qi, p0)
    lists = H.gpu_select(case, qi, p)
    assert case.ctx.get_status() == 0
    swaps = 0
    for l in range(w.n_layers):
        for b in range(w.batch):
            for h in range(case.Hl):
                what = "layer %d seq %d list %d" % (l, b, h)
                base, full, s = case.oracle_select(l, b, h, qi[l, b], p)
                if p.radius == 0:
                    swaps += H.check_selection(lists[l][b][h], full, s, what)
                else:
                    swaps += H.check_selection(base_lists[l][b][h], base, s, what)
                    lo, hi = H.orc.candidate_range(case.cur[b], p.sinks, p.recent)
                    want = H.orc.neighbors(base_lists[l][b][h], p.radius, p.nmode, lo, hi)
                    assert np.array_equal(lists[l][b][h], want), "%s: expanded list is not the neighbour rule of the GPU's selection" % what
    out, lse = H.gpu_attention(case, q, p)
    assert case.ctx.get_status() == 0
    worst = 0.0
    for l in range(w.n_layers):
        for b in range(w.batch):
            for h in range(case.Ha):
                ref, ref_lse = case.oracle_attention(l, b, h, q[l, b], lists[l][b][h * case.Hl // case.Ha], p)
                got = out[l, b, h * case.ga:(h + 1) * case.ga]
                worst = max(worst, np.abs(got - ref).max())
                assert np.allclose(lse[l, b, h * case.ga:(h + 1) * case.ga], ref_lse, atol=2e-3 if w.dtype == wl.BF16 else 1e-5, rtol=1e-5)
    assert worst <= H.ATTN_TOL[w.dtype], worst
    if dense_too:
        pd = tb().select_params(-1)
        outd, _ = H.gpu_attention(case, q, pd)
        for l in range(w.n_layers):
            for b in range(w.batch):
                for h in range(case.Ha):
                    ref, _ = case.oracle_attention(l, b, h, q[l, b], None, p, dense=True)
                    assert np.abs(outd[l, b, h * case.ga:(h + 1) * case.ga] - ref).max() <= H.ATTN_TOL[w.dtype]
    return swaps, worst


def test_cfg1_fp32_full_size(H):
    # configs[0]: single layer, 8 = 8 heads, fp32, 4096 tokens, budget 256 + 4 sinks + 64 recent
    w = wl.workload(1)
    case = H.Case(w)
    p = tb().select_params(w.budget, w.sinks, w.recent)
    swaps, worst = full_pipeline_check(H, case, p, dense_too=True)
    assert swaps == 0


def test_bf16_gqa_ragged_batch(H):
    # Llama-shaped heads (32 query / 8 KV), two layers, ragged lengths that end mid-tile
    w = wl.workload(2, n_layers=2, batch=3, lengths=[5000, 3333, 257], budget=300, sinks=3, recent=17, outlier_channels=4)
    case = H.Case(w)
    p = tb().select_params(w.budget, w.sinks, w.recent)
    full_pipeline_check(H, case, p, dense_too=True)


def test_cluster_path_long_sequence(H):
    # one sequence, two KV heads: the selection is spread over a thread-block cluster of 8
    w = wl.workload(4, n_layers=1, n_q_heads=8, n_kv_heads=2, lengths=[20011], budget=777, sinks=16, recent=256, planted=0)
    case = H.Case(w)
    p = tb().select_params(w.budget, w.sinks, w.recent)
    full_pipeline_check(H, case, p)


def test_attention_merge_shapes_with_eight_heads_per_group(H):
    # Groups of eight query heads fill every lane of the accumulator layout (groups of four leave half of it as
    # padding).  Three launch shapes of the bf16 attention kernel: a cluster of 16 blocks whose warps hold two
    # tiles (taken as one 32-token tile) or one; a cluster of a few blocks with three tiles per warp; and one
    # block per problem, which writes its result without the cluster exchange.
    for lengths, budget, sinks, recent in (([40000], 3000, 5, 130), ([9000], 1100, 0, 40), ([2500, 2400, 2300, 2200], 300, 2, 9)):
        w = wl.workload(2, n_layers=1, batch=len(lengths), n_q_heads=16, n_kv_heads=2, lengths=lengths, budget=budget,
                        sinks=sinks, recent=recent)
        full_pipeline_check(H, H.Case(w), tb().select_params(w.budget, w.sinks, w.recent), dense_too=len(lengths) == 1 and lengths[0] < 10000)


def _random_shapes(n, seed):
    # seeded draws over group size, KV heads, batch, lengths (a few long ones), budget, sinks, window, neighbour rule:
    # between them they reach every launch shape of the selection and attention kernels
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        g, hkv = int(rng.choice([1, 2, 4, 8])), int(rng.choice([1, 2, 4]))
        batch = int(rng.choice([1, 1, 1, 2, 3, 5, 24]))
        top = 140000 if batch == 1 and i % 4 == 0 else 30000 if batch == 1 else 6000 if batch < 24 else 2500
        lengths = [int(rng.integers(40, top)) for _ in range(batch)]
        budget = int(rng.integers(8, max(9, min(3500, max(lengths)))))
        cases.append((g, hkv, lengths, budget, int(rng.choice([0, 0, 1, 4, 16])), int(rng.choice([0, 0, 7, 64, 300])),
                      int(rng.choice([0, 0, 0, 1, 2])), int(rng.choice([0, 1]))))
    return cases


@pytest.mark.parametrize("shape", _random_shapes(32, 20250307),
                         ids=lambda c: "g%d_kv%d_b%d_L%d_B%d_s%d_w%d_r%d%s" % (c[0], c[1], len(c[2]), max(c[2]), c[3], c[4], c[5], c[6], "dc"[c[7]]))
def test_random_shapes(H, shape):
    g, hkv, lengths, budget, sinks, recent, radius, nmode = shape
    w = wl.workload(2, n_layers=1, batch=len(lengths), n_q_heads=g * hkv, n_kv_heads=hkv, lengths=lengths, budget=budget,
                    sinks=sinks, recent=recent, radius=radius, nmode=nmode)
    full_pipeline_check(H, H.Case(w), tb().select_params(w.budget, w.sinks, w.recent, radius, nmode))


def test_imp_dim_16_and_fp32_gqa(H):
    w = wl.workload(1, n_q_heads=4, n_kv_heads=2, imp_dim=16, lengths=[1500], budget=100, sinks=2, recent=5)
    full_pipeline_check(H, H.Case(w), tb().select_params(w.budget, w.sinks, w.recent))
    w = wl.workload(2, n_layers=1, n_q_heads=16, n_kv_heads=2, imp_dim=16, lengths=[3000], budget=64)
    full_pipeline_check(H, H.Case(w), tb().select_params(w.budget, 0, 0))


def test_scores_match_oracle_and_selection_is_exact_topk_of_them(H):
    w = wl.workload(2, n_layers=1, batch=2, lengths=[4100, 900], budget=200, sinks=1, recent=9)
    case = H.Case(w)
    q, qi = H.queries(w)
    scores = torch.full((w.batch, w.n_kv_heads, case.cap), float("nan"), device="cuda")
    case.ctx.score_tokens(0, None, w.batch, torch.from_numpy(qi[0]).cuda(), scores, scale=0.5)
    p = tb().select_params(w.budget, w.sinks, w.recent)
    lists = H.gpu_select(case, qi, p)
    sc = scores.cpu().numpy()
    for b in range(w.batch):
        L = case.cur[b]
        for h in range(w.n_kv_heads):
            _, _, s = case.oracle_select(0, b, h, qi[0, b], p)
            assert np.allclose(sc[b, h, :L], 0.5 * s, rtol=1e-5, atol=1e-5)
            assert np.all(np.isnan(sc[b, h, L:]))                       # tail untouched
            # the fused kernel ranks by these very fp32 values: exact top-k, ties to the lower index
            lo, hi = H.orc.candidate_range(L, p.sinks, p.recent)
            cand = np.arange(lo, hi)
            order = np.lexsort((cand, -sc[b, h, lo:hi].astype(np.float64)))
            assert np.array_equal(lists[0][b][h], np.sort(cand[order[:w.budget]]))


def test_exact_ties_keep_lower_positions(H):
    w = wl.workload(2, n_layers=1, n_q_heads=4, n_kv_heads=1, lengths=[3000], budget=50)
    case = H.Case(w)
    q, qi = H.queries(w)
    p = tb().select_params(w.budget, 0, 0)
    _, _, s = case.oracle_select(0, 0, 0, qi[0, 0], p)
    order = np.argsort(-s)
    # duplicate the projected key of the token ranked 49th (boundary) at five later and earlier positions
    src = order[48]
    dup = [int(x) for x in order[200:205]]
    for t in dup:
        case.Kimp[0][0][0, t] = case.Kimp[0][0][0, src]
    case.ctx.kimp[0, 0, 0, :3000] = H.to_dev(case.Kimp[0][0][0, :3000], w.dtype)
    lists = H.gpu_select(case, qi, p)
    _, full, s2 = case.oracle_select(0, 0, 0, qi[0, 0], p)
    assert np.array_equal(lists[0][0][0], full)                            # bit-equal scores: no tolerance
    tied = sorted(dup + [int(src)])
    assert set(tied[:2]) <= set(full.tolist()) and not (set(tied[2:]) & set(full.tolist()))
    # all scores equal (zero query): the first `budget` candidates win; -0.0 and +0.0 tie
    zero = np.zeros_like(qi)
    zero[0, 0, 0, 0] = -0.0
    lists = H.gpu_select(case, zero, tb().select_params(50, 7, 3))
    assert np.array_equal(lists[0][0][0], np.arange(7, 57))


def test_edge_cases(H):
    w = wl.workload(2, n_layers=1, batch=4, n_q_heads=8, n_kv_heads=2, lengths=[1, 40, 300, 513], budget=64)
    case = H.Case(w, max_budget=1024)
    q, qi = H.queries(w)
    # L <= S + W for the two short sequences (no candidates -> dense); budget > candidates for the others
    p = tb().select_params(1000, 8, 32)
    lists = H.gpu_select(case, qi, p)
    for h in range(2):
        assert len(lists[0][0][h]) == 0 and len(lists[0][1][h]) == 0
        assert np.array_equal(lists[0][2][h], np.arange(8, 300 - 32))
        assert np.array_equal(lists[0][3][h], np.arange(8, 513 - 32))
    out, _ = H.gpu_attention(case, q, p)
    for b in range(4):
        for h in range(2):
            ref, _ = case.oracle_attention(0, b, h, q[0, b], None, p, dense=True)   # everything attended
            assert np.abs(out[0, b, h * 4:(h + 1) * 4] - ref).max() <= 2e-3
    # budget 0: sinks + window only
    p0 = tb().select_params(0, 8, 32)
    full_pipeline_check(H, case, p0)
    # budget 1
    full_pipeline_check(H, case, tb().select_params(1, 0, 0))


@pytest.mark.parametrize("nmode", [0, 1])
@pytest.mark.parametrize("radius", [1, 2])
def test_neighbor_modes(H, nmode, radius):
    w = wl.workload(5, n_layers=1, batch=2, n_q_heads=8, n_kv_heads=2, lengths=[2500, 1800], budget=120, recent=16,
                    radius=radius, nmode=nmode, decode_steps=0)
    case = H.Case(w)
    q, qi = H.queries(w)
    p = tb().select_params(w.budget, 0, w.recent, radius, nmode)
    lists = H.gpu_select(case, qi, p)
    for b in range(2):
        for h in range(2):
            base, full, s = case.oracle_select(0, b, h, qi[0, b], p)
            assert np.array_equal(lists[0][b][h], full)
    full_pipeline_check(H, case, p)


def test_interval_trajectory_with_appends(H):
    # configs[4] in miniature: selection refreshed every P steps, +-1 neighbours, one token appended
    # per step, keys projected in deferred batches of W tokens
    P, Wn, steps = 4, 8, 10
    w = wl.workload(5, n_layers=2, batch=2, n_q_heads=8, n_kv_heads=2, lengths=[1200, 700], budget=90, recent=Wn,
                    radius=1, interval=P, decode_steps=steps)
    case = H.Case(w, extra_len=steps)
    stored = None
    for t in range(steps):
        if t > 0:
            case.append_step(t)
            if (case.cur[0] - case.proj[0]) >= Wn:                      # the window wrapped: project its tokens
                case.project_range(list(case.proj), [case.proj[b] + Wn for b in range(w.batch)])
        p = tb().select_params(w.budget, 0, Wn, 1, 0, P, t)
        q, qi = H.queries(w, t)
        lists = H.gpu_select(case, qi, p)
        if t % P == 0:
            for l in range(2):
                for b in range(2):
                    for h in range(2):
                        _, full, _ = case.oracle_select(l, b, h, qi[l, b], p)
                        assert np.array_equal(lists[l][b][h], full)
            stored = lists
        else:
            for l in range(2):
                for b in range(2):
                    for h in range(2):
                        assert np.array_equal(lists[l][b][h], stored[l][b][h])     # stale list reused
        out, _ = H.gpu_attention(case, q, p)
        for l in range(2):
            for b in range(2):
                for h in range(2):
                    ref, _ = case.oracle_attention(l, b, h, q[l, b], stored[l][b][h], p)
                    assert np.abs(out[l, b, h * 4:(h + 1) * 4] - ref).max() <= 2e-3


def test_full_budget_equals_dense(H):
    w = wl.workload(1, lengths=[1111], budget=2000, sinks=4, recent=64, n_q_heads=4, n_kv_heads=4)
    case = H.Case(w, max_budget=2000)
    q, qi = H.queries(w)
    p = tb().select_params(2000, 4, 64)
    H.gpu_select(case, qi, p)
    sparse, _ = H.gpu_attention(case, q, p)
    dense, _ = H.gpu_attention(case, q, tb().select_params(-1))
    assert np.abs(sparse - dense).max() <= 1e-6


def test_caller_lists_and_bad_index_status(H):
    w = wl.workload(2, n_layers=1, n_q_heads=8, n_kv_heads=2, lengths=[600], budget=32)
    case = H.Case(w)
    q, qi = H.queries(w)
    cap = case.ctx.index_capacity
    r = np.random.Generator(np.random.PCG64(5))
    idx = np.zeros((1, 1, 2, cap), np.int32)
    mine = [np.sort(r.choice(np.arange(5, 590), 20, replace=False)).astype(np.int32) for _ in range(2)]
    for h in range(2):
        idx[0, 0, h, :20] = mine[h]
    cnt = np.full((1, 1, 2), 20, np.int32)
    p = tb().select_params(32, 5, 10)
    out, _ = H.gpu_attention(case, q, p, idx=torch.from_numpy(idx).cuda(), cnt=torch.from_numpy(cnt).cuda())
    for h in range(2):
        ref, _ = case.oracle_attention(0, 0, h, q[0, 0], mine[h], p)
        assert np.abs(out[0, 0, h * 4:(h + 1) * 4] - ref).max() <= 2e-3
    assert case.ctx.get_status() == 0
    idx[0, 0, 1, 3] = 600                                                # one past the end: skipped and reported
    out2, _ = H.gpu_attention(case, q, p, idx=torch.from_numpy(idx).cuda(), cnt=torch.from_numpy(cnt).cuda())
    assert case.ctx.get_status() == tb().TB_ERR_BAD_INDEX
    assert case.ctx.get_status() == 0                                    # reading clears it
    ref, _ = case.oracle_attention(0, 0, 1, q[0, 0], np.delete(mine[1], 3), p)
    assert np.abs(out2[0, 0, 4:8] - ref).max() <= 2e-3


def test_error_codes_change_nothing(H):
    b = tb()
    w = wl.workload(2, n_layers=1, n_q_heads=8, n_kv_heads=2, lengths=[100], budget=16)
    case = H.Case(w, extra_len=4, project=None)
    q, qi = H.queries(w)
    qi_d = torch.from_numpy(qi).cuda()
    with pytest.raises(b.TBError) as e:
        case.ctx.select_topk(0, 1, None, 1, qi_d, b.select_params(16))
    assert e.value.status == b.TB_ERR_UNPROJECTED
    out = torch.zeros(1, 1, 8, 128, device="cuda")
    with pytest.raises(b.TBError) as e:
        case.ctx.sparse_decode_attention(0, 1, None, 1, H.to_dev(q, w.dtype), b.select_params(16), out)
    assert e.value.status == b.TB_ERR_STATE
    with pytest.raises(b.TBError) as e:
        case.ctx.select_topk(0, 1, None, 1, qi_d, b.select_params(17))
    assert e.value.status == b.TB_ERR_CAPACITY
    k = torch.zeros(5, 2, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(b.TBError) as e:
        case.ctx.append_kv(0, 1, None, [5], k, k)
    assert e.value.status == b.TB_ERR_CAPACITY
    assert case.ctx.get_length(0, 0) == (100, 0)
    with pytest.raises(b.TBError) as e:
        case.ctx.project_keys(0, 1, None, [10], [20])                    # would leave positions 0..9 unprojected
    assert e.value.status == b.TB_ERR_INVALID_ARG
    # the deferred-projection rule: only the candidates need projecting
    case.project_range([0], [60])
    case.ctx.select_topk(0, 1, None, 1, qi_d, b.select_params(16, 0, 40))
    with pytest.raises(b.TBError) as e:
        case.ctx.select_topk(0, 1, None, 1, qi_d, b.select_params(16, 0, 39))
    assert e.value.status == b.TB_ERR_UNPROJECTED


def test_bit_reproducible(H):
    w = wl.workload(2, n_layers=2, batch=2, lengths=[9000, 4000], budget=500)
    case = H.Case(w, project="oracle-only")
    q, qi = H.queries(w)
    p = tb().select_params(w.budget, 0, 0)
    a = H.gpu_select(case, qi, p)
    oa, la = H.gpu_attention(case, q, p)
    b = H.gpu_select(case, qi, p)
    ob, lb = H.gpu_attention(case, q, p)
    assert all(np.array_equal(x, y) for l in range(2) for s in range(2) for x, y in zip(a[l][s], b[l][s]))
    assert np.array_equal(oa, ob) and np.array_equal(la, lb)


def _crafted_scores_case(H, scores_per_head, budget, sinks=0, recent=0):
    """A cluster-sized problem (one sequence, L = len(scores)) whose importance scores are exactly the
    given values: K_imp rows are score * e_0 and the importance query is e_0."""
    L = scores_per_head.shape[1]
    n_heads = scores_per_head.shape[0]
    w = wl.workload(2, n_layers=1, n_q_heads=n_heads, n_kv_heads=n_heads, lengths=[L], budget=budget, sinks=sinks, recent=recent)
    case = H.Case(w, project="oracle-only")
    for h in range(n_heads):
        kimp = np.zeros((L, w.imp_dim), np.float32)
        kimp[:, 0] = scores_per_head[h]
        bits = wl.to_storage(kimp, w.dtype)
        assert np.array_equal(wl.storage_to_f32(bits, w.dtype)[:, 0], scores_per_head[h]), "scores must be bf16-exact"
        case.Kimp[0][0][h, :L] = bits
        case.ctx.kimp[0, 0, h, :L] = H.to_dev(bits, w.dtype)
    qi = np.zeros((1, 1, n_heads, w.imp_dim), np.float32)
    qi[..., 0] = 1.0
    p = tb().select_params(budget, sinks, recent)
    lists = H.gpu_select(case, qi, p)
    assert case.ctx.get_status() == 0
    for h in range(n_heads):
        _, full, _ = case.oracle_select(0, 0, h, qi[0, 0], p)
        assert np.array_equal(lists[0][0][h], full), "head %d" % h     # exact scores: no tolerance
    return lists


def test_cluster_selection_unusual_distributions(H):
    """Paths of the cluster radix select that ordinary data never takes (20011 tokens, 2 heads: a cluster of 8)."""
    r = np.random.Generator(np.random.PCG64(77))
    L = 20011
    # every score equal: the threshold bin holds everything, the lowest positions win
    _crafted_scores_case(H, np.zeros((2, L), np.float32), budget=777, sinks=5, recent=9)
    _crafted_scores_case(H, np.full((2, L), -3.5, np.float32), budget=1)
    # scores over ~400 binades and both signs: more non-empty first-digit bins than a block may publish
    expo = r.integers(-100, 101, size=(2, L))
    sign = r.choice([-1.0, 1.0], size=(2, L))
    _crafted_scores_case(H, (sign * np.exp2(expo)).astype(np.float32), budget=2500)
    # a few distinct values: thousands of exact ties at the threshold, spread over all blocks
    vals = r.integers(0, 12, size=(2, L)).astype(np.float32)
    _crafted_scores_case(H, vals, budget=3000)                          # ~1670 per value: the quota ends inside a class
    _crafted_scores_case(H, r.integers(0, 3, size=(2, L)).astype(np.float32), budget=9000)   # class of ~6670 keys
    # the budget ends exactly at a class boundary (whole threshold bin taken)
    v = np.zeros((2, L), np.float32)
    v[:, ::7] = 4.0
    _crafted_scores_case(H, v, budget=int((v[0] == 4.0).sum()))


def _crafted_batch_case(H, scores, budget, sinks=0, recent=0):
    """Many problems in one launch (scores[seq, head, position], equal lengths): K_imp rows are
    score * e_0 and the importance query is e_0, so the importance scores are exactly `scores`."""
    n_seq, n_heads, L = scores.shape
    w = wl.workload(2, n_layers=1, n_q_heads=n_heads, n_kv_heads=n_heads, batch=n_seq, lengths=[L] * n_seq, budget=budget,
                    sinks=sinks, recent=recent)
    case = H.Case(w, project="oracle-only")
    for b in range(n_seq):
        for h in range(n_heads):
            kimp = np.zeros((L, w.imp_dim), np.float32)
            kimp[:, 0] = scores[b, h]
            bits = wl.to_storage(kimp, w.dtype)
            assert np.array_equal(wl.storage_to_f32(bits, w.dtype)[:, 0], scores[b, h]), "scores must be bf16-exact"
            case.Kimp[0][b][h, :L] = bits
            case.ctx.kimp[0, b, h, :L] = H.to_dev(bits, w.dtype)
    qi = np.zeros((1, n_seq, n_heads, w.imp_dim), np.float32)
    qi[..., 0] = 1.0
    p = tb().select_params(budget, sinks, recent)
    lists = H.gpu_select(case, qi, p)
    assert case.ctx.get_status() == 0
    for b in range(n_seq):
        for h in range(n_heads):
            _, full, _ = case.oracle_select(0, b, h, qi[0, b], p)
            assert np.array_equal(lists[0][b][h], full), "seq %d head %d" % (b, h)   # exact scores: no tolerance
    return lists


def _bf16_exact(x):
    return wl.storage_to_f32(wl.to_storage(x.astype(np.float32), wl.BF16), wl.BF16)


def test_many_problem_selection_kernel(H):
    """Launches with hundreds of problems take the one-block-per-problem kernel (40 sequences x 8 heads
    here).  Its first digit is placed from a sample of each problem's scores; these cases put the
    threshold in every kind of bin that digit has, and on the general path behind it."""
    r = np.random.Generator(np.random.PCG64(78))
    n_seq, n_heads = 40, 8
    # ordinary data, long enough to be sampled, ending mid-tile; and too short to be sampled
    _crafted_batch_case(H, _bf16_exact(r.standard_normal((n_seq, n_heads, 5003))), budget=400, sinks=2, recent=31)
    _crafted_batch_case(H, _bf16_exact(r.standard_normal((n_seq, n_heads, 1501))), budget=100)
    # every score equal, and a few distinct values: the threshold bin is one crowded class of ties
    _crafted_batch_case(H, np.full((n_seq, n_heads, 3001), 1.5, np.float32), budget=200, sinks=1, recent=3)
    _crafted_batch_case(H, r.integers(0, 5, size=(n_seq, n_heads, 4099)).astype(np.float32), budget=1000)
    # a handful of huge scores at positions the sample does not see, budget below their number: the
    # threshold lies in the open-ended top bin
    L = 4096
    s = _bf16_exact(r.standard_normal((n_seq, n_heads, L)))
    s[:, :, 7::509] = _bf16_exact(1000.0 + 8.0 * r.integers(0, 64, size=s[:, :, 7::509].shape))
    _crafted_batch_case(H, s, budget=5)
    # the sampled positions (every 64th of the candidates) hold large scores, everything else small
    # ones, and the budget reaches deep into the small ones: the threshold lies below the sampled range
    s = _bf16_exact(0.01 * r.standard_normal((n_seq, n_heads, L)))
    s[:, :, ::64] = _bf16_exact(50.0 + r.standard_normal((n_seq, n_heads, L // 64)))
    _crafted_batch_case(H, s, budget=2000)
    # scores over ~400 binades and both signs
    expo = r.integers(-100, 101, size=(n_seq, n_heads, 3000))
    sign = r.choice([-1.0, 1.0], size=expo.shape)
    _crafted_batch_case(H, (sign * np.exp2(expo)).astype(np.float32), budget=700)
    # budget covers every candidate; no candidates at all
    _crafted_batch_case(H, _bf16_exact(r.standard_normal((n_seq, n_heads, 600))), budget=600)
    _crafted_batch_case(H, _bf16_exact(r.standard_normal((n_seq, n_heads, 300))), budget=10, sinks=100, recent=200)


def test_selection_of_very_long_problems(H):
    """A single problem of 270K candidates: the parked-key cluster kernel with its rows' first digits on
    chip.  One of 700K: more rows per block than shared memory holds digits for, so they live in the
    workspace; ordinary scores, and a few distinct values (crowded threshold bins: the bin is cut again from
    the parked keys, then the general path)."""
    r = np.random.Generator(np.random.PCG64(79))
    _crafted_scores_case(H, _bf16_exact(r.standard_normal((1, 270001))), budget=5000, sinks=4, recent=64)
    _crafted_scores_case(H, _bf16_exact(r.standard_normal((1, 700001))), budget=9000, sinks=4, recent=64)
    _crafted_scores_case(H, r.integers(0, 40, size=(1, 700001)).astype(np.float32), budget=30000)


@pytest.mark.parametrize("act", [0, 1, 2])
def test_predictor_forward_matches_oracle(H, act):
    """q = W2 act(W1 LN(h)) against the fp64 oracle on the same stored bytes: fp32 accumulation over
    4096 and 512 terms of O(1) values, so 2e-4 absolute on outputs of magnitude ~2 is ample."""
    import torch
    # bf16 8B shapes at 1 token (matrix-vector kernels), 5 and 20 tokens (tensor-core tiles, one and two of them);
    # bf16 with sizes the tiles do not divide; fp32, odd sizes
    for cfg, over, E, hid in ((2, dict(batch=1), 4096, 512), (2, dict(batch=5), 4096, 512), (2, dict(batch=20), 4096, 512),
                              (2, dict(batch=7), 1000, 72), (1, dict(batch=3), 1000, 72)):
        w = wl.workload(cfg, **over)
        Hs, ln_w, ln_b, W1, W2 = wl.gen_predictor(w, 1, model_dim=E, hidden_dim=hid, slots=4)
        ref = H.orc.predict_queries(Hs, ln_w, ln_b, W1, W2, w.dtype, eps=1e-5, act=act)       # [tokens, slots * heads * d']
        dev = [H.to_dev(a, w.dtype) for a in (Hs, ln_w, ln_b, W1, W2)]
        scratch = torch.empty(w.batch * hid, dtype=torch.float32, device="cuda")
        q = torch.full((4, w.batch, w.n_q_heads, w.imp_dim), float("nan"), dtype=torch.float32, device="cuda")
        st = tb().predict_importance_queries(*dev, w.dtype, w.n_q_heads, 4, w.imp_dim, scratch, q, ln_eps=1e-5, activation=act)
        assert st == tb().TB_OK
        torch.cuda.synchronize()
        got = q.cpu().numpy()                                                                  # [slot, token, head, d']
        want = ref.reshape(w.batch, 4, w.n_q_heads, w.imp_dim).transpose(1, 0, 2, 3)
        assert np.isfinite(got).all()
        assert np.abs(got - want).max() <= 2e-4, np.abs(got - want).max()


def test_predictor_output_feeds_selection(H):
    """The predictor's output block is the q_imp argument of tb_select_topk for its consumer layers:
    selecting with it on the GPU equals selecting with the oracle's queries in the oracle."""
    import torch
    w = wl.workload(2, n_layers=4, batch=2, lengths=[3000, 1800], budget=200)
    case = H.Case(w)
    Hs, ln_w, ln_b, W1, W2 = wl.gen_predictor(w, 0, model_dim=1024, hidden_dim=512, slots=4)
    dev = [H.to_dev(a, w.dtype) for a in (Hs, ln_w, ln_b, W1, W2)]
    scratch = torch.empty(w.batch * 512, dtype=torch.float32, device="cuda")
    q = torch.empty((4, w.batch, w.n_q_heads, w.imp_dim), dtype=torch.float32, device="cuda")
    assert tb().predict_importance_queries(*dev, w.dtype, w.n_q_heads, 4, w.imp_dim, scratch, q) == tb().TB_OK
    p = tb().select_params(w.budget)
    lists = H.gpu_select(case, q.cpu().numpy(), p)
    assert case.ctx.get_status() == 0
    ref = H.orc.predict_queries(Hs, ln_w, ln_b, W1, W2, w.dtype).reshape(w.batch, 4, w.n_q_heads, w.imp_dim).transpose(1, 0, 2, 3)
    for l in range(4):
        for b in range(w.batch):
            for h in range(w.n_kv_heads):
                _, full, s = case.oracle_select(l, b, h, np.ascontiguousarray(ref[l, b], dtype=np.float32), p)
                H.check_selection(lists[l][b][h], full, s, "layer %d seq %d head %d" % (l, b, h))


def test_kv_cache_in_pinned_host_memory(H):
    """Offloaded KV: with the K|V cache in page-locked host memory every call works unchanged and gives
    the same bits as with the cache on the device (same kernels, same order of operations); a pointer
    the device cannot address is refused at tb_create."""
    import ctypes
    import torch
    w = wl.workload(2, n_layers=2, batch=2, lengths=[2500, 1111], budget=150, sinks=2, recent=9)
    p = tb().select_params(w.budget, w.sinks, w.recent)
    q, qi = H.queries(w, 0)
    res = []
    for on_host in (False, True):
        case = H.Case(w, extra_len=4, kv_on_host=on_host)
        assert case.ctx.kv.is_cuda != on_host
        lists = H.gpu_select(case, qi, p)
        out, lse = H.gpu_attention(case, q, p)
        case.append_step(0)                                   # one decode step: append (over the link), project, attend
        out2, lse2 = H.gpu_attention(case, q, p)
        assert case.ctx.get_status() == 0
        res.append((lists, out, lse, out2, lse2))
        if on_host:
            case.project_all()                                # the new token's projected key (reads K over the link)
            full_pipeline_check(H, case, p, step=1)           # and it matches the oracle
    (la, oa, sa, oa2, sa2), (lb, ob, sb, ob2, sb2) = res
    assert all(np.array_equal(x, y) for l in range(2) for s in range(2) for x, y in zip(la[l][s], lb[l][s]))
    assert np.array_equal(oa, ob) and np.array_equal(sa, sb) and np.array_equal(oa2, ob2) and np.array_equal(sa2, sb2)
    # pageable host memory is not addressable by the device: refused, nothing launched
    b = tb()
    cfg = b.tb_config(1, 8, 8, 128, 32, b.TB_BF16, 1, 256, 16, 0, 0, 0)
    sizes = [ctypes.c_size_t() for _ in range(4)]
    assert b.lib().tb_query_sizes(ctypes.byref(cfg), *[ctypes.byref(s) for s in sizes]) == b.TB_OK
    dev = [torch.empty(s.value + 256, dtype=torch.uint8, device="cuda") for s in sizes]
    pageable = torch.empty(sizes[0].value + 256, dtype=torch.uint8)
    al = lambda t: ctypes.c_void_p((t.data_ptr() + 255) & ~255)
    h = ctypes.c_void_p()
    assert b.lib().tb_create(ctypes.byref(cfg), al(pageable), al(dev[1]), al(dev[2]), al(dev[3]), ctypes.byref(h)) == b.TB_ERR_INVALID_ARG
    assert b.lib().tb_create(ctypes.byref(cfg), al(dev[0]), al(pageable), al(dev[2]), al(dev[3]), ctypes.byref(h)) == b.TB_ERR_INVALID_ARG


def test_group_max_reduction(H):
    """TB_GROUP_MAX (a token's score is the largest of its group's g head scores): materialised scores
    against the oracle, the fused selection = exact top-k of those very fp32 values, on the cluster
    kernel (one long sequence), on the many-problem kernel (40 sequences) and through the whole pipeline."""
    b_ = tb()
    # cluster kernel + score kernel, g = 4
    w = wl.workload(2, n_layers=1, batch=2, lengths=[9000, 700], budget=300, sinks=2, recent=5)
    case = H.Case(w)
    q, qi = H.queries(w)
    p = b_.select_params(w.budget, w.sinks, w.recent, reduce=b_.TB_GROUP_MAX)
    scores = torch.full((w.batch, w.n_kv_heads, case.cap), float("nan"), device="cuda")
    case.ctx.score_tokens(0, None, w.batch, torch.from_numpy(qi[0]).cuda(), scores, reduce=b_.TB_GROUP_MAX)
    lists = H.gpu_select(case, qi, p)
    sc = scores.cpu().numpy()
    for b in range(w.batch):
        L = case.cur[b]
        for h in range(w.n_kv_heads):
            _, _, s = case.oracle_select(0, b, h, qi[0, b], p)
            assert np.allclose(sc[b, h, :L], s, rtol=1e-5, atol=1e-5)
            ssum = H.orc.score(qi[0, b][h * w.group:(h + 1) * w.group], np.ascontiguousarray(case.Kimp[0][b][h, :L]), w.dtype)
            assert not np.allclose(s, ssum)                                # and it is not the sum reduction
            lo, hi = H.orc.candidate_range(L, p.sinks, p.recent)
            cand = np.arange(lo, hi)
            order = np.lexsort((cand, -sc[b, h, lo:hi].astype(np.float64)))
            assert np.array_equal(lists[0][b][h], np.sort(cand[order[:w.budget]]))
    full_pipeline_check(H, case, p)
    # many-problem kernel: 40 sequences x 8 KV heads in one launch, fp32 storage and d' = 16 as well
    for cfg, over in ((2, dict(n_layers=1, batch=40, lengths=[2300 + 37 * i for i in range(40)], budget=128)),
                      (1, dict(n_layers=1, n_q_heads=16, n_kv_heads=8, imp_dim=16, batch=40, lengths=[2100 + 11 * i for i in range(40)],
                               budget=64, sinks=1, recent=3))):
        w = wl.workload(cfg, **over)
        case = H.Case(w)
        q, qi = H.queries(w)
        p = b_.select_params(w.budget, w.sinks, w.recent, reduce=b_.TB_GROUP_MAX)
        lists = H.gpu_select(case, qi, p)
        assert case.ctx.get_status() == 0
        for b in range(w.batch):
            for h in range(w.n_kv_heads):
                _, full, s = case.oracle_select(0, b, h, qi[0, b], p)
                H.check_selection(lists[0][b][h], full, s, "seq %d head %d" % (b, h))


@pytest.mark.parametrize("nmode", [0, 1])
def test_many_problem_selection_with_neighbours_and_attention(H, nmode):
    """The one-block-per-problem selection kernel in the full pipeline: 32 sequences x 8 KV heads per
    launch, neighbour expansion from its pre-expansion lists, attention from the stored lists."""
    w = wl.workload(5, n_layers=1, batch=32, lengths=[2100 + 29 * i for i in range(32)], budget=120, sinks=2, recent=16, radius=1)
    case = H.Case(w)
    p = tb().select_params(w.budget, w.sinks, w.recent, radius=1, nmode=nmode)
    full_pipeline_check(H, case, p)


def test_long_problem_cluster_kernel_unusual_distributions(H):
    """Problems beyond 48K candidates take the cluster kernel that parks its keys (70001 tokens, 2 heads
    here).  Cases for each way its threshold search can go: a bin cut again, the open bin above the
    sampled bracket, the open bin below it and massive ties (general path on the parked keys)."""
    r = np.random.Generator(np.random.PCG64(80))
    L = 70001
    _crafted_scores_case(H, _bf16_exact(r.standard_normal((2, L))), budget=3000, sinks=3, recent=40)
    # every score equal; a few distinct values (tens of thousands of ties at the threshold)
    _crafted_scores_case(H, np.full((2, L), 2.25, np.float32), budget=500, sinks=5, recent=9)
    _crafted_scores_case(H, r.integers(0, 4, size=(2, L)).astype(np.float32), budget=20000)
    # a hundred huge scores where the sample does not look, budget below their number: the threshold is far
    # above the bracket
    s = _bf16_exact(r.standard_normal((2, L)))
    s[:, 11::701] = _bf16_exact(1000.0 + 8.0 * r.integers(0, 64, size=s[:, 11::701].shape))
    _crafted_scores_case(H, s, budget=37)
    # 3000 scores just above everything else, spread so thinly that the bracket's top slice holds them all
    s = _bf16_exact(r.standard_normal((2, L)))
    s[:, 5::23] = _bf16_exact(6.0 + 0.5 * r.random(s[:, 5::23].shape))
    _crafted_scores_case(H, s, budget=1500)
    # the sampled positions hold large scores, the rest small ones, and the budget reaches deep into the
    # small ones: the threshold lies below the bracket
    s = _bf16_exact(0.01 * r.standard_normal((2, L)))
    for i in range(64):
        s[:, (i * L) // 64] = 50.0 + i
    _crafted_scores_case(H, s, budget=30000)
    # ~400 binades, both signs
    expo = r.integers(-100, 101, size=(2, L))
    sign = r.choice([-1.0, 1.0], size=(2, L))
    _crafted_scores_case(H, (sign * np.exp2(expo)).astype(np.float32), budget=9000)
