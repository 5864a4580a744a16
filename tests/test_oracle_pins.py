"""Pins for the CPU oracle: each test checks it against something other than itself -- a numpy
float64 library routine, brute force on tiny inputs, a closed form, an invariant the paper fixes,
or a value the paper prints (tests/golden/)."""
import itertools
import os

import numpy as np
import pytest

from paper_2503_07518_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
F32, BF16 = 0, 1


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def rand_storage(r, shape, dtype, scale=1.0):
    return wl.to_storage((r.standard_normal(shape) * scale).astype(np.float32), dtype)


def f64(x, dtype):
    return wl.storage_to_f32(x, dtype).astype(np.float64)


# ------------------------------------------------------------------ storage rounding

def test_bf16_rounding_special_cases(orc):
    # ties go to the even mantissa; one rounding step only (a detour through fp32 would turn
    # 1 + 2^-8 + 2^-30 into the tie 1 + 2^-8 and then round it DOWN)
    x = np.array([1.0, 1 + 2.0**-8, 1 + 3 * 2.0**-8, 1 + 2.0**-8 + 2.0**-30, -(1 + 2.0**-8 + 2.0**-30),
                  0.0, -0.0, 2.0**-133, 2.0**-134, 1.5 * 2.0**-133, 3.3895313892515355e38, 1e39, np.inf])
    want = np.array([1.0, 1.0, 1 + 2.0**-6, 1 + 2.0**-7, -(1 + 2.0**-7), 0.0, -0.0, 2.0**-133, 0.0,
                     2.0**-132, 3.3895313892515355e38, np.inf, np.inf])
    got = f64(orc.round_to_storage(x, BF16), BF16)
    assert np.array_equal(got, want)
    assert np.signbit(got[6]) and not np.signbit(got[5])


def test_bf16_rounding_matches_bit_trick_on_fp32_inputs(orc):
    x = (rng(1).standard_normal(20000) * np.exp(rng(2).uniform(-20, 20, 20000))).astype(np.float32)
    assert np.array_equal(orc.round_to_storage(x.astype(np.float64), BF16), wl.f32_to_bf16_bits(x))
    assert np.array_equal(orc.widen(wl.f32_to_bf16_bits(x), BF16), wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(x)).astype(np.float64))


# ------------------------------------------------------------------ P3: projection = K @ W

@pytest.mark.parametrize("dtype", [F32, BF16])
def test_project_keys_is_float64_matmul(orc, dtype):
    r = rng(3)
    T, D, dp = 37, 128, 32
    K = rand_storage(r, (T, D), dtype)
    W = rand_storage(r, (D, dp), dtype, 1 / np.sqrt(D))
    out, exact = orc.project_keys(K, W, dtype, want_f64=True)
    ref = f64(K, dtype) @ f64(W, dtype)                      # numpy float64 GEMM
    assert np.allclose(exact, ref, rtol=1e-13, atol=1e-13)
    # K @ W^T (transposed operand) or a dropped channel would be far outside this
    assert exact.shape == (T, dp)
    ulp = 2.0 ** (np.floor(np.log2(np.abs(ref))) - (7 if dtype == BF16 else 23))   # spacing at |ref|
    assert np.all(np.abs(f64(out, dtype) - ref) <= 0.5 * ulp)                      # correctly rounded
    # non-square W catches an index swap: W[c, j] vs W[j, c]
    W2 = W.copy()
    W2[0, 1], W2[1, 0] = W[1, 0], W[0, 1]
    if not np.array_equal(W2, W):
        out2 = orc.project_keys(K, W2, dtype)
        assert not np.array_equal(out2, out)


# ------------------------------------------------------------------ scores = q . K_imp

@pytest.mark.parametrize("dtype", [F32, BF16])
@pytest.mark.parametrize("g", [1, 4])
def test_scores_are_float64_dot_products(orc, dtype, g):
    r = rng(4 + g)
    L, dp = 300, 32
    kimp = rand_storage(r, (L, dp), dtype, 3.0)
    qi = r.standard_normal((g, dp)).astype(np.float32)
    s = orc.score(qi, kimp, dtype, orc.GROUP_SUM, 0.5)
    ref = 0.5 * (f64(kimp, dtype) @ qi.astype(np.float64).sum(0))
    assert np.allclose(s, ref, rtol=1e-12, atol=1e-12)
    smax = orc.score(qi, kimp, dtype, orc.GROUP_MAX, 1.0)
    refmax = (f64(kimp, dtype) @ qi.astype(np.float64).T).max(1)
    assert np.allclose(smax, refmax, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ P4/P5: selection

def lexsort_select(s, S, W, k):
    L = len(s)
    lo, hi = min(S, L), max(min(S, L), L - W)
    cand = np.arange(lo, hi)
    order = np.lexsort((cand, -s[cand]))                      # score descending, then index ascending
    return np.sort(cand[order[:min(k, len(cand))]])


@pytest.mark.parametrize("seed", range(6))
def test_select_equals_stable_argsort(orc, seed):
    r = rng(100 + seed)
    L = int(r.integers(1, 3000))
    S, W = int(r.integers(0, 40)), int(r.integers(0, 200))
    k = int(r.integers(0, L + 5))
    s = r.standard_normal(L)
    if seed % 2:                                              # many exact ties
        s = np.round(s * 4) / 4
    got = orc.select(s, S, W, k)
    assert np.array_equal(got, lexsort_select(s, S, W, k))
    assert np.all(np.diff(got) > 0)


def test_select_brute_force_all_subsets(orc):
    # the kept set maximises the score sum; among maximisers it is the lexicographically smallest
    r = rng(7)
    for trial in range(40):
        L = int(r.integers(1, 12))
        S, W = int(r.integers(0, 3)), int(r.integers(0, 3))
        s = r.integers(-2, 3, L).astype(np.float64)           # few distinct values: ties everywhere
        lo, hi = min(S, L), max(min(S, L), L - W)
        k = int(r.integers(0, hi - lo + 2))
        kk = min(k, hi - lo)
        best = max(itertools.combinations(range(lo, hi), kk),
                   key=lambda c: (sum(s[list(c)]), tuple(-i for i in c))) if kk > 0 else ()
        assert tuple(orc.select(s, S, W, k)) == tuple(best), (L, S, W, k, s)


def test_select_boundary_duplicates_keep_lowest_indices(orc):
    s = np.linspace(0.0, 1.0, 64)
    dup = [5, 17, 33, 40, 59]
    s[dup] = 7.0
    s[[2, 3]] = 9.0                                           # two clear winners
    got = orc.select(s, 0, 0, 5)                              # room for 3 of the 5 equal scores
    assert list(got) == [2, 3, 5, 17, 33]
    neg = np.zeros(8)
    neg[[1, 4]] = -0.0                                        # -0.0 ties with +0.0
    assert list(orc.select(neg, 0, 0, 3)) == [0, 1, 2]


def test_select_edge_cases(orc):
    s = rng(8).standard_normal(50)
    assert len(orc.select(s, 0, 0, 0)) == 0                   # no budget: sinks + window only
    assert list(orc.select(s, 10, 45, 8)) == []               # L <= S + W: no candidates
    assert list(orc.select(s, 4, 6, 1000)) == list(range(4, 44))   # budget >= candidates: all of them
    assert orc.candidate_range(50, 4, 6) == (4, 44)
    assert orc.candidate_range(3, 4, 6) == (3, 3)


# ------------------------------------------------------------------ P6: neighbour fetching

def test_neighbors_radius_zero_is_identity(orc):
    idx = np.array([3, 4, 9, 20], np.int32)
    for mode in (orc.NEIGHBOR_DILATE, orc.NEIGHBOR_CLUSTER):
        assert np.array_equal(orc.neighbors(idx, 0, mode, 2, 30), idx)


@pytest.mark.parametrize("r_", [1, 2, 3])
def test_neighbors_dilate_is_binary_dilation(orc, r_):
    r = rng(9 + r_)
    lo, hi = 5, 400
    idx = np.sort(r.choice(np.arange(lo, hi), 60, replace=False)).astype(np.int32)
    mask = np.zeros(hi + 10, int)
    mask[idx] = 1
    dil = np.convolve(mask, np.ones(2 * r_ + 1, int), mode="same") > 0
    want = np.array([p for p in np.flatnonzero(dil) if lo <= p < hi])
    got = orc.neighbors(idx, r_, orc.NEIGHBOR_DILATE, lo, hi)
    assert np.array_equal(got, want)
    assert set(idx) <= set(got)


def test_neighbors_cluster_worked_example(orc):
    d = {}
    for line in open(os.path.join(GOLDEN, "neighbor_cluster_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        d[k] = [int(x) for x in v]
    got = orc.neighbors(np.array(d["selected"], np.int32), d["r"][0], orc.NEIGHBOR_CLUSTER, d["lo"][0], d["hi"][0])
    assert list(got) == d["expanded"]
    assert len(got) == 2 * len(d["selected"])


def test_neighbors_cluster_gives_2B_unique_positions(orc):
    # "2B unique positions": holds whenever runs are far enough apart and away from the ends
    r = rng(12)
    starts = np.arange(100, 5000, 60)
    idx = np.concatenate([np.arange(s, s + int(r.integers(1, 12))) for s in starts]).astype(np.int32)
    for rad in (1, 2):
        got = orc.neighbors(idx, rad, orc.NEIGHBOR_CLUSTER, 10, 6000)
        assert len(got) == (1 + rad) * len(idx)
        assert len(np.unique(got)) == len(got) and np.all(np.diff(got) > 0)
        assert set(idx) <= set(got)
    # clipping at the candidate range, collisions merge
    got = orc.neighbors(np.array([10, 11, 13], np.int32), 1, orc.NEIGHBOR_CLUSTER, 10, 15)
    assert list(got) == [10, 11, 12, 13, 14]
    assert np.all((got >= 10) & (got < 15))


# ------------------------------------------------------------------ P2/P11: attention

@pytest.mark.parametrize("dtype", [F32, BF16])
def test_dense_attention_is_float64_softmax(orc, dtype):
    r = rng(13)
    L, D, g = 77, 128, 4
    q, K, V = rand_storage(r, (g, D), dtype), rand_storage(r, (L, D), dtype), rand_storage(r, (L, D), dtype)
    out, lse = orc.dense_attention(q, K, V, dtype)
    x = f64(q, dtype) @ f64(K, dtype).T / np.sqrt(D)
    p = np.exp(x - x.max(1, keepdims=True))
    p /= p.sum(1, keepdims=True)
    assert np.allclose(out, p @ f64(V, dtype), rtol=1e-12, atol=1e-13)
    assert np.allclose(lse, np.log(np.exp(x).sum(1)), rtol=1e-12)
    # swapping the roles of K and V must change the result
    out_swapped, _ = orc.dense_attention(q, V, K, dtype)
    assert not np.allclose(out_swapped, out)


def test_attention_invariants(orc):
    r = rng(14)
    L, D, g = 200, 128, 2
    q, K, V = rand_storage(r, (g, D), F32), rand_storage(r, (L, D), F32), rand_storage(r, (L, D), F32)
    A = np.sort(r.choice(L, 50, replace=False)).astype(np.int32)
    out, lse = orc.attention(q, K, V, A, F32)
    Vf = V[A].astype(np.float64)
    assert np.all(out <= Vf.max(0) + 1e-12) and np.all(out >= Vf.min(0) - 1e-12)   # convex combination
    perm = r.permutation(len(A))
    out_p, lse_p = orc.attention(q, K, V, A[perm], F32)
    assert np.allclose(out_p, out, rtol=1e-12, atol=1e-13) and np.allclose(lse_p, lse, rtol=1e-13)
    # split-K merge of any partition equals the unsplit result
    parts = np.array_split(perm, 3)
    os_, ls_ = zip(*[orc.attention(q, K, V, A[p], F32) for p in parts])
    M = np.max(ls_, 0)
    wts = np.exp(np.array(ls_) - M)
    merged = (np.array(os_) * wts[:, :, None]).sum(0) / wts.sum(0)[:, None]
    assert np.allclose(merged, out, rtol=1e-11, atol=1e-13)
    assert np.allclose(M + np.log(wts.sum(0)), lse, rtol=1e-12)
    # single attended row: output is that V row, lse is its logit
    o1, l1 = orc.attention(q, K, V, np.array([7], np.int32), F32)
    assert np.allclose(o1, np.broadcast_to(V[7].astype(np.float64), (g, D)))
    assert np.allclose(l1, (q.astype(np.float64) @ K[7].astype(np.float64)) / np.sqrt(D))
    # sm_scale is honoured
    o2, _ = orc.attention(q, K, V, A, F32, sm_scale=0.0)
    assert np.allclose(o2, np.broadcast_to(Vf.mean(0), (g, D)))


# ------------------------------------------------------------------ P1/P7: the chained step

def make_units(orc, r, n, L, cap_L, D, dp, dtype, cap):
    units, W = [], rand_storage(r, (D, dp), dtype, 1 / np.sqrt(D))
    for _ in range(n):
        K, V = rand_storage(r, (cap_L, D), dtype), rand_storage(r, (cap_L, D), dtype)
        units.append(orc.Unit(K, V, orc.project_keys(K, W, dtype), cap))
    return units


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_full_budget_sparse_equals_dense_bitwise(orc, dtype):
    # Sec. 4 policy by construction: sinks + all candidates + window = every token
    r = rng(15)
    L, D, dp, g = 333, 128, 32, 4
    units = make_units(orc, r, 3, L, L, D, dp, dtype, L)
    qi = [r.standard_normal((g, dp)).astype(np.float32) for _ in units]
    qs = [rand_storage(r, (g, D), dtype) for _ in units]
    out = orc.step_units(units, [L] * 3, qi, qs, [1] * 3, g=g, D=D, dp=dp, dtype=dtype, budget=L, sinks=5, recent=20,
                         n_threads=2)
    for i, u in enumerate(units):
        dense, _ = orc.dense_attention(qs[i], u.K[:L], u.V[:L], dtype)
        assert np.array_equal(out[i], dense)
        assert u.cnt[0] == L - 25


def test_interval_reuses_stale_list_and_window_slides(orc):
    r = rng(16)
    L0, D, dp, g, S, Wn, Bud, P = 300, 128, 32, 2, 3, 8, 20, 4
    steps = 9
    units = make_units(orc, r, 2, L0, L0 + steps, D, dp, BF16, 3 * Bud)
    prev = None
    for t in range(steps):
        L = L0 + t
        refresh = int(orc.is_prediction_step(t, P))
        assert refresh == int(t in (0, 4, 8))
        qi = [r.standard_normal((g, dp)).astype(np.float32) for _ in units]
        qs = [rand_storage(r, (g, D), BF16) for _ in units]
        out = orc.step_units(units, [L] * 2, qi, qs, [refresh] * 2, g=g, D=D, dp=dp, dtype=BF16, budget=Bud, sinks=S,
                             recent=Wn, radius=1, nmode=orc.NEIGHBOR_DILATE)
        lists = [u.idx[:u.cnt[0]].copy() for u in units]
        if not refresh:
            assert all(np.array_equal(a, b) for a, b in zip(lists, prev))    # stale list untouched
        else:
            # a refresh equals the separately computed pipeline at the current length
            for i, u in enumerate(units):
                s = orc.score(qi[i], u.Kimp[:L], BF16)
                base = orc.select(s, S, Wn, Bud)
                lo, hi = orc.candidate_range(L, S, Wn)
                assert np.array_equal(lists[i], orc.neighbors(base, 1, orc.NEIGHBOR_DILATE, lo, hi))
        prev = lists
        for i, u in enumerate(units):
            A = orc.attended_set(L, S, Wn, lists[i])
            assert len(np.unique(A)) == len(A) == S + len(lists[i]) + Wn      # three disjoint parts
            assert np.all(A[-Wn:] == np.arange(L - Wn, L))                     # window follows L every step
            ref, _ = orc.attention(qs[i], u.K[:L], u.V[:L], A, BF16)
            assert np.array_equal(out[i], ref)


def test_interval_one_is_per_step_selection(orc):
    # P = 1: every step predicts, and each step's stored list is the plain definition (numpy float64
    # scores, lexsort) at that step's length and with that step's importance query -- not a stale one
    r = rng(17)
    L0, D, dp, g, S, Wn, Bud = 128, 128, 16, 2, 2, 4, 10
    units = make_units(orc, rng(18), 1, L0, L0 + 3, D, dp, F32, Bud)
    for t in range(3):
        assert orc.is_prediction_step(t, 1)
        L = L0 + t
        qi = [r.standard_normal((g, dp)).astype(np.float32)]
        qs = [rand_storage(r, (g, D), F32)]
        orc.step_units(units, [L], qi, qs, [int(orc.is_prediction_step(t, 1))], g=g, D=D, dp=dp, dtype=F32, budget=Bud, sinks=S,
                       recent=Wn)
        s = f64(units[0].Kimp[:L], F32) @ qi[0].astype(np.float64).sum(0)
        assert np.array_equal(units[0].idx[:units[0].cnt[0]], lexsort_select(s, S, Wn, Bud))


def test_prediction_steps_are_the_multiples_of_the_interval(orc):
    # Sec. 3.4: the pipeline runs once every N steps, starting with the first sparse step (nothing to
    # reuse before it); T steps cost ceil(T / N) predictions ("T to about T/N"), 16 at N = 16 over 256 steps
    for P in (1, 2, 4, 16):
        steps = [t for t in range(256) if orc.is_prediction_step(t, P)]
        assert steps == list(range(0, 256, P)) and len(steps) == -(-256 // P)
        gaps = np.diff(steps)
        assert len(gaps) == 0 or np.all(gaps == P)                   # exactly P - 1 reuse steps between two predictions
    assert sum(orc.is_prediction_step(t, 16) for t in range(256)) == 16
    assert sum(orc.is_prediction_step(t, 4) for t in range(9)) == 3  # steps 0, 4, 8


# ------------------------------------------------------------------ values the paper prints

def test_table6_parameter_counts_fix_projection_shape():
    # params = n_prod (E*512 + 512*Hq*G*d' + 2E)  [LN + two bias-free linears per producer]
    #        + n_prod * n_layers * Hkv * D * d'     [a D x d' key projection per layer AND per KV head]
    G, dp, hidden = 4, 16, 512
    for line in open(os.path.join(GOLDEN, "table6_param_counts.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, nl, E, Hq, Hkv, D, exact = line.split()
        nl, E, Hq, Hkv, D, exact = map(int, (nl, E, Hq, Hkv, D, exact))
        n_prod = nl // G
        per_head = n_prod * (E * hidden + hidden * Hq * G * dp + 2 * E) + n_prod * nl * Hkv * D * dp
        assert per_head == exact, name
        shared = n_prod * (E * hidden + hidden * Hq * G * dp + 2 * E) + n_prod * nl * D * dp
        assert shared != exact                                     # one matrix per layer would not fit the table


def test_attended_row_counts_match_paper_budgets(orc):
    for line in open(os.path.join(GOLDEN, "rule_budget_examples.txt")):
        if line.startswith("#") or not line.strip():
            continue
        L, S, W, bud, total, red = line.split()
        L, S, W, bud, total = map(int, (L, S, W, bud, total))
        s = rng(L).standard_normal(L)
        I = orc.select(s, S, W, bud)
        A = orc.attended_set(L, S, W, I)
        assert len(A) == total == S + bud + W
        if red != "-":
            assert "%.2f" % (L / len(A)) == red


def test_planted_tokens_are_all_recalled(orc):
    # closed form: a planted key scores 0.9*|q|*sqrt(d') ~ 0.9*sqrt(g*d')*sqrt(d'), far above the
    # (1 - 2048/131072) quantile of the N(0, |q|^2) background
    w = wl.workload(4, n_layers=1)
    L = w.lengths[0]
    W = wl.gen_W(w, 0)
    K, _ = wl.gen_KV(w, 0, 0)
    _, qi = wl.gen_queries(w, 0, 0)
    K = K[:1].copy()                                               # one KV head is enough
    w1 = w.scaled(n_kv_heads=1, n_q_heads=w.group)
    pos = wl.plant_keys(w1, 0, 0, K, W[:1], qi[:w.group])
    kimp = orc.project_keys(K[0], W[0], BF16)
    s = orc.score(qi[:w.group], kimp, BF16)
    qn = np.linalg.norm(qi[:w.group].astype(np.float64).sum(0))
    assert np.all(np.abs(s[pos[0]] / (0.9 * qn * np.sqrt(w.imp_dim)) - 1) < 0.05)
    I = orc.select(s, w.sinks, w.recent, w.budget)
    assert len(I) == w.budget
    assert set(pos[0]) <= set(I)


# ------------------------------------------------------------------ importance-query predictor (Sec. 3.1, App. A)

@pytest.mark.parametrize("dtype", [F32, BF16])
@pytest.mark.parametrize("act", [0, 1, 2])
def test_predictor_is_layernorm_then_two_float64_matmuls(orc, dtype, act):
    """q = W2 act(W1 LN(h)): every stage against numpy / math library routines in float64, with a
    layer norm that has both weight and bias and linears without bias (Table 6)."""
    import math
    r = rng(310 + act)
    n_tok, E, hid, heads, slots, dp = 3, 96, 40, 4, 2, 8
    out = slots * heads * dp
    H = rand_storage(r, (n_tok, E), dtype, 2.0)
    H[1] = wl.to_storage((wl.storage_to_f32(H[1], dtype) + 7.0).astype(np.float32), dtype)    # a token with a large mean
    ln_w, ln_b = rand_storage(r, (E,), dtype), rand_storage(r, (E,), dtype, 0.3)
    W1, W2 = rand_storage(r, (hid, E), dtype, E ** -0.5), rand_storage(r, (out, hid), dtype, hid ** -0.5)
    q = orc.predict_queries(H, ln_w, ln_b, W1, W2, dtype, eps=1e-5, act=act)
    h = f64(H, dtype)
    x = (h - h.mean(axis=1, keepdims=True)) / np.sqrt(h.var(axis=1, keepdims=True) + 1e-5) * f64(ln_w, dtype) + f64(ln_b, dtype)
    pre = x @ f64(W1, dtype).T
    if act == 0:
        u = np.array([[0.5 * v * (1.0 + math.erf(v / math.sqrt(2.0))) for v in row] for row in pre])
    elif act == 1:
        u = pre / (1.0 + np.exp(-pre))
    else:
        u = np.maximum(pre, 0.0)
    ref = u @ f64(W2, dtype).T
    assert q.shape == (n_tok, out)
    assert np.allclose(q, ref, rtol=1e-12, atol=1e-12)


def test_predictor_closed_forms(orc):
    """Special cases with known answers: a constant hidden state normalises to the LN bias alone; GELU
    at 0, +1, -1 (0, Phi(1), -Phi(-1)); identity-like weights pass the normalised input through."""
    E = 8
    one = np.ones((1, E), np.float32)
    eye = np.eye(E, dtype=np.float32)
    # constant token: (h - mean) = 0, so x = ln_b whatever ln_w is; ReLU and identity weights return it
    b = np.linspace(0.5, 4.0, E).astype(np.float32)
    q = orc.predict_queries(3.25 * one, 9.0 * one[0], b, eye, eye, F32, act=2)
    assert np.allclose(q[0], b, rtol=0, atol=1e-12)
    # h = (+1, -1, +1, -1, ...): mean 0, variance 1, so x = h / sqrt(1 + eps); GELU(x) by its closed form
    h = np.tile(np.array([1.0, -1.0], np.float32), E // 2)[None]
    q = orc.predict_queries(h, one[0], 0 * one[0], eye, eye, F32, eps=0.0, act=0)
    assert np.allclose(q[0, 0], 0.8413447460685429, atol=1e-12) and np.allclose(q[0, 1], -0.15865525393145707, atol=1e-12)
    q = orc.predict_queries(h, one[0], 0 * one[0], eye, eye, F32, eps=0.0, act=1)
    assert np.allclose(q[0, 0], 1.0 / (1.0 + np.exp(-1.0)), atol=1e-12) and np.allclose(q[0, 1], -1.0 / (1.0 + np.exp(1.0)), atol=1e-12)
    # scale invariance of the layer norm (eps = 0): 5 h gives the same queries as h
    r = rng(311)
    H = r.standard_normal((2, E)).astype(np.float32)
    W1, W2 = r.standard_normal((6, E)).astype(np.float32), r.standard_normal((4, 6)).astype(np.float32)
    qa = orc.predict_queries(H, one[0], b, W1, W2, F32, eps=0.0)
    qb = orc.predict_queries((4.0 * H).astype(np.float32), one[0], b, W1, W2, F32, eps=0.0)   # 4 h is exact in fp32
    assert np.allclose(qa, qb, rtol=1e-12, atol=1e-12)


def test_per_layer_projection_is_the_sum_of_the_heads_projections(orc):
    """One list per layer (App. "additional evaluation", head-less predictor): the projection of a token's
    concatenated key [Hkv*D] by the stacked W_K [Hkv*D][d'] is the sum over heads of the per-head
    projections; checked on integer-valued inputs, where both sides are exact."""
    rng = np.random.default_rng(5)
    Hkv, T, D, dp = 4, 9, 128, 16
    K = rng.integers(-3, 4, size=(Hkv, T, D)).astype(np.float32)
    W = rng.integers(-2, 3, size=(Hkv, D, dp)).astype(np.float32)
    _, cat = orc.project_keys(np.ascontiguousarray(np.concatenate(list(K), axis=1)), np.ascontiguousarray(np.concatenate(list(W), axis=0)),
                              orc.F32, want_f64=True)
    per_head = sum(orc.project_keys(np.ascontiguousarray(K[h]), np.ascontiguousarray(W[h]), orc.F32, want_f64=True)[1] for h in range(Hkv))
    assert np.array_equal(cat, per_head)
    assert np.array_equal(cat, np.einsum("htc,hcj->tj", K.astype(np.float64), W.astype(np.float64)))
