"""Boundary behaviour of the C ABI on the GPU: errors found before the first launch, the bounded-wait
path of the selection kernel in its safe form, and the analytic byte counter behind every roofline
figure."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2503_07518_b200 import workloads as wl  # noqa: E402
from test_gpu_parity import H, tb  # noqa: E402,F401


def test_bounded_wait_runs_out_and_the_context_stays_usable(H):
    """One tile's barrier is armed without its copy being requested (diagnostic hook, single-block launch
    only, so nothing else is in flight and no other block waits).  The wait gives up after its poll
    limit, the kernel finishes normally, the status word says TB_ERR_TIMEOUT, and the next ordinary call
    on the same context is clean and exact."""
    b_ = tb()
    w = wl.workload(2, n_layers=1, n_q_heads=4, n_kv_heads=1, lengths=[900], budget=50)     # 4 tiles, one block
    case = H.Case(w)
    q, qi = H.queries(w)
    p = b_.select_params(w.budget, 0, 0)
    clean = H.gpu_select(case, qi, p)
    assert case.ctx.get_status() == 0
    case.ctx.set_wait_diagnostics(poll_limit=2000, drop_tile=1)
    n0 = case.ctx.launch_count()
    lost = H.gpu_select(case, qi, p)
    assert case.ctx.launch_count() > n0                                  # the kernel ran and returned
    assert case.ctx.get_status() == b_.TB_ERR_TIMEOUT
    assert case.ctx.get_status() == 0                                    # reading clears it
    assert len(lost[0][0][0]) == w.budget and np.all((lost[0][0][0] >= 0) & (lost[0][0][0] < 900))   # void, but in range
    case.ctx.set_wait_diagnostics(0, -1)
    again = H.gpu_select(case, qi, p)
    assert case.ctx.get_status() == 0
    _, full, _ = case.oracle_select(0, 0, 0, qi[0, 0], p)
    assert np.array_equal(again[0][0][0], clean[0][0][0]) and np.array_equal(again[0][0][0], full)
    out, _ = H.gpu_attention(case, q, p)                                 # and attention from the stored list still matches
    ref, _ = case.oracle_attention(0, 0, 0, q[0, 0], full, p)
    assert np.abs(out[0, 0] - ref).max() <= 2e-3


def test_wait_diagnostics_are_refused_by_multi_block_launches(H):
    """The hook never reaches a launch in which another block could be left waiting: such a call returns
    TB_ERR_UNSUPPORTED and launches nothing."""
    b_ = tb()
    w = wl.workload(2, n_layers=1, n_q_heads=8, n_kv_heads=2, lengths=[5000], budget=50)    # two lists, clusters
    case = H.Case(w)
    _, qi = H.queries(w)
    case.ctx.set_wait_diagnostics(poll_limit=2000, drop_tile=0)
    n0 = case.ctx.launch_count()
    with pytest.raises(b_.TBError) as e:
        H.gpu_select(case, qi, b_.select_params(w.budget))
    assert e.value.status == b_.TB_ERR_UNSUPPORTED and case.ctx.launch_count() == n0
    case.ctx.set_wait_diagnostics(0, -1)
    H.gpu_select(case, qi, b_.select_params(w.budget))
    assert case.ctx.get_status() == 0


def test_oversized_neighbour_span_is_refused_before_anything_runs(H):
    """Neighbour expansion keeps one bit per candidate on chip (up to 1,638,272 candidates).  A longer
    sequence is selected from without neighbours, and refused with them -- before the selection kernel of
    the same call is launched, not after it."""
    b_ = tb()
    L = 1_700_000
    ctx = b_.Context(1, 1, 1, 128, 32, b_.TB_BF16, 1, L + 8, 64, max_radius=1)
    ctx.set_projection(0, torch.zeros(1, 128, 32, dtype=torch.bfloat16, device="cuda"))
    k = torch.zeros(L, 1, 128, dtype=torch.bfloat16, device="cuda")
    k[::1000, 0, 0] = 1.0
    ctx.append_kv(0, 1, None, [L], k, k)
    ctx.project_keys(0, 1, None, [0], [L])
    qi = torch.ones(1, 1, 1, 32, device="cuda")
    idx = torch.zeros(1, 1, 1, ctx.index_capacity, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, 1, 1, dtype=torch.int32, device="cuda")
    ctx.select_topk(0, 1, None, 1, qi, b_.select_params(64), idx, cnt)           # all scores equal: the first 64 positions
    torch.cuda.synchronize()
    assert cnt.item() == 64 and np.array_equal(idx[0, 0, 0, :64].cpu().numpy(), np.arange(64))
    n0 = ctx.launch_count()
    with pytest.raises(b_.TBError) as e:
        ctx.select_topk(0, 1, None, 1, qi, b_.select_params(64, radius=1), idx, cnt)
    assert e.value.status == b_.TB_ERR_UNSUPPORTED
    assert ctx.launch_count() == n0 and ctx.get_length(0, 0) == (L, L)
    out = torch.empty(1, 1, 128, device="cuda")
    ctx.sparse_decode_attention(0, 1, None, 1, k[:1, 0], b_.select_params(64), out)   # the stored list is still the first call's
    assert ctx.get_status() == 0


def test_byte_counter_reproduces_the_papers_bandwidth_reduction(H):
    """tb_last_step_bytes is the numerator of every roofline figure.  At 64K tokens with about 8K
    accessed (128 sinks + 7808 selected + 256 recent) the K/V bytes of a sparse step are 1/8.00 of the
    dense step's (Sec. 4.2: "8x" KV-access reduction); the selection reads d' elements per candidate
    and key stream."""
    b_ = tb()
    L, S, W, B = 65536, 128, 256, 7808
    ctx = b_.Context(1, 32, 8, 128, 32, b_.TB_BF16, 1, L + 8, B)
    ctx.set_projection(0, torch.zeros(8, 128, 32, dtype=torch.bfloat16, device="cuda"))
    k = torch.zeros(L, 8, 128, dtype=torch.bfloat16, device="cuda")
    ctx.append_kv(0, 1, None, [L], k, k)
    ctx.project_keys(0, 1, None, [0], [L])
    p = b_.select_params(B, S, W)
    ctx.select_topk(0, 1, None, 1, torch.ones(1, 1, 32, 32, device="cuda"), p)
    assert ctx.last_step_bytes() == (L - S - W) * 8 * 32 * 2
    q = torch.zeros(1, 32, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.empty(1, 32, 128, device="cuda")
    ctx.sparse_decode_attention(0, 1, None, 1, q, p, out)
    sparse = ctx.last_step_bytes()
    ctx.sparse_decode_attention(0, 1, None, 1, q, b_.select_params(-1), out)
    dense = ctx.last_step_bytes()
    assert sparse == (S + B + W) * 8 * 2 * 128 * 2 == 8192 * 8 * 512
    assert dense == L * 8 * 512 and dense / sparse == 8.0
    assert ctx.get_status() == 0


def test_captured_graphs_replay_a_growing_sequence(H):
    """Device-resident lengths: two CUDA graphs, captured once -- a refresh step (append, projection of the
    unprojected tokens, selection with neighbours, attention) and a reuse step (append, attention from the stale
    lists) -- are replayed over a decode trajectory.  Every replay must see the sequence one token longer:
    lists and attention are checked against the oracle at each step's true length, the projected keys
    against the oracle's projection, and the device counters against the lengths at the end."""
    b_ = tb()
    P, Wn, steps = 4, 8, 11
    w = wl.workload(5, n_layers=2, batch=2, n_q_heads=8, n_kv_heads=2, lengths=[1200, 700], budget=90, recent=Wn,
                    radius=1, interval=P, decode_steps=steps)
    case = H.Case(w, extra_len=steps + 2)
    ctx = case.ctx
    ctx.use_device_lengths(True, growth_reserve=steps + 2)
    dt = torch.bfloat16
    k_new = torch.zeros(w.n_layers, w.batch, w.n_kv_heads, w.head_dim, dtype=dt, device="cuda")
    v_new = torch.zeros_like(k_new)
    q_d = torch.zeros(w.n_layers, w.batch, w.n_q_heads, w.head_dim, dtype=dt, device="cuda")
    qi_d = torch.zeros(w.n_layers, w.batch, w.n_q_heads, w.imp_dim, device="cuda")
    out = torch.zeros(w.n_layers, w.batch, w.n_q_heads, w.head_dim, device="cuda")
    cap = ctx.index_capacity
    idx = torch.zeros(w.n_layers, w.batch, w.n_kv_heads, cap, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(w.n_layers, w.batch, w.n_kv_heads, dtype=torch.int32, device="cuda")
    p_refresh = b_.select_params(w.budget, 0, Wn, 1, 0, P, 0)
    p_reuse = b_.select_params(w.budget, 0, Wn, 1, 0, P, 1)

    def one_step(p):
        for l in range(w.n_layers):
            ctx.append_kv(l, 1, None, [1] * w.batch, k_new[l], v_new[l])
        if p.step % P == 0:
            ctx.project_keys(0, w.n_layers, None, None, None, n_seq=w.batch)
        ctx.select_topk(0, w.n_layers, None, w.batch, qi_d, p, idx, cnt)
        for l in range(w.n_layers):
            ctx.sparse_decode_attention(l, 1, None, w.batch, q_d[l], p, out[l])

    stream = torch.cuda.Stream()
    graphs = {}
    with torch.cuda.stream(stream):
        for name, p in (("refresh", p_refresh), ("reuse", p_reuse)):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                one_step(p)
            graphs[name] = g
        ctx.sync_lengths(stream)                       # capturing advanced only the host mirrors: back to the truth
        assert [ctx.get_length(0, b) for b in range(w.batch)] == [(1200, 1200), (700, 700)]
        stored = None
        for t in range(steps):
            # this step's inputs, and the host copies of the rows the graph will append
            Ks = [[wl.gen_KV(w, l, b, n_tokens=1, start=t + 1) for b in range(w.batch)] for l in range(w.n_layers)]
            for l in range(w.n_layers):
                for b in range(w.batch):
                    K, V = Ks[l][b]
                    case.K[l][b][:, case.cur[b]] = K[:, 0]
                    case.V[l][b][:, case.cur[b]] = V[:, 0]
                    k_new[l, b] = H.to_dev(K[:, 0], w.dtype)
                    v_new[l, b] = H.to_dev(V[:, 0], w.dtype)
            case.cur = [c + 1 for c in case.cur]
            q, qi = H.queries(w, t)
            q_d.copy_(H.to_dev(q, w.dtype))
            qi_d.copy_(torch.from_numpy(qi).cuda())
            refresh = H.orc.is_prediction_step(t, P)
            graphs["refresh" if refresh else "reuse"].replay()
            torch.cuda.synchronize()
            assert ctx.get_status(stream) == 0
            p = b_.select_params(w.budget, 0, Wn, 1, 0, P, t)
            idx_h, cnt_h, out_h = idx.cpu().numpy(), cnt.cpu().numpy(), out.cpu().numpy()
            lists = [[[idx_h[l, b, h, :cnt_h[l, b, h]] for h in range(2)] for b in range(w.batch)] for l in range(w.n_layers)]
            if refresh:
                for l in range(w.n_layers):
                    for b in range(w.batch):
                        L = case.cur[b]
                        dev = H.to_host(ctx.kimp[l, b, :, :L], w.dtype)           # the device's own projected keys
                        for h in range(2):
                            # newly projected rows obey the projection's error bound
                            lo_new = case.proj[b]
                            ref = H.orc.project_keys(np.ascontiguousarray(case.K[l][b][h, lo_new:L]), np.ascontiguousarray(case.W[l][h]), w.dtype)
                            assert H.projection_excess(dev[h, lo_new:L], ref, case.K[l][b][h, lo_new:L], case.W[l][h], w.dtype) <= 1.0
                            s = H.orc.score(qi[l, b][h * 4:(h + 1) * 4], np.ascontiguousarray(dev[h]), w.dtype)
                            base = H.orc.select(s, 0, Wn, w.budget)
                            lo, hi = H.orc.candidate_range(L, 0, Wn)
                            assert np.array_equal(lists[l][b][h], H.orc.neighbors(base, 1, 0, lo, hi)), (t, l, b, h)
                case.proj = list(case.cur)
                stored = [[[x.copy() for x in lb_] for lb_ in ll_] for ll_ in lists]
            else:
                assert all(np.array_equal(lists[l][b][h], stored[l][b][h]) for l in range(2) for b in range(2) for h in range(2))
            for l in range(w.n_layers):
                for b in range(w.batch):
                    for h in range(2):
                        ref, _ = case.oracle_attention(l, b, h, q[l, b], stored[l][b][h], p)
                        assert np.abs(out_h[l, b, h * 4:(h + 1) * 4] - ref).max() <= 2e-3, (t, l, b, h)
        ctx.sync_lengths(stream)
        assert [ctx.get_length(1, b) for b in range(w.batch)] == [(1200 + steps, 1200 + 9), (700 + steps, 700 + 9)]   # last refresh at t = 8
    ctx.use_device_lengths(False)
    # back on host-carried lengths the same context goes on as usual
    full = H.gpu_select(case, H.queries(w, 99)[1], b_.select_params(w.budget, 0, Wn, 0))
    assert ctx.get_status() == 0 and len(full[0][0][0]) == w.budget


@pytest.mark.parametrize("on_host", [False, True])
def test_resident_rows_and_important_buffer_give_the_same_bits(H, on_host):
    """Offloaded-KV options (Sec. 4.4) and the paper's contiguous Important buffer (Sec. 3.3): device copies of
    the sink and window rows kept current by the appends, and the selected rows migrated into a contiguous
    buffer at every refresh.  Both only change where a row is read from, so every output must be bit-equal to
    the plain index-driven gather -- over a trajectory in which the window slides, the selection is reused for
    P steps, and the sink / window sizes asked for are smaller than, equal to and larger than the copies."""
    b_ = tb()
    P, steps = 3, 7
    w = wl.workload(5, n_layers=2, batch=2, n_q_heads=8, n_kv_heads=2, lengths=[900, 333], budget=60, sinks=5, recent=12,
                    radius=1, interval=P, decode_steps=steps)

    def run(resident, important):
        outs = []
        ctx_args = dict(extra_len=steps + 2, kv_on_host=on_host, project=None)
        # the copies must be bound before the first append: build the context by hand, then fill it
        case = H.Case.__new__(H.Case)
        case.w, case.lengths = w, list(w.lengths)
        case.cap = max(case.lengths) + steps + 2
        case.ctx = b_.Context(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.imp_dim, w.dtype, w.batch, case.cap, w.budget,
                              w.radius, kv_on_host=on_host)
        if resident:
            case.ctx.bind_resident_rows(sinks=8, window=16)
        if important:
            case.ctx.bind_important_buffer()
        case.Hi = case.Hl = case.Ha = w.n_kv_heads
        case.gl = case.ga = w.group
        case.K = [[None] * w.batch for _ in range(w.n_layers)]
        case.V = [[None] * w.batch for _ in range(w.n_layers)]
        case.Kimp = [[np.zeros((2, case.cap, w.imp_dim), np.uint16) for _ in range(w.batch)] for _ in range(w.n_layers)]
        case.W = []
        for l in range(w.n_layers):
            case.W.append(wl.gen_W(w, l))
            case.ctx.set_projection(l, H.to_dev(case.W[l], w.dtype))
            Ks, Vs = [], []
            for b in range(w.batch):
                K, V = wl.gen_KV(w, l, b)
                case.K[l][b] = np.zeros((2, case.cap, w.head_dim), K.dtype)
                case.V[l][b] = np.zeros_like(case.K[l][b])
                case.K[l][b][:, :w.lengths[b]] = K
                case.V[l][b][:, :w.lengths[b]] = V
                Ks.append(K), Vs.append(V)
            case._append_layer(l, Ks, Vs)
        case.cur, case.proj = list(w.lengths), [0] * w.batch
        case.project_all(compare=False)
        for t in range(steps):
            if t > 0:
                case.append_step(t)
                case.project_range(list(case.proj), list(case.cur), compare=False)
            q, qi = H.queries(w, t)
            # sink / window sizes below, at and above what the copies hold
            S, Wn = [(5, 12), (8, 16), (11, 20)][t % 3] if t % P == 0 else last
            last = (S, Wn)
            p = b_.select_params(w.budget, S, Wn, 1, 0, P, t)
            lists = H.gpu_select(case, qi, p)
            out, lse = H.gpu_attention(case, q, p)
            assert case.ctx.get_status() == 0
            outs.append((lists, out, lse))
        return case, outs

    base_case, base = run(False, False)
    for resident, important in ((True, False), (False, True), (True, True)):
        _, got = run(resident, important)
        for t in range(steps):
            assert all(np.array_equal(x, y) for l in range(2) for s in range(2) for x, y in zip(base[t][0][l][s], got[t][0][l][s]))
            assert np.array_equal(base[t][1], got[t][1]) and np.array_equal(base[t][2], got[t][2]), (resident, important, t)
    # and the common result is the oracle's (last step, stored lists)
    q, _ = H.queries(w, steps - 1)
    p = b_.select_params(w.budget, *[(5, 12), (8, 16), (11, 20)][((steps - 1) // P * P) % 3], 1, 0, P, steps - 1)
    for l in range(2):
        for b in range(2):
            for h in range(2):
                ref, _ = base_case.oracle_attention(l, b, h, q[l, b], base[-1][0][l][b][h], p)
                assert np.abs(base[-1][1][l, b, h * 4:(h + 1) * 4] - ref).max() <= 2e-3
