"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (score+select per
group of 4 layers, attention per layer).  The caches are drawn on the device exactly as bench.py draws
them; the oracle then checks sampled (layer, sequence, KV head) units on the very bytes the device holds
(units are independent, so a sample of whole units is a sample of whole results)."""
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


class DeviceCase:
    """Full-size state built the way bench.py builds it, plus the per-step inputs."""

    def __init__(self, w, extra_len=8):
        import bench
        from paper_2503_07518_b200 import binding as tb
        self.tb, self.w = tb, w
        self.ctx = tb.Context(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.imp_dim, w.dtype, w.batch,
                              max(w.lengths) + extra_len, w.budget, w.radius)
        bench.fill_caches(self.ctx, w, torch, tb)
        self.cur = list(w.lengths)
        gen = torch.Generator(device="cuda")
        gen.manual_seed(1234)
        self.gen = gen
        self.new_queries()
        self.out = torch.empty(w.n_layers, w.batch, w.n_q_heads, w.head_dim, device="cuda")
        self.lse = torch.empty(w.n_layers, w.batch, w.n_q_heads, device="cuda")
        cap = self.ctx.index_capacity
        self.idx = torch.empty(w.n_layers, w.batch, w.n_kv_heads, cap, dtype=torch.int32, device="cuda")
        self.cnt = torch.empty(w.n_layers, w.batch, w.n_kv_heads, dtype=torch.int32, device="cuda")

    def new_queries(self):
        w = self.w
        self.q = torch.randn(w.n_layers, w.batch, w.n_q_heads, w.head_dim, generator=self.gen, device="cuda").to(torch.bfloat16)
        self.qi = torch.randn(w.n_layers, w.batch, w.n_q_heads, w.imp_dim, generator=self.gen, device="cuda")

    def step(self, p):
        """bench.py's schedule; also copies the stored lists out.  With neighbour fetching on a refresh
        step, the same selection launch is first run with radius 0 (bit-reproducible), so that the
        expansion can be checked exactly against the GPU's own pre-expansion lists."""
        w = self.w
        if p.radius > 0 and p.step % p.interval == 0:
            if not hasattr(self, "idx0"):
                self.idx0, self.cnt0 = torch.empty_like(self.idx), torch.empty_like(self.cnt)
            p0 = self.tb.select_params(p.budget, p.sinks, p.recent, 0, p.nmode, p.interval, p.step, p.reduce, p.score_scale)
            for l0 in range(0, w.n_layers, 4):
                n = min(4, w.n_layers - l0)
                self.ctx.select_topk(l0, n, None, w.batch, self.qi[l0:l0 + n], p0, self.idx0[l0:l0 + n], self.cnt0[l0:l0 + n])
        for l0 in range(0, w.n_layers, 4):
            n = min(4, w.n_layers - l0)
            self.ctx.select_topk(l0, n, None, w.batch, self.qi[l0:l0 + n], p, self.idx[l0:l0 + n], self.cnt[l0:l0 + n])
            for l in range(l0, l0 + n):
                self.ctx.sparse_decode_attention(l, 1, None, w.batch, self.q[l], p, self.out[l], lse=self.lse[l])
        torch.cuda.synchronize()
        assert self.ctx.get_status() == 0

    def unit_host(self, H, l, b, h):
        """Host copies of one unit's cache rows and inputs (storage bytes)."""
        w, L = self.w, self.cur[b]
        kv = H.to_host(self.ctx.kv[l, b, h, :L], w.dtype)                  # [L, 2, D]
        K, V = np.ascontiguousarray(kv[:, 0]), np.ascontiguousarray(kv[:, 1])
        Kimp = H.to_host(self.ctx.kimp[l, b, h, :L], w.dtype)
        g = w.group
        q = H.to_host(self.q[l, b, h * g:(h + 1) * g], w.dtype)
        qi = self.qi[l, b, h * g:(h + 1) * g].cpu().numpy()
        return K, V, Kimp, q, qi


def check_unit(H, case, l, b, h, p, W_host=None, stored=None):
    """Projection bound (if W given), selection parity on the device's K_imp bytes, attention parity."""
    orc, w = H.orc, case.w
    K, V, Kimp, q, qi = case.unit_host(H, l, b, h)
    L = case.cur[b]
    if W_host is not None:
        ref = orc.project_keys(K, np.ascontiguousarray(W_host), w.dtype)
        assert H.projection_excess(Kimp, ref, K, W_host, w.dtype) <= 1.0
    n = int(case.cnt[l, b, h].item())
    got = case.idx[l, b, h, :n].cpu().numpy()
    if stored is None:
        s = orc.score(qi, Kimp, w.dtype)
        base = orc.select(s, p.sinks, p.recent, p.budget)
        lo, hi = orc.candidate_range(L, p.sinks, p.recent)
        if p.radius > 0:
            # the GPU's pre-expansion list obeys the selection rule, and the stored list is exactly the
            # oracle's neighbour rule applied to it
            n0 = int(case.cnt0[l, b, h].item())
            got0 = case.idx0[l, b, h, :n0].cpu().numpy()
            H.check_selection(got0, base, s, "layer %d seq %d head %d" % (l, b, h))
            assert np.array_equal(got, orc.neighbors(got0, p.radius, p.nmode, lo, hi))
        else:
            H.check_selection(got, base, s, "layer %d seq %d head %d" % (l, b, h))
    else:
        assert np.array_equal(got, stored)
    A = orc.attended_set(L, p.sinks, p.recent, got)
    ref, ref_lse = orc.attention(q, K, V, A, w.dtype)
    g = w.group
    dev = case.out[l, b, h * g:(h + 1) * g].cpu().numpy()
    assert np.abs(dev - ref).max() <= H.ATTN_TOL[w.dtype]
    assert np.abs(case.lse[l, b, h * g:(h + 1) * g].cpu().numpy() - ref_lse).max() <= 2e-3
    return got


def test_config2_llama8b_32k_full(H):
    w = wl.workload(2)                                       # 32 layers, 32/8 heads, 32768 tokens, budget 3276
    case = DeviceCase(w)
    p = case.tb.select_params(w.budget, w.sinks, w.recent)
    case.step(p)
    assert int(case.cnt.min()) == int(case.cnt.max()) == w.budget
    for (l, h) in [(0, 0), (3, 7), (13, 2), (31, 5)]:
        check_unit(H, case, l, 0, h, p)
    # dense rule at full size on one unit
    dense = torch.empty_like(case.out[5])
    case.ctx.sparse_decode_attention(5, 1, None, 1, case.q[5], case.tb.select_params(-1), dense)
    K, V, _, q, _ = case.unit_host(H, 5, 0, 3)
    ref, _ = H.orc.dense_attention(q, K, V, w.dtype)
    assert np.abs(dense[0, 12:16].cpu().numpy() - ref).max() <= 2e-3


def test_config3_batched_ragged(H):
    w = wl.workload(3, n_layers=4)                           # all 16 ragged sequences, 4 of the 32 layers
    case = DeviceCase(w)
    p = case.tb.select_params(w.budget, 0, 0)
    case.step(p)
    longest, shortest = int(np.argmax(w.lengths)), int(np.argmin(w.lengths))
    for (l, b, h) in [(0, longest, 0), (1, shortest, 3), (2, 7, 6), (3, 11, 1)]:
        check_unit(H, case, l, b, h, p)


def test_config4_long_context_planted_recall(H):
    w = wl.workload(4, n_layers=4)                           # 131072 tokens, budget 2048 + 16 sinks + 256 recent
    case = DeviceCase(w)
    L = w.lengths[0]
    # plant 64 keys per (layer, KV head) whose projection has cosine 0.9 with the summed importance query
    planted = {}
    qi_host = case.qi.cpu().numpy()
    for l in (0, 2):
        # this layer's W_K exactly as bench.py drew it (first draw of the layer's seeded generator)
        gen = torch.Generator(device="cuda")
        gen.manual_seed(wl.seed_for(w.cfg_id, l, 0, wl.TAG_K))
        Wd = (torch.randn(w.n_kv_heads, w.head_dim, w.imp_dim, generator=gen, device="cuda") / np.sqrt(w.head_dim)).to(torch.bfloat16)
        Wl = H.to_host(Wd, w.dtype)
        K = H.to_host(case.ctx.kv[l, 0, :, :L, 0], w.dtype)                 # [Hkv, L, D]
        pos = wl.plant_keys(w, l, 0, K, Wl, qi_host[l, 0])
        for h in range(w.n_kv_heads):
            rows = torch.from_numpy(pos[h].astype(np.int64)).cuda()
            case.ctx.kv[l, 0, h, rows, 0] = H.to_dev(K[h, pos[h]], w.dtype)
        case.ctx.project_keys(l, 1, None, [0], [L])                          # re-project (planted rows changed)
        planted[l] = (pos, Wl)
    p = case.tb.select_params(w.budget, w.sinks, w.recent)
    case.step(p)
    for l, (pos, Wl) in planted.items():
        for h in range(w.n_kv_heads):
            n = int(case.cnt[l, 0, h].item())
            got = set(case.idx[l, 0, h, :n].cpu().numpy().tolist())
            assert n == w.budget and set(pos[h].tolist()) <= got, "planted tokens missed in layer %d head %d" % (l, h)
    check_unit(H, case, 0, 0, 2, p, W_host=planted[0][1][2])
    check_unit(H, case, 3, 0, 6, p)


def test_config5_interval_trajectory(H):
    # batch 8 x 65536 tokens, 2 of the 32 layers, P = 16, +-1 neighbours, window 16, 34 decode steps
    P = 16
    w = wl.workload(5, n_layers=2)
    steps = 2 * P + 2
    case = DeviceCase(w, extra_len=steps + 16)
    proj = list(w.lengths)
    units = [(0, 0, 0), (1, 5, 7)]
    stored = {}
    for t in range(steps):
        kn = torch.randn(w.n_layers, w.batch, w.n_kv_heads, w.head_dim, generator=case.gen, device="cuda").to(torch.bfloat16)
        vn = torch.randn(w.n_layers, w.batch, w.n_kv_heads, w.head_dim, generator=case.gen, device="cuda").to(torch.bfloat16)
        case.new_queries()
        for l in range(w.n_layers):
            case.ctx.append_kv(l, 1, None, [1] * w.batch, kn[l], vn[l])
            if t % P == 0 and t > 0:
                case.ctx.project_keys(l, 1, None, proj, [x + P for x in proj])
        if t % P == 0 and t > 0:
            proj = [x + P for x in proj]
        case.cur = [x + 1 for x in case.cur]
        p = case.tb.select_params(w.budget, 0, w.recent, 1, 0, P, t)
        case.step(p)
        if t in (0, 1, P - 1, P, P + 1, 2 * P, 2 * P + 1):
            for u in units:
                if t % P == 0:
                    stored[u] = check_unit(H, case, *u, p)
                else:
                    check_unit(H, case, *u, p, stored=stored[u])
