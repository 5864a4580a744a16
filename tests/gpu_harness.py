"""Glue for the GPU parity tests: moves seeded host inputs into a device context through the C ABI,
runs the CPU oracle on the same bytes, and compares with the parity rules.

Parity rules:
  project_keys   |gpu - oracle| <= one unit in the last place of the storage type
                 + D * 2^-24 * sum_c |K_c W_c|  (forward error bound of the fp32 accumulation)
  select_topk    identical index sets, except swaps of tokens whose oracle scores differ by at most
                 1e-5 relative (fp32 vs fp64 accumulation may order such a pair either way)
  attention      max-abs error 2e-3 (bf16 storage) / 1e-5 (fp32 storage), same index list both sides
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import tb_oracle as orc
from paper_2503_07518_b200 import binding as tb
from paper_2503_07518_b200 import workloads as wl

ATTN_TOL = {wl.BF16: 2e-3, wl.F32: 1e-5}


def to_dev(arr: np.ndarray, dtype: int, device="cuda"):
    """numpy storage array (uint16 bf16 bits / float32) -> torch tensor of the storage type."""
    if dtype == wl.BF16:
        return torch.from_numpy(np.ascontiguousarray(arr).view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(arr)).to(device)


def to_host(t: torch.Tensor, dtype: int) -> np.ndarray:
    if dtype == wl.BF16:
        return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return t.contiguous().cpu().numpy()


class Case:
    """A workload instantiated on the host (numpy) and on the device (tb.Context)."""

    def __init__(self, w: wl.Workload, max_budget=None, max_radius=None, extra_len=0, project="device", kv_on_host=False,
                 list_scope=tb.TB_SCOPE_KV_HEAD):
        self.w = w
        self.lengths = list(w.lengths)
        self.cap = max(self.lengths) + extra_len
        self.ctx = tb.Context(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.imp_dim, w.dtype, w.batch, self.cap,
                              max_budget or max(1, w.budget), w.radius if max_radius is None else max_radius, kv_on_host=kv_on_host,
                              list_scope=list_scope)
        # Heads per (layer, sequence) under the selection scope: key streams of the projected-key cache,
        # lists, attention units; importance queries per list and query heads per attention unit.
        self.Hi, self.Hl = self.ctx.n_key_heads, self.ctx.n_lists
        self.Ha = max(self.Hl, w.n_kv_heads)
        self.gl = w.group if list_scope == tb.TB_SCOPE_KV_HEAD else 1
        self.ga = w.n_q_heads // self.Ha
        self.K = [[None] * w.batch for _ in range(w.n_layers)]     # [layer][seq] -> [Hkv, cap, D] storage
        self.V = [[None] * w.batch for _ in range(w.n_layers)]
        self.Kimp = [[None] * w.batch for _ in range(w.n_layers)]  # oracle's projection, [Hkv, cap, d']
        self.W = []
        for l in range(w.n_layers):
            Wl = wl.gen_W(w, l)
            self.W.append(Wl)
            self.ctx.set_projection(l, to_dev(Wl, w.dtype))
            for b in range(w.batch):
                K, V = wl.gen_KV(w, l, b)
                self.K[l][b] = np.zeros((w.n_kv_heads, self.cap, w.head_dim), K.dtype)
                self.V[l][b] = np.zeros_like(self.K[l][b])
                self.Kimp[l][b] = np.zeros((self.Hi, self.cap, w.imp_dim), K.dtype)
                self.K[l][b][:, :self.lengths[b]] = K
                self.V[l][b][:, :self.lengths[b]] = V
            self._append_layer(l, [self.K[l][b][:, :self.lengths[b]] for b in range(w.batch)],
                               [self.V[l][b][:, :self.lengths[b]] for b in range(w.batch)])
        self.cur = list(self.lengths)                              # current length per sequence
        self.proj = [0] * w.batch
        if project:
            self.project_all(compare=(project == "device"))

    # ---- cache maintenance ----------------------------------------------------------------------
    def _append_layer(self, l, Ks, Vs):
        w = self.w
        k = np.concatenate([np.ascontiguousarray(np.transpose(x, (1, 0, 2))) for x in Ks], 0)   # [sum n, Hkv, D]
        v = np.concatenate([np.ascontiguousarray(np.transpose(x, (1, 0, 2))) for x in Vs], 0)
        self.ctx.append_kv(l, 1, None, [x.shape[1] for x in Ks], to_dev(k, w.dtype), to_dev(v, w.dtype))

    def append_step(self, step):
        """Append one new token per sequence in every layer (decode)."""
        w = self.w
        for l in range(w.n_layers):
            Ks, Vs = [], []
            for b in range(w.batch):
                K, V = wl.gen_KV(w, l, b, n_tokens=1, start=step + 1)
                self.K[l][b][:, self.cur[b]] = K[:, 0]
                self.V[l][b][:, self.cur[b]] = V[:, 0]
                Ks.append(K), Vs.append(V)
            self._append_layer(l, Ks, Vs)
        self.cur = [c + 1 for c in self.cur]

    def project_range(self, begin, end, compare=True):
        """Project positions [begin[b], end[b]) on the device, check against the oracle (<= 1 ulp),
        then make the device cache hold the oracle's bytes so later stages see identical inputs."""
        w = self.w
        self.ctx.project_keys(0, w.n_layers, None, begin, end)
        worst = 0
        for l in range(w.n_layers):
            for b in range(w.batch):
                if end[b] <= begin[b]:
                    continue
                # one list per layer: the token's concatenated key [Hkv*D] times the stacked W_K [Hkv*D][d']
                Ks = [self.K[l][b][h, begin[b]:end[b]] for h in range(w.n_kv_heads)] if self.Hi == w.n_kv_heads else \
                    [np.concatenate([self.K[l][b][h, begin[b]:end[b]] for h in range(w.n_kv_heads)], axis=1)]
                Ws = [self.W[l][h] for h in range(w.n_kv_heads)] if self.Hi == w.n_kv_heads else \
                    [np.concatenate([self.W[l][h] for h in range(w.n_kv_heads)], axis=0)]
                for h in range(self.Hi):
                    self.Kimp[l][b][h, begin[b]:end[b]] = orc.project_keys(
                        np.ascontiguousarray(Ks[h]), np.ascontiguousarray(Ws[h]), w.dtype)
                if compare:
                    dev = to_host(self.ctx.kimp[l, b, :, begin[b]:end[b]], w.dtype)
                    for h in range(self.Hi):
                        worst = max(worst, projection_excess(dev[h], self.Kimp[l][b][h, begin[b]:end[b]], Ks[h], Ws[h], w.dtype))
                self.ctx.kimp[l, b, :, begin[b]:end[b]] = to_dev(self.Kimp[l][b][:, begin[b]:end[b]], w.dtype)
        for b in range(w.batch):
            self.proj[b] = max(self.proj[b], end[b])
        if compare:
            assert worst <= 1.0, "project_keys outside its error bound by a factor %.3f" % worst
        return worst

    def project_all(self, compare=True):
        return self.project_range([0] * self.w.batch, list(self.cur), compare)

    # ---- oracle side --------------------------------------------------------------------------------
    def oracle_select(self, l, b, h, q_imp, p):
        """Oracle list (after neighbours) and the fp64 scores, on the oracle's K_imp bytes.  h = list
        head; q_imp = the (layer, sequence)'s importance queries [Hl * gl][d']."""
        w, L = self.w, self.cur[b]
        s = orc.score(q_imp[h * self.gl:(h + 1) * self.gl], np.ascontiguousarray(self.Kimp[l][b][h * self.Hi // self.Hl, :L]), w.dtype,
                      reduce=getattr(p, "reduce", orc.GROUP_SUM))
        base = orc.select(s, p.sinks, p.recent, p.budget)
        lo, hi = orc.candidate_range(L, p.sinks, p.recent)
        full = orc.neighbors(base, p.radius, p.nmode, lo, hi) if p.radius > 0 else base
        return base, full, s

    def oracle_attention(self, l, b, h, q, I, p, dense=False):
        """h = attention unit (a KV head with its group, or one query head); I = the list it reads."""
        w, L = self.w, self.cur[b]
        hk = h * w.n_kv_heads // self.Ha
        K = np.ascontiguousarray(self.K[l][b][hk, :L])
        V = np.ascontiguousarray(self.V[l][b][hk, :L])
        qh = np.ascontiguousarray(q[h * self.ga:(h + 1) * self.ga])
        A = np.arange(L, dtype=np.int32) if dense else orc.attended_set(L, p.sinks, p.recent, I)
        return orc.attention(qh, K, V, A, w.dtype)


def projection_excess(dev, ref, K, W, dtype) -> float:
    """max over elements of |dev - ref| / (ulp(ref) + D 2^-24 sum_c |K_c W_c|); <= 1 passes."""
    d, r = wl.storage_to_f32(dev, dtype).astype(np.float64), wl.storage_to_f32(ref, dtype).astype(np.float64)
    Kf, Wf = wl.storage_to_f32(K, dtype).astype(np.float64), wl.storage_to_f32(W, dtype).astype(np.float64)
    mant = 7 if dtype == wl.BF16 else 23
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(r), 2.0 ** -126))) - mant)
    bound = ulp + Kf.shape[1] * 2.0 ** -24 * (np.abs(Kf) @ np.abs(Wf))
    return float((np.abs(d - r) / bound).max()) if d.size else 0.0


def ulp_distance(a: np.ndarray, b: np.ndarray, dtype: int) -> int:
    """Largest distance, in representable values of the storage type, between two arrays."""
    if dtype == wl.BF16:
        ia, ib = a.astype(np.int64), b.astype(np.int64)
        sign = 0x8000
    else:
        ia, ib = a.view(np.uint32).astype(np.int64), b.view(np.uint32).astype(np.int64)
        sign = 0x80000000
    ia = np.where(ia & sign, -(ia & (sign - 1)), ia)          # sign-magnitude -> monotone integers
    ib = np.where(ib & sign, -(ib & (sign - 1)), ib)
    return int(np.abs(ia - ib).max()) if ia.size else 0


def check_selection(gpu_idx: np.ndarray, orc_idx: np.ndarray, scores: np.ndarray, what=""):
    """Index sets must be identical; a swap (i only on the GPU, j only in the oracle) is accepted iff
    the two oracle scores agree to 1e-5 relative.  Returns the number of accepted swaps."""
    assert np.all(np.diff(gpu_idx) > 0), "%s: GPU list not strictly ascending" % what
    assert len(gpu_idx) == len(orc_idx), "%s: count %d vs oracle %d" % (what, len(gpu_idx), len(orc_idx))
    g, o = set(gpu_idx.tolist()), set(orc_idx.tolist())
    if g == o:
        return 0
    only_g = sorted(g - o, key=lambda i: scores[i])
    only_o = sorted(o - g, key=lambda i: scores[i])
    assert len(only_g) == len(only_o)
    for i, j in zip(only_g, only_o):
        si, sj = scores[i], scores[j]
        assert abs(si - sj) <= 1e-5 * max(abs(si), abs(sj)), "%s: tokens %d/%d scores %r/%r are not a near-tie" % (what, i, j, si, sj)
    return len(only_g)


def gpu_select(case: Case, q_imp_all: np.ndarray, p, layer_begin=0, layer_count=None):
    """q_imp_all [layer_count][B][Hl * gl][d'] -> lists [layer_count][B][Hl] of numpy arrays."""
    w = case.w
    lc = w.n_layers - layer_begin if layer_count is None else layer_count
    cap = case.ctx.index_capacity
    idx = torch.full((lc, w.batch, case.Hl, cap), -1, dtype=torch.int32, device="cuda")
    cnt = torch.full((lc, w.batch, case.Hl), -1, dtype=torch.int32, device="cuda")
    case.ctx.select_topk(layer_begin, lc, None, w.batch, torch.from_numpy(np.ascontiguousarray(q_imp_all, np.float32)).cuda(),
                         p, idx, cnt)
    torch.cuda.synchronize()
    idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
    return [[[idx[l, b, h, :cnt[l, b, h]].copy() for h in range(case.Hl)] for b in range(w.batch)] for l in range(lc)]


def gpu_attention(case: Case, q_all: np.ndarray, p, idx=None, cnt=None, layer_begin=0, layer_count=None, want_lse=True):
    """q_all [layer_count][B][Hq][D] storage -> out [layer_count][B][Hq][D] fp32 (and lse)."""
    w = case.w
    lc = w.n_layers - layer_begin if layer_count is None else layer_count
    out = torch.full((lc, w.batch, w.n_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((lc, w.batch, w.n_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    case.ctx.sparse_decode_attention(layer_begin, lc, None, w.batch, to_dev(q_all, w.dtype), p, out, idx=idx, cnt=cnt,
                                     lse=lse if want_lse else None)
    torch.cuda.synchronize()
    return out.cpu().numpy(), lse.cpu().numpy()


def queries(w: wl.Workload, step=0, layers=None):
    """q [L][B][Hq][D] storage and q_imp [L][B][Hq][d'] fp32 for one decode step."""
    layers = range(w.n_layers) if layers is None else layers
    qs, qis = [], []
    for l in layers:
        pairs = [wl.gen_queries(w, l, b, step) for b in range(w.batch)]
        qs.append(np.stack([p[0] for p in pairs]))
        qis.append(np.stack([p[1] for p in pairs]))
    return np.stack(qs), np.stack(qis)
