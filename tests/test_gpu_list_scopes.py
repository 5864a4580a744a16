"""GPU parity for the selection scopes other than one list per KV head (paper Sec. 3.1: importance is
predicted per head; App. "additional evaluation": a head-less predictor, one importance per token and
layer): one list per query head, one list per layer.  The oracle needs no new arithmetic for them: a
per-query-head unit is a group of one whose keys are its KV head's, and a per-layer unit scores the
[Hkv*D] x d' projection of the concatenated key and hands its one list to every head."""
import ctypes

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2503_07518_b200 import workloads as wl  # noqa: E402
from test_gpu_parity import H, full_pipeline_check, tb  # noqa: E402,F401


CASES = [
    # cluster kernel (few problems), bf16 tensor-core attention with a group of one / of four
    (2, dict(n_layers=2, batch=2, lengths=[5000, 777], budget=200, sinks=3, recent=9)),
    # fp32 storage, d' = 16, g = 2
    (1, dict(n_layers=1, n_q_heads=8, n_kv_heads=4, imp_dim=16, batch=3, lengths=[1500, 260, 2049], budget=100, sinks=1, recent=4)),
]


@pytest.mark.parametrize("scope", [1, 2])
@pytest.mark.parametrize("ci", range(len(CASES)))
def test_scope_pipeline_matches_oracle(H, scope, ci):
    """Projection (per-layer scope: summed over the KV heads), selection and attention from the stored
    lists, dense attention too, with and without neighbours and across an append + reuse step."""
    b_ = tb()
    cfg, over = CASES[ci]
    w = wl.workload(cfg, **over)
    case = H.Case(w, max_radius=2, extra_len=4, list_scope=scope)          # Case checks the projection
    assert case.Hl == (w.n_q_heads if scope == 1 else 1) and case.Hi == (w.n_kv_heads if scope == 1 else 1)
    p = b_.select_params(w.budget, w.sinks, w.recent)
    full_pipeline_check(H, case, p, dense_too=True)
    pn = b_.select_params(w.budget, w.sinks, w.recent, radius=2, nmode=b_.TB_NEIGHBOR_DILATE)
    full_pipeline_check(H, case, b_.select_params(w.budget, w.sinks, w.recent, radius=1, nmode=b_.TB_NEIGHBOR_CLUSTER), step=3)
    full_pipeline_check(H, case, pn, step=1)                               # leaves the DILATE lists stored for the reuse step below
    # a decode step that appends and reuses the stored lists (interval 4, step 1)
    case.append_step(0)
    case.project_range(list(case.proj), list(case.cur))
    q, qi = H.queries(w, 2)
    stored = H.gpu_select(case, qi[:, :, :case.Hl * case.gl], b_.select_params(w.budget, w.sinks, w.recent, radius=2, interval=4, step=1))
    out, _ = H.gpu_attention(case, q, pn)
    for l in range(w.n_layers):
        for b in range(w.batch):
            for h in range(case.Ha):
                ref, _ = case.oracle_attention(l, b, h, q[l, b], stored[l][b][h * case.Hl // case.Ha], pn)
                assert np.abs(out[l, b, h * case.ga:(h + 1) * case.ga] - ref).max() <= H.ATTN_TOL[w.dtype]


def test_per_query_head_lists_many_problems(H):
    """One list per query head turns 24 sequences x 32 query heads into 768 problems of one launch:
    the one-block-per-problem selection kernel, then attention with a group of one."""
    b_ = tb()
    w = wl.workload(2, n_layers=1, batch=24, lengths=[1800 + 53 * i for i in range(24)], budget=96)
    case = H.Case(w, list_scope=b_.TB_SCOPE_Q_HEAD)
    full_pipeline_check(H, case, b_.select_params(w.budget, w.sinks, w.recent))


def test_per_query_head_lists_reduce_to_group_lists(H):
    """If the g importance queries of every group are equal, a group's sum is g times each of them, so
    per-query-head lists must equal the per-KV-head list of the same inputs (and so must the outputs)."""
    b_ = tb()
    w = wl.workload(2, n_layers=1, batch=2, lengths=[3000, 901], budget=150, sinks=2, recent=6)
    q, qi = H.queries(w)
    qi = np.repeat(qi[:, :, ::w.group], w.group, axis=2)                   # every head of a group gets the group's first query
    p = b_.select_params(w.budget, w.sinks, w.recent)
    kv_case = H.Case(w)
    kv_lists = H.gpu_select(kv_case, qi, p)
    kv_out, _ = H.gpu_attention(kv_case, q, p)
    q_case = H.Case(w, list_scope=b_.TB_SCOPE_Q_HEAD)
    q_lists = H.gpu_select(q_case, qi, b_.select_params(w.budget, w.sinks, w.recent, reduce=b_.TB_PER_QHEAD))
    q_out, _ = H.gpu_attention(q_case, q, p)
    for b in range(w.batch):
        for hq in range(w.n_q_heads):
            assert np.array_equal(q_lists[0][b][hq], kv_lists[0][b][hq // w.group])
    assert np.abs(q_out - kv_out).max() <= H.ATTN_TOL[w.dtype]


def test_scope_argument_checks(H):
    b_ = tb()
    w = wl.workload(2, n_layers=1, batch=1, lengths=[600], budget=32)
    case = H.Case(w)                                                      # lists per KV head
    _, qi = H.queries(w)
    with pytest.raises(b_.TBError) as e:
        H.gpu_select(case, qi, b_.select_params(w.budget, w.sinks, w.recent, reduce=b_.TB_PER_QHEAD))
    assert e.value.status == b_.TB_ERR_UNSUPPORTED
    cfg = b_.tb_config(1, 8, 8, 128, 32, b_.TB_BF16, 1, 256, 16, 0, 0, 7)  # no such scope
    sizes = [ctypes.c_size_t() for _ in range(4)]
    assert b_.lib().tb_query_sizes(ctypes.byref(cfg), *[ctypes.byref(x) for x in sizes]) == b_.TB_ERR_INVALID_ARG
    # sizes follow the scope: per-layer keeps one projected key per token, per-query-head g times the lists
    def sizes_of(scope):
        c = b_.tb_config(2, 32, 8, 128, 32, b_.TB_BF16, 2, 4096, 256, 0, 0, scope)
        out = [ctypes.c_size_t() for _ in range(4)]
        assert b_.lib().tb_query_sizes(ctypes.byref(c), *[ctypes.byref(x) for x in out]) == b_.TB_OK
        return [x.value for x in out]
    kvh, qh, lay = sizes_of(0), sizes_of(1), sizes_of(2)
    assert kvh[0] == qh[0] == lay[0] and kvh[1] == qh[1] == 8 * lay[1]
    assert qh[2] > kvh[2] > lay[2]
