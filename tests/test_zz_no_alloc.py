"""The allocation-free attention entry point (tb_sparse_decode_attention_static) must give what the
context-based entry point gives.  It serves callers that cannot allocate device memory at call time
(fixed memory pools, threads on which cudaMalloc is forbidden): its split-K scratch is a fixed array
inside the library, shared by every call, so this file calls it twice in a row with different inputs
to show that nothing stale leaks from one call into the next.  Collected last on purpose."""
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


@pytest.mark.parametrize("cfg", [2, 1])
def test_static_entry_matches_context_entry_twice(H, cfg):
    from paper_2503_07518_b200 import binding as tb
    if cfg == 2:       # bf16, GQA 4: the tensor-core kernel
        w = wl.workload(2, n_layers=2, batch=2, lengths=[5000, 2100], budget=400, sinks=4, recent=32)
    else:              # fp32, one query head per KV head
        w = wl.workload(1, n_layers=2, batch=2, lengths=[3000, 700], budget=200, sinks=4, recent=64)
    case = H.Case(w, project="oracle-only")
    p = tb.select_params(w.budget, w.sinks, w.recent)
    cap = case.ctx.index_capacity
    tol = H.ATTN_TOL[w.dtype]
    for call in range(2):                                   # two calls in a row, different queries and layer
        layer = call
        q, qi = H.queries(w, step=call)
        idx = torch.zeros(1, w.batch, w.n_kv_heads, cap, dtype=torch.int32, device="cuda")
        cnt = torch.zeros(1, w.batch, w.n_kv_heads, dtype=torch.int32, device="cuda")
        case.ctx.select_topk(layer, 1, None, w.batch, torch.from_numpy(qi[layer:layer + 1]).cuda(), p, idx, cnt)
        q_dev = H.to_dev(q[layer], w.dtype)
        ref = torch.full((w.batch, w.n_q_heads, w.head_dim), float("nan"), device="cuda")
        ref_lse = torch.full((w.batch, w.n_q_heads), float("nan"), device="cuda")
        case.ctx.sparse_decode_attention(layer, 1, None, w.batch, q_dev, p, ref, idx=idx, cnt=cnt, lse=ref_lse)
        out = torch.full_like(ref, float("nan"))
        lse = torch.full_like(ref_lse, float("nan"))
        st = tb.sparse_decode_attention_static(case.ctx.kv[layer], w.dtype, w.n_q_heads, w.n_kv_heads, w.head_dim, case.cap,
                                               None, case.cur, q_dev, out, idx=idx, cnt=cnt, idx_stride=cap, sinks=w.sinks,
                                               recent=w.recent, lse=lse)
        assert st == tb.TB_OK
        torch.cuda.synchronize()
        assert torch.isfinite(out).all()
        assert (out - ref).abs().max().item() <= tol
        assert (lse - ref_lse).abs().max().item() <= tol
        # dense rule through the same entry point
        dense_ref = torch.empty_like(ref)
        case.ctx.sparse_decode_attention(layer, 1, None, w.batch, q_dev, tb.select_params(-1), dense_ref)
        st = tb.sparse_decode_attention_static(case.ctx.kv[layer], w.dtype, w.n_q_heads, w.n_kv_heads, w.head_dim, case.cap,
                                               None, case.cur, q_dev, out)
        assert st == tb.TB_OK
        torch.cuda.synchronize()
        assert (out - dense_ref).abs().max().item() <= tol
        # the sparse result against the oracle on the caller's lists, every sequence and KV head; one dense unit
        sparse = torch.full_like(ref, float("nan"))
        st = tb.sparse_decode_attention_static(case.ctx.kv[layer], w.dtype, w.n_q_heads, w.n_kv_heads, w.head_dim, case.cap,
                                               None, case.cur, q_dev, sparse, idx=idx, cnt=cnt, idx_stride=cap, sinks=w.sinks,
                                               recent=w.recent)
        assert st == tb.TB_OK
        torch.cuda.synchronize()
        sp, o = sparse.cpu().numpy(), out.cpu().numpy()
        got_idx, got_cnt = idx.cpu().numpy(), cnt.cpu().numpy()
        for b in range(w.batch):
            for h in range(w.n_kv_heads):
                refo, _ = case.oracle_attention(layer, b, h, q[layer, b], got_idx[0, b, h, :got_cnt[0, b, h]], p)
                assert np.abs(sp[b, h * w.group:(h + 1) * w.group] - refo).max() <= tol
        refo, _ = case.oracle_attention(layer, 1, 0, q[layer, 1], None, p, dense=True)
        assert np.abs(o[1, :w.group] - refo).max() <= tol
        assert tb.static_get_status() == 0
    assert case.ctx.get_status() == 0


def test_static_entry_reports_an_out_of_range_list_entry(H):
    """A caller list entry equal to the sequence length is skipped (no access outside the cache) and
    shows up once in the entry point's own status word; the rest of the list is attended as usual."""
    from paper_2503_07518_b200 import binding as tb
    w = wl.workload(2, n_layers=1, n_q_heads=8, n_kv_heads=2, lengths=[600], budget=32)
    case = H.Case(w, project="oracle-only")
    q, _ = H.queries(w)
    r = np.random.Generator(np.random.PCG64(6))
    mine = [np.sort(r.choice(np.arange(5, 590), 20, replace=False)).astype(np.int32) for _ in range(2)]
    idx = np.zeros((1, 2, 24), np.int32)
    for h in range(2):
        idx[0, h, :20] = mine[h]
    idx[0, 1, 7] = 600                                                    # one past the end
    cnt = np.full((1, 2), 20, np.int32)
    q_dev = H.to_dev(q[0], w.dtype)
    out = torch.full((1, w.n_q_heads, w.head_dim), float("nan"), device="cuda")
    assert tb.static_get_status() == 0
    st = tb.sparse_decode_attention_static(case.ctx.kv[0], w.dtype, w.n_q_heads, w.n_kv_heads, w.head_dim, case.cap, None,
                                           case.cur, q_dev, out, idx=torch.from_numpy(idx).cuda(), cnt=torch.from_numpy(cnt).cuda(),
                                           idx_stride=24, sinks=5, recent=10)
    assert st == tb.TB_OK
    assert tb.static_get_status() == tb.TB_ERR_BAD_INDEX
    assert tb.static_get_status() == 0                                    # reading clears it
    p = tb.select_params(32, 5, 10)
    o = out.cpu().numpy()
    for h, lst in enumerate([mine[0], np.delete(mine[1], 7)]):
        refo, _ = case.oracle_attention(0, 0, h, q[0, 0], lst, p)
        assert np.abs(o[0, h * 4:(h + 1) * 4] - refo).max() <= 2e-3


def test_static_entry_rejects_what_its_scratch_cannot_hold(H):
    from paper_2503_07518_b200 import binding as tb
    kv = torch.zeros(3 * 8 * 64 * 2 * 128, dtype=torch.bfloat16, device="cuda")
    q = torch.zeros(3 * 32 * 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(3 * 32 * 128, device="cuda")
    # 3 sequences x 32 query heads = 96 > TB_STATIC_MAX_QHEADS
    st = tb.sparse_decode_attention_static(kv, tb.TB_BF16, 32, 8, 128, 64, None, [64, 64, 64], q, out)
    assert st == tb.TB_ERR_CAPACITY
    assert tb.lib().tb_status_string(st) == b"capacity exceeded"
    st = tb.sparse_decode_attention_static(kv, tb.TB_BF16, 32, 8, 128, 64, None, [64, 65], q, out)   # longer than the cache
    assert st == tb.TB_ERR_INVALID_ARG
    st = tb.sparse_decode_attention_static(kv, tb.TB_BF16, 32, 8, 96, 64, None, [64], q, out)
    assert st == tb.TB_ERR_UNSUPPORTED
    # a cache the device cannot address (pageable host memory) is refused, not handed to a kernel
    st = tb.sparse_decode_attention_static(torch.zeros(8 * 64 * 2 * 128, dtype=torch.bfloat16), tb.TB_BF16, 32, 8, 128, 64,
                                           None, [64], q, out)
    assert st == tb.TB_ERR_INVALID_ARG
