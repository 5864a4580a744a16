"""The C-ABI library builds for sm_100a, loads without a GPU, and exports every entry point the
public header declares (no compute calls here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libpath():
    from paper_2503_07518_b200 import build
    return build.build()


def declared_functions():
    src = open(os.path.join(ROOT, "include", "tokenbutler.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(tb_[a-z_]+)\s*\(", src)))


def test_header_declares_the_path_entry_points():
    names = declared_functions()
    for must in ("tb_append_kv", "tb_project_keys", "tb_score_tokens", "tb_select_topk", "tb_sparse_decode_attention"):
        assert must in names


def test_library_exports_every_declared_symbol(libpath):
    lib = ctypes.CDLL(libpath)
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_names(libpath):
    from paper_2503_07518_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()


def test_host_validation_needs_no_gpu(libpath):
    from paper_2503_07518_b200 import binding as b
    L = b.lib()
    cfg = b.tb_config(2, 8, 8, 128, 32, b.TB_BF16, 1, 1024, 64, 1, 0, 0)
    sizes = [ctypes.c_size_t() for _ in range(4)]
    assert L.tb_query_sizes(ctypes.byref(cfg), *[ctypes.byref(s) for s in sizes]) == b.TB_OK
    assert sizes[0].value == 2 * 1 * 8 * 1024 * 2 * 128 * 2            # interleaved K|V rows
    assert sizes[1].value == 2 * 1 * 8 * 1024 * 32 * 2                  # projected keys
    bad = b.tb_config(2, 8, 8, 96, 32, b.TB_BF16, 1, 1024, 64, 1, 0, 0)
    assert L.tb_query_sizes(ctypes.byref(bad), *[ctypes.byref(s) for s in sizes]) == b.TB_ERR_UNSUPPORTED
    bad = b.tb_config(2, 9, 8, 128, 32, b.TB_BF16, 1, 1024, 64, 1, 0, 0)
    assert L.tb_query_sizes(ctypes.byref(bad), *[ctypes.byref(s) for s in sizes]) == b.TB_ERR_INVALID_ARG
    assert L.tb_status_string(b.TB_ERR_UNPROJECTED) == b"candidate keys not projected"


def test_predictor_host_validation_needs_no_gpu(libpath):
    from paper_2503_07518_b200 import binding as b
    L = b.lib()
    one = ctypes.c_void_p(16)                           # any aligned non-null address: never dereferenced on these paths
    ok = dict(dtype=b.TB_BF16, model_dim=4096, hidden_dim=512, n_q_heads=32, n_slots=4, imp_dim=32, activation=b.TB_ACT_GELU,
              ln_eps=1e-5, ln_weight=16, ln_bias=16, w1=16, w2=16)

    def call(n_tokens=1, hidden=one, **over):
        p = b.tb_predictor(**{**ok, **over})
        return L.tb_predict_importance_queries(ctypes.byref(p), hidden, n_tokens, one, one, None)

    assert call(w1=None) == b.TB_ERR_INVALID_ARG
    assert call(hidden=None) == b.TB_ERR_INVALID_ARG
    assert call(n_tokens=0) == b.TB_ERR_INVALID_ARG
    assert call(activation=7) == b.TB_ERR_INVALID_ARG
    assert call(ln_weight=24) == b.TB_ERR_INVALID_ARG      # not 16-byte aligned
    assert call(model_dim=4100) == b.TB_ERR_UNSUPPORTED    # rows are read 16 bytes at a time
    assert call(n_tokens=65) == b.TB_ERR_CAPACITY
