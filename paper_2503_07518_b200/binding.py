"""ctypes binding of libtokenbutler.so: the same entry points as include/tokenbutler.h, argument
marshalling only.  torch supplies device memory and streams; every step of the path runs in the
library's CUDA kernels.  There is no CPU fallback: if the library is missing, loading raises."""
from __future__ import annotations

import ctypes as C
import os

import torch

TB_OK = 0
TB_ERR_INVALID_ARG, TB_ERR_UNSUPPORTED, TB_ERR_CAPACITY, TB_ERR_UNPROJECTED = -1, -2, -3, -4
TB_ERR_STATE, TB_ERR_CUDA, TB_ERR_TIMEOUT, TB_ERR_BAD_INDEX = -5, -6, -7, -8
TB_F32, TB_BF16 = 0, 1
TB_GROUP_SUM, TB_GROUP_MAX, TB_PER_QHEAD = 0, 1, 2
TB_SCOPE_KV_HEAD, TB_SCOPE_Q_HEAD, TB_SCOPE_LAYER = 0, 1, 2
TB_NEIGHBOR_DILATE, TB_NEIGHBOR_CLUSTER = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtokenbutler.so")

EXPORTS = ["tb_query_sizes", "tb_create", "tb_destroy", "tb_index_capacity", "tb_set_projection", "tb_reset_sequence",
           "tb_get_length", "tb_append_kv", "tb_project_keys", "tb_score_tokens", "tb_select_topk",
           "tb_sparse_decode_attention", "tb_sparse_decode_attention_static", "tb_static_get_status", "tb_predict_importance_queries", "tb_get_status", "tb_set_wait_diagnostics", "tb_use_device_lengths", "tb_sync_lengths", "tb_resident_rows_bytes", "tb_bind_resident_rows", "tb_important_buffer_bytes", "tb_bind_important_buffer", "tb_last_step_bytes", "tb_launch_count", "tb_status_string"]


class tb_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "n_q_heads", "n_kv_heads", "head_dim", "imp_dim", "kv_dtype",
                                         "max_batch", "max_seq_len", "max_budget", "max_radius", "device",
                                         "list_scope")]


class tb_select_params(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("budget", "sinks", "recent", "radius", "nmode", "interval", "step", "reduce")] + \
               [("score_scale", C.c_float)]


class tb_predictor(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("dtype", "model_dim", "hidden_dim", "n_q_heads", "n_slots", "imp_dim", "activation")] + \
               [("ln_eps", C.c_float)] + [(n, C.c_void_p) for n in ("ln_weight", "ln_bias", "w1", "w2")]


TB_ACT_GELU, TB_ACT_SILU, TB_ACT_RELU = 0, 1, 2


class TBError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__("%s: %s (%d)" % (what, lib().tb_status_string(status).decode(), status))


_lib = None


def lib():
    """Load the CUDA library (built in-tree by paper_2503_07518_b200.build); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libtokenbutler.so has not been built: run `python -m paper_2503_07518_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        L.tb_status_string.restype = C.c_char_p
        L.tb_last_step_bytes.restype = C.c_uint64
        L.tb_launch_count.restype = C.c_uint64
        L.tb_index_capacity.restype = C.c_int32
        vp, i32, ip = C.c_void_p, C.c_int32, C.POINTER(C.c_int32)
        L.tb_query_sizes.argtypes = [C.POINTER(tb_config)] + [C.POINTER(C.c_size_t)] * 4
        L.tb_create.argtypes = [C.POINTER(tb_config), vp, vp, vp, vp, C.POINTER(vp)]
        L.tb_destroy.argtypes = [vp]
        L.tb_index_capacity.argtypes = [vp]
        L.tb_set_projection.argtypes = [vp, i32, vp, vp]
        L.tb_reset_sequence.argtypes = [vp, i32]
        L.tb_get_length.argtypes = [vp, i32, i32, ip, ip]
        L.tb_append_kv.argtypes = [vp, i32, i32, ip, ip, i32, vp, vp, vp]
        L.tb_project_keys.argtypes = [vp, i32, i32, ip, ip, ip, i32, vp]
        L.tb_score_tokens.argtypes = [vp, i32, ip, i32, vp, i32, C.c_float, vp, vp]
        L.tb_select_topk.argtypes = [vp, i32, i32, ip, i32, vp, C.POINTER(tb_select_params), vp, vp, vp]
        L.tb_sparse_decode_attention.argtypes = [vp, i32, i32, ip, i32, vp, C.POINTER(tb_select_params), vp, vp, C.c_float,
                                                 vp, vp, vp]
        L.tb_sparse_decode_attention_static.argtypes = [vp, i32, i32, i32, i32, i32, ip, ip, i32, vp, vp, vp, i32, i32, i32,
                                                        C.c_float, vp, vp, vp]
        L.tb_static_get_status.argtypes = [vp, ip]
        L.tb_predict_importance_queries.argtypes = [vp, vp, i32, vp, vp, vp]
        L.tb_get_status.argtypes = [vp, vp, ip]
        L.tb_set_wait_diagnostics.argtypes = [vp, i32, i32]
        L.tb_use_device_lengths.argtypes = [vp, i32, i32]
        L.tb_sync_lengths.argtypes = [vp, vp]
        L.tb_resident_rows_bytes.restype = C.c_size_t
        L.tb_resident_rows_bytes.argtypes = [C.POINTER(tb_config), i32, i32]
        L.tb_bind_resident_rows.argtypes = [vp, vp, C.c_size_t, i32, i32]
        L.tb_important_buffer_bytes.restype = C.c_size_t
        L.tb_important_buffer_bytes.argtypes = [C.POINTER(tb_config)]
        L.tb_bind_important_buffer.argtypes = [vp, vp, C.c_size_t]
        L.tb_last_step_bytes.argtypes = [vp]
        L.tb_launch_count.argtypes = [vp]
        L.tb_status_string.argtypes = [i32]
        _lib = L
    return _lib


def _ints(x):
    if x is None:
        return None
    return (C.c_int32 * len(x))(*[int(v) for v in x])


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def select_params(budget, sinks=0, recent=0, radius=0, nmode=TB_NEIGHBOR_DILATE, interval=1, step=0,
                  reduce=TB_GROUP_SUM, score_scale=1.0):
    return tb_select_params(budget, sinks, recent, radius, nmode, interval, step, reduce, score_scale)


def torch_dtype(kv_dtype):
    return torch.bfloat16 if kv_dtype == TB_BF16 else torch.float32


TB_STATIC_MAX_QHEADS = 64


def sparse_decode_attention_static(kv, kv_dtype, n_q_heads, n_kv_heads, head_dim, max_seq_len, seq_slots, seq_lens, q, out,
                                   idx=None, cnt=None, idx_stride=0, sinks=0, recent=0, sm_scale=0.0, lse=None, stream=None):
    """Attention without a context or workspace, for callers that cannot allocate device memory
    (fixed memory pools, threads where cudaMalloc is forbidden): scratch lives inside the library.
    Only marshals arguments for tb_sparse_decode_attention_static; returns its status code."""
    return lib().tb_sparse_decode_attention_static(_ptr(kv), kv_dtype, n_q_heads, n_kv_heads, head_dim, max_seq_len,
                                                   _ints(seq_slots), _ints(seq_lens), len(seq_lens), _ptr(q), _ptr(idx),
                                                   _ptr(cnt), idx_stride, sinks, recent, sm_scale, _ptr(out), _ptr(lse),
                                                   _stream(stream))


def static_get_status(stream=None):
    """Status word of the allocation-free entry point on the current device (read and cleared)."""
    v = C.c_int32()
    st = lib().tb_static_get_status(_stream(stream), C.byref(v))
    if st != TB_OK:
        raise TBError(st, "tb_static_get_status")
    return v.value


def predict_importance_queries(hidden, ln_weight, ln_bias, w1, w2, dtype, n_q_heads, n_slots, imp_dim, scratch, q_imp,
                               ln_eps=1e-5, activation=TB_ACT_GELU, stream=None):
    """Predictor forward q = W2 act(W1 LN(h)) for the rows of `hidden` [tokens, model_dim]; writes q_imp
    [n_slots, tokens, n_q_heads, imp_dim].  Only marshals arguments for tb_predict_importance_queries;
    returns its status code."""
    p = tb_predictor(dtype, hidden.shape[1], w1.shape[0], n_q_heads, n_slots, imp_dim, activation, ln_eps,
                     ln_weight.data_ptr(), ln_bias.data_ptr(), w1.data_ptr(), w2.data_ptr())
    return lib().tb_predict_importance_queries(C.byref(p), _ptr(hidden), hidden.shape[0], _ptr(scratch), _ptr(q_imp), _stream(stream))


class Context:
    """Owns the four device regions (torch tensors) and the tb_ctx bound to them.  Methods carry the
    names of the C entry points and only marshal arguments."""

    def __init__(self, n_layers, n_q_heads, n_kv_heads, head_dim, imp_dim, kv_dtype, max_batch, max_seq_len,
                 max_budget, max_radius=0, device=0, kv_on_host=False, list_scope=TB_SCOPE_KV_HEAD):
        L = lib()
        self.cfg = tb_config(n_layers, n_q_heads, n_kv_heads, head_dim, imp_dim, kv_dtype, max_batch, max_seq_len,
                             max_budget, max_radius, device, list_scope)
        # heads of the projected-key cache / lists per (layer, sequence) under the selection scope
        self.n_key_heads = 1 if list_scope == TB_SCOPE_LAYER else n_kv_heads
        self.n_lists = {TB_SCOPE_KV_HEAD: n_kv_heads, TB_SCOPE_Q_HEAD: n_q_heads, TB_SCOPE_LAYER: 1}.get(list_scope, n_kv_heads)
        sizes = [C.c_size_t() for _ in range(4)]
        st = L.tb_query_sizes(C.byref(self.cfg), *[C.byref(s) for s in sizes])
        if st != TB_OK:
            raise TBError(st, "tb_query_sizes")
        self.sizes = [s.value for s in sizes]
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        dt = torch_dtype(kv_dtype)
        es = 2 if kv_dtype == TB_BF16 else 4
        # caller-owned regions; kv / kimp exposed as typed views in the documented layouts
        # (kv_on_host: the cache in page-locked host memory, addressed by the device through the same pointer)
        kv_flat = torch.empty(self.sizes[0] // es, dtype=dt, pin_memory=True) if kv_on_host else \
            torch.empty(self.sizes[0] // es, dtype=dt, device=self.device)
        self.kv = kv_flat.view(n_layers, max_batch, n_kv_heads, max_seq_len, 2, head_dim)
        self.kimp = torch.empty(self.sizes[1] // es, dtype=dt, device=self.device).view(
            n_layers, max_batch, self.n_key_heads, max_seq_len, imp_dim)
        self.state = torch.empty(self.sizes[2], dtype=torch.uint8, device=self.device)
        self.workspace = torch.empty(self.sizes[3], dtype=torch.uint8, device=self.device)
        h = C.c_void_p()
        st = L.tb_create(C.byref(self.cfg), _ptr(self.kv), _ptr(self.kimp), _ptr(self.state), _ptr(self.workspace), C.byref(h))
        if st != TB_OK:
            raise TBError(st, "tb_create")
        self.h = h
        self.index_capacity = L.tb_index_capacity(h)

    def close(self):
        if getattr(self, "h", None):
            lib().tb_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @staticmethod
    def _chk(st, what):
        if st != TB_OK:
            raise TBError(st, what)

    def set_projection(self, layer, W, stream=None):
        self._chk(lib().tb_set_projection(self.h, layer, _ptr(W), _stream(stream)), "tb_set_projection")

    def reset_sequence(self, seq):
        self._chk(lib().tb_reset_sequence(self.h, seq), "tb_reset_sequence")

    def get_length(self, layer, seq):
        a, b = C.c_int32(), C.c_int32()
        self._chk(lib().tb_get_length(self.h, layer, seq, C.byref(a), C.byref(b)), "tb_get_length")
        return a.value, b.value

    def append_kv(self, layer_begin, layer_count, seq_ids, n_new, k, v, stream=None):
        self._chk(lib().tb_append_kv(self.h, layer_begin, layer_count, _ints(seq_ids), _ints(n_new), len(n_new), _ptr(k),
                                     _ptr(v), _stream(stream)), "tb_append_kv")

    def project_keys(self, layer_begin, layer_count, seq_ids, pos_begin, pos_end, stream=None, n_seq=None):
        """pos_begin = pos_end = None: every listed sequence's unprojected tokens (n_seq says how many sequences)."""
        n = len(pos_begin) if pos_begin is not None else n_seq
        self._chk(lib().tb_project_keys(self.h, layer_begin, layer_count, _ints(seq_ids), _ints(pos_begin), _ints(pos_end),
                                        n, _stream(stream)), "tb_project_keys")

    def bind_resident_rows(self, sinks, window):
        """Allocates (torch) and binds device copies of the first `sinks` and the `window` most recent tokens' rows."""
        n = lib().tb_resident_rows_bytes(C.byref(self.cfg), sinks, window)
        self.resident_rows = torch.empty(max(n, 256), dtype=torch.uint8, device=self.device)
        self._chk(lib().tb_bind_resident_rows(self.h, _ptr(self.resident_rows), n, sinks, window), "tb_bind_resident_rows")

    def bind_important_buffer(self):
        """Allocates (torch) and binds the contiguous Important buffer."""
        n = lib().tb_important_buffer_bytes(C.byref(self.cfg))
        self.important_buffer = torch.empty(max(n, 256), dtype=torch.uint8, device=self.device)
        self._chk(lib().tb_bind_important_buffer(self.h, _ptr(self.important_buffer), n), "tb_bind_important_buffer")

    def use_device_lengths(self, on=True, growth_reserve=0):
        self._chk(lib().tb_use_device_lengths(self.h, int(on), growth_reserve), "tb_use_device_lengths")

    def sync_lengths(self, stream=None):
        self._chk(lib().tb_sync_lengths(self.h, _stream(stream)), "tb_sync_lengths")

    def score_tokens(self, layer, seq_ids, n_seq, q_imp, scores, reduce=TB_GROUP_SUM, scale=1.0, stream=None):
        self._chk(lib().tb_score_tokens(self.h, layer, _ints(seq_ids), n_seq, _ptr(q_imp), reduce, scale, _ptr(scores),
                                        _stream(stream)), "tb_score_tokens")

    def select_topk(self, layer_begin, layer_count, seq_ids, n_seq, q_imp, params, idx_out=None, cnt_out=None, stream=None):
        self._chk(lib().tb_select_topk(self.h, layer_begin, layer_count, _ints(seq_ids), n_seq, _ptr(q_imp), C.byref(params),
                                       _ptr(idx_out), _ptr(cnt_out), _stream(stream)), "tb_select_topk")

    def sparse_decode_attention(self, layer_begin, layer_count, seq_ids, n_seq, q, params, out, idx=None, cnt=None,
                                sm_scale=0.0, lse=None, stream=None):
        self._chk(lib().tb_sparse_decode_attention(self.h, layer_begin, layer_count, _ints(seq_ids), n_seq, _ptr(q),
                                                   C.byref(params), _ptr(idx), _ptr(cnt), sm_scale, _ptr(out), _ptr(lse),
                                                   _stream(stream)), "tb_sparse_decode_attention")

    def get_status(self, stream=None):
        v = C.c_int32()
        self._chk(lib().tb_get_status(self.h, _stream(stream), C.byref(v)), "tb_get_status")
        return v.value

    def set_wait_diagnostics(self, poll_limit=0, drop_tile=-1):
        self._chk(lib().tb_set_wait_diagnostics(self.h, poll_limit, drop_tile), "tb_set_wait_diagnostics")

    def last_step_bytes(self):
        return lib().tb_last_step_bytes(self.h)

    def launch_count(self):
        return lib().tb_launch_count(self.h)
