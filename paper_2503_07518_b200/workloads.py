"""Seeded synthetic inputs for the decode hot path -- shared by the tests, the benchmark and the
CPU oracle's drivers.  This module holds NONE of the method's arithmetic: it only draws random
tensors with the shapes, value distributions and structure of the five benchmark workloads and
converts them to the storage type.

Value recipe: K, V, q, q_imp ~ N(0,1); W_K ~ N(0, 1/D) per (layer, KV head); seeds are a fixed
function of (workload, layer, sequence, tensor tag) so any single unit can be regenerated alone.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass, field

import numpy as np

F32, BF16 = 0, 1
TAG_K, TAG_V, TAG_Q, TAG_QIMP, TAG_W, TAG_AUX, TAG_PRED = 1, 2, 3, 4, 5, 6, 7
BASE_SEED = 250307518


@dataclass
class Workload:
    name: str
    cfg_id: int
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    imp_dim: int
    dtype: int                      # F32 / BF16 storage of K, V, K_imp, q
    lengths: list                   # context length per sequence (before any decode append)
    budget: int
    sinks: int = 0
    recent: int = 0
    radius: int = 0
    nmode: int = 0                  # 0 = DILATE (+-r), 1 = CLUSTER (run-boundary placement)
    interval: int = 1
    decode_steps: int = 1
    outlier_channels: int = 0       # channels per (layer, KV head) whose keys are scaled x8
    planted: int = 0                # planted tokens per (layer, KV head), cosine 0.9 with the importance query
    group: int = field(init=False)

    def __post_init__(self):
        self.group = self.n_q_heads // self.n_kv_heads

    @property
    def max_len(self):
        return max(self.lengths) + self.decode_steps

    def elem_size(self):
        return 2 if self.dtype == BF16 else 4

    def scaled(self, **kw):
        return dataclasses.replace(self, **kw)


def seed_for(cfg_id: int, layer: int, seq: int, tag: int) -> int:
    return BASE_SEED + 1000003 * cfg_id + 1009 * layer + 17 * seq + tag


def _rng(cfg_id, layer, seq, tag):
    return np.random.Generator(np.random.PCG64(seed_for(cfg_id, layer, seq, tag)))


def ragged_lengths(cfg_id: int, batch: int, lo: int, hi: int) -> list:
    """Per-sequence context lengths, uniform in [lo, hi] (the batched-serving workload)."""
    r = _rng(cfg_id, 0, 0, TAG_AUX)
    return [int(x) for x in r.integers(lo, hi + 1, size=batch)]


def workload(cfg: int, **over) -> Workload:
    """The five benchmark workloads (1-based).  Keyword overrides shrink them for tests."""
    if cfg == 1:
        w = Workload("cfg1_fp32_4k", 1, 1, 1, 8, 8, 128, 32, F32, [4096], budget=256, sinks=4, recent=64)
    elif cfg == 2:
        w = Workload("cfg2_llama8b_32k", 2, 32, 1, 32, 8, 128, 32, BF16, [32768], budget=3276, outlier_channels=4)
    elif cfg == 3:
        w = Workload("cfg3_batched_serving", 3, 32, 16, 32, 8, 128, 32, BF16, ragged_lengths(3, 16, 8192, 16384),
                     budget=1024)
    elif cfg == 4:
        w = Workload("cfg4_long_context_128k", 4, 32, 1, 32, 8, 128, 32, BF16, [131072], budget=2048, sinks=16,
                     recent=256, planted=64)
    elif cfg == 5:
        w = Workload("cfg5_interval_neighbors", 5, 32, 8, 32, 8, 128, 32, BF16, [65536] * 8, budget=3276, sinks=0,
                     recent=16, radius=1, nmode=0, interval=16, decode_steps=256)
    else:
        raise ValueError(cfg)
    return w.scaled(**over) if over else w


# ---------------------------------------------------------------------------------------------
# storage conversion (format only)

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even.  Inputs are finite."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + r) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


def to_storage(x: np.ndarray, dtype: int) -> np.ndarray:
    return f32_to_bf16_bits(x) if dtype == BF16 else np.ascontiguousarray(x, dtype=np.float32)


def storage_to_f32(x: np.ndarray, dtype: int) -> np.ndarray:
    return bf16_bits_to_f32(x) if dtype == BF16 else x


# ---------------------------------------------------------------------------------------------
# host generation, one (layer, sequence) at a time

def gen_W(w: Workload, layer: int) -> np.ndarray:
    """Key projection W_K of one layer: [Hkv, D, d'] ~ N(0, 1/D), storage type."""
    r = _rng(w.cfg_id, layer, 0, TAG_W)
    x = r.standard_normal((w.n_kv_heads, w.head_dim, w.imp_dim), dtype=np.float32) * np.float32(1.0 / np.sqrt(w.head_dim))
    return to_storage(x, w.dtype)


def outlier_channels(w: Workload, layer: int) -> np.ndarray:
    """[Hkv, n] distinct channel ids per KV head whose key entries are scaled by 8."""
    r = _rng(w.cfg_id, layer, 0, TAG_AUX)
    return np.stack([r.choice(w.head_dim, size=w.outlier_channels, replace=False) for _ in range(w.n_kv_heads)])


def gen_KV(w: Workload, layer: int, seq: int, n_tokens: int | None = None, start: int = 0):
    """K, V of one (layer, sequence): [Hkv, n, D] each, storage type.  `start` > 0 draws the rows
    appended during decode from an independent stream (tag offset) so prefixes stay reproducible."""
    n = w.lengths[seq] if n_tokens is None else n_tokens
    rk = _rng(w.cfg_id, layer, seq, TAG_K + 100 * start)
    rv = _rng(w.cfg_id, layer, seq, TAG_V + 100 * start)
    K = rk.standard_normal((w.n_kv_heads, n, w.head_dim), dtype=np.float32)
    V = rv.standard_normal((w.n_kv_heads, n, w.head_dim), dtype=np.float32)
    if w.outlier_channels:
        ch = outlier_channels(w, layer)
        for h in range(w.n_kv_heads):
            K[h][:, ch[h]] *= np.float32(8.0)
    return to_storage(K, w.dtype), to_storage(V, w.dtype)


def gen_queries(w: Workload, layer: int, seq: int, step: int = 0):
    """q [Hq, D] (storage type) and importance queries q_imp [Hq, d'] (fp32) of one decode step."""
    rq = _rng(w.cfg_id, layer, seq, TAG_Q + 100 * step)
    ri = _rng(w.cfg_id, layer, seq, TAG_QIMP + 100 * step)
    q = rq.standard_normal((w.n_q_heads, w.head_dim), dtype=np.float32)
    qi = ri.standard_normal((w.n_q_heads, w.imp_dim), dtype=np.float32)
    return to_storage(q, w.dtype), qi


def plant_keys(w: Workload, layer: int, seq: int, K: np.ndarray, W: np.ndarray, q_imp: np.ndarray):
    """Long-context workload: overwrite `planted` rows per KV head with keys whose projection has
    cosine 0.9 with the group's summed importance query and a typical norm.

    k = pinv(W)^T u + (I - W pinv(W)) z,  u = rho (0.9 qhat + sqrt(0.19) nhat),  rho = sqrt(d').
    Built in fp64, rounded to the storage type.  Returns positions [Hkv, planted]."""
    r = _rng(w.cfg_id, layer, seq, TAG_AUX + 100)
    L = K.shape[1]
    lo, hi = w.sinks, L - w.recent
    Wf = storage_to_f32(W, w.dtype).astype(np.float64)
    pos_all = []
    for h in range(w.n_kv_heads):
        Wh = Wf[h]                                              # [D, d']
        qt = q_imp[h * w.group:(h + 1) * w.group].astype(np.float64).sum(0)
        qhat = qt / np.linalg.norm(qt)
        pinv = np.linalg.pinv(Wh)                               # [d', D]
        pos = np.sort(r.choice(np.arange(lo, hi), size=w.planted, replace=False))
        for p in pos:
            n = r.standard_normal(w.imp_dim)
            n -= n.dot(qhat) * qhat
            n /= np.linalg.norm(n)
            u = np.sqrt(w.imp_dim) * (0.9 * qhat + np.sqrt(0.19) * n)
            z = r.standard_normal(w.head_dim)
            k = pinv.T @ u + (z - Wh @ (pinv @ z))
            K[h, p] = to_storage(k.astype(np.float32), w.dtype)
        pos_all.append(pos)
    return np.stack(pos_all)


def gen_predictor(w: Workload, producer: int, model_dim: int = 4096, hidden_dim: int = 512, slots: int = 4, step: int = 0):
    """Inputs of one producer layer's importance-query predictor, in the storage type: hidden states
    [batch, model_dim] (unit-variance channels, a shared offset and 8 channels scaled by 20: residual
    streams have a few massive channels), layer-norm weight ~ 1 and bias ~ 0, W1 [hidden, model_dim]
    ~ N(0, 1/model_dim), W2 [slots * q_heads * imp_dim, hidden] ~ N(0, 4/hidden)."""
    r = _rng(w.cfg_id, producer, 0, TAG_PRED)
    ln_w = 1.0 + 0.1 * r.standard_normal(model_dim)
    ln_b = 0.02 * r.standard_normal(model_dim)
    W1 = r.standard_normal((hidden_dim, model_dim)) * model_dim ** -0.5
    W2 = r.standard_normal((slots * w.n_q_heads * w.imp_dim, hidden_dim)) * 2.0 * hidden_dim ** -0.5
    big = r.choice(model_dim, size=8, replace=False)
    rh = _rng(w.cfg_id, producer, step, TAG_PRED + 8)
    H = rh.standard_normal((w.batch, model_dim)) + 0.25
    H[:, big] *= 20.0
    return tuple(to_storage(np.ascontiguousarray(a, dtype=np.float32), w.dtype) for a in (H, ln_w, ln_b, W1, W2))
