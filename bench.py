#!/usr/bin/env python
"""Benchmark of the TokenButler decode hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--impl ours|reference]

One "step" = one decode step of the whole path over the workload's batch: fused importance scoring +
top-B selection (launched per group of G=4 consumer layers, as the paper batches predictor work per
producer), neighbour expansion where the workload has it, and sparse attention per layer, over all
layers.  Default workload: the Llama-3-8B-shaped decode at 32K context (32 layers, budget 10%).
The printed JSON line carries the device-timed throughput (inputs resident in HBM), the same metric
end to end through the public API with pinned host buffers, the roofline of the dominant kernel
measured live with CUDA events, and the CPU oracle timed on a bounded sample of the same workload.
Run without --config, the line also carries a `workloads` block with the same measurements, in brief, for
the batched-serving, long-context and prediction-interval workloads (configs 3, 4, 5) at their full sizes.
Every timed region is K steps between device events; it is repeated until at least 0.3 s have been timed
and the median repeat is reported (min and max beside it).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2503_07518_b200 import workloads as wl  # noqa: E402

GROUP_LAYERS = 4          # consumer layers served by one producer (paper: G = 4)
METRIC = "decode_tokens_per_s"
UNIT = "tokens/s"

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# captures summarised under profiles/ (None until a capture exists for that workload).
NCU_TRAFFIC_BYTES = {
    ("cfg2_llama8b_32k", "select_kernel"): 67_221_760 + 848_896,   # profiles/select_kernel_cfg2_32k.md
    ("cfg2_llama8b_32k", "attn_kernel"): 13_598_208,               # profiles/attn_mma_kernel_cfg2_32k.md
    ("cfg3_batched_serving", "select_kernel"): 398_907_392 + 5_187_840,   # profiles/select_wave_kernel_cfg3_batched.md
    ("cfg4_long_context_128k", "select_kernel"): 268_011_264 + 3_980_544,  # profiles/select_cw_kernel_cfg4_128k.md
    ("cfg5_interval_neighbors", "attn_kernel"): 309_490_432 + 4_711_680,   # profiles/attn_mma_kernel_cfg5_interval.md
}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# --------------------------------------------------------------------------------------------------
# CPU oracle leg (cpu_baseline and --impl reference)

def oracle_sample(w: wl.Workload, n_layers: int, passes: int, threads: int, max_units: int = 0):
    """Times the oracle, as it stands, on the (sequence, KV head) units of `n_layers` layers of the
    workload (at most `max_units` of them if given), host-generated inputs.  Returns (seconds per pass
    list, units in the sample)."""
    from oracle import tb_oracle as orc
    orc.build()
    units, qis, qs, Ls = [], [], [], []
    cap = (2 * w.radius + 1) * w.budget
    for l in range(n_layers):
        W = wl.gen_W(w, l)
        for b in range(w.batch):
            if max_units and len(units) >= max_units:
                break
            K, V = wl.gen_KV(w, l, b)
            q, qi = wl.gen_queries(w, l, b)
            for h in range(w.n_kv_heads):
                if max_units and len(units) >= max_units:
                    break
                Kh, Vh = np.ascontiguousarray(K[h]), np.ascontiguousarray(V[h])
                units.append(orc.Unit(Kh, Vh, orc.project_keys(Kh, np.ascontiguousarray(W[h]), w.dtype), cap))
                qis.append(qi[h * w.group:(h + 1) * w.group])
                qs.append(q[h * w.group:(h + 1) * w.group])
                Ls.append(w.lengths[b])
    times = []
    for _ in range(passes):
        t0 = time.perf_counter()
        orc.step_units(units, Ls, qis, qs, [1] * len(units), g=w.group, D=w.head_dim, dp=w.imp_dim, dtype=w.dtype,
                       budget=w.budget, sinks=w.sinks, recent=w.recent, radius=w.radius, nmode=w.nmode, n_threads=threads)
        times.append(time.perf_counter() - t0)
    return times, len(units)


def cpu_leg(w: wl.Workload, sample_layers: int, passes: int, max_units: int = 0, threads: int = 0):
    threads = threads or len(os.sched_getaffinity(0))
    times, n_units = oracle_sample(w, sample_layers, passes, threads, max_units)
    total_units = w.n_layers * w.batch * w.n_kv_heads
    step_s = [t * total_units / n_units for t in times]          # units are independent: linear scaling
    return {"times": step_s, "threads": min(threads, n_units),
            "sample": "%d of %d (layer, sequence, KV head) units of %s (layer 0 first), one refresh step each pass, "
                      "scaled linearly to the whole step" % (n_units, total_units, w.name)}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # bounded sample per step so that K steps end within minutes: a layer's 8 heads for short runs,
    # down to a single (layer, sequence, KV head) unit for long ones
    passes = args.steps + args.warmup
    max_units = 8 if passes <= 25 else (2 if passes <= 250 else 1)
    leg = cpu_leg(w, 1, passes, max_units)
    t = leg["times"][args.warmup:]
    ms = 1e3 * float(np.mean(t))
    val = w.batch / (ms * 1e-3)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": {"workload": w.name},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": leg["threads"], "kind": "oracle", "sample": leg["sample"]},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------------
# multi-GPU: the path shards by (sequence, layer, KV head) with no exchange step, so N GPUs run N
# replicas of the workload (weak scaling); the only communication is the barrier and the max-over-ranks
# of the device-measured time.

def max_over_ranks(ms: float, device="cpu") -> float:
    """The slowest rank's time (every rank gets it).  No-op without an initialised process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(batch_per_rank: int, world: int, ms_per_step: float) -> float:
    """Tokens all ranks decode per second: every rank advances `batch_per_rank` sequences per step."""
    return batch_per_rank * world / (ms_per_step * 1e-3)


# --------------------------------------------------------------------------------------------------
# device leg

class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.stop_flag, self.max_mhz = [], set(), False, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def sample(self):
        if not self.nv:
            return
        nv = self.nv
        try:
            self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
            r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
            names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                     "hw_power_brake_slowdown": 0x80}
            for k, bit in names.items():
                if r & bit:
                    self.reasons.add(k)
        except Exception:
            pass

    def run(self):
        while not self.stop_flag:
            self.sample()
            time.sleep(0.01)

    def summary(self):
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def fill_caches(ctx, w, torch, tbh):
    """Seeded synthetic K/V drawn on the device (N(0,1), outlier channels x8 where the workload has
    them), appended and projected through the library's own entry points."""
    dt = tbh.torch_dtype(w.dtype)
    gen = torch.Generator(device="cuda")
    total = sum(w.lengths)
    ev = []
    for l in range(w.n_layers):
        gen.manual_seed(wl.seed_for(w.cfg_id, l, 0, wl.TAG_K))
        Wl = (torch.randn(w.n_kv_heads, w.head_dim, w.imp_dim, generator=gen, device="cuda") / np.sqrt(w.head_dim)).to(dt)
        ctx.set_projection(l, Wl)
        k = torch.randn(total, w.n_kv_heads, w.head_dim, generator=gen, device="cuda")
        if w.outlier_channels:
            ch = wl.outlier_channels(w, l)
            for h in range(w.n_kv_heads):
                k[:, h, torch.from_numpy(ch[h]).cuda()] *= 8.0
        v = torch.randn(total, w.n_kv_heads, w.head_dim, generator=gen, device="cuda")
        ctx.append_kv(l, 1, None, w.lengths, k.to(dt), v.to(dt))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.project_keys(l, 1, None, [0] * w.batch, w.lengths)          # the batched (post-prefill) projection
        e1.record()
        ev.append((e0, e1))
        del k, v
    torch.cuda.synchronize()
    ms = float(np.median([a.elapsed_time(b) for a, b in ev]))
    es = 2 if w.dtype == wl.BF16 else 4
    nbytes = total * w.n_kv_heads * (w.head_dim + w.imp_dim) * es       # K rows read + projected rows written
    return {"us_per_layer": ms * 1e3, "bytes_per_layer": nbytes, "gbs": nbytes / (ms * 1e-3) / 1e9}


def dist_env(torch, dist):
    """(world, rank, local) of this process; the NCCL group (barrier + max-over-ranks only) is set up once."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1 and not dist.is_initialized():
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    return world, rank, local


def storage_name(w):
    return "bf16" if w.dtype == wl.BF16 else "f32"


def measure_static(args, w, brief=False):
    """Workloads whose lengths do not change (configs 1-4): the step is captured once in a CUDA graph and
    replayed.  Returns the JSON line as a dict (without the CPU baseline).  `brief`: the step, its two
    kernels and the end-to-end figure only (the entries of the default run's `workloads` block)."""
    import torch
    import torch.distributed as dist
    from paper_2503_07518_b200 import binding as tbh
    from paper_2503_07518_b200 import build
    build.build()
    world, rank, local = dist_env(torch, dist)

    p = tbh.select_params(w.budget, w.sinks, w.recent, w.radius, w.nmode)
    scope = {"kv_head": tbh.TB_SCOPE_KV_HEAD, "q_head": tbh.TB_SCOPE_Q_HEAD, "layer": tbh.TB_SCOPE_LAYER}[args.list_scope]
    ctx = tbh.Context(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.imp_dim, w.dtype, w.batch, max(w.lengths) + 8,
                      w.budget, w.radius, device=local, kv_on_host=args.offload_kv, list_scope=scope)
    if args.resident_rows:                                   # device copies of the sink and window rows (offloaded KV)
        ctx.bind_resident_rows(max(w.sinks, 1), max(w.recent, 1))
    if args.important_buffer:
        ctx.bind_important_buffer()
    proj_info = fill_caches(ctx, w, torch, tbh)
    dt = tbh.torch_dtype(w.dtype)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(wl.seed_for(w.cfg_id, 0, 0, wl.TAG_Q))
    q = torch.randn(w.n_layers, w.batch, w.n_q_heads, w.head_dim, generator=gen, device="cuda").to(dt)
    qi = torch.randn(w.n_layers, w.batch, w.n_q_heads, w.imp_dim, generator=gen, device="cuda")
    if scope == tbh.TB_SCOPE_LAYER:                          # the head-less predictor: one importance query per layer
        qi = qi[:, :, :1].contiguous()
    out = torch.empty(w.n_layers, w.batch, w.n_q_heads, w.head_dim, device="cuda")
    # end-to-end leg: two sets of device buffers, so that a step's inputs arrive while the step before it computes
    bufs = [(q, qi, out), (q.clone(), qi.clone(), torch.empty_like(out))]
    q_host, qi_host = q.cpu().pin_memory(), qi.cpu().pin_memory()
    out_host = torch.empty_like(out, device="cpu").pin_memory()

    groups = [(l, min(GROUP_LAYERS, w.n_layers - l)) for l in range(0, w.n_layers, GROUP_LAYERS)]
    sel_bytes, att_bytes = [], []

    def step_launches(record=False, b=0):
        # model-faithful schedule: at each producer the selections of its consumer layers, then
        # attention layer by layer
        q_, qi_, out_ = bufs[b]
        for (l0, n) in groups:
            ctx.select_topk(l0, n, None, w.batch, qi_[l0:l0 + n], p)
            if record:
                sel_bytes.append(ctx.last_step_bytes())
            for l in range(l0, l0 + n):
                ctx.sparse_decode_attention(l, 1, None, w.batch, q_[l], p, out_[l])
                if record:
                    att_bytes.append(ctx.last_step_bytes())

    stream = torch.cuda.Stream()
    s_sel = torch.cuda.Stream()

    def step_overlapped(b=0):
        # The same launches with each producer group's selection on a second stream, beside the attention of
        # the group before it (a producer predicts for the layers after it, Sec. 3.1, so its selection does not
        # wait for their attention).  Pays where attention is slow: rows fetched over the host link.
        q_, qi_, out_ = bufs[b]
        ev = [torch.cuda.Event() for _ in groups]
        start = torch.cuda.Event()
        start.record(stream)
        s_sel.wait_event(start)
        with torch.cuda.stream(s_sel):
            ctx.select_topk(groups[0][0], groups[0][1], None, w.batch, qi_[groups[0][0]:groups[0][0] + groups[0][1]], p)
            ev[0].record(s_sel)
        for gi, (l0, n) in enumerate(groups):
            stream.wait_event(ev[gi])
            if gi + 1 < len(groups):
                l1, n1 = groups[gi + 1]
                with torch.cuda.stream(s_sel):
                    ctx.select_topk(l1, n1, None, w.batch, qi_[l1:l1 + n1], p)
                    ev[gi + 1].record(s_sel)
            for l in range(l0, l0 + n):
                ctx.sparse_decode_attention(l, 1, None, w.batch, q_[l], p, out_[l])

    with torch.cuda.stream(stream):
        n0 = ctx.launch_count()
        step_launches(record=True)
        launches_per_step = ctx.launch_count() - n0
        torch.cuda.synchronize()
        assert ctx.get_status(stream) == 0, "device status set during warm-up"
        if args.profile:
            # plain launches only (no graphs, no extra passes): the command line profilers are given
            for _ in range(args.warmup + args.steps):
                step_launches()
            torch.cuda.synchronize()
            return {"profile_run": w.name, "layers": w.n_layers, "launches_per_step": int(launches_per_step)}

        def capture(fn):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                fn()
            return g

        g_step = [capture(lambda: step_launches(b=0)), capture(lambda: step_launches(b=1))]
        g_sel = capture(lambda: [ctx.select_topk(l0, n, None, w.batch, qi[l0:l0 + n], p) for (l0, n) in groups])
        g_att = capture(lambda: [ctx.sparse_decode_attention(l, 1, None, w.batch, q[l], p, out[l]) for l in range(w.n_layers)])

        def timed(fn, steps, warmup, sampler=None, min_ms=300.0, stats=None, tail=None):
            """K steps between two events on the launching stream (barrier + synchronise on both sides),
            max over ranks; repeated until min_ms of device time have been timed.  Returns the median
            repeat in ms per step; `stats` receives min / max / repeats."""
            for _ in range(warmup):
                fn()
            torch.cuda.synchronize()
            if sampler:
                sampler.start()
            reps, total = [], 0.0
            while True:
                if world > 1:
                    dist.barrier()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(steps):
                    fn()
                if tail:
                    tail()                                  # joins work on other streams to the launching stream
                e1.record(stream)
                if sampler:
                    while not e1.query():
                        time.sleep(0.002)
                torch.cuda.synchronize()
                if world > 1:
                    dist.barrier()
                ms = max_over_ranks(e0.elapsed_time(e1), "cuda")       # the same number on every rank: a common exit
                reps.append(ms / steps)
                total += ms
                if total >= min_ms or len(reps) >= 400:
                    break
            if sampler:
                sampler.sample()
                sampler.stop_flag = True
            if stats is not None:
                stats.update({"min": float(np.min(reps)), "max": float(np.max(reps)), "repeats": len(reps)})
            return float(np.median(reps))

        sampler = ClockSampler(local)
        step_stats = {}
        ms_step = timed(g_step[0].replay, args.steps, args.warmup, sampler, stats=step_stats)

        # End to end through the public API: every step copies its queries and importance queries in from
        # page-locked host memory and its outputs back.  The copies run on two copy streams and the steps
        # alternate between two sets of device buffers, so step i+1's inputs cross the link while step i
        # computes and step i's outputs go back while step i+1 computes; events keep every buffer's
        # producer and consumer in order.
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_done = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]
        counter = [0]

        def e2e_step():
            b = counter[0] & 1
            counter[0] += 1
            q_, qi_, out_ = bufs[b]
            s_in.wait_event(ev_done[b])                     # the step that last read this set is through
            with torch.cuda.stream(s_in):
                q_.copy_(q_host, non_blocking=True)
                qi_.copy_(qi_host, non_blocking=True)
                ev_in[b].record(s_in)
            stream.wait_event(ev_in[b])
            stream.wait_event(ev_out[b])                    # this set's previous outputs have left
            g_step[b].replay()
            ev_done[b].record(stream)
            s_out.wait_event(ev_done[b])
            with torch.cuda.stream(s_out):
                out_host.copy_(out_, non_blocking=True)
                ev_out[b].record(s_out)

        def e2e_region_end():
            stream.wait_event(ev_out[0])
            stream.wait_event(ev_out[1])

        ms_e2e = timed(e2e_step, args.steps, args.warmup, tail=e2e_region_end)
        kstats_s, kstats_a = {}, {}
        ms_sel = timed(g_sel.replay, max(20, args.steps // 4), 3, min_ms=100.0, stats=kstats_s) / len(groups)
        ms_att = timed(g_att.replay, max(20, args.steps // 4), 3, min_ms=100.0, stats=kstats_a) / w.n_layers
        offload_info = None
        if args.offload_kv:
            # the comparison the paper draws for offloaded KV: the same step attending to every cached token
            p_dense = tbh.select_params(-1)
            g_dense = capture(lambda: [ctx.sparse_decode_attention(l, 1, None, w.batch, q[l], p_dense, out[l]) for l in range(w.n_layers)])
            ms_dense = timed(g_dense.replay, 3, 1, min_ms=0.0)
            dense_bytes = float(sum(w.lengths)) * w.n_layers * w.n_kv_heads * 2 * w.head_dim * (2 if w.dtype == wl.BF16 else 4)
            g_ov = capture(step_overlapped)
            ms_ov = timed(g_ov.replay, 3, 1, min_ms=0.0)
            res_rows = (min(w.sinks, min(w.lengths)) + min(w.recent, min(w.lengths))) if args.resident_rows else 0
            link_bytes = float(np.sum(att_bytes)) - float(res_rows) * w.n_layers * w.batch * w.n_kv_heads * 2 * w.head_dim * (2 if w.dtype == wl.BF16 else 4)
            offload_info = {"kv_placement": "page-locked host memory, rows fetched by the attention kernel over the host link",
                            "resident_sink_and_window_rows": bool(args.resident_rows),
                            "dense_step_us": ms_dense * 1e3, "dense_link_gbs": dense_bytes / (ms_dense * 1e-3) / 1e9,
                            "sparse_step_us": ms_step * 1e3, "sparse_link_bytes_per_step": link_bytes,
                            "sparse_link_gbs": link_bytes / (ms_step * 1e-3) / 1e9,
                            "sparse_step_us_selection_overlapped": ms_ov * 1e3,
                            "selection_us_per_step": ms_sel * len(groups) * 1e3,
                            "overlap_achieved": (ms_step - ms_ov) / max(1e-9, ms_sel * len(groups)),
                            "sparse_speedup_over_dense": ms_dense / min(ms_step, ms_ov)}
        ms_all = ms_pred = pred_bytes = None
        if not brief:
            # Upper bound, not the method's schedule: the importance queries of all layers at once, so the
            # selection runs as one call over every layer (many problems per launch) before the attentions.
            g_all = capture(lambda: (ctx.select_topk(0, w.n_layers, None, w.batch, qi, p),
                                     [ctx.sparse_decode_attention(l, 1, None, w.batch, q[l], p, out[l]) for l in range(w.n_layers)]))
            ms_all = timed(g_all.replay, max(20, args.steps // 4), 3, min_ms=100.0)
            # The step before the path, reported beside it (not inside the timed step): the importance-query
            # predictor of one producer layer, 8B-shaped (model dim 4096, hidden 512), random weights; 16 weight
            # sets are cycled so that every call reads its 8 MB from HBM, not from L2.
            E, HID, n_sets = 4096, 512, 16
            n_out = GROUP_LAYERS * w.n_q_heads * w.imp_dim
            pw = [(torch.randn(E, generator=gen, device="cuda").to(dt), torch.randn(E, generator=gen, device="cuda").to(dt),
                   (torch.randn(HID, E, generator=gen, device="cuda") * E ** -0.5).to(dt),
                   (torch.randn(n_out, HID, generator=gen, device="cuda") * HID ** -0.5).to(dt)) for _ in range(n_sets)]
            hs = torch.randn(w.batch, E, generator=gen, device="cuda").to(dt)
            p_scratch = torch.empty(w.batch * HID, device="cuda")
            p_out = torch.empty(GROUP_LAYERS, w.batch, w.n_q_heads, w.imp_dim, device="cuda")
            g_pred = capture(lambda: [tbh.predict_importance_queries(hs, a, b, w1, w2, w.dtype, w.n_q_heads, GROUP_LAYERS, w.imp_dim,
                                                                     p_scratch, p_out, stream=stream) for (a, b, w1, w2) in pw])
            ms_pred = timed(g_pred.replay, 20, 3, min_ms=50.0) / n_sets
            pred_bytes = (HID * E + n_out * HID + 2 * E + w.batch * E) * (2 if w.dtype == wl.BF16 else 4)
        assert ctx.get_status(stream) == 0, "device status set during the timed region"

    peak, peak_kind = measured_peaks()
    tokens = w.batch * world
    sel_b, att_b = float(np.mean(sel_bytes)), float(np.mean(att_bytes))
    step_bytes = float(np.sum(sel_bytes) + np.sum(att_bytes))
    dom = ("select_kernel", sel_b, ms_sel) if ms_sel * len(groups) >= ms_att * w.n_layers else ("attn_kernel", att_b, ms_att)
    achieved = dom[1] / (dom[2] * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": whole_job_tokens_per_s(w.batch, world, ms_step), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "us_per_step": ms_step * 1e3,
        "us_per_step_min": step_stats["min"] * 1e3, "us_per_step_max": step_stats["max"] * 1e3, "timed_repeats": step_stats["repeats"],
        "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": storage_name(w), "data": "synthetic",
        "config": {"workload": w.name + ("+offloaded_kv" if args.offload_kv else "") +
                   ("+lists_per_" + args.list_scope if args.list_scope != "kv_head" else ""), "layers": w.n_layers, "batch_per_gpu": w.batch,
                   "q_heads": w.n_q_heads,
                   "kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "imp_dim": w.imp_dim,
                   "kv_storage": storage_name(w), "accumulation": "f32", "context": w.lengths if len(set(w.lengths)) > 1 else w.lengths[0],
                   "budget": w.budget, "sinks": w.sinks, "recent": w.recent, "radius": w.radius, "interval": w.interval,
                   "schedule": "score+select per %d layers, attention per layer, CUDA-graph replay" % GROUP_LAYERS,
                   "timing": "median of %d repeats of %d steps (>= 0.3 s of device time)" % (step_stats["repeats"], args.steps),
                   "l2": "inputs larger than L2: %.0f MB touched per step" % (step_bytes / 1e6)},
        "step_hbm_gbs": step_bytes / (ms_step * 1e-3) / 1e9, "step_bytes": step_bytes,
        "step_frac_of_peak": step_bytes / (ms_step * 1e-3) / 1e9 / peak,
        "step_frac_of_nominal_8tbs": step_bytes / (ms_step * 1e-3) / 1e9 / 8000.0,
        "gpu_launches": int(launches_per_step * args.steps),
        "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": UNIT, "us_per_step": ms_e2e * 1e3,
                "h2d_bytes_per_step": q_host.numel() * q_host.element_size() + qi_host.numel() * 4,
                "d2h_bytes_per_step": out_host.numel() * 4,
                "how": "copies on two copy streams, two sets of device buffers: a step's copies overlap its neighbours' compute"},
        "roofline": {"bound": "hbm", "kernel": dom[0], "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": "of " + peak_kind, "traffic": NCU_TRAFFIC_BYTES.get((w.name, dom[0])),
                     "bytes_per_launch": dom[1], "us_per_launch": dom[2] * 1e3},
        "kernels": {"select_kernel": {"us_per_launch": ms_sel * 1e3, "bytes_per_launch": sel_b,
                                      "gbs": sel_b / (ms_sel * 1e-3) / 1e9, "frac": sel_b / (ms_sel * 1e-3) / 1e9 / peak,
                                      "launches_per_step": len(groups)},
                    "attn_kernel": {"us_per_launch": ms_att * 1e3, "bytes_per_launch": att_b,
                                    "gbs": att_b / (ms_att * 1e-3) / 1e9, "frac": att_b / (ms_att * 1e-3) / 1e9 / peak,
                                    "launches_per_step": w.n_layers}},
        "prefill_projection": proj_info,
        "clocks": sampler.summary(),
    }
    if not brief:
        line["upper_bound_all_layers_one_select_call"] = {
            "us_per_step": ms_all * 1e3, "step_frac_of_peak": step_bytes / (ms_all * 1e-3) / 1e9 / peak,
            "note": "selection for all layers in one call; needs every layer's importance query up front, which the "
                    "per-producer schedule does not have"}
        line["predictor_forward"] = {
            "us_per_producer": ms_pred * 1e3, "bytes_per_producer": pred_bytes, "gbs": pred_bytes / (ms_pred * 1e-3) / 1e9,
            "producers_per_step": len(groups), "step_incl_predictor_us": ms_step * 1e3 + len(groups) * ms_pred * 1e3,
            "note": "importance-query MLP of one producer layer; the step before the path, timed alone and added to the "
                    "step in step_incl_predictor_us"}
        line["offloaded_kv"] = offload_info
    del g_step, g_sel, g_att, ctx
    torch.cuda.empty_cache()
    return line


def measure_trajectory(args, w):
    """Workloads that decode: every step appends one token per sequence and layer, keys are projected
    in deferred batches of `recent` tokens, the selection (with neighbour expansion) is refreshed every
    `interval` steps and reused in between, attention runs every step.  Lengths change each step, so
    the launches are issued directly (kernel parameters carry the lengths); a step's GPU time is
    milliseconds, far above the launch cost.  Returns the JSON line as a dict."""
    import torch
    import torch.distributed as dist
    from paper_2503_07518_b200 import binding as tbh
    from paper_2503_07518_b200 import build
    build.build()

    world, rank, local = dist_env(torch, dist)
    P, Wn = w.interval, w.recent
    steps = max(P, args.steps // P * P)                      # whole refresh periods
    warm = max(P, (args.warmup + P - 1) // P * P)
    total = 2 * warm + 3 * steps                              # device-timed pass + end-to-end pass + graph-replay pass
    ctx = tbh.Context(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.imp_dim, w.dtype, w.batch, max(w.lengths) + total + Wn,
                      w.budget, w.radius, device=local, kv_on_host=args.offload_kv)
    if args.resident_rows:
        ctx.bind_resident_rows(max(w.sinks, 1), max(w.recent, 1))
    if args.important_buffer:
        ctx.bind_important_buffer()
    fill_caches(ctx, w, torch, tbh)
    dt = tbh.torch_dtype(w.dtype)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(wl.seed_for(w.cfg_id, 0, 0, wl.TAG_Q))
    shape_q = (w.n_layers, w.batch, w.n_q_heads)
    q = torch.randn(*shape_q, w.head_dim, generator=gen, device="cuda").to(dt)
    qi = torch.randn(*shape_q, w.imp_dim, generator=gen, device="cuda")
    k_new = torch.randn(w.n_layers, w.batch, w.n_kv_heads, w.head_dim, generator=gen, device="cuda").to(dt)
    v_new = torch.randn(w.n_layers, w.batch, w.n_kv_heads, w.head_dim, generator=gen, device="cuda").to(dt)
    out = torch.empty(*shape_q, w.head_dim, device="cuda")
    host = [t.cpu().pin_memory() for t in (q, qi, k_new, v_new)]
    out_host = torch.empty_like(out, device="cpu").pin_memory()
    groups = [(l, min(GROUP_LAYERS, w.n_layers - l)) for l in range(0, w.n_layers, GROUP_LAYERS)]
    proj = list(w.lengths)                                    # projected length per sequence (same in every layer)
    ones = [1] * w.batch
    bytes_sel, bytes_att = [0.0], [0.0]
    # the lists' realised lengths: copied out at every refresh (a copy kernel per producer group inside the timed
    # region), read back after the run, so that the attention bytes are what was gathered, not the (2r+1) B bound
    n_refresh_max = total // P + 2
    cnt_log = torch.zeros(n_refresh_max, w.n_layers, w.batch, w.n_kv_heads, dtype=torch.int32, device="cuda")
    es = 2 if w.dtype == wl.BF16 else 4

    # end-to-end leg: a second set of input / output buffers, so that a step's copies overlap its neighbours' compute
    dev_sets = [(q, qi, k_new, v_new, out), (q.clone(), qi.clone(), k_new.clone(), v_new.clone(), torch.empty_like(out))]

    def step(t, b=0):
        q, qi, k_new, v_new, out = dev_sets[b]
        p = tbh.select_params(w.budget, w.sinks, w.recent, w.radius, w.nmode, P, t)
        refresh = t % P == 0
        for (l0, n) in groups:
            for l in range(l0, l0 + n):
                ctx.append_kv(l, 1, None, ones, k_new[l], v_new[l])
                if refresh and t > 0:                         # the window wrapped: project its tokens in one batch
                    ctx.project_keys(l, 1, None, proj, [x + Wn for x in proj])
            # launches only on refresh steps
            ctx.select_topk(l0, n, None, w.batch, qi[l0:l0 + n], p, None, cnt_log[t // P, l0:l0 + n] if refresh else None)
            if refresh:
                bytes_sel[0] += ctx.last_step_bytes()
            for l in range(l0, l0 + n):
                ctx.sparse_decode_attention(l, 1, None, w.batch, q[l], p, out[l])
        if refresh and t > 0:
            for b in range(w.batch):
                proj[b] += Wn

    stream = torch.cuda.Stream()
    sampler = ClockSampler(local)
    with torch.cuda.stream(stream):
        t = 0
        for _ in range(warm):
            step(t)
            t += 1
        torch.cuda.synchronize()
        assert ctx.get_status(stream) == 0, "device status set during warm-up"
        if world > 1:
            dist.barrier()
        bytes_sel[0] = bytes_att[0] = 0.0
        t_first = t
        n0 = ctx.launch_count()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        sampler.start()
        ev[0].record(stream)
        for i in range(steps):
            step(t)
            t += 1
            ev[i + 1].record(stream)
        while not ev[-1].query():
            time.sleep(0.002)
        torch.cuda.synchronize()
        sampler.sample()
        sampler.stop_flag = True
        launches = ctx.launch_count() - n0
        per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
        ms_step = max_over_ranks(ev[0].elapsed_time(ev[-1]), "cuda") / steps
        refresh_ms = float(np.mean(per_step[0::P]))
        reuse_ms = float(np.mean([x for i, x in enumerate(per_step) if i % P]))
        # rows gathered per timed step: sinks + the list stored at the step's last refresh + window, per KV head
        cnt_host = cnt_log.cpu().numpy().astype(np.int64)
        for ts in range(t_first, t_first + steps):
            L_now = w.lengths[0] + ts + 1
            rows = min(w.sinks, L_now) * cnt_host[ts // P].size + int(cnt_host[ts // P].sum()) + min(w.recent, L_now) * cnt_host[ts // P].size
            bytes_att[0] += float(rows) * 2 * w.head_dim * es
        step_bytes = (bytes_sel[0] + bytes_att[0]) / steps
        att_bytes = bytes_att[0] / steps / w.n_layers
        bound_rows = (w.sinks + ((2 * w.radius + 1) if w.nmode == 0 else (1 + w.radius)) * w.budget + w.recent) * w.batch * w.n_kv_heads
        att_bytes_bound = float(bound_rows) * 2 * w.head_dim * es
        sel_bytes = bytes_sel[0] / max(1, steps // P) / len(groups)
        # end to end: the step's new K/V rows and queries come from pinned host memory, outputs go back; the copies
        # run on two copy streams and the steps alternate between two sets of device buffers (as in the static
        # workloads), events keep every buffer's producer and consumer in order
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_done = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(steps):
            b = i & 1
            s_in.wait_event(ev_done[b])                     # the step that last read this set is through
            with torch.cuda.stream(s_in):
                for dst, src in zip(dev_sets[b][:4], host):
                    dst.copy_(src, non_blocking=True)
                ev_in[b].record(s_in)
            stream.wait_event(ev_in[b])
            stream.wait_event(ev_out[b])                    # this set's previous outputs have left
            step(t, b)
            t += 1
            ev_done[b].record(stream)
            s_out.wait_event(ev_done[b])
            with torch.cuda.stream(s_out):
                out_host.copy_(dev_sets[b][4], non_blocking=True)
                ev_out[b].record(s_out)
        stream.wait_event(ev_out[0])
        stream.wait_event(ev_out[1])
        e1.record(stream)
        torch.cuda.synchronize()
        ms_e2e = e0.elapsed_time(e1) / steps
        # the two main kernels alone (same state, no appends): attention of every layer, refresh of every group
        pr = tbh.select_params(w.budget, w.sinks, w.recent, w.radius, w.nmode, P, 0)

        def alone(fn, reps):
            fn()
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            for _ in range(reps):
                fn()
            a1.record(stream)
            torch.cuda.synchronize()
            return a0.elapsed_time(a1) / reps

        att_ms = alone(lambda: [ctx.sparse_decode_attention(l, 1, None, w.batch, q[l], pr, out[l]) for l in range(w.n_layers)], 5) / w.n_layers
        sel_ms = alone(lambda: [ctx.select_topk(l0, n, None, w.batch, qi[l0:l0 + n], pr) for (l0, n) in groups], 3) / len(groups)
        assert ctx.get_status(stream) == 0, "device status set during the timed region"

        # The same trajectory as two CUDA graphs captured once (refresh step / reuse step) and replayed: the
        # kernels read the lengths from the device counters that the append and projection kernels advance.
        ctx.use_device_lengths(True, growth_reserve=warm + steps + 2 * P)
        cnt_g = torch.zeros(w.n_layers, w.batch, w.n_kv_heads, dtype=torch.int32, device="cuda")

        def graph_step(refresh):
            p = tbh.select_params(w.budget, w.sinks, w.recent, w.radius, w.nmode, P, 0 if refresh else 1)
            for (l0, n) in groups:
                for l in range(l0, l0 + n):
                    ctx.append_kv(l, 1, None, ones, k_new[l], v_new[l])
                    if refresh:                               # the tokens that left the window since the last refresh
                        ctx.project_keys(l, 1, None, None, None, n_seq=w.batch)
                ctx.select_topk(l0, n, None, w.batch, qi[l0:l0 + n], p, None, cnt_g[l0:l0 + n] if refresh else None)
                for l in range(l0, l0 + n):
                    ctx.sparse_decode_attention(l, 1, None, w.batch, q[l], p, out[l])

        graphs = {}
        for refresh in (True, False):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                graph_step(refresh)
            graphs[refresh] = g
        ctx.sync_lengths(stream)                              # capturing moved only the host mirrors
        for i in range(warm):
            graphs[i % P == 0].replay()
        torch.cuda.synchronize()
        gv = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        gv[0].record(stream)
        for i in range(steps):
            graphs[i % P == 0].replay()
            gv[i + 1].record(stream)
        torch.cuda.synchronize()
        assert ctx.get_status(stream) == 0, "device status set during the graph-replay pass"
        g_per = [gv[i].elapsed_time(gv[i + 1]) for i in range(steps)]
        ms_graph = max_over_ranks(gv[0].elapsed_time(gv[-1]), "cuda") / steps
        graph_refresh_ms = float(np.mean(g_per[0::P]))
        graph_reuse_ms = float(np.mean([x for i, x in enumerate(g_per) if i % P]))
        ctx.sync_lengths(stream)
        ctx.use_device_lengths(False)

    peak, peak_kind = measured_peaks()
    tokens = w.batch * world
    line = {
        "metric": METRIC, "value": whole_job_tokens_per_s(w.batch, world, ms_step), "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warm,
        "ms_per_step": ms_step, "us_per_step": ms_step * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": storage_name(w), "data": "synthetic",
        "config": {"workload": w.name + ("+offloaded_kv" if args.offload_kv else "") + ("+resident_rows" if args.resident_rows else "") +
                   ("+important_buffer" if args.important_buffer else ""),
                   "layers": w.n_layers, "batch_per_gpu": w.batch, "context": w.lengths[0], "budget": w.budget,
                   "recent": w.recent, "radius": w.radius, "neighbor_mode": "dilate" if w.nmode == 0 else "cluster",
                   "interval": P, "schedule": "per layer: append, (deferred projection), attention; select+expand per 4 layers on "
                   "refresh steps; direct launches", "l2": "inputs larger than L2: %.0f MB touched per step" % (step_bytes / 1e6)},
        "refresh_step_us": refresh_ms * 1e3, "reuse_step_us": reuse_ms * 1e3,
        "graph_replay": {"us_per_step": ms_graph * 1e3, "refresh_step_us": graph_refresh_ms * 1e3, "reuse_step_us": graph_reuse_ms * 1e3,
                         "step_frac_of_peak": step_bytes / (ms_graph * 1e-3) / 1e9 / peak,
                         "note": "the same steps as two CUDA graphs captured once (refresh / reuse) and replayed; lengths read "
                                 "from device counters advanced by the append and projection kernels"},
        "step_hbm_gbs": step_bytes / (ms_step * 1e-3) / 1e9, "step_bytes": step_bytes,
        "step_bytes_note": "realised: the stored lists' lengths read back after the run (upper bound per attention launch: %.1f MB)" % (att_bytes_bound / 1e6),
        "step_frac_of_peak": step_bytes / (ms_step * 1e-3) / 1e9 / peak,
        "step_frac_of_nominal_8tbs": step_bytes / (ms_step * 1e-3) / 1e9 / 8000.0, "gpu_launches": int(launches),
        "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": UNIT, "us_per_step": ms_e2e * 1e3,
                "h2d_bytes_per_step": sum(h.numel() * h.element_size() for h in host), "d2h_bytes_per_step": out_host.numel() * 4,
                "how": "copies on two copy streams, two sets of device buffers: a step's copies overlap its neighbours' compute"},
        "kernels": {"select_kernel+neighbor_kernel": {"us_per_launch": sel_ms * 1e3, "bytes_per_launch": sel_bytes,
                                                      "gbs": sel_bytes / (sel_ms * 1e-3) / 1e9, "launches_per_refresh": len(groups)},
                    "attn_kernel": {"us_per_launch": att_ms * 1e3, "bytes_per_launch": att_bytes,
                                    "gbs": att_bytes / (att_ms * 1e-3) / 1e9, "launches_per_step": w.n_layers}},
        "roofline": {"bound": "hbm", "kernel": "attn_mma_kernel", "achieved": att_bytes / (att_ms * 1e-3) / 1e9,
                     "peak": peak, "unit": "GB/s", "frac": att_bytes / (att_ms * 1e-3) / 1e9 / peak, "peak_kind": "of " + peak_kind,
                     "traffic": NCU_TRAFFIC_BYTES.get((w.name, "attn_kernel")) if w.nmode == 0 else None,
                     "bytes_per_launch": att_bytes, "us_per_launch": att_ms * 1e3},
        "clocks": sampler.summary(),
    }
    del ctx
    torch.cuda.empty_cache()
    return line


def measure_list_layouts(args, w):
    """Does it matter to the attention kernel where the listed rows lie?  (The paper's design migrates the
    selected rows into a contiguous Important buffer, Sec. 3.3; this build gathers them by index from the
    cache where they are.)  Same shapes, same list length, three layouts of the caller-supplied lists:
    random positions, runs of three consecutive positions, one contiguous block.  Prints one JSON line."""
    import torch
    import torch.distributed as dist
    from paper_2503_07518_b200 import binding as tbh
    from paper_2503_07518_b200 import build
    build.build()
    dist_env(torch, dist)
    ctx = tbh.Context(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.imp_dim, w.dtype, w.batch, max(w.lengths) + 8,
                      w.budget, w.radius)
    fill_caches(ctx, w, torch, tbh)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(wl.seed_for(w.cfg_id, 0, 0, wl.TAG_Q))
    q = torch.randn(w.n_layers, w.batch, w.n_q_heads, w.head_dim, generator=gen, device="cuda").to(tbh.torch_dtype(w.dtype))
    out = torch.empty(w.n_layers, w.batch, w.n_q_heads, w.head_dim, device="cuda")
    cap = ctx.index_capacity
    n_list = min(cap, ((2 * w.radius + 1) if w.nmode == 0 else (1 + w.radius)) * w.budget) // 3 * 3
    L = min(w.lengths)
    lo, hi = min(w.sinks, L), L - w.recent
    r = np.random.Generator(np.random.PCG64(wl.seed_for(w.cfg_id, 0, 0, wl.TAG_AUX)))
    units = w.n_layers * w.batch * w.n_kv_heads

    def lists(kind):
        rows = np.zeros((units, cap), np.int32)
        for u in range(units):
            if kind == "random":
                rows[u, :n_list] = np.sort(r.choice(np.arange(lo, hi), n_list, replace=False))
            elif kind == "runs_of_3":
                c = np.sort(r.choice(np.arange(lo, hi - 3, 3), n_list // 3, replace=False))
                rows[u, :n_list] = (c[:, None] + np.arange(3)[None, :]).reshape(-1)
            else:
                start = int(r.integers(lo, hi - n_list))
                rows[u, :n_list] = np.arange(start, start + n_list)
        return torch.from_numpy(rows.reshape(w.n_layers, w.batch, w.n_kv_heads, cap)).cuda()

    cnt = torch.full((w.n_layers, w.batch, w.n_kv_heads), n_list, dtype=torch.int32, device="cuda")
    p = tbh.select_params(w.budget, w.sinks, w.recent, w.radius, w.nmode)
    res = {}
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for kind in ("random", "runs_of_3", "contiguous"):
            idx = lists(kind)
            g = torch.cuda.CUDAGraph()
            for _ in range(2):
                for l in range(w.n_layers):
                    ctx.sparse_decode_attention(l, 1, None, w.batch, q[l], p, out[l], idx=idx[l:l + 1], cnt=cnt[l:l + 1])
            torch.cuda.synchronize()
            with torch.cuda.graph(g, stream=stream):
                for l in range(w.n_layers):
                    ctx.sparse_decode_attention(l, 1, None, w.batch, q[l], p, out[l], idx=idx[l:l + 1], cnt=cnt[l:l + 1])
            reps = []
            for _ in range(12):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(4):
                    g.replay()
                e1.record(stream)
                torch.cuda.synchronize()
                reps.append(e0.elapsed_time(e1) / 4 / w.n_layers * 1e3)
            res[kind] = {"us_per_layer": float(np.median(reps)), "min": float(np.min(reps)), "max": float(np.max(reps))}
        assert ctx.get_status(stream) == 0
    rows = (min(w.sinks, L) + n_list + min(w.recent, L)) * w.batch * w.n_kv_heads
    bytes_layer = rows * 2 * w.head_dim * (2 if w.dtype == wl.BF16 else 4)
    for v in res.values():
        v["gbs"] = bytes_layer / (v["us_per_layer"] * 1e-6) / 1e9
    print(json.dumps({"attention_list_layouts": res, "workload": w.name, "layers": w.n_layers, "batch": w.batch,
                      "rows_per_kv_head": rows // (w.batch * w.n_kv_heads), "bytes_per_layer": bytes_layer,
                      "note": "caller-supplied lists of equal length; the K|V rows are gathered by index from the cache in all three"}))


def brief_entry(line):
    """What the default run's `workloads` block keeps of another workload's line."""
    keep = ("us_per_step", "us_per_step_min", "us_per_step_max", "timed_repeats", "steps", "warmup", "value", "step_bytes", "graph_replay",
            "step_hbm_gbs", "step_frac_of_peak", "step_frac_of_nominal_8tbs", "refresh_step_us", "reuse_step_us", "roofline",
            "kernels", "e2e", "clocks", "gpu_launches")
    out = {k: line[k] for k in keep if k in line}
    out["config"] = {k: line["config"][k] for k in ("workload", "layers", "batch_per_gpu", "context", "budget", "schedule") if k in line["config"]}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", type=int, default=0,
                    help="workload 1..5; default: the 32K Llama-3-8B-shaped decode (2) as the line's value, plus a brief "
                         "`workloads` block for 3, 4 and 5")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (debugging)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-layers", type=int, default=2, help="layers in the CPU oracle's sample")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="default run without the `workloads` block")
    ap.add_argument("--profile", action="store_true", help="only warm-up + steps of plain launches (for ncu)")
    ap.add_argument("--offload-kv", action="store_true",
                    help="K|V cache in page-locked host memory (selected rows cross the host link); also times the dense step")
    ap.add_argument("--resident-rows", action="store_true",
                    help="with --offload-kv: device copies of the sink and window rows (only the selected rows cross the link)")
    ap.add_argument("--important-buffer", action="store_true",
                    help="the paper's contiguous Important buffer: selected rows migrated at every refresh, attended from there")
    ap.add_argument("--list-scope", default="kv_head", choices=["kv_head", "q_head", "layer"],
                    help="which heads share an index list (configs 1-4; default: one list per KV head)")
    ap.add_argument("--context", type=int, default=0,
                    help="override every sequence's context length (e.g. --config 4 --context 1048576 --layers 8)")
    ap.add_argument("--budget", type=int, default=0,
                    help="override the selection budget (e.g. --config 4 --budget 8192: the paper's latency setting, Sec. 4.3)")
    ap.add_argument("--list-layouts", action="store_true",
                    help="time the attention kernel on random / runs-of-3 / contiguous caller lists of the workload's shapes")
    ap.add_argument("--neighbors", default=None, choices=["dilate", "cluster"],
                    help="neighbour rule of the interval workload (default: its own, +-r dilation)")
    args = ap.parse_args()
    default_run = args.config == 0
    w = wl.workload(args.config or 2)
    if args.layers:
        w = w.scaled(n_layers=args.layers)
    if args.context:
        w = w.scaled(lengths=[args.context] * w.batch, name="%s@%d" % (w.name, args.context))
    if args.neighbors:
        w = w.scaled(nmode=0 if args.neighbors == "dilate" else 1)
    if args.budget:
        w = w.scaled(budget=args.budget, name="%s,budget=%d" % (w.name, args.budget))
    if args.impl == "reference":
        run_reference(args, w)
        return
    if args.warmup < 3:
        args.warmup = 3
    if args.list_layouts:
        measure_list_layouts(args, w)
        return

    def measure(wk, brief=False):
        if wk.decode_steps > 1:
            a2 = argparse.Namespace(**vars(args))
            a2.steps = min(args.steps, wk.decode_steps if not brief else 10 * wk.interval)
            return measure_trajectory(a2, wk)
        return measure_static(args, wk, brief=brief)

    line = measure(w)
    world, rank = int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0"))
    if "profile_run" not in line:
        extra = default_run and not args.no_extra and not args.profile and world == 1 and not args.offload_kv and \
            not args.important_buffer and \
            args.list_scope == "kv_head" and not args.layers and not args.context and not args.budget
        if extra:
            line["workloads"] = {}
            for cfg in (3, 4, 5):
                wk = wl.workload(cfg)
                if args.neighbors:
                    wk = wk.scaled(nmode=0 if args.neighbors == "dilate" else 1) if cfg == 5 else wk
                line["workloads"][wk.name] = brief_entry(measure(wk, brief=True))
        if rank == 0 and world == 1 and not args.no_cpu and args.list_scope == "kv_head" and w.decode_steps <= 1:
            leg = cpu_leg(w, args.cpu_layers, 3)                      # the oracle sample is per KV head
            best = min(leg["times"])
            one = cpu_leg(w, 1, 1, max_units=2, threads=1)            # and on one thread
            line["cpu_baseline"] = {"value": w.batch / best, "unit": UNIT, "cores": leg["threads"], "kind": "oracle",
                                    "sample": leg["sample"], "ms_per_step": best * 1e3,
                                    "value_1_thread": w.batch / one["times"][0], "sample_1_thread": one["sample"]}
    if rank == 0:
        print(json.dumps(line))
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
