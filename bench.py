#!/usr/bin/env python
"""Benchmark of the Focus-dLLM per-step sparse-attention path on B200.

One "step" = one non-block-entry denoising step of the 32-layer, 32K-context workload: the past-confidence
indicator, dense attention of the I_active rows in layers 0..16 (layer 16 also yields the sink set), and for
layers 17..31 block scoring against the cached pooled keys, Top-C selection and block-sparse attention.
Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import contextlib
import datetime
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "sparse attn step latency (ms) at 32K ctx"


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=float(d["hbm_gbs"]), tf_burst=float(d["bf16_tflops"]),
                    tf_sust=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), src="measured")
    return dict(hbm=6650.0, tf_burst=1590.0, tf_sust=1400.0, src="fallback")


class ClockSampler:
    """Samples SM clock, power and throttle reasons while the timed regions run: through NVML from a thread of this
    process (a sample every 2 ms, so that a region of tens of milliseconds holds a dozen), else with nvidia-smi
    (25 ms).  Both only read.

    Every sample carries a timestamp of the machine clock; `window()` brackets a timed region with host wall-clock
    times, and `stop()` keeps only the samples that fall inside a window, so that the median is a clock under load
    and not one taken while the host was building a graph."""
    Q = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    INTERVAL_MS = 25
    NVML_INTERVAL_MS = 2

    def __init__(self, index: int):
        self.index, self.proc, self.lines, self.windows, self.source = index, None, [], [], "nvidia-smi"

    def _start_nvml(self) -> bool:
        """One line per sample, in nvidia-smi's own CSV layout, appended to self.lines by a thread."""
        try:
            import pynvml as nv
            nv.nvmlInit()
            try:                                                   # the device torch calls `index`, whatever NVML's order
                uuid = str(torch.cuda.get_device_properties(self.index).uuid)
                h = nv.nvmlDeviceGetHandleByUUID(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
            except Exception:
                h = nv.nvmlDeviceGetHandleByIndex(self.index)
            cmax = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            nv.nvmlDeviceGetCurrentClocksEventReasons(h)
        except Exception:
            return False
        stop = threading.Event()
        act = lambda r, m: "Active" if r & m else "Not Active"

        def loop():
            while not stop.is_set():
                try:
                    ts = datetime.datetime.now()
                    clk = nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)
                    watts = nv.nvmlDeviceGetPowerUsage(h) / 1000.0
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
                    # bits: 0x4 sw power cap, 0x8 hw slowdown, 0x20 sw thermal slowdown, 0x40 hw thermal slowdown
                    self.lines.append(f"{ts:%Y/%m/%d %H:%M:%S.%f}, {self.index}, {clk}, {cmax}, {watts:.2f}, {r:#x}, "
                                      f"{act(r, 0x8)}, {act(r, 0x40)}, {act(r, 0x20)}, {act(r, 0x4)}\n")
                except Exception:
                    pass
                stop.wait(self.NVML_INTERVAL_MS / 1000)

        class _Stopper:
            terminate = staticmethod(stop.set)
        self.proc, self.INTERVAL_MS, self.source = _Stopper(), self.NVML_INTERVAL_MS, "nvml"
        self.t = threading.Thread(target=loop, daemon=True)
        self.t.start()
        t0 = time.time()
        while not self.lines and time.time() - t0 < 2.0:
            time.sleep(0.005)
        return True

    def start(self):
        if self._start_nvml():
            return
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", str(self.INTERVAL_MS)],
                                         stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.t.start()
            t0 = time.time()
            while not self.lines and time.time() - t0 < 5.0:      # first sample in hand before any timed region
                time.sleep(0.01)
        except Exception:
            self.proc = None

    def window(self, headline=False):
        """Context manager marking a timed region; samples stamped inside it count as 'under load'."""
        sampler = self

        class _W:
            def __enter__(self):
                self.t0 = datetime.datetime.now()

            def __exit__(self, *exc):
                sampler.windows.append((self.t0, datetime.datetime.now(), headline))
        return _W()

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(2 * self.INTERVAL_MS / 1000)
        self.proc.terminate()
        self.t.join(timeout=2)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        sm, sm_head, mx, watts, reasons, counts = [], [], [], [], set(), {n: 0 for n in names}
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 10:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f")
                clk, cmax = float(f[2]), float(f[3])
            except ValueError:
                continue
            mx.append(cmax)
            inside = [h for a, z, h in self.windows if a <= ts <= z]
            if not inside:
                continue
            sm.append(clk)
            if any(inside):
                sm_head.append(clk)
            try:
                watts.append(float(f[4]))
            except ValueError:
                pass
            for n, v in zip(names, f[6:10]):
                if v.lower().startswith("active"):
                    reasons.add(n)
                    counts[n] += 1
        note = None
        if not sm and mx:                                  # a very short region can fall between two samples
            note = "no sample fell inside a timed region; clocks of the samples around it"
            for ln in self.lines:
                f = [x.strip() for x in ln.split(",")]
                try:
                    sm.append(float(f[2]))
                except (ValueError, IndexError):
                    pass
        out = {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "samples_in_headline_region": len(sm_head),
                "sm_mhz_headline_region": statistics.median(sm_head) if sm_head else None,
                "power_w": statistics.median(watts) if watts else None,
                "interval_ms": self.INTERVAL_MS, "source": self.source, "reasons": sorted(reasons),
                "reason_share": {n: round(c / len(sm), 3) for n, c in counts.items() if c and sm}}
        if note:
            out["note"] = note
        return out


# --------------------------------------------------------------------------------------------------
# CPU oracle arm (also the cpu_baseline leg of the default arm)
# --------------------------------------------------------------------------------------------------
class OracleSample:
    """The CPU oracle on a bounded sample of one step: `heads` of the H heads, one dense layer, the probe-layer
    sink scores and one sparse layer (pooling included); `run()` times one pass and scales it to the whole step
    (all heads, the dense/sparse layer schedule).  Inputs are generated once, outside the timed part."""

    def __init__(self, w, heads=tuple(range(8))):
        from paper_2602_02159_b200 import workloads as wl
        self.w, s = w, w.shape
        hpg = s.H // s.Hkv
        self.kvh = sorted({h // hpg for h in heads if h < s.H})
        qh = [h for g in self.kvh for h in range(g * hpg, (g + 1) * hpg)]
        c_prev, _ = wl.gen_confidence(w.seed, s.N)
        self.conf, self.masked = wl.full_conf(s, c_prev), wl.gen_masked(w)
        self.sparse_layer = min(w.probe_layer + 1, w.n_layers - 1)
        self.lay = {}
        for layer in (0, w.probe_layer, self.sparse_layer):
            if layer not in self.lay:
                t = wl.gen_qkv(s, layer, threads=0)
                self.lay[layer] = tuple(wl.storage_to_f64(t[n][self.kvh] if n != "Q" else t[n][:, qh], s.dtype)
                                        for n in "QKV")

    def run(self):
        from oracle import focus_oracle as fo
        w, s = self.w, self.w.shape
        scale = 1.0 / math.sqrt(s.d)
        Ld, Lp, Ls = self.lay[0], self.lay[w.probe_layer], self.lay[self.sparse_layer]
        t0 = time.perf_counter()
        focus, active = fo.select_queries(self.conf, self.masked, w.blk_lo, w.blk_hi, w.k, w.w, s.M, s.L)
        t1 = time.perf_counter()
        fo.dense_attn(Ld[0][active - s.M], Ld[1], Ld[2], scale)
        t2 = time.perf_counter()
        S = fo.sink_scores(Lp[0][active - s.M], Lp[1], scale)
        sinks = fo.find_sinks(S, w.n_sink, 0, s.M)
        t3 = time.perf_counter()
        R = fo.score_blocks(Ls[0][focus - s.M], fo.pool_keys(Ls[1], s.M, s.B), fo.PER_KV_GROUP)
        blocks, _ = fo.select_blocks(R, w.C, sinks, s.B)
        fo.sparse_attn(Ls[0][active - s.M], Ls[1], Ls[2], s.M, s.B, blocks, sinks, scale)
        t4 = time.perf_counter()
        f = s.Hkv / len(self.kvh)
        n_dense, n_sparse = w.probe_layer + 1, w.n_layers - w.probe_layer - 1
        est = (t1 - t0) + f * (n_dense * (t2 - t1) + (t3 - t2) + n_sparse * (t4 - t3))
        try:
            from threadpoolctl import threadpool_info
            cores = max([i.get("num_threads", 1) for i in threadpool_info()] or [1])
        except Exception:
            cores = os.cpu_count() or 1
        sample = (f"{len(self.kvh)} of {s.Hkv} KV heads; 1 dense layer + probe-layer sink scores + 1 sparse layer "
                  f"(pooling included), {t4 - t0:.2f} s of oracle time per pass, scaled by heads and by the schedule "
                  f"{n_dense} dense / {n_sparse} sparse layers")
        return est * 1e3, cores, sample


def run_reference(args):
    from paper_2602_02159_b200 import workloads as wl
    if int(os.environ.get("RANK", "0")) != 0:
        return
    w = wl.config(args.config)
    smp = OracleSample(w)
    vals, timed_s = [], 0.0
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        ms, cores, sample = smp.run()
        if i >= args.warmup:
            vals.append(ms)
            timed_s += time.perf_counter() - t0
    v = float(np.mean(vals))
    # `value` is an extrapolation: each timed pass runs a bounded sample of a step (see cpu_baseline.sample) and is
    # scaled to the whole step, so steps x value is far more than the wall time of this run
    out = {"impl": "reference", "metric": METRIC, "value": v, "unit": "ms", "n_gpus": args.gpus, "steps": len(vals),
           "warmup": args.warmup, "ms_per_step": v, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
           "dtype": "f64", "data": "synthetic", "extrapolated": True, "timed_passes": len(vals),
           "timed_s": round(timed_s, 3),
           "config": {"workload": w.name, "rows": "I_active (paper)", "note": "CPU oracle, bounded sample scaled to a step"},
           "cpu_baseline": {"value": v, "unit": "ms", "cores": cores, "kind": "oracle", "sample": sample},
           "e2e": {"value": v, "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


# --------------------------------------------------------------------------------------------------
# CUDA arm
# --------------------------------------------------------------------------------------------------
def run_focus(args):
    import torch
    import torch.distributed as dist

    from paper_2602_02159_b200 import binding as fb
    from paper_2602_02159_b200 import build as fbuild
    from paper_2602_02159_b200 import step as fstep
    from paper_2602_02159_b200 import workloads as wl

    from paper_2602_02159_b200 import replicas
    rank, world, local = replicas.env_ranks()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    replicas.init("nccl", torch.device("cuda", local))
    if rank == 0:
        fbuild.build()
    if world > 1:
        replicas.barrier()
    ctx = fb.Context(local, workspace_bytes=512 << 20)
    w = wl.config(args.config)
    if args.layers:
        import dataclasses
        w = dataclasses.replace(w, n_layers=args.layers, probe_layer=min(w.probe_layer, max(0, args.layers // 2)))
    s = w.shape
    P = peaks()
    dev = torch.device("cuda", local)
    NL, probe = w.n_layers, w.probe_layer
    n_dense, n_sparse = probe + 1, NL - probe - 1

    # ---- inputs: per-layer Q/K/V (seed = layer index; replicas offset the seed), confidence, masks -------------
    t_gen = time.perf_counter()
    Qs, Ks, Vs, Kbars = [], [], [], []
    Q_host = torch.empty(NL, s.N, s.H, s.d, dtype=torch.bfloat16).pin_memory()
    for l in range(NL):
        t = wl.gen_qkv(s, replicas.replica_seed(l, rank), threads=0)
        Q_host[l].copy_(torch.from_numpy(t["Q"].view(np.int16)).view(torch.bfloat16))
        Qs.append(Q_host[l].to(dev, non_blocking=True))
        Ks.append(fstep.to_device(t["K"], s.dtype, dev))
        Vs.append(fstep.to_device(t["V"], s.dtype, dev))
        del t
    c_prev, _ = wl.gen_confidence(w.seed, s.N)
    conf_host = torch.from_numpy(wl.full_conf(s, c_prev)).pin_memory()
    masked_host = torch.from_numpy(wl.gen_masked(w)).pin_memory()
    conf, masked = conf_host.to(dev), masked_host.to(dev)
    t_gen = time.perf_counter() - t_gen

    results = {}
    for rows in ("active", "gen"):
        b = fstep.StepBuffers(w, rows=rows, device=dev)
        O_all = torch.zeros(NL, b.max_rows, s.H, s.d, dtype=torch.bfloat16, device=dev)
        lse_probe = torch.zeros(s.H, b.max_active, dtype=torch.float32, device=dev)
        results[rows] = dict(b=b, O=O_all, lse_probe=lse_probe)
    # pooled keys are cached per KV-cache refresh (prompt keys do not change between the steps of a block)
    for l in range(NL):
        kb = torch.zeros(s.Hkv, s.nb, s.d, dtype=torch.float32, device=dev) if l > probe else None
        if kb is not None:
            fb.focus_pool_keys(ctx, results["active"]["b"].shape, Ks[l], kb)
        Kbars.append(kb)
    torch.cuda.synchronize()

    ev = lambda: torch.cuda.Event(enable_timing=True)

    def step(rows, dense_only=False, kbar=True, marks=None, probe_lse_for_active=True, pre_layer=None, post_layer=None):
        """Enqueue one denoising step.  marks: list collecting (kind, start_event, end_event) per attention call;
        pre_layer(l) / post_layer(l): called before / after layer l is enqueued (the end-to-end run waits there for
        the layer's inputs and sends the layer's output home)."""
        r = results[rows]
        b, O_all = r["b"], r["O"]
        fstep.select_queries(ctx, b, conf, masked)
        last_dense = NL - 1 if dense_only else probe
        for l in range(last_dense + 1):
            if pre_layer is not None:
                pre_layer(l)
            if marks is not None:
                e0, e1 = ev(), ev(); e0.record()
            fstep.dense_layer(ctx, b, Qs[l], Ks[l], Vs[l], O=O_all[l])
            if marks is not None:
                e1.record(); marks.append(("dense", e0, e1))
            if post_layer is not None:
                post_layer(l)
        if dense_only:
            return
        # probe layer: LSE of the I_active rows (from the dense pass when the attention rows are I_active)
        if rows == "active":
            fstep.find_sinks(ctx, b, Qs[probe], Ks[probe], b.lse)
        else:
            # attention rows are the whole gen region: one more dense pass over the I_active rows yields their LSE
            fb.focus_dense_attn(ctx, b.shape, Qs[probe], s.M, s.N, b.active_idx, b.n_active, b.max_active, Ks[probe],
                                Vs[probe], results["active"]["O"][probe], r["lse_probe"])
            fstep.find_sinks(ctx, b, Qs[probe], Ks[probe], r["lse_probe"])
        for l in range(probe + 1, NL):
            if pre_layer is not None:
                pre_layer(l)
            if marks is not None:
                e0, e1 = ev(), ev(); e0.record()
            fstep.sparse_layer(ctx, b, Qs[l], Ks[l], Vs[l], Kbar=Kbars[l] if kbar else None, O=O_all[l])
            if marks is not None:
                e1.record(); marks.append(("sparse", e0, e1))
            if post_layer is not None:
                post_layer(l)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            replicas.barrier()
            torch.cuda.synchronize()

    sampler = None

    def timed(fn, steps, warmup, with_marks=False, headline=False):
        # every timed region starts from an idle part: what ran before (seconds of gen-row attention, say) would
        # otherwise decide under which power state this region is measured; the back-to-back figure is `sustained`
        sync_all()
        time.sleep(args.cooldown_s)
        for _ in range(warmup):
            fn(None)
        sync_all()
        marks = [] if with_marks else None
        evs = [(ev(), ev()) for _ in range(steps)]
        n0 = fb.focus_launch_count()
        with (sampler.window(headline) if sampler is not None else contextlib.nullcontext()):
            for a, z in evs:
                a.record(); fn(marks); z.record()
            sync_all()
        launches = fb.focus_launch_count() - n0
        ms = [a.elapsed_time(z) for a, z in evs]
        tot = float(sum(ms))
        tot = replicas.max_over_ranks(tot, dev)
        return tot / steps, launches, marks

    K, W = args.steps, max(args.warmup, 3)
    # eager pass with CUDA-event marks around every attention call (per-call durations; the roofline uses them only
    # with --no-graph, otherwise the per-launch average of a graph of those launches, see below)
    sampler = ClockSampler(local)
    sampler.INTERVAL_MS = max(5, args.clock_interval_ms)
    sampler.start()
    ms_eager, launches, marks = timed(lambda m: step("active", marks=m), K, W, with_marks=True,
                                      headline=args.no_graph)
    assert ctx.poll_status() == 0, "device status word set during the timed region"
    # the same step captured once into a CUDA graph (counts stay on the device, so nothing needs the host)
    graph = None
    if not args.no_graph:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            step("active")
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        n0 = fb.focus_launch_count()
        with torch.cuda.graph(graph):
            step("active")
        launches = fb.focus_launch_count() - n0          # kernels per replayed step
    if graph is not None:
        ms_step, _, _ = timed(lambda m: graph.replay(), K, W, headline=True)
        launches *= K
    else:
        ms_step = ms_eager
    assert ctx.poll_status() == 0, "device status word set during the timed region"

    # The sampler stops here: with nvidia-smi polling every 25 ms the per-launch figures below came out 5-8 % slower
    # (measured by alternating runs), while the step time above did not move beyond its run-to-run spread.
    clocks = sampler.stop()
    sampler = None
    dense_t = [a.elapsed_time(z) for kind, a, z in marks if kind == "dense"]
    sparse_t = [a.elapsed_time(z) for kind, a, z in marks if kind == "sparse"]
    # The dominant kernel in the launch mode of the headline number: the dense-attention launches of one step (each on
    # its own layer's K/V, 537 MB apiece) captured alone into a graph; average time per launch over K replays,
    # gaps between the launches included.
    def per_launch_in_graph(rows, kind, steps):
        """Average time per launch of the step's dense (or sparse) layers, captured alone into a graph."""
        r_ = results[rows]
        layers = range(probe + 1) if kind == "dense" else range(probe + 1, NL)
        if len(layers) == 0:
            return None
        b_ = r_["b"]
        q_rows_, n_rows_, max_rows_ = b_._rows()

        def run():
            for l in layers:
                if kind == "dense":
                    fstep.dense_layer(ctx, b_, Qs[l], Ks[l], Vs[l], O=r_["O"][l])
                elif kind == "sparse":                     # sink set from the last full step
                    fstep.sparse_layer(ctx, b_, Qs[l], Ks[l], Vs[l], Kbar=Kbars[l], O=r_["O"][l])
                else:                                      # the attention call alone, on the lists the last layer call left
                    fb.focus_sparse_attn(ctx, b_.shape, Qs[l], b_.q_base, b_.n_q, q_rows_, n_rows_, max_rows_, Ks[l],
                                         Vs[l], fb.HEADS_PER_KV_GROUP, b_.block_idx, b_.max_blocks, b_.block_cnt,
                                         b_.sink_idx, b_.sink_keep, w.n_sink, r_["O"][l], b_.lse)
        run()
        torch.cuda.synchronize()
        g_ = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_):
            run()
        ms_, _, _ = timed(lambda m: g_.replay(), steps, W)
        return ms_ / len(layers)

    dense_graph_ms = sparse_graph_ms = None
    if graph is not None:
        dense_graph_ms = per_launch_in_graph("active", "dense", K)
        sparse_graph_ms = per_launch_in_graph("active", "sparse", K)
    # practical read ceiling: the library's read-only streaming probe over two 2 GiB buffers in turn (launch gaps
    # are 2 % of a pass of that size), per pass inside a graph
    probe_out = torch.zeros(1, dtype=torch.int32, device="cuda")
    probe_bytes = 2 << 30
    probe_bufs = [torch.randint(0, 255, (probe_bytes,), dtype=torch.uint8, device="cuda") for _ in range(2)]
    stream_gbs = probe_bytes / (graph_time_us(lambda l: fb.focus_stream_read(ctx, probe_bufs[l], probe_bytes, probe_out),
                                              2, warm=3, reps=20) * 1e-6) / 1e9
    del probe_bufs
    eb = 2
    kv_bytes = 2 * s.Hkv * s.L * s.d * eb
    na = int(results["active"]["b"].n_active.item())
    qo_bytes = 2 * na * s.H * s.d * eb
    dense_eager_ms = float(np.mean(dense_t))
    dense_ms = dense_graph_ms if dense_graph_ms is not None else dense_eager_ms
    dense_gbs = (kv_bytes + qo_bytes) / (dense_ms * 1e-3) / 1e9
    retained_keys = w.C * s.B + w.n_sink + s.N                      # upper bound per head (sinks inside blocks are skipped)
    sparse_bytes = 2 * s.Hkv * retained_keys * s.d * eb + qo_bytes
    sparse_eager_ms = float(np.mean(sparse_t)) if sparse_t else float("nan")
    sparse_ms = sparse_graph_ms if sparse_graph_ms is not None else sparse_eager_ms

    # ---- own dense baseline (every layer dense), cold pooled keys, gen-region rows -----------------------
    ms_dense_step, _, _ = timed(lambda m: step("active", dense_only=True), max(2, K // 4), 2)
    ms_cold, _, _ = timed(lambda m: step("active", kbar=False), max(2, K // 2), 2)
    gen = {}
    if not args.skip_gen:
        ms_gen, _, gm = timed(lambda m: step("gen", marks=m), max(2, K // 4), 2, with_marks=True)
        ms_gen_dense, _, _ = timed(lambda m: step("gen", dense_only=True), 2, 1)
        gd_eager = float(np.mean([a.elapsed_time(z) for k_, a, z in gm if k_ == "dense"]))
        gs_eager = float(np.mean([a.elapsed_time(z) for k_, a, z in gm if k_ == "sparse"]))
        gd, gs, gsa = gd_eager, gs_eager, None
        if graph is not None:                              # same launch mode as the paper-row figures
            gd = per_launch_in_graph("gen", "dense", max(2, K // 4)) or gd_eager
            gs = per_launch_in_graph("gen", "sparse", max(2, K // 4)) or gs_eager
            gsa = per_launch_in_graph("gen", "sparse_attn", max(2, K // 4))
        fl_dense = 4.0 * s.N * s.L * s.d * s.H
        fl_sparse = 4.0 * s.N * retained_keys * s.d * s.H
        gen = {"rows": s.N, "ms_per_step": ms_gen, "dense_ms_per_step": ms_gen_dense,
               "speedup_vs_own_dense": ms_gen_dense / ms_gen,
               "dense_layer_ms": gd, "dense_layer_tflops": fl_dense / gd / 1e9,
               "sparse_layer_ms": gs, "sparse_retained_tflops": fl_sparse / gs / 1e9,
               "sparse_dense_equiv_tflops": fl_dense / gs / 1e9,
               "dense_layer_eager_marks_ms": gd_eager, "sparse_layer_eager_marks_ms": gs_eager,
               # these launches are timed alone in millisecond replays (burst conditions): frac is of the burst peak, the
               # sustained-peak and nominal fractions stand beside it
               "roofline": tensor_roofline(fl_dense / gd / 1e9, P, "attn_tc_wide_kernel<false> (dense layer, 512 gen rows)"),
               "sparse_roofline": tensor_roofline(fl_sparse / gs / 1e9, P,
                                                  "sparse layer on retained blocks, 512 gen rows: selection kernel + "
                                                  "sparse attention kernel"),
               "sparse_attn_only_ms": gsa,
               "sparse_attn_only_roofline": tensor_roofline(fl_sparse / gsa / 1e9, P,
                                                            "sparse attention kernel alone (lists from the last layer call)")
               if gsa else None}
    assert ctx.poll_status() == 0

    # ---- end to end through the C ABI with host buffers (K/V cache resident: it is model state, Eq. 3) -------
    r = results["active"]
    bact = r["b"]
    O_host = torch.empty(NL, bact.max_rows, s.H, s.d, dtype=torch.bfloat16).pin_memory()
    idx_host = torch.empty(bact.max_active + bact.sink_idx.numel() + 2, dtype=torch.int32).pin_memory()
    h2d = conf_host.numel() * 4 + masked_host.numel() + Q_host.numel() * 2
    d2h = O_host.numel() * 2 + idx_host.numel() * 4

    copy_stream, back_stream = torch.cuda.Stream(), torch.cuda.Stream()
    q_ready = [torch.cuda.Event() for _ in range(NL)]
    o_ready = [torch.cuda.Event() for _ in range(NL)]

    def e2e_step(_m):
        # the layers' Q rows arrive on a copy stream, layer by layer, while earlier layers compute; every layer waits
        # for its own rows only, and its output goes back on a third stream as soon as it exists
        main = torch.cuda.current_stream()
        conf.copy_(conf_host, non_blocking=True)
        masked.copy_(masked_host, non_blocking=True)
        copy_stream.wait_stream(main)                    # the previous step may still be reading the Q buffers
        with torch.cuda.stream(copy_stream):
            for l in range(NL):
                Qs[l].copy_(Q_host[l], non_blocking=True)
                q_ready[l].record(copy_stream)
        def send_home(l):
            o_ready[l].record(main)
            back_stream.wait_event(o_ready[l])
            with torch.cuda.stream(back_stream):
                O_host[l].copy_(r["O"][l], non_blocking=True)

        step("active", pre_layer=lambda l: main.wait_event(q_ready[l]), post_layer=send_home)
        idx_host[:bact.max_active].copy_(bact.active_idx, non_blocking=True)
        idx_host[bact.max_active:bact.max_active + bact.sink_idx.numel()].copy_(bact.sink_idx, non_blocking=True)
        main.wait_stream(back_stream)
        main.synchronize()

    ms_e2e_all, _, _ = timed(e2e_step, max(2, K // 2), 2)

    # The same step with only the rows that are read crossing PCIe.  After the indicator the host reads I_focus and
    # I_active back (a few hundred bytes), gathers those rows of every layer's Q in pinned memory (index bookkeeping on
    # the host, no arithmetic) and uploads them as a compact [layer, row] array; the library is handed local row
    # numbers.  Layers run as graphs of a few layers each so that the gather of the next chunk overlaps the GPU work of
    # the current one; every chunk's outputs go home inside the next chunk's graph, on a second captured stream.
    bc = fstep.StepBuffers(w, rows="compact", device=dev)
    MA = bc.max_active
    Qc = torch.zeros(NL, MA, s.H, s.d, dtype=torch.bfloat16, device=dev)
    Oc = torch.zeros(NL, MA, s.H, s.d, dtype=torch.bfloat16, device=dev)
    Qc_host = torch.zeros(NL, MA, s.H, s.d, dtype=torch.bfloat16).pin_memory()
    Oc_host = torch.zeros(NL, MA, s.H, s.d, dtype=torch.bfloat16).pin_memory()
    sel_dev = torch.zeros(2 + max(1, w.k) + MA, dtype=torch.int32, device=dev)
    sel_host = torch.zeros(2 + max(1, w.k) + MA, dtype=torch.int32).pin_memory()
    sink_host = torch.zeros(bc.sink_idx.numel(), dtype=torch.int32).pin_memory()
    # chunk sizes: what precedes the first graph (indicator, read-back, gather and upload of the first chunk's rows) and
    # what follows the last (its outputs going home) is serial, so the first and the last chunk are short
    if NL >= 12:
        bounds = [0] + [2 + round(i * (NL - 4) / 3) for i in range(4)] + [NL]
    else:
        nc = max(1, min(4, NL // 2))
        bounds = [round(i * NL / nc) for i in range(nc + 1)]
    n_chunks = len(bounds) - 1
    chunk_ready = [torch.cuda.Event() for _ in range(n_chunks)]

    def chunk_layers(c, home_prev):
        side = torch.cuda.Stream()
        cur = torch.cuda.current_stream()
        if home_prev and c > 0:                          # outputs of the previous chunk go home beside this chunk's work
            side.wait_stream(cur)
            with torch.cuda.stream(side):
                Oc_host[bounds[c - 1]:bounds[c]].copy_(Oc[bounds[c - 1]:bounds[c]], non_blocking=True)
        for l in range(bounds[c], bounds[c + 1]):
            if l <= probe:
                fstep.dense_layer(ctx, bc, Qc[l], Ks[l], Vs[l], O=Oc[l])
                if l == probe:
                    fstep.find_sinks(ctx, bc, Qc[l], Ks[l], bc.lse)
            else:
                fstep.sparse_layer(ctx, bc, Qc[l], Ks[l], Vs[l], Kbar=Kbars[l], O=Oc[l])
        if home_prev and c > 0:
            cur.wait_stream(side)

    chunk_graphs = None
    if graph is not None:
        # warm every call of the compact path once (function attributes, occupancy queries) before capturing
        fstep.select_queries(ctx, bc, conf, masked)
        bc.set_local_focus(results["active"]["b"].focus_idx.cpu().numpy()[:int(results["active"]["b"].n_focus.item())],
                           results["active"]["b"].active_idx.cpu().numpy()[:na])
        for c in range(n_chunks):
            chunk_layers(c, False)
        torch.cuda.synchronize()
        chunk_graphs = []
        for c in range(n_chunks):
            g_ = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_):
                chunk_layers(c, True)
            chunk_graphs.append(g_)

    e2e_marks = []                                       # host clock at the phase boundaries of every end-to-end step

    def e2e_compact_step(_m):
        main = torch.cuda.current_stream()
        tm = [time.perf_counter()]
        conf.copy_(conf_host, non_blocking=True)
        masked.copy_(masked_host, non_blocking=True)
        fstep.select_queries(ctx, bc, conf, masked)
        sel_dev[0:1].copy_(bc.n_focus, non_blocking=True); sel_dev[1:2].copy_(bc.n_active, non_blocking=True)
        sel_dev[2:2 + bc.focus_idx.numel()].copy_(bc.focus_idx, non_blocking=True)
        sel_dev[2 + bc.focus_idx.numel():].copy_(bc.active_idx, non_blocking=True)
        sel_host.copy_(sel_dev, non_blocking=True)
        main.synchronize()
        tm.append(time.perf_counter())                   # indicator done, index sets on the host
        nf_, na_ = int(sel_host[0]), int(sel_host[1])
        fpos = sel_host[2:2 + nf_]
        apos = sel_host[2 + bc.focus_idx.numel():2 + bc.focus_idx.numel() + na_]
        bc.set_local_focus(fpos.tolist(), apos.tolist())
        rows_idx = (apos - s.M).to(torch.int64)
        for c in range(n_chunks):
            for l in range(bounds[c], bounds[c + 1]):
                torch.index_select(Q_host[l], 0, rows_idx, out=Qc_host[l, :na_])
            with torch.cuda.stream(copy_stream):
                if c == 0:
                    copy_stream.wait_stream(main)
                for l in range(bounds[c], bounds[c + 1]):    # one contiguous block per layer: plain DMA from pinned memory
                    Qc[l, :na_].copy_(Qc_host[l, :na_], non_blocking=True)
                chunk_ready[c].record(copy_stream)
            main.wait_event(chunk_ready[c])
            if chunk_graphs is not None:
                chunk_graphs[c].replay()
            else:
                chunk_layers(c, True)
            if c == 0:
                tm.append(time.perf_counter())           # first chunk gathered, uploaded and launched
        Oc_host[bounds[-2]:].copy_(Oc[bounds[-2]:], non_blocking=True)
        sink_host.copy_(bc.sink_idx, non_blocking=True)
        tm.append(time.perf_counter())                   # everything enqueued
        main.synchronize()
        tm.append(time.perf_counter())
        e2e_marks.append(tm)

    ms_e2e, _, _ = timed(e2e_compact_step, max(2, K // 2), 2)
    h2d_c = conf_host.numel() * 4 + masked_host.numel() + NL * na * s.H * s.d * 2 + 4 * max(1, w.k)
    e2e_phases = None
    if e2e_marks:
        tail = e2e_marks[-max(2, K // 2):]               # the timed steps
        med = lambda i: float(np.median([(t[i + 1] - t[i]) * 1e3 for t in tail]))
        e2e_phases = {"indicator_and_readback_ms": round(med(0), 3), "first_chunk_gather_upload_launch_ms": round(med(1), 3),
                      "remaining_enqueue_ms": round(med(2), 3), "wait_for_the_device_ms": round(med(3), 3),
                      "note": "host clock between the phase boundaries of the timed end-to-end steps (medians)"}
    d2h_c = Oc_host.numel() * 2 + sel_host.numel() * 4 + sink_host.numel() * 4

    # ---- sustained leg: the same graph replayed back to back for >= 2 s of device time, clocks sampled inside --------
    sustained = None
    if graph is not None and args.sustain_s > 0:
        n_rep = max(K, int(math.ceil(args.sustain_s * 1e3 / ms_step)))
        sus = ClockSampler(local)
        sus.INTERVAL_MS, sus.NVML_INTERVAL_MS = 25, 10
        sus.start()
        a, z = ev(), ev()
        sync_all()
        with sus.window(True):
            a.record()
            for _ in range(n_rep):
                graph.replay()
            z.record()
            sync_all()
        tot = replicas.max_over_ranks(a.elapsed_time(z), dev)
        ck = sus.stop()
        sustained = {"ms_per_step": tot / n_rep, "replays": n_rep, "seconds": tot / 1e3, "sm_mhz_median": ck["sm_mhz"],
                     "clock_samples": ck["samples"], "power_w_median": ck["power_w"], "reasons": ck["reasons"],
                     "reason_share": ck.get("reason_share", {}),
                     "ms_x_mhz": (tot / n_rep) * ck["sm_mhz"] if ck["sm_mhz"] else None,
                     "burst_ms_x_mhz": ms_step * clocks["sm_mhz_headline_region"] if clocks.get("sm_mhz_headline_region") else None,
                     "note": "back-to-back replays of the headline graph; the headline value above is a burst of K replays"}
    if rank != 0:
        replicas.shutdown()
        return
    # ---- CPU oracle on a bounded sample (rank 0, N = 1 only) ------------------------------------------------
    cpu = None
    if world == 1 and not args.skip_cpu:
        smp = OracleSample(w)
        v, cores, sample = min((smp.run() for _ in range(3)), key=lambda r: r[0])
        cpu = {"value": v, "unit": "ms", "cores": cores, "kind": "oracle", "sample": sample}

    # dram__bytes_read.sum + dram__bytes_write.sum of one dense-layer launch of this shape (32 heads, L = 32768,
    # I_active rows) from the ncu capture of that kernel summarised under profiles/
    traffic = 541_483_264 if (args.config == 2 and not args.layers) else None
    out = {
        "metric": METRIC, "value": ms_step, "unit": "ms", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_step, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "L": s.L, "gen": s.N, "heads": s.H, "kv_heads": s.Hkv, "head_dim": s.d,
                   "layers": NL, "dense_layers": n_dense, "sparse_layers": n_sparse, "kv_block": s.B, "keep_blocks": w.C,
                   "n_sink": w.n_sink, "k": w.k, "w": w.w, "rows": f"I_active ({na} rows, the paper's query set)",
                   "pooled_keys": "cached per KV-cache refresh", "l2": "inputs larger than L2 (17 GB of K/V per step)",
                   "multi_gpu": "independent replicas, no data-path collective", "input_gen_s": round(t_gen, 1)},
        "gpu_launches": int(launches),
        "steps_per_s_all_replicas": world * 1e3 / ms_step,     # the latency metric does not add up over replicas; this does
        "launch_mode": "one CUDA graph replay per step" if graph is not None else "eager C-ABI calls",
        "eager_ms_per_step": ms_eager,
        "clocks": clocks,
        "speedup_vs_own_dense": ms_dense_step / ms_step,
        "own_dense_ms_per_step": ms_dense_step,
        "cold_pooled_keys_ms_per_step": ms_cold,
        "stages": {"dense_layer_ms": dense_ms, "dense_layer_GBps": dense_gbs, "sparse_layer_ms": sparse_ms,
                   "sparse_layer_GBps": sparse_bytes / (sparse_ms * 1e-3) / 1e9,
                   "sparse_layer_frac_of_hbm": sparse_bytes / (sparse_ms * 1e-3) / 1e9 / P["hbm"],
                   "per_layer_sparse_vs_dense": dense_ms / sparse_ms,
                   "timing": "average per launch of a graph holding only those launches" if graph is not None else "CUDA-event marks around eager calls",
                   "dense_layer_eager_marks_ms": dense_eager_ms, "sparse_layer_eager_marks_ms": sparse_eager_ms},
        "roofline": {"bound": "hbm", "achieved": dense_gbs, "peak": P["hbm"], "unit": "GB/s", "frac": dense_gbs / P["hbm"],
                     "traffic": traffic, "kernel": "attn_tc_kernel incl. its in-cluster split merge (dense layer, I_active rows)",
                     "read_only_stream_GBps": stream_gbs, "frac_of_read_only_stream": dense_gbs / stream_gbs,
                     "bytes_per_launch": kv_bytes + qo_bytes, "peak_source": f"{P['src']} copy bandwidth"},
        "sparse_roofline": {"bound": "hbm", "achieved": sparse_bytes / (sparse_ms * 1e-3) / 1e9, "peak": P["hbm"], "unit": "GB/s",
                            "frac": sparse_bytes / (sparse_ms * 1e-3) / 1e9 / P["hbm"],
                            "frac_of_nominal": sparse_bytes / (sparse_ms * 1e-3) / 1e9 / 8000.0,
                            "kernel": "sparse layer, I_active rows: selection kernel + sparse attention kernel on retained K/V "
                                      f"({retained_keys} keys per head)", "bytes_per_launch": sparse_bytes,
                            "peak_source": f"{P['src']} copy bandwidth; nominal 8000"},
        "gen_mode": gen,
        "e2e": {"value": ms_e2e, "unit": "ms", "h2d_bytes_per_step": int(h2d_c), "d2h_bytes_per_step": int(d2h_c),
                "resident": "K/V cache stays in HBM between steps (approximate KV cache, Eq. 3); confidence and masks come "
                            "from pinned host memory; after the indicator the host reads I_focus / I_active back, gathers "
                            "those rows of every layer's Q in pinned memory and uploads only them (chunks of layers, the "
                            "gather of the next chunk overlapping the GPU work of the current one); outputs of the "
                            "I_active rows of every layer and the index sets go back to pinned memory",
                "host_phases": e2e_phases,
                "launch_mode": f"{n_chunks} CUDA graphs of {[bounds[i + 1] - bounds[i] for i in range(n_chunks)]} layers per step + eager indicator call"
                               if chunk_graphs is not None else "eager C-ABI calls"},
        "e2e_all_gen_rows": {"value": ms_e2e_all, "unit": "ms", "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                             "note": "all 512 gen rows of Q of every layer uploaded although only the I_active rows are read "
                                     "(PCIe-bound); layer by layer on a copy stream, outputs back on a third stream"},
        "sustained": sustained,
        "paper_context": "paper reports >29x end-to-end speedup at 32K on H200 (whole model vs no KV cache): context only",
    }
    if cpu:
        out["cpu_baseline"] = cpu
    print(json.dumps(out))


def tensor_roofline(tflops, P, kernel):
    """Roofline object of a tensor-bound launch timed alone: fraction of the measured burst bf16 peak, with the
    sustained and nominal fractions beside it."""
    return {"bound": "tensor", "achieved": tflops, "peak": P["tf_burst"], "unit": "TFLOP/s", "frac": tflops / P["tf_burst"],
            "frac_of_sustained": tflops / P["tf_sust"], "frac_of_nominal": tflops / 2250.0, "kernel": kernel,
            "peak_source": f"{P['src']} burst bf16 (cuBLAS 8192^3); sustained {P['tf_sust']}, nominal 2250"}


def graph_time_us(fn, n_layers, warm=10, reps=50):
    """Per-call latency in microseconds of fn(l), l = 0..n_layers-1 (rotating layer copies, so that the inputs of a
    call are not in L2 from the call before), replayed as one CUDA graph: `warm` untimed replays, then `reps` replays
    timed one by one with CUDA events; the median replay divided by the calls per replay."""
    import torch
    for l in range(n_layers):
        fn(l)
    torch.cuda.synchronize()
    gr = torch.cuda.CUDAGraph()
    with torch.cuda.graph(gr):
        for l in range(n_layers):
            fn(l)
    torch.cuda.synchronize()
    time.sleep(0.3)                                  # start from an idle part (see `timed` in run_focus)
    for _ in range(warm):
        gr.replay()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for a, z in evs:
        a.record(); gr.replay(); z.record()
    torch.cuda.synchronize()
    return statistics.median(a.elapsed_time(z) for a, z in evs) / n_layers * 1e3


def run_sweep(args):
    """Config 4: one attention layer, 32 heads, d 128, bf16, gen 256; context x keep ratio.  Per point: latency of
    the sparse layer (selection + attention) and of the attention call alone, for the gen-region rows (256) and for
    the paper's I_active rows, retained-FLOP TFLOP/s, HBM GB/s, and the ratio to the own dense attention."""
    import torch

    from paper_2602_02159_b200 import binding as fb
    from paper_2602_02159_b200 import build as fbuild
    from paper_2602_02159_b200 import step as fstep
    from paper_2602_02159_b200 import workloads as wl
    fbuild.build()
    torch.cuda.set_device(0)
    ctx = fb.Context(0, workspace_bytes=1 << 30)
    P = peaks()
    out = []
    for L in wl.SWEEP_L:
        w0 = wl.config(4, L=L, keep_den=1)
        s = w0.shape
        layer_bytes = 2 * s.Hkv * s.L * s.d * 2
        NL = max(2, min(8, -(-400_000_000 // layer_bytes)))          # rotate layers: > 3x L2 in total
        g = torch.Generator(device="cuda").manual_seed(L)
        mk = lambda *sh: (torch.randn(*sh, device="cuda", generator=g) / s.d ** 0.5).to(torch.bfloat16)
        Qs = [mk(s.N, s.H, s.d) for _ in range(NL)]
        Ks = [mk(s.Hkv, s.L, s.d) for _ in range(NL)]
        Vs = [mk(s.Hkv, s.L, s.d) for _ in range(NL)]
        c_prev, _ = wl.gen_confidence(0, s.N)
        conf = torch.from_numpy(wl.full_conf(s, c_prev)).cuda()
        masked = torch.from_numpy(wl.gen_masked(w0)).cuda()

        def graph_time(fn):
            return graph_time_us(fn, NL)

        for rows in ("gen", "active"):
            dense_us = None
            for den in wl.SWEEP_KEEP_DEN:
                w = wl.config(4, L=L, keep_den=den)
                b = fstep.StepBuffers(w, rows=rows)
                fstep.select_queries(ctx, b, conf, masked)
                ba = fstep.StepBuffers(w, rows="active")
                fstep.select_queries(ctx, ba, conf, masked)
                fstep.dense_layer(ctx, ba, Qs[0], Ks[0], Vs[0])
                fstep.find_sinks(ctx, ba, Qs[0], Ks[0], ba.lse)
                b.sink_idx.copy_(ba.sink_idx)
                Kb = []
                for l in range(NL):
                    kb = torch.zeros(s.Hkv, s.nb, s.d, dtype=torch.float32, device="cuda")
                    fb.focus_pool_keys(ctx, b.shape, Ks[l], kb)
                    Kb.append(kb)
                if dense_us is None:
                    dense_us = graph_time(lambda l: fstep.dense_layer(ctx, b, Qs[l], Ks[l], Vs[l]))
                layer_us = graph_time(lambda l: fstep.sparse_layer(ctx, b, Qs[l], Ks[l], Vs[l], Kbar=Kb[l]))
                q_rows, n_rows, max_rows = b._rows()
                attn_us = graph_time(lambda l: fb.focus_sparse_attn(
                    ctx, b.shape, Qs[l], s.M, s.N, q_rows, n_rows, max_rows, Ks[l], Vs[l], fb.HEADS_PER_KV_GROUP,
                    b.block_idx, b.max_blocks, b.block_cnt, b.sink_idx, b.sink_keep, w.n_sink, b.O, b.lse))
                n_q = s.N if rows == "gen" else int(b.n_active.item())
                keys = w.C * s.B + w.n_sink + s.N
                flops = 4.0 * n_q * keys * s.d * s.H
                byts = 2.0 * s.Hkv * keys * s.d * 2 + 2.0 * n_q * s.H * s.d * 2
                tf, gbs = flops / attn_us / 1e6, byts / attn_us / 1e3
                out.append({"L": L, "rows": rows, "n_q": n_q, "keep": f"1/{den}", "blocks": w.C, "retained_keys": keys,
                            "sparse_layer_us": round(layer_us, 2), "sparse_attn_us": round(attn_us, 2),
                            "dense_attn_us": round(dense_us, 2), "attn_vs_dense": round(dense_us / attn_us, 2),
                            "retained_TFLOPs": round(tf, 1), "frac_tensor_sustained": round(tf / P["tf_sust"], 3),
                            "dense_equiv_TFLOPs": round(4.0 * n_q * s.L * s.d * s.H / attn_us / 1e6, 1),
                            "GBps": round(gbs, 1), "frac_hbm": round(gbs / P["hbm"], 3)})
                assert ctx.poll_status() == 0
        del Qs, Ks, Vs
        torch.cuda.empty_cache()
    print(json.dumps({"sweep": out, "peaks": P,
                      "timing": "median of 50 CUDA-graph replays after 10 warm-up replays, per call"}))


def run_stages(args):
    """Per-stage latency of one configuration (graph replay over a few rotating layer copies so that inputs do not
    sit in L2), for the paper's I_active rows and for the gen-region rows."""
    import torch

    from paper_2602_02159_b200 import binding as fb
    from paper_2602_02159_b200 import build as fbuild
    from paper_2602_02159_b200 import step as fstep
    from paper_2602_02159_b200 import workloads as wl
    fbuild.build()
    torch.cuda.set_device(0)
    ctx = fb.Context(0, workspace_bytes=512 << 20)
    P = peaks()
    w = wl.config(args.config)
    s = w.shape
    eb = 4 if s.dtype == "f32" else 2
    layer_bytes = 2 * s.Hkv * s.L * s.d * eb
    NL = max(2, min(8, -(-400_000_000 // layer_bytes)))
    Qs, Ks, Vs, Kb = [], [], [], []
    for l in range(NL):
        t = wl.gen_qkv(s, l)
        Qs.append(fstep.to_device(t["Q"], s.dtype)); Ks.append(fstep.to_device(t["K"], s.dtype))
        Vs.append(fstep.to_device(t["V"], s.dtype))
    c_prev, _ = wl.gen_confidence(w.seed, s.N)
    conf = torch.from_numpy(wl.full_conf(s, c_prev)).cuda()
    masked = torch.from_numpy(wl.gen_masked(w)).cuda()
    ba = fstep.StepBuffers(w, rows="active")
    bg = fstep.StepBuffers(w, rows="gen")
    for b in (ba, bg):
        fstep.select_queries(ctx, b, conf, masked)
    for l in range(NL):
        kb = torch.zeros(s.Hkv, s.nb, s.d, dtype=torch.float32, device="cuda")
        fb.focus_pool_keys(ctx, ba.shape, Ks[l], kb)
        Kb.append(kb)
    fstep.dense_layer(ctx, ba, Qs[0], Ks[0], Vs[0])
    fstep.find_sinks(ctx, ba, Qs[0], Ks[0], ba.lse)
    bg.sink_idx.copy_(ba.sink_idx)
    lse_keep = ba.lse.clone()
    torch.cuda.synchronize()

    def graph_time(fn):
        return round(graph_time_us(fn, NL), 2)

    na = int(ba.n_active.item())
    keys = w.C * s.B + w.n_sink + s.N
    out = {"workload": w.name, "n_active": na, "retained_keys_per_head": keys, "layers_rotated": NL,
           "timing": "median of 50 CUDA-graph replays after 10 warm-up replays, per call", "us": {}}
    u = out["us"]
    u["select_queries"] = graph_time(lambda l: fstep.select_queries(ctx, ba, conf, masked))
    u["find_sinks (with LSE of the dense pass)"] = graph_time(lambda l: fstep.find_sinks(ctx, ba, Qs[l], Ks[l], lse_keep))
    u["pool_keys"] = graph_time(lambda l: fb.focus_pool_keys(ctx, ba.shape, Ks[l], Kb[l]))
    u["score_blocks cold (streams K)"] = graph_time(lambda l: fb.focus_score_blocks(
        ctx, ba.shape, Qs[l], s.M, ba.focus_idx, ba.n_focus, max(1, w.k), Ks[l], None, 0, ba.R))
    # loop-closing stages: confidence from logits (LLaDA vocabulary, bf16) for the I_active rows, KV refresh of those rows
    V = 126464
    logits = (torch.randn(s.N, V, device="cuda") * 2).to(torch.bfloat16)
    cconf = torch.zeros(ba.max_active, dtype=torch.float32, device="cuda")
    ctok = torch.zeros(ba.max_active, dtype=torch.int32, device="cuda")
    t_conf = graph_time(lambda l: fb.focus_confidence(ctx, logits, fb.BF16, V, V, s.M, s.N, ba.active_idx, ba.n_active,
                                                      ba.max_active, cconf, ctok))
    u["confidence (Eq. 2), I_active rows x 126464 vocab"] = {"us": t_conf, "GBps": round(na * V * 2 / t_conf / 1e3, 1)}
    del logits
    if s.dtype == "bf16":
        Kn = torch.randn(ba.max_active, s.Hkv, s.d, device="cuda").to(torch.bfloat16)
        u["update_kv (Eq. 3), I_active rows"] = graph_time(lambda l: fb.focus_update_kv(
            ctx, ba.shape, Ks[l], Vs[l], Kn, Kn, ba.active_idx, ba.n_active, ba.max_active))
        # a block-entry style refresh of 64 prompt rows spread over the prompt, then the pooled keys of their blocks
        prow = torch.arange(0, s.M, max(1, s.M // 64), dtype=torch.int32, device="cuda")[:64].contiguous()
        pn = torch.tensor([prow.numel()], dtype=torch.int32, device="cuda")
        u["update_pooled_keys (64 refreshed prompt rows)"] = graph_time(lambda l: fb.focus_update_pooled_keys(
            ctx, ba.shape, Ks[l], Kb[l], prow, pn, prow.numel()))
    # the state update that ends a step: new confidences of the I_active rows in, two positions unmasked
    st_conf, st_masked = conf.clone(), masked.clone()
    st_x = torch.zeros(s.L, dtype=torch.int32, device="cuda")
    picked = torch.zeros(2, dtype=torch.int32, device="cuda"); n_picked = torch.zeros(1, dtype=torch.int32, device="cuda")
    u["commit_step (end of a step, I_active rows, 2 unmasked)"] = graph_time(lambda l: fb.focus_commit_step(
        ctx, cconf, ctok, s.M, ba.active_idx, ba.n_active, ba.max_active, s.L, w.blk_lo, w.blk_hi, 2, st_conf, st_masked,
        st_x, picked, n_picked))
    for name, b in (("I_active rows", ba), ("gen rows", bg)):
        q_rows, n_rows, max_rows = b._rows()
        n_q = na if b is ba else s.N
        d_us = graph_time(lambda l: fstep.dense_layer(ctx, b, Qs[l], Ks[l], Vs[l]))
        l_us = graph_time(lambda l: fstep.sparse_layer(ctx, b, Qs[l], Ks[l], Vs[l], Kbar=Kb[l]))
        a_us = graph_time(lambda l: fb.focus_sparse_attn(
            ctx, b.shape, Qs[l], s.M, s.N, q_rows, n_rows, max_rows, Ks[l], Vs[l], fb.HEADS_PER_KV_GROUP, b.block_idx,
            b.max_blocks, b.block_cnt, b.sink_idx, b.sink_keep, w.n_sink, b.O, b.lse))
        fl_d, fl_s = 4.0 * n_q * s.L * s.d * s.H, 4.0 * n_q * keys * s.d * s.H
        by_d = 2.0 * s.Hkv * s.L * s.d * eb
        by_s = 2.0 * s.Hkv * keys * s.d * eb
        u[name] = {"n_q": n_q, "dense_attn": d_us, "sparse_layer (score+select+attn)": l_us, "sparse_attn": a_us,
                   "dense_TFLOPs": round(fl_d / d_us / 1e6, 1), "dense_GBps": round(by_d / d_us / 1e3, 1),
                   "sparse_retained_TFLOPs": round(fl_s / a_us / 1e6, 1), "sparse_GBps": round(by_s / a_us / 1e3, 1),
                   "sparse_attn_vs_dense": round(d_us / a_us, 2)}
    assert ctx.poll_status() == 0
    out["peaks"] = P
    print(json.dumps(out))


def spawn_ranks(n, argv):
    """`bench.py --gpus N` started as a plain process: start the N ranks here (one per GPU, rendezvous on 127.0.0.1)
    the way an outer launcher would have, and hand their exit code back."""
    import socket
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        port = so.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]
    return subprocess.call(cmd)


def run_stub(args):
    """Host-only stand-in for the step (no GPU, gloo): exercises the launcher, the rendezvous, the barrier and the
    max-over-ranks timing that the real arm uses, and prints a line of the same outer shape."""
    from paper_2602_02159_b200 import replicas
    rank, world, _ = replicas.init("gloo")
    replicas.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(0.001 * (1 + rank))                 # rank r takes r + 1 ms per step: the slowest rank sets the time
    ms = replicas.max_over_ranks((time.perf_counter() - t0) * 1e3) / max(1, args.steps)
    replicas.barrier()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": ms, "unit": "ms", "n_gpus": world, "steps": args.steps,
                          "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": False, "scaling": "weak",
                          "stub": True}))
    replicas.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="focus", choices=["focus", "reference"])
    ap.add_argument("--config", type=int, default=2,
                    help="workload: 2 = the headline 32-layer step; 5 = the paper's own hyper-parameters on that shape")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (quick runs)")
    ap.add_argument("--skip-gen", action="store_true", help="skip the gen-region-rows (tensor-bound) measurements")
    ap.add_argument("--no-graph", action="store_true", help="time eager C-ABI calls instead of a CUDA graph replay")
    ap.add_argument("--stages", action="store_true", help="per-stage latencies of --config (0..3) instead of the step")
    ap.add_argument("--sweep", action="store_true", help="run the context x keep-ratio sweep (config 4) instead")
    ap.add_argument("--clock-interval-ms", type=int, default=25, help="nvidia-smi sampling period during timed regions")
    ap.add_argument("--skip-cpu", action="store_true", help="skip the CPU oracle baseline leg")
    ap.add_argument("--sustain-s", type=float, default=2.0,
                    help="seconds of back-to-back graph replays for the sustained figure (0 = skip)")
    ap.add_argument("--cooldown-s", type=float, default=0.5, help="idle time before each timed region")
    ap.add_argument("--stub-step", action="store_true", help=argparse.SUPPRESS)   # host-only step: tests of the launcher
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not (args.stages or args.sweep):
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    if args.stub_step:
        run_stub(args)
    elif args.stages:
        run_stages(args)
    elif args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_focus(args)


if __name__ == "__main__":
    main()
