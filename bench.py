#!/usr/bin/env python
"""Benchmark of the selection hot path: selection tokens*layers/s on one B200 (or N replicas).

A "step" is one pass of the whole path over one synthetic batch: full selection
(Definition 1) at layer 0, then one cascade step (Algorithm 1) at each of the
layers 1..L-1, every layer's X a distinct HBM-resident tensor.  The same layers
are also pushed through full selection at every layer ("independent" selection)
to report the cascade speedup.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..4] [--impl reference]

Prints ONE JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle
on the host cores instead (a deliberately plain program: a reported baseline).
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_03110_b200 import workloads as wl  # noqa: E402

METRIC = "selection tokens*layers/s (full at layer 0 + cascade at layers 1..L-1)"
UNIT = "tokens*layers/s"

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per launch of the dominant kernel.
# These are NOT measured by this program: they are the figures of earlier `ncu` captures of the
# same kernel on the same workload (one launch each), printed as `traffic_static` with their
# origin beside them.  Keyed by (kernel, workload).
NCU_TRAFFIC_BYTES = {
    # cascade launch on configs[3]: mean of the captured layers 1 (77.2 MB) and 30 (104.3 MB)
    ("gram_tc_cascade", 4): 90.75e6,
    # fused cascade launches of layers 1-2 on the smaller workloads
    ("gram_tc_cascade", 1): 9.53e6,
    ("gram_tc_cascade", 2): 28.9e6,
    ("gram_tc_cascade", 3): 21.08e6,
}
NCU_TRAFFIC_SOURCE = ("static: mean DRAM read+write bytes per launch from earlier ncu captures of this "
                      "kernel on this workload (summaries under profiles/), not measured in this run")


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            m = json.load(f)
        return dict(hbm_gbs=m["hbm_gbs"], bf16_burst=m["bf16_tflops"],
                    bf16_sustained=m.get("bf16_tflops_sustained", m["bf16_tflops"]), src="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, src="fallback")


# ------------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, device_index: int):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.h = None

    def run(self):
        if self.h is None:
            return
        while not self._stop_evt.is_set():
            try:
                self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                bits = self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop_evt.wait(0.01)

    def finish(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def jaccard(a, b):
    a, b = set(a), set(b)
    return 1.0 if not (a or b) else len(a & b) / len(a | b)


# ------------------------------------------------------------------------------------------
def reference_arm(args, cfg):
    """The fp64 CPU oracle on the host cores, same metric, bounded sample per step."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_lay = min(cfg.L, args.ref_layers)
    layers = [lb.X for lb in wl.generate_layers(cfg, seed=0, n_layers=n_lay)]
    X64 = [[wl.as_f64(X[b]) for b in range(cfg.B)] for X in layers]

    def one_step():
        t0 = time.perf_counter()
        R = [oracle.select_full(X64[0][b], cfg.tau)[0] for b in range(cfg.B)]
        t_full = time.perf_counter() - t0
        t_c = []
        for l in range(1, n_lay):
            t1 = time.perf_counter()
            R = [oracle.cascade_step(X64[l][b], cfg.tau, R[b]).rep for b in range(cfg.B)]
            t_c.append(time.perf_counter() - t1)
        return t_full, (float(np.mean(t_c)) if t_c else t_full)

    for _ in range(args.ref_warmup):
        one_step()
    est, wall = [], []
    for _ in range(args.steps):
        t0 = time.perf_counter()
        t_full, t_casc = one_step()
        wall.append(time.perf_counter() - t0)
        est.append(t_full + (cfg.L - 1) * t_casc)      # scaled to the L-layer pipeline
    t_step = float(np.mean(est))
    value = cfg.B * cfg.T * cfg.L / t_step
    sample = (f"layers 0..{n_lay - 1} of workload {cfg.cfg_id} computed in full by the oracle; "
              f"step time = t(full, layer 0) + {cfg.L - 1} x mean t(cascade step)")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.ref_warmup, "ms_per_step": 1e3 * t_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_dict(cfg),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
        # ms_per_step is NOT the wall time of a step of this run: only `layers_computed` of the L
        # layers are computed, the rest is scaled from the mean cascade step (a lower bound of the
        # oracle's cost where the representative set grows over the layers)
        "extrapolated": n_lay < cfg.L, "layers_computed": n_lay, "layers": cfg.L,
        "wall_s_per_step": float(np.mean(wall)),
    }
    print(json.dumps(line))


L2_BYTES = 126e6


def step_bytes(cfg):
    return cfg.L * cfg.B * cfg.T * cfg.d * cfg.es


def workload_dict(cfg):
    mib = step_bytes(cfg) / 2**20
    if step_bytes(cfg) > L2_BYTES:
        l2 = f"every layer is a distinct HBM-resident tensor; one step streams {mib:.0f} MiB (> 126 MB L2)"
    else:
        l2 = (f"one step reads only {mib:.0f} MiB (< 126 MB L2): L2 is flushed by a 256 MiB write before "
              "every timed step, each step is bracketed by its own CUDA events, the flush is outside them")
    return {"workload": f"configs[{cfg.cfg_id - 1}] {cfg.name}", "B": cfg.B, "T": cfg.T, "d": cfg.d,
            "L": cfg.L, "tau": cfg.tau, "prototypes": cfg.P, "storage": cfg.dtype, "l2": l2, "seed": 0}


# ------------------------------------------------------------------------------------------
def sweep(args):
    """configs[4]: d = 4096, bf16, one layer transition X1 = X0 + 0.02 N(0, I); full selection on
    X1 against one cascade step on X1 from R(X0), per T and r/T.  Times are CUDA-event means over
    graph replays of ten calls each, with a 256 MiB write before every call so that it starts with a
    cold L2; the time of the writes alone is measured the same way and subtracted."""
    import torch
    from paper_2605_03110_b200 import binding as ada
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    peaks = measured_peaks()
    steps = max(5, min(args.steps, 20))

    reps = 10
    side = torch.cuda.Stream()

    def graph_of(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for _ in range(reps):
                    flush.zero_()
                    fn(side)
        return g

    def time_graph(g):
        for _ in range(2):
            g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / (steps * reps)         # microseconds per call + flush

    t_flush = time_graph(graph_of(lambda st: None))

    def timed_call(fn):
        fn(None)                                                   # first-call set-up outside capture
        torch.cuda.synchronize()
        return time_graph(graph_of(fn)) - t_flush

    print("| T | r/T | r | full us | cascade us | speedup | T/r (paper) | 1/(2q-q^2) | full TFLOP/s | "
          "cascade: X once GB/s | cascade TFLOP/s |")
    print("|---|---|---|---|---|---|---|---|---|---|---|")
    for T in wl.SWEEP_T:
        ctx = ada.ada_create(1, T, 4096, ada.ADA_BF16)
        ada.ada_set_engine(ctx, args.engine)
        for q in wl.SWEEP_Q:
            cfg = wl.sweep_config(T, q)
            X0, X1 = [torch.from_numpy(lb.X.view(np.int16)).view(torch.bfloat16).to(dev)
                      for lb in wl.generate_layers(cfg, seed=0)]
            idx, cnt, _ = ada.ada_select_full(ctx, X0, cfg.tau, want_gamma=False)
            r = int(cnt[0])
            i2 = torch.empty_like(idx)
            c2 = torch.empty_like(cnt)
            out = ada.CascadeOut(1, T, dev, want_gamma=False)
            t_full = timed_call(lambda st: ada.ada_select_full(ctx, X1, cfg.tau, i2, c2, want_gamma=False,
                                                               stream=st))
            t_casc = timed_call(lambda st: ada.ada_cascade_step(ctx, X1, cfg.tau, idx, cnt, out=out,
                                                                stream=st))
            d = 4096
            f_full = d * T * (T - 1.0)
            f_casc = d * r * (r - 1.0) + 2.0 * d * (T - r) * r
            qq = r / T
            print(f"| {T} | {q:g} | {r} | {t_full:.1f} | {t_casc:.1f} | {t_full / t_casc:.2f} | "
                  f"{T / r:.1f} | {1.0 / (2 * qq - qq * qq):.2f} | {f_full / t_full / 1e6:.0f} | "
                  f"{T * d * 2 / t_casc / 1e3:.0f} | {f_casc / t_casc / 1e6:.0f} |")
            sys.stdout.flush()
        ada.ada_destroy(ctx)
    print(f"peaks ({peaks['src']}): HBM {peaks['hbm_gbs']} GB/s, bf16 {peaks['bf16_burst']} TFLOP/s burst / "
          f"{peaks['bf16_sustained']} sustained")


def hbm_point(ada, dev, T, q, peaks, args):
    """One HBM-bound point of the crossover sweep (d = 4096, bf16, few representatives): the
    cascade step on X1 from R(X0).  Reports the fused Gram launch (CUDA events around the launch,
    L2 flushed by a 256 MiB write before every call) and the whole ada_cascade_step call (graph
    replays of [flush, call], the flush-only graph subtracted) against the copy bandwidth, with
    T*d*2 bytes (every row of X once) as the algorithmic traffic."""
    import torch
    cfg = wl.sweep_config(T, q)
    X0, X1 = [torch.from_numpy(lb.X.view(np.int16)).view(torch.bfloat16).to(dev)
              for lb in wl.generate_layers(cfg, seed=0)]
    ctx = ada.ada_create(1, T, cfg.d, ada.ADA_BF16, device=dev.index or 0)
    if args.no_cooperative:
        ada.ada_set_cooperative(ctx, False)
    idx, cnt, _ = ada.ada_select_full(ctx, X0, cfg.tau, want_gamma=False)
    out = ada.CascadeOut(1, T, dev, want_gamma=False)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    ada.ada_cascade_step(ctx, X1, cfg.tau, idx, cnt, out=out)          # first-call set-up
    torch.cuda.synchronize()
    r = int(cnt[0])
    n = 10
    ada.ada_profile_enable(ctx, True)
    for _ in range(n):
        flush.zero_()
        ada.ada_cascade_step(ctx, X1, cfg.tau, idx, cnt, out=out)
    torch.cuda.synchronize()
    prof = {k: v for k, v in ada.ada_profile_read(ctx).items() if v[0]}
    ada.ada_profile_enable(ctx, False)
    k_gram = max(prof, key=lambda k: prof[k][1])
    us_launch = prof[k_gram][1] * 1e3 / prof[k_gram][0]
    # whole call, from graph replays
    side = torch.cuda.Stream()

    def graph_of(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for _ in range(n):
                    flush.zero_()
                    fn(side)
        return g

    def time_graph(g):
        for _ in range(2):
            g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(5):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / (5 * n)

    us_flush = time_graph(graph_of(lambda st: None))
    us_call = time_graph(graph_of(lambda st: ada.ada_cascade_step(ctx, X1, cfg.tau, idx, cnt, out=out,
                                                                  stream=st))) - us_flush
    st_, _ = ada.ada_device_status(ctx)
    assert st_ == 0
    ada.ada_destroy(ctx)
    nbytes = T * cfg.d * 2
    gbs_launch, gbs_call = nbytes / us_launch / 1e3, nbytes / us_call / 1e3
    return {"workload": f"configs[4] sweep point T={T}, r/T={q:g} (r={r}), d={cfg.d}, bf16", "kernel": k_gram,
            "bound": "hbm", "algorithmic_bytes_per_launch": nbytes, "kernels_per_call": {k: v[0] // n for k, v in prof.items()},
            "launch_us": us_launch, "achieved": gbs_launch, "unit": "GB/s", "peak": peaks["hbm_gbs"],
            "frac": gbs_launch / peaks["hbm_gbs"], "peak_source": f"copy bandwidth, {peaks['src']}",
            "whole_call_us": us_call, "whole_call_gbs": gbs_call, "whole_call_frac": gbs_call / peaks["hbm_gbs"],
            "l2": "256 MiB write before every call"}


def overlap_bench(args, cfg):
    """Section 8.4: the selection of layer l+1 on one stream while the nearest-representative map
    and the attention on the representatives (Eq. 2) of layer l run on another.  The layers of
    `cfg` stand in for Q, K, V (h heads of d/h); serial order on one stream against the two-stream
    order, CUDA events around the whole chain, inputs resident in HBM.  Prints a table."""
    import torch
    from paper_2605_03110_b200 import binding as ada
    from paper_2605_03110_b200.pipeline import SelectionAttentionPipeline
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    h = args.heads or 32
    T, d, L = cfg.T, cfg.d, cfg.L
    d_h = d // h
    layers = [torch.from_numpy(lb.X[0].view(np.int16)).view(torch.bfloat16).to(dev).view(T, h, d_h)
              for lb in wl.generate_layers(cfg, seed=0)]
    outs = [torch.zeros((T, h, d_h), dtype=torch.float32, device=dev) for _ in range(2)]
    pipe = SelectionAttentionPipeline(T, h, d_h, cfg.tau, dev)
    out_of = lambda l: outs[l & 1]

    def timed(fn):
        for _ in range(max(2, args.warmup)):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.steps

    st = torch.cuda.current_stream()

    def selection_only():
        for l in range(L):
            pipe._select(l, layers[l], st)

    def consumers_only():
        for l in range(L):
            pipe._consume(l, layers[l], out_of(l), st)

    ms_sel = timed(selection_only)
    ms_con = timed(consumers_only)            # on the sets the last selection pass left behind
    ms_serial = timed(lambda: pipe.run(layers, [out_of(l) for l in range(L)], overlap=False))
    ms_over = timed(lambda: pipe.run(layers, [out_of(l) for l in range(L)], overlap=True))
    r_last = int(pipe.sets[(L - 1) % len(pipe.sets)].rep_out_cnt[0])
    # the attention call alone, on the last layer's set (gather + Eq. 2 + expansion)
    last = pipe.sets[(L - 1) % len(pipe.sets)]
    X = layers[L - 1]
    ms_att = timed(lambda: ada.ada_attention_reps(pipe.con, X, X, X, last.rep_out[0], last.rep_out_cnt,
                                                  nearest_idx=pipe.near[0], out=outs[0]))
    ms_att_reps = timed(lambda: ada.ada_attention_reps(pipe.con, X, X, X, last.rep_out[0], last.rep_out_cnt,
                                                       out=outs[0]))
    assert ada.ada_device_status(pipe.sel)[0] == 0 and ada.ada_device_status(pipe.con)[0] == 0
    pipe.close()
    print(f"workload configs[{cfg.cfg_id - 1}] {cfg.name}: T={T} d={d} L={L}, {h} heads of {d_h}; r at the last "
          f"layer {r_last}; {args.steps} eager passes per figure (launches from Python)")
    print("| chain | ms per L layers |")
    print("|---|---|")
    print(f"| selection alone (full + {L - 1} cascade steps) | {ms_sel:.3f} |")
    print(f"| consumers alone (nearest-representative map + attention on the representatives, {L} layers) | {ms_con:.3f} |")
    print(f"| both, one stream | {ms_serial:.3f} |")
    print(f"| both, two streams (selection of layer l+1 beside the consumers of layer l) | {ms_over:.3f} |")
    gf = 2 * 2.0 * r_last * r_last * d_h * h / 1e9
    print(f"attention on the representatives alone, r = {r_last}: {ms_att_reps * 1e3:.1f} us without the expansion "
          f"({gf:.1f} GFLOP in the two contractions of Eq. 2 -> {gf / ms_att_reps:.0f} TFLOP/s), "
          f"{ms_att * 1e3:.1f} us with it ({T * d * 4 / 1e6:.0f} MB of fp32 output rows)")


def heads_bench(args, cfg):
    """Per-head selection (Section 8.5) on the layers of `cfg` read as (T, h, d/h): the whole
    L-layer cascade pipeline with one representative set per head, beside the shared-set pipeline
    on the same tensors.  CUDA-graph replay of one step, CUDA events, inputs resident in HBM.
    Prints a table instead of the JSON line."""
    import torch
    from paper_2605_03110_b200 import binding as ada
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    h = args.heads
    assert cfg.B == 1 and cfg.dtype == "bf16" and cfg.d % h == 0
    T, d, L, d_h = cfg.T, cfg.d, cfg.L, cfg.d // h
    layers = [torch.from_numpy(lb.X[0].view(np.int16)).view(torch.bfloat16).to(dev)
              for lb in wl.generate_layers(cfg, seed=0)]
    side = torch.cuda.Stream()
    peaks = measured_peaks()

    def pipeline(kind):
        nb = h if kind == "heads" else 1
        ctx = ada.ada_create(nb, T, d_h if kind == "heads" else d, ada.ADA_BF16)
        outs = [ada.CascadeOut(nb, T, dev, want_gamma=False) for _ in range(2)]
        view = (lambda X: X.view(T, h, d_h)) if kind == "heads" else (lambda X: X.view(1, T, d))
        full = ada.ada_select_full_heads if kind == "heads" else ada.ada_select_full
        step = ada.ada_cascade_step_heads if kind == "heads" else ada.ada_cascade_step

        def run(st, n_layers=L):
            full(ctx, view(layers[0]), cfg.tau, outs[0].rep_out, outs[0].rep_out_cnt, want_gamma=False,
                 stream=st)
            cur = 0
            for l in range(1, n_layers):
                step(ctx, view(layers[l]), cfg.tau, outs[cur].rep_out, outs[cur].rep_out_cnt,
                     out=outs[1 - cur], stream=st)
                cur = 1 - cur
            return outs[cur]

        def graph_time(fn):
            fn(None)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    fn(side)
            for _ in range(max(3, args.warmup)):
                g.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(args.steps):
                g.replay()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / args.steps

        ms_pipe = graph_time(run)
        ms_full = graph_time(lambda st: run(st, 1))
        last = run(None)
        torch.cuda.synchronize()
        r = last.rep_out_cnt.cpu().numpy()
        st_, _ = ada.ada_device_status(ctx)
        assert st_ == 0
        ada.ada_destroy(ctx)
        return ms_pipe, ms_full, r

    rows = []
    for kind in ("shared", "heads"):
        ms_pipe, ms_full, r = pipeline(kind)
        ms_step = (ms_pipe - ms_full) / (L - 1)
        rows.append((kind, ms_pipe, ms_full, ms_step, r))
    x_bytes = T * d * 2
    print(f"workload configs[{cfg.cfg_id - 1}] {cfg.name}: T={T} d={d} L={L} bf16, heads h={h} d_h={d_h}; "
          f"{args.steps} graph replays after {max(3, args.warmup)} warm-up")
    print("| sets | step (L layers) ms | tokens*layers/s | full selection us | cascade step us | "
          "cascade step: X once GB/s | r at the last layer |")
    print("|---|---|---|---|---|---|---|")
    for kind, ms_pipe, ms_full, ms_step, r in rows:
        rr = f"{int(r[0])}" if kind == "shared" else f"{int(r.min())}..{int(r.max())} (mean {r.mean():.0f})"
        print(f"| {'one per head' if kind == 'heads' else 'one shared'} | {ms_pipe:.3f} | "
              f"{T * L / (ms_pipe * 1e-3):.3e} | {ms_full * 1e3:.1f} | {ms_step * 1e3:.1f} | "
              f"{x_bytes / (ms_step * 1e-3) / 1e9:.0f} | {rr} |")
    print(f"peaks ({peaks['src']}): HBM {peaks['hbm_gbs']} GB/s")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=4, choices=[1, 2, 3, 4])
    ap.add_argument("--layers", type=int, default=0, help="override L (0 = the configuration's)")
    ap.add_argument("--engine", type=int, default=0,
                    help="0 auto, 1 force the FFMA Gram, 2 the one-CTA tcgen05 kernel, 3 the pair-CTA one")
    ap.add_argument("--ref-layers", type=int, default=4)
    ap.add_argument("--ref-warmup", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sustained", action="store_true", help="skip the >= 1 s replay loop")
    ap.add_argument("--no-hbm-points", action="store_true",
                    help="skip the two HBM-bound cross-Gram points (sweep, r/T = 0.01)")
    ap.add_argument("--sweep", action="store_true",
                    help="crossover sweep (configs[4]): full selection vs one cascade step per (T, r/T); "
                         "prints a table instead of the JSON line")
    ap.add_argument("--hbm-only", action="store_true",
                    help="only the two HBM-bound cross-Gram points (one JSON line each)")
    ap.add_argument("--overlap", action="store_true",
                    help="selection / attention pipelining on two streams (Section 8.4) on --workload 3 or 4 "
                         "(--heads h, default 32); prints a table instead of the JSON line")
    ap.add_argument("--causal", action="store_true",
                    help="cascade steps with ADA_CROSS_CAUSAL (line 8 restricted to s < t)")
    ap.add_argument("--no-cooperative", action="store_true",
                    help="launch the fused cascade kernel as an ordinary grid (for profilers)")
    ap.add_argument("--no-dep-launch", action="store_true",
                    help="launch the kernels without programmatic stream serialization")
    ap.add_argument("--no-graph", action="store_true",
                    help="launch every call from Python instead of replaying a CUDA graph of one step")
    ap.add_argument("--heads", type=int, default=0,
                    help="per-head selection (one set per head, d_h = d / HEADS) beside the shared-set "
                         "pipeline on --workload 3 or 4; prints a table instead of the JSON line")
    args = ap.parse_args()

    if args.hbm_only:
        import torch
        from paper_2605_03110_b200 import binding as ada
        torch.cuda.set_device(0)
        for Tq in (16384, 8192):
            print(json.dumps(hbm_point(ada, torch.device("cuda", 0), Tq, 0.01, measured_peaks(), args)))
        return
    if args.overlap:
        cfg = wl.CONFIGS[args.workload]
        overlap_bench(args, wl.scaled(cfg, L=args.layers) if args.layers else cfg)
        return
    if args.heads:
        cfg = wl.CONFIGS[args.workload]
        heads_bench(args, wl.scaled(cfg, L=args.layers) if args.layers else cfg)
        return
    if args.sweep:
        sweep(args)
        return
    cfg = wl.CONFIGS[args.workload]
    if args.layers:
        cfg = wl.scaled(cfg, L=args.layers)
    if args.impl == "reference":
        reference_arm(args, cfg)
        return

    import torch
    import torch.distributed as dist
    from paper_2605_03110_b200 import binding as ada
    from paper_2605_03110_b200 import replicas

    rep = replicas.from_env()
    rank, world, local = rep.rank, rep.world, rep.local_rank
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    replicas.init_process_group(rep, "nccl", dev)
    ada.lib()                                                   # fail loudly if not built

    # ---- inputs: every rank draws its own replica (weak scaling, no data-path collective) ----
    # Host copies live in pinned memory (they feed the end-to-end leg); plain numpy copies are
    # kept only for the few layers the CPU-baseline leg recomputes.
    want_e2e = not args.no_e2e
    want_cpu = rep.rank == 0 and rep.world == 1 and not args.no_cpu_baseline
    host_layers, pin, dev_layers = [], [], []
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32

    def as_torch(X):
        if X.dtype == np.uint16:
            return torch.from_numpy(X.view(np.int16)).view(torch.bfloat16)
        return torch.from_numpy(X)

    for lb in wl.generate_layers(cfg, seed=rep.seed):
        t = as_torch(lb.X)
        if want_e2e:
            t = t.pin_memory()
            pin.append(t)
        dev_layers.append(t.to(dev))
        if want_cpu and lb.layer < args.ref_layers:
            host_layers.append(lb.X)
    B, T, d, L = cfg.B, cfg.T, cfg.d, cfg.L
    ctx = ada.ada_create(B, T, d, ada.ADA_BF16 if cfg.dtype == "bf16" else ada.ADA_F32, device=local)
    ada.ada_set_engine(ctx, args.engine)
    if args.no_cooperative:
        ada.ada_set_cooperative(ctx, False)
    if args.no_dep_launch:
        ada.ada_set_dependent_launch(ctx, False)
    stream = torch.cuda.current_stream()
    cflags = ada.ADA_CROSS_CAUSAL if args.causal else 0

    i32 = dict(dtype=torch.int32, device=dev)
    idx = [torch.empty((B, T), **i32) for _ in range(2)]
    cnt = [torch.empty((B,), **i32) for _ in range(2)]
    outs = [ada.CascadeOut(B, T, dev, want_gamma=False) for _ in range(2)]
    r_hist = torch.zeros((L, 3, B), **i32)                      # rep count, adds, removes per layer

    def cascade_pipeline(record=False):
        ada.ada_select_full(ctx, dev_layers[0], cfg.tau, outs[0].rep_out, outs[0].rep_out_cnt,
                            want_gamma=False, stream=stream)
        cur = 0
        if record:
            r_hist[0, 0].copy_(outs[0].rep_out_cnt)
        for l in range(1, L):
            nxt = 1 - cur
            ada.ada_cascade_step(ctx, dev_layers[l], cfg.tau, outs[cur].rep_out, outs[cur].rep_out_cnt,
                                 out=outs[nxt], flags=cflags, stream=stream)
            cur = nxt
            if record:
                r_hist[l, 0].copy_(outs[cur].rep_out_cnt)
                r_hist[l, 1].copy_(outs[cur].add_cnt)
                r_hist[l, 2].copy_(outs[cur].rem_cnt)
        return outs[cur]

    def independent_pipeline(keep=None):
        for l in range(L):
            ada.ada_select_full(ctx, dev_layers[l], cfg.tau, idx[0], cnt[0], want_gamma=False,
                                stream=stream)
            if keep is not None:
                keep.append((idx[0].clone(), cnt[0].clone()))

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    flush_l2 = step_bytes(cfg) <= L2_BYTES
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if flush_l2 else None

    def timed(fn, steps, warmup, cold=True):
        for _ in range(warmup):
            fn()
        barrier()
        sampler = ClockSampler(local)
        sampler.start()
        if not (flush_l2 and cold):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(steps):
                fn()
            e1.record(stream)
            barrier()
            total_ms = e0.elapsed_time(e1)
        else:
            # inputs smaller than L2: a cold L2 for every step, the flush outside the brackets
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                  for _ in range(steps)]
            for a, b in ev:
                flush_buf.zero_()
                a.record(stream)
                fn()
                b.record(stream)
            barrier()
            total_ms = sum(a.elapsed_time(b) for a, b in ev)
        clocks = sampler.finish()
        ms = replicas.max_over_ranks(rep, total_ms, dev)
        return ms / steps, clocks

    # ---- headline: cascade pipeline, inputs resident in HBM ----
    # One step (all L layers, every launch of the path) is captured once into a CUDA graph and
    # replayed: the calls are stream-ordered and never synchronise, so the graph holds exactly
    # the kernels an eager step launches.
    step_fn, indep_fn = cascade_pipeline, independent_pipeline
    if not args.no_graph:
        cascade_pipeline(); independent_pipeline()              # first-call set-up outside capture
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        g_casc, g_ind = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            stream = side
            with torch.cuda.graph(g_casc, stream=side):
                cascade_pipeline()
            with torch.cuda.graph(g_ind, stream=side):
                independent_pipeline()
        stream = torch.cuda.current_stream()
        step_fn, indep_fn = g_casc.replay, g_ind.replay
    ms_step, clocks = timed(step_fn, args.steps, args.warmup)
    value = replicas.whole_job_throughput(rep, B * T * L, ms_step * 1e-3)

    # ---- independent selection (full Gram at every layer) for the cascade speedup ----
    ms_indep, _ = timed(indep_fn, max(3, args.steps // 2), 3)
    ms_warm = timed(step_fn, args.steps, 1, cold=False)[0] if flush_l2 else None

    # ---- per-kernel times (events on the launching stream) and roofline of the dominant kernel ----
    cascade_pipeline(record=True)
    torch.cuda.synchronize()
    hist = r_hist.cpu().numpy().astype(np.int64)                # (L, 3, B)
    # Every launch is bracketed by CUDA events on the launching stream.  A spin kernel is queued
    # first so that the host runs ahead of the GPU: the brackets then measure the GPU working
    # through a full queue, not the host's launch latency.
    ada.ada_profile_enable(ctx, True)
    n_prof = 3
    for _ in range(n_prof):
        torch.cuda._sleep(int(2.0e7))
        cascade_pipeline()
        torch.cuda.synchronize()
    prof = ada.ada_profile_read(ctx)
    ada.ada_profile_enable(ctx, False)
    kernels = {k: {"launches": c // n_prof, "ms_per_step": ms / n_prof}
               for k, (c, ms) in prof.items() if c}
    dom = max(kernels, key=lambda k: kernels[k]["ms_per_step"])
    r_in = hist[:-1, 0, :]                                      # inherited count at layers 1..L-1
    r_valid = r_in - hist[1:, 2, :]
    flops = {
        "tri_full": float(d) * T * (T - 1) * B,
        "tri_rep": float(np.sum(d * r_in * (r_in - 1))),
        "cross": float(np.sum(2.0 * d * (T - r_in) * r_valid)),
    }
    peaks = measured_peaks()
    es = cfg.es
    if "cascade" in dom:
        alg, bound = flops["tri_rep"] + flops["cross"], "tensor"
        per = "d*r*(r-1) + 2*d*(T-r)*r_valid flop per launch"
    elif "cross" in dom:
        alg, bound, per = flops["cross"], "tensor", "2*d*(T-r)*r_valid flop per launch"
    elif "tri" in dom:
        alg, bound, per = flops["tri_full"] + flops["tri_rep"], "tensor", "d*n*(n-1) flop per launch"
    else:
        alg, bound, per = float(L * B * T * d * es), "hbm", "d*es bytes per token"
    secs = kernels[dom]["ms_per_step"] * 1e-3
    if bound == "tensor" and cfg.dtype == "bf16":
        peak, unit, achieved = peaks["bf16_sustained"], "TFLOP/s", alg / secs / 1e12
        peak_note = f"cuBLAS bf16 sustained, {peaks['src']}"
    elif bound == "tensor" and "tc" in dom:
        # fp32 storage on the tensor cores: every fp32 product is six bf16 products (three-term
        # split), so the ceiling for ALGORITHMIC fp32 flops is the bf16 peak / 6
        peak, unit, achieved = peaks["bf16_sustained"] / 6.0, "TFLOP/s", alg / secs / 1e12
        peak_note = f"cuBLAS bf16 sustained / 6 (fp32 as six bf16 products), {peaks['src']}"
    elif bound == "tensor":
        # fp32 FFMA kernel: 148 SMs x 128 lanes x 2 flop x max SM clock
        peak, unit, achieved = 148 * 128 * 2 * 1.965e9 / 1e12, "TFLOP/s", alg / secs / 1e12
        bound, peak_note = "alu", "148 SMs x 128 FFMA lanes x 2 flop x 1.965 GHz (derived)"
    else:
        peak, unit, achieved = peaks["hbm_gbs"], "GB/s", alg / secs / 1e9
        peak_note = f"copy bandwidth, {peaks['src']}"
    roofline = {"kernel": dom, "bound": bound, "achieved": achieved, "peak": peak, "unit": unit,
                "frac": achieved / peak, "peak_source": peak_note,
                "algorithmic_per_launch": per,
                "avg_launch_ms": kernels[dom]["ms_per_step"] / kernels[dom]["launches"],
                "traffic": NCU_TRAFFIC_BYTES.get((dom, cfg.cfg_id)),
                "traffic_source": NCU_TRAFFIC_SOURCE if (dom, cfg.cfg_id) in NCU_TRAFFIC_BYTES else None}
    if bound == "tensor" and cfg.dtype == "bf16":
        roofline["frac_sustained"] = achieved / peaks["bf16_sustained"]
        roofline["frac_burst"] = achieved / peaks["bf16_burst"]
        # the whole timed step (every launch of the path, graph replay): all algorithmic flops of a
        # step over ms_per_step -- free of the per-launch event brackets of the figure above
        step_tf = sum(flops.values()) / (ms_step * 1e-3) / 1e12
        roofline["whole_step"] = {"achieved": step_tf, "unit": "TFLOP/s",
                                  "frac_burst": step_tf / peaks["bf16_burst"],
                                  "frac_sustained": step_tf / peaks["bf16_sustained"]}

    # ---- sustained: the same graph replayed for at least a second (a 1 kW part settles to lower
    # clocks under load; the K-step figure above is the short-run one) ----
    sustained = None
    if not args.no_sustained:
        n_sus = max(args.steps, int(np.ceil(1100.0 / ms_step)))
        ms_sus, clk_sus = timed(step_fn, n_sus, 1)
        sustained = {"ms_per_step": ms_sus, "steps": n_sus,
                     "value": replicas.whole_job_throughput(rep, B * T * L, ms_sus * 1e-3), "unit": UNIT,
                     "clocks": clk_sus,
                     "ms_x_sm_mhz": (ms_sus * clk_sus["sm_mhz"]) if clk_sus.get("sm_mhz") else None}

    # ---- the full-selection Gram on this workload (Definition 1 at every layer), per launch ----
    roofline_full = None
    ada.ada_profile_enable(ctx, True)
    for _ in range(n_prof):
        torch.cuda._sleep(int(2.0e7))
        independent_pipeline()
        torch.cuda.synchronize()
    prof_i = {k: v for k, v in ada.ada_profile_read(ctx).items() if v[0] and "tri" in k}
    ada.ada_profile_enable(ctx, False)
    if prof_i:
        k_full = max(prof_i, key=lambda k: prof_i[k][1])
        n_l, ms_l = prof_i[k_full]
        secs_full = ms_l * 1e-3 / n_l
        ach = flops["tri_full"] / secs_full / 1e12
        roofline_full = {"kernel": k_full, "bound": "tensor" if "tc" in k_full else "alu",
                         "algorithmic_per_launch": "d*T*(T-1) flop per launch (lower triangle)",
                         "avg_launch_ms": secs_full * 1e3, "achieved": ach, "unit": "TFLOP/s"}
        if cfg.dtype == "bf16" and "tc" in k_full:
            roofline_full.update({"peak_burst": peaks["bf16_burst"], "peak_sustained": peaks["bf16_sustained"],
                                  "frac_burst": ach / peaks["bf16_burst"],
                                  "frac_sustained": ach / peaks["bf16_sustained"],
                                  "peak_source": f"cuBLAS bf16, {peaks['src']}"})

    # ---- cross-Gram where it is HBM-bound: the r/T = 0.01 points of the crossover sweep ----
    roofline_cross_hbm = None
    if cfg.cfg_id == 4 and not args.no_hbm_points and rank == 0:
        roofline_cross_hbm = [hbm_point(ada, dev, Tq, 0.01, peaks, args) for Tq in (16384, 8192)]

    # ---- set statistics: consecutive-layer Jaccard (independent) and cascade-vs-full Jaccard ----
    keep = []
    independent_pipeline(keep)
    torch.cuda.synchronize()
    indep = [[i[b, :int(c[b])].cpu().numpy() for b in range(B)] for i, c in keep]
    casc_sets = []
    ada.ada_select_full(ctx, dev_layers[0], cfg.tau, outs[0].rep_out, outs[0].rep_out_cnt,
                        want_gamma=False)
    cur = 0
    casc_sets.append([outs[0].rep_out[b, :int(outs[0].rep_out_cnt[b])].cpu().numpy() for b in range(B)])
    for l in range(1, L):
        ada.ada_cascade_step(ctx, dev_layers[l], cfg.tau, outs[cur].rep_out, outs[cur].rep_out_cnt,
                             out=outs[1 - cur], flags=cflags)
        cur = 1 - cur
        casc_sets.append([outs[cur].rep_out[b, :int(outs[cur].rep_out_cnt[b])].cpu().numpy()
                          for b in range(B)])
    j_consec = [float(np.mean([jaccard(indep[l][b], indep[l + 1][b]) for b in range(B)]))
                for l in range(L - 1)]
    j_cvf = [float(np.mean([jaccard(indep[l][b], casc_sets[l][b]) for b in range(B)]))
             for l in range(L)]
    st, n_zero = ada.ada_device_status(ctx)
    assert st == 0, ada.status_string(st)
    ops_indep = L * ada.ada_gram_op_count(False, T, d)
    ops_casc = ada.ada_gram_op_count(False, T, d) + int(
        np.mean([sum(ada.ada_gram_op_count(True, T, d, int(r_in[l, b])) for l in range(L - 1))
                 for b in range(B)]))

    # ---- end to end: HOST buffers through the C ABI, copies inside the timed region ----
    e2e = None
    if not args.no_e2e:
        hi = lambda *s: torch.empty(s, dtype=torch.int32).pin_memory()  # noqa: E731
        h_idx, h_cnt = [hi(B, T), hi(B, T)], [hi(B), hi(B)]
        h_add, h_addc, h_rem, h_remc = hi(B, T), hi(B), hi(B, T), hi(B)

        def e2e_pipeline():
            ada.ada_select_full_host(ctx, pin[0], cfg.tau, h_idx[0], h_cnt[0])
            c = 0
            for l in range(1, L):
                ada.ada_cascade_step_host(ctx, pin[l], cfg.tau, h_idx[c], h_cnt[c], h_idx[1 - c],
                                          h_cnt[1 - c], h_add, h_addc, h_rem, h_remc, flags=cflags)
                c = 1 - c

        for _ in range(2):
            e2e_pipeline()
        barrier()
        n_e2e = max(3, args.steps // 2)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)                       # the host calls run on this stream and wait for it
        for _ in range(n_e2e):
            e2e_pipeline()
        e1.record(stream)
        barrier()
        t_e2e = replicas.max_over_ranks(rep, e0.elapsed_time(e1) * 1e-3 / n_e2e, dev)
        n_tok = B * T
        h2d = L * n_tok * d * es + (L - 1) * (n_tok * 4 + B * 4)
        d2h = (n_tok * 4 + B * 4) + (L - 1) * 3 * (n_tok * 4 + B * 4)
        e2e = {"value": world * B * T * L / t_e2e, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": 1e3 * t_e2e,
               "api": "ada_select_full_host + ada_cascade_step_host, pinned host tensors"}

    # ---- the oracle on this machine's host cores (rank 0, N = 1 only), bounded sample ----
    cpu_baseline, parity_sample = None, None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        n_lay = min(L, args.ref_layers)
        t_c, band, mism = [], 0, 0
        t0 = time.perf_counter()
        R = [oracle.select_full(wl.as_f64(host_layers[0][b]), cfg.tau)[0] for b in range(B)]
        t_full = time.perf_counter() - t0
        for l in range(n_lay):
            if l > 0:
                t1 = time.perf_counter()
                R = [oracle.cascade_step(wl.as_f64(host_layers[l][b]), cfg.tau, R[b],
                                         causal=args.causal).rep
                     for b in range(B)]
                t_c.append(time.perf_counter() - t1)
            mism += sum(R[b].tolist() != casc_sets[l][b].tolist() for b in range(B))
        t_est = t_full + (L - 1) * (float(np.mean(t_c)) if t_c else t_full)
        cpu_baseline = {"value": B * T * L / t_est, "unit": UNIT, "cores": oracle.num_threads(),
                        "kind": "oracle",
                        "sample": f"layers 0..{n_lay - 1} computed in full (fp64); step time = "
                                  f"t(full, layer 0) + {L - 1} x mean t(cascade step)",
                        "t_full_s": t_full, "t_cascade_step_s": float(np.mean(t_c)) if t_c else None}
        parity_sample = {"layers_checked": n_lay, "set_mismatches": mism}
        if cfg.cfg_id == 1:      # the small fp32 configuration: also one host thread
            nthr = oracle.num_threads()
            oracle.set_threads(1)
            t0 = time.perf_counter()
            R1 = [oracle.select_full(wl.as_f64(host_layers[0][b]), cfg.tau)[0] for b in range(B)]
            t_f1 = time.perf_counter() - t0
            t1 = time.perf_counter()
            if n_lay > 1:
                [oracle.cascade_step(wl.as_f64(host_layers[1][b]), cfg.tau, R1[b], causal=args.causal)
                 for b in range(B)]
            t_c1 = time.perf_counter() - t1 if n_lay > 1 else t_f1
            oracle.set_threads(nthr)
            cpu_baseline["one_thread_value"] = B * T * L / (t_f1 + (L - 1) * t_c1)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": ("bf16 x bf16 -> f32" if cfg.dtype == "bf16" else
                      ("f32" if args.engine == 1 else "f32 as 3 bf16 terms (6 cross products) -> f32")),
            "data": "synthetic", "config": workload_dict(cfg), "clocks": clocks, "e2e": e2e,
            "warm_l2_ms_per_step": ms_warm,
            "gpu_launches": args.steps * sum(k["launches"] for k in kernels.values()),
            "roofline": roofline, "roofline_full": roofline_full,
            "roofline_cross_hbm": roofline_cross_hbm, "sustained": sustained,
            "cpu_baseline": cpu_baseline,
            "independent": {"value": world * B * T * L / (ms_indep * 1e-3), "unit": UNIT,
                            "ms_per_step": ms_indep},
            "cascade_speedup": ms_indep / ms_step,
            "kernels": kernels,
            "algorithmic_gflop_per_step": {k: v / 1e9 for k, v in flops.items()},
            "gram_ops": {"independent": ops_indep, "cascade": ops_casc,
                         "saved_frac": 1.0 - ops_casc / ops_indep},
            "sets": {"r_layer0": [int(x) for x in hist[0, 0]], "r_last": [int(x) for x in hist[-1, 0]],
                     "jaccard_consecutive_independent_mean": float(np.mean(j_consec)) if j_consec else None,
                     "jaccard_cascade_vs_full_mean": float(np.mean(j_cvf)),
                     "jaccard_cascade_vs_full_last": j_cvf[-1]},
            "parity_sample": parity_sample, "zero_norm_rows": n_zero,
            "engine": "ffma" if args.engine == 1 else "auto", "cuda_graph": not args.no_graph,
            "cross_check": "causal (s < t)" if args.causal else "as printed in Algorithm 1 (all valid representatives)",
        }
        print(json.dumps(line))
    ada.ada_destroy(ctx)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
