#!/usr/bin/env python
"""Benchmark of the MGRIT-GRU hot path on B200:  python bench.py --gpus N --steps K --warmup W

One step = one pass of the whole path over one batch of seeded synthetic per-frame features:
input projections, MGRIT forward of every layer, loss head, MGRIT adjoint of every layer,
time-parallel weight gradients, SGD update.  Metric: timesteps x batch per second (T*B / step time),
summed over the N independent replicas (the path does not shard across GPUs: replicas only).

Prints ONE JSON line.  `--impl reference` times the fp64 CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "MGRIT-GRU fwd+adjoint timesteps*batch/sec"
UNIT = "timesteps*batch/s"
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of the fused forward-step kernel per (row x hidden
# unit).  A constant taken from an `ncu --set full --clock-control none` capture of that kernel, NOT measured in a
# bench run: 17.4 B on the default workload's own level-0 sweep (four dependent steps of 16384 rows in one launch,
# H = 1024: 1166 MB).  Traffic grows in proportion to rows x hidden units, so a workload's per-launch traffic is this
# figure x the rows x H its launches process.
NCU_DRAM_BYTES_PER_ROW_UNIT = {"forward_step": {1024: 17.4}}
NOMINAL_BF16_TFLOPS = 2250.0       # dense bf16, vendor figure (context only)


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            d = json.load(f)
        return d, "measured"
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


# ------------------------------------------------------------------------------------------ CPU oracle leg
def oracle_step(w, d, T, Bsz):
    """The same training step computed by the fp64 oracle (as it stands) on a T x Bsz sample."""
    import numpy as np
    from oracle import mgrit_gru_oracle as O
    f64 = lambda a: a.astype(np.float64)
    layers = [[f64(l[n]) for n in ("W_ih", "W_hh", "b_ih", "b_hh")] for l in d["layers"]]
    x, h0 = f64(d["x"]), f64(d["h0"])
    kw = dict(cf=w.cf, levels=w.levels, cell=w.cell, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse)
    hs, inp = [], x
    for P in layers:
        h, _ = O.mgrit_forward(*P, inp, h0, iters=w.iters_fwd, **kw)
        hs.append(h)
        inp = h
    loss, dhT, dWc, dbc = O.xent_head(hs[-1][-1], f64(d["W_c"]), f64(d["b_c"]), d["labels"])
    seed = np.zeros_like(hs[-1])
    seed[-1] = dhT
    for l in range(len(layers) - 1, -1, -1):
        inp = x if l == 0 else hs[l - 1]
        lam, lam0, g, _ = O.mgrit_adjoint(*layers[l], inp, h0, hs[l], seed, iters=w.iters_adj, want_dx=l > 0, **kw)
        for i, n in enumerate(("dW_ih", "dW_hh", "db_ih", "db_hh")):
            layers[l][i] = O.sgd_update(layers[l][i], g[n], 1e-3)
        seed = g.get("dx")
    return loss


def cpu_sample_shape(w):
    """A bounded sample of the workload: same widths, levels and cycle counts, shorter and narrower batch."""
    unit = w.cf ** (w.levels - 1)
    T = min(w.T, max(unit * 4, 256 if w.H >= 512 else w.T))
    T = (T // unit) * unit
    Bsz = min(w.B, 8 if w.H >= 512 else w.B)
    return T, Bsz


def time_oracle(w, steps=1, warmup=0):
    from paper_2203_04738_b200.synthetic import make_inputs
    T, Bsz = cpu_sample_shape(w)
    d = make_inputs(w, T=T, B=Bsz)
    for _ in range(warmup):
        oracle_step(w, d, T, Bsz)
    ts = []
    for _ in range(max(1, steps)):
        t0 = time.perf_counter()
        oracle_step(w, d, T, Bsz)
        ts.append(time.perf_counter() - t0)
    sec = sum(ts) / len(ts)
    try:
        import threadpoolctl
        cores = max([p.get("num_threads", 1) for p in threadpoolctl.threadpool_info()] or [1])
    except Exception:
        cores = os.cpu_count() or 1
    return {"value": T * Bsz / sec, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"same step on T={T}, B={Bsz} of workload '{w.name}' (fp64 NumPy, {len(ts)} run(s), {sec:.2f} s each)"}, sec


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """nvidia-smi polled every 20 ms in a child process.  It is started before the warm-up steps (the tool needs
    a few hundred ms to produce its first line) and every line carries its own timestamp, so stop() can keep the
    samples that fall inside the timed region [t0, t1] (host wall clock)."""
    Q = "timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
        "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"

    def __init__(self, index):
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "20",
                                       "-i", str(index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.p = None

    def stop(self, t0=None, t1=None):
        import datetime
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.p.terminate()
        try:
            out, _ = self.p.communicate(timeout=5)
        except Exception:
            self.p.kill()
            out = ""
        self.p = None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        self.rows = []
        for line in out.strip().splitlines():
            f = [s.strip() for s in line.split(",")]
            if len(f) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f")
                self.rows.append((ts, float(f[1]), float(f[2]), [n for n, v in zip(names, f[4:8]) if v.lower().startswith("active")]))
            except ValueError:
                continue
        return self.window(t0, t1)

    def window(self, t0, t1):
        """Clock summary of the samples inside [t0, t1] (host wall clock); valid after stop()."""
        rows = getattr(self, "rows", [])
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        inside = [r for r in rows if t0 is not None and t0 <= r[0] <= t1]
        scope = "timed region"
        if not inside:        # region shorter than the polling period: take the samples nearest to it
            scope = "nearest to the timed region"
            mid = t0 + (t1 - t0) / 2 if t0 is not None else None
            inside = sorted(rows, key=lambda r: abs((r[0] - mid).total_seconds()))[:3] if mid is not None else rows
        sm = [r[1] for r in inside]
        reasons = sorted({n for r in inside for n in r[3]})
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(r[2] for r in inside) if inside else None,
                "reasons": reasons, "samples": len(sm), "scope": scope}


# ------------------------------------------------------------------------------------------ GPU helpers
OPERAND_NAMES = {0: "fp32 (FFMA)", 1: "tf32 tensor cores, three-term split", 2: "bf16 tensor cores", 3: "tf32 tensor cores, single pass"}
OPERAND_DTYPES = {0: "f32", 1: "tf32x3", 2: "bf16", 3: "tf32"}


def describe(w, T, Bsz):
    return (f"{w.name}: {w.layers}-layer GRU I={w.I} H={w.H} B={Bsz} T={T}, cf={w.cf}, levels={w.levels}, "
            f"iters fwd/adj={w.iters_fwd}/{w.iters_adj}, relax fine/coarse={'FCF' if w.relax_fine else 'F'}/"
            f"{'FCF' if w.relax_coarse else 'F'}, implicit cell, {w.classes}-class xent on h_T, SGD, "
            f"operands {OPERAND_NAMES[w.operands]}")


def time_gpu_step(w, T, serial, steps, warmup, dev, use_graph=True):
    """Device-resident inputs; returns (ms per step, wall-clock window of the timed region).  The same step as the
    headline (all layers forward, head, adjoint, gradients, SGD) with MGRIT or with the serial sweep + exact BPTT."""
    import datetime
    import torch
    from paper_2203_04738_b200 import binding as B
    from paper_2203_04738_b200.synthetic import make_inputs
    from paper_2203_04738_b200.train_step import GraphedTrainingStep, alloc_buffers, training_step
    d = make_inputs(w, T=T)
    up = lambda a: torch.from_numpy(a).to(dev)
    layers = [{n: up(l[n]) for n in ("W_ih", "W_hh", "b_ih", "b_hh")} for l in d["layers"]]
    W_c, b_c, labels, h0, x = up(d["W_c"]), up(d["b_c"]), up(d["labels"]), up(d["h0"]), up(d["x"])
    buf = alloc_buffers(w, T, w.B, dev, serial=serial, flags=B.FLAG_SKIP_DUPLICATE_FRELAX)
    step = lambda: training_step(w, layers, W_c, b_c, x, h0, labels, buf)
    if use_graph:
        try:
            step = GraphedTrainingStep(w, layers, W_c, b_c, x, h0, labels, buf)
        except Exception as e:
            sys.stderr.write(f"bench: CUDA graph capture failed ({e!r}); launching from the host\n")
    for _ in range(max(warmup, 3)):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = datetime.datetime.now()
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    t1 = datetime.datetime.now()
    return e0.elapsed_time(e1) / steps, (t0, t1)


# ------------------------------------------------------------------------------------------ main
def time_lstm(w, T, dev):
    """One Implicit-LSTM layer of the workload's shape: MGRIT forward (the workload's forward cycles), adjoint cycles
    seeded at the last step, all gradients and dx; next to it the serial sweep + exact BPTT (levels = 1).  Host launches."""
    import numpy as np
    import torch
    from paper_2203_04738_b200 import binding as B
    rng = np.random.default_rng(w.seed + 17)
    k = 1.0 / np.sqrt(w.H)
    shapes = dict(W_ih=(4 * w.H, w.I), W_hh=(4 * w.H, w.H), b_ih=(4 * w.H,), b_hh=(4 * w.H,))
    p = {n: torch.from_numpy(rng.uniform(-k, k, sh).astype(np.float32)).to(dev) for n, sh in shapes.items()}
    x = torch.from_numpy(np.maximum(rng.standard_normal((T, w.B, w.I)), 0).astype(np.float32)).to(dev)
    u0 = torch.zeros(2, w.B, w.H, device=dev)
    dhT = torch.from_numpy(rng.standard_normal((w.B, w.H)).astype(np.float32)).to(dev)
    out = {}
    for leg, levels in (("mgrit", w.levels), ("serial", 1)):
        kw = dict(cf=w.cf, levels=levels, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse, operands=w.operands)
        cf_ = B.make_cfg(T, w.B, w.I, w.H, iters=w.iters_fwd if levels > 1 else 1, **kw)
        ca_ = B.make_cfg(T, w.B, w.I, w.H, iters=w.iters_adj if levels > 1 else 1, **kw)
        nf, na = B.lstm_workspace_bytes(cf_)[0], B.lstm_workspace_bytes(ca_)[1]
        wsf, wsa = torch.empty(nf, dtype=torch.uint8, device=dev), torch.empty(na, dtype=torch.uint8, device=dev)

        def step():
            u, gi, _ = B.mgrit_lstm_forward(cf_, p, x, u0, ws=wsf)
            return B.mgrit_lstm_adjoint(ca_, p, x, u0, gi, u, dhT=dhT, want_du=False, ws=wsa)

        for _ in range(2):
            step()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(3):
            step()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / 3
        out[f"{leg}_ms"] = ms
        if leg == "mgrit":
            B.profile_enable(True)
            step()
            prof = B.profile_read()
            by_size = {}
            for name, tms_, fl_ in B.profile_records():
                e = by_size.setdefault(f"{name}@{fl_ / 1e9:.2f}GF", [0, 0.0])
                e[0] += 1
                e[1] += tms_
            out["kernel_by_size"] = {kk: {"launches_per_step": v[0], "avg_us": v[1] / v[0] * 1e3, "ms_per_step": v[1],
                                          "tflops": float(kk.split("@")[1][:-2]) * 1e9 / (v[1] / v[0] * 1e-3) / 1e12}
                                     for kk, v in by_size.items()}
            B.profile_enable(False)
            out["kernel_breakdown"] = {kk: {"ms_per_step": v[0], "launches_per_step": v[1],
                                            "tflops": (v[2] / (v[0] * 1e-3) / 1e12) if v[0] > 0 else None} for kk, v in prof.items()}
        del wsf, wsa
        torch.cuda.empty_cache()
    out.update({"value": T * w.B / (out["mgrit_ms"] * 1e-3), "unit": UNIT, "steps": 3, "launch": "host launches",
                "speedup_vs_serial": out["serial_ms"] / out["mgrit_ms"],
                "what": f"one Implicit-LSTM layer, T={T}, B={w.B}, I={w.I}, H={w.H}, operands {OPERAND_NAMES[w.operands]}: "
                        f"{w.iters_fwd} forward / {w.iters_adj} adjoint cycles + gradients; serial = sweep + exact BPTT"})
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="train")
    ap.add_argument("--T", type=int, default=None, help="override the sequence length (sweeps)")
    ap.add_argument("--serial", action="store_true", help="time the GPU serial sweep + exact BPTT instead of MGRIT")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel from the host instead of replaying a CUDA graph")
    ap.add_argument("--no-kernel-timing", action="store_true", help="skip the per-kernel CUDA-event pass")
    ap.add_argument("--no-serial", action="store_true", help="skip the GPU serial-sweep leg (gpu_serial)")
    ap.add_argument("--no-sweep", action="store_true", help="skip the sequence-length sweep (t_sweep)")
    ap.add_argument("--operands", default=None, choices=["fp32", "tf32", "bf16", "tf32_1pass"],
                    help="override the workload's operand mode (tf32: three-term split on the tensor cores, fp32-level accuracy)")
    ap.add_argument("--lstm", action="store_true", help="also time one Implicit-LSTM layer of the workload's shape (key lstm)")
    ap.add_argument("--stacked", action="store_true", help="also time the step with all layers in one state (one MGRIT cycle for the stack)")
    args = ap.parse_args()

    from paper_2203_04738_b200.synthetic import WORKLOADS, make_inputs
    w = WORKLOADS[args.workload]
    if args.operands:
        import dataclasses
        w = dataclasses.replace(w, operands={"fp32": 0, "tf32": 1, "bf16": 2, "tf32_1pass": 3}[args.operands])
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    T = args.T or w.T
    # bytes one step streams: x, gi and the states of every layer (fp32)
    stream_mb = 4.0 * T * w.B * (w.I + w.layers * 4 * w.H) / 1e6
    l2_note = (f"inputs larger than L2 (x, gi and states, {stream_mb:.0f} MB, are re-streamed from HBM every step)" if stream_mb > 126.0
               else f"working set {stream_mb:.1f} MB fits the 126 MB L2 and no flush is done: an L2-resident side case, not the headline configuration")
    config = {"workload": describe(w, T, w.B),
              "solver": "serial sweep + BPTT" if args.serial else "MGRIT",
              "l2": l2_note,
              "parallelism": f"replicas x{args.gpus} (no sharding, no collective)"}

    if args.impl == "reference":
        if rank != 0:
            return
        cb, sec = time_oracle(w, steps=args.steps, warmup=min(args.warmup, 1))
        # this arm times a bounded sample of the workload (same widths, levels and cycle counts): say so
        Ts, Bs = cpu_sample_shape(w)
        config = {"workload": describe(w, Ts, Bs) + f" -- a bounded sample of '{w.name}' (T={w.T}, B={w.B}), which the fp64 "
                              "oracle cannot finish within minutes",
                  "solver": "MGRIT (fp64 NumPy oracle on the host cores)", "l2": "n/a (CPU)",
                  "parallelism": "host threads of the BLAS library"}
        print(json.dumps({"metric": METRIC, "value": cb["value"], "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
                          "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
                          "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config, "impl": "reference",
                          "cpu_baseline": cb, "gpu_launches": 0,
                          "e2e": {"value": cb["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    import torch
    import torch.distributed as dist
    from paper_2203_04738_b200 import binding as B
    from paper_2203_04738_b200.replicas import job_throughput, max_over_ranks
    from paper_2203_04738_b200.train_step import GraphedTrainingStep, HostInputPipeline, alloc_buffers, training_step

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    d = make_inputs(w, T=T)
    up = lambda a: torch.from_numpy(a).to(dev)
    layers = [{n: up(l[n]) for n in ("W_ih", "W_hh", "b_ih", "b_hh")} for l in d["layers"]]
    W_c, b_c, labels, h0 = up(d["W_c"]), up(d["b_c"]), up(d["labels"]), up(d["h0"])
    x_host = torch.from_numpy(d["x"]).pin_memory()
    x = x_host.to(dev)
    # cycles after the first skip re-doing the F-relaxation that the previous cycle just finished (identical results)
    buf = alloc_buffers(w, T, w.B, dev, serial=args.serial, flags=B.FLAG_SKIP_DUPLICATE_FRELAX)
    loss_host = torch.empty(1).pin_memory()

    def eager_step():
        return training_step(w, layers, W_c, b_c, x, h0, labels, buf)

    # The step is captured once into a CUDA graph and replayed (same kernels, same order, same buffers).
    graphed = None
    if not args.no_graph:
        try:
            graphed = GraphedTrainingStep(w, layers, W_c, b_c, x, h0, labels, buf)
        except Exception as e:      # capture unavailable here: launch from the host
            sys.stderr.write(f"bench: CUDA graph capture failed ({e!r}); launching from the host\n")
            graphed = None
    step = graphed if graphed is not None else eager_step
    config["launch"] = "one CUDA graph replay per step" if graphed is not None else "host launches"

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    import datetime
    sampler = ClockSampler(local_rank) if rank == 0 else None
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    l0 = B.kernel_launches()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    wall0 = datetime.datetime.now()
    e0.record()
    t_host = time.perf_counter()
    marks = []                                  # one event after every step: median and best step beside the mean
    for _ in range(args.steps):
        loss = step()
        marks.append(torch.cuda.Event(enable_timing=True))
        marks[-1].record()
    host_ms = (time.perf_counter() - t_host) * 1e3 / args.steps     # CPU time to enqueue one step (no sync inside)
    e1.record()
    barrier()
    wall1 = datetime.datetime.now()
    ms = e0.elapsed_time(e1)
    per_step = sorted(a.elapsed_time(b) for a, b in zip([e0] + marks[:-1], marks))
    step_stats = {"median_ms": per_step[len(per_step) // 2], "best_ms": per_step[0], "worst_ms": per_step[-1],
                  "what": "single steps of the timed region (this rank), from an event recorded after every step"}
    launches = graphed.launches * args.steps if graphed is not None else B.kernel_launches() - l0
    windows = {"headline": (wall0, wall1)}      # the clock sampler keeps running through the later legs
    ms = max_over_ranks(ms, dev)
    ms_step = ms / args.steps
    value = job_throughput(T * w.B, ms_step, world)

    # the forward solves alone (projections + MGRIT forward of every layer), host launches
    fwd_only = None
    if world == 1 and not args.no_kernel_timing:
        from paper_2203_04738_b200.train_step import forward_pass
        for _ in range(3):
            forward_pass(layers, x, h0, buf)
        torch.cuda.synchronize()
        nf = max(3, args.steps // 2)
        e0.record()
        for _ in range(nf):
            forward_pass(layers, x, h0, buf)
        e1.record()
        torch.cuda.synchronize()
        fms = e0.elapsed_time(e1) / nf
        fwd_only = {"ms_per_step": fms, "value": T * w.B / (fms * 1e-3), "unit": UNIT, "steps": nf,
                    "what": "input projections + forward solve of every layer only (no head, adjoint, gradients or update)"}

    # end to end: inputs start in pinned host memory, the loss is read back, every step
    e2e = None
    if not args.no_e2e:
        # Every step's input is copied from pinned host memory inside the timed region; the copy of step k+1
        # runs on a side stream while step k computes (two device buffers), and the loss is read back every step.
        pipe = HostInputPipeline(x.shape, x.dtype, dev)
        e2e_graphs = None
        if graphed is not None:     # one captured step per input buffer of the pipeline
            try:
                e2e_graphs = [GraphedTrainingStep(w, layers, W_c, b_c, xb_, h0, labels, buf) for xb_ in pipe.bufs]
            except Exception as e:
                sys.stderr.write(f"bench: CUDA graph capture failed ({e!r}); launching from the host\n")
        barrier()
        e0.record()
        pipe.submit(x_host)
        for k in range(args.steps):
            xk = pipe.acquire()
            if k + 1 < args.steps:
                pipe.submit(x_host)
            loss = e2e_graphs[k % 2]() if e2e_graphs else training_step(w, layers, W_c, b_c, xk, h0, labels, buf)
            pipe.release()
            loss_host.copy_(loss, non_blocking=True)
            torch.cuda.current_stream().synchronize()
        e1.record()
        barrier()
        ms2 = e0.elapsed_time(e1)
        ms2 = max_over_ranks(ms2, dev)
        e2e = {"value": job_throughput(T * w.B, ms2 / args.steps, world), "unit": UNIT,
               "h2d_bytes_per_step": x_host.numel() * 4, "d2h_bytes_per_step": 4,
               "overlap": "input copy of step k+1 on a side stream during step k (all copies inside the timed region)"}

    # per-kernel timing pass (CUDA events around every GEMM-shaped launch; outside the timed region so
    # that the event records do not perturb it)
    roofline, breakdown, by_size, roofline_by_class = None, None, None, None
    if rank == 0 and not args.no_kernel_timing:
        torch.cuda.synchronize()
        nprof = 2
        B.profile_enable(True)
        for _ in range(nprof):
            eager_step()
        prof = B.profile_read()
        by_size = {}
        for name, tms_, fl_ in B.profile_records():
            e = by_size.setdefault(f"{name}@{fl_ / 1e9:.2f}GF", [0, 0.0])
            e[0] += 1
            e[1] += tms_
        by_size = {k: {"launches_per_step": v[0] // nprof, "avg_us": v[1] / v[0] * 1e3, "ms_per_step": v[1] / nprof,
                       "tflops": float(k.split("@")[1][:-2]) * 1e9 / (v[1] / v[0] * 1e-3) / 1e12} for k, v in by_size.items()}
        B.profile_enable(False)
        peaks, pk = measured_peaks()
        bf16 = w.operands == 2
        breakdown = {k: {"ms_per_step": v[0] / nprof, "launches_per_step": v[1] // nprof,
                         "tflops": (v[2] / (v[0] * 1e-3) / 1e12) if v[0] > 0 else None} for k, v in prof.items()}
        # The dominant KERNEL: classes that time one kernel per record (the adjoint-step class times its operand
        # packing kernel together with the product, the gradient class a whole pass of several kernels).
        single = {k: v for k, v in prof.items() if k not in ("adjoint_step", "gradient_gemms")}
        name, (tms, n, fl) = max(single.items(), key=lambda kv: kv[1][0])
        if bf16:
            peak = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
            burst = float(peaks["bf16_tflops"])
            bound, note = "tensor", (f"bf16 dense cuBLAS figures ({pk}): `peak`/`frac` use the sustained one (the kernel is timed inside "
                                     "whole steps), `frac_burst` the burst one, `frac_nominal` the vendor's 2250 TFLOP/s")
        elif w.operands in (1, 3):
            # tf32 products: the measured bf16 figures scaled by the nominal tf32 : bf16 ratio (1.1 : 2.25 PFLOP/s dense);
            # the recorded flops are those the tensor cores execute (three products per element in the split mode)
            ratio = 1.1 / 2.25
            peak = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])) * ratio
            burst = float(peaks["bf16_tflops"]) * ratio
            bound, note = "tensor", f"tf32: bf16 dense cuBLAS figures ({pk}) x the nominal tf32:bf16 ratio 1.1/2.25"
        else:
            # fp32 FFMA: 148 SMs x 128 lanes x 2 flop x max SM clock
            peak = burst = 148 * 128 * 2 * float(peaks.get("sm_max_mhz", 1965.0)) * 1e6 / 1e12
            bound, note = "alu", "fp32 FFMA: 148 SMs x 128 lanes x 2 flop x max SM clock"
        if tms > 0 and n > 0:
            achieved = fl / (tms * 1e-3) / 1e12
            units = (fl / n) / (6.0 * w.H)          # (row x hidden unit) pairs of an average launch
            roofline = {"kernel": name, "bound": bound, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                        "frac": achieved / peak, "frac_sustained": achieved / peak, "frac_burst": achieved / burst,
                        "frac_nominal": achieved / NOMINAL_BF16_TFLOPS if bf16 else None, "peak_burst": burst,
                        "traffic": (NCU_DRAM_BYTES_PER_ROW_UNIT[name][w.H] * units
                                    if w.H in NCU_DRAM_BYTES_PER_ROW_UNIT.get(name, {}) else None),
                        "traffic_note": "DRAM bytes per average launch = a constant from an ncu capture of this kernel (bytes per "
                                        "row x hidden unit at this H) x the launch's rows x H; not measured in this run",
                        # per cell evaluation the method moves 3H of gi + H written + H/(cf-1) read of state, fp32:
                        # 16H + 4H/(cf-1) bytes; this implementation also writes and reads a bf16 copy of the state
                        # and re-reads the fp32 state every step: 24H bytes
                        "algorithmic_bytes": (16.0 + 4.0 / (w.cf - 1)) * units if name == "forward_step" else None,
                        # input projection 6 (bf16 copy), previous state 4 + 2 (its bf16 copy), new state 4 + 2
                        "implementation_bytes": 18.0 * units if name == "forward_step" else None,
                        "avg_launch_us": tms / n * 1e3, "launches_per_step": n // nprof,
                        "share_of_gemm_time": tms / max(sum(v[0] for v in prof.values()), 1e-9), "peak_source": note}
        roofline_by_class = {k: {"tflops": v[2] / (v[0] * 1e-3) / 1e12, "frac_sustained": v[2] / (v[0] * 1e-3) / 1e12 / peak,
                                 "frac_burst": v[2] / (v[0] * 1e-3) / 1e12 / burst, "ms_per_step": v[0] / nprof}
                             for k, v in prof.items() if v[0] > 0 and k not in ("forward_serial_chain", "adjoint_serial_chain")}
        for k in ("forward_serial_chain", "adjoint_serial_chain"):     # latency-bound: time per dependent step
            if prof[k][0] > 0:
                nsteps = prof[k][2] / (2.0 * w.B * 3.0 * w.H * w.H)
                roofline_by_class[k] = {"us_per_dependent_step": prof[k][0] * 1e3 / nsteps, "ms_per_step": prof[k][0] / nprof}

    # ---- the same GPU's serial sweep + exact BPTT on the same workload, and the speed-up over it as T grows
    gpu_serial, t_sweep = None, None
    if rank == 0 and world == 1 and not args.serial:
        from paper_2203_04738_b200.synthetic import WORKLOADS as _W
        if not args.no_serial:
            ms_s, win = time_gpu_step(w, T, True, 5, 3, dev, use_graph=not args.no_graph)
            windows["gpu_serial"] = win
            gpu_serial = {"ms_per_step": ms_s, "value": T * w.B / (ms_s * 1e-3), "unit": UNIT, "steps": 5,
                          "speedup_mgrit_over_serial": ms_s / ms_step,
                          "what": "same step with gru_serial_forward / gru_serial_backward (exact sweep + BPTT) instead of MGRIT"}
        if not args.no_sweep:
            wl = _W["long"]
            t_sweep = {"workload": describe(wl, "{512,1024,2048,4096}", wl.B), "points": []}
            for Ts in (512, 1024, 2048, 4096):
                ms_m, win_m = time_gpu_step(wl, Ts, False, 5, 3, dev, use_graph=not args.no_graph)
                ms_r, win_r = time_gpu_step(wl, Ts, True, 3, 3, dev, use_graph=not args.no_graph)
                windows[f"sweep_T{Ts}_mgrit"] = win_m
                windows[f"sweep_T{Ts}_serial"] = win_r
                t_sweep["points"].append({"T": Ts, "mgrit_ms": ms_m, "serial_ms": ms_r, "speedup": ms_r / ms_m})
                torch.cuda.empty_cache()
    stacked = None
    if rank == 0 and world == 1 and args.stacked and w.layers > 1:
        from paper_2203_04738_b200.train_step import stacked_training_step
        cfg_s = B.make_cfg(T, w.B, w.I, w.H, cf=w.cf, levels=w.levels, iters=w.iters_fwd, relax_fine=w.relax_fine,
                           relax_coarse=w.relax_coarse, operands=w.operands)
        nf, na = B.stack_workspace_bytes(cfg_s, w.layers)
        wsf, wsa = torch.empty(nf, dtype=torch.uint8, device=dev), torch.empty(na, dtype=torch.uint8, device=dev)
        h0s = torch.zeros(w.layers, w.B, w.H, device=dev)
        sstep = lambda: stacked_training_step(w, layers, W_c, b_c, x, h0s, labels, ws_fwd=wsf, ws_adj=wsa, ws_head=buf.ws_head)
        stacked_launch = "host launches"
        if not args.no_graph:      # thousands of small launches on the coarsest level: replay them from a CUDA graph
            from paper_2203_04738_b200.train_step import GraphedTrainingStep
            sstep = GraphedTrainingStep(w, layers, W_c, b_c, x, h0s, labels, None, step_fn=sstep)
            stacked_launch = f"CUDA graph replay ({sstep.launches} kernels per step)"
        for _ in range(2):
            sstep()
        torch.cuda.synchronize()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        for _ in range(3):
            sstep()
        s1.record()
        torch.cuda.synchronize()
        ms_st = s0.elapsed_time(s1) / 3
        stacked = {"ms_per_step": ms_st, "value": T * w.B / (ms_st * 1e-3), "unit": UNIT, "steps": 3, "launch": stacked_launch,
                   "what": "all layers in one time-step state, one MGRIT cycle for the stack (generic step kernels: not tuned)"}
        del wsf, wsa
    lstm = None
    if rank == 0 and world == 1 and args.lstm:
        lstm = time_lstm(w, T, dev)
    clocks = None
    if sampler:
        clocks = sampler.stop(*windows["headline"])
        for k, win in windows.items():
            if k == "headline":
                continue
            c = sampler.window(*win)
            if k == "gpu_serial" and gpu_serial:
                gpu_serial["clocks"] = c
            elif t_sweep:
                Ts, leg = k.split("_")[1][1:], k.split("_")[2]
                for pt in t_sweep["points"]:
                    if str(pt["T"]) == Ts:
                        pt[f"clocks_{leg}"] = {"sm_mhz": c["sm_mhz"], "reasons": c["reasons"], "samples": c["samples"]}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cpu, _ = time_oracle(w)
    status = B.last_device_status()
    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
           "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": OPERAND_DTYPES[w.operands], "data": "synthetic", "config": config, "clocks": clocks,
           "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu,
           "step_stats": step_stats, "forward_only": fwd_only, "gpu_serial": gpu_serial, "t_sweep": t_sweep, "stacked_state": stacked, "lstm": lstm, "roofline_by_class": roofline_by_class,
           "paper_context": "the paper reports up to 6.5x over serial training on 288 Xeon cores (32 MPI ranks x 9 threads) for T=128; "
                            "another machine and workload: context, not a target",
           "host_enqueue_ms_per_step": host_ms, "kernel_breakdown": breakdown, "kernel_by_size": by_size, "loss": float(loss.item()), "device_status": status}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
