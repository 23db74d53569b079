#!/usr/bin/env python
"""Benchmark of the LapSum forward+backward hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c5] [--impl reference]

A step is one lapsum_forward + lapsum_backward over one batch of the named
workload (default c5: one row of 10^8 scores, k = 20000, alpha = -0.02, the
configuration the headline metric is quoted on).  One JSON line is printed by
rank 0.  With --gpus N > 1 (launched through torch.distributed.run) every rank
runs an independent replica of the workload (the solver has no cross-GPU data
path), timed as the maximum over ranks.

--impl reference times the CPU oracle (oracle/) instead, each step on a
bounded sample of the same workload.
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

METRIC = "fwd+bwd scores/s"
UNIT = "scores/s"
# algorithmic bytes per score (fp32): forward = read r for the stream pass + read r and write p for the mask;
# backward = read (r, v) for the reduction + read (r, v) and write grad
BYTES_PER_SCORE = {"stream_band": 4, "cdf_map": 8, "vjp_reduce": 8, "vjp_map": 12, "row_block_forward": 8,
                   "row_block_backward": 12, "rs_onesweep": 8, "rs_histogram": 4, "tile_aggregate": 4}
L2_BYTES = 126 * 1024 * 1024
# DRAM bytes per score of the dominant kernels, from one ncu capture each (dram__bytes_read.sum +
# dram__bytes_write.sum divided by the scores of the captured launch; pure streams, so traffic scales with n).
# Source: the ncu full-set capture of the bracket-path kernels at n = 5e7, summarised with the other profiles.
NCU_TRAFFIC_PER_SCORE = {"vjp_map": (400.0 + 157.7) / 50.0, "cdf_map": (200.0 + 144.7) / 50.0,
                         "vjp_reduce": (400.0 + 3.7) / 50.0, "stream_band": (200.4 + 4.8) / 50.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Polls SM clock, power and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.stop_flag, self.ok = [], threading.Event(), False
        try:
            import pynvml

            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_sm = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.max_sm = None

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self.stop_flag.is_set():
            try:
                sm = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                power = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                self.samples.append((time.perf_counter(), sm, reasons, power))
            except Exception:
                pass
            time.sleep(self.period)

    def summary(self, t0: float, t1: float):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_sm, "reasons": ["unavailable"], "samples": 0}
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        window = "timed region"
        if len(inside) < 3:
            inside, window = self.samples, "warm-up + timed region"
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
        }
        seen = set()
        for s in inside:
            for bit, name in names.items():
                if s[2] & bit:
                    seen.add(name)
        return {"sm_mhz": float(np.median([s[1] for s in inside])), "sm_max_mhz": self.max_sm,
                "reasons": sorted(seen), "power_w_max": max(s[3] for s in inside), "samples": len(inside),
                "window": window}


def cpu_model() -> str:
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def oracle_step(O, r, v, k, alpha):
    f = O.forward(r, k, alpha)
    O.backward(v, r, f.b, alpha)


def cpu_baseline(w, r, v, budget_n: int):
    """The oracle as it stands, one thread, on a bounded prefix of the same workload."""
    from oracle import lapsum_oracle as O

    if w.rows > 1:
        rows = max(1, min(w.rows, budget_n // w.n))
        rs, vs, k = r[:rows], v[:rows], w.k
        sample = f"first {rows} of {w.rows} rows, n={w.n}, k={w.k:g}"
        scores = rows * w.n
    else:
        m = min(w.n, budget_n)
        k = w.k if m == w.n else max(1.0, round(w.k * m / w.n))
        rs, vs = r[:, :m], v[:, :m]
        sample = (f"the whole row of {w.n} scores, k={k:g}, one forward+backward" if m == w.n else
                  f"first {m} of {w.n} scores of the row, k scaled to {k:g} (same k/n)")
        scores = m
    O.lib()
    t0 = time.perf_counter()
    oracle_step(O, rs, vs, k, w.alpha)
    dt = time.perf_counter() - t0
    return {"value": scores / dt, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
            "seconds": round(dt, 3), "host_cores": os.cpu_count(), "cpu_model": cpu_model()}


def run_reference(args, w):
    from paper_2608_06912_b200 import inputs as I
    from oracle import lapsum_oracle as O

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    O.lib()
    m = min(w.n, 2_000_000) if w.rows == 1 else w.n
    rows = 1 if w.rows == 1 else max(1, min(w.rows, 2_000_000 // w.n))
    ws = I.scaled(w, m) if w.rows == 1 and m != w.n else w
    r = I.make_scores(ws)[:rows]
    v = I.make_upstream(ws)[:rows]
    scores = rows * ws.n
    for _ in range(args.warmup):
        oracle_step(O, r, v, ws.k, ws.alpha)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(O, r, v, ws.k, ws.alpha)
    dt = time.perf_counter() - t0
    ms = dt / args.steps * 1e3
    value = scores / (ms * 1e-3)
    sample = (f"each step: oracle forward+backward on {rows} row(s) of {ws.n} scores "
              f"(k={ws.k:g}, alpha={ws.alpha:g}), the {w.name} recipe at reduced size")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "rows": w.rows, "n": w.n, "k": w.k, "alpha": w.alpha, "recipe": w.recipe,
                   "sampled": {"rows": rows, "n": ws.n, "k": ws.k}},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                         "host_cores": os.cpu_count(), "cpu_model": cpu_model()},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="c5")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-baseline-scores", type=int, default=100_000_000)
    ap.add_argument("--rows", type=int, default=0, help="run only the first ROWS rows of a batched workload")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--path", default="auto", choices=["auto", "block", "fullsort", "bracket"])
    ap.add_argument("--sort-payload", action="store_true", help="radix sorts carry the index payload (76 B/score)")
    ap.add_argument("--band-capacity", type=int, default=0, help="scores the middle-band buffer holds (0: the library's default)")
    ap.add_argument("--dtype", default="f32", choices=["f32", "f16", "bf16"],
                    help="storage type of scores, upstream gradient, mask and gradient (arithmetic stays fp32)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    from paper_2608_06912_b200 import inputs as I

    base = args.config.split("@")[0]
    w = I.WORKLOADS[base]
    if "@" in args.config:
        w = I.scaled(w, int(float(args.config.split("@")[1])))
    full_rows = w.rows
    if args.rows and args.rows < w.rows:
        import dataclasses as _dc

        w = _dc.replace(w, rows=args.rows)

    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch

    import paper_2608_06912_b200 as L
    from paper_2608_06912_b200 import dist as D

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product has no CPU path")
    rank, local_rank, world = D.init("nccl")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world != args.gpus and rank == 0:
        print(f"note: --gpus {args.gpus} but WORLD_SIZE={world}; using {world}", file=sys.stderr)

    # every rank runs an independent replica of the workload (its own seeds): weak scaling, no data-path collective
    import dataclasses

    wr = w if rank == 0 else dataclasses.replace(w, seed_r=w.seed_r + 101 * rank, seed_v=w.seed_v + 101 * rank)
    if w.rows != full_rows:   # a slice of a batched workload: draw the whole batch, keep its first rows
        wfull = dataclasses.replace(wr, rows=full_rows)
        r_np = np.ascontiguousarray(I.make_scores(wfull)[: w.rows])
        v_np = np.ascontiguousarray(I.make_upstream(wfull)[: w.rows])
    else:
        r_np, v_np = I.make_scores(wr), I.make_upstream(wr)
    io = {"f32": L.IO_F32, "f16": L.IO_F16, "bf16": L.IO_BF16}[args.dtype]
    esz = 4 if io == L.IO_F32 else 2
    r_pin = torch.from_numpy(r_np).to(L.IO_TORCH[io]).pin_memory()   # 16-bit runs: the scores rounded to the storage type
    v_pin = torch.from_numpy(v_np).to(L.IO_TORCH[io]).pin_memory()
    if io != L.IO_F32:   # what the CPU baseline is given: the same values, up-converted (exact)
        r_np, v_np = r_pin.float().numpy(), v_pin.float().numpy()
    r = r_pin.to(dev)
    v = v_pin.to(dev)
    p = torch.empty_like(r)
    g = torch.empty_like(r)
    b = torch.empty(w.rows, device=dev)
    force = {"auto": L.PATH_AUTO, "block": L.PATH_BLOCK, "fullsort": L.PATH_FULLSORT, "bracket": L.PATH_BRACKET}[args.path]
    prm = L.default_params(force_path=force, sort_payload=1 if args.sort_payload else 0, io_dtype=io,
                           band_capacity=args.band_capacity)
    ws = L.Workspace(w.rows, w.n, prm, seed=w.seed_sampler)
    stream = torch.cuda.current_stream()

    def fwd():
        L.lapsum_forward_io(r, None, None, w.k, w.alpha, p, b, ws, stream)

    def bwd():
        L.lapsum_backward_io(v, r, b, None, w.alpha, g, None, None, ws, stream)

    def step():
        fwd()
        bwd()

    resident = 4 * esz * w.scores
    flush = resident <= 2 * L2_BYTES * 2  # working set (r, v, p, grad) comparable to L2: flush between steps
    flush_buf = torch.empty(512 * 1024 * 1024, dtype=torch.uint8, device=dev) if flush else None

    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    st0 = ws.status()
    path = L.PATH_NAMES[st0.path]
    dominant = {"bracket": "vjp_map", "fullsort": "rs_onesweep", "block": "row_block_forward"}[path]
    L.lapsum_profile_enable(ws, [dominant], max_records=max(16, args.steps * (8 if path == "fullsort" else 2)))

    ev0 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps if flush else 1)]
    ev1 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps if flush else 1)]
    launches0 = L.lapsum_launch_count()
    D.barrier()
    torch.cuda.synchronize()
    t_host0 = time.perf_counter()
    if flush:
        for i in range(args.steps):
            flush_buf.fill_(i & 255)  # untimed: evicts the previous step's lines from L2
            ev0[i].record(stream)
            step()
            ev1[i].record(stream)
    else:
        ev0[0].record(stream)
        for _ in range(args.steps):
            step()
        ev1[0].record(stream)
    torch.cuda.synchronize()
    t_host1 = time.perf_counter()
    D.barrier()
    launches = L.lapsum_launch_count() - launches0
    total_ms = sum(a.elapsed_time(z) for a, z in zip(ev0, ev1))
    total_ms = D.max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / args.steps
    value = world * w.scores / (ms_per_step * 1e-3)
    prof = L.lapsum_profile_read(ws, stream)
    L.lapsum_profile_disable(ws)
    sampler.stop_flag.set()
    sampler.join(timeout=2)
    clocks = sampler.summary(t_host0, t_host1)
    st = ws.status()

    peak, peak_kind = load_peaks()
    k_launches, k_ms = prof.get(dominant, (0, 0.0))
    units = w.n if path != "block" else w.scores
    alg_bytes = BYTES_PER_SCORE[dominant] * units * esz // 4
    avg_ms = k_ms / max(1, k_launches)
    achieved = alg_bytes / (avg_ms * 1e-3) / 1e9 if k_launches else None
    if path == "fullsort":
        alg_bytes = (16 if args.sort_payload else 8) * units  # keys are 32-bit whatever the storage type; with payload (key, index) pairs
    traffic = (NCU_TRAFFIC_PER_SCORE[dominant] * units if dominant in NCU_TRAFFIC_PER_SCORE and path == "bracket"
               and io == L.IO_F32 else None)
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": (achieved / peak) if achieved else None, "traffic": traffic,
                "traffic_source": ("ncu capture of this kernel at n = 5e7, scaled by n"
                                   if traffic else None),
                "peak_kind": f"of {peak_kind}",
                "algorithmic_bytes_per_launch": alg_bytes, "avg_launch_ms": avg_ms, "launches_timed": k_launches}
    if traffic and k_launches:
        # what the DRAM really moved (ncu) over the same launch time: below `achieved` where the back-to-front second
        # passes find the tail of the row still in L2
        roofline["dram_gbs"] = traffic / (avg_ms * 1e-3) / 1e9
        roofline["dram_frac"] = roofline["dram_gbs"] / peak
    # whole-step view: algorithmic bytes of forward + backward over the step time.  Full sort: histogram 4 + four
    # passes of 8 (keys only; 12 + 3 x 16 with the index payload) + tile aggregates 4 + mask 8, backward 20.
    fullsort_bytes = (76 if args.sort_payload else 48) + 20
    if io != L.IO_F32:  # 16-bit storage halves every read of r, v and every write of p, grad; sort keys stay 32-bit
        fullsort_bytes = (2 + (10 if args.sort_payload else 6) + (48 if args.sort_payload else 24) + 4 + 4) + 10
    step_bytes = {"bracket": 32 * esz // 4, "fullsort": fullsort_bytes, "block": 20 * esz // 4}[path] * w.scores
    roofline["step_algorithmic_bytes_per_score"] = step_bytes // w.scores
    roofline["step_algorithmic_gbs"] = step_bytes / (ms_per_step * 1e-3) / 1e9
    roofline["step_frac"] = roofline["step_algorithmic_gbs"] / peak

    # untimed second pass: per-step times for the median, and forward / backward apart
    reps = max(5, min(args.steps, 50))
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(reps)]
    for i in range(reps):
        if flush:
            flush_buf.fill_(i & 255)
        evs[i][0].record(stream)
        fwd()
        evs[i][1].record(stream)
        bwd()
        evs[i][2].record(stream)
    torch.cuda.synchronize()
    fwd_ms = [e[0].elapsed_time(e[1]) for e in evs]
    bwd_ms = [e[1].elapsed_time(e[2]) for e in evs]
    tot_ms = [e[0].elapsed_time(e[2]) for e in evs]
    split = {"steps": reps, "step_ms_median": float(np.median(tot_ms)), "step_ms_mean": float(np.mean(tot_ms)),
             "forward_ms_median": float(np.median(fwd_ms)), "forward_ms_mean": float(np.mean(fwd_ms)),
             "backward_ms_median": float(np.median(bwd_ms)), "backward_ms_mean": float(np.mean(bwd_ms)),
             "what": "a second, untimed pass with events between the two calls of every step"}

    # per-kernel breakdown of one untimed pass (events around every kernel)
    L.lapsum_profile_enable(ws, None, max_records=512)
    for _ in range(3):
        step()
    breakdown = {name: {"launches": n // 3, "ms_per_step": ms / 3} for name, (n, ms) in
                 L.lapsum_profile_read(ws, stream).items()}
    L.lapsum_profile_disable(ws)

    e2e = None
    if not args.no_e2e and io == L.IO_F32:  # the host-buffer entry point serves fp32 storage
        p_pin = torch.empty_like(r_pin).pin_memory()
        g_pin = torch.empty_like(r_pin).pin_memory()
        b_pin = torch.empty(w.rows).pin_memory()
        staging = torch.empty(4 * w.scores + w.rows, device=dev)

        def e2e_step():
            # the library's host-buffer call: copies in, forward, backward, copies out, all enqueued on `stream`
            L.lapsum_forward_backward_host(r_pin, v_pin, w.k, w.alpha, p_pin, g_pin, b_pin, staging, ws, stream)

        e2e_step()
        torch.cuda.synchronize()
        D.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.e2e_steps):
            e2e_step()
        e1.record(stream)
        torch.cuda.synchronize()
        D.barrier()
        e_ms = D.max_over_ranks(e0.elapsed_time(e1), dev) / args.e2e_steps
        e2e = {"value": world * w.scores / (e_ms * 1e-3), "unit": UNIT, "ms_per_step": e_ms,
               "h2d_bytes_per_step": 2 * 4 * w.scores, "d2h_bytes_per_step": 2 * 4 * w.scores + 4 * w.rows,
               "steps": args.e2e_steps,
               "what": "lapsum_forward_backward_host: pinned host r, v -> device, forward + backward, p, grad, b -> pinned host"}
        assert torch.isfinite(b_pin).all()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(w, r_np, v_np, args.cpu_baseline_scores)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "ms_per_step_median": split["step_ms_median"],
            "forward_ms": split["forward_ms_median"], "backward_ms": split["backward_ms_median"], "split": split,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "io_dtype": args.dtype, "data": "synthetic",
            "config": {"workload": w.name + ("" if io == L.IO_F32 else "_" + args.dtype), "rows": w.rows, "n": w.n, "k": w.k, "alpha": w.alpha, "recipe": w.recipe,
                       "path": path, "parallelism": "replicas" if world > 1 else "single",
                       "storage": args.dtype + " scores, upstream gradient, mask and gradient; fp32 arithmetic and thresholds",
                       "l2": ("512 MiB scratch written between timed steps (L2 flush)" if flush else
                              f"inputs (r, v, p, grad: {esz * w.scores // 10**6} MB each) exceed the 126 MB L2, no flush")},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu,
            "kernels": breakdown,
            "solver": {"fallbacks": st.fallbacks, "status_bits": st.status_bits, "n_M": st.n_M, "K": st.K,
                       "lookback_timeouts": st.lookback_timeouts, "b": float(b[0].item())},
        }
        print(json.dumps(line), flush=True)
    D.finalize()


if __name__ == "__main__":
    main()
