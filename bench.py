#!/usr/bin/env python
"""Benchmark of the PairBalance ordering path.

A step is one balancing step of the whole path (difference forming, balancing core, running-sum
update, permutation slots) over one batch of synthetic stale gradients [2][m][d].  The default
workload is the GPT-2-small-sized one (m=64, n=128, d=124,000,000, bf16).

  python bench.py --gpus N --steps K --warmup W          native CUDA path (C ABI)
  python bench.py --impl reference ...                   the CPU oracle on a bounded sample

Prints ONE JSON line on rank 0.  With N > 1 (torchrun) every rank runs an independent replica
on its own GPU: the path does not shard (one shared running sum, sequential decisions).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2302_00845_b200 import synth  # noqa: E402

METRIC = "balanced_examples_per_sec"
UNIT = "examples/s"
L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic per launch from ncu captures (dram__bytes_read.sum + dram__bytes_write.sum),
# keyed by kernel kind and workload; valid only while the kernel source hash matches.
NCU_TRAFFIC: dict = {}   # filled below, after source_hash is defined


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="gpt2", choices=sorted(synth.WORKLOADS) + ["herding"])
    ap.add_argument("--herding-total", type=int, default=1_000_000, help="vectors of the herding study (all workers)")
    ap.add_argument("--herding-epochs", type=int, default=4)
    ap.add_argument("--herding-seeds", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kernel-events", action="store_true",
                    help="do not record per-kernel events inside the timed region")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--no-side-workloads", action="store_true",
                    help="skip the brief runs of the other configurations after the headline one")
    ap.add_argument("--oracle-child", default="", help=argparse.SUPPRESS)
    ap.add_argument("--independent", action="store_true",
                    help="ID-GraB (PairBal) mode: one running sum per worker (the uncoordinated baseline)")
    ap.add_argument("--d", type=int, default=0, help="override d (smaller cases for profiler captures)")
    ap.add_argument("--m", type=int, default=0, help="override m")
    return ap.parse_args()


def pick_workload(args) -> synth.Workload:
    wl = synth.WORKLOADS["tiny" if args.workload == "herding" else args.workload]
    if args.d:
        wl = wl.scaled(d=args.d, name=f"{wl.name}@d={args.d}")
    if args.m:
        wl = wl.scaled(m=args.m, name=f"{wl.name}@m={args.m}")
    return wl


# ------------------------------------------------------------------------------------------
def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 200 ms while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.lines = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "200",
                 "-i", str(index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = [l for (t, l) in self.lines if t0 <= t <= t1 + 0.3] or [l for (_, l) in self.lines]
        for l in rows:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); smax.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def algorithmic_bytes(kind: str, wl: synth.Workload) -> float:
    """Bytes one launch of a kernel kind must move: inputs once per pass; r read in pass 1,
    read and written in pass 2 (or once each in the fused step)."""
    inp = 2.0 * wl.m * wl.d * wl.elem_bytes
    if kind == "gram":
        return inp + 4.0 * wl.d
    if kind in ("update", "fused"):
        return inp + 8.0 * wl.d
    return 0.0


def aggregate_replicas(ms_local: float, examples_local: int, world: int, device: str):
    """Whole-job throughput of `world` independent replicas: every rank processed
    `examples_local` examples; the job's time is the slowest rank's (max over ranks).
    Returns (examples per second over all ranks, that time in ms)."""
    ms = ms_local
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([ms_local], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return examples_local * world / (ms * 1e-3), ms


def source_hash(files=None) -> str:
    """Hash of the kernel sources a traffic figure was captured with (all of csrc by default)."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2302_00845_b200", "csrc")
    for f in sorted(files or os.listdir(csrc)):
        h.update(open(os.path.join(csrc, f), "rb").read())
    return h.hexdigest()[:16]


# captured with ncu --set full (profiles/*.md); gpt2 figures were taken at d = 8,000,000 and are
# scaled by d to a full-size launch (traffic grows in proportion to d)
NCU_TRAFFIC.update({
    ("gram", "gpt2"): {"bytes": 2.089630e+09 * 15.5, "files": ["kernels_umma.cu", "ptx.cuh"], "source": "0c33b575267f3440"},
    ("update", "gpt2"): {"bytes": 2.112607e+09 * 15.5, "files": ["kernels_generic.cu"], "source": "ffc0c65e39a2c529"},
    # lstm: captured at d = 4,194,304, scaled by d
    ("gram", "lstm"): {"bytes": 5.576481e+08 * (13_500_000 / 4_194_304), "files": ["kernels_umma.cu", "ptx.cuh"], "source": "0c33b575267f3440"},
    ("update", "lstm"): {"bytes": 5.671585e+08 * (13_500_000 / 4_194_304), "files": ["kernels_generic.cu"], "source": "ffc0c65e39a2c529"},
    # mid, at full size.  Pass 2: bytes of a cold launch (ncu flushes L2 between replays)
    ("gram", "mid"): {"bytes": 1.445166e+08, "files": ["kernels_fma.cu", "ptx.cuh"], "source": "76d0347672d85fa9"},
    ("update", "mid"): {"bytes": 1.420818e+08, "files": ["kernels_generic.cu"], "source": "ffc0c65e39a2c529"},
})


# ------------------------------------------------------------------------------------------
def oracle_sample(wl, grads_dev, seconds: float):
    """The CPU oracle, as it stands, timed on a bounded sample: the pairs of the first workers of
    one step (at most 8 GB of rows copied to the host), balanced position after position with the
    running sum carried, until the time budget is used."""
    import oracle
    row_bytes = 2 * wl.d * wl.elem_bytes
    ms = int(max(1, min(wl.m, (8 << 30) // row_bytes)))
    host = [(synth.to_host(grads_dev[0, i]), synth.to_host(grads_dev[1, i])) for i in range(ms)]
    n_big = 1 << 20
    o = oracle.PairBalanceOracle(ms, n_big, wl.d)
    o.begin_epoch()
    done = 0
    t0 = time.perf_counter()
    while True:
        o.balance_one(done % ms, host[done % ms][0], host[done % ms][1])
        done += 1
        t_used = time.perf_counter() - t0
        if t_used >= seconds or done >= ms * (n_big // 2):
            break
    o.close()
    return {"value": 2.0 * done / t_used, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": f"{done} positions ({2 * done} examples) over the pairs of the first {ms} of "
                      f"{wl.m} workers at full d={wl.d}, running sum carried, {t_used:.1f} s"}


def run_reference(args):
    """The oracle timed on the host cores: each step is a bounded sample of a balancing step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    wl = pick_workload(args)
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    # sample: S workers per step, sized from one probe so the whole run ends within minutes
    S_cap = min(wl.m, 4)
    sub = wl.scaled(m=S_cap)
    gs = synth.GradientStream(sub, device=dev)
    g = gs.step(0)
    host = [(synth.to_host(g[0, i]), synth.to_host(g[1, i])) for i in range(S_cap)]
    probe = oracle.PairBalanceOracle(1, 2, wl.d)
    probe.begin_epoch()
    t0 = time.perf_counter()
    probe.balance_one(0, host[0][0], host[0][1])
    t_pos = time.perf_counter() - t0
    probe.close()
    total_steps = args.steps + args.warmup
    S = int(max(1, min(S_cap, 120.0 / max(t_pos * total_steps, 1e-9))))
    n_o = 2 * total_steps
    o = oracle.PairBalanceOracle(S, n_o, wl.d)
    o.begin_epoch()
    for _ in range(args.warmup):
        for i in range(S):
            o.balance_one(i, host[i][0], host[i][1])
    t0 = time.perf_counter()
    for _ in range(args.steps):
        for i in range(S):
            o.balance_one(i, host[i][0], host[i][1])
    dt = time.perf_counter() - t0
    o.close()
    value = 2.0 * S * args.steps / dt
    sample = (f"each step balances the first {S} of {wl.m} workers' pairs at full d={wl.d} "
              f"({wl.dtype}); same rows every step, running sum carried")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": wl.name, "m": wl.m, "n": wl.n, "d": wl.d,
                                        "storage": wl.dtype, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------
class Run:
    """One workload set up on the current device: handle, input buffers, the step closure."""

    def __init__(self, wl, local: int, independent: bool = False):
        from paper_2302_00845_b200 import binding
        self.independent = independent
        self.wl = wl
        m, n, d = wl.m, wl.n, wl.d
        self.step_bytes = 2 * m * d * wl.elem_bytes
        total_mem = torch.cuda.get_device_properties(local).total_memory
        self.nbuf = 2 if 2 * self.step_bytes < 0.5 * total_mem else 1
        # consecutive steps read different buffers: once those exceed L2 nothing survives between steps
        self.flush_mode = ("inputs_larger_than_l2" if self.step_bytes * self.nbuf >= 2 * L2_BYTES
                           else "l2_flush_between_steps")
        self.prob = None
        if wl.kind == "logreg":
            # gradients are produced on the device by the library's own kernel, every step
            self.prob = synth.LogregProblem(wl, device="cuda")
            self.bufs = [torch.empty(2, m, d, device="cuda") for _ in range(self.nbuf)]
        else:
            gs = synth.GradientStream(wl, device="cuda")
            self.bufs = [gs.step(k) for k in range(self.nbuf)]
        self.flush = (torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda")
                      if self.flush_mode != "inputs_larger_than_l2" else None)
        self.h = binding.CdGrab(m, n, d, wl.dtype, independent=independent)
        self.stream = torch.cuda.current_stream()
        self.state = {"step": 0}

    def one_step(self):
        h, wl, st = self.h, self.wl, self.state
        if st["step"] % (wl.n // 2) == 0:
            if st["step"]:
                h.end_epoch()
            h.begin_epoch()
        buf = self.bufs[st["step"] % self.nbuf]
        if self.prob is not None:
            h.logreg_grads(self.prob.X, self.prob.y, self.prob.w, buf)   # gradient kernel, then the step
        h.step(buf)                                                       # (faster than cdgrab_step_logreg)
        st["step"] += 1

    def timed_region(self, steps: int, barrier) -> float:
        """CUDA-event time of `steps` steps in ms (the L2 flushes between them are not timed)."""
        stream = self.stream
        if self.flush is None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            e0.record(stream)
            for _ in range(steps):
                self.one_step()
            e1.record(stream)
            barrier()
            return e0.elapsed_time(e1)
        evs = []
        barrier()
        for _ in range(steps):
            self.flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            self.one_step()
            b.record(stream)
            evs.append((a, b))
        barrier()
        return sum(a.elapsed_time(b) for a, b in evs)

    def measure(self, steps: int, warmup: int, barrier, want_events: bool):
        """Warm up, time `steps` steps, and time the kernels.  Per-kernel event pairs sit inside the
        timed region when a step is long enough not to notice them; a step of tens of microseconds
        would be slowed by the records themselves (and they keep a launch from queueing behind its
        predecessor), so there the kernels are timed over a second pass of the same steps."""
        h = self.h
        for _ in range(max(3, warmup)):
            self.one_step()
        barrier()
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record(self.stream)
        for _ in range(3):
            self.one_step()
        p1.record(self.stream)
        barrier()
        events_inside = want_events and p0.elapsed_time(p1) / 3 >= 1.0
        launches0 = h.launch_count
        if events_inside:
            h.profile_enable(True)
        t0 = time.time()
        ms = self.timed_region(steps, barrier)
        t1 = time.time()
        launches = h.launch_count - launches0
        prof = h.profile_read() if events_inside else {}
        h.profile_enable(False)
        if want_events and not events_inside:
            h.profile_enable(True)
            self.timed_region(steps, barrier)
            prof = h.profile_read()
            h.profile_enable(False)
        h.check_status()
        kernel_events = "none" if not want_events else ("timed_region" if events_inside else "second_pass_of_same_steps")
        return {"ms": ms, "launches": launches, "prof": prof, "kernel_events": kernel_events, "wall": (t0, t1)}

    def model_bytes(self) -> float:
        if self.independent:     # every worker has its own running sum: read twice, written once
            return 2.0 * self.step_bytes + 12.0 * self.wl.m * self.wl.d
        b2 = 2.0 * self.step_bytes + 12.0 * self.wl.d
        b1 = 1.0 * self.step_bytes + 8.0 * self.wl.d
        return b1 if self.h.path in ("fused", "literal") else b2

    def close(self):
        self.h.destroy()
        self.bufs = None
        self.flush = None
        self.prob = None
        torch.cuda.empty_cache()


NOMINAL_HBM_GBS = 8000.0     # the public HBM3e figure for the part, beside the measured copy rate


def roofline_of(prof: dict, wl, peak: float, peak_kind: str):
    """Roofline of the kernel with the largest summed time among the event pairs."""
    if not prof:
        return None
    dom = max(prof, key=lambda kname: prof[kname][0])
    tot_ms, cnt = prof[dom]
    avg_ms = tot_ms / cnt
    ab = algorithmic_bytes(dom, wl)
    achieved = ab / (avg_ms * 1e-3) / 1e9
    tr = NCU_TRAFFIC.get((dom, wl.name))
    traffic = tr["bytes"] if tr and tr.get("source") == source_hash(tr.get("files")) else None
    return {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "traffic": traffic, "peak_kind": peak_kind,
            "peak_nominal": NOMINAL_HBM_GBS, "frac_of_nominal": achieved / NOMINAL_HBM_GBS,
            "above_measured_peak": achieved > peak,   # the measured peak is a copy, not a bound on reads
            "avg_launch_ms": avg_ms, "algorithmic_bytes_per_launch": ab,
            "kernels": {kname: {"ms_total": v[0], "launches": v[1],
                                "share": v[0] / sum(x[0] for x in prof.values())}
                        for kname, v in prof.items()}}


# steps timed for the workloads reported beside the headline one (each well under two seconds)
SIDE_STEPS = {"tiny": 200, "logreg": 200, "mid": 400, "lstm": 100, "gpt2": 10}


def side_workloads(main_name: str, local: int, barrier, peak: float, with_oracle: bool):
    """The other configurations of the metric, each timed briefly on the same device: path, time
    per step, model bytes per second.  With the CPU-baseline leg on, the first steps of an epoch
    are also replayed through the oracle (near-tie count and raw sign agreement)."""
    out = []
    for name in ("tiny", "logreg", "mid", "lstm", "gpt2"):
        if name == main_name:
            continue
        wl = synth.WORKLOADS[name]
        free = torch.cuda.mem_get_info()[0]
        if 2.2 * 2 * wl.m * wl.d * wl.elem_bytes > free:
            out.append({"workload": name, "skipped": "not enough free device memory"})
            continue
        run = Run(wl, local)
        res = run.measure(SIDE_STEPS[name], 3, barrier, True)
        ms_step = res["ms"] / SIDE_STEPS[name]
        gbs = run.model_bytes() / (ms_step * 1e-3) / 1e9
        entry = {"workload": name, "m": wl.m, "n": wl.n, "d": wl.d, "storage": wl.dtype, "path": run.h.path,
                 "steps": SIDE_STEPS[name], "ms_per_step": ms_step, "cache": run.flush_mode,
                 "launches_per_step": res["launches"] / SIDE_STEPS[name],
                 "step_model_bytes": run.model_bytes(), "step_model_gbs": gbs, "frac_of_peak": gbs / peak,
                 "frac_of_nominal": gbs / NOMINAL_HBM_GBS,
                 "kernels_ms_per_launch": {k: v[0] / v[1] for k, v in res["prof"].items() if v[1]}}
        run.close()
        if with_oracle:
            entry.update(first_steps_vs_oracle(wl))
        out.append(entry)
    return out


def first_steps_vs_oracle(wl, seconds: float = 4.0):
    """Part of the CPU-baseline leg: the first steps of an epoch on the device and, on the same
    bytes, through the oracle in replay mode (it adopts the device's sign inside the tie band and
    counts those positions; its own signs give the raw agreement)."""
    import numpy as np
    import oracle
    from paper_2302_00845_b200 import binding
    tau = 1e-6 if wl.dtype == "f32" else 1e-3
    n_o = min(wl.n, 64)
    h = binding.CdGrab(wl.m, n_o, wl.d, wl.dtype)
    o = oracle.PairBalanceOracle(wl.m, n_o, wl.d)
    prob = synth.LogregProblem(wl.scaled(n=n_o), device="cuda") if wl.kind == "logreg" else None
    gs = None if prob is not None else synth.GradientStream(wl, device="cuda")
    buf = torch.empty(2, wl.m, wl.d, dtype=wl.torch_dtype, device="cuda")
    h.begin_epoch(); o.begin_epoch()
    t0 = time.perf_counter()
    k = 0
    equal = 0
    while k < n_o // 2:
        if prob is not None:
            h.logreg_grads(prob.X, prob.y, prob.w, buf)
        else:
            gs.step(k, out=buf)
        h.step(buf)
        s = h.signs()[:, k].cpu().numpy()
        o.step(synth.to_host(buf), replay=s, tau=tau)
        equal += int((o.own_signs()[:, k] == s).sum())
        k += 1
        if time.perf_counter() - t0 > seconds:
            break
    res = {"oracle_steps": k, "near_ties": o.near_ties, "mismatches_outside_band": o.mismatches,
           "raw_agreement": equal / float(k * wl.m)}
    h.destroy(); o.close()
    return res


def one_thread_oracle(name: str, seconds: float):
    """The oracle on one host thread (a child process, OMP_NUM_THREADS=1, inputs drawn on the CPU)."""
    env = dict(os.environ, OMP_NUM_THREADS="1", CUDA_VISIBLE_DEVICES="")
    try:
        res = subprocess.run([sys.executable, os.path.abspath(__file__), "--oracle-child", name,
                              "--cpu-seconds", str(seconds)], env=env, capture_output=True, text=True, timeout=300)
        return json.loads(res.stdout.strip().splitlines()[-1])
    except Exception as e:  # noqa: BLE001
        return {"workload": name, "error": str(e)[:200]}


def oracle_child(name: str, seconds: float):
    """Child of one_thread_oracle: times whole balancing steps of one workload on this process's threads."""
    import numpy as np
    import oracle
    wl = synth.WORKLOADS[name]
    n_o = min(wl.n, 64)
    if wl.kind == "logreg":
        prob = synth.LogregProblem(wl.scaled(n=n_o), device="cpu")
        X, y, w = prob.X.numpy(), prob.y.numpy(), prob.w.numpy()

        def step_rows(k):
            g = np.empty((2, wl.m, wl.d), dtype=np.float32)
            for i in range(wl.m):
                for q in range(2):
                    g[q, i] = oracle.logistic_grad(X[i, 2 * k + q], y[i, 2 * k + q], w).astype(np.float32)
            return g
        rows = [step_rows(k) for k in range(2)]
    else:
        gs = synth.GradientStream(wl, device="cpu")
        rows = [synth.to_host(gs.step(k)) for k in range(2)]
    o = oracle.PairBalanceOracle(wl.m, 1 << 20, wl.d)
    o.begin_epoch()
    done = 0
    t0 = time.perf_counter()
    while True:
        o.step(rows[done % 2])
        done += 1
        dt = time.perf_counter() - t0
        if dt >= seconds or done >= (1 << 19):
            break
    o.close()
    print(json.dumps({"workload": name, "value": 2.0 * wl.m * done / dt, "unit": UNIT, "cores": oracle.threads(),
                      "ms_per_step": 1e3 * dt / done, "steps": done}), flush=True)


def run_native(args):
    from paper_2302_00845_b200 import build
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    wl = pick_workload(args)
    m, n, d = wl.m, wl.n, wl.d
    run = Run(wl, local, independent=args.independent)
    h = run.h
    sampler = ClockSampler(local) if rank == 0 else None
    res = run.measure(args.steps, args.warmup, barrier, not args.no_kernel_events)
    clocks = sampler.stop(*res["wall"]) if sampler else None
    value, ms = aggregate_replicas(res["ms"], 2 * m * args.steps, world, "cuda")

    peak, peak_kind = peaks()
    roof = roofline_of(res["prof"], wl, peak, peak_kind)
    model = run.model_bytes()
    step_gbs = model / (ms / args.steps * 1e-3) / 1e9

    # ---- end to end through the host-buffer call ----------------------------------------------
    e2e = None
    if not args.no_e2e and world == 1:
        e2e = run_e2e(h, wl, run.bufs[0], run.state, run.one_step)

    cpu = None
    with_oracle = rank == 0 and world == 1 and not args.no_cpu_baseline
    if with_oracle:
        torch.cuda.synchronize()
        cpu = oracle_sample(wl, run.bufs[0], args.cpu_seconds)
    path, step_bytes, nbuf, flush_mode = h.path, run.step_bytes, run.nbuf, run.flush_mode
    run.close()

    # ---- the other configurations of the metric, briefly, after the headline one ---------------
    side = None
    if rank == 0 and world == 1 and not args.no_side_workloads and not args.d and not args.m and not args.independent:
        side = side_workloads(wl.name, local, barrier, peak, with_oracle)
        if with_oracle:
            cpu["one_thread"] = [one_thread_oracle(name, 3.0) for name in ("tiny", "logreg", "mid")]

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": {"workload": wl.name, "m": m, "n": n, "d": d, "storage": wl.dtype, "accumulate": "f32",
                       "path": path, "step_input_bytes": step_bytes, "input_buffers": nbuf,
                       "cache": flush_mode, "kernel_events": res["kernel_events"],
                       "parallelism": "replicas" if world > 1 else "single",
                       "order": "independent" if args.independent else "coordinated",
                       "step_model_bytes": model, "step_model_gbs": step_gbs,
                       "step_model_frac_of_peak": step_gbs / peak,
                       "step_model_frac_of_nominal": step_gbs / NOMINAL_HBM_GBS},
            "roofline": roof, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": res["launches"],
            "clocks": clocks, "workloads": side,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_herding(args):
    """The paper's synthetic herding study as a workload: N vectors ~ Unif[0,1)^16, centred and
    normalised, split over m in {5, 10, 20, 50, 100} workers; a few epochs of coordinated
    PairBalance orders (each epoch staged in HBM and balanced by one cdgrab_step_many call) against
    random reshuffling, the parallel herding objective (Eq. 7) evaluated on the device after every
    epoch.  One JSON line: value = balanced examples per second over all PairBalance epochs."""
    from paper_2302_00845_b200 import binding, build
    if int(os.environ.get("RANK", "0")) != 0:
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    build.build()
    N, d, E = args.herding_total, 16, args.herding_epochs
    table, total_ms, total_examples, launches = [], 0.0, 0, 0
    for m in (5, 10, 20, 50, 100):
        n = (N // m) & ~1
        rows = torch.arange(m, device="cuda")[:, None]
        for seed in range(args.herding_seeds):
            z = synth.herding_vectors(m * n, d, seed, "cuda").reshape(m, n, d)
            cur = synth.random_orders(m, n, 1000 * seed, "cuda")
            pb = [binding.herding_objective(z, cur)]
            rr = [pb[0]]
            out = torch.empty(m, n, dtype=torch.int32, device="cuda")
            ms = []
            with binding.CdGrab(m, n, d, "f32") as h:
                h.set_perms(cur.cpu().numpy())
                for ep in range(E):
                    # this epoch's gradients in visiting order, staged as [n/2][2][m][d]
                    g = z[rows, cur.long()].reshape(m, n // 2, 2, d).permute(1, 2, 0, 3).contiguous()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    before = h.launch_count
                    torch.cuda.synchronize()
                    e0.record()
                    h.begin_epoch()
                    h.step_many(g)
                    h.end_epoch(out)
                    e1.record()
                    torch.cuda.synchronize()
                    launches += h.launch_count - before
                    ms.append(e0.elapsed_time(e1))
                    cur = out.clone()
                    pb.append(binding.herding_objective(z, cur))
                    rr.append(binding.herding_objective(z, synth.random_orders(m, n, 1000 * seed + ep + 1, "cuda")))
                h.check_status()
                path = h.path
            total_ms += sum(ms)
            total_examples += E * m * n
            table.append({"m": m, "n": n, "seed": seed, "path": path, "pairbalance": pb, "random_reshuffling": rr,
                          "ms_per_epoch": sum(ms) / E, "us_per_step": 1e3 * sum(ms) / E / (n // 2)})
    line = {"metric": METRIC, "value": total_examples / (total_ms * 1e-3), "unit": UNIT, "n_gpus": 1,
            "steps": E * len(table), "warmup": 0, "ms_per_step": total_ms / (E * len(table)), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "herding", "total_vectors": N, "d": d, "epochs": E, "seeds": args.herding_seeds,
                       "step": "one epoch of PairBalance orders (cdgrab_begin_epoch, cdgrab_step_many over n/2 staged "
                               "steps, cdgrab_end_epoch)"},
            "gpu_launches": launches, "herding": table}
    print(json.dumps(line), flush=True)


def run_e2e(h, wl, dev_buf, state, one_step):
    """Same metric through cdgrab_step_host: every step copies its [2][m][d] input from pinned host
    memory and reads the sign table back."""
    import psutil
    from paper_2302_00845_b200 import binding  # noqa: F401
    step_bytes = 2 * wl.m * wl.d * wl.elem_bytes
    if psutil.virtual_memory().available < 2.5 * step_bytes:
        return {"value": None, "unit": UNIT, "h2d_bytes_per_step": step_bytes, "d2h_bytes_per_step": 0,
                "note": "not enough host memory for a pinned copy of one step"}
    host = torch.empty(dev_buf.shape, dtype=dev_buf.dtype, pin_memory=True)
    host.copy_(dev_buf)
    staging = torch.empty_like(dev_buf)
    signs_host = torch.empty(wl.m, wl.n // 2, dtype=torch.int8, pin_memory=True)
    stream = torch.cuda.current_stream()
    lib = binding.lib()
    steps = 3 if step_bytes > (1 << 30) else 10

    def e2e_step():
        if state["step"] % (wl.n // 2) == 0:
            if state["step"]:
                h.end_epoch()
            h.begin_epoch()
        h.step_host(host, staging)
        state["step"] += 1
        rc = lib.cdgrab_get_signs(h._h, signs_host.data_ptr(), stream.cuda_stream)
        assert rc == 0
        stream.synchronize()  # the caller reads the step's result

    e2e_step()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        e2e_step()
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    return {"value": 2.0 * wl.m * steps / dt, "unit": UNIT, "h2d_bytes_per_step": step_bytes,
            "d2h_bytes_per_step": wl.m * (wl.n // 2), "steps": steps, "ms_per_step": 1e3 * dt / steps}


def main():
    args = parse_args()
    if args.oracle_child:
        oracle_child(args.oracle_child, args.cpu_seconds)
    elif args.workload == "herding" and args.impl == "native":
        run_herding(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_native(args)


if __name__ == "__main__":
    main()
