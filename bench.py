#!/usr/bin/env python
"""Benchmark of the parameter-server update path: updates/s and achieved HBM bandwidth.

One step = one update window of the learner event stream: the c = floor(lambda/n) pushGradient
messages of a group, the fused sumGradients + applyUpdate launch, and the pullWeights copies the
learners of that window make.  Default workload: the ImageNet-scale model (60 965 224 fp32
weights, lambda = 54, n = 18, c = 3, momentum 0.9, weight decay 5e-4) on synthetic gradient
streams, one distinct buffer per learner so every byte comes from HBM.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

With N > 1 (under torchrun) every rank runs an independent replica of the server: the path has
no exchange step on one node, so there is no collective in the timed region.
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

from paper_1509_04210_b200 import synth  # noqa: E402

METRIC = "ps_updates_per_sec"
UNIT = "updates/s"
FALLBACK_HBM_GBS = 6650.0


# DRAM traffic of one launch, from ncu captures summarised under profiles/ (dram__bytes_read.sum +
# dram__bytes_write.sum).  The windowed update kernel was captured on a smaller vector with the same
# launch shape (the full-size launch holds 26 GB of distinct buffers) and is scaled by the vector
# length; the copy and leaf kernels were captured at full size.  Each record is valid only for the
# kernel sources it was taken on.
NCU_TRAFFIC = {
    # (kernel, workload, updates, gradient vectors, weight copies)
    ("update", "imagenet", 18, 54, 54): {"bytes_per_weight": 438.71, "sources": ("update.cu", "kernels.cuh", "vec.cuh"),
                                         "sha": "9bd3787d26f56bbe", "source": "profiles/update_kernel_imagenet_window18.md"},
    # (kernel, destinations)
    ("snapshot", 1): {"bytes_per_launch_at": (60965224, 433.7e6), "sources": ("snapshot.cu", "kernels.cuh"),
                      "sha": "a821be77c12fccc9", "source": "profiles/snapshot_kernel_imagenet_pull.md"},
    # (kernel, fan-in, bytes per gradient element)
    ("leaf", 3, 4): {"bytes_per_launch_at": (60965224, 926.5e6), "sources": ("leaf.cu", "kernels.cuh", "vec.cuh"),
                     "sha": "aac70d5e74ad45de", "source": "profiles/leaf_average_kernel_imagenet_fanin3.md"},
}


def sources_sha(files):
    import hashlib

    h = hashlib.sha256()
    for f in files:
        with open(os.path.join(ROOT, "paper_1509_04210_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def kernel_sources_sha():
    return sources_sha(("update.cu", "kernels.cuh", "vec.cuh"))


def ncu_traffic(key, nparams):
    """Bytes per launch from the recorded capture, or None if there is none for this kernel and
    launch shape or the kernel's sources have changed since."""
    rec = NCU_TRAFFIC.get(key)
    if rec is None or rec["sha"] != sources_sha(rec["sources"]):
        return None
    if "bytes_per_launch_at" in rec:
        n, b = rec["bytes_per_launch_at"]
        return float(b) if n == nparams else None
    return rec["bytes_per_weight"] * nparams


def measured_hbm_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


ADAGRAD = False   # set from --optimizer


def state_bytes(w):
    """Read + write of the weights, and of the state vector when the rule keeps one (velocity with
    momentum, squared-gradient sum with AdaGrad)."""
    return 16 if (w.momentum != 0.0 or ADAGRAD) else 8


def update_bytes_per_param(w):
    """Algorithmic bytes one update moves per weight: c gradient reads + weights and state."""
    g = 2 if w.grad_dtype == synth.GRAD_BF16 else 4
    return w.c * g + state_bytes(w)


EV_PUSH, EV_STEP, EV_PULL, EV_PULL_SKIP, EV_BROADCAST = 1, 2, 3, 4, 5


def make_windows(w, count, seed=synth.MASTER_SEED, from_oracle=False, fanin=0):
    """Event windows (arrays of event records): a window runs from the first push of a group to
    the last pull before the next group's first push.  The CUDA arm takes the events from the
    library's scheduler, the reference arm from the oracle's."""
    if from_oracle:
        from oracle import rudra_oracle as ora

        osched = ora.OracleScheduler(w.lam, w.n, w.mode, seed, w.lognormal_sigma, w.downcast, fanin)
        more = lambda k: osched.run(k)
    else:
        from paper_1509_04210_b200 import binding as rb

        sched = rb.Scheduler(w.lam, w.n, w.mode, seed, w.lognormal_sigma, w.downcast, fanin)
        more = lambda k: sched.next(k)
    windows, cur, stepped = [], [], False
    while len(windows) < count:
        for ev in more(4096):
            if ev["kind"] == EV_PUSH and stepped:
                windows.append(np.array(cur, dtype=ev.dtype))
                cur, stepped = [], False
                if len(windows) == count:
                    break
            cur.append(ev)
            if ev["kind"] == EV_STEP:
                stepped = True
    return windows


def default_window(w, views=False):
    """Updates packed into one launch by default: the gradients lambda learners can have waiting at
    once make n = lambda / c updates (every learner blocks on its push until the server has taken
    it), capped by the launch tables (32 updates, 128 gradients, 128 pull destinations; with
    zero-copy pulls a version is one destination however many learners take it)."""
    pulls_per_update = 1 if views else (w.lam if (w.downcast or w.mode == synth.HARDSYNC) else w.c)
    return max(1, min(w.n, 32, 128 // w.c, 128 // pulls_per_update))


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons while the timed region runs (read-only NVML queries)."""

    def __init__(self, index, period=0.005):
        super().__init__(daemon=True)
        self.period, self.samples, self.reasons, self.max_mhz = period, [], set(), None
        self._halt = threading.Event()
        self._h = None
        try:
            import pynvml

            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def run(self):
        if self._h is None:
            return
        nv = self._nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._halt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._halt.set()
        self.join(timeout=2.0)
        return {
            "sm_mhz": float(np.median(self.samples)) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


def visible_gpu_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ---------------------------------------------------------------------------------------------
# CPU oracle legs (the reported baseline and the --impl reference arm)
# ---------------------------------------------------------------------------------------------
def oracle_run(w, windows, nsample, grads_host, warmup=0, budget_s=None, max_windows=None, adagrad=False, keep=None):
    """Times the oracle, as it stands, over event windows (from the start of the event stream) on
    the first nsample weights; the first ``warmup`` windows run untimed.  keep: a list that receives
    the oracle server, so that the caller can compare its weights with the library's."""
    from oracle import rudra_oracle as ora

    ps = ora.OraclePS(nsample, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
    ps.set_grad_dtype(w.grad_dtype)
    if adagrad:
        ps.set_optimizer(ora.OPT_ADAGRAD, 1e-8)
    ps.set_weights(synth.initial_weights(nsample, w.theta_std))
    done, t0 = -warmup, time.perf_counter()
    for win in windows:
        if done == 0:
            t0 = time.perf_counter()
        for kind, learner, pulled_ts in zip(win["kind"].tolist(), win["learner"].tolist(), win["pulled_ts"].tolist()):
            if kind == ora.PUSH:
                ps.push(grads_host[learner % len(grads_host)], pulled_ts)
            elif kind == ora.STEP:
                ps.step()
            elif kind == ora.PULL:
                ps.pull()
            elif kind == ora.BROADCAST:
                for _ in range(w.lam):
                    ps.pull()
        done += 1
        if max_windows is not None and done >= max_windows:
            break
        if budget_s is not None and time.perf_counter() - t0 >= budget_s:
            break
    dt = time.perf_counter() - t0
    if keep is not None:
        keep.append(ps)
    return done, dt


def oracle_run_all_cores(w, windows, grads_host, cores, budget_s, adagrad=False):
    """The same oracle, one unmodified single-threaded instance per core on disjoint slices of the
    vector (the path is element-wise, so slicing changes nothing); returns (windows done, seconds)."""
    import threading as th

    n = len(grads_host[0])
    bounds = [n * i // cores for i in range(cores + 1)]
    results = [None] * cores
    # fix the number of windows from a short probe so that all threads do the same work
    probe_done, probe_dt = oracle_run(w, windows, min(n, 1 << 20), [g[: 1 << 20] for g in grads_host], warmup=0,
                                      max_windows=2, adagrad=adagrad)
    per_window = probe_dt / probe_done * (n / cores) / min(n, 1 << 20)
    todo = max(2, min(len(windows), int(budget_s / max(per_window, 1e-9))))

    def work(i):
        sl = [np.ascontiguousarray(g[bounds[i]: bounds[i + 1]]) for g in grads_host]
        results[i] = oracle_run(w, windows, bounds[i + 1] - bounds[i], sl, warmup=0, max_windows=todo, adagrad=adagrad)

    threads = [th.Thread(target=work, args=(i,)) for i in range(cores)]
    t0 = time.perf_counter()
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    return todo, time.perf_counter() - t0


def host_gradients(w, nsample, count):
    return [synth.gradient(nsample, l, 0, w.grad_std, w.grad_dtype) for l in range(count)]


def run_reference(args, w):
    """--impl reference: the CPU oracle on the same workload, metric and unit."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import rudra_oracle as ora

    ora.build()
    # Each step handles a bounded sample of the vector so that the whole run ends within a few
    # minutes whatever --steps is: about 75 s of oracle work at ~60 M weight-updates per second
    # and core, never more than a quarter of a large vector.
    nsample = w.nparams
    if w.nparams > (1 << 22):
        per_step = int(75.0 * 60e6 / (args.steps + args.warmup) / max(w.c, 1) * 3)
        nsample = max(1 << 16, min(w.nparams // 4, per_step))
    windows = make_windows(w, args.warmup + args.steps, from_oracle=True)
    grads = host_gradients(w, nsample, min(w.lam, 8))
    done, dt = oracle_run(w, windows, nsample, grads, warmup=args.warmup, adagrad=args.optimizer == "adagrad")
    frac = nsample / w.nparams
    value = done / dt * frac
    sample = "first %d of %d weights (%.0f%%), %d distinct host gradient buffers, rate scaled by the fraction" % (
        nsample, w.nparams, 100 * frac, len(grads))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 / value, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                         "cpu_model": cpu_model()},
        "timed_seconds": dt, "timed_windows": done, "sample_fraction": frac,
        "ms_per_step_note": "ms_per_step is 1000 / value, the time a full-size window would take at the sampled rate; "
                            "the run itself timed %d windows of the sample in %.1f s" % (done, dt),
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def workload_config(w):
    return {
        "workload": w.name, "nparams": w.nparams, "lambda": w.lam, "n": w.n, "c": w.c, "alpha0": w.alpha0,
        "momentum": w.momentum, "weight_decay": w.weight_decay,
        "grad_dtype": "bf16" if w.grad_dtype == synth.GRAD_BF16 else "f32",
        "scheduler": {0: "hardsync", 1: "softsync_rounds", 2: "softsync_timed"}[w.mode],
        "l2": ("inputs larger than L2 (one distinct %.0f MB gradient buffer per learner, %.0f MB of weights and state)"
               % (w.nparams * (2 if w.grad_dtype == synth.GRAD_BF16 else 4) / 1e6, w.nparams * 8 / 1e6))
              if w.nparams * 8 > 126e6 else "weights and state fit in L2: launch-bound workload, no HBM roofline claim",
        "parallelism": "replicas",
    }


# ---------------------------------------------------------------------------------------------
# the CUDA arm
# ---------------------------------------------------------------------------------------------
def link_probe(torch, pinned_src, pinned_dst, reps=6):
    """GB/s per direction of plain pinned-memory copies over the host link, a host-to-device and a
    device-to-host copy in flight at the same time on two streams: the ceiling of the end-to-end leg."""
    n = min(pinned_src.numel() * pinned_src.element_size(), pinned_dst.numel() * pinned_dst.element_size())
    src = pinned_src.view(torch.uint8)[:n]
    dst = pinned_dst.view(torch.uint8)[:n]
    d_in = torch.empty(n, dtype=torch.uint8, device="cuda")
    d_out = torch.empty(n, dtype=torch.uint8, device="cuda")
    up, down = torch.cuda.Stream(), torch.cuda.Stream()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    torch.cuda.synchronize()
    for timed in (False, True):
        if timed:
            ev[0].record(up)
            ev[2].record(down)
        for _ in range(reps if timed else 1):
            with torch.cuda.stream(up):
                d_in.copy_(src, non_blocking=True)
            with torch.cuda.stream(down):
                dst.copy_(d_out, non_blocking=True)
        if timed:
            ev[1].record(up)
            ev[3].record(down)
        torch.cuda.synchronize()
    return {"h2d_gbs": n * reps / (ev[0].elapsed_time(ev[1]) * 1e-3) / 1e9,
            "d2h_gbs": n * reps / (ev[2].elapsed_time(ev[3]) * 1e-3) / 1e9,
            "how": "plain copies of one %.0f MB pinned buffer each way at the same time, %d repetitions" % (n / 1e6, reps)}


def parity_with_oracle(rb, torch, w, windows, grads_host, oracle_ps, W, stream):
    """Runs ``windows`` (from the start of the event stream) through the library on device copies of
    the oracle's own inputs and compares the whole weight and state vectors with the oracle's."""
    N = w.nparams
    ps = rb.ParameterServer(N, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
    ps.set_option(rb.OPT_GRAD_DTYPE, w.grad_dtype)
    if ADAGRAD:
        ps.set_option(rb.OPT_OPTIMIZER, rb.OPTIM_ADAGRAD)
    ps.set_weights(torch.from_numpy(synth.initial_weights(N, w.theta_std)).cuda())
    ps.sync()
    ps.set_stream(stream)
    dev = [torch.from_numpy(g.view(np.int16) if g.dtype == np.uint16 else g).cuda() for g in grads_host]
    slots = [torch.empty(N, dtype=torch.float32, device="cuda") for _ in range(len(dev))]
    gtable = rb.pointer_table([dev[l % len(dev)] for l in range(w.lam)])
    stable = rb.pointer_table([slots[l % len(slots)] for l in range(w.lam)])
    step = max(W, 1)
    updates = 0
    for i in range(0, len(windows), step):
        chunk = np.concatenate(windows[i:i + step])
        updates += ps.run_events(chunk, gtable, stable, W)
    th = torch.empty(N, dtype=torch.float32, device="cuda")
    st = torch.empty(N, dtype=torch.float32, device="cuda")
    ps.export_state(th, st)
    ps.sync()

    def rel(got, want):
        want = want.astype(np.float64)
        den = np.maximum(np.abs(want), max(float(np.sqrt(np.mean(want * want))), 1e-30))
        return float(np.max(np.abs(got.astype(np.float64) - want) / den))

    want_th, ts = oracle_ps.pull()
    out = {"updates": updates, "weights_compared": N, "max_rel_err_weights": rel(th.cpu().numpy(), want_th),
           "max_rel_err_state": rel(st.cpu().numpy(), oracle_ps.state()) if (w.momentum != 0.0 or ADAGRAD) else None,
           "timestamps_equal": int(ts) == ps.timestamp() == updates,
           "bar": 1e-5 if updates == 1 else 1e-4,
           "error": "|library - oracle| / max(|oracle|, rms(oracle)), maximum over the vector",
           "how": "the windows the timed oracle just handled, through rudra_ps_run_events on device copies of the same inputs"}
    ps.close()
    return out


def cpu_model():
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    import platform

    return platform.processor() or platform.machine()


def batch_shape(w, batch):
    """(updates, gradient vectors, weight copies) one backlog asks of the server."""
    kinds = batch["kind"]
    updates = int((kinds == EV_STEP).sum())
    copies = int((kinds == EV_PULL).sum()) + w.lam * int((kinds == EV_BROADCAST).sum())
    return updates, updates * w.c, copies


class DeviceRun:
    """One parameter server with everything resident in HBM, driven over a workload's event stream."""

    def __init__(self, rb, torch, w, args, seed, stream, views=False, fanin=0):
        self.rb, self.torch, self.w, self.stream, self.views = rb, torch, w, stream, views
        N = w.nparams
        self.nbufs = min(w.lam, args.buffers) if args.buffers else w.lam
        self.bufs = [synth.device_gradient(N, l, w.grad_std, w.grad_dtype, seed) for l in range(self.nbufs)]
        self.nslots = 0 if views else self.nbufs
        self.slots = [torch.empty(N, dtype=torch.float32, device="cuda") for _ in range(self.nslots)]
        ps = rb.ParameterServer(N, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
        ps.set_option(rb.OPT_GRAD_DTYPE, w.grad_dtype)
        if ADAGRAD:
            ps.set_option(rb.OPT_OPTIMIZER, rb.OPTIM_ADAGRAD)
        ps.set_weights(synth.device_initial_weights(N, w.theta_std, seed))
        if views:
            ps.enable_views(w.lam + 1)
        if fanin:
            ps.set_option(rb.OPT_TREE_FANIN, fanin)   # learners -> leaves -> this server (Section 3.3)
        ps.sync()
        ps.set_stream(stream)
        self.ps = ps
        self.gtable = rb.pointer_table([self.bufs[l % self.nbufs] for l in range(w.lam)])
        self.stable = None if views else rb.pointer_table([self.slots[l % self.nslots] for l in range(w.lam)])
        self.pool = []

    def events(self, count):
        """Timing event pairs made (and recorded once) ahead of the timed region, so that none is created in it."""
        for _ in range(count):
            pair = (self.torch.cuda.Event(enable_timing=True), self.torch.cuda.Event(enable_timing=True))
            pair[0].record(self.stream)
            pair[1].record(self.stream)
            self.pool.append(pair)

    def pair(self):
        if self.pool:
            return self.pool.pop()
        return self.torch.cuda.Event(enable_timing=True), self.torch.cuda.Event(enable_timing=True)

    def messages(self, win, upd_events, pull_events=None):
        """One message at a time through push / step / pull."""
        ps, bufs, slots, stream = self.ps, self.bufs, self.slots, self.stream
        for kind, learner, pulled_ts in zip(win["kind"].tolist(), win["learner"].tolist(), win["pulled_ts"].tolist()):
            if kind == EV_PUSH:
                ps.push(bufs[learner % self.nbufs], pulled_ts)
            elif kind == EV_STEP:
                e0, e1 = self.pair()
                e0.record(stream)
                ps.step()
                e1.record(stream)
                upd_events.append((e0, e1))
            elif kind == EV_PULL:
                if pull_events is None:
                    ps.pull(slots[learner % self.nslots])
                else:
                    e0, e1 = self.pair()
                    e0.record(stream)
                    ps.pull(slots[learner % self.nslots])
                    e1.record(stream)
                    pull_events.append((e0, e1, 1))
            elif kind == EV_BROADCAST:
                if pull_events is None:
                    ps.pull_many(slots)
                else:
                    e0, e1 = self.pair()
                    e0.record(stream)
                    ps.pull_many(slots)
                    e1.record(stream)
                    pull_events.append((e0, e1, len(slots)))

    def backlog(self, chunk, W, timed, host_s, with_events=True, address=None):
        """A backlog of update windows through one rudra_ps_run_events call (chunk: a contiguous event
        array that the caller keeps alive).  with_events: bracket the call with two timing events."""
        if with_events:
            e0, e1 = self.pair()
            e0.record(self.stream)
        t0 = time.perf_counter()
        self.ps.run_events_at(address or chunk.ctypes.data, len(chunk), self.gtable, self.stable, W)
        host_s.append(time.perf_counter() - t0)
        if with_events:
            e1.record(self.stream)
            timed.append((e0, e1))

    def close(self):
        self.ps.close()
        self.bufs, self.slots = [], []


def rounded_warmup(warmup, W):
    """Warm-up windows really run: whole backlogs, so that the timed backlogs start where a round of
    the learners starts, and at least two of them (the first launches after set-up run 1-2 % slow)."""
    return warmup if W == 0 else max(2, -(-warmup // W)) * W


def timed_region(run, w, windows, warmup, steps, W, barrier, sampler_factory=None):
    """Warm-up, then exactly ``steps`` update windows between two events.  With a backlog size W the
    warm-up is rounded up to whole backlogs so that the timed backlogs start where a round of the
    learners starts; the timed windows are handed over as backlogs of W (the last may be shorter).
    Every launch is bracketed by timing events when the workload streams from HBM (the roofline is
    formed from those); for L2-resident, launch-bound workloads only every eighth call is, so that
    the event records do not slow the host loop that is the bottleneck there."""
    torch, stream, ps = run.torch, run.stream, run.ps
    warm = rounded_warmup(warmup, W)
    wins = windows[: warm + steps]
    assert len(wins) == warm + steps
    if W == 0:
        warm_batches, batches = wins[:warm], wins[warm:]
    else:
        warm_batches = [np.concatenate(wins[i:i + W]) for i in range(0, warm, W)]
        batches = [np.concatenate(wins[i:i + W]) for i in range(warm, warm + steps, W)]
    stride = 1 if (W == 0 or w.nparams * 8 > 126e6) else 8
    all_shapes = [batch_shape(w, b) for b in batches]
    shapes = all_shapes[::stride]
    addresses = [None] * len(batches) if W == 0 else [b.ctypes.data for b in batches]
    junk, host_s = [], []
    for b in warm_batches:
        run.messages(b, junk) if W == 0 else run.backlog(b, W, junk, [])
    run.pool.extend(junk)
    run.events((steps if W == 0 else len(batches)) + 4)
    barrier()
    sampler = sampler_factory() if sampler_factory else None
    if sampler:
        sampler.start()
    c0 = ps.counters()
    start, end = run.pair()
    timed = []
    start.record(stream)
    for i, b in enumerate(batches):
        run.messages(b, timed) if W == 0 else run.backlog(b, W, timed, host_s, i % stride == 0, addresses[i])
    end.record(stream)
    barrier()
    clocks = sampler.stop() if sampler else None
    c1 = ps.counters()
    return {
        "ms": start.elapsed_time(end), "launch_ms": [a.elapsed_time(b) for a, b in timed], "shapes": shapes,
        "host_us": [1e6 * t for t in host_s], "warmup_done": warm, "clocks": clocks,
        "launches": c1["launches"] - c0["launches"], "pulls": c1["pulls"] - c0["pulls"],
        "copies": c1["weight_copies"] - c0["weight_copies"], "batches": len(batches), "views": run.views,
        "launches_sampled_every": stride, "all_shapes": all_shapes,
    }


def path_bytes_of(w, N, region):
    """Algorithmic bytes of everything the timed region's run_events calls asked for."""
    g = 2 if w.grad_dtype == synth.GRAD_BF16 else 4
    extra = max(0, region["launches"] - region["batches"])          # copy launches split off: one more read of the weights each
    vectors = sum(v for _, v, _ in region["all_shapes"])
    copies = region["copies"] if region.get("views") else sum(c for _, _, c in region["all_shapes"])
    return float(N) * (vectors * g + state_bytes(w) * region["batches"] + 4 * copies + 4 * extra)


def launch_shapes(w, N, W, region):
    """Per launch shape (number of updates a run_events call carried): launches, device time and the
    algorithmic bytes of one call.  A call is one fused launch; where the library splits a broadcast
    off into a copy launch (one more read of the weights) the extra launches are spread evenly."""
    g = 2 if w.grad_dtype == synth.GRAD_BF16 else 4
    sb = state_bytes(w)
    extra_per_call = max(0, region["launches"] - region["batches"]) / max(region["batches"], 1)
    out = {}
    total_updates = max(1, sum(u for u, _, _ in region["shapes"]))
    for (updates, vectors, copies), ms in zip(region["shapes"], region["launch_ms"]):
        if region.get("views"):   # shared versions: a version is written once however many learners take it
            copies = region["copies"] * updates / total_updates
        rec = out.setdefault((updates, vectors, copies), {"updates": updates, "gradient_vectors": vectors,
                                                          "weight_copies": copies, "launches": 0, "ms": 0.0})
        rec["launches"] += 1
        rec["ms"] += ms
        rec["bytes_per_launch"] = float(N) * (vectors * g + sb + 4 * copies + 4 * extra_per_call)
    for rec in out.values():
        rec["avg_launch_us"] = 1e3 * rec.pop("ms") / rec["launches"]
        rec["gbs"] = rec["bytes_per_launch"] / (rec["avg_launch_us"] * 1e-6) / 1e9
    return out


def run_ours(args, w):
    global ADAGRAD
    import torch
    import torch.distributed as dist
    from paper_1509_04210_b200 import binding as rb
    from paper_1509_04210_b200 import probe

    from paper_1509_04210_b200 import replicas

    rank, local_rank, world = replicas.rank_info()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU implementation")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    rb.lib()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    N = w.nparams
    seed = replicas.replica_seed(synth.MASTER_SEED, rank)
    stream = torch.cuda.Stream()
    views = args.pull == "views"
    W = default_window(w, views) if args.window < 0 else args.window
    if views and W == 0:
        raise SystemExit("--pull views is served through rudra_ps_run_events: use --window >= 1")
    if args.tree and W == 0:
        raise SystemExit("--tree is served through rudra_ps_run_events: use --window >= 1")
    run = DeviceRun(rb, torch, w, args, seed, stream, views, args.tree)
    ps, bufs, slots, nbufs = run.ps, run.bufs, run.slots, run.nbufs
    # smallest power of two that every gradient buffer and slot starts on (full speed needs 1 KB)
    buf_align = min([(t.data_ptr() & -t.data_ptr()) for t in bufs + slots] + [1 << 21])
    warm_done = rounded_warmup(args.warmup, W)
    extra_steps = 0 if (W == 0 or views or args.tree) else min(args.steps, 216)
    # a short timed region holds few full-window launches: after it, finish the learners' round and
    # time ten more full backlogs, reported beside the roofline (not part of `value`)
    more = 10 if (W >= 1 and args.steps // max(W, 1) < 10) else 0
    tail = (-args.steps) % W if more else 0
    windows = make_windows(w, warm_done + args.steps + tail + more * W + extra_steps, fanin=args.tree)
    extra_windows = windows[warm_done + args.steps + tail + more * W:]
    region = timed_region(run, w, windows, args.warmup, args.steps, W, barrier,
                          lambda: ClockSampler(visible_gpu_index(local_rank)))
    more_launches = None
    if more:
        at = warm_done + args.steps
        if tail:
            run.backlog(np.concatenate(windows[at: at + tail]), W, [], [])
        run.events(more + 2)
        mev, mbytes = [], []
        gb = 2 if w.grad_dtype == synth.GRAD_BF16 else 4
        for i in range(more):
            chunk = np.concatenate(windows[at + tail + i * W: at + tail + (i + 1) * W])
            _, vectors, ncopies = batch_shape(w, chunk)
            mbytes.append(float(N) * (vectors * gb + state_bytes(w) + 4 * ncopies))
            run.backlog(chunk, W, mev, [])
        torch.cuda.synchronize()
        mus = [1e3 * a.elapsed_time(b) for a, b in mev]
        more_launches = {"launches": more, "avg_launch_us": float(np.mean(mus)), "min": min(mus), "max": max(mus),
                         "bytes_per_launch": float(np.mean(mbytes)),
                         "gbs": float(np.sum(mbytes)) / (float(np.sum(mus)) * 1e-6) / 1e9}
    ms, launch_ms, clocks = region["ms"], region["launch_ms"], region["clocks"]
    kern_ms = float(sum(launch_ms))
    launches, pulls, copies = region["launches"], region["pulls"], region["copies"]
    g = 2 if w.grad_dtype == synth.GRAD_BF16 else 4
    sb = state_bytes(w)

    # The same server, continuing the same event stream, driven one message at a time (push, step,
    # pull as separate calls and launches): the unbatched figure beside the backlog figure, and the
    # launch times of the copy kernel that serves a pull by itself.
    single, pull_roof = None, None
    if extra_steps:
        run.events(2 * extra_steps + len(extra_windows) * (w.c + 1) + 4)
        sev, pev = [], []
        barrier()
        s0, s1 = run.pair()
        s0.record(stream)
        for win in extra_windows:
            run.messages(win, sev, pev)
        s1.record(stream)
        barrier()
        sms = replicas.max_over_ranks([s0.elapsed_time(s1)], device="cuda")[0]
        upd_us = 1e3 * float(np.mean([a.elapsed_time(b) for a, b in sev]))
        single = {"value": replicas.whole_job_rate(extra_steps, world, sms), "unit": UNIT, "steps": extra_steps,
                  "update_kernel_us": upd_us,
                  "update_kernel_gbs": update_bytes_per_param(w) * N / (upd_us * 1e-6) / 1e9}
        if pev:
            ndst = pev[0][2]
            pull_us = 1e3 * float(np.mean([a.elapsed_time(b) for a, b, k in pev if k == ndst]))
            pull_roof = {"us": pull_us, "ndst": ndst, "launches": sum(1 for x in pev if x[2] == ndst),
                         "bytes": float(N) * (4 + 4 * ndst)}

    shapes = launch_shapes(w, N, W, region) if W != 0 else {}
    # the launch shape the roofline describes: the full window (W updates) seen most often, else the largest seen
    full = None
    if shapes:
        whole = [b for b in shapes.values() if b["updates"] == W]
        full = max(whole, key=lambda b: b["launches"]) if whole else shapes[max(shapes)]

    # What HBM delivers on this GPU, in this run, for the same mix of reads and writes as one
    # full-window launch of the dominant kernel: a probe kernel that only streams that many vectors
    # in and out (the probe's tables hold 64 of each).
    mix = None
    if full and not views and w.grad_dtype == synth.GRAD_F32 and N * 8 > 126e6 and nbufs == w.lam:
        nr = min(64, full["gradient_vectors"] + sb // 8)
        nw = min(64, full["weight_copies"] + sb // 8)
        extra = [torch.empty(N, dtype=torch.float32, device="cuda") for _ in range(4)]
        srcs = (bufs + extra[:2])[-nr:] if nr <= len(bufs) + 2 else None
        dsts = (slots + extra[2:])[-nw:] if nw <= len(slots) + 2 else None
        if srcs and dsts:
            for _ in range(3):
                probe.stream_probe(srcs, dsts, N, stream)
            p0, p1 = run.pair()
            reps = 10
            p0.record(stream)
            for _ in range(reps):
                probe.stream_probe(srcs, dsts, N, stream)
            p1.record(stream)
            torch.cuda.synchronize()
            mix = {"gbs": 4.0 * N * (nr + nw) * reps / (p0.elapsed_time(p1) * 1e-3) / 1e9, "reads": nr, "writes": nw,
                   "launch_reads": full["gradient_vectors"] + sb // 8, "launch_writes": full["weight_copies"] + sb // 8,
                   "launches": reps,
                   "how": "rudra_stream_probe (librudra_probe.so): that many vectors streamed in and out, same access "
                          "shape, no arithmetic; its tables hold 64 of each"}
        del extra, srcs, dsts

    e2e_ms, e2e_steps, h0, h1, link = float('nan'), 0, None, None, None
    no_e2e = args.kernel_only or bool(args.tree)   # a leaf's relay has no host-buffer form: the tree is measured on the device
    if not no_e2e:
        # end to end through the C interface with host buffers: gradients travel host -> device inside
        # the timed region and every pulled copy of the weights travels device -> host
        e2e_steps = min(args.steps, 16 if N > (1 << 24) else 200)
        nhost = min(nbufs, 8)
        hg = []
        for l in range(nhost):
            t = torch.empty(N, dtype=bufs[0].dtype).pin_memory()
            t.copy_(bufs[l])
            hg.append(t)
        hdst = [torch.empty(N, dtype=torch.float32).pin_memory() for _ in range(4)]
        torch.cuda.synchronize()
        ps2 = rb.ParameterServer(N, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
        ps2.set_option(rb.OPT_GRAD_DTYPE, w.grad_dtype)
        if args.optimizer == "adagrad":
            ps2.set_option(rb.OPT_OPTIMIZER, rb.OPTIM_ADAGRAD)
        ps2.set_weights(synth.device_initial_weights(N, w.theta_std, seed))
        ps2.sync()
        ps2.set_stream(stream)

        def run_window_host(win):
            k = 0
            for kind, learner, pulled_ts in zip(win["kind"].tolist(), win["learner"].tolist(), win["pulled_ts"].tolist()):
                if kind == EV_PUSH:
                    ps2.push_host(hg[learner % nhost], pulled_ts)
                elif kind == EV_STEP:
                    ps2.step()
                elif kind == EV_PULL:
                    ps2.pull_host(hdst[k % 4])
                    k += 1
                elif kind == EV_BROADCAST:
                    ps2.pull_host(hdst[0])   # one copy leaves the device; learners on the host share it

        e2e_warm = min(args.warmup, 3)
        for win in windows[:e2e_warm]:
            run_window_host(win)
        ps2.sync()
        barrier()
        h0 = ps2.counters()
        s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s2.record(stream)
        for win in windows[e2e_warm: e2e_warm + e2e_steps]:
            run_window_host(win)
        ps2.sync()            # uploads, updates and downloads run on three streams: wait for all of them
        e2.record(stream)
        barrier()
        h1 = ps2.counters()
        e2e_ms = s2.elapsed_time(e2)
        ps2.close()
        # what the host link gives plain copies of the same buffers, both directions at once
        link = link_probe(torch, hg[0], hdst[0]) if N > (1 << 24) else None
        del hg, hdst

    ms, e2e_ms = replicas.max_over_ranks([ms, e2e_ms], device="cuda")

    # the paper's other model shape and the broadcast-heavy shape, short runs on the same GPU
    others = None
    if world == 1 and w.name == "imagenet" and not args.kernel_only and not args.no_other_workloads and not args.tree:
        run.close()
        del bufs, slots
        torch.cuda.empty_cache()
        others = {}
        for name, osteps, owarm in (("tiny", 2000, 100), ("cifar10", 6000, 300), ("mid", 800, 40), ("stress", 40, 4),
                                    ("imagenet72m", 180, 18),
                                    ("imagenet_zero_copy_pulls", 360, 18), ("imagenet_adagrad", 360, 18)):
            # the last two: the default workload with learners sharing weight versions by pointer
            # (rudra_ps_enable_views) and with AdaGrad at the server (Section 5.5)
            oviews = name == "imagenet_zero_copy_pulls"
            was_adagrad, ADAGRAD = ADAGRAD, ADAGRAD or name == "imagenet_adagrad"
            ow = w if name.startswith("imagenet_") else synth.WORKLOADS[name]
            if name == "imagenet_adagrad":
                import dataclasses

                ow = dataclasses.replace(ow, momentum=0.0)
            orun = DeviceRun(rb, torch, ow, args, seed, stream, views=oviews)
            oW = default_window(ow, oviews)
            owin = make_windows(ow, rounded_warmup(owarm, oW) + osteps)
            reg = timed_region(orun, ow, owin, owarm, osteps, oW, barrier)
            og = 2 if ow.grad_dtype == synth.GRAD_BF16 else 4
            osb = 16 if ow.momentum else 8
            obytes = path_bytes_of(ow, ow.nparams, reg)
            others[name] = {
                "value": osteps / (reg["ms"] * 1e-3), "unit": UNIT, "steps": osteps, "warmup": reg["warmup_done"],
                "nparams": ow.nparams, "lambda": ow.lam, "n": ow.n, "c": ow.c,
                "grad_dtype": "bf16" if ow.grad_dtype == synth.GRAD_BF16 else "f32", "window": oW,
                "bytes_per_param_per_step": obytes / ow.nparams / osteps,
                "hbm_gbs": obytes / (reg["ms"] * 1e-3) / 1e9,
                "gpu_launches": reg["launches"], "avg_launch_us": 1e3 * float(np.mean(reg["launch_ms"])),
                "host_us_per_call": float(np.median(reg["host_us"])),
                "roofline_claim": ow.nparams * 8 > 126e6,
            }
            del og, osb
            orun.close()
            del orun
            ADAGRAD = was_adagrad
            torch.cuda.empty_cache()
        # the same ImageNet-scale stream behind the two-level server tree of Section 3.3 (18 leaves of 3
        # learners on this GPU, their averaging fused into the root's launch), and the leaf's own kernel
        k = 3
        trun = DeviceRun(rb, torch, w, args, seed, stream, fanin=k)
        tsteps, twarm = 360, W
        treg = timed_region(trun, w, make_windows(w, rounded_warmup(twarm, W) + tsteps, fanin=k), twarm, tsteps, W, barrier)
        tbytes = path_bytes_of(w, N, treg)
        avg = torch.empty(N, dtype=torch.float32, device="cuda")
        for i in range(3):
            rb.leaf_average(trun.bufs[3 * i: 3 * i + k], w.grad_dtype, N, avg, stream)
        l0, l1 = trun.pair()
        reps = 18
        l0.record(stream)
        for i in range(reps):
            rb.leaf_average(trun.bufs[3 * (i % 18): 3 * (i % 18) + k], w.grad_dtype, N, avg, stream)
        l1.record(stream)
        torch.cuda.synchronize()
        leaf_us = 1e3 * l0.elapsed_time(l1) / reps
        # the other form of the relay, one message at a time: every leaf runs its averaging kernel and
        # the root receives one float vector per leaf (what crosses the link when leaves sit on other GPUs)
        mrun = DeviceRun(rb, torch, w, args, seed, stream)
        mwin = make_windows(w, 2 * W + 108, fanin=k)
        avgs = [torch.empty(N, dtype=torch.float32, device="cuda") for _ in range(w.lam // k)]
        held = {}

        def relay_window(win):
            for kind, learner, pulled_ts in zip(win["kind"].tolist(), win["learner"].tolist(), win["pulled_ts"].tolist()):
                if kind == EV_PUSH:
                    held.setdefault(learner // k, []).append((mrun.bufs[learner], pulled_ts))
                elif kind == 6:   # RELAY
                    msg = held.pop(learner)
                    rb.leaf_average([b for b, _ in msg], w.grad_dtype, N, avgs[learner], stream)
                    mrun.ps.push_group([avgs[learner]], [p for _, p in msg])
                elif kind == EV_STEP:
                    mrun.ps.step()
                elif kind == EV_PULL:
                    mrun.ps.pull(mrun.slots[learner])

        for win in mwin[: 2 * W]:
            relay_window(win)
        barrier()
        m0, m1 = mrun.pair()
        m0.record(stream)
        for win in mwin[2 * W:]:
            relay_window(win)
        m1.record(stream)
        barrier()
        relay_rate = 108 / (m0.elapsed_time(m1) * 1e-3)
        mrun.close()
        del mrun, avgs
        torch.cuda.empty_cache()
        peak_now = measured_hbm_peak()[0]
        others["imagenet_tree_fanin3"] = {
            "value": tsteps / (treg["ms"] * 1e-3), "unit": UNIT, "steps": tsteps, "window": W, "fanin": k,
            "relay": "leaves share the root's GPU: raw gradients handed over, averaged inside the update kernel",
            "materialised_relay_one_message_at_a_time": {
                "value": relay_rate, "unit": UNIT, "steps": 108,
                "how": "every leaf runs rudra_leaf_average, the root takes one float vector per leaf "
                       "(rudra_ps_push_group), step and pull as separate calls; compare one_message_at_a_time"},
            "bytes_per_param_per_step": tbytes / N / tsteps, "hbm_gbs": tbytes / (treg["ms"] * 1e-3) / 1e9,
            "gpu_launches": treg["launches"], "avg_launch_us": 1e3 * float(np.mean(treg["launch_ms"])),
            "host_us_per_call": float(np.median(treg["host_us"])),
            "roofline_leaf": {
                "kernel": "leaf_average_kernel (a leaf's mean of its %d learners' gradients, one float vector out)" % k,
                "bound": "hbm", "achieved": float(N) * (k * g + 4) / (leaf_us * 1e-6) / 1e9, "peak": peak_now, "unit": "GB/s",
                "frac": float(N) * (k * g + 4) / (leaf_us * 1e-6) / 1e9 / peak_now, "launches_timed": reps,
                "avg_launch_us": leaf_us, "bytes_per_launch": float(N) * (k * g + 4),
                "traffic": ncu_traffic(("leaf", k, g), N)},
        }
        trun.close()
        del trun, avg
        torch.cuda.empty_cache()

    if rank == 0:
        peak, peak_kind = measured_hbm_peak()
        # bytes the whole path must move per step: every gradient once, weights/state per launch, pulls
        if W == 0:
            path_bytes = N * (args.steps * (w.c * g + sb) + 8 * pulls)
            kern_bytes = float(N * args.steps * (w.c * g + sb))     # the timed launches are the update kernels only
            achieved = kern_bytes / (kern_ms * 1e-3) / 1e9 if kern_ms > 0 else float("nan")
            roof_launches, roof_us, roof_bytes = len(launch_ms), 1e3 * kern_ms / max(len(launch_ms), 1), kern_bytes / max(len(launch_ms), 1)
            label = "update_kernel (fused sumGradients + applyUpdate), one update per launch"
        else:
            path_bytes = path_bytes_of(w, N, region)
            achieved, roof_launches, roof_us, roof_bytes = full["gbs"], full["launches"], full["avg_launch_us"], full["bytes_per_launch"]
            label = "update_kernel (fused sumGradients + applyUpdate), %d-update window with its %d pulls%s" % (
                full["updates"], full["weight_copies"],
                "" if launches == region["batches"] else " + the copy kernel the library splits off for a broadcast")
        value = replicas.whole_job_rate(args.steps, world, ms)
        cfg = workload_config(w)
        cfg["parallelism"] = "replicas x%d (one independent server per GPU)" % world
        cfg["window"] = W
        cfg["buffer_alignment_bytes"] = buf_align
        cfg["warmup_done"] = region["warmup_done"]
        cfg["launches_timed_every"] = region["launches_sampled_every"]
        cfg["pull"] = ("zero-copy: learners share a pointer to the version they pulled (rudra_ps_enable_views)" if views
                       else "copy into each learner's slot")
        cfg["window_note"] = ("messages handled one at a time (push / step / pull)" if W == 0 else
                              "backlog of %d update windows per rudra_ps_run_events call; warm-up rounded up to whole backlogs" % W)
        other_shapes = [b for k, b in sorted(shapes.items()) if b is not full]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None,
            "dtype": "f32" if w.grad_dtype == synth.GRAD_F32 else "f32 arithmetic on bf16 gradients (widened exactly)",
            "data": "synthetic",
            "config": cfg,
            "hbm_gbs_whole_path": path_bytes / (ms * 1e-3) / 1e9,
            "bytes_per_param_per_step": path_bytes / N / args.steps,
            "pulls_per_step": pulls / args.steps,
            "weight_copies_per_step": copies / args.steps,
            "host_us_per_call": None if not region["host_us"] else {
                "call": "rudra_ps_run_events through the Python binding", "median": float(np.median(region["host_us"])),
                "max": float(max(region["host_us"])), "calls": len(region["host_us"])},
            "one_message_at_a_time": single,
            "gpu_launches": launches,
            "clocks": clocks,
            "e2e": None if no_e2e else {
                "value": replicas.whole_job_rate(e2e_steps, world, e2e_ms), "unit": UNIT, "steps": e2e_steps,
                "h2d_bytes_per_step": (h1["h2d_bytes"] - h0["h2d_bytes"]) // e2e_steps,
                "d2h_bytes_per_step": (h1["d2h_bytes"] - h0["d2h_bytes"]) // e2e_steps,
                "link": None if not link else dict(
                    link, achieved_h2d_gbs=(h1["h2d_bytes"] - h0["h2d_bytes"]) / (e2e_ms * 1e-3) / 1e9,
                    achieved_d2h_gbs=(h1["d2h_bytes"] - h0["d2h_bytes"]) / (e2e_ms * 1e-3) / 1e9),
            },
            "roofline": {
                "kernel": label,
                "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "peak_kind": "of %s" % peak_kind, "launches_timed": roof_launches, "avg_launch_us": roof_us,
                "bytes_per_launch": roof_bytes,
                "launch_us": None if not launch_ms else {
                    "min": 1e3 * min(launch_ms), "median": 1e3 * float(np.median(launch_ms)), "max": 1e3 * max(launch_ms)},
                "frac_of_8TBs_datasheet": achieved / 8000.0,
                "traffic": None if (W == 0 or not full or views) else ncu_traffic(
                    ("update", w.name, full["updates"], full["gradient_vectors"], full["weight_copies"]), N),
                "mix_ceiling": mix,
                "frac_of_mix_ceiling": None if not mix else achieved / mix["gbs"],
                "other_launch_shapes": other_shapes,
                "more_full_window_launches": None if not more_launches or views else dict(
                    more_launches,
                    note="the same server right after the timed region, the round finished first; not part of value"),
            },
            "roofline_pull": None if not pull_roof else {
                "kernel": "snapshot_kernel (pullWeights: one read of the weights, %d written cop%s)" % (
                    pull_roof["ndst"], "y" if pull_roof["ndst"] == 1 else "ies"),
                "bound": "hbm", "achieved": pull_roof["bytes"] / (pull_roof["us"] * 1e-6) / 1e9, "peak": peak, "unit": "GB/s",
                "frac": pull_roof["bytes"] / (pull_roof["us"] * 1e-6) / 1e9 / peak, "peak_kind": "of %s" % peak_kind,
                "launches_timed": pull_roof["launches"], "avg_launch_us": pull_roof["us"],
                "bytes_per_launch": pull_roof["bytes"], "traffic": ncu_traffic(("snapshot", pull_roof["ndst"]), N),
                "where": "the one-message-at-a-time leg of this run: every pull a launch of its own",
            },
            "other_workloads": others,
        }
        if world == 1 and not args.no_cpu_baseline and not args.kernel_only:
            from oracle import rudra_oracle as ora

            ora.build()
            nh = min(w.lam, 6)
            hostg = [synth.device_gradient(N, l, w.grad_std, w.grad_dtype, seed) for l in range(nh)]
            grads = [t.cpu().numpy() if w.grad_dtype == synth.GRAD_F32 else t.view(torch.int16).cpu().numpy().view(np.uint16)
                     for t in hostg]
            del hostg
            kept = []
            done, dt = oracle_run(w, windows, N, grads, warmup=1, budget_s=12.0, max_windows=args.steps,
                                  adagrad=args.optimizer == "adagrad", keep=kept)
            line["cpu_baseline"] = {
                "value": done / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
                "sample": "%d full-size update windows of the same event stream (%d distinct gradient buffers), %.1f s"
                          % (done, nh, dt),
                "host_cores_available": os.cpu_count(), "cpu_model": cpu_model(),
            }
            # The windows the oracle just went through, once more through the library on the same
            # bytes: every weight and every state value of the full-size vector compared.
            if not args.tree:   # (the tree's events have no flat-server replay in the timed oracle loop)
                line["cpu_baseline"]["parity"] = parity_with_oracle(rb, torch, w, windows[: done + 1], grads, kept[0], W, stream)
            del kept
            cores = os.cpu_count() or 1
            if cores > 1:
                done_all, dt_all = oracle_run_all_cores(w, windows, grads, cores, 8.0, adagrad=args.optimizer == "adagrad")
                line["cpu_baseline"]["all_cores"] = {
                    "value": done_all / dt_all, "unit": UNIT, "cores": cores,
                    "kind": "oracle, one unmodified single-threaded instance per core on disjoint slices of the vector",
                    "sample": "%d full-size update windows, %.1f s (slicing and per-thread copies of the inputs included)"
                              % (done_all, dt_all),
                }
        print(json.dumps(line), flush=True)
    if others is None:
        run.close()
    if world > 1:
        dist.destroy_process_group()


def run_probe_mixes(args, w):
    """--probe-mixes: what HBM delivers for mixes of reads and writes (rudra_stream_probe), as a table."""
    import torch
    from paper_1509_04210_b200 import probe

    N = w.nparams
    pool = [torch.zeros(N, dtype=torch.float32, device="cuda") for _ in range(120)]
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    print("vector length %d floats, distinct vectors rotating through a pool of %d, 8 timed launches each" % (N, len(pool)))
    for nr, nw in [(54, 0), (0, 54), (27, 27), (56, 56), (20, 8), (56, 2), (2, 56), (40, 16), (16, 40), (8, 0), (0, 8)]:
        def launch(i):
            srcs = [pool[(i * 7 + l) % 60] for l in range(nr)]
            dsts = [pool[60 + (i * 5 + l) % 60] for l in range(nw)]
            probe.stream_probe(srcs, dsts, N, stream)
        for i in range(2):
            launch(i)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(8):
            launch(i)
        e1.record(stream)
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) / 8 * 1e3
        print("reads %2d writes %2d  write share %.2f  %8.1f us  %6.0f GB/s"
              % (nr, nw, nw / (nr + nw), us, 4.0 * N * (nr + nw) / us * 1e-3), flush=True)


def run_leaf_average(args, w):
    """--leaf-average K: the leaf's averaging kernel alone on the workload's vector length (no bench line)."""
    import torch
    from paper_1509_04210_b200 import binding as rb

    N, k = w.nparams, args.leaf_average
    g = 2 if w.grad_dtype == synth.GRAD_BF16 else 4
    nbuf = max(k, (args.buffers or min(54, int(6e9 // (N * g)))) // k * k)
    bufs = [synth.device_gradient(N, l, w.grad_std, w.grad_dtype) for l in range(nbuf)]
    avg = torch.empty(N, dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    groups = [bufs[i:i + k] for i in range(0, nbuf, k)]
    for grp in groups[:3]:
        rb.leaf_average(grp, w.grad_dtype, N, avg, stream)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 3 * len(groups)
    e0.record(stream)
    for i in range(reps):
        rb.leaf_average(groups[i % len(groups)], w.grad_dtype, N, avg, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    us = 1e3 * e0.elapsed_time(e1) / reps
    peak, kind = measured_hbm_peak()
    print(json.dumps({"kernel": "leaf_average_kernel", "nparams": N, "k": k, "grad_bytes": g, "launches": reps,
                      "avg_launch_us": us, "bytes_per_launch": float(N) * (k * g + 4),
                      "gbs": float(N) * (k * g + 4) / (us * 1e-6) / 1e9, "peak": peak, "peak_kind": kind,
                      "frac": float(N) * (k * g + 4) / (us * 1e-6) / 1e9 / peak}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1800,
                    help="timed update windows (default: 100 rounds of the 54 learners at the ImageNet-scale workload)")
    ap.add_argument("--warmup", type=int, default=36)
    ap.add_argument("--workload", default="imagenet", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--window", type=int, default=-1,
                    help="update windows handed to the server per call: 0 = one message at a time, "
                         "-1 = what lambda blocked learners can have waiting (n = lambda/c updates)")
    ap.add_argument("--pull", default="copy", choices=["copy", "views"],
                    help="copy: every pull writes the learner's own slot; views: zero-copy shared weight versions")
    ap.add_argument("--optimizer", default="sgd", choices=["sgd", "adagrad"],
                    help="momentum SGD with weight decay (Section 4.2) or AdaGrad at the server (Section 5.5)")
    ap.add_argument("--tree", type=int, default=0, metavar="FANIN",
                    help="learners send to leaves of a two-level server tree (Section 3.3), FANIN learners per leaf")
    ap.add_argument("--leaf-average", type=int, default=0, metavar="K",
                    help="time the leaf's averaging kernel for K gradients per leaf (no bench line) and exit")
    ap.add_argument("--probe-mixes", action="store_true",
                    help="print what HBM delivers for several mixes of reads and writes (no bench line) and exit")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the short cifar10 and stress runs that the default workload's line carries")
    ap.add_argument("--kernel-only", action="store_true",
                    help="device-resident timed region only: no end-to-end leg, no CPU baseline (profiler captures)")
    ap.add_argument("--nparams", type=int, default=0,
                    help="override the vector length (small cases for profiler captures; not a bench line)")
    ap.add_argument("--buffers", type=int, default=0,
                    help="distinct gradient buffers and learner slots (default: one per learner)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    w = synth.WORKLOADS[args.workload]
    if args.optimizer == "adagrad":
        import dataclasses

        global ADAGRAD
        ADAGRAD = True
        w = dataclasses.replace(w, name=w.name + "+adagrad", momentum=0.0)
    if args.pull == "views" and w.downcast:
        import dataclasses

        # with shared versions the down-cast needs no broadcast: each learner takes the current
        # version when it starts its next mini-batch (the integers of the trace are the same)
        w = dataclasses.replace(w, name=w.name + "+views", downcast=False)
    if args.nparams:
        import dataclasses

        w = dataclasses.replace(w, name=w.name + "@%d" % args.nparams, nparams=args.nparams)
    if args.probe_mixes:
        run_probe_mixes(args, w)
        return
    if args.leaf_average:
        run_leaf_average(args, w)
        return
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
