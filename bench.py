#!/usr/bin/env python
"""Benchmark of the CLT-k step: learner-elements/s (n*d / step time) and HBM roofline fraction.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload resnet50] [--impl reference]

One "step" is one scalecom_step call (selection on the leader, fused learner
pass over all n learners, weight update) on seeded synthetic gradients of the
named workload.  N > 1 (under torchrun) runs N independent replicas: the
method keeps all n logical learners inside one GPU, so nothing is exchanged.
Rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "learner-elements/s per CLT-k step (n*d/step time)"
UNIT = "learner-elements/s"
FALLBACK_HBM_GBS = 6650.0            # earlier measurement on this machine, used only if MEASURED_PEAKS.json is absent
NOMINAL_HBM_GBS = 8000.0
MAX_BATCHES = 24                     # distinct gradient batches kept resident; steps cycle through them

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture of this
# command with --batches 2) by workload and kernel, with the day of the capture; absent: not captured.
NCU_TRAFFIC = {"resnet50": {"learner_pass_kernel": 2.4326e9, "topk_select_kernel": 2.119e8, "captured": "2026-11-25"},
               "resnet50_n16": {"learner_pass_kernel": 4.8896e9, "captured": "2026-11-25"}}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet50",
                    help="tiny, resnet50 (default, the headline), transformer_base, resnet50_n<N>, gpt2_medium, or "
                         "all: every configuration in turn, one JSON line each, then the learner sweep's fit")
    ap.add_argument("--late-steps", type=int, default=0,
                    help="untimed steps run before the timed region (beyond --warmup): late in a run error feedback "
                         "has piled coordinates up under the threshold and the selection has more candidates")
    ap.add_argument("--repeats", type=int, default=4,
                    help="further timed regions of --steps steps after the headline one, reported as median/min/max")
    ap.add_argument("--batches", type=int, default=MAX_BATCHES,
                    help="distinct gradient batches kept in HBM (steps cycle through them); small values keep "
                         "the footprint low for profiler captures")
    ap.add_argument("--selector", default="topk", choices=["topk", "chunk", "layer_topk"],
                    help="leader selection: exact top-k (the headline path), the chunk-wise selector, or exact top-k "
                         "inside every layer (needs --layers)")
    ap.add_argument("--layers", action="store_true",
                    help="with --selector chunk on a ResNet-50-shaped workload: the paper's per-layer rate rule "
                         "(25X / 50X / 400X, first layer whole) instead of one rate; k becomes the sum of the layers' keeps")
    ap.add_argument("--deployment", default="one-gpu", choices=["one-gpu", "learner-per-gpu"],
                    help="one-gpu (default, the headline): all n learners of the workload in each GPU's memory; "
                         "learner-per-gpu: every rank is one learner (n = number of ranks), indices broadcast and "
                         "kept values all-gathered over NCCL between the library's calls")
    ap.add_argument("--exchange", default="collective", choices=["collective", "peer", "peer-flags"],
                    help="learner-per-gpu only: all-gather of the kept values by NCCL (collective); fused into the "
                         "compressing kernel as stores into the peers' mapped buffers, a one-word all-reduce as fence "
                         "(peer); or the same with flag words the reducing kernel waits for instead of the fence "
                         "(peer-flags; one rank per GPU)")
    ap.add_argument("--l2-keep", type=int, default=1, choices=[0, 1],
                    help="SCALECOM_OPT_L2_KEEP: 0 streams the leader's vectors with the default L2 policy (for A/B runs and captures)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    return ap.parse_args()


def get_workload(name):
    from paper_2104_11125_b200 import workloads as W
    if name in W.CONFIGS:
        return W.CONFIGS[name]
    if name.startswith("resnet50_n"):
        return W.sweep(int(name[len("resnet50_n"):]))
    raise SystemExit("unknown workload %r (have %s, resnet50_n<N>)" % (name, ", ".join(W.CONFIGS)))


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler(threading.Thread):
    """Polls SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, device_index):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception as e:  # pragma: no cover
            self.error = repr(e)

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
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.001)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


def job_value(n, d, world, ms_step):
    """Whole-job learner-elements/s: every rank processed n*d learner-coordinates per step."""
    return n * d * world / (ms_step * 1e-3)


def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(values)
    t = torch.tensor(list(values), dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


REFERENCE_BUDGET_S = 240.0           # the --impl reference arm runs full steps of the workload when they fit this


def oracle_rate():
    """Learner-coordinates per second the single-threaded oracle usually reaches (sizing only, never reported)."""
    return 6.5e7


def run_reference(args):
    """The CPU oracle as it stands (one thread) on host cores: full steps of the bench workload when
    steps + warmup of them fit the budget, else steps over the first coordinates of every vector."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import oracle
    from paper_2104_11125_b200 import workloads as W
    full = get_workload(args.workload)
    total = args.steps + args.warmup
    est_full = full.n * full.d / oracle_rate()                         # seconds per full step
    if est_full * total <= REFERENCE_BUDGET_S:
        w = full
    else:
        w = full.scaled(max(1 << 20, int(full.d * REFERENCE_BUDGET_S / (est_full * total))))
    prof = W.profile(w, "cpu")
    nb = min(total, 2 if w.n * w.d > 1e8 else 4)
    batches = [[g.numpy() for g in W.gradients(w, s, "cpu", prof)] for s in range(nb)]
    osel = "chunk" if args.selector == "chunk" else "topk"        # (per-layer rates are not part of this arm)
    m = [x.numpy() for x in W.initial_memory(w, "cpu")]
    th = W.initial_weights(w, "cpu").numpy()
    t = 0
    for _ in range(args.warmup):
        oracle.step(batches[t % nb], m, th, t, w.k, w.beta, w.lr, want_gathered=False, selector=osel)
        t += 1
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.step(batches[t % nb], m, th, t, w.k, w.beta, w.lr, want_gathered=False, selector=osel)
        t += 1
    dt = time.perf_counter() - t0
    value = w.n * w.d * args.steps / dt
    if w.d == full.d:
        sample = "full steps of the workload (n=%d, d=%d, k=%d), %d gradient batches in turn" % (w.n, w.d, w.k, nb)
    else:
        sample = "first %d of %d coordinates per learner (same recipe, n=%d, k=%d), every step" % (w.d, full.d, w.n, w.k)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": full.name, "n": full.n, "d": full.d, "k": full.k, "beta": full.beta, "lr": full.lr,
                   "selector": args.selector},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def time_oracle(w, batches_dev, selector="topk", layers=None, budget_s=12.0):
    """cpu_baseline leg: the oracle, as it stands, on one of this machine's host cores, for about budget_s seconds: full
    steps of the bench workload where one fits the budget (up to four of them), else steps over the first
    coordinates of every learner's vectors (the same recipe at a smaller d; not with per-layer rates).  Beside it,
    for the exact selector, the same routines with their loops spread over all host cores."""
    import numpy as np
    import oracle
    est = w.n * w.d / oracle_rate()                                    # seconds per full step
    d_s = w.d if est <= budget_s or layers is not None else max(1 << 20, int(w.d * budget_s / est))
    k_s = w.k if d_s == w.d else max(1, w.k * d_s // w.d)
    steps = max(1, min(4, int(budget_s / max(est * d_s / w.d, 1e-9))))
    what = "full steps of the bench workload" if d_s == w.d else "steps over the first %d coordinates of every vector" % d_s
    osel = "topk" if selector == "layer_topk" else selector

    def run(threads):
        m = [np.zeros(d_s, np.float32) for _ in range(w.n)]
        th = np.zeros(d_s, np.float32)
        dt = 0.0
        for s in range(steps):
            g = [np.ascontiguousarray(x[:d_s].cpu().numpy()) for x in batches_dev[s % len(batches_dev)]]
            t0 = time.perf_counter()
            oracle.step(g, m, th, s, k_s, w.beta, w.lr, want_gathered=False, selector=osel, layers=layers, threads=threads)
            dt += time.perf_counter() - t0
        return dt

    dt = run(1)
    out = {"value": w.n * d_s * steps / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": "%d %s (n=%d, d=%d, k=%d), %.1f s" % (steps, what, w.n, w.d, w.k, dt)}
    cores = oracle.host_cores()
    if cores > 1 and osel == "topk" and layers is None:
        dtp = run(cores)
        out["all_cores"] = {"value": w.n * d_s * steps / dtp, "unit": UNIT, "cores": cores, "kind": "oracle, loops spread over threads",
                            "sample": "the same %d steps, %.1f s" % (steps, dtp), "nproc": os.cpu_count()}
    return out


def run_learner_per_gpu(args):
    """Every rank is one learner of Algorithm 1: select on the leader, index broadcast, compress, all-gather of
    the kept values, reduce + weight update.  One JSON line from rank 0; the time is the max over ranks."""
    import torch
    import torch.distributed as dist
    from paper_2104_11125_b200 import binding, multi, workloads as W

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    else:
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % (29400 + os.getpid() % 500),
                                world_size=1, rank=0, device_id=dev)
    w = dataclasses.replace(get_workload(args.workload), n=world)
    K, Wm = args.steps, max(args.warmup, 3)
    prof = W.profile(w, dev)
    nb = max(1, min(K + Wm, args.batches, 4 * MAX_BATCHES))
    grads = [W.gradients(w, s, dev, prof, learners=[rank])[0] for s in range(nb)]
    mem = torch.zeros(w.d, device=dev, dtype=torch.float32)          # Algorithm 1: memory starts at zero
    flush = torch.empty(64 << 20, device=dev, dtype=torch.float32)  # 256 MB: written between timed intervals
    theta = W.initial_weights(w, dev)
    node = multi.LearnerRank(w.d, w.k, w.beta, w.lr, exchange=args.exchange,
                             selector=binding.SELECTOR_CHUNK if args.selector == "chunk" else binding.SELECTOR_TOPK)
    ctx = node.engine

    def barrier():
        dist.barrier()
        torch.cuda.synchronize()

    t = 0
    for _ in range(Wm):
        node.step(grads[t % nb], mem, theta, t)
        t += 1
    # the memory vector is the same 4d bytes every step and would sit in L2 from one step to the next, which a
    # training iteration between two steps would not allow: each step is timed by itself, L2 flushed before it
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    launches0 = ctx.query(binding.Q_KERNEL_LAUNCHES)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    for a, b in evs:
        flush.zero_()
        a.record()
        node.step(grads[t % nb], mem, theta, t)
        b.record()
        t += 1
    barrier()
    clocks = sampler.stop()
    ms_step = sum(a.elapsed_time(b) for a, b in evs) / K
    launches = ctx.query(binding.Q_KERNEL_LAUNCHES) - launches0
    assert ctx.status() == 0, "device status %d" % ctx.status()

    # the library's three calls one by one (CUDA events around each call, no collective in between)
    def call_ms(fn, reps=30):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for i, (a, b) in enumerate(evs):
            flush.zero_()
            a.record()
            fn(i)
            b.record()
        torch.cuda.synchronize()
        ms = sorted(a.elapsed_time(b) for a, b in evs)
        return ms[len(ms) // 2]

    sel_ms = call_ms(lambda i: ctx.select(grads[i % nb], mem, node.idx))
    cmp_ms = call_ms(lambda i: ctx.compress(grads[i % nb], mem, node.idx, node.own))
    red_ms = call_ms(lambda i: ctx.reduce_rows(node.rows, node.val, node.idx, theta))
    assert ctx.status() == 0
    ms_step, sel_ms, cmp_ms, red_ms = max_over_ranks([ms_step, sel_ms, cmp_ms, red_ms], dev)
    if rank == 0:
        peak, peak_src = measured_peak()
        cmp_gbs = 12.0 * w.d / (cmp_ms * 1e-3) / 1e9
        print(json.dumps({
            "metric": METRIC, "value": world * w.d / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": Wm, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "n": world, "d": w.d, "k": w.k, "beta": w.beta, "lr": w.lr,
                       "parallelism": "learner per GPU: index broadcast (NCCL) + " +
                                      {"peer": "kept values stored into the peers' mapped rows by the compressing kernel, "
                                               "one-word all-reduce as fence",
                                       "peer-flags": "kept values and flag words stored into the peers' mapped buffers by the "
                                                     "compressing kernel, the reducing kernel waits for the flags",
                                       "collective": "all-gather of kept values (NCCL)"}[args.exchange],
                       "selector": args.selector, "gradient_batches_resident": nb,
                       "l2": "flushed (256 MB written) before every timed step and call",
                       "exchange_bytes_per_rank_per_step": node.exchange_bytes()},
            "roofline": {"bound": "hbm", "kernel": "scalecom_compress (index list -> bitmap, single-learner pass)",
                         "achieved": cmp_gbs, "peak": peak, "unit": "GB/s", "frac": cmp_gbs / peak, "traffic": None,
                         "peak_source": peak_src, "algorithmic_bytes_per_launch": 12.0 * w.d, "avg_launch_ms": cmp_ms},
            "call_ms": {"scalecom_select": sel_ms, "scalecom_compress": cmp_ms, "scalecom_reduce_rows": red_ms,
                        "note": "median of 30 calls, CUDA events around each call (about 6 us of event overhead each), L2 flushed before each"},
            "gpu_launches": launches, "clocks": clocks,
        }))
    node.close()
    dist.destroy_process_group()


def fit_line(xs, ys):
    """Least-squares slope and intercept of ys over xs."""
    n = len(xs)
    mx, my = sum(xs) / n, sum(ys) / n
    sxx = sum((x - mx) ** 2 for x in xs)
    slope = sum((x - mx) * (y - my) for x, y in zip(xs, ys)) / sxx
    return slope, my - slope * mx


def bench_workload(args, name, world, rank, dev, stream, barrier, steps=None, late_steps=0, cpu_baseline=True, e2e=True):
    """Time one workload on this rank's GPU and (rank 0) return its JSON line as a dict."""
    import torch
    import paper_2104_11125_b200 as sc
    from paper_2104_11125_b200 import binding, workloads as W

    local = dev.index
    w = get_workload(name)
    layers = None
    if args.layers:
        if args.selector == "topk" or w.kind != "resnet50":
            raise SystemExit("--layers needs --selector chunk or layer_topk and a ResNet-50-shaped workload")
        layers = W.resnet50_layer_keep(w)
        w = W.Workload(w.name + "+layers", w.wid, w.kind, w.n, w.d, sum(layers[1]), w.beta, w.lr, w.steps, w.c)
    K, Wm = steps or args.steps, max(args.warmup, 3)
    prof = W.profile(w, dev)
    # gradient batches kept resident: as many as fit beside the memories in about 60 % of the free device memory
    free, _ = torch.cuda.mem_get_info(dev)
    per_batch = 4 * w.n * w.d
    fit = max(1, int((0.6 * free - per_batch) // per_batch))
    nb = max(1, min(K + Wm, args.batches, MAX_BATCHES, fit))
    batches = [W.gradients(w, s, dev, prof) for s in range(nb)]
    mem = W.initial_memory(w, dev)
    theta = W.initial_weights(w, dev)
    idx = torch.empty(w.k, device=dev, dtype=torch.int32)
    val = torch.empty(w.k, device=dev, dtype=torch.float32)

    ctx = sc.Context(w.d, w.n, w.k, w.beta, w.lr, stream=stream)
    if args.selector == "layer_topk":
        if layers is None:
            raise SystemExit("--selector layer_topk needs --layers")
        ctx.set_option(binding.OPT_SELECTOR, binding.SELECTOR_LAYER_TOPK)
    if args.selector == "chunk":
        ctx.set_option(binding.OPT_SELECTOR, binding.SELECTOR_CHUNK)
    if layers is not None:
        ctx.set_layers(*layers)
    if not args.l2_keep:
        ctx.set_option(binding.OPT_L2_KEEP, 0)
    torch.cuda.synchronize()
    step = ctx.prepare_step(batches, mem, theta, idx, val)        # pointer tables marshalled once per batch

    # ---- device-resident timing ---------------------------------------------------------------------
    # Region A: K steps back to back, nothing else on the stream -> the headline value.
    # Region B: the same K steps again with the library's per-kernel CUDA events switched on -> the
    # per-kernel durations behind the roofline block (the extra events cost about 2 % of a step,
    # which is why they are kept out of region A).
    # Region A is then repeated a few times: the median says how far one K-step region can be trusted.
    t = 0
    for _ in range(Wm + late_steps):
        step(t % nb, t)
        t += 1
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ctx.query(binding.Q_KERNEL_LAUNCHES)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    ev0.record(stream)
    for _ in range(K):
        step(t % nb, t)
        t += 1
    ev1.record(stream)
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    launches = ctx.query(binding.Q_KERNEL_LAUNCHES) - launches0
    ctx.set_option(binding.OPT_KERNEL_TIMING, 1)
    ctx.set_option(binding.OPT_KERNEL_SPANS, 1)
    evb0, evb1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    evb0.record(stream)
    for _ in range(K):
        step(t % nb, t)
        t += 1
    evb1.record(stream)
    barrier()
    ms_total_b = evb0.elapsed_time(evb1)
    assert ctx.status() == 0, "device status %d" % ctx.status()
    kms, ksteps = ctx.kernel_ms()
    sms, ssteps = ctx.kernel_span_ms()
    ctx.set_option(binding.OPT_KERNEL_TIMING, 0)
    ctx.set_option(binding.OPT_KERNEL_SPANS, 0)
    paths = ctx.query(binding.Q_LAST_TOPK_PATH)
    cands = ctx.query(binding.Q_LAST_CANDIDATES)
    one_kernel = ctx.query(binding.Q_FUSED_SMALL) > 0                  # the whole step is one cooperative kernel
    repeats = []
    for _ in range(args.repeats):
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        r0.record(stream)
        for _ in range(K):
            step(t % nb, t)
            t += 1
        r1.record(stream)
        torch.cuda.synchronize()
        repeats.append(r0.elapsed_time(r1) / K)
    clocks = sampler.stop()

    # ---- end to end through the host-buffer entry point ------------------------------------------------
    e2e_ms = None
    if e2e and not args.no_e2e:
        hb = [[g.cpu().pin_memory() for g in batches[s]] for s in range(min(2, nb))]
        hidx = torch.empty(w.k, dtype=torch.int32).pin_memory()
        hval = torch.empty(w.k, dtype=torch.float32).pin_memory()
        ke = max(3, min(K, 20))
        for s in range(2):
            ctx.step_host(hb[s % len(hb)], mem, theta, t, hidx, hval)
            t += 1
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for s in range(ke):
            ctx.step_host(hb[s % len(hb)], mem, theta, t, hidx, hval)
            t += 1
        e1.record(stream)
        barrier()
        e2e_ms = e0.elapsed_time(e1) / ke
        del hb

    # ---- max over ranks --------------------------------------------------------------------------------
    ms_total, e2e_max = max_over_ranks([ms_total, e2e_ms or 0.0], dev)
    e2e_ms = e2e_max if e2e_ms is not None else None

    out = None
    if rank == 0:
        ms_step = ms_total / K
        peak, peak_src = measured_peak()
        lp_ms = kms[1] / max(ksteps, 1)
        tk_ms = kms[0] / max(ksteps, 1)
        tk_bytes = 8.0 * w.d + 4.0 * w.k
        # the one-kernel step does the selection's reads too: the step's algorithmic bytes are its kernel's
        lp_bytes = 12.0 * w.n * w.d + (tk_bytes if one_kernel else 0.0)
        lp_gbs = lp_bytes / (lp_ms * 1e-3) / 1e9
        traffic = NCU_TRAFFIC.get(w.name, {})
        sel_kernel = {"topk": "topk_select_kernel", "chunk": "chunk_select_kernel", "layer_topk": "layer_topk_kernel"}[args.selector]
        main_kernel = "small_step_kernel" if one_kernel else "learner_pass_kernel"
        lp_span = sms[1] / max(ssteps, 1)
        in_kernel = {"note": "first block start to last block end on the GPU timer, no launch gap or event overhead; "
                             "same steps as the event figures",
                     main_kernel: lp_span, "step_frac" if one_kernel else "learner_frac": lp_bytes / (lp_span * 1e-3) / 1e9 / peak}
        sel_block = None
        if not one_kernel:
            tk_gbs = tk_bytes / (tk_ms * 1e-3) / 1e9
            tk_span = sms[0] / max(ssteps, 1)
            sel_block = {"achieved": tk_gbs, "frac": tk_gbs / peak, "avg_launch_ms": tk_ms,
                         "algorithmic_bytes_per_launch": tk_bytes, "traffic": traffic.get(sel_kernel),
                         "frac_of_nominal_8TBs": tk_gbs / NOMINAL_HBM_GBS}
            in_kernel[sel_kernel] = tk_span
            in_kernel["selection_frac"] = tk_bytes / (tk_span * 1e-3) / 1e9 / peak
        out = {
            "metric": METRIC, "value": job_value(w.n, w.d, world, ms_step), "unit": UNIT, "n_gpus": world,
            "steps": K, "warmup": Wm, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "n": w.n, "d": w.d, "k": w.k, "beta": w.beta, "lr": w.lr,
                       "parallelism": "replicas only" if world > 1 else "single GPU, n logical learners",
                       "l2": "inputs larger than L2 (%.2f GB of g+m per step), no flush" % (8e-9 * w.n * w.d)
                             if 8 * w.n * w.d > 126e6 else
                             "g+m (%.0f MB) fit L2: the memories stay cached from step to step, the gradients cycle through "
                             "%d resident batches (%.0f MB) and come from HBM" % (8e-6 * w.n * w.d, nb, 4e-6 * nb * w.n * w.d),
                       "gradient_batches_resident": nb, "selector": args.selector, "l2_keep": args.l2_keep,
                       "steps_before_timing": Wm + late_steps,
                       "selection_path_last_step": paths, "selection_candidates_last_step": cands,
                       "kernels_per_step": 1 if one_kernel else 2,
                       "weight_update": "fused into the learner pass"},
            "roofline": {"bound": "hbm", "kernel": main_kernel, "achieved": lp_gbs, "peak": peak,
                         "unit": "GB/s", "frac": lp_gbs / peak, "traffic": traffic.get(main_kernel),
                         "traffic_captured": traffic.get("captured"),
                         "peak_source": peak_src, "algorithmic_bytes_per_launch": lp_bytes, "avg_launch_ms": lp_ms,
                         "frac_of_nominal_8TBs": lp_gbs / NOMINAL_HBM_GBS,
                         "steps_timed": ksteps, "ms_per_step_with_kernel_events": ms_total_b / K,
                         "in_kernel_ms": in_kernel},
            "gpu_launches": launches,
            "clocks": clocks,
        }
        if sel_block is not None:
            out["roofline"][sel_kernel] = sel_block
        if repeats:
            rs = sorted(repeats)
            out["repeats"] = {"regions": len(rs), "steps_each": K, "ms_per_step_median": rs[len(rs) // 2],
                              "ms_per_step_min": rs[0], "ms_per_step_max": rs[-1],
                              "note": "the K-step region timed again; the headline is the first region alone"}
        if e2e_ms is not None:
            out["e2e"] = {"value": job_value(w.n, w.d, world, e2e_ms), "unit": UNIT,
                          "h2d_bytes_per_step": 4 * w.n * w.d, "d2h_bytes_per_step": 8 * w.k,
                          "ms_per_step": e2e_ms, "api": "scalecom_step_host (pinned host gradients in, idx/val out)"}
        if world == 1 and cpu_baseline and not args.no_cpu_baseline:
            out["cpu_baseline"] = time_oracle(w, batches, selector=args.selector, layers=layers)
    ctx.close()
    del batches, mem, theta, idx, val, step
    torch.cuda.empty_cache()
    return out


ALL_WORKLOADS = ["tiny", "resnet50", "transformer_base", "resnet50_n8", "resnet50_n32", "resnet50_n64", "resnet50_n128",
                 "gpt2_medium"]


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.deployment == "learner-per-gpu":
        run_learner_per_gpu(args)
        return

    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    stream = torch.cuda.Stream(device=dev)
    if args.workload != "all":
        out = bench_workload(args, args.workload, world, rank, dev, stream, barrier, late_steps=args.late_steps)
        if rank == 0:
            print(json.dumps(out))
    else:
        # every configuration, one JSON line each (not the driver's single-line mode), then the learner sweep's fit
        lines = {}
        for name in ALL_WORKLOADS:
            out = bench_workload(args, name, world, rank, dev, stream, barrier, cpu_baseline=False, e2e=False)
            if rank == 0:
                lines[name] = out
                print(json.dumps(out), flush=True)
        late = bench_workload(args, "resnet50", world, rank, dev, stream, barrier, late_steps=args.late_steps or 1500,
                              cpu_baseline=False, e2e=False)
        if rank == 0:
            late["config"]["note"] = "late in a run: the steps before timing let error feedback pile coordinates up under the threshold"
            print(json.dumps(late), flush=True)
            peak, _ = measured_peak()
            ns = [8, 32, 64, 128]
            ts = [lines["resnet50_n%d" % n]["ms_per_step"] for n in ns]
            slope, icpt = fit_line(ns, ts)
            d = lines["resnet50_n8"]["config"]["d"]
            print(json.dumps({
                "learner_sweep_fit": {"n": ns, "ms_per_step": ts, "slope_ms_per_learner": slope, "intercept_ms": icpt,
                                      "12d_over_measured_peak_ms": 12.0 * d / (peak * 1e9) * 1e3,
                                      "12d_over_nominal_8TBs_ms": 12.0 * d / (NOMINAL_HBM_GBS * 1e9) * 1e3,
                                      "selection_ms_by_events": [lines["resnet50_n%d" % n]["roofline"]["topk_select_kernel"]["avg_launch_ms"] for n in ns],
                                      "note": "step time is linear in the number of simulated learners (12 d bytes each), "
                                              "the intercept is the selection: the paper's constant-in-n claim is about "
                                              "communication volume, not about n learners simulated in one GPU"}}), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
