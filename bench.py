#!/usr/bin/env python
"""Benchmark of the fused finite-difference PDE-residual hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl fpde|reference]

One "step" = one fused forward (all residual fields + loss) plus one adjoint (gradient of that
loss, boundary correction included) over one synthetic grid, through the C ABI.  The default
workload is the 3-D unsteady Navier-Stokes (Taylor-Green) configuration, 128^3 x 16 space-time
points, four fields: the paper's headline operator and the largest configuration; its 2.5 GB of
per-step traffic is far beyond L2, so back-to-back steps need no cache flush.

Prints ONE JSON line (rank 0).  `value` is grid points per second over all GPUs (replicas: the
path has no exchange step, so N GPUs run N independent grids, weak scaling).
`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2607_18020_b200 import workloads as W

METRIC = "grid-points/s for fused fwd+bwd residual loss"
UNIT = "grid-points/s"
DEFAULT_WORKLOAD = "ns_tgv_128x16"

# Algorithmic bytes per grid point (fp32, every array touched once): forward reads fields and
# sources and writes residuals; the adjoint reads the upstream arrays plus the fields its
# Jacobian needs and writes one gradient per field.
ALGO_BYTES = {                      # op: (fwd, bwd)
    W.BURGERS_1D_T: (8, 12),
    W.POISSON_2D: (12, 8),
    W.GRAYSCOTT_2D: (16, 24),
    W.HELMHOLTZ_3D_O4: (12, 8),
    W.NS_3D_T: (32, 44),
    W.NS_2D_STEADY: (24, 32),
    W.NS_3D_STEADY: (32, 44),
}
KERNEL_NAMES = {                    # op: (fwd kernel, bwd kernel)
    W.BURGERS_1D_T: ("burgers_fwd_kernel", "burgers_bwd_kernel"),
    W.POISSON_2D: ("lap2d_kernel<PoissonFwd>", "lap2d_kernel<PoissonBwd>"),
    W.GRAYSCOTT_2D: ("lap2d_kernel<GrayScottFwd>", "lap2d_kernel<GrayScottBwd>"),
    W.HELMHOLTZ_3D_O4: ("star3d_kernel<fwd>", "star3d_tma_kernel<bwd>"),
    W.NS_3D_T: ("ns_fwd_kernel", "ns_bwd_kernel"),
    W.NS_2D_STEADY: ("ns2d_kernel<fwd>", "ns2d_kernel<bwd>"),
    W.NS_3D_STEADY: ("ns3d_kernel<fwd>", "ns3d_kernel<bwd>"),
}
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures
# summarised under profiles/; None where no capture has been taken yet.
NCU_TRAFFIC_BYTES = {
    # half-size capture (64 planes) x 2: traffic is proportional to the number of planes
    ("ns_tgv_128x16", "ns_fwd_kernel"): 2 * 518003968,
    ("ns_tgv_128x16", "ns_bwd_kernel"): 2 * 762521088,
    ("grayscott_4096", "lap2d_kernel<GrayScottFwd>"): 222671616,
    ("grayscott_4096", "lap2d_kernel<GrayScottBwd>"): 366043648,
    ("helmholtz_256", "star3d_kernel<fwd>"): 171900000,
    ("helmholtz_256", "star3d_tma_kernel<bwd>"): 97610000,
    ("ns2d_steady_4096", "ns2d_kernel<fwd>"): 362135040,
    ("ns2d_steady_4096", "ns2d_kernel<bwd>"): 511582720,
    ("ns3d_steady_256", "ns3d_kernel<fwd>"): 516224256,
    ("ns3d_steady_256", "ns3d_kernel<bwd>"): 735408896,
    ("grayscott_4096", "fused2d_kernel<grayscott_2d>"): 235188736,
    ("ns2d_steady_4096", "fused2d_kernel<ns_2d_steady>"): 372255488,
}
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0            # the vendor figure the workload text quotes; fractions of it go beside the measured ones
LAUNCHES_PER_STEP = 3               # forward kernel, loss finalise, adjoint kernel


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------------------
# clocks: sampled through NVML (read-only) while the timed region runs
# ------------------------------------------------------------------------------------------
_REASONS = {0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x10: "sync_boost",
            0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}


class ClockSampler:
    """Reads SM clock and clock-event reasons through NVML while the timed loops run.  The period is
    kept coarse (25 ms): polling NVML every few milliseconds was measured to slow the kernels under
    test by ~7 %."""

    def __init__(self, torch, device_index: int, period_s: float = 0.025):
        self.samples, self.stamps, self.reasons, self.max_mhz = [], [], set(), None
        self.period = period_s
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            p = torch.cuda.get_device_properties(device_index)
            bus = "%08x:%02x:%02x.0" % (p.pci_domain_id, p.pci_bus_id, p.pci_device_id)
            self._h = pynvml.nvmlDeviceGetHandleByPciBusId(bus.encode())
            self._nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception as exc:      # NVML unavailable: report that instead of numbers
            self.error = repr(exc)

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                self.stamps.append(time.perf_counter())
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in _REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()

    def mhz_between(self, t0: float, t1: float):
        """Median SM clock of the samples taken in [t0, t1] (host clock), else the sample nearest to it."""
        inside = [m for m, t in zip(self.samples, self.stamps) if t0 <= t <= t1]
        if inside:
            return statistics.median(inside)
        if not self.samples:
            return None
        mid = 0.5 * (t0 + t1)
        return min(zip(self.samples, self.stamps), key=lambda p: abs(p[1] - mid))[0]

    def summary(self):
        if self._h is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "error": getattr(self, "error", "nvml unavailable")}
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------
def oracle_sample(name: str, planes: int, seed: int = 42):
    """A bounded sample of a workload: its first `planes` slices along the slowest axis, taken
    as a grid of its own (same spacings, same recipe)."""
    cfg = W.CONFIGS[name]
    shape = list(cfg["shape"])
    planes = max(5, min(shape[0], planes))
    full = W.make(name, seed=seed, shape=[planes] + shape[1:], spacing=_spacing_of(name))
    return full


def _spacing_of(name):
    cfg = W.CONFIGS[name]
    hs = []
    for n, (lo, hi), b in zip(cfg["shape"], cfg["domain"], cfg["bc"]):
        hs.append((hi - lo) / n if b == W.PERIODIC else (hi - lo) / (n - 1))
    return tuple(hs)


def time_oracle(w, reps: int):
    import oracle
    best = float("inf")
    for _ in range(reps):
        t0 = time.perf_counter()
        oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
        best = min(best, time.perf_counter() - t0)
    return best


def _oracle_worker(args):
    """One worker of the all-cores leg: the oracle, as it stands, on this worker's own sample (the
    first `planes` slices of the workload's recipe under the worker's own seed)."""
    name, planes, seed, reps, t_go = args
    w = oracle_sample(name, planes, seed=seed)
    import oracle
    oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)      # warm-up: page-in, library load
    while time.time() < t_go:                       # all workers start their timed passes together
        time.sleep(0.001)
    t0 = time.time()
    for _ in range(reps):
        oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    return t0, time.time(), w.npoints * reps


def cpu_baseline_all_cores(name: str, planes_per_worker: int, reps: int = 2):
    """P = os.cpu_count() processes, each running the single-thread oracle on its own sample at the
    same time; aggregate points per second over the window from the first start to the last end."""
    import multiprocessing as mp
    P = min(os.cpu_count() or 1, 64)                # one process per host core (at most 64: each holds ~250 MB)
    n0 = W.CONFIGS[name]["shape"][0]
    planes = max(5, min(planes_per_worker, n0))
    ctx = mp.get_context("spawn")
    t_go = time.time() + 8.0 + 0.1 * P                      # imports, sample generation and the warm-up pass come first
    with ctx.Pool(P) as pool:
        out = pool.map(_oracle_worker, [(name, planes, 1042 + i, reps, t_go) for i in range(P)], chunksize=1)
    t_first, t_last = min(o[0] for o in out), max(o[1] for o in out)
    pts = sum(o[2] for o in out)
    late = sum(1 for o in out if o[0] > t_go + 0.5)
    return {"value": pts / (t_last - t_first), "cores": P, "planes_per_worker": planes, "reps": reps,
            "seconds": t_last - t_first, "late_starters": late}


def cpu_baseline(name: str):
    """The oracle as it stands, fwd + bwd, on a bounded sample: one thread, and one process per host
    core running at the same time (the oracle itself is single-threaded and stays so)."""
    cfg_shape = W.CONFIGS[name]["shape"]
    per_plane = int(np.prod(cfg_shape[1:]))
    planes = max(5, min(cfg_shape[0], int(8.0e6 // per_plane) or 1))
    w = oracle_sample(name, planes)
    t = time_oracle(w, 3)
    single = w.npoints / t
    out = {"value": single, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": "first %d of %d slices along axis 0 of %s (%d points), fp64 fwd+bwd incl. loss, best of 3"
                     % (w.shape[0], cfg_shape[0], name, w.npoints),
           "seconds": t, "host_cores": os.cpu_count()}
    try:
        allc = cpu_baseline_all_cores(name, max(5, int(2.0e6 // per_plane) or 1))
        out.update({"single_thread": single, "value": allc["value"], "cores": allc["cores"],
                    "sample": "%d processes at once, each the single-thread oracle on its own seeded sample of %d "
                              "slices along axis 0 of %s, %d passes each (fp64 fwd+bwd incl. loss); single_thread = "
                              "one process on %d slices, best of 3"
                              % (allc["cores"], allc["planes_per_worker"], name, allc["reps"], w.shape[0]),
                    "seconds_all_cores": allc["seconds"], "late_starters": allc["late_starters"]})
    except Exception as exc:             # no multiprocessing here: the one-thread figure stands
        out["all_cores_error"] = repr(exc)
    return out


def run_reference(args, rank):
    """--impl reference: the CPU oracle on a bounded sample, one sample pass per step."""
    if rank != 0:
        return
    name = args.workload
    cfg_shape = W.CONFIGS[name]["shape"]
    per_plane = int(np.prod(cfg_shape[1:]))
    # keep the whole run near two minutes whatever K and W are (the oracle does ~2.5e6 points/s)
    budget_points = 120.0 * 2.5e6 / max(1, args.steps + args.warmup)
    planes = max(5, min(cfg_shape[0], int(budget_points // per_plane)))
    w = oracle_sample(name, planes)
    import oracle
    for _ in range(args.warmup):
        oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    dt = time.perf_counter() - t0
    value = w.npoints * args.steps / dt
    sample = "first %d of %d slices along axis 0 (%d points per step)" % (w.shape[0], cfg_shape[0], w.npoints)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": name, "shape": list(w.shape), "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------------------
# GPU legs
# ------------------------------------------------------------------------------------------
class DeviceProblem:
    def __init__(self, torch, B, w):
        self.w, self.B, self.torch = w, B, torch
        self.fields = [torch.from_numpy(f).cuda() for f in w.fields]
        self.sources = [torch.from_numpy(s).cuda() for s in w.sources]
        ne = len(W.OP_META[w.op]["residuals"])
        self.res = [torch.empty(w.shape, dtype=torch.float32, device="cuda") for _ in range(ne)]
        self.grads = [torch.empty(w.shape, dtype=torch.float32, device="cuda") for _ in w.fields]
        self.loss = torch.zeros(ne + 1, dtype=torch.float64, device="cuda")
        self.ws = torch.empty(B.workspace_bytes(w.op, w.shape), dtype=torch.uint8, device="cuda")
        self.gscale = [2.0 / B.row_count(w.op, w.shape)] * ne

        # the C arguments of the three calls, marshalled once: on small grids the per-call marshalling
        # costs more host time than the kernels take
        self.ws2 = torch.empty(B.fwd_bwd_workspace_bytes(w.op, w.shape), dtype=torch.uint8, device="cuda")
        self.step = B.PreparedStep(w.op, self.fields, self.sources, self.res, self.grads, self.loss, w.shape, w.spacing,
                                   w.coeffs, w.bc, workspace=self.ws, gscale=self.gscale, fwd_bwd_workspace=self.ws2)
        self._store_res = not B.has_single_pass(w.op)          # two-kernel operators need the intermediate

    def fwd(self):
        self.step.fwd()

    def bwd(self):
        self.step.bwd()

    def fwd_bwd(self):
        """The loss-specialised pass: loss + dL/dfield, residual arrays not stored."""
        self.step.fwd_bwd(store_residuals=self._store_res)


class SlabProblem:
    """One grid split into x-slabs, one per rank: fwd() = field halo exchange + forward kernel,
    bwd() = residual halo exchange + adjoint kernel + loss all-reduce."""

    def __init__(self, torch, B, w, world, rank, dist):
        from paper_2607_18020_b200 import slabs as S
        self.S, self.dist, self.w = S, dist, w
        self.rank = S.SlabRank(torch, B, S.plans(w.op, w.shape, world)[rank], w.spacing, w.coeffs)
        self.rank.load_owned(w.fields, w.sources)
        self.R = self.rank.plan.radius
        self.loss = torch.zeros(self.rank.ne + 1, dtype=torch.float64, device="cuda")
        # launches over plane ranges (inner planes while the halos are in flight) only pay with real transfers
        self.chunks = self.rank.chunk_plan() if world > 1 else None

    def fwd(self):
        ex = self.S.post_exchange(self.rank.plan, self.rank.field_stack, 2 * self.R, self.dist)
        if self.chunks is not None:             # planes away from the halos while the halos are in flight
            self.rank.fwd_inner(self.chunks[0])
            ex.wait()
            self.rank.fwd_edges(self.chunks[0])
        else:
            ex.wait()
            self.rank.fwd()

    def bwd(self):
        ex = self.S.post_exchange(self.rank.plan, self.rank.res_stack, self.R, self.dist)
        self.loss.copy_(self.rank.loss)             # this slab's share; the shares add up to the grid's loss
        work = self.dist.all_reduce(self.loss, op=self.dist.ReduceOp.SUM, async_op=True) if self.dist is not None else None
        if self.chunks is not None:
            self.rank.bwd_inner(self.chunks[1])
            ex.wait()
            self.rank.bwd_edges(self.chunks[1])
        else:
            ex.wait()
            self.rank.bwd()
        if work is not None:
            work.wait()


def timed_steps(torch, prob, steps, warmup, barrier, flush=None, inner_events=False):
    """K back-to-back steps between two events.  With inner_events, every forward and adjoint call
    is bracketed by its own events as well (per-call durations; the extra records sit between
    launches, so this variant is used for the per-kernel figures, not for the headline)."""
    for _ in range(warmup):
        prob.fwd(); prob.bwd()
    first, last = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)] if inner_events else None
    barrier(); torch.cuda.synchronize()
    first.record()
    for k in range(steps):
        if flush is not None:
            flush.fill_(k)
        if inner_events:
            ev[k][0].record(); prob.fwd(); ev[k][1].record(); prob.bwd(); ev[k][2].record()
        else:
            prob.fwd(); prob.bwd()
    last.record()
    torch.cuda.synchronize(); barrier()
    total_ms = first.elapsed_time(last)
    if not inner_events:
        return total_ms, None, None
    fwd_ms = [e[0].elapsed_time(e[1]) for e in ev]
    bwd_ms = [e[1].elapsed_time(e[2]) for e in ev]
    return total_ms, fwd_ms, bwd_ms


def e2e_steps(torch, B, w, steps, warmup, barrier):
    """The same step from pinned HOST buffers through fpde_loss_grad_host: per step, H2D of every
    field/source, forward, adjoint, D2H of every gradient and of the loss, then a stream sync (the
    caller reads the loss)."""
    # the fields (and the gradients) are slices of ONE pinned buffer each: evenly spaced arrays let the
    # library move a range of planes of all of them in one strided copy
    hf_all = torch.stack([torch.from_numpy(f) for f in w.fields]).pin_memory()
    hg_all = torch.empty((len(w.fields),) + tuple(w.shape), dtype=torch.float32).pin_memory()
    hf, hg = list(hf_all.unbind(0)), list(hg_all.unbind(0))
    hs = [torch.from_numpy(s).pin_memory() for s in w.sources]
    ne = len(W.OP_META[w.op]["residuals"])
    hl = torch.zeros(ne + 1, dtype=torch.float64).pin_memory()
    arena = torch.empty(B.host_arena_bytes(w.op, w.shape), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        B.fpde_loss_grad_host(w.op, hf, hs, hg, hl, w.shape, w.spacing, w.coeffs, w.bc, arena)
        stream.synchronize()
        return float(hl[-1])

    for _ in range(warmup):
        step()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(); torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        loss = step()
    e1.record()
    torch.cuda.synchronize(); barrier()
    nbytes = w.npoints * 4
    return e0.elapsed_time(e1), nbytes * (len(hf) + len(hs)), nbytes * len(hg) + 8 * (ne + 1), loss


def graph_points_per_s(torch, prob, N, pairs, replays):
    """`pairs` forward+adjoint pairs captured into one CUDA graph and replayed; None if capture is
    not possible here."""
    try:
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            prob.fwd(); prob.bwd()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        with torch.cuda.graph(g):
            for _ in range(pairs):
                prob.fwd(); prob.bwd()
        for _ in range(2):
            g.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(replays):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return N * pairs * replays / (e0.elapsed_time(e1) * 1e-3)
    except Exception:
        torch.cuda.synchronize()
        return None


def single_pass_figures(torch, prob, steps, warmup, flush, peak):
    """fpde_fwd_bwd (one kernel: residuals stay in registers, loss and gradients come out): cold
    per-call median and a warm back-to-back figure.  Algorithmic bytes: every field and source
    read once, every gradient written once."""
    w = prob.w
    N = w.npoints
    bpp = 4 * (2 * len(w.fields) + len(w.sources))
    for _ in range(warmup):
        prob.fwd_bwd()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(steps)]
    torch.cuda.synchronize()
    for k in range(steps):
        flush.fill_(k)
        ev[k][0].record(); prob.fwd_bwd(); ev[k][1].record()
    torch.cuda.synchronize()
    ms = statistics.median(e[0].elapsed_time(e[1]) for e in ev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        prob.fwd_bwd()
    e1.record(); torch.cuda.synchronize()
    warm_ms = e0.elapsed_time(e1) / steps
    gbs = bpp * N / (ms * 1e-3) / 1e9

    class OneCall:                      # the same step for the graph helper (one call instead of a pair)
        fwd = staticmethod(prob.fwd_bwd)
        bwd = staticmethod(lambda: None)

    return {"ms": ms, "points_per_s": N / (ms * 1e-3), "warm_points_per_s": N / (warm_ms * 1e-3),
            "graph_points_per_s": graph_points_per_s(torch, OneCall, N, pairs=10, replays=max(3, steps // 10)),
            "algorithmic_bytes_per_point": bpp, "gbs": gbs, "frac": gbs / peak,
            "what": "fpde_fwd_bwd, residual arrays not stored; launches: 1 kernel + loss finalise"}


def rotating_figures(torch, B, w, prob, steps, peak):
    """Cold without a flush: the step runs back to back over three sets of arrays in turn (each set
    larger than half of L2, all three several times L2), so every array comes from DRAM, nothing of
    a flush has to be written back, and consecutive launches overlap as they do in use."""
    fb, bb = ALGO_BYTES[w.op]
    N = w.npoints
    probs = [prob] + [DeviceProblem(torch, B, w) for _ in range(2)]
    for q in probs:
        q.fwd(); q.bwd()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for k in range(steps):
        q = probs[k % 3]
        q.fwd(); q.bwd()
    e1.record(); torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    del probs
    return {"ms_per_step": ms, "points_per_s": N / (ms * 1e-3), "frac_pair": (fb + bb) * N / (ms * 1e-3) / 1e9 / peak,
            "what": "%d steps back to back over three sets of arrays in turn (no flush, every array from DRAM)" % steps}


def sustained_figures(torch, prob, N, pair_bytes, peak, seconds=1.0):
    """The step back to back for about a second; the figure is that of the second half (the SM clock
    settles under the power cap a few tenths of a second into a sustained load)."""
    for _ in range(3):
        prob.fwd(); prob.bwd()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(20):
        prob.fwd(); prob.bwd()
    e1.record(); torch.cuda.synchronize()
    n = max(40, int(seconds * 1e3 / max(e0.elapsed_time(e1) / 20, 1e-3)))
    half = n // 2
    sm = ClockSampler(torch, torch.cuda.current_device())
    ea, eb, ec = (torch.cuda.Event(enable_timing=True) for _ in range(3))
    sm.start()
    ea.record()
    for k in range(n):
        if k == half:
            eb.record()
        prob.fwd(); prob.bwd()
    ec.record(); torch.cuda.synchronize()
    sm.stop()
    ms = eb.elapsed_time(ec) / (n - half)
    clk = sm.summary()
    return {"ms_per_step": ms, "points_per_s": N / (ms * 1e-3), "frac_pair": pair_bytes / (ms * 1e-3) / 1e9 / peak,
            "sm_mhz_median": clk.get("sm_mhz"), "reasons": clk.get("reasons"),
            "ms_x_mhz": None if clk.get("sm_mhz") is None else ms * clk["sm_mhz"],
            "what": "second half of a ~%.0f s back-to-back run" % seconds}


class CleanFlush:
    """An L2 flush that leaves the cache clean: the 256 MiB write, then a read of another 256 MiB.
    After the write alone the whole L2 holds dirty lines, and the first kernel that follows pays
    for writing them back (about 126 MB of DRAM traffic that is not its own)."""

    def __init__(self, torch, write_buf):
        self.w = write_buf
        self.r = torch.zeros(64 << 20, dtype=torch.float32, device="cuda")
        self.acc = torch.zeros((), dtype=torch.float32, device="cuda")

    def fill_(self, k):
        self.w.fill_(k)
        self.acc += self.r.sum()


def config_line(torch, B, name, steps, warmup, peak):
    """Secondary figures for one configuration: per-call medians with an L2 flush (a 256 MiB
    write) before every step, so small grids are measured cold like large ones."""
    w = W.make(name, seed=42)
    prob = DeviceProblem(torch, B, w)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    _, f_ms, b_ms = timed_steps(torch, prob, steps, warmup, lambda: None, flush=flush, inner_events=True)
    fm, bm = statistics.median(f_ms), statistics.median(b_ms)
    fb, bb = ALGO_BYTES[w.op]
    N = w.npoints
    out = {"shape": list(w.shape), "points": N, "ms_fwd": fm, "ms_bwd": bm, "ms_fwd_min": min(f_ms), "ms_bwd_min": min(b_ms),
           "points_per_s": N / ((fm + bm) * 1e-3),
           "gbs_fwd": fb * N / (fm * 1e-3) / 1e9, "gbs_bwd": bb * N / (bm * 1e-3) / 1e9,
           "gbs_pair": (fb + bb) * N / ((fm + bm) * 1e-3) / 1e9}
    out["frac_pair"] = out["gbs_pair"] / peak
    out["frac_pair_min"] = (fb + bb) * N / ((min(f_ms) + min(b_ms)) * 1e-3) / 1e9 / peak
    out["timing"] = "cold: 256 MiB L2 flush before every step, per-call medians (and minima) of %d steps after %d" % (steps, warmup)
    # the same with the cache left clean (write, then read another buffer): what the kernels do when
    # they do not also have to write back the flush's dirty lines
    clean = CleanFlush(torch, flush)
    _, f_ms, b_ms = timed_steps(torch, prob, steps, warmup, lambda: None, flush=clean, inner_events=True)
    fc, bc = statistics.median(f_ms), statistics.median(b_ms)
    out["clean_l2"] = {"ms_fwd": fc, "ms_bwd": bc, "frac_pair": (fb + bb) * N / ((fc + bc) * 1e-3) / 1e9 / peak,
                       "what": "flush = 256 MiB write followed by a 256 MiB read (no dirty lines left in L2)"}
    del clean
    # warm, back to back (working sets below L2 stay resident: say so), and the same pairs replayed
    # from one CUDA graph, which removes the host launch gaps of the latency-bound small grids
    total_ms, _, _ = timed_steps(torch, prob, steps, 3, lambda: None)
    out["warm_points_per_s"] = N * steps / (total_ms * 1e-3)
    out["frac_warm"] = (fb + bb) * N * steps / (total_ms * 1e-3) / 1e9 / peak
    out["l2_resident"] = bool((fb + bb) * N < (100 << 20))
    out["graph_points_per_s"] = graph_points_per_s(torch, prob, N, pairs=10, replays=max(3, steps // 10))
    if not out["l2_resident"]:
        out["rotating"] = rotating_figures(torch, B, w, prob, steps, peak)
        out["sustained"] = sustained_figures(torch, prob, N, (fb + bb) * N, peak)
    if B.has_single_pass(w.op):
        out["single_pass"] = single_pass_figures(torch, prob, steps, warmup, flush, peak)
    else:
        # the same pair through the one-call entry point (forward, loss sum, adjoint queued by the
        # library; the adjoint then knows its upstream arrays are residuals it wrote itself)
        for _ in range(3):
            prob.fwd_bwd()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            prob.fwd_bwd()
        e1.record(); torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        out["fwd_bwd_call"] = {"warm_points_per_s": N / (ms * 1e-3), "ms": ms,
                               "frac_pair": (fb + bb) * N / (ms * 1e-3) / 1e9 / peak}
    del prob, flush
    torch.cuda.empty_cache()
    return out


def max_over_ranks(x: float, dist, device) -> float:
    """Slowest rank's figure (the job is as slow as its slowest replica); identity on one rank."""
    if dist is None:
        return x
    import torch
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(world: int, points_per_rank: int, steps: int, slowest_ms: float) -> float:
    """Whole-job throughput of `world` independent replicas: all points processed / slowest time."""
    return world * points_per_rank * steps / (slowest_ms * 1e-3)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=list(W.CONFIG_ORDER + W.EXTRA_CONFIGS))
    ap.add_argument("--impl", default="fpde", choices=["fpde", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip per-config figures and the CPU baseline")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--single-pass", action="store_true",
                    help="time fpde_fwd_bwd (one kernel: loss + gradient, residual arrays not stored) as the step; "
                         "only for operators that have a single-pass kernel")
    ap.add_argument("--one-call", action="store_true",
                    help="time fpde_fwd_bwd as the step for any operator (forward, loss and adjoint queued by one call; "
                         "operators without a single-pass kernel pass their residual arrays as the intermediate)")
    ap.add_argument("--slabs", action="store_true",
                    help="strong scaling: ONE grid split into x-slabs, one per rank, with halo exchange "
                         "(default: independent replicas, weak scaling)")
    ap.add_argument("--shape", default=None, help="override the grid extents, e.g. 64,128,128,16 (profiling runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "fpde" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    from paper_2607_18020_b200 import binding as B
    B.lib()                                   # fail loudly if the CUDA library is missing
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()

    peak, peak_src = measured_peak()
    shape = [int(x) for x in args.shape.split(",")] if args.shape else None
    w = W.make(args.workload, seed=42 if args.slabs else 42 + rank, shape=shape,
               spacing=_spacing_of(args.workload) if shape else None)
    prob = SlabProblem(torch, B, w, world, rank, dist) if args.slabs else DeviceProblem(torch, B, w)
    if args.single_pass:
        if not B.has_single_pass(w.op):
            raise SystemExit("--single-pass: operator %s has no single-pass kernel" % w.op)
        prob.fwd, prob.bwd = prob.fwd_bwd, (lambda: None)
    if args.one_call:
        prob.fwd, prob.bwd = prob.fwd_bwd, (lambda: None)
    N = w.npoints

    sampler = ClockSampler(torch, local_rank)
    sampler.start()
    total_ms, _, _ = timed_steps(torch, prob, args.steps, args.warmup, barrier)
    # same K steps again with an event pair around every call: per-kernel durations for the roofline
    _, fwd_ms, bwd_ms = timed_steps(torch, prob, args.steps, 0, barrier, inner_events=True)
    # The K-step block repeated (every block timed like the first, a host sync and a time stamp
    # between blocks) until about 0.3 s have passed, with the clock sampler running across all of
    # them: median and fastest block, and per block ms x SM MHz, so that a reader can tell a faster
    # kernel from a faster clock.  `value` stays the first block's (the K steps the contract names).
    blocks = []
    if world == 1 and not args.slabs:
        n_blocks = max(10, min(200, int(300.0 / max(total_ms, 1e-3)) + 1))
        for _ in range(n_blocks):
            t0 = time.perf_counter()
            ms, _, _ = timed_steps(torch, prob, args.steps, 0, barrier)
            blocks.append((ms, t0, time.perf_counter()))
    sampler.stop()
    total_ms = max_over_ranks(total_ms, dist, "cuda")
    value = job_value(1 if args.slabs else world, N, args.steps, total_ms)

    e2e_k = max(1, min(args.steps, 20))
    if args.no_e2e or args.slabs:
        e2e_ms, h2d, d2h = float("nan"), 0, 0
    else:
        e2e_ms, h2d, d2h, _ = e2e_steps(torch, B, w, e2e_k, 3, barrier)
    e2e_ms = max_over_ranks(e2e_ms, dist, "cuda")
    e2e_value = None if e2e_ms != e2e_ms else job_value(world, N, e2e_k, e2e_ms)
    if e2e_ms != e2e_ms:
        e2e_ms = None

    fb, bb = ALGO_BYTES[w.op]
    knames = KERNEL_NAMES[w.op]
    f_avg, b_avg = sum(fwd_ms) / len(fwd_ms), sum(bwd_ms) / len(bwd_ms)
    if args.single_pass:        # every field and source read once, every gradient written once
        fb, bb = 4 * (2 * len(w.fields) + len(w.sources)), 0
        knames = ("fused2d_kernel<%s>" % w.op, "-")
        b_avg = 0.0
    elif args.one_call:         # the pair's bytes against the time of the one call
        fb, bb = fb + bb, 0
        knames = ("fpde_fwd_bwd(%s)" % w.op, "-")
        b_avg = 0.0
    dom = 1 if b_avg >= f_avg else 0
    Nk = N // world if args.slabs else N       # grid points one rank's kernels process (own planes)
    dom_bytes = (fb, bb)[dom] * Nk
    dom_ms = (f_avg, b_avg)[dom]
    dom_name = knames[dom]
    achieved = dom_bytes / (dom_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": dom_name, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_source": peak_src,
                "traffic": NCU_TRAFFIC_BYTES.get((args.workload, dom_name)),
                "algorithmic_bytes": dom_bytes, "avg_ms": dom_ms,
                "other_kernel": None if (args.single_pass or args.one_call) else
                                {"kernel": knames[1 - dom], "avg_ms": (f_avg, b_avg)[1 - dom],
                                 "note": "forward figure includes the one-block loss finalise launch",
                                 "achieved": (fb, bb)[1 - dom] * Nk / ((f_avg, b_avg)[1 - dom] * 1e-3) / 1e9},
                "pair_achieved": (fb + bb) * Nk * args.steps / (total_ms * 1e-3) / 1e9,
                "pair_frac": (fb + bb) * Nk * args.steps / (total_ms * 1e-3) / 1e9 / peak}
    roofline["frac_of_nominal_8000"] = achieved / NOMINAL_HBM_GBS
    roofline["pair_frac_of_nominal_8000"] = roofline["pair_achieved"] / NOMINAL_HBM_GBS
    if blocks:
        b_ms = [b[0] / args.steps for b in blocks]
        b_mhz = [sampler.mhz_between(b[1], b[2]) for b in blocks]
        pair_bytes = (fb + bb) * Nk
        roofline["blocks"] = {
            "n": len(blocks), "steps_per_block": args.steps,
            "ms_per_step_median": statistics.median(b_ms), "ms_per_step_min": min(b_ms),
            "pair_frac_median": pair_bytes / (statistics.median(b_ms) * 1e-3) / 1e9 / peak,
            "pair_frac_best": pair_bytes / (min(b_ms) * 1e-3) / 1e9 / peak,
            "ms_x_mhz": [None if m is None else round(t * m, 1) for t, m in zip(b_ms, b_mhz)],
            "sm_mhz": b_mhz,
            "what": "the K-step block repeated back to back; ms_x_mhz = ms per step x median SM MHz sampled during the block"}
    if args.slabs:
        roofline["note"] = "per-call times include the halo exchange of the step (and the loss all-reduce)"
    elif not (args.single_pass or args.one_call):
        # the dominant kernel launched K times back to back between ONE pair of events: its
        # per-launch time with the ramp and tail of consecutive launches overlapping
        # (programmatic dependent launch) as they do inside a step
        call = prob.bwd if dom == 1 else prob.fwd
        for _ in range(3):
            call()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        s0.record()
        for _ in range(args.steps):
            call()
        s1.record(); torch.cuda.synchronize()
        sus_ms = s0.elapsed_time(s1) / args.steps
        roofline["back_to_back"] = {"avg_ms": sus_ms, "achieved": dom_bytes / (sus_ms * 1e-3) / 1e9,
                                    "frac": dom_bytes / (sus_ms * 1e-3) / 1e9 / peak,
                                    "what": "%d consecutive launches of the dominant kernel between one event pair" % args.steps}

    # The same step over about two seconds: on these parts the SM clock comes down from its boost
    # value a few tenths of a second into a sustained load (power management), and these kernels
    # are bound by instruction issue and latency, so the long-run figure is the lower one.
    sustained = None
    if world == 1 and not args.no_extras and not args.slabs:
        s_sampler = ClockSampler(torch, local_rank)
        n_sus = max(200, int(2000.0 / max(total_ms / args.steps, 1e-3)))
        half = n_sus // 2
        ea, eb, ec = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        torch.cuda.synchronize()
        s_sampler.start()
        ea.record()
        for k in range(n_sus):
            if k == half:
                eb.record()
            prob.fwd(); prob.bwd()
        ec.record(); torch.cuda.synchronize()
        s_sampler.stop()
        sus_ms = eb.elapsed_time(ec) / (n_sus - half)
        s_clk = s_sampler.summary()
        sustained = {"steps": n_sus, "seconds": ea.elapsed_time(ec) * 1e-3, "ms_per_step": sus_ms,
                     "value": N / (sus_ms * 1e-3), "pair_frac": (fb + bb) * Nk / (sus_ms * 1e-3) / 1e9 / peak,
                     "pair_frac_of_nominal_8000": (fb + bb) * Nk / (sus_ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
                     "ms_x_mhz": None if s_clk.get("sm_mhz") is None else sus_ms * s_clk["sm_mhz"],
                     "clocks": s_clk, "what": "second half of a ~2 s back-to-back run of the same step"}
        roofline["sustained"] = {k: sustained[k] for k in ("ms_per_step", "pair_frac", "pair_frac_of_nominal_8000", "ms_x_mhz")}
        roofline["sustained"].update({"sm_mhz_median": s_clk.get("sm_mhz"), "reasons": s_clk.get("reasons"),
                                      "what": sustained["what"]})

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "strong" if args.slabs else "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "operator": w.op, "shape": list(w.shape), "points": N,
                   "fields": len(w.fields), "step": "fpde_fwd_bwd (single pass)" if args.single_pass else
                           ("fpde_fwd_bwd (one call)" if args.one_call else "fpde_fwd + fpde_bwd"),
                   "parallelism": ("x-slabs x%d of one grid, halo exchange per step" if args.slabs
                                   else "replicas x%d (no exchange step)") % world,
                   "l2": "per-step traffic %.0f MB >> L2, no flush needed" % ((fb + bb) * N / 1e6)
                         if (fb + bb) * N > (256 << 20) else "working set fits L2: warm-cache number"},
        "clocks": sampler.summary(),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_k, "ms_per_step": None if e2e_ms is None else e2e_ms / e2e_k,
                "what": "fpde_loss_grad_host from pinned host buffers: H2D fields, fwd, bwd, D2H gradients + loss, sync"},
        "gpu_launches": (2 if args.single_pass else LAUNCHES_PER_STEP) * args.steps,
        "roofline": roofline,
        "sustained": sustained,
        "loss": float(prob.loss[-1].item()),
    }
    if world == 1 and not args.no_extras:
        del prob
        torch.cuda.empty_cache()
        line["per_config"] = {name: config_line(torch, B, name, 100, 50, peak) for name in W.CONFIG_ORDER + W.EXTRA_CONFIGS}
        # the same figures in short, inside a key every reader of the line keeps: per workload the
        # pair's fraction of the measured peak cold (L2 flushed by a write), cold with a clean L2,
        # cold over rotating sets of arrays (no flush), back to back, over a second of sustained
        # load, the CUDA-graph figure, and the single-pass / one-call entry point
        short = {}
        for name, c in line["per_config"].items():
            sp, fc = c.get("single_pass"), c.get("fwd_bwd_call")
            short[name] = {"frac_cold": round(c["frac_pair"], 4), "frac_cold_best": round(c["frac_pair_min"], 4),
                           "frac_clean": round(c["clean_l2"]["frac_pair"], 4), "frac_warm": round(c["frac_warm"], 4),
                           "frac_cold_of_nominal_8000": round(c["gbs_pair"] / NOMINAL_HBM_GBS, 4),
                           "points_per_s_cold": c["points_per_s"], "graph_points_per_s": c["graph_points_per_s"],
                           "l2_resident": c["l2_resident"]}
            if sp:
                short[name]["single_pass"] = {"frac": round(sp["frac"], 4), "points_per_s": sp["points_per_s"],
                                              "graph_points_per_s": sp["graph_points_per_s"]}
            if fc:
                short[name]["fwd_bwd_call_frac"] = round(fc["frac_pair"], 4)
            if c.get("rotating"):
                short[name]["frac_rotating"] = round(c["rotating"]["frac_pair"], 4)
            if c.get("sustained"):
                short[name]["sustained"] = {"frac": round(c["sustained"]["frac_pair"], 4), "sm_mhz": c["sustained"]["sm_mhz_median"],
                                            "ms_x_mhz": c["sustained"]["ms_x_mhz"]}
        line["roofline"]["per_workload"] = short
        line["cpu_baseline"] = cpu_baseline(args.workload)
        line["config"]["cpu_sample"] = line["cpu_baseline"]["sample"]
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
