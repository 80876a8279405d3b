#!/usr/bin/env python
"""Benchmark of GDN draft-tree verify + commit (libtreewy) on B200.

A step is one pass of the whole hot path -- treewy_tree_prepare, treewy_verify,
treewy_commit -- over one batch of the 35B-shaped workload (256 sequences x 32 value heads,
16 shared q/k heads, random trees of 32 nodes).  Metric: node*heads/s per layer.

Layer rotation: the bench keeps two independent layer buffer sets; step s prepares and
verifies set s%2 and commits the other set (verified one step earlier).  Every step still
does one prepare + one verify + one commit over a full batch, but a state is committed only
after ~1 GB of other traffic has passed through the 126 MB L2 -- as in serving, where commit
follows the rest of the forward pass -- so no kernel is timed on an L2-resident state.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config ID] [--impl reference]

Timing: after W warm-up steps, blocks of exactly K steps are timed back to back with CUDA events on
the launching stream (at least five blocks, tens of milliseconds in all); `value` and `ms_per_step`
are the median block, min and max stand beside them.  The other benchmark workloads are timed with
the same code and reported under `workloads`.

N > 1 (under torchrun) runs N independent replicas, one per GPU: the path has no exchange
step, so there is no data-path collective (weak scaling).
"""
from __future__ import annotations

import argparse
import contextlib
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2608_20961_b200 import footprint, replicas  # noqa: E402
from paper_2608_20961_b200 import workloads as wl  # noqa: E402

METRIC = "gdn_tree_verify_commit_node_heads_per_s_per_layer"
UNIT = "node*heads/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0          # the nominal HBM3e figure the target also names; context, not the denominator
OTHER_WORKLOADS = (1, 3, 4, 6)    # timed beside the headline workload: 35B-chain5, 397B-wide64, ragged-stress, wide128

# DRAM bytes per launch of the verify kernel on the bench workload: dram__bytes_read.sum +
# dram__bytes_write.sum of the latest ncu capture at batch 96 (151.9 MB + 41.1 MB), scaled by 256/96
# (traffic is linear in the batch).  Writes still dirty in L2 at kernel end are not in it.
VERIFY_DRAM_TRAFFIC = {2: {"bytes": int((151.9e6 + 41.1e6) * 256 / 96),
                           "source": "ncu capture at batch 96 scaled by 256/96: profiles/kernels_35B-tree32_b96.md"}}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), float(p.get("bf16_tflops", 0.0)), "measured"
    return FALLBACK_HBM_GBS, 1590.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.001):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                bits = get_reasons(self.h)
                for name, bit in names.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except (ValueError, IndexError):
            return local
    return local


class LayerSet:
    """Device buffers of one GDN layer for one batch of draft trees, and the library calls on them
    with their arguments marshalled once (``binding.prebound``): a decoding loop calls the library
    with the same buffers step after step, and on the small workloads the Python work of building
    structs and pointer objects per call would otherwise be a visible part of the step."""

    def __init__(self, w: wl.Workload, dev: torch.device):
        from paper_2608_20961_b200 import binding as tw
        self.tw, self.w = tw, w
        d = lambda t: t.to(dev)
        self.off, self.par = d(w.node_offsets), d(w.parent)
        self.alpha, self.beta = d(w.alpha), d(w.beta)
        self.q, self.k, self.v, self.S0 = d(w.q), d(w.k), d(w.v), d(w.S0).clone()
        self.acc = d(w.accepted)
        self.O = torch.empty((w.T, w.H_v, 128), dtype=w.io_dtype, device=dev)
        self.U = torch.empty((w.T, w.H_v, 128), dtype=torch.float32, device=dev)
        self.status = torch.zeros(w.B, dtype=torch.int32, device=dev)
        self.tree = tw.Tree.empty(self.off, self.par, w.H_v, w.max_nodes)
        wide = w.max_nodes > 64          # trees of more than 64 nodes go through the wide-tree calls
        self.prepare = tw.prebound(tw.treewy_tree_prepare_wide if wide else tw.treewy_tree_prepare,
                                   self.tree, self.alpha, self.status)
        self.verify = tw.prebound(tw.treewy_verify_wide if wide else tw.treewy_verify, self.S0, self.q, self.k,
                                  self.v, self.beta, self.tree, w.H_qk, self.O, self.U, self.status)
        self.commit = tw.prebound(tw.treewy_commit_wide if wide else tw.treewy_commit, self.S0, self.U, self.k,
                                  self.tree, w.H_qk, self.acc, None, self.status)
        self._half = self._fused = None
        self._flip = 0
        self._wide = wide

    def raw_step_calls(self):
        """The three calls as plain binding calls on the CURRENT stream (for capture in a CUDA graph)."""
        tw, w = self.tw, self.w
        prep = tw.treewy_tree_prepare_wide if self._wide else tw.treewy_tree_prepare
        ver = tw.treewy_verify_wide if self._wide else tw.treewy_verify
        com = tw.treewy_commit_wide if self._wide else tw.treewy_commit
        return (lambda: prep(self.tree, self.alpha, self.status),
                lambda: ver(self.S0, self.q, self.k, self.v, self.beta, self.tree, w.H_qk, self.O, self.U, self.status),
                lambda: com(self.S0, self.U, self.k, self.tree, w.H_qk, self.acc, None, self.status))

    def _half_calls(self):
        """verify / commit with the pseudo-values kept in fp16 (own buffer)."""
        if self._half is None:
            tw, w = self.tw, self.w
            self.U16 = torch.empty((w.T, w.H_v, 128), dtype=torch.float16, device=self.O.device)
            self._half = (tw.prebound(tw.treewy_verify_half_u, self.S0, self.q, self.k, self.v, self.beta, self.tree,
                                      w.H_qk, self.O, self.U16, self.status),
                          tw.prebound(tw.treewy_commit_half_u, self.S0, self.U16, self.k, self.tree, w.H_qk, self.acc,
                                      None, self.status))
        return self._half

    def verify_half(self):
        self._half_calls()[0]()

    def commit_half(self):
        self._half_calls()[1]()

    def commit_verify(self):
        """Commit of the previous round fused into this round's verify (U double-buffered)."""
        if self._fused is None:
            tw, w = self.tw, self.w
            self.U2 = torch.empty_like(self.U)
            mk = lambda u_prev, u_new: tw.prebound(tw.treewy_commit_verify, self.S0, u_prev, self.k, self.tree,
                                                   self.acc, self.q, self.k, self.v, self.beta, self.tree, w.H_qk,
                                                   self.O, u_new, True, self.status)
            self._fused = (mk(self.U, self.U2), mk(self.U2, self.U))
        self._fused[self._flip]()
        self._flip ^= 1


def pass_bytes(w: wl.Workload) -> footprint.PassBytes:
    off = w.node_offsets.tolist()
    par = w.parent.tolist()
    nodes, plen = [], []
    for b in range(w.B):
        t = par[off[b]:off[b + 1]]
        depth = wl.tree_depths(t)
        a = int(w.accepted[b])
        nodes.append(len(t))
        plen.append(depth[a] + 1 if a >= 0 else 0)
    return footprint.algorithmic_bytes(nodes, plen, w.H_v, w.H_qk, io_elem=w.S0.element_size(),
                                       o_elem=w.S0.element_size())


def oracle_inputs(w: wl.Workload):
    f = lambda t: t.to(torch.float64).numpy()
    return (w.node_offsets.numpy(), w.parent.numpy(), f(w.S0), f(w.q), f(w.k), f(w.v), f(w.alpha),
            f(w.beta), w.accepted.numpy())


def time_oracle(w: wl.Workload, n_seq: int, min_seconds: float = 10.0):
    """The CPU oracle, as it stands, on the first n_seq sequences, repeated until at least
    min_seconds have passed; returns (units/s, seconds, passes, sub-batch, threads)."""
    from oracle import treewy_oracle
    treewy_oracle.build()
    treewy_oracle.set_max_nodes(max(64, w.max_nodes))   # (64 unless the workload has wider trees)
    sub = w.select_sequences(range(min(n_seq, w.B)))
    args = oracle_inputs(sub)
    passes, t0 = 0, time.perf_counter()
    while True:
        treewy_oracle.prepare(args[0], args[1], args[6])
        treewy_oracle.verify_commit(*args)
        passes += 1
        dt = time.perf_counter() - t0
        if dt >= min_seconds or passes >= 64:
            break
    return passes * sub.T * sub.H_v / dt, dt, passes, sub, treewy_oracle.num_threads()


def run_reference(args, rank: int):
    """Reference arm: the fp64 CPU oracle on the host cores, rank 0 only."""
    if rank != 0:
        return
    w = wl.make_workload(args.config, B=args.ref_seqs)
    from oracle import treewy_oracle
    treewy_oracle.build()
    oargs = oracle_inputs(w)
    units = w.T * w.H_v

    def step():
        treewy_oracle.prepare(oargs[0], oargs[1], oargs[6])
        treewy_oracle.verify_commit(*oargs)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = units * args.steps / dt
    full = wl._DEFAULTS[args.config]
    sample = f"{w.B} of {full[1]} sequences of workload {full[0]} per step, all heads"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": full[0], "B": full[1], "H_v": w.H_v, "H_qk": w.H_qk,
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": treewy_oracle.num_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def timed_blocks(step, steps: int, dev, stream, start: int = 0, min_total_ms: float = 40.0, sampler=None):
    """Times blocks of exactly `steps` steps back to back with CUDA events on the launching stream:
    at least five blocks, more when a block is short, so that the whole timed region lasts tens of
    milliseconds.  Barrier and device synchronisation on both sides.  Returns the per-block times
    (ms, this rank) and the index of the next step."""
    ev = lambda: torch.cuda.Event(enable_timing=True)
    p0, p1 = ev(), ev()
    p0.record(stream)
    for i in range(steps):                      # pilot block: sizes the run, not reported
        step(start + i)
    p1.record(stream)
    torch.cuda.synchronize(dev)
    start += steps
    pilot = max(p0.elapsed_time(p1), 1e-3)
    n_blocks = int(min(400, max(5, -(-min_total_ms // pilot))))
    marks = [ev() for _ in range(n_blocks + 1)]
    replicas.barrier(dev)
    torch.cuda.synchronize(dev)
    ctx = sampler if sampler is not None else contextlib.nullcontext()
    with ctx:
        marks[0].record(stream)
        for blk in range(n_blocks):
            for i in range(steps):
                step(start + blk * steps + i)
            marks[blk + 1].record(stream)
        torch.cuda.synchronize(dev)
    replicas.barrier(dev)
    return [marks[i].elapsed_time(marks[i + 1]) for i in range(n_blocks)], start + n_blocks * steps


def block_stats(block_ms, steps: int, dev):
    """Median / min / max over the blocks of the time per step, each the MAX over ranks."""
    s = sorted(block_ms)
    med = 0.5 * (s[(len(s) - 1) // 2] + s[len(s) // 2])
    f = lambda x: replicas.max_over_ranks(x, dev) / steps
    return {"median": f(med), "min": f(s[0]), "max": f(s[-1]), "blocks": len(s),
            "series": [round(x / steps, 5) for x in block_ms]}   # this rank's blocks in time order


def kernel_times(sets, dev, stream, reps: int):
    """Per-call durations (ms), separate pass: events around every call on the launching stream."""
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(reps)]
    for i in range(reps):
        a, b = sets[i % 2], sets[(i + 1) % 2]
        ev[i][0].record(stream)
        a.prepare()
        ev[i][1].record(stream)
        a.verify()
        ev[i][2].record(stream)
        b.commit()
        ev[i][3].record(stream)
    torch.cuda.synchronize(dev)
    return [sum(e[j].elapsed_time(e[j + 1]) for e in ev) / reps for j in range(3)]


def kernel_times_back_to_back(sets, dev, stream, reps: int):
    """Per-call durations (ms) without an event between launches: `reps` launches of ONE entry point
    back to back, the two layer sets alternating (so no launch finds its inputs in L2), one event pair
    around them.  An event pair around every single launch adds the launch latency that consecutive
    launches hide; this is the duration ncu reports for the kernels."""
    out = []
    for name in ("prepare", "verify", "commit"):
        calls = [getattr(s_, name) for s_ in sets]
        for i in range(4):
            calls[i % 2]()
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(reps):
            calls[i % 2]()
        e1.record(stream)
        torch.cuda.synchronize(dev)
        out.append(e0.elapsed_time(e1) / reps)
    for s_ in sets:            # (commit ran without a fresh verify: leave every set verified again)
        s_.prepare(), s_.verify()
    torch.cuda.synchronize(dev)
    return out


def host_cost_per_call(ls: LayerSet, dev, n: int = 100):
    """Host time of one enqueue (microseconds): n calls of each entry point through its marshalled
    C call, no synchronisation inside, wall clock / n.  The queue is drained between the three."""
    out = {}
    for name in ("prepare", "verify", "commit"):
        call = getattr(ls, name)
        torch.cuda.synchronize(dev)
        t0 = time.perf_counter()
        for _ in range(n):
            call()
        out[name] = (time.perf_counter() - t0) / n * 1e6
        torch.cuda.synchronize(dev)
    return out


def graph_replay_ms_per_step(sets, dev, steps: int) -> float:
    """The same step captured in a CUDA graph and replayed: what a caller sees whose host does not have
    to enqueue the launches one by one (the paper's chain path runs under a CUDA graph, Section 4)."""
    calls = [s_.raw_step_calls() for s_ in sets]

    def raw_step(i: int):
        a, b = calls[i % 2], calls[(i + 1) % 2]
        a[0](), a[1](), b[2]()

    n = 2 * ((steps + 1) // 2)            # an even number of steps: a replay leaves the rotation where it was
    side = torch.cuda.Stream(dev)
    side.wait_stream(torch.cuda.current_stream(dev))
    with torch.cuda.stream(side):
        raw_step(0), raw_step(1)
    torch.cuda.current_stream(dev).wait_stream(side)
    torch.cuda.synchronize(dev)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(n):
            raw_step(i)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = max(3, int(40.0 / max(1e-3, n * 0.05)) // 10)
    stream = torch.cuda.current_stream(dev)
    e0.record(stream)
    for _ in range(reps):
        graph.replay()
    e1.record(stream)
    torch.cuda.synchronize(dev)
    return e0.elapsed_time(e1) / (reps * n)


def n_launches(w: wl.Workload) -> int:
    """Kernels per prepare + verify + commit step: a bf16 batch whose trees may exceed 32 nodes verifies
    in two launches (one per size class)."""
    return 4 if w.io_dtype == torch.bfloat16 and 32 < w.max_nodes <= 64 else 3


def measure_workload(w: wl.Workload, dev, stream, steps: int, warmup: int, sampler=None, min_total_ms: float = 40.0):
    """The step (prepare + verify + commit, two layer sets rotated) on one workload: block-median time,
    per-kernel times, roofline fractions against the measured and the nominal bandwidth."""
    pb = pass_bytes(w)
    sets = [LayerSet(w, dev) for _ in range(2)]
    for s_ in sets:                      # every set holds a verified tree before step 0
        s_.prepare(), s_.verify()
    torch.cuda.synchronize(dev)

    def step(i: int):
        a, b = sets[i % 2], sets[(i + 1) % 2]
        a.prepare()
        a.verify()
        b.commit()

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize(dev)
    blocks, nxt = timed_blocks(step, steps, dev, stream, start=warmup, sampler=sampler, min_total_ms=min_total_ms)
    st = block_stats(blocks, steps, dev)
    kt = kernel_times(sets, dev, stream, max(3, min(steps, 50)))
    kb = kernel_times_back_to_back(sets, dev, stream, max(4, min(steps, 50)))
    graph_ms = graph_replay_ms_per_step(sets, dev, steps)
    assert not any(int(s_.status.max()) for s_ in sets), "a sequence was flagged"
    hbm, tf, which = measured_peaks()
    roof_ms = max(pb.total / (hbm * 1e9), pb.tensor_flops / (tf * 1e12)) * 1e3
    nominal_ms = pb.total / (NOMINAL_HBM_GBS * 1e9) * 1e3
    rec = {
        "ms_per_step": st["median"], "ms_per_step_min": st["min"], "ms_per_step_max": st["max"],
        "blocks": st["blocks"], "steps_per_block": steps, "ms_per_step_blocks": st["series"],
        "kernel_ms": {"prepare": kt[0], "verify": kt[1], "commit": kt[2]},
        "kernel_ms_back_to_back": {"prepare": kb[0], "verify": kb[1], "commit": kb[2]},
        "kernel_gbs": {"prepare": pb.prepare / kb[0] / 1e6, "verify": pb.verify / kb[1] / 1e6,
                       "commit": pb.commit / kb[2] / 1e6},
        "step_roofline": {"bytes": pb.total, "tensor_flops": pb.tensor_flops, "roof_ms": roof_ms,
                          "frac": roof_ms / st["median"], "peak_source": f"of {which}",
                          "frac_of_nominal_8tbs": nominal_ms / st["median"]},
        "gpu_launches_per_step": n_launches(w),
        "graph_replay_ms_per_step": graph_ms,   # the same steps replayed from a CUDA graph
    }
    return rec, sets, pb, kb


def run_ours(args, rank: int, size: int, local: int):
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libtreewy has no CPU path")
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    from paper_2608_20961_b200 import binding as tw
    tw.load_library()
    stream = torch.cuda.current_stream(dev)
    hbm, tf, which = measured_peaks()

    w = wl.make_workload(args.config, B=args.batch, prefix_device=str(dev))
    units = w.T * w.H_v
    clocks = ClockSampler(physical_gpu_index(local))
    main, sets, pb, kt = measure_workload(w, dev, stream, args.steps, args.warmup, sampler=clocks,
                                           min_total_ms=40.0)   # (long enough for a dozen clock samples; beyond ~50 ms of this load the board nears its power limit)
    ms_per_step = main["ms_per_step"]
    value = size * units / (ms_per_step * 1e-3)

    verify_gbs = pb.verify / (kt[1] * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "treewy_verify", "achieved": verify_gbs, "peak": hbm,
                "duration_ms": kt[1], "duration_source": "CUDA events around consecutive launches of the kernel "
                                                         "(kernel_ms_back_to_back); kernel_ms has an event pair per launch",
                "unit": "GB/s", "frac": verify_gbs / hbm, "peak_source": f"of {which}",
                "frac_of_nominal_8tbs": verify_gbs / NOMINAL_HBM_GBS,
                "traffic": VERIFY_DRAM_TRAFFIC.get(args.config, {}).get("bytes"),
                "traffic_source": VERIFY_DRAM_TRAFFIC.get(args.config, {}).get("source"),
                "algorithmic_bytes_per_launch": pb.verify}

    # end to end through the user-level API: pinned host inputs in, outputs back, every step;
    # consecutive steps are pipelined over upload / compute / download streams
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ke = max(4, min(args.steps, 20))
    layer = tw.VerifyCommitLayer(sets[0].S0, w.H_qk, w.T, w.max_nodes)
    names = ("q", "k", "v", "alpha", "beta", "parent", "node_offsets", "accepted")
    hosts = [{n: getattr(w, n).contiguous().clone().pin_memory() for n in names} for _ in range(2)]
    O_hosts = [torch.empty((w.T, w.H_v, 128), dtype=w.io_dtype).pin_memory() for _ in range(2)]
    h2d = sum(t.numel() * t.element_size() for t in hosts[0].values())
    d2h = O_hosts[0].numel() * O_hosts[0].element_size()
    for i in range(4):
        layer.step_async(hosts[i & 1], O_hosts[i & 1])
    layer.synchronize()
    torch.cuda.synchronize(dev)
    replicas.barrier(dev)
    e0.record(stream)
    layer.s_up.wait_event(e0)
    for i in range(ke):
        layer.step_async(hosts[i & 1], O_hosts[i & 1])
    for st in (layer.s_up, layer.s_run, layer.s_down):
        stream.wait_stream(st)
    e1.record(stream)
    torch.cuda.synchronize(dev)
    e2e_ms = replicas.max_over_ranks(e0.elapsed_time(e1), dev)
    e2e = {"value": size * units * ke / (e2e_ms * 1e-3), "unit": UNIT, "steps": ke,
           "ms_per_step": e2e_ms / ke, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
           "note": "pinned host buffers; upload, kernels and download pipelined over three streams"}
    del layer, hosts, O_hosts

    def variant(step, warm_first=None):
        if warm_first is not None:
            warm_first()
        for i in range(max(args.warmup, 3)):
            step(i)
        torch.cuda.synchronize(dev)
        blocks, _ = timed_blocks(step, args.steps, dev, stream, start=max(args.warmup, 3), min_total_ms=20.0)
        return block_stats(blocks, args.steps, dev)

    # the same hot path with the commit of round r fused into the verify of round r+1
    # (treewy_commit_verify): step = prepare + commit_verify on one layer set, sets rotated
    fused = None
    if w.io_dtype == torch.bfloat16 and w.max_nodes <= 32:
        st = variant(lambda i: (sets[i % 2].prepare(), sets[i % 2].commit_verify()))
        fbytes = pb.total - w.B * w.H_v * 128 * 128 * w.S0.element_size()   # the state is read once
        fused = {"what": "prepare + treewy_commit_verify(single_kernel=1) per step: the previous round's commit "
                         "and this round's verify in one kernel, state read once and written once",
                 "ms_per_step": st["median"], "ms_per_step_min": st["min"], "ms_per_step_max": st["max"],
                 "value": size * units / (st["median"] * 1e-3), "unit": UNIT,
                 "algorithmic_bytes": fbytes, "roof_ms": fbytes / (hbm * 1e9) * 1e3,
                 "frac": fbytes / (hbm * 1e9) * 1e3 / st["median"],
                 "frac_of_nominal_8tbs": fbytes / (NOMINAL_HBM_GBS * 1e9) * 1e3 / st["median"],
                 "gpu_launches_per_step": 2}
        assert not any(int(s_.status.max()) for s_ in sets), "a sequence was flagged"

    # the three calls with U kept in fp16 (treewy_verify_half_u / treewy_commit_half_u): same step shape
    half_u = None
    if w.io_dtype == torch.bfloat16 and w.max_nodes <= 64:
        st = variant(lambda i: (sets[i % 2].prepare(), sets[i % 2].verify_half(), sets[(i + 1) % 2].commit_half()),
                     warm_first=lambda: [s_.verify_half() for s_ in sets])
        off_, par_ = w.node_offsets.tolist(), w.parent.tolist()
        plen_total = sum(wl.tree_depths(par_[off_[b]:off_[b + 1]])[int(w.accepted[b])] + 1
                         for b in range(w.B) if int(w.accepted[b]) >= 0)   # path rows commit reads, per head
        hbytes = pb.total - 2 * w.T * w.H_v * 128 - 2 * plen_total * w.H_v * 128   # U: 2 bytes instead of 4
        half_u = {"what": "prepare + treewy_verify_half_u + treewy_commit_half_u per step: U stored as fp16",
                  "ms_per_step": st["median"], "value": size * units / (st["median"] * 1e-3), "unit": UNIT,
                  "algorithmic_bytes": hbytes, "roof_ms": hbytes / (hbm * 1e9) * 1e3,
                  "frac": hbytes / (hbm * 1e9) * 1e3 / st["median"], "gpu_launches_per_step": n_launches(w)}
        assert not any(int(s_.status.max()) for s_ in sets), "a sequence was flagged"

    # the scheme the method replaces, measured on the same inputs: every node's state written out
    storeall = None
    snap_bytes = w.T * w.H_v * 128 * 128 * w.S0.element_size()
    if w.io_dtype == torch.bfloat16 and w.max_nodes <= 64 and snap_bytes < 40e9 and not args.no_snapshot_compare:
        Snap = torch.empty((w.T, w.H_v, 128, 128), dtype=w.io_dtype, device=dev)
        s0 = sets[0]
        for _ in range(2):
            tw.treewy_snapshot_all(s0.S0, s0.U, s0.k, s0.tree, w.H_qk, Snap, s0.status)
        torch.cuda.synchronize(dev)
        e0.record(stream)
        for _ in range(3):
            tw.treewy_snapshot_all(s0.S0, s0.U, s0.k, s0.tree, w.H_qk, Snap, s0.status)
        e1.record(stream)
        torch.cuda.synchronize(dev)
        snap_ms = e0.elapsed_time(e1) / 3
        del Snap
        storeall = {"what": "treewy_snapshot_all: one state per draft node instead of one per sequence",
                    "ms": snap_ms, "bytes_written": snap_bytes, "commit_ms": kt[2],
                    "time_over_commit": snap_ms / kt[2],
                    "state_bytes_over_commit": snap_bytes / (w.B * w.H_v * 128 * 128 * w.S0.element_size())}

    set_bytes = sum(t.numel() * t.element_size()
                    for t in (sets[0].S0, sets[0].q, sets[0].k, sets[0].v, sets[0].O, sets[0].U))
    if set_bytes > 126e6:
        l2_note = (f"inputs larger than L2: two layer sets ({set_bytes / 1e9:.2f} GB each) rotated, commit "
                   "runs one step after its verify")
    else:
        l2_note = (f"two layer sets ({set_bytes / 1e6:.0f} MB each, {2 * set_bytes / 1e6:.0f} MB together against a "
                   "126 MB L2) rotated, commit runs one step after its verify: this small configuration is "
                   "partly L2-resident and is not the headline workload")
    host_us = host_cost_per_call(sets[0], dev)
    del sets
    torch.cuda.empty_cache()

    # the other benchmark workloads, same step and timing code (no end-to-end or CPU leg)
    others = {}
    if not args.no_other_workloads and args.batch is None:
        for cid in OTHER_WORKLOADS:
            if cid == args.config:
                continue
            wo = wl.make_workload(cid, prefix_device=str(dev))
            rec, osets, _, _ = measure_workload(wo, dev, stream, args.steps, args.warmup)
            rec["value"] = size * wo.T * wo.H_v / (rec["ms_per_step"] * 1e-3)
            if wo.io_dtype == torch.bfloat16 and wo.max_nodes <= 32:   # the fused round on this workload too
                fstep = lambda i, s_=osets: (s_[i % 2].prepare(), s_[i % 2].commit_verify())
                for i in range(max(args.warmup, 3)):
                    fstep(i)
                torch.cuda.synchronize(dev)
                fb, _ = timed_blocks(fstep, args.steps, dev, stream, start=max(args.warmup, 3), min_total_ms=20.0)
                rec["fused_commit_verify_ms_per_step"] = block_stats(fb, args.steps, dev)["median"]
            rec["config"] = {"B": wo.B, "H_v": wo.H_v, "H_qk": wo.H_qk, "T": wo.T, "max_nodes": wo.max_nodes}
            rec["host_us_per_call"] = host_cost_per_call(osets[0], dev)
            others[wo.name] = rec
            del osets, wo
            torch.cuda.empty_cache()

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": size, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.io_dtype == torch.bfloat16 else "f32",
        "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H_v": w.H_v, "H_qk": w.H_qk, "T": w.T,
                   "max_nodes": w.max_nodes, "seed": w.seed,
                   "l2": l2_note,
                   "timing": f"median of {main['blocks']} back-to-back blocks of {args.steps} steps "
                             "(CUDA events on the launching stream, MAX over ranks)",
                   "parallelism": f"replicas x{size}, no collective"},
        "ms_per_step_min": main["ms_per_step_min"], "ms_per_step_max": main["ms_per_step_max"],
        "blocks": main["blocks"], "ms_per_step_blocks": main["ms_per_step_blocks"],
        "clocks": clocks.summary(), "e2e": e2e,
        "gpu_launches": n_launches(w) * args.steps * main["blocks"],   # inside the timed region
        "roofline": roofline,
        "step_roofline": main["step_roofline"],
        "kernel_ms": main["kernel_ms"], "kernel_ms_back_to_back": main["kernel_ms_back_to_back"],
        "kernel_gbs": main["kernel_gbs"],
        "host_us_per_call": host_us,
        "graph_replay_ms_per_step": main["graph_replay_ms_per_step"],
        "footprint": footprint.footprint_report(w.max_nodes, w.H_v, w.H_qk),
        "snapshot_comparator": storeall,
        "fused_commit_verify": fused, "half_u": half_u,
        "workloads": others,
    }
    if rank == 0 and size == 1 and not args.no_cpu_baseline:
        v, dt, passes, sub, cores = time_oracle(w, args.cpu_seqs)
        out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                               "seconds": dt,
                               "sample": f"first {sub.B} of {w.B} sequences, all heads, {passes} passes"}
    if rank == 0:
        print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=2, help="workload id (2 = the metric's)")
    ap.add_argument("--batch", type=int, default=None,
                    help="override the workload's batch size (profiling captures on a small case)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-seqs", type=int, default=256, help="sequences the CPU baseline times")
    ap.add_argument("--ref-seqs", type=int, default=16, help="sequences per reference-arm step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-snapshot-compare", action="store_true")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="time the selected workload only (profiling captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank, size, local = replicas.world()
    if args.impl == "reference":
        run_reference(args, rank)
        return
    rank, size, local = replicas.init()
    try:
        run_ours(args, rank, size, local)
    finally:
        replicas.shutdown()


if __name__ == "__main__":
    main()
