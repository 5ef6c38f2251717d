#!/usr/bin/env python
"""Benchmark of the batched token sampler: rows sampled per second and the fraction of
the HBM roofline on the metric workload (B=256 rows, V=152064, bf16, top-k + top-p).

A "step" is one pass of the whole sampling path over one batch: one `albireo_sample`
call (penalties -> temperature -> top-k -> min-p/top-p -> softmax/logprob -> race).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference] [--all-configs]

The K timed launches are one CUDA graph, replayed until the timed region lasts at least 50 ms (so
that the clock samples fall inside it); `ms_per_step` is the region divided by all its launches.
The line also carries the spread of isolated cold-L2 calls, the duration of the stream alone in the
same harness (`roofline.read_ceiling_us`), and one compact record per configuration (`per_config`).
Calls are launched with programmatic stream serialisation by default (each kernel waits for the one
ahead of it before it touches memory; only its set-up overlaps that kernel's tail); the figure for
plain launches is in the same line (`roofline.plain_launch_us`), `--no-pdl` makes it the headline.
With --gpus N > 1 and no WORLD_SIZE in the environment the N ranks are started here.

N > 1 (launched by torch.distributed.run, one rank per GPU): rows are independent
(section 6.1 of the paper), so every rank samples its own B rows with global row ids
`rank * B + b` and there is no data-path collective ("weak" scaling).

`--impl reference` times the CPU oracle instead (rank 0 only), each step a bounded
sample of the same workload.
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

METRIC = "rows_sampled_per_s"
UNIT = "rows/s"
N_ROTATING = 8            # distinct logits buffers, so that no call finds its rows in L2
FALLBACK_HBM_GBS = 6650.0



def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy read+write)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.samples = []
        self.stop = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception as e:   # NVML missing: report that, do not guess
            self.err = repr(e)
        self.thread = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        nv = self.nv
        while not self.stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                    else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.samples.append((time.perf_counter(), mhz, int(reasons)))
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.ok:
            self.thread.start()

    def finish(self, t0: float, t1: float):
        if not self.ok:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvml unavailable"]}
        self.stop.set()
        self.thread.join(timeout=2)
        nv = self.nv
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        used = inside if len(inside) >= 3 else self.samples
        names = {
            "gpu_idle": 0x1, "applications_clocks_setting": 0x2, "sw_power_cap": 0x4, "hw_slowdown": 0x8,
            "sync_boost": 0x10, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
            "hw_power_brake_slowdown": 0x80, "display_clock_setting": 0x100,
        }
        bits = 0
        for s in used:
            bits |= s[2]
        reasons = sorted(n for n, m in names.items() if bits & m and n != "gpu_idle")
        return {"sm_mhz": statistics.median(s[1] for s in used) if used else None,
                "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples_in_timed_region": len(inside), "samples_total": len(self.samples)}


def describe(w) -> str:
    def one(a, fmt):
        if a is None:
            return "off"
        return fmt % a[0] if np.all(a == a[0]) else "per-row"
    return (f"{w.name}: B={w.B} V={w.V} {'bf16' if w.dtype == 1 else 'f32'} T={one(w.temperature, '%.2g')} "
            f"top_k={one(w.top_k, '%d')} top_p={one(w.top_p, '%.2g')} min_p={one(w.min_p, '%.2g')} "
            f"history={'none' if w.history_ids is None else str(int(w.history_ids.size)) + ' ids'}")


def algorithmic_bytes(w) -> int:
    """Bytes one launch must move: every logit once, the history CSR, per-row scalars, outputs."""
    n_param_arrays = sum(a is not None for a in (w.temperature, w.top_k, w.top_p, w.min_p, w.repetition_penalty,
                                                 w.presence_penalty, w.frequency_penalty))
    return w.logit_bytes + w.history_bytes + w.B * (4 * n_param_arrays + 8 + 8)


def run_reference(args, w):
    """The CPU oracle as it stands, on the host cores, on a bounded sample of the workload."""
    from oracle import albireo_oracle as O
    cores = len(os.sched_getaffinity(0))
    rows = min(w.B, max(cores, args.ref_rows))
    sub = w.rows(0, rows)
    for _ in range(min(args.warmup, 1)):
        O.sample(sub, threads=cores)
    times = []
    for _ in range(args.steps):
        t0 = time.perf_counter()
        O.sample(sub, threads=cores)
        times.append(time.perf_counter() - t0)
    per_step = sum(times) / len(times)
    value = rows / per_step
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": min(args.warmup, 1), "ms_per_step": per_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": describe(w), "sample": f"first {rows} rows of the batch per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"first {rows} of {w.B} rows per step, {args.steps} steps, one thread per core"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_sequence_parallel(args, rank, world, local_rank):
    """Secondary mode (section 6.1): the batch's logits start as vocabulary shards [s, v/t], one per
    rank; a step is all-to-all + sample local rows + gather of the tokens ("a2a"), or the gather-to-one
    arrangement it replaces ("gather").  Total work is fixed as N grows (strong scaling)."""
    import torch
    import torch.distributed as dist
    from paper_2606_01927_b200 import _build
    _build.build()
    from paper_2606_01927_b200 import binding, sequence_parallel as SP, workloads as W
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if not dist.is_initialized():
        if world == 1:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29571")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    w = W.make(args.workload)
    s_rows, V = w.B, w.V
    if V % world or (V // world * w.elem_size) % 16:
        raise SystemExit("the vocabulary does not split into 16-byte aligned shards over this many ranks")
    vs = V // world
    t_full = binding.workload_tensors(w, dev)
    full = t_full.pop("logits")
    shards = [full[:, rank * vs:(rank + 1) * vs].contiguous()]
    shards += [torch.roll(shards[0], shifts=i, dims=0).contiguous() for i in range(1, N_ROTATING)]
    del full
    lay = SP.layout(s_rows)
    htot = 0 if w.history_ids is None else int(w.history_ids.size)
    sampler = binding.Sampler(max_rows=s_rows, max_vocab=V, max_history_total=htot, device=dev)
    meta_all = {k: v for k, v in t_full.items() if k != "step"}
    meta_local = SP.scatter_metadata(meta_all if rank == 0 else None, lay, dev)
    fn = SP.cuda_sample_fn(sampler)
    recv = torch.empty((world, lay.rows, vs), dtype=shards[0].dtype, device=dev)
    peer_bufs = None
    if args.sequence_parallel == "peer":
        # every rank's shard lives in symmetric memory (one buffer per rotation); the "LM head" output is copied in once
        peer_bufs = []
        for sh in shards:
            mine, peers, handle = SP.peer_shards(lay.s_padded, vs, sh.dtype, dev)
            mine[:s_rows].copy_(sh)
            peer_bufs.append((peers, handle))
        torch.cuda.synchronize(dev)
        dist.barrier()

    def step(i):
        if args.sequence_parallel == "peer":
            peers, handle = peer_bufs[i % N_ROTATING]
            return SP.peer_sample_step(sampler, peers, handle, meta_local, lay, step=w.step)
        if args.sequence_parallel == "a2a":
            return SP.sample_step(fn, shards[i % N_ROTATING], meta_local, lay, step=w.step, recv=recv)
        return SP.gather_then_sample_step(fn, shards[i % N_ROTATING], meta_all, s_rows, step=w.step)

    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        for i in range(args.warmup):
            step(i)
    torch.cuda.synchronize(dev)
    # the K steps as one CUDA graph (collectives included): from the host they are launch-bound
    graph = None
    if not args.no_graph:
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                for i in range(args.steps):
                    step(i)
            graph.replay()
            torch.cuda.synchronize(dev)
        except Exception as exc:                    # a library that cannot be captured: time the host-launched steps
            print(f"[bench] graph capture of the sequence-parallel step failed ({exc}); launching from the host",
                  file=sys.stderr)
            graph = None
            torch.cuda.synchronize(dev)
    dist.barrier()
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        e0.record(stream)
        if graph is not None:
            graph.replay()
        else:
            for i in range(args.steps):
                step(i)
        e1.record(stream)
    torch.cuda.synchronize(dev)
    dist.barrier()
    tt = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    ms = float(tt.item()) / args.steps
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": s_rows / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": describe(w), "mode": "sequence-parallel " + args.sequence_parallel,
                       "rows_per_gpu": lay.rows,
                       "launch": "one CUDA graph of K steps (collectives + one kernel each)" if graph is not None
                       else "K steps from the host (collectives + one kernel each)"},
            "gpu_launches": args.steps}))
    dist.destroy_process_group()


def cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def ncu_traffic(name: str):
    """dram bytes (read + write) per launch from the ncu captures summarised under profiles/ (a small
    data file written beside those summaries); None for a workload without a capture."""
    try:
        with open(os.path.join(ROOT, "profiles", "ncu_traffic.json")) as f:
            return json.load(f).get(name, {}).get("dram_bytes_per_launch")
    except Exception:
        return None


def percentile(xs, q):
    xs = sorted(xs)
    if not xs:
        return None
    k = (len(xs) - 1) * q
    lo, hi = int(k), min(int(k) + 1, len(xs) - 1)
    return xs[lo] + (xs[hi] - xs[lo]) * (k - lo)


def measure(args, name, rank, world, dev, *, clocks=None, calls=200, min_region_ms=50.0, ceiling=True):
    """Times one workload on this rank: the K launches as one CUDA graph replayed until the timed region
    is at least `min_region_ms` long (CUDA events on the launching stream), then `calls` isolated calls
    with cold L2, then the stream alone in the same graph harness.  Returns a dict of raw figures."""
    import torch
    import torch.distributed as dist
    from paper_2606_01927_b200 import binding, workloads as W

    if args.no_graph:
        calls = min(calls, 20)                   # (profiler runs: few launches beside the timed ones)
    w = W.make(name)
    if args.rows and args.rows < w.B:
        w = w.rows(0, args.rows)                 # a smaller case of the same workload (profiler captures)
        w.name = name
    if args.variant == "f16":
        w = W.as_f16(w)
    elif args.variant == "exp1":
        w = W.with_exp1(w)
    elif args.variant == "feedback":
        w = W.with_backfill(w)
    w.row_base = rank * w.B                      # global row ids: draws do not depend on the sharding
    htot = 0 if w.history_ids is None else int(w.history_ids.size)
    sampler = binding.Sampler(max_rows=w.B, max_vocab=w.V, max_history_total=htot, device=dev, host_staging=True)
    t = binding.workload_tensors(w, dev)
    logits0 = t.pop("logits")
    # rotating copies (rows rolled so the copies are not byte-identical): at least 8, and enough of them
    # to be several times the 126 MB L2
    n_rot = max(N_ROTATING, -(-600_000_000 // max(1, w.logit_bytes)))
    n_rot = min(n_rot, 64)
    bufs = [logits0] + [torch.roll(logits0, shifts=i, dims=0).contiguous() for i in range(1, n_rot)]
    out_tok = torch.empty(w.B, dtype=torch.int32, device=dev)
    out_lp = torch.empty(w.B, dtype=torch.float32, device=dev)
    flags = binding.FLAG_FORCE_GENERAL if args.general_path else 0
    if args.variant == "fullvocab":
        flags |= binding.FLAG_LOGPROB_FULL_VOCAB
    if args.pdl:
        flags |= binding.FLAG_PROGRAMMATIC_LAUNCH
    stream = torch.cuda.Stream(device=dev)
    if args.variant == "feedback":
        t["backfill_ids"] = torch.zeros(w.backfill_len, dtype=torch.int32, device=dev)
        t["feedback_ring"] = torch.full((2 * w.B,), -1, dtype=torch.int64).pin_memory()

    top_kw = {}
    if w.num_top:                                  # the workload asks for top-N lists: they are part of the call
        top_kw = dict(num_top=w.num_top,
                      out_top_ids=torch.empty((w.B, w.num_top), dtype=torch.int32, device=dev),
                      out_top_logprobs=torch.empty((w.B, w.num_top), dtype=torch.float32, device=dev))

    def step(i, st, fl=None):
        sampler.albireo_sample(bufs[i % n_rot], **t, out_tokens=out_tok, out_logprobs=out_lp, stream=st,
                               row_base=w.row_base, flags=flags if fl is None else fl, **top_kw)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    steps = args.steps
    with torch.cuda.stream(stream):
        for i in range(args.warmup):
            step(i, stream)
    torch.cuda.synchronize(dev)

    graph = None
    if not args.no_graph:
        # the K launches of the timed region as one CUDA graph: the region is launch-bound otherwise
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for i in range(steps):
                step(i, stream)
        graph.replay()                              # one untimed replay (uploads the graph)
        torch.cuda.synchronize(dev)
        # how long is one replay?  (untimed probe; decides how many replays the timed region takes)
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            p0.record(stream); graph.replay(); p1.record(stream)
        torch.cuda.synchronize(dev)
        one_ms = max(p0.elapsed_time(p1), 1e-3)
        replays = max(1, int(-(-min_region_ms // one_ms)))
    else:
        replays = 1
    if world > 1:                                    # every rank the same number of replays
        rr = torch.tensor([replays], dtype=torch.int64, device=dev)
        dist.all_reduce(rr, op=dist.ReduceOp.MAX)
        replays = int(rr.item())

    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    if clocks is not None:
        clocks.start()
    n_before = sampler.launch_count()
    barrier()
    t_wall0 = time.perf_counter()
    with torch.cuda.stream(stream):
        e0.record(stream)
        for _ in range(replays):
            if graph is not None:
                graph.replay()
            else:
                for i in range(steps):
                    step(i, stream)
        e1.record(stream)
    barrier()
    t_wall1 = time.perf_counter()
    launches = steps * replays if graph is not None else sampler.launch_count() - n_before
    elapsed_ms = e0.elapsed_time(e1)
    clock_info = clocks.finish(t_wall0, t_wall1) if clocks is not None else None
    if world > 1:
        tt = torch.tensor([elapsed_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        elapsed_ms = float(tt.item())
    ms_per_step = elapsed_ms / (steps * replays)

    # isolated calls with cold L2 (the rotation sees to that), each bracketed by its own events
    iso = []
    with torch.cuda.stream(stream):
        for i in range(calls):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            step(i, stream, flags & ~binding.FLAG_PROGRAMMATIC_LAUNCH)   # (a call alone has no kernel ahead to overlap)
            b.record(stream)
            iso.append((a, b))
    torch.cuda.synchronize(dev)
    iso_us = [a.elapsed_time(b) * 1e3 for a, b in iso]

    # the stream alone, in the same harness: same buffers, same rotation, one graph of K launches
    ceiling_us = None
    if ceiling and graph is not None and args.variant == "none":
        sink = torch.zeros(w.B, dtype=torch.int32, device=dev)
        with torch.cuda.stream(stream):
            for i in range(3):
                sampler.albireo_stream_only(bufs[i % n_rot], sink, stream=stream)
        torch.cuda.synchronize(dev)
        g2 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g2, stream=stream):
            for i in range(steps):
                sampler.albireo_stream_only(bufs[i % n_rot], sink, stream=stream)
        g2.replay()
        torch.cuda.synchronize(dev)
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps2 = max(1, replays // 2)
        with torch.cuda.stream(stream):
            c0.record(stream)
            for _ in range(reps2):
                g2.replay()
            c1.record(stream)
        torch.cuda.synchronize(dev)
        ceiling_us = c0.elapsed_time(c1) * 1e3 / (steps * reps2)
        del g2

    res = dict(w=w, sampler=sampler, t=t, bufs=bufs, stream=stream, flags=flags, graph=graph is not None,
               ms_per_step=ms_per_step, replays=replays, launches=launches, elapsed_ms=elapsed_ms,
               iso_us=iso_us, ceiling_us=ceiling_us, clock_info=clock_info, n_rot=n_rot)
    return res


def measure_e2e(args, res, rank, world, dev):
    """The same metric through the host-buffer entry of the C ABI: pinned host inputs copied in, tokens
    and log-probabilities copied back, every step, inside the timed region."""
    import torch
    import torch.distributed as dist
    from paper_2606_01927_b200 import binding
    w, sampler, stream, flags = res["w"], res["sampler"], res["stream"], res["flags"]
    th = binding.workload_tensors(w, "cpu", pinned=True)
    h_logits = th.pop("logits")
    th.pop("exp1", None); th.pop("backfill_index", None)      # device-only options: the host entry runs the plain call
    h_tok = torch.empty(w.B, dtype=torch.int32, pin_memory=True)
    h_lp = torch.empty(w.B, dtype=torch.float32, pin_memory=True)
    h2d = sum(int(v.numel() * v.element_size()) for v in [h_logits] + [x for x in th.values() if torch.is_tensor(x)])
    d2h = int(h_tok.numel() * 4 + h_lp.numel() * 4)

    def e2e_step():
        sampler.albireo_sample_host(h_logits, **th, out_tokens=h_tok, out_logprobs=h_lp, stream=stream,
                                    row_base=w.row_base, flags=flags)
    for _ in range(3):
        e2e_step()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize(dev)
    t0 = time.perf_counter()
    for _ in range(args.e2e_steps):
        e2e_step()
    torch.cuda.synchronize(dev)
    e2e_s = (time.perf_counter() - t0) / args.e2e_steps
    if world > 1:
        tt = torch.tensor([e2e_s], dtype=torch.float64, device=dev)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        e2e_s = float(tt.item())
    return {"value": world * w.B / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "ms_per_step": e2e_s * 1e3, "steps": args.e2e_steps}


def cpu_baseline(w):
    """The oracle as it stands on the machine's cores: whole batches, one thread per core, until ~15 s of CPU
    work are done; and one pass on a single thread over a bounded sample of the rows."""
    from oracle import albireo_oracle as O
    cores = len(os.sched_getaffinity(0))
    reps, cpu_s, best = 0, 0.0, float("inf")
    while reps < 2 or (cpu_s < 12.0 and reps < 32):
        t0 = time.perf_counter()
        O.sample(w, threads=cores)
        dt = time.perf_counter() - t0
        best = min(best, dt)
        cpu_s += dt * cores
        reps += 1
    n1 = min(w.B, 16)
    sub = w.rows(0, n1)
    t0 = time.perf_counter()
    O.sample(sub, threads=1)
    one = time.perf_counter() - t0
    return {"value": w.B / best, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"all {w.B} rows of the batch, {reps} passes (best of them), one thread per core, "
                      f"~{cpu_s:.0f} s of CPU work in total",
            "single_thread": {"value": n1 / one, "unit": UNIT, "sample": f"first {n1} rows, one pass, one thread"},
            "cpu_model": cpu_model()}


def roofline_of(w, res, peak, peak_src):
    alg = algorithmic_bytes(w)
    ms = res["ms_per_step"]
    achieved = alg / (ms * 1e-3) / 1e9
    iso = res["iso_us"]
    r = {
        "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
        "traffic": ncu_traffic(w.name),
        "algorithmic_bytes_per_launch": alg, "kernel": "albireo_sample_kernel",
        "launch_us_avg_timed_region": ms * 1e3,
        "cold_l2_call_us": {"calls": len(iso), "p10": percentile(iso, 0.1), "p50": percentile(iso, 0.5),
                            "p90": percentile(iso, 0.9),
                            "note": "one call between two events each: includes the events' own cost"},
        "read_ceiling_us": res["ceiling_us"],
        "peak_source": peak_src, "frac_of_8TBps_nominal": achieved / 8000.0,
    }
    if res["ceiling_us"]:
        r["frac_of_read_ceiling"] = res["ceiling_us"] / (ms * 1e3)
        r["read_ceiling_note"] = ("albireo_stream_only: the same bytes through the same ring in the same launch shape "
                                  "and graph harness, nothing else")
    return r


def spawn_ranks(n):
    """`bench.py --gpus N` run plainly: start the N ranks (one process per GPU) and pass their output through."""
    import socket
    import subprocess
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        port = so.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="albireo", choices=["albireo", "reference"])
    ap.add_argument("--workload", default="configM")
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--ref-rows", type=int, default=64, help="rows per step of the reference arm")
    ap.add_argument("--no-graph", action="store_true", help="launch each step from Python instead of one CUDA graph")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--general-path", action="store_true", help="force every row down the general path")
    ap.add_argument("--variant", default="none", choices=["none", "f16", "exp1", "feedback", "fullvocab"],
                    help="the same workload as binary16 logits, with a pre-generated Exp(1) table, or with the "
                         "early-feedback targets (next input ids + pinned host ring), or with log-probabilities "
                         "relative to the full vocabulary")
    ap.add_argument("--sequence-parallel", default=None, choices=["a2a", "gather", "peer"],
                    help="secondary mode: logits start as per-rank vocabulary shards; time all-to-all + sample + "
                         "gather (a2a), the gather-to-one-rank arrangement it replaces (gather), or the step without an "
                         "exchange: the sampler reads the peers' shards in place from symmetric memory (peer)")
    ap.add_argument("--pdl", action="store_true", default=True,
                    help="(default) launch every call with programmatic stream serialisation "
                         "(ALBIREO_FLAG_PROGRAMMATIC_LAUNCH): a call's set-up overlaps the tail of the kernel ahead of it in "
                         "the stream, as it would overlap the tail of the LM-head GEMM in a decode step; the kernel waits for "
                         "that kernel before it touches memory, results are identical")
    ap.add_argument("--no-pdl", dest="pdl", action="store_false",
                    help="plain launches; the default run reports this figure too, as roofline.plain_launch_us")
    ap.add_argument("--all-configs", action="store_true",
                    help="also time configs 1-5 and put one compact record per config into `per_config`")
    ap.add_argument("--no-per-config", action="store_true", help="(default run) leave `per_config` out")
    ap.add_argument("--rows", type=int, default=0,
                    help="take only the first ROWS rows of the workload: a small case of the same kernel for a profiler "
                         "capture; a line printed with this flag is not the metric")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        spawn_ranks(args.gpus)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    from paper_2606_01927_b200 import workloads as W

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, W.make(args.workload))
        return
    if args.sequence_parallel:
        run_sequence_parallel(args, rank, world, local_rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2606_01927_b200 import _build
    _build.build()

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the sampler has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    clocks = ClockSampler(local_rank)
    res = measure(args, args.workload, rank, world, dev, clocks=clocks)
    w = res["w"]
    e2e = measure_e2e(args, res, rank, world, dev)
    value = world * w.B / (res["ms_per_step"] * 1e-3)

    # the same region with the other launch mode (plain launches when the run uses programmatic dependent
    # launch, and the other way round), reported beside the headline
    other_us = None
    if world == 1 and not args.no_graph and not args.rows:
        import copy
        a2 = copy.copy(args); a2.pdl = not args.pdl
        res["bufs"] = None
        rp = measure(a2, args.workload, rank, world, dev, calls=0, min_region_ms=20.0, ceiling=False)
        other_us = rp["ms_per_step"] * 1e3
        del rp

    per_config = None
    if world == 1 and (args.all_configs or not args.no_per_config):
        peak, peak_src = measured_peak()
        per_config = []
        for name in ("config1", "config2", "configM", "config3", "config4", "config5"):
            if name == args.workload:
                r = res
            else:
                res["bufs"] = None                   # (one workload's buffers at a time)
                torch.cuda.empty_cache()
                r = measure(args, name, rank, world, dev, calls=50, min_region_ms=20.0, ceiling=True)
            wi = r["w"]
            alg = algorithmic_bytes(wi)
            per_config.append({
                "workload": wi.name, "B": wi.B, "V": wi.V, "us_per_call": r["ms_per_step"] * 1e3,
                "rows_per_s": wi.B / (r["ms_per_step"] * 1e-3),
                "achieved_gbs": alg / (r["ms_per_step"] * 1e-3) / 1e9,
                "frac": alg / (r["ms_per_step"] * 1e-3) / 1e9 / peak,
                "read_ceiling_us": r["ceiling_us"], "replays": r["replays"],
                "cold_l2_call_us_p50": percentile(r["iso_us"], 0.5)})
            if r is not res:
                del r
            res.setdefault("bufs", None)

    if rank == 0:
        peak, peak_src = measured_peak()
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": {W.F32: "f32", W.BF16: "bf16", W.F16: "f16"}.get(w.dtype, "f32"),
            "data": "synthetic",
            "config": {
                "workload": describe(w), "rows_per_gpu": w.B, "accum": "f32 element-wise, 2^40 fixed-point masses",
                "l2": f"{res['n_rot']} rotating logits buffers ({res['n_rot'] * w.logit_bytes / 1e6:.0f} MB per GPU) so no call finds its rows in the 126 MB L2",
                "launch": (f"one CUDA graph of K launches, replayed {res['replays']} times inside the timed region" if res["graph"] else "K launches from the host")
                          + ("; programmatic dependent launch between the calls (plain launches: roofline.plain_launch_us)" if args.pdl else "; plain launches"),
                "path": "general path forced" if args.general_path else "automatic",
                "variant": args.variant,
                "programmatic_launch": bool(args.pdl),
            },
            "replays": res["replays"], "timed_region_ms": res["elapsed_ms"],
            "tokens_per_s": value,
            "roofline": dict(roofline_of(w, res, peak, peak_src),
                             **({("plain_launch_us" if args.pdl else "programmatic_launch_us"): other_us,
                                 ("plain_launch_frac" if args.pdl else "programmatic_launch_frac"):
                                     algorithmic_bytes(w) / (other_us * 1e-6) / 1e9 / peak}
                                if other_us else {})),
            "e2e": e2e,
            "gpu_launches": res["launches"],
            "clocks": res["clock_info"],
        }
        if per_config is not None:
            line["per_config"] = per_config
        if world == 1 and not args.skip_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(w)
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
