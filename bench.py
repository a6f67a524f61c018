#!/usr/bin/env python
"""Benchmark of the SharpV pruning hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl sharpv|reference]

One "step" is one pass of the whole path over one batch of synthetic video tokens:
score frames -> per-frame top-k + gather -> calibration -> K/V compaction.  Prints one JSON
line (rank 0).  With N > 1 every rank runs the same-shaped batch on its own GPU (videos are
independent: no data-path collective, weak scaling) and the time is the max over ranks.
`--impl reference` times the CPU oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2511_08003_b200 import workloads as W  # noqa: E402

METRIC = "pruning throughput (visual tokens/s)"
UNIT = "visual tokens/s"
FALLBACK_HBM_GBS = 6650.0
# kernels launched per step by each entry point (score, select, calibrate, compact)
LAUNCHES_PER_STEP = {"score": 2, "select": 2, "calibrate": 2, "compact": 1}
# DRAM bytes per launch of the dominant kernel from an ncu capture (profiles/); None = not captured
NCU_TRAFFIC_BYTES = {("onevision_7b", "compact"): 266_712_320}   # profiles/kv_compact_kernel_onevision_7b.md


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="onevision_7b", choices=list(W.PRESETS))
    ap.add_argument("--impl", default="sharpv", choices=["sharpv", "reference"])
    ap.add_argument("--M", type=float, default=0.788,
                    help="degradation threshold; 0.788 keeps about 39 %% of the synthetic visual tokens "
                         "(the paper's reported memory ratio); the paper's default 0.2 keeps all of them")
    ap.add_argument("--w", type=float, default=1.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--stage", default=None, choices=["score", "select", "calibrate", "compact"],
                    help="profiling aid: after the warm-up run only this entry point --steps times "
                         "(L2 flushed before each) and print its mean duration")
    ap.add_argument("--inplace", action="store_true",
                    help="compact the K/V cache in place (kv_dst == kv_src) instead of into a second cache")
    ap.add_argument("--rope", action="store_true",
                    help="compact with rotary re-encoding of the keys (rotary_dim = head_dim, base 1e6)")
    ap.add_argument("--layers", type=int, default=None,
                    help="override the number of K/V layers (profiling aid: smaller device footprint)")
    ap.add_argument("--frames", type=int, default=None,
                    help="override the frame count of a single-video workload (profiling aid)")
    return ap.parse_args()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(wl, n_keep_tokens, t_keep, stage):
    e = wl.elem_bytes
    if stage == "score":
        return wl.n_visual * wl.d * e + wl.n_visual * 4 + wl.total_frames * 8
    if stage == "select":
        return wl.n_visual * 4 + wl.total_frames * 4 + 2 * n_keep_tokens * wl.d * e + n_keep_tokens * 4
    if stage == "calibrate":
        return 2 * wl.n_visual * wl.d * e + wl.n_visual * 4 + t_keep * 4
    if stage == "compact":
        planes = wl.num_layers * 2 * wl.num_kv_heads
        return 2 * planes * t_keep * wl.head_dim * e + t_keep * 4
    raise KeyError(stage)


# ------------------------------------------------------------------------------------- oracle
def oracle_step(wl, orc, M, w, nthreads, kv_layers=None):
    """One full pass of the path in the oracle.  kv_layers limits the compaction to a prefix of
    the layers (bounded sample); returns (seconds per stage, kept counts)."""
    t = {}
    t0 = time.perf_counter()
    s = orc.score_frames(wl.tokens, wl.video_frame_offsets, wl.f, w=w, nthreads=nthreads)
    t["score"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    idx, _ = orc.select_tokens(s["importance"], s["k"], wl.f)
    orc.gather_rows(wl.tokens, idx)
    t["select"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    c = orc.kv_calibrate_prune(wl.hidden, wl.tokens, wl.seq_offsets, wl.vis_begin, wl.vis_count, wl.vis_offsets,
                               M, nthreads=nthreads)
    t["calibrate"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    if wl.kv is not None:
        L = wl.num_layers if kv_layers is None else kv_layers
        orc.kv_compact(wl.kv, c["kept_pos"], layer_begin=0, layer_end=L, dst=wl._kv_dst, nthreads=nthreads)
        t["compact"] = (time.perf_counter() - t0) * (wl.num_layers / L)
    return t, idx.size, c["kept_pos"].size


def host_workload(name, with_kv_layers=None, frames=None, layers=None):
    kw = {}
    if frames:
        kw["n_frames"] = frames
    if layers:
        kw["num_layers"] = layers
    wl = W.PRESETS[name](**kw)
    W.fill_tokens(wl)
    W.fill_hidden(wl)
    if with_kv_layers:
        # K/V values never influence a decision: the oracle's compaction is timed on the first
        # `with_kv_layers` layers of an all-layer-shaped cache and scaled to all layers
        full = wl.num_layers
        wl.num_layers = with_kv_layers
        W.fill_kv(wl)
        wl.num_layers = full
        wl._kv_dst = np.zeros_like(wl.kv)
    return wl


def run_reference(args):
    from oracle import sharpv_oracle as orc
    cores = os.cpu_count() or 1
    kv_layers = 4
    wl = host_workload(args.workload, with_kv_layers=kv_layers)
    for _ in range(min(args.warmup, 1)):
        oracle_step(wl, orc, args.M, args.w, cores, kv_layers)
    t0 = time.perf_counter()
    scaled = 0.0
    for _ in range(args.steps):
        t, n_keep, t_keep = oracle_step(wl, orc, args.M, args.w, cores, kv_layers)
        scaled += sum(t.values())
    wall = time.perf_counter() - t0
    ms = scaled / args.steps * 1e3
    value = wl.n_visual / (ms * 1e-3)
    sample = (f"every step: full score, select+gather and calibration of the workload; K/V compaction timed on "
              f"{kv_layers} of {wl.num_layers} layers and scaled; {cores} OpenMP threads; wall {wall:.1f} s")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "M": args.M, "w": args.w},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU from a thread while the timed region runs
    (NVML, read-only queries)."""

    REASONS = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40}

    def __init__(self, index, period_s=0.005, pci_bus_id=None):
        import threading
        self.samples, self.reason_bits, self.max_mhz = [], 0, None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nvml = pynvml
            try:
                self._h = pynvml.nvmlDeviceGetHandleByPciBusId(pci_bus_id.encode()) if pci_bus_id else None
            except Exception:
                self._h = None
            if self._h is None:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nvml = None
            return
        self._period = period_s
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def _run(self):
        nv = self._nvml
        while not self._stop.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
            except Exception:
                pass
            self._stop.wait(self._period)

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": []}
        if self._thread is None:
            return out
        self._stop.set()
        self._thread.join(timeout=2)
        if self.samples:
            out["sm_mhz"] = statistics.median(self.samples)
            out["samples"] = len(self.samples)
        out["reasons"] = sorted(n for n, bit in self.REASONS.items() if self.reason_bits & bit)
        return out


# ------------------------------------------------------------------------------------- ranks
def max_over_ranks(ms, device, world):
    """Slowest rank's time: the job is as fast as its slowest replica."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank, world, ms_per_step):
    """Every rank processes its own batch of the same size (weak scaling): units of all ranks per second."""
    return world * units_per_rank / (ms_per_step * 1e-3)


# ------------------------------------------------------------------------------------- GPU arm
def run_sharpv(args):
    import torch
    import torch.distributed as dist

    from paper_2511_08003_b200 import binding as sv

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    sv.lib()                                            # fail loudly before any work if not built

    wl = host_workload(args.workload, frames=args.frames, layers=args.layers)
    F, f, d, T, NV = wl.total_frames, wl.f, wl.d, wl.total_seq_tokens, wl.n_visual
    tdt = torch.float32 if wl.dtype == W.F32 else torch.bfloat16

    def dev_tokens(a):
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)
        return torch.from_numpy(a).to(dev)

    def pinned(a):
        t = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()
        return t.view(torch.bfloat16) if a.dtype == np.uint16 else t

    # Rotating copies of the token and hidden-state matrices: consecutive launches of one kernel
    # read different copies, and a copy is only read again after more than twice the L2 capacity of
    # other data has gone through the cache, so every timed launch starts from HBM.
    L2_BYTES = 126 << 20
    in_bytes = wl.tokens.nbytes
    ncopies = max(1, -(-2 * L2_BYTES // in_bytes) + 1) if in_bytes < 2 * L2_BYTES else 1
    tok_copies = [dev_tokens(wl.tokens) for _ in range(ncopies)]
    hid_copies = [dev_tokens(wl.hidden) for _ in range(ncopies)]
    tokens, hidden = tok_copies[0], hid_copies[0]
    tabs = {k: torch.from_numpy(getattr(wl, k)).to(dev) for k in
            ("video_frame_offsets", "seq_offsets", "vis_begin", "vis_count", "vis_offsets")}
    gen = torch.Generator(device=dev)
    gen.manual_seed(wl.seed * 1000 + 3)
    kv = torch.empty(wl.kv_shape(), dtype=tdt, device=dev)
    for l in range(wl.num_layers):                      # N(0,1) K/V, drawn on the device layer by layer
        kv[l] = torch.randn(wl.kv_shape()[1:], dtype=torch.float32, device=dev, generator=gen).to(tdt)
    kv_dst = torch.zeros_like(kv)

    # preallocated outputs and workspaces: nothing is allocated inside a step
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    o_score = {"importance": torch.empty(NV, dtype=torch.float32, device=dev),
               "ratio": torch.empty(F, dtype=torch.float32, device=dev),
               "k": torch.empty(F, dtype=torch.int32, device=dev)}
    ws_score = torch.empty(sv.sharpv_score_frames_workspace_bytes(F, f, d), dtype=torch.uint8, device=dev)
    o_sel = {"kept_index": torch.empty(NV, dtype=torch.int32, device=dev),
             "kept_offsets": torch.empty(F + 1, dtype=torch.int32, device=dev),
             "num_kept": torch.empty(1, dtype=torch.int32, device=dev),
             "tokens": torch.empty((NV, d), dtype=tdt, device=dev)}
    ws_sel = torch.empty(sv.sharpv_select_tokens_workspace_bytes(F, f), dtype=torch.uint8, device=dev)
    o_cal = {"cos": torch.empty(NV, dtype=torch.float32, device=dev),
             "kept_pos": torch.empty(T, dtype=torch.int32, device=dev),
             "kept_seq_offsets": torch.empty(wl.num_videos + 1, dtype=torch.int32, device=dev)}
    ws_cal = torch.empty(sv.sharpv_kv_calibrate_prune_workspace_bytes(T, wl.num_videos), dtype=torch.uint8,
                         device=dev)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)      # > 2x the 126 MB L2
    stream = torch.cuda.current_stream()

    def stage_score(i=0):
        sv.sharpv_score_frames(tok_copies[i % ncopies], tabs["video_frame_offsets"], F, f, w=args.w, out=o_score,
                               workspace=ws_score, status_word=status)

    def stage_select(i=0):
        sv.sharpv_select_tokens(o_score["importance"], o_score["k"], F, f, tokens=tok_copies[i % ncopies],
                                capacity=NV, out=o_sel, workspace=ws_sel, status_word=status)

    def stage_calibrate(i=0):
        sv.sharpv_kv_calibrate_prune(hid_copies[i % ncopies], tok_copies[i % ncopies], tabs["seq_offsets"],
                                     tabs["vis_begin"], tabs["vis_count"], tabs["vis_offsets"], T, M=args.M,
                                     capacity=T, out=o_cal, workspace=ws_cal, status_word=status)

    ws_rope = (torch.empty(sv.sharpv_kv_compact_rope_workspace_bytes(T, wl.head_dim), dtype=torch.uint8, device=dev)
               if args.rope else None)

    def stage_compact(i=0):
        if args.rope:
            sv.sharpv_kv_compact_rope(kv, kv_dst, o_cal["kept_pos"], o_cal["kept_seq_offsets"], tabs["seq_offsets"],
                                      T, wl.head_dim, 1.0e6, workspace=ws_rope, status_word=status)
            return
        sv.sharpv_kv_compact(kv, kv if args.inplace else kv_dst, o_cal["kept_pos"], o_cal["kept_seq_offsets"],
                             capacity=T, status_word=status)

    stages = [("score", stage_score), ("select", stage_select), ("calibrate", stage_calibrate),
              ("compact", stage_compact)]

    def step():
        for _, fn in stages:
            fn()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed_launches(fn, n):
        """n back-to-back launches between one pair of events (an event pair around a single launch
        costs several microseconds on its own); returns the mean milliseconds per launch.  The n
        launches (each with its own rotating input copy) are captured into one CUDA graph first, so
        that the time of the Python caller between two launches is not in the measurement."""
        g = torch.cuda.CUDAGraph()
        cs = torch.cuda.Stream()
        cs.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(cs):
            with torch.cuda.graph(g, stream=cs):
                for i in range(n):
                    fn(i)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        flush.zero_()
        a.record(stream)
        g.replay()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n

    W_ = max(args.warmup, 3)
    for _ in range(W_):
        flush.zero_()
        step()
    torch.cuda.synchronize()
    n_keep = int(o_sel["num_kept"].item())
    t_keep = int(o_cal["kept_seq_offsets"][-1].item())
    assert int(status.item()) == 0, "device status word set"

    if args.stage:
        fn = dict(stages)[args.stage]
        ms = timed_launches(fn, args.steps)
        nbytes = algorithmic_bytes(wl, n_keep, t_keep, args.stage)
        print(json.dumps({"stage": args.stage, "workload": args.workload, "frames": F, "ms": ms,
                          "algorithmic_bytes": nbytes, "GBps": nbytes / (ms * 1e-3) / 1e9,
                          "kept_stage_one": n_keep, "kept_stage_two": t_keep, "input_copies": ncopies}))
        return

    # The library calls only enqueue kernels (no allocation, no sync), so one step is captured
    # into a CUDA graph and replayed: the GPU never waits for the Python caller.
    graph = torch.cuda.CUDAGraph()
    cap_stream = torch.cuda.Stream()
    cap_stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(cap_stream):
        with torch.cuda.graph(graph, stream=cap_stream):
            step()
    torch.cuda.synchronize()
    for _ in range(W_):
        graph.replay()
    torch.cuda.synchronize()

    # ---- timed region: K graph replays back to back between one pair of events.  A step reads and
    # writes several times the L2 capacity, so each step finds its inputs in HBM, not in cache.
    try:
        pr = torch.cuda.get_device_properties(dev)
        bus = f"{pr.pci_domain_id:08x}:{pr.pci_bus_id:02x}:{pr.pci_device_id:02x}.0"
    except Exception:
        bus = None
    sampler = ClockSampler(local_rank, pci_bus_id=bus) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    flush.zero_()
    barrier()
    wall0 = time.perf_counter()
    e0.record(stream)
    for _ in range(args.steps):
        graph.replay()
    e1.record(stream)
    barrier()
    wall = time.perf_counter() - wall0
    total_ms = e0.elapsed_time(e1)

    # ---- per-entry-point launch durations from HBM-cold inputs, in the same region of the run
    stage_n = max(10, min(args.steps, 100))
    stage_ms = {name: timed_launches(fn, stage_n) for name, fn in stages}

    # ---- secondary number: stage two chained behind stage one (it sees only the tokens stage one kept).
    # The survivors' features, hidden rows and K/V rows are laid out once with torch indexing (set-up,
    # not timed); calibration and compaction then run on that smaller sequence set.
    chained = None
    if world == 1 and wl.num_videos == 1 and n_keep > 0:
        idx = o_sel["kept_index"][:n_keep].long()
        pos = torch.cat([idx, torch.arange(NV, T, device=dev)])            # survivors, then the text tokens
        c_vis = tokens.index_select(0, idx).contiguous()
        c_hid = hidden.index_select(0, pos).contiguous()
        c_kv = kv.index_select(3, pos).contiguous()
        c_dst = torch.zeros_like(c_kv)
        Tc = int(pos.numel())
        i32 = lambda v: torch.tensor(v, dtype=torch.int32, device=dev)
        c_tabs = (i32([0, Tc]), i32([0]), i32([n_keep]), i32([0]))
        c_out = {"cos": torch.empty(n_keep, dtype=torch.float32, device=dev),
                 "kept_pos": torch.empty(Tc, dtype=torch.int32, device=dev),
                 "kept_seq_offsets": torch.empty(2, dtype=torch.int32, device=dev)}
        c_ws = torch.empty(sv.sharpv_kv_calibrate_prune_workspace_bytes(Tc, 1), dtype=torch.uint8, device=dev)

        def chained_stage_two(i=0):
            sv.sharpv_kv_calibrate_prune(c_hid, c_vis, *c_tabs, Tc, M=args.M, capacity=Tc, out=c_out,
                                         workspace=c_ws, status_word=status)
            sv.sharpv_kv_compact(c_kv, c_dst, c_out["kept_pos"], c_out["kept_seq_offsets"], capacity=Tc,
                                 status_word=status)

        chained_stage_two()
        torch.cuda.synchronize()
        c_ms = timed_launches(chained_stage_two, stage_n)
        c_keep = int(c_out["kept_seq_offsets"][-1].item())
        chained = {"seq_tokens": Tc, "kept_stage_two": c_keep, "stage_two_ms": round(c_ms, 5),
                   "token_budget": round((c_keep - (T - NV)) / NV, 4),
                   "note": "calibration + compaction on the survivors of stage one; token_budget = visual "
                           "tokens left after both stages / visual tokens in"}
        del c_kv, c_dst
    clocks = sampler.stop() if sampler else None

    total_ms = max_over_ranks(total_ms, dev, world)
    ms_per_step = total_ms / args.steps
    value = whole_job_throughput(NV, world, ms_per_step)

    # ---- end to end: inputs start in pinned host memory, results are read back every step
    h_tokens, h_hidden = pinned(wl.tokens), pinned(wl.hidden)
    h_idx = torch.empty(NV, dtype=torch.int32).pin_memory()
    h_pos = torch.empty(T, dtype=torch.int32).pin_memory()
    h_cnt = torch.empty(F + 1, dtype=torch.int32).pin_memory()
    h_kso = torch.empty(wl.num_videos + 1, dtype=torch.int32).pin_memory()

    def e2e_step():
        tokens.copy_(h_tokens, non_blocking=True)
        hidden.copy_(h_hidden, non_blocking=True)
        step()
        h_idx.copy_(o_sel["kept_index"], non_blocking=True)
        h_cnt.copy_(o_sel["kept_offsets"], non_blocking=True)
        h_pos.copy_(o_cal["kept_pos"], non_blocking=True)
        h_kso.copy_(o_cal["kept_seq_offsets"], non_blocking=True)
        torch.cuda.synchronize()

    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    e2e_ms = max_over_ranks(e2e_ms, dev, world)
    h2d = h_tokens.numel() * h_tokens.element_size() + h_hidden.numel() * h_hidden.element_size()
    d2h = (h_idx.numel() + h_pos.numel() + h_cnt.numel() + h_kso.numel()) * 4

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    kernels = {}
    for name, _ in stages:
        b = algorithmic_bytes(wl, n_keep, t_keep, name)
        gbs = b / (stage_ms[name] * 1e-3) / 1e9
        kernels[name] = {"ms": round(stage_ms[name], 5), "algorithmic_bytes": b, "GBps": round(gbs, 1),
                         "frac": round(gbs / peak, 4), "launches": LAUNCHES_PER_STEP[name]}
    dom = max(stage_ms, key=stage_ms.get)
    roofline = {"bound": "hbm", "kernel": dom, "achieved": kernels[dom]["GBps"], "peak": peak, "unit": "GB/s",
                "frac": kernels[dom]["frac"], "peak_source": f"of {peak_kind}",
                "traffic": NCU_TRAFFIC_BYTES.get((args.workload, dom))}

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        from oracle import sharpv_oracle as orc
        cores = os.cpu_count() or 1
        kv_layers = 2
        hw = host_workload(args.workload, with_kv_layers=kv_layers)
        best = None
        t0 = time.perf_counter()
        reps = 0
        while reps < 3 and time.perf_counter() - t0 < 25:
            t, _, _ = oracle_step(hw, orc, args.M, args.w, cores, kv_layers)
            tot = sum(t.values())
            best = tot if best is None else min(best, tot)
            reps += 1
        cpu = {"value": NV / best, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"best of {reps} full passes of the same workload (K/V compaction timed on {kv_layers} of "
                         f"{wl.num_layers} layers and scaled), {cores} OpenMP threads"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": W_, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "frames": F, "tokens_per_frame": f, "d": d, "storage": wl.dtype,
                   "visual_tokens": NV, "seq_tokens": T, "kv": list(wl.kv_shape()), "M": args.M, "w": args.w,
                   "kept_stage_one": n_keep, "kept_stage_two": t_keep, "kv_in_place": bool(args.inplace), "kv_rope": bool(args.rope),
                   "launch": "one CUDA graph replay per step, steps back to back",
                   "l2": "inputs larger than L2: a step streams several times the 126 MB L2 (K/V alone is "
                         "larger), and the per-kernel timings rotate through input copies totalling more than "
                         "twice the L2"},
        "kv_compaction_GBps": kernels["compact"]["GBps"], "chained": chained,
        "roofline": roofline, "kernels": kernels,
        "cpu_baseline": cpu,
        "e2e": {"value": whole_job_throughput(NV, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "note": "tokens and hidden state copied from pinned host memory every step, kept-index lists "
                        "read back; the K/V cache is device-resident model state"},
        "gpu_launches": sum(LAUNCHES_PER_STEP.values()) * args.steps,
        "clocks": clocks, "wall_s": round(wall, 3),
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) == 0:
            run_reference(args)
        return
    run_sharpv(args)


if __name__ == "__main__":
    main()
