#!/usr/bin/env python
"""Benchmark of the W4A4 bitmap-sparse SpMM (one JSON line on stdout).

Workload of the headline line: LLaMA-2-7B-shaped attention projections, W 4096x4096 INT4 at 50 %
uniform sparsity, X 4096xN INT4 with N = 8, fused fp16 dequant output. One pass = one SpMM on each
of R distinct encoded weight buffers (R * bytes > 3x the L2 size, so every launch streams its
weights from HBM); one step = as many passes as make the timed region at least half a second. The
other configurations (1024x1024; sparsity {30, 50, 70 %} x N {1, 8, 16, 32}; the 7B-shaped FFN with
row-varying density; the 13B-shaped decoder layer; the 70B-shaped FFN N sweep) are reported in the
same line under "sweep".

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-sweep]
  python bench.py --only M,K,s,N[,int32|fp16[,K_L[,N_max[,q4]]]]     one case with the kernel's stage
                                                               timers (the command of the ncu captures)

With --gpus N > 1 and no torchrun environment the script starts itself N times under
torch.distributed.run (one replica per GPU, no data-path collective).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

METRIC = "w4a4_spmm_achieved_hbm_gbs"
UNIT = "GB/s"
HEAD = dict(M=4096, K=4096, s=0.5, N=8, seed=201)
WORKLOAD = ("llama2-7b attention projection 4096x4096 INT4, 50% uniform sparsity, N=8, fused fp16 dequant; "
            "bytes counted at local tiles of 16x1024, one union-mask bit per 2x1 values")
HEAD_K_L = 1024                       # tile width the byte count of both arms refers to
CONTRACT_PEAK_GBS = 8000.0
L2_BYTES_FALLBACK = 126 * 1024 * 1024
MIN_TIMED_SECONDS = 0.5


def io_bytes(M: int, K: int, N: int, fp16: bool) -> int:
    """X, Y and (fp16 output) the two scale vectors."""
    return N * ((K + 1) // 2) + N * M * (2 if fp16 else 4) + (2 * (M + N) if fp16 else 0)


def algorithmic_bytes(stats: dict, N: int, fp16: bool) -> int:
    """What the method must move once per call: packed INT4 values of the active union-mask
    positions, union bitmaps, per-tile offsets, X, Y and (fp16 output) the two scale vectors.
    Padding of the stored payload is NOT counted: it shows up as traffic above this figure."""
    w = stats["bytes_payload"] + stats["bytes_bitmap"] + stats["bytes_offsets"]
    return w + io_bytes(stats["M"], stats["K"], N, fp16)


def bytes_q1(stats: dict, N: int, fp16: bool) -> int:
    """The same call with a per-element bitmap (one bit per weight, 16x64 local tiles): only the
    true nonzeros are stored. Closed form from the handle's own nonzero count."""
    M, K = stats["M"], stats["K"]
    mp, kp = (M + 15) // 16 * 16, (K + 63) // 64 * 64
    n_lt = (mp // 16) * (kp // 64)
    bits = stats.get("weight_bits", 4)
    return (stats["nnz"] * bits + 7) // 8 + mp * kp // 8 + 4 * (n_lt + 1) + io_bytes(M, K, N, fp16)


def bytes_dense_int4(stats: dict, N: int, fp16: bool) -> int:
    """The same call on the dense weight at its own bit width (INT4, or INT2 for the W2A4 rows): no
    bitmap, no pruning exploited."""
    M, K = stats["M"], stats["K"]
    return (M * K * stats.get("weight_bits", 4) + 7) // 8 + io_bytes(M, K, N, fp16)


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period: float = 0.02):
        super().__init__(daemon=True)
        self.period, self.samples, self.reasons, self.max_mhz = period, [], set(), None
        self._stop_evt = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.dev = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.dev, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def sample(self):
        if self.nv is None:
            return
        nv = self.nv
        try:
            self.samples.append(nv.nvmlDeviceGetClockInfo(self.dev, nv.NVML_CLOCK_SM))
            r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.dev)
            names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20,
                     "hw_thermal_slowdown": 0x40, "hw_power_brake_slowdown": 0x80,
                     "sync_boost": 0x10, "applications_clocks_setting": 0x2}
            for k, bit in names.items():
                if r & bit:
                    self.reasons.add(k)
        except Exception:
            pass

    def run(self):
        while not self._stop_evt.is_set():
            self.sample()
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def visible_device_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ------------------------------------------------------------------------------------------------
def reference_arm(args, rank: int):
    """The CPU oracle, as it stands, timed on the host cores (the reference of this build)."""
    if rank != 0:
        return
    import oracle
    from paper_2608_09291_b200 import workloads
    oracle.build()
    W = workloads.make_weight(HEAD["M"], HEAD["K"], HEAD["s"], HEAD["seed"])
    X = workloads.make_x(HEAD["K"], 32, HEAD["seed"])[: HEAD["N"]]
    s_w, s_x = workloads.make_scales(HEAD["M"], 32, HEAD["seed"])
    st = oracle.encode(W, 16, HEAD_K_L, 2, 1)["stats"]
    stats = dict(M=HEAD["M"], K=HEAD["K"], bytes_payload=st["bytes_payload"],
                 bytes_bitmap=st["bytes_bitmap"], bytes_offsets=st["bytes_offsets"])
    per_call = algorithmic_bytes(stats, HEAD["N"], True)
    calls_per_step = 2

    def step():
        for _ in range(calls_per_step):
            oracle.dequant(oracle.spmm_dense(W, X), s_w, s_x[: HEAD["N"]])

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = per_call * calls_per_step * args.steps / dt / 1e9
    sample = (f"{calls_per_step} oracle SpMMs (naive masked-dense INT32 GEMM + fp64 dequant) of the "
              f"4096x4096 s=0.5 N=8 case per step")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "flush": "n/a (CPU)"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------------------------
def max_over_ranks(seconds: float, dist, device: str) -> float:
    """Replicas only: every rank runs the same step on its own GPU with no data-path collective;
    the job's time is the slowest rank's."""
    if dist is None:
        return seconds
    import torch
    t = torch.tensor([seconds], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


class Case:
    """R replicas of one encoded weight plus device inputs; a 'pass' = one SpMM per replica."""

    def __init__(self, binding, torch, W, s_w, X, s_x, N_max, replicas, fmt=None, flags=0):
        self.torch, self.b = torch, binding
        self.sw = [binding.SparseWeight(W, s_w, fmt=fmt, max_N=N_max, flags=flags) for _ in range(replicas)]
        self.stats = self.sw[0].stats
        self.Xh = torch.from_numpy(binding.pack_int4(X)).pin_memory()
        self.Xd = self.Xh.cuda()
        self.sxd = torch.from_numpy(s_x.copy()).cuda() if s_x is not None else None
        self.M, self.K = W.shape
        self.Y16 = torch.empty((N_max, self.M), dtype=torch.float16, device="cuda")
        self.Y32 = torch.empty((N_max, self.M), dtype=torch.int32, device="cuda")

    def enqueue_pass(self, N, fp16):
        xs = self.sxd if fp16 else None
        out = self.Y16 if fp16 else self.Y32
        for sw in self.sw:
            sw.spmm(self.Xd, N, xs, out=out[:N])

    def graph(self, N, fp16):
        torch = self.torch
        g = torch.cuda.CUDAGraph()
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            self.enqueue_pass(N, fp16)          # warm-up outside capture
        torch.cuda.current_stream().wait_stream(s)
        torch.cuda.synchronize()
        with torch.cuda.graph(g):
            self.enqueue_pass(N, fp16)
        return g

    def time_passes(self, N, fp16, passes, warmup):
        """Median-free plain timing: total device time of `passes` graph replays / launches."""
        torch = self.torch
        g = self.graph(N, fp16)
        for _ in range(warmup):
            g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(passes):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        for sw in self.sw:
            sw.check()
        return e0.elapsed_time(e1) * 1e-3 / (passes * len(self.sw))   # seconds per launch

    def time_isolated(self, N, fp16, launches=40):
        """One launch at a time: events around every single call with a synchronisation in between,
        so that nothing of the next launch overlaps it (the pipelined figure of time_passes lets a
        launch's prologue run under its predecessor). Median over the launches, in seconds."""
        torch = self.torch
        xs = self.sxd if fp16 else None
        out = self.Y16 if fp16 else self.Y32
        ts = []
        for i in range(launches + 3):
            sw = self.sw[i % len(self.sw)]
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            sw.spmm(self.Xd, N, xs, out=out[:N])
            e1.record()
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(e0.elapsed_time(e1) * 1e-3)
        return float(np.median(ts))

    def close(self):
        for sw in self.sw:
            sw.close()


def replicas_for(stats, l2_bytes):
    return max(3, int(np.ceil(3.2 * l2_bytes / max(1, stats_bytes(stats)))))


def stats_bytes(stats):
    return stats["bytes_total"]


def run_ours(args, rank: int, local_rank: int, world: int):
    import torch
    from paper_2608_09291_b200 import build as libbuild
    if rank == 0:
        libbuild.build()
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    else:
        dist = None
        torch.cuda.set_device(local_rank)
    from paper_2608_09291_b200 import binding, workloads

    l2 = torch.cuda.get_device_properties(local_rank).L2_cache_size or L2_BYTES_FALLBACK
    peak_gbs, peak_kind = measured_peaks()

    # ---- headline case -----------------------------------------------------------------------
    W = workloads.make_weight(HEAD["M"], HEAD["K"], HEAD["s"], HEAD["seed"])
    Xall = workloads.make_x(HEAD["K"], 32, HEAD["seed"])
    s_w, s_x = workloads.make_scales(HEAD["M"], 32, HEAD["seed"])
    head_fmt = (16, HEAD_K_L, 2, 1)
    probe = binding.us_encode(W, s_w, head_fmt, 32, binding.US_ENCODE_HOST_ONLY)
    pstats = binding.us_get_stats(probe)
    binding.us_destroy(probe)
    R = replicas_for(pstats, l2)
    head = Case(binding, torch, W, s_w, Xall, s_x, 32, R, fmt=head_fmt)
    N = HEAD["N"]
    alg = algorithmic_bytes(head.stats, N, True)
    g = head.graph(N, True)
    # passes per step: the timed region (steps x passes x R launches) lasts at least half a second
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    t_probe = time.perf_counter()
    for _ in range(10):
        g.replay()
    torch.cuda.synchronize()
    t_pass = max(1e-6, (time.perf_counter() - t_probe) / 10)
    passes = max(1, int(np.ceil(MIN_TIMED_SECONDS / (t_pass * max(1, args.steps)))))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        for _ in range(passes):
            g.replay()
    barrier()
    sampler = ClockSampler(visible_device_index(local_rank))
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        for _ in range(passes):
            g.replay()
    e1.record()
    sampler.sample()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    barrier()
    for sw in head.sw:
        sw.check()
    dt = max_over_ranks(e0.elapsed_time(e1) * 1e-3, dist, "cuda")
    launches = args.steps * passes * R
    per_launch = dt / launches
    value = alg * launches * world / dt / 1e9
    t_iso = head.time_isolated(N, True)
    q1, dn = bytes_q1(head.stats, N, True), bytes_dense_int4(head.stats, N, True)

    # ---- end to end: host buffers, H2D of X and scales, D2H of Y inside the timed region --------
    # One step = R SpMMs, each with its own (X | activation scales) block in pinned host memory and
    # its own Y block: batched copies in, the R library calls, batched copies of all results back to
    # pinned host memory. The step is captured once as a CUDA graph -- the copies are memcpy nodes
    # that read / write the host buffers at every replay.
    x_bytes = head.Xh[:N].numel()
    sx_off = (x_bytes + 15) // 16 * 16
    blk = (sx_off + 2 * N + 255) // 256 * 256
    in_h = torch.zeros((R, blk), dtype=torch.uint8).pin_memory()
    in_h[:, :x_bytes] = head.Xh[:N].reshape(-1)
    in_h[:, sx_off:sx_off + 2 * N] = torch.from_numpy(s_x[:N].copy()).view(torch.uint8)
    in_d = torch.empty_like(in_h, device="cuda")
    Yh = torch.empty((R, N, HEAD["M"]), dtype=torch.float16).pin_memory()
    Yd = torch.empty((R, N, HEAD["M"]), dtype=torch.float16, device="cuda")

    # The R SpMMs go in four chunks: a chunk's results travel back (on a second stream) while the
    # next chunk computes, and the later chunks' inputs travel in (on a third) under the first one.
    n_chunks = min(4, R)
    bounds = [R * c // n_chunks for c in range(n_chunks + 1)]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

    def e2e_enqueue():
        main = torch.cuda.current_stream()
        s_in.wait_stream(main)
        s_out.wait_stream(main)
        arrived = []
        with torch.cuda.stream(s_in):
            for c in range(n_chunks):
                a, b = bounds[c], bounds[c + 1]
                in_d[a:b].copy_(in_h[a:b], non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(s_in)
                arrived.append(ev)
        for c in range(n_chunks):
            a, b = bounds[c], bounds[c + 1]
            main.wait_event(arrived[c])
            for r in range(a, b):
                head.sw[r].spmm(in_d[r, :x_bytes].view(N, -1), N, in_d[r, sx_off:sx_off + 2 * N].view(torch.float16),
                                out=Yd[r])
            done = torch.cuda.Event()
            done.record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(done)
                Yh[a:b].copy_(Yd[a:b], non_blocking=True)
        main.wait_stream(s_in)
        main.wait_stream(s_out)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        e2e_enqueue()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    e2e_graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(e2e_graph):
        e2e_enqueue()

    def e2e_step():
        e2e_graph.replay()
        torch.cuda.synchronize()   # the step's results are in host memory from here on

    for _ in range(3):
        e2e_step()
    ref16 = head.Y16[:N].cpu()   # every replica holds the same W and gets the same X: same Y
    if not all(torch.equal(Yh[r], ref16) for r in range(R)):
        raise RuntimeError("end-to-end result differs from the device-resident run")
    e2e_steps = max(3, min(args.steps, 50))
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    t_e2e = max_over_ranks(time.perf_counter() - t0, dist, "cuda")
    e2e_value = alg * R * e2e_steps * world / t_e2e / 1e9
    h2d = in_h.numel()
    d2h = Yh.numel() * 2

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {
            "workload": WORKLOAD,
            "step": f"{passes} passes of one SpMM on each of {R} distinct weight buffers",
            "replicas_per_pass": R, "passes_per_step": passes, "format": list(head.stats["fmt"]),
            "flush": f"inputs larger than L2: {R} x {head.stats['bytes_total']} B of weights rotate "
                     f"through a {l2} B L2",
            "launch": "CUDA graph of one step, replayed",
            "parallelism": "replicas only" if world > 1 else "1 gpu",
        },
        "us_per_spmm": per_launch * 1e6,
        "us_per_spmm_isolated": t_iso * 1e6,
        "dense_equiv_tops": 2.0 * HEAD["M"] * HEAD["K"] * N / per_launch / 1e12,
        "pct_of_8tbs": 100.0 * (alg / per_launch / 1e9) / CONTRACT_PEAK_GBS,
        "bytes_q1": q1, "pct_of_8tbs_on_q1_bytes": 100.0 * (q1 / per_launch / 1e9) / CONTRACT_PEAK_GBS,
        "bytes_dense_int4": dn, "us_dense_int4_at_8tbs": dn / CONTRACT_PEAK_GBS / 1e3,
        "clocks": clocks,
        "gpu_launches": launches,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps},
        "roofline": {"bound": "hbm", "achieved": alg / per_launch / 1e9, "peak": peak_gbs,
                     "unit": "GB/s", "frac": alg / per_launch / 1e9 / peak_gbs, "peak_kind": peak_kind,
                     "traffic": TRAFFIC_BYTES_PER_LAUNCH, "algorithmic_bytes": alg,
                     "stored_bytes": binding.us_spmm_bytes(head.sw[0].handle, N, True),
                     "kernel": kernel_label(binding, head.sw[0].handle, N) + " on 4096x4096 s=0.5 N=8 fp16"},
        "stats": {k: head.stats[k] for k in ("nnz", "sum_P", "bytes_payload", "bytes_payload_padded",
                                             "bytes_bitmap", "bytes_offsets", "pmr", "fill")},
    }
    head.close()

    if rank == 0 and not args.no_sweep:
        out["sweep"] = sweep(binding, torch, workloads, l2, peak_gbs)
        big = [r for r in out["sweep"] if r["case"] == "ffn70b_up" and r["N"] == 8]
        if big:   # the shape on which a bandwidth roofline is physically reachable
            r = big[0]
            out["roofline_large"] = {"bound": "hbm", "achieved": r["gbs"], "peak": peak_gbs, "unit": "GB/s",
                                     "frac": r["gbs"] / peak_gbs, "pct_of_8tbs": r["pct_of_8tbs"],
                                     "us": r["us"], "algorithmic_bytes": r["alg_bytes"],
                                     "traffic": TRAFFIC_BYTES_PER_LAUNCH_LARGE,
                                     "kernel": r["kernel"] + " on 28672x8192 s=0.6 N=8 int32"}
        # the same two shapes in the folded format (one mask bit per 2 x 2 weights): more bytes per launch,
        # fewer decode instructions per weight; its own byte count, time and fractions
        for key, case_name, shape in (("roofline_q4", "attn7b_q4", "4096x4096 s=0.5 N=8 fp16"),
                                      ("roofline_large_q4", "ffn70b_up_q4", "28672x8192 s=0.6 N=8 int32")):
            hit = [r for r in out["sweep"] if r["case"] == case_name and r["N"] == 8 and r["sparsity"] in (0.5, 0.6)]
            if hit:
                r = hit[0]
                out[key] = {"bound": "hbm", "achieved": r["gbs"], "peak": peak_gbs, "unit": "GB/s",
                            "frac": r["gbs"] / peak_gbs, "pct_of_8tbs": r["pct_of_8tbs"], "us": r["us"],
                            "algorithmic_bytes": r["alg_bytes"], "traffic": None, "format": r["format"],
                            "kernel": r["kernel"] + " on " + shape}
    if rank == 0:
        out["cpu_baseline"] = cpu_baseline(W, Xall[:N], s_w, s_x[:N], pstats)
        print(json.dumps(out))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def kernel_label(binding, handle, N):
    """The dominant (only) kernel of a call and its launch geometry."""
    g = binding.us_launch_info(handle, N)
    return (f"us_spmm_kernel (n-tiles {max(1, 1 << (max(N, 1) - 1).bit_length()) // 8 or 1}, {g['grid']} CTAs x "
            f"{g['block'] // 32} warps, {g['smem_bytes']} B shared memory)")


# Measured DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch, from the ncu
# captures of the same kernel build (one launch each; commands in the capture summaries).
TRAFFIC_BYTES_PER_LAUNCH = 7_969_024          # 4096x4096, s = 0.5, N = 8, fp16: 7.9690 MB read, 0 written
TRAFFIC_BYTES_PER_LAUNCH_LARGE = 101_235_968  # 28672x8192, s = 0.6, N = 8, int32: 98.02 MB read + 3.22 MB written


def sweep(binding, torch, workloads, l2, peak_gbs):
    rows = []

    def run_case(name, M, K, s, seed, Ns, outs, row_varying=False, flags=0, q4=False, w2=False):
        """q4: the folded format (16, K_L, 2, 2) -- one mask bit per 2 x 2 weights -- at the K_L the
        library picks for this shape, instead of the default (16, K_L, 2, 1)."""
        W = workloads.make_weight_w2(M, K, s, seed) if w2 else workloads.make_weight(M, K, s, seed, row_varying)
        Nmax = max(Ns)
        X = workloads.make_x(K, Nmax, seed)
        s_w, s_x = workloads.make_scales(M, Nmax, seed)
        probe = binding.us_encode(W, None, None, Nmax, binding.US_ENCODE_HOST_ONLY | flags)
        st = binding.us_get_stats(probe)
        binding.us_destroy(probe)
        fmt = None
        if q4 or w2:   # w2: INT2 weights, which live in the folded format only
            fmt = (16, st["fmt"][1], 2, 2)
            if w2:
                flags |= binding.US_ENCODE_W2
            probe = binding.us_encode(W, None, fmt, Nmax, binding.US_ENCODE_HOST_ONLY | flags)
            st = binding.us_get_stats(probe)
            binding.us_destroy(probe)
        R = replicas_for(st, l2)
        case = Case(binding, torch, W, s_w, X, s_x, Nmax, R, fmt=fmt, flags=flags)
        for fp16 in outs:
            for N in Ns:
                passes = max(3, int(2e-2 / max(1e-6, 3e-6 * R)))
                t = case.time_passes(N, fp16, passes=min(passes, 200), warmup=3)
                t_iso = case.time_isolated(N, fp16, launches=20)
                alg = algorithmic_bytes(case.stats, N, fp16)
                q1, dn = bytes_q1(case.stats, N, fp16), bytes_dense_int4(case.stats, N, fp16)
                rows.append({"case": name, "M": M, "K": K, "sparsity": s, "N": N, "out": "fp16" if fp16 else "int32",
                             "us": t * 1e6, "us_isolated": t_iso * 1e6, "alg_bytes": alg,
                             "stored_bytes": binding.us_spmm_bytes(case.sw[0].handle, N, fp16),
                             "gbs": alg / t / 1e9, "pct_of_8tbs": 100 * alg / t / 1e9 / CONTRACT_PEAK_GBS,
                             "frac_of_measured": alg / t / 1e9 / peak_gbs,
                             "bytes_q1": q1, "pct_of_8tbs_on_q1_bytes": 100 * q1 / t / 1e9 / CONTRACT_PEAK_GBS,
                             "bytes_dense_int4": dn, "us_dense_int4_at_8tbs": dn / CONTRACT_PEAK_GBS / 1e3,
                             "dense_equiv_tops": 2.0 * M * K * N / t / 1e12, "replicas": R,
                             "pmr": case.stats["pmr"], "format": list(case.stats["fmt"]),
                             "weight_bits": case.stats["weight_bits"],
                             "kernel": kernel_label(binding, case.sw[0].handle, N)})
        case.close()
        del case
        torch.cuda.empty_cache()

    SORT = binding.US_ENCODE_SORT_ROWS
    run_case("single1024", 1024, 1024, 0.5, 0, [8], [False])                                  # config 1
    for i, s in enumerate((0.3, 0.5, 0.7)):                                                    # config 2
        run_case("attn7b", 4096, 4096, s, 200 + i, [1, 8, 16, 32], [True])
    run_case("attn7b_qkv_fused", 12288, 4096, 0.5, 210, [8], [True])   # Q, K, V stacked: one launch
    run_case("ffn7b_up", 11008, 4096, 0.5, 300, [1, 8, 32], [True, False], row_varying=True, flags=SORT)     # config 3
    run_case("ffn7b_gate", 11008, 4096, 0.5, 301, [8], [True, False], row_varying=True, flags=SORT)
    run_case("ffn7b_down", 4096, 11008, 0.5, 302, [1, 8, 32], [True, False], row_varying=True, flags=SORT)
    run_case("ffn70b_up", 28672, 8192, 0.6, 500, [1, 4, 8, 16, 32, 64], [False])               # config 5
    run_case("ffn70b_down", 8192, 28672, 0.6, 501, [1, 4, 8, 16, 32, 64], [False])
    # Bitmap-aware row pairing inside each strip (the per-strip form of Alg. 1): fewer union bits.
    run_case("attn7b_paired", 4096, 4096, 0.5, 201, [8], [True], flags=binding.US_ENCODE_PAIR_ROWS)
    run_case("ffn70b_up_paired", 28672, 8192, 0.6, 500, [8], [False], flags=binding.US_ENCODE_PAIR_ROWS)
    # The paper's 2 x 2 union mask (Q = 4) in the folded kernel layout: more bytes, fewer decode
    # instructions per weight. Same matrices and seeds as the rows above.
    for i, s in enumerate((0.3, 0.5, 0.7)):
        run_case("attn7b_q4", 4096, 4096, s, 200 + i, [1, 8, 16, 32], [True], q4=True)
    run_case("ffn7b_up_q4", 11008, 4096, 0.5, 300, [8, 32], [True], row_varying=True, flags=SORT, q4=True)
    run_case("ffn7b_down_q4", 4096, 11008, 0.5, 302, [8, 32], [True], row_varying=True, flags=SORT, q4=True)
    run_case("ffn70b_up_q4", 28672, 8192, 0.6, 500, [1, 8, 16, 32, 64], [False], q4=True)
    run_case("ffn70b_down_q4", 8192, 28672, 0.6, 501, [1, 8, 16, 32, 64], [False], q4=True)
    # W2A4 (Sec. VII-B): INT2 weights, one payload byte per union-mask bit of the folded format
    run_case("attn7b_w2a4", 4096, 4096, 0.5, 201, [1, 8, 32], [True], w2=True)
    run_case("ffn70b_up_w2a4", 28672, 8192, 0.6, 500, [1, 8, 16, 32], [False], w2=True)
    run_case("ffn70b_down_w2a4", 8192, 28672, 0.6, 501, [1, 8, 16, 32], [False], w2=True)
    for s in (0.3, 0.5, 0.7):                                                                  # config 4
        rows.append(layer_chain(binding, torch, workloads, l2, s))
        rows.append(layer_chain_requant(binding, torch, workloads, l2, s))
    return rows


def layer_chain(binding, torch, workloads, l2, sparsity=0.5):
    """All seven projections of one LLaMA-2-13B-shaped decoder layer (Q, K, V, O 5120x5120; gate, up
    13824x5120; down 5120x13824) at the given sparsity, N = 16, fp16 output, back to back on one stream
    (one CUDA graph; consecutive launches overlap through programmatic dependent launch). Several
    copies of the layer rotate so that the weights come from HBM."""
    shapes = [(5120, 5120)] * 4 + [(13824, 5120)] * 2 + [(5120, 13824)]
    N = 16
    mats = []
    for i, (m, k) in enumerate(shapes):
        W = workloads.make_weight(m, k, sparsity, 410 + i)
        s_w, _ = workloads.make_scales(m, N, 410 + i)
        mats.append((W, s_w))
    layer_bytes = 0
    copies = []
    while layer_bytes * len(copies) < 3.2 * l2 or len(copies) < 2:
        layer = [binding.SparseWeight(W, s_w, max_N=N) for W, s_w in mats]
        layer_bytes = sum(sw.stats["bytes_total"] for sw in layer)
        copies.append(layer)
    alg = sum(algorithmic_bytes(sw.stats, N, True) for sw in copies[0])
    xs = {k: torch.from_numpy(binding.pack_int4(workloads.make_x(k, N, 77))).cuda() for k in (5120, 13824)}
    _, s_x = workloads.make_scales(8, N, 77)
    sxd = torch.from_numpy(s_x.copy()).cuda()
    outs = {m: torch.empty((N, m), dtype=torch.float16, device="cuda") for m in (5120, 13824)}

    def enqueue():
        for layer in copies:
            for sw in layer:
                sw.spmm(xs[sw.K], N, sxd, out=outs[sw.M])

    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        enqueue()
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        enqueue()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 20
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    for layer in copies:
        for sw in layer:
            sw.check()
    t = e0.elapsed_time(e1) * 1e-3 / (reps * len(copies))
    row = {"case": "layer13b_chain", "M": 0, "K": 0, "sparsity": sparsity, "N": N, "out": "fp16", "us": t * 1e6,
           "alg_bytes": alg, "stored_bytes": layer_bytes, "gbs": alg / t / 1e9,
           "pct_of_8tbs": 100 * alg / t / 1e9 / CONTRACT_PEAK_GBS, "frac_of_measured": alg / t / 1e9 / measured_peaks()[0],
           "dense_equiv_tops": 2.0 * sum(m * k for m, k in shapes) * N / t / 1e12, "replicas": len(copies),
           "pmr": copies[0][0].stats["pmr"], "launches_per_unit": len(shapes)}
    for layer in copies:
        for sw in layer:
            sw.close()
    torch.cuda.empty_cache()
    return row


def layer_chain_requant(binding, torch, workloads, l2, sparsity=0.5):
    """The same seven weight matrices as layer_chain, as a chain of four chained calls: [Q;K;V]
    stacked into one 15360 x 5120 matrix, O, [gate;up] stacked into 27648 x 5120, down. Activations
    travel as fp16; each call quantises its input per token to INT4 while staging it and leaves the
    absmax its successor needs (O reads the Q columns, down reads the gate columns: the attention
    and the gating in between are not this library's work). One CUDA graph, several layer copies."""
    H, F, N = 5120, 13824, 16
    base = [(H, H)] * 4 + [(F, H)] * 2 + [(H, F)]
    Ws = [workloads.make_weight(m, k, sparsity, 410 + i) for i, (m, k) in enumerate(base)]
    groups = [([0, 1, 2], (0, H)), ([3], (0, H)), ([4, 5], (0, F)), ([6], (0, 0))]
    mats = []
    for g, (idx, rng) in enumerate(groups):
        W = np.concatenate([Ws[i] for i in idx], axis=0)
        mats.append((W, workloads.make_chain_weight_scales(W.shape[0], W.shape[1], 410 + g), rng))
    del Ws
    layer_bytes, copies = 0, []
    while layer_bytes * len(copies) < 3.2 * l2 or len(copies) < 2:
        layer = [binding.SparseWeight(W, s_w, max_N=N) for W, s_w, _ in mats]
        layer_bytes = sum(sw.stats["bytes_total"] for sw in layer)
        copies.append(layer)
    alg = sum(sw.stats["bytes_payload"] + sw.stats["bytes_bitmap"] + sw.stats["bytes_offsets"] + 2 * sw.M +
              2 * N * sw.K + 2 * N * sw.M + 8 * N for sw in copies[0])
    X0 = torch.from_numpy(workloads.make_x_f16(H, N, 77)).cuda()
    a0 = binding.absmax_f16(X0)
    outs = [torch.empty((N, W.shape[0]), dtype=torch.float16, device="cuda") for W, _, _ in mats]
    amaxs = [binding.new_amax() for _ in mats]

    def enqueue():
        for layer in copies:
            src, src_amax = X0, a0
            for sw, (_, _, rng), Y, am in zip(layer, mats, outs, amaxs):
                sw.spmm_requant(src, N, src_amax, out=Y, y_amax=am, amax_range=rng)
                src, src_amax = Y[:, rng[0]:rng[1]], am

    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        enqueue()
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        enqueue()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 20
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    for layer in copies:
        for sw in layer:
            sw.check()
    assert bool(torch.isfinite(outs[-1]).all())
    t = e0.elapsed_time(e1) * 1e-3 / (reps * len(copies))
    row = {"case": "layer13b_chain_requant", "M": 0, "K": 0, "sparsity": sparsity, "N": N, "out": "fp16", "us": t * 1e6,
           "alg_bytes": alg, "stored_bytes": layer_bytes, "gbs": alg / t / 1e9,
           "pct_of_8tbs": 100 * alg / t / 1e9 / CONTRACT_PEAK_GBS, "frac_of_measured": alg / t / 1e9 / measured_peaks()[0],
           "dense_equiv_tops": 2.0 * sum(m * k for m, k in base) * N / t / 1e12, "replicas": len(copies),
           "pmr": copies[0][0].stats["pmr"], "launches_per_unit": len(mats)}
    for layer in copies:
        for sw in layer:
            sw.close()
    torch.cuda.empty_cache()
    return row


def cpu_baseline(W, X, s_w, s_x, stats):
    import oracle
    oracle.build()
    N = X.shape[0]
    per_call = algorithmic_bytes(stats, N, True)
    oracle.dequant(oracle.spmm_dense(W, X), s_w, s_x)
    calls, t0 = 0, time.perf_counter()
    while time.perf_counter() - t0 < 10.0 or calls < 3:
        oracle.dequant(oracle.spmm_dense(W, X), s_w, s_x)
        calls += 1
    dt = time.perf_counter() - t0
    return {"value": per_call * calls / dt / 1e9, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{calls} calls of the oracle (naive masked-dense INT32 GEMM, OpenMP over rows, "
                      f"+ fp64 dequant) on the 4096x4096 s=0.5 N=8 case, {dt:.1f} s",
            "ms_per_spmm": dt / calls * 1e3}


def run_only(args):
    import torch
    from paper_2608_09291_b200 import build as libbuild
    libbuild.build()
    from paper_2608_09291_b200 import binding, workloads
    f = args.only.split(",")
    M, K, s, N = int(f[0]), int(f[1]), float(f[2]), int(f[3])
    fp16 = len(f) > 4 and f[4] == "fp16"
    # K_L > 0 picks the tile width; a seventh field "q4" the folded format (16, K_L, 2, 2)
    fmt = (16, int(f[5]), 2, 2 if (len(f) > 7 and f[7] == "q4") else 1) if len(f) > 5 and int(f[5]) > 0 else None
    n_max = int(f[6]) if len(f) > 6 else N   # largest N the handles are encoded for
    torch.cuda.set_device(0)
    l2 = torch.cuda.get_device_properties(0).L2_cache_size or L2_BYTES_FALLBACK
    W = workloads.make_weight(M, K, s, seed=1)
    X = workloads.make_x(K, n_max, seed=1)
    s_w, s_x = workloads.make_scales(M, n_max, seed=1)
    probe = binding.us_encode(W, None, fmt, n_max, binding.US_ENCODE_HOST_ONLY)
    st = binding.us_get_stats(probe)
    binding.us_destroy(probe)
    case = Case(binding, torch, W, s_w, X, s_x, n_max, replicas_for(st, l2), fmt=fmt)
    for _ in range(max(1, args.warmup)):
        case.enqueue_pass(N, fp16)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        case.enqueue_pass(N, fp16)
    e1.record()
    torch.cuda.synchronize()
    for sw in case.sw:
        sw.check()
    t = e0.elapsed_time(e1) * 1e-3 / (args.steps * len(case.sw))
    alg = algorithmic_bytes(case.stats, N, fp16)
    t_graph = case.time_passes(N, fp16, passes=max(3, args.steps), warmup=3)
    # one more pass with the stage timers of ONE handle in the middle of the pass on (not part of
    # the timing above): a single launch in the steady state of back-to-back launches
    probe = case.sw[len(case.sw) // 2]
    binding.us_stage_timers(probe.handle, 1)
    case.enqueue_pass(N, fp16)
    torch.cuda.synchronize()
    d = binding.us_stage_timers(probe.handle, 0, read=True, per_cta=192)
    ctas = [c for c in d.pop("ctas") if c[3]]
    ck = d.pop("checkpoints")
    timers = {k: (v / max(1, d["warps"]) if k in ("wait", "decode", "epilogue", "lifetime", "prologue") else v)
              for k, v in d.items()}
    timers["checkpoints"] = [v / max(1, d["warps"]) for v in ck]
    if ctas:
        t0 = min(c[0] for c in ctas)
        q = lambda xs: [int(np.percentile(xs, pc)) for pc in (0, 50, 100)]
        timers["cta_ns_min_med_max"] = {"start": q([c[0] - t0 for c in ctas]), "past_wait": q([c[4] - t0 for c in ctas]),
                                        "x_stage": q([c[2] - c[4] for c in ctas]), "tail": q([c[3] - c[1] for c in ctas]),
                                        "x_staged": q([c[2] - t0 for c in ctas]), "end": q([c[3] - t0 for c in ctas]),
                                        "loop": q([c[3] - c[2] for c in ctas])}
    print(json.dumps({"only": args.only, "us_per_launch_graph": t_graph * 1e6, "gbs_graph": alg / t_graph / 1e9,
                      "us_per_launch_stream_order": t * 1e6, "alg_bytes": alg,
                      "stored_bytes": binding.us_spmm_bytes(case.sw[0].handle, N, fp16),
                      "gbs": alg / t / 1e9, "replicas": len(case.sw), "format": list(case.stats["fmt"]),
                      "launch": binding.us_launch_info(case.sw[0].handle, N),
                      "stage_cycles_per_warp": timers}))
    case.close()


def torchrun_command(argv, gpus: int, port: int = 29541):
    """The command that starts `gpus` replica processes of this script on one node."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(gpus),
            "--master-addr", "127.0.0.1", "--master-port", str(port), str(Path(__file__).resolve())] + list(argv)


def run_chain():
    import torch
    from paper_2608_09291_b200 import build as libbuild
    libbuild.build()
    from paper_2608_09291_b200 import binding, workloads
    torch.cuda.set_device(0)
    l2 = torch.cuda.get_device_properties(0).L2_cache_size or L2_BYTES_FALLBACK
    for s in (0.3, 0.5, 0.7):
        print(json.dumps(layer_chain(binding, torch, workloads, l2, s)))
        print(json.dumps(layer_chain_requant(binding, torch, workloads, l2, s)))


def main(argv=None):
    argv = list(sys.argv[1:] if argv is None else argv)
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--only", default=None, metavar="M,K,s,N[,int32|fp16[,K_L[,N_max[,q4]]]]",
                    help="time one case only, with the kernel's stage timers: the small run of the ncu captures")
    ap.add_argument("--chain", action="store_true",
                    help="time only the 13B-shaped layer, as seven plain calls and as a chain of four chained calls")
    args = ap.parse_args(argv)
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus < 1:
        ap.error("--gpus must be at least 1")
    if "WORLD_SIZE" not in os.environ and args.gpus > 1 and not args.only:
        # replicas only: start one process per GPU (no data-path collective; the ranks meet for the
        # barrier around the timed region and the maximum over ranks)
        os.execvp(sys.executable, torchrun_command(argv, args.gpus))
    if world != args.gpus and not args.only:
        sys.exit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world}: launch with "
                 f"torch.distributed.run --nproc-per-node {args.gpus}, or without it")
    if args.impl == "reference":
        reference_arm(args, rank)
        return
    if args.only:
        run_only(args)
        return
    if args.chain:
        run_chain()
        return
    run_ours(args, rank, local_rank, world)


if __name__ == "__main__":
    main()
