#!/usr/bin/env python
"""Benchmark of the W4A16 GEMM hot path on B200.

A "step" is one pass of the decode sweep K=11008, N=4096 (MLP down-projection shape),
M in {1,2,4,8,16}: five calls of w4a16_gemm through the C ABI, each on a different copy of
the packed weights so that every call streams its weights from HBM (the copies total more
than 512 MB; B200's L2 is 126 MB).  The metric is effective HBM bandwidth = algorithmic
bytes (packed weights + FP16 scales + 4-bit zeros + activations + output) / time.

Prints ONE JSON line (see the keys below).  `--impl reference` times the CPU oracle on the
host cores instead.  Under torchrun each rank runs an independent replica (the path has no
exchange step) and rank 0 reports the aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "w4a16_gemm_effective_hbm_bandwidth"
UNIT = "GB/s"
SWEEP_K, SWEEP_N, SWEEP_M = 11008, 4096, (1, 2, 4, 8, 16)
WORKLOAD = "config2_down_proj_decode_K11008_N4096_M1-2-4-8-16"
MIN_ROTATION_BYTES = 512 << 20
PATH_NAMES = {1: "gemm_simple_kernel", 2: "gemm_decode_kernel", 3: "gemm_tile_kernel"}

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# capture summarised under profiles/ (None until captured)
# DRAM read + write of one M=16 K=11008 N=4096 launch, by the kernel the library picks for it (ncu; None = not
# captured since that kernel last changed)
NCU_TRAFFIC_BYTES = {"gemm_tile_kernel": 24134016,      # read 24.13 MB, write 0
                     "gemm_decode_kernel": 23817984}    # read 23.82 MB, write 0 (<2, 2, cluster>)
NCU_TRAFFIC_BYTES_TILE = 192325632    # gemm_tile_kernel<256>, M=4096 K=N=8192 (read 136.1 MB + write 56.2 MB)


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["hbm_gbs"]), float(d.get("bf16_tflops", 1590.0)), "measured"
        except Exception:
            pass
    return 6650.0, 1590.0, "fallback"


def _rank_world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), \
        int(os.environ.get("LOCAL_RANK", "0"))


# ------------------------------------------------------------------------------ ranks
def max_over_ranks(seconds, dist, device):
    """The slowest rank's time: replicas run independently, the job is as slow as its slowest rank."""
    if dist is None:
        return float(seconds)
    import torch
    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(step_bytes, steps, world, seconds):
    """Aggregate effective bandwidth in GB/s: every rank moves step_bytes per step (weak scaling)."""
    return step_bytes * steps * world / seconds / 1e9


# ------------------------------------------------------------------------------ clocks
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                    "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ------------------------------------------------------------------------------ reference arm
def run_reference(args):
    """The CPU oracle, as it stands, timed on the host cores.  Each step is a bounded sample
    of the workload: the same five GEMMs restricted to the first `cols` output columns."""
    rank, world, _ = _rank_world()
    if rank != 0:
        return
    import oracle
    from paper_2601_16536_b200 import workloads as wl
    K, N = SWEEP_K, SWEEP_N
    cols = 256
    w = wl.draw_weights(K, N, 2000)
    acts = [wl.draw_activations(M, K, 2000 + i) for i, M in enumerate(SWEEP_M)]
    frac = cols / N

    def step():
        for M, A in zip(SWEEP_M, acts):
            oracle.gemm(A, w["Wq"], w["S"], w["Z"], M, N, K, 128, cols=(0, cols))

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    step_bytes = sum(wl.algorithmic_bytes(M, K, N) for M in SWEEP_M) * frac
    val = step_bytes * args.steps / dt / 1e9
    sample = "first %d of %d output columns of each of the 5 GEMMs per step" % (cols, N)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "group": 128, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------ our arm
def _to_dev(a, torch):
    if a.dtype == np.uint32:
        return torch.from_numpy(a.view(np.int32)).cuda()
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.float16)).cuda()
    return torch.from_numpy(a).cuda()


class Layer:
    """One weight matrix: `copies` packed replicas in distinct device memory (cold-L2 rotation)."""

    def __init__(self, K, N, seed, torch, B, wl, min_bytes=MIN_ROTATION_BYTES, max_copies=32):
        self.K, self.N = K, N
        self.raw = wl.draw_weights(K, N, seed)
        per = K * N // 2 + (K // 128) * N * 5 // 2
        self.copies = max(2, min(max_copies, -(-min_bytes // per)))
        rw, rs, rz = (_to_dev(self.raw[k], torch) for k in ("Wq", "S", "Z"))
        self.packed = [B.w4a16_pack(rw, rs, rz, N, K) for _ in range(self.copies)]
        torch.cuda.synchronize()
        self.next = 0

    def take(self):
        pw = self.packed[self.next]
        self.next = (self.next + 1) % self.copies
        return pw


def _capture(fn, n, torch):
    """A CUDA graph of n consecutive calls of fn (launches recorded once, replayed without
    per-call host work, so the device time of back-to-back kernels is what gets measured)."""
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for _ in range(n):
            fn()
    return g


def _time_calls(fn, n_warm, n_timed, torch, per_graph=32):
    """Seconds per call: `fn` captured per_graph times into a CUDA graph, replayed."""
    for _ in range(max(3, n_warm)):
        fn()
    torch.cuda.synchronize()
    g = _capture(fn, per_graph, torch)
    reps = max(1, n_timed // per_graph)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e-3 / (reps * per_graph)


def run_ours(args):
    import torch
    rank, world, local = _rank_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    from paper_2601_16536_b200 import binding as B
    from paper_2601_16536_b200 import workloads as wl
    B.load()
    hbm_peak, tc_peak, peak_kind = _peaks()

    K, N = SWEEP_K, SWEEP_N
    layer = Layer(K, N, 2000, torch, B, wl)
    acts_np = [wl.draw_activations(M, K, 2000 + i) for i, M in enumerate(SWEEP_M)]
    acts = [_to_dev(a, torch) for a in acts_np]
    outs = [torch.empty((M, N), dtype=torch.float16, device="cuda") for M in SWEEP_M]
    splits = [args.split_k for M in SWEEP_M]   # 0 = the library's own schedule
    ws_need = max([B.w4a16_workspace_bytes(M, N, K, 128, s) for M, s in zip(SWEEP_M, splits)] + [16384])
    extra_cases = []
    if args.configs:
        for c in wl.CASES:
            if c.config in args.configs and not (c.config == 2):
                if world > 1 and c.config != 2:
                    continue        # the per-case table is a 1-GPU report
                extra_cases.append(c)
        # the tensor-bound config 5 goes last: right after its long launches (and their FP16 references)
        # the GPU runs the next short launches 30-40 % slower for a while (power state), which used to
        # land on whichever small layer came next
        extra_cases.sort(key=lambda c: c.config == 5)
        for c in extra_cases:
            ws_need = max(ws_need, B.w4a16_workspace_bytes(c.M, c.N, c.K, 128, 0))
    ws = B.ensure_workspace(ws_need)

    def step():
        for A, C, s in zip(acts, outs, splits):
            B.w4a16_gemm(A, layer.take(), C, split_k=s)

    launches_per_step = len(SWEEP_M)   # one kernel per GEMM: the Split-K reduce is inside it
    step_bytes = sum(wl.algorithmic_bytes(M, K, N) for M in SWEEP_M)

    # ---- main timed region: W warm-up steps, exactly K steps, device events, max over ranks.
    # The steps are captured into CUDA graphs (one rotation through the weight copies each) and
    # replayed, so the timed region holds exactly steps x 5 kernel launches and no host work.
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    chunk = max(1, min(args.steps, layer.copies))
    g_main = _capture(step, chunk, torch)
    reps, rem = divmod(args.steps, chunk)
    g_rem = _capture(step, rem, torch) if rem else None
    g_main.replay()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    if not args.no_clocks:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g_main.replay()
    if g_rem is not None:
        g_rem.replay()
    e1.record()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    elapsed = e0.elapsed_time(e1) * 1e-3
    if not args.no_clocks:
        # keep the same load running until the sampler has seen ~0.6 s of it
        t_end = time.perf_counter() + max(0.0, 0.6 - elapsed)
        while time.perf_counter() < t_end:
            g_main.replay()
            torch.cuda.synchronize()
    clocks = sampler.stop()
    elapsed = max_over_ranks(elapsed, dist, "cuda")
    assert B.w4a16_device_status() == 0, "a kernel reported a device-side timeout"
    value = whole_job_value(step_bytes, args.steps, world, elapsed)

    # ---- per-case numbers (each M alone, same rotation)
    cases = []
    per_call = {}
    for i, M in enumerate(SWEEP_M):
        sec = _time_calls(lambda: B.w4a16_gemm(acts[i], layer.take(), outs[i], split_k=splits[i]),
                          20, args.case_calls, torch)
        byts = wl.algorithmic_bytes(M, K, N)
        per_call[M] = sec
        cases.append({"config": 2, "layer": "down_proj", "M": M, "K": K, "N": N, "split_k": splits[i],
                      "path": PATH_NAMES.get(B.w4a16_choose_path(M, N, K), "?"),
                      "us": sec * 1e6, "eff_GBps": byts / sec / 1e9, "tflops": 2.0 * M * N * K / sec / 1e12,
                      "roofline_frac": max(byts / (hbm_peak * 1e9), 2.0 * M * N * K / (tc_peak * 1e12)) / sec})
    # split_k = 1 ("data parallel" in the paper's comparison) beside the chosen split
    for i, M in enumerate(SWEEP_M):
        sec = _time_calls(lambda: B.w4a16_gemm(acts[i], layer.take(), outs[i], split_k=1), 10,
                          max(50, args.case_calls // 4), torch)
        cases[i]["us_split_k_1"] = sec * 1e6

    # cuBLAS / PyTorch FP16 x FP16 on pre-dequantized weights: a reference point, not our path
    if not args.no_cublas:
        w16 = [B.w4a16_dequant(layer.packed[0]).clone() for _ in range(6)]
        idx = [0]

        def mm(i):
            torch.matmul(acts[i], w16[idx[0] % len(w16)], out=outs[i])
            idx[0] += 1
        for i, M in enumerate(SWEEP_M):
            sec = _time_calls(lambda: mm(i), 10, max(50, args.case_calls // 4), torch)
            cases[i]["torch_fp16_matmul_us"] = sec * 1e6
            cases[i]["speedup_vs_fp16"] = sec / per_call[M]
        del w16

    # other configs on request (each case alone, rotating copies)
    cur = None
    cur_w16 = None
    for c in extra_cases:
        if cur is None or (cur.K, cur.N) != (c.K, c.N):
            cur = None
            cur_w16 = None
            torch.cuda.empty_cache()
            cur = Layer(c.K, c.N, c.seed, torch, B, wl)
        A = _to_dev(wl.draw_activations(c.M, c.K, c.seed, c.a_sigma, c.outliers), torch)
        C = torch.empty((c.M, c.N), dtype=torch.float16, device="cuda")
        s = 0
        sec = _time_calls(lambda: B.w4a16_gemm(A, cur.take(), C, split_k=s), 10,
                          max(20, args.case_calls // 4), torch)
        byts = wl.algorithmic_bytes(c.M, c.K, c.N)
        fl = 2.0 * c.M * c.N * c.K
        rec = {"config": c.config, "layer": c.name, "M": c.M, "K": c.K, "N": c.N, "split_k": s,
               "path": PATH_NAMES.get(B.w4a16_choose_path(c.M, c.N, c.K), "?"),
               "us": sec * 1e6, "eff_GBps": byts / sec / 1e9, "tflops": fl / sec / 1e12,
               "bound": "tensor" if fl / (tc_peak * 1e12) > byts / (hbm_peak * 1e9) else "hbm",
               "roofline_frac": max(byts / (hbm_peak * 1e9), fl / (tc_peak * 1e12)) / sec}
        if c.config == 6:
            # the paper's Figure 2 comparison: one slice ("data parallel") beside the chosen schedule
            sec1 = _time_calls(lambda: B.w4a16_gemm(A, cur.take(), C, split_k=1), 5,
                               max(20, args.case_calls // 8), torch)
            rec["us_split_k_1"] = sec1 * 1e6
            rec["splitk_speedup"] = sec1 / sec
        if not args.no_cublas:
            if cur_w16 is None:
                ncopy = max(2, min(6, (MIN_ROTATION_BYTES // 2) // (c.K * c.N * 2) + 1))
                cur_w16 = [B.w4a16_dequant(cur.packed[0]).clone() for _ in range(ncopy)]
            k16 = [0]

            def mm16():
                torch.matmul(A, cur_w16[k16[0] % len(cur_w16)], out=C)
                k16[0] += 1
            sec16 = _time_calls(mm16, 5, max(20, args.case_calls // 8), torch, per_graph=8)
            rec["torch_fp16_matmul_us"] = sec16 * 1e6
            rec["speedup_vs_fp16"] = sec16 / sec
        cases.append(rec)

    # ---- end to end through the host-buffer entry point (H2D of A and D2H of C inside the region)
    hA = [torch.from_numpy(a.view(np.float16)).pin_memory() for a in acts_np]
    hC = [torch.empty((M, N), dtype=torch.float16).pin_memory() for M in SWEEP_M]

    def step_e2e():
        for i in range(len(SWEEP_M)):
            B.w4a16_gemm_host(hA[i], acts[i], layer.take(), outs[i], hC[i], split_k=splits[i])

    for _ in range(max(3, args.warmup)):
        step_e2e()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step_e2e()
    torch.cuda.synchronize()
    e2e_elapsed = time.perf_counter() - t0
    e2e_elapsed = max_over_ranks(e2e_elapsed, dist, "cuda")
    e2e_value = whole_job_value(step_bytes, args.steps, world, e2e_elapsed)

    # ---- roofline of the dominant kernel (the decode GEMM kernel at M = 16, the heaviest call)
    dom_M = SWEEP_M[-1]
    dom_bytes = wl.algorithmic_bytes(dom_M, K, N)
    achieved = dom_bytes / per_call[dom_M] / 1e9
    dom_kernel = PATH_NAMES.get(B.w4a16_choose_path(dom_M, N, K), "?")
    roofline = {"bound": "hbm", "kernel": dom_kernel, "case": "M=%d K=%d N=%d" % (dom_M, K, N),
                "achieved": achieved, "peak": hbm_peak, "peak_kind": "of " + peak_kind, "unit": "GB/s",
                "frac": achieved / hbm_peak, "traffic": NCU_TRAFFIC_BYTES.get(dom_kernel),
                "algorithmic_bytes_per_launch": dom_bytes,
                "launch_us": per_call[dom_M] * 1e6,
                "sweep_frac": value / world / hbm_peak}

    # ---- CPU baseline: the oracle on the full sweep once (rank 0, N = 1 only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        worst, reps_cpu, dt = 0.0, 0, 0.0
        while dt < 10.0 and reps_cpu < 64:     # whole steps until about 10 s of CPU work
            t0 = time.perf_counter()
            refs = [oracle.gemm(acts_np[i], layer.raw["Wq"], layer.raw["S"], layer.raw["Z"], M, N, K, 128)
                    for i, M in enumerate(SWEEP_M)]
            dt += time.perf_counter() - t0
            reps_cpu += 1
        for i, M in enumerate(SWEEP_M):
            got = outs[i].cpu().numpy().astype(np.float64)   # result of the last timed call
            worst = max(worst, float(np.max(np.abs(got - refs[i]) / (1.0 + np.abs(refs[i])))))
        cpu = {"value": step_bytes * reps_cpu / dt / 1e9, "unit": UNIT, "cores": oracle.num_threads(),
               "kind": "oracle",
               "sample": "%d full steps (all 5 GEMMs, all columns), %.1f s of CPU time" % (reps_cpu, dt),
               "max_elem_err_vs_gpu": worst}

    # the tensor-bound end of the path: the largest prefill case that was timed (config 5)
    roofline_tensor = None
    big = [c for c in cases if c["config"] == 5]
    if big:
        b = max(big, key=lambda c: c["M"])
        peaks = {}
        try:
            peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        except Exception:
            pass
        sustained = float(peaks.get("bf16_tflops_sustained", 1400.0))
        roofline_tensor = {"bound": "tensor", "kernel": b["path"], "case": "M=%d K=%d N=%d" % (b["M"], b["K"], b["N"]),
                           "achieved": b["tflops"], "peak": tc_peak, "peak_kind": "of " + peak_kind +
                           " (burst; FP16 takes the BF16 figure, same nominal rate)", "unit": "TFLOP/s",
                           "frac": b["tflops"] / tc_peak, "frac_of_sustained_peak": b["tflops"] / sustained,
                           "launch_us": b["us"], "traffic": NCU_TRAFFIC_BYTES_TILE}
    # config 4: the four layers of one transformer block, summed per batch size
    block_sums = {}
    for c in cases:
        if c["config"] == 4:
            block_sums.setdefault(c["M"], 0.0)
            block_sums[c["M"]] += c["us"]

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": elapsed / args.steps * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "group": 128, "accumulate": "f32", "split_k": splits,
                       "l2": "cold: %d packed weight copies (%d MB) rotated, every call reads HBM"
                             % (layer.copies, layer.copies * (K * N // 2) >> 20),
                       "launch": "CUDA graphs of %d steps, replayed" % chunk,
                       "multi_gpu": "replicas only"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT,
                    "h2d_bytes_per_step": sum(2 * M * K for M in SWEEP_M),
                    "d2h_bytes_per_step": sum(2 * M * N for M in SWEEP_M),
                    "ms_per_step": e2e_elapsed / args.steps * 1e3,
                    "note": "activations from pinned host memory, result to pinned host memory; "
                            "packed weights resident in HBM"},
            "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline,
            "roofline_tensor": roofline_tensor,
            "config4_block_us_by_M": block_sums,
            "cpu_baseline": cpu,
            "cases": cases,
        }))
    del ws
    if dist:
        dist.destroy_process_group()


def run_one(args):
    """One shape alone: `--one M,K,N` packs rotating weight copies, makes --calls plain stream
    launches (no CUDA graph) and prints the mean device time per call.  The small, launch-by-launch
    command used for profiler captures."""
    import torch
    from paper_2601_16536_b200 import binding as B
    from paper_2601_16536_b200 import workloads as wl
    torch.cuda.set_device(0)
    M, K, N = args.one
    layer = Layer(K, N, 1, torch, B, wl, min_bytes=args.rotation_mb << 20)
    A = _to_dev(wl.draw_activations(M, K, 1), torch)
    C = torch.empty((M, N), dtype=torch.float16, device="cuda")
    ws = B.ensure_workspace(max(B.w4a16_workspace_bytes(M, N, K, 128, args.split_k), 16384))
    for _ in range(3):
        B.w4a16_gemm(A, layer.take(), C, split_k=args.split_k, path=args.path)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.calls):
        B.w4a16_gemm(A, layer.take(), C, split_k=args.split_k, path=args.path)
    e1.record()
    torch.cuda.synchronize()
    assert B.w4a16_device_status() == 0
    us = e0.elapsed_time(e1) * 1e3 / args.calls
    byts = wl.algorithmic_bytes(M, K, N)
    out = {"one": [M, K, N], "path": args.path, "split_k": args.split_k, "calls": args.calls,
           "us_per_call_stream": us, "copies": layer.copies}
    if args.graph:
        # the same call inside replayed CUDA graphs: device time of back-to-back launches
        g_us = _time_calls(lambda: B.w4a16_gemm(A, layer.take(), C, split_k=args.split_k, path=args.path),
                           3, max(args.calls, 64), torch, per_graph=min(32, max(2, layer.copies))) * 1e6
        hbm_peak, tc_peak, _ = _peaks()
        out.update(us_per_call_graph=g_us, eff_GBps=byts / g_us / 1e3, tflops=2.0 * M * N * K / g_us / 1e6,
                   roofline_frac=max(byts / (hbm_peak * 1e3), 2.0 * M * N * K / (tc_peak * 1e6)) / g_us)
    print(json.dumps(out))
    del ws


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--split-k", type=int, default=0, help="force one split factor (0 = automatic)")
    ap.add_argument("--configs", type=lambda s: [int(x) for x in s.split(",")], default=[1, 3, 4, 5, 6],
                    help="besides the timed config-2 step, report every case of these configs (2 = none)")
    ap.add_argument("--case-calls", type=int, default=400)
    ap.add_argument("--no-cublas", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-clocks", action="store_true", help="do not sample nvidia-smi clocks")
    ap.add_argument("--one", type=lambda s: [int(x) for x in s.split(",")], default=None,
                    help="M,K,N: time this one shape with plain stream launches and exit")
    ap.add_argument("--calls", type=int, default=20, help="launches of --one")
    ap.add_argument("--graph", action="store_true", help="--one: also time the call inside CUDA graphs")
    ap.add_argument("--path", type=int, default=0, help="kernel path of --one (0 auto, 1 simple, 2 decode, 3 tile)")
    ap.add_argument("--rotation-mb", type=int, default=512, help="bytes of rotating weight copies of --one")
    args = ap.parse_args()
    if args.one:
        run_one(args)
        return
    if args.impl == "reference":
        args.steps = 5 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args)
    else:
        args.steps = 2000 if args.steps is None else args.steps
        args.warmup = max(3, 20 if args.warmup is None else args.warmup)
        run_ours(args)


if __name__ == "__main__":
    main()
