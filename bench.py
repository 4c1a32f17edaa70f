#!/usr/bin/env python
"""Benchmark of the W4A16 GEMM hot path on B200.

A "step" is one pass of the decode sweep K=11008, N=4096 (MLP down-projection shape),
M in {1,2,4,8,16}: five calls of w4a16_gemm through the C ABI, each on a different copy of
the packed weights so that every call streams its weights from HBM (the copies total more
than 512 MB; B200's L2 is 126 MB).  The metric is effective HBM bandwidth = algorithmic
bytes (packed weights + FP16 scales + 4-bit zeros + activations + output) / time.

The LAST line of stdout is one compact JSON object (the headline: value, roofline, e2e,
cpu_baseline, clocks ...; under 4 KB).  The bulky per-case table (every case of every config,
explicit split_k sweep, warm-L2 times, FP16 x FP16 reference) is written to
--cases-file and echoed on earlier stdout lines prefixed "CASE ".  `--impl reference` times the
CPU oracle on the host cores instead.  Under torchrun each rank runs an independent replica (the
path has no exchange step) and rank 0 reports the aggregate; `--gpus N` without torchrun starts
the N ranks itself.
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
E2E_STREAMS = 2
PATH_NAMES = {1: "gemm_simple_kernel", 2: "gemm_decode_kernel", 3: "gemm_tile_kernel"}

# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under profiles/
# (None = not captured since that kernel last changed).  Decode kernel: the mean of the five launches of a
# step, M = 1 / 2 / 4 / 8 / 16 at K = 11008, N = 4096: 23.482 / 23.505 / 23.549 / 23.636 / 23.813 MB read, 0 written.
NCU_TRAFFIC_BYTES = {"gemm_decode_kernel": 23597000}
NCU_TRAFFIC_BYTES_TILE = 189215000    # gemm_tile_kernel<256>, M=4096 K=N=8192 (read 135.2 MB + write 54.0 MB, mean of two launches)


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


def _replay_times(graph, reps, torch):
    """Device seconds of each of `reps` replays of one graph (CUDA events on the launching stream)."""
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
    ev[0].record()
    for r in range(reps):
        graph.replay()
        ev[r + 1].record()
    torch.cuda.synchronize()
    return [ev[r].elapsed_time(ev[r + 1]) * 1e-3 for r in range(reps)]


def _time_calls(fn, n_warm, n_timed, torch, per_graph=32, reps=5):
    """Seconds per call of `fn` inside replayed CUDA graphs of `per_graph` calls: (median, min) over
    at least `reps` replays (and at least n_timed calls in total)."""
    for _ in range(max(3, n_warm)):
        fn()
    torch.cuda.synchronize()
    g = _capture(fn, per_graph, torch)
    g.replay()
    torch.cuda.synchronize()
    reps = max(reps, -(-n_timed // per_graph))
    t = [x / per_graph for x in _replay_times(g, reps, torch)]
    return statistics.median(t), min(t)


def summary_line(d):
    """The compact last line: the headline object serialised without the per-case table."""
    return json.dumps(d, separators=(",", ":"))


def emit(summary, cases, cases_file, out=None):
    """Write the per-case table to `cases_file` (if it can be written) and as "CASE {...}" lines, then
    the compact summary as the LAST line of `out`."""
    out = out or sys.stdout
    if cases_file:
        try:
            os.makedirs(os.path.dirname(os.path.abspath(cases_file)), exist_ok=True)
            with open(cases_file, "w") as f:
                json.dump({"summary": summary, "cases": cases}, f, indent=1)
            summary = dict(summary, cases_file=os.path.relpath(cases_file, ROOT))
        except OSError:
            pass
    for c in cases:
        out.write("CASE " + json.dumps(c, separators=(",", ":")) + "\n")
    out.write(summary_line(summary) + "\n")
    out.flush()


def _r(x, nd=4):
    return None if x is None else round(float(x), nd)


def _case_record(c_config, layer, M, K, N, sec_med, sec_min, path, peaks, wl):
    hbm_peak, tc_peak = peaks
    byts = wl.algorithmic_bytes(M, K, N)
    fl = 2.0 * M * N * K
    t_hbm, t_tc = byts / (hbm_peak * 1e9), fl / (tc_peak * 1e12)
    return {"config": c_config, "layer": layer, "M": M, "K": K, "N": N, "path": path,
            "us": _r(sec_med * 1e6, 3), "us_min": _r(sec_min * 1e6, 3),
            "eff_GBps": _r(byts / sec_med / 1e9, 1), "tflops": _r(fl / sec_med / 1e12, 2),
            "bound": "tensor" if t_tc > t_hbm else "hbm",
            "roofline_frac": _r(max(t_hbm, t_tc) / sec_med),
            # the same against the nominal peaks (8 TB/s, 2250 TFLOP/s dense FP16)
            "roofline_frac_nominal": _r(max(byts / 8e12, fl / 2250e12) / sec_med)}


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
    peaks = (hbm_peak, tc_peak)

    K, N = SWEEP_K, SWEEP_N
    layer = Layer(K, N, 2000, torch, B, wl)
    acts_np = [wl.draw_activations(M, K, 2000 + i) for i, M in enumerate(SWEEP_M)]
    acts = [_to_dev(a, torch) for a in acts_np]
    outs = [torch.empty((M, N), dtype=torch.float16, device="cuda") for M in SWEEP_M]
    splits = [args.split_k for M in SWEEP_M]   # 0 = the library's own schedule
    ws_need = max([B.w4a16_workspace_bytes(M, N, K, 128, s) for M in SWEEP_M for s in (0, 1, 2, 4, 8, 16)]
                  + [16384])
    extra_cases = []
    if args.configs and world == 1:          # the per-case table is a 1-GPU report
        extra_cases = [c for c in wl.CASES if c.config in args.configs and c.config != 2]
        # the tensor-bound config 5 goes last: right after its long launches (and their FP16 references)
        # the GPU runs the next short launches 30-40 % slower for a while (power state)
        extra_cases.sort(key=lambda c: c.config == 5)
        for c in extra_cases:
            for s in (0, 2, 4, 8, 16):
                if s <= c.K // 128:
                    ws_need = max(ws_need, B.w4a16_workspace_bytes(c.M, c.N, c.K, 128, s))
    ws = B.ensure_workspace(ws_need)

    def step():
        for A, C, s in zip(acts, outs, splits):
            B.w4a16_gemm(A, layer.take(), C, split_k=s)

    launches_per_step = len(SWEEP_M)   # one kernel per GEMM: the Split-K reduce is inside it
    step_bytes = sum(wl.algorithmic_bytes(M, K, N) for M in SWEEP_M)

    # ---- main timed region.  W warm-up steps; then the region of exactly `steps` steps is captured
    # into a CUDA graph (no host work inside) and replayed `reps` times, each replay bracketed by
    # CUDA events on the launching stream.  ms_per_step is the median replay (the minimum is reported
    # beside it); reps is sized so that the timed work is at least ~0.15 s whatever --steps is.
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    g_main = _capture(step, args.steps, torch)
    g_main.replay()
    torch.cuda.synchronize()
    probe = _replay_times(g_main, 2, torch)[-1]
    reps = max(20, min(2000, int(0.15 / max(probe, 1e-6)) + 1))
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    if not args.no_clocks:
        sampler.start()
    rep_times = _replay_times(g_main, reps, torch)
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    timed_total = sum(rep_times)
    if not args.no_clocks:
        # keep the same load running until the sampler has seen ~0.6 s of it
        t_end = time.perf_counter() + max(0.0, 0.6 - timed_total)
        while time.perf_counter() < t_end:
            g_main.replay()
            torch.cuda.synchronize()
    clocks = sampler.stop()
    elapsed = max_over_ranks(statistics.median(rep_times), dist, "cuda")     # one region of `steps` steps
    elapsed_min = max_over_ranks(min(rep_times), dist, "cuda")
    assert B.w4a16_device_status() == 0, "a kernel reported a device-side timeout"
    value = whole_job_value(step_bytes, args.steps, world, elapsed)

    # ---- per-case numbers (each M alone, same rotation, same launch form)
    cases = []
    per_call = {}
    extras_error = None
    sweep_splits = (1, 2, 4, 8, 16)

    def split_sweep(rec, A, lay, C, M, Kc, Nc, calls):
        """Explicit split_k beside the library's own schedule (the paper takes S as an input)."""
        best_s, best = None, None
        rec["us_by_split_k"] = {}
        for s in sweep_splits:
            if s > Kc // 128:
                continue
            try:
                sec, _ = _time_calls(lambda: B.w4a16_gemm(A, lay.take(), C, split_k=s), 5, calls, torch)
            except B.W4A16Error:
                continue
            rec["us_by_split_k"][str(s)] = _r(sec * 1e6, 3)
            if best is None or sec < best:
                best_s, best = s, sec
        rec["us_split_k_1"] = rec["us_by_split_k"].get("1")
        rec["best_explicit_split_k"] = best_s
        rec["auto_vs_best_explicit"] = _r(rec["us"] / (best * 1e6), 3) if best else None

    for i, M in enumerate(SWEEP_M):
        med, mn = _time_calls(lambda: B.w4a16_gemm(acts[i], layer.take(), outs[i], split_k=splits[i]),
                              20, args.case_calls, torch)
        per_call[M] = med
        rec = _case_record(2, "down_proj", M, K, N, med, mn, PATH_NAMES.get(B.w4a16_choose_path(M, N, K), "?"),
                           peaks, wl)
        rec["split_k"] = splits[i]
        rec["chosen_split_k"] = B.w4a16_choose_split_k(M, N, K)
        cases.append(rec)
    try:
        if rank == 0 and world == 1 and not args.headline_only:
            for i, M in enumerate(SWEEP_M):
                split_sweep(cases[i], acts[i], layer, outs[i], M, K, N, max(64, args.case_calls // 4))
                # warm L2: the same packed copy every call (23 MB stay in the 126 MB L2) -- labelled, not the metric
                sec, _ = _time_calls(lambda: B.w4a16_gemm(acts[i], layer.packed[0], outs[i], split_k=splits[i]),
                                     5, max(64, args.case_calls // 4), torch)
                cases[i]["us_warm_l2"] = _r(sec * 1e6, 3)

            # format variants on the same shape (Eq. 1's symmetric case, smaller groups, BF16): same value recipe,
            # their own algorithmic bytes (no Z traffic when symmetric, more scales with smaller groups)
            for vname, group, sym, bf in (("symmetric_g128", 128, True, False), ("asymmetric_g64", 64, False, False),
                                          ("asymmetric_g32", 32, False, False), ("bf16_g128", 128, False, True)):
                flags = (B.FLAG_SYMMETRIC if sym else 0) | (B.FLAG_BF16 if bf else 0)
                raw = wl.draw_weights(K, N, 2100, group, sym, bf)
                dt = torch.bfloat16 if bf else torch.float16
                rw = _to_dev(raw["Wq"], torch)
                rs = torch.from_numpy(raw["S"].view(np.int16)).cuda().view(dt)
                rz = None if sym else _to_dev(raw["Z"], torch)
                per = wl.algorithmic_bytes(0, K, N, group, sym)
                packs = [B.w4a16_pack(rw, rs, rz, N, K, group, flags) for _ in range(max(2, -(-MIN_ROTATION_BYTES // per)))]
                turn = [0]

                def take_v():
                    turn[0] += 1
                    return packs[turn[0] % len(packs)]
                for M in (1, 8, 16):
                    Av = torch.from_numpy(wl.draw_activations(M, K, 2100 + M, bf16=bf).view(np.int16)).cuda().view(dt)
                    Cv = torch.empty((M, N), dtype=dt, device="cuda")
                    med, mn = _time_calls(lambda: B.w4a16_gemm(Av, take_v(), Cv), 10, max(64, args.case_calls // 4), torch)
                    byts = wl.algorithmic_bytes(M, K, N, group, sym)
                    cases.append({"config": "2-variant", "layer": vname, "M": M, "K": K, "N": N, "us": _r(med * 1e6, 3),
                                  "us_min": _r(mn * 1e6, 3), "algorithmic_bytes": byts, "eff_GBps": _r(byts / med / 1e9, 1),
                                  "roofline_frac": _r(byts / (hbm_peak * 1e9) / med), "bound": "hbm"})
                del packs, rw, rs, rz
                torch.cuda.empty_cache()

            # cuBLAS / PyTorch FP16 x FP16 on pre-dequantized weights: a reference point, not our path
            if not args.no_cublas:
                w16 = [B.w4a16_dequant(layer.packed[0]).clone() for _ in range(6)]
                idx = [0]

                def mm(i):
                    torch.matmul(acts[i], w16[idx[0] % len(w16)], out=outs[i])
                    idx[0] += 1
                for i, M in enumerate(SWEEP_M):
                    sec, _ = _time_calls(lambda: mm(i), 10, max(50, args.case_calls // 4), torch)
                    cases[i]["torch_fp16_matmul_us"] = _r(sec * 1e6, 3)
                    cases[i]["speedup_vs_fp16"] = _r(sec / per_call[M], 3)
                del w16

            # other configs (each case alone, rotating copies)
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
                med, mn = _time_calls(lambda: B.w4a16_gemm(A, cur.take(), C, split_k=0), 10,
                                      max(20, args.case_calls // 4), torch)
                rec = _case_record(c.config, c.name, c.M, c.K, c.N, med, mn,
                                   PATH_NAMES.get(B.w4a16_choose_path(c.M, c.N, c.K), "?"), peaks, wl)
                rec["split_k"] = 0
                rec["chosen_split_k"] = B.w4a16_choose_split_k(c.M, c.N, c.K)
                if c.config in (3, 6):
                    split_sweep(rec, A, cur, C, c.M, c.K, c.N, max(20, args.case_calls // 8))
                    if rec.get("us_split_k_1"):
                        rec["splitk_speedup"] = _r(rec["us_split_k_1"] / rec["us"], 3)
                if not args.no_cublas:
                    if cur_w16 is None:
                        ncopy = max(2, min(6, (MIN_ROTATION_BYTES // 2) // (c.K * c.N * 2) + 1))
                        cur_w16 = [B.w4a16_dequant(cur.packed[0]).clone() for _ in range(ncopy)]
                    k16 = [0]

                    def mm16():
                        torch.matmul(A, cur_w16[k16[0] % len(cur_w16)], out=C)
                        k16[0] += 1
                    sec16, _ = _time_calls(mm16, 5, max(20, args.case_calls // 8), torch, per_graph=8)
                    rec["torch_fp16_matmul_us"] = _r(sec16 * 1e6, 3)
                    rec["speedup_vs_fp16"] = _r(sec16 / med, 3)
                cases.append(rec)
            cur = None
            cur_w16 = None
    except Exception as exc:   # the headline below does not depend on the optional table
        extras_error = "%s: %s" % (type(exc).__name__, exc)

    # ---- end to end through the host-buffer entry point (H2D of A and D2H of C inside the region).  Calls go
    # round-robin to E2E_STREAMS streams, each with staging buffers of its own, so that the copies of one call
    # overlap the kernel of the call before it; every call still does its own H2D, GEMM and D2H in order.
    e2e_streams = [torch.cuda.Stream() for _ in range(E2E_STREAMS)]
    e2e_handles = [st.cuda_stream for st in e2e_streams]
    stage = []
    for _ in range(E2E_STREAMS):
        stage.append([(torch.from_numpy(a.view(np.float16)).pin_memory(),
                       torch.empty((M, K), dtype=torch.float16, device="cuda"),
                       torch.empty((M, N), dtype=torch.float16, device="cuda"),
                       torch.empty((M, N), dtype=torch.float16).pin_memory()) for a, M in zip(acts_np, SWEEP_M)])
    turn = [0]

    def step_e2e():
        for i in range(len(SWEEP_M)):
            sid = turn[0] % E2E_STREAMS
            turn[0] += 1
            hA, dA, dC, hC = stage[sid][i]
            B.w4a16_gemm_host(hA, dA, layer.take(), dC, hC, split_k=splits[i], stream=e2e_handles[sid])

    torch.cuda.synchronize()
    for _ in range(max(3, args.warmup)):
        step_e2e()
    torch.cuda.synchronize()
    e2e_steps = max(args.steps, 200)      # long enough to time on the wall clock
    e2e_times = []
    for _ in range(5):
        if dist:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            step_e2e()
        torch.cuda.synchronize()
        e2e_times.append(time.perf_counter() - t0)
    e2e_elapsed = max_over_ranks(statistics.median(e2e_times), dist, "cuda")
    e2e_value = whole_job_value(step_bytes, e2e_steps, world, e2e_elapsed)
    # the results that came back to the host are the ones the device-resident path produces, bit for bit
    # (same inputs, same schedule: any difference would mean calls on different streams disturbed each other)
    # (every packed copy holds the same weights, so whichever copy the last overlapping calls used, their
    # results must equal the sequential call's)
    for i, M in enumerate(SWEEP_M):
        want = B.w4a16_gemm(acts[i], layer.packed[0], split_k=splits[i]).cpu()
        for sid in range(E2E_STREAMS):
            assert torch.equal(stage[sid][i][3], want), \
                "end-to-end result differs from the device-resident call (M = %d, stream %d)" % (M, sid)
    assert B.w4a16_device_status() == 0

    # ---- roofline of the dominant kernel.  Every launch of the timed region is gemm_decode_kernel (one
    # per GEMM), so its average launch duration over the region is region time / launches, and the
    # algorithmic bytes of an average launch are step bytes / launches per step.
    dom_kernel = PATH_NAMES.get(B.w4a16_choose_path(SWEEP_M[0], N, K), "?")
    launch_us = elapsed / (args.steps * launches_per_step) * 1e6
    bytes_per_launch = step_bytes / launches_per_step
    achieved = bytes_per_launch / launch_us / 1e3
    heavy = SWEEP_M[-1]
    roofline = {"bound": "hbm", "kernel": dom_kernel,
                "launches": "the %d launches of a step, averaged over the timed region" % launches_per_step,
                "achieved": _r(achieved, 1), "peak": hbm_peak, "peak_kind": "of " + peak_kind, "unit": "GB/s",
                "frac": _r(achieved / hbm_peak), "frac_of_nominal_8TBps": _r(achieved / 8000.0),
                "traffic": NCU_TRAFFIC_BYTES.get(dom_kernel),
                "algorithmic_bytes_per_launch": int(bytes_per_launch), "launch_us": _r(launch_us, 3),
                "launch_us_by_M": {str(M): _r(per_call[M] * 1e6, 3) for M in SWEEP_M},
                "frac_by_M": {str(M): _r(wl.algorithmic_bytes(M, K, N) / per_call[M] / 1e9 / hbm_peak)
                              for M in SWEEP_M},
                "heaviest_launch": "M=%d: %s" % (heavy, PATH_NAMES.get(B.w4a16_choose_path(heavy, N, K), "?"))}

    # ---- CPU baseline: the oracle on whole steps (rank 0, N = 1 only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        worst, reps_cpu, dt = 0.0, 0, 0.0
        step()
        torch.cuda.synchronize()
        while dt < 10.0 and reps_cpu < 64:     # whole steps until about 10 s of CPU work
            t0 = time.perf_counter()
            refs = [oracle.gemm(acts_np[i], layer.raw["Wq"], layer.raw["S"], layer.raw["Z"], M, N, K, 128)
                    for i, M in enumerate(SWEEP_M)]
            dt += time.perf_counter() - t0
            reps_cpu += 1
        for i, M in enumerate(SWEEP_M):
            got = outs[i].cpu().numpy().astype(np.float64)   # result of the last call
            worst = max(worst, float(np.max(np.abs(got - refs[i]) / (1.0 + np.abs(refs[i])))))
        cpu = {"value": _r(step_bytes * reps_cpu / dt / 1e9, 5), "unit": UNIT, "cores": oracle.num_threads(),
               "kind": "oracle",
               "sample": "%d full steps (all 5 GEMMs, all columns), %.1f s of CPU time" % (reps_cpu, dt),
               "max_elem_err_vs_gpu": _r(worst, 6)}

    # the tensor-bound end of the path: the largest prefill case that was timed (config 5)
    roofline_tensor = None
    big = [c for c in cases if c["config"] == 5]
    if big:
        b = max(big, key=lambda c: c["M"])
        pk = {}
        try:
            pk = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        except Exception:
            pass
        sustained = float(pk.get("bf16_tflops_sustained", 1400.0))
        roofline_tensor = {"bound": "tensor", "kernel": b["path"], "case": "M=%d K=%d N=%d" % (b["M"], b["K"], b["N"]),
                           "achieved": b["tflops"], "peak": tc_peak,
                           "peak_kind": "of " + peak_kind + " (burst; FP16 takes the BF16 figure, same nominal rate)",
                           "unit": "TFLOP/s", "frac": _r(b["tflops"] / tc_peak),
                           "frac_of_sustained_peak": _r(b["tflops"] / sustained),
                           "frac_of_nominal_2250": _r(b["tflops"] / 2250.0),
                           "launch_us": b["us"], "traffic": NCU_TRAFFIC_BYTES_TILE}
    # config 4: the four layers of one transformer block, summed per batch size
    block_sums = {}
    for c in cases:
        if c["config"] == 4:
            block_sums[str(c["M"])] = _r(block_sums.get(str(c["M"]), 0.0) + c["us"], 2)

    if rank == 0:
        summary = {
            "metric": METRIC, "value": _r(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": _r(elapsed / args.steps * 1e3, 6),
            "ms_per_step_min": _r(elapsed_min / args.steps * 1e3, 6), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "group": 128, "accumulate": "f32", "split_k": splits[0],
                       "l2": "cold: %d packed weight copies (%d MB) rotated, every call reads HBM"
                             % (layer.copies, layer.copies * (K * N // 2) >> 20),
                       "launch": "one CUDA graph of the %d steps, replayed %d times; ms_per_step = median replay"
                                 % (args.steps, reps),
                       "timed_s": _r(timed_total, 4), "multi_gpu": "replicas only"},
            "clocks": clocks,
            "e2e": {"value": _r(e2e_value, 2), "unit": UNIT,
                    "h2d_bytes_per_step": sum(2 * M * K for M in SWEEP_M),
                    "d2h_bytes_per_step": sum(2 * M * N for M in SWEEP_M),
                    "ms_per_step": _r(e2e_elapsed / e2e_steps * 1e3, 6), "steps": e2e_steps,
                    "streams": E2E_STREAMS,
                    "note": "A from pinned host memory, C to pinned host memory, weights resident; wall clock"},
            "gpu_launches": launches_per_step * args.steps * reps,
            "roofline": roofline,
            "roofline_tensor": roofline_tensor,
            "config4_block_us_by_M": block_sums,
            "cpu_baseline": cpu,
        }
        if extras_error:
            summary["cases_error"] = extras_error[:200]
        emit(summary, cases, args.cases_file)
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
                           3, max(args.calls, 64), torch, per_graph=min(32, max(2, layer.copies)))[0] * 1e6
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
    ap.add_argument("--cases-file", default=os.path.join(ROOT, "gpurun_out", "bench_cases.json"),
                    help="where the per-case table goes ('' = nowhere)")
    ap.add_argument("--headline-only", action="store_true",
                    help="skip the per-case table (other configs, split_k sweep, FP16 reference)")
    args = ap.parse_args()
    if args.one:
        run_one(args)
        return
    world_env = os.environ.get("WORLD_SIZE")
    if args.gpus < 1:
        raise SystemExit("--gpus must be at least 1")
    if world_env is None and args.gpus > 1:
        # not under torchrun: start the N replicas ourselves (one process per GPU, rendezvous on 127.0.0.1)
        import socket
        with socket.socket() as s:
            s.bind(("127.0.0.1", 0))
            port = s.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    if world_env is not None and int(world_env) != args.gpus:
        raise SystemExit("--gpus %d but WORLD_SIZE=%s: launch one rank per GPU" % (args.gpus, world_env))
    if args.impl == "reference":
        args.steps = 5 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args)
    else:
        args.steps = 100 if args.steps is None else args.steps
        args.warmup = max(3, 20 if args.warmup is None else args.warmup)
        run_ours(args)


if __name__ == "__main__":
    main()
