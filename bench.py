"""Benchmark of the dual-trit-plane decode linears on B200.

One step = one pass of the hot path over the seven decode linears of a LLaMA-3-8B layer at
batch 1 (q, k, v, o, gate, up, down), one ptqtp_gemv call per matrix, on packed planes that are
already resident in HBM.  Steps rotate over `--sets` distinct copies of the layer (default 8,
928 MB) so that every packed byte comes from HBM, not from L2.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

prints ONE JSON line (rank 0).  With N > 1 (under torchrun) every rank runs an independent
replica on its own GPU: the layer has no exchange step, so there is no collective on the data
path; times are the maximum over ranks.

`--impl reference` times the CPU oracle (plain C loops, fp64) on the host cores instead.
"""
import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2509_16989_b200.inputs import LLAMA3_8B, LLAMA3_8B_UNIQUE, make_case  # noqa: E402

METRIC = "dual-trit-plane GEMV effective HBM GB/s at batch 1 (us/layer in us_per_layer)"
UNIT = "GB/s"
WORKLOAD = "llama3-8b decode linears (q,k,v,o 4096x4096|1024x4096, gate/up 14336x4096, down 4096x14336), batch 1"
MATRICES = ("q", "k", "v", "o", "gate", "up", "down")
UNIQUE_OF = {"q": "qo", "o": "qo", "k": "kv", "v": "kv", "gate": "gate_up", "up": "gate_up", "down": "down"}
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum over algorithmic bytes in the ncu capture of the 14336x4096 launch of
# the current GEMV kernel (profiles/gemv2_gate_up_14336x4096.md); set to None when the kernel changes
DRAM_TRAFFIC_RATIO = 31239424.0 / 31232000.0
FALLBACK_HBM_GBS = 6650.0


def algorithmic_bytes(N, K, M=1):
    """Bytes the method itself must move for one call: 2-bit planes, fp16 scale pairs, x and y."""
    return N * K // 2 + 4 * N * K // 128 + 2 * M * K + 2 * M * N


def weight_bytes(N, K):
    return N * K // 2 + 4 * N * K // 128


STEP_BYTES = sum(algorithmic_bytes(*LLAMA3_8B[m]) for m in MATRICES)
STEP_WEIGHT_BYTES = sum(weight_bytes(*LLAMA3_8B[m]) for m in MATRICES)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


# ----------------------------------------------------------------------------- replicas
def max_over_ranks(ms, world, device=None):
    """Slowest rank's time: the job is as fast as its slowest replica (no-op for one rank)."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput_gbs(ms_per_step, world, step_bytes=None):
    """Whole-job GB/s of `world` independent replicas that each move step_bytes per step (weak scaling)."""
    return world * (STEP_BYTES if step_bytes is None else step_bytes) / (ms_per_step * 1e-3) / 1e9


# ----------------------------------------------------------------------------- clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only) every 20 ms."""

    REASONS = (("hw_slowdown", 0x8), ("sw_thermal_slowdown", 0x20), ("hw_thermal_slowdown", 0x40),
               ("sw_power_cap", 0x4), ("hw_power_brake", 0x80))

    def __init__(self, torch_device):
        super().__init__(daemon=True)
        self.samples = []          # (t, sm_mhz, reasons bitmask)
        self.sm_max = None
        self._stop_evt = threading.Event()
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self._nv = pynvml
            h = None
            try:
                uuid = str(torch.cuda.get_device_properties(torch_device).uuid)
                if not uuid.startswith("GPU-"):
                    uuid = "GPU-" + uuid
                h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            except Exception:
                h = pynvml.nvmlDeviceGetHandleByIndex(torch_device)
            self._h = h
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def sample_now(self):
        """One sample taken by the caller (a short timed region may end before the thread's next turn)."""
        if self._h is None:
            return
        nv = self._nv
        try:
            mhz = int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
            try:
                rs = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
            except Exception:
                rs = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
            self.samples.append((time.perf_counter(), mhz, rs))
        except Exception:
            pass

    def run(self):
        if self._h is None:
            return
        while not self._stop_evt.is_set():
            self.sample_now()
            self._stop_evt.wait(0.02)

    def stop(self):
        self._stop_evt.set()

    def summary(self, t0, t1):
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        window = "timed region"
        if len(inside) < 3 and len(self.samples) > len(inside):
            inside = list(self.samples)
            window = "whole run (timed region shorter than 3 samples)"
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": [], "samples": 0, "window": "none"}
        mask = 0
        for s in inside:
            mask |= s[2]
        reasons = [name for name, bit in self.REASONS if mask & bit]
        return {"sm_mhz": float(np.median([s[1] for s in inside])), "sm_max_mhz": self.sm_max,
                "reasons": reasons, "samples": len(inside), "window": window}


# ----------------------------------------------------------------------------- CPU oracle legs
def oracle_layer_time(cases, rows_frac, threads):
    """One pass of the fp64 oracle over the first rows of each of the seven matrices; returns seconds, bytes."""
    from oracle.c_oracle import layer_fp64_c
    t0 = time.perf_counter()
    nbytes = 0
    for m in MATRICES:
        c = cases[UNIQUE_OF[m]]
        rows = max(8, int(round(c["N"] * rows_frac)))
        rows = min(rows, c["N"])
        layer_fp64_c(c["T1"][:rows], c["T2"][:rows], c["alpha1"][:rows], c["alpha2"][:rows], c["x"],
                     threads=threads)
        nbytes += algorithmic_bytes(rows, c["K"])
    return time.perf_counter() - t0, nbytes


def make_cases():
    return {u: make_case(N, K, seed=i) for i, (u, (N, K)) in enumerate(sorted(LLAMA3_8B_UNIQUE.items()))}


def cpu_baseline(cases, budget_s=4.0):
    from oracle.c_oracle import max_threads
    threads = max_threads()
    oracle_layer_time(cases, 0.02, threads)                     # warm-up, builds the C library
    t_probe, b_probe = oracle_layer_time(cases, 0.05, threads)
    frac = min(1.0, max(0.05, 0.05 * (budget_s / 3.0) / max(t_probe, 1e-6)))
    best = None
    spent = 0.0
    reps = 0
    while reps < 3 or (spent < budget_s and reps < 20):
        t, b = oracle_layer_time(cases, frac, threads)
        spent += t
        reps += 1
        gbs = b / t / 1e9
        best = gbs if best is None else max(best, gbs)
    return {"value": best, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "first %.0f%% of the rows of each of the 7 matrices, best of %d passes, %.1f s of wall time"
                      % (100 * frac, reps, spent)}


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return 0
    from oracle.c_oracle import max_threads
    cases = make_cases()
    threads = max_threads()
    oracle_layer_time(cases, 0.01, threads)
    t_probe, _ = oracle_layer_time(cases, 0.05, threads)
    budget = 150.0 / max(1, args.steps + args.warmup)
    frac = min(1.0, max(0.002, 0.05 * budget / max(t_probe, 1e-6)))
    for _ in range(args.warmup):
        oracle_layer_time(cases, frac, threads)
    total_t, total_b = 0.0, 0
    for _ in range(args.steps):
        t, b = oracle_layer_time(cases, frac, threads)
        total_t += t
        total_b += b
    gbs = total_b / total_t / 1e9
    sample = "each step: first %.2f%% of the rows of each of the 7 matrices" % (100 * frac)
    line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": sample},
            "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------- GPU arm
def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2509_16989_b200 import binding, build

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    build.build()
    binding.lib()

    def dev(a):
        return torch.from_numpy(np.ascontiguousarray(a)).to(device)

    cases = make_cases()
    stream = torch.cuda.Stream(device=device)
    R = args.sets

    # set 0 is packed from the seeded planes; the other sets are byte copies at distinct addresses
    base = {}
    for u, c in cases.items():
        packed, st = binding.ptqtp_pack(dev(c["T1"]), dev(c["T2"]), dev(c["alpha1"]), dev(c["alpha2"]))
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        base[u] = packed
    sets = []
    for r in range(R):
        sets.append({m: (base[UNIQUE_OF[m]] if (r == 0 and m in ("q", "k", "gate", "down"))
                         else base[UNIQUE_OF[m]].clone()) for m in MATRICES})
    xs = {m: dev(cases[UNIQUE_OF[m]]["x"]) for m in MATRICES}
    ys = {m: torch.empty(LLAMA3_8B[m][0], dtype=torch.float16, device=device) for m in MATRICES}
    torch.cuda.synchronize()

    def step(r):
        for m in MATRICES:
            N, K = LLAMA3_8B[m]
            binding.ptqtp_gemv(sets[r][m], N, K, xs[m], y=ys[m], stream=stream)

    # warm every buffer once outside any capture, then capture the steps as CUDA graphs
    for r in range(R):
        step(r)
    stream.synchronize()
    graphs = None
    big = None
    huge = None
    if not args.no_graph:
        graphs = []
        for r in range(R):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                step(r)
            graphs.append(g)
        big = torch.cuda.CUDAGraph()
        with torch.cuda.graph(big, stream=stream):
            for r in range(R):
                step(r)
        # eight rotations in one graph: a graph boundary drains the chain of overlapping launches
        huge = torch.cuda.CUDAGraph()
        with torch.cuda.graph(huge, stream=stream):
            for _ in range(8):
                for r in range(R):
                    step(r)
        # first replays upload the graphs to the device: part of the set-up, like packing the matrices
        with torch.cuda.stream(stream):
            for g in graphs + [big, huge]:
                g.replay()
        stream.synchronize()

    def run_steps(k, start=0):
        with torch.cuda.stream(stream):
            i = 0
            if graphs is None:
                while i < k:
                    step((start + i) % R)
                    i += 1
                return
            while i < k and (start + i) % R != 0:
                graphs[(start + i) % R].replay()
                i += 1
            while k - i >= 8 * R:
                huge.replay()
                i += 8 * R
            while k - i >= R:
                big.replay()
                i += R
            while i < k:
                graphs[(start + i) % R].replay()
                i += 1

    def barrier():
        if world > 1:
            dist.barrier()

    sampler = ClockSampler(local)
    sampler.start()

    run_steps(max(args.warmup, 3))
    stream.synchronize()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    t_begin = time.perf_counter()
    e0.record(stream)
    run_steps(args.steps)
    e1.record(stream)
    sampler.sample_now()                                 # the GPU is still working on the enqueued steps
    stream.synchronize()
    torch.cuda.synchronize()
    t_end = time.perf_counter()
    barrier()
    ms = max_over_ranks(e0.elapsed_time(e1), world, device)
    clocks = sampler.summary(t_begin, t_end)
    ms_per_step = ms / args.steps
    value = job_throughput_gbs(ms_per_step, world)

    # ---- parity spot check of what was just timed (sampled rows, fp64 oracle) ----
    parity = None
    if rank == 0:
        from oracle.c_oracle import layer_fp64_c, max_threads
        from oracle.layer import parity_metrics
        step(0)
        stream.synchronize()
        worst_rel, worst_frac = 0.0, 0.0
        for m in ("q", "k", "gate", "down"):
            c = cases[UNIQUE_OF[m]]
            rows = np.unique(np.random.default_rng(1).integers(0, c["N"], 512))
            ref = layer_fp64_c(c["T1"][rows], c["T2"][rows], c["alpha1"][rows], c["alpha2"][rows], c["x"],
                               threads=max_threads())
            got = ys[m].cpu().numpy()[rows]
            rel, mab, bound = parity_metrics(got, ref, c["x"])[0]
            worst_rel = max(worst_rel, rel)
            worst_frac = max(worst_frac, mab / bound)
        parity = {"rel_l2_max": worst_rel, "max_abs_over_bound": worst_frac,
                  "ok": bool(worst_rel <= 1e-3 and worst_frac <= 1.0), "rows_sampled_per_matrix": 512}

    # ---- end to end: host x in pinned memory -> H2D, GEMV, D2H of y, one sync per step ----
    e2e_steps = min(args.steps, 2000)
    xh = {m: torch.from_numpy(cases[UNIQUE_OF[m]]["x"].copy()).pin_memory() for m in MATRICES}
    yh = {m: torch.empty(LLAMA3_8B[m][0], dtype=torch.float16).pin_memory() for m in MATRICES}

    def e2e_calls(r):
        for m in MATRICES:
            N, K = LLAMA3_8B[m]
            binding.ptqtp_gemv_host(sets[r][m], N, K, xh[m], yh[m], xs[m], ys[m], stream=stream)

    # the host-buffer calls of a step are captured once per layer copy, like the device-resident steps
    e2e_graphs = None
    if not args.no_graph:
        with torch.cuda.stream(stream):
            e2e_calls(0)
            stream.synchronize()
            e2e_graphs = []
            for r in range(R):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    e2e_calls(r)
                e2e_graphs.append(g)

    def e2e_step(r):
        with torch.cuda.stream(stream):
            if e2e_graphs is None:
                e2e_calls(r)
            else:
                e2e_graphs[r].replay()
        stream.synchronize()

    for i in range(3):
        e2e_step(i % R)
    barrier()
    torch.cuda.synchronize()
    e0.record(stream)
    for i in range(e2e_steps):
        e2e_step(i % R)
    e1.record(stream)
    stream.synchronize()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, device)
    e2e_value = job_throughput_gbs(e2e_ms / e2e_steps, world)
    h2d = sum(2 * LLAMA3_8B[m][1] for m in MATRICES)
    d2h = sum(2 * LLAMA3_8B[m][0] for m in MATRICES)

    # ---- per-shape detail: steady state over rotating buffers > 2x L2, and isolated cold calls ----
    detail = {}
    if rank == 0 and not args.no_detail:
        l2 = torch.cuda.get_device_properties(device).L2_cache_size
        flush = torch.empty(max(2 * l2, 256 << 20), dtype=torch.uint8, device=device)
        for u, (N, K) in sorted(LLAMA3_8B_UNIQUE.items()):
            nbuf = max(4, -(-(2 * l2 + (64 << 20)) // base[u].numel()))
            bufs = [base[u]] + [base[u].clone() for _ in range(nbuf - 1)]
            x = xs["down" if u == "down" else "q"]
            y = torch.empty(N, dtype=torch.float16, device=device)
            with torch.cuda.stream(stream):
                for b in bufs[:2]:
                    binding.ptqtp_gemv(b, N, K, x, y=y, stream=stream)
                stream.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    for b in bufs:
                        binding.ptqtp_gemv(b, N, K, x, y=y, stream=stream)
                reps = max(3, int(2000 / nbuf))
                g.replay()
                stream.synchronize()
                e0.record(stream)
                for _ in range(reps):
                    g.replay()
                e1.record(stream)
                stream.synchronize()
                us = 1e3 * e0.elapsed_time(e1) / (reps * nbuf)
                iso = []
                for i in range(12):
                    flush.fill_(i)
                    e0.record(stream)
                    binding.ptqtp_gemv(bufs[i % nbuf], N, K, x, y=y, stream=stream)
                    e1.record(stream)
                    stream.synchronize()
                    iso.append(1e3 * e0.elapsed_time(e1))
            nb = algorithmic_bytes(N, K)
            detail[u] = {"N": N, "K": K, "bytes": nb, "us_steady": us, "gbs_steady": nb / us / 1e3,
                         "us_isolated_median": float(np.median(iso)), "buffers": nbuf}
            del bufs
        del flush
        # the same step without any overlap of consecutive launches (plain launches, no speculative execution)
        if graphs is not None:
            old_level = binding.ptqtp_set_overlap(0)
            try:
                with torch.cuda.stream(stream):
                    step(0)
                    stream.synchronize()
                    plain = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(plain, stream=stream):
                        for r in range(R):
                            step(r)
                    plain.replay()
                    stream.synchronize()
                    e0.record(stream)
                    for _ in range(20):
                        plain.replay()
                    e1.record(stream)
                    stream.synchronize()
                detail["step_without_overlap"] = {"us_per_layer": 1e3 * e0.elapsed_time(e1) / (20 * R),
                                                  "what": "ptqtp_set_overlap(0): every launch waits for the one before it"}
                del plain
            finally:
                binding.ptqtp_set_overlap(old_level)

    sampler.stop()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    peak, peak_kind = measured_peak()
    launches = 7 * args.steps
    achieved = STEP_BYTES / (ms_per_step * 1e-3) / 1e9       # per GPU: bytes of a launch / its mean duration
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "l2": "inputs larger than L2: steps rotate over %d layer copies (%d MB)"
                   % (R, R * STEP_WEIGHT_BYTES >> 20), "launch": "cuda graph" if graphs else "plain launches",
                   "parallelism": "replicas only" if world > 1 else "1 gpu", "bytes_per_step": STEP_BYTES,
                   "overlap": "library default (ptqtp_set_overlap level 2): programmatic dependent launch with "
                              "speculative execution; the CTAs of consecutive launches share SMs"},
        "us_per_layer": 1e3 * ms_per_step,
        "weight_gbs": STEP_WEIGHT_BYTES / (ms_per_step * 1e-3) / 1e9,
        "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": "of " + peak_kind,
                     "traffic": None if DRAM_TRAFFIC_RATIO is None else DRAM_TRAFFIC_RATIO * STEP_BYTES / 7.0,
                     "kernel": "gemv2_kernel (7 launches per step; mean over the step)",
                     "bytes_per_launch_mean": STEP_BYTES / 7.0, "us_per_launch_mean": 1e3 * ms_per_step / 7.0},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "us_per_layer": 1e3 * e2e_ms / e2e_steps,
                "launch": ("cuda graph of the 7 ptqtp_gemv_host calls" if e2e_graphs else "plain calls")
                          + ", one stream synchronisation per step"},
        "gpu_launches": launches, "clocks": clocks, "parity": parity, "shapes": detail,
    }
    if world == 1 and not args.no_cpu:
        line["cpu_baseline"] = cpu_baseline(cases)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=100)
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--sets", type=int, default=8, help="distinct layer copies the steps rotate over")
    ap.add_argument("--no-graph", action="store_true", help="plain launches instead of CUDA graphs")
    ap.add_argument("--no-detail", action="store_true", help="skip the per-shape measurements")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    args = ap.parse_args()
    if args.steps < 1:
        ap.error("--steps must be >= 1")
    if args.impl == "reference":
        return run_reference(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
