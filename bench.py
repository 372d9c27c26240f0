"""Benchmark of the dual-trit-plane decode linears on B200.

One step = one pass of the hot path over the seven decode linears of a LLaMA-3-8B layer at
batch 1 (q, k, v, o, gate, up, down), one ptqtp_gemv call per matrix, on packed planes that are
already resident in HBM.  Steps rotate over `--sets` distinct copies of the layer (default 8,
928 MB) so that every packed byte comes from HBM, not from L2.  The timed steps are one CUDA graph
(up to 512 steps per graph), so a run of 20 steps has no graph boundary inside it.

The library's default is plain launches; this program opts in to overlap level 2 (programmatic
dependent launch with speculative execution) as a decoder would whose packed blobs never change while
GEMV calls are in flight, and says so in `config.overlap`.

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
# dram__bytes_read.sum + dram__bytes_write.sum per launch in the ncu captures of the current batch-1 kernel, one
# launch per shape (profiles/gemv4_llama3_8b_shapes.md, profiles/gemv2_gate_up_14336x4096.md); None where no capture
# of the current kernel exists
DRAM_TRAFFIC_BYTES = {3: {"qo": 8958720.0, "kv": 2274048.0, "gate_up": 31241216.0, "down": 31261440.0},
                      2: {"qo": None, "kv": None, "gate_up": 31239424.0, "down": None}}
KERNEL_NAME = {2: "gemv2_kernel", 3: "gemv4_kernel"}
DTYPE = {2: "int16 block-fixed-point x int2 codes -> int32 (dp4a), f32 scale epilogue",
         3: "int15 block-fixed-point x int2 codes -> int32 (int8 mma), f32 scale epilogue"}
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
GRAPH_STEPS = 512            # steps per CUDA graph of the timed run (a 20-step run is one graph)


class Chain:
    """CUDA-graph timing of a list of launch functions on one stream."""

    def __init__(self, torch, stream):
        self.torch, self.stream = torch, stream
        self.e0 = torch.cuda.Event(enable_timing=True)
        self.e1 = torch.cuda.Event(enable_timing=True)

    def capture(self, fn):
        torch, st = self.torch, self.stream
        with torch.cuda.stream(st):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=st):
                fn()
            g.replay()                                   # the first replay uploads the graph: part of the set-up
            st.synchronize()
        return g

    def time_ms(self, graphs):
        """Replays the graphs back to back once; device time in ms."""
        torch, st = self.torch, self.stream
        with torch.cuda.stream(st):
            self.e0.record(st)
            for g in graphs:
                g.replay()
            self.e1.record(st)
            st.synchronize()
        return self.e0.elapsed_time(self.e1)


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
    fmt = args.format
    # the decode case: packed blobs are immutable while GEMV calls are in flight, so the opt-in overlap applies
    binding.ptqtp_set_overlap(2)

    def dev(a):
        return torch.from_numpy(np.ascontiguousarray(a)).to(device)

    cases = make_cases()
    stream = torch.cuda.Stream(device=device)
    chain = Chain(torch, stream)
    R = args.sets

    def pack_all(f):
        out = {}
        for u, c in cases.items():
            packed, st = binding.ptqtp_pack(dev(c["T1"]), dev(c["T2"]), dev(c["alpha1"]), dev(c["alpha2"]), fmt=f)
            torch.cuda.synchronize()
            assert int(st.item()) == 0
            out[u] = packed
        return out

    # set 0 is packed from the seeded planes; the other sets are byte copies at distinct addresses
    base = pack_all(fmt)
    sets = []
    for r in range(R):
        sets.append({m: (base[UNIQUE_OF[m]] if (r == 0 and m in ("q", "k", "gate", "down"))
                         else base[UNIQUE_OF[m]].clone()) for m in MATRICES})
    xs = {m: dev(cases[UNIQUE_OF[m]]["x"]) for m in MATRICES}
    ys = {m: torch.empty(LLAMA3_8B[m][0], dtype=torch.float16, device=device) for m in MATRICES}
    torch.cuda.synchronize()

    def step(r, f=fmt, layer_sets=None):
        for m in MATRICES:
            N, K = LLAMA3_8B[m]
            binding.ptqtp_gemv((layer_sets or sets)[r][m], N, K, xs[m], y=ys[m], stream=stream, fmt=f)

    def steps_fn(k, start=0, **kw):
        def fn():
            for i in range(k):
                step((start + i) % R, **kw)
        return fn

    # warm every buffer once outside any capture, then capture the timed steps
    with torch.cuda.stream(stream):
        steps_fn(R)()
    stream.synchronize()
    timed_graphs, warm_graphs = None, None
    if not args.no_graph:
        per = min(args.steps, GRAPH_STEPS)
        full = chain.capture(steps_fn(per))
        timed_graphs = [full] * (args.steps // per)
        if args.steps % per:
            timed_graphs.append(chain.capture(steps_fn(args.steps % per, start=(args.steps // per) * per)))
        nwarm = max(args.warmup, 3)
        warm_graphs = [chain.capture(steps_fn(min(nwarm, GRAPH_STEPS)))] * -(-nwarm // GRAPH_STEPS)

    def barrier():
        if world > 1:
            dist.barrier()

    sampler = ClockSampler(local)
    sampler.start()

    if timed_graphs is None:
        with torch.cuda.stream(stream):
            steps_fn(max(args.warmup, 3))()
    else:
        chain.time_ms(warm_graphs)
    stream.synchronize()
    barrier()
    torch.cuda.synchronize()
    t_begin = time.perf_counter()
    if timed_graphs is None:
        with torch.cuda.stream(stream):
            chain.e0.record(stream)
            steps_fn(args.steps)()
            chain.e1.record(stream)
            sampler.sample_now()
            stream.synchronize()
        ms_local = chain.e0.elapsed_time(chain.e1)
    else:
        with torch.cuda.stream(stream):
            chain.e0.record(stream)
            for g in timed_graphs:
                g.replay()
            chain.e1.record(stream)
            sampler.sample_now()                         # the GPU is still working on the enqueued steps
            stream.synchronize()
        ms_local = chain.e0.elapsed_time(chain.e1)
    torch.cuda.synchronize()
    t_end = time.perf_counter()
    barrier()
    ms = max_over_ranks(ms_local, world, device)
    ms_per_step = ms / args.steps
    value = job_throughput_gbs(ms_per_step, world)
    # a short timed region ends before the sampler thread's next turn: keep the GPU under the same load a little
    # longer so that the clocks are seen under load (not part of the timed region)
    extended = False
    if timed_graphs is not None and ms < 200.0:
        t_load = time.perf_counter()
        while time.perf_counter() - t_load < 0.25:
            chain.time_ms(timed_graphs[:1])
        t_end = time.perf_counter()
        extended = True
    clocks = sampler.summary(t_begin, t_end)
    if extended and clocks["window"] == "timed region":
        clocks["window"] = "timed region plus 0.25 s of replays of the same graph directly after it"

    # ---- parity spot check of what was just timed (sampled rows, fp64 oracle) ----
    parity = None
    if rank == 0:
        from oracle.c_oracle import layer_fp64_c, max_threads
        from oracle.layer import parity_metrics
        with torch.cuda.stream(stream):
            step(0)
        stream.synchronize()
        worst_rel, worst_frac = 0.0, 0.0
        refs = {}
        for m in ("q", "k", "gate", "down"):
            c = cases[UNIQUE_OF[m]]
            rows = np.unique(np.random.default_rng(1).integers(0, c["N"], 512))
            ref = layer_fp64_c(c["T1"][rows], c["T2"][rows], c["alpha1"][rows], c["alpha2"][rows], c["x"],
                               threads=max_threads())
            refs[m] = (rows, ref, c["x"])
            got = ys[m].cpu().numpy()[rows]
            rel, mab, bound = parity_metrics(got, ref, c["x"])[0]
            worst_rel = max(worst_rel, rel)
            worst_frac = max(worst_frac, mab / bound)
        parity = {"rel_l2_max": worst_rel, "max_abs_over_bound": worst_frac,
                  "ok": bool(worst_rel <= 1e-3 and worst_frac <= 1.0), "rows_sampled_per_matrix": 512}

    # ---- end to end: host x in pinned memory -> H2D, GEMV, y into pinned host memory, one sync per step ----
    e2e_steps = min(args.steps, 2000)
    xh = {m: torch.from_numpy(cases[UNIQUE_OF[m]]["x"].copy()).pin_memory() for m in MATRICES}
    yh = {m: torch.empty(LLAMA3_8B[m][0], dtype=torch.float16).pin_memory() for m in MATRICES}

    # the seven calls of a step are independent of one another (own x, own y): each runs on a stream of its own, forked
    # from and joined to the step's stream, so their copies and kernels overlap
    side = [torch.cuda.Stream(device=device) for _ in MATRICES]

    def e2e_calls(r):
        fork = torch.cuda.Event()
        fork.record(stream)
        for s_m, m in zip(side, MATRICES):
            N, K = LLAMA3_8B[m]
            s_m.wait_event(fork)
            binding.ptqtp_gemv_host(sets[r][m], N, K, xh[m], yh[m], xs[m], ys[m], stream=s_m, fmt=fmt)
            join = torch.cuda.Event()
            join.record(s_m)
            stream.wait_event(join)

    # the host-buffer calls of a step are captured once per layer copy, like the device-resident steps
    e2e_graphs = None
    if not args.no_graph:
        with torch.cuda.stream(stream):
            e2e_calls(0)
            stream.synchronize()
        e2e_graphs = [chain.capture(lambda r=r: e2e_calls(r)) for r in range(R)]

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
    chain.e0.record(stream)
    for i in range(e2e_steps):
        e2e_step(i % R)
    chain.e1.record(stream)
    stream.synchronize()
    e2e_ms = max_over_ranks(chain.e0.elapsed_time(chain.e1), world, device)
    e2e_value = job_throughput_gbs(e2e_ms / e2e_steps, world)
    h2d = sum(2 * LLAMA3_8B[m][1] for m in MATRICES)
    d2h = sum(2 * LLAMA3_8B[m][0] for m in MATRICES)
    # what the host-buffer calls left in pinned memory, against the same oracle rows
    e2e_parity_ok = None
    if rank == 0:
        e2e_parity_ok = True
        for m, (rows, ref, x) in refs.items():
            rel, mab, bound = parity_metrics(yh[m].numpy()[rows], ref, x)[0]
            e2e_parity_ok = bool(e2e_parity_ok and rel <= 1e-3 and mab <= bound)

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

            def calls():
                for b in bufs:
                    binding.ptqtp_gemv(b, N, K, x, y=y, stream=stream, fmt=fmt)

            with torch.cuda.stream(stream):
                calls()
                stream.synchronize()
            g = chain.capture(calls)
            reps = max(3, int(2000 / nbuf))
            us = 1e3 * chain.time_ms([g] * reps) / (reps * nbuf)
            iso = []
            with torch.cuda.stream(stream):
                for i in range(12):
                    flush.fill_(i)
                    chain.e0.record(stream)
                    binding.ptqtp_gemv(bufs[i % nbuf], N, K, x, y=y, stream=stream, fmt=fmt)
                    chain.e1.record(stream)
                    stream.synchronize()
                    iso.append(1e3 * chain.e0.elapsed_time(chain.e1))
                iso_whole = []                           # the same lone call with the whole-SM launch configuration
                for i in range(12):
                    flush.fill_(i)
                    chain.e0.record(stream)
                    binding.ptqtp_gemv_cfg(bufs[i % nbuf], N, K, x, y=y, k_split=-1, stream=stream, fmt=fmt)
                    chain.e1.record(stream)
                    stream.synchronize()
                    iso_whole.append(1e3 * chain.e0.elapsed_time(chain.e1))
            nb = algorithmic_bytes(N, K)
            detail[u] = {"N": N, "K": K, "bytes": nb, "us_steady": us, "gbs_steady": nb / us / 1e3,
                         "us_isolated_median": float(np.median(iso)),
                         "us_isolated_whole_sm_median": float(np.median(iso_whole)), "buffers": nbuf}
            del bufs, g
        del flush
        detail["step_isolated_sum"] = {
            "us_per_layer": sum(detail[UNIQUE_OF[m]]["us_isolated_median"] for m in MATRICES),
            "what": "sum over the 7 matrices of the isolated, cold-L2, event-timed single calls above"}
        if not args.no_graph:
            # The layer as a decoder issues it: every call's x is written on the stream directly before it is used.
            #   x_q = f(y_down of the layer before); x_k = x_v = x_q; x_o = f(y_q); x_gate = x_up = f(y_o);
            #   x_down = y_gate * y_up   (f = one elementwise kernel, standing in for attention / norms)
            # 7 GEMV calls + 4 elementwise kernels per layer.  k, v and up start early under their speculative pass; a
            # call behind an elementwise kernel starts when that kernel has finished (it releases its dependents only
            # at its end), so q, o, gate and down run alone on the GPU.
            xd = {"a": torch.zeros(4096, dtype=torch.float16, device=device),
                  "o": torch.zeros(4096, dtype=torch.float16, device=device),
                  "m": torch.zeros(4096, dtype=torch.float16, device=device),
                  "d": torch.zeros(14336, dtype=torch.float16, device=device)}
            ys["down"].zero_()

            def dep_layer(r):
                g4 = lambda m, x: binding.ptqtp_gemv(sets[r][m], *LLAMA3_8B[m], x, y=ys[m], stream=stream, fmt=fmt)
                torch.add(ys["down"], 0.5, out=xd["a"])
                g4("q", xd["a"]); g4("k", xd["a"]); g4("v", xd["a"])
                torch.add(ys["q"], 0.25, out=xd["o"])
                g4("o", xd["o"])
                torch.add(ys["o"], 0.125, out=xd["m"])
                g4("gate", xd["m"]); g4("up", xd["m"])
                torch.mul(ys["gate"], ys["up"], out=xd["d"])
                g4("down", xd["d"])

            def dep_steps():
                for i in range(4 * R):
                    dep_layer(i % R)

            with torch.cuda.stream(stream):
                dep_layer(0)
                stream.synchronize()
            gd = chain.capture(dep_steps)
            detail["step_dependent"] = {
                "us_per_layer": 1e3 * chain.time_ms([gd] * 10) / (10 * 4 * R),
                "what": "7 ptqtp_gemv + 4 elementwise kernels per layer; every x is produced on the stream directly "
                        "before its first use (q, o, gate, down start only when the elementwise kernel ahead of them has ended)"}
            for lvl in (1, 0):
                old_level = binding.ptqtp_set_overlap(lvl)
                try:
                    with torch.cuda.stream(stream):
                        dep_layer(0)
                        stream.synchronize()
                    gd1 = chain.capture(dep_steps)
                    detail["step_dependent"]["us_per_layer_level%d" % lvl] = 1e3 * chain.time_ms([gd1] * 10) / (10 * 4 * R)
                    del gd1
                finally:
                    binding.ptqtp_set_overlap(old_level)
            del gd
            # Four launches per layer (format 3): q, k, v in one launch and gate, up with the gated pair epilogue in
            # one launch (ptqtp_gemv_multi over the separately packed blobs), o and down as before.  First with
            # independent activations like the headline step, then as a decoder issues it: down reads the gated
            # output directly, the other activations come from one elementwise kernel each.
            if fmt == 3:
                yg = torch.zeros(14336, dtype=torch.float16, device=device)

                def four(r, dep):
                    S_ = sets[r]
                    if dep:
                        torch.add(ys["down"], 0.5, out=xd["a"])
                    binding.ptqtp_gemv_multi([S_["q"], S_["k"], S_["v"]], [4096, 1024, 1024], 4096, xd["a"] if dep else xs["q"],
                                             ys=[ys["q"], ys["k"], ys["v"]], stream=stream)
                    if dep:
                        torch.add(ys["q"], 0.25, out=xd["o"])
                    binding.ptqtp_gemv(S_["o"], 4096, 4096, xd["o"] if dep else xs["o"], y=ys["o"], stream=stream, fmt=3)
                    if dep:
                        torch.add(ys["o"], 0.125, out=xd["m"])
                    binding.ptqtp_gemv_multi([S_["gate"], S_["up"]], [14336, 14336], 4096, xd["m"] if dep else xs["gate"],
                                             ys=[yg], epilogue=binding.EPILOGUE_GATED_PAIR, stream=stream)
                    binding.ptqtp_gemv(S_["down"], 4096, 14336, yg if dep else xs["down"], y=ys["down"], stream=stream, fmt=3)

                four_bytes = STEP_BYTES - 2 * 2 * 4096 - 2 * 4096 - 2 * 14336      # x of k, v, up and one y not moved
                for dep, key in ((False, "four_launch_layer"), (True, "four_launch_layer_dependent")):
                    with torch.cuda.stream(stream):
                        four(0, dep)
                        stream.synchronize()
                    g4l = chain.capture(lambda dep=dep: [four(i % R, dep) for i in range(4 * R)])
                    us4 = 1e3 * chain.time_ms([g4l] * 10) / (10 * 4 * R)
                    detail[key] = {"us_per_layer": us4, "gbs": four_bytes / us4 / 1e3, "bytes": four_bytes,
                                   "launches": "ptqtp_gemv_multi(q,k,v) + ptqtp_gemv(o) + ptqtp_gemv_multi(gate,up; gated pair) "
                                               "+ ptqtp_gemv(down)" + (" + 3 elementwise kernels; down reads the gated output" if dep else "")}
                    del g4l
            # the same independent step without any overlap of consecutive launches: the library default
            old_level = binding.ptqtp_set_overlap(0)
            try:
                with torch.cuda.stream(stream):
                    step(0)
                    stream.synchronize()
                plain = chain.capture(steps_fn(R))
                detail["step_without_overlap"] = {
                    "us_per_layer": 1e3 * chain.time_ms([plain] * 20) / (20 * R),
                    "what": "ptqtp_set_overlap(0), the library default: plain launches, every call waits for the one before it"}
                del plain
            finally:
                binding.ptqtp_set_overlap(old_level)
            # the other batch-1 kernel (CUDA cores: masks + integer dot products on format 2) on the same step
            other = 2 if fmt == 3 else 3
            base_o = pack_all(other)
            sets_o = [{m: base_o[UNIQUE_OF[m]].clone() for m in MATRICES} for _ in range(R)]
            with torch.cuda.stream(stream):
                steps_fn(R, f=other, layer_sets=sets_o)()
                stream.synchronize()
            go = chain.capture(steps_fn(4 * R, f=other, layer_sets=sets_o))
            detail["step_other_format"] = {"format": other, "kernel": KERNEL_NAME[other],
                                           "us_per_layer": 1e3 * chain.time_ms([go] * 10) / (10 * 4 * R)}
            del go, sets_o, base_o
            # the small-batch call on the gate/up shape (format 3: warp MMAs for few rows, the tcgen05 kernel for many)
            if fmt == 3:
                Ng, Kg = LLAMA3_8B["gate"]
                small = {}
                for M in (2, 16, 64):
                    Xb = torch.randn((M, Kg), generator=torch.Generator(device=device).manual_seed(M), device=device,
                                     dtype=torch.float32).to(torch.float16)
                    Yb = torch.empty((M, Ng), dtype=torch.float16, device=device)
                    call = lambda: [binding.ptqtp_gemm_skinny(sets[r]["gate"], Ng, Kg, Xb, Y=Yb, stream=stream, fmt=3)
                                    for r in range(R)]
                    with torch.cuda.stream(stream):
                        call()
                        stream.synchronize()
                    gb = chain.capture(lambda: [call() for _ in range(4)])
                    small["M%d_us" % M] = 1e3 * chain.time_ms([gb] * 10) / (10 * 4 * R)
                    del gb
                detail["small_batch_gate_14336x4096"] = small

    sampler.stop()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    peak, peak_kind = measured_peak()
    launches = 7 * args.steps
    achieved = STEP_BYTES / (ms_per_step * 1e-3) / 1e9       # per GPU: bytes of a launch / its mean duration
    traffic = [DRAM_TRAFFIC_BYTES[fmt][UNIQUE_OF[m]] for m in MATRICES]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": DTYPE[fmt], "data": "synthetic",
        "config": {"workload": WORKLOAD, "l2": "inputs larger than L2: steps rotate over %d layer copies (%d MB)"
                   % (R, R * STEP_WEIGHT_BYTES >> 20),
                   "launch": ("one cuda graph per %d steps" % min(args.steps, GRAPH_STEPS)) if timed_graphs else "plain launches",
                   "parallelism": "replicas only" if world > 1 else "1 gpu", "bytes_per_step": STEP_BYTES,
                   "packed_format": fmt,
                   "overlap": "opt-in ptqtp_set_overlap(2): programmatic dependent launch with speculative execution "
                              "(packed blobs are immutable during the run); the library default is plain launches, see "
                              "shapes.step_without_overlap"},
        "us_per_layer": 1e3 * ms_per_step,
        "weight_gbs": STEP_WEIGHT_BYTES / (ms_per_step * 1e-3) / 1e9,
        "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": "of " + peak_kind,
                     "traffic": None if any(t is None for t in traffic) else sum(traffic) / 7.0,
                     "kernel": "%s (7 launches per step; mean over the step)" % KERNEL_NAME[fmt],
                     "bytes_per_launch_mean": STEP_BYTES / 7.0, "us_per_launch_mean": 1e3 * ms_per_step / 7.0},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "us_per_layer": 1e3 * e2e_ms / e2e_steps, "parity_ok": e2e_parity_ok,
                "launch": ("cuda graph of the 7 ptqtp_gemv_host calls, each on a stream of its own forked from the step's stream"
                           if e2e_graphs else "plain calls, each on a stream of its own forked from the step's stream")
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
    ap.add_argument("--format", type=int, default=3, choices=(2, 3),
                    help="packed format of the timed step: 3 = tiles in int8 MMA operand order, 2 = CUDA-core kernel")
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
