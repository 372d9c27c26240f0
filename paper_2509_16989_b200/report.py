"""Measurements of the workloads other than the benchmark's headline step (run on a B200).

    python -m paper_2509_16989_b200.report [--only 0,2,3] [--format 3]

Batch-1 calls use the packed format given by --format (default 3: tiles in int8 MMA operand order; 2: the
CUDA-core kernel); the small-batch calls (M > 1) use format 2 unless a line says format 3.  The program opts in to overlap level 2, as
a decoder would whose packed blobs never change while GEMV calls are in flight.

  0  Qwen3-0.6B up_proj 3072 x 1024, batch 1
  2  batch sweep M in {1,...,64} of ptqtp_gemm_skinny on the 14336 x 4096 gate/up shape (and ptqtp_gemv at M = 1) on
     format 2, then M in {2,...,64} on format 3 for the four distinct LLaMA-3-8B shapes
  3  LLaMA-3-70B shapes, planes with P(0) = 0.5, batch 1 and 8
  5  a LLaMA-3-8B layer with stacked matrices: q, k, v packed as one 6144 x 4096 matrix, and also gate, up as one
     28672 x 4096 matrix (rows are independent, so a caller may stack matrices that share their input and
     slice y): five or four calls per layer instead of seven
  6  the seven linears of a LLaMA-3-70B-shaped layer as one chain of calls
  4  the 32-layer stack of LLaMA-3-8B-shaped linears from decomposed weights: W ~ N(0, 0.02^2) with 0.1 % of the
     entries times 20, drawn on the device, 224 distinct matrices decomposed by ptqtp_decompose and packed; one decode
     step = 224 calls in one CUDA graph; reports the time per token, the decomposition time and the reconstruction
     error ||W - (alpha1 T1 + alpha2 T2)||_F / ||W||_F per matrix type (tests/test_gpu_stack.py checks parity of
     such a stack against the CPU oracle)

Every timing is a CUDA-event steady state inside a CUDA graph that walks over distinct packed buffers
totalling more than twice the L2 size, so the planes come from HBM.  One JSON line per result.
"""
import argparse
import json
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2509_16989_b200 import binding  # noqa: E402
from paper_2509_16989_b200.inputs import LLAMA3_8B, LLAMA3_70B, QWEN3_0P6B_UP, make_case, make_weights_device  # noqa: E402

FMT = binding.FORMAT_V3          # packed format of the batch-1 calls (--format)


def algorithmic_bytes(N, K, M=1):
    return N * K // 2 + 4 * N * K // 128 + 2 * M * K + 2 * M * N


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


class Timer:
    def __init__(self):
        self.stream = torch.cuda.Stream()
        self.e0 = torch.cuda.Event(enable_timing=True)
        self.e1 = torch.cuda.Event(enable_timing=True)
        self.l2 = torch.cuda.get_device_properties(0).L2_cache_size

    def copies(self, packed):
        n = max(3, -(-(2 * self.l2 + (64 << 20)) // packed.numel()))
        return [packed] + [packed.clone() for _ in range(n - 1)]

    def steady_us(self, calls, reps=None):
        """calls: list of zero-argument functions launching on self.stream; returns us per call."""
        st = self.stream
        with torch.cuda.stream(st):
            calls[0]()
            st.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=st):
                for c in calls:
                    c()
            g.replay()
            st.synchronize()
            reps = reps or max(3, 1500 // len(calls))
            self.e0.record(st)
            for _ in range(reps):
                g.replay()
            self.e1.record(st)
            st.synchronize()
        return 1e3 * self.e0.elapsed_time(self.e1) / (reps * len(calls))


def emit(**kw):
    print(json.dumps(kw))
    sys.stdout.flush()


def gemv_case(T, name, N, K, p_zero=0.4, seed=0, batches=(1,)):
    c = make_case(N, K, seed=seed, M=max(batches), p_zero=p_zero)
    Xall = dev(np.atleast_2d(c["x"]))
    packed, bufs = None, None
    for M in batches:
        want = FMT if M == 1 else binding.FORMAT_V2
        if packed is None or want != have:
            del packed, bufs
            torch.cuda.empty_cache()
            packed, st = binding.ptqtp_pack(dev(c["T1"]), dev(c["T2"]), dev(c["alpha1"]), dev(c["alpha2"]), fmt=want)
            bufs = T.copies(packed)
            have = want
        if M == 1:
            x = Xall[0].contiguous()
            y = torch.empty(N, dtype=torch.float16, device="cuda")
            us = T.steady_us([lambda b=b: binding.ptqtp_gemv(b, N, K, x, y=y, stream=T.stream, fmt=FMT) for b in bufs])
            call = "ptqtp_gemv (format %d)" % FMT
        else:
            X = Xall[:M].contiguous()
            Y = torch.empty((M, N), dtype=torch.float16, device="cuda")
            us = T.steady_us([lambda b=b: binding.ptqtp_gemm_skinny(b, N, K, X, Y=Y, stream=T.stream) for b in bufs])
            call = "ptqtp_gemm_skinny"
            ws = torch.empty(binding.gemm_skinny_workspace_size(N, K, M), dtype=torch.uint8, device="cuda")
            us_ws = T.steady_us([lambda b=b: binding.ptqtp_gemm_skinny_ws(b, N, K, X, Y=Y, workspace=ws, stream=T.stream)
                                 for b in bufs])
            nb = algorithmic_bytes(N, K, M)
            emit(workload=name, call="ptqtp_gemm_skinny_ws", N=N, K=K, M=M, p_zero=p_zero, us=round(us_ws, 3),
                 gbs=round(nb / us_ws / 1e3, 1), bytes=nb, buffers=len(bufs))
        nb = algorithmic_bytes(N, K, M)
        emit(workload=name, call=call, N=N, K=K, M=M, p_zero=p_zero, us=round(us, 3), gbs=round(nb / us / 1e3, 1),
             bytes=nb, buffers=len(bufs))
    return packed


def config0(T):
    N, K = QWEN3_0P6B_UP
    gemv_case(T, "cfg0 qwen3-0.6b up_proj", N, K)


def config2(T):
    N, K = LLAMA3_8B["gate"]
    c = make_case(N, K, seed=2, M=64)
    packed, st = binding.ptqtp_pack(dev(c["T1"]), dev(c["T2"]), dev(c["alpha1"]), dev(c["alpha2"]), fmt=binding.FORMAT_V2)
    bufs = T.copies(packed)
    Xall = dev(c["x"])
    for M in (1, 2, 4, 8, 16, 32, 64):
        X = Xall[:M].contiguous()
        Y = torch.empty((M, N), dtype=torch.float16, device="cuda")
        us = T.steady_us([lambda b=b: binding.ptqtp_gemm_skinny(b, N, K, X, Y=Y, stream=T.stream) for b in bufs])
        nb = algorithmic_bytes(N, K, M)
        emit(workload="cfg2 gate/up batch sweep", call="ptqtp_gemm_skinny", N=N, K=K, M=M, us=round(us, 3),
             us_per_batch_row=round(us / M, 3), gbs=round(nb / us / 1e3, 1), bytes=nb)
        ws = torch.empty(binding.gemm_skinny_workspace_size(N, K, M), dtype=torch.uint8, device="cuda")
        us = T.steady_us([lambda b=b: binding.ptqtp_gemm_skinny_ws(b, N, K, X, Y=Y, workspace=ws, stream=T.stream)
                          for b in bufs])
        emit(workload="cfg2 gate/up batch sweep", call="ptqtp_gemm_skinny_ws", N=N, K=K, M=M, us=round(us, 3),
             us_per_batch_row=round(us / M, 3), gbs=round(nb / us / 1e3, 1), bytes=nb)
    del bufs
    torch.cuda.empty_cache()
    # the same sweep on format 3 (M = 2..7: warp-MMA passes of four rows; M >= 8: the tcgen05 kernel), every 8B shape
    for name in ("gate", "down", "q", "k"):
        N, K = LLAMA3_8B[name]
        c = make_case(N, K, seed=2, M=64)
        packed, st = binding.ptqtp_pack(dev(c["T1"]), dev(c["T2"]), dev(c["alpha1"]), dev(c["alpha2"]), fmt=binding.FORMAT_V3)
        bufs = T.copies(packed)
        Xall = dev(c["x"])
        for M in (2, 4, 8, 16, 32, 64):
            X = Xall[:M].contiguous()
            Y = torch.empty((M, N), dtype=torch.float16, device="cuda")
            us = T.steady_us([lambda b=b: binding.ptqtp_gemm_skinny(b, N, K, X, Y=Y, stream=T.stream, fmt=binding.FORMAT_V3)
                              for b in bufs])
            nb = algorithmic_bytes(N, K, M)
            emit(workload="cfg2 format 3 batch sweep " + name, call="ptqtp_gemm_skinny", N=N, K=K, M=M, us=round(us, 3),
                 us_per_batch_row=round(us / M, 3), gbs=round(nb / us / 1e3, 1), bytes=nb)
        del bufs
        torch.cuda.empty_cache()


def config3(T):
    for name, (N, K) in sorted(LLAMA3_70B.items()):
        gemv_case(T, "cfg3 llama3-70b " + name, N, K, p_zero=0.5, seed=3, batches=(1, 8))
        torch.cuda.empty_cache()


def config5(T):
    # the chain walks over enough copies of the layer to exceed twice the L2 size
    variants = [
        ("stacked q/k/v", [("qkv", 6144, 4096), ("o", 4096, 4096), ("gate", 14336, 4096), ("up", 14336, 4096),
                           ("down", 4096, 14336)]),
        ("stacked q/k/v and gate/up", [("qkv", 6144, 4096), ("o", 4096, 4096), ("gate_up", 28672, 4096),
                                       ("down", 4096, 14336)]),
        ("stacked q/k/v, gate/up interleaved with the gated pair epilogue (ptqtp_gemv_swiglu)",
         [("qkv", 6144, 4096), ("o", 4096, 4096), ("swiglu", 28672, 4096), ("down", 4096, 14336)]),
    ]
    for what, shapes in variants:
        base = {}
        for i, (name, N, K) in enumerate(shapes):
            c = make_case(N, K, seed=50 + i)
            packed, st = binding.ptqtp_pack(dev(c["T1"]), dev(c["T2"]), dev(c["alpha1"]), dev(c["alpha2"]), fmt=FMT)
            base[name] = (packed, dev(c["x"]), torch.empty(N, dtype=torch.float16, device="cuda"))
        layer_bytes = sum(base[n][0].numel() for n, _, _ in shapes)
        copies = max(4, -(-(2 * T.l2 + (64 << 20)) // layer_bytes))
        layers = [{n: (base[n][0] if l == 0 else base[n][0].clone()) for n, _, _ in shapes} for l in range(copies)]
        calls = []
        for l in range(copies):
            for name, N, K in shapes:
                if name == "swiglu":
                    calls.append(lambda p=layers[l][name], N=N, K=K, x=base[name][1], y=base[name][2][:N // 2]:
                                 binding.ptqtp_gemv_swiglu(p, N, K, x, y=y, stream=T.stream, fmt=FMT))
                else:
                    calls.append(lambda p=layers[l][name], N=N, K=K, x=base[name][1], y=base[name][2]:
                                 binding.ptqtp_gemv(p, N, K, x, y=y, stream=T.stream, fmt=FMT))
        us = T.steady_us(calls) * len(shapes)
        nb = sum(algorithmic_bytes(N, K) - (N if name == "swiglu" else 0) for name, N, K in shapes)
        emit(workload="cfg5 llama3-8b layer, " + what, call="%d x ptqtp_gemv (format %d)" % (len(shapes), FMT), us_per_layer=round(us, 3),
             gbs=round(nb / us / 1e3, 1), bytes=nb, layer_copies=copies)
        del layers, base, calls
        torch.cuda.empty_cache()


def config6(T):
    # the seven linears of a LLaMA-3-70B-shaped layer as one chain of calls, two copies of the layer (> 2x L2)
    order = [("q", "qo"), ("k", "kv"), ("v", "kv"), ("o", "qo"), ("gate", "gate_up"), ("up", "gate_up"), ("down", "down")]
    base = {}
    for i, u in enumerate(sorted(LLAMA3_70B)):
        N, K = LLAMA3_70B[u]
        c = make_case(N, K, seed=60 + i)
        packed, st = binding.ptqtp_pack(dev(c["T1"]), dev(c["T2"]), dev(c["alpha1"]), dev(c["alpha2"]), fmt=FMT)
        base[u] = (packed, dev(c["x"]), torch.empty(N, dtype=torch.float16, device="cuda"))
    calls = []
    for l in range(2):
        for name, u in order:
            p = base[u][0] if (l == 0 and name in ("q", "k", "gate", "down")) else base[u][0].clone()
            N, K = LLAMA3_70B[u]
            calls.append(lambda p=p, N=N, K=K, x=base[u][1], y=base[u][2]: binding.ptqtp_gemv(p, N, K, x, y=y, stream=T.stream, fmt=FMT))
    us = T.steady_us(calls, reps=40) * len(order)
    nb = sum(algorithmic_bytes(*LLAMA3_70B[u]) for _, u in order)
    emit(workload="cfg6 llama3-70b-shaped layer as one chain", call="7 x ptqtp_gemv (format %d)" % FMT, us_per_layer=round(us, 3),
         gbs=round(nb / us / 1e3, 1), bytes=nb, layer_copies=2)


def config4(T, layers=32):
    names = ("q", "k", "v", "o", "gate", "up", "down")
    stack, err2, w2, sweeps = [], {m: 0.0 for m in names}, {m: 0.0 for m in names}, []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dec_ms = 0.0
    for l in range(layers):
        layer = {}
        for mi, m in enumerate(names):
            N, K = LLAMA3_8B[m]
            W = make_weights_device(N, K, seed=1000 + 7 * l + mi)
            torch.cuda.synchronize()
            e0.record()
            T1, T2, a1, a2, info = binding.ptqtp_decompose(W, details=True)
            e1.record()
            torch.cuda.synchronize()
            dec_ms += e0.elapsed_time(e1)
            sweeps.append(info["sweeps"])
            layer[m], st = binding.ptqtp_pack(T1, T2, a1, a2, fmt=FMT)
            # reconstruction error with the fp16 scales that were packed (plain torch arithmetic on the device)
            What = (a1.float().repeat_interleave(128, dim=1) * T1.float() + a2.float().repeat_interleave(128, dim=1) * T2.float())
            err2[m] += float(((W - What).double() ** 2).sum())
            w2[m] += float((W.double() ** 2).sum())
            del W, What, T1, T2, a1, a2
        stack.append(layer)
    xs = {m: torch.randn(LLAMA3_8B[m][1], device="cuda").half() for m in names}
    ys = {m: torch.empty(LLAMA3_8B[m][0], dtype=torch.float16, device="cuda") for m in names}
    calls = [lambda p=layer[m], m=m: binding.ptqtp_gemv(p, *LLAMA3_8B[m], xs[m], y=ys[m], stream=T.stream, fmt=FMT)
             for layer in stack for m in names]
    us = T.steady_us(calls, reps=20) * len(calls)
    nb = layers * sum(algorithmic_bytes(*LLAMA3_8B[m]) for m in names)
    emit(workload="cfg4 %d-layer llama3-8b linear stack, weights decomposed on the GPU, batch 1" % layers,
         call="%d x ptqtp_gemv (format %d)" % (len(calls), FMT), us_per_token=round(us, 1), us_per_layer=round(us / layers, 3),
         gbs=round(nb / us / 1e3, 1), bytes=nb, distinct_decomposed_layers=layers,
         reconstruction_error={m: round((err2[m] / w2[m]) ** 0.5, 4) for m in names},
         reconstruction_error_all=round((sum(err2.values()) / sum(w2.values())) ** 0.5, 4),
         decompose_ms_total=round(dec_ms, 1), decompose_ms_per_layer=round(dec_ms / layers, 2),
         sweeps_min=int(min(sweeps)), sweeps_max=int(max(sweeps)))


def main():
    global FMT
    ap = argparse.ArgumentParser()
    ap.add_argument("--only", default="0,2,3,4,5,6")
    ap.add_argument("--format", type=int, default=3, choices=(2, 3))
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise RuntimeError("needs a CUDA device")
    binding.lib()
    FMT = args.format
    binding.ptqtp_set_overlap(2)
    T = Timer()
    which = set(int(v) for v in args.only.split(","))
    if 0 in which:
        config0(T)
    if 2 in which:
        config2(T)
    if 3 in which:
        config3(T)
    if 5 in which:
        config5(T)
    if 6 in which:
        config6(T)
    if 4 in which:
        config4(T)



if __name__ == "__main__":
    main()
