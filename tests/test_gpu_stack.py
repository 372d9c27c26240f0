"""Realistic-weight stack: 32 layers of LLaMA-3-8B-shaped linears whose planes come from the oracle's
progressive trit-plane decomposition of W ~ N(0, 0.02^2) with 0.1 % of entries multiplied by 20.

Checks parity of the GEMV on decomposed planes (every row, every matrix type), the reconstruction error range,
and that one decode step (224 GEMV calls in one CUDA graph, replayed) reproduces the results of plain calls bit
for bit.  One layer is decomposed (the oracle needs about 20 s of CPU time per layer); the other 31 are byte
copies of its packed blobs at distinct addresses.  The step is timed by `python -m paper_2509_16989_b200.report 4`."""
import numpy as np
import pytest
import torch

from oracle.c_oracle import decompose_c, layer_fp64_c, max_threads
from oracle.decompose import reconstruction_error
from paper_2509_16989_b200 import binding
from paper_2509_16989_b200.inputs import LLAMA3_8B, make_activations, make_weights
from gpu_util import assert_parity, dev

pytestmark = pytest.mark.gpu
NAMES = ("q", "k", "v", "o", "gate", "up", "down")


def test_config4_stack_parity_and_error():
    blobs, errs = {}, {}
    for mi, m in enumerate(NAMES):
        N, K = LLAMA3_8B[m]
        W = make_weights(N, K, seed=1000 + mi)
        d = decompose_c(W)
        errs[m] = reconstruction_error(W, d["T1"], d["T2"], d["alpha1_fp16"], d["alpha2_fp16"])
        assert 0.10 < errs[m] < 0.25
        assert set(np.unique(d["T1"])) <= {-1, 0, 1} and set(np.unique(d["T2"])) <= {-1, 0, 1}
        packed, st = binding.ptqtp_pack(dev(d["T1"]), dev(d["T2"]), dev(d["alpha1_fp16"]), dev(d["alpha2_fp16"]))
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        x = make_activations(K, seed=70 + mi)
        y = binding.ptqtp_gemv(packed, N, K, dev(x)).cpu().numpy()
        ref = layer_fp64_c(d["T1"], d["T2"], d["alpha1_fp16"], d["alpha2_fp16"], x, threads=max_threads())
        assert_parity(y, ref, x, m)
        blobs[m] = packed
        del d, W
    stack = [{m: (blobs[m] if i == 0 else blobs[m].clone()) for m in NAMES} for i in range(32)]
    xs = {m: dev(make_activations(LLAMA3_8B[m][1], seed=5)) for m in NAMES}
    ys = {m: torch.empty(LLAMA3_8B[m][0], dtype=torch.float16, device="cuda") for m in NAMES}
    stream = torch.cuda.Stream()

    def step():
        for layer in stack:
            for m in NAMES:
                N, K = LLAMA3_8B[m]
                binding.ptqtp_gemv(layer[m], N, K, xs[m], y=ys[m], stream=stream)

    with torch.cuda.stream(stream):
        step()
        stream.synchronize()
        first = {m: ys[m].cpu().numpy().copy() for m in NAMES}
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            step()
        for _ in range(3):
            g.replay()
        stream.synchronize()
    for m in NAMES:                                   # every layer holds the same planes: the last one's result
        assert np.array_equal(ys[m].cpu().numpy().view(np.uint16), first[m].view(np.uint16))
