"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA tests/benchmark.

Holds no arithmetic of the method: only random draws and the public layer shapes.
Draw order per case is fixed (x, T1, T2, alpha1, alpha2) so both sides see identical bits.
"""
import numpy as np

GROUP = 128

# (N out, K in) of the decode linears the workloads name.
QWEN3_0P6B_UP = (3072, 1024)
LLAMA3_8B = {
    "q": (4096, 4096), "k": (1024, 4096), "v": (1024, 4096), "o": (4096, 4096),
    "gate": (14336, 4096), "up": (14336, 4096), "down": (4096, 14336),
}
LLAMA3_8B_UNIQUE = {"qo": (4096, 4096), "kv": (1024, 4096), "gate_up": (14336, 4096),
                    "down": (4096, 14336)}
LLAMA3_70B = {"qo": (8192, 8192), "kv": (1024, 8192), "gate_up": (28672, 8192),
              "down": (8192, 28672)}


def random_trits(rng, shape, p_zero):
    """iid trits with P(0) = p_zero and P(-1) = P(+1) = (1 - p_zero) / 2, int8."""
    u = rng.random(shape, dtype=np.float32)
    pm = np.float32((1.0 - p_zero) / 2.0)
    t = np.zeros(shape, dtype=np.int8)
    t[u < pm] = -1
    t[u >= np.float32(1.0) - pm] = 1
    return t


def make_case(N, K, seed=0, M=1, p_zero=0.4, sigma1=0.02, sigma2=0.01, G=GROUP):
    """One synthetic PTQTP linear: fp16 x ~ N(0,1), iid trit planes, fp16 |N(0, sigma)| scales."""
    rng = np.random.default_rng(seed)
    xshape = (K,) if M == 1 else (M, K)
    x = rng.standard_normal(xshape, dtype=np.float32).astype(np.float16)
    T1 = random_trits(rng, (N, K), p_zero)
    T2 = random_trits(rng, (N, K), p_zero)
    a1 = np.abs(rng.normal(0.0, sigma1, (N, K // G))).astype(np.float16)
    a2 = np.abs(rng.normal(0.0, sigma2, (N, K // G))).astype(np.float16)
    return dict(N=N, K=K, M=M, G=G, x=x, T1=T1, T2=T2, alpha1=a1, alpha2=a2)


def make_weights(N, K, seed=0, sigma=0.02, outlier_frac=1e-3, outlier_gain=20.0):
    """fp32 W ~ N(0, sigma^2) with a fraction of entries (uniform positions) multiplied by a gain."""
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((N, K), dtype=np.float32) * np.float32(sigma)).astype(np.float32)
    n_out = int(round(outlier_frac * N * K))
    if n_out:
        pos = rng.choice(N * K, size=n_out, replace=False)
        W.reshape(-1)[pos] *= np.float32(outlier_gain)
    return W


def make_activations(K, seed=0, M=1):
    rng = np.random.default_rng(seed)
    shape = (K,) if M == 1 else (M, K)
    return rng.standard_normal(shape, dtype=np.float32).astype(np.float16)


def make_weights_device(N, K, seed=0, sigma=0.02, outlier_frac=1e-3, outlier_gain=20.0, device="cuda"):
    """The same distribution as make_weights, drawn on the device with torch's generator (for workloads that are
    too large to draw on the host: each entry is an outlier with probability outlier_frac, independently)."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    W = torch.randn((N, K), generator=g, device=device, dtype=torch.float32) * sigma
    mask = torch.rand((N, K), generator=g, device=device) < outlier_frac
    return torch.where(mask, W * outlier_gain, W).contiguous()
