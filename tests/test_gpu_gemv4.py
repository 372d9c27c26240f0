"""GPU parity of the format-3 batch-1 kernel (int8 warp MMAs on codes in fragment order) against the fp64 oracle:
launch configurations, exact integer cases, the gated pair epilogue, stream order under the overlap levels, and the
give-up path of its bounded waits.  Shapes that every format shares are covered in test_gpu_gemv.py (FORMATS)."""
import numpy as np
import pytest
import torch

from oracle.layer import layer_fp64
from paper_2509_16989_b200 import binding
from paper_2509_16989_b200.inputs import LLAMA3_8B_UNIQUE, make_case
from gpu_util import assert_parity, dev, oracle_y, pack_case

pytestmark = pytest.mark.gpu
V3 = binding.FORMAT_V3


@pytest.fixture(autouse=True)
def decode_overlap_level():
    old = binding.ptqtp_set_overlap(2)
    yield
    binding.ptqtp_set_overlap(old)


def _smem_bytes(N, K, warps, depth, units, per_sm):
    """Shared memory of a launch, from the kernel's layout: x as read (2 K bytes), a staging area of 1120 bytes per
    warp, the partial sums, the fp16 rows, the table of the CTA's shares (64 bytes), one mbarrier per ring slot and one for x, the ring (tiles of 4352 bytes)
    from a 128-byte boundary."""
    S, nrb = -(-K // 512), -(-((N + 1) // 2) // 8)
    rows_cap = 16 * -(-nrb // min(per_sm * 148, nrb))
    off = 2 * K + warps * 1120 + rows_cap * S * 4 + rows_cap * 2
    off = -(-off // 16) * 16 + 64 + (warps * depth + 1) * 8
    return -(-off // 128) * 128 + warps * depth * units * 4352


@pytest.mark.parametrize("per_sm", [1, 2])
@pytest.mark.parametrize("units", [1, 2])
@pytest.mark.parametrize("depth", [2, 3, 4, 6])
@pytest.mark.parametrize("warps", [1, 2, 3, 4, 7, 8, 16])
def test_launch_configurations(warps, depth, units, per_sm):
    for N, K in ((67, 8192), (1000, 14336), (4, 2048), (2400, 1024), (333, 640), (23, 128)):
        c = make_case(N, K, seed=warps * 10 + depth)
        packed = pack_case(c, V3)
        cfg = dict(rows_per_warp=units, k_split=warps, depth=depth, ctas_per_sm=per_sm, fmt=V3)
        budget = (228 // per_sm - 1) * 1024
        fits = warps * per_sm <= 16 and _smem_bytes(N, K, warps, depth, units, per_sm) <= budget
        if not fits:
            with pytest.raises(binding.PtqtpError) as e:
                binding.ptqtp_gemv_cfg(packed, N, K, dev(c["x"]), **cfg)
            assert e.value.status == binding.ERR_CONFIG
            continue
        y = binding.ptqtp_gemv_cfg(packed, N, K, dev(c["x"]), **cfg)
        torch.cuda.synchronize()
        assert_parity(y.cpu().numpy(), oracle_y(c), c["x"],
                      "warps=%d depth=%d units=%d per_sm=%d N=%d K=%d" % (warps, depth, units, per_sm, N, K))


def test_whole_sm_configuration_and_rejections():
    c = make_case(1000, 4096, seed=3)
    packed = pack_case(c, V3)
    y = binding.ptqtp_gemv_cfg(packed, 1000, 4096, dev(c["x"]), k_split=-1, fmt=V3)
    torch.cuda.synchronize()
    assert_parity(y.cpu().numpy(), oracle_y(c), c["x"], "whole SM")
    for bad in (dict(rows_per_warp=3), dict(rows_per_warp=4), dict(arith=3), dict(arith=4), dict(k_split=17), dict(depth=5),
                dict(depth=8), dict(ctas_per_sm=5), dict(k_split=16, ctas_per_sm=2)):
        with pytest.raises(binding.PtqtpError) as e:
            binding.ptqtp_gemv_cfg(packed, 1000, 4096, dev(c["x"]), fmt=V3, **bad)
        assert e.value.status == binding.ERR_CONFIG


def test_exact_for_integer_activations():
    # small integer activations, scales 1 and 2: every product and sum is an integer below 2^11, so the fp16
    # result must equal the exact integer sum
    N, K = 300, 4096
    c = make_case(N, K, seed=12)
    rng = np.random.default_rng(3)
    c["x"] = rng.integers(-3, 4, K).astype(np.float16)
    c["alpha1"] = np.ones_like(c["alpha1"])
    c["alpha2"] = np.full_like(c["alpha2"], 2.0)
    exact = (c["T1"].astype(np.int64) @ c["x"].astype(np.int64)) + 2 * (c["T2"].astype(np.int64) @ c["x"].astype(np.int64))
    assert np.all(np.abs(exact) < 2048)
    y = binding.ptqtp_gemv(pack_case(c, V3), N, K, dev(c["x"]), fmt=V3)
    torch.cuda.synchronize()
    assert np.array_equal(y.cpu().numpy().astype(np.int64), exact)


def test_every_field_and_group_position_is_wired_to_its_output():
    # one non-zero trit at a time: y must be alpha * x[col] in exactly one row, for positions that walk through
    # every (row within a tile, plane, column within a 512-column superblock) combination at least once
    N, K = 48, 1536
    rng = np.random.default_rng(5)
    c = make_case(N, K, seed=5)
    c["x"] = rng.integers(1, 30, K).astype(np.float16)
    a1 = rng.integers(1, 8, c["alpha1"].shape).astype(np.float16)
    a2 = rng.integers(1, 8, c["alpha2"].shape).astype(np.float16) * np.float16(0.5)
    z = np.zeros((N, K), np.int8)
    for plane in (0, 1):
        T = z.copy()
        # row r carries one trit at column (37 r + 11 j) for 32 values of j: all residues of columns mod 512 get hit
        for r in range(N):
            for j in range(32):
                T[r, (37 * r + 53 * j + 512 * (j % 3)) % K] = 1 if (r + j) % 2 == 0 else -1
        cc = dict(c, T1=T if plane == 0 else z, T2=z if plane == 0 else T, alpha1=a1, alpha2=a2)
        ref = layer_fp64(cc["T1"], cc["T2"], a1, a2, c["x"])
        y = binding.ptqtp_gemv(pack_case(cc, V3), N, K, dev(c["x"]), fmt=V3)
        torch.cuda.synchronize()
        assert np.array_equal(y.cpu().numpy().astype(np.float64), ref.astype(np.float16).astype(np.float64)), plane


@pytest.mark.parametrize("pairs,K", [(1, 128), (3, 1152), (64, 4096), (515, 2048), (300, 14336), (7168, 4096)])
def test_gated_pair_epilogue_matches_oracle(pairs, K):
    N = 2 * pairs
    c = make_case(N, K, seed=900 + pairs)
    c["alpha1"] = (c["alpha1"].astype(np.float32) * 4).astype(np.float16)          # gate values of order 1
    y = binding.ptqtp_gemv_swiglu(pack_case(c, V3), N, K, dev(c["x"]), fmt=V3)
    torch.cuda.synchronize()
    y = y.cpu().numpy().astype(np.float64)
    t = oracle_y(c)
    g, u = t[0::2], t[1::2]
    ref = g / (1.0 + np.exp(-g)) * u
    B = 2e-3 * float(np.abs(c["x"].astype(np.float64)).max()) * np.sqrt(K)
    bound = B * (1.1 * np.abs(u) + np.abs(g / (1.0 + np.exp(-g)))) + 2.0 ** -10 * np.abs(ref) + 1e-7
    assert np.all(np.isfinite(y)) and y.shape == (pairs,)
    assert np.all(np.abs(y - ref) <= bound)
    assert np.linalg.norm(y - ref) <= 1e-3 * np.linalg.norm(ref) + 1e-6


@pytest.mark.parametrize("level", [0, 1, 2])
@pytest.mark.parametrize("graph", [False, True])
def test_chain_keeps_stream_order(graph, level):
    # y1 = layer1(x), y2 = layer2(y1), y3 = layer1(y2): a call that used x before its predecessor had written it
    # would be caught.  Checked link by link against the oracle; all levels give the same bits.
    N = K = 2048
    c1, c2 = make_case(N, K, seed=50), make_case(N, K, seed=51)
    c1["alpha1"] = (c1["alpha1"].astype(np.float32) * 1.5).astype(np.float16)
    c2["alpha1"] = (c2["alpha1"].astype(np.float32) * 1.5).astype(np.float16)
    p1, p2 = pack_case(c1, V3), pack_case(c2, V3)
    x = dev(c1["x"])
    ys = [torch.empty(N, dtype=torch.float16, device="cuda") for _ in range(3)]
    binding.ptqtp_set_overlap(level)

    def chain():
        binding.ptqtp_gemv(p1, N, K, x, y=ys[0], fmt=V3)
        binding.ptqtp_gemv(p2, N, K, ys[0], y=ys[1], fmt=V3)
        binding.ptqtp_gemv(p1, N, K, ys[1], y=ys[2], fmt=V3)

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        chain()
        stream.synchronize()
        if graph:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for _ in range(8):
                    chain()
        for y in ys:
            y.zero_()
        for _ in range(5):
            if graph:
                g.replay()
            else:
                for _ in range(8):
                    chain()
        stream.synchronize()
    h = [y.cpu().numpy() for y in ys]
    for cc, xin, yout, what in ((c1, c1["x"], h[0], "link 1"), (c2, h[0], h[1], "link 2"), (c1, h[1], h[2], "link 3")):
        assert_parity(yout, oracle_y(dict(cc, x=xin)), xin, what)
    binding.ptqtp_set_overlap(0)
    with torch.cuda.stream(stream):
        chain()
        stream.synchronize()
    for y, ref in zip(ys, h):
        assert np.array_equal(y.cpu().numpy().view(np.uint16), ref.view(np.uint16))


def test_speculative_read_sees_activations_written_just_before():
    N, K = 512, 4096
    c = make_case(N, K, seed=60)
    packed = pack_case(c, V3)
    xa = c["x"].copy()
    xb = c["x"].copy()
    xb[K - 3] = np.float16(-float(xb[K - 3]) + 0.25)
    da, db = dev(xa), dev(xb)
    x = torch.empty(K, dtype=torch.float16, device="cuda")
    ys = [torch.empty(N, dtype=torch.float16, device="cuda") for _ in range(6)]
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i, y in enumerate(ys):
            src = da if i % 2 == 0 else db
            if i % 3 == 0:
                x.copy_(src)
            else:
                torch.add(src, 0, out=x)
            binding.ptqtp_gemv(packed, N, K, x, y=y, fmt=V3)
        stream.synchronize()
    ra, rb = oracle_y(dict(c, x=xa)), oracle_y(dict(c, x=xb))
    for i, y in enumerate(ys):
        assert_parity(y.cpu().numpy(), ra if i % 2 == 0 else rb, xa if i % 2 == 0 else xb, "call %d" % i)
    assert np.array_equal(ys[0].cpu().numpy().view(np.uint16), ys[2].cpu().numpy().view(np.uint16))
    assert not np.array_equal(ys[0].cpu().numpy().view(np.uint16), ys[1].cpu().numpy().view(np.uint16))


@pytest.mark.parametrize("fmt", [binding.FORMAT_V2, V3])
def test_default_level_keeps_packed_in_stream_order(fmt):
    # library default (level 0): a blob written by another kernel directly ahead on the stream (a device-to-device
    # clone here) is read only after that kernel has finished
    binding.ptqtp_set_overlap(0)
    N, K = 4096, 4096
    cs = [make_case(N, K, seed=80 + i) for i in range(2)]
    srcs = [pack_case(c, fmt) for c in cs]
    x = dev(cs[0]["x"])
    ys = [torch.empty(N, dtype=torch.float16, device="cuda") for _ in range(6)]
    blob = torch.empty_like(srcs[0])
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i, y in enumerate(ys):
            torch.add(srcs[i % 2], 0, out=blob)          # an elementwise kernel rewrites the whole blob
            binding.ptqtp_gemv(blob, N, K, x, y=y, fmt=fmt)
        stream.synchronize()
    refs = [oracle_y(dict(c, x=cs[0]["x"])) for c in cs]
    for i, y in enumerate(ys):
        assert_parity(y.cpu().numpy(), refs[i % 2], cs[0]["x"], "call %d" % i)


def test_bounded_wait_gives_up_reports_and_recovers():
    # one mbarrier of the first CTA is told to expect 16 bytes more than its copy brings: the wait runs out after the
    # poll limit, the rows of that warp come out as NaN, the status word reports it, and the kernel ends normally.
    # After the word is cleared the next call is healthy again.
    N, K = 2400, 2048
    c = make_case(N, K, seed=66)
    packed = pack_case(c, V3)
    ref = oracle_y(c)
    binding.ptqtp_kernel_status_clear()
    assert binding.ptqtp_kernel_status() == 0
    old = binding.ptqtp_set_wait_limit(1 << 10)
    try:
        binding.ptqtp_test_fail_next_wait(1)
        y = binding.ptqtp_gemv(packed, N, K, dev(c["x"]), fmt=V3)
        torch.cuda.synchronize()
    finally:
        binding.ptqtp_set_wait_limit(old)
        binding.ptqtp_test_fail_next_wait(0)
    h = y.cpu().numpy().astype(np.float64)
    bad = np.isnan(h)
    assert bad.any() and not bad.all()
    assert bad[:16].all()                                 # the first CTA's first row block is among them
    assert_parity(h[~bad], ref[~bad], c["x"], "rows of the healthy warps")
    assert binding.ptqtp_kernel_status() == binding.ERR_CUDA
    assert binding.ptqtp_kernel_status() == binding.ERR_CUDA      # the word stays set until it is cleared
    binding.ptqtp_kernel_status_clear()
    y = binding.ptqtp_gemv(packed, N, K, dev(c["x"]), fmt=V3)
    torch.cuda.synchronize()
    assert_parity(y.cpu().numpy(), ref, c["x"], "after the failure")
    assert binding.ptqtp_kernel_status() == 0


@pytest.mark.parametrize("name", sorted(LLAMA3_8B_UNIQUE))
def test_llama3_8b_shapes_whole_sm_launch(name):
    N, K = LLAMA3_8B_UNIQUE[name]
    c = make_case(N, K, seed=11)
    y = binding.ptqtp_gemv_cfg(pack_case(c, V3), N, K, dev(c["x"]), k_split=-1, fmt=V3)
    torch.cuda.synchronize()
    assert_parity(y.cpu().numpy(), oracle_y(c), c["x"], name)


@pytest.mark.parametrize("level", [0, 2])
@pytest.mark.parametrize("Ns,K", [((4096, 1024, 1024), 4096), ((5, 33, 130, 7), 1152), ((1000,), 2048), ((14336, 14336), 4096),
                                  ((64, 2400), 14336), ((16, 16, 16, 16), 128)])
def test_several_matrices_in_one_launch_give_the_bits_of_separate_calls(Ns, K, level):
    binding.ptqtp_set_overlap(level)
    cs = [make_case(N, K, seed=500 + 7 * j + N) for j, N in enumerate(Ns)]
    x = cs[0]["x"]
    packed = [pack_case(c, V3) for c in cs]
    ys = binding.ptqtp_gemv_multi(packed, list(Ns), K, dev(x))
    torch.cuda.synchronize()
    for j, (c, p, y) in enumerate(zip(cs, packed, ys)):
        alone = binding.ptqtp_gemv(p, c["N"], K, dev(x), fmt=V3)
        torch.cuda.synchronize()
        assert np.array_equal(y.cpu().numpy().view(np.uint16), alone.cpu().numpy().view(np.uint16)), j
        assert_parity(y.cpu().numpy(), oracle_y(dict(c, x=x)), x, "matrix %d of %s" % (j, Ns))


@pytest.mark.parametrize("N,K", [(16, 128), (300, 1152), (14336, 4096), (2401, 2048)])
def test_gated_pair_of_two_matrices_in_one_launch(N, K):
    cg, cu = make_case(N, K, seed=600 + N), make_case(N, K, seed=601 + N)
    cg["alpha1"] = (cg["alpha1"].astype(np.float32) * 4).astype(np.float16)          # gate values of order 1
    x = cg["x"]
    (y,) = binding.ptqtp_gemv_multi([pack_case(cg, V3), pack_case(cu, V3)], [N, N], K, dev(x),
                                    epilogue=binding.EPILOGUE_GATED_PAIR)
    torch.cuda.synchronize()
    y = y.cpu().numpy().astype(np.float64)
    g, u = oracle_y(dict(cg, x=x)), oracle_y(dict(cu, x=x))
    ref = g / (1.0 + np.exp(-g)) * u
    B = 2e-3 * float(np.abs(x.astype(np.float64)).max()) * np.sqrt(K)
    bound = B * (1.1 * np.abs(u) + np.abs(g / (1.0 + np.exp(-g)))) + 2.0 ** -10 * np.abs(ref) + 1e-7
    assert y.shape == (N,) and np.all(np.isfinite(y))
    assert np.all(np.abs(y - ref) <= bound)
    assert np.linalg.norm(y - ref) <= 1e-3 * np.linalg.norm(ref) + 1e-6
    # the same bits as the interleaved single-matrix form of the epilogue
    inter = dict(N=2 * N, K=K, x=x, **{k: np.stack([cg[k], cu[k]], axis=1).reshape(2 * N, -1) for k in ("T1", "T2", "alpha1", "alpha2")})
    yi = binding.ptqtp_gemv_swiglu(pack_case(inter, V3), 2 * N, K, dev(x), fmt=V3)
    torch.cuda.synchronize()
    assert np.array_equal(yi.cpu().numpy().astype(np.float64), y)


def test_several_matrices_argument_checks():
    K = 1024
    cs = [make_case(64, K, seed=1), make_case(32, K, seed=2)]
    p3 = [pack_case(c, V3) for c in cs]
    x = dev(cs[0]["x"])
    with pytest.raises(binding.PtqtpError) as e:             # gated pair needs equal N
        binding.ptqtp_gemv_multi(p3, [64, 32], K, x, epilogue=binding.EPILOGUE_GATED_PAIR)
    assert e.value.status == binding.ERR_SHAPE
    with pytest.raises(binding.PtqtpError) as e:             # more than four matrices
        binding.ptqtp_gemv_multi([p3[0]] * 5, [64] * 5, K, x)
    assert e.value.status == binding.ERR_SHAPE
    with pytest.raises(binding.PtqtpError) as e:
        binding.ptqtp_gemv_multi(p3, [64, 32], K, x, epilogue=7)
    assert e.value.status == binding.ERR_CONFIG


@pytest.mark.parametrize("level", [0, 2])
@pytest.mark.parametrize("N,K,M", [(1, 128, 2), (5, 256, 3), (7, 1152, 4), (33, 2048, 2), (130, 3200, 4), (257, 5120, 3),
                                   (64, 14336, 4), (1000, 6144, 7), (37, 36864, 4), (192, 3072, 64), (2400, 4096, 9),
                                   (14336, 4096, 2), (4096, 14336, 4), (1024, 4096, 3), (4096, 4096, 8)])
def test_small_batch_on_the_batch1_layout(N, K, M, level):
    # ptqtp_gemm_skinny on format 3: passes of up to four rows on the kernel whose MMA columns are the batch rows, or
    # (more rows, larger matrices) one pass on the tcgen05 kernel
    binding.ptqtp_set_overlap(level)
    c = make_case(N, K, seed=700 + N + M, M=M)
    packed = pack_case(c, V3)
    Y = binding.ptqtp_gemm_skinny(packed, N, K, dev(c["x"]), fmt=V3)
    torch.cuda.synchronize()
    assert_parity(Y.cpu().numpy(), np.atleast_2d(oracle_y(c)), c["x"], "N=%d K=%d M=%d" % (N, K, M))
    assert binding.ptqtp_kernel_status() == 0


def test_small_batch_on_the_batch1_layout_is_exact_on_integers():
    N, K, M = 96, 4096, 4
    c = make_case(N, K, seed=13, M=M)
    rng = np.random.default_rng(4)
    c["x"] = rng.integers(-3, 4, (M, K)).astype(np.float16)
    c["alpha1"] = np.ones_like(c["alpha1"])
    c["alpha2"] = np.full_like(c["alpha2"], 2.0)
    exact = (c["x"].astype(np.int64) @ c["T1"].astype(np.int64).T) + 2 * (c["x"].astype(np.int64) @ c["T2"].astype(np.int64).T)
    assert np.all(np.abs(exact) < 2048)
    for m in (2, 3, 4):
        Y = binding.ptqtp_gemm_skinny(pack_case(c, V3), N, K, dev(c["x"][:m].copy()), fmt=V3)
        torch.cuda.synchronize()
        assert np.array_equal(Y.cpu().numpy().astype(np.int64), exact[:m]), m
