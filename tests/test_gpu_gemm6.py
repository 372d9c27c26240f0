"""GPU parity of the tcgen05 small-batch kernel on format 3 (fp16 trits from tensor memory against fp16
activations, fp32 accumulators in tensor memory) against the fp64 oracle: ragged shapes, every batch size class,
every K split of a cluster, exact integer cases, the library's dispatch and the give-up path of its bounded waits."""
import numpy as np
import pytest
import torch

from paper_2509_16989_b200 import binding
from paper_2509_16989_b200.inputs import make_case
from gpu_util import assert_parity, dev, oracle_y, pack_case

pytestmark = pytest.mark.gpu
V3 = binding.FORMAT_V3


def _run(c, packed, N, K, **kw):
    Y = binding.ptqtp_gemm_skinny_cfg(packed, N, K, dev(c["x"]), path=6, **kw)
    torch.cuda.synchronize()
    return Y.cpu().numpy()


@pytest.mark.parametrize("N,K,M", [(1, 128, 2), (5, 256, 5), (7, 1152, 16), (33, 2048, 17), (130, 3200, 31),
                                   (257, 5120, 32), (64, 14336, 33), (1000, 6144, 48), (37, 36864, 49),
                                   (192, 3072, 64), (2400, 4096, 9), (129, 640, 2), (255, 512, 64), (256, 384, 20)])
def test_ragged_shapes_and_batch_sizes(N, K, M):
    c = make_case(N, K, seed=900 + N + M, M=M)
    Y = _run(c, pack_case(c, V3), N, K)
    assert_parity(Y, np.atleast_2d(oracle_y(c)), np.atleast_2d(c["x"]), "N=%d K=%d M=%d" % (N, K, M))
    assert binding.ptqtp_kernel_status() == 0


@pytest.mark.parametrize("k_split", [1, 2, 4, 8])
@pytest.mark.parametrize("N,K,M", [(300, 4096, 24), (130, 1536, 64), (2050, 512, 7), (48, 7168, 40)])
def test_every_k_split(N, K, M, k_split):
    # a cluster of k_split CTAs shares the columns of a block of 128 rows (some CTAs get no superblock when K is short)
    c = make_case(N, K, seed=77 + k_split, M=M)
    Y = _run(c, pack_case(c, V3), N, K, k_split=k_split)
    assert_parity(Y, oracle_y(c), c["x"], "N=%d K=%d M=%d split %d" % (N, K, M, k_split))
    assert binding.ptqtp_kernel_status() == 0


@pytest.mark.parametrize("N,K,M", [(14336, 4096, 64), (4096, 14336, 16), (1024, 4096, 37), (4096, 4096, 8),
                                   (28672, 4096, 33)])
def test_full_size_shapes(N, K, M):
    c = make_case(N, K, seed=5 + M, M=M)
    Y = _run(c, pack_case(c, V3), N, K)
    assert_parity(Y, oracle_y(c), c["x"], "N=%d K=%d M=%d" % (N, K, M))
    assert binding.ptqtp_kernel_status() == 0


def test_exact_on_integers():
    # integer activations, scales 1 and 2: every product and every fp32 sum is exact, so the result is the integer
    # matrix product for every batch size class and K split
    N, K, M = 200, 4096, 64
    c = make_case(N, K, seed=13, M=M)
    rng = np.random.default_rng(4)
    c["x"] = rng.integers(-3, 4, (M, K)).astype(np.float16)
    c["alpha1"] = np.ones_like(c["alpha1"])
    c["alpha2"] = np.full_like(c["alpha2"], 2.0)
    exact = (c["x"].astype(np.int64) @ c["T1"].astype(np.int64).T) + 2 * (c["x"].astype(np.int64) @ c["T2"].astype(np.int64).T)
    assert np.all(np.abs(exact) < 2048)
    packed = pack_case(c, V3)
    for m in (1, 15, 16, 17, 33, 64):
        for k_split in (1, 4):
            cm = dict(c, x=c["x"][:m].copy())
            Y = _run(cm, packed, N, K, k_split=k_split)
            assert np.array_equal(Y.astype(np.int64), exact[:m]), (m, k_split)


def test_rows_do_not_depend_on_their_neighbours():
    # row m of the result is a function of row m of X alone: the same row inside batches of different size and at a
    # different position gives the same bits
    N, K = 300, 2048
    c = make_case(N, K, seed=31, M=40)
    packed = pack_case(c, V3)
    full = _run(c, packed, N, K, k_split=2)
    part = _run(dict(c, x=c["x"][8:24].copy()), packed, N, K, k_split=2)
    assert np.array_equal(full[8:24].view(np.uint16), part.view(np.uint16))


def test_library_dispatch():
    # the library takes the tcgen05 kernel where its fixed cost pays: many rows, or a matrix of some size
    def same(a, b):
        torch.cuda.synchronize()
        return np.array_equal(a.cpu().numpy().view(np.uint16), b.cpu().numpy().view(np.uint16))
    N, K = 4096, 4096
    c = make_case(N, K, seed=40, M=64)
    packed = pack_case(c, V3)
    for M, path in ((64, 6), (16, 6), (4, 5)):
        X = dev(c["x"][:M].copy())
        assert same(binding.ptqtp_gemm_skinny(packed, N, K, X, fmt=V3), binding.ptqtp_gemm_skinny_cfg(packed, N, K, X, path=path)), M
    N, K = 520, 3072
    c = make_case(N, K, seed=41, M=64)
    packed = pack_case(c, V3)
    for M, path in ((64, 6), (8, 5), (7, 5)):
        X = dev(c["x"][:M].copy())
        assert same(binding.ptqtp_gemm_skinny(packed, N, K, X, fmt=V3), binding.ptqtp_gemm_skinny_cfg(packed, N, K, X, path=path)), M


def test_argument_checks():
    N, K = 64, 512
    c = make_case(N, K, seed=1, M=8)
    x = dev(c["x"])
    p3 = pack_case(c, V3)
    for kw in (dict(path=4), dict(path=6, k_split=3), dict(path=6, k_split=16)):
        with pytest.raises(binding.PtqtpError) as e:
            binding.ptqtp_gemm_skinny_cfg(p3, N, K, x, **kw)
        assert e.value.status == binding.ERR_CONFIG


@pytest.mark.parametrize("k_split", [1, 4])
def test_bounded_wait_gives_up_reports_and_recovers(k_split):
    # the first wait of every CTA is made to give up: all rows come out as NaN, the status word reports it, the
    # CTAs still meet at their cluster barriers and free their tensor memory, and the next call is healthy
    N, K, M = 700, 2048, 12
    c = make_case(N, K, seed=66, M=M)
    packed = pack_case(c, V3)
    ref = oracle_y(c)
    binding.ptqtp_kernel_status_clear()
    assert binding.ptqtp_kernel_status() == 0
    try:
        binding.ptqtp_test_fail_next_wait(1)
        Y = _run(c, packed, N, K, k_split=k_split)
    finally:
        binding.ptqtp_test_fail_next_wait(0)
    assert np.isnan(Y.astype(np.float64)).all()
    assert binding.ptqtp_kernel_status() == binding.ERR_CUDA
    binding.ptqtp_kernel_status_clear()
    for _ in range(3):                                       # tensor memory was freed: later launches allocate again
        Y = _run(c, packed, N, K, k_split=k_split)
    assert_parity(Y, ref, c["x"], "after the failure")
    assert binding.ptqtp_kernel_status() == 0


def test_many_launches_on_two_streams_give_the_same_bits():
    # tensor memory is allocated and freed by every CTA: launches that share the SMs (two streams, back to back) must
    # neither starve one another nor change a result
    N, K = 2400, 2048
    cs = [make_case(N, K, seed=300 + i, M=M) for i, M in enumerate((9, 24, 40, 64))]
    packed = [pack_case(c, V3) for c in cs]
    xs = [dev(c["x"]) for c in cs]
    want = []
    for c, p, x in zip(cs, packed, xs):
        want.append(binding.ptqtp_gemm_skinny_cfg(p, N, K, x, path=6).cpu().numpy().view(np.uint16))
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [[torch.empty((x.shape[0], N), dtype=torch.float16, device="cuda") for x in xs] for _ in range(2)]
    torch.cuda.synchronize()
    for rep in range(25):
        for si, st in enumerate(streams):
            with torch.cuda.stream(st):
                for i in range(4):
                    j = (i + si + rep) % 4
                    binding.ptqtp_gemm_skinny_cfg(packed[j], N, K, xs[j], Y=outs[si][j], path=6, k_split=(1, 2, 4)[rep % 3],
                                                  stream=st)
    torch.cuda.synchronize()
    assert binding.ptqtp_kernel_status() == 0
    # the sum over a cluster is in rank order, but the split changes which partial sums exist: compare like with like
    for si in range(2):
        for j in range(4):
            got = outs[si][j].cpu().numpy()
            assert_parity(got, oracle_y(cs[j]), cs[j]["x"], "stream %d case %d" % (si, j))
    for j in range(4):
        a = binding.ptqtp_gemm_skinny_cfg(packed[j], N, K, xs[j], path=6).cpu().numpy().view(np.uint16)
        assert np.array_equal(a, want[j])
