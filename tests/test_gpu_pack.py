"""GPU pack/unpack: bit-exact round trip and byte equality with the independent format writer."""
import numpy as np
import pytest
import torch

from oracle import packed_format as pf
from paper_2509_16989_b200 import binding
from paper_2509_16989_b200.inputs import LLAMA3_8B_UNIQUE, QWEN3_0P6B_UP, make_case
from gpu_util import FORMATS, dev

pytestmark = pytest.mark.gpu


WRITERS = {binding.FORMAT_V1: pf.pack_reference, binding.FORMAT_V2: pf.pack_reference_v2,
           binding.FORMAT_V3: pf.pack_reference_v3}
READERS = {binding.FORMAT_V1: pf.unpack_reference, binding.FORMAT_V2: pf.unpack_reference_v2,
           binding.FORMAT_V3: pf.unpack_reference_v3}


def reference_blob(c, fmt):
    return WRITERS[fmt](c["T1"], c["T2"], c["alpha1"], c["alpha2"])


def reference_unpack(blob, fmt):
    return READERS[fmt](blob)


def roundtrip(c, fmt):
    packed, st = binding.ptqtp_pack(dev(c["T1"]), dev(c["T2"]), dev(c["alpha1"]), dev(c["alpha2"]), fmt=fmt)
    T1, T2, a1, a2, st2 = binding.ptqtp_unpack(packed, c["N"], c["K"], fmt=fmt)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and int(st2.item()) == 0
    assert np.array_equal(T1.cpu().numpy(), c["T1"])
    assert np.array_equal(T2.cpu().numpy(), c["T2"])
    assert np.array_equal(a1.cpu().numpy().view(np.uint16), c["alpha1"].view(np.uint16))
    assert np.array_equal(a2.cpu().numpy().view(np.uint16), c["alpha2"].view(np.uint16))
    return packed.cpu().numpy()


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("N,K", [(1, 128), (2, 128), (3, 256), (7, 1152), (33, 2048), (130, 3200), (9, 4224),
                                 (64, 14336), (17, 512), (16, 640), QWEN3_0P6B_UP])
def test_roundtrip_and_bytes_match_reference_writer(N, K, fmt):
    c = make_case(N, K, seed=N + K)
    blob = roundtrip(c, fmt)
    ref = reference_blob(c, fmt)
    assert blob.size == ref.size == binding.packed_size(N, K, fmt=fmt)
    assert np.array_equal(blob, ref)
    t1, t2, a1, a2 = reference_unpack(blob, fmt)        # the independent CPU reader agrees too
    assert np.array_equal(t1, c["T1"]) and np.array_equal(t2, c["T2"])
    assert np.array_equal(a1.view(np.uint16), c["alpha1"].view(np.uint16))
    assert np.array_equal(a2.view(np.uint16), c["alpha2"].view(np.uint16))


@pytest.mark.parametrize("fmt", FORMATS)
def test_all_nine_pairs_at_every_position(fmt):
    # row r holds pair number r at every column; then a rolling pattern so that each lane-block
    # position sees every pair next to every other pair.
    K = 2048
    pairs = [(a, b) for a in (-1, 0, 1) for b in (-1, 0, 1)]
    T1 = np.zeros((18, K), np.int8)
    T2 = np.zeros((18, K), np.int8)
    for r, (a, b) in enumerate(pairs):
        T1[r, :] = a
        T2[r, :] = b
        idx = (np.arange(K) + r) % 9
        T1[9 + r, :] = np.array([p[0] for p in pairs], np.int8)[idx]
        T2[9 + r, :] = np.array([p[1] for p in pairs], np.int8)[idx]
    c = make_case(18, K, seed=1)
    c["T1"], c["T2"] = T1, T2
    blob = roundtrip(c, fmt)
    assert np.array_equal(blob, reference_blob(c, fmt))


@pytest.mark.parametrize("fmt", FORMATS)
def test_scale_bit_patterns_are_carried_verbatim(fmt):
    c = make_case(4, 1024, seed=5)
    special = np.array([0x0000, 0x8000, 0x0001, 0x83FF, 0x7BFF, 0xFBFF, 0x7C00, 0xFC00, 0x7E00, 0x7C01,
                        0xFFFF, 0x3C00, 0x0400, 0x03FF, 0xBC00, 0x1234], np.uint16)
    a1 = np.resize(special, c["alpha1"].shape).astype(np.uint16)
    a2 = np.resize(special[::-1], c["alpha2"].shape).astype(np.uint16)
    c["alpha1"], c["alpha2"] = a1.view(np.float16), a2.view(np.float16)
    roundtrip(c, fmt)


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("name", sorted(LLAMA3_8B_UNIQUE))
def test_roundtrip_llama3_8b_shapes(name, fmt):
    N, K = LLAMA3_8B_UNIQUE[name]
    roundtrip(make_case(N, K, seed=7), fmt)


@pytest.mark.parametrize("fmt", FORMATS)
def test_invalid_trit_sets_device_status_and_kernel_completes(fmt):
    c = make_case(5, 1024, seed=9)
    bad = c["T2"].copy()
    bad[3, 700] = 2
    packed, st = binding.ptqtp_pack(dev(c["T1"]), dev(bad), dev(c["alpha1"]), dev(c["alpha2"]), fmt=fmt)
    torch.cuda.synchronize()
    assert int(st.item()) == binding.ERR_TRIT
    # the offending entry is stored as 0, everything else intact
    T1, T2, a1, a2, st2 = binding.ptqtp_unpack(packed, 5, 1024, fmt=fmt)
    torch.cuda.synchronize()
    fixed = bad.copy()
    fixed[3, 700] = 0
    assert np.array_equal(T2.cpu().numpy(), fixed) and np.array_equal(T1.cpu().numpy(), c["T1"])
    bad[3, 700] = -128
    _, st = binding.ptqtp_pack(dev(c["T1"]), dev(bad), dev(c["alpha1"]), dev(c["alpha2"]), fmt=fmt)
    assert int(st.item()) == binding.ERR_TRIT


@pytest.mark.parametrize("fmt", FORMATS)
def test_unpack_reports_header_mismatch(fmt):
    c = make_case(8, 1024, seed=10)
    packed, _ = binding.ptqtp_pack(dev(c["T1"]), dev(c["T2"]), dev(c["alpha1"]), dev(c["alpha2"]), fmt=fmt)
    other_shape = (24, 512) if fmt == binding.FORMAT_V3 else (4, 2048)
    assert binding.packed_size(*other_shape, fmt=fmt) == packed.numel()
    *_, st = binding.ptqtp_unpack(packed, *other_shape, fmt=fmt)      # same byte size, different shape
    torch.cuda.synchronize()
    assert int(st.item()) == binding.ERR_FORMAT
    for other in FORMATS:
        if other != fmt and binding.packed_size(8, 1024, fmt=other) <= packed.numel():
            *_, st = binding.ptqtp_unpack(packed, 8, 1024, fmt=other)    # a blob of another format
            assert int(st.item()) == binding.ERR_FORMAT
    packed[0] = 0
    *_, st = binding.ptqtp_unpack(packed, 8, 1024, fmt=fmt)
    assert int(st.item()) == binding.ERR_FORMAT


@pytest.mark.parametrize("fmt", FORMATS)
def test_header_parses_on_host(fmt):
    c = make_case(6, 1152, seed=11)
    packed, _ = binding.ptqtp_pack(dev(c["T1"]), dev(c["T2"]), dev(c["alpha1"]), dev(c["alpha2"]), fmt=fmt)
    assert binding.ptqtp_parse_header(bytes(packed[:256].cpu().numpy())) == (6, 1152, fmt)


@pytest.mark.parametrize("fmt", FORMATS)
def test_guard_bands_untouched(fmt):
    c = make_case(9, 1152, seed=12)
    size = binding.packed_size(9, 1152, fmt=fmt)
    buf = torch.full((size + 512,), 0xA5, dtype=torch.uint8, device="cuda")
    view = buf[256:256 + size]
    binding.ptqtp_pack(dev(c["T1"]), dev(c["T2"]), dev(c["alpha1"]), dev(c["alpha2"]), packed=view, fmt=fmt)
    torch.cuda.synchronize()
    host = buf.cpu().numpy()
    assert np.all(host[:256] == 0xA5) and np.all(host[256 + size:] == 0xA5)
    assert np.array_equal(host[256:256 + size], reference_blob(c, fmt))
