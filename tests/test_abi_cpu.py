"""CPU-only checks of the C ABI: the library builds, loads and exports what include/ptqtp.h declares,
host-side validation returns the documented codes, and the size/header helpers agree with the
independent format description.  No kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import packed_format as pf
from paper_2509_16989_b200 import binding, build
from paper_2509_16989_b200.inputs import make_case

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ptqtp.h")).read()
    return sorted(set(re.findall(r"PTQTP_API[^;(]*?\b(ptqtp_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = declared_symbols()
    assert len(names) >= 17 and set(names) == set(binding.EXPORTS)
    for n in names:
        assert getattr(L, n) is not None
    assert L.ptqtp_version() >= 100


def test_packed_size_is_memory_formula_plus_header_and_padding(L):
    for N, K in ((3072, 1024), (4096, 4096), (1024, 4096), (14336, 4096), (4096, 14336), (8192, 28672)):
        for fmt, lay in ((1, pf.layout), (2, pf.layout_v2), (3, pf.layout_v3)):
            got = binding.packed_size(N, K, fmt=fmt)
            assert got == lay(N, K)["total"]
            assert got == pf.HEADER_BYTES + pf.memory_formula_bits(N, K) // 8      # no padding at these shapes
    # format 1: K not a multiple of 1024 pads the code and scale regions to the next multiple
    assert binding.packed_size(7, 1152, fmt=1) == 256 + 7 * 2048 // 2 + 4 * 7 * 16
    # format 2: an odd N stores one more row; a unit whose size is not a multiple of 16 is padded
    assert binding.packed_size(7, 1152, fmt=2) == 256 + 4 * (1152 + 72 + 8) == pf.layout_v2(7, 1152)["total"]
    assert binding.packed_size(3, 4224, fmt=2) == 256 + 2 * (2176 * 2 + 128 + 8 + 8) == pf.layout_v2(3, 4224)["total"]
    # format 3: whole tiles of 16 rows x 512 columns, 4352 bytes each
    assert binding.packed_size(7, 1152, fmt=3) == 256 + 1 * 3 * 4352 == pf.layout_v3(7, 1152)["total"]
    assert binding.packed_size(33, 512, fmt=3) == 256 + 3 * 1 * 4352 == pf.layout_v3(33, 512)["total"]
    for bad in ((0, 128), (4, 0), (4, 100), (-1, 128)):
        assert binding.packed_size(*bad) == 0
    assert L.ptqtp_packed_size(ctypes.byref(binding.Shape(4, 128, 64, 1))) == 0
    assert L.ptqtp_packed_size(ctypes.byref(binding.Shape(4, 128, 128, 4))) == 0
    assert L.ptqtp_packed_size(ctypes.byref(binding.Shape(4, 128, 128, 0))) == 0


def test_parse_header_accepts_reference_blob_and_rejects_damage(L):
    c = make_case(3, 1152, seed=2)
    blob2 = pf.pack_reference_v2(c["T1"], c["T2"], c["alpha1"], c["alpha2"])
    assert binding.ptqtp_parse_header(bytes(blob2[:256])) == (3, 1152, 2)
    bad2 = blob2[:256].copy()
    bad2[40] ^= 8         # bytes per row pair no longer match the shape
    with pytest.raises(binding.PtqtpError):
        binding.ptqtp_parse_header(bytes(bad2))
    blob3 = pf.pack_reference_v3(c["T1"], c["T2"], c["alpha1"], c["alpha2"])
    assert binding.ptqtp_parse_header(bytes(blob3[:256])) == (3, 1152, 3)
    bad3 = blob3[:256].copy()
    bad3[40] ^= 8         # bytes per tile no longer 4352
    with pytest.raises(binding.PtqtpError):
        binding.ptqtp_parse_header(bytes(bad3))
    blob = pf.pack_reference(c["T1"], c["T2"], c["alpha1"], c["alpha2"])
    assert binding.ptqtp_parse_header(bytes(blob[:256])) == (3, 1152, 1)
    bad = blob[:256].copy()
    bad[0] ^= 1
    with pytest.raises(binding.PtqtpError) as e:
        binding.ptqtp_parse_header(bytes(bad))
    assert e.value.status == binding.ERR_FORMAT
    bad = blob[:256].copy()
    bad[16] += 1          # N no longer matches the recorded offsets
    with pytest.raises(binding.PtqtpError):
        binding.ptqtp_parse_header(bytes(bad))
    with pytest.raises(binding.PtqtpError) as e:
        binding.ptqtp_parse_header(bytes(blob[:16]))
    assert e.value.status == binding.ERR_SIZE


def test_host_side_validation_codes(L):
    shape = binding.make_shape(8, 256)
    sp = ctypes.byref(shape)
    ok_ptr = ctypes.c_void_p(0x10000)           # never dereferenced: validation fails first
    odd_ptr = ctypes.c_void_p(0x10008)
    size = binding.packed_size(8, 256)
    assert L.ptqtp_gemv(sp, None, size, ok_ptr, ok_ptr, None) == binding.ERR_NULL
    assert L.ptqtp_gemv(sp, ok_ptr, size, None, ok_ptr, None) == binding.ERR_NULL
    assert L.ptqtp_gemv(None, ok_ptr, size, ok_ptr, ok_ptr, None) == binding.ERR_NULL
    assert L.ptqtp_gemv(sp, odd_ptr, size, ok_ptr, ok_ptr, None) == binding.ERR_ALIGN
    assert L.ptqtp_gemv(sp, ok_ptr, size, odd_ptr, ok_ptr, None) == binding.ERR_ALIGN
    assert L.ptqtp_gemv(sp, ok_ptr, size - 1, ok_ptr, ok_ptr, None) == binding.ERR_SIZE
    bad = binding.make_shape(8, 200)
    assert L.ptqtp_gemv(ctypes.byref(bad), ok_ptr, size, ok_ptr, ok_ptr, None) == binding.ERR_SHAPE
    assert L.ptqtp_gemm_skinny(sp, ok_ptr, size, 0, ok_ptr, ok_ptr, None) == binding.ERR_SHAPE
    assert L.ptqtp_gemm_skinny(sp, ok_ptr, size, 65, ok_ptr, ok_ptr, None) == binding.ERR_SHAPE
    assert L.ptqtp_gemv_cfg(sp, ok_ptr, size, ok_ptr, ok_ptr, -1, 0, 0, 0, -1, None) == binding.ERR_CONFIG
    assert L.ptqtp_pack(sp, ok_ptr, ok_ptr, ok_ptr, None, ok_ptr, size, None, None) == binding.ERR_NULL
    assert L.ptqtp_pack(sp, ok_ptr, odd_ptr, ok_ptr, ok_ptr, ok_ptr, size, None, None) == binding.ERR_ALIGN
    assert L.ptqtp_unpack(sp, ok_ptr, size - 4, ok_ptr, ok_ptr, ok_ptr, ok_ptr, None, None) == binding.ERR_SIZE
    assert L.ptqtp_gemv_host(sp, ok_ptr, size, None, ok_ptr, ok_ptr, ok_ptr, None) == binding.ERR_NULL
    # gated pair epilogue: format 2 only, an even number of rows
    assert L.ptqtp_gemv_swiglu(sp, ok_ptr, size, None, ok_ptr, None) == binding.ERR_NULL
    assert L.ptqtp_gemv_swiglu(sp, ok_ptr, size, ok_ptr, odd_ptr, None) == binding.ERR_ALIGN
    odd_rows = binding.make_shape(7, 256)
    assert L.ptqtp_gemv_swiglu(ctypes.byref(odd_rows), ok_ptr, size, ok_ptr, ok_ptr, None) == binding.ERR_SHAPE
    v1 = binding.make_shape(8, 256, fmt=binding.FORMAT_V1)
    assert L.ptqtp_gemv_swiglu(ctypes.byref(v1), ok_ptr, binding.packed_size(8, 256, fmt=binding.FORMAT_V1), ok_ptr, ok_ptr,
                               None) == binding.ERR_CONFIG
    # format 1 is a batch-1 layout; the workspace calls read format 2 only
    for fmt in (binding.FORMAT_V1, binding.FORMAT_V3):
        sh = binding.make_shape(8, 256, fmt=fmt)
        sz = binding.packed_size(8, 256, fmt=fmt)
        if fmt == binding.FORMAT_V1:
            assert L.ptqtp_gemm_skinny(ctypes.byref(sh), ok_ptr, sz, 2, ok_ptr, ok_ptr, None) == binding.ERR_CONFIG
        assert L.ptqtp_gemm_skinny_ws(ctypes.byref(sh), ok_ptr, sz, 2, ok_ptr, ok_ptr, ok_ptr, 1 << 20, None) == binding.ERR_CONFIG
        assert L.ptqtp_gemm_skinny_workspace_size(ctypes.byref(sh), 2) == 0
    # the kernel choice of the small-batch call exists for format 3 only; paths 0, 5, 6; splits 0, 1, 2, 4, 8
    s3 = binding.make_shape(8, 256, fmt=binding.FORMAT_V3)
    z3 = binding.packed_size(8, 256, fmt=binding.FORMAT_V3)
    assert L.ptqtp_gemm_skinny_cfg(sp, ok_ptr, size, 8, ok_ptr, ok_ptr, 6, 0, None) == binding.ERR_CONFIG
    assert L.ptqtp_gemm_skinny_cfg(ctypes.byref(s3), ok_ptr, z3, 8, ok_ptr, ok_ptr, 4, 0, None) == binding.ERR_CONFIG
    assert L.ptqtp_gemm_skinny_cfg(ctypes.byref(s3), ok_ptr, z3, 8, ok_ptr, ok_ptr, 6, 3, None) == binding.ERR_CONFIG
    assert L.ptqtp_gemm_skinny_cfg(ctypes.byref(s3), ok_ptr, z3, 0, ok_ptr, ok_ptr, 6, 0, None) == binding.ERR_SHAPE
    assert L.ptqtp_gemm_skinny_cfg(ctypes.byref(s3), ok_ptr, z3, 8, odd_ptr, ok_ptr, 6, 0, None) == binding.ERR_ALIGN
    assert L.ptqtp_gemm_skinny_cfg(ctypes.byref(s3), ok_ptr, z3, 8, None, ok_ptr, 6, 0, None) == binding.ERR_NULL
    assert L.ptqtp_gemm_skinny_cfg(ctypes.byref(s3), ok_ptr, z3 - 16, 8, ok_ptr, ok_ptr, 6, 0, None) == binding.ERR_SIZE


def test_decompose_host_side_checks(L):
    ok_ptr, odd_ptr = ctypes.c_void_p(0x10000), ctypes.c_void_p(0x10008)
    need = L.ptqtp_decompose_workspace_size(8, 256, 128, 50)
    off = binding.DecomposeOffsets()
    assert L.ptqtp_decompose_layout(8, 256, 128, 50, ctypes.byref(off)) == binding.OK
    assert off.total_bytes == need and off.sweeps_offset == 0 and off.delta_offset == 64
    assert off.error_offset == 64 + 51 * 8 and off.alpha2_offset - off.alpha1_offset == 16 * 8
    assert off.lambda_offset + 16 * 8 == need
    assert L.ptqtp_decompose_layout(8, 250, 128, 50, ctypes.byref(off)) == binding.ERR_SHAPE
    args = lambda **kw: [kw.get("W", ok_ptr), 8, kw.get("k", 256), 128, 50, ctypes.c_double(kw.get("eps", 1e-4)), 1, ok_ptr, ok_ptr,
                         kw.get("a1", ok_ptr), ok_ptr, ok_ptr, kw.get("size", need), None]
    assert L.ptqtp_decompose(*args(W=None)) == binding.ERR_NULL
    assert L.ptqtp_decompose(*args(k=200)) == binding.ERR_SHAPE
    assert L.ptqtp_decompose(*args(eps=-1.0)) == binding.ERR_SHAPE
    assert L.ptqtp_decompose(*args(a1=odd_ptr)) == binding.ERR_ALIGN
    assert L.ptqtp_decompose(*args(size=need - 1)) == binding.ERR_SIZE


def test_process_wide_settings_defaults_and_setters(L):
    # plain launches are the default: every buffer, the packed blob included, follows stream order
    assert L.ptqtp_set_overlap(1) == 0
    assert L.ptqtp_set_overlap(7) == 1
    assert L.ptqtp_set_overlap(-3) == 2
    assert L.ptqtp_set_overlap(0) == 0
    assert L.ptqtp_set_wait_limit(1000) == 1 << 22
    assert L.ptqtp_set_wait_limit(0) == 1000
    assert L.ptqtp_set_wait_limit(1 << 22) == 1


def test_status_strings(L):
    seen = set()
    for code in range(0, -9, -1):
        s = binding.status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 9
    assert binding.status_string(-99) == "unknown status"


def test_binding_refuses_cpu_tensors(L):
    import torch
    with pytest.raises(TypeError):
        binding.ptqtp_gemv(torch.zeros(binding.packed_size(8, 128), dtype=torch.uint8), 8, 128,
                           torch.zeros(128, dtype=torch.float16))


def test_reference_format2_roundtrip_layout_and_damage_detection():
    c = make_case(5, 4224, seed=4)                       # odd N, two full slices and a 128-column tail
    blob = pf.pack_reference_v2(c["T1"], c["T2"], c["alpha1"], c["alpha2"])
    t1, t2, a1, a2 = pf.unpack_reference_v2(blob)
    assert np.array_equal(t1, c["T1"]) and np.array_equal(t2, c["T2"])
    assert np.array_equal(a1.view(np.uint16), c["alpha1"].view(np.uint16))
    assert np.array_equal(a2.view(np.uint16), c["alpha2"].view(np.uint16))
    # the body is slice-major: 3 row pairs x 2176 bytes of slice 0, 3 x 2176 of slice 1, 3 x 144 of the tail slice.
    # One byte by hand: row pair 1 (rows 2, 3), column 2048 + 64*3 + 16*2 + 5 = 2277:
    # slice 1, lane block 3, sub-block 2, byte 5 -> unit offset 16 * (2 * 32 + 3) + 5
    run = 3 * 2176
    off = 256 + run + 1 * 2176 + 16 * (2 * 32 + 3) + 5
    want = ((int(c["T1"][2, 2277]) + 1) | (int(c["T2"][2, 2277]) + 1) << 2 | (int(c["T1"][3, 2277]) + 1) << 4
            | (int(c["T2"][3, 2277]) + 1) << 6)
    assert int(blob[off]) == want
    # scale quad of row pair 0, group 17 (slice 1, second group): after the 2048 code bytes of that unit
    q = 256 + run + 2048 + 8 * 1
    assert bytes(blob[q:q + 8]) == (c["alpha1"][0, 17].tobytes() + c["alpha2"][0, 17].tobytes()
                                    + c["alpha1"][1, 17].tobytes() + c["alpha2"][1, 17].tobytes())
    # the tail unit of row pair 0: 128 columns -> 2 lane blocks, 128 code bytes, one quad, 8 bytes of zero padding
    tail = 256 + 2 * run
    assert bytes(blob[tail + 128:tail + 136]) == (c["alpha1"][0, 32].tobytes() + c["alpha2"][0, 32].tobytes()
                                                  + c["alpha1"][1, 32].tobytes() + c["alpha2"][1, 32].tobytes())
    assert not blob[tail + 136:tail + 144].any()
    assert blob.size == 256 + 2 * run + 3 * 144
    # the missing row 5 is trit 0 (code 1) with zero scales: first byte of row pair 2 in slice 0
    last = 256 + 2 * 2176
    assert (int(blob[last]) >> 4) == 0b0101
    bad = blob.copy()
    bad[256] |= 3
    with pytest.raises(ValueError):
        pf.unpack_reference_v2(bad)
    bad = blob.copy()
    bad[tail + 140] = 1
    with pytest.raises(ValueError):
        pf.unpack_reference_v2(bad)


def test_reference_format3_roundtrip_layout_and_damage_detection():
    c = make_case(21, 1152, seed=4)                      # 11 row pairs -> 2 row blocks; 1152 columns -> 3 superblocks
    blob = pf.pack_reference_v3(c["T1"], c["T2"], c["alpha1"], c["alpha2"])
    t1, t2, a1, a2 = pf.unpack_reference_v3(blob)
    assert np.array_equal(t1, c["T1"]) and np.array_equal(t2, c["T2"])
    assert np.array_equal(a1.view(np.uint16), c["alpha1"].view(np.uint16))
    assert np.array_equal(a2.view(np.uint16), c["alpha2"].view(np.uint16))
    assert blob.size == 256 + 2 * 3 * 4352

    def column_byte(rp, col):
        return ((int(c["T1"][2 * rp, col]) + 1) | (int(c["T2"][2 * rp, col]) + 1) << 2
                | (int(c["T1"][2 * rp + 1, col]) + 1) << 4 | (int(c["T2"][2 * rp + 1, col]) + 1) << 6)

    # One byte by hand: row pair 9 (rows 18, 19) = row block 1, g = 1; column 700 = superblock 1, column 188 of it:
    # group 1 (h = 0, t / 2 = 1), column 60 of the group = k-step 7 (chunk 3, s = 1), second half (t % 2 = 1), e = 0
    # -> t = 3, lane 4 * 1 + 3 = 7, byte 512 * 3 + 16 * 7 + 8 * 1 + 4 * 0 + 0 of tile (sb 1, rb 1) = tile number 1 * 2 + 1
    off = 256 + 3 * 4352 + 512 * 3 + 16 * 7 + 8
    assert int(blob[off]) == column_byte(9, 700)
    # column 700 + 256 = 956 is group 3 of the same superblock: h = 1, same lane, four bytes further
    assert int(blob[off + 4]) == column_byte(9, 956)
    # scale quad of row pair 9, group 5 (superblock 1, t = 1): lane 4 * 1 + 1 = 5 of the same tile
    q = 256 + 3 * 4352 + 4096 + 8 * 5
    assert bytes(blob[q:q + 8]) == (c["alpha1"][18, 5].tobytes() + c["alpha2"][18, 5].tobytes()
                                    + c["alpha1"][19, 5].tobytes() + c["alpha2"][19, 5].tobytes())
    # row 21 does not exist: row pair 10 (row block 1, g = 2) has trit 0 (code 1) and zero scales in its upper half
    first = 256 + 1 * 4352 + 16 * (4 * 2 + 0)
    assert (int(blob[first]) >> 4) == 0b0101
    assert not blob[256 + 4352 + 4096 + 8 * 8 + 4:256 + 4352 + 4096 + 8 * 8 + 8].any()
    # columns 1152 .. 1535 of superblock 2 do not exist: group 1 of that superblock (t = 2, 3 with h = 0) holds 0x55
    pad = 256 + (2 * 2 + 0) * 4352 + 16 * 2
    assert int(blob[pad]) == 0x55
    bad = blob.copy()
    bad[256] |= 3
    with pytest.raises(ValueError):
        pf.unpack_reference_v3(bad)
    bad = blob.copy()
    bad[pad] = 0x54
    with pytest.raises(ValueError):
        pf.unpack_reference_v3(bad)


def test_reference_format_roundtrip_and_damage_detection():
    c = make_case(6, 1280, seed=3)
    blob = pf.pack_reference(c["T1"], c["T2"], c["alpha1"], c["alpha2"])
    t1, t2, a1, a2 = pf.unpack_reference(blob)
    assert np.array_equal(t1, c["T1"]) and np.array_equal(t2, c["T2"])
    assert np.array_equal(a1.view(np.uint16), c["alpha1"].view(np.uint16))
    assert np.array_equal(a2.view(np.uint16), c["alpha2"].view(np.uint16))
    # one trit, one bit position: column 37 of row 2, plane 2 -> lane block 1, e = 5, word 2, bits 10..11
    c["T2"][2, 37] = -1
    b2 = pf.pack_reference(c["T1"], c["T2"], c["alpha1"], c["alpha2"])
    off = 256 + (2 * 2 + 0) * 512 + 1 * 16 + 2 * 4
    word = int.from_bytes(bytes(b2[off:off + 4]), "little")
    assert (word >> 10) & 3 == 0
    bad = blob.copy()
    bad[256] |= 3                       # code 3 does not exist
    with pytest.raises(ValueError):
        pf.unpack_reference(bad)
