"""Byte-level writer/reader of the packed-plane blob, from the format's description.  Test infrastructure only.

Format "PTQTP-B200 v1" (storage model of Appendix B "Memory Saving": 2 bits per trit per plane and
one fp16 scale per plane per 128-column group):

  bytes [0, 256)   header: b"PTQTPB2\\0", u32 version = 1, u32 format = 1, i32 N, i32 K, i32 group = 128,
                   i32 K_pad, u64 codes offset, u64 scales offset, u64 total size; rest zero
  codes            for each row i, for each 1024-column slice s: 512 bytes = 32 lane blocks of 16 bytes.
                   Lane block l holds columns s*1024 + 32*l + e (e = 0..31) as 4 little-endian u32:
                   word 0 = plane 1, e 0..15; word 1 = plane 1, e 16..31; word 2, 3 = plane 2 likewise.
                   Inside a word, offset e' = e mod 16 occupies bits [16*(e'//8) + 2*(e'%8), +2) with the
                   code trit + 1.  Columns >= K (padding up to a multiple of 1024) hold trit 0.
  scales           for each row i, for each group g < K_pad/128: u16 alpha1 bits, u16 alpha2 bits
                   (zero for padding groups).

Format 2 (same header with format = 2; the K_pad slot holds 2048 * ceil(K/2048), the scales-offset slot the
bytes of one row pair over all slices):

  body             for each slice s of up to 2048 columns, for each row pair p (rows 2p, 2p+1; a missing odd row
                   counts as trit 0, scales 0), one unit with A = columns/64 lane blocks: 4*A atoms of 16 bytes, atom
                   (i, l) at byte 16*(i*A + l) holding columns 2048 s + 64 l + 16 i + e (e = 0..15), one byte
                   per column = code(2p, plane 1) | code(2p, plane 2) << 2 | code(2p+1, plane 1) << 4
                   | code(2p+1, plane 2) << 6; then A/2 quads of 4 little-endian u16 (alpha1[2p], alpha2[2p],
                   alpha1[2p+1], alpha2[2p+1]) for the slice's 128-column groups; then zero padding to a
                   multiple of 16 bytes.

Format 3 (same header with format = 3; the K_pad slot holds 512 * ceil(K/512), the scales-offset slot the bytes of
one tile, 4352):

  body             tiles of 8 row pairs (16 rows) x 512 columns (four 128-column groups), 4352 bytes each, stored
                   superblock-major: tile (sb, rb) -- columns 512 sb .., row pairs 8 rb .. -- at byte
                   256 + (sb * ceil(ceil(N/2)/8) + rb) * 4352.  Rows >= N and columns >= K count as trit 0 with
                   scales 0.  A tile is 8 chunks of 512 bytes, then 32 scale quads of 8 bytes.  Chunk c holds,
                   for l = 4 g + t (g = 0..7 the row pair within the tile, t = 0..3), 16 bytes at 512 c + 16 l:
                   four little-endian words (s, h), s = 0, 1, h = 0, 1, at byte 8 s + 4 h; byte e of word (s, h)
                   is the column byte (as in format 2: code(2p, plane 1) | code(2p, plane 2) << 2 |
                   code(2p+1, plane 1) << 4 | code(2p+1, plane 2) << 6) of row pair p = 8 rb + g and column
                   512 sb + 128 (2 h + t // 2) + 8 (2 c + s) + 4 (t % 2) + e.  Scale quad l = 4 g + t at byte
                   4096 + 8 l: alpha1[2p], alpha2[2p], alpha1[2p+1], alpha2[2p+1] (u16 each) of group 4 sb + t.

Written independently of the CUDA pack/unpack kernels (plain numpy bit operations) so that the two
can be compared byte for byte.
"""
import struct

import numpy as np

HEADER_BYTES = 256
MAGIC = b"PTQTPB2\x00"


def layout(N, K):
    if N <= 0 or K <= 0 or K % 128:
        raise ValueError("N > 0 and K a positive multiple of 128 required")
    K_pad = (K + 1023) // 1024 * 1024
    codes_off = HEADER_BYTES
    scales_off = codes_off + N * (K_pad // 1024) * 512
    total = scales_off + N * (K_pad // 128) * 4
    return dict(N=N, K=K, K_pad=K_pad, codes_off=codes_off, scales_off=scales_off, total=total)


def memory_formula_bits(N, K, G=128):
    """Appendix B: M_PTQTP = 2*n*d*2 + ceil(d/k)*2n*16 bits."""
    return 2 * N * K * 2 + -(-K // G) * 2 * N * 16


def _bit_positions():
    # for column offset e (0..31) of a lane block and plane p: (word index, bit position)
    pos = np.zeros((2, 32, 2), dtype=np.int64)
    for p in range(2):
        for e in range(32):
            word = 2 * p + e // 16
            e16 = e % 16
            pos[p, e] = (word, 16 * (e16 // 8) + 2 * (e16 % 8))
    return pos


def pack_reference(T1, T2, alpha1, alpha2):
    """Planes int8 [N,K], scales fp16 [N,K/128] -> blob (numpy uint8)."""
    T1 = np.asarray(T1, dtype=np.int8)
    T2 = np.asarray(T2, dtype=np.int8)
    N, K = T1.shape
    L = layout(N, K)
    if np.any(np.abs(T1) > 1) or np.any(np.abs(T2) > 1):
        raise ValueError("trit out of range")
    blob = np.zeros(L["total"], dtype=np.uint8)
    hdr = MAGIC + struct.pack("<IIiiiiQQQ", 1, 1, N, K, 128, L["K_pad"], L["codes_off"], L["scales_off"],
                              L["total"])
    blob[:len(hdr)] = np.frombuffer(hdr, dtype=np.uint8)
    Kp = L["K_pad"]
    words = np.zeros((N, Kp // 32, 4), dtype=np.uint64)
    pos = _bit_positions()
    for p, T in enumerate((T1, T2)):
        q = np.ones((N, Kp), dtype=np.uint64)                 # padding: trit 0 -> code 1
        q[:, :K] = (T.astype(np.int64) + 1).astype(np.uint64)
        q = q.reshape(N, Kp // 32, 32)
        for e in range(32):
            word, bit = pos[p, e]
            words[:, :, word] |= q[:, :, e] << np.uint64(bit)
    blob[L["codes_off"]:L["scales_off"]] = words.astype("<u4").reshape(-1).view(np.uint8)
    sc = np.zeros((N, Kp // 128, 2), dtype="<u2")
    sc[:, :K // 128, 0] = np.asarray(alpha1, dtype=np.float16).view(np.uint16)
    sc[:, :K // 128, 1] = np.asarray(alpha2, dtype=np.float16).view(np.uint16)
    blob[L["scales_off"]:] = sc.reshape(-1).view(np.uint8)
    return blob


def parse_header(blob):
    hdr = bytes(np.asarray(blob[:HEADER_BYTES], dtype=np.uint8))
    if hdr[:8] != MAGIC:
        raise ValueError("bad magic")
    version, fmt, N, K, group, K_pad, codes_off, scales_off, total = struct.unpack("<IIiiiiQQQ", hdr[8:56])
    if version != 1 or fmt != 1 or group != 128:
        raise ValueError("bad version/format/group")
    if any(hdr[56:]):
        raise ValueError("header padding not zero")
    return dict(N=N, K=K, K_pad=K_pad, codes_off=codes_off, scales_off=scales_off, total=total)


def unpack_reference(blob):
    """blob (numpy uint8) -> T1, T2 int8 [N,K], alpha1, alpha2 fp16 [N,K/128]."""
    blob = np.asarray(blob, dtype=np.uint8)
    H = parse_header(blob)
    N, K, Kp = H["N"], H["K"], H["K_pad"]
    L = layout(N, K)
    if any(H[k] != L[k] for k in ("K_pad", "codes_off", "scales_off", "total")) or blob.size < L["total"]:
        raise ValueError("header inconsistent with its shape")
    words = blob[L["codes_off"]:L["scales_off"]].view("<u4").astype(np.uint64).reshape(N, Kp // 32, 4)
    pos = _bit_positions()
    planes = []
    for p in range(2):
        q = np.zeros((N, Kp // 32, 32), dtype=np.int64)
        for e in range(32):
            word, bit = pos[p, e]
            q[:, :, e] = ((words[:, :, word] >> np.uint64(bit)) & np.uint64(3)).astype(np.int64)
        if np.any(q == 3):
            raise ValueError("code 3 found")
        q = q.reshape(N, Kp)
        if np.any(q[:, K:] != 1):
            raise ValueError("padding columns must hold trit 0")
        planes.append((q[:, :K] - 1).astype(np.int8))
    sc = blob[L["scales_off"]:L["total"]].view("<u2").reshape(N, Kp // 128, 2)
    if np.any(sc[:, K // 128:, :] != 0):
        raise ValueError("padding scales must be zero")
    a1 = sc[:, :K // 128, 0].copy().view(np.float16)
    a2 = sc[:, :K // 128, 1].copy().view(np.float16)
    return planes[0], planes[1], a1, a2


# ----------------------------------------------------------------------------- format 2
def layout_v2(N, K):
    if N <= 0 or K <= 0 or K % 128:
        raise ValueError("N > 0 and K a positive multiple of 128 required")
    nrp = (N + 1) // 2
    slices = (K + 2047) // 2048
    units = []                                   # (first column, columns, byte offset of the slice's run, unit bytes)
    off = 0
    strip = 0
    for sl in range(slices):
        cols = min(2048, K - 2048 * sl)
        size = -(-(cols + cols // 16) // 16) * 16
        units.append((2048 * sl, cols, off, size))
        off += nrp * size                        # slice-major: the units of a slice for all row pairs are contiguous
        strip += size
    return dict(N=N, K=K, nrp=nrp, slices=slices, units=units, strip=strip, codes_off=HEADER_BYTES,
                total=HEADER_BYTES + off)


def pack_reference_v2(T1, T2, alpha1, alpha2):
    """Planes int8 [N,K], scales fp16 [N,K/128] -> format-2 blob (numpy uint8)."""
    T1 = np.asarray(T1, dtype=np.int8)
    T2 = np.asarray(T2, dtype=np.int8)
    N, K = T1.shape
    L = layout_v2(N, K)
    if np.any(np.abs(T1) > 1) or np.any(np.abs(T2) > 1):
        raise ValueError("trit out of range")
    nrp = L["nrp"]
    q = np.ones((2, 2 * nrp, K), dtype=np.uint8)                  # [plane, row, column]; a missing row is trit 0
    q[0, :N] = (T1.astype(np.int16) + 1).astype(np.uint8)
    q[1, :N] = (T2.astype(np.int16) + 1).astype(np.uint8)
    col_byte = (q[0, 0::2] | (q[1, 0::2] << 2) | (q[0, 1::2] << 4) | (q[1, 1::2] << 6)).astype(np.uint8)
    sc = np.zeros((2 * nrp, K // 128, 2), dtype="<u2")             # [row, group, plane]
    sc[:N, :, 0] = np.asarray(alpha1, dtype=np.float16).view(np.uint16)
    sc[:N, :, 1] = np.asarray(alpha2, dtype=np.float16).view(np.uint16)
    quads = np.concatenate([sc[0::2], sc[1::2]], axis=2)           # [row pair, group, 4]
    blob = np.zeros(L["total"], dtype=np.uint8)
    hdr = MAGIC + struct.pack("<IIiiiiQQQ", 1, 2, N, K, 128, 2048 * L["slices"], L["codes_off"], L["strip"],
                              L["total"])
    blob[:len(hdr)] = np.frombuffer(hdr, dtype=np.uint8)
    for c0, cols, off, size in L["units"]:
        A = cols // 64
        run = blob[L["codes_off"] + off:L["codes_off"] + off + nrp * size].reshape(nrp, size)   # one unit per row pair
        atoms = col_byte[:, c0:c0 + cols].reshape(nrp, A, 4, 16)   # [row pair, lane block, i, e]
        run[:, :4 * A * 16] = atoms.transpose(0, 2, 1, 3).reshape(nrp, -1)
        g0 = c0 // 128
        run[:, 64 * A:64 * A + 4 * A] = (
            np.ascontiguousarray(quads[:, g0:g0 + A // 2]).reshape(nrp, -1).view(np.uint8))
    return blob


def unpack_reference_v2(blob):
    """Format-2 blob (numpy uint8) -> T1, T2 int8 [N,K], alpha1, alpha2 fp16 [N,K/128]."""
    blob = np.asarray(blob, dtype=np.uint8)
    hdr = bytes(blob[:HEADER_BYTES])
    if hdr[:8] != MAGIC:
        raise ValueError("bad magic")
    version, fmt, N, K, group, K_pad, codes_off, stride, total = struct.unpack("<IIiiiiQQQ", hdr[8:56])
    if version != 1 or fmt != 2 or group != 128 or any(hdr[56:]):
        raise ValueError("bad version/format/group")
    L = layout_v2(N, K)
    if (K_pad, codes_off, stride, total) != (2048 * L["slices"], L["codes_off"], L["strip"], L["total"]):
        raise ValueError("header inconsistent with its shape")
    if blob.size < L["total"]:
        raise ValueError("blob too small")
    nrp = L["nrp"]
    col_byte = np.zeros((nrp, K), dtype=np.uint8)
    quads = np.zeros((nrp, K // 128, 4), dtype="<u2")
    for c0, cols, off, size in L["units"]:
        A = cols // 64
        run = blob[L["codes_off"] + off:L["codes_off"] + off + nrp * size].reshape(nrp, size)   # one unit per row pair
        atoms = run[:, :4 * A * 16].reshape(nrp, 4, A, 16)
        col_byte[:, c0:c0 + cols] = atoms.transpose(0, 2, 1, 3).reshape(nrp, cols)
        g0 = c0 // 128
        quads[:, g0:g0 + A // 2] = np.ascontiguousarray(run[:, 64 * A:68 * A]).view("<u2").reshape(nrp, A // 2, 4)
        if np.any(run[:, 68 * A:size] != 0):
            raise ValueError("unit padding must be zero")
    planes = []
    for plane in range(2):
        t = np.zeros((2 * nrp, K), dtype=np.int16)
        for r in range(2):
            code = (col_byte >> (4 * r + 2 * plane)) & 3
            if np.any(code == 3):
                raise ValueError("code 3 found")
            t[r::2] = code.astype(np.int16) - 1
        if 2 * nrp > N and np.any(t[N:] != 0):
            raise ValueError("the missing odd row must hold trit 0")
        planes.append(t[:N].astype(np.int8))
    if 2 * nrp > N and np.any(quads[-1, :, 2:] != 0):
        raise ValueError("the missing odd row must have zero scales")
    a1 = np.zeros((2 * nrp, K // 128), dtype=np.uint16)
    a2 = np.zeros((2 * nrp, K // 128), dtype=np.uint16)
    a1[0::2], a2[0::2], a1[1::2], a2[1::2] = quads[:, :, 0], quads[:, :, 1], quads[:, :, 2], quads[:, :, 3]
    return planes[0], planes[1], a1[:N].view(np.float16), a2[:N].view(np.float16)


# ----------------------------------------------------------------------------- format 3
TILE_V3 = 4352


def layout_v3(N, K):
    if N <= 0 or K <= 0 or K % 128:
        raise ValueError("N > 0 and K a positive multiple of 128 required")
    nrp = (N + 1) // 2
    nrb = (nrp + 7) // 8
    sbs = (K + 511) // 512
    return dict(N=N, K=K, nrp=nrp, nrb=nrb, sbs=sbs, codes_off=HEADER_BYTES,
                total=HEADER_BYTES + nrb * sbs * TILE_V3)


def _tile_maps_v3():
    """For every code byte of a tile: (row pair within the tile, column within the superblock); for every scale
    quad: (row pair within the tile, group within the superblock).  Written out from the format description."""
    rp = np.zeros(4096, dtype=np.int64)
    col = np.zeros(4096, dtype=np.int64)
    for c in range(8):
        for g in range(8):
            for t in range(4):
                for s in range(2):
                    for h in range(2):
                        for e in range(4):
                            b = 512 * c + 16 * (4 * g + t) + 8 * s + 4 * h + e
                            rp[b] = g
                            col[b] = 128 * (2 * h + t // 2) + 8 * (2 * c + s) + 4 * (t % 2) + e
    qrp = np.repeat(np.arange(8), 4)
    qgrp = np.tile(np.arange(4), 8)
    return rp, col, qrp, qgrp


def pack_reference_v3(T1, T2, alpha1, alpha2):
    """Planes int8 [N,K], scales fp16 [N,K/128] -> format-3 blob (numpy uint8)."""
    T1 = np.asarray(T1, dtype=np.int8)
    T2 = np.asarray(T2, dtype=np.int8)
    N, K = T1.shape
    L = layout_v3(N, K)
    if np.any(np.abs(T1) > 1) or np.any(np.abs(T2) > 1):
        raise ValueError("trit out of range")
    nrb, sbs = L["nrb"], L["sbs"]
    rows, cols = 16 * nrb, 512 * sbs
    q = np.ones((2, rows, cols), dtype=np.uint8)                   # [plane, row, column]; padding is trit 0
    q[0, :N, :K] = (T1.astype(np.int16) + 1).astype(np.uint8)
    q[1, :N, :K] = (T2.astype(np.int16) + 1).astype(np.uint8)
    col_byte = (q[0, 0::2] | (q[1, 0::2] << 2) | (q[0, 1::2] << 4) | (q[1, 1::2] << 6)).astype(np.uint8)
    sc = np.zeros((rows, 4 * sbs, 2), dtype="<u2")                 # [row, group, plane]
    sc[:N, :K // 128, 0] = np.asarray(alpha1, dtype=np.float16).view(np.uint16)
    sc[:N, :K // 128, 1] = np.asarray(alpha2, dtype=np.float16).view(np.uint16)
    quads = np.concatenate([sc[0::2], sc[1::2]], axis=2)           # [row pair, group, 4]
    blob = np.zeros(L["total"], dtype=np.uint8)
    hdr = MAGIC + struct.pack("<IIiiiiQQQ", 1, 3, N, K, 128, 512 * sbs, L["codes_off"], TILE_V3, L["total"])
    blob[:len(hdr)] = np.frombuffer(hdr, dtype=np.uint8)
    rp, col, qrp, qgrp = _tile_maps_v3()
    for sb in range(sbs):
        for rb in range(nrb):
            off = HEADER_BYTES + (sb * nrb + rb) * TILE_V3
            blob[off:off + 4096] = col_byte[8 * rb + rp, 512 * sb + col]
            blob[off + 4096:off + TILE_V3] = np.ascontiguousarray(quads[8 * rb + qrp, 4 * sb + qgrp]).reshape(-1).view(np.uint8)
    return blob


def unpack_reference_v3(blob):
    """Format-3 blob (numpy uint8) -> T1, T2 int8 [N,K], alpha1, alpha2 fp16 [N,K/128]."""
    blob = np.asarray(blob, dtype=np.uint8)
    hdr = bytes(blob[:HEADER_BYTES])
    if hdr[:8] != MAGIC:
        raise ValueError("bad magic")
    version, fmt, N, K, group, K_pad, codes_off, tile, total = struct.unpack("<IIiiiiQQQ", hdr[8:56])
    if version != 1 or fmt != 3 or group != 128 or any(hdr[56:]):
        raise ValueError("bad version/format/group")
    L = layout_v3(N, K)
    if (K_pad, codes_off, tile, total) != (512 * L["sbs"], L["codes_off"], TILE_V3, L["total"]):
        raise ValueError("header inconsistent with its shape")
    if blob.size < L["total"]:
        raise ValueError("blob too small")
    nrb, sbs = L["nrb"], L["sbs"]
    col_byte = np.zeros((8 * nrb, 512 * sbs), dtype=np.uint8)
    quads = np.zeros((8 * nrb, 4 * sbs, 4), dtype="<u2")
    rp, col, qrp, qgrp = _tile_maps_v3()
    for sb in range(sbs):
        for rb in range(nrb):
            off = HEADER_BYTES + (sb * nrb + rb) * TILE_V3
            col_byte[8 * rb + rp, 512 * sb + col] = blob[off:off + 4096]
            quads[8 * rb + qrp, 4 * sb + qgrp] = blob[off + 4096:off + TILE_V3].view("<u2").reshape(32, 4)
    t = np.zeros((2, 16 * nrb, 512 * sbs), dtype=np.int16)
    for plane in range(2):
        for r in range(2):
            code = (col_byte >> (4 * r + 2 * plane)) & 3
            if np.any(code == 3):
                raise ValueError("code 3 found")
            t[plane, r::2] = code.astype(np.int16) - 1
    if np.any(t[:, N:] != 0) or np.any(t[:, :, K:] != 0):
        raise ValueError("padding rows and columns must hold trit 0")
    a = np.zeros((2, 16 * nrb, 4 * sbs), dtype=np.uint16)
    a[0, 0::2], a[1, 0::2], a[0, 1::2], a[1, 1::2] = quads[:, :, 0], quads[:, :, 1], quads[:, :, 2], quads[:, :, 3]
    if np.any(a[:, N:] != 0) or np.any(a[:, :, K // 128:] != 0):
        raise ValueError("padding scales must be zero")
    return (t[0, :N, :K].astype(np.int8), t[1, :N, :K].astype(np.int8),
            np.ascontiguousarray(a[0, :N, :K // 128]).view(np.float16), np.ascontiguousarray(a[1, :N, :K // 128]).view(np.float16))
