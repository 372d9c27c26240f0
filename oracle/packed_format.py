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
