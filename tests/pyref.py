"""Independent pure-Python statements used to pin the C oracle.

Nothing here is shared with the oracle or with the CUDA library: exact rational
arithmetic for the quantiser (Eq. 2-3), Python big-int strings for the key encoder
(Sec. 3.3) and a second, separately written reader / writer of the stream container.
"""
from __future__ import annotations

import math
import struct
from fractions import Fraction

import numpy as np


# ---------------------------------------------------------------- values

def exact_level(v: float, S: float, b: float, kmax: int = 4096) -> int:
    """ceil(log_b(S/|v|)) in exact rational arithmetic: least k >= 0 with |v| * b^k >= S."""
    a, s, bb = Fraction(abs(float(v))), Fraction(float(S)), Fraction(float(b))
    k, p = 0, Fraction(1)
    while a * p < s:
        p *= bb
        k += 1
        if k > kmax:
            raise OverflowError
    return k


def naive_tree_sum(x: np.ndarray) -> float:
    """Pairwise sum over the zero-padded power-of-two range, level by level (iterative,
    not the oracle's recursion)."""
    a = np.abs(np.asarray(x, np.float32)).astype(np.float64)
    n2 = 1
    while n2 < a.size:
        n2 *= 2
    a = np.concatenate([a, np.zeros(n2 - a.size)])
    while a.size > 1:
        a = a[0::2] + a[1::2]
    return float(a[0]) if a.size else 0.0


# ------------------------------------------------------------------ keys

def bits_of(x: int, width: int) -> str:
    assert 0 <= x < (1 << width) or (width == 0 and x == 0)
    return format(x, "b").zfill(width) if width else ""


def level_widths(M: int, l: int):
    return [-((-(f + 1) * M) // (1 << l)) for f in range(1 << l)]


def alg2_paper(keys, l: int):
    """Algorithm 2: one chain of deltas from 0, one M, BK = flag||delta per key."""
    deltas, pre = [], 0
    for k in keys:
        deltas.append(int(k) - pre)
        pre = int(k)
    M = max(1, max(deltas).bit_length()) if deltas else 1
    w = level_widths(M, l)
    bk = ""
    for dlt in deltas:
        f = next(i for i, wi in enumerate(w) if dlt.bit_length() <= wi)
        bk += bits_of(f, l) + bits_of(dlt, w[f])
    return bk, M


# ------------------------------------------------------------- container

MAGIC = 0x31475346


def write_stream(keys, codes, n: int, S: float, b: float, tau: int, l: int, group_log2: int) -> bytes:
    """Second writer: builds every blob as a Python bit string."""
    T = 1 << group_log2
    G = (n + T - 1) // T
    groups = [[] for _ in range(G)]
    for k, q in zip(keys, codes):
        groups[int(k) >> group_log2].append((int(k), int(q)))
    directory = b""
    blobs = b""
    off = (64 + 8 * G) // 4
    for g, items in enumerate(groups):
        if not items:
            directory += struct.pack("<II", 0, off)
            continue
        pre, deltas = g * T, []
        for k, _ in items:
            deltas.append(k - pre)
            pre = k
        M = max(1, max(deltas).bit_length())
        w = level_widths(M, l)
        flags = [next(i for i, wi in enumerate(w) if dlt.bit_length() <= wi) for dlt in deltas]
        s = "".join(bits_of((0x80 if q < 0 else 0) | (abs(q) - 1), 8) for _, q in items)
        s += "".join(bits_of(f, l) for f in flags)
        s += "".join(bits_of(dlt, w[f]) for dlt, f in zip(deltas, flags))
        s += "0" * (-len(s) % 32)
        blob = int(s, 2).to_bytes(len(s) // 8, "big")
        directory += struct.pack("<II", len(items) | (M << 24), off)
        blobs += blob
        off += len(blob) // 4
    total = 64 + 8 * G + len(blobs)
    header = struct.pack("<IIIIQQQddBBHI", MAGIC, 1, 0, tau, n, len(keys), total, S, b, l, group_log2, 0, G)
    assert len(header) == 64
    return header + directory + blobs


def read_stream(buf: bytes):
    """Second reader -> dict(header fields), keys, signed codes."""
    (magic, ver, status, tau, n, d, total, S, b, l, glog, zero, G) = struct.unpack("<IIIIQQQddBBHI", buf[:64])
    assert magic == MAGIC and ver == 1 and zero == 0
    hdr = dict(status=status, tau=tau, n=n, d=d, total=total, S=S, b=b, l=l, group_log2=glog, G=G)
    keys, codes = [], []
    if status != 0:
        return hdr, keys, codes
    T = 1 << glog
    assert G == (n + T - 1) // T and total == len(buf)
    for g in range(G):
        a, off = struct.unpack_from("<II", buf, 64 + 8 * g)
        count, M = a & 0xFFFFFF, a >> 24
        if count == 0:
            continue
        nxt = struct.unpack_from("<I", buf, 64 + 8 * (g + 1) + 4)[0] if g + 1 < G else total // 4
        blob = buf[4 * off:4 * nxt]
        s = bin(int.from_bytes(blob, "big"))[2:].zfill(8 * len(blob))
        w = level_widths(M, l)
        pos_f, pos_d, pre = 8 * count, 8 * count + l * count, g * T
        for i in range(count):
            c = int(s[8 * i:8 * i + 8], 2)
            f = int(s[pos_f + l * i:pos_f + l * i + l], 2)
            dlt = int(s[pos_d:pos_d + w[f]], 2)
            pos_d += w[f]
            pre += dlt
            keys.append(pre)
            codes.append(-((c & 0x7F) + 1) if c & 0x80 else (c & 0x7F) + 1)
        assert set(s[pos_d:]) <= {"0"} and len(s) - pos_d < 32
    return hdr, keys, codes
