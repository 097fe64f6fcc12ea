"""An independent reader of the packet stream, written from the format definition
(global header + fixed-size packets; packet = header {s, y_r, centroid distribution} +
(PID, CID) pairs, Fig. 2 of the paper; the centroid distribution is {min, max} for PQ and
{l2-norm, 0} for QSGD), used by the tests to check both encoders.  It shares
no code with the oracle or with the CUDA library."""
from __future__ import annotations

import struct
from dataclasses import dataclass
from typing import List

import numpy as np


@dataclass
class Packet:
    s: int
    y: int
    lo: float
    hi: float
    pid: np.ndarray   # uint64
    cid: np.ndarray   # uint64
    pad_bits_zero: bool


@dataclass
class Stream:
    magic: int
    version: int
    quantizer: int
    s: int
    d: int
    R: int
    packet_bits: int
    header_bits: int
    client_id: int
    seed: int
    round: int
    scale_B: float
    k: int
    packets: List[Packet]


def _bits_of(packet: np.ndarray) -> np.ndarray:
    """bit i of the packet = bit (i mod 8) of byte i // 8 (little-endian words)."""
    return np.unpackbits(packet, bitorder="little")


def _field(bits: np.ndarray, start: int, width: int) -> int:
    v = 0
    for i in range(width):
        v |= int(bits[start + i]) << i
    return v


def parse(stream: np.ndarray) -> Stream:
    raw = np.ascontiguousarray(stream, dtype=np.uint8).tobytes()
    (magic, version, quantizer, s, d, R, packet_bits, header_bits, client_id, seed, rnd, zero, scale_B,
     k) = struct.unpack_from("<IHBBQIIIIQIIdQ", raw, 0)
    assert zero == 0
    out = Stream(magic, version, quantizer, s, d, R, packet_bits, header_bits, client_id, seed, rnd,
                 scale_B, k, [])
    nbytes = packet_bits // 8
    assert len(raw) == 64 + R * nbytes
    for r in range(R):
        pkt = np.frombuffer(raw, dtype=np.uint8, count=nbytes, offset=64 + r * nbytes)
        bits = _bits_of(pkt)
        ps = _field(bits, 0, 8)
        y = _field(bits, 8, 8)
        lo = struct.unpack("<f", struct.pack("<I", _field(bits, 16, 32)))[0]
        hi = struct.unpack("<f", struct.pack("<I", _field(bits, 48, 32)))[0]
        hdr_zero = not bits[80:header_bits].any()
        w = ps + y
        P = (packet_bits - header_bits) // w
        body = bits[header_bits:header_bits + P * w].reshape(P, w).astype(np.uint64)
        wp = (np.uint64(1) << np.arange(ps, dtype=np.uint64))
        wc = (np.uint64(1) << np.arange(y, dtype=np.uint64))
        pid = (body[:, :ps] * wp).sum(axis=1, dtype=np.uint64)
        cid = (body[:, ps:] * wc).sum(axis=1, dtype=np.uint64)
        pad_zero = hdr_zero and not bits[header_bits + P * w:].any()
        out.packets.append(Packet(ps, y, lo, hi, pid, cid, pad_zero))
    return out


def dequantize(pk: Packet) -> np.ndarray:
    """centroid value of each record: uniform grid of 2^y points on [lo, hi]."""
    if pk.hi == pk.lo:
        return np.full(pk.cid.shape, np.float32(pk.lo), dtype=np.float32)
    L = float(2 ** pk.y - 1)
    step = (np.float64(pk.hi) - np.float64(pk.lo)) / L
    return (np.float64(pk.lo) + pk.cid.astype(np.float64) * step).astype(np.float32)


def dequantize_qsgd(pk: Packet) -> np.ndarray:
    """QSGD record: top bit of the CID = sign, the rest = level on a grid of 2^(y-1) - 1 steps
    of the packet's l2-norm (kept in the first centroid field)."""
    sq = 2 ** (pk.y - 1) - 1
    level = (pk.cid & np.uint64(sq)).astype(np.float64)
    negative = ((pk.cid >> np.uint64(pk.y - 1)) & np.uint64(1)).astype(bool)
    mag = (level * (np.float64(pk.lo) / np.float64(sq))).astype(np.float32)
    return np.where(negative, -mag, mag).astype(np.float32)


# ---- unframed stream (version 2) ---------------------------------------------------------------------------------
# header (64 bytes, as version 1 with version = 2) | n_y[33] u32 | cap[33] u32 | total body bits u64 |
# directory: R x u64 bit offsets | body: blocks in descending code length, each {lo 32, hi 32, records in ascending
# position: Golomb-Rice(position - previous position - 1, previous = -1 at the start of a block) then CID (y bits)};
# Rice parameter m = floor(log2(d // P)); a value v is sent as v >> m one-bits, a zero bit, then the low m bits.

@dataclass
class UnframedStream:
    head: Stream                 # packets: one Packet per block (s = 0: the blocks carry no s field)
    total_bits: int
    directory: np.ndarray
    n_y: List[int]
    cap: List[int]
    tail_zero: bool


def parse_unframed(stream: np.ndarray) -> UnframedStream:
    raw = np.ascontiguousarray(stream, dtype=np.uint8).tobytes()
    (magic, version, quantizer, s, d, R, packet_bits, header_bits, client_id, seed, rnd, zero, scale_B,
     k) = struct.unpack_from("<IHBBQIIIIQIIdQ", raw, 0)
    assert version == 2 and zero == 0
    n_y = list(struct.unpack_from("<33I", raw, 64))
    cap = list(struct.unpack_from("<33I", raw, 64 + 132))
    total_bits = struct.unpack_from("<Q", raw, 64 + 264)[0]
    directory = np.frombuffer(raw, dtype="<u8", count=R, offset=64 + 264 + 8).copy()
    head_bytes = 64 + 264 + 8 + 8 * R
    assert len(raw) == head_bytes + ((total_bits + 63) // 64) * 8
    bits = np.unpackbits(np.frombuffer(raw, dtype=np.uint8, offset=head_bytes), bitorder="little")
    out = Stream(magic, version, quantizer, s, d, R, packet_bits, header_bits, client_id, seed, rnd, scale_B, k, [])
    pos, r = 0, 0
    for y in range(32, 0, -1):
        for _ in range(n_y[y]):
            assert directory[r] == pos
            P = cap[y]
            m = max(0, (d // P).bit_length() - 1)
            lo = struct.unpack("<f", struct.pack("<I", _field(bits, pos, 32)))[0]
            hi = struct.unpack("<f", struct.pack("<I", _field(bits, pos + 32, 32)))[0]
            pos += 64
            pids, cids = [], []
            prev = 0
            for _j in range(P):
                q = 0
                while bits[pos]:
                    q += 1
                    pos += 1
                pos += 1
                delta = (q << m) | _field(bits, pos, m)
                pos += m
                cids.append(_field(bits, pos, y))
                pos += y
                pids.append(prev + delta)
                prev = prev + delta + 1
            out.packets.append(Packet(0, y, lo, hi, np.array(pids, dtype=np.uint64), np.array(cids, dtype=np.uint64), True))
            r += 1
    assert pos == total_bits and r == R
    return UnframedStream(out, total_bits, directory, n_y, cap, not bits[pos:].any())
