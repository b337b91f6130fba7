"""CPU oracle of the exponent / sign+mantissa Huffman codec — TEST INFRASTRUCTURE ONLY.

Thin ctypes access to ``zc_oracle.c`` (plain single-threaded C, compiled with gcc
into ``libzc_oracle.so`` next to this file).  Only the tests, the smoke check and
the benchmark's CPU-baseline leg may import this package; the CUDA library and
its Python binding never do, and share no code with it.

Every function takes and returns numpy arrays; nothing here knows about CUDA.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

BF16, FP8_E4M3, FP4_E2M1, SCALE_U8, FP8_E5M2 = 1, 2, 3, 4, 5
RAW, HUFF = 0, 1
POLICY_AUTO, POLICY_HUFF_ALL, POLICY_RAW_ALL, POLICY_STATIC = 0, 1, 2, 3
L_MAX = 12

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "zc_oracle.c")
_LIB = os.path.join(_HERE, "libzc_oracle.so")


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc if the shared object is missing or stale."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-Wall", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u8p, u32p, u64p = C.POINTER(C.c_uint8), C.POINTER(C.c_uint32), C.POINTER(C.c_uint64)
        L.zo_bf16_value.restype = C.c_double
        L.zo_bf16_value.argtypes = [C.c_uint16]
        L.zo_e4m3_value.restype = C.c_double
        L.zo_e4m3_value.argtypes = [C.c_uint8]
        L.zo_e5m2_value.restype = C.c_double
        L.zo_e5m2_value.argtypes = [C.c_uint8]
        L.zo_e2m1_value.restype = C.c_double
        L.zo_e2m1_value.argtypes = [C.c_uint8]
        L.zo_group.restype = C.c_int
        L.zo_group.argtypes = [C.c_int]
        L.zo_n_syms.restype = C.c_uint64
        L.zo_n_syms.argtypes = [C.c_int, C.c_uint64]
        L.zo_input_bytes.restype = C.c_uint64
        L.zo_input_bytes.argtypes = [C.c_int, C.c_uint64]
        L.zo_split.restype = None
        L.zo_split.argtypes = [C.c_int, u8p, C.c_uint64, u8p, u8p]
        L.zo_merge.restype = None
        L.zo_merge.argtypes = [C.c_int, u8p, u8p, C.c_uint64, u8p]
        L.zo_histogram.restype = None
        L.zo_histogram.argtypes = [u8p, C.c_uint64, u64p]
        L.zo_code_lengths.restype = C.c_int
        L.zo_code_lengths.argtypes = [u64p, C.c_int, u8p]
        L.zo_static_lengths.restype = C.c_int
        L.zo_static_lengths.argtypes = [u64p, C.c_int, u8p]
        L.zo_dict_wants_rebuild.restype = C.c_int
        L.zo_dict_wants_rebuild.argtypes = [C.c_double, C.c_double, C.c_double]
        L.zo_canonical_codes.restype = None
        L.zo_canonical_codes.argtypes = [u8p, u32p]
        L.zo_payload_bits.restype = C.c_uint64
        L.zo_payload_bits.argtypes = [u64p, u8p]
        L.zo_choose_mode.restype = C.c_int
        L.zo_choose_mode.argtypes = [u64p, u8p, C.c_int]
        L.zo_container_bound.restype = C.c_uint64
        L.zo_container_bound.argtypes = [C.c_int, C.c_uint64, C.c_uint32]
        L.zo_compress.restype = C.c_int64
        L.zo_compress.argtypes = [C.c_int, u8p, C.c_uint64, C.c_uint32, C.POINTER(C.c_int), u8p, u8p, C.c_uint64]
        L.zo_decompress.restype = C.c_int64
        L.zo_decompress.argtypes = [u8p, C.c_uint64, u8p, C.c_uint64]
        L.zo_decompress_chunk.restype = C.c_int64
        L.zo_decompress_chunk.argtypes = [u8p, C.c_uint64, C.c_uint32, u8p, C.c_uint64]
        L.zo_stream_stats_of.restype = None
        L.zo_stream_stats_of.argtypes = [u64p, u8p, C.c_int, C.c_void_p]
        _lib = L
    return _lib


def _p(a: np.ndarray, ty):
    return a.ctypes.data_as(C.POINTER(ty))


def _bytes(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    return a.view(np.uint8).reshape(-1)


# ---- element values -------------------------------------------------------------------------

def bf16_value(bits: int) -> float:
    return lib().zo_bf16_value(bits)


def e4m3_value(bits: int) -> float:
    return lib().zo_e4m3_value(bits)


def e5m2_value(bits: int) -> float:
    return lib().zo_e5m2_value(bits)


def e2m1_value(nibble: int) -> float:
    return lib().zo_e2m1_value(nibble)


# ---- geometry -------------------------------------------------------------------------------

def e5m2_element_fields(data):
    """FP8 E5M2 split the way Sec. 3.2 states it: the 5 exponent bits of every element on one side, the sign and
    the 2 mantissa bits on the other ((sign << 2) | mantissa), one symbol per element.  Returns two uint8 arrays."""
    x = _bytes(data)
    return ((x >> 2) & 0x1F).astype(np.uint8), (((x >> 7) << 2) | (x & 3)).astype(np.uint8)


def e5m2_element_payload_bits(data, L: int = L_MAX):
    """Payload bits of an E5M2 tensor coded per element with that split (an optimal prefix code per stream, length
    limit L, stored at its field width when the code does not save 1/64: the AUTO rule with 5- and 3-bit raw
    symbols).  Returns (exponent bits, sign+mantissa bits).  Plain arithmetic on the two histograms."""
    out = []
    for syms, width in zip(e5m2_element_fields(data), (5, 3)):
        hist = np.bincount(syms, minlength=256).astype(np.uint64)
        coded = payload_bits(hist, code_lengths(hist, L)) if syms.size else 0
        raw = width * int(syms.size)
        out.append(coded if 64 * coded <= 63 * raw else raw)
    return tuple(out)


def group(fmt: int) -> int:
    return lib().zo_group(fmt)


def n_syms(fmt: int, n_elems: int) -> int:
    return lib().zo_n_syms(fmt, n_elems)


def input_bytes(fmt: int, n_elems: int) -> int:
    return lib().zo_input_bytes(fmt, n_elems)


# ---- split / merge / histogram ---------------------------------------------------------------

def split(fmt: int, data, n_elems: int):
    """Return the exponent symbol stream and the sign+mantissa symbol stream."""
    d = _bytes(data)
    assert d.size >= input_bytes(fmt, n_elems)
    ns = n_syms(fmt, n_elems)
    s0 = np.zeros(max(ns, 1), np.uint8)
    s1 = np.zeros(max(ns, 1), np.uint8)
    lib().zo_split(fmt, _p(d, C.c_uint8), n_elems, _p(s0, C.c_uint8), _p(s1, C.c_uint8))
    return s0[:ns], s1[:ns]


def merge(fmt: int, s0, s1, n_elems: int) -> np.ndarray:
    s0 = np.ascontiguousarray(s0, np.uint8)
    s1 = np.ascontiguousarray(s1, np.uint8)
    out = np.zeros(max(input_bytes(fmt, n_elems), 1), np.uint8)
    lib().zo_merge(fmt, _p(s0, C.c_uint8), _p(s1, C.c_uint8), n_elems, _p(out, C.c_uint8))
    return out[: input_bytes(fmt, n_elems)]


def symbol_histogram(syms) -> np.ndarray:
    s = np.ascontiguousarray(syms, np.uint8)
    h = np.zeros(256, np.uint64)
    lib().zo_histogram(_p(s, C.c_uint8), s.size, _p(h, C.c_uint64))
    return h


def histogram(fmt: int, data, n_elems: int) -> np.ndarray:
    """hist[2][256]: counts of each stream's symbols over the whole tensor."""
    s0, s1 = split(fmt, data, n_elems)
    return np.stack([symbol_histogram(s0), symbol_histogram(s1)])


# ---- codebook --------------------------------------------------------------------------------

def code_lengths(hist, L: int = L_MAX) -> np.ndarray:
    h = np.ascontiguousarray(hist, np.uint64)
    assert h.shape == (256,)
    out = np.zeros(256, np.uint8)
    rc = lib().zo_code_lengths(_p(h, C.c_uint64), L, _p(out, C.c_uint8))
    if rc:
        raise ValueError(f"zo_code_lengths failed: {rc}")
    return out


def static_lengths(hist, L: int = L_MAX) -> np.ndarray:
    """Code lengths of a static dictionary (Sec. 3.3): every symbol gets a code."""
    h = np.ascontiguousarray(hist, np.uint64)
    assert h.shape == (256,)
    out = np.zeros(256, np.uint8)
    rc = lib().zo_static_lengths(_p(h, C.c_uint64), L, _p(out, C.c_uint8))
    if rc:
        raise ValueError(f"zo_static_lengths failed: {rc}")
    return out


def canonical_codes(lengths) -> np.ndarray:
    l = np.ascontiguousarray(lengths, np.uint8)
    out = np.zeros(256, np.uint32)
    lib().zo_canonical_codes(_p(l, C.c_uint8), _p(out, C.c_uint32))
    return out


def payload_bits(hist, lengths) -> int:
    h = np.ascontiguousarray(hist, np.uint64)
    l = np.ascontiguousarray(lengths, np.uint8)
    return lib().zo_payload_bits(_p(h, C.c_uint64), _p(l, C.c_uint8))


def choose_mode(hist, lengths, policy: int) -> int:
    h = np.ascontiguousarray(hist, np.uint64)
    l = np.ascontiguousarray(lengths, np.uint8)
    return lib().zo_choose_mode(_p(h, C.c_uint64), _p(l, C.c_uint8), policy)


@dataclass
class Codebook:
    modes: list          # [2] RAW / HUFF
    lengths: np.ndarray  # [2][256] u8
    codes: np.ndarray    # [2][256] u32


def build_codebook(hist2, policy: int = POLICY_AUTO) -> Codebook:
    hist2 = np.ascontiguousarray(hist2, np.uint64).reshape(2, 256)
    lens = np.stack([(static_lengths if policy == POLICY_STATIC else code_lengths)(hist2[s]) for s in range(2)])
    codes = np.stack([canonical_codes(lens[s]) for s in range(2)])
    modes = [choose_mode(hist2[s], lens[s], policy) for s in range(2)]
    return Codebook(modes, lens, codes)


class StaticDictionary:
    """A precomputed dictionary for K/V cache tensors and the rule that replaces it (Sec. 3.3): built from the
    histogram of a representative tensor, reused for the tensors that follow, replaced when a tensor's ratio
    (container bytes / input bytes) exceeds the baseline by more than `tolerance` (relative)."""

    def __init__(self, hist2, tolerance: float):
        self.tolerance = float(tolerance)
        self.codebook = build_codebook(hist2, POLICY_STATIC)
        self.baseline = None
        self.n_rebuilds = 0

    def observe(self, input_bytes: int, container_bytes: int) -> bool:
        ratio = container_bytes / input_bytes
        if self.baseline is None:
            self.baseline = ratio
            return False
        return bool(lib().zo_dict_wants_rebuild(self.baseline, ratio, self.tolerance))

    def rebuild(self, hist2) -> None:
        self.codebook = build_codebook(hist2, POLICY_STATIC)
        self.baseline = None
        self.n_rebuilds += 1


# ---- container -------------------------------------------------------------------------------

def container_bound(fmt: int, n_elems: int, chunk_bytes: int) -> int:
    return lib().zo_container_bound(fmt, n_elems, chunk_bytes)


def compress(fmt: int, data, n_elems: int, chunk_bytes: int, cb: Codebook) -> np.ndarray:
    d = _bytes(data)
    if d.size == 0:
        d = np.zeros(1, np.uint8)
    cap = container_bound(fmt, n_elems, chunk_bytes)
    if cap == 0:
        raise ValueError("bad format or chunk size")
    out = np.zeros(cap, np.uint8)
    modes = (C.c_int * 2)(*cb.modes)
    lens = np.ascontiguousarray(cb.lengths, np.uint8).reshape(2, 256)
    n = lib().zo_compress(fmt, _p(d, C.c_uint8), n_elems, chunk_bytes, modes, _p(lens, C.c_uint8),
                          _p(out, C.c_uint8), cap)
    if n < 0:
        raise ValueError(f"zo_compress failed: {n}")
    return out[:n].copy()


def decompress(container, out_bytes: int) -> np.ndarray:
    c = np.ascontiguousarray(container, np.uint8)
    out = np.zeros(max(out_bytes, 1), np.uint8)
    n = lib().zo_decompress(_p(c, C.c_uint8), c.size, _p(out, C.c_uint8), out_bytes)
    if n < 0:
        raise ValueError(f"zo_decompress failed: {n}")
    return out[:n]


def decompress_chunk(container, chunk: int, chunk_bytes: int) -> np.ndarray:
    c = np.ascontiguousarray(container, np.uint8)
    out = np.zeros(chunk_bytes, np.uint8)
    n = lib().zo_decompress_chunk(_p(c, C.c_uint8), c.size, chunk, _p(out, C.c_uint8), chunk_bytes)
    if n < 0:
        raise ValueError(f"zo_decompress_chunk failed: {n}")
    return out[:n]


# ---- stats -----------------------------------------------------------------------------------

class _StreamStats(C.Structure):
    _fields_ = [("n_syms", C.c_uint64), ("raw_bits", C.c_uint64), ("payload_bits", C.c_uint64),
                ("mode", C.c_uint32), ("n_active", C.c_uint32), ("max_len", C.c_uint32), ("pad", C.c_uint32),
                ("avg_len", C.c_double), ("entropy_bits", C.c_double)]


def stream_stats(hist, lengths, mode: int) -> dict:
    h = np.ascontiguousarray(hist, np.uint64)
    l = np.ascontiguousarray(lengths, np.uint8)
    st = _StreamStats()
    lib().zo_stream_stats_of(_p(h, C.c_uint64), _p(l, C.c_uint8), mode, C.byref(st))
    return {k: getattr(st, k) for k, _ in _StreamStats._fields_ if k != "pad"}


def read_tables(container, stream: int):
    """chunk_off16[n_chunks] and sub_end[n_chunks][32] of a HUFF stream as int64 arrays (plain unpacking)."""
    hd = parse_header(container)
    c = np.ascontiguousarray(container, np.uint8)
    sec, nc, w = hd["streams"][stream]["section_off"], hd["n_chunks"], hd["sub_end_bytes"]
    off16 = np.frombuffer(c[sec + 256: sec + 256 + 4 * nc].tobytes(), "<u4").astype(np.int64)
    tab = sec + 256 + ((4 * nc + 15) // 16) * 16
    sub_end = np.frombuffer(c[tab: tab + 32 * w * nc].tobytes(), "<u2" if w == 2 else "<u4").reshape(nc, 32).astype(np.int64)
    return off16, sub_end, tab


def parse_header(container) -> dict:
    """Decode the 128-byte header into a dict (plain struct unpacking, for tests and reports)."""
    import struct
    b = bytes(np.ascontiguousarray(container, np.uint8)[:128])
    magic, version, fmt, n_streams, n_elems, chunk_bytes, n_chunks, lmax, g, subs, sub_w = struct.unpack_from(
        "<4sHBBQIIBBBB", b, 0)
    total, payload_off, payload_bytes = struct.unpack_from("<QQQ", b, 32)
    streams = []
    for s in range(2):
        mode, = struct.unpack_from("<B", b, 64 + 32 * s)
        ns, pbits, sec = struct.unpack_from("<QQQ", b, 64 + 32 * s + 8)
        streams.append(dict(mode=mode, n_syms=ns, payload_bits=pbits, section_off=sec))
    return dict(magic=magic, version=version, format=fmt, n_streams=n_streams, n_elems=n_elems,
                chunk_bytes=chunk_bytes, n_chunks=n_chunks, l_max=lmax, group=g, subchunks=subs, sub_end_bytes=sub_w,
                total_bytes=total, payload_off=payload_off, payload_bytes=payload_bytes, streams=streams)
