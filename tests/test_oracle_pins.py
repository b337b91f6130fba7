"""Pins of the CPU oracle against facts it does not define itself.

Each test ties one oracle function to something fixed by the paper's statement of
the formats, by coding theory, or by an independent library routine, so that a
dropped term, a wrong bit position or a swapped operand fails at least one test.
"""
import heapq
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle as zo

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
FORMATS = [zo.BF16, zo.FP8_E4M3, zo.FP4_E2M1, zo.SCALE_U8, zo.FP8_E5M2]


# --------------------------------------------------------------------------------------------
# element formats and field split
# --------------------------------------------------------------------------------------------

def _golden_format_rows():
    rows = []
    for line in open(os.path.join(GOLDEN, "format_values.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        fmt, bits, val, e, sm = line.split()
        rows.append((fmt, int(bits, 16), float(val), int(e), int(sm, 16)))
    return rows


@pytest.mark.parametrize("row", _golden_format_rows(), ids=lambda r: f"{r[0]}_{r[1]:X}")
def test_golden_bit_patterns(row):
    fmt, bits, val, e, sm = row
    if fmt == "bf16":
        got = zo.bf16_value(bits)
        s0, s1 = zo.split(zo.BF16, np.array([bits], np.uint16), 1)
    elif fmt == "e4m3":
        got = zo.e4m3_value(bits)
        s0, s1 = zo.split(zo.FP8_E4M3, np.array([bits], np.uint8), 1)
    else:
        got = zo.e2m1_value(bits)
        s0, s1 = zo.split(zo.FP4_E2M1, np.array([bits], np.uint8), 2)   # second element = 0
    assert got == val and math.copysign(1, got) == math.copysign(1, val)
    assert (int(s0[0]), int(s1[0])) == (e, sm)


def test_bf16_values_match_torch_for_all_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    ref = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    got = np.array([zo.bf16_value(int(b)) for b in bits])
    assert np.array_equal(np.isnan(ref), np.isnan(got))
    ok = ~np.isnan(ref)
    assert np.array_equal(ref[ok], got[ok])
    assert np.array_equal(np.signbit(ref[ok]), np.signbit(got[ok]))


def test_e4m3_values_match_torch_for_all_patterns():
    bits = np.arange(256, dtype=np.uint8)
    ref = torch.from_numpy(bits.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = np.array([zo.e4m3_value(int(b)) for b in bits])
    assert np.array_equal(np.isnan(ref), np.isnan(got))
    ok = ~np.isnan(ref)
    assert np.array_equal(ref[ok], got[ok])
    assert got[0x7E] == 448.0 and np.nanmax(got) == 448.0


def test_e5m2_values_match_torch_for_all_patterns():
    bits = np.arange(256, dtype=np.uint8)
    ref = torch.from_numpy(bits.copy()).view(torch.float8_e5m2).to(torch.float64).numpy()
    got = np.array([zo.e5m2_value(int(b)) for b in bits])
    assert np.array_equal(np.isnan(ref), np.isnan(got))
    ok = ~np.isnan(ref)
    assert np.array_equal(ref[ok], got[ok])
    assert got[0x7B] == 57344.0 and got[0x7C] == np.inf and got[0x01] == 2.0 ** -16


def test_split_fields_rebuild_the_value_e5m2():
    """E5M2 (Sec. 3.2): the coded field holds the upper four exponent bits, the other field sign, lowest exponent
    bit and mantissa; read back that way the two fields give the element's value for every pattern."""
    bits = np.arange(256, dtype=np.uint8)
    data = np.stack([bits, bits[::-1]], axis=1).reshape(-1)
    hi, rest = zo.split(zo.FP8_E5M2, data, data.size)
    ref = torch.from_numpy(data.copy()).view(torch.float8_e5m2).to(torch.float64).numpy()
    for half, sl in ((0, slice(0, None, 2)), (1, slice(1, None, 2))):
        e_hi = ((hi >> (4 * half)) & 0xF).astype(np.int64)
        f = (rest >> (4 * half)) & 0xF
        s = f >> 3
        ee = 2 * e_hi + ((f >> 2) & 1)
        m = (f & 3).astype(np.float64)
        val = np.where(ee == 0, np.ldexp(m / 4.0, -14), np.ldexp(1.0 + m / 4.0, ee - 15))
        val = np.where(s == 1, -val, val)
        r = ref[sl]
        ok = np.isfinite(r)
        assert np.array_equal(val[ok], r[ok])
        assert (ee[~ok] == 31).all()
    # 1.0 = 0 01111 00 (0x3C) and -2^-14 = 1 00001 00 (0x84): upper exponent bits 7 and 0, rest 0100 and 1100
    hi, rest = zo.split(zo.FP8_E5M2, np.array([0x3C, 0x84], np.uint8), 2)
    assert (int(hi[0]), int(rest[0])) == (0x07, 0xC4)


def test_e2m1_value_set():
    assert [zo.e2m1_value(i) for i in range(8)] == [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    assert [zo.e2m1_value(8 + i) for i in range(1, 8)] == [-0.5, -1.0, -1.5, -2.0, -3.0, -4.0, -6.0]


def test_split_fields_rebuild_the_value_bf16():
    """The two fields, read as sign / biased exponent / mantissa, must give the element's value."""
    bits = np.arange(65536, dtype=np.uint16)
    e, sm = zo.split(zo.BF16, bits, bits.size)
    e = e.astype(np.int64); s = sm >> 7; m = (sm & 0x7F).astype(np.float64)
    normal = (e > 0) & (e < 255)
    val = np.where(e == 0, np.ldexp(m / 128.0, -126), np.ldexp(1.0 + m / 128.0, np.clip(e, 1, 254) - 127))
    val = np.where(s == 1, -val, val)
    ref = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    sel = normal | (e == 0)
    assert np.array_equal(val[sel], ref[sel])


def test_split_fields_rebuild_the_value_fp8_and_grouping():
    bits = np.arange(256, dtype=np.uint8)
    # element i paired with element 255-i: symbol k = fields of elements 2k (low nibble) and 2k+1 (high nibble)
    data = np.stack([bits, bits[::-1]], axis=1).reshape(-1)
    e, sm = zo.split(zo.FP8_E4M3, data, data.size)
    ref = torch.from_numpy(data.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    for half, sl in ((0, slice(0, None, 2)), (1, slice(1, None, 2))):
        ee = ((e >> (4 * half)) & 0xF).astype(np.int64)
        f = (sm >> (4 * half)) & 0xF
        s = f >> 3; m = (f & 7).astype(np.float64)
        val = np.where(ee == 0, np.ldexp(m / 8.0, -6), np.ldexp(1.0 + m / 8.0, ee - 7))
        val = np.where(s == 1, -val, val)
        r = ref[sl]
        ok = ~np.isnan(r)
        assert np.array_equal(val[ok], r[ok])
    # a hand vector: bytes 7E 08 -> exponent symbol 0x1F, sign+mantissa symbol 0x06
    e, sm = zo.split(zo.FP8_E4M3, np.array([0x7E, 0x08], np.uint8), 2)
    assert (int(e[0]), int(sm[0])) == (0x1F, 0x06)


def test_split_fp4_grouping_and_values():
    # four elements 0x7 (+6), 0x1 (.5), 0xD (-3), 0x2 (1.0) packed low nibble first: bytes 0x17, 0x2D
    data = np.array([0x17, 0x2D], np.uint8)
    e, sm = zo.split(zo.FP4_E2M1, data, 4)
    # exponent fields 3,0,2,1 at bit positions 0,2,4,6 ; sign+mantissa fields 1,1,3,0
    assert int(e[0]) == (3 | (0 << 2) | (2 << 4) | (1 << 6))
    assert int(sm[0]) == (1 | (1 << 2) | (3 << 4) | (0 << 6))
    # every nibble value: the fields rebuild the value
    for nib in range(16):
        e, sm = zo.split(zo.FP4_E2M1, np.array([nib], np.uint8), 2)
        ee, f = int(e[0]) & 3, int(sm[0]) & 3
        s, m = f >> 1, f & 1
        val = (0.5 * m) if ee == 0 else (1 + 0.5 * m) * 2.0 ** (ee - 1)
        assert (-val if s else val) == zo.e2m1_value(nib)


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("n", [0, 1, 2, 3, 4, 5, 7, 8, 9, 1000, 4097])
def test_merge_inverts_split(fmt, n):
    if fmt == zo.FP4_E2M1 and n % 2:
        n += 1
    rng = np.random.default_rng(n + 17 * fmt)
    data = rng.integers(0, 256, zo.input_bytes(fmt, n), dtype=np.uint8)
    s0, s1 = zo.split(fmt, data, n)
    assert s0.size == s1.size == -(-n // zo.group(fmt))
    assert np.array_equal(zo.merge(fmt, s0, s1, n), data)


def test_scale_bytes_split_into_odd_and_even_offsets():
    """Sec. 3.4 / 4.4: the scaling factors are coded as a stream of bytes.  Here: bytes at odd offsets are the
    symbols of stream 0, bytes at even offsets those of stream 1; a missing last odd byte counts as zero."""
    s0, s1 = zo.split(zo.SCALE_U8, np.array([0x7A, 0x7B, 0x7C, 0x7D, 0x7E], np.uint8), 5)
    assert list(s0) == [0x7B, 0x7D, 0x00] and list(s1) == [0x7A, 0x7C, 0x7E]
    assert zo.n_syms(zo.SCALE_U8, 5) == 3 and zo.input_bytes(zo.SCALE_U8, 5) == 5 and zo.group(zo.SCALE_U8) == 2
    assert list(zo.merge(zo.SCALE_U8, s0, s1, 5)) == [0x7A, 0x7B, 0x7C, 0x7D, 0x7E]
    # the two histograms are the plain byte counts of the two halves
    rng = np.random.default_rng(8)
    d = rng.integers(0, 256, 10001, dtype=np.uint8)
    h = zo.histogram(zo.SCALE_U8, d, d.size)
    assert np.array_equal(h[1], np.bincount(d[0::2], minlength=256))
    odd = np.bincount(d[1::2], minlength=256); odd[0] += 1              # the zero that stands for the missing byte
    assert np.array_equal(h[0], odd)


def test_tail_fields_are_zero():
    # 3 FP8 elements -> 2 symbols, the missing 4th element contributes zero fields
    e, sm = zo.split(zo.FP8_E4M3, np.array([0xFF, 0xFF, 0xFF], np.uint8), 3)
    assert (int(e[1]), int(sm[1])) == (0x0F, 0x0F)
    e, sm = zo.split(zo.FP4_E2M1, np.array([0xFF], np.uint8), 2)
    assert (int(e[0]), int(sm[0])) == (0x0F, 0x0F)


def test_histogram_counts():
    rng = np.random.default_rng(3)
    data = rng.integers(0, 65536, 50000, dtype=np.uint16)
    h = zo.histogram(zo.BF16, data, data.size)
    assert h.shape == (2, 256) and int(h[0].sum()) == int(h[1].sum()) == data.size
    assert np.array_equal(h[0], np.bincount((data >> 7) & 0xFF, minlength=256).astype(np.uint64))
    assert np.array_equal(h[1], np.bincount(((data >> 15) << 7) | (data & 0x7F), minlength=256).astype(np.uint64))


# --------------------------------------------------------------------------------------------
# code lengths
# --------------------------------------------------------------------------------------------

def _hist_of(counts):
    h = np.zeros(256, np.uint64)
    h[: len(counts)] = counts
    return h


def _kraft(lens):
    return sum(2.0 ** -int(l) for l in lens if l)


def _huffman_cost(counts):
    """Cost of a textbook Huffman tree: sum of all internal node weights."""
    heap = list(counts)
    heapq.heapify(heap)
    cost = 0
    while len(heap) > 1:
        a, b = heapq.heappop(heap), heapq.heappop(heap)
        cost += a + b
        heapq.heappush(heap, a + b)
    return cost


def _brute_best_cost(counts, L):
    """Minimum of sum count*len over every length vector with Kraft sum <= 1 and max <= L."""
    n = len(counts)
    best = None
    for lens in itertools.product(range(1, L + 1), repeat=n):
        if sum(1 << (L - l) for l in lens) <= (1 << L):
            c = sum(a * l for a, l in zip(counts, lens))
            if best is None or c < best:
                best = c
    return best


def _golden_huffman():
    out = {}
    for line in open(os.path.join(GOLDEN, "huffman_worked.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        parts = [p.strip() for p in line.split("|")]
        out[parts[0]] = parts[1:]
    return out


def test_golden_code_lengths_and_codes():
    g = _golden_huffman()
    for name in ("ex1", "ex2", "ex3", "ex5"):
        counts, L, lens, codes = g[name]
        counts = [int(x) for x in counts.split()]
        lens = [int(x) for x in lens.split()]
        got = zo.code_lengths(_hist_of(counts), int(L))
        assert list(got[: len(counts)]) == lens, name
        assert not got[len(counts):].any()
        cw = zo.canonical_codes(got)
        assert [format(int(cw[i]), f"0{lens[i]}b") for i in range(len(counts))] == codes.split(), name
    # RFC 1951 3.2.2 assignment example: lengths are given
    _, _, lens, codes = g["ex4"]
    l = np.zeros(256, np.uint8)
    lens = [int(x) for x in lens.split()]
    l[: len(lens)] = lens
    cw = zo.canonical_codes(l)
    assert [format(int(cw[i]), f"0{lens[i]}b") for i in range(len(lens))] == codes.split()


@pytest.mark.parametrize("L", [3, 4, 5])
def test_lengths_are_optimal_by_brute_force_small(L):
    rng = np.random.default_rng(100 + L)
    for trial in range(120):
        n = int(rng.integers(2, 7 if L > 3 else 8))
        if n > (1 << L):
            continue
        kind = trial % 4
        if kind == 0:
            counts = rng.integers(1, 10, n)
        elif kind == 1:
            counts = rng.integers(1, 1000, n)
        elif kind == 2:
            counts = (2 ** rng.integers(0, 10, n))
        else:
            counts = np.sort(rng.integers(1, 4, n))
        counts = [int(c) for c in counts]
        lens = zo.code_lengths(_hist_of(counts), L)[:n]
        assert lens.min() >= 1 and lens.max() <= L
        assert abs(_kraft(lens) - 1.0) < 1e-12
        assert sum(c * int(l) for c, l in zip(counts, lens)) == _brute_best_cost(counts, L), (counts, list(lens))


def test_lengths_match_textbook_huffman_cost_when_limit_is_loose():
    rng = np.random.default_rng(7)
    for trial in range(300):
        n = int(rng.integers(2, 9))
        counts = [int(c) for c in rng.integers(1, 5000, n)]
        lens = zo.code_lengths(_hist_of(counts), 12)[:n]
        assert abs(_kraft(lens) - 1.0) < 1e-12
        assert sum(c * int(l) for c, l in zip(counts, lens)) == _huffman_cost(counts)
    # also for full 256-symbol alphabets whose Huffman depth stays below 12
    for trial in range(20):
        counts = [int(c) for c in rng.integers(1000, 2000, 256)]
        lens = zo.code_lengths(_hist_of(counts), 12)
        assert abs(_kraft(lens) - 1.0) < 1e-12
        assert sum(c * int(l) for c, l in zip(counts, lens)) == _huffman_cost(counts)


def test_limit_binds_on_fibonacci_counts():
    fib = [1, 1]
    while len(fib) < 20:
        fib.append(fib[-1] + fib[-2])
    lens = zo.code_lengths(_hist_of(fib), 12)[:20]
    assert lens.max() == 12 and abs(_kraft(lens) - 1.0) < 1e-12
    cost = sum(c * int(l) for c, l in zip(fib, lens))
    assert cost > _huffman_cost(fib)                       # the unrestricted tree is 19 deep
    # more frequent symbols never get longer codes
    assert all(lens[i] >= lens[i + 1] for i in range(19))


def test_entropy_bounds():
    rng = np.random.default_rng(11)
    for trial in range(50):
        n = int(rng.integers(2, 257))
        counts = rng.integers(1, 10000, n).astype(np.float64)
        if trial % 2:
            counts = np.floor(counts * np.exp(-0.08 * np.arange(n))) + 1
        h = _hist_of(counts.astype(np.uint64))
        lens = zo.code_lengths(h, 12)
        p = counts / counts.sum()
        H = -(p * np.log2(p)).sum()
        avg = (counts * lens[:n]).sum() / counts.sum()
        assert H <= avg + 1e-12
        if _huffman_cost([int(c) for c in counts]) == int((counts * lens[:n]).sum()):   # limit not binding
            assert avg < H + 1
        st = zo.stream_stats(h, lens, zo.HUFF)
        assert abs(st["entropy_bits"] - H) < 1e-9 and abs(st["avg_len"] - avg) < 1e-12
        assert st["payload_bits"] == int((counts * lens[:n]).sum()) == zo.payload_bits(h, lens)
        assert st["n_active"] == n and st["max_len"] == lens.max()


def test_degenerate_alphabets():
    assert not zo.code_lengths(np.zeros(256, np.uint64)).any()
    h = np.zeros(256, np.uint64); h[200] = 5
    l = zo.code_lengths(h)
    assert l[200] == 1 and l.sum() == 1
    h[3] = 5
    l = zo.code_lengths(h)
    assert l[200] == 1 and l[3] == 1
    assert list(zo.canonical_codes(l)[[3, 200]]) == [0, 1]


def test_codes_are_prefix_free_and_ordered():
    rng = np.random.default_rng(5)
    counts = np.floor(1e6 * np.exp(-0.3 * np.arange(40))).astype(np.uint64) + 1
    h = np.zeros(256, np.uint64); h[rng.permutation(256)[:40]] = counts
    l = zo.code_lengths(h)
    cw = zo.canonical_codes(l)
    strs = {v: format(int(cw[v]), f"0{int(l[v])}b") for v in range(256) if l[v]}
    items = sorted(strs.values())
    for a, b in zip(items, items[1:]):
        assert not b.startswith(a)
    order = sorted(strs, key=lambda v: (int(l[v]), v))
    padded = [strs[v].ljust(12, "0") for v in order]
    assert padded == sorted(padded)          # canonical: numeric order follows (length, symbol)


def test_auto_policy_arithmetic():
    h = np.zeros(256, np.uint64); h[:] = 100           # uniform bytes: 8 bits each -> RAW
    l = zo.code_lengths(h)
    assert zo.choose_mode(h, l, zo.POLICY_AUTO) == zo.RAW
    assert zo.choose_mode(h, l, zo.POLICY_HUFF_ALL) == zo.HUFF
    assert zo.choose_mode(h, l, zo.POLICY_RAW_ALL) == zo.RAW
    # exactly at the threshold 64*bits == 63*8*n -> HUFF ; one bit more -> RAW
    h = np.zeros(256, np.uint64); l = np.zeros(256, np.uint8)
    h[0], l[0] = 64, 7
    h[1], l[1] = 8, 7                                    # bits = 504 = 63*8*72/72... n = 72, 63*8*72 = 36288 = 64*567
    n = 72
    bits = 64 * 7 + 8 * 7
    assert (64 * bits <= 63 * 8 * n) == (zo.choose_mode(h, l, zo.POLICY_AUTO) == zo.HUFF)
    for b7, b8 in ((63, 1), (62, 2), (0, 64), (64, 0)):
        h = np.zeros(256, np.uint64); l = np.zeros(256, np.uint8)
        h[0], l[0] = b7, 7
        h[1], l[1] = b8, 9
        want = zo.HUFF if 64 * (7 * b7 + 9 * b8) <= 63 * 8 * 64 else zo.RAW
        assert zo.choose_mode(h, l, zo.POLICY_AUTO) == want
    assert zo.choose_mode(np.zeros(256, np.uint64), np.zeros(256, np.uint8), zo.POLICY_HUFF_ALL) == zo.RAW


# --------------------------------------------------------------------------------------------
# container
# --------------------------------------------------------------------------------------------

def _bits_of_piece(piece_bytes, nbits):
    """Read a chunk piece as a bit string: bit k = bit 31-(k%32) of little-endian word k//32."""
    words = np.frombuffer(bytes(piece_bytes), dtype="<u4")
    return "".join(format(int(w), "032b") for w in words)[:nbits]


def _dict_decode(bitstr, codes):
    """Independent prefix decoder: grow a candidate string until it equals a code word."""
    inv = {v: k for k, v in codes.items()}
    out, cur = [], ""
    for b in bitstr:
        cur += b
        if cur in inv:
            out.append(inv[cur]); cur = ""
    assert cur == ""
    return out


def test_golden_message_bitstream():
    g = _golden_huffman()
    msg, bits, word, stored = g["msg1"]
    sym = {"A": 1, "B": 2, "C": 3, "D": 4}                # exponent values of BF16 elements, sm = 0
    elems = np.array([sym[ch] << 7 for ch in msg.split()], np.uint16)
    hist = zo.histogram(zo.BF16, elems, elems.size)
    assert list(hist[0][1:5]) == [5, 2, 1, 1]
    cb = zo.build_codebook(hist, zo.POLICY_HUFF_ALL)
    assert list(cb.lengths[0][1:5]) == [1, 2, 3, 3]
    cont = zo.compress(zo.BF16, elems, elems.size, 1024, cb)
    hd = zo.parse_header(cont)
    assert hd["magic"] == b"ZC10" and hd["total_bytes"] == cont.size and hd["n_chunks"] == 1
    # the sign+mantissa stream holds one symbol only: its single chunk is constant and takes no bits at all
    assert hd["streams"][0]["payload_bits"] == 15 and hd["streams"][1]["payload_bits"] == 0
    sec1 = hd["streams"][1]["section_off"]
    assert int.from_bytes(cont[sec1 + 256: sec1 + 260].tobytes(), "little") == 1      # it "starts" behind stream 0's piece
    assert not cont[sec1 + 256 + 16: sec1 + 256 + 16 + 64].any() and hd["payload_bytes"] == 16
    p = hd["payload_off"]
    assert cont[p:p + 4].tobytes() == bytes(int(x, 16) for x in stored.split())
    assert int.from_bytes(cont[p:p + 4].tobytes(), "little") == int(word, 16)
    assert _bits_of_piece(cont[p:p + 16], 15) == bits
    sec = hd["streams"][0]["section_off"]
    assert np.array_equal(cont[sec:sec + 256], cb.lengths[0])
    assert hd["sub_end_bytes"] == 2                       # 1 KiB chunks use the narrow table
    sub_end = np.frombuffer(cont[sec + 256 + 16: sec + 256 + 16 + 64].tobytes(), "<u2")
    assert list(sub_end) == [15] * 32                     # 9 symbols all fall in subchunk 0 (16 symbols each)
    assert np.array_equal(zo.decompress(cont, elems.size * 2), elems.view(np.uint8))


def _random_tensor(fmt, n, seed, skew=True):
    rng = np.random.default_rng(seed)
    if n == 0:
        return np.zeros(0, np.uint8)
    if fmt == zo.SCALE_U8:                                # E8M0-like scale bytes: a narrow bell around 120
        return np.clip(np.round(rng.normal(120, 1.5, n)), 0, 255).astype(np.uint8)
    if fmt == zo.BF16:
        x = (rng.standard_normal(n) * 0.02).astype(np.float32)
        return torch.from_numpy(x).to(torch.bfloat16).view(torch.uint8).numpy().reshape(-1).copy()
    if fmt == zo.FP8_E4M3:
        x = rng.standard_normal(n).astype(np.float32)
        x = np.clip(x / (np.abs(x).max() / 448.0), -448, 448) if n else x
        return torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy().reshape(-1).copy()
    if fmt == zo.FP8_E5M2:
        x = (rng.standard_normal(n) * 0.02).astype(np.float32)
        return torch.from_numpy(x).to(torch.float8_e5m2).view(torch.uint8).numpy().reshape(-1).copy()
    v = rng.choice(16, size=n, p=np.array([6, 5, 4, 3, 2, 1, 1, 1, 6, 5, 4, 3, 2, 1, 1, 1]) / 46.0).astype(np.uint8)
    return (v[0::2] | (v[1::2] << 4)).astype(np.uint8)


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("policy", [zo.POLICY_AUTO, zo.POLICY_HUFF_ALL, zo.POLICY_RAW_ALL])
@pytest.mark.parametrize("chunk_bytes", [2048, 16384])
def test_container_invariants_and_independent_decode(fmt, policy, chunk_bytes):
    G = zo.group(fmt)
    cs = chunk_bytes // 2
    n = (3 * cs + cs // 2 + 37) * G                       # 3 full chunks + a ragged one
    if fmt == zo.FP4_E2M1:
        n -= n % 2
    data = _random_tensor(fmt, n, 42 + fmt)
    hist = zo.histogram(fmt, data, n)
    cb = zo.build_codebook(hist, policy)
    cont = zo.compress(fmt, data, n, chunk_bytes, cb)
    hd = zo.parse_header(cont)
    ns = -(-n // G)
    assert hd["total_bytes"] == cont.size and hd["n_elems"] == n and hd["n_chunks"] == -(-ns // cs)
    assert hd["group"] == G and hd["l_max"] == 12 and hd["subchunks"] == 32
    assert cont.size <= zo.container_bound(fmt, n, chunk_bytes)
    syms = zo.split(fmt, data, n)
    any_huff = False
    for s in range(2):
        st = hd["streams"][s]
        assert st["mode"] == cb.modes[s] and st["n_syms"] == ns and st["section_off"] % 16 == 0
        if st["mode"] == zo.RAW:
            assert st["payload_bits"] == 8 * ns
            sec = st["section_off"]
            assert np.array_equal(cont[sec:sec + ns], syms[s])
            continue
        any_huff = True
        lens = cb.lengths[s].astype(np.int64)
        assert st["payload_bits"] == int((hist[s].astype(np.int64) * lens).sum())
        sec = st["section_off"]
        nc = hd["n_chunks"]
        off16, sub_end, _ = zo.read_tables(cont, s)
        assert hd["sub_end_bytes"] == (2 if chunk_bytes <= 8192 else 4)
        code_str = {v: format(int(cb.codes[s][v]), f"0{int(lens[v])}b") for v in range(256) if lens[v]}
        total_bits = 0
        for c in range(nc):
            sy = syms[s][c * cs:(c + 1) * cs]
            # subchunk end bits are the running sums of the code lengths of each 32nd of the chunk
            want = [int(lens[sy[: min(len(sy), (j + 1) * (cs // 32))]].sum()) for j in range(32)]
            assert list(sub_end[c]) == want
            nbits = int(sub_end[c][31])
            total_bits += nbits
            lo = hd["payload_off"] + 16 * int(off16[c])
            assert lo % 16 == 0
            piece = cont[lo: lo + ((nbits + 127) // 128) * 16]
            bitstr = _bits_of_piece(piece, len(piece) * 8)
            assert set(bitstr[nbits:]) <= {"0"}           # padding bits are zero
            assert _dict_decode(bitstr[:nbits], code_str) == list(sy)
        assert total_bits == st["payload_bits"]
        assert np.all(np.diff(off16) > 0) or nc == 1
    if any_huff:
        assert not cont[-16:].any()
        assert hd["payload_off"] + hd["payload_bytes"] + 16 == cont.size
    else:
        assert hd["payload_bytes"] == 0 and hd["payload_off"] == cont.size
    assert np.array_equal(zo.decompress(cont, data.size), data)
    # random access: each chunk alone gives its slice of the tensor
    for c in range(hd["n_chunks"]):
        got = zo.decompress_chunk(cont, c, chunk_bytes)
        assert np.array_equal(got, data[c * chunk_bytes: c * chunk_bytes + got.size])
        assert got.size == min(chunk_bytes, data.size - c * chunk_bytes)


@pytest.mark.parametrize("fmt", FORMATS)
def test_round_trip_edge_sizes(fmt):
    G = zo.group(fmt)
    chunk_bytes = 1024
    cs = chunk_bytes // 2
    sizes = [0, 1, G - 1, G, G + 1, 2 * G, cs * G - 1, cs * G, cs * G + 1, cs * G + G, 2 * cs * G, 5 * cs * G + 3 * G]
    for n in sorted(set(sizes)):
        if n < 0 or (fmt == zo.FP4_E2M1 and n % 2):
            continue
        for policy in (zo.POLICY_AUTO, zo.POLICY_HUFF_ALL):
            data = _random_tensor(fmt, n, 1000 + n)
            hist = zo.histogram(fmt, data, n)
            cb = zo.build_codebook(hist, policy)
            cont = zo.compress(fmt, data, n, chunk_bytes, cb)
            assert zo.parse_header(cont)["total_bytes"] == cont.size
            assert np.array_equal(zo.decompress(cont, data.size), data), (fmt, n, policy)


def test_round_trip_special_patterns():
    # all-zero tensor: one active symbol per stream; every chunk is constant and takes no payload at all
    z = np.zeros(5000, np.uint16)
    cb = zo.build_codebook(zo.histogram(zo.BF16, z, z.size), zo.POLICY_HUFF_ALL)
    cont = zo.compress(zo.BF16, z, z.size, 1024, cb)
    hd = zo.parse_header(cont)
    assert hd["streams"][0]["payload_bits"] == 0 and hd["streams"][1]["payload_bits"] == 0 and hd["payload_bytes"] == 0
    assert np.array_equal(zo.decompress(cont, z.size * 2), z.view(np.uint8))
    # one element that differs: only its chunk (512 symbols) is coded, one bit per symbol plus the odd one's code
    z[1700] = 0x3F80
    cb = zo.build_codebook(zo.histogram(zo.BF16, z, z.size), zo.POLICY_HUFF_ALL)
    cont = zo.compress(zo.BF16, z, z.size, 1024, cb)
    hd = zo.parse_header(cont)
    assert hd["streams"][0]["payload_bits"] == 512 and hd["streams"][1]["payload_bits"] == 0
    assert hd["payload_bytes"] == 64
    assert np.array_equal(zo.decompress(cont, z.size * 2), z.view(np.uint8))
    for c in range(hd["n_chunks"]):
        assert np.array_equal(zo.decompress_chunk(cont, c, 1024), z.view(np.uint8)[1024 * c: 1024 * (c + 1)])
    # the rule is per stream: with noise in the sign+mantissa bits that stream is stored raw, and the constant
    # exponent stream still costs nothing
    rng = np.random.default_rng(9)
    noisy = (np.uint16(0x3F80) | rng.integers(0, 128, 5000).astype(np.uint16) | (rng.integers(0, 2, 5000).astype(np.uint16) << 15))
    cb = zo.build_codebook(zo.histogram(zo.BF16, noisy, noisy.size), zo.POLICY_AUTO)
    assert cb.modes == [zo.HUFF, zo.RAW]
    cont = zo.compress(zo.BF16, noisy, noisy.size, 1024, cb)
    hd = zo.parse_header(cont)
    assert hd["streams"][0]["payload_bits"] == 0 and hd["payload_bytes"] == 0
    # one chunk with another exponent in it: that chunk alone pays (one bit per symbol, two for the odd symbol)
    noisy[2000] = np.uint16(0x4000) | (noisy[2000] & np.uint16(0x807F))
    cb = zo.build_codebook(zo.histogram(zo.BF16, noisy, noisy.size), zo.POLICY_AUTO)
    assert cb.modes == [zo.HUFF, zo.RAW]
    cont = zo.compress(zo.BF16, noisy, noisy.size, 1024, cb)
    assert zo.parse_header(cont)["streams"][0]["payload_bits"] == 512
    assert np.array_equal(zo.decompress(cont, noisy.size * 2), noisy.view(np.uint8))
    # NaN / inf / -0 / subnormal patterns are ordinary symbols
    pats = np.array([0x7FC0, 0xFFC1, 0x7F80, 0xFF80, 0x8000, 0x0001, 0x807F, 0x7FFF] * 300, np.uint16)
    cb = zo.build_codebook(zo.histogram(zo.BF16, pats, pats.size), zo.POLICY_HUFF_ALL)
    cont = zo.compress(zo.BF16, pats, pats.size, 1024, cb)
    assert np.array_equal(zo.decompress(cont, pats.size * 2), pats.view(np.uint8))
    # every FP8 byte value
    allb = np.tile(np.arange(256, dtype=np.uint8), 40)
    cb = zo.build_codebook(zo.histogram(zo.FP8_E4M3, allb, allb.size), zo.POLICY_HUFF_ALL)
    cont = zo.compress(zo.FP8_E4M3, allb, allb.size, 1024, cb)
    assert np.array_equal(zo.decompress(cont, allb.size), allb)


@pytest.mark.parametrize("chunk_bytes", [1024, 8192, 16384])
def test_container_bound_is_met_by_a_constructed_worst_case(chunk_bytes):
    """The capacity bound against a container that is as large as the format allows: a dictionary made on a steep
    histogram gives some symbols 12-bit codes, and a tensor of whole chunks made of nothing but those symbols (in
    both streams, both coded) fills every piece to 12 bits per symbol.  Its size, worked out here from the layout
    (header, two table sections, pieces, guard), must be exactly the bound; anything else stays below it."""
    steep = np.ones((2, 256), np.uint64)
    steep[:, :20] = (np.uint64(1) << np.arange(40, 20, -1, dtype=np.uint64))      # twenty heavy symbols push the rest to the limit
    cb = zo.build_codebook(steep, zo.POLICY_HUFF_ALL)
    assert cb.modes == [zo.HUFF, zo.HUFF]
    long0 = np.flatnonzero(cb.lengths[0] == 12)
    long1 = np.flatnonzero(cb.lengths[1] == 12)
    assert long0.size >= 2 and long1.size >= 2
    n_chunks, cs = 5, chunk_bytes // 2
    n = n_chunks * cs                                                # BF16: one element per symbol, whole chunks
    rng = np.random.default_rng(4)
    e = long0[rng.integers(0, long0.size, n)].astype(np.uint16)      # exponent symbols
    sm = long1[rng.integers(0, long1.size, n)].astype(np.uint16)     # sign+mantissa symbols
    data = ((e << 7) | (sm & 0x7F) | ((sm >> 7) << 15)).astype(np.uint16).view(np.uint8)
    s0, s1 = zo.split(zo.BF16, data, n)
    assert np.array_equal(s0, e.astype(np.uint8)) and np.array_equal(s1, sm.astype(np.uint8))
    cont = zo.compress(zo.BF16, data, n, chunk_bytes, cb)
    width = 2 if chunk_bytes <= 8192 else 4
    tables = 256 + ((4 * n_chunks + 15) // 16) * 16 + 32 * width * n_chunks
    piece = ((cs * 12 // 8 + 15) // 16) * 16
    want = 128 + 2 * tables + 2 * n_chunks * piece + 16
    assert cont.size == want
    assert zo.container_bound(zo.BF16, n, chunk_bytes) == want
    assert np.array_equal(zo.decompress(cont, data.size), data)
    # a ragged tensor and ordinary data stay below the bound
    assert zo.container_bound(zo.BF16, n + 7, chunk_bytes) >= want


def test_e5m2_split_as_the_paper_states_it():
    """Sec. 3.2: E5M2 gives 5 bits to the exponent and the rest to sign and mantissa.  The per-element fields rebuild
    the value of every one of the 256 patterns (torch's float8_e5m2 is the independent reference), and on Gaussian
    weights the per-element code of the full exponent beats the byte-symbol reading that codes its upper four
    bits (the format id the kernels serve)."""
    pats = np.arange(256, dtype=np.uint8)
    e5, sm3 = zo.e5m2_element_fields(pats)
    assert e5.max() == 31 and sm3.max() == 7
    ref = torch.from_numpy(pats.copy()).view(torch.float8_e5m2).to(torch.float32).numpy()
    for x in range(256):
        s, m, e = int(sm3[x]) >> 2, int(sm3[x]) & 3, int(e5[x])
        if e == 31:
            val = float("inf") if m == 0 else float("nan")
        elif e == 0:
            val = m / 4.0 * 2.0 ** -14
        else:
            val = (1 + m / 4.0) * 2.0 ** (e - 15)
        val = -val if s else val
        assert (np.isnan(val) and np.isnan(ref[x])) or val == ref[x], x
    # hand vector: 0x3C = +1.0 (exponent 15, mantissa 0), 0xC2 = -(2 + 1) = -3.0 (exponent 16, mantissa 2)
    e5, sm3 = zo.e5m2_element_fields(np.array([0x3C, 0xC2], np.uint8))
    assert list(e5) == [15, 16] and list(sm3) == [0, 6]
    assert zo.e5m2_value(0x3C) == 1.0 and zo.e5m2_value(0xC2) == -3.0
    # ratios on synthetic weights
    rng = np.random.default_rng(12)
    w = torch.from_numpy((rng.standard_normal(1 << 20) * 0.02).astype(np.float32)).to(torch.float8_e5m2).view(torch.uint8).numpy()
    be, bs = zo.e5m2_element_payload_bits(w)
    exact = (be + bs) / (8 * w.size)
    h = zo.histogram(zo.FP8_E5M2, w, w.size)
    cb = zo.build_codebook(h, zo.POLICY_AUTO)
    bits = [zo.payload_bits(h[s], cb.lengths[s]) if cb.modes[s] == zo.HUFF else 8 * int(h[s].sum()) for s in range(2)]
    grouped = sum(bits) / (8 * w.size)
    assert exact < grouped < 1.0
    assert 0.60 < exact < 0.75 and 0.65 < grouped < 0.80
    print(f"E5M2 payload ratios: exponent/mantissa split per element {exact:.4f}, byte symbols of the upper exponent bits {grouped:.4f}")


def test_static_dictionary_from_another_tensor():
    """A code built on one tensor encodes another (Sec. 3.3 precomputed dictionaries) as long as it
    covers its symbols; a symbol without a code is an error, not silent damage."""
    a = _random_tensor(zo.BF16, 20000, 1)
    b = _random_tensor(zo.BF16, 20000, 2)
    ha = zo.histogram(zo.BF16, a, 20000)
    hb = zo.histogram(zo.BF16, b, 20000)
    cb = zo.build_codebook(ha + 1, zo.POLICY_HUFF_ALL)     # +1: every symbol gets a code
    cont = zo.compress(zo.BF16, b, 20000, 4096, cb)
    assert np.array_equal(zo.decompress(cont, b.size), b)
    hd = zo.parse_header(cont)
    assert hd["streams"][0]["payload_bits"] == int((hb[0].astype(np.int64) * cb.lengths[0]).sum())
    cb2 = zo.build_codebook(ha, zo.POLICY_HUFF_ALL)
    missing = np.flatnonzero((ha[0] == 0))
    bad = b.copy().view(np.uint16)
    bad[0] = int(missing[0]) << 7
    with pytest.raises(ValueError):
        zo.compress(zo.BF16, bad, 20000, 4096, cb2)


def test_static_dictionary_lengths_cover_every_symbol():
    """A precomputed dictionary (Sec. 3.3) must be able to code a tensor it was not counted on: all 256 symbols
    get a code, the code is complete (Kraft sum exactly 1), and wherever the length limit does not bind its cost
    on the raised counts is that of a textbook Huffman tree."""
    rng = np.random.default_rng(21)
    for trial in range(40):
        n = int(rng.integers(0, 257))
        h = np.zeros(256, np.uint64)
        h[rng.permutation(256)[:n]] = rng.integers(1, 1 << int(rng.integers(1, 34)), n).astype(np.uint64)
        lens = zo.static_lengths(h)
        assert lens.min() >= 1 and lens.max() <= 12
        assert sum(1 << (12 - int(l)) for l in lens) == 1 << 12
        # frequent symbols never get longer codes than rarer ones
        order = np.argsort(h, kind="stable")
        assert all(lens[order[i]] >= lens[order[i + 1]] or h[order[i]] == h[order[i + 1]] for i in range(255))
    assert np.array_equal(zo.static_lengths(np.zeros(256, np.uint64)), np.full(256, 8))
    assert np.array_equal(zo.static_lengths(np.full(256, 12345, np.uint64)), np.full(256, 8))
    for trial in range(20):                      # Huffman depth stays below 12: the limit is loose
        counts = rng.integers(1000, 2000, 256).astype(np.uint64)
        lens = zo.static_lengths(counts)
        raised = [256 * int(c) + 1 for c in counts]
        assert sum(r * int(l) for r, l in zip(raised, lens)) == _huffman_cost(raised)
    # a symbol that never occurred costs a long code; the frequent ones make room for them with one more bit at the end
    h = _hist_of([1 << 20, 1 << 19, 1 << 18, 1 << 17])
    lens = zo.static_lengths(h)
    assert list(lens[:4]) == [1, 2, 3, 4] and lens[4:].min() >= 11
    cb = zo.build_codebook(np.stack([h, np.zeros(256, np.uint64)]), zo.POLICY_STATIC)
    assert cb.modes == [zo.HUFF, zo.RAW] and np.array_equal(cb.lengths[0], lens)


def test_static_dictionary_codes_a_tensor_with_unseen_symbols():
    a = _random_tensor(zo.BF16, 20000, 1)
    b = _random_tensor(zo.BF16, 20000, 2).copy()
    ha = zo.histogram(zo.BF16, a, 20000)
    unseen = np.flatnonzero(ha[0] == 0)
    b.view(np.uint16)[:50] = (unseen[:50].astype(np.uint16) << 7)      # exponents the dictionary never saw
    cb = zo.build_codebook(ha, zo.POLICY_STATIC)
    cont = zo.compress(zo.BF16, b, 20000, 4096, cb)
    assert np.array_equal(zo.decompress(cont, b.size), b)
    hb = zo.histogram(zo.BF16, b, 20000)
    assert zo.parse_header(cont)["streams"][0]["payload_bits"] == int((hb[0].astype(np.int64) * cb.lengths[0]).sum())
    # a tensor without elements is all header, whatever the dictionary's modes say
    empty = zo.compress(zo.BF16, np.zeros(0, np.uint8), 0, 4096, cb)
    assert empty.size == 128 and [st["mode"] for st in zo.parse_header(empty)["streams"]] == [zo.RAW, zo.RAW]
    assert zo.decompress(empty, 0).size == 0


def test_dictionary_replacement_rule():
    """Sec. 3.3: a dictionary stays while the ratio holds and is replaced when it gets worse; the first tensor
    after a (re)build sets the baseline."""
    h = np.stack([_hist_of([100, 50, 20, 5]), _hist_of([10] * 256)])
    d = zo.StaticDictionary(h, 0.05)
    assert d.observe(1000, 700) is False and d.baseline == 0.7
    assert d.observe(1000, 734) is False         # 0.734 <= 0.7 * 1.05
    assert d.observe(1000, 736) is True
    assert d.observe(2000, 1400) is False        # ratios, not sizes, are compared
    assert d.observe(1000, 600) is False         # better than the baseline never triggers
    d.rebuild(h)
    assert d.baseline is None and d.n_rebuilds == 1
    assert d.observe(1000, 900) is False and d.baseline == 0.9
    assert zo.StaticDictionary(h, 0.0).observe(10, 7) is False
    d0 = zo.StaticDictionary(h, 0.0)
    d0.observe(10, 7)
    assert d0.observe(10, 7) is False and d0.observe(1000, 701) is True


def test_damaged_container_is_rejected():
    data = _random_tensor(zo.BF16, 3000, 9)
    cb = zo.build_codebook(zo.histogram(zo.BF16, data, 3000), zo.POLICY_AUTO)
    cont = zo.compress(zo.BF16, data, 3000, 1024, cb)
    hd = zo.parse_header(cont)
    for off, val in ((0, 0x58), (6, 9), (16, 7), (20, 99), (64, 5)):
        bad = cont.copy(); bad[off] = val
        with pytest.raises(ValueError):
            zo.decompress(bad, data.size)
    bad = cont.copy()
    _, _, tab = zo.read_tables(cont, 0)
    bad[tab + hd["sub_end_bytes"] * 5] ^= 0x10             # a subchunk boundary moves
    with pytest.raises(ValueError):
        zo.decompress(bad, data.size)


def test_synthetic_ratios_are_in_the_paper_s_neighbourhood():
    """Gaussian BF16 weights: exponent stream near 0.32, total near 0.66 (abstract: 'up to 62%');
    FP8 E4M3 per-tensor scale: total near 0.82 (abstract: 'up to 83%').  Context, not a target."""
    n = 1 << 20
    d = _random_tensor(zo.BF16, n, 77)
    h = zo.histogram(zo.BF16, d, n)
    cb = zo.build_codebook(h, zo.POLICY_AUTO)
    assert cb.modes == [zo.HUFF, zo.RAW]
    r = zo.payload_bits(h[0], cb.lengths[0]) / (8 * n)
    assert 0.30 < r < 0.35
    cont = zo.compress(zo.BF16, d, n, 65536, cb)
    assert 0.64 < cont.size / d.size < 0.69
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(n) * 0.02).astype(np.float32)
    x = x / (np.abs(x).max() / 448.0)
    d8 = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy().copy()
    h = zo.histogram(zo.FP8_E4M3, d8, n)
    cb = zo.build_codebook(h, zo.POLICY_AUTO)
    assert cb.modes == [zo.HUFF, zo.RAW]
    cont = zo.compress(zo.FP8_E4M3, d8, n, 65536, cb)
    assert 0.78 < cont.size / d8.size < 0.86
