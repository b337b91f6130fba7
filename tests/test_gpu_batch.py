"""The batched entry points against the CPU oracle: many tensors per call, bit-exact.

Containers given to the batched decoder are made by the oracle; containers made by the batched encoder are
compared with the oracle's byte for byte.  Everything goes through the C ABI (via the ctypes binding).
"""
import numpy as np
import pytest
import torch

import oracle as zo
from paper_2508_19263_b200 import binding as zc
from test_gpu_parity import _weights

pytestmark = pytest.mark.gpu
FORMATS = [zc.FMT_BF16, zc.FMT_FP8_E4M3, zc.FMT_FP4_E2M1, zc.FMT_SCALE_U8, zc.FMT_FP8_E5M2]
DEV = "cuda"


def _sizes(fmt, chunk_bytes):
    """Element counts from nothing to dozens of chunks, ragged ends included."""
    G = zo.group(fmt)
    cs = chunk_bytes // 2
    sizes = [0, 2 * G, cs * G, cs * G + 2 * G, 3 * cs * G - 2 * G, 40 * cs * G + 6 * G, 0, 7 * cs * G, 29 * cs * G + cs * G // 2,
             64 * cs * G, 2 * G, 11 * cs * G + 10 * G]
    return [n - (n % 2) if fmt == zc.FMT_FP4_E2M1 else n for n in sizes]


def _oracle_containers(fmt, sizes, chunk_bytes, seed):
    policies = [zc.POLICY_AUTO, zc.POLICY_HUFF_ALL, zc.POLICY_RAW_ALL]
    datas, conts = [], []
    for i, n in enumerate(sizes):
        data = _weights(fmt, n, seed + i)
        cb = zo.build_codebook(zo.histogram(fmt, data, n), policies[i % 3])
        datas.append(data)
        conts.append(zo.compress(fmt, data, n, chunk_bytes, cb))
    return datas, conts


def _to_dev(a, pad=0):
    t = torch.full((max(a.size, 16) + pad,), 0xEE, dtype=torch.uint8, device=DEV)
    t[: a.size] = torch.from_numpy(a.copy()).to(DEV)
    return t


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("chunk_bytes", [1024, 4096, 16384])
def test_batched_decoder_restores_every_tensor(fmt, chunk_bytes):
    sizes = _sizes(fmt, chunk_bytes)
    datas, conts = _oracle_containers(fmt, sizes, chunk_bytes, 1000 * fmt + chunk_bytes)
    plans = [zc.plan(fmt, n, chunk_bytes) for n in sizes]
    d_comps = [_to_dev(c) for c in conts]
    d_outs = [torch.full((p.input_bytes + 64,), 0xEE, dtype=torch.uint8, device=DEV) for p in plans]
    ws = torch.full((256,), 0x5A, dtype=torch.uint8, device=DEV)
    batch = zc.DecompressBatch(plans, d_comps, [c.size for c in conts], d_outs)
    for _ in range(2):                                               # the second call reuses the workspace as it is
        zc.decompress_batch(batch, ws)
        assert zc.batch_status(ws) == (zc.OK, None)
        for p, data, out in zip(plans, datas, d_outs):
            back = out.cpu().numpy()
            assert np.array_equal(back[: p.input_bytes], data[: p.input_bytes])
            assert (back[p.input_bytes:] == 0xEE).all()


def test_batched_decoder_many_small_tensors_span_several_launches():
    fmt, chunk_bytes = zc.FMT_BF16, 1024
    rng = np.random.default_rng(7)
    sizes = [int(v) for v in rng.integers(0, 3000, 1100)]
    datas, conts = _oracle_containers(fmt, sizes, chunk_bytes, 5)
    plans = [zc.plan(fmt, n, chunk_bytes) for n in sizes]
    d_comps = [_to_dev(c) for c in conts]
    d_outs = [torch.full((p.input_bytes + 16,), 0xEE, dtype=torch.uint8, device=DEV) for p in plans]
    ws = torch.zeros(256, dtype=torch.uint8, device=DEV)
    zc.decompress_batch(zc.DecompressBatch(plans, d_comps, [c.size for c in conts], d_outs), ws)
    assert zc.batch_status(ws) == (zc.OK, None)
    for p, data, out in zip(plans, datas, d_outs):
        back = out.cpu().numpy()
        assert np.array_equal(back[: p.input_bytes], data[: p.input_bytes])
        assert (back[p.input_bytes:] == 0xEE).all()


@pytest.mark.parametrize("victim", [0, 5, 11])
def test_batched_decoder_names_the_damaged_tensor_and_decodes_the_rest(victim):
    fmt, chunk_bytes = zc.FMT_FP8_E4M3, 4096
    sizes = _sizes(fmt, chunk_bytes)
    datas, conts = _oracle_containers(fmt, sizes, chunk_bytes, 77)
    bad = conts[victim].copy()
    bad[17] ^= 0x40                                                  # chunk_bytes field of the header
    conts[victim] = bad
    plans = [zc.plan(fmt, n, chunk_bytes) for n in sizes]
    d_comps = [_to_dev(c) for c in conts]
    d_outs = [torch.full((p.input_bytes + 16,), 0xEE, dtype=torch.uint8, device=DEV) for p in plans]
    ws = torch.zeros(256, dtype=torch.uint8, device=DEV)
    zc.decompress_batch(zc.DecompressBatch(plans, d_comps, [c.size for c in conts], d_outs), ws)
    assert zc.batch_status(ws) == (zc.E_CORRUPT, victim)
    for t, (p, data, out) in enumerate(zip(plans, datas, d_outs)):
        back = out.cpu().numpy()
        if t == victim:
            assert (back == 0xEE).all()                              # nothing of it was written
        else:
            assert np.array_equal(back[: p.input_bytes], data[: p.input_bytes])


def test_batch_argument_checks():
    pa, pb = zc.plan(zc.FMT_BF16, 5000, 4096), zc.plan(zc.FMT_BF16, 5000, 8192)
    pc = zc.plan(zc.FMT_FP8_E4M3, 5000, 4096)
    d = [torch.zeros(1 << 15, dtype=torch.uint8, device=DEV) for _ in range(2)]
    o = [torch.zeros(1 << 15, dtype=torch.uint8, device=DEV) for _ in range(2)]
    ws = torch.zeros(256, dtype=torch.uint8, device=DEV)
    for plans in ([pa, pb], [pa, pc]):
        with pytest.raises(zc.ZcError) as e:
            zc.decompress_batch(zc.DecompressBatch(plans, d, [1 << 15] * 2, o), ws)
        assert e.value.status == zc.E_INVALID_ARG
    with pytest.raises(zc.ZcError) as e:
        zc.decompress_batch(zc.DecompressBatch([pa, pa], d, [1 << 15, 64], o), ws)
    assert e.value.status == zc.E_CORRUPT
    zc.decompress_batch(zc.DecompressBatch([], [], [], []), ws)      # nothing to do


# ---- the batched encoder ----

def _batch_compress(fmt, sizes, chunk_bytes, seed, policies):
    datas = [_weights(fmt, n, seed + i) for i, n in enumerate(sizes)]
    plans = [zc.plan(fmt, n, chunk_bytes) for n in sizes]
    hists = [zo.histogram(fmt, d, n) for d, n in zip(datas, sizes)]
    cbs = [zc.build_codebook(p, h, policies[i % len(policies)]) for i, (p, h) in enumerate(zip(plans, hists))]
    ocbs = [zo.build_codebook(h, policies[i % len(policies)]) for i, h in enumerate(hists)]
    d_ins = [_to_dev(d) for d in datas]
    d_outs = [torch.full((p.max_compressed_bytes + 64,), 0xA5, dtype=torch.uint8, device=DEV) for p in plans]
    batch = zc.CompressBatch(plans, d_ins, [o[: p.max_compressed_bytes] for o, p in zip(d_outs, plans)])
    batch.set_codebooks(cbs)
    ws = torch.full((batch.workspace_bytes,), 0x5A, dtype=torch.uint8, device=DEV)
    return datas, plans, ocbs, d_outs, batch, ws


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("chunk_bytes", [1024, 4096, 16384])
def test_batched_encoder_writes_the_oracle_s_containers(fmt, chunk_bytes):
    sizes = _sizes(fmt, chunk_bytes)
    policies = [zc.POLICY_AUTO, zc.POLICY_HUFF_ALL, zc.POLICY_RAW_ALL]
    datas, plans, ocbs, d_outs, batch, ws = _batch_compress(fmt, sizes, chunk_bytes, 3000 * fmt + chunk_bytes, policies)
    for _ in range(2):                                               # twice in a row on the same workspace
        got_sizes = zc.compress_batch(batch, ws)
        assert zc.batch_status(ws) == (zc.OK, None)
        for n, data, p, ocb, out, nbytes in zip(sizes, datas, plans, ocbs, d_outs, got_sizes):
            want = zo.compress(fmt, data, n, chunk_bytes, ocb)
            cont = out.cpu().numpy()
            assert nbytes == want.size
            assert np.array_equal(cont[:nbytes], want)
            assert (cont[p.max_compressed_bytes:] == 0xA5).all()     # canary after the buffer


def test_batched_encoder_many_small_tensors_and_the_batched_decoder_after_it():
    fmt, chunk_bytes = zc.FMT_BF16, 1024
    rng = np.random.default_rng(11)
    sizes = [int(v) for v in rng.integers(0, 6000, 700)]
    datas, plans, ocbs, d_outs, batch, ws = _batch_compress(fmt, sizes, chunk_bytes, 9, [zc.POLICY_AUTO, zc.POLICY_HUFF_ALL])
    got_sizes = zc.compress_batch(batch, ws)
    for n, data, ocb, out, nbytes in zip(sizes, datas, ocbs, d_outs, got_sizes):
        want = zo.compress(fmt, data, n, chunk_bytes, ocb)
        assert nbytes == want.size and np.array_equal(out[:nbytes].cpu().numpy(), want)
    backs = [torch.full((p.input_bytes + 16,), 0xEE, dtype=torch.uint8, device=DEV) for p in plans]
    zc.decompress_batch(zc.DecompressBatch(plans, d_outs, got_sizes, backs), ws)
    assert zc.batch_status(ws) == (zc.OK, None)
    for p, data, back in zip(plans, datas, backs):
        assert np.array_equal(back[: p.input_bytes].cpu().numpy(), data[: p.input_bytes])


@pytest.mark.parametrize("fmt", [zc.FMT_BF16, zc.FMT_FP8_E4M3])
def test_batched_encoder_with_codebooks_shared_between_tensors(fmt):
    """Pages of a K/V cache share their dictionaries (Sec. 3.3): three static codebooks serve 40 tensors, a few
    tensors bring their own; every container equals the oracle's with the same code."""
    chunk_bytes = 4096
    rng = np.random.default_rng(3)
    G = zo.group(fmt)
    sizes = [int(v) * 2 * G for v in rng.integers(1, 12000, 40)] + [0, 2 * G]
    datas = [_weights(fmt, n, 500 + i) for i, n in enumerate(sizes)]
    plans = [zc.plan(fmt, n, chunk_bytes) for n in sizes]
    hists = [zo.histogram(fmt, d, n) for d, n in zip(datas, sizes)]
    shared = [zc.build_codebook(plans[k], hists[k], zc.POLICY_STATIC) for k in range(3)]
    oshared = [zo.build_codebook(hists[k], zo.POLICY_STATIC) for k in range(3)]
    cbs, ocbs = [], []
    for i in range(len(sizes)):
        if i % 7 == 6:                                               # its own codebook
            cbs.append(zc.build_codebook(plans[i], hists[i], zc.POLICY_AUTO))
            ocbs.append(zo.build_codebook(hists[i], zo.POLICY_AUTO))
        else:
            cbs.append(shared[i % 3])
            ocbs.append(oshared[i % 3])
    d_ins = [_to_dev(d) for d in datas]
    d_outs = [torch.full((p.max_compressed_bytes,), 0xA5, dtype=torch.uint8, device=DEV) for p in plans]
    batch = zc.CompressBatch(plans, d_ins, d_outs)
    batch.set_codebooks(cbs)
    ws = torch.full((batch.workspace_bytes,), 0x5A, dtype=torch.uint8, device=DEV)
    for _ in range(2):
        got = zc.compress_batch(batch, ws)
        for n, data, ocb, out, nbytes in zip(sizes, datas, ocbs, d_outs, got):
            want = zo.compress(fmt, data, n, chunk_bytes, ocb)
            assert nbytes == want.size and np.array_equal(out[:nbytes].cpu().numpy(), want)
    backs = [torch.full((p.input_bytes + 16,), 0xEE, dtype=torch.uint8, device=DEV) for p in plans]
    dws = torch.zeros(256, dtype=torch.uint8, device=DEV)
    zc.decompress_batch(zc.DecompressBatch(plans, d_outs, got, backs), dws)
    assert zc.batch_status(dws) == (zc.OK, None)
    for p, data, back in zip(plans, datas, backs):
        assert np.array_equal(back[: p.input_bytes].cpu().numpy(), data[: p.input_bytes])


def test_batched_encoder_reports_a_symbol_without_code_and_its_tensor():
    fmt, chunk_bytes = zc.FMT_BF16, 4096
    sizes = [30000, 50000, 20000]
    datas = [_weights(fmt, n, 40 + i) for i, n in enumerate(sizes)]
    plans = [zc.plan(fmt, n, chunk_bytes) for n in sizes]
    hists = [zo.histogram(fmt, d, n) for d, n in zip(datas, sizes)]
    missing = int(np.flatnonzero(hists[1][0] == 0)[0])
    bad = datas[1].copy().view(np.uint16); bad[777] = missing << 7
    datas[1] = bad.view(np.uint8)
    cbs = [zc.build_codebook(p, h, zc.POLICY_HUFF_ALL) for p, h in zip(plans, hists)]
    d_ins = [_to_dev(d) for d in datas]
    d_outs = [torch.zeros(p.max_compressed_bytes, dtype=torch.uint8, device=DEV) for p in plans]
    batch = zc.CompressBatch(plans, d_ins, d_outs)
    batch.set_codebooks(cbs)
    ws = torch.zeros(batch.workspace_bytes, dtype=torch.uint8, device=DEV)
    with pytest.raises(zc.ZcError) as e:
        zc.compress_batch(batch, ws)
    assert e.value.status == zc.E_NO_CODE
    assert zc.batch_status(ws) == (zc.E_NO_CODE, 1)


def test_compress_batch_argument_checks():
    pa, pb = zc.plan(zc.FMT_BF16, 5000, 4096), zc.plan(zc.FMT_BF16, 5000, 8192)
    d = [torch.zeros(1 << 15, dtype=torch.uint8, device=DEV) for _ in range(2)]
    o = [torch.zeros(1 << 15, dtype=torch.uint8, device=DEV) for _ in range(2)]
    cb = zc.build_codebook(pa, np.ones((2, 256)), zc.POLICY_AUTO)
    batch = zc.CompressBatch([pa, pb], d, o)
    batch.set_codebooks([cb, cb])
    ws = torch.zeros(1 << 16, dtype=torch.uint8, device=DEV)
    with pytest.raises(zc.ZcError) as e:
        zc.compress_batch(batch, ws)
    assert e.value.status == zc.E_INVALID_ARG
    batch = zc.CompressBatch([pa, pa], d, [o[0], o[1][:100]])
    batch.set_codebooks([cb, cb])
    with pytest.raises(zc.ZcError) as e:
        zc.compress_batch(batch, ws)
    assert e.value.status == zc.E_BUFFER_TOO_SMALL
    batch = zc.CompressBatch([pa, pa], d, o)
    batch.set_codebooks([cb, cb])
    with pytest.raises(zc.ZcError) as e:
        zc.compress_batch(batch, ws[:256])
    assert e.value.status == zc.E_BUFFER_TOO_SMALL


# ---- the batched histogram ----

@pytest.mark.parametrize("fmt", FORMATS)
def test_batched_histogram_counts_every_tensor(fmt):
    G = zo.group(fmt)
    rng = np.random.default_rng(fmt)
    sizes = [0, 2 * G, 8 * G - 2 * G, 8 * G, 8 * G + 2 * G, 100000 * G + 6 * G, 0, 16 * G, 3 * G * 2, 1 << 21, 12345 * 2 * G] + \
            [int(v) * 2 * G for v in rng.integers(0, 5000, 40)]
    datas = [_weights(fmt, n, 500 + i) for i, n in enumerate(sizes)]
    plans = [zc.plan(fmt, n, 4096) for n in sizes]
    d_ins = [_to_dev(d) for d in datas]
    d_hists = torch.full((len(sizes), 2, 256), -1, dtype=torch.int64, device=DEV)
    zc.histogram_batch(zc.HistogramBatch(plans, d_ins), d_hists)
    got = d_hists.cpu().numpy().astype(np.uint64)
    for i, (n, data) in enumerate(zip(sizes, datas)):
        assert np.array_equal(got[i], zo.histogram(fmt, data, n)), f"tensor {i} ({n} elements)"


# ---- XOR-delta forms (delta checkpoints, Sec. 3.1 / 4.1) ----

def _checkpoint_pair(fmt, n, seed):
    """Two tensors that differ little: the second one is the first with a few low mantissa bits flipped here and
    there and a sprinkling of completely different elements."""
    rng = np.random.default_rng(seed)
    a = _weights(fmt, n, seed)
    b = a.copy()
    if b.size:
        flip = rng.random(b.size) < 0.3
        b[flip] ^= rng.integers(0, 4, int(flip.sum()), dtype=np.uint8)
        wild = rng.random(b.size) < 0.002
        b[wild] = rng.integers(0, 256, int(wild.sum()), dtype=np.uint8)
    return a, b


@pytest.mark.parametrize("fmt", [zc.FMT_BF16, zc.FMT_FP8_E4M3])
@pytest.mark.parametrize("chunk_bytes", [1024, 4096, 16384])
def test_xor_delta_single_calls_match_the_oracle_on_the_xor(fmt, chunk_bytes):
    G = zo.group(fmt)
    cs = chunk_bytes // 2
    for n in [0, 2 * G, 5 * cs * G + cs * G // 3 + 2 * G, 23 * cs * G + 6 * G]:
        base, cur = _checkpoint_pair(fmt, n, chunk_bytes + n)
        delta = base ^ cur                                            # the plain definition of what is coded
        p = zc.plan(fmt, n, chunk_bytes)
        d_cur, d_base = _to_dev(cur), _to_dev(base)
        hist = zc.histogram(p, d_cur, d_base=d_base).cpu().numpy().astype(np.uint64)
        assert np.array_equal(hist, zo.histogram(fmt, delta, n))
        cb, ocb = zc.build_codebook(p, hist, zc.POLICY_AUTO), zo.build_codebook(hist, zc.POLICY_AUTO)
        d_out = torch.full((p.max_compressed_bytes,), 0xA5, dtype=torch.uint8, device=DEV)
        ws = torch.empty(p.workspace_bytes, dtype=torch.uint8, device=DEV)
        nbytes = zc.compress(p, cb, d_cur, d_out, ws, d_base=d_base)
        want = zo.compress(fmt, delta, n, chunk_bytes, ocb)
        assert nbytes == want.size and np.array_equal(d_out[:nbytes].cpu().numpy(), want)
        d_back = torch.full((p.input_bytes + 32,), 0xEE, dtype=torch.uint8, device=DEV)
        zc.decompress(p, d_out, nbytes, d_back, ws, d_base=d_base)
        assert zc.device_status(p, ws) == zc.OK
        back = d_back.cpu().numpy()
        assert np.array_equal(back[: p.input_bytes], cur[: p.input_bytes]) and (back[p.input_bytes:] == 0xEE).all()


def _mixed_delta(fmt, chunk_bytes):
    """base, current, their XOR and the element count: chunks 0, 3, 5, 8, 10 and the ragged end unchanged; 1-2 mantissa
    bits only; 4 lowest exponent bit only; 6-7 everything; 9 mantissa bits in its first half."""
    G = zo.group(fmt)
    cs = chunk_bytes // 2
    n_syms = 11 * cs + cs // 3 + 5
    n = n_syms * G
    rng = np.random.default_rng(chunk_bytes + fmt)
    base = _weights(fmt, n, 5 + chunk_bytes)[: 2 * n_syms].copy()
    delta = np.zeros_like(base)
    if fmt == zc.FMT_BF16:
        view, mant, expo, full = delta.view(np.uint16), 0x0003, 0x0080, 0x10000     # sign 15, exponent 14..7, mantissa 6..0
    else:
        view, mant, expo, full = delta, 0x03, 0x08, 0x100                             # sign 7, exponent 6..3, mantissa 2..0
    per_chunk = 2 * cs // view.itemsize
    def span(c0, c1): return view[c0 * per_chunk: c1 * per_chunk]
    d = span(1, 3); d[:] = rng.integers(0, mant + 1, d.size) * (rng.random(d.size) < 0.4)
    d = span(4, 5); d[:] = (rng.random(d.size) < 0.05) * expo
    d = span(6, 8); d[:] = rng.integers(0, full, d.size) * (rng.random(d.size) < 0.2)
    d = span(9, 10); d[: d.size // 2] = rng.integers(0, mant + 1, d.size // 2)
    return base, base ^ delta, delta, n


@pytest.mark.parametrize("fmt", [zc.FMT_BF16, zc.FMT_FP8_E4M3])
@pytest.mark.parametrize("chunk_bytes", [2048, 4096, 16384, 65536])
def test_xor_delta_with_unchanged_stretches(fmt, chunk_bytes):
    """A later checkpoint in which whole stretches did not move, stretches where only the low mantissa bits moved (the
    exponent stream of those chunks is constant, the other stream is not), stretches where only exponent bits
    moved, ordinary stretches, and an unchanged ragged end: every mix of constant and coded chunks in the two
    streams, with both streams Huffman-coded."""
    cs = chunk_bytes // 2
    base, cur, delta, n = _mixed_delta(fmt, chunk_bytes)
    p = zc.plan(fmt, n, chunk_bytes)
    d_cur, d_base = _to_dev(cur), _to_dev(base)
    hist = zc.histogram(p, d_cur, d_base=d_base).cpu().numpy().astype(np.uint64)
    assert np.array_equal(hist, zo.histogram(fmt, delta, n))
    for policy in (zc.POLICY_HUFF_ALL, zc.POLICY_AUTO):
        cb, ocb = zc.build_codebook(p, hist, policy), zo.build_codebook(hist, policy)
        d_out = torch.full((p.max_compressed_bytes,), 0xA5, dtype=torch.uint8, device=DEV)
        ws = torch.empty(p.workspace_bytes, dtype=torch.uint8, device=DEV)
        nbytes = zc.compress(p, cb, d_cur, d_out, ws, d_base=d_base)
        want = zo.compress(fmt, delta, n, chunk_bytes, ocb)
        assert nbytes == want.size and np.array_equal(d_out[:nbytes].cpu().numpy(), want)
        if policy == zc.POLICY_HUFF_ALL:
            hd = zo.parse_header(want)
            assert all(st["payload_bits"] < 8 * 4 * cs for st in hd["streams"])      # most chunks of either stream cost nothing
        d_back = torch.full((p.input_bytes + 32,), 0xEE, dtype=torch.uint8, device=DEV)
        zc.decompress(p, d_out, nbytes, d_back, ws, d_base=d_base)
        assert zc.device_status(p, ws) == zc.OK
        back = d_back.cpu().numpy()
        assert np.array_equal(back[: p.input_bytes], cur[: p.input_bytes]) and (back[p.input_bytes:] == 0xEE).all()


def test_xor_delta_batched_calls():
    fmt, chunk_bytes = zc.FMT_BF16, 4096
    sizes = _sizes(fmt, chunk_bytes)
    pairs = [_checkpoint_pair(fmt, n, 900 + i) for i, n in enumerate(sizes)]
    plans = [zc.plan(fmt, n, chunk_bytes) for n in sizes]
    d_bases = [_to_dev(a) for a, _ in pairs]
    d_curs = [_to_dev(b) for _, b in pairs]
    d_bases[3] = None                                                 # one tensor of the batch without a base
    deltas = [(b if i == 3 else a ^ b) for i, (a, b) in enumerate(pairs)]
    d_hists = torch.zeros((len(sizes), 2, 256), dtype=torch.int64, device=DEV)
    zc.histogram_batch(zc.HistogramBatch(plans, d_curs, d_bases), d_hists)
    hists = d_hists.cpu().numpy().astype(np.uint64)
    for i, (n, d) in enumerate(zip(sizes, deltas)):
        assert np.array_equal(hists[i], zo.histogram(fmt, d, n))
    cbs = zc.build_codebooks(plans, hists, zc.POLICY_AUTO)
    d_outs = [torch.zeros(p.max_compressed_bytes, dtype=torch.uint8, device=DEV) for p in plans]
    batch = zc.CompressBatch(plans, d_curs, d_outs, d_bases)
    batch.set_codebooks(cbs)
    ws = torch.empty(batch.workspace_bytes, dtype=torch.uint8, device=DEV)
    got = zc.compress_batch(batch, ws)
    for i, (n, d) in enumerate(zip(sizes, deltas)):
        want = zo.compress(fmt, d, n, chunk_bytes, zo.build_codebook(hists[i], zc.POLICY_AUTO))
        assert got[i] == want.size and np.array_equal(d_outs[i][: got[i]].cpu().numpy(), want)
    backs = [torch.full((p.input_bytes + 16,), 0xEE, dtype=torch.uint8, device=DEV) for p in plans]
    zc.decompress_batch(zc.DecompressBatch(plans, d_outs, got, backs, d_bases), ws)
    assert zc.batch_status(ws) == (zc.OK, None)
    for p, (a, b), back in zip(plans, pairs, backs):
        out = back.cpu().numpy()
        assert np.array_equal(out[: p.input_bytes], b[: p.input_bytes]) and (out[p.input_bytes:] == 0xEE).all()


def test_batched_calls_at_bench_size_on_sampled_chunks():
    """Tensors of the size class the benchmark times (a 14336 x 4096 and a 4096 x 4096 BF16 matrix and a 1024 x 4096
    one, 4 KiB chunks, the batched calls): the oracle decodes sampled chunks one by one, properties that hold at
    any size cover the rest."""
    fmt, chunk_bytes = zc.FMT_BF16, 4096
    shapes = [(14336, 4096), (4096, 4096), (1024, 4096)]
    g = torch.Generator(device=DEV); g.manual_seed(99)
    d_ins, plans = [], []
    for r, c in shapes:
        x = (torch.randn(r * c, generator=g, device=DEV) * 0.02).to(torch.bfloat16)
        d_ins.append(x.view(torch.uint8))
        plans.append(zc.plan(fmt, r * c, chunk_bytes))
    n_t = len(plans)
    d_hists = torch.zeros((n_t, 2, 256), dtype=torch.int64, device=DEV)
    zc.histogram_batch(zc.HistogramBatch(plans, d_ins), d_hists)
    hists = d_hists.cpu().numpy().astype(np.uint64)
    for t in range(n_t):
        assert int(hists[t, 0].sum()) == plans[t].n_syms and int(hists[t, 1].sum()) == plans[t].n_syms
    cbs = zc.build_codebooks(plans, hists, zc.POLICY_AUTO)
    d_outs = [torch.empty(p.max_compressed_bytes, dtype=torch.uint8, device=DEV) for p in plans]
    enc = zc.CompressBatch(plans, d_ins, d_outs)
    enc.set_codebooks(cbs)
    ws = torch.empty(enc.workspace_bytes, dtype=torch.uint8, device=DEV)
    sizes = zc.compress_batch(enc, ws)
    rng = np.random.default_rng(0)
    for t in range(n_t):
        p = plans[t]
        cont = d_outs[t][: sizes[t]].cpu().numpy()
        assert zc.validate_container(p, cont) == zc.OK
        hd = zo.parse_header(cont)
        assert hd["total_bytes"] == sizes[t] and hd["n_chunks"] == p.n_chunks
        for s in range(2):
            mode, lens, _ = cbs[t].get(s)
            want_bits = int((hists[t, s].astype(np.int64) * lens).sum()) if mode == zc.MODE_HUFF else 8 * p.n_syms
            assert hd["streams"][s]["payload_bits"] == want_bits
        data = d_ins[t].cpu().numpy()
        for c in [0, 1, p.n_chunks - 1] + [int(v) for v in rng.integers(0, p.n_chunks, 10)]:
            got = zo.decompress_chunk(cont, c, chunk_bytes)
            assert np.array_equal(got, data[c * chunk_bytes: c * chunk_bytes + got.size]), (t, c)
    d_backs = [torch.empty(p.input_bytes, dtype=torch.uint8, device=DEV) for p in plans]
    zc.decompress_batch(zc.DecompressBatch(plans, d_outs, sizes, d_backs), ws)
    assert zc.batch_status(ws) == (zc.OK, None)
    for b, x in zip(d_backs, d_ins):
        assert torch.equal(b, x)


@pytest.mark.parametrize("fmt", [zc.FMT_BF16, zc.FMT_FP8_E4M3])
@pytest.mark.parametrize("chunk_bytes", [2048, 4096, 65536])
def test_whole_containers_at_bench_size_equal_the_oracle_s(fmt, chunk_bytes):
    """Tensors of the size class the benchmark times, in one batched call that crosses tensor boundaries: every byte
    of every container against the oracle (not a sample).  The large tensor has thousands of batches, far more
    than blocks run at a time, so its chunks are placed through many rounds of the look-back; the ragged one ends
    in the middle of a chunk."""
    G = zo.group(fmt)
    sizes = [(24 << 20) * G, (3 << 20) * G + 1234 * G + 2 * G, 0, (7 << 20) * G]     # 48 MiB, 6 MiB + a bit, nothing, 14 MiB of BF16
    g = torch.Generator(device=DEV); g.manual_seed(7 + chunk_bytes)
    d_ins, plans, datas = [], [], []
    for i, n in enumerate(sizes):
        x = torch.randn(max(n, 16), generator=g, device=DEV) * (0.02 / (1 + i))
        if fmt == zc.FMT_BF16:
            b = x.to(torch.bfloat16).view(torch.uint8)[: 2 * n]
        else:
            b = (x / (x.abs().max() / 448)).clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8)[:n]
        d_ins.append(b.contiguous() if n else torch.zeros(16, dtype=torch.uint8, device=DEV))
        datas.append(b.cpu().numpy().copy() if n else np.zeros(0, np.uint8))
        plans.append(zc.plan(fmt, n, chunk_bytes))
    n_t = len(plans)
    d_hists = torch.zeros((n_t, 2, 256), dtype=torch.int64, device=DEV)
    zc.histogram_batch(zc.HistogramBatch(plans, d_ins), d_hists)
    hists = d_hists.cpu().numpy().astype(np.uint64)
    cbs = zc.build_codebooks(plans, hists, zc.POLICY_AUTO)
    d_outs = [torch.empty(p.max_compressed_bytes, dtype=torch.uint8, device=DEV) for p in plans]
    enc = zc.CompressBatch(plans, d_ins, d_outs)
    enc.set_codebooks(cbs)
    ws = torch.empty(enc.workspace_bytes, dtype=torch.uint8, device=DEV)
    got_sizes = zc.compress_batch(enc, ws)
    for t in range(n_t):
        assert np.array_equal(hists[t], zo.histogram(fmt, datas[t], sizes[t]))
        want = zo.compress(fmt, datas[t], sizes[t], chunk_bytes, zo.build_codebook(hists[t], zo.POLICY_AUTO))
        assert got_sizes[t] == want.size
        assert np.array_equal(d_outs[t][: got_sizes[t]].cpu().numpy(), want), f"container of tensor {t} differs"
    d_backs = [torch.empty(max(p.input_bytes, 16), dtype=torch.uint8, device=DEV) for p in plans]
    zc.decompress_batch(zc.DecompressBatch(plans, d_outs, got_sizes, d_backs), ws)
    assert zc.batch_status(ws) == (zc.OK, None)
    for p, b, x in zip(plans, d_backs, d_ins):
        assert torch.equal(b[: p.input_bytes], x[: p.input_bytes])
