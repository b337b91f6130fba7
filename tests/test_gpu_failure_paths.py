"""Failure handling on the device, without faulting or hanging anything.

* A damaged payload (not only damaged tables): every lane must consume exactly the bits of its subchunk, so damage
  that changes the length of a code is reported as ZC_E_CORRUPT, and the decoder stays inside its buffers whatever
  the payload says.
* Bounded waits: with the test hooks of include/zc_test_hooks.h a look-back waits for a word that nobody posts,
  resp. the decoder waits for a copy that was never started; the wait limit is set low, the kernels give up by
  themselves, the call reports ZC_E_DEVICE_TIMEOUT, and the next ordinary call on the same workspace works.
* The largest chunk size zc_plan accepts, with both streams coded.
"""
import numpy as np
import pytest
import torch

import oracle as zo
from paper_2508_19263_b200 import binding as zc

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _bf16_weights(n, seed, std=0.02):
    rng = np.random.default_rng(seed)
    x = torch.from_numpy((rng.standard_normal(n) * std).astype(np.float32))
    return x.to(torch.bfloat16).view(torch.uint8).numpy().reshape(-1).copy()


def _oracle_container(fmt, data, n, chunk_bytes, policy=zo.POLICY_AUTO):
    return zo.compress(fmt, data, n, chunk_bytes, zo.build_codebook(zo.histogram(fmt, data, n), policy))


@pytest.mark.parametrize("chunk_bytes", [4096, 16384])
@pytest.mark.parametrize("batched", [False, True])
def test_damaged_payload_bits_are_reported(chunk_bytes, batched):
    fmt, n = zc.FMT_BF16, 40 * chunk_bytes // 2 + 77
    data = _bf16_weights(n, 5)
    cont = _oracle_container(fmt, data, n, chunk_bytes)
    hd = zo.parse_header(cont)
    assert hd["streams"][0]["mode"] == zo.HUFF
    p = zc.plan(fmt, n, chunk_bytes)
    ws = torch.zeros(max(p.workspace_bytes, 256), dtype=torch.uint8, device=DEV)
    payload_off = hd["total_bytes"] - 16 - hd["payload_bytes"]
    rng = np.random.default_rng(1)
    reported = 0
    for trial in range(12):
        bad = cont.copy()
        at = payload_off + int(rng.integers(0, hd["payload_bytes"] - 64))
        bad[at] ^= 1 << int(rng.integers(0, 8))
        d_comp = torch.from_numpy(bad).to(DEV)
        d_out = torch.full((p.input_bytes + 64,), 0xEE, dtype=torch.uint8, device=DEV)
        if batched:
            zc.decompress_batch(zc.DecompressBatch([p], [d_comp], [bad.size], [d_out]), ws)
            st = zc.batch_status(ws)[0]
        else:
            zc.decompress(p, d_comp, bad.size, d_out, ws)
            st = zc.device_status(p, ws)
        assert st in (zc.OK, zc.E_CORRUPT)
        back = d_out.cpu().numpy()
        assert (back[p.input_bytes:] == 0xEE).all()                  # nothing written past the tensor, whatever the bits say
        # A flipped bit that turns a code into another code of the same length cannot be seen (the payload carries no
        # checksum); one that changes a length shifts the end of its subchunk, and that is reported.
        reported += st == zc.E_CORRUPT
    assert reported >= 2
    # the untouched container still decodes on the same workspace
    d_out = torch.empty(p.input_bytes, dtype=torch.uint8, device=DEV)
    zc.decompress(p, torch.from_numpy(cont).to(DEV), cont.size, d_out, ws)
    assert zc.device_status(p, ws) == zc.OK
    assert np.array_equal(d_out.cpu().numpy(), data[: p.input_bytes])


def test_payload_of_garbage_stays_in_bounds():
    """Valid header and tables, payload replaced by random bytes: lanes run far past their subchunks."""
    fmt, chunk_bytes, n = zc.FMT_BF16, 4096, 64 * 2048
    data = _bf16_weights(n, 9)
    cont = _oracle_container(fmt, data, n, chunk_bytes)
    hd = zo.parse_header(cont)
    payload_off = hd["total_bytes"] - 16 - hd["payload_bytes"]
    bad = cont.copy()
    bad[payload_off: payload_off + hd["payload_bytes"]] = np.random.default_rng(3).integers(0, 256, hd["payload_bytes"], dtype=np.uint8)
    p = zc.plan(fmt, n, chunk_bytes)
    ws = torch.zeros(256, dtype=torch.uint8, device=DEV)
    d_out = torch.full((p.input_bytes + 64,), 0xEE, dtype=torch.uint8, device=DEV)
    zc.decompress(p, torch.from_numpy(bad).to(DEV), bad.size, d_out, ws)
    assert zc.device_status(p, ws) == zc.E_CORRUPT
    assert (d_out.cpu().numpy()[p.input_bytes:] == 0xEE).all()


@pytest.mark.parametrize("chunk_bytes", [2048, 4096])
def test_a_look_back_that_nobody_answers_gives_up(chunk_bytes):
    """chunk_bytes 2048 runs the row encoder, 4096 the slot encoder."""
    fmt, n = zc.FMT_BF16, 3000 * chunk_bytes // 2
    data = _bf16_weights(n, 21)
    p = zc.plan(fmt, n, chunk_bytes)
    hist = zo.histogram(fmt, data, n)
    cb = zc.build_codebook(p, hist, zc.POLICY_AUTO)
    d_in = torch.from_numpy(data).to(DEV)
    d_out = torch.empty(p.max_compressed_bytes, dtype=torch.uint8, device=DEV)
    ws = torch.zeros(p.workspace_bytes, dtype=torch.uint8, device=DEV)
    try:
        zc.test_set_wait_limit(1 << 9)
        zc.test_stall_encoder(1)                 # batch 0 of the tensor is never packed
        with pytest.raises(zc.ZcError) as e:
            zc.compress(p, cb, d_in, d_out, ws)
        assert e.value.status == zc.E_DEVICE_TIMEOUT
    finally:
        zc.test_stall_encoder(0)
        zc.test_set_wait_limit(0)
    torch.cuda.synchronize()
    nbytes = zc.compress(p, cb, d_in, d_out, ws)             # the same workspace, an ordinary call
    want = zo.compress(fmt, data, n, chunk_bytes, zo.build_codebook(hist, zo.POLICY_AUTO))
    assert nbytes == want.size and np.array_equal(d_out[:nbytes].cpu().numpy(), want)


@pytest.mark.parametrize("batched", [False, True])
def test_a_copy_that_never_comes_gives_up(batched):
    fmt, chunk_bytes, n = zc.FMT_BF16, 4096, 500 * 2048
    data = _bf16_weights(n, 22)
    cont = _oracle_container(fmt, data, n, chunk_bytes)
    p = zc.plan(fmt, n, chunk_bytes)
    d_comp = torch.from_numpy(cont).to(DEV)
    d_out = torch.empty(p.input_bytes, dtype=torch.uint8, device=DEV)
    ws = torch.zeros(256, dtype=torch.uint8, device=DEV)

    def run():
        if batched:
            zc.decompress_batch(zc.DecompressBatch([p], [d_comp], [cont.size], [d_out]), ws)
            return zc.batch_status(ws)[0]
        zc.decompress(p, d_comp, cont.size, d_out, ws)
        return zc.device_status(p, ws)

    try:
        zc.test_set_wait_limit(1 << 6)
        zc.test_stall_decoder(True)
        assert run() == zc.E_DEVICE_TIMEOUT
    finally:
        zc.test_stall_decoder(False)
        zc.test_set_wait_limit(0)
    assert run() == zc.OK
    assert np.array_equal(d_out.cpu().numpy(), data[: p.input_bytes])


@pytest.mark.parametrize("fmt", [zc.FMT_BF16, zc.FMT_FP8_E4M3, zc.FMT_SCALE_U8])
def test_largest_chunk_size_with_both_streams_coded(fmt):
    chunk_bytes = 65536
    G = zo.group(fmt)
    n = (5 * chunk_bytes // 2 + 1000) * G
    rng = np.random.default_rng(17)
    if fmt == zc.FMT_BF16:
        data = _bf16_weights(n, 17)
    elif fmt == zc.FMT_SCALE_U8:
        data = np.clip(np.round(rng.normal(120, 1.5, n)), 0, 255).astype(np.uint8)
    else:
        x = torch.from_numpy((rng.standard_normal(n) * 0.02).astype(np.float32))
        data = (x / (x.abs().max() / 448)).to(torch.float8_e4m3fn).view(torch.uint8).numpy().copy()
    p = zc.plan(fmt, n, chunk_bytes)
    hist = zo.histogram(fmt, data, n)
    cb = zc.build_codebook(p, hist, zc.POLICY_HUFF_ALL)
    d_in = torch.from_numpy(data).to(DEV)
    d_out = torch.empty(p.max_compressed_bytes, dtype=torch.uint8, device=DEV)
    ws = torch.zeros(p.workspace_bytes, dtype=torch.uint8, device=DEV)
    nbytes = zc.compress(p, cb, d_in, d_out, ws)
    want = zo.compress(fmt, data, n, chunk_bytes, zo.build_codebook(hist, zo.POLICY_HUFF_ALL))
    assert nbytes == want.size and np.array_equal(d_out[:nbytes].cpu().numpy(), want)
    d_back = torch.empty(p.input_bytes, dtype=torch.uint8, device=DEV)
    zc.decompress(p, d_out, nbytes, d_back, ws)
    assert zc.device_status(p, ws) == zc.OK
    assert np.array_equal(d_back.cpu().numpy(), data[: p.input_bytes])
