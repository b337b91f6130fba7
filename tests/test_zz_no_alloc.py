"""zc_compress_noalloc: compression for callers that are not allowed to allocate device memory.

Such callers (a serving loop that must stay off the allocator, a plugin that only receives input and
output buffers, code running under an exhausted memory pool) cannot hand the library a workspace.  The
entry point keeps its scratch in a fixed device array inside the library instead.  This test calls it
through the C ABI twice in a row, on different tensors, and requires the containers to be byte-identical
to those of zc_compress, which takes the scratch from the caller.  It runs last in the suite on purpose.
"""
import numpy as np
import pytest
import torch

import oracle as zo
from paper_2508_19263_b200 import binding as zc
from paper_2508_19263_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _compress_both_ways(fmt, d_in, n, chunk_bytes, policy):
    p = zc.plan(fmt, n, chunk_bytes)
    hist = zc.histogram(p, d_in).cpu().numpy().astype(np.uint64)
    cb = zc.build_codebook(p, hist, policy)
    d_ref = torch.full((p.max_compressed_bytes,), 0x11, dtype=torch.uint8, device=DEV)
    d_new = torch.full((p.max_compressed_bytes,), 0x22, dtype=torch.uint8, device=DEV)
    d_ws = torch.empty(p.workspace_bytes, dtype=torch.uint8, device=DEV)
    n_ref = zc.compress(p, cb, d_in, d_ref, d_ws)
    n_new = zc.compress_noalloc(p, cb, d_in, d_new)
    assert n_new == n_ref
    assert torch.equal(d_new[:n_new], d_ref[:n_ref])              # integer work: bit-exact, no tolerance
    # the CPU oracle writes the same container
    want = zo.compress(fmt, d_in.cpu().numpy(), n, chunk_bytes, zo.build_codebook(hist, policy))
    assert n_new == want.size and np.array_equal(d_new[:n_new].cpu().numpy(), want)
    # the asynchronous form: nothing comes back with the call, the status is read from the built-in scratch
    d_async = torch.full((p.max_compressed_bytes,), 0x33, dtype=torch.uint8, device=DEV)
    assert zc.compress_noalloc(p, cb, d_in, d_async, sync=False) is None
    assert zc.noalloc_status() == zc.OK
    assert torch.equal(d_async[:n_new], d_new[:n_new])
    # and the container decodes back to the input
    d_back = torch.empty(p.input_bytes, dtype=torch.uint8, device=DEV)
    zc.decompress(p, d_new, n_new, d_back, d_ws)
    assert zc.device_status(p, d_ws) == zc.OK
    assert torch.equal(d_back, d_in[: p.input_bytes])
    return n_new


def test_noalloc_matches_compress_on_two_calls_in_a_row():
    # first call: BF16 weights, several chunks and a ragged tail; the built-in scratch is left dirty by it
    spec = wl.TensorSpec("a", (300, 4099), 0.02, 11)
    d_in, n, _ = wl.make_weight(spec, zc.FMT_BF16, DEV)
    first = _compress_both_ways(zc.FMT_BF16, d_in, n, 8192, zc.POLICY_AUTO)
    # second call right after it: another format, other chunk size, both streams coded
    spec = wl.TensorSpec("b", (512, 4096), 0.01, 12)
    d_in, n, _ = wl.make_weight(spec, zc.FMT_FP8_E4M3, DEV)
    second = _compress_both_ways(zc.FMT_FP8_E4M3, d_in, n, 4096, zc.POLICY_HUFF_ALL)
    assert first > 0 and second > 0
    # and the first tensor once more: stale scratch of the second call must not matter
    spec = wl.TensorSpec("a", (300, 4099), 0.02, 11)
    d_in, n, _ = wl.make_weight(spec, zc.FMT_BF16, DEV)
    assert _compress_both_ways(zc.FMT_BF16, d_in, n, 8192, zc.POLICY_AUTO) == first


def test_noalloc_refuses_plans_beyond_its_scratch():
    n = (zc.NOALLOC_MAX_CHUNKS + 1) * 512                          # 1 KiB chunks of BF16: 512 elements each
    p = zc.plan(zc.FMT_BF16, n, 1024)
    assert p.n_chunks == zc.NOALLOC_MAX_CHUNKS + 1
    cb = zc.build_codebook(p, np.ones((2, 256)), zc.POLICY_AUTO)
    d_in = torch.zeros(16, dtype=torch.uint8, device=DEV)          # never read: the call is refused before any launch
    d_out = torch.zeros(p.max_compressed_bytes, dtype=torch.uint8, device=DEV)
    with pytest.raises(zc.ZcError) as e:
        zc.compress_noalloc(p, cb, d_in, d_out)
    assert e.value.status == zc.E_TOO_LARGE
    # exactly at the limit it is accepted
    n = zc.NOALLOC_MAX_CHUNKS * 512
    p = zc.plan(zc.FMT_BF16, n, 1024)
    d_in = torch.zeros(2 * n, dtype=torch.uint8, device=DEV)
    hist = zc.histogram(p, d_in).cpu().numpy().astype(np.uint64)
    cb = zc.build_codebook(p, hist, zc.POLICY_HUFF_ALL)
    d_out = torch.zeros(p.max_compressed_bytes, dtype=torch.uint8, device=DEV)
    d_ws = torch.empty(p.workspace_bytes, dtype=torch.uint8, device=DEV)
    assert zc.compress_noalloc(p, cb, d_in, d_out) == zc.compress(p, cb, d_in, d_out.clone(), d_ws)
