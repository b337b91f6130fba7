"""K/V cache tensors coded at run time with precomputed dictionaries (Sec. 3.3, Sec. 5.2), against the CPU oracle.

One dictionary per kind of tensor (K, V) is built from the first step's tensor and reused for the pages of the
following steps without a histogram pass; when a page's ratio exceeds the baseline by more than the tolerance the
dictionary is rebuilt from that page and the page is coded again.  The same flow is run with the oracle's
statement of the rule and the oracle's coder; decisions and containers have to agree bit for bit.
"""
import numpy as np
import pytest
import torch

import oracle as zo
from paper_2508_19263_b200 import binding as zc
from paper_2508_19263_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _kv_page(fmt, which, step, tokens, drift):
    """[2, 2, tokens, 128] K or V page: Gaussian per channel, channel std log-normal, magnitude scaled by `drift`.
    FP8 uses one fixed scale for all steps, as a serving stack with a static K/V scale does."""
    g = torch.Generator(device="cpu").manual_seed(77 + which)
    std = torch.exp(torch.randn((2, 128), generator=g))
    g = torch.Generator(device="cpu").manual_seed(1000 * step + which)
    x = torch.randn((2, 2, tokens, 128), generator=g) * std.reshape(1, 2, 1, 128) * drift
    n = x.numel()
    if fmt == zc.FMT_BF16:
        return wl.to_bf16_bytes(x).to(DEV), n
    return wl.to_e4m3_bytes(x, torch.tensor(30.0 / 448.0)).to(DEV), n


@pytest.mark.parametrize("fmt", [zc.FMT_BF16, zc.FMT_FP8_E4M3])
@pytest.mark.parametrize("chunk_bytes", [1024, 4096])
def test_kv_pages_with_static_dictionaries_follow_the_oracle(fmt, chunk_bytes):
    tol = 0.03
    drifts = [1.0, 1.0, 1.05, 1.0, 1 / 64.0, 1 / 64.0, 1 / 60.0, 8.0, 8.0]      # two regime changes
    tokens = [50] * len(drifts)                  # pages of one size (12.5 chunks of 4 KiB in BF16), as in a paged cache
    dicts, odicts = {}, {}
    decisions, stored = [], []
    for step, (drift, tok) in enumerate(zip(drifts, tokens)):
        pages = [_kv_page(fmt, w, step, tok, drift) for w in range(2)]
        plans = [zc.plan(fmt, n, chunk_bytes) for _, n in pages]
        datas = [t.cpu().numpy() for t, _ in pages]
        if step == 0:
            for w in range(2):                   # the dictionaries: from the first page of each kind
                hist = zc.histogram(plans[w], pages[w][0]).cpu().numpy().astype(np.uint64)
                ohist = zo.histogram(fmt, datas[w], pages[w][1])
                assert np.array_equal(hist, ohist)
                dicts[w], odicts[w] = zc.Dictionary(plans[w], hist, tol), zo.StaticDictionary(ohist, tol)
        # both pages in one call, no histogram pass
        d_outs = [torch.full((p.max_compressed_bytes,), 0xEE, dtype=torch.uint8, device=DEV) for p in plans]
        enc = zc.CompressBatch(plans, [t for t, _ in pages], d_outs)
        enc.set_codebooks([dicts[w].codebook for w in range(2)])
        ws = torch.empty(enc.workspace_bytes, dtype=torch.uint8, device=DEV)
        sizes = zc.compress_batch(enc, ws)
        for w in range(2):
            p, data, n = plans[w], datas[w], pages[w][1]
            want = zo.compress(fmt, data, n, chunk_bytes, odicts[w].codebook)
            assert np.array_equal(d_outs[w][: sizes[w]].cpu().numpy(), want), (step, w)
            got_flag, want_flag = dicts[w].observe(p.input_bytes, sizes[w]), odicts[w].observe(data.size, want.size)
            assert got_flag == want_flag, (step, w)
            decisions.append(got_flag)
            if got_flag:
                hist = zc.histogram(p, pages[w][0]).cpu().numpy().astype(np.uint64)
                dicts[w].rebuild(p, hist)
                odicts[w].rebuild(zo.histogram(fmt, data, n))
                ws1 = torch.empty(p.workspace_bytes, dtype=torch.uint8, device=DEV)
                sizes[w] = zc.compress(p, dicts[w].codebook, pages[w][0], d_outs[w], ws1)
                want2 = zo.compress(fmt, data, n, chunk_bytes, odicts[w].codebook)
                assert np.array_equal(d_outs[w][: sizes[w]].cpu().numpy(), want2), (step, w)
                assert want2.size < want.size    # the new dictionary fits the page better
                assert dicts[w].observe(p.input_bytes, sizes[w]) is False and odicts[w].observe(data.size, want2.size) is False
            stored.append((p, pages[w][0], d_outs[w], sizes[w]))
    # the regime changes, and only they, replaced dictionaries
    per_step = [decisions[2 * s] or decisions[2 * s + 1] for s in range(len(drifts))]
    assert per_step == [False, False, False, False, True, False, False, True, False]
    assert all(dicts[w].info.n_rebuilds == odicts[w].n_rebuilds for w in range(2))

    # every stored page decodes, in one call; one of them also chunk by chunk
    plans = [s[0] for s in stored]
    backs = [torch.full((p.input_bytes + 16,), 0xEE, dtype=torch.uint8, device=DEV) for p in plans]
    ws = torch.zeros(256, dtype=torch.uint8, device=DEV)
    zc.decompress_batch(zc.DecompressBatch(plans, [s[2] for s in stored], [s[3] for s in stored], backs), ws)
    assert zc.batch_status(ws) == (zc.OK, None)
    for (p, d_in, _, _), back in zip(stored, backs):
        assert torch.equal(back[: p.input_bytes], d_in[: p.input_bytes]) and bool((back[p.input_bytes:] == 0xEE).all())
    p, d_in, d_comp, nbytes = max(stored, key=lambda s: s[0].n_chunks)
    ws1 = torch.empty(p.workspace_bytes, dtype=torch.uint8, device=DEV)
    for c in (0, p.n_chunks // 2, p.n_chunks - 1):
        lo, hi = c * chunk_bytes, min((c + 1) * chunk_bytes, p.input_bytes)
        out = torch.full((hi - lo + 16,), 0xEE, dtype=torch.uint8, device=DEV)
        zc.decompress_chunks(p, d_comp, nbytes, c, 1, out, ws1)
        assert zc.device_status(p, ws1) == zc.OK
        assert torch.equal(out[: hi - lo], d_in[lo:hi]) and bool((out[hi - lo:] == 0xEE).all())
