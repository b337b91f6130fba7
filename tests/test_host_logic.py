"""Host-side logic of libzc against the oracle, and the shape of the C ABI.  Needs no GPU."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle as zo
from paper_2508_19263_b200 import binding as zc
from paper_2508_19263_b200 import build as zbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FORMATS = [zc.FMT_BF16, zc.FMT_FP8_E4M3, zc.FMT_FP4_E2M1, zc.FMT_SCALE_U8, zc.FMT_FP8_E5M2]


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(zbuild.LIB)
    declared = set()
    for hdr in os.listdir(os.path.join(ROOT, "include")):
        text = open(os.path.join(ROOT, "include", hdr)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        declared |= set(re.findall(r"\b(zc_[a-z0-9_]+)\s*\(", text))
    assert {"zc_plan", "zc_histogram", "zc_build_codebook", "zc_compress", "zc_decompress", "zc_stats"} <= declared
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in include/ but not exported"


def test_enums_match_the_oracle_s_numbering():
    assert (zc.FMT_BF16, zc.FMT_FP8_E4M3, zc.FMT_FP4_E2M1, zc.FMT_SCALE_U8, zc.FMT_FP8_E5M2) == \
        (zo.BF16, zo.FP8_E4M3, zo.FP4_E2M1, zo.SCALE_U8, zo.FP8_E5M2)
    assert (zc.POLICY_AUTO, zc.POLICY_HUFF_ALL, zc.POLICY_RAW_ALL, zc.POLICY_STATIC) == \
        (zo.POLICY_AUTO, zo.POLICY_HUFF_ALL, zo.POLICY_RAW_ALL, zo.POLICY_STATIC)
    assert (zc.MODE_RAW, zc.MODE_HUFF) == (zo.RAW, zo.HUFF)


@pytest.mark.parametrize("fmt", FORMATS)
def test_plan_geometry(fmt):
    for n in [0, 2, 6, 1000, 4096, 65536 * 3 + 10, 1 << 24]:
        for cb in [1024, 8192, 32768, 65536]:
            p = zc.plan(fmt, n, cb)
            assert p.n_syms == zo.n_syms(fmt, n)
            assert p.input_bytes == zo.input_bytes(fmt, n)
            assert p.n_chunks == -(-p.n_syms // (cb // 2))
            assert p.info.syms_per_chunk == cb // 2 and p.info.syms_per_subchunk == cb // 64
            assert p.info.group == zo.group(fmt)
            assert p.max_compressed_bytes == zo.container_bound(fmt, n, cb)
            assert p.workspace_bytes >= 256 + 8 * p.n_chunks and p.workspace_bytes % 256 == 0


def test_every_accepted_chunk_size_has_a_launch_shape():
    """Whatever zc_plan accepts, the encoder (any number of coded streams, every class of pack slots) and the
    decoder (one or both streams coded) have a launch shape for; beyond the limit the plan itself is refused.
    Half-size slots never leave room for fewer worker warps than the ordinary ones."""
    for cb in range(1024, 65536 + 1, 1024):
        p = zc.plan(zc.FMT_BF16, 1 << 20, cb)
        for n_coded in (0, 1, 2):
            for slots in (0, 1, 2):
                assert zc.test_encoder_workers(p, n_coded, slots) >= 1, (cb, n_coded, slots)
            assert zc.test_encoder_workers(p, n_coded, 2) >= zc.test_encoder_workers(p, n_coded, 0)
            assert zc.test_encoder_workers(p, n_coded, 3) == 0
        for both in (False, True):
            assert zc.test_decoder_warps(p, both) >= 8, (cb, both)


def test_plan_rejects_bad_arguments():
    for cb in [0, 512, 1000, 1025, 65536 + 1024, 131072, 262144, 1 << 20]:
        with pytest.raises(zc.ZcError) as e:
            zc.plan(zc.FMT_BF16, 100, cb)
        assert e.value.status == zc.E_INVALID_ARG
    with pytest.raises(zc.ZcError) as e:
        zc.plan(7, 100, 1024)
    assert e.value.status == zc.E_UNSUPPORTED
    with pytest.raises(zc.ZcError) as e:
        zc.plan(zc.FMT_FP4_E2M1, 101, 1024)
    assert e.value.status == zc.E_INVALID_ARG
    p = zc.plan(zc.FMT_BF16, 10, 1024)
    with pytest.raises(zc.ZcError) as e:
        zc.build_codebook(p, np.zeros((2, 256)), 9)
    assert e.value.status == zc.E_UNSUPPORTED
    assert zc.strerror(zc.E_CORRUPT) and zc.strerror(99) == "unknown status"


def _adversarial_histograms(rng):
    H = []
    for n in [1, 2, 3, 5, 8, 16, 17, 31, 64, 100, 255, 256]:
        H.append(("equal", np.concatenate([np.full(n, 7), np.zeros(256 - n)])))
        fib = [1, 1]
        while len(fib) < n:
            fib.append(min(fib[-1] + fib[-2], 1 << 40))
        H.append(("fib", np.concatenate([np.array(fib[:n]), np.zeros(256 - n)])))
        H.append(("pow2", np.concatenate([2 ** np.minimum(np.arange(n), 40), np.zeros(256 - n)])))
        H.append(("pow2rev", np.concatenate([2 ** np.minimum(np.arange(n), 40)[::-1], np.zeros(256 - n)])))
        H.append(("big", np.concatenate([rng.integers((1 << 33) - 5, (1 << 33) + 5, n), np.zeros(256 - n)])))
        H.append(("fewvalues", np.concatenate([rng.integers(1, 4, n), np.zeros(256 - n)])))
    out = []
    for name, h in H:
        h = h.astype(np.uint64)
        out.append((name, h))
        out.append((name + "_perm", h[rng.permutation(256)]))
    return out


def _compare_codebook(h2, policy):
    p = zc.plan(zc.FMT_BF16, 16, 1024)
    got = zc.build_codebook(p, h2, policy)
    want = zo.build_codebook(h2, policy)
    for s in range(2):
        mode, lens, codes = got.get(s)
        assert np.array_equal(lens, want.lengths[s]), (s, h2[s][:16])
        assert np.array_equal(codes, want.codes[s])
        assert mode == want.modes[s]


def test_codebook_matches_oracle_on_adversarial_histograms():
    rng = np.random.default_rng(0)
    H = _adversarial_histograms(rng)
    for i in range(0, len(H) - 1, 2):
        h2 = np.stack([H[i][1], H[i + 1][1]])
        for policy in (zc.POLICY_AUTO, zc.POLICY_HUFF_ALL, zc.POLICY_RAW_ALL, zc.POLICY_STATIC):
            _compare_codebook(h2, policy)


def test_codebook_matches_oracle_on_random_histograms():
    rng = np.random.default_rng(1)
    for trial in range(1500):
        h2 = np.zeros((2, 256), np.uint64)
        for s in range(2):
            n = int(rng.integers(0, 257)) if trial % 3 else int(rng.integers(0, 12))
            kind = trial % 5
            if kind == 0:
                c = rng.integers(1, 6, n)                                 # many ties
            elif kind == 1:
                c = np.floor(1e7 * np.exp(-rng.uniform(0.05, 1.0) * np.arange(n))) + 1   # skewed: limit binds
            elif kind == 2:
                c = rng.integers(1, 1 << 30, n)
            elif kind == 3:
                c = 2 ** rng.integers(0, 30, n)
            else:
                c = np.floor(rng.exponential(1000.0, n)) + 1
            idx = rng.permutation(256)[:n]
            h2[s, idx] = np.asarray(c, dtype=np.uint64)
        _compare_codebook(h2, zc.POLICY_AUTO)
        if trial % 4 == 0:
            _compare_codebook(h2, zc.POLICY_STATIC)


def test_dictionary_object_follows_the_replacement_rule():
    """zc_dict_*: the same decisions as the oracle's statement of the rule on seeded sequences of sizes, the same
    codebooks after every rebuild, and the argument checks."""
    rng = np.random.default_rng(5)
    p = zc.plan(zc.FMT_BF16, 1 << 16, 4096)
    for trial in range(20):
        tol = float(rng.choice([0.0, 0.01, 0.05, 0.25]))
        h = rng.integers(0, 1 << 20, (2, 256)).astype(np.uint64) * (rng.random((2, 256)) < 0.4)
        d, o = zc.Dictionary(p, h, tol), zo.StaticDictionary(h, tol)
        ratio = 0.7
        for step in range(60):
            ratio = min(max(ratio * float(rng.uniform(0.97, 1.04)), 0.05), 1.2)
            nin = int(rng.integers(1, 1 << 30))
            nout = int(round(nin * ratio))
            got, want = d.observe(nin, nout), o.observe(nin, nout)
            assert got == want, (trial, step)
            if got:
                h = rng.integers(0, 1 << 16, (2, 256)).astype(np.uint64)
                d.rebuild(p, h)
                o.rebuild(h)
            cb = d.codebook
            for s in range(2):
                mode, lens, codes = cb.get(s)
                assert mode == o.codebook.modes[s] and np.array_equal(lens, o.codebook.lengths[s])
                assert np.array_equal(codes, o.codebook.codes[s]) and lens.min() >= 1
        info = d.info
        assert info.n_observed == 60 and info.n_rebuilds == o.n_rebuilds and info.tolerance == tol
        assert bool(info.has_baseline) == (o.baseline is not None)
        if o.baseline is not None:
            assert info.baseline_ratio == o.baseline
    h = np.ones((2, 256), np.uint64)
    for bad in (-0.1, float("nan"), float("inf")):
        with pytest.raises(zc.ZcError):
            zc.Dictionary(p, h, bad)
    d = zc.Dictionary(p, h, 0.1)
    with pytest.raises(zc.ZcError):
        d.observe(0, 10)


def test_codebook_on_workload_like_histograms():
    import torch
    from paper_2508_19263_b200 import workloads as wl
    for name, fmt, t, n in wl.small_cases("cpu"):
        data = t.numpy()
        h = zo.histogram(fmt, data, n)
        for policy in (zc.POLICY_AUTO, zc.POLICY_HUFF_ALL):
            _compare_codebook(h, policy)


@pytest.mark.parametrize("fmt", FORMATS)
def test_word_level_split_and_merge_match_oracle(fmt):
    rng = np.random.default_rng(fmt)
    cases = [rng.integers(0, 256, 16, dtype=np.uint8) for _ in range(3000)]
    cases += [np.full(16, v, np.uint8) for v in (0, 0xFF, 0x80, 0x7F, 0x0F, 0xF0, 0x55, 0xAA)]
    for b in range(16):
        for bit in range(8):
            x = np.zeros(16, np.uint8); x[b] = 1 << bit
            cases.append(x)
    n_elems = {zc.FMT_BF16: 8, zc.FMT_FP8_E4M3: 16, zc.FMT_FP4_E2M1: 32, zc.FMT_SCALE_U8: 16, zc.FMT_FP8_E5M2: 16}[fmt]
    for x in cases:
        e, sm = zc.test_split16(fmt, x)
        we, wsm = zo.split(fmt, x, n_elems)
        assert np.array_equal(e, we) and np.array_equal(sm, wsm), x
        assert np.array_equal(zc.test_merge16(fmt, e, sm), x)


def _container(fmt, n, chunk_bytes, policy, seed=0):
    rng = np.random.default_rng(seed)
    nb = zo.input_bytes(fmt, n)
    if fmt == zo.BF16:
        import torch
        data = torch.from_numpy((rng.standard_normal(n) * 0.02).astype(np.float32)).to(torch.bfloat16).view(torch.uint8).numpy().copy()
    else:
        data = rng.choice(256, size=nb, p=np.r_[np.full(16, 0.04), np.full(240, 0.36 / 240)]).astype(np.uint8)
    hist = zo.histogram(fmt, data, n)
    cb = zo.build_codebook(hist, policy)
    return data, hist, cb, zo.compress(fmt, data, n, chunk_bytes, cb)


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("policy", [zc.POLICY_AUTO, zc.POLICY_HUFF_ALL, zc.POLICY_RAW_ALL])
@pytest.mark.parametrize("cbytes", [2048, 16384])
def test_validate_accepts_oracle_containers_and_rejects_damage(fmt, policy, cbytes):
    n = 5 * (cbytes // 2) + 36
    data, hist, cb, cont = _container(fmt, n, cbytes, policy)
    p = zc.plan(fmt, n, cbytes)
    assert zc.validate_container(p, cont) == zc.OK
    assert cont.size <= p.max_compressed_bytes
    # a plan with other parameters does not accept it
    assert zc.validate_container(zc.plan(fmt, n + 2, cbytes), cont) == zc.E_CORRUPT
    assert zc.validate_container(zc.plan(fmt, n, 2 * cbytes), cont) == zc.E_CORRUPT
    assert zc.validate_container(p, cont[:-1]) == zc.E_CORRUPT
    hd = zo.parse_header(cont)
    for off in (0, 4, 6, 7, 8, 16, 20, 24, 25, 26, 27, 32, 40, 48, 64, 72, 80, 88, 96, 104, 112, 120):
        bad = cont.copy(); bad[off] ^= 0x01
        assert zc.validate_container(p, bad) == zc.E_CORRUPT, off
    for s in range(2):
        if hd["streams"][s]["mode"] != zo.HUFF:
            continue
        sec = hd["streams"][s]["section_off"]
        used = np.flatnonzero(cont[sec:sec + 256])
        bad = cont.copy(); bad[sec + used[0]] += 1                    # Kraft sum no longer 1
        assert zc.validate_container(p, bad) == zc.E_CORRUPT
        bad = cont.copy(); bad[sec + 256] ^= 1                        # first chunk offset
        assert zc.validate_container(p, bad) == zc.E_CORRUPT
        _, _, tab = zo.read_tables(cont, s)
        bad = cont.copy(); bad[tab + hd["sub_end_bytes"] * 7 + 1] ^= 0x40   # a subchunk end jumps
        assert zc.validate_container(p, bad) == zc.E_CORRUPT
        bad = cont.copy(); bad[-3] = 1                                # guard not zero
        assert zc.validate_container(p, bad) == zc.E_CORRUPT


def test_stats_match_oracle():
    n = 40000
    data, hist, ocb, cont = _container(zo.BF16, n, 4096, zo.POLICY_AUTO)
    p = zc.plan(zc.FMT_BF16, n, 4096)
    cb = zc.build_codebook(p, hist, zc.POLICY_AUTO)
    for header in (None, cont[:128]):
        st = zc.stats(p, cb, hist, header)
        tot = 0
        for s in range(2):
            want = zo.stream_stats(hist[s], ocb.lengths[s], ocb.modes[s])
            got = st.stream[s]
            assert (got.n_syms, got.raw_bits, got.payload_bits, got.mode, got.n_active_symbols, got.max_len) == \
                   (want["n_syms"], want["raw_bits"], want["payload_bits"], want["mode"], want["n_active"], want["max_len"])
            assert abs(got.avg_len - want["avg_len"]) <= 1e-12 * max(1.0, want["avg_len"])
            assert abs(got.entropy_bits - want["entropy_bits"]) <= 1e-12 * max(1.0, want["entropy_bits"])
            tot += want["payload_bits"]
        assert st.in_bytes == 2 * n
        assert abs(st.ratio_payload - tot / (16.0 * n)) < 1e-15
        if header is not None:
            assert st.out_bytes == cont.size and abs(st.ratio_container - cont.size / (2.0 * n)) < 1e-15
            hd = zo.parse_header(cont)
            assert st.stream[0].payload_bits == hd["streams"][0]["payload_bits"]
        else:
            assert st.out_bytes == 0


def test_threaded_codebook_builder_matches_the_single_one():
    rng = np.random.default_rng(3)
    n = 37
    hists = np.zeros((n, 2, 256), np.uint64)
    for t in range(n):
        k = int(rng.integers(1, 256))
        hists[t, 0, rng.choice(256, k, replace=False)] = rng.integers(1, 1 << 20, k)
        hists[t, 1] = rng.integers(0, 1000, 256)
    hists[5] = 0                                                       # an empty tensor
    plans = [zc.plan(zc.FMT_BF16, int(hists[t, 0].sum()), 4096) for t in range(n)]
    for policy in (zc.POLICY_AUTO, zc.POLICY_HUFF_ALL, zc.POLICY_RAW_ALL):
        for threads in (0, 1, 3, 64):
            many = zc.build_codebooks(plans, hists, policy, threads)
            assert len(many) == n
            for t in range(n):
                one = zc.build_codebook(plans[t], hists[t], policy)
                for s in range(2):
                    a, b = many[t].get(s), one.get(s)
                    assert a[0] == b[0] and np.array_equal(a[1], b[1]) and np.array_equal(a[2], b[2])
    assert zc.build_codebooks([], np.zeros((0, 2, 256), np.uint64)) == []


def test_codebook_builder_against_the_oracle_s_on_a_million_histograms(tmp_path):
    """tests/codebook_fuzz.c, one process per core: ties, Fibonacci, powers of two, counts near 2^33, ...

    ZC_FUZZ_HISTOGRAMS sets the total (default 10^6, or 125 000 per core where fewer than 8 cores are available)."""
    import subprocess
    exe = str(tmp_path / "codebook_fuzz")
    src = os.path.join(os.path.dirname(os.path.abspath(__file__)), "codebook_fuzz.c")
    subprocess.check_call(["gcc", "-O2", "-std=c99", "-Wall", "-o", exe, src, "-ldl"])
    cores = len(os.sched_getaffinity(0))
    total = int(os.environ.get("ZC_FUZZ_HISTOGRAMS", min(1_000_000, 125_000 * cores)))
    per = -(-total // cores)
    procs = [subprocess.Popen([exe, zbuild.build_library(), zo.build(), str(per), str(1000 + i)],
                              stdout=subprocess.PIPE, text=True) for i in range(cores)]
    outs = [p.communicate()[0] for p in procs]
    for p, out in zip(procs, outs):
        assert p.returncode == 0 and out.startswith("ok "), out[-2000:]
    assert sum(int(o.split()[1]) for o in outs) >= total
