"""The input generators' casts against the oracle's value tables.  Needs no GPU.

The synthetic workloads are fp32 draws cast to BF16 / FP8 / MXFP4 by `workloads.py` (torch casts and a hand-written
E2M1 quantiser).  Here every cast is checked against the definition of the format as the oracle states it: the
produced bit pattern must be the code whose value (oracle value function) is nearest to the input, ties going to
the code with an even last mantissa bit, magnitudes beyond the largest finite value saturating where the
generator says so.  The search for the nearest code is written out here and uses nothing but the value tables.
"""
import numpy as np
import torch

import oracle as zo
from paper_2508_19263_b200 import workloads as wl


def _nearest_codes(table, mags):
    """table[c] = value of magnitude code c (ascending); returns the code nearest to each magnitude, ties to even."""
    table = np.asarray(table, np.float64)
    assert np.all(np.diff(table) > 0)
    hi = np.clip(np.searchsorted(table, mags, side="left"), 0, len(table) - 1)
    lo = np.clip(hi - 1, 0, len(table) - 1)
    d_lo, d_hi = np.abs(mags - table[lo]), np.abs(table[hi] - mags)
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    return np.where(pick_hi, hi, lo)


def _samples(seed, n, scale_lo=-20, scale_hi=6):
    """fp32 values over many binades, plus exact midpoints between neighbours of a coarse grid (ties)."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal(n) * np.exp2(rng.integers(scale_lo, scale_hi, n))
    return x.astype(np.float32)


def test_bf16_cast_is_round_to_nearest_even_on_the_oracle_s_values():
    table = [zo.bf16_value(c) for c in range(0x7F80)]                    # finite magnitudes, ascending
    x = _samples(1, 20000)
    # exact ties: halfway between two neighbouring BF16 values
    c = np.random.default_rng(2).integers(0x100, 0x7000, 4000)
    ties = ((np.array(table)[c] + np.array(table)[c + 1]) / 2).astype(np.float32)
    assert np.all(ties.astype(np.float64) == (np.array(table)[c] + np.array(table)[c + 1]) / 2)
    x = np.concatenate([x, ties, -ties])
    got = wl.to_bf16_bytes(torch.from_numpy(x)).numpy().view(np.uint16)
    want = _nearest_codes(table, np.abs(x.astype(np.float64))) | (np.signbit(x).astype(np.int64) << 15)
    assert np.array_equal(got, want.astype(np.uint16))


def test_e4m3_cast_is_round_to_nearest_even_and_saturates_on_the_oracle_s_values():
    table = [zo.e4m3_value(c) for c in range(0x7F)]                      # 0x7F is NaN
    assert table[-1] == 448.0
    x = _samples(3, 20000, -12, 12)
    c = np.random.default_rng(4).integers(0, 0x7E, 2000)
    ties = ((np.array(table)[c] + np.array(table)[c + 1]) / 2).astype(np.float32)
    x = np.concatenate([x, ties, -ties, np.float32([448.0, 500.0, -1e9, 464.0, 465.0])])
    for scale in (1.0, 0.03125, 3.0):
        y = (torch.from_numpy(x) / torch.tensor(scale)).numpy().astype(np.float64)    # the generator divides in fp32
        got = wl.to_e4m3_bytes(torch.from_numpy(x), torch.tensor(scale)).numpy()
        want = _nearest_codes(table, np.minimum(np.abs(y), 448.0)) | (np.signbit(y).astype(np.int64) << 7)
        assert np.array_equal(got, want.astype(np.uint8)), scale


def test_e5m2_cast_is_round_to_nearest_even_on_the_oracle_s_values():
    table = [zo.e5m2_value(c) for c in range(0x7C)]                      # 0x7C is infinity
    x = _samples(5, 20000, -14, 10)
    x = x[np.abs(x) < 57344.0]
    c = np.random.default_rng(6).integers(0, 0x7B, 2000)
    ties = ((np.array(table)[c] + np.array(table)[c + 1]) / 2).astype(np.float32)
    x = np.concatenate([x, ties, -ties])
    got = torch.from_numpy(x).to(torch.float8_e5m2).view(torch.uint8).numpy()
    want = _nearest_codes(table, np.abs(x.astype(np.float64))) | (np.signbit(x).astype(np.int64) << 7)
    assert np.array_equal(got, want.astype(np.uint8))
    spec = wl.llama8b_stack(3, n_layers=1)[1]
    data, n, _ = wl.make_weight(spec, zo.FP8_E5M2, "cpu")                # the generator's own E5M2 path
    assert n == spec.n_elems and data.numel() == n


def test_mxfp4_quantiser_against_the_oracle_s_e2m1_values_and_the_block_scale_rule():
    table = [zo.e2m1_value(c) for c in range(8)]
    assert table == [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    assert [zo.e2m1_value(c | 8) for c in range(1, 8)] == [-v for v in table[1:]]
    rng = np.random.default_rng(7)
    x = (rng.standard_normal((4000, 32)) * np.exp2(rng.integers(-30, 20, (4000, 1)))).astype(np.float32)
    x[5] = 0.0                                                           # an all-zero block
    x[6, :] = np.float32([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0] * 4) * np.float32(4.0)   # every tie, amax 24 -> e = 2
    x[7, :] = -x[6, :]
    packed, scales = wl.to_mxfp4_bytes(torch.from_numpy(x))
    packed, scales = packed.numpy(), scales.numpy()
    assert scales.shape == (4000,) and packed.shape == (4000 * 16,)
    amax = np.abs(x.astype(np.float64)).max(axis=1)
    # shared exponent: the largest power of two not above amax, less the exponent of E2M1's largest binade (2)
    e = np.where(amax > 0, np.floor(np.log2(np.where(amax > 0, amax, 1.0))) - 2, -127).clip(-127, 127)
    assert np.array_equal(scales, (e + 127).astype(np.uint8))
    assert np.all(np.exp2(e[amax > 0] + 2) <= amax[amax > 0]) and np.all(amax[amax > 0] < np.exp2(e[amax > 0] + 3))
    y = x.astype(np.float64) * np.exp2(-e)[:, None]
    want = _nearest_codes(table, np.minimum(np.abs(y), 6.0)) | (np.signbit(y).astype(np.int64) << 3)
    nib = np.stack([packed & 0xF, packed >> 4], axis=1).reshape(4000, 32)
    assert np.array_equal(nib, want)
    # decoded values: within half of the widest step (1) of the scaled input, or, saturated, less than 2 below it
    dec = np.vectorize(zo.e2m1_value)(nib) * np.exp2(e)[:, None]
    assert np.all(np.abs(dec - x) < np.exp2(e)[:, None] * 2.0 + 1e-300)
