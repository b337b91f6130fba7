"""Seeded synthetic tensors shaped like the paper's workloads.

This module only *makes inputs*: Gaussian draws, the quantisers that turn them
into BF16 / FP8 E4M3 / packed FP4 E2M1 bytes, and the tensor lists of the five
benchmark configurations.  It contains none of the codec's arithmetic (no field
split, histogram, code construction, packing or decoding) and is the one module
that both the CUDA library's callers and the CPU oracle's callers may use.

The paper measures on real checkpoints, model weights and K/V caches (Sec. 4);
those are not available offline, so these tensors stand in for them: same
shapes, same storage formats, Gaussian values with the stated spreads.

Every generator returns a ``torch.uint8`` tensor holding the raw element bytes
(little-endian BF16, one byte per FP8 element, two FP4 elements per byte with
the even element in the low nibble) plus the element count.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Iterator, List, Optional, Tuple

import torch

BF16, FP8_E4M3, FP4_E2M1, SCALE_U8, FP8_E5M2 = 1, 2, 3, 4, 5
FORMAT_NAMES = {BF16: "bf16", FP8_E4M3: "fp8_e4m3", FP4_E2M1: "fp4_e2m1", FP8_E5M2: "fp8_e5m2"}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _randn(shape, std: float, seed: int, device) -> torch.Tensor:
    return torch.randn(shape, generator=_gen(seed, device), device=device, dtype=torch.float32) * std


# ---- quantisers (input preparation only) ---------------------------------------------------

def to_bf16_bytes(x: torch.Tensor) -> torch.Tensor:
    """fp32 -> BF16 with round-to-nearest-even, returned as bytes."""
    return x.to(torch.bfloat16).contiguous().view(torch.uint8).reshape(-1)


def to_e4m3_bytes(x: torch.Tensor, scale: torch.Tensor) -> torch.Tensor:
    """fp32 -> FP8 E4M3 of x/scale, clamped to +-448 before the RNE cast, as bytes."""
    y = (x / scale).clamp_(-448.0, 448.0)
    return y.to(torch.float8_e4m3fn).contiguous().view(torch.uint8).reshape(-1)


_E2M1_THRESH = (0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0)
_E2M1_TIE_UP = (0.75, 1.75, 3.5)     # ties go to the neighbour with an even mantissa bit


def to_mxfp4_bytes(x: torch.Tensor, block: int = 32) -> Tuple[torch.Tensor, torch.Tensor]:
    """fp32 rows -> MXFP4: one E8M0 scale byte per `block` elements along the last axis and
    E2M1 elements (RNE, saturating), two per byte with the even element in the low nibble.
    Returns (packed element bytes, scale bytes)."""
    assert x.shape[-1] % block == 0
    xb = x.reshape(-1, block)
    amax = xb.abs().amax(dim=1, keepdim=True)
    # shared exponent = floor(log2(amax)) - emax(E2M1), emax = 2; an all-zero block takes the smallest scale
    e = torch.floor(torch.log2(torch.where(amax > 0, amax, torch.ones_like(amax)))) - 2.0
    e = torch.where(amax > 0, e, torch.full_like(e, -127.0)).clamp_(-127.0, 127.0)
    scale_bytes = (e + 127.0).to(torch.uint8).reshape(-1)
    y = xb * torch.exp2(-e)
    ay = y.abs().clamp_(max=6.0)
    code = torch.zeros_like(ay, dtype=torch.int32)
    for t in _E2M1_THRESH:
        code += (ay > t).to(torch.int32)
    for t in _E2M1_TIE_UP:
        code += (ay == t).to(torch.int32)
    code |= (torch.signbit(y).to(torch.int32) << 3)
    code = code.reshape(-1, 2)
    packed = (code[:, 0] | (code[:, 1] << 4)).to(torch.uint8)
    return packed.contiguous(), scale_bytes.contiguous()


# ---- tensor lists of the benchmark configurations ---------------------------------------------

@dataclass
class TensorSpec:
    name: str
    shape: Tuple[int, ...]
    std: float
    seed: int

    @property
    def n_elems(self) -> int:
        return math.prod(self.shape)


def llama8b_stack(config_id: int, n_layers: int = 32, hidden: int = 4096, kv: int = 1024,
                  ffn: int = 14336, vocab: int = 128256, include_embedding: bool = True) -> List[TensorSpec]:
    """The 225 weight tensors of a Llama-8B-shaped stack: layer l draws N(0, (0.02/sqrt(l+1))^2),
    the embedding N(0, 0.02^2).  seed = 1000*config + 10*layer + index."""
    out = []
    for l in range(n_layers):
        std = 0.02 / math.sqrt(l + 1)
        shapes = [("q", (hidden, hidden)), ("k", (kv, hidden)), ("v", (kv, hidden)), ("o", (hidden, hidden)),
                  ("gate", (ffn, hidden)), ("up", (ffn, hidden)), ("down", (hidden, ffn))]
        for i, (nm, shp) in enumerate(shapes):
            out.append(TensorSpec(f"layers.{l}.{nm}", shp, std, 1000 * config_id + 10 * l + i))
    if include_embedding:
        out.append(TensorSpec("embedding", (vocab, hidden), 0.02, 1000 * config_id + 10 * n_layers))
    return out


def make_weight(spec: TensorSpec, fmt: int, device) -> Tuple[torch.Tensor, int, Optional[torch.Tensor]]:
    """Generate one weight tensor in `fmt`.  Returns (element bytes, n_elems, side scales or None).
    FP8 uses one fp32 scale per output row (amax_row/448); FP4 uses MX blocks of 32 along the row."""
    x = _randn(spec.shape, spec.std, spec.seed, device)
    if fmt == BF16:
        return to_bf16_bytes(x), spec.n_elems, None
    if fmt == FP8_E4M3:
        scale = (x.abs().amax(dim=-1, keepdim=True) / 448.0).clamp_(min=1e-30)
        return to_e4m3_bytes(x, scale), spec.n_elems, scale.reshape(-1)
    if fmt == FP8_E5M2:                          # the wide-range FP8 format: cast as it is (RNE), no scale
        return x.to(torch.float8_e5m2).view(torch.uint8).reshape(-1), spec.n_elems, None
    if fmt == FP4_E2M1:
        packed, scales = to_mxfp4_bytes(x)
        return packed, spec.n_elems, scales
    if fmt == SCALE_U8:                          # the E8M0 block scales of the tensor's MXFP4 form, as a byte stream
        _, scales = to_mxfp4_bytes(x)
        return scales, scales.numel(), None
    raise ValueError(fmt)


def checkpoint_pair(spec: TensorSpec, device, rel_step: float = 0.03, frozen_rows: float = 0.0) -> Tuple[torch.Tensor, torch.Tensor, int]:
    """Two consecutive BF16 checkpoints of one weight tensor: the earlier one is the tensor of `make_weight`, the
    later one is every weight moved by a relative step N(0, rel_step^2) (seed + 7) before the BF16 cast, so that
    most exponents and the upper mantissa bits stay the same.  frozen_rows: share of the leading rows (first
    dimension) that the step leaves untouched (1.0: a frozen tensor, the later checkpoint equals the earlier one).
    Returns (later bytes, earlier bytes, n_elems)."""
    x = _randn(spec.shape, spec.std, spec.seed, device)
    base = to_bf16_bytes(x)
    step = 1.0 + rel_step * torch.randn(spec.shape, generator=_gen(spec.seed + 7, device), device=device, dtype=torch.float32)
    keep = int(round(frozen_rows * spec.shape[0]))
    if keep:
        step[:keep] = 1.0
    x.mul_(step)
    return to_bf16_bytes(x), base, spec.n_elems


def frozen_rows_of(spec: TensorSpec) -> float:
    """The *_delta_frozen workloads: the tensors of the even layers did not change at all, in all other tensors the
    first half of the rows did not change (three quarters of the weights are untouched in all)."""
    parts = spec.name.split(".")
    if parts[0] == "layers" and int(parts[1]) % 2 == 0:
        return 1.0
    return 0.5


def config1_tensor(device) -> Tuple[torch.Tensor, int]:
    """One 1024x1024 FP8 E4M3 weight tensor, N(0, 0.02^2), per-tensor scale amax/448, seed 0."""
    x = _randn((1024, 1024), 0.02, 0, device)
    scale = x.abs().amax() / 448.0
    return to_e4m3_bytes(x, scale), 1024 * 1024


def kv_cache_tensor(fmt: int, layer: int, which: int, device, batch: int = 8, kv_heads: int = 8,
                    seq: int = 32768, head_dim: int = 128) -> Tuple[torch.Tensor, int]:
    """K (which=0) or V (which=1) cache of one layer, [batch, kv_heads, seq, head_dim] with head_dim
    contiguous.  Per (tensor, head): channel std = exp(N(0,1)), four distinct channels scaled x10;
    values are Gaussian per channel.  FP8 uses one per-tensor scale amax/448."""
    seed = 5000 + 10 * layer + which
    g = _gen(seed, device)
    std = torch.exp(torch.randn((kv_heads, head_dim), generator=g, device=device))
    for h in range(kv_heads):
        idx = torch.randperm(head_dim, generator=g, device=device)[:4]
        std[h, idx] *= 10.0
    x = torch.randn((batch, kv_heads, seq, head_dim), generator=g, device=device, dtype=torch.float32)
    x *= std.reshape(1, kv_heads, 1, head_dim)
    n = batch * kv_heads * seq * head_dim
    if fmt == BF16:
        return to_bf16_bytes(x), n
    if fmt == FP8_E4M3:
        return to_e4m3_bytes(x, x.abs().amax() / 448.0), n
    raise ValueError(fmt)


def small_cases(device="cpu") -> Iterator[Tuple[str, int, torch.Tensor, int]]:
    """Reduced versions of the five configurations for quick parity runs: (name, fmt, bytes, n_elems)."""
    t, n = config1_tensor(device)
    yield "cfg1_fp8_1024x1024", FP8_E4M3, t, n
    for fmt in (BF16, FP8_E4M3, FP4_E2M1):
        spec = TensorSpec("layers.3.k_small", (96, 4096), 0.02 / 2.0, 2033)
        b, n, _ = make_weight(spec, fmt, device)
        yield f"weights_{FORMAT_NAMES[fmt]}_96x4096", fmt, b, n
    for fmt in (BF16, FP8_E4M3):
        b, n = kv_cache_tensor(fmt, 0, 0, device, batch=1, kv_heads=2, seq=1024, head_dim=128)
        yield f"kv_{FORMAT_NAMES[fmt]}_1x2x1024x128", fmt, b, n
