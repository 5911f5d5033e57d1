"""Seeded synthetic workloads: matrix shape sets, flat-shard layouts, input tensors.

This module only *describes inputs*: which matrices exist, how a padded flat
FSDP-style shard buffer is cut into segments, and how seeded random tensors are
drawn.  It contains none of the optimizer's arithmetic, so both the CUDA
binding's tests and the independent CPU oracle may use it.

The paper evaluates on LLM weight matrices whose shapes it does not list; the
Llama-style shape sets below stand in for them.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass
from typing import List, Sequence, Tuple

import numpy as np

Shape = Tuple[int, int]

QUINTIC = (3.4445, -4.7750, 2.0315)   # legacy constant-coefficient quintic (Section 6.6 names it, prints no values)
NS_STEPS = 5                          # "five NS iterations" (Section 7.4, Muon comparison set-up)
ALIGN_ELEMS = 128                     # pad alignment of every segment start, in elements


# --------------------------------------------------------------------------- shape sets
def shapes_tiny() -> List[Shape]:
    """One transformer layer with d=256: Wq, Wk, Wv, Wo, W_up, W_down."""
    return [(256, 256)] * 4 + [(1024, 256), (256, 1024)]


def shapes_1b(layers: int = 16) -> List[Shape]:
    """1B-class Llama-style stack: d=2048, ffn 5632, GQA with 8 KV heads of dim 64."""
    per = [(2048, 2048), (2048, 2048), (512, 2048), (512, 2048), (5632, 2048), (5632, 2048), (2048, 5632)]
    return per * layers


def shapes_llama8b(layers: int = 32) -> List[Shape]:
    """Llama-3-8B matrix set: Wq, Wo, Wk, Wv, gate, up, down per layer."""
    per = [(4096, 4096), (4096, 4096), (1024, 4096), (1024, 4096), (14336, 4096), (14336, 4096), (4096, 14336)]
    return per * layers


def shapes_moe(layers: int = 4, experts: int = 64) -> List[Shape]:
    """Many-small-matrix stress: per layer 64 experts x {gate, up, down} plus four attention matrices."""
    per = [(1408, 2048)] * (2 * experts) + [(2048, 1408)] * experts + [(2048, 2048)] * 4
    return per * layers


def shapes_odd() -> List[Shape]:
    """Ragged shapes that exercise unaligned heads/tails, zero-row shards and 1x1."""
    return [(37, 53), (130, 7), (5, 1000), (64, 64), (1, 1), (300, 129)]


CONFIGS = {
    "tiny": shapes_tiny,
    "1b": shapes_1b,
    "llama8b": shapes_llama8b,
    "moe": shapes_moe,
}


def ns_flops(shapes: Sequence[Shape], steps: int = NS_STEPS) -> Tuple[int, int]:
    """(dense-equivalent, symmetry-exploiting) flop counts of `steps` NS iterations."""
    dense = sym = 0
    for m, n in shapes:
        s, l = min(m, n), max(m, n)
        dense += 4 * s * s * l + 2 * s ** 3
        sym += 3 * s * s * l + s ** 3
    return dense * steps, sym * steps


# --------------------------------------------------------------------------- layouts
@dataclass(frozen=True)
class Segment:
    matrix: int        # index into the shape list
    elem_begin: int    # first element (row-major linear index) of the matrix this segment holds
    elem_count: int    # number of consecutive elements
    flat_offset: int   # element offset in the flat buffer (= shard * shard_len + offset inside the shard)


@dataclass(frozen=True)
class Layout:
    shapes: Tuple[Shape, ...]
    num_shards: int
    shard_len: int             # elements per shard, a multiple of `align`
    align: int
    segments: Tuple[Segment, ...]

    @property
    def flat_len(self) -> int:
        return self.num_shards * self.shard_len

    @property
    def payload(self) -> int:
        return sum(m * n for m, n in self.shapes)


def _up(x: int, a: int) -> int:
    return (x + a - 1) // a * a


def layout_per_param(shapes: Sequence[Shape], num_shards: int, align: int = ALIGN_ELEMS) -> Layout:
    """Per-parameter ceil-chunk row split (the uneven ceil-chunk sharding of Sections 4.4 and 5.5).

    Shard r holds rows [r*ceil(m/S), min(m, (r+1)*ceil(m/S))) of every matrix; inside a
    shard the pieces are packed in matrix order, each start aligned up to `align`
    elements.  Trailing shards may hold no rows of a small matrix.
    """
    segs: List[Segment] = []
    shard_len = 0
    per_shard: List[List[Tuple[int, int, int, int]]] = []
    for r in range(num_shards):
        off = 0
        rows: List[Tuple[int, int, int, int]] = []
        for i, (m, n) in enumerate(shapes):
            ch = -(-m // num_shards)
            r0 = min(m, r * ch)
            k = min(m, (r + 1) * ch) - r0
            if k <= 0 or n == 0:
                continue
            off = _up(off, align)
            rows.append((i, r0 * n, k * n, off))
            off += k * n
        per_shard.append(rows)
        shard_len = max(shard_len, _up(off, align))
    shard_len = max(shard_len, align)
    for r, rows in enumerate(per_shard):
        for (i, eb, ec, off) in rows:
            segs.append(Segment(i, eb, ec, r * shard_len + off))
    return Layout(tuple(shapes), num_shards, shard_len, align, tuple(segs))


def layout_flat_concat(shapes: Sequence[Shape], num_shards: int, align: int = ALIGN_ELEMS) -> Layout:
    """Flat concatenation of all matrices cut into S nearly equal parts.

    The cut points are element positions rounded up to a multiple of `align`, so a cut
    usually falls inside a matrix (and inside a row).  Inside a shard the pieces keep
    their order and each start is aligned up to `align` elements.
    """
    total = sum(m * n for m, n in shapes)
    target = _up(-(-total // num_shards), align) if total else align
    starts = []
    acc = 0
    for m, n in shapes:
        starts.append(acc)
        acc += m * n
    per_shard: List[List[Tuple[int, int, int, int]]] = []
    shard_len = 0
    for r in range(num_shards):
        lo, hi = min(total, r * target), min(total, (r + 1) * target)
        off = 0
        rows = []
        for i, (m, n) in enumerate(shapes):
            b = max(lo, starts[i])
            e = min(hi, starts[i] + m * n)
            if e <= b:
                continue
            off = _up(off, align)
            rows.append((i, b - starts[i], e - b, off))
            off += e - b
        per_shard.append(rows)
        shard_len = max(shard_len, _up(off, align))
    shard_len = max(shard_len, align)
    segs = [Segment(i, eb, ec, r * shard_len + off) for r, rows in enumerate(per_shard) for (i, eb, ec, off) in rows]
    return Layout(tuple(shapes), num_shards, shard_len, align, tuple(segs))


# --------------------------------------------------------------------------- seeded data
def stream_seed(config: str, step: int, matrix: int, role: str) -> int:
    """One independent 63-bit seed per (config, step, matrix index, role)."""
    h = hashlib.sha256(f"{config}|{step}|{matrix}|{role}".encode()).digest()
    return int.from_bytes(h[:8], "little") & ((1 << 63) - 1)


def _rng(config: str, step: int, matrix: int, role: str) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(stream_seed(config, step, matrix, role)))


def param_np(config: str, matrix: int, shape: Shape, std: float = 0.02) -> np.ndarray:
    """fp32 parameters ~ N(0, std^2)."""
    return (_rng(config, 0, matrix, "param").standard_normal(shape, dtype=np.float32) * np.float32(std)).astype(np.float32)


def grad_np(config: str, step: int, matrix: int, shape: Shape, std: float = 1e-3, row_scaled: bool = False) -> np.ndarray:
    """fp32 gradient draw.  row_scaled: Z ~ N(0,1) times one scale per row, log-uniform in [1e-4, 1e-2]."""
    g = _rng(config, step, matrix, "grad")
    z = g.standard_normal(shape, dtype=np.float32)
    if row_scaled:
        rho = np.exp(g.uniform(np.log(1e-4), np.log(1e-2), size=(shape[0], 1))).astype(np.float32)
        return (z * rho).astype(np.float32)
    return (z * np.float32(std)).astype(np.float32)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Input-format helper: fp32 array -> uint16 bf16 bit patterns (round to nearest even).

    Used only to *produce inputs* that are stored as bf16; implemented through torch's
    cast so that it shares nothing with the oracle's or the kernels' rounding code.
    """
    import torch

    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> the fp32 values they denote (exact widening)."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


def device_draw(config: str, step: int, matrix: int, role: str, shape: Shape, device, *, std: float,
                dtype, row_scaled: bool = False):
    """Seeded draw directly on a torch device (bench and full-size tests).

    The stream differs from the numpy one; consumers that need the values on the host
    copy the tensor back, so parity never depends on RNG portability.
    """
    import torch

    gen = torch.Generator(device=device)
    gen.manual_seed(stream_seed(config, step, matrix, role))
    z = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    if row_scaled:
        u = torch.rand((shape[0], 1), generator=gen, device=device, dtype=torch.float32)
        lo, hi = float(np.log(1e-4)), float(np.log(1e-2))
        z.mul_(torch.exp(u * (hi - lo) + lo))
    else:
        z.mul_(std)
    return z.to(dtype)
