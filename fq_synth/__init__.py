"""Seeded synthetic inputs for the elastic dequantize-and-matmul path.

This module only *draws numbers*: real-valued weight matrices, activation
vectors, per-layer bit-widths and elastic configuration chains.  It contains
none of the method's arithmetic (no quantiser, no packing, no dequantisation,
no matmul) so that the CPU oracle and the CUDA library can both be fed from it
without sharing any code that is under test.

Every tensor element is a pure function of (key, element index): the generator
is counter based (SplitMix64, Steele/Lea/Flood 2014: output_i =
finalise(key + (i + 1) * 0x9E3779B97F4A7C15)), evaluated with wrapping 64-bit
integer arithmetic only.  A "normal" variate is the centred sum of twelve
16-bit uniform fields (Irwin-Hall with n = 12, range +-6 sigma) scaled in
float64 and rounded once to float32, so the same bits come out of torch on a
CPU, torch on a GPU, or any row subset computed on its own -- there is no
transcendental function whose last bit could differ between devices.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Sequence, Tuple

import numpy as np
import torch

MASTER_SEED = 2501_07139

_M64 = (1 << 64) - 1


def _s64(v: int) -> int:
    """Two's-complement view of an unsigned 64-bit constant (torch has no uint64 math)."""
    v &= _M64
    return v - (1 << 64) if v >= (1 << 63) else v


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_MUL1 = _s64(0xBF58476D1CE4E5B9)
_MUL2 = _s64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _finalise(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _MUL1
    z = (z ^ _lsr(z, 27)) * _MUL2
    return z ^ _lsr(z, 31)


def splitmix64(key: int, counter: torch.Tensor) -> torch.Tensor:
    """SplitMix64 output number `counter` (int64 tensor, >= 0) of the stream seeded with `key`."""
    return _finalise((counter + 1) * _GOLDEN + _s64(key))


def splitmix64_scalar(key: int, counter: int) -> int:
    """Pure-Python SplitMix64, used to derive per-tensor keys."""
    z = (key + (counter + 1) * 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def tensor_key(config: int, layer: int, tensor: int, master: int = MASTER_SEED) -> int:
    """Key of one tensor: a hash chain over (master seed, config, layer, tensor id)."""
    k = splitmix64_scalar(master, config)
    k = splitmix64_scalar(k, layer)
    return splitmix64_scalar(k, tensor)


TENSOR_W, TENSOR_X, TENSOR_BITS, TENSOR_CHAIN = 0, 1, 2, 3

_IH_MEAN = 6 * 65535                    # mean of twelve uniform 16-bit fields
_IH_STD = math.sqrt(65536.0 ** 2 - 1.0)  # their standard deviation


def normal_f32(key: int, start: int, count: int, sigma: float,
               device: torch.device | str = "cpu") -> torch.Tensor:
    """`count` approximately-normal float32 values with standard deviation `sigma`:
    elements start .. start+count-1 of the infinite stream that belongs to `key`."""
    if count == 0:
        return torch.empty(0, dtype=torch.float32, device=device)
    e = torch.arange(start, start + count, dtype=torch.int64, device=device)
    total = torch.zeros(count, dtype=torch.int64, device=device)
    for j in range(3):
        h = splitmix64(key, e * 3 + j)
        for sh in (0, 16, 32, 48):
            total += (h >> sh) & 0xFFFF
    scale = float(sigma) / _IH_STD
    return ((total - _IH_MEAN).to(torch.float64) * scale).to(torch.float32)


def weight_rows(key: int, n0: int, n1: int, k_in: int, sigma: float = 0.02,
                device: torch.device | str = "cpu", chunk_rows: int = 2048) -> torch.Tensor:
    """Rows n0..n1-1 of the float32 weight matrix W[N][K] that belongs to `key`
    (element (n, k) is stream element n*K + k), W ~ N(0, sigma^2)."""
    out = torch.empty((n1 - n0, k_in), dtype=torch.float32, device=device)
    for r0 in range(n0, n1, chunk_rows):
        r1 = min(n1, r0 + chunk_rows)
        out[r0 - n0:r1 - n0] = normal_f32(key, r0 * k_in, (r1 - r0) * k_in, sigma, device).view(r1 - r0, k_in)
    return out


def activations(key: int, rows: int, k_in: int, dtype: torch.dtype = torch.float16,
                device: torch.device | str = "cpu") -> torch.Tensor:
    """Activation matrix X[rows][K] ~ N(0, 1), rounded once (nearest-even) to `dtype`."""
    return normal_f32(key, 0, rows * k_in, 1.0, device).view(rows, k_in).to(dtype)


# ---------------------------------------------------------------------------
# Layer stacks (shapes of the linear layers of Llama-2 decoders)
# ---------------------------------------------------------------------------

@dataclass(frozen=True)
class LayerShape:
    name: str      # e.g. "blk3.q"
    block: int
    module: int    # 0 = attention (q, k, v, o), 1 = MLP (gate, up, down)
    phase: int     # dependency phase inside a block: {q,k,v}=0, o=1, {gate,up}=2, down=3
    n_out: int
    k_in: int


_STACKS = {
    "7b": (32, 4096, 11008),
    "13b": (40, 5120, 13824),
}


def stack_shapes(model: str, n_blocks: int | None = None) -> List[LayerShape]:
    """The linear layers of a Llama-2-shaped decoder stack in execution order."""
    blocks, hidden, ffn = _STACKS[model]
    if n_blocks is not None:
        blocks = n_blocks
    out: List[LayerShape] = []
    for b in range(blocks):
        for nm, ph, n, k, mod in (("q", 0, hidden, hidden, 0), ("k", 0, hidden, hidden, 0),
                                  ("v", 0, hidden, hidden, 0), ("o", 1, hidden, hidden, 0),
                                  ("gate", 2, ffn, hidden, 1), ("up", 2, ffn, hidden, 1),
                                  ("down", 3, hidden, ffn, 1)):
            out.append(LayerShape(f"blk{b}.{nm}", b, mod, ph, n, k))
    return out


def stack_phases(shapes: Sequence[LayerShape]) -> List[int]:
    """Global dependency phase of every layer: a layer may start only when every layer
    of the previous phase has finished ({q,k,v} -> o -> {gate,up} -> down -> next block)."""
    return [4 * s.block + s.phase for s in shapes]


def draw_bits(key: int, n_layers: int, choices: Sequence[int]) -> np.ndarray:
    """One bit-width per layer, i.i.d. uniform over `choices`."""
    rng = np.random.Generator(np.random.PCG64(key & _M64))
    return np.asarray(choices, dtype=np.uint8)[rng.integers(0, len(choices), size=n_layers)]


def average_bits(bits: Sequence[int], shapes: Sequence[LayerShape]) -> float:
    """Parameter-weighted mean bit-width (scale/zero metadata excluded)."""
    w = np.array([s.n_out * s.k_in for s in shapes], dtype=np.float64)
    return float((np.asarray(bits, dtype=np.float64) * w).sum() / w.sum())


def config_chain(key: int, shapes: Sequence[LayerShape], n_configs: int, avg_hi: float,
                 avg_lo: float, floor_bits: int, start_bits: int = 8) -> List[np.ndarray]:
    """A one-way chain of elastic configurations.

    Starts with every layer at `start_bits`.  For each of `n_configs` equally spaced
    targets from `avg_hi` down to `avg_lo`, a seeded random module (the attention or
    the MLP matrices of one block) that is still above `floor_bits` is lowered by one
    bit, again and again, until the parameter-weighted average is <= the target.
    Along the chain no layer's bit-width ever increases.
    """
    rng = np.random.Generator(np.random.PCG64(key & _M64))
    bits = np.full(len(shapes), start_bits, dtype=np.uint8)
    modules = sorted({(s.block, s.module) for s in shapes})
    members = {m: [i for i, s in enumerate(shapes) if (s.block, s.module) == m] for m in modules}
    targets = np.linspace(avg_hi, avg_lo, n_configs)
    chain: List[np.ndarray] = []
    for t in targets:
        while average_bits(bits, shapes) > t + 1e-12:
            live = [m for m in modules if bits[members[m][0]] > floor_bits]
            if not live:
                break
            m = live[int(rng.integers(0, len(live)))]
            bits[members[m]] -= 1
        chain.append(bits.copy())
    return chain


def sample_rows(key: int, n_out: int, count: int) -> np.ndarray:
    """Sorted distinct output rows to spot-check: always the first and last row, the rows
    on either side of a 16- and a 128-row tile edge when they exist, the rest seeded."""
    fixed = [r for r in (0, 15, 16, 127, 128, n_out - 1) if 0 <= r < n_out]
    rng = np.random.Generator(np.random.PCG64(key & _M64))
    extra = rng.integers(0, n_out, size=max(0, count)).tolist()
    return np.asarray(sorted(set(fixed + extra)), dtype=np.int64)
