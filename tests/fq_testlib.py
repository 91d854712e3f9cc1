"""Shared helpers of the GPU parity tests: make a layer from seeded inputs, quantise it with the
CPU oracle, hand the codes to the library."""
from __future__ import annotations

import numpy as np
import torch

import fq_synth as S
from oracle import fq_oracle as O

GEMV_TOL = 1e-3     # relative L2, decode
GEMM_TOL = 5e-3     # relative L2, prefill


def make_layer(cfg: int, layer: int, n_out: int, k_in: int, bits: int):
    """Seeded W -> oracle quantiser.  Returns numpy (codes u8, scales u16, zeros u16)."""
    w = S.weight_rows(S.tensor_key(cfg, layer, S.TENSOR_W), 0, n_out, k_in).numpy()
    return O.quantize(w, bits)


def to_dev(codes, scales, zeros):
    return (torch.from_numpy(codes).cuda(), torch.from_numpy(scales.view(np.float16)).cuda(),
            torch.from_numpy(zeros.view(np.float16)).cuda())


def x_fp16(cfg: int, layer: int, rows: int, k_in: int) -> torch.Tensor:
    return S.activations(S.tensor_key(cfg, layer, S.TENSOR_X), rows, k_in, torch.float16)


def x_bf16(cfg: int, layer: int, rows: int, k_in: int) -> torch.Tensor:
    return S.activations(S.tensor_key(cfg, layer, S.TENSOR_X), rows, k_in, torch.bfloat16)


def bits_of(t: torch.Tensor) -> np.ndarray:
    """uint16 bit patterns of an fp16 / bf16 tensor (on any device)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def f64_of(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()
