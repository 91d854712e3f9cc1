"""ctypes front end of the CPU oracle (fq_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
"CPU baseline" leg of the benchmark; never by the library that is under test.
The C file is compiled on first use with the system gcc (no CUDA involved).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading
from typing import Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fq_oracle.c")
_LIB = os.path.join(_HERE, "libfq_oracle.so")
_lock = threading.Lock()
_lib = None

GROUP = 128


def build(force: bool = False) -> str:
    """Compile fq_oracle.c into libfq_oracle.so next to it (if stale) and return the path."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off",
                                   "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        i64, u8p, u16p, u32p = C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p
        lib.fqo_f16_to_f64.restype = C.c_double
        lib.fqo_f16_to_f64.argtypes = [C.c_uint16]
        lib.fqo_f64_to_f16.restype = C.c_uint16
        lib.fqo_f64_to_f16.argtypes = [C.c_double]
        lib.fqo_bf16_to_f64.restype = C.c_double
        lib.fqo_bf16_to_f64.argtypes = [C.c_uint16]
        lib.fqo_quantize.restype = None
        lib.fqo_quantize.argtypes = [C.c_void_p, i64, i64, C.c_int, u8p, u16p, u16p]
        lib.fqo_pack_bitstream.restype = None
        lib.fqo_pack_bitstream.argtypes = [u8p, i64, i64, C.c_int, u32p]
        lib.fqo_unpack_bitstream.restype = None
        lib.fqo_unpack_bitstream.argtypes = [u32p, i64, i64, C.c_int, u8p]
        lib.fqo_pack_planes.restype = None
        lib.fqo_pack_planes.argtypes = [u8p, i64, i64, u32p]
        lib.fqo_child_codes.restype = None
        lib.fqo_child_codes.argtypes = [u32p, i64, i64, C.c_int, u8p]
        lib.fqo_dequant_one.restype = C.c_double
        lib.fqo_dequant_one.argtypes = [C.c_uint, C.c_int, C.c_int, C.c_uint16, C.c_uint16]
        lib.fqo_dequant.restype = None
        lib.fqo_dequant.argtypes = [u8p, u16p, u16p, i64, i64, C.c_int, C.c_int, C.c_void_p]
        lib.fqo_matmul.restype = None
        lib.fqo_matmul.argtypes = [u8p, u16p, u16p, i64, i64, C.c_int, C.c_int,
                                   u16p, i64, i64, C.c_int, C.c_void_p]
        lib.fqo_footprint.restype = C.c_uint64
        lib.fqo_footprint.argtypes = [C.c_void_p, C.c_void_p, u8p, i64]
        _lib = lib
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


# ---- scalar conversions ----------------------------------------------------

def f16_to_f64(h: int) -> float:
    return _load().fqo_f16_to_f64(int(h))


def f64_to_f16(v: float) -> int:
    return _load().fqo_f64_to_f16(float(v))


def bf16_to_f64(b: int) -> float:
    return _load().fqo_bf16_to_f64(int(b))


# ---- quantiser ---------------------------------------------------------------

def quantize(w: np.ndarray, bits: int):
    """W float32 [N][K] -> (codes uint8 [N][K], scales uint16 [N][K/128], zeros uint16 [N][K/128])."""
    w = _c(w, np.float32)
    n, k = w.shape
    assert k % GROUP == 0 and 2 <= bits <= 8
    codes = np.empty((n, k), np.uint8)
    scales = np.empty((n, k // GROUP), np.uint16)
    zeros = np.empty((n, k // GROUP), np.uint16)
    _load().fqo_quantize(_p(w), n, k, bits, _p(codes), _p(scales), _p(zeros))
    return codes, scales, zeros


# ---- formats -------------------------------------------------------------------

def pack_bitstream(codes: np.ndarray, bits: int) -> np.ndarray:
    codes = _c(codes, np.uint8)
    n, k = codes.shape
    assert (k * bits) % 32 == 0
    out = np.empty((n, k * bits // 32), np.uint32)
    _load().fqo_pack_bitstream(_p(codes), n, k, bits, _p(out))
    return out


def unpack_bitstream(packed: np.ndarray, k_in: int, bits: int) -> np.ndarray:
    packed = _c(packed, np.uint32)
    n = packed.shape[0]
    codes = np.empty((n, k_in), np.uint8)
    _load().fqo_unpack_bitstream(_p(packed), n, k_in, bits, _p(codes))
    return codes


def pack_planes(q8: np.ndarray) -> np.ndarray:
    """uint8 [N][K] -> uint32 [8][N][K/32], most significant plane first."""
    q8 = _c(q8, np.uint8)
    n, k = q8.shape
    assert k % 32 == 0
    out = np.empty((8, n, k // 32), np.uint32)
    _load().fqo_pack_planes(_p(q8), n, k, _p(out))
    return out


def child_codes(planes: np.ndarray, k_in: int, bits: int) -> np.ndarray:
    """Codes of the b-bit child, read from the first b planes only."""
    planes = _c(planes[:bits], np.uint32)
    n = planes.shape[1]
    codes = np.empty((n, k_in), np.uint8)
    _load().fqo_child_codes(_p(planes), n, k_in, bits, _p(codes))
    return codes


# ---- dequantisation and matmul ----------------------------------------------------

def dequant_one(q: int, bits: int, parent_bits: int, scale: int, zero: int) -> float:
    return _load().fqo_dequant_one(int(q), bits, parent_bits, int(scale), int(zero))


def dequant(codes, scales, zeros, bits: int, parent_bits: int | None = None) -> np.ndarray:
    codes, scales, zeros = _c(codes, np.uint8), _c(scales, np.uint16), _c(zeros, np.uint16)
    n, k = codes.shape
    out = np.empty((n, k), np.float64)
    _load().fqo_dequant(_p(codes), _p(scales), _p(zeros), n, k, bits,
                        bits if parent_bits is None else parent_bits, _p(out))
    return out


def matmul(codes, scales, zeros, bits: int, x_bits: np.ndarray, x_is_bf16: bool = False,
           parent_bits: int | None = None) -> np.ndarray:
    """Y[m][n] = sum_k X[m][k] * w^[n][k] in float64.  x_bits: uint16 [M][K] (fp16 or bf16 patterns)."""
    codes, scales, zeros = _c(codes, np.uint8), _c(scales, np.uint16), _c(zeros, np.uint16)
    x_bits = _c(x_bits, np.uint16)
    if x_bits.ndim == 1:
        x_bits = x_bits[None, :]
    n, k = codes.shape
    m = x_bits.shape[0]
    assert x_bits.shape[1] == k
    y = np.empty((m, n), np.float64)
    _load().fqo_matmul(_p(codes), _p(scales), _p(zeros), n, k, bits,
                       bits if parent_bits is None else parent_bits,
                       _p(x_bits), m, k, 1 if x_is_bf16 else 0, _p(y))
    return y


def gemv(codes, scales, zeros, bits, x_bits, parent_bits=None) -> np.ndarray:
    """Decode: x fp16 patterns [K] or [B][K]."""
    return matmul(codes, scales, zeros, bits, x_bits, False, parent_bits)


def gemm(codes, scales, zeros, bits, x_bits, parent_bits=None) -> np.ndarray:
    """Prefill: X bf16 patterns [M][K]."""
    return matmul(codes, scales, zeros, bits, x_bits, True, parent_bits)


# ---- footprint ---------------------------------------------------------------------

def footprint(n_out: Sequence[int], k_in: Sequence[int], bits: Sequence[int]) -> int:
    n = _c(n_out, np.int64)
    k = _c(k_in, np.int64)
    b = _c(bits, np.uint8)
    return int(_load().fqo_footprint(_p(n), _p(k), _p(b), len(b)))


# ---- one-way transitions (Sec. II-C, Sec. III-B) -------------------------------------

def transition(n_out: Sequence[int], k_in: Sequence[int], nested: Sequence[bool], from_bits: Sequence[int],
               to_bits: Sequence[int]) -> dict:
    """Memory accounting of moving from one elastic configuration to another, layer by layer.

    The paper asks that a transition only ever lowers a module's bit-width (Sec. III-B, the one-way
    constraint) and that as little memory as possible has to be brought in (Sec. II-C).  Per layer:
      nested layer  : the child keeps a prefix of the parent's planes; lowering frees the dropped planes
                      (N*K*(b0-b1)/8 bytes) and loads nothing, raising loads the re-appended planes;
                      scale/zero words are shared by every width and never move;
      packed layer  : widths are separate stored variants; a change frees the old variant and loads the
                      new one, codes and scale/zero words (4 bytes per group of 128) alike.
    Returns bytes_freed, bytes_loaded, layers_changed, one_way (no layer goes up) and the footprints of
    both configurations."""
    freed = loaded = changed = 0
    one_way = True
    for n, k, nest, b0, b1 in zip(n_out, k_in, nested, from_bits, to_bits):
        n, k, b0, b1 = int(n), int(k), int(b0), int(b1)
        if b0 == b1:
            continue
        changed += 1
        if b1 > b0:
            one_way = False
        if nest:
            if b1 < b0:
                freed += n * k * (b0 - b1) // 8
            else:
                loaded += n * k * (b1 - b0) // 8
        else:
            meta = n * (k // 128) * 4
            freed += n * k * b0 // 8 + meta
            loaded += n * k * b1 // 8 + meta
    return {"bytes_freed": freed, "bytes_loaded": loaded, "layers_changed": changed, "one_way": one_way,
            "footprint_from": footprint(n_out, k_in, from_bits), "footprint_to": footprint(n_out, k_in, to_bits)}


def rel_l2(got: np.ndarray, ref: np.ndarray) -> float:
    """||got - ref||_2 / ||ref||_2 over all elements (0 if both are all-zero)."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    den = float(np.sqrt((ref * ref).sum()))
    num = float(np.sqrt(((got - ref) ** 2).sum()))
    return num / den if den > 0 else num
