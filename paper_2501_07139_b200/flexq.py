"""ctypes binding of libflexq.so: argument marshalling only.

Every method has the name of the C function it calls.  torch is used for device memory
and streams; all computation happens inside the library's CUDA kernels.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

FQ_FMT_PACKED = 0
FQ_FMT_PLANES = 1
FQ_MAX_BATCH = 8

_HERE = os.path.dirname(os.path.abspath(__file__))
# FLEXQ_LIBRARY selects the file: unset = libflexq.so, "checked" = libflexq_checked.so (the bounds-checked build,
# `python -m paper_2501_07139_b200.build --checked`), anything else = a path.
_LIB_PATH = {None: os.path.join(_HERE, "libflexq.so"), "": os.path.join(_HERE, "libflexq.so"),
             "checked": os.path.join(_HERE, "libflexq_checked.so")}.get(os.environ.get("FLEXQ_LIBRARY"),
                                                                        os.environ.get("FLEXQ_LIBRARY"))
_lib = None

EXPORTS = [
    "fq_create", "fq_destroy", "fq_store_bytes", "fq_quantize_layer", "fq_pack_layer",
    "fq_set_config", "fq_gemv", "fq_gemv_batched", "fq_gemv_stack", "fq_gemm", "fq_export_layer",
    "fq_export_meta", "fq_storage_bytes", "fq_active_bits", "fq_status", "fq_strerror", "fq_gemv_static", "fq_transition", "fq_save", "fq_load", "fq_search_chain", "fq_prune_chain", "fq_sqdiff",
    "fq_set_wait_limit_ns", "fq_code_bytes", "fq_meta_bytes", "fq_stream_read", "fq_gemm_two_pass",
    "fq_host_variant", "fq_transition_swap",
]


class TransitionReport(C.Structure):
    _fields_ = [("bytes_freed", C.c_uint64), ("bytes_loaded", C.c_uint64), ("footprint_from", C.c_uint64),
                ("footprint_to", C.c_uint64), ("layers_changed", C.c_int), ("one_way", C.c_int)]


class SwapReport(C.Structure):
    _fields_ = [("bytes_loaded", C.c_uint64), ("bytes_freed", C.c_uint64), ("peak_extra_bytes", C.c_uint64),
                ("resident_bytes", C.c_uint64), ("footprint_from", C.c_uint64), ("footprint_to", C.c_uint64),
                ("layers_changed", C.c_int), ("one_way", C.c_int)]


class FlexQError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {fq_strerror(code)} ({code})")


def lib_path() -> str:
    return _LIB_PATH


def lib():
    """Loads libflexq.so (once).  Raises if it is missing: build it with
    `python -m paper_2501_07139_b200.build` or `__graft_entry__.build()`."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise FileNotFoundError(f"{_LIB_PATH} not built; run `python -m paper_2501_07139_b200.build`")
    L = C.CDLL(_LIB_PATH)
    vp, i, u64 = C.c_void_p, C.c_int, C.c_uint64
    L.fq_create.argtypes = [C.POINTER(vp), i, i]
    L.fq_destroy.argtypes = [vp]
    L.fq_store_bytes.argtypes = [i, i, i, i]
    L.fq_store_bytes.restype = C.c_size_t
    L.fq_quantize_layer.argtypes = [vp, i, i, i, i, vp, vp, vp, vp]
    L.fq_pack_layer.argtypes = [vp, i, i, i, i, i, i, vp, vp, vp, vp, vp]
    L.fq_set_config.argtypes = [vp, vp, i, C.POINTER(u64), vp]
    L.fq_transition.argtypes = [vp, vp, i, i, C.POINTER(TransitionReport), vp]
    L.fq_host_variant.argtypes = [vp, i, i, i, i, vp]
    L.fq_transition_swap.argtypes = [vp, vp, i, i, C.POINTER(SwapReport), vp]
    L.fq_save.argtypes = [vp, C.c_char_p, C.POINTER(u64)]
    L.fq_load.argtypes = [vp, C.c_char_p]
    L.fq_search_chain.argtypes = [vp, vp, vp, i, i, i, i, vp, C.POINTER(i), C.POINTER(C.c_double)]
    L.fq_prune_chain.argtypes = [vp, i, i, i, vp, C.c_double, vp, vp, C.POINTER(u64), C.POINTER(u64)]
    L.fq_sqdiff.argtypes = [vp, vp, C.c_size_t, vp, vp]
    L.fq_gemv.argtypes = [vp, i, vp, vp, vp]
    L.fq_gemv_batched.argtypes = [vp, i, vp, i, vp, vp]
    L.fq_gemv_static.argtypes = [vp, i, vp, vp, vp]
    L.fq_gemv_stack.argtypes = [vp, i, vp, vp, vp, vp, i, vp]
    L.fq_gemm.argtypes = [vp, i, vp, i, i, vp, i, vp]
    L.fq_gemm_two_pass.argtypes = [vp, i, vp, i, i, vp, i, vp]
    L.fq_export_layer.argtypes = [vp, i, i, vp, vp]
    L.fq_export_meta.argtypes = [vp, i, i, vp, vp, vp]
    L.fq_storage_bytes.argtypes = [vp]
    L.fq_storage_bytes.restype = u64
    L.fq_active_bits.argtypes = [vp, i]
    L.fq_status.argtypes = [vp]
    L.fq_set_wait_limit_ns.argtypes = [vp, u64]
    L.fq_stream_read.argtypes = [vp, vp, C.c_size_t, vp]
    L.fq_code_bytes.argtypes = [i, i, i]
    L.fq_code_bytes.restype = C.c_size_t
    L.fq_meta_bytes.argtypes = [i, i, i]
    L.fq_meta_bytes.restype = C.c_size_t
    L.fq_strerror.argtypes = [i]
    L.fq_strerror.restype = C.c_char_p
    for name in EXPORTS:
        fn = getattr(L, name)
        if fn.restype is C.c_int or fn.restype is None:
            fn.restype = C.c_int
    _lib = L
    return L


def fq_strerror(code: int) -> str:
    return lib().fq_strerror(int(code)).decode()


def fq_store_bytes(n_out: int, k_in: int, bits: int, fmt: int) -> int:
    return int(lib().fq_store_bytes(n_out, k_in, bits, fmt))


def fq_code_bytes(n_out: int, k_in: int, bits: int) -> int:
    return int(lib().fq_code_bytes(n_out, k_in, bits))


def fq_meta_bytes(n_out: int, k_in: int, group: int = 128) -> int:
    return int(lib().fq_meta_bytes(n_out, k_in, group))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(rc: int, where: str) -> int:
    if rc != 0:
        raise FlexQError(rc, where)
    return rc


def fq_search_chain(cost, sens, foot, stems: int, branches: int):
    """Algorithm 1 on host tables [module][level]; returns (chain as a list of level lists, curve cost)."""
    import numpy as np
    c = np.ascontiguousarray(cost, np.float64)
    s_ = np.ascontiguousarray(sens, np.float64)
    f = np.ascontiguousarray(foot, np.uint64)
    m, lv = c.shape
    chain = np.zeros((m * (lv - 1) + 1, m), np.uint8)
    n_states, curve = C.c_int(0), C.c_double(0.0)
    _check(lib().fq_search_chain(c.ctypes.data, s_.ctypes.data, f.ctypes.data, m, lv, stems, branches, chain.ctypes.data,
                                 C.byref(n_states), C.byref(curve)), "fq_search_chain")
    return chain[:n_states.value].tolist(), float(curve.value)


def fq_prune_chain(chain, n_levels: int, foot, fraction: float):
    """Sec. III-C; returns (pruned chain, set of dropped (module, level), storage before, storage after)."""
    import numpy as np
    ch = np.ascontiguousarray(chain, np.uint8)
    f = np.ascontiguousarray(foot, np.uint64)
    n_states, m = ch.shape
    out = np.zeros_like(ch)
    dropped = np.zeros((m, n_levels), np.uint8)
    before, after = C.c_uint64(0), C.c_uint64(0)
    _check(lib().fq_prune_chain(ch.ctypes.data, n_states, m, n_levels, f.ctypes.data, float(fraction), out.ctypes.data,
                                dropped.ctypes.data, C.byref(before), C.byref(after)), "fq_prune_chain")
    return out.tolist(), {(int(a), int(b)) for a, b in zip(*np.nonzero(dropped))}, int(before.value), int(after.value)


def fq_sqdiff(a: torch.Tensor, b: torch.Tensor) -> torch.Tensor:
    """Device tensor [sum (a-b)^2, sum b^2] (float64) over two bf16 tensors of the same size."""
    assert a.dtype == torch.bfloat16 and b.dtype == torch.bfloat16 and a.is_contiguous() and b.is_contiguous()
    assert a.numel() == b.numel()
    out = torch.empty(2, dtype=torch.float64, device=a.device)
    _check(lib().fq_sqdiff(a.data_ptr(), b.data_ptr(), a.numel(), out.data_ptr(), _stream()), "fq_sqdiff")
    return out


def fq_quantize_layer(w: torch.Tensor, bits: int, group: int = 128):
    """W float32 [N][K] on the GPU -> (codes uint8 [N][K], scales fp16 [N][K/128], zeros fp16 [N][K/128])."""
    assert w.is_cuda and w.dtype == torch.float32 and w.is_contiguous()
    n, k = w.shape
    codes = torch.empty((n, k), dtype=torch.uint8, device=w.device)
    scales = torch.empty((n, k // group), dtype=torch.float16, device=w.device)
    zeros = torch.empty((n, k // group), dtype=torch.float16, device=w.device)
    with torch.cuda.device(w.device):
        _check(lib().fq_quantize_layer(w.data_ptr(), n, k, bits, group, codes.data_ptr(), scales.data_ptr(),
                                       zeros.data_ptr(), _stream()), "fq_quantize_layer")
    return codes, scales, zeros


class FlexQ:
    """One library context.  Keeps the retained device buffers (the stored variants) alive."""

    def __init__(self, n_layers: int, device: int = 0):
        self._h = C.c_void_p()
        self.device = torch.device("cuda", device)
        _check(lib().fq_create(C.byref(self._h), device, n_layers), "fq_create")
        self.n_layers = n_layers
        self._keep = {}          # (layer, bits) -> stored variant retained by the context
        self._stack_keep = None

    # -- lifetime -----------------------------------------------------------------
    def fq_destroy(self):
        if self._h:
            lib().fq_destroy(self._h)
            self._h = C.c_void_p()
            self._keep.clear()

    def __del__(self):
        try:
            self.fq_destroy()
        except Exception:
            pass

    # -- packing --------------------------------------------------------------------
    def fq_pack_layer(self, layer: int, codes: torch.Tensor, scales: torch.Tensor, zeros: torch.Tensor,
                      bits: int, fmt: int = FQ_FMT_PACKED, group: int = 128):
        assert codes.is_cuda and codes.dtype == torch.uint8 and codes.is_contiguous()
        assert scales.dtype == torch.float16 and zeros.dtype == torch.float16
        n, k = codes.shape
        sb = fq_store_bytes(n, k, bits, fmt)
        if sb == 0 or group != 128:
            # let the library name the problem
            _check(lib().fq_pack_layer(self._h, layer, n, k, bits, group, fmt, codes.data_ptr(), scales.data_ptr(),
                                       zeros.data_ptr(), codes.data_ptr(), _stream()), "fq_pack_layer")
        store = torch.empty(sb, dtype=torch.uint8, device=self.device)
        _check(lib().fq_pack_layer(self._h, layer, n, k, bits, group, fmt, codes.data_ptr(),
                                   scales.contiguous().data_ptr(), zeros.contiguous().data_ptr(),
                                   store.data_ptr(), _stream()), "fq_pack_layer")
        self._keep[(layer, bits)] = store
        return store

    # -- configuration -------------------------------------------------------------------
    def fq_set_config(self, bits: Sequence[int]) -> int:
        arr = (C.c_uint8 * len(bits))(*[int(b) for b in bits])
        fp = C.c_uint64(0)
        _check(lib().fq_set_config(self._h, arr, len(bits), C.byref(fp), _stream()), "fq_set_config")
        return int(fp.value)

    def fq_transition(self, bits: Sequence[int], require_one_way: bool = True) -> dict:
        arr = (C.c_uint8 * len(bits))(*[int(b) for b in bits])
        rep = TransitionReport()
        _check(lib().fq_transition(self._h, arr, len(bits), 1 if require_one_way else 0, C.byref(rep), _stream()),
               "fq_transition")
        return {"bytes_freed": int(rep.bytes_freed), "bytes_loaded": int(rep.bytes_loaded),
                "layers_changed": int(rep.layers_changed), "one_way": bool(rep.one_way),
                "footprint_from": int(rep.footprint_from), "footprint_to": int(rep.footprint_to)}

    def fq_host_variant(self, layer: int, n_out: int, k_in: int, bits: int, store_host: torch.Tensor) -> None:
        """Registers a PACKED variant whose stored bytes lie in the (page-locked) host tensor `store_host`."""
        if store_host.device.type != "cpu" or not store_host.is_contiguous():
            raise ValueError("store_host must be a contiguous host tensor")
        if store_host.numel() * store_host.element_size() < fq_store_bytes(n_out, k_in, bits, FQ_FMT_PACKED):
            raise ValueError("store_host is smaller than fq_store_bytes")
        self._keep[("host", layer, bits)] = store_host       # the library reads it at every swap-in
        _check(lib().fq_host_variant(self._h, layer, n_out, k_in, bits, store_host.data_ptr()), "fq_host_variant")

    def fq_transition_swap(self, bits: Sequence[int], require_one_way: bool = True) -> dict:
        arr = (C.c_uint8 * len(bits))(*[int(b) for b in bits])
        rep = SwapReport()
        _check(lib().fq_transition_swap(self._h, arr, len(bits), 1 if require_one_way else 0, C.byref(rep), _stream()),
               "fq_transition_swap")
        return {k: int(getattr(rep, k)) for k, _ in SwapReport._fields_}

    def fq_save(self, path: str) -> int:
        """Writes every stored variant to `path`; returns the bytes written."""
        n = C.c_uint64(0)
        _check(lib().fq_save(self._h, os.fsencode(path), C.byref(n)), "fq_save")
        return int(n.value)

    def fq_load(self, path: str):
        """Registers the layers of a file written by fq_save (the library allocates their device buffers)."""
        _check(lib().fq_load(self._h, os.fsencode(path)), "fq_load")

    def fq_storage_bytes(self) -> int:
        return int(lib().fq_storage_bytes(self._h))

    def fq_active_bits(self, layer: int) -> int:
        rc = lib().fq_active_bits(self._h, layer)
        if rc < 0:
            raise FlexQError(rc, "fq_active_bits")
        return rc

    def fq_status(self) -> int:
        return int(lib().fq_status(self._h))

    def fq_stream_read(self, buf: torch.Tensor):
        """One read-only pass over a device buffer (measurement support)."""
        _check(lib().fq_stream_read(self._h, buf.data_ptr(), buf.numel() * buf.element_size(), _stream()), "fq_stream_read")

    def fq_set_wait_limit_ns(self, ns: int):
        """Limit of every device-side wait of the decode kernels (0 restores the default of 2 s)."""
        _check(lib().fq_set_wait_limit_ns(self._h, int(ns)), "fq_set_wait_limit_ns")

    # -- decode --------------------------------------------------------------------------
    def fq_gemv(self, layer: int, x: torch.Tensor, y: torch.Tensor):
        _check(lib().fq_gemv(self._h, layer, x.data_ptr(), y.data_ptr(), _stream()), "fq_gemv")
        return y

    def fq_gemv_static(self, layer: int, x: torch.Tensor, y: torch.Tensor):
        """fq_gemv without any device allocation: split-K scratch lives in a fixed array inside the
        library (see include/flexq.h).  Raises FlexQError(-9) when the layer does not fit."""
        _check(lib().fq_gemv_static(self._h, layer, x.data_ptr(), y.data_ptr(), _stream()), "fq_gemv_static")
        return y

    def fq_gemv_batched(self, layer: int, x: torch.Tensor, y: torch.Tensor):
        _check(lib().fq_gemv_batched(self._h, layer, x.data_ptr(), x.shape[0], y.data_ptr(), _stream()),
               "fq_gemv_batched")
        return y

    def fq_gemv_stack(self, layers: Sequence[int], xs: Sequence[torch.Tensor], ys: Sequence[torch.Tensor],
                      phases: Optional[Sequence[int]] = None, batch: int = 1):
        n = len(layers)
        la = (C.c_int * n)(*[int(v) for v in layers])
        xa = (C.c_void_p * n)(*[t.data_ptr() for t in xs])
        ya = (C.c_void_p * n)(*[t.data_ptr() for t in ys])
        pa = (C.c_int * n)(*[int(v) for v in phases]) if phases is not None else None
        self._stack_keep = (la, xa, ya, pa)
        _check(lib().fq_gemv_stack(self._h, n, la, xa, ya, pa, batch, _stream()), "fq_gemv_stack")

    def stack_args(self, layers, xs, ys, phases=None):
        """Pre-marshalled argument arrays for repeated fq_gemv_stack_raw calls."""
        n = len(layers)
        la = (C.c_int * n)(*[int(v) for v in layers])
        xa = (C.c_void_p * n)(*[t.data_ptr() for t in xs])
        ya = (C.c_void_p * n)(*[t.data_ptr() for t in ys])
        pa = (C.c_int * n)(*[int(v) for v in phases]) if phases is not None else None
        return (n, la, xa, ya, pa)

    def fq_gemv_stack_raw(self, args, batch: int = 1):
        n, la, xa, ya, pa = args
        _check(lib().fq_gemv_stack(self._h, n, la, xa, ya, pa, batch, _stream()), "fq_gemv_stack")

    # -- prefill --------------------------------------------------------------------------
    def fq_gemm(self, layer: int, X: torch.Tensor, Y: torch.Tensor):
        assert X.dtype == torch.bfloat16 and Y.dtype == torch.bfloat16
        _check(lib().fq_gemm(self._h, layer, X.data_ptr(), X.shape[0], X.stride(0), Y.data_ptr(), Y.stride(0),
                             _stream()), "fq_gemm")
        return Y

    def fq_gemm_two_pass(self, layer: int, X: torch.Tensor, Y: torch.Tensor):
        """The comparison point of fq_gemm: dequantise to a bf16 workspace, then a plain tcgen05 GEMM."""
        assert X.dtype == torch.bfloat16 and Y.dtype == torch.bfloat16
        _check(lib().fq_gemm_two_pass(self._h, layer, X.data_ptr(), X.shape[0], X.stride(0), Y.data_ptr(), Y.stride(0),
                                      _stream()), "fq_gemm_two_pass")
        return Y

    # -- export (tests / reporting) ----------------------------------------------------------
    def fq_export_layer(self, layer: int, bits: int, n_out: int, k_in: int) -> torch.Tensor:
        out = torch.empty(n_out * k_in * bits // 32, dtype=torch.int32, device=self.device)
        _check(lib().fq_export_layer(self._h, layer, bits, out.data_ptr(), _stream()), "fq_export_layer")
        return out

    def fq_export_meta(self, layer: int, bits: int, n_out: int, k_in: int):
        s = torch.empty((n_out, k_in // 128), dtype=torch.float16, device=self.device)
        z = torch.empty((n_out, k_in // 128), dtype=torch.float16, device=self.device)
        _check(lib().fq_export_meta(self._h, layer, bits, s.data_ptr(), z.data_ptr(), _stream()), "fq_export_meta")
        return s, z
