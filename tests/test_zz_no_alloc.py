"""fq_gemv_static: the decode call for users who may not allocate device memory.

Some callers of this library run inside a fixed memory budget (a serving loop that has handed
all remaining memory to a KV cache, a plug-in living next to another allocator, a thread that
must not hit the device-wide synchronisation behind cudaMalloc).  For them fq_gemv_static keeps
its scratch -- the per-blob partial sums that two thread blocks exchange when they share a strip of
the matrix -- in an array that is part of the library image.  This test checks, through the C ABI,
that it returns exactly what fq_gemv returns (both add the blob sums in blob order, so the results
are bit-identical) and what the CPU oracle computes, twice in a row (the second call starts from the
scratch contents the first one left behind), with two contexts taking turns on the one array, and
that an oversized layer is refused.

Collected last on purpose: if it fails, `pytest -x` has already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import fq_oracle as O
from fq_testlib import GEMV_TOL, bits_of, f64_of, make_layer, to_dev, x_fp16

pytestmark = pytest.mark.gpu


def test_static_scratch_gemv_matches_fq_gemv_and_oracle_twice():
    import paper_2501_07139_b200 as P
    # ragged rows; strips of every layer are shared between thread blocks, so the scratch is in use
    specs = [(1000, 4096 + 128, 8, 8, P.FQ_FMT_PACKED), (300, 2304, 3, 3, P.FQ_FMT_PACKED),
             (520, 1536, 8, 5, P.FQ_FMT_PLANES)]
    ctxs = [P.FlexQ(len(specs)), P.FlexQ(len(specs))]          # two contexts share the built-in array
    layers = []
    for i, (nn, kk, stored, b, fmt) in enumerate(specs):
        codes, s, z = make_layer(120, i, nn, kk, stored)
        layers.append((codes, s, z))
        for fq in ctxs:
            fq.fq_pack_layer(i, *to_dev(codes, s, z), stored, fmt)
    for fq in ctxs:
        fq.fq_set_config([b for (_, _, _, b, _) in specs])
    for rep in range(2):               # two calls in a row share the same built-in array
        for i, (nn, kk, stored, b, fmt) in enumerate(specs):
            fq = ctxs[(rep + i) % 2]
            x = x_fp16(120, 10 * rep + i, 1, kk).cuda()
            y_ref = torch.empty(nn, dtype=torch.float16, device="cuda")
            y_new = torch.full((nn,), float("nan"), dtype=torch.float16, device="cuda")
            fq.fq_gemv(i, x, y_ref)
            fq.fq_gemv_static(i, x, y_new)
            torch.cuda.synchronize()
            assert fq.fq_status() == 0
            assert torch.equal(y_new, y_ref), (rep, i)
            codes, s, z = layers[i]
            if fmt == P.FQ_FMT_PLANES:
                ref = O.gemv(codes >> (8 - b), s, z, b, bits_of(x), parent_bits=8)[0]
            else:
                ref = O.gemv(codes, s, z, b, bits_of(x))[0]
            got = f64_of(y_new)
            assert np.all(np.isfinite(got))
            assert O.rel_l2(got, ref) <= GEMV_TOL, (rep, i, O.rel_l2(got, ref))
            assert np.max(np.abs(got - ref)) <= 4 * GEMV_TOL * np.max(np.abs(ref)), (rep, i)
    for fq in ctxs:
        fq.fq_destroy()


def test_static_scratch_gemv_rejects_oversized_layer():
    import paper_2501_07139_b200 as P
    n, k = 32768, 8192                 # 1024 strips x 16 blobs x 256 B = 4 MiB > the built-in 2 MiB
    fq = P.FlexQ(1)
    codes = torch.zeros((n, k), dtype=torch.uint8, device="cuda")
    s = torch.ones((n, k // 128), dtype=torch.float16, device="cuda")
    z = torch.zeros((n, k // 128), dtype=torch.float16, device="cuda")
    fq.fq_pack_layer(0, codes, s, z, 8, P.FQ_FMT_PACKED)
    x = torch.zeros(1, k, dtype=torch.float16, device="cuda")
    y = torch.empty(n, dtype=torch.float16, device="cuda")
    with pytest.raises(P.FlexQError) as e:
        fq.fq_gemv_static(0, x, y)
    assert e.value.code == -9
    fq.fq_gemv(0, x, y)                # the call that uses the context's workspace still serves it
    assert fq.fq_status() == 0
    fq.fq_destroy()
