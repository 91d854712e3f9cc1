"""fq_gemv_static: the decode call for users who may not allocate device memory.

Some callers of this library run inside a fixed memory budget (a serving loop that has handed
all remaining memory to a KV cache, a plug-in living next to another allocator, a thread that
must not hit the device-wide synchronisation behind cudaMalloc).  For them fq_gemv_static keeps
its split-K scratch in an array that is part of the library image.  This test checks, through
the C ABI, that it returns what fq_gemv returns, twice in a row (the second call starts from the
scratch contents the first one left behind), and that an oversized layer is refused.

Collected last on purpose: if it fails, `pytest -x` has already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import fq_oracle as O
from fq_testlib import GEMV_TOL, f64_of, make_layer, to_dev, x_fp16

pytestmark = pytest.mark.gpu


def test_static_scratch_gemv_matches_fq_gemv_twice():
    import paper_2501_07139_b200 as P
    n, k = 1000, 4096 + 128            # ragged rows; 8-bit codes split K into several chunks
    fq = P.FlexQ(2)
    shapes_bits = [(n, k, 8), (300, 2304, 3)]
    for i, (nn, kk, b) in enumerate(shapes_bits):
        fq.fq_pack_layer(i, *to_dev(*make_layer(120, i, nn, kk, b)), b, P.FQ_FMT_PACKED)
    for rep in range(2):               # two calls in a row share the same built-in array
        for i, (nn, kk, b) in enumerate(shapes_bits):
            x = x_fp16(120, 10 * rep + i, 1, kk).cuda()
            y_ref = torch.empty(nn, dtype=torch.float16, device="cuda")
            y_new = torch.full((nn,), float("nan"), dtype=torch.float16, device="cuda")
            fq.fq_gemv(i, x, y_ref)
            fq.fq_gemv_static(i, x, y_new)
            torch.cuda.synchronize()
            assert fq.fq_status() == 0
            got, ref = f64_of(y_new), f64_of(y_ref)
            assert np.all(np.isfinite(got))
            assert O.rel_l2(got, ref) <= GEMV_TOL, (rep, i, O.rel_l2(got, ref))
    fq.fq_destroy()


def test_static_scratch_gemv_rejects_oversized_layer():
    import paper_2501_07139_b200 as P
    n, k = 32768, 8192                 # 1024 row pairs x 16 chunks x 256 B = 4 MiB > the built-in 2 MiB
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
    fq.fq_gemv(0, x, y)                # the allocating call still serves it
    assert fq.fq_status() == 0
    fq.fq_destroy()
