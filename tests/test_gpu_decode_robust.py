"""Decode kernel, beyond plain parity: activations that are not finite or badly scaled, configuration
switches and stack launches issued back to back without a synchronisation, a device-side wait that is
made to run out, and the promise that the decode calls do not allocate."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import fq_oracle as O
from fq_testlib import GEMV_TOL, bits_of, f64_of, make_layer, to_dev, x_fp16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import paper_2501_07139_b200 as P
    P.lib()
    return P


def test_outlier_inside_a_group_keeps_the_tolerance(P):
    """One activation 2^10 times larger than its neighbours: the group's fixed-point scale follows the
    outlier, the small values keep an absolute error of 2^-15 of it (Sec. II-A keeps 16-bit arithmetic)."""
    n, k, b = 200, 2304, 5
    codes, s, z = make_layer(130, 0, n, k, b)
    fq = P.FlexQ(1)
    fq.fq_pack_layer(0, *to_dev(codes, s, z), b, P.FQ_FMT_PACKED)
    x = x_fp16(130, 0, 1, k)
    x[0, 700] = 1024.0
    x = x.cuda()
    y = torch.full((n,), float("nan"), dtype=torch.float16, device="cuda")
    fq.fq_gemv(0, x, y)
    assert fq.fq_status() == 0
    ref = O.gemv(codes, s, z, b, bits_of(x))[0]
    got = f64_of(y)
    assert O.rel_l2(got, ref) <= GEMV_TOL
    assert np.max(np.abs(got - ref)) <= 4 * GEMV_TOL * np.max(np.abs(ref))
    fq.fq_destroy()


@pytest.mark.parametrize("bad", [float("inf"), float("-inf"), float("nan")])
def test_non_finite_activation_is_not_swallowed(P, bad):
    """The oracle's fp64 sum is infinite or NaN in every row when an activation is; the kernel must not turn
    that into a finite number (its fixed-point conversion cannot represent the value: the group's factor
    becomes NaN and every row sum comes out NaN)."""
    n, k, b = 96, 1024, 4
    codes, s, z = make_layer(131, 0, n, k, b)
    fq = P.FlexQ(1)
    fq.fq_pack_layer(0, *to_dev(codes, s, z), b, P.FQ_FMT_PACKED)
    x = x_fp16(131, 0, 1, k)
    x[0, 300] = bad
    x = x.cuda()
    y = torch.zeros((n,), dtype=torch.float16, device="cuda")
    fq.fq_gemv(0, x, y)
    assert fq.fq_status() == 0
    ref = O.gemv(codes, s, z, b, bits_of(x))[0]
    assert not np.isfinite(ref).any()
    assert not np.isfinite(f64_of(y)).any()
    fq.fq_destroy()


def test_switches_and_stack_launches_back_to_back(P):
    """Three configuration switches, each followed by a stack launch, with no synchronisation in between:
    every launch must run with the table of its own configuration (the tables are staged through pinned
    buffers that take turns)."""
    shapes = [(256, 1024), (192, 512), (320, 1536), (256, 1024)]
    L = len(shapes)
    fq = P.FlexQ(L)
    parents = []
    for i, (n, k) in enumerate(shapes):
        q8, s, z = make_layer(132, i, n, k, 8)
        parents.append((q8, s, z))
        fq.fq_pack_layer(i, *to_dev(q8, s, z), 8, P.FQ_FMT_PLANES)
    xs = [x_fp16(132, i, 1, k).cuda() for i, (n, k) in enumerate(shapes)]
    configs = [[8, 7, 6, 5], [5, 4, 6, 3], [2, 3, 4, 2]]
    outs = []
    for cfg in configs:
        ys = [torch.full((n,), float("nan"), dtype=torch.float16, device="cuda") for n, k in shapes]
        fq.fq_set_config(cfg)
        fq.fq_gemv_stack(list(range(L)), xs, ys, [0, 0, 1, 2], 1)      # no synchronisation before the next switch
        outs.append(ys)
    assert fq.fq_status() == 0
    for cfg, ys in zip(configs, outs):
        fq.fq_set_config(cfg)
        for i, (n, k) in enumerate(shapes):
            y1 = torch.empty((n,), dtype=torch.float16, device="cuda")
            fq.fq_gemv(i, xs[i], y1)
            torch.cuda.synchronize()
            assert torch.equal(ys[i], y1), (cfg, i)
            q8, s, z = parents[i]
            ref = O.gemv(q8 >> (8 - cfg[i]), s, z, cfg[i], bits_of(xs[i]), parent_bits=8)[0]
            assert O.rel_l2(f64_of(ys[i]), ref) <= GEMV_TOL, (cfg, i)
    fq.fq_destroy()


def test_a_wait_that_runs_out_is_reported_and_leaves_the_context_usable(P):
    """With a limit of one nanosecond the first wait of the launch that is not satisfied at once gives up: the
    kernel records the time-out, every role leaves its loop, the producer waits for its copies in flight and
    the launch returns.  fq_status reports the code and cleans up; the next launch is correct again."""
    shapes = [(256, 512), (256, 512), (96, 512), (512, 256), (130, 512), (256, 1280)]
    bits = [3, 8, 5, 4, 6, 2]
    fq = P.FlexQ(len(shapes))
    for i, ((n, k), b) in enumerate(zip(shapes, bits)):
        fq.fq_pack_layer(i, *to_dev(*make_layer(99, i, n, k, b)), b, P.FQ_FMT_PACKED)
    xs = [x_fp16(99, i, 1, k).cuda() for i, (n, k) in enumerate(shapes)]
    want = [torch.empty((n,), dtype=torch.float16, device="cuda") for n, k in shapes]
    for i in range(len(shapes)):
        fq.fq_gemv(i, xs[i], want[i])
    assert fq.fq_status() == 0
    ys = [torch.zeros((n,), dtype=torch.float16, device="cuda") for n, k in shapes]
    fq.fq_set_wait_limit_ns(1)
    fq.fq_gemv_stack(list(range(len(shapes))), xs, ys, [0, 0, 0, 1, 2, 3], 1)
    assert fq.fq_status() == -8                       # FQ_ERR_TIMEOUT, and the launch has returned
    assert P.fq_strerror(-8) == "device-side wait timed out"
    assert fq.fq_status() == 0                        # reported once, counters reset
    fq.fq_set_wait_limit_ns(0)                        # back to the default
    for rep in range(2):
        fq.fq_gemv_stack(list(range(len(shapes))), xs, ys, [0, 0, 0, 1, 2, 3], 1)
    assert fq.fq_status() == 0
    for i in range(len(shapes)):
        assert torch.equal(ys[i], want[i]), i
    fq.fq_destroy()


def test_decode_calls_do_not_allocate(P):
    """After the layers are packed, the first fq_gemv, fq_gemv_batched(8) and fq_gemv_stack calls leave the
    amount of free device memory unchanged (the split-K scratch was reserved at pack time; the op table of a
    stack call goes to a buffer that only grows when a longer list is seen)."""
    shapes = [(1024, 2048), (512, 4096), (2048, 1024)]
    bits = [4, 8, 3]
    fq = P.FlexQ(len(shapes))
    for i, ((n, k), b) in enumerate(zip(shapes, bits)):
        fq.fq_pack_layer(i, *to_dev(*make_layer(133, i, n, k, b)), b, P.FQ_FMT_PACKED)
    xs1 = [x_fp16(133, i, 1, k).cuda() for i, (n, k) in enumerate(shapes)]
    xs8 = [x_fp16(133, 10 + i, 8, k).cuda() for i, (n, k) in enumerate(shapes)]
    ys1 = [torch.empty((1, n), dtype=torch.float16, device="cuda") for n, k in shapes]
    ys8 = [torch.empty((8, n), dtype=torch.float16, device="cuda") for n, k in shapes]
    # one stack call first: it creates the (small) table buffers that later calls reuse
    fq.fq_gemv_stack(list(range(len(shapes))), xs1, ys1, [0, 1, 2], 1)
    fq.fq_gemv_stack(list(range(len(shapes))), xs8, ys8, [0, 1, 2], 8)
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for i in range(len(shapes)):
        fq.fq_gemv(i, xs1[i], ys1[i])
        fq.fq_gemv_batched(i, xs8[i], ys8[i])
    fq.fq_gemv_stack(list(range(len(shapes))), xs1, ys1, [0, 0, 1], 1)      # another op table of the same size
    fq.fq_gemv_stack(list(range(len(shapes))), xs8, ys8, None, 8)
    torch.cuda.synchronize()
    assert fq.fq_status() == 0
    assert torch.cuda.mem_get_info()[0] == free0
    fq.fq_destroy()


@pytest.mark.parametrize("fmt_bits", [(0, 4), (1, 5)])
def test_layer_wider_than_the_batch1_kernel_holds(P, fmt_bits):
    """k_in = 16384 is more than the batch-1 kernel keeps in shared memory (14336): fq_gemv and a batch-1
    fq_gemv_stack then run in the batch kernel; fq_gemv_static, which has no other kernel, refuses."""
    fmt, bits = fmt_bits
    n, k = 96, 16384
    stored = 8 if fmt == 1 else bits
    codes, s, z = make_layer(160, bits, n, k, stored)
    fq = P.FlexQ(2)
    fq.fq_pack_layer(0, *to_dev(codes, s, z), stored, fmt)
    small = make_layer(160, 9, 64, 512, 4)
    fq.fq_pack_layer(1, *to_dev(*small), 4, P.FQ_FMT_PACKED)
    fq.fq_set_config([bits, 4])
    x = x_fp16(160, bits, 1, k).cuda()[0]
    y = torch.full((n,), float("nan"), dtype=torch.float16, device="cuda")
    fq.fq_gemv(0, x, y)
    assert fq.fq_status() == 0
    ref = (O.gemv(codes >> (8 - bits), s, z, bits, bits_of(x[None]), parent_bits=8) if fmt == 1
           else O.gemv(codes, s, z, bits, bits_of(x[None])))[0]
    got = f64_of(y)
    assert np.all(np.isfinite(got)) and O.rel_l2(got, ref) <= GEMV_TOL
    assert np.max(np.abs(got - ref)) <= 4 * GEMV_TOL * np.max(np.abs(ref))
    # the same layer inside a dependency-ordered batch-1 stack next to a narrow one
    x1 = x_fp16(160, 7, 1, 512).cuda()[0]
    ys = [torch.full((n,), float("nan"), dtype=torch.float16, device="cuda"),
          torch.full((64,), float("nan"), dtype=torch.float16, device="cuda")]
    fq.fq_gemv_stack([0, 1], [x, x1], ys, [0, 1], 1)
    assert fq.fq_status() == 0
    assert O.rel_l2(f64_of(ys[0]), ref) <= GEMV_TOL
    ref1 = O.gemv(*small, 4, bits_of(x1[None]))[0]
    assert O.rel_l2(f64_of(ys[1]), ref1) <= GEMV_TOL
    with pytest.raises(P.FlexQError) as e:
        fq.fq_gemv_static(0, x, y)
    assert e.value.code == -3
    fq.fq_destroy()
