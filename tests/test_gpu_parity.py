"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import fq_synth as S
from oracle import fq_oracle as O
from fq_testlib import (GEMV_TOL, bits_of, f64_of, make_layer, to_dev, x_fp16)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import paper_2501_07139_b200 as P
    P.lib()
    return P


# ----------------------------------------------------------------------------- quantiser
@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8])
def test_quantizer_bit_exact(P, bits):
    n, k = 150, 1152
    w = S.weight_rows(S.tensor_key(90, bits, S.TENSOR_W), 0, n, k)
    w[3, 128:256] = 0.0125                 # constant group
    w[4, :128] = 0.0                       # all-zero group
    w[5, 0] = 3.0                          # outlier
    rc, rs, rz = O.quantize(w.numpy(), bits)
    c, s, z = P.fq_quantize_layer(w.cuda(), bits)
    torch.cuda.synchronize()
    assert np.array_equal(c.cpu().numpy(), rc)
    assert np.array_equal(bits_of(s), rs)
    assert np.array_equal(bits_of(z), rz)


# ----------------------------------------------------------------------------- packing / export / footprint
@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("shape", [(16, 128), (40, 384), (129, 1024)])
def test_pack_export_packed_bit_exact(P, bits, shape):
    n, k = shape
    codes, s, z = make_layer(91, bits, n, k, bits)
    fq = P.FlexQ(1)
    fq.fq_pack_layer(0, *to_dev(codes, s, z), bits, P.FQ_FMT_PACKED)
    out = fq.fq_export_layer(0, bits, n, k).cpu().numpy().view(np.uint32).reshape(n, -1)
    assert np.array_equal(out, O.pack_bitstream(codes, bits))
    es, ez = fq.fq_export_meta(0, bits, n, k)
    assert np.array_equal(bits_of(es), s) and np.array_equal(bits_of(ez), z)
    assert fq.fq_set_config([bits]) == O.footprint([n], [k], [bits])
    fq.fq_destroy()


@pytest.mark.parametrize("shape", [(16, 128), (40, 384), (129, 1024)])
def test_pack_export_planes_bit_exact_and_nested(P, shape):
    n, k = shape
    q8, s, z = make_layer(92, 0, n, k, 8)
    fq = P.FlexQ(1)
    code_buf = fq.fq_pack_layer(0, *to_dev(q8, s, z), 8, P.FQ_FMT_PLANES)
    before = code_buf.clone()
    ref = O.pack_planes(q8)
    for b in range(2, 9):
        assert fq.fq_set_config([b]) == O.footprint([n], [k], [b])
        out = fq.fq_export_layer(0, b, n, k).cpu().numpy().view(np.uint32).reshape(b, n, k // 32)
        assert np.array_equal(out, ref[:b])
        assert np.array_equal(O.child_codes(out, k, b), q8 >> (8 - b))
    assert torch.equal(before, code_buf)            # switching configurations moved no weight byte
    assert fq.fq_storage_bytes() == O.footprint([n], [k], [8])
    fq.fq_destroy()


def test_packed_multi_variant_config_and_errors(P):
    n, k = 32, 256
    fq = P.FlexQ(2)
    variants = {}
    for b in (3, 8):
        variants[b] = make_layer(93, 0, n, k, b)
        fq.fq_pack_layer(0, *to_dev(*variants[b]), b, P.FQ_FMT_PACKED)
    v1 = make_layer(93, 1, n, k, 4)
    fq.fq_pack_layer(1, *to_dev(*v1), 4, P.FQ_FMT_PACKED)
    assert fq.fq_active_bits(0) == 3
    assert fq.fq_set_config([8, 4]) == O.footprint([n, n], [k, k], [8, 4])
    assert fq.fq_storage_bytes() == O.footprint([n, n, n], [k, k, k], [3, 8, 4])
    with pytest.raises(P.FlexQError) as e:
        fq.fq_set_config([5, 4])
    assert e.value.code == -5 and fq.fq_active_bits(0) == 8      # unchanged after the failed call
    with pytest.raises(P.FlexQError) as e:
        fq.fq_set_config([9, 4])
    assert e.value.code == -2
    with pytest.raises(P.FlexQError) as e:
        fq.fq_set_config([8])
    assert e.value.code == -1
    x = x_fp16(93, 0, 1, k).cuda()
    y = torch.empty(n, dtype=torch.float16, device="cuda")
    fq.fq_gemv(0, x, y)
    ref = O.gemv(*variants[8], 8, bits_of(x))[0]
    assert O.rel_l2(f64_of(y), ref) <= GEMV_TOL
    fq.fq_destroy()


# ----------------------------------------------------------------------------- GEMV
def _gemv_case(P, fmt, bits, n, k, batch, cfg):
    stored = 8 if fmt == P.FQ_FMT_PLANES else bits
    codes, s, z = make_layer(cfg, bits, n, k, stored)
    fq = P.FlexQ(1)
    fq.fq_pack_layer(0, *to_dev(codes, s, z), stored, fmt)
    fq.fq_set_config([bits])
    x = x_fp16(cfg, bits, batch, k).cuda()
    y = torch.full((batch, n), float("nan"), dtype=torch.float16, device="cuda")
    if batch == 1:
        fq.fq_gemv(0, x, y)
    else:
        fq.fq_gemv_batched(0, x, y)
    assert fq.fq_status() == 0
    if fmt == P.FQ_FMT_PLANES:
        ref = O.gemv(codes >> (8 - bits), s, z, bits, bits_of(x), parent_bits=8)
    else:
        ref = O.gemv(codes, s, z, bits, bits_of(x))
    got = f64_of(y)
    assert np.all(np.isfinite(got))
    for b in range(batch):
        assert O.rel_l2(got[b], ref[b]) <= GEMV_TOL, (bits, b, O.rel_l2(got[b], ref[b]))
        # element by element too: a norm alone would hide one bad row among a thousand
        assert np.max(np.abs(got[b] - ref[b])) <= 4 * GEMV_TOL * np.max(np.abs(ref[b])), (bits, b)
    fq.fq_destroy()
    return codes, s, z


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("shape", [(16, 128), (200, 2304), (1000, 4096 + 128)])
def test_gemv_packed_parity(P, bits, shape):
    _gemv_case(P, P.FQ_FMT_PACKED, bits, shape[0], shape[1], 1, 94)


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("shape", [(16, 128), (200, 2304)])
def test_gemv_planes_parity(P, bits, shape):
    _gemv_case(P, P.FQ_FMT_PLANES, bits, shape[0], shape[1], 1, 95)


@pytest.mark.parametrize("batch", [2, 5, 8])
@pytest.mark.parametrize("fmt_bits", [(0, 4), (0, 3), (0, 8), (1, 5), (1, 2)])
def test_gemv_batched_parity(P, batch, fmt_bits):
    fmt, bits = fmt_bits
    _gemv_case(P, fmt, bits, 200, 1280, batch, 96)


@pytest.mark.parametrize("fmt_bits", [(0, 2), (0, 3), (0, 4), (0, 7), (0, 8), (1, 3), (1, 8)])
def test_gemv_one_hot_is_bit_exact(P, fmt_bits):
    """x = e_k recovers column k of the dequantised matrix through the real kernel, bit for bit."""
    fmt, bits = fmt_bits
    n, k = 48, 512
    stored = 8 if fmt == 1 else bits
    codes, s, z = make_layer(97, bits, n, k, stored)
    fq = P.FlexQ(1)
    fq.fq_pack_layer(0, *to_dev(codes, s, z), stored, fmt)
    fq.fq_set_config([bits])
    child = codes >> (8 - bits) if fmt == 1 else codes
    w_hat = O.dequant(child, s, z, bits, 8 if fmt == 1 else None)
    y = torch.empty(n, dtype=torch.float16, device="cuda")
    for kk in (0, 1, 7, 8, 31, 32, 127, 128, 255, 256, 300, 511):
        x = torch.zeros(1, k, dtype=torch.float16)
        x[0, kk] = 1.0
        fq.fq_gemv(0, x.cuda(), y)
        assert np.array_equal(f64_of(y), w_hat[:, kk]), kk
    fq.fq_destroy()


def test_gemv_exact_integer_row_sums_and_zero_codes(P):
    rng = np.random.default_rng(12)
    n, k = 64, 1024
    codes = rng.integers(0, 256, size=(n, k), dtype=np.uint8)
    s = np.full((n, k // 128), 0x3C00, np.uint16)
    z = np.zeros((n, k // 128), np.uint16)
    fq = P.FlexQ(1)
    fq.fq_pack_layer(0, *to_dev(codes, s, z), 8, P.FQ_FMT_PACKED)
    x = torch.full((1, k), 2.0 ** -8, dtype=torch.float16).cuda()
    y = torch.empty(n, dtype=torch.float16, device="cuda")
    fq.fq_gemv(0, x, y)
    exact = codes.astype(np.int64).sum(1) / 256.0
    assert np.array_equal(f64_of(y), exact.astype(np.float16).astype(np.float64))
    fq.fq_destroy()
    # every code equal to its zero point -> y == 0
    codes2, s2, z2 = make_layer(98, 0, n, k, 6)
    zc = np.repeat(z2.view(np.float16).astype(np.uint8), 128, axis=1)
    fq = P.FlexQ(1)
    fq.fq_pack_layer(0, *to_dev(zc, s2, z2), 6, P.FQ_FMT_PACKED)
    xr = x_fp16(98, 0, 1, k).cuda()
    fq.fq_gemv(0, xr, y)
    assert float(y.float().abs().max()) <= 2e-3 * float(np.abs(O.gemv(codes2, s2, z2, 6, bits_of(xr))).max())
    fq.fq_destroy()


def test_config0_single_layer_4bit(P):
    """4096 x 4096, 4-bit, group 128: footprint 8 912 896 bytes and GEMV parity."""
    n = k = 4096
    codes, s, z = make_layer(0, 0, n, k, 4)
    fq = P.FlexQ(1)
    fq.fq_pack_layer(0, *to_dev(codes, s, z), 4, P.FQ_FMT_PACKED)
    assert fq.fq_set_config([4]) == 8_912_896
    x = x_fp16(0, 0, 1, k).cuda()
    y = torch.empty(n, dtype=torch.float16, device="cuda")
    fq.fq_gemv(0, x, y)
    rows = S.sample_rows(1, n, 64)
    ref = O.gemv(codes[rows], s[rows], z[rows], 4, bits_of(x))[0]
    assert O.rel_l2(f64_of(y)[rows], ref) <= GEMV_TOL
    out = fq.fq_export_layer(0, 4, n, k).cpu().numpy().view(np.uint32).reshape(n, -1)
    assert np.array_equal(out[rows], O.pack_bitstream(codes[rows], 4))
    fq.fq_destroy()


# ----------------------------------------------------------------------------- stack
@pytest.mark.parametrize("batch", [1, 4])
def test_gemv_stack_matches_per_layer_calls(P, batch):
    shapes = [(256, 512), (256, 512), (96, 512), (512, 256), (130, 512), (256, 1280)]
    bits = [3, 8, 5, 4, 6, 2]
    phases = [0, 0, 0, 1, 2, 3]
    fq = P.FlexQ(len(shapes))
    layers = []
    for i, ((n, k), b) in enumerate(zip(shapes, bits)):
        c, s, z = make_layer(99, i, n, k, b)
        fq.fq_pack_layer(i, *to_dev(c, s, z), b, P.FQ_FMT_PACKED)
        layers.append((c, s, z))
    xs = [x_fp16(99, i, batch, k).cuda() for i, (n, k) in enumerate(shapes)]
    y_single = [torch.empty((batch, n), dtype=torch.float16, device="cuda") for n, k in shapes]
    for i in range(len(shapes)):
        fq.fq_gemv_batched(i, xs[i], y_single[i])
    for ph in (None, phases):
        ys = [torch.full((batch, n), float("nan"), dtype=torch.float16, device="cuda") for n, k in shapes]
        for rep in range(3):                     # repeated launches reuse self-resetting counters
            fq.fq_gemv_stack(list(range(len(shapes))), xs, ys, ph, batch)
        assert fq.fq_status() == 0
        for i in range(len(shapes)):
            assert torch.equal(ys[i], y_single[i]), (ph, i)
    ref = O.gemv(*layers[3], bits[3], bits_of(xs[3]))
    assert O.rel_l2(f64_of(y_single[3]), ref) <= GEMV_TOL
    fq.fq_destroy()


def test_gemv_argument_errors(P):
    fq = P.FlexQ(2)
    x = torch.zeros(1, 256, dtype=torch.float16, device="cuda")
    y = torch.zeros(32, dtype=torch.float16, device="cuda")
    with pytest.raises(P.FlexQError) as e:
        fq.fq_gemv(0, x, y)
    assert e.value.code == -6
    c, s, z = make_layer(100, 0, 32, 256, 4)
    fq.fq_pack_layer(0, *to_dev(c, s, z), 4)
    with pytest.raises(P.FlexQError) as e:
        fq.fq_gemv(0, x.view(-1)[1:].view(1, -1), y)      # misaligned x
    assert e.value.code == -4
    with pytest.raises(P.FlexQError) as e:
        fq.fq_gemv(5, x, y)
    assert e.value.code == -1
    with pytest.raises(P.FlexQError) as e:
        fq.fq_pack_layer(1, torch.zeros((4, 100), dtype=torch.uint8, device="cuda"),
                         torch.zeros((4, 1), dtype=torch.float16, device="cuda"),
                         torch.zeros((4, 1), dtype=torch.float16, device="cuda"), 4)
    assert e.value.code == -3
    fq.fq_destroy()


def test_stack_after_single_calls_with_split_k(P):
    """Split-K arrival counters and partial sums must never share workspace bytes: a per-layer call
    followed by a stack call over wide layers (several K chunks) once left rows unwritten."""
    n, k = 1024, 4096
    fq = P.FlexQ(2)
    layers = [make_layer(101, i, n, k, 3) for i in range(2)]
    for i, l in enumerate(layers):
        fq.fq_pack_layer(i, *to_dev(*l), 3, P.FQ_FMT_PACKED)
    xs = [x_fp16(101, i, 1, k).cuda() for i in range(2)]
    y_single = [torch.empty((1, n), dtype=torch.float16, device="cuda") for _ in range(2)]
    for rep in range(2):
        for i in range(2):
            fq.fq_gemv_batched(i, xs[i], y_single[i])
        ys = [torch.full((1, n), float("nan"), dtype=torch.float16, device="cuda") for _ in range(2)]
        fq.fq_gemv_stack([0, 1], xs, ys, None, 1)
        assert fq.fq_status() == 0
        for i in range(2):
            assert torch.equal(ys[i], y_single[i])
    ref = O.gemv(*layers[1], 3, bits_of(xs[1]))
    assert O.rel_l2(f64_of(y_single[1]), ref) <= GEMV_TOL
    fq.fq_destroy()


def test_gemv_stack_phases_carry_real_data_dependencies(P):
    """A chain in which every op reads what the previous phase wrote (x of op i+1 IS y of op i): the values
    must equal those of separate calls in sequence, launch after launch.  A phase that started before the
    previous one had published all of its outputs would read stale or poisoned activations."""
    dims = [1024, 2048, 1024, 4096, 1024]                      # k_in of op 0, then n_out of every op
    bits = [8, 4, 3, 5]
    L = len(bits)
    fq = P.FlexQ(L)
    for i in range(L):
        fq.fq_pack_layer(i, *to_dev(*make_layer(101, i, dims[i + 1], dims[i], bits[i])), bits[i], P.FQ_FMT_PACKED)
    x0 = (x_fp16(101, 0, 1, dims[0]) * 4).cuda()
    # reference: one call after the other; scale so that the chain neither dies out nor overflows
    seq = [x0[0]]
    for i in range(L):
        y = torch.empty(dims[i + 1], dtype=torch.float16, device="cuda")
        fq.fq_gemv(i, seq[-1], y)
        seq.append(y)
    torch.cuda.synchronize()
    assert all(torch.isfinite(t).all() and t.abs().max() > 0 for t in seq)
    bufs = [x0[0].clone()] + [torch.empty(dims[i + 1], dtype=torch.float16, device="cuda") for i in range(L)]
    for rep in range(25):
        for t in bufs[1:]:
            t.fill_(float("nan"))                              # poison: an early reader would see NaN
        fq.fq_gemv_stack(list(range(L)), bufs[:-1], bufs[1:], list(range(L)), 1)
        torch.cuda.synchronize()
        for i in range(L):
            assert torch.equal(bufs[i + 1], seq[i + 1]), (rep, i)
    assert fq.fq_status() == 0
    fq.fq_destroy()
