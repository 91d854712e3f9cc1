"""GPU parity of the prefill path against the fp64 CPU oracle: the fused kernel behind fq_gemm (blobs
dequantised inside the tcgen05 GEMM) and its two-pass comparison point fq_gemm_two_pass."""
import numpy as np
import pytest
import torch

import fq_synth as S
from oracle import fq_oracle as O
from fq_testlib import GEMM_TOL, bits_of, f64_of, make_layer, to_dev, x_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import paper_2501_07139_b200 as P
    P.lib()
    return P


@pytest.fixture(params=["fused", "two_pass"])
def which(request):
    return request.param


def _gemm(fq, which, layer, x, y):
    return fq.fq_gemm(layer, x, y) if which == "fused" else fq.fq_gemm_two_pass(layer, x, y)


def _ref(codes, s, z, bits, fmt, x):
    if fmt == 1:
        return O.gemm(codes >> (8 - bits), s, z, bits, bits_of(x), parent_bits=8)
    return O.gemm(codes, s, z, bits, bits_of(x))


@pytest.mark.parametrize("fmt_bits", [(0, 2), (0, 3), (0, 4), (0, 5), (0, 6), (0, 7), (0, 8), (1, 3), (1, 6), (1, 8)])
def test_gemm_small_every_element(P, which, fmt_bits):
    fmt, bits = fmt_bits
    n, k, m = 300, 384, 200                      # ragged against the 128 x 256 x 64 tiles
    stored = 8 if fmt == 1 else bits
    codes, s, z = make_layer(110, bits, n, k, stored)
    fq = P.FlexQ(1)
    fq.fq_pack_layer(0, *to_dev(codes, s, z), stored, fmt)
    fq.fq_set_config([bits])
    x = x_bf16(110, bits, m, k).cuda()
    y = torch.full((m, n + 4), float("nan"), dtype=torch.bfloat16, device="cuda")[:, :]   # ldy = n + 4 (multiple of 8)
    _gemm(fq, which, 0, x, y)
    assert fq.fq_status() == 0
    got = f64_of(y)[:, :n]
    ref = _ref(codes, s, z, bits, fmt, x)
    assert np.all(np.isfinite(got))
    err = O.rel_l2(got, ref)
    assert err <= GEMM_TOL, (fmt, bits, err)
    # element by element too (bf16 rounding of X-dot-w^ alone is 2^-9 of the value; sums are ~sqrt(k) larger than terms)
    assert np.max(np.abs(got - ref)) <= 4 * GEMM_TOL * np.max(np.abs(ref)), (fmt, bits)
    assert torch.isnan(y[:, n:].float()).all()   # columns beyond n_out are not written
    fq.fq_destroy()


@pytest.mark.parametrize("m", [1, 127, 129, 600])
def test_gemm_token_counts(P, which, m):
    n, k = 512, 1024
    codes, s, z = make_layer(111, 0, n, k, 4)
    fq = P.FlexQ(1)
    fq.fq_pack_layer(0, *to_dev(codes, s, z), 4, P.FQ_FMT_PACKED)
    x = x_bf16(111, m, m, k).cuda()
    y = torch.empty((m, n), dtype=torch.bfloat16, device="cuda")
    _gemm(fq, which, 0, x, y)
    assert fq.fq_status() == 0
    rows = sorted(set([0, m - 1, m // 2, min(m - 1, 127), min(m - 1, 128)]))
    ref = O.gemm(codes, s, z, 4, bits_of(x[rows]))
    assert O.rel_l2(f64_of(y)[rows], ref) <= GEMM_TOL
    fq.fq_destroy()


@pytest.mark.parametrize("bits", [3, 4])
def test_gemm_more_tiles_than_sms(P, which, bits):
    """9 x 17 = 153 output tiles of 256 x 256 on 148 SMs: the fused kernel cuts the (tile, K stage) sequence into equal
    runs, so tiles are shared between two CTAs (partial sums through the workspace); sampled rows against the oracle,
    and the two kernels against each other (a shared tile adds two fp32 partial sums, so the last bf16 bit may differ)."""
    n, k, m = 17 * 256 - 40, 640, 9 * 256 - 3
    codes, s, z = make_layer(115, bits, n, k, bits)
    fq = P.FlexQ(1)
    fq.fq_pack_layer(0, *to_dev(codes, s, z), bits, P.FQ_FMT_PACKED)
    x = x_bf16(115, bits, m, k).cuda()
    y = torch.full((m, n), float("nan"), dtype=torch.bfloat16, device="cuda")
    for _ in range(2):                                   # twice: the partial-sum flags of the first launch are stale in the second
        _gemm(fq, which, 0, x, y)
    assert fq.fq_status() == 0
    other = torch.empty_like(y)
    _gemm(fq, "two_pass" if which == "fused" else "fused", 0, x, other)
    a, b = y.float(), other.float()
    assert bool(((a - b).abs() <= 2.0 ** -7 * b.abs() + 1e-3).all())
    assert float((a != b).float().mean()) < 0.02
    rows = [int(r) for r in S.sample_rows(115, m, 40)]
    ref = O.gemm(codes, s, z, bits, bits_of(x[rows]))
    got = f64_of(y)[rows]
    assert np.all(np.isfinite(f64_of(y)))
    assert O.rel_l2(got, ref) <= GEMM_TOL
    assert np.max(np.abs(got - ref)) <= 4 * GEMM_TOL * np.max(np.abs(ref))
    fq.fq_destroy()


def test_gemm_identity_probe_recovers_weights(P, which):
    """X = identity rows: Y[m][n] = bf16(w^[n][m]); checks operand orientation and every k position."""
    n, k = 256, 256
    codes, s, z = make_layer(112, 0, n, k, 8)
    fq = P.FlexQ(1)
    fq.fq_pack_layer(0, *to_dev(codes, s, z), 8, P.FQ_FMT_PACKED)
    x = torch.eye(k, dtype=torch.bfloat16, device="cuda")
    y = torch.empty((k, n), dtype=torch.bfloat16, device="cuda")
    _gemm(fq, which, 0, x, y)
    S_ = np.repeat(s.view(np.float16).astype(np.float64), 128, axis=1)
    Z_ = np.repeat(z.view(np.float16).astype(np.float64), 128, axis=1)
    exact = (codes.astype(np.float64) - Z_) * S_                       # [n][k], exact products
    want = torch.from_numpy(exact.T.copy()).to(torch.bfloat16).double().numpy()   # one rounding to bf16
    assert np.array_equal(f64_of(y), want)
    fq.fq_destroy()


def test_gemm_7b_block_at_prefill_size_sampled(P, which):
    """First block of the 7B-shaped stack at M = 4 x 2048 tokens, bits from {2,3,4,6,8}: sampled outputs."""
    shapes = S.stack_shapes("7b", 1)
    bits = S.draw_bits(S.tensor_key(3, 0, S.TENSOR_BITS), len(shapes), [2, 3, 4, 6, 8])
    m = 8192
    fq = P.FlexQ(len(shapes))
    xs = {}
    for i, sh in enumerate(shapes):
        w = S.weight_rows(S.tensor_key(3, i, S.TENSOR_W), 0, sh.n_out, sh.k_in, device="cuda")
        c, s, z = P.fq_quantize_layer(w, int(bits[i]))
        fq.fq_pack_layer(i, c, s, z, int(bits[i]), P.FQ_FMT_PACKED)
        if sh.k_in not in xs:
            xs[sh.k_in] = S.activations(S.tensor_key(3, sh.k_in, S.TENSOR_X), m, sh.k_in, torch.bfloat16, device="cuda")
        del w, c, s, z
    rng = np.random.default_rng(33)
    for i, sh in enumerate(shapes):
        x = xs[sh.k_in]
        y = torch.empty((m, sh.n_out), dtype=torch.bfloat16, device="cuda")
        _gemm(fq, which, i, x, y)
        assert fq.fq_status() == 0
        trows = sorted(set([0, 127, 128, m - 1] + rng.integers(0, m, 12).tolist()))
        nrows = S.sample_rows(2000 + i, sh.n_out, 40)
        w = np.concatenate([S.weight_rows(S.tensor_key(3, i, S.TENSOR_W), int(r), int(r) + 1, sh.k_in).numpy() for r in nrows])
        c, s, z = O.quantize(w, int(bits[i]))
        ref = O.gemm(c, s, z, int(bits[i]), bits_of(x[trows]))
        got = f64_of(y[trows][:, torch.from_numpy(nrows).cuda()])
        err = O.rel_l2(got, ref)
        assert err <= GEMM_TOL, (sh.name, int(bits[i]), err)
        del y
    fq.fq_destroy()


def test_gemm_argument_errors(P):
    fq = P.FlexQ(1)
    c, s, z = make_layer(113, 0, 64, 256, 4)
    fq.fq_pack_layer(0, *to_dev(c, s, z), 4)
    x = torch.zeros((8, 256), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    import ctypes as C
    L = P.lib()
    st = torch.cuda.current_stream().cuda_stream
    assert L.fq_gemm(fq._h, 0, x.data_ptr(), 8, 250, y.data_ptr(), 64, st) == -3      # ldx < k_in
    assert L.fq_gemm(fq._h, 0, x.data_ptr(), 0, 256, y.data_ptr(), 64, st) == -3      # M < 1
    assert L.fq_gemm(fq._h, 0, x.data_ptr() + 2, 8, 256, y.data_ptr(), 64, st) == -4  # misaligned X
    assert L.fq_gemm(fq._h, 3, x.data_ptr(), 8, 256, y.data_ptr(), 64, st) == -1
    fq.fq_gemm(0, x, y)
    assert fq.fq_status() == 0 and float(y.float().abs().max()) == 0.0
    fq.fq_destroy()
