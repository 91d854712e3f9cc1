"""Pins for the CPU oracle: each oracle function is checked against something that is
not the oracle -- numpy's float16 / packbits / matmul, closed forms, hand-worked groups,
exhaustive enumeration, and the accounting figures the paper prints."""
import os

import numpy as np
import pytest

from oracle import fq_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split("=")
                out[k.strip()] = v.strip()
    return out


# --------------------------------------------------------------------------- fp16 / bf16

def test_f16_to_f64_all_patterns_match_numpy():
    h = np.arange(65536, dtype=np.uint16)
    ref = h.view(np.float16).astype(np.float64)
    got = np.array([O.f16_to_f64(int(v)) for v in h])
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], ref[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(ref[~nan]))


def test_f64_to_f16_values_midpoints_and_edges_match_numpy():
    h = np.arange(0x7C00, dtype=np.uint16)                     # all finite non-negative halves
    v = h.view(np.float16).astype(np.float64)
    cases = [v, -v]
    mid = (v[:-1] + v[1:]) / 2                                   # exact ties between neighbours
    cases += [mid, -mid, np.nextafter(mid, np.inf), np.nextafter(mid, -np.inf)]
    cases.append(np.array([65504.0, 65519.99, 65520.0, 65520.01, 1e9, -1e9, np.inf, -np.inf,
                           2.0 ** -24, 2.0 ** -25, np.nextafter(2.0 ** -25, 1), 2.0 ** -26,
                           1e-300, 5e-324, 0.0, -0.0, 1 / 3, 0.1, 1e-5, 6.1e-5]))
    rng = np.random.default_rng(1)
    cases.append(rng.standard_normal(20000) * np.exp(rng.uniform(-12, 12, 20000)))
    allv = np.concatenate(cases)
    with np.errstate(over="ignore"):
        ref = allv.astype(np.float16).view(np.uint16)
    got = np.array([O.f64_to_f16(float(x)) for x in allv], dtype=np.uint16)
    assert np.array_equal(got, ref)


def test_f64_to_f16_is_single_rounding_not_via_float32():
    # 1 + 2^-11 + 2^-30 lies just above a tie: direct rounding goes up, rounding through
    # float32 first would land on the tie and go down (to even).
    v = 1.0 + 2.0 ** -11 + 2.0 ** -30
    assert O.f64_to_f16(v) == 0x3C01
    assert np.float32(v).astype(np.float16).view(np.uint16) == 0x3C00


def test_bf16_to_f64_matches_bit_definition():
    for b in (0x0000, 0x3F80, 0xBF80, 0x4049, 0x0001, 0x7F7F, 0x8000, 0x3DCD):
        ref = np.array([b << 16], dtype=np.uint32).view(np.float32)[0]
        assert O.bf16_to_f64(b) == float(ref)


# --------------------------------------------------------------------------- quantiser

def test_quantizer_hand_worked_group():
    # b = 4: mn = -0.75, mx = 1.125 -> S = 1.875 / 15 = 0.125 exactly, z = 6.
    w = np.zeros((1, 128), np.float32)
    for k in range(128):
        w[0, k] = ((k % 16) - 6) * 0.125          # lands exactly on code k % 16
    w[0, 16] = 0.0625                              # w/S = 0.5 -> ties-to-even -> 0 -> q = 6
    w[0, 17] = 0.1875                              # w/S = 1.5 -> 2 -> q = 8
    w[0, 18] = -0.0625                             # -0.5 -> -0 -> q = 6
    w[0, 19] = 0.3125                              # 2.5 -> 2 -> q = 8
    codes, s, z = O.quantize(w, 4)
    expect = np.array([k % 16 for k in range(128)], np.uint8)
    expect[16], expect[17], expect[18], expect[19] = 6, 8, 6, 8
    assert np.array_equal(codes[0], expect)
    assert s[0, 0] == 0x3000                       # fp16(0.125)
    assert z[0, 0] == 0x4600                       # fp16(6.0)


def test_quantizer_rounds_the_scale_before_the_codes():
    # b = 4, mn = 0, mx = 1: (mx - mn) / 15 = 0.0666... is not an fp16 number.  Between 2^-4 and 2^-3 fp16
    # steps by 2^-14; 0.0666667 = 2^-4 + 68.27 * 2^-14 rounds to 2^-4 + 68 * 2^-14 = 0.066650390625 = 0x2C44.
    # The codes are computed against THAT scale: 0.4999 / 0.066650390625 = 7.5003 -> 8, whereas against the
    # unrounded 1/15 it would be 7.4985 -> 7.  (z = rint(0 / s) = 0.)
    w = np.full((1, 128), 0.25, np.float32)        # 0.25 / s = 3.7509 -> 4 either way
    w[0, 0], w[0, 1], w[0, 2] = 0.0, 1.0, 0.4999
    codes, s, z = O.quantize(w, 4)
    assert s[0, 0] == 0x2C44 and z[0, 0] == 0x0000
    assert codes[0, 0] == 0 and codes[0, 1] == 15 and codes[0, 2] == 8
    assert np.all(codes[0, 3:] == 4)


def test_quantizer_degenerate_and_clamped_groups():
    w = np.full((2, 128), 0.25, np.float32)        # constant group: range 0 -> s = 2^-14
    w[1] = 0.0
    w[1, 5] = 1e-9                                  # range/qmax underflows fp16 -> s = 2^-14
    codes, s, z = O.quantize(w, 3)
    assert s[0, 0] == 0x0400 and s[1, 0] == 0x0400
    assert z[0, 0] == 0x0000                       # -mn/S negative -> clamped to 0
    assert np.all(codes[0] == 7)                   # 0.25 / 2^-14 = 4096 -> clamped to qmax
    assert np.all(codes[1] == 0) and z[1, 0] == 0


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8])
def test_quantizer_invariants(bits):
    rng = np.random.default_rng(bits)
    w = (rng.standard_normal((24, 512)) * 0.02).astype(np.float32)
    codes, s, z = O.quantize(w, bits)
    qmax = 2 ** bits - 1
    assert codes.max() <= qmax
    S = s.view(np.float16).astype(np.float64)
    Z = z.view(np.float16).astype(np.float64)
    assert np.all(Z == np.round(Z)) and Z.min() >= 0 and Z.max() <= qmax
    wg = w.reshape(24, 4, 128).astype(np.float64)
    cg = codes.reshape(24, 4, 128).astype(np.float64)
    # the group's minimum and maximum land within one code of 0 and qmax
    amin, amax = wg.argmin(-1), wg.argmax(-1)
    assert np.all(np.take_along_axis(cg, amin[..., None], -1) <= 1)
    assert np.all(np.take_along_axis(cg, amax[..., None], -1) >= qmax - 1)
    # reconstruction error of unclamped codes is at most half a step
    err = np.abs(wg - (cg - Z[..., None]) * S[..., None])
    inner = (cg > 0) & (cg < qmax)
    assert np.all(err[inner] <= 0.5 * np.broadcast_to(S[..., None], err.shape)[inner] * (1 + 1e-9))
    # clamped codes may be off by at most one more step (scale rounding to fp16)
    assert np.all(err <= 1.5 * S[..., None] + 1e-12)


# --------------------------------------------------------------------------- packed format

def _np_bitstream(codes, bits):
    """Independent construction with numpy: LSB-first bits of each code, concatenated."""
    n, k = codes.shape
    b = np.unpackbits(codes[..., None], axis=-1, bitorder="little")[..., :bits]     # [n][k][bits]
    by = np.packbits(b.reshape(n, k * bits), axis=-1, bitorder="little")             # bytes
    return by.view("<u4")


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("k", [128, 256, 4096])
def test_pack_bitstream_matches_numpy_packbits_and_round_trips(bits, k):
    rng = np.random.default_rng(100 * bits + k)
    qmax = 2 ** bits - 1
    codes = rng.integers(0, qmax + 1, size=(5, k), dtype=np.uint8)
    codes[0] = 0
    codes[1] = qmax
    codes[2] = np.where(np.arange(k) % 2 == 0, 0, qmax)
    packed = O.pack_bitstream(codes, bits)
    assert packed.shape == (5, k * bits // 32)
    assert packed.nbytes == 5 * k * bits // 8
    assert np.array_equal(packed, _np_bitstream(codes, bits))
    assert np.array_equal(O.unpack_bitstream(packed, k, bits), codes)


@pytest.mark.parametrize("k", [11008, 13824])
def test_pack_bitstream_round_trip_model_widths(k):
    rng = np.random.default_rng(k)
    for bits in (3, 5, 7):
        codes = rng.integers(0, 2 ** bits, size=(2, k), dtype=np.uint8)
        assert np.array_equal(O.unpack_bitstream(O.pack_bitstream(codes, bits), k, bits), codes)


def test_pack_4bit_is_eight_nibbles_per_word_and_8bit_is_the_bytes():
    rng = np.random.default_rng(7)
    c4 = rng.integers(0, 16, size=(3, 128), dtype=np.uint8)
    p4 = O.pack_bitstream(c4, 4)
    ref = (c4.reshape(3, 16, 8).astype(np.uint64) * (16 ** np.arange(8, dtype=np.uint64))).sum(-1)
    assert np.array_equal(p4.astype(np.uint64), ref)
    c8 = rng.integers(0, 256, size=(3, 128), dtype=np.uint8)
    assert np.array_equal(O.pack_bitstream(c8, 8).view(np.uint8), c8)


# --------------------------------------------------------------------------- nested format

def test_nested_invariant_exhaustive():
    q8 = np.tile(np.arange(256, dtype=np.uint8), (2, 1))          # every parent code, K = 256
    q8[1] = q8[1][::-1]
    planes = O.pack_planes(q8)
    assert planes.shape == (8, 2, 8)
    bits_ref = np.unpackbits(q8[..., None], axis=-1, bitorder="little")   # [n][k][p]
    for t in range(8):                                              # stored plane t = parent bit 7 - t
        ref = np.packbits(bits_ref[..., 7 - t], axis=-1, bitorder="little").view("<u4")
        assert np.array_equal(planes[t], ref)
        assert int(np.unpackbits(planes[t].view(np.uint8)).sum()) == int(bits_ref[..., 7 - t].sum())
    for b in range(2, 9):
        assert np.array_equal(O.child_codes(planes, 256, b), q8 >> (8 - b))
    # dropping planes never changes the retained bytes: the b-bit child is a prefix
    for b in range(2, 8):
        assert planes[:b].tobytes() == planes.tobytes()[: b * 2 * 8 * 4]


# --------------------------------------------------------------------------- dequantisation

def test_dequant_closed_form_hand_cases():
    one, half = 0x3C00, 0x3800
    for q in range(256):
        assert O.dequant_one(q, 8, 8, one, 0x0000) == float(q)              # s = 1, z = 0
        assert O.dequant_one(q, 8, 8, half, O.f64_to_f16(q)) == 0.0         # q == z
    assert O.dequant_one(5, 4, 4, half, O.f64_to_f16(7)) == -1.0            # (5 - 7) * 0.5
    # one rounding of the exact product: 255 * fp16(0.1) = 25.4937..., fp16 spacing there is 2^-6
    s = O.f64_to_f16(0.1)
    exact = 255 * float(np.array([s], np.uint16).view(np.float16)[0])
    assert O.dequant_one(255, 8, 8, s, 0) == float(np.float16(exact))
    # monotone in q
    vals = [O.dequant_one(q, 8, 8, s, O.f64_to_f16(100)) for q in range(256)]
    assert all(b > a for a, b in zip(vals, vals[1:]))


def test_dequant_nested_child_midpoint_fill():
    s = O.f64_to_f16(0.0123)
    z = O.f64_to_f16(131)
    S = float(np.array([s], np.uint16).view(np.float16)[0])
    for q8 in range(256):
        w8 = O.dequant_one(q8, 8, 8, s, z)
        for b in range(2, 8):
            qb = q8 >> (8 - b)
            wb = O.dequant_one(qb, b, 8, s, z)
            d = (qb << (8 - b)) + (1 << (7 - b)) - 131                       # parent units
            assert wb == float(np.float16(d * S))
            assert abs(wb - w8) <= (1 << (7 - b)) * S + 2 ** -11 * (abs(w8) + abs(wb))


def test_dequant_matrix_matches_numpy_closed_form():
    rng = np.random.default_rng(3)
    w = (rng.standard_normal((8, 256)) * 0.02).astype(np.float32)
    for bits in (2, 4, 7, 8):
        codes, s, z = O.quantize(w, bits)
        S = np.repeat(s.view(np.float16).astype(np.float64), 128, axis=1)
        Z = np.repeat(z.view(np.float16).astype(np.float64), 128, axis=1)
        ref = ((codes.astype(np.float64) - Z) * S).astype(np.float16).astype(np.float64)
        assert np.array_equal(O.dequant(codes, s, z, bits), ref)


# --------------------------------------------------------------------------- GEMV / GEMM

def _f32_to_bf16_bits(a):
    u = np.ascontiguousarray(a, np.float32).view(np.uint32).astype(np.uint64)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8])
def test_gemv_and_gemm_brute_force_vs_numpy(bits):
    rng = np.random.default_rng(10 + bits)
    n, k, m = 16, 256, 8
    w = (rng.standard_normal((n, k)) * 0.02).astype(np.float32)
    codes, s, z = O.quantize(w, bits)
    S = np.repeat(s.view(np.float16).astype(np.float64), 128, axis=1)
    Z = np.repeat(z.view(np.float16).astype(np.float64), 128, axis=1)
    w_hat = ((codes.astype(np.float64) - Z) * S).astype(np.float16).astype(np.float64)
    x16 = rng.standard_normal((m, k)).astype(np.float16)
    y = O.gemv(codes, s, z, bits, x16.view(np.uint16))
    ref = x16.astype(np.float64) @ w_hat.T
    assert y.shape == (m, n)
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-13)
    xb = _f32_to_bf16_bits(rng.standard_normal((m, k)).astype(np.float32))
    xb_val = (xb.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    Y = O.gemm(codes, s, z, bits, xb)
    assert np.allclose(Y, xb_val @ w_hat.T, rtol=1e-12, atol=1e-13)
    # a transposed-operand mistake would show here: y is not symmetric in (m, n)
    assert not np.allclose(Y[:8, :8], Y[:8, :8].T)


def test_gemv_one_hot_recovers_columns_and_zero_codes_give_zero():
    rng = np.random.default_rng(5)
    w = (rng.standard_normal((16, 128)) * 0.02).astype(np.float32)
    codes, s, z = O.quantize(w, 5)
    w_hat = O.dequant(codes, s, z, 5)
    for kk in (0, 1, 63, 127):
        x = np.zeros(128, np.float16)
        x[kk] = 1.0
        assert np.array_equal(O.gemv(codes, s, z, 5, x.view(np.uint16))[0], w_hat[:, kk])
    zc = np.repeat(z.view(np.float16).astype(np.uint8), 128, axis=1)      # every code equals its zero point
    x = rng.standard_normal(128).astype(np.float16)
    assert np.all(O.gemv(zc, s, z, 5, x.view(np.uint16)) == 0.0)


def test_gemv_exact_integer_row_sums():
    rng = np.random.default_rng(6)
    codes = rng.integers(0, 256, size=(8, 512), dtype=np.uint8)
    s = np.full((8, 4), 0x3C00, np.uint16)         # 1.0
    z = np.zeros((8, 4), np.uint16)
    x = np.full(512, 2.0 ** -8, np.float16)
    y = O.gemv(codes, s, z, 8, x.view(np.uint16))[0]
    assert np.array_equal(y, codes.astype(np.int64).sum(1) / 256.0)


def test_gemv_nested_child_uses_parent_scale_and_midpoint():
    rng = np.random.default_rng(8)
    w = (rng.standard_normal((4, 256)) * 0.02).astype(np.float32)
    q8, s, z = O.quantize(w, 8)
    x = rng.standard_normal(256).astype(np.float16)
    S = np.repeat(s.view(np.float16).astype(np.float64), 128, axis=1)
    Z = np.repeat(z.view(np.float16).astype(np.float64), 128, axis=1)
    for b in (2, 3, 5, 8):
        qb = q8 >> (8 - b)
        h = (1 << (7 - b)) if b < 8 else 0
        d = qb.astype(np.float64) * (1 << (8 - b)) + h - Z
        ref = x.astype(np.float64) @ (d * S).astype(np.float16).astype(np.float64).T
        got = O.gemv(qb, s, z, b, x.view(np.uint16), parent_bits=8)[0]
        assert np.allclose(got, ref, rtol=1e-12, atol=1e-13)


# --------------------------------------------------------------------------- footprint

def test_footprint_closed_forms():
    assert O.footprint([4096], [4096], [4]) == 8_388_608 + 524_288 == 8_912_896
    import fq_synth as S
    sh = S.stack_shapes("7b")
    n, k = [s.n_out for s in sh], [s.k_in for s in sh]
    assert len(sh) == 224 and sum(a * b for a, b in zip(n, k)) == 6_476_005_376
    assert O.footprint(n, k, [4] * 224) == 3_238_002_688 + 202_375_168
    assert O.footprint(n, k, [8] * 224) == 6_678_380_544
    sh13 = S.stack_shapes("13b")
    assert O.footprint([s.n_out for s in sh13], [s.k_in for s in sh13], [8] * 280) == 13_084_262_400
    # mixed bits: the sum of per-layer terms, written out independently
    bits = S.draw_bits(11, 224, [3, 4, 5, 6, 8])
    ref = sum(a * b * int(c) // 8 + a * (b // 128) * 4 for a, b, c in zip(n, k, bits))
    assert O.footprint(n, k, bits) == ref


def test_footprint_against_paper_accounting_figures():
    g = _golden("paper_accounting.txt")
    assert abs(2.0 ** int(g["design_space_log2"]) / float(g["design_space_value"]) - 1) < 5e-3
    import fq_synth as S
    sh = S.stack_shapes("7b")
    n, k = [s.n_out for s in sh], [s.k_in for s in sh]
    chain = S.config_chain(S.tensor_key(2, 0, S.TENSOR_CHAIN), sh, 12, 7.0, 3.5, 3)
    fps = [O.footprint(n, k, c) / 1e9 for c in chain]
    lo, hi = float(g["table1_footprint_min_gb"]), float(g["table1_footprint_max_gb"])
    # Table I's footprint rows (3.0 ... 6.0 GB) bracket the 7B linear-layer stack at 3.5 ... 7.0 bits
    assert lo <= min(fps) <= lo + 0.3 and hi - 0.3 <= max(fps) <= hi
    assert all(b <= a for a, b in zip(fps, fps[1:]))
    # the nested parent (storage set by the largest precision) stays under the AnyPrecision bound
    assert O.footprint(n, k, [8] * 224) / 1e9 < float(g["anyprecision_storage_max_gb"])
    # lowering one module by one bit moves the footprint by well under the ~100 MB granularity
    att = O.footprint(n[:4], k[:4], [8] * 4) - O.footprint(n[:4], k[:4], [7] * 4)
    mlp = O.footprint(n[4:7], k[4:7], [8] * 3) - O.footprint(n[4:7], k[4:7], [7] * 3)
    assert att == 4 * 4096 * 4096 // 8 and mlp == 3 * 11008 * 4096 // 8
    assert max(att, mlp) / 1e6 < float(g["granularity_mb"])
    # stored QMs at 2.5 + 4.0 + 5.0 + 7.5 bits per weight: the linear layers account for most of 17 GB
    tot_bits = sum(float(v) for v in g["fq_storage_bits"].split())
    gb = 6_476_005_376 * tot_bits / 8 / 1e9
    assert 0.85 * float(g["fq_storage_gb"]) < gb < float(g["fq_storage_gb"])


# --------------------------------------------------------------------------- one-way transitions

def test_transition_accounting_closed_forms_and_invariants():
    import fq_synth as S
    sh = S.stack_shapes("7b")
    n, k = [s.n_out for s in sh], [s.k_in for s in sh]
    g = _golden("paper_accounting.txt")
    # nested: replacing one attention module (q,k,v,o) of the 8-bit model by its 3-bit version (the
    # paper's interchangeability example, Sec. III) frees 5 planes of 4 matrices and loads nothing
    to = [8] * 224
    to[0:4] = [3] * 4
    t = O.transition(n, k, [True] * 224, [8] * 224, to)
    assert t["bytes_freed"] == 4 * 4096 * 4096 * 5 // 8 == 41_943_040 and t["bytes_loaded"] == 0
    assert t["layers_changed"] == 4 and t["one_way"]
    # what is freed is exactly the drop in footprint (scale/zero words are shared by all widths)
    assert t["footprint_from"] - t["footprint_to"] == t["bytes_freed"]
    assert t["bytes_freed"] / 1e6 < float(g["granularity_mb"])
    # going back up is not one-way and loads what was freed
    back = O.transition(n, k, [True] * 224, to, [8] * 224)
    assert not back["one_way"] and back["bytes_loaded"] == t["bytes_freed"] and back["bytes_freed"] == 0
    # packed: widths are separate variants, a change swaps codes AND scale/zero words
    p = O.transition([4096], [4096], [False], [8], [3])
    meta = 4096 * 32 * 4
    assert p["bytes_freed"] == 4096 * 4096 + meta and p["bytes_loaded"] == 4096 * 4096 * 3 // 8 + meta and p["one_way"]
    assert p["bytes_freed"] - p["bytes_loaded"] == p["footprint_from"] - p["footprint_to"]
    # no change, nothing moves
    z = O.transition(n, k, [True] * 224, to, to)
    assert z == {"bytes_freed": 0, "bytes_loaded": 0, "layers_changed": 0, "one_way": True,
                 "footprint_from": z["footprint_from"], "footprint_to": z["footprint_from"]}
    # the seeded chains are one-way and every step frees exactly its footprint gap and loads nothing
    chain = S.config_chain(S.tensor_key(2, 0, S.TENSOR_CHAIN), sh, 12, 7.0, 3.5, 3)
    for a, b in zip(chain, chain[1:]):
        t = O.transition(n, k, [True] * 224, a, b)
        assert t["one_way"] and t["bytes_loaded"] == 0 and t["bytes_freed"] == t["footprint_from"] - t["footprint_to"] > 0
    # brute force on a tiny mixed case, written out independently
    nn, kk, nest, f, tt = [32, 64, 16], [256, 128, 384], [True, False, True], [8, 6, 4], [5, 4, 7]
    t = O.transition(nn, kk, nest, f, tt)
    assert t["bytes_freed"] == 32 * 256 * 3 // 8 + (64 * 128 * 6 // 8 + 64 * 4)
    assert t["bytes_loaded"] == (64 * 128 * 4 // 8 + 64 * 4) + 16 * 384 * 3 // 8
    assert t["layers_changed"] == 3 and not t["one_way"]
