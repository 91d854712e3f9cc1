"""Full-size elastic configurations in the nested format (one stored 8-bit parent per layer, children read its leading bits):
the 7B-shaped stack with its 12-configuration chain and the 13B-shaped stack with its 16-configuration
chain.  Footprints are compared bit-for-bit with the oracle, decode / prefill outputs on sampled rows."""
import time

import numpy as np
import pytest
import torch

import fq_synth as S
from oracle import fq_oracle as O
from fq_testlib import GEMM_TOL, GEMV_TOL, bits_of, f64_of

pytestmark = pytest.mark.gpu


def _build_nested(P, cfg, shapes, device):
    fq = P.FlexQ(len(shapes))
    stores = []
    for i, sh in enumerate(shapes):
        w = S.weight_rows(S.tensor_key(cfg, i, S.TENSOR_W), 0, sh.n_out, sh.k_in, device=device)
        c, s, z = P.fq_quantize_layer(w, 8)
        stores.append(fq.fq_pack_layer(i, c, s, z, 8, P.FQ_FMT_PLANES))
        del w, c, s, z
    torch.cuda.synchronize()
    return fq, stores


class _ParentRows:
    """Oracle-quantised 8-bit parent codes of a few sampled rows per layer (CPU, generated row by row)."""

    def __init__(self, cfg, shapes, rows_per_layer):
        self.rows, self.q8, self.s, self.z = [], [], [], []
        for i, sh in enumerate(shapes):
            rows = S.sample_rows(5000 + i, sh.n_out, rows_per_layer)
            w = np.concatenate([S.weight_rows(S.tensor_key(cfg, i, S.TENSOR_W), int(r), int(r) + 1, sh.k_in).numpy()
                                for r in rows])
            q8, s, z = O.quantize(w, 8)
            self.rows.append(rows); self.q8.append(q8); self.s.append(s); self.z.append(z)

    def gemv(self, i, b, xbits):
        return O.gemv(self.q8[i] >> (8 - b), self.s[i], self.z[i], b, xbits, parent_bits=8)

    def gemm(self, i, b, xbits):
        return O.gemm(self.q8[i] >> (8 - b), self.s[i], self.z[i], b, xbits, parent_bits=8)


def _check_decode(fq, shapes, ref, bits, xs, batch, tol):
    L = len(shapes)
    ys = [torch.full((batch, sh.n_out), float("nan"), dtype=torch.float16, device="cuda") for sh in shapes]
    fq.fq_gemv_stack(list(range(L)), xs, ys, S.stack_phases(shapes), batch)
    assert fq.fq_status() == 0
    num = den = 0.0
    for i in range(L):
        got_all = f64_of(ys[i])
        assert np.all(np.isfinite(got_all)), shapes[i].name
        want = ref.gemv(i, int(bits[i]), bits_of(xs[i]))           # [batch][rows]
        got = got_all[:, ref.rows[i]]
        num += float(((got - want) ** 2).sum()); den += float((want ** 2).sum())
        assert O.rel_l2(got, want) <= tol, (shapes[i].name, int(bits[i]))         # the stated tolerance, per matrix
        assert np.max(np.abs(got - want)) <= 4 * tol * np.max(np.abs(want)), (shapes[i].name, int(bits[i]))
    assert np.sqrt(num / den) <= tol, np.sqrt(num / den)


def test_config2_7b_nested_chain():
    import paper_2501_07139_b200 as P
    device = torch.device("cuda", 0)
    shapes = S.stack_shapes("7b")
    L = len(shapes)
    n, k = [s.n_out for s in shapes], [s.k_in for s in shapes]
    fq, stores = _build_nested(P, 2, shapes, device)
    assert fq.fq_storage_bytes() == O.footprint(n, k, [8] * L) == 6_678_380_544
    chain = S.config_chain(S.tensor_key(2, 0, S.TENSOR_CHAIN), shapes, 12, 7.0, 3.5, 3)
    ref = _ParentRows(2, shapes, 58)
    xs = [S.activations(S.tensor_key(2, i, S.TENSOR_X), 1, sh.k_in).to(device) for i, sh in enumerate(shapes)]
    probe = [0, 100, 223]
    before = [stores[i].clone() for i in probe]
    ptrs = [t.data_ptr() for t in stores]
    prev = np.full(L, 8)
    switch_us = []
    for ci, bits in enumerate(chain):
        assert np.all(bits <= prev) and bits.min() >= 3                    # one-way transitions only
        prev = bits
        t0 = time.perf_counter()
        fp = fq.fq_set_config([int(b) for b in bits])
        switch_us.append((time.perf_counter() - t0) * 1e6)
        assert fp == O.footprint(n, k, bits)
        assert abs(S.average_bits(bits, shapes) - np.linspace(7.0, 3.5, 12)[ci]) < 0.06
        if ci in (0, 5, 11):
            _check_decode(fq, shapes, ref, bits, xs, 1, GEMV_TOL)
    # switching configurations moved no weights: same buffers, same bytes
    assert [t.data_ptr() for t in stores] == ptrs
    for t, i in zip(before, probe):
        assert torch.equal(t, stores[i])
    assert max(switch_us) < 5000, switch_us                                 # host bookkeeping only
    fq.fq_destroy()


def test_config4_13b_nested_chain_decode_and_prefill():
    import paper_2501_07139_b200 as P
    device = torch.device("cuda", 0)
    shapes = S.stack_shapes("13b")
    L = len(shapes)
    n, k = [s.n_out for s in shapes], [s.k_in for s in shapes]
    fq, stores = _build_nested(P, 4, shapes, device)
    assert L == 280 and fq.fq_storage_bytes() == 13_084_262_400
    chain = S.config_chain(S.tensor_key(4, 0, S.TENSOR_CHAIN), shapes, 16, 6.0, 2.5, 2)
    for bits in chain:
        assert fq.fq_set_config([int(b) for b in bits]) == O.footprint(n, k, bits)
    ref = _ParentRows(4, shapes, 26)
    x1 = [S.activations(S.tensor_key(4, i, S.TENSOR_X), 1, sh.k_in).to(device) for i, sh in enumerate(shapes)]
    x8 = [S.activations(S.tensor_key(4, 1000 + i, S.TENSOR_X), 8, sh.k_in).to(device) for i, sh in enumerate(shapes)]
    for ci in (0, 15):
        bits = chain[ci]
        fq.fq_set_config([int(b) for b in bits])
        _check_decode(fq, shapes, ref, bits, x1, 1, GEMV_TOL)
        _check_decode(fq, shapes, ref, bits, x8, 8, GEMV_TOL)
    # prefill at 1 x 2048 tokens on the first and the last block, lowest configuration (2-bit children occur)
    bits = chain[15]
    assert bits.min() == 2
    m = 2048
    xb = {kk: S.activations(S.tensor_key(4, kk, S.TENSOR_X), m, kk, torch.bfloat16, device=device) for kk in sorted(set(k))}
    trows = [0, 127, 128, 1000, m - 1]
    for i in list(range(7)) + list(range(L - 7, L)):
        sh = shapes[i]
        y = torch.empty((m, sh.n_out), dtype=torch.bfloat16, device=device)
        fq.fq_gemm(i, xb[sh.k_in], y)
        assert fq.fq_status() == 0
        want = ref.gemm(i, int(bits[i]), bits_of(xb[sh.k_in][trows]))
        got = f64_of(y[trows][:, torch.from_numpy(ref.rows[i]).cuda()])
        assert O.rel_l2(got, want) <= GEMM_TOL, (sh.name, int(bits[i]))
    fq.fq_destroy()
