"""Ensemble generation end to end on a small nested stack: the tables measured with fq_gemm / fq_sqdiff against
the fp64 oracle, then the library's search and pruning against the oracle's on the same tables."""
from collections import namedtuple

import numpy as np
import pytest
import torch

from oracle import fq_oracle as O
from oracle import fq_search as OS
from fq_testlib import bits_of, make_layer, to_dev, x_bf16

pytestmark = pytest.mark.gpu
Shape = namedtuple("Shape", "n_out k_in")


def test_sqdiff_matches_numpy():
    import paper_2501_07139_b200 as P
    g = torch.Generator().manual_seed(5)
    a = torch.randn(333, 257, generator=g).to(torch.bfloat16).cuda()
    b = torch.randn(333, 257, generator=g).to(torch.bfloat16).cuda()
    got = P.fq_sqdiff(a, b).cpu().numpy()
    a64, b64 = a.double().cpu().numpy(), b.double().cpu().numpy()
    assert np.allclose(got, [((a64 - b64) ** 2).sum(), (b64 ** 2).sum()], rtol=1e-12)


def test_tables_search_and_pruning_on_a_small_stack():
    import paper_2501_07139_b200 as P
    from paper_2501_07139_b200 import search as SR
    shapes = [Shape(64, 256), Shape(64, 256), Shape(96, 256), Shape(64, 384)] * 2
    modules = [[0, 1], [2, 3], [4, 5], [6, 7]]
    levels = [8, 5, 3]
    tokens, sens_tokens = 48, 16
    fq = P.FlexQ(len(shapes))
    layers = [make_layer(150, i, sh.n_out, sh.k_in, 8) for i, sh in enumerate(shapes)]
    for i, lay in enumerate(layers):
        fq.fq_pack_layer(i, *to_dev(*lay), 8, P.FQ_FMT_PLANES)
    calib = {k: x_bf16(150, k, tokens, k) for k in (256, 384)}
    out = SR.generate_ensemble(fq, shapes, modules, levels, {k: v.cuda() for k, v in calib.items()},
                               stems=2, branches=3, sens_tokens=sens_tokens, prune_fraction=0.5)
    assert fq.fq_status() == 0
    # tables against the oracle (fp64 outputs of the same codes; the kernel rounds w^ and Y to bf16)
    def rel_err(i, b, rows):
        codes, s, z = layers[i]
        xb = bits_of(calib[shapes[i].k_in])[:rows]
        y8 = O.gemm(codes, s, z, 8, xb, parent_bits=8)
        yb = O.gemm(codes >> (8 - b), s, z, b, xb, parent_bits=8)
        return float(((yb - y8) ** 2).sum() / (y8 ** 2).sum())
    for m, mod in enumerate(modules):
        for li, b in enumerate(levels):
            ref_c = sum(rel_err(i, b, tokens) for i in mod) if li else 0.0
            ref_s = sum(rel_err(i, b, sens_tokens) for i in mod) if li else 0.0
            assert abs(out["cost"][m][li] - ref_c) <= 0.05 * ref_c + 1e-12, (m, b, out["cost"][m][li], ref_c)
            assert abs(out["sens"][m][li] - ref_s) <= 0.05 * ref_s + 1e-12
            assert out["foot"][m][li] == sum(shapes[i].n_out * shapes[i].k_in * b // 8 for i in mod)
        assert out["cost"][m][0] == 0.0 and out["cost"][m][1] < out["cost"][m][2]      # fewer bits, larger error
    # the search and the pruning are index work on the measured tables: identical to the oracle's
    ref_chain, ref_curve = OS.search_chain(out["cost"], out["sens"], out["foot"], 2, 3)
    assert out["chain"] == ref_chain and out["curve"] == ref_curve
    rp, rd, rb, ra = OS.prune_chain(ref_chain, 3, out["foot"], 0.5)
    assert (out["pruned_chain"], out["dropped"], out["storage_before"], out["storage_after"]) == (rp, rd, rb, ra)
    # the chain is a valid one-way sequence of configurations for the runtime
    n, k = [s.n_out for s in shapes], [s.k_in for s in shapes]
    bits = SR.chain_to_bits(out["chain"], modules, levels, len(shapes))
    fq.fq_set_config(bits[0])
    for b0, b1 in zip(bits, bits[1:]):
        rep = fq.fq_transition(b1, require_one_way=True)
        assert rep == O.transition(n, k, [True] * len(shapes), b0, b1) and rep["bytes_loaded"] == 0
    fq.fq_destroy()
