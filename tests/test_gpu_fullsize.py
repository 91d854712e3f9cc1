"""Full-size parity: the 7B-shaped mixed-bit stack, built and launched exactly as bench.py does
(GPU quantiser -> packer -> one persistent fq_gemv_stack launch with dependency phases), checked
against the CPU oracle on sampled output rows of every matrix."""
import numpy as np
import pytest
import torch

import fq_synth as S
from oracle import fq_oracle as O
from fq_testlib import GEMV_TOL, bits_of, f64_of

pytestmark = pytest.mark.gpu


def test_7b_stack_sampled_rows_match_oracle():
    import bench
    import paper_2501_07139_b200 as P
    device = torch.device("cuda", 0)
    shapes = S.stack_shapes("7b")
    L = len(shapes)
    bits = S.draw_bits(S.tensor_key(bench.CONFIG_ID, 0, S.TENSOR_BITS), L, bench.BIT_CHOICES)
    fq = bench.build_stack(P, shapes, bits, device)
    footprint = fq.fq_set_config([int(b) for b in bits])
    assert footprint == O.footprint([s.n_out for s in shapes], [s.k_in for s in shapes], bits)
    xs = [S.activations(S.tensor_key(bench.CONFIG_ID, i, S.TENSOR_X), 1, sh.k_in).to(device)
          for i, sh in enumerate(shapes)]
    ys = [torch.full((sh.n_out,), float("nan"), dtype=torch.float16, device=device) for sh in shapes]
    fq.fq_gemv_stack(list(range(L)), xs, ys, S.stack_phases(shapes), 1)
    assert fq.fq_status() == 0
    worst, num, den = 0.0, 0.0, 0.0
    for i, sh in enumerate(shapes):
        got_all = f64_of(ys[i])
        assert np.all(np.isfinite(got_all)), shapes[i].name
        rows = S.sample_rows(1000 + i, sh.n_out, 58)            # 64 rows of every matrix
        # contiguous runs of rows are generated and quantised on the CPU, one row at a time
        w = np.concatenate([S.weight_rows(S.tensor_key(bench.CONFIG_ID, i, S.TENSOR_W), int(r), int(r) + 1,
                                          sh.k_in).numpy() for r in rows])
        c, s, z = O.quantize(w, int(bits[i]))
        ref = O.gemv(c, s, z, int(bits[i]), bits_of(xs[i]))[0]
        got = got_all[rows]
        err = float(np.sqrt(((got - ref) ** 2).sum()) / np.sqrt((ref ** 2).sum()))
        worst = max(worst, err)
        num += float(((got - ref) ** 2).sum())
        den += float((ref ** 2).sum())
        assert err <= GEMV_TOL, (sh.name, int(bits[i]), err)          # the stated tolerance, per matrix
        # ... and no single output is off by more than a few times that (a norm alone would hide one bad row)
        assert np.max(np.abs(got - ref)) <= 4 * GEMV_TOL * np.max(np.abs(ref)), (sh.name, int(bits[i]))
    assert np.sqrt(num / den) <= GEMV_TOL, (np.sqrt(num / den), worst)
    fq.fq_destroy()
