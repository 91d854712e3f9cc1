"""fq_transition (one-way configuration switch, Sec. II-C / III-B) against the oracle's accounting."""
import numpy as np
import pytest
import torch

from oracle import fq_oracle as O
from fq_testlib import GEMV_TOL, bits_of, f64_of, make_layer, to_dev, x_fp16

pytestmark = pytest.mark.gpu


def test_transition_reports_match_oracle_and_respect_one_way():
    import paper_2501_07139_b200 as P
    shapes = [(64, 512), (40, 384), (129, 1024)]          # two nested layers around one packed layer
    nested = [True, False, True]
    fq = P.FlexQ(3)
    q8a = make_layer(130, 0, *shapes[0], 8)
    q8c = make_layer(130, 2, *shapes[2], 8)
    fq.fq_pack_layer(0, *to_dev(*q8a), 8, P.FQ_FMT_PLANES)
    packed = {b: make_layer(130, 1, *shapes[1], b) for b in (6, 4)}
    for b in (6, 4):
        fq.fq_pack_layer(1, *to_dev(*packed[b]), b, P.FQ_FMT_PACKED)
    fq.fq_pack_layer(2, *to_dev(*q8c), 8, P.FQ_FMT_PLANES)
    n, k = [s[0] for s in shapes], [s[1] for s in shapes]
    cur = [8, 6, 8]
    assert fq.fq_set_config(cur) == O.footprint(n, k, cur)
    store_before = fq._keep[(0, 8)].clone()
    for nxt in ([6, 6, 8], [6, 4, 5], [3, 4, 2]):          # a one-way chain
        rep = fq.fq_transition(nxt)
        assert rep == O.transition(n, k, nested, cur, nxt)
        assert rep["one_way"] and [fq.fq_active_bits(i) for i in range(3)] == nxt
        cur = nxt
    assert torch.equal(store_before, fq._keep[(0, 8)])     # switching moves no weight byte
    # raising a layer is refused when one-way is required, and nothing changes
    with pytest.raises(P.FlexQError) as e:
        fq.fq_transition([3, 4, 5])
    assert e.value.code == -10 and [fq.fq_active_bits(i) for i in range(3)] == cur
    rep = fq.fq_transition([3, 6, 5], require_one_way=False)
    assert rep == O.transition(n, k, nested, cur, [3, 6, 5]) and not rep["one_way"]
    # argument checks are those of fq_set_config
    for bad, code in (([3, 5, 5], -5), ([3, 6, 9], -2), ([3, 6], -1)):
        with pytest.raises(P.FlexQError) as e:
            fq.fq_transition(bad, require_one_way=False)
        assert e.value.code == code
    # the configuration reached by transitions decodes like the one set directly
    x = x_fp16(130, 9, 1, k[2]).cuda()
    y = torch.empty(n[2], dtype=torch.float16, device="cuda")
    fq.fq_gemv(2, x, y)
    ref = O.gemv(q8c[0] >> 3, q8c[1], q8c[2], 5, bits_of(x), parent_bits=8)[0]
    assert O.rel_l2(f64_of(y), ref) <= GEMV_TOL and fq.fq_status() == 0
    fq.fq_destroy()
