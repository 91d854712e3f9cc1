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


def test_swap_transition_loads_before_it_releases_and_decodes_bit_identically():
    """Swap model (Sec. II-C): only the active variants are on the device, the others wait in page-locked host
    memory; a one-way chain of swaps against a context that keeps everything resident."""
    import fq_synth as S
    import paper_2501_07139_b200 as P
    dev = torch.device("cuda", 0)
    shapes = [(2048, 4096), (1000, 2048), (4096, 1024)]
    variants = (8, 5, 3)
    ref = P.FlexQ(4)                                       # everything resident
    fq = P.FlexQ(4)                                        # swap model
    sizes = {}
    for i, (n, k) in enumerate(shapes):
        w = S.weight_rows(S.tensor_key(140, i, S.TENSOR_W), 0, n, k, device=dev)
        for b in variants:
            c, s, z = P.fq_quantize_layer(w, b)
            store = ref.fq_pack_layer(i, c, s, z, b, P.FQ_FMT_PACKED)
            sizes[(i, b)] = store.numel()
            assert store.numel() == P.fq_store_bytes(n, k, b, P.FQ_FMT_PACKED)
            fq.fq_host_variant(i, n, k, b, store.cpu().pin_memory())
    # layer 3: a nested parent, resident in both
    w = S.weight_rows(S.tensor_key(140, 3, S.TENSOR_W), 0, 512, 1024, device=dev)
    c, s, z = P.fq_quantize_layer(w, 8)
    ref.fq_pack_layer(3, c, s, z, 8, P.FQ_FMT_PLANES)
    fq.fq_pack_layer(3, c, s, z, 8, P.FQ_FMT_PLANES)
    all_shapes = shapes + [(512, 1024)]
    xs = [S.activations(S.tensor_key(140, i, S.TENSOR_X), 1, k).to(dev)[0] for i, (n, k) in enumerate(all_shapes)]

    def same_outputs(cfg):
        ref.fq_set_config(cfg)
        for i, (n, k) in enumerate(all_shapes):
            ya = torch.full((n,), float("nan"), dtype=torch.float16, device=dev)
            yb = torch.full((n,), float("nan"), dtype=torch.float16, device=dev)
            ref.fq_gemv(i, xs[i], ya)
            fq.fq_gemv(i, xs[i], yb)
            assert torch.equal(ya, yb), (cfg, i)
        ys = [torch.empty(n, dtype=torch.float16, device=dev) for n, _ in all_shapes]
        yr = [torch.empty(n, dtype=torch.float16, device=dev) for n, _ in all_shapes]
        fq.fq_gemv_stack(list(range(4)), xs, ys, None, 1)
        ref.fq_gemv_stack(list(range(4)), xs, yr, None, 1)
        assert all(torch.equal(a, b) for a, b in zip(ys, yr))
        assert fq.fq_status() == 0 and ref.fq_status() == 0

    n_all, k_all = [s[0] for s in all_shapes], [s[1] for s in all_shapes]
    # nothing usable before the first swap: the packed layers have no resident variant
    with pytest.raises(P.FlexQError):
        fq.fq_set_config([8, 8, 8, 8])
    cur = [8, 8, 8, 8]
    rep = fq.fq_transition_swap(cur)
    assert rep["bytes_loaded"] == sum(sizes[(i, 8)] for i in range(3)) and rep["bytes_freed"] == 0
    assert rep["resident_bytes"] == rep["bytes_loaded"] and rep["footprint_to"] == O.footprint(n_all, k_all, cur)
    same_outputs(cur)
    resident = rep["resident_bytes"]
    for nxt in ([8, 5, 8, 6], [3, 5, 8, 6], [3, 3, 5, 4], [3, 3, 3, 2]):
        torch.cuda.synchronize()
        free0 = torch.cuda.mem_get_info()[0]
        rep = fq.fq_transition_swap(nxt)
        changed = [i for i in range(3) if cur[i] != nxt[i]]
        loaded = sum(sizes[(i, nxt[i])] for i in changed)
        freed = sum(sizes[(i, cur[i])] for i in changed)
        assert rep["bytes_loaded"] == loaded and rep["bytes_freed"] == freed and rep["one_way"] == 1
        assert rep["layers_changed"] == sum(1 for a, b in zip(cur, nxt) if a != b)
        # a layer's replacement is resident before the layer's old variant goes, one layer at a time
        assert rep["peak_extra_bytes"] == max(sizes[(i, nxt[i])] for i in changed)
        resident += loaded - freed
        assert rep["resident_bytes"] == resident
        assert rep["footprint_from"] == O.footprint(n_all, k_all, cur) and rep["footprint_to"] == O.footprint(n_all, k_all, nxt)
        torch.cuda.synchronize()
        free1 = torch.cuda.mem_get_info()[0]
        assert free1 - free0 >= (freed - loaded) - (8 << 20)          # the memory really went back (pool granularity aside)
        cur = nxt
        same_outputs(cur)
    # one-way is enforced before anything moves; a width that was never registered is refused
    with pytest.raises(P.FlexQError) as e:
        fq.fq_transition_swap([5, 3, 3, 2])
    assert e.value.code == -10 and [fq.fq_active_bits(i) for i in range(4)] == cur
    with pytest.raises(P.FlexQError) as e:
        fq.fq_transition_swap([3, 3, 2, 2])
    assert e.value.code == -5 and [fq.fq_active_bits(i) for i in range(4)] == cur
    # going back up is a swap like any other when the caller allows it
    rep = fq.fq_transition_swap([8, 3, 3, 7], require_one_way=False)
    assert rep["one_way"] == 0 and rep["bytes_loaded"] == sizes[(0, 8)] and rep["bytes_freed"] == sizes[(0, 3)]
    same_outputs([8, 3, 3, 7])
    fq.fq_destroy()
    ref.fq_destroy()
