"""fq_save / fq_load: the ensemble on disk (the paper's "storage cost" is the size of these stored variants)."""
import os
import struct

import numpy as np
import pytest
import torch

from oracle import fq_oracle as O
from fq_testlib import bits_of, make_layer, to_dev, x_fp16

pytestmark = pytest.mark.gpu


def _parse(path):
    """Independent reader of the file format stated in include/flexq.h."""
    raw = open(path, "rb").read()
    assert raw[:8] == b"FLEXQ1\0\0"
    n_layers, zero = struct.unpack_from("<II", raw, 8)
    assert zero == 0
    off, layers = 16, []
    for _ in range(n_layers):
        reg, n, k, fmt, active, mask = struct.unpack_from("<6I", raw, off)
        off += 24
        variants = {}
        for b in range(2, 9):
            if mask >> b & 1:
                (nbytes,) = struct.unpack_from("<Q", raw, off)
                off += 8
                variants[b] = raw[off:off + nbytes]
                off += nbytes
        layers.append(dict(reg=reg, n=n, k=k, fmt=fmt, active=active, variants=variants))
    assert off == len(raw)
    return layers


def test_save_load_round_trip(tmp_path):
    import paper_2501_07139_b200 as P
    path = os.path.join(tmp_path, "ensemble.flexq")
    shapes = [(129, 1024), (40, 384)]
    fq = P.FlexQ(3)                                        # layer 2 stays unregistered
    q8 = make_layer(140, 0, *shapes[0], 8)
    fq.fq_pack_layer(0, *to_dev(*q8), 8, P.FQ_FMT_PLANES)
    packed = {b: make_layer(140, 1, *shapes[1], b) for b in (3, 6)}
    for b in (3, 6):
        fq.fq_pack_layer(1, *to_dev(*packed[b]), b, P.FQ_FMT_PACKED)
    fq.fq_set_config([5, 6])
    written = fq.fq_save(path)
    assert written == os.path.getsize(path)
    # the file holds exactly the stored variants, byte for byte, and its payload is the storage footprint
    L = _parse(path)
    assert [l["reg"] for l in L] == [1, 1, 0] and L[0]["active"] == 5 and L[1]["active"] == 6
    assert sorted(L[0]["variants"]) == [8] and sorted(L[1]["variants"]) == [3, 6]
    for (layer, b), t in fq._keep.items():
        assert L[layer]["variants"][b] == t.cpu().numpy().tobytes()
    payload = sum(len(v) for l in L for v in l["variants"].values())
    assert payload == sum(P.fq_store_bytes(l["n"], l["k"], b, l["fmt"]) for l in L for b in l["variants"])
    assert written == 16 + 24 * 3 + 8 * 3 + payload
    # a fresh context loaded from the file behaves like the original
    g = P.FlexQ(3)
    g.fq_load(path)
    assert g.fq_storage_bytes() == fq.fq_storage_bytes() == O.footprint([129, 40, 40], [1024, 384, 384], [8, 3, 6])
    assert [g.fq_active_bits(i) for i in range(2)] == [5, 6]
    for b in range(2, 9):                                  # nested children re-derived from the loaded planes
        out = g.fq_export_layer(0, b, *shapes[0]).cpu().numpy().view(np.uint32)
        assert np.array_equal(out.reshape(-1), O.pack_planes(q8[0])[:b].reshape(-1))
    for b in (3, 6):
        out = g.fq_export_layer(1, b, *shapes[1]).cpu().numpy().view(np.uint32).reshape(shapes[1][0], -1)
        assert np.array_equal(out, O.pack_bitstream(packed[b][0], b))
    for layer, (n, k) in enumerate(shapes):
        x = x_fp16(140, 7 + layer, 1, k).cuda()
        y0 = torch.empty(n, dtype=torch.float16, device="cuda")
        y1 = torch.empty(n, dtype=torch.float16, device="cuda")
        fq.fq_gemv(layer, x, y0)
        g.fq_gemv(layer, x, y1)
        torch.cuda.synchronize()
        assert np.array_equal(bits_of(y0), bits_of(y1))
    assert fq.fq_status() == 0 and g.fq_status() == 0
    # errors: loading into a context that already has layers, a missing file, a damaged file
    with pytest.raises(P.FlexQError) as e:
        g.fq_load(path)
    assert e.value.code == -1
    h = P.FlexQ(3)
    with pytest.raises(P.FlexQError) as e:
        h.fq_load(path + ".missing")
    assert e.value.code == -11
    bad = os.path.join(tmp_path, "bad.flexq")
    open(bad, "wb").write(open(path, "rb").read()[:-100])
    with pytest.raises(P.FlexQError) as e:
        h.fq_load(bad)
    assert e.value.code == -11
    h.fq_load(path)                                        # the failed attempts changed nothing
    assert h.fq_storage_bytes() == fq.fq_storage_bytes()
    for c in (fq, g, h):
        c.fq_destroy()
