"""A fixed set of calls through the library (decode in every format and width, a dependency-ordered stack, a batch,
the fused prefill kernel, pack / export), every output placed between guard words.  Used twice by
test_gpu_checked_build.py: in-process with the normal library, and as a child process (`python
tests/fq_checked_cases.py out.pt`) with FLEXQ_LIBRARY=checked, i.e. the build whose kernels verify every index."""
from __future__ import annotations

import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import fq_synth as S  # noqa: E402

GUARD = 64            # fp16 / bf16 elements before and after every output
SENTINEL = -12345.0


def guarded(n: int, dtype, dev):
    buf = torch.full((n + 2 * GUARD,), SENTINEL, dtype=dtype, device=dev)
    return buf, buf[GUARD:GUARD + n]


def guards_intact(buf: torch.Tensor) -> bool:
    return bool((buf[:GUARD] == SENTINEL).all()) and bool((buf[-GUARD:] == SENTINEL).all())


def run_cases(P) -> dict:
    dev = torch.device("cuda", 0)
    out, bufs = {}, []

    # 1. one ragged layer in every width and both formats, batch 1 and batch 3
    n, k = 300, 1152
    w = S.weight_rows(S.tensor_key(150, 0, S.TENSOR_W), 0, n, k, device=dev)
    x1 = S.activations(S.tensor_key(150, 1, S.TENSOR_X), 1, k).to(dev)[0]
    x3 = S.activations(S.tensor_key(150, 2, S.TENSOR_X), 3, k).to(dev)
    for fmt in (P.FQ_FMT_PACKED, P.FQ_FMT_PLANES):
        for b in range(2, 9):
            fq = P.FlexQ(1)
            if fmt == P.FQ_FMT_PLANES:
                c, s, z = P.fq_quantize_layer(w, 8)
                fq.fq_pack_layer(0, c, s, z, 8, fmt)
                fq.fq_set_config([b])
            else:
                c, s, z = P.fq_quantize_layer(w, b)
                fq.fq_pack_layer(0, c, s, z, b, fmt)
            buf, y = guarded(n, torch.float16, dev)
            fq.fq_gemv(0, x1, y)
            bufs.append(buf)
            out[f"gemv_f{fmt}_b{b}"] = y.clone()
            buf3, y3 = guarded(3 * n, torch.float16, dev)
            fq.fq_gemv_batched(0, x3, y3.view(3, n))
            bufs.append(buf3)
            out[f"gemv3_f{fmt}_b{b}"] = y3.clone()
            out[f"export_f{fmt}_b{b}"] = fq.fq_export_layer(0, b, n, k)
            assert fq.fq_status() == 0, (fmt, b, fq.fq_status())
            fq.fq_destroy()

    # 2. two decoder blocks of the 7B-shaped stack, mixed widths, dependency-ordered, one launch
    shapes = S.stack_shapes("7b", 2)
    L = len(shapes)
    bits = S.draw_bits(S.tensor_key(151, 0, S.TENSOR_BITS), L, [3, 4, 5, 6, 8])
    fq = P.FlexQ(L)
    for i, (sh, b) in enumerate(zip(shapes, bits)):
        wi = S.weight_rows(S.tensor_key(151, i, S.TENSOR_W), 0, sh.n_out, sh.k_in, device=dev)
        c, s, z = P.fq_quantize_layer(wi, int(b))
        fq.fq_pack_layer(i, c, s, z, int(b), P.FQ_FMT_PACKED)
    xs = [S.activations(S.tensor_key(151, i, S.TENSOR_X), 1, sh.k_in).to(dev)[0] for i, sh in enumerate(shapes)]
    ys = []
    for sh in shapes:
        buf, y = guarded(sh.n_out, torch.float16, dev)
        bufs.append(buf)
        ys.append(y)
    fq.fq_gemv_stack(list(range(L)), xs, ys, S.stack_phases(shapes), 1)
    for i, y in enumerate(ys):
        out[f"stack_{i}"] = y.clone()
    assert fq.fq_status() == 0
    # 3. the fused prefill kernel on two of its matrices, ragged token counts
    for i, m in ((0, 200), (6, 600)):
        sh = shapes[i]
        x = S.activations(S.tensor_key(151, 100 + i, S.TENSOR_X), m, sh.k_in, torch.bfloat16, device=dev)
        buf, y = guarded(m * sh.n_out, torch.bfloat16, dev)
        fq.fq_gemm(i, x, y.view(m, sh.n_out))
        bufs.append(buf)
        out[f"gemm_{i}"] = y.clone()
    assert fq.fq_status() == 0
    fq.fq_destroy()
    torch.cuda.synchronize()
    out["guards_intact"] = torch.tensor([all(guards_intact(b) for b in bufs)])
    return {k: v.cpu() for k, v in out.items()}


if __name__ == "__main__":
    import paper_2501_07139_b200 as P
    assert os.path.basename(P.lib_path()) == "libflexq_checked.so", P.lib_path()
    torch.save(run_cases(P), sys.argv[1])
