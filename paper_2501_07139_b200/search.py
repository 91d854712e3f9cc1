"""Ensemble generation on a nested stack: builds the per-module tables with the prefill kernel and runs the
library's tree search (Sec. III-B, Algorithm 1) and pruning (Sec. III-C) on them.

The paper evaluates candidates by perplexity on a calibration set; without trained weights and datasets the
evaluation here is the relative output error of each linear layer on seeded calibration activations,
|| Y_b - Y_8 ||^2 / || Y_8 ||^2, summed over the layers of a module (and over modules for a configuration).
The library does the heavy work: fq_gemm for the outputs, fq_sqdiff for the two fp64 sums of every comparison,
fq_code_bytes for the sizes, fq_search_chain / fq_prune_chain for the search.  This module only divides each pair
of sums and adds the per-layer ratios and sizes up per module (a few hundred host operations)."""
from __future__ import annotations

from typing import Dict, List, Sequence

import torch

from . import flexq as F


def module_tables(fq: "F.FlexQ", shapes: Sequence, modules: Sequence[Sequence[int]], levels: Sequence[int],
                  calib: Dict[int, torch.Tensor], sens_tokens: int):
    """cost, sens, foot tables [module][level] of a stack whose layers are nested (8-bit parents).

    shapes[i] has n_out / k_in; modules[j] lists the layers of module j; levels are bit-widths from n_up down
    to n_low; calib[k_in] is a bf16 [tokens][k_in] activation matrix.  cost uses every token, sens only the
    first `sens_tokens` (the cheaper, pre-generated analysis of Sec. III-B)."""
    L = len(shapes)
    n_lev = len(levels)
    err = [[None] * n_lev for _ in range(L)]
    err_s = [[None] * n_lev for _ in range(L)]
    cur = [int(levels[0])] * L
    fq.fq_set_config(cur)
    for i, sh in enumerate(shapes):
        x = calib[sh.k_in]
        y_up = torch.empty((x.shape[0], sh.n_out), dtype=torch.bfloat16, device=x.device)
        y = torch.empty_like(y_up)
        fq.fq_gemm(i, x, y_up)
        for li, b in enumerate(levels):
            if li == 0:
                err[i][0] = err_s[i][0] = torch.zeros(2, dtype=torch.float64, device=x.device)
                continue
            cur[i] = int(b)
            fq.fq_set_config(cur)
            fq.fq_gemm(i, x, y)
            err[i][li] = F.fq_sqdiff(y, y_up)
            err_s[i][li] = F.fq_sqdiff(y[:sens_tokens].contiguous(), y_up[:sens_tokens].contiguous())
        cur[i] = int(levels[0])
        fq.fq_set_config(cur)
    torch.cuda.synchronize()

    def rel(t):
        d2, b2 = (float(v) for v in t.cpu())
        return d2 / b2 if b2 > 0 else 0.0

    cost = [[sum(rel(err[i][li]) for i in mod) for li in range(n_lev)] for mod in modules]
    sens = [[sum(rel(err_s[i][li]) for i in mod) for li in range(n_lev)] for mod in modules]
    foot = [[sum(F.fq_code_bytes(shapes[i].n_out, shapes[i].k_in, int(b)) for i in mod) for b in levels] for mod in modules]
    return cost, sens, foot


def chain_to_bits(chain: List[List[int]], modules: Sequence[Sequence[int]], levels: Sequence[int], n_layers: int):
    """Per-layer bit vectors (what fq_set_config / fq_transition take) of a chain of module-level states."""
    out = []
    for st in chain:
        bits = [0] * n_layers
        for m, l in enumerate(st):
            for i in modules[m]:
                bits[i] = int(levels[l])
        out.append(bits)
    return out


def generate_ensemble(fq, shapes, modules, levels, calib, stems: int = 2, branches: int = 3, sens_tokens: int = 32,
                      prune_fraction: float = 0.0):
    cost, sens, foot = module_tables(fq, shapes, modules, levels, calib, sens_tokens)
    chain, curve = F.fq_search_chain(cost, sens, foot, stems, branches)
    pruned, dropped, before, after = F.fq_prune_chain(chain, len(levels), foot, prune_fraction)
    return {"cost": cost, "sens": sens, "foot": foot, "chain": chain, "curve": curve, "pruned_chain": pruned,
            "dropped": dropped, "storage_before": before, "storage_after": after}
