#!/usr/bin/env python
"""Benchmark of the elastic mixed-bit decode path on B200.

One "step" is one pass of the hot path over the Llama-2-7B-shaped layer stack: a batch-1
fp16 activation vector goes through all 224 packed mixed-bit matrices (bits per matrix drawn
from {3,4,5,6,8}, group 128) in ONE persistent fq_gemv_stack launch that honours the
dependency order {q,k,v} -> o -> {gate,up} -> down -> next block.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--blocks B]

Prints one JSON line (rank 0).  N > 1 runs N independent replicas (the path does not shard).
`--impl reference` times the CPU oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import fq_synth as S

METRIC = "mixed-bit dequant-GEMV weight GB/s"
UNIT = "GB/s"
CONFIG_ID = 1                      # the 7B decode stack
BIT_CHOICES = [3, 4, 5, 6, 8]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


def read_ncu_traffic(footprint_bytes):
    """DRAM bytes per stack launch derived from the committed ncu capture of a small case
    (traffic / algorithmic bytes there, times this launch's algorithmic bytes).  None when the
    kernel source changed after the counters were taken."""
    import hashlib
    try:
        with open(os.path.join(ROOT, "profiles", "gemv_stack_traffic.json")) as f:
            d = json.load(f)
        h = hashlib.sha256()
        for name in ("fq_gemv1.cu", "fq_gemv_core.cuh"):                 # the batch-1 decode kernel and its arithmetic
            with open(os.path.join(ROOT, "paper_2501_07139_b200", "csrc", name), "rb") as f:
                h.update(f.read())
        sha = h.hexdigest()
        if sha != d["source_sha256"]:
            return None, "kernel changed since the ncu capture"
        return d["ratio"] * footprint_bytes, d["note"]
    except Exception:
        return None, "no ncu capture recorded"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        n_inside = len(self.rows)                      # samples that arrived while the timed region ran
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows[:max(n_inside, 1)]:
            p = [c.strip() for c in r.split(",")]
            if len(p) < 6:
                continue
            try:
                sm.append(float(p[0])); mx.append(float(p[1]))
            except ValueError:
                continue
            for n, v in zip(names, p[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(value: float, device) -> float:
    """The slowest rank's figure (replicas are timed together: barrier, events, max over ranks)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def build_stack(P, shapes, bits, device):
    """Seeded weights -> GPU quantiser -> packed layers.  Returns the context."""
    fq = P.FlexQ(len(shapes), device.index or 0)
    for i, (sh, b) in enumerate(zip(shapes, bits)):
        w = S.weight_rows(S.tensor_key(CONFIG_ID, i, S.TENSOR_W), 0, sh.n_out, sh.k_in, device=device)
        c, s, z = P.fq_quantize_layer(w, int(b))
        fq.fq_pack_layer(i, c, s, z, int(b), P.FQ_FMT_PACKED)
        del w, c, s, z
    torch.cuda.synchronize()
    return fq


PREFILL_CONFIG_ID = 3
PREFILL_BITS = [2, 3, 4, 6, 8]
PREFILL_TOKENS = 4 * 2048


def prefill_pass(P, device, blocks, steps, warmup, tokens=PREFILL_TOKENS):
    """Prefill / calibration-evaluation workload: bf16 activations of 4 x 2048 tokens through every matrix
    of the 7B-shaped stack (bits seeded from {2,3,4,6,8}), one fq_gemm call per matrix.  Returns a dict."""
    shapes = S.stack_shapes("7b", blocks)
    L = len(shapes)
    bits = S.draw_bits(S.tensor_key(PREFILL_CONFIG_ID, 0, S.TENSOR_BITS), L, PREFILL_BITS)
    fq = P.FlexQ(L, device.index or 0)
    for i, (sh, b) in enumerate(zip(shapes, bits)):
        w = S.weight_rows(S.tensor_key(PREFILL_CONFIG_ID, i, S.TENSOR_W), 0, sh.n_out, sh.k_in, device=device)
        c, sc, z = P.fq_quantize_layer(w, int(b))
        fq.fq_pack_layer(i, c, sc, z, int(b), P.FQ_FMT_PACKED)
        del w, c, sc, z
    m = tokens
    xs = {k: S.activations(S.tensor_key(PREFILL_CONFIG_ID, k, S.TENSOR_X), m, k, torch.bfloat16, device=device)
          for k in sorted({sh.k_in for sh in shapes})}
    ys = {n: torch.empty((m, n), dtype=torch.bfloat16, device=device) for n in sorted({sh.n_out for sh in shapes})}

    def one_pass():
        for i, sh in enumerate(shapes):
            fq.fq_gemm(i, xs[sh.k_in], ys[sh.n_out])

    def one_pass_two():                             # the comparison point: dequantise to bf16, then a plain tcgen05 GEMM
        for i, sh in enumerate(shapes):
            fq.fq_gemm_two_pass(i, xs[sh.k_in], ys[sh.n_out])

    def timed(fn):
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    ms = timed(one_pass)
    ms_two = timed(one_pass_two)
    status = fq.fq_status()
    fq.fq_destroy()
    if status != 0:
        raise RuntimeError(f"device status {status} after the prefill pass")
    flop = sum(2.0 * m * sh.n_out * sh.k_in for sh in shapes)
    return {"ms_per_pass": ms, "tflops": flop / (ms * 1e-3) / 1e12, "flop_per_pass": flop, "tokens": m,
            "matrices": L, "average_bits": S.average_bits(bits, shapes), "gpu_launches_per_pass": L,
            "two_pass": {"ms_per_pass": ms_two, "tflops": flop / (ms_two * 1e-3) / 1e12, "gpu_launches_per_pass": 2 * L}}


def _time_ms(fn, steps, warmup=3):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def config_report(P, device, steps, brief=False):
    """The other workloads of the problem statement, one JSON object each (printed by --all-configs):
    config 0 (one 4096x4096 4-bit layer, rotated over copies larger than L2), config 2 (7B-shaped nested
    stack, 12-configuration chain) and config 4 (13B-shaped nested stack, 16 configurations, batch 1 / 8
    decode and prefill at 2048 tokens).  brief: only the first, a middle and the last configuration of each
    chain and no ensemble search -- what the default bench line carries in its `configs` object."""
    peaks, kind = measured_peaks()
    out = []
    # ---- config 0
    n = k = 4096
    copies = 32                                           # 32 x 8.9 MB = 285 MB > 126 MB L2
    fq = P.FlexQ(copies, device.index or 0)
    w = S.weight_rows(S.tensor_key(0, 0, S.TENSOR_W), 0, n, k, device=device)
    c, sc, z = P.fq_quantize_layer(w, 4)
    for i in range(copies):
        fq.fq_pack_layer(i, c, sc, z, 4, P.FQ_FMT_PACKED)
    x = S.activations(S.tensor_key(0, 0, S.TENSOR_X), 1, k).to(device)
    ys = [torch.empty(n, dtype=torch.float16, device=device) for _ in range(copies)]
    fp1 = fq.fq_set_config([4] * copies) // copies

    def per_layer():
        for i in range(copies):
            fq.fq_gemv(i, x, ys[i])
    args = fq.stack_args(list(range(copies)), [x] * copies, ys, None)
    t_call = _time_ms(per_layer, steps) / copies
    t_stack = _time_ms(lambda: fq.fq_gemv_stack_raw(args, 1), steps) / copies
    out.append({"config": 0, "workload": "4096x4096 4-bit g=128 GEMV, rotated over 32 stored copies (cold L2)",
                "footprint_bytes": fp1, "us_per_layer_separate_calls": t_call * 1e3, "us_per_layer_one_launch": t_stack * 1e3,
                "GBps_separate_calls": fp1 / t_call / 1e6, "GBps_one_launch": fp1 / t_stack / 1e6,
                "frac_of_measured_hbm_one_launch": fp1 / t_stack / 1e6 / peaks["hbm_gbs"]})
    fq.fq_destroy()
    del fq, ys
    # ---- configs 2 and 4: nested stacks and their chains
    for cfg, model, n_cfg, hi, lo, floor in ((2, "7b", 12, 7.0, 3.5, 3), (4, "13b", 16, 6.0, 2.5, 2)):
        shapes = S.stack_shapes(model)
        L = len(shapes)
        fq = P.FlexQ(L, device.index or 0)
        stores = []
        for i, sh in enumerate(shapes):
            w = S.weight_rows(S.tensor_key(cfg, i, S.TENSOR_W), 0, sh.n_out, sh.k_in, device=device)
            c, sc, z = P.fq_quantize_layer(w, 8)
            stores.append(fq.fq_pack_layer(i, c, sc, z, 8, P.FQ_FMT_PLANES))
            del w, c, sc, z
        chain = S.config_chain(S.tensor_key(cfg, 0, S.TENSOR_CHAIN), shapes, n_cfg, hi, lo, floor)
        phases = S.stack_phases(shapes)
        rows = []
        steps_freed, steps_loaded = [], []
        for batch in ((1,) if cfg == 2 else (1, 8)):
            xs = [S.activations(S.tensor_key(cfg, i, S.TENSOR_X), batch, sh.k_in).to(device) for i, sh in enumerate(shapes)]
            ys = [torch.empty((batch, sh.n_out), dtype=torch.float16, device=device) for sh in shapes]
            args_dep = fq.stack_args(list(range(L)), xs, ys, phases)
            args_free = fq.stack_args(list(range(L)), xs, ys, None)
            for ci, bits in enumerate(chain):
                if brief and ci not in ((0, n_cfg // 2 - 1, n_cfg - 1) if cfg == 2 else (0, n_cfg - 1)):
                    continue
                t0 = time.perf_counter()
                if ci == 0 or batch != 1 or brief:
                    fp = fq.fq_set_config([int(b) for b in bits])
                else:                                            # the chain is one-way: every step is a transition
                    rep = fq.fq_transition([int(b) for b in bits], require_one_way=True)
                    fp = rep["footprint_to"]
                    steps_freed.append(rep["bytes_freed"]); steps_loaded.append(rep["bytes_loaded"])
                switch_us = (time.perf_counter() - t0) * 1e6
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); fq.fq_gemv_stack_raw(args_dep, batch); e1.record(); torch.cuda.synchronize()
                first_ms = e0.elapsed_time(e1)                     # first pass after the switch (table rebuilt)
                ms = _time_ms(lambda: fq.fq_gemv_stack_raw(args_dep, batch), steps)
                ms_free = _time_ms(lambda: fq.fq_gemv_stack_raw(args_free, batch), steps)
                rows.append({"batch": batch, "config_index": ci, "average_bits": S.average_bits(bits, shapes),
                             "footprint_bytes": fp, "set_config_host_us": switch_us, "first_pass_ms": first_ms,
                             "ms_per_pass": ms, "GBps": fp / ms / 1e6, "frac": fp / ms / 1e6 / peaks["hbm_gbs"],
                             "ms_unordered": ms_free, "GBps_unordered": fp / ms_free / 1e6})
            del xs, ys
        entry = {"config": cfg, "workload": f"{model}-shaped stack, nested format (one 8-bit parent per layer), {n_cfg}-configuration chain",
                 "storage_bytes": fq.fq_storage_bytes(), "weight_bytes_moved_by_switches": 0, "decode": rows}
        if steps_freed:
            entry["transitions"] = {"steps": len(steps_freed), "one_way": True, "bytes_loaded_total": int(sum(steps_loaded)),
                                    "granularity_bytes_max": int(max(steps_freed)), "granularity_bytes_mean": float(np.mean(steps_freed)),
                                    "note": "fq_transition per chain step: memory a deployment can release; nothing has to be loaded"}
        if cfg == 2 and not brief:
            # the offline side on the same stack: tables measured with the prefill kernel, tree search, pruning
            from paper_2501_07139_b200 import search as SR
            levels = [8, 5, 3]
            mods = {}
            for i, sh in enumerate(shapes):
                mods.setdefault((sh.block, sh.module), []).append(i)
            modules = [mods[k] for k in sorted(mods)]
            calib = {kk: S.activations(S.tensor_key(cfg, kk, S.TENSOR_X), 2048, kk, torch.bfloat16, device=device)
                     for kk in sorted({sh.k_in for sh in shapes})}
            torch.cuda.synchronize(); t0 = time.perf_counter()
            cost, sens, foot = SR.module_tables(fq, shapes, modules, levels, calib, 256)
            t_tab = time.perf_counter() - t0
            t0 = time.perf_counter()
            ens, curve = P.fq_search_chain(cost, sens, foot, 2, 3)
            t_search = time.perf_counter() - t0
            pruned, dropped, before, after = P.fq_prune_chain(ens, len(levels), foot, 0.5)
            fps = [sum(foot[m][l] for m, l in enumerate(st)) for st in ens]
            entry["ensemble_search"] = {
                "modules": len(modules), "levels_bits": levels, "stems": 2, "branches": 3, "calibration_tokens": 2048,
                "evaluation": "relative output error of the linear layers (stand-in for calibration perplexity)",
                "table_seconds_gpu": t_tab, "table_fq_gemm_calls": len(shapes) * len(levels), "search_seconds_host": t_search,
                "configurations": len(ens), "curve_cost": curve,
                "granularity_bytes_max": int(max(a - b for a, b in zip(fps, fps[1:]))),
                "code_bytes_first_last": [int(fps[0]), int(fps[-1])],
                "pruning_50pct": {"dropped_mid_modules": len(dropped), "storage_code_bytes_before": before,
                                  "storage_code_bytes_after": after}}
            del calib
        if cfg == 4:
            bits = chain[-1]
            fq.fq_set_config([int(b) for b in bits])
            m = 2048
            xb = {kk: S.activations(S.tensor_key(cfg, kk, S.TENSOR_X), m, kk, torch.bfloat16, device=device)
                  for kk in sorted({sh.k_in for sh in shapes})}
            yb = {nn: torch.empty((m, nn), dtype=torch.bfloat16, device=device) for nn in sorted({sh.n_out for sh in shapes})}

            def pf():
                for i, sh in enumerate(shapes):
                    fq.fq_gemm(i, xb[sh.k_in], yb[sh.n_out])
            def pf_two():
                for i, sh in enumerate(shapes):
                    fq.fq_gemm_two_pass(i, xb[sh.k_in], yb[sh.n_out])
            ms = _time_ms(pf, max(1, steps // 4), 2)
            ms_two = _time_ms(pf_two, max(1, steps // 4), 2)
            flop = sum(2.0 * m * sh.n_out * sh.k_in for sh in shapes)
            entry["prefill"] = {"tokens": m, "average_bits": S.average_bits(bits, shapes), "ms_per_pass": ms,
                                "tflops": flop / ms / 1e9, "frac_of_measured_sustained_bf16": flop / ms / 1e9 / peaks["bf16_tflops_sustained"],
                                "two_pass": {"ms_per_pass": ms_two, "tflops": flop / ms_two / 1e9}}
        if fq.fq_status() != 0:
            raise RuntimeError("device status after config report")
        out.append(entry)
        fq.fq_destroy()
        del fq, stores
        torch.cuda.empty_cache()
    return out


def oracle_inputs(shapes, bits, n_layers, device_for_gen):
    """Quantised matrices and activations of the first `n_layers` matrices of the workload, as the CPU oracle takes them."""
    from oracle import fq_oracle as O
    O.build()
    items = []
    for i in range(n_layers):
        sh, b = shapes[i], int(bits[i])
        w = S.weight_rows(S.tensor_key(CONFIG_ID, i, S.TENSOR_W), 0, sh.n_out, sh.k_in, device=device_for_gen)
        codes, sc, zr = O.quantize(w.cpu().numpy(), b)
        x = S.activations(S.tensor_key(CONFIG_ID, i, S.TENSOR_X), 1, sh.k_in, torch.float16)
        xb = x.view(torch.int16).numpy().view(np.uint16)
        items.append((codes, sc, zr, b, xb, sh.n_out * sh.k_in * b // 8 + sh.n_out * (sh.k_in // 128) * 4))
    return items


def oracle_pass(items):
    """One timed pass of the CPU oracle's GEMV over `items`.  Returns (bytes processed, seconds)."""
    from oracle import fq_oracle as O
    total_bytes, total_s = 0, 0.0
    for codes, sc, zr, b, xb, nbytes in items:
        t0 = time.perf_counter()
        O.gemv(codes, sc, zr, b, xb)
        total_s += time.perf_counter() - t0
        total_bytes += nbytes
    return total_bytes, total_s


def oracle_pass_threads(items, threads):
    """The same pass with the rows of every matrix dealt to `threads` host threads (the oracle's C routine is
    called once per row slice and releases the interpreter lock; the arithmetic of a row is unchanged)."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import fq_oracle as O
    total_bytes, total_s = 0, 0.0
    with ThreadPoolExecutor(max_workers=threads) as pool:
        for codes, sc, zr, b, xb, nbytes in items:
            n = codes.shape[0]
            cuts = [n * t // threads for t in range(threads + 1)]
            slices = [(codes[a:e], sc[a:e], zr[a:e]) for a, e in zip(cuts, cuts[1:]) if e > a]
            t0 = time.perf_counter()
            list(pool.map(lambda p: O.gemv(p[0], p[1], p[2], b, xb), slices))
            total_s += time.perf_counter() - t0
            total_bytes += nbytes
    return total_bytes, total_s


def prefill_oracle_leg(shapes, bits, tokens, n_matrices, rows_per_matrix, device):
    """The CPU oracle's prefill GEMM on a bounded sample: `rows_per_matrix` sampled token rows of the first
    `n_matrices` matrices of the prefill stack (all output columns of those rows).  Returns (flop, seconds)."""
    from oracle import fq_oracle as O
    flop, secs = 0.0, 0.0
    for i in range(n_matrices):
        sh, b = shapes[i], int(bits[i])
        w = S.weight_rows(S.tensor_key(PREFILL_CONFIG_ID, i, S.TENSOR_W), 0, sh.n_out, sh.k_in).numpy()
        c, sc, z = O.quantize(w, b)
        x = S.activations(S.tensor_key(PREFILL_CONFIG_ID, sh.k_in, S.TENSOR_X), tokens, sh.k_in, torch.bfloat16, device=device)
        rows = S.sample_rows(PREFILL_CONFIG_ID * 1000 + i, tokens, rows_per_matrix)[:rows_per_matrix]
        xb = np.ascontiguousarray(x[torch.from_numpy(rows).to(device)].cpu().view(torch.int16).numpy().view(np.uint16))
        del x
        t0 = time.perf_counter()
        O.gemm(c, sc, z, b, xb)
        secs += time.perf_counter() - t0
        flop += 2.0 * len(rows) * sh.n_out * sh.k_in
    return flop, secs


def transition_leg(P, device, blocks=4, high=8, low=4):
    """Swap-model transitions (Sec. II-C) on `blocks` decoder blocks of the 7B-shaped stack: every matrix has a
    `high`- and a `low`-bit variant in page-locked host memory; after loading the all-`high` configuration, each
    step lowers the seven matrices of one block (one module of the chain) with fq_transition_swap: the `low`
    variants are copied in, then the `high` ones released.  Timed per step with CUDA events."""
    shapes = S.stack_shapes("7b", blocks)
    L = len(shapes)
    tmp = P.FlexQ(L, device.index or 0)
    fq = P.FlexQ(L, device.index or 0)
    for i, sh in enumerate(shapes):
        w = S.weight_rows(S.tensor_key(CONFIG_ID, i, S.TENSOR_W), 0, sh.n_out, sh.k_in, device=device)
        for b in (high, low):
            c, sc, z = P.fq_quantize_layer(w, b)
            store = tmp.fq_pack_layer(i, c, sc, z, b, P.FQ_FMT_PACKED)
            fq.fq_host_variant(i, sh.n_out, sh.k_in, b, store.cpu().pin_memory())
        del w, c, sc, z
    tmp.fq_destroy()
    torch.cuda.empty_cache()
    cfg = [high] * L
    rep0 = fq.fq_transition_swap(cfg)
    torch.cuda.synchronize()
    steps = []
    for blk in range(blocks):
        for i in range(7 * blk, 7 * blk + 7):
            cfg[i] = low
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        rep = fq.fq_transition_swap(cfg)
        e1.record()
        torch.cuda.synchronize()
        steps.append((e0.elapsed_time(e1), rep))
    status = fq.fq_status()
    fq.fq_destroy()
    if status != 0:
        raise RuntimeError(f"device status {status} after the transition leg")
    ms = sorted(t for t, _ in steps)[len(steps) // 2]
    rep = steps[-1][1]
    return {"workload": f"{blocks} blocks of the 7B-shaped stack, packed variants of {high} and {low} bits in page-locked host "
                        f"memory; each step lowers one block's seven matrices {high} -> {low} (fq_transition_swap)",
            "initial_load_bytes": rep0["bytes_loaded"], "steps": len(steps), "ms_per_step_median": ms,
            "bytes_loaded_per_step": rep["bytes_loaded"], "bytes_freed_per_step": rep["bytes_freed"],
            "peak_extra_bytes": rep["peak_extra_bytes"],
            "granularity_bytes": rep["footprint_from"] - rep["footprint_to"],
            "h2d_gbs": rep["bytes_loaded"] / (ms * 1e-3) / 1e9}


def oracle_desc(n_layers):
    return f"oracle GEMV over the first {n_layers} matrices of the stack ({n_layers / 7:.2g} blocks), single thread"


REF_BUDGET_S = 150.0          # CPU seconds the whole reference run may take, over all its steps


def run_reference(args, rank):
    if rank != 0:
        return
    shapes = S.stack_shapes("7b", args.blocks)
    bits = S.draw_bits(S.tensor_key(CONFIG_ID, 0, S.TENSOR_BITS), len(shapes), BIT_CHOICES)
    gen_dev = "cuda" if torch.cuda.is_available() else "cpu"
    items = oracle_inputs(shapes, bits, min(args.ref_layers, len(shapes)), gen_dev)
    # bound the run: one untimed pass gives each matrix's cost, a step is the longest prefix of the sample
    # that keeps (warmup + steps) passes inside the budget
    per = [oracle_pass([it])[1] for it in items]
    n_layers, acc = 0, 0.0
    for t in per:
        if n_layers >= 1 and (acc + t) * (args.warmup + args.steps) > REF_BUDGET_S:
            break
        acc += t; n_layers += 1
    items = items[:n_layers]
    desc = oracle_desc(n_layers)
    if n_layers == 1 and per[0] * (args.warmup + args.steps) > REF_BUDGET_S:
        # even one matrix per step would pass the budget: a step is the first rows of the first matrix
        codes, sc, zr, b, xb, nbytes = items[0]
        n = codes.shape[0]
        rows = int(max(32, min(n, n * REF_BUDGET_S / (per[0] * (args.warmup + args.steps)))))
        items = [(codes[:rows], sc[:rows], zr[:rows], b, xb, nbytes * rows // n)]
        desc = f"oracle GEMV over the first {rows} of {n} output rows of the first matrix of the stack, single thread"
    times, byts = [], 0
    for step in range(args.warmup + args.steps):
        byts, secs = oracle_pass(items)
        if step >= args.warmup:
            times.append(secs)
    t = float(np.mean(times))
    val = byts / t / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"llama2-7b-shaped decode stack, {len(shapes)} matrices, bits {BIT_CHOICES}, g=128, batch 1",
                   "sample": desc},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="default 400 (20 for --impl reference)")
    ap.add_argument("--warmup", type=int, default=None, help="default 10 (1 for --impl reference)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--blocks", type=int, default=32, help="decoder blocks of the 7B-shaped stack (32 = full)")
    ap.add_argument("--ref-layers", type=int, default=7,
                    help="--impl reference: matrices per step at most (fewer when warmup + steps would pass the time budget)")
    ap.add_argument("--cpu-layers", type=int, default=28, help="matrices the cpu_baseline leg times the CPU oracle on")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-prefill", action="store_true", help="skip the prefill (tensor-core GEMM) leg")
    ap.add_argument("--prefill-steps", type=int, default=3)
    ap.add_argument("--prefill-tokens", type=int, default=PREFILL_TOKENS)
    ap.add_argument("--prefill-only", action="store_true", help="run only the prefill leg and print its object")
    ap.add_argument("--no-transition", action="store_true", help="skip the swap-transition leg")
    ap.add_argument("--no-configs", action="store_true", help="leave the `configs` object (configs 0, 2, 4 in brief) out of the line")
    ap.add_argument("--all-configs", action="store_true",
                    help="instead of the bench line, print one JSON object per other workload (configs 0, 2, 4)")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 400 if args.impl == "ours" else 20
    if args.warmup is None:
        args.warmup = 10 if args.impl == "ours" else 1
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch.distributed as dist
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)

    import paper_2501_07139_b200 as P
    P.lib()                                      # fails loudly if the CUDA library is missing

    if args.all_configs:
        for obj in config_report(P, device, max(3, args.steps // 5)):
            print(json.dumps(obj), flush=True)
        return
    if args.prefill_only:
        pf = prefill_pass(P, device, args.blocks, args.prefill_steps, 3, args.prefill_tokens)
        print(json.dumps({"prefill_only": pf}), flush=True)
        return

    shapes = S.stack_shapes("7b", args.blocks)
    L = len(shapes)
    bits = S.draw_bits(S.tensor_key(CONFIG_ID, 0, S.TENSOR_BITS), L, BIT_CHOICES)
    phases = S.stack_phases(shapes)
    fq = build_stack(P, shapes, bits, device)
    footprint = fq.fq_set_config([int(b) for b in bits])

    # activations: one seeded fp16 vector per matrix; host copies are pinned for the end-to-end leg
    k_off = np.concatenate([[0], np.cumsum([s.k_in for s in shapes])])
    n_off = np.concatenate([[0], np.cumsum([s.n_out for s in shapes])])
    x_host = torch.empty(int(k_off[-1]), dtype=torch.float16).pin_memory()
    for i, sh in enumerate(shapes):
        x_host[k_off[i]:k_off[i + 1]] = S.activations(S.tensor_key(CONFIG_ID, i, S.TENSOR_X), 1, sh.k_in)[0]
    y_host = torch.empty(int(n_off[-1]), dtype=torch.float16).pin_memory()
    x_dev = x_host.to(device)
    y_dev = torch.zeros(int(n_off[-1]), dtype=torch.float16, device=device)
    xs = [x_dev[k_off[i]:k_off[i + 1]] for i in range(L)]
    ys = [y_dev[n_off[i]:n_off[i + 1]] for i in range(L)]
    layers = list(range(L))
    args_dep = fq.stack_args(layers, xs, ys, phases)
    args_free = fq.stack_args(layers, xs, ys, None)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1) / steps, device)

    def step_dev():
        fq.fq_gemv_stack_raw(args_dep, 1)

    def step_free():
        fq.fq_gemv_stack_raw(args_free, 1)

    def step_e2e():
        x_dev.copy_(x_host, non_blocking=True)
        fq.fq_gemv_stack_raw(args_dep, 1)
        y_host.copy_(y_dev, non_blocking=True)

    for _ in range(args.warmup):
        step_dev()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ms = timed(step_dev, args.steps)
    clocks = sampler.stop() if rank == 0 else None
    for _ in range(3):
        step_free()
    ms_free = timed(step_free, args.steps)
    for _ in range(3):
        step_e2e()
    ms_e2e = timed(step_e2e, args.steps)
    status = fq.fq_status()
    if status != 0:
        raise RuntimeError(f"device status {status} after the timed region")

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks, peak_kind = measured_peaks()
    # a second denominator: what a read-only pass over 4 GiB reaches on this GPU right now
    probe = torch.empty(1 << 30, dtype=torch.int32, device=device)
    for _ in range(2):
        fq.fq_stream_read(probe)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(5):
        fq.fq_stream_read(probe)
    e1.record()
    torch.cuda.synchronize()
    stream_gbs = 5 * probe.numel() * 4 / (e0.elapsed_time(e1) * 1e-3) / 1e9
    del probe
    gbs = footprint / (ms * 1e-3) / 1e9
    traffic, traffic_note = read_ncu_traffic(footprint)
    line = {
        "metric": METRIC, "value": gbs * world, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f16", "data": "synthetic",
        "config": {
            "workload": f"llama2-7b-shaped decode stack: {L} matrices ({args.blocks} blocks), per-matrix bits seeded from "
                        f"{BIT_CHOICES}, g=128, packed format, batch-1 fp16 GEMV, one persistent launch per pass, "
                        f"dependency phases honoured",
            "average_bits": S.average_bits(bits, shapes), "footprint_bytes": footprint,
            "l2": "each pass streams the whole stack (>> 126 MB L2), no flush needed",
            "replicas": world,
        },
        "e2e": {"value": footprint / (ms_e2e * 1e-3) / 1e9 * world, "unit": UNIT,
                "h2d_bytes_per_step": int(x_host.numel() * 2), "d2h_bytes_per_step": int(y_host.numel() * 2),
                "ms_per_step": ms_e2e},
        "gpu_launches": args.steps,
        "unordered": {"value": footprint / (ms_free * 1e-3) / 1e9 * world, "unit": UNIT, "ms_per_step": ms_free,
                      "note": "same pass without the dependency phases (every matrix independent)"},
        "roofline": {
            "bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": gbs / peaks["hbm_gbs"], "peak_kind": f"of {peak_kind}",
            "frac_of_nominal_8TBs": gbs / 8000.0,
            "kernel": "gemv1_kernel (one launch per pass; algorithmic bytes = footprint of the configuration)",
            "stream_read_gbs": stream_gbs, "frac_of_stream_read": gbs / stream_gbs,
            "traffic": traffic, "traffic_note": traffic_note,
        },
        "clocks": clocks,
    }
    fq.fq_destroy()
    del fq
    torch.cuda.empty_cache()
    if not args.no_prefill and world == 1:
        pf = prefill_pass(P, device, args.blocks, args.prefill_steps, 3, args.prefill_tokens)
        burst, sustained = peaks.get("bf16_tflops", 1590.0), peaks.get("bf16_tflops_sustained", 1400.0)
        line["prefill"] = {
            "metric": "prefill dequant-GEMM TFLOP/s", "value": pf["tflops"], "unit": "TFLOP/s", "ms_per_pass": pf["ms_per_pass"],
            "workload": f"bf16 activations {pf['tokens']} tokens through {pf['matrices']} matrices of the 7B-shaped stack, "
                        f"bits seeded from {PREFILL_BITS} (average {pf['average_bits']:.2f}), one fq_gemm (fused kernel) per matrix",
            "dtype": "bf16", "gpu_launches_per_pass": pf["gpu_launches_per_pass"],
            "roofline": {"bound": "tensor", "achieved": pf["tflops"], "peak": sustained, "unit": "TFLOP/s",
                         "frac": pf["tflops"] / sustained, "peak_kind": f"of {peak_kind} (sustained bf16, the pass is a long step)",
                         "frac_of_burst": pf["tflops"] / burst, "traffic": None,
                         "kernel": "gemm_fused_kernel (tcgen05; blobs dequantised inside); flops = 2*M*N*K per matrix"},
            "two_pass": dict(pf["two_pass"], note="comparison point: dequant_kernel + gemm_kernel (fq_gemm_two_pass)",
                             frac=pf["two_pass"]["tflops"] / sustained),
        }
    if not args.no_transition and world == 1:
        line["transition"] = transition_leg(P, device)
    if not args.no_configs and world == 1 and args.blocks == 32:
        line["configs"] = config_report(P, device, 5, brief=True)
    if not args.no_cpu_baseline:
        n_layers = min(args.cpu_layers, L)
        items = oracle_inputs(shapes, bits, n_layers, device)
        cores = len(os.sched_getaffinity(0))
        byts1, secs1 = oracle_pass(items[:min(7, n_layers)])
        byts, secs = oracle_pass_threads(items, cores)
        line["cpu_baseline"] = {"value": byts / secs / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": oracle_desc(n_layers).replace("single thread", f"rows of each matrix dealt to {cores} host threads"),
                                "single_thread": {"value": byts1 / secs1 / 1e9, "unit": UNIT, "cores": 1,
                                                  "sample": oracle_desc(min(7, n_layers))}}
        if "prefill" in line:
            pshapes = S.stack_shapes("7b", args.blocks)
            pbits = S.draw_bits(S.tensor_key(PREFILL_CONFIG_ID, 0, S.TENSOR_BITS), len(pshapes), PREFILL_BITS)
            pflop, psecs = prefill_oracle_leg(pshapes, pbits, args.prefill_tokens, min(7, len(pshapes)), 16, device)
            line["prefill"]["cpu_baseline"] = {
                "value": pflop / psecs / 1e12, "unit": "TFLOP/s", "cores": 1, "kind": "oracle",
                "sample": f"16 sampled token rows of each of the first {min(7, len(pshapes))} matrices, all output columns, "
                          f"CPU oracle (fp64), single thread",
                "full_pass_seconds_extrapolated": psecs / pflop * pf["flop_per_pass"]}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
