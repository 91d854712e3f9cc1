"""CPU oracle of the offline side: tree search for an ensemble of elastic configurations (Sec. III-B,
Algorithm 1) and pruning of mid-precision modules (Sec. III-C), on per-module tables.

Test infrastructure only: plain Python, slow, written from the paper's description.  Tables are
[module][level] with level 0 = n_up and the last level = n_low."""
from __future__ import annotations

from typing import List, Sequence, Tuple


def evaluate(state: Sequence[int], cost) -> float:
    """calibrationEval stand-in: the sum of the per-module terms, in module order."""
    c = 0.0
    for m, l in enumerate(state):
        c += float(cost[m][l])
    return c


def curve(chain, cost) -> float:
    """Sum of the evaluation over the configurations of a chain, added one by one in chain order (the
    built-in sum() compensates rounding since Python 3.12, a plain loop does not)."""
    c = 0.0
    for st in chain:
        c += evaluate(st, cost)
    return c


def footprint(state: Sequence[int], foot) -> int:
    return sum(int(foot[m][l]) for m, l in enumerate(state))


def search_chain(cost, sens, foot, stems: int, branches: int) -> Tuple[List[List[int]], float]:
    """Algorithm 1.  Returns (chain of configurations, sum of the evaluation over the chain)."""
    n_mod, n_lev = len(cost), len(cost[0])
    ensembles = [[[0] * n_mod]]                                   # list([QM(n_up)])
    low = [n_lev - 1] * n_mod
    while ensembles[0][-1] != low:                                # every stem advances one step per iteration
        pool = []
        for si, ens in enumerate(ensembles):
            last = ens[-1]
            # candidateGenerator: lower one module to its next lower precision (one-way)
            cands = [m for m in range(n_mod) if last[m] + 1 < n_lev]
            # analysisFilter: the #branch candidates with the smallest pre-generated sensitivity
            cands = sorted(cands, key=lambda m: float(sens[m][last[m] + 1]))[:branches]
            for m in cands:
                nxt = list(last)
                nxt[m] += 1
                pool.append((evaluate(nxt, cost), footprint(nxt, foot), si, nxt))   # calibrationEval
        pool.sort(key=lambda t: (t[0], t[1]))                     # rank (stable: generation order breaks ties)
        new = []
        for _, _, si, nxt in pool:
            if len(new) == stems:
                break
            if any(e[-1] == nxt for e in new):
                continue
            new.append(ensembles[si] + [nxt])
        ensembles = new
    best = min(range(len(ensembles)), key=lambda i: (curve(ensembles[i], cost), i))
    return ensembles[best], curve(ensembles[best], cost)


def prune_chain(chain, n_levels: int, foot, fraction: float):
    """Sec. III-C.  Returns (pruned chain, dropped (module, level) pairs, storage before, storage after)."""
    n_mod = len(chain[0])
    items = []
    for m in range(n_mod):
        for l in range(1, n_levels - 1):                          # modules of the mid-precision models only
            uses = [t for t, st in enumerate(chain) if st[m] == l]
            items.append((len(uses), sum(uses), m, l))            # usage, then usage at lower footprints
    items.sort(key=lambda t: (t[0], t[1]))                        # least important first (stable)
    n_drop = int(fraction * len(items) + 1e-9)
    dropped = {(m, l) for _, _, m, l in items[:n_drop]}
    before = sum(int(foot[m][l]) for m in range(n_mod) for l in range(n_levels))
    after = before - sum(int(foot[m][l]) for m, l in dropped)
    pruned = []
    for st in chain:
        row = []
        for m, l in enumerate(st):
            while (m, l) in dropped:
                l += 1
            row.append(l)
        pruned.append(row)
    return pruned, dropped, before, after


def brute_force_best_chain(cost, foot):
    """Every one-way chain of a tiny problem (exponential): the smallest sum of the evaluation over a chain."""
    n_mod, n_lev = len(cost), len(cost[0])
    low = tuple([n_lev - 1] * n_mod)
    from functools import lru_cache

    @lru_cache(maxsize=None)
    def best_from(state):
        here = evaluate(state, cost)
        if state == low:
            return here
        opts = []
        for m in range(n_mod):
            if state[m] + 1 < n_lev:
                nxt = list(state)
                nxt[m] += 1
                opts.append(best_from(tuple(nxt)))
        return here + min(opts)

    return best_from(tuple([0] * n_mod))
