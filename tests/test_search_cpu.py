"""Tree search (Sec. III-B, Algorithm 1) and pruning (Sec. III-C): the oracle against closed forms and brute
force, and the library's host implementation against the oracle (index work: bit-exact).  No GPU needed."""
import itertools

import numpy as np
import pytest

from oracle import fq_search as OS


def _tables(seed, n_mod, n_lev, integer=False):
    rng = np.random.default_rng(seed)
    inc = rng.integers(1, 6, (n_mod, n_lev - 1)).astype(float) if integer else rng.uniform(0.1, 1.0, (n_mod, n_lev - 1))
    cost = np.concatenate([np.zeros((n_mod, 1)), np.cumsum(inc, axis=1)], axis=1)      # grows as precision drops
    sens = cost * rng.uniform(0.5, 1.5, cost.shape) if not integer else cost.copy()
    size = rng.integers(1, 5, (n_mod, 1)) * 1000
    foot = (size * np.linspace(8, 3, n_lev)[None, :]).astype(np.uint64)
    return cost, sens, foot


def _check_chain(chain, n_mod, n_lev):
    assert len(chain) == n_mod * (n_lev - 1) + 1
    assert chain[0] == [0] * n_mod and chain[-1] == [n_lev - 1] * n_mod
    for a, b in zip(chain, chain[1:]):
        d = [y - x for x, y in zip(a, b)]
        assert sorted(d) == [0] * (n_mod - 1) + [1]            # one module, one level, never back up


# ---------------------------------------------------------------------------------------- oracle pins
def test_oracle_two_level_search_is_the_sorted_order():
    # with two stored models a chain is an order in which modules drop; the sum over the chain is
    # sum_m c_m * (number of configurations after the drop), minimal when the cheapest drop first
    cost, sens, foot = _tables(1, 7, 2)
    chain, curve = OS.search_chain(cost, cost, foot, stems=1, branches=7)
    _check_chain(chain, 7, 2)
    order = [int(np.nonzero(np.array(b) - np.array(a))[0][0]) for a, b in zip(chain, chain[1:])]
    assert order == list(np.argsort(cost[:, 1], kind="stable"))
    c = np.sort(cost[:, 1])
    assert abs(curve - sum(c[i] * (7 - i) for i in range(7))) < 1e-12


def test_oracle_against_brute_force_and_greedy():
    for seed in range(6):
        cost, sens, foot = _tables(10 + seed, 3, 3)
        best = OS.brute_force_best_chain(cost, foot)
        for stems, branches in ((1, 3), (2, 3), (4, 2), (9, 3)):
            chain, curve = OS.search_chain(cost, sens, foot, stems, branches)
            _check_chain(chain, 3, 3)
            assert curve >= best - 1e-12                       # no chain beats the exhaustive optimum
            assert abs(curve - sum(sum(cost[m][l] for m, l in enumerate(s)) for s in chain)) < 1e-9
        # one stem, no filtering: every step takes the cheapest successor (written out independently)
        chain, _ = OS.search_chain(cost, sens, foot, 1, 3)
        st = [0, 0, 0]
        for nxt in chain[1:]:
            opts = []
            for m in range(3):
                if st[m] < 2:
                    t = list(st); t[m] += 1
                    opts.append((sum(cost[i][t[i]] for i in range(3)), sum(int(foot[i][t[i]]) for i in range(3)), m, t))
            st = min(opts)[3]
            assert nxt == st


def test_oracle_one_branch_follows_the_sensitivity_table():
    cost, sens, foot = _tables(3, 5, 3)
    chain, _ = OS.search_chain(cost, sens, foot, stems=3, branches=1)
    st = [0] * 5
    for nxt in chain[1:]:
        m = min((m for m in range(5) if st[m] < 2), key=lambda m: (sens[m][st[m] + 1], m))
        st[m] += 1
        assert nxt == st


def test_oracle_pruning_hand_case():
    # 2 modules, levels (8, 5, 3): module 0 sits at the mid level in 3 configurations, module 1 in 1
    chain = [[0, 0], [1, 0], [1, 1], [1, 2], [2, 2]]
    foot = [[800, 500, 300], [80, 50, 30]]
    pruned, dropped, before, after = OS.prune_chain(chain, 3, foot, 0.5)
    assert dropped == {(1, 1)} and before == 1760 and after == 1710
    assert pruned == [[0, 0], [1, 0], [1, 2], [1, 2], [2, 2]]
    assert OS.prune_chain(chain, 3, foot, 0.0)[0] == chain
    allp, d, _, a = OS.prune_chain(chain, 3, foot, 1.0)
    assert d == {(0, 1), (1, 1)} and a == 1760 - 550 and all(l in (0, 2) for st in allp for l in st)
    # equal use: the one used at the larger footprints (earlier in the chain) goes first
    chain2 = [[0, 0], [1, 0], [2, 0], [2, 1], [2, 2]]
    assert OS.prune_chain(chain2, 3, foot, 0.5)[1] == {(0, 1)}


# ---------------------------------------------------------------------------------------- library vs oracle
@pytest.mark.parametrize("integer", [False, True])
def test_native_search_and_pruning_match_oracle(integer):
    import paper_2501_07139_b200 as P
    for seed, (n_mod, n_lev) in enumerate([(3, 2), (4, 3), (6, 4), (8, 3), (16, 3)]):
        cost, sens, foot = _tables(40 + seed, n_mod, n_lev, integer)
        for stems, branches in ((1, 1), (1, n_mod), (2, 3), (4, 2), (8, 5)):
            ref_chain, ref_curve = OS.search_chain(cost, sens, foot, stems, branches)
            chain, curve = P.fq_search_chain(cost, sens, foot, stems, branches)
            assert chain == ref_chain and curve == ref_curve, (seed, stems, branches)
            for frac in (0.0, 0.25, 0.5, 0.75, 1.0):
                rp, rd, rb, ra = OS.prune_chain(ref_chain, n_lev, foot, frac)
                p, d, b, a = P.fq_prune_chain(chain, n_lev, foot, frac)
                assert (p, d, b, a) == (rp, rd, rb, ra), (seed, frac)
                assert all(y >= x for s0, s1 in zip(p, p[1:]) for x, y in zip(s0, s1))    # still one-way
    with pytest.raises(P.FlexQError):
        P.fq_search_chain(np.zeros((2, 1)), np.zeros((2, 1)), np.zeros((2, 1), np.uint64), 1, 1)
