"""Verification-tree design and width choice (paper Sec. III-C): the oracle's plain greedy against brute
force, and the package's heap-based builder against the oracle.  CPU only (the module under test is
host-side logic; importing it does not load the CUDA library)."""
import importlib.util
import itertools
from pathlib import Path

import numpy as np
import pytest

import oracle
import workloads as wl

_spec = importlib.util.spec_from_file_location("arca", Path(__file__).resolve().parent.parent / "paper_2505_23219_b200" / "arca.py")
arca = importlib.util.module_from_spec(_spec)
_spec.loader.exec_module(arca)


def _all_prefix_closed_trees(acc, width):
    """Every tree of `width` nodes over the candidate tree: sets of rank paths closed under taking prefixes."""
    cands = [()]
    for l in range(len(acc)):
        cands += [p + (r,) for p in cands if len(p) == l for r in range(len(acc[l]))]
    cands = [c for c in cands if c]
    for pick in itertools.combinations(cands, width - 1):
        s = set(pick)
        if all(p[:-1] in s or len(p) == 1 for p in s):
            yield s


def _value(acc, paths):
    return 1.0 + sum(np.prod([acc[l][r] for l, r in enumerate(p)]) for p in paths)


@pytest.mark.parametrize("acc", [[[0.7, 0.2, 0.05], [0.5, 0.3], [0.4, 0.1]], [[0.9, 0.6], [0.8, 0.1, 0.05], [0.3]],
                                 [[0.3, 0.3, 0.2], [0.9, 0.2], [0.9]]])
def test_greedy_tree_maximises_the_expected_acceptance_length(acc):
    for width in range(1, 8):
        parent, prob = oracle.arca_tree(acc, width)
        best = max(_value(acc, t) for t in _all_prefix_closed_trees(acc, width))
        assert len(parent) == width and parent[0] == -1 and all(0 <= parent[i] < i for i in range(1, width))
        assert abs(oracle.expected_acceptance(prob) - best) < 1e-12


def test_width_one_gives_acceptance_length_one():
    parent, prob = oracle.arca_tree(arca.synthetic_accuracies(), 1)
    assert parent == [-1] and oracle.expected_acceptance(prob) == 1.0          # paper Table I, width 1


def test_expected_acceptance_is_the_sum_of_path_products():
    acc = [[0.5, 0.25], [0.5]]
    parent, prob = oracle.arca_tree(acc, 4)          # root, (0), (1), (0, 0): 1 + 0.5 + 0.25 + 0.25
    assert parent == [-1, 0, 0, 1] and abs(oracle.expected_acceptance(prob) - 2.0) < 1e-15


@pytest.mark.parametrize("seed", range(6))
def test_package_builder_equals_the_oracle(seed):
    rng = np.random.default_rng(seed)
    caps = [int(rng.integers(1, 6)) for _ in range(int(rng.integers(1, 6)))]
    acc = [sorted((float(x) for x in rng.uniform(0.05, 0.95, c)), reverse=True) for c in caps]
    if seed % 2:                                      # unsorted ranks take the full-frontier path
        acc = [list(rng.permutation(a)) for a in acc]
    total = 1 + sum(int(np.prod(caps[:l + 1])) for l in range(len(caps)))
    for width in sorted({1, 2, 3, 7, 16, min(40, total), min(64, total)}):
        if width > total:
            continue
        parent, paths, prob = arca.build_tree(acc, width)
        want_parent, want_prob = oracle.arca_tree(acc, width)
        assert parent == want_parent
        assert np.allclose(prob, want_prob, rtol=1e-13, atol=0)
        assert abs(arca.expected_tokens(prob) - oracle.expected_acceptance(want_prob)) < 1e-12


def test_synthetic_accuracies_reproduce_the_benchmark_tree():
    parent, _, _ = arca.build_tree(arca.synthetic_accuracies(), 64)
    assert parent == wl.medusa_tree(64)               # the input generator's own construction of the same tree


def test_width_choice_is_the_argmax_of_tokens_per_second():
    acc = arca.synthetic_accuracies()
    lat = {1: 100.0, 4: 101.0, 16: 104.0, 64: 110.0, 128: 200.0, 256: 400.0}
    best, rows = arca.choose_width(lat, acc)
    obest, table = oracle.best_width(lat, acc)
    assert best == obest == 64
    for w, l, tau, tps in rows:
        assert abs(tau - table[w][0]) < 1e-12 and abs(tps - table[w][1]) < 1e-6 * tps
    taus = [r[2] for r in rows]
    assert all(a < b for a, b in zip(taus, taus[1:]))         # more nodes never lower the expectation
    flat = {w: 100.0 for w in lat}
    assert arca.choose_width(flat, acc)[0] == 256 and oracle.best_width(flat, acc)[0] == 256
