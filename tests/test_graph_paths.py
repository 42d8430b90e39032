"""Path finding in the dataflow graph (Sec. 3.1): the oracle and the library's host-side search
against the examples the paper states in words, and against brute force on random graphs."""
import itertools
import os

import numpy as np
import pytest

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def _examples():
    ex, cur = [], None
    for line in open(os.path.join(HERE, "golden", "paths_paper_examples.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, *rest = line.split()
        if key == "example":
            cur = {"name": rest[0], "paths": []}
        elif key in ("u2l", "l2u"):
            cur[key] = [tuple(int(x) for x in e.split(">")) for e in rest]
        elif key == "k":
            cur["k"] = int(rest[0])
        elif key == "targets":
            cur["targets"] = [int(x) for x in rest]
        elif key == "path":
            cur["paths"].append([int(x) for x in rest])
        elif key == "end":
            ex.append(cur)
    return ex


@pytest.mark.parametrize("ex", _examples(), ids=lambda e: e["name"])
def test_paths_of_the_papers_examples(ex):
    got = oracle.find_paths(ex["u2l"], ex["l2u"], ex["k"], ex["targets"])
    assert sorted(got) == sorted(ex["paths"])
    import paper_2207_02849_b200 as bt
    n = 1 + max(max(a, b) for a, b in ex["u2l"] + ex["l2u"])
    assert sorted(bt.betty_find_paths(n, ex["u2l"], ex["l2u"], ex["k"], ex["targets"])) == sorted(ex["paths"])


def _brute_force(n, u2l, l2u, k, targets):
    """Every simple sequence of problems, filtered by the rule: first edge upper-to-lower, the
    rest lower-to-upper, ends on a target, never returns to k."""
    U, L = set(u2l), set(l2u)
    out = []
    others = [i for i in range(n) if i != k]
    for m in range(1, n):
        for seq in itertools.permutations(others, m):
            if (k, seq[0]) not in U:
                continue
            if all((seq[i], seq[i + 1]) in L for i in range(m - 1)) and seq[-1] in targets:
                out.append([k] + list(seq))
    return out


@pytest.mark.parametrize("seed", range(8))
def test_paths_against_brute_force_on_random_graphs(seed):
    import paper_2207_02849_b200 as bt
    rng = np.random.default_rng(seed)
    n = 6
    k = n - 1
    # lower-to-upper edges go from a lower index to a higher one, upper-to-lower the other way
    l2u = [(a, b) for a in range(n) for b in range(a + 1, n) if rng.random() < 0.45]
    u2l = [(a, b) for a in range(n) for b in range(a) if rng.random() < 0.45]
    targets = [a for a, b in l2u if b == k] or [0]
    ref = sorted(_brute_force(n, u2l, l2u, k, set(targets)))
    assert sorted(oracle.find_paths(u2l, l2u, k, targets)) == ref
    assert sorted(bt.betty_find_paths(n, u2l, l2u, k, targets)) == ref


def test_find_paths_reports_the_needed_size_when_the_buffer_is_too_small():
    import ctypes as C
    import paper_2207_02849_b200 as bt
    from paper_2207_02849_b200 import binding
    eu, el = binding._edges([(3, 2), (3, 0)]), binding._edges([(0, 2)])
    t = (C.c_int32 * 1)(2)
    buf = (C.c_int32 * 3)()
    n_paths, n_ints = C.c_int32(0), C.c_int32(0)
    st = bt.lib().betty_find_paths(4, eu, 2, el, 1, 3, t, 1, buf, 3, C.byref(n_paths), C.byref(n_ints))
    assert st == bt.BETTY_ERR_WORKSPACE and n_paths.value == 2 and n_ints.value == 3 + 4
    assert list(buf) == [2, 3, 2]                       # the first record still fits
    assert bt.lib().betty_find_paths(4, eu, 2, el, 1, 9, t, 1, None, 0, C.byref(n_paths), None) == bt.BETTY_ERR_INVALID_ARG
