"""ersd_optimal_tree (Algorithm 3's priority-queue construction, host code of the library) against
the oracle's definition (the k most probable vertices) -- no GPU needed.  Several trees can tie,
so what is compared is what is unique: the expected number of accepted tokens; the tree itself is
checked for validity and for the form ersd_verify_tree takes."""
import ctypes as C

import numpy as np
import pytest

from oracle import tree_oracle as to
from paper_2504_15475_b200 import build as ersd_build


@pytest.fixture(scope="module")
def ersd():
    ersd_build.build()
    from paper_2504_15475_b200 import binding
    binding.lib()
    return binding


def paths_of(parent):
    """Child-rank tuples of a parent array whose siblings ascend by rank."""
    nchild = [0] * len(parent)
    path = [()] * len(parent)
    for n in range(1, len(parent)):
        p = parent[n]
        path[n] = path[p] + (nchild[p],)
        nchild[p] += 1
    return path[1:]


@pytest.mark.parametrize("accept", [[0.6, 0.25, 0.1], [0.9, 0.05], [0.35, 0.3, 0.2, 0.1], [0.8], [1.0, 0.4],
                                    [0.52, 0.17, 0.08, 0.05, 0.03, 0.02]])
@pytest.mark.parametrize("k", [0, 1, 2, 5, 9, 16, 40])
def test_library_tree_is_optimal_and_well_formed(ersd, accept, k):
    parent, expected = ersd.ersd_optimal_tree(accept, k)
    assert len(parent) == k + 1 and parent[0] == -1
    assert all(0 <= parent[n] < n for n in range(1, k + 1))
    paths = paths_of(parent)
    assert sorted(paths) == paths                              # lexicographic vertex order
    assert to.is_valid_tree(paths)
    assert expected == pytest.approx(to.expected_accepted(paths, accept), abs=1e-12)
    if k <= 16:
        ref = to.top_k_vertices(accept, k) if k else []
        assert expected == pytest.approx(sum(r for r, _ in ref), abs=1e-12)
    if k:
        assert ersd.ersd_tree_depth(parent) == max(len(p) for p in paths)


def test_random_acceptance_profiles(ersd):
    rng = np.random.default_rng(4)
    for _ in range(40):
        c = int(rng.integers(1, 6))
        accept = np.sort(rng.uniform(0.01, 0.95, size=c))[::-1].tolist()
        k = int(rng.integers(1, 9))
        parent, expected = ersd.ersd_optimal_tree(accept, k)
        assert expected == pytest.approx(sum(r for r, _ in to.top_k_vertices(accept, k)), abs=1e-12)
        assert expected == pytest.approx(to.best_tree_by_search(accept, min(k, 6)), abs=1e-12) or k > 6


def test_named_strategies_and_errors(ersd):
    assert ersd.ersd_optimal_tree([0.8], 5)[0] == [-1, 0, 1, 2, 3, 4]                 # sequence drafting
    assert ersd.ersd_optimal_tree([0.3, 0.29, 0.28, 0.27], 4)[0] == [-1, 0, 0, 0, 0]   # batch drafting
    L = ersd.lib()
    par = (C.c_int32 * 4)()
    good = (C.c_double * 2)(0.5, 0.2)
    assert L.ersd_optimal_tree(None, 2, 3, par, None) == -1
    assert L.ersd_optimal_tree(good, 2, -1, par, None) == -1
    assert L.ersd_optimal_tree((C.c_double * 2)(0.2, 0.5), 2, 3, par, None) == -1     # increasing ranks
    assert L.ersd_optimal_tree((C.c_double * 1)(1.5), 1, 3, par, None) == -1
    assert L.ersd_optimal_tree(good, 2, 300, par, None) == -3
