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


# ----------------------------------------------------------------------------- empirical acceptance profile
def test_acceptance_profile_worked_example():
    """Section 5's empirical R on a tree small enough to count by hand.  Tree: root 0 with children
    1, 2 (ranks 0, 1); node 1 with children 3, 4; node 2 with child 5.  Four verified paths."""
    from oracle import tree_oracle as to
    parent = [-1, 0, 0, 1, 1, 2]
    paths = [[0, 1, 3], [0, 2, -1], [0, -1, -1], [0, 1, -1]]
    # trials: root verified 4 times -> ranks 0 and 1 tried 4 times each; node 1 verified twice ->
    # ranks 0, 1 twice each; node 2 verified once -> rank 0 once.  hits: rank 0: 0->1 twice, 1->3 once;
    # rank 1: 0->2 once.
    acc, tri = to.acceptance_profile(paths, parent, 2)
    assert tri == [7, 6] and acc == [3 / 7, 1 / 6]
    from paper_2504_15475_b200 import binding
    got, got_tri = binding.ersd_acceptance_profile(np.array(paths, np.int32), parent, 2)
    assert got_tri == tri and got == pytest.approx(acc, abs=0)
    # a third rank was never tried: 0; an estimate that rises with the rank is capped by the library
    got3, tri3 = binding.ersd_acceptance_profile(np.array(paths, np.int32), parent, 3)
    assert tri3 == [7, 6, 0] and got3[2] == 0.0
    rising = [[0, 2, -1]] * 3 + [[0, 1, -1]]
    raw, _ = to.acceptance_profile(rising, parent, 2)
    capped, _ = binding.ersd_acceptance_profile(np.array(rising, np.int32), parent, 2)
    # (rank 0: tried 4 times at the root, 3 at node 2, once at node 1, accepted once; rank 1: tried 4 + 1 times, accepted 3 times)
    assert raw == [0.125, 0.6] and capped == [0.125, 0.125]
    # a path that is not a root path of the tree is refused
    with pytest.raises(binding.ErsdError):
        binding.ersd_acceptance_profile(np.array([[0, 3, -1]], np.int32), parent, 2)


def test_acceptance_profile_recovers_a_known_profile_and_feeds_the_builder():
    """Paths simulated from a 0-th order source with known per-rank acceptance: the library's
    profile equals the oracle's count, estimates the source, and the tree built from it is the tree
    of the true profile."""
    from oracle import tree_oracle as to
    from paper_2504_15475_b200 import binding
    rng = np.random.default_rng(5)
    true = [0.55, 0.2, 0.08]
    parent, _ = binding.ersd_optimal_tree(true, 12)
    n = len(parent)
    kids = [[m for m in range(1, n) if parent[m] == v] for v in range(n)]
    D = binding.ersd_tree_depth(parent)
    paths = np.full((20000, D + 1), -1, np.int32)
    for b in range(paths.shape[0]):
        cur, d = 0, 0
        paths[b, 0] = 0
        while kids[cur]:
            u, nxt, lo = rng.random(), None, 0.0
            for r, m in enumerate(kids[cur]):      # at most one child is accepted, rank r with probability true[r]
                if lo <= u < lo + true[r]:
                    nxt = m
                lo += true[r]
            if nxt is None:
                break
            cur, d = nxt, d + 1
            paths[b, d] = cur
    want, want_tri = to.acceptance_profile(paths.tolist(), parent, 3)
    got, got_tri = binding.ersd_acceptance_profile(paths, parent, 3)
    assert got_tri == want_tri and got == pytest.approx(want, abs=1e-15)
    for r in range(3):
        assert abs(got[r] - true[r]) < 4.5 * np.sqrt(true[r] * (1 - true[r]) / got_tri[r])
    rebuilt, _ = binding.ersd_optimal_tree(got, 12)
    assert rebuilt == parent
