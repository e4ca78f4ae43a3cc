"""Pins of the optimal-tree oracle (Section 4, Algorithm 3's objective): the "k most probable
vertices" definition against an exhaustive search over all valid trees, the structure the paper
states (a valid tree, descendants never more probable than ancestors), and the special cases
that reduce to the paper's named strategies."""
import itertools

import pytest

from oracle import tree_oracle as to


ACCEPTS = [[0.6, 0.25, 0.1], [0.9, 0.05], [0.5, 0.5, 0.5], [0.35, 0.3, 0.2, 0.1], [0.8], [1.0, 0.4]]


@pytest.mark.parametrize("accept", ACCEPTS)
@pytest.mark.parametrize("k", [1, 2, 3, 4, 5, 6])
def test_top_k_vertices_maximise_the_expected_number_of_accepted_tokens(accept, k):
    top = to.top_k_vertices(accept, k)
    paths = [p for _, p in top]
    assert len(paths) == k and to.is_valid_tree(paths)          # the top k form a valid tree
    best = to.best_tree_by_search(accept, k)                    # every valid tree, exhaustively
    assert to.expected_accepted(paths, accept) == pytest.approx(best, abs=1e-12)
    # a plausible mistake -- dropping the sibling rule or a level -- must lose to the optimum
    chain = [tuple([0] * d) for d in range(1, k + 1)]
    assert to.expected_accepted(chain, accept) <= best + 1e-12


def test_acceptance_probability_never_grows_along_a_path():
    accept = [0.7, 0.2, 0.05]
    for depth in (1, 2, 3):
        for path in itertools.product(range(3), repeat=depth):
            r = to.vertex_probability(path, accept)
            assert r <= to.vertex_probability(path[:-1], accept) + 1e-15
            if path[-1] > 0:
                assert r <= to.vertex_probability(path[:-1] + (path[-1] - 1,), accept) + 1e-15


def test_special_cases_reduce_to_the_named_strategies():
    # one possible child per node: the optimum is sequence drafting (a chain)
    paths = [p for _, p in to.top_k_vertices([0.8], 5)]
    assert sorted(paths) == [tuple([0] * d) for d in range(1, 6)]
    assert to.parent_array(paths) == [-1, 0, 1, 2, 3, 4]
    # deeper vertices worthless (first-child acceptance tiny, siblings likely): batch drafting
    paths = [p for _, p in to.top_k_vertices([0.3, 0.29, 0.28, 0.27], 4)]
    assert sorted(paths) == [(0,), (1,), (2,), (3,)]
    assert to.parent_array(paths) == [-1, 0, 0, 0, 0]
    # expected tokens of a chain with acceptance a: a + a^2 + ... (geometric)
    a = 0.8
    assert to.expected_accepted([tuple([0] * d) for d in range(1, 6)], [a]) == pytest.approx(
        sum(a ** d for d in range(1, 6)))


def test_parent_array_is_in_the_librarys_form():
    paths = [p for _, p in to.top_k_vertices([0.6, 0.25, 0.1], 6)]
    parent = to.parent_array(paths)
    assert parent[0] == -1 and all(0 <= parent[n] < n for n in range(1, len(parent)))
