"""Pins of the oracle's sequence and tree verification (no GPU)."""
import math

import numpy as np
import pytest

import oracle
from oracle import ersd_oracle_np as onp
from paper_2504_15475_b200 import workloads as wl


def softmax(z, T=1.0):
    s = np.asarray(z, dtype=np.float64) / T
    p = np.exp(s - s.max())
    return p / p.sum()


def match_closed_form(p, q):
    return sum(1.0 / np.maximum(p / p[i], q / q[i]).sum() for i in range(len(p)))


def small_rows(rng, B, rows, V, spread):
    tgt = rng.normal(size=(B, rows, V)).astype(np.float32)
    drf = (tgt + spread * rng.normal(size=(B, rows, V))).astype(np.float32)
    return tgt, drf


def test_simple_ersd_two_outcomes():
    """Algorithm 2 (k = 1): winners agree -> (draft token, sample of the next target row);
    they differ -> the target winner alone."""
    rng = np.random.default_rng(0)
    B, V = 4000, 5
    tgt, drf = small_rows(rng, B, 2, V, 1.0)
    out = oracle.verify(tgt, drf[:, :1], seeds=np.arange(B) + 10, T=1.0)
    acc = out["accept_len"] == 1
    assert 0.2 < acc.mean() < 0.95
    assert (out["tokens"][acc, 0] == out["draft_tok"][acc, 0]).all()
    assert (out["tokens"][acc, 1] == out["target_tok"][acc, 1]).all() and (out["tokens"][acc, 1] >= 0).all()
    rej = ~acc
    assert (out["tokens"][rej, 0] == out["target_tok"][rej, 0]).all()
    assert (out["tokens"][rej, 0] != out["draft_tok"][rej, 0]).all()
    assert (out["tokens"][rej, 1] == -1).all()


def test_sequence_accept_length_law():
    """Accept in order until the first disagreement (Section 2); with one independent race per
    position, Pr{L >= j} = prod_{i<j} m_i with m_i the closed-form match probability."""
    rng = np.random.default_rng(1)
    k, V, B = 4, 6, 60_000
    tgt1, drf1 = small_rows(rng, 1, k + 1, V, 0.8)
    tgt = np.repeat(tgt1, B, axis=0)
    drf = np.repeat(drf1[:, :k], B, axis=0)
    out = oracle.verify(tgt, drf, seeds=np.arange(B, dtype=np.uint64) * 7919 + 1, T=1.0)
    m = [match_closed_form(softmax(tgt1[0, j]), softmax(drf1[0, j])) for j in range(k)]
    L = out["accept_len"]
    surv = 1.0
    for j in range(1, k + 1):
        surv *= m[j - 1]
        got = (L >= j).mean()
        assert abs(got - surv) < 4.5 * math.sqrt(surv * (1 - surv) / B), (j, got, surv)
    # emitted tokens: target winners up to and including position L, then -1
    for j in range(k + 1):
        live = L >= j
        assert (out["tokens"][live, j] == out["target_tok"][live, j]).all()
        assert (out["tokens"][~live, j] == -1).all()
    # the bonus token after k acceptances is a sample of the last target row
    full = L == k
    cnt = np.bincount(out["tokens"][full, k], minlength=V)
    from scipy import stats
    assert stats.chisquare(cnt, softmax(tgt1[0, k]) * full.sum()).pvalue > 1e-3


def test_identical_models_accept_everything():
    rng = np.random.default_rng(2)
    tgt, _ = small_rows(rng, 50, 6, 40, 0.0)
    out = oracle.verify(tgt, tgt[:, :5].copy(), seeds=np.arange(50), T=0.7)
    assert (out["accept_len"] == 5).all() and (out["tokens"] >= 0).all()


def test_numpy_version_agrees_on_sequence_and_tree():
    rng = np.random.default_rng(3)
    B, k, V = 6, 4, 33
    tgt, drf = small_rows(rng, B, k + 1, V, 0.7)
    seeds = np.arange(B, dtype=np.uint64) + 1000
    out = oracle.verify(tgt, drf[:, :k], seeds, T=0.9)
    tok_np, acc_np = onp.verify(tgt, drf[:, :k], seeds, float(np.float32(0.9)))
    assert (acc_np == out["accept_len"]).all()
    for b in range(B):
        L = acc_np[b]
        assert list(tok_np[b, :L + 1]) == list(out["tokens"][b, :L + 1])
    for parent in (wl.TREE_4x4, wl.TREE_SPECINFER, wl.star_parent(5)):
        nodes = len(parent)
        tgt, drf = small_rows(rng, B, nodes, V, 0.7)
        res = oracle.verify_tree(tgt, drf, parent, seeds, T=0.9)
        ys = onp.verify_tree(tgt, drf, list(parent), seeds, float(np.float32(0.9)))
        for b in range(B):
            n = res["accept_len"][b] + 1
            assert list(res["tokens"][b, :n]) == ys[b]
            assert (res["tokens"][b, n:] == -1).all()


def test_chain_tree_is_the_sequence_variant():
    """The tree strategy subsumes the sequence strategy (Section 2): a chain gives the same
    emitted tokens and accept length, position for position."""
    rng = np.random.default_rng(4)
    B, k, V = 40, 5, 50
    tgt, drf = small_rows(rng, B, k + 1, V, 0.6)
    seeds = np.arange(B, dtype=np.uint64) * 3 + 5
    seq = oracle.verify(tgt, drf[:, :k], seeds, T=1.0)
    tree = oracle.verify_tree(tgt, drf, wl.chain_parent(k), seeds, T=1.0)
    assert (tree["accept_len"] == seq["accept_len"]).all()
    assert (tree["tokens"] == seq["tokens"]).all()
    assert tree["depth"] == k


def test_star_tree_is_batch_drafting():
    """Batch drafting = the first k arrivals under Q (Section 3): two tokens if the target winner
    is among them, else one; acceptance is non-decreasing in k and reaches 1 at k = V."""
    rng = np.random.default_rng(5)
    B, V = 3000, 6
    seeds = np.arange(B, dtype=np.uint64) + 77
    tgt1 = rng.normal(size=(1, 1, V)).astype(np.float32)
    drf1 = (tgt1 + rng.normal(size=(1, 1, V))).astype(np.float32)
    prev = None
    rates = []
    for c in range(1, V + 1):
        tgt = np.repeat(np.repeat(tgt1, c + 1, axis=1), B, axis=0)
        drf = np.repeat(np.repeat(drf1, c + 1, axis=1), B, axis=0)
        res = oracle.verify_tree(tgt, drf, wl.star_parent(c), seeds, T=1.0)
        acc = res["accept_len"]
        assert set(np.unique(acc)) <= {0, 1}
        hit = (res["arrivals"][:, 0, :c] == res["target_tok"][:, 0:1]).any(axis=1)
        assert (hit == (acc == 1)).all()
        if prev is not None:
            assert (acc >= prev).all()       # same races, one more candidate
        prev = acc
        rates.append(acc.mean())
    assert rates[-1] == 1.0
    m = match_closed_form(softmax(tgt1[0, 0]), softmax(drf1[0, 0]))
    assert abs(rates[0] - m) < 4.5 * math.sqrt(m * (1 - m) / B)


@pytest.mark.parametrize("parent", [wl.TREE_4x4, wl.TREE_SPECINFER])
def test_tree_walk_follows_algorithm_5(parent):
    rng = np.random.default_rng(6)
    B, V, nodes = 400, 12, len(parent)
    tgt, drf = small_rows(rng, B, nodes, V, 0.5)
    seeds = np.arange(B, dtype=np.uint64) + 1
    res = oracle.verify_tree(tgt, drf, parent, seeds, T=1.0)
    D, max_c, nchild, rank = oracle.tree_shape(parent)
    assert res["tokens"].shape == (B, D + 1)
    accepted = np.zeros(nodes)
    for b in range(B):
        L = res["accept_len"][b]
        path = res["path"][b]
        assert path[0] == 0 and (path[L + 1:] == -1).all()
        for d in range(1, L + 1):
            n, par = path[d], path[d - 1]
            assert parent[n] == par                                   # a root path
            # the accepted child carries the token the target race chose at its parent
            assert res["arrivals"][b, par, rank[n]] == res["tokens"][b, d - 1]
            assert res["tokens"][b, d - 1] == res["target_tok"][b, par]
            accepted[n] += 1
        last = path[L]
        assert res["tokens"][b, L] == res["target_tok"][b, last]
        kids = [m for m in range(nodes) if parent[m] == last]
        assert all(res["arrivals"][b, last, rank[m]] != res["tokens"][b, L] for m in kids)
        # siblings carry distinct tokens (sampling without replacement)
        for n in range(nodes):
            a = res["arrivals"][b, n, :nchild[n]]
            assert len(set(a.tolist())) == nchild[n]
    # a descendant is accepted no more often than its ancestor (Section 4)
    for n in range(1, nodes):
        if parent[n] > 0:
            assert accepted[n] <= accepted[parent[n]]


def test_position_offsets_and_sequence_ids_select_the_race():
    rng = np.random.default_rng(7)
    B, k, V = 3, 2, 20
    tgt, drf = small_rows(rng, B, k + 1, V, 0.5)
    seeds = np.array([5, 5, 5], dtype=np.uint64)
    a = oracle.verify(tgt, drf[:, :k], seeds, T=1.0, seq_ids=[9, 9, 9], pos_offsets=[0, 1, 100])
    # sequence 1 at offset 1 races position 1 with the stream sequence 0 uses at its row 1
    k01 = oracle.row_keys(tgt[1, 0], 1.0, 5, 9, 1)
    assert a["target_tok"][1, 0] == np.argmin(k01)
    k2 = oracle.row_keys(tgt[2, 1], 1.0, 5, 9, 101)
    assert a["target_tok"][2, 1] == np.argmin(k2)


def test_workload_recipe_shapes():
    w = wl.scaled(wl.CONFIGS["c2"], B=2, V=512)
    x = wl.make_inputs(w, call=3)
    assert x["target"].shape == (2, 5, 512) and x["draft"].shape == (2, 4, 512)
    y = wl.make_inputs(w, call=3)
    assert (x["target"].view(dtype=__import__("torch").int16) == y["target"].view(dtype=__import__("torch").int16)).all()
    assert (x["seeds"] == y["seeds"]).all()
    z = wl.make_inputs(w, call=4)
    assert not (x["seeds"] == z["seeds"]).all()
    t = wl.make_inputs(wl.scaled(wl.CONFIGS["c4"], B=1, V=256))
    assert t["target"].shape == (1, 17, 256) and t["draft"].shape == (1, 17, 256)
    c5 = wl.make_inputs(wl.scaled(wl.CONFIGS["c5"], B=4, V=256))
    assert c5["temps"].shape == (4, 6)
    assert set(np.unique(c5["temps"].numpy()).astype(np.float64).round(3).tolist()) <= {0.6, 0.8, 1.0}
    c1 = wl.make_inputs(wl.CONFIGS["c1"])
    assert c1["seeds"].tolist() == [0] and c1["target"].dtype == __import__("torch").float32


def test_token_given_verification_agrees_with_the_row_given_one():
    """Drafting first (winners of the draft rows) and then verifying the given tokens is the
    sequence procedure of Section 3 cut in two: same accepted prefix, same emitted tokens."""
    rng = np.random.default_rng(11)
    B, k, V = 40, 5, 300
    tgt = rng.normal(size=(B, k + 1, V)).astype(np.float32) * 2
    drf = (tgt[:, :k] + rng.normal(size=(B, k, V)).astype(np.float32) * 0.7).astype(np.float32)
    seeds = rng.integers(0, 2**63, size=B).astype(np.uint64)
    full = oracle.verify(tgt, drf, seeds, T=0.9)
    drafted, _ = oracle.race_sample(drf, seeds, T=0.9)
    got = oracle.verify_tokens(tgt, drafted[..., 0], seeds, T=0.9)
    assert (drafted[..., 0] == full["draft_tok"]).all()
    assert (got["accept_len"] == full["accept_len"]).all()
    assert (got["tokens"] == full["tokens"]).all()
    assert 0 < got["accept_len"].mean() < k                   # both outcomes occur


def test_token_given_verification_outcomes_of_algorithm_2():
    """k = 1: a drafted token equal to the target winner gives two tokens, any other gives the
    target winner alone; a wrong later token cuts the prefix exactly there."""
    rng = np.random.default_rng(12)
    B, V = 30, 50
    tgt = rng.normal(size=(B, 2, V)).astype(np.float32)
    seeds = np.arange(B, dtype=np.uint64) + 5
    win, _ = oracle.race_sample(tgt, seeds, T=1.0)
    hit = oracle.verify_tokens(tgt, win[:, :1, 0], seeds, T=1.0)
    assert (hit["accept_len"] == 1).all() and (hit["tokens"] == win[..., 0]).all()
    miss = oracle.verify_tokens(tgt, (win[:, :1, 0] + 1) % V, seeds, T=1.0)
    assert (miss["accept_len"] == 0).all()
    assert (miss["tokens"][:, 0] == win[:, 0, 0]).all() and (miss["tokens"][:, 1] == -1).all()
    tgt3 = rng.normal(size=(B, 4, V)).astype(np.float32)
    w3, _ = oracle.race_sample(tgt3, seeds, T=1.0)
    d = w3[:, :3, 0].copy()
    d[:, 1] = (d[:, 1] + 3) % V                               # second drafted token wrong
    cut = oracle.verify_tokens(tgt3, d, seeds, T=1.0)
    assert (cut["accept_len"] == 1).all() and (cut["tokens"][:, 2:] == -1).all()
    assert (cut["tokens"][:, :2] == w3[:, :2, 0]).all()
