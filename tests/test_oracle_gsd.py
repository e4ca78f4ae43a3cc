"""Pins of the oracle's greedy speculative decoding (Algorithms 1 and 4) -- no GPU.

GSD is the paper's comparison verifier: a ratio test per drafted token and, on rejection, a sample
of the residual law.  What the paper and the mathematics fix: the acceptance probability of a
token drafted from Q is 1 - D_TV[P, Q] (Section 3), the emitted token follows P exactly
(losslessness of rejection sampling with the residual), the recursion of Algorithm 4 over several
candidates drafted without replacement has an acceptance probability that a few lines of numpy
enumerate exactly on a tiny alphabet, and Lemma 3.1 orders ERSD's match rate against GSD's.
"""
import itertools
import math

import numpy as np
import pytest
from scipy import stats

import oracle
from paper_2504_15475_b200 import workloads as wl


def softmax(z, T=1.0):
    s = np.asarray(z, dtype=np.float64) / T
    p = np.exp(s - s.max())
    return p / p.sum()


def tv(p, q):
    return 0.5 * np.abs(p - q).sum()


def rows_for(rng, V, spread=1.0, scale=1.2):
    zt = (scale * rng.normal(size=V)).astype(np.float32)
    zd = (zt + spread * rng.normal(size=V)).astype(np.float32)
    return zt, zd


def draft_with_independent_races(drf, seeds, T, c=1):
    """Tokens drafted from the draft rows: first c arrivals of an exponential race (a sample
    without replacement, Section 3), with seeds of their own."""
    tok, _ = oracle.race_sample(drf, seeds, T=T, c=c)
    return tok


def test_ratio_test_uniforms_are_uniform_and_separate_from_the_race():
    n = 20000
    u = np.array([oracle.gsd_uniform(99, 5, node, 0) for node in range(n)])
    assert (u > 0).all() and (u < 1).all()
    assert stats.kstest(u, "uniform").pvalue > 1e-3
    # another child rank, sequence or seed: another stream
    assert oracle.gsd_uniform(99, 5, 7, 0) != oracle.gsd_uniform(99, 5, 7, 1)
    assert oracle.gsd_uniform(99, 5, 7, 0) != oracle.gsd_uniform(99, 6, 7, 0)
    assert oracle.gsd_uniform(99, 5, 7, 0) != oracle.gsd_uniform(98, 5, 7, 0)
    # not a word of the drafting race of the same node (last counter word 0)
    race_words = {oracle.token_word(99, 5, 7, i) for i in range(8)}
    assert int(oracle.gsd_uniform(99, 5, 7, 0) * 2**32) not in race_words


def simple_runs(V=8, B=60_000, T=0.9, seed=3, spread=0.6):
    # rows whose residual max(P - Q, 0) has at least three tokens and whose acceptance is mid-range
    while True:
        rng = np.random.default_rng(seed)
        zt, zd = rows_for(rng, V, spread)
        pp, qq = softmax(zt, T), softmax(zd, T)
        if (pp > qq).sum() >= 3 and 0.3 < 1 - tv(pp, qq) < 0.9:
            break
        seed += 1
    zt2 = (1.3 * rng.normal(size=V)).astype(np.float32)
    tgt = np.broadcast_to(np.stack([zt, zt2]), (B, 2, V)).copy()
    drf = np.broadcast_to(zd, (B, 1, V)).copy()
    seeds = np.arange(B, dtype=np.uint64) * 7919 + 11
    tok = draft_with_independent_races(drf, seeds + np.uint64(1 << 40), T)[..., 0]
    out = oracle.gsd_verify(tgt, drf, tok, seeds, T=T)
    T = float(np.float32(T))                                    # (the temperature travels as a float)
    return softmax(zt, T), softmax(zd, T), softmax(zt2, T), tok[:, 0], out


def test_simple_gsd_accepts_with_probability_one_minus_total_variation():
    """Section 3: the acceptance probability of greedy decoding is 1 - D_TV[P, Q]."""
    p, q, _, _, out = simple_runs()
    B = out["accept_len"].shape[0]
    want = 1.0 - tv(p, q)
    got = (out["accept_len"] == 1).mean()
    assert abs(got - want) < 4.5 * math.sqrt(want * (1 - want) / B), (got, want)
    assert 0.2 < want < 0.95                                    # both outcomes are well populated


def test_simple_gsd_outcomes_and_laws():
    """Algorithm 1: accepted -> (drafted token, sample of the next target row); rejected -> one
    sample of max(P - Q, 0) / sum.  Overall the first emitted token follows P (losslessness)."""
    p, q, p2, drafted, out = simple_runs()
    V = p.shape[0]
    acc = out["accept_len"] == 1
    y = out["tokens"]
    assert (y[acc, 0] == drafted[acc]).all() and (y[acc, 1] >= 0).all()
    assert (y[~acc, 1] == -1).all() and (y[~acc, 0] >= 0).all()
    # the test that was applied is the one stated: P(x)/Q(x) > u
    r, u = out["ratio"][:, 0], out["unif"][:, 0]
    np.testing.assert_allclose(r, p[drafted] / q[drafted], rtol=1e-12)
    assert ((r > u) == acc).all()
    # first token ~ P
    cnt = np.bincount(y[:, 0], minlength=V)
    assert stats.chisquare(cnt, p * len(y)).pvalue > 1e-3
    assert stats.chisquare(cnt, q * len(y)).pvalue < 1e-12     # (not the draft law)
    # rejected branch ~ residual; accepted branch ~ min(p, q) / sum: neither is P
    res = np.maximum(p - q, 0.0)
    res /= res.sum()
    cnt_r = np.bincount(y[~acc, 0], minlength=V)
    keep = res > 0
    assert (cnt_r[~keep] == 0).all()
    assert stats.chisquare(cnt_r[keep], res[keep] * cnt_r.sum()).pvalue > 1e-3
    assert stats.chisquare(cnt_r + 1e-9, p * cnt_r.sum()).pvalue < 1e-12
    m = np.minimum(p, q)
    cnt_a = np.bincount(y[acc, 0], minlength=V)
    assert stats.chisquare(cnt_a, m / m.sum() * cnt_a.sum()).pvalue > 1e-3
    # the token after an acceptance is a sample of the next target row
    cnt2 = np.bincount(y[acc, 1], minlength=V)
    assert stats.chisquare(cnt2, p2 * cnt2.sum()).pvalue > 1e-3


def test_sequence_gsd_accept_length_law_and_special_cases():
    """Tokens are verified in order until the first rejection (Section 2): with independent
    uniforms Pr{L >= j} = prod_{i<j} (1 - D_TV[P_i, Q_i]).  Identical models accept everything."""
    rng = np.random.default_rng(8)
    k, V, B, T = 4, 7, 50_000, 1.0
    tgt1 = (1.2 * rng.normal(size=(1, k + 1, V))).astype(np.float32)
    drf1 = (tgt1[:, :k] + 0.7 * rng.normal(size=(1, k, V))).astype(np.float32)
    tgt, drf = np.repeat(tgt1, B, axis=0), np.repeat(drf1, B, axis=0)
    seeds = np.arange(B, dtype=np.uint64) * 104729 + 5
    tok = draft_with_independent_races(drf, seeds + np.uint64(1 << 41), T)[..., 0]
    out = oracle.gsd_verify(tgt, drf, tok, seeds, T=T)
    L = out["accept_len"]
    surv = 1.0
    for j in range(1, k + 1):
        surv *= 1.0 - tv(softmax(tgt1[0, j - 1]), softmax(drf1[0, j - 1]))
        got = (L >= j).mean()
        assert abs(got - surv) < 4.5 * math.sqrt(surv * (1 - surv) / B), (j, got, surv)
    for j in range(k + 1):
        assert (out["tokens"][L >= j, j] >= 0).all() and (out["tokens"][L < j, j] == -1).all()
    acc_all = L == k
    assert (out["tokens"][acc_all, :k] == tok[acc_all]).all()
    same = oracle.gsd_verify(tgt[:500], tgt[:500, :k].copy(),
                             draft_with_independent_races(tgt[:500, :k].copy(), seeds[:500], T)[..., 0], seeds[:500], T=T)
    assert (same["accept_len"] == k).all() and (same["tokens"] >= 0).all()


def test_lemma_3_1_orders_the_two_verifiers():
    """Lemma 3.1: 1 - D_TV >= P_accept(ERSD) >= D_HM, and 1 - D_TV is what GSD achieves: on the
    same rows GSD's acceptance rate is not below ERSD's match rate (up to Monte-Carlo error), and
    ERSD's stays above the harmonic-mean distance."""
    rng = np.random.default_rng(12)
    V, B, T = 8, 40_000, 1.0
    zt, zd = rows_for(rng, V, spread=1.3)
    p, q = softmax(zt), softmax(zd)
    tgt = np.broadcast_to(np.stack([zt, zt]), (B, 2, V)).copy()
    drf = np.broadcast_to(zd, (B, 1, V)).copy()
    seeds = np.arange(B, dtype=np.uint64) + 1000
    ersd = oracle.verify(tgt, drf, seeds, T=T)
    tok = draft_with_independent_races(drf, seeds + np.uint64(1 << 42), T)[..., 0]
    gsd = oracle.gsd_verify(tgt, drf, tok, seeds, T=T)
    a_e, a_g = (ersd["accept_len"] == 1).mean(), (gsd["accept_len"] == 1).mean()
    se = 4.5 * math.sqrt(0.25 / B)
    d_hm = (p * q / (p + q)).sum()
    assert a_g + se >= a_e >= d_hm - se
    assert abs(a_g - (1 - tv(p, q))) < se
    assert a_g - a_e > se                                       # on these rows the gap is visible


def exact_batch_acceptance(p, q, c):
    """Pr{some candidate accepted} of Algorithm 4 at one vertex with c candidates drafted without
    replacement from q, by enumeration over the ordered candidate tuples (tiny alphabets)."""
    V = len(p)
    total = 0.0
    for order in itertools.permutations(range(V), c):
        pt, qd, w_draw, rej = p.copy(), q.copy(), 1.0, 1.0
        acc = 0.0
        for x in order:
            if qd[x] <= 0:
                w_draw = 0.0
                break
            w_draw *= qd[x]
            a = min(1.0, pt[x] / qd[x])
            acc += rej * a
            rej *= 1.0 - a
            pt = np.maximum(pt - qd, 0.0)
            if pt.sum() > 0:
                pt = pt / pt.sum()
            qd = qd.copy()
            qd[x] = 0.0
            if qd.sum() > 0:
                qd = qd / qd.sum()
        total += w_draw * acc
    return total


@pytest.mark.parametrize("c", [1, 2, 3])
def test_tree_gsd_at_one_vertex_matches_the_enumerated_recursion(c):
    """Algorithm 4 on a star with c candidates: acceptance rate against the exact enumeration of
    the recursion (residual target law, rejected token removed from the draft law), and the
    emitted first token still follows P."""
    rng = np.random.default_rng(20 + c)
    V, B, T = 4, 60_000, 1.0
    zt, zd = rows_for(rng, V, spread=1.0, scale=1.0)
    p, q = softmax(zt), softmax(zd)
    parent = wl.star_parent(c)
    nodes = c + 1
    tgt = np.broadcast_to(zt, (B, nodes, V)).copy()
    drf = np.broadcast_to(zd, (B, nodes, V)).copy()
    seeds = np.arange(B, dtype=np.uint64) * 31 + 7
    arr = draft_with_independent_races(drf[:, :1], seeds + np.uint64(1 << 43), T, c=c)[:, 0, :]   # [B, c]
    tok = np.full((B, nodes), -1, np.int32)
    tok[:, 1:] = arr
    out = oracle.gsd_verify_tree(tgt, drf, tok, parent, seeds, T=T)
    want = exact_batch_acceptance(p, q, c)
    got = (out["accept_len"] == 1).mean()
    assert abs(got - want) < 4.5 * math.sqrt(want * (1 - want) / B), (c, got, want)
    if c == 1:
        assert abs(want - (1 - tv(p, q))) < 1e-12
    cnt = np.bincount(out["tokens"][:, 0], minlength=V)
    assert stats.chisquare(cnt, p * B).pvalue > 1e-3
    acc = out["accept_len"] == 1
    # an accepted sequence continues with a sample of the accepted child's target row; the path is a root path
    assert (out["tokens"][acc, 1] >= 0).all() and (out["tokens"][~acc, 1] == -1).all()
    assert (out["path"][:, 0] == 0).all()
    for b in np.flatnonzero(acc)[:200]:
        m = out["path"][b, 1]
        assert parent[m] == 0 and tok[b, m] == out["tokens"][b, 0]


def test_chain_tree_gsd_is_sequence_gsd():
    """The tree strategy subsumes the sequence strategy (Section 2)."""
    rng = np.random.default_rng(31)
    B, k, V, T = 300, 5, 40, 0.8
    tgt = (1.5 * rng.normal(size=(B, k + 1, V))).astype(np.float32)
    drf = (tgt + 0.5 * rng.normal(size=(B, k + 1, V))).astype(np.float32)
    seeds = np.arange(B, dtype=np.uint64) + 77
    tok = draft_with_independent_races(drf[:, :k], seeds + np.uint64(1 << 44), T)[..., 0]
    seq = oracle.gsd_verify(tgt, drf[:, :k].copy(), tok, seeds, T=T)
    tree_tok = np.full((B, k + 1), -1, np.int32)
    tree_tok[:, 1:] = tok
    tree = oracle.gsd_verify_tree(tgt, drf, tree_tok, wl.chain_parent(k), seeds, T=T)
    assert (tree["accept_len"] == seq["accept_len"]).all()
    assert (tree["tokens"] == seq["tokens"]).all()
    assert 0 < seq["accept_len"].mean() < k


def test_gsd_per_row_temperatures():
    """The ratio of position j is formed at that row's temperature."""
    rng = np.random.default_rng(41)
    B, k, V = 4, 3, 30
    tgt = (2.0 * rng.normal(size=(B, k + 1, V))).astype(np.float32)
    drf = (tgt[:, :k] + 0.4 * rng.normal(size=(B, k, V))).astype(np.float32)
    seeds = np.arange(B, dtype=np.uint64) + 3
    t = (0.5 + 0.13 * np.arange(B * (k + 1)).reshape(B, k + 1)).astype(np.float32)
    tok = np.stack([np.argmax(drf[:, j], axis=-1) for j in range(k)], axis=1).astype(np.int32)
    out = oracle.gsd_verify(tgt, drf, tok, seeds, T=9.0, temps=t)
    for b in range(B):
        for j in range(k):
            if np.isnan(out["ratio"][b, j]):
                continue
            p, q = softmax(tgt[b, j], float(t[b, j])), softmax(drf[b, j], float(t[b, j]))
            assert out["ratio"][b, j] == pytest.approx(p[tok[b, j]] / q[tok[b, j]], rel=1e-12)
            assert out["unif"][b, j] == oracle.gsd_uniform(int(seeds[b]), b, j, 0)
