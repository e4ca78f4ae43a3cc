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


# ----------------------------------------------------------------------------- per-row temperatures
def distinct_temps(B, rows):
    """A temperature table in which every entry differs (0.35 .. ~2), as float32."""
    return (0.35 + 0.11 * np.arange(B * rows).reshape(B, rows)).astype(np.float32)


def test_per_row_temperatures_reach_their_rows_in_sequence_verification():
    """p = softmax(z / T) with T the temperature of THAT row (Section 3: the winner of a race is
    a sample of the row's law); the draft row of position j is raced at the temperature of
    target row j, with the same race variables."""
    rng = np.random.default_rng(21)
    B, k, V = 3, 4, 96
    rows = k + 1
    tgt = (3.0 * rng.normal(size=(B, rows, V))).astype(np.float32)
    drf = (tgt + 0.3 * rng.normal(size=(B, rows, V))).astype(np.float32)[:, :k]
    seeds = np.array([11, 22, 33], dtype=np.uint64)
    t = distinct_temps(B, rows)
    out = oracle.verify(tgt, drf, seeds, T=123.0, temps=t)      # the scalar must be ignored
    differs = 0
    for b in range(B):
        for j in range(rows):
            kt = oracle.row_keys(tgt[b, j], float(t[b, j]), int(seeds[b]), b, j)
            assert out["target_tok"][b, j] == np.argmin(kt)
            assert out["target_key"][b, j, 0] == kt.min()
            # the same row raced at a neighbouring entry's temperature has another key
            other = oracle.row_keys(tgt[b, j], float(t[(b + 1) % B, (j + 1) % rows]), int(seeds[b]), b, j)
            differs += int(other.min() != kt.min())
            if j < k:
                kd = oracle.row_keys(drf[b, j], float(t[b, j]), int(seeds[b]), b, j)
                assert out["draft_tok"][b, j] == np.argmin(kd)
                assert out["draft_key"][b, j, 0] == kd.min()
    assert differs == B * rows
    # the separately written numpy statement, given the same table, agrees
    tok_np, acc_np = onp.verify(tgt, drf, seeds, 123.0, temps=t.astype(np.float64))
    assert (acc_np == out["accept_len"]).all()
    for b in range(B):
        L = acc_np[b]
        assert list(tok_np[b, :L + 1]) == list(out["tokens"][b, :L + 1])
    # and the table matters: one scalar temperature gives other winners somewhere
    flat = oracle.verify(tgt, drf, seeds, T=1.0)
    assert (flat["target_key"][..., 0] != out["target_key"][..., 0]).any()


def test_per_row_temperatures_reach_their_nodes_in_tree_verification():
    """Algorithm 5 with one temperature per node: node n's target row and draft row are both
    raced at temps[b, n]."""
    rng = np.random.default_rng(22)
    parent = wl.TREE_SPECINFER
    nodes = len(parent)
    B, V = 2, 80
    tgt = (3.0 * rng.normal(size=(B, nodes, V))).astype(np.float32)
    drf = (tgt + 0.3 * rng.normal(size=(B, nodes, V))).astype(np.float32)
    seeds = np.array([5, 6], dtype=np.uint64)
    t = distinct_temps(B, nodes)
    res = oracle.verify_tree(tgt, drf, parent, seeds, T=55.0, temps=t)
    _, _, nchild, _ = oracle.tree_shape(parent)
    for b in range(B):
        for n in range(nodes):
            kt = oracle.row_keys(tgt[b, n], float(t[b, n]), int(seeds[b]), b, n)
            assert res["target_tok"][b, n] == np.argmin(kt)
            if nchild[n]:
                kd = oracle.row_keys(drf[b, n], float(t[b, n]), int(seeds[b]), b, n)
                want = np.argsort(kd, kind="stable")[:nchild[n]]
                assert list(res["arrivals"][b, n, :nchild[n]]) == list(want)
    ys = onp.verify_tree(tgt, drf, list(parent), seeds, 55.0, temps=t.astype(np.float64))
    for b in range(B):
        n = res["accept_len"][b] + 1
        assert list(res["tokens"][b, :n]) == ys[b]


def test_winner_law_per_row_temperature():
    """Losslessness (Section 3) row by row: in ONE call whose rows alternate between two
    temperatures, the winners of the rows at T_a follow softmax(z / T_a) and those at T_b follow
    softmax(z / T_b).  Negative controls: the same counts fit neither the other row's
    temperature (indices swapped) nor the scalar T of the call."""
    from scipy import stats
    z = np.array([0.4, -1.1, 1.3, 0.0, 0.7], np.float32)
    V, R = z.shape[0], 120_000
    Ta, Tb, Tscalar = 0.5, 1.6, 1.0
    logits = np.broadcast_to(z, (2, R, V)).copy()
    temps = np.empty((2, R), np.float32)
    temps[0, 0::2], temps[0, 1::2] = Ta, Tb
    temps[1, 0::2], temps[1, 1::2] = Tb, Ta
    tok, _ = oracle.race_sample(logits, seeds=[77, 78], T=Tscalar, temps=temps)
    tok = tok[..., 0]
    groups = {(0, 0): Ta, (0, 1): Tb, (1, 0): Tb, (1, 1): Ta}
    for (b, parity), T_true in groups.items():
        cnt = np.bincount(tok[b, parity::2], minlength=V)
        n = cnt.sum()
        T_other = Tb if T_true == Ta else Ta
        assert stats.chisquare(cnt, softmax(z, T_true) * n).pvalue > 1e-3, (b, parity)
        assert stats.chisquare(cnt, softmax(z, T_other) * n).pvalue < 1e-12
        assert stats.chisquare(cnt, softmax(z, Tscalar) * n).pvalue < 1e-12


def test_shared_race_at_per_row_temperature_matches_the_closed_form():
    """Draft and target row of a position share the race AND the temperature: the match rate of
    position j is sum_i 1 / sum_l max(p_l / p_i, q_l / q_i) with p, q = softmax(. / temps[b, j])
    (the coupling of Section 3), not the value at another row's temperature."""
    rng = np.random.default_rng(23)
    k, V, B = 2, 6, 40_000
    rows = k + 1
    tgt1 = (1.5 * rng.normal(size=(1, rows, V))).astype(np.float32)
    drf1 = (tgt1 + 1.0 * rng.normal(size=(1, rows, V))).astype(np.float32)[:, :k]
    tgt, drf = np.repeat(tgt1, B, axis=0), np.repeat(drf1, B, axis=0)
    t_row = np.array([0.4, 2.5, 1.0], np.float32)
    temps = np.repeat(t_row[None, :], B, axis=0)
    out = oracle.verify(tgt, drf, np.arange(B, dtype=np.uint64) + 3, T=1.0, temps=temps)
    m = [match_closed_form(softmax(tgt1[0, j], float(t_row[j])), softmax(drf1[0, j], float(t_row[j]))) for j in range(k)]
    m_swapped = [match_closed_form(softmax(tgt1[0, j], float(t_row[1 - j])), softmax(drf1[0, j], float(t_row[1 - j]))) for j in range(k)]
    hit = out["draft_tok"] == out["target_tok"][:, :k]
    for j in range(k):
        sd = math.sqrt(m[j] * (1 - m[j]) / B)
        assert abs(hit[:, j].mean() - m[j]) < 4.5 * sd, (j, hit[:, j].mean(), m[j])
        assert abs(hit[:, j].mean() - m_swapped[j]) > 8 * sd   # the pin can tell the rows apart
