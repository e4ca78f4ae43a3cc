"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test names the statement it checks.  None of them compares the oracle with
the CUDA library: these are the checks that make the oracle trustworthy before
any kernel is compared with it.
"""
import itertools
import math
import os

import numpy as np
import pytest
from scipy import stats

import oracle
from oracle import ersd_oracle_np as onp

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def softmax(z, T=1.0):
    s = np.asarray(z, dtype=np.float64) / T
    p = np.exp(s - s.max())
    return p / p.sum()


# ----------------------------------------------------------------------------- Philox
def test_philox_known_answers():
    """Published Philox4x32-10 vectors (Salmon et al. 2011, Random123 known-answer table)."""
    n = 0
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(t, 16) for t in line.split()]
        got = oracle.philox4x32_10(w[0:4], w[4:6])
        assert [int(g) for g in got] == w[6:10]
        got_np = onp.philox4x32_10([w[0]], [w[1]], [w[2]], [w[3]], w[4], w[5])
        assert [int(g[0]) for g in got_np] == w[6:10]
        n += 1
    assert n == 3


def test_philox_two_separately_written_versions_agree():
    rng = np.random.default_rng(7)
    ctr = rng.integers(0, 2**32, size=(4000, 4), dtype=np.uint64)
    key = rng.integers(0, 2**32, size=2, dtype=np.uint64)
    ref = onp.philox4x32_10(ctr[:, 0], ctr[:, 1], ctr[:, 2], ctr[:, 3], int(key[0]), int(key[1]))
    for n in range(0, 4000, 37):
        got = oracle.philox4x32_10(ctr[n], key)
        assert [int(g) for g in got] == [int(ref[j][n]) for j in range(4)]


def test_token_word_layout():
    """Token i owns word i & 3 of the block with counter (i >> 2, position, sequence, 0),
    key = (low, high) half of the seed."""
    seed, seq, pos = 0x0123456789ABCDEF, 5, 77
    for i in (0, 1, 2, 3, 4, 7, 1023, 128255):
        block = oracle.philox4x32_10([i >> 2, pos, seq, 0], [seed & 0xFFFFFFFF, seed >> 32])
        assert oracle.token_word(seed, seq, pos, i) == int(block[i & 3])
    # distinct positions / sequences / seeds give distinct streams
    base = [oracle.token_word(seed, seq, pos, i) for i in range(64)]
    assert base != [oracle.token_word(seed, seq, pos + 1, i) for i in range(64)]
    assert base != [oracle.token_word(seed, seq + 1, pos, i) for i in range(64)]
    assert base != [oracle.token_word(seed + 1, seq, pos, i) for i in range(64)]
    assert base != [oracle.token_word(seed + (1 << 32), seq, pos, i) for i in range(64)]


# ----------------------------------------------------------------------------- Exp(1) variate
def test_exp_variate_inverts_the_exponential_cdf():
    """e solves 1 - exp(-e) = (x + 1/2) / 2^32 (inverse-CDF sampling of Exp(1), Section 3)."""
    for x in (0, 1, 2, 255, 2**16, 2**23 + 1, 2**31, 2**32 - 2, 2**32 - 1):
        e = oracle.exp_variate(x)
        w = (x + 0.5) / 2**32
        assert -math.expm1(-e) == pytest.approx(w, rel=1e-14)
    assert oracle.exp_variate(0) == pytest.approx(0.5 / 2**32, rel=1e-9)
    assert oracle.exp_variate(2**32 - 1) == pytest.approx(33 * math.log(2), rel=1e-9)
    xs = [0, 5, 1000, 2**20, 2**31, 2**32 - 1]
    es = [oracle.exp_variate(x) for x in xs]
    assert es == sorted(es) and len(set(es)) == len(es)


def test_race_exponentials_are_exp1():
    """Kolmogorov-Smirnov and moments of 4e5 race variables against Exp(1)."""
    n = 400_000
    keys = oracle.row_keys(np.zeros(n, np.float32), 1.0, seed=12345, seq_id=3, position=9)
    e = np.exp(keys)  # logits are zero, so key = ln e
    assert stats.kstest(e, "expon").pvalue > 1e-3
    assert abs(e.mean() - 1.0) < 4 / math.sqrt(n)
    assert abs(e.var() - 1.0) < 4 * math.sqrt(8.0 / n)
    # independence across tokens: lag-1 correlation vanishes
    assert abs(np.corrcoef(e[:-1], e[1:])[0, 1]) < 4 / math.sqrt(n)
    # the separately written numpy version draws the same variables
    np.testing.assert_allclose(onp.race_exponentials(4096, 12345, 3, 9), e[:4096], rtol=1e-12)


# ----------------------------------------------------------------------------- winner law
@pytest.mark.parametrize("V,T", [(2, 1.0), (3, 0.7), (4, 1.0), (8, 1.3)])
def test_winner_follows_softmax(V, T):
    """Losslessness (Section 3): the race winner under P is distributed exactly as P."""
    rng = np.random.default_rng(100 + V)
    z = (rng.normal(size=V) * 1.5).astype(np.float32)
    R = 300_000
    tok, _ = oracle.race_sample(z, seeds=[999 + V], T=T, broadcast_rows=R)
    counts = np.bincount(tok.reshape(-1), minlength=V)
    assert counts.sum() == R
    chi = stats.chisquare(counts, softmax(z, T) * R)
    assert chi.pvalue > 1e-3, (counts / R, softmax(z, T))


def test_winner_law_rejects_a_wrong_sign_or_missing_temperature():
    """The chi-square pin has teeth: the same counts do not fit softmax(-z/T) or softmax(z)."""
    z = np.array([0.3, -1.2, 1.1, 0.0], np.float32)
    R, T = 300_000, 0.5
    tok, _ = oracle.race_sample(z, seeds=[4242], T=T, broadcast_rows=R)
    counts = np.bincount(tok.reshape(-1), minlength=4)
    assert stats.chisquare(counts, softmax(z, T) * R).pvalue > 1e-3
    assert stats.chisquare(counts, softmax(-z, T) * R).pvalue < 1e-12
    assert stats.chisquare(counts, softmax(z, 1.0) * R).pvalue < 1e-12


def test_arrival_order_is_plackett_luce():
    """The ordered arrivals are a sample without replacement from Q (Appendix A, remark after
    Algorithm 4): Pr{order} = prod_r q_(r) / (1 - q_(1) - ... - q_(r-1)).  V = 4, all 24 orders."""
    z = np.array([0.8, -0.5, 0.1, 1.4], np.float32)
    q = softmax(z)
    R = 400_000
    tok, key = oracle.race_sample(z, seeds=[77], T=1.0, c=4, broadcast_rows=R)
    tok = tok.reshape(R, 4)
    assert (np.sort(tok, axis=1) == np.arange(4)).all()          # distinct: no replacement
    assert (np.diff(key.reshape(R, 5)[:, :4], axis=1) >= 0).all()  # ascending arrival keys
    code = (tok * np.array([64, 16, 4, 1])).sum(axis=1)
    expected, observed = [], []
    for perm in itertools.permutations(range(4)):
        pr, rest = 1.0, 1.0
        for i in perm:
            pr *= q[i] / rest
            rest -= q[i]
        expected.append(pr * R)
        observed.append(int((code == sum(v * m for v, m in zip(perm, (64, 16, 4, 1)))).sum()))
    assert sum(observed) == R
    assert stats.chisquare(observed, expected).pvalue > 1e-3


# ----------------------------------------------------------------------------- coupling
def match_closed_form(p, q):
    """Pr{I_P = I_Q} = sum_i 1 / sum_j max(p_j/p_i, q_j/q_i): integrate exp(-e_i) times
    prod_{j != i} Pr{e_j >= e_i max(p_j/p_i, q_j/q_i)} over e_i (shared e, Section 3)."""
    return sum(1.0 / np.maximum(p / p[i], q / q[i]).sum() for i in range(len(p)))


def coupled_winners(zp, zq, R, seed, T=1.0):
    tp, _ = oracle.race_sample(zp, seeds=[seed], T=T, broadcast_rows=R)
    tq, _ = oracle.race_sample(zq, seeds=[seed], T=T, broadcast_rows=R)
    return tp.reshape(-1), tq.reshape(-1)


@pytest.mark.parametrize("V,spread", [(3, 0.5), (8, 1.0), (16, 2.0)])
def test_coupling_match_rate_and_lemma_bounds(V, spread):
    """Shared randomness: match rate equals the closed form and lies inside the bounds of the
    first-arrival lemma, D_HM[P,Q] <= Pr{accept} <= 1 - D_TV[P,Q]."""
    rng = np.random.default_rng(V)
    zp = rng.normal(size=V).astype(np.float32)
    zq = (zp + spread * rng.normal(size=V)).astype(np.float32)
    p, q = softmax(zp), softmax(zq)
    R = 400_000
    tp, tq = coupled_winners(zp, zq, R, seed=31337 + V)
    rate = (tp == tq).mean()
    m = match_closed_form(p, q)
    assert abs(rate - m) < 4 * math.sqrt(m * (1 - m) / R)
    d_hm = (p * q / (p + q)).sum()
    d_tv = 0.5 * np.abs(p - q).sum()
    assert d_hm - 1e-12 <= m <= 1 - d_tv + 1e-12
    assert d_hm - 4 / math.sqrt(R) < rate < 1 - d_tv + 4 / math.sqrt(R)
    # both marginals stay exact under the coupling
    assert stats.chisquare(np.bincount(tp, minlength=V), p * R).pvalue > 1e-3
    assert stats.chisquare(np.bincount(tq, minlength=V), q * R).pvalue > 1e-3


def test_poisson_matching_lemma_conditional_bound():
    """Pr{I_P != I_Q | I_Q = i} <= 1 - (1 + q_i / p_i)^-1 (Appendix B), and the exact
    conditional value 1 - (1/q_i) / sum_j max(p_j/p_i, q_j/q_i)."""
    rng = np.random.default_rng(5)
    V = 6
    zp = rng.normal(size=V).astype(np.float32)
    zq = (zp + rng.normal(size=V)).astype(np.float32)
    p, q = softmax(zp), softmax(zq)
    R = 600_000
    tp, tq = coupled_winners(zp, zq, R, seed=2024)
    for i in range(V):
        sel = tq == i
        n = int(sel.sum())
        miss = (tp[sel] != i).mean()
        bound = 1 - 1 / (1 + q[i] / p[i])
        exact = 1 - (1 / np.maximum(p / p[i], q / q[i]).sum()) / q[i]
        assert exact <= bound + 1e-12
        assert abs(miss - exact) < 4.5 * math.sqrt(max(exact * (1 - exact), 1e-4) / n)
        assert miss <= bound + 4.5 / math.sqrt(n)


def test_identical_laws_always_match():
    z = np.random.default_rng(1).normal(size=50).astype(np.float32)
    tp, tq = coupled_winners(z, z.copy(), 20_000, seed=8)
    assert (tp == tq).all()


def test_different_positions_are_independent_races():
    """One race per drafted position (Section 3): winners at two positions are independent."""
    z = np.array([0.0, 0.4, -0.3], np.float32)
    R = 200_000
    tok, _ = oracle.race_sample(z, seeds=[3], T=1.0, broadcast_rows=2 * R)
    a, b = tok.reshape(-1)[0::2], tok.reshape(-1)[1::2]
    table = np.zeros((3, 3))
    np.add.at(table, (a, b), 1)
    assert stats.chi2_contingency(table)[1] > 1e-3


# ----------------------------------------------------------------------------- log form = definition
@pytest.mark.parametrize("V", [1, 2, 5, 64, 1000, 4096])
def test_log_form_equals_definition_form(V):
    """argmin_i (ln e_i - z_i/T) = argmin_i e_i / softmax(z/T)_i, and the keys differ from
    ln t_i by the constant -ln Z."""
    rng = np.random.default_rng(V)
    z = (-1.1 * np.log(rng.permutation(V) + 1.0) + rng.normal(size=V)).astype(np.float32)
    for T in (0.6, 1.0):
        c = min(V, 5)
        tok_l, key_l = oracle.race_sample(z.reshape(1, 1, V).repeat(40, axis=1), seeds=[V], T=T, c=c)
        tok_d, t_d = oracle.race_sample_def(z.reshape(1, 1, V).repeat(40, axis=1), seeds=[V], T=T, c=c)
        assert (tok_l == tok_d).all()
        diff = key_l[..., :c] - np.log(t_d[..., :c])
        assert np.ptp(diff) < 1e-9
        s = z.astype(np.float64) / float(np.float32(T))  # the interface carries T as fp32
        ln_z = s.max() + math.log(np.exp(s - s.max()).sum())
        assert diff.mean() == pytest.approx(-ln_z, abs=1e-9)


def test_numpy_version_agrees_on_keys_and_winners():
    rng = np.random.default_rng(11)
    V = 777
    z = rng.normal(size=V).astype(np.float32) * 2
    for pos in range(6):
        t = onp.arrival_times(z, 0.8, seed=99, seq_id=2, position=pos)
        keys = oracle.row_keys(z, 0.8, seed=99, seq_id=2, position=pos)
        assert np.argmin(t) == np.argmin(keys)
        tok, _ = oracle.first_arrivals(keys, 4)
        assert list(onp.first_arrivals(t, 4)) == list(tok)


def test_bf16_rows_are_read_as_their_exact_values():
    import torch
    z = torch.randn(300, generator=torch.Generator().manual_seed(0)) * 3
    zb = z.to(torch.bfloat16)
    bits = zb.view(torch.int16).numpy().view(np.uint16)
    k_bits = oracle.row_keys(bits, 0.9, 5, 0, 0)
    k_f32 = oracle.row_keys(zb.float().numpy(), 0.9, 5, 0, 0)
    assert (k_bits == k_f32).all()


# ----------------------------------------------------------------------------- special values
def test_ties_masks_and_greedy():
    # T == 0: greedy, lowest index among equal maxima
    z = np.array([1.0, 3.0, 3.0, -2.0], np.float32)
    tok, key = oracle.race_sample(z.reshape(1, 1, 4), seeds=[1], T=0.0, c=3)
    assert list(tok.reshape(-1)) == [1, 2, 0] and key[0, 0, 0] == -3.0
    # -inf and NaN never win; a fully masked row gives -1
    z = np.array([-np.inf, np.nan, 0.5, -np.inf], np.float32)
    tok, key = oracle.race_sample(z.reshape(1, 1, 4), seeds=[1], T=1.0, c=2)
    assert list(tok.reshape(-1)) == [2, -1] and np.isinf(key[0, 0, 1])
    z = np.array([-np.inf, np.nan], np.float32)
    tok, key = oracle.race_sample(z.reshape(1, 1, 2), seeds=[1], T=1.0, c=1)
    assert tok.reshape(-1)[0] == -1 and np.isinf(key[0, 0, 0])
    # +inf logit always wins, lowest index first
    z = np.array([0.0, np.inf, np.inf], np.float32)
    tok, _ = oracle.race_sample(z.reshape(1, 1, 3), seeds=[1], T=1.0, c=2)
    assert list(tok.reshape(-1)) == [1, 2]
    # exact key ties go to the lowest token id
    tok, _ = oracle.first_arrivals(np.array([2.0, 1.0, 1.0, 1.0, 3.0]), 4)
    assert list(tok) == [1, 2, 3, 0]
