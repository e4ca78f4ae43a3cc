"""Comparison of libersd's results with the CPU oracle's (used by the GPU tests and the smoke check).

Bar: tokens and accept lengths bit-equal.  The one allowed exception is a row
whose two best oracle keys differ by less than NEAR_TIE (natural-log units, i.e.
relative 1e-5 in arrival time): there either of the two may win; such rows are
counted and returned.  Winner keys must agree within KEY_TOL absolute.
"""
from __future__ import annotations

import numpy as np

import oracle
from paper_2504_15475_b200 import workloads as wl

NEAR_TIE = 1e-5
KEY_TOL = 2e-5


def _cmp_rows(name, got_tok, got_key, ref_tok, ref_key_pairs):
    """Per-row winners: returns the boolean mask of near-tie rows where the tokens differ."""
    got_tok = np.asarray(got_tok)
    ref_tok = np.asarray(ref_tok)
    gap = ref_key_pairs[..., 1] - ref_key_pairs[..., 0]
    differ = got_tok != ref_tok
    bad = differ & ~(gap < NEAR_TIE)
    assert not bad.any(), "%s: %d winners differ outside near-ties, first at %s (gpu %s, oracle %s, gap %s)" % (
        name, int(bad.sum()), np.argwhere(bad)[0], got_tok[bad][0], ref_tok[bad][0], gap[bad][0])
    if got_key is not None:
        same = ~differ & (ref_tok >= 0)
        err = np.abs(np.asarray(got_key, dtype=np.float64)[same] - ref_key_pairs[..., 0][same])
        finite = np.isfinite(ref_key_pairs[..., 0][same])
        assert (err[finite] <= KEY_TOL).all(), "%s: winner key off by %g" % (name, err[finite].max())
        missing = ~differ & (ref_tok < 0)
        assert np.isinf(np.asarray(got_key)[missing]).all()
    return differ


def check_verify(inp, out, seq_ids=None, pos_offsets=None):
    """inp: dict from workloads.make_inputs (any device); out: dict from binding.verify(want_rows=True).
    Returns the number of near-tie rows on which GPU and oracle legitimately differ."""
    tgt = wl.as_numpy_logits(inp["target"])
    drf = wl.as_numpy_logits(inp["draft"])
    seeds = wl.seeds_as_u64(inp["seeds"])
    temps = None if inp.get("temps") is None else inp["temps"].cpu().numpy()
    g = {k: v.cpu().numpy() for k, v in out.items()}
    if inp.get("parent") is None:
        ref = oracle.verify(tgt, drf, seeds, T=inp["T"], temps=temps, seq_ids=seq_ids,
                            pos_offsets=pos_offsets)
        d1 = _cmp_rows("target", g["target_tok"], g["target_key"], ref["target_tok"], ref["target_key"])
        d2 = _cmp_rows("draft", g["draft_tok"], g["draft_key"], ref["draft_tok"], ref["draft_key"])
        flips = int(d1.sum() + d2.sum())
        B, rows = ref["tokens"].shape
        k = rows - 1
        for b in range(B):
            if d1[b].any() or d2[b].any():
                # near-tie in this sequence: the scan must be right for the winners the GPU chose
                tt, dt = g["target_tok"][b], g["draft_tok"][b]
                L = 0
                while L < k and tt[L] >= 0 and dt[L] == tt[L]:
                    L += 1
                exp = np.where(np.arange(rows) <= L, tt, -1)
                assert g["accept_len"][b] == L and (g["tokens"][b] == exp).all()
            else:
                assert g["accept_len"][b] == ref["accept_len"][b], (b, g["accept_len"][b], ref["accept_len"][b])
                assert (g["tokens"][b] == ref["tokens"][b]).all(), (b, g["tokens"][b], ref["tokens"][b])
        return flips
    parent = inp["parent"]
    ref = oracle.verify_tree(tgt, drf, parent, seeds, T=inp["T"], temps=temps, seq_ids=seq_ids,
                             pos_offsets=pos_offsets)
    D, max_c, nchild, rank = oracle.tree_shape(parent)
    d1 = _cmp_rows("target", g["target_tok"], g["target_key"], ref["target_tok"], ref["target_key"])
    B, nodes = ref["target_tok"].shape
    # token drafted at node n = arrival rank[n] of its parent's race
    ref_dtok = np.full((B, nodes), -1, np.int32)
    ref_dkey = np.full((B, nodes, 2), np.inf)
    for n in range(1, nodes):
        ref_dtok[:, n] = ref["arrivals"][:, parent[n], rank[n]]
        ref_dkey[:, n, 0] = ref["arrival_key"][:, parent[n], rank[n]]
        # a near-tie with either neighbour in the arrival order may swap this slot
        nxt = ref["arrival_key"][:, parent[n], rank[n] + 1]
        gap = nxt - ref_dkey[:, n, 0]
        if rank[n] > 0:
            gap = np.minimum(gap, ref_dkey[:, n, 0] - ref["arrival_key"][:, parent[n], rank[n] - 1])
        ref_dkey[:, n, 1] = ref_dkey[:, n, 0] + gap
    d2 = _cmp_rows("draft", g["draft_tok"][:, 1:], g["draft_key"][:, 1:], ref_dtok[:, 1:], ref_dkey[:, 1:])
    assert (g["draft_tok"][:, 0] == -1).all()
    flips = int(d1.sum() + d2.sum())
    for b in range(B):
        if d1[b].any() or d2[b].any():
            # near-tie in this sequence: the walk must be right for the winners the GPU chose
            tt, dt = g["target_tok"][b], g["draft_tok"][b]
            cur, toks, path = 0, [], []
            while True:
                toks.append(int(tt[cur]))
                path.append(cur)
                nxt = [m for m in range(1, nodes) if parent[m] == cur and tt[cur] >= 0 and dt[m] == tt[cur]]
                if not nxt:
                    break
                cur = nxt[0]
            L = len(toks) - 1
            assert g["accept_len"][b] == L
            assert list(g["tokens"][b, :L + 1]) == toks and (g["tokens"][b, L + 1:] == -1).all()
            assert list(g["path"][b, :L + 1]) == path and (g["path"][b, L + 1:] == -1).all()
            continue
        assert g["accept_len"][b] == ref["accept_len"][b]
        assert (g["tokens"][b] == ref["tokens"][b]).all(), (b, g["tokens"][b], ref["tokens"][b])
        assert (g["path"][b] == ref["path"][b]).all()
    return flips


def check_sample(logits, seeds, T, got_tok, got_key, c=1, temps=None, seq_ids=None, pos_offsets=None):
    ref_tok, ref_key = oracle.race_sample(wl.as_numpy_logits(logits), wl.seeds_as_u64(seeds), T=T, c=c,
                                          temps=temps, seq_ids=seq_ids, pos_offsets=pos_offsets)
    got_tok = got_tok.cpu().numpy()
    got_key = None if got_key is None else got_key.cpu().numpy()
    gaps = np.diff(ref_key, axis=-1)                     # gap to the next arrival, per slot
    gap = gaps.copy()
    gap[..., 1:] = np.minimum(gaps[..., 1:], gaps[..., :-1])  # or to the previous one
    pairs = np.stack([ref_key[..., :c], ref_key[..., :c] + gap], axis=-1)
    differ = _cmp_rows("sample", got_tok, got_key, ref_tok, pairs)
    return int(differ.sum())
