"""Second, separately written statement of the race in numpy (TEST INFRASTRUCTURE).

It follows the paper's own form (Section 3): arrival time t_i = e_i / p_i with
p = softmax(z / T), winner = argmin_i t_i, the first c arrivals = the c smallest
t_i.  It exists to cross-check ``ersd_oracle.c`` (which works with
ln e_i - z_i / T) on small inputs; it shares no code with it and none with the
CUDA library.  Sequence verification follows Algorithm 2 extended per
position; the tree walk follows Algorithm 5.
"""
from __future__ import annotations

import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_MASK = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)


def philox4x32_10(c0, c1, c2, c3, k0: int, k1: int):
    """Vectorised Philox4x32-10 (Salmon et al. 2011); counters are uint32 arrays."""
    c0 = np.asarray(c0, dtype=np.uint64)
    c1 = np.asarray(c1, dtype=np.uint64)
    c2 = np.asarray(c2, dtype=np.uint64)
    c3 = np.asarray(c3, dtype=np.uint64)
    k0 = int(k0) & 0xFFFFFFFF
    k1 = int(k1) & 0xFFFFFFFF
    for _ in range(10):
        prod0 = _M0 * c0
        prod1 = _M1 * c2
        new0 = (prod1 >> _S32) ^ c1 ^ np.uint64(k0)
        new1 = prod1 & _MASK
        new2 = (prod0 >> _S32) ^ c3 ^ np.uint64(k1)
        new3 = prod0 & _MASK
        c0, c1, c2, c3 = new0, new1, new2, new3
        k0 = (k0 + _W0) & 0xFFFFFFFF
        k1 = (k1 + _W1) & 0xFFFFFFFF
    return [a.astype(np.uint32) for a in (c0, c1, c2, c3)]


def race_exponentials(V: int, seed: int, seq_id: int, position: int) -> np.ndarray:
    """e_i for i < V: token i owns word i mod 4 of the block with counter (i div 4, pos, seq, 0)."""
    nblk = (V + 3) // 4
    blk = np.arange(nblk, dtype=np.uint64)
    z = np.zeros(nblk, dtype=np.uint64)
    words = philox4x32_10(blk, z + np.uint64(position), z + np.uint64(seq_id), z,
                          seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    x = np.stack(words, axis=1).reshape(-1)[:V].astype(np.float64)
    w = (x + 0.5) / 4294967296.0
    return -np.log1p(-w)


def arrival_times(z: np.ndarray, T: float, seed: int, seq_id: int, position: int) -> np.ndarray:
    z = np.asarray(z, dtype=np.float64)
    z = np.where(np.isnan(z), -np.inf, z)
    s = z / T
    p = np.exp(s - s.max())
    p = p / p.sum()
    e = race_exponentials(z.shape[0], seed, seq_id, position)
    with np.errstate(divide="ignore"):
        return np.where(p > 0, e / np.where(p > 0, p, 1.0), np.inf)


def first_arrivals(t: np.ndarray, c: int) -> np.ndarray:
    order = np.argsort(t, kind="stable")  # stable: equal times by ascending token id
    out = np.full(c, -1, dtype=np.int64)
    for r in range(min(c, t.shape[0])):
        if np.isfinite(t[order[r]]):
            out[r] = order[r]
    return out


def _temperature(T: float, temps, b: int, r: int) -> float:
    """Temperature of row r of sequence b: temps[b][r] where a table is given, else T.  The
    draft row and the target row of a position are raced at the same temperature."""
    return float(T) if temps is None else float(temps[b][r])


def verify(target: np.ndarray, draft: np.ndarray, seeds, T: float, temps=None):
    B, rows, V = target.shape
    k = rows - 1
    tokens = np.full((B, rows), -1, dtype=np.int64)
    accept = np.zeros(B, dtype=np.int64)
    for b in range(B):
        L = 0
        for j in range(rows):
            Tj = _temperature(T, temps, b, j)
            tp = first_arrivals(arrival_times(target[b, j], Tj, int(seeds[b]), b, j), 1)[0]
            tokens[b, j] = tp
            if j == k:
                break
            tq = first_arrivals(arrival_times(draft[b, j], Tj, int(seeds[b]), b, j), 1)[0]
            if tq != tp or tp < 0:
                break
            L += 1
        accept[b] = L
    return tokens, accept


def verify_tree(target: np.ndarray, draft: np.ndarray, parent, seeds, T: float, temps=None):
    B, nodes, V = target.shape
    children = [[] for _ in range(nodes)]
    for m in range(1, nodes):
        children[parent[m]].append(m)
    out = []
    for b in range(B):
        y, cur = [], 0
        while True:
            Tn = _temperature(T, temps, b, cur)
            w = first_arrivals(arrival_times(target[b, cur], Tn, int(seeds[b]), b, cur), 1)[0]
            y.append(int(w))
            nxt = None
            if children[cur] and w >= 0:
                arr = first_arrivals(arrival_times(draft[b, cur], Tn, int(seeds[b]), b, cur),
                                     len(children[cur]))
                for r, m in enumerate(children[cur]):
                    if arr[r] == w:
                        nxt = m
            if nxt is None:
                break
            cur = nxt
        out.append(y)
    return out
