"""ctypes front end of the fp64 CPU oracle (TEST INFRASTRUCTURE, not product code).

Only the tests, the smoke check and the benchmark's CPU-baseline leg import
this package.  It compiles ``ersd_oracle.c`` with gcc on first use and exposes
its functions on numpy arrays.  Logit arrays are float32 or, for bf16, the raw
16-bit patterns as uint16.  Nothing here touches the CUDA library.

What each function computes is stated, with the passage of the paper it
follows, in ``ersd_oracle.c``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ersd_oracle.c")
_LIB = os.path.join(_HERE, "libersd_oracle.so")

F32, BF16 = 0, 1
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle into a shared object next to its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-shared", "-fPIC",
                           "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.ersd_oracle_exp_variate.restype = C.c_double
        _lib.ersd_oracle_exp_variate.argtypes = [C.c_uint32]
        _lib.ersd_oracle_token_word.restype = C.c_uint32
        _lib.ersd_oracle_token_word.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32]
        _lib.ersd_oracle_max_threads.restype = C.c_int
        _lib.ersd_oracle_gsd_uniform.restype = C.c_double
        _lib.ersd_oracle_gsd_uniform.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32]
    return _lib


def max_threads() -> int:
    return int(lib().ersd_oracle_max_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dtype_of(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError("logits must be float32 or uint16 (bf16 bit patterns), got %s" % a.dtype)


def _opt(a, dtype):
    return None if a is None else np.ascontiguousarray(a, dtype=dtype)


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().ersd_oracle_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def exp_variate(x: int) -> float:
    return float(lib().ersd_oracle_exp_variate(C.c_uint32(int(x))))


def token_word(seed: int, seq_id: int, position: int, i: int) -> int:
    return int(lib().ersd_oracle_token_word(C.c_uint64(int(seed)), C.c_uint32(int(seq_id)),
                                            C.c_uint32(int(position)), C.c_uint32(int(i))))


def row_keys(row: np.ndarray, T: float, seed: int, seq_id: int, position: int) -> np.ndarray:
    row = np.ascontiguousarray(row)
    keys = np.empty(row.shape[0], dtype=np.float64)
    lib().ersd_oracle_row_keys(_p(row), C.c_int(_dtype_of(row)), C.c_int(row.shape[0]),
                               C.c_double(float(T)), C.c_uint64(int(seed)),
                               C.c_uint32(int(seq_id)), C.c_uint32(int(position)), _p(keys))
    return keys


def row_times_def(row: np.ndarray, T: float, seed: int, seq_id: int, position: int) -> np.ndarray:
    row = np.ascontiguousarray(row)
    t = np.empty(row.shape[0], dtype=np.float64)
    lib().ersd_oracle_row_times_def(_p(row), C.c_int(_dtype_of(row)), C.c_int(row.shape[0]),
                                    C.c_double(float(T)), C.c_uint64(int(seed)),
                                    C.c_uint32(int(seq_id)), C.c_uint32(int(position)), _p(t))
    return t


def first_arrivals(keys: np.ndarray, c: int):
    keys = np.ascontiguousarray(keys, dtype=np.float64)
    tok = np.empty(c, dtype=np.int32)
    key = np.empty(c + 1, dtype=np.float64)
    lib().ersd_oracle_first_arrivals(_p(keys), C.c_int(keys.shape[0]), C.c_int(c), _p(tok), _p(key))
    return tok, key


def race_sample(logits: np.ndarray, seeds, T: float = 1.0, c: int = 1, temps=None,
                seq_ids=None, pos_offsets=None, broadcast_rows: int | None = None):
    """logits [B, R, V] (or one row [V] raced ``broadcast_rows`` times as B=1, R=rows).

    Returns (tok [B, R, c] int32, key [B, R, c+1] float64).
    """
    logits = np.ascontiguousarray(logits)
    if broadcast_rows is not None:
        assert logits.ndim == 1
        B, R, V = 1, int(broadcast_rows), logits.shape[0]
        sb, sr = 0, 0
    else:
        B, R, V = logits.shape
        sb, sr = R * V, V
    seeds = np.ascontiguousarray(seeds, dtype=np.uint64)
    assert seeds.shape == (B,)
    temps = _opt(temps, np.float32)
    if temps is not None:
        assert temps.shape == (B, R)
    seq_ids = _opt(seq_ids, np.uint32)
    pos_offsets = _opt(pos_offsets, np.uint32)
    tok = np.empty((B, R, c), dtype=np.int32)
    key = np.empty((B, R, c + 1), dtype=np.float64)
    lib().ersd_oracle_race_sample(
        _p(logits), C.c_int(_dtype_of(logits)), C.c_int64(sb), C.c_int64(sr), _p(seeds),
        _p(seq_ids), _p(pos_offsets), C.c_int(B), C.c_int(R), C.c_int(V), C.c_float(float(T)),
        _p(temps), C.c_int64(R), C.c_int64(1), C.c_int(c), _p(tok), _p(key))
    return tok, key


def race_sample_def(logits: np.ndarray, seeds, T: float = 1.0, c: int = 1,
                    broadcast_rows: int | None = None):
    """Same races in the paper's t = e / softmax(z/T) form (small V)."""
    logits = np.ascontiguousarray(logits)
    if broadcast_rows is not None:
        B, R, V = 1, int(broadcast_rows), logits.shape[0]
        sb, sr = 0, 0
    else:
        B, R, V = logits.shape
        sb, sr = R * V, V
    seeds = np.ascontiguousarray(seeds, dtype=np.uint64)
    tok = np.empty((B, R, c), dtype=np.int32)
    t = np.empty((B, R, c + 1), dtype=np.float64)
    lib().ersd_oracle_race_sample_def(
        _p(logits), C.c_int(_dtype_of(logits)), C.c_int64(sb), C.c_int64(sr), _p(seeds),
        C.c_int(B), C.c_int(R), C.c_int(V), C.c_float(float(T)), C.c_int(c), _p(tok), _p(t))
    return tok, t


def verify(target: np.ndarray, draft: np.ndarray, seeds, T: float = 1.0, temps=None,
           seq_ids=None, pos_offsets=None):
    """target [B, k+1, V], draft [B, k, V] -> dict of the sequence-ERSD results."""
    target = np.ascontiguousarray(target)
    draft = np.ascontiguousarray(draft)
    B, rows, V = target.shape
    k = rows - 1
    assert draft.shape == (B, k, V) and draft.dtype == target.dtype
    seeds = np.ascontiguousarray(seeds, dtype=np.uint64)
    assert seeds.shape == (B,)
    temps = _opt(temps, np.float32)
    if temps is not None:
        assert temps.shape == (B, rows)
    seq_ids = _opt(seq_ids, np.uint32)
    pos_offsets = _opt(pos_offsets, np.uint32)
    out = dict(
        tokens=np.empty((B, rows), np.int32), accept_len=np.empty(B, np.int32),
        draft_tok=np.empty((B, k), np.int32), target_tok=np.empty((B, rows), np.int32),
        draft_key=np.empty((B, k, 2), np.float64), target_key=np.empty((B, rows, 2), np.float64))
    lib().ersd_oracle_verify(
        _p(target), _p(draft), C.c_int(_dtype_of(target)), C.c_int64(V), C.c_int64(V), _p(seeds),
        _p(seq_ids), _p(pos_offsets), C.c_int(B), C.c_int(k), C.c_int(V), C.c_float(float(T)),
        _p(temps), C.c_int64(rows), C.c_int64(1), _p(out["tokens"]), _p(out["accept_len"]),
        _p(out["draft_tok"]), _p(out["target_tok"]), _p(out["draft_key"]), _p(out["target_key"]))
    return out


def verify_tokens(target: np.ndarray, draft_tokens: np.ndarray, seeds, T: float = 1.0, temps=None,
                  seq_ids=None, pos_offsets=None):
    """Verification when the drafted tokens are given (Algorithm 2's verification lines, extended
    to a drafted sequence as Section 3 describes: accept in order until the first rejection).

    target [B, k+1, V]; draft_tokens [B, k] (token drafted at position j, i.e. the draft row's race
    winner under the SAME race variables, produced earlier).  Position j's target winner is
    argmin_i e_i / p_i with that position's race; position j is accepted iff it equals
    draft_tokens[b, j]; the output is the target winners up to and including the first
    rejection (or the extra token of position k when all k are accepted).
    Returns dict(tokens [B, k+1] (-1 padded), accept_len [B], target_tok, target_key [B, k+1, 2]).
    """
    target = np.ascontiguousarray(target)
    B, rows, V = target.shape
    k = rows - 1
    draft_tokens = np.asarray(draft_tokens)
    assert draft_tokens.shape == (B, k)
    tok, key = race_sample(target, seeds, T=T, c=1, temps=temps, seq_ids=seq_ids, pos_offsets=pos_offsets)
    ttok = tok[..., 0]
    tokens = np.full((B, rows), -1, np.int32)
    accept = np.zeros(B, np.int32)
    for b in range(B):
        L = 0
        while L < k and ttok[b, L] >= 0 and ttok[b, L] == draft_tokens[b, L]:
            L += 1
        tokens[b, :L + 1] = ttok[b, :L + 1]
        accept[b] = L
    return dict(tokens=tokens, accept_len=accept, target_tok=ttok.astype(np.int32), target_key=key)


def tree_shape(parent):
    """(depth D, max children, children counts, sibling ranks) of a parent array."""
    parent = np.asarray(parent, dtype=np.int64)
    n = parent.shape[0]
    depth = np.zeros(n, np.int64)
    nchild = np.zeros(n, np.int64)
    rank = np.zeros(n, np.int64)
    for m in range(1, n):
        assert 0 <= parent[m] < m
        depth[m] = depth[parent[m]] + 1
        rank[m] = nchild[parent[m]]
        nchild[parent[m]] += 1
    return int(depth.max()), int(max(1, nchild.max())), nchild, rank


def verify_tree(target: np.ndarray, draft: np.ndarray, parent, seeds, T: float = 1.0,
                temps=None, seq_ids=None, pos_offsets=None):
    """target, draft [B, N+1, V]; parent [N+1] with parent[0] = -1 -> dict of tree-ERSD results."""
    target = np.ascontiguousarray(target)
    draft = np.ascontiguousarray(draft)
    B, nodes, V = target.shape
    assert draft.shape == target.shape and draft.dtype == target.dtype
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    assert parent.shape == (nodes,) and parent[0] == -1
    D, max_c, _, _ = tree_shape(parent)
    seeds = np.ascontiguousarray(seeds, dtype=np.uint64)
    temps = _opt(temps, np.float32)
    if temps is not None:
        assert temps.shape == (B, nodes)
    seq_ids = _opt(seq_ids, np.uint32)
    pos_offsets = _opt(pos_offsets, np.uint32)
    out = dict(
        tokens=np.empty((B, D + 1), np.int32), accept_len=np.empty(B, np.int32),
        path=np.empty((B, D + 1), np.int32), arrivals=np.empty((B, nodes, max_c), np.int32),
        target_tok=np.empty((B, nodes), np.int32),
        arrival_key=np.empty((B, nodes, max_c + 1), np.float64),
        target_key=np.empty((B, nodes, 2), np.float64), depth=D, max_children=max_c)
    lib().ersd_oracle_verify_tree(
        _p(target), _p(draft), C.c_int(_dtype_of(target)), C.c_int64(V), C.c_int64(V),
        _p(parent), _p(seeds), _p(seq_ids), _p(pos_offsets), C.c_int(B), C.c_int(nodes - 1),
        C.c_int(V), C.c_float(float(T)), _p(temps), C.c_int64(nodes), C.c_int64(1), C.c_int(D),
        C.c_int(max_c), _p(out["tokens"]), _p(out["accept_len"]), _p(out["path"]),
        _p(out["arrivals"]), _p(out["target_tok"]), _p(out["arrival_key"]), _p(out["target_key"]))
    return out


def gsd_uniform(seed: int, seq_id: int, node: int, rank: int = 0) -> float:
    """The uniform of the ratio test of child `rank` of node (or position) `node`."""
    return float(lib().ersd_oracle_gsd_uniform(C.c_uint64(int(seed)), C.c_uint32(int(seq_id)),
                                               C.c_uint32(int(node)), C.c_uint32(int(rank))))


def gsd_verify(target: np.ndarray, draft: np.ndarray, draft_tokens, seeds, T: float = 1.0, temps=None,
               seq_ids=None, pos_offsets=None):
    """Sequence GSD (Algorithm 1 position by position).  target [B, k+1, V], draft [B, k, V],
    draft_tokens [B, k] -> dict(tokens [B, k+1] (-1 padded), accept_len [B], ratio, unif [B, k],
    last_times [B, 2])."""
    target = np.ascontiguousarray(target)
    draft = np.ascontiguousarray(draft)
    B, rows, V = target.shape
    k = rows - 1
    assert draft.shape == (B, k, V) and draft.dtype == target.dtype
    tok = np.ascontiguousarray(draft_tokens, dtype=np.int32)
    assert tok.shape == (B, k)
    seeds = np.ascontiguousarray(seeds, dtype=np.uint64)
    temps = _opt(temps, np.float32)
    if temps is not None:
        assert temps.shape == (B, rows)
    seq_ids = _opt(seq_ids, np.uint32)
    pos_offsets = _opt(pos_offsets, np.uint32)
    out = dict(tokens=np.empty((B, rows), np.int32), accept_len=np.empty(B, np.int32),
               ratio=np.empty((B, k), np.float64), unif=np.empty((B, k), np.float64),
               last_times=np.full((B, 2), np.inf))
    lib().ersd_oracle_gsd_verify(
        _p(target), _p(draft), _p(tok), C.c_int(_dtype_of(target)), _p(seeds), _p(seq_ids), _p(pos_offsets),
        C.c_int(B), C.c_int(k), C.c_int(V), C.c_float(float(T)), _p(temps), C.c_int64(rows), C.c_int64(1),
        _p(out["tokens"]), _p(out["accept_len"]), _p(out["ratio"]), _p(out["unif"]), _p(out["last_times"]))
    return out


def gsd_verify_tree(target: np.ndarray, draft: np.ndarray, draft_tokens, parent, seeds, T: float = 1.0,
                    temps=None, seq_ids=None, pos_offsets=None):
    """Tree GSD (Algorithm 4).  target, draft [B, N+1, V]; draft_tokens [B, N+1] (entry 0 unused);
    parent [N+1] -> dict(tokens [B, D+1], accept_len [B], path [B, D+1], last_times [B, 2])."""
    target = np.ascontiguousarray(target)
    draft = np.ascontiguousarray(draft)
    B, nodes, V = target.shape
    assert draft.shape == target.shape and draft.dtype == target.dtype
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    D, _, _, _ = tree_shape(parent)
    tok = np.ascontiguousarray(draft_tokens, dtype=np.int32)
    assert tok.shape == (B, nodes)
    seeds = np.ascontiguousarray(seeds, dtype=np.uint64)
    temps = _opt(temps, np.float32)
    seq_ids = _opt(seq_ids, np.uint32)
    pos_offsets = _opt(pos_offsets, np.uint32)
    out = dict(tokens=np.empty((B, D + 1), np.int32), accept_len=np.empty(B, np.int32),
               path=np.empty((B, D + 1), np.int32), last_times=np.full((B, 2), np.inf), depth=D)
    lib().ersd_oracle_gsd_verify_tree(
        _p(target), _p(draft), _p(tok), C.c_int(_dtype_of(target)), _p(parent), _p(seeds), _p(seq_ids),
        _p(pos_offsets), C.c_int(B), C.c_int(nodes - 1), C.c_int(V), C.c_float(float(T)), _p(temps),
        C.c_int64(nodes), C.c_int64(1), C.c_int(D), _p(out["tokens"]), _p(out["accept_len"]), _p(out["path"]),
        _p(out["last_times"]))
    return out
