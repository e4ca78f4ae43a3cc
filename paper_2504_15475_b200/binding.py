"""Thin ctypes binding of libersd.so: argument marshalling only.

The functions carry the names of the C entry points in ``include/ersd.h`` and
take torch CUDA tensors (used for device memory and the current stream only).
Every step of the computation runs in the library's kernels.  Loading fails
loudly when the library has not been built: there is no CPU path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("ERSD_LIBRARY") or os.path.join(_HERE, "libersd.so")  # ERSD_LIBRARY: another build of libersd

ERSD_F32, ERSD_BF16 = 0, 1
ERSD_OK = 0
ERSD_MAX_TOP_C, ERSD_MAX_ROWS, ERSD_MAX_SPLIT = 64, 256, 32
ERSD_NOALLOC_MAX_ROWS = 1024
ERSD_ENOALLOC_LIMIT = -6

EXPORTS = ("ersd_race_sample", "ersd_verify", "ersd_verify_tokens", "ersd_verify_noalloc", "ersd_verify_tree", "ersd_gsd_verify", "ersd_gsd_verify_tree", "ersd_tree_depth", "ersd_optimal_tree",
           "ersd_acceptance_profile", "ersd_row_keys", "ersd_workspace_bytes", "ersd_workspace_init", "ersd_status_string",
           "ersd_last_cuda_error", "ersd_last_launch", "ersd_version")


class ErsdOpts(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("top_c", C.c_uint32), ("split_v", C.c_uint32),
        ("block_threads", C.c_uint32),
        ("ld_target", C.c_int64), ("ld_draft", C.c_int64),
        ("temps", C.c_void_p), ("temp_stride_b", C.c_int64), ("temp_stride_r", C.c_int64),
        ("seq_ids", C.c_void_p), ("pos_offsets", C.c_void_p),
        ("out_draft_tok", C.c_void_p), ("out_draft_key", C.c_void_p),
        ("out_target_tok", C.c_void_p), ("out_target_key", C.c_void_p),
        ("out_path", C.c_void_p), ("out_key", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("kernel_path", C.c_uint32), ("reserved1", C.c_uint32),
        ("near_tie_count", C.c_void_p),
    ]


class ErsdError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().ersd_status_string(status).decode()
        if status == -4:
            msg += " (cudaError %d)" % lib().ersd_last_cuda_error()
        super().__init__("%s: %s [%d]" % (where, msg, status))


_lib = None


def lib():
    """The loaded library; raises if libersd.so is missing (build it with ``build.py``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libersd.so not found at %s: run `python -m paper_2504_15475_b200.build` "
                               "(there is no CPU fallback)" % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        vp, i, f = C.c_void_p, C.c_int, C.c_float
        L.ersd_race_sample.argtypes = [vp, i, vp, i, i, i, f, vp, C.POINTER(ErsdOpts), vp]
        L.ersd_verify.argtypes = [vp, vp, i, vp, i, i, i, f, vp, vp, C.POINTER(ErsdOpts), vp]
        L.ersd_verify_noalloc.argtypes = L.ersd_verify.argtypes
        L.ersd_verify_tokens.argtypes = L.ersd_verify.argtypes
        L.ersd_verify_tree.argtypes = [vp, vp, i, C.POINTER(C.c_int32), vp, i, i, i, f, vp, vp,
                                       C.POINTER(ErsdOpts), vp]
        L.ersd_gsd_verify.argtypes = [vp, vp, vp, i, vp, i, i, i, f, vp, vp, C.POINTER(ErsdOpts), vp]
        L.ersd_gsd_verify_tree.argtypes = [vp, vp, vp, i, C.POINTER(C.c_int32), vp, i, i, i, f, vp, vp,
                                           C.POINTER(ErsdOpts), vp]
        L.ersd_tree_depth.argtypes = [C.POINTER(C.c_int32), i]
        L.ersd_optimal_tree.argtypes = [C.POINTER(C.c_double), i, i, C.POINTER(C.c_int32), C.POINTER(C.c_double)]
        L.ersd_optimal_tree.restype = i
        L.ersd_acceptance_profile.argtypes = [C.POINTER(C.c_int32), C.POINTER(C.c_int32), i, i, i,
                                              C.POINTER(C.c_double), C.POINTER(C.c_int64)]
        L.ersd_acceptance_profile.restype = i
        L.ersd_row_keys.argtypes = [vp, i, i, f, C.c_uint64, C.c_uint32, C.c_uint32, i, vp, vp]
        L.ersd_workspace_bytes.argtypes = [i, i]
        L.ersd_workspace_bytes.restype = C.c_size_t
        L.ersd_workspace_init.argtypes = [vp, C.c_size_t, vp]
        L.ersd_status_string.argtypes = [i]
        L.ersd_status_string.restype = C.c_char_p
        L.ersd_last_launch.restype = C.c_char_p
        for name in ("ersd_race_sample", "ersd_verify", "ersd_verify_tokens", "ersd_verify_noalloc", "ersd_verify_tree", "ersd_tree_depth",
                     "ersd_gsd_verify", "ersd_gsd_verify_tree",
                     "ersd_row_keys", "ersd_workspace_init", "ersd_last_cuda_error", "ersd_version"):
            getattr(L, name).restype = i
        _lib = L
    return _lib


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return ERSD_F32
    if t.dtype == torch.bfloat16:
        return ERSD_BF16
    raise TypeError("logits must be float32 or bfloat16, got %s" % t.dtype)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _check(status: int, where: str):
    if status != ERSD_OK:
        raise ErsdError(status, where)


def _dev(t: torch.Tensor, dtype, name: str):
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor" % name)
    if dtype is not None and t.dtype != dtype:
        raise TypeError("%s must be %s" % (name, dtype))
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    return t


def _sizes(logits: torch.Tensor, V: Optional[int]):
    """(B, rows, V) of a logits tensor [B, rows, ld]; V defaults to ld (rows without padding)."""
    B, rows, ld = logits.shape
    if V is None:
        return B, rows, ld
    if not 1 <= int(V) <= ld:
        raise ValueError("V must be between 1 and the row length of the tensor")
    return B, rows, int(V)


def make_opts(*, top_c: int = 0, split_v: int = 0, block_threads: int = 0, ld_target: int = 0, ld_draft: int = 0,
              temps: Optional[torch.Tensor] = None, temp_strides: Sequence[int] = (0, 0),
              seq_ids: Optional[torch.Tensor] = None, pos_offsets: Optional[torch.Tensor] = None,
              out_draft_tok=None, out_draft_key=None, out_target_tok=None, out_target_key=None,
              out_path=None, out_key=None, workspace: Optional[torch.Tensor] = None,
              kernel_path: int = 0, near_tie_count: Optional[torch.Tensor] = None) -> ErsdOpts:
    o = ErsdOpts()
    o.struct_size = C.sizeof(ErsdOpts)
    o.top_c, o.split_v, o.block_threads = top_c, split_v, block_threads
    o.kernel_path = kernel_path
    o.ld_target, o.ld_draft = ld_target, ld_draft
    if temps is not None:
        _dev(temps, torch.float32, "temps")
        o.temps = temps.data_ptr()
        o.temp_stride_b, o.temp_stride_r = int(temp_strides[0]), int(temp_strides[1])
    if seq_ids is not None:
        o.seq_ids = _dev(seq_ids, torch.int32, "seq_ids").data_ptr()
    if pos_offsets is not None:
        o.pos_offsets = _dev(pos_offsets, torch.int32, "pos_offsets").data_ptr()
    for name, t, dt in (("out_draft_tok", out_draft_tok, torch.int32),
                        ("out_draft_key", out_draft_key, torch.float32),
                        ("out_target_tok", out_target_tok, torch.int32),
                        ("out_target_key", out_target_key, torch.float32),
                        ("out_path", out_path, torch.int32), ("out_key", out_key, torch.float32)):
        if t is not None:
            setattr(o, name, _dev(t, dt, name).data_ptr())
    if workspace is not None:
        o.workspace = workspace.data_ptr()
        o.workspace_bytes = workspace.numel() * workspace.element_size()
    if near_tie_count is not None:  # int32 tensor of one element that the call adds to
        o.near_tie_count = _dev(near_tie_count, torch.int32, "near_tie_count").data_ptr()
    return o


def ersd_last_launch() -> str:
    """Which kernel the last call of this thread launched, and in what shape."""
    return lib().ersd_last_launch().decode()


def ersd_version() -> int:
    return int(lib().ersd_version())


def ersd_workspace_bytes(B: int, rows_per_seq: int) -> int:
    return int(lib().ersd_workspace_bytes(B, rows_per_seq))


def ersd_workspace_init(workspace: torch.Tensor, stream=None) -> None:
    _check(lib().ersd_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(),
                                     _stream(stream)), "ersd_workspace_init")


def ersd_tree_depth(parent: Sequence[int]) -> int:
    arr = (C.c_int32 * len(parent))(*[int(p) for p in parent])
    return int(lib().ersd_tree_depth(arr, len(parent) - 1))


def ersd_optimal_tree(accept: Sequence[float], k: int):
    """(parent array [k + 1], expected number of accepted tokens) of the best k-token draft tree for
    per-rank acceptance probabilities `accept` (host function, Algorithm 3)."""
    a = (C.c_double * len(accept))(*[float(x) for x in accept])
    parent = (C.c_int32 * (k + 1))()
    expected = C.c_double(0.0)
    _check(lib().ersd_optimal_tree(a, len(accept), int(k), parent, C.byref(expected)), "ersd_optimal_tree")
    return list(parent), float(expected.value)


def ersd_acceptance_profile(paths, parent: Sequence[int], max_children: int):
    """(accept [max_children], trials [max_children]) from the accepted paths ([B, D+1] node ids,
    -1 padded: opts.out_path of a tree verification, any device) over the draft tree `parent`:
    the empirical per-rank acceptance probabilities that ersd_optimal_tree takes (host function)."""
    pt = torch.as_tensor(paths).detach().to("cpu", torch.int32).contiguous()
    B = int(pt.shape[0])
    par = (C.c_int32 * len(parent))(*[int(x) for x in parent])
    acc = (C.c_double * max_children)()
    tri = (C.c_int64 * max_children)()
    _check(lib().ersd_acceptance_profile(C.cast(pt.data_ptr(), C.POINTER(C.c_int32)), par, B, len(parent) - 1,
                                         int(max_children), acc, tri), "ersd_acceptance_profile")
    return list(acc), list(tri)


def ersd_race_sample(logits: torch.Tensor, seeds: torch.Tensor, T: float, out_tok: torch.Tensor,
                     opts: Optional[ErsdOpts] = None, stream=None, V: Optional[int] = None) -> None:
    """logits [B, R, V] (f32/bf16), seeds int64 [B] (the uint64 bit patterns), out_tok int32 [B, R, c].
    Padded rows: pass the tensor [B, R, ld], the vocabulary size as ``V`` and opts.ld_target = ld."""
    _dev(logits, None, "logits")
    _dev(seeds, torch.int64, "seeds")
    _dev(out_tok, torch.int32, "out_tok")
    B, R, V = _sizes(logits, V)
    _check(lib().ersd_race_sample(_ptr(logits), _dtype_code(logits), _ptr(seeds), B, R, V, float(T),
                                  _ptr(out_tok), C.byref(opts) if opts is not None else None,
                                  _stream(stream)), "ersd_race_sample")


def ersd_verify(target_logits: torch.Tensor, draft_logits: Optional[torch.Tensor], seeds: torch.Tensor,
                T: float, out_tokens: torch.Tensor, out_accept_len: torch.Tensor,
                opts: Optional[ErsdOpts] = None, stream=None, V: Optional[int] = None) -> None:
    """target [B, k+1, V], draft [B, k, V], out_tokens int32 [B, k+1], out_accept_len int32 [B].
    Padded rows: tensors [B, rows, ld], the vocabulary size as ``V``, opts.ld_target / ld_draft = ld."""
    _dev(target_logits, None, "target_logits")
    B, rows, V = _sizes(target_logits, V)
    if draft_logits is not None:
        _dev(draft_logits, target_logits.dtype, "draft_logits")
    _dev(seeds, torch.int64, "seeds")
    _dev(out_tokens, torch.int32, "out_tokens")
    _dev(out_accept_len, torch.int32, "out_accept_len")
    _check(lib().ersd_verify(_ptr(target_logits), _ptr(draft_logits), _dtype_code(target_logits),
                             _ptr(seeds), B, rows - 1, V, float(T), _ptr(out_tokens),
                             _ptr(out_accept_len), C.byref(opts) if opts is not None else None,
                             _stream(stream)), "ersd_verify")


def ersd_verify_tokens(target_logits: torch.Tensor, draft_tokens: Optional[torch.Tensor], seeds: torch.Tensor,
                       T: float, out_tokens: torch.Tensor, out_accept_len: torch.Tensor,
                       opts: Optional[ErsdOpts] = None, stream=None, V: Optional[int] = None) -> None:
    """target [B, k+1, V], draft_tokens int32 [B, k] (drafted earlier with the same races),
    out_tokens int32 [B, k+1], out_accept_len int32 [B]."""
    _dev(target_logits, None, "target_logits")
    B, rows, V = _sizes(target_logits, V)
    if draft_tokens is not None:
        _dev(draft_tokens, torch.int32, "draft_tokens")
    _dev(seeds, torch.int64, "seeds")
    _dev(out_tokens, torch.int32, "out_tokens")
    _dev(out_accept_len, torch.int32, "out_accept_len")
    _check(lib().ersd_verify_tokens(_ptr(target_logits), _ptr(draft_tokens), _dtype_code(target_logits),
                                    _ptr(seeds), B, rows - 1, V, float(T), _ptr(out_tokens),
                                    _ptr(out_accept_len), C.byref(opts) if opts is not None else None,
                                    _stream(stream)), "ersd_verify_tokens")


def ersd_gsd_verify(target_logits: torch.Tensor, draft_logits: Optional[torch.Tensor],
                    draft_tokens: Optional[torch.Tensor], seeds: torch.Tensor, T: float, out_tokens: torch.Tensor,
                    out_accept_len: torch.Tensor, opts: Optional[ErsdOpts] = None, stream=None,
                    V: Optional[int] = None) -> None:
    """Greedy speculative decoding (Algorithm 1 position by position) on the same logits.
    target [B, k+1, V], draft [B, k, V], draft_tokens int32 [B, k]; out_tokens int32 [B, k+1]."""
    _dev(target_logits, None, "target_logits")
    B, rows, V = _sizes(target_logits, V)
    if draft_logits is not None:
        _dev(draft_logits, target_logits.dtype, "draft_logits")
    if draft_tokens is not None:
        _dev(draft_tokens, torch.int32, "draft_tokens")
    _dev(seeds, torch.int64, "seeds")
    _dev(out_tokens, torch.int32, "out_tokens")
    _dev(out_accept_len, torch.int32, "out_accept_len")
    _check(lib().ersd_gsd_verify(_ptr(target_logits), _ptr(draft_logits), _ptr(draft_tokens),
                                 _dtype_code(target_logits), _ptr(seeds), B, rows - 1, V, float(T),
                                 _ptr(out_tokens), _ptr(out_accept_len),
                                 C.byref(opts) if opts is not None else None, _stream(stream)), "ersd_gsd_verify")


def ersd_gsd_verify_tree(target_logits: torch.Tensor, draft_logits: Optional[torch.Tensor],
                         draft_tokens: Optional[torch.Tensor], parent: Sequence[int], seeds: torch.Tensor,
                         T: float, out_tokens: torch.Tensor, out_accept_len: torch.Tensor,
                         opts: Optional[ErsdOpts] = None, stream=None, V: Optional[int] = None) -> None:
    """Tree GSD (Algorithm 4).  target, draft [B, N+1, V]; draft_tokens int32 [B, N+1] (entry 0
    unused); parent: host list [N+1]; out_tokens int32 [B, D+1]."""
    _dev(target_logits, None, "target_logits")
    B, rows, V = _sizes(target_logits, V)
    if draft_logits is not None:
        _dev(draft_logits, target_logits.dtype, "draft_logits")
    if draft_tokens is not None:
        _dev(draft_tokens, torch.int32, "draft_tokens")
    _dev(seeds, torch.int64, "seeds")
    _dev(out_tokens, torch.int32, "out_tokens")
    _dev(out_accept_len, torch.int32, "out_accept_len")
    arr = (C.c_int32 * len(parent))(*[int(x) for x in parent])
    _check(lib().ersd_gsd_verify_tree(_ptr(target_logits), _ptr(draft_logits), _ptr(draft_tokens),
                                      _dtype_code(target_logits), arr, _ptr(seeds), B, rows - 1, V, float(T),
                                      _ptr(out_tokens), _ptr(out_accept_len),
                                      C.byref(opts) if opts is not None else None, _stream(stream)),
           "ersd_gsd_verify_tree")


def ersd_verify_noalloc(target_logits: torch.Tensor, draft_logits: Optional[torch.Tensor],
                        seeds: torch.Tensor, T: float, out_tokens: torch.Tensor,
                        out_accept_len: torch.Tensor, opts: Optional[ErsdOpts] = None, stream=None,
                        V: Optional[int] = None) -> None:
    """ersd_verify for callers that cannot allocate device memory: same arguments and results,
    scratch built into the library, B * (k + 1) <= ERSD_NOALLOC_MAX_ROWS.  Calls on one device
    share that scratch, so they must not overlap on the GPU."""
    _dev(target_logits, None, "target_logits")
    B, rows, V = _sizes(target_logits, V)
    if draft_logits is not None:
        _dev(draft_logits, target_logits.dtype, "draft_logits")
    _dev(seeds, torch.int64, "seeds")
    _dev(out_tokens, torch.int32, "out_tokens")
    _dev(out_accept_len, torch.int32, "out_accept_len")
    _check(lib().ersd_verify_noalloc(_ptr(target_logits), _ptr(draft_logits), _dtype_code(target_logits),
                                     _ptr(seeds), B, rows - 1, V, float(T), _ptr(out_tokens),
                                     _ptr(out_accept_len), C.byref(opts) if opts is not None else None,
                                     _stream(stream)), "ersd_verify_noalloc")


def ersd_verify_tree(target_logits: torch.Tensor, draft_logits: Optional[torch.Tensor],
                     parent: Sequence[int], seeds: torch.Tensor, T: float, out_tokens: torch.Tensor,
                     out_accept_len: torch.Tensor, opts: Optional[ErsdOpts] = None, stream=None,
                     V: Optional[int] = None) -> None:
    """target, draft [B, N+1, V]; parent: host list [N+1]; out_tokens int32 [B, D+1]."""
    _dev(target_logits, None, "target_logits")
    B, nodes, V = _sizes(target_logits, V)
    if draft_logits is not None:
        _dev(draft_logits, target_logits.dtype, "draft_logits")
    _dev(seeds, torch.int64, "seeds")
    _dev(out_tokens, torch.int32, "out_tokens")
    _dev(out_accept_len, torch.int32, "out_accept_len")
    arr = (C.c_int32 * len(parent))(*[int(p) for p in parent])
    _check(lib().ersd_verify_tree(_ptr(target_logits), _ptr(draft_logits), _dtype_code(target_logits),
                                  arr, _ptr(seeds), B, nodes - 1, V, float(T), _ptr(out_tokens),
                                  _ptr(out_accept_len), C.byref(opts) if opts is not None else None,
                                  _stream(stream)), "ersd_verify_tree")


def ersd_row_keys(row: torch.Tensor, T: float, seed: int, seq_id: int, position: int, mode: int,
                  out_keys: torch.Tensor, stream=None) -> None:
    _dev(row, None, "row")
    _dev(out_keys, torch.float32, "out_keys")
    _check(lib().ersd_row_keys(_ptr(row), _dtype_code(row), row.shape[0], float(T),
                               C.c_uint64(seed & (2**64 - 1)), seq_id, position, mode, _ptr(out_keys),
                               _stream(stream)), "ersd_row_keys")


# --------------------------------------------------------------------------- conveniences
def verify(target_logits, draft_logits, seeds, T=1.0, temps=None, parent=None, split_v=0,
           want_rows=False, seq_ids=None, pos_offsets=None, block_threads=0, kernel_path=0):
    """Allocate outputs, call ersd_verify / ersd_verify_tree, return a dict of device tensors."""
    B, rows, V = target_logits.shape
    dev = target_logits.device
    D = rows - 1 if parent is None else ersd_tree_depth(parent)
    out = dict(tokens=torch.empty(B, D + 1, dtype=torch.int32, device=dev),
               accept_len=torch.empty(B, dtype=torch.int32, device=dev))
    kw = dict(split_v=split_v, block_threads=block_threads, seq_ids=seq_ids, pos_offsets=pos_offsets,
              kernel_path=kernel_path)
    if temps is not None:
        kw.update(temps=temps, temp_strides=(temps.stride(0), temps.stride(1)))
    if want_rows:
        n_d = rows - 1 if parent is None else rows
        out["draft_tok"] = torch.empty(B, n_d, dtype=torch.int32, device=dev)
        out["draft_key"] = torch.empty(B, n_d, dtype=torch.float32, device=dev)
        out["target_tok"] = torch.empty(B, rows, dtype=torch.int32, device=dev)
        out["target_key"] = torch.empty(B, rows, dtype=torch.float32, device=dev)
        kw.update(out_draft_tok=out["draft_tok"], out_draft_key=out["draft_key"],
                  out_target_tok=out["target_tok"], out_target_key=out["target_key"])
        if parent is not None:
            out["path"] = torch.empty(B, D + 1, dtype=torch.int32, device=dev)
            kw.update(out_path=out["path"])
    opts = make_opts(**kw)
    if parent is None:
        ersd_verify(target_logits, draft_logits, seeds, T, out["tokens"], out["accept_len"], opts)
    else:
        ersd_verify_tree(target_logits, draft_logits, parent, seeds, T, out["tokens"],
                         out["accept_len"], opts)
    return out


def verify_host(target_logits, draft_logits, seeds, T=1.0, temps=None, parent=None, device="cuda"):
    """End-to-end call on HOST tensors: copy in, verify on the GPU, copy the result back."""
    tgt = target_logits.to(device, non_blocking=True)
    drf = draft_logits.to(device, non_blocking=True) if draft_logits is not None else None
    sd = seeds.to(device, non_blocking=True)
    tp = temps.to(device, non_blocking=True) if temps is not None else None
    out = verify(tgt, drf, sd, T, temps=tp, parent=parent)
    return out["tokens"].cpu(), out["accept_len"].cpu()
