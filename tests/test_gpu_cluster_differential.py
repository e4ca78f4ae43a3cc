"""Differential test of the two kernels: seeded random shapes, temperatures and masks; the cluster
kernel and the streaming kernel must agree bit for bit (tokens, accept lengths, per-row winners
and keys), and a sample of the cases is also checked against the CPU oracle."""
import os

import numpy as np
import pytest
import torch

from paper_2504_15475_b200 import workloads as wl

from parity_util import check_verify

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ersd():
    from paper_2504_15475_b200 import binding
    binding.lib()
    assert torch.cuda.is_available()
    return binding


def random_case(rng: np.random.Generator, g: torch.Generator):
    B = int(rng.integers(1, 6))
    k = int(rng.integers(0, 9))
    V = int(rng.choice([int(rng.integers(1, 64)), int(rng.integers(64, 5000)), int(rng.integers(5000, 70000)),
                        int(rng.integers(70000, 160000))]))
    V8 = (V + 7) // 8 * 8                       # rows padded to 16-byte boundaries
    dtype = "bf16" if rng.random() < 0.7 else "f32"
    T = float(rng.choice([0.0, 0.3, 0.7, 1.0, 1.0, 1.7]))
    style = rng.integers(0, 4)
    if style == 0:
        t = wl.zipf_rows(B * (k + 1), V, g, "cpu").view(B, k + 1, V)
    elif style == 1:
        t = torch.randn(B, k + 1, V, generator=g) * float(rng.uniform(0.1, 4.0))
    elif style == 2:                            # few distinct values: many ties in bf16
        t = torch.randint(-3, 4, (B, k + 1, V), generator=g).float() * 0.5
    else:                                       # peaked
        t = torch.full((B, k + 1, V), -20.0) + torch.randn(B, k + 1, V, generator=g)
        t[..., int(rng.integers(0, V))] = 3.0
    d = t[:, :k] + float(rng.uniform(0.0, 1.5)) * torch.randn(B, k, V, generator=g)
    if rng.random() < 0.4:                      # masked ranges, infinities, NaNs
        lo = int(rng.integers(0, V))
        t[:, :, lo:lo + int(rng.integers(1, V + 1))] = float("-inf")
        if k > 0 and rng.random() < 0.5:
            d[:, 0, int(rng.integers(0, V))] = float("inf")
        if rng.random() < 0.3:
            t[0, 0, int(rng.integers(0, V))] = float("nan")
    big_t = torch.full((B, k + 1, V8), 70.0)
    big_d = torch.full((B, max(k, 1), V8), 70.0)
    big_t[:, :, :V] = t
    if k > 0:
        big_d[:, :k, :V] = d
    temps = None
    if rng.random() < 0.3:
        temps = torch.tensor(rng.choice([0.0, 0.5, 1.0, 2.0], size=(B, k + 1)), dtype=torch.float32)
    return dict(B=B, k=k, V=V, ld=V8, dtype=dtype, T=T, temps=temps,
                target=wl._storage(big_t, dtype), draft=wl._storage(big_d[:, :k].contiguous(), dtype) if k > 0 else None,
                seeds=wl.make_seeds(int(rng.integers(0, 1 << 30)), 0, B))


def run(ersd, case, path):
    B, k, V, ld = case["B"], case["k"], case["V"], case["ld"]
    out = dict(tokens=torch.full((B, k + 1), -7, dtype=torch.int32, device="cuda"),
               accept_len=torch.full((B,), -7, dtype=torch.int32, device="cuda"),
               target_tok=torch.full((B, k + 1), -7, dtype=torch.int32, device="cuda"),
               target_key=torch.full((B, k + 1), -7.0, dtype=torch.float32, device="cuda"),
               draft_tok=torch.full((B, k), -7, dtype=torch.int32, device="cuda"),
               draft_key=torch.full((B, k), -7.0, dtype=torch.float32, device="cuda"))
    kw = dict(ld_target=ld, ld_draft=ld, kernel_path=path, out_target_tok=out["target_tok"],
              out_target_key=out["target_key"])
    if k > 0:
        kw.update(out_draft_tok=out["draft_tok"], out_draft_key=out["draft_key"])
    if case["temps"] is not None:
        tp = case["temps"].cuda()
        kw.update(temps=tp, temp_strides=(tp.stride(0), tp.stride(1)))
    ersd.ersd_verify(case["target"].cuda(), case["draft"].cuda() if k > 0 else None, case["seeds"].cuda(), case["T"],
                     out["tokens"], out["accept_len"], ersd.make_opts(**kw), V=V)
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("chunk", range(int(os.environ.get("ERSD_DIFFERENTIAL_CHUNKS", "6"))))  # 25 cases each
def test_random_cases_agree_between_the_kernels(ersd, chunk):
    rng = np.random.default_rng(1234 + chunk)
    g = torch.Generator().manual_seed(99 + chunk)
    for n in range(25):
        case = random_case(rng, g)
        a = run(ersd, case, 2)
        b = run(ersd, case, 1)
        for name in a:
            same = (a[name] == b[name]) | (torch.isnan(a[name].float()) & torch.isnan(b[name].float()))
            assert same.all(), (chunk, n, name, {q: case[q] for q in ("B", "k", "V", "dtype", "T")}, a[name], b[name])
        if n % 5 == 0 and case["temps"] is None:       # and the oracle agrees with both
            V = case["V"]
            inp = dict(target=case["target"][:, :, :V].contiguous(),
                       draft=case["draft"][:, :, :V].contiguous() if case["k"] > 0 else
                       torch.empty(case["B"], 0, V, dtype=case["target"].dtype),
                       seeds=case["seeds"], T=case["T"], temps=None, parent=None)
            check_verify(inp, a)


# ------------------------------------------------------------------ races of several arrivals
def random_parent(rng: np.random.Generator, n_nodes: int, max_children: int):
    """A random draft tree: node n hangs under an earlier node that still has room for a child."""
    parent, nchild = [-1], [0]
    for n in range(1, n_nodes):
        room = [m for m in range(n) if nchild[m] < max_children]
        m = int(rng.choice(room))
        parent.append(m)
        nchild[m] += 1
        nchild.append(0)
    return parent


def random_rows(rng, g, B, rows, V):
    style = rng.integers(0, 4)
    if style == 0:
        t = wl.zipf_rows(B * rows, V, g, "cpu").view(B, rows, V)
    elif style == 1:
        t = torch.randn(B, rows, V, generator=g) * float(rng.uniform(0.1, 4.0))
    elif style == 2:                            # few distinct values: many ties in bf16
        t = torch.randint(-3, 4, (B, rows, V), generator=g).float() * 0.5
    else:                                       # peaked
        t = torch.full((B, rows, V), -20.0) + torch.randn(B, rows, V, generator=g)
        t[..., int(rng.integers(0, V))] = 3.0
    if rng.random() < 0.3:                      # a masked range
        lo = int(rng.integers(0, V))
        t[:, :, lo:lo + int(rng.integers(1, V + 1))] = float("-inf")
    return t


@pytest.mark.parametrize("chunk", range(4))  # 15 trees and 15 sampling calls each
def test_random_trees_and_first_arrivals_agree_between_the_kernels(ersd, chunk):
    rng = np.random.default_rng(4321 + chunk)
    g = torch.Generator().manual_seed(77 + chunk)
    for n in range(15):
        # tree verification
        B = int(rng.integers(1, 4))
        nodes = int(rng.integers(2, 20))
        parent = random_parent(rng, nodes, int(rng.integers(2, 9)))
        V = int(rng.choice([int(rng.integers(8, 3000)), int(rng.integers(3000, 60000)), int(rng.integers(60000, 160000))]))
        V = (V + 7) // 8 * 8
        dtype = "bf16" if rng.random() < 0.7 else "f32"
        T = float(rng.choice([0.0, 0.4, 1.0, 1.0, 1.6]))
        t = random_rows(rng, g, B, nodes, V)
        d = t + float(rng.uniform(0.0, 1.5)) * torch.randn(B, nodes, V, generator=g)
        inp = dict(target=wl._storage(t, dtype), draft=wl._storage(d, dtype),
                   seeds=wl.make_seeds(int(rng.integers(0, 1 << 30)), 0, B), T=T, temps=None, parent=parent)
        outs = []
        for path in (2, 1):
            out = ersd.verify(inp["target"].cuda(), inp["draft"].cuda(), inp["seeds"].cuda(), T, parent=parent,
                              want_rows=True, kernel_path=path)
            torch.cuda.synchronize()
            outs.append(out)
        for name in outs[0]:
            a, b = outs[0][name], outs[1][name]
            assert ((a == b) | (torch.isnan(a.float()) & torch.isnan(b.float()))).all(), (chunk, n, name, parent, V, dtype, T)
        if n % 3 == 0:
            check_verify(inp, outs[0])
        # the first c arrivals of single races
        R, c = int(rng.integers(1, 4)), int(rng.integers(2, 33))
        rows = wl._storage(random_rows(rng, g, B, R, V), dtype)
        got = []
        for path in (2, 1):
            tok = torch.full((B, R, c), -7, dtype=torch.int32, device="cuda")
            key = torch.full((B, R, c), -7.0, dtype=torch.float32, device="cuda")
            ersd.ersd_race_sample(rows.cuda(), inp["seeds"].cuda(), T, tok,
                                  ersd.make_opts(kernel_path=path, top_c=c, out_key=key))
            torch.cuda.synchronize()
            got.append((tok, key))
        assert (got[0][0] == got[1][0]).all() and (got[0][1] == got[1][1]).all(), (chunk, n, "sample", V, dtype, T, c)
