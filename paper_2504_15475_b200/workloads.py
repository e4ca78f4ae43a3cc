"""Seeded synthetic inputs: Zipf-shaped logit rows, seeds and tree shapes.

This module only makes inputs.  It holds none of the method's arithmetic (no
race, no Philox stream of the method, no verification) and is the one module
that both the CPU oracle's tests and the CUDA path's tests feed from, so that
both sides see the same bits.

The rows stand in for next-token distributions of a large target model and a
small draft model over Llama-/Qwen-sized vocabularies (the paper's experiments
use Llama-3.1-70B-Instruct and Llama-3.2-1B, whose weights are not available
here):

    target[b, r, pi(rho)] = -s * ln(rho) + N(0, 1),  rho = 1..V,
    draft[b, j, :]        = target_fp32[b, j, :] + sigma * N(0, 1),

with pi a fresh random permutation per row, s the Zipf exponent, everything
generated in fp32 and cast once (round to nearest even) to the storage type.
"""
from __future__ import annotations

import dataclasses
from typing import Optional, Sequence

import torch

_MASK64 = (1 << 64) - 1


def splitmix64(x: int) -> int:
    """One output of the SplitMix64 mixer (Steele, Lea, Flood 2014) for state x."""
    x = (x + 0x9E3779B97F4A7C15) & _MASK64
    z = x
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def make_seeds(global_seed: int, call: int, B: int) -> torch.Tensor:
    """Per-sequence 64-bit race seeds, returned as int64 bit patterns [B]."""
    out = []
    for b in range(B):
        s = splitmix64(splitmix64(splitmix64(global_seed) ^ call) ^ b)
        out.append(s - (1 << 64) if s >= (1 << 63) else s)
    return torch.tensor(out, dtype=torch.int64)


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    B: int
    k: int                      # drafted tokens per sequence (tree: N = number of draft nodes)
    V: int
    dtype: str                  # "f32" | "bf16"
    sigma: float = 1.0          # std of the draft perturbation
    T: float = 1.0
    zipf: float = 1.1           # exponent s; zipf_range overrides it per row
    zipf_range: Optional[tuple] = None
    temps_choices: Optional[tuple] = None   # one temperature per sequence, drawn from these
    parent: Optional[tuple] = None          # tree variant: parent[n] for n = 0..N
    config_id: int = 0
    zero_seed: bool = False     # config 1 fixes the race seed to 0

    @property
    def rows_target(self) -> int:
        return self.k + 1

    @property
    def is_tree(self) -> bool:
        return self.parent is not None


TREE_4x4 = (-1, 0, 0, 0, 0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12)
# "3 sequences with the first two drafted tokens in common" (the SpecInfer shape of Section 5)
TREE_SPECINFER = (-1, 0, 1, 2, 2, 2, 3, 4, 5)

CONFIGS = {
    "c1": Workload("c1", B=1, k=4, V=1024, dtype="f32", sigma=0.5, T=1.0, config_id=1,
                   zero_seed=True),
    "c2": Workload("c2", B=8, k=4, V=32000, dtype="bf16", sigma=0.5, T=1.0, config_id=2),
    "c3": Workload("c3", B=64, k=8, V=128256, dtype="bf16", sigma=1.0, T=1.0, config_id=3),
    "c4": Workload("c4", B=32, k=16, V=151936, dtype="bf16", sigma=1.0, T=1.0, config_id=4,
                   parent=TREE_4x4),
    "c5": Workload("c5", B=256, k=5, V=128256, dtype="bf16", sigma=1.0, T=1.0, config_id=5,
                   zipf_range=(0.9, 1.3), temps_choices=(0.6, 0.8, 1.0)),
}
C3_SWEEP = [(sigma, T) for sigma in (0.25, 1.0, 2.0) for T in (0.7, 1.0)]


def _storage(x: torch.Tensor, dtype: str) -> torch.Tensor:
    if dtype == "bf16":
        return x.to(torch.bfloat16)
    if dtype == "f32":
        return x
    raise ValueError(dtype)


def zipf_rows(rows: int, V: int, gen: torch.Generator, device, zipf: float = 1.1,
              zipf_range: Optional[tuple] = None) -> torch.Tensor:
    """fp32 [rows, V]: -s ln(rank) + N(0,1) scattered by a random permutation per row."""
    out = torch.empty(rows, V, dtype=torch.float32, device=device)
    log_rank = torch.log(torch.arange(1, V + 1, dtype=torch.float32, device=device))
    chunk = max(1, min(rows, (1 << 25) // max(V, 1)))
    for r0 in range(0, rows, chunk):
        r1 = min(rows, r0 + chunk)
        n = r1 - r0
        if zipf_range is not None:
            s = torch.empty(n, 1, device=device).uniform_(zipf_range[0], zipf_range[1],
                                                          generator=gen)
        else:
            s = torch.full((n, 1), float(zipf), device=device)
        perm = torch.rand(n, V, generator=gen, device=device).argsort(dim=1)
        base = -s * log_rank.unsqueeze(0)
        noise = torch.randn(n, V, generator=gen, device=device)
        out[r0:r1] = torch.gather(base, 1, perm) + noise
    return out


def make_inputs(w: Workload, call: int = 0, device="cpu", sigma: Optional[float] = None,
                T: Optional[float] = None, global_seed: int = 2504_15475):
    """Inputs of one verify call for workload w.

    Returns a dict: target [B, rows, V], draft [B, k or N+1, V] (storage dtype),
    seeds int64 [B], T (float), temps (float32 [B, rows] or None), parent (list or None).
    """
    sigma = w.sigma if sigma is None else sigma
    T = w.T if T is None else T
    gen = torch.Generator(device=device)
    gen.manual_seed(1000 * w.config_id + call)
    rows = w.rows_target
    tgt32 = zipf_rows(w.B * rows, w.V, gen, device, w.zipf, w.zipf_range).view(w.B, rows, w.V)
    n_draft = rows if w.is_tree else w.k
    draft32 = tgt32[:, :n_draft, :] + sigma * torch.randn(w.B, n_draft, w.V, generator=gen,
                                                           device=device)
    temps = None
    if w.temps_choices is not None:
        pick = torch.randint(0, len(w.temps_choices), (w.B,), generator=gen, device=device)
        per_seq = torch.tensor(w.temps_choices, dtype=torch.float32, device=device)[pick]
        temps = per_seq.unsqueeze(1).expand(w.B, rows).contiguous()
    if w.zero_seed:
        seeds = torch.zeros(w.B, dtype=torch.int64)
    else:
        seeds = make_seeds(global_seed + w.config_id, call, w.B)
    return dict(target=_storage(tgt32, w.dtype).contiguous(),
                draft=_storage(draft32, w.dtype).contiguous(), seeds=seeds.to(device), T=float(T),
                temps=temps, parent=list(w.parent) if w.is_tree else None)


def scaled(w: Workload, B: Optional[int] = None, V: Optional[int] = None,
           k: Optional[int] = None) -> Workload:
    """A smaller (or larger) copy of a workload with the same recipe."""
    return dataclasses.replace(w, B=w.B if B is None else B, V=w.V if V is None else V,
                               k=w.k if k is None else k)


def as_numpy_logits(t: torch.Tensor):
    """Host numpy view of a logit tensor: float32 as is, bf16 as its uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view("uint16")
    return t.numpy()


def seeds_as_u64(seeds: torch.Tensor):
    return seeds.detach().cpu().contiguous().numpy().view("uint64")


def chain_parent(k: int) -> Sequence[int]:
    return [-1] + list(range(k))


def star_parent(k: int) -> Sequence[int]:
    return [-1] + [0] * k
