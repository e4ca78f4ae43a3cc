"""Greedy speculative decoding on the GPU (ersd_gsd_verify, ersd_gsd_verify_tree) against the CPU
oracle's Algorithms 1 and 4, through the C boundary, on the same seeded inputs.

Bar: emitted tokens and accept lengths equal the oracle's.  Both sides decide in double precision,
so the allowed exceptions are decisions within rounding of each other, which the oracle's outputs
expose: a ratio test with |ratio - u| < 1e-9 * ratio, or a final race whose two best arrival times
are closer than 1e-5 relative (the near-tie window); such sequences are counted."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_15475_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ersd():
    from paper_2504_15475_b200 import binding
    binding.lib()
    assert torch.cuda.is_available()
    return binding


def draft_tokens(ersd, draft, seeds, T, c=1, temps=None):
    """Tokens drafted on the GPU: the first c arrivals of every draft row's race (a sample without
    replacement of that row's law)."""
    B, R, V = draft.shape
    tok = torch.empty(B, R, c, dtype=torch.int32, device="cuda")
    kw = {}
    if temps is not None:
        kw = dict(temps=temps, temp_strides=(temps.stride(0), temps.stride(1)))
    ersd.ersd_race_sample(draft, seeds, T, tok, ersd.make_opts(top_c=c, **kw))
    return tok


def ambiguous(ref):
    """Sequences whose outcome hangs on a decision within rounding (see the module docstring)."""
    amb = np.zeros(ref["accept_len"].shape[0], bool)
    if "ratio" in ref:
        r, u = ref["ratio"], ref["unif"]
        with np.errstate(invalid="ignore"):
            amb |= (np.abs(r - u) < 1e-9 * np.maximum(r, 1e-300)).any(axis=1)
    t = ref["last_times"]
    with np.errstate(invalid="ignore"):
        amb |= (t[:, 1] - t[:, 0]) < 1e-5 * t[:, 0]
    return amb


@pytest.mark.parametrize("name,scale", [("c1", {}), ("c2", {}), ("c5", dict(B=12)), ("c3", dict(B=4)),
                                        ("c2", dict(B=300, V=3000))])
def test_sequence_gsd_against_the_oracle(ersd, name, scale):
    w = wl.scaled(wl.CONFIGS[name], **scale)
    inp = wl.make_inputs(w, call=5)
    tgt, drf, seeds = inp["target"].cuda(), inp["draft"].cuda(), inp["seeds"].cuda()
    temps = None if inp.get("temps") is None else inp["temps"].cuda()
    kw = {} if temps is None else dict(temps=temps, temp_strides=(temps.stride(0), temps.stride(1)))
    t_d = None if temps is None else temps[:, :w.k].contiguous()
    tok = draft_tokens(ersd, drf, seeds, inp["T"], temps=t_d)[..., 0].contiguous()
    out = torch.full((w.B, w.k + 1), -9, dtype=torch.int32, device="cuda")
    acc = torch.full((w.B,), -9, dtype=torch.int32, device="cuda")
    for rep in range(2):                        # twice: the call leaves the workspace as it found it
        ersd.ersd_gsd_verify(tgt, drf, tok, seeds, inp["T"], out, acc, ersd.make_opts(**kw))
    torch.cuda.synchronize()
    ref = oracle.gsd_verify(wl.as_numpy_logits(inp["target"]), wl.as_numpy_logits(inp["draft"]),
                            tok.cpu().numpy(), wl.seeds_as_u64(inp["seeds"]), T=inp["T"],
                            temps=None if temps is None else inp["temps"].numpy())
    amb = ambiguous(ref)
    assert amb.sum() <= 1
    ok = ~amb
    assert (acc.cpu().numpy()[ok] == ref["accept_len"][ok]).all()
    assert (out.cpu().numpy()[ok] == ref["tokens"][ok]).all()
    assert 0 < ref["accept_len"].mean() < w.k or w.B == 1   # both outcomes occur
    # an ERSD call afterwards finds its workspace in order
    from parity_util import check_verify
    res = ersd.verify(tgt, drf, seeds, inp["T"], temps=temps, want_rows=True)
    torch.cuda.synchronize()
    check_verify(inp, res)


def test_sequence_gsd_options_and_errors(ersd):
    w = wl.scaled(wl.CONFIGS["c2"], B=5, V=5000)
    inp = wl.make_inputs(w, call=9)
    tgt, drf, seeds = inp["target"].cuda(), inp["draft"].cuda(), inp["seeds"].cuda()
    seq = torch.tensor([7, 7, 9, 11, 12], dtype=torch.int32, device="cuda")
    off = torch.tensor([0, 5, 100, 3, 0], dtype=torch.int32, device="cuda")
    tok = torch.randint(0, w.V, (w.B, w.k), dtype=torch.int32, device="cuda")   # any tokens may be verified
    ws = torch.empty(ersd.ersd_workspace_bytes(w.B, w.k + 1), dtype=torch.uint8, device="cuda")
    ersd.ersd_workspace_init(ws)
    out = torch.empty(w.B, w.k + 1, dtype=torch.int32, device="cuda")
    acc = torch.empty(w.B, dtype=torch.int32, device="cuda")
    ersd.ersd_gsd_verify(tgt, drf, tok, seeds, 0.8, out, acc, ersd.make_opts(seq_ids=seq, pos_offsets=off, workspace=ws))
    torch.cuda.synchronize()
    assert (ws == 0).all()                                       # left zeroed
    ref = oracle.gsd_verify(wl.as_numpy_logits(inp["target"]), wl.as_numpy_logits(inp["draft"]), tok.cpu().numpy(),
                            wl.seeds_as_u64(inp["seeds"]), T=0.8, seq_ids=seq.cpu().numpy(), pos_offsets=off.cpu().numpy())
    assert not ambiguous(ref).any()
    assert (acc.cpu().numpy() == ref["accept_len"]).all() and (out.cpu().numpy() == ref["tokens"]).all()
    for bad_T in (0.0, -1.0, float("nan")):
        with pytest.raises(ersd.ErsdError) as e:
            ersd.ersd_gsd_verify(tgt, drf, tok, seeds, bad_T, out, acc)
        assert e.value.status == -1
    with pytest.raises(ersd.ErsdError) as e:
        ersd.ersd_gsd_verify(tgt, drf, None, seeds, 1.0, out, acc)
    assert e.value.status == -1
    # no drafts: one sample of the only target row
    ersd.ersd_gsd_verify(tgt[:, :1].contiguous(), None, None, seeds, 1.0, out[:, :1].contiguous(), acc)
    torch.cuda.synchronize()
    assert (acc == 0).all()


@pytest.mark.parametrize("parent,B,V", [(wl.TREE_4x4, 6, 20000), (wl.TREE_SPECINFER, 4, 151936), (wl.star_parent(5), 8, 4097),
                                         (wl.chain_parent(4), 5, 32000), ([-1], 3, 1000)])
def test_tree_gsd_against_the_oracle(ersd, parent, B, V):
    nodes = len(parent)
    w = wl.Workload("gsdtree", B=B, k=nodes - 1, V=V, dtype="bf16", sigma=0.7, T=1.0, config_id=50, parent=tuple(parent))
    inp = wl.make_inputs(w, call=2)
    tgt, drf, seeds = inp["target"].cuda(), inp["draft"].cuda(), inp["seeds"].cuda()
    _, max_c, nchild, rank = oracle.tree_shape(parent)
    arr = draft_tokens(ersd, drf, seeds, inp["T"], c=max_c)      # [B, nodes, max_c]: arrivals of every node's draft race
    tok = torch.full((B, nodes), -1, dtype=torch.int32, device="cuda")
    for n in range(1, nodes):
        tok[:, n] = arr[:, parent[n], rank[n]]
    D = ersd.ersd_tree_depth(parent)
    out = torch.full((B, D + 1), -9, dtype=torch.int32, device="cuda")
    acc = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    path = torch.full((B, D + 1), -9, dtype=torch.int32, device="cuda")
    ersd.ersd_gsd_verify_tree(tgt, drf, tok, parent, seeds, inp["T"], out, acc, ersd.make_opts(out_path=path))
    torch.cuda.synchronize()
    ref = oracle.gsd_verify_tree(wl.as_numpy_logits(inp["target"]), wl.as_numpy_logits(inp["draft"]), tok.cpu().numpy(),
                                 parent, wl.seeds_as_u64(inp["seeds"]), T=inp["T"])
    amb = ambiguous(ref)
    assert amb.sum() <= 1
    ok = ~amb
    assert (acc.cpu().numpy()[ok] == ref["accept_len"][ok]).all()
    assert (out.cpu().numpy()[ok] == ref["tokens"][ok]).all()
    assert (path.cpu().numpy()[ok] == ref["path"][ok]).all()


def test_gsd_and_ersd_acceptance_on_the_same_rows(ersd):
    """Section 3 on synthetic Zipf rows at vocabulary size: GSD accepts the first drafted token with
    probability 1 - D_TV, ERSD's match rate lies between D_HM and that (Lemma 3.1); summed over
    the rows of config 3's sigma = 1 point both counts fall within 4.5 sigma of those sums."""
    import math
    w = wl.scaled(wl.CONFIGS["c3"], B=64)
    inp = wl.make_inputs(w, call=1, sigma=1.0, T=1.0, device="cuda")
    tgt, drf, seeds = inp["target"], inp["draft"], inp["seeds"]
    res = ersd.verify(tgt, drf, seeds, 1.0)
    tok = draft_tokens(ersd, drf, seeds + 12345, 1.0)[..., 0].contiguous()     # drafted with races of their own
    out = torch.empty(w.B, w.k + 1, dtype=torch.int32, device="cuda")
    acc = torch.empty(w.B, dtype=torch.int32, device="cuda")
    ersd.ersd_gsd_verify(tgt, drf, tok, seeds, 1.0, out, acc)
    torch.cuda.synchronize()
    p = torch.softmax(tgt[:, 0].double(), -1)
    q = torch.softmax(drf[:, 0].double(), -1)
    a_gsd = (1.0 - 0.5 * (p - q).abs().sum(-1)).cpu().numpy()
    d_hm = (p * q / (p + q)).sum(-1).cpu().numpy()
    got_g = int((acc >= 1).sum().item())
    got_e = int((res["accept_len"] >= 1).sum().item())
    sd = math.sqrt((a_gsd * (1 - a_gsd)).sum())
    assert abs(got_g - a_gsd.sum()) < 4.5 * sd, (got_g, a_gsd.sum())
    assert d_hm.sum() - 4.5 * sd <= got_e <= a_gsd.sum() + 4.5 * sd, (got_e, d_hm.sum(), a_gsd.sum())
