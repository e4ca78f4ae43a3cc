"""Sequence verification on the cluster kernel (one thread-block cluster per position; calls of
few rows) against the CPU oracle, through the C boundary.  `kernel_path=2` forces the cluster
kernel, `1` the streaming one."""
import numpy as np
import pytest
import torch

from paper_2504_15475_b200 import workloads as wl

from parity_util import KEY_TOL, check_verify

pytestmark = pytest.mark.gpu

CLUSTER, STREAMING = 2, 1


@pytest.fixture(scope="module")
def ersd():
    from paper_2504_15475_b200 import binding
    binding.lib()
    assert torch.cuda.is_available()
    return binding


def run(ersd, inp, path, **kw):
    out = ersd.verify(inp["target"].cuda(), inp["draft"].cuda() if inp["draft"] is not None else None,
                      inp["seeds"].cuda(), inp["T"], temps=None if inp.get("temps") is None else inp["temps"].cuda(),
                      want_rows=True, kernel_path=path, **kw)
    torch.cuda.synchronize()
    return out


def same(a, b):
    return all((a[k] == b[k]).all() for k in a)


@pytest.mark.parametrize("name,scale", [("c1", {}), ("c2", {}), ("c3", dict(B=3)), ("c5", dict(B=4))])
def test_configurations(ersd, name, scale):
    w = wl.scaled(wl.CONFIGS[name], **scale)
    for call in (0, 1):
        inp = wl.make_inputs(w, call=call)
        out = run(ersd, inp, CLUSTER)
        check_verify(inp, out)
        assert same(out, run(ersd, inp, STREAMING))      # the two kernels decide in the same arithmetic


@pytest.mark.parametrize("V", [1, 5, 8, 9, 2047, 2048, 2049, 4100, 33000, 151936])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_vocabulary_sizes(ersd, V, dtype):
    ld = (V + 7) // 8 * 8                                # rows padded to 16-byte boundaries
    B, k = 2, 3
    g = torch.Generator().manual_seed(V)
    t = wl.zipf_rows(B * (k + 1), V, g, "cpu").view(B, k + 1, V)
    d = t[:, :k] + 0.7 * torch.randn(B, k, V, generator=g)
    big_t = torch.full((B, k + 1, ld), 60.0)
    big_d = torch.full((B, k, ld), 60.0)                 # the padding must never be raced
    big_t[:, :, :V] = t
    big_d[:, :, :V] = d
    big_t, big_d = wl._storage(big_t, dtype), wl._storage(big_d, dtype)
    seeds = wl.make_seeds(41, V % 977, B)
    tok = torch.empty(B, k + 1, dtype=torch.int32, device="cuda")
    acc = torch.empty(B, dtype=torch.int32, device="cuda")
    ersd.ersd_verify(big_t.cuda(), big_d.cuda(), seeds.cuda(), 0.9, tok, acc,
                     ersd.make_opts(ld_target=ld, ld_draft=ld, kernel_path=CLUSTER), V=V)
    torch.cuda.synchronize()
    import oracle
    ref = oracle.verify(wl.as_numpy_logits(big_t[:, :, :V].contiguous()),
                        wl.as_numpy_logits(big_d[:, :, :V].contiguous()), wl.seeds_as_u64(seeds), T=0.9)
    assert (tok.cpu().numpy() == ref["tokens"]).all() and (acc.cpu().numpy() == ref["accept_len"]).all()


def test_special_values_greedy_and_invalid_temperatures(ersd):
    V = 5000
    g = torch.Generator().manual_seed(9)
    t = torch.randn(5, 3, V, generator=g)
    d = t[:, :2] + 0.1 * torch.randn(5, 2, V, generator=g)
    t[0, 0, :] = float("-inf")                        # fully masked target row -> -1, nothing accepted
    t[1, 0, 5] = float("nan")
    t[1, 0, 100:] = float("-inf")
    d[1, 0, 4017] = float("inf")                      # +inf always wins (odd position, far into the row)
    t[2, 0, :] = float("-inf")
    t[2, 0, 123] = 0.0                                # single live token
    d[2, 0, :] = float("nan")
    d[2, 0, 123] = -3.0
    for dtype in ("f32", "bf16"):
        inp = dict(target=wl._storage(t, dtype), draft=wl._storage(d, dtype), seeds=wl.make_seeds(3, 0, 5),
                   T=0.8, temps=None, parent=None)
        out = run(ersd, inp, CLUSTER)
        check_verify(inp, out)
        assert same(out, run(ersd, inp, STREAMING))
        tok = out["tokens"].cpu().numpy()
        assert tok[0, 0] == -1 and out["accept_len"][0].item() == 0
        assert out["draft_tok"][1, 0].item() == 4017
        assert tok[2, 0] == 123 and out["accept_len"][2].item() >= 1
        # greedy: the lowest index among the maxima, draft and target alike
        inp0 = dict(inp, T=0.0)
        out0 = run(ersd, inp0, CLUSTER)
        check_verify(inp0, out0)
        assert same(out0, run(ersd, inp0, STREAMING))
        # per-row temperatures, one of them invalid: that row has no arrivals
        temps = torch.tensor([[1.0, 0.5, 2.0]] * 5)
        temps[3, 1] = -1.0
        inp1 = dict(inp, temps=temps)
        out1 = run(ersd, inp1, CLUSTER)
        assert out1["target_tok"][3, 1].item() == -1 and out1["draft_tok"][3, 1].item() == -1
        assert out1["accept_len"][3].item() <= 1
        assert same(out1, run(ersd, inp1, STREAMING))


def test_sequence_ids_position_offsets_and_per_sequence_temperatures(ersd):
    w = wl.Workload("opts", B=4, k=3, V=3000, dtype="bf16", sigma=0.8, T=1.0, config_id=44)
    inp = wl.make_inputs(w)
    inp["temps"] = torch.tensor([[0.5, 0.7, 1.0, 1.3], [1.0, 1.0, 0.0, 1.0], [2.0, 0.6, 0.6, 0.6], [1.0, 0.9, 1.0, 1.0]])
    seq = torch.tensor([7, 7, 9, 1000000], dtype=torch.int32)
    off = torch.tensor([0, 4, 123456, 1], dtype=torch.int32)
    out = run(ersd, inp, CLUSTER, seq_ids=seq.cuda(), pos_offsets=off.cuda())
    check_verify(inp, out, seq_ids=seq.numpy().astype(np.uint32), pos_offsets=off.numpy().astype(np.uint32))
    assert same(out, run(ersd, inp, STREAMING, seq_ids=seq.cuda(), pos_offsets=off.cuda()))


def test_identical_rows_accept_everything_and_k0(ersd):
    B, k, V = 3, 6, 40000
    g = torch.Generator().manual_seed(2)
    t = wl.zipf_rows(B * (k + 1), V, g, "cpu").view(B, k + 1, V).to(torch.bfloat16)
    inp = dict(target=t, draft=t[:, :k].contiguous(), seeds=wl.make_seeds(5, 0, B), T=1.0, temps=None, parent=None)
    out = run(ersd, inp, CLUSTER)
    check_verify(inp, out)
    assert (out["accept_len"] == k).all() and (out["tokens"] >= 0).all()
    # no drafted position at all: one race per sequence
    tok = torch.empty(B, 1, dtype=torch.int32, device="cuda")
    acc = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    ersd.ersd_verify(t[:, :1].contiguous().cuda(), None, inp["seeds"].cuda(), 1.0, tok, acc,
                     ersd.make_opts(kernel_path=CLUSTER))
    torch.cuda.synchronize()
    assert (acc == 0).all() and (tok[:, 0] == out["target_tok"][:, 0]).all()


def test_given_tokens(ersd):
    import oracle
    w = wl.scaled(wl.CONFIGS["c2"], B=6)
    inp = wl.make_inputs(w, call=91)
    dev = {k: (v.cuda() if torch.is_tensor(v) else v) for k, v in inp.items()}
    drafted = torch.empty(w.B, w.k, 1, dtype=torch.int32, device="cuda")
    ersd.ersd_race_sample(dev["draft"], dev["seeds"], inp["T"], drafted, ersd.make_opts(kernel_path=CLUSTER))
    dtok = drafted[..., 0].contiguous()
    spoil = torch.zeros_like(dtok, dtype=torch.bool)
    spoil[::3, 1] = True                              # rejections at position 1 in every third sequence
    dtok = torch.where(spoil, (dtok + 1) % w.V, dtok)
    tok = torch.full((w.B, w.k + 1), -7, dtype=torch.int32, device="cuda")
    acc = torch.full((w.B,), -7, dtype=torch.int32, device="cuda")
    ttok = torch.empty(w.B, w.k + 1, dtype=torch.int32, device="cuda")
    tkey = torch.empty(w.B, w.k + 1, dtype=torch.float32, device="cuda")
    gtok = torch.empty(w.B, w.k, dtype=torch.int32, device="cuda")
    ersd.ersd_verify_tokens(dev["target"], dtok, dev["seeds"], inp["T"], tok, acc,
                            ersd.make_opts(out_target_tok=ttok, out_target_key=tkey, out_draft_tok=gtok,
                                           kernel_path=CLUSTER))
    torch.cuda.synchronize()
    ref = oracle.verify_tokens(wl.as_numpy_logits(inp["target"]), dtok.cpu().numpy(),
                               wl.seeds_as_u64(inp["seeds"]), T=inp["T"])
    assert (ttok.cpu().numpy() == ref["target_tok"]).all()
    assert (tok.cpu().numpy() == ref["tokens"]).all() and (acc.cpu().numpy() == ref["accept_len"]).all()
    assert np.abs(tkey.cpu().numpy() - ref["target_key"][..., 0]).max() <= KEY_TOL
    assert (gtok == dtok).all()


def test_workspace_shared_with_the_streaming_kernel_over_many_calls(ersd):
    """Both kernels count a sequence's finished positions in the same workspace and leave it
    clean: calls of either kind, in any order, on one caller-owned workspace."""
    w = wl.scaled(wl.CONFIGS["c2"], B=5)
    ws = torch.zeros(ersd.ersd_workspace_bytes(w.B, w.k + 1), dtype=torch.uint8, device="cuda")
    ersd.ersd_workspace_init(ws)
    tok = torch.empty(w.B, w.k + 1, dtype=torch.int32, device="cuda")
    acc = torch.empty(w.B, dtype=torch.int32, device="cuda")
    import oracle
    for call in range(24):
        inp = wl.make_inputs(w, call=call)
        path = (CLUSTER, STREAMING, CLUSTER, CLUSTER)[call % 4]
        ersd.ersd_verify(inp["target"].cuda(), inp["draft"].cuda(), inp["seeds"].cuda(), inp["T"], tok, acc,
                         ersd.make_opts(kernel_path=path, workspace=ws))
        torch.cuda.synchronize()
        ref = oracle.verify(wl.as_numpy_logits(inp["target"]), wl.as_numpy_logits(inp["draft"]),
                            wl.seeds_as_u64(inp["seeds"]), T=inp["T"])
        assert (tok.cpu().numpy() == ref["tokens"]).all() and (acc.cpu().numpy() == ref["accept_len"]).all()


def test_no_alloc_entry_takes_the_cluster_kernel_too(ersd):
    w = wl.scaled(wl.CONFIGS["c2"], B=4)
    inp = wl.make_inputs(w, call=3)
    tok = torch.empty(w.B, w.k + 1, dtype=torch.int32, device="cuda")
    acc = torch.empty(w.B, dtype=torch.int32, device="cuda")
    ref = run(ersd, inp, STREAMING)
    for path in (0, CLUSTER, STREAMING):
        ersd.ersd_verify_noalloc(inp["target"].cuda(), inp["draft"].cuda(), inp["seeds"].cuda(), inp["T"], tok, acc,
                                 ersd.make_opts(kernel_path=path))
        torch.cuda.synchronize()
        assert (tok == ref["tokens"]).all() and (acc == ref["accept_len"]).all()


@pytest.mark.parametrize("gap", [1e-4, -1e-4])
def test_screening_keys_too_close_to_call(ersd, gap):
    """Draft and target rows whose two best keys differ by less than the screening precision:
    the exact key decides both, whichever of the two tokens leads."""
    import oracle
    B, k, V, T = 4, 2, 128256, 1.0
    seeds = wl.make_seeds(31, 1, B)
    flat = np.zeros((B, k + 1, V), dtype=np.float32)
    tok2, key2 = oracle.race_sample(flat, wl.seeds_as_u64(seeds), T=T, c=2)
    t = torch.zeros(B, k + 1, V)
    for b in range(B):
        for r in range(k + 1):
            second = int(tok2[b, r, 1])
            t[b, r, second] = float((key2[b, r, 1] - key2[b, r, 0] - gap) * T)
    d = t[:, :k].clone()
    d[0, 0] = 0.0                                      # one drafted position without the engineered tie
    inp = dict(target=t, draft=d, seeds=seeds, T=T, temps=None, parent=None)
    out = run(ersd, inp, CLUSTER)
    check_verify(inp, out)
    assert same(out, run(ersd, inp, STREAMING))
    want = tok2[:, :, 0] if gap > 0 else tok2[:, :, 1]
    assert (out["target_tok"].cpu().numpy() == want).all()


def test_a_chain_given_as_a_tree(ersd):
    """A draft tree without branching (what the tree builder returns when first children are
    accepted often) takes the cluster kernel too, with the tree entry point's output layout."""
    parent, expected = ersd.ersd_optimal_tree([0.9, 0.02], 6)
    assert list(parent) == wl.chain_parent(6) and expected > 3.0
    w = wl.Workload("chain_tree", B=3, k=6, V=30000, dtype="bf16", sigma=0.5, T=0.9, config_id=61,
                    parent=tuple(parent))
    inp = wl.make_inputs(w)
    outs = {}
    for path in (CLUSTER, STREAMING):
        out = ersd.verify(inp["target"].cuda(), inp["draft"].cuda(), inp["seeds"].cuda(), inp["T"],
                          parent=list(parent), want_rows=True, kernel_path=path)
        torch.cuda.synchronize()
        check_verify(inp, out)
        outs[path] = out
    assert same(outs[CLUSTER], outs[STREAMING])
    assert (outs[CLUSTER]["draft_tok"][:, 0] == -1).all()


def test_where_the_cluster_kernel_does_not_apply(ersd):
    B, V = 2, 1024
    seeds = wl.make_seeds(1, 0, B).cuda()
    # trees whose races want more than 32 arrivals
    parent = wl.star_parent(33)
    t = torch.randn(B, len(parent), V).to(torch.bfloat16).cuda()
    tok = torch.empty(B, 2, dtype=torch.int32, device="cuda")
    acc = torch.empty(B, dtype=torch.int32, device="cuda")
    with pytest.raises(ersd.ErsdError) as e:
        ersd.ersd_verify_tree(t, t, parent, seeds, 1.0, tok, acc, ersd.make_opts(kernel_path=CLUSTER))
    assert e.value.status == -3
    # more than 32 positions
    k = 32
    t = torch.randn(B, k + 1, V).to(torch.bfloat16).cuda()
    tok = torch.empty(B, k + 1, dtype=torch.int32, device="cuda")
    with pytest.raises(ersd.ErsdError) as e:
        ersd.ersd_verify(t, t[:, :k].contiguous(), seeds, 1.0, tok, acc, ersd.make_opts(kernel_path=CLUSTER))
    assert e.value.status == -3
    ersd.ersd_verify(t, t[:, :k].contiguous(), seeds, 1.0, tok, acc, None)   # the library picks the streaming kernel
    torch.cuda.synchronize()
    assert (acc == k).all()
