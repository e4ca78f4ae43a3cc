"""The latency path for races that want several arrivals (ersd_cluster_top_kernel: one thread-block
cluster per position, every block hands its own first arrivals to the cluster's first block)
against the CPU oracle, through the C boundary: race sampling with top_c > 1 (batch drafting) and
tree verification (Algorithm 5).  `kernel_path=2` forces the cluster kernel, `1` the streaming one."""
import numpy as np
import pytest
import torch

from paper_2504_15475_b200 import workloads as wl

from parity_util import check_sample, check_verify

pytestmark = pytest.mark.gpu

CLUSTER, STREAMING = 2, 1


@pytest.fixture(scope="module")
def ersd():
    from paper_2504_15475_b200 import binding
    binding.lib()
    assert torch.cuda.is_available()
    return binding


def sample(ersd, logits, seeds, T, c, path, **kw):
    """First c arrivals of the races over `logits` [B, R, V]; rows are padded to a multiple of
    eight elements with large logits that must never arrive."""
    B, R, V = logits.shape
    ld = (V + 7) // 8 * 8
    big = torch.full((B, R, ld), 60.0, dtype=logits.dtype)
    big[:, :, :V] = logits
    tok = torch.full((B, R, c), -7, dtype=torch.int32, device="cuda")
    key = torch.full((B, R, c), -7.0, dtype=torch.float32, device="cuda")
    ersd.ersd_race_sample(big.cuda(), seeds.cuda(), T, tok,
                          ersd.make_opts(kernel_path=path, top_c=c, out_key=key, ld_target=ld, **kw), V=V)
    torch.cuda.synchronize()
    return tok, key


def verify_tree(ersd, inp, path, **kw):
    out = ersd.verify(inp["target"].cuda(), inp["draft"].cuda(), inp["seeds"].cuda(), inp["T"],
                      parent=list(inp["parent"]), want_rows=True, kernel_path=path, **kw)
    torch.cuda.synchronize()
    return out


def same(a, b):
    return all((a[k] == b[k]).all() for k in a)


# ------------------------------------------------------------------ sampling: first c arrivals
@pytest.mark.parametrize("V", [8, 40, 2047, 2049, 8200, 33000, 128256, 151936, 250001])
@pytest.mark.parametrize("c", [2, 8, 32])
def test_first_arrivals_at_many_vocabulary_sizes(ersd, V, c):
    B, R = 2, 2
    g = torch.Generator().manual_seed(V + c)
    for dtype in (torch.bfloat16, torch.float32):
        logits = wl.zipf_rows(B * R, V, g, "cpu").view(B, R, V).to(dtype)
        seeds = wl.make_seeds(71, (V + c) % 1000, B)
        tok, key = sample(ersd, logits, seeds, 0.9, c, CLUSTER)
        assert check_sample(logits, seeds, 0.9, tok, key, c=c) == 0
        assert "ersd_cluster_top_kernel" in ersd.ersd_last_launch()
        tok_s, key_s = sample(ersd, logits, seeds, 0.9, c, STREAMING)
        assert (tok == tok_s).all() and (key == key_s).all()     # the same arithmetic decides in both kernels


@pytest.mark.parametrize("c", [3, 4, 17, 31])
@pytest.mark.parametrize("T", [0.4, 1.0, 2.0])
def test_first_arrivals_at_full_vocabulary(ersd, c, T):
    B, R, V = 3, 2, 128256
    g = torch.Generator().manual_seed(int(10 * T) + c)
    logits = wl.zipf_rows(B * R, V, g, "cpu").view(B, R, V).to(torch.bfloat16)
    logits[1, 1, 5::2] = float("-inf")                     # half of one row masked
    seeds = wl.make_seeds(72, c, B)
    tok, key = sample(ersd, logits, seeds, T, c, CLUSTER)
    assert check_sample(logits, seeds, T, tok, key, c=c) == 0
    assert all(len(set(r.tolist())) == c for r in tok.view(-1, c).cpu())


def test_every_cluster_size_gives_the_same_arrivals(ersd):
    B, V, c = 3, 40000, 8                                 # 20 tiles: clusters of 1 to 16 blocks stage 20 to 2 tiles each
    g = torch.Generator().manual_seed(78)
    logits = wl.zipf_rows(B, V, g, "cpu").view(B, 1, V).to(torch.bfloat16)
    seeds = wl.make_seeds(73, 0, B)
    ref_tok, ref_key = sample(ersd, logits, seeds, 1.0, c, STREAMING)
    assert check_sample(logits, seeds, 1.0, ref_tok, ref_key, c=c) == 0
    for blocks in (1, 2, 4, 8, 16):
        tok, key = sample(ersd, logits, seeds, 1.0, c, CLUSTER, split_v=blocks)
        assert (tok == ref_tok).all() and (key == ref_key).all()


def test_two_blocks_to_a_row_of_full_length(ersd):
    """Two blocks to a row of 128256 logits and 32 arrivals wanted: 32 tiles to a block, hundreds of
    groups on its list and a hundred survivors."""
    B, V, c = 2, 128256, 32
    g = torch.Generator().manual_seed(79)
    logits = wl.zipf_rows(B, V, g, "cpu").view(B, 1, V).to(torch.bfloat16)
    seeds = wl.make_seeds(73, 1, B)
    tok, key = sample(ersd, logits, seeds, 1.0, c, CLUSTER, split_v=2)
    assert "ersd_cluster_top_kernel" in ersd.ersd_last_launch()
    assert check_sample(logits, seeds, 1.0, tok, key, c=c) == 0
    tok_s, key_s = sample(ersd, logits, seeds, 1.0, c, STREAMING)
    assert (tok == tok_s).all() and (key == key_s).all()


def test_rows_with_fewer_tokens_than_arrivals_wanted(ersd):
    """Rows where fewer than c tokens have positive probability: the arrivals there are, then -1
    and +inf keys; a row of NaN or without any token gives no arrival at all."""
    B, R, V, c = 1, 4, 50000, 8
    logits = torch.full((B, R, V), float("-inf"))
    logits[0, 0, [3, 49999, 20000]] = torch.tensor([1.0, 2.0, 0.5])
    logits[0, 1, 7] = 0.0
    logits[0, 3, :] = float("nan")
    seeds = wl.make_seeds(74, 0, B)
    tok, key = sample(ersd, logits, seeds, 1.0, c, CLUSTER)
    assert check_sample(logits, seeds, 1.0, tok, key, c=c) == 0
    t = tok.cpu().numpy()[0]
    assert sorted(t[0, :3].tolist()) == [3, 20000, 49999] and (t[0, 3:] == -1).all()
    assert t[1, 0] == 7 and (t[1, 1:] == -1).all() and (t[2:] == -1).all()
    assert torch.isinf(key[0, 0, 3:]).all() and torch.isinf(key[0, 2:]).all()


@pytest.mark.parametrize("V", [4096, 128256])
def test_greedy_rows_of_tied_logits(ersd, V):
    """T = 0 on rows whose logits tie: every index has the same key, the order is by index, and a
    block finds far more survivors than it lists (it then picks its arrivals one at a time)."""
    B, R, c = 2, 2, 8
    logits = torch.zeros(B, R, V, dtype=torch.bfloat16)
    logits[0, 1, 100:] = -1.0                              # ties among the first hundred only
    logits[1, 0, ::3] = 2.0                                # every third index leads
    logits[1, 1, V - 5:] = 5.0                             # fewer leaders than arrivals wanted, then the tied rest
    seeds = wl.make_seeds(75, 0, B)
    tok, key = sample(ersd, logits, seeds, 0.0, c, CLUSTER)
    assert check_sample(logits, seeds, 0.0, tok, key, c=c) == 0
    t = tok.cpu().numpy()
    assert t[0, 0].tolist() == list(range(8)) and t[0, 1].tolist() == list(range(8))
    assert t[1, 0].tolist() == list(range(0, 24, 3))
    assert t[1, 1].tolist() == list(range(V - 5, V)) + [0, 1, 2]
    tok_s, key_s = sample(ersd, logits, seeds, 0.0, c, STREAMING)
    assert (tok == tok_s).all() and (key == key_s).all()
    if V > 100000:   # clusters of four: a block has more tied groups (4096) than its list holds and goes through all its indices
        tok_4, key_4 = sample(ersd, logits, seeds, 0.0, c, CLUSTER, split_v=4)
        assert (tok == tok_4).all() and (key == key_4).all()


@pytest.mark.parametrize("c", [2, 4, 8, 32])
@pytest.mark.parametrize("gap", [1e-4, -1e-4])
def test_last_arrival_too_close_to_call_by_screening(ersd, c, gap):
    """The c-th and the (c+1)-th arrival closer than the screening precision (about 1.4e-3) but far
    beyond the near-tie window: the exact keys must decide which of the two is among the first c."""
    import oracle
    B, V, T = 4, 128256, 1.0
    seeds = wl.make_seeds(76, c, B)
    flat = np.zeros((B, 1, V), dtype=np.float32)
    tokc, keyc = oracle.race_sample(flat, wl.seeds_as_u64(seeds), T=T, c=c + 1)
    logits = torch.zeros(B, 1, V, dtype=torch.float32)
    want = []
    for b in range(B):
        last, after = int(tokc[b, 0, c - 1]), int(tokc[b, 0, c])
        # raise the logit of the (c+1)-th arrival until its key sits `gap` above (or below) the c-th
        logits[b, 0, after] = float((keyc[b, 0, c] - keyc[b, 0, c - 1] - gap) * T)
        want.append(last if gap > 0 else after)
    tok, key = sample(ersd, logits, seeds, T, c, CLUSTER)
    assert check_sample(logits, seeds, T, tok, key, c=c) == 0
    got = tok.cpu().numpy()[:, 0]
    for b in range(B):
        assert want[b] in got[b].tolist()
        assert got[b, :c - 1].tolist() == tokc[b, 0, :c - 1].tolist()
    tok_s, key_s = sample(ersd, logits, seeds, T, c, STREAMING)
    assert (tok == tok_s).all() and (key == key_s).all()


def test_per_row_temperatures_and_counters(ersd):
    B, R, V, c = 2, 3, 70000, 4
    g = torch.Generator().manual_seed(5)
    logits = wl.zipf_rows(B * R, V, g, "cpu").view(B, R, V).to(torch.bfloat16)
    seeds = wl.make_seeds(77, 0, B)
    temps = torch.tensor([[0.5, 0.0, 1.5], [1.0, 2.0, 0.25]], dtype=torch.float32)
    seq_ids = torch.tensor([9, 4], dtype=torch.int32)
    off = torch.tensor([100, 7], dtype=torch.int32)
    tok, key = sample(ersd, logits, seeds, 1.0, c, CLUSTER, temps=temps.cuda(), temp_strides=(R, 1),
                      seq_ids=seq_ids.cuda(), pos_offsets=off.cuda())
    assert check_sample(logits, seeds, 1.0, tok, key, c=c, temps=temps.numpy(),
                        seq_ids=seq_ids.numpy().astype(np.uint32), pos_offsets=off.numpy().astype(np.uint32)) == 0


# ------------------------------------------------------------------ tree verification
TREES = {
    "star8": wl.star_parent(8),
    "c4": wl.TREE_4x4,
    "specinfer": wl.TREE_SPECINFER,
    "bushy": (-1, 0, 0, 0, 1, 1, 1, 2, 2, 4, 4, 4, 4, 9, 9),
    "star32": wl.star_parent(32),
}


@pytest.mark.parametrize("shape", sorted(TREES))
@pytest.mark.parametrize("B,V,dtype", [(1, 128256, "bf16"), (3, 9000, "bf16"), (2, 151936, "bf16"), (2, 40000, "f32")])
def test_tree_verification(ersd, shape, B, V, dtype):
    parent = tuple(TREES[shape])
    for sigma in (0.3, 1.5):                               # drafts that are accepted often, and seldom
        w = wl.Workload("tree_" + shape, B=B, k=len(parent) - 1, V=V, dtype=dtype, sigma=sigma, T=0.9,
                        config_id=80, parent=parent)
        inp = wl.make_inputs(w, call=int(sigma * 10))
        out = verify_tree(ersd, inp, CLUSTER)
        assert "ersd_cluster_top_kernel" in ersd.ersd_last_launch()
        check_verify(inp, out)
        assert same(out, verify_tree(ersd, inp, STREAMING))


@pytest.mark.parametrize("V", [4096, 128256])
def test_greedy_tree_over_tied_logits(ersd, V):
    """T = 0 with draft and target rows of equal logits everywhere: both roles of a position list
    every group (more than a block's candidate list holds), arrivals are the lowest indices, the
    target's winner is the first child's token at every level."""
    parent = tuple(TREES["c4"])
    B, n = 2, len(parent)
    t = torch.zeros(B, n, V, dtype=torch.bfloat16)
    t[1, :, 1000:] = -3.0                                  # second sequence: ties among the first thousand only
    inp = dict(target=t, draft=t.clone(), seeds=wl.make_seeds(83, 0, B), T=0.0, temps=None, parent=list(parent))
    out = verify_tree(ersd, inp, CLUSTER)
    assert "ersd_cluster_top_kernel" in ersd.ersd_last_launch()
    check_verify(inp, out)
    assert (out["accept_len"] == 4).all() and (out["tokens"] == 0).all()
    assert out["draft_tok"][0, 1:5].tolist() == [0, 1, 2, 3]
    assert same(out, verify_tree(ersd, inp, STREAMING))


def test_tree_verification_repeats_bit_for_bit_and_leaves_the_workspace_clean(ersd):
    parent = tuple(TREES["c4"])
    w = wl.Workload("tree_rep", B=2, k=len(parent) - 1, V=128256, dtype="bf16", sigma=0.5, T=1.0, config_id=81,
                    parent=parent)
    inp = wl.make_inputs(w)
    first = verify_tree(ersd, inp, CLUSTER)
    check_verify(inp, first)
    for n in range(20):
        path = STREAMING if n % 5 == 4 else CLUSTER        # the two kernels share the workspace's counters
        assert same(first, verify_tree(ersd, inp, path))


def test_small_trees_take_this_kernel_by_default(ersd):
    parent = tuple(TREES["star8"])
    w = wl.Workload("tree_def", B=1, k=8, V=128256, dtype="bf16", sigma=0.5, T=1.0, config_id=82, parent=parent)
    inp = wl.make_inputs(w)
    out = ersd.verify(inp["target"].cuda(), inp["draft"].cuda(), inp["seeds"].cuda(), inp["T"],
                      parent=list(parent), want_rows=True)
    torch.cuda.synchronize()
    assert "ersd_cluster_top_kernel" in ersd.ersd_last_launch()
    assert "1 row(s) per cluster>: 10 clusters" in ersd.ersd_last_launch()   # root's draft row, nine target rows
    check_verify(inp, out)
    mid = wl.scaled(wl.CONFIGS["c4"], B=4, V=128256)      # 68 positions: draft and target row of a node in one cluster
    inp = wl.make_inputs(mid)
    out = ersd.verify(inp["target"].cuda(), inp["draft"].cuda(), inp["seeds"].cuda(), inp["T"],
                      parent=list(inp["parent"]), want_rows=True)
    torch.cuda.synchronize()
    assert "2 row(s) per cluster>: 68 clusters" in ersd.ersd_last_launch()
    check_verify(inp, out)
    big = wl.scaled(wl.CONFIGS["c4"], B=8)                # 136 rows: the streaming kernel's job
    inp = wl.make_inputs(big)
    out = ersd.verify(inp["target"].cuda(), inp["draft"].cuda(), inp["seeds"].cuda(), inp["T"],
                      parent=list(inp["parent"]), want_rows=True)
    torch.cuda.synchronize()
    assert "ersd_race_kernel" in ersd.ersd_last_launch()
    check_verify(inp, out)


def test_where_this_kernel_does_not_apply(ersd):
    B, V = 1, 4096
    seeds = wl.make_seeds(1, 0, B).cuda()
    tok = torch.empty(B, 1, 33, dtype=torch.int32, device="cuda")
    row = torch.randn(B, 1, V).to(torch.bfloat16).cuda()
    with pytest.raises(ersd.ErsdError) as e:               # more than 32 arrivals per race
        ersd.ersd_race_sample(row, seeds, 1.0, tok, ersd.make_opts(kernel_path=CLUSTER, top_c=33))
    assert e.value.status == -3
    near = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(ersd.ErsdError) as e:               # near-ties are counted by the streaming kernel
        ersd.ersd_race_sample(row, seeds, 1.0, tok, ersd.make_opts(kernel_path=CLUSTER, top_c=4, near_tie_count=near))
    assert e.value.status == -3
    parent = wl.star_parent(33)
    t = torch.randn(B, len(parent), V).to(torch.bfloat16).cuda()
    out = torch.empty(B, 2, dtype=torch.int32, device="cuda")
    acc = torch.empty(B, dtype=torch.int32, device="cuda")
    with pytest.raises(ersd.ErsdError) as e:
        ersd.ersd_verify_tree(t, t, parent, seeds, 1.0, out, acc, ersd.make_opts(kernel_path=CLUSTER))
    assert e.value.status == -3
    ersd.ersd_verify_tree(t, t, parent, seeds, 1.0, out, acc, None)    # the library picks the streaming kernel
    torch.cuda.synchronize()
    assert (acc == 1).all()                                # draft rows = target rows: the first child is accepted
