"""The latency path of race sampling (one thread-block cluster per logit row) against the CPU
oracle, through the C boundary.  `kernel_path=2` forces the cluster kernel, `1` the streaming one."""
import numpy as np
import pytest
import torch

from paper_2504_15475_b200 import workloads as wl

from parity_util import check_sample

pytestmark = pytest.mark.gpu

CLUSTER, STREAMING = 2, 1


@pytest.fixture(scope="module")
def ersd():
    from paper_2504_15475_b200 import binding
    binding.lib()
    assert torch.cuda.is_available()
    return binding


def sample(ersd, logits, seeds, T, path, **kw):
    """Races `logits` [B, R, V] from rows padded to a multiple of eight elements (so that rows of
    any length start on 16-byte boundaries); the padding holds large logits that must never win."""
    B, R, V = logits.shape
    ld = (V + 7) // 8 * 8
    big = torch.full((B, R, ld), 60.0, dtype=logits.dtype)
    big[:, :, :V] = logits
    tok = torch.full((B, R, 1), -7, dtype=torch.int32, device="cuda")
    key = torch.full((B, R, 1), -7.0, dtype=torch.float32, device="cuda")
    ersd.ersd_race_sample(big.cuda(), seeds.cuda(), T, tok,
                          ersd.make_opts(kernel_path=path, out_key=key, ld_target=ld, **kw), V=V)
    torch.cuda.synchronize()
    return tok, key


# one tile is 2048 indices; a cluster of 16 blocks holds 64 tiles at a time (131072 indices)
@pytest.mark.parametrize("V", [1, 7, 8, 9, 1023, 2048, 2049, 4100, 8192, 8200, 20000, 33000, 65536, 128256,
                               131072, 131080, 151936, 300001])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_vocabulary_sizes(ersd, V, dtype):
    B, R = 2, 3
    g = torch.Generator().manual_seed(V)
    logits = wl.zipf_rows(B * R, V, g, "cpu").view(B, R, V).to(dtype)
    seeds = wl.make_seeds(21, V % 1000, B)
    tok, key = sample(ersd, logits, seeds, 0.9, CLUSTER)
    assert check_sample(logits, seeds, 0.9, tok, key) == 0


@pytest.mark.parametrize("T", [0.3, 1.0, 2.5])
def test_many_rows_at_full_vocabulary(ersd, T):
    B, R, V = 48, 2, 128256
    g = torch.Generator().manual_seed(int(T * 10))
    logits = wl.zipf_rows(B * R, V, g, "cpu").view(B, R, V).to(torch.bfloat16)
    seeds = wl.make_seeds(22, int(T * 10), B)
    tok, key = sample(ersd, logits, seeds, T, CLUSTER)
    assert check_sample(logits, seeds, T, tok, key) <= 1          # near-tie rows, if any
    tok_s, key_s = sample(ersd, logits, seeds, T, STREAMING)
    assert (tok == tok_s).all() and (key == key_s).all()          # the two kernels decide in the same arithmetic


def test_flat_and_peaked_rows(ersd):
    V = 128256
    flat = torch.zeros(1, 1, V)
    peaked = torch.full((1, 1, V), -30.0)
    peaked[0, 0, 77777] = 5.0
    two = torch.full((1, 1, V), -40.0)
    two[0, 0, 5] = 1.0
    two[0, 0, 128255] = 1.0
    logits = torch.cat([flat, peaked, two], 0).to(torch.bfloat16)
    seeds = wl.make_seeds(23, 0, 3)
    for T in (0.5, 1.0):
        tok, key = sample(ersd, logits, seeds, T, CLUSTER)
        assert check_sample(logits, seeds, T, tok, key) == 0
    assert tok[1, 0, 0].item() == 77777


def test_special_values(ersd):
    V = 5003
    g = torch.Generator().manual_seed(9)
    z = torch.randn(6, 1, V, generator=g)
    z[0, 0, :] = float("-inf")                     # nothing has positive probability: -1
    z[1, 0, 5] = float("nan")
    z[1, 0, 100:] = float("-inf")
    z[2, 0, 4017] = float("inf")                   # +inf always wins
    z[2, 0, 5002] = float("inf")                   # ... the lowest index among several
    z[3, 0, :] = float("nan")
    z[3, 0, 2048] = -3.0                           # single live token
    z[4, 0, :] = float("nan")                      # -1
    z[5, 0, :] = float("-inf")
    z[5, 0, 5002] = -10.0                          # a live token in the ragged last group
    for dtype in (torch.float32, torch.bfloat16):
        logits = z.to(dtype)
        seeds = wl.make_seeds(3, 0, 6)
        tok, key = sample(ersd, logits, seeds, 0.8, CLUSTER)
        assert check_sample(logits, seeds, 0.8, tok, key) == 0
        t = tok[:, 0, 0].cpu().tolist()
        assert t[0] == -1 and t[2] == 4017 and t[3] == 2048 and t[4] == -1 and t[5] == 5002
        assert torch.isinf(key[0, 0, 0]) and key[0, 0, 0] > 0
        assert torch.isinf(key[2, 0, 0]) and key[2, 0, 0] < 0


def test_greedy_rows_take_the_lowest_index_among_the_maxima(ersd):
    B, R, V = 2, 2, 70000
    g = torch.Generator().manual_seed(1)
    logits = (torch.randn(B, R, V, generator=g) * 0.3).to(torch.bfloat16)   # bf16: many equal maxima
    logits[1, 1, :] = 0.25                                                   # all equal: index 0
    seeds = wl.make_seeds(5, 0, B)
    tok, key = sample(ersd, logits, seeds, 0.0, CLUSTER)
    assert check_sample(logits, seeds, 0.0, tok, key) == 0
    f = logits.float()
    am = (f == f.max(-1, keepdim=True).values).float().argmax(-1)
    assert (tok[..., 0].cpu() == am).all() and tok[1, 1, 0].item() == 0


def test_per_row_temperatures_sequence_ids_offsets_and_strides(ersd):
    B, R, V, ld = 4, 3, 3000, 3008
    g = torch.Generator().manual_seed(44)
    big = wl.zipf_rows(B * R, ld, g, "cpu").view(B, R, ld).to(torch.bfloat16)
    logits = big[:, :, :V].contiguous()
    temps = torch.tensor([[0.5, 0.7, 1.0], [1.0, 0.0, 1.0], [2.0, 0.6, 0.6], [1.0, -1.0, float("nan")]])
    seq = torch.tensor([7, 7, 9, 1000000], dtype=torch.int32)
    off = torch.tensor([0, 4, 123456, 1], dtype=torch.int32)
    seeds = wl.make_seeds(6, 0, B)
    tok = torch.full((B, R, 1), -7, dtype=torch.int32, device="cuda")
    key = torch.full((B, R, 1), -7.0, dtype=torch.float32, device="cuda")
    opts = ersd.make_opts(kernel_path=CLUSTER, out_key=key, ld_target=ld, temps=temps.cuda(), temp_strides=(R, 1),
                          seq_ids=seq.cuda(), pos_offsets=off.cuda())
    ersd.ersd_race_sample(big.cuda(), seeds.cuda(), 1.0, tok, opts, V=V)
    torch.cuda.synchronize()
    # rows with an invalid temperature have no arrivals (the oracle has no notion of them)
    assert tok[3, 1, 0].item() == -1 and tok[3, 2, 0].item() == -1
    temps_ok = temps.clone()
    temps_ok[3, 1] = 1.0
    temps_ok[3, 2] = 1.0
    ersd.ersd_race_sample(big.cuda(), seeds.cuda(), 1.0, tok,
                          ersd.make_opts(kernel_path=CLUSTER, out_key=key, ld_target=ld, temps=temps_ok.cuda(),
                                         temp_strides=(R, 1), seq_ids=seq.cuda(), pos_offsets=off.cuda()), V=V)
    torch.cuda.synchronize()
    assert check_sample(logits, seeds, 1.0, tok, key, temps=temps_ok.numpy(),
                        seq_ids=seq.numpy().astype(np.uint32), pos_offsets=off.numpy().astype(np.uint32)) == 0


def test_where_the_cluster_kernel_does_not_apply(ersd):
    B, R, V = 2, 2, 1003
    logits = torch.randn(B, R, V).to(torch.bfloat16).cuda()      # rows of 2006 bytes: not 16-byte aligned
    seeds = wl.make_seeds(1, 0, B).cuda()
    tok = torch.empty(B, R, 33, dtype=torch.int32, device="cuda")
    with pytest.raises(ersd.ErsdError) as e:
        ersd.ersd_race_sample(logits, seeds, 1.0, tok, ersd.make_opts(kernel_path=CLUSTER))
    assert e.value.status == -3
    ok = torch.randn(B, R, 1024).to(torch.bfloat16).cuda()
    with pytest.raises(ersd.ErsdError) as e:   # (up to 32 arrivals per race take the cluster kernel of their own)
        ersd.ersd_race_sample(ok, seeds, 1.0, tok, ersd.make_opts(kernel_path=CLUSTER, top_c=33))
    assert e.value.status == -3
    with pytest.raises(ersd.ErsdError) as e:
        ersd.ersd_race_sample(ok, seeds, 1.0, tok, ersd.make_opts(kernel_path=3))
    assert e.value.status == -1
    # left to the library, such calls take the streaming kernel
    ersd.ersd_race_sample(logits, seeds, 1.0, tok, ersd.make_opts(top_c=4))
    ersd.ersd_race_sample(logits, seeds, 1.0, tok, None)
    torch.cuda.synchronize()


def test_default_choice_gives_the_same_tokens_as_either_kernel(ersd):
    V = 32000
    for B in (1, 8, 200):                       # few rows: cluster kernel; many: streaming kernel
        g = torch.Generator().manual_seed(B)
        logits = wl.zipf_rows(B, V, g, "cpu").view(B, 1, V).to(torch.bfloat16)
        seeds = wl.make_seeds(8, B, B)
        tok = torch.empty(B, 1, 1, dtype=torch.int32, device="cuda")
        ersd.ersd_race_sample(logits.cuda(), seeds.cuda(), 1.0, tok, None)
        torch.cuda.synchronize()
        tok_c, _ = sample(ersd, logits, seeds, 1.0, CLUSTER)
        tok_s, _ = sample(ersd, logits, seeds, 1.0, STREAMING)
        assert (tok == tok_c).all() and (tok == tok_s).all()


def test_drafting_loop_one_position_at_a_time(ersd):
    """Algorithm 2's drafting line run position by position (R = 1, pos_offsets advancing) equals
    the oracle's race of all positions at once."""
    B, k, V = 3, 5, 50000
    g = torch.Generator().manual_seed(12)
    logits = wl.zipf_rows(B * k, V, g, "cpu").view(B, k, V).to(torch.bfloat16)
    seeds = wl.make_seeds(9, 0, B)
    dev = logits.cuda()
    got = torch.empty(B, k, 1, dtype=torch.int32, device="cuda")
    for j in range(k):
        off = torch.full((B,), j, dtype=torch.int32, device="cuda")
        row = dev[:, j:j + 1, :].contiguous()
        tok = torch.empty(B, 1, 1, dtype=torch.int32, device="cuda")
        ersd.ersd_race_sample(row, seeds.cuda(), 0.7, tok, ersd.make_opts(kernel_path=CLUSTER, pos_offsets=off))
        got[:, j] = tok[:, 0]
    torch.cuda.synchronize()
    assert check_sample(logits, seeds, 0.7, got, None) == 0


def test_repeated_calls_agree_bit_for_bit(ersd):
    B, V = 4, 128256
    g = torch.Generator().manual_seed(3)
    logits = wl.zipf_rows(B, V, g, "cpu").view(B, 1, V).to(torch.bfloat16).cuda()
    seeds = wl.make_seeds(10, 0, B).cuda()
    first = None
    for _ in range(50):
        tok = torch.empty(B, 1, 1, dtype=torch.int32, device="cuda")
        key = torch.empty(B, 1, 1, dtype=torch.float32, device="cuda")
        ersd.ersd_race_sample(logits, seeds, 1.0, tok, ersd.make_opts(kernel_path=CLUSTER, out_key=key))
        if first is None:
            first = (tok, key)
        else:
            assert (tok == first[0]).all() and (key == first[1]).all()
    torch.cuda.synchronize()


@pytest.mark.parametrize("gap", [1e-4, -1e-4, 3e-3, -3e-3])
def test_screening_keys_too_close_to_call_are_decided_exactly(ersd, gap):
    """Two tokens whose keys differ by less than the screening precision (about 1.4e-3) but by
    far more than the near-tie window: the exact key must decide, whichever of the two leads."""
    import oracle
    B, V, T = 6, 128256, 1.0
    seeds = wl.make_seeds(31, 0, B)
    flat = np.zeros((B, 1, V), dtype=np.float32)
    tok2, key2 = oracle.race_sample(flat, wl.seeds_as_u64(seeds), T=T, c=2)
    logits = torch.zeros(B, 1, V, dtype=torch.float32)
    want = []
    for b in range(B):
        first, second = int(tok2[b, 0, 0]), int(tok2[b, 0, 1])
        # raise the runner-up's logit until its key sits `gap` above (or below) the leader's
        logits[b, 0, second] = float((key2[b, 0, 1] - key2[b, 0, 0] - gap) * T)
        want.append(first if gap > 0 else second)
    tok, key = sample(ersd, logits, seeds, T, CLUSTER)
    assert check_sample(logits, seeds, T, tok, key) == 0
    assert tok[:, 0, 0].cpu().tolist() == want
    tok_s, key_s = sample(ersd, logits, seeds, T, STREAMING)
    assert (tok == tok_s).all() and (key == key_s).all()


def test_every_cluster_size_gives_the_same_result(ersd):
    B, V = 5, 40000                                   # 20 tiles: clusters of 1 to 16 blocks stage 20 to 2 tiles each
    g = torch.Generator().manual_seed(77)
    logits = wl.zipf_rows(B, V, g, "cpu").view(B, 1, V).to(torch.bfloat16)
    seeds = wl.make_seeds(12, 0, B)
    ref_tok, ref_key = sample(ersd, logits, seeds, 1.0, STREAMING)
    assert check_sample(logits, seeds, 1.0, ref_tok, ref_key) == 0
    for blocks in (1, 2, 4, 8, 16):
        tok, key = sample(ersd, logits, seeds, 1.0, CLUSTER, split_v=blocks)
        assert (tok == ref_tok).all() and (key == ref_key).all()
    tok = torch.empty(B, 1, 1, dtype=torch.int32, device="cuda")
    for bad in (3, 32):                               # not a power of two; more than a cluster holds
        with pytest.raises(ersd.ErsdError) as e:
            ersd.ersd_race_sample(logits.cuda(), seeds.cuda(), 1.0, tok, ersd.make_opts(kernel_path=CLUSTER, split_v=bad))
        assert e.value.status == -3
    big = torch.zeros(1, 1, 300000, dtype=torch.float32).cuda()   # 147 tiles of fp32: too many for one block
    with pytest.raises(ersd.ErsdError) as e:
        ersd.ersd_race_sample(big, seeds[:1].cuda(), 1.0, tok[:1], ersd.make_opts(kernel_path=CLUSTER, split_v=1))
    assert e.value.status == -3
