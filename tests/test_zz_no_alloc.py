"""ersd_verify_noalloc: the verify entry point for callers that cannot allocate device memory
(pre-planned memory pools, latency-critical sections, fully committed devices).  Its scratch is a
fixed array inside the library that every call on a device shares, so the checks here are: same
results as ersd_verify on two calls in a row (the second call finds the first one's leftovers in
the scratch), and a clear refusal beyond the built-in capacity.  Collected last on purpose."""
import pytest
import torch

from paper_2504_15475_b200 import workloads as wl
from parity_util import check_verify

pytestmark = pytest.mark.gpu


def test_noalloc_matches_verify_on_two_calls_in_a_row():
    from paper_2504_15475_b200 import binding as ersd
    ersd.lib()
    configs = [wl.scaled(wl.CONFIGS["c2"], B=8), wl.scaled(wl.CONFIGS["c5"], B=5, V=40000),
               wl.scaled(wl.CONFIGS["c2"], B=8)]
    for call, w in enumerate(configs):
        inp = wl.make_inputs(w, call=200 + call)
        tgt, drf, seeds = inp["target"].cuda(), inp["draft"].cuda(), inp["seeds"].cuda()
        kw = {}
        if inp["temps"] is not None:
            t = inp["temps"].cuda()
            kw = dict(temps=t, temp_strides=(t.stride(0), t.stride(1)))
        for split in (0, 3):
            ref_tok = torch.full((w.B, w.k + 1), -9, dtype=torch.int32, device="cuda")
            ref_acc = torch.full((w.B,), -9, dtype=torch.int32, device="cuda")
            ersd.ersd_verify(tgt, drf, seeds, inp["T"], ref_tok, ref_acc, ersd.make_opts(split_v=split, **kw))
            for rep in range(2):                      # two calls in a row through the new entry point
                tok = torch.full((w.B, w.k + 1), -9, dtype=torch.int32, device="cuda")
                acc = torch.full((w.B,), -9, dtype=torch.int32, device="cuda")
                dkey = torch.empty(w.B, w.k, dtype=torch.float32, device="cuda")
                ref_dkey = torch.empty(w.B, w.k, dtype=torch.float32, device="cuda")
                rows = dict(draft_tok=torch.empty(w.B, w.k, dtype=torch.int32, device="cuda"),
                            target_tok=torch.empty(w.B, w.k + 1, dtype=torch.int32, device="cuda"),
                            target_key=torch.empty(w.B, w.k + 1, dtype=torch.float32, device="cuda"))
                ersd.ersd_verify_noalloc(tgt, drf, seeds, inp["T"], tok, acc,
                                         ersd.make_opts(split_v=split, out_draft_key=dkey,
                                                        out_draft_tok=rows["draft_tok"],
                                                        out_target_tok=rows["target_tok"],
                                                        out_target_key=rows["target_key"], **kw))
                ersd.ersd_verify(tgt, drf, seeds, inp["T"], ref_tok, ref_acc,
                                 ersd.make_opts(split_v=split, out_draft_key=ref_dkey, **kw))
                torch.cuda.synchronize()
                assert (tok == ref_tok).all(), (call, split, rep)
                assert (acc == ref_acc).all(), (call, split, rep)
                assert (dkey - ref_dkey).abs().max().item() <= 2e-5   # the key tolerance of the parity tests
                if split == 0:
                    # and against the oracle itself: every row's winners and keys, the accepted prefix
                    # (a near-tie row may take either winner; check_verify counts those)
                    check_verify(inp, dict(tokens=tok, accept_len=acc, draft_key=dkey, **rows))


def test_noalloc_refuses_sizes_beyond_its_scratch():
    from paper_2504_15475_b200 import binding as ersd
    B, k, V = 205, 4, 64                               # 205 * 5 = 1025 rows > 1024
    assert B * (k + 1) > ersd.ERSD_NOALLOC_MAX_ROWS
    tgt = torch.zeros(B, k + 1, V, dtype=torch.bfloat16, device="cuda")
    drf = torch.zeros(B, k, V, dtype=torch.bfloat16, device="cuda")
    seeds = torch.zeros(B, dtype=torch.int64, device="cuda")
    tok = torch.full((B, k + 1), -9, dtype=torch.int32, device="cuda")
    acc = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    with pytest.raises(ersd.ErsdError) as e:
        ersd.ersd_verify_noalloc(tgt, drf, seeds, 1.0, tok, acc)
    assert e.value.status == ersd.ERSD_ENOALLOC_LIMIT and "ERSD_NOALLOC_MAX_ROWS" in str(e.value)
    torch.cuda.synchronize()
    assert (tok == -9).all() and (acc == -9).all()     # nothing was launched
    # the largest size that fits is accepted
    B = 1024 // (k + 1)
    ersd.ersd_verify_noalloc(tgt[:B], drf[:B], seeds[:B], 1.0, tok[:B], acc[:B])
    ref_tok = torch.empty_like(tok[:B])
    ref_acc = torch.empty_like(acc[:B])
    ersd.ersd_verify(tgt[:B], drf[:B], seeds[:B], 1.0, ref_tok, ref_acc)
    torch.cuda.synchronize()
    assert (tok[:B] == ref_tok).all() and (acc[:B] == ref_acc).all()
    # a caller-supplied workspace contradicts the point of this entry and is refused
    ws = torch.zeros(ersd.ersd_workspace_bytes(B, k + 1), dtype=torch.uint8, device="cuda")
    with pytest.raises(ersd.ErsdError) as e:
        ersd.ersd_verify_noalloc(tgt[:B], drf[:B], seeds[:B], 1.0, tok[:B], acc[:B], ersd.make_opts(workspace=ws))
    assert e.value.status == -1


def test_noalloc_refused_call_puts_nothing_on_the_stream():
    """Argument errors are found before anything is enqueued: a refused call leaves the outputs as
    they were, and the next valid call still agrees with ersd_verify."""
    from paper_2504_15475_b200 import binding as ersd
    w = wl.scaled(wl.CONFIGS["c2"], B=3, V=4096)
    inp = wl.make_inputs(w, call=300)
    tgt, drf, seeds = inp["target"].cuda(), inp["draft"].cuda(), inp["seeds"].cuda()
    tok = torch.full((w.B, w.k + 1), -9, dtype=torch.int32, device="cuda")
    acc = torch.full((w.B,), -9, dtype=torch.int32, device="cuda")
    for bad in (dict(T=-1.0), dict(T=float("nan")), dict(draft=None), dict(opts=ersd.make_opts(kernel_path=3)),
                dict(opts=ersd.make_opts(block_threads=96))):
        with pytest.raises(ersd.ErsdError) as e:
            ersd.ersd_verify_noalloc(tgt, bad.get("draft", drf) if "draft" in bad else drf, seeds,
                                     bad.get("T", inp["T"]), tok, acc, bad.get("opts"))
        assert e.value.status == -1, bad                  # ERSD_EINVAL
        torch.cuda.synchronize()
        assert (tok == -9).all() and (acc == -9).all()
    ersd.ersd_verify_noalloc(tgt, drf, seeds, inp["T"], tok, acc)
    ref_tok, ref_acc = torch.empty_like(tok), torch.empty_like(acc)
    ersd.ersd_verify(tgt, drf, seeds, inp["T"], ref_tok, ref_acc)
    torch.cuda.synchronize()
    assert (tok == ref_tok).all() and (acc == ref_acc).all()
