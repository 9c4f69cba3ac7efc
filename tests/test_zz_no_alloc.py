"""tree_accept_noalloc: the accept step for callers that are not allowed to
allocate device memory (its argmax scratch is a fixed array inside the
library).  Checked through the C ABI against tree_accept with a caller
workspace and against the oracle, bit for bit, on two calls in a row with different inputs, so that
whatever the first call left in the shared scratch cannot leak into the second.
Collected last on purpose: a run that stops at the first failure has already
run every other test."""
import numpy as np
import pytest
import torch

import paper_2603_08088_b200 as tv
from oracle import tree_verify_oracle as orc
from workloads import CONFIGS, make_case, bf16_bits

pytestmark = pytest.mark.gpu

OUTS = ("argmax_tok", "accept_len", "best_path", "accepted_nodes", "next_token", "safe_idx", "candidates")


def _outputs(B, N, P, Dp1, dev):
    z = lambda *s: torch.full(s, -3, dtype=torch.int32, device=dev)
    return dict(argmax_tok=z(B, N), accept_len=z(B), best_path=z(B), accepted_nodes=z(B, Dp1), next_token=z(B),
                safe_idx=z(B, P, Dp1), candidates=z(B, P, Dp1))


def _run_both(cfg, seed):
    dev = "cuda"
    case = make_case(cfg, seed=seed, device=dev, with_cache=False, ragged_nodes=True)
    B, N, V = case["logits"].shape
    P, Dp1 = case["retrieve"].shape[1], case["retrieve"].shape[2]
    a, b = _outputs(B, N, P, Dp1, dev), _outputs(B, N, P, Dp1, dev)
    st_a = torch.zeros(B, dtype=torch.int32, device=dev)
    st_b = torch.zeros(B, dtype=torch.int32, device=dev)
    ws = torch.zeros(tv.tv_accept_workspace_bytes(B, N, V), dtype=torch.uint8, device=dev)
    tv.tree_accept(case["logits"], case["tokens"], case["retrieve"], case["n_nodes"], a["argmax_tok"],
                   a["accept_len"], a["best_path"], a["accepted_nodes"], a["next_token"], ws, st_a,
                   safe_idx=a["safe_idx"], candidates=a["candidates"])
    tv.tree_accept_noalloc(case["logits"], case["tokens"], case["retrieve"], case["n_nodes"], b["argmax_tok"],
                           b["accept_len"], b["best_path"], b["accepted_nodes"], b["next_token"], st_b,
                           safe_idx=b["safe_idx"], candidates=b["candidates"])
    torch.cuda.synchronize()
    for k in OUTS:
        assert torch.equal(a[k], b[k]), f"{k} differs between tree_accept and tree_accept_noalloc"
    assert torch.equal(st_a, st_b)
    # and directly against the oracle, not only through the other entry point
    n_nodes = case["n_nodes"].cpu().numpy()
    am = orc.argmax_rows(bf16_bits(case["logits"]), n_nodes)
    ref = orc.greedy_accept(case["retrieve"].cpu().numpy(), case["tokens"].cpu().numpy(), n_nodes, am)
    assert np.array_equal(b["argmax_tok"].cpu().numpy(), am)
    for k in ("accept_len", "best_path", "accepted_nodes", "next_token", "safe_idx", "candidates"):
        assert np.array_equal(b[k].cpu().numpy(), ref[k]), f"{k} differs from the oracle"
    assert np.array_equal(st_b.cpu().numpy(), ref["status"])
    return a


def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    big = CONFIGS[4].scaled(L=1, B=6, S_lo=1, S_hi=4, Scap=16, V=153600)       # 6*60*19 scratch entries
    small = CONFIGS[2].scaled(L=1, B=3, S_lo=1, S_hi=4, Scap=16, V=9000, Hq=8, Hkv=2)
    first = _run_both(big, seed=11)
    second = _run_both(small, seed=12)      # smaller problem: most of the scratch still holds call one's pairs
    third = _run_both(big, seed=13)
    assert not torch.equal(first["argmax_tok"], third["argmax_tok"])
    assert int(second["accept_len"].max()) >= 1


def test_noalloc_rejects_problems_beyond_its_scratch():
    assert tv.tv_accept_noalloc_max_bytes() == 32768 * 8
    cfg = CONFIGS[4].scaled(L=1, S_lo=1, S_hi=4, Scap=16, B=16, V=16384 * 36)   # 16*60*36 > 32768 entries
    dev = "cuda"
    B, N, V, P, Dp1 = cfg.B, cfg.N, cfg.V, 10, cfg.D + 1
    logits = torch.zeros(1, dtype=torch.bfloat16, device=dev)     # never read: the call is rejected first
    o = _outputs(B, N, P, Dp1, dev)
    i32 = lambda *s: torch.zeros(s, dtype=torch.int32, device=dev)
    lib = tv.load()
    rc = lib.tree_accept_noalloc(logits.data_ptr(), i32(B, N).data_ptr(), i32(B, P, Dp1).data_ptr(), i32(B).data_ptr(),
                                 B, N, V, P, Dp1, o["argmax_tok"].data_ptr(), None, None, o["accept_len"].data_ptr(),
                                 o["best_path"].data_ptr(), o["accepted_nodes"].data_ptr(), o["next_token"].data_ptr(),
                                 i32(B).data_ptr(), None)
    assert rc == 3 and b"built-in scratch" in lib.tv_last_error()
