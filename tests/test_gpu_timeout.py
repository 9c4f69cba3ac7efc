"""The failure path of tree_verify_attn: every wait inside the kernel is bounded, and when one expires the
launch must end by itself - all roles leave their loops, the tensor memory is freed, TV_ST_TIMEOUT is raised
for every sequence - and the device must go on working.  The expiry is produced the harmless way: a test
entry point (treeverify_debug.h) launches the kernel with a limit of two milliseconds and a producer warp
that issues no copy, so the wait of the MMA-issuing warp for its first operands runs out - or with pieces of
cut units that are never announced, so the bounded poll of the merging piece runs out.  Nothing traps, faults or
waits without limit."""
import numpy as np
import pytest
import torch

import paper_2603_08088_b200 as tv
from workloads import CONFIGS, make_case
from gpu_util import i32

pytestmark = pytest.mark.gpu

SHAPES = [
    ("one_row_tile", 0, dict(B=2, S_lo=100, S_hi=300, Scap=320, N=15)),
    ("two_row_tiles_cut_units", 4, dict(B=6, L=1, V=0)),
]


@pytest.mark.parametrize("name,ci,over", SHAPES, ids=[s[0] for s in SHAPES])
def test_expired_wait_ends_the_launch_with_a_status_and_the_next_launch_is_unharmed(name, ci, over):
    cfg = CONFIGS[ci].scaled(**over)
    d = make_case(cfg, seed=31 + ci, device="cuda", with_logits=False)
    B, N, Hq, Hkv, dh = cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.d
    bits = torch.zeros(B, N, (N + 31) // 32, dtype=torch.int32, device="cuda")
    status = torch.zeros(B, dtype=torch.int32, device="cuda")
    tv.tree_build_mask(d["parent"], d["n_nodes"], N - 1, 1, bits, status)
    ws = torch.zeros(max(256, tv.tv_attn_workspace_bytes(B, N, Hq, Hkv, dh, cfg.Scap)), dtype=torch.uint8, device="cuda")
    args = (d["q"][0], d["k_cache"][0], d["v_cache"][0], d["k_tree"][0], d["v_tree"][0], d["prefix_len"], d["n_nodes"],
            bits, dh ** -0.5)

    def normal():
        out = torch.full((B, N, Hq, dh), 3.0, dtype=torch.bfloat16, device="cuda")
        lse = torch.full((B, Hq, N), 3.0, dtype=torch.float32, device="cuda")
        tv.tree_verify_attn(*args, out, ws, status, lse=lse)
        torch.cuda.synchronize()
        return out, lse

    before = normal()
    assert (i32(status) == 0).all()
    # mode 0 of the test entry point is an ordinary launch (short limit, nothing withheld): same bits, no flag
    out0 = torch.zeros_like(before[0])
    tv.tv_debug_attn_expire(*args, out0, ws, status, 500_000_000, 0)
    torch.cuda.synchronize()
    assert (i32(status) == 0).all() and torch.equal(out0, before[0])

    modes = [1, 1, 1] + ([2, 2] if ci == 4 else [])       # 2: the merger's poll (only the second shape has cut units)
    for rep, mode in enumerate(modes):
        junk = torch.zeros_like(before[0])
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        tv.tv_debug_attn_expire(*args, junk, ws, status, 2_000_000, mode)    # 2 ms; 1: producer issues nothing
        t1.record()
        torch.cuda.synchronize()                                             # the launch returned by itself
        assert (i32(status) & tv.TV_ST_TIMEOUT != 0).all(), f"status {i32(status).tolist()}"
        assert (i32(status) & ~tv.TV_ST_TIMEOUT == 0).all()
        ms = t0.elapsed_time(t1)
        assert 1.5 <= ms <= 200.0, f"the expiring launch took {ms} ms"
        status.zero_()
        after = normal()                                                     # tensor memory was freed, barriers are fresh
        assert (i32(status) == 0).all()
        assert torch.equal(after[0], before[0]) and torch.equal(after[1], before[1])
