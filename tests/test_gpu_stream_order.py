"""Launch overlap between the kernels of a step (programmatic stream serialisation) must never let a kernel
read what the kernel in front is still writing, nor lose a status bit.

  - kv_commit directly followed by tree_verify_attn (no mask launch in between): the attention reads
    prefix_len before its own wait, so it must only start when the commit is complete;
  - tree_build_mask directly followed by a one-layer attention that raises a status bit itself (a tree
    that does not fit the cache in the in-cache layout; a page id outside the pool): the mask kernel stores
    status last, and the attention's bit must survive it.
All calls of a test go to one stream with no synchronisation in between, many times over."""
import numpy as np
import pytest
import torch

import paper_2603_08088_b200 as tv
from oracle import tree_verify_oracle as orc
from workloads import CONFIGS, make_case, case_to_numpy, bf16_bits
from gpu_util import to_device, f32, i32, assert_attention_close, oracle_visibility

pytestmark = pytest.mark.gpu


def test_attention_directly_behind_commit_sees_the_new_prefix():
    """A step, then at once another attention over the same tree with the mask of the step: its keys are the
    prefix as the commit left it.  The prefix lengths are chosen so that the committed rows open a new key
    tile (126 -> 134 rows) or fill the last one, and the values are N(0,1), so stale lengths or rows move
    the output by far more than the tolerance."""
    cfg = CONFIGS[2].scaled(B=6, Hq=8, Hkv=2, S_lo=126, S_hi=126, Scap=256, N=64, V=2048, std=1.0)
    for rep in range(6):
        case = make_case(cfg, seed=7700 + rep)
        case["prefix_len"][:] = torch.tensor([126, 127, 120, 1, 250 - 8, 128], dtype=torch.int32)
        d = to_device(case)
        P, Dp1 = case["retrieve"].shape[1], cfg.D + 1
        buf = tv.StepBuffers(cfg.L, cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.d, cfg.Scap, cfg.V, P, Dp1)
        out2 = torch.full((cfg.B, cfg.N, cfg.Hq, cfg.d), 3.0, dtype=torch.bfloat16, device="cuda")
        lse2 = torch.full((cfg.B, cfg.Hq, cfg.N), 3.0, dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        tv.verify_step(d, buf, cfg.d ** -0.5)            # mask, attention, accept, commit
        tv.tree_verify_attn(d["q"][0], d["k_cache"][0], d["v_cache"][0], d["k_tree"][0], d["v_tree"][0],
                            d["prefix_len"], d["n_nodes"], buf.anc_bits, cfg.d ** -0.5, out2, buf.attn_ws, buf.status,
                            lse=lse2)
        torch.cuda.synchronize()
        ref = orc.verify_step(case_to_numpy(case), cfg.d ** -0.5, use_given_retrieve=False)
        assert (ref["accept"]["accept_len"] == cfg.D).all()            # planted: every prefix grows by D + 1 rows
        assert np.array_equal(i32(d["prefix_len"]), ref["prefix_len"])
        assert (i32(buf.status) == 0).all()
        c = case_to_numpy(case)
        vis = oracle_visibility(case["parent"], case["n_nodes"])
        want, want_lse = orc.tree_attention(c["q"][0], ref["k_cache"][0], ref["v_cache"][0], c["k_tree"][0], c["v_tree"][0],
                                            ref["prefix_len"], c["n_nodes"], vis[:, 0], cfg.d ** -0.5)
        assert_attention_close(out2, lse2, want, want_lse, f"attention behind the commit, repetition {rep}")
        # the same rows over the old prefix are far away: the check above can tell the two apart
        old, _ = orc.tree_attention(c["q"][0], c["k_cache"][0], c["v_cache"][0], c["k_tree"][0], c["v_tree"][0],
                                    c["prefix_len"], c["n_nodes"], vis[:, 0], cfg.d ** -0.5)
        assert np.abs(old - want).max() > 0.2


def test_status_bits_raised_by_a_one_layer_attention_survive_the_mask_kernel():
    cfg = CONFIGS[0].scaled(B=2, S_lo=100, S_hi=100, Scap=128, N=15)
    case = make_case(cfg, seed=12, with_logits=False)
    g = to_device(case)
    B, N, Hq, Hkv, d = cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.d
    bits = torch.zeros(B, N, 1, dtype=torch.int32, device="cuda")
    ws = torch.zeros(max(256, tv.tv_attn_workspace_bytes(B, N, Hq, Hkv, d, cfg.Scap)), dtype=torch.uint8, device="cuda")
    out = torch.zeros(B, N, Hq, d, dtype=torch.bfloat16, device="cuda")
    # in-cache layout: 120 + 15 rows do not fit 128; 100 + 15 do
    S = torch.tensor([120, 100], dtype=torch.int32, device="cuda")
    # paged layout: one page per sequence, the second sequence names a page outside the pool of 3
    kp = torch.zeros(3, Hkv, 128, d, dtype=torch.bfloat16, device="cuda")
    bt = torch.tensor([[1], [3]], dtype=torch.int32, device="cuda")
    statuses = []
    for rep in range(40):
        st1 = torch.full((B,), 64, dtype=torch.int32, device="cuda")       # the mask call overwrites it
        tv.tree_build_mask(g["parent"], g["n_nodes"], N - 1, 1, bits, st1)
        tv.tree_verify_attn(g["q"][0], g["k_cache"][0], g["v_cache"][0], None, None, S, g["n_nodes"], bits, d ** -0.5,
                            out, ws, st1)
        st2 = torch.full((B,), 64, dtype=torch.int32, device="cuda")
        tv.tree_build_mask(g["parent"], g["n_nodes"], N - 1, 1, bits, st2)
        tv.tree_verify_attn_paged(g["q"][0], kp, kp, bt, g["k_tree"][0], g["v_tree"][0], g["prefix_len"], g["n_nodes"],
                                  bits, d ** -0.5, out, ws, st2)
        statuses.append((st1, st2))
    torch.cuda.synchronize()
    for rep, (st1, st2) in enumerate(statuses):
        assert i32(st1).tolist() == [tv.TV_ST_CAPACITY, 0], f"repetition {rep}: {i32(st1).tolist()}"
        assert i32(st2).tolist() == [0, tv.TV_ST_BAD_INDEX], f"repetition {rep}: {i32(st2).tolist()}"
