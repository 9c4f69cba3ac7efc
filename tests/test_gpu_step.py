"""A whole verification step on the GPU against the oracle: the five configs
(reduced where the fp64 oracle would take minutes; the attention of the
full-size configs is covered head-by-head in test_gpu_attn.py), the
commit-equivalence property, and the host-buffer entry point."""
import numpy as np
import pytest
import torch

import paper_2603_08088_b200 as tv
from oracle import tree_verify_oracle as orc
from workloads import CONFIGS, make_case, case_to_numpy, bf16_bits
from gpu_util import to_device, f32, i32, ATTN_ATOL

pytestmark = pytest.mark.gpu

STEP_CASES = [
    ("tiny", 0, {}),
    ("llama7b_layer", 1, dict(Hq=8, Hkv=8, S_lo=300, S_hi=300, Scap=384)),
    ("gqa8b_ragged", 2, dict(B=4, Hq=16, Hkv=4, S_lo=60, S_hi=500, Scap=640, V=128256)),
    ("full_step", 4, dict(B=5, L=3, Hq=16, Hkv=4, S_lo=30, S_hi=260, Scap=320, V=153600)),
    # the variant whose ten candidate rows name all 60 nodes (ten chains from the root)
    ("full_step_covering_rows", 4, dict(B=4, L=2, Hq=16, Hkv=4, S_lo=30, S_hi=260, Scap=320, V=20000, tree="chains")),
]


def run_step(cfg, case, given_rows):
    d = to_device(case)
    P = case["retrieve"].shape[1]
    buf = tv.StepBuffers(cfg.L, cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.d, cfg.Scap, cfg.V, P, cfg.D + 1,
                         want_dense=True, want_lse=True, want_gather=True)
    tv.verify_step(d, buf, cfg.d ** -0.5, retrieve=d["retrieve"] if given_rows else None)
    torch.cuda.synchronize()
    return d, buf


@pytest.mark.parametrize("name,ci,over", STEP_CASES, ids=[s[0] for s in STEP_CASES])
def test_whole_step_matches_oracle(name, ci, over):
    cfg = CONFIGS[ci].scaled(**over)
    case = make_case(cfg, seed=1000 * ci + 7, ragged_nodes=(cfg.B > 2 and cfg.tree != "chains"))
    given_rows = cfg.P > 0
    ref = orc.verify_step(case_to_numpy(case), cfg.d ** -0.5, use_given_retrieve=given_rows)
    d, buf = run_step(cfg, case, given_rows)
    mk = ref["mask"]
    assert np.array_equal(i32(buf.anc_bits).view(np.uint32), mk["anc_bits"])
    assert np.array_equal(i32(buf.dense), mk["dense"])
    assert np.array_equal(i32(buf.depth), mk["depth"])
    assert np.array_equal(i32(buf.anc_table), mk["anc_table"])
    if not given_rows:
        assert np.array_equal(i32(buf.retrieve), mk["retrieve"]) and np.array_equal(i32(buf.n_paths), mk["n_paths"])
    err = np.abs(f32(buf.out).astype(np.float64) - ref["out"]).max()
    assert err <= ATTN_ATOL, f"attention max-abs error {err}"
    lg, lr = f32(buf.lse).astype(np.float64), ref["lse"]
    assert (np.isneginf(lg) == np.isneginf(lr)).all()
    assert np.abs(np.where(np.isneginf(lr), 0, lg) - np.where(np.isneginf(lr), 0, lr)).max() <= 2e-3
    acc = ref["accept"]
    assert np.array_equal(i32(buf.argmax_tok), ref["argmax"])
    for k in ("accept_len", "best_path", "accepted_nodes", "next_token"):
        assert np.array_equal(i32(getattr(buf, k)), acc[k]), k
    assert np.array_equal(i32(buf.safe_idx), acc["safe_idx"]) and np.array_equal(i32(buf.candidates), acc["candidates"])
    assert np.array_equal(i32(buf.status), ref["status"])
    assert np.array_equal(bf16_bits(d["k_cache"]), ref["k_cache"]), "committed K bytes differ"
    assert np.array_equal(bf16_bits(d["v_cache"]), ref["v_cache"]), "committed V bytes differ"
    assert np.array_equal(i32(d["prefix_len"]), ref["prefix_len"])
    if cfg.plant != "none":
        full = case["n_nodes"].numpy() == cfg.N
        assert (acc["accept_len"][full] >= case["plant_depth"][full]).all()


def test_commit_equivalence_follow_up_decode():
    """After the commit a 1-node verify equals causal decode over prefix (+)
    accepted path (commit equivalence, Section 3.1)."""
    cfg = CONFIGS[2].scaled(B=3, Hq=8, Hkv=2, S_lo=100, S_hi=300, Scap=384, V=4096)
    case = make_case(cfg, seed=99)
    d, buf = run_step(cfg, case, False)
    A = i32(buf.accept_len)
    nodes = i32(buf.accepted_nodes)
    assert (A == cfg.D).all()                       # the planted path is accepted to full depth
    S0 = case["prefix_len"].numpy()
    S1 = i32(d["prefix_len"])
    assert (S1 == S0 + A + 1).all()
    one = CONFIGS[2].scaled(B=3, Hq=8, Hkv=2, S_lo=1, S_hi=1, Scap=384, N=1, D=0, V=0, tree="uniform", plant="none")
    nxt = make_case(one, seed=100, with_cache=False, with_logits=False)
    dn = to_device(nxt)
    dn["k_cache"], dn["v_cache"], dn["prefix_len"] = d["k_cache"], d["v_cache"], d["prefix_len"]
    buf1 = tv.StepBuffers(1, 3, 1, 8, 2, 128, 384, 0, 1, 1, want_lse=True)
    tv.verify_step(dn, buf1, 128 ** -0.5)
    torch.cuda.synchronize()
    # sequential reference: prefix rows, then the accepted nodes' tree rows in path order, then the new token
    cn, nn = case_to_numpy(case), case_to_numpy(nxt)
    for b in range(3):
        kc = np.concatenate([cn["k_cache"][0, b, :, :S0[b]], cn["k_tree"][0, b, nodes[b, :A[b] + 1]].transpose(1, 0, 2)], 1)
        vc = np.concatenate([cn["v_cache"][0, b, :, :S0[b]], cn["v_tree"][0, b, nodes[b, :A[b] + 1]].transpose(1, 0, 2)], 1)
        pad = np.zeros((2, 4, 128), dtype=np.uint16)
        out, lse = orc.tree_attention(nn["q"][0][b:b + 1], np.concatenate([kc, pad], 1)[None], np.concatenate([vc, pad], 1)[None],
                                      nn["k_tree"][0][b:b + 1], nn["v_tree"][0][b:b + 1], S1[b:b + 1], np.array([1]),
                                      np.ones((1, 1, 1), dtype=np.uint8), 128 ** -0.5)
        assert np.abs(f32(buf1.out)[0, b] - out[0]).max() <= ATTN_ATOL
        assert np.abs(f32(buf1.lse)[0, b] - lse[0]).max() <= 2e-3


def test_host_buffer_step_matches_device_step():
    cfg = CONFIGS[4].scaled(B=3, L=2, Hq=8, Hkv=2, S_lo=50, S_hi=200, Scap=256, V=20000)
    case = make_case(cfg, seed=4242)
    ref = orc.verify_step(case_to_numpy(case), cfg.d ** -0.5)
    P, Dp1 = case["retrieve"].shape[1], cfg.D + 1
    pin = lambda t: t.contiguous().pin_memory()
    host = {k: pin(case[k]) for k in ("parent", "n_nodes", "tokens", "q", "k_tree", "v_tree", "logits")}
    host["retrieve_indices"] = pin(case["retrieve"])
    host["out"] = torch.zeros(cfg.L, cfg.B, cfg.N, cfg.Hq, cfg.d, dtype=torch.bfloat16).pin_memory()
    for k, shape in (("accept_len", (cfg.B,)), ("accepted_nodes", (cfg.B, Dp1)), ("next_token", (cfg.B,)), ("status", (cfg.B,))):
        host[k] = torch.full(shape, -5, dtype=torch.int32).pin_memory()
    kc, vc, S = case["k_cache"].cuda(), case["v_cache"].cuda(), case["prefix_len"].cuda()
    staging = torch.zeros(tv.tv_step_staging_bytes(cfg.L, cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.d, cfg.Scap, cfg.V, P, Dp1),
                          dtype=torch.uint8, device="cuda")
    tv.tv_verify_step_host(host, kc, vc, S, staging, cfg.d ** -0.5, cfg.V)
    assert np.abs(host["out"].float().numpy() - ref["out"]).max() <= ATTN_ATOL
    for k in ("accept_len", "accepted_nodes", "next_token"):
        assert np.array_equal(host[k].numpy(), ref["accept"][k]), k
    assert np.array_equal(host["status"].numpy(), ref["status"])
    assert np.array_equal(bf16_bits(kc), ref["k_cache"]) and np.array_equal(bf16_bits(vc), ref["v_cache"])
    assert np.array_equal(i32(S), ref["prefix_len"])
