"""tv_debug_attn_stream_only (treeverify_debug.h): the K/V stream of the attention launch with nothing computed.
It must end by itself without raising a status, leave the output alone, and leave the device in a state in which
the next real launch - on the same workspace - gives the oracle's result."""
import numpy as np
import pytest
import torch

import paper_2603_08088_b200 as tv
from workloads import CONFIGS, make_case, bf16_bits
from gpu_util import i32, f32, oracle_attention_slice, oracle_visibility, ATTN_ATOL

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("ci,over", [(4, dict(B=6, L=3, V=0)), (1, dict(L=2, V=0))], ids=["two_row_tiles", "one_row_tile"])
def test_stream_only_launch_computes_nothing_and_harms_nothing(ci, over):
    cfg = CONFIGS[ci].scaled(**over)
    d = make_case(cfg, seed=77 + ci, device="cuda", with_logits=False)
    L, B, N, Hq, Hkv, dh = cfg.L, cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.d
    bits = torch.zeros(B, N, (N + 31) // 32, dtype=torch.int32, device="cuda")
    status = torch.zeros(B, dtype=torch.int32, device="cuda")
    tv.tree_build_mask(d["parent"], d["n_nodes"], N - 1, 1, bits, status)
    dense = oracle_visibility(d["parent"], d["n_nodes"], bits_gpu=bits)[:, 0]
    ws = torch.zeros(max(256, tv.tv_attn_workspace_bytes(B, N, Hq, Hkv, dh, cfg.Scap)), dtype=torch.uint8, device="cuda")
    out = torch.full((L, B, N, Hq, dh), 3.0, dtype=torch.bfloat16, device="cuda")
    for _ in range(3):
        tv.tv_debug_attn_stream_only(d["q"], d["k_cache"], d["v_cache"], d["k_tree"], d["v_tree"], d["prefix_len"],
                                     d["n_nodes"], bits, out, ws, status)
    torch.cuda.synchronize()
    assert (i32(status) == 0).all()
    assert (out == 3.0).all()                       # nothing was written
    tv.tree_verify_attn_layers(d["q"], d["k_cache"], d["v_cache"], d["k_tree"], d["v_tree"], d["prefix_len"], d["n_nodes"],
                               bits, dh ** -0.5, out, ws, status)
    torch.cuda.synchronize()
    assert (i32(status) == 0).all()
    G = Hq // Hkv
    S0, n_nodes = i32(d["prefix_len"]), i32(d["n_nodes"])
    for (l, b, hk) in {(0, 0, 0), (L - 1, B - 1, Hkv - 1)}:
        case_np = {"q": bf16_bits(d["q"][l:l + 1]), "k_cache": bf16_bits(d["k_cache"][l:l + 1]),
                   "v_cache": bf16_bits(d["v_cache"][l:l + 1]), "k_tree": bf16_bits(d["k_tree"][l:l + 1]),
                   "v_tree": bf16_bits(d["v_tree"][l:l + 1]), "prefix_len": S0, "n_nodes": n_nodes}
        ref_out, _ = oracle_attention_slice(case_np, 0, b, hk, G, dense, dh ** -0.5)
        got = f32(out[l, b:b + 1, :, hk * G:(hk + 1) * G])
        assert np.abs(got - ref_out).max() <= ATTN_ATOL
