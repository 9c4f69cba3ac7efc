"""Seeded random shapes through tree_verify_attn in its three cache layouts (contiguous with separate tree
buffers, tree inside the cache, paged).  Each case is checked against the fp64 oracle (max-abs 2e-2) and the
three layouts against each other bit for bit: they run the same tiles with the same arithmetic."""
import numpy as np
import pytest
import torch

import paper_2603_08088_b200 as tv
from oracle import tree_verify_oracle as orc
from workloads import CONFIGS, make_case, case_to_numpy
from gpu_util import to_device, i32, assert_attention_close, oracle_visibility

pytestmark = pytest.mark.gpu


def random_cfg(rng):
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 3]))
    G = int(rng.choice([1, 2, 4, 8]))
    N = int(rng.choice([1, 2, 7, 15, 33, 60, 64, 65, 100, 129, 150]))
    B = int(rng.integers(1, 5))
    S_hi = int(rng.choice([0, 5, 130, 400, 900]))
    S_lo = int(rng.integers(0, S_hi + 1))
    Scap = ((S_hi + N + 127) // 128) * 128 + int(rng.choice([0, 128]))
    D = int(min(N - 1, rng.integers(1, 9))) if N > 1 else 0
    return CONFIGS[0].scaled(B=B, Hq=Hkv * G, Hkv=Hkv, d=d, L=1, S_lo=S_lo, S_hi=S_hi, Scap=Scap, N=N, D=max(D, 0), V=0,
                             tree="uniform", std=float(rng.choice([1.0, 0.3])))


@pytest.mark.parametrize("seed", list(range(14)))
def test_random_shape_three_layouts(seed):
    rng = np.random.default_rng(1000 + seed)
    cfg = random_cfg(rng)
    if cfg.N == 1:
        cfg = cfg.scaled(D=0)
    case = make_case(cfg, seed=500 + seed, ragged_nodes=(cfg.B > 1), with_logits=False)
    dev = "cuda"
    g = to_device(case)
    B, N, Hq, Hkv, d, Scap = cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.d, cfg.Scap
    W = (N + 31) // 32
    bits = torch.zeros(B, N, W, dtype=torch.int32, device=dev)
    dense = torch.zeros(B, 1, N, N, dtype=torch.uint8, device=dev)
    status = torch.zeros(B, dtype=torch.int32, device=dev)
    tv.tree_build_mask(g["parent"], g["n_nodes"], max(N - 1, 0), 1, bits, status, dense_mask=dense)
    ws = torch.zeros(max(256, tv.tv_attn_workspace_bytes(B, N, Hq, Hkv, d, Scap)), dtype=torch.uint8, device=dev)
    scale = d ** -0.5
    outs = []
    # contiguous cache, separate tree buffers
    out, lse = torch.full((B, N, Hq, d), 3.0, dtype=torch.bfloat16, device=dev), torch.zeros(B, Hq, N, device=dev)
    tv.tree_verify_attn(g["q"][0], g["k_cache"][0], g["v_cache"][0], g["k_tree"][0], g["v_tree"][0], g["prefix_len"],
                        g["n_nodes"], bits, scale, out, ws, status, lse=lse)
    outs.append((out, lse))
    # tree rows inside the cache
    kc, vc = case["k_cache"][0].clone(), case["v_cache"][0].clone()
    for b, S in enumerate(case["prefix_len"].tolist()):
        kc[b, :, S:S + N] = case["k_tree"][0, b].permute(1, 0, 2)
        vc[b, :, S:S + N] = case["v_tree"][0, b].permute(1, 0, 2)
    out, lse = torch.full((B, N, Hq, d), 3.0, dtype=torch.bfloat16, device=dev), torch.zeros(B, Hq, N, device=dev)
    tv.tree_verify_attn(g["q"][0], kc.to(dev), vc.to(dev), None, None, g["prefix_len"], g["n_nodes"], bits, scale, out, ws,
                        status, lse=lse)
    outs.append((out, lse))
    # pages scattered over a pool
    nb = Scap // 128
    order = rng.permutation(B * nb + 2)
    bt = torch.from_numpy(order[:B * nb].reshape(B, nb).astype(np.int32))
    def paginate(c):
        pool = torch.zeros(B * nb + 2, Hkv, 128, d, dtype=c.dtype)
        for b in range(B):
            pool[bt[b].long()] = c[b].reshape(Hkv, nb, 128, d).permute(1, 0, 2, 3)
        return pool
    out, lse = torch.full((B, N, Hq, d), 3.0, dtype=torch.bfloat16, device=dev), torch.zeros(B, Hq, N, device=dev)
    tv.tree_verify_attn_paged(g["q"][0], paginate(case["k_cache"][0]).to(dev), paginate(case["v_cache"][0]).to(dev),
                              bt.to(dev), g["k_tree"][0], g["v_tree"][0], g["prefix_len"], g["n_nodes"], bits, scale, out,
                              ws, status, lse=lse)
    outs.append((out, lse))
    torch.cuda.synchronize()
    assert (i32(status) == 0).all(), f"{cfg}: status {i32(status)}"
    case_np = case_to_numpy(case)
    vis = oracle_visibility(case["parent"], case["n_nodes"], dense_gpu=dense, bits_gpu=bits)   # the oracle's own mask
    ref_out, ref_lse = orc.tree_attention(case_np["q"][0], case_np["k_cache"][0], case_np["v_cache"][0],
                                          case_np["k_tree"][0], case_np["v_tree"][0], case_np["prefix_len"],
                                          case_np["n_nodes"], vis[:, 0], scale)
    assert_attention_close(outs[0][0], outs[0][1], ref_out, ref_lse, str(cfg))
    for o, l in outs[1:]:
        assert torch.equal(o.view(torch.int16), outs[0][0].view(torch.int16)) and torch.equal(l, outs[0][1]), str(cfg)
