"""Context split on one GPU: the members of an R-way split are run one after the other (each on its own
slice of the prefix cache), their (out, lse) are stacked as an all-gather would leave them, and
tree_merge_partials must reproduce the attention over the whole prefix (oracle, max-abs 2e-2) and the
oracle's merge of the very same partials (one bf16 rounding apart)."""
import numpy as np
import pytest
import torch

import paper_2603_08088_b200 as tv
from paper_2603_08088_b200 import dist as tvd
from oracle import tree_verify_oracle as orc
from workloads import CONFIGS, make_case, case_to_numpy, bf16_bits
from gpu_util import f32, ATTN_ATOL, oracle_visibility

pytestmark = pytest.mark.gpu


def run_split(case, R):
    """Returns o_parts[R,B,N,Hq,d] bf16, lse_parts[R,B,Hq,N] fp32 (device) and the oracle's dense mask of the same trees (numpy; the CUDA mask
    is checked equal to it)."""
    L, B, N, Hq, d = case["q"].shape
    Hkv, Scap = case["k_cache"].shape[2], case["k_cache"].shape[3]
    dev = case["q"].device
    bits = torch.zeros(B, N, (N + 31) // 32, dtype=torch.int32, device=dev)
    dense = torch.zeros(B, 1, N, N, dtype=torch.uint8, device=dev)
    status = torch.zeros(B, dtype=torch.int32, device=dev)
    tv.tree_build_mask(case["parent"], case["n_nodes"], N - 1, 1, bits, status, dense_mask=dense)
    ws = torch.zeros(max(256, tv.tv_attn_workspace_bytes(B, N, Hq, Hkv, d, Scap)), dtype=torch.uint8, device=dev)
    S = case["prefix_len"]
    o_parts, l_parts = [], []
    for r in range(R):
        lo, hi = tvd.split_prefix(S, r, R)
        kc = torch.full_like(case["k_cache"][0], float("nan"))       # rows past the local range: poison
        vc = torch.full_like(case["v_cache"][0], float("nan"))
        for b in range(B):
            n_loc = int(hi[b] - lo[b])
            kc[b, :, :n_loc] = case["k_cache"][0][b, :, int(lo[b]):int(hi[b])]
            vc[b, :, :n_loc] = case["v_cache"][0][b, :, int(lo[b]):int(hi[b])]
        out = torch.empty(B, N, Hq, d, dtype=torch.bfloat16, device=dev)
        lse = torch.empty(B, Hq, N, dtype=torch.float32, device=dev)
        tv.tree_verify_attn(case["q"][0], kc, vc, case["k_tree"][0], case["v_tree"][0], (hi - lo).to(torch.int32),
                            case["n_nodes"], bits if r == R - 1 else torch.zeros_like(bits), d ** -0.5, out, ws,
                            status, lse=lse)
        torch.cuda.synchronize()
        o_parts.append(out)
        l_parts.append(lse)
    assert (status.cpu().numpy() == 0).all()
    return (torch.stack(o_parts), torch.stack(l_parts),
            oracle_visibility(case["parent"], case["n_nodes"], dense_gpu=dense, bits_gpu=bits))


@pytest.mark.parametrize("ci,over,R", [(0, dict(B=3, S_lo=0, S_hi=300, Scap=320), 2),
                                       (2, dict(B=4, Hq=8, Hkv=2, S_lo=1, S_hi=700, Scap=768), 3),
                                       (3, dict(B=2, Hq=8, Hkv=2, S_lo=1000, S_hi=1100, Scap=1152), 8),
                                       (1, dict(Hq=4, Hkv=4, S_lo=129, S_hi=129, Scap=256), 1)])
def test_context_split_merge_parity(ci, over, R):
    cfg = CONFIGS[ci].scaled(L=1, V=0, **over)
    case = make_case(cfg, seed=900 + ci, device="cuda", ragged_nodes=(cfg.B > 1), with_logits=False)
    o_parts, l_parts, dense = run_split(case, R)
    B, N, Hq, d = cfg.B, cfg.N, cfg.Hq, cfg.d
    out = torch.full((B, N, Hq, d), 3.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, Hq, N), 3.0, dtype=torch.float32, device="cuda")
    tv.tree_merge_partials(o_parts, l_parts, out, lse)
    torch.cuda.synchronize()
    got, got_lse = f32(out).astype(np.float64), lse.cpu().numpy().astype(np.float64)
    # (1) against the oracle's merge of the same partials: only the final bf16 rounding and fp32 weights differ
    ref, ref_lse = orc.merge_partials(f32(o_parts), l_parts.cpu().numpy())
    assert np.abs(got - ref).max() <= 2.0 ** -8 * max(1.0, np.abs(ref).max()) + 1e-6
    assert np.array_equal(np.isneginf(got_lse), np.isneginf(ref_lse))
    fin = np.isfinite(ref_lse)
    assert np.abs(got_lse[fin] - ref_lse[fin]).max() < 1e-4
    # (2) against the attention over the whole prefix
    c = case_to_numpy(case)
    full, full_lse = orc.tree_attention(c["q"][0], c["k_cache"][0], c["v_cache"][0], c["k_tree"][0], c["v_tree"][0],
                                        c["prefix_len"], c["n_nodes"], dense[:, 0], d ** -0.5)
    assert np.abs(got - full).max() <= ATTN_ATOL
    assert np.array_equal(np.isneginf(got_lse), np.isneginf(full_lse))
    assert np.abs(got_lse[fin] - full_lse[fin]).max() < 2e-3


def test_merge_ignores_empty_ranges_and_their_payload():
    R, B, N, Hq, d = 3, 1, 2, 2, 16
    o = torch.randn(R, B, N, Hq, d, device="cuda").to(torch.bfloat16)
    o[1] = float("nan")                                   # an empty range may hold anything
    l = torch.zeros(R, B, Hq, N, device="cuda")
    l[1] = float("-inf")
    l[:, 0, 1, 1] = float("-inf")                          # one row without any key
    out = torch.empty(B, N, Hq, d, dtype=torch.bfloat16, device="cuda")
    lse = torch.empty(B, Hq, N, device="cuda")
    tv.tree_merge_partials(o, l, out, lse)
    torch.cuda.synchronize()
    ref, ref_lse = orc.merge_partials(f32(o), l.cpu().numpy())
    assert not torch.isnan(out.float()).any()
    assert np.abs(f32(out) - ref).max() <= 2.0 ** -8 * 4
    assert (f32(out)[0, 1, 1] == 0).all() and lse[0, 1, 1].item() == float("-inf")
    assert np.isclose(lse[0, 0, 0].item(), np.log(2.0), atol=1e-6)


def test_context_split_attention_single_process_is_plain_attention():
    """Outside a process group the orchestration reduces to one member that owns everything."""
    cfg = CONFIGS[0].scaled(B=2, S_lo=5, S_hi=200, Scap=256)
    case = make_case(cfg, seed=31, device="cuda", ragged_nodes=True, with_logits=False)
    L, B, N, Hq, d = case["q"].shape
    bits = torch.zeros(B, N, (N + 31) // 32, dtype=torch.int32, device="cuda")
    status = torch.zeros(B, dtype=torch.int32, device="cuda")
    tv.tree_build_mask(case["parent"], case["n_nodes"], N - 1, 1, bits, status)
    ws = torch.zeros(max(256, tv.tv_attn_workspace_bytes(B, N, Hq, cfg.Hkv, d, cfg.Scap)), dtype=torch.uint8, device="cuda")
    out, lse = tvd.context_split_attention(case["q"][0], case["k_cache"][0], case["v_cache"][0], case["k_tree"][0],
                                           case["v_tree"][0], case["prefix_len"], case["n_nodes"], bits, d ** -0.5,
                                           ws, status, owns_tree=True)
    ref = torch.empty_like(out)
    tv.tree_verify_attn(case["q"][0], case["k_cache"][0], case["v_cache"][0], case["k_tree"][0], case["v_tree"][0],
                        case["prefix_len"], case["n_nodes"], bits, d ** -0.5, ref, ws, status)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), ref.view(torch.int16))      # one part, weight 1: unchanged
