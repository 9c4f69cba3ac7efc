"""tree_verify_attn on the GPU against the fp64 oracle (max-abs 2e-2), plus the
checks that pin the mask through the whole kernel: closed forms, leak canaries,
NaN-poisoned padding, non-ancestor perturbation, state safety."""
import math

import numpy as np
import pytest
import torch

import paper_2603_08088_b200 as tv
from oracle import tree_verify_oracle as orc
from workloads import (CONFIGS, make_case, case_to_numpy, bf16_bits, random_parent_tree, topk_expansion_tree,
                       chain_tree)
from gpu_util import to_device, f32, assert_attention_close, oracle_attention_slice, oracle_visibility, ATTN_ATOL

pytestmark = pytest.mark.gpu


def gpu_attention(case, layer=0, simt=False):
    """case: device tensors.  Returns (out, lse, anc_bits, dense) for one layer; `dense` is the ORACLE's
    mask of the same trees (the CUDA mask is checked equal to it here and then dropped), so that every
    expected value below comes from the oracle alone."""
    L, B, N, Hq, d = case["q"].shape
    Hkv, Scap = case["k_cache"].shape[2], case["k_cache"].shape[3]
    dev = case["q"].device
    W = (N + 31) // 32
    bits = torch.zeros(B, N, W, dtype=torch.int32, device=dev)
    dense = torch.zeros(B, 1, N, N, dtype=torch.uint8, device=dev)
    status = torch.zeros(B, dtype=torch.int32, device=dev)
    tv.tree_build_mask(case["parent"], case["n_nodes"], N - 1, 1, bits, status, dense_mask=dense)
    out = torch.full((B, N, Hq, d), 3.0, dtype=torch.bfloat16, device=dev)
    lse = torch.full((B, Hq, N), 3.0, dtype=torch.float32, device=dev)
    scale = d ** -0.5
    if simt:
        tv.tv_debug_attn_simt(case["q"][layer], case["k_cache"][layer], case["v_cache"][layer],
                              case["k_tree"][layer], case["v_tree"][layer], case["prefix_len"],
                              case["n_nodes"], bits, scale, out, lse=lse)
    else:
        ws = torch.zeros(max(256, tv.tv_attn_workspace_bytes(B, N, Hq, Hkv, d, Scap)), dtype=torch.uint8, device=dev)
        tv.tree_verify_attn(case["q"][layer], case["k_cache"][layer], case["v_cache"][layer],
                            case["k_tree"][layer], case["v_tree"][layer], case["prefix_len"],
                            case["n_nodes"], bits, scale, out, ws, status, lse=lse)
    torch.cuda.synchronize()
    assert (status.cpu().numpy() == 0).all(), f"status {status.cpu().numpy()}"
    dense = torch.from_numpy(oracle_visibility(case["parent"], case["n_nodes"], dense_gpu=dense, bits_gpu=bits))
    return out, lse, bits, dense


def oracle_attention(case_np, dense, layer=0):
    d = case_np["q"].shape[-1]
    return orc.tree_attention(case_np["q"][layer], case_np["k_cache"][layer], case_np["v_cache"][layer],
                              case_np["k_tree"][layer], case_np["v_tree"][layer], case_np["prefix_len"],
                              case_np["n_nodes"], dense[:, 0], d ** -0.5)


SMALL = [
    # name, base config, overrides: several key tiles, ragged tails, both head dims, G in {1,2,4}
    ("tiny_full", 0, {}),
    ("d64_g2_ragged", 0, dict(B=3, S_lo=0, S_hi=300, Scap=320, N=15)),
    ("d128_g1", 1, dict(Hq=4, Hkv=4, S_lo=129, S_hi=129, Scap=256, N=60)),
    ("d128_g4_ragged", 2, dict(B=4, Hq=8, Hkv=2, S_lo=1, S_hi=700, Scap=768, N=64)),
    ("d128_g4_n128", 3, dict(B=2, Hq=8, Hkv=2, S_lo=383, S_hi=385, Scap=512, N=128)),
    ("d128_g4_n60", 4, dict(B=3, L=2, Hq=8, Hkv=2, S_lo=100, S_hi=520, Scap=640, V=0)),
]


@pytest.mark.parametrize("name,ci,over", SMALL, ids=[s[0] for s in SMALL])
@pytest.mark.parametrize("simt", [False, True], ids=["tc", "simt"])
def test_attention_parity_small(name, ci, over, simt):
    cfg = CONFIGS[ci].scaled(**over)
    case = make_case(cfg, seed=1000 * ci + 1, ragged_nodes=(cfg.B > 1), with_logits=False)
    # rows past the prefix and padded tree slots hold NaN: they must never reach an output
    S = case["prefix_len"].numpy()
    n = case["n_nodes"].numpy()
    nan = torch.tensor(float("nan"), dtype=torch.bfloat16)
    for b in range(cfg.B):
        case["k_cache"][:, b, :, S[b]:] = nan
        case["v_cache"][:, b, :, S[b]:] = nan
        case["k_tree"][:, b, n[b]:] = nan
        case["v_tree"][:, b, n[b]:] = nan
        case["q"][:, b, n[b]:] = nan
    dcase = to_device(case)
    case_np = case_to_numpy(case)
    for layer in range(cfg.L):
        out, lse, bits, dense = gpu_attention(dcase, layer, simt=simt)
        ref_out, ref_lse = oracle_attention(case_np, dense.cpu().numpy(), layer)
        assert_attention_close(out, lse, ref_out, ref_lse, name)
        got = f32(out)
        for b in range(cfg.B):                       # padded rows are exact zeros / -inf
            assert (got[b, n[b]:] == 0).all()
            assert np.isneginf(f32(lse)[b, :, n[b]:]).all()


GROUPS = [
    # (query heads per KV head, KV heads, nodes, d): group sizes that do not divide the 128-row tile leave rows of
    # every tile unused (128 // G nodes per tile), and large groups put few nodes into a tile
    (3, 2, 50, 128), (5, 1, 30, 128), (6, 2, 64, 64), (7, 4, 26, 128), (12, 1, 21, 128), (24, 1, 11, 64),
    (128, 1, 3, 128), (7, 1, 129, 128),
]


@pytest.mark.parametrize("G,Hkv,N,d", GROUPS, ids=[f"G{g}_kv{h}_N{n}_d{d}" for g, h, n, d in GROUPS])
def test_group_sizes_that_do_not_divide_the_row_tile(G, Hkv, N, d):
    cfg = CONFIGS[0].scaled(B=3, Hq=G * Hkv, Hkv=Hkv, d=d, S_lo=0, S_hi=700, Scap=1024, N=N, D=min(6, N - 1), V=0,
                            tree="uniform")
    case = make_case(cfg, seed=4200 + G, ragged_nodes=True, with_logits=False)
    dcase = to_device(case)
    case_np = case_to_numpy(case)
    n = case["n_nodes"].numpy()
    out, lse, bits, dense = gpu_attention(dcase, 0)
    ref_out, ref_lse = oracle_attention(case_np, dense.cpu().numpy(), 0)
    assert_attention_close(out, lse, ref_out, ref_lse, f"G={G}")
    got = f32(out)
    for b in range(cfg.B):
        assert (got[b, n[b]:] == 0).all()
    # all layers in one launch and the paged layout walk the same row tiles
    L = 2
    cfg2 = cfg.scaled(L=L)
    case2 = make_case(cfg2, seed=4300 + G, ragged_nodes=True, with_logits=False)
    g2 = to_device(case2)
    B, Hq = cfg.B, cfg.Hq
    bits2 = torch.zeros(B, N, (N + 31) // 32, dtype=torch.int32, device="cuda")
    st = torch.zeros(B, dtype=torch.int32, device="cuda")
    tv.tree_build_mask(g2["parent"], g2["n_nodes"], N - 1, 1, bits2, st)
    ws = torch.zeros(max(256, tv.tv_attn_workspace_bytes(B, N, Hq, Hkv, d, cfg.Scap)), dtype=torch.uint8, device="cuda")
    out2 = torch.full((L, B, N, Hq, d), 3.0, dtype=torch.bfloat16, device="cuda")
    lse2 = torch.zeros(L, B, Hq, N, device="cuda")
    tv.tree_verify_attn_layers(g2["q"], g2["k_cache"], g2["v_cache"], g2["k_tree"], g2["v_tree"], g2["prefix_len"],
                               g2["n_nodes"], bits2, d ** -0.5, out2, ws, st, lse=lse2)
    torch.cuda.synchronize()
    assert (st.cpu().numpy() == 0).all()
    vis = oracle_visibility(case2["parent"], case2["n_nodes"], bits_gpu=bits2)
    cn = case_to_numpy(case2)
    for l in range(L):
        r_out, r_lse = orc.tree_attention(cn["q"][l], cn["k_cache"][l], cn["v_cache"][l], cn["k_tree"][l], cn["v_tree"][l],
                                          cn["prefix_len"], cn["n_nodes"], vis[:, 0], d ** -0.5)
        assert_attention_close(out2[l], lse2[l], r_out, r_lse, f"G={G}, layer {l}")


@pytest.mark.parametrize("B", [33, 70, 512])
def test_many_sequences_up_to_the_maximum(B):
    """The schedule table is built 32 sequences at a time and searched per work item; the library takes up to
    512 sequences.  Short ragged sequences, so that most CTAs walk many units."""
    cfg = CONFIGS[0].scaled(B=B, Hq=4, Hkv=2, d=64, S_lo=0, S_hi=300, Scap=384, N=9, D=4, V=0, tree="uniform")
    case = make_case(cfg, seed=9000 + B, ragged_nodes=True, with_logits=False)
    dcase = to_device(case)
    out, lse, bits, dense = gpu_attention(dcase, 0)
    ref_out, ref_lse = oracle_attention(case_to_numpy(case), dense.cpu().numpy(), 0)
    assert_attention_close(out, lse, ref_out, ref_lse, f"B={B}")
    if B == 512:                # one more sequence is refused, nothing is launched
        big = CONFIGS[0].scaled(B=513, Hq=4, Hkv=2, d=64, S_lo=0, S_hi=10, Scap=128, N=9, D=4, V=0, tree="uniform")
        g = to_device(make_case(big, seed=1, with_logits=False))
        ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
        st = torch.zeros(513, dtype=torch.int32, device="cuda")
        o = torch.zeros(513, 9, 4, 64, dtype=torch.bfloat16, device="cuda")
        b513 = torch.zeros(513, 9, 1, dtype=torch.int32, device="cuda")
        with pytest.raises(tv.TreeVerifyError):
            tv.tree_verify_attn(g["q"][0], g["k_cache"][0], g["v_cache"][0], g["k_tree"][0], g["v_tree"][0], g["prefix_len"],
                                g["n_nodes"], b513, 0.125, o, ws, st)


@pytest.mark.parametrize("d,G", [(128, 4), (64, 1), (128, 8)])
def test_prefix_lengths_on_and_around_tile_boundaries(d, G):
    """Prefixes of 0, 127, 128, 129, 255, 256, 257 keys and one that fills the cache to its last row: the ragged
    last prefix tile has 127, 0 (it does not exist), 1 ... valid keys.  Rows behind each prefix hold NaN."""
    S = np.array([0, 127, 128, 129, 255, 256, 257, 512], dtype=np.int32)
    B, Scap, N = len(S), 512, 33
    cfg = CONFIGS[0].scaled(B=B, Hq=2 * G, Hkv=2, d=d, S_lo=0, S_hi=Scap, Scap=Scap, N=N, D=6, V=0, tree="uniform")
    case = make_case(cfg, seed=777 + d + G, ragged_nodes=True, with_logits=False)
    case["prefix_len"] = torch.from_numpy(S.copy())
    nan = torch.tensor(float("nan"), dtype=torch.bfloat16)
    for b in range(B):
        case["k_cache"][:, b, :, S[b]:] = nan
        case["v_cache"][:, b, :, S[b]:] = nan
    out, lse, bits, dense = gpu_attention(to_device(case), 0)
    ref_out, ref_lse = oracle_attention(case_to_numpy(case), dense.cpu().numpy(), 0)
    assert_attention_close(out, lse, ref_out, ref_lse, f"d={d} G={G}")


BUDGETS = [(16, 10), (32, 10), (64, 4), (64, 16), (128, 10), (200, 12), (256, 10), (256, 16)]


@pytest.mark.parametrize("N,D", BUDGETS, ids=[f"M{n}_D{d}" for n, d in BUDGETS])
def test_budget_sweep_shapes(N, D):
    """Node budgets and depth bounds of the paper's sweep (Table 2: M in 16..256, Dmax in 4..16);
    more than 128 nodes means two tree key tiles and eight mask words per row."""
    cfg = CONFIGS[2].scaled(B=3, Hq=8, Hkv=2, S_lo=100, S_hi=420, Scap=512, N=N, D=D, tree="spine", V=0)
    case = make_case(cfg, seed=7000 + N + D, ragged_nodes=True, with_logits=False)
    n = case["n_nodes"].numpy()
    nan = torch.tensor(float("nan"), dtype=torch.bfloat16)
    for b in range(cfg.B):
        case["k_tree"][:, b, n[b]:] = nan
        case["v_tree"][:, b, n[b]:] = nan
    dcase = to_device(case)
    out, lse, bits, dense = gpu_attention(dcase)
    ref_out, ref_lse = oracle_attention(case_to_numpy(case), dense.cpu().numpy())
    assert_attention_close(out, lse, ref_out, ref_lse, f"M={N} D={D}")
    out2, lse2, _, _ = gpu_attention(dcase, simt=True)
    assert_attention_close(out2, lse2, ref_out, ref_lse, f"simt M={N} D={D}")


def _tree_case(parent, S, Hq, Hkv, d, Scap, seed, std=1.0):
    N = len(parent)
    cfg = CONFIGS[0].scaled(B=1, Hq=Hq, Hkv=Hkv, d=d, S_lo=S, S_hi=S, Scap=Scap, N=N, D=min(3, N - 1), std=std, V=0)
    case = make_case(cfg, seed=seed, with_logits=False)
    case["parent"] = torch.from_numpy(parent[None].astype(np.int32))
    return case


@pytest.mark.parametrize("S", [0, 1, 16, 200])
@pytest.mark.parametrize("d", [64, 128])
def test_closed_form_zero_keys_pins_the_visible_count(S, d):
    """K = 0 => lse = ln(S + depth + 1) and out = mean of the visible V rows."""
    rng = np.random.default_rng(S + d)
    parent = topk_expansion_tree(40, 6, 4, rng)
    case = _tree_case(parent, S, 4, 2, d, 256, seed=S)
    case["k_cache"].zero_()
    case["k_tree"].zero_()
    out, lse, bits, dense = gpu_attention(to_device(case))
    ref_out, ref_lse = oracle_attention(case_to_numpy(case), dense.cpu().numpy())
    vis = dense.cpu().numpy()[0, 0]
    want = np.log(S + vis.sum(1))
    assert np.abs(f32(lse)[0] - want[None, :]).max() < 1e-4
    assert np.abs(ref_lse[0] - want[None, :]).max() < 1e-12
    assert_attention_close(out, lse, ref_out, ref_lse, "zero keys")


@pytest.mark.parametrize("S", [0, 1, 16])
def test_leak_canary_one_hot_values(S):
    """Tree V rows are 100 * e_j and tree keys score alike, so a leaked
    non-ancestor or a missing ancestor moves the output by far more than 2e-2."""
    rng = np.random.default_rng(40 + S)
    N, d = 60, 64
    parent = topk_expansion_tree(N, 6, 10, rng)
    case = _tree_case(parent, S, 2, 1, d, 64, seed=S + 9)
    case["v_tree"].zero_()
    for j in range(N):
        case["v_tree"][0, 0, j, 0, j % d] = 100.0
    case["v_cache"].zero_()
    case["k_tree"].zero_()
    case["k_cache"].zero_()
    out, lse, bits, dense = gpu_attention(to_device(case))
    ref_out, ref_lse = oracle_attention(case_to_numpy(case), dense.cpu().numpy())
    vis = dense.cpu().numpy()[0, 0].astype(np.float64)
    want = np.zeros((N, d))
    for i in range(N):
        for j in np.flatnonzero(vis[i]):
            want[i, j % d] += 100.0 / (S + vis[i].sum())
    assert np.abs(ref_out[0, :, 0] - want).max() < 1e-9
    got = f32(out)[0]
    for h in range(2):
        assert np.abs(got[:, h] - want).max() <= 0.26      # 100/k rounded to bf16: half-ulp of 64..128 is 0.25
    # a leak of one key would shift some entry by >= 100/(S+8) > 4


MOVES = [
    # name, S, N, index of the dominant key (prefix row, or S + tree node)
    ("ragged_prefix_tile_second_half", 242, 8, 200),
    ("first_tile_of_the_item_second_half", 100, 8, 80),
    ("tree_tile_second_half", 40, 128, 40 + 100),
    ("whole_tile_then_ragged_tile", 370, 8, 340),
    # full, unmasked prefix tiles: the fast path's row-sum check has to reject the tile and the careful path redo it
    ("full_tile_first_half", 600, 8, 260),
    ("full_tile_second_half", 600, 8, 350),
    ("opening_tile_early_key", 600, 8, 5),
    ("opening_tile_late_key", 600, 8, 120),
    ("last_full_tile_last_key", 640, 8, 639),
    # a jump of about 2^367: 2^x overflows in the fast path, the factor of the rescale underflows to zero
    ("extreme_jump_in_a_full_tile", 600, 8, 350),
    ("extreme_jump_in_the_tree_tile", 40, 128, 40 + 100),
]


@pytest.mark.parametrize("name,S,N,big", MOVES, ids=[m[0] for m in MOVES])
@pytest.mark.parametrize("d", [64, 128])
def test_reference_maximum_moving_inside_a_tile(name, S, N, big, d):
    """The softmax keeps a lazy reference maximum and rescales only when the maximum grows by more than 2^8.
    Masked key tiles are worked through in two halves of 64 keys; here one key in the SECOND half of such a
    tile scores 2^12 above everything before it, so the reference moves after the first half has already
    produced its probabilities: they have to move with it.  All other scores are 0, so every visible key
    before the dominant one has weight 1 and that one 2^12.2: the output is a known mixture."""
    parent = chain_tree(N)                          # node i sees nodes 0..i: tree key j is visible to rows >= j
    case = _tree_case(parent, S, 2, 1, d, 384 if S < 384 else 768, seed=S + N)
    case["k_cache"].zero_()
    case["k_tree"].zero_()
    case["q"].fill_(1.0)
    amp = 0.75 * (128 / d) ** 0.5                   # score = d * amp / sqrt(d); 12.24 in log2 units for both head dims
    if name.startswith("extreme"):
        amp *= 30.0
    if big < S:
        case["k_cache"][0, 0, 0, big] = amp
    else:
        case["k_tree"][0, 0, big - S, 0] = amp
    out, lse, bits, dense = gpu_attention(to_device(case))
    ref_out, ref_lse = oracle_attention(case_to_numpy(case), dense.cpu().numpy())
    assert_attention_close(out, lse, ref_out, ref_lse, name)
    # the oracle's rows that see the dominant key are that key's V row up to the 2^-12 share of the others
    cn = case_to_numpy(case)
    vbig = orc.decode_bf16(cn["v_cache"][0][0, 0, big] if big < S else cn["v_tree"][0][0, big - S, 0])
    rows = range(N) if big < S else range(big - S, N)
    for i in rows:
        assert np.abs(ref_out[0, i, 0] - vbig).max() < 0.5      # the other keys share less than 0.1 of the weight


def test_non_ancestor_perturbation_leaves_rows_bit_identical():
    rng = np.random.default_rng(5)
    parent = topk_expansion_tree(64, 7, 8, rng)
    case = _tree_case(parent, 300, 8, 2, 128, 512, seed=3, std=128 ** -0.5)
    dcase = to_device(case)
    out1, lse1, bits, dense = gpu_attention(dcase)
    vis = dense.cpu().numpy()[0, 0]
    victim = 63
    dcase["k_tree"][0, 0, victim] = 30.0
    dcase["v_tree"][0, 0, victim] = -50.0
    out2, lse2, _, _ = gpu_attention(dcase)
    a, b = bf16_bits(out1), bf16_bits(out2)
    unaffected = np.flatnonzero(vis[:, victim] == 0)
    assert len(unaffected) >= 50
    assert np.array_equal(a[0, unaffected], b[0, unaffected])
    assert np.array_equal(f32(lse1)[0][:, unaffected], f32(lse2)[0][:, unaffected])
    assert not np.array_equal(a[0, victim], b[0, victim])


def test_state_safety_cache_and_inputs_are_not_written():
    cfg = CONFIGS[2].scaled(B=2, Hq=8, Hkv=2, S_lo=200, S_hi=400, Scap=512)
    dcase = to_device(make_case(cfg, seed=8, with_logits=False))
    before = {k: dcase[k].clone() for k in ("k_cache", "v_cache", "k_tree", "v_tree", "q", "prefix_len")}
    gpu_attention(dcase)
    for k, v in before.items():
        assert torch.equal(v, dcase[k]), f"{k} was modified by tree_verify_attn"


def test_chain_tree_is_causal_attention_and_one_node_is_decode():
    for N in (1, 37):
        case = _tree_case(chain_tree(N), 150, 4, 4, 128, 256, seed=N, std=0.3)
        out, lse, bits, dense = gpu_attention(to_device(case))
        cn = case_to_numpy(case)
        q = torch.from_numpy(orc.decode_bf16(cn["q"][0]))[0].permute(1, 0, 2)
        k = torch.cat([torch.from_numpy(orc.decode_bf16(cn["k_cache"][0]))[0, :, :150],
                       torch.from_numpy(orc.decode_bf16(cn["k_tree"][0]))[0].permute(1, 0, 2)], 1)
        v = torch.cat([torch.from_numpy(orc.decode_bf16(cn["v_cache"][0]))[0, :, :150],
                       torch.from_numpy(orc.decode_bf16(cn["v_tree"][0]))[0].permute(1, 0, 2)], 1)
        allow = torch.ones(N, 150 + N).tril(diagonal=150).bool()
        ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=allow, scale=128 ** -0.5)
        err = np.abs(f32(out)[0] - ref.permute(1, 0, 2).numpy()).max()
        assert err <= ATTN_ATOL


def test_repeated_launches_are_bit_reproducible_and_never_time_out():
    """Units cut between CTAs are merged by whichever piece finishes last; the result must not depend on
    that order, and the bounded waits must never expire (they once did when a wait could lag two barrier
    phases behind)."""
    cfg = CONFIGS[4].scaled(L=1, V=0)
    dcase = make_case(cfg, seed=4001, device="cuda", with_logits=False)
    B, N = cfg.B, cfg.N
    bits = torch.zeros(B, N, (N + 31) // 32, dtype=torch.int32, device="cuda")
    status = torch.zeros(B, dtype=torch.int32, device="cuda")
    tv.tree_build_mask(dcase["parent"], dcase["n_nodes"], N - 1, 1, bits, status)
    ws = torch.zeros(tv.tv_attn_workspace_bytes(B, N, cfg.Hq, cfg.Hkv, cfg.d, cfg.Scap), dtype=torch.uint8, device="cuda")
    first = None
    for it in range(60):
        out = torch.zeros(B, N, cfg.Hq, cfg.d, dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros(B, cfg.Hq, N, dtype=torch.float32, device="cuda")
        tv.tree_verify_attn(dcase["q"][0], dcase["k_cache"][0], dcase["v_cache"][0], dcase["k_tree"][0],
                            dcase["v_tree"][0], dcase["prefix_len"], dcase["n_nodes"], bits, cfg.d ** -0.5, out,
                            ws, status, lse=lse)
        torch.cuda.synchronize()
        assert (status == 0).all(), f"launch {it}: status {status.cpu().tolist()}"
        if first is None:
            first = (out, lse)
        else:
            assert torch.equal(out, first[0]) and torch.equal(lse, first[1]), f"launch {it} differs from launch 0"


def test_back_to_back_launches_on_one_workspace_match_isolated_launches():
    """The layers of a step are launched back to back on one stream and one workspace, and a launch may
    start while the one in front is still draining.  Every launch must give exactly what it gives alone:
    no partial, counter or output of a neighbouring launch may leak in."""
    cfg = CONFIGS[4].scaled(L=4, B=6, V=0)
    dcase = make_case(cfg, seed=4100, device="cuda", with_logits=False)
    B, N, L = cfg.B, cfg.N, cfg.L
    bits = torch.zeros(B, N, (N + 31) // 32, dtype=torch.int32, device="cuda")
    status = torch.zeros(B, dtype=torch.int32, device="cuda")
    tv.tree_build_mask(dcase["parent"], dcase["n_nodes"], N - 1, 1, bits, status)
    nbytes = tv.tv_attn_workspace_bytes(B, N, cfg.Hq, cfg.Hkv, cfg.d, cfg.Scap)
    ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")

    def launch(layer, out, lse, workspace):
        tv.tree_verify_attn(dcase["q"][layer], dcase["k_cache"][layer], dcase["v_cache"][layer],
                            dcase["k_tree"][layer], dcase["v_tree"][layer], dcase["prefix_len"], dcase["n_nodes"],
                            bits, cfg.d ** -0.5, out, workspace, status, lse=lse)

    alone = []
    for layer in range(L):                      # isolated: own workspace, synchronised on both sides
        out = torch.zeros(B, N, cfg.Hq, cfg.d, dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros(B, cfg.Hq, N, dtype=torch.float32, device="cuda")
        launch(layer, out, lse, torch.zeros(nbytes, dtype=torch.uint8, device="cuda"))
        torch.cuda.synchronize()
        alone.append((out, lse))
    for rep in range(5):                        # back to back, 3 rounds over the layers, nothing in between
        outs = [torch.zeros(B, N, cfg.Hq, cfg.d, dtype=torch.bfloat16, device="cuda") for _ in range(3 * L)]
        lses = [torch.zeros(B, cfg.Hq, N, dtype=torch.float32, device="cuda") for _ in range(3 * L)]
        torch.cuda.synchronize()
        for i in range(3 * L):
            launch(i % L, outs[i], lses[i], ws)
        torch.cuda.synchronize()
        assert (status == 0).all(), f"status {status.cpu().tolist()}"
        for i in range(3 * L):
            assert torch.equal(outs[i], alone[i % L][0]) and torch.equal(lses[i], alone[i % L][1]), \
                f"round {rep}, launch {i} (layer {i % L}) differs from the isolated launch"


FULL = [(1, [(0, 0), (0, 17), (0, 31)]), (2, [(0, 0), (3, 5), (7, 7)]), (3, [(0, 0), (3, 7)]),
        (4, [(0, 0), (9, 3), (15, 7)])]


@pytest.mark.parametrize("ci,samples", FULL, ids=[CONFIGS[c].name for c, _ in FULL])
def test_attention_full_size_sampled_heads(ci, samples):
    """Full-size configs in the launch configuration the bench uses; the oracle
    checks sampled (sequence, KV head) slices one by one."""
    cfg = CONFIGS[ci].scaled(L=min(CONFIGS[ci].L, 2), V=0)
    dcase = make_case(cfg, seed=1000 * ci, device="cuda", with_logits=False)
    layer = cfg.L - 1
    out, lse, bits, dense = gpu_attention(dcase, layer)
    vis = dense.cpu().numpy()[:, 0]
    G = cfg.Hq // cfg.Hkv
    case_np = {k: (bf16_bits(v[layer:layer + 1]) if v.dtype == torch.bfloat16 else v.cpu().numpy())
               for k, v in dcase.items() if isinstance(v, torch.Tensor)}
    got_out, got_lse = f32(out), f32(lse)
    assert np.isfinite(got_out).all()
    for (b, hk) in samples:
        ref_out, ref_lse = oracle_attention_slice(case_np, 0, b, hk, G, vis, cfg.d ** -0.5)
        err = np.abs(got_out[b:b + 1, :, hk * G:(hk + 1) * G] - ref_out).max()
        assert err <= ATTN_ATOL, f"(b={b}, hk={hk}): {err}"
        assert np.abs(got_lse[b:b + 1, hk * G:(hk + 1) * G] - ref_lse).max() <= 2e-3


def test_layers_call_one_launch_many_layers_and_its_limits():
    """tree_verify_attn_layers: all layers in one launch (as many as the workspace has counters for), against the
    oracle layer by layer; the same call as one launch per layer agrees to the rounding of the partials."""
    L = 35
    cfg = CONFIGS[0].scaled(B=3, L=L, S_lo=0, S_hi=600, Scap=640, N=15, Hq=8, Hkv=2, V=0)
    case = make_case(cfg, seed=77, ragged_nodes=True, with_logits=False)
    d = to_device(case)
    B, N, Hq, Hkv, dh = cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.d
    bits = torch.zeros(B, N, 1, dtype=torch.int32, device="cuda")
    status = torch.zeros(B, dtype=torch.int32, device="cuda")
    tv.tree_build_mask(d["parent"], d["n_nodes"], N - 1, 1, bits, status)
    need = tv.tv_attn_workspace_bytes(B, N, Hq, Hkv, dh, cfg.Scap)
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")

    def run(flags, workspace):
        out = torch.full((L, B, N, Hq, dh), 3.0, dtype=torch.bfloat16, device="cuda")
        lse = torch.full((L, B, Hq, N), 3.0, dtype=torch.float32, device="cuda")
        n0 = tv.tv_launch_count()
        tv.tree_verify_attn_layers(d["q"], d["k_cache"], d["v_cache"], d["k_tree"], d["v_tree"], d["prefix_len"],
                                   d["n_nodes"], bits, dh ** -0.5, out, workspace, status, lse=lse, flags=flags)
        torch.cuda.synchronize()
        assert (status.cpu().numpy() == 0).all()
        return out, lse, tv.tv_launch_count() - n0

    out, lse, launches = run(tv.TV_ATTN_STABLE_INPUTS, ws)
    assert launches == 2                                    # the workspace holds the counters of 32 layers
    vis = oracle_visibility(case["parent"], case["n_nodes"], bits_gpu=bits)
    cn = case_to_numpy(case)
    for l in range(L):
        ref_out, ref_lse = orc.tree_attention(cn["q"][l], cn["k_cache"][l], cn["v_cache"][l], cn["k_tree"][l],
                                              cn["v_tree"][l], cn["prefix_len"], cn["n_nodes"], vis[:, 0], dh ** -0.5)
        assert_attention_close(out[l], lse[l], ref_out, ref_lse, f"layer {l}")
    out2, lse2, launches2 = run(tv.TV_ATTN_LAUNCH_PER_LAYER, ws)
    assert launches2 == L
    assert (out.float() - out2.float()).abs().max().item() <= 2.0 ** -5
    # room for the counters of a single layer: still correct, one launch per layer
    per_layer = (B * Hkv * 2 * 8 + 255) // 256 * 256
    small = torch.zeros(need - 31 * per_layer, dtype=torch.uint8, device="cuda")
    out3, lse3, launches3 = run(0, small)
    assert launches3 == L and torch.equal(out3, out2) and torch.equal(lse3, lse2)
    with pytest.raises(tv.TreeVerifyError):                 # not even one layer of counters
        run(0, torch.zeros(need - 32 * per_layer, dtype=torch.uint8, device="cuda"))


def test_layers_call_with_padded_layer_strides_is_bit_equal_to_the_dense_call():
    """The layer strides are arguments of their own: tensors whose layers lie further apart than their size
    (a view into a larger allocation) give the same bits as dense ones."""
    L = 3
    cfg = CONFIGS[0].scaled(B=3, L=L, S_lo=0, S_hi=500, Scap=512, N=40, Hq=8, Hkv=2, d=128, V=0)
    case = to_device(make_case(cfg, seed=61, ragged_nodes=True, with_logits=False))
    B, N, Hq, Hkv, d, Scap = cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.d, cfg.Scap
    bits = torch.zeros(B, N, (N + 31) // 32, dtype=torch.int32, device="cuda")
    st = torch.zeros(B, dtype=torch.int32, device="cuda")
    tv.tree_build_mask(case["parent"], case["n_nodes"], N - 1, 1, bits, st)
    ws = torch.zeros(tv.tv_attn_workspace_bytes(B, N, Hq, Hkv, d, Scap), dtype=torch.uint8, device="cuda")

    def padded(t, pad):
        per = t[0].numel()
        big = torch.full((L * (per + pad),), 7.0, dtype=t.dtype, device=t.device)
        v = torch.as_strided(big, t.shape, (per + pad,) + t[0].stride())
        v.copy_(t)
        return v

    def run(q, kc, vc, kt, vt, out):
        tv.tree_verify_attn_layers(q, kc, vc, kt, vt, case["prefix_len"], case["n_nodes"], bits, d ** -0.5, out, ws, st)
        torch.cuda.synchronize()
        assert (st.cpu().numpy() == 0).all()
        return out

    dense = run(case["q"], case["k_cache"], case["v_cache"], case["k_tree"], case["v_tree"],
                torch.zeros(L, B, N, Hq, d, dtype=torch.bfloat16, device="cuda"))
    out_p = padded(torch.zeros(L, B, N, Hq, d, dtype=torch.bfloat16, device="cuda"), 24)
    got = run(padded(case["q"], 8), padded(case["k_cache"], 4096), padded(case["v_cache"], 4096), padded(case["k_tree"], 16),
              padded(case["v_tree"], 16), out_p)
    assert torch.equal(got, dense)
    per = B * N * Hq * d                       # the gaps between the layers of the output were left alone
    gaps = torch.as_strided(out_p, (L, 24), (per + 24, 1), per)
    assert (gaps == 7.0).all()
