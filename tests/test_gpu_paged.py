"""Paged committed cache on the GPU against the oracle: tree_verify_attn_paged (pages of 128 rows named by a
block table) and kv_commit_paged.  Attention max-abs 2e-2 and bit-equal to the contiguous layout; committed
bytes bit-exact."""
import numpy as np
import pytest
import torch

import paper_2603_08088_b200 as tv
from oracle import tree_verify_oracle as orc
from workloads import CONFIGS, make_case, case_to_numpy
from gpu_util import to_device, i32, assert_attention_close, oracle_visibility

pytestmark = pytest.mark.gpu
R = 128


def to_pages(cache, prefix_len, rng, spare=3, fill=None):
    """cache [B,Hkv,Scap,d] (host, bf16) -> (pages [n_pages,Hkv,128,d], block_table [B,max_blocks]): the rows of
    every sequence cut into pages, pages scattered over the pool in random order, `spare` pages nobody owns."""
    B, Hkv, Scap, d = cache.shape
    nb = (Scap + R - 1) // R
    n_pages = B * nb + spare
    order = rng.permutation(n_pages)
    pages = torch.zeros(n_pages, Hkv, R, d, dtype=cache.dtype) if fill is None else torch.full((n_pages, Hkv, R, d), fill, dtype=cache.dtype)
    bt = np.zeros((B, nb), dtype=np.int32)
    for b in range(B):
        for t in range(nb):
            pg = int(order[b * nb + t])
            bt[b, t] = pg
            rows = cache[b, :, t * R:min(Scap, (t + 1) * R)]
            pages[pg, :, :rows.shape[1]] = rows
    return pages, torch.from_numpy(bt)


CASES = [
    ("tiny", 0, dict(Scap=256)),
    ("d64_g2_ragged", 0, dict(B=3, S_lo=0, S_hi=300, Scap=384, N=15)),
    ("d128_g4_ragged", 2, dict(B=4, Hq=8, Hkv=2, S_lo=1, S_hi=700, Scap=768, N=64)),
    ("d128_g4_n128_tile_edge", 3, dict(B=2, Hq=8, Hkv=2, S_lo=383, S_hi=385, Scap=512, N=128)),
    ("d128_g4_n60_split", 4, dict(B=3, L=1, Hq=8, Hkv=2, S_lo=100, S_hi=2300, Scap=2304, V=0)),
]


@pytest.mark.parametrize("name,ci,over", CASES, ids=[c[0] for c in CASES])
def test_paged_attention_matches_oracle_and_contiguous_layout(name, ci, over):
    cfg = CONFIGS[ci].scaled(**over)
    case = make_case(cfg, seed=1000 * ci + 9, ragged_nodes=(cfg.B > 1), with_logits=False)
    rng = np.random.default_rng(ci)
    S = case["prefix_len"].numpy()
    kc, vc = case["k_cache"][0].clone(), case["v_cache"][0].clone()
    nan = torch.tensor(float("nan"), dtype=torch.bfloat16)
    for b in range(cfg.B):                      # rows past the prefix hold NaN, as do the pages nobody owns
        kc[b, :, S[b]:] = nan
        vc[b, :, S[b]:] = nan
    kp, bt = to_pages(kc, S, rng, fill=float("nan"))
    vp, _ = to_pages(vc, S, np.random.default_rng(ci), fill=float("nan"))
    # the oracle's view through the block table is the contiguous cache
    assert np.array_equal(orc.paged_to_contiguous(kp.view(torch.int16).numpy(), bt.numpy())[:, :, :cfg.Scap],
                          kc.view(torch.int16).numpy())
    dev = "cuda"
    B, N, Hq, d = cfg.B, cfg.N, cfg.Hq, cfg.d
    W = (N + 31) // 32
    bits = torch.zeros(B, N, W, dtype=torch.int32, device=dev)
    dense = torch.zeros(B, 1, N, N, dtype=torch.uint8, device=dev)
    status = torch.zeros(B, dtype=torch.int32, device=dev)
    g = to_device(case)
    tv.tree_build_mask(g["parent"], g["n_nodes"], N - 1, 1, bits, status, dense_mask=dense)
    ws = torch.zeros(max(256, tv.tv_attn_workspace_bytes(B, N, Hq, cfg.Hkv, d, cfg.Scap)), dtype=torch.uint8, device=dev)
    out = torch.full((B, N, Hq, d), 3.0, dtype=torch.bfloat16, device=dev)
    lse = torch.full((B, Hq, N), 3.0, dtype=torch.float32, device=dev)
    kpd, vpd, btd = kp.to(dev), vp.to(dev), bt.to(dev)
    tv.tree_verify_attn_paged(g["q"][0], kpd, vpd, btd, g["k_tree"][0], g["v_tree"][0], g["prefix_len"], g["n_nodes"],
                              bits, d ** -0.5, out, ws, status, lse=lse)
    torch.cuda.synchronize()
    assert (i32(status) == 0).all()
    case_np = case_to_numpy(case)
    vis = oracle_visibility(case["parent"], case["n_nodes"], dense_gpu=dense, bits_gpu=bits)    # the oracle's own mask
    ref_out, ref_lse = orc.tree_attention(case_np["q"][0], case_np["k_cache"][0], case_np["v_cache"][0],
                                          case_np["k_tree"][0], case_np["v_tree"][0], case_np["prefix_len"],
                                          case_np["n_nodes"], vis[:, 0], d ** -0.5)
    assert_attention_close(out, lse, ref_out, ref_lse, name)
    out2, lse2 = torch.zeros_like(out), torch.zeros_like(lse)
    tv.tree_verify_attn(g["q"][0], kc.to(dev), vc.to(dev), g["k_tree"][0], g["v_tree"][0], g["prefix_len"], g["n_nodes"],
                        bits, d ** -0.5, out2, ws, status, lse=lse2)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16)) and torch.equal(lse, lse2)
    assert torch.equal(kpd.view(torch.int16).cpu(), kp.view(torch.int16)), "the pages are an input"


def test_paged_attention_bad_page_id_is_flagged_and_reads_nothing_outside():
    cfg = CONFIGS[0].scaled(B=2, S_lo=200, S_hi=200, Scap=256, N=15)
    case = make_case(cfg, seed=12, with_logits=False)
    rng = np.random.default_rng(3)
    kp, bt = to_pages(case["k_cache"][0], None, rng)
    vp, _ = to_pages(case["v_cache"][0], None, np.random.default_rng(3))
    bt[1, 1] = kp.shape[0]                           # one past the pool
    bt[0, 1] = bt[0, 0]                              # a repeated page is legal: the table is only an indirection
    dev = "cuda"
    B, N, Hq, d = cfg.B, cfg.N, cfg.Hq, cfg.d
    g = to_device(case)
    bits = torch.zeros(B, N, 1, dtype=torch.int32, device=dev)
    status = torch.zeros(B, dtype=torch.int32, device=dev)
    tv.tree_build_mask(g["parent"], g["n_nodes"], N - 1, 1, bits, status)
    ws = torch.zeros(max(256, tv.tv_attn_workspace_bytes(B, N, Hq, cfg.Hkv, d, cfg.Scap)), dtype=torch.uint8, device=dev)
    out = torch.zeros(B, N, Hq, d, dtype=torch.bfloat16, device=dev)
    tv.tree_verify_attn_paged(g["q"][0], kp.to(dev), vp.to(dev), bt.to(dev), g["k_tree"][0], g["v_tree"][0],
                              g["prefix_len"], g["n_nodes"], bits, d ** -0.5, out, ws, status)
    torch.cuda.synchronize()
    assert i32(status).tolist() == [0, tv.TV_ST_BAD_INDEX]
    assert torch.isfinite(out.float()).all()


def test_paged_commit_bytes_exact_and_step_equivalence():
    """kv_commit_paged against the oracle (pages, lengths, flags, bit-exact, guard bands), and the whole step on
    pages - mask, paged attention, accept, paged commit - equal to the oracle's contiguous step seen through
    the block table."""
    cfg = CONFIGS[4].scaled(B=4, L=2, Hq=8, Hkv=2, S_lo=60, S_hi=500, Scap=512, V=4096)
    case = make_case(cfg, seed=4322)
    case["prefix_len"][0] = 125                      # the accepted segment of b=0 crosses a page boundary
    case_np = case_to_numpy(case)
    ref = orc.verify_step(case_np, cfg.d ** -0.5)
    dev = "cuda"
    L, B, N, Hq, d = cfg.L, cfg.B, cfg.N, cfg.Hq, cfg.d
    bt = None
    kps, vps = [], []
    for l in range(L):                                # one block table for all layers, as in a serving stack
        kp, bt_l = to_pages(case["k_cache"][l], None, np.random.default_rng(8))
        vp, _ = to_pages(case["v_cache"][l], None, np.random.default_rng(8))
        bt = bt_l
        kps.append(kp)
        vps.append(vp)
    pad = 4096
    def guarded(t):
        flat = torch.full((t.numel() + 2 * pad,), 0x1234, dtype=torch.int16, device=dev)
        flat[pad:-pad] = t.view(torch.int16).reshape(-1).to(dev)
        return flat, flat[pad:-pad].view(t.shape).view(torch.bfloat16)
    kflat, kpd = guarded(torch.stack(kps))
    vflat, vpd = guarded(torch.stack(vps))
    btd = bt.to(dev)
    g = to_device(case)
    W = (N + 31) // 32
    bits = torch.zeros(B, N, W, dtype=torch.int32, device=dev)
    status = torch.zeros(B, dtype=torch.int32, device=dev)
    tv.tree_build_mask(g["parent"], g["n_nodes"], N - 1, 1, bits, status)
    ws = torch.zeros(max(256, tv.tv_attn_workspace_bytes(B, N, Hq, cfg.Hkv, d, cfg.Scap)), dtype=torch.uint8, device=dev)
    out = torch.zeros(L, B, N, Hq, d, dtype=torch.bfloat16, device=dev)
    for l in range(L):
        tv.tree_verify_attn_paged(g["q"][l], kpd[l], vpd[l], btd, g["k_tree"][l], g["v_tree"][l], g["prefix_len"],
                                  g["n_nodes"], bits, d ** -0.5, out[l], ws, status)
    Dp1 = g["retrieve"].shape[2]
    z = lambda *s: torch.zeros(s, dtype=torch.int32, device=dev)
    am, alen, best, anodes, nxt = z(B, N), z(B), z(B), z(B, Dp1), z(B)
    aws = torch.zeros(max(16, tv.tv_accept_workspace_bytes(B, N, cfg.V)), dtype=torch.uint8, device=dev)
    tv.tree_accept(g["logits"], g["tokens"], g["retrieve"], g["n_nodes"], am, alen, best, anodes, nxt, aws, status)
    tv.kv_commit_paged(kpd, vpd, btd, g["k_tree"], g["v_tree"], anodes, alen, g["prefix_len"], status)
    torch.cuda.synchronize()
    assert (i32(status) == 0).all()
    for flat in (kflat, vflat):
        assert (flat[:pad] == 0x1234).all() and (flat[-pad:] == 0x1234).all(), "commit wrote outside the pool"
    assert np.array_equal(i32(alen), ref["accept"]["accept_len"]) and np.array_equal(i32(g["prefix_len"]), ref["prefix_len"])
    # oracle on pages, fed with the GPU-independent oracle acceptance
    k_np = torch.stack(kps).view(torch.int16).numpy().view(np.uint16)
    v_np = torch.stack(vps).view(torch.int16).numpy().view(np.uint16)
    rk, rv, rS, rst = orc.kv_commit_paged(k_np, v_np, bt.numpy(), case_np["k_tree"], case_np["v_tree"],
                                          ref["accept"]["accepted_nodes"], ref["accept"]["accept_len"], case_np["prefix_len"])
    assert np.array_equal(kpd.view(torch.int16).cpu().numpy().view(np.uint16), rk), "committed K pages differ"
    assert np.array_equal(vpd.view(torch.int16).cpu().numpy().view(np.uint16), rv), "committed V pages differ"
    # ... which is the contiguous step's cache seen through the block table
    for l in range(L):
        assert np.array_equal(orc.paged_to_contiguous(rk[l], bt.numpy())[:, :, :cfg.Scap], ref["k_cache"][l])
    for l in range(L):
        err = np.abs(out[l].float().cpu().numpy().astype(np.float64) - ref["out"][l]).max()
        assert err <= 2e-2


def test_paged_commit_flags():
    rng = np.random.default_rng(2)
    L, B, Hkv, d, N, Dp1, n_pages, nb = 2, 4, 2, 64, 9, 4, 12, 2
    u16 = lambda *s_: torch.from_numpy(rng.integers(0, 2 ** 16, size=s_).astype(np.int16)).view(torch.bfloat16)
    kp, vp = u16(L, n_pages, Hkv, R, d), u16(L, n_pages, Hkv, R, d)
    kt, vt = u16(L, B, N, Hkv, d), u16(L, B, N, Hkv, d)
    bt = np.array([[7, 2], [0, 12], [3, 8], [4, 5]], dtype=np.int32)       # b=1: its second page is outside the pool
    nodes = np.array([[0, 2, 5, 8], [0, 1, 3, 0], [0, 3, 9, 0], [0, 1, 2, 3]], dtype=np.int32)   # b=2: node 9 >= N
    A = np.array([3, 2, 2, 3], dtype=np.int32)
    S = np.array([253, 126, 0, 100], dtype=np.int32)                        # b=0: 253 + 4 > 256
    status_in = np.array([0, 0, 0, orc.ST_BAD_TREE], dtype=np.int32)
    dev = "cuda"
    kpd, vpd = kp.to(dev), vp.to(dev)
    Sd = torch.from_numpy(S).to(dev)
    st = torch.from_numpy(status_in).to(dev)
    tv.kv_commit_paged(kpd, vpd, torch.from_numpy(bt).to(dev), kt.to(dev), vt.to(dev), torch.from_numpy(nodes).to(dev),
                       torch.from_numpy(A).to(dev), Sd, st)
    torch.cuda.synchronize()
    asu = lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)
    rk, rv, rS, rst = orc.kv_commit_paged(asu(kp), asu(vp), bt, asu(kt), asu(vt), nodes, A, S, status_in)
    assert rst.tolist() == [orc.ST_CAPACITY, orc.ST_BAD_INDEX, orc.ST_BAD_INDEX, orc.ST_BAD_TREE]
    assert np.array_equal(i32(st), rst) and np.array_equal(i32(Sd), rS)
    assert np.array_equal(asu(kpd), rk) and np.array_equal(asu(vpd), rv) and np.array_equal(rk, asu(kp))


def test_paged_layers_call_equals_layer_by_layer_calls():
    """All layers over the paged cache in one launch (tree_verify_attn_paged_layers) against one
    tree_verify_attn_paged call per layer (the units are cut at other places, so the two agree to the rounding of
    the partials, not bit for bit) and against the oracle."""
    cfg = CONFIGS[4].scaled(B=5, L=3, Hq=8, Hkv=2, S_lo=60, S_hi=900, Scap=1024, V=0)
    case = make_case(cfg, seed=4400, ragged_nodes=True, with_logits=False)
    dev = "cuda"
    L, B, N, Hq, d = cfg.L, cfg.B, cfg.N, cfg.Hq, cfg.d
    kps, vps, bt = [], [], None
    for l in range(L):                                # one block table for all layers
        kp, bt = to_pages(case["k_cache"][l], None, np.random.default_rng(5))
        vp, _ = to_pages(case["v_cache"][l], None, np.random.default_rng(5))
        kps.append(kp)
        vps.append(vp)
    k_pages, v_pages = torch.stack(kps).to(dev), torch.stack(vps).to(dev)
    g = to_device(case)
    btd = bt.to(dev)
    bits = torch.zeros(B, N, (N + 31) // 32, dtype=torch.int32, device=dev)
    status = torch.zeros(B, dtype=torch.int32, device=dev)
    tv.tree_build_mask(g["parent"], g["n_nodes"], N - 1, 1, bits, status)
    ws = torch.zeros(tv.tv_attn_workspace_bytes(B, N, Hq, cfg.Hkv, d, cfg.Scap), dtype=torch.uint8, device=dev)
    one = torch.zeros(L, B, N, Hq, d, dtype=torch.bfloat16, device=dev)
    lse_one = torch.zeros(L, B, Hq, N, dtype=torch.float32, device=dev)
    for l in range(L):
        tv.tree_verify_attn_paged(g["q"][l], k_pages[l], v_pages[l], btd, g["k_tree"][l], g["v_tree"][l], g["prefix_len"],
                                  g["n_nodes"], bits, d ** -0.5, one[l], ws, status, lse=lse_one[l])
    allq = torch.full_like(one, 3.0)
    lse_all = torch.full_like(lse_one, 3.0)
    tv.tree_verify_attn_paged_layers(g["q"], k_pages, v_pages, btd, g["k_tree"], g["v_tree"], g["prefix_len"], g["n_nodes"],
                                     bits, d ** -0.5, allq, ws, status, lse=lse_all)
    torch.cuda.synchronize()
    assert (i32(status) == 0).all()
    assert (allq.float() - one.float()).abs().max().item() <= 2.0 ** -7
    both_inf = torch.isinf(lse_all) & torch.isinf(lse_one)
    assert torch.equal(torch.isinf(lse_all), torch.isinf(lse_one))
    assert torch.where(both_inf, torch.zeros_like(lse_all), lse_all - lse_one).abs().max().item() <= 1e-4
    # and against the oracle, layer by layer
    case_np = case_to_numpy(case)
    vis = oracle_visibility(case["parent"], case["n_nodes"], bits_gpu=bits)
    for l in range(L):
        ref_out, ref_lse = orc.tree_attention(case_np["q"][l], case_np["k_cache"][l], case_np["v_cache"][l],
                                              case_np["k_tree"][l], case_np["v_tree"][l], case_np["prefix_len"],
                                              case_np["n_nodes"], vis[:, 0], d ** -0.5)
        assert_attention_close(allq[l], lse_all[l], ref_out, ref_lse, f"layer {l}")
