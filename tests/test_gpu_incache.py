"""In-cache tree layout on the GPU against the oracle: tree_verify_attn with the tree's K/V rows behind
the prefix inside the cache (k_tree = v_tree = NULL), and kv_commit_inplace, the path-index commit as
a full reorder inside the cache (Section 3.1).  Attention max-abs 2e-2, committed bytes bit-exact."""
import numpy as np
import pytest
import torch

import paper_2603_08088_b200 as tv
from oracle import tree_verify_oracle as orc
from workloads import CONFIGS, make_case, case_to_numpy
from gpu_util import to_device, i32, assert_attention_close, oracle_visibility

pytestmark = pytest.mark.gpu


def place_tree_in_cache(case):
    """Copies of the case's caches with node i's K/V written at row prefix_len[b] + i (what a forward pass
    that extends the cache in place leaves behind).  Host tensors [L,B,Hkv,Scap,d]."""
    kc, vc = case["k_cache"].clone(), case["v_cache"].clone()
    N = case["k_tree"].shape[2]
    for b, S in enumerate(case["prefix_len"].tolist()):
        kc[:, b, :, S:S + N] = case["k_tree"][:, b].permute(0, 2, 1, 3)
        vc[:, b, :, S:S + N] = case["v_tree"][:, b].permute(0, 2, 1, 3)
    return kc, vc


CASES = [
    ("tiny", 0, dict(Scap=256)),
    ("d64_g2_ragged", 0, dict(B=3, S_lo=0, S_hi=300, Scap=320, N=15)),
    ("d128_g4_ragged", 2, dict(B=4, Hq=8, Hkv=2, S_lo=1, S_hi=700, Scap=768, N=64)),
    ("d128_g4_n128_tile_edge", 3, dict(B=2, Hq=8, Hkv=2, S_lo=383, S_hi=385, Scap=520, N=128)),
    ("d128_g4_n60_split", 4, dict(B=3, L=1, Hq=8, Hkv=2, S_lo=100, S_hi=520, Scap=640, V=0)),
]


@pytest.mark.parametrize("name,ci,over", CASES, ids=[c[0] for c in CASES])
def test_incache_attention_matches_oracle_and_separate_buffers(name, ci, over):
    cfg = CONFIGS[ci].scaled(**over)
    case = make_case(cfg, seed=1000 * ci + 7, ragged_nodes=(cfg.B > 1), with_logits=False)
    S = case["prefix_len"].numpy()
    n = case["n_nodes"].numpy()
    kc, vc = place_tree_in_cache(case)
    nan = torch.tensor(float("nan"), dtype=torch.bfloat16)
    for b in range(cfg.B):                      # rows behind the tree's active nodes must never reach an output
        kc[:, b, :, S[b] + n[b]:] = nan
        vc[:, b, :, S[b] + n[b]:] = nan
    dev = "cuda"
    B, N, Hq, d = cfg.B, cfg.N, cfg.Hq, cfg.d
    W = (N + 31) // 32
    bits = torch.zeros(B, N, W, dtype=torch.int32, device=dev)
    dense = torch.zeros(B, 1, N, N, dtype=torch.uint8, device=dev)
    status = torch.zeros(B, dtype=torch.int32, device=dev)
    tv.tree_build_mask(case["parent"].to(dev), case["n_nodes"].to(dev), N - 1, 1, bits, status, dense_mask=dense)
    ws = torch.zeros(max(256, tv.tv_attn_workspace_bytes(B, N, Hq, cfg.Hkv, d, cfg.Scap)), dtype=torch.uint8, device=dev)
    out = torch.full((B, N, Hq, d), 3.0, dtype=torch.bfloat16, device=dev)
    lse = torch.full((B, Hq, N), 3.0, dtype=torch.float32, device=dev)
    kcd, vcd = kc.to(dev), vc.to(dev)
    tv.tree_verify_attn(case["q"][0].to(dev), kcd[0], vcd[0], None, None, case["prefix_len"].to(dev),
                        case["n_nodes"].to(dev), bits, d ** -0.5, out, ws, status, lse=lse)
    torch.cuda.synchronize()
    assert (i32(status) == 0).all()
    # the oracle sees the definition: separate tree buffers
    case_np = case_to_numpy(case)
    vis = oracle_visibility(case["parent"], case["n_nodes"], dense_gpu=dense, bits_gpu=bits)    # the oracle's own mask
    ref_out, ref_lse = orc.tree_attention(case_np["q"][0], case_np["k_cache"][0], case_np["v_cache"][0],
                                          case_np["k_tree"][0], case_np["v_tree"][0], case_np["prefix_len"],
                                          case_np["n_nodes"], vis[:, 0], d ** -0.5)
    assert_attention_close(out, lse, ref_out, ref_lse, name)
    # and the two layouts of the same kernel agree bit for bit (same tiles, same arithmetic)
    out2 = torch.zeros_like(out)
    lse2 = torch.zeros_like(lse)
    g = to_device(case)
    tv.tree_verify_attn(g["q"][0], g["k_cache"][0], g["v_cache"][0], g["k_tree"][0], g["v_tree"][0], g["prefix_len"],
                        g["n_nodes"], bits, d ** -0.5, out2, ws, status, lse=lse2)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16)) and torch.equal(lse, lse2)
    # the cache is an input: not one byte of it changed
    assert torch.equal(kcd.view(torch.int16).cpu(), kc.view(torch.int16)) and torch.equal(vcd.view(torch.int16).cpu(), vc.view(torch.int16))


def test_incache_tree_that_does_not_fit_is_flagged():
    cfg = CONFIGS[0].scaled(B=2, S_lo=100, S_hi=100, Scap=112, N=15)
    case = make_case(cfg, seed=11, with_logits=False)
    dev = "cuda"
    B, N, Hq, d = cfg.B, cfg.N, cfg.Hq, cfg.d
    S = torch.tensor([100, 90], dtype=torch.int32)        # 100 + 15 > 112; 90 + 15 fits
    bits = torch.zeros(B, N, 1, dtype=torch.int32, device=dev)
    status = torch.zeros(B, dtype=torch.int32, device=dev)
    tv.tree_build_mask(case["parent"].to(dev), case["n_nodes"].to(dev), N - 1, 1, bits, status)
    ws = torch.zeros(max(256, tv.tv_attn_workspace_bytes(B, N, Hq, cfg.Hkv, d, cfg.Scap)), dtype=torch.uint8, device=dev)
    out = torch.zeros(B, N, Hq, d, dtype=torch.bfloat16, device=dev)
    tv.tree_verify_attn(case["q"][0].to(dev), case["k_cache"][0].to(dev), case["v_cache"][0].to(dev), None, None,
                        S.to(dev), case["n_nodes"].to(dev), bits, d ** -0.5, out, ws, status)
    torch.cuda.synchronize()
    assert i32(status).tolist() == [tv.TV_ST_CAPACITY, 0]
    assert torch.isfinite(out.float()).all()
    with pytest.raises(tv.TreeVerifyError):               # one of the two tree pointers alone is an argument error
        tv.tree_verify_attn(case["q"][0].to(dev), case["k_cache"][0].to(dev), case["v_cache"][0].to(dev),
                            case["k_tree"][0].to(dev), None, S.to(dev), case["n_nodes"].to(dev), bits, d ** -0.5,
                            out, ws, status)


def gpu_commit_inplace(kc, vc, nodes, A, S, Nmax, status_in=None):
    dev = "cuda"
    B = kc.shape[1]
    pad = 4096
    def guarded(a):
        t = torch.from_numpy(a.view(np.int16))
        flat = torch.full((t.numel() + 2 * pad,), 0x1234, dtype=torch.int16, device=dev)
        flat[pad:-pad] = t.reshape(-1).to(dev)
        return flat, flat[pad:-pad].view(t.shape)
    kflat, kcd = guarded(kc)
    vflat, vcd = guarded(vc)
    Sd = torch.from_numpy(S.astype(np.int32)).to(dev)
    st = torch.zeros(B, dtype=torch.int32, device=dev) if status_in is None else torch.from_numpy(status_in.astype(np.int32)).to(dev)
    tv.kv_commit_inplace(kcd.view(torch.bfloat16), vcd.view(torch.bfloat16), torch.from_numpy(nodes.astype(np.int32)).to(dev),
                         torch.from_numpy(A.astype(np.int32)).to(dev), Sd, Nmax, st)
    torch.cuda.synchronize()
    for flat in (kflat, vflat):
        assert (flat[:pad] == 0x1234).all() and (flat[-pad:] == 0x1234).all(), "commit wrote outside the cache"
    return kcd.cpu().numpy().view(np.uint16), vcd.cpu().numpy().view(np.uint16), i32(Sd), i32(st)


@pytest.mark.parametrize("d,Hkv", [(64, 2), (128, 8), (128, 1), (256, 3)])
def test_inplace_commit_bytes_exact(d, Hkv):
    rng = np.random.default_rng(100 + d + Hkv)
    L, B, Scap, N, Dp1 = 3, 6, 48, 17, 7
    u16 = lambda *s: rng.integers(0, 2 ** 16, size=s).astype(np.uint16)
    kc, vc = u16(L, B, Hkv, Scap, d), u16(L, B, Hkv, Scap, d)
    nodes = np.zeros((B, Dp1), dtype=np.int32)
    A = np.array([6, 0, 3, 2, 1, 4], dtype=np.int32)
    for b in range(B):
        nodes[b, 1:A[b] + 1] = np.sort(rng.choice(np.arange(1, N), size=A[b], replace=False))
    nodes[0, :7] = [0, 1, 3, 4, 5, 9, 10]        # chains of overlaps: rows 3, 4, 5 are sources and destinations
    nodes[5, :5] = [0, 2, 3, 4, 16]
    nodes[4, :2] = [0, 5]
    S = np.array([0, 31, 27, 20, 30, 31], dtype=np.int32)     # b=5: source row 31 + 16 = 47, the last row
    status_in = np.array([0, 0, 0, orc.ST_BAD_TREE, 0, 0])
    got = gpu_commit_inplace(kc, vc, nodes, A, S, N, status_in)
    ref = orc.kv_commit_inplace(kc, vc, nodes, A, S, N, status_in)
    for g, r, what in zip(got, ref, ("k", "v", "prefix_len", "status")):
        assert np.array_equal(g, r), f"{what} differs"
    assert got[2].tolist() == [7, 32, 31, 20, 32, 36]
    # capacity (segment or source row past the end), bad node id, bad length: flagged and untouched
    S_bad = np.array([44, 0, 0, 0, 40, 32], dtype=np.int32)
    nodes_bad = nodes.copy()
    nodes_bad[2, 1] = N
    A_bad = A.copy()
    A_bad[3] = Dp1
    got = gpu_commit_inplace(kc, vc, nodes_bad, A_bad, S_bad, N)
    ref = orc.kv_commit_inplace(kc, vc, nodes_bad, A_bad, S_bad, N)
    for g, r, what in zip(got, ref, ("k", "v", "prefix_len", "status")):
        assert np.array_equal(g, r), f"{what} differs"
    assert got[3].tolist() == [orc.ST_CAPACITY, 0, orc.ST_BAD_INDEX, orc.ST_BAD_INDEX, 0, orc.ST_CAPACITY]


def test_inplace_commit_longest_supported_path_and_argument_errors():
    rng = np.random.default_rng(5)
    L, B, Hkv, Scap, d, N, Dp1 = 1, 2, 2, 300, 128, 256, 128      # Dp1 * d / 8 = 2048: eight pieces per thread
    kc = rng.integers(0, 2 ** 16, size=(L, B, Hkv, Scap, d)).astype(np.uint16)
    vc = rng.integers(0, 2 ** 16, size=(L, B, Hkv, Scap, d)).astype(np.uint16)
    nodes = np.zeros((B, Dp1), dtype=np.int32)
    nodes[0] = np.arange(Dp1) * 2                         # every other node: each row both source and destination
    nodes[1, :3] = [0, 200, 255]
    A = np.array([Dp1 - 1, 2], dtype=np.int32)
    S = np.array([40, 44], dtype=np.int32)
    got = gpu_commit_inplace(kc, vc, nodes, A, S, N)
    ref = orc.kv_commit_inplace(kc, vc, nodes, A, S, N)
    for g, r in zip(got, ref):
        assert np.array_equal(g, r)
    z = torch.zeros(1, dtype=torch.int32, device="cuda")
    big = torch.zeros(1, 1, 1, 8, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(tv.TreeVerifyError):               # Dp1 * d / 8 > 2048
        tv.kv_commit_inplace(big, big, torch.zeros(1, 129, dtype=torch.int32, device="cuda"), z, z, 4, z)


def test_step_with_incache_layout_equals_step_with_separate_buffers():
    """Mask, in-cache attention, accept and in-place commit give, on the committed rows, exactly what the
    separate-buffer step gives; a following one-node verify then reads the same prefix (commit
    equivalence, Section 3.1)."""
    cfg = CONFIGS[4].scaled(B=4, L=2, Hq=8, Hkv=2, S_lo=60, S_hi=400, Scap=512, V=4096)
    case = make_case(cfg, seed=4321)
    case_np = case_to_numpy(case)
    ref = orc.verify_step(case_np, cfg.d ** -0.5)
    dev = "cuda"
    kc, vc = place_tree_in_cache(case)
    kcd, vcd = kc.to(dev), vc.to(dev)
    B, N, Hq, d, L = cfg.B, cfg.N, cfg.Hq, cfg.d, cfg.L
    W = (N + 31) // 32
    bits = torch.zeros(B, N, W, dtype=torch.int32, device=dev)
    status = torch.zeros(B, dtype=torch.int32, device=dev)
    S = case["prefix_len"].to(dev)
    nn = case["n_nodes"].to(dev)
    tv.tree_build_mask(case["parent"].to(dev), nn, N - 1, 1, bits, status)
    ws = torch.zeros(max(256, tv.tv_attn_workspace_bytes(B, N, Hq, cfg.Hkv, d, cfg.Scap)), dtype=torch.uint8, device=dev)
    out = torch.zeros(L, B, N, Hq, d, dtype=torch.bfloat16, device=dev)
    for l in range(L):
        tv.tree_verify_attn(case["q"][l].to(dev), kcd[l], vcd[l], None, None, S, nn, bits, d ** -0.5, out[l], ws, status)
    retrieve = case["retrieve"].to(dev)
    Dp1 = retrieve.shape[2]
    z = lambda *s: torch.zeros(s, dtype=torch.int32, device=dev)
    am, alen, best, anodes, nxt = z(B, N), z(B), z(B), z(B, Dp1), z(B)
    aws = torch.zeros(max(16, tv.tv_accept_workspace_bytes(B, N, cfg.V)), dtype=torch.uint8, device=dev)
    tv.tree_accept(case["logits"].to(dev), case["tokens"].to(dev), retrieve, nn, am, alen, best, anodes, nxt, aws, status)
    tv.kv_commit_inplace(kcd, vcd, anodes, alen, S, N, status)
    torch.cuda.synchronize()
    assert (i32(status) == 0).all()
    assert np.array_equal(i32(alen), ref["accept"]["accept_len"]) and np.array_equal(i32(anodes), ref["accept"]["accepted_nodes"])
    assert np.array_equal(i32(S), ref["prefix_len"])
    got_k = kcd.cpu().view(torch.int16).numpy().view(np.uint16)
    got_v = vcd.cpu().view(torch.int16).numpy().view(np.uint16)
    for b in range(B):
        T = int(ref["prefix_len"][b])
        assert np.array_equal(got_k[:, b, :, :T], ref["k_cache"][:, b, :, :T]), "committed K rows differ"
        assert np.array_equal(got_v[:, b, :, :T], ref["v_cache"][:, b, :, :T]), "committed V rows differ"
    for l in range(L):
        err = np.abs(out[l].float().cpu().numpy().astype(np.float64) - ref["out"][l]).max()
        assert err <= 2e-2
