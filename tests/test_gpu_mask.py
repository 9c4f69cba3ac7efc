"""tree_build_mask on the GPU against the oracle: bit-exact on every output."""
import numpy as np
import pytest
import torch

import paper_2603_08088_b200 as tv
from oracle import tree_verify_oracle as orc
from workloads import CONFIGS, chain_tree, star_tree, random_parent_tree, topk_expansion_tree

pytestmark = pytest.mark.gpu


def run_mask(parent, n_nodes, Dcap, Pcap):
    dev = "cuda"
    B, Nmax = parent.shape
    W = (Nmax + 31) // 32
    i32 = dict(dtype=torch.int32, device=dev)
    guard = 64
    bufs = {
        "anc_bits": torch.full((B * Nmax * W + 2 * guard,), 0x5A5A5A5A, **i32),
        "dense": torch.full((B * Nmax * Nmax + 2 * guard,), 0xA5, dtype=torch.uint8, device=dev),
        "depth": torch.full((B * Nmax + 2 * guard,), -7, **i32),
        "anc_table": torch.full((B * (Dcap + 1) * Nmax + 2 * guard,), -7, **i32),
        "retrieve": torch.full((B * Pcap * (Dcap + 1) + 2 * guard,), -7, **i32),
        "n_paths": torch.full((B + 2 * guard,), -7, **i32),
        "status": torch.full((B + 2 * guard,), -7, **i32),
    }
    core = {k: v[guard:-guard] for k, v in bufs.items()}
    tv.tree_build_mask(torch.from_numpy(parent).to(dev), torch.from_numpy(n_nodes.astype(np.int32)).to(dev),
                       Dcap, Pcap, core["anc_bits"], core["status"], dense_mask=core["dense"],
                       depth=core["depth"], anc_table=core["anc_table"], retrieve_indices=core["retrieve"],
                       n_paths=core["n_paths"])
    torch.cuda.synchronize()
    for k, v in bufs.items():      # guard bands untouched
        fill = v[0].item()
        assert (v[:guard] == fill).all() and (v[-guard:] == fill).all(), f"{k}: wrote outside its array"
    return {
        "anc_bits": core["anc_bits"].cpu().numpy().view(np.uint32).reshape(B, Nmax, W),
        "dense": core["dense"].cpu().numpy().reshape(B, 1, Nmax, Nmax),
        "depth": core["depth"].cpu().numpy().reshape(B, Nmax),
        "anc_table": core["anc_table"].cpu().numpy().reshape(B, Dcap + 1, Nmax),
        "retrieve": core["retrieve"].cpu().numpy().reshape(B, Pcap, Dcap + 1),
        "n_paths": core["n_paths"].cpu().numpy(),
        "status": core["status"].cpu().numpy(),
    }


def check(parent, n_nodes, Dcap, Pcap):
    got = run_mask(parent, n_nodes, Dcap, Pcap)
    ref = orc.build_mask(parent, n_nodes, Dcap, Pcap)
    for k in ref:
        assert np.array_equal(got[k], ref[k]), f"{k} differs from the oracle"
    return got


@pytest.mark.parametrize("ci", range(5))
def test_mask_parity_on_the_five_configs(ci):
    cfg = CONFIGS[ci]
    rng = np.random.default_rng(1000 * ci)
    parent = np.zeros((cfg.B, cfg.N), dtype=np.int32)
    for b in range(cfg.B):
        parent[b] = (random_parent_tree(cfg.N, cfg.D, rng) if cfg.tree == "uniform"
                     else topk_expansion_tree(cfg.N, cfg.D, cfg.topk, rng))
    n = np.full(cfg.B, cfg.N, dtype=np.int32)
    got = check(parent, n, cfg.D, cfg.N)
    assert (got["status"] == 0).all()
    check(parent, n, cfg.D, cfg.P if cfg.P else 3)      # capped rows: truncation bit and kept rows


def test_mask_ragged_batch_special_trees_and_padding_garbage():
    rng = np.random.default_rng(77)
    Nmax = 100
    trees = [chain_tree(100), star_tree(64), random_parent_tree(33, 5, rng), np.array([-1], dtype=np.int32),
             topk_expansion_tree(97, 8, 6, rng), random_parent_tree(2, 1, rng)]
    parent = rng.integers(-9, 200, size=(len(trees), Nmax)).astype(np.int32)   # garbage in the padding
    n = np.zeros(len(trees), dtype=np.int32)
    for b, t in enumerate(trees):
        parent[b, :len(t)] = t
        n[b] = len(t)
    check(parent, n, 99, Nmax)
    check(parent[2:], n[2:], 8, 7)


@pytest.mark.parametrize("Nmax", [1, 31, 32, 33, 128, 129, 257, 1024])
def test_mask_sizes_around_word_boundaries(Nmax):
    rng = np.random.default_rng(Nmax)
    D = min(6, Nmax - 1)
    parent = np.stack([random_parent_tree(Nmax, D, rng) if Nmax > 1 else np.array([-1], dtype=np.int32)
                       for _ in range(3)])
    check(parent, np.full(3, Nmax, dtype=np.int32), D, min(Nmax, 64))


def test_malformed_trees_set_status_and_zero_outputs():
    base = np.array([-1, 0, 1, 2, 3, 1, 0, 6], dtype=np.int32)
    cases = []
    for kind in ["ok", "root", "range_hi", "range_neg", "order", "self", "depth"]:
        p = base.copy()
        if kind == "root":
            p[0] = 0
        elif kind == "range_hi":
            p[3] = 8
        elif kind == "range_neg":
            p[3] = -1
        elif kind == "order":
            p[2] = 4
        elif kind == "self":
            p[2] = 2
        elif kind == "depth":
            p[6] = 4          # depth 5 > Dcap
        cases.append(p)
    parent = np.stack(cases)
    n = np.full(len(cases), 8, dtype=np.int32)
    got = check(parent, n, 4, 8)
    assert got["status"].tolist() == [0] + [orc.ST_BAD_TREE] * 6
    n_bad = np.array([0, 9, -3, 8, 8, 8, 8], dtype=np.int32)      # n_nodes outside 1..Nmax
    got = check(np.stack([base] * 7), n_bad, 4, 8)
    assert got["status"].tolist() == [orc.ST_BAD_TREE] * 3 + [0] * 4
