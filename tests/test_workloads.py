"""Input generators: shapes, determinism and the structural promises the
configs make (tree depth, node order, planted rows present)."""
import numpy as np
import torch

from workloads import CONFIGS, make_case, leaf_paths


def _small(cfg):
    return cfg.scaled(L=min(cfg.L, 2), S_lo=min(cfg.S_lo, 40), S_hi=min(cfg.S_hi, 90), Scap=128,
                      V=min(cfg.V, 2048) if cfg.V else 0, B=min(cfg.B, 3))


def test_cases_are_deterministic_and_well_formed():
    for ci, cfg in enumerate(CONFIGS):
        c = _small(cfg)
        a = make_case(c, seed=1000 * ci)
        b = make_case(c, seed=1000 * ci)
        for k in ("parent", "tokens", "retrieve", "prefix_len", "q", "k_cache", "v_tree"):
            assert torch.equal(a[k], b[k]), k
        par = a["parent"].numpy()
        assert a["q"].shape == (c.L, c.B, c.N, c.Hq, c.d)
        assert a["k_cache"].shape == (c.L, c.B, c.Hkv, c.Scap, c.d)
        for bb in range(c.B):
            assert par[bb, 0] == -1 and all(0 <= par[bb, i] < i for i in range(1, c.N))
            rows = leaf_paths(par[bb])
            assert max(len(r) for r in rows) == c.D + 1
        S = a["prefix_len"].numpy()
        assert (S >= c.S_lo).all() and (S <= c.S_hi).all()
        if c.V:
            assert a["logits"].shape == (c.B, c.N, c.V)


def test_ragged_nodes_pad_with_device_defined_fill():
    c = _small(CONFIGS[2])
    a = make_case(c, seed=5, ragged_nodes=True)
    n = a["n_nodes"].numpy()
    par = a["parent"].numpy()
    assert n[0] == c.N and (n >= 1).all()
    for b in range(c.B):
        assert (par[b, n[b]:] == 0).all()
        r = a["retrieve"].numpy()[b]
        assert r.max() < n[b]


def test_covering_chains_tree_rows_name_every_node():
    """The second variant of the full-step config: ten chains from the root, nine of depth 6 and one of
    depth 5, so that the ten candidate rows of seven columns cover all 60 nodes."""
    import numpy as np
    from workloads import CONFIGS, make_case, covering_chains_tree, leaf_paths
    p = covering_chains_tree(60, 10, 6, np.random.default_rng(3))
    rows = leaf_paths(p)
    assert len(rows) == 10 and sorted(len(r) - 1 for r in rows) == [5] + [6] * 9
    assert sorted(n for r in rows for n in r[1:]) == list(range(1, 60)) and all(r[0] == 0 for r in rows)
    assert (p[1:] < np.arange(1, 60)).all() and p[0] == -1
    cfg = CONFIGS[4].scaled(L=1, B=3, S_lo=4, S_hi=9, Scap=32, V=64, tree="chains")
    case = make_case(cfg, seed=1)
    r = case["retrieve"].numpy()
    assert r.shape == (3, 10, 7)
    for b in range(3):
        named = set(int(x) for x in r[b].ravel() if x >= 0)
        assert named == set(range(60))
