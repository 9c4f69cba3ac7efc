"""Integer and byte outputs of a whole step at the FULL size of the two batched configurations (the ragged
GQA batch with vocabulary 128256, and the 32-layer step with vocabulary 153600 and a cache of 2.2 G elements
per tensor, i.e. element offsets past 2^31), in the call sequence bench.py times.  Everything the oracle can
state exactly is compared bit for bit: mask words, depths, ancestor table, candidate rows, argmax tokens,
safe indices, gathered candidates, accepted lengths, winning rows, node lists, next tokens, status, the
advanced prefix lengths and every byte of the committed cache, layer by layer (the host never holds more
than one layer of the cache twice)."""
import numpy as np
import pytest
import torch

import paper_2603_08088_b200 as tv
from oracle import tree_verify_oracle as orc
from workloads import CONFIGS, make_case, bf16_bits
from gpu_util import i32, f32, oracle_attention_slice, ATTN_ATOL

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("ci", [2, 4], ids=[CONFIGS[2].name, CONFIGS[4].name])
def test_full_size_step_integers_and_committed_bytes(ci):
    cfg = CONFIGS[ci]
    need = 2 * 2 * cfg.L * cfg.B * cfg.Hkv * cfg.Scap * cfg.d * 2 + (4 << 30)       # cache + pre-commit copy + the rest
    if torch.cuda.mem_get_info()[0] < need:
        pytest.skip(f"needs {need >> 30} GiB of free device memory")
    d = make_case(cfg, seed=1000 * ci + 3, device="cuda")
    given_rows = cfg.P > 0
    P, Dp1 = d["retrieve"].shape[1], cfg.D + 1
    k_before, v_before = d["k_cache"].clone(), d["v_cache"].clone()
    S0 = i32(d["prefix_len"]).copy()
    buf = tv.StepBuffers(cfg.L, cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.d, cfg.Scap, cfg.V, P, Dp1, want_dense=True,
                         want_gather=True)
    tv.verify_step(d, buf, cfg.d ** -0.5, retrieve=d["retrieve"] if given_rows else None)
    torch.cuda.synchronize()

    # ---- mask and tensorisation
    parent, n_nodes = i32(d["parent"]), i32(d["n_nodes"])
    mk = orc.build_mask(parent, n_nodes, cfg.D, P, emit_paths=not given_rows)
    assert np.array_equal(i32(buf.anc_bits).view(np.uint32), mk["anc_bits"])
    assert np.array_equal(i32(buf.dense), mk["dense"])
    assert np.array_equal(i32(buf.depth), mk["depth"])
    assert np.array_equal(i32(buf.anc_table), mk["anc_table"])
    if not given_rows:
        assert np.array_equal(i32(buf.retrieve), mk["retrieve"]) and np.array_equal(i32(buf.n_paths), mk["n_paths"])
    rows = i32(d["retrieve"]) if given_rows else mk["retrieve"]

    # ---- attention of the one launch that covers all layers: sampled (layer, sequence, KV head) slices against the
    # oracle (its own mask), first and last layers included
    G = cfg.Hq // cfg.Hkv
    for (l, b, hk) in {(0, 0, 0), (cfg.L - 1, cfg.B - 1, cfg.Hkv - 1), (cfg.L // 2, cfg.B // 2, 3)}:
        case_np = {"q": bf16_bits(d["q"][l:l + 1]), "k_cache": bf16_bits(k_before[l:l + 1]), "v_cache": bf16_bits(v_before[l:l + 1]),
                   "k_tree": bf16_bits(d["k_tree"][l:l + 1]), "v_tree": bf16_bits(d["v_tree"][l:l + 1]),
                   "prefix_len": S0, "n_nodes": n_nodes}
        ref_out, _ = oracle_attention_slice(case_np, 0, b, hk, G, mk["dense"][:, 0], cfg.d ** -0.5)
        got = f32(buf.out[l, b:b + 1, :, hk * G:(hk + 1) * G])
        assert np.abs(got - ref_out).max() <= ATTN_ATOL, f"attention of layer {l}, sequence {b}, KV head {hk}"

    # ---- argmax over the full vocabulary, gather, acceptance
    am = orc.argmax_rows(bf16_bits(d["logits"]), n_nodes)
    assert np.array_equal(i32(buf.argmax_tok), am)
    acc = orc.greedy_accept(rows, i32(d["tokens"]), n_nodes, am)
    for k in ("accept_len", "best_path", "accepted_nodes", "next_token", "safe_idx", "candidates"):
        assert np.array_equal(i32(getattr(buf, k)), acc[k]), k
    assert (acc["accept_len"] >= d["plant_depth"]).all()           # the planted paths are found
    status = mk["status"] | acc["status"]

    # ---- commit: every byte of every layer (offsets pass 2^31 elements in the upper layers of the 32-layer cache)
    new_len = None
    for l in range(cfg.L):
        kt, vt = bf16_bits(d["k_tree"][l:l + 1]), bf16_bits(d["v_tree"][l:l + 1])
        kc, vc, new_len, st = orc.kv_commit(bf16_bits(k_before[l:l + 1]), bf16_bits(v_before[l:l + 1]), kt, vt,
                                            acc["accepted_nodes"], acc["accept_len"], S0, status)
        assert np.array_equal(bf16_bits(d["k_cache"][l:l + 1]), kc), f"committed K bytes differ in layer {l}"
        assert np.array_equal(bf16_bits(d["v_cache"][l:l + 1]), vc), f"committed V bytes differ in layer {l}"
        assert not np.array_equal(kc, bf16_bits(k_before[l:l + 1]))     # something was committed
    assert np.array_equal(i32(buf.status), st)
    assert (st == 0).all()
    assert np.array_equal(i32(d["prefix_len"]), new_len)
    assert np.array_equal(new_len, S0 + acc["accept_len"] + 1)
