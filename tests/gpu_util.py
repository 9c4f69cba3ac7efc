"""Glue shared by the GPU parity tests: run the CUDA library on a case and the
oracle on the same host copy, and compare."""
import numpy as np
import torch

from oracle import tree_verify_oracle as orc
from workloads import bf16_bits, case_to_numpy

ATTN_ATOL = 2e-2     # max-abs bound on attention outputs (bf16 in, fp32 accumulate, bf16 out)
LSE_ATOL = 2e-3      # fp32 log-sum-exp against fp64


def to_device(case, device="cuda"):
    out = {}
    for k, v in case.items():
        out[k] = v.to(device) if isinstance(v, torch.Tensor) else v
    return out


def f32(t):
    return t.detach().float().cpu().numpy()


def i32(t):
    return t.detach().cpu().numpy()


def assert_attention_close(out_gpu, lse_gpu, out_ref, lse_ref, what=""):
    got = f32(out_gpu).astype(np.float64)
    assert np.isfinite(got).all(), f"{what}: non-finite attention output"
    err = np.abs(got - out_ref).max() if got.size else 0.0
    assert err <= ATTN_ATOL, f"{what}: attention max-abs error {err}"
    if lse_gpu is not None:
        lg = f32(lse_gpu).astype(np.float64)
        both_inf = np.isneginf(lg) & np.isneginf(lse_ref)
        assert (np.isneginf(lg) == np.isneginf(lse_ref)).all(), f"{what}: -inf pattern of lse differs"
        d = np.abs(np.where(both_inf, 0.0, lg) - np.where(both_inf, 0.0, lse_ref)).max() if lg.size else 0.0
        assert d <= LSE_ATOL, f"{what}: lse error {d}"
    return err


def oracle_attention_slice(case_np, layer, b, hk, G, vis, scale):
    """Oracle attention for one (layer, sequence, KV head): slices the inputs so the oracle sees
    B=1, Hkv=1, Hq=G."""
    q = case_np["q"][layer][b:b + 1, :, hk * G:(hk + 1) * G]
    kc = case_np["k_cache"][layer][b:b + 1, hk:hk + 1]
    vc = case_np["v_cache"][layer][b:b + 1, hk:hk + 1]
    kt = case_np["k_tree"][layer][b:b + 1, :, hk:hk + 1]
    vt = case_np["v_tree"][layer][b:b + 1, :, hk:hk + 1]
    return orc.tree_attention(q, kc, vc, kt, vt, case_np["prefix_len"][b:b + 1], case_np["n_nodes"][b:b + 1],
                              vis[b:b + 1], scale)


def oracle_visibility(parent, n_nodes, dense_gpu=None, bits_gpu=None):
    """The tree mask the ORACLE builds from the parent arrays, as dense[B,1,N,N] u8 (numpy).  The attention
    parity tests feed this one to the oracle's attention, never the mask the CUDA kernel produced; when the
    CUDA mask is passed in as well it must be the same bit for bit."""
    parent = np.asarray(parent.detach().cpu().numpy() if isinstance(parent, torch.Tensor) else parent)
    n_nodes = np.asarray(n_nodes.detach().cpu().numpy() if isinstance(n_nodes, torch.Tensor) else n_nodes)
    B, N = parent.shape
    # the ancestor relation does not depend on the depth bound once it covers the deepest node: take the
    # deepest level of these trees (a plain parent walk) so that the oracle's loops stay short
    deepest = 0
    for b in range(B):
        for i in range(int(n_nodes[b])):
            k, j = 0, i
            while j > 0 and k <= N:
                j = int(parent[b, j])
                k += 1
            deepest = max(deepest, k)
    mk = orc.build_mask(parent, n_nodes, min(deepest, max(N - 1, 0)), 1, emit_paths=False)
    assert (mk["status"] & orc.ST_BAD_TREE == 0).all(), "the oracle rejects a tree of this case"
    if dense_gpu is not None:
        assert np.array_equal(i32(dense_gpu), mk["dense"]), "CUDA dense mask differs from the oracle's"
    if bits_gpu is not None:
        assert np.array_equal(i32(bits_gpu).view(np.uint32), mk["anc_bits"]), "CUDA ancestor words differ from the oracle's"
    return mk["dense"]
