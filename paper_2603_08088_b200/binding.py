"""ctypes binding of libtreeverify.so: the same entry points as
include/treeverify.h, taking torch tensors (device memory) and doing argument
marshalling only.  There is no fallback of any kind: if the shared library is
missing or a call fails, an exception is raised.
"""
import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libtreeverify.so")

TV_OK, TV_ERR_INVALID_ARG, TV_ERR_CUDA, TV_ERR_WORKSPACE = 0, 1, 2, 3
TV_ST_BAD_TREE, TV_ST_BAD_INDEX, TV_ST_CAPACITY, TV_ST_TIMEOUT, TV_ST_PATHS_TRUNCATED = 1, 2, 4, 8, 16
TV_ATTN_STABLE_INPUTS = 1
TV_ATTN_LAUNCH_PER_LAYER = 2

EXPORTS = ["tv_last_error", "tv_version", "tv_launch_count", "tree_build_mask", "tv_attn_workspace_bytes", "tree_verify_attn",
           "tree_verify_attn_layers", "tree_verify_attn_paged_layers",
           "tv_accept_workspace_bytes", "tree_accept", "tree_node_scores", "tree_merge_partials", "tv_accept_noalloc_max_bytes", "tree_accept_noalloc",
           "tv_sample_workspace_bytes", "tree_accept_sample",
           "kv_commit", "kv_commit_inplace", "tree_verify_attn_paged", "kv_commit_paged", "tv_step_staging_bytes",
           "tv_verify_step_host"]


class TreeVerifyError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"treeverify error {code}: {msg}")
        self.code = code


_c_int, _c_vp, _c_sz, _c_i64, _c_f = ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int64, ctypes.c_float


class StepHostArgs(ctypes.Structure):
    _fields_ = [(n, _c_vp) for n in (
        "parent", "n_nodes", "tokens", "retrieve_indices", "q", "k_tree", "v_tree", "logits", "out",
        "accept_len", "accepted_nodes", "next_token", "status", "k_cache", "v_cache", "prefix_len", "staging")]
    _fields_ += [("staging_bytes", _c_sz)]
    _fields_ += [(n, _c_int) for n in ("L", "B", "Nmax", "Hq", "Hkv", "d", "Scap", "V", "P", "Dp1")]
    _fields_ += [("scale", _c_f), ("stream", _c_vp)]


_lib = None


def load():
    """Load the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2603_08088_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    lib.tv_last_error.restype = ctypes.c_char_p
    lib.tv_last_error.argtypes = []
    lib.tv_version.restype = _c_int
    lib.tv_launch_count.restype = ctypes.c_ulonglong
    lib.tv_launch_count.argtypes = []
    lib.tree_build_mask.restype = _c_int
    lib.tree_build_mask.argtypes = [_c_vp, _c_vp, _c_int, _c_int, _c_int, _c_int] + [_c_vp] * 8
    lib.tv_attn_workspace_bytes.restype = _c_sz
    lib.tv_attn_workspace_bytes.argtypes = [_c_int] * 6
    lib.tree_verify_attn.restype = _c_int
    lib.tree_verify_attn.argtypes = [_c_vp] * 8 + [_c_int] * 6 + [_c_f, _c_vp, _c_vp, _c_vp, _c_sz, _c_vp, _c_vp]
    lib.tree_verify_attn_layers.restype = _c_int
    lib.tree_verify_attn_layers.argtypes = ([_c_vp] * 8 + [_c_int] * 7 + [_c_f] + [_c_i64] * 3 + [_c_vp, _c_i64, _c_vp, _c_vp, _c_sz,
                                            _c_vp, ctypes.c_uint, _c_vp])
    lib.tree_verify_attn_paged_layers.restype = _c_int
    lib.tree_verify_attn_paged_layers.argtypes = ([_c_vp] * 9 + [_c_int] * 8 + [_c_f] + [_c_i64] * 3 + [_c_vp, _c_i64, _c_vp, _c_vp,
                                                  _c_sz, _c_vp, ctypes.c_uint, _c_vp])
    lib.tv_accept_workspace_bytes.restype = _c_sz
    lib.tv_accept_workspace_bytes.argtypes = [_c_int] * 3
    lib.tree_accept.restype = _c_int
    lib.tree_accept.argtypes = [_c_vp] * 4 + [_c_int] * 5 + [_c_vp] * 7 + [_c_vp, _c_sz, _c_vp, _c_vp]
    lib.tree_node_scores.restype = _c_int
    lib.tree_node_scores.argtypes = [_c_vp] * 4 + [_c_int] * 3 + [_c_vp, _c_vp, _c_vp]
    lib.tree_merge_partials.restype = _c_int
    lib.tree_merge_partials.argtypes = [_c_vp, _c_vp] + [_c_int] * 5 + [_c_vp, _c_vp, _c_vp]
    lib.tv_accept_noalloc_max_bytes.restype = _c_sz
    lib.tv_accept_noalloc_max_bytes.argtypes = []
    lib.tree_accept_noalloc.restype = _c_int
    lib.tree_accept_noalloc.argtypes = [_c_vp] * 4 + [_c_int] * 5 + [_c_vp] * 7 + [_c_vp, _c_vp]
    lib.kv_commit.restype = _c_int
    lib.kv_commit.argtypes = [_c_vp] * 7 + [_c_int] * 7 + [_c_i64, _c_i64, _c_vp, _c_vp]
    lib.tv_sample_workspace_bytes.restype = _c_sz
    lib.tv_sample_workspace_bytes.argtypes = [_c_int] * 3
    lib.tree_accept_sample.restype = _c_int
    lib.tree_accept_sample.argtypes = [_c_vp] * 6 + [_c_f] + [_c_int] * 4 + [_c_vp] * 4 + [_c_sz, _c_vp, _c_vp]
    lib.tree_verify_attn_paged.restype = _c_int
    lib.tree_verify_attn_paged.argtypes = [_c_vp] * 9 + [_c_int] * 7 + [_c_f, _c_vp, _c_vp, _c_vp, _c_sz, _c_vp, _c_vp]
    lib.kv_commit_paged.restype = _c_int
    lib.kv_commit_paged.argtypes = [_c_vp] * 8 + [_c_int] * 8 + [_c_i64, _c_i64, _c_vp, _c_vp]
    lib.kv_commit_inplace.restype = _c_int
    lib.kv_commit_inplace.argtypes = [_c_vp] * 5 + [_c_int] * 7 + [_c_i64, _c_vp, _c_vp]
    lib.tv_step_staging_bytes.restype = _c_sz
    lib.tv_step_staging_bytes.argtypes = [_c_int] * 10
    lib.tv_verify_step_host.restype = _c_int
    lib.tv_verify_step_host.argtypes = [ctypes.POINTER(StepHostArgs)]
    if hasattr(lib, "tv_debug_attn_expire"):
        lib.tv_debug_attn_expire.restype = _c_int
        lib.tv_debug_attn_expire.argtypes = ([_c_vp] * 8 + [_c_int] * 6 + [_c_f, _c_vp, _c_vp, _c_vp, _c_sz, _c_vp,
                                              ctypes.c_ulonglong, _c_int, _c_vp])
    if hasattr(lib, "tv_debug_attn_stream_only"):
        lib.tv_debug_attn_stream_only.restype = _c_int
        lib.tv_debug_attn_stream_only.argtypes = ([_c_vp] * 8 + [_c_int] * 7 + [_c_i64] * 3 + [_c_vp, _c_i64, _c_vp, _c_sz,
                                                   _c_vp, _c_vp])
    if hasattr(lib, "tv_debug_attn_simt"):
        lib.tv_debug_attn_simt.restype = _c_int
        lib.tv_debug_attn_simt.argtypes = [_c_vp] * 8 + [_c_int] * 6 + [_c_f, _c_vp, _c_vp, _c_vp]
    _lib = lib
    return lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_contiguous(), "treeverify takes dense tensors"
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(rc):
    if rc != TV_OK:
        raise TreeVerifyError(rc, load().tv_last_error().decode())


def tv_version():
    return load().tv_version()


def tv_launch_count():
    return int(load().tv_launch_count())


def tv_attn_workspace_bytes(B, Nmax, Hq, Hkv, d, Scap):
    return load().tv_attn_workspace_bytes(B, Nmax, Hq, Hkv, d, Scap)


def tv_accept_workspace_bytes(B, Nmax, V):
    return load().tv_accept_workspace_bytes(B, Nmax, V)


def tv_step_staging_bytes(L, B, Nmax, Hq, Hkv, d, Scap, V, P, Dp1):
    return load().tv_step_staging_bytes(L, B, Nmax, Hq, Hkv, d, Scap, V, P, Dp1)


def tree_build_mask(parent, n_nodes, Dcap, Pcap, anc_bits, status, dense_mask=None, depth=None,
                    anc_table=None, retrieve_indices=None, n_paths=None, stream=None):
    B, Nmax = parent.shape
    _check(load().tree_build_mask(_ptr(parent), _ptr(n_nodes), B, Nmax, Dcap, Pcap, _ptr(anc_bits),
                                  _ptr(dense_mask), _ptr(depth), _ptr(anc_table), _ptr(retrieve_indices),
                                  _ptr(n_paths), _ptr(status), _stream(stream)))


def tree_verify_attn(q, k_cache, v_cache, k_tree, v_tree, prefix_len, n_nodes, anc_bits, scale, out,
                     workspace, status, lse=None, stream=None):
    B, Nmax, Hq, d = q.shape
    _, Hkv, Scap, _ = k_cache.shape
    _check(load().tree_verify_attn(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(k_tree), _ptr(v_tree),
                                   _ptr(prefix_len), _ptr(n_nodes), _ptr(anc_bits), B, Nmax, Hq, Hkv, d, Scap,
                                   float(scale), _ptr(out), _ptr(lse), _ptr(workspace),
                                   workspace.numel() * workspace.element_size(), _ptr(status), _stream(stream)))


def tree_verify_attn_layers(q, k_cache, v_cache, k_tree, v_tree, prefix_len, n_nodes, anc_bits, scale, out,
                            workspace, status, lse=None, flags=0, stream=None):
    """All layers of a step in one call: q, out [L,B,Nmax,Hq,d], k_cache, v_cache [L,B,Hkv,Scap,d], k_tree, v_tree
    [L,B,Nmax,Hkv,d] (or None: in-cache layout), lse [L,B,Hq,Nmax] or None; layer strides are taken from the tensors."""
    L, B, Nmax, Hq, d = q.shape
    _, _, Hkv, Scap, _ = k_cache.shape
    for t in (q, k_cache, v_cache, k_tree, v_tree, out, lse):
        assert t is None or t.shape[0] == L
        assert t is None or t[0].is_contiguous(), "treeverify takes dense layers"
    assert k_cache.stride(0) == v_cache.stride(0) and (k_tree is None or k_tree.stride(0) == v_tree.stride(0))
    assert lse is None or lse.is_contiguous()
    _check(load().tree_verify_attn_layers(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(),
                                          None if k_tree is None else k_tree.data_ptr(),
                                          None if v_tree is None else v_tree.data_ptr(), _ptr(prefix_len), _ptr(n_nodes),
                                          _ptr(anc_bits), L, B, Nmax, Hq, Hkv, d, Scap, float(scale), q.stride(0),
                                          k_cache.stride(0), 0 if k_tree is None else k_tree.stride(0), out.data_ptr(),
                                          out.stride(0), None if lse is None else lse.data_ptr(), _ptr(workspace),
                                          workspace.numel() * workspace.element_size(), _ptr(status), int(flags),
                                          _stream(stream)))


def tree_verify_attn_paged_layers(q, k_pages, v_pages, block_table, k_tree, v_tree, prefix_len, n_nodes, anc_bits, scale,
                                  out, workspace, status, lse=None, flags=0, stream=None):
    """All layers over a paged cache: k_pages, v_pages [L,n_pages,Hkv,128,d], one block table [B,max_blocks]."""
    L, B, Nmax, Hq, d = q.shape
    _, n_pages, Hkv, _, _ = k_pages.shape
    assert lse is None or lse.is_contiguous()
    _check(load().tree_verify_attn_paged_layers(q.data_ptr(), k_pages.data_ptr(), v_pages.data_ptr(), _ptr(block_table),
                                                k_tree.data_ptr(), v_tree.data_ptr(), _ptr(prefix_len), _ptr(n_nodes),
                                                _ptr(anc_bits), L, B, Nmax, Hq, Hkv, d, n_pages, block_table.shape[1],
                                                float(scale), q.stride(0), k_pages.stride(0), k_tree.stride(0),
                                                out.data_ptr(), out.stride(0), None if lse is None else lse.data_ptr(),
                                                _ptr(workspace), workspace.numel() * workspace.element_size(),
                                                _ptr(status), int(flags), _stream(stream)))


def tv_debug_attn_expire(q, k_cache, v_cache, k_tree, v_tree, prefix_len, n_nodes, anc_bits, scale, out, workspace, status,
                         wait_limit_ns, mode, lse=None, stream=None):
    """Test aid (treeverify_debug.h): tree_verify_attn with a short limit on its bounded waits and, with mode bit 0,
    a producer that never delivers, so that a wait expires."""
    B, Nmax, Hq, d = q.shape
    _, Hkv, Scap, _ = k_cache.shape
    _check(load().tv_debug_attn_expire(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(k_tree), _ptr(v_tree),
                                       _ptr(prefix_len), _ptr(n_nodes), _ptr(anc_bits), B, Nmax, Hq, Hkv, d, Scap,
                                       float(scale), _ptr(out), _ptr(lse), _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _ptr(status), int(wait_limit_ns),
                                       int(mode), _stream(stream)))


def tv_debug_attn_stream_only(q, k_cache, v_cache, k_tree, v_tree, prefix_len, n_nodes, anc_bits, out, workspace, status,
                              stream=None):
    """Tuning aid (treeverify_debug.h): the K/V stream of tree_verify_attn_layers alone - same launch, schedule and
    copies, no MMA, no softmax, no output.  Shapes as in tree_verify_attn_layers."""
    L, B, Nmax, Hq, d = q.shape
    _, _, Hkv, Scap, _ = k_cache.shape
    _check(load().tv_debug_attn_stream_only(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), k_tree.data_ptr(),
                                            v_tree.data_ptr(), _ptr(prefix_len), _ptr(n_nodes), _ptr(anc_bits), L, B, Nmax,
                                            Hq, Hkv, d, Scap, q.stride(0), k_cache.stride(0), k_tree.stride(0),
                                            out.data_ptr(), out.stride(0), _ptr(workspace),
                                            workspace.numel() * workspace.element_size(), _ptr(status), _stream(stream)))


def tv_debug_attn_simt(q, k_cache, v_cache, k_tree, v_tree, prefix_len, n_nodes, anc_bits, scale, out,
                       lse=None, stream=None):
    B, Nmax, Hq, d = q.shape
    _, Hkv, Scap, _ = k_cache.shape
    _check(load().tv_debug_attn_simt(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(k_tree), _ptr(v_tree),
                                     _ptr(prefix_len), _ptr(n_nodes), _ptr(anc_bits), B, Nmax, Hq, Hkv, d, Scap,
                                     float(scale), _ptr(out), _ptr(lse), _stream(stream)))


def tree_accept(logits, tokens, retrieve_indices, n_nodes, argmax_tok, accept_len, best_path, accepted_nodes,
                next_token, workspace, status, safe_idx=None, candidates=None, stream=None):
    B, Nmax, V = logits.shape
    P, Dp1 = retrieve_indices.shape[1], retrieve_indices.shape[2]
    _check(load().tree_accept(_ptr(logits), _ptr(tokens), _ptr(retrieve_indices) if P > 0 else None, _ptr(n_nodes),
                              B, Nmax, V, P, Dp1, _ptr(argmax_tok), _ptr(safe_idx), _ptr(candidates),
                              _ptr(accept_len), _ptr(best_path), _ptr(accepted_nodes), _ptr(next_token),
                              _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(status),
                              _stream(stream)))


def tree_node_scores(logits, tokens, parent, n_nodes, scores, status, stream=None):
    B, Nmax, V = logits.shape
    _check(load().tree_node_scores(_ptr(logits), _ptr(tokens), _ptr(parent), _ptr(n_nodes), B, Nmax, V,
                                   _ptr(scores), _ptr(status), _stream(stream)))


def tree_merge_partials(o_parts, lse_parts, out, lse=None, stream=None):
    R, B, Nmax, Hq, d = o_parts.shape
    _check(load().tree_merge_partials(_ptr(o_parts), _ptr(lse_parts), R, B, Nmax, Hq, d, _ptr(out),
                                      _ptr(lse) if lse is not None else None, _stream(stream)))


def tv_sample_workspace_bytes(B, Nmax, V):
    return load().tv_sample_workspace_bytes(B, Nmax, V)


def tree_accept_sample(logits, tokens, parent, n_nodes, u_node, u_bonus, temperature, accept_len, accepted_nodes,
                       next_token, workspace, status, stream=None):
    """Sampling-mode acceptance over the tree; u_node [B,Nmax] and u_bonus [B] are float32 uniforms in [0,1)."""
    B, Nmax, V = logits.shape
    _check(load().tree_accept_sample(_ptr(logits), _ptr(tokens), _ptr(parent), _ptr(n_nodes), _ptr(u_node),
                                     _ptr(u_bonus), float(temperature), B, Nmax, V, accepted_nodes.shape[1],
                                     _ptr(accept_len), _ptr(accepted_nodes), _ptr(next_token), _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _ptr(status), _stream(stream)))


def tv_accept_noalloc_max_bytes():
    return load().tv_accept_noalloc_max_bytes()


def tree_accept_noalloc(logits, tokens, retrieve_indices, n_nodes, argmax_tok, accept_len, best_path,
                        accepted_nodes, next_token, status, safe_idx=None, candidates=None, stream=None):
    """tree_accept without a caller workspace: the scratch is a fixed array inside the library, for
    callers that may not allocate device memory.  Raises TreeVerifyError (code 3) past its size limit."""
    B, Nmax, V = logits.shape
    P, Dp1 = retrieve_indices.shape[1], retrieve_indices.shape[2]
    _check(load().tree_accept_noalloc(_ptr(logits), _ptr(tokens), _ptr(retrieve_indices) if P > 0 else None,
                                      _ptr(n_nodes), B, Nmax, V, P, Dp1, _ptr(argmax_tok), _ptr(safe_idx),
                                      _ptr(candidates), _ptr(accept_len), _ptr(best_path), _ptr(accepted_nodes),
                                      _ptr(next_token), _ptr(status), _stream(stream)))


def kv_commit(k_cache, v_cache, k_tree, v_tree, accepted_nodes, accept_len, prefix_len, status, stream=None):
    L, B, Hkv, Scap, d = k_cache.shape
    Nmax = k_tree.shape[2]
    Dp1 = accepted_nodes.shape[1]
    _check(load().kv_commit(_ptr(k_cache), _ptr(v_cache), _ptr(k_tree), _ptr(v_tree), _ptr(accepted_nodes),
                            _ptr(accept_len), _ptr(prefix_len), L, B, Nmax, Hkv, d, Scap, Dp1,
                            k_cache.stride(0), k_tree.stride(0), _ptr(status), _stream(stream)))


def tree_verify_attn_paged(q, k_pages, v_pages, block_table, k_tree, v_tree, prefix_len, n_nodes, anc_bits, scale, out,
                           workspace, status, lse=None, stream=None):
    """k_pages, v_pages [n_pages,Hkv,128,d] (one layer), block_table [B,max_blocks] int32."""
    B, Nmax, Hq, d = q.shape
    n_pages, Hkv = k_pages.shape[0], k_pages.shape[1]
    assert k_pages.shape[2] == 128 and block_table.shape[0] == B
    _check(load().tree_verify_attn_paged(_ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(block_table), _ptr(k_tree),
                                         _ptr(v_tree), _ptr(prefix_len), _ptr(n_nodes), _ptr(anc_bits), B, Nmax, Hq,
                                         Hkv, d, n_pages, block_table.shape[1], float(scale), _ptr(out), _ptr(lse),
                                         _ptr(workspace), workspace.numel() * workspace.element_size(),
                                         _ptr(status), _stream(stream)))


def kv_commit_paged(k_pages, v_pages, block_table, k_tree, v_tree, accepted_nodes, accept_len, prefix_len, status,
                    stream=None):
    """k_pages, v_pages [L,n_pages,Hkv,128,d]."""
    L, n_pages, Hkv, _, d = k_pages.shape
    B, Nmax = k_tree.shape[1], k_tree.shape[2]
    _check(load().kv_commit_paged(_ptr(k_pages), _ptr(v_pages), _ptr(block_table), _ptr(k_tree), _ptr(v_tree),
                                  _ptr(accepted_nodes), _ptr(accept_len), _ptr(prefix_len), L, B, Nmax, Hkv, d,
                                  n_pages, block_table.shape[1], accepted_nodes.shape[1], k_pages.stride(0),
                                  k_tree.stride(0), _ptr(status), _stream(stream)))


def kv_commit_inplace(k_cache, v_cache, accepted_nodes, accept_len, prefix_len, Nmax, status, stream=None):
    """In-cache layout: node i's K/V are rows prefix_len[b] + i of the cache; the accepted path is gathered to
    the front of that region and prefix_len advances."""
    L, B, Hkv, Scap, d = k_cache.shape
    Dp1 = accepted_nodes.shape[1]
    _check(load().kv_commit_inplace(_ptr(k_cache), _ptr(v_cache), _ptr(accepted_nodes), _ptr(accept_len),
                                    _ptr(prefix_len), L, B, Nmax, Hkv, d, Scap, Dp1, k_cache.stride(0),
                                    _ptr(status), _stream(stream)))


def tv_verify_step_host(host, k_cache, v_cache, prefix_len, staging, scale, V, stream=None):
    """``host``: dict of pinned CPU tensors parent, n_nodes, tokens, retrieve_indices (or None), q, k_tree,
    v_tree, logits and outputs out, accept_len, accepted_nodes, next_token, status."""
    L, B, Nmax, Hq, d = host["q"].shape
    Hkv, Scap = k_cache.shape[2], k_cache.shape[3]
    Dp1 = host["accepted_nodes"].shape[1]
    r = host.get("retrieve_indices")
    P = r.shape[1] if r is not None else host["P"]
    a = StepHostArgs()
    for name in ("parent", "n_nodes", "tokens", "q", "k_tree", "v_tree", "logits", "out", "accept_len",
                 "accepted_nodes", "next_token", "status"):
        setattr(a, name, _ptr(host[name]))
    a.retrieve_indices = _ptr(r)
    a.k_cache, a.v_cache, a.prefix_len = _ptr(k_cache), _ptr(v_cache), _ptr(prefix_len)
    a.staging, a.staging_bytes = _ptr(staging), staging.numel() * staging.element_size()
    a.L, a.B, a.Nmax, a.Hq, a.Hkv, a.d, a.Scap, a.V, a.P, a.Dp1 = L, B, Nmax, Hq, Hkv, d, Scap, V, P, Dp1
    a.scale = float(scale)
    a.stream = _stream(stream)
    _check(load().tv_verify_step_host(ctypes.byref(a)))
