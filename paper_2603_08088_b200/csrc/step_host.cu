// tv_verify_step_host: one verification step driven from host buffers.
// Copies the per-step inputs into a caller-provided device staging area,
// enqueues the four calls of the step in the paper's order (tensorise + mask,
// attention per layer, gather + accept, commit; Section 3), copies the
// per-step results back and waits for the stream.  The KV cache and
// prefix_len are resident device state and are not copied.
#include "common.cuh"

namespace {

struct Staging {
  size_t parent, n_nodes, tokens, retrieve, q, k_tree, v_tree, logits, out, anc_bits, status, argmax,
      accept_len, best_path, accepted, next_token, n_paths, attn_ws, accept_ws, total;
  size_t attn_ws_bytes, accept_ws_bytes;
};

size_t up256(size_t x) { return (x + 255) & ~size_t(255); }

Staging layout(int L, int B, int Nmax, int Hq, int Hkv, int d, int Scap, int V, int P, int Dp1) {
  Staging s{};
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t at = off;
    off += up256(bytes ? bytes : 1);
    return at;
  };
  const size_t W = (Nmax + 31) / 32;
  s.parent = take(sizeof(int32_t) * B * Nmax);
  s.n_nodes = take(sizeof(int32_t) * B);
  s.tokens = take(sizeof(int32_t) * B * Nmax);
  s.retrieve = take(sizeof(int32_t) * B * P * Dp1);
  s.q = take(sizeof(tv_bf16) * (size_t)L * B * Nmax * Hq * d);
  s.k_tree = take(sizeof(tv_bf16) * (size_t)L * B * Nmax * Hkv * d);
  s.v_tree = take(sizeof(tv_bf16) * (size_t)L * B * Nmax * Hkv * d);
  s.logits = take(sizeof(tv_bf16) * (size_t)B * Nmax * V);
  s.out = take(sizeof(tv_bf16) * (size_t)L * B * Nmax * Hq * d);
  s.anc_bits = take(sizeof(uint32_t) * B * Nmax * W);
  s.status = take(sizeof(int32_t) * B);
  s.argmax = take(sizeof(int32_t) * B * Nmax);
  s.accept_len = take(sizeof(int32_t) * B);
  s.best_path = take(sizeof(int32_t) * B);
  s.accepted = take(sizeof(int32_t) * B * Dp1);
  s.next_token = take(sizeof(int32_t) * B);
  s.n_paths = take(sizeof(int32_t) * B);
  s.attn_ws_bytes = tv_attn_workspace_bytes(B, Nmax, Hq, Hkv, d, Scap);
  s.attn_ws = take(s.attn_ws_bytes);
  s.accept_ws_bytes = tv_accept_workspace_bytes(B, Nmax, V);
  s.accept_ws = take(s.accept_ws_bytes);
  s.total = off;
  return s;
}

}  // namespace

extern "C" size_t tv_step_staging_bytes(int L, int B, int Nmax, int Hq, int Hkv, int d, int Scap, int V,
                                        int P, int Dp1) {
  if (L < 0 || B < 0 || Nmax < 1 || Hq < 1 || Hkv < 1 || d < 1 || V < 1 || P < 0 || Dp1 < 1) return 0;
  return layout(L, B, Nmax, Hq, Hkv, d, Scap, V, P, Dp1).total;
}

extern "C" int tv_verify_step_host(const tv_step_host_args* a) {
  TV_REQUIRE(a, "tv_verify_step_host: NULL args");
  TV_REQUIRE(a->parent && a->n_nodes && a->tokens && a->q && a->k_tree && a->v_tree && a->logits && a->out &&
                 a->accept_len && a->accepted_nodes && a->next_token && a->status && a->k_cache && a->v_cache &&
                 a->prefix_len && a->staging,
             "tv_verify_step_host: NULL pointer");
  TV_REQUIRE(a->L >= 1 && a->B >= 1 && a->Nmax >= 1 && a->V >= 1 && a->P >= 1 && a->Dp1 >= 1 && a->Dp1 <= a->Nmax,
             "tv_verify_step_host: bad dimension");
  TV_REQUIRE((reinterpret_cast<uintptr_t>(a->staging) & 255u) == 0, "tv_verify_step_host: staging must be 256-byte aligned");
  const int L = a->L, B = a->B, Nmax = a->Nmax, Hq = a->Hq, Hkv = a->Hkv, d = a->d, Scap = a->Scap, V = a->V,
            P = a->P, Dp1 = a->Dp1;
  const Staging s = layout(L, B, Nmax, Hq, Hkv, d, Scap, V, P, Dp1);
  if (a->staging_bytes < s.total)
    return tv::fail(TV_ERR_WORKSPACE, "tv_verify_step_host: staging of %zu bytes, need %zu", a->staging_bytes, s.total);
  char* base = static_cast<char*>(a->staging);
  cudaStream_t st = (cudaStream_t)a->stream;
  auto dptr = [&](size_t off) { return base + off; };
#define TV_H2D(field, off, bytes) TV_CUDA_OK(cudaMemcpyAsync(dptr(off), a->field, (bytes), cudaMemcpyHostToDevice, st))
  TV_H2D(parent, s.parent, sizeof(int32_t) * B * Nmax);
  TV_H2D(n_nodes, s.n_nodes, sizeof(int32_t) * B);
  TV_H2D(tokens, s.tokens, sizeof(int32_t) * B * Nmax);
  if (a->retrieve_indices) TV_H2D(retrieve_indices, s.retrieve, sizeof(int32_t) * B * P * Dp1);
  TV_H2D(q, s.q, sizeof(tv_bf16) * (size_t)L * B * Nmax * Hq * d);
  TV_H2D(k_tree, s.k_tree, sizeof(tv_bf16) * (size_t)L * B * Nmax * Hkv * d);
  TV_H2D(v_tree, s.v_tree, sizeof(tv_bf16) * (size_t)L * B * Nmax * Hkv * d);
  TV_H2D(logits, s.logits, sizeof(tv_bf16) * (size_t)B * Nmax * V);
#undef TV_H2D
  int32_t* d_n_nodes = reinterpret_cast<int32_t*>(dptr(s.n_nodes));
  int32_t* d_status = reinterpret_cast<int32_t*>(dptr(s.status));
  int32_t* d_retrieve = reinterpret_cast<int32_t*>(dptr(s.retrieve));
  uint32_t* d_bits = reinterpret_cast<uint32_t*>(dptr(s.anc_bits));
  int rc = tree_build_mask(reinterpret_cast<int32_t*>(dptr(s.parent)), d_n_nodes, B, Nmax, Dp1 - 1, P, d_bits,
                           nullptr, nullptr, nullptr, a->retrieve_indices ? nullptr : d_retrieve,
                           reinterpret_cast<int32_t*>(dptr(s.n_paths)), d_status, a->stream);
  if (rc != TV_OK) return rc;
  const size_t q_layer = (size_t)B * Nmax * Hq * d, t_layer = (size_t)B * Nmax * Hkv * d,
               c_layer = (size_t)B * Hkv * Scap * d;
  tv_bf16* d_q = reinterpret_cast<tv_bf16*>(dptr(s.q));
  tv_bf16* d_kt = reinterpret_cast<tv_bf16*>(dptr(s.k_tree));
  tv_bf16* d_vt = reinterpret_cast<tv_bf16*>(dptr(s.v_tree));
  tv_bf16* d_out = reinterpret_cast<tv_bf16*>(dptr(s.out));
  for (int l = 0; l < L; ++l) {
    rc = tree_verify_attn(d_q + l * q_layer, a->k_cache + l * c_layer, a->v_cache + l * c_layer,
                          d_kt + l * t_layer, d_vt + l * t_layer, a->prefix_len, d_n_nodes, d_bits,
                          B, Nmax, Hq, Hkv, d, Scap, a->scale, d_out + l * q_layer, nullptr,
                          dptr(s.attn_ws), s.attn_ws_bytes, d_status, a->stream);
    if (rc != TV_OK) return rc;
  }
  int32_t* d_alen = reinterpret_cast<int32_t*>(dptr(s.accept_len));
  int32_t* d_acc = reinterpret_cast<int32_t*>(dptr(s.accepted));
  int32_t* d_next = reinterpret_cast<int32_t*>(dptr(s.next_token));
  rc = tree_accept(reinterpret_cast<tv_bf16*>(dptr(s.logits)), reinterpret_cast<int32_t*>(dptr(s.tokens)),
                   d_retrieve, d_n_nodes, B, Nmax, V, P, Dp1, reinterpret_cast<int32_t*>(dptr(s.argmax)),
                   nullptr, nullptr, d_alen, reinterpret_cast<int32_t*>(dptr(s.best_path)), d_acc, d_next,
                   dptr(s.accept_ws), s.accept_ws_bytes, d_status, a->stream);
  if (rc != TV_OK) return rc;
  rc = kv_commit(a->k_cache, a->v_cache, d_kt, d_vt, d_acc, d_alen, a->prefix_len, L, B, Nmax, Hkv, d, Scap, Dp1,
                 (int64_t)c_layer, (int64_t)t_layer, d_status, a->stream);
  if (rc != TV_OK) return rc;
  TV_CUDA_OK(cudaMemcpyAsync(a->out, d_out, sizeof(tv_bf16) * (size_t)L * q_layer, cudaMemcpyDeviceToHost, st));
  TV_CUDA_OK(cudaMemcpyAsync(a->accept_len, d_alen, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, st));
  TV_CUDA_OK(cudaMemcpyAsync(a->accepted_nodes, d_acc, sizeof(int32_t) * B * Dp1, cudaMemcpyDeviceToHost, st));
  TV_CUDA_OK(cudaMemcpyAsync(a->next_token, d_next, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, st));
  TV_CUDA_OK(cudaMemcpyAsync(a->status, d_status, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, st));
  TV_CUDA_OK(cudaStreamSynchronize(st));
  return TV_OK;
}
