// tv_verify_step_host: one verification step driven from host buffers.
// Copies the per-step inputs into a caller-provided device staging area,
// enqueues the four calls of the step in the paper's order (tensorise + mask,
// attention per layer, gather + accept, commit; Section 3), copies the
// per-step results back and waits for the stream.  The KV cache and
// prefix_len are resident device state and are not copied.
//
// The step is bound by the host link (hundreds of MB each way), so the copies
// are pipelined against the kernels: an input stream feeds Q and the tree K/V
// layer by layer and the logits last, the caller's stream runs a layer as soon
// as its inputs have landed, and an output stream returns a layer's result as
// soon as it is complete, while later layers are still coming in (the link is
// full duplex).
#include "common.cuh"

#include <mutex>
#include <vector>

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

// Per-device copy streams and a growing pool of timing-free events, created on first use and kept.
struct Pipes {
  cudaStream_t in = nullptr, out = nullptr;
  std::vector<cudaEvent_t> events;
};

cudaError_t get_pipes(int n_events, Pipes** result) {
  static std::mutex mu;
  static Pipes pipes[64];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  Pipes& p = pipes[dev];
  if (!p.in) {
    if ((e = cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking)) != cudaSuccess) return e;
    if ((e = cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking)) != cudaSuccess) return e;
  }
  while ((int)p.events.size() < n_events) {
    cudaEvent_t ev;
    if ((e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming)) != cudaSuccess) return e;
    p.events.push_back(ev);
  }
  *result = &p;
  return cudaSuccess;
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
  // Everything the four calls below would refuse is refused here, before the first copy is queued: a call that
  // returns an error has then never touched the host buffers or the staging area.
  TV_REQUIRE(a->B <= 512 && a->Nmax <= 256 && (long long)a->B * a->Nmax <= 65535,
             "tv_verify_step_host: need B <= 512, Nmax <= 256, B * Nmax <= 65535");
  TV_REQUIRE(a->d == 64 || a->d == 128, "tv_verify_step_host: d must be 64 or 128");
  TV_REQUIRE(a->Hq >= 1 && a->Hkv >= 1 && a->Hq % a->Hkv == 0 && a->Hq / a->Hkv <= 128,
             "tv_verify_step_host: need Hq %% Hkv == 0 and Hq / Hkv <= 128");
  TV_REQUIRE(a->Scap >= 1 && a->scale > 0.f && a->L <= 65535 && a->Dp1 <= 1024,
             "tv_verify_step_host: need Scap >= 1, scale > 0, L <= 65535, Dp1 <= 1024");
  TV_REQUIRE((long long)a->B * a->Hkv * ((a->Scap + 127) / 128 + 8) < (1ll << 31),
             "tv_verify_step_host: B * Hkv * Scap is too large for the attention's tile scheduler");
  TV_REQUIRE(tv::aligned16(a->k_cache) && tv::aligned16(a->v_cache), "tv_verify_step_host: the caches must be 16-byte aligned");
  const int L = a->L, B = a->B, Nmax = a->Nmax, Hq = a->Hq, Hkv = a->Hkv, d = a->d, Scap = a->Scap, V = a->V,
            P = a->P, Dp1 = a->Dp1;
  const Staging s = layout(L, B, Nmax, Hq, Hkv, d, Scap, V, P, Dp1);
  if (a->staging_bytes < s.total)
    return tv::fail(TV_ERR_WORKSPACE, "tv_verify_step_host: staging of %zu bytes, need %zu", a->staging_bytes, s.total);
  char* base = static_cast<char*>(a->staging);
  cudaStream_t st = (cudaStream_t)a->stream;
  auto dptr = [&](size_t off) { return base + off; };
  // events: 0 entry, 1 small inputs in, 2 logits in, 3 step done, 4 results out, 5 + l layer inputs in,
  // 5 + L + l layer computed.  One call at a time per device uses them (the call is synchronous).
  Pipes* pp = nullptr;
  TV_CUDA_OK(get_pipes(5 + 2 * L, &pp));
  cudaStream_t s_in = pp->in, s_out = pp->out;
  cudaEvent_t* ev = pp->events.data();
  // From here on copies are in flight on the two private streams: if anything fails further down, the three
  // streams are drained before the error is returned, so that the caller may free or reuse its buffers at once.
  auto body = [&]() -> int {
  // work already queued on the caller's stream may still use the staging area and the host buffers
  TV_CUDA_OK(cudaEventRecord(ev[0], st));
  TV_CUDA_OK(cudaStreamWaitEvent(s_in, ev[0], 0));
  TV_CUDA_OK(cudaStreamWaitEvent(s_out, ev[0], 0));
  const size_t q_layer = (size_t)B * Nmax * Hq * d, t_layer = (size_t)B * Nmax * Hkv * d,
               c_layer = (size_t)B * Hkv * Scap * d;
  tv_bf16* d_q = reinterpret_cast<tv_bf16*>(dptr(s.q));
  tv_bf16* d_kt = reinterpret_cast<tv_bf16*>(dptr(s.k_tree));
  tv_bf16* d_vt = reinterpret_cast<tv_bf16*>(dptr(s.v_tree));
  tv_bf16* d_out = reinterpret_cast<tv_bf16*>(dptr(s.out));
#define TV_H2D(field, off, bytes) TV_CUDA_OK(cudaMemcpyAsync(dptr(off), a->field, (bytes), cudaMemcpyHostToDevice, s_in))
  TV_H2D(parent, s.parent, sizeof(int32_t) * B * Nmax);
  TV_H2D(n_nodes, s.n_nodes, sizeof(int32_t) * B);
  TV_H2D(tokens, s.tokens, sizeof(int32_t) * B * Nmax);
  if (a->retrieve_indices) TV_H2D(retrieve_indices, s.retrieve, sizeof(int32_t) * B * P * Dp1);
#undef TV_H2D
  TV_CUDA_OK(cudaEventRecord(ev[1], s_in));
  for (int l = 0; l < L; ++l) {
    TV_CUDA_OK(cudaMemcpyAsync(d_q + l * q_layer, a->q + l * q_layer, sizeof(tv_bf16) * q_layer, cudaMemcpyHostToDevice, s_in));
    TV_CUDA_OK(cudaMemcpyAsync(d_kt + l * t_layer, a->k_tree + l * t_layer, sizeof(tv_bf16) * t_layer, cudaMemcpyHostToDevice, s_in));
    TV_CUDA_OK(cudaMemcpyAsync(d_vt + l * t_layer, a->v_tree + l * t_layer, sizeof(tv_bf16) * t_layer, cudaMemcpyHostToDevice, s_in));
    TV_CUDA_OK(cudaEventRecord(ev[5 + l], s_in));
  }
  TV_CUDA_OK(cudaMemcpyAsync(dptr(s.logits), a->logits, sizeof(tv_bf16) * (size_t)B * Nmax * V, cudaMemcpyHostToDevice, s_in));
  TV_CUDA_OK(cudaEventRecord(ev[2], s_in));

  int32_t* d_n_nodes = reinterpret_cast<int32_t*>(dptr(s.n_nodes));
  int32_t* d_status = reinterpret_cast<int32_t*>(dptr(s.status));
  int32_t* d_retrieve = reinterpret_cast<int32_t*>(dptr(s.retrieve));
  uint32_t* d_bits = reinterpret_cast<uint32_t*>(dptr(s.anc_bits));
  TV_CUDA_OK(cudaStreamWaitEvent(st, ev[1], 0));
  int rc = tree_build_mask(reinterpret_cast<int32_t*>(dptr(s.parent)), d_n_nodes, B, Nmax, Dp1 - 1, P, d_bits,
                           nullptr, nullptr, nullptr, a->retrieve_indices ? nullptr : d_retrieve,
                           reinterpret_cast<int32_t*>(dptr(s.n_paths)), d_status, a->stream);
  if (rc != TV_OK) return rc;
  for (int l = 0; l < L; ++l) {
    TV_CUDA_OK(cudaStreamWaitEvent(st, ev[5 + l], 0));
    rc = tree_verify_attn(d_q + l * q_layer, a->k_cache + l * c_layer, a->v_cache + l * c_layer,
                          d_kt + l * t_layer, d_vt + l * t_layer, a->prefix_len, d_n_nodes, d_bits,
                          B, Nmax, Hq, Hkv, d, Scap, a->scale, d_out + l * q_layer, nullptr,
                          dptr(s.attn_ws), s.attn_ws_bytes, d_status, a->stream);
    if (rc != TV_OK) return rc;
    TV_CUDA_OK(cudaEventRecord(ev[5 + L + l], st));
    TV_CUDA_OK(cudaStreamWaitEvent(s_out, ev[5 + L + l], 0));
    TV_CUDA_OK(cudaMemcpyAsync(a->out + l * q_layer, d_out + l * q_layer, sizeof(tv_bf16) * q_layer, cudaMemcpyDeviceToHost, s_out));
  }
  int32_t* d_alen = reinterpret_cast<int32_t*>(dptr(s.accept_len));
  int32_t* d_acc = reinterpret_cast<int32_t*>(dptr(s.accepted));
  int32_t* d_next = reinterpret_cast<int32_t*>(dptr(s.next_token));
  TV_CUDA_OK(cudaStreamWaitEvent(st, ev[2], 0));
  rc = tree_accept(reinterpret_cast<tv_bf16*>(dptr(s.logits)), reinterpret_cast<int32_t*>(dptr(s.tokens)),
                   d_retrieve, d_n_nodes, B, Nmax, V, P, Dp1, reinterpret_cast<int32_t*>(dptr(s.argmax)),
                   nullptr, nullptr, d_alen, reinterpret_cast<int32_t*>(dptr(s.best_path)), d_acc, d_next,
                   dptr(s.accept_ws), s.accept_ws_bytes, d_status, a->stream);
  if (rc != TV_OK) return rc;
  rc = kv_commit(a->k_cache, a->v_cache, d_kt, d_vt, d_acc, d_alen, a->prefix_len, L, B, Nmax, Hkv, d, Scap, Dp1,
                 (int64_t)c_layer, (int64_t)t_layer, d_status, a->stream);
  if (rc != TV_OK) return rc;
  TV_CUDA_OK(cudaEventRecord(ev[3], st));
  TV_CUDA_OK(cudaStreamWaitEvent(s_out, ev[3], 0));
  TV_CUDA_OK(cudaMemcpyAsync(a->accept_len, d_alen, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, s_out));
  TV_CUDA_OK(cudaMemcpyAsync(a->accepted_nodes, d_acc, sizeof(int32_t) * B * Dp1, cudaMemcpyDeviceToHost, s_out));
  TV_CUDA_OK(cudaMemcpyAsync(a->next_token, d_next, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, s_out));
  TV_CUDA_OK(cudaMemcpyAsync(a->status, d_status, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, s_out));
  TV_CUDA_OK(cudaEventRecord(ev[4], s_out));
  TV_CUDA_OK(cudaStreamWaitEvent(st, ev[4], 0));
  TV_CUDA_OK(cudaStreamSynchronize(st));
  return TV_OK;
  };
  const int rc_step = body();
  if (rc_step != TV_OK) {
    cudaStreamSynchronize(s_in);
    cudaStreamSynchronize(s_out);
    cudaStreamSynchronize(st);
  }
  return rc_step;
}
