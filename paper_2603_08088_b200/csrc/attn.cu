// tree_verify_attn entry point.
#include "common.cuh"

extern "C" TV_API int tv_debug_attn_simt(const tv_bf16* q, const tv_bf16* k_cache, const tv_bf16* v_cache,
                                  const tv_bf16* k_tree, const tv_bf16* v_tree,
                                  const int32_t* prefix_len, const int32_t* n_nodes,
                                  const uint32_t* anc_bits,
                                  int B, int Nmax, int Hq, int Hkv, int d, int Scap, float scale,
                                  tv_bf16* out, float* lse, tv_stream stream);

extern "C" size_t tv_attn_workspace_bytes(int B, int Nmax, int Hq, int Hkv, int d, int Scap) {
  (void)B; (void)Nmax; (void)Hq; (void)Hkv; (void)d; (void)Scap;
  return 256;
}

extern "C" int tree_verify_attn(const tv_bf16* q,
                                const tv_bf16* k_cache, const tv_bf16* v_cache,
                                const tv_bf16* k_tree, const tv_bf16* v_tree,
                                const int32_t* prefix_len, const int32_t* n_nodes,
                                const uint32_t* anc_bits,
                                int B, int Nmax, int Hq, int Hkv, int d, int Scap, float scale,
                                tv_bf16* out, float* lse,
                                void* workspace, size_t workspace_bytes,
                                int32_t* status, tv_stream stream) {
  TV_REQUIRE(status && workspace, "tree_verify_attn: NULL pointer");
  TV_REQUIRE(Nmax <= 128, "tree_verify_attn: Nmax must be <= 128");
  if (workspace_bytes < tv_attn_workspace_bytes(B, Nmax, Hq, Hkv, d, Scap))
    return tv::fail(TV_ERR_WORKSPACE, "tree_verify_attn: workspace too small");
  return tv_debug_attn_simt(q, k_cache, v_cache, k_tree, v_tree, prefix_len, n_nodes, anc_bits,
                            B, Nmax, Hq, Hkv, d, Scap, scale, out, lse, stream);
}
