/*
 * treeverify_debug.h - test and tuning aids exported by libtreeverify.so next
 * to the public interface of treeverify.h.  None of them is on the product
 * path: the library never calls them, the Python step never calls them; the
 * parity tests use the first as an on-device cross-check of the tensor-core
 * kernel and the second to see a bounded wait expire; bench.py uses the third
 * to time the kernel's memory side alone.
 */
#ifndef TREEVERIFY_DEBUG_H_
#define TREEVERIFY_DEBUG_H_

#include "treeverify.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * tree_verify_attn computed by a plain CUDA-core kernel (one warp per query
 * row, fp32 online softmax): same arguments and results, no workspace, no
 * status.  A second, independently written GPU implementation of Sections
 * 2.3 / 3.3 for cross-checks.
 */
TV_API int tv_debug_attn_simt(const tv_bf16* q, const tv_bf16* k_cache, const tv_bf16* v_cache,
                              const tv_bf16* k_tree, const tv_bf16* v_tree,
                              const int32_t* prefix_len, const int32_t* n_nodes, const uint32_t* anc_bits,
                              int B, int Nmax, int Hq, int Hkv, int d, int Scap, float scale,
                              tv_bf16* out, float* lse, tv_stream stream);

/*
 * tree_verify_attn with the limit of every bounded wait inside the kernel set
 * to wait_limit_ns (the product uses 2 s).  mode bit 0: the producer warp
 * issues no copy at all, so the first wait of the MMA-issuing warp expires.
 * mode bit 1: the pieces of units that are cut between CTAs store their
 * partials but never announce them, so the poll of the piece that merges
 * expires (a launch without a cut unit is then an ordinary launch).
 * The launch then ends by itself: every role leaves its loop, the tensor
 * memory is freed, and TV_ST_TIMEOUT is ORed into status[b] of every
 * sequence (out and lse are unspecified).  Nothing traps or faults; the next
 * launch on the device works as usual.  mode 0 is an ordinary launch.
 * (Section 4.3 of the paper, the failure dump on a runtime error, is the
 * nearest counterpart.)
 */
TV_API int tv_debug_attn_expire(const tv_bf16* q, const tv_bf16* k_cache, const tv_bf16* v_cache,
                                const tv_bf16* k_tree, const tv_bf16* v_tree,
                                const int32_t* prefix_len, const int32_t* n_nodes, const uint32_t* anc_bits,
                                int B, int Nmax, int Hq, int Hkv, int d, int Scap, float scale,
                                tv_bf16* out, float* lse, void* workspace, size_t workspace_bytes,
                                int32_t* status, unsigned long long wait_limit_ns, int mode, tv_stream stream);

/*
 * The K/V stream of tree_verify_attn_layers alone: the same launch, schedule
 * and TMA copies, but the warp that would issue the MMAs only hands every
 * shared-memory slot back as soon as its tile has landed, and no softmax
 * runs.  Nothing is computed and out is not written (it is only validated);
 * status is left alone unless a wait expires.  Timing it against the
 * algorithmic bytes of the call shows what the memory side of the kernel can
 * deliver, i.e. how much of the real launch's time is not memory.  The
 * arguments have the meaning they have in tree_verify_attn_layers; the
 * inputs must be stable while the kernel in front runs (the launch may start
 * reading them early).  The paper has no counterpart.
 */
TV_API int tv_debug_attn_stream_only(const tv_bf16* q, const tv_bf16* k_cache, const tv_bf16* v_cache,
                                     const tv_bf16* k_tree, const tv_bf16* v_tree,
                                     const int32_t* prefix_len, const int32_t* n_nodes, const uint32_t* anc_bits,
                                     int L, int B, int Nmax, int Hq, int Hkv, int d, int Scap,
                                     int64_t q_layer_stride, int64_t cache_layer_stride, int64_t tree_layer_stride,
                                     tv_bf16* out, int64_t out_layer_stride,
                                     void* workspace, size_t workspace_bytes, int32_t* status, tv_stream stream);

/*
 * Live only in a library built with -DTV_TRACE: while a device buffer of
 * 160 * 4 * 256 uint64 is registered here, every tree_verify_attn launch
 * records a per-CTA, per-role timeline (tag << 48 | globaltimer ns) into it.
 * NULL switches it off.
 */
TV_API void tv_debug_set_attn_trace(unsigned long long* device_buffer);

#ifdef __cplusplus
}
#endif
#endif /* TREEVERIFY_DEBUG_H_ */
