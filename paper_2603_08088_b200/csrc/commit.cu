// kv_commit: path-index commit with the prefix-sharing fast reorder
// (Section 3.1).  The committed prefix is never moved; the accepted nodes' K/V
// rows are gathered from the tree ("branch") buffers and appended behind it,
// for every layer and KV head, in one launch.  A second one-warp launch then
// advances prefix_len, so no copy CTA can observe the updated length.
//
// Each (layer, sequence, accepted slot) is one CTA; a thread moves 16 bytes,
// so a head row of d bf16 is written by d/8 adjacent threads (coalesced on
// both sides: the source row [node, h, :] and the destination row [h, S+j, :]).
#include "common.cuh"

namespace {

// Decides, identically in both kernels, whether sequence b commits.
// Returns the status bits to raise (0 = commit).
__device__ __forceinline__ int commit_check(const int32_t* accepted_nodes, int A, int S, int st_in,
                                            int Nmax, int Scap, int Dp1, int b) {
  if (st_in & tv::kFatalStatus) return -1;            // skipped, nothing new to report
  if (A < 0 || A >= Dp1) return TV_ST_BAD_INDEX;
  for (int j = 0; j <= A; ++j) {
    const int node = accepted_nodes[(size_t)b * Dp1 + j];
    if (node < 0 || node >= Nmax) return TV_ST_BAD_INDEX;
  }
  if (S < 0 || S + A + 1 > Scap) return TV_ST_CAPACITY;
  return 0;
}

__global__ void __launch_bounds__(256)
commit_copy_kernel(uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                   const uint4* __restrict__ k_tree, const uint4* __restrict__ v_tree,
                   const int32_t* __restrict__ accepted_nodes, const int32_t* __restrict__ accept_len,
                   const int32_t* __restrict__ prefix_len, const int32_t* __restrict__ status,
                   int B, int Nmax, int Hkv, int dvec, int Scap, int Dp1,
                   int64_t cache_layer_vec, int64_t tree_layer_vec) {
  const int j = blockIdx.x, b = blockIdx.y, l = blockIdx.z;
  const int A = accept_len[b];
  if (j > A) return;
  const int S = prefix_len[b];
  if (commit_check(accepted_nodes, A, S, status[b], Nmax, Scap, Dp1, b) != 0) return;
  const int node = accepted_nodes[(size_t)b * Dp1 + j];
  const size_t src = (size_t)l * tree_layer_vec + ((size_t)b * Nmax + node) * Hkv * dvec;          // [node, h, :]
  const size_t dst = (size_t)l * cache_layer_vec + ((size_t)b * Hkv * Scap + (size_t)(S + j)) * dvec;  // [h=0, S+j, :]
  const int per = Hkv * dvec;
  for (int t = threadIdx.x; t < 2 * per; t += blockDim.x) {
    const int kv = t >= per;
    const int u = kv ? t - per : t;
    const int h = u / dvec, c = u - h * dvec;
    const uint4 val = kv ? v_tree[src + u] : k_tree[src + u];
    uint4* out = kv ? v_cache : k_cache;
    out[dst + (size_t)h * Scap * dvec + c] = val;
  }
}

__global__ void commit_finish_kernel(const int32_t* __restrict__ accepted_nodes,
                                     const int32_t* __restrict__ accept_len,
                                     int32_t* __restrict__ prefix_len, int32_t* __restrict__ status,
                                     int B, int Nmax, int Scap, int Dp1) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int A = accept_len[b];
  const int S = prefix_len[b];
  const int r = commit_check(accepted_nodes, A, S, status[b], Nmax, Scap, Dp1, b);
  if (r == 0) prefix_len[b] = S + A + 1;
  else if (r > 0) status[b] |= r;
}

}  // namespace

extern "C" int kv_commit(tv_bf16* k_cache, tv_bf16* v_cache,
                         const tv_bf16* k_tree, const tv_bf16* v_tree,
                         const int32_t* accepted_nodes, const int32_t* accept_len,
                         int32_t* prefix_len,
                         int L, int B, int Nmax, int Hkv, int d, int Scap, int Dp1,
                         int64_t cache_layer_stride, int64_t tree_layer_stride,
                         int32_t* status, tv_stream stream) {
  TV_REQUIRE(k_cache && v_cache && k_tree && v_tree && accepted_nodes && accept_len && prefix_len && status,
             "kv_commit: NULL pointer");
  TV_REQUIRE(L >= 0 && B >= 0 && Nmax >= 1 && Hkv >= 1 && d >= 8 && Scap >= 1 && Dp1 >= 1,
             "kv_commit: bad dimension");
  TV_REQUIRE(d % 8 == 0, "kv_commit: d must be a multiple of 8 (16-byte rows)");
  TV_REQUIRE(cache_layer_stride % 8 == 0 && tree_layer_stride % 8 == 0, "kv_commit: layer strides must be multiples of 8 elements");
  TV_REQUIRE(tv::aligned16(k_cache) && tv::aligned16(v_cache) && tv::aligned16(k_tree) && tv::aligned16(v_tree),
             "kv_commit: tensors must be 16-byte aligned");
  TV_REQUIRE(B <= 65535 && L <= 65535, "kv_commit: B and L must be <= 65535");
  if (L == 0 || B == 0) return TV_OK;
  const int dvec = d / 8;
  cudaStream_t s = (cudaStream_t)stream;
  int threads = 2 * Hkv * dvec;
  threads = threads > 256 ? 256 : ((threads + 31) / 32) * 32;
  commit_copy_kernel<<<dim3(Dp1, B, L), threads, 0, s>>>(
      reinterpret_cast<uint4*>(k_cache), reinterpret_cast<uint4*>(v_cache),
      reinterpret_cast<const uint4*>(k_tree), reinterpret_cast<const uint4*>(v_tree),
      accepted_nodes, accept_len, prefix_len, status, B, Nmax, Hkv, dvec, Scap, Dp1,
      cache_layer_stride / 8, tree_layer_stride / 8);
  TV_CUDA_OK(cudaGetLastError());
  commit_finish_kernel<<<(B + 127) / 128, 128, 0, s>>>(accepted_nodes, accept_len, prefix_len, status,
                                                       B, Nmax, Scap, Dp1);
  TV_CUDA_OK(cudaGetLastError());
  tv::count_launches(2);
  return TV_OK;
}
