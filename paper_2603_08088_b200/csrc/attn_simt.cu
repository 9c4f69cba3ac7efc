// A plain CUDA-core tree-attention kernel: one warp per (node, query head)
// row, 32 keys per step, fp32 online softmax.  It exists as an on-device
// cross-check for the tensor-core kernel (tv_debug_attn_simt); it is not the
// fast path.  Same semantics as tree_verify_attn: prefix rows [0, S_b) are
// all visible, tree key j is visible to node i iff bit j of anc_bits[b,i] is
// set, padded rows give 0 / -inf, rows past the prefix and padded tree slots
// are never multiplied in (their V rows are staged as zeros).
#include "common.cuh"
#include "treeverify_debug.h"

#include <cuda_bf16.h>

namespace {

constexpr int kWarps = 8;
constexpr int kTile = 32;

template <int D>
__global__ void __launch_bounds__(kWarps * 32)
attn_simt_kernel(const tv_bf16* __restrict__ q, const tv_bf16* __restrict__ k_cache,
                 const tv_bf16* __restrict__ v_cache, const tv_bf16* __restrict__ k_tree,
                 const tv_bf16* __restrict__ v_tree, const int32_t* __restrict__ prefix_len,
                 const int32_t* __restrict__ n_nodes, const uint32_t* __restrict__ anc_bits,
                 int Nmax, int Hq, int Hkv, int Scap, float scale,
                 tv_bf16* __restrict__ out, float* __restrict__ lse) {
  constexpr int KW = D / 2 + 1;                       // padded K row stride in 32-bit words
  constexpr int E = D / 32;                           // output dims per lane
  __shared__ uint32_t ks[kTile * KW];
  __shared__ __align__(16) uint32_t vs[kTile * D / 2];
  __shared__ float qs[kWarps][D];

  const int G = Hq / Hkv;
  const int W = (Nmax + 31) / 32;
  const int b = blockIdx.y / Hkv, hk = blockIdx.y % Hkv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = blockIdx.x * kWarps + warp;           // packed row: node * G + group member
  const int node = r / G, h = hk * G + (r % G);
  int n = n_nodes[b];
  n = n < 0 ? 0 : (n > Nmax ? Nmax : n);
  int S = prefix_len[b];
  S = S < 0 ? 0 : (S > Scap ? Scap : S);
  const bool row_exists = node < Nmax;
  const bool row_valid = node < n;

  if (row_exists) {
    const tv_bf16* qrow = q + (((size_t)b * Nmax + node) * Hq + h) * D;
    for (int c = lane; c < D; c += 32) qs[warp][c] = __uint_as_float((uint32_t)qrow[c] << 16);
  }
  float m = -INFINITY, l = 0.f;
  float acc[E];
#pragma unroll
  for (int e = 0; e < E; ++e) acc[e] = 0.f;

  const int prefix_tiles = (S + kTile - 1) / kTile;
  const int tree_tiles = (Nmax + kTile - 1) / kTile;
  const uint4* kc = reinterpret_cast<const uint4*>(k_cache + ((size_t)b * Hkv + hk) * Scap * D);
  const uint4* vc = reinterpret_cast<const uint4*>(v_cache + ((size_t)b * Hkv + hk) * Scap * D);
  constexpr int VPR = D / 8;                           // uint4 per row

  for (int t = 0; t < prefix_tiles + tree_tiles; ++t) {
    const bool in_tree = t >= prefix_tiles;
    const int key0 = in_tree ? (t - prefix_tiles) * kTile : t * kTile;
    const int limit = in_tree ? n : S;
    __syncthreads();
    for (int idx = threadIdx.x; idx < kTile * VPR; idx += kWarps * 32) {
      const int j = idx / VPR, c = idx - j * VPR;
      const int key = key0 + j;
      uint4 kk = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
      if (key < limit) {
        if (in_tree) {
          const size_t off = (((size_t)b * Nmax + key) * Hkv + hk) * VPR + c;
          kk = reinterpret_cast<const uint4*>(k_tree)[off];
          vv = reinterpret_cast<const uint4*>(v_tree)[off];
        } else {
          kk = kc[(size_t)key * VPR + c];
          vv = vc[(size_t)key * VPR + c];
        }
      }
      uint32_t* kd = ks + j * KW + c * 4;
      kd[0] = kk.x; kd[1] = kk.y; kd[2] = kk.z; kd[3] = kk.w;
      reinterpret_cast<uint4*>(vs)[idx] = vv;
    }
    __syncthreads();
    if (!row_valid) continue;

    const int key = key0 + lane;
    bool visible = key < limit;
    if (in_tree && visible)
      visible = (anc_bits[((size_t)b * Nmax + node) * W + (key >> 5)] >> (key & 31)) & 1u;
    float dot = 0.f;
    const uint32_t* krow = ks + lane * KW;
#pragma unroll 8
    for (int w = 0; w < D / 2; ++w) {
      const uint32_t kk = krow[w];
      dot = fmaf(qs[warp][2 * w], __uint_as_float(kk << 16), dot);
      dot = fmaf(qs[warp][2 * w + 1], __uint_as_float(kk & 0xffff0000u), dot);
    }
    const float s = visible ? dot * scale : -INFINITY;
    float tmax = s;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, off));
    const float m_new = fmaxf(m, tmax);
    if (m_new == -INFINITY) continue;                   // nothing visible yet (warp-uniform)
    const float p = visible ? __expf(s - m_new) : 0.f;
    const float alpha = (m == -INFINITY) ? 0.f : __expf(m - m_new);
    float psum = p;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, off);
    l = l * alpha + psum;
    m = m_new;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] *= alpha;
    for (int j = 0; j < kTile; ++j) {
      const float pj = __shfl_sync(0xffffffffu, p, j);
      const uint32_t* vrow = vs + j * (D / 2) + lane * (E / 2);
#pragma unroll
      for (int e = 0; e < E / 2; ++e) {
        const uint32_t vv = vrow[e];
        acc[2 * e] = fmaf(pj, __uint_as_float(vv << 16), acc[2 * e]);
        acc[2 * e + 1] = fmaf(pj, __uint_as_float(vv & 0xffff0000u), acc[2 * e + 1]);
      }
    }
  }

  if (!row_exists) return;
  tv_bf16* orow = out + (((size_t)b * Nmax + node) * Hq + h) * D + lane * E;
  const float inv = (row_valid && l > 0.f) ? 1.f / l : 0.f;
#pragma unroll
  for (int e = 0; e < E; e += 2) {
    __nv_bfloat162 pk = __floats2bfloat162_rn(acc[e] * inv, acc[e + 1] * inv);
    *reinterpret_cast<__nv_bfloat162*>(orow + e) = pk;
  }
  if (lse && lane == 0)
    lse[((size_t)b * Hq + h) * Nmax + node] = (row_valid && l > 0.f) ? m + logf(l) : -INFINITY;
}

}  // namespace

// Same arguments as tree_verify_attn without the workspace.  Debug / cross-check only.
extern "C" TV_API int tv_debug_attn_simt(const tv_bf16* q, const tv_bf16* k_cache, const tv_bf16* v_cache,
                                  const tv_bf16* k_tree, const tv_bf16* v_tree,
                                  const int32_t* prefix_len, const int32_t* n_nodes,
                                  const uint32_t* anc_bits,
                                  int B, int Nmax, int Hq, int Hkv, int d, int Scap, float scale,
                                  tv_bf16* out, float* lse, tv_stream stream) {
  TV_REQUIRE(q && k_cache && v_cache && k_tree && v_tree && prefix_len && n_nodes && anc_bits && out,
             "tv_debug_attn_simt: NULL pointer");
  TV_REQUIRE(B >= 0 && Nmax >= 1 && Hq >= 1 && Hkv >= 1 && Hq % Hkv == 0 && Scap >= 1 && (d == 64 || d == 128),
             "tv_debug_attn_simt: bad dimension");
  TV_REQUIRE(tv::aligned16(q) && tv::aligned16(k_cache) && tv::aligned16(v_cache) && tv::aligned16(k_tree) &&
                 tv::aligned16(v_tree) && tv::aligned16(out),
             "tv_debug_attn_simt: tensors must be 16-byte aligned");
  if (B == 0) return TV_OK;
  const int R = Nmax * (Hq / Hkv);
  dim3 grid((R + kWarps - 1) / kWarps, B * Hkv);
  cudaStream_t s = (cudaStream_t)stream;
  if (d == 128)
    attn_simt_kernel<128><<<grid, kWarps * 32, 0, s>>>(q, k_cache, v_cache, k_tree, v_tree, prefix_len, n_nodes,
                                                       anc_bits, Nmax, Hq, Hkv, Scap, scale, out, lse);
  else
    attn_simt_kernel<64><<<grid, kWarps * 32, 0, s>>>(q, k_cache, v_cache, k_tree, v_tree, prefix_len, n_nodes,
                                                      anc_bits, Nmax, Hq, Hkv, Scap, scale, out, lse);
  TV_CUDA_OK(cudaGetLastError());
  tv::count_launches(1);
  return TV_OK;
}
