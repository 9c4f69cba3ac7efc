// kv_commit: path-index commit with the prefix-sharing fast reorder
// (Section 3.1).  The committed prefix is never moved; the accepted nodes' K/V
// rows are gathered from the tree ("branch") buffers and appended behind it,
// for every layer and KV head, in one launch.  A second one-warp launch then
// advances prefix_len, so no copy CTA can observe the updated length.
//
// Each (layer, sequence) is one CTA; a thread moves 16 bytes at a time, so a
// head row of d bf16 is written by d/8 adjacent threads (coalesced on both
// sides: the source row [node, h, :] and the destination row [h, S+j, :]).
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

// One CTA per (layer, sequence): the per-sequence scalars and the node list are fetched together and validated by
// all threads at once (the same decision as commit_check), then the CTA moves every 16-byte piece of the accepted
// segment, K and V, all heads; the pieces of a row are adjacent threads on both sides.
constexpr int kCopyThreads = 256;
constexpr int kCopyMaxDp1 = 1024;

__global__ void __launch_bounds__(kCopyThreads)
commit_copy_kernel(uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                   const uint4* __restrict__ k_tree, const uint4* __restrict__ v_tree,
                   const int32_t* __restrict__ accepted_nodes, const int32_t* __restrict__ accept_len,
                   const int32_t* __restrict__ prefix_len, const int32_t* __restrict__ status,
                   int B, int Nmax, int Hkv, int dvec, int Scap, int Dp1,
                   int64_t cache_layer_vec, int64_t tree_layer_vec) {
  tv::pdl_enter();
  __shared__ int s_nodes[kCopyMaxDp1];
  const int b = blockIdx.x, l = blockIdx.y;
  const int A = accept_len[b];
  const int S = prefix_len[b];
  const int st = status[b];
  for (int j = threadIdx.x; j < Dp1; j += kCopyThreads) s_nodes[j] = accepted_nodes[(size_t)b * Dp1 + j];
  int bad = (st & tv::kFatalStatus) || A < 0 || A >= Dp1 || S < 0 || S + A + 1 > Scap;
  __syncthreads();
  if (!bad)
    for (int j = threadIdx.x; j <= A; j += kCopyThreads) bad |= (s_nodes[j] < 0 || s_nodes[j] >= Nmax);
  if (__syncthreads_or(bad)) return;
  const size_t src0 = (size_t)l * tree_layer_vec + (size_t)b * Nmax * Hkv * dvec;       // [node, h, :]
  const size_t dst0 = (size_t)l * cache_layer_vec + (size_t)b * Hkv * Scap * dvec;      // [h, row, :]
  const int per = Hkv * dvec;                   // pieces of one node's row over all heads
  const int total = 2 * (A + 1) * per;
  // four pieces per thread and round: the loads of a round are all issued before the first store
  for (int t0 = threadIdx.x; t0 < total; t0 += 4 * kCopyThreads) {
    uint4 val[4];
    uint4* dst[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int t = t0 + i * kCopyThreads;
      dst[i] = nullptr;
      if (t < total) {
        const int kv = t >= (A + 1) * per;
        const int u = kv ? t - (A + 1) * per : t;
        const int j = u / per, w = u - j * per;
        const int h = w / dvec, c = w - h * dvec;
        val[i] = (kv ? v_tree : k_tree)[src0 + (size_t)s_nodes[j] * per + w];
        dst[i] = (kv ? v_cache : k_cache) + dst0 + ((size_t)h * Scap + S + j) * dvec + c;
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (dst[i]) *dst[i] = val[i];
  }
}

__global__ void commit_finish_kernel(const int32_t* __restrict__ accepted_nodes,
                                     const int32_t* __restrict__ accept_len,
                                     int32_t* __restrict__ prefix_len, int32_t* __restrict__ status,
                                     int B, int Nmax, int Scap, int Dp1) {
  // This kernel writes prefix_len, which a tree_verify_attn launch directly behind it reads before its own
  // wait: the next launch must not start until this grid is complete, so nothing is released early here.
  tv::pdl_wait_only();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int A = accept_len[b];
  const int S = prefix_len[b];
  const int r = commit_check(accepted_nodes, A, S, status[b], Nmax, Scap, Dp1, b);
  if (r == 0) prefix_len[b] = S + A + 1;
  else if (r > 0) status[b] |= r;
}

// In-cache layout: the tree's K/V rows were written into the cache itself, node i at row S + i, and the commit
// reorders them in place: row S + j takes the old row S + accepted_nodes[j], j = 0..A.  Source and destination
// ranges overlap (a row can be the source of one slot and the destination of another), so the copy is a gather
// from the state BEFORE the commit: one CTA owns all the rows of a (layer, sequence, KV head, K or V), reads
// every row it needs into registers, and only writes after a barrier.
constexpr int kInplaceThreads = 256;
constexpr int kInplaceMaxPerThread = 8;
constexpr int kInplaceMaxPieces = kInplaceThreads * kInplaceMaxPerThread;

// One CTA per (layer, sequence, K or V, group of `hpc` KV heads).  The per-sequence scalars and the node list are
// fetched together (one round trip), validated by all threads at once, and then every 16-byte piece of the
// accepted segments of the CTA's heads is read, a barrier passes, and the pieces that move are written.
__global__ void __launch_bounds__(kInplaceThreads)
commit_inplace_kernel(uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                      const int32_t* __restrict__ accepted_nodes, const int32_t* __restrict__ accept_len,
                      const int32_t* __restrict__ prefix_len, const int32_t* __restrict__ status,
                      int B, int Nmax, int Hkv, int dvec, int Scap, int Dp1, int hpc, int64_t cache_layer_vec) {
  __shared__ int s_nodes[kInplaceMaxPieces];
  const int kv = blockIdx.x & 1, h0 = (blockIdx.x >> 1) * hpc, b = blockIdx.y, l = blockIdx.z;
  const int A = accept_len[b];
  const int S = prefix_len[b];
  const int st = status[b];
  for (int j = threadIdx.x; j < Dp1; j += kInplaceThreads) s_nodes[j] = accepted_nodes[(size_t)b * Dp1 + j];
  // the same decision as commit_check plus the source-row bound, taken by all threads together
  int bad = (st & tv::kFatalStatus) || A < 0 || A >= Dp1 || S < 0 || S + A + 1 > Scap;
  __syncthreads();
  if (!bad)
    for (int j = threadIdx.x; j <= A; j += kInplaceThreads) {
      const int node = s_nodes[j];
      bad |= (node < 0 || node >= Nmax || S + node >= Scap);
    }
  if (__syncthreads_or(bad)) return;
  uint4* base = (kv ? v_cache : k_cache) + (size_t)l * cache_layer_vec + ((size_t)b * Hkv + h0) * (size_t)Scap * dvec;
  const int per_head = (A + 1) * dvec;           // 16-byte pieces of one head's accepted segment
  const int total = hpc * per_head;
  uint4 held[kInplaceMaxPerThread];
#pragma unroll
  for (int i = 0; i < kInplaceMaxPerThread; ++i) {
    const int t = threadIdx.x + i * kInplaceThreads;
    if (t < total) {
      const int h = t / per_head, u = t - h * per_head;
      const int j = u / dvec, c = u - j * dvec;
      held[i] = base[((size_t)h * Scap + S + s_nodes[j]) * dvec + c];
    }
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < kInplaceMaxPerThread; ++i) {
    const int t = threadIdx.x + i * kInplaceThreads;
    if (t < total) {
      const int h = t / per_head, u = t - h * per_head;
      const int j = u / dvec, c = u - j * dvec;
      if (s_nodes[j] != j) base[((size_t)h * Scap + S + j) * dvec + c] = held[i];
    }
  }
}

// prefix_len and status of the in-place commit (after every copy CTA has finished)
__global__ void commit_inplace_finish_kernel(const int32_t* __restrict__ accepted_nodes,
                                             const int32_t* __restrict__ accept_len,
                                             int32_t* __restrict__ prefix_len, int32_t* __restrict__ status,
                                             int B, int Nmax, int Scap, int Dp1) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int A = accept_len[b];
  const int S = prefix_len[b];
  int r = commit_check(accepted_nodes, A, S, status[b], Nmax, Scap, Dp1, b);
  if (r == 0)
    for (int j = 0; j <= A; ++j)
      if (S + accepted_nodes[(size_t)b * Dp1 + j] >= Scap) r = TV_ST_CAPACITY;     // a source row outside the cache
  if (r == 0) prefix_len[b] = S + A + 1;
  else if (r > 0) status[b] |= r;
}

// Paged cache: pages [n_pages,Hkv,128,d] per layer, block_table[b, t] = page of rows 128 t .. 128 t + 127 of
// sequence b.  Row S + j of the sequence is row (S + j) % 128 of page block_table[b, (S + j) / 128].
constexpr int kPageRows = 128;

__device__ __forceinline__ bool paged_segment_ok(const int32_t* block_table, int b, int S, int A, int max_blocks,
                                                 int n_pages) {
  for (int t = S / kPageRows; t <= (S + A) / kPageRows; ++t) {
    const int pg = block_table[(size_t)b * max_blocks + t];
    if (pg < 0 || pg >= n_pages) return false;
  }
  return true;
}

__global__ void __launch_bounds__(kCopyThreads)
commit_paged_kernel(uint4* __restrict__ k_pages, uint4* __restrict__ v_pages, const int32_t* __restrict__ block_table,
                    const uint4* __restrict__ k_tree, const uint4* __restrict__ v_tree,
                    const int32_t* __restrict__ accepted_nodes, const int32_t* __restrict__ accept_len,
                    const int32_t* __restrict__ prefix_len, const int32_t* __restrict__ status,
                    int B, int Nmax, int Hkv, int dvec, int n_pages, int max_blocks, int Dp1,
                    int64_t page_layer_vec, int64_t tree_layer_vec) {
  __shared__ int s_nodes[kCopyMaxDp1];
  const int b = blockIdx.x, l = blockIdx.y;
  const int A = accept_len[b];
  const int S = prefix_len[b];
  const int st = status[b];
  for (int j = threadIdx.x; j < Dp1; j += kCopyThreads) s_nodes[j] = accepted_nodes[(size_t)b * Dp1 + j];
  int bad = (st & tv::kFatalStatus) || A < 0 || A >= Dp1 || S < 0 || S + A + 1 > max_blocks * kPageRows;
  __syncthreads();
  if (!bad) {
    for (int j = threadIdx.x; j <= A; j += kCopyThreads) bad |= (s_nodes[j] < 0 || s_nodes[j] >= Nmax);
    if (threadIdx.x == 0) bad |= !paged_segment_ok(block_table, b, S, A, max_blocks, n_pages);
  }
  if (__syncthreads_or(bad)) return;
  const size_t src0 = (size_t)l * tree_layer_vec + (size_t)b * Nmax * Hkv * dvec;       // [node, h, :]
  const size_t dst0 = (size_t)l * page_layer_vec;                                       // [page, h, row, :]
  const int per = Hkv * dvec;
  const int total = 2 * (A + 1) * per;
  for (int t = threadIdx.x; t < total; t += kCopyThreads) {
    const int kv = t >= (A + 1) * per;
    const int u = kv ? t - (A + 1) * per : t;
    const int j = u / per, w = u - j * per;
    const int h = w / dvec, c = w - h * dvec;
    const int row = S + j;
    const int pg = block_table[(size_t)b * max_blocks + row / kPageRows];
    const uint4 val = (kv ? v_tree : k_tree)[src0 + (size_t)s_nodes[j] * per + w];
    (kv ? v_pages : k_pages)[dst0 + (((size_t)pg * Hkv + h) * kPageRows + row % kPageRows) * dvec + c] = val;
  }
}

__global__ void commit_paged_finish_kernel(const int32_t* __restrict__ accepted_nodes,
                                           const int32_t* __restrict__ accept_len,
                                           const int32_t* __restrict__ block_table,
                                           int32_t* __restrict__ prefix_len, int32_t* __restrict__ status,
                                           int B, int Nmax, int n_pages, int max_blocks, int Dp1) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int A = accept_len[b];
  const int S = prefix_len[b];
  int r = commit_check(accepted_nodes, A, S, status[b], Nmax, max_blocks * kPageRows, Dp1, b);
  if (r == 0 && !paged_segment_ok(block_table, b, S, A, max_blocks, n_pages)) r = TV_ST_BAD_INDEX;
  if (r == 0) prefix_len[b] = S + A + 1;
  else if (r > 0) status[b] |= r;
}

}  // namespace

extern "C" int kv_commit_paged(tv_bf16* k_pages, tv_bf16* v_pages, const int32_t* block_table,
                               const tv_bf16* k_tree, const tv_bf16* v_tree,
                               const int32_t* accepted_nodes, const int32_t* accept_len,
                               int32_t* prefix_len,
                               int L, int B, int Nmax, int Hkv, int d, int n_pages, int max_blocks, int Dp1,
                               int64_t page_layer_stride, int64_t tree_layer_stride,
                               int32_t* status, tv_stream stream) {
  TV_REQUIRE(k_pages && v_pages && block_table && k_tree && v_tree && accepted_nodes && accept_len && prefix_len && status,
             "kv_commit_paged: NULL pointer");
  TV_REQUIRE(L >= 0 && B >= 0 && Nmax >= 1 && Hkv >= 1 && d >= 8 && n_pages >= 1 && max_blocks >= 1 && Dp1 >= 1,
             "kv_commit_paged: bad dimension");
  TV_REQUIRE(max_blocks <= (1 << 20), "kv_commit_paged: max_blocks must be <= 2^20");
  TV_REQUIRE(d % 8 == 0, "kv_commit_paged: d must be a multiple of 8 (16-byte rows)");
  TV_REQUIRE(page_layer_stride % 8 == 0 && tree_layer_stride % 8 == 0, "kv_commit_paged: layer strides must be multiples of 8 elements");
  TV_REQUIRE(tv::aligned16(k_pages) && tv::aligned16(v_pages) && tv::aligned16(k_tree) && tv::aligned16(v_tree),
             "kv_commit_paged: tensors must be 16-byte aligned");
  TV_REQUIRE(L <= 65535 && Dp1 <= kCopyMaxDp1, "kv_commit_paged: L must be <= 65535 and Dp1 <= 1024");
  if (L == 0 || B == 0) return TV_OK;
  cudaStream_t s = (cudaStream_t)stream;
  commit_paged_kernel<<<dim3(B, L), kCopyThreads, 0, s>>>(
      reinterpret_cast<uint4*>(k_pages), reinterpret_cast<uint4*>(v_pages), block_table,
      reinterpret_cast<const uint4*>(k_tree), reinterpret_cast<const uint4*>(v_tree), accepted_nodes, accept_len,
      prefix_len, status, B, Nmax, Hkv, d / 8, n_pages, max_blocks, Dp1, page_layer_stride / 8, tree_layer_stride / 8);
  TV_CUDA_OK(cudaGetLastError());
  commit_paged_finish_kernel<<<(B + 127) / 128, 128, 0, s>>>(accepted_nodes, accept_len, block_table, prefix_len, status,
                                                             B, Nmax, n_pages, max_blocks, Dp1);
  TV_CUDA_OK(cudaGetLastError());
  tv::count_launches(2);
  return TV_OK;
}

extern "C" int kv_commit_inplace(tv_bf16* k_cache, tv_bf16* v_cache,
                                 const int32_t* accepted_nodes, const int32_t* accept_len,
                                 int32_t* prefix_len,
                                 int L, int B, int Nmax, int Hkv, int d, int Scap, int Dp1,
                                 int64_t cache_layer_stride,
                                 int32_t* status, tv_stream stream) {
  TV_REQUIRE(k_cache && v_cache && accepted_nodes && accept_len && prefix_len && status, "kv_commit_inplace: NULL pointer");
  TV_REQUIRE(L >= 0 && B >= 0 && Nmax >= 1 && Hkv >= 1 && d >= 8 && Scap >= 1 && Dp1 >= 1,
             "kv_commit_inplace: bad dimension");
  TV_REQUIRE(d % 8 == 0, "kv_commit_inplace: d must be a multiple of 8 (16-byte rows)");
  TV_REQUIRE(cache_layer_stride % 8 == 0, "kv_commit_inplace: the layer stride must be a multiple of 8 elements");
  TV_REQUIRE(tv::aligned16(k_cache) && tv::aligned16(v_cache), "kv_commit_inplace: tensors must be 16-byte aligned");
  TV_REQUIRE(B <= 65535 && L <= 65535 && Hkv <= 32767, "kv_commit_inplace: B and L must be <= 65535, Hkv <= 32767");
  TV_REQUIRE((long long)Dp1 * (d / 8) <= kInplaceMaxPieces,
             "kv_commit_inplace: Dp1 * d / 8 must be <= 2048 (the accepted segment of a head is staged in registers)");
  if (L == 0 || B == 0) return TV_OK;
  cudaStream_t s = (cudaStream_t)stream;
  int hpc = 1;       // KV heads per CTA: the largest divisor of Hkv whose longest possible segments fit the registers
  for (int c = 1; c <= Hkv; ++c)
    if (Hkv % c == 0 && (long long)c * Dp1 * (d / 8) <= kInplaceMaxPieces) hpc = c;
  commit_inplace_kernel<<<dim3(2 * (Hkv / hpc), B, L), kInplaceThreads, 0, s>>>(
      reinterpret_cast<uint4*>(k_cache), reinterpret_cast<uint4*>(v_cache), accepted_nodes, accept_len, prefix_len,
      status, B, Nmax, Hkv, d / 8, Scap, Dp1, hpc, cache_layer_stride / 8);
  TV_CUDA_OK(cudaGetLastError());
  commit_inplace_finish_kernel<<<(B + 127) / 128, 128, 0, s>>>(accepted_nodes, accept_len, prefix_len, status,
                                                               B, Nmax, Scap, Dp1);
  TV_CUDA_OK(cudaGetLastError());
  tv::count_launches(2);
  return TV_OK;
}

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
  TV_REQUIRE(L <= 65535, "kv_commit: L must be <= 65535");
  TV_REQUIRE(Dp1 <= kCopyMaxDp1, "kv_commit: Dp1 must be <= 1024");
  if (L == 0 || B == 0) return TV_OK;
  const int dvec = d / 8;
  cudaStream_t s = (cudaStream_t)stream;
  TV_CUDA_OK(tv::launch_pdl(commit_copy_kernel, dim3(B, L), dim3(kCopyThreads), 0, s,
                            reinterpret_cast<uint4*>(k_cache), reinterpret_cast<uint4*>(v_cache),
                            reinterpret_cast<const uint4*>(k_tree), reinterpret_cast<const uint4*>(v_tree),
                            accepted_nodes, accept_len, prefix_len, status, B, Nmax, Hkv, dvec, Scap, Dp1,
                            cache_layer_stride / 8, tree_layer_stride / 8));
  TV_CUDA_OK(tv::launch_pdl(commit_finish_kernel, dim3((B + 127) / 128), dim3(128), 0, s, accepted_nodes, accept_len,
                            prefix_len, status, B, Nmax, Scap, Dp1));
  tv::count_launches(2);
  return TV_OK;
}
