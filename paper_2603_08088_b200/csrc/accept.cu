// tree_accept: teacher argmax over the vocabulary (an HBM-bound scan of the
// logits), the accelerator-safe path gather (Section 2.5 / 3.2) and greedy
// acceptance along root-to-leaf rows (Section 2.3).
//
// Phase 1 (argmax_scan_kernel) streams logits[B,Nmax,V] once with 16-byte
// streaming loads; every CTA reduces one vocabulary chunk of one row to a (value,
// index) pair in scratch.  Phase 2 (accept_kernel), one CTA per sequence,
// folds the chunk pairs in index order, then remaps, gathers and compares.
// Ties resolve to the lowest index at every level of the reduction.
#include "common.cuh"

#include <cuda_bf16.h>

#include <mutex>

namespace {

constexpr int kScanThreads = 256;
constexpr int kVecPerThread = 8;                                   // 16-byte loads in flight per thread
constexpr int kChunkElems = kScanThreads * kVecPerThread * 8;      // 16384 logits per CTA

struct ArgPair {
  float val;
  int32_t idx;
};

__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16) {
  return __uint_as_float(bits16 << 16);
}

// (v, i) beats (bv, bi) when it is larger, or equal with a lower index.
__device__ __forceinline__ void take_better(float& bv, int& bi, float v, int i) {
  if (v > bv || (v == bv && i < bi)) {
    bv = v;
    bi = i;
  }
}

__device__ __forceinline__ float vec8_max(const uint4& u) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
  __nv_bfloat162 m = __hmax2(__hmax2(h[0], h[1]), __hmax2(h[2], h[3]));
  const float r = fmaxf(__low2float(m), __high2float(m));   // max of a NaN and x is x
  return r == r ? r : -INFINITY;                            // an all-NaN vector can never win
}

// Persistent scan: the (row, vocabulary chunk) items are dealt round-robin to a grid of a few CTAs per SM, and a
// CTA requests the vectors of its next item before it reduces the ones it holds, so the memory pipe never drains
// at an item boundary.
__global__ void __launch_bounds__(kScanThreads, 3)
argmax_scan_kernel(const tv_bf16* __restrict__ logits, const int32_t* __restrict__ n_nodes,
                   int Nmax, int V, int n_chunks, int n_items, ArgPair* __restrict__ partial) {
  tv::pdl_enter();
  const int tid = threadIdx.x;
  const bool vec_ok = ((V & 7) == 0) && ((reinterpret_cast<uintptr_t>(logits) & 15u) == 0);
  __shared__ float sv[2][kScanThreads / 32];      // two sets, taken in turn: one barrier per item suffices
  __shared__ int si[2][kScanThreads / 32];
  int set = 0;
  const uint4 kLowest = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);     // bf16 -inf

  // item -> (row, chunk, active); padded rows are never read
  auto locate = [&](int item, int& row, int& chunk) -> bool {
    if (item >= n_items) return false;
    row = item / n_chunks;
    chunk = item - row * n_chunks;
    const int b = row / Nmax;
    return row - b * Nmax < n_nodes[b];
  };
  auto fetch = [&](int row, int chunk, uint4* u) {
    const uint4* vbase = reinterpret_cast<const uint4*>(logits + (size_t)row * V);
    const int v0 = (chunk * kChunkElems) >> 3, v1 = min(V, (chunk + 1) * kChunkElems) >> 3;
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
      const int vi = v0 + k * kScanThreads + tid;
      u[k] = vi < v1 ? __ldcs(vbase + vi) : kLowest;
    }
  };

  int item = blockIdx.x;
  int row = 0, chunk = 0;
  bool active = locate(item, row, chunk);
  uint4 u[kVecPerThread];
  if (active && vec_ok) fetch(row, chunk, u);
  while (item < n_items) {
    const int nitem = item + gridDim.x;
    int nrow = 0, nchunk = 0;
    const bool nactive = locate(nitem, nrow, nchunk);
    uint4 un[kVecPerThread];
    if (nactive && vec_ok) fetch(nrow, nchunk, un);
    if (active) {
      const int c0 = chunk * kChunkElems;
      const int c1 = min(V, c0 + kChunkElems);
      float best = -INFINITY;
      int best_i = 0x7fffffff;
      if (vec_ok) {
        const int v0 = c0 >> 3, v1 = c1 >> 3;      // vector range of this chunk
        int best_vec = -1;
#pragma unroll
        for (int k = 0; k < kVecPerThread; ++k) {
          const float m = vec8_max(u[k]);
          if (v0 + k * kScanThreads + tid < v1 && (m > best || best_vec < 0)) {   // increasing index order: strict > keeps the first
            best = m;
            best_vec = k;
          }
        }
        if (best_vec >= 0) {
          uint4 w = u[0];
#pragma unroll
          for (int k = 1; k < kVecPerThread; ++k) if (best_vec == k) w = u[k];
          const uint32_t e[4] = {w.x, w.y, w.z, w.w};
          float bv = -INFINITY;
          int bi = 0x7fffffff;
#pragma unroll
          for (int t = 0; t < 8; ++t) {
            const uint32_t bits = (t & 1) ? (e[t >> 1] >> 16) : (e[t >> 1] & 0xffffu);
            float f = bf16_bits_to_float(bits);
            f = f == f ? f : -INFINITY;
            take_better(bv, bi, f, t);
          }
          best = bv;
          best_i = (v0 + best_vec * kScanThreads + tid) * 8 + bi;
        }
      } else {
        const tv_bf16* base = logits + (size_t)row * V;
        for (int v = c0 + tid; v < c1; v += kScanThreads) {
          float f = bf16_bits_to_float(base[v]);
          f = f == f ? f : -INFINITY;
          take_better(best, best_i, f, v);
        }
      }
      // warp, then block reduction with the same rule
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, off);
        const int oi = __shfl_xor_sync(0xffffffffu, best_i, off);
        take_better(best, best_i, ov, oi);
      }
      if ((tid & 31) == 0) {
        sv[set][tid >> 5] = best;
        si[set][tid >> 5] = best_i;
      }
      __syncthreads();
      if (tid == 0) {
        for (int w = 1; w < kScanThreads / 32; ++w) take_better(best, best_i, sv[set][w], si[set][w]);
        ArgPair out;
        out.val = best;
        out.idx = best_i;
        partial[(size_t)row * n_chunks + chunk] = out;
      }
      set ^= 1;              // the next item writes the other set; this one is rewritten only after the next barrier
    }
    item = nitem;
    row = nrow;
    chunk = nchunk;
    active = nactive;
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) u[k] = un[k];
  }
}

__global__ void __launch_bounds__(256)
accept_kernel(const ArgPair* __restrict__ partial, int n_chunks,
              const int32_t* __restrict__ tokens, const int32_t* __restrict__ retrieve,
              const int32_t* __restrict__ n_nodes,
              int Nmax, int P, int Dp1,
              int32_t* __restrict__ argmax_tok, int32_t* __restrict__ safe_idx,
              int32_t* __restrict__ candidates, int32_t* __restrict__ accept_len,
              int32_t* __restrict__ best_path, int32_t* __restrict__ accepted_nodes,
              int32_t* __restrict__ next_token, int32_t* __restrict__ status) {
  tv::pdl_enter();
  extern __shared__ int32_t am[];          // [Nmax] teacher argmax of this sequence
  __shared__ unsigned long long best_key;  // (accepted length << 32) | ~row : max = longest, then lowest row
  __shared__ int bad_index;
  const int b = blockIdx.x;
  const int tid = threadIdx.x, nt = blockDim.x;
  int n = n_nodes[b];
  n = n < 0 ? 0 : (n > Nmax ? Nmax : n);
  if (tid == 0) {
    best_key = 0xffffffffull;              // length 0, row 0
    bad_index = 0;
  }
  for (int i = tid; i < Nmax; i += nt) {
    int tok = -1;
    if (i < n) {
      const ArgPair* pp = partial + ((size_t)b * Nmax + i) * n_chunks;
      float bv = -INFINITY;
      int bi = 0x7fffffff;
      for (int c0 = 0; c0 < n_chunks; c0 += 8) {       // eight pairs requested together, folded in chunk order
        ArgPair p8[8];
#pragma unroll
        for (int k = 0; k < 8; ++k)
          if (c0 + k < n_chunks) p8[k] = pp[c0 + k];
#pragma unroll
        for (int k = 0; k < 8; ++k)
          if (c0 + k < n_chunks) take_better(bv, bi, p8[k].val, p8[k].idx);
      }
      tok = bi;
    }
    am[i] = tok;
    argmax_tok[(size_t)b * Nmax + i] = tok;
  }
  __syncthreads();

  const int32_t* rows = retrieve + (size_t)b * P * Dp1;
  const int32_t* tok_b = tokens + (size_t)b * Nmax;
  for (int p = tid; p < P; p += nt) {
    int a = 0;
    bool chain = true;
    bool prev_ok = false;
    int prev_safe = 0;
    for (int j = 0; j < Dp1; ++j) {
      const int r = rows[p * Dp1 + j];
      const bool ok = r >= 0 && r < n;
      if (r < -1 || r >= n) bad_index = 1;
      const int s = ok ? r : 0;            // remap BEFORE the gather: s is always in [0, Nmax)
      const int cand = tok_b[s];
      if (safe_idx) safe_idx[((size_t)b * P + p) * Dp1 + j] = s;
      if (candidates) candidates[((size_t)b * P + p) * Dp1 + j] = cand;
      if (j > 0 && chain) {
        if (ok && prev_ok && cand == am[prev_safe]) a = j;
        else chain = false;
      }
      prev_ok = ok;
      prev_safe = s;
    }
    const unsigned long long key = ((unsigned long long)a << 32) | (unsigned long long)(0xffffffffu - (unsigned)p);
    atomicMax(&best_key, key);
  }
  __syncthreads();
  const int A = (int)(best_key >> 32);
  const int pstar = (int)(0xffffffffu - (unsigned)(best_key & 0xffffffffull));
  for (int j = tid; j < Dp1; j += nt) {
    int node = 0;
    if (j <= A && P > 0) {
      const int r = rows[pstar * Dp1 + j];
      node = (r >= 0 && r < n) ? r : 0;
    }
    accepted_nodes[(size_t)b * Dp1 + j] = node;
    if (j == A) next_token[b] = am[node];
  }
  if (tid == 0) {
    accept_len[b] = A;
    best_path[b] = pstar;
    if (bad_index) atomicOr(&status[b], TV_ST_BAD_INDEX);
  }
}

// One thread per (sequence, node): score of the node's proposed token in the logits of its parent's slot.
__global__ void node_scores_kernel(const tv_bf16* __restrict__ logits, const int32_t* __restrict__ tokens,
                                   const int32_t* __restrict__ parent, const int32_t* __restrict__ n_nodes,
                                   int B, int Nmax, int V, float* __restrict__ scores, int32_t* __restrict__ status) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= B * Nmax) return;
  const int b = idx / Nmax, k = idx - b * Nmax;
  int n = n_nodes[b];
  n = n < 0 ? 0 : (n > Nmax ? Nmax : n);
  float val = 0.f;
  if (k >= 1 && k < n) {
    const int p = parent[idx];
    const int sp = (p >= 0 && p < n) ? p : 0;          // dummy-root remap before the gather
    const int t = tokens[idx];
    const bool ok = t >= 0 && t < V;
    const int st = ok ? t : 0;                          // in-range vocabulary index
    const float g = bf16_bits_to_float(logits[((size_t)b * Nmax + sp) * V + st]);
    val = ok ? g : -INFINITY;
    if (!ok) atomicOr(&status[b], TV_ST_BAD_INDEX);
  }
  scores[idx] = val;
}

int scan_chunks(int V) { return (V + kChunkElems - 1) / kChunkElems; }

// CTAs of the persistent scan: three per SM (what its registers allow).
int scan_ctas() {
  static int n = [] {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148 * 3;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return 148 * 3;
    return sms * 3;
  }();
  return n;
}

// Scratch of tree_accept_noalloc: a fixed device array that lives in the library image, so that callers
// who may not allocate device memory can still run the accept step.  Every GPU that loads the library
// holds these 256 KiB until the process exits.
constexpr size_t kStaticPairs = 32768;                       // (row, vocabulary chunk) pairs
static __device__ __align__(256) unsigned char g_accept_scratch[kStaticPairs * sizeof(ArgPair)];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of g_accept_scratch on the current device.  In host code the symbol's name is only a
// stand-in, not an address a kernel can use; the runtime hands out the real one, once per device.
int static_scratch(void** out) {
  int dev = -1;
  TV_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices)
    return tv::fail(TV_ERR_INVALID_ARG, "tree_accept_noalloc: device ordinal %d is not supported", dev);
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    TV_CUDA_OK(cudaGetSymbolAddress(&p, g_accept_scratch));
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return TV_OK;
}

}  // namespace

extern "C" size_t tv_accept_workspace_bytes(int B, int Nmax, int V) {
  if (B <= 0 || Nmax <= 0 || V <= 0) return 16;
  return (size_t)B * Nmax * scan_chunks(V) * sizeof(ArgPair);
}

extern "C" int tree_accept(const tv_bf16* logits, const int32_t* tokens,
                           const int32_t* retrieve_indices, const int32_t* n_nodes,
                           int B, int Nmax, int V, int P, int Dp1,
                           int32_t* argmax_tok, int32_t* safe_idx, int32_t* candidates,
                           int32_t* accept_len, int32_t* best_path, int32_t* accepted_nodes,
                           int32_t* next_token,
                           void* workspace, size_t workspace_bytes,
                           int32_t* status, tv_stream stream) {
  TV_REQUIRE(logits && tokens && n_nodes && argmax_tok && accept_len && best_path && accepted_nodes &&
                 next_token && status && workspace,
             "tree_accept: NULL required pointer");
  TV_REQUIRE(B >= 0 && Nmax >= 1 && Nmax <= 8192 && V >= 1 && P >= 0 && Dp1 >= 1,
             "tree_accept: need B >= 0, 1 <= Nmax <= 8192, V >= 1, P >= 0, Dp1 >= 1");
  TV_REQUIRE(P == 0 || retrieve_indices, "tree_accept: retrieve_indices is NULL with P > 0");
  TV_REQUIRE(B * (long long)Nmax <= 65535, "tree_accept: B*Nmax exceeds 65535 rows");
  TV_REQUIRE((reinterpret_cast<uintptr_t>(workspace) & 7u) == 0, "tree_accept: workspace must be 8-byte aligned");
  if (workspace_bytes < tv_accept_workspace_bytes(B, Nmax, V))
    return tv::fail(TV_ERR_WORKSPACE, "tree_accept: workspace of %zu bytes, need %zu", workspace_bytes,
                    tv_accept_workspace_bytes(B, Nmax, V));
  if (B == 0) return TV_OK;
  const int n_chunks = scan_chunks(V);
  ArgPair* partial = static_cast<ArgPair*>(workspace);
  cudaStream_t s = (cudaStream_t)stream;
  const long long n_items = (long long)B * Nmax * n_chunks;
  TV_REQUIRE(n_items < (1ll << 31), "tree_accept: B * Nmax * ceil(V / 16384) must stay below 2^31");
  const int scan_grid = (int)(n_items < (long long)scan_ctas() ? n_items : scan_ctas());
  TV_CUDA_OK(tv::launch_pdl(argmax_scan_kernel, dim3(scan_grid), dim3(kScanThreads), 0, s, logits, n_nodes, Nmax, V,
                            n_chunks, (int)n_items, partial));
  TV_CUDA_OK(tv::launch_pdl(accept_kernel, dim3(B), dim3(256), Nmax * sizeof(int32_t), s, partial, n_chunks, tokens,
                            retrieve_indices, n_nodes, Nmax, P, Dp1, argmax_tok, safe_idx, candidates, accept_len, best_path,
                            accepted_nodes, next_token, status));
  tv::count_launches(2);
  return TV_OK;
}

extern "C" size_t tv_accept_noalloc_max_bytes(void) { return kStaticPairs * sizeof(ArgPair); }

extern "C" int tree_accept_noalloc(const tv_bf16* logits, const int32_t* tokens,
                                   const int32_t* retrieve_indices, const int32_t* n_nodes,
                                   int B, int Nmax, int V, int P, int Dp1,
                                   int32_t* argmax_tok, int32_t* safe_idx, int32_t* candidates,
                                   int32_t* accept_len, int32_t* best_path, int32_t* accepted_nodes,
                                   int32_t* next_token, int32_t* status, tv_stream stream) {
  TV_REQUIRE(B >= 0 && Nmax >= 1 && V >= 1, "tree_accept_noalloc: need B >= 0, Nmax >= 1, V >= 1");
  const size_t need = tv_accept_workspace_bytes(B, Nmax, V);
  if (need > kStaticPairs * sizeof(ArgPair))
    return tv::fail(TV_ERR_WORKSPACE,
                    "tree_accept_noalloc: B*Nmax*ceil(V/%d) = %zu scratch entries, the built-in scratch holds %zu; "
                    "use tree_accept with a caller workspace",
                    kChunkElems, need / sizeof(ArgPair), kStaticPairs);
  void* scratch = nullptr;
  const int rc = static_scratch(&scratch);
  if (rc != TV_OK) return rc;
  return tree_accept(logits, tokens, retrieve_indices, n_nodes, B, Nmax, V, P, Dp1, argmax_tok, safe_idx, candidates,
                     accept_len, best_path, accepted_nodes, next_token, scratch, kStaticPairs * sizeof(ArgPair),
                     status, stream);
}

extern "C" int tree_node_scores(const tv_bf16* logits, const int32_t* tokens, const int32_t* parent,
                                const int32_t* n_nodes, int B, int Nmax, int V, float* scores,
                                int32_t* status, tv_stream stream) {
  TV_REQUIRE(logits && tokens && parent && n_nodes && scores && status, "tree_node_scores: NULL pointer");
  TV_REQUIRE(B >= 0 && Nmax >= 1 && V >= 1, "tree_node_scores: need B >= 0, Nmax >= 1, V >= 1");
  if (B == 0) return TV_OK;
  const int total = B * Nmax;
  node_scores_kernel<<<(total + 127) / 128, 128, 0, (cudaStream_t)stream>>>(logits, tokens, parent, n_nodes, B, Nmax, V,
                                                                             scores, status);
  TV_CUDA_OK(cudaGetLastError());
  tv::count_launches(1);
  return TV_OK;
}
