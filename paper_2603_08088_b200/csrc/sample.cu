// tree_accept_sample: sampling-mode acceptance over the tree (Section 2.2: an acceptance rule "rejection
// sampling style" that keeps the teacher's distribution; Section 3.3: the node scores are what it consumes).
// The rule is speculative sampling for proposals without a draft probability (q = one-hot), walked down the
// tree: at the current node the children are tried in node order, child k with token x is accepted iff
// u_node[k] < p(x) / (1 - mass rejected so far at this node), a rejected token's mass is removed; when no
// child passes, the next token is drawn from what is left of p by inversion of the cumulative sum in
// vocabulary order at u_bonus.  p = softmax(logits / T) of the current node's row.
//
// Phase 1 (row_stats_kernel) streams logits[B,Nmax,V] once, like the argmax scan: every CTA reduces one
// vocabulary chunk of one row to (max, sum of 2^((l - max) k)), k = log2(e) / T.  Phase 2
// (sample_walk_kernel), one CTA per sequence: folds the chunk pairs per row in chunk order, gathers the mass
// of every node's token in its parent's row, walks the tree with one thread, and then all threads draw the
// next token from the last node's row (segment sums in vocabulary order, a serial prefix over the segments,
// a rescan of the segment that holds the target).  All arithmetic in fp32.
#include "common.cuh"

#include <cuda_bf16.h>

namespace {

constexpr int kStatThreads = 256;
constexpr int kStatVecPerThread = 4;
constexpr int kStatChunk = kStatThreads * kStatVecPerThread * 8;      // 8192 logits per CTA
constexpr int kWalkThreads = 256;
constexpr int kMaxNodes = 256;
constexpr float kLog2e = 1.4426950408889634f;

struct RowStat {
  float m;      // maximum of the chunk (raw logit units); -inf for an empty chunk
  float s;      // sum over the chunk of 2^((l - m) * k)
};

__device__ __forceinline__ float bf16_to_float(uint32_t bits16) { return __uint_as_float(bits16 << 16); }

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Unnormalised mass of a vocabulary entry with logit l in a row whose maximum is M: 2^((l - M) k); 0 for NaN
// and -inf (fmaxf returns its other operand for a NaN, and 2^-150 flushes to 0).
__device__ __forceinline__ float mass_of(float l, float M, float k) {
  return ex2_approx(fmaxf((l - M) * k, -150.f));
}

// (m, s) <- (m, s) merged with (mo, so): s = sum of 2^((l - m) k) over a set whose maximum is m.
__device__ __forceinline__ void merge_pair(float& m, float& s, float mo, float so, float k) {
  const float M = fmaxf(m, mo);
  if (M > -INFINITY) {
    s = (m > -INFINITY ? s * ex2_approx((m - M) * k) : 0.f) + (mo > -INFINITY ? so * ex2_approx((mo - M) * k) : 0.f);
    m = M;
  }
}

__global__ void __launch_bounds__(kStatThreads)
row_stats_kernel(const tv_bf16* __restrict__ logits, const int32_t* __restrict__ n_nodes, int Nmax, int V,
                 int n_chunks, float k, RowStat* __restrict__ stats) {
  const int row = blockIdx.y;
  const int b = row / Nmax, i = row - b * Nmax;
  if (i >= n_nodes[b]) return;
  const int c0 = blockIdx.x * kStatChunk;
  const int c1 = min(V, c0 + kStatChunk);
  const uint16_t* base = reinterpret_cast<const uint16_t*>(logits) + (size_t)row * V;
  const int tid = threadIdx.x;
  // the chunk's values of this thread stay in registers between the two passes (maximum, then sum)
  float vals[kStatVecPerThread * 8];
  const bool vec_ok = ((V & 7) == 0) && ((reinterpret_cast<uintptr_t>(logits) & 15u) == 0);
#pragma unroll
  for (int q = 0; q < kStatVecPerThread; ++q) {
    const int v0 = c0 + (q * kStatThreads + tid) * 8;
    if (vec_ok && v0 + 8 <= c1) {
      const uint4 u = __ldcs(reinterpret_cast<const uint4*>(base + v0));
      const uint32_t e[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
      for (int t = 0; t < 8; ++t) vals[q * 8 + t] = bf16_to_float((t & 1) ? (e[t >> 1] >> 16) : (e[t >> 1] & 0xffffu));
    } else {
#pragma unroll
      for (int t = 0; t < 8; ++t) vals[q * 8 + t] = (v0 + t < c1) ? bf16_to_float(base[v0 + t]) : -INFINITY;
    }
  }
  // per thread, then per warp (pairs merged by shuffles), then one barrier and a fold of the eight warp pairs
  float m = -INFINITY;
#pragma unroll
  for (int t = 0; t < kStatVecPerThread * 8; ++t) m = fmaxf(m, vals[t]);      // a NaN never becomes the maximum
  float s = 0.f;
  if (m > -INFINITY) {
#pragma unroll
    for (int t = 0; t < kStatVecPerThread * 8; ++t) s += mass_of(vals[t], m, k);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float mo = __shfl_xor_sync(0xffffffffu, m, off);
    const float so = __shfl_xor_sync(0xffffffffu, s, off);
    merge_pair(m, s, mo, so, k);
  }
  __shared__ float red_m[kStatThreads / 32], red_s[kStatThreads / 32];
  if ((tid & 31) == 0) {
    red_m[tid >> 5] = m;
    red_s[tid >> 5] = s;
  }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < kStatThreads / 32; ++w) merge_pair(m, s, red_m[w], red_s[w], k);
    RowStat out;
    out.m = m;
    out.s = s;
    stats[(size_t)row * n_chunks + blockIdx.x] = out;
  }
}


__global__ void __launch_bounds__(kWalkThreads)
sample_walk_kernel(const tv_bf16* __restrict__ logits, const RowStat* __restrict__ stats, int n_chunks,
                   const int32_t* __restrict__ tokens, const int32_t* __restrict__ parent,
                   const int32_t* __restrict__ n_nodes, const float* __restrict__ u_node,
                   const float* __restrict__ u_bonus, float k, int Nmax, int V, int Dp1,
                   int32_t* __restrict__ accept_len, int32_t* __restrict__ accepted_nodes,
                   int32_t* __restrict__ next_token, int32_t* __restrict__ status) {
  __shared__ float sM[kMaxNodes], sZ[kMaxNodes], sE[kMaxNodes], sU[kMaxNodes];   // row max, row sum, token mass, uniform
  __shared__ int sPar[kMaxNodes], sTok[kMaxNodes], sRej[kMaxNodes];
  __shared__ float sWarp[kWalkThreads / 32];
  __shared__ int sLast, sNrej, sHit, sBad;
  __shared__ float sTarget;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int n = n_nodes[b];
  n = n < 0 ? 0 : (n > Nmax ? Nmax : n);
  const uint16_t* lg = reinterpret_cast<const uint16_t*>(logits) + (size_t)b * Nmax * V;
  if (tid == 0) sBad = 0;
  // ---- per-row maximum and sum: the chunk pairs folded in chunk order (one pass, rescaling as the maximum grows)
  for (int i = tid; i < n; i += kWalkThreads) {
    const RowStat* rs = stats + ((size_t)b * Nmax + i) * n_chunks;
    float M = -INFINITY, Z = 0.f;
    for (int c = 0; c < n_chunks; ++c) {
      const RowStat r = rs[c];
      if (r.m > -INFINITY) {
        const float Mn = fmaxf(M, r.m);
        Z = Z * exp2f((M - Mn) * k) + r.s * exp2f((r.m - Mn) * k);       // M = -inf the first time: 0 * 0
        M = Mn;
      }
    }
    sM[i] = M;
    sZ[i] = Z;
    const int p = parent[(size_t)b * Nmax + i];
    sPar[i] = (p >= 0 && p < n) ? p : 0;                 // dummy-root remap (Section 3.2)
    sTok[i] = tokens[(size_t)b * Nmax + i];
    sU[i] = u_node[(size_t)b * Nmax + i];
  }
  __syncthreads();
  // ---- mass of every node's token in its parent's row (the node score of Section 3.3, exponentiated)
  for (int i = tid; i < n; i += kWalkThreads) {
    float e = 0.f;
    if (i >= 1) {
      const int x = sTok[i];
      if (x >= 0 && x < V) {
        e = mass_of(bf16_to_float(lg[(size_t)sPar[i] * V + x]), sM[sPar[i]], k);
      } else {
        sBad = 1;            // benign race: every writer stores 1
      }
    }
    sE[i] = e;
  }
  __syncthreads();
  // ---- the walk (one thread, shared memory only; at most Nmax steps in all)
  if (tid == 0) {
    int c = 0, depth = 0, nrej = 0;
    float rem = n > 0 ? sZ[0] : 0.f;
    for (int j = 0; j < Dp1; ++j) accepted_nodes[(size_t)b * Dp1 + j] = 0;
    while (depth < Dp1 - 1) {
      int acc = -1;
      for (int kk = c + 1; kk < n; ++kk) {
        if (sPar[kk] != c) continue;
        const int x = sTok[kk];
        if (x < 0 || x >= V) continue;
        bool dup = false;
        for (int r = 0; r < nrej; ++r) dup |= (sRej[r] == x);
        if (dup) continue;
        const float prob = rem > 0.f ? sE[kk] / rem : 0.f;
        if (sU[kk] < prob) {
          acc = kk;
          break;
        }
        sRej[nrej++] = x;
        rem -= sE[kk];
      }
      if (acc < 0) break;
      ++depth;
      accepted_nodes[(size_t)b * Dp1 + depth] = acc;
      c = acc;
      nrej = 0;
      rem = sZ[c];
    }
    accept_len[b] = depth;
    sLast = c;
    sNrej = nrej;
    sTarget = u_bonus[b] * fmaxf(rem, 0.f);       // in units of the remaining (unnormalised) mass
    sHit = -1;
    if (sBad) atomicOr(status + b, TV_ST_BAD_INDEX);
  }
  __syncthreads();
  // ---- next token: the first entry of row c, rejected tokens left out, whose cumulative mass in vocabulary
  // order exceeds the target.  The row is streamed 64 entries per thread and step (one 128-byte line each, a
  // warp reads 4 KB in a row); the running sum passes from step to step through a block-wide scan.
  if (n == 0) {
    if (tid == 0) next_token[b] = -1;       // no row to draw from
    return;
  }
  const int c = sLast, nrej = sNrej;
  const float M = sM[c], target = sTarget;
  const uint16_t* row = lg + (size_t)c * V;
  const bool vec_ok = ((V & 7) == 0) && ((reinterpret_cast<uintptr_t>(logits) & 15u) == 0);
  constexpr int kPerThread = 64;
  float carried = 0.f;                 // cumulative mass of everything before this step
  int last_with_mass = -1;             // fallback when rounding leaves the target above the scanned total
  for (int base = 0; base < V; base += kWalkThreads * kPerThread) {
    const int v0 = base + tid * kPerThread;
    float vals[kPerThread];
    if (vec_ok && v0 + kPerThread <= V) {
#pragma unroll
      for (int q = 0; q < kPerThread / 8; ++q) {
        const uint4 u = __ldg(reinterpret_cast<const uint4*>(row + v0) + q);
        const uint32_t e[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int t = 0; t < 8; ++t) vals[q * 8 + t] = bf16_to_float((t & 1) ? (e[t >> 1] >> 16) : (e[t >> 1] & 0xffffu));
      }
    } else {
#pragma unroll
      for (int t = 0; t < kPerThread; ++t) vals[t] = (v0 + t < V) ? bf16_to_float(row[v0 + t]) : -INFINITY;
    }
    float sum = 0.f;
#pragma unroll
    for (int t = 0; t < kPerThread; ++t) {
      vals[t] = mass_of(vals[t], M, k);
      sum += vals[t];
    }
    for (int r = 0; r < nrej; ++r) {               // rejected tokens that fall into this thread's 64 entries
      const int off = sRej[r] - v0;
      if (off >= 0 && off < kPerThread) {
        float m_r = 0.f;
#pragma unroll
        for (int t = 0; t < kPerThread; ++t) m_r = (t == off) ? vals[t] : m_r;
        sum -= m_r;
#pragma unroll
        for (int t = 0; t < kPerThread; ++t) vals[t] = (t == off) ? 0.f : vals[t];
      }
    }
    sum = fmaxf(sum, 0.f);
    // block-wide inclusive scan of the thread sums, in thread (= vocabulary) order
    float incl = sum;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const float o = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += o;
    }
    if (lane == 31) sWarp[warp] = incl;
    __syncthreads();
    float before = carried;
    for (int w = 0; w < warp; ++w) before += sWarp[w];
    float step_total = 0.f;
    for (int w = 0; w < kWalkThreads / 32; ++w) step_total += sWarp[w];
    const float excl = before + incl - sum;          // cumulative mass before this thread's entries
    if (excl <= target && target < excl + sum) {     // the crossing lies in this thread's entries
      float cum = excl;
      int hit = -1;
#pragma unroll
      for (int t = 0; t < kPerThread; ++t) {
        cum += vals[t];
        if (hit < 0 && cum > target) hit = v0 + t;
      }
      if (hit < 0) {                                 // rounding inside the 64 entries: the last one with mass
#pragma unroll
        for (int t = 0; t < kPerThread; ++t)
          if (vals[t] > 0.f) hit = v0 + t;
      }
      if (hit >= 0) sHit = hit;
    }
    {
      int lw = -1;
#pragma unroll
      for (int t = 0; t < kPerThread; ++t)
        if (vals[t] > 0.f) lw = v0 + t;
      last_with_mass = max(last_with_mass, lw);
    }
    carried += step_total;
    __syncthreads();
    if (sHit >= 0) break;                            // uniform: read after the barrier
  }
  if (sHit < 0) {
    // the target was not below the scanned total (u_bonus close to 1 and rounding): the last entry with mass
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) last_with_mass = max(last_with_mass, __shfl_xor_sync(0xffffffffu, last_with_mass, off));
    __shared__ int sLastMass[kWalkThreads / 32];
    if (lane == 0) sLastMass[warp] = last_with_mass;
    __syncthreads();
    if (tid == 0) {
      int lm = -1;
      for (int w = 0; w < kWalkThreads / 32; ++w) lm = max(lm, sLastMass[w]);
      sHit = lm >= 0 ? lm : V - 1;
    }
    __syncthreads();
  }
  if (tid == 0) next_token[b] = sHit;
}

int stat_chunks(int V) { return (V + kStatChunk - 1) / kStatChunk; }

}  // namespace

extern "C" size_t tv_sample_workspace_bytes(int B, int Nmax, int V) {
  if (B <= 0 || Nmax <= 0 || V <= 0) return 16;
  return (size_t)B * Nmax * stat_chunks(V) * sizeof(RowStat);
}

extern "C" int tree_accept_sample(const tv_bf16* logits, const int32_t* tokens, const int32_t* parent,
                                  const int32_t* n_nodes, const float* u_node, const float* u_bonus,
                                  float temperature, int B, int Nmax, int V, int Dp1,
                                  int32_t* accept_len, int32_t* accepted_nodes, int32_t* next_token,
                                  void* workspace, size_t workspace_bytes,
                                  int32_t* status, tv_stream stream) {
  TV_REQUIRE(logits && tokens && parent && n_nodes && u_node && u_bonus && accept_len && accepted_nodes && next_token &&
                 workspace && status,
             "tree_accept_sample: NULL pointer");
  TV_REQUIRE(B >= 0 && Nmax >= 1 && Nmax <= kMaxNodes && V >= 1 && Dp1 >= 1,
             "tree_accept_sample: need B >= 0, 1 <= Nmax <= 256, V >= 1, Dp1 >= 1");
  TV_REQUIRE(temperature > 0.f, "tree_accept_sample: temperature must be > 0 (tree_accept is the greedy rule)");
  TV_REQUIRE((long long)B * Nmax <= 65535, "tree_accept_sample: B * Nmax must be <= 65535");
  if (workspace_bytes < tv_sample_workspace_bytes(B, Nmax, V))
    return tv::fail(TV_ERR_WORKSPACE, "tree_accept_sample: workspace of %zu bytes, need %zu", workspace_bytes,
                    tv_sample_workspace_bytes(B, Nmax, V));
  if (B == 0) return TV_OK;
  const int n_chunks = stat_chunks(V);
  const float k = kLog2e / temperature;
  RowStat* stats = static_cast<RowStat*>(workspace);
  cudaStream_t s = (cudaStream_t)stream;
  row_stats_kernel<<<dim3(n_chunks, B * Nmax), kStatThreads, 0, s>>>(logits, n_nodes, Nmax, V, n_chunks, k, stats);
  TV_CUDA_OK(cudaGetLastError());
  sample_walk_kernel<<<B, kWalkThreads, 0, s>>>(logits, stats, n_chunks, tokens, parent, n_nodes, u_node, u_bonus, k,
                                                Nmax, V, Dp1, accept_len, accepted_nodes, next_token, status);
  TV_CUDA_OK(cudaGetLastError());
  tv::count_launches(2);
  return TV_OK;
}
