// tree_build_mask: tree tensorisation (dummy-root remap, depth, ancestor table,
// structural invariants - Section 3.2) and the ancestor-or-self tree mask
// (Sections 2.4, 3.3) as per-row bit words plus an optional dense 4D mask.
//
// One CTA per sequence.  The work is a few KB of integer traffic per
// sequence, so the kernel is latency bound by design: a single launch, every
// array written once, all walks bounded because parent[i] < i is checked first.
#include "common.cuh"

namespace {

__global__ void __launch_bounds__(1024)
build_mask_kernel(const int32_t* __restrict__ parent, const int32_t* __restrict__ n_nodes,
                  int Nmax, int Dcap, int Pcap, int W,
                  uint32_t* __restrict__ anc_bits, uint8_t* __restrict__ dense,
                  int32_t* __restrict__ depth, int32_t* __restrict__ anc_table,
                  int32_t* __restrict__ retrieve, int32_t* __restrict__ n_paths,
                  int32_t* __restrict__ status) {
  tv::pdl_enter();
  extern __shared__ int32_t sm[];
  int32_t* sp = sm;                 // safe parent (sentinel and padding -> 0)
  int32_t* dep = sm + Nmax;
  int32_t* has_child = sm + 2 * Nmax;
  __shared__ int bad;
  __shared__ int n_leaves;

  const int b = blockIdx.x;
  const int tid = threadIdx.x;
  const int nt = blockDim.x;
  const int n_in = n_nodes[b];
  const bool n_ok = n_in >= 1 && n_in <= Nmax;
  const int n = n_ok ? n_in : 0;
  if (tid == 0) {
    bad = n_ok ? 0 : 1;
    n_leaves = 0;
  }
  __syncthreads();

  // Range + topological order; the sentinel of the root and every padded slot
  // become the dummy index 0, so all later walks stay inside [0, n).
  for (int i = tid; i < Nmax; i += nt) {
    int p = 0;
    if (i < n) {
      p = parent[(size_t)b * Nmax + i];
      if (i == 0) {
        if (p != -1) bad = 1;
        p = 0;
      } else if (p < 0 || p >= i) {
        bad = 1;
        p = 0;
      }
    }
    sp[i] = p;
    has_child[i] = 0;
  }
  __syncthreads();

  // Depth = number of parent steps to reach row 0 (strictly decreasing ids: at most i steps).
  for (int i = tid; i < Nmax; i += nt) {
    int steps = 0;
    if (i < n) {
      int cur = i;
      while (cur != 0) {
        cur = sp[cur];
        ++steps;
      }
      if (steps > Dcap) bad = 1;
      if (i > 0) has_child[sp[i]] = 1;
    }
    dep[i] = steps;
  }
  __syncthreads();

  const size_t rowbase = (size_t)b * Nmax;
  if (bad) {
    for (int i = tid; i < Nmax * W; i += nt) anc_bits[rowbase * W + i] = 0u;
    if (dense) for (int i = tid; i < Nmax * Nmax; i += nt) dense[rowbase * Nmax + i] = 0;
    if (depth) for (int i = tid; i < Nmax; i += nt) depth[rowbase + i] = 0;
    if (anc_table) for (int i = tid; i < (Dcap + 1) * Nmax; i += nt) anc_table[(size_t)b * (Dcap + 1) * Nmax + i] = 0;
    if (retrieve) for (int i = tid; i < Pcap * (Dcap + 1); i += nt) retrieve[(size_t)b * Pcap * (Dcap + 1) + i] = -1;
    if (tid == 0) {
      if (n_paths) n_paths[b] = 0;
      status[b] = TV_ST_BAD_TREE;
    }
    return;
  }

  // Bit rows, depth and the ancestor table: thread i owns column i / row i.
  for (int i = tid; i < Nmax; i += nt) {
    uint32_t* row = anc_bits + (rowbase + i) * W;
    for (int w = 0; w < W; ++w) row[w] = 0u;
    if (i < n) {
      int cur = i;
      while (true) {
        row[cur >> 5] |= 1u << (cur & 31);
        if (cur == 0) break;
        cur = sp[cur];
      }
    }
    if (depth) depth[rowbase + i] = dep[i];
    if (anc_table) {
      int cur = i;
      int32_t* col = anc_table + (size_t)b * (Dcap + 1) * Nmax + i;
      for (int l = 0; l <= Dcap; ++l) {
        col[(size_t)l * Nmax] = cur;
        cur = sp[cur];
      }
    }
  }
  if (retrieve)
    for (int i = tid; i < Pcap * (Dcap + 1); i += nt) retrieve[(size_t)b * Pcap * (Dcap + 1) + i] = -1;
  __syncthreads();   // the block's own global writes above are visible below

  if (dense) {
    for (int idx = tid; idx < Nmax * Nmax; idx += nt) {
      const int i = idx / Nmax, j = idx - i * Nmax;
      dense[rowbase * Nmax + idx] = (uint8_t)((anc_bits[(rowbase + i) * W + (j >> 5)] >> (j & 31)) & 1u);
    }
  }

  // One candidate row per leaf, leaves in increasing node id.
  for (int i = tid; i < n; i += nt) {
    if (has_child[i]) continue;
    int rank = 0;
    for (int j = 0; j < i; ++j) rank += has_child[j] ? 0 : 1;
    atomicAdd(&n_leaves, 1);
    if (retrieve && rank < Pcap) {
      int32_t* row = retrieve + ((size_t)b * Pcap + rank) * (Dcap + 1);
      int cur = i;
      for (int l = dep[i]; l >= 0; --l) {
        row[l] = cur;
        cur = sp[cur];
      }
    }
  }
  __syncthreads();
  if (tid == 0) {
    int st = 0;
    if (retrieve) {
      if (n_leaves > Pcap) st |= TV_ST_PATHS_TRUNCATED;
      n_paths[b] = n_leaves < Pcap ? n_leaves : Pcap;
    } else if (n_paths) {
      n_paths[b] = n_leaves;
    }
    status[b] = st;
  }
}

}  // namespace

extern "C" int tree_build_mask(const int32_t* parent, const int32_t* n_nodes,
                               int B, int Nmax, int Dcap, int Pcap,
                               uint32_t* anc_bits, uint8_t* dense_mask, int32_t* depth,
                               int32_t* anc_table, int32_t* retrieve_indices, int32_t* n_paths,
                               int32_t* status, tv_stream stream) {
  TV_REQUIRE(parent && n_nodes && anc_bits && status, "tree_build_mask: NULL required pointer");
  TV_REQUIRE(B >= 0 && Nmax >= 1 && Nmax <= 1024, "tree_build_mask: need B >= 0, 1 <= Nmax <= 1024");
  TV_REQUIRE(Dcap >= 0 && Dcap < Nmax, "tree_build_mask: need 0 <= Dcap < Nmax");
  TV_REQUIRE(!retrieve_indices || (Pcap >= 1 && n_paths), "tree_build_mask: retrieve_indices needs Pcap >= 1 and n_paths");
  if (B == 0) return TV_OK;
  const int W = (Nmax + 31) / 32;
  int threads = ((Nmax + 31) / 32) * 32;
  if (threads < 128) threads = 128;
  const size_t smem = 3 * (size_t)Nmax * sizeof(int32_t);
  TV_CUDA_OK(tv::launch_pdl(build_mask_kernel, dim3(B), dim3(threads), smem, (cudaStream_t)stream,
                            parent, n_nodes, Nmax, Dcap, Pcap, W, anc_bits, dense_mask, depth, anc_table,
                            retrieve_indices, n_paths, status));
  tv::count_launches(1);
  return TV_OK;
}
