/*
 * treeverify - the teacher tree-verification step of EAGLE-3-style tree
 * speculative decoding, as a C-ABI library of sm_100a CUDA kernels.
 *
 * One step = tree_build_mask, then tree_verify_attn once per layer, then
 * tree_accept, then kv_commit, all enqueued on one stream.  No call
 * synchronises, allocates or keeps state (except tv_verify_step_host, which
 * waits for its own copies); every launch is asynchronous on the stream given.
 *
 * Conventions
 *   - Pointers are DEVICE pointers owned by the caller unless a parameter is
 *     marked "host".  Arrays are dense, row-major, last index fastest.
 *   - tv_bf16 is the raw 16-bit pattern of a bfloat16.
 *   - Node 0 of every tree is the root (the last sampled token): it is a
 *     real query row with its own K/V and logits, parent[0] = -1 is the only
 *     sentinel, and 0 is the dummy index every sentinel is remapped to
 *     before a gather (Section 3.2, "Dummy-root indexing", with N = M + 1).
 *   - n_nodes[b] <= Nmax nodes of sequence b are active; slots past it are
 *     padding and can never influence an active output (Section 3.2,
 *     "Padding and batch semantics"; Section 3.3, "No leakage to padded slots").
 *   - Return value: TV_OK or a TV_ERR_* code for errors the host can see
 *     (nothing is launched then); tv_last_error() gives a message.
 *   - Data-dependent errors are reported per sequence in status[B] (device,
 *     bit field TV_ST_*).  tree_build_mask overwrites status[b]; the other
 *     calls OR into it.  A sequence with a fatal bit gets no commit.
 */
#ifndef TREEVERIFY_H_
#define TREEVERIFY_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define TV_API __attribute__((visibility("default")))
#else
#define TV_API
#endif

typedef uint16_t tv_bf16;
typedef void* tv_stream;      /* a cudaStream_t; NULL is the legacy default stream */

enum {
  TV_OK = 0,
  TV_ERR_INVALID_ARG = 1,     /* NULL pointer, bad dimension, unsupported shape, misalignment */
  TV_ERR_CUDA = 2,            /* a launch, copy or tensor-map encode failed */
  TV_ERR_WORKSPACE = 3        /* workspace smaller than tv_*_workspace_bytes says */
};

enum {
  TV_ST_BAD_TREE = 1,         /* a structural invariant of the tree failed (fatal) */
  TV_ST_BAD_INDEX = 2,        /* a path / node index outside its range (fatal) */
  TV_ST_CAPACITY = 4,         /* the accepted segment does not fit the cache (fatal) */
  TV_ST_TIMEOUT = 8,          /* a bounded wait inside a kernel expired (fatal) */
  TV_ST_PATHS_TRUNCATED = 16  /* more leaves than path rows; the first Pcap were kept */
};

/* Message of the last TV_ERR_* returned on this host thread ("" if none). */
TV_API const char* tv_last_error(void);

/* Library version, major*100 + minor. */
TV_API int tv_version(void);

/* Number of kernels this library has launched in this process so far
 * (diagnostics: lets a caller verify that its work ran in these kernels). */
TV_API unsigned long long tv_launch_count(void);

/*
 * Tree tensorisation and tree mask (Section 3.2: dummy-root remap, depth,
 * ancestor table A[0,k]=k, A[l+1,k]=parent~(A[l,k]), structural invariants;
 * Section 2.4 / 3.3: node k sees node j iff j is an ancestor of k or k itself
 * and both are valid).
 *
 *   parent[B,Nmax]  in  parent[b,0] must be -1; 0 <= parent[b,i] < i for
 *                       1 <= i < n_nodes[b] (topological order); slots past
 *                       n_nodes[b] are ignored.
 *   n_nodes[B]      in  1..Nmax
 *   Dcap                largest depth (edges from the root) a node may have
 *   Pcap                rows of retrieve_indices
 *   anc_bits[B,Nmax,W]  out, W = ceil(Nmax/32): bit (j%32) of word j/32 of
 *                       row i is set iff i sees j.  Required.
 *   dense_mask[B,1,Nmax,Nmax] out or NULL: 1 = visible, 0 = masked (the
 *                       additive mask of Section 2.4 is visible ? 0 : -inf).
 *   depth[B,Nmax]       out or NULL
 *   anc_table[B,Dcap+1,Nmax] out or NULL; every entry is in [0,Nmax).
 *   retrieve_indices[B,Pcap,Dcap+1] out or NULL: one row per leaf, leaves in
 *                       increasing node id, root first, -1 after the leaf and
 *                       in unused rows.
 *   n_paths[B]          out or NULL (required with retrieve_indices)
 *   status[B]           out: 0, TV_ST_BAD_TREE (all outputs of the sequence
 *                       zero, its retrieve rows -1) or TV_ST_PATHS_TRUNCATED.
 * Limits: 1 <= Nmax <= 1024, 0 <= Dcap < Nmax.
 */
TV_API int tree_build_mask(const int32_t* parent, const int32_t* n_nodes,
                    int B, int Nmax, int Dcap, int Pcap,
                    uint32_t* anc_bits, uint8_t* dense_mask, int32_t* depth,
                    int32_t* anc_table, int32_t* retrieve_indices, int32_t* n_paths,
                    int32_t* status, tv_stream stream);

/* Flags of tree_verify_attn_layers. */
enum {
  TV_ATTN_LAUNCH_PER_LAYER = 2, /* one launch per layer, exactly as L calls of tree_verify_attn would issue them (for
                                 comparison; the default is one launch for all layers) */
  TV_ATTN_STABLE_INPUTS = 1   /* the caller promises: the kernel directly in front of this call on the stream does
                                 not write prefix_len, n_nodes or rows [0, prefix_len) of the cache - or it does, but
                                 lets no successor start before it has completed.  tree_build_mask in front (the
                                 usual step) satisfies it; kv_commit in front does not. */
};

/* Scratch needed by tree_verify_attn and tree_verify_attn_layers for these dimensions (bytes). */
TV_API size_t tv_attn_workspace_bytes(int B, int Nmax, int Hq, int Hkv, int d, int Scap);

/*
 * Tree attention of one layer: the attention sub-step of TeacherTreeEval
 * (Section 2.3) under the tree mask (Section 3.3).  Every active node i and
 * query head h (KV head h / (Hq/Hkv)) attends the committed prefix rows
 * [0, prefix_len[b]) of the cache and the tree keys j whose bit is set in
 * anc_bits[b,i]; softmax of scale * <q,k> with fp32 accumulation.
 *
 *   q[B,Nmax,Hq,d]                 in  bf16
 *   k_cache,v_cache[B,Hkv,Scap,d]  in  bf16, one layer; never written
 *                                      (state safety, Section 3.3); rows at
 *                                      or past prefix_len[b] are ignored even
 *                                      if they hold NaN.
 *   k_tree,v_tree[B,Nmax,Hkv,d]    in  bf16, the speculative ("branch") K/V;
 *                                      or both NULL = in-cache layout: the
 *                                      teacher forward extended the cache in
 *                                      place (Section 3.1) and node i's K/V
 *                                      are rows prefix_len[b] + i of k_cache /
 *                                      v_cache, written behind the committed
 *                                      prefix and not part of it until
 *                                      kv_commit_inplace.  A tree that does not
 *                                      fit (prefix_len[b] + n_nodes[b] > Scap)
 *                                      gets TV_ST_CAPACITY and an unspecified
 *                                      output.
 *   prefix_len[B], n_nodes[B]      in
 *   anc_bits[B,Nmax,W]             in  from tree_build_mask
 *   out[B,Nmax,Hq,d]               out bf16; padded rows are written as 0
 *   lse[B,Hq,Nmax]                 out or NULL, fp32 log-sum-exp of the
 *                                      scaled scores; -inf for padded rows
 *   workspace                      device scratch, 256-byte aligned, at least
 *                                      tv_attn_workspace_bytes(...) bytes; needs
 *                                      no initialisation; calls that share one
 *                                      must be issued in one stream
 *   status[B]                      in/out: TV_ST_TIMEOUT is ORed in if a
 *                                      bounded wait expired (outputs invalid)
 * Limits: d in {64,128}; Nmax <= 256 (the node budgets of the paper's sweep);
 * Hq % Hkv == 0, Hq / Hkv <= 128; B <= 512; all tensors 16-byte aligned;
 * 0 <= prefix_len[b] <= Scap; scale > 0.
 * CUDA graphs: every call of this header only launches on the given stream, so a
 * step can be captured into a CUDA graph and replayed; the split-KV counters in
 * the workspace are cleared by the piece that merges, so a replay (which
 * repeats the call's internal epoch) finds them unused.
 * Stream order: the kernel is launched with programmatic stream serialisation,
 * so it may be scheduled while the kernel in front of it still runs (if that
 * kernel allows it), but it reads and writes nothing of the problem before
 * every earlier kernel of the stream has finished: only its own set-up
 * (barriers, tensor memory, descriptor fetch) overlaps.  Reading
 * the committed prefix earlier than that is what tree_verify_attn_layers
 * offers, under a promise by the caller.
 */
TV_API int tree_verify_attn(const tv_bf16* q,
                     const tv_bf16* k_cache, const tv_bf16* v_cache,
                     const tv_bf16* k_tree, const tv_bf16* v_tree,
                     const int32_t* prefix_len, const int32_t* n_nodes,
                     const uint32_t* anc_bits,
                     int B, int Nmax, int Hq, int Hkv, int d, int Scap, float scale,
                     tv_bf16* out, float* lse,
                     void* workspace, size_t workspace_bytes,
                     int32_t* status, tv_stream stream);

/*
 * tree_verify_attn for all L layers of a step in one call (Section 2.3: the
 * teacher evaluates the whole tree in one forward; every layer attends under
 * the same mask and the same prefix lengths).  Layer l reads q, k_cache,
 * v_cache, k_tree, v_tree (both NULL: in-cache layout) at l times the given
 * layer stride (elements), writes out at l * out_layer_stride and lse (dense
 * [L,B,Hq,Nmax], or NULL).  Arguments, limits and results are those of
 * tree_verify_attn, layer by layer (outputs agree with L single calls to the
 * rounding of the split-KV partials: units are cut at other places).
 * What it adds: the inputs of all layers are there when the call is made, so
 * all layers run in ONE launch - their (sequence, KV head) units form one
 * tile space that is cut evenly over the SMs - with one pipeline fill, one
 * tail and at most one cut unit per SM for the whole step instead of per
 * layer.  The workspace of tv_attn_workspace_bytes holds the counters of 32
 * layers per launch; more layers (or a smaller workspace, down to the
 * counters of one layer) are served by more launches.  A caller whose layers
 * depend on each other has to issue single-layer calls instead.
 * flags: TV_ATTN_STABLE_INPUTS lets the launch read prefix_len, n_nodes and
 * committed-prefix rows while the kernel in front still runs (see the flag);
 * TV_ATTN_LAUNCH_PER_LAYER issues one launch per layer, as L single calls
 * would (for comparison).
 */
TV_API int tree_verify_attn_layers(const tv_bf16* q,
                     const tv_bf16* k_cache, const tv_bf16* v_cache,
                     const tv_bf16* k_tree, const tv_bf16* v_tree,
                     const int32_t* prefix_len, const int32_t* n_nodes,
                     const uint32_t* anc_bits,
                     int L, int B, int Nmax, int Hq, int Hkv, int d, int Scap, float scale,
                     int64_t q_layer_stride, int64_t cache_layer_stride, int64_t tree_layer_stride,
                     tv_bf16* out, int64_t out_layer_stride, float* lse,
                     void* workspace, size_t workspace_bytes,
                     int32_t* status, unsigned flags, tv_stream stream);

/*
 * tree_verify_attn over a paged committed cache (Section 3.1 speaks of
 * backend-specific KV layouts behind one cache interface; this is the block
 * layout of serving stacks).  A page holds 128 consecutive rows - one key tile
 * of the kernel - of all KV heads: k_pages, v_pages [n_pages,Hkv,128,d] bf16
 * (one layer).  block_table[B,max_blocks] names, for sequence b, the page of
 * rows 128 t .. 128 t + 127 at [b, t]; only entries t < ceil(prefix_len[b]/128)
 * are read.  The capacity of a sequence is 128 * max_blocks rows.  The tree's
 * K/V come in their own buffers.  Everything else - arguments, outputs,
 * workspace (tv_attn_workspace_bytes with any Scap), limits, stream order - is
 * as for tree_verify_attn.  A page id outside [0, n_pages) raises
 * TV_ST_BAD_INDEX for the sequence (its output is unspecified; nothing is
 * read outside the pool).
 */
TV_API int tree_verify_attn_paged(const tv_bf16* q,
                     const tv_bf16* k_pages, const tv_bf16* v_pages,
                     const int32_t* block_table,
                     const tv_bf16* k_tree, const tv_bf16* v_tree,
                     const int32_t* prefix_len, const int32_t* n_nodes,
                     const uint32_t* anc_bits,
                     int B, int Nmax, int Hq, int Hkv, int d, int n_pages, int max_blocks, float scale,
                     tv_bf16* out, float* lse,
                     void* workspace, size_t workspace_bytes,
                     int32_t* status, tv_stream stream);

/*
 * tree_verify_attn_paged for all L layers of a step in one launch: k_pages,
 * v_pages [L,n_pages,Hkv,128,d] with layer stride page_layer_stride (elements;
 * the layout kv_commit_paged writes), one block table for all layers.
 * Otherwise as tree_verify_attn_layers (flags: TV_ATTN_STABLE_INPUTS, which
 * here also covers the block table).
 */
TV_API int tree_verify_attn_paged_layers(const tv_bf16* q,
                     const tv_bf16* k_pages, const tv_bf16* v_pages,
                     const int32_t* block_table,
                     const tv_bf16* k_tree, const tv_bf16* v_tree,
                     const int32_t* prefix_len, const int32_t* n_nodes,
                     const uint32_t* anc_bits,
                     int L, int B, int Nmax, int Hq, int Hkv, int d, int n_pages, int max_blocks, float scale,
                     int64_t q_layer_stride, int64_t page_layer_stride, int64_t tree_layer_stride,
                     tv_bf16* out, int64_t out_layer_stride, float* lse,
                     void* workspace, size_t workspace_bytes,
                     int32_t* status, unsigned flags, tv_stream stream);

/* Scratch needed by tree_accept (bytes). */
TV_API size_t tv_accept_workspace_bytes(int B, int Nmax, int V);

/*
 * Safe path gather, teacher argmax and greedy acceptance.
 *   - gather (Section 2.5; Section 3.2): an index r of a candidate row is
 *     usable iff 0 <= r < n_nodes[b]; every other value is remapped to the
 *     dummy index 0 BEFORE tokens[] is read, and the slot is excluded from
 *     acceptance by its validity flag.  r < -1 or r >= n_nodes[b] also
 *     raises TV_ST_BAD_INDEX.
 *   - argmax (greedy selection, Section 2.1, temperature 0 as in Section 5):
 *     the lowest v that maximises logits[b,i,v]; values compare as floats;
 *     inputs are NaN-free by contract (a NaN never wins).
 *   - accept (Section 2.3): along each row, node j is accepted while its
 *     token equals the teacher argmax at node j-1 of the row; the longest
 *     accepted prefix over all rows wins, ties go to the lowest row.
 *
 *   logits[B,Nmax,V]          in  bf16
 *   tokens[B,Nmax]            in  draft token of every node (node 0: the last sampled token)
 *   retrieve_indices[B,P,Dp1] in  left-aligned root-to-leaf rows, -1 padded
 *   argmax_tok[B,Nmax]        out (-1 for padded rows)
 *   safe_idx,candidates[B,P,Dp1] out or NULL
 *   accept_len[B]             out accepted draft tokens, 0..Dp1-1 (root and bonus token not counted)
 *   best_path[B]              out winning row
 *   accepted_nodes[B,Dp1]     out first accept_len+1 entries = root..last accepted node, rest 0
 *   next_token[B]             out teacher argmax at the last accepted node (the bonus token)
 *   workspace                 device scratch >= tv_accept_workspace_bytes(B,Nmax,V), 16-byte aligned
 *   status[B]                 in/out
 */
TV_API int tree_accept(const tv_bf16* logits, const int32_t* tokens,
                const int32_t* retrieve_indices, const int32_t* n_nodes,
                int B, int Nmax, int V, int P, int Dp1,
                int32_t* argmax_tok, int32_t* safe_idx, int32_t* candidates,
                int32_t* accept_len, int32_t* best_path, int32_t* accepted_nodes,
                int32_t* next_token,
                void* workspace, size_t workspace_bytes,
                int32_t* status, tv_stream stream);

/*
 * Node verification scores (Section 3.3, "Mapping teacher outputs to node
 * verification scores"): the teacher's logit of every node's proposed token,
 * taken from the logits row of the node's parent slot (that row predicts the
 * node's token): scores[b,k] = logits[b, parent~[b,k], tokens[b,k]], the input
 * of a score-based (non-greedy) acceptance rule.  An in-range gather over the
 * vocabulary, guarded by valid: the sentinel parent is remapped to 0, the root
 * and padded slots give 0, a token outside [0,V) gives -inf and raises
 * TV_ST_BAD_INDEX (its index is remapped to 0 before the gather).
 *   logits[B,Nmax,V] bf16, tokens[B,Nmax], parent[B,Nmax], n_nodes[B]  in
 *   scores[B,Nmax] fp32  out;  status[B]  in/out
 */
TV_API int tree_node_scores(const tv_bf16* logits, const int32_t* tokens, const int32_t* parent,
                            const int32_t* n_nodes, int B, int Nmax, int V, float* scores,
                            int32_t* status, tv_stream stream);

/*
 * Attention over a key set that was split in R disjoint ranges (Section 6,
 * "Limitations and future work": longer-context workloads and multi-device
 * serving; the attention is Section 2.4).  Each member of a context-split group
 * runs tree_verify_attn over its own range of the committed prefix (the tree's
 * keys belong to exactly one member; the others pass all-zero anc_bits) and
 * keeps out and lse; after the partials of all members have been gathered into
 * local memory, this call combines them per query row:
 *   out = sum_r w_r O_r / sum_r w_r,  w_r = exp(lse_r - max_r lse_r),
 *   lse = max_r lse_r + log sum_r w_r.
 * A range without visible keys has lse_r = -inf and weight 0 (its O_r is not
 * read); a row without any key gives zeros and -inf.
 *   o_parts[R,B,Nmax,Hq,d] bf16, lse_parts[R,B,Hq,Nmax] fp32 (natural log)  in, device, local memory
 *   out[B,Nmax,Hq,d] bf16  out;  lse[B,Hq,Nmax] fp32  out, may be NULL
 * d must be a multiple of 8, o_parts and out 16-byte aligned.
 */
TV_API int tree_merge_partials(const tv_bf16* o_parts, const float* lse_parts, int R, int B, int Nmax, int Hq, int d,
                               tv_bf16* out, float* lse, tv_stream stream);

/*
 * tree_accept for callers that cannot allocate device memory (the paper has
 * no counterpart; this is a convenience of this library).  Some hosts of this
 * code may not call cudaMalloc at all: a plugin inside a serving runtime that
 * owns the whole memory pool, code running while another component captures a
 * stream, or a process whose allocator budget is fixed at start-up.  For them
 * the scratch of the argmax reduction is a fixed 256 KiB array inside the
 * library image (every GPU that loads the library holds it until exit).
 * Same arguments and results as tree_accept, without the workspace.
 *   - Limit: B * Nmax * ceil(V / 16384) <= 32768 scratch entries
 *     (tv_accept_noalloc_max_bytes() / 8); larger problems are rejected with
 *     TV_ERR_WORKSPACE and must use tree_accept.
 *   - The first call on each device looks up the array's device address (with
 *     that device current); make that first call outside any stream capture.
 *   - All calls on a device share the one array, which keeps the previous
 *     call's contents.  Nothing in it has to start at zero (every entry that
 *     is read is written first by the same call), but two calls whose kernels
 *     overlap on the GPU (different streams) race on it: serialise them.
 *   - No cudaMalloc, cudaFree or allocating library routine is called.
 */
TV_API size_t tv_accept_noalloc_max_bytes(void);
TV_API int tree_accept_noalloc(const tv_bf16* logits, const int32_t* tokens,
                               const int32_t* retrieve_indices, const int32_t* n_nodes,
                               int B, int Nmax, int V, int P, int Dp1,
                               int32_t* argmax_tok, int32_t* safe_idx, int32_t* candidates,
                               int32_t* accept_len, int32_t* best_path, int32_t* accepted_nodes,
                               int32_t* next_token, int32_t* status, tv_stream stream);

/* Scratch needed by tree_accept_sample (bytes). */
TV_API size_t tv_sample_workspace_bytes(int B, int Nmax, int V);

/*
 * Sampling-mode acceptance (temperature > 0) over the tree.  Section 2.2 asks
 * for an acceptance rule "rejection sampling style" under which the output
 * keeps the teacher's distribution, Section 3.3 names the node scores as its
 * input; no formula is printed, so this is the reading: speculative sampling
 * for proposals without a draft probability (q = one-hot on the proposed
 * token), walked down the tree.  With p = softmax(logits[b,c,:] / temperature)
 * at the current node c (the root first):
 *   - the children of c (parent[k] = c after the dummy-root remap, valid
 *     slots, increasing node id) are tried in turn; a token already rejected
 *     at c is skipped; child k with token x is accepted iff
 *       u_node[b,k] < p(x) / (1 - mass rejected so far at c);
 *     otherwise x is rejected and its mass removed;
 *   - an accepted child becomes the current node (at most Dp1 - 1 of them);
 *   - when no child passes, next_token is drawn from p without the rejected
 *     tokens: the first v whose cumulative mass in vocabulary order exceeds
 *     u_bonus[b] times the remaining mass.
 * Every token that leaves the step is then distributed as under plain
 * sampling from the teacher; temperature -> 0 gives tree_accept's greedy rule.
 * The uniforms are inputs (the library draws nothing): u_node[B,Nmax] and
 * u_bonus[B], float32 in [0,1).  All probabilities are computed in fp32.
 *
 *   logits[B,Nmax,V] bf16, tokens[B,Nmax], parent[B,Nmax], n_nodes[B]   in
 *   accept_len[B], accepted_nodes[B,Dp1] (first accept_len+1 valid, rest 0),
 *   next_token[B] (-1 for a sequence without nodes)                     out
 *   status[B]  in/out: TV_ST_BAD_INDEX is ORed in if a valid non-root slot
 *              proposes a token outside [0,V) (that child is never accepted).
 * The tree is taken as validated by tree_build_mask (parent[k] < k).
 * Limits: Nmax <= 256, B * Nmax <= 65535, temperature > 0.
 */
TV_API int tree_accept_sample(const tv_bf16* logits, const int32_t* tokens, const int32_t* parent,
                              const int32_t* n_nodes, const float* u_node, const float* u_bonus,
                              float temperature, int B, int Nmax, int V, int Dp1,
                              int32_t* accept_len, int32_t* accepted_nodes, int32_t* next_token,
                              void* workspace, size_t workspace_bytes,
                              int32_t* status, tv_stream stream);

/*
 * Path-index commit with the prefix-sharing fast reorder (Section 3.1): the
 * committed prefix keeps its place and only the accepted segment is gathered
 * behind it, in place, for all layers in one call:
 *   cache[l,b,h,prefix_len[b]+j,:] = tree[l,b,accepted_nodes[b,j],h,:], j = 0..accept_len[b]
 *   prefix_len[b] += accept_len[b] + 1
 * A chain tree makes this the length-based commit of Section 3.1.
 *
 *   k_cache,v_cache   in/out [L,B,Hkv,Scap,d] with layer stride cache_layer_stride (elements)
 *   k_tree,v_tree     in     [L,B,Nmax,Hkv,d] with layer stride tree_layer_stride (elements)
 *   accepted_nodes[B,Dp1], accept_len[B]  in (device; read by the kernel)
 *   prefix_len[B]     in/out
 *   status[B]         in/out: a sequence with a fatal bit already set is
 *                     skipped; TV_ST_CAPACITY if the segment would pass Scap,
 *                     TV_ST_BAD_INDEX if accept_len or a node id is out of
 *                     range; such a sequence is left untouched.
 * Must follow the last tree_verify_attn of the step on the same stream.
 * Limits: d*2 bytes a multiple of 16; tensors 16-byte aligned; Dp1 <= 1024;
 * L <= 65535.
 */
TV_API int kv_commit(tv_bf16* k_cache, tv_bf16* v_cache,
              const tv_bf16* k_tree, const tv_bf16* v_tree,
              const int32_t* accepted_nodes, const int32_t* accept_len,
              int32_t* prefix_len,
              int L, int B, int Nmax, int Hkv, int d, int Scap, int Dp1,
              int64_t cache_layer_stride, int64_t tree_layer_stride,
              int32_t* status, tv_stream stream);

/*
 * kv_commit on the paged cache of tree_verify_attn_paged: accepted row j of
 * sequence b goes to row (S+j) % 128 of page block_table[b, (S+j) / 128],
 * S = prefix_len[b], for all layers; prefix_len[b] += accept_len[b] + 1.  The
 * pages under the accepted segment must already be in the block table (the
 * caller allocates pages; the library never does).
 *   k_pages,v_pages   in/out [L,n_pages,Hkv,128,d] with layer stride page_layer_stride (elements)
 *   k_tree,v_tree     in     [L,B,Nmax,Hkv,d] with layer stride tree_layer_stride
 *   status[B]         in/out as for kv_commit; capacity = 128 * max_blocks;
 *                     TV_ST_BAD_INDEX also for a page id outside [0, n_pages)
 *                     under the segment.  A flagged sequence is left untouched.
 * Limits as for kv_commit; max_blocks <= 2^20.
 */
TV_API int kv_commit_paged(tv_bf16* k_pages, tv_bf16* v_pages, const int32_t* block_table,
              const tv_bf16* k_tree, const tv_bf16* v_tree,
              const int32_t* accepted_nodes, const int32_t* accept_len,
              int32_t* prefix_len,
              int L, int B, int Nmax, int Hkv, int d, int n_pages, int max_blocks, int Dp1,
              int64_t page_layer_stride, int64_t tree_layer_stride,
              int32_t* status, tv_stream stream);

/*
 * Path-index commit as a full reorder inside the cache (Section 3.1, "full
 * reordering"), for the in-cache layout of tree_verify_attn: node i's K/V are
 * rows prefix_len[b] + i, and the accepted path is gathered to the front of
 * that region, for all layers in one call:
 *   cache[l,b,h,S+j,:] = OLD cache[l,b,h,S+accepted_nodes[b,j],:], j = 0..accept_len[b], S = prefix_len[b]
 *   prefix_len[b] += accept_len[b] + 1
 * Source and destination rows overlap (with accepted_nodes = {0,2,3} row S+2
 * is the source of slot 1 and the destination of slot 2), so every source row
 * is read before any row is written: the result is the gather from the state
 * before the call, whatever the order of the node ids.  Rows behind the
 * accepted segment keep their (now stale) speculative contents; rows below S
 * are never touched.
 *
 *   k_cache,v_cache   in/out [L,B,Hkv,Scap,d] with layer stride cache_layer_stride (elements)
 *   accepted_nodes[B,Dp1], accept_len[B]  in (device)
 *   prefix_len[B]     in/out
 *   status[B]         in/out, as for kv_commit; TV_ST_CAPACITY also if a
 *                     source row S + node lies at or past Scap.
 * Limits: Dp1 * d / 8 <= 2048; d*2 bytes a multiple of 16; tensors 16-byte
 * aligned; Hkv <= 32767.
 */
TV_API int kv_commit_inplace(tv_bf16* k_cache, tv_bf16* v_cache,
              const int32_t* accepted_nodes, const int32_t* accept_len,
              int32_t* prefix_len,
              int L, int B, int Nmax, int Hkv, int d, int Scap, int Dp1,
              int64_t cache_layer_stride,
              int32_t* status, tv_stream stream);

/*
 * One whole verification step driven from HOST buffers (Section 3 call
 * order: tensorise + mask, attention per layer, gather + accept, commit).
 * Per-step inputs are copied host->device into `staging`, the four calls
 * above run, and the per-step results are copied back; the call returns after
 * the stream has drained.  The KV cache and prefix_len stay resident on the
 * device (they are the committed state, not a per-step input).
 */
typedef struct tv_step_host_args {
  /* host, pinned memory recommended */
  const int32_t* parent;            /* [B,Nmax] */
  const int32_t* n_nodes;           /* [B] */
  const int32_t* tokens;            /* [B,Nmax] */
  const int32_t* retrieve_indices;  /* [B,P,Dp1] or NULL: use the rows tree_build_mask emits */
  const tv_bf16* q;                 /* [L,B,Nmax,Hq,d] */
  const tv_bf16* k_tree;            /* [L,B,Nmax,Hkv,d] */
  const tv_bf16* v_tree;            /* [L,B,Nmax,Hkv,d] */
  const tv_bf16* logits;            /* [B,Nmax,V] */
  tv_bf16* out;                     /* [L,B,Nmax,Hq,d] host out */
  int32_t* accept_len;              /* [B] host out */
  int32_t* accepted_nodes;          /* [B,Dp1] host out */
  int32_t* next_token;              /* [B] host out */
  int32_t* status;                  /* [B] host out */
  /* device, resident */
  tv_bf16* k_cache;                 /* [L,B,Hkv,Scap,d] */
  tv_bf16* v_cache;
  int32_t* prefix_len;              /* [B] in/out */
  void* staging;                    /* device scratch >= tv_step_staging_bytes(...) , 256-byte aligned */
  size_t staging_bytes;
  int L, B, Nmax, Hq, Hkv, d, Scap, V, P, Dp1;
  float scale;
  tv_stream stream;
} tv_step_host_args;

TV_API size_t tv_step_staging_bytes(int L, int B, int Nmax, int Hq, int Hkv, int d, int Scap, int V, int P, int Dp1);
TV_API int tv_verify_step_host(const tv_step_host_args* args);

#ifdef __cplusplus
}
#endif
#endif /* TREEVERIFY_H_ */
