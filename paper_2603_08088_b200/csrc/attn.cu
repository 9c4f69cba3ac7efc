// tree_verify_attn: GQA tree attention for sm_100a (Sections 2.3, 2.4, 3.3).
//
// Packing.  For one sequence b and KV head hk, the G = Hq/Hkv query heads of
// every tree node share the same K/V, so (node, group member) pairs are packed
// into dense MMA rows r = node_local * G + g.  A row tile holds 128 rows =
// 128/G nodes; a CTA owns MT (1 or 2) row tiles and streams 128-key tiles of
// the committed prefix, then one tile of the tree's own keys.
//
// Pipeline (one CTA per SM, 12 warps):
//   warp 0      TMA producer: Q tiles once per work item, then K and V tiles
//               through a 5-slot shared-memory ring (128-byte swizzled boxes).
//   warp 1      tcgen05.mma issuer (one thread): S = Q K^T for a whole 128-key
//               tile (N = 128; 64-key MMAs re-read Q from shared memory twice as
//               often and run at 2/3 of the rate), O += P V with P read from
//               TMEM; completion goes to mbarriers with tcgen05.commit.  With
//               two row tiles it serves them in turn, so the softmax of one row
//               tile runs while the tensor pipe works for the other.
//   warps 4-7   softmax warpgroup for row tile 0: one thread per row, online
//   warps 8-11  softmax with lazy rescale; tile 1 likewise.  The ancestor
//               bitmask of the row is applied only on the tree tile(s), the
//               prefix length only on the ragged last prefix tile.
// TMEM: S0 | S1 | O0 | O1, 128 columns each; P (bf16) overlays the first 64
// columns of its S.  With one row tile the two S buffers alternate by key tile.
//
// Code size matters here: instruction fetches compete with the K/V stream for
// L2 and HBM, and code that runs once per work item (set-up, epilogue, merge)
// is fetched cold every time.  Cold paths are therefore written as loops, not
// unrolled, and the timeline marks are compiled out unless -DTV_TRACE is given.
//
// Work split.  All key tiles of all (layer, b, hk) units of the launch - one
// layer, or all layers of a step - form one linear space that
// is cut evenly over the CTA groups (a group = the CTAs that hold the row
// tiles of the same unit and walk the same keys together, so the second reader
// hits L2).  A unit cut in pieces leaves partials (normalised O in bf16, m, l) in the
// workspace; the piece that draws the last ticket on the unit's counter merges them.
// Counters carry a per-call epoch, so the workspace needs no initialisation.
//
// Every wait on an mbarrier is bounded: on expiry the CTA raises
// TV_ST_TIMEOUT for all sequences, all roles leave their loops, outstanding
// copies are given time to land, TMEM is freed and the kernel returns.
#include "common.cuh"
#include "treeverify_debug.h"

#include <cuda.h>
#include <cuda_bf16.h>

#include <atomic>
#include <chrono>

namespace {

constexpr int kTileN = 128;        // keys per tile
constexpr int kTileM = 128;        // rows per row tile
constexpr int kSlots = 5;          // K/V ring slots
constexpr int kThreads = 384;
constexpr int kMaxB = 512;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;            // in log2 units
constexpr float kMaxFastSum = 16384.0f;               // 64 keys x 2^threshold: largest row sum the fast path accepts
// Of every 16 element pairs of the softmax fast path, three take 2^x on the FMA pipe (measured optimum between
// the special-function unit and the FMA pipe: 2/16 and 4/16 are 1-2 % slower on the 32-layer and the
// long-context shape, 1/16 and 5/16 far slower).
#ifndef TV_POLY_SEL
#define TV_POLY_SEL(i) ((((i) & 7) == 3) || (((i) & 15) == 7))
#endif
constexpr unsigned long long kWaitLimitNs = 2000000000ull;
// virtual tiles charged per unit by the scheduler (32-layer shape, five seeds: 2 is 0.2-2 % faster than 4,
// 0 and 1 are slower)
#ifndef TV_SETUP_COST
#define TV_SETUP_COST 2
#endif
constexpr int kSetupCost = TV_SETUP_COST;
constexpr int kMaxGroups = 160;
// do not spread a small problem over more CTA groups than this allows (measured on the 7B-shaped single
// sequence: 12 -> 26 us, 6 -> 22 us, 4 -> 23 us per launch)
#ifndef TV_MIN_VT
#define TV_MIN_VT 6
#endif
constexpr int kMinVirtualTilesPerGroup = TV_MIN_VT;
constexpr int kTraceCap = 256;     // events per (CTA, role) kept by the optional trace

// ---------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the wait was abandoned (timeout here or abort raised elsewhere).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          unsigned long long limit_ns) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++spins & 255u) == 0) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > limit_ns) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// Programmatic dependent launch.  gdc_wait: every kernel launched before this one in the stream has finished and
// its writes are visible.  gdc_launch_dependents: the next kernel in the stream may be scheduled once every CTA of
// this grid has got here or has exited.
__device__ __forceinline__ void gdc_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void gdc_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// One lane of a converged warp (the compiler keeps what it guards in the uniform datapath).
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
  return pred != 0;
}
// 32 bytes per thread in one store (a whole sector); the address must be 32-byte aligned.
__device__ __forceinline__ void st_global_32B(void* p, uint4 a, uint4 b) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w),
               "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Tiled TMA loads.  The one for the cache carries an L2 eviction-priority hint: the committed K/V prefix is read once per
// launch, and letting it leave L2 first keeps Q, the partials and the kernel's own code resident.
// (The outermost coordinate of every tensor is the layer.)
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                                 int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                            int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;
  d |= 2ull << 61;
  return d;
}
// Instruction descriptor, kind::f16: bf16 x bf16 -> fp32, M = 128, A K-major.
__host__ __device__ constexpr uint32_t instr_desc(int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(kTileM >> 4) << 24);
}
// tcgen05.mma, kind::f16, one CTA.  The 64-bit shared-memory descriptors are given as (low, high) words: the
// high word of every descriptor used here is one constant, so the issuing thread only adds an offset to a
// low word per MMA.
__device__ __forceinline__ void mma_ss_lohi(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                            uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void mma_ts_lohi(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                            uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
        "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]),
        "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]),
        "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Optional timeline for tuning: role r of this CTA appends (tag, time since kernel start of CTA 0).
struct Tracer {
  unsigned long long* base;
  int n;
  __device__ __forceinline__ void init(unsigned long long* trace, int role) {
    base = trace ? trace + ((size_t)blockIdx.x * 4 + role) * kTraceCap : nullptr;
    n = 0;
  }
  __device__ __forceinline__ void mark(uint32_t tag) {
#ifndef TV_TRACE
    (void)tag;        // compiled out: even switched off, the marks cost several per cent of the kernel's time
    return;
#endif
    if (base && n < kTraceCap) base[n++] = ((unsigned long long)tag << 48) | (globaltimer_ns() & 0xffffffffffffull);
  }
};

#ifdef TV_PROF
#define TV_PROF_T(var) do { var = clock(); } while (0)
#define TV_PROF_USE(x) asm volatile("{.reg .b32 t; mov.b32 t, %0;}" ::"r"(x))
#else
#define TV_PROF_T(var) do { } while (0)
#define TV_PROF_USE(x) do { } while (0)
#endif
// Packed fp32 pair arithmetic (one issue slot for two lanes of work).
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) { return __fadd2_rn(a, b); }
// 2^x for a pair on the FMA pipe (the special-function unit is the scarce resource of the softmax):
// x = n + f with n = round(x), f in [-0.5, 0.5]; 2^f by a cubic (relative error 7.5e-5, far below the
// bf16 rounding of P), 2^n by an add into the exponent field.  x is clamped to [-125, 16].
__device__ __forceinline__ float2 exp2_poly2(float2 x) {
  x.x = fminf(fmaxf(x.x, -125.f), 16.f);
  x.y = fminf(fmaxf(x.y, -125.f), 16.f);
  const float2 t = fadd2(x, make_float2(12582912.f, 12582912.f));          // 1.5 * 2^23: low mantissa bits = n
  const float2 n = fadd2(t, make_float2(-12582912.f, -12582912.f));
  const float2 f = ffma2(n, make_float2(-1.f, -1.f), x);
  float2 p = ffma2(f, make_float2(0.0551716685f, 0.0551716685f), make_float2(0.2426111251f, 0.2426111251f));
  p = ffma2(p, f, make_float2(0.6932609677f, 0.6932609677f));
  p = ffma2(p, f, make_float2(0.9999280572f, 0.9999280572f));
  float2 r;
  r.x = __int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23));
  r.y = __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23));
  return r;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// Epoch-tagged arrival counter: value = (epoch << 16) | count; a value with another epoch counts as zero, so
// the counters need no initialisation.  `seen` is a value of the counter read earlier.  Returns the count
// after this arrival.
__device__ __forceinline__ int bump_counter(unsigned long long* c, unsigned long long seen, unsigned long long epoch) {
  while (true) {
    const unsigned long long assumed = seen;
    const int cnt = ((assumed >> 16) == epoch) ? (int)(assumed & 0xffffu) : 0;
    seen = atomicCAS(c, assumed, (epoch << 16) | (unsigned long long)(cnt + 1));
    if (seen == assumed) return cnt + 1;
  }
}

// ---------------------------------------------------------------- kernel parameters
struct AttnParams {
  const int32_t* prefix_len;
  const int32_t* n_nodes;
  const uint32_t* anc_bits;
  tv_bf16* out;
  float* lse;
  int32_t* status;
  tv_bf16* part_o;               // [slots][D/8][MT*128][8] bf16 normalised outputs, column-group major
  float* part_ml;                // [slots][2][MT*128]  (m in log2 units, then l)
  unsigned long long* counters;  // [B*Hkv*NP][2]: tickets claimed, partials ready (epoch-tagged)
  unsigned long long epoch;      // 48-bit tag of this call
  int B, Nmax, Hq, Hkv, Scap, G, NPT, NP, W, groups;
  int TT;                        // key tiles of the tree's own K/V: ceil(Nmax / 128), 1 or 2
  uint32_t q_box_bytes;
  unsigned long long* trace;     // optional event trace [cta][role 0..3][kTraceCap] of (tag << 48 | ns), or NULL          // bytes of one Q box {64, G, NPT}: 16 KB when G divides 128
  int tree_in_cache;             // the tree's K/V rows live in the cache behind the prefix (rows S_b + node)
  const int32_t* block_table;    // paged cache: page of key tile j of sequence b at [b * max_blocks + j]; else nullptr
  int max_blocks, n_pages;
  int out_al32;                  // out is 32-byte aligned: rows can be written 32 bytes per thread and store
  float scale_log2e;             // scale * log2(e)
  float scale;
  int early;                     // the caller promises that the kernel in front leaves prefix_len, n_nodes, the block
                                 // table and the committed rows alone: they are read before the grid-dependency wait
  unsigned long long wait_limit_ns;   // limit of every bounded wait
  int debug;                     // bit 0: the producer issues no copy at all; bit 1: pieces of cut units store their
                                 // partials but never announce them (both exercise the expiry of a bounded wait);
                                 // bit 2: the K/V stream alone - the issuing warp only hands every slot back as
                                 // soon as it is full, no MMA, no softmax, no output (what the memory side can do)
  int L;                         // layers in this launch: their units form one tile space, layer after layer
  long long out_layer_stride;    // elements between the outputs of two layers (lse is dense, [L,B,Hq,Nmax])
};

struct Item {
  int b, hk, j0, j1, len, S, n, layer;
};

// Shared bookkeeping of the linear tile space: cum[b] = sum of len over b' < b, len_b = ceil(S_b/128) + 1.
// The schedule works in a "virtual" tile space: every (sequence, KV head) unit is charged kSetupCost
// virtual tiles in front of its real key tiles, the price of starting a unit (Q load, pipeline refill,
// epilogue).  Cutting that space evenly gives CTAs that start more units fewer real tiles, and a cut that
// falls into a unit's setup region snaps to the unit boundary, which saves a split.
struct Sched {
  const int* cum;    // cum[b] = sum over b' < b of (len_b' + kSetupCost)
  const int* gs;     // gs[k] = first virtual tile of CTA group k, gs[groups] = total
  int B, Hkv;
  int total;         // layers * Hkv * cum[B]; the host refuses problems whose tile count does not fit 31 bits
  int per_layer;     // Hkv * cum[B]: the units of a layer tile one such stretch, layer after layer
  __device__ __forceinline__ int group_start(int k, int) const { return gs[k]; }
  __device__ __forceinline__ int find_b(int g) const {
    int lo = 0, hi = B - 1;   // largest b with Hkv*cum[b] <= g
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (Hkv * cum[mid] <= g) lo = mid; else hi = mid - 1;
    }
    return lo;
  }
};

template <int D, int MT>
struct SmemLayout {
  static constexpr int kHalf = 64 * 128 * 2;               // one 64-column, 128-row swizzled box: 16 KB
  static constexpr int kTileBytes = (D / 64) * kHalf;      // a 128 x D bf16 tile
  static constexpr int kQ = 0;
  static constexpr int kRing = MT * kTileBytes;
  static constexpr int kBars = kRing + kSlots * kTileBytes;
  // barrier indices (8 bytes each)
  static constexpr int Q_FULL = 0, Q_EMPTY = 1, KV_FULL = 2, KV_EMPTY = 2 + kSlots, S_FULL = 2 + 2 * kSlots,
                       P_READY = S_FULL + 2, O_DONE = P_READY + 2, ITEM_DONE = O_DONE + 2, EPI = ITEM_DONE + 2,
                       NBARS = EPI + 1;
  static constexpr int kMisc = kBars + NBARS * 8;          // tmem ptr, abort flag, last flag
  static constexpr int kCum = kMisc + 16;
  static constexpr int kGs = kCum + (kMaxB + 1) * 4;
  static constexpr int kTotal = kGs + (kMaxGroups + 1) * 4;
};

// ---------------------------------------------------------------- the kernel
template <int D, int MT>
__global__ void __launch_bounds__(kThreads, 1)
tree_attn_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kc,
                 const __grid_constant__ CUtensorMap map_vc, const __grid_constant__ CUtensorMap map_kt,
                 const __grid_constant__ CUtensorMap map_vt, const AttnParams prm) {
  using L = SmemLayout<D, MT>;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bars = sbase + L::kBars;
  auto bar = [&](int i) { return bars + 8u * i; };
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kMisc + 4);
  volatile int* last_flag = reinterpret_cast<volatile int*>(smem + L::kMisc + 8);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + L::kMisc);
  int* cum = reinterpret_cast<int*>(smem + L::kCum);
  int* gs = reinterpret_cast<int*>(smem + L::kGs);
  const unsigned long long wait_limit = prm.wait_limit_ns;

  // ---- setup: schedule table, barriers, TMEM
  if (threadIdx.x == 64) {     // fetch the five TMA descriptors while the rest of the set-up runs
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_q) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_kc) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_vc) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_kt) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_vt) : "memory");
  }
  // Without the caller's promise nothing of the problem is read before every earlier kernel of the stream has
  // finished (a kernel in front may still be writing prefix_len, and lines of it cached by an earlier launch on
  // this SM are only dropped by the wait).
  if (!prm.early) gdc_wait();
  if (warp == 0) {
    int run = 0;
#pragma unroll 1
    for (int base = 0; base < prm.B; base += 32) {
      const int b = base + lane;
      int len = 0;
      if (b < prm.B) {
        int S = prm.prefix_len[b];
        S = S < 0 ? 0 : (S > prm.Scap ? prm.Scap : S);
        len = (S + kTileN - 1) / kTileN + prm.TT + kSetupCost;
      }
      int inc = len;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      if (b < prm.B) cum[b] = run + inc - len;
      run += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (lane == 0) cum[prm.B] = run;
  }
  if (threadIdx.x == 32) {
    mbar_init(bar(L::Q_FULL), 1);
    mbar_init(bar(L::Q_EMPTY), 1);
#pragma unroll 1
    for (int s = 0; s < kSlots; ++s) {
      mbar_init(bar(L::KV_FULL + s), 1);
      mbar_init(bar(L::KV_EMPTY + s), 1);
    }
    for (int s = 0; s < 2; ++s) {                // index = S buffer
      mbar_init(bar(L::S_FULL + s), 1);
      mbar_init(bar(L::P_READY + s), 128);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar(L::O_DONE + s), 1);
      mbar_init(bar(L::ITEM_DONE + s), 1);
    }
    mbar_init(bar(L::EPI), MT * 128);
    *abort_flag = ((sbase & 1023u) != 0) ? 1 : 0;   // swizzled tiles need a 1024-byte aligned base
    *last_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32((const void*)tmem_slot))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // Small problems use fewer CTA groups, so that a unit is cut into few pieces (each piece costs a partial
  // write and a merge) and every group still gets a worthwhile share of tiles.
  int groups;
  {
    const unsigned total = (unsigned)(prm.Hkv * cum[prm.B]) * (unsigned)prm.L;
    const unsigned want = total / (unsigned)kMinVirtualTilesPerGroup;
    groups = want < 1u ? 1 : (want < (unsigned)prm.groups ? (int)want : prm.groups);
    // A group count just above a multiple of the unit count is rounded down to it: with units of equal length
    // (one sequence, all heads) every unit is then cut into the same number of equal pieces and no cut falls
    // just behind a unit boundary.  Not worth more than 1/16 of the groups.
    {
      const int units = prm.B * prm.Hkv * prm.L, over = groups % units;
      if (groups > units && over * 16 <= groups) groups -= over;
    }
    // gs[k] = floor(total * k / groups) in 32-bit arithmetic: total = q * groups + r
    const unsigned q = total / (unsigned)groups, r = total % (unsigned)groups;
#pragma unroll 1
    for (int k = threadIdx.x; k <= prm.groups; k += kThreads)
      gs[k] = k <= groups ? (int)(k * q + (k * r) / (unsigned)groups) : (int)total;
  }
  __syncthreads();

  Sched sch{cum, gs, prm.B, prm.Hkv, prm.Hkv * cum[prm.B] * prm.L, prm.Hkv * cum[prm.B]};
  const int group = blockIdx.x / prm.NP;
  const int pair = blockIdx.x % prm.NP;
  const int g_begin = sch.group_start(group, groups);        // groups past the last used one get an empty range
  const int g_end = sch.group_start(group + 1, groups);

  // Walks the items of this CTA's range; identical in every role.
  auto next_item = [&](int& g, Item& it) -> bool {
    while (g < g_end) {
      const int layer = (int)((unsigned)g / (unsigned)sch.per_layer);
      const int gl = g - layer * sch.per_layer;                   // place inside the layer
      const int b = sch.find_b(gl);
      const int lenv = cum[b + 1] - cum[b];                       // setup region + real tiles
      const unsigned local = (unsigned)(gl - prm.Hkv * cum[b]);
      const int hk = (int)(local / (unsigned)lenv);
      const int r0 = (int)(local - (unsigned)hk * (unsigned)lenv);
      const int room = g_end - g;
      const int r1 = (lenv - r0) < room ? lenv : r0 + room;
      g += r1 - r0;
      const int j0 = r0 > kSetupCost ? r0 - kSetupCost : 0;
      const int j1 = r1 > kSetupCost ? r1 - kSetupCost : 0;
      if (j1 <= j0) continue;                                     // only setup tiles of this unit fall in the range
      it.b = b;
      it.hk = hk;
      it.layer = layer;
      it.j0 = j0;
      it.j1 = j1;
      it.len = lenv - kSetupCost;
      int S = prm.prefix_len[b];
      it.S = S < 0 ? 0 : (S > prm.Scap ? prm.Scap : S);
      int n = prm.n_nodes[b];
      it.n = n < 0 ? 0 : (n > prm.Nmax ? prm.Nmax : n);
      return true;
    }
    return false;
  };

  constexpr uint32_t kIdescQK = instr_desc(kTileN, false);
  constexpr uint32_t kIdescPV = instr_desc(D, true);
  constexpr uint32_t kTmemS0 = 0, kTmemO0 = 256;

  if (warp == 0) {
    // =========================================================== TMA producer
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    if (!*abort_flag && !(prm.debug & 1)) {        // the whole warp walks the items; one elected lane issues the copies
      int g = g_begin;
      Item it;
      uint32_t item_idx = 0, fill = 0;
      bool ok = true;
      Tracer tr;
      tr.init(lane == 0 ? prm.trace : nullptr, 0);
      tr.mark(0);
      uint64_t kv_policy;      // the committed prefix is streamed once: first in line for eviction from L2
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(kv_policy));
      // Overlap with the kernel in front (programmatic dependent launch).  With the caller's promise (prm.early)
      // that this kernel leaves prefix_len, n_nodes, the block table and the committed rows alone, the first
      // prefix tiles are requested at once; Q and the tree's K/V - what a preceding kernel may still be
      // producing - wait for that kernel to finish.  Only then may the next kernel be scheduled, so that at
      // most two launches are in flight.
      // status[] may still be written by the kernel in front (tree_build_mask stores it last), so a flag found
      // before the wait is kept here and raised after it.
      bool synced = false;
      int bad_page_b = -1;
      auto sync_with_predecessor = [&]() {
        gdc_wait();
        if (elect_one()) gdc_launch_dependents();
        if (bad_page_b >= 0 && lane == 0) atomicOr(prm.status + bad_page_b, TV_ST_BAD_INDEX);
        bad_page_b = -1;
        __syncwarp();
        synced = true;
      };
      auto load_q = [&]() {
        if (elect_one()) {
          mbar_expect_tx(bar(L::Q_FULL), MT * (D / 64) * prm.q_box_bytes);
#pragma unroll
          for (int t = 0; t < MT; ++t)
#pragma unroll
            for (int h = 0; h < D / 64; ++h)
              tma_load_5d(sbase + L::kQ + t * L::kTileBytes + h * L::kHalf, &map_q, bar(L::Q_FULL), h * 64,
                          it.hk * prm.G, (pair * MT + t) * prm.NPT, it.b, it.layer);
        }
        __syncwarp();
      };
      if (!prm.early) sync_with_predecessor();
      while (ok && next_item(g, it)) {
        ok = mbar_wait(bar(L::Q_EMPTY), (item_idx & 1) ^ 1, abort_flag, wait_limit);
        if (!ok) break;
        tr.mark(0x1000u | item_idx);
        bool q_pending = !synced;          // first item: Q goes out after the first prefix tiles
        if (!q_pending) load_q();
        ++item_idx;
        // paged cache: the page of a prefix key tile comes from the block table, fetched one tile ahead of its use
        auto page_of = [&](int jj) -> int {
          if (!prm.block_table || jj >= it.len - prm.TT || jj >= it.j1) return 0;
          int pg = prm.block_table[(size_t)it.b * prm.max_blocks + jj];
          if ((unsigned)pg >= (unsigned)prm.n_pages) {       // reported; the tile then reads page 0
            if (!synced) bad_page_b = it.b;                  // (only the first item can get here before the wait)
            else if (lane == 0) atomicOr(prm.status + it.b, TV_ST_BAD_INDEX);
            pg = 0;
          }
          return pg;
        };
        int page_next = page_of(it.j0);
        for (int j = it.j0; j < it.j1 && ok; ++j) {
          const int tt = j - (it.len - prm.TT);      // >= 0: index of the tree key tile
          const bool tree = tt >= 0;
          const int page = page_next;
          page_next = page_of(j + 1);
          const int row0 = prm.block_table ? 0 : j * kTileN;                                // of the tile in its slab
          const int slab = (prm.block_table ? page : it.b) * prm.Hkv + it.hk;               // (page or sequence, KV head)
#pragma unroll
          for (int kv = 0; kv < 2; ++kv) {
            const uint32_t slot = fill % kSlots, round = fill / kSlots;
            if (q_pending && (tree || fill >= (uint32_t)kSlots)) {      // before the first wait for a ring slot
              sync_with_predecessor();
              load_q();
              q_pending = false;
            }
            ok = mbar_wait(bar(L::KV_EMPTY + slot), (round & 1) ^ 1, abort_flag, wait_limit);
            if (!ok) break;
            tr.mark(0x2000u | (fill & 0xfffu));
            const uint32_t dst = sbase + L::kRing + slot * L::kTileBytes;
            if (elect_one()) {
              mbar_expect_tx(bar(L::KV_FULL + slot), L::kTileBytes);
#pragma unroll
              for (int h = 0; h < D / 64; ++h) {
                if (tree && prm.tree_in_cache)
                  tma_load_4d_hint(dst + h * L::kHalf, kv ? &map_vc : &map_kc, bar(L::KV_FULL + slot), h * 64,
                                   it.S + tt * kTileN, it.b * prm.Hkv + it.hk, it.layer, kv_policy);
                else if (tree)
                  tma_load_5d(dst + h * L::kHalf, kv ? &map_vt : &map_kt, bar(L::KV_FULL + slot), h * 64, it.hk, tt * kTileN, it.b,
                              it.layer);
                else
                  tma_load_4d_hint(dst + h * L::kHalf, kv ? &map_vc : &map_kc, bar(L::KV_FULL + slot), h * 64, row0, slab,
                                   it.layer, kv_policy);
              }
            }
            __syncwarp();
            ++fill;
          }
        }
        if (ok && q_pending) {
          sync_with_predecessor();
          load_q();
        }
      }
      if (!synced) sync_with_predecessor();        // a CTA without work still has to let the next kernel go
    } else {
      gdc_wait();
      if (elect_one()) gdc_launch_dependents();
    }
  } else if (warp == 1) {
    // =========================================================== MMA issuer
    // One thread issues every MMA of the CTA.  S of a key tile is a full 128-key tile (N = 128: with 64-key
    // MMAs the Q operand is re-read from shared memory twice as often and the pipe runs at 2/3 of its rate).
    // P overlays the first 64 columns of its S buffer, so S of the next key tile can only be computed after
    // the PV that reads P; the tensor pipe runs MMAs in issue order, which gives that for free.
    //   two row tiles (buffer = row tile):  wait P_t -> O_t += P_t V -> S_t = Q_t K_next^T, t = 0, 1 in turn, so
    //     that the softmax of one row tile runs while the pipe works for the other one;
    //   one row tile (buffers alternate by key tile):  S_next = Q K_next^T -> wait P -> O += P V.
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    if (!*abort_flag) {      // the whole warp walks the items; one elected lane issues
      int g = g_begin;
      Item it;
      uint32_t item_idx = 0, fill = 0, tj = 0;
      bool ok = true;
      Tracer tr;
      tr.init(lane == 0 ? prm.trace : nullptr, 1);
      tr.mark(0);
      // descriptor words: low = start address >> 4 | LBO field, high = SBO 1024 B | version 1 | 128-byte swizzle
      const uint32_t desc_hi = (uint32_t)(smem_desc(0, 0, 1024) >> 32);
      const uint32_t q_lo = (uint32_t)smem_desc(sbase + L::kQ, 16, 1024);   // K-major: LBO unused
      const uint32_t k_lo = (uint32_t)smem_desc(sbase + L::kRing, 16, 1024);
      const uint32_t v_lo = (uint32_t)smem_desc(sbase + L::kRing, L::kHalf, 1024);  // MN-major: LBO = next 64 columns
      constexpr int kHalf16 = L::kHalf >> 4, kTile16 = L::kTileBytes >> 4;
      // S(buf) = Q_t K^T for the 128 keys of the K tile in `slot`
      auto issue_qk = [&](int t, int buf, uint32_t slot) {
        const uint32_t qa = q_lo + t * kTile16, ka = k_lo + slot * kTile16;
        if (elect_one()) {
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            const uint32_t off = (ks / 4) * kHalf16 + (ks % 4) * 2;        // 16 columns = 32 bytes inside a swizzled row
            mma_ss_lohi(tmem + kTmemS0 + buf * 128, qa + off, ka + off, desc_hi, kIdescQK, ks > 0);
          }
          mma_commit(bar(L::S_FULL + buf));
        }
        __syncwarp();
      };
      // O_t += P(buf) V for the 128 keys of the V tile in `slot`
      auto issue_pv = [&](int t, int buf, uint32_t slot, bool first_tile) {
        const uint32_t va = v_lo + slot * kTile16;
        if (elect_one()) {
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)            // 16 keys = 16 rows of 128 bytes = 8 packed P columns
            mma_ts_lohi(tmem + kTmemO0 + t * 128, tmem + kTmemS0 + buf * 128 + ks * 8, va + ks * 128, desc_hi, kIdescPV,
                        (!first_tile || ks > 0) ? 1u : 0u);
        // With two row tiles the S tile that the softmax waits for next is committed after this PV, so its
        // completion is known without a commit of its own (a commit stalls the pipe for some 45 cycles).
          if (MT == 1) mma_commit(bar(L::O_DONE + t));
        }
        __syncwarp();
      };
      while (ok && next_item(g, it)) {
        const int nt = it.j1 - it.j0;
        ok = mbar_wait(bar(L::Q_FULL), item_idx & 1, abort_flag, wait_limit);
        if (!ok) break;
        tr.mark(0x1000u | item_idx);
        if (prm.debug & 4) {       // stream only: every tile of the item is released as soon as it has landed
#pragma unroll 1
          for (int f = 0; f < 2 * nt && ok; ++f) {
            const uint32_t ff = fill + f;
            ok = mbar_wait(bar(L::KV_FULL + ff % kSlots), (ff / kSlots) & 1, abort_flag, wait_limit);
            if (ok && elect_one()) mbar_arrive(bar(L::KV_EMPTY + ff % kSlots));
            __syncwarp();
          }
          if (elect_one()) mbar_arrive(bar(L::Q_EMPTY));
          __syncwarp();
          fill += 2 * nt;
          ++item_idx;
          continue;
        }
        {
          const uint32_t slot = fill % kSlots;
          ok = mbar_wait(bar(L::KV_FULL + slot), (fill / kSlots) & 1, abort_flag, wait_limit);
          if (!ok) break;
          tc_fence_after();
          if (MT == 2) {
            issue_qk(0, 0, slot);
            issue_qk(1, 1, slot);
          } else {
            issue_qk(0, tj & 1, slot);
          }
          if (elect_one()) mma_commit(bar(L::KV_EMPTY + slot));
          if (nt == 1 && elect_one()) mma_commit(bar(L::Q_EMPTY));
        }
        for (int jt = 0; jt < nt && ok; ++jt, ++tj) {
          const uint32_t fv = fill + 2 * jt + 1, vslot = fv % kSlots;
          const uint32_t fk = fv + 1, kslot = fk % kSlots;
          const bool more = jt + 1 < nt;
          if (MT == 2) {
#pragma unroll
            for (int t = 0; t < 2; ++t) {
              ok = mbar_wait(bar(L::P_READY + t), tj & 1, abort_flag, wait_limit);
              if (!ok) break;
              if (t == 0) {
                ok = mbar_wait(bar(L::KV_FULL + vslot), (fv / kSlots) & 1, abort_flag, wait_limit);
                if (ok && more) ok = mbar_wait(bar(L::KV_FULL + kslot), (fk / kSlots) & 1, abort_flag, wait_limit);
                if (!ok) break;
              }
              tc_fence_after();
              tr.mark(0x4000u | ((2 * tj + t) & 0xfffu));
              issue_pv(t, t, vslot, jt == 0);
              if (!more && elect_one()) mma_commit(bar(L::ITEM_DONE + t));      // all MMAs of the item's row tile are done
              if (more) issue_qk(t, t, kslot);
              tr.mark(0x2000u | ((2 * tj + t) & 0xfffu));
            }
            if (!ok) break;
          } else {
            const int buf = tj & 1;
            if (more) {
              ok = mbar_wait(bar(L::KV_FULL + kslot), (fk / kSlots) & 1, abort_flag, wait_limit);
              if (!ok) break;
              tc_fence_after();
              issue_qk(0, buf ^ 1, kslot);
            }
            ok = mbar_wait(bar(L::P_READY + buf), (tj >> 1) & 1, abort_flag, wait_limit);
            if (ok) ok = mbar_wait(bar(L::KV_FULL + vslot), (fv / kSlots) & 1, abort_flag, wait_limit);
            if (!ok) break;
            tc_fence_after();
            tr.mark(0x4000u | (tj & 0xfffu));
            issue_pv(0, buf, vslot, jt == 0);
            if (!more && elect_one()) mma_commit(bar(L::ITEM_DONE));
            tr.mark(0x2000u | (tj & 0xfffu));
          }
          if (elect_one()) {
            mma_commit(bar(L::KV_EMPTY + vslot));
            if (more) mma_commit(bar(L::KV_EMPTY + kslot));
            if (jt + 2 == nt) mma_commit(bar(L::Q_EMPTY));
          }
          __syncwarp();
        }
        fill += 2 * nt;
        ++item_idx;
      }
    }
  } else if (warp >= 4) {
    // =========================================================== softmax / epilogue warpgroups
    // Register budget: the CTA starts with 168 registers per thread; warps 0-3 give up 96 each (168 -> 72) and
    // warps 4-11 take 48 each (168 -> 216).  4 x 96 = 8 x 48: the increase below can only complete once the
    // other warpgroup has released enough, so any other split has to keep 4 (168 - low) >= 8 (high - 168) or the
    // kernel never gets past this instruction.
    asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
    const int wg = (warp - 4) >> 2;                  // row tile of this warpgroup
    const int row = ((warp & 3) << 5) | lane;        // TMEM lane = row inside the tile
    const uint32_t lane_addr = (uint32_t)((warp & 3) << 5) << 16;
    const bool wg_active = wg < MT;
    gdc_wait();      // anc_bits, the workspace and the outputs may belong to the kernel in front until it is done
    // in-cache layout: a tree that does not fit behind its prefix is reported, not read past the capacity (rows
    // past Scap arrive as zeros and the sequence's output is unspecified).  Raised after the wait: status[] may
    // be written by the kernel in front until then.
    if (prm.tree_in_cache && blockIdx.x == 0)
#pragma unroll 1
      for (int b = threadIdx.x - 128; b < prm.B; b += kThreads - 128) {
        int S = prm.prefix_len[b];
        S = S < 0 ? 0 : (S > prm.Scap ? prm.Scap : S);
        if (S + prm.n_nodes[b] > prm.Scap) atomicOr(prm.status + b, TV_ST_CAPACITY);
      }
    if (wg_active && !*abort_flag && !(prm.debug & 4)) {
      int g = g_begin;
      Item it;
      uint32_t fill = 0, tj = 0, epi_phase = 0, item_cnt = 0;   // tj: key tiles handled so far (all items)
      bool ok = true;
      Tracer tr;
      tr.init((threadIdx.x & 127) == 0 ? prm.trace : nullptr, 2 + wg);
      tr.mark(0);
#ifdef TV_PROF
      unsigned int prof[12] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u}, pc0 = 0, pc1 = 0, pc2 = 0, pend = 0;
      // 0 wait S, 1 ld, 2 compute, 3 hand-over, 4 tiles, 5 between tiles, 6 start -> first S, 7 wait ITEM_DONE,
      // 8 epilogue (whole or piece), 9 items, 10 first tile of an item: from item start to its S
      const unsigned int prof_start = clock();
      const long long prof_c0 = clock64();
      const unsigned long long prof_g0 = globaltimer_ns();   // cycles: wait S, ld, compute, hand-over; tiles
#endif
      // Rendezvous of the softmax warpgroups through an mbarrier, so that it is bounded like every other wait.
      // All 32 lanes wait together and agree on the outcome, so that the warp-wide TMEM instructions
      // below are never executed by a part of a warp.
      auto wwait = [&](uint32_t b_, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, mbar_wait(b_, parity, abort_flag, wait_limit));
      };
      auto epi_sync = [&]() -> bool {
        mbar_arrive(bar(L::EPI));
        const bool r = wwait(bar(L::EPI), epi_phase & 1);
        ++epi_phase;
        return r;
      };
      while (ok && next_item(g, it)) {
#ifdef TV_PROF
        const unsigned int pitem = clock();
        unsigned int ep[6], ep_kind = 0, ep_others = 0, ep_own = 0;
#endif
        const int nt = it.j1 - it.j0;
        const int node = (pair * MT + wg) * prm.NPT + row / prm.G;
        const int gm = row % prm.G;
        const bool row_exists = row < prm.NPT * prm.G && node < prm.Nmax;
        const bool row_active = row_exists && node < it.n;
        uint32_t anc[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
        if (row_active) {
#pragma unroll
          for (int w = 0; w < 8; ++w)
            if (w < prm.W) anc[w] = prm.anc_bits[((size_t)it.b * prm.Nmax + node) * prm.W + w];
        }
        float m_used = -INFINITY;      // running reference maximum, in log2 units (score * scale * log2e)
        float l_sum = 0.f;
        // A piece of a cut unit draws its ticket early (thread 128 only): the counter is read at the start of
        // the item and the compare-and-swap is issued when the last key tile begins, so that both round trips
        // are hidden behind the softmax of that tile; the outcome is looked at in the epilogue.
        const bool piece = !(it.j0 == 0 && it.j1 == it.len);
        unsigned long long* claim_ctr =
            prm.counters + ((((size_t)it.layer * prm.B + it.b) * prm.Hkv + it.hk) * prm.NP + pair) * 2;
        unsigned long long claim_assumed = 0, claim_ret = 1;
        int claim_cnt = 0;
        if (piece && threadIdx.x == 128) claim_assumed = *reinterpret_cast<volatile unsigned long long*>(claim_ctr);
        const uint32_t o_addr_loop = tmem + lane_addr + kTmemO0 + wg * 128;
        // key tiles below this index are full tiles of the committed prefix (no mask of any kind)
        const int j_full = min(it.S / kTileN, it.len - prm.TT);
        for (int jt = 0; jt < nt && ok; ++jt, ++tj) {
          const int j = it.j0 + jt;
          const bool full_tile = j < j_full;
          int tt = -1, valid_keys = kTileN;          // tt >= 0: index of the tree key tile
          if (!full_tile) {
            tt = j - (it.len - prm.TT);
            valid_keys = tt >= 0 ? max(0, min(kTileN, it.n - tt * kTileN)) : min(kTileN, it.S - j * kTileN);
          }
          const bool tree = tt >= 0;
          if (piece && threadIdx.x == 128 && jt == nt - 1) {
            claim_cnt = ((claim_assumed >> 16) == prm.epoch) ? (int)(claim_assumed & 0xffffu) : 0;
            claim_ret = atomicCAS(claim_ctr, claim_assumed, (prm.epoch << 16) | (unsigned long long)(claim_cnt + 1));
          }
          // ---- V rows past the valid keys may hold anything (stale cache rows, padded tree slots): zero
          // them so that 0 * NaN never reaches O.  Idempotent, so both warpgroups may do it.  Rows that lie
          // outside the tensor arrive as zeros from the copy itself: a tree tile whose tree is full (the
          // usual case) needs nothing.
          if (valid_keys < kTileN && !(tree && !prm.tree_in_cache && tt * kTileN + valid_keys >= prm.Nmax)) {
            const uint32_t f = fill + 2 * jt + 1, slot = f % kSlots;
            ok = wwait(bar(L::KV_FULL + slot), (f / kSlots) & 1);
            if (!ok) break;
            if (row >= valid_keys) {
              uint8_t* vrow = smem + L::kRing + slot * L::kTileBytes + row * 128;
#pragma unroll
              for (int h = 0; h < D / 64; ++h)
#pragma unroll
                for (int c = 0; c < 8; ++c)
                  *reinterpret_cast<uint4*>(vrow + h * L::kHalf + c * 16) = make_uint4(0, 0, 0, 0);
            }
            fence_proxy_async_smem();
          }
          // S buffer of this key tile: the row tile's own one, or alternating by key tile when the CTA has one
          // row tile; its barriers complete once per use of the buffer.
          const int buf = (MT == 2) ? wg : (int)(tj & 1u);
          const uint32_t use_par = (MT == 2) ? (tj & 1u) : ((tj >> 1) & 1u);
          const uint32_t s_base = tmem + lane_addr + kTmemS0 + buf * 128;
          tr.mark(0x0800u | (tj & 0x7ffu));
          TV_PROF_T(pc0);
#ifdef TV_PROF
          if (jt > 0) prof[5] += pc0 - pend;
#endif
          ok = wwait(bar(L::S_FULL + buf), use_par);
          if (!ok) break;
          tc_fence_after();
          TV_PROF_T(pc1);
#ifdef TV_PROF
          prof[0] += pc1 - pc0;
          if (tj == 0) prof[6] = pc1 - prof_start;
          if (jt == 0) prof[10] += pc1 - pitem;
#endif
          tr.mark(0x1000u | (tj & 0xfffu));
          // ---- whole-tile fast path (full, unmasked tiles): all 128 scores of the row in one load and P with
          // the reference maximum as it stands; the row sum then tells whether anything left the lazy-rescale
          // range (all P are >= 0, so the sum bounds every element; NaN and infinity fail the comparison).  P
          // is only stored once the check has passed, so on a failure the scores are still in S and the chunk
          // loop below does the tile again, maximum first.  A row without a reference yet (the first tile of
          // an item) takes the score of the tile's first key: it is one of the row's scores, hence not above
          // their maximum, and if it lies too far below it the check fails like any other.
          bool tile_done = false;
          if (full_tile) {
            uint32_t sall[128];
            tmem_ld32(s_base, sall);
            tmem_ld32(s_base + 32, sall + 32);
            tmem_ld32(s_base + 64, sall + 64);
            tmem_ld32(s_base + 96, sall + 96);
            tmem_wait_ld();
            const float* sa = reinterpret_cast<const float*>(sall);
            const float2 c2 = make_float2(prm.scale_log2e, prm.scale_log2e);
            const bool opens = (m_used == -INFINITY);
            const float m_ref = opens ? sa[0] * prm.scale_log2e : m_used;
            const float2 nm2 = make_float2(-m_ref, -m_ref);
            float2 sum = make_float2(0.f, 0.f);
            uint32_t pkk[64];
#pragma unroll
            for (int i = 0; i < 64; ++i) {
              const float2 x = ffma2(make_float2(sa[2 * i], sa[2 * i + 1]), c2, nm2);
              float2 pv;
              if (TV_POLY_SEL(i)) {
                pv = exp2_poly2(x);
              } else {
                pv.x = fast_exp2(x.x);
                pv.y = fast_exp2(x.y);
              }
              sum = fadd2(sum, pv);
              pkk[i] = pack_bf16(pv.x, pv.y);
            }
            const float fsum = sum.x + sum.y;
            const bool overflow = row_active && !(fsum <= 2.f * kMaxFastSum);
            if (!__any_sync(0xffffffffu, overflow)) {
              l_sum += fsum;
              if (opens && row_active) m_used = m_ref;
#pragma unroll
              for (int q = 0; q < 8; ++q)
                asm volatile(
                    "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                    ::"r"(s_base + q * 8), "r"(pkk[q * 8 + 0]), "r"(pkk[q * 8 + 1]), "r"(pkk[q * 8 + 2]), "r"(pkk[q * 8 + 3]),
                      "r"(pkk[q * 8 + 4]), "r"(pkk[q * 8 + 5]), "r"(pkk[q * 8 + 6]), "r"(pkk[q * 8 + 7])
                    : "memory");
              tile_done = true;
            }
          }
#pragma unroll
          for (int h = 0; h < 2 && !tile_done; ++h) {
            const int valid_half = min(64, max(0, valid_keys - 64 * h));
            uint32_t sreg[64];
            const uint32_t s_addr = s_base + h * 64;
            TV_PROF_T(pc0);
            tmem_ld32(s_addr, sreg);
            tmem_ld32(s_addr + 32, sreg + 32);
            tmem_wait_ld();
            TV_PROF_USE(sreg[31]);
            TV_PROF_USE(sreg[63]);
            TV_PROF_T(pc1);
            float* s = reinterpret_cast<float*>(sreg);
            const bool masked = tree || valid_half < 64;
            if (masked) {
              // two 32-bit words of this chunk: ancestor bits on a tree tile, a length mask on the ragged tile
              uint32_t w0, w1;
              if (tree) {
                const uint32_t a0 = tt > 0 ? anc[4] : anc[0], a1 = tt > 0 ? anc[5] : anc[1];
                const uint32_t a2 = tt > 0 ? anc[6] : anc[2], a3 = tt > 0 ? anc[7] : anc[3];
                w0 = h ? a2 : a0;
                w1 = h ? a3 : a1;
              } else {
                w0 = valid_half >= 32 ? 0xffffffffu : ((1u << valid_half) - 1u);
                w1 = valid_half >= 64 ? 0xffffffffu : (valid_half <= 32 ? 0u : ((1u << (valid_half - 32)) - 1u));
              }
#pragma unroll
              for (int c = 0; c < 32; ++c) {
                if (!((w0 >> c) & 1u)) s[c] = -INFINITY;
                if (!((w1 >> c) & 1u)) s[32 + c] = -INFINITY;
              }
            }
            uint32_t pk[32];                 // P of this chunk, bf16 pairs
            const bool first = (jt == 0 && h == 0);
            // the tiles that get here (first of an item, masked, or rejected by the fast path) take the true
            // maximum of the chunk first
            {
              float mx0 = s[0], mx1 = s[1], mx2_ = s[2], mx3 = s[3];
#pragma unroll
              for (int c = 4; c < 64; c += 4) {
                mx0 = fmaxf(mx0, s[c]);
                mx1 = fmaxf(mx1, s[c + 1]);
                mx2_ = fmaxf(mx2_, s[c + 2]);
                mx3 = fmaxf(mx3, s[c + 3]);
              }
              const float mx2 = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2_, mx3)) * prm.scale_log2e;
              // ---- lazy rescale: move the reference maximum only when it would grow by more than the
              // threshold.  The TMEM accesses are warp-wide (.sync.aligned), so the warp rescales as soon as
              // one of its rows has to; rows that keep their maximum multiply by 1.
              const bool moves = (mx2 > m_used + kRescaleThreshold || m_used == -INFINITY) && mx2 > -INFINITY;
              const bool scales = moves && !first && m_used > -INFINITY;
              const float alpha = scales ? fast_exp2(m_used - mx2) : 1.f;
              if (moves) m_used = mx2;
              l_sum *= alpha;
              if (__any_sync(0xffffffffu, scales)) {
                tr.mark(0x9000u | (tj & 0xfffu));
                // O must be at rest.  With two row tiles the PV of the previous key tile was issued before the
                // S = Q K^T this warpgroup has just waited for, and the pipe runs in issue order: it is done.
                // With one row tile the next S is issued ahead of the PV: wait for its completion (number tj - 1).
                if (MT == 1) ok = wwait(bar(L::O_DONE + wg), (tj - 1) & 1);
                if (!ok) break;
                tc_fence_after();
#pragma unroll 1
                for (int q = 0; q < D / 32; ++q) {
                  uint32_t o[32];
                  tmem_ld32(o_addr_loop + q * 32, o);
                  tmem_wait_ld();
#pragma unroll
                  for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                  tmem_st32(o_addr_loop + q * 32, o);
                }
                // The tile's first 64 keys already have their P in TMEM, formed with the old reference: it moves
                // with O (l_sum has just been rescaled for them too).
                if (h == 1) {
                  uint32_t pp[32];
                  tmem_ld32(s_base, pp);
                  tmem_wait_ld();
#pragma unroll
                  for (int c = 0; c < 32; ++c)
                    pp[c] = pack_bf16(__uint_as_float(pp[c] << 16) * alpha, __uint_as_float(pp[c] & 0xffff0000u) * alpha);
                  tmem_st32(s_base, pp);
                }
              }
              // ---- P = exp2(s * c - m), row sum in fp32, P rounded to bf16 (masked scores give exactly 0)
              const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
              float ls0 = 0.f, ls1 = 0.f;
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                const float p0 = fast_exp2(fmaf(s[2 * i], prm.scale_log2e, neg_m));
                const float p1 = fast_exp2(fmaf(s[2 * i + 1], prm.scale_log2e, neg_m));
                ls0 += p0;
                ls1 += p1;
                pk[i] = pack_bf16(p0, p1);
              }
              l_sum += ls0 + ls1;
            }
            if (!ok) break;
            TV_PROF_USE(pk[31]);
            TV_PROF_USE(pk[15]);
            TV_PROF_USE(__float_as_uint(l_sum));
            TV_PROF_T(pc2);
#ifdef TV_PROF
            prof[1] += pc1 - pc0;
            prof[2] += pc2 - pc1;
#endif
            // ---- P over the start of the S buffer (columns already read): 16 keys = 8 packed columns per store
#pragma unroll
            for (int q = 0; q < 4; ++q)
              asm volatile(
                  "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                  ::"r"(s_base + h * 32 + q * 8), "r"(pk[q * 8 + 0]), "r"(pk[q * 8 + 1]), "r"(pk[q * 8 + 2]), "r"(pk[q * 8 + 3]),
                    "r"(pk[q * 8 + 4]), "r"(pk[q * 8 + 5]), "r"(pk[q * 8 + 6]), "r"(pk[q * 8 + 7])
                  : "memory");
          }
          if (!ok) break;
          TV_PROF_T(pc0);
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(bar(L::P_READY + buf));
          TV_PROF_T(pc1);
#ifdef TV_PROF
          prof[3] += pc1 - pc0;
          prof[4] += 1;
          pend = pc1;
#endif
          tr.mark(0x2000u | (tj & 0xfffu));
        }
        if (!ok) break;
        // ---- epilogue of the item: wait for the last PV into this O buffer
        {
          // Wait for every MMA of the item.  This barrier completes once per item, so its phase is never
          // more than one away from the one waited for (a parity wait cannot tell phases two apart, which
          // is why the per-PV barrier O_DONE is not used here: both last PVs may or may not be done yet).
          TV_PROF_T(pc0);
          ok = wwait(bar(L::ITEM_DONE + wg), item_cnt & 1);
          ++item_cnt;
          if (!ok) break;
          tc_fence_after();
          TV_PROF_T(pc1);
#ifdef TV_PROF
          prof[7] += pc1 - pc0;
#endif
          tr.mark(0x5000u);
#ifdef TV_PROF
          for (int i = 0; i < 6; ++i) ep[i] = pc1;
#endif
          const uint32_t o_addr = o_addr_loop;
          const bool whole = (it.j0 == 0 && it.j1 == it.len);
          const int h = it.hk * prm.G + gm;
          tv_bf16* orow = prm.out + (size_t)it.layer * prm.out_layer_stride + (((size_t)it.b * prm.Nmax + node) * prm.Hq + h) * D;
          float* lse_p = prm.lse ? prm.lse + (((size_t)it.layer * prm.B + it.b) * prm.Hq + h) * prm.Nmax + node : nullptr;
          // Normalised bf16 output of this row, 32 columns at a time (one copy of the loop for every use: the
          // epilogue is cold code, fetched while the other CTAs still stream K/V).
          auto store_rows = [&](uint4* dst, size_t stride_u4, float inv, bool do_store, bool zero) {
#pragma unroll 1
            for (int q = 0; q < D / 32; ++q) {
              uint32_t o[32];
              tmem_ld32(o_addr + q * 32, o);
              tmem_wait_ld();
              if (do_store) {
                uint4 v[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                  v[c].x = pack_bf16(__uint_as_float(o[8 * c + 0]) * inv, __uint_as_float(o[8 * c + 1]) * inv);
                  v[c].y = pack_bf16(__uint_as_float(o[8 * c + 2]) * inv, __uint_as_float(o[8 * c + 3]) * inv);
                  v[c].z = pack_bf16(__uint_as_float(o[8 * c + 4]) * inv, __uint_as_float(o[8 * c + 5]) * inv);
                  v[c].w = pack_bf16(__uint_as_float(o[8 * c + 6]) * inv, __uint_as_float(o[8 * c + 7]) * inv);
                  if (zero) v[c] = make_uint4(0, 0, 0, 0);       // rows of padded nodes: O may hold anything
                }
                if (stride_u4 == 1 && prm.out_al32) {     // a row of the output: whole 32-byte sectors per store
                  st_global_32B(dst + q * 4, v[0], v[1]);
                  st_global_32B(dst + q * 4 + 2, v[2], v[3]);
                } else {
#pragma unroll
                  for (int c = 0; c < 4; ++c) dst[(size_t)(q * 4 + c) * stride_u4] = v[c];
                }
              }
            }
          };
          if (whole) {
            const float inv = (row_active && l_sum > 0.f) ? 1.f / l_sum : 0.f;
            store_rows(reinterpret_cast<uint4*>(orow), 1, inv, row_exists, !row_active);
            if (row_exists && lse_p)
              *lse_p = (row_active && l_sum > 0.f) ? (m_used + log2f(l_sum)) / kLog2e : -INFINITY;
            tc_fence_before();
          } else {
            // ---- a piece of a unit.  The pieces of a unit draw tickets on the unit's "claimed" counter (the
            // draw was started while the last key tile was still being processed): the piece with the last
            // ticket becomes the merger and keeps its O in TMEM; every other piece leaves its normalised
            // output O/l (bf16) and (m, l) in its CTA's slot and then bumps the unit's "ready" counter.  The
            // merger waits (bounded) until all other pieces are ready - they hold tickets, so they are in
            // their epilogue - and combines out = sum_p w_p O_p / sum_p w_p with w_p = l_p 2^(m_p - max m).
            // Every piece enters the sum as its bf16-rounded normalised output, the merger's own included,
            // and the sum runs in piece order with one fused multiply-add per piece, so the result does not
            // depend on which piece merges.  Both counters carry the call's epoch: no initialisation needed.
            // Partial outputs are stored column-group major, [slot][D/8][MT*128 rows][8 bf16]: a warp writes
            // and reads 512 contiguous bytes per instruction.
            constexpr int kRows = MT * 128;
            const int rr = wg * 128 + row;
            // The unit's real tiles occupy [real0, uend) of the virtual tile space.  CTA groups k_first..k_last
            // hold them, one piece each (a group between the two lies wholly inside the unit), and this CTA's
            // group is one of them: two short walks over the cut table find both ends.
            const int real0 = it.layer * sch.per_layer + prm.Hkv * cum[it.b] + it.hk * (it.len + kSetupCost) + kSetupCost;
            const int uend = real0 + it.len;
            int k_first = group, k_last = group;
            while (gs[k_first] > real0) --k_first;
            while (gs[k_last + 1] < uend) ++k_last;
            const int n_frag = k_last - k_first + 1;
            // slot of the piece CTA group k holds: slot 1 of its CTA if the unit starts in that group, else slot 0
            auto piece_slot = [&](int k) -> int { return (k * prm.NP + pair) * 2 + (k == k_first ? 1 : 0); };
            const int my_slot = piece_slot(group);
            unsigned long long* ctr = claim_ctr;
            TV_PROF_T(ep[1]);
            if (threadIdx.x == 128) {
              int ticket;
              if (claim_ret == claim_assumed) {
                ticket = claim_cnt + 1;                      // the early draw went through
              } else {
                ticket = bump_counter(ctr, claim_ret, prm.epoch);
              }
              const int merger = (ticket == n_frag) ? 1 : 0;
              if (merger) {
                // wait until the other n_frag - 1 pieces have published their partials
                const unsigned long long t0 = globaltimer_ns();
                while (true) {
                  const unsigned long long v = *reinterpret_cast<volatile unsigned long long*>(ctr + 1);
                  const int ready = ((v >> 16) == prm.epoch) ? (int)(v & 0xffffu) : 0;
                  if (ready >= n_frag - 1) break;
                  if (*abort_flag || globaltimer_ns() - t0 > wait_limit) {
                    *abort_flag = 1;
                    break;
                  }
                }
                __threadfence();
                // every piece has drawn its ticket and published: nobody touches the two counters again in
                // this launch.  Clearing them lets the same launch be replayed with the same epoch (a captured
                // CUDA graph) and find them unused.
                *reinterpret_cast<volatile unsigned long long*>(ctr) = 0ull;
                *reinterpret_cast<volatile unsigned long long*>(ctr + 1) = 0ull;
              }
              *last_flag = merger;
            }
            ok = epi_sync();
            if (!ok || *abort_flag) { ok = false; break; }
            tr.mark(0x7000u | (*last_flag ? 1u : 0u));
            TV_PROF_T(ep[2]);
#ifdef TV_PROF
            ep_kind = (*last_flag ? 2u : 1u) | ((unsigned)n_frag << 4);
#endif
            const float inv_own = (row_active && l_sum > 0.f) ? 1.f / l_sum : 0.f;
            if (!*last_flag) {
              uint4* po = reinterpret_cast<uint4*>(prm.part_o) + (size_t)my_slot * (D / 8) * kRows;
              float* pml = prm.part_ml + (size_t)my_slot * 2 * kRows;
              store_rows(po + rr, kRows, inv_own, row_active, false);
              if (row_active) {
                pml[rr] = m_used;
                pml[kRows + rr] = l_sum;
              }
              tc_fence_before();
              TV_PROF_T(ep[3]);
              __threadfence();
              TV_PROF_T(ep[4]);
              tr.mark(0x6000u);
              ok = epi_sync();
              if (!ok) break;
              TV_PROF_T(ep[5]);
              if (threadIdx.x == 128 && !(prm.debug & 2)) {      // (debug bit 1: the piece is never announced)
                const unsigned long long seen = *reinterpret_cast<volatile unsigned long long*>(ctr + 1);
                bump_counter(ctr + 1, seen, prm.epoch);
              }
            } else {
              // ---- pass 1: reference maximum and total weight of the row.  (m, l) of the first four pieces
              // are fetched together (one round trip; a unit rarely has more), the rest one by one.  Loads are
              // issued by every thread (row rr always lies inside a slot; rows that are not active read stale
              // bytes and are masked by selects): no thread-divergent branch sits between the warp-wide TMEM ops.
              float pm[4], w4[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const int k = k_first + i;
                const bool other = k <= k_last && k != group;
                const float* q_ml = prm.part_ml + (size_t)piece_slot(other ? k : group) * 2 * kRows;
                const float m_k = __ldcg(q_ml + rr), l_k = __ldcg(q_ml + kRows + rr);
                pm[i] = other ? m_k : (k == group ? m_used : -INFINITY);
                w4[i] = other ? l_k : (k == group ? l_sum : 0.f);
              }
              float mm = fmaxf(fmaxf(pm[0], pm[1]), fmaxf(pm[2], pm[3]));
#pragma unroll 1
              for (int k = k_first + 4; k <= k_last; ++k)
                mm = fmaxf(mm, k == group ? m_used : __ldcg(prm.part_ml + (size_t)piece_slot(k) * 2 * kRows + rr));
              float lt = 0.f;
#pragma unroll
              for (int i = 0; i < 4; ++i) {       // weights w_p = l_p 2^(m_p - mm), summed in piece order
                w4[i] *= fast_exp2(pm[i] - mm);
                lt += w4[i];
              }
              auto late_weight = [&](int k) -> float {     // pieces past the fourth
                if (k == group) return l_sum * fast_exp2(m_used - mm);
                const float* q_ml = prm.part_ml + (size_t)piece_slot(k) * 2 * kRows;
                return __ldcg(q_ml + kRows + rr) * fast_exp2(__ldcg(q_ml + rr) - mm);
              };
#pragma unroll 1
              for (int k = k_first + 4; k <= k_last; ++k) lt += late_weight(k);
              if (!row_active) lt = 0.f;
              const float inv = (row_active && lt > 0.f) ? 1.f / lt : 0.f;
              TV_PROF_USE(__float_as_uint(inv));
              TV_PROF_T(ep[3]);
              // ---- pass 2: 64 output columns at a time, pieces in order (one fused multiply-add per piece and
              // element, two elements per instruction); the own piece comes from TMEM and enters as its
              // bf16-rounded normalised output, like every other piece
              const float2 inv_own2 = make_float2(inv_own, inv_own), inv2 = make_float2(inv, inv);
#pragma unroll 1
              for (int hq = 0; hq < D / 64; ++hq) {
                float2 acc[32];
#pragma unroll
                for (int c = 0; c < 32; ++c) acc[c] = make_float2(0.f, 0.f);
#pragma unroll 1
                for (int k = k_first; k <= k_last; ++k) {
                  const int i = k - k_first;
                  float w = i == 0 ? w4[0] : (i == 1 ? w4[1] : (i == 2 ? w4[2] : w4[3]));
                  if (i >= 4) w = late_weight(k);
                  const float2 w2 = make_float2(w, w);
                  if (k == group) {
                    TV_PROF_T(pc0);
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                      uint32_t o[32];
                      tmem_ld32(o_addr + (hq * 2 + q) * 32, o);
                      tmem_wait_ld();
#pragma unroll
                      for (int c = 0; c < 16; ++c) {
                        const float2 t = __fmul2_rn(make_float2(__uint_as_float(o[2 * c]), __uint_as_float(o[2 * c + 1])), inv_own2);
                        const uint32_t own = pack_bf16(t.x, t.y);
                        acc[q * 16 + c] = ffma2(w2, make_float2(__uint_as_float(own << 16), __uint_as_float(own & 0xffff0000u)),
                                                acc[q * 16 + c]);
                      }
                    }
#ifdef TV_PROF
                    TV_PROF_USE(__float_as_uint(acc[31].y));
                    ep_own += clock() - pc0;
#endif
                    continue;
                  }
                  const uint4* q_o = reinterpret_cast<const uint4*>(prm.part_o) + (size_t)piece_slot(k) * (D / 8) * kRows;
                  uint4 v[8];
                  TV_PROF_T(pc0);
#pragma unroll
                  for (int c = 0; c < 8; ++c) v[c] = __ldcg(q_o + (size_t)(hq * 8 + c) * kRows + rr);
#pragma unroll
                  for (int c = 0; c < 8; ++c) {
                    const uint32_t wv[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                      acc[4 * c + e] = ffma2(w2, make_float2(__uint_as_float(wv[e] << 16), __uint_as_float(wv[e] & 0xffff0000u)),
                                             acc[4 * c + e]);
                  }
#ifdef TV_PROF
                  TV_PROF_USE(__float_as_uint(acc[31].y));
                  ep_others += clock() - pc0;
#endif
                }
                if (row_exists) {
#pragma unroll
                  for (int c = 0; c < 8; c += 2) {
                    uint4 v[2];
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                      float2 t[4];
#pragma unroll
                      for (int x = 0; x < 4; ++x) t[x] = __fmul2_rn(acc[4 * (c + e) + x], inv2);
                      v[e].x = pack_bf16(t[0].x, t[0].y);
                      v[e].y = pack_bf16(t[1].x, t[1].y);
                      v[e].z = pack_bf16(t[2].x, t[2].y);
                      v[e].w = pack_bf16(t[3].x, t[3].y);
                      if (!row_active) v[e] = make_uint4(0, 0, 0, 0);
                    }
                    if (prm.out_al32) {
                      st_global_32B(orow + hq * 64 + c * 8, v[0], v[1]);
                    } else {
                      *reinterpret_cast<uint4*>(orow + hq * 64 + c * 8) = v[0];
                      *reinterpret_cast<uint4*>(orow + hq * 64 + c * 8 + 8) = v[1];
                    }
                  }
                }
              }
              if (row_exists && lse_p) *lse_p = (row_active && lt > 0.f) ? (mm + log2f(lt)) / kLog2e : -INFINITY;
              tc_fence_before();
              TV_PROF_T(ep[4]);
              ok = epi_sync();   // keeps the two warpgroups' barrier phases in step with the other branch
              if (!ok) break;
              TV_PROF_T(ep[5]);
            }
          }
        }
        tr.mark(0x8000u);
#ifdef TV_PROF
        prof[8] += clock() - pc1;
        if (tr.base && prof[9] < 24) {
          unsigned long long* e = tr.base + prof[9] * 8;
          e[0] = ep_kind; e[1] = ep_own;
          for (int i = 1; i < 6; ++i) e[1 + i] = ep[i] - ep[i - 1];
          e[7] = ep_others;      // pass 2: cycles from the loads of the other pieces to the end of their sums
        }
        prof[9] += 1;
#endif
        fill += 2 * nt;
      }
#ifdef TV_PROF
      if (tr.base)
      {
        for (int i = 0; i < 12; ++i) tr.base[kTraceCap - 16 + i] = prof[i];
        tr.base[kTraceCap - 2] = clock64() - prof_c0;
        tr.base[kTraceCap - 1] = globaltimer_ns() - prof_g0;
      }
#endif
    }
  } else {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
  }

  // ---- teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // give copies that may still be in flight time to land before the shared memory is released
    const unsigned long long t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) {
    }
    if (threadIdx.x == 0)
#pragma unroll 1
      for (int b = 0; b < prm.B; ++b) atomicOr(&prm.status[b], TV_ST_TIMEOUT);
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

bool encode_map(CUtensorMap* m, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides_bytes,
                const cuuint32_t* box) {
  cuuint32_t ones[5] = {1, 1, 1, 1, 1};
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims, strides_bytes, box, ones,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct Geometry {
  int G, NPT, n_row_tiles, MT, NP, sms, groups, grid;
  size_t ml_off, o_off, counters_off, counters_per_layer, total;
};

int sm_count() {
  static int sms = [] {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    return n;
  }();
  return sms;
}

constexpr int kCounterLayers = 32;      // layers whose counters the workspace of tv_attn_workspace_bytes holds

Geometry geometry(int B, int Nmax, int Hq, int Hkv, int d, bool query_device) {
  Geometry g{};
  g.G = Hq / Hkv;
  g.NPT = kTileM / g.G;
  g.n_row_tiles = (Nmax + g.NPT - 1) / g.NPT;
  g.MT = g.n_row_tiles > 1 ? 2 : 1;
  g.NP = (g.n_row_tiles + g.MT - 1) / g.MT;
  g.sms = query_device ? sm_count() : 148;
  g.groups = g.sms / g.NP > 0 ? g.sms / g.NP : 1;
  g.grid = g.groups * g.NP;
  // workspace: (m,l) pairs, partial O (both sized for 160 SMs so the size does not depend on the device), then
  // the units' counters, layer after layer: as many layers as fit behind the partials can share one launch
  const size_t max_ctas = 160 > g.grid ? 160 : g.grid;
  size_t off = 0;
  g.ml_off = off;
  off += max_ctas * 2 * (size_t)g.MT * 128 * 2 * sizeof(float);
  off = (off + 255) & ~size_t(255);
  g.o_off = off;
  off += max_ctas * 2 * (size_t)g.MT * 128 * d * sizeof(tv_bf16);
  off = (off + 255) & ~size_t(255);
  g.counters_off = off;
  g.counters_per_layer = ((size_t)B * Hkv * g.NP * 2 * sizeof(unsigned long long) + 255) & ~size_t(255);
  g.total = off + kCounterLayers * g.counters_per_layer;
  return g;
}

std::atomic<unsigned long long*> g_trace{nullptr};

// Tag of a call in its workspace counters (48 bits, never repeated within a process): the only state the
// library keeps for this entry point besides the cached driver entry point and device attributes.
unsigned long long next_epoch() {
  static std::atomic<unsigned long long> ctr{
      (unsigned long long)std::chrono::steady_clock::now().time_since_epoch().count() * 2654435761ull};
  return ctr.fetch_add(1, std::memory_order_relaxed) & 0xffffffffffffull;
}

template <int D, int MT>
cudaError_t launch(const Geometry& g, const CUtensorMap* maps, const AttnParams& prm, cudaStream_t s) {
  using L = SmemLayout<D, MT>;
  static std::atomic<bool> configured[64];
  auto kern = tree_attn_kernel<D, MT>;
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64 || !configured[dev].load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev].store(true, std::memory_order_release);
  }
  // Programmatic stream serialisation: this launch may be scheduled while the kernel in front is still
  // running (if that kernel allows it); the kernel itself waits before it touches anything that kernel writes.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(g.grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = L::kTotal;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, maps[0], maps[1], maps[2], maps[3], maps[4], prm);
}

struct AttnOptions {
  bool early = false;                              // TV_ATTN_STABLE_INPUTS was promised
  unsigned long long wait_limit_ns = kWaitLimitNs;
  int debug = 0;
};

// Layer strides of a call (elements); a single-layer call has L = 1 and strides that are never used.
struct LayerStrides {
  int64_t q = 0, cache = 0, tree = 0, out = 0;
};

// One launch over L layers.  Both layouts of the committed cache: contiguous [L,B,Hkv,Scap,d]
// (block_table == nullptr) or, for one layer, pages [n_pages,Hkv,128,d] named by block_table[B,max_blocks]
// (then Scap = 128 * max_blocks).  The layer is the outermost coordinate of every tensor map.
int attn_launch(const tv_bf16* q, const tv_bf16* k_cache, const tv_bf16* v_cache,
                const int32_t* block_table, int n_pages, int max_blocks,
                const tv_bf16* k_tree, const tv_bf16* v_tree, bool in_cache,
                const int32_t* prefix_len, const int32_t* n_nodes, const uint32_t* anc_bits,
                int L, const LayerStrides& ls, int B, int Nmax, int Hq, int Hkv, int d, int Scap, float scale,
                tv_bf16* out, float* lse, void* workspace, int32_t* status, const AttnOptions& opt, cudaStream_t s) {
  const Geometry g = geometry(B, Nmax, Hq, Hkv, d, true);
  CUtensorMap maps[5];
  {
    const cuuint64_t e = 2;
    const cuuint64_t layers = (cuuint64_t)L;
    // a stride of a dimension of extent 1 is never used, but has to be a valid one
    const cuuint64_t q_ls = L > 1 ? (cuuint64_t)ls.q * e : (cuuint64_t)B * Nmax * Hq * d * e;
    const cuuint64_t t_ls = L > 1 ? (cuuint64_t)ls.tree * e : (cuuint64_t)B * Nmax * Hkv * d * e;
    cuuint64_t qd[5] = {(cuuint64_t)d, (cuuint64_t)Hq, (cuuint64_t)Nmax, (cuuint64_t)B, layers};
    cuuint64_t qs[4] = {(cuuint64_t)d * e, (cuuint64_t)Hq * d * e, (cuuint64_t)Nmax * Hq * d * e, q_ls};
    cuuint32_t qb[5] = {64, (cuuint32_t)g.G, (cuuint32_t)g.NPT, 1, 1};
    // rows of one (sequence, KV head) slab, or of one (page, KV head) slab of 128 rows
    const cuuint64_t slab_rows = block_table ? (cuuint64_t)kTileN : (cuuint64_t)Scap;
    const cuuint64_t slabs = block_table ? (cuuint64_t)n_pages * Hkv : (cuuint64_t)B * Hkv;
    const cuuint64_t c_ls = L > 1 ? (cuuint64_t)ls.cache * e : slabs * slab_rows * d * e;
    cuuint64_t cd[4] = {(cuuint64_t)d, slab_rows, slabs, layers};
    cuuint64_t cs[3] = {(cuuint64_t)d * e, slab_rows * d * e, c_ls};
    cuuint32_t cb[4] = {64, kTileN, 1, 1};
    cuuint64_t td[5] = {(cuuint64_t)d, (cuuint64_t)Hkv, (cuuint64_t)Nmax, (cuuint64_t)B, layers};
    cuuint64_t ts[4] = {(cuuint64_t)d * e, (cuuint64_t)Hkv * d * e, (cuuint64_t)Nmax * Hkv * d * e, t_ls};
    cuuint32_t tb[5] = {64, 1, kTileN, 1, 1};
    const bool ok = encode_map(&maps[0], q, 5, qd, qs, qb) && encode_map(&maps[1], k_cache, 4, cd, cs, cb) &&
                    encode_map(&maps[2], v_cache, 4, cd, cs, cb) &&
                    (in_cache ? (maps[3] = maps[1], maps[4] = maps[2], true)      // placeholders the kernel never uses
                              : (encode_map(&maps[3], k_tree, 5, td, ts, tb) && encode_map(&maps[4], v_tree, 5, td, ts, tb)));
    if (!ok) return tv::fail(TV_ERR_CUDA, "tree_verify_attn: cuTensorMapEncodeTiled failed");
  }
  AttnParams prm{};
  prm.prefix_len = prefix_len;
  prm.n_nodes = n_nodes;
  prm.anc_bits = anc_bits;
  prm.out = out;
  prm.lse = lse;
  prm.status = status;
  // The launch touches the workspace only after its grid-dependency wait, that is after every earlier kernel of
  // the stream has completed: consecutive launches may share it although they overlap on the device.
  char* ws = static_cast<char*>(workspace);
  prm.counters = reinterpret_cast<unsigned long long*>(ws + g.counters_off);
  prm.part_ml = reinterpret_cast<float*>(ws + g.ml_off);
  prm.part_o = reinterpret_cast<tv_bf16*>(ws + g.o_off);
  prm.epoch = next_epoch();
  prm.B = B; prm.Nmax = Nmax; prm.Hq = Hq; prm.Hkv = Hkv; prm.Scap = Scap;
  prm.G = g.G; prm.NPT = g.NPT; prm.NP = g.NP; prm.W = (Nmax + 31) / 32; prm.groups = g.groups;
  prm.TT = (Nmax + kTileN - 1) / kTileN;
  prm.scale = scale;
  prm.tree_in_cache = in_cache ? 1 : 0;
  prm.block_table = block_table;
  prm.max_blocks = max_blocks;
  prm.n_pages = n_pages;
  prm.out_al32 = ((reinterpret_cast<uintptr_t>(out) & 31u) == 0 && (L == 1 || (ls.out * 2) % 32 == 0)) ? 1 : 0;
  prm.q_box_bytes = 64u * (uint32_t)g.G * (uint32_t)g.NPT * 2u;
  prm.trace = g_trace.load(std::memory_order_relaxed);
  prm.scale_log2e = scale * kLog2e;
  prm.early = opt.early ? 1 : 0;
  prm.wait_limit_ns = opt.wait_limit_ns;
  prm.debug = opt.debug;
  prm.L = L;
  prm.out_layer_stride = ls.out;
  cudaError_t e;
  if (d == 128) e = g.MT == 2 ? launch<128, 2>(g, maps, prm, s) : launch<128, 1>(g, maps, prm, s);
  else e = g.MT == 2 ? launch<64, 2>(g, maps, prm, s) : launch<64, 1>(g, maps, prm, s);
  if (e != cudaSuccess) return tv::fail(TV_ERR_CUDA, "tree_verify_attn: launch failed: %s", cudaGetErrorString(e));
  tv::count_launches(1);
  return TV_OK;
}

int attn_entry(const tv_bf16* q,
               const tv_bf16* k_cache, const tv_bf16* v_cache,
               const int32_t* block_table, int n_pages, int max_blocks,
               const tv_bf16* k_tree, const tv_bf16* v_tree,
               const int32_t* prefix_len, const int32_t* n_nodes,
               const uint32_t* anc_bits,
               int L, const LayerStrides& ls, int B, int Nmax, int Hq, int Hkv, int d, int Scap, float scale,
               tv_bf16* out, float* lse,
               void* workspace, size_t workspace_bytes,
               int32_t* status, const AttnOptions& opt, tv_stream stream) {
  TV_REQUIRE(q && k_cache && v_cache && prefix_len && n_nodes && anc_bits && out && status && workspace,
             "tree_verify_attn: NULL pointer");
  TV_REQUIRE((k_tree == nullptr) == (v_tree == nullptr), "tree_verify_attn: k_tree and v_tree must both be given or both be NULL");
  const bool in_cache = (k_tree == nullptr);       // the tree's K/V rows sit in the cache behind the prefix
  TV_REQUIRE(B >= 0 && B <= kMaxB, "tree_verify_attn: need 0 <= B <= 512");
  TV_REQUIRE(Nmax >= 1 && Nmax <= 256, "tree_verify_attn: Nmax must be in 1..256");
  TV_REQUIRE(d == 64 || d == 128, "tree_verify_attn: d must be 64 or 128");
  TV_REQUIRE(Hq >= 1 && Hkv >= 1 && Hq % Hkv == 0 && Hq / Hkv <= kTileM, "tree_verify_attn: need Hq %% Hkv == 0 and Hq/Hkv <= 128");
  TV_REQUIRE(Scap >= 1 && scale > 0.f, "tree_verify_attn: need Scap >= 1 and scale > 0");
  TV_REQUIRE(tv::aligned16(q) && tv::aligned16(k_cache) && tv::aligned16(v_cache) && tv::aligned16(k_tree) &&
                 tv::aligned16(v_tree) && tv::aligned16(out),
             "tree_verify_attn: tensors must be 16-byte aligned");
  TV_REQUIRE((reinterpret_cast<uintptr_t>(workspace) & 255u) == 0, "tree_verify_attn: workspace must be 256-byte aligned");
  if (B == 0 || L == 0) return TV_OK;
  const Geometry g = geometry(B, Nmax, Hq, Hkv, d, true);
  const long long tiles_per_layer = (long long)B * Hkv * ((Scap + kTileN - 1) / kTileN + 2 + kSetupCost);
  TV_REQUIRE(tiles_per_layer < (1ll << 31), "tree_verify_attn: B * Hkv * Scap is too large for the tile scheduler");
  if (g.grid > 160) return tv::fail(TV_ERR_INVALID_ARG, "tree_verify_attn: device with more than 160 SMs is not supported");
  if (workspace_bytes < g.counters_off + g.counters_per_layer)
    return tv::fail(TV_ERR_WORKSPACE, "tree_verify_attn: workspace of %zu bytes, need %zu", workspace_bytes,
                    g.counters_off + g.counters_per_layer);
  // Layers that share a launch: as many as the workspace has counters for and as the 31-bit tile space holds.
  long long per_launch = (long long)((workspace_bytes - g.counters_off) / g.counters_per_layer);
  const long long by_tiles = ((1ll << 31) - 1) / tiles_per_layer;
  if (per_launch > by_tiles) per_launch = by_tiles;
  if (per_launch > 65535) per_launch = 65535;
  AttnOptions o = opt;
  for (int l0 = 0; l0 < L; l0 += (int)per_launch) {
    const int nl = L - l0 < per_launch ? L - l0 : (int)per_launch;
    const tv_bf16* kc = k_cache + (size_t)l0 * ls.cache;
    const tv_bf16* vc = v_cache + (size_t)l0 * ls.cache;
    const int rc = attn_launch(q + (size_t)l0 * ls.q, kc, vc, block_table, n_pages, max_blocks,
                               in_cache ? kc : k_tree + (size_t)l0 * ls.tree, in_cache ? vc : v_tree + (size_t)l0 * ls.tree,
                               in_cache, prefix_len, n_nodes, anc_bits, nl, ls, B, Nmax, Hq, Hkv, d, Scap, scale,
                               out + (size_t)l0 * ls.out, lse ? lse + (size_t)l0 * B * Hq * Nmax : nullptr, workspace, status,
                               o, (cudaStream_t)stream);
    if (rc != TV_OK) return rc;
    o.early = true;       // behind a tree_verify_attn launch of this very call the inputs are stable
  }
  return TV_OK;
}

}  // namespace

// Tuning aid, live only in a library built with -DTV_TRACE: while a device buffer of 160 * 4 * 256 u64 is
// registered here, every tree_verify_attn launch records a per-CTA, per-role timeline (tag << 48 |
// globaltimer ns) into it.  NULL switches it off.
extern "C" TV_API void tv_debug_set_attn_trace(unsigned long long* device_buffer) {
  g_trace.store(device_buffer, std::memory_order_relaxed);
}

// Test aid for the failure path: tree_verify_attn with the limit of every bounded wait set to wait_limit_ns and,
// with mode bit 0, a producer warp that issues no copy at all, so that the first wait of the MMA issuer expires;
// with mode bit 1, pieces of cut units that never announce their partials, so that the poll of the merging piece expires.
// The launch must then end by itself with TV_ST_TIMEOUT in status[] of every sequence and leave the GPU usable.
extern "C" TV_API int tv_debug_attn_expire(const tv_bf16* q, const tv_bf16* k_cache, const tv_bf16* v_cache,
                                           const tv_bf16* k_tree, const tv_bf16* v_tree, const int32_t* prefix_len,
                                           const int32_t* n_nodes, const uint32_t* anc_bits, int B, int Nmax, int Hq,
                                           int Hkv, int d, int Scap, float scale, tv_bf16* out, float* lse,
                                           void* workspace, size_t workspace_bytes, int32_t* status,
                                           unsigned long long wait_limit_ns, int mode, tv_stream stream) {
  AttnOptions opt;
  opt.wait_limit_ns = wait_limit_ns;
  opt.debug = mode;
  return attn_entry(q, k_cache, v_cache, nullptr, 0, 0, k_tree, v_tree, prefix_len, n_nodes, anc_bits, 1, LayerStrides{}, B,
                    Nmax, Hq, Hkv, d, Scap, scale, out, lse, workspace, workspace_bytes, status, opt, stream);
}

extern "C" TV_API int tv_debug_attn_stream_only(const tv_bf16* q, const tv_bf16* k_cache, const tv_bf16* v_cache,
                                                const tv_bf16* k_tree, const tv_bf16* v_tree, const int32_t* prefix_len,
                                                const int32_t* n_nodes, const uint32_t* anc_bits, int L, int B, int Nmax,
                                                int Hq, int Hkv, int d, int Scap, int64_t q_layer_stride,
                                                int64_t cache_layer_stride, int64_t tree_layer_stride, tv_bf16* out,
                                                int64_t out_layer_stride, void* workspace, size_t workspace_bytes,
                                                int32_t* status, tv_stream stream) {
  TV_REQUIRE(L >= 0 && L <= 65535, "tv_debug_attn_stream_only: need 0 <= L <= 65535");
  TV_REQUIRE(q_layer_stride % 8 == 0 && cache_layer_stride % 8 == 0 && tree_layer_stride % 8 == 0 && out_layer_stride % 8 == 0,
             "tv_debug_attn_stream_only: layer strides must be multiples of 8 elements");
  AttnOptions opt;
  opt.early = true;
  opt.debug = 4;
  LayerStrides ls;
  ls.q = q_layer_stride;
  ls.cache = cache_layer_stride;
  ls.tree = tree_layer_stride;
  ls.out = out_layer_stride;
  return attn_entry(q, k_cache, v_cache, nullptr, 0, 0, k_tree, v_tree, prefix_len, n_nodes, anc_bits, L, ls, B, Nmax, Hq,
                    Hkv, d, Scap, 1.0f, out, nullptr, workspace, workspace_bytes, status, opt, stream);
}

extern "C" size_t tv_attn_workspace_bytes(int B, int Nmax, int Hq, int Hkv, int d, int Scap) {
  (void)Scap;
  if (B <= 0 || Nmax <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || Hq / Hkv > kTileM || d <= 0) return 256;
  return geometry(B, Nmax, Hq, Hkv, d, false).total;
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
  return attn_entry(q, k_cache, v_cache, nullptr, 0, 0, k_tree, v_tree, prefix_len, n_nodes, anc_bits, 1, LayerStrides{}, B,
                    Nmax, Hq, Hkv, d, Scap, scale, out, lse, workspace, workspace_bytes, status, AttnOptions{}, stream);
}

extern "C" int tree_verify_attn_paged(const tv_bf16* q,
                                      const tv_bf16* k_pages, const tv_bf16* v_pages,
                                      const int32_t* block_table,
                                      const tv_bf16* k_tree, const tv_bf16* v_tree,
                                      const int32_t* prefix_len, const int32_t* n_nodes,
                                      const uint32_t* anc_bits,
                                      int B, int Nmax, int Hq, int Hkv, int d, int n_pages, int max_blocks, float scale,
                                      tv_bf16* out, float* lse,
                                      void* workspace, size_t workspace_bytes,
                                      int32_t* status, tv_stream stream) {
  TV_REQUIRE(block_table && k_tree && v_tree, "tree_verify_attn_paged: NULL pointer");
  TV_REQUIRE(n_pages >= 1 && max_blocks >= 1 && max_blocks <= (1 << 20) && (long long)n_pages * Hkv < (1ll << 31),
             "tree_verify_attn_paged: need n_pages >= 1, 1 <= max_blocks <= 2^20, n_pages * Hkv < 2^31");
  return attn_entry(q, k_pages, v_pages, block_table, n_pages, max_blocks, k_tree, v_tree, prefix_len, n_nodes, anc_bits,
                    1, LayerStrides{}, B, Nmax, Hq, Hkv, d, max_blocks * kTileN, scale, out, lse, workspace, workspace_bytes,
                    status, AttnOptions{}, stream);
}

extern "C" int tree_verify_attn_layers(const tv_bf16* q,
                                       const tv_bf16* k_cache, const tv_bf16* v_cache,
                                       const tv_bf16* k_tree, const tv_bf16* v_tree,
                                       const int32_t* prefix_len, const int32_t* n_nodes,
                                       const uint32_t* anc_bits,
                                       int L, int B, int Nmax, int Hq, int Hkv, int d, int Scap, float scale,
                                       int64_t q_layer_stride, int64_t cache_layer_stride, int64_t tree_layer_stride,
                                       tv_bf16* out, int64_t out_layer_stride, float* lse,
                                       void* workspace, size_t workspace_bytes,
                                       int32_t* status, unsigned flags, tv_stream stream) {
  TV_REQUIRE(L >= 0 && L <= 65535, "tree_verify_attn_layers: need 0 <= L <= 65535");
  TV_REQUIRE(q_layer_stride % 8 == 0 && cache_layer_stride % 8 == 0 && tree_layer_stride % 8 == 0 && out_layer_stride % 8 == 0,
             "tree_verify_attn_layers: layer strides must be multiples of 8 elements");
  TV_REQUIRE((flags & ~(unsigned)(TV_ATTN_STABLE_INPUTS | TV_ATTN_LAUNCH_PER_LAYER)) == 0, "tree_verify_attn_layers: unknown flag");
  AttnOptions opt;
  opt.early = (flags & TV_ATTN_STABLE_INPUTS) != 0;
  LayerStrides ls;
  ls.q = q_layer_stride;
  ls.cache = cache_layer_stride;
  ls.tree = tree_layer_stride;
  ls.out = out_layer_stride;
  if (flags & TV_ATTN_LAUNCH_PER_LAYER) {      // exactly what L calls of tree_verify_attn issue
    for (int l = 0; l < L; ++l) {
      const int rc = attn_entry(q + (size_t)l * ls.q, k_cache + (size_t)l * ls.cache, v_cache + (size_t)l * ls.cache, nullptr,
                                0, 0, k_tree ? k_tree + (size_t)l * ls.tree : nullptr,
                                v_tree ? v_tree + (size_t)l * ls.tree : nullptr, prefix_len, n_nodes, anc_bits, 1,
                                LayerStrides{}, B, Nmax, Hq, Hkv, d, Scap, scale, out + (size_t)l * ls.out,
                                lse ? lse + (size_t)l * B * Hq * Nmax : nullptr, workspace, workspace_bytes, status, opt,
                                stream);
      if (rc != TV_OK) return rc;
      opt.early = true;      // behind a tree_verify_attn launch of this very call the inputs are stable
    }
    return TV_OK;
  }
  return attn_entry(q, k_cache, v_cache, nullptr, 0, 0, k_tree, v_tree, prefix_len, n_nodes, anc_bits, L, ls, B, Nmax, Hq,
                    Hkv, d, Scap, scale, out, lse, workspace, workspace_bytes, status, opt, stream);
}

extern "C" int tree_verify_attn_paged_layers(const tv_bf16* q,
                                             const tv_bf16* k_pages, const tv_bf16* v_pages,
                                             const int32_t* block_table,
                                             const tv_bf16* k_tree, const tv_bf16* v_tree,
                                             const int32_t* prefix_len, const int32_t* n_nodes,
                                             const uint32_t* anc_bits,
                                             int L, int B, int Nmax, int Hq, int Hkv, int d, int n_pages, int max_blocks,
                                             float scale,
                                             int64_t q_layer_stride, int64_t page_layer_stride, int64_t tree_layer_stride,
                                             tv_bf16* out, int64_t out_layer_stride, float* lse,
                                             void* workspace, size_t workspace_bytes,
                                             int32_t* status, unsigned flags, tv_stream stream) {
  TV_REQUIRE(block_table && k_tree && v_tree, "tree_verify_attn_paged_layers: NULL pointer");
  TV_REQUIRE(n_pages >= 1 && max_blocks >= 1 && max_blocks <= (1 << 20) && (long long)n_pages * Hkv < (1ll << 31),
             "tree_verify_attn_paged_layers: need n_pages >= 1, 1 <= max_blocks <= 2^20, n_pages * Hkv < 2^31");
  TV_REQUIRE(L >= 0 && L <= 65535, "tree_verify_attn_paged_layers: need 0 <= L <= 65535");
  TV_REQUIRE(q_layer_stride % 8 == 0 && page_layer_stride % 8 == 0 && tree_layer_stride % 8 == 0 && out_layer_stride % 8 == 0,
             "tree_verify_attn_paged_layers: layer strides must be multiples of 8 elements");
  TV_REQUIRE((flags & ~(unsigned)TV_ATTN_STABLE_INPUTS) == 0, "tree_verify_attn_paged_layers: unknown flag");
  AttnOptions opt;
  opt.early = (flags & TV_ATTN_STABLE_INPUTS) != 0;
  LayerStrides ls;
  ls.q = q_layer_stride;
  ls.cache = page_layer_stride;
  ls.tree = tree_layer_stride;
  ls.out = out_layer_stride;
  return attn_entry(q, k_pages, v_pages, block_table, n_pages, max_blocks, k_tree, v_tree, prefix_len, n_nodes, anc_bits, L,
                    ls, B, Nmax, Hq, Hkv, d, max_blocks * kTileN, scale, out, lse, workspace, workspace_bytes, status, opt,
                    stream);
}
