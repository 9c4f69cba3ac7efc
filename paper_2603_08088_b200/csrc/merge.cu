// tree_merge_partials: attention over a key set that was split in R disjoint ranges (one per GPU of a
// context-split group), from the per-range outputs and log-sum-exps (Section 6, "Limitations and future
// work": longer-context, multi-device serving; the attention is Section 2.4).  For every query row
//   out = sum_r w_r O_r / sum_r w_r,  w_r = exp(lse_r - max_r lse_r),  lse = max + log sum_r w_r.
// Pure streaming: R reads of the partials, one write; one thread per (row, 8 output columns).
#include "common.cuh"

#include <cuda_bf16.h>

namespace {

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

__global__ void merge_partials_kernel(const uint4* __restrict__ o_parts, const float* __restrict__ lse_parts, int R,
                                      int B, int Nmax, int Hq, int d8, uint4* __restrict__ out,
                                      float* __restrict__ lse_out) {
  const long long total = (long long)B * Nmax * Hq * d8;
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= total) return;
  const int cg = (int)(t % d8);
  const long long row = t / d8;                       // (b * Nmax + node) * Hq + h
  const int h = (int)(row % Hq);
  const long long bn = row / Hq;
  const int node = (int)(bn % Nmax);
  const int b = (int)(bn / Nmax);
  const long long rows = (long long)B * Nmax * Hq;
  const long long lse_idx = ((long long)b * Hq + h) * Nmax + node;
  float m = -INFINITY;
#pragma unroll 4
  for (int r = 0; r < R; ++r) m = fmaxf(m, __ldg(lse_parts + (long long)r * rows + lse_idx));
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  float tot = 0.f;
  if (m > -INFINITY) {
    // four ranges at a time: all loads of a group are in flight together; the payload of an empty range
    // (weight 0) may be anything, so it is replaced by zeros rather than multiplied
    for (int r0 = 0; r0 < R; r0 += 4) {
      float w[4];
      uint4 v[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int r = r0 + k < R ? r0 + k : R - 1;
        w[k] = __ldg(lse_parts + (long long)r * rows + lse_idx);
        v[k] = __ldg(o_parts + ((long long)r * rows + row) * d8 + cg);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float wk = (r0 + k < R) ? expf(w[k] - m) : 0.f;
        if (!(wk > 0.f)) v[k] = make_uint4(0u, 0u, 0u, 0u);
        tot += wk;
        acc[0] = fmaf(wk, bf16_lo(v[k].x), acc[0]);
        acc[1] = fmaf(wk, bf16_hi(v[k].x), acc[1]);
        acc[2] = fmaf(wk, bf16_lo(v[k].y), acc[2]);
        acc[3] = fmaf(wk, bf16_hi(v[k].y), acc[3]);
        acc[4] = fmaf(wk, bf16_lo(v[k].z), acc[4]);
        acc[5] = fmaf(wk, bf16_hi(v[k].z), acc[5]);
        acc[6] = fmaf(wk, bf16_lo(v[k].w), acc[6]);
        acc[7] = fmaf(wk, bf16_hi(v[k].w), acc[7]);
      }
    }
  }
  const float inv = tot > 0.f ? 1.f / tot : 0.f;
  uint4 o;
  o.x = pack_bf16(acc[0] * inv, acc[1] * inv);
  o.y = pack_bf16(acc[2] * inv, acc[3] * inv);
  o.z = pack_bf16(acc[4] * inv, acc[5] * inv);
  o.w = pack_bf16(acc[6] * inv, acc[7] * inv);
  out[row * d8 + cg] = o;
  if (lse_out && cg == 0) lse_out[lse_idx] = tot > 0.f ? m + logf(tot) : -INFINITY;
}

}  // namespace

extern "C" int tree_merge_partials(const tv_bf16* o_parts, const float* lse_parts, int R, int B, int Nmax, int Hq, int d,
                                   tv_bf16* out, float* lse, tv_stream stream) {
  TV_REQUIRE(o_parts && lse_parts && out, "tree_merge_partials: NULL pointer");
  TV_REQUIRE(R >= 1 && B >= 0 && Nmax >= 1 && Hq >= 1 && d >= 8 && d % 8 == 0,
             "tree_merge_partials: need R >= 1, B >= 0, Nmax >= 1, Hq >= 1, d a multiple of 8");
  TV_REQUIRE(tv::aligned16(o_parts) && tv::aligned16(out), "tree_merge_partials: tensors must be 16-byte aligned");
  if (B == 0) return TV_OK;
  const long long total = (long long)B * Nmax * Hq * (d / 8);
  TV_REQUIRE((total + 255) / 256 < (1ll << 31), "tree_merge_partials: problem too large for one launch");
  merge_partials_kernel<<<(unsigned)((total + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
      reinterpret_cast<const uint4*>(o_parts), lse_parts, R, B, Nmax, Hq, d / 8, reinterpret_cast<uint4*>(out), lse);
  TV_CUDA_OK(cudaGetLastError());
  tv::count_launches(1);
  return TV_OK;
}
