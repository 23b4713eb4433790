// Shared by the two persistent decode-stack kernels (decode_stack.cu, decode_fused.cu): the split of a
// layer's neurons over the CTAs, the grid-wide events, and the RMSNorm of one token row.
//
// Work split.  The compacted neurons of a layer (Ipad, a multiple of 128, padding rows zero) are cut
// into units of 16; CTA c owns the contiguous units [bounds[c], bounds[c + 1]) (equal shares, built on
// the host), whatever the number of surviving neurons: every SM streams the same share of the
// gate|up weights, so a pruned layer is faster in proportion.  A CTA's range is walked in items of at
// most 8 units = 128 weight rows, the M side of one MMA; an item with r rows occupies r gate rows and
// r up rows of a stage (256 r bytes per 64-wide K-step) and the MMA reads 128 rows from each start:
// the rows past r are whatever the stage slot held before and only feed accumulator lanes that the
// epilogue ignores.
#pragma once
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace mlpmoe {
namespace dec {

using namespace ptx;

constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int NORM_VEC = 8;                           // float4 per lane the RMSNorm phase keeps in registers
constexpr uint32_t ARRIVALS_PER_CTA = 4;              // every epilogue warp arrives once per event

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async;" ::: "memory"); }
// The four epilogue warps (threads 64..191) only.
__device__ __forceinline__ void epilogue_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Event e has happened once counter[e] has reached the number of arrivals of a full grid.
__device__ __forceinline__ bool event_passed(const uint32_t* counter, uint32_t target) {
  return ld_acquire_u32(counter) >= target;
}
__device__ __forceinline__ bool event_wait(const uint32_t* counter, uint32_t target, volatile uint32_t* abort_flag,
                                           uint64_t limit_ns) {
  if (event_passed(counter, target)) return true;
  const uint64_t t0 = globaltimer_ns();
  uint32_t polls = 0;
  while (true) {
    if (event_passed(counter, target)) return true;
    __nanosleep(64);
    if ((++polls & 15u) == 0) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > limit_ns) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

// A CTA's phase A items of one layer.
struct Items {
  int lo, hi;                                        // units
  __device__ __forceinline__ Items(const DecodeStackLayer* L, int cta) : lo(L->bounds[cta]), hi(L->bounds[cta + 1]) {}
  __device__ __forceinline__ int count() const { return (hi - lo + kDecMaxUnitsPerItem - 1) / kDecMaxUnitsPerItem; }
  __device__ __forceinline__ int unit0(int i) const { return lo + i * kDecMaxUnitsPerItem; }
  __device__ __forceinline__ int rows(int i) const {
    const int left = hi - unit0(i);
    return kDecUnit * (left < kDecMaxUnitsPerItem ? left : kDecMaxUnitsPerItem);
  }
};

// RMSNorm of token row t by the four epilogue warps of a CTA (quad = warp % 4): r = x / sqrt(mean(x^2) + eps),
// rounded to bf16.  Each warp takes a quarter of the row and keeps it in registers; the four partial sums
// of squares meet in shared memory.  Every warp of the four must call this (named barrier), also when
// `active` is false (a wait has given up: no memory is touched then).
__device__ __forceinline__ void norm_row(const float* __restrict__ x, __nv_bfloat16* __restrict__ xnorm, int64_t t, int64_t d,
                                         float eps, int quad, int lane, volatile float* norm_part, bool active) {
  const float* row = x + t * d;
  const int64_t q = (d / 4 + 3) / 4 * 4;                 // columns per warp, a multiple of 4
  const int64_t c0 = static_cast<int64_t>(quad) * q, c1 = c0 + q < d ? c0 + q : d;
  float4 v[NORM_VEC];
  float ss = 0.f;
  if (active) {
#pragma unroll
    for (int i = 0; i < NORM_VEC; ++i) {
      const int64_t k = c0 + (static_cast<int64_t>(i) * 32 + lane) * 4;
      v[i] = k < c1 ? __ldcg(reinterpret_cast<const float4*>(row + k)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int i = 0; i < NORM_VEC; ++i) ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
    for (int64_t k = c0 + (static_cast<int64_t>(NORM_VEC) * 32 + lane) * 4; k < c1; k += 128) {   // rows wider than the register window
      const float4 w4 = __ldcg(reinterpret_cast<const float4*>(row + k));
      ss += w4.x * w4.x + w4.y * w4.y + w4.z * w4.z + w4.w * w4.w;
    }
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
  }
  if (lane == 0) norm_part[quad] = ss;
  epilogue_bar_sync();
  const float total = norm_part[0] + norm_part[1] + norm_part[2] + norm_part[3];
  epilogue_bar_sync();                                   // norm_part may be overwritten by the next row
  if (active) {
    const float inv = 1.0f / sqrtf(total / static_cast<float>(d) + eps);
    __nv_bfloat16* out = xnorm + t * d;
    auto store4 = [&](int64_t k, const float4& f) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(f.x * inv, f.y * inv), hi = __floats2bfloat162_rn(f.z * inv, f.w * inv);
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&lo);
      pk.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(out + k) = pk;
    };
#pragma unroll
    for (int i = 0; i < NORM_VEC; ++i) {
      const int64_t k = c0 + (static_cast<int64_t>(i) * 32 + lane) * 4;
      if (k < c1) store4(k, v[i]);
    }
    for (int64_t k = c0 + (static_cast<int64_t>(NORM_VEC) * 32 + lane) * 4; k < c1; k += 128)
      store4(k, __ldcg(reinterpret_cast<const float4*>(row + k)));
  }
}

}  // namespace dec
}  // namespace mlpmoe
