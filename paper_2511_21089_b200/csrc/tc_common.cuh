// Shared by the single-CTA and CTA-pair prefill kernels: tile constants, epilogue arguments and
// the two epilogues (TMEM accumulator -> global memory).
#pragma once
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace mlpmoe {
namespace tc {

constexpr int BM = 128;        // rows of one CTA's A tile = TMEM lanes
constexpr int BK = 64;         // K elements per stage: one 128-byte swizzled row of bf16
constexpr int UMMA_K = 16;
constexpr int NUM_THREADS = 192;

enum { EPI_SWIGLU = 0, EPI_OUT = 1 };

struct EpiArgs {
  const float* scale;   // EPI_SWIGLU: per-neuron scale (effective alpha of the neuron's branch)
  const float* R;       // EPI_OUT, optional fp32 residual
  void* out;            // H (bf16) or Y (fp32 / bf16)
  int64_t rows;         // valid rows (tokens)
  int64_t cols;         // valid output columns (EPI_OUT: d_model)
  int64_t ld;           // output row pitch in elements
  int out_bf16;         // EPI_OUT only
  uint32_t* status;
};

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Accumulator columns [0, half) hold gate, [half, 2*half) hold up, for the `half` neurons starting
// at compacted index neuron0.  This thread owns token `row` (its TMEM lane).
// H[row, neuron0 + j] = bf16( silu(gate_j) * up_j * scale[neuron0 + j] )   (Section 3.1, inner bracket)
__device__ __forceinline__ void epilogue_swiglu(uint32_t taddr, const EpiArgs& ep, int64_t row, int64_t neuron0, int half) {
  __nv_bfloat16* H = static_cast<__nv_bfloat16*>(ep.out);
#pragma unroll 1
  for (int c = 0; c < half; c += 32) {
    uint32_t g[32], u[32];
    ptx::tmem_ld_32x32(taddr + c, g);
    ptx::tmem_ld_32x32(taddr + half + c, u);
    ptx::tmem_ld_wait();
    const int64_t col0 = neuron0 + c;
    const float4* sc4 = reinterpret_cast<const float4*>(ep.scale + col0);
    uint32_t packed[16];
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
      const float4 s = __ldg(sc4 + i / 4);
      const float sv[4] = {s.x, s.y, s.z, s.w};
      float h[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float gv = __uint_as_float(g[i + e]);
        h[e] = __fdividef(gv, 1.0f + __expf(-gv)) * __uint_as_float(u[i + e]) * sv[e];
      }
      packed[i / 2] = pack_bf16(h[0], h[1]);
      packed[i / 2 + 1] = pack_bf16(h[2], h[3]);
    }
    if (row < ep.rows) {
      uint4* dst = reinterpret_cast<uint4*>(H + row * ep.ld + col0);
#pragma unroll
      for (int v = 0; v < 4; ++v) dst[v] = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
    }
  }
}

// Y[row, col_base + j] = (R[row, col_base + j] +) acc_j for j < bn, clipped to ep.cols (a multiple of 4).
__device__ __forceinline__ void epilogue_out(uint32_t taddr, const EpiArgs& ep, int64_t row, int64_t col_base, int bn) {
#pragma unroll 1
  for (int c = 0; c < bn; c += 32) {
    uint32_t a[32];
    ptx::tmem_ld_32x32(taddr + c, a);
    ptx::tmem_ld_wait();
    const int64_t col0 = col_base + c;
    if (row < ep.rows) {
#pragma unroll
      for (int v = 0; v < 8; ++v) {
        const int64_t col = col0 + 4 * v;
        if (col < ep.cols) {
          float4 o = make_float4(__uint_as_float(a[4 * v]), __uint_as_float(a[4 * v + 1]), __uint_as_float(a[4 * v + 2]),
                                 __uint_as_float(a[4 * v + 3]));
          if (ep.R != nullptr) {
            const float4 r = *reinterpret_cast<const float4*>(ep.R + row * ep.ld + col);
            o.x += r.x; o.y += r.y; o.z += r.z; o.w += r.w;
          }
          if (ep.out_bf16) {
            *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(ep.out) + row * ep.ld + col) =
                make_uint2(pack_bf16(o.x, o.y), pack_bf16(o.z, o.w));
          } else {
            *reinterpret_cast<float4*>(static_cast<float*>(ep.out) + row * ep.ld + col) = o;
          }
        }
      }
    }
  }
}

}  // namespace tc
}  // namespace mlpmoe
