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

enum { EPI_SWIGLU = 0, EPI_OUT = 1, EPI_SWIGLU_SPLIT3 = 2 };

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

// As epilogue_swiglu with the fp32 value h = silu(gate) * up * scale (accurate exp) written as its three-way
// bf16 split: piece s of H[row, j] goes to column s * ep.cols + j of a row of 3 * ep.cols (= ep.ld) elements.
// taddr2 != 0: a second accumulator of the same shape (the correction terms) is added to gate and up first.
__device__ __forceinline__ void epilogue_swiglu_split3(uint32_t taddr, const EpiArgs& ep, int64_t row, int64_t neuron0, int half,
                                                       uint32_t taddr2) {
  __nv_bfloat16* H = static_cast<__nv_bfloat16*>(ep.out);
#pragma unroll 1
  for (int c = 0; c < half; c += 16) {
    uint32_t g[16], u[16];
    ptx::tmem_ld_32x16(taddr + c, g);
    ptx::tmem_ld_32x16(taddr + half + c, u);
    ptx::tmem_ld_wait();
    if (taddr2 != 0) {
      uint32_t g2[16], u2[16];
      ptx::tmem_ld_32x16(taddr2 + c, g2);
      ptx::tmem_ld_32x16(taddr2 + half + c, u2);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        g[i] = __float_as_uint(__uint_as_float(g[i]) + __uint_as_float(g2[i]));
        u[i] = __float_as_uint(__uint_as_float(u[i]) + __uint_as_float(u2[i]));
      }
    }
    const int64_t col0 = neuron0 + c;
    uint32_t pk[3][8];
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
      __nv_bfloat16 p[3][2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const float gv = __uint_as_float(g[i + e]);
        const float h = gv / (1.0f + expf(-gv)) * __uint_as_float(u[i + e]) * __ldg(ep.scale + col0 + i + e);
        const __nv_bfloat16 a = __float2bfloat16_rn(h);
        const float r1 = h - __bfloat162float(a);
        const __nv_bfloat16 b = __float2bfloat16_rn(r1);
        p[0][e] = a; p[1][e] = b; p[2][e] = __float2bfloat16_rn(r1 - __bfloat162float(b));
      }
#pragma unroll
      for (int s = 0; s < 3; ++s) {
        __nv_bfloat162 v2(p[s][0], p[s][1]);
        pk[s][i / 2] = *reinterpret_cast<uint32_t*>(&v2);
      }
    }
    if (row < ep.rows) {
#pragma unroll
      for (int s = 0; s < 3; ++s) {
        uint4* dst = reinterpret_cast<uint4*>(H + row * ep.ld + s * ep.cols + col0);
        dst[0] = make_uint4(pk[s][0], pk[s][1], pk[s][2], pk[s][3]);
        dst[1] = make_uint4(pk[s][4], pk[s][5], pk[s][6], pk[s][7]);
      }
    }
  }
}

// Y[row, col_base + j] = (R[row, col_base + j] +) acc_j for j < bn, clipped to ep.cols (a multiple of 4).
// taddr2 != 0: a second accumulator of the same shape is added first (fp32, round to nearest).
__device__ __forceinline__ void epilogue_out(uint32_t taddr, const EpiArgs& ep, int64_t row, int64_t col_base, int bn,
                                             uint32_t taddr2 = 0) {
#pragma unroll 1
  for (int c = 0; c < bn; c += 32) {
    uint32_t a[32];
    ptx::tmem_ld_32x32(taddr + c, a);
    ptx::tmem_ld_wait();
    if (taddr2 != 0) {
      uint32_t b[32];
      ptx::tmem_ld_32x32(taddr2 + c, b);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 32; ++i) a[i] = __float_as_uint(__uint_as_float(a[i]) + __uint_as_float(b[i]));
    }
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

// ---------------------------------------------------------------------------------------------
// Epilogues that leave through shared memory and TMA: each epilogue warp owns two 4 KB staging
// tiles (32 rows x 128 bytes, 128-byte swizzle, 1024-byte aligned) and alternates between them.
// Lane r writes row r; the 16-byte chunk c of a row sits at chunk position c ^ (r % 8), which is
// both what the swizzled tensor map expects and free of bank conflicts.  One lane issues the
// bulk tensor store, which is clipped to the tensor's extent (rows >= n, columns >= d).
// ---------------------------------------------------------------------------------------------
constexpr int STAGING_TILE_BYTES = 4096;
constexpr int STAGING_BYTES_PER_WARP = 2 * STAGING_TILE_BYTES;

__device__ __forceinline__ void staging_write16(uint8_t* tile, int lane, int chunk, uint4 v) {
  *reinterpret_cast<uint4*>(tile + lane * 128 + ((chunk ^ (lane & 7)) << 4)) = v;
}

__device__ __forceinline__ float silu_mul(uint32_t g_bits, uint32_t u_bits, float sc) {
  const float g = __uint_as_float(g_bits);
  return __fdividef(g, 1.0f + __expf(-g)) * __uint_as_float(u_bits) * sc;
}

// gate|up epilogue for one 128-neuron tile.  tm_h: bf16 [n x Ipad], box 64 x 32.  `tiles_stored`
// counts this warp's staging tiles so far (selects the buffer).  `release` is called as soon as
// the accumulator has been read completely, before the arithmetic and the stores finish.
template <typename Release>
__device__ __forceinline__ void epilogue_swiglu_tma(uint32_t taddr, const float* __restrict__ scale, const CUtensorMap* tm_h,
                                                    uint8_t* staging, uint32_t& tiles_stored, int lane, int32_t row0,
                                                    int32_t neuron0, Release release) {
  uint32_t g[2][32], u[2][32];
  ptx::tmem_ld_32x32(taddr, g[0]);
  ptx::tmem_ld_32x32(taddr + 128, u[0]);
#pragma unroll
  for (int s = 0; s < 4; ++s) {          // four groups of 32 neurons
    ptx::tmem_ld_wait();
    if (s < 3) {
      ptx::tmem_ld_32x32(taddr + 32 * (s + 1), g[(s + 1) & 1]);
      ptx::tmem_ld_32x32(taddr + 128 + 32 * (s + 1), u[(s + 1) & 1]);
    } else {
      release();
    }
    uint8_t* tile = staging + (tiles_stored & 1u) * STAGING_TILE_BYTES;
    if ((s & 1) == 0) {                   // a new 64-neuron staging tile: its previous store must have been read
      if (lane == 0) ptx::tma_store_wait_read<1>();
      __syncwarp();
    }
    const float4* sc4 = reinterpret_cast<const float4*>(scale + neuron0 + 32 * s);
#pragma unroll
    for (int q = 0; q < 4; ++q) {         // 8 neurons -> one 16-byte chunk
      const float4 s0 = __ldg(sc4 + 2 * q), s1 = __ldg(sc4 + 2 * q + 1);
      const uint32_t* gg = &g[s & 1][8 * q];
      const uint32_t* uu = &u[s & 1][8 * q];
      uint4 v;
      v.x = pack_bf16(silu_mul(gg[0], uu[0], s0.x), silu_mul(gg[1], uu[1], s0.y));
      v.y = pack_bf16(silu_mul(gg[2], uu[2], s0.z), silu_mul(gg[3], uu[3], s0.w));
      v.z = pack_bf16(silu_mul(gg[4], uu[4], s1.x), silu_mul(gg[5], uu[5], s1.y));
      v.w = pack_bf16(silu_mul(gg[6], uu[6], s1.z), silu_mul(gg[7], uu[7], s1.w));
      staging_write16(tile, lane, 4 * (s & 1) + q, v);
    }
    if ((s & 1) == 1) {
      ptx::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        ptx::tma_store_2d(tm_h, tile, neuron0 + 32 * (s - 1), row0);
        ptx::tma_store_commit();
      }
      ++tiles_stored;
    }
  }
}

// down epilogue, fp32 output: bn accumulator columns (a multiple of 32) starting at col_base.
// tm_y: fp32 [n x d], box 32 x 32.  accumulate != 0 adds onto Y (the residual stream updated
// in place), otherwise Y is overwritten.
template <typename Release>
__device__ __forceinline__ void epilogue_out_tma(uint32_t taddr, const CUtensorMap* tm_y, uint8_t* staging,
                                                 uint32_t& tiles_stored, int lane, int32_t row0, int32_t col_base, int bn,
                                                 int accumulate, Release release) {
  uint32_t a[2][32];
  ptx::tmem_ld_32x32(taddr, a[0]);
  const int chunks = bn / 32;
#pragma unroll 1
  for (int c = 0; c < chunks; c += 2) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int cc = c + e;
      if (cc < chunks) {
        ptx::tmem_ld_wait();
        if (cc + 1 < chunks) ptx::tmem_ld_32x32(taddr + 32 * (cc + 1), a[(e + 1) & 1]);
        else release();
        uint8_t* tile = staging + (tiles_stored & 1u) * STAGING_TILE_BYTES;
        if (lane == 0) ptx::tma_store_wait_read<1>();
        __syncwarp();
#pragma unroll
        for (int q = 0; q < 8; ++q)
          staging_write16(tile, lane, q, make_uint4(a[e][4 * q], a[e][4 * q + 1], a[e][4 * q + 2], a[e][4 * q + 3]));
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          if (accumulate) ptx::tma_reduce_add_2d(tm_y, tile, col_base + 32 * cc, row0);
          else ptx::tma_store_2d(tm_y, tile, col_base + 32 * cc, row0);
          ptx::tma_store_commit();
        }
        ++tiles_stored;
      }
    }
  }
}

}  // namespace tc
}  // namespace mlpmoe
