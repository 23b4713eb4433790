// Decode path (n_tokens <= 64): the layer is bound by streaming the weights from HBM once, so
// both kernels put the WEIGHTS on the 128-row side of the tensor-core tile and the few tokens
// on the narrow side (N = 16, 32 or 64), and keep a deep TMA ring of weight tiles in flight.
//
//   kernel 1 (Section 3.1, inner bracket): per CTA 128 neurons; two accumulators
//       G[j, t] = sum_k Wg'[j, k] X[t, k],   U[j, t] = sum_k Wu'[j, k] X[t, k]
//     live in the same TMEM lanes, so each epilogue thread owns one neuron and writes
//       Hd[t, j] = bf16( silu(G) * U * scale[j] ).
//   kernel 2 (outer product + branch sum): per CTA a 128-row slab of WdT and one slice of the
//     contraction range (split-K); partial sums go to a workspace and the warp that arrives
//     last for a 32-row group adds the slices in fixed order (deterministic, no spinning) and
//     writes Y[t, m] = (R[t, m] +) sum_j Hd[t, j] WdT[m, j].
//
// Warp roles as in the prefill kernels: warp 0 TMA producer, warp 1 TMEM owner + MMA issuer,
// warps 2..5 epilogue.
//
// Back-to-back kernels: both kernels are launched with programmatic stream serialization, use
// little enough shared memory (about 120 KB and 98 KB) and tensor memory (256 + 128 columns) for a
// CTA of each to share an SM, and their producers start streaming WEIGHT tiles - which no earlier
// kernel writes - before waiting for the previous kernel; only the activation tiles wait.  The
// weight stream of the next kernel thus starts while the previous kernel drains.
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace mlpmoe {
namespace {

using namespace ptx;

constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int NUM_THREADS = 192;
constexpr int MAXN = kDecodeMaxTokens;            // widest token tile

// kernel 1: stage = 256 weight rows (128 gate + 128 up) + token tile
constexpr int K1_W_BYTES = 256 * BK * 2;
constexpr int K1_STAGE_BYTES = K1_W_BYTES + MAXN * BK * 2;
constexpr int K1_STAGES = 3;
constexpr int K1_BAR_OFFSET = K1_STAGES * K1_STAGE_BYTES;
constexpr int K1_SMEM_BYTES = K1_BAR_OFFSET + 256 + 1024;
// kernel 2: stage = 128 rows of WdT + activation tile
constexpr int K2_W_BYTES = 128 * BK * 2;
constexpr int K2_STAGE_BYTES = K2_W_BYTES + MAXN * BK * 2;
constexpr int K2_STAGES = 4;
constexpr int K2_BAR_OFFSET = K2_STAGES * K2_STAGE_BYTES;
constexpr int K2_SMEM_BYTES = K2_BAR_OFFSET + 256 + 1024;

__device__ __forceinline__ uint8_t* align_1024(uint8_t* p) {
  return reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~static_cast<uintptr_t>(1023));
}

// Reads `npad` fp32 columns of this thread's TMEM lane into v[0..npad).
__device__ __forceinline__ void load_acc_row(uint32_t taddr, int npad, float (&v)[MAXN]) {
#pragma unroll
  for (int c = 0; c < MAXN; c += 16) {     // npad is 16, 32 or 64: uniform across the CTA
    if (c < npad) {
      uint32_t r[16];
      tmem_ld_32x16(taddr + c, r);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) v[c + i] = __uint_as_float(r[i]);
    }
  }
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
decode_gateup_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x,
                     const float* __restrict__ scale, __nv_bfloat16* __restrict__ Hd, int64_t n, int64_t Ipad,
                     int num_tiles, int num_k_blocks, int npad, uint32_t* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align_1024(smem_raw);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + K1_BAR_OFFSET);
  uint64_t* empty_bar = full_bar + K1_STAGES;
  uint64_t* tfull_bar = empty_bar + K1_STAGES;
  uint64_t* tempty_bar = tfull_bar + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  constexpr uint32_t TMEM_COLS = 4 * MAXN;     // 2 buffers x (G | U)

  if (threadIdx.x == 0) {
    for (int s = 0; s < K1_STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull_bar[a], 1); mbar_init(&tempty_bar[a], 4); }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) { tmem_alloc(tmem_slot, TMEM_COLS); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  griddep_launch_dependents();          // the next kernel may begin its set-up
  const uint32_t stage_tx = K1_W_BYTES + static_cast<uint32_t>(npad) * BK * 2;

  if (warp == 0) {
    if (lane == 0) {
      prefetch_tensormap(&tm_w);
      prefetch_tensormap(&tm_x);
      int stage = 0; uint32_t phase = 0; bool ok = true;
      // weight tiles go out at once; the token tiles of those first stages follow once the kernel
      // that writes X has completed
      bool waited = false;
      int deferred = 0, def_stage[K1_STAGES], def_kb[K1_STAGES];
      auto flush = [&]() {
        griddep_wait();
        for (int i = 0; i < deferred; ++i)
          tma_load_2d(smem + def_stage[i] * K1_STAGE_BYTES + K1_W_BYTES, &tm_x, def_kb[i] * BK, 0, &full_bar[def_stage[i]]);
        waited = true;
      };
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        for (int kb = 0; kb < num_k_blocks; ++kb) {
          if (!waited && deferred == K1_STAGES) flush();
          if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
          uint8_t* s = smem + stage * K1_STAGE_BYTES;
          mbar_expect_tx(&full_bar[stage], stage_tx);
          tma_load_2d(s, &tm_w, kb * BK, tile * 256, &full_bar[stage]);
          if (waited) {
            tma_load_2d(s + K1_W_BYTES, &tm_x, kb * BK, 0, &full_bar[stage]);
          } else {
            def_stage[deferred] = stage;
            def_kb[deferred] = kb;
            ++deferred;
          }
          if (++stage == K1_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!waited) flush();
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = make_idesc_bf16_f32(128, static_cast<uint32_t>(npad));
      int stage = 0, acc = 0; uint32_t phase = 0, acc_phase = 0; bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        if (!mbar_wait_bounded(&tempty_bar[acc], acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t g_tmem = tmem_base + static_cast<uint32_t>(acc * 2 * MAXN);
        const uint32_t u_tmem = g_tmem + MAXN;
        for (int kb = 0; kb < num_k_blocks; ++kb) {
          if (!mbar_wait_bounded(&full_bar[stage], phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t s = smem_u32(smem + stage * K1_STAGE_BYTES);
          const uint64_t wg_desc = make_desc_sw128_kmajor(s);
          const uint64_t wu_desc = make_desc_sw128_kmajor(s + 128 * BK * 2);
          const uint64_t x_desc = make_desc_sw128_kmajor(s + K1_W_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint32_t accum = (kb | k) != 0 ? 1u : 0u;
            umma_bf16(g_tmem, wg_desc + 2 * k, x_desc + 2 * k, idesc, accum);
            umma_bf16(u_tmem, wu_desc + 2 * k, x_desc + 2 * k, idesc, accum);
          }
          umma_commit(&empty_bar[stage]);
          if (++stage == K1_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(&tfull_bar[acc]);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    griddep_wait();                       // Hd may still be read by the previous layer's second kernel
    const int quad = warp % 4;
    int acc = 0; uint32_t acc_phase = 0;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
      bool ok = mbar_wait_bounded(&tfull_bar[acc], acc_phase, abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + static_cast<uint32_t>(acc * 2 * MAXN) + (static_cast<uint32_t>(quad * 32) << 16);
      float g[MAXN], u[MAXN];
      load_acc_row(taddr, npad, g);
      load_acc_row(taddr + MAXN, npad, u);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tempty_bar[acc]);
      const int64_t j = static_cast<int64_t>(tile) * 128 + quad * 32 + lane;   // compacted neuron index
      const float sc = scale[j];
#pragma unroll
      for (int t = 0; t < MAXN; ++t) {
        if (t < n) {
          const float gv = g[t];
          const float h = __fdividef(gv, 1.0f + __expf(-gv)) * u[t] * sc;
          Hd[static_cast<int64_t>(t) * Ipad + j] = __float2bfloat16_rn(h);
        }
      }
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, TMEM_COLS); }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, kStatusTimeout);
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
decode_down_kernel(const __grid_constant__ CUtensorMap tm_wd, const __grid_constant__ CUtensorMap tm_h,
                   float* __restrict__ partial, uint32_t* __restrict__ counters, const float* R,
                   void* Y, int y_bf16, int accumulate, int64_t n, int64_t d, int num_m_blocks, int splits,
                   int total_k_blocks, int npad, uint32_t* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align_1024(smem_raw);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + K2_BAR_OFFSET);
  uint64_t* empty_bar = full_bar + K2_STAGES;
  uint64_t* tfull_bar = empty_bar + K2_STAGES;
  uint64_t* tempty_bar = tfull_bar + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  constexpr uint32_t TMEM_COLS = 2 * MAXN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < K2_STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull_bar[a], 1); mbar_init(&tempty_bar[a], 4); }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) { tmem_alloc(tmem_slot, TMEM_COLS); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  griddep_launch_dependents();          // the next kernel may begin its set-up
  const uint32_t stage_tx = K2_W_BYTES + static_cast<uint32_t>(npad) * BK * 2;
  const int num_items = num_m_blocks * splits;

  // work item -> (m block, split); split s covers k blocks [s*KB/S, (s+1)*KB/S)
  if (warp == 0) {
    if (lane == 0) {
      prefetch_tensormap(&tm_wd);
      prefetch_tensormap(&tm_h);
      int stage = 0; uint32_t phase = 0; bool ok = true;
      bool waited = false;                 // as in the first kernel: weights first, Hd tiles after the wait
      int deferred = 0, def_stage[K2_STAGES], def_kb[K2_STAGES];
      auto flush = [&]() {
        griddep_wait();
        for (int i = 0; i < deferred; ++i)
          tma_load_2d(smem + def_stage[i] * K2_STAGE_BYTES + K2_W_BYTES, &tm_h, def_kb[i] * BK, 0, &full_bar[def_stage[i]]);
        waited = true;
      };
      for (int item = blockIdx.x; ok && item < num_items; item += gridDim.x) {
        const int m_blk = item % num_m_blocks, sp = item / num_m_blocks;
        const int kb0 = static_cast<int>(static_cast<int64_t>(sp) * total_k_blocks / splits);
        const int kb1 = static_cast<int>(static_cast<int64_t>(sp + 1) * total_k_blocks / splits);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!waited && deferred == K2_STAGES) flush();
          if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
          uint8_t* s = smem + stage * K2_STAGE_BYTES;
          mbar_expect_tx(&full_bar[stage], stage_tx);
          tma_load_2d(s, &tm_wd, kb * BK, m_blk * 128, &full_bar[stage]);
          if (waited) {
            tma_load_2d(s + K2_W_BYTES, &tm_h, kb * BK, 0, &full_bar[stage]);
          } else {
            def_stage[deferred] = stage;
            def_kb[deferred] = kb;
            ++deferred;
          }
          if (++stage == K2_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!waited) flush();
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = make_idesc_bf16_f32(128, static_cast<uint32_t>(npad));
      int stage = 0, acc = 0; uint32_t phase = 0, acc_phase = 0; bool ok = true;
      for (int item = blockIdx.x; ok && item < num_items; item += gridDim.x) {
        const int sp = item / num_m_blocks;
        const int kb0 = static_cast<int>(static_cast<int64_t>(sp) * total_k_blocks / splits);
        const int kb1 = static_cast<int>(static_cast<int64_t>(sp + 1) * total_k_blocks / splits);
        if (kb1 == kb0) continue;            // empty slice: no accumulator is produced for it
        if (!mbar_wait_bounded(&tempty_bar[acc], acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * MAXN);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait_bounded(&full_bar[stage], phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t s = smem_u32(smem + stage * K2_STAGE_BYTES);
          const uint64_t w_desc = make_desc_sw128_kmajor(s);
          const uint64_t h_desc = make_desc_sw128_kmajor(s + K2_W_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_bf16(d_tmem, w_desc + 2 * k, h_desc + 2 * k, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
          umma_commit(&empty_bar[stage]);
          if (++stage == K2_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(&tfull_bar[acc]);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    griddep_wait();                       // partial sums, counters and Y belong to earlier kernels until now
    const int quad = warp % 4;
    int acc = 0; uint32_t acc_phase = 0;
    for (int item = blockIdx.x; item < num_items; item += gridDim.x) {
      const int m_blk = item % num_m_blocks, sp = item / num_m_blocks;
      const int kb0 = static_cast<int>(static_cast<int64_t>(sp) * total_k_blocks / splits);
      const int kb1 = static_cast<int>(static_cast<int64_t>(sp + 1) * total_k_blocks / splits);
      float v[MAXN];
      if (kb1 > kb0) {                       // uniform across the CTA: an empty slice issues no MMA and no commit
        bool ok = mbar_wait_bounded(&tfull_bar[acc], acc_phase, abort_flag);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        tc_fence_after();
        const uint32_t taddr = tmem_base + static_cast<uint32_t>(acc * MAXN) + (static_cast<uint32_t>(quad * 32) << 16);
        load_acc_row(taddr, npad, v);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tempty_bar[acc]);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      } else {
#pragma unroll
        for (int t = 0; t < MAXN; ++t) v[t] = 0.f;
      }
      const int64_t m = static_cast<int64_t>(m_blk) * 128 + quad * 32 + lane;    // output feature of this thread
      const bool m_ok = m < d;
      if (accumulate) {
        // Y (fp32) already holds the residual: every slice adds its part, no staging and no hand-over
        if (m_ok) {
#pragma unroll
          for (int t = 0; t < MAXN; ++t)
            if (t < n) atomicAdd(static_cast<float*>(Y) + static_cast<int64_t>(t) * d + m, v[t]);
        }
        continue;
      }
      // 1. publish this slice's partial row
      if (m_ok) {
        float4* dst = reinterpret_cast<float4*>(partial + (static_cast<int64_t>(sp) * d + m) * npad);
#pragma unroll
        for (int t = 0; t < MAXN; t += 4)
          if (t < npad) dst[t / 4] = make_float4(v[t], v[t + 1], v[t + 2], v[t + 3]);
      }
      __threadfence();
      __syncwarp();
      // 2. count arrivals for this 32-row group; the last warp reduces
      uint32_t old = 0;
      if (lane == 0) old = atomicAdd(&counters[m_blk * 4 + quad], 1u);
      old = __shfl_sync(0xFFFFFFFFu, old, 0);
      if (old == static_cast<uint32_t>(splits - 1)) {
        __threadfence();
        if (m_ok) {
          float accv[MAXN];
#pragma unroll
          for (int t = 0; t < MAXN; ++t) accv[t] = 0.f;
          for (int s2 = 0; s2 < splits; ++s2) {
            const float4* src = reinterpret_cast<const float4*>(partial + (static_cast<int64_t>(s2) * d + m) * npad);
#pragma unroll
            for (int t = 0; t < MAXN; t += 4) {
              if (t < npad) {
                const float4 p = __ldcg(src + t / 4);
                accv[t] += p.x; accv[t + 1] += p.y; accv[t + 2] += p.z; accv[t + 3] += p.w;
              }
            }
          }
          // all residual loads first, then all stores: R may alias Y (in-place residual stream), and a
          // load placed after a store to a possibly aliasing address would wait for it
          if (R != nullptr) {
#pragma unroll
            for (int t = 0; t < MAXN; ++t)
              if (t < n) accv[t] += __ldcg(R + static_cast<int64_t>(t) * d + m);
          }
#pragma unroll
          for (int t = 0; t < MAXN; ++t) {
            if (t < n) {
              if (y_bf16) static_cast<__nv_bfloat16*>(Y)[static_cast<int64_t>(t) * d + m] = __float2bfloat16_rn(accv[t]);
              else static_cast<float*>(Y)[static_cast<int64_t>(t) * d + m] = accv[t];
            }
          }
        }
        __syncwarp();
        if (lane == 0) counters[m_blk * 4 + quad] = 0;    // ready for the next call
      }
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, TMEM_COLS); }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, kStatusTimeout);
}

}  // namespace

cudaError_t decode_init() {
  cudaError_t e = cudaFuncSetAttribute(decode_gateup_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, K1_SMEM_BYTES);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(decode_down_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, K2_SMEM_BYTES);
}

cudaError_t launch_decode_gateup(const DecodeArgs& a, int num_sms, cudaStream_t st) {
  if (a.n == 0) return cudaSuccess;
  const int tiles1 = static_cast<int>(a.Ipad / 128);
  const int kb1 = static_cast<int>((a.d + BK - 1) / BK);
  const int grid1 = tiles1 < num_sms ? tiles1 : num_sms;
  return launch_pdl(decode_gateup_kernel, dim3(grid1), dim3(NUM_THREADS), K1_SMEM_BYTES, st, a.tm_w, a.tm_x, a.scale,
                    static_cast<__nv_bfloat16*>(a.Hd), a.n, a.Ipad, tiles1, kb1, a.npad, a.status);
}

cudaError_t launch_decode_down(const DecodeArgs& a, int num_sms, cudaStream_t st) {
  if (a.n == 0) return cudaSuccess;
  const int m_blocks = static_cast<int>((a.d + 127) / 128);
  const int items = m_blocks * a.splits;
  const int grid2 = items < num_sms ? items : num_sms;
  return launch_pdl(decode_down_kernel, dim3(grid2), dim3(NUM_THREADS), K2_SMEM_BYTES, st, a.tm_wd, a.tm_h, a.partial, a.counters,
                    a.R, a.Y, a.y_bf16, a.accumulate, a.n, a.d, m_blocks, a.splits, static_cast<int>(a.Ipad / BK), a.npad, a.status);
}

}  // namespace mlpmoe
