// Decode of a whole pre-norm stack (n_tokens <= 64) in ONE persistent, cooperatively launched
// kernel: x <- x + MLPMoE_l(RMSNorm(x)) for l = 0 .. L-1.  One CTA per SM; every CTA walks the same
// static sequence of phases per layer
//     N: RMSNorm of the token rows into the bf16 activation buffer
//     A: gate|up, H = bf16(silu(G) * U * scale), 128 neurons per work item      (Section 3.1)
//     B: down + branch sum, K slices added straight into the fp32 stream x
// separated by grid-wide events (one global arrival counter, bounded waits).  The producer warp
// never stops at an event with an empty ring: weight tiles depend on no earlier phase, so it keeps
// issuing them and only holds back the small activation tile of each stage until the event it
// needs has passed.  HBM therefore keeps streaming weights across phase and layer boundaries.
//
// Warp roles: warp 0 TMA producer, warp 1 TMEM owner + MMA issuer, warps 2..5 epilogue (and the
// RMSNorm phase).  Weights sit on the 128-row side of the MMA, tokens on N = 16 / 32 / 64.
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace mlpmoe {
namespace {

using namespace ptx;

constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int NUM_THREADS = 192;
constexpr int MAXN = kDecodeMaxTokens;
constexpr int STAGES = 5;
constexpr int W_BYTES = 256 * BK * 2;                 // phase A: 128 gate + 128 up rows; phase B uses the first half
constexpr int STAGE_BYTES = W_BYTES + MAXN * BK * 2;  // + token tile
constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
constexpr int SMEM_BYTES = BAR_OFFSET + 256 + 1024;
constexpr uint32_t TMEM_COLS = 4 * MAXN;              // 2 buffers x (G | U)
constexpr uint64_t WAIT_NS = 1000000000ull;
constexpr uint32_t ARRIVALS_PER_CTA = 4;              // every epilogue warp arrives once per event

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async;" ::: "memory"); }

// Events are numbered in program order, 3 per layer (N, A, B), and each has its own arrival counter
// (a CTA without work in a phase arrives at once, so one shared counter would let early arrivals
// at later events stand in for missing arrivals at earlier ones).  Event e has happened once
// counter[e] has reached arrivals_per_event.
__device__ __forceinline__ bool event_passed(const uint32_t* counter, uint32_t target) {
  return ld_acquire_u32(counter) >= target;
}
__device__ __forceinline__ bool event_wait(const uint32_t* counter, uint32_t target, volatile uint32_t* abort_flag) {
  if (event_passed(counter, target)) return true;
  const uint64_t t0 = globaltimer_ns();
  uint32_t polls = 0;
  while (true) {
    if (event_passed(counter, target)) return true;
    __nanosleep(64);
    if ((++polls & 15u) == 0) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > WAIT_NS) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

__device__ __forceinline__ void load_acc(uint32_t taddr, int npad, float (&v)[MAXN]) {
#pragma unroll
  for (int c = 0; c < MAXN; c += 16) {
    if (c < npad) {
      uint32_t r[16];
      tmem_ld_32x16(taddr + c, r);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) v[c + i] = __uint_as_float(r[i]);
    }
  }
}

// A CTA's share of phase B of one layer: units (128-row block of WdT, K-step) in block-major order,
// dealt in equal contiguous ranges; a range is cut at block boundaries into items.
struct BItem {
  int m_blk, kb_lo, kb_hi;
};
__device__ __forceinline__ int b_items(int cta, int ctas, int m_blocks, int kb2, BItem (&out)[4]) {
  const int64_t units = static_cast<int64_t>(m_blocks) * kb2;
  const int64_t lo = units * cta / ctas, hi = units * (cta + 1) / ctas;
  int n = 0;
  for (int64_t u = lo; u < hi && n < 4;) {
    const int m = static_cast<int>(u / kb2);
    const int64_t end = (static_cast<int64_t>(m) + 1) * kb2 < hi ? (static_cast<int64_t>(m) + 1) * kb2 : hi;
    out[n].m_blk = m;
    out[n].kb_lo = static_cast<int>(u - static_cast<int64_t>(m) * kb2);
    out[n].kb_hi = static_cast<int>(end - static_cast<int64_t>(m) * kb2);
    ++n;
    u = end;
  }
  return n;
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
decode_stack_kernel(const DecodeStackLayer* __restrict__ layers, int n_layers,
                    const __grid_constant__ CUtensorMap tm_x,   // xnorm [n x d] bf16, box 64 x npad
                    float* x, __nv_bfloat16* xnorm, int64_t n, int64_t d, int npad, float eps, uint32_t* event_counter,
                    uint32_t* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + BAR_OFFSET);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* tfull_bar = empty_bar + STAGES;
  uint64_t* tempty_bar = tfull_bar + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int cta = blockIdx.x, ctas = gridDim.x;
  const uint32_t per_event = static_cast<uint32_t>(ctas) * ARRIVALS_PER_CTA;
  const int m_blocks = static_cast<int>((d + 127) / 128);
  const int kb1 = static_cast<int>((d + BK - 1) / BK);

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull_bar[a], 1); mbar_init(&tempty_bar[a], 4); }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) { tmem_alloc(tmem_slot, TMEM_COLS); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t act_bytes = static_cast<uint32_t>(npad) * BK * 2;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tensormap(&tm_x);
      int stage = 0; uint32_t phase = 0; bool ok = true;
      // activation tiles that wait for the current gating event: (stage, tensor map, K-step)
      int deferred = 0, def_stage[STAGES], def_kb[STAGES];
      const CUtensorMap* def_map = nullptr;
      const uint32_t* gate = event_counter;  // counter of the gating event
      bool gate_open = false;
      auto flush = [&]() {
        fence_async_proxy();               // what the acquire made visible must be seen by the TMA reads
        for (int i = 0; i < deferred; ++i)
          tma_load_2d(smem + def_stage[i] * STAGE_BYTES + W_BYTES, def_map, def_kb[i] * BK, 0, &full_bar[def_stage[i]]);
        deferred = 0;
        gate_open = true;
      };
      // issues one stage: weights at once, the token tile as soon as the gate is open
      auto issue = [&](const CUtensorMap* wmap, int wrow, uint32_t wbytes, const CUtensorMap* amap, int kb) -> bool {
        if (!gate_open && (deferred == STAGES || event_passed(gate, per_event))) {
          if (deferred == STAGES && !event_wait(gate, per_event, abort_flag)) return false;
          flush();
        }
        if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, WAIT_NS)) return false;
        uint8_t* s = smem + stage * STAGE_BYTES;
        mbar_expect_tx(&full_bar[stage], wbytes + act_bytes);
        tma_load_2d(s, wmap, kb * BK, wrow, &full_bar[stage]);
        if (gate_open) {
          tma_load_2d(s + W_BYTES, amap, kb * BK, 0, &full_bar[stage]);
        } else {
          def_stage[deferred] = stage; def_kb[deferred] = kb; ++deferred;
        }
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        return true;
      };
      for (int l = 0; ok && l < n_layers; ++l) {
        const DecodeStackLayer* L = layers + l;
        const int Ipad = L->Ipad;
        // phase A needs event N(l): index 3l
        if (deferred > 0) { if (!event_wait(gate, per_event, abort_flag)) { ok = false; break; } flush(); }
        gate = event_counter + 3 * l; gate_open = false; def_map = &tm_x;
        for (int tile = cta; ok && tile < Ipad / 128; tile += ctas)
          for (int kb = 0; kb < kb1; ++kb)
            if (!issue(&L->tm_wgu, tile * 256, W_BYTES, &tm_x, kb)) { ok = false; break; }
        if (!ok) break;
        // phase B needs event A(l): index 3l + 1
        if (deferred > 0) { if (!event_wait(gate, per_event, abort_flag)) { ok = false; break; } flush(); }
        gate = event_counter + 3 * l + 1; gate_open = false; def_map = &L->tm_hd;
        BItem it[4];
        const int nit = b_items(cta, ctas, m_blocks, Ipad / BK, it);
        for (int i = 0; ok && i < nit; ++i)
          for (int kb = it[i].kb_lo; kb < it[i].kb_hi; ++kb)
            if (!issue(&L->tm_wdt, it[i].m_blk * 128, W_BYTES / 2, &L->tm_hd, kb)) { ok = false; break; }
      }
      if (ok && deferred > 0 && event_wait(gate, per_event, abort_flag)) flush();
    }
  }
  else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = make_idesc_bf16_f32(128, static_cast<uint32_t>(npad));
      int stage = 0, acc = 0; uint32_t phase = 0, acc_phase = 0; bool ok = true;
      // one accumulator item: two_acc = gate and up (phase A), else one accumulator (phase B)
      auto run_item = [&](int kbs, bool two_acc) -> bool {
        if (!mbar_wait_bounded(&tempty_bar[acc], acc_phase ^ 1u, abort_flag, WAIT_NS)) return false;
        tc_fence_after();
        const uint32_t g_tmem = tmem_base + static_cast<uint32_t>(acc * 2 * MAXN);
        for (int kb = 0; kb < kbs; ++kb) {
          if (!mbar_wait_bounded(&full_bar[stage], phase, abort_flag, WAIT_NS)) return false;
          tc_fence_after();
          const uint32_t s = smem_u32(smem + stage * STAGE_BYTES);
          const uint64_t w0 = make_desc_sw128_kmajor(s);
          const uint64_t w1 = make_desc_sw128_kmajor(s + 128 * BK * 2);
          const uint64_t xd = make_desc_sw128_kmajor(s + W_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint32_t accum = (kb | k) != 0 ? 1u : 0u;
            umma_bf16(g_tmem, w0 + 2 * k, xd + 2 * k, idesc, accum);
            if (two_acc) umma_bf16(g_tmem + MAXN, w1 + 2 * k, xd + 2 * k, idesc, accum);
          }
          umma_commit(&empty_bar[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        umma_commit(&tfull_bar[acc]);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
        return true;
      };
      for (int l = 0; ok && l < n_layers; ++l) {
        const int Ipad = layers[l].Ipad;
        for (int tile = cta; ok && tile < Ipad / 128; tile += ctas) ok = run_item(kb1, true);
        BItem it[4];
        const int nit = b_items(cta, ctas, m_blocks, Ipad / BK, it);
        for (int i = 0; ok && i < nit; ++i) ok = run_item(it[i].kb_hi - it[i].kb_lo, false);
      }
    }
  }
  else {
    // ------------------------------------------- epilogue warps (+ RMSNorm phase)
    const int quad = warp % 4;
    int acc = 0; uint32_t acc_phase = 0;
    bool ok = true;
    auto arrive_event = [&](int e) {       // this warp's part of the phase is written and visible
      __threadfence();
      __syncwarp();
      if (lane == 0) atomicAdd(event_counter + e, 1u);
    };
    auto wait_acc = [&]() -> bool {
      bool w = mbar_wait_bounded(&tfull_bar[acc], acc_phase, abort_flag, WAIT_NS);
      w = __all_sync(0xFFFFFFFFu, w);
      if (w) tc_fence_after();
      return w;
    };
    auto release_acc = [&]() {
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tempty_bar[acc]);
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    };
    for (int l = 0; ok && l < n_layers; ++l) {
      const DecodeStackLayer* L = layers + l;
      const int Ipad = L->Ipad;
      // ---- phase N: x is final once every K slice of the previous layer has been added
      if (l > 0) {
        bool w = event_wait(event_counter + 3 * l - 1, per_event, abort_flag);
        w = __all_sync(0xFFFFFFFFu, w);
        if (!w) { ok = false; break; }
      }
      for (int t = cta; t < n; t += ctas) {
        // each of the four warps sums the whole row (16 KB from L2) and writes its quarter of it
        const float* row = x + static_cast<int64_t>(t) * d;
        float ss = 0.f;
        for (int64_t k = lane * 4; k < d; k += 128) {
          const float4 v = __ldcg(reinterpret_cast<const float4*>(row + k));
          ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
        const float inv = 1.0f / sqrtf(ss / static_cast<float>(d) + eps);
        const int64_t q = (d / 4 + 3) / 4 * 4;                 // columns per warp, a multiple of 4
        const int64_t c0 = static_cast<int64_t>(quad) * q, c1 = c0 + q < d ? c0 + q : d;
        for (int64_t k = c0 + lane * 4; k < c1; k += 128) {
          const float4 v = __ldcg(reinterpret_cast<const float4*>(row + k));
          __nv_bfloat162 lo = __floats2bfloat162_rn(v.x * inv, v.y * inv), hi = __floats2bfloat162_rn(v.z * inv, v.w * inv);
          uint2 pk;
          pk.x = *reinterpret_cast<uint32_t*>(&lo);
          pk.y = *reinterpret_cast<uint32_t*>(&hi);
          *reinterpret_cast<uint2*>(xnorm + static_cast<int64_t>(t) * d + k) = pk;
        }
      }
      arrive_event(3 * l);                                       // event N(l)
      // ---- phase A: Hd = bf16(silu(G) * U * scale)
      __nv_bfloat16* Hd = L->Hd;
      for (int tile = cta; ok && tile < Ipad / 128; tile += ctas) {
        if (!wait_acc()) { ok = false; break; }
        const uint32_t taddr = tmem_base + static_cast<uint32_t>(acc * 2 * MAXN) + (static_cast<uint32_t>(quad * 32) << 16);
        float g[MAXN], u[MAXN];
        load_acc(taddr, npad, g);
        load_acc(taddr + MAXN, npad, u);
        release_acc();
        const int64_t j = static_cast<int64_t>(tile) * 128 + quad * 32 + lane;
        const float sc = L->scale[j];
#pragma unroll
        for (int t = 0; t < MAXN; ++t) {
          if (t < n) {
            const float gv = g[t];
            Hd[static_cast<int64_t>(t) * Ipad + j] = __float2bfloat16_rn(__fdividef(gv, 1.0f + __expf(-gv)) * u[t] * sc);
          }
        }
      }
      if (!ok) break;
      arrive_event(3 * l + 1);                                   // event A(l)
      // ---- phase B: every K slice adds its part into x
      BItem it[4];
      const int nit = b_items(cta, ctas, m_blocks, Ipad / BK, it);
      for (int i = 0; ok && i < nit; ++i) {
        if (!wait_acc()) { ok = false; break; }
        const uint32_t taddr = tmem_base + static_cast<uint32_t>(acc * 2 * MAXN) + (static_cast<uint32_t>(quad * 32) << 16);
        float v[MAXN];
        load_acc(taddr, npad, v);
        release_acc();
        const int64_t m = static_cast<int64_t>(it[i].m_blk) * 128 + quad * 32 + lane;
        if (m < d) {
#pragma unroll
          for (int t = 0; t < MAXN; ++t)
            if (t < n) atomicAdd(x + static_cast<int64_t>(t) * d + m, v[t]);
        }
      }
      if (!ok) break;
      arrive_event(3 * l + 2);                                   // event B(l)
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, TMEM_COLS); }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, kStatusTimeout);
}

}  // namespace

cudaError_t decode_stack_init(int* max_ctas_per_sm) {
  cudaError_t e = cudaFuncSetAttribute(decode_stack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (e != cudaSuccess) return e;
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(max_ctas_per_sm, decode_stack_kernel, NUM_THREADS, SMEM_BYTES);
}

// layers_dev: n_layers records in device memory (64-byte aligned).  event_counter: 3 * n_layers zeros.
cudaError_t launch_decode_stack(const DecodeStackLayer* layers_dev, int n_layers, const CUtensorMap& tm_x, float* x, void* xnorm,
                                int64_t n, int64_t d, int npad, float eps, uint32_t* event_counter, uint32_t* status,
                                int num_sms, cudaStream_t st) {
  if (n == 0 || n_layers == 0) return cudaSuccess;
  __nv_bfloat16* xn = static_cast<__nv_bfloat16*>(xnorm);
  void* args[] = {const_cast<DecodeStackLayer**>(&layers_dev), &n_layers, const_cast<CUtensorMap*>(&tm_x), &x, &xn, &n, &d, &npad,
                  &eps, &event_counter, &status};
  // cooperative launch: the grid-wide events need every CTA resident at once
  return cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(decode_stack_kernel), dim3(num_sms), dim3(NUM_THREADS), args,
                                     SMEM_BYTES, st);
}

}  // namespace mlpmoe
