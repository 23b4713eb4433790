// Decode of a whole pre-norm stack for at most 16 tokens in ONE persistent, cooperatively launched
// kernel: x <- x + MLPMoE_l(RMSNorm(x)) for l = 0 .. L-1, with BOTH GEMMs of a layer on the CTA that
// owns the neurons.  Every CTA owns an equal contiguous share of each layer's compacted neurons
// (16-neuron units, decode_common.cuh), walked in items of r <= 128 neurons, and runs per item
//     A: G|U = Wg'|Wu'[item] Xn^T over K = d_model; h = bf16(silu(G) * U * scale) written straight
//        into shared memory as the token operand of phase B                        (Section 3.1)
//     B: for every block of 128 output columns, Wd'^T[block, item's r neurons] h^T, added into
//        the fp32 stream x with atomics: the branch sum of Section 3.1 is the sum over the items
// so H never goes through global memory and no CTA waits for another between A and B.  Per layer
// two grid-wide events remain (arrival counters in global memory, bounded waits): x is final once
// every CTA has added its items' parts (event B) and the normalised rows are ready once every
// token row is done (event N).  With few tokens the price, one partial sum of x per item
// (#CTAs x n x d_model fp32 atomics per layer), is small next to the weight stream.
//
// Warp roles: warp 0 TMA producer (it keeps issuing weight stages across events and only holds back
// the token tile of a phase A stage until event N has passed), warp 1 TMEM owner + MMA issuer, warps
// 2..5 epilogues and the RMSNorm phase.  Weights sit on the 128-row side of the MMA, tokens on N = 16.
// Every stage carries 256 r bytes of weights: in phase A r gate rows and r up rows x 64 K (128-byte
// swizzle), in phase B r / 16 sub-tiles of 128 output columns x 16 neurons (32-byte swizzle), so the K
// extent of phase B is exactly the item's r neurons.  The weights come from a stage-tiled copy
// (launch_retile_decode, kDecTiledFused): a CTA's stages of a layer are one contiguous run of ready-made
// shared-memory images, fetched with plain bulk copies.
#include <cuda_bf16.h>

#include "decode_common.cuh"

namespace mlpmoe {
namespace {

using namespace ptx;
using namespace dec;

constexpr int NUM_THREADS = 192;
constexpr int NPAD = 16;                              // token rows of the MMA's N side
constexpr int STAGES = 6;
constexpr int W_BYTES = 256 * BK * 2;                 // weight bytes of a full stage (r = 128)
constexpr int ACT_BYTES = NPAD * BK * 2;              // token tile of a phase A stage
constexpr int STAGE_BYTES = W_BYTES + ACT_BYTES;
constexpr int BAR_BYTES = 1024;
constexpr int HSUB_BYTES = NPAD * 32;                 // h of 16 neurons: 16 token rows of 32 bytes
constexpr int HBUF_BYTES = 8 * HSUB_BYTES;            // h of an item: up to 8 sub-tiles
constexpr int RING_OFFSET = BAR_BYTES + HBUF_BYTES;
constexpr int SMEM_BYTES = RING_OFFSET + STAGES * STAGE_BYTES + 1024;
static_assert(SMEM_BYTES <= 232448, "exceeds the 227 KB of shared memory a CTA may use");
static_assert(HBUF_BYTES % 1024 == 0 && STAGE_BYTES % 1024 == 0, "swizzled tiles start on 1024-byte boundaries");
constexpr uint32_t TMEM_COLS = 64;                    // G | U (32 columns), then 2 phase B buffers of 16
constexpr uint32_t ACC_B0 = 2 * NPAD;                 // first column of the phase B buffers

// Shared-memory operand descriptor for a K-major bf16 tile of 16 K (rows of 32 bytes) under the 32-byte
// swizzle, 8-row groups 256 bytes apart (fields as make_desc_sw128_kmajor; swizzle mode 6 = 32 B).
__device__ __forceinline__ uint64_t make_desc_sw32_kmajor(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>(256 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(6) << 61;
  return d;
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
decode_fused_kernel(const DecodeStackLayer* __restrict__ layers, int n_layers,
                    const __grid_constant__ CUtensorMap tm_x,   // xnorm [n x d] bf16, box 64 x 16
                    float* x, __nv_bfloat16* xnorm, int64_t n, int64_t d, float eps, uint32_t* event_counter,
                    uint32_t* status, uint64_t WAIT_NS, uint32_t extra_arrivals) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* tfull_a = empty_bar + STAGES;               // G|U complete
  uint64_t* h_ready = tfull_a + 1;                      // h of the item is in shared memory (4 epilogue warps)
  uint64_t* tfull_b = h_ready + 1;                      // [2] phase B buffer complete
  uint64_t* tempty_b = tfull_b + 2;                     // [2] phase B buffer read (4 epilogue warps)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_b + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  const ClockProbe probe = clock_probe_begin();
  volatile float* norm_part = reinterpret_cast<volatile float*>(tmem_slot + 4);   // one partial sum of squares per epilogue warp
  uint8_t* hbuf = smem + BAR_BYTES;
  uint8_t* ring = smem + RING_OFFSET;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int cta = blockIdx.x, ctas = gridDim.x;
  const uint32_t per_event = static_cast<uint32_t>(ctas) * ARRIVALS_PER_CTA + extra_arrivals;   // extra: 0 outside tests
  const int n_mb = static_cast<int>((d + 127) / 128);         // phase B: blocks of 128 output columns
  const int kb1 = static_cast<int>((d + BK - 1) / BK);

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(tfull_a, 1);
    mbar_init(h_ready, 4);
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull_b[a], 1); mbar_init(&tempty_b[a], 4); }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) { tmem_alloc(tmem_slot, TMEM_COLS); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tensormap(&tm_x);
      int stage = 0; uint32_t phase = 0;
      // token tiles of phase A stages that wait for event N of their layer: (stage, K-step), oldest first
      int def_head = 0, deferred = 0, def_stage[STAGES], def_kb[STAGES], def_layer[STAGES];
      int open_layer = -1;                 // event N of this layer (and of every earlier one) has been seen
      auto gate_is_open = [&](int l) -> bool {
        if (l <= open_layer) return true;
        if (!event_passed(event_counter + 2 * l, per_event)) return false;
        open_layer = l;
        fence_async_proxy();               // what the acquire made visible must be seen by the TMA reads
        return true;
      };
      auto drain = [&](bool block) -> bool {
        while (deferred > 0) {
          const int h = def_head;
          if (!gate_is_open(def_layer[h])) {
            if (!block) return true;
            if (!event_wait(event_counter + 2 * def_layer[h], per_event, abort_flag, WAIT_NS)) return false;
            block = false;
            continue;
          }
          tma_load_2d(ring + def_stage[h] * STAGE_BYTES + W_BYTES, &tm_x, def_kb[h] * BK, 0, &full_bar[def_stage[h]]);
          def_head = def_head + 1 == STAGES ? 0 : def_head + 1;
          --deferred;
        }
        return true;
      };
      bool ok = true;
      for (int l = 0; ok && l < n_layers; ++l) {
        const DecodeStackLayer* L = layers + l;
        const Items items(L, cta);
        const uint8_t* src = L->tiled + L->a_off[cta];            // the CTA's stages of this layer, one contiguous run
        for (int item = 0; ok && item < items.count(); ++item) {
          const uint32_t wb = static_cast<uint32_t>(items.rows(item)) * 256u;   // weight bytes of every stage of the item
          // phase A: r gate rows | r up rows x 64 K, and the token tile
          for (int kb = 0; ok && kb < kb1; ++kb) {
            // (blocking when the slot to refill still waits for its own token tile)
            if (deferred > 0 && !drain(def_stage[def_head] == stage)) { ok = false; break; }
            if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, WAIT_NS)) { ok = false; break; }
            uint8_t* s = ring + stage * STAGE_BYTES;
            mbar_expect_tx(&full_bar[stage], wb + ACT_BYTES);
            bulk_load_1d(s, src, wb, &full_bar[stage]);
            src += wb;
            if (deferred == 0 && gate_is_open(l)) {
              tma_load_2d(s + W_BYTES, &tm_x, kb * BK, 0, &full_bar[stage]);
            } else {
              int t = def_head + deferred;
              if (t >= STAGES) t -= STAGES;
              def_stage[t] = stage; def_kb[t] = kb; def_layer[t] = l;
              ++deferred;
            }
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
          }
          // phase B: 128 output columns x the item's neurons; the token operand is in shared memory
          for (int mb = 0; ok && mb < n_mb; ++mb) {
            if (deferred > 0 && !drain(def_stage[def_head] == stage)) { ok = false; break; }
            if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, WAIT_NS)) { ok = false; break; }
            mbar_expect_tx(&full_bar[stage], wb);
            bulk_load_1d(ring + stage * STAGE_BYTES, src, wb, &full_bar[stage]);
            src += wb;
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
          }
        }
      }
      while (ok && deferred > 0) ok = drain(true);
    }
  }
  else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = make_idesc_bf16_f32(128, NPAD);
      int stage = 0, buf = 0; uint32_t phase = 0, buf_phase = 0, h_phase = 0; bool ok = true;
      for (int l = 0; ok && l < n_layers; ++l) {
        const Items items(layers + l, cta);
        for (int item = 0; ok && item < items.count(); ++item) {
          const int r = items.rows(item);
          // phase A.  G|U may be overwritten: the epilogue read them before it signalled h_ready, which
          // the phase B MMAs issued before these waited for.
          for (int kb = 0; kb < kb1; ++kb) {
            if (!mbar_wait_bounded(&full_bar[stage], phase, abort_flag, WAIT_NS)) { ok = false; break; }
            tc_fence_after();
            const uint32_t s = smem_u32(ring + stage * STAGE_BYTES);
            const uint64_t w0 = make_desc_sw128_kmajor(s), w1 = make_desc_sw128_kmajor(s + static_cast<uint32_t>(r) * BK * 2);
            const uint64_t xd = make_desc_sw128_kmajor(s + W_BYTES);
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) {
              const uint32_t accum = (kb | k) != 0 ? 1u : 0u;
              umma_bf16(tmem_base, w0 + 2 * k, xd + 2 * k, idesc, accum);
              umma_bf16(tmem_base + NPAD, w1 + 2 * k, xd + 2 * k, idesc, accum);
            }
            umma_commit(&empty_bar[stage]);
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          umma_commit(tfull_a);
          // phase B
          if (!mbar_wait_bounded(h_ready, h_phase, abort_flag, WAIT_NS)) { ok = false; break; }
          h_phase ^= 1u;
          tc_fence_after();
          for (int mb = 0; ok && mb < n_mb; ++mb) {
            if (!mbar_wait_bounded(&tempty_b[buf], buf_phase ^ 1u, abort_flag, WAIT_NS)) { ok = false; break; }
            if (!mbar_wait_bounded(&full_bar[stage], phase, abort_flag, WAIT_NS)) { ok = false; break; }
            tc_fence_after();
            const uint32_t acc = tmem_base + ACC_B0 + static_cast<uint32_t>(buf * NPAD);
            const uint32_t s = smem_u32(ring + stage * STAGE_BYTES), hs = smem_u32(hbuf);
            for (int k16 = 0; k16 < r / 16; ++k16)
              umma_bf16(acc, make_desc_sw32_kmajor(s + static_cast<uint32_t>(k16) * 4096u),
                        make_desc_sw32_kmajor(hs + static_cast<uint32_t>(k16 * HSUB_BYTES)), idesc, k16 != 0 ? 1u : 0u);
            umma_commit(&empty_bar[stage]);
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            umma_commit(&tfull_b[buf]);
            buf ^= 1;
            if (buf == 0) buf_phase ^= 1u;
          }
        }
      }
    }
  }
  else {
    // ------------------------------------------- epilogue warps (+ RMSNorm phase)
    const int quad = warp % 4;
    int buf = 0; uint32_t buf_phase = 0, a_phase = 0;
    bool ok = true;
    auto arrive_event = [&](int e) {       // this warp's part of the phase is written and visible
      __threadfence();
      __syncwarp();
      if (lane == 0) atomicAdd(event_counter + e, 1u);
    };
    // Once a wait has given up (ok == false) a warp skips all further work but still walks every
    // loop, so that the four warps keep meeting at the named barrier of the RMSNorm phase.
    for (int l = 0; l < n_layers; ++l) {
      const DecodeStackLayer* L = layers + l;
      // ---- phase N: x is final once every CTA has added the parts of its items of the previous layer
      if (ok && l > 0) {
        bool w = event_wait(event_counter + 2 * l - 1, per_event, abort_flag, WAIT_NS);
        ok = __all_sync(0xFFFFFFFFu, w);
      }
      for (int t = cta; t < n; t += ctas) norm_row(x, xnorm, t, d, eps, quad, lane, norm_part, ok);
      if (ok) arrive_event(2 * l);                               // event N(l)
      const Items items(L, cta);
      for (int item = 0; item < items.count(); ++item) {
        // ---- phase A epilogue: h = bf16(silu(G) * U * scale), this thread's neuron for all 16 token rows
        if (ok && !mbar_wait_bounded(tfull_a, a_phase, abort_flag, WAIT_NS)) ok = false;
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) continue;
        a_phase ^= 1u;
        tc_fence_after();
        const uint32_t lane_base = static_cast<uint32_t>(quad * 32) << 16;
        uint32_t g[NPAD], u[NPAD];
        tmem_ld_32x16(tmem_base + lane_base, g);
        tmem_ld_32x16(tmem_base + lane_base + NPAD, u);
        const int j = quad * 32 + lane;                          // neuron within the item
        const bool mine = j < items.rows(item);                  // accumulator lanes past the item's rows hold nothing
        const float sc = mine ? L->scale[static_cast<int64_t>(items.unit0(item)) * kDecUnit + j] : 0.f;
        tmem_ld_wait();
        // K-major token operand in sub-tiles of 16 neurons under the 32-byte swizzle: token row t is 32 bytes,
        // its 16-byte piece c (8 neurons) sits at piece position c ^ ((t / 4) % 2)
        if (mine) {
          uint8_t* hk = hbuf + (j / 16) * HSUB_BYTES;
          const int piece = (j % 16) / 8, within = (j % 8) * 2;
#pragma unroll
          for (int t = 0; t < NPAD; ++t) {
            const float gv = __uint_as_float(g[t]);
            const __nv_bfloat16 hv = __float2bfloat16_rn(__fdividef(gv, 1.0f + __expf(-gv)) * __uint_as_float(u[t]) * sc);
            *reinterpret_cast<__nv_bfloat16*>(hk + t * 32 + ((piece ^ ((t >> 2) & 1)) << 4) + within) = hv;
          }
        }
        fence_proxy_async_smem();            // the MMAs read h through the async proxy
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(h_ready);
        // ---- phase B epilogues: every block of 128 output columns adds its part into x
        for (int mb = 0; mb < n_mb; ++mb) {
          if (ok && !mbar_wait_bounded(&tfull_b[buf], buf_phase, abort_flag, WAIT_NS)) ok = false;
          ok = __all_sync(0xFFFFFFFFu, ok);
          if (!ok) break;
          tc_fence_after();
          uint32_t v[NPAD];
          tmem_ld_32x16(tmem_base + ACC_B0 + static_cast<uint32_t>(buf * NPAD) + lane_base, v);
          tmem_ld_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tempty_b[buf]);
          buf ^= 1;
          if (buf == 0) buf_phase ^= 1u;
          const int64_t m0 = static_cast<int64_t>(mb) * 128 + quad * 32 + lane;
          if (m0 < d) {
#pragma unroll
            for (int t = 0; t < NPAD; ++t)
              if (t < n) atomicAdd(x + static_cast<int64_t>(t) * d + m0, __uint_as_float(v[t]));
          }
        }
      }
      if (ok) arrive_event(2 * l + 1);                           // event B(l)
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, TMEM_COLS); }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, kStatusTimeout);
  if (blockIdx.x == 0 && threadIdx.x == 0) clock_probe_end(status, probe);
}

}  // namespace

cudaError_t decode_fused_init(int* max_ctas_per_sm) {
  cudaError_t e = cudaFuncSetAttribute(decode_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (e != cudaSuccess) return e;
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(max_ctas_per_sm, decode_fused_kernel, NUM_THREADS, SMEM_BYTES);
}

// layers_dev: n_layers records in device memory (`tiled` in the kDecTiledFused layout; tm_hd and Hd unused).
// event_counter: 2 * n_layers zeros.  n <= 16 (the caller uses it up to kDecodeFusedMaxTokens).
cudaError_t launch_decode_fused(const DecodeStackLayer* layers_dev, int n_layers, const CUtensorMap& tm_x, float* x, void* xnorm,
                                int64_t n, int64_t d, float eps, uint32_t* event_counter, uint32_t* status, int num_sms,
                                const WaitCfg& wait, cudaStream_t st) {
  if (n == 0 || n_layers == 0) return cudaSuccess;
  __nv_bfloat16* xn = static_cast<__nv_bfloat16*>(xnorm);
  uint64_t wait_ns = wait.limit_ns;
  uint32_t extra = wait.extra_arrivals;
  void* args[] = {const_cast<DecodeStackLayer**>(&layers_dev), &n_layers, const_cast<CUtensorMap*>(&tm_x), &x, &xn, &n, &d,
                  &eps, &event_counter, &status, &wait_ns, &extra};
  // cooperative launch: the grid-wide events need every CTA resident at once
  return cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(decode_fused_kernel), dim3(num_sms), dim3(NUM_THREADS), args,
                                     SMEM_BYTES, st);
}

}  // namespace mlpmoe
