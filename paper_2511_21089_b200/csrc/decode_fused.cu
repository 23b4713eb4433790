// Decode of a whole pre-norm stack for at most 16 tokens in ONE persistent, cooperatively launched
// kernel: x <- x + MLPMoE_l(RMSNorm(x)) for l = 0 .. L-1, with BOTH GEMMs of a layer on the CTA that
// owns the neurons.  CTA c owns the 128 compacted neurons of gate|up tile c (c + #CTAs, ...) and
// runs, per layer and tile,
//     A: G|U = Wg'|Wu'[tile] Xn^T over K = d_model; h = bf16(silu(G) * U * scale) written straight
//        into shared memory as the token operand of phase B                        (Section 3.1)
//     B: for every block of 256 output columns, Wd'^T[block, tile's 128 neurons] h^T, added into
//        the fp32 stream x with atomics: the branch sum of Section 3.1 is the sum over the tiles
// so H never goes through global memory and no CTA waits for another between A and B.  Per layer
// two grid-wide events remain (arrival counters in global memory, bounded waits): x is final once
// every CTA has added its tiles' parts (event B) and the normalised rows are ready once every
// token row is done (event N).  With few tokens the price, one partial sum of x per tile
// (Ipad / 128 x n x d_model fp32 atomics per layer), is small next to the weight stream.
//
// The CTAs beyond the number of tiles (36 of 148 at the Llama-8B shape) own no neurons; at every
// layer boundary they request the next layer's first stages into L2 while HBM would idle (+2 to 3.5 %).
//
// Warp roles as in decode_stack.cu: warp 0 TMA producer (it keeps issuing weight tiles across
// events and only holds back the token tile of a phase A stage until event N has passed), warp 1
// TMEM owner + MMA issuer, warps 2..5 epilogues and the RMSNorm phase.  Weights sit on the 128-row
// side of the MMA, tokens on N = 16.  Every stage carries 256 weight rows x 64 K = 32 KB, and the
// weights come from a stage-tiled copy (launch_retile_decode): a CTA's stages of a layer are one
// contiguous 3 MB run of ready-made shared-memory images, fetched with plain bulk copies, which HBM
// serves about 5 % faster than 256 row pieces of 128 bytes.
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace mlpmoe {
namespace {

using namespace ptx;

constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int NUM_THREADS = 192;
constexpr int NPAD = 16;                              // token rows of the MMA's N side
constexpr int STAGES = 6;
constexpr int W_BYTES = 256 * BK * 2;                 // 256 weight rows per stage in both phases
constexpr int ACT_BYTES = NPAD * BK * 2;              // token tile of a phase A stage
constexpr int STAGE_BYTES = W_BYTES + ACT_BYTES;
constexpr int BAR_BYTES = 1024;
constexpr int HBUF_BYTES = 2 * ACT_BYTES;             // h of the tile: two K-steps of 16 tokens x 64 neurons
constexpr int RING_OFFSET = BAR_BYTES + HBUF_BYTES;
constexpr int SMEM_BYTES = RING_OFFSET + STAGES * STAGE_BYTES + 1024;
static_assert(SMEM_BYTES <= 232448, "exceeds the 227 KB of shared memory a CTA may use");
static_assert(HBUF_BYTES % 1024 == 0 && STAGE_BYTES % 1024 == 0, "swizzled tiles start on 1024-byte boundaries");
constexpr uint32_t TMEM_COLS = 128;                   // G | U (32 columns), then 2 buffers x 2 halves x 16 for phase B
constexpr uint32_t ACC_B0 = 2 * NPAD;                 // first column of the phase B buffers
constexpr uint32_t ARRIVALS_PER_CTA = 1;              // one arrival per CTA and event, after its four epilogue warps have met
constexpr int HELPER_STAGES = 32;                     // stages per tile that a CTA without tiles requests into L2 at a layer boundary
constexpr int NORM_VEC = 8;                           // float4 per lane the RMSNorm phase keeps in registers

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async;" ::: "memory"); }
// The four epilogue warps (threads 64..191) only.
__device__ __forceinline__ void epilogue_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Events are numbered in program order, 2 per layer (N at 2l, B at 2l + 1), each with its own
// arrival counter; event e has happened once counter[e] has reached arrivals_per_event.
__device__ __forceinline__ bool event_passed(const uint32_t* counter, uint32_t target) {
  return ld_acquire_u32(counter) >= target;
}
__device__ __forceinline__ bool event_wait(const uint32_t* counter, uint32_t target, volatile uint32_t* abort_flag,
                                           uint64_t WAIT_NS) {
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
  uint64_t* h_ready = tfull_a + 1;                      // h of the tile is in shared memory (4 epilogue warps)
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
  const int m_blocks = static_cast<int>((d + 255) / 256);     // phase B: blocks of 256 output columns
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
      // A CTA without a tile in any layer helps the others over the layer boundaries: when three
      // quarters of the owners have finished layer l (HBM starts to idle while x is completed and
      // normalised), it asks for the stages of layer l + 1 that lie just beyond the owners' rings to be
      // brought into L2, from where the owners then refill their rings faster than HBM would serve
      // them.  Only where the owners are many enough to be bound by HBM (at least 70 % of the CTAs):
      // with fewer owners each is bound by what one SM can take in, and the requests measured slower.
      int max_tiles = 0;
      for (int l = 0; l < n_layers; ++l) max_tiles = layers[l].Ipad / 128 > max_tiles ? layers[l].Ipad / 128 : max_tiles;
      if (cta >= max_tiles) {                              // no tile in any layer: this producer has nothing else to do
        const int helpers = ctas - max_tiles, me = cta - max_tiles;
        const int cpt = kb1 + 2 * m_blocks;
        for (int l = 0; ok && l + 1 < n_layers; ++l) {
          const DecodeStackLayer* Ln = layers + l + 1;
          const int tiles_next = Ln->Ipad / 128, tiles_this = layers[l].Ipad / 128;
          // (the CTAs without a tile in layer l arrive at its event B at once)
          if (10 * tiles_next < 7 * ctas) continue;
          const uint32_t idle_arrivals = static_cast<uint32_t>(ctas - tiles_this) * ARRIVALS_PER_CTA;
          const uint32_t owners_done = static_cast<uint32_t>(tiles_this) * 3u / 4u + 1u;
          if (!event_wait(event_counter + 2 * l + 1, idle_arrivals + owners_done * ARRIVALS_PER_CTA, abort_flag, WAIT_NS)) { ok = false; break; }
          for (int tile = me; tile < tiles_next; tile += helpers)
            for (int s = STAGES; s < STAGES + HELPER_STAGES && s < kb1; ++s)
              bulk_prefetch_l2(Ln->tiled + (static_cast<int64_t>(tile) * cpt + s) * W_BYTES, W_BYTES);
        }
      }
      for (int l = 0; ok && l < n_layers; ++l) {
        const DecodeStackLayer* L = layers + l;
        const uint8_t* tiled = L->tiled;
        const int chunks_per_tile = kb1 + 2 * m_blocks;
        for (int tile = cta; ok && tile < L->Ipad / 128; tile += ctas) {
          // phase A: 256 rows of Wgu (128 gate | 128 up) x 64 K, and the token tile
          for (int kb = 0; ok && kb < kb1; ++kb) {
            // (blocking when the slot to refill still waits for its own token tile)
            if (deferred > 0 && !drain(def_stage[def_head] == stage)) { ok = false; break; }
            if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, WAIT_NS)) { ok = false; break; }
            uint8_t* s = ring + stage * STAGE_BYTES;
            mbar_expect_tx(&full_bar[stage], W_BYTES + ACT_BYTES);
            bulk_load_1d(s, tiled + (static_cast<int64_t>(tile) * chunks_per_tile + kb) * W_BYTES, W_BYTES, &full_bar[stage]);
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
          // phase B: 256 rows of WdT x the tile's 128 neurons, 64 at a time; the token operand is in shared memory
          for (int blk = 0; ok && blk < m_blocks; ++blk)
            for (int ks = 0; ks < 2; ++ks) {
              if (deferred > 0 && !drain(def_stage[def_head] == stage)) { ok = false; break; }
              if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, WAIT_NS)) { ok = false; break; }
              mbar_expect_tx(&full_bar[stage], W_BYTES);
              bulk_load_1d(ring + stage * STAGE_BYTES, tiled + (static_cast<int64_t>(tile) * chunks_per_tile + kb1 + blk * 2 + ks) * W_BYTES,
                           W_BYTES, &full_bar[stage]);
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
      const uint64_t h0 = make_desc_sw128_kmajor(smem_u32(hbuf)), h1 = make_desc_sw128_kmajor(smem_u32(hbuf + ACT_BYTES));
      int stage = 0, buf = 0; uint32_t phase = 0, buf_phase = 0, h_phase = 0; bool ok = true;
      for (int l = 0; ok && l < n_layers; ++l) {
        const int Ipad = layers[l].Ipad;
        for (int tile = cta; ok && tile < Ipad / 128; tile += ctas) {
          // phase A.  G|U may be overwritten: the epilogue read them before it signalled h_ready, which
          // the phase B MMAs issued before these waited for.
          for (int kb = 0; kb < kb1; ++kb) {
            if (!mbar_wait_bounded(&full_bar[stage], phase, abort_flag, WAIT_NS)) { ok = false; break; }
            tc_fence_after();
            const uint32_t s = smem_u32(ring + stage * STAGE_BYTES);
            const uint64_t w0 = make_desc_sw128_kmajor(s), w1 = make_desc_sw128_kmajor(s + 128 * BK * 2);
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
          for (int blk = 0; ok && blk < m_blocks; ++blk) {
            if (!mbar_wait_bounded(&tempty_b[buf], buf_phase ^ 1u, abort_flag, WAIT_NS)) { ok = false; break; }
            tc_fence_after();
            const uint32_t acc = tmem_base + ACC_B0 + static_cast<uint32_t>(buf * 2 * NPAD);
            for (int ks = 0; ks < 2; ++ks) {
              if (!mbar_wait_bounded(&full_bar[stage], phase, abort_flag, WAIT_NS)) { ok = false; break; }
              tc_fence_after();
              const uint32_t s = smem_u32(ring + stage * STAGE_BYTES);
              const uint64_t w0 = make_desc_sw128_kmajor(s), w1 = make_desc_sw128_kmajor(s + 128 * BK * 2);
              const uint64_t hd = ks == 0 ? h0 : h1;
#pragma unroll
              for (int k = 0; k < BK / UMMA_K; ++k) {
                const uint32_t accum = (ks | k) != 0 ? 1u : 0u;
                umma_bf16(acc, w0 + 2 * k, hd + 2 * k, idesc, accum);
                umma_bf16(acc + NPAD, w1 + 2 * k, hd + 2 * k, idesc, accum);
              }
              umma_commit(&empty_bar[stage]);
              if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
            if (!ok) break;
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
    // One arrival per CTA (592 arrivals on one counter took longer than the meeting of four warps): every
    // thread makes its writes visible, the four warps meet, one thread arrives.  Called by all four warps
    // also after a wait has given up, so that the named barrier stays balanced.
    auto arrive_event = [&](int e) {
      if (ok) __threadfence();
      epilogue_bar_sync();
      if (ok && quad == 0 && lane == 0) atomicAdd(event_counter + e, 1u);
    };
    // Once a wait has given up (ok == false) a warp skips all further work but still walks every
    // loop, so that the four warps keep meeting at the named barrier of the RMSNorm phase.
    for (int l = 0; l < n_layers; ++l) {
      const DecodeStackLayer* L = layers + l;
      const int Ipad = L->Ipad;
      // ---- phase N: x is final once every CTA has added the parts of its tiles of the previous layer
      if (ok && l > 0) {
        bool w = event_wait(event_counter + 2 * l - 1, per_event, abort_flag, WAIT_NS);
        ok = __all_sync(0xFFFFFFFFu, w);
      }
      for (int t = cta; t < n; t += ctas) {
        // each warp takes a quarter of the row, keeps it in registers, and the four partial sums of
        // squares meet in shared memory
        const float* row = x + static_cast<int64_t>(t) * d;
        const int64_t q = (d / 4 + 3) / 4 * 4;                 // columns per warp, a multiple of 4
        const int64_t c0 = static_cast<int64_t>(quad) * q, c1 = c0 + q < d ? c0 + q : d;
        float4 v[NORM_VEC];
        float ss = 0.f;
        if (ok) {
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
        if (ok) {
          const float inv = 1.0f / sqrtf(total / static_cast<float>(d) + eps);
          __nv_bfloat16* out = xnorm + static_cast<int64_t>(t) * d;
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
      arrive_event(2 * l);                               // event N(l)
      for (int tile = cta; tile < Ipad / 128; tile += ctas) {
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
        const int j = quad * 32 + lane;                          // neuron within the tile
        const float sc = L->scale[static_cast<int64_t>(tile) * 128 + j];
        tmem_ld_wait();
        // K-major token operand under the 128-byte swizzle: token row t is 128 bytes (64 neurons), its
        // 16-byte chunk c sits at chunk position c ^ (t % 8); neurons 64..127 form the second K-step
        uint8_t* hk = hbuf + (j / 64) * ACT_BYTES;
        const int chunk = (j % 64) / 8, within = (j % 8) * 2;
#pragma unroll
        for (int t = 0; t < NPAD; ++t) {
          const float gv = __uint_as_float(g[t]);
          const __nv_bfloat16 hv = __float2bfloat16_rn(__fdividef(gv, 1.0f + __expf(-gv)) * __uint_as_float(u[t]) * sc);
          *reinterpret_cast<__nv_bfloat16*>(hk + t * 128 + ((chunk ^ (t & 7)) << 4) + within) = hv;
        }
        fence_proxy_async_smem();            // the MMAs read h through the async proxy
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(h_ready);
        // ---- phase B epilogues: every block of 256 output columns adds its part into x
        for (int blk = 0; blk < m_blocks; ++blk) {
          if (ok && !mbar_wait_bounded(&tfull_b[buf], buf_phase, abort_flag, WAIT_NS)) ok = false;
          ok = __all_sync(0xFFFFFFFFu, ok);
          if (!ok) break;
          tc_fence_after();
          const uint32_t acc = tmem_base + ACC_B0 + static_cast<uint32_t>(buf * 2 * NPAD) + lane_base;
          uint32_t lo[NPAD], hi[NPAD];
          tmem_ld_32x16(acc, lo);
          tmem_ld_32x16(acc + NPAD, hi);
          tmem_ld_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tempty_b[buf]);
          buf ^= 1;
          if (buf == 0) buf_phase ^= 1u;
          const int64_t m0 = static_cast<int64_t>(blk) * 256 + quad * 32 + lane;
#pragma unroll
          for (int t = 0; t < NPAD; ++t) {
            if (t < n) {
              if (m0 < d) atomicAdd(x + static_cast<int64_t>(t) * d + m0, __uint_as_float(lo[t]));
              if (m0 + 128 < d) atomicAdd(x + static_cast<int64_t>(t) * d + m0 + 128, __uint_as_float(hi[t]));
            }
          }
        }
      }
      arrive_event(2 * l + 1);                           // event B(l)
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

// layers_dev: n_layers records in device memory (`tiled` set; tm_wgu, tm_wdt, tm_hd and Hd unused).  event_counter: 2 * n_layers zeros.  n <= 16
// (the caller uses it up to kDecodeFusedMaxTokens).
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
