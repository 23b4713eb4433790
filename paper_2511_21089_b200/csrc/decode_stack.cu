// Decode of a whole pre-norm stack (n_tokens <= 128) in ONE persistent, cooperatively launched
// kernel: x <- x + MLPMoE_l(RMSNorm(x)) for l = 0 .. L-1.  One CTA per SM; every CTA walks the same
// static sequence of phases per layer
//     N: RMSNorm of the token rows into the bf16 activation buffer
//     A: gate|up, H = bf16(silu(G) * U * scale), 128 neurons per work item      (Section 3.1)
//     B: down + branch sum, 256 output columns per work item, K slices added straight into the
//        fp32 stream x
// separated by grid-wide events (one global arrival counter, bounded waits).  The producer warp
// never stops at an event with an empty ring: weight tiles depend on no earlier phase, so it keeps
// issuing them and only holds back the small activation tile of each stage until the event it
// needs has passed.  HBM therefore keeps streaming weights across phase and layer boundaries.
// Both phases use the same stage: 256 weight rows x 64 K (two accumulators of 128 rows: gate and
// up of the same neurons in phase A, two neighbouring blocks of output columns in phase B) next to
// one token tile, so every stage carries 32 KB of weights.  Where the layers have a stage-tiled
// copy (launch_retile_decode) the weights of a stage are one contiguous, ready-made shared-memory
// image fetched by a plain bulk copy (2 to 4 % faster than the 256 row pieces of a tensor tile);
// otherwise they come from the packed operands through tensor maps.
//
// Warp roles: warp 0 TMA producer, warp 1 TMEM owner + MMA issuer, warps 2..5 epilogue (and the
// RMSNorm phase).  Weights sit on the 128-row side of the MMA, tokens on N = 16 / 32 / 64 / 128.
// The kernel is built twice: for at most 64 token rows (two accumulator buffers in 256 TMEM columns)
// and for 128 (all 512 columns).
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace mlpmoe {
namespace {

using namespace ptx;

constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int NUM_THREADS = 192;
constexpr int MAX_STAGES = 6;
constexpr int W_BYTES = 256 * BK * 2;                 // 256 weight rows per stage in both phases
// A stage is the weight tile plus a token tile of npad rows; the ring takes as many stages as fit
// (6 for npad 16 and 32, 5 for npad 64, 4 for npad 128), the barriers sit in front of it.
constexpr int BAR_BYTES = 1024;
constexpr int RING_BYTES = 216 * 1024;
constexpr int SMEM_BYTES = BAR_BYTES + RING_BYTES + 1024;
static_assert(SMEM_BYTES <= 232448, "exceeds the 227 KB of shared memory a CTA may use");
__host__ __device__ constexpr int stage_bytes_for(int npad) { return W_BYTES + npad * BK * 2; }
__host__ __device__ constexpr int stages_for(int npad) {
  return RING_BYTES / stage_bytes_for(npad) < MAX_STAGES ? RING_BYTES / stage_bytes_for(npad) : MAX_STAGES;
}
constexpr uint32_t ARRIVALS_PER_CTA = 1;              // one arrival per CTA and event, after its four epilogue warps have met
constexpr int NORM_VEC = 8;                           // float4 per lane the RMSNorm phase keeps in registers

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async;" ::: "memory"); }
// The four epilogue warps (threads 64..191) only.
__device__ __forceinline__ void epilogue_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Events are numbered in program order, 3 per layer (N, A, B), and each has its own arrival counter
// (a CTA without work in a phase arrives at once, so one shared counter would let early arrivals
// at later events stand in for missing arrivals at earlier ones).  Event e has happened once
// counter[e] has reached arrivals_per_event.
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

// Issues the loads of one accumulator's first npad columns; the values are valid after tmem_ld_wait().
template <int MAXN>
__device__ __forceinline__ void load_acc_async(uint32_t taddr, int npad, uint32_t (&v)[MAXN]) {
#pragma unroll
  for (int c = 0; c < MAXN; c += 16) {
    if (c < npad) {
      uint32_t(&r)[16] = *reinterpret_cast<uint32_t(*)[16]>(&v[c]);
      tmem_ld_32x16(taddr + c, r);
    }
  }
}

// A CTA's share of phase B of one layer: units (256-row block of WdT, K-step) in block-major order,
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

// One CTA's weight K-steps of the whole stack in program order: per layer first phase A (its
// gate|up tiles, all K-steps of each), then phase B (its items).  The producer walks the
// sequence.
struct StepIter {
  const DecodeStackLayer* layers;
  int n_layers, cta, ctas, m_blocks, kb1;
  int l, ph, idx, kb, nit;       // ph 0: idx = gate|up tile; ph 1: idx = item number
  BItem it[4];
  bool done;
  __device__ __forceinline__ void settle() {      // moves to the first phase at or after (l, ph) that has work
    while (!done) {
      const int Ipad = layers[l].Ipad;
      if (ph == 0) {
        idx = cta;
        kb = 0;
        if (idx < Ipad / 128) return;
        ph = 1;
      }
      nit = b_items(cta, ctas, m_blocks, Ipad / BK, it);
      idx = 0;
      if (nit > 0) { kb = it[0].kb_lo; return; }
      ph = 0;
      if (++l == n_layers) done = true;
    }
  }
  __device__ __forceinline__ void init(const DecodeStackLayer* layers_, int n_layers_, int cta_, int ctas_, int m_blocks_, int kb1_) {
    layers = layers_; n_layers = n_layers_; cta = cta_; ctas = ctas_; m_blocks = m_blocks_; kb1 = kb1_;
    l = 0; ph = 0; idx = 0; kb = 0; nit = 0;
    done = n_layers == 0;
    settle();
  }
  __device__ __forceinline__ const CUtensorMap* wmap() const { return ph == 0 ? &layers[l].tm_wgu : &layers[l].tm_wdt; }
  __device__ __forceinline__ int wrow() const { return (ph == 0 ? idx : it[idx].m_blk) * 256; }
  __device__ __forceinline__ int event() const { return 3 * l + ph; }     // the event its activation tile waits for
  // The same 256 x 64 weight tile in the stage-tiled copy (see launch_retile_decode): chunk kb of gate|up
  // tile idx, or, for phase B, the chunk of output block m_blk and K-step kb = 2 * (gate|up tile) + half.
  __device__ __forceinline__ const uint8_t* wtiled() const {
    const int64_t cpt = kb1 + 2 * m_blocks;
    const int64_t chunk = ph == 0 ? static_cast<int64_t>(idx) * cpt + kb
                                  : static_cast<int64_t>(kb / 2) * cpt + kb1 + it[idx].m_blk * 2 + kb % 2;
    return layers[l].tiled + chunk * W_BYTES;
  }
  __device__ __forceinline__ void advance() {
    ++kb;
    if (ph == 0) {
      if (kb < kb1) return;
      idx += ctas;
      kb = 0;
      if (idx < layers[l].Ipad / 128) return;
      ph = 1;
      settle();
    } else {
      if (kb < it[idx].kb_hi) return;
      if (++idx < nit) { kb = it[idx].kb_lo; return; }
      ph = 0;
      if (++l == n_layers) { done = true; return; }
      settle();
    }
  }
};

template <int MAXN>                                   // token rows the accumulators hold: 64 or 128
__global__ void __launch_bounds__(NUM_THREADS, 1)
decode_stack_kernel(const DecodeStackLayer* __restrict__ layers, int n_layers,
                    const __grid_constant__ CUtensorMap tm_x,   // xnorm [n x d] bf16, box 64 x npad
                    float* x, __nv_bfloat16* xnorm, int64_t n, int64_t d, int npad, float eps, uint32_t* event_counter,
                    uint32_t* status, uint64_t WAIT_NS, uint32_t extra_arrivals) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem);
  uint64_t* empty_bar = full_bar + MAX_STAGES;
  uint64_t* tfull_bar = empty_bar + MAX_STAGES;
  uint64_t* tempty_bar = tfull_bar + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  const ClockProbe probe = clock_probe_begin();
  constexpr uint32_t TMEM_COLS = 4 * MAXN;              // 2 buffers x (G | U)
  volatile float* norm_part = reinterpret_cast<volatile float*>(tmem_slot + 4);   // one partial sum of squares per epilogue warp
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int cta = blockIdx.x, ctas = gridDim.x;
  const uint32_t per_event = static_cast<uint32_t>(ctas) * ARRIVALS_PER_CTA + extra_arrivals;   // extra: 0 outside tests
  const int m_blocks = static_cast<int>((d + 255) / 256);     // phase B: blocks of 256 output columns
  const int kb1 = static_cast<int>((d + BK - 1) / BK);

  if (threadIdx.x == 0) {
    for (int s = 0; s < MAX_STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
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
  uint8_t* ring = smem + BAR_BYTES;
  const int STAGES = stages_for(npad), STAGE_BYTES = stage_bytes_for(npad);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tensormap(&tm_x);
      int stage = 0; uint32_t phase = 0;
      // activation tiles that wait for the current gating event: (stage, K-step) of map def_map
      int deferred = 0, def_stage[MAX_STAGES], def_kb[MAX_STAGES];
      const CUtensorMap* def_map = &tm_x;
      int gate_ev = 0;                     // index of the gating event
      bool gate_open = false;
      auto flush = [&]() {
        fence_async_proxy();               // what the acquire made visible must be seen by the TMA reads
        for (int i = 0; i < deferred; ++i)
          tma_load_2d(ring + def_stage[i] * STAGE_BYTES + W_BYTES, def_map, def_kb[i] * BK, 0, &full_bar[def_stage[i]]);
        deferred = 0;
        gate_open = true;
      };
      StepIter cur;
      cur.init(layers, n_layers, cta, ctas, m_blocks, kb1);
      bool ok = true;
      while (ok && !cur.done) {
        const int ev = cur.event();
        if (ev != gate_ev) {
          // a new phase: the deferred tiles of the previous one go first (events pass in order)
          if (deferred > 0) {
            if (!event_wait(event_counter + gate_ev, per_event, abort_flag, WAIT_NS)) { ok = false; break; }
            flush();
          }
          gate_ev = ev;
          gate_open = false;
          def_map = cur.ph == 0 ? &tm_x : &layers[cur.l].tm_hd;
        }
        if (!gate_open && (deferred == STAGES || event_passed(event_counter + gate_ev, per_event))) {
          if (deferred == STAGES && !event_wait(event_counter + gate_ev, per_event, abort_flag, WAIT_NS)) { ok = false; break; }
          flush();
        }
        if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, WAIT_NS)) { ok = false; break; }
        uint8_t* s = ring + stage * STAGE_BYTES;
        mbar_expect_tx(&full_bar[stage], W_BYTES + act_bytes);
        const int kc = cur.kb;     // every CTA walks K in the same order: staggered starts measured 3 % slower
        if (layers[cur.l].tiled != nullptr) bulk_load_1d(s, cur.wtiled(), W_BYTES, &full_bar[stage]);
        else tma_load_2d(s, cur.wmap(), kc * BK, cur.wrow(), &full_bar[stage]);
        if (gate_open) {
          tma_load_2d(s + W_BYTES, def_map, kc * BK, 0, &full_bar[stage]);
        } else {
          def_stage[deferred] = stage; def_kb[deferred] = kc; ++deferred;
        }
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        cur.advance();
      }
      if (ok && deferred > 0 && event_wait(event_counter + gate_ev, per_event, abort_flag, WAIT_NS)) flush();
    }
  }
  else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = make_idesc_bf16_f32(128, static_cast<uint32_t>(npad));
      int stage = 0, acc = 0; uint32_t phase = 0, acc_phase = 0; bool ok = true;
      // one work item: two accumulators of 128 weight rows each
      auto run_item = [&](int kbs) -> bool {
        if (!mbar_wait_bounded(&tempty_bar[acc], acc_phase ^ 1u, abort_flag, WAIT_NS)) return false;
        tc_fence_after();
        const uint32_t g_tmem = tmem_base + static_cast<uint32_t>(acc * 2 * MAXN);
        for (int kb = 0; kb < kbs; ++kb) {
          if (!mbar_wait_bounded(&full_bar[stage], phase, abort_flag, WAIT_NS)) return false;
          tc_fence_after();
          const uint32_t s = smem_u32(ring + stage * STAGE_BYTES);
          const uint64_t w0 = make_desc_sw128_kmajor(s);
          const uint64_t w1 = make_desc_sw128_kmajor(s + 128 * BK * 2);
          const uint64_t xd = make_desc_sw128_kmajor(s + W_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint32_t accum = (kb | k) != 0 ? 1u : 0u;
            umma_bf16(g_tmem, w0 + 2 * k, xd + 2 * k, idesc, accum);
            umma_bf16(g_tmem + MAXN, w1 + 2 * k, xd + 2 * k, idesc, accum);
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
        for (int tile = cta; ok && tile < Ipad / 128; tile += ctas) ok = run_item(kb1);
        BItem it[4];
        const int nit = b_items(cta, ctas, m_blocks, Ipad / BK, it);
        for (int i = 0; ok && i < nit; ++i) ok = run_item(it[i].kb_hi - it[i].kb_lo);
      }
    }
  }
  else {
    // ------------------------------------------- epilogue warps (+ RMSNorm phase)
    const int quad = warp % 4;
    int acc = 0; uint32_t acc_phase = 0;
    bool ok = true;
    // One arrival per CTA (592 arrivals on one counter took longer than the meeting of four warps): every
    // thread makes its writes visible, the four warps meet, one thread arrives.  Called by all four warps
    // also after a wait has given up, so that the named barrier stays balanced.
    auto arrive_event = [&](int e) {
      if (ok) __threadfence();
      epilogue_bar_sync();
      if (ok && quad == 0 && lane == 0) atomicAdd(event_counter + e, 1u);
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
    // Once a wait has given up (ok == false) a warp skips all further work but still walks every
    // loop, so that the four warps keep meeting at the named barrier of the RMSNorm phase.
    for (int l = 0; l < n_layers; ++l) {
      const DecodeStackLayer* L = layers + l;
      const int Ipad = L->Ipad;
      // ---- phase N: x is final once every K slice of the previous layer has been added
      if (ok && l > 0) {
        bool w = event_wait(event_counter + 3 * l - 1, per_event, abort_flag, WAIT_NS);
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
      arrive_event(3 * l);                               // event N(l)
      // ---- phase A: Hd = bf16(silu(G) * U * scale)
      __nv_bfloat16* Hd = L->Hd;
      for (int tile = cta; tile < Ipad / 128; tile += ctas) {
        if (ok && !wait_acc()) ok = false;
        if (!ok) continue;
        const uint32_t taddr = tmem_base + static_cast<uint32_t>(acc * 2 * MAXN) + (static_cast<uint32_t>(quad * 32) << 16);
        const int64_t j = static_cast<int64_t>(tile) * 128 + quad * 32 + lane;
        const float sc = L->scale[j];
#pragma unroll
        for (int c = 0; c < MAXN; c += 32) {                   // 32 tokens at a time: gate and up columns together
          if (c < npad) {
            uint32_t g[32], u[32];
            tmem_ld_32x16(taddr + c, *reinterpret_cast<uint32_t(*)[16]>(&g[0]));
            tmem_ld_32x16(taddr + MAXN + c, *reinterpret_cast<uint32_t(*)[16]>(&u[0]));
            if (c + 16 < npad) {
              tmem_ld_32x16(taddr + c + 16, *reinterpret_cast<uint32_t(*)[16]>(&g[16]));
              tmem_ld_32x16(taddr + MAXN + c + 16, *reinterpret_cast<uint32_t(*)[16]>(&u[16]));
            }
            tmem_ld_wait();
            if (c + 32 >= npad) release_acc();                 // the last columns have been read
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const int t = c + i;
              if (t < n) {
                const float gv = __uint_as_float(g[i]);
                Hd[static_cast<int64_t>(t) * Ipad + j] = __float2bfloat16_rn(__fdividef(gv, 1.0f + __expf(-gv)) * __uint_as_float(u[i]) * sc);
              }
            }
          }
        }
      }
      arrive_event(3 * l + 1);                           // event A(l)
      // ---- phase B: every K slice adds its part into x
      BItem it[4];
      const int nit = b_items(cta, ctas, m_blocks, Ipad / BK, it);
      for (int i = 0; i < nit; ++i) {
        if (ok && !wait_acc()) ok = false;
        if (!ok) continue;
        const uint32_t taddr = tmem_base + static_cast<uint32_t>(acc * 2 * MAXN) + (static_cast<uint32_t>(quad * 32) << 16);
#pragma unroll
        for (int half = 0; half < 2; ++half) {                 // the two blocks of 128 output columns
          const int64_t m = static_cast<int64_t>(it[i].m_blk) * 256 + half * 128 + quad * 32 + lane;
#pragma unroll
          for (int c0 = 0; c0 < MAXN; c0 += 64) {              // 64 token rows at a time
            if (c0 < npad) {
              uint32_t v[64];
              load_acc_async(taddr + half * MAXN + c0, npad - c0, v);
              tmem_ld_wait();
              if (half == 1 && c0 + 64 >= npad) release_acc();   // the last columns have been read
              if (m < d) {
#pragma unroll
                for (int t = 0; t < 64; ++t)
                  if (c0 + t < n) atomicAdd(x + static_cast<int64_t>(c0 + t) * d + m, __uint_as_float(v[t]));
              }
            }
          }
        }
      }
      arrive_event(3 * l + 2);                           // event B(l)
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

cudaError_t decode_stack_init(int* max_ctas_per_sm) {
  cudaError_t e = cudaFuncSetAttribute(decode_stack_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_stack_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (e != cudaSuccess) return e;
  int a = 0, b = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, decode_stack_kernel<64>, NUM_THREADS, SMEM_BYTES);
  if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, decode_stack_kernel<128>, NUM_THREADS, SMEM_BYTES);
  *max_ctas_per_sm = a < b ? a : b;
  return e;
}

// layers_dev: n_layers records in device memory (64-byte aligned).  event_counter: 3 * n_layers zeros.
cudaError_t launch_decode_stack(const DecodeStackLayer* layers_dev, int n_layers, const CUtensorMap& tm_x, float* x, void* xnorm,
                                int64_t n, int64_t d, int npad, float eps, uint32_t* event_counter, uint32_t* status,
                                int num_sms, const WaitCfg& wait, cudaStream_t st) {
  if (n == 0 || n_layers == 0) return cudaSuccess;
  __nv_bfloat16* xn = static_cast<__nv_bfloat16*>(xnorm);
  uint64_t wait_ns = wait.limit_ns;
  uint32_t extra = wait.extra_arrivals;
  void* args[] = {const_cast<DecodeStackLayer**>(&layers_dev), &n_layers, const_cast<CUtensorMap*>(&tm_x), &x, &xn, &n, &d, &npad,
                  &eps, &event_counter, &status, &wait_ns, &extra};
  // cooperative launch: the grid-wide events need every CTA resident at once
  const void* kernel = npad <= 64 ? reinterpret_cast<const void*>(decode_stack_kernel<64>)
                                  : reinterpret_cast<const void*>(decode_stack_kernel<128>);
  return cudaLaunchCooperativeKernel(kernel, dim3(num_sms), dim3(NUM_THREADS), args, SMEM_BYTES, st);
}

}  // namespace mlpmoe
