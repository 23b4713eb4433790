// Prefill of a whole pre-norm stack (n_tokens > 128) in ONE persistent kernel on CTA pairs:
//     x <- x + MLPMoE_l(RMSNorm(x))   for l = 0 .. L-1,
// every layer being the two GEMMs of Section 3.1
//     H = bf16( silu(Xn Wg'^T) * (Xn Wu'^T) * scale ),     x += H WdT^T   (branch sum inside the K loop).
// Token rows are independent through the whole stack, so there is no barrier between layers: each
// pair walks a host-built sequence of work items that spans all layers, and an item only waits
// (bounded) for the items of ITS 256-token block that it reads from:
//     norm item (layer l, block m, part)  reads x rows of block m:   all down items of (l-1, m)
//     gate|up tile (l, m, 128 neurons)    reads the normalised rows: all norm parts of (l, m)
//     down item (l, m, columns, K slice)  reads H rows of block m:   all gate|up tiles of (l, m)
// counted per (layer, block) in global memory.  Pairs that finish a layer's items early go on with
// the next layer's items of blocks that are already complete, so the SMs neither drain nor refill
// at a layer boundary, and the RMSNorm needs no launch of its own.
//
// The tiles, the pipeline and the first six warp roles are those of the single-layer kernel in
// tc_layer.cu (tcgen05 cta_group::2, M = 256, TMA 128B-swizzled K-major stages, two TMEM
// accumulators, epilogues through swizzled shared memory and TMA store / reduce-add).  Two more
// warps per CTA walk the pair's own sequence of norm items, apart from the GEMM pipeline: a norm
// part runs as soon as its block's down items are in, not when an epilogue warp gets round to it.
// No load uses cluster multicast.  Every wait is bounded.
#include <algorithm>
#include <utility>
#include <vector>

#include "tc_common.cuh"

namespace mlpmoe {
namespace {

using namespace ptx;
using namespace tc;

constexpr int STAGES = 6;
constexpr int A_BYTES = BM * BK * 2;                 // 16 KB
constexpr int B_HALF_MAX_BYTES = 128 * BK * 2;       // up to 128 weight rows per CTA
constexpr int STAGE_BYTES = A_BYTES + B_HALF_MAX_BYTES;
constexpr int STAGING_OFFSET = STAGES * STAGE_BYTES;                 // epilogue staging tiles, 8 KB per epilogue warp
constexpr int BAR_OFFSET = STAGING_OFFSET + 4 * STAGING_BYTES_PER_WARP;
constexpr int SMEM_BYTES = BAR_OFFSET + 256 + 1024;
static_assert(SMEM_BYTES <= 232448, "exceeds the 227 KB of shared memory a CTA may use");
constexpr int ACC_STRIDE = 256;                      // TMEM columns per accumulator buffer
constexpr int TMEM_COLS = 512;
constexpr int STACK_THREADS = 256;                   // producer, MMA, 4 epilogue and 2 norm warps
constexpr uint32_t ARRIVALS_PER_ITEM = 8;            // 4 epilogue warps in each of the two CTAs
constexpr int NORM_PARTS = kStackNormParts;          // norm items per 256-token block
constexpr uint32_t ARRIVALS_PER_NORM_ITEM = 4;       // 2 norm warps in each of the two CTAs
constexpr int NORM_ROWS_PER_WARP = 256 / NORM_PARTS / 4;
static_assert(NORM_PARTS * ARRIVALS_PER_NORM_ITEM == kStackNormArrivals, "the preset of the grouped-branch launches");
constexpr int NORM_VEC = 8;                          // float4 per lane and row kept in registers (d <= 1024 in one go)

struct StackParams {
  const TcStackLayer* layers;
  float* x;               // [n x d] fp32 residual stream, updated in place
  __nv_bfloat16* xnorm;   // [n x d] bf16, RMSNorm output = A operand of the gate|up tiles
  int64_t n, d;
  int m_pairs, kb1, bn, n2;
  float eps;
  const int2* items;            // per-pair sequences, concatenated: (code, layer); GEMM items of all pairs, then norm items
  const int32_t* list_offsets;  // [pairs + 1] GEMM sequences, then [pairs + 1] norm sequences
  uint32_t* done_norm;    // [L x m_pairs] arrivals of norm items
  uint32_t* done_gu;      // [L x m_pairs] arrivals of gate|up tiles
  uint32_t* done_dn;      // [L x m_pairs] arrivals of down items
  uint32_t* status;
  uint64_t wait_ns;       // limit of every bounded wait
  uint32_t extra;         // added to the target of every wait for other CTAs' arrivals (0 outside tests)
  int out_add;            // down items add their tile into x (the residual stream) / overwrite it (grouped branches)
};

struct Item {
  int type, m_pair, col, layer;
};
__device__ __forceinline__ Item decode_item(int2 e) {
  Item t;
  t.type = static_cast<int>(static_cast<uint32_t>(e.x) >> 30);
  t.col = (e.x >> 16) & 0x3FFF;
  t.m_pair = e.x & 0xFFFF;
  t.layer = e.y;
  return t;
}

__device__ __forceinline__ uint32_t ld_acquire_gpu(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// Bounded wait until `*counter` has reached `target`.
__device__ __forceinline__ bool wait_count(const uint32_t* counter, uint32_t target, volatile uint32_t* abort_flag,
                                           uint64_t WAIT_NS) {
  if (ld_acquire_gpu(counter) >= target) return true;
  const uint64_t t0 = globaltimer_ns();
  uint32_t polls = 0;
  while (true) {
    if (ld_acquire_gpu(counter) >= target) return true;
    __nanosleep(100);
    if ((++polls & 15u) == 0) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > WAIT_NS) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

// RMSNorm of ROWS token rows by one warp: r = x / sqrt(mean(x^2) + eps), rounded to bf16.  The loads
// of all rows are issued before the first reduction, so the rows share one round trip to L2.
template <int ROWS>
__device__ __forceinline__ void norm_rows(const float* __restrict__ x, __nv_bfloat16* __restrict__ xnorm, int64_t row0, int64_t n,
                                          int64_t d, float eps, int lane) {
  float4 v[ROWS][NORM_VEC];
  float ss[ROWS];
#pragma unroll
  for (int r = 0; r < ROWS; ++r) {
    const float* row = x + (row0 + r) * d;
#pragma unroll
    for (int i = 0; i < NORM_VEC; ++i) {
      const int64_t k = (static_cast<int64_t>(i) * 32 + lane) * 4;
      v[r][i] = (k < d && row0 + r < n) ? __ldcg(reinterpret_cast<const float4*>(row + k)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
#pragma unroll
  for (int r = 0; r < ROWS; ++r) {
    ss[r] = 0.f;
#pragma unroll
    for (int i = 0; i < NORM_VEC; ++i) ss[r] += v[r][i].x * v[r][i].x + v[r][i].y * v[r][i].y + v[r][i].z * v[r][i].z + v[r][i].w * v[r][i].w;
    if (row0 + r < n) {
      const float* row = x + (row0 + r) * d;
      for (int64_t k = (static_cast<int64_t>(NORM_VEC) * 32 + lane) * 4; k < d; k += 128) {    // rows wider than the register window
        const float4 w = __ldcg(reinterpret_cast<const float4*>(row + k));
        ss[r] += w.x * w.x + w.y * w.y + w.z * w.z + w.w * w.w;
      }
    }
    for (int o = 16; o > 0; o >>= 1) ss[r] += __shfl_xor_sync(0xFFFFFFFFu, ss[r], o);
  }
#pragma unroll
  for (int r = 0; r < ROWS; ++r) {
    if (row0 + r >= n) continue;
    const float inv = 1.0f / sqrtf(ss[r] / static_cast<float>(d) + eps);
    const float* row = x + (row0 + r) * d;
    __nv_bfloat16* out = xnorm + (row0 + r) * d;
#pragma unroll
    for (int i = 0; i < NORM_VEC; ++i) {
      const int64_t k = (static_cast<int64_t>(i) * 32 + lane) * 4;
      if (k < d)
        *reinterpret_cast<uint2*>(out + k) = make_uint2(pack_bf16(v[r][i].x * inv, v[r][i].y * inv), pack_bf16(v[r][i].z * inv, v[r][i].w * inv));
    }
    for (int64_t k = (static_cast<int64_t>(NORM_VEC) * 32 + lane) * 4; k < d; k += 128) {
      const float4 w = __ldcg(reinterpret_cast<const float4*>(row + k));
      *reinterpret_cast<uint2*>(out + k) = make_uint2(pack_bf16(w.x * inv, w.y * inv), pack_bf16(w.z * inv, w.w * inv));
    }
  }
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(STACK_THREADS, 1)
tc_stack_kernel(const __grid_constant__ CUtensorMap tm_x,        // Xn  [n x d] bf16   box 64 x 128
                const __grid_constant__ CUtensorMap tm_y,        // x   [n x d] fp32   box 32 x 32
                const StackParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + BAR_OFFSET);   // used in the even CTA
  uint64_t* empty_bar = full_bar + STAGES;                               // per CTA
  uint64_t* tfull_bar = empty_bar + STAGES;                              // per CTA
  uint64_t* tempty_bar = tfull_bar + 2;                                  // used in the even CTA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  const ClockProbe probe = clock_probe_begin();
  const uint64_t WAIT_NS = p.wait_ns;

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const uint32_t rank = cluster_ctarank();

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);       // one arrive.expect_tx by the even CTA's producer + bytes of both CTAs
      mbar_init(&empty_bar[s], 1);      // one commit arrival
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&tfull_bar[a], 1);      // one commit arrival
      mbar_init(&tempty_bar[a], 8);     // 4 epilogue warps of each CTA
    }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                   // both CTAs' barriers and TMEM exist before any remote signal
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  griddep_launch_dependents();
  griddep_wait();                       // inputs written by earlier kernels are complete and visible
  const int list_begin = p.list_offsets[cluster_id_x()];
  const int list_end = p.list_offsets[cluster_id_x() + 1];

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tensormap(&tm_x);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      // token blocks (below 64) of the current layer whose normalised rows / H rows are known to be complete
      uint64_t ready[2] = {0, 0};
      int ready_layer = -1;
      for (int i = list_begin; ok && i < list_end; ++i) {
        const Item t = decode_item(p.items[i]);
        const TcStackLayer* L = p.layers + t.layer;
        const bool down = t.type == kItemDown;
        if (t.layer != ready_layer) { ready_layer = t.layer; ready[0] = ready[1] = 0; }
        const int bn = down ? p.bn : 256;
        const int half_rows = bn / 2;
        const int ksplit = L->ksplit;
        const int n_blk = down ? t.col / ksplit : t.col, kslice = down ? t.col % ksplit : 0;
        const int kb_lo = down ? kslice * L->kb2 / ksplit : 0;
        const int kb_hi = down ? (kslice + 1) * L->kb2 / ksplit : p.kb1;
        const CUtensorMap* ma = down ? &L->tm_h_ld : &tm_x;
        const CUtensorMap* mb = down ? &L->tm_wdt : &L->tm_wgu;
        const int row_a = (t.m_pair * 2 + static_cast<int>(rank)) * BM;
        const int row_b = n_blk * bn + static_cast<int>(rank) * half_rows;
        const uint32_t stage_tx = 2u * static_cast<uint32_t>(A_BYTES + half_rows * BK * 2);   // bytes of both CTAs
        // the A operand of this item: normalised rows (all norm parts of the block) or H rows (all gate|up tiles)
        const uint32_t* counter = (down ? p.done_gu : p.done_norm) + static_cast<int64_t>(t.layer) * p.m_pairs + t.m_pair;
        const uint32_t target = down ? static_cast<uint32_t>(L->n1) * ARRIVALS_PER_ITEM : NORM_PARTS * ARRIVALS_PER_NORM_ITEM;
        const bool known = t.m_pair < 64 && ((ready[down ? 1 : 0] >> t.m_pair) & 1u);
        if (!known) {
          if (!wait_count(counter, target + p.extra, abort_flag, WAIT_NS)) { ok = false; break; }
          fence_proxy_async_all();       // the TMA loads below must observe what that acquire made visible
          if (t.m_pair < 64) ready[down ? 1 : 0] |= uint64_t(1) << t.m_pair;
        }
        for (int kb = kb_lo; kb < kb_hi; ++kb) {
          if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, WAIT_NS)) { ok = false; break; }
          uint8_t* sa = smem + stage * STAGE_BYTES;
          const uint32_t full_even = map_to_cta(smem_u32(&full_bar[stage]), 0);
          if (rank == 0) mbar_expect_tx(&full_bar[stage], stage_tx);
          tma_load_2d_pair(sa, ma, kb * BK, row_a, full_even);
          tma_load_2d_pair(sa + A_BYTES, mb, kb * BK, row_b, full_even);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      // tail: leave only after the MMAs have released every stage (their commits target these barriers)
      for (int i = 0; ok && i < STAGES; ++i) {
        if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, WAIT_NS)) break;
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------- MMA issuer (even CTA only)
    if (rank == 0 && lane == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int i = list_begin; ok && i < list_end; ++i) {
        const Item t = decode_item(p.items[i]);
        const TcStackLayer* L = p.layers + t.layer;
        const bool down = t.type == kItemDown;
        const int ksplit = L->ksplit;
        const int kslice = down ? t.col % ksplit : 0;
        const int kb_lo = down ? kslice * L->kb2 / ksplit : 0;
        const int kb_hi = down ? (kslice + 1) * L->kb2 / ksplit : p.kb1;
        const uint32_t idesc = make_idesc_bf16_f32(256, static_cast<uint32_t>(down ? p.bn : 256));
        if (!mbar_wait_bounded(&tempty_bar[acc], acc_phase ^ 1u, abort_flag, WAIT_NS)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * ACC_STRIDE);
        for (int kb = kb_lo; kb < kb_hi; ++kb) {
          if (!mbar_wait_bounded(&full_bar[stage], phase, abort_flag, WAIT_NS)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * STAGE_BYTES);
          const uint64_t a_desc = make_desc_sw128_kmajor(sa);
          const uint64_t b_desc = make_desc_sw128_kmajor(sa + A_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_bf16_pair(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb > kb_lo || k > 0) ? 1u : 0u);
          umma_commit_pair(&empty_bar[stage], 3);      // frees this stage in both CTAs
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit_pair(&tfull_bar[acc], 3);          // accumulator complete, both CTAs' epilogues may read
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else if (warp >= 6) {
    // ------------------------------------------------------------- norm warps
    const int nbegin = p.list_offsets[cluster_count_x() + 1 + cluster_id_x()];
    const int nend = p.list_offsets[cluster_count_x() + 2 + cluster_id_x()];
    for (int i = nbegin; i < nend; ++i) {
      const Item t = decode_item(p.items[i]);
      const int64_t cidx = static_cast<int64_t>(t.layer) * p.m_pairs + t.m_pair;
      if (t.layer > 0) {
        // x rows of the block are final once every down item of the previous layer has added its part
        bool ok = true;
        if (lane == 0)
          ok = wait_count(p.done_dn + cidx - p.m_pairs, static_cast<uint32_t>(p.n2 * p.layers[t.layer - 1].ksplit) * ARRIVALS_PER_ITEM + p.extra, abort_flag, WAIT_NS);
        ok = __all_sync(0xFFFFFFFFu, ok);    // also orders every lane's reads after lane 0's acquire
        if (!ok) break;
      }
      const int64_t row0 = static_cast<int64_t>(t.m_pair) * 256 + t.col * (256 / NORM_PARTS) +
                           (static_cast<int64_t>(rank) * 2 + (warp - 6)) * NORM_ROWS_PER_WARP;
      norm_rows<NORM_ROWS_PER_WARP>(p.x, p.xnorm, row0, p.n, p.d, p.eps, lane);
      __threadfence();                   // this warp's rows are visible device-wide before the arrival is
      __syncwarp();
      if (lane == 0) atomicAdd(p.done_norm + cidx, 1u);
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int quad = warp % 4;
    uint8_t* staging = smem + STAGING_OFFSET + (warp - 2) * STAGING_BYTES_PER_WARP;
    uint32_t tiles_stored = 0;
    int acc = 0;
    uint32_t acc_phase = 0;
    if (lane == 0) prefetch_tensormap(&tm_y);
    for (int i = list_begin; i < list_end; ++i) {
      const Item t = decode_item(p.items[i]);
      const TcStackLayer* L = p.layers + t.layer;
      const int64_t cidx = static_cast<int64_t>(t.layer) * p.m_pairs + t.m_pair;
      bool ok = mbar_wait_bounded(&tfull_bar[acc], acc_phase, abort_flag, WAIT_NS);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after();
      const int32_t row0 = (t.m_pair * 2 + static_cast<int>(rank)) * BM + quad * 32;
      const uint32_t taddr = tmem_base + static_cast<uint32_t>(acc * ACC_STRIDE) + (static_cast<uint32_t>(quad * 32) << 16);
      const uint32_t tempty_even = map_to_cta(smem_u32(&tempty_bar[acc]), 0);
      auto release = [&]() {               // the accumulator buffer may be overwritten by the next tile's MMAs
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(tempty_even);
      };
      if (t.type == kItemGateUp) {
        epilogue_swiglu_tma(taddr, L->scale, &L->tm_h_st, staging, tiles_stored, lane, row0, t.col * 128, release);
      } else {
        epilogue_out_tma(taddr, &tm_y, staging, tiles_stored, lane, row0, (t.col / L->ksplit) * p.bn, p.bn, p.out_add, release);
      }
      if (lane == 0) {
        tma_store_wait_all<0>();           // this warp's part of H (or of x) has been written ...
        fence_proxy_async_all();
        __threadfence();                   // ... and is visible device-wide before the arrival is
        atomicAdd((t.type == kItemGateUp ? p.done_gu : p.done_dn) + cidx, 1u);
      }
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
    if (lane == 0) tma_store_wait_all<0>();   // this warp's bulk stores have completed
  }

  __syncwarp();
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                   // neither CTA leaves while the other may still signal or read it
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status, kStatusTimeout);
  if (blockIdx.x == 0 && threadIdx.x == 0) clock_probe_end(p.status, probe);
}

inline int32_t encode_item(int type, int col, int m_pair) {
  return static_cast<int32_t>((static_cast<uint32_t>(type) << 30) | (static_cast<uint32_t>(col) << 16) | static_cast<uint32_t>(m_pair));
}

}  // namespace

cudaError_t tc_stack_init() {
  return cudaFuncSetAttribute(tc_stack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
}

// Work sequences of every CTA pair for the whole stack.  The GEMM items have one global order (a
// stream over layers and token blocks, see below) and go, in that order, to the pair with the
// least estimated work so far, so the deal keeps balancing across layer boundaries; norm parts go
// round-robin, in (layer, block, part) order, to the pairs' norm warps.  Every sequence (a pair's
// GEMM items; a pair's norm parts) is the global order restricted to its items and every item
// comes after the items it waits for, so with all pairs resident the waits cannot form a cycle.
// items: GEMM items of pair 0, 1, ... then norm items of pair 0, 1, ..., as (code, layer);
// offsets: [pairs + 1] for the GEMM sequences followed by [pairs + 1] for the norm sequences.
void tc_stack_schedule(int64_t n, int64_t d, const int64_t* Ipad, const int* ksplit, int n_layers, int bn, int num_sms,
                       std::vector<int32_t>* items, std::vector<int32_t>* offsets) {
  const int pairs = num_sms / 2 > 0 ? num_sms / 2 : 1;
  const int m_pairs = static_cast<int>((n + 255) / 256);
  const int n2 = static_cast<int>((d + bn - 1) / bn);
  const int64_t kb1 = (d + BK - 1) / BK;
  auto kstep_cycles = [](int width) {
    const int64_t mma = 2 * width, fill = (A_BYTES + (width / 2) * BK * 2) / 50;
    return mma > fill ? mma : fill;
  };
  std::vector<int64_t> load(pairs, 0);
  std::vector<std::vector<int32_t>> lists(pairs), norm_lists(pairs);
  int next = 0;                          // ties go round-robin
  auto give = [&](int32_t code, int layer, int64_t cost) {
    int c = next;
    for (int i = 0; i < pairs; ++i) {
      const int cand = (next + i) % pairs;
      if (load[cand] < load[c]) c = cand;
    }
    lists[c].push_back(code);
    lists[c].push_back(layer);
    load[c] += cost;
    next = (c + 1) % pairs;
  };
  int norm_next = 0;
  for (int l = 0; l < n_layers; ++l)
    for (int m = 0; m < m_pairs; ++m)
      for (int part = 0; part < NORM_PARTS; ++part) {
        norm_lists[norm_next].push_back(encode_item(kItemNorm, part, m));
        norm_lists[norm_next].push_back(l);
        norm_next = (norm_next + 1) % pairs;
      }
  // The GEMM items as one stream over (layer, group of token blocks): slot s holds the gate|up tiles
  // of its group and the down items of the group `lag` slots earlier, also across layer boundaries.
  // A group is one token block when the layers' weights fit in L2 (they can be re-read at will) and
  // 8 token blocks otherwise (the weights are streamed from HBM once per group, the tiles of a group
  // walking the weight tiles together).  lag < groups per layer, so a block's down items still come
  // before its gate|up tiles of the next layer.  The further back in the order the items that an
  // item waits for, the less a pair that runs a little ahead of the others has to wait: 7/16 of the
  // groups leaves the down items about as far behind their block's tiles as the next layer's tiles
  // are behind the block's down items plus the time its norm takes.
  bool fits_l2 = true;
  for (int l = 0; l < n_layers; ++l) fits_l2 = fits_l2 && 3 * d * Ipad[l] * 2 <= kWeightsFitL2Bytes;
  const int group = fits_l2 ? 1 : 8;
  const int n_groups = (m_pairs + group - 1) / group;
  int lag = (7 * n_groups + 8) / 16;
  if (lag > n_groups - 1) lag = n_groups - 1;
  const int slots = n_layers * n_groups;
  for (int sl = 0; sl < slots + lag; ++sl) {
    if (sl < slots) {
      const int l = sl / n_groups, g = sl % n_groups;
      const int n1 = static_cast<int>(Ipad[l] / 128);
      const int64_t cost_g = kb1 * kstep_cycles(256) + 1500;
      const int g0 = g * group, g1 = g0 + group < m_pairs ? g0 + group : m_pairs;
      for (int nb = 0; nb < n1; ++nb)
        for (int m = g0; m < g1; ++m) give(encode_item(kItemGateUp, nb, m), l, cost_g);
    }
    if (sl >= lag) {
      const int l = (sl - lag) / n_groups, g = (sl - lag) % n_groups;
      const int64_t cost_d = (Ipad[l] / BK) * kstep_cycles(bn) / ksplit[l] + 1500 + 24 * bn;
      const int g0 = g * group, g1 = g0 + group < m_pairs ? g0 + group : m_pairs;
      for (int m = g0; m < g1; ++m)
        for (int nb = 0; nb < n2 * ksplit[l]; ++nb) give(encode_item(kItemDown, nb, m), l, cost_d);
    }
  }
  items->clear();
  offsets->clear();
  for (int pass = 0; pass < 2; ++pass) {
    offsets->push_back(static_cast<int32_t>(items->size() / 2));
    for (int c = 0; c < pairs; ++c) {
      const std::vector<int32_t>& src = pass == 0 ? lists[c] : norm_lists[c];
      items->insert(items->end(), src.begin(), src.end());
      offsets->push_back(static_cast<int32_t>(items->size() / 2));
    }
  }
}

// Work sequences for grouped branches (per-token branch selection): every 256-row block of the
// gathered token matrix belongs to ONE branch, whose weights are the block's "layer" record.  A
// block has the gate|up tiles of its branch and then its down items (one K slice), nothing else:
// no norm parts (the norm sequences are empty; the caller presets the norm counters to their
// target) and no dependency between blocks.  Same form as tc_stack_schedule: one global order
// (slot s: the gate|up tiles of block s, then the down items of block s - lag), dealt to the pair
// with the least estimated work; an item only waits for items earlier in that order.
void tc_stack_group_schedule(const int32_t* block_layer, int n_blocks, int64_t d, const int64_t* Ipad, int bn, int num_sms,
                             std::vector<int32_t>* items, std::vector<int32_t>* offsets) {
  const int pairs = num_sms / 2 > 0 ? num_sms / 2 : 1;
  const int n2 = static_cast<int>((d + bn - 1) / bn);
  const int64_t kb1 = (d + BK - 1) / BK;
  auto kstep_cycles = [](int width) {
    const int64_t mma = 2 * width, fill = (A_BYTES + (width / 2) * BK * 2) / 50;
    return mma > fill ? mma : fill;
  };
  // (estimated work, pair) as a min-heap: this schedule is rebuilt at every call, so dealing an item costs log(pairs)
  std::vector<std::pair<int64_t, int>> heap;
  for (int c = 0; c < pairs; ++c) heap.emplace_back(0, c);
  auto later = [](const std::pair<int64_t, int>& a, const std::pair<int64_t, int>& b) { return a > b; };
  std::vector<std::vector<int32_t>> lists(pairs);
  auto give = [&](int32_t code, int layer, int64_t cost) {
    std::pop_heap(heap.begin(), heap.end(), later);
    std::pair<int64_t, int>& top = heap.back();
    lists[top.second].push_back(code);
    lists[top.second].push_back(layer);
    top.first += cost;
    std::push_heap(heap.begin(), heap.end(), later);
  };
  // the down items of a block come about a wave and a half of gate|up tiles after the block's own tiles
  int64_t tiles = 0;
  for (int r = 0; r < n_blocks; ++r) tiles += Ipad[block_layer[r]] / 128;
  const int64_t per_block = n_blocks > 0 ? (tiles + n_blocks - 1) / n_blocks : 1;
  int lag = static_cast<int>((3 * pairs + 2 * per_block - 1) / (2 * per_block)) + 1;
  if (lag > n_blocks) lag = n_blocks;
  for (int sl = 0; sl < n_blocks + lag; ++sl) {
    if (sl < n_blocks) {
      const int l = block_layer[sl];
      const int64_t cost_g = kb1 * kstep_cycles(256) + 1500;
      for (int nb = 0; nb < static_cast<int>(Ipad[l] / 128); ++nb) give(encode_item(kItemGateUp, nb, sl), l, cost_g);
    }
    if (sl >= lag) {
      const int r = sl - lag, l = block_layer[r];
      const int64_t cost_d = (Ipad[l] / BK) * kstep_cycles(bn) + 1500 + 24 * bn;
      for (int nb = 0; nb < n2; ++nb) give(encode_item(kItemDown, nb, r), l, cost_d);
    }
  }
  items->clear();
  offsets->clear();
  offsets->push_back(0);
  for (int c = 0; c < pairs; ++c) {
    items->insert(items->end(), lists[c].begin(), lists[c].end());
    offsets->push_back(static_cast<int32_t>(items->size() / 2));
  }
  for (int c = 0; c <= pairs; ++c) offsets->push_back(static_cast<int32_t>(items->size() / 2));    // empty norm sequences
}

cudaError_t launch_tc_stack(const TcStackArgs& a, int num_sms, cudaStream_t st) {
  if (a.n == 0 || a.n_layers == 0) return cudaSuccess;
  StackParams p{};
  p.layers = a.layers;
  p.x = a.x;
  p.xnorm = static_cast<__nv_bfloat16*>(a.xnorm);
  p.n = a.n;
  p.d = a.d;
  p.m_pairs = static_cast<int>((a.n + 255) / 256);
  p.kb1 = static_cast<int>((a.d + BK - 1) / BK);
  p.bn = a.bn;
  p.n2 = static_cast<int>((a.d + a.bn - 1) / a.bn);
  p.eps = a.eps;
  p.items = reinterpret_cast<const int2*>(a.items);
  p.list_offsets = a.list_offsets;
  p.done_norm = a.counters;
  p.done_gu = a.counters + static_cast<int64_t>(a.n_layers) * p.m_pairs;
  p.done_dn = a.counters + 2 * static_cast<int64_t>(a.n_layers) * p.m_pairs;
  p.status = a.status;
  p.wait_ns = a.wait.limit_ns;
  p.extra = a.wait.extra_arrivals;
  p.out_add = a.out_add;
  const int pairs = num_sms / 2 > 0 ? num_sms / 2 : 1;
  return launch_pdl(tc_stack_kernel, dim3(2 * pairs), dim3(STACK_THREADS), SMEM_BYTES, st, a.tm_x, a.tm_y, p);
}

}  // namespace mlpmoe
