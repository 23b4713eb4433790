// One persistent kernel per layer call for n_tokens > 128: both GEMMs of the layer
//     H = bf16( silu(X Wg'^T) * (X Wu'^T) * scale )          (Section 3.1, inner bracket)
//     Y = (R +) H WdT^T                                       (outer product + branch sum)
// run on CTA pairs (tcgen05 cta_group::2, see below) from one tile list: first every gate|up
// tile, then every down tile.  A down tile of a 256-token block may only read H once all
// gate|up tiles of that block have been stored; the epilogue warps count finished tiles per
// block in global memory and the producers of down tiles wait (bounded) for the count.  Fusing
// the two GEMMs removes a launch and lets down tiles fill the SMs that the last, partial wave
// of gate|up tiles would leave idle.
//
// CTA pairs: one tcgen05.mma of shape 256 x N x 16 spans two SMs; each CTA stages its own 128
// token rows of A and only HALF of the N weight rows of B, and both SMs' tensor cores read both
// halves.  Per CTA and K-step that is 16 KB (A) + N/2 x 128 B (B) of shared-memory fill for
// 128 x N x 64 multiply-accumulates, two thirds of a lone CTA's at N = 256; the L2 -> SM fill
// rate is what bounds these kernels at small K.
//
//   gate|up tile: N = 256 = 128 gate rows (staged by the even CTA) | 128 up rows (odd CTA) of
//                 the same 128 neurons; K = d_model.
//   down tile:    N = bn (multiple of 32, <= 256, chosen per call); K = all surviving neurons
//                 of all surviving branches, one fp32 accumulator.
//
// Roles per CTA (192 threads): warp 0 TMA producer; warp 1 TMEM owner and, in the even CTA,
// MMA issuer for the pair; warps 2..5 epilogue of this CTA's 128 rows (through swizzled shared
// memory and TMA stores).  Barriers: "empty" and "accumulator full" per CTA, reached by
// multicast commits; "full" and "accumulator empty" live in the even CTA and are signalled from
// both.  No load uses cluster multicast.  Every wait is bounded.
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
constexpr uint32_t ARRIVALS_PER_GATEUP_TILE = 8;     // 4 epilogue warps in each of the two CTAs

struct LayerParams {
  const float* scale;     // [Ipad] per-neuron scale
  const float* R;         // optional fp32 residual [n x d]
  void* Y;                // [n x d] fp32 or bf16
  int64_t n, d;
  int y_bf16;
  int out_mode;           // TcLayerArgs::OUT_*
  int m_pairs;            // 256-token blocks
  int n1, kb1;            // gate|up: tiles per token block (Ipad / 128), K-steps (d / 64)
  int n2, kb2, bn;        // down: tiles per token block, K-steps (Ipad / 64), tile width
  int ksplit;             // down tiles are cut into this many K slices (> 1 only when Y is accumulated into)
  const int32_t* tile_list;     // per-cluster tile sequences, concatenated (see encode_tile)
  const int32_t* list_offsets;  // [clusters + 1] start of each cluster's sequence
  uint32_t* done;         // [m_pairs] finished gate|up tile arrivals; zero between calls
  uint32_t* passed;       // [m_pairs] down-tile producers that have seen the block complete; zero between calls
  uint32_t* status;
  uint64_t wait_ns;       // limit of every bounded wait
  uint32_t extra;         // added to the target of every wait for other CTAs' arrivals (0 outside tests)
};

struct Tile {
  int is_down, m_pair, n_blk, kslice;
};

// Tile code: bit 31 = down tile, bits 16..30 = tile index along the output columns, bits 0..15 =
// 256-token block.
// For down tiles the column field holds column_tile * ksplit + K slice.
__device__ __forceinline__ Tile decode_tile(int32_t code, int ksplit) {
  Tile t;
  t.is_down = (static_cast<uint32_t>(code) >> 31) & 1;
  const int col = (code >> 16) & 0x7FFF;
  t.n_blk = t.is_down ? col / ksplit : col;
  t.kslice = t.is_down ? col % ksplit : 0;
  t.m_pair = code & 0xFFFF;
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

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
tc_layer_kernel(const __grid_constant__ CUtensorMap tm_x,        // X   [n x d]        box 64 x 128
                const __grid_constant__ CUtensorMap tm_wgu,      // Wgu [2 Ipad x d]   box 64 x 128
                const __grid_constant__ CUtensorMap tm_h_st,     // H   [n x Ipad]     box 64 x 32   (epilogue stores)
                const __grid_constant__ CUtensorMap tm_h_ld,     // H   [n x Ipad]     box 64 x 128  (A operand of down)
                const __grid_constant__ CUtensorMap tm_wdt,      // WdT [d x Ipad]     box 64 x bn/2
                const __grid_constant__ CUtensorMap tm_y,        // Y   [n x d] fp32   box 32 x 32
                const LayerParams p) {
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
  griddep_launch_dependents();          // the next kernel may begin its set-up
  griddep_wait();                       // inputs written by earlier kernels are complete and visible
  // this CTA pair's tile sequence (the same for every role of both CTAs)
  const int list_begin = p.list_offsets[cluster_id_x()];
  const int list_end = p.list_offsets[cluster_id_x() + 1];

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tensormap(&tm_x);
      prefetch_tensormap(&tm_wgu);
      prefetch_tensormap(&tm_h_ld);
      prefetch_tensormap(&tm_wdt);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int i = list_begin; ok && i < list_end; ++i) {
        const Tile t = decode_tile(p.tile_list[i], p.ksplit);
        const int bn = t.is_down ? p.bn : 256;
        const int half_rows = bn / 2;
        const int kb_lo = t.is_down ? t.kslice * p.kb2 / p.ksplit : 0;
        const int kb_hi = t.is_down ? (t.kslice + 1) * p.kb2 / p.ksplit : p.kb1;
        const CUtensorMap* ma = t.is_down ? &tm_h_ld : &tm_x;
        const CUtensorMap* mb = t.is_down ? &tm_wdt : &tm_wgu;
        const int row_a = (t.m_pair * 2 + static_cast<int>(rank)) * BM;
        const int row_b = t.n_blk * bn + static_cast<int>(rank) * half_rows;
        const uint32_t stage_tx = 2u * static_cast<uint32_t>(A_BYTES + half_rows * BK * 2);   // bytes of both CTAs
        if (t.is_down) {
          // H rows of this token block are complete once every gate|up tile of the block has arrived
          if (!wait_count(p.done + t.m_pair, static_cast<uint32_t>(p.n1) * ARRIVALS_PER_GATEUP_TILE + p.extra, abort_flag, WAIT_NS)) { ok = false; break; }
          fence_proxy_async_all();       // the TMA loads below must observe what that acquire made visible
          // the last of the 2 * n2 * ksplit producers of this block to get here re-arms the counters for the next call
          if (atomicAdd(p.passed + t.m_pair, 1u) == static_cast<uint32_t>(2 * p.n2 * p.ksplit - 1)) {
            p.done[t.m_pair] = 0;
            p.passed[t.m_pair] = 0;
          }
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
        const Tile t = decode_tile(p.tile_list[i], p.ksplit);
        const int kb_lo = t.is_down ? t.kslice * p.kb2 / p.ksplit : 0;
        const int kb_hi = t.is_down ? (t.kslice + 1) * p.kb2 / p.ksplit : p.kb1;
        const uint32_t idesc = make_idesc_bf16_f32(256, static_cast<uint32_t>(t.is_down ? p.bn : 256));
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
  } else {
    // ---------------------------------------------------------------- epilogue
    const int quad = warp % 4;
    uint8_t* staging = smem + STAGING_OFFSET + (warp - 2) * STAGING_BYTES_PER_WARP;
    uint32_t tiles_stored = 0;
    int acc = 0;
    uint32_t acc_phase = 0;
    if (lane == 0) {
      prefetch_tensormap(&tm_h_st);
      prefetch_tensormap(&tm_y);
    }
    EpiArgs ep{};
    ep.R = p.R;
    ep.out = p.Y;
    ep.rows = p.n;
    ep.cols = p.d;
    ep.ld = p.d;
    ep.out_bf16 = p.y_bf16;
    for (int i = list_begin; i < list_end; ++i) {
      const Tile t = decode_tile(p.tile_list[i], p.ksplit);
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
      if (!t.is_down) {
        epilogue_swiglu_tma(taddr, p.scale, &tm_h_st, staging, tiles_stored, lane, row0, t.n_blk * 128, release);
        if (lane == 0) {
          tma_store_wait_all<0>();         // this warp's part of H has been written ...
          fence_proxy_async_all();
          __threadfence();                 // ... and is visible device-wide before the arrival is
          atomicAdd(p.done + t.m_pair, 1u);
        }
      } else if (p.out_mode != TcLayerArgs::OUT_DIRECT) {
        epilogue_out_tma(taddr, &tm_y, staging, tiles_stored, lane, row0, t.n_blk * p.bn, p.bn,
                         p.out_mode == TcLayerArgs::OUT_TMA_ADD, release);
      } else {
        epilogue_out(taddr, ep, static_cast<int64_t>(row0) + lane, static_cast<int64_t>(t.n_blk) * p.bn, p.bn);
        release();
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

}  // namespace

cudaError_t tc_layer_init() {
  return cudaFuncSetAttribute(tc_layer_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
}

// Width of the down-projection tile (a multiple of 32, 64..256): the one that minimises
// waves x (time of one K-step), where a K-step costs the larger of its tensor-core time
// (2 x width cycles for a 256 x width x 64 step) and the time to fill one CTA's stage from L2
// (16 KB of A + width/2 rows of B at about 50 bytes per cycle per SM, the rate these kernels
// see).  Narrow tiles need fewer waves but re-read A more often; ties go to the wider tile.
int tc_layer_down_bn(int64_t n, int64_t d, int num_sms) {
  const int64_t pairs = num_sms / 2 > 0 ? num_sms / 2 : 1;
  const int64_t m_pairs = (n + 255) / 256;
  int best = 256;
  int64_t best_cost = -1;
  for (int bn = 256; bn >= 64; bn -= 32) {
    const int64_t tiles = m_pairs * ((d + bn - 1) / bn);
    const int64_t mma_cycles = 2 * bn;
    const int64_t fill_cycles = (A_BYTES + (bn / 2) * BK * 2) / 50;
    const int64_t step = mma_cycles > fill_cycles ? mma_cycles : fill_cycles;
    const int64_t cost = ((tiles + pairs - 1) / pairs) * step;
    if (best_cost < 0 || cost < best_cost) { best = bn; best_cost = cost; }
  }
  return best;
}

namespace {
inline int32_t encode_tile(bool is_down, int n_blk, int m_pair) {
  return static_cast<int32_t>((is_down ? 0x80000000u : 0u) | (static_cast<uint32_t>(n_blk) << 16) | static_cast<uint32_t>(m_pair));
}
// Estimated cycles of one K-step of a 256 x bn pair tile: tensor-core time or L2 fill time.
inline int64_t kstep_cycles(int bn) {
  const int64_t mma = 2 * bn, fill = (A_BYTES + (bn / 2) * BK * 2) / 50;
  return mma > fill ? mma : fill;
}
}  // namespace

// Static tile schedule: which CTA pair runs which tiles, in which order.  A greedy list scheduler
// over estimated tile costs.  Token blocks are taken in groups; a group's gate|up tiles run with
// the token block fastest (tiles in flight share weight tiles, the group shares one pass over the
// weights), and its down tiles become eligible once the simulation has finished every gate|up
// tile of their token block, so that they are handed to pairs that would otherwise idle at the end
// of a wave.  Every pair's sequence follows one global order in which a down tile comes after all
// gate|up tiles of its token block: the waits inside the kernel therefore cannot form a cycle.
int64_t tc_layer_schedule(int64_t n, int64_t d, int64_t Ipad, int bn, int ksplit, int num_sms, std::vector<int32_t>* tiles,
                          std::vector<int32_t>* offsets) {
  const int pairs = num_sms / 2 > 0 ? num_sms / 2 : 1;
  const int m_pairs = static_cast<int>((n + 255) / 256);
  const int n1 = static_cast<int>(Ipad / 128), n2 = static_cast<int>((d + bn - 1) / bn) * ksplit;   // down items per token block
  const int64_t cost_g = ((d + BK - 1) / BK) * kstep_cycles(256) + 1500;
  const int64_t cost_d = (Ipad / BK) * kstep_cycles(bn) / ksplit + 1500 + 24 * bn;     // + exposed part of the epilogue
  // Group size.  Weights that fit in L2 can be re-read at will: take the token blocks one by one, so
  // that they complete (and their down tiles become eligible) one by one.  Larger weights are
  // streamed from HBM once per group: take enough token blocks to keep every pair busy on one pass
  // over the weight tiles, and at least 8.
  int group = (pairs + n1 - 1) / n1 + 1;
  const bool weights_fit_l2 = 3 * d * Ipad * 2 <= kWeightsFitL2Bytes;
  if (weights_fit_l2) group = 1;        // one token block after the other: blocks complete one by one, early
  else if (group < 8) group = 8;
  if (group > m_pairs) group = m_pairs;
  std::vector<int32_t> g_order;
  g_order.reserve(static_cast<size_t>(m_pairs) * n1);
  for (int g0 = 0; g0 < m_pairs; g0 += group)
    for (int nb = 0; nb < n1; ++nb)
      for (int m = g0; m < g0 + group && m < m_pairs; ++m) g_order.push_back(encode_tile(false, nb, m));
  std::vector<int64_t> avail(pairs, 0);
  std::vector<std::vector<int32_t>> lists(pairs);
  if (weights_fit_l2) {
    // Small layer: every gate|up tile (token block after token block), then every down item in the
    // same block order, dealt round-robin.  Blocks complete progressively during the first phase, so
    // by the time a pair reaches a down item its block has long been complete; the items are short
    // enough (K slices) for the plain deal to balance.
    int c = 0;
    for (int32_t code : g_order) {
      lists[c].push_back(code);
      avail[c] += cost_g;
      c = (c + 1) % pairs;
    }
    for (int m = 0; m < m_pairs; ++m)
      for (int nb = 0; nb < n2; ++nb) {
        lists[c].push_back(encode_tile(true, nb, m));
        avail[c] += cost_d;
        c = (c + 1) % pairs;
      }
    g_order.clear();
  }
  std::vector<int> g_left(m_pairs, n1);
  std::vector<int64_t> block_done_at(m_pairs, 0);
  struct Ready { int64_t at; int32_t code; };
  std::vector<Ready> d_ready;          // FIFO of eligible down tiles
  size_t d_head = 0, g_next = 0;
  const size_t total = weights_fit_l2 ? 0 : static_cast<size_t>(m_pairs) * (n1 + n2);
  size_t assigned = 0;
  // down tiles are the large items: no pair takes more than its share of them while gate|up tiles remain
  const int d_quota = static_cast<int>((static_cast<int64_t>(m_pairs) * n2 + pairs - 1) / pairs);
  std::vector<int> d_taken(pairs, 0);
  // pending completions of simulated gate|up tiles: (finish time, token block)
  std::vector<std::pair<int64_t, int>> running;
  auto retire = [&](int64_t now) {
    for (size_t i = 0; i < running.size();) {
      if (running[i].first <= now) {
        const int m = running[i].second;
        if (block_done_at[m] < running[i].first) block_done_at[m] = running[i].first;
        if (--g_left[m] == 0)
          // eligible one gate|up tile time after the simulated completion: real tiles finish a little
          // off the estimate, and a pair that reaches a down tile too early stalls on it
          for (int nb = 0; nb < n2; ++nb) d_ready.push_back({block_done_at[m] + cost_g, encode_tile(true, nb, m)});
        running[i] = running.back();
        running.pop_back();
      } else {
        ++i;
      }
    }
  };
  while (assigned < total) {
    int c = 0;
    for (int i = 1; i < pairs; ++i)
      if (avail[i] < avail[c]) c = i;
    int64_t now = avail[c];
    retire(now);
    int cd = -1;                         // the earliest-free pair that still has room for a down tile
    if (d_head < d_ready.size() && (d_ready[d_head].at <= now || g_next >= g_order.size())) {
      for (int i = 0; i < pairs; ++i)
        if (d_taken[i] < d_quota && (cd < 0 || avail[i] < avail[cd])) cd = i;
      if (cd < 0 && g_next >= g_order.size()) cd = c;    // everyone has a share and nothing else is left
    }
    if (cd >= 0) {
      ++d_taken[cd];
      lists[cd].push_back(d_ready[d_head].code);
      const int64_t t0 = avail[cd] > d_ready[d_head].at ? avail[cd] : d_ready[d_head].at;
      avail[cd] = t0 + cost_d;
      ++d_head;
    } else if (g_next < g_order.size()) {
      const int32_t code = g_order[g_next++];
      lists[c].push_back(code);
      avail[c] = now + cost_g;
      running.push_back({avail[c], static_cast<int>(code & 0xFFFF)});
    } else {
      // only down tiles whose gate|up tiles are still running in the simulation remain: advance time
      int64_t next = -1;
      for (const auto& r : running)
        if (next < 0 || r.first < next) next = r.first;
      avail[c] = next > now ? next : now + 1;
      continue;
    }
    ++assigned;
  }
  tiles->clear();
  offsets->assign(1, 0);
  for (int c = 0; c < pairs; ++c) {
    tiles->insert(tiles->end(), lists[c].begin(), lists[c].end());
    offsets->push_back(static_cast<int32_t>(tiles->size()));
  }
  int64_t makespan = 0;                 // simulated finish time of the last pair, in cycles of the cost model
  for (int c = 0; c < pairs; ++c) makespan = avail[c] > makespan ? avail[c] : makespan;
  return makespan;
}

// Number of K slices per down tile (1..4): the one whose simulated schedule finishes first.
// Slicing is only possible when Y is accumulated into (each slice adds its part), and only matters
// when a CTA pair gets few tiles: whole down tiles, several times longer than gate|up tiles, then
// cannot be balanced across the pairs.
int tc_layer_ksplit(int64_t n, int64_t d, int64_t Ipad, int bn, int out_mode, int num_sms) {
  if (out_mode != TcLayerArgs::OUT_TMA_ADD) return 1;
  const int64_t pairs = num_sms / 2 > 0 ? num_sms / 2 : 1;
  const int64_t m_pairs = (n + 255) / 256;
  if (m_pairs * (Ipad / 128 + (d + bn - 1) / bn) >= 24 * pairs) return 1;
  int best = 1;
  int64_t best_t = -1;
  std::vector<int32_t> t, o;
  for (int k = 1; k <= 4; ++k) {
    if (k > 1 && (Ipad / BK) / k < 8) break;
    const int64_t span = tc_layer_schedule(n, d, Ipad, bn, k, num_sms, &t, &o);
    if (best_t < 0 || span < best_t - best_t / 50) { best = k; best_t = span; }   // a finer cut must win by 2 %
  }
  return best;
}

cudaError_t launch_tc_layer(const TcLayerArgs& a, int num_sms, cudaStream_t st) {
  if (a.n == 0) return cudaSuccess;
  LayerParams p{};
  p.scale = a.scale;
  p.R = a.R;
  p.Y = a.Y;
  p.n = a.n;
  p.d = a.d;
  p.y_bf16 = a.y_bf16;
  p.out_mode = a.out_mode;
  p.m_pairs = static_cast<int>((a.n + 255) / 256);
  p.n1 = static_cast<int>(a.Ipad / 128);
  p.kb1 = static_cast<int>((a.d + BK - 1) / BK);
  p.bn = a.bn;
  p.n2 = static_cast<int>((a.d + a.bn - 1) / a.bn);
  p.kb2 = static_cast<int>(a.Ipad / BK);
  p.ksplit = a.ksplit;
  p.tile_list = a.tile_list;
  p.list_offsets = a.list_offsets;
  p.done = a.done;
  p.passed = a.passed;
  p.status = a.status;
  p.wait_ns = a.wait.limit_ns;
  p.extra = a.wait.extra_arrivals;
  const int pairs = num_sms / 2 > 0 ? num_sms / 2 : 1;     // pairs without tiles have empty sequences
  return launch_pdl(tc_layer_kernel, dim3(2 * pairs), dim3(NUM_THREADS), SMEM_BYTES, st, a.tm_x, a.tm_wgu, a.tm_h_st, a.tm_h_ld,
                    a.tm_wdt, a.tm_y, p);
}

}  // namespace mlpmoe
