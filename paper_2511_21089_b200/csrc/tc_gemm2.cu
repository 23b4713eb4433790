// Prefill GEMMs on CTA pairs (tcgen05 cta_group::2).  One tcgen05.mma of shape 256 x N x 16
// spans two SMs: each CTA stages its own 128 token rows of A and only HALF of the N weight rows
// of B, and the tensor cores of both SMs read the two halves from both shared memories.  Per
// CTA and K-step that is 16 KB (A) + N/2 x 128 B (B) of shared-memory fill for 128 x N x 64
// multiply-accumulates - two thirds of what a lone CTA needs at N = 256 - which matters because
// these kernels are bound by the L2 -> SM fill rate, not by the tensor pipes.
//
//   gate|up : N = 256 = 128 gate rows (staged by the even CTA) | 128 up rows (odd CTA) of the
//             same 128 neurons; epilogue H = bf16(silu(gate) * up * scale)   (Section 3.1)
//   down    : N = bn (runtime, multiple of 32, <= 256); Y = (R +) H * WdT^T, the K loop running
//             over all surviving neurons of all surviving branches in one accumulator.
//
// Roles per CTA (192 threads): warp 0 TMA producer; warp 1 TMEM owner and, in the even CTA only,
// MMA issuer for the pair; warps 2..5 epilogue of this CTA's 128 rows.  Barriers: each CTA has
// its own "empty" and "accumulator full" barriers, reached by multicast commits from the issuing
// thread; the "full" and "accumulator empty" barriers that the issuer waits on live in the even
// CTA and are signalled from both CTAs.  No load uses cluster multicast.
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
constexpr uint64_t WAIT_NS = 1000000000ull;
enum { OUT_DIRECT = 0, OUT_TMA_STORE = 1, OUT_TMA_ADD = 2 };   // how the down epilogue leaves

template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
tc_pair_gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                    const __grid_constant__ CUtensorMap tm_out, const EpiArgs ep, int num_m_pairs, int num_n_blocks,
                    int num_k_blocks, int bn, int out_mode) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + BAR_OFFSET);   // used in the even CTA
  uint64_t* empty_bar = full_bar + STAGES;                               // per CTA
  uint64_t* tfull_bar = empty_bar + STAGES;                              // per CTA
  uint64_t* tempty_bar = tfull_bar + 2;                                  // used in the even CTA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const uint32_t rank = cluster_ctarank();
  const int BN = (EPI == EPI_SWIGLU) ? 256 : bn;
  const int half_rows = BN / 2;

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
  const int num_tiles = num_m_pairs * num_n_blocks;
  const int first_tile = static_cast<int>(cluster_id_x());
  const int tile_step = static_cast<int>(cluster_count_x());

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tensormap(&tm_a);
      prefetch_tensormap(&tm_b);
      const uint32_t stage_tx = 2u * static_cast<uint32_t>(A_BYTES + half_rows * BK * 2);   // bytes of both CTAs
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = first_tile; ok && tile < num_tiles; tile += tile_step) {
        const int m_pair = tile % num_m_pairs, n_blk = tile / num_m_pairs;
        const int row_a = (m_pair * 2 + static_cast<int>(rank)) * BM;
        const int row_b = n_blk * BN + static_cast<int>(rank) * half_rows;
        for (int kb = 0; kb < num_k_blocks; ++kb) {
          if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, WAIT_NS)) { ok = false; break; }
          uint8_t* sa = smem + stage * STAGE_BYTES;
          const uint32_t full_even = map_to_cta(smem_u32(&full_bar[stage]), 0);
          if (rank == 0) mbar_expect_tx(&full_bar[stage], stage_tx);
          tma_load_2d_pair(sa, &tm_a, kb * BK, row_a, full_even);
          tma_load_2d_pair(sa + A_BYTES, &tm_b, kb * BK, row_b, full_even);
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
      const uint32_t idesc = make_idesc_bf16_f32(256, static_cast<uint32_t>(BN));
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int tile = first_tile; ok && tile < num_tiles; tile += tile_step) {
        if (!mbar_wait_bounded(&tempty_bar[acc], acc_phase ^ 1u, abort_flag, WAIT_NS)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * ACC_STRIDE);
        for (int kb = 0; kb < num_k_blocks; ++kb) {
          if (!mbar_wait_bounded(&full_bar[stage], phase, abort_flag, WAIT_NS)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * STAGE_BYTES);
          const uint64_t a_desc = make_desc_sw128_kmajor(sa);
          const uint64_t b_desc = make_desc_sw128_kmajor(sa + A_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_bf16_pair(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
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
    if (lane == 0) prefetch_tensormap(&tm_out);
    for (int tile = first_tile; tile < num_tiles; tile += tile_step) {
      const int m_pair = tile % num_m_pairs, n_blk = tile / num_m_pairs;
      bool ok = mbar_wait_bounded(&tfull_bar[acc], acc_phase, abort_flag, WAIT_NS);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after();
      const int32_t row0 = (m_pair * 2 + static_cast<int>(rank)) * BM + quad * 32;
      const uint32_t taddr = tmem_base + static_cast<uint32_t>(acc * ACC_STRIDE) + (static_cast<uint32_t>(quad * 32) << 16);
      const uint32_t tempty_even = map_to_cta(smem_u32(&tempty_bar[acc]), 0);
      auto release = [&]() {               // the accumulator buffer may be overwritten by the next tile's MMAs
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(tempty_even);
      };
      if (EPI == EPI_SWIGLU) {
        epilogue_swiglu_tma(taddr, ep.scale, &tm_out, staging, tiles_stored, lane, row0, n_blk * 128, release);
      } else if (out_mode != OUT_DIRECT) {
        epilogue_out_tma(taddr, &tm_out, staging, tiles_stored, lane, row0, n_blk * BN, BN, out_mode == OUT_TMA_ADD, release);
      } else {
        epilogue_out(taddr, ep, static_cast<int64_t>(row0) + lane, static_cast<int64_t>(n_blk) * BN, BN);
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
  if (threadIdx.x == 0 && *abort_flag) atomicExch(ep.status, kStatusTimeout);
}

}  // namespace

cudaError_t tc_pair_init() {
  cudaError_t e = cudaFuncSetAttribute(tc_pair_gemm_kernel<EPI_SWIGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(tc_pair_gemm_kernel<EPI_OUT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
}

// Width of the down-projection tile (a multiple of 32, 64..256): the one that minimises
// waves x (time of one K-step), where a K-step costs the larger of its tensor-core time
// (2 x width cycles for a 256 x width x 64 step) and the time to fill one CTA's stage from L2
// (16 KB of A + width/2 rows of B at about 50 bytes per cycle per SM, the rate these kernels
// see).  Narrow tiles need fewer waves but re-read A more often; ties go to the wider tile.
int tc_pair_down_bn(int64_t n, int64_t d, int num_sms) {
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

cudaError_t launch_tc_pair_gateup(const TcGateUpArgs& a, int num_sms, cudaStream_t st) {
  if (a.n == 0) return cudaSuccess;
  const int m_pairs = static_cast<int>((a.n + 255) / 256);
  const int n_blocks = static_cast<int>(a.Ipad / 128);
  const int k_blocks = static_cast<int>((a.d + BK - 1) / BK);
  EpiArgs ep{};
  ep.scale = a.scale;
  ep.out = a.H;
  ep.rows = a.n;
  ep.cols = a.Ipad;
  ep.ld = a.Ipad;
  ep.status = a.status;
  const int tiles = m_pairs * n_blocks;
  const int pairs = tiles < num_sms / 2 ? tiles : num_sms / 2;
  return launch_pdl(tc_pair_gemm_kernel<EPI_SWIGLU>, dim3(2 * pairs), dim3(NUM_THREADS), SMEM_BYTES, st, a.tm_x, a.tm_w, a.tm_out,
                    ep, m_pairs, n_blocks, k_blocks, 256, static_cast<int>(OUT_TMA_STORE));
}

cudaError_t launch_tc_pair_down(const TcDownArgs& a, int bn, int num_sms, cudaStream_t st) {
  if (a.n == 0) return cudaSuccess;
  const int m_pairs = static_cast<int>((a.n + 255) / 256);
  const int n_blocks = static_cast<int>((a.d + bn - 1) / bn);
  const int k_blocks = static_cast<int>(a.Ipad / BK);
  EpiArgs ep{};
  ep.R = a.R;
  ep.out = a.Y;
  ep.rows = a.n;
  ep.cols = a.d;
  ep.ld = a.d;
  ep.out_bf16 = a.y_bf16;
  ep.status = a.status;
  const int tiles = m_pairs * n_blocks;
  const int pairs = tiles < num_sms / 2 ? tiles : num_sms / 2;
  // fp32 output leaves through TMA: plain store without a residual, add-in-place when the residual
  // is the output buffer itself; other combinations use the direct (per-thread) epilogue
  int mode = OUT_DIRECT;
  if (!a.y_bf16 && a.R == nullptr) mode = OUT_TMA_STORE;
  else if (!a.y_bf16 && a.R == a.Y) mode = OUT_TMA_ADD;
  return launch_pdl(tc_pair_gemm_kernel<EPI_OUT>, dim3(2 * pairs), dim3(NUM_THREADS), SMEM_BYTES, st, a.tm_h, a.tm_w, a.tm_out, ep,
                    m_pairs, n_blocks, k_blocks, bn, mode);
}

}  // namespace mlpmoe
