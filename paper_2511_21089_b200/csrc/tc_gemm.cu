// Prefill path on the 5th-generation tensor cores (sm_100a): two persistent, warp-specialised
// GEMM kernels with bf16 operands staged by TMA into 128-byte-swizzled shared memory, tcgen05.mma
// accumulating in fp32 in tensor memory, and a double-buffered accumulator so that the epilogue
// of one tile runs under the MMAs of the next.
//
//   gate|up  (Section 3.1, inner bracket):   one 128 x 256 accumulator holds gate (columns 0..127)
//            and up (columns 128..255) of the same 128 neurons; the epilogue computes
//            H = bf16( silu(gate) * up * scale ), scale[j] = effective alpha of neuron j's branch.
//   down     (Section 3.1, outer product and branch sum): Y = (R +) H * WdT^T with the K loop
//            running over every surviving neuron of every surviving branch in one accumulator.
//
// Warp roles (192 threads): warp 0 = TMA producer (one lane), warp 1 = TMEM owner + MMA issuer
// (one lane), warps 2..5 = epilogue (TMEM lane quadrant = warp index mod 4).
#include "tc_common.cuh"

namespace mlpmoe {
namespace {

using namespace ptx;
using namespace tc;

template <int BN, int STAGES>
struct Cfg {
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
  static constexpr int SMEM_BYTES = BAR_OFFSET + 256 + 1024;   // barriers + slack for 1024-byte alignment
  static constexpr int TMEM_COLS = 2 * BN;                      // two accumulator buffers
};

template <int BN, int STAGES, int EPI>
__global__ void __launch_bounds__(NUM_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b, const EpiArgs ep,
               int num_m_blocks, int num_n_blocks, int num_k_blocks, int kseg, int two_acc) {
  // K loop over num_k_blocks = terms * kseg blocks of 64: term t multiplies segment a_seg(t) of A's row by segment
  // b_seg(t) of B's row.  One term (kseg = num_k_blocks) is the plain product; the six terms of the fast fp32
  // mode pair the three-way splits of both operands as (0,0) (0,1) (0,2) (1,0) (1,1) (2,0).
  // two_acc (six-term mode): the leading term (0,0) and the five correction terms, 2^-8 and less of it,
  // accumulate in two accumulators that the epilogue adds.  The tensor cores' fp32 accumulation loses a
  // little on every add in proportion to the running sum; keeping the number of adds into the large sum
  // at a sixth, and the long tail of adds on a sum 2^-8 as large, keeps the total within fp32 round-off.
  using C = Cfg<BN, STAGES>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + C::BAR_OFFSET);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* tfull_bar = empty_bar + STAGES;
  uint64_t* tempty_bar = tfull_bar + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  // accumulator buffers: two (the epilogue of a tile runs under the MMAs of the next) unless the two accumulators
  // of a tile in two_acc mode already fill the 512 columns of tensor memory
  const uint32_t acc_stride = two_acc ? 2u * BN : static_cast<uint32_t>(BN);
  const int nbuf = 2u * acc_stride <= 512u ? 2 : 1;
  const uint32_t tmem_cols = static_cast<uint32_t>(nbuf) * acc_stride;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&tfull_bar[a], 1);
      mbar_init(&tempty_bar[a], 4);
    }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  griddep_launch_dependents();          // the next kernel may begin its set-up
  griddep_wait();                       // inputs written by earlier kernels are complete and visible
  const int num_tiles = num_m_blocks * num_n_blocks;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tensormap(&tm_a);
      prefetch_tensormap(&tm_b);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        const int m_blk = tile % num_m_blocks, n_blk = tile / num_m_blocks;
        for (int kb = 0; kb < num_k_blocks; ++kb) {
          if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
          uint8_t* sa = smem + stage * C::STAGE_BYTES;
          mbar_expect_tx(&full_bar[stage], C::STAGE_BYTES);
          const int term = kb / kseg, r = kb % kseg;
          const int a_seg = term < 3 ? 0 : (term < 5 ? 1 : 2), b_seg = term < 3 ? term : (term < 5 ? term - 3 : 0);
          tma_load_2d(sa, &tm_a, (a_seg * kseg + r) * BK, m_blk * BM, &full_bar[stage]);
          tma_load_2d(sa + C::A_BYTES, &tm_b, (b_seg * kseg + r) * BK, n_blk * BN, &full_bar[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      // tail: leave only after the MMAs have released every stage (their commits target these barriers)
      for (int i = 0; ok && i < STAGES; ++i) {
        if (!mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag)) break;
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16_f32(BM, BN);
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        if (!mbar_wait_bounded(&tempty_bar[acc], acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_main = tmem_base + static_cast<uint32_t>(acc) * acc_stride;
        for (int kb = 0; kb < num_k_blocks; ++kb) {
          const bool corr = two_acc && kb >= kseg;               // a correction term
          const uint32_t d_tmem = corr ? d_main + BN : d_main;
          const int kb_first = corr ? kseg : 0;
          if (!mbar_wait_bounded(&full_bar[stage], phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * C::STAGE_BYTES);
          const uint64_t a_desc = make_desc_sw128_kmajor(sa);
          const uint64_t b_desc = make_desc_sw128_kmajor(sa + C::A_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advancing 16 elements along K inside the swizzled row = +32 bytes = +2 in the address field
            umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb != kb_first || k != 0) ? 1u : 0u);
          }
          umma_commit(&empty_bar[stage]);       // stage is free once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(&tfull_bar[acc]);           // accumulator complete
        if (++acc == nbuf) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int quad = warp % 4;
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
      const int m_blk = tile % num_m_blocks, n_blk = tile / num_m_blocks;
      bool ok = mbar_wait_bounded(&tfull_bar[acc], acc_phase, abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after();
      const int64_t row = static_cast<int64_t>(m_blk) * BM + quad * 32 + lane;
      const uint32_t taddr = tmem_base + static_cast<uint32_t>(acc) * acc_stride + (static_cast<uint32_t>(quad * 32) << 16);
      if (EPI == EPI_SWIGLU)
        epilogue_swiglu(taddr, ep, row, static_cast<int64_t>(n_blk) * (BN / 2), BN / 2);
      else if (EPI == EPI_SWIGLU_SPLIT3)
        epilogue_swiglu_split3(taddr, ep, row, static_cast<int64_t>(n_blk) * (BN / 2), BN / 2, two_acc ? taddr + BN : 0u);
      else
        epilogue_out(taddr, ep, row, static_cast<int64_t>(n_blk) * BN, BN, two_acc ? taddr + BN : 0u);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tempty_bar[acc]);
      if (++acc == nbuf) { acc = 0; acc_phase ^= 1u; }
    }
  }

  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, tmem_cols);
  }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(ep.status, kStatusTimeout);
}

constexpr int GU_BN = 256, GU_STAGES = 4;
constexpr int DN_BN = 128, DN_STAGES = 6;

}  // namespace

cudaError_t tc_gemm_init() {
  cudaError_t e = cudaFuncSetAttribute(tc_gemm_kernel<GU_BN, GU_STAGES, EPI_SWIGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       Cfg<GU_BN, GU_STAGES>::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(tc_gemm_kernel<GU_BN, GU_STAGES, EPI_SWIGLU_SPLIT3>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           Cfg<GU_BN, GU_STAGES>::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(tc_gemm_kernel<DN_BN, DN_STAGES, EPI_OUT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              Cfg<DN_BN, DN_STAGES>::SMEM_BYTES);
}

cudaError_t launch_tc_gateup(const TcGateUpArgs& a, int num_sms, cudaStream_t st) {
  if (a.n == 0) return cudaSuccess;
  const int m_blocks = static_cast<int>((a.n + BM - 1) / BM);
  const int n_blocks = static_cast<int>(a.Ipad / (GU_BN / 2));
  const int k_blocks = static_cast<int>((a.d + BK - 1) / BK);
  EpiArgs ep{};
  ep.scale = a.scale;
  ep.out = a.H;
  ep.rows = a.n;
  ep.cols = a.Ipad;
  ep.ld = a.split3 ? 3 * a.Ipad : a.Ipad;
  ep.status = a.status;
  const int tiles = m_blocks * n_blocks;
  const int grid = tiles < num_sms ? tiles : num_sms;
  if (a.split3)
    return launch_pdl(tc_gemm_kernel<GU_BN, GU_STAGES, EPI_SWIGLU_SPLIT3>, dim3(grid), dim3(NUM_THREADS),
                      Cfg<GU_BN, GU_STAGES>::SMEM_BYTES, st, a.tm_x, a.tm_w, ep, m_blocks, n_blocks, 6 * k_blocks, k_blocks, 1);
  return launch_pdl(tc_gemm_kernel<GU_BN, GU_STAGES, EPI_SWIGLU>, dim3(grid), dim3(NUM_THREADS),
                    Cfg<GU_BN, GU_STAGES>::SMEM_BYTES, st, a.tm_x, a.tm_w, ep, m_blocks, n_blocks, k_blocks, k_blocks, 0);
}

cudaError_t launch_tc_down(const TcDownArgs& a, int num_sms, cudaStream_t st) {
  if (a.n == 0) return cudaSuccess;
  const int m_blocks = static_cast<int>((a.n + BM - 1) / BM);
  const int n_blocks = static_cast<int>((a.d + DN_BN - 1) / DN_BN);
  const int k_blocks = static_cast<int>(a.Ipad / BK);
  EpiArgs ep{};
  ep.R = a.R;
  ep.out = a.Y;
  ep.rows = a.n;
  ep.cols = a.d;
  ep.ld = a.d;
  ep.out_bf16 = a.y_bf16;
  ep.status = a.status;
  const int tiles = m_blocks * n_blocks;
  const int grid = tiles < num_sms ? tiles : num_sms;
  return launch_pdl(tc_gemm_kernel<DN_BN, DN_STAGES, EPI_OUT>, dim3(grid), dim3(NUM_THREADS), Cfg<DN_BN, DN_STAGES>::SMEM_BYTES,
                    st, a.tm_h, a.tm_w, ep, m_blocks, n_blocks, a.split3 ? 6 * k_blocks : k_blocks, k_blocks, a.split3 ? 1 : 0);
}

}  // namespace mlpmoe
