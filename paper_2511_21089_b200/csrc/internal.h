// Internal launch interface between the C-ABI host code and the kernel files.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>
#include <vector>

namespace mlpmoe {

// Launch with programmatic stream serialization: the kernel may begin (set-up only) while its
// predecessor in the stream drains; every kernel launched this way executes griddepcontrol.wait
// before it touches global memory.
// Overlap is switched off (plain stream order) while a handle records per-kernel CUDA events:
// an event between two overlapped kernels would not mark the end of the first one.
inline bool& pdl_overlap_enabled() {
  static thread_local bool on = true;
  return on;
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = pdl_overlap_enabled() ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

constexpr int kGroup = 128;      // neurons per interleaved gate|up group in the packed operand
// A layer's packed weights (3 * d_model * surviving neurons * 2 bytes) count as L2-resident below this size:
// the prefill schedules may then re-read them at will instead of streaming them once per group of token blocks.
constexpr int64_t kWeightsFitL2Bytes = int64_t(48) << 20;
constexpr int kDecodeMaxTokens = 64;
constexpr int kDecodeStackMaxTokens = 128;  // most tokens the persistent decode-stack kernel takes (its 128-row build)

// Limits of the bounded waits of one launch.  Ordinary launches use the defaults; the test hook
// mlpmoe_debug_set_wait shortens the limit and adds `extra_arrivals` to the target of every wait of
// one CTA for work of other CTAs, so that such a wait runs out and the give-up path can be tested.
struct WaitCfg {
  uint64_t limit_ns = 1000000000ull;
  uint32_t extra_arrivals = 0;
};

// Device status word values (written by kernels whose bounded waits run out).
constexpr uint32_t kStatusOk = 0;
constexpr uint32_t kStatusTimeout = 1;

// ------------------------------------------------------------------ pack.cu --
// dst[c * rows + r] = src[r * cols + c]
cudaError_t launch_transpose(const void* src, void* dst, int64_t rows, int64_t cols, int elem_size, cudaStream_t st);
// Packed gate|up operand: rows [2*kGroup*q, +kGroup) = gate rows of compacted neurons [kGroup*q, +kGroup),
// next kGroup rows = their up rows; each row d contiguous elements.  Rows past n_active are zero.
cudaError_t launch_gather_gateup(const void* Wg_c, const void* Wu_c, const int32_t* src_row, void* Wgu,
                                 int64_t n_active, int64_t n_active_pad, int64_t d, int elem_size, cudaStream_t st);
// Packed down operand, K-major: WdT[m * n_active_pad + j'] = Wd_c[src_row[j'] * d + m]; columns past n_active zero.
cudaError_t launch_gather_down_t(const void* Wd_c, const int32_t* src_row, void* WdT, int64_t n_active,
                                 int64_t n_active_pad, int64_t d, int elem_size, cudaStream_t st);
// Per neuron row: non-zero counts of the gate, up and down rows: out[0*I + j], out[1*I + j], out[2*I + j].
cudaError_t launch_row_nnz(const void* Wg_c, const void* Wu_c, const void* Wd_c, int32_t* out, int64_t I, int64_t d,
                           int elem_size, cudaStream_t st);

// Three-way bf16 split of an fp32 matrix [rows x K] (row pitch src_pitch) into [rows x 3 Kp] bf16: segment s holds
// piece s of every element (p0 + p1 + p2 = 24 significand bits of the value), K padded with zeros to Kp (multiple of 64).
cudaError_t launch_split3(const float* src, void* dst, int64_t rows, int64_t K, int64_t Kp, int64_t src_pitch, cudaStream_t st);

// Neuron-structured Fade variant: score[j] = sum of squares of neuron j's gate and up rows (float64, terms added
// one after the other, gate row first); zero_rows clears the listed rows of both canonical matrices.
cudaError_t launch_neuron_scores(const void* Wg_c, const void* Wu_c, double* score, int64_t I, int64_t d, int elem_size, cudaStream_t st);
cudaError_t launch_zero_rows(void* A, void* B, const int32_t* rows_dev, int64_t n_rows, int64_t d, int elem_size, cudaStream_t st);

// Per-token branch selection (route.cu): stable grouping of the tokens by selected branch, the per-token
// compensation factor, the row gather, and the sum of the branches' output rows back into y.
cudaError_t launch_route_scan(const uint8_t* select, const uint8_t* avail, int64_t n, int B, int64_t list_stride, int32_t* pos,
                              int32_t* lists, int32_t* counts, cudaStream_t st);
cudaError_t launch_route_coef(const int32_t* pos, int64_t n, int B, int n_avail, int compensate, float* coef, cudaStream_t st);
cudaError_t launch_gather_rows(const void* src, const int32_t* list, int64_t n_rows, int64_t row_bytes, void* out, cudaStream_t st);
cudaError_t launch_gather_branches(const void* src, const int32_t* lists, int64_t list_stride, const int32_t* counts,
                                   const int32_t* rowbase, int b_lo, int b_hi, int64_t row_bytes, void* out, int blocks_per_branch,
                                   cudaStream_t st);
cudaError_t launch_fill_u32(uint32_t* dst, uint32_t value, int64_t count, cudaStream_t st);
cudaError_t launch_route_combine(const void* Ye, int ye_bf16, const int32_t* pos, const int32_t* rowbase, const float* coef, int64_t n,
                                 int B, int b_lo, int b_hi, int64_t d, int first, float* y, cudaStream_t st);

// Fade: exact rank selection on magnitude bit patterns, then masking (Section 3.2).
struct FadeSeg {
  void* base;      // first element of the slice (contiguous m elements)
  int64_t m;       // number of elements
  int64_t rank;    // 0-based rank lo of the threshold order statistic
};
// work: device scratch of fade_work_bytes(nseg) bytes.  Zeroes every element with |w| <= (rank-th smallest |w|).
size_t fade_work_bytes(int nseg);
cudaError_t launch_fade(const FadeSeg* segs_host, int nseg, void* work, int elem_size, cudaStream_t st);

// Stage-tiled copy of the packed bf16 operands for the fused few-token decode kernel: per tile of 128
// compacted neurons one contiguous run of 32 KB chunks, each the 128-byte-swizzled shared-memory image
// of one stage (256 rows x 64 K): first ceil(d / 64) chunks of Wgu rows [256 t, 256 t + 256) (K-step
// after K-step), then per block of 256 output columns two chunks of WdT[block rows, the tile's
// neurons 0..63 | 64..127].  Rows / columns past d are zero.
size_t decode_tiled_bytes(int64_t n_active_pad, int64_t d);
cudaError_t launch_retile_decode(const void* Wgu, const void* WdT, void* tiled, int64_t n_active_pad, int64_t d, cudaStream_t st);

// r = x / sqrt(mean(x^2) + eps), out bf16 (elem_size 2) or fp32 (4).
cudaError_t launch_rmsnorm(const float* x, void* r, int64_t n, int64_t d, float eps, int out_elem_size, cudaStream_t st);

// ------------------------------------------------------------- simt_gemm.cu --
// fp32 path.  H[n x ldh] = silu(X Wg'^T) * (X Wu'^T) * scale, Wgu packed as above.
cudaError_t launch_simt_gateup(const float* X, const float* Wgu, const float* scale, float* H, int64_t n, int64_t d,
                               int64_t n_active_pad, cudaStream_t st);
// Y[n x d] = (R +) H[n x K] * WdT[d x K]^T
cudaError_t launch_simt_down(const float* H, const float* WdT, const float* R, float* Y, int64_t n, int64_t d,
                             int64_t K, cudaStream_t st);

// --------------------------------------------------------------- tc_gemm.cu --
struct TcGateUpArgs {
  CUtensorMap tm_x;     // X   [n x d]            bf16, box 64 x 128, 128B swizzle
  CUtensorMap tm_w;     // Wgu [2*Ipad x d]       bf16, box 64 x 256
  const float* scale;   // [Ipad]
  void* H;              // [n x Ipad] bf16
  int64_t n, d, Ipad;
  uint32_t* status;
  // split3 != 0 (fast fp32 mode): both operands are three-way bf16 splits [rows x 3 dp], dp = d rounded up to 64;
  // the K loop runs the six piece products x0 w0, x0 w1, x0 w2, x1 w0, x1 w1, x2 w0, and H is written as the
  // three-way split [n x 3 Ipad] of the fp32 value.
  int split3 = 0;
};
struct TcDownArgs {
  CUtensorMap tm_h;     // H   [n x Ipad]         bf16, box 64 x 128
  CUtensorMap tm_w;     // WdT [d x Ipad]         bf16, box 64 x 128
  const float* R;       // optional fp32 residual [n x d]
  void* Y;              // [n x d] fp32 or bf16
  int y_bf16;
  int64_t n, d, Ipad;
  uint32_t* status;
  int split3 = 0;       // fast fp32 mode: H and WdT are three-way splits [rows x 3 Ipad]; six piece products
};
cudaError_t launch_tc_gateup(const TcGateUpArgs& a, int num_sms, cudaStream_t st);
cudaError_t launch_tc_down(const TcDownArgs& a, int num_sms, cudaStream_t st);
cudaError_t tc_gemm_init();   // opt in to the large dynamic shared memory sizes (once per process)

// -------------------------------------------------------------- tc_layer.cu --
// Both GEMMs of a layer call in one persistent CTA-pair kernel (n > 128).
struct TcLayerArgs {
  enum { OUT_DIRECT = 0, OUT_TMA_STORE = 1, OUT_TMA_ADD = 2 };   // how the down epilogue leaves
  CUtensorMap tm_x;      // X   [n x d]       bf16, box 64 x 128
  CUtensorMap tm_wgu;    // Wgu [2 Ipad x d]  bf16, box 64 x 128
  CUtensorMap tm_h_st;   // H   [n x Ipad]    bf16, box 64 x 32
  CUtensorMap tm_h_ld;   // H   [n x Ipad]    bf16, box 64 x 128
  CUtensorMap tm_wdt;    // WdT [d x Ipad]    bf16, box 64 x bn/2
  CUtensorMap tm_y;      // Y   [n x d]       fp32, box 32 x 32 (unused by OUT_DIRECT)
  const float* scale;
  const float* R;
  void* Y;
  int y_bf16, out_mode, bn, ksplit;
  int64_t n, d, Ipad;
  const int32_t* tile_list;     // device: per-pair tile sequences from tc_layer_schedule
  const int32_t* list_offsets;  // device: [num_sms / 2 + 1]
  uint32_t* done;        // [ceil(n / 256)] zero between calls
  uint32_t* passed;      // [ceil(n / 256)] zero between calls
  uint32_t* status;
  WaitCfg wait;
};
cudaError_t tc_layer_init();
int tc_layer_down_bn(int64_t n, int64_t d, int num_sms);
int tc_layer_ksplit(int64_t n, int64_t d, int64_t Ipad, int bn, int out_mode, int num_sms);
int64_t tc_layer_schedule(int64_t n, int64_t d, int64_t Ipad, int bn, int ksplit, int num_sms, std::vector<int32_t>* tiles,
                          std::vector<int32_t>* offsets);
cudaError_t launch_tc_layer(const TcLayerArgs& a, int num_sms, cudaStream_t st);

// -------------------------------------------------------------- tc_stack.cu --
// Whole pre-norm stack (n > 128) in one persistent CTA-pair kernel.  One record per layer in
// device memory; work items are (code, layer) pairs, code = type << 30 | column << 16 | token block.
constexpr int kItemGateUp = 0, kItemDown = 1, kItemNorm = 2;
constexpr int kStackNormParts = 16;    // norm items per 256-token block
constexpr uint32_t kStackNormArrivals = kStackNormParts * 4;   // arrivals a gate|up tile waits for (2 norm warps in each CTA of the pair)
struct alignas(64) TcStackLayer {
  CUtensorMap tm_wgu;    // Wgu [2 Ipad x d]  bf16, box 64 x 128
  CUtensorMap tm_h_st;   // H   [n x Ipad]    bf16, box 64 x 32
  CUtensorMap tm_h_ld;   // H   [n x Ipad]    bf16, box 64 x 128
  CUtensorMap tm_wdt;    // WdT [d x Ipad]    bf16, box 64 x bn/2
  const float* scale;    // [Ipad]
  int32_t n1;            // gate|up tiles per token block (Ipad / 128)
  int32_t kb2;           // K-steps of the down GEMM (Ipad / 64)
  int32_t ksplit;        // K slices per down tile
  int32_t pad_[11];
};
struct TcStackArgs {
  const TcStackLayer* layers;    // device, n_layers records
  int n_layers;
  CUtensorMap tm_x;      // Xn [n x d] bf16, box 64 x 128
  CUtensorMap tm_y;      // x  [n x d] fp32, box 32 x 32
  float* x;
  void* xnorm;
  int64_t n, d;
  int bn;
  float eps;
  const int32_t* items;          // device: (code, layer) pairs, 8-byte aligned
  const int32_t* list_offsets;   // device: [num_sms / 2 + 1], in items
  uint32_t* counters;            // device: [3 x n_layers x ceil(n / 256)], zero at launch
  uint32_t* status;
  WaitCfg wait;
  int out_add = 1;               // down items accumulate into x (stack) or overwrite it (grouped branches)
};
cudaError_t tc_stack_init();
void tc_stack_group_schedule(const int32_t* block_layer, int n_blocks, int64_t d, const int64_t* Ipad, int bn, int num_sms,
                             std::vector<int32_t>* items, std::vector<int32_t>* offsets);
void tc_stack_schedule(int64_t n, int64_t d, const int64_t* Ipad, const int* ksplit, int n_layers, int bn, int num_sms,
                       std::vector<int32_t>* items, std::vector<int32_t>* offsets);
cudaError_t launch_tc_stack(const TcStackArgs& a, int num_sms, cudaStream_t st);

// ---------------------------------------------------------------- decode.cu --
struct DecodeArgs {
  CUtensorMap tm_w;     // Wgu [2*Ipad x d]  box 64 x 64
  CUtensorMap tm_x;     // X   [n x d]       box 64 x npad
  CUtensorMap tm_wd;    // WdT [d x Ipad]    box 64 x 128
  CUtensorMap tm_h;     // Hd  [n x Ipad]    box 64 x npad
  const float* scale;
  void* Hd;             // [n x Ipad] bf16 workspace
  float* partial;       // [splits x d x npad] fp32 workspace
  uint32_t* counters;   // [d / 128] arrival counters, zero between calls
  const float* R;
  void* Y;
  int y_bf16;
  int64_t n, d, Ipad;
  int npad, splits;
  int accumulate;       // 1: Y (fp32) already holds the residual and every K slice adds into it
  uint32_t* status;
};
cudaError_t launch_decode_gateup(const DecodeArgs& a, int num_sms, cudaStream_t st);
cudaError_t launch_decode_down(const DecodeArgs& a, int num_sms, cudaStream_t st);
cudaError_t decode_init();

// ----------------------------------------------------------- decode_stack.cu --
// One record per layer of a decode stack, read by the persistent stack kernel from device memory.
struct alignas(64) DecodeStackLayer {
  CUtensorMap tm_wgu;    // Wgu [2 Ipad x d]  box 64 x 256
  CUtensorMap tm_wdt;    // WdT [d x Ipad]    box 64 x 256
  CUtensorMap tm_hd;     // Hd  [n x Ipad]    box 64 x npad
  const float* scale;    // [Ipad]
  __nv_bfloat16* Hd;     // [n x Ipad]
  const uint8_t* tiled;  // stage-tiled weight copy of the fused few-token kernel (decode_tiled_bytes), else null
  int32_t Ipad;
  int32_t pad_[9];
};
static_assert(sizeof(DecodeStackLayer) == 448, "record layout");
cudaError_t decode_stack_init(int* max_ctas_per_sm);
cudaError_t launch_decode_stack(const DecodeStackLayer* layers_dev, int n_layers, const CUtensorMap& tm_x, float* x, void* xnorm,
                                int64_t n, int64_t d, int npad, float eps, uint32_t* event_counter, uint32_t* status,
                                int num_sms, const WaitCfg& wait, cudaStream_t st);

// ----------------------------------------------------------- decode_fused.cu --
// Decode stack for at most kDecodeFusedMaxTokens tokens: both GEMMs of a layer on the CTA that owns the neurons.
constexpr int kDecodeFusedMaxTokens = 13;   // above, the partial sums per tile (fp32 atomics) cost more than the dependency saved (measured: even at 14)
cudaError_t decode_fused_init(int* max_ctas_per_sm);
cudaError_t launch_decode_fused(const DecodeStackLayer* layers_dev, int n_layers, const CUtensorMap& tm_x, float* x, void* xnorm,
                                int64_t n, int64_t d, float eps, uint32_t* event_counter, uint32_t* status, int num_sms,
                                const WaitCfg& wait, cudaStream_t st);

}  // namespace mlpmoe
