// C-ABI entry points and the host side of the library: argument checks, the weight packer's
// control flow, the branch scheduler (Section 3.3 -> K-list), Fade set-up (Section 3.2) and the
// dispatch of mlpmoe_forward onto the prefill / decode / fp32 kernels.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/mlpmoe.h"
#include "internal.h"

using namespace mlpmoe;

namespace {

#define CK(expr)                                   \
  do {                                             \
    cudaError_t e__ = (expr);                      \
    if (e__ != cudaSuccess) return MLPMOE_ERR_CUDA; \
  } while (0)

inline int64_t round_up(int64_t a, int64_t b) { return (a + b - 1) / b * b; }

// Activation workspace; may be shared by the layers of a stack.
struct Workspace {
  void* H = nullptr;       // [max_tokens x Ipad_max] layer dtype: silu(gate)*up*scale
  void* xnorm = nullptr;   // [max_tokens x d] layer dtype: RMSNorm output / host-call staging of x
  float* yres = nullptr;   // [max_tokens x d] fp32: host-call staging of y / the residual stream
  int64_t max_tokens = 0, Ipad_max = 0, d = 0;
  int elem_size = 0;
  int refs = 0;
};

void ws_release(Workspace* w) {
  if (!w) return;
  if (--w->refs > 0) return;
  cudaFree(w->H);
  cudaFree(w->xnorm);
  cudaFree(w->yres);
  delete w;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

// Row-major matrix [outer x inner] of bf16 (elem_size 2) or fp32 (4) with row pitch `pitch_elems`;
// box = 128 bytes x box_outer rows, 128-byte swizzle.
bool make_tmap_t(CUtensorMap* m, const void* ptr, int64_t inner, int64_t outer, int64_t pitch_elems, int box_outer,
                 int elem_size) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(inner), static_cast<cuuint64_t>(outer)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(pitch_elems) * elem_size};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(128 / elem_size), static_cast<cuuint32_t>(box_outer)};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, elem_size == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
            const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
bool make_tmap(CUtensorMap* m, const void* ptr, int64_t inner, int64_t outer, int64_t pitch_elems, int box_outer) {
  return make_tmap_t(m, ptr, inner, outer, pitch_elems, box_outer, 2);
}

// ------------------------------------------------------------ host logic ----
// floor(s * (m - 1)) on the exact value of the double s, 0 <= s < 1.
int64_t fade_position_exact(double s, int64_t m) {
  if (s <= 0.0 || m <= 1) return 0;
  int exp = 0;
  const double mant = std::frexp(s, &exp);                       // s = mant * 2^exp, mant in [0.5, 1)
  const unsigned long long M = static_cast<unsigned long long>(std::ldexp(mant, 53));   // exact: 53-bit integer
  const int shift = 53 - exp;                                    // s = M * 2^-shift, shift >= 53
  unsigned __int128 P = static_cast<unsigned __int128>(M) * static_cast<unsigned __int128>(m - 1);
  if (shift >= 128) return 0;
  return static_cast<int64_t>(P >> shift);
}

int64_t fade_position_default(int b, int B, int64_t m) {
  return static_cast<int64_t>((static_cast<__int128>(9) * b * (m - 1)) / (static_cast<__int128>(10) * B));
}

struct Schedule {
  std::vector<int32_t> branches;
  std::vector<int64_t> seg_start, seg_len;
  int64_t n_active = 0;
};

// Surviving branches (alpha != 0 and at least one live neuron) and the maximal runs of live
// neurons inside them, in ascending order.
void build_schedule(int B, const int64_t* d_b, const float* alpha_eff, const uint8_t* live, Schedule* out) {
  out->branches.clear();
  out->seg_start.clear();
  out->seg_len.clear();
  out->n_active = 0;
  int64_t off = 0;
  for (int b = 0; b < B; ++b) {
    const int64_t lo = off, hi = off + d_b[b];
    off = hi;
    if (alpha_eff[b] == 0.0f) continue;
    bool any = false;
    int64_t run = -1;
    for (int64_t j = lo; j < hi; ++j) {
      const bool alive = live == nullptr || live[j] != 0;
      if (alive) {
        any = true;
        if (run < 0) run = j;
      } else if (run >= 0) {
        out->seg_start.push_back(run);
        out->seg_len.push_back(j - run);
        out->n_active += j - run;
        run = -1;
      }
    }
    if (run >= 0) {
      out->seg_start.push_back(run);
      out->seg_len.push_back(hi - run);
      out->n_active += hi - run;
    }
    if (any) out->branches.push_back(b);
  }
}

mlpmoe_status_t prune_alpha_host(int B, const float* alpha, const uint8_t* keep, int compensate, float* out) {
  int K = 0;
  for (int b = 0; b < B; ++b) K += keep[b] ? 1 : 0;
  if (K == 0) return MLPMOE_ERR_EMPTY_KEEP_SET;
  const double c = compensate ? std::sqrt(static_cast<double>(B) / static_cast<double>(K)) : 1.0;
  for (int b = 0; b < B; ++b) out[b] = keep[b] ? static_cast<float>(c * static_cast<double>(alpha[b])) : 0.0f;
  return MLPMOE_OK;
}

mlpmoe_status_t check_partition(int64_t d_inter, int B, const int64_t* d_b, int64_t granule) {
  if (B <= 0 || d_b == nullptr) return MLPMOE_ERR_INVALID_ARG;
  int64_t sum = 0;
  for (int b = 0; b < B; ++b) {
    if (d_b[b] <= 0 || d_b[b] % granule != 0) return MLPMOE_ERR_BAD_PARTITION;
    sum += d_b[b];
  }
  return sum == d_inter ? MLPMOE_OK : MLPMOE_ERR_BAD_PARTITION;
}

// Per-token branch selection (mlpmoe_forward_routed): one single-branch layer per available branch, made
// from the parent's canonical weights and current gates, and the buffers of the grouping step.
struct Routed {
  int64_t version = -1;                    // parent's schedule version the children were built for
  std::vector<mlpmoe_layer_s*> child;      // [B]; nullptr where alpha_b = 0
  int n_avail = 0;
  uint8_t* avail = nullptr;                // device [B]
  int32_t *pos = nullptr, *lists = nullptr, *counts = nullptr, *rowbase = nullptr;   // device: [max_tokens x B], [B x max_tokens], [B], [B]
  float* coef = nullptr;                   // device [max_tokens]
  void *Xe = nullptr, *Ye = nullptr;       // gathered rows of one branch; outputs of the branches of one pass
  int64_t ye_rows = 0;                     // rows of Ye (and, grouped, of Xe and Hg)
  std::vector<int32_t> counts_host, rowbase_host;
  // bf16 layers: all branches of a pass in ONE launch of the stack kernel, the branches as its "layers"
  bool grouped = false;
  TcStackLayer* recs = nullptr;            // device [B]
  void* Hg = nullptr;                      // [ye_rows x h_pitch] bf16
  int64_t h_pitch = 0;
  int bn = 256;
  int32_t* items = nullptr;                // device: work items + offsets of the current launch
  int64_t items_cap = 0;
  uint32_t* group_counters = nullptr;      // device [3 x B x blocks]
  int64_t counters_cap = 0;
  std::vector<int32_t> items_host, block_layer;
  std::vector<int64_t> ipad_host;
  Workspace* no_ws = nullptr;              // what the per-branch layers share in grouped mode: sizes only, no memory
};

}  // namespace

struct mlpmoe_layer_s {
  int device = 0, num_sms = 0;
  int64_t d = 0, I = 0, Ipad_max = 0, max_tokens = 0;
  int B = 0;
  mlpmoe_dtype_t dtype = MLPMOE_BF16;
  int elem_size = 2;
  std::vector<int64_t> d_b, offs;
  std::vector<float> alpha_create, alpha_eff;
  void *Wg_c = nullptr, *Wu_c = nullptr, *Wd_c = nullptr;   // canonical copies, [I x d] each (neuron-major)
  void *Wgu = nullptr, *WdT = nullptr;                      // packed operands
  float* scale = nullptr;                                   // [Ipad_max]
  int32_t* src_row = nullptr;                               // [I] compacted neuron -> original neuron
  int32_t* row_nnz = nullptr;                               // [3 I]
  std::vector<int32_t> row_nnz_host;
  Schedule sched;
  int64_t Ipad = 0;
  Workspace* ws = nullptr;
  void* fade_work = nullptr;
  float* partial = nullptr;
  DecodeStackLayer* stack_dev = nullptr;                    // layer records of the persistent decode-stack kernel
  uint32_t* stack_counter = nullptr;                        // its grid-wide event counter
  std::vector<DecodeStackLayer> stack_host;                 // what stack_dev currently holds
  void* dec_tiled = nullptr;                                // stage-tiled weight copy of the fused few-token decode kernel,
  int64_t dec_tiled_version = -1;                           //   built at the first such call after a (re)schedule
  // persistent prefill-stack kernel (buffers live in the first layer's handle, sized at the first call
  // with a new stack / token count)
  TcStackLayer* pstack_dev = nullptr;
  int32_t* pstack_items = nullptr;                          // work items, then the per-pair offsets
  uint32_t* pstack_counters = nullptr;
  int64_t pstack_layer_cap = 0, pstack_item_cap = 0, pstack_counter_cap = 0, pstack_n_items = 0;
  int pstack_bn = 0;
  int64_t version = 0;                                      // bumped by every reschedule
  int64_t uid = 0;                                          // process-wide, never reused (a freed handle's address can be)
  Routed* routed = nullptr;                                 // built by the first mlpmoe_forward_routed
  // what the last mlpmoe_stack_prepare / first mlpmoe_stack_forward set up for a stack that starts with this layer
  std::vector<int64_t> plan_key;
  int plan_kind = 0;                                        // PLAN_*
  bool plan_fused = false;                                  // decode: the few-token kernel
  int plan_npad = 0;
  CUtensorMap plan_tm_x;                                    // normalised rows [n x d] as the kernels' token operand
  WaitCfg wait;                                             // bounded-wait limits of this handle's launches (test hook)
  int decode_kernel = 0;                                    // test hook: 0 = by rule, 1 = few-token kernel, 2 = the 14..64-token kernel
  // fast fp32 mode (fp32 layers): three-way bf16 splits of the packed operands and of the activations
  bool fast32 = false;
  int64_t dp = 0;                                           // d rounded up to the 64-wide K-step
  void *Wgu3 = nullptr, *WdT3 = nullptr;                    // [2 Ipad_max x 3 dp], [d x 3 Ipad_max] bf16
  void *X3 = nullptr, *H3 = nullptr;                        // [max_tokens x 3 dp], [max_tokens x 3 Ipad_max] bf16
  uint32_t* counters = nullptr;
  uint32_t* block_done = nullptr;                           // [2 x ceil(max_tokens / 256)] gate|up completion counters
  int64_t max_blocks = 0;
  int32_t* tile_sched = nullptr;                            // device: tile sequences + offsets of the fused prefill kernel
  int64_t sched_capacity = 0, sched_n = -1, sched_Ipad = -1;
  int sched_bn = 0, sched_ksplit = 0, sched_tiles = 0, sched_out_mode = -1;
  std::vector<int32_t> sched_host;
  int max_splits = 1;
  uint32_t* status = nullptr;
  int64_t launches = 0;
  CUtensorMap tm_wgu, tm_wdt;      // single-CTA boxes: 64 x 256 and 64 x 128
  CUtensorMap tm_wdt256;           // WdT with box 64 x 256 (decode-stack kernel)
  CUtensorMap tm_wgu_pair;         // CTA-pair box: 64 x 128
  // optional per-kernel event timing
  bool timing = false;
  std::vector<cudaEvent_t> events;
  size_t events_used = 0;
  struct Span { int kind; size_t a, b; };
  std::vector<Span> spans;
};

namespace {

constexpr size_t kEventPool = 2048;
constexpr size_t kStatusBytes = 64;        // status word, then (at byte 16) the clock probe of the last persistent-kernel launch
constexpr int kMaxStackLayers = 256;       // layers one persistent decode-stack launch can take
enum { SPAN_GATEUP = 0, SPAN_DOWN = 1, SPAN_RMSNORM = 2 };

// Records an event on `st` and returns its index in the pool, or -1 when timing is off / the pool is used up.
long rec_event(mlpmoe_layer_s* h, cudaStream_t st) {
  if (!h->timing || h->events_used >= h->events.size()) return -1;
  if (cudaEventRecord(h->events[h->events_used], st) != cudaSuccess) return -1;
  return static_cast<long>(h->events_used++);
}
void add_span(mlpmoe_layer_s* h, int kind, long a, long b) {
  if (a >= 0 && b >= 0) h->spans.push_back({kind, static_cast<size_t>(a), static_cast<size_t>(b)});
}

void free_layer(mlpmoe_layer_s* h);
void free_routed(Routed* r) {
  if (!r) return;
  for (mlpmoe_layer_s* c : r->child) free_layer(c);
  cudaFree(r->avail); cudaFree(r->pos); cudaFree(r->lists); cudaFree(r->counts); cudaFree(r->rowbase); cudaFree(r->coef);
  cudaFree(r->Xe); cudaFree(r->Ye); cudaFree(r->recs); cudaFree(r->Hg); cudaFree(r->items); cudaFree(r->group_counters);
  ws_release(r->no_ws);
  delete r;
}

void free_layer(mlpmoe_layer_s* h) {
  if (!h) return;
  free_routed(h->routed);
  for (cudaEvent_t e : h->events) cudaEventDestroy(e);
  cudaFree(h->Wg_c); cudaFree(h->Wu_c); cudaFree(h->Wd_c);
  cudaFree(h->Wgu); cudaFree(h->WdT);
  cudaFree(h->scale); cudaFree(h->src_row); cudaFree(h->row_nnz);
  cudaFree(h->fade_work); cudaFree(h->partial); cudaFree(h->counters); cudaFree(h->block_done); cudaFree(h->tile_sched); cudaFree(h->stack_dev); cudaFree(h->stack_counter); cudaFree(h->status);
  cudaFree(h->pstack_dev); cudaFree(h->pstack_items); cudaFree(h->pstack_counters); cudaFree(h->dec_tiled);
  cudaFree(h->Wgu3); cudaFree(h->WdT3); cudaFree(h->X3); cudaFree(h->H3);
  ws_release(h->ws);
  delete h;
}

// Fast fp32 mode: the three-way bf16 splits of the current packed operands.
mlpmoe_status_t refresh_fast32(mlpmoe_layer_s* h, cudaStream_t st) {
  CK(launch_split3(static_cast<const float*>(h->Wgu), h->Wgu3, 2 * h->Ipad, h->d, h->dp, h->d, st));
  CK(launch_split3(static_cast<const float*>(h->WdT), h->WdT3, h->d, h->Ipad, h->Ipad, h->Ipad, st));
  return MLPMOE_OK;
}

// Recompute liveness, the K-list, the per-neuron scale and the packed operands from the
// canonical weights and the effective gates.  Synchronises `st`.
mlpmoe_status_t reschedule(mlpmoe_layer_s* h, cudaStream_t st) {
  h->version += 1;
  CK(launch_row_nnz(h->Wg_c, h->Wu_c, h->Wd_c, h->row_nnz, h->I, h->d, h->elem_size, st));
  h->row_nnz_host.resize(3 * h->I);
  CK(cudaMemcpyAsync(h->row_nnz_host.data(), h->row_nnz, sizeof(int32_t) * 3 * h->I, cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  std::vector<uint8_t> live(h->I);
  for (int64_t j = 0; j < h->I; ++j)
    live[j] = (h->row_nnz_host[j] > 0 && h->row_nnz_host[h->I + j] > 0 && h->row_nnz_host[2 * h->I + j] > 0) ? 1 : 0;
  build_schedule(h->B, h->d_b.data(), h->alpha_eff.data(), live.data(), &h->sched);
  const int64_t n_active = h->sched.n_active;
  h->Ipad = round_up(n_active > 0 ? n_active : 1, kGroup);

  std::vector<int32_t> src(static_cast<size_t>(n_active > 0 ? n_active : 1));
  std::vector<float> scale(static_cast<size_t>(h->Ipad), 0.0f);
  int64_t jj = 0;
  int b = 0;
  for (size_t sgi = 0; sgi < h->sched.seg_start.size(); ++sgi) {
    const int64_t s0 = h->sched.seg_start[sgi], len = h->sched.seg_len[sgi];
    while (h->offs[b + 1] <= s0) ++b;
    for (int64_t j = s0; j < s0 + len; ++j, ++jj) {
      src[jj] = static_cast<int32_t>(j);
      scale[jj] = h->alpha_eff[b];
    }
  }
  if (n_active > 0) CK(cudaMemcpyAsync(h->src_row, src.data(), sizeof(int32_t) * n_active, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(h->scale, scale.data(), sizeof(float) * h->Ipad, cudaMemcpyHostToDevice, st));
  CK(launch_gather_gateup(h->Wg_c, h->Wu_c, h->src_row, h->Wgu, n_active, h->Ipad, h->d, h->elem_size, st));
  CK(launch_gather_down_t(h->Wd_c, h->src_row, h->WdT, n_active, h->Ipad, h->d, h->elem_size, st));
  CK(cudaStreamSynchronize(st));    // the host vectors above go out of scope
  if (h->fast32) {
    mlpmoe_status_t fs = refresh_fast32(h, st);
    if (fs != MLPMOE_OK) return fs;
  }
  if (h->dtype == MLPMOE_BF16) {
    if (!make_tmap(&h->tm_wgu, h->Wgu, h->d, 2 * h->Ipad, h->d, 256)) return MLPMOE_ERR_CUDA;
    if (!make_tmap(&h->tm_wdt, h->WdT, h->Ipad, h->d, h->Ipad, 128)) return MLPMOE_ERR_CUDA;
    if (!make_tmap(&h->tm_wdt256, h->WdT, h->Ipad, h->d, h->Ipad, 256)) return MLPMOE_ERR_CUDA;
    if (!make_tmap(&h->tm_wgu_pair, h->Wgu, h->d, 2 * h->Ipad, h->d, 128)) return MLPMOE_ERR_CUDA;
  }
  return MLPMOE_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The tile sequences of the fused prefill kernel for n tokens: chosen and uploaded (host work and one
// asynchronous copy into a buffer sized at create) at the first call with this token count / output
// mode since the last reschedule.
mlpmoe_status_t ensure_tile_schedule(mlpmoe_layer_s* h, int64_t n, int bn, int out_mode, cudaStream_t st) {
  if (h->sched_n == n && h->sched_Ipad == h->Ipad && h->sched_bn == bn && h->sched_out_mode == out_mode) return MLPMOE_OK;
  const int ksplit = tc_layer_ksplit(n, h->d, h->Ipad, bn, out_mode, h->num_sms);
  std::vector<int32_t> tiles, offs;
  tc_layer_schedule(n, h->d, h->Ipad, bn, ksplit, h->num_sms, &tiles, &offs);
  if (static_cast<int64_t>(tiles.size() + offs.size()) > h->sched_capacity) return MLPMOE_ERR_UNSUPPORTED;
  h->sched_host = tiles;
  h->sched_host.insert(h->sched_host.end(), offs.begin(), offs.end());
  h->sched_tiles = static_cast<int>(tiles.size());
  CK(cudaMemcpyAsync(h->tile_sched, h->sched_host.data(), sizeof(int32_t) * h->sched_host.size(), cudaMemcpyHostToDevice, st));
  h->sched_n = n; h->sched_Ipad = h->Ipad; h->sched_bn = bn; h->sched_ksplit = ksplit; h->sched_out_mode = out_mode;
  return MLPMOE_OK;
}

mlpmoe_status_t forward_impl(mlpmoe_layer_s* h, const void* x, void* y, int64_t n, const float* residual,
                             mlpmoe_dtype_t y_dtype, cudaStream_t st) {
  if (!h || n < 0) return MLPMOE_ERR_INVALID_ARG;
  if (n == 0) return MLPMOE_OK;
  if (!x || !y || n > h->max_tokens || !aligned16(x) || !aligned16(y) || (residual && !aligned16(residual)))
    return MLPMOE_ERR_INVALID_ARG;
  pdl_overlap_enabled() = !h->timing;
  if (y_dtype != MLPMOE_FP32 && !(y_dtype == MLPMOE_BF16 && h->dtype == MLPMOE_BF16)) return MLPMOE_ERR_UNSUPPORTED;
  if (h->dtype == MLPMOE_FP32 && h->fast32 && n > kDecodeMaxTokens) {
    // tensor-core path: every product of the two GEMMs as six bf16 piece products with fp32 accumulation
    TcGateUpArgs g;
    TcDownArgs dn;
    CK(launch_split3(static_cast<const float*>(x), h->X3, n, h->d, h->dp, h->d, st));
    if (!make_tmap(&g.tm_x, h->X3, 3 * h->dp, n, 3 * h->dp, 128)) return MLPMOE_ERR_CUDA;
    if (!make_tmap(&g.tm_w, h->Wgu3, 3 * h->dp, 2 * h->Ipad, 3 * h->dp, 256)) return MLPMOE_ERR_CUDA;
    g.scale = h->scale;
    g.H = h->H3;
    g.n = n; g.d = h->d; g.Ipad = h->Ipad;
    g.status = h->status;
    g.split3 = 1;
    if (!make_tmap(&dn.tm_h, h->H3, 3 * h->Ipad, n, 3 * h->Ipad, 128)) return MLPMOE_ERR_CUDA;
    if (!make_tmap(&dn.tm_w, h->WdT3, 3 * h->Ipad, h->d, 3 * h->Ipad, 128)) return MLPMOE_ERR_CUDA;
    dn.R = residual;
    dn.Y = y;
    dn.y_bf16 = 0;
    dn.n = n; dn.d = h->d; dn.Ipad = h->Ipad;
    dn.status = h->status;
    dn.split3 = 1;
    const long e0 = rec_event(h, st);
    CK(launch_tc_gateup(g, h->num_sms, st));
    const long e1 = rec_event(h, st);
    CK(launch_tc_down(dn, h->num_sms, st));
    const long e2 = rec_event(h, st);
    add_span(h, SPAN_GATEUP, e0, e1);
    add_span(h, SPAN_DOWN, e1, e2);
    h->launches += 3;
    return MLPMOE_OK;
  }
  if (h->dtype == MLPMOE_FP32) {
    float* H = static_cast<float*>(h->ws->H);
    const long e0 = rec_event(h, st);
    CK(launch_simt_gateup(static_cast<const float*>(x), static_cast<const float*>(h->Wgu), h->scale, H, n, h->d, h->Ipad, st));
    const long e1 = rec_event(h, st);
    CK(launch_simt_down(H, static_cast<const float*>(h->WdT), residual, static_cast<float*>(y), n, h->d, h->Ipad, st));
    const long e2 = rec_event(h, st);
    add_span(h, SPAN_GATEUP, e0, e1);
    add_span(h, SPAN_DOWN, e1, e2);
    h->launches += 2;
    return MLPMOE_OK;
  }
  if (n <= kDecodeMaxTokens) {
    DecodeArgs a;
    a.npad = n <= 16 ? 16 : (n <= 32 ? 32 : 64);
    a.tm_w = h->tm_wgu;
    a.tm_wd = h->tm_wdt;
    if (!make_tmap(&a.tm_x, x, h->d, n, h->d, a.npad)) return MLPMOE_ERR_CUDA;
    if (!make_tmap(&a.tm_h, h->ws->H, h->Ipad, n, h->Ipad, a.npad)) return MLPMOE_ERR_CUDA;
    a.scale = h->scale;
    a.Hd = h->ws->H;
    a.partial = h->partial;
    a.counters = h->counters;
    a.R = residual;
    a.Y = y;
    a.y_bf16 = y_dtype == MLPMOE_BF16;
    a.n = n; a.d = h->d; a.Ipad = h->Ipad;
    const int m_blocks = static_cast<int>((h->d + 127) / 128);
    a.accumulate = (residual == y && y_dtype == MLPMOE_FP32) ? 1 : 0;
    // accumulate mode needs no staging buffer, so it can cut K finer (two work items per SM)
    int splits = (a.accumulate ? 2 * h->num_sms : h->num_sms) / m_blocks;
    if (!a.accumulate && splits > h->max_splits) splits = h->max_splits;
    if (splits > h->Ipad / 64 / 8) splits = static_cast<int>(h->Ipad / 64 / 8);
    if (splits < 1) splits = 1;
    a.splits = splits;
    a.status = h->status;
    const long e0 = rec_event(h, st);
    CK(launch_decode_gateup(a, h->num_sms, st));
    const long e1 = rec_event(h, st);
    CK(launch_decode_down(a, h->num_sms, st));
    const long e2 = rec_event(h, st);
    add_span(h, SPAN_GATEUP, e0, e1);
    add_span(h, SPAN_DOWN, e1, e2);
    h->launches += 2;
    return MLPMOE_OK;
  }
  if (n > 128) {
    // one fused CTA-pair kernel: gate|up tiles, then down tiles
    TcLayerArgs a;
    a.bn = tc_layer_down_bn(n, h->d, h->num_sms);
    if (!make_tmap(&a.tm_x, x, h->d, n, h->d, 128)) return MLPMOE_ERR_CUDA;
    a.tm_wgu = h->tm_wgu_pair;
    if (!make_tmap(&a.tm_h_st, h->ws->H, h->Ipad, n, h->Ipad, 32)) return MLPMOE_ERR_CUDA;
    if (!make_tmap(&a.tm_h_ld, h->ws->H, h->Ipad, n, h->Ipad, 128)) return MLPMOE_ERR_CUDA;
    if (!make_tmap(&a.tm_wdt, h->WdT, h->Ipad, h->d, h->Ipad, a.bn / 2)) return MLPMOE_ERR_CUDA;
    a.out_mode = TcLayerArgs::OUT_DIRECT;
    if (y_dtype == MLPMOE_FP32 && residual == nullptr) a.out_mode = TcLayerArgs::OUT_TMA_STORE;
    else if (y_dtype == MLPMOE_FP32 && residual == y) a.out_mode = TcLayerArgs::OUT_TMA_ADD;
    if (a.out_mode != TcLayerArgs::OUT_DIRECT) {
      if (!make_tmap_t(&a.tm_y, y, h->d, n, h->d, 32, 4)) return MLPMOE_ERR_CUDA;
    } else {
      a.tm_y = a.tm_h_st;       // not used by the direct epilogue; any valid map
    }
    a.scale = h->scale;
    a.R = residual;
    a.Y = y;
    a.y_bf16 = y_dtype == MLPMOE_BF16;
    a.n = n; a.d = h->d; a.Ipad = h->Ipad;
    mlpmoe_status_t src = ensure_tile_schedule(h, n, a.bn, a.out_mode, st);
    if (src != MLPMOE_OK) return src;
    a.ksplit = h->sched_ksplit;
    a.tile_list = h->tile_sched;
    a.list_offsets = h->tile_sched + h->sched_tiles;
    a.done = h->block_done;
    a.passed = h->block_done + h->max_blocks;
    a.status = h->status;
    a.wait = h->wait;
    const long e0 = rec_event(h, st);
    CK(launch_tc_layer(a, h->num_sms, st));
    const long e1 = rec_event(h, st);
    add_span(h, SPAN_GATEUP, e0, e1);      // the fused kernel is reported in the first slot
    h->launches += 1;
    return MLPMOE_OK;
  }
  // 65..128 tokens: one CTA per tile, two kernels
  TcGateUpArgs g;
  if (!make_tmap(&g.tm_x, x, h->d, n, h->d, 128)) return MLPMOE_ERR_CUDA;
  g.tm_w = h->tm_wgu;
  g.scale = h->scale;
  g.H = h->ws->H;
  g.n = n; g.d = h->d; g.Ipad = h->Ipad;
  g.status = h->status;
  TcDownArgs dn;
  if (!make_tmap(&dn.tm_h, h->ws->H, h->Ipad, n, h->Ipad, 128)) return MLPMOE_ERR_CUDA;
  dn.tm_w = h->tm_wdt;
  dn.R = residual;
  dn.Y = y;
  dn.y_bf16 = y_dtype == MLPMOE_BF16;
  dn.n = n; dn.d = h->d; dn.Ipad = h->Ipad;
  dn.status = h->status;
  const long e0 = rec_event(h, st);
  CK(launch_tc_gateup(g, h->num_sms, st));
  const long e1 = rec_event(h, st);
  CK(launch_tc_down(dn, h->num_sms, st));
  const long e2 = rec_event(h, st);
  add_span(h, SPAN_GATEUP, e0, e1);
  add_span(h, SPAN_DOWN, e1, e2);
  h->launches += 2;
  return MLPMOE_OK;
}

// The persistent decode-stack kernel needs one CTA of it to fit on every SM (checked once).
bool stack_kernel_ok() {
  static int state = -1;
  if (state < 0) {
    int per_sm = 0;
    int per_sm_fused = 0;
    state = (decode_stack_init(&per_sm) == cudaSuccess && per_sm >= 1 && decode_fused_init(&per_sm_fused) == cudaSuccess &&
             per_sm_fused >= 1) ? 1 : 0;
  }
  return state == 1;
}

mlpmoe_status_t check_stack(const mlpmoe_handle_t* layers, int32_t n_layers, int64_t n) {
  if (!layers || n_layers <= 0 || n < 0) return MLPMOE_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l) {
    if (!layers[l]) return MLPMOE_ERR_INVALID_ARG;
    if (layers[l]->d != layers[0]->d || layers[l]->dtype != layers[0]->dtype) return MLPMOE_ERR_INVALID_ARG;
    if (n > layers[l]->max_tokens) return MLPMOE_ERR_INVALID_ARG;
  }
  return MLPMOE_OK;
}

enum { PLAN_NONE = 0, PLAN_DECODE = 1, PLAN_PREFILL_STACK = 2, PLAN_PER_LAYER = 3 };

// What a stack call's set-up depends on: the token count, the shared workspace, and every layer's identity
// (a process-wide id, never reused) and schedule version.
std::vector<int64_t> stack_key(const mlpmoe_handle_t* layers, int32_t n_layers, int64_t n) {
  std::vector<int64_t> key;
  key.reserve(4 + 2 * static_cast<size_t>(n_layers));
  key.push_back(n);
  key.push_back(n_layers);
  key.push_back(reinterpret_cast<int64_t>(layers[0]->ws->H));
  key.push_back(reinterpret_cast<int64_t>(layers[0]->ws->xnorm));
  for (int l = 0; l < n_layers; ++l) {
    key.push_back(layers[l]->uid);
    key.push_back(layers[l]->version);
  }
  return key;
}

// Set-up of the persistent decode kernels for this stack and token count: the stage-tiled weight copies
// (allocated at the first decode set-up of a layer, rebuilt after a reschedule), the layer records and
// the token operand's tensor map.
mlpmoe_status_t plan_decode(const mlpmoe_handle_t* layers, int32_t n_layers, int64_t n, cudaStream_t st) {
  mlpmoe_layer_s* h0 = layers[0];
  const int npad = n <= 16 ? 16 : (n <= 32 ? 32 : (n <= 64 ? 64 : 128));
  bool tiled = true;
  for (int l = 0; tiled && l < n_layers; ++l) {
    mlpmoe_layer_s* h = layers[l];
    if (h->dec_tiled != nullptr && h->dec_tiled_version == h->version) continue;
    if (h->dec_tiled == nullptr && cudaMalloc(&h->dec_tiled, decode_tiled_bytes(h->Ipad_max, h->d)) != cudaSuccess) {
      cudaGetLastError();
      h->dec_tiled = nullptr;
      tiled = false;          // without memory for the copy the 14..64-token kernel reads the packed operands through tensor maps
      break;
    }
    CK(launch_retile_decode(h->Wgu, h->WdT, h->dec_tiled, h->Ipad, h->d, st));
    h->dec_tiled_version = h->version;
  }
  h0->stack_host.assign(static_cast<size_t>(n_layers), DecodeStackLayer());
  std::memset(h0->stack_host.data(), 0, sizeof(DecodeStackLayer) * h0->stack_host.size());
  for (int l = 0; l < n_layers; ++l) {
    mlpmoe_layer_s* h = layers[l];
    DecodeStackLayer& r = h0->stack_host[l];
    r.tm_wgu = h->tm_wgu;
    r.tm_wdt = h->tm_wdt256;
    if (!make_tmap(&r.tm_hd, h->ws->H, h->Ipad, n, h->Ipad, npad)) return MLPMOE_ERR_CUDA;
    r.scale = h->scale;
    r.Hd = static_cast<__nv_bfloat16*>(h->ws->H);
    r.tiled = tiled ? static_cast<const uint8_t*>(h->dec_tiled) : nullptr;
    r.Ipad = static_cast<int32_t>(h->Ipad);
  }
  CK(cudaMemcpyAsync(h0->stack_dev, h0->stack_host.data(), sizeof(DecodeStackLayer) * h0->stack_host.size(), cudaMemcpyHostToDevice, st));
  if (!make_tmap(&h0->plan_tm_x, h0->ws->xnorm, h0->d, n, h0->d, npad)) return MLPMOE_ERR_CUDA;
  // Which of the two decode kernels: the few-token kernel keeps both GEMMs of a neuron tile on the tile's owner, so with
  // few tiles (pruned stacks) few SMs do all the work, while the other kernel spreads its down phase over all SMs.
  // Measured crossovers on 4096 x 14336 layers (tiles per layer over SMs: tokens up to which the few-token kernel wins):
  // 112/148: 13, 102/148: 12, 90/148 and 70/148: 7, 56/148 and below: none.
  int64_t tiles = 0;
  for (int l = 0; l < n_layers; ++l) tiles += layers[l]->Ipad / 128;
  const double owners = static_cast<double>(tiles) / n_layers / h0->num_sms;
  int fused_max = owners > 0.71 ? kDecodeFusedMaxTokens : (owners > 0.64 ? 12 : (owners > 0.38 ? 7 : 0));
  if (h0->decode_kernel == 1) fused_max = 16;              // the few-token kernel holds 16 token rows
  if (h0->decode_kernel == 2) fused_max = 0;
  h0->plan_fused = tiled && n <= fused_max;
  h0->plan_npad = npad;
  return MLPMOE_OK;
}

// Set-up of the persistent prefill-stack kernel: the work sequences (host), the layer records, and the
// device buffers that hold them (re-allocated when they are too small, which synchronises `st`).
mlpmoe_status_t plan_prefill_stack(const mlpmoe_handle_t* layers, int32_t n_layers, int64_t n, cudaStream_t st) {
  mlpmoe_layer_s* h0 = layers[0];
  const int64_t d = h0->d;
  const int bn = tc_layer_down_bn(n, d, h0->num_sms);
  const int64_t m_pairs = (n + 255) / 256;
  std::vector<TcStackLayer> recs(static_cast<size_t>(n_layers));
  std::memset(recs.data(), 0, sizeof(TcStackLayer) * recs.size());
  std::vector<int64_t> Ipad(n_layers);
  std::vector<int> ksplit(n_layers);
  for (int l = 0; l < n_layers; ++l) {
    mlpmoe_layer_s* h = layers[l];
    Ipad[l] = h->Ipad;
    ksplit[l] = tc_layer_ksplit(n, d, h->Ipad, bn, TcLayerArgs::OUT_TMA_ADD, h0->num_sms);
    recs[l].tm_wgu = h->tm_wgu_pair;
    if (!make_tmap(&recs[l].tm_h_st, h->ws->H, h->Ipad, n, h->Ipad, 32)) return MLPMOE_ERR_CUDA;
    if (!make_tmap(&recs[l].tm_h_ld, h->ws->H, h->Ipad, n, h->Ipad, 128)) return MLPMOE_ERR_CUDA;
    if (!make_tmap(&recs[l].tm_wdt, h->WdT, h->Ipad, d, h->Ipad, bn / 2)) return MLPMOE_ERR_CUDA;
    recs[l].scale = h->scale;
    recs[l].n1 = static_cast<int32_t>(h->Ipad / 128);
    recs[l].kb2 = static_cast<int32_t>(h->Ipad / 64);
    recs[l].ksplit = ksplit[l];
  }
  std::vector<int32_t> items, offs;
  tc_stack_schedule(n, d, Ipad.data(), ksplit.data(), n_layers, bn, h0->num_sms, &items, &offs);
  const int64_t need_items = static_cast<int64_t>(items.size() + offs.size());
  const int64_t need_counters = 3 * static_cast<int64_t>(n_layers) * m_pairs;
  if (need_items > h0->pstack_item_cap || need_counters > h0->pstack_counter_cap || n_layers > h0->pstack_layer_cap) {
    CK(cudaStreamSynchronize(st));     // earlier launches may still read the old buffers
    cudaFree(h0->pstack_items); cudaFree(h0->pstack_counters); cudaFree(h0->pstack_dev);
    h0->pstack_items = nullptr; h0->pstack_counters = nullptr; h0->pstack_dev = nullptr;
    h0->pstack_item_cap = h0->pstack_counter_cap = h0->pstack_layer_cap = 0;
    if (cudaMalloc(reinterpret_cast<void**>(&h0->pstack_items), sizeof(int32_t) * need_items) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&h0->pstack_counters), sizeof(uint32_t) * need_counters) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&h0->pstack_dev), sizeof(TcStackLayer) * n_layers) != cudaSuccess) {
      cudaGetLastError();
      return MLPMOE_ERR_ALLOC;
    }
    h0->pstack_item_cap = need_items; h0->pstack_counter_cap = need_counters; h0->pstack_layer_cap = n_layers;
  }
  items.insert(items.end(), offs.begin(), offs.end());
  h0->pstack_n_items = static_cast<int64_t>(items.size() - offs.size());
  CK(cudaMemcpyAsync(h0->pstack_items, items.data(), sizeof(int32_t) * items.size(), cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(h0->pstack_dev, recs.data(), sizeof(TcStackLayer) * recs.size(), cudaMemcpyHostToDevice, st));
  CK(cudaStreamSynchronize(st));       // the host vectors above go out of scope
  if (!make_tmap(&h0->plan_tm_x, h0->ws->xnorm, d, n, d, 128)) return MLPMOE_ERR_CUDA;
  h0->pstack_bn = bn;
  return MLPMOE_OK;
}

// Which kernel family runs this stack call, and its set-up.  Cached in the first layer's handle under
// stack_key(); a call with another stack, token count, workspace or schedule version plans again.
mlpmoe_status_t plan_stack(const mlpmoe_handle_t* layers, int32_t n_layers, int64_t n, cudaStream_t st) {
  mlpmoe_layer_s* h0 = layers[0];
  std::vector<int64_t> key = stack_key(layers, n_layers, n);
  if (h0->plan_kind != PLAN_NONE && key == h0->plan_key) return MLPMOE_OK;
  h0->plan_kind = PLAN_NONE;
  h0->plan_key.clear();
  int kind = PLAN_PER_LAYER;
  if (h0->dtype == MLPMOE_BF16 && n <= kDecodeStackMaxTokens && n_layers <= kMaxStackLayers && h0->d <= 32768 && stack_kernel_ok()) {
    // decode: the whole stack in one persistent kernel (weights keep streaming across layer boundaries)
    kind = PLAN_DECODE;
  } else if (h0->dtype == MLPMOE_BF16 && n > 128 && n_layers <= kMaxStackLayers) {
    // The one-launch stack kernel pays where layers are short (weights that stay in L2: its gain is
    // what a layer boundary costs); long layers run faster one launch per layer, on the cost-aware
    // tile schedule of the single-layer kernel (measured on 4096 x 14336 layers).
    bool use_stack = true;
    for (int l = 0; l < n_layers; ++l)
      use_stack = use_stack && layers[l]->ws == h0->ws && 3 * layers[l]->d * layers[l]->Ipad * 2 <= kWeightsFitL2Bytes;
    if (use_stack) kind = PLAN_PREFILL_STACK;
  }
  mlpmoe_status_t rc = MLPMOE_OK;
  if (kind == PLAN_DECODE) {
    rc = plan_decode(layers, n_layers, n, st);
  } else if (kind == PLAN_PREFILL_STACK) {
    rc = plan_prefill_stack(layers, n_layers, n, st);
  } else if (h0->dtype == MLPMOE_BF16 && n > 128) {
    // one fused-kernel launch per layer: choose and upload every layer's tile sequences now
    for (int l = 0; rc == MLPMOE_OK && l < n_layers; ++l)
      rc = ensure_tile_schedule(layers[l], n, tc_layer_down_bn(n, layers[l]->d, layers[l]->num_sms), TcLayerArgs::OUT_TMA_ADD, st);
  }
  if (rc != MLPMOE_OK) return rc;
  h0->plan_kind = kind;
  h0->plan_key = std::move(key);
  return MLPMOE_OK;
}

mlpmoe_status_t run_decode_stack(const mlpmoe_handle_t* layers, int32_t n_layers, float* x, int64_t n, float eps, cudaStream_t st) {
  mlpmoe_layer_s* h0 = layers[0];
  CK(cudaMemsetAsync(h0->stack_counter, 0, sizeof(uint32_t) * 3 * n_layers, st));
  const long e0 = rec_event(h0, st);
  if (h0->plan_fused) {
    // both GEMMs of a layer on the CTA that owns the neurons (no H round trip, one dependency less per layer)
    CK(launch_decode_fused(h0->stack_dev, n_layers, h0->plan_tm_x, x, h0->ws->xnorm, n, h0->d, eps, h0->stack_counter, h0->status,
                           h0->num_sms, h0->wait, st));
  } else {
    CK(launch_decode_stack(h0->stack_dev, n_layers, h0->plan_tm_x, x, h0->ws->xnorm, n, h0->d, h0->plan_npad, eps, h0->stack_counter,
                           h0->status, h0->num_sms, h0->wait, st));
  }
  const long e1 = rec_event(h0, st);
  add_span(h0, SPAN_GATEUP, e0, e1);
  h0->launches += 1;
  return MLPMOE_OK;
}

mlpmoe_status_t run_prefill_stack(const mlpmoe_handle_t* layers, int32_t n_layers, float* x, int64_t n, float eps, cudaStream_t st) {
  mlpmoe_layer_s* h0 = layers[0];
  const int64_t m_pairs = (n + 255) / 256;
  TcStackArgs a;
  a.layers = h0->pstack_dev;
  a.n_layers = n_layers;
  a.tm_x = h0->plan_tm_x;
  if (!make_tmap_t(&a.tm_y, x, h0->d, n, h0->d, 32, 4)) return MLPMOE_ERR_CUDA;     // x is the caller's: encoded per call
  a.x = x;
  a.xnorm = h0->ws->xnorm;
  a.n = n;
  a.d = h0->d;
  a.bn = h0->pstack_bn;
  a.eps = eps;
  a.items = h0->pstack_items;
  a.list_offsets = h0->pstack_items + h0->pstack_n_items;
  a.counters = h0->pstack_counters;
  a.status = h0->status;
  a.wait = h0->wait;
  pdl_overlap_enabled() = !h0->timing;
  CK(cudaMemsetAsync(h0->pstack_counters, 0, sizeof(uint32_t) * 3 * n_layers * m_pairs, st));
  const long e0 = rec_event(h0, st);
  CK(launch_tc_stack(a, h0->num_sms, st));
  const long e1 = rec_event(h0, st);
  add_span(h0, SPAN_GATEUP, e0, e1);       // the one kernel of the step is reported in the first slot
  h0->launches += 1;
  return MLPMOE_OK;
}

// Layer construction.  `layout` is one of the public layouts or kLayoutCanonical (all three matrices
// neuron-major, [d_inter x d_model]: what the handle keeps); with `share` the layer uses that
// workspace instead of allocating one (it must be large enough).
constexpr int kLayoutCanonical = 2;
mlpmoe_status_t create_impl(mlpmoe_handle_t* out, int64_t d_model, int64_t d_inter, int32_t B, const int64_t* d_b,
                            const void* W_gate, const void* W_up, const void* W_down, const float* alpha, mlpmoe_dtype_t dtype,
                            int layout, int64_t max_tokens, Workspace* share, cudaStream_t st) {
  if (!out) return MLPMOE_ERR_INVALID_ARG;
  *out = nullptr;
  if (d_model <= 0 || d_inter <= 0 || max_tokens <= 0 || !W_gate || !W_up || !W_down) return MLPMOE_ERR_INVALID_ARG;
  if (dtype != MLPMOE_BF16 && dtype != MLPMOE_FP32) return MLPMOE_ERR_INVALID_ARG;
  mlpmoe_status_t ps = check_partition(d_inter, B, d_b, 16);
  if (ps != MLPMOE_OK) return ps;
  if (d_model % 8 != 0) return MLPMOE_ERR_UNSUPPORTED;
  if (d_inter > (int64_t(1) << 30) || d_model > (int64_t(1) << 30)) return MLPMOE_ERR_UNSUPPORTED;
  int dev = 0;
  CK(cudaGetDevice(&dev));
  cudaDeviceProp prop;
  CK(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) return MLPMOE_ERR_UNSUPPORTED;     // kernels are built for sm_100a only
  CK(tc_gemm_init());
  CK(tc_layer_init());
  CK(tc_stack_init());
  CK(decode_init());

  mlpmoe_layer_s* h = new (std::nothrow) mlpmoe_layer_s();
  if (!h) return MLPMOE_ERR_ALLOC;
  static std::atomic<int64_t> next_uid{1};
  h->uid = next_uid.fetch_add(1);
  h->device = dev;
  h->num_sms = prop.multiProcessorCount;
  h->d = d_model;
  h->I = d_inter;
  h->B = B;
  h->dtype = dtype;
  h->elem_size = dtype == MLPMOE_BF16 ? 2 : 4;
  h->max_tokens = max_tokens;
  h->Ipad_max = round_up(d_inter, kGroup);
  h->d_b.assign(d_b, d_b + B);
  h->offs.resize(B + 1);
  h->offs[0] = 0;
  for (int b = 0; b < B; ++b) h->offs[b + 1] = h->offs[b] + d_b[b];
  h->alpha_create.resize(B);
  for (int b = 0; b < B; ++b) h->alpha_create[b] = alpha ? alpha[b] : 1.0f;
  h->alpha_eff = h->alpha_create;

  const size_t es = static_cast<size_t>(h->elem_size);
  const size_t mat = static_cast<size_t>(d_model) * d_inter * es;
  const int m_blocks = static_cast<int>((d_model + 127) / 128);
  h->max_splits = h->num_sms / m_blocks + 1;
  h->max_blocks = (max_tokens + 255) / 256;
  h->sched_capacity = h->max_blocks * (h->Ipad_max / 128 + 4 * ((d_model + 63) / 64)) + h->num_sms / 2 + 2;
  bool ok = true;
  if (share) {
    if (share->elem_size != h->elem_size || share->max_tokens < max_tokens || share->Ipad_max < h->Ipad_max || share->d < d_model) {
      delete h;
      return MLPMOE_ERR_INVALID_ARG;
    }
    h->ws = share;
    share->refs += 1;
  } else {
    h->ws = new (std::nothrow) Workspace();
    ok = h->ws != nullptr;
    if (ok) {
      h->ws->refs = 1;
      h->ws->max_tokens = max_tokens;
      h->ws->Ipad_max = h->Ipad_max;
      h->ws->d = d_model;
      h->ws->elem_size = h->elem_size;
    }
  }
  ok = ok && cudaMalloc(&h->Wg_c, mat) == cudaSuccess && cudaMalloc(&h->Wu_c, mat) == cudaSuccess &&
       cudaMalloc(&h->Wd_c, mat) == cudaSuccess &&
       cudaMalloc(&h->Wgu, static_cast<size_t>(2 * h->Ipad_max) * d_model * es) == cudaSuccess &&
       cudaMalloc(&h->WdT, static_cast<size_t>(h->Ipad_max) * d_model * es) == cudaSuccess &&
       cudaMalloc(&h->scale, sizeof(float) * h->Ipad_max) == cudaSuccess &&
       cudaMalloc(&h->src_row, sizeof(int32_t) * d_inter) == cudaSuccess &&
       cudaMalloc(&h->row_nnz, sizeof(int32_t) * 3 * d_inter) == cudaSuccess &&
       cudaMalloc(&h->fade_work, fade_work_bytes(2 * B)) == cudaSuccess &&
       cudaMalloc(&h->partial, sizeof(float) * static_cast<size_t>(h->max_splits) * d_model * kDecodeMaxTokens) == cudaSuccess &&
       cudaMalloc(&h->counters, sizeof(uint32_t) * m_blocks * 4) == cudaSuccess &&
       cudaMalloc(reinterpret_cast<void**>(&h->stack_dev), sizeof(DecodeStackLayer) * kMaxStackLayers) == cudaSuccess &&
       cudaMalloc(reinterpret_cast<void**>(&h->stack_counter), sizeof(uint32_t) * 3 * kMaxStackLayers) == cudaSuccess &&
       cudaMalloc(&h->block_done, sizeof(uint32_t) * 2 * h->max_blocks) == cudaSuccess &&
       cudaMalloc(&h->tile_sched, sizeof(int32_t) * h->sched_capacity) == cudaSuccess &&
       cudaMalloc(&h->status, kStatusBytes) == cudaSuccess;
  if (ok && !share)
    ok = cudaMalloc(&h->ws->H, static_cast<size_t>(max_tokens) * h->Ipad_max * es) == cudaSuccess &&
         cudaMalloc(&h->ws->xnorm, static_cast<size_t>(max_tokens) * d_model * es) == cudaSuccess &&
         cudaMalloc(reinterpret_cast<void**>(&h->ws->yres), static_cast<size_t>(max_tokens) * d_model * sizeof(float)) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    free_layer(h);
    return MLPMOE_ERR_ALLOC;
  }
  mlpmoe_status_t rc = MLPMOE_OK;
  auto fail = [&](mlpmoe_status_t s) { free_layer(h); return s; };
  if (cudaMemsetAsync(h->counters, 0, sizeof(uint32_t) * m_blocks * 4, st) != cudaSuccess ||
      cudaMemsetAsync(h->block_done, 0, sizeof(uint32_t) * 2 * h->max_blocks, st) != cudaSuccess ||
      cudaMemsetAsync(h->status, 0, kStatusBytes, st) != cudaSuccess)
    return fail(MLPMOE_ERR_CUDA);
  // canonical copies: one row of d contiguous weights per intermediate neuron, for all three matrices
  cudaError_t e;
  if (layout == kLayoutCanonical) {
    e = cudaMemcpyAsync(h->Wg_c, W_gate, mat, cudaMemcpyDeviceToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h->Wu_c, W_up, mat, cudaMemcpyDeviceToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h->Wd_c, W_down, mat, cudaMemcpyDeviceToDevice, st);
  } else if (layout == MLPMOE_LAYOUT_PAPER) {
    e = launch_transpose(W_gate, h->Wg_c, d_model, d_inter, h->elem_size, st);
    if (e == cudaSuccess) e = launch_transpose(W_up, h->Wu_c, d_model, d_inter, h->elem_size, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h->Wd_c, W_down, mat, cudaMemcpyDeviceToDevice, st);
  } else {
    e = cudaMemcpyAsync(h->Wg_c, W_gate, mat, cudaMemcpyDeviceToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h->Wu_c, W_up, mat, cudaMemcpyDeviceToDevice, st);
    if (e == cudaSuccess) e = launch_transpose(W_down, h->Wd_c, d_model, d_inter, h->elem_size, st);
  }
  if (e != cudaSuccess) return fail(MLPMOE_ERR_CUDA);
  rc = reschedule(h, st);
  if (rc != MLPMOE_OK) return fail(rc);
  *out = h;
  return MLPMOE_OK;
}

// The per-branch layers and buffers of mlpmoe_forward_routed, (re)built when the parent's weights or
// gates have changed since.  Allocates and synchronises `st`.
constexpr int64_t kRoutedPassBranches = 8;      // Ye holds max_tokens x min(B, this) rows; more selected rows take more passes
mlpmoe_status_t ensure_routed(mlpmoe_layer_s* h, cudaStream_t st) {
  if (h->routed && h->routed->version == h->version) return MLPMOE_OK;
  CK(cudaStreamSynchronize(st));           // earlier routed calls may still use what is replaced below
  if (!h->routed) {
    Routed* r = new (std::nothrow) Routed();
    if (!r) return MLPMOE_ERR_ALLOC;
    h->routed = r;
    r->child.assign(h->B, nullptr);
    r->grouped = h->dtype == MLPMOE_BF16 && h->B <= kMaxStackLayers;
    r->ye_rows = h->max_tokens * (h->B < kRoutedPassBranches ? h->B : kRoutedPassBranches);
    if (r->grouped) r->ye_rows = round_up(r->ye_rows, 256) + 256 * static_cast<int64_t>(h->B);   // every branch's rows start a 256-row block
    const size_t row = static_cast<size_t>(h->d) * h->elem_size;
    if (cudaMalloc(reinterpret_cast<void**>(&r->avail), h->B) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&r->pos), sizeof(int32_t) * h->max_tokens * h->B) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&r->lists), sizeof(int32_t) * h->max_tokens * h->B) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&r->counts), sizeof(int32_t) * h->B) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&r->rowbase), sizeof(int32_t) * h->B) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&r->coef), sizeof(float) * h->max_tokens) != cudaSuccess ||
        cudaMalloc(&r->Xe, row * (r->grouped ? r->ye_rows : h->max_tokens)) != cudaSuccess ||
        (r->grouped && cudaMalloc(reinterpret_cast<void**>(&r->recs), sizeof(TcStackLayer) * h->B) != cudaSuccess) ||
        cudaMalloc(&r->Ye, sizeof(float) * static_cast<size_t>(h->d) * r->ye_rows) != cudaSuccess) {
      cudaGetLastError();
      free_routed(r);
      h->routed = nullptr;
      return MLPMOE_ERR_ALLOC;
    }
  }
  Routed* r = h->routed;
  for (mlpmoe_layer_s*& c : r->child) { free_layer(c); c = nullptr; }
  r->version = -1;
  // widest branch first: its workspace serves all the others
  std::vector<int> order;
  for (int b = 0; b < h->B; ++b)
    if (h->alpha_eff[b] != 0.0f) order.push_back(b);
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return h->d_b[a] > h->d_b[b]; });
  r->n_avail = static_cast<int>(order.size());
  Workspace* ws = nullptr;
  if (r->grouped) {
    // the grouped launch has its own buffers (Xe, Hg, Ye): the per-branch layers get a workspace without memory
    if (!r->no_ws) {
      r->no_ws = new (std::nothrow) Workspace();
      if (!r->no_ws) return MLPMOE_ERR_ALLOC;
      r->no_ws->refs = 1;
      r->no_ws->max_tokens = h->max_tokens;
      r->no_ws->Ipad_max = h->Ipad_max;
      r->no_ws->d = h->d;
      r->no_ws->elem_size = h->elem_size;
    }
    ws = r->no_ws;
  }
  const size_t row = static_cast<size_t>(h->d) * h->elem_size;
  for (int b : order) {
    const size_t off = static_cast<size_t>(h->offs[b]) * row;
    const int64_t width = h->d_b[b];
    const float alpha = h->alpha_eff[b];
    mlpmoe_layer_s* c = nullptr;
    mlpmoe_status_t rc = create_impl(&c, h->d, width, 1, &width, static_cast<const char*>(h->Wg_c) + off,
                                     static_cast<const char*>(h->Wu_c) + off, static_cast<const char*>(h->Wd_c) + off, &alpha, h->dtype,
                                     kLayoutCanonical, h->max_tokens, ws, st);
    if (rc != MLPMOE_OK) return rc;
    // the child only ever runs forward: its canonical copies are not needed once the operands are packed
    CK(cudaStreamSynchronize(st));
    cudaFree(c->Wg_c); cudaFree(c->Wu_c); cudaFree(c->Wd_c);
    c->Wg_c = c->Wu_c = c->Wd_c = nullptr;
    c->wait = h->wait;
    r->child[b] = c;
    if (!ws) ws = c->ws;
  }
  if (r->grouped) {
    // one "layer" record per branch: its packed weights, and its columns of the shared H buffer
    int64_t pitch = kGroup;
    for (int b : order) pitch = std::max(pitch, r->child[b]->Ipad);
    if (pitch > r->h_pitch) {
      cudaFree(r->Hg);
      r->Hg = nullptr;
      r->h_pitch = 0;
      if (cudaMalloc(&r->Hg, sizeof(__nv_bfloat16) * static_cast<size_t>(r->ye_rows) * pitch) != cudaSuccess) {
        cudaGetLastError();
        return MLPMOE_ERR_ALLOC;
      }
      r->h_pitch = pitch;
    }
    r->bn = tc_layer_down_bn(r->ye_rows, h->d, h->num_sms);
    std::vector<TcStackLayer> recs(static_cast<size_t>(h->B));
    std::memset(recs.data(), 0, sizeof(TcStackLayer) * recs.size());
    r->ipad_host.assign(h->B, kGroup);
    for (int b : order) {
      mlpmoe_layer_s* c = r->child[b];
      recs[b].tm_wgu = c->tm_wgu_pair;
      if (!make_tmap(&recs[b].tm_h_st, r->Hg, c->Ipad, r->ye_rows, r->h_pitch, 32)) return MLPMOE_ERR_CUDA;
      if (!make_tmap(&recs[b].tm_h_ld, r->Hg, c->Ipad, r->ye_rows, r->h_pitch, 128)) return MLPMOE_ERR_CUDA;
      if (!make_tmap(&recs[b].tm_wdt, c->WdT, c->Ipad, h->d, c->Ipad, r->bn / 2)) return MLPMOE_ERR_CUDA;
      recs[b].scale = c->scale;
      recs[b].n1 = static_cast<int32_t>(c->Ipad / 128);
      recs[b].kb2 = static_cast<int32_t>(c->Ipad / 64);
      recs[b].ksplit = 1;
      r->ipad_host[b] = c->Ipad;
    }
    CK(cudaMemcpyAsync(r->recs, recs.data(), sizeof(TcStackLayer) * recs.size(), cudaMemcpyHostToDevice, st));
    CK(cudaStreamSynchronize(st));
  }
  std::vector<uint8_t> avail(h->B, 0);
  for (int b : order) avail[b] = 1;
  CK(cudaMemcpyAsync(r->avail, avail.data(), h->B, cudaMemcpyHostToDevice, st));
  CK(cudaStreamSynchronize(st));
  r->counts_host.assign(h->B, 0);
  r->rowbase_host.assign(h->B, 0);
  r->version = h->version;
  return MLPMOE_OK;
}

}  // namespace

extern "C" {

mlpmoe_status_t mlpmoe_create(mlpmoe_handle_t* out, int64_t d_model, int64_t d_inter, int32_t B, const int64_t* d_b,
                              const void* W_gate, const void* W_up, const void* W_down, const float* alpha,
                              mlpmoe_dtype_t dtype, mlpmoe_layout_t layout, int64_t max_tokens, void* stream) {
  if (layout != MLPMOE_LAYOUT_PAPER && layout != MLPMOE_LAYOUT_LINEAR) return MLPMOE_ERR_INVALID_ARG;
  return create_impl(out, d_model, d_inter, B, d_b, W_gate, W_up, W_down, alpha, dtype, static_cast<int>(layout), max_tokens, nullptr,
                     static_cast<cudaStream_t>(stream));
}

void mlpmoe_destroy(mlpmoe_handle_t h) { free_layer(h); }

mlpmoe_status_t mlpmoe_share_workspace(mlpmoe_handle_t h, mlpmoe_handle_t donor) {
  if (!h || !donor) return MLPMOE_ERR_INVALID_ARG;
  if (h->ws == donor->ws) return MLPMOE_OK;
  const Workspace* w = donor->ws;
  if (w->elem_size != h->elem_size || w->max_tokens < h->max_tokens || w->Ipad_max < h->Ipad_max || w->d < h->d)
    return MLPMOE_ERR_INVALID_ARG;
  ws_release(h->ws);
  h->ws = donor->ws;
  h->ws->refs += 1;
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_fade(mlpmoe_handle_t h, const double* s, void* stream) {
  if (!h) return MLPMOE_ERR_INVALID_ARG;
  if (s) {
    for (int b = 0; b < h->B; ++b)
      if (!(s[b] >= 0.0 && s[b] < 1.0)) return MLPMOE_ERR_BAD_SCHEDULE;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  std::vector<FadeSeg> segs;
  for (int b = 0; b < h->B; ++b) {
    const int64_t m = h->d * h->d_b[b];
    if (s ? (s[b] == 0.0) : (b == 0)) continue;      // the dense backbone / "leave untouched"
    const int64_t lo = s ? fade_position_exact(s[b], m) : fade_position_default(b, h->B, m);
    for (int proj = 0; proj < 2; ++proj) {
      FadeSeg g;
      g.base = static_cast<char*>(proj == 0 ? h->Wg_c : h->Wu_c) + static_cast<size_t>(h->offs[b]) * h->d * h->elem_size;
      g.m = m;
      g.rank = lo;
      segs.push_back(g);
    }
  }
  CK(launch_fade(segs.data(), static_cast<int>(segs.size()), h->fade_work, h->elem_size, st));
  CK(cudaStreamSynchronize(st));     // segs is host memory read by an async copy
  return reschedule(h, st);
}

mlpmoe_status_t mlpmoe_set_fast_fp32(mlpmoe_handle_t h, int32_t enable, void* stream) {
  if (!h) return MLPMOE_ERR_INVALID_ARG;
  if (h->dtype != MLPMOE_FP32) return MLPMOE_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!enable) { h->fast32 = false; return MLPMOE_OK; }
  if (h->Wgu3 == nullptr) {
    h->dp = round_up(h->d, 64);
    const size_t e2 = sizeof(__nv_bfloat16);
    if (cudaMalloc(&h->Wgu3, static_cast<size_t>(2 * h->Ipad_max) * 3 * h->dp * e2) != cudaSuccess ||
        cudaMalloc(&h->WdT3, static_cast<size_t>(h->d) * 3 * h->Ipad_max * e2) != cudaSuccess ||
        cudaMalloc(&h->X3, static_cast<size_t>(h->max_tokens) * 3 * h->dp * e2) != cudaSuccess ||
        cudaMalloc(&h->H3, static_cast<size_t>(h->max_tokens) * 3 * h->Ipad_max * e2) != cudaSuccess) {
      cudaGetLastError();
      cudaFree(h->Wgu3); cudaFree(h->WdT3); cudaFree(h->X3); cudaFree(h->H3);
      h->Wgu3 = h->WdT3 = h->X3 = h->H3 = nullptr;
      return MLPMOE_ERR_ALLOC;
    }
  }
  mlpmoe_status_t rc = refresh_fast32(h, st);
  if (rc != MLPMOE_OK) return rc;
  h->fast32 = true;
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_fade_structured(mlpmoe_handle_t h, const double* s, void* stream) {
  if (!h) return MLPMOE_ERR_INVALID_ARG;
  if (s) {
    for (int b = 0; b < h->B; ++b)
      if (!(s[b] >= 0.0 && s[b] < 1.0)) return MLPMOE_ERR_BAD_SCHEDULE;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // scores of all neurons (device, float64, fixed summation order), then the selection on the host
  double* score_dev = nullptr;
  int32_t* rows_dev = nullptr;
  if (cudaMalloc(reinterpret_cast<void**>(&score_dev), sizeof(double) * h->I) != cudaSuccess) { cudaGetLastError(); return MLPMOE_ERR_ALLOC; }
  std::vector<double> score(static_cast<size_t>(h->I));
  cudaError_t e = launch_neuron_scores(h->Wg_c, h->Wu_c, score_dev, h->I, h->d, h->elem_size, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(score.data(), score_dev, sizeof(double) * h->I, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  cudaFree(score_dev);
  if (e != cudaSuccess) return MLPMOE_ERR_CUDA;
  std::vector<int32_t> drop;
  std::vector<int32_t> order;
  for (int b = 0; b < h->B; ++b) {
    if (s ? (s[b] == 0.0) : (b == 0)) continue;                   // the dense backbone / "leave untouched"
    const int64_t m = h->d_b[b];
    // q = floor(s_b * d_b) in exact arithmetic
    const int64_t q = s ? fade_position_exact(s[b], m + 1)
                        : static_cast<int64_t>((static_cast<__int128>(9) * b * m) / (static_cast<__int128>(10) * h->B));
    if (q <= 0) continue;
    order.resize(static_cast<size_t>(m));
    for (int64_t i = 0; i < m; ++i) order[i] = static_cast<int32_t>(h->offs[b] + i);
    // ascending score, ties to the lower index (stable): the first q go
    std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) { return score[x] < score[y]; });
    drop.insert(drop.end(), order.begin(), order.begin() + q);
  }
  if (!drop.empty()) {
    if (cudaMalloc(reinterpret_cast<void**>(&rows_dev), sizeof(int32_t) * drop.size()) != cudaSuccess) { cudaGetLastError(); return MLPMOE_ERR_ALLOC; }
    e = cudaMemcpyAsync(rows_dev, drop.data(), sizeof(int32_t) * drop.size(), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = launch_zero_rows(h->Wg_c, h->Wu_c, rows_dev, static_cast<int64_t>(drop.size()), h->d, h->elem_size, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    cudaFree(rows_dev);
    if (e != cudaSuccess) return MLPMOE_ERR_CUDA;
  }
  return reschedule(h, st);
}

mlpmoe_status_t mlpmoe_prune(mlpmoe_handle_t h, const uint8_t* keep, int32_t compensate, void* stream) {
  if (!h || !keep) return MLPMOE_ERR_INVALID_ARG;
  std::vector<float> a(h->B);
  mlpmoe_status_t rc = prune_alpha_host(h->B, h->alpha_create.data(), keep, compensate, a.data());
  if (rc != MLPMOE_OK) return rc;
  std::vector<float> saved = h->alpha_eff;
  h->alpha_eff = a;
  rc = reschedule(h, static_cast<cudaStream_t>(stream));
  if (rc != MLPMOE_OK) h->alpha_eff = saved;
  return rc;
}

mlpmoe_status_t mlpmoe_prune_first_k(mlpmoe_handle_t h, int32_t K, void* stream) {
  if (!h) return MLPMOE_ERR_INVALID_ARG;
  if (K <= 0) return MLPMOE_ERR_EMPTY_KEEP_SET;
  if (K > h->B) return MLPMOE_ERR_INVALID_ARG;
  std::vector<uint8_t> keep(h->B);
  for (int b = 0; b < h->B; ++b) keep[b] = b < K ? 1 : 0;
  return mlpmoe_prune(h, keep.data(), 1, stream);
}

mlpmoe_status_t mlpmoe_forward(mlpmoe_handle_t h, const void* x, void* y, int64_t n_tokens, void* stream) {
  return forward_impl(h, x, y, n_tokens, nullptr, MLPMOE_FP32, static_cast<cudaStream_t>(stream));
}

mlpmoe_status_t mlpmoe_forward_ex(mlpmoe_handle_t h, const void* x, void* y, int64_t n_tokens, const float* residual,
                                  mlpmoe_dtype_t y_dtype, void* stream) {
  return forward_impl(h, x, y, n_tokens, residual, y_dtype, static_cast<cudaStream_t>(stream));
}

mlpmoe_status_t mlpmoe_forward_routed(mlpmoe_handle_t h, const void* x, float* y, int64_t n, const uint8_t* select,
                                      int32_t compensate, void* stream) {
  if (!h || n < 0) return MLPMOE_ERR_INVALID_ARG;
  if (n == 0) return MLPMOE_OK;
  if (!x || !y || !select || n > h->max_tokens || !aligned16(x) || !aligned16(y)) return MLPMOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  mlpmoe_status_t rc = ensure_routed(h, st);
  if (rc != MLPMOE_OK) return rc;
  Routed* r = h->routed;
  const int B = h->B;
  // group the tokens by branch; the per-branch counts come back to the host (one synchronisation per call)
  CK(launch_route_scan(select, r->avail, n, B, h->max_tokens, r->pos, r->lists, r->counts, st));
  CK(launch_route_coef(r->pos, n, B, r->n_avail, compensate ? 1 : 0, r->coef, st));
  CK(cudaMemcpyAsync(r->counts_host.data(), r->counts, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  // passes: consecutive branches whose rows fit the output buffer together
  std::vector<int> pass_end;               // one past the last branch of each pass
  int64_t used = 0;
  for (int b = 0; b < B; ++b) {
    const int64_t cnt = r->grouped ? round_up(r->counts_host[b], 256) : r->counts_host[b];
    if (used + cnt > r->ye_rows) {
      pass_end.push_back(b);
      used = 0;
    }
    r->rowbase_host[b] = static_cast<int32_t>(used);
    used += cnt;
  }
  pass_end.push_back(B);
  CK(cudaMemcpyAsync(r->rowbase, r->rowbase_host.data(), sizeof(int32_t) * B, cudaMemcpyHostToDevice, st));
  const size_t row = static_cast<size_t>(h->d) * h->elem_size;
  const size_t ye_row = sizeof(float) * static_cast<size_t>(h->d);     // branch outputs stay fp32 until they are summed
  int b0 = 0;
  for (size_t p = 0; r->grouped && p < pass_end.size(); ++p) {
    // the pass's branches in one launch: gathered rows of branch b at rows rowbase[b] .. of Xe, 256-row blocks
    r->block_layer.clear();
    {
      // about 8 blocks of 256 threads per SM over the pass's branches
      int per_branch = (8 * h->num_sms + (pass_end[p] - b0) - 1) / (pass_end[p] - b0);
      CK(launch_gather_branches(x, r->lists, h->max_tokens, r->counts, r->rowbase, b0, pass_end[p], row, r->Xe, per_branch, st));
      h->launches += 1;
    }
    for (int b = b0; b < pass_end[p]; ++b) {
      const int64_t cnt = r->counts_host[b];
      if (cnt == 0 || !r->child[b]) continue;
      // blocks are numbered by their position in Xe: the block index is the row offset / 256
      const int first_block = r->rowbase_host[b] / 256, n_blk = static_cast<int>((cnt + 255) / 256);
      if (static_cast<int>(r->block_layer.size()) < first_block + n_blk) r->block_layer.resize(first_block + n_blk, -1);
      for (int q = 0; q < n_blk; ++q) r->block_layer[first_block + q] = b;
    }
    const int n_blocks = static_cast<int>(r->block_layer.size());
    if (n_blocks > 0) {
      // every block of a pass is in use (the branches' padded row ranges are laid end to end)
      for (int q = 0; q < n_blocks; ++q)
        if (r->block_layer[q] < 0) return MLPMOE_ERR_CUDA;
      std::vector<int32_t> offs;
      tc_stack_group_schedule(r->block_layer.data(), n_blocks, h->d, r->ipad_host.data(), r->bn, h->num_sms, &r->items_host, &offs);
      const int64_t n_items = static_cast<int64_t>(r->items_host.size());
      r->items_host.insert(r->items_host.end(), offs.begin(), offs.end());
      const int64_t need_items = static_cast<int64_t>(r->items_host.size());
      const int64_t need_counters = 3 * static_cast<int64_t>(B) * n_blocks;
      if (need_items > r->items_cap || need_counters > r->counters_cap) {
        CK(cudaStreamSynchronize(st));
        cudaFree(r->items); cudaFree(r->group_counters);
        r->items = nullptr; r->group_counters = nullptr;
        r->items_cap = r->counters_cap = 0;
        if (cudaMalloc(reinterpret_cast<void**>(&r->items), sizeof(int32_t) * 2 * need_items) != cudaSuccess ||
            cudaMalloc(reinterpret_cast<void**>(&r->group_counters), sizeof(uint32_t) * 2 * need_counters) != cudaSuccess) {
          cudaGetLastError();
          return MLPMOE_ERR_ALLOC;
        }
        r->items_cap = 2 * need_items;
        r->counters_cap = 2 * need_counters;
      }
      CK(cudaMemcpyAsync(r->items, r->items_host.data(), sizeof(int32_t) * need_items, cudaMemcpyHostToDevice, st));
      if (p + 1 < pass_end.size()) CK(cudaStreamSynchronize(st));     // items_host is rebuilt by the next pass
      CK(cudaMemsetAsync(r->group_counters, 0, sizeof(uint32_t) * need_counters, st));
      // there is no norm step: its counters start at the value the gate|up tiles wait for
      CK(launch_fill_u32(r->group_counters, kStackNormArrivals, static_cast<int64_t>(B) * n_blocks, st));
      const int64_t rows = static_cast<int64_t>(n_blocks) * 256;
      TcStackArgs a;
      a.layers = r->recs;
      a.n_layers = B;
      if (!make_tmap(&a.tm_x, r->Xe, h->d, rows, h->d, 128)) return MLPMOE_ERR_CUDA;
      if (!make_tmap_t(&a.tm_y, r->Ye, h->d, rows, h->d, 32, 4)) return MLPMOE_ERR_CUDA;
      a.x = static_cast<float*>(r->Ye);
      a.xnorm = r->Xe;
      a.n = rows;
      a.d = h->d;
      a.bn = r->bn;
      a.eps = 0.0f;
      a.items = r->items;
      a.list_offsets = r->items + n_items;
      a.counters = r->group_counters;
      a.status = h->status;
      a.wait = h->wait;
      a.out_add = 0;
      pdl_overlap_enabled() = !h->timing;
      CK(launch_tc_stack(a, h->num_sms, st));
      h->launches += 2;
    }
    CK(launch_route_combine(r->Ye, 0, r->pos, r->rowbase, r->coef, n, B, b0, pass_end[p], h->d, p == 0, y, st));
    h->launches += 1;
    b0 = pass_end[p];
  }
  if (r->grouped) {
    h->launches += 2;
    return MLPMOE_OK;
  }
  for (size_t p = 0; p < pass_end.size(); ++p) {
    for (int b = b0; b < pass_end[p]; ++b) {
      const int64_t cnt = r->counts_host[b];
      if (cnt == 0 || !r->child[b]) continue;
      CK(launch_gather_rows(x, r->lists + static_cast<int64_t>(b) * h->max_tokens, cnt, row, r->Xe, st));
      r->child[b]->timing = false;
      rc = forward_impl(r->child[b], r->Xe, static_cast<char*>(r->Ye) + static_cast<size_t>(r->rowbase_host[b]) * ye_row, cnt, nullptr,
                        MLPMOE_FP32, st);
      if (rc != MLPMOE_OK) return rc;
      h->launches += 1 + r->child[b]->launches;
      r->child[b]->launches = 0;
    }
    CK(launch_route_combine(r->Ye, 0, r->pos, r->rowbase, r->coef, n, B, b0, pass_end[p], h->d, p == 0, y, st));
    h->launches += 1;
    b0 = pass_end[p];
  }
  h->launches += 2;
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_forward_host(mlpmoe_handle_t h, const void* x_host, float* y_host, int64_t n, void* stream) {
  if (!h || n < 0) return MLPMOE_ERR_INVALID_ARG;
  if (n == 0) return MLPMOE_OK;
  if (!x_host || !y_host || n > h->max_tokens) return MLPMOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CK(cudaMemcpyAsync(h->ws->xnorm, x_host, static_cast<size_t>(n) * h->d * h->elem_size, cudaMemcpyHostToDevice, st));
  mlpmoe_status_t rc = forward_impl(h, h->ws->xnorm, h->ws->yres, n, nullptr, MLPMOE_FP32, st);
  if (rc != MLPMOE_OK) return rc;
  CK(cudaMemcpyAsync(y_host, h->ws->yres, static_cast<size_t>(n) * h->d * sizeof(float), cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_rmsnorm(const float* x, void* r, int64_t n_tokens, int64_t d_model, float eps,
                               mlpmoe_dtype_t out_dtype, void* stream) {
  if (n_tokens < 0 || d_model <= 0 || d_model % 4 != 0) return MLPMOE_ERR_INVALID_ARG;
  if (n_tokens == 0) return MLPMOE_OK;
  if (!x || !r || !aligned16(x) || !aligned16(r)) return MLPMOE_ERR_INVALID_ARG;
  pdl_overlap_enabled() = true;
  CK(launch_rmsnorm(x, r, n_tokens, d_model, eps, out_dtype == MLPMOE_BF16 ? 2 : 4, static_cast<cudaStream_t>(stream)));
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_stack_prepare(const mlpmoe_handle_t* layers, int32_t n_layers, int64_t n, void* stream) {
  mlpmoe_status_t rc = check_stack(layers, n_layers, n);
  if (rc != MLPMOE_OK) return rc;
  if (n == 0) return MLPMOE_OK;
  return plan_stack(layers, n_layers, n, static_cast<cudaStream_t>(stream));
}

mlpmoe_status_t mlpmoe_stack_forward(const mlpmoe_handle_t* layers, int32_t n_layers, float* x, int64_t n, float eps,
                                     void* stream) {
  mlpmoe_status_t rc = check_stack(layers, n_layers, n);
  if (rc != MLPMOE_OK) return rc;
  if (n == 0) return MLPMOE_OK;
  if (!x || !aligned16(x)) return MLPMOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // a no-op after mlpmoe_stack_prepare for this stack and token count; otherwise the set-up happens here
  rc = plan_stack(layers, n_layers, n, st);
  if (rc != MLPMOE_OK) return rc;
  if (layers[0]->plan_kind == PLAN_DECODE) return run_decode_stack(layers, n_layers, x, n, eps, st);
  if (layers[0]->plan_kind == PLAN_PREFILL_STACK) return run_prefill_stack(layers, n_layers, x, n, eps, st);
  for (int l = 0; l < n_layers; ++l) {
    mlpmoe_layer_s* h = layers[l];
    pdl_overlap_enabled() = !h->timing;
    const long e0 = rec_event(h, st);
    CK(launch_rmsnorm(x, h->ws->xnorm, n, h->d, eps, h->elem_size, st));
    const long e1 = rec_event(h, st);
    add_span(h, SPAN_RMSNORM, e0, e1);
    h->launches += 1;
    rc = forward_impl(h, h->ws->xnorm, x, n, x, MLPMOE_FP32, st);
    if (rc != MLPMOE_OK) return rc;
  }
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_stack_forward_host(const mlpmoe_handle_t* layers, int32_t n_layers, const float* x_host,
                                          float* y_host, int64_t n, float eps, void* stream) {
  mlpmoe_status_t rc = check_stack(layers, n_layers, n);
  if (rc != MLPMOE_OK) return rc;
  if (n == 0) return MLPMOE_OK;
  if (!x_host || !y_host) return MLPMOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  mlpmoe_layer_s* h0 = layers[0];
  const size_t bytes = static_cast<size_t>(n) * h0->d * sizeof(float);
  CK(cudaMemcpyAsync(h0->ws->yres, x_host, bytes, cudaMemcpyHostToDevice, st));
  rc = mlpmoe_stack_forward(layers, n_layers, h0->ws->yres, n, eps, stream);
  if (rc != MLPMOE_OK) return rc;
  CK(cudaMemcpyAsync(y_host, h0->ws->yres, bytes, cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_get_klist(mlpmoe_handle_t h, int32_t* branches, int32_t* n_branches, int64_t* seg_start,
                                 int64_t* seg_len, int32_t* n_segs) {
  if (!h) return MLPMOE_ERR_INVALID_ARG;
  const Schedule& s = h->sched;
  if (branches) std::memcpy(branches, s.branches.data(), sizeof(int32_t) * s.branches.size());
  if (n_branches) *n_branches = static_cast<int32_t>(s.branches.size());
  if (seg_start) std::memcpy(seg_start, s.seg_start.data(), sizeof(int64_t) * s.seg_start.size());
  if (seg_len) std::memcpy(seg_len, s.seg_len.data(), sizeof(int64_t) * s.seg_len.size());
  if (n_segs) *n_segs = static_cast<int32_t>(s.seg_start.size());
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_get_alpha(mlpmoe_handle_t h, float* alpha) {
  if (!h || !alpha) return MLPMOE_ERR_INVALID_ARG;
  std::memcpy(alpha, h->alpha_eff.data(), sizeof(float) * h->B);
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_get_active_neurons(mlpmoe_handle_t h, int64_t* n_active) {
  if (!h || !n_active) return MLPMOE_ERR_INVALID_ARG;
  *n_active = h->sched.n_active;
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_nnz(mlpmoe_handle_t h, int64_t* nnz_gate, int64_t* nnz_up, int64_t* nnz_down) {
  if (!h) return MLPMOE_ERR_INVALID_ARG;
  // row_nnz_host is refreshed by every reschedule (create, fade, prune), the only calls that change weights
  int64_t* outs[3] = {nnz_gate, nnz_up, nnz_down};
  for (int which = 0; which < 3; ++which) {
    if (!outs[which]) continue;
    for (int b = 0; b < h->B; ++b) {
      int64_t c = 0;
      for (int64_t j = h->offs[b]; j < h->offs[b + 1]; ++j) c += h->row_nnz_host[which * h->I + j];
      outs[which][b] = c;
    }
  }
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_get_weights(mlpmoe_handle_t h, void* W_gate, void* W_up, void* W_down, void* stream) {
  if (!h) return MLPMOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (W_gate) CK(launch_transpose(h->Wg_c, W_gate, h->I, h->d, h->elem_size, st));
  if (W_up) CK(launch_transpose(h->Wu_c, W_up, h->I, h->d, h->elem_size, st));
  if (W_down)
    CK(cudaMemcpyAsync(W_down, h->Wd_c, static_cast<size_t>(h->I) * h->d * h->elem_size, cudaMemcpyDeviceToDevice, st));
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_get_status(mlpmoe_handle_t h) {
  if (!h) return MLPMOE_ERR_INVALID_ARG;
  uint32_t w = 0;
  CK(cudaDeviceSynchronize());
  CK(cudaMemcpy(&w, h->status, sizeof(w), cudaMemcpyDeviceToHost));
  // the per-branch layers of routed calls report through their parent
  bool child_timeout = false;
  if (h->routed)
    for (mlpmoe_layer_s* c : h->routed->child)
      if (c && mlpmoe_get_status(c) == MLPMOE_ERR_DEVICE_TIMEOUT) child_timeout = true;
  if (w == kStatusOk) return child_timeout ? MLPMOE_ERR_DEVICE_TIMEOUT : MLPMOE_OK;
  // A kernel gave up: the dependency counters that its work items leave at zero in a normal run may hold
  // anything.  Re-arm the handle (the counters that are not zeroed before every launch, and the status word).
  CK(cudaMemset(h->block_done, 0, sizeof(uint32_t) * 2 * h->max_blocks));
  CK(cudaMemset(h->counters, 0, sizeof(uint32_t) * ((h->d + 127) / 128) * 4));
  CK(cudaMemset(h->status, 0, sizeof(uint32_t)));
  return MLPMOE_ERR_DEVICE_TIMEOUT;
}

mlpmoe_status_t mlpmoe_debug_set_decode_kernel(mlpmoe_handle_t h, int32_t kernel) {
  if (!h || kernel < 0 || kernel > 2) return MLPMOE_ERR_INVALID_ARG;
  h->decode_kernel = kernel;
  h->plan_kind = PLAN_NONE;            // the next stack call chooses again
  h->plan_key.clear();
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_debug_set_wait(mlpmoe_handle_t h, uint64_t limit_ns, uint32_t extra_arrivals) {
  if (!h) return MLPMOE_ERR_INVALID_ARG;
  h->wait = WaitCfg();
  if (limit_ns != 0) h->wait.limit_ns = limit_ns;
  h->wait.extra_arrivals = extra_arrivals;
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_get_workspace(mlpmoe_handle_t h, void** H, int64_t* H_bytes, void** xnorm, int64_t* xnorm_bytes,
                                     float** yres, int64_t* yres_bytes, int64_t* n_active_pad) {
  if (!h) return MLPMOE_ERR_INVALID_ARG;
  const Workspace* w = h->ws;
  if (H) *H = w->H;
  if (H_bytes) *H_bytes = w->max_tokens * w->Ipad_max * w->elem_size;
  if (xnorm) *xnorm = w->xnorm;
  if (xnorm_bytes) *xnorm_bytes = w->max_tokens * w->d * w->elem_size;
  if (yres) *yres = w->yres;
  if (yres_bytes) *yres_bytes = w->max_tokens * w->d * static_cast<int64_t>(sizeof(float));
  if (n_active_pad) *n_active_pad = h->Ipad;
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_get_kernel_clock(mlpmoe_handle_t h, double* sm_mhz, double* kernel_us) {
  if (!h) return MLPMOE_ERR_INVALID_ARG;
  uint64_t probe[2] = {0, 0};
  CK(cudaDeviceSynchronize());
  CK(cudaMemcpy(probe, reinterpret_cast<const char*>(h->status) + 16, sizeof(probe), cudaMemcpyDeviceToHost));
  if (sm_mhz) *sm_mhz = probe[1] ? static_cast<double>(probe[0]) / static_cast<double>(probe[1]) * 1e3 : 0.0;
  if (kernel_us) *kernel_us = static_cast<double>(probe[1]) * 1e-3;
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_get_launch_count(mlpmoe_handle_t h, int64_t* launches) {
  if (!h || !launches) return MLPMOE_ERR_INVALID_ARG;
  *launches = h->launches;
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_set_timing(mlpmoe_handle_t h, int32_t enable) {
  if (!h) return MLPMOE_ERR_INVALID_ARG;
  if (enable && h->events.empty()) {
    h->events.reserve(kEventPool);
    for (size_t i = 0; i < kEventPool; ++i) {
      cudaEvent_t e;
      CK(cudaEventCreate(&e));
      h->events.push_back(e);
    }
  }
  h->timing = enable != 0;
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_get_timing(mlpmoe_handle_t h, double* ms, int64_t* launches) {
  if (!h || !ms || !launches) return MLPMOE_ERR_INVALID_ARG;
  CK(cudaDeviceSynchronize());
  for (int k = 0; k < 3; ++k) { ms[k] = 0.0; launches[k] = 0; }
  for (const auto& sp : h->spans) {
    float t = 0.f;
    CK(cudaEventElapsedTime(&t, h->events[sp.a], h->events[sp.b]));
    ms[sp.kind] += t;
    launches[sp.kind] += 1;
  }
  h->spans.clear();
  h->events_used = 0;
  return MLPMOE_OK;
}

const char* mlpmoe_status_string(mlpmoe_status_t s) {
  switch (s) {
    case MLPMOE_OK: return "ok";
    case MLPMOE_ERR_INVALID_ARG: return "invalid argument";
    case MLPMOE_ERR_BAD_PARTITION: return "bad partition of d_inter";
    case MLPMOE_ERR_EMPTY_KEEP_SET: return "empty keep set";
    case MLPMOE_ERR_BAD_SCHEDULE: return "sparsity ratio outside [0, 1)";
    case MLPMOE_ERR_UNSUPPORTED: return "unsupported shape, dtype or device";
    case MLPMOE_ERR_ALLOC: return "allocation failed";
    case MLPMOE_ERR_CUDA: return "CUDA call failed";
    case MLPMOE_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
  }
  return "unknown status";
}

// ---- host-only helpers ------------------------------------------------------
mlpmoe_status_t mlpmoe_host_fade_position(double s, int64_t m, int64_t* lo) {
  if (!lo || m <= 0) return MLPMOE_ERR_INVALID_ARG;
  if (!(s >= 0.0 && s < 1.0)) return MLPMOE_ERR_BAD_SCHEDULE;
  *lo = fade_position_exact(s, m);
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_host_fade_position_default(int32_t b, int32_t B, int64_t m, int64_t* lo) {
  if (!lo || m <= 0 || B <= 0 || b < 0 || b >= B) return MLPMOE_ERR_INVALID_ARG;
  *lo = fade_position_default(b, B, m);
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_host_prune_alpha(int32_t B, const float* alpha, const uint8_t* keep, int32_t compensate,
                                        float* alpha_eff) {
  if (B <= 0 || !alpha || !keep || !alpha_eff) return MLPMOE_ERR_INVALID_ARG;
  return prune_alpha_host(B, alpha, keep, compensate, alpha_eff);
}

mlpmoe_status_t mlpmoe_host_schedule(int32_t B, const int64_t* d_b, const float* alpha_eff, const uint8_t* live,
                                     int32_t* branches, int32_t* n_branches, int64_t* seg_start, int64_t* seg_len,
                                     int32_t* n_segs, int64_t* n_active) {
  if (B <= 0 || !d_b || !alpha_eff) return MLPMOE_ERR_INVALID_ARG;
  int64_t I = 0;
  for (int b = 0; b < B; ++b) {
    if (d_b[b] <= 0) return MLPMOE_ERR_BAD_PARTITION;
    I += d_b[b];
  }
  Schedule s;
  build_schedule(B, d_b, alpha_eff, live, &s);
  if (branches) std::memcpy(branches, s.branches.data(), sizeof(int32_t) * s.branches.size());
  if (n_branches) *n_branches = static_cast<int32_t>(s.branches.size());
  if (seg_start) std::memcpy(seg_start, s.seg_start.data(), sizeof(int64_t) * s.seg_start.size());
  if (seg_len) std::memcpy(seg_len, s.seg_len.data(), sizeof(int64_t) * s.seg_len.size());
  if (n_segs) *n_segs = static_cast<int32_t>(s.seg_start.size());
  if (n_active) *n_active = s.n_active;
  (void)I;
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_host_tile_schedule(int64_t n_tokens, int64_t d_model, int64_t n_active_pad, int32_t bn,
                                          int32_t ksplit, int32_t num_sms, int32_t* tiles, int32_t* n_tiles,
                                          int32_t* offsets) {
  if (n_tokens <= 0 || d_model <= 0 || n_active_pad <= 0 || n_active_pad % 128 != 0 || bn < 32 || bn > 256 || bn % 32 != 0 ||
      num_sms < 2 || ksplit < 1 || ksplit > 4 || !tiles || !n_tiles || !offsets)
    return MLPMOE_ERR_INVALID_ARG;
  std::vector<int32_t> t, o;
  tc_layer_schedule(n_tokens, d_model, n_active_pad, bn, ksplit, num_sms, &t, &o);
  std::memcpy(tiles, t.data(), sizeof(int32_t) * t.size());
  std::memcpy(offsets, o.data(), sizeof(int32_t) * o.size());
  *n_tiles = static_cast<int32_t>(t.size());
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_host_stack_schedule(int64_t n_tokens, int64_t d_model, int32_t n_layers, const int64_t* n_active_pad,
                                           const int32_t* ksplit, int32_t bn, int32_t num_sms, int32_t* items,
                                           int64_t item_capacity, int64_t* n_items, int32_t* offsets) {
  if (n_tokens <= 0 || d_model <= 0 || n_layers <= 0 || !n_active_pad || !ksplit || bn < 32 || bn > 256 || bn % 32 != 0 ||
      num_sms < 2 || !items || !n_items || !offsets)
    return MLPMOE_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l)
    if (n_active_pad[l] <= 0 || n_active_pad[l] % 128 != 0 || ksplit[l] < 1 || ksplit[l] > 4) return MLPMOE_ERR_INVALID_ARG;
  std::vector<int32_t> t, o;
  std::vector<int> ks(ksplit, ksplit + n_layers);
  tc_stack_schedule(n_tokens, d_model, n_active_pad, ks.data(), n_layers, bn, num_sms, &t, &o);
  *n_items = static_cast<int64_t>(t.size() / 2);
  if (static_cast<int64_t>(t.size() / 2) > item_capacity) return MLPMOE_ERR_INVALID_ARG;
  std::memcpy(items, t.data(), sizeof(int32_t) * t.size());
  std::memcpy(offsets, o.data(), sizeof(int32_t) * o.size());
  return MLPMOE_OK;
}

mlpmoe_status_t mlpmoe_host_group_schedule(const int32_t* block_branch, int32_t n_blocks, int64_t d_model, int32_t n_branches,
                                           const int64_t* n_active_pad, int32_t bn, int32_t num_sms, int32_t* items,
                                           int64_t item_capacity, int64_t* n_items, int32_t* offsets) {
  if (!block_branch || n_blocks < 0 || d_model <= 0 || n_branches <= 0 || !n_active_pad || bn < 32 || bn > 256 || bn % 32 != 0 ||
      num_sms < 2 || !items || !n_items || !offsets)
    return MLPMOE_ERR_INVALID_ARG;
  for (int b = 0; b < n_branches; ++b)
    if (n_active_pad[b] <= 0 || n_active_pad[b] % 128 != 0) return MLPMOE_ERR_INVALID_ARG;
  for (int r = 0; r < n_blocks; ++r)
    if (block_branch[r] < 0 || block_branch[r] >= n_branches) return MLPMOE_ERR_INVALID_ARG;
  std::vector<int32_t> t, o;
  tc_stack_group_schedule(block_branch, n_blocks, d_model, n_active_pad, bn, num_sms, &t, &o);
  *n_items = static_cast<int64_t>(t.size() / 2);
  if (static_cast<int64_t>(t.size() / 2) > item_capacity) return MLPMOE_ERR_INVALID_ARG;
  std::memcpy(items, t.data(), sizeof(int32_t) * t.size());
  std::memcpy(offsets, o.data(), sizeof(int32_t) * o.size());
  return MLPMOE_OK;
}

}  // extern "C"
