// Per-token branch selection (dynamic routing over branches; Section 7, Limitation 2, and Section 8
// name it as future work, the rule is this library's own and is stated in mlpmoe.h): the glue
// around the per-branch GEMMs.  Tokens are grouped by selected branch (a stable scan per branch),
// their rows gathered into one contiguous block per branch, every branch evaluated on its own
// block by the layer kernels (bf16: all blocks in one launch of the stack kernel, the branches as
// its layer records), and the blocks' outputs summed back per token with the token's compensation
// factor sqrt(B' / |S_t|) (Section 3.3 with K = |S_t|).  All HBM-bound.
#include "internal.h"

namespace mlpmoe {
namespace {

constexpr int SCAN_THREADS = 1024;

// One block per branch b: position of every selecting token among the branch's tokens, in token
// order.  pos[t * B + b] = that position or -1; lists[b * list_stride + position] = t; counts[b].
__global__ void __launch_bounds__(SCAN_THREADS) route_scan_kernel(const uint8_t* __restrict__ select,
                                                                  const uint8_t* __restrict__ avail, int64_t n, int B,
                                                                  int64_t list_stride, int32_t* __restrict__ pos,
                                                                  int32_t* __restrict__ lists, int32_t* __restrict__ counts) {
  __shared__ int warp_total[SCAN_THREADS / 32];
  __shared__ int chunk_total;
  const int b = blockIdx.x;
  const int lane = threadIdx.x % 32, warp = threadIdx.x / 32;
  const bool branch_ok = avail[b] != 0;
  int running = 0;
  for (int64_t base = 0; base < n; base += SCAN_THREADS) {
    const int64_t t = base + threadIdx.x;
    const bool f = branch_ok && t < n && select[t * B + b] != 0;
    const unsigned ballot = __ballot_sync(0xFFFFFFFFu, f);
    const int before = __popc(ballot & ((1u << lane) - 1u));
    if (lane == 0) warp_total[warp] = __popc(ballot);
    __syncthreads();
    if (warp == 0) {
      int v = warp_total[lane];
      for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xFFFFFFFFu, v, o);
        if (lane >= o) v += u;
      }
      warp_total[lane] = v;              // inclusive totals of the warps
      if (lane == 31) chunk_total = v;
    }
    __syncthreads();
    const int p = running + (warp > 0 ? warp_total[warp - 1] : 0) + before;
    if (t < n) pos[t * B + b] = f ? p : -1;
    if (f) lists[static_cast<int64_t>(b) * list_stride + p] = static_cast<int32_t>(t);
    running += chunk_total;
    __syncthreads();                     // warp_total is rewritten by the next chunk
  }
  if (threadIdx.x == 0) counts[b] = running;
}

// coef[t] = sqrt(B' / |S_t|) (1 without compensation), 0 for a token that selects nothing.  The
// quotient and the root are taken in double and rounded once.
__global__ void route_coef_kernel(const int32_t* __restrict__ pos, int64_t n, int B, int n_avail, int compensate,
                                  float* __restrict__ coef) {
  const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (t >= n) return;
  int k = 0;
  for (int b = 0; b < B; ++b) k += pos[t * B + b] >= 0 ? 1 : 0;
  float c = 0.0f;
  if (k > 0) c = compensate ? static_cast<float>(sqrt(static_cast<double>(n_avail) / static_cast<double>(k))) : 1.0f;
  coef[t] = c;
}

// out row r = src row list[r]; rows are row_vecs 16-byte vectors long.
__global__ void gather_rows_kernel(const uint4* __restrict__ src, const int32_t* __restrict__ list, int64_t n_rows,
                                   int64_t row_vecs, uint4* __restrict__ out) {
  const int64_t total = n_rows * row_vecs;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t r = i / row_vecs, v = i % row_vecs;
    out[i] = src[static_cast<int64_t>(list[r]) * row_vecs + v];
  }
}

// All branches b_lo <= b < b_hi in one launch (blockIdx.y = b - b_lo): row p < counts[b] of branch b goes to row
// rowbase[b] + p of out.  The counts are read on the device.
__global__ void gather_branches_kernel(const uint4* __restrict__ src, const int32_t* __restrict__ lists, int64_t list_stride,
                                       const int32_t* __restrict__ counts, const int32_t* __restrict__ rowbase, int b_lo,
                                       int64_t row_vecs, uint4* __restrict__ out) {
  const int b = b_lo + blockIdx.y;
  const int64_t total = static_cast<int64_t>(counts[b]) * row_vecs;
  const int32_t* list = lists + static_cast<int64_t>(b) * list_stride;
  uint4* dst = out + static_cast<int64_t>(rowbase[b]) * row_vecs;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t r = i / row_vecs, v = i % row_vecs;
    dst[i] = src[static_cast<int64_t>(list[r]) * row_vecs + v];
  }
}

__global__ void fill_u32_kernel(uint32_t* __restrict__ dst, uint32_t value, int64_t count) {
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < count; i += static_cast<int64_t>(gridDim.x) * blockDim.x)
    dst[i] = value;
}

__device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xFFFF0000u), __uint_as_float(u.y << 16),
                     __uint_as_float(u.y & 0xFFFF0000u));
}

// One block per token: y[t] = (first ? 0 : y[t]) + coef[t] * sum over the branches b_lo <= b < b_hi that the token
// selected, in ascending b, of row (rowbase[b] + pos[t, b]) of Ye.  d is a multiple of 4.
template <typename T>
__global__ void route_combine_kernel(const T* __restrict__ Ye, const int32_t* __restrict__ pos, const int32_t* __restrict__ rowbase,
                                     const float* __restrict__ coef, int B, int b_lo, int b_hi, int64_t d, int first,
                                     float* __restrict__ y) {
  const int64_t t = blockIdx.x;
  const float c = coef[t];
  const int32_t* prow = pos + t * B;
  for (int64_t col = static_cast<int64_t>(threadIdx.x) * 4; col < d; col += static_cast<int64_t>(blockDim.x) * 4) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int b = b_lo; b < b_hi; ++b) {
      const int32_t p = prow[b];
      if (p < 0) continue;
      const float4 v = load4(Ye + (static_cast<int64_t>(rowbase[b]) + p) * d + col);
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    float4 out = make_float4(c * acc.x, c * acc.y, c * acc.z, c * acc.w);
    if (!first) {
      const float4 old = *reinterpret_cast<const float4*>(y + t * d + col);
      out.x += old.x; out.y += old.y; out.z += old.z; out.w += old.w;
    }
    *reinterpret_cast<float4*>(y + t * d + col) = out;
  }
}

}  // namespace

cudaError_t launch_route_scan(const uint8_t* select, const uint8_t* avail, int64_t n, int B, int64_t list_stride, int32_t* pos,
                              int32_t* lists, int32_t* counts, cudaStream_t st) {
  route_scan_kernel<<<B, SCAN_THREADS, 0, st>>>(select, avail, n, B, list_stride, pos, lists, counts);
  return cudaGetLastError();
}

cudaError_t launch_route_coef(const int32_t* pos, int64_t n, int B, int n_avail, int compensate, float* coef, cudaStream_t st) {
  route_coef_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, st>>>(pos, n, B, n_avail, compensate, coef);
  return cudaGetLastError();
}

cudaError_t launch_gather_rows(const void* src, const int32_t* list, int64_t n_rows, int64_t row_bytes, void* out, cudaStream_t st) {
  if (n_rows == 0) return cudaSuccess;
  const int64_t total = n_rows * (row_bytes / 16);
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  gather_rows_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(static_cast<const uint4*>(src), list, n_rows, row_bytes / 16,
                                                                  static_cast<uint4*>(out));
  return cudaGetLastError();
}

cudaError_t launch_gather_branches(const void* src, const int32_t* lists, int64_t list_stride, const int32_t* counts,
                                   const int32_t* rowbase, int b_lo, int b_hi, int64_t row_bytes, void* out, int blocks_per_branch,
                                   cudaStream_t st) {
  if (b_hi <= b_lo) return cudaSuccess;
  gather_branches_kernel<<<dim3(static_cast<unsigned>(blocks_per_branch), static_cast<unsigned>(b_hi - b_lo)), 256, 0, st>>>(
      static_cast<const uint4*>(src), lists, list_stride, counts, rowbase, b_lo, row_bytes / 16, static_cast<uint4*>(out));
  return cudaGetLastError();
}

cudaError_t launch_fill_u32(uint32_t* dst, uint32_t value, int64_t count, cudaStream_t st) {
  if (count == 0) return cudaSuccess;
  int64_t blocks = (count + 255) / 256;
  if (blocks > 1024) blocks = 1024;
  fill_u32_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(dst, value, count);
  return cudaGetLastError();
}

cudaError_t launch_route_combine(const void* Ye, int ye_bf16, const int32_t* pos, const int32_t* rowbase, const float* coef, int64_t n,
                                 int B, int b_lo, int b_hi, int64_t d, int first, float* y, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  int threads = static_cast<int>((d / 4 + 31) / 32 * 32);
  if (threads > 1024) threads = 1024;
  if (ye_bf16)
    route_combine_kernel<__nv_bfloat16><<<static_cast<unsigned>(n), threads, 0, st>>>(static_cast<const __nv_bfloat16*>(Ye), pos, rowbase,
                                                                                    coef, B, b_lo, b_hi, d, first, y);
  else
    route_combine_kernel<float><<<static_cast<unsigned>(n), threads, 0, st>>>(static_cast<const float*>(Ye), pos, rowbase, coef, B, b_lo,
                                                                            b_hi, d, first, y);
  return cudaGetLastError();
}

}  // namespace mlpmoe
