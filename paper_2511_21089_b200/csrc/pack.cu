// Set-up kernels: weight packer (slice / transpose / interleave, Section 3.1), Fractal Fade
// (exact rank selection + masking, Section 3.2), per-neuron non-zero counts for the scheduler,
// and the RMSNorm helper of the stack harness.  All HBM-bound copies.
#include "internal.h"

namespace mlpmoe {
namespace {

// ------------------------------------------------------------- transpose ----
template <typename T>
__global__ void transpose_kernel(const T* __restrict__ src, T* __restrict__ dst, int64_t rows, int64_t cols) {
  __shared__ T tile[32][33];
  const int64_t c0 = static_cast<int64_t>(blockIdx.x) * 32, r0 = static_cast<int64_t>(blockIdx.y) * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int64_t r = r0 + i, c = c0 + threadIdx.x;
    if (r < rows && c < cols) tile[i][threadIdx.x] = src[r * cols + c];
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int64_t c = c0 + i, r = r0 + threadIdx.x;
    if (r < rows && c < cols) dst[c * rows + r] = tile[threadIdx.x][i];
  }
}

// ------------------------------------------------------ gate|up gather ------
// One block per packed row; 16-byte vectors (d * elem_size is a multiple of 16).
__global__ void gather_gateup_kernel(const uint4* __restrict__ Wg_c, const uint4* __restrict__ Wu_c,
                                     const int32_t* __restrict__ src_row, uint4* __restrict__ Wgu, int64_t n_active,
                                     int64_t row_vecs) {
  const int64_t r = blockIdx.x;
  const int64_t q = r / (2 * kGroup);
  const int within = static_cast<int>(r % (2 * kGroup));
  const bool is_up = within >= kGroup;
  const int64_t j = q * kGroup + (within % kGroup);
  uint4* out = Wgu + r * row_vecs;
  if (j < n_active) {
    const uint4* in = (is_up ? Wu_c : Wg_c) + static_cast<int64_t>(src_row[j]) * row_vecs;
    for (int64_t v = threadIdx.x; v < row_vecs; v += blockDim.x) out[v] = in[v];
  } else {
    for (int64_t v = threadIdx.x; v < row_vecs; v += blockDim.x) out[v] = make_uint4(0, 0, 0, 0);
  }
}

// -------------------------------------------------- down gather+transpose ---
template <typename T>
__global__ void gather_down_t_kernel(const T* __restrict__ Wd_c, const int32_t* __restrict__ src_row, T* __restrict__ WdT,
                                     int64_t n_active, int64_t n_active_pad, int64_t d) {
  __shared__ T tile[32][33];
  const int64_t j0 = static_cast<int64_t>(blockIdx.x) * 32, m0 = static_cast<int64_t>(blockIdx.y) * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int64_t j = j0 + i, m = m0 + threadIdx.x;
    T v = T(0);
    if (j < n_active && m < d) v = Wd_c[static_cast<int64_t>(src_row[j]) * d + m];
    tile[i][threadIdx.x] = v;
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int64_t m = m0 + i, j = j0 + threadIdx.x;
    if (m < d && j < n_active_pad) WdT[m * n_active_pad + j] = tile[threadIdx.x][i];
  }
}

// ------------------------------------------- stage-tiled copy for decode ---
// One thread per 16-byte piece of the destination.  A chunk is 256 rows of 128 bytes; piece c of row r
// goes to piece position c ^ (r % 8) of that row (the 128-byte swizzle of the shared-memory tiles).
__global__ void retile_decode_kernel(const uint4* __restrict__ Wgu, const uint4* __restrict__ WdT, uint4* __restrict__ out,
                                     int64_t Ipad, int64_t d, int kb1, int m_blocks, int64_t total) {
  const int64_t q = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (q >= total) return;
  const int chunks_per_tile = kb1 + 2 * m_blocks;
  const int c = static_cast<int>(q % 8), r = static_cast<int>((q / 8) % 256);
  const int64_t chunk_id = q / 2048;
  const int chunk = static_cast<int>(chunk_id % chunks_per_tile);
  const int64_t tile = chunk_id / chunks_per_tile;
  uint4 v = make_uint4(0, 0, 0, 0);
  if (chunk < kb1) {
    const int64_t col = static_cast<int64_t>(chunk) * 64 + c * 8;                 // K coordinate (elements)
    if (col < d) v = Wgu[((tile * 256 + r) * d + col) / 8];
  } else {
    const int blk = (chunk - kb1) / 2, ks = (chunk - kb1) % 2;
    const int64_t row = static_cast<int64_t>(blk) * 256 + r;                      // output column of the layer
    if (row < d) v = WdT[(row * Ipad + tile * 128 + ks * 64 + c * 8) / 8];
  }
  out[chunk_id * 2048 + r * 8 + (c ^ (r & 7))] = v;
}

// ------------------------------------------------ three-way bf16 split -------
// dst[r][s * Kp + k] = piece s of src[r][k] (s = 0, 1, 2; zero for K <= k < Kp), where
//   p0 = bf16(v), p1 = bf16(v - p0), p2 = bf16(v - p0 - p1)      (differences exact in fp32)
// so that p0 + p1 + p2 carries 24 significand bits of v.  One thread per 8 elements of a row.
__global__ void split3_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, int64_t rows, int64_t K, int64_t Kp,
                              int64_t src_pitch) {
  const int64_t chunks = Kp / 8;
  const int64_t q = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (q >= rows * chunks) return;
  const int64_t r = q / chunks, k0 = (q % chunks) * 8;
  __nv_bfloat16 p[3][8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float v = k0 + i < K ? src[r * src_pitch + k0 + i] : 0.f;
    const __nv_bfloat16 a = __float2bfloat16_rn(v);
    const float r1 = v - __bfloat162float(a);
    const __nv_bfloat16 b = __float2bfloat16_rn(r1);
    const __nv_bfloat16 c = __float2bfloat16_rn(r1 - __bfloat162float(b));
    p[0][i] = a; p[1][i] = b; p[2][i] = c;
  }
#pragma unroll
  for (int sgm = 0; sgm < 3; ++sgm)
    *reinterpret_cast<uint4*>(dst + r * 3 * Kp + sgm * Kp + k0) = *reinterpret_cast<const uint4*>(p[sgm]);
}

// ------------------------------------------- neuron scores / row zeroing ----
// score[j] = sum_k Wg_c[j][k]^2 + sum_k Wu_c[j][k]^2 in float64, accumulated one term after the other in
// that order (gate row first) with separately rounded multiply and add, so that a host program adding the
// same terms in the same order gets the same bits.  One thread per neuron (a set-up kernel).
template <typename T>
__device__ __forceinline__ double widen(T v);
template <>
__device__ __forceinline__ double widen<uint16_t>(uint16_t v) { return static_cast<double>(__uint_as_float(static_cast<uint32_t>(v) << 16)); }
template <>
__device__ __forceinline__ double widen<uint32_t>(uint32_t v) { return static_cast<double>(__uint_as_float(v)); }

template <typename T>
__global__ void neuron_score_kernel(const T* __restrict__ Wg_c, const T* __restrict__ Wu_c, double* __restrict__ score, int64_t I, int64_t d) {
  const int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (j >= I) return;
  double acc = 0.0;
  for (int which = 0; which < 2; ++which) {
    const T* row = (which == 0 ? Wg_c : Wu_c) + j * d;
    for (int64_t k = 0; k < d; ++k) {
      const double w = widen<T>(row[k]);
      acc = __dadd_rn(acc, __dmul_rn(w, w));
    }
  }
  score[j] = acc;
}

// Zeroes rows rows[i] (i < n_rows) of the two [I x d] matrices; one block per row.
template <typename T>
__global__ void zero_rows_kernel(T* __restrict__ A, T* __restrict__ B, const int32_t* __restrict__ rows, int64_t d) {
  const int64_t j = rows[blockIdx.x];
  for (int64_t k = threadIdx.x; k < d; k += blockDim.x) {
    A[j * d + k] = 0;
    B[j * d + k] = 0;
  }
}

// ------------------------------------------------------------ row nnz -------
template <typename T>
__device__ __forceinline__ bool is_nonzero(T v);
template <>
__device__ __forceinline__ bool is_nonzero<uint16_t>(uint16_t v) { return (v & 0x7FFFu) != 0; }
template <>
__device__ __forceinline__ bool is_nonzero<uint32_t>(uint32_t v) { return (v & 0x7FFFFFFFu) != 0; }

// One warp per (matrix, neuron row).
template <typename T>
__global__ void row_nnz_kernel(const T* __restrict__ Wg_c, const T* __restrict__ Wu_c, const T* __restrict__ Wd_c,
                               int32_t* __restrict__ out, int64_t I, int64_t d) {
  const int64_t w = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) / 32;
  const int lane = threadIdx.x % 32;
  if (w >= 3 * I) return;
  const int which = static_cast<int>(w / I);
  const int64_t j = w % I;
  const T* row = (which == 0 ? Wg_c : which == 1 ? Wu_c : Wd_c) + j * d;
  int cnt = 0;
  for (int64_t k = lane; k < d; k += 32) cnt += is_nonzero<T>(row[k]) ? 1 : 0;
  for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xFFFFFFFFu, cnt, o);
  if (lane == 0) out[w] = cnt;
}

// --------------------------------------------------------------- Fade -------
// Keys: magnitude bit patterns as 32-bit integers (order of non-negative floats equals the
// order of their bit patterns).  bf16 magnitudes are placed in the upper half so that the
// same digit positions serve both types.
template <typename T>
__device__ __forceinline__ uint32_t mag_key(T v);
template <>
__device__ __forceinline__ uint32_t mag_key<uint16_t>(uint16_t v) { return static_cast<uint32_t>(v & 0x7FFFu) << 16; }
template <>
__device__ __forceinline__ uint32_t mag_key<uint32_t>(uint32_t v) { return v & 0x7FFFFFFFu; }

struct FadeSegDev {
  void* base;
  int64_t m;
  int64_t rank;
};
struct FadeState {          // per segment
  uint32_t prefix;          // digits fixed so far (upper bits of the threshold key)
  uint32_t pad;
  int64_t remaining;        // rank among the elements that match the prefix
  uint32_t hist[256];
};

__global__ void fade_init_kernel(const FadeSegDev* segs, FadeState* st, int nseg) {
  const int s = blockIdx.x;
  if (s >= nseg) return;
  if (threadIdx.x == 0) {
    st[s].prefix = 0;
    st[s].remaining = segs[s].rank;
  }
  for (int i = threadIdx.x; i < 256; i += blockDim.x) st[s].hist[i] = 0;
}

// Histogram of digit `pass` (8 bits, most significant first) over elements matching the prefix.
template <typename T>
__global__ void fade_hist_kernel(const FadeSegDev* segs, FadeState* st, int pass) {
  __shared__ uint32_t h[256];
  const int s = blockIdx.y;
  for (int i = threadIdx.x; i < 256; i += blockDim.x) h[i] = 0;
  __syncthreads();
  const T* base = static_cast<const T*>(segs[s].base);
  const int64_t m = segs[s].m;
  const int shift = 24 - 8 * pass;
  const uint32_t himask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
  const uint32_t prefix = st[s].prefix;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < m;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const uint32_t key = mag_key<T>(base[i]);
    if ((key & himask) == prefix) atomicAdd(&h[(key >> shift) & 0xFFu], 1u);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 256; i += blockDim.x)
    if (h[i]) atomicAdd(&st[s].hist[i], h[i]);
}

// Pick the digit whose bin holds the wanted rank; fix it in the prefix; clear the histogram.
__global__ void fade_select_kernel(FadeState* st, int pass) {
  const int s = blockIdx.x;
  if (threadIdx.x == 0) {
    const int shift = 24 - 8 * pass;
    int64_t rem = st[s].remaining;
    int digit = 255;
    for (int b = 0; b < 256; ++b) {
      const int64_t c = st[s].hist[b];
      if (rem < c) { digit = b; break; }
      rem -= c;
    }
    st[s].prefix |= static_cast<uint32_t>(digit) << shift;
    st[s].remaining = rem;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 256; i += blockDim.x) st[s].hist[i] = 0;
}

// Zero every element whose magnitude key is <= the threshold key (keeps the sign bit, as a
// multiplication by a 0/1 mask does).
template <typename T>
__global__ void fade_mask_kernel(const FadeSegDev* segs, const FadeState* st) {
  const int s = blockIdx.y;
  T* base = static_cast<T*>(segs[s].base);
  const int64_t m = segs[s].m;
  const uint32_t thr = st[s].prefix;
  constexpr T sign = static_cast<T>(T(1) << (8 * sizeof(T) - 1));
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < m;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const T v = base[i];
    if (mag_key<T>(v) <= thr) base[i] = v & sign;
  }
}

// ------------------------------------------------------------- RMSNorm ------
__device__ __forceinline__ uint16_t f32_to_bf16_rn(float f) {
  uint32_t u = __float_as_uint(f);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return static_cast<uint16_t>(u >> 16);
}

// One warp per token row: pass 1 sums the squares, pass 2 re-reads the row (now in L1) and writes
// the normalised values.  HBM traffic = one read of x and one write of r.
template <bool OUT_BF16>
__global__ void __launch_bounds__(256) rmsnorm_kernel(const float* __restrict__ x, void* __restrict__ r, int64_t n, int64_t d,
                                                      float eps) {
  const int64_t t = static_cast<int64_t>(blockIdx.x) * (blockDim.x / 32) + threadIdx.x / 32;
  const int lane = threadIdx.x % 32;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may begin its set-up
  asm volatile("griddepcontrol.wait;" ::: "memory");                // x written by the previous kernel is complete
  if (t >= n) return;
  const float4* row = reinterpret_cast<const float4*>(x + t * d);
  const int64_t nv = d / 4;
  float ss = 0.f;
#pragma unroll 8
  for (int64_t v = lane; v < nv; v += 32) {
    const float4 a = row[v];
    ss += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
  }
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
  const float inv = 1.0f / sqrtf(ss / static_cast<float>(d) + eps);
#pragma unroll 8
  for (int64_t v = lane; v < nv; v += 32) {
    const float4 a = row[v];
    if (OUT_BF16) {
      uint2 o;
      o.x = static_cast<uint32_t>(f32_to_bf16_rn(a.x * inv)) | (static_cast<uint32_t>(f32_to_bf16_rn(a.y * inv)) << 16);
      o.y = static_cast<uint32_t>(f32_to_bf16_rn(a.z * inv)) | (static_cast<uint32_t>(f32_to_bf16_rn(a.w * inv)) << 16);
      reinterpret_cast<uint2*>(static_cast<uint16_t*>(r) + t * d)[v] = o;
    } else {
      reinterpret_cast<float4*>(static_cast<float*>(r) + t * d)[v] = make_float4(a.x * inv, a.y * inv, a.z * inv, a.w * inv);
    }
  }
}

// One warp per token row with the whole row in registers (d <= 128 NV): every load of the row is in
// flight before the first use, and the row crosses the memory system once.  The sum of squares adds
// the same terms in the same order as rmsnorm_kernel.
template <bool OUT_BF16, int NV>
__global__ void __launch_bounds__(256) rmsnorm_reg_kernel(const float* __restrict__ x, void* __restrict__ r, int64_t n,
                                                          int64_t d, float eps) {
  const int64_t t = static_cast<int64_t>(blockIdx.x) * (blockDim.x / 32) + threadIdx.x / 32;
  const int lane = threadIdx.x % 32;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (t >= n) return;
  const float4* row = reinterpret_cast<const float4*>(x + t * d);
  const int64_t nv = d / 4;
  float4 a[NV];
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int64_t v = static_cast<int64_t>(i) * 32 + lane;
    a[i] = v < nv ? __ldcs(row + v) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) ss += a[i].x * a[i].x + a[i].y * a[i].y + a[i].z * a[i].z + a[i].w * a[i].w;
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
  const float inv = 1.0f / sqrtf(ss / static_cast<float>(d) + eps);
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int64_t v = static_cast<int64_t>(i) * 32 + lane;
    if (v >= nv) continue;
    if (OUT_BF16) {
      uint2 o;
      o.x = static_cast<uint32_t>(f32_to_bf16_rn(a[i].x * inv)) | (static_cast<uint32_t>(f32_to_bf16_rn(a[i].y * inv)) << 16);
      o.y = static_cast<uint32_t>(f32_to_bf16_rn(a[i].z * inv)) | (static_cast<uint32_t>(f32_to_bf16_rn(a[i].w * inv)) << 16);
      reinterpret_cast<uint2*>(static_cast<uint16_t*>(r) + t * d)[v] = o;
    } else {
      reinterpret_cast<float4*>(static_cast<float*>(r) + t * d)[v] = make_float4(a[i].x * inv, a[i].y * inv, a[i].z * inv, a[i].w * inv);
    }
  }
}

// Few rows (decode): one 256-thread block per row, so that a row's loads are all in flight at once.
template <bool OUT_BF16>
__global__ void __launch_bounds__(256) rmsnorm_block_kernel(const float* __restrict__ x, void* __restrict__ r, int64_t n,
                                                            int64_t d, float eps) {
  const int64_t t = blockIdx.x;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const float4* row = reinterpret_cast<const float4*>(x + t * d);
  const int64_t nv = d / 4;
  float ss = 0.f;
  for (int64_t v = threadIdx.x; v < nv; v += blockDim.x) {
    const float4 a = row[v];
    ss += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
  }
  __shared__ float red[8];
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
  if (threadIdx.x % 32 == 0) red[threadIdx.x / 32] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) tot += red[i];
  const float inv = 1.0f / sqrtf(tot / static_cast<float>(d) + eps);
  for (int64_t v = threadIdx.x; v < nv; v += blockDim.x) {
    const float4 a = row[v];
    if (OUT_BF16) {
      uint2 o;
      o.x = static_cast<uint32_t>(f32_to_bf16_rn(a.x * inv)) | (static_cast<uint32_t>(f32_to_bf16_rn(a.y * inv)) << 16);
      o.y = static_cast<uint32_t>(f32_to_bf16_rn(a.z * inv)) | (static_cast<uint32_t>(f32_to_bf16_rn(a.w * inv)) << 16);
      reinterpret_cast<uint2*>(static_cast<uint16_t*>(r) + t * d)[v] = o;
    } else {
      reinterpret_cast<float4*>(static_cast<float*>(r) + t * d)[v] = make_float4(a.x * inv, a.y * inv, a.z * inv, a.w * inv);
    }
  }
}

inline unsigned cdiv(int64_t a, int64_t b) { return static_cast<unsigned>((a + b - 1) / b); }

}  // namespace

cudaError_t launch_transpose(const void* src, void* dst, int64_t rows, int64_t cols, int elem_size, cudaStream_t st) {
  if (rows == 0 || cols == 0) return cudaSuccess;
  dim3 grid(cdiv(cols, 32), cdiv(rows, 32)), block(32, 8);
  if (elem_size == 2)
    transpose_kernel<uint16_t><<<grid, block, 0, st>>>(static_cast<const uint16_t*>(src), static_cast<uint16_t*>(dst), rows, cols);
  else
    transpose_kernel<uint32_t><<<grid, block, 0, st>>>(static_cast<const uint32_t*>(src), static_cast<uint32_t*>(dst), rows, cols);
  return cudaGetLastError();
}

cudaError_t launch_gather_gateup(const void* Wg_c, const void* Wu_c, const int32_t* src_row, void* Wgu, int64_t n_active,
                                 int64_t n_active_pad, int64_t d, int elem_size, cudaStream_t st) {
  if (n_active_pad == 0) return cudaSuccess;
  const int64_t row_vecs = d * elem_size / 16;
  gather_gateup_kernel<<<static_cast<unsigned>(2 * n_active_pad), 128, 0, st>>>(
      static_cast<const uint4*>(Wg_c), static_cast<const uint4*>(Wu_c), src_row, static_cast<uint4*>(Wgu), n_active, row_vecs);
  return cudaGetLastError();
}

cudaError_t launch_gather_down_t(const void* Wd_c, const int32_t* src_row, void* WdT, int64_t n_active,
                                 int64_t n_active_pad, int64_t d, int elem_size, cudaStream_t st) {
  if (n_active_pad == 0) return cudaSuccess;
  dim3 grid(cdiv(n_active_pad, 32), cdiv(d, 32)), block(32, 8);
  if (elem_size == 2)
    gather_down_t_kernel<uint16_t><<<grid, block, 0, st>>>(static_cast<const uint16_t*>(Wd_c), src_row,
                                                           static_cast<uint16_t*>(WdT), n_active, n_active_pad, d);
  else
    gather_down_t_kernel<uint32_t><<<grid, block, 0, st>>>(static_cast<const uint32_t*>(Wd_c), src_row,
                                                           static_cast<uint32_t*>(WdT), n_active, n_active_pad, d);
  return cudaGetLastError();
}

cudaError_t launch_row_nnz(const void* Wg_c, const void* Wu_c, const void* Wd_c, int32_t* out, int64_t I, int64_t d,
                           int elem_size, cudaStream_t st) {
  const int64_t warps = 3 * I;
  const unsigned blocks = cdiv(warps * 32, 256);
  if (elem_size == 2)
    row_nnz_kernel<uint16_t><<<blocks, 256, 0, st>>>(static_cast<const uint16_t*>(Wg_c), static_cast<const uint16_t*>(Wu_c),
                                                     static_cast<const uint16_t*>(Wd_c), out, I, d);
  else
    row_nnz_kernel<uint32_t><<<blocks, 256, 0, st>>>(static_cast<const uint32_t*>(Wg_c), static_cast<const uint32_t*>(Wu_c),
                                                     static_cast<const uint32_t*>(Wd_c), out, I, d);
  return cudaGetLastError();
}

size_t decode_tiled_bytes(int64_t n_active_pad, int64_t d) {
  const int64_t chunks_per_tile = (d + 63) / 64 + 2 * ((d + 255) / 256);
  return static_cast<size_t>(n_active_pad / 128 * chunks_per_tile) * 32768;
}

cudaError_t launch_retile_decode(const void* Wgu, const void* WdT, void* tiled, int64_t n_active_pad, int64_t d, cudaStream_t st) {
  const int64_t total = static_cast<int64_t>(decode_tiled_bytes(n_active_pad, d) / 16);
  if (total == 0) return cudaSuccess;
  retile_decode_kernel<<<cdiv(total, 256), 256, 0, st>>>(static_cast<const uint4*>(Wgu), static_cast<const uint4*>(WdT),
                                                        static_cast<uint4*>(tiled), n_active_pad, d,
                                                        static_cast<int>((d + 63) / 64), static_cast<int>((d + 255) / 256), total);
  return cudaGetLastError();
}

cudaError_t launch_split3(const float* src, void* dst, int64_t rows, int64_t K, int64_t Kp, int64_t src_pitch, cudaStream_t st) {
  if (rows == 0) return cudaSuccess;
  const int64_t total = rows * (Kp / 8);
  split3_kernel<<<cdiv(total, 256), 256, 0, st>>>(src, static_cast<__nv_bfloat16*>(dst), rows, K, Kp, src_pitch);
  return cudaGetLastError();
}

cudaError_t launch_neuron_scores(const void* Wg_c, const void* Wu_c, double* score, int64_t I, int64_t d, int elem_size, cudaStream_t st) {
  if (I == 0) return cudaSuccess;
  if (elem_size == 2)
    neuron_score_kernel<uint16_t><<<cdiv(I, 64), 64, 0, st>>>(static_cast<const uint16_t*>(Wg_c), static_cast<const uint16_t*>(Wu_c), score, I, d);
  else
    neuron_score_kernel<uint32_t><<<cdiv(I, 64), 64, 0, st>>>(static_cast<const uint32_t*>(Wg_c), static_cast<const uint32_t*>(Wu_c), score, I, d);
  return cudaGetLastError();
}

cudaError_t launch_zero_rows(void* A, void* B, const int32_t* rows_dev, int64_t n_rows, int64_t d, int elem_size, cudaStream_t st) {
  if (n_rows == 0) return cudaSuccess;
  if (elem_size == 2)
    zero_rows_kernel<uint16_t><<<static_cast<unsigned>(n_rows), 256, 0, st>>>(static_cast<uint16_t*>(A), static_cast<uint16_t*>(B), rows_dev, d);
  else
    zero_rows_kernel<uint32_t><<<static_cast<unsigned>(n_rows), 256, 0, st>>>(static_cast<uint32_t*>(A), static_cast<uint32_t*>(B), rows_dev, d);
  return cudaGetLastError();
}

size_t fade_work_bytes(int nseg) { return static_cast<size_t>(nseg) * (sizeof(FadeSegDev) + sizeof(FadeState)); }

cudaError_t launch_fade(const FadeSeg* segs_host, int nseg, void* work, int elem_size, cudaStream_t st) {
  if (nseg == 0) return cudaSuccess;
  static_assert(sizeof(FadeSeg) == sizeof(FadeSegDev), "segment records must match");
  FadeSegDev* segs = static_cast<FadeSegDev*>(work);
  FadeState* state = reinterpret_cast<FadeState*>(segs + nseg);
  cudaError_t e = cudaMemcpyAsync(segs, segs_host, sizeof(FadeSegDev) * nseg, cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return e;
  int64_t max_m = 0;
  for (int i = 0; i < nseg; ++i) max_m = segs_host[i].m > max_m ? segs_host[i].m : max_m;
  unsigned bx = cdiv(max_m, 256 * 16);
  if (bx > 1024) bx = 1024;
  if (bx < 1) bx = 1;
  dim3 grid(bx, nseg);
  fade_init_kernel<<<nseg, 256, 0, st>>>(segs, state, nseg);
  const int passes = elem_size == 2 ? 2 : 4;   // bf16 keys carry 15 significant bits in the upper half
  for (int p = 0; p < passes; ++p) {
    if (elem_size == 2)
      fade_hist_kernel<uint16_t><<<grid, 256, 0, st>>>(segs, state, p);
    else
      fade_hist_kernel<uint32_t><<<grid, 256, 0, st>>>(segs, state, p);
    fade_select_kernel<<<nseg, 256, 0, st>>>(state, p);
  }
  if (elem_size == 2)
    fade_mask_kernel<uint16_t><<<grid, 256, 0, st>>>(segs, state);
  else
    fade_mask_kernel<uint32_t><<<grid, 256, 0, st>>>(segs, state);
  return cudaGetLastError();
}

cudaError_t launch_rmsnorm(const float* x, void* r, int64_t n, int64_t d, float eps, int out_elem_size, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  if (n <= 1024) {     // not enough rows to fill the GPU with one warp per row
    if (out_elem_size == 2)
      return launch_pdl(rmsnorm_block_kernel<true>, dim3(static_cast<unsigned>(n)), dim3(256), 0, st, x, r, n, d, eps);
    return launch_pdl(rmsnorm_block_kernel<false>, dim3(static_cast<unsigned>(n)), dim3(256), 0, st, x, r, n, d, eps);
  }
  if (out_elem_size == 2 && d <= 1024)
    return launch_pdl(rmsnorm_reg_kernel<true, 8>, dim3(cdiv(n, 8)), dim3(256), 0, st, x, r, n, d, eps);
  if (out_elem_size == 2 && d <= 4096)
    return launch_pdl(rmsnorm_reg_kernel<true, 32>, dim3(cdiv(n, 8)), dim3(256), 0, st, x, r, n, d, eps);
  if (out_elem_size == 2)
    return launch_pdl(rmsnorm_kernel<true>, dim3(cdiv(n, 8)), dim3(256), 0, st, x, r, n, d, eps);
  return launch_pdl(rmsnorm_kernel<false>, dim3(cdiv(n, 8)), dim3(256), 0, st, x, r, n, d, eps);
}

}  // namespace mlpmoe
