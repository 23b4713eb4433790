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

// ------------------------------------------ stage-tiled copies for decode ---
// One thread per 16-byte piece (8 bf16) of the destination; layouts in internal.h.
// Packed gate|up operand: neuron j's gate row is row (j / 128) * 256 + j % 128, its up row 128 further.
__device__ __forceinline__ uint4 load_gateup_piece(const uint4* __restrict__ Wgu, int64_t j, int proj, int64_t k, int64_t d) {
  if (k >= d) return make_uint4(0, 0, 0, 0);
  const int64_t row = (j / kGroup) * (2 * kGroup) + proj * kGroup + j % kGroup;
  return Wgu[(row * d + k) / 8];
}

// Phase A stages of every item of CTA blockIdx.y (grid.x strides over the CTA's pieces), and for the fused
// layout the item's phase B stages behind them.
__global__ void retile_items_kernel(int kind, const uint4* __restrict__ Wgu, const uint4* __restrict__ WdT, uint8_t* __restrict__ out,
                                    const int32_t* __restrict__ bounds, const int64_t* __restrict__ a_off, int64_t Ipad, int64_t d) {
  const int cta = blockIdx.y;
  const int lo = bounds[cta], hi = bounds[cta + 1];
  const int kb1 = static_cast<int>((d + 63) / 64), n_mb = static_cast<int>((d + 127) / 128);
  const int64_t stages_per_item = kb1 + (kind == kDecTiledFused ? n_mb : 0);
  int64_t item_base = a_off[cta];
  for (int u0 = lo; u0 < hi; u0 += kDecMaxUnitsPerItem) {
    const int r = kDecUnit * ((hi - u0) < kDecMaxUnitsPerItem ? (hi - u0) : kDecMaxUnitsPerItem);
    const int64_t n0 = static_cast<int64_t>(u0) * kDecUnit;
    const int64_t pieces_per_stage = 16 * r;                       // 256 r bytes
    const int64_t pieces = pieces_per_stage * stages_per_item;
    for (int64_t q = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; q < pieces; q += static_cast<int64_t>(gridDim.x) * blockDim.x) {
      const int64_t stage = q / pieces_per_stage;
      const int p = static_cast<int>(q % pieces_per_stage);
      uint4 v;
      int64_t dst;                                                 // piece position inside the stage
      if (stage < kb1) {
        const int R = p / 8, c = p % 8;                            // row of the stage (gate rows, then up rows), piece of the row
        v = load_gateup_piece(Wgu, n0 + R % r, R / r, stage * 64 + c * 8, d);
        dst = R * 8 + (c ^ (R & 7));                               // 128-byte swizzle
      } else {
        const int64_t mb = stage - kb1;
        const int k16 = p / 256, m = (p % 256) / 2, c = p % 2;     // sub-tile, output column of the block, piece of the 32-byte row
        const int64_t col = mb * 128 + m;
        v = col < d ? WdT[(col * Ipad + n0 + k16 * 16 + c * 8) / 8] : make_uint4(0, 0, 0, 0);
        dst = static_cast<int64_t>(k16) * 256 + m * 2 + (c ^ ((m >> 2) & 1));   // 32-byte swizzle
      }
      reinterpret_cast<uint4*>(out + item_base)[stage * pieces_per_stage + dst] = v;
    }
    item_base += pieces * 16;
  }
}

// Phase B region of the stack layout: chunk (block of 256 output columns, K-step) = 256 rows x 128 bytes.
__global__ void retile_down_chunks_kernel(const uint4* __restrict__ WdT, uint4* __restrict__ out, int64_t Ipad, int64_t d, int64_t total) {
  const int64_t q = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (q >= total) return;
  const int c = static_cast<int>(q % 8), r = static_cast<int>((q / 8) % 256);
  const int64_t chunk = q / 2048;
  const int64_t kb2 = Ipad / 64;
  const int64_t blk = chunk / kb2, kb = chunk % kb2;
  const int64_t col = blk * 256 + r;
  const uint4 v = col < d ? WdT[(col * Ipad + kb * 64 + c * 8) / 8] : make_uint4(0, 0, 0, 0);
  out[chunk * 2048 + r * 8 + (c ^ (r & 7))] = v;
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

int64_t decode_tiled_b_base(int64_t n_active_pad, int64_t d) { return n_active_pad * 256 * ((d + 63) / 64); }

size_t decode_tiled_bytes(int kind, int64_t n_active_pad, int64_t d) {
  if (kind == kDecTiledFused) return static_cast<size_t>(n_active_pad * 256 * ((d + 63) / 64 + (d + 127) / 128));
  return static_cast<size_t>(decode_tiled_b_base(n_active_pad, d) + ((d + 255) / 256) * (n_active_pad / 64) * 32768);
}

void decode_split(int kind, int64_t n_active_pad, int64_t d, int ctas, int32_t* bounds, int64_t* a_off) {
  const int64_t units = n_active_pad / kDecUnit;
  const int64_t stages = (d + 63) / 64 + (kind == kDecTiledFused ? (d + 127) / 128 : 0);
  for (int c = 0; c <= ctas; ++c) {
    bounds[c] = static_cast<int32_t>(units * c / ctas);
    a_off[c] = static_cast<int64_t>(bounds[c]) * kDecUnit * 256 * stages;
  }
}

cudaError_t launch_retile_decode(int kind, const void* Wgu, const void* WdT, void* tiled, const int32_t* bounds_dev,
                                 const int64_t* a_off_dev, int ctas, int64_t n_active_pad, int64_t d, cudaStream_t st) {
  if (n_active_pad == 0 || ctas <= 0) return cudaSuccess;
  retile_items_kernel<<<dim3(64, ctas), 256, 0, st>>>(kind, static_cast<const uint4*>(Wgu), static_cast<const uint4*>(WdT),
                                                      static_cast<uint8_t*>(tiled), bounds_dev, a_off_dev, n_active_pad, d);
  if (kind == kDecTiledStack) {
    const int64_t total = ((d + 255) / 256) * (n_active_pad / 64) * 2048;
    retile_down_chunks_kernel<<<cdiv(total, 256), 256, 0, st>>>(
        static_cast<const uint4*>(WdT), reinterpret_cast<uint4*>(static_cast<uint8_t*>(tiled) + decode_tiled_b_base(n_active_pad, d)),
        n_active_pad, d, total);
  }
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
  if (out_elem_size == 2)
    return launch_pdl(rmsnorm_kernel<true>, dim3(cdiv(n, 8)), dim3(256), 0, st, x, r, n, d, eps);
  return launch_pdl(rmsnorm_kernel<false>, dim3(cdiv(n, 8)), dim3(256), 0, st, x, r, n, d, eps);
}

}  // namespace mlpmoe
