// fp32 mode of the layer (Section 3.1 equations in plain FMA arithmetic): used when the
// weights are fp32.  Two tiled kernels over the same packed operands as the tensor-core path:
//   gate|up:  H[t, j] = silu(sum_k X[t,k] Wg'[j,k]) * (sum_k X[t,k] Wu'[j,k]) * scale[j]
//   down:     Y[t, m] = (R[t, m] +) sum_j H[t, j] WdT[m, j]      (all surviving branches in one sum)
#include "internal.h"

namespace mlpmoe {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, THREADS = 256;

// Loads a 64 x 16 tile of a K-major matrix (row pitch ld) into smem as [k][row], zero-filling
// rows >= rows_total and k >= K.  256 threads, one float4 each.
__device__ __forceinline__ void load_tile(const float* __restrict__ M, int64_t row0, int64_t rows_total, int64_t ld, int64_t k0,
                                          int64_t K, float (*s)[BM + 4]) {
  const int r = threadIdx.x / 4, kq = (threadIdx.x % 4) * 4;
  const int64_t row = row0 + r, k = k0 + kq;
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (row < rows_total && k < K) v = *reinterpret_cast<const float4*>(M + row * ld + k);
  s[kq + 0][r] = v.x;
  s[kq + 1][r] = v.y;
  s[kq + 2][r] = v.z;
  s[kq + 3][r] = v.w;
}

__global__ void __launch_bounds__(THREADS) simt_gateup_kernel(const float* __restrict__ X, const float* __restrict__ Wgu,
                                                              const float* __restrict__ scale, float* __restrict__ H,
                                                              int64_t n, int64_t d, int64_t Ipad) {
  __shared__ float As[BK][BM + 4], Bg[BK][BN + 4], Bu[BK][BN + 4];
  const int64_t t0 = static_cast<int64_t>(blockIdx.y) * BM;
  const int64_t j0 = static_cast<int64_t>(blockIdx.x) * BN;          // compacted neuron index
  const int64_t q = j0 / kGroup, jin = j0 % kGroup;                    // a 64-neuron tile never straddles a group
  const int64_t grow = q * 2 * kGroup + jin, urow = grow + kGroup;     // packed rows of the gate / up weights
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  float ag[4][4] = {}, au[4][4] = {};
  for (int64_t k0 = 0; k0 < d; k0 += BK) {
    load_tile(X, t0, n, d, k0, d, As);
    load_tile(Wgu, grow, 2 * Ipad, d, k0, d, Bg);
    load_tile(Wgu, urow, 2 * Ipad, d, k0, d, Bu);
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float a[4], bg[4], bu[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        a[i] = As[k][ty * 4 + i];
        bg[i] = Bg[k][tx * 4 + i];
        bu[i] = Bu[k][tx * 4 + i];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          ag[i][j] = fmaf(a[i], bg[j], ag[i][j]);
          au[i][j] = fmaf(a[i], bu[j], au[i][j]);
        }
    }
    __syncthreads();
  }
  const float4 sc = *reinterpret_cast<const float4*>(scale + j0 + tx * 4);
  const float s[4] = {sc.x, sc.y, sc.z, sc.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t t = t0 + ty * 4 + i;
    if (t >= n) continue;
    float h[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float g = ag[i][j];
      h[j] = (g / (1.0f + expf(-g))) * au[i][j] * s[j];
    }
    *reinterpret_cast<float4*>(H + t * Ipad + j0 + tx * 4) = make_float4(h[0], h[1], h[2], h[3]);
  }
}

__global__ void __launch_bounds__(THREADS) simt_down_kernel(const float* __restrict__ H, const float* __restrict__ WdT,
                                                            const float* __restrict__ R, float* __restrict__ Y, int64_t n,
                                                            int64_t d, int64_t K) {
  __shared__ float As[BK][BM + 4], Bs[BK][BN + 4];
  const int64_t t0 = static_cast<int64_t>(blockIdx.y) * BM;
  const int64_t m0 = static_cast<int64_t>(blockIdx.x) * BN;
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  float acc[4][4] = {};
  for (int64_t k0 = 0; k0 < K; k0 += BK) {
    load_tile(H, t0, n, K, k0, K, As);
    load_tile(WdT, m0, d, K, k0, K, Bs);
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        a[i] = As[k][ty * 4 + i];
        b[i] = Bs[k][tx * 4 + i];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t t = t0 + ty * 4 + i;
    const int64_t m = m0 + tx * 4;
    if (t >= n || m >= d) continue;     // d is a multiple of 4, so a float4 is all-in or all-out
    float4 v = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    if (R != nullptr) {
      const float4 r = *reinterpret_cast<const float4*>(R + t * d + m);
      v.x += r.x; v.y += r.y; v.z += r.z; v.w += r.w;
    }
    *reinterpret_cast<float4*>(Y + t * d + m) = v;
  }
}

}  // namespace

cudaError_t launch_simt_gateup(const float* X, const float* Wgu, const float* scale, float* H, int64_t n, int64_t d,
                               int64_t Ipad, cudaStream_t st) {
  if (n == 0 || Ipad == 0) return cudaSuccess;
  dim3 grid(static_cast<unsigned>(Ipad / BN), static_cast<unsigned>((n + BM - 1) / BM));
  simt_gateup_kernel<<<grid, THREADS, 0, st>>>(X, Wgu, scale, H, n, d, Ipad);
  return cudaGetLastError();
}

cudaError_t launch_simt_down(const float* H, const float* WdT, const float* R, float* Y, int64_t n, int64_t d, int64_t K,
                             cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  dim3 grid(static_cast<unsigned>((d + BN - 1) / BN), static_cast<unsigned>((n + BM - 1) / BM));
  simt_down_kernel<<<grid, THREADS, 0, st>>>(H, WdT, R, Y, n, d, K);
  return cudaGetLastError();
}

}  // namespace mlpmoe
