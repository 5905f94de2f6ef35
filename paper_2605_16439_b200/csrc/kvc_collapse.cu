// Load-time collapse of a factored key reconstructor (kvc_collapse_theta).  Sec. 3.1 calls the reconstructor a two-layer
// network; Alg. 1 applies one matrix theta[h] (m x n) per KV head to the compressed scores, which is exact when the two
// layers are linear along the token axis: theta[h] = W1[h] W2[h], W1 (m x k), W2 (k x n).  The product is taken once,
// before decoding, with fp32 accumulation and one rounding to the storage type.  Plain shared-memory tiling: this runs
// once per (layer, ratio), not on the decode path.
#include <cuda_bf16.h>

#include "kvc_internal.cuh"

namespace kvc {

constexpr int CL_TILE = 64, CL_K = 16;

__device__ __forceinline__ float cl_load(const float* p) { return *p; }
__device__ __forceinline__ float cl_load(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void cl_store(float* p, float v) { *p = v; }
__device__ __forceinline__ void cl_store(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// grid (ceil(n/64), ceil(m/64), H_kv), 256 threads: thread (ty, tx) owns rows ty + 16 i, columns tx + 16 j of the tile
template <typename T>
__global__ void __launch_bounds__(256) collapse_theta_kernel(const T* __restrict__ W1, const T* __restrict__ W2, T* __restrict__ theta,
                                                             int m, int k, int n) {
  __shared__ float a_sm[CL_K][CL_TILE + 1];   // [kk][row]
  __shared__ float b_sm[CL_K][CL_TILE + 1];   // [kk][column]
  const int h = blockIdx.z, row0 = blockIdx.y * CL_TILE, col0 = blockIdx.x * CL_TILE;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const T* A = W1 + (size_t)h * m * k;
  const T* B = W2 + (size_t)h * k * n;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < k; k0 += CL_K) {
    for (int e = threadIdx.x; e < CL_TILE * CL_K; e += 256) {
      const int r = e / CL_K, kk = e % CL_K;                  // W1: k contiguous
      a_sm[kk][r] = (row0 + r < m && k0 + kk < k) ? cl_load(A + (size_t)(row0 + r) * k + k0 + kk) : 0.f;
      const int kb = e / CL_TILE, c = e % CL_TILE;            // W2: n contiguous
      b_sm[kb][c] = (k0 + kb < k && col0 + c < n) ? cl_load(B + (size_t)(k0 + kb) * n + col0 + c) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < CL_K; ++kk) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { av[i] = a_sm[kk][ty + 16 * i]; bv[i] = b_sm[kk][tx + 16 * i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
  T* out = theta + (size_t)h * m * n;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int r = row0 + ty + 16 * i, c = col0 + tx + 16 * j;
      if (r < m && c < n) cl_store(out + (size_t)r * n + c, acc[i][j]);
    }
}

cudaError_t launch_collapse_theta(const void* W1, const void* W2, void* theta, int H_kv, int m, int k, int n, int dtype,
                                  cudaStream_t st) {
  const dim3 grid((unsigned)ceil_div(n, CL_TILE), (unsigned)ceil_div(m, CL_TILE), (unsigned)H_kv);
  if (dtype == KVC_BF16)
    collapse_theta_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(W1), static_cast<const __nv_bfloat16*>(W2),
                                                              static_cast<__nv_bfloat16*>(theta), m, k, n);
  else
    collapse_theta_kernel<float><<<grid, 256, 0, st>>>(static_cast<const float*>(W1), static_cast<const float*>(W2),
                                                      static_cast<float*>(theta), m, k, n);
  return cudaGetLastError();
}

}  // namespace kvc
