// Prefill-stage compression (Sec. 3.2): key row selection by the fixed index set and the
// sequence-level value projection V_tilde = U (V - 1 mu^T), one n-token block at a time.
#include "kvc_internal.cuh"

namespace kvc {

// Row of vision token (block r, offset i) inside a (sequence, KV head)'s vision K/V: the grouping of Alg. 1 step 1.
__host__ __device__ __forceinline__ long long vision_row(long long r, int n, int i) { return r * n + i; }

// (block, offset) of every vision token as the key selection addresses them: thread (r, i) writes to entry vision_row(r, n, i)
__global__ void export_groups_kernel(int32_t* __restrict__ out, int R, int n) {
  const long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= (long long)R * n) return;
  const int r = (int)(x / n), i = (int)(x - (long long)r * n);
  const long long t = vision_row(r, n, i);
  out[2 * t] = r;
  out[2 * t + 1] = i;
}

cudaError_t launch_export_groups(int32_t* d_out, int R, int n, cudaStream_t st) {
  const long long total = (long long)R * n;
  export_groups_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(d_out, R, n);
  return cudaGetLastError();
}

// K_tilde[b,h,r,j,:] = K_vis[b,h,r*n + idx[h][j],:].  One warp copies RPI rows per step.
template <typename T>
__global__ void __launch_bounds__(256) gather_keys_kernel(const T* __restrict__ K_vis, T* __restrict__ Kc,
                                                          const int32_t* __restrict__ idx, int H_kv, int R,
                                                          int n, int m, long long total_rows) {
  constexpr int EPV = Elems16<T>::N;
  constexpr int LPR = D / EPV;
  constexpr int RPI = 32 / LPR;
  const int lane = threadIdx.x & 31, sub = lane / LPR, c = lane % LPR;
  const long long warp = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const long long row = warp * RPI + sub;          // flat (b, h, r, j)
  if (row >= total_rows) return;
  const int j = (int)(row % m);
  const long long bhr = row / m;
  const int h = (int)((bhr / R) % H_kv);
  const int src = idx[h * m + j];
  const long long blk = bhr % R, seq_head = bhr / R;
  const uint4 v = __ldg(reinterpret_cast<const uint4*>(K_vis + (seq_head * R * n + vision_row(blk, n, src)) * D + c * EPV));
  *reinterpret_cast<uint4*>(Kc + row * D + c * EPV) = v;
}

// V_tilde tile [32 rows j][D] of one block = U[h][j0:j0+32, :] (V_blk - 1 mu^T), fp32 CUDA cores.
// Centering is applied when the V tile is staged, in the paper's order (centre, then project).
template <typename T>
__global__ void __launch_bounds__(256) project_values_kernel(const T* __restrict__ V_vis, T* __restrict__ Vc,
                                                             const T* __restrict__ U, const T* __restrict__ mu,
                                                             int H_kv, int R, int n, int m) {
  __shared__ float Usm[32][33];
  __shared__ float Vsm[32][D];
  const int bhr = blockIdx.x, j0 = blockIdx.y * 32;
  const int h = (bhr / R) % H_kv;
  const int tid = threadIdx.x, c = tid & (D - 1), jg = tid >> 7;   // 2 groups of 16 rows
  const T* Vb = V_vis + (size_t)bhr * n * D;
  const T* Uh = U + (size_t)h * m * n;
  const float mu_c = to_f32(mu[h * D + c]);
  float acc[16];
#pragma unroll
  for (int k = 0; k < 16; ++k) acc[k] = 0.f;
  for (int i0 = 0; i0 < n; i0 += 32) {
    for (int x = tid; x < 32 * 32; x += 256) {
      const int jj = x >> 5, ii = x & 31;
      Usm[jj][ii] = (j0 + jj < m && i0 + ii < n) ? to_f32(Uh[(size_t)(j0 + jj) * n + i0 + ii]) : 0.f;
    }
    for (int x = tid; x < 32 * D; x += 256) {
      const int ii = x >> 7, cc = x & (D - 1);
      Vsm[ii][cc] = (i0 + ii < n) ? to_f32(Vb[(size_t)(i0 + ii) * D + cc]) - to_f32(mu[h * D + cc]) : 0.f;
    }
    __syncthreads();
#pragma unroll 4
    for (int ii = 0; ii < 32; ++ii) {
      const float v = Vsm[ii][c];
#pragma unroll
      for (int k = 0; k < 16; ++k) acc[k] = fmaf(Usm[jg * 16 + k][ii], v, acc[k]);
    }
    __syncthreads();
  }
  (void)mu_c;
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    const int j = j0 + jg * 16 + k;
    if (j < m) store_elem(Vc + ((size_t)bhr * m + j) * D + c, acc[k]);
  }
}

template <typename T>
static cudaError_t launch_keys_t(const kvc_layer* L, const void* K_vis, int B, int R, void* Kc, cudaStream_t st) {
  constexpr int RPI = 32 / (D / Elems16<T>::N);
  const int H_kv = L->desc.H_kv, n = L->desc.n, m = L->m;
  const long long total_rows = (long long)B * H_kv * R * m;
  const long long warps = (total_rows + RPI - 1) / RPI;
  ProfScope prof(KVC_KERNEL_GATHER_KEYS, st);
  gather_keys_kernel<T><<<(unsigned)((warps + 7) / 8), 256, 0, st>>>(
      static_cast<const T*>(K_vis), static_cast<T*>(Kc), L->d_idx, H_kv, R, n, m, total_rows);
  return cudaGetLastError();
}

template <typename T>
static cudaError_t launch_values_t(const kvc_layer* L, const void* V_vis, int B, int R, void* Vc, cudaStream_t st) {
  const int H_kv = L->desc.H_kv, n = L->desc.n, m = L->m;
  cudaError_t e;
  ProfScope prof(KVC_KERNEL_PROJECT_VALUES, st);
  {
    bool used = false;
    e = launch_project_values_tc(L, V_vis, B, R, Vc, st, &used);       // bf16: tcgen05, accumulator in tensor memory
    if (used || e != cudaSuccess) return e;
    e = launch_project_values_mma(L, V_vis, B, R, Vc, st, &used);      // bf16: mma.sync (kept as the comparison kernel)
    if (used || e != cudaSuccess) return e;
  }
  dim3 grid((unsigned)(B * H_kv * R), (unsigned)ceil_div(m, 32));
  project_values_kernel<T><<<grid, 256, 0, st>>>(static_cast<const T*>(V_vis), static_cast<T*>(Vc),
                                                 static_cast<const T*>(L->desc.U),
                                                 static_cast<const T*>(L->desc.mu), H_kv, R, n, m);
  return cudaGetLastError();
}

cudaError_t launch_compress_keys(const kvc_layer* L, const void* K_vis, int B, int R, void* Kc, cudaStream_t st) {
  return L->desc.dtype == KVC_BF16 ? launch_keys_t<__nv_bfloat16>(L, K_vis, B, R, Kc, st)
                                   : launch_keys_t<float>(L, K_vis, B, R, Kc, st);
}
cudaError_t launch_compress_values(const kvc_layer* L, const void* V_vis, int B, int R, void* Vc, cudaStream_t st) {
  return L->desc.dtype == KVC_BF16 ? launch_values_t<__nv_bfloat16>(L, V_vis, B, R, Vc, st)
                                   : launch_values_t<float>(L, V_vis, B, R, Vc, st);
}

}  // namespace kvc
