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
// A (sequence, KV head) of the source has `pitch` rows (R n for a uniform batch).  idx == nullptr copies the first m
// rows of every block (m = n: a side stored verbatim); R_b != nullptr gives the blocks each sequence has (the others
// are left untouched).
template <typename T>
__global__ void __launch_bounds__(256) gather_keys_kernel(const T* __restrict__ K_vis, T* __restrict__ Kc,
                                                          const int32_t* __restrict__ idx, int H_kv, int R,
                                                          int n, int m, long long total_rows, long long pitch,
                                                          const int* __restrict__ R_b) {
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
  const int src = idx ? idx[h * m + j] : j;
  const long long blk = bhr % R, seq_head = bhr / R;
  if (R_b && blk >= R_b[seq_head / H_kv]) return;
  const uint4 v = __ldg(reinterpret_cast<const uint4*>(K_vis + (seq_head * pitch + vision_row(blk, n, src)) * D + c * EPV));
  *reinterpret_cast<uint4*>(Kc + row * D + c * EPV) = v;
}

// V_tilde tile [32 rows j][D] of one block = U[h][j0:j0+32, :] (V_blk - 1 mu^T), fp32 CUDA cores.
// Centering is applied when the V tile is staged, in the paper's order (centre, then project).
template <typename T>
__global__ void __launch_bounds__(256) project_values_kernel(const T* __restrict__ V_vis, T* __restrict__ Vc,
                                                             const T* __restrict__ U, const T* __restrict__ mu,
                                                             int H_kv, int R, int n, int m, long long pitch,
                                                             const int* __restrict__ R_b) {
  __shared__ float Usm[32][33];
  __shared__ float Vsm[32][D];
  const int bhr = blockIdx.x, j0 = blockIdx.y * 32;
  const int h = (bhr / R) % H_kv;
  if (R_b && bhr % R >= R_b[bhr / R / H_kv]) return;              // a block this sequence does not have
  const int tid = threadIdx.x, c = tid & (D - 1), jg = tid >> 7;   // 2 groups of 16 rows
  const T* Vb = V_vis + ((size_t)(bhr / R) * pitch + (size_t)vision_row(bhr % R, n, 0)) * D;
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
      static_cast<const T*>(K_vis), static_cast<T*>(Kc), L->d_idx, H_kv, R, n, m, total_rows, (long long)R * n, nullptr);
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
                                                 static_cast<const T*>(L->desc.mu), H_kv, R, n, m, (long long)R * n, nullptr);
  return cudaGetLastError();
}

// ---- batches with per-sequence lengths ---------------------------------------------------------------------------
// Sequence b has N_v[b] vision rows: R_b[b] = floor(N_v[b] / n) whole blocks are compressed, the N_v[b] mod n rows
// left over stay uncompressed and become the first T_b[b] rows of the caller's text buffers.  Lengths that do not
// fit (N_v[b] outside [0, N_cap], more than R_max blocks, more than T_cap rows left over) are clamped and reported.
__global__ void ragged_lengths_kernel(const int* __restrict__ N_v, int B, int n, int N_cap, int R_max, int T_cap,
                                      int* __restrict__ R_b, int* __restrict__ T_b, int* status) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  int nv = N_v[b];
  bool bad = nv < 0 || nv > N_cap;
  nv = nv < 0 ? 0 : (nv > N_cap ? N_cap : nv);
  int r = nv / n, t = nv - r * n;
  if (r > R_max) { bad = true; r = R_max; t = 0; }
  if (t > T_cap) { bad = true; t = T_cap; }
  R_b[b] = r;
  T_b[b] = t;
  if (bad) atomicExch(status, (int)KVC_ERR_BOUNDS);
}

// rows [R_b n, R_b n + T_b) of a (sequence, KV head)'s vision K and V -> rows [0, T_b) of its text buffers
template <typename T>
__global__ void __launch_bounds__(256) copy_tail_kernel(const T* __restrict__ K_vis, const T* __restrict__ V_vis,
                                                        T* __restrict__ K_tail, T* __restrict__ V_tail,
                                                        const int* __restrict__ R_b, const int* __restrict__ T_b,
                                                        int H_kv, int n, long long N_cap, long long T_cap) {
  constexpr int EPV = Elems16<T>::N;
  constexpr int LPR = D / EPV;
  const int bh = blockIdx.x, b = bh / H_kv;
  const int rows = T_b[b];
  const long long first = (long long)R_b[b] * n;
  for (int x = blockIdx.y * blockDim.x + threadIdx.x; x < rows * LPR; x += gridDim.y * blockDim.x) {
    const int row = x / LPR, c = x - row * LPR;
    const size_t so = ((size_t)bh * N_cap + first + row) * D + c * EPV, dst = ((size_t)bh * T_cap + row) * D + c * EPV;
    *reinterpret_cast<uint4*>(K_tail + dst) = __ldg(reinterpret_cast<const uint4*>(K_vis + so));
    *reinterpret_cast<uint4*>(V_tail + dst) = __ldg(reinterpret_cast<const uint4*>(V_vis + so));
  }
}

template <typename T>
static cudaError_t launch_ragged_t(const kvc_layer* L, const void* K_vis, const void* V_vis, int B, int N_cap,
                                   const int* N_v, int R_max, void* Kc, void* Vc, void* K_tail, void* V_tail, int T_cap,
                                   int* R_b, int* T_b, cudaStream_t st) {
  constexpr int RPI = 32 / (D / Elems16<T>::N);
  const int H_kv = L->desc.H_kv, n = L->desc.n;
  ragged_lengths_kernel<<<ceil_div(B, 128), 128, 0, st>>>(N_v, B, n, N_cap, R_max, T_cap, R_b, T_b, L->d_cstatus);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (R_max > 0) {
    // key side: the retained rows, or all n rows of a block when the side is stored verbatim
    {
      const bool verbatim = L->passthrough || L->mode == KVC_MODE_V_ONLY;
      const long long total_rows = (long long)B * H_kv * R_max * L->mk;
      ProfScope prof(KVC_KERNEL_GATHER_KEYS, st);
      gather_keys_kernel<T><<<(unsigned)(((total_rows + RPI - 1) / RPI + 7) / 8), 256, 0, st>>>(
          static_cast<const T*>(K_vis), static_cast<T*>(Kc), verbatim ? nullptr : L->d_idx, H_kv, R_max, n, L->mk, total_rows,
          (long long)N_cap, R_b);
      e = cudaGetLastError();
      if (e != cudaSuccess) return e;
    }
    ProfScope prof(KVC_KERNEL_PROJECT_VALUES, st);
    if (L->passthrough || L->mode == KVC_MODE_K_ONLY) {
      const long long total_rows = (long long)B * H_kv * R_max * n;
      gather_keys_kernel<T><<<(unsigned)(((total_rows + RPI - 1) / RPI + 7) / 8), 256, 0, st>>>(
          static_cast<const T*>(V_vis), static_cast<T*>(Vc), nullptr, H_kv, R_max, n, n, total_rows, (long long)N_cap, R_b);
    } else {
      dim3 grid((unsigned)(B * H_kv * R_max), (unsigned)ceil_div(L->m, 32));
      project_values_kernel<T><<<grid, 256, 0, st>>>(static_cast<const T*>(V_vis), static_cast<T*>(Vc),
                                                     static_cast<const T*>(L->desc.U), static_cast<const T*>(L->desc.mu),
                                                     H_kv, R_max, n, L->m, (long long)N_cap, R_b);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  if (T_cap > 0) {
    const int per = ceil_div((n - 1) * (D / Elems16<T>::N), 256);
    copy_tail_kernel<T><<<dim3((unsigned)(B * H_kv), (unsigned)(per < 1 ? 1 : per)), 256, 0, st>>>(
        static_cast<const T*>(K_vis), static_cast<const T*>(V_vis), static_cast<T*>(K_tail), static_cast<T*>(V_tail), R_b, T_b,
        H_kv, n, N_cap, T_cap);
    e = cudaGetLastError();
  }
  return e;
}

cudaError_t launch_compress_ragged(const kvc_layer* L, const void* K_vis, const void* V_vis, int B, int N_cap,
                                   const int* N_v, int R_max, void* Kc, void* Vc, void* K_tail, void* V_tail, int T_cap,
                                   int* R_b, int* T_b, cudaStream_t st) {
  return L->desc.dtype == KVC_BF16
             ? launch_ragged_t<__nv_bfloat16>(L, K_vis, V_vis, B, N_cap, N_v, R_max, Kc, Vc, K_tail, V_tail, T_cap, R_b, T_b, st)
             : launch_ragged_t<float>(L, K_vis, V_vis, B, N_cap, N_v, R_max, Kc, Vc, K_tail, V_tail, T_cap, R_b, T_b, st);
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
