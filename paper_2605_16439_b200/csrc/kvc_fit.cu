// Parameter fits from activations, on the device and in fp64 (calibration-time work, not the decode path):
//   FitValuePCA (App. C, Alg. 2; Sec. 3.1 "Sequence-Level Low-Rank Compression for Values"): mu = mean over the pooled
//     blocks and their n positions, U = the top m eigenvectors of the n x n token covariance of the centred values
//     (= the top m left singular vectors of the pooled centred columns);
//   the key reconstructor for a fixed retained index set as the minimiser of the reconstruction term of Alg. 2:
//     theta = (K_r K_r^T)^+ K_r K^T with K_r the retained rows, the pseudo-inverse taken through the eigen-decomposition.
// Both rest on one hand-written solver: the cyclic Jacobi method for symmetric matrices with the round-robin ordering,
// in which the n/2 rotations of a round act on disjoint index pairs, so a round is one data-parallel update
// A <- J^T A J, Q <- Q J in which every 2 x 2 block of A is transformed in place by the rotations of its row pair and
// its column pair.
#include <vector>

#include "kvc_internal.cuh"

namespace kvc {

constexpr int FIT_TILE = 64;            // covariance tile per CTA
constexpr int FIT_KC = 32;              // channels per staged chunk
constexpr int FIT_MAX_SWEEPS = 40;
constexpr double FIT_OFF_TOL2 = 1e-22;  // stop when (off-diagonal norm / diagonal norm)^2 falls below this

static inline int even_up(int x) { return (x + 1) & ~1; }

// per-head regions of the fit workspace, in doubles
struct FitLayout {
  int ne;                 // n rounded up to even (the Jacobi pairing needs an even size; the extra index is all zero)
  size_t mat;             // ne * ne
  size_t off_M[4];        // four ne x ne matrices
  size_t off_lam;         // [ne]
  size_t off_inv;         // [ne]
  size_t off_rot;         // [ne] as double2 [ne / 2]
  size_t off_order;       // [ne] ints (in a region of ne doubles)
  size_t off_idx;         // [ne] ints
  size_t off_norm;        // [2]: off-diagonal and diagonal sums of squares
  size_t off_sum;         // [D]
  size_t per_head;
};

static FitLayout fit_layout(int n) {
  FitLayout f{};
  f.ne = even_up(n);
  f.mat = (size_t)f.ne * f.ne;
  size_t off = 0;
  for (int i = 0; i < 4; ++i) { f.off_M[i] = off; off += f.mat; }
  f.off_lam = off; off += f.ne;
  f.off_inv = off; off += f.ne;
  f.off_rot = off; off += f.ne;
  f.off_order = off; off += f.ne;
  f.off_idx = off; off += f.ne;
  f.off_norm = off; off += 2;
  f.off_sum = off; off += D;
  f.per_head = (off + 31) / 32 * 32;
  return f;
}

// ---- pooled sums and second moments ---------------------------------------------------------------------------
// sum[h][c] += sum over sequences and rows of X[b, h, row, c]
template <typename T>
__global__ void __launch_bounds__(256) fit_sum_kernel(const T* __restrict__ X, int B, int H_kv, long long rows, double* sum,
                                                      size_t head_stride) {
  const int h = blockIdx.x, c = threadIdx.x & (D - 1);
  const long long total = (long long)B * rows;
  double acc = 0.0;
  for (long long rr = (long long)blockIdx.y * 2 + (threadIdx.x >> 7); rr < total; rr += (long long)gridDim.y * 2) {
    const long long b = rr / rows, i = rr - b * rows;
    acc += (double)to_f32(X[((b * H_kv + h) * rows + i) * D + c]);
  }
  atomicAdd(sum + (size_t)h * head_stride + c, acc);
}

// C[h][i][j] = sum over blocks s and channels c of (X_s[i][c] - mu_c)(X_s[j][c] - mu_c), mu = sum / count (0 if !center)
template <typename T>
__global__ void __launch_bounds__(256) fit_moment_kernel(const T* __restrict__ X, int B, int R, int H_kv, int n, int ne,
                                                         double* __restrict__ ws, size_t head_stride, size_t off_C,
                                                         size_t off_sum, int center) {
  __shared__ double As[FIT_KC][FIT_TILE + 1], Bs[FIT_KC][FIT_TILE + 1];
  __shared__ double mu[D];
  const int h = blockIdx.z, i0 = blockIdx.y * FIT_TILE, j0 = blockIdx.x * FIT_TILE;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  double* C = ws + (size_t)h * head_stride + off_C;
  if (tid < D) mu[tid] = center ? ws[(size_t)h * head_stride + off_sum + tid] / ((double)B * R * n) : 0.0;
  __syncthreads();
  double acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;
  const int lrow = tid >> 2, lc = (tid & 3) * 8;          // staging: 64 rows x 4 groups of 8 channels
  for (int s = 0; s < B * R; ++s) {
    const int b = s / R, r = s - b * R;
    const T* blk = X + (((size_t)b * H_kv + h) * R + r) * (size_t)n * D;
    for (int c0 = 0; c0 < D; c0 += FIT_KC) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int c = c0 + lc + e;
        As[lc + e][lrow] = i0 + lrow < n ? (double)to_f32(blk[(size_t)(i0 + lrow) * D + c]) - mu[c] : 0.0;
        Bs[lc + e][lrow] = j0 + lrow < n ? (double)to_f32(blk[(size_t)(j0 + lrow) * D + c]) - mu[c] : 0.0;
      }
      __syncthreads();
#pragma unroll 8
      for (int k = 0; k < FIT_KC; ++k) {
        double av[4], bv[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) { av[e] = As[k][ty * 4 + e]; bv[e] = Bs[k][tx * 4 + e]; }
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int bb = 0; bb < 4; ++bb) acc[a][bb] = fma(av[a], bv[bb], acc[a][bb]);
      }
      __syncthreads();
    }
  }
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int bb = 0; bb < 4; ++bb) {
      const int i = i0 + ty * 4 + a, j = j0 + tx * 4 + bb;
      if (i < n && j < n) C[(size_t)i * ne + j] = acc[a][bb];
    }
}

// ---- cyclic Jacobi with the round-robin ordering --------------------------------------------------------------
// Round k of a sweep over an even number ne of indices: index ne-1 meets k; (k + j) mod (ne-1) meets (k - j) mod (ne-1).
__device__ __forceinline__ void round_pair(int k, int j, int ne, int& p, int& q) {
  const int nm1 = ne - 1;
  int a, b;
  if (j == 0) { a = nm1; b = k; }
  else { a = (k + j) % nm1; b = (k - j + nm1) % nm1; }
  p = a < b ? a : b;
  q = a < b ? b : a;
}

__global__ void jacobi_rotations_kernel(const double* __restrict__ ws, size_t head_stride, size_t off_A, size_t off_rot,
                                        int ne, int k, double* ws_out) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x, h = blockIdx.y;
  if (j >= ne / 2) return;
  const double* A = ws + (size_t)h * head_stride + off_A;
  int p, q;
  round_pair(k, j, ne, p, q);
  const double app = A[(size_t)p * ne + p], aqq = A[(size_t)q * ne + q], apq = A[(size_t)p * ne + q];
  double c = 1.0, s = 0.0;
  if (fabs(apq) > 1e-300 && fabs(apq) > 1e-18 * sqrt(fabs(app) * fabs(aqq))) {
    const double th = (aqq - app) / (2.0 * apq);
    const double t = (th >= 0.0 ? 1.0 : -1.0) / (fabs(th) + sqrt(th * th + 1.0));
    c = 1.0 / sqrt(t * t + 1.0);
    s = t * c;
  }
  double2* rot = reinterpret_cast<double2*>(ws_out + (size_t)h * head_stride + off_rot);
  rot[j] = make_double2(c, s);
}

// A <- J^T A J on the 2 x 2 block (row pair ja, column pair jb); Q <- Q J on rows (2 ja, 2 ja + 1), column pair jb
__global__ void __launch_bounds__(128) jacobi_apply_kernel(double* __restrict__ ws, size_t head_stride, size_t off_A,
                                                           size_t off_Q, size_t off_rot, int ne, int k) {
  const int jb = blockIdx.x * blockDim.x + threadIdx.x, ja = blockIdx.y, h = blockIdx.z;
  if (jb >= ne / 2) return;
  double* A = ws + (size_t)h * head_stride + off_A;
  double* Q = ws + (size_t)h * head_stride + off_Q;
  const double2* rot = reinterpret_cast<const double2*>(ws + (size_t)h * head_stride + off_rot);
  int p, q, pc, qc;
  round_pair(k, ja, ne, p, q);
  round_pair(k, jb, ne, pc, qc);
  const double2 ra = rot[ja], rb = rot[jb];
  const double b00 = A[(size_t)p * ne + pc], b01 = A[(size_t)p * ne + qc];
  const double b10 = A[(size_t)q * ne + pc], b11 = A[(size_t)q * ne + qc];
  // rows: J_a^T B
  const double x00 = ra.x * b00 - ra.y * b10, x01 = ra.x * b01 - ra.y * b11;
  const double x10 = ra.y * b00 + ra.x * b10, x11 = ra.y * b01 + ra.x * b11;
  // columns: (.) J_b
  double y00 = rb.x * x00 - rb.y * x01, y01 = rb.y * x00 + rb.x * x01;
  double y10 = rb.x * x10 - rb.y * x11, y11 = rb.y * x10 + rb.x * x11;
  if (ja == jb) { y01 = 0.0; y10 = 0.0; }                      // the annihilated pair, exactly
  A[(size_t)p * ne + pc] = y00; A[(size_t)p * ne + qc] = y01;
  A[(size_t)q * ne + pc] = y10; A[(size_t)q * ne + qc] = y11;
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const size_t row = (size_t)(2 * ja + e) * ne;
    const double u = Q[row + pc], v = Q[row + qc];
    Q[row + pc] = rb.x * u - rb.y * v;
    Q[row + qc] = rb.y * u + rb.x * v;
  }
}

__global__ void __launch_bounds__(256) fit_norms_kernel(double* __restrict__ ws, size_t head_stride, size_t off_A,
                                                        size_t off_norm, int ne) {
  __shared__ double red[2][8];
  const int h = blockIdx.y;
  const double* A = ws + (size_t)h * head_stride + off_A;
  double off = 0.0, dg = 0.0;
  for (size_t x = (size_t)blockIdx.x * 256 + threadIdx.x; x < (size_t)ne * ne; x += (size_t)gridDim.x * 256) {
    const size_t i = x / ne, j = x - i * ne;
    const double v = A[x];
    if (i == j) dg += v * v; else off += v * v;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    off += __shfl_xor_sync(0xffffffffu, off, o);
    dg += __shfl_xor_sync(0xffffffffu, dg, o);
  }
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = off; red[1][threadIdx.x >> 5] = dg; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) { off += red[0][w]; dg += red[1][w]; }
    atomicAdd(ws + (size_t)h * head_stride + off_norm, off);
    atomicAdd(ws + (size_t)h * head_stride + off_norm + 1, dg);
  }
}

__global__ void fit_identity_kernel(double* __restrict__ ws, size_t head_stride, size_t off_Q, int ne) {
  const int h = blockIdx.y;
  double* Q = ws + (size_t)h * head_stride + off_Q;
  for (size_t x = (size_t)blockIdx.x * blockDim.x + threadIdx.x; x < (size_t)ne * ne; x += (size_t)gridDim.x * blockDim.x)
    Q[x] = (x / ne == x % ne) ? 1.0 : 0.0;
}

// eigenvalues = the diagonal; order[rank] = index, descending (ties by index; indices >= n_valid go last)
__global__ void fit_rank_kernel(double* __restrict__ ws, size_t head_stride, size_t off_A, size_t off_lam, size_t off_order,
                                int ne, int n_valid) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x, h = blockIdx.y;
  if (i >= ne) return;
  const double* A = ws + (size_t)h * head_stride + off_A;
  double* lam = ws + (size_t)h * head_stride + off_lam;
  int* order = reinterpret_cast<int*>(ws + (size_t)h * head_stride + off_order);
  const double li = A[(size_t)i * ne + i];
  int rank = 0;
  for (int j = 0; j < ne; ++j) {
    const double lj = A[(size_t)j * ne + j];
    const bool vi = i < n_valid, vj = j < n_valid;
    const bool before = (vj && !vi) || (vi == vj && (lj > li || (lj == li && j < i)));
    rank += before ? 1 : 0;
  }
  order[rank] = i;
  lam[i] = li;
}

// U[h][j][:] = eigenvector of rank j, sign fixed so that its entry of largest magnitude is positive
template <typename T>
__global__ void __launch_bounds__(128) fit_emit_basis_kernel(const double* __restrict__ ws, size_t head_stride, size_t off_Q,
                                                             size_t off_lam, size_t off_order, int ne, int n, int m,
                                                             T* __restrict__ U, double* __restrict__ eig) {
  __shared__ double best[4];
  __shared__ double sgn_s;
  const int j = blockIdx.x, h = blockIdx.y, tid = threadIdx.x;
  const double* Q = ws + (size_t)h * head_stride + off_Q;
  const int* order = reinterpret_cast<const int*>(ws + (size_t)h * head_stride + off_order);
  const int col = order[j];
  if (eig && tid == 0) eig[(size_t)h * n + j] = ws[(size_t)h * head_stride + off_lam + col];
  if (j >= m) return;
  double bv = 0.0;                       // entry of largest magnitude (first one on ties)
  for (int i = tid; i < n; i += 128) {
    const double v = Q[(size_t)i * ne + col];
    if (fabs(v) > fabs(bv)) bv = v;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const double ov = __shfl_xor_sync(0xffffffffu, bv, o);
    if (fabs(ov) > fabs(bv)) bv = ov;
  }
  if ((tid & 31) == 0) best[tid >> 5] = bv;
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < 4; ++w) if (fabs(best[w]) > fabs(bv)) bv = best[w];
    sgn_s = bv < 0.0 ? -1.0 : 1.0;
  }
  __syncthreads();
  const double sg = sgn_s;
  for (int i = tid; i < n; i += 128) store_elem(U + ((size_t)h * m + j) * n + i, (float)(sg * Q[(size_t)i * ne + col]));
}

template <typename T>
__global__ void fit_emit_mean_kernel(const double* __restrict__ ws, size_t head_stride, size_t off_sum, double count,
                                     T* __restrict__ mu) {
  const int h = blockIdx.x, c = threadIdx.x;
  store_elem(mu + h * D + c, (float)(ws[(size_t)h * head_stride + off_sum + c] / count));
}

// ---- least-squares pieces ------------------------------------------------------------------------------------
// A[j][j'] = C[idx[j]][idx[j']] (me x me, zero beyond m)
__global__ void fit_select_kernel(double* __restrict__ ws, size_t head_stride, size_t off_C, size_t off_A, size_t off_idx,
                                  int ne, int me, int m) {
  const int h = blockIdx.y;
  const double* C = ws + (size_t)h * head_stride + off_C;
  double* A = ws + (size_t)h * head_stride + off_A;
  const int* idx = reinterpret_cast<const int*>(ws + (size_t)h * head_stride + off_idx);
  for (size_t x = (size_t)blockIdx.x * blockDim.x + threadIdx.x; x < (size_t)me * me; x += (size_t)gridDim.x * blockDim.x) {
    const int j = (int)(x / me), k = (int)(x % me);
    A[x] = (j < m && k < m) ? C[(size_t)idx[j] * ne + idx[k]] : 0.0;
  }
}

// inv[i] = 1 / lam[i] where lam[i] > rcond * max lam, else 0 (one block per head)
__global__ void __launch_bounds__(256) fit_pinv_kernel(double* __restrict__ ws, size_t head_stride, size_t off_A, size_t off_inv,
                                                       int me, int m, double rcond) {
  __shared__ double red[8];
  const int h = blockIdx.x, tid = threadIdx.x;
  const double* A = ws + (size_t)h * head_stride + off_A;
  double mx = 0.0;
  for (int i = tid; i < me; i += 256) mx = fmax(mx, A[(size_t)i * me + i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((tid & 31) == 0) red[tid >> 5] = mx;
  __syncthreads();
  mx = red[0];
  for (int w = 1; w < 8; ++w) mx = fmax(mx, red[w]);
  double* inv = ws + (size_t)h * head_stride + off_inv;
  for (int i = tid; i < me; i += 256) {
    const double l = A[(size_t)i * me + i];
    inv[i] = (l > 0.0 && l > rcond * mx) ? 1.0 / l : 0.0;
  }
  (void)m;
}

// T1[i][c] = inv[i] * sum_j Q[j][i] C[idx[j]][c]        (i < me, c < n)
__global__ void __launch_bounds__(256) fit_project_kernel(double* __restrict__ ws, size_t head_stride, size_t off_C, size_t off_Q,
                                                          size_t off_T, size_t off_inv, size_t off_idx, int ne, int me, int m,
                                                          int n) {
  __shared__ double Qs[16][17], Cs[16][17];
  const int h = blockIdx.z, i0 = blockIdx.y * 16, c0 = blockIdx.x * 16, ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
  const double* C = ws + (size_t)h * head_stride + off_C;
  const double* Q = ws + (size_t)h * head_stride + off_Q;
  const int* idx = reinterpret_cast<const int*>(ws + (size_t)h * head_stride + off_idx);
  double acc = 0.0;
  for (int j0 = 0; j0 < m; j0 += 16) {
    Qs[ty][tx] = (j0 + ty < m && i0 + tx < me) ? Q[(size_t)(j0 + ty) * me + i0 + tx] : 0.0;      // Qs[j][i]
    Cs[ty][tx] = (j0 + ty < m && c0 + tx < n) ? C[(size_t)idx[j0 + ty] * ne + c0 + tx] : 0.0;   // Cs[j][c]
    __syncthreads();
#pragma unroll
    for (int j = 0; j < 16; ++j) acc = fma(Qs[j][ty], Cs[j][tx], acc);
    __syncthreads();
  }
  if (i0 + ty < me && c0 + tx < n)
    ws[(size_t)h * head_stride + off_T + (size_t)(i0 + ty) * ne + c0 + tx] = acc * ws[(size_t)h * head_stride + off_inv + i0 + ty];
}

// theta[h][j][c] = sum_i Q[j][i] T1[i][c]
template <typename T>
__global__ void __launch_bounds__(256) fit_emit_theta_kernel(const double* __restrict__ ws, size_t head_stride, size_t off_Q,
                                                             size_t off_T, int ne, int me, int m, int n, T* __restrict__ theta) {
  __shared__ double Qs[16][17], Ts[16][17];
  const int h = blockIdx.z, j0 = blockIdx.y * 16, c0 = blockIdx.x * 16, ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
  const double* Q = ws + (size_t)h * head_stride + off_Q;
  const double* T1 = ws + (size_t)h * head_stride + off_T;
  double acc = 0.0;
  for (int i0 = 0; i0 < me; i0 += 16) {
    Qs[ty][tx] = (j0 + ty < m && i0 + tx < me) ? Q[(size_t)(j0 + ty) * me + i0 + tx] : 0.0;      // Qs[j][i]
    Ts[ty][tx] = (i0 + ty < me && c0 + tx < n) ? T1[(size_t)(i0 + ty) * ne + c0 + tx] : 0.0;    // Ts[i][c]
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 16; ++i) acc = fma(Qs[ty][i], Ts[i][tx], acc);
    __syncthreads();
  }
  if (j0 + ty < m && c0 + tx < n) store_elem(theta + ((size_t)h * m + j0 + ty) * n + c0 + tx, (float)acc);
}

// ---- host side -------------------------------------------------------------------------------------------------
// eigen-decomposition of the size x size matrices at off_A (overwritten by their diagonal form), eigenvectors to off_Q
static cudaError_t jacobi_eigen(double* ws, size_t head_stride, size_t off_A, size_t off_Q, size_t off_rot, size_t off_norm,
                                int H, int size, cudaStream_t st, int* sweeps_out) {
  fit_identity_kernel<<<dim3(64, H), 256, 0, st>>>(ws, head_stride, off_Q, size);
  cudaError_t e = cudaGetLastError();
  std::vector<double> norms((size_t)2 * H);
  int sweep = 0;
  for (; e == cudaSuccess && sweep < FIT_MAX_SWEEPS; ++sweep) {
    for (int h = 0; h < H && e == cudaSuccess; ++h)
      e = cudaMemsetAsync(ws + (size_t)h * head_stride + off_norm, 0, 2 * sizeof(double), st);
    if (e != cudaSuccess) break;
    fit_norms_kernel<<<dim3(32, H), 256, 0, st>>>(ws, head_stride, off_A, off_norm, size);
    for (int h = 0; h < H && e == cudaSuccess; ++h)
      e = cudaMemcpyAsync(&norms[2 * h], ws + (size_t)h * head_stride + off_norm, 2 * sizeof(double), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) break;
    bool done = true;
    for (int h = 0; h < H; ++h) done = done && !(norms[2 * h] > FIT_OFF_TOL2 * norms[2 * h + 1]);
    if (done) break;
    for (int k = 0; k < size - 1; ++k) {
      jacobi_rotations_kernel<<<dim3(ceil_div(size / 2, 128), H), 128, 0, st>>>(ws, head_stride, off_A, off_rot, size, k, ws);
      jacobi_apply_kernel<<<dim3(ceil_div(size / 2, 128), size / 2, H), 128, 0, st>>>(ws, head_stride, off_A, off_Q, off_rot, size, k);
    }
    e = cudaGetLastError();
  }
  if (sweeps_out) *sweeps_out = sweep;
  return e;
}

template <typename T>
static cudaError_t moments(const T* X, int B, int R, int H, int n, const FitLayout& f, double* ws, size_t off_C, bool center,
                           cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(ws, 0, (size_t)H * f.per_head * sizeof(double), st);
  if (e != cudaSuccess) return e;
  if (center) fit_sum_kernel<T><<<dim3(H, 64), 256, 0, st>>>(X, B, H, (long long)R * n, ws + f.off_sum, f.per_head);
  const int tiles = ceil_div(n, FIT_TILE);
  fit_moment_kernel<T><<<dim3(tiles, tiles, H), 256, 0, st>>>(X, B, R, H, n, f.ne, ws, f.per_head, off_C, f.off_sum, center ? 1 : 0);
  return cudaGetLastError();
}

template <typename T>
static cudaError_t fit_pca_t(const void* V_vis, int B, int R, int H, int n, int m, void* U_out, void* mu_out, double* eig_out,
                             double* ws, cudaStream_t st, int* sweeps) {
  const FitLayout f = fit_layout(n);
  cudaError_t e = moments<T>(static_cast<const T*>(V_vis), B, R, H, n, f, ws, f.off_M[0], true, st);
  if (e != cudaSuccess) return e;
  e = jacobi_eigen(ws, f.per_head, f.off_M[0], f.off_M[1], f.off_rot, f.off_norm, H, f.ne, st, sweeps);
  if (e != cudaSuccess) return e;
  fit_rank_kernel<<<dim3(ceil_div(f.ne, 128), H), 128, 0, st>>>(ws, f.per_head, f.off_M[0], f.off_lam, f.off_order, f.ne, n);
  fit_emit_basis_kernel<T><<<dim3(eig_out ? n : m, H), 128, 0, st>>>(ws, f.per_head, f.off_M[1], f.off_lam, f.off_order, f.ne, n, m,
                                                                     static_cast<T*>(U_out), eig_out);
  fit_emit_mean_kernel<T><<<H, D, 0, st>>>(ws, f.per_head, f.off_sum, (double)B * R * n, static_cast<T*>(mu_out));
  e = cudaGetLastError();
  return e != cudaSuccess ? e : cudaStreamSynchronize(st);
}

template <typename T>
static cudaError_t fit_theta_t(const void* K_vis, int B, int R, int H, int n, int m, const int32_t* idx, int idx_per_head,
                               double rcond, void* theta_out, double* ws, cudaStream_t st, int* sweeps) {
  const FitLayout f = fit_layout(n);
  const int me = even_up(m);
  cudaError_t e = moments<T>(static_cast<const T*>(K_vis), B, R, H, n, f, ws, f.off_M[0], false, st);
  for (int h = 0; h < H && e == cudaSuccess; ++h)
    e = cudaMemcpyAsync(ws + (size_t)h * f.per_head + f.off_idx, idx + (idx_per_head ? (size_t)h * m : 0), (size_t)m * sizeof(int32_t),
                        cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return e;
  fit_select_kernel<<<dim3(64, H), 256, 0, st>>>(ws, f.per_head, f.off_M[0], f.off_M[1], f.off_idx, f.ne, me, m);
  e = jacobi_eigen(ws, f.per_head, f.off_M[1], f.off_M[2], f.off_rot, f.off_norm, H, me, st, sweeps);
  if (e != cudaSuccess) return e;
  fit_pinv_kernel<<<H, 256, 0, st>>>(ws, f.per_head, f.off_M[1], f.off_inv, me, m, rcond);
  fit_project_kernel<<<dim3(ceil_div(n, 16), ceil_div(me, 16), H), 256, 0, st>>>(ws, f.per_head, f.off_M[0], f.off_M[2], f.off_M[3],
                                                                              f.off_inv, f.off_idx, f.ne, me, m, n);
  fit_emit_theta_kernel<T><<<dim3(ceil_div(n, 16), ceil_div(m, 16), H), 256, 0, st>>>(ws, f.per_head, f.off_M[2], f.off_M[3], f.ne, me, m,
                                                                                    n, static_cast<T*>(theta_out));
  e = cudaGetLastError();
  return e != cudaSuccess ? e : cudaStreamSynchronize(st);
}

}  // namespace kvc

using namespace kvc;

extern "C" {

size_t kvc_fit_workspace_bytes(int H_kv, int n) {
  if (H_kv < 1 || n < 1) return 0;
  return align_up((size_t)H_kv * fit_layout(n).per_head * sizeof(double), 256);
}

static int fit_args_ok(const void* X, int B, int R, int H_kv, int n, int m, int dtype, const void* out, const void* ws) {
  if (!X || !out || !ws) return KVC_ERR_ARG;
  if (B < 1 || R < 1 || H_kv < 1 || n < 1 || m < 1 || m > n || H_kv > 65535) return KVC_ERR_SHAPE;
  if (dtype != KVC_F32 && dtype != KVC_BF16) return KVC_ERR_DTYPE;
  if (reinterpret_cast<uintptr_t>(ws) & 255) return KVC_ERR_WORKSPACE;
  return KVC_OK;
}

int kvc_fit_value_pca(const void* V_vis, int B, int R, int H_kv, int n, int m, kvc_dtype dtype, void* U_out, void* mu_out,
                      double* eig_out, void* workspace, void* stream, int* sweeps_out) {
  const int s = fit_args_ok(V_vis, B, R, H_kv, n, m, (int)dtype, U_out, workspace);
  if (s != KVC_OK) return s;
  if (!mu_out) return KVC_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  double* ws = static_cast<double*>(workspace);
  return cuda_status(dtype == KVC_BF16
                         ? fit_pca_t<__nv_bfloat16>(V_vis, B, R, H_kv, n, m, U_out, mu_out, eig_out, ws, st, sweeps_out)
                         : fit_pca_t<float>(V_vis, B, R, H_kv, n, m, U_out, mu_out, eig_out, ws, st, sweeps_out));
}

int kvc_fit_key_reconstructor(const void* K_vis, int B, int R, int H_kv, int n, int m, const int32_t* idx, int idx_per_head,
                              double rcond, kvc_dtype dtype, void* theta_out, void* workspace, void* stream, int* sweeps_out) {
  const int s = fit_args_ok(K_vis, B, R, H_kv, n, m, (int)dtype, theta_out, workspace);
  if (s != KVC_OK) return s;
  if (!idx || !(rcond >= 0.0)) return KVC_ERR_ARG;
  for (int h = 0; h < (idx_per_head ? H_kv : 1); ++h)
    for (int j = 0; j < m; ++j) {
      const int32_t v = idx[(size_t)h * m + j];
      if (v < 0 || v >= n || (j > 0 && v <= idx[(size_t)h * m + j - 1])) return KVC_ERR_BOUNDS;
    }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  double* ws = static_cast<double*>(workspace);
  return cuda_status(dtype == KVC_BF16
                         ? fit_theta_t<__nv_bfloat16>(K_vis, B, R, H_kv, n, m, idx, idx_per_head, rcond, theta_out, ws, st, sweeps_out)
                         : fit_theta_t<float>(K_vis, B, R, H_kv, n, m, idx, idx_per_head, rcond, theta_out, ws, st, sweeps_out));
}

}  // extern "C"
