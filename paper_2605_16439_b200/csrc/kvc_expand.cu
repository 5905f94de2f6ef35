// Steps 2 and 3 of Algorithm 1 for one KV head: L_img = S_full theta, P = exp(L_img - rowmax),
// W = P U^T.  Rows are the (sequence, query head in group, block) triples that share theta[h] and
// U[h]; every row keeps its own running maximum (the joint softmax over all blocks and the text is
// completed by the log-sum-exp merge of the output kernel), and the n axis may be split over
// several CTAs, each emitting an unnormalised partial (W, max, sum).
//
// This translation unit holds the CUDA-core fp32 version, used for fp32 storage (1e-4 parity) and
// as the fallback shape-agnostic path.  It also serves the one-sided variants (App. G): with verbatim
// keys the score row already has n entries and the expansion is the identity (id_theta); with verbatim
// values the weight row has n entries and equals P (id_U).  The score row has a.m entries (pitch a.ms),
// the weight row a.mv entries (pitch a.msv).
#include "kvc_async.cuh"
#include "kvc_internal.cuh"

namespace kvc {

template <typename T>
__global__ void __launch_bounds__(256) expand_kernel(DecodeArgs a) {
  extern __shared__ __align__(16) float smem[];
  const int ms = a.ms, m = a.m, n = a.n, msv = a.msv, mv = a.mv;
  float* Ssm = smem;                          // [EXP_ROWS][ms]
  float* Wacc = Ssm + EXP_ROWS * ms;          // [EXP_ROWS][msv]
  float* Lsm = Wacc + EXP_ROWS * msv;         // [EXP_ROWS][EXP_IC]
  float* Usm = Lsm + EXP_ROWS * EXP_IC;       // [64][EXP_IC + 1]
  float* rowmax = Usm + 64 * (EXP_IC + 1);    // [EXP_ROWS]
  float* rowsum = rowmax + EXP_ROWS;
  float* rowscale = rowsum + EXP_ROWS;

  const int split = blockIdx.x, rt = blockIdx.y, h = blockIdx.z;
  const int nrows_h = a.B * a.G * a.R;
  const int row0 = rt * EXP_ROWS;
  const int i_begin = split * a.ws.IR, i_end = min(n, i_begin + a.ws.IR);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const T* theta = static_cast<const T*>(a.theta) + (size_t)h * m * n;
  const T* U = static_cast<const T*>(a.U) + (size_t)h * mv * n;
  const float* S = a.S + (size_t)h * nrows_h * ms;

  for (int x = tid; x < EXP_ROWS * ms; x += 256) {
    const int r = x / ms, j = x - r * ms;
    Ssm[x] = (row0 + r < nrows_h && j < m) ? S[(size_t)(row0 + r) * ms + j] : 0.f;
  }
  for (int x = tid; x < EXP_ROWS * msv; x += 256) Wacc[x] = 0.f;
  if (tid < EXP_ROWS) { rowmax[tid] = -INFINITY; rowsum[tid] = 0.f; }
  __syncthreads();

  const int ii = tid & 63, rg = tid >> 6;      // column in chunk, group of 4 rows
  for (int i0 = i_begin; i0 < i_end; i0 += EXP_IC) {
    // ---- L chunk: [EXP_ROWS x EXP_IC] = S [EXP_ROWS x m] . theta[:, i0:i0+IC]
    {
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      const bool ok = i0 + ii < i_end;
      if (ok && a.id_theta) {
#pragma unroll
        for (int k = 0; k < 4; ++k) acc[k] = Ssm[(rg * 4 + k) * ms + i0 + ii];
      } else if (ok) {
        const T* tp = theta + i0 + ii;
        for (int j = 0; j < m; ++j) {
          const float t = to_f32(tp[(size_t)j * n]);
#pragma unroll
          for (int k = 0; k < 4; ++k) acc[k] = fmaf(Ssm[(rg * 4 + k) * ms + j], t, acc[k]);
        }
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) Lsm[(rg * 4 + k) * EXP_IC + ii] = ok ? acc[k] : -INFINITY;
    }
    __syncthreads();
    // ---- running max, P = exp(L - max), running sum: warp w owns rows 2w and 2w+1
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int r = warp * 2 + rr;
      const float l0 = Lsm[r * EXP_IC + lane], l1 = Lsm[r * EXP_IC + lane + 32];
      float cm = fmaxf(l0, l1);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, o));
      const float m_old = rowmax[r], m_new = fmaxf(m_old, cm);
      const float p0 = __expf(l0 - m_new), p1 = __expf(l1 - m_new);
      float ps = p0 + p1;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
      Lsm[r * EXP_IC + lane] = p0;
      Lsm[r * EXP_IC + lane + 32] = p1;
      if (lane == 0) {
        const float sc = (m_old == -INFINITY) ? 0.f : __expf(m_old - m_new);
        rowscale[r] = sc;
        rowsum[r] = rowsum[r] * sc + ps;
        rowmax[r] = m_new;
      }
    }
    __syncthreads();
    if (a.id_U) {
      // W = P: the columns of this CTA's range written so far follow the running maximum, the chunk's columns are P
      for (int x = tid; x < EXP_ROWS * (i0 - i_begin); x += 256) {
        const int r = x / (i0 - i_begin), j = i_begin + (x - r * (i0 - i_begin));
        Wacc[r * msv + j] *= rowscale[r];
      }
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (i0 + ii < i_end) Wacc[(rg * 4 + k) * msv + i0 + ii] = Lsm[(rg * 4 + k) * EXP_IC + ii];
      __syncthreads();
      continue;
    }
    // ---- W[:, j] = W[:, j] * scale + P . U[j, i0:i0+IC]^T, 64 rows of U at a time
    for (int j0 = 0; j0 < mv; j0 += 64) {
      for (int x = tid; x < 64 * EXP_IC; x += 256) {
        const int jj = x >> 6, i2 = x & 63;
        const bool ok = (j0 + jj < mv) && (i0 + i2 < i_end);
        Usm[jj * (EXP_IC + 1) + i2] = ok ? to_f32(U[(size_t)(j0 + jj) * n + i0 + i2]) : 0.f;
      }
      __syncthreads();
      {
        const int jj = ii;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int i2 = 0; i2 < EXP_IC; ++i2) {
          const float u = Usm[jj * (EXP_IC + 1) + i2];
#pragma unroll
          for (int k = 0; k < 4; ++k) acc[k] = fmaf(Lsm[(rg * 4 + k) * EXP_IC + i2], u, acc[k]);
        }
        if (j0 + jj < mv) {
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int r = rg * 4 + k;
            Wacc[r * msv + j0 + jj] = Wacc[r * msv + j0 + jj] * rowscale[r] + acc[k];
          }
        }
      }
      __syncthreads();
    }
  }

  float* Wout = a.W + ((size_t)split * a.H_kv + h) * nrows_h * msv;
  for (int x = tid; x < EXP_ROWS * msv; x += 256) {
    const int r = x / msv;
    if (row0 + r < nrows_h) Wout[(size_t)(row0 + r) * msv + (x - r * msv)] = Wacc[x];
  }
  if (tid < EXP_ROWS && row0 + tid < nrows_h)
    a.wstat[((size_t)split * a.H_kv + h) * nrows_h + row0 + tid] = make_float2(rowmax[tid], rowsum[tid]);
}

// rho = 0: theta = U = I, so L_img = S_comp and W = P.  One warp per row; writes the combined format.
__global__ void __launch_bounds__(256) passthrough_softmax_kernel(DecodeArgs a) {
  grid_dep_wait();
  grid_dep_launch();
  const int nrows = a.H_kv * a.B * a.G * a.R;
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= nrows) return;
  const float* s = a.S + (size_t)row * a.ms;
  float* w = a.Wcomb + (size_t)row * a.ms;
  float mx = -INFINITY;
  for (int j = lane; j < a.m; j += 32) mx = fmaxf(mx, s[j]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float sum = 0.f;
  for (int j = lane; j < a.ms; j += 32) {
    const float p = j < a.m ? __expf(s[j] - mx) : 0.f;
    w[j] = p;
    sum += p;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (lane == 0) a.statc[row] = make_float4(mx, sum, 0.f, 0.f);
}

// The n-split partials of one row combined relative to the row's overall maximum:
//   Wcomb[row][:] = sum_s e^{max_s - max} W_s[row][:],   statc[row] = (max, sum_s e^{max_s - max} sum_s).
// One warp per row (KV head, sequence, head in group, block).
__global__ void __launch_bounds__(256) combine_kernel(DecodeArgs a) {
  grid_dep_wait();
  grid_dep_launch();
  const int nrows = a.H_kv * a.B * a.G * a.R;
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= nrows) return;
  const int NS = a.ws.NS;
  float2 st = make_float2(-INFINITY, 0.f);
  if (lane < NS) st = a.wstat[(size_t)lane * nrows + row];
  float mx = st.x;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  const float my_sc = lane < NS ? __expf(st.x - mx) : 0.f;
  float sum = my_sc * st.y;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  float sc[MAX_NS];
#pragma unroll
  for (int s = 0; s < MAX_NS; ++s) sc[s] = __shfl_sync(0xffffffffu, my_sc, s);
  const size_t sstride = (size_t)nrows * a.msv;
  const float* wp = a.W + (size_t)row * a.msv;
  float* wo = a.Wcomb + (size_t)row * a.msv;
  for (int j = lane; j < a.msv; j += 32) {
    float v[MAX_NS];
#pragma unroll
    for (int s = 0; s < MAX_NS; ++s) v[s] = s < NS ? __ldcg(wp + s * sstride + j) : 0.f;
    float w = 0.f;
#pragma unroll
    for (int s = 0; s < MAX_NS; ++s) w = fmaf(sc[s], v[s], w);
    wo[j] = w;
  }
  if (lane == 0) a.statc[row] = make_float4(mx, sum, 0.f, 0.f);
}

static size_t expand_smem_bytes(int ms, int msv) {
  return sizeof(float) * ((size_t)EXP_ROWS * (ms + msv) + EXP_ROWS * EXP_IC + 64 * (EXP_IC + 1) + 3 * EXP_ROWS);
}

template <typename T>
static cudaError_t launch_expand_t(const DecodeArgs& a, cudaStream_t st) {
  const size_t smem = expand_smem_bytes(a.ms, a.msv);
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(expand_kernel<T>), smem);
  if (e != cudaSuccess) return e;
  dim3 grid(a.ws.NS, ceil_div(a.B * a.G * a.R, EXP_ROWS), a.H_kv);
  expand_kernel<T><<<grid, 256, smem, st>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_expand(const DecodeArgs& a, int dtype, cudaStream_t st) {
  if (a.R == 0) return cudaSuccess;
  const int nrows = a.H_kv * a.B * a.G * a.R;
  if (a.passthrough) {
    ProfScope prof(KVC_KERNEL_EXPAND, st);
    return launch_dependent(passthrough_softmax_kernel, dim3(ceil_div(nrows, 8)), dim3(256), 0, st, a);
  }
  cudaError_t e;
  {
    ProfScope prof(KVC_KERNEL_EXPAND, st);
    if (a.ws.use_mma) e = launch_expand_mma(a, st);
    else e = dtype == KVC_BF16 ? launch_expand_t<__nv_bfloat16>(a, st) : launch_expand_t<float>(a, st);
  }
  if (e != cudaSuccess) return e;
  ProfScope prof(KVC_KERNEL_COMBINE, st);
  return launch_dependent(combine_kernel, dim3(ceil_div(nrows, 8)), dim3(256), 0, st, a);
}

}  // namespace kvc
