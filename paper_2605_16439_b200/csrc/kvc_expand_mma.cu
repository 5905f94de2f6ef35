// Steps 2 and 3 of Algorithm 1 on the tensor cores (bf16 operands, fp32 accumulation):
//   L = S theta[h]   ->   P = exp(L - running row max)   ->   W += P U[h]^T
// for 64 rows (sequence, head-in-group, block) of one KV head and one range of the n axis.
// Same contract as the CUDA-core kernel: every (row, n-split) emits an unnormalised partial
// (W, max, sum); the output kernel combines the splits.
//
// Warp-level mma.sync.m16n8k16: each of the 4 warps owns 16 rows; theta and U chunks of 64 vision
// positions are staged in shared memory with cp.async and read with ldmatrix (theta transposed,
// since the contraction runs over its leading index).
#include "kvc_async.cuh"
#include "kvc_internal.cuh"

namespace kvc {

constexpr int XM_ROWS = 64;   // rows per CTA
constexpr int XM_IC = 64;     // vision positions per chunk
constexpr int XM_LD = 72;     // smem row stride of theta / U chunks in elements (64 + 8 pad: conflict-free ldmatrix)

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem, bool pred) {
  const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
  const int sz = pred ? 16 : 0;   // 0 source bytes: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;\n" ::: "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* p) {
  const unsigned s = (unsigned)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(s));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* p) {
  const unsigned s = (unsigned)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(s));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// NT_W: 8-column tiles of W held per warp (columns of this CTA's column group, <= NT_W * 8)
template <int NT_W>
__global__ void __launch_bounds__(128) expand_mma_kernel(DecodeArgs a) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int ms = a.ms, m = a.m, n = a.n;
  const int ldS = ms + 8;
  __nv_bfloat16* Ssm = reinterpret_cast<__nv_bfloat16*>(smem_raw);   // [XM_ROWS][ldS]
  __nv_bfloat16* Tsm = Ssm + XM_ROWS * ldS;                            // [ms][XM_LD]   theta chunk
  __nv_bfloat16* Usm = Tsm + ms * XM_LD;                               // [cgw][XM_LD]  U chunk

  const int CG = a.ws.CG, cgw = a.ws.cgw;
  const int split = blockIdx.x, rt = blockIdx.y / CG, cg = blockIdx.y % CG, h = blockIdx.z;
  const int col0 = cg * cgw, ncols = min(cgw, ms - col0);
  const int nrows_h = a.B * a.G * a.R;
  const int row0 = rt * XM_ROWS;
  const int i_begin = split * a.ws.IR, i_end = min(n, i_begin + a.ws.IR);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const __nv_bfloat16* theta = static_cast<const __nv_bfloat16*>(a.theta) + (size_t)h * m * n;
  const __nv_bfloat16* U = static_cast<const __nv_bfloat16*>(a.U) + (size_t)h * m * n;
  const __nv_bfloat16* S = a.Sb + (size_t)h * nrows_h * ms;

  auto load_params = [&](int i0) {
    for (int x = tid; x < ms * 8; x += 128) {
      const int j = x >> 3, c = x & 7;
      const bool ok = j < m && i0 + c * 8 < i_end;
      cp_async16(&Tsm[j * XM_LD + c * 8], ok ? theta + (size_t)j * n + i0 + c * 8 : theta, ok);
    }
    for (int x = tid; x < ncols * 8; x += 128) {
      const int jj = x >> 3, c = x & 7;
      const bool ok = col0 + jj < m && i0 + c * 8 < i_end;
      cp_async16(&Usm[jj * XM_LD + c * 8], ok ? U + (size_t)(col0 + jj) * n + i0 + c * 8 : U, ok);
    }
  };
  // theta and U are parameters (never written by this library): fetch the first chunk while the score
  // kernel is still running, then wait for its scores
  load_params(i_begin);
  grid_dep_wait();
  grid_dep_launch();
  {
    const int cpr = ms >> 3;   // 16-byte pieces per row
    for (int x = tid; x < XM_ROWS * cpr; x += 128) {
      const int r = x / cpr, c = x - r * cpr;
      const bool ok = row0 + r < nrows_h;
      cp_async16(&Ssm[r * ldS + c * 8], ok ? S + (size_t)(row0 + r) * ms + c * 8 : S, ok);
    }
  }

  float accW[NT_W][4];
#pragma unroll
  for (int i = 0; i < NT_W; ++i)
#pragma unroll
    for (int k = 0; k < 4; ++k) accW[i][k] = 0.f;
  float mrow[2] = {-INFINITY, -INFINITY}, lsum[2] = {0.f, 0.f};

  for (int i0 = i_begin; i0 < i_end; i0 += XM_IC) {
    if (i0 != i_begin) {
      __syncthreads();            // every warp is done with the previous chunk
      load_params(i0);
    }
    cp_async_commit();
    cp_async_wait_all();
    __syncthreads();
    if (i0 == i_begin && ms > m) {
      // the columns m..ms of S are padding of the score buffer: make them exact zeros
      const int pad = ms - m;
      for (int x = tid; x < XM_ROWS * pad; x += 128) {
        const int r = x / pad, c = x - r * pad;
        Ssm[r * ldS + m + c] = __float2bfloat16_rn(0.f);
      }
      __syncthreads();
    }

    // ---- L chunk [16 x 64] per warp
    float accL[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int k = 0; k < 4; ++k) accL[i][k] = 0.f;
    for (int k0 = 0; k0 < ms; k0 += 16) {
      uint32_t af[4];
      ldmatrix_x4(af, &Ssm[(warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * ldS + k0 + (lane >> 4) * 8]);
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        uint32_t bf[4];
        ldmatrix_x4_trans(bf, &Tsm[(k0 + (lane & 7) + ((lane >> 3) & 1) * 8) * XM_LD + np * 16 + (lane >> 4) * 8]);
        mma_bf16(accL[2 * np], af, bf[0], bf[1]);
        mma_bf16(accL[2 * np + 1], af, bf[2], bf[3]);
      }
    }
    // ---- running max, P = exp(L - max)
    const int valid = i_end - i0;                  // columns of this chunk that exist
    float cm[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int col = nt * 8 + 2 * t + (k & 1);
        if (col >= valid) accL[nt][k] = -INFINITY;
        cm[k >> 1] = fmaxf(cm[k >> 1], accL[nt][k]);
      }
    float sc[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      cm[r] = fmaxf(cm[r], __shfl_xor_sync(0xffffffffu, cm[r], 1));
      cm[r] = fmaxf(cm[r], __shfl_xor_sync(0xffffffffu, cm[r], 2));
      const float m_new = fmaxf(mrow[r], cm[r]);
      sc[r] = (mrow[r] == -INFINITY) ? 0.f : __expf(mrow[r] - m_new);
      mrow[r] = m_new;
      lsum[r] *= sc[r];
    }
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float p = __expf(accL[nt][k] - mrow[k >> 1]);
        accL[nt][k] = p;
        lsum[k >> 1] += p;
      }
    if (sc[0] != 1.f || sc[1] != 1.f) {
#pragma unroll
      for (int nt = 0; nt < NT_W; ++nt) {
        accW[nt][0] *= sc[0]; accW[nt][1] *= sc[0];
        accW[nt][2] *= sc[1]; accW[nt][3] *= sc[1];
      }
    }
    // ---- W [16 x ncols] += P [16 x 64] . U[col0:col0+ncols, chunk]^T
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      uint32_t pf[4];
      pf[0] = pack_bf16(accL[2 * kk][0], accL[2 * kk][1]);
      pf[1] = pack_bf16(accL[2 * kk][2], accL[2 * kk][3]);
      pf[2] = pack_bf16(accL[2 * kk + 1][0], accL[2 * kk + 1][1]);
      pf[3] = pack_bf16(accL[2 * kk + 1][2], accL[2 * kk + 1][3]);
#pragma unroll
      for (int np = 0; np < NT_W / 2; ++np) {
        if (np * 16 < ncols) {
          uint32_t bf[4];
          ldmatrix_x4(bf, &Usm[(np * 16 + (lane & 7) + (lane >> 4) * 8) * XM_LD + kk * 16 + ((lane >> 3) & 1) * 8]);
          mma_bf16(accW[2 * np], pf, bf[0], bf[1]);
          mma_bf16(accW[2 * np + 1], pf, bf[2], bf[3]);
        }
      }
    }
  }

  // ---- partial results of this (row tile, column group, n-split)
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    lsum[r] += __shfl_xor_sync(0xffffffffu, lsum[r], 1);
    lsum[r] += __shfl_xor_sync(0xffffffffu, lsum[r], 2);
  }
  float* Wout = a.W + ((size_t)split * a.H_kv + h) * nrows_h * ms;
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int row = row0 + warp * 16 + g + r * 8;
    if (row >= nrows_h) continue;
#pragma unroll
    for (int nt = 0; nt < NT_W; ++nt) {
      const int col = col0 + nt * 8 + 2 * t;
      if (nt * 8 < ncols && col < ms)
        *reinterpret_cast<float2*>(&Wout[(size_t)row * ms + col]) = make_float2(accW[nt][2 * r], accW[nt][2 * r + 1]);
    }
    if (t == 0 && cg == 0)
      a.wstat[((size_t)split * a.H_kv + h) * nrows_h + row] = make_float2(mrow[r], lsum[r]);
  }
}

size_t expand_mma_smem_bytes(int ms, int cgw) {
  return sizeof(__nv_bfloat16) * ((size_t)XM_ROWS * (ms + 8) + (size_t)ms * XM_LD + (size_t)cgw * XM_LD);
}

template <int NT_W>
static cudaError_t launch_nt(const DecodeArgs& a, cudaStream_t st) {
  const size_t smem = expand_mma_smem_bytes(a.ms, a.ws.cgw);
  {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(expand_mma_kernel<NT_W>), smem);
    if (e != cudaSuccess) return e;
  }
  dim3 grid(a.ws.NS, ceil_div(a.B * a.G * a.R, XM_ROWS) * a.ws.CG, a.H_kv);
  return launch_dependent(expand_mma_kernel<NT_W>, grid, dim3(128), smem, st, a);
}

cudaError_t launch_expand_mma(const DecodeArgs& a, cudaStream_t st) {
  const int nt = ceil_div(a.ws.cgw, 8);
  if (nt <= 8) return launch_nt<8>(a, st);
  if (nt <= 16) return launch_nt<16>(a, st);
  if (nt <= 24) return launch_nt<24>(a, st);
  return launch_nt<32>(a, st);
}

}  // namespace kvc
