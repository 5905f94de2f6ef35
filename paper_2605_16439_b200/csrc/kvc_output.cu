// Step 4 of Algorithm 1 plus the text values and the final normalisation:
//   y = sum_r W_r V_tilde_r + (sum P) mu + P_txt V_txt,   out = y / (sum of all exp terms).
// One streaming pass over the compressed values and the text values; bound by HBM bandwidth.
// Every CTA owns one split (a vision block or a chunk of text rows) of one (sequence, KV head)
// for all G query heads of the group; the last CTA of a (sequence, KV head) to finish merges the
// split partials by log-sum-exp and writes the output rows.
#include "kvc_internal.cuh"

namespace kvc {

template <typename T, int GT>
__global__ void __launch_bounds__(256) output_kernel(DecodeArgs a) {
  constexpr int EPV = Elems16<T>::N;
  constexpr int LPR = D / EPV;
  constexpr int RPI = 32 / LPR;
  constexpr int WARPS = 8;
  constexpr int UNROLL = 4;
  static_assert(GT <= WARPS, "one warp prepares the weights of one query head");

  extern __shared__ __align__(16) float smem[];
  const int wrows = max(a.ms, TXT_CHUNK);
  float* Wc = smem;                              // [wrows][GT]  weights of this split, row-major by row
  float* red = Wc + (size_t)wrows * GT;          // [WARPS][GT][D]
  __shared__ float s_max[MAX_G], s_sum[MAX_G];
  __shared__ int s_last;

  const int nsplit = a.ws.nsplit;
  const int bh = blockIdx.x / nsplit, split = blockIdx.x % nsplit;
  const int b = bh / a.H_kv, h = bh % a.H_kv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int sub = lane / LPR, c = lane % LPR;
  const bool is_txt = split >= a.R;
  const int nrows_h = a.B * a.G * a.R;

  int nrows;
  const T* rows;
  int t0 = 0;
  if (is_txt) {
    t0 = (split - a.R) * TXT_CHUNK;
    nrows = min(TXT_CHUNK, a.T - t0);
    rows = static_cast<const T*>(a.V_txt) + ((size_t)bh * a.T_cap + t0) * D;
  } else {
    nrows = a.m;
    rows = static_cast<const T*>(a.Vc) + ((size_t)bh * a.R + split) * a.m * D;
  }

  for (int g0 = 0; g0 < a.G; g0 += GT) {
    // ---- weights of this split for heads g0 .. g0+GT-1, relative to one maximum per head
    if (is_txt) {
      if (warp < GT && g0 + warp < a.G) {
        const float* s = a.s_txt + ((size_t)bh * a.G + g0 + warp) * a.Ts + t0;
        float mx = -INFINITY;
        for (int t = lane; t < nrows; t += 32) mx = fmaxf(mx, s[t]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float sum = 0.f;
        for (int t = lane; t < nrows; t += 32) {
          const float p = __expf(s[t] - mx);
          Wc[t * GT + warp] = p;
          sum += p;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) { s_max[g0 + warp] = mx; s_sum[g0 + warp] = sum; }
      }
    } else {
      if (warp < GT && g0 + warp < a.G) {
        const int row_id = (b * a.G + g0 + warp) * a.R + split;
        float mx = -INFINITY;
        for (int s = 0; s < a.ws.NS; ++s)
          mx = fmaxf(mx, a.wstat[((size_t)s * a.H_kv + h) * nrows_h + row_id].x);
        float sum = 0.f;
        for (int s = 0; s < a.ws.NS; ++s) {
          const float2 st = a.wstat[((size_t)s * a.H_kv + h) * nrows_h + row_id];
          const float sc = __expf(st.x - mx);
          sum += sc * st.y;
          const float* wp = a.W + (((size_t)s * a.H_kv + h) * nrows_h + row_id) * a.ms;
          for (int j = lane; j < nrows; j += 32) {
            const float w = sc * wp[j];
            Wc[j * GT + warp] = (s == 0) ? w : Wc[j * GT + warp] + w;
          }
        }
        if (lane == 0) { s_max[g0 + warp] = mx; s_sum[g0 + warp] = sum; }
      }
    }
    __syncthreads();
    // unused head slots of the register tile read zero weights
    if (g0 + GT > a.G) {
      for (int x = tid; x < nrows * GT; x += 256)
        if (g0 + (x % GT) >= a.G) Wc[x] = 0.f;
      __syncthreads();
    }

    // ---- stream the rows: acc[g][e] += w[row][g] * x[row][e]
    float acc[GT][EPV];
#pragma unroll
    for (int g = 0; g < GT; ++g)
#pragma unroll
      for (int e = 0; e < EPV; ++e) acc[g][e] = 0.f;

    for (int base = warp * RPI; base < nrows; base += WARPS * RPI * UNROLL) {
      uint4 v[UNROLL];
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        const int row = base + u * WARPS * RPI + sub;
        v[u] = make_uint4(0, 0, 0, 0);
        if (row < nrows) v[u] = __ldg(reinterpret_cast<const uint4*>(rows + (size_t)row * D + c * EPV));
      }
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        const int row = base + u * WARPS * RPI + sub;
        if (row < nrows) {
          float x[EPV];
          unpack16(v[u], x, (T*)nullptr);
#pragma unroll
          for (int g = 0; g < GT; ++g) {
            const float w = Wc[row * GT + g];
#pragma unroll
            for (int e = 0; e < EPV; ++e) acc[g][e] = fmaf(w, x[e], acc[g][e]);
          }
        }
      }
    }
    // ---- reduce over the rows held by different lanes and warps
#pragma unroll
    for (int g = 0; g < GT; ++g)
#pragma unroll
      for (int e = 0; e < EPV; ++e) {
        float v = acc[g][e];
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (sub == 0) red[(warp * GT + g) * D + c * EPV + e] = v;
      }
    __syncthreads();
    for (int x = tid; x < GT * D; x += 256) {
      const int g = x / D, col = x % D;
      if (g0 + g < a.G) {
        float y = 0.f;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) y += red[(w * GT + g) * D + col];
        if (!is_txt && !a.passthrough)
          y = fmaf(s_sum[g0 + g], to_f32(static_cast<const T*>(a.mu)[h * D + col]), y);
        a.ypart[(((size_t)bh * a.G + g0 + g) * nsplit + split) * D + col] = y;
      }
    }
    __syncthreads();
  }
  if (tid < a.G) a.ystat[((size_t)bh * a.G + tid) * nsplit + split] = make_float2(s_max[tid], s_sum[tid]);

  // ---- the last split of this (sequence, KV head) merges all partials
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(&a.cnt[bh], 1) == nsplit - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  for (int x = tid; x < a.G * D; x += 256) {
    const int g = x / D, col = x % D;
    const float2* st = a.ystat + ((size_t)bh * a.G + g) * nsplit;
    const float* yp = a.ypart + ((size_t)bh * a.G + g) * nsplit * D + col;
    float mx = -INFINITY;
    for (int s = 0; s < nsplit; ++s) mx = fmaxf(mx, __ldcg(&st[s]).x);
    float num = 0.f, den = 0.f;
    for (int s = 0; s < nsplit; ++s) {
      const float2 v = __ldcg(&st[s]);
      const float sc = __expf(v.x - mx);
      den = fmaf(sc, v.y, den);
      num = fmaf(sc, __ldcg(yp + (size_t)s * D), num);
    }
    store_elem(static_cast<T*>(a.out) + ((size_t)b * a.H_kv * a.G + h * a.G + g) * D + col, num / den);
  }
}

template <typename T, int GT>
static cudaError_t launch_output_g(const DecodeArgs& a, cudaStream_t st) {
  const size_t smem = sizeof(float) * ((size_t)max(a.ms, TXT_CHUNK) * GT + 8 * GT * D);
  cudaError_t e = cudaFuncSetAttribute(output_kernel<T, GT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const unsigned grid = (unsigned)(a.B * a.H_kv * a.ws.nsplit);
  output_kernel<T, GT><<<grid, 256, smem, st>>>(a);
  return cudaGetLastError();
}

template <typename T>
static cudaError_t launch_output_t(const DecodeArgs& a, cudaStream_t st) {
  if (a.G == 1) return launch_output_g<T, 1>(a, st);
  if (a.G == 2) return launch_output_g<T, 2>(a, st);
  if (a.G <= 4) return launch_output_g<T, 4>(a, st);
  return launch_output_g<T, 8>(a, st);
}

cudaError_t launch_output(const DecodeArgs& a, int dtype, cudaStream_t st) {
  ProfScope prof(KVC_KERNEL_OUTPUT, st);
  return dtype == KVC_BF16 ? launch_output_t<__nv_bfloat16>(a, st) : launch_output_t<float>(a, st);
}

}  // namespace kvc
