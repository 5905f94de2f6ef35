// Step 1 of Algorithm 1 plus the text logits: S_comp = sigma q K_tilde^T, s_txt = sigma q K_txt^T.
// One streaming pass over the compressed keys and the text keys; bound by HBM bandwidth.
#include "kvc_internal.cuh"

namespace kvc {

// Each CTA scores SCORE_TILE_ROWS consecutive rows of one (sequence, KV head) against GT query
// heads held in registers.  A row of D elements is covered by LPR lanes with one 16-byte load
// each; a warp therefore reads RPI whole rows (512 contiguous bytes) per load instruction.
template <typename T, int GT>
__global__ void __launch_bounds__(256) scores_kernel(DecodeArgs a, int tiles_vis, int tiles_txt) {
  constexpr int EPV = Elems16<T>::N;
  constexpr int LPR = D / EPV;             // lanes per row
  constexpr int RPI = 32 / LPR;            // rows per warp load
  constexpr int WARPS = 8;
  constexpr int ROWS_PER_WARP = SCORE_TILE_ROWS / WARPS;
  constexpr int ITERS = ROWS_PER_WARP / RPI;

  const int tiles_per_bh = tiles_vis + tiles_txt;
  const int bh = blockIdx.x / tiles_per_bh;
  const int tile = blockIdx.x % tiles_per_bh;
  const int b = bh / a.H_kv, h = bh % a.H_kv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane / LPR, c = lane % LPR;

  // the arrival counters of the output kernel's split merge are cleared here, one launch earlier
  if (blockIdx.x == 0)
    for (int i = threadIdx.x; i < a.B * a.H_kv; i += blockDim.x) a.cnt[i] = 0;

  const bool is_txt = tile >= tiles_vis;
  const int nrows = is_txt ? a.T : a.R * a.m;
  const int row0 = (is_txt ? tile - tiles_vis : tile) * SCORE_TILE_ROWS + warp * ROWS_PER_WARP;
  const T* base = is_txt
      ? static_cast<const T*>(a.K_txt) + (size_t)bh * a.T_cap * D
      : static_cast<const T*>(a.Kc) + (size_t)bh * a.R * a.m * D;

  const float sigma = rsqrtf((float)D);
  for (int g0 = 0; g0 < a.G; g0 += GT) {
    float qf[GT][EPV];
#pragma unroll
    for (int g = 0; g < GT; ++g) {
      if (g0 + g < a.G) {
        load16(static_cast<const T*>(a.q) + ((size_t)b * a.H_kv * a.G + h * a.G + g0 + g) * D + c * EPV, qf[g]);
#pragma unroll
        for (int e = 0; e < EPV; ++e) qf[g][e] *= sigma;
      } else {
#pragma unroll
        for (int e = 0; e < EPV; ++e) qf[g][e] = 0.f;
      }
    }
    uint4 v[ITERS];
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
      const int row = row0 + it * RPI + sub;
      v[it] = make_uint4(0, 0, 0, 0);
      if (row < nrows) v[it] = __ldg(reinterpret_cast<const uint4*>(base + (size_t)row * D + c * EPV));
    }
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
      const int row = row0 + it * RPI + sub;
      float x[EPV];
      unpack16(v[it], x, (T*)nullptr);
      float acc[GT];
#pragma unroll
      for (int g = 0; g < GT; ++g) {
        acc[g] = 0.f;
#pragma unroll
        for (int e = 0; e < EPV; ++e) acc[g] = fmaf(qf[g][e], x[e], acc[g]);
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) acc[g] += __shfl_xor_sync(0xffffffffu, acc[g], o);
      }
      if (c == 0 && row < nrows) {
#pragma unroll
        for (int g = 0; g < GT; ++g) {
          if (g0 + g >= a.G) break;
          if (is_txt) {
            a.s_txt[((size_t)bh * a.G + g0 + g) * a.Ts + row] = acc[g];
          } else {
            const int r = row / a.m, j = row - r * a.m;
            a.S[((((size_t)h * a.B + b) * a.G + g0 + g) * a.R + r) * a.ms + j] = acc[g];
          }
        }
      }
    }
  }
}

template <typename T>
static cudaError_t launch_scores_t(const DecodeArgs& a, cudaStream_t st) {
  const int tiles_vis = ceil_div(a.R * a.m, SCORE_TILE_ROWS);
  const int tiles_txt = ceil_div(a.T, SCORE_TILE_ROWS);
  const unsigned grid = (unsigned)(a.B * a.H_kv * (tiles_vis + tiles_txt));
  if (grid == 0) return cudaSuccess;
  ProfScope prof(KVC_KERNEL_SCORES, st);
  if (a.G == 1) scores_kernel<T, 1><<<grid, 256, 0, st>>>(a, tiles_vis, tiles_txt);
  else if (a.G == 2) scores_kernel<T, 2><<<grid, 256, 0, st>>>(a, tiles_vis, tiles_txt);
  else if (a.G <= 4) scores_kernel<T, 4><<<grid, 256, 0, st>>>(a, tiles_vis, tiles_txt);
  else scores_kernel<T, 8><<<grid, 256, 0, st>>>(a, tiles_vis, tiles_txt);
  return cudaGetLastError();
}

cudaError_t launch_scores(const DecodeArgs& a, int dtype, cudaStream_t st) {
  return dtype == KVC_BF16 ? launch_scores_t<__nv_bfloat16>(a, st) : launch_scores_t<float>(a, st);
}

}  // namespace kvc
