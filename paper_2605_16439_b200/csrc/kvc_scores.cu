// Step 1 of Algorithm 1 plus the text logits: S_comp = sigma q K_tilde^T, s_txt = sigma q K_txt^T.
// One streaming pass over the compressed keys and the text keys; bound by HBM bandwidth.
#include "kvc_async.cuh"
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
  if (blockIdx.x == 0) {
    for (int i = threadIdx.x; i <= a.B * a.H_kv; i += blockDim.x) a.cnt[i] = 0;   // counters + status word
    __syncthreads();
    check_seq_lengths(a, threadIdx.x, blockDim.x);
  }

  const bool is_txt = tile >= tiles_vis;
  const int nrows = is_txt ? seq_T(a, b) : seq_R(a, b) * a.m;
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
            const size_t o = ((((size_t)h * a.B + b) * a.G + g0 + g) * a.R + r) * a.ms + j;
            if (a.ws.use_mma) a.Sb[o] = __float2bfloat16_rn(acc[g]);
            else a.S[o] = acc[g];
          }
        }
      }
    }
  }
}


// ---- bf16 storage: the dot products run on the tensor cores (mma.sync m16n8k16) -------------------
// A warp scores a tile of 16 rows against up to 8 * NG query heads.  Lane (g, t) loads, for rows g
// and g + 8, the 16-byte pieces t, t+4, t+8, t+12 of the 256-byte row straight from global memory
// (every byte of every 32-byte sector is used) and feeds them to the MMA as A fragments; because a
// dot product does not care about the order of its terms, the k index of the MMA is a fixed
// permutation of the row's element index, and the B fragments (the queries, one head per column)
// are loaded with the same permutation.  The MMA does the cross-lane reduction that would
// otherwise cost shuffles.
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

constexpr int SM_TILE = 16;           // rows per warp tile
constexpr int SM_WARPS = 8;

template <int NG>
__global__ void __launch_bounds__(256, 4) scores_mma_kernel(DecodeArgs a, int tv, int tt, int tiles_per_cta) {
  using T = __nv_bfloat16;
  const int tiles_per_bh = tv + tt;
  const int total = a.B * a.H_kv * tiles_per_bh;
  const int tile_begin = blockIdx.x * tiles_per_cta;
  const int tile_end = min(total, tile_begin + tiles_per_cta);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int VR = a.R * a.m;
  const float sigma = rsqrtf((float)D);

  // the expansion kernel may start now: it prefetches parameters, then waits for this grid to finish
  grid_dep_launch();

  if (blockIdx.x == 0) {
    for (int i = threadIdx.x; i <= a.B * a.H_kv; i += blockDim.x) a.cnt[i] = 0;   // counters + status word
    __syncthreads();
    check_seq_lengths(a, threadIdx.x, blockDim.x);
  }

  int cur_bh = -1;
  uint4 qf[NG][4];
  for (int tile = tile_begin + warp; tile < tile_end; tile += SM_WARPS) {
    const int bh = tile / tiles_per_bh, lt = tile - bh * tiles_per_bh;
    const bool is_txt = lt >= tv;
    const int row0 = (is_txt ? lt - tv : lt) * SM_TILE;
    const int nrows = is_txt ? seq_T(a, bh / a.H_kv) : seq_R(a, bh / a.H_kv) * a.m;
    const T* base = is_txt ? static_cast<const T*>(a.K_txt) + (size_t)bh * a.T_cap * D
                           : static_cast<const T*>(a.Kc) + (size_t)bh * VR * D;
    const int ra = row0 + g, rb = row0 + g + 8;
    uint4 va[4], vb[4];
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      va[kk] = ra < nrows ? __ldg(reinterpret_cast<const uint4*>(base + (size_t)ra * D + kk * 32 + t * 8)) : make_uint4(0, 0, 0, 0);
      vb[kk] = rb < nrows ? __ldg(reinterpret_cast<const uint4*>(base + (size_t)rb * D + kk * 32 + t * 8)) : make_uint4(0, 0, 0, 0);
    }
    if (bh != cur_bh) {
      cur_bh = bh;
#pragma unroll
      for (int ng = 0; ng < NG; ++ng) {
        const int head = ng * 8 + g;     // this lane's column of the B operand
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          qf[ng][kk] = head < a.G ? __ldg(reinterpret_cast<const uint4*>(static_cast<const T*>(a.q) +
                                          ((size_t)bh * a.G + head) * D + kk * 32 + t * 8))
                                  : make_uint4(0, 0, 0, 0);
      }
    }
    const int b = bh / a.H_kv, h = bh - b * a.H_kv;
#pragma unroll
    for (int ng = 0; ng < NG; ++ng) {
      float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        mma_16816(c, va[kk].x, vb[kk].x, va[kk].y, vb[kk].y, qf[ng][kk].x, qf[ng][kk].y);
        mma_16816(c, va[kk].z, vb[kk].z, va[kk].w, vb[kk].w, qf[ng][kk].z, qf[ng][kk].w);
      }
      // c[0], c[1]: row ra, heads 2t, 2t+1 of this group of 8;  c[2], c[3]: row rb
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int head = ng * 8 + 2 * t + (k & 1);
        const int row = (k < 2) ? ra : rb;
        if (head < a.G && row < nrows) {
          const float v = c[k] * sigma;
          if (is_txt) {
            a.s_txt[((size_t)bh * a.G + head) * a.Ts + row] = v;
          } else {
            const int r = row / a.m, j = row - r * a.m;
            const size_t o = ((((size_t)h * a.B + b) * a.G + head) * a.R + r) * a.ms + j;
            if (a.ws.use_mma) a.Sb[o] = __float2bfloat16_rn(v);
            else a.S[o] = v;
          }
        }
      }
    }
  }
}

static cudaError_t launch_scores_mma(const DecodeArgs& a, cudaStream_t st) {
  const int tv = ceil_div(a.R * a.m, SM_TILE), tt = ceil_div(a.T, SM_TILE);
  const long long total = (long long)a.B * a.H_kv * (tv + tt);
  if (total == 0) return cudaSuccess;
  // one resident wave: (CTAs that fit per SM) x (SM count) CTAs, each a contiguous run of tiles
  static int slots[2] = {0, 0};
  const int ng = a.G <= 8 ? 0 : 1;
  if (slots[ng] == 0) {
    int dev = 0, sms = 0, per_sm = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (ng == 0) cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, scores_mma_kernel<1>, 256, 0);
    else cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, scores_mma_kernel<2>, 256, 0);
    slots[ng] = (sms > 0 ? sms : 148) * (per_sm > 0 ? per_sm : 2);
  }
  int tiles_per_cta = (int)((total + slots[ng] - 1) / slots[ng]);
  tiles_per_cta = ceil_div(tiles_per_cta, SM_WARPS) * SM_WARPS;
  const unsigned grid = (unsigned)((total + tiles_per_cta - 1) / tiles_per_cta);
  if (a.G <= 8) scores_mma_kernel<1><<<grid, 256, 0, st>>>(a, tv, tt, tiles_per_cta);
  else scores_mma_kernel<2><<<grid, 256, 0, st>>>(a, tv, tt, tiles_per_cta);
  return cudaGetLastError();
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
  if (dtype == KVC_BF16) {
    ProfScope prof(KVC_KERNEL_SCORES, st);
    return launch_scores_mma(a, st);
  }
  return dtype == KVC_BF16 ? launch_scores_t<__nv_bfloat16>(a, st) : launch_scores_t<float>(a, st);
}

}  // namespace kvc
