// Step 4 of Algorithm 1 plus the text values and the final normalisation:
//   y = sum_r W_r V_tilde_r + (sum P) mu + P_txt V_txt,   out = y / (sum of all exp terms).
// One streaming pass over the compressed values and the text values; bound by HBM bandwidth.
//
// The value rows of a (sequence, KV head) form two contiguous runs in memory: R*m compressed vision
// rows and T text rows.  Each run is cut into parts of at most OUT_PART_ROWS rows, independent of
// the block structure, and one CTA owns one part for all G query heads of the group.  The CTA first
// asks the bulk-copy engine (cp.async.bulk, mbarrier completion) for all rows of its part, then
// prepares the per-row weights while the copies are in flight: for a vision row (block r, offset j)
// the n-split partials of W combined relative to one maximum per head and part, for a text row
// exp(s - max).  It then forms the weighted sum of the rows from shared memory and writes one
// partial (max, sum, y) per head.  A second, tiny kernel merges the partials of all parts by
// log-sum-exp and writes the output rows.
#include "kvc_async.cuh"
#include "kvc_internal.cuh"

namespace kvc {

constexpr int OUT_STAGE_ROWS = 64;
constexpr int OUT_STAGES = OUT_PART_ROWS / OUT_STAGE_ROWS;
constexpr int OUT_WARPS = 8;
static_assert(OUT_PART_ROWS == 256, "one thread prepares the weights of one row of the part");

template <typename T, int GT>
__global__ void __launch_bounds__(256, (GT <= 2 ? 3 : 1)) output_kernel(DecodeArgs a) {
  constexpr int EPV = Elems16<T>::N;
  constexpr int LPR = D / EPV;               // lanes per row
  constexpr int RPI = 32 / LPR;              // rows per warp step
  constexpr uint32_t ROW_BYTES = D * sizeof(T);
  constexpr uint32_t STAGE_BYTES = OUT_STAGE_ROWS * ROW_BYTES;
  static_assert(GT <= OUT_WARPS, "one warp prepares the statistics of one query head");

  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* ring = smem_raw;                                              // [OUT_STAGES][STAGE_BYTES]
  float* Wc = reinterpret_cast<float*>(ring + OUT_STAGES * STAGE_BYTES);       // [OUT_PART_ROWS][GT]
  float* red = Wc + OUT_PART_ROWS * GT;                                        // [OUT_WARPS][GT][D]
  __shared__ __align__(8) uint64_t bars[OUT_STAGES];
  __shared__ float s_max[MAX_G], s_sum[MAX_G];

  const int nsplit = a.ws.nsplit, Pv = a.ws.Pv;
  const int bh = blockIdx.x / nsplit, part = blockIdx.x % nsplit;
  const int b = bh / a.H_kv, h = bh % a.H_kv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int sub = lane / LPR, c = lane % LPR;
  const bool is_txt = part >= Pv;
  const int nrows_h = a.B * a.G * a.R;
  const int NS = a.ws.NS, m = a.m, VR = a.R * a.m;

  int row_a, nrows;                                  // first row of the part within its run, row count
  const T* rows;
  if (is_txt) {
    row_a = (part - Pv) * OUT_PART_ROWS;
    nrows = min(OUT_PART_ROWS, a.T - row_a);
    rows = static_cast<const T*>(a.V_txt) + ((size_t)bh * a.T_cap + row_a) * D;
  } else {
    row_a = part * a.ws.pr;
    nrows = min(a.ws.pr, VR - row_a);
    rows = static_cast<const T*>(a.Vc) + ((size_t)bh * VR + row_a) * D;
  }
  const int nchunks = ceil_div(nrows, OUT_STAGE_ROWS);

  if (tid == 0) {
    for (int s = 0; s < OUT_STAGES; ++s) mbar_init(&bars[s], 1);
    fence_mbar_init();
    for (int ch = 0; ch < nchunks; ++ch) {
      const uint32_t bytes = (uint32_t)min(OUT_STAGE_ROWS, nrows - ch * OUT_STAGE_ROWS) * ROW_BYTES;
      mbar_expect_tx(&bars[ch], bytes);
      bulk_g2s(ring + ch * STAGE_BYTES, rows + (size_t)ch * OUT_STAGE_ROWS * D, bytes, &bars[ch]);
    }
  }
  // The value rows were written before the kernel this one follows; everything below reads what the
  // score and expansion kernels produced, so wait for them here (the copies are already in flight).
  grid_dep_wait();
  grid_dep_launch();
  __syncthreads();                                  // barriers initialised before anyone polls them

  // this thread's row of the part, and for a vision row its block and offset
  const int row = tid;
  const bool row_ok = row < nrows;
  int r_blk = 0, j_off = 0;
  if (!is_txt && row_ok) { r_blk = (row_a + row) / m; j_off = (row_a + row) - r_blk * m; }
  const size_t sstride_stat = (size_t)a.H_kv * nrows_h;
  const size_t sstride_W = sstride_stat * a.ms;

  bool timed_out = false;
  for (int g0 = 0; g0 < a.G; g0 += GT) {
    // ---- one reference maximum and the probability mass per head for this part
    if (warp < GT && g0 + warp < a.G) {
      const int gh = g0 + warp;
      if (is_txt) {
        const float* s = a.s_txt + ((size_t)bh * a.G + gh) * a.Ts + row_a;
        float v[OUT_PART_ROWS / 32];
        float mx = -INFINITY;
#pragma unroll
        for (int k = 0; k < OUT_PART_ROWS / 32; ++k) {
          const int t = lane + 32 * k;
          v[k] = t < nrows ? s[t] : -INFINITY;
          mx = fmaxf(mx, v[k]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float sum = 0.f;
#pragma unroll
        for (int k = 0; k < OUT_PART_ROWS / 32; ++k) {
          const int t = lane + 32 * k;
          const float p = __expf(v[k] - mx);
          if (t < nrows) Wc[t * GT + warp] = p;
          sum += p;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) { s_max[gh] = mx; s_sum[gh] = sum; }
      } else {
        // statistics (max, sum) of every (block touched by the part, n-split): entry e = blk * NS + s
        const int r_lo = row_a / m, r_hi = (row_a + nrows - 1) / m;
        const int ne = (r_hi - r_lo + 1) * NS;
        const float2* st = a.wstat + (size_t)h * nrows_h + (size_t)(b * a.G + gh) * a.R;
        float mx = -INFINITY;
        for (int e = lane; e < ne; e += 32) {
          const int blk = e / NS, s = e - blk * NS;
          mx = fmaxf(mx, st[s * sstride_stat + r_lo + blk].x);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        // the probability mass of a block is counted by the part that holds the block's first row
        float sum = 0.f;
        for (int e = lane; e < ne; e += 32) {
          const int blk = e / NS, s = e - blk * NS;
          const int first = (r_lo + blk) * m;
          if (first >= row_a && first < row_a + nrows) {
            const float2 v = st[s * sstride_stat + r_lo + blk];
            sum = fmaf(__expf(v.x - mx), v.y, sum);
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) { s_max[gh] = mx; s_sum[gh] = sum; }
      }
    }
    // ---- vision rows: fetch the n-split partials of W for the first head before the barrier
    float wv[MAX_NS], xs[MAX_NS];
    auto fetch = [&](int gh) {
      const size_t row_id = (size_t)(b * a.G + gh) * a.R + r_blk;
      const float* wp = a.W + ((size_t)h * nrows_h + row_id) * a.ms + j_off;
      const float2* sp = a.wstat + (size_t)h * nrows_h + row_id;
#pragma unroll
      for (int s = 0; s < MAX_NS; ++s) {
        const bool ok = s < NS;
        wv[s] = ok ? __ldcg(wp + s * sstride_W) : 0.f;
        xs[s] = ok ? __ldcg(&sp[s * sstride_stat]).x : -INFINITY;
      }
    };
    const bool vis_row = !is_txt && row_ok;
    if (vis_row) fetch(g0);
    __syncthreads();
    if (!is_txt) {
#pragma unroll
      for (int g = 0; g < GT; ++g) {
        float w = 0.f;
        if (vis_row && g0 + g < a.G) {
          if (g > 0) fetch(g0 + g);
          const float mx = s_max[g0 + g];
#pragma unroll
          for (int s = 0; s < MAX_NS; ++s) w = fmaf(__expf(xs[s] - mx), wv[s], w);
        }
        if (row_ok) Wc[row * GT + g] = w;
      }
    } else if (g0 + GT > a.G) {
      for (int x = tid; x < nrows * GT; x += 256)
        if (g0 + (x % GT) >= a.G) Wc[x] = 0.f;
    }
    __syncthreads();

    // ---- weighted sum of the rows from shared memory: acc[g][e] += w[row][g] * x[row][e]
    float acc[GT][EPV];
#pragma unroll
    for (int g = 0; g < GT; ++g)
#pragma unroll
      for (int e = 0; e < EPV; ++e) acc[g][e] = 0.f;

    for (int ch = 0; ch < nchunks; ++ch) {
      // every stage is filled exactly once (phase 0); later passes over the heads find it complete
      if (!timed_out && !mbar_wait_bounded(&bars[ch], 0u)) timed_out = true;
      const int crow0 = ch * OUT_STAGE_ROWS;
      const int crows = min(OUT_STAGE_ROWS, nrows - crow0);
      const unsigned char* sbase = ring + ch * STAGE_BYTES;
      if (!timed_out) {
#pragma unroll 2
        for (int rr = warp * RPI + sub; rr < crows; rr += OUT_WARPS * RPI) {
          const uint4 v = *reinterpret_cast<const uint4*>(sbase + (size_t)rr * ROW_BYTES + c * 16);
          float x[EPV];
          unpack16(v, x, (T*)nullptr);
#pragma unroll
          for (int g = 0; g < GT; ++g) {
            const float w = Wc[(crow0 + rr) * GT + g];
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
        for (int w = 0; w < OUT_WARPS; ++w) y += red[(w * GT + g) * D + col];
        if (!is_txt && !a.passthrough)
          y = fmaf(s_sum[g0 + g], to_f32(static_cast<const T*>(a.mu)[h * D + col]), y);
        a.ypart[(((size_t)bh * a.G + g0 + g) * nsplit + part) * D + col] = y;
      }
    }
    __syncthreads();
  }
  if (tid < a.G) a.ystat[((size_t)bh * a.G + tid) * nsplit + part] = make_float2(s_max[tid], s_sum[tid]);
  if (timed_out && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
}

// out[b,hq,:] = sum_p e^{max_p - M} y_p / sum_p e^{max_p - M} l_p over the parts p of (b, hq): one warp per head.
template <typename T>
__global__ void __launch_bounds__(256) merge_kernel(DecodeArgs a) {
  grid_dep_wait();
  const int nsplit = a.ws.nsplit;
  const int head = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;   // flat (b, h, g)
  if (head >= a.B * a.H_kv * a.G) return;
  const float2* st = a.ystat + (size_t)head * nsplit;
  const float* yp = a.ypart + (size_t)head * nsplit * D;
  float mx = -INFINITY;
  for (int p = lane; p < nsplit; p += 32) mx = fmaxf(mx, st[p].x);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float den = 0.f;
  float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int p = 0; p < nsplit; ++p) {
    const float2 v = st[p];
    const float sc = __expf(v.x - mx);
    den = fmaf(sc, v.y, den);
    const float4 y = *reinterpret_cast<const float4*>(yp + (size_t)p * D + lane * 4);
    num.x = fmaf(sc, y.x, num.x); num.y = fmaf(sc, y.y, num.y);
    num.z = fmaf(sc, y.z, num.z); num.w = fmaf(sc, y.w, num.w);
  }
  const float inv = 1.f / den;
  T* o = static_cast<T*>(a.out) + (size_t)head * D + lane * 4;
  store_elem(o, num.x * inv); store_elem(o + 1, num.y * inv);
  store_elem(o + 2, num.z * inv); store_elem(o + 3, num.w * inv);
}

template <typename T, int GT>
static cudaError_t launch_output_g(const DecodeArgs& a, cudaStream_t st) {
  const size_t smem = (size_t)OUT_PART_ROWS * D * sizeof(T) + sizeof(float) * ((size_t)OUT_PART_ROWS * GT + OUT_WARPS * GT * D);
  static size_t configured = 0;
  if (smem > configured) {
    cudaError_t e = cudaFuncSetAttribute(output_kernel<T, GT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  const unsigned grid = (unsigned)(a.B * a.H_kv * a.ws.nsplit);
  return launch_dependent(output_kernel<T, GT>, dim3(grid), dim3(256), smem, st, a);
}

template <typename T>
static cudaError_t launch_output_t(const DecodeArgs& a, cudaStream_t st) {
  cudaError_t e;
  {
    ProfScope prof(KVC_KERNEL_OUTPUT, st);
    if (a.G == 1) e = launch_output_g<T, 1>(a, st);
    else if (a.G == 2) e = launch_output_g<T, 2>(a, st);
    else if (a.G <= 4) e = launch_output_g<T, 4>(a, st);
    else e = launch_output_g<T, 8>(a, st);
  }
  if (e != cudaSuccess) return e;
  ProfScope prof(KVC_KERNEL_MERGE, st);
  const unsigned grid = (unsigned)ceil_div(a.B * a.H_kv * a.G, 8);
  return launch_dependent(merge_kernel<T>, dim3(grid), dim3(256), 0, st, a);
}

cudaError_t launch_output(const DecodeArgs& a, int dtype, cudaStream_t st) {
  return dtype == KVC_BF16 ? launch_output_t<__nv_bfloat16>(a, st) : launch_output_t<float>(a, st);
}

}  // namespace kvc
