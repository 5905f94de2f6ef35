// Step 4 of Algorithm 1 plus the text values and the final normalisation:
//   y = sum_r W_r V_tilde_r + (sum P) mu + P_txt V_txt,   out = y / (sum of all exp terms).
// One streaming pass over the compressed values and the text values; bound by HBM bandwidth.
//
// Persistent, warp-specialised kernel.  The value rows of all (sequence, KV head) pairs are cut into
// chunks of at most OUT_CHUNK rows that never straddle a vision block or the vision/text boundary;
// the flat chunk list is divided evenly over a grid of one resident wave, CTA c streaming chunks
// [c*cpc, (c+1)*cpc).  One producer warp keeps a ring of OUT_STAGES stages full with the bulk-copy
// engine (cp.async.bulk + mbarrier): per stage the rows of a chunk and, per query head, the matching
// slice of the combined W row plus its (max, sum), or the matching slice of the text logits.  Eight
// consumer warps turn each stage into a weighted sum of its rows with an online-softmax running
// maximum per head, so no thread of the kernel issues a global load on the critical path.  When the
// chunk range of a CTA leaves a (sequence, KV head), the consumers reduce their accumulators and
// write one partial (max, sum, y) per head; a second, tiny kernel merges the partials by log-sum-exp.
#include "kvc_async.cuh"
#include "kvc_internal.cuh"

namespace kvc {

constexpr int OUT_STAGES = 4;
constexpr int OUT_WARPS = 8;                       // consumer warps
constexpr int OUT_THREADS = (OUT_WARPS + 1) * 32;  // + one producer warp

struct ChunkRef {
  int bh, h, b;
  bool is_txt;
  int r;          // vision block (vision chunks)
  int j0;         // first row of the chunk within its block, or first text row
  int rows;       // rows in the chunk
};

__device__ __forceinline__ ChunkRef chunk_ref(const DecodeArgs& a, int q) {
  ChunkRef c;
  c.bh = q / a.ws.chunks_per_bh;
  const int lc = q - c.bh * a.ws.chunks_per_bh;
  c.b = c.bh / a.H_kv;
  c.h = c.bh - c.b * a.H_kv;
  const int nvis = a.R * a.ws.cpb;
  c.is_txt = lc >= nvis;
  if (c.is_txt) {
    c.r = 0;
    c.j0 = (lc - nvis) * OUT_CHUNK;
    c.rows = min(OUT_CHUNK, seq_T(a, c.b) - c.j0);   // <= 0 for chunks beyond the sequence's text length
  } else {
    c.r = lc / a.ws.cpb;
    c.j0 = (lc - c.r * a.ws.cpb) * OUT_CHUNK;
    c.rows = c.r < seq_R(a, c.b) ? min(OUT_CHUNK, a.mv - c.j0) : 0;   // 0 for a block the sequence does not have
  }
  return c;
}

template <typename T, int GT>
struct OutSmem {
  static constexpr uint32_t ROW_BYTES = D * sizeof(T);
  static constexpr uint32_t DATA_BYTES = OUT_CHUNK * ROW_BYTES;
  static constexpr uint32_t W_BYTES = GT * OUT_CHUNK * sizeof(float);       // weights or logits, [GT][OUT_CHUNK]
  static constexpr uint32_t STAT_BYTES = GT * sizeof(float4);               // (max, sum, 0, 0) per head
  static constexpr uint32_t STAGE_BYTES = DATA_BYTES + W_BYTES + ((STAT_BYTES + 127) / 128) * 128;
  static constexpr uint32_t RED_BYTES = OUT_WARPS * GT * D * sizeof(float);
  static constexpr uint32_t TOTAL = OUT_STAGES * STAGE_BYTES + RED_BYTES;
};

template <typename T, int GT>
__global__ void __launch_bounds__(OUT_THREADS) output_kernel(DecodeArgs a, int g_base) {
  using SM = OutSmem<T, GT>;
  constexpr int EPV = Elems16<T>::N;
  constexpr int LPR = D / EPV;               // lanes per row
  constexpr int RPI = 32 / LPR;              // rows per warp step

  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* ring = smem_raw;
  float* red = reinterpret_cast<float*>(ring + OUT_STAGES * SM::STAGE_BYTES);   // [OUT_WARPS][GT][D]
  __shared__ __align__(8) uint64_t full_bar[OUT_STAGES], empty_bar[OUT_STAGES];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long total = (long long)a.B * a.H_kv * a.ws.chunks_per_bh;
  const int q_begin = blockIdx.x * a.ws.cpc;
  const int q_end = (int)min((long long)q_begin + a.ws.cpc, total);
  const int nrows_h = a.B * a.G * a.R;
  const int gcount = min(GT, a.G - g_base);    // heads handled by this launch

  if (tid == 0) {
    for (int s = 0; s < OUT_STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], OUT_WARPS); }
    fence_mbar_init();
  }
  __syncthreads();

  if (warp == OUT_WARPS) {
    // ================= producer warp =================
    if (lane == 0) {
      bool dead = false;
      // copies of one chunk: the value rows (written before the kernels this one follows) and, per head,
      // the weights / logits produced by the kernels this one follows
      auto issue = [&](int q, int stage, bool data, bool weights) {
        const ChunkRef c = chunk_ref(a, q);
        unsigned char* sbase = ring + stage * SM::STAGE_BYTES;
        if (c.rows <= 0) {                       // no rows: the stage completes at once
          if (data) mbar_expect_tx(&full_bar[stage], 0);
          return;
        }
        const uint32_t wbytes = (uint32_t)((c.rows + 3) & ~3) * (uint32_t)sizeof(float);
        const uint32_t data_bytes = (uint32_t)c.rows * SM::ROW_BYTES;
        if (data) {
          mbar_expect_tx(&full_bar[stage], data_bytes + gcount * wbytes +
                                               (c.is_txt ? 0u : (uint32_t)gcount * (uint32_t)sizeof(float4)));
          const T* src = c.is_txt ? static_cast<const T*>(a.V_txt) + ((size_t)c.bh * a.T_cap + c.j0) * D
                                  : static_cast<const T*>(a.Vc) + (((size_t)c.bh * a.R + c.r) * a.mv + c.j0) * D;
          bulk_g2s(sbase, src, data_bytes, &full_bar[stage]);
        }
        if (weights) {
          float* wdst = reinterpret_cast<float*>(sbase + SM::DATA_BYTES);
          float4* sdst = reinterpret_cast<float4*>(sbase + SM::DATA_BYTES + SM::W_BYTES);
          for (int g = 0; g < gcount; ++g) {
            if (c.is_txt) {
              bulk_g2s(wdst + g * OUT_CHUNK, a.s_txt + ((size_t)c.bh * a.G + g_base + g) * a.Ts + c.j0, wbytes,
                       &full_bar[stage]);
            } else {
              const size_t row_id = (size_t)c.h * nrows_h + (size_t)(c.b * a.G + g_base + g) * a.R + c.r;
              bulk_g2s(wdst + g * OUT_CHUNK, a.Wcomb + row_id * a.msv + c.j0, wbytes, &full_bar[stage]);
              bulk_g2s(sdst + g, a.statc + row_id, (uint32_t)sizeof(float4), &full_bar[stage]);
            }
          }
        }
      };
      const int n = q_end - q_begin;
      const int n_pre = min(n, OUT_STAGES);
      for (int it = 0; it < n_pre; ++it) issue(q_begin + it, it, true, false);
      grid_dep_wait();
      grid_dep_launch();
      for (int it = 0; it < n_pre; ++it) issue(q_begin + it, it, false, true);
      for (int it = n_pre; it < n; ++it) {
        const int stage = it % OUT_STAGES, use = it / OUT_STAGES;
        if (!mbar_wait_bounded(&empty_bar[stage], (uint32_t)(use - 1) & 1u)) { dead = true; break; }
        issue(q_begin + it, stage, true, true);
      }
      if (dead) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
    }
    return;
  }

  // ================= consumer warps =================
  const int sub = lane / LPR, c16 = lane % LPR;
  float acc[GT][EPV];
  float run_max[GT], run_sum[GT];
  auto reset = [&]() {
#pragma unroll
    for (int g = 0; g < GT; ++g) {
      run_max[g] = -INFINITY;
      run_sum[g] = 0.f;
#pragma unroll
      for (int e = 0; e < EPV; ++e) acc[g][e] = 0.f;
    }
  };
  reset();
  float mu_sum[GT];                 // probability mass of the vision blocks seen in this piece (for the mu term)
#pragma unroll
  for (int g = 0; g < GT; ++g) mu_sum[g] = 0.f;

  bool dead = false;
  for (int q = q_begin, it = 0; q < q_end; ++q, ++it) {
    const int stage = it % OUT_STAGES, use = it / OUT_STAGES;
    const ChunkRef c = chunk_ref(a, q);
    if (!dead && !mbar_wait_bounded(&full_bar[stage], (uint32_t)use & 1u)) dead = true;
    const unsigned char* sbase = ring + stage * SM::STAGE_BYTES;
    const float* wsm = reinterpret_cast<const float*>(sbase + SM::DATA_BYTES);
    const float4* ssm = reinterpret_cast<const float4*>(sbase + SM::DATA_BYTES + SM::W_BYTES);
    if (!dead && c.rows > 0) {
      // ---- reference maximum of the chunk per head, running maximum of the piece
      float scale[GT];              // factor applied to the chunk's stored weights (vision) / unused (text)
#pragma unroll
      for (int g = 0; g < GT; ++g) {
        scale[g] = 0.f;
        if (g < gcount) {
          float cm, csum = 0.f;
          if (c.is_txt) {
            float v0 = lane < c.rows ? wsm[g * OUT_CHUNK + lane] : -INFINITY;
            float v1 = lane + 32 < c.rows ? wsm[g * OUT_CHUNK + lane + 32] : -INFINITY;
            cm = fmaxf(v0, v1);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, o));
          } else {
            const float4 st = ssm[g];
            cm = st.x;
            csum = c.j0 == 0 ? st.y : 0.f;     // a block's probability mass is counted with its first chunk
          }
          const float m_new = fmaxf(run_max[g], cm);
          const float resc = run_max[g] == -INFINITY ? 0.f : __expf(run_max[g] - m_new);
          if (resc != 1.f) {
            run_sum[g] *= resc;
            mu_sum[g] *= resc;
#pragma unroll
            for (int e = 0; e < EPV; ++e) acc[g][e] *= resc;
          }
          run_max[g] = m_new;
          if (c.is_txt) {
            // p = exp(s - max) per row; every warp needs the sum only once: warp 0 keeps it
            float p0 = lane < c.rows ? __expf(wsm[g * OUT_CHUNK + lane] - m_new) : 0.f;
            float p1 = lane + 32 < c.rows ? __expf(wsm[g * OUT_CHUNK + lane + 32] - m_new) : 0.f;
            float ps = p0 + p1;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
            run_sum[g] += ps;
            scale[g] = m_new;                   // text rows: weight = exp(s - scale)
          } else {
            scale[g] = __expf(cm - m_new);      // vision rows: weight = W * scale
            run_sum[g] = fmaf(csum, scale[g], run_sum[g]);
            mu_sum[g] = fmaf(csum, scale[g], mu_sum[g]);
          }
        }
      }
      // ---- acc[g][e] += w[row][g] * x[row][e]
#pragma unroll 2
      for (int rr = warp * RPI + sub; rr < c.rows; rr += OUT_WARPS * RPI) {
        const uint4 v = *reinterpret_cast<const uint4*>(sbase + (size_t)rr * SM::ROW_BYTES + c16 * 16);
        float x[EPV];
        unpack16(v, x, (T*)nullptr);
#pragma unroll
        for (int g = 0; g < GT; ++g) {
          if (g < gcount) {
            const float sv = wsm[g * OUT_CHUNK + rr];
            const float w = c.is_txt ? __expf(sv - scale[g]) : sv * scale[g];
#pragma unroll
            for (int e = 0; e < EPV; ++e) acc[g][e] = fmaf(w, x[e], acc[g][e]);
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[stage]);

    // ---- end of this CTA's piece of the (sequence, KV head): reduce over warps, write the partial
    const bool piece_end = (q + 1 == q_end) || ((q + 1) / a.ws.chunks_per_bh != c.bh);
    if (piece_end) {
#pragma unroll
      for (int g = 0; g < GT; ++g)
#pragma unroll
        for (int e = 0; e < EPV; ++e) {
          float v = acc[g][e];
#pragma unroll
          for (int o = LPR; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
          if (sub == 0) red[(warp * GT + g) * D + c16 * EPV + e] = v;
        }
      named_barrier_sync(1, OUT_WARPS * 32);
      const int c_first = (int)(((long long)c.bh * a.ws.chunks_per_bh) / a.ws.cpc);
      const int slot = blockIdx.x - c_first;
      for (int x = tid; x < GT * D; x += OUT_WARPS * 32) {
        const int g = x / D, col = x % D;
        if (g < gcount) {
          float y = 0.f;
#pragma unroll
          for (int w = 0; w < OUT_WARPS; ++w) y += red[(w * GT + g) * D + col];
          // all warps hold the same run_max / mu_sum (they saw the same chunks)
          float ms_g = 0.f;
#pragma unroll
          for (int k = 0; k < GT; ++k) if (k == g) ms_g = mu_sum[k];
          if (!a.passthrough && !a.id_U) y = fmaf(ms_g, to_f32(static_cast<const T*>(a.mu)[c.h * D + col]), y);
          a.ypart[(((size_t)c.bh * a.G + g_base + g) * a.ws.nsplit + slot) * D + col] = y;
        }
      }
      if (tid < gcount) {
        float mx = 0.f, sm = 0.f;
#pragma unroll
        for (int k = 0; k < GT; ++k) if (k == tid) { mx = run_max[k]; sm = run_sum[k]; }
        a.ystat[((size_t)c.bh * a.G + g_base + tid) * a.ws.nsplit + slot] = make_float2(mx, sm);
      }
      named_barrier_sync(1, OUT_WARPS * 32);      // red is reused by the next piece
      reset();
#pragma unroll
      for (int g = 0; g < GT; ++g) mu_sum[g] = 0.f;
    }
  }
  if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
}

// out[b,hq,:] = sum_p e^{max_p - M} y_p / sum_p e^{max_p - M} l_p over the partials p of (b, hq): one warp per head.
template <typename T>
__global__ void __launch_bounds__(256) merge_kernel(DecodeArgs a) {
  grid_dep_wait();
  grid_dep_launch();
  const int head = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;   // flat (b, h, g)
  if (head >= a.B * a.H_kv * a.G) return;
  const int bh = head / a.G;
  const int c_first = (int)(((long long)bh * a.ws.chunks_per_bh) / a.ws.cpc);
  const int c_last = (int)(((long long)(bh + 1) * a.ws.chunks_per_bh - 1) / a.ws.cpc);
  const int np = c_last - c_first + 1;
  const float2* st = a.ystat + (size_t)head * a.ws.nsplit;
  const float* yp = a.ypart + (size_t)head * a.ws.nsplit * D;
  float mx = -INFINITY;
  for (int p = lane; p < np; p += 32) mx = fmaxf(mx, st[p].x);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float den = 0.f;
  float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int p = 0; p < np; ++p) {
    const float2 v = st[p];
    if (v.x == -INFINITY) continue;              // a piece without rows (text chunks beyond T)
    const float sc = __expf(v.x - mx);
    den = fmaf(sc, v.y, den);
    const float4 y = *reinterpret_cast<const float4*>(yp + (size_t)p * D + lane * 4);
    num.x = fmaf(sc, y.x, num.x); num.y = fmaf(sc, y.y, num.y);
    num.z = fmaf(sc, y.z, num.z); num.w = fmaf(sc, y.w, num.w);
  }
  const float inv = den > 0.f ? 1.f / den : 0.f;     // a sequence without any row: a zero output row
  T* o = static_cast<T*>(a.out) + (size_t)head * D + lane * 4;
  store_elem(o, num.x * inv); store_elem(o + 1, num.y * inv);
  store_elem(o + 2, num.z * inv); store_elem(o + 3, num.w * inv);
}

template <typename T, int GT>
static cudaError_t launch_output_g(const DecodeArgs& a, cudaStream_t st) {
  const size_t smem = OutSmem<T, GT>::TOTAL;
  {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(output_kernel<T, GT>), smem);
    if (e != cudaSuccess) return e;
  }
  for (int g_base = 0; g_base < a.G; g_base += GT) {
    cudaError_t e = launch_dependent(output_kernel<T, GT>, dim3(a.ws.out_ctas), dim3(OUT_THREADS), smem, st, a, g_base);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

template <typename T>
static cudaError_t launch_output_t(const DecodeArgs& a, cudaStream_t st) {
  cudaError_t e;
  {
    ProfScope prof(KVC_KERNEL_OUTPUT, st);
    if (a.ws.GT == 1) e = launch_output_g<T, 1>(a, st);
    else if (a.ws.GT == 2) e = launch_output_g<T, 2>(a, st);
    else if (a.ws.GT == 4) e = launch_output_g<T, 4>(a, st);
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
