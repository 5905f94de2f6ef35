// Split path, third kernel: Alg. 1 step 4, the text rows and the normalisation,
//   y = sum_r W_r V_tilde_r + (sum P) mu + P_txt V_txt,   out = y / (sum of all exponentials),
// as one streaming pass over V_tilde and over K_txt / V_txt, bound by HBM bandwidth.
//
// Work items are tiles of 64 rows: the text rows of a (sequence, KV head) in 64-row tiles, and the m rows of every
// block of V_tilde in 64-row tiles.  Both item lists are dealt in contiguous runs to one persistent CTA per SM; a CTA
// first takes its text run (which needs nothing from the expansion kernel, so it may run while that kernel finishes),
// then its run of value tiles.  A producer thread keeps a ring of TMA-filled stages full: a text stage holds 64 rows of
// K_txt and V_txt, a value stage 64 rows of V_tilde and the matching 64 columns of the partial weights of the block's
// G heads for every range of the n axis.  Eight consumer warps = 4 groups of 16 rows x 2 halves of the head dimension;
// all products are mma.sync m16n8k16 with the value rows transposed (head dimension as M, heads as N).
//   text tile    logits = q K_txt^T, online softmax per head, y^T += V_txt^T P^T
//   value tile   W[g][j] = sum_s 2^(max_s - max) Wp_s[g][j]  (the ranges joined while the B fragment is built),
//                y^T += V_tilde^T W^T; the probability mass of the block and the mu term come from the range sums
// A run of tiles of one (sequence, KV head) leaves one partial (max, sum, y) per head; the last run of that pair to
// arrive merges them by log-sum-exp and writes `out`.
#include "kvc_split.cuh"

namespace kvc {

constexpr int SO_WARPS = 8;
constexpr int SO_CONS = SO_WARPS * 32;
constexpr int SO_THREADS = SO_CONS + 32;
constexpr uint32_t SO_HALF = SP_OUT_ROWS * 128;       // 64 rows x 64 channels
constexpr int SO_QLD = 136;

template <int NH>
__global__ void __launch_bounds__(SO_THREADS, 1)
split_output_kernel(const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmKt,
                    const __grid_constant__ CUtensorMap tmVt, const __grid_constant__ CUtensorMap tmW, const SplitArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* sm = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
  __shared__ __align__(8) uint64_t full_bar[SP_MAX_STAGES], empty_bar[SP_MAX_STAGES];
  __shared__ int s_last;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < a.o_stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], SO_WARPS); }
    fence_mbar_init();
  }
  __syncthreads();

  const int G = a.G, R = a.R, NS = a.NS, vt = a.vt;
  const long long BH = (long long)a.B * a.H_kv;
  const int tt = (a.T + SP_OUT_ROWS - 1) / SP_OUT_ROWS;          // text tiles per (sequence, KV head)
  const int vb = R * vt;                                          // value tiles per (sequence, KV head)
  const long long tot_t = BH * tt, tot_v = BH * vb;
  // each list is dealt to the first min(grid, items) CTAs, so that every CTA that takes part owns at least one item and
  // the runs that hold tiles of one pair belong to consecutive CTAs
  const long long gt = tot_t < (long long)gridDim.x ? tot_t : (long long)gridDim.x;
  const long long gv = tot_v < (long long)gridDim.x ? tot_v : (long long)gridDim.x;
  const bool in_t = (long long)blockIdx.x < gt, in_v = (long long)blockIdx.x < gv;
  const long long tlo = in_t ? run_begin(blockIdx.x, tot_t, gt) : 0, thi = in_t ? run_begin(blockIdx.x + 1, tot_t, gt) : 0;
  const long long vlo = in_v ? run_begin(blockIdx.x, tot_v, gv) : 0, vhi = in_v ? run_begin(blockIdx.x + 1, tot_v, gv) : 0;
  const uint32_t w_bytes = (uint32_t)(NS * G) * 128u;

  if (warp == SO_WARPS) {
    // ================= producer =================
    if (lane != 0) return;
    tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmW);
    if (a.T > 0) { tma_prefetch_desc(&tmKt); tma_prefetch_desc(&tmVt); }
    uint32_t slot = 0, phase = 1;
    for (long long i = tlo; i < thi; ++i) {
      const int bh = (int)(i / tt), tile = (int)(i - (long long)bh * tt);
      const int b = bh / a.H_kv, h = bh - b * a.H_kv;
      if (!mbar_wait_bounded(&empty_bar[slot], phase)) { atomicExch(a.status, (int)KVC_ERR_TIMEOUT); return; }
      unsigned char* dst = sm + slot * a.o_stage_bytes;
      mbar_expect_tx(&full_bar[slot], 4 * SO_HALF);
      const int y = tile * SP_OUT_ROWS;
      tma_load_4d(dst, &tmKt, 0, y, h, b, &full_bar[slot]);
      tma_load_4d(dst + SO_HALF, &tmKt, 64, y, h, b, &full_bar[slot]);
      tma_load_4d(dst + 2 * SO_HALF, &tmVt, 0, y, h, b, &full_bar[slot]);
      tma_load_4d(dst + 3 * SO_HALF, &tmVt, 64, y, h, b, &full_bar[slot]);
      if (++slot == (uint32_t)a.o_stages) { slot = 0; phase ^= 1u; }
    }
    grid_dep_wait();                               // the partial weights come from the expansion kernel
    for (long long i = vlo; i < vhi; ++i) {
      const int bh = (int)(i / vb), rem = (int)(i - (long long)bh * vb);
      const int b = bh / a.H_kv, h = bh - b * a.H_kv;
      const int r = rem / vt, jt = rem - r * vt;
      if (!mbar_wait_bounded(&empty_bar[slot], phase)) { atomicExch(a.status, (int)KVC_ERR_TIMEOUT); return; }
      unsigned char* dst = sm + slot * a.o_stage_bytes;
      mbar_expect_tx(&full_bar[slot], 2 * SO_HALF + w_bytes);
      tma_load_5d(dst, &tmV, 0, jt * SP_OUT_ROWS, r, h, b, &full_bar[slot]);
      tma_load_5d(dst + SO_HALF, &tmV, 64, jt * SP_OUT_ROWS, r, h, b, &full_bar[slot]);
      tma_load_4d(dst + 2 * SO_HALF, &tmW, jt * SP_OUT_ROWS, (b * R + r) * G, 0, h, &full_bar[slot]);
      if (++slot == (uint32_t)a.o_stages) { slot = 0; phase ^= 1u; }
    }
    return;
  }

  // ================= consumers =================
  grid_dep_launch();
  const int gid = lane >> 2, t4 = lane & 3;
  const int rg = warp & 3, dh = warp >> 2;          // 16-row group of a tile; half of the head dimension
  const int l7 = lane & 7, lhi = lane >> 4, lmid = (lane >> 3) & 1;
  const int lrow = l7 + lmid * 8;                   // ldmatrix address pattern A: rows 0-15 by lanes 0-15, twice
  const int lrowB = l7 + lhi * 8;                   // pattern B: rows 0-7 | 0-7 | 8-15 | 8-15
  const uint32_t sm_u = smem_addr(sm);
  const uint32_t q_u = sm_u + a.o_off_q;
  __nv_bfloat16* q_sm = reinterpret_cast<__nv_bfloat16*>(sm + a.o_off_q);        // [16][SO_QLD]
  float2* fac = reinterpret_cast<float2*>(sm + a.o_off_fac);                     // [R*NS][16]: (factor, scaled row sum)
  float* red = reinterpret_cast<float*>(sm + a.o_off_red);                       // [8 warps][NH*8][64]
  float* tmax = reinterpret_cast<float*>(sm + a.o_off_stat);                     // [8][16]
  float* tsum = tmax + SO_WARPS * 16;                                            // [8][16]
  float* hmax = tsum + SO_WARPS * 16;                                            // [16] reference maximum of the segment
  float* hsum = hmax + 16;                                                       // [16] its sum of exponentials

  uint32_t slot = 0, phase = 0;
  bool dead = false;
  auto wait_full = [&]() {
    if (!dead && !mbar_wait_bounded(&full_bar[slot], phase)) dead = true;
    __syncwarp();
  };
  auto release = [&]() {
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[slot]);
    if (++slot == (uint32_t)a.o_stages) { slot = 0; phase ^= 1u; }
  };

  float yacc[4][NH][4];
  auto zero_acc = [&]() {
#pragma unroll
    for (int mt = 0; mt < 4; ++mt)
#pragma unroll
      for (int nh = 0; nh < NH; ++nh)
#pragma unroll
        for (int e = 0; e < 4; ++e) yacc[mt][nh][e] = 0.f;
  };

  // End of a run of tiles of one (sequence, KV head): the accumulators of the 4 row groups are summed per half of the
  // head dimension, the partial goes to slot `pslot`, and the last run of the pair to arrive merges all of them.
  // hmax / hsum hold the run's reference maximum and sum per head; mu_w[g] (by reference: hsum-like array) adds mu.
  auto flush = [&](int bh, int pslot, bool add_mu) {
    const int b = bh / a.H_kv, h = bh - b * a.H_kv;
    float* mine = red + (size_t)warp * (NH * 8 * 64);
#pragma unroll
    for (int nh = 0; nh < NH; ++nh)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        float* yp = mine + (nh * 8 + 2 * t4 + e) * 64;
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
          yp[mt * 16 + gid] = yacc[mt][nh][e];
          yp[mt * 16 + gid + 8] = yacc[mt][nh][2 + e];
        }
      }
    named_barrier_sync(1, SO_CONS);
    const int nslot = a.nslot_v + a.nslot_t;
    const size_t pbase = ((size_t)bh * nslot + pslot) * G;
    for (int idx = tid; idx < G * D; idx += SO_CONS) {
      const int g = idx >> 7, col = idx & (D - 1);
      const float* rp = red + (size_t)((col >> 6) * 4) * (NH * 8 * 64) + g * 64 + (col & 63);
      float y = rp[0] + rp[NH * 8 * 64] + rp[2 * NH * 8 * 64] + rp[3 * NH * 8 * 64];
      if (add_mu) y = fmaf(hsum[g], __bfloat162float(a.mu[h * D + col]), y);
      a.py[(pbase + g) * D + col] = y;
    }
    if (tid < G) a.pml[pbase + tid] = make_float2(hmax[tid], hsum[tid]);
    __threadfence();
    named_barrier_sync(1, SO_CONS);
    // how many runs hold tiles of this pair: those of the CTAs that own its first and last tile, per kind
    const int cv0 = vb > 0 ? run_owner((long long)bh * vb, tot_v, gv) : 0;
    const int nsv = vb > 0 ? run_owner((long long)(bh + 1) * vb - 1, tot_v, gv) - cv0 + 1 : 0;
    const int ct0 = tt > 0 ? run_owner((long long)bh * tt, tot_t, gt) : 0;
    const int nst = tt > 0 ? run_owner((long long)(bh + 1) * tt - 1, tot_t, gt) - ct0 + 1 : 0;
    if (tid == 0) s_last = atomicAdd(&a.cnt[bh], 1) + 1 == nsv + nst ? 1 : 0;
    named_barrier_sync(1, SO_CONS);
    if (s_last) {
      __threadfence();
      const size_t p0 = (size_t)bh * nslot * G;
      for (int idx = tid; idx < G * (D / 4); idx += SO_CONS) {
        const int g = idx >> 5, col = (idx & 31) * 4;
        float M = -INFINITY;
        for (int k = 0; k < nsv + nst; ++k) {
          const int p = k < nsv ? k : a.nslot_v + (k - nsv);
          M = fmaxf(M, __ldcg(&a.pml[p0 + (size_t)p * G + g]).x);
        }
        float den = 0.f;
        float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int k = 0; k < nsv + nst; ++k) {
          const int p = k < nsv ? k : a.nslot_v + (k - nsv);
          const float2 ml = __ldcg(&a.pml[p0 + (size_t)p * G + g]);
          const float w = ml.x == -INFINITY ? 0.f : fast_exp2(ml.x - M);
          den = fmaf(w, ml.y, den);
          const float4 y = __ldcg(reinterpret_cast<const float4*>(a.py + (p0 + (size_t)p * G + g) * D + col));
          num.x = fmaf(w, y.x, num.x); num.y = fmaf(w, y.y, num.y); num.z = fmaf(w, y.z, num.z); num.w = fmaf(w, y.w, num.w);
        }
        const float inv = 1.f / den;
        uint2 o;
        o.x = pack2_bf16(num.x * inv, num.y * inv); o.y = pack2_bf16(num.z * inv, num.w * inv);
        *reinterpret_cast<uint2*>(a.out + ((size_t)b * a.H_kv * G + (size_t)h * G + g) * D + col) = o;
      }
    }
    named_barrier_sync(1, SO_CONS);
  };

  // ------------------------------------------------------------------ text runs
  {
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};   // heads gid and gid + 8
    // brings the per-warp online-softmax state of the run to one maximum per head and leaves its partial
    auto flush_text = [&](int bh) {
      if (t4 == 0) { tmax[warp * 16 + gid] = m_run[0]; tmax[warp * 16 + gid + 8] = m_run[1]; }
      named_barrier_sync(1, SO_CONS);
      float scl[2];
#pragma unroll
      for (int hr = 0; hr < 2; ++hr) {
        const int head = gid + 8 * hr;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < SO_WARPS; ++w) M = fmaxf(M, tmax[w * 16 + head]);
        scl[hr] = m_run[hr] == -INFINITY ? 0.f : fast_exp2(m_run[hr] - M);
        float l = l_run[hr] * scl[hr];
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        if (t4 == 0) tsum[warp * 16 + head] = dh == 0 ? l : 0.f;     // the two halves of a row group hold the same sums
        if (warp == 0 && t4 == 0) hmax[head] = M;
      }
#pragma unroll
      for (int nh = 0; nh < NH; ++nh) {
        const float c0s = __shfl_sync(0xffffffffu, scl[nh], (2 * t4) * 4);
        const float c1s = __shfl_sync(0xffffffffu, scl[nh], (2 * t4 + 1) * 4);
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
          yacc[mt][nh][0] *= c0s; yacc[mt][nh][1] *= c1s;
          yacc[mt][nh][2] *= c0s; yacc[mt][nh][3] *= c1s;
        }
      }
      named_barrier_sync(1, SO_CONS);
      if (tid < 16) {
        float l = 0.f;
#pragma unroll
        for (int w = 0; w < SO_WARPS; ++w) l += tsum[w * 16 + tid];
        hsum[tid] = l;
      }
      named_barrier_sync(1, SO_CONS);
      const int ct0 = run_owner((long long)bh * tt, tot_t, gt);
      flush(bh, a.nslot_v + (int)blockIdx.x - ct0, false);
    };

    int cur_bh = -1;
    for (long long i = tlo; i < thi; ++i) {
      const int bh = (int)(i / tt), tile = (int)(i - (long long)bh * tt);
      if (bh != cur_bh) {
        if (cur_bh >= 0) flush_text(cur_bh);
        cur_bh = bh;
        const int b = bh / a.H_kv, h = bh - b * a.H_kv;
        // queries of the pair: [16 heads][128], heads >= G are zero rows
        for (int idx = tid; idx < 256; idx += SO_CONS) {
          const int g = idx >> 4, piece = idx & 15;
          uint4 v = make_uint4(0u, 0u, 0u, 0u);
          if (g < G) v = *reinterpret_cast<const uint4*>(a.q + ((size_t)b * a.H_kv * G + (size_t)h * G + g) * D + piece * 8);
          *reinterpret_cast<uint4*>(q_sm + g * SO_QLD + piece * 8) = v;
        }
        named_barrier_sync(1, SO_CONS);
        zero_acc();
        m_run[0] = m_run[1] = -INFINITY;
        l_run[0] = l_run[1] = 0.f;
      }
      wait_full();
      const uint32_t kt_u = sm_u + slot * a.o_stage_bytes, vt_u = kt_u + 2 * SO_HALF;
      const int t_first = tile * SP_OUT_ROWS + rg * 16;
      if (t_first < a.T) {
        const uint32_t rowB = (uint32_t)((rg * 16 + lrowB) * 128);
        // logits [16 heads][16 text rows] = q K_txt^T
        float cc[2][4];
        {
          float c2[2][2][4];
#pragma unroll
          for (int x = 0; x < 2; ++x)
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
              for (int e = 0; e < 4; ++e) c2[x][nt][e] = 0.f;
#pragma unroll
          for (int kh = 0; kh < 2; ++kh) {
            uint32_t bk[4][4], aq[4][4];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
              const int ks = kh * 4 + x;
              ldsm_x4(bk[x], kt_u + kh * SO_HALF + rowB + (uint32_t)((((x * 2 + lmid)) ^ l7) << 4));
              ldsm_x4(aq[x], q_u + (uint32_t)((lrow * SO_QLD + ks * 16 + lhi * 8) * 2));
            }
#pragma unroll
            for (int x = 0; x < 4; ++x) {
              mma_bf16_16816(c2[x & 1][0], aq[x], bk[x][0], bk[x][1]);
              mma_bf16_16816(c2[x & 1][1], aq[x], bk[x][2], bk[x][3]);
            }
          }
#pragma unroll
          for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) cc[nt][e] = c2[0][nt][e] + c2[1][nt][e];
        }
        // cc[nt][e]: head gid + 8 (e >> 1), text row t_first + nt*8 + 2 t4 + (e & 1)
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int t = t_first + nt * 8 + 2 * t4 + (e & 1);
            cc[nt][e] = t < a.T ? cc[nt][e] * SP_QSCALE : -INFINITY;
          }
        float scl[2];
#pragma unroll
        for (int hr = 0; hr < 2; ++hr) {
          float mx = fmaxf(fmaxf(cc[0][2 * hr], cc[0][2 * hr + 1]), fmaxf(cc[1][2 * hr], cc[1][2 * hr + 1]));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
          const float m_new = fmaxf(m_run[hr], mx);              // finite: the 16 rows hold at least one valid row
          scl[hr] = fast_exp2(m_run[hr] - m_new);                // 0 on the first tile
          m_run[hr] = m_new;
          float ps = 0.f;
#pragma unroll
          for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int k = 0; k < 2; ++k) {
              const float p = fast_exp2(cc[nt][2 * hr + k] - m_new);
              cc[nt][2 * hr + k] = p;
              ps += p;
            }
          l_run[hr] = l_run[hr] * scl[hr] + ps;
        }
#pragma unroll
        for (int nh = 0; nh < NH; ++nh) {
          const float c0s = __shfl_sync(0xffffffffu, scl[nh], (2 * t4) * 4);
          const float c1s = __shfl_sync(0xffffffffu, scl[nh], (2 * t4 + 1) * 4);
          if (c0s != 1.f || c1s != 1.f) {
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
              yacc[mt][nh][0] *= c0s; yacc[mt][nh][1] *= c1s;
              yacc[mt][nh][2] *= c0s; yacc[mt][nh][3] *= c1s;
            }
          }
        }
        // y^T[64 of 128][heads] += V_txt^T[64][16 rows] P^T[16 rows][heads]
        uint32_t pb[2][2];
        pb[0][0] = pack2_bf16(cc[0][0], cc[0][1]); pb[0][1] = pack2_bf16(cc[1][0], cc[1][1]);
        pb[1][0] = pack2_bf16(cc[0][2], cc[0][3]); pb[1][1] = pack2_bf16(cc[1][2], cc[1][3]);
        uint32_t av[4][4];
#pragma unroll
        for (int mt = 0; mt < 4; ++mt)
          ldsm_x4_t(av[mt], vt_u + dh * SO_HALF + rowB + (uint32_t)((((mt * 2 + lmid)) ^ l7) << 4));
#pragma unroll
        for (int mt = 0; mt < 4; ++mt)
#pragma unroll
          for (int nh = 0; nh < NH; ++nh) mma_bf16_16816(yacc[mt][nh], av[mt], pb[nh][0], pb[nh][1]);
      }
      release();
    }
    if (cur_bh >= 0) flush_text(cur_bh);
  }

  // ------------------------------------------------------------------ value runs
  grid_dep_wait();                                   // row statistics and partial weights of the expansion kernel
  {
    int cur_bh = -1, cur_b = 0, cur_h = 0;
    bool has_first = false;
    auto flush_values = [&](int bh) {
      // hmax holds the vision-only maximum per head; the run that holds the pair's first tile carries the whole
      // probability mass of the vision positions (and with it the mu term), the others none
      if (!has_first && tid < 16) hsum[tid] = 0.f;
      named_barrier_sync(1, SO_CONS);
      const int cv0 = run_owner((long long)bh * vb, tot_v, gv);
      flush(bh, (int)blockIdx.x - cv0, has_first);
    };
    for (long long i = vlo; i < vhi; ++i) {
      const int bh = (int)(i / vb), rem = (int)(i - (long long)bh * vb);
      const int r = rem / vt, jt = rem - r * vt;
      if (bh != cur_bh) {
        if (cur_bh >= 0) flush_values(cur_bh);
        cur_bh = bh;
        cur_b = bh / a.H_kv; cur_h = bh - cur_b * a.H_kv;
        has_first = rem == 0;
        // row statistics of every (block, range, head) of the pair -> maximum per head, factor per entry, mass per head
        const int ne = R * NS;
        for (int idx = tid; idx < ne * 16; idx += SO_CONS) {
          const int e = idx >> 4, g = idx & 15, rr = e / NS, s = e - rr * NS;
          float2 v = make_float2(-INFINITY, 0.f);
          if (g < G) v = __ldcg(&a.stat[((size_t)cur_h * NS + s) * a.rows_h + (size_t)(cur_b * R + rr) * G + g]);
          fac[idx] = v;
        }
        named_barrier_sync(1, SO_CONS);
        for (int g = warp; g < 16; g += SO_WARPS) {
          float mx = -INFINITY;
          for (int e = lane; e < ne; e += 32) mx = fmaxf(mx, fac[e * 16 + g].x);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
          float l = 0.f;
          for (int e = lane; e < ne; e += 32) {
            const float2 v = fac[e * 16 + g];
            const float f = g < G ? fast_exp2(v.x - mx) : 0.f;
            fac[e * 16 + g] = make_float2(f, f * v.y);
            l += f * v.y;
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
          if (lane == 0) { hmax[g] = g < G ? mx : -INFINITY; hsum[g] = g < G ? l : 0.f; }
        }
        named_barrier_sync(1, SO_CONS);
        zero_acc();
      }
      wait_full();
      const uint32_t v_u = sm_u + slot * a.o_stage_bytes;
      const unsigned char* wp = sm + slot * a.o_stage_bytes + 2 * SO_HALF;      // [NS][G][64] bf16
      if (jt * SP_OUT_ROWS + rg * 16 < a.m) {
        // B fragments: the weights of heads gid (+8) for rows 2 t4, 2 t4 + 1 (+8) of this row group, ranges joined
        uint32_t bw[NH][2];
#pragma unroll
        for (int nh = 0; nh < NH; ++nh) {
          const int g = gid + 8 * nh;
          float w0 = 0.f, w1 = 0.f, w2 = 0.f, w3 = 0.f;
          if (g < G) {
            for (int s = 0; s < NS; ++s) {
              const float f = fac[(r * NS + s) * 16 + g].x;
              const unsigned char* row = wp + (size_t)(s * G + g) * 128 + (rg * 16 + 2 * t4) * 2;
              const uint32_t lo = *reinterpret_cast<const uint32_t*>(row), hi = *reinterpret_cast<const uint32_t*>(row + 16);
              w0 = fmaf(f, __uint_as_float(lo << 16), w0); w1 = fmaf(f, __uint_as_float(lo & 0xffff0000u), w1);
              w2 = fmaf(f, __uint_as_float(hi << 16), w2); w3 = fmaf(f, __uint_as_float(hi & 0xffff0000u), w3);
            }
          }
          bw[nh][0] = pack2_bf16(w0, w1);
          bw[nh][1] = pack2_bf16(w2, w3);
        }
        const uint32_t rowB = (uint32_t)((rg * 16 + lrowB) * 128);
        uint32_t av[4][4];
#pragma unroll
        for (int mt = 0; mt < 4; ++mt)
          ldsm_x4_t(av[mt], v_u + dh * SO_HALF + rowB + (uint32_t)((((mt * 2 + lmid)) ^ l7) << 4));
#pragma unroll
        for (int mt = 0; mt < 4; ++mt)
#pragma unroll
          for (int nh = 0; nh < NH; ++nh) mma_bf16_16816(yacc[mt][nh], av[mt], bw[nh][0], bw[nh][1]);
      }
      release();
    }
    if (cur_bh >= 0) flush_values(cur_bh);
  }
  if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
}

cudaError_t launch_split_output(const CUtensorMap* tm, const SplitArgs& a, const SplitPlan& p, cudaStream_t st) {
  ProfScope prof(KVC_KERNEL_SPLIT_OUTPUT, st);
  if (a.G > 8) {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(split_output_kernel<2>), p.o_smem);
    if (e != cudaSuccess) return e;
    return launch_dependent(split_output_kernel<2>, dim3(p.o_grid), dim3(SO_THREADS), p.o_smem, st, tm[0], tm[1], tm[2], tm[3], a);
  }
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(split_output_kernel<1>), p.o_smem);
  if (e != cudaSuccess) return e;
  return launch_dependent(split_output_kernel<1>, dim3(p.o_grid), dim3(SO_THREADS), p.o_smem, st, tm[0], tm[1], tm[2], tm[3], a);
}

}  // namespace kvc
