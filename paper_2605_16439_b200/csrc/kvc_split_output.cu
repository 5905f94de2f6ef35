// Split path, third kernel: Alg. 1 step 4, the text rows and the normalisation,
//   y = sum_r W_r V_tilde_r + (sum P) mu + P_txt V_txt,   out = y / (sum of all exponentials),
// as one streaming pass over V_tilde and over K_txt / V_txt, bound by HBM bandwidth.
//
// Work items are tiles of 64 rows: the text rows of a (sequence, KV head) and the m rows of every block of its V_tilde.
// A pair's tiles go to `cpb` CTAs (as many as the SMs allow, the same number for every pair), each taking an equal share
// of the text tiles and of the value tiles; with more pairs than SMs a CTA takes whole pairs one after the other.  A CTA
// first takes its text tiles (which need nothing from the expansion kernel, so they may run while that kernel finishes),
// then its value tiles.  A producer thread keeps a ring of TMA-filled stages full: a text stage holds 64 rows of K_txt
// and V_txt, a value stage 64 rows of V_tilde and the matching 64 columns of the partial weights of the block's G heads
// for every range of the n axis.  The eight consumer warps form two groups of four; tile k of the CTA's list goes to
// group k mod 2 and each warp of the group takes 16 of its rows over the whole head dimension; all products are mma.sync
// m16n8k16 with the value rows transposed (head dimension as M, heads as N).
//   text tile    logits = q K_txt^T, online softmax per head, y^T += V_txt^T P^T
//   value tile   W[g][j] = sum_s 2^(max_s - max) Wp_s[g][j]  (the ranges joined while the B fragment is built),
//                y^T += V_tilde^T W^T; the probability mass of the vision positions and the mu term come from the range sums
// The text part and the value part of a CTA meet in shared memory at one maximum per head.  With one CTA per pair the
// result is normalised and written; otherwise the CTA leaves one partial (max, sum, y) per head and the last CTA of the
// pair to arrive merges them by log-sum-exp.
#include "kvc_split.cuh"

namespace kvc {

constexpr int SO_WARPS = 8;
constexpr int SO_CONS = SO_WARPS * 32;
constexpr int SO_THREADS = SO_CONS + 32;
constexpr uint32_t SO_HALF = SP_OUT_ROWS * 128;       // 64 rows x 64 channels

template <int NH>
__global__ void __launch_bounds__(SO_THREADS, 1)
split_output_kernel(const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmKt,
                    const __grid_constant__ CUtensorMap tmVt, const __grid_constant__ CUtensorMap tmW, const SplitArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* sm = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
  __shared__ __align__(8) uint64_t full_bar[SP_MAX_STAGES], empty_bar[SP_MAX_STAGES];
  __shared__ uint32_t released[SP_MAX_STAGES];
  __shared__ int s_last;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < a.o_stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], SP_GROUP); released[s] = 0u; }
    fence_mbar_init();
  }
  __syncthreads();

  const int G = a.G, R = a.R, NS = a.NS, vt = a.vt, nst = a.o_stages, cpb = a.o_cpb;
  const int BH = a.B * a.H_kv;
  const int tt = (a.T + SP_OUT_ROWS - 1) / SP_OUT_ROWS;          // text tiles per (sequence, KV head)
  const int vb = R * vt;                                          // value tiles per (sequence, KV head)
  // this CTA's pairs and its share of their tiles
  const int bh_first = cpb > 1 ? (int)blockIdx.x / cpb : (int)blockIdx.x;
  const int bh_step = cpb > 1 ? BH : (int)gridDim.x;
  const int part = cpb > 1 ? (int)blockIdx.x % cpb : 0;
  const int t0 = (int)((long long)part * tt / cpb), t1 = (int)((long long)(part + 1) * tt / cpb);
  const int v0 = (int)((long long)part * vb / cpb), v1 = (int)((long long)(part + 1) * vb / cpb);
  const int per_bh = (t1 - t0) + (v1 - v0);                      // ring ordinals per pair: text tiles, then value tiles
  const uint32_t w_bytes = (uint32_t)(NS * G) * 128u;

  if (warp == SO_WARPS) {
    // ================= producer =================
    if (lane != 0) return;
    tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmW);
    if (a.T > 0) { tma_prefetch_desc(&tmKt); tma_prefetch_desc(&tmVt); }
    uint32_t slot = 0, phase = 1;
    bool waited = false;
    for (int bh = bh_first; bh < BH; bh += bh_step) {
      const int b = bh / a.H_kv, h = bh - b * a.H_kv;
      for (int tile = t0; tile < t1; ++tile) {
        if (!mbar_wait_bounded(&empty_bar[slot], phase)) { atomicExch(a.status, (int)KVC_ERR_TIMEOUT); return; }
        unsigned char* dst = sm + slot * a.o_stage_bytes;
        mbar_expect_tx(&full_bar[slot], 4 * SO_HALF);
        const int y = tile * SP_OUT_ROWS;
        tma_load_4d(dst, &tmKt, 0, y, h, b, &full_bar[slot]);
        tma_load_4d(dst + SO_HALF, &tmKt, 64, y, h, b, &full_bar[slot]);
        tma_load_4d(dst + 2 * SO_HALF, &tmVt, 0, y, h, b, &full_bar[slot]);
        tma_load_4d(dst + 3 * SO_HALF, &tmVt, 64, y, h, b, &full_bar[slot]);
        if (++slot == (uint32_t)nst) { slot = 0; phase ^= 1u; }
      }
      if (!waited) { grid_dep_wait(); waited = true; }     // the partial weights come from the expansion kernel
      for (int rem = v0; rem < v1; ++rem) {
        const int r = rem / vt, jt = rem - r * vt;
        if (!mbar_wait_bounded(&empty_bar[slot], phase)) { atomicExch(a.status, (int)KVC_ERR_TIMEOUT); return; }
        unsigned char* dst = sm + slot * a.o_stage_bytes;
        mbar_expect_tx(&full_bar[slot], 2 * SO_HALF + w_bytes);
        tma_load_5d(dst, &tmV, 0, jt * SP_OUT_ROWS, r, h, b, &full_bar[slot]);
        tma_load_5d(dst + SO_HALF, &tmV, 64, jt * SP_OUT_ROWS, r, h, b, &full_bar[slot]);
        tma_load_4d(dst + 2 * SO_HALF, &tmW, jt * SP_OUT_ROWS, (b * R + r) * G, 0, h, &full_bar[slot]);
        if (++slot == (uint32_t)nst) { slot = 0; phase ^= 1u; }
      }
    }
    return;
  }

  // ================= consumers: tile k of the CTA's list goes to warp group k mod 2, 16 rows to each of its warps =================
  grid_dep_launch();
  constexpr int NGRP = SO_WARPS / SP_GROUP;
  const int grp = warp / SP_GROUP, rg = warp % SP_GROUP;      // warp group; the 16-row group of a tile this warp takes
  const int gid = lane >> 2, t4 = lane & 3;
  const int l7 = lane & 7, lhi = lane >> 4, lmid = (lane >> 3) & 1;
  const int lrowB = l7 + lhi * 8;                   // ldmatrix address pattern: rows 0-7 | 0-7 | 8-15 | 8-15
  const uint32_t sm_u = smem_addr(sm);
  float2* fac = reinterpret_cast<float2*>(sm + a.o_off_fac);                     // [R*NS][16]: (factor, scaled row sum)
  float* red = reinterpret_cast<float*>(sm + a.o_off_red);                       // [8 warps][NH*8][128]
  float* tbuf = reinterpret_cast<float*>(sm + a.o_off_q);                        // [16][128] text part of the pair
  float* tmax = reinterpret_cast<float*>(sm + a.o_off_stat);                     // [8][16]
  float* tsum = tmax + SO_WARPS * 16;                                            // [8][16]
  float* hmax = tsum + SO_WARPS * 16;                                            // [16] maximum over the vision logits
  float* hsum = hmax + 16;                                                       // [16] probability mass carried by this CTA
  float* txm = hsum + 16;                                                        // [16] maximum over this CTA's text rows
  float* txl = txm + 16;                                                         // [16] their sum of exponentials
  float* mlm = txl + 16;                                                         // merge: [cpb][16] maxima, sums -> weights

  bool dead = false, waited = false;
  auto wait_full = [&](long long k) {
    const uint32_t slot = (uint32_t)(k % nst), round = (uint32_t)(k / nst);
    if (!dead && !(wait_round(released, slot, round) && mbar_wait_bounded(&full_bar[slot], round & 1u))) dead = true;
    __syncwarp();
  };
  auto release = [&](long long k) {
    __syncwarp();
    if (lane == 0) release_slot(released, empty_bar, (uint32_t)(k % nst));
  };

  float yacc[8][NH][4];
  auto zero_acc = [&]() {
#pragma unroll
    for (int mt = 0; mt < 8; ++mt)
#pragma unroll
      for (int nh = 0; nh < NH; ++nh)
#pragma unroll
        for (int e = 0; e < 4; ++e) yacc[mt][nh][e] = 0.f;
  };
  // every warp parks its accumulator tile [heads][128] for the fixed-order sum over the warps
  auto park_acc = [&]() {
    float* mine = red + (size_t)warp * (NH * 8 * D);
#pragma unroll
    for (int nh = 0; nh < NH; ++nh)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        float* yp = mine + (nh * 8 + 2 * t4 + e) * D;
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
          yp[mt * 16 + gid] = yacc[mt][nh][e];
          yp[mt * 16 + gid + 8] = yacc[mt][nh][2 + e];
        }
      }
  };

  long long kbase = 0;                              // ring ordinal of the current pair's first tile
  for (int bh = bh_first; bh < BH; bh += bh_step, kbase += per_bh) {
    const int b = bh / a.H_kv, h = bh - b * a.H_kv;
    // ------------------------------------------------------------------ text tiles
    if (t1 > t0) {
      // A fragments of the logit product: rows = the heads of the group (gid, gid + 8), k = the 128 channels
      uint32_t qa[8][4];
      {
        const __nv_bfloat16* q0 = a.q + ((size_t)b * a.H_kv * G + (size_t)h * G) * D;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const int k0 = ks * 16 + 2 * t4;
          qa[ks][0] = gid < G ? *reinterpret_cast<const uint32_t*>(q0 + (size_t)gid * D + k0) : 0u;
          qa[ks][1] = gid + 8 < G ? *reinterpret_cast<const uint32_t*>(q0 + (size_t)(gid + 8) * D + k0) : 0u;
          qa[ks][2] = gid < G ? *reinterpret_cast<const uint32_t*>(q0 + (size_t)gid * D + k0 + 8) : 0u;
          qa[ks][3] = gid + 8 < G ? *reinterpret_cast<const uint32_t*>(q0 + (size_t)(gid + 8) * D + k0 + 8) : 0u;
        }
      }
      zero_acc();
      float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};   // heads gid and gid + 8
      long long k = kbase;
      k += ((grp - (int)(k % NGRP)) + NGRP) % NGRP;
      for (; k < kbase + (t1 - t0); k += NGRP) {
        const int tile = t0 + (int)(k - kbase);
        wait_full(k);
        const uint32_t kt_u = sm_u + (uint32_t)(k % nst) * a.o_stage_bytes, vt_u = kt_u + 2 * SO_HALF;
        const int t_first = tile * SP_OUT_ROWS + rg * 16;
        if (t_first < a.T) {
          const uint32_t rowB = (uint32_t)((rg * 16 + lrowB) * 128);
          // logits [16 heads][16 text rows] = q K_txt^T, two accumulation chains per 8-row group
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
            for (int ks = 0; ks < 8; ++ks) {
              uint32_t bk[4];
              ldsm_x4(bk, kt_u + (ks >> 2) * SO_HALF + rowB + (uint32_t)(((((ks & 3) * 2 + lmid)) ^ l7) << 4));
              mma_bf16_16816(c2[ks & 1][0], qa[ks], bk[0], bk[1]);
              mma_bf16_16816(c2[ks & 1][1], qa[ks], bk[2], bk[3]);
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
            scl[hr] = fast_exp2(m_run[hr] - m_new);                // 0 on the first group
            m_run[hr] = m_new;
            float ps = 0.f;
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
              for (int x = 0; x < 2; ++x) {
                const float p = fast_exp2(cc[nt][2 * hr + x] - m_new);
                cc[nt][2 * hr + x] = p;
                ps += p;
              }
            l_run[hr] = l_run[hr] * scl[hr] + ps;
          }
          // the accumulator's columns are heads: fetch their factors from the lanes that own those heads as rows
#pragma unroll
          for (int nh = 0; nh < NH; ++nh) {
            const float c0s = __shfl_sync(0xffffffffu, scl[nh], (2 * t4) * 4);
            const float c1s = __shfl_sync(0xffffffffu, scl[nh], (2 * t4 + 1) * 4);
            if (c0s != 1.f || c1s != 1.f) {
#pragma unroll
              for (int mt = 0; mt < 8; ++mt) {
                yacc[mt][nh][0] *= c0s; yacc[mt][nh][1] *= c1s;
                yacc[mt][nh][2] *= c0s; yacc[mt][nh][3] *= c1s;
              }
            }
          }
          // y^T[128][heads] += V_txt^T[128][16 rows] P^T[16 rows][heads]
          uint32_t pb[2][2];
          pb[0][0] = pack2_bf16(cc[0][0], cc[0][1]); pb[0][1] = pack2_bf16(cc[1][0], cc[1][1]);
          pb[1][0] = pack2_bf16(cc[0][2], cc[0][3]); pb[1][1] = pack2_bf16(cc[1][2], cc[1][3]);
#pragma unroll
          for (int mt = 0; mt < 8; ++mt) {
            uint32_t av[4];
            ldsm_x4_t(av, vt_u + (mt >> 2) * SO_HALF + rowB + (uint32_t)(((((mt & 3) * 2 + lmid)) ^ l7) << 4));
#pragma unroll
            for (int nh = 0; nh < NH; ++nh) mma_bf16_16816(yacc[mt][nh], av, pb[nh][0], pb[nh][1]);
          }
        }
        release(k);
      }
      // the per-warp online-softmax states meet at one maximum per head; the sum over the warps goes to tbuf
      if (t4 == 0) { tmax[warp * 16 + gid] = m_run[0]; tmax[warp * 16 + gid + 8] = m_run[1]; }
      named_barrier_sync(1, SO_CONS);
      {
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
          if (t4 == 0) tsum[warp * 16 + head] = l;
          if (warp == 0 && t4 == 0) txm[head] = M;
        }
#pragma unroll
        for (int nh = 0; nh < NH; ++nh) {
          const float c0s = __shfl_sync(0xffffffffu, scl[nh], (2 * t4) * 4);
          const float c1s = __shfl_sync(0xffffffffu, scl[nh], (2 * t4 + 1) * 4);
#pragma unroll
          for (int mt = 0; mt < 8; ++mt) {
            yacc[mt][nh][0] *= c0s; yacc[mt][nh][1] *= c1s;
            yacc[mt][nh][2] *= c0s; yacc[mt][nh][3] *= c1s;
          }
        }
      }
      park_acc();
      named_barrier_sync(1, SO_CONS);
      for (int idx = tid; idx < G * D; idx += SO_CONS) {
        const float* rp = red + idx;
        float y = 0.f;
#pragma unroll
        for (int w = 0; w < SO_WARPS; ++w) y += rp[(size_t)w * (NH * 8 * D)];
        tbuf[idx] = y;
      }
      if (tid < 16) {
        float l = 0.f;
#pragma unroll
        for (int w = 0; w < SO_WARPS; ++w) l += tsum[w * 16 + tid];
        txl[tid] = l;
      }
    } else if (tid < 16) {
      txm[tid] = -INFINITY;
      txl[tid] = 0.f;
    }

    // ------------------------------------------------------------------ value tiles
    if (!waited) { grid_dep_wait(); waited = true; }  // row statistics and partial weights of the expansion kernel
    // row statistics of every (block, range, head) of the pair -> maximum per head, factor per entry, mass per head
    const int ne = R * NS;
    for (int idx = tid; idx < ne * 16; idx += SO_CONS) {
      const int e = idx >> 4, g = idx & 15, rr = e / NS, s = e - rr * NS;
      float2 v = make_float2(-INFINITY, 0.f);
      if (g < G) v = __ldcg(&a.stat[((size_t)h * NS + s) * a.rows_h + (size_t)(b * R + rr) * G + g]);
      fac[idx] = v;
    }
    named_barrier_sync(1, SO_CONS);                   // also: tbuf, txm, txl are in place; red is free again
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
      // the first CTA of the pair carries the whole probability mass of the vision positions (and with it the mu term)
      if (lane == 0) { hmax[g] = g < G ? mx : -INFINITY; hsum[g] = (g < G && part == 0) ? l : 0.f; }
    }
    named_barrier_sync(1, SO_CONS);
    zero_acc();
    {
      const long long kv = kbase + (t1 - t0);
      long long k = kv;
      k += ((grp - (int)(k % NGRP)) + NGRP) % NGRP;
      for (; k < kv + (v1 - v0); k += NGRP) {
        const int rem = v0 + (int)(k - kv);
        const int r = rem / vt, jt = rem - r * vt;
        wait_full(k);
        const uint32_t v_u = sm_u + (uint32_t)(k % nst) * a.o_stage_bytes;
        const unsigned char* wp = sm + (size_t)(k % nst) * a.o_stage_bytes + 2 * SO_HALF;      // [NS][G][64] bf16
        const float2* fr = fac + (size_t)r * NS * 16;
        if (jt * SP_OUT_ROWS + rg * 16 < a.m) {
          // B fragments: the weights of heads gid (+8) for rows 2 t4, 2 t4 + 1 (+8) of this row group, ranges joined
          uint32_t bw[NH][2];
#pragma unroll
          for (int nh = 0; nh < NH; ++nh) {
            const int g = gid + 8 * nh;
            float w0 = 0.f, w1 = 0.f, w2 = 0.f, w3 = 0.f;
            if (g < G) {
              const unsigned char* row = wp + (size_t)g * 128 + (rg * 16 + 2 * t4) * 2;
              for (int s = 0; s < NS; ++s) {
                const float f = fr[s * 16 + g].x;
                const uint32_t lo = *reinterpret_cast<const uint32_t*>(row), hi = *reinterpret_cast<const uint32_t*>(row + 16);
                row += (size_t)G * 128;
                w0 = fmaf(f, __uint_as_float(lo << 16), w0); w1 = fmaf(f, __uint_as_float(lo & 0xffff0000u), w1);
                w2 = fmaf(f, __uint_as_float(hi << 16), w2); w3 = fmaf(f, __uint_as_float(hi & 0xffff0000u), w3);
              }
            }
            bw[nh][0] = pack2_bf16(w0, w1);
            bw[nh][1] = pack2_bf16(w2, w3);
          }
          const uint32_t rowB = (uint32_t)((rg * 16 + lrowB) * 128);
#pragma unroll
          for (int mt = 0; mt < 8; ++mt) {
            uint32_t av[4];
            ldsm_x4_t(av, v_u + (mt >> 2) * SO_HALF + rowB + (uint32_t)(((((mt & 3) * 2 + lmid)) ^ l7) << 4));
#pragma unroll
            for (int nh = 0; nh < NH; ++nh) mma_bf16_16816(yacc[mt][nh], av, bw[nh][0], bw[nh][1]);
          }
        }
        release(k);
      }
    }

    // ------------------------------------------------------------------ the two parts meet; output or partial + merge
    park_acc();
    named_barrier_sync(1, SO_CONS);
    const size_t pbase = ((size_t)bh * cpb + part) * G;
    for (int idx = tid; idx < G * D; idx += SO_CONS) {
      const int g = idx >> 7, col = idx & (D - 1);
      const float* rp = red + idx;
      float yv = 0.f;
#pragma unroll
      for (int w = 0; w < SO_WARPS; ++w) yv += rp[(size_t)w * (NH * 8 * D)];
      yv = fmaf(hsum[g], __bfloat162float(a.mu[h * D + col]), yv);
      const float mv = hmax[g], mt_ = txm[g], M = fmaxf(mv, mt_);
      const float fv = fast_exp2(mv - M), ft = mt_ == -INFINITY ? 0.f : fast_exp2(mt_ - M);
      const float y = fmaf(fv, yv, ft * tbuf[idx]);
      if (cpb == 1) {
        const float l = fmaf(fv, hsum[g], ft * txl[g]);
        a.out[((size_t)b * a.H_kv * G + (size_t)h * G + g) * D + col] = __float2bfloat16_rn(y / l);
      } else {
        a.py[(pbase + g) * D + col] = y;
      }
    }
    if (cpb > 1) {
      if (tid < G) {
        const float mv = hmax[tid], mt_ = txm[tid], M = fmaxf(mv, mt_);
        const float fv = fast_exp2(mv - M), ft = mt_ == -INFINITY ? 0.f : fast_exp2(mt_ - M);
        a.pml[pbase + tid] = make_float2(M, fmaf(fv, hsum[tid], ft * txl[tid]));
      }
      named_barrier_sync(1, SO_CONS);
      if (tid == 0) {
        __threadfence();                  // the partial of every thread (ordered before by the barrier) before the arrival
        s_last = atomicAdd(&a.cnt[bh], 1) + 1 == cpb ? 1 : 0;
        __threadfence();                  // the arrival before the reads of the other CTAs' partials
      }
      named_barrier_sync(1, SO_CONS);
      if (s_last) {
        const size_t p0 = (size_t)bh * cpb * G;
        // (max, sum) of every partial into shared memory, then one weight 2^(max_p - max) / sum per (partial, head)
        for (int idx = tid; idx < cpb * 16; idx += SO_CONS) {
          const int p = idx >> 4, g = idx & 15;
          const float2 ml = g < G ? __ldcg(&a.pml[p0 + (size_t)p * G + g]) : make_float2(-INFINITY, 0.f);
          mlm[idx] = ml.x;
          mlm[cpb * 16 + idx] = ml.y;
        }
        named_barrier_sync(1, SO_CONS);
        if (tid < 16) {
          float M = -INFINITY, den = 0.f;
          for (int p = 0; p < cpb; ++p) M = fmaxf(M, mlm[p * 16 + tid]);
          for (int p = 0; p < cpb; ++p) den = fmaf(fast_exp2(mlm[p * 16 + tid] - M), mlm[cpb * 16 + p * 16 + tid], den);
          const float inv = 1.f / den;
          for (int p = 0; p < cpb; ++p) mlm[p * 16 + tid] = fast_exp2(mlm[p * 16 + tid] - M) * inv;
        }
        named_barrier_sync(1, SO_CONS);
        for (int idx = tid; idx < G * (D / 4); idx += SO_CONS) {
          const int g = idx >> 5, col = (idx & 31) * 4;
          float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
          auto acc4 = [&](const float4& y, float w) {
            num.x = fmaf(w, y.x, num.x); num.y = fmaf(w, y.y, num.y); num.z = fmaf(w, y.z, num.z); num.w = fmaf(w, y.w, num.w);
          };
          const float* src = a.py + (p0 + g) * D + col;
          int p = 0;
          for (; p + 8 <= cpb; p += 8) {
            float4 y[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) y[x] = __ldcg(reinterpret_cast<const float4*>(src + (size_t)(p + x) * G * D));
#pragma unroll
            for (int x = 0; x < 8; ++x) acc4(y[x], mlm[(p + x) * 16 + g]);
          }
          for (; p + 2 <= cpb; p += 2) {
            float4 y[2];
#pragma unroll
            for (int x = 0; x < 2; ++x) y[x] = __ldcg(reinterpret_cast<const float4*>(src + (size_t)(p + x) * G * D));
#pragma unroll
            for (int x = 0; x < 2; ++x) acc4(y[x], mlm[(p + x) * 16 + g]);
          }
          for (; p < cpb; ++p) acc4(__ldcg(reinterpret_cast<const float4*>(src + (size_t)p * G * D)), mlm[p * 16 + g]);
          uint2 o;
          o.x = pack2_bf16(num.x, num.y); o.y = pack2_bf16(num.z, num.w);
          *reinterpret_cast<uint2*>(a.out + ((size_t)b * a.H_kv * G + (size_t)h * G + g) * D + col) = o;
        }
      }
    }
    named_barrier_sync(1, SO_CONS);                   // red, tbuf and the statistics are free for the next pair
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
