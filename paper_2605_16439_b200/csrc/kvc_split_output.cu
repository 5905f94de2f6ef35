// Split path, last kernel: Alg. 1 step 4 and the normalisation,
//   y = sum_r W_r V_tilde_r + (sum P) mu  (+ the text kernel's P_txt V_txt),   out = y / (sum of all exponentials),
// as one streaming pass over V_tilde, bound by HBM bandwidth.
//
// Work items are tiles of 64 rows of a block of V_tilde.  A pair's tiles go to `cpb` CTAs (as many as the SMs allow, the
// same number for every pair), each taking an equal share; with more pairs than SMs a CTA takes whole pairs one after
// the other.  A producer thread keeps a ring of TMA-filled stages full: 64 rows of V_tilde and the matching 64 columns of
// the partial weights of the block's G heads for every range of the n axis.  The consumer warps form groups of four; tile
// k of the CTA's list goes to group k mod NGRP and each warp of the group takes 16 of its rows over the whole head
// dimension; the product is mma.sync m16n8k16 with the value rows transposed (head dimension as M, heads as N):
//   W[g][j] = sum_s 2^(max_s - max) Wp_s[g][j]  (the ranges joined while the B fragment is built),  y^T += V_tilde^T W^T;
//   the probability mass of the vision positions and the mu term come from the range sums.
// Every CTA leaves one partial (max, sum, y) per head; the last CTA of the pair to arrive merges the pair's partials and
// those the text CTAs of the expansion kernel left by log-sum-exp and writes `out`.
#include "kvc_split.cuh"

namespace kvc {

constexpr uint32_t SO_HALF = SP_OUT_ROWS * 128;       // 64 rows x 64 channels

// NH = 8-head tiles of the group (1: G <= 8, 2: G <= 16); NGRP = warp groups of four (a tile is a chain of dependent
// steps per warp, so more groups, each on its own tile, keep more tiles in work)
template <int NH, int NGRP>
__global__ void __launch_bounds__(NGRP * SP_GROUP * 32 + 32, 1)
split_output_kernel(const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmW, const SplitArgs a) {
  constexpr int SO_WARPS = NGRP * SP_GROUP;
  constexpr int SO_CONS = SO_WARPS * 32;
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
  const int v0 = (int)((long long)part * vb / cpb), v1 = (int)((long long)(part + 1) * vb / cpb);
  const int per_bh = v1 - v0;                                     // ring ordinals per pair
  const int nct = (tt + SP_TEXT_CHUNK - 1) / SP_TEXT_CHUNK;       // partials the text kernel left per pair
  const uint32_t w_bytes = (uint32_t)(NS * G) * 128u;

  if (warp == SO_WARPS) {
    // ================= producer =================
    if (lane != 0) return;
    tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmW);
    uint32_t slot = 0, phase = 1;
    bool waited = false;
    for (int bh = bh_first; bh < BH; bh += bh_step) {
      const int b = bh / a.H_kv, h = bh - b * a.H_kv;
      if (!waited) { grid_dep_wait(); waited = true; }     // the partial weights come from the expansion kernel
      int r = v0 / vt, jt = v0 - r * vt;
      for (int rem = v0; rem < v1; ++rem) {
        if (!mbar_wait_bounded(&empty_bar[slot], phase)) { atomicExch(a.status, (int)KVC_ERR_TIMEOUT); return; }
        unsigned char* dst = sm + slot * a.o_stage_bytes;
        mbar_expect_tx(&full_bar[slot], 2 * SO_HALF + w_bytes);
        tma_load_4d(dst, &tmV, 0, jt * SP_OUT_ROWS, 0, bh * R + r, &full_bar[slot]);      // both 64-channel halves in one copy
        tma_load_4d(dst + 2 * SO_HALF, &tmW, jt * SP_OUT_ROWS, (b * R + r) * G, 0, h, &full_bar[slot]);
        if (++slot == (uint32_t)nst) { slot = 0; phase ^= 1u; }
        if (++jt == vt) { jt = 0; ++r; }
      }
    }
    return;
  }

  // ================= consumers: tile k of the CTA's list goes to warp group k mod 2, 16 rows to each of its warps =================
  grid_dep_launch();
  const int grp = warp / SP_GROUP, rg = warp % SP_GROUP;      // warp group; the 16-row group of a tile this warp takes
  const int gid = lane >> 2, t4 = lane & 3;
  const int l7 = lane & 7, lhi = lane >> 4, lmid = (lane >> 3) & 1;
  const int lrowB = l7 + lhi * 8;                   // ldmatrix address pattern: rows 0-7 | 0-7 | 8-15 | 8-15
  const uint32_t sm_u = smem_addr(sm);
  float2* fac = reinterpret_cast<float2*>(sm + a.o_off_fac);                     // [R*NS][17]: (factor, scaled row sum) per head; the odd pitch spreads a head's entries over the banks
  float* red = reinterpret_cast<float*>(sm + a.o_off_red);                       // [8 warps][NH*8][128]
  float* vbuf = reinterpret_cast<float*>(sm + a.o_off_q);                        // [16][128] value part of the pair
  float* hmax = reinterpret_cast<float*>(sm + a.o_off_stat);                     // [16] maximum over the vision logits
  float* hsum = hmax + 16;                                                       // [16] probability mass carried by this CTA
  float* mlm = hsum + 16;                                                        // merge: [partials][16] maxima, sums -> weights

  bool dead = false, waited = false;
  // ring position of this warp group's next tile: ordinal ko, slot = ko mod stages, round = ko div stages
  int ko = 0;
  uint32_t slot = 0, round = 0;
  auto seek = [&](int k) {                          // forward to ordinal k >= ko
    int d = k - ko;
    ko = k;
    while (d > 0) {
      const int step = d < nst - (int)slot ? d : nst - (int)slot;
      slot += (uint32_t)step;
      d -= step;
      if (slot == (uint32_t)nst) { slot = 0; ++round; }
    }
  };
  auto wait_full = [&]() {
    if (!dead && !(wait_round(released, slot, round) && mbar_wait_bounded(&full_bar[slot], round & 1u))) dead = true;
    __syncwarp();
  };
  auto release = [&]() {
    __syncwarp();
    if (lane == 0) release_slot(released, empty_bar, slot);
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
  // Fixed-order sum of the warps' accumulator tiles [heads][128] into dst: eight warps at a time park theirs in shared
  // memory and every thread adds up its elements.
  auto reduce_acc = [&](float* dst) {
#pragma unroll 1
    for (int round = 0; round < SO_WARPS / 8; ++round) {
      if ((warp >> 3) == round) {
        float* mine = red + (size_t)(warp & 7) * (NH * 8 * D);
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
      }
      named_barrier_sync(1, SO_CONS);
      for (int idx = tid; idx < G * D; idx += SO_CONS) {
        const float* rp = red + idx;
        float y = round ? dst[idx] : 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) y += rp[(size_t)w * (NH * 8 * D)];
        dst[idx] = y;
      }
      named_barrier_sync(1, SO_CONS);
    }
  };

  int kbase = 0;                                    // ring ordinal of the current pair's first tile
  for (int bh = bh_first; bh < BH; bh += bh_step, kbase += per_bh) {
    const int b = bh / a.H_kv, h = bh - b * a.H_kv;
    // ------------------------------------------------------------------ value tiles
    if (!waited) { grid_dep_wait(); waited = true; }  // row statistics and partial weights of the expansion kernel
    // row statistics of every (block, range, head) of the pair -> maximum per head, factor per entry, mass per head
    const int ne = R * NS;
    for (int idx = tid; idx < ne * 16; idx += SO_CONS) {
      const int e = idx >> 4, g = idx & 15, rr = e / NS, s = e - rr * NS;
      float2 v = make_float2(-INFINITY, 0.f);
      if (g < G) v = __ldcg(&a.stat[((size_t)h * NS + s) * a.rows_h + (size_t)(b * R + rr) * G + g]);
      fac[e * SO_FAC_PITCH + g] = v;
    }
    named_barrier_sync(1, SO_CONS);
    for (int g = warp; g < 16; g += SO_WARPS) {
      float mx = -INFINITY;
      for (int e = lane; e < ne; e += 32) mx = fmaxf(mx, fac[e * SO_FAC_PITCH + g].x);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      float l = 0.f;
      for (int e = lane; e < ne; e += 32) {
        const float2 v = fac[e * SO_FAC_PITCH + g];
        const float f = g < G ? fast_exp2(v.x - mx) : 0.f;
        fac[e * SO_FAC_PITCH + g] = make_float2(f, f * v.y);
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
      const int kv = kbase;
      int k = kv;
      k += ((grp - (k % NGRP)) + NGRP) % NGRP;
      for (; k < kv + (v1 - v0); k += NGRP) {
        const int rem = v0 + (k - kv);
        const int r = rem / vt, jt = rem - r * vt;
        seek(k);
        wait_full();
        const uint32_t v_u = sm_u + slot * a.o_stage_bytes;
        const unsigned char* wp = sm + (size_t)slot * a.o_stage_bytes + 2 * SO_HALF;      // [NS][G][64] bf16
        const float2* fr = fac + (size_t)r * NS * SO_FAC_PITCH;
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
                const float f = fr[s * SO_FAC_PITCH + g].x;
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
        release();
      }
    }

    // ------------------------------------------------------------------ partial of this CTA; the last CTA of the pair merges
    // the pair's value partials and the text kernel's partials by log-sum-exp
    reduce_acc(vbuf);
    const size_t pbase = ((size_t)bh * cpb + part) * G;
    for (int idx = tid; idx < G * D; idx += SO_CONS) {
      const int g = idx >> 7, col = idx & (D - 1);
      a.py[(pbase + g) * D + col] = fmaf(hsum[g], __bfloat162float(a.mu[h * D + col]), vbuf[idx]);
    }
    if (tid < G) a.pml[pbase + tid] = make_float2(hmax[tid], hsum[tid]);
    named_barrier_sync(1, SO_CONS);
    if (tid == 0) {
      s_last = 1;
      if (cpb > 1) {
        __threadfence();                // the partial of every thread (ordered before by the barrier) before the arrival
        s_last = atomicAdd(&a.cnt[bh], 1) + 1 == cpb ? 1 : 0;
        __threadfence();                // the arrival before the reads of the other CTAs' partials
      }
    }
    named_barrier_sync(1, SO_CONS);
    if (s_last) {
      const int np = cpb + nct;                       // partials of the pair: value CTAs, then text chunks
      const size_t p0 = (size_t)bh * cpb * G, q0 = (size_t)bh * nct * G;
      // (max, sum) of every partial into shared memory, then one weight 2^(max_p - max) / sum per (partial, head)
      for (int idx = tid; idx < np * 16; idx += SO_CONS) {
        const int p = idx >> 4, g = idx & 15;
        float2 ml = make_float2(-INFINITY, 0.f);
        if (g < G) ml = p < cpb ? __ldcg(&a.pml[p0 + (size_t)p * G + g]) : __ldcg(&a.tpml[q0 + (size_t)(p - cpb) * G + g]);
        mlm[idx] = ml.x;
        mlm[np * 16 + idx] = ml.y;
      }
      named_barrier_sync(1, SO_CONS);
      if (tid < 16) {
        float M = -INFINITY, den = 0.f;
        for (int p = 0; p < np; ++p) M = fmaxf(M, mlm[p * 16 + tid]);
        for (int p = 0; p < np; ++p) {
          const float x = mlm[p * 16 + tid];
          den = fmaf(x == -INFINITY ? 0.f : fast_exp2(x - M), mlm[np * 16 + p * 16 + tid], den);
        }
        const float inv = 1.f / den;
        for (int p = 0; p < np; ++p) {
          const float x = mlm[p * 16 + tid];
          mlm[p * 16 + tid] = x == -INFINITY ? 0.f : fast_exp2(x - M) * inv;
        }
      }
      named_barrier_sync(1, SO_CONS);
      for (int idx = tid; idx < G * (D / 4); idx += SO_CONS) {
        const int g = idx >> 5, col = (idx & 31) * 4;
        float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
        auto acc4 = [&](const float4& y, float w) {
          num.x = fmaf(w, y.x, num.x); num.y = fmaf(w, y.y, num.y); num.z = fmaf(w, y.z, num.z); num.w = fmaf(w, y.w, num.w);
        };
        auto src = [&](int p) {
          return reinterpret_cast<const float4*>(p < cpb ? a.py + (p0 + (size_t)p * G + g) * D + col
                                                         : a.tpy + (q0 + (size_t)(p - cpb) * G + g) * D + col);
        };
        // eight partials' loads in flight at a time, the last group predicated (a pair has 2 + 3 partials at config 2: one
        // round trip instead of three)
        for (int p = 0; p < np; p += 8) {
          float4 y[8];
#pragma unroll
          for (int x = 0; x < 8; ++x)
            if (p + x < np) y[x] = __ldcg(src(p + x));
#pragma unroll
          for (int x = 0; x < 8; ++x)
            if (p + x < np) acc4(y[x], mlm[(p + x) * 16 + g]);
        }
        uint2 o;
        o.x = pack2_bf16(num.x, num.y); o.y = pack2_bf16(num.z, num.w);
        *reinterpret_cast<uint2*>(a.out + ((size_t)b * a.H_kv * G + (size_t)h * G + g) * D + col) = o;
      }
    }
    named_barrier_sync(1, SO_CONS);                   // red and the statistics are free for the next pair
  }
  if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
}

template <int NH, int NGRP>
static cudaError_t launch_output_inst(const CUtensorMap* tm, const SplitArgs& a, const SplitPlan& p, cudaStream_t st) {
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(split_output_kernel<NH, NGRP>), p.o_smem);
  if (e != cudaSuccess) return e;
  return launch_dependent(split_output_kernel<NH, NGRP>, dim3(p.o_grid), dim3(NGRP * SP_GROUP * 32 + 32), p.o_smem, st, tm[0], tm[3], a);
}

cudaError_t launch_split_output(const CUtensorMap* tm, const SplitArgs& a, const SplitPlan& p, cudaStream_t st) {
  ProfScope prof(KVC_KERNEL_SPLIT_OUTPUT, st);
  // up to 8 heads per KV head: 16 consumer warps; more: the accumulators of two head tiles leave registers for 8
  return a.G > 8 ? launch_output_inst<2, 2>(tm, a, p, st) : launch_output_inst<1, 4>(tm, a, p, st);
}

}  // namespace kvc
