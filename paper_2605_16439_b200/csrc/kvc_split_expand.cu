// Split path, second kernel: Alg. 1 steps 2 and 3 for 128 expansion rows of a KV head and one range [n0, n0 + NW) of
// the n positions of a block, as two dense products on tcgen05 with the accumulators in tensor memory:
//   L[128 x NW]  = S[128 x m] theta[h][m x range]            A = S tile (K-major), B = theta rows (MN-major)
//   P = 2^(L - rowmax) (bf16, in shared memory as the next A operand), rowsum
//   Wp[128 x m]  = P[128 x NW] U[h][m x range]^T              A = P (K-major), B = rows of U (K-major), in passes of
//                                                             at most 512 columns; the logits' columns are reused
// Every operand tile is read as the TMA engine lays it down (128-byte swizzle).  The partial weights of the range, still
// relative to the range's own row maximum, go to the workspace as bf16 with (rowmax, rowsum); the output kernel joins the
// ranges of a row.  One CTA per (KV head, row tile, range); warps 0-7 = one lane per expansion row and half of the columns
// (softmax, epilogue), warp 8 = MMA issue, warp 9 = TMA producer.
#include "kvc_split.cuh"
#include "kvc_tcgen05.cuh"

namespace kvc {

constexpr int SE_THREADS = 10 * 32;      // warps 0-7: softmax and epilogue, warp 8: MMA issue, warp 9: TMA producer

struct ExpandBars {
  uint64_t full[SP_MAX_STAGES], empty[SP_MAX_STAGES];
  uint64_t l_done;      // the logits are complete in tensor memory
  uint64_t p_ready;     // the probabilities are in shared memory and the logits have been read (4 warps)
  uint64_t w_done;      // a pass of the weights is complete
  uint64_t w_free;      // a pass of the weights has been read back (4 warps)
};

// ---- the text rows, on the SMs the expansion leaves idle ----
// Plain attention of the decode query over K_txt / V_txt (Sec. 3.2: the text K/V stay uncompressed and join the softmax
// of the reconstructed vision positions), flash-style, as partials: the CTAs behind the expansion CTAs of the grid each
// take a run of (sequence, KV head, chunk of up to 192 text rows) items and leave (max, sum, y) per head and item in
// the workspace; the output kernel merges them with the vision part.  An item is a chain of round trips (queries, three
// tiles, the warps' states meeting in shared memory, the partial's store), so a CTA runs NG of them side by side: group g =
// warps 4g..4g+3 (16 rows of every 64-row tile each) with its own stages, barriers and producer thread (lane 0 of warp
// 9 - g; one stage per tile of a chunk, refilled for the next chunk as soon as its tile has been read), taking every NG-th
// item of the CTA's run.
constexpr uint32_t ST_HALF = SP_OUT_ROWS * 128;       // 64 rows x 64 channels
constexpr uint32_t ST_STAGE = 4 * ST_HALF;            // K and V rows of a tile
constexpr int ST_WARPS = 4;
constexpr int ST_CONS = ST_WARPS * 32;

constexpr uint32_t SP_SMEM_LIMIT_EXPAND = 232448;      // shared memory of a CTA, static part included
constexpr int ST_STAT = 2 * ST_WARPS * 16 + 16;       // floats of a group's statistics: maxima [4][16], sums [4][16], maximum [16]
// a group's shared memory: its stages and the four warps' parked accumulators [G heads][128]; two groups fit up to G = 7
__host__ __device__ constexpr uint32_t st_group_bytes(int G) { return ((uint32_t)SP_TEXT_CHUNK * ST_STAGE + (uint32_t)ST_WARPS * G * D * 4 + 1023u) & ~1023u; }
__host__ __device__ constexpr int st_groups(int G) { return 2u * st_group_bytes(G) + 1024u + 4096u <= SP_SMEM_LIMIT_EXPAND ? 2 : 1; }

template <int NH>
__device__ __forceinline__ void text_role(const CUtensorMap& tmKt, const CUtensorMap& tmVt, const SplitArgs& a, unsigned char* sm_cta,
                                          ExpandBars& bars, float* stat_cta /*[NG][ST_STAT]*/) {
  const int NG = st_groups(a.G);
  const int tid_cta = threadIdx.x, warp_cta = tid_cta >> 5, lane = tid_cta & 31;
  const int G = a.G;
  const int tt = (a.T + SP_OUT_ROWS - 1) / SP_OUT_ROWS;
  const int nct = (tt + SP_TEXT_CHUNK - 1) / SP_TEXT_CHUNK;
  const long long items = (long long)a.B * a.H_kv * nct;
  const int j = (int)blockIdx.x - a.e_grid;
  const int i0 = (int)(items * j / a.tx_grid), i1 = (int)(items * (j + 1) / a.tx_grid);
  if (tid_cta == 0) {
    for (int s = 0; s < NG * SP_TEXT_CHUNK; ++s) { mbar_init(&bars.full[s], 1); mbar_init(&bars.empty[s], ST_WARPS); }
    fence_mbar_init();
  }
  __syncthreads();
  grid_dep_launch();
  // group of this warp: consumers 4g..4g+3, producer 9 - g
  const int grp = warp_cta >= 10 - NG ? 9 - warp_cta : warp_cta / ST_WARPS;
  if (grp >= NG) return;
  unsigned char* sm = sm_cta + (size_t)grp * st_group_bytes(a.G);
  uint64_t* full = bars.full + grp * SP_TEXT_CHUNK;
  uint64_t* empty = bars.empty + grp * SP_TEXT_CHUNK;
  float* tmax = stat_cta + grp * ST_STAT, *tsum = tmax + ST_WARPS * 16, *txm = tsum + ST_WARPS * 16;
  if (warp_cta >= 10 - NG) {
    if (lane == 0) {
      tma_prefetch_desc(&tmKt); tma_prefetch_desc(&tmVt);
      uint32_t phase = 1;
      for (int it = i0 + grp; it < i1; it += NG, phase ^= 1u) {
        const int bh = it / nct, ci = it - bh * nct;
        const int b = bh / a.H_kv, h = bh - b * a.H_kv;
        const int t0 = ci * SP_TEXT_CHUNK, t1 = min(tt, t0 + SP_TEXT_CHUNK);
        for (int tile = t0; tile < t1; ++tile) {
          const int s = tile - t0;
          if (!mbar_wait_bounded(&empty[s], phase)) { atomicExch(a.status, (int)KVC_ERR_TIMEOUT); return; }
          unsigned char* dst = sm + (uint32_t)s * ST_STAGE;
          mbar_expect_tx(&full[s], ST_STAGE);
          const int y = tile * SP_OUT_ROWS;
          tma_load_5d(dst, &tmKt, 0, y, 0, h, b, &full[s]);                    // both 64-channel halves per copy
          tma_load_5d(dst + 2 * ST_HALF, &tmVt, 0, y, 0, h, b, &full[s]);
        }
        // a stage the chunk does not use still turns its barriers once, so that every stage is in the same round
        for (int s = t1 - t0; s < SP_TEXT_CHUNK; ++s) {
          if (!mbar_wait_bounded(&empty[s], phase)) { atomicExch(a.status, (int)KVC_ERR_TIMEOUT); return; }
          mbar_expect_tx(&full[s], 0);
        }
      }
    }
    return;
  }
  const int warp = warp_cta - grp * ST_WARPS, tid = tid_cta - grp * ST_CONS;     // within the group
  const int rg = warp;                              // the 16-row group of a tile this warp takes
  const int gid = lane >> 2, t4 = lane & 3;
  const int l7 = lane & 7, lhi = lane >> 4, lmid = (lane >> 3) & 1;
  const int lrowB = l7 + lhi * 8;                   // ldmatrix address pattern: rows 0-7 | 0-7 | 8-15 | 8-15
  const uint32_t sm_u = smem_addr(sm);
  float* red = reinterpret_cast<float*>(sm + SP_TEXT_CHUNK * ST_STAGE);          // [4 warps][G][128]
  bool dead = false;
  uint32_t phase = 0;
  for (int it = i0 + grp; it < i1; it += NG, phase ^= 1u) {
    const int bh = it / nct, ci = it - bh * nct;
    const int b = bh / a.H_kv, h = bh - b * a.H_kv;
    const int t0 = ci * SP_TEXT_CHUNK, t1 = min(tt, t0 + SP_TEXT_CHUNK);
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
    float yacc[8][NH][4];
#pragma unroll
    for (int mt = 0; mt < 8; ++mt)
#pragma unroll
      for (int nh = 0; nh < NH; ++nh)
#pragma unroll
        for (int e = 0; e < 4; ++e) yacc[mt][nh][e] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};   // heads gid and gid + 8
    for (int s = 0; s < SP_TEXT_CHUNK; ++s) {
      const int tile = t0 + s;
      if (!dead && !mbar_wait_bounded(&full[s], phase)) dead = true;
      __syncwarp();
      if (tile < t1) {
        const uint32_t kt_u = sm_u + (uint32_t)s * ST_STAGE, vt_u = kt_u + 2 * ST_HALF;
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
                ldsm_x4(bk, kt_u + (ks >> 2) * ST_HALF + rowB + (uint32_t)(((((ks & 3) * 2 + lmid)) ^ l7) << 4));
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
              ldsm_x4_t(av, vt_u + (mt >> 2) * ST_HALF + rowB + (uint32_t)(((((mt & 3) * 2 + lmid)) ^ l7) << 4));
  #pragma unroll
              for (int nh = 0; nh < NH; ++nh) mma_bf16_16816(yacc[mt][nh], av, pb[nh][0], pb[nh][1]);
            }
          }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);
    }
    // the per-warp online-softmax states meet at one maximum per head
    if (t4 == 0) { tmax[warp * 16 + gid] = m_run[0]; tmax[warp * 16 + gid + 8] = m_run[1]; }
    named_barrier_sync(1 + grp, ST_CONS);
    {
      float scl[2];
#pragma unroll
      for (int hr = 0; hr < 2; ++hr) {
        const int head = gid + 8 * hr;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < ST_WARPS; ++w) M = fmaxf(M, tmax[w * 16 + head]);
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
    {
      float* mine = red + (size_t)warp * (G * D);
#pragma unroll
      for (int nh = 0; nh < NH; ++nh)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int head = nh * 8 + 2 * t4 + e;
          if (head < G) {
            float* yp = mine + head * D;
#pragma unroll
            for (int mt = 0; mt < 8; ++mt) {
              yp[mt * 16 + gid] = yacc[mt][nh][e];
              yp[mt * 16 + gid + 8] = yacc[mt][nh][2 + e];
            }
          }
        }
    }
    named_barrier_sync(1 + grp, ST_CONS);
    const size_t pbase = ((size_t)bh * nct + ci) * G;
    for (int idx = tid; idx < G * D; idx += ST_CONS) {
      const float* rp = red + idx;
      float y = 0.f;
#pragma unroll
      for (int w = 0; w < ST_WARPS; ++w) y += rp[(size_t)w * (G * D)];
      a.tpy[pbase * D + idx] = dead ? 0.f : y;
    }
    if (tid < G) {
      float l = 0.f;
#pragma unroll
      for (int w = 0; w < ST_WARPS; ++w) l += tsum[w * 16 + tid];
      a.tpml[pbase + tid] = make_float2(txm[tid], l);
    }
    named_barrier_sync(1 + grp, ST_CONS);                 // red and the statistics are free for the next item
  }
  if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
}

template <int NH>
__global__ void __launch_bounds__(SE_THREADS, 1)
split_expand_kernel(const __grid_constant__ CUtensorMap tmS, const __grid_constant__ CUtensorMap tmTh,
                    const __grid_constant__ CUtensorMap tmU, const __grid_constant__ CUtensorMap tmWs,
                    const __grid_constant__ CUtensorMap tmKt, const __grid_constant__ CUtensorMap tmVt, const SplitArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* sm = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
  __shared__ __align__(8) ExpandBars bars;
  __shared__ uint32_t s_tmem;
  __shared__ float s_tstat[2 * ST_STAT];
  __shared__ float s_rstat[512];                  // row maxima and row sums of the two column halves
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if ((int)blockIdx.x >= a.e_grid) {             // a text CTA (it uses no tensor memory)
    text_role<NH>(tmKt, tmVt, a, sm, bars, s_tstat);
    return;
  }

  // CTA -> (KV head, row tile, range): the ranges of a tile are neighbours (they share the S tile in L2)
  const int s = blockIdx.x % a.NS;
  const int ht = blockIdx.x / a.NS;
  const int tile = ht % a.ntile, h = ht / a.ntile;
  const int n0 = s * a.NW;
  const int ngrp = a.NW >> 6;                          // 64-column groups of the range
  const uint32_t p_bytes = (uint32_t)a.NW * 256u;      // P: [NW/64][128 rows][128 B]
  unsigned char* ring = sm + p_bytes;

  if (tid == 0) {
    for (int i = 0; i < a.e_stages; ++i) { mbar_init(&bars.full[i], 1); mbar_init(&bars.empty[i], 1); }
    mbar_init(&bars.l_done, 1);
    mbar_init(&bars.p_ready, 8);
    mbar_init(&bars.w_done, 1);
    mbar_init(&bars.w_free, 8);
    fence_mbar_init();
  }
  if (warp == 8) tmem_alloc(&s_tmem, (uint32_t)a.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = s_tmem;
  const uint32_t th_bytes = (uint32_t)ngrp * 8192u;    // theta rows of a chunk: [group][64 rows][128 B]
  // The CTAs of a (KV head, range) walk the same theta and U chunks; each starts at another chunk (its row tile's number),
  // so that they do not all ask the L2 slice that holds a line for it at the same moment.  The sums run over the same terms.
  auto chunk1 = [&](int i) { const int k = i + tile % a.nk1; return k < a.nk1 ? k : k - a.nk1; };
  auto chunk2 = [&](int i) { const int k = i + tile % ngrp; return k < ngrp ? k : k - ngrp; };
  const uint32_t u_box = (uint32_t)a.brow * 128u;

  if (warp == 9) {
    // ---------------- producer ----------------
    if (lane == 0) {
      tma_prefetch_desc(&tmS); tma_prefetch_desc(&tmTh); tma_prefetch_desc(&tmU);
      uint32_t slot = 0, phase = 1;
      bool ok = true;
      // the first ring of stages: theta rows (parameters, never written by the library) before the dependency wait,
      // the scores of the kernel before after it
      const int npre = a.nk1 < a.e_stages ? a.nk1 : a.e_stages;
      for (int i = 0; i < npre; ++i) {
        const int kc = chunk1(i);
        unsigned char* dst = ring + i * a.e_stage_bytes;
        mbar_expect_tx(&bars.full[i], 16384u + th_bytes);
        tma_load_4d(dst + 16384, &tmTh, 0, kc * 64, n0 >> 6, h, &bars.full[i]);
      }
      grid_dep_wait();
      grid_dep_launch();                      // only now: the output kernel relies on the score kernel being complete
      for (int i = 0; i < npre; ++i) tma_load_3d(ring + i * a.e_stage_bytes, &tmS, chunk1(i) * 64, tile * SP_TILE_ROWS, h, &bars.full[i]);
      slot = (uint32_t)npre;
      if (slot == (uint32_t)a.e_stages) { slot = 0; phase ^= 1u; }
      for (int i = npre; i < a.nk1 && ok; ++i) {
        const int kc = chunk1(i);
        if (!mbar_wait_bounded(&bars.empty[slot], phase)) { ok = false; break; }
        unsigned char* dst = ring + slot * a.e_stage_bytes;
        mbar_expect_tx(&bars.full[slot], 16384u + th_bytes);
        tma_load_4d(dst + 16384, &tmTh, 0, kc * 64, n0 >> 6, h, &bars.full[slot]);
        tma_load_3d(dst, &tmS, kc * 64, tile * SP_TILE_ROWS, h, &bars.full[slot]);
        if (++slot == (uint32_t)a.e_stages) { slot = 0; phase ^= 1u; }
      }
      for (int wp = 0; wp < a.npass && ok; ++wp)
        for (int i = 0; i < ngrp && ok; ++i) {
          const int kc = chunk2(i);
          if (!mbar_wait_bounded(&bars.empty[slot], phase)) { ok = false; break; }
          unsigned char* dst = ring + slot * a.e_stage_bytes;
          mbar_expect_tx(&bars.full[slot], (uint32_t)a.nbox * u_box);
          for (int bx = 0; bx < a.nbox; ++bx)
            tma_load_3d(dst + bx * u_box, &tmU, n0 + kc * 64, wp * a.prow + bx * a.brow, h, &bars.full[slot]);
          if (++slot == (uint32_t)a.e_stages) { slot = 0; phase ^= 1u; }
        }
      if (!ok) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
    }
  } else if (warp == 8) {
    // ---------------- MMA issue ----------------
    const uint32_t sm_u = smem_addr(sm), ring_u = sm_u + p_bytes;
    const uint32_t idesc_L = umma_idesc_bf16(128, a.NW, 0, 1);
    const uint32_t idesc_W = umma_idesc_bf16(128, a.brow, 0, 0);
    uint32_t slot = 0, phase = 0;
    bool dead = false;
    auto wait_on = [&](uint64_t* bar, uint32_t parity) {
      if (!dead && !mbar_wait_bounded(bar, parity)) dead = true;
      __syncwarp();
    };
    for (int i = 0; i < a.nk1; ++i) {
      const int kc = chunk1(i);
      wait_on(&bars.full[slot], phase);
      tc_fence_after();
      if (lane == 0) {
        const uint32_t s_u = ring_u + slot * a.e_stage_bytes, th_u = s_u + 16384u;
        const int ksteps = min(4, (a.m - kc * 64 + 15) >> 4);
        for (int ks = 0; ks < ksteps; ++ks) {
          const uint64_t adesc = umma_smem_desc(s_u + (uint32_t)(ks * 32), 16u, 1024u, UMMA_LAYOUT_SW128);
          const uint64_t bdesc = umma_smem_desc(th_u + (uint32_t)(ks * 2048), 8192u, 1024u, UMMA_LAYOUT_SW128);
          umma_bf16(tb, adesc, bdesc, idesc_L, (i | ks) ? 1u : 0u);
        }
        umma_commit(&bars.empty[slot]);
        if (i == a.nk1 - 1) umma_commit(&bars.l_done);
      }
      __syncwarp();
      if (++slot == (uint32_t)a.e_stages) { slot = 0; phase ^= 1u; }
    }
    wait_on(&bars.p_ready, 0);
    for (int wp = 0; wp < a.npass; ++wp) {
      if (wp > 0) wait_on(&bars.w_free, (uint32_t)((wp - 1) & 1));
      tc_fence_after();
      for (int i = 0; i < ngrp; ++i) {
        const int kc = chunk2(i);
        wait_on(&bars.full[slot], phase);
        tc_fence_after();
        if (lane == 0) {
          const uint32_t u_u = ring_u + slot * a.e_stage_bytes;
          const uint32_t p_u = sm_u + (uint32_t)kc * 16384u;
#pragma unroll 1                 // rolled: this code runs once per CTA, and its first pass is paced by instruction fetch
          for (int ks = 0; ks < 4; ++ks) {
            const uint64_t adesc = umma_smem_desc(p_u + (uint32_t)(ks * 32), 16u, 1024u, UMMA_LAYOUT_SW128);
#pragma unroll 1
            for (int bx = 0; bx < a.nbox; ++bx) {
              const uint64_t bdesc = umma_smem_desc(u_u + bx * u_box + (uint32_t)(ks * 32), 16u, 1024u, UMMA_LAYOUT_SW128);
              umma_bf16(tb + (uint32_t)(bx * a.brow), adesc, bdesc, idesc_W, (i | ks) ? 1u : 0u);
            }
          }
          umma_commit(&bars.empty[slot]);
          if (i == ngrp - 1) umma_commit(&bars.w_done);
        }
        __syncwarp();
        if (++slot == (uint32_t)a.e_stages) { slot = 0; phase ^= 1u; }
      }
    }
    if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
  } else {
    // ---------------- warps 0-7: lane <-> expansion row (lane quarter = warp mod 4), half of the columns each ----------------
    const int qw = warp & 3, hf = warp >> 2;
    const int row = qw * 32 + lane;                            // row of the tile = tensor-memory lane
    const long long rho = (long long)tile * SP_TILE_ROWS + row;
    const bool valid = rho < a.rows_h;
    const uint32_t trow = tb + ((uint32_t)(qw * 32) << 16);
    const int cw = a.NW >> 1, cb = hf * cw;                    // this warp's columns of the logits: [cb, cb + cw), 32-column steps
    bool ok = mbar_wait_bounded(&bars.l_done, 0);
    __syncwarp();
    tc_fence_after();
    // pass 1: row maximum (32 columns per load, the next load in flight while one is reduced); the halves meet in shared memory
    float mx = -INFINITY;
    {
      uint32_t ra[32], rb[32];
      tmem_ld_issue_x32(trow + (uint32_t)cb, ra);
      for (int c0 = 0; c0 < cw; c0 += 64) {
        tmem_ld_wait_x32(ra);
        if (c0 + 32 < cw) tmem_ld_issue_x32(trow + (uint32_t)(cb + c0 + 32), rb);
#pragma unroll
        for (int k = 0; k < 32; ++k) mx = fmaxf(mx, __uint_as_float(ra[k]));
        if (c0 + 32 < cw) {
          tmem_ld_wait_x32(rb);
          if (c0 + 64 < cw) tmem_ld_issue_x32(trow + (uint32_t)(cb + c0 + 64), ra);
#pragma unroll
          for (int k = 0; k < 32; ++k) mx = fmaxf(mx, __uint_as_float(rb[k]));
        }
      }
    }
    s_rstat[hf * 128 + row] = mx;
    named_barrier_sync(3, 256);
    mx = fmaxf(mx, s_rstat[(hf ^ 1) * 128 + row]);
    // pass 2: probabilities relative to it, as the K-major A operand of the second product
    float sum = 0.f;
    unsigned char* p_row = sm + (uint32_t)row * 128u;
    {
      uint32_t ra[32];
      auto emit = [&](int c0, const uint32_t (&r)[32]) {       // 32 columns -> four 16-byte pieces of the row
        uint32_t w[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const float p0 = fast_exp2(__uint_as_float(r[2 * k]) - mx), p1 = fast_exp2(__uint_as_float(r[2 * k + 1]) - mx);
          sum += p0 + p1;
          w[k] = pack2_bf16(p0, p1);
        }
        unsigned char* g = p_row + (uint32_t)(c0 >> 6) * 16384u;
        const int piece = (c0 & 63) >> 3;
#pragma unroll
        for (int q = 0; q < 4; ++q)
          *reinterpret_cast<uint4*>(g + (((piece + q) ^ (row & 7)) << 4)) = make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
      };
      for (int c0 = cb; c0 < cb + cw; c0 += 32) {
        tmem_ld_issue_x32(trow + (uint32_t)c0, ra);
        tmem_ld_wait_x32(ra);
        emit(c0, ra);
      }
    }
    s_rstat[256 + hf * 128 + row] = sum;
    fence_proxy_async();                                       // P is read by the tensor core (async proxy)
    tc_fence_before();
    named_barrier_sync(3, 256);
    if (hf == 0 && valid && ok) a.stat[((size_t)h * a.NS + s) * a.rows_h + rho] = make_float2(mx, sum + s_rstat[256 + 128 + row]);
    __syncwarp();
    if (lane == 0) mbar_arrive(&bars.p_ready);
    // the weights of the range, pass by pass.  The last pass goes through the shared memory of P (dead by then): 64-column
    // tiles in the swizzled row layout, stored by the TMA engine (rows and columns outside the tensor are clipped), the
    // two halves of the warps taking alternate tiles; earlier passes (retained lengths above 512) store from registers.
    __nv_bfloat16* wrow = a.Wp + (((size_t)h * a.NS + s) * a.rows_h + (valid ? rho : 0)) * a.ms;
    const int ntile = a.NW >> 6;                                 // staging tiles of 16 KB in the region of P
    const int tph = ntile >= 2 ? ntile >> 1 : 1;                 // staging tiles per half
    const bool issuer = qw == 0 && lane == 0;                    // the thread of this half that owns its bulk stores
    for (int wp = 0; wp < a.npass; ++wp) {
      if (ok && !mbar_wait_bounded(&bars.w_done, (uint32_t)(wp & 1))) ok = false;
      __syncwarp();
      tc_fence_after();
      const int j0 = wp * a.prow;
      if (wp == a.npass - 1) {
        if (ntile >= 2 || hf == 0) {
          const int step = ntile >= 2 ? 2 : 1;
          int li = 0;
          for (int cg = ntile >= 2 ? hf : 0; cg * 64 < a.prow && j0 + cg * 64 < a.m; cg += step, ++li) {
            const int c0 = cg * 64;
            unsigned char* tile_sm = sm + (uint32_t)((ntile >= 2 ? hf * tph : 0) + li % tph) * 16384u;
            if (li >= tph) {                                     // the store that last read this tile has to be done with it
              if (issuer) { if (tph >= 2) bulk_wait_group_read<1>(); else bulk_wait_group_read<0>(); }
              named_barrier_sync(4 + hf, 128);
            }
            const int ncol = min(64, a.prow - c0);
            uint32_t ra[32];
            for (int cc = 0; cc < ncol; cc += 32) {
              tmem_ld_issue_x32(trow + (uint32_t)(c0 + cc), ra);
              tmem_ld_wait_x32(ra);
              unsigned char* g = tile_sm + (uint32_t)row * 128u;
              const int piece = cc >> 3;
#pragma unroll
              for (int q = 0; q < 4; ++q)
                *reinterpret_cast<uint4*>(g + (((piece + q) ^ (row & 7)) << 4)) =
                    make_uint4(pack2_bf16(__uint_as_float(ra[8 * q]), __uint_as_float(ra[8 * q + 1])),
                               pack2_bf16(__uint_as_float(ra[8 * q + 2]), __uint_as_float(ra[8 * q + 3])),
                               pack2_bf16(__uint_as_float(ra[8 * q + 4]), __uint_as_float(ra[8 * q + 5])),
                               pack2_bf16(__uint_as_float(ra[8 * q + 6]), __uint_as_float(ra[8 * q + 7])));
            }
            fence_proxy_async();
            named_barrier_sync(4 + hf, 128);
            if (issuer && ok) {
              tma_store_4d(&tmWs, tile_sm, j0 + c0, tile * SP_TILE_ROWS, s, h);
              bulk_commit_group();
            }
          }
          if (issuer) bulk_wait_group_all();
        }
      } else if (hf == 0) {
        for (int c0 = 0; c0 < a.prow && j0 + c0 < a.ms; c0 += 16) {
          float v[16];
          tmem_ld_x16(trow + (uint32_t)c0, v);
          if (valid && ok) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const int j = j0 + c0 + 8 * half;
              if (j < a.ms)
                *reinterpret_cast<uint4*>(wrow + j) =
                    make_uint4(pack2_bf16(v[8 * half], v[8 * half + 1]), pack2_bf16(v[8 * half + 2], v[8 * half + 3]),
                               pack2_bf16(v[8 * half + 4], v[8 * half + 5]), pack2_bf16(v[8 * half + 6], v[8 * half + 7]));
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars.w_free);
    }
    if (!ok && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 8) tmem_dealloc(tb, (uint32_t)a.tmem_cols);
}

template <int NH>
static cudaError_t launch_expand_inst(const CUtensorMap* tm, const SplitArgs& a, size_t smem, cudaStream_t st) {
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(split_expand_kernel<NH>), smem);
  if (e != cudaSuccess) return e;
  return launch_dependent(split_expand_kernel<NH>, dim3(a.e_grid + a.tx_grid), dim3(SE_THREADS), smem, st, tm[0], tm[1], tm[2], tm[3],
                          tm[4], tm[5], a);
}

// tm: S, theta, U, partial weights (store), K_txt, V_txt
cudaError_t launch_split_expand(const CUtensorMap* tm, const SplitArgs& a, const SplitPlan& p, cudaStream_t st) {
  // a text CTA needs its stages and the reduction buffer of its four warps
  const size_t text_smem = (size_t)st_groups(a.G) * st_group_bytes(a.G) + 1024;
  const size_t smem = a.tx_grid > 0 && text_smem > p.e_smem ? text_smem : p.e_smem;
  ProfScope prof(KVC_KERNEL_SPLIT_EXPAND, st);
  return a.G > 8 ? launch_expand_inst<2>(tm, a, smem, st) : launch_expand_inst<1>(tm, a, smem, st);
}

}  // namespace kvc
