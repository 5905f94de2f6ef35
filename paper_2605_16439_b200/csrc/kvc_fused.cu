// Algorithm 1 as ONE kernel for bf16 storage: compressed scores, expansion by theta, joint softmax with
// the text logits, re-projection by U^T, product with the compressed values, mu term, normalisation.
//
// Work unit = one KV head h, NB sequences and RB vision blocks of each (NB*RB*G <= 16 expansion rows),
// plus a slice of the sequences' text rows.  A persistent CTA streams, per unit, through a ring of large
// shared-memory stages filled by the TMA engine (tiled tensor maps, 128-byte swizzle):
//   pass A   stage c = rows [16 JC c, 16 JC (c+1)) of K_tilde of every block of the unit  +  the same rows
//            of theta[h] (all n columns).  Scores S_c = sigma q K_c^T go through shared memory as bf16 and
//            are multiplied into the logits L += S_c theta_c, which stay in registers (rows x n, fp32).
//   text     stage = TCH rows of K_txt and V_txt per sequence; every warp runs an online-softmax
//            attention over its own 16-row tiles.
//   softmax  one maximum per (sequence, head) over all blocks of the unit and its text rows; P = 2^(L - max).
//   pass C   stage c = rows of V_tilde + the same rows of U[h]:  W_c = P U_c^T (split over the warps' column
//            ranges, reduced through shared memory), then y += W_c V_c.
// theta/U rows (L2-resident, shared by all sequences) and capsule rows (HBM) arrive interleaved in the same
// stages, so both streams stay busy for the whole unit.  All matrix products run on mma.sync m16n8k16.
// A unit that holds every block of its sequences writes `out` directly; otherwise the units of a
// (sequence, KV head) leave (max, sum, y) partials and the last one to arrive merges them.
#include "kvc_tma.cuh"
#include "kvc_internal.cuh"

namespace kvc {

constexpr int FW = 8;                        // consumer warps
constexpr int FTHREADS = (FW + 1) * 32;      // + one producer warp
constexpr int FCONS = FW * 32;
constexpr int FMAX_STAGES = 8;
constexpr int QLD = 136;                     // row stride of the query tile in elements (272 B: conflict-free ldmatrix)
constexpr int SLD = 24;                      // row stride of the 16-column score / weight tiles (48 B)
constexpr uint32_t SMEM_LIMIT = 232448;      // 227 KB per CTA on sm_100

struct FusedArgs {
  const __nv_bfloat16* q;
  const __nv_bfloat16* mu;
  __nv_bfloat16* out;
  int B, H_kv, G, R, m, n, T;
  int NB, RB, nbg, nrg, units, JC, NJ, TCH, Tper, ncg, stages;
  uint32_t par_bytes, k_half_bytes, txt_half_bytes, stage_bytes;
  uint32_t off_q, off_S, off_W, off_wred, off_rstat, off_tstat, off_hstat, off_yred;
  float* part_y;      // [B*H_kv][nrg][G][D]  partial outputs (only when nrg > 1)
  float2* part_ml;    // [B*H_kv][nrg][G]     (max in log2 units, sum)
  int* cnt;           // [B*H_kv] arrival counters, zero between calls
  int* status;        // device status word
};

__device__ __forceinline__ void consumer_sync() { named_barrier_sync(1, FCONS); }

template <int MT, int NTW, int NH>
__global__ void __launch_bounds__(FTHREADS, 1)
fused_decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const __grid_constant__ CUtensorMap tmKt, const __grid_constant__ CUtensorMap tmVt,
                    const __grid_constant__ CUtensorMap tmTh, const __grid_constant__ CUtensorMap tmU,
                    const FusedArgs a) {
  constexpr int ROWS = 16 * MT;
  constexpr int KK = (NTW + 1) / 2;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* sm = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
  __shared__ __align__(8) uint64_t full_bar[FMAX_STAGES], empty_bar[FMAX_STAGES];
  __shared__ int s_last;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < a.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], FW); }
    fence_mbar_init();
  }
  // score and weight tiles start as zeros: their padding rows and columns are read by the MMAs
  {
    uint32_t* z = reinterpret_cast<uint32_t*>(sm + a.off_S);
    const int words = (2 * ROWS * SLD + (ROWS + 16) * SLD) / 2;
    for (int i = tid; i < words; i += FTHREADS) z[i] = 0u;
  }
  __syncthreads();

  const int per_h = a.nbg * a.nrg;

  if (warp == FW) {
    // ================= producer: one thread feeds the ring =================
    if (lane != 0) return;
    tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmTh); tma_prefetch_desc(&tmU);
    if (a.T > 0) { tma_prefetch_desc(&tmKt); tma_prefetch_desc(&tmVt); }
    bool dead = false, first = true;
    uint32_t it = 0;
    for (int u = blockIdx.x; u < a.units && !dead; u += gridDim.x) {
      const int h = u / per_h, rem = u - h * per_h;
      const int bg = rem / a.nrg, rg = rem - bg * a.nrg;
      const int b0 = bg * a.NB, r0 = rg * a.RB;
      const int ts0 = rg * a.Tper;
      const int ts1 = min(a.T, ts0 + a.Tper);
      const int nts = ts1 > ts0 ? (ts1 - ts0 + a.TCH - 1) / a.TCH : 0;
      for (int pass = 0; pass < 2 && !dead; ++pass) {
        const CUtensorMap* tp = pass == 0 ? &tmTh : &tmU;
        const CUtensorMap* tk = pass == 0 ? &tmK : &tmV;
        for (int c = 0; c < a.NJ; ++c, ++it) {
          const uint32_t slot = it % a.stages, use = it / a.stages;
          if (use > 0 && !mbar_wait_bounded(&empty_bar[slot], (use - 1) & 1u)) { dead = true; break; }
          unsigned char* dst = sm + slot * a.stage_bytes;
          const int j0 = c * 16 * a.JC;
          mbar_expect_tx(&full_bar[slot], a.par_bytes + 2 * a.k_half_bytes);
          tma_load_4d(dst, tp, 0, j0, 0, h, &full_bar[slot]);                 // parameters: never written by this library
          if (first) { grid_dep_wait(); first = false; }                       // everything else may come from the stream's previous kernel
          tma_load_5d(dst + a.par_bytes, tk, 0, j0, r0, h, b0, &full_bar[slot]);
          tma_load_5d(dst + a.par_bytes + a.k_half_bytes, tk, 64, j0, r0, h, b0, &full_bar[slot]);
        }
        if (pass == 0) {
          for (int ts = 0; ts < nts && !dead; ++ts, ++it) {
            const uint32_t slot = it % a.stages, use = it / a.stages;
            if (use > 0 && !mbar_wait_bounded(&empty_bar[slot], (use - 1) & 1u)) { dead = true; break; }
            unsigned char* dst = sm + slot * a.stage_bytes;
            const int y = ts0 + ts * a.TCH;
            mbar_expect_tx(&full_bar[slot], 4 * a.txt_half_bytes);
            tma_load_4d(dst, &tmKt, 0, y, h, b0, &full_bar[slot]);
            tma_load_4d(dst + a.txt_half_bytes, &tmKt, 64, y, h, b0, &full_bar[slot]);
            tma_load_4d(dst + 2 * a.txt_half_bytes, &tmVt, 0, y, h, b0, &full_bar[slot]);
            tma_load_4d(dst + 3 * a.txt_half_bytes, &tmVt, 64, y, h, b0, &full_bar[slot]);
          }
        }
      }
    }
    if (dead) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
    return;
  }

  // ================= consumers =================
  const int gid = lane >> 2, t4 = lane & 3;
  const int G = a.G, RB = a.RB, JC = a.JC, ncg = a.ncg;
  const int WPG = FW / a.NB;                       // warps per sequence of the unit
  const int bl = warp / WPG, wig = warp - bl * WPG;
  const int c0 = warp * ncg * 8;                   // first column of L owned by this warp
  const int rows16 = 16 * JC;                      // rows of one block inside a stage
  const uint32_t sm_u = smem_addr(sm);
  const uint32_t q_u = sm_u + a.off_q, S_u = sm_u + a.off_S, W_u = sm_u + a.off_W;
  __nv_bfloat16* q_sm = reinterpret_cast<__nv_bfloat16*>(sm + a.off_q);
  __nv_bfloat16* S_sm = reinterpret_cast<__nv_bfloat16*>(sm + a.off_S);
  __nv_bfloat16* W_sm = reinterpret_cast<__nv_bfloat16*>(sm + a.off_W);
  float* wred = reinterpret_cast<float*>(sm + a.off_wred);
  float* rmax = reinterpret_cast<float*>(sm + a.off_rstat);
  float* rsum = rmax + FW * ROWS;
  float* tmax = reinterpret_cast<float*>(sm + a.off_tstat);
  float* tsum = tmax + FW * 16;
  float* hmax = reinterpret_cast<float*>(sm + a.off_hstat);
  float* hsum = hmax + a.NB * 16;
  float* vsum = hsum + a.NB * 16;
  float* yred = reinterpret_cast<float*>(sm + a.off_yred);
  const float qscale = 0.08838834764831845f * 1.4426950408889634f;   // sigma = 1/sqrt(128), logits kept in log2 units
  const int lrow = (lane & 7) + ((lane >> 3) & 1) * 8;              // ldmatrix row pattern: rows 0-15 in lanes 0-15, repeated
  const int lhi = lane >> 4;

  grid_dep_wait();
  grid_dep_launch();
  if (blockIdx.x == 0 && tid == 0) *a.status = 0;

  uint32_t it = 0;
  bool dead = false;

  for (int u = blockIdx.x; u < a.units; u += gridDim.x) {
    const int h = u / per_h, rem = u - h * per_h;
    const int bg = rem / a.nrg, rg = rem - bg * a.nrg;
    const int b0 = bg * a.NB, r0 = rg * a.RB;
    const int nbv = min(a.NB, a.B - b0);
    const int ts0 = rg * a.Tper;
    const int ts1 = min(a.T, ts0 + a.Tper);
    const int nts = ts1 > ts0 ? (ts1 - ts0 + a.TCH - 1) / a.TCH : 0;

    // ---- queries of the unit's sequences: [NB][16 heads][128], heads >= G and absent sequences are zero rows
    for (int idx = tid; idx < a.NB * 256; idx += FCONS) {
      const int tb = idx >> 8, g = (idx >> 4) & 15, piece = idx & 15;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (tb < nbv && g < G)
        v = *reinterpret_cast<const uint4*>(a.q + ((size_t)(b0 + tb) * a.H_kv * G + (size_t)h * G + g) * D + piece * 8);
      *reinterpret_cast<uint4*>(q_sm + (tb * 16 + g) * QLD + piece * 8) = v;
    }
    consumer_sync();
    uint32_t qf[NH][8][2];                          // B operand of the score MMA: heads of sequence bl
#pragma unroll
    for (int nh = 0; nh < NH; ++nh)
#pragma unroll
      for (int k2 = 0; k2 < 4; ++k2) {
        uint32_t r[4];
        ldsm_x4(r, q_u + (uint32_t)(((bl * 16 + nh * 8 + (lane & 7)) * QLD + k2 * 32 + (lane >> 3) * 8) * 2));
        qf[nh][2 * k2][0] = r[0]; qf[nh][2 * k2][1] = r[1];
        qf[nh][2 * k2 + 1][0] = r[2]; qf[nh][2 * k2 + 1][1] = r[3];
      }

    // expansion rows held by this lane: rho = mt*16 + gid + 8*hr  <->  (sequence, block, head)
    bool rvalid[MT][2];
    int rhead[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int hr = 0; hr < 2; ++hr) {
        const int rho = mt * 16 + gid + 8 * hr;
        const int bi = rho / G, g = rho - bi * G;
        const int rbl = bi / RB, rrl = bi - rbl * RB;
        rvalid[mt][hr] = rho < a.NB * RB * G && rbl < nbv && r0 + rrl < a.R;
        rhead[mt][hr] = rvalid[mt][hr] ? rbl * 16 + g : 0;
      }

    float accL[MT][NTW][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NTW; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) accL[mt][nt][e] = 0.f;

    // =============================== pass A: scores and expansion by theta ===============================
    int buf = 0;
    for (int c = 0; c < a.NJ; ++c, ++it) {
      const uint32_t slot = it % a.stages, use = it / a.stages;
      if (!dead && !mbar_wait_bounded(&full_bar[slot], use & 1u)) dead = true;
      const uint32_t par_u = sm_u + slot * a.stage_bytes, k_u = par_u + a.par_bytes;
      for (int s = 0; s < JC; ++s) {
        if ((c * JC + s) * 16 >= a.m) break;
        // S_c[rows of my blocks][16] = sigma q K_c^T
        for (int rl = wig; rl < RB; rl += WPG) {
          const int bi = bl * RB + rl;
          const int row = bi * rows16 + s * 16 + lrow;
          float sc[NH][4];
#pragma unroll
          for (int nh = 0; nh < NH; ++nh)
#pragma unroll
            for (int e = 0; e < 4; ++e) sc[nh][e] = 0.f;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            uint32_t af[4];
            ldsm_x4(af, k_u + (ks >> 2) * a.k_half_bytes + swz(row, (ks & 3) * 2 + lhi));
#pragma unroll
            for (int nh = 0; nh < NH; ++nh) mma_bf16_16816(sc[nh], af, qf[nh][ks][0], qf[nh][ks][1]);
          }
          __nv_bfloat16* Sb = S_sm + buf * (ROWS * SLD);
#pragma unroll
          for (int nh = 0; nh < NH; ++nh)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int head = nh * 8 + 2 * t4 + (e & 1), j = gid + (e >> 1) * 8;
              if (head < G) Sb[(bi * G + head) * SLD + j] = __float2bfloat16_rn(sc[nh][e] * qscale);
            }
        }
        consumer_sync();
        // L[:, my columns] += S_c theta_c
        uint32_t af[MT][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
          ldsm_x4(af[mt], S_u + (uint32_t)((buf * (ROWS * SLD) + (mt * 16 + lrow) * SLD + lhi * 8) * 2));
#pragma unroll
        for (int np = 0; np < KK; ++np) {
          if (2 * np < ncg) {
            int col = c0 + np * 16 + lhi * 8;
            if (col >= a.n) col = c0;
            const int row = (col >> 6) * rows16 + s * 16 + lrow;
            uint32_t bf[4];
            ldsm_x4_t(bf, par_u + swz(row, (col & 63) >> 3));
            const int n1 = 2 * np + 1 < NTW ? 2 * np + 1 : NTW - 1;
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
              mma_bf16_16816(accL[mt][2 * np], af[mt], bf[0], bf[1]);
              if (2 * np + 1 < NTW && 2 * np + 1 < ncg) mma_bf16_16816(accL[mt][n1], af[mt], bf[2], bf[3]);
            }
          }
        }
        buf ^= 1;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[slot]);
    }

    // =============================== text rows: online-softmax attention per warp ===============================
    float yacc[16][4];
#pragma unroll
    for (int nt = 0; nt < 16; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) yacc[nt][e] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    for (int ts = 0; ts < nts; ++ts, ++it) {
      const uint32_t slot = it % a.stages, use = it / a.stages;
      if (!dead && !mbar_wait_bounded(&full_bar[slot], use & 1u)) dead = true;
      const uint32_t kt_u = sm_u + slot * a.stage_bytes, vt_u = kt_u + 2 * a.txt_half_bytes;
      for (int tile = wig; tile * 16 < a.TCH; tile += WPG) {
        const int t_first = ts0 + ts * a.TCH + tile * 16;
        if (t_first >= ts1) break;
        const int row0 = bl * a.TCH + tile * 16;
        float cc[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) cc[nt][e] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          uint32_t aq[4], bk[4];
          ldsm_x4(aq, q_u + (uint32_t)(((bl * 16 + lrow) * QLD + ks * 16 + lhi * 8) * 2));
          ldsm_x4(bk, kt_u + (ks >> 2) * a.txt_half_bytes +
                          swz(row0 + (lane & 7) + lhi * 8, (ks & 3) * 2 + ((lane >> 3) & 1)));
          mma_bf16_16816(cc[0], aq, bk[0], bk[1]);
          mma_bf16_16816(cc[1], aq, bk[2], bk[3]);
        }
        // cc[nt][e]: head gid + 8*(e>>1), text row t_first + nt*8 + 2*t4 + (e&1)
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int t = t_first + nt * 8 + 2 * t4 + (e & 1);
            cc[nt][e] = t < ts1 ? cc[nt][e] * qscale : -INFINITY;
          }
#pragma unroll
        for (int hr = 0; hr < 2; ++hr) {
          float mx = fmaxf(fmaxf(cc[0][2 * hr], cc[0][2 * hr + 1]), fmaxf(cc[1][2 * hr], cc[1][2 * hr + 1]));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
          const float m_new = fmaxf(m_run[hr], mx);              // finite: the tile has at least one valid row
          const float scl = fast_exp2(m_run[hr] - m_new);        // 0 on the first tile
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
          l_run[hr] = l_run[hr] * scl + ps;
          if (scl != 1.f) {
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) { yacc[nt][2 * hr] *= scl; yacc[nt][2 * hr + 1] *= scl; }
          }
        }
        uint32_t pa[4];
        pa[0] = pack2_bf16(cc[0][0], cc[0][1]); pa[1] = pack2_bf16(cc[0][2], cc[0][3]);
        pa[2] = pack2_bf16(cc[1][0], cc[1][1]); pa[3] = pack2_bf16(cc[1][2], cc[1][3]);
#pragma unroll
        for (int np = 0; np < 8; ++np) {
          const int col = np * 16 + lhi * 8;
          uint32_t bv[4];
          ldsm_x4_t(bv, vt_u + (col >> 6) * a.txt_half_bytes + swz(row0 + lrow, (col & 63) >> 3));
          mma_bf16_16816(yacc[2 * np], pa, bv[0], bv[1]);
          mma_bf16_16816(yacc[2 * np + 1], pa, bv[2], bv[3]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[slot]);
    }

    // =============================== joint softmax over the unit's blocks and text rows ===============================
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int hr = 0; hr < 2; ++hr) {
        float mx = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < NTW; ++nt)
          if (nt < ncg) mx = fmaxf(mx, fmaxf(accL[mt][nt][2 * hr], accL[mt][nt][2 * hr + 1]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        if (t4 == 0) rmax[warp * ROWS + mt * 16 + gid + 8 * hr] = rvalid[mt][hr] ? mx : -INFINITY;
      }
    if (t4 == 0) { tmax[warp * 16 + gid] = m_run[0]; tmax[warp * 16 + gid + 8] = m_run[1]; }
    consumer_sync();
    if (tid < a.NB * 16) {
      const int tb = tid >> 4, g = tid & 15;
      float mx = 0.f;
      if (g < G && tb < nbv) {
        mx = -INFINITY;
        for (int rl = 0; rl < RB; ++rl)
          if (r0 + rl < a.R)
            for (int w = 0; w < FW; ++w) mx = fmaxf(mx, rmax[w * ROWS + (tb * RB + rl) * G + g]);
        for (int w = tb * WPG; w < (tb + 1) * WPG; ++w) mx = fmaxf(mx, tmax[w * 16 + g]);
      }
      hmax[tid] = mx;
    }
    consumer_sync();
    uint32_t pf[MT][KK][4];                         // P as A operand of the re-projection (bf16), this warp's columns
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
      for (int hr = 0; hr < 2; ++hr) {
        const bool ok = rvalid[mt][hr];
        const float M = hmax[rhead[mt][hr]];
        float sum = 0.f;
#pragma unroll
        for (int nt = 0; nt < NTW; ++nt)
#pragma unroll
          for (int k = 0; k < 2; ++k) {
            const float p = (ok && nt < ncg) ? fast_exp2(accL[mt][nt][2 * hr + k] - M) : 0.f;
            accL[mt][nt][2 * hr + k] = p;
            sum += p;
          }
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        sum += __shfl_xor_sync(0xffffffffu, sum, 2);
        if (t4 == 0) rsum[warp * ROWS + mt * 16 + gid + 8 * hr] = sum;
      }
#pragma unroll
      for (int kk = 0; kk < KK; ++kk) {
        pf[mt][kk][0] = pack2_bf16(accL[mt][2 * kk][0], accL[mt][2 * kk][1]);
        pf[mt][kk][1] = pack2_bf16(accL[mt][2 * kk][2], accL[mt][2 * kk][3]);
        const int n1 = 2 * kk + 1 < NTW ? 2 * kk + 1 : NTW - 1;
        pf[mt][kk][2] = 2 * kk + 1 < NTW ? pack2_bf16(accL[mt][n1][0], accL[mt][n1][1]) : 0u;
        pf[mt][kk][3] = 2 * kk + 1 < NTW ? pack2_bf16(accL[mt][n1][2], accL[mt][n1][3]) : 0u;
      }
    }
    // the text accumulators move to the same reference maximum
#pragma unroll
    for (int hr = 0; hr < 2; ++hr) {
      const int head = gid + 8 * hr;
      const float M = hmax[bl * 16 + head];
      const float scl = m_run[hr] == -INFINITY ? 0.f : fast_exp2(m_run[hr] - M);
      float l = l_run[hr] * scl;
      l += __shfl_xor_sync(0xffffffffu, l, 1);
      l += __shfl_xor_sync(0xffffffffu, l, 2);
#pragma unroll
      for (int nt = 0; nt < 16; ++nt) { yacc[nt][2 * hr] *= scl; yacc[nt][2 * hr + 1] *= scl; }
      if (t4 == 0) tsum[warp * 16 + head] = l;
    }
    consumer_sync();
    if (tid < a.NB * 16) {
      const int tb = tid >> 4, g = tid & 15;
      float vs = 0.f, tsm = 0.f;
      if (g < G && tb < nbv) {
        for (int rl = 0; rl < RB; ++rl)
          if (r0 + rl < a.R)
            for (int w = 0; w < FW; ++w) vs += rsum[w * ROWS + (tb * RB + rl) * G + g];
        for (int w = tb * WPG; w < (tb + 1) * WPG; ++w) tsm += tsum[w * 16 + g];
      }
      vsum[tid] = vs;
      hsum[tid] = vs + tsm;
    }

    // =============================== pass C: re-projection by U^T and product with V_tilde ===============================
    for (int c = 0; c < a.NJ; ++c, ++it) {
      const uint32_t slot = it % a.stages, use = it / a.stages;
      if (!dead && !mbar_wait_bounded(&full_bar[slot], use & 1u)) dead = true;
      const uint32_t par_u = sm_u + slot * a.stage_bytes, v_u = par_u + a.par_bytes;
      for (int s = 0; s < JC; ++s) {
        if ((c * JC + s) * 16 >= a.m) break;
        // partial W_c[rows][16] over this warp's columns of P
        float wc[MT][2][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) wc[mt][nt][e] = 0.f;
#pragma unroll
        for (int kk = 0; kk < KK; ++kk) {
          if (2 * kk < ncg) {
            int col = c0 + kk * 16 + ((lane >> 3) & 1) * 8;
            if (col >= a.n) col = c0;
            const int row = (col >> 6) * rows16 + s * 16 + (lane & 7) + lhi * 8;
            uint32_t bu[4];
            ldsm_x4(bu, par_u + swz(row, (col & 63) >> 3));
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
              mma_bf16_16816(wc[mt][0], pf[mt][kk], bu[0], bu[1]);
              mma_bf16_16816(wc[mt][1], pf[mt][kk], bu[2], bu[3]);
            }
          }
        }
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int hr = 0; hr < 2; ++hr)
              *reinterpret_cast<float2*>(&wred[(warp * ROWS + mt * 16 + gid + 8 * hr) * 16 + nt * 8 + 2 * t4]) =
                  make_float2(wc[mt][nt][2 * hr], wc[mt][nt][2 * hr + 1]);
        consumer_sync();
        for (int idx = tid; idx < ROWS * 16; idx += FCONS) {
          float w = 0.f;
#pragma unroll
          for (int x = 0; x < FW; ++x) w += wred[x * ROWS * 16 + idx];
          W_sm[(idx >> 4) * SLD + (idx & 15)] = __float2bfloat16_rn(w);
        }
        consumer_sync();
        // y[heads of sequence bl] += W_c[rows of block] V_c[block]
        for (int rl = wig; rl < RB; rl += WPG) {
          if (r0 + rl >= a.R || bl >= nbv) continue;
          const int bi = bl * RB + rl;
          uint32_t aw[4];
          ldsm_x4(aw, W_u + (uint32_t)(((bi * G + lrow) * SLD + lhi * 8) * 2));
          const int row = bi * rows16 + s * 16 + lrow;
#pragma unroll
          for (int np = 0; np < 8; ++np) {
            const int col = np * 16 + lhi * 8;
            uint32_t bv[4];
            ldsm_x4_t(bv, v_u + (col >> 6) * a.k_half_bytes + swz(row, (col & 63) >> 3));
            mma_bf16_16816(yacc[2 * np], aw, bv[0], bv[1]);
            mma_bf16_16816(yacc[2 * np + 1], aw, bv[2], bv[3]);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[slot]);
    }

    // =============================== unit end: reduce over warps, mu term, normalise or leave a partial ===============================
    for (int k = 0; k < WPG; ++k) {
      if (wig == k) {
#pragma unroll
        for (int hr = 0; hr < 2; ++hr) {
          const int head = gid + 8 * hr;
          if (head < G) {
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) {
              float2* p = reinterpret_cast<float2*>(&yred[(bl * 16 + head) * D + nt * 8 + 2 * t4]);
              float2 v = make_float2(yacc[nt][2 * hr], yacc[nt][2 * hr + 1]);
              if (k > 0) { const float2 o = *p; v.x += o.x; v.y += o.y; }
              *p = v;
            }
          }
        }
      }
      consumer_sync();
    }
    if (a.nrg == 1) {
      for (int idx = tid; idx < nbv * G * 64; idx += FCONS) {
        const int cp = idx & 63, g = (idx >> 6) % G, tb = idx / (64 * G);
        const float2 y = *reinterpret_cast<const float2*>(&yred[(tb * 16 + g) * D + 2 * cp]);
        const __nv_bfloat162 mu2 = *reinterpret_cast<const __nv_bfloat162*>(a.mu + h * D + 2 * cp);
        const float vs = vsum[tb * 16 + g], inv = 1.f / hsum[tb * 16 + g];
        const __nv_bfloat162 o = __floats2bfloat162_rn(fmaf(vs, __low2float(mu2), y.x) * inv, fmaf(vs, __high2float(mu2), y.y) * inv);
        *reinterpret_cast<__nv_bfloat162*>(a.out + ((size_t)(b0 + tb) * a.H_kv * G + (size_t)h * G + g) * D + 2 * cp) = o;
      }
    } else {
      // NB == 1 here: one sequence, several units along the block axis
      const int bh = b0 * a.H_kv + h;
      const size_t pbase = ((size_t)bh * a.nrg + rg) * G;
      for (int idx = tid; idx < G * D; idx += FCONS) {
        const int g = idx >> 7, col = idx & (D - 1);
        a.part_y[(pbase + g) * D + col] = fmaf(vsum[g], __bfloat162float(a.mu[h * D + col]), yred[g * D + col]);
      }
      if (tid < G) a.part_ml[pbase + tid] = make_float2(hmax[tid], hsum[tid]);
      __threadfence();
      consumer_sync();
      if (tid == 0) {
        const int old = atomicAdd(&a.cnt[bh], 1);
        s_last = old == a.nrg - 1 ? 1 : 0;
        if (s_last) a.cnt[bh] = 0;                  // every unit of (sequence, head) has arrived: ready for the next call
      }
      consumer_sync();
      if (s_last) {
        __threadfence();
        const size_t p0 = (size_t)bh * a.nrg * G;
        for (int idx = tid; idx < G * D; idx += FCONS) {
          const int g = idx >> 7, col = idx & (D - 1);
          float M = -INFINITY;
          for (int p = 0; p < a.nrg; ++p) M = fmaxf(M, __ldcg(&a.part_ml[p0 + (size_t)p * G + g]).x);
          float num = 0.f, den = 0.f;
          for (int p = 0; p < a.nrg; ++p) {
            const float2 ml = __ldcg(&a.part_ml[p0 + (size_t)p * G + g]);
            const float w = fast_exp2(ml.x - M);
            den = fmaf(w, ml.y, den);
            num = fmaf(w, __ldcg(&a.part_y[(p0 + (size_t)p * G + g) * D + col]), num);
          }
          a.out[((size_t)b0 * a.H_kv * G + (size_t)h * G + g) * D + col] = __float2bfloat16_rn(num / den);
        }
      }
    }
    consumer_sync();
  }
  if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
}

// ------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

bool encode_tensor_map_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                            const uint64_t* strides_bytes, const uint32_t* box) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t gd[5], gs[4];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) { gd[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) gs[i] = strides_bytes[i];
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gd, gs, bx, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

FusedPlan plan_fused(const kvc_layer* L, int B, int R) {
  FusedPlan p{};
  const int G = L->G, n = L->desc.n, m = L->m, H_kv = L->desc.H_kv;
  if (L->desc.dtype != KVC_BF16 || L->passthrough || R < 1 || B < 1 || n % 64 != 0 || n > 1024 || G > 16) return p;
  if (reinterpret_cast<uintptr_t>(L->desc.theta) & 15 || reinterpret_cast<uintptr_t>(L->desc.U) & 15) return p;
  const int sms = L->num_sms > 0 ? L->num_sms : 148;
  p.MT = 1;
  const int cap = 16 * p.MT;
  p.RB = R < cap / G ? R : cap / G;
  p.NB = 1;
  if (p.RB == R) {
    // whole sequences per unit: more sequences per unit share one pass over theta[h] and U[h]
    double best = 0;
    for (int nb = 1; nb <= 4; nb *= 2) {
      if (nb > 1 && (nb * R * G > cap || nb > B)) break;
      const long long units = (long long)H_kv * ceil_div(B, nb);
      const double cost = (double)ceil_div((int)units, sms) * ((double)nb * R * m * 512.0 + 4.0 * m * n);
      if (nb == 1 || cost < best) { best = cost; p.NB = nb; }
    }
  }
  p.nbg = ceil_div(B, p.NB);
  p.nrg = ceil_div(R, p.RB);
  p.units = H_kv * p.nbg * p.nrg;
  if (p.nrg > 1 && (long long)B * H_kv > KVC_MAX_COUNTERS) return p;
  p.ncg = n / 64;
  const uint32_t chunk = (uint32_t)p.NB * p.RB * 4096u + (uint32_t)n * 32u;
  int jc = (int)(65536u / chunk);
  const int jmax = ceil_div(m, 16) < 16 ? ceil_div(m, 16) : 16;
  p.JC = jc < 1 ? 1 : (jc > jmax ? jmax : jc);
  p.NJ = ceil_div(m, 16 * p.JC);
  p.par_bytes = (uint32_t)p.ncg * p.JC * 2048u;
  p.k_half_bytes = (uint32_t)p.NB * p.RB * p.JC * 2048u;
  p.stage_bytes = p.par_bytes + 2 * p.k_half_bytes;
  int tch = (int)(p.stage_bytes / (p.NB * 512u)) & ~15;
  p.TCH = tch > 256 ? 256 : tch;
  if (p.TCH < 16) return p;
  p.txt_half_bytes = (uint32_t)p.NB * p.TCH * 128u;
  const int rows = 16 * p.MT;
  uint32_t off = 0;
  auto take = [&](uint32_t bytes) { uint32_t o = off; off = (off + bytes + 127u) & ~127u; return o; };
  p.off_q = take((uint32_t)p.NB * 16 * QLD * 2);
  p.off_S = take((uint32_t)(2 * rows * SLD + (rows + 16) * SLD) * 2);
  p.off_W = p.off_S + (uint32_t)2 * rows * SLD * 2;
  p.off_wred = take((uint32_t)FW * rows * 16 * 4);
  p.off_rstat = take((uint32_t)2 * FW * rows * 4);
  p.off_tstat = take((uint32_t)2 * FW * 16 * 4);
  p.off_hstat = take((uint32_t)3 * p.NB * 16 * 4);
  p.off_yred = take((uint32_t)p.NB * 16 * D * 4);
  p.misc_bytes = off;
  const uint32_t avail = SMEM_LIMIT - 1024u - 2048u - p.misc_bytes;   // alignment slack; static shared memory and its padding
  int stages = (int)(avail / p.stage_bytes);
  p.stages = stages > FMAX_STAGES ? FMAX_STAGES : stages;
  if (p.stages < 2) return p;
  p.smem_bytes = (size_t)p.stages * p.stage_bytes + p.misc_bytes + 1024u;
  p.grid = p.units < sms ? p.units : sms;
  p.ok = 1;
  return p;
}

template <int MT, int NTW, int NH>
static cudaError_t launch_inst(const CUtensorMap* tm, const FusedArgs& fa, const FusedPlan& p, cudaStream_t st) {
  static size_t configured = 0;
  if (p.smem_bytes > configured) {
    cudaError_t e = cudaFuncSetAttribute(fused_decode_kernel<MT, NTW, NH>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)p.smem_bytes);
    if (e != cudaSuccess) return e;
    configured = p.smem_bytes;
  }
  return launch_dependent(fused_decode_kernel<MT, NTW, NH>, dim3(p.grid), dim3(FTHREADS), p.smem_bytes, st, tm[0], tm[1],
                          tm[2], tm[3], tm[4], tm[5], fa);
}

cudaError_t launch_fused(const kvc_layer* L, const DecodeArgs& a, const FusedPlan& p, cudaStream_t st, bool* encoded) {
  const int H_kv = a.H_kv, m = a.m, n = a.n, R = a.R, B = a.B;
  CUtensorMap tm[6];
  *encoded = false;
  {
    const uint64_t dims[5] = {(uint64_t)D, (uint64_t)m, (uint64_t)R, (uint64_t)H_kv, (uint64_t)B};
    const uint64_t str[4] = {256ull, (uint64_t)m * 256, (uint64_t)R * m * 256, (uint64_t)H_kv * R * m * 256};
    const uint32_t box[5] = {64u, (uint32_t)(16 * p.JC), (uint32_t)p.RB, 1u, (uint32_t)p.NB};
    if (!encode_tensor_map_bf16(&tm[0], a.Kc, 5, dims, str, box)) return cudaSuccess;
    if (!encode_tensor_map_bf16(&tm[1], a.Vc, 5, dims, str, box)) return cudaSuccess;
  }
  if (a.T > 0) {
    const uint64_t dims[4] = {(uint64_t)D, (uint64_t)a.T, (uint64_t)H_kv, (uint64_t)B};
    const uint64_t str[3] = {256ull, (uint64_t)a.T_cap * 256, (uint64_t)H_kv * a.T_cap * 256};
    const uint32_t box[4] = {64u, (uint32_t)p.TCH, 1u, (uint32_t)p.NB};
    if (!encode_tensor_map_bf16(&tm[2], a.K_txt, 4, dims, str, box)) return cudaSuccess;
    if (!encode_tensor_map_bf16(&tm[3], a.V_txt, 4, dims, str, box)) return cudaSuccess;
  } else {
    tm[2] = tm[0];
    tm[3] = tm[1];
  }
  {
    // theta, U [H_kv][m][n] viewed as (64 columns, m rows, n/64 column groups, H_kv): a box lands as [group][row][64]
    const uint64_t dims[4] = {64ull, (uint64_t)m, (uint64_t)p.ncg, (uint64_t)H_kv};
    const uint64_t str[3] = {(uint64_t)n * 2, 128ull, (uint64_t)m * n * 2};
    const uint32_t box[4] = {64u, (uint32_t)(16 * p.JC), (uint32_t)p.ncg, 1u};
    if (!encode_tensor_map_bf16(&tm[4], a.theta, 4, dims, str, box)) return cudaSuccess;
    if (!encode_tensor_map_bf16(&tm[5], a.U, 4, dims, str, box)) return cudaSuccess;
  }
  *encoded = true;

  FusedArgs fa{};
  fa.q = static_cast<const __nv_bfloat16*>(a.q);
  fa.mu = static_cast<const __nv_bfloat16*>(a.mu);
  fa.out = static_cast<__nv_bfloat16*>(a.out);
  fa.B = B; fa.H_kv = H_kv; fa.G = a.G; fa.R = R; fa.m = m; fa.n = n; fa.T = a.T;
  fa.NB = p.NB; fa.RB = p.RB; fa.nbg = p.nbg; fa.nrg = p.nrg; fa.units = p.units; fa.JC = p.JC; fa.NJ = p.NJ;
  fa.TCH = p.TCH; fa.ncg = p.ncg; fa.stages = p.stages;
  fa.Tper = (ceil_div(a.T > 0 ? a.T : 1, p.nrg) + 15) & ~15;
  fa.par_bytes = p.par_bytes; fa.k_half_bytes = p.k_half_bytes; fa.txt_half_bytes = p.txt_half_bytes;
  fa.stage_bytes = p.stage_bytes;
  const uint32_t ring = (uint32_t)p.stages * p.stage_bytes;
  fa.off_q = ring + p.off_q; fa.off_S = ring + p.off_S; fa.off_W = ring + p.off_W; fa.off_wred = ring + p.off_wred;
  fa.off_rstat = ring + p.off_rstat; fa.off_tstat = ring + p.off_tstat; fa.off_hstat = ring + p.off_hstat;
  fa.off_yred = ring + p.off_yred;
  fa.part_y = a.fpart_y;
  fa.part_ml = a.fpart_ml;
  fa.cnt = L->d_cnt;
  fa.status = a.status;

  ProfScope prof(KVC_KERNEL_FUSED, st);
  const bool nh2 = a.G > 8;
  if (p.ncg <= 4) return nh2 ? launch_inst<1, 4, 2>(tm, fa, p, st) : launch_inst<1, 4, 1>(tm, fa, p, st);
  if (p.ncg <= 9) return nh2 ? launch_inst<1, 9, 2>(tm, fa, p, st) : launch_inst<1, 9, 1>(tm, fa, p, st);
  return nh2 ? launch_inst<1, 16, 2>(tm, fa, p, st) : launch_inst<1, 16, 1>(tm, fa, p, st);
}

}  // namespace kvc
