// Algorithm 1 as ONE kernel for bf16 storage: compressed scores, expansion by theta, joint softmax with
// the text logits, re-projection by U^T, product with the compressed values, mu term, normalisation.
//
// Work unit = one KV head h, NB sequences and RB vision blocks of each (NB*RB*G <= 16 expansion rows),
// plus a slice of the sequences' text rows.  A persistent CTA streams, per unit, through a ring of large
// shared-memory stages filled by the TMA engine (tiled tensor maps, 128-byte swizzle).  A stage of pass A holds
// rows [16 JC c, 16 JC (c+1)) of K_tilde of every block of the unit and the same rows of theta[h] (all n
// columns); a stage of pass C holds the same rows of V_tilde and of U[h]; a text stage holds TCH rows of K_txt
// and V_txt per sequence.  theta/U rows (L2-resident, shared by all sequences) and capsule rows (HBM) thus
// arrive interleaved and both streams stay busy for the whole unit.
//
// The consumer warps are specialised, and the two groups run one stage apart instead of meeting at a barrier:
//   value warps      pass A: S_c = sigma q K_c^T (bf16 tile in shared memory)           -> expansion warps
//                    text:   online-softmax attention over their own 16-row tiles
//                    pass C: y^T += V_c^T W_c^T                                          <- expansion warps
//   expansion warps  pass A: L += S_c theta_c, logits in registers (rows x n, fp32), each warp a column range
//                    softmax: P = 2^(L - max), one maximum per (sequence, head) over the unit's blocks and text
//                    pass C: W_c = P U_c^T, split over the column ranges and reduced through shared memory
// All matrix products run on mma.sync m16n8k16; the products with value rows are taken transposed (head
// dimension as M, heads as N) so that a group of up to 8 heads costs one 8-wide tile.  A unit that holds every
// block of its sequences writes `out` directly; otherwise the units of a (sequence, KV head) leave
// (max, sum, y) partials and the last one to arrive merges them.
#include <mutex>
#include <new>

#include "kvc_fused.cuh"

namespace kvc {

// EW expansion warps, VW value warps, one producer warp.  Every expansion warp owns up to KTW 16-column groups of
// the logits; NH = 8-head tiles of the group (1: G <= 8, 2: G <= 16); MT = 16-row tiles of expansion rows per unit
template <int EW, int VW, int KTW, int NH, int MT>
__global__ void __launch_bounds__((EW + VW + 1) * 32, 1)
fused_decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const __grid_constant__ CUtensorMap tmKt, const __grid_constant__ CUtensorMap tmVt,
                    const __grid_constant__ CUtensorMap tmTh, const __grid_constant__ CUtensorMap tmU,
                    const FusedArgs a) {
  constexpr int CW = EW + VW;                 // consumer warps
  constexpr int FCONS = CW * 32;
  constexpr int FTHREADS = FCONS + 32;
  constexpr int RT = ROWS * MT;               // expansion rows of a unit
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* sm = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
  __shared__ __align__(8) FusedBars bars;
  __shared__ int s_last;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < a.stages; ++s) { mbar_init(&bars.full[s], 1); mbar_init(&bars.empty[s], CW); }
    fence_mbar_init();
  }
  // score and weight tiles start as zeros: their padding rows and columns are read by the MMAs
  {
    uint32_t* z = reinterpret_cast<uint32_t*>(sm + a.off_S);
    const int words = (2 * RT * a.sld + 2 * (RT + 16) * SLD) / 2;
    for (int i = tid; i < words; i += FTHREADS) z[i] = 0u;
  }
  __syncthreads();

  const int per_h = a.nbg * a.nrg;

  if (warp == CW) {
    // ================= producer: one thread feeds the ring =================
    // It walks the stage sequence of this CTA's units: per unit NJ stages of pass A, the text stages, NJ stages
    // of pass C.  A slot is refilled as soon as every consumer warp has released it.
    if (lane != 0) return;
    tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmTh); tma_prefetch_desc(&tmU);
    if (a.T > 0) { tma_prefetch_desc(&tmKt); tma_prefetch_desc(&tmVt); }
    bool first = true;
    uint32_t slot = 0, phase = 1;              // parity to wait for on the empty barrier: 1 passes on a fresh barrier
    for (int u = blockIdx.x; u < a.units; u += gridDim.x) {
      const int h = u / per_h, rem = u - h * per_h;
      const int bg = rem / a.nrg, rg = rem - bg * a.nrg;
      const int b0 = bg * a.NB, r0 = rg * a.RB;
      const RowRanges tr = row_ranges(a, rg);
      const int nts = tr.na + tr.nb;
      if (first && a.R > 0) {
        // while the stream's previous kernel drains: the K_tilde rows of the first ring of stages are asked into L2 (a
        // prefetch consumes no data, so it need not wait for that kernel; the loads below do)
        for (int c = 0; c < a.NJ && c < a.stages; ++c) {
          tma_prefetch_l2_5d(&tmK, 0, c * 16 * a.JC, r0, h, b0);
          tma_prefetch_l2_5d(&tmK, 64, c * 16 * a.JC, r0, h, b0);
        }
      }
      for (int part = 0; part < 3; ++part) {
        const int count = part == 1 ? nts : a.NJ;
        for (int c = 0; c < count; ++c) {
          if (!mbar_wait_bounded(&bars.empty[slot], phase)) { atomicExch(a.status, (int)KVC_ERR_TIMEOUT); return; }
          unsigned char* dst = sm + slot * a.stage_bytes;
          uint64_t* bar = &bars.full[slot];
          if (part == 1) {
            const bool lead = c < tr.na;
            const int y = lead ? tr.a0 + c * a.TCH : tr.b0 + (c - tr.na) * a.TCH;
            const CUtensorMap* mk = lead ? &tmK : &tmKt;
            const CUtensorMap* mv = lead ? &tmV : &tmVt;
            mbar_expect_tx(bar, 4 * a.txt_half_bytes);
            if (first) { grid_dep_wait(); first = false; }
            tma_load_4d(dst, mk, 0, y, h, b0, bar);
            tma_load_4d(dst + a.txt_half_bytes, mk, 64, y, h, b0, bar);
            tma_load_4d(dst + 2 * a.txt_half_bytes, mv, 0, y, h, b0, bar);
            tma_load_4d(dst + 3 * a.txt_half_bytes, mv, 64, y, h, b0, bar);
          } else {
            const CUtensorMap* tp = part == 0 ? &tmTh : &tmU;
            const CUtensorMap* tk = part == 0 ? &tmK : &tmV;
            const int j0 = c * 16 * a.JC;
            mbar_expect_tx(bar, a.par_bytes + 2 * a.k_half_bytes);
            tma_load_4d(dst, tp, 0, j0, 0, h, bar);                  // parameters: never written by this library
            if (first && !a.early) { grid_dep_wait(); first = false; }   // the capsule rows: late unless known to be settled
            tma_load_5d(dst + a.par_bytes, tk, 0, j0, r0, h, b0, bar);
            tma_load_5d(dst + a.par_bytes + a.k_half_bytes, tk, 64, j0, r0, h, b0, bar);
          }
          if (++slot == (uint32_t)a.stages) { slot = 0; phase ^= 1u; }
        }
      }
    }
    return;
  }

  // ================= consumers: common set-up =================
  const int gid = lane >> 2, t4 = lane & 3;
  const int G = a.G, RB = a.RB, JC = a.JC;
  const int rows16 = 16 * JC;                      // rows of one block inside a stage
  const int sld = a.sld;
  const uint32_t sm_u = smem_addr(sm);
  const uint32_t q_u = sm_u + a.off_q, S_u = sm_u + a.off_S, W_u = sm_u + a.off_W;
  __nv_bfloat16* q_sm = reinterpret_cast<__nv_bfloat16*>(sm + a.off_q);
  __nv_bfloat16* S_sm = reinterpret_cast<__nv_bfloat16*>(sm + a.off_S);      // [2][RT][sld]
  __nv_bfloat16* W_sm = reinterpret_cast<__nv_bfloat16*>(sm + a.off_W);      // [2][RT + 16][SLD]
  float* wred = reinterpret_cast<float*>(sm + a.off_wred);                   // [2][EW][RT][16]
  float* rmax = reinterpret_cast<float*>(sm + a.off_rstat);                  // [EW][RT]
  float* rsum = rmax + EW * RT;
  float* tmax = reinterpret_cast<float*>(sm + a.off_tstat);                  // [VW][16]
  float* tsum = tmax + VW * 16;
  float* hmax = reinterpret_cast<float*>(sm + a.off_hstat);                  // [NB][16]
  float* hsum = hmax + a.NB * 16;
  float* vsum = hsum + a.NB * 16;
  float* hvmax = vsum + a.NB * 16;                                           // maximum over the vision logits only
  float* hfv = hvmax + a.NB * 16;                                            // 2^(hvmax - hmax): moves the vision weights to the joint maximum
  float* rowf = hfv + a.NB * 16;                                             // [RT] that factor per expansion row
  float* yred = reinterpret_cast<float*>(sm + a.off_yred);                   // [VW][yhg][D]
  const float qscale = 0.08838834764831845f * 1.4426950408889634f;   // sigma = 1/sqrt(128), logits kept in log2 units
  const int l7 = lane & 7;
  const int lrow = l7 + ((lane >> 3) & 1) * 8;     // ldmatrix address pattern A: rows 0-15 by lanes 0-15, twice
  const int lhi = lane >> 4;
  const int lrowB = l7 + lhi * 8;                  // address pattern B: rows 0-7 | 0-7 | 8-15 | 8-15
  const int lmid = (lane >> 3) & 1;
  const int WPG = VW / a.NB;                       // value warps per sequence of the unit

  if (warp >= EW && blockIdx.x < a.units) {
    // the queries of the first unit: into L2 (and the TLB) before the wait, read after it
    const int u = blockIdx.x, h = u / per_h, rem = u - h * per_h, b0 = (rem / a.nrg) * a.NB;
    const int vt = tid - EW * 32;
    if (vt < a.NB * 32) {
      const int tb = vt >> 5, g = (vt >> 1) & 15, half = vt & 1;     // 128-byte halves of a 256-byte query row
      if (b0 + tb < a.B && g < a.G) prefetch_l2(a.q + ((size_t)(b0 + tb) * a.H_kv * a.G + (size_t)h * a.G + g) * D + half * 64);
    }
  }
  grid_dep_wait();
  grid_dep_launch();
  if (blockIdx.x == 0 && tid == 0) *a.status = 0;

  uint32_t slot = 0, phase = 0;
  uint32_t si = 0, wi = 0;                         // score tiles and weight tiles handed over so far (buffer = count & 1)
  bool dead = false;
  // every lane of the calling warp waits; the lanes leave the polling loop together again before any warp-wide instruction
  auto wait_on = [&](uint64_t* bar, uint32_t parity) {
    if (!dead && !mbar_wait_bounded(bar, parity)) dead = true;
    __syncwarp();
  };
  // the stage in `slot` has been consumed by this warp
  auto release = [&]() {
    __syncwarp();
    if (lane == 0) mbar_arrive(&bars.empty[slot]);
    if (++slot == (uint32_t)a.stages) { slot = 0; phase ^= 1u; }
  };

  if (warp < EW) {
    // ======================================================================================================
    // expansion warps: L += S theta, softmax, W = P U^T
    // ======================================================================================================
    const int ETH = EW * 32;
    const int KT = a.n >> 4;
    const int kt0 = warp * a.ktw;
    const int my_kt = max(0, min(a.ktw, KT - kt0));
    // byte offsets of this warp's fragments inside a parameter tile [column group][row][64]
    uint32_t th_off[KTW], u_off[KTW];              // theta: [k = row][n = col] read transposed;  U: [n = row][k = col]
#pragma unroll
    for (int kt = 0; kt < KTW; ++kt) {
      const int ktc = kt < my_kt ? kt0 + kt : 0;
      const int col_t = ktc * 16 + lhi * 8, col_u = ktc * 16 + lmid * 8;
      th_off[kt] = (uint32_t)(((col_t >> 6) * rows16 + lrow) * 128 + ((((col_t & 63) >> 3) ^ l7) << 4));
      u_off[kt] = (uint32_t)(((col_u >> 6) * rows16 + lrowB) * 128 + ((((col_u & 63) >> 3) ^ l7) << 4));
    }

    for (int u = blockIdx.x; u < a.units; u += gridDim.x) {
      const int h = u / per_h, rem = u - h * per_h;
      const int bg = rem / a.nrg, rg = rem - bg * a.nrg;
      const int b0 = bg * a.NB, r0 = rg * a.RB;
      const int nbv = min(a.NB, a.B - b0);
      const int rbv = min(RB, a.R - r0);
      const RowRanges tr = row_ranges(a, rg);
      const int nts = tr.na + tr.nb;
      (void)h;

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
          rvalid[mt][hr] = rho < a.NB * RB * G && rbl < nbv && rrl < rbv;
          rhead[mt][hr] = rvalid[mt][hr] ? rbl * 16 + g : 0;
        }

      float accL[MT][2 * KTW][4];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < 2 * KTW; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) accL[mt][nt][e] = 0.f;

      // ---------------- pass A: L[:, my column groups] += S theta ----------------
      for (int c = 0; c < a.NJ; ++c) {
        wait_on(&bars.full[slot], phase);
        const uint32_t par_u = sm_u + slot * a.stage_bytes;
        const int nsub = min(JC, (a.m - c * rows16 + 15) >> 4);          // 16-row sub-chunks with rows below m
        const uint32_t sbuf = si & 1u;
        named_barrier_sync(BAR_S_READY + (int)sbuf, FCONS);
        for (int s = 0; s < nsub; ++s) {
          uint32_t as[MT][4];
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
            ldsm_x4(as[mt], S_u + (uint32_t)((sbuf * (RT * sld) + (mt * 16 + lrow) * sld + s * 16 + lhi * 8) * 2));
#pragma unroll
          for (int kq = 0; kq < KTW; kq += 4) {                 // fragments of 4 column groups in flight at a time
            uint32_t bf[4][4];
#pragma unroll
            for (int x = 0; x < 4; ++x)
              if (kq + x < KTW && kq + x < my_kt) ldsm_x4_t(bf[x], par_u + th_off[(kq + x < KTW) ? kq + x : 0] + (uint32_t)(s * 2048));
#pragma unroll
            for (int x = 0; x < 4; ++x)
              if (kq + x < KTW && kq + x < my_kt) {
                const int kt = (kq + x < KTW) ? kq + x : 0;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                  mma_bf16_16816(accL[mt][2 * kt], as[mt], bf[x][0], bf[x][1]);
                  mma_bf16_16816(accL[mt][2 * kt + 1], as[mt], bf[x][2], bf[x][3]);
                }
              }
          }
        }
        named_barrier_arrive(BAR_S_FREE + (int)sbuf, FCONS);
        ++si;
        release();
      }
      // ---------------- the text stages belong to the value warps: this warp only hands their slots back, as they
      // fill, between the steps of the softmax below (a look at the barrier, no wait, until the last step) ----------------
      int ts_done = 0;
      auto pass_text = [&](bool block) {
        while (ts_done < nts) {
          if (block) {
            wait_on(&bars.full[slot], phase);
          } else {
            int ok = 0;
            if (lane == 0) ok = mbar_test_wait(&bars.full[slot], phase) ? 1 : 0;
            if (!__shfl_sync(0xffffffffu, ok, 0)) break;
          }
          release();
          ++ts_done;
        }
      };

      // ---------------- softmax of the vision logits relative to the vision-only maximum, while the value warps attend
      // the text rows; the text rows' maxima and sums join afterwards through one factor per (sequence, head) ----------------
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int hr = 0; hr < 2; ++hr) {
          float mx = -INFINITY;
#pragma unroll
          for (int nt = 0; nt < 2 * KTW; ++nt)
            if (nt < 2 * my_kt) mx = fmaxf(mx, fmaxf(accL[mt][nt][2 * hr], accL[mt][nt][2 * hr + 1]));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
          if (t4 == 0) rmax[warp * RT + mt * 16 + gid + 8 * hr] = rvalid[mt][hr] ? mx : -INFINITY;
        }
      pass_text(false);
      named_barrier_sync(2, ETH);                                     // row maxima of every expansion warp
      if (warp == 0) {
        // maximum of every expansion row over the warps, then of every (sequence, head) over its blocks
        for (int x = lane; x < RT; x += 32) {
          float mx = -INFINITY;
#pragma unroll
          for (int w = 0; w < EW; ++w) mx = fmaxf(mx, rmax[w * RT + x]);
          rmax[x] = mx;
        }
        __syncwarp();
        for (int x = lane; x < a.NB * 16; x += 32) {
          const int tb = x >> 4, g = x & 15;
          float mx = 0.f;
          if (g < G && tb < nbv) {
            mx = -INFINITY;
            for (int rl = 0; rl < rbv; ++rl) mx = fmaxf(mx, rmax[(tb * RB + rl) * G + g]);
          }
          hvmax[x] = mx;
        }
      }
      pass_text(false);
      named_barrier_sync(2, ETH);                                     // vision maxima per (sequence, head)
      uint32_t pf[MT][KTW][4];                        // P (bf16) of this warp's column groups, as MMA operand fragments
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
        for (int hr = 0; hr < 2; ++hr) {
          const bool ok = rvalid[mt][hr];
          const float M = hvmax[rhead[mt][hr]];
          float sum = 0.f;
#pragma unroll
          for (int nt = 0; nt < 2 * KTW; ++nt)
#pragma unroll
            for (int k = 0; k < 2; ++k) {
              const float p = (ok && nt < 2 * my_kt) ? fast_exp2(accL[mt][nt][2 * hr + k] - M) : 0.f;
              accL[mt][nt][2 * hr + k] = p;
              sum += p;
            }
          sum += __shfl_xor_sync(0xffffffffu, sum, 1);
          sum += __shfl_xor_sync(0xffffffffu, sum, 2);
          if (t4 == 0) rsum[warp * RT + mt * 16 + gid + 8 * hr] = sum;
        }
#pragma unroll
        for (int kt = 0; kt < KTW; ++kt) {
          pf[mt][kt][0] = pack2_bf16(accL[mt][2 * kt][0], accL[mt][2 * kt][1]);
          pf[mt][kt][1] = pack2_bf16(accL[mt][2 * kt][2], accL[mt][2 * kt][3]);
          pf[mt][kt][2] = pack2_bf16(accL[mt][2 * kt + 1][0], accL[mt][2 * kt + 1][1]);
          pf[mt][kt][3] = pack2_bf16(accL[mt][2 * kt + 1][2], accL[mt][2 * kt + 1][3]);
        }
      }
      pass_text(false);
      named_barrier_sync(2, ETH);                                     // row sums of every expansion warp
      if (warp == 0) {
        for (int x = lane; x < RT; x += 32) {
          float sm_ = 0.f;
#pragma unroll
          for (int w = 0; w < EW; ++w) sm_ += rsum[w * RT + x];
          rsum[x] = sm_;
        }
      }
      pass_text(true);
      named_barrier_sync(1, FCONS);                                   // B1: the text maxima are in place
      if (warp == 0) {
        // joint maximum of every (sequence, head) and the factor that moves its vision weights to it
        for (int x = lane; x < a.NB * 16; x += 32) {
          const int tb = x >> 4, g = x & 15;
          float mx = 0.f, f = 0.f;
          if (g < G && tb < nbv) {
            mx = hvmax[x];
            for (int w = tb * WPG; w < (tb + 1) * WPG; ++w) mx = fmaxf(mx, tmax[w * 16 + g]);
            f = fast_exp2(hvmax[x] - mx);
          }
          hmax[x] = mx;
          hfv[x] = f;
        }
      }
      named_barrier_sync(1, FCONS);                                   // B2: head maxima
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int hr = 0; hr < 2; ++hr)
          if (warp == 0 && t4 == 0) rowf[mt * 16 + gid + 8 * hr] = rvalid[mt][hr] ? hfv[rhead[mt][hr]] : 0.f;
      named_barrier_sync(1, FCONS);                                   // B3: text sums are in place
      if (warp == 0) {
        for (int x = lane; x < a.NB * 16; x += 32) {
          const int tb = x >> 4, g = x & 15;
          float vs = 0.f, tsm = 0.f;
          if (g < G && tb < nbv) {
            for (int rl = 0; rl < rbv; ++rl) vs += rsum[(tb * RB + rl) * G + g];
            vs *= hfv[x];
            for (int w = tb * WPG; w < (tb + 1) * WPG; ++w) tsm += tsum[w * 16 + g];
          }
          vsum[x] = vs;
          hsum[x] = vs + tsm;
        }
      }
      named_barrier_sync(1, FCONS);                                   // B4: head sums

      // ---------------- pass C: W = P U^T, reduced over the expansion warps ----------------
      for (int c = 0; c < a.NJ; ++c) {
        wait_on(&bars.full[slot], phase);
        const uint32_t par_u = sm_u + slot * a.stage_bytes;
        const int nsub = min(JC, (a.m - c * rows16 + 15) >> 4);
        for (int s = 0; s < nsub; ++s) {
          float wc[MT][2][4];
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
              for (int e = 0; e < 4; ++e) wc[mt][nt][e] = 0.f;
#pragma unroll
          for (int kq = 0; kq < KTW; kq += 4) {
            uint32_t bu[4][4];
#pragma unroll
            for (int x = 0; x < 4; ++x)
              if (kq + x < KTW && kq + x < my_kt) ldsm_x4(bu[x], par_u + u_off[(kq + x < KTW) ? kq + x : 0] + (uint32_t)(s * 2048));
#pragma unroll
            for (int x = 0; x < 4; ++x)
              if (kq + x < KTW && kq + x < my_kt) {
                const int kt = (kq + x < KTW) ? kq + x : 0;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                  mma_bf16_16816(wc[mt][0], pf[mt][kt], bu[x][0], bu[x][1]);
                  mma_bf16_16816(wc[mt][1], pf[mt][kt], bu[x][2], bu[x][3]);
                }
              }
          }
          const uint32_t wbuf = wi & 1u;
          float* wr = wred + (wbuf * EW + warp) * (RT * 16);
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
              for (int hr = 0; hr < 2; ++hr)
                *reinterpret_cast<float2*>(&wr[(mt * 16 + gid + 8 * hr) * 16 + nt * 8 + 2 * t4]) =
                    make_float2(wc[mt][nt][2 * hr], wc[mt][nt][2 * hr + 1]);
          named_barrier_sync(2, ETH);
          if (wi >= 2) named_barrier_sync(BAR_W_FREE + (int)wbuf, FCONS);   // the value warps are done with this buffer's previous tile
          for (int idx = tid; idx < RT * 16; idx += ETH) {
            const float* wp = wred + wbuf * EW * (RT * 16) + idx;
            float w = 0.f;
#pragma unroll
            for (int x = 0; x < EW; ++x) w += wp[x * RT * 16];
            W_sm[wbuf * ((RT + 16) * SLD) + (idx >> 4) * SLD + (idx & 15)] = __float2bfloat16_rn(w * rowf[idx >> 4]);
          }
          named_barrier_arrive(BAR_W_READY + (int)wbuf, FCONS);
          ++wi;
        }
        release();
      }
    }
  } else {
    // ======================================================================================================
    // value warps: scores, text attention, y^T += V^T W^T, output
    // ======================================================================================================
    const int VTH = VW * 32;
    const int vw = warp - EW, vtid = tid - EW * 32;
    const int bl = vw / WPG, wig = vw - bl * WPG;
    const int msplit = a.msplit, mshift = a.mshift;           // a task covers the row tiles mt with (mt >> mshift) == its group

    for (int u = blockIdx.x; u < a.units; u += gridDim.x) {
      const int h = u / per_h, rem = u - h * per_h;
      const int bg = rem / a.nrg, rg = rem - bg * a.nrg;
      const int b0 = bg * a.NB, r0 = rg * a.RB;
      const int nbv = min(a.NB, a.B - b0);
      const int rbv = min(RB, a.R - r0);
      const RowRanges tr = row_ranges(a, rg);
      const int nts = tr.na + tr.nb;

      // ---- queries of the unit's sequences: [NB][16 heads][128], heads >= G and absent sequences are zero rows
      for (int idx = vtid; idx < a.NB * 256; idx += VTH) {
        const int tb = idx >> 8, g = (idx >> 4) & 15, piece = idx & 15;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (tb < nbv && g < G)
          v = *reinterpret_cast<const uint4*>(a.q + ((size_t)(b0 + tb) * a.H_kv * G + (size_t)h * G + g) * D + piece * 8);
        *reinterpret_cast<uint4*>(q_sm + (tb * 16 + g) * QLD + piece * 8) = v;
      }
      named_barrier_sync(3, VTH);
      uint32_t qf[NH][8][2];                          // B operand of the score MMA: heads of sequence bl
#pragma unroll
      for (int nh = 0; nh < NH; ++nh)
#pragma unroll
        for (int k2 = 0; k2 < 4; ++k2) {
          uint32_t r[4];
          ldsm_x4(r, q_u + (uint32_t)(((bl * 16 + nh * 8 + l7) * QLD + k2 * 32 + (lane >> 3) * 8) * 2));
          qf[nh][2 * k2][0] = r[0]; qf[nh][2 * k2][1] = r[1];
          qf[nh][2 * k2 + 1][0] = r[2]; qf[nh][2 * k2 + 1][1] = r[3];
        }

      // ---------------- pass A: S[rows of block][16] = sigma q K^T for my (block, sub-chunk) tasks ----------------
      for (int c = 0; c < a.NJ; ++c) {
        wait_on(&bars.full[slot], phase);
        const uint32_t k_u = sm_u + slot * a.stage_bytes + a.par_bytes;
        const int nsub = min(JC, (a.m - c * rows16 + 15) >> 4);
        const uint32_t sbuf = si & 1u;
        if (si >= 2) named_barrier_sync(BAR_S_FREE + (int)sbuf, FCONS);   // the expansion warps are done with this buffer's previous tile
        __nv_bfloat16* Sb = S_sm + sbuf * (RT * sld);
        for (int task = wig; task < RB * nsub; task += WPG) {
          const int rl = nsub == 1 ? task : task / nsub, s = task - rl * nsub;
          const int bi = bl * RB + rl;
          const uint32_t rowoff = k_u + (uint32_t)((bi * rows16 + s * 16 + lrow) * 128);
          uint32_t af[8][4];
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            ldsm_x4(af[ks], rowoff + (ks >> 2) * a.k_half_bytes + (uint32_t)(((((ks & 3) * 2 + lhi)) ^ l7) << 4));
          float sc[NH][2][4];
#pragma unroll
          for (int nh = 0; nh < NH; ++nh)
#pragma unroll
            for (int x = 0; x < 2; ++x)
#pragma unroll
              for (int e = 0; e < 4; ++e) sc[nh][x][e] = 0.f;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
#pragma unroll
            for (int nh = 0; nh < NH; ++nh) mma_bf16_16816(sc[nh][ks & 1], af[ks], qf[nh][ks][0], qf[nh][ks][1]);
#pragma unroll
          for (int nh = 0; nh < NH; ++nh)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int head = nh * 8 + 2 * t4 + (e & 1), j = gid + (e >> 1) * 8;
              if (head < G) Sb[(bi * G + head) * sld + s * 16 + j] = __float2bfloat16_rn((sc[nh][0][e] + sc[nh][1][e]) * qscale);
            }
        }
        named_barrier_arrive(BAR_S_READY + (int)sbuf, FCONS);
        ++si;
        release();
      }

      // ---------------- text rows: online-softmax attention per warp ----------------
      // yacc[mt][nh]: y^T tile, rows = head-dimension mt*16 + gid (+8), columns = heads nh*8 + 2*t4 (+1) of sequence bl
      float yacc[8][NH][4];
#pragma unroll
      for (int mt = 0; mt < 8; ++mt)
#pragma unroll
        for (int nh = 0; nh < NH; ++nh)
#pragma unroll
          for (int e = 0; e < 4; ++e) yacc[mt][nh][e] = 0.f;
      float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};   // heads gid and gid + 8
      for (int ts = 0; ts < nts; ++ts) {
        wait_on(&bars.full[slot], phase);
        const uint32_t kt_u = sm_u + slot * a.stage_bytes, vt_u = kt_u + 2 * a.txt_half_bytes;
        for (int tile = wig; tile * 16 < a.TCH; tile += WPG) {
          const int ts1 = ts < tr.na ? tr.a1 : tr.b1;               // end of the row range this stage belongs to
          const int t_first = (ts < tr.na ? tr.a0 + ts * a.TCH : tr.b0 + (ts - tr.na) * a.TCH) + tile * 16;
          if (t_first >= ts1) break;
          const int row0 = bl * a.TCH + tile * 16;
          const uint32_t rowB = (uint32_t)((row0 + lrowB) * 128);
          // logits [16 heads][16 text rows] = q K_txt^T
          float cc[2][4];
          {
            float c2[2][2][4];                       // two accumulation chains per tile column
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
                ldsm_x4(bk[x], kt_u + kh * a.txt_half_bytes + rowB + (uint32_t)((((x * 2 + lmid)) ^ l7) << 4));
                ldsm_x4(aq[x], q_u + (uint32_t)(((bl * 16 + lrow) * QLD + ks * 16 + lhi * 8) * 2));
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
          // cc[nt][e]: head gid + 8*(e>>1), text row t_first + nt*8 + 2*t4 + (e&1)
#pragma unroll
          for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int t = t_first + nt * 8 + 2 * t4 + (e & 1);
              cc[nt][e] = t < ts1 ? cc[nt][e] * qscale : -INFINITY;
            }
          float scl[2];
#pragma unroll
          for (int hr = 0; hr < 2; ++hr) {
            float mx = fmaxf(fmaxf(cc[0][2 * hr], cc[0][2 * hr + 1]), fmaxf(cc[1][2 * hr], cc[1][2 * hr + 1]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run[hr], mx);              // finite: the tile has at least one valid row
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
          uint32_t av[8][4];
#pragma unroll
          for (int mt = 0; mt < 8; ++mt)
            ldsm_x4_t(av[mt], vt_u + (mt >> 2) * a.txt_half_bytes + rowB + (uint32_t)(((((mt & 3) * 2 + lmid)) ^ l7) << 4));
#pragma unroll
          for (int mt = 0; mt < 8; ++mt)
#pragma unroll
            for (int nh = 0; nh < NH; ++nh) mma_bf16_16816(yacc[mt][nh], av[mt], pb[nh][0], pb[nh][1]);
        }
        release();
      }

      // ---------------- joint softmax: the text accumulators move to the unit's reference maximum ----------------
      if (t4 == 0) { tmax[vw * 16 + gid] = m_run[0]; tmax[vw * 16 + gid + 8] = m_run[1]; }
      named_barrier_sync(1, FCONS);                                   // B1
      named_barrier_sync(1, FCONS);                                   // B2: head maxima
      {
        float scl[2];
#pragma unroll
        for (int hr = 0; hr < 2; ++hr) {
          const int head = gid + 8 * hr;
          const float M = hmax[bl * 16 + head];
          scl[hr] = m_run[hr] == -INFINITY ? 0.f : fast_exp2(m_run[hr] - M);
          float l = l_run[hr] * scl[hr];
          l += __shfl_xor_sync(0xffffffffu, l, 1);
          l += __shfl_xor_sync(0xffffffffu, l, 2);
          if (t4 == 0) tsum[vw * 16 + head] = l;
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
      named_barrier_sync(1, FCONS);                                   // B3
      named_barrier_sync(1, FCONS);                                   // B4: head sums

      // ---------------- pass C: y^T[128][heads] += V^T[128][16 rows of block] W^T[16][heads of block] ----------------
      for (int c = 0; c < a.NJ; ++c) {
        wait_on(&bars.full[slot], phase);
        const uint32_t v_u = sm_u + slot * a.stage_bytes + a.par_bytes;
        const int nsub = min(JC, (a.m - c * rows16 + 15) >> 4);
        for (int s = 0; s < nsub; ++s) {
          const uint32_t wbuf = wi & 1u;
          named_barrier_sync(BAR_W_READY + (int)wbuf, FCONS);
          for (int task = wig; task < RB * msplit; task += WPG) {          // my (block, row-tile group) tasks
            const int rl = task >> (3 - mshift), mg = task & (msplit - 1);
            if (rl >= rbv || bl >= nbv) continue;
            const int bi = bl * RB + rl;
            uint32_t bw[4];
            ldsm_x4(bw, W_u + (uint32_t)((wbuf * ((RT + 16) * SLD) + (bi * G + lrowB) * SLD + lmid * 8) * 2));
            const uint32_t rowoff = v_u + (uint32_t)((bi * rows16 + s * 16 + lrowB) * 128);
            uint32_t av[8][4];
#pragma unroll
            for (int mt = 0; mt < 8; ++mt)
              if ((mt >> mshift) == mg)
                ldsm_x4_t(av[mt], rowoff + (mt >> 2) * a.k_half_bytes + (uint32_t)(((((mt & 3) * 2 + lmid)) ^ l7) << 4));
#pragma unroll
            for (int mt = 0; mt < 8; ++mt)
              if ((mt >> mshift) == mg) {
#pragma unroll
                for (int nh = 0; nh < NH; ++nh) mma_bf16_16816(yacc[mt][nh], av[mt], bw[2 * nh], bw[2 * nh + 1]);
              }
          }
          named_barrier_arrive(BAR_W_FREE + (int)wbuf, FCONS);
          ++wi;
        }
        release();
      }

      // ---------------- unit end: reduce over the value warps, mu term, normalise or leave a partial ----------------
      const int bh = b0 * a.H_kv + h;                    // used when the block axis is split (NB == 1)
      const size_t pbase = ((size_t)bh * a.nrg + rg) * G;
      const int YHG = a.yhg;
      for (int g0 = 0; g0 < G; g0 += YHG) {
        // every warp parks its tile columns of heads g0 .. g0+YHG-1; then the warps of a sequence are summed
#pragma unroll
        for (int nh = 0; nh < NH; ++nh)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int head = nh * 8 + 2 * t4 + e;
            if (head >= g0 && head < g0 + YHG && head < G) {
              float* yp = yred + (vw * YHG + (head - g0)) * D;
#pragma unroll
              for (int mt = 0; mt < 8; ++mt) {
                yp[mt * 16 + gid] = yacc[mt][nh][e];
                yp[mt * 16 + gid + 8] = yacc[mt][nh][2 + e];
              }
            }
          }
        named_barrier_sync(3, VTH);
        const int hg = min(YHG, G - g0);
        for (int idx = vtid; idx < nbv * hg * D; idx += VTH) {
          const int col = idx & (D - 1), gg = (idx >> 7) % hg, tb = idx / (D * hg);
          const int g = g0 + gg;
          float y = 0.f;
          for (int w = tb * WPG; w < (tb + 1) * WPG; ++w) y += yred[(w * YHG + gg) * D + col];
          if (a.R > 0) y = fmaf(vsum[tb * 16 + g], __bfloat162float(a.mu[h * D + col]), y);
          if (a.nrg == 1)
            a.out[((size_t)(b0 + tb) * a.H_kv * G + (size_t)h * G + g) * D + col] = __float2bfloat16_rn(y / hsum[tb * 16 + g]);
          else
            a.part_y[(pbase + g) * D + col] = y;
        }
        named_barrier_sync(3, VTH);
      }
      if (a.nrg > 1) {
        // one sequence, several units along the block axis: the last unit to arrive merges the partials
        if (vtid < G) a.part_ml[pbase + vtid] = make_float2(hmax[vtid], hsum[vtid]);
        __threadfence();
        named_barrier_sync(3, VTH);
        if (vtid == 0) {
          s_last = arrive_is_last(&a.cnt[bh], a.token, a.nrg) ? 1 : 0;
        }
        named_barrier_sync(3, VTH);
        if (s_last) {
          __threadfence();
          const size_t p0 = (size_t)bh * a.nrg * G;
          // weights of the partials, w[p][g] = 2^(max_p - max) / sum: first all (max, sum) pairs into shared memory
          float* mlm = yred;                              // [nrg*G] maxima, then [nrg*G] sums, then [nrg*G] weights
          const int npg = a.nrg * G;
          const bool in_smem = 3 * npg <= VW * YHG * D;
          if (in_smem) {
            for (int idx = vtid; idx < npg; idx += VTH) {
              const float2 ml = __ldcg(&a.part_ml[p0 + idx]);
              mlm[idx] = ml.x;
              mlm[npg + idx] = ml.y;
            }
            named_barrier_sync(3, VTH);
            if (vtid < G) {
              float M = -INFINITY, den = 0.f;
              for (int p = 0; p < a.nrg; ++p) M = fmaxf(M, mlm[p * G + vtid]);
              for (int p = 0; p < a.nrg; ++p) den = fmaf(fast_exp2(mlm[p * G + vtid] - M), mlm[npg + p * G + vtid], den);
              const float inv = 1.f / den;
              for (int p = 0; p < a.nrg; ++p) mlm[2 * npg + p * G + vtid] = fast_exp2(mlm[p * G + vtid] - M) * inv;
            }
            named_barrier_sync(3, VTH);
            // four output columns per thread, up to eight partials' loads in flight: the merge is a chain of L2 round trips
            for (int idx = vtid; idx < G * (D / 4); idx += VTH) {
              const int g = idx >> 5, col = (idx & 31) * 4;
              const float* yp = a.part_y + (p0 + g) * D + col;
              const float* wp = mlm + 2 * npg + g;
              float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
              auto acc = [&](const float4& y, float w) {
                num.x = fmaf(w, y.x, num.x); num.y = fmaf(w, y.y, num.y); num.z = fmaf(w, y.z, num.z); num.w = fmaf(w, y.w, num.w);
              };
              int p = 0;
              for (; p + 8 <= a.nrg; p += 8) {
                float4 y[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) y[k] = __ldcg(reinterpret_cast<const float4*>(yp + (size_t)(p + k) * G * D));
#pragma unroll
                for (int k = 0; k < 8; ++k) acc(y[k], wp[(p + k) * G]);
              }
              for (; p + 4 <= a.nrg; p += 4) {
                float4 y[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) y[k] = __ldcg(reinterpret_cast<const float4*>(yp + (size_t)(p + k) * G * D));
#pragma unroll
                for (int k = 0; k < 4; ++k) acc(y[k], wp[(p + k) * G]);
              }
              for (; p < a.nrg; ++p) acc(__ldcg(reinterpret_cast<const float4*>(yp + (size_t)p * G * D)), wp[p * G]);
              uint2 o;
              o.x = pack2_bf16(num.x, num.y); o.y = pack2_bf16(num.z, num.w);
              *reinterpret_cast<uint2*>(a.out + ((size_t)b0 * a.H_kv * G + (size_t)h * G + g) * D + col) = o;
            }
          } else {
            for (int idx = vtid; idx < G * D; idx += VTH) {
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
        named_barrier_sync(3, VTH);
      }
    }
  }
  if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
}

}  // namespace kvc

// The tensor maps over the capsule store and the parameters depend only on (B, R, capsule pointer, box shape), not on
// the text length: a decode loop re-encodes them for the same few stores again and again, so a handle keeps the last few.
struct kvc_map_cache {
  struct Entry {
    bool valid;
    int B, R, tc, JC, RB, NB;
    const void* Kc;
    CUtensorMap tm[4];          // K_tilde, V_tilde, theta, U
  };
  std::mutex mu;
  Entry e[8];
  int next;
};

namespace kvc {

kvc_map_cache* map_cache_create() {
  kvc_map_cache* c = new (std::nothrow) kvc_map_cache();
  if (c) { for (auto& x : c->e) x.valid = false; c->next = 0; }
  return c;
}
void map_cache_destroy(kvc_map_cache* c) { delete c; }

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
                            const uint64_t* strides_bytes, const uint32_t* box, bool swizzle128) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t gd[5], gs[4];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) { gd[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) gs[i] = strides_bytes[i];
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gd, gs, bx, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// expansion and value warps for a block length n (the 16-column groups of the logits are dealt to the expansion warps)
static void warp_split(int n, int* ew, int* vw, int* ktw_max) {
  const int KT = n / 16;
  if (KT <= 16) { *ew = 4; *vw = 8; *ktw_max = 4; }          // n <= 256
  else if (KT <= 40) { *ew = 5; *vw = 10; *ktw_max = 8; }    // n <= 640 (24 x 24 grids: 576): the value warps carry most of the work
  else { *ew = 11; *vw = 4; *ktw_max = 6; }                  // n <= 1024: the expansion dominates
}

FusedPlan plan_fused(const kvc_layer* L, int B, int R) {
  if (L->use_tc == -2) return FusedPlan{};      // the three-phase kernels were asked for
  if (L->use_tc >= 0 && L->use_tc != 3) {
    // The tensor-memory variant pays per tcgen05.mma, not per expansion row: it wins for long blocks once two row
    // tiles per unit still give most SMs a unit (measured on the n = 1024, G = 7 shape: ahead from batch 16 on,
    // behind at batches 1-4 where units of half the size halve the latency).
    if (L->use_tc != 1) {
      // pairs of CTAs per (sequence, KV head): ahead of the single-CTA variant on the n = 1024, G = 7 shape from batch 16 on
      // when a sequence has more expansion rows than one CTA's two row tiles (8 blocks: 122 vs 154 us at batch 32; with 2
      // blocks the 64-row unit is mostly padding: 105 vs 45 us)
      const FusedPlan t2 = plan_fused_pair(L, B, R);
      if (t2.ok && (L->use_tc == 2 || (L->desc.n > 640 && R * L->G > 32 && t2.units >= 96))) return t2;
    }
    const FusedPlan t = plan_fused_tc(L, B, R);
    if (t.ok && (L->use_tc > 0 || (L->desc.n > 640 && t.MT == 2 && t.units >= 96))) return t;
  }
  FusedPlan p{};
  const int G = L->G, n = L->desc.n, m = L->m, H_kv = L->desc.H_kv;
  if (L->desc.dtype != KVC_BF16 || L->passthrough || R < 1 || B < 1 || n % 64 != 0 || n > 1024 || G > 16) return p;
  if (reinterpret_cast<uintptr_t>(L->desc.theta) & 15 || reinterpret_cast<uintptr_t>(L->desc.U) & 15) return p;
  const int sms = L->num_sms > 0 ? L->num_sms : 148;
  int ktw_max = 0;
  warp_split(n, &p.EW, &p.VW, &ktw_max);
  p.ktw = ceil_div(n / 16, p.EW);
  // two row tiles per unit when the logits of both still fit the expansion warps' registers (n <= 256)
  p.MT = (n <= 256 && G * R > ROWS) ? 2 : 1;
  const int cap = ROWS * p.MT;
  p.RB = R < cap / G ? R : cap / G;
  p.NB = 1;
  if (p.RB == R) {
    // whole sequences per unit: more sequences per unit share one pass over theta[h] and U[h]
    double best = 0;
    for (int nb = 1; nb <= 4; nb *= 2) {
      if (nb > 1 && (nb * R * G > cap || nb > B || p.VW % nb != 0)) break;
      const long long units = (long long)H_kv * ceil_div(B, nb);
      const double cost = (double)ceil_div((int)units, sms) * ((double)nb * R * m * 512.0 + 4.0 * m * n);
      if (nb == 1 || cost < best) { best = cost; p.NB = nb; }
    }
  }
  p.nbg = ceil_div(B, p.NB);
  p.nrg = ceil_div(R, p.RB);
  p.units = H_kv * p.nbg * p.nrg;
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
  {
    // the 8 row tiles of a value block go to `msplit` tasks so that the warps of a sequence share the work evenly
    const int wpg = p.VW / p.NB;
    int best = 1 << 30;
    for (int sh = 3; sh >= 0; --sh) {            // sh = 3: one task per block
      const int ms = 8 >> sh, cost = ceil_div(p.RB * ms, wpg) * ((1 << sh) + 1);
      if (cost < best) { best = cost; p.msplit = ms; p.mshift = sh; }
    }
  }
  p.sld = 16 * p.JC + 8;
  uint32_t off = 0;
  auto take = [&](uint32_t bytes) { uint32_t o = off; off = (off + bytes + 127u) & ~127u; return o; };
  p.off_q = take((uint32_t)p.NB * 16 * QLD * 2);
  const int rt = ROWS * p.MT;
  p.off_S = take((uint32_t)(2 * rt * p.sld + 2 * (rt + 16) * SLD) * 2);
  p.off_W = p.off_S + (uint32_t)2 * rt * p.sld * 2;
  p.off_wred = take((uint32_t)2 * p.EW * rt * 16 * 4);
  p.off_rstat = take((uint32_t)2 * p.EW * rt * 4);
  p.off_tstat = take((uint32_t)2 * p.VW * 16 * 4);
  p.off_hstat = take((uint32_t)(5 * p.NB * 16 + rt) * 4);
  p.yhg = G > 4 ? 8 : (G > 2 ? 4 : 2);
  p.off_yred = take((uint32_t)p.VW * p.yhg * D * 4);
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

// Text-only attention (no vision blocks: the uncompressed comparator and R == 0 calls) through the same kernel:
// only text stages, the rows of a (sequence, KV head) cut into `nrg` slices whose partials are merged.
FusedPlan plan_fused_text(const kvc_layer* L, int B, int T) {   // T = all plain rows (leading segment + text)
  FusedPlan p{};
  const int G = L->G, H_kv = L->desc.H_kv;
  if (L->desc.dtype != KVC_BF16 || B < 1 || T < 1 || G > 16) return p;
  const int sms = L->num_sms > 0 ? L->num_sms : 148;
  p.EW = 4; p.VW = 8; p.ktw = 0; p.MT = 1;
  p.NB = 1; p.RB = 1; p.nbg = B;
  // slices: enough units for every SM, cut so that the persistent CTAs are evenly loaded, slices of >= 256 rows
  const long long bh = (long long)B * H_kv;
  int best_ns = 1;
  double best_eff = 0;
  for (int ns = 1; ns <= 16; ++ns) {
    if (ns > 1 && T / ns < 256) break;
    const long long units = bh * ns;
    const long long grid = units < sms ? units : sms;
    const double eff = (double)units / (double)(((units + grid - 1) / grid) * sms);
    if (eff > best_eff + 0.02) { best_eff = eff; best_ns = ns; }
  }
  p.nrg = best_ns;
  p.units = (int)(bh * p.nrg);
  p.ncg = 1; p.JC = 1; p.NJ = 0;
  p.TCH = 128;
  p.par_bytes = 0; p.k_half_bytes = 0;
  p.txt_half_bytes = (uint32_t)p.TCH * 128u;
  p.stage_bytes = 4 * p.txt_half_bytes;
  p.msplit = 1; p.mshift = 3;
  p.sld = 24;
  uint32_t off = 0;
  auto take = [&](uint32_t bytes) { uint32_t o = off; off = (off + bytes + 127u) & ~127u; return o; };
  p.off_q = take((uint32_t)p.NB * 16 * QLD * 2);
  const int rt = ROWS * p.MT;
  p.off_S = take((uint32_t)(2 * rt * p.sld + 2 * (rt + 16) * SLD) * 2);
  p.off_W = p.off_S + (uint32_t)2 * rt * p.sld * 2;
  p.off_wred = take((uint32_t)2 * p.EW * rt * 16 * 4);
  p.off_rstat = take((uint32_t)2 * p.EW * rt * 4);
  p.off_tstat = take((uint32_t)2 * p.VW * 16 * 4);
  p.off_hstat = take((uint32_t)(5 * p.NB * 16 + rt) * 4);
  p.yhg = G > 4 ? 8 : (G > 2 ? 4 : 2);
  p.off_yred = take((uint32_t)p.VW * p.yhg * D * 4);
  p.misc_bytes = off;
  const uint32_t avail = SMEM_LIMIT - 1024u - 2048u - p.misc_bytes;
  p.stages = (int)(avail / p.stage_bytes) > 3 ? 3 : (int)(avail / p.stage_bytes);
  if (p.stages < 2) return p;
  p.smem_bytes = (size_t)p.stages * p.stage_bytes + p.misc_bytes + 1024u;
  p.grid = p.units < sms ? p.units : sms;
  p.ok = 1;
  return p;
}

template <int EW, int VW, int KTW, int NH, int MT>
static cudaError_t launch_inst(const CUtensorMap* tm, const FusedArgs& fa, const FusedPlan& p, cudaStream_t st) {
  {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(fused_decode_kernel<EW, VW, KTW, NH, MT>), p.smem_bytes);
    if (e != cudaSuccess) return e;
  }
  return launch_dependent(fused_decode_kernel<EW, VW, KTW, NH, MT>, dim3(p.grid), dim3((EW + VW + 1) * 32), p.smem_bytes, st, tm[0],
                          tm[1], tm[2], tm[3], tm[4], tm[5], fa);
}

template <int NH>
static cudaError_t launch_nh(const CUtensorMap* tm, const FusedArgs& fa, const FusedPlan& p, cudaStream_t st) {
  if (p.EW == 4) return p.MT == 2 ? launch_inst<4, 8, 4, NH, 2>(tm, fa, p, st) : launch_inst<4, 8, 4, NH, 1>(tm, fa, p, st);
  if (p.EW == 5) return launch_inst<5, 10, 8, NH, 1>(tm, fa, p, st);
  return launch_inst<11, 4, 6, NH, 1>(tm, fa, p, st);
}

cudaError_t launch_fused(const kvc_layer* L, const DecodeArgs& a, const FusedPlan& p, cudaStream_t st, bool* encoded) {
  const int H_kv = a.H_kv, m = a.m, n = a.n, R = a.R, B = a.B;
  CUtensorMap tm[6];
  *encoded = false;
  const bool compressed = R > 0 && !a.passthrough;
  bool cached = false;
  if (compressed && L->maps) {
    std::lock_guard<std::mutex> lock(L->maps->mu);
    for (const auto& x : L->maps->e)
      if (x.valid && x.B == B && x.R == R && x.tc == p.tc && x.JC == p.JC && x.RB == p.RB && x.NB == p.NB && x.Kc == a.Kc) {
        tm[0] = x.tm[0]; tm[1] = x.tm[1]; tm[4] = x.tm[2]; tm[5] = x.tm[3];
        cached = true;
        break;
      }
  }
  if (compressed && !cached) {
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
  const int S0 = (R > 0 && a.passthrough) ? R * n : 0;   // rho = 0: the store holds K and V verbatim, attended as plain rows
  if (S0 > 0) {
    const uint64_t dims[4] = {(uint64_t)D, (uint64_t)S0, (uint64_t)H_kv, (uint64_t)B};
    const uint64_t str[3] = {256ull, (uint64_t)S0 * 256, (uint64_t)H_kv * S0 * 256};
    const uint32_t box[4] = {64u, (uint32_t)p.TCH, 1u, (uint32_t)p.NB};
    if (!encode_tensor_map_bf16(&tm[0], a.Kc, 4, dims, str, box)) return cudaSuccess;
    if (!encode_tensor_map_bf16(&tm[1], a.Vc, 4, dims, str, box)) return cudaSuccess;
    if (a.T == 0) { tm[2] = tm[0]; tm[3] = tm[1]; }
    tm[4] = tm[0]; tm[5] = tm[1];
  } else if (R == 0) {
    tm[0] = tm[2]; tm[1] = tm[3]; tm[4] = tm[2]; tm[5] = tm[3];          // never used: no vision stages
  } else if (!cached) {
    // theta, U [H_kv][m][n] viewed as (64 columns, m rows, n/64 column groups, H_kv): a box lands as [group][row][64]
    const uint64_t dims[4] = {64ull, (uint64_t)m, (uint64_t)p.ncg, (uint64_t)H_kv};
    const uint64_t str[3] = {(uint64_t)n * 2, 128ull, (uint64_t)m * n * 2};
    const uint32_t box[4] = {64u, (uint32_t)(16 * p.JC), (uint32_t)(p.tc == 2 ? p.ncg / 2 : p.ncg), 1u};
    const uint32_t box_tc[4] = {64u, 128u, 1u, 1u};     // tensor-memory variant: U by 64-column groups, 128 rows at a time
    if (!encode_tensor_map_bf16(&tm[4], a.theta, 4, dims, str, box)) return cudaSuccess;
    if (!encode_tensor_map_bf16(&tm[5], a.U, 4, dims, str, p.tc ? box_tc : box)) return cudaSuccess;
    if (L->maps) {
      std::lock_guard<std::mutex> lock(L->maps->mu);
      auto& x = L->maps->e[L->maps->next];
      L->maps->next = (L->maps->next + 1) % 8;
      x.B = B; x.R = R; x.tc = p.tc; x.JC = p.JC; x.RB = p.RB; x.NB = p.NB; x.Kc = a.Kc;
      x.tm[0] = tm[0]; x.tm[1] = tm[1]; x.tm[2] = tm[4]; x.tm[3] = tm[5];
      x.valid = true;
    }
  }
  *encoded = true;

  FusedArgs fa{};
  fa.q = static_cast<const __nv_bfloat16*>(a.q);
  fa.mu = static_cast<const __nv_bfloat16*>(a.mu);
  fa.out = static_cast<__nv_bfloat16*>(a.out);
  const bool plain = R == 0 || a.passthrough;            // text-only mode
  fa.B = B; fa.H_kv = H_kv; fa.G = a.G; fa.R = plain ? 0 : R; fa.m = plain ? 1 : m; fa.n = plain ? 64 : n; fa.T = a.T;
  fa.S0 = S0;
  fa.NB = p.NB; fa.RB = p.RB; fa.nbg = p.nbg; fa.nrg = p.nrg; fa.units = p.units; fa.JC = p.JC; fa.NJ = p.NJ;
  fa.TCH = p.TCH; fa.ncg = p.ncg; fa.stages = p.stages;
  fa.ktw = p.ktw; fa.msplit = p.msplit; fa.mshift = p.mshift; fa.sld = p.sld; fa.yhg = p.yhg;
  fa.Tper = (ceil_div(S0 + a.T > 0 ? S0 + a.T : 1, p.nrg) + 15) & ~15;
  fa.par_bytes = p.par_bytes; fa.k_half_bytes = p.k_half_bytes; fa.txt_half_bytes = p.txt_half_bytes;
  fa.stage_bytes = p.stage_bytes;
  const uint32_t ring = (uint32_t)p.stages * p.stage_bytes;
  fa.off_q = ring + p.off_q; fa.off_S = ring + p.off_S; fa.off_W = ring + p.off_W; fa.off_wred = ring + p.off_wred;
  fa.off_rstat = ring + p.off_rstat; fa.off_tstat = ring + p.off_tstat; fa.off_hstat = ring + p.off_hstat;
  fa.off_yred = ring + p.off_yred;
  fa.off_P = ring + p.off_P; fa.off_rtab = ring + p.off_rtab; fa.tmem_cols = p.tmem_cols; fa.UT = p.UT; fa.nu = p.nu;
  fa.off_xstat = ring + p.off_xstat; fa.off_wrecv = ring + p.off_wrecv;
  fa.part_y = a.fpart_y;
  fa.part_ml = a.fpart_ml;
  fa.cnt = a.fcnt;
  fa.token = a.token;
  fa.status = a.status;
  fa.early = a.early_capsules;

  ProfScope prof(p.tc == 2 ? KVC_KERNEL_FUSED_PAIR : (p.tc ? KVC_KERNEL_FUSED_TC : KVC_KERNEL_FUSED), st);
  if (p.tc) return launch_fused_tc_kernel(tm, fa, p, st);
  return a.G > 8 ? launch_nh<2>(tm, fa, p, st) : launch_nh<1>(tm, fa, p, st);
}

}  // namespace kvc
