// Algorithm 1 as one kernel for bf16 storage, with the two expansions on the 5th-generation tensor cores:
//   L^T[n x rows] += theta_c^T[n x 16] S_c^T[16 x rows]   (Alg. 1 step 2; logits accumulate in tensor memory)
//   W^T[m x rows]  = U[m x n] P^T[n x rows]                (Alg. 1 step 3, re-projection of the probabilities)
// `rows` = the expansion rows of a work unit (sequence, block, head) = the N dimension of both products; the large
// dimensions (n for the logits, m for the weights) are the M dimension of tcgen05.mma, in tiles of 128, and the
// operand tiles are read exactly as the TMA engine lays them down (128-byte swizzle): theta_c as an MN-major A
// operand, 128-row tiles of a 64-column group of U as a K-major A operand.  Work units and the ring are those of
// kvc_fused.cu; the stage sequence of a unit is: pass A (theta rows + K_tilde rows), then the column groups of U
// interleaved with the text stages, then the V_tilde stages.  Warp roles:
//   warps 0-3        softmax of the vision logits read back from tensor memory (one lane per column of L^T), relative
//                    to the vision-only maximum; P as a bf16 operand in shared memory; when W^T is complete they move
//                    it to the weight tiles, scaled to the joint maximum of vision and text rows
//   value warps      S_c = sigma q K_c^T (mma.sync; bf16 tile in shared memory in UMMA core-matrix order), text rows
//                    flash-style, y^T += V_c^T W_c^T, unit end: reduction, mu term, output or partial + merge
//   MMA warp         one thread issues every tcgen05.mma and commits completion to the mbarriers that free the
//                    stage, the score tile and the accumulators
//   producer warp    one thread feeds the ring through tensor maps
//
// Measured on B200: one tcgen05.mma of K = 16 occupies the tensor pipe for about 129 cycles at M = 128 and about 85
// at M = 64 whatever N <= 128 is (one row of A per cycle, A from shared or tensor memory alike).  The cost of a unit
// is therefore (n/128) (m/16) + (m/128) (n/16) MMAs whatever its number of expansion rows: the variant pays off
// for long blocks with as many rows per unit as the grid allows (see plan_fused in kvc_fused.cu).
#include "kvc_fused.cuh"
#include "kvc_tcgen05.cuh"

namespace kvc {

constexpr int BAR_P_READY = 12;                // probabilities written (warps 0-3 arrive, the MMA warp waits)
constexpr int BAR_END = 13;                    // every tensor-memory user is done: the MMA warp may free it

// Order of the stages between pass A and the V_tilde stages: `nu` stages of U (tensor core) and `nts` text stages
// (value warps).  The first TEXT_LEAD text stages go first, because the re-projection cannot start before the softmax
// is done; after that the two kinds alternate.  (iu, it) = stages of either kind issued so far.
constexpr int TEXT_LEAD = 3;
__device__ __forceinline__ bool next_is_text(int iu, int it, int nu, int nts) {
  return it < nts && (it < TEXT_LEAD || iu >= nu || it - TEXT_LEAD < iu);
}

struct TcBars {
  uint64_t full[FMAX_STAGES], empty[FMAX_STAGES];
  uint64_t s_free[2];      // the MMAs that read score tile b have completed
  uint64_t w_done;         // W^T of the unit is complete
  uint64_t l_done;         // the logits of the unit are complete
  uint64_t l_free;         // the logits of the unit have been read back (4 warps)
  uint64_t x_data;         // pair mode: the peer's statistics and partial weights of the unit have landed here
  uint64_t x_ready;        // pair mode: the peer's re-projection of the unit is complete: its weight tiles may be written
  uint64_t m_data;         // pair mode, CTA 0: the peer's partial output of the unit has landed here
};

// Reduces 16 per-lane values over the 32 lanes of a warp (maximum or sum) in 31 shuffles: after the first exchange
// every step halves the rows a lane keeps; lane l (and l + 16) returns the total of row l & 15.
template <bool IS_MAX>
__device__ __forceinline__ float lane_reduce16(float (&x)[16], int lane) {
  auto op = [](float p, float q) { return IS_MAX ? fmaxf(p, q) : p + q; };
#pragma unroll
  for (int r = 0; r < 16; ++r) x[r] = op(x[r], __shfl_xor_sync(0xffffffffu, x[r], 16));
  float y8[8], y4[4], y2[2];
  const bool u8 = lane & 8, u4 = lane & 4, u2 = lane & 2, u1 = lane & 1;
#pragma unroll
  for (int k = 0; k < 8; ++k) y8[k] = op(u8 ? x[8 + k] : x[k], __shfl_xor_sync(0xffffffffu, u8 ? x[k] : x[8 + k], 8));
#pragma unroll
  for (int k = 0; k < 4; ++k) y4[k] = op(u4 ? y8[4 + k] : y8[k], __shfl_xor_sync(0xffffffffu, u4 ? y8[k] : y8[4 + k], 4));
#pragma unroll
  for (int k = 0; k < 2; ++k) y2[k] = op(u2 ? y4[2 + k] : y4[k], __shfl_xor_sync(0xffffffffu, u2 ? y4[k] : y4[2 + k], 2));
  return op(u1 ? y2[1] : y2[0], __shfl_xor_sync(0xffffffffu, u1 ? y2[0] : y2[1], 1));
}

// EW = 4 or 8 softmax / conversion warps (warps 0 .. EW-1: one or two per tensor-memory lane quarter), VW value warps
// PAIR: the two CTAs of a cluster share a (sequence, KV head): both compute the scores of all its blocks, CTA c keeps
// the logits and the partial weights of columns [c n/2, (c+1) n/2) (its half of theta and U), the partial weights of the
// other CTA's half of the m rows are sent to it through distributed shared memory, and each CTA multiplies its half of
// the V_tilde rows (and attends its half of the text rows); the two outputs are merged like those of any split sequence.
template <int EW, int VW, int NH, int MT, bool PAIR>
__global__ void __launch_bounds__((EW + VW + 2) * 32, 1)
fused_decode_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                       const __grid_constant__ CUtensorMap tmKt, const __grid_constant__ CUtensorMap tmVt,
                       const __grid_constant__ CUtensorMap tmTh, const __grid_constant__ CUtensorMap tmU,
                       const FusedArgs a) {
  constexpr int TEW = EW;
  constexpr int TSTEP = EW / 4;               // the tiles of a lane quarter are dealt to its TSTEP warps
  constexpr int CW = TEW + VW;                // warps that meet at the softmax barriers
  constexpr int FCONS = CW * 32;
  constexpr int MMA_WARP = CW, PROD_WARP = CW + 1;
  constexpr int FTHREADS = (CW + 2) * 32;
  constexpr int RT = ROWS * MT;               // expansion rows of a unit = N of the expansion MMAs
  constexpr int SREADY = VW * 32 + 32;        // value warps arrive, the MMA warp waits
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* sm = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
  __shared__ __align__(8) TcBars bars;
  __shared__ int s_last;
  __shared__ uint32_t s_tmem;
  __shared__ float2 s_mlpeer[8];            // pair mode, CTA 0: (maximum, sum) of the peer's partial output per head

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < a.stages; ++s) { mbar_init(&bars.full[s], 1); mbar_init(&bars.empty[s], VW + 1); }
    for (int b = 0; b < 2; ++b) mbar_init(&bars.s_free[b], 1);
    mbar_init(&bars.w_done, 1);
    mbar_init(&bars.l_done, 1);
    mbar_init(&bars.l_free, TEW);
    mbar_init(&bars.x_data, 1);
    mbar_init(&bars.x_ready, 1);
    mbar_init(&bars.m_data, 1);
    fence_mbar_init();
  }
  if (warp == MMA_WARP) tmem_alloc(&s_tmem, (uint32_t)a.tmem_cols);
  const int JC = a.JC;
  const uint32_t s_buf_bytes = (uint32_t)(JC * RT * 32);            // score tile buffer: [JC][2 halves][RT/8][8][8]
  // score tiles start as zeros: the rows of absent (sequence, block, head) triples are read by the MMAs
  {
    uint32_t* z = reinterpret_cast<uint32_t*>(sm + a.off_S);
    const int words = (int)(2 * s_buf_bytes) / 4;
    for (int i = tid; i < words; i += FTHREADS) z[i] = 0u;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if constexpr (PAIR) cluster_sync_all();      // the peer's barriers exist before anything is sent to them
  const uint32_t tb = s_tmem;                  // tensor memory: L^T tiles at columns [0, NT*RT), W^T tiles after them
  const int ncgl = PAIR ? a.ncg >> 1 : a.ncg;  // 64-column groups of theta / U this CTA works on
  const int NT = PAIR ? a.n >> 8 : (a.n + 127) >> 7;
  const int NJ0 = PAIR ? (a.NJ + 1) >> 1 : a.NJ;   // pair mode: CTA 0 takes the first NJ0 stages of the m axis in the value pass
  const int MTL = (a.m + 127) >> 7;            // 128-row tiles of W^T (rows of U)
  const uint32_t w_col = (uint32_t)(NT * RT);
  // W^T tiles beyond the allocated columns take the columns of L^T, whose logits are dead once P is in shared memory
  // (long retained lengths in pair mode: 4 + 4 tiles of 64 columns fill the 512, tiles 4.. of W^T overlay L^T)
  const int wown = (a.tmem_cols - NT * RT) / RT;
  const bool overlay = MTL > wown;
  auto wcol = [&](int t) -> uint32_t { return t < wown ? w_col + (uint32_t)(t * RT) : (uint32_t)((t - wown) * RT); };
  const bool w_tail64 = a.m - 128 * (MTL - 1) <= 64;   // the last tile of W^T holds at most 64 rows of U: M = 64
  const int ugroups = (MTL + a.UT - 1) / a.UT; // stages per 64-column group of U: UT row tiles each

  const int per_h = a.nbg * a.nrg;
  const int rows16 = 16 * JC;                      // rows of one block inside a stage
  const uint32_t sm_u = smem_addr(sm);

  if (warp == PROD_WARP) {
    // ================= producer: one thread feeds the ring =================
    if (lane != 0) { if constexpr (PAIR) cluster_exit_sync(); return; }
    tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmTh); tma_prefetch_desc(&tmU);
    if (a.T > 0) { tma_prefetch_desc(&tmKt); tma_prefetch_desc(&tmVt); }
    bool first = true;
    uint32_t slot = 0, phase = 1;              // parity to wait for on the empty barrier: 1 passes on a fresh barrier
    for (int u = blockIdx.x; u < a.units; u += gridDim.x) {
      const int h = u / per_h, rem = u - h * per_h;
      const int bg = rem / a.nrg, rg = rem - bg * a.nrg;
      // pair mode: the units 2k, 2k+1 of a (sequence, head) are the two CTAs (rank rk) of a cluster on block group k
      const int rk = PAIR ? (rg & 1) : 0;
      const int b0 = bg * a.NB, r0 = PAIR ? (rg >> 1) * a.RB : rg * a.RB;
      const RowRanges tr = row_ranges(a, rg);
      const int nts = tr.na + tr.nb;
      const int cg0 = PAIR ? rk * ncgl : 0;          // first column group of this CTA
      const int c2first = (PAIR && rk) ? NJ0 : 0, c2count = PAIR ? (rk ? a.NJ - NJ0 : NJ0) : a.NJ;
      // stage sequence of a unit: NJ stages of pass A (theta rows + K_tilde rows); then the column groups of U and
      // the text stages, interleaved so that the tensor core (U) and the value warps (text) both have work; then
      // NJ stages of V_tilde rows
      for (int part = 0; part < 3; ++part) {
        const int count = part == 1 ? a.nu + nts : (part == 0 ? a.NJ : c2count);
        int iu = 0, it = 0;
        for (int cc = 0; cc < count; ++cc) {
          const bool is_text = part == 1 && next_is_text(iu, it, a.nu, nts);
          const int c = part == 1 ? (is_text ? it++ : iu++) : cc;
          if (!mbar_wait_bounded(&bars.empty[slot], phase)) {
            atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
            if constexpr (PAIR) cluster_exit_sync();
            return;
          }
          unsigned char* dst = sm + slot * a.stage_bytes;
          uint64_t* bar = &bars.full[slot];
          if (is_text) {
            const int y = tr.b0 + c * a.TCH;
            mbar_expect_tx(bar, 4 * a.txt_half_bytes);
            tma_load_4d(dst, &tmKt, 0, y, h, b0, bar);
            tma_load_4d(dst + a.txt_half_bytes, &tmKt, 64, y, h, b0, bar);
            tma_load_4d(dst + 2 * a.txt_half_bytes, &tmVt, 0, y, h, b0, bar);
            tma_load_4d(dst + 3 * a.txt_half_bytes, &tmVt, 64, y, h, b0, bar);
          } else if (part == 1) {
            // 64 columns of U[h], row tiles [t0, t0 + nt_) of 128 rows each (rows past m are zero-filled)
            const int cg = c / ugroups, t0 = (c - cg * ugroups) * a.UT;
            const int nt_ = min(a.UT, MTL - t0);
            mbar_expect_tx(bar, (uint32_t)nt_ * 16384u);
            for (int t = 0; t < nt_; ++t) tma_load_4d(dst + t * 16384, &tmU, 0, (t0 + t) * 128, cg0 + cg, h, bar);
          } else if (part == 0) {
            const int j0 = c * rows16;
            mbar_expect_tx(bar, a.par_bytes + 2 * a.k_half_bytes);
            tma_load_4d(dst, &tmTh, 0, j0, cg0, h, bar);             // parameters: never written by this library
            if (first) { grid_dep_wait(); first = false; }            // everything else may come from the stream's previous kernel
            tma_load_5d(dst + a.par_bytes, &tmK, 0, j0, r0, h, b0, bar);
            tma_load_5d(dst + a.par_bytes + a.k_half_bytes, &tmK, 64, j0, r0, h, b0, bar);
          } else {
            const int j0 = (c2first + c) * rows16;
            mbar_expect_tx(bar, 2 * a.k_half_bytes);
            tma_load_5d(dst + a.par_bytes, &tmV, 0, j0, r0, h, b0, bar);
            tma_load_5d(dst + a.par_bytes + a.k_half_bytes, &tmV, 64, j0, r0, h, b0, bar);
          }
          if (++slot == (uint32_t)a.stages) { slot = 0; phase ^= 1u; }
        }
      }
    }
    if constexpr (PAIR) cluster_exit_sync();
    return;
  }

  grid_dep_wait();
  grid_dep_launch();
  if (blockIdx.x == 0 && tid == 0) *a.status = 0;

  uint32_t slot = 0, phase = 0;
  uint32_t si = 0;                                 // score tiles handed over so far (buffer = si & 1)
  uint32_t ucount = 0;                             // units this CTA has started
  uint32_t vunit = 0;                              // units whose outputs the value warps have merged through the pair (pair mode)
  bool dead = false;
  // every lane of the calling warp waits; the lanes leave the polling loop together again before any warp-wide instruction
  auto wait_on = [&](uint64_t* bar, uint32_t parity) {
    if (!dead && !mbar_wait_bounded(bar, parity)) dead = true;
    __syncwarp();
  };
  auto advance = [&]() { if (++slot == (uint32_t)a.stages) { slot = 0; phase ^= 1u; } };

  if (warp == MMA_WARP) {
    // ======================================================================================================
    // MMA warp: lane 0 issues the expansion MMAs of every stage
    // ======================================================================================================
    const uint32_t S_u = sm_u + a.off_S, P_u = sm_u + a.off_P;
    const uint32_t cg_bytes = (uint32_t)rows16 * 128u;            // one 64-column group of a parameter tile
    const uint32_t idesc_L_full = umma_idesc_bf16(128, RT, 1, 0);
    const uint32_t idesc_L_half = umma_idesc_bf16(64, RT, 1, 0);
    const uint32_t idesc_W = umma_idesc_bf16(128, RT, 0, 0), idesc_W64 = umma_idesc_bf16(64, RT, 0, 0);
    const bool half_tail = !PAIR && (a.n & 127) != 0;             // n = 64 (mod 128): the last tile of L^T has 64 rows
    for (int u = blockIdx.x; u < a.units; u += gridDim.x, ++ucount) {
      const int rem = u % per_h;
      const int rg = rem % a.nrg;
      const RowRanges tr = row_ranges(a, rg);
      const int nts = tr.na + tr.nb;
      // ---------------- pass A ----------------
      if (ucount > 0) wait_on(&bars.l_free, (ucount - 1) & 1u);    // the previous unit's logits have been read back
      for (int c = 0; c < a.NJ; ++c) {
        wait_on(&bars.full[slot], phase);
        const uint32_t sbuf = si & 1u;
        named_barrier_sync(BAR_S_READY + (int)sbuf, SREADY);
        tc_fence_after();
        if (lane == 0) {
          const uint32_t par_u = sm_u + slot * a.stage_bytes;
          const int nsub = min(JC, (a.m - c * rows16 + 15) >> 4);
          for (int s = 0; s < nsub; ++s) {
            const uint64_t bdesc = umma_smem_desc(S_u + sbuf * s_buf_bytes + (uint32_t)(s * RT * 32), (uint32_t)(RT * 16), 128u, UMMA_LAYOUT_NONE);
            for (int t = 0; t < NT; ++t) {
              const uint64_t adesc = umma_smem_desc(par_u + (uint32_t)(2 * t) * cg_bytes + (uint32_t)(s * 2048), cg_bytes, 1024u, UMMA_LAYOUT_SW128);
              umma_bf16(tb + (uint32_t)(t * RT), adesc, bdesc, (half_tail && t == NT - 1) ? idesc_L_half : idesc_L_full, (c | s) ? 1u : 0u);
            }
          }
          umma_commit(&bars.empty[slot]);
          umma_commit(&bars.s_free[sbuf]);
          if (c == a.NJ - 1) umma_commit(&bars.l_done);
        }
        __syncwarp();
        ++si;
        advance();
      }
      // ---------------- W^T[m x rows] = U P^T: one stage = 64 columns of U, UT row tiles; text stages pass by ----------------
      for (int iu = 0, it = 0; iu + it < a.nu + nts;) {
        if (!next_is_text(iu, it, a.nu, nts)) {
          const int i = iu++;
          wait_on(&bars.full[slot], phase);
          if (i == 0) named_barrier_sync(BAR_P_READY, TEW * 32 + 32);    // the probabilities of the unit are in shared memory
          tc_fence_after();
          if (lane == 0) {
            const uint32_t par_u = sm_u + slot * a.stage_bytes;
            const int cg = i / ugroups, t0 = (i - cg * ugroups) * a.UT;
            const int nt_ = min(a.UT, MTL - t0);
            for (int t = 0; t < nt_; ++t)
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) {
                const uint64_t adesc = umma_smem_desc(par_u + (uint32_t)(t * 16384 + kk * 32), 16u, 1024u, UMMA_LAYOUT_SW128);
                const uint64_t bdesc = umma_smem_desc(P_u + (uint32_t)(cg * RT * 128 + kk * 32), 16u, 1024u, UMMA_LAYOUT_SW128);
                umma_bf16(tb + wcol(t0 + t), adesc, bdesc, (w_tail64 && t0 + t == MTL - 1) ? idesc_W64 : idesc_W,
                          (cg | kk) ? 1u : 0u);
              }
            umma_commit(&bars.empty[slot]);
            if (i == a.nu - 1) umma_commit(&bars.w_done);
          }
          __syncwarp();
          advance();
        } else {
          ++it;
          wait_on(&bars.full[slot], phase);
          if (lane == 0) mbar_arrive(&bars.empty[slot]);
          advance();
        }
      }
      // ---------------- the V_tilde stages belong to the value warps ----------------
      const int c2count = PAIR ? ((rg & 1) ? a.NJ - NJ0 : NJ0) : a.NJ;
      for (int c = 0; c < c2count; ++c) {
        wait_on(&bars.full[slot], phase);
        if (lane == 0) mbar_arrive(&bars.empty[slot]);
        advance();
      }
    }
    tc_fence_before();
    named_barrier_sync(BAR_END, (CW + 1) * 32);
    tmem_dealloc(tb, (uint32_t)a.tmem_cols);
    if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
    if constexpr (PAIR) cluster_exit_sync();
    return;
  }

  // ================= softmax / conversion warps and value warps: common set-up =================
  const int gid = lane >> 2, t4 = lane & 3;
  const int G = a.G, RB = a.RB;
  const uint32_t q_u = sm_u + a.off_q, W_u = sm_u + a.off_W;
  __nv_bfloat16* q_sm = reinterpret_cast<__nv_bfloat16*>(sm + a.off_q);
  unsigned char* S_sm = sm + a.off_S;                                        // [2][JC][2][RT/8][8][8] bf16
  __nv_bfloat16* W_sm = reinterpret_cast<__nv_bfloat16*>(sm + a.off_W);      // [ceil(m/16)][RT + 16][SLD]; shares its region with P
  float* rmax = reinterpret_cast<float*>(sm + a.off_rstat);                  // [TEW][RT]
  float* rsum = rmax + TEW * RT;
  float* tmax = reinterpret_cast<float*>(sm + a.off_tstat);                  // [VW][16]
  float* tsum = tmax + VW * 16;
  float* hmax = reinterpret_cast<float*>(sm + a.off_hstat);                  // [NB][16]
  float* hsum = hmax + a.NB * 16;
  float* vsum = hsum + a.NB * 16;
  float* hvmax = vsum + a.NB * 16;                                           // maximum over the vision logits only
  float* hfv = hvmax + a.NB * 16;                                            // 2^(hvmax - hmax): moves the vision weights to the joint maximum
  float* hfp = hfv + a.NB * 16;                                              // pair mode: the same for the peer's partial weights
  float* rowf = hfp + a.NB * 16;                                             // [2][RT] those factors per expansion row
  float* xstat = reinterpret_cast<float*>(sm + a.off_xstat);                 // pair mode, written by the peer: [16] maxima, [RT] row sums
  int* rtab = reinterpret_cast<int*>(sm + a.off_rtab);                       // [RT] head slot of an expansion row, -1 if unused
  float* yred = reinterpret_cast<float*>(sm + a.off_yred);                   // [VW][yhg][D]
  const float qscale = 0.08838834764831845f * 1.4426950408889634f;   // sigma = 1/sqrt(128), logits kept in log2 units
  const int l7 = lane & 7;
  const int lrow = l7 + ((lane >> 3) & 1) * 8;     // ldmatrix address pattern A: rows 0-15 by lanes 0-15, twice
  const int lhi = lane >> 4;
  const int lrowB = l7 + lhi * 8;                  // address pattern B: rows 0-7 | 0-7 | 8-15 | 8-15
  const int lmid = (lane >> 3) & 1;
  const int WPG = VW / a.NB;                       // value warps per sequence of the unit
  // expansion rows of a block: G heads; pair mode pads them to 8 or 16 so that a block's rows start a 16-byte piece of the
  // weight tiles, which it keeps as [row of U][expansion row] (the layout the peer CTA sends and this CTA adds to in place)
  const int GP = PAIR ? (G <= 8 ? 8 : 16) : G;
  constexpr int WLD = RT + 8;                      // pair mode: row stride of the weight tiles in elements

  if (warp < TEW) {
    // ======================================================================================================
    // warps 0-3: joint softmax on the logits in tensor memory, then W^T -> weight tiles
    // ======================================================================================================
    const int wq = warp & 3, wh = warp >> 2;                      // lane quarter; which of the quarter's warps
    const uint32_t tq = tb + ((uint32_t)(wq * 32) << 16);
    const bool half_tail = (a.n & 127) != 0;
    unsigned char* P_sm = sm + a.off_P;                           // [n/64][RT][64] bf16, 128-byte swizzle
    for (int u = blockIdx.x; u < a.units; u += gridDim.x, ++ucount) {
      const int h = u / per_h, rem = u - h * per_h;
      const int bg = rem / a.nrg, rg = rem - bg * a.nrg;
      const int rk = PAIR ? (rg & 1) : 0;           // pair mode: rank in the cluster; block group rg >> 1
      const int b0 = bg * a.NB, r0 = PAIR ? (rg >> 1) * a.RB : rg * a.RB;
      const int nbv = min(a.NB, a.B - b0);
      const int rbv = min(RB, a.R - r0);
      (void)h;
      named_barrier_sync(2, TEW * 32);           // every warp is done with the previous unit's tables
      // expansion row rho <-> (sequence, block, head): head slot of the row, -1 if the unit has no such row
      auto row_slot = [&](int rho) {
        const int bi = rho / GP, g = rho - bi * GP;
        const int rbl = bi / RB, rrl = bi - rbl * RB;
        return (g < G && rho < a.NB * RB * GP && rbl < nbv && rrl < rbv) ? rbl * 16 + g : -1;
      };
      if (warp == 0)
        for (int x = lane; x < RT; x += 32) rtab[x] = row_slot(x);

      // ---------------- maxima of the logits, 16 expansion rows (one tensor-memory load) at a time ----------------
      // (the loops over the 16-row groups are kept rolled: this code runs once per unit, and instruction fetch of the
      // unrolled copies cost more than the loop overhead saves)
      wait_on(&bars.l_done, ucount & 1u);
      tc_fence_after();
#pragma unroll 1
      for (int hh = 0; hh < MT; ++hh) {
        float mx[16];
#pragma unroll
        for (int r = 0; r < 16; ++r) mx[r] = -INFINITY;
        uint32_t nx[16];
        __syncwarp();
        if (wh < NT) tmem_ld_issue_x16(tq + (uint32_t)(wh * RT + hh * 16), nx);
        for (int t = wh; t < NT; t += TSTEP) {
          float v[16];
          tmem_ld_wait_x16(nx);
#pragma unroll
          for (int r = 0; r < 16; ++r) v[r] = __uint_as_float(nx[r]);
          if (t + TSTEP < NT) tmem_ld_issue_x16(tq + (uint32_t)((t + TSTEP) * RT + hh * 16), nx);   // in flight while tile t is reduced
          if (!(half_tail && t == NT - 1) || lane < 16) {
#pragma unroll
            for (int r = 0; r < 16; ++r) mx[r] = fmaxf(mx[r], v[r]);
          }
        }
        const float mine = lane_reduce16<true>(mx, lane);            // row hh*16 + (lane & 15)
        if (lane < 16) rmax[warp * RT + hh * 16 + lane] = row_slot(hh * 16 + lane) >= 0 ? mine : -INFINITY;
      }
      named_barrier_sync(2, TEW * 32);
      if (warp == 0) {
        // maximum of every expansion row over the warps, then of every (sequence, head) over its blocks: the softmax of
        // the vision logits is taken relative to it, the text rows join at the unit's weight hand-over
        for (int x = lane; x < RT; x += 32) {
          float m_ = -INFINITY;
#pragma unroll
          for (int w = 0; w < TEW; ++w) m_ = fmaxf(m_, rmax[w * RT + x]);
          rmax[x] = m_;
        }
        __syncwarp();
        for (int x = lane; x < a.NB * 16; x += 32) {
          const int tb_ = x >> 4, g = x & 15;
          float m_ = 0.f;
          if (g < G && tb_ < nbv) {
            m_ = -INFINITY;
            for (int rl = 0; rl < rbv; ++rl) m_ = fmaxf(m_, rmax[(tb_ * RB + rl) * GP + g]);
          }
          hvmax[x] = m_;
        }
      }
      named_barrier_sync(2, TEW * 32);

      // ---------------- P = 2^(L - max) as the bf16 operand of the re-projection; row sums ----------------
#pragma unroll 1
      for (int hh = 0; hh < MT; ++hh) {
        float Mr[16], sum[16];                        // rows without a (sequence, block, head) get the reference +inf: P = 0
#pragma unroll
        for (int r = 0; r < 16; ++r) {
          const int slot_ = rtab[hh * 16 + r];
          Mr[r] = slot_ >= 0 ? hvmax[slot_] : INFINITY;
          sum[r] = 0.f;
        }
        uint32_t nx[16];
        __syncwarp();
        if (wh < NT) tmem_ld_issue_x16(tq + (uint32_t)(wh * RT + hh * 16), nx);
        for (int t = wh; t < NT; t += TSTEP) {
          float v[16];
          tmem_ld_wait_x16(nx);
#pragma unroll
          for (int r = 0; r < 16; ++r) v[r] = __uint_as_float(nx[r]);
          if (t + TSTEP < NT) tmem_ld_issue_x16(tq + (uint32_t)((t + TSTEP) * RT + hh * 16), nx);   // in flight while tile t is processed
          const bool tail = half_tail && t == NT - 1;
          const bool lane_ok = !tail || lane < 16;
          const int i = t * 128 + (tail ? wq * 16 : wq * 32) + lane;          // column of L = row of L^T
          // element (row, column i) of P: column group i / 64, 128-byte rows, 16-byte pieces XOR-ed with the row modulo 8
          unsigned char* pb = P_sm + (uint32_t)((i >> 6) * (RT * 128) + hh * 2048) + (uint32_t)((i & 7) * 2);
          const uint32_t c8s = (uint32_t)(((i & 63) >> 3) << 4);
          if (lane_ok) {
#pragma unroll
            for (int r = 0; r < 16; ++r) {
              const float p = fast_exp2(v[r] - Mr[r]);
              sum[r] += p;
              *reinterpret_cast<__nv_bfloat16*>(pb + r * 128 + (c8s ^ (uint32_t)((r & 7) << 4))) = __float2bfloat16_rn(p);
            }
          }
        }
        const float mine = lane_reduce16<false>(sum, lane);
        if (lane < 16) rsum[warp * RT + hh * 16 + lane] = mine;
      }
      fence_proxy_async();                                             // P is read by the tensor core (async proxy)
      tc_fence_before();
      __syncwarp();
      if (lane == 0 && !overlay) mbar_arrive(&bars.l_free);          // (with W^T tiles over L^T: after they have been read)
      named_barrier_arrive(BAR_P_READY, TEW * 32 + 32);
      named_barrier_sync(2, TEW * 32);                                // row sums of every warp
      if (warp == 0) {
        for (int x = lane; x < RT; x += 32) {
          float s_ = 0.f;
#pragma unroll
          for (int w = 0; w < TEW; ++w) s_ += rsum[w * RT + x];
          rsum[x] = s_;
        }
      }
      const int NS = (a.m + 15) >> 4;
      // rows of W^T this CTA turns into weight tiles; in pair mode the other rows go to the peer
      const int oj0 = (PAIR && rk) ? NJ0 * rows16 : 0;
      const int oj1 = PAIR ? min(NS * 16, (rk ? a.NJ : NJ0) * rows16) : NS * 16;
      wait_on(&bars.w_done, ucount & 1u);
      tc_fence_after();
      if constexpr (PAIR) {
        // ---- my re-projection is complete and P is dead: the peer may write into my weight tiles (they share P's region);
        // then send: maxima and row sums of my columns, and my partial weights of the peer's rows (bf16), straight into
        // the peer's weight tiles ----
        const uint32_t peer = (uint32_t)rk ^ 1u;
        if (tid == 0) mbar_arrive_cluster(map_to_cta(smem_addr(&bars.x_ready), peer));
        if (!dead && !mbar_wait_cluster_bounded(&bars.x_ready, ucount & 1u)) dead = true;
        __syncwarp();
        if (warp == 0) {
          const uint32_t xs = map_to_cta(smem_addr(xstat), peer);
          for (int x = lane; x < 16; x += 32) st_cluster_f32(xs + 4u * x, hvmax[x]);
          for (int x = lane; x < RT; x += 32) st_cluster_f32(xs + 4u * (16 + x), rsum[x]);
        }
        const int pj0 = rk ? 0 : NJ0 * rows16, pj1 = rk ? min(NS * 16, NJ0 * rows16) : NS * 16;
        const uint32_t wr = map_to_cta(smem_addr(W_sm), peer);
        for (int t = wh; t < MTL; t += TSTEP) {
          const bool t64 = w_tail64 && t == MTL - 1;
          const int j = t * 128 + (t64 ? wq * 16 : wq * 32) + lane;
          const bool mine = j >= pj0 && j < pj1 && (!t64 || lane < 16);
#pragma unroll 1
          for (int hh = 0; hh < MT; ++hh) {
            float v[16];
            __syncwarp();
            tmem_ld_x16(tq + wcol(t) + (uint32_t)(hh * 16), v);
            if (mine) {
              const uint32_t dst = wr + (uint32_t)(((j - pj0) * WLD + hh * 16) * 2);
              st_cluster_v4(dst, pack2_bf16(v[0], v[1]), pack2_bf16(v[2], v[3]), pack2_bf16(v[4], v[5]), pack2_bf16(v[6], v[7]));
              st_cluster_v4(dst + 16u, pack2_bf16(v[8], v[9]), pack2_bf16(v[10], v[11]), pack2_bf16(v[12], v[13]), pack2_bf16(v[14], v[15]));
            }
          }
        }
        named_barrier_sync(2, TEW * 32);                              // every warp has sent
        if (tid == 0) mbar_arrive_cluster(map_to_cta(smem_addr(&bars.x_data), peer));
        if (!dead && !mbar_wait_cluster_bounded(&bars.x_data, ucount & 1u)) dead = true;   // the peer's half has landed
        __syncwarp();
      }
      named_barrier_sync(1, FCONS);                                   // B1: maxima and sums of the text rows from the value warps
      if (warp == 0) {
        for (int x = lane; x < a.NB * 16; x += 32) {
          const int tb_ = x >> 4, g = x & 15;
          float M = 0.f, fo = 0.f, fp = 0.f, vs = 0.f, tsm = 0.f;
          if (g < G && tb_ < nbv) {
            float Mv = hvmax[x];
            if constexpr (PAIR) Mv = fmaxf(Mv, xstat[x]);            // vision maximum over both halves of the columns
            M = Mv;
            for (int w = tb_ * WPG; w < (tb_ + 1) * WPG; ++w) M = fmaxf(M, tmax[w * 16 + g]);
            fo = fast_exp2(hvmax[x] - M);
            for (int rl = 0; rl < rbv; ++rl) vs += rsum[(tb_ * RB + rl) * GP + g];
            vs *= fo;
            if constexpr (PAIR) {
              fp = fast_exp2(xstat[x] - M);
              float vp = 0.f;
              for (int rl = 0; rl < rbv; ++rl) vp += xstat[16 + (tb_ * RB + rl) * GP + g];
              vs = rk ? 0.f : fmaf(vp, fp, vs);                      // the sum of the vision probabilities is counted by CTA 0 alone
            }
            for (int w = tb_ * WPG; w < (tb_ + 1) * WPG; ++w) {
              const float tm_ = tmax[w * 16 + g];
              if (tm_ != -INFINITY) tsm = fmaf(tsum[w * 16 + g], fast_exp2(tm_ - M), tsm);
            }
          }
          hmax[x] = M;
          hfv[x] = fo;
          hfp[x] = fp;
          vsum[x] = vs;
          hsum[x] = vs + tsm;
        }
        __syncwarp();
        for (int x = lane; x < RT; x += 32) {                        // factors of every expansion row
          const int slot_ = rtab[x];
          rowf[x] = slot_ >= 0 ? hfv[slot_] : 0.f;
          rowf[RT + x] = slot_ >= 0 ? hfp[slot_] : 0.f;
        }
      }
      named_barrier_sync(1, FCONS);                                   // B2: joint maxima, sums and the factors

      // ---------------- my rows of W^T from tensor memory to the weight tiles, at the joint maximum ----------------
      for (int t = wh; t < MTL; t += TSTEP) {
        const bool t64 = w_tail64 && t == MTL - 1;                   // a 64-row tile: 16 rows in the first lanes of every quarter
        const int j = t * 128 + (t64 ? wq * 16 : wq * 32) + lane;    // row of U
        const bool mine = j >= oj0 && j < oj1 && (!t64 || lane < 16);
        __nv_bfloat16* wt = W_sm + ((j - oj0) >> 4) * ((RT + 16) * SLD) + (j & 15);      // [expansion row][row of U] tiles
        __nv_bfloat16* wp = W_sm + (j - oj0) * WLD;                                       // pair mode: [row of U][expansion row]
#pragma unroll 1
        for (int hh = 0; hh < MT; ++hh) {
          float v[16];
          __syncwarp();
          tmem_ld_x16(tq + wcol(t) + (uint32_t)(hh * 16), v);
          if (mine) {
            if constexpr (PAIR) {
              // the peer's partial sits where the result goes: add in place
              uint4* rp = reinterpret_cast<uint4*>(wp + hh * 16);
              const uint4 r0_ = rp[0], r1_ = rp[1];
              const uint32_t rw[8] = {r0_.x, r0_.y, r0_.z, r0_.w, r1_.x, r1_.y, r1_.z, r1_.w};
              uint32_t ow[8];
#pragma unroll
              for (int k = 0; k < 8; ++k) {
                const float2 pr = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&rw[k]));
                ow[k] = pack2_bf16(fmaf(pr.x, rowf[RT + hh * 16 + 2 * k], v[2 * k] * rowf[hh * 16 + 2 * k]),
                                   fmaf(pr.y, rowf[RT + hh * 16 + 2 * k + 1], v[2 * k + 1] * rowf[hh * 16 + 2 * k + 1]));
              }
              rp[0] = make_uint4(ow[0], ow[1], ow[2], ow[3]);
              rp[1] = make_uint4(ow[4], ow[5], ow[6], ow[7]);
            } else {
#pragma unroll
              for (int r = 0; r < 16; ++r) wt[(hh * 16 + r) * SLD] = __float2bfloat16_rn(v[r] * rowf[hh * 16 + r]);
            }
          }
        }
      }
      tc_fence_before();
      if (overlay) {
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars.l_free);
      }
      named_barrier_arrive(BAR_W_READY, FCONS);
    }
    named_barrier_sync(BAR_END, (CW + 1) * 32);
    if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
    if constexpr (PAIR) cluster_exit_sync();
    return;
  }

  // ======================================================================================================
  // value warps: scores, text attention, y^T += V^T W^T, output
  // ======================================================================================================
  // the stage in `slot` has been consumed by this warp
  auto release = [&]() {
    __syncwarp();
    if (lane == 0) mbar_arrive(&bars.empty[slot]);
    advance();
  };
  const int VTH = VW * 32;
  const int vw = warp - TEW, vtid = tid - TEW * 32;
  const int bl = vw / WPG, wig = vw - bl * WPG;
  const int msplit = a.msplit, mshift = a.mshift;           // a task covers the row tiles mt with (mt >> mshift) == its group

  for (int u = blockIdx.x; u < a.units; u += gridDim.x) {
    const int h = u / per_h, rem = u - h * per_h;
    const int bg = rem / a.nrg, rg = rem - bg * a.nrg;
    const int rk = PAIR ? (rg & 1) : 0;
    const int b0 = bg * a.NB, r0 = PAIR ? (rg >> 1) * a.RB : rg * a.RB;
    const int nbv = min(a.NB, a.B - b0);
    const int rbv = min(RB, a.R - r0);
    const RowRanges tr = row_ranges(a, rg);
    const int nts = tr.na + tr.nb;
    const int c2first = (PAIR && rk) ? NJ0 : 0, c2count = PAIR ? (rk ? a.NJ - NJ0 : NJ0) : a.NJ;
    (void)r0;

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
      if (si >= 2) wait_on(&bars.s_free[sbuf], ((si >> 1) - 1) & 1u);   // the MMAs that read this buffer's previous tile are complete
      unsigned char* Sb = S_sm + sbuf * s_buf_bytes;
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
            if (head < G) {
              // element (row rho, column j) of sub-chunk s, K-major core matrices of 8 rows x 8 columns
              const int rho = bi * GP + head;
              *reinterpret_cast<__nv_bfloat16*>(Sb + s * (RT * 32) + (j >> 3) * (RT * 16) + (rho >> 3) * 128 + (rho & 7) * 16 + (j & 7) * 2) =
                  __float2bfloat16_rn((sc[nh][0][e] + sc[nh][1][e]) * qscale);
            }
          }
      }
      fence_proxy_async();                                              // the tile is read by the tensor core (async proxy)
      named_barrier_arrive(BAR_S_READY + (int)sbuf, SREADY);
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
    for (int iu = 0, it = 0; iu + it < a.nu + nts;) {
      if (!next_is_text(iu, it, a.nu, nts)) {            // a stage of U: the tensor core's
        ++iu;
        wait_on(&bars.full[slot], phase);
        release();
        continue;
      }
      const int ts = it++;
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

    // ---------------- joint softmax: maxima and sums of this warp's text rows out, the joint maximum back ----------------
#pragma unroll
    for (int hr = 0; hr < 2; ++hr) {
      float l = l_run[hr];
      l += __shfl_xor_sync(0xffffffffu, l, 1);
      l += __shfl_xor_sync(0xffffffffu, l, 2);
      if (t4 == 0) { tmax[vw * 16 + gid + 8 * hr] = m_run[hr]; tsum[vw * 16 + gid + 8 * hr] = l; }
    }
    named_barrier_sync(1, FCONS);                                   // B1
    named_barrier_sync(1, FCONS);                                   // B2: joint maxima and sums
    {
      float scl[2];
#pragma unroll
      for (int hr = 0; hr < 2; ++hr) {
        const float M = hmax[bl * 16 + gid + 8 * hr];
        scl[hr] = m_run[hr] == -INFINITY ? 0.f : fast_exp2(m_run[hr] - M);
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

    // ---------------- y^T[128][heads] += V^T[128][16 rows of block] W^T[16][heads of block], all weights in place ----------------
    named_barrier_sync(BAR_W_READY, FCONS);
    for (int c = 0; c < c2count; ++c) {
      wait_on(&bars.full[slot], phase);
      const uint32_t v_u = sm_u + slot * a.stage_bytes + a.par_bytes;
      const int nsub = min(JC, (a.m - (c2first + c) * rows16 + 15) >> 4);
      const int ntask = RB * msplit;
      for (int task = wig; task < nsub * ntask; task += WPG) {          // my (sub-chunk, block, row-tile group) tasks
        const int s = task / ntask, tk = task - s * ntask;
        const int rl = tk >> (3 - mshift), mg = tk & (msplit - 1);
        if (rl >= rbv || bl >= nbv) continue;
        const int bi = bl * RB + rl;
        uint32_t bw[4];
        if constexpr (PAIR)      // tiles kept as [row of U][expansion row]: transposing load; rows of U by lmid, heads by lhi
          ldsm_x4_t(bw, W_u + (uint32_t)((((c * JC + s) * 16 + lmid * 8 + l7) * WLD + bi * GP + lhi * 8) * 2));
        else
          ldsm_x4(bw, W_u + (uint32_t)(((c * JC + s) * ((RT + 16) * SLD) + (bi * G + lrowB) * SLD + lmid * 8) * 2));
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
      release();
    }
    named_barrier_sync(3, VTH);                                     // the weight tiles share their region with the reduction buffer

    // ---------------- unit end: reduce over the value warps, mu term, normalise or leave a partial ----------------
    const int bh = b0 * a.H_kv + h;                    // used when the block axis is split (NB == 1)
    const size_t pbase = ((size_t)bh * a.nrg + rg) * G;
    const int YHG = a.yhg;
    // pair mode, one block group per sequence: the two outputs of the pair are merged through distributed shared memory
    // (CTA 1 sends, CTA 0 merges and writes); the buffers are regions that are dead by now: the query tile for this CTA's
    // output, the score tiles for the peer's
    const bool pmerge = PAIR && a.nrg == 2 && G <= 8;
    float* ybuf0 = reinterpret_cast<float*>(sm + a.off_q);
    float* ybuf1 = reinterpret_cast<float*>(sm + a.off_S);
    const uint32_t ypeer = PAIR ? map_to_cta(smem_addr(ybuf1), 0u) : 0u;
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
        else if (pmerge) {
          if (rk) st_cluster_f32(ypeer + (uint32_t)((g * D + col) * 4), y); else ybuf0[g * D + col] = y;
        } else
          a.part_y[(pbase + g) * D + col] = y;
      }
      named_barrier_sync(3, VTH);
    }
    if (pmerge) {
      if (rk) {
        if (vtid < G) {
          const uint32_t mp = map_to_cta(smem_addr(&s_mlpeer[vtid]), 0u);
          st_cluster_f32(mp, hmax[vtid]);
          st_cluster_f32(mp + 4u, hsum[vtid]);
        }
        named_barrier_sync(3, VTH);                                   // every value of this CTA's output has been sent
        if (vtid == 0) mbar_arrive_cluster(map_to_cta(smem_addr(&bars.m_data), 0u));
      } else {
        named_barrier_sync(3, VTH);                                   // this CTA's output is in its buffer
        if (!dead && !mbar_wait_cluster_bounded(&bars.m_data, vunit & 1u)) dead = true;
        __syncwarp();
        for (int idx = vtid; idx < G * D; idx += VTH) {
          const int g = idx >> 7, col = idx & (D - 1);
          const float M0 = hmax[g], M1 = s_mlpeer[g].x, M = fmaxf(M0, M1);
          const float w0 = fast_exp2(M0 - M), w1 = fast_exp2(M1 - M);
          const float num = fmaf(ybuf0[idx], w0, ybuf1[idx] * w1), den = fmaf(hsum[g], w0, s_mlpeer[g].y * w1);
          a.out[((size_t)b0 * a.H_kv * G + (size_t)h * G + g) * D + col] = __float2bfloat16_rn(num / den);
        }
        named_barrier_sync(3, VTH);                                   // the buffers are read: the next unit may overwrite them
      }
      ++vunit;
    } else if (a.nrg > 1) {
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
  named_barrier_sync(BAR_END, (CW + 1) * 32);
  if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
  if constexpr (PAIR) cluster_exit_sync();
}

// ------------------------------------------------------------------------------------------ host side
FusedPlan plan_fused_tc(const kvc_layer* L, int B, int R) {
  FusedPlan p{};
  const int G = L->G, n = L->desc.n, m = L->m, H_kv = L->desc.H_kv;
  if (L->desc.dtype != KVC_BF16 || L->passthrough || R < 1 || B < 1 || n % 64 != 0 || n > 1024 || G > 16) return p;
  if (reinterpret_cast<uintptr_t>(L->desc.theta) & 15 || reinterpret_cast<uintptr_t>(L->desc.U) & 15) return p;
  const int sms = L->num_sms > 0 ? L->num_sms : 148;
  p.tc = 1;
  p.EW = 4;
  p.VW = n <= 256 ? 8 : 10;
  p.ktw = 0;
  // the logits live in tensor memory: two row tiles per unit whenever a sequence has more than 16 expansion rows
  p.MT = G * R > ROWS ? 2 : 1;
  if (p.MT == 2 && n > 256) { p.EW = 8; p.VW = 6; }     // 32 rows x long blocks: the softmax is the larger share, the value warps have slack
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
  if (p.stage_bytes < 16384u) p.stage_bytes = 16384u;                  // a stage also holds 128 rows x 64 columns of U
  const int mtiles = ceil_div(m, 128);
  p.UT = (int)(p.stage_bytes / 16384u) < mtiles ? (int)(p.stage_bytes / 16384u) : mtiles;
  p.nu = p.ncg * ceil_div(mtiles, p.UT);
  int tch = (int)(p.stage_bytes / (p.NB * 512u)) & ~15;
  p.TCH = tch > 256 ? 256 : tch;
  if (p.TCH < 16) return p;
  p.txt_half_bytes = (uint32_t)p.NB * p.TCH * 128u;
  {
    const int wpg = p.VW / p.NB;
    int best = 1 << 30;
    for (int sh = 3; sh >= 0; --sh) {            // sh = 3: one task per block
      const int ms = 8 >> sh, cost = ceil_div(p.JC * p.RB * ms, wpg) * ((1 << sh) + 1);
      if (cost < best) { best = cost; p.msplit = ms; p.mshift = sh; }
    }
  }
  p.sld = 0;
  const int rt = ROWS * p.MT;
  p.yhg = G > 4 ? 8 : (G > 2 ? 4 : 2);
  uint32_t off = 0;
  auto take = [&](uint32_t bytes) { uint32_t o = off; off = (off + bytes + 127u) & ~127u; return o; };
  // one region right after the ring (1024-byte aligned) serves, in turn: P (operand of the re-projection MMAs), the
  // weight tiles of all m rows (written once those MMAs are complete), the reduction buffer of the unit end
  const uint32_t p_bytes = (uint32_t)rt * n * 2, yred_bytes = (uint32_t)p.VW * p.yhg * D * 4;
  const uint32_t w_bytes = (uint32_t)ceil_div(m, 16) * (rt + 16) * SLD * 2;
  uint32_t r0_bytes = p_bytes > yred_bytes ? p_bytes : yred_bytes;
  if (w_bytes > r0_bytes) r0_bytes = w_bytes;
  p.off_P = take(r0_bytes);
  p.off_yred = p.off_P;
  p.off_W = p.off_P;
  p.off_q = take((uint32_t)p.NB * 16 * QLD * 2);
  p.off_S = take((uint32_t)(2 * p.JC * rt * 32));
  p.off_wred = 0;
  p.off_rstat = take((uint32_t)2 * p.EW * rt * 4);
  p.off_tstat = take((uint32_t)2 * p.VW * 16 * 4);
  p.off_hstat = take((uint32_t)(6 * p.NB * 16 + 2 * rt) * 4);
  p.off_rtab = take((uint32_t)rt * 4);
  p.misc_bytes = off;
  const int nt = (n + 127) / 128;
  int cols = 32;
  while (cols < nt * rt + mtiles * rt) cols *= 2;
  p.tmem_cols = cols;
  if (cols > 512) return p;
  if (SMEM_LIMIT < 1024u + 2048u + p.misc_bytes + 2 * p.stage_bytes) return p;
  const uint32_t avail = SMEM_LIMIT - 1024u - 2048u - p.misc_bytes;   // alignment slack; static shared memory and its padding
  int stages = (int)(avail / p.stage_bytes);
  p.stages = stages > FMAX_STAGES ? FMAX_STAGES : stages;
  if (p.stages < 2) return p;
  p.smem_bytes = (size_t)p.stages * p.stage_bytes + p.misc_bytes + 1024u;
  p.grid = p.units < sms ? p.units : sms;
  p.ok = 1;
  return p;
}

// Pair mode: one (sequence, KV head) per cluster of two CTAs, all its blocks in one unit of up to 64 expansion rows.
FusedPlan plan_fused_pair(const kvc_layer* L, int B, int R) {
  FusedPlan p{};
  const int G = L->G, n = L->desc.n, m = L->m, H_kv = L->desc.H_kv;
  const int GP = G <= 8 ? 8 : 16;                                      // expansion rows per block, padded
  if (L->desc.dtype != KVC_BF16 || L->passthrough || R < 1 || B < 1 || n % 256 != 0 || n > 1024 || G > 16 || m < 32) return p;
  if (reinterpret_cast<uintptr_t>(L->desc.theta) & 15 || reinterpret_cast<uintptr_t>(L->desc.U) & 15) return p;
  const int sms = L->num_sms > 0 ? L->num_sms : 148;
  p.tc = 2;
  p.EW = 4; p.VW = 8; p.ktw = 0;
  p.MT = 4;
  const int rt = ROWS * p.MT;
  p.NB = 1; p.nbg = B;
  p.RB = R < 64 / GP ? R : 64 / GP;            // blocks per pair: up to 64 padded expansion rows
  p.nrg = 2 * ceil_div(R, p.RB);               // every pair leaves two partial outputs per (sequence, head)
  p.units = H_kv * B * p.nrg;
  p.ncg = n / 64;
  const int ncgl = p.ncg / 2;
  const uint32_t chunk = (uint32_t)p.RB * 4096u + (uint32_t)(n / 2) * 32u;
  int jc = (int)(49152u / chunk);
  const int jmax = ceil_div(m, 32) < 16 ? ceil_div(m, 32) : 16;       // at least two stages along m: one per CTA in the value pass
  p.JC = jc < 1 ? 1 : (jc > jmax ? jmax : jc);
  p.NJ = ceil_div(m, 16 * p.JC);
  if (p.NJ < 2) return p;
  p.par_bytes = (uint32_t)ncgl * p.JC * 2048u;
  p.k_half_bytes = (uint32_t)p.RB * p.JC * 2048u;
  p.stage_bytes = p.par_bytes + 2 * p.k_half_bytes;
  if (p.stage_bytes < 16384u) p.stage_bytes = 16384u;
  const int mtiles = ceil_div(m, 128);
  p.UT = (int)(p.stage_bytes / 16384u) < mtiles ? (int)(p.stage_bytes / 16384u) : mtiles;
  p.nu = ncgl * ceil_div(mtiles, p.UT);
  int tch = (int)(p.stage_bytes / 512u) & ~15;
  p.TCH = tch > 256 ? 256 : tch;
  if (p.TCH < 16) return p;
  p.txt_half_bytes = (uint32_t)p.TCH * 128u;
  {
    int best = 1 << 30;
    for (int sh = 3; sh >= 0; --sh) {
      const int ms = 8 >> sh, cost = ceil_div(p.JC * p.RB * ms, p.VW) * ((1 << sh) + 1);
      if (cost < best) { best = cost; p.msplit = ms; p.mshift = sh; }
    }
  }
  p.sld = 0;
  p.yhg = G > 4 ? 8 : (G > 2 ? 4 : 2);
  uint32_t off = 0;
  auto take = [&](uint32_t bytes) { uint32_t o = off; off = (off + bytes + 127u) & ~127u; return o; };
  const int nj0 = (p.NJ + 1) / 2;                                      // stages of the m axis of CTA 0 (the larger share)
  const uint32_t p_bytes = (uint32_t)rt * (n / 2) * 2, yred_bytes = (uint32_t)p.VW * p.yhg * D * 4;
  const uint32_t w_bytes = (uint32_t)nj0 * p.JC * 16 * (rt + 8) * 2;     // [rows of U of CTA 0][expansion rows + 8]
  uint32_t r0_bytes = p_bytes > yred_bytes ? p_bytes : yred_bytes;
  if (w_bytes > r0_bytes) r0_bytes = w_bytes;
  p.off_P = take(r0_bytes);
  p.off_yred = p.off_P;
  p.off_W = p.off_P;
  p.off_wrecv = 0;
  p.off_xstat = take((uint32_t)(16 + rt) * 4);
  p.off_q = take((uint32_t)16 * QLD * 2);
  p.off_S = take((uint32_t)(2 * p.JC * rt * 32));
  p.off_wred = 0;
  p.off_rstat = take((uint32_t)2 * p.EW * rt * 4);
  p.off_tstat = take((uint32_t)2 * p.VW * 16 * 4);
  p.off_hstat = take((uint32_t)(6 * 16 + 2 * rt) * 4);
  p.off_rtab = take((uint32_t)rt * 4);
  p.misc_bytes = off;
  // tensor memory: n/256 tiles of L^T, then the tiles of W^T; W^T tiles that do not fit behind them take the columns of
  // L^T (dead by then), so up to n/256 more
  const int lcols = (n / 256) * rt;
  int cols = 32;
  while (cols < lcols + mtiles * rt && cols < 512) cols *= 2;
  p.tmem_cols = cols;
  if (lcols + mtiles * rt > 512 && mtiles - (512 - lcols) / rt > n / 256) return p;
  if (SMEM_LIMIT < 1024u + 2048u + p.misc_bytes + 2 * p.stage_bytes) return p;
  const uint32_t avail = SMEM_LIMIT - 1024u - 2048u - p.misc_bytes;
  int stages = (int)(avail / p.stage_bytes);
  p.stages = stages > FMAX_STAGES ? FMAX_STAGES : stages;
  if (p.stages < 2) return p;
  p.smem_bytes = (size_t)p.stages * p.stage_bytes + p.misc_bytes + 1024u;
  const int pairs = p.units / 2, slots = sms / 2;
  p.grid = 2 * (pairs < slots ? pairs : slots);
  p.ok = 1;
  return p;
}

template <int EW, int VW, int NH, int MT, bool PAIR>
static cudaError_t launch_tc_inst(const CUtensorMap* tm, const FusedArgs& fa, const FusedPlan& p, cudaStream_t st) {
  {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(fused_decode_tc_kernel<EW, VW, NH, MT, PAIR>), p.smem_bytes);
    if (e != cudaSuccess) return e;
  }
  if (!PAIR)
    return launch_dependent(fused_decode_tc_kernel<EW, VW, NH, MT, PAIR>, dim3(p.grid), dim3((EW + VW + 2) * 32), p.smem_bytes, st, tm[0],
                            tm[1], tm[2], tm[3], tm[4], tm[5], fa);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.grid);
  cfg.blockDim = dim3((EW + VW + 2) * 32);
  cfg.dynamicSmemBytes = p.smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, fused_decode_tc_kernel<EW, VW, NH, MT, PAIR>, tm[0], tm[1], tm[2], tm[3], tm[4], tm[5], fa);
}

template <int NH>
static cudaError_t launch_tc_nh(const CUtensorMap* tm, const FusedArgs& fa, const FusedPlan& p, cudaStream_t st) {
  if (p.tc == 2) return launch_tc_inst<4, 8, NH, 4, true>(tm, fa, p, st);
  if (p.EW == 8) return launch_tc_inst<8, 6, NH, 2, false>(tm, fa, p, st);
  if (p.VW == 8) return p.MT == 2 ? launch_tc_inst<4, 8, NH, 2, false>(tm, fa, p, st) : launch_tc_inst<4, 8, NH, 1, false>(tm, fa, p, st);
  return launch_tc_inst<4, 10, NH, 1, false>(tm, fa, p, st);
}

cudaError_t launch_fused_tc_kernel(const CUtensorMap* tm, const FusedArgs& fa, const FusedPlan& p, cudaStream_t st) {
  return fa.G > 8 ? launch_tc_nh<2>(tm, fa, p, st) : launch_tc_nh<1>(tm, fa, p, st);
}

}  // namespace kvc
