// Resident-parameter decode kernel (see kvc_resident.cuh): Algorithm 1 for short blocks in one kernel, per work item
//   vision block r:  S = sigma q K_tilde_r^T (step 1), L = S theta (step 2), P = 2^(L - M) with M the running maximum of the
//                    (sequence, query head), W = P U^T (step 3), y += W V_tilde_r (step 4), vision mass += sum P
//   text chunk:      s = sigma q K_txt^T, p = 2^(s - M), y += p V_txt
// and at the end of a (sequence, KV head): y += (vision mass) mu, out = y / (sum of all p), through a log-sum-exp merge
// when several CTAs share the pair.  All products are mma.sync m16n8k16 (bf16 in, fp32 accumulate) with the 16 rows of
// the A operand = the query heads of the group (zero-padded): the K extents are m and n, a few hundred, and a block is
// a few microseconds of HBM time, so the kernel is built around the load stream, not the tensor pipe: one producer
// thread keeps a ring of 16 KB tiles full while eight consumer warps walk the items.
#include "kvc_fused.cuh"
#include "kvc_resident.cuh"

namespace kvc {

constexpr int RS_THREADS = (RS_WARPS + 1) * 32;
constexpr int RS_CONS = RS_WARPS * 32;
constexpr uint32_t RS_SMEM_LIMIT = 232448;
constexpr int RS_TLD = 68;                                                   // row pitch of the fp32 text scores
constexpr float RS_QSCALE = 0.08838834764831845f * 1.4426950408889634f;      // sigma = 1/sqrt(128), logits in log2 units

__global__ void __launch_bounds__(RS_THREADS, 1)
resident_decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                       const __grid_constant__ CUtensorMap tmKt, const __grid_constant__ CUtensorMap tmVt,
                       const __grid_constant__ CUtensorMap tmTh, const __grid_constant__ CUtensorMap tmU,
                       const ResidentArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* sm = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
  __shared__ __align__(8) uint64_t full_bar[RS_MAX_STAGES], empty_bar[RS_MAX_STAGES], par_bar;
  __shared__ int s_last;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int h = blockIdx.x / a.cph, c = blockIdx.x - h * a.cph;
  const long long items_h = (long long)a.B * a.items_b;
  const int lo = (int)(c * items_h / a.cph), hi = (int)((c + 1) * items_h / a.cph);
  const int nst = a.stages;
  if (tid == 0) {
    for (int s = 0; s < nst; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], RS_WARPS); }
    mbar_init(&par_bar, 1);
    fence_mbar_init();
  }
  __syncthreads();

  if (warp == RS_WARPS) {
    // ================= producer =================
    if (lane != 0 || lo >= hi) return;
    tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmTh); tma_prefetch_desc(&tmU);
    if (a.T > 0) { tma_prefetch_desc(&tmKt); tma_prefetch_desc(&tmVt); }
    // the parameters of the head: fixed at inference (Sec. 3.2), so they need not wait for the stream's previous kernel
    mbar_expect_tx(&par_bar, 2u * a.par_bytes);
    tma_load_4d(sm + a.off_theta, &tmTh, 0, 0, 0, h, &par_bar);
    tma_load_4d(sm + a.off_U, &tmU, 0, 0, 0, h, &par_bar);
    grid_dep_wait();
    uint32_t slot = 0, phase = 1;
    auto tile = [&](const CUtensorMap* tm, int row0, int idx3) -> bool {
      if (!mbar_wait_bounded(&empty_bar[slot], phase)) { atomicExch(a.status, (int)KVC_ERR_TIMEOUT); return false; }
      unsigned char* dst = sm + a.off_ring + slot * RS_TILE_BYTES;
      mbar_expect_tx(&full_bar[slot], RS_TILE_BYTES);
      tma_load_3d(dst, tm, 0, row0, idx3, &full_bar[slot]);
      tma_load_3d(dst + RS_TILE_BYTES / 2, tm, 64, row0, idx3, &full_bar[slot]);
      if (++slot == (uint32_t)nst) { slot = 0; phase ^= 1u; }
      return true;
    };
    for (int it = lo; it < hi; ++it) {
      const int b = it / a.items_b, k = it - b * a.items_b, bh = b * a.H_kv + h;
      if (k < a.R) {
        for (int t = 0; t < a.kt; ++t) if (!tile(&tmK, t * RS_TILE_ROWS, bh * a.R + k)) return;
        for (int t = 0; t < a.kt; ++t) if (!tile(&tmV, t * RS_TILE_ROWS, bh * a.R + k)) return;
      } else {
        if (!tile(&tmKt, (k - a.R) * RS_TILE_ROWS, bh)) return;
        if (!tile(&tmVt, (k - a.R) * RS_TILE_ROWS, bh)) return;
      }
    }
    return;
  }

  // ================= consumers =================
  grid_dep_wait();
  grid_dep_launch();
  if (blockIdx.x == 0 && tid == 0) *a.status = 0;
  const int gid = lane >> 2, t4 = lane & 3;
  const int arow = (lane & 7) + ((lane >> 3) & 1) * 8, asel = lane >> 4;   // ldmatrix lane roles (row of the 16, second half)
  const uint32_t sm_u = smem_addr(sm);
  const uint32_t th_u = sm_u + a.off_theta, U_u = sm_u + a.off_U, ring_u = sm_u + a.off_ring;
  const uint32_t S_u = sm_u + a.off_S, P_u = sm_u + a.off_P, W_u = sm_u + a.off_W;
  __nv_bfloat16* Ssm = reinterpret_cast<__nv_bfloat16*>(sm + a.off_S);
  __nv_bfloat16* Psm = reinterpret_cast<__nv_bfloat16*>(sm + a.off_P);
  __nv_bfloat16* Wsm = reinterpret_cast<__nv_bfloat16*>(sm + a.off_W);
  float* Tsm = reinterpret_cast<float*>(sm + a.off_T);
  float* wmax = reinterpret_cast<float*>(sm + a.off_stat);       // [8][16]
  float* wsum = wmax + RS_WARPS * 16;                            // [8][16]
  float* rowM = wsum + RS_WARPS * 16;                            // running maximum per query head of the group
  float* rowL = rowM + 16;                                       // running sum of all probabilities
  float* rowV = rowL + 16;                                       // running sum of the vision probabilities
  float* rowC = rowV + 16;                                       // rescale factor of the current text chunk
  const int pS = a.pitchS, pP = a.pitchP, pW = a.pitchW, mp = a.mp, G = a.G;
  const int NTW = a.n / 64;                                      // 8-column tiles of the logits per warp
  const int wt = mp / 8;                                         // 8-column tiles of the weights
  const uint32_t panel = (uint32_t)mp * 128u;                    // bytes of one 64-column panel of theta / U

  if (tid < 16) { rowM[tid] = -INFINITY; rowL[tid] = 0.f; rowV[tid] = 0.f; }
  float yacc[2][4];
#pragma unroll
  for (int x = 0; x < 2; ++x)
#pragma unroll
    for (int e = 0; e < 4; ++e) yacc[x][e] = 0.f;
  named_barrier_sync(1, RS_CONS);

  uint32_t slot = 0, phase = 0;
  bool dead = false, par_ready = false;
  int cur_b = -1;
  uint32_t qa[8][4];
  auto next_tile = [&]() -> uint32_t {          // waits for the ring's next tile, returns its shared-memory address
    if (!dead && !mbar_wait_bounded(&full_bar[slot], phase)) dead = true;
    __syncwarp();
    return ring_u + slot * RS_TILE_BYTES;
  };
  auto release_tile = [&]() {
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[slot]);
    if (++slot == (uint32_t)nst) { slot = 0; phase ^= 1u; }
  };

  for (int it = lo; it < hi; ++it) {
    const int b = it / a.items_b, k = it - b * a.items_b, bh = b * a.H_kv + h;
    const bool vis = k < a.R;
    if (b != cur_b) {
      cur_b = b;
      // A fragments of the score product: rows = the query heads of the group (gid, gid + 8), k = the 128 channels
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
    // ---- step 1: scores of the item's key rows; a warp takes 8 rows of every tile
    const int ntile = vis ? a.kt : 1;
    for (int t = 0; t < ntile; ++t) {
      const uint32_t st_u = next_tile();
      float acc2[2][4];
#pragma unroll
      for (int x = 0; x < 2; ++x)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc2[x][e] = 0.f;
      const int row = warp * 8 + (lane & 7);
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const int cc = 4 * x + (lane >> 3);          // 16-byte piece of the 256-byte row
        uint32_t bf[4];
        ldsm_x4(bf, st_u + (uint32_t)(cc >> 3) * (RS_TILE_BYTES / 2) + (uint32_t)row * 128u + (uint32_t)(((cc & 7) ^ (row & 7)) << 4));
        mma_bf16_16816(acc2[x & 1], qa[2 * x], bf[0], bf[1]);
        mma_bf16_16816(acc2[x & 1], qa[2 * x + 1], bf[2], bf[3]);
      }
      const int col = t * RS_TILE_ROWS + warp * 8 + 2 * t4;    // key row of acc[0] / acc[2]; acc[1] / acc[3] the next one
      const float v0 = (acc2[0][0] + acc2[1][0]) * RS_QSCALE, v1 = (acc2[0][1] + acc2[1][1]) * RS_QSCALE;
      const float v2 = (acc2[0][2] + acc2[1][2]) * RS_QSCALE, v3 = (acc2[0][3] + acc2[1][3]) * RS_QSCALE;
      if (vis) {
        if (col < mp) {
          *reinterpret_cast<uint32_t*>(Ssm + gid * pS + col) = pack2_bf16(v0, v1);
          *reinterpret_cast<uint32_t*>(Ssm + (gid + 8) * pS + col) = pack2_bf16(v2, v3);
        }
      } else {
        *reinterpret_cast<float2*>(Tsm + gid * RS_TLD + col) = make_float2(v0, v1);
        *reinterpret_cast<float2*>(Tsm + (gid + 8) * RS_TLD + col) = make_float2(v2, v3);
      }
      release_tile();
    }
    named_barrier_sync(1, RS_CONS);

    if (vis) {
      if (!par_ready) {
        if (!dead && !mbar_wait_bounded(&par_bar, 0)) dead = true;
        par_ready = true;
      }
      // ---- step 2: L[16 x n] = S[16 x m] theta[m x n]; warp w holds columns [w n/8, (w+1) n/8)
      float lacc[4][4];
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int e = 0; e < 4; ++e) lacc[x][e] = 0.f;
      for (int ks = 0; ks < mp / 16; ++ks) {
        uint32_t af[4];
        ldsm_x4(af, S_u + (uint32_t)(arow * pS + ks * 16 + asel * 8) * 2u);
        const int krow = ks * 16 + arow;
#pragma unroll
        for (int np = 0; np < 2; ++np) {
          if (2 * np < NTW) {
            int nt = 2 * np + asel;
            nt = nt < NTW ? nt : NTW - 1;
            const int col8 = warp * NTW + nt;
            uint32_t bf[4];
            ldsm_x4_t(bf, th_u + (uint32_t)(col8 >> 3) * panel + (uint32_t)krow * 128u + (uint32_t)(((col8 & 7) ^ (krow & 7)) << 4));
            mma_bf16_16816(lacc[2 * np], af, bf[0], bf[1]);
            if (2 * np + 1 < NTW) mma_bf16_16816(lacc[2 * np + 1], af, bf[2], bf[3]);
          }
        }
      }
      // ---- softmax pieces of the block relative to the running maximum of each query head
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
        if (nt < NTW) {
          mx0 = fmaxf(mx0, fmaxf(lacc[nt][0], lacc[nt][1]));
          mx1 = fmaxf(mx1, fmaxf(lacc[nt][2], lacc[nt][3]));
        }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      if (t4 == 0) { wmax[warp * 16 + gid] = mx0; wmax[warp * 16 + gid + 8] = mx1; }
      named_barrier_sync(1, RS_CONS);
      float bm0 = wmax[gid], bm1 = wmax[gid + 8];
#pragma unroll
      for (int w = 1; w < RS_WARPS; ++w) { bm0 = fmaxf(bm0, wmax[w * 16 + gid]); bm1 = fmaxf(bm1, wmax[w * 16 + gid + 8]); }
      const float Mo0 = rowM[gid], Mo1 = rowM[gid + 8];
      const float Mn0 = fmaxf(Mo0, bm0), Mn1 = fmaxf(Mo1, bm1);
      const float c0 = Mo0 == -INFINITY ? 0.f : fast_exp2(Mo0 - Mn0), c1 = Mo1 == -INFINITY ? 0.f : fast_exp2(Mo1 - Mn1);
      float s0 = 0.f, s1 = 0.f;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
        if (nt < NTW) {
          const float p0 = fast_exp2(lacc[nt][0] - Mn0), p1 = fast_exp2(lacc[nt][1] - Mn0);
          const float p2 = fast_exp2(lacc[nt][2] - Mn1), p3 = fast_exp2(lacc[nt][3] - Mn1);
          s0 += p0 + p1;
          s1 += p2 + p3;
          const int colp = (warp * NTW + nt) * 8 + 2 * t4;
          *reinterpret_cast<uint32_t*>(Psm + gid * pP + colp) = pack2_bf16(p0, p1);
          *reinterpret_cast<uint32_t*>(Psm + (gid + 8) * pP + colp) = pack2_bf16(p2, p3);
        }
      s0 += __shfl_xor_sync(0xffffffffu, s0, 1); s0 += __shfl_xor_sync(0xffffffffu, s0, 2);
      s1 += __shfl_xor_sync(0xffffffffu, s1, 1); s1 += __shfl_xor_sync(0xffffffffu, s1, 2);
      if (t4 == 0) { wsum[warp * 16 + gid] = s0; wsum[warp * 16 + gid + 8] = s1; }
#pragma unroll
      for (int x = 0; x < 2; ++x) { yacc[x][0] *= c0; yacc[x][1] *= c0; yacc[x][2] *= c1; yacc[x][3] *= c1; }
      named_barrier_sync(1, RS_CONS);
      if (warp == 0 && lane < 16) {
        float bm = wmax[lane], ss = wsum[lane];
#pragma unroll
        for (int w = 1; w < RS_WARPS; ++w) { bm = fmaxf(bm, wmax[w * 16 + lane]); ss += wsum[w * 16 + lane]; }
        const float Mo = rowM[lane], Mn = fmaxf(Mo, bm);
        const float cc = Mo == -INFINITY ? 0.f : fast_exp2(Mo - Mn);
        rowL[lane] = rowL[lane] * cc + ss;
        rowV[lane] = rowV[lane] * cc + ss;
        rowM[lane] = Mn;
      }
      // ---- step 3: W[16 x m] = P[16 x n] U^T; the 8-column tiles w, w + 8, w + 16 of the m axis go to warp w
      float wacc[3][4];
#pragma unroll
      for (int x = 0; x < 3; ++x)
#pragma unroll
        for (int e = 0; e < 4; ++e) wacc[x][e] = 0.f;
      if (warp < wt) {
        for (int ks = 0; ks < a.n / 16; ++ks) {
          uint32_t af[4];
          ldsm_x4(af, P_u + (uint32_t)(arow * pP + ks * 16 + asel * 8) * 2u);
          const int kcol = ks * 16 + ((lane >> 3) & 1) * 8;
          const uint32_t pan = (uint32_t)(kcol >> 6) * panel;
          const int chunk = (kcol & 63) >> 3;
          {
            int tile = warp + 8 * asel;
            tile = tile < wt ? tile : warp;
            const int j = tile * 8 + (lane & 7);
            uint32_t bf[4];
            ldsm_x4(bf, U_u + pan + (uint32_t)j * 128u + (uint32_t)((chunk ^ (j & 7)) << 4));
            mma_bf16_16816(wacc[0], af, bf[0], bf[1]);
            if (warp + 8 < wt) mma_bf16_16816(wacc[1], af, bf[2], bf[3]);
          }
          if (warp + 16 < wt) {
            const int j = (warp + 16) * 8 + (lane & 7);
            uint32_t bf[4];
            ldsm_x4(bf, U_u + pan + (uint32_t)j * 128u + (uint32_t)((chunk ^ (j & 7)) << 4));
            mma_bf16_16816(wacc[2], af, bf[0], bf[1]);
          }
        }
#pragma unroll
        for (int x = 0; x < 3; ++x)
          if (warp + 8 * x < wt) {
            const int colw = (warp + 8 * x) * 8 + 2 * t4;
            *reinterpret_cast<uint32_t*>(Wsm + gid * pW + colw) = pack2_bf16(wacc[x][0], wacc[x][1]);
            *reinterpret_cast<uint32_t*>(Wsm + (gid + 8) * pW + colw) = pack2_bf16(wacc[x][2], wacc[x][3]);
          }
      }
      named_barrier_sync(1, RS_CONS);
    } else {
      // ---- text chunk: warp w owns query heads 2w and 2w + 1 (64 scores each)
      const int base = (k - a.R) * RS_TILE_ROWS;
#pragma unroll
      for (int rr = 0; rr < 2; ++rr) {
        const int row = 2 * warp + rr;
        const float sa = base + lane < a.T ? Tsm[row * RS_TLD + lane] : -INFINITY;
        const float sb = base + lane + 32 < a.T ? Tsm[row * RS_TLD + lane + 32] : -INFINITY;
        float cm = fmaxf(sa, sb);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, o));
        const float Mo = rowM[row], Mn = fmaxf(Mo, cm);
        const float pa = fast_exp2(sa - Mn), pb = fast_exp2(sb - Mn);
        float ps = pa + pb;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
        Wsm[row * pW + lane] = __float2bfloat16_rn(pa);
        Wsm[row * pW + lane + 32] = __float2bfloat16_rn(pb);
        __syncwarp();
        if (lane == 0) {
          const float cc = Mo == -INFINITY ? 0.f : fast_exp2(Mo - Mn);
          rowC[row] = cc;
          rowL[row] = rowL[row] * cc + ps;
          rowV[row] *= cc;
          rowM[row] = Mn;
        }
      }
      named_barrier_sync(1, RS_CONS);
      const float c0 = rowC[gid], c1 = rowC[gid + 8];
#pragma unroll
      for (int x = 0; x < 2; ++x) { yacc[x][0] *= c0; yacc[x][1] *= c0; yacc[x][2] *= c1; yacc[x][3] *= c1; }
    }

    // ---- step 4: y[16 x 128] += W (or p) times the item's value rows; warp w holds channels [16w, 16w + 16)
    {
      const int kmax = vis ? mp : RS_TILE_ROWS;
      for (int t = 0; t < ntile; ++t) {
        const uint32_t st_u = next_tile() + (uint32_t)(warp >> 2) * (RS_TILE_BYTES / 2);
        const int cb = (2 * warp) & 7;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          if (t * RS_TILE_ROWS + ks * 16 < kmax) {
            uint32_t af[4], bf[4];
            ldsm_x4(af, W_u + (uint32_t)(arow * pW + t * RS_TILE_ROWS + ks * 16 + asel * 8) * 2u);
            const int krow = ks * 16 + arow;
            ldsm_x4_t(bf, st_u + (uint32_t)krow * 128u + (uint32_t)(((cb + asel) ^ (krow & 7)) << 4));
            mma_bf16_16816(yacc[0], af, bf[0], bf[1]);
            mma_bf16_16816(yacc[1], af, bf[2], bf[3]);
          }
        }
        release_tile();
      }
    }

    // ---- end of this CTA's items of the (sequence, KV head): the centring term, then the result or a partial
    if (it + 1 == hi || (it + 1) / a.items_b != b) {
      const int first = (int)((((long long)b * a.items_b + 1) * a.cph - 1) / items_h);
      const int last = (int)((((long long)(b + 1) * a.items_b) * a.cph - 1) / items_h);
      const int expected = last - first + 1, ps = c - first;
      named_barrier_sync(1, RS_CONS);                    // the statistics of the last item are complete
#pragma unroll
      for (int x = 0; x < 2; ++x)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const int row = gid + 8 * hf;
          if (row < G) {
            const int ch = warp * 16 + x * 8 + 2 * t4;
            const float vm = rowV[row];
            const float y0 = fmaf(vm, __bfloat162float(a.mu[h * D + ch]), yacc[x][2 * hf]);
            const float y1 = fmaf(vm, __bfloat162float(a.mu[h * D + ch + 1]), yacc[x][2 * hf + 1]);
            if (expected == 1) {
              const float inv = 1.f / rowL[row];
              *reinterpret_cast<uint32_t*>(a.out + ((size_t)bh * G + row) * D + ch) = pack2_bf16(y0 * inv, y1 * inv);
            } else {
              *reinterpret_cast<float2*>(a.py + (((size_t)bh * a.slots + ps) * 16 + row) * D + ch) = make_float2(y0, y1);
            }
          }
        }
      if (expected > 1) {
        if (warp == 0 && lane < 16) a.pml[((size_t)bh * a.slots + ps) * 16 + lane] = make_float2(rowM[lane], rowL[lane]);
        __threadfence();
        named_barrier_sync(1, RS_CONS);
        if (tid == 0) s_last = arrive_is_last(a.cnt + bh, a.token, expected) ? 1 : 0;
        named_barrier_sync(1, RS_CONS);
        if (s_last) {
          __threadfence();
          const float2* ml = a.pml + (size_t)bh * a.slots * 16;
          const float* py = a.py + (size_t)bh * a.slots * 16 * D;
          for (int x = tid; x < G * (D / 2); x += RS_CONS) {
            const int row = x / (D / 2), cp = x - row * (D / 2);
            float Ms = -INFINITY;
            for (int s = 0; s < expected; ++s) Ms = fmaxf(Ms, __ldcg(&ml[s * 16 + row].x));
            float den = 0.f, n0 = 0.f, n1 = 0.f;
            for (int s = 0; s < expected; ++s) {
              const float2 v = __ldcg(&ml[s * 16 + row]);
              const float f = fast_exp2(v.x - Ms);
              const float2 y = __ldcg(reinterpret_cast<const float2*>(py + ((size_t)s * 16 + row) * D + 2 * cp));
              den = fmaf(f, v.y, den);
              n0 = fmaf(f, y.x, n0);
              n1 = fmaf(f, y.y, n1);
            }
            const float inv = 1.f / den;
            *reinterpret_cast<uint32_t*>(a.out + ((size_t)bh * G + row) * D + 2 * cp) = pack2_bf16(n0 * inv, n1 * inv);
          }
        }
      }
      named_barrier_sync(1, RS_CONS);
      if (tid < 16) { rowM[tid] = -INFINITY; rowL[tid] = 0.f; rowV[tid] = 0.f; }
#pragma unroll
      for (int x = 0; x < 2; ++x)
#pragma unroll
        for (int e = 0; e < 4; ++e) yacc[x][e] = 0.f;
      named_barrier_sync(1, RS_CONS);
    }
  }
  if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
}

// ---- host ------------------------------------------------------------------------------------------------------
static int cph_max(const kvc_layer* L) {
  const int sms = L->num_sms > 0 ? L->num_sms : 148;
  const int c = sms / L->desc.H_kv;
  return c < 1 ? 1 : c;
}
// partial slots per (sequence, KV head): the runs of cph CTAs over B equal intervals meet an interval at most cph / B + 2 times
static int slots_per_pair(const kvc_layer* L, int B) {
  const int cm = cph_max(L), s = cm / (B > 0 ? B : 1) + 3;
  return s < cm ? s : cm;
}

ResidentPlan plan_resident(const kvc_layer* L, int B, int R, int T) {
  ResidentPlan p{};
  const int n = L->desc.n, m = L->m, G = L->G;
  if (L->desc.dtype != KVC_BF16 || L->passthrough || L->mode != KVC_MODE_KV || R < 1 || B < 1 || n % 64 != 0 || n > 256 ||
      G > 16)
    return p;
  if ((reinterpret_cast<uintptr_t>(L->desc.theta) | reinterpret_cast<uintptr_t>(L->desc.U)) & 15) return p;
  p.mp = (m + 15) & ~15;
  if (p.mp > 192) return p;                       // three 8-column weight tiles per warp at most
  p.ncg = n / 64;
  p.kt = ceil_div(m, RS_TILE_ROWS);
  p.ct = ceil_div(T, RS_TILE_ROWS);
  p.items_b = R + p.ct;
  const long long items_h = (long long)B * p.items_b;
  p.cph = (int)(items_h < cph_max(L) ? items_h : cph_max(L));
  p.grid = p.cph * L->desc.H_kv;
  p.pitchS = p.mp + 8;
  p.pitchP = n + 8;
  p.pitchW = (p.mp > RS_TILE_ROWS ? p.mp : RS_TILE_ROWS) + 8;
  p.par_bytes = (uint32_t)p.ncg * (uint32_t)p.mp * 128u;
  const uint32_t tiles = 16u * 2u * (uint32_t)(p.pitchS + p.pitchP + p.pitchW) + 16u * RS_TLD * 4u + (2u * RS_WARPS * 16u + 64u) * 4u;
  const uint32_t fixed = 2u * p.par_bytes + ((tiles + 127u) & ~127u) + 1024u + 2048u;
  if (fixed + 3u * RS_TILE_BYTES > RS_SMEM_LIMIT) return p;
  p.stages = (int)((RS_SMEM_LIMIT - fixed) / RS_TILE_BYTES);
  if (p.stages > RS_MAX_STAGES) p.stages = RS_MAX_STAGES;
  uint32_t off = 0;
  auto take = [&](uint32_t bytes) { uint32_t o = off; off = (off + bytes + 127u) & ~127u; return o; };
  p.off_theta = take(p.par_bytes);
  p.off_U = take(p.par_bytes);
  p.off_ring = take((uint32_t)p.stages * RS_TILE_BYTES);
  p.off_S = take(16u * 2u * (uint32_t)p.pitchS);
  p.off_P = take(16u * 2u * (uint32_t)p.pitchP);
  p.off_W = take(16u * 2u * (uint32_t)p.pitchW);
  p.off_T = take(16u * RS_TLD * 4u);
  p.off_stat = take((2u * RS_WARPS * 16u + 64u) * 4u);
  p.smem = (size_t)off + 1024;
  p.ok = 1;
  return p;
}

ResidentWs resident_ws(const kvc_layer* L, int B) {
  ResidentWs w{};
  const size_t bh = (size_t)B * L->desc.H_kv, sl = (size_t)slots_per_pair(L, B);
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  w.off_py = take(bh * sl * 16 * D * sizeof(float));
  w.off_pml = take(bh * sl * 16 * sizeof(float2));
  w.off_cnt = take(bh * sizeof(unsigned long long));
  w.bytes = off;
  return w;
}

cudaError_t launch_resident(const kvc_layer* L, const DecodeArgs& a, const ResidentPlan& p, cudaStream_t st, bool* encoded) {
  const int H_kv = a.H_kv, m = L->m, n = a.n, R = a.R, B = a.B;
  *encoded = false;
  CUtensorMap tm[6];
  {
    // K_tilde, V_tilde as (channels, m rows of a block, blocks): rows past a block's last are zero-filled
    const uint64_t dims[3] = {(uint64_t)D, (uint64_t)m, (uint64_t)B * H_kv * R};
    const uint64_t str[2] = {256ull, (uint64_t)m * 256};
    const uint32_t box[3] = {64u, (uint32_t)RS_TILE_ROWS, 1u};
    if (!encode_tensor_map_bf16(&tm[0], a.Kc, 3, dims, str, box)) return cudaSuccess;
    if (!encode_tensor_map_bf16(&tm[1], a.Vc, 3, dims, str, box)) return cudaSuccess;
  }
  if (a.T > 0) {
    const uint64_t dims[3] = {(uint64_t)D, (uint64_t)a.T, (uint64_t)B * H_kv};
    const uint64_t str[2] = {256ull, (uint64_t)a.T_cap * 256};
    const uint32_t box[3] = {64u, (uint32_t)RS_TILE_ROWS, 1u};
    if (!encode_tensor_map_bf16(&tm[2], a.K_txt, 3, dims, str, box)) return cudaSuccess;
    if (!encode_tensor_map_bf16(&tm[3], a.V_txt, 3, dims, str, box)) return cudaSuccess;
  } else {
    tm[2] = tm[0];
    tm[3] = tm[1];
  }
  {
    // theta, U [H_kv][m][n] viewed as (64 columns, m rows, n/64 column panels, H_kv): a box lands as [panel][row][64]
    const uint64_t dims[4] = {64ull, (uint64_t)m, (uint64_t)p.ncg, (uint64_t)H_kv};
    const uint64_t str[3] = {(uint64_t)n * 2, 128ull, (uint64_t)m * n * 2};
    const uint32_t box[4] = {64u, (uint32_t)p.mp, (uint32_t)p.ncg, 1u};
    if (!encode_tensor_map_bf16(&tm[4], a.theta, 4, dims, str, box)) return cudaSuccess;
    if (!encode_tensor_map_bf16(&tm[5], a.U, 4, dims, str, box)) return cudaSuccess;
  }
  *encoded = true;
  const ResidentWs w = resident_ws(L, B);
  char* ws = static_cast<char*>(a.resident_base);
  ResidentArgs ra{};
  ra.q = static_cast<const __nv_bfloat16*>(a.q);
  ra.mu = static_cast<const __nv_bfloat16*>(a.mu);
  ra.out = static_cast<__nv_bfloat16*>(a.out);
  ra.py = reinterpret_cast<float*>(ws + w.off_py);
  ra.pml = reinterpret_cast<float2*>(ws + w.off_pml);
  ra.cnt = reinterpret_cast<unsigned long long*>(ws + w.off_cnt);
  ra.token = a.token;
  ra.status = a.status;
  ra.B = B; ra.H_kv = H_kv; ra.G = a.G; ra.R = R; ra.m = m; ra.mp = p.mp; ra.n = n; ra.T = a.T;
  ra.ncg = p.ncg; ra.kt = p.kt; ra.ct = p.ct; ra.items_b = p.items_b; ra.cph = p.cph; ra.stages = p.stages;
  ra.slots = slots_per_pair(L, B);
  ra.pitchS = p.pitchS; ra.pitchP = p.pitchP; ra.pitchW = p.pitchW;
  ra.par_bytes = p.par_bytes;
  ra.off_theta = p.off_theta; ra.off_U = p.off_U; ra.off_ring = p.off_ring; ra.off_S = p.off_S; ra.off_P = p.off_P;
  ra.off_W = p.off_W; ra.off_T = p.off_T; ra.off_stat = p.off_stat;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(resident_decode_kernel), p.smem);
  if (e != cudaSuccess) return e;
  ProfScope prof(KVC_KERNEL_RESIDENT, st);
  return launch_dependent(resident_decode_kernel, dim3(p.grid), dim3(RS_THREADS), p.smem, st, tm[0], tm[1], tm[2], tm[3], tm[4],
                          tm[5], ra);
}

}  // namespace kvc
