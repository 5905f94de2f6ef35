// Resident-parameter decode kernel (see kvc_resident.cuh): Algorithm 1 for short blocks in one kernel.  Per work item,
// with the products taken transposed so that the long axis is the M side of mma.sync m16n8k16 and the (up to 8) query
// heads of the KV head are its N side:
//   vision block r:  S^T[m x G] = K_tilde_r q^T          (step 1; A = key rows as stored, B = the queries)
//                    L^T[n x G] = theta^T S^T            (step 2; A = theta read transposed from shared memory)
//                    P = 2^(L - M), M the running maximum of the (sequence, query head)
//                    W^T[m x G] = U P^T                  (step 3; A = U as stored)
//                    y^T[d x G] += V_tilde_r^T W^T       (step 4; A = value rows read transposed)
//   text chunk:      s^T = K_txt q^T, p = 2^(s - M), y^T += V_txt^T p^T
// The accumulator of one product becomes the B operand of the next without leaving the registers (bf16 pairs moved
// across the lanes by movmatrix).  A warp owns its items from the first key row to the last value row: it issues its own
// TMA loads into its own ring of 16-row pieces and waits on its own mbarriers, so the eight warps of a CTA run eight
// independent chains and hide each other's latencies.  theta[h] and U[h] are shared by the CTA and loaded once.
#include "kvc_fused.cuh"
#include "kvc_resident.cuh"

namespace kvc {

constexpr int RS_THREADS = RS_WARPS * 32;
constexpr uint32_t RS_SMEM_LIMIT = 232448;
constexpr uint32_t RS_HALF = RS_PIECE_BYTES / 2;
constexpr float RS_QSCALE = 0.08838834764831845f * 1.4426950408889634f;      // sigma = 1/sqrt(128), logits in log2 units

// transpose of an 8 x 8 matrix of 16-bit elements held as one register per lane (row lane / 4, columns 2 (lane % 4), + 1)
__device__ __forceinline__ uint32_t movm_t(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(y) : "r"(x));
  return y;
}

// RAGGED: per-sequence block counts and text lengths are read from device arrays (the uniform instance carries none of that code)
template <int NT16, bool RAGGED>
__global__ void __launch_bounds__(RS_THREADS, 1)
resident_decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                       const __grid_constant__ CUtensorMap tmKt, const __grid_constant__ CUtensorMap tmVt,
                       const __grid_constant__ CUtensorMap tmTh, const __grid_constant__ CUtensorMap tmU,
                       const ResidentArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* sm = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
  __shared__ __align__(8) uint64_t full_bar[RS_WARPS][RS_MAX_SLOTS], par_bar;
  __shared__ int s_last;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int h = blockIdx.x / a.cph, c = blockIdx.x - h * a.cph;
  const int units_h = a.B * a.cpb;
  const int np = a.mp / 16, G = a.G;
  if (tid == 0) {
    for (int w = 0; w < RS_WARPS; ++w)
      for (int s = 0; s < RS_MAX_SLOTS; ++s) mbar_init(&full_bar[w][s], 1);
    mbar_init(&par_bar, 1);
    fence_mbar_init();
  }
  __syncthreads();
  if (tid == 0 && c < units_h) {
    tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmTh); tma_prefetch_desc(&tmU);
    if (a.T > 0) { tma_prefetch_desc(&tmKt); tma_prefetch_desc(&tmVt); }
    // the parameters of the head: fixed at inference (Sec. 3.2), so they need not wait for the stream's previous kernel
    mbar_expect_tx(&par_bar, 2u * a.par_bytes);
    tma_load_4d(sm + a.off_theta, &tmTh, 0, 0, 0, h, &par_bar);
    tma_load_4d(sm + a.off_U, &tmU, 0, 0, 0, h, &par_bar);
  }
  // Everything the stream's previous kernel may have written (queries, text rows, workspace) is touched only after the
  // dependency wait; the capsule rows are not among it when a.early is set, and their first pieces are asked for at once.
  bool waited = false;
  auto dep_wait = [&]() {
    if (waited) return;
    grid_dep_wait();
    grid_dep_launch();
    if (blockIdx.x == 0 && tid == 0) *a.status = 0;
    waited = true;
  };
  constexpr bool ragged = RAGGED;                               // the lengths are inputs like the queries: read after the wait
  if (!a.early || ragged) dep_wait();
  if (ragged) __syncthreads();                                  // the status word is cleared before a length is reported
  if (ragged && blockIdx.x == 0)
    for (int bb = tid; bb < a.B; bb += RS_THREADS) {
      const bool bad = (a.R_b && (a.R_b[bb] < 0 || a.R_b[bb] > a.R)) || (a.T_b && (a.T_b[bb] < 0 || a.T_b[bb] > a.T));
      if (bad) atomicExch(a.status, (int)KVC_ERR_BOUNDS);
    }

  const uint32_t sm_u = smem_addr(sm);
  const uint32_t th_u = sm_u + a.off_theta, U_u = sm_u + a.off_U;
  const uint32_t panel = (uint32_t)a.mp * 128u;                  // bytes of one 64-column panel of theta / U
  // ldmatrix lane roles: the lane supplies the address of row (lane & 7) of 8 x 8 matrix (lane >> 3)
  const int r8 = lane & 7, mat = lane >> 3;
  const int rowA = r8 + (mat & 1) * 8, selA = mat >> 1;          // plain: matrices (rows 0-7 | 8-15) x (k 0-7 | 8-15)
  const int rowT = r8 + (mat >> 1) * 8, selT = mat & 1;          // transposed: stored rows are the k index

  uint32_t pbits = 0;                                            // parity of the next completion of each of this warp's slots
  bool dead = false, par_ready = false;

  for (int u = c; u < units_h; u += a.cph) {
    const int b = u / a.cpb, part = u - b * a.cpb, bh = b * a.H_kv + h;
    const int ulo = part * a.items_b / a.cpb, uhi = (part + 1) * a.items_b / a.cpb;
    const int ni = uhi - ulo;
    // blocks and text rows this sequence takes part with; an item beyond them is skipped (no loads, no arithmetic)
    int Rb = a.R, Tb = a.T;
    if (RAGGED && a.R_b) { Rb = a.R_b[b]; Rb = Rb < 0 ? 0 : (Rb > a.R ? a.R : Rb); }
    if (RAGGED && a.T_b) { Tb = a.T_b[b]; Tb = Tb < 0 ? 0 : (Tb > a.T ? a.T : Tb); }
    auto valid = [&](int k) { return !RAGGED || (k < a.R ? k < Rb : (k - a.R) * RS_TEXT_ROWS < Tb); };
    const int wlo = ulo + ni * warp / RS_WARPS, whi = ulo + ni * (warp + 1) / RS_WARPS;
    // the ring pieces of the CTA go to the warps that have items in this unit (with fewer than 8 items: one item each)
    const int nact = ni < RS_WARPS ? ni : RS_WARPS;
    const int nsl = a.slots / nact < RS_MAX_SLOTS ? a.slots / nact : RS_MAX_SLOTS;
    auto region = [&](int w) { return (size_t)(ni < RS_WARPS ? ni * w / RS_WARPS : w) * nsl * RS_PIECE_BYTES; };
    unsigned char* ring_p = sm + a.off_ring + region(warp);
    const uint32_t ring_u = smem_addr(ring_p);
    uint32_t use_slot = 0, iss_slot = 0;                         // slots of the next piece consumed / issued by this warp

    // ---- this warp's load stream: the pieces of its items in the order it consumes them
    int p_k = wlo, p_idx = 0;
    auto issue_next = [&]() {
      if (p_idx == 0) while (p_k < whi && !valid(p_k)) ++p_k;
      if (p_k >= whi) return;
      const bool vis = p_k < a.R;
      const int half = vis ? np : RS_TEXT_ROWS / RS_PIECE_ROWS;
      if (!vis) dep_wait();
      if (lane == 0) {
        unsigned char* dst = ring_p + iss_slot * RS_PIECE_BYTES;
        uint64_t* bar = &full_bar[warp][iss_slot];
        const bool second = p_idx >= half;
        const int piece = second ? p_idx - half : p_idx;
        const CUtensorMap* tm = vis ? (second ? &tmV : &tmK) : (second ? &tmVt : &tmKt);
        const int row0 = vis ? piece * RS_PIECE_ROWS : (p_k - a.R) * RS_TEXT_ROWS + piece * RS_PIECE_ROWS;
        const int idx3 = vis ? bh * a.R + p_k : bh;
        mbar_expect_tx(bar, RS_PIECE_BYTES);
        tma_load_4d(dst, tm, 0, row0, 0, idx3, bar);               // both 64-channel halves of the 16 rows in one copy
      }
      if (++iss_slot == (uint32_t)nsl) iss_slot = 0;
      if (++p_idx == 2 * half) { p_idx = 0; ++p_k; }
    };
    auto wait_piece = [&]() -> uint32_t {
      const uint32_t slot = use_slot, parity = (pbits >> slot) & 1u;
      if (!mbar_test_wait(&full_bar[warp][slot], parity))          // usually complete already: one immediate look first
        if (!dead && !mbar_wait_bounded(&full_bar[warp][slot], parity)) dead = true;
      pbits ^= 1u << slot;
      __syncwarp();
      return ring_u + slot * RS_PIECE_BYTES;
    };
    // every lane has read the piece (ldmatrix has returned its data): its slot takes the next load of the stream
    auto done_piece = [&]() {
      __syncwarp();
      if (++use_slot == (uint32_t)nsl) use_slot = 0;
      issue_next();
    };
    for (int s = 0; s < nsl; ++s) issue_next();
    dep_wait();

    float yacc[8][4];
#pragma unroll
    for (int x = 0; x < 8; ++x)
#pragma unroll
      for (int e = 0; e < 4; ++e) yacc[x][e] = 0.f;
    float rM0 = -INFINITY, rM1 = -INFINITY, rL0 = 0.f, rL1 = 0.f, rV0 = 0.f, rV1 = 0.f;   // query heads 2t and 2t + 1
    uint32_t qb[8][2];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) { qb[ks][0] = 0u; qb[ks][1] = 0u; }
    if (wlo < whi && g < G) {
      // B fragments of the score product: k = the 128 channels, n = the query heads of the group (zero beyond G)
      const __nv_bfloat16* q0 = a.q + ((size_t)b * a.H_kv * G + (size_t)h * G + g) * D;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        qb[ks][0] = *reinterpret_cast<const uint32_t*>(q0 + ks * 16 + 2 * t);
        qb[ks][1] = *reinterpret_cast<const uint32_t*>(q0 + ks * 16 + 8 + 2 * t);
      }
    }
    // scores of one 16-row piece against the queries: v[0..3] = (row g, heads 2t, 2t+1), (row g + 8, heads 2t, 2t+1)
    auto score_piece = [&](uint32_t st, float (&v)[4]) {
      float c[4][4];                                // four chains of two products each
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) c[i][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const int cc = 2 * ks + selA;               // 16-byte piece of the 256-byte row
        uint32_t af[4];
        ldsm_x4(af, st + (uint32_t)(cc >> 3) * RS_HALF + (uint32_t)rowA * 128u + (uint32_t)(((cc & 7) ^ (rowA & 7)) << 4));
        mma_bf16_16816(c[ks & 3], af, qb[ks][0], qb[ks][1]);
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) v[e] = ((c[0][e] + c[1][e]) + (c[2][e] + c[3][e])) * RS_QSCALE;
    };
    // y^T += (value rows of the piece)^T times the B fragment (k = the 16 rows, n = the heads)
    auto value_piece = [&](uint32_t st, uint32_t b0, uint32_t b1) {
#pragma unroll
      for (int ct = 0; ct < 8; ++ct) {
        const int cch = 2 * ct + selT;
        uint32_t af[4];
        ldsm_x4_t(af, st + (uint32_t)(cch >> 3) * RS_HALF + (uint32_t)rowT * 128u + (uint32_t)(((cch & 7) ^ (rowT & 7)) << 4));
        mma_bf16_16816(yacc[ct], af, b0, b1);
      }
    };
    auto rescale = [&](float cr0, float cr1) {
#pragma unroll
      for (int ct = 0; ct < 8; ++ct) { yacc[ct][0] *= cr0; yacc[ct][1] *= cr1; yacc[ct][2] *= cr0; yacc[ct][3] *= cr1; }
    };
    auto over_rows = [&](float& x0, float& x1, bool is_max) {     // reduction over the 8 row groups of a column (lanes g)
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) {
        const float y0 = __shfl_xor_sync(0xffffffffu, x0, o), y1 = __shfl_xor_sync(0xffffffffu, x1, o);
        x0 = is_max ? fmaxf(x0, y0) : x0 + y0;
        x1 = is_max ? fmaxf(x1, y1) : x1 + y1;
      }
    };

    for (int k = wlo; k < whi; ++k) {
      if (!valid(k)) continue;
      if (k < a.R) {
        // ---- step 1: S^T, kept as B fragments (k = key rows, n = heads)
        uint32_t Sb[RS_MAX_MP16][2];
#pragma unroll
        for (int pc = 0; pc < RS_MAX_MP16; ++pc) {
          Sb[pc][0] = 0u; Sb[pc][1] = 0u;
          if (pc < np) {
            float v[4];
            score_piece(wait_piece(), v);
            Sb[pc][0] = movm_t(pack2_bf16(v[0], v[1]));
            Sb[pc][1] = movm_t(pack2_bf16(v[2], v[3]));
            done_piece();
          }
        }
        if (!par_ready) {
          if (!dead && !mbar_wait_bounded(&par_bar, 0)) dead = true;
          par_ready = true;
        }
        // ---- step 2: L^T[n x G] = theta^T S^T, 16 positions per row tile; the row tiles are independent accumulators,
        // so the loop over them is the inner one
        float lacc[NT16][4];
#pragma unroll
        for (int it = 0; it < NT16; ++it)
#pragma unroll
          for (int e = 0; e < 4; ++e) lacc[it][e] = 0.f;
#pragma unroll
        for (int ks = 0; ks < RS_MAX_MP16; ++ks) {
          if (ks < np) {
            const int jrow = 16 * ks + rowT;
            const uint32_t rbase = th_u + (uint32_t)jrow * 128u;
#pragma unroll
            for (int it = 0; it < NT16; ++it) {
              const int ic = 2 * it + selT;
              uint32_t af[4];
              ldsm_x4_t(af, rbase + (uint32_t)(ic >> 3) * panel + (uint32_t)(((ic & 7) ^ (jrow & 7)) << 4));
              mma_bf16_16816(lacc[it], af, Sb[ks][0], Sb[ks][1]);
            }
          }
        }
        // ---- softmax pieces of the block relative to the running maximum of each head
        float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
        for (int it = 0; it < NT16; ++it) {
          m0 = fmaxf(m0, fmaxf(lacc[it][0], lacc[it][2]));
          m1 = fmaxf(m1, fmaxf(lacc[it][1], lacc[it][3]));
        }
        over_rows(m0, m1, true);
        const float Mn0 = fmaxf(rM0, m0), Mn1 = fmaxf(rM1, m1);
        const float cr0 = rM0 == -INFINITY ? 0.f : fast_exp2(rM0 - Mn0), cr1 = rM1 == -INFINITY ? 0.f : fast_exp2(rM1 - Mn1);
        float s0 = 0.f, s1 = 0.f;
        uint32_t Pb[NT16][2];
#pragma unroll
        for (int it = 0; it < NT16; ++it) {
          const float p0 = fast_exp2(lacc[it][0] - Mn0), p1 = fast_exp2(lacc[it][1] - Mn1);
          const float p2 = fast_exp2(lacc[it][2] - Mn0), p3 = fast_exp2(lacc[it][3] - Mn1);
          s0 += p0 + p2;
          s1 += p1 + p3;
          Pb[it][0] = movm_t(pack2_bf16(p0, p1));
          Pb[it][1] = movm_t(pack2_bf16(p2, p3));
        }
        over_rows(s0, s1, false);
        rL0 = rL0 * cr0 + s0; rL1 = rL1 * cr1 + s1;
        rV0 = rV0 * cr0 + s0; rV1 = rV1 * cr1 + s1;
        rM0 = Mn0; rM1 = Mn1;
        rescale(cr0, cr1);
        // ---- step 3: W^T[m x G] = U P^T, kept as B fragments for step 4 (two accumulators per row tile: the chain over
        // the n axis is the long one here)
        uint32_t Wb[RS_MAX_MP16][2];
#pragma unroll
        for (int jt = 0; jt < RS_MAX_MP16; ++jt) {
          Wb[jt][0] = 0u; Wb[jt][1] = 0u;
          if (jt < np) {
            float w0[4] = {0.f, 0.f, 0.f, 0.f}, w1[4] = {0.f, 0.f, 0.f, 0.f};
            const int jrow = 16 * jt + rowA;
            const uint32_t rbase = U_u + (uint32_t)jrow * 128u;
#pragma unroll
            for (int ks = 0; ks < NT16; ++ks) {
              const int ic = 2 * ks + selA;
              uint32_t af[4];
              ldsm_x4(af, rbase + (uint32_t)(ic >> 3) * panel + (uint32_t)(((ic & 7) ^ (jrow & 7)) << 4));
              if (ks & 1) mma_bf16_16816(w1, af, Pb[ks][0], Pb[ks][1]);
              else mma_bf16_16816(w0, af, Pb[ks][0], Pb[ks][1]);
            }
            Wb[jt][0] = movm_t(pack2_bf16(w0[0] + w1[0], w0[1] + w1[1]));
            Wb[jt][1] = movm_t(pack2_bf16(w0[2] + w1[2], w0[3] + w1[3]));
          }
        }
        // ---- step 4: y^T += V_tilde^T W^T
#pragma unroll
        for (int pc = 0; pc < RS_MAX_MP16; ++pc) {
          if (pc < np) {
            value_piece(wait_piece(), Wb[pc][0], Wb[pc][1]);
            done_piece();
          }
        }
      } else {
        // ---- text chunk of 64 rows
        const int base = (k - a.R) * RS_TEXT_ROWS;
        float sc[4][4];
#pragma unroll
        for (int pc = 0; pc < 4; ++pc) {
          score_piece(wait_piece(), sc[pc]);
          const int row = base + pc * RS_PIECE_ROWS + g;
          if (row >= Tb) { sc[pc][0] = -INFINITY; sc[pc][1] = -INFINITY; }
          if (row + 8 >= Tb) { sc[pc][2] = -INFINITY; sc[pc][3] = -INFINITY; }
          done_piece();
        }
        float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
        for (int pc = 0; pc < 4; ++pc) {
          m0 = fmaxf(m0, fmaxf(sc[pc][0], sc[pc][2]));
          m1 = fmaxf(m1, fmaxf(sc[pc][1], sc[pc][3]));
        }
        over_rows(m0, m1, true);
        const float Mn0 = fmaxf(rM0, m0), Mn1 = fmaxf(rM1, m1);
        const float cr0 = rM0 == -INFINITY ? 0.f : fast_exp2(rM0 - Mn0), cr1 = rM1 == -INFINITY ? 0.f : fast_exp2(rM1 - Mn1);
        float s0 = 0.f, s1 = 0.f;
        uint32_t Tb_frag[4][2];
#pragma unroll
        for (int pc = 0; pc < 4; ++pc) {
          const float p0 = fast_exp2(sc[pc][0] - Mn0), p1 = fast_exp2(sc[pc][1] - Mn1);
          const float p2 = fast_exp2(sc[pc][2] - Mn0), p3 = fast_exp2(sc[pc][3] - Mn1);
          s0 += p0 + p2;
          s1 += p1 + p3;
          Tb_frag[pc][0] = movm_t(pack2_bf16(p0, p1));
          Tb_frag[pc][1] = movm_t(pack2_bf16(p2, p3));
        }
        over_rows(s0, s1, false);
        rL0 = rL0 * cr0 + s0; rL1 = rL1 * cr1 + s1;
        rV0 *= cr0; rV1 *= cr1;
        rM0 = Mn0; rM1 = Mn1;
        rescale(cr0, cr1);
#pragma unroll
        for (int pc = 0; pc < 4; ++pc) {
          const uint32_t st = wait_piece();
          if (RAGGED && a.T_b) {
            // rows past the sequence's text length hold whatever the caller's buffer holds (a zero probability does not
            // silence a NaN): cleared in shared memory before the product
            const int nv = Tb - (base + pc * RS_PIECE_ROWS);
            if (nv < RS_PIECE_ROWS && lane < 16)
              for (int r = nv < 0 ? 0 : nv; r < RS_PIECE_ROWS; ++r)
                asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};\n" ::"r"(st + (uint32_t)(lane >> 3) * RS_HALF + (uint32_t)r * 128u + (uint32_t)(lane & 7) * 16u), "r"(0u) : "memory");
            fence_proxy_async();                   // the cleared rows precede the copy that refills the slot
            __syncwarp();
          }
          value_piece(st, Tb_frag[pc][0], Tb_frag[pc][1]);
          done_piece();
        }
      }
    }

    // ---- end of the unit: the warps' results meet in shared memory (each warp's ring is idle: all its pieces are consumed)
    float* segy = reinterpret_cast<float*>(ring_p);              // [8 heads][D]
    float* segs = segy + 8 * D;                                  // max[8], sum[8], vision sum[8], valid
    if (wlo < whi) {
#pragma unroll
      for (int ct = 0; ct < 8; ++ct) {
        const int ch = 16 * ct + g;
        segy[(2 * t) * D + ch] = yacc[ct][0];
        segy[(2 * t + 1) * D + ch] = yacc[ct][1];
        segy[(2 * t) * D + ch + 8] = yacc[ct][2];
        segy[(2 * t + 1) * D + ch + 8] = yacc[ct][3];
      }
      if (g == 0) {
        segs[2 * t] = rM0; segs[2 * t + 1] = rM1;
        segs[8 + 2 * t] = rL0; segs[8 + 2 * t + 1] = rL1;
        segs[16 + 2 * t] = rV0; segs[16 + 2 * t + 1] = rV1;
      }
    }
    __syncthreads();
    const int head = warp;                                      // merge: warp = query head, lane = 4 channels
    auto has_items = [&](int w) { return ni * (w + 1) / RS_WARPS > ni * w / RS_WARPS; };
    if (head < G) {
      float Mx = -INFINITY;
#pragma unroll
      for (int w = 0; w < RS_WARPS; ++w) {
        const float* ss = reinterpret_cast<const float*>(sm + a.off_ring + region(w)) + 8 * D;
        if (has_items(w)) Mx = fmaxf(Mx, ss[head]);
      }
      float Ls = 0.f, Vs = 0.f;
      float4 y = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int w = 0; w < RS_WARPS; ++w) {
        const float* sy = reinterpret_cast<const float*>(sm + a.off_ring + region(w));
        const float* ss = sy + 8 * D;
        if (has_items(w) && ss[head] != -INFINITY) {
          const float f = fast_exp2(ss[head] - Mx);
          Ls = fmaf(f, ss[8 + head], Ls);
          Vs = fmaf(f, ss[16 + head], Vs);
          const float4 v = *reinterpret_cast<const float4*>(sy + head * D + lane * 4);
          y.x = fmaf(f, v.x, y.x); y.y = fmaf(f, v.y, y.y); y.z = fmaf(f, v.z, y.z); y.w = fmaf(f, v.w, y.w);
        }
      }
      const uint2 mraw = *reinterpret_cast<const uint2*>(a.mu + h * D + lane * 4);     // the centring term (sum P) mu
      y.x = fmaf(Vs, __uint_as_float(mraw.x << 16), y.x);
      y.y = fmaf(Vs, __uint_as_float(mraw.x & 0xffff0000u), y.y);
      y.z = fmaf(Vs, __uint_as_float(mraw.y << 16), y.z);
      y.w = fmaf(Vs, __uint_as_float(mraw.y & 0xffff0000u), y.w);
      if (a.cpb == 1) {
        const float inv = Ls > 0.f ? 1.f / Ls : 0.f;          // a sequence without any row: a zero output row
        *reinterpret_cast<uint2*>(a.out + ((size_t)bh * G + head) * D + lane * 4) =
            make_uint2(pack2_bf16(y.x * inv, y.y * inv), pack2_bf16(y.z * inv, y.w * inv));
      } else {
        *reinterpret_cast<float4*>(a.py + (((size_t)bh * RS_MAX_CPB + part) * 8 + head) * D + lane * 4) = y;
        if (lane == 0) a.pml[((size_t)bh * RS_MAX_CPB + part) * 8 + head] = make_float2(Mx, Ls);
      }
    }
    if (a.cpb > 1) {
      __threadfence();
      __syncthreads();
      if (tid == 0) s_last = arrive_is_last(a.cnt + bh, a.token, a.cpb) ? 1 : 0;
      __syncthreads();
      if (s_last && head < G) {
        __threadfence();
        const float2* ml = a.pml + (size_t)bh * RS_MAX_CPB * 8 + head;
        const float* py = a.py + ((size_t)bh * RS_MAX_CPB * 8 + head) * D + lane * 4;
        float2 st[RS_MAX_CPB];
        float4 ys[RS_MAX_CPB];
#pragma unroll
        for (int s = 0; s < RS_MAX_CPB; ++s) {
          st[s] = make_float2(-INFINITY, 0.f);
          ys[s] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (s < a.cpb) {
            st[s] = __ldcg(ml + s * 8);
            ys[s] = __ldcg(reinterpret_cast<const float4*>(py + (size_t)s * 8 * D));
          }
        }
        float Ms = -INFINITY;
#pragma unroll
        for (int s = 0; s < RS_MAX_CPB; ++s) Ms = fmaxf(Ms, st[s].x);
        float den = 0.f;
        float4 y = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int s = 0; s < RS_MAX_CPB; ++s) {
          const float f = st[s].x == -INFINITY ? 0.f : fast_exp2(st[s].x - Ms);
          den = fmaf(f, st[s].y, den);
          y.x = fmaf(f, ys[s].x, y.x); y.y = fmaf(f, ys[s].y, y.y); y.z = fmaf(f, ys[s].z, y.z); y.w = fmaf(f, ys[s].w, y.w);
        }
        const float inv = den > 0.f ? 1.f / den : 0.f;
        *reinterpret_cast<uint2*>(a.out + ((size_t)bh * G + head) * D + lane * 4) =
            make_uint2(pack2_bf16(y.x * inv, y.y * inv), pack2_bf16(y.z * inv, y.w * inv));
      }
    }
    fence_proxy_async();                // the warps' results, written to their rings with ordinary stores, precede the copies
    __syncthreads();                    // the rings take the next unit's pieces
  }
  dep_wait();
  if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
}

// ---- host ------------------------------------------------------------------------------------------------------
ResidentPlan plan_resident(const kvc_layer* L, int B, int R, int T) {
  ResidentPlan p{};
  const int n = L->desc.n, m = L->m, G = L->G, H_kv = L->desc.H_kv;
  if (L->desc.dtype != KVC_BF16 || L->passthrough || L->mode != KVC_MODE_KV || R < 1 || B < 1 || n % 64 != 0 || n > 256 ||
      G > 8)
    return p;
  if ((reinterpret_cast<uintptr_t>(L->desc.theta) | reinterpret_cast<uintptr_t>(L->desc.U)) & 15) return p;
  p.mp = (m + 15) & ~15;
  if (p.mp > 16 * RS_MAX_MP16) return p;
  const int sms = L->num_sms > 0 ? L->num_sms : 148;
  p.ncg = n / 64;
  p.ct = ceil_div(T, RS_TEXT_ROWS);
  p.items_b = R + p.ct;
  long long cpb = sms / ((long long)B * H_kv);
  if (cpb > RS_MAX_CPB) cpb = RS_MAX_CPB;
  if (cpb > p.items_b) cpb = p.items_b;
  if (cpb < 1) cpb = 1;
  p.cpb = (int)cpb;
  const long long units_h = (long long)B * p.cpb;
  const int cmax = sms / H_kv > 0 ? sms / H_kv : 1;
  p.cph = (int)(units_h < cmax ? units_h : cmax);
  p.grid = p.cph * H_kv;
  p.par_bytes = (uint32_t)p.ncg * (uint32_t)p.mp * 128u;
  const uint32_t fixed = 2u * p.par_bytes + 1024u + 2048u;
  if (fixed + 3u * RS_WARPS * RS_PIECE_BYTES > RS_SMEM_LIMIT) return p;
  p.slots = (int)((RS_SMEM_LIMIT - fixed) / RS_PIECE_BYTES);
  if (p.slots > RS_MAX_SLOTS * RS_WARPS) p.slots = RS_MAX_SLOTS * RS_WARPS;
  if (p.slots < 3 * RS_WARPS) return p;            // a warp's region also stages its result (4 KB + statistics) at the end of a unit
  p.off_theta = 0;
  p.off_U = p.par_bytes;
  p.off_ring = 2u * p.par_bytes;
  p.smem = (size_t)p.off_ring + (size_t)p.slots * RS_PIECE_BYTES + 1024;
  p.ok = 1;
  return p;
}

ResidentWs resident_ws(const kvc_layer* L, int B) {
  ResidentWs w{};
  // partials exist only while several units share a (sequence, KV head), i.e. while there are fewer pairs than SMs
  const int sms = L->num_sms > 0 ? L->num_sms : 148;
  const size_t bh = (size_t)B * L->desc.H_kv;
  const size_t with_parts = bh <= (size_t)sms / 2 ? bh : 0;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  w.off_py = take(with_parts * RS_MAX_CPB * 8 * D * sizeof(float));
  w.off_pml = take(with_parts * RS_MAX_CPB * 8 * sizeof(float2));
  w.off_cnt = take(bh * sizeof(unsigned long long));
  w.bytes = off;
  return w;
}

cudaError_t launch_resident(const kvc_layer* L, const DecodeArgs& a, const ResidentPlan& p, cudaStream_t st, bool* encoded) {
  const int H_kv = a.H_kv, m = L->m, n = a.n, R = a.R, B = a.B;
  *encoded = false;
  CUtensorMap tm[6];
  {
    // K_tilde, V_tilde as (64 channels, m rows of a block, channel half, blocks): a box lands as [half][16 rows][64];
    // rows past a block's last are zero-filled
    const uint64_t dims[4] = {64ull, (uint64_t)m, 2ull, (uint64_t)B * H_kv * R};
    const uint64_t str[3] = {256ull, 128ull, (uint64_t)m * 256};
    const uint32_t box[4] = {64u, (uint32_t)RS_PIECE_ROWS, 2u, 1u};
    if (!encode_tensor_map_bf16(&tm[0], a.Kc, 4, dims, str, box)) return cudaSuccess;
    if (!encode_tensor_map_bf16(&tm[1], a.Vc, 4, dims, str, box)) return cudaSuccess;
  }
  if (a.T > 0) {
    const uint64_t dims[4] = {64ull, (uint64_t)a.T, 2ull, (uint64_t)B * H_kv};
    const uint64_t str[3] = {256ull, 128ull, (uint64_t)a.T_cap * 256};
    const uint32_t box[4] = {64u, (uint32_t)RS_PIECE_ROWS, 2u, 1u};
    if (!encode_tensor_map_bf16(&tm[2], a.K_txt, 4, dims, str, box)) return cudaSuccess;
    if (!encode_tensor_map_bf16(&tm[3], a.V_txt, 4, dims, str, box)) return cudaSuccess;
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
  ra.ncg = p.ncg; ra.ct = p.ct; ra.items_b = p.items_b; ra.cpb = p.cpb; ra.cph = p.cph; ra.slots = p.slots;
  ra.early = a.early_capsules;
  ra.R_b = a.R_b; ra.T_b = a.T_b;
  ra.par_bytes = p.par_bytes;
  ra.off_theta = p.off_theta; ra.off_U = p.off_U; ra.off_ring = p.off_ring;
  const bool rg = a.R_b != nullptr || a.T_b != nullptr;
  void (*kernel)(CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, ResidentArgs) =
      n == 64    ? (rg ? resident_decode_kernel<4, true> : resident_decode_kernel<4, false>)
      : n == 128 ? (rg ? resident_decode_kernel<8, true> : resident_decode_kernel<8, false>)
      : n == 192 ? (rg ? resident_decode_kernel<12, true> : resident_decode_kernel<12, false>)
                 : (rg ? resident_decode_kernel<16, true> : resident_decode_kernel<16, false>);
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), p.smem);
  if (e != cudaSuccess) return e;
  ProfScope prof(KVC_KERNEL_RESIDENT, st);
  return launch_dependent(kernel, dim3(p.grid), dim3(RS_THREADS), p.smem, st, tm[0], tm[1], tm[2], tm[3], tm[4], tm[5], ra);
}

}  // namespace kvc
