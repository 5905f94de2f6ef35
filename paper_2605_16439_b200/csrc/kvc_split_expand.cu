// Split path, second kernel: Alg. 1 steps 2 and 3 for 128 expansion rows of a KV head and one range [n0, n0 + NW) of
// the n positions of a block, as two dense products on tcgen05 with the accumulators in tensor memory:
//   L[128 x NW]  = S[128 x m] theta[h][m x range]            A = S tile (K-major), B = theta rows (MN-major)
//   P = 2^(L - rowmax) (bf16, in shared memory as the next A operand), rowsum
//   Wp[128 x m]  = P[128 x NW] U[h][m x range]^T              A = P (K-major), B = rows of U (K-major), in passes of
//                                                             at most 512 columns; the logits' columns are reused
// Every operand tile is read as the TMA engine lays it down (128-byte swizzle).  The partial weights of the range, still
// relative to the range's own row maximum, go to the workspace as bf16 with (rowmax, rowsum); the output kernel joins the
// ranges of a row.  One CTA per (KV head, row tile, range); warps 0-3 = one lane per expansion row (softmax, epilogue),
// warp 4 = MMA issue, warp 5 = TMA producer.
#include "kvc_split.cuh"
#include "kvc_tcgen05.cuh"

namespace kvc {

constexpr int SE_THREADS = 6 * 32;

struct ExpandBars {
  uint64_t full[SP_MAX_STAGES], empty[SP_MAX_STAGES];
  uint64_t l_done;      // the logits are complete in tensor memory
  uint64_t p_ready;     // the probabilities are in shared memory and the logits have been read (4 warps)
  uint64_t w_done;      // a pass of the weights is complete
  uint64_t w_free;      // a pass of the weights has been read back (4 warps)
};

__global__ void __launch_bounds__(SE_THREADS, 1)
split_expand_kernel(const __grid_constant__ CUtensorMap tmS, const __grid_constant__ CUtensorMap tmTh,
                    const __grid_constant__ CUtensorMap tmU, const __grid_constant__ CUtensorMap tmWs, const SplitArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* sm = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
  __shared__ __align__(8) ExpandBars bars;
  __shared__ uint32_t s_tmem;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

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
    mbar_init(&bars.p_ready, 4);
    mbar_init(&bars.w_done, 1);
    mbar_init(&bars.w_free, 4);
    fence_mbar_init();
  }
  if (warp == 4) tmem_alloc(&s_tmem, (uint32_t)a.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = s_tmem;
  const uint32_t th_bytes = (uint32_t)ngrp * 8192u;    // theta rows of a chunk: [group][64 rows][128 B]
  const uint32_t u_box = (uint32_t)a.brow * 128u;

  if (warp == 5) {
    // ---------------- producer ----------------
    if (lane == 0) {
      tma_prefetch_desc(&tmS); tma_prefetch_desc(&tmTh); tma_prefetch_desc(&tmU);
      uint32_t slot = 0, phase = 1;
      bool waited = false;
      bool ok = true;
      for (int kc = 0; kc < a.nk1 && ok; ++kc) {
        if (!mbar_wait_bounded(&bars.empty[slot], phase)) { ok = false; break; }
        unsigned char* dst = ring + slot * a.e_stage_bytes;
        mbar_expect_tx(&bars.full[slot], 16384u + th_bytes);
        tma_load_4d(dst + 16384, &tmTh, 0, kc * 64, n0 >> 6, h, &bars.full[slot]);   // parameters: never written by the library
        if (!waited) {
          grid_dep_wait();                    // the scores come from the kernel before
          grid_dep_launch();                  // only now: the output kernel relies on that kernel being complete
          waited = true;
        }
        tma_load_3d(dst, &tmS, kc * 64, tile * SP_TILE_ROWS, h, &bars.full[slot]);
        if (++slot == (uint32_t)a.e_stages) { slot = 0; phase ^= 1u; }
      }
      for (int wp = 0; wp < a.npass && ok; ++wp)
        for (int kc = 0; kc < ngrp && ok; ++kc) {
          if (!mbar_wait_bounded(&bars.empty[slot], phase)) { ok = false; break; }
          unsigned char* dst = ring + slot * a.e_stage_bytes;
          mbar_expect_tx(&bars.full[slot], (uint32_t)a.nbox * u_box);
          for (int bx = 0; bx < a.nbox; ++bx)
            tma_load_3d(dst + bx * u_box, &tmU, n0 + kc * 64, wp * a.prow + bx * a.brow, h, &bars.full[slot]);
          if (++slot == (uint32_t)a.e_stages) { slot = 0; phase ^= 1u; }
        }
      if (!ok) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
    }
  } else if (warp == 4) {
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
    for (int kc = 0; kc < a.nk1; ++kc) {
      wait_on(&bars.full[slot], phase);
      tc_fence_after();
      if (lane == 0) {
        const uint32_t s_u = ring_u + slot * a.e_stage_bytes, th_u = s_u + 16384u;
        const int ksteps = min(4, (a.m - kc * 64 + 15) >> 4);
        for (int ks = 0; ks < ksteps; ++ks) {
          const uint64_t adesc = umma_smem_desc(s_u + (uint32_t)(ks * 32), 16u, 1024u, UMMA_LAYOUT_SW128);
          const uint64_t bdesc = umma_smem_desc(th_u + (uint32_t)(ks * 2048), 8192u, 1024u, UMMA_LAYOUT_SW128);
          umma_bf16(tb, adesc, bdesc, idesc_L, (kc | ks) ? 1u : 0u);
        }
        umma_commit(&bars.empty[slot]);
        if (kc == a.nk1 - 1) umma_commit(&bars.l_done);
      }
      __syncwarp();
      if (++slot == (uint32_t)a.e_stages) { slot = 0; phase ^= 1u; }
    }
    wait_on(&bars.p_ready, 0);
    for (int wp = 0; wp < a.npass; ++wp) {
      if (wp > 0) wait_on(&bars.w_free, (uint32_t)((wp - 1) & 1));
      tc_fence_after();
      for (int kc = 0; kc < ngrp; ++kc) {
        wait_on(&bars.full[slot], phase);
        tc_fence_after();
        if (lane == 0) {
          const uint32_t u_u = ring_u + slot * a.e_stage_bytes;
          const uint32_t p_u = sm_u + (uint32_t)kc * 16384u;
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            const uint64_t adesc = umma_smem_desc(p_u + (uint32_t)(ks * 32), 16u, 1024u, UMMA_LAYOUT_SW128);
            for (int bx = 0; bx < a.nbox; ++bx) {
              const uint64_t bdesc = umma_smem_desc(u_u + bx * u_box + (uint32_t)(ks * 32), 16u, 1024u, UMMA_LAYOUT_SW128);
              umma_bf16(tb + (uint32_t)(bx * a.brow), adesc, bdesc, idesc_W, (kc | ks) ? 1u : 0u);
            }
          }
          umma_commit(&bars.empty[slot]);
          if (kc == ngrp - 1) umma_commit(&bars.w_done);
        }
        __syncwarp();
        if (++slot == (uint32_t)a.e_stages) { slot = 0; phase ^= 1u; }
      }
    }
    if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
  } else {
    // ---------------- warps 0-3: lane <-> expansion row ----------------
    const int row = warp * 32 + lane;                          // row of the tile = tensor-memory lane
    const long long rho = (long long)tile * SP_TILE_ROWS + row;
    const bool valid = rho < a.rows_h;
    const uint32_t trow = tb + ((uint32_t)(warp * 32) << 16);
    bool ok = mbar_wait_bounded(&bars.l_done, 0);
    __syncwarp();
    tc_fence_after();
    // pass 1: row maximum over the range (32 columns per load, the next load in flight while one is reduced)
    float mx = -INFINITY;
    {
      uint32_t ra[32], rb[32];
      tmem_ld_issue_x32(trow, ra);
      for (int c0 = 0; c0 < a.NW; c0 += 64) {
        tmem_ld_wait_x32(ra);
        tmem_ld_issue_x32(trow + (uint32_t)(c0 + 32), rb);
#pragma unroll
        for (int k = 0; k < 32; ++k) mx = fmaxf(mx, __uint_as_float(ra[k]));
        tmem_ld_wait_x32(rb);
        if (c0 + 64 < a.NW) tmem_ld_issue_x32(trow + (uint32_t)(c0 + 64), ra);
#pragma unroll
        for (int k = 0; k < 32; ++k) mx = fmaxf(mx, __uint_as_float(rb[k]));
      }
    }
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
      for (int c0 = 0; c0 < a.NW; c0 += 32) {
        tmem_ld_issue_x32(trow + (uint32_t)c0, ra);
        tmem_ld_wait_x32(ra);
        emit(c0, ra);
      }
    }
    if (valid && ok) a.stat[((size_t)h * a.NS + s) * a.rows_h + rho] = make_float2(mx, sum);
    fence_proxy_async();                                       // P is read by the tensor core (async proxy)
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(&bars.p_ready);
    // the weights of the range, pass by pass.  The last pass goes through the shared memory of P (dead by then): 64-column
    // tiles in the swizzled row layout, stored by the TMA engine (rows and columns outside the tensor are clipped);
    // earlier passes (retained lengths above 512) store from registers.
    __nv_bfloat16* wrow = a.Wp + (((size_t)h * a.NS + s) * a.rows_h + (valid ? rho : 0)) * a.ms;
    const int ntile = a.NW >> 6;                                 // staging tiles of 16 KB in the region of P
    for (int wp = 0; wp < a.npass; ++wp) {
      if (ok && !mbar_wait_bounded(&bars.w_done, (uint32_t)(wp & 1))) ok = false;
      __syncwarp();
      tc_fence_after();
      const int j0 = wp * a.prow;
      if (wp == a.npass - 1) {
        int cg = 0;
        for (int c0 = 0; c0 < a.prow && j0 + c0 < a.m; c0 += 64, ++cg) {
          unsigned char* tile_sm = sm + (uint32_t)(cg % ntile) * 16384u;
          if (cg >= ntile) {                                     // the store that last read this tile has to be done with it
            if (tid == 0) { if (ntile >= 4) bulk_wait_group_read<3>(); else if (ntile >= 2) bulk_wait_group_read<1>(); else bulk_wait_group_read<0>(); }
            named_barrier_sync(2, 128);
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
          named_barrier_sync(2, 128);
          if (tid == 0 && ok) {
            tma_store_4d(&tmWs, tile_sm, j0 + c0, tile * SP_TILE_ROWS, s, h);
            bulk_commit_group();
          }
        }
        if (tid == 0) bulk_wait_group_all();
      } else {
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
  if (warp == 4) tmem_dealloc(tb, (uint32_t)a.tmem_cols);
}

cudaError_t launch_split_expand(const CUtensorMap& tmS, const CUtensorMap& tmTh, const CUtensorMap& tmU, const CUtensorMap& tmWs,
                                const SplitArgs& a, const SplitPlan& p, cudaStream_t st) {
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(split_expand_kernel), p.e_smem);
  if (e != cudaSuccess) return e;
  ProfScope prof(KVC_KERNEL_SPLIT_EXPAND, st);
  return launch_dependent(split_expand_kernel, dim3(p.e_grid), dim3(SE_THREADS), p.e_smem, st, tmS, tmTh, tmU, tmWs, a);
}

}  // namespace kvc
