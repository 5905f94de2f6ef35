// Value compression on the 5th-generation tensor cores (bf16 storage): V_tilde[b,h,r] = U[h] (V[b,h,r] - 1 mu[h]^T),
// Sec. 3.1 "Sequence-Level Low-Rank Compression for Values", taken as  U V - (U 1) mu^T  with the row sums of U
// computed once per layer.  One CTA produces a [128 rows of U] x [128 channels] tile of one block:
//   producer warp   streams 64-column slices of U[h] and the matching 64 rows of the block's V through a ring of
//                   TMA-filled stages (128-byte swizzle)
//   MMA warp        one thread issues tcgen05.mma M = 128, N = 128, K = 16: the U slice is the K-major A operand, the V
//                   rows (channels contiguous) the MN-major B operand, read as the TMA engine laid them down; the
//                   accumulator (128 lanes x 128 fp32 columns) lives in tensor memory; tcgen05.commit frees the stages
//   warps 0-3       epilogue: one lane per output row reads the accumulator back, subtracts usum[j] mu[c], rounds to
//                   bf16 and stores the row
// Two CTAs fit an SM (3 stages of 32 KB, 128 tensor-memory columns each), so one CTA's epilogue overlaps the other's
// main loop.
#include "kvc_tma.cuh"
#include "kvc_tcgen05.cuh"
#include "kvc_internal.cuh"

namespace kvc {

constexpr int CT_STAGES = 3;
constexpr int CT_BM = 128, CT_BK = 64;
constexpr uint32_t CT_U_BYTES = CT_BM * CT_BK * 2;          // 16 KB
constexpr uint32_t CT_V_HALF = CT_BK * 64 * 2;              // 8 KB: 64 rows x 64 channels
constexpr uint32_t CT_STAGE = CT_U_BYTES + 2 * CT_V_HALF;   // 32 KB
constexpr uint32_t CT_TMEM_COLS = 128;

struct CompressTcArgs {
  __nv_bfloat16* Vc;        // [B*H_kv*R][m][D]
  const float* usum;        // [H_kv][m] row sums of U
  const __nv_bfloat16* mu;  // [H_kv][D]
  int H_kv, R, n, m, mtiles, blocks;   // blocks = B*H_kv*R
  int* status;
};

__global__ void __launch_bounds__(6 * 32, 2)
project_values_tc_kernel(const __grid_constant__ CUtensorMap tmU, const __grid_constant__ CUtensorMap tmV, const CompressTcArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* sm = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
  __shared__ __align__(8) uint64_t full_bar[CT_STAGES], empty_bar[CT_STAGES], done_bar;
  __shared__ uint32_t s_tmem;
  __shared__ float s_mu[D];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // CTA -> (KV head, sequence, block, row tile): consecutive CTAs share U[h]
  const int mt = blockIdx.x % a.mtiles;
  const int rest = blockIdx.x / a.mtiles;              // = (h * B + b) * R + r
  const int per_h = a.blocks / a.H_kv;                 // B * R
  const int h = rest / per_h, br = rest - h * per_h;
  const int b = br / a.R, r = br - b * a.R;
  const int bhr = (b * a.H_kv + h) * a.R + r;
  const int nk = a.n / CT_BK;

  if (tid == 0) {
    for (int s = 0; s < CT_STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(&done_bar, 1);
    fence_mbar_init();
  }
  if (warp == 4) tmem_alloc(&s_tmem, CT_TMEM_COLS);
  if (tid < D) s_mu[tid] = __bfloat162float(a.mu[h * D + tid]);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = s_tmem;

  if (warp == 5) {
    // ---------------- producer ----------------
    if (lane == 0) {
      tma_prefetch_desc(&tmU); tma_prefetch_desc(&tmV);
      uint32_t slot = 0, phase = 1;
      for (int kc = 0; kc < nk; ++kc) {
        if (!mbar_wait_bounded(&empty_bar[slot], phase)) { atomicExch(a.status, (int)KVC_ERR_TIMEOUT); break; }
        unsigned char* dst = sm + slot * CT_STAGE;
        mbar_expect_tx(&full_bar[slot], CT_STAGE);
        tma_load_3d(dst, &tmU, kc * CT_BK, mt * CT_BM, h, &full_bar[slot]);
        tma_load_2d(dst + CT_U_BYTES, &tmV, 0, bhr * a.n + kc * CT_BK, &full_bar[slot]);
        tma_load_2d(dst + CT_U_BYTES + CT_V_HALF, &tmV, 64, bhr * a.n + kc * CT_BK, &full_bar[slot]);
        if (++slot == CT_STAGES) { slot = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 4) {
    // ---------------- MMA issue ----------------
    const uint32_t idesc = umma_idesc_bf16(128, 128, 0, 1);
    const uint32_t sm_u = smem_addr(sm);
    uint32_t slot = 0, phase = 0;
    bool dead = false;
    for (int kc = 0; kc < nk; ++kc) {
      if (!dead && !mbar_wait_bounded(&full_bar[slot], phase)) dead = true;
      __syncwarp();
      tc_fence_after();
      if (lane == 0) {
        const uint32_t u_u = sm_u + slot * CT_STAGE, v_u = u_u + CT_U_BYTES;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          // A: rows of U, 16 of the slice's 64 columns; B: 16 rows of V (two groups of 8), 128 channels in two halves
          const uint64_t adesc = umma_smem_desc(u_u + (uint32_t)(ks * 32), 16u, 1024u, UMMA_LAYOUT_SW128);
          const uint64_t bdesc = umma_smem_desc(v_u + (uint32_t)(ks * 2048), CT_V_HALF, 1024u, UMMA_LAYOUT_SW128);
          umma_bf16(tb, adesc, bdesc, idesc, (kc | ks) ? 1u : 0u);
        }
        umma_commit(&empty_bar[slot]);
        if (kc == nk - 1) umma_commit(&done_bar);
      }
      __syncwarp();
      if (++slot == CT_STAGES) { slot = 0; phase ^= 1u; }
    }
    if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
  } else {
    // ---------------- epilogue: V_tilde[j][c] = acc - usum[j] * mu[c] ----------------
    const bool ok = mbar_wait_bounded(&done_bar, 0);
    __syncwarp();
    tc_fence_after();
    const int j = mt * CT_BM + warp * 32 + lane;
    const float us = j < a.m ? a.usum[h * a.m + j] : 0.f;
    __nv_bfloat16* outp = a.Vc + ((size_t)bhr * a.m + (j < a.m ? j : 0)) * D;
#pragma unroll
    for (int c0 = 0; c0 < D; c0 += 16) {
      float v[16];
      tmem_ld_x16(tb + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
      if (j < a.m && ok) {
        uint32_t w[8];
#pragma unroll
        for (int k = 0; k < 8; ++k)
          w[k] = pack2_bf16(fmaf(-us, s_mu[c0 + 2 * k], v[2 * k]), fmaf(-us, s_mu[c0 + 2 * k + 1], v[2 * k + 1]));
        *reinterpret_cast<uint4*>(outp + c0) = make_uint4(w[0], w[1], w[2], w[3]);
        *reinterpret_cast<uint4*>(outp + c0 + 8) = make_uint4(w[4], w[5], w[6], w[7]);
      }
    }
    if (!ok && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 4) tmem_dealloc(tb, CT_TMEM_COLS);
}

// bf16, n a multiple of 64, 16-byte aligned pointers; *used == false if this path does not apply
cudaError_t launch_project_values_tc(const kvc_layer* L, const void* V_vis, int B, int R, void* Vc, cudaStream_t st, bool* used) {
  *used = false;
  const int n = L->desc.n, m = L->m, H_kv = L->desc.H_kv;
  if (L->desc.dtype != KVC_BF16 || n % CT_BK != 0 || !L->d_usum) return cudaSuccess;
  if ((reinterpret_cast<uintptr_t>(V_vis) | reinterpret_cast<uintptr_t>(Vc) | reinterpret_cast<uintptr_t>(L->desc.U) |
       reinterpret_cast<uintptr_t>(L->desc.mu)) & 15)
    return cudaSuccess;
  const long long rows_v = (long long)B * H_kv * R * n;
  if (rows_v >= (1ll << 31)) return cudaSuccess;
  CUtensorMap tmU, tmV;
  {
    const uint64_t dims[3] = {(uint64_t)n, (uint64_t)m, (uint64_t)H_kv};
    const uint64_t str[2] = {(uint64_t)n * 2, (uint64_t)m * n * 2};
    const uint32_t box[3] = {64u, (uint32_t)CT_BM, 1u};
    if (!encode_tensor_map_bf16(&tmU, L->desc.U, 3, dims, str, box)) return cudaSuccess;
  }
  {
    const uint64_t dims[2] = {(uint64_t)D, (uint64_t)rows_v};
    const uint64_t str[1] = {256ull};
    const uint32_t box[2] = {64u, (uint32_t)CT_BK};
    if (!encode_tensor_map_bf16(&tmV, V_vis, 2, dims, str, box)) return cudaSuccess;
  }
  *used = true;
  CompressTcArgs a{};
  a.Vc = static_cast<__nv_bfloat16*>(Vc);
  a.usum = L->d_usum;
  a.mu = static_cast<const __nv_bfloat16*>(L->desc.mu);
  a.H_kv = H_kv; a.R = R; a.n = n; a.m = m;
  a.mtiles = ceil_div(m, CT_BM);
  a.blocks = B * H_kv * R;
  a.status = L->d_cstatus;
  const size_t smem = (size_t)CT_STAGES * CT_STAGE + 1024;
  {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(project_values_tc_kernel), smem);
    if (e != cudaSuccess) return e;
  }
  project_values_tc_kernel<<<(unsigned)(a.blocks * a.mtiles), 6 * 32, smem, st>>>(tmU, tmV, a);
  return cudaGetLastError();
}

}  // namespace kvc
