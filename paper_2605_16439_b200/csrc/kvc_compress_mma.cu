// Value compression on the tensor cores (bf16 storage): V_tilde[b,h,r] = U[h] (V[b,h,r] - 1 mu[h]^T), Sec. 3.1
// "Sequence-Level Low-Rank Compression for Values", taken as  U V - (U 1) mu^T  with the row sums of U computed
// once per layer.  One CTA produces a [128 rows of U] x [128 channels] tile of one block: a producer thread
// streams 64-column slices of U[h] and the matching 64 rows of the block's V through a ring of TMA-filled stages
// (128-byte swizzle), eight consumer warps (4 along the rows x 2 along the channels) run mma.sync m16n8k16.
#include "kvc_tma.cuh"
#include "kvc_internal.cuh"

namespace kvc {

constexpr int CM_STAGES = 4;
constexpr int CM_BM = 128, CM_BK = 64;
constexpr uint32_t CM_U_BYTES = CM_BM * CM_BK * 2;          // 16 KB
constexpr uint32_t CM_V_HALF = CM_BK * 64 * 2;              // 8 KB: 64 rows x 64 channels
constexpr uint32_t CM_STAGE = CM_U_BYTES + 2 * CM_V_HALF;   // 32 KB
constexpr int CM_WARPS = 8;

struct CompressArgs {
  __nv_bfloat16* Vc;        // [B*H_kv*R][m][D]
  const float* usum;        // [H_kv][m] row sums of U
  const __nv_bfloat16* mu;  // [H_kv][D]
  int H_kv, R, n, m, mtiles, blocks;   // blocks = B*H_kv*R
  int* status;
};

// row sums of U (fp32), one warp per row
template <typename T>
__global__ void __launch_bounds__(256) usum_kernel(const T* __restrict__ U, float* __restrict__ usum, int rows, int n) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  float s = 0.f;
  for (int i = lane; i < n; i += 32) s += to_f32(U[(size_t)row * n + i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) usum[row] = s;
}

__global__ void __launch_bounds__((CM_WARPS + 1) * 32, 1)
project_values_mma_kernel(const __grid_constant__ CUtensorMap tmU, const __grid_constant__ CUtensorMap tmV, const CompressArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* sm = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
  __shared__ __align__(8) uint64_t full_bar[CM_STAGES], empty_bar[CM_STAGES];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < CM_STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], CM_WARPS); }
    fence_mbar_init();
  }
  __syncthreads();

  // CTA -> (KV head, sequence, block, row tile): consecutive CTAs share U[h]
  const int mt = blockIdx.x % a.mtiles;
  const int rest = blockIdx.x / a.mtiles;              // = (h * B + b) * R + r
  const int per_h = a.blocks / a.H_kv;                 // B * R
  const int h = rest / per_h, br = rest - h * per_h;
  const int b = br / a.R, r = br - b * a.R;
  const int bhr = (b * a.H_kv + h) * a.R + r;
  const int nk = a.n / CM_BK;

  if (warp == CM_WARPS) {
    if (lane != 0) return;
    tma_prefetch_desc(&tmU); tma_prefetch_desc(&tmV);
    uint32_t slot = 0, phase = 1;
    for (int kc = 0; kc < nk; ++kc) {
      if (!mbar_wait_bounded(&empty_bar[slot], phase)) { atomicExch(a.status, (int)KVC_ERR_TIMEOUT); return; }
      unsigned char* dst = sm + slot * CM_STAGE;
      mbar_expect_tx(&full_bar[slot], CM_STAGE);
      tma_load_3d(dst, &tmU, kc * CM_BK, mt * CM_BM, h, &full_bar[slot]);
      tma_load_2d(dst + CM_U_BYTES, &tmV, 0, bhr * a.n + kc * CM_BK, &full_bar[slot]);
      tma_load_2d(dst + CM_U_BYTES + CM_V_HALF, &tmV, 64, bhr * a.n + kc * CM_BK, &full_bar[slot]);
      if (++slot == CM_STAGES) { slot = 0; phase ^= 1u; }
    }
    return;
  }

  const int gid = lane >> 2, t4 = lane & 3;
  const int wm = warp & 3, wn = warp >> 2;             // rows wm*32.., channels wn*64..
  const int l7 = lane & 7, lrow = l7 + ((lane >> 3) & 1) * 8, lhi = lane >> 4;
  const uint32_t sm_u = smem_addr(sm);
  float acc[2][8][4];
#pragma unroll
  for (int mi = 0; mi < 2; ++mi)
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[mi][nt][e] = 0.f;

  uint32_t slot = 0, phase = 0;
  bool dead = false;
  for (int kc = 0; kc < nk; ++kc) {
    if (!dead && !mbar_wait_bounded(&full_bar[slot], phase)) dead = true;
    const uint32_t u_u = sm_u + slot * CM_STAGE, v_u = u_u + CM_U_BYTES + wn * CM_V_HALF;
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      uint32_t af[2][4], bf[4][4];
#pragma unroll
      for (int mi = 0; mi < 2; ++mi)
        ldsm_x4(af[mi], u_u + (uint32_t)((wm * 32 + mi * 16 + lrow) * 128) + (uint32_t)(((ks * 2 + lhi) ^ l7) << 4));
#pragma unroll
      for (int np = 0; np < 4; ++np)
        ldsm_x4_t(bf[np], v_u + (uint32_t)((ks * 16 + lrow) * 128) + (uint32_t)(((np * 2 + lhi) ^ l7) << 4));
#pragma unroll
      for (int mi = 0; mi < 2; ++mi)
#pragma unroll
        for (int np = 0; np < 4; ++np) {
          mma_bf16_16816(acc[mi][2 * np], af[mi], bf[np][0], bf[np][1]);
          mma_bf16_16816(acc[mi][2 * np + 1], af[mi], bf[np][2], bf[np][3]);
        }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[slot]);
    if (++slot == CM_STAGES) { slot = 0; phase ^= 1u; }
  }

  // V_tilde[j][c] = acc - usum[j] * mu[c]
  __nv_bfloat16* outp = a.Vc + (size_t)bhr * a.m * D;
#pragma unroll
  for (int mi = 0; mi < 2; ++mi)
#pragma unroll
    for (int hr = 0; hr < 2; ++hr) {
      const int j = mt * CM_BM + wm * 32 + mi * 16 + gid + 8 * hr;
      if (j < a.m) {
        const float us = a.usum[h * a.m + j];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          const int c = wn * 64 + nt * 8 + 2 * t4;
          const __nv_bfloat162 mu2 = *reinterpret_cast<const __nv_bfloat162*>(a.mu + h * D + c);
          const __nv_bfloat162 o = __floats2bfloat162_rn(fmaf(-us, __low2float(mu2), acc[mi][nt][2 * hr]),
                                                         fmaf(-us, __high2float(mu2), acc[mi][nt][2 * hr + 1]));
          *reinterpret_cast<__nv_bfloat162*>(outp + (size_t)j * D + c) = o;
        }
      }
    }
  if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
}

cudaError_t compute_usum(const kvc_layer* L, float* usum) {
  const int rows = L->desc.H_kv * L->m;
  if (L->desc.dtype == KVC_BF16)
    usum_kernel<__nv_bfloat16><<<ceil_div(rows, 8), 256>>>(static_cast<const __nv_bfloat16*>(L->desc.U), usum, rows, L->desc.n);
  else
    usum_kernel<float><<<ceil_div(rows, 8), 256>>>(static_cast<const float*>(L->desc.U), usum, rows, L->desc.n);
  return cudaGetLastError();
}

// bf16, n a multiple of 64, 16-byte aligned pointers; *used == false if this path does not apply
cudaError_t launch_project_values_mma(const kvc_layer* L, const void* V_vis, int B, int R, void* Vc, cudaStream_t st, bool* used) {
  *used = false;
  const int n = L->desc.n, m = L->m, H_kv = L->desc.H_kv;
  if (L->desc.dtype != KVC_BF16 || n % CM_BK != 0 || !L->d_usum) return cudaSuccess;
  if ((reinterpret_cast<uintptr_t>(V_vis) | reinterpret_cast<uintptr_t>(Vc) | reinterpret_cast<uintptr_t>(L->desc.U) |
       reinterpret_cast<uintptr_t>(L->desc.mu)) & 15)
    return cudaSuccess;
  const long long rows_v = (long long)B * H_kv * R * n;
  if (rows_v >= (1ll << 31)) return cudaSuccess;
  CUtensorMap tmU, tmV;
  {
    const uint64_t dims[3] = {(uint64_t)n, (uint64_t)m, (uint64_t)H_kv};
    const uint64_t str[2] = {(uint64_t)n * 2, (uint64_t)m * n * 2};
    const uint32_t box[3] = {64u, (uint32_t)CM_BM, 1u};
    if (!encode_tensor_map_bf16(&tmU, L->desc.U, 3, dims, str, box)) return cudaSuccess;
  }
  {
    const uint64_t dims[2] = {(uint64_t)D, (uint64_t)rows_v};
    const uint64_t str[1] = {256ull};
    const uint32_t box[2] = {64u, (uint32_t)CM_BK};
    if (!encode_tensor_map_bf16(&tmV, V_vis, 2, dims, str, box)) return cudaSuccess;
  }
  *used = true;
  CompressArgs a{};
  a.Vc = static_cast<__nv_bfloat16*>(Vc);
  a.usum = L->d_usum;
  a.mu = static_cast<const __nv_bfloat16*>(L->desc.mu);
  a.H_kv = H_kv; a.R = R; a.n = n; a.m = m;
  a.mtiles = ceil_div(m, CM_BM);
  a.blocks = B * H_kv * R;
  a.status = L->d_cstatus;
  const size_t smem = (size_t)CM_STAGES * CM_STAGE + 1024;
  {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(project_values_mma_kernel), smem);
    if (e != cudaSuccess) return e;
  }
  project_values_mma_kernel<<<(unsigned)(a.blocks * a.mtiles), (CM_WARPS + 1) * 32, smem, st>>>(tmU, tmV, a);
  return cudaGetLastError();
}

}  // namespace kvc
