// Split path, first kernel: the compressed scores of Alg. 1 step 1,
//   S[h][(b R + r) G + g][j] = sigma log2(e) q[b, hG + g, :] . K_tilde[b, h, r, j, :]      (bf16, fp32 accumulation)
// One streaming pass over K_tilde, bound by HBM bandwidth.  The R m key rows of a (sequence, KV head) are contiguous in
// the capsule store; they are cut into tiles of 128 rows and the flat tile list is dealt in contiguous runs to one
// persistent CTA per SM.  A producer thread keeps a ring of TMA-filled 32 KB stages full (128-byte swizzle).  Each of
// the sixteen consumer warps takes 8 rows of every tile (a tile is a chain of dependent steps per warp, so its latency,
// not its instruction count, sets the pace: more and shorter chains): the queries of the KV head (up to 16, zero-padded) are the A
// operand held in registers, the key rows the B operand read with ldmatrix, and a lane ends up with two consecutive key
// rows of one head.
#include "kvc_split.cuh"

namespace kvc {

constexpr int SS_WARPS = 16;
constexpr int SS_THREADS = (SS_WARPS + 1) * 32;
constexpr uint32_t SS_HALF = SP_TILE_ROWS * 128;      // one 64-channel half of a tile
constexpr uint32_t SS_STAGE = 2 * SS_HALF;

__global__ void __launch_bounds__(SS_THREADS, 1)
split_scores_kernel(const __grid_constant__ CUtensorMap tmK, const SplitArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* sm = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
  __shared__ __align__(8) uint64_t full_bar[SP_MAX_STAGES], empty_bar[SP_MAX_STAGES];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < a.s_stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], SS_WARPS); }
    fence_mbar_init();
  }
  __syncthreads();

  const long long BH = (long long)a.B * a.H_kv;
  const long long total = BH * a.s_tiles_bh;
  const long long lo = run_begin(blockIdx.x, total, gridDim.x), hi = run_begin(blockIdx.x + 1, total, gridDim.x);
  const int nst = a.s_stages;

  if (warp == SS_WARPS) {
    if (lane != 0) return;
    tma_prefetch_desc(&tmK);
    {
      // while the stream's previous kernel drains: the first ring of tiles is asked into L2 (a prefetch consumes no
      // data, so it need not wait for that kernel; the loads below do)
      int pbh = (int)(lo / a.s_tiles_bh), pt = (int)(lo - (long long)pbh * a.s_tiles_bh);
      for (int k = 0; k < nst && lo + k < hi; ++k) {
        tma_prefetch_l2_4d(&tmK, 0, pt * SP_TILE_ROWS, 0, pbh);
        if (++pt == a.s_tiles_bh) { pt = 0; ++pbh; }
      }
    }
    if (!a.early) grid_dep_wait();                // the capsule rows: late unless known to be settled (the queries are read by the consumers, after their wait)
    uint32_t slot = 0, phase = 1;
    int bh = (int)(lo / a.s_tiles_bh), t = (int)(lo - (long long)bh * a.s_tiles_bh) - 1;
    for (int it = (int)(hi - lo); it > 0; --it) {
      if (++t == a.s_tiles_bh) { t = 0; ++bh; }
      if (!mbar_wait_bounded(&empty_bar[slot], phase)) { atomicExch(a.status, (int)KVC_ERR_TIMEOUT); return; }
      unsigned char* dst = sm + slot * SS_STAGE;
      mbar_expect_tx(&full_bar[slot], SS_STAGE);
      tma_load_4d(dst, &tmK, 0, t * SP_TILE_ROWS, 0, bh, &full_bar[slot]);      // both 64-channel halves in one copy
      if (++slot == (uint32_t)nst) { slot = 0; phase ^= 1u; }
    }
    return;
  }

  grid_dep_wait();
  grid_dep_launch();
  // per-call device state of the path: status word, arrival counters of the output kernel's runs
  if (blockIdx.x == 0 && tid == 0) *a.status = 0;
  for (long long i = (long long)blockIdx.x * (SS_WARPS * 32) + tid; i < BH; i += (long long)gridDim.x * (SS_WARPS * 32)) a.cnt[i] = 0;

  const int gid = lane >> 2, t4 = lane & 3;
  const int G = a.G, m = a.m, Rm = a.R * a.m;
  const uint32_t sm_u = smem_addr(sm);
  bool dead = false;
  int cur_bh = -1;
  uint32_t qa[8][4];
  uint32_t slot = 0, phase = 0;
  int bh = (int)(lo / a.s_tiles_bh), t = (int)(lo - (long long)bh * a.s_tiles_bh) - 1;
  for (int it = (int)(hi - lo); it > 0; --it) {
    if (++t == a.s_tiles_bh) { t = 0; ++bh; }
    const int b = bh / a.H_kv, h = bh - b * a.H_kv;
    if (bh != cur_bh) {
      cur_bh = bh;
      // A fragments of the score product: rows = the heads of the group (gid, gid + 8), k = the 128 channels
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
    if (!dead && !mbar_wait_bounded(&full_bar[slot], phase)) dead = true;
    __syncwarp();
    const uint32_t st_u = sm_u + slot * SS_STAGE;
    // (block, row in block) of the tile's first key row; the rows of a lane follow by small steps
    const int g0 = t * SP_TILE_ROWS;
    const int r_t = g0 / m, j_t = g0 - r_t * m;
    __nv_bfloat16* S_h = a.S + (size_t)h * a.rows_h * a.ms;
    const int bR = b * a.R;
    {
      const int row0 = warp * 8;                   // this warp's 8 rows: two accumulation chains over the channel halves
      float acc2[2][4];
#pragma unroll
      for (int x = 0; x < 2; ++x)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc2[x][e] = 0.f;
      const int row = row0 + (lane & 7);
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        // four 8 x 8 matrices: the 16-byte pieces 4x .. 4x+3 of rows row0 .. row0+7 (pieces 0-7 in the first half)
        const int c = 4 * x + (lane >> 3);
        uint32_t bf[4];
        ldsm_x4(bf, st_u + (uint32_t)(c >> 3) * SS_HALF + (uint32_t)row * 128u + (uint32_t)((((c & 7) ^ (row & 7))) << 4));
        mma_bf16_16816(acc2[x & 1], qa[2 * x], bf[0], bf[1]);
        mma_bf16_16816(acc2[x & 1], qa[2 * x + 1], bf[2], bf[3]);
      }
      // acc[e]: head gid + 8 (e >> 1), key row g0 + row0 + 2 t4 + (e & 1) of the (sequence, KV head)
      const int off = row0 + 2 * t4;
      if (!dead && g0 + off < Rm) {
        int r = r_t, j = j_t + off;
        if (m >= SP_TILE_ROWS) { if (j >= m) { j -= m; ++r; } }
        else { const int dr = j / m; r += dr; j -= dr * m; }
        int r1 = r, j1 = j + 1;
        if (j1 == m) { j1 = 0; ++r1; }
        const bool second = g0 + off + 1 < Rm;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          const int head = gid + 8 * hh;
          if (head >= G) continue;
          const float v0 = (acc2[0][2 * hh] + acc2[1][2 * hh]) * SP_QSCALE, v1 = (acc2[0][2 * hh + 1] + acc2[1][2 * hh + 1]) * SP_QSCALE;
          __nv_bfloat16* p0 = S_h + ((size_t)(bR + r) * G + head) * a.ms + j;
          if (second && r1 == r && (j & 1) == 0) {
            *reinterpret_cast<uint32_t*>(p0) = pack2_bf16(v0, v1);
          } else {
            *p0 = __float2bfloat16_rn(v0);
            if (second) S_h[((size_t)(bR + r1) * G + head) * a.ms + j1] = __float2bfloat16_rn(v1);
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[slot]);
    if (++slot == (uint32_t)nst) { slot = 0; phase ^= 1u; }
  }
  if (dead && lane == 0) atomicExch(a.status, (int)KVC_ERR_TIMEOUT);
}

cudaError_t launch_split_scores(const CUtensorMap& tmK, const SplitArgs& a, const SplitPlan& p, cudaStream_t st) {
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(split_scores_kernel), p.s_smem);
  if (e != cudaSuccess) return e;
  ProfScope prof(KVC_KERNEL_SPLIT_SCORES, st);
  return launch_dependent(split_scores_kernel, dim3(p.s_grid), dim3(SS_THREADS), p.s_smem, st, tmK, a);
}

}  // namespace kvc
