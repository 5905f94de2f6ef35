// The three-kernel bf16 decode path ("split" path): Algorithm 1 cut at the two places where the work changes shape.
//   split_scores_kernel   step 1: S = sigma q K_tilde^T for every retained key row, one streaming pass over K_tilde (HBM)
//   split_expand_kernel   steps 2-3 as two dense products per 128 expansion rows of a KV head and per range of the n
//                         positions, on tcgen05 with the logits and the weights in tensor memory:
//                           L = S theta[:, range],  P = 2^(L - rowmax),  W_part = P U[:, range]^T  (+ rowmax, rowsum)
//   split_output_kernel   step 4 and the text rows: one streaming pass over V_tilde (weights = the range partials of W
//                         joined on the fly) and over K_txt / V_txt (flash-style), partial (max, sum, y) per segment,
//                         merged by the last segment of a (sequence, KV head) to arrive
// The intermediates S and W_part are a few MB, written once and read back once or a few times from L2.  The expansion rows
// of a KV head are ordered rho = (b R + r) G + g, so the G rows of a block are adjacent.
#pragma once

#include "kvc_tma.cuh"
#include "kvc_internal.cuh"

namespace kvc {

constexpr int SP_TILE_ROWS = 128;      // retained key rows per stage of the score kernel; expansion rows per expansion CTA
constexpr int SO_FAC_PITCH = 17;     // float2 entries per (block, range) row of the output kernel's factor table
constexpr int SP_OUT_ROWS = 64;        // value rows (and text rows) per stage of the output kernel
constexpr int SP_MAX_STAGES = 12;
constexpr int SP_TEXT_CHUNK = 3;       // 64-row tiles of text per CTA of the text kernel (96 KB of stages: two CTAs per SM)

struct SplitPlan {
  int ok;
  int rows_h;          // expansion rows per KV head: B R G
  int ntile;           // 128-row tiles of them
  int NS, NW;          // ranges of the n axis and their width (a multiple of 64, at most 256)
  int ms;              // row pitch of S and W_part in elements (m rounded up to 8)
  int nk1;             // 64-row chunks of the m axis (K steps of the first product)
  int npass, prow;     // the weights of a tile are produced in npass passes of prow columns (<= 512 tensor-memory columns)
  int nbox, brow;      // a pass reads nbox boxes of brow rows of U per 64-column chunk (brow <= 256, a multiple of 16)
  int tmem_cols;
  int e_stages; uint32_t e_stage_bytes, e_p_bytes; size_t e_smem; int e_grid;
  int s_tiles_bh;      // 128-row tiles of the R m key rows of a (sequence, KV head)
  int s_stages, s_grid; size_t s_smem;
  int vt;              // 64-row tiles per block of V_tilde
  int o_stages, o_grid; uint32_t o_stage_bytes, o_w_bytes; size_t o_smem;
  int o_cpb;              // CTAs of the output kernel per (sequence, KV head) = its partial slots
  uint32_t o_off_q, o_off_fac, o_off_red, o_off_stat;   // behind the ring
};

// workspace regions of the split path (byte offsets inside the caller's workspace)
struct SplitWs {
  size_t off_S;      // bf16 [H_kv][rows_h][ms]
  size_t off_Wp;     // bf16 [H_kv][NS][rows_h][ms]
  size_t off_stat;   // float2 [H_kv][NS][rows_h]  (row maximum in log2 units, row sum)
  size_t off_py;     // fp32 [B*H_kv][o_cpb][G][D]
  size_t off_pml;    // float2 [B*H_kv][o_cpb][G]
  size_t off_cnt;    // int [B*H_kv]  arrivals of the output kernel's CTAs, cleared by the score kernel
  size_t off_tpy;    // fp32 [B*H_kv][chunks][G][D]   partials of the text kernel
  size_t off_tpml;   // float2 [B*H_kv][chunks][G]
  size_t bytes;
};

SplitPlan plan_split(const kvc_layer* L, int B, int R);
SplitWs split_ws(const kvc_layer* L, const SplitPlan& p, int B, int R, int T);
cudaError_t launch_split(const kvc_layer* L, const DecodeArgs& a, const SplitPlan& p, cudaStream_t st, bool* encoded);

struct SplitArgs {
  const __nv_bfloat16* q;
  const __nv_bfloat16* mu;
  __nv_bfloat16* out;
  __nv_bfloat16* S;
  __nv_bfloat16* Wp;
  float2* stat;
  float* py;
  float2* pml;
  float* tpy;        // text kernel: [B*H_kv][chunks][G][D]
  float2* tpml;      // [B*H_kv][chunks][G]
  int* cnt;
  int* status;
  int early;         // 1: capsule rows may be loaded before the stream's previous kernel has finished (see kvc.h)
  int B, H_kv, G, R, m, n, T;
  int rows_h, ntile, NS, NW, ms, nk1, npass, prow, nbox, brow, tmem_cols;
  int e_stages; uint32_t e_stage_bytes;
  int e_grid, tx_grid;   // expansion CTAs; text CTAs behind them in the same grid
  int s_tiles_bh, s_stages;
  int vt, o_stages; uint32_t o_stage_bytes;
  int o_cpb;
  uint32_t o_off_q, o_off_fac, o_off_red, o_off_stat;
};

// sigma = 1/sqrt(128), logits kept in log2 units
constexpr float SP_QSCALE = 0.08838834764831845f * 1.4426950408889634f;

// Stage rings whose tiles go to groups of SP_GROUP warps (tile k of a CTA's list to group k mod 2, ring slot k mod stages):
// a group may reach the full barrier of its slot before the slot's previous round has even been filled, and the barrier's
// parity alone cannot tell round w from round w - 2.  So every slot carries a count of the warps that have released it
// over all rounds; the consumers of round w first wait (bounded) until every warp of the rounds before has released,
// which pins the barrier's current phase to round w.
constexpr int SP_GROUP = 4;            // warps that share a tile
__device__ __forceinline__ bool wait_round(const volatile uint32_t* released, uint32_t slot, uint32_t round, uint32_t group = SP_GROUP) {
  for (uint32_t i = 0; i < (1u << 24); ++i)
    if (released[slot] >= round * group) return true;
  return false;
}
__device__ __forceinline__ void release_slot(uint32_t* released, uint64_t* empty_bar, uint32_t slot) {
  atomicAdd(&released[slot], 1u);
  __threadfence_block();
  mbar_arrive(&empty_bar[slot]);
}

// Item i of `tot` items dealt in contiguous runs to `grid` CTAs: CTA c owns [c tot / grid, (c+1) tot / grid).
__host__ __device__ __forceinline__ long long run_begin(long long c, long long tot, long long grid) { return c * tot / grid; }
// the CTA that owns item i
__host__ __device__ __forceinline__ int run_owner(long long i, long long tot, long long grid) {
  return (int)(((i + 1) * grid - 1) / tot);
}

}  // namespace kvc
