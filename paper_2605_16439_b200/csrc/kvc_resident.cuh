// One-kernel bf16 decode path for short blocks whose parameters fit shared memory ("resident" path): theta[h] and U[h]
// are loaded once per CTA and stay in shared memory, the capsule rows and the text rows stream through a ring of
// 64-row tiles, and a CTA walks a contiguous run of work items (one vision block or one 64-row text chunk each) of its
// KV head, carrying flash-style running (max, sum, y) per query head across the items of a (sequence, KV head).
#pragma once

#include "kvc_tma.cuh"
#include "kvc_internal.cuh"

namespace kvc {

constexpr int RS_TILE_ROWS = 64;                  // rows per ring tile (16 KB: two 64-channel halves, 128-byte swizzle)
constexpr uint32_t RS_TILE_BYTES = RS_TILE_ROWS * 256u;
constexpr int RS_WARPS = 8;                       // consumer warps (+ one producer warp)
constexpr int RS_MAX_STAGES = 8;

struct ResidentPlan {
  int ok;
  int mp;            // m rounded up to 16: rows of the parameter panels, K extent of the first product
  int ncg;           // n / 64 column panels of theta and U
  int kt;            // 64-row tiles per block side
  int ct;            // 64-row text chunks per (sequence, KV head) at this T
  int items_b;       // work items per (sequence, KV head): R + ct
  int cph;           // CTAs per KV head
  int grid;
  int stages;
  int pitchS, pitchP, pitchW;                        // row pitches in elements
  uint32_t par_bytes;                                // bytes of one parameter matrix in shared memory
  uint32_t off_theta, off_U, off_ring, off_S, off_P, off_W, off_T, off_stat;
  size_t smem;
};

struct ResidentWs {
  size_t off_py;     // fp32 [B*H_kv][slots][16][D]
  size_t off_pml;    // float2 [B*H_kv][slots][16]
  size_t off_cnt;    // u64 [B*H_kv] arrival words (token, count)
  size_t bytes;
};

ResidentPlan plan_resident(const kvc_layer* L, int B, int R, int T);
ResidentWs resident_ws(const kvc_layer* L, int B);
cudaError_t launch_resident(const kvc_layer* L, const DecodeArgs& a, const ResidentPlan& p, cudaStream_t st, bool* encoded);

struct ResidentArgs {
  const __nv_bfloat16* q;
  const __nv_bfloat16* mu;
  __nv_bfloat16* out;
  float* py;
  float2* pml;
  unsigned long long* cnt;
  unsigned int token;
  int* status;
  int B, H_kv, G, R, m, mp, n, T;
  int ncg, kt, ct, items_b, cph, stages;
  int slots;         // partial slots per (sequence, KV head) in py / pml
  int pitchS, pitchP, pitchW;
  uint32_t par_bytes;
  uint32_t off_theta, off_U, off_ring, off_S, off_P, off_W, off_T, off_stat;
};

}  // namespace kvc
