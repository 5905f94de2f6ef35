// One-kernel bf16 decode path for short blocks whose parameters fit shared memory ("resident" path): theta[h] and U[h]
// are loaded once per CTA and stay in shared memory.  The work of a (sequence, KV head) is a list of items (one vision
// block or one 64-row text chunk each); it is cut into `cpb` units, a CTA takes whole units of its KV head, and inside a
// unit every WARP walks its own items from its own ring of 16-row pieces, carrying flash-style (max, sum, y) per query
// head in registers: no barrier of the CTA until the unit ends, when the warps' results are merged through shared
// memory (and the units of a pair through the workspace).
#pragma once

#include "kvc_tma.cuh"
#include "kvc_internal.cuh"

namespace kvc {

constexpr int RS_PIECE_ROWS = 16;                 // rows per ring piece (4 KB: two 64-channel halves, 128-byte swizzle)
constexpr uint32_t RS_PIECE_BYTES = RS_PIECE_ROWS * 256u;
constexpr int RS_TEXT_ROWS = 64;                  // text rows per item
constexpr int RS_WARPS = 8;
constexpr int RS_MAX_SLOTS = 8;                   // pieces in flight per warp
constexpr int RS_MAX_CPB = 16;                    // units per (sequence, KV head)
constexpr int RS_MAX_MP16 = 8;                    // m <= 128

struct ResidentPlan {
  int ok;
  int mp;            // m rounded up to 16: rows of the parameter panels
  int ncg;           // n / 64 column panels of theta and U
  int ct;            // text items per (sequence, KV head) at this T
  int items_b;       // items per (sequence, KV head): R + ct
  int cpb;           // units per (sequence, KV head)
  int cph;           // CTAs per KV head
  int grid;
  int slots;         // ring pieces of the CTA; a unit deals them to the warps that have items
  uint32_t par_bytes;
  uint32_t off_theta, off_U, off_ring;
  size_t smem;
};

struct ResidentWs {
  size_t off_py;     // fp32 [B*H_kv][RS_MAX_CPB][8][D]
  size_t off_pml;    // float2 [B*H_kv][RS_MAX_CPB][8]
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
  int ncg, ct, items_b, cpb, cph, slots;
  const int* R_b;    // per-sequence block counts (<= R) and text lengths (<= T), device arrays; nullptr: R and T for all
  const int* T_b;
  int early;         // 1: vision pieces may be loaded before the stream's previous kernel has finished (see kvc.h)
  uint32_t par_bytes;
  uint32_t off_theta, off_U, off_ring;
};

}  // namespace kvc
