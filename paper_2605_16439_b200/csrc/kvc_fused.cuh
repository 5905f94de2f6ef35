// Definitions shared by the one-kernel decode paths: kernel arguments, shared-memory ring barriers, named-barrier
// ids and the row ranges of the plain K/V rows of a work unit.
#pragma once

#include "kvc_tma.cuh"
#include "kvc_internal.cuh"

namespace kvc {

constexpr int FMAX_STAGES = 8;
constexpr int QLD = 136;                     // row stride of the query tile in elements (272 B: conflict-free ldmatrix)
constexpr int SLD = 24;                      // row stride of the 16-column weight tile (48 B)
constexpr int ROWS = 16;                     // expansion rows per MMA row tile; a unit holds MT of them
constexpr uint32_t SMEM_LIMIT = 232448;      // 227 KB per CTA on sm_100

struct FusedArgs {
  const __nv_bfloat16* q;
  const __nv_bfloat16* mu;
  __nv_bfloat16* out;
  int B, H_kv, G, R, m, n, T;
  int S0;             // text-only mode: rows of a leading K/V segment (verbatim vision rows of a rho = 0 store), else 0
  int NB, RB, nbg, nrg, units, JC, NJ, TCH, Tper, ncg, stages;
  int ktw;            // 16-column groups of L per expansion warp
  int msplit, mshift; // the 8 row tiles of a value block go to msplit = 8 >> mshift tasks
  int sld;            // row stride of the score tile in elements (16 JC + 8)
  int yhg;            // heads per round of the final reduction over the value warps
  uint32_t par_bytes, k_half_bytes, txt_half_bytes, stage_bytes;
  uint32_t off_q, off_S, off_W, off_wred, off_rstat, off_tstat, off_hstat, off_yred;
  uint32_t off_P, off_rtab;   // tensor-memory variant: probabilities as an MMA operand; head slot of every expansion row
  int tmem_cols;              // tensor-memory variant: columns to allocate (power of two >= 32)
  int UT, nu;                 // tensor-memory variant: 128-row tiles of U per stage; stages of U per unit
  uint32_t off_xstat, off_wrecv;   // pair mode of the tensor-memory variant: what the peer CTA writes
  float* part_y;      // [B*H_kv][nrg][G][D]  partial outputs (only when nrg > 1)
  float2* part_ml;    // [B*H_kv][nrg][G]     (max in log2 units, sum)
  unsigned long long* cnt;   // [B*H_kv] arrival words in the caller's workspace (see arrive_is_last)
  unsigned int token;        // this call's token, never 0
  int* status;        // device status word
  int early;          // 1: capsule rows may be loaded before the stream's previous kernel has finished (see kvc.h)
};

// shared-memory barriers of one CTA
struct FusedBars {
  uint64_t full[FMAX_STAGES], empty[FMAX_STAGES];   // ring: data landed / every consumer warp done
};
// Named barriers (bar.arrive by the writers or readers that move on, bar.sync by the side that has to wait), all
// counting every consumer thread: 1 all consumers, 2 expansion warps, 3 value warps, then per tile buffer b:
constexpr int BAR_S_READY = 4;   // + b: score tile written (value warps arrive, expansion warps wait)
constexpr int BAR_S_FREE = 6;    // + b: score tile read     (expansion warps arrive, value warps wait)
constexpr int BAR_W_READY = 8;   // + b: weight tile written (expansion warps arrive, value warps wait)
constexpr int BAR_W_FREE = 10;   // + b: weight tile read    (value warps arrive, expansion warps wait)

// The plain K/V rows a unit attends over: its slice [g0, g1) of the concatenation [leading segment | text rows], as a
// range of the leading segment (a0, a1; tensor maps tmK / tmV) and a range of the text rows (b0, b1; tmKt / tmVt)
struct RowRanges { int a0, a1, b0, b1, na, nb; };
__device__ __forceinline__ RowRanges row_ranges(const FusedArgs& a, int rg) {
  RowRanges r;
  const int g0 = rg * a.Tper, g1 = min(a.S0 + a.T, g0 + a.Tper);
  r.a0 = min(g0, a.S0); r.a1 = min(g1, a.S0);
  r.b0 = max(g0, a.S0) - a.S0; r.b1 = max(g1, a.S0) - a.S0;
  r.na = r.a1 > r.a0 ? (r.a1 - r.a0 + a.TCH - 1) / a.TCH : 0;
  r.nb = r.b1 > r.b0 ? (r.b1 - r.b0 + a.TCH - 1) / a.TCH : 0;
  return r;
}

// Arrival of one unit of a (sequence, KV head) whose partials are merged by the last unit to arrive.  The word lives in
// the caller's workspace, which is never initialised: it packs (token of the call that last touched it, arrivals of
// that call), so whatever an earlier call or nobody left there reads as "no arrivals yet" for a new token.  The last
// arriver clears the word, which also keeps a replayed launch (same token) correct.  Call after __threadfence().
// One atomic add per arrival once the word carries the call's token; only the arrivals that still find another token
// (the first of a call, and those racing with it) take the compare-and-swap path that installs it.
__device__ __forceinline__ bool arrive_is_last(unsigned long long* word, unsigned int token, int expected) {
  const unsigned long long mine = (unsigned long long)token << 32;
  for (;;) {
    const unsigned long long old = atomicAdd(word, 1ull);
    if ((unsigned int)(old >> 32) == token) {
      const bool last = (int)(unsigned int)old + 1 == expected;
      if (last) *reinterpret_cast<volatile unsigned long long*>(word) = 0ull;     // every arrival of the call has been counted
      return last;
    }
    // a word of another call (or never written): this add counted nothing.  Install (token, 1) unless somebody else does first
    unsigned long long seen = old + 1ull;
    for (;;) {
      if ((unsigned int)(seen >> 32) == token) break;                 // installed by another arrival: count this one above
      const unsigned long long prev = atomicCAS(word, seen, mine | 1ull);
      if (prev == seen) {
        if (expected == 1) *reinterpret_cast<volatile unsigned long long*>(word) = 0ull;
        return expected == 1;
      }
      seen = prev;
    }
  }
}

// tensor-memory variant of the kernel (kvc_fused_tc.cu): tm = the six tensor maps in the order of the kernel arguments
cudaError_t launch_fused_tc_kernel(const CUtensorMap* tm, const FusedArgs& fa, const FusedPlan& p, cudaStream_t st);

}  // namespace kvc
