// Internal declarations shared by the KVCapsule CUDA translation units (not part of the ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvc.h"

namespace kvc {

constexpr int D = 128;              // head dimension (all supported models)
constexpr int MAX_G = 16;           // query heads per KV head
constexpr int SCORE_TILE_ROWS = 64; // K rows per CTA in the score kernel
constexpr int OUT_CHUNK = 64;       // value rows per ring stage of the output kernel
constexpr int EXP_ROWS = 16;        // rows per CTA in the generic expansion kernel
constexpr int EXP_IC = 64;          // vision positions per inner chunk of the expansion
constexpr int EXP_TARGET_CTAS = 296;
constexpr int MAX_NS = 16;          // upper bound of the n-axis splits of the expansion

inline __host__ __device__ int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline __host__ __device__ size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- 16-byte vector access, converted to fp32 -----------------------------------------------
template <typename T> struct Elems16;
template <> struct Elems16<float> { static constexpr int N = 4; };
template <> struct Elems16<__nv_bfloat16> { static constexpr int N = 8; };

__device__ __forceinline__ void unpack16(const uint4& v, float (&f)[4], float*) {
  f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
  f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}
__device__ __forceinline__ void unpack16(const uint4& v, float (&f)[8], __nv_bfloat16*) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
template <typename T>
__device__ __forceinline__ void load16(const T* p, float (&f)[Elems16<T>::N]) {
  uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
  unpack16(v, f, (T*)nullptr);
}
__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_elem(float* p, float x) { *p = x; }
__device__ __forceinline__ void store_elem(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

// ---- workspace layout of one decode call -----------------------------------------------------
struct WsLayout {
  int use_mma;     // 1: tensor-core expansion (bf16 S), 0: CUDA-core fp32 expansion
  int NS;          // splits of the n axis in the expansion kernel
  int IR;          // vision positions per split (multiple of EXP_IC)
  int CG, cgw;     // tensor-core expansion: column groups of W and their width (multiple of 16)
  // output kernel: the value rows of a (sequence, KV head) are cut into chunks of <= OUT_CHUNK rows
  // (cpb per vision block, ct for the text run); CTA c streams chunks [c*cpc, (c+1)*cpc) of the flat list
  int cpb, ct, chunks_per_bh, cpc, out_ctas, GT;
  int nsplit;      // partial slots per (sequence, KV head): CTAs that can touch its chunk range
  int Ts;          // row stride of the text logits (T rounded up to a multiple of 4)
  size_t off_S;    // fp32 or bf16 [H_kv][B][G][R][ms]   compressed scores, sigma applied
  size_t off_stxt; // fp32 [B][H_kv][G][T]       text logits
  size_t off_W;    // fp32 [NS][H_kv][B*G*R][msv] unnormalised P U^T per split (msv: pitch of a weight row)
  size_t off_wstat;// float2 [NS][H_kv][B*G*R]   (max, sum) per row and split
  size_t off_Wc;   // fp32 [H_kv][B*G*R][msv]    the splits combined, relative to one maximum per row
  size_t off_statc;// float4 [H_kv][B*G*R]       (max, sum, 0, 0) of the combined row
  size_t off_ypart;// fp32 [B][H_kv][G][nsplit][D]
  size_t off_ystat;// float2 [B][H_kv][G][nsplit]
  size_t off_cnt;  // int [B*H_kv] arrival counters, then one int device status word
  size_t off_fpy;  // fp32 [B*H_kv][nrg][G][D]  partial outputs of the one-kernel path (units that split the block axis)
  size_t off_fpml; // float2 [B*H_kv][nrg][G]   their (max, sum)
  size_t off_fcnt; // u64 [B*H_kv]              arrival words of the one-kernel path: (call token, arrivals)
  size_t off_split;// the regions of the three-kernel bf16 path (kvc_split.cuh), 0 bytes when the shape does not take it
  size_t off_resident; // the regions of the resident-parameter bf16 path (kvc_resident.cuh), likewise
  size_t total;
};

// Launch plan of the one-kernel bf16 decode path (kvc_fused.cu); ok == 0 when the shape is served by the
// three-phase path instead.
struct FusedPlan {
  int ok;
  int MT;            // 16-row tiles of expansion rows per unit
  int NB, RB;        // sequences and vision blocks per unit
  int nbg, nrg;      // unit groups along the batch and the block axis
  int units;         // H_kv * nbg * nrg
  int JC, NJ;        // 16-row sub-chunks of the m axis per stage; stages per pass over the m axis
  int TCH;           // text rows per stage and sequence
  int ncg;           // n / 64
  int EW, VW, ktw;   // expansion warps, value warps; 16-column groups of the logits per expansion warp
  int msplit, mshift;// the 8 row tiles of a value block go to msplit = 8 >> mshift tasks
  int sld;           // row stride of the score tile
  int yhg;           // heads per round of the final reduction over the value warps
  int stages, grid;
  uint32_t par_bytes, k_half_bytes, txt_half_bytes, stage_bytes, misc_bytes;
  uint32_t off_q, off_S, off_W, off_wred, off_rstat, off_tstat, off_hstat, off_yred;   // relative to the end of the ring
  int tc;            // 1: the expansions run on tcgen05 with the logits in tensor memory (kvc_fused_tc.cu); 2: its pair mode
  uint32_t off_P, off_rtab, off_xstat, off_wrecv;
  int tmem_cols;
  int UT, nu;        // 128-row tiles of U per stage and stages of U per unit (tensor-memory variant)
  size_t smem_bytes;
};

}  // namespace kvc

struct kvc_map_cache;     // tensor maps of recent decode calls on a handle (kvc_fused.cu)

struct kvc_layer {
  kvc_layer_desc desc;   // idx pointer cleared after the copy
  int m;                 // retained length
  int ms;                // row stride of score buffers (m rounded up to 16)
  int mode;              // KVC_MODE_KV, or one side kept verbatim (App. G): KVC_MODE_K_ONLY, KVC_MODE_V_ONLY
  int capsules_fresh;    // set by kvc_compress*, cleared by the next decode call on the handle (which then reads the store late)
  int mk, mv;            // stored rows per block on the key side (n in the V-only mode) and on the value side (n in the K-only mode)
  int G;
  int passthrough;       // ratio_permille == 0
  int device;
  int num_sms;
  int use_tc;            // expansions of the one-kernel decode path: 0 chosen per shape, 1 tcgen05, 2 tcgen05 in pairs of CTAs,
                         // -1 mma.sync (environment KVC_EXPANSION=tcgen05 | pair | mma when the handle is created)
  int32_t* d_idx;        // device [H_kv][m]
  int* d_cstatus;        // device status word of the compress kernels (cleared by every kvc_compress call)
  float* d_usum;         // device [H_kv][m] row sums of U (value compression:  U (V - 1 mu^T) = U V - (U 1) mu^T)
  kvc_map_cache* maps;   // host: tensor maps keyed by (B, R, capsule pointer, launch plan); guarded by its own mutex
};

namespace kvc {

WsLayout ws_layout(const kvc_layer* L, int B, int R, int T_cap);
int cuda_status(cudaError_t e);   // KVC_OK or KVC_ERR_CUDA, remembering the error for kvc_last_cuda_error
FusedPlan plan_fused(const kvc_layer* L, int B, int R);
FusedPlan plan_fused_tc(const kvc_layer* L, int B, int R);     // tensor-memory variant; ok == 0 if the shape does not fit it
FusedPlan plan_fused_pair(const kvc_layer* L, int B, int R);   // its pair mode (clusters of two CTAs)
FusedPlan plan_fused_text(const kvc_layer* L, int B, int T);   // R == 0: text rows only

struct DecodeArgs {
  const void* q;
  const void* Kc;      // K_tilde  [B][H_kv][R][m][D]
  const void* Vc;      // V_tilde
  const void* K_txt;
  const void* V_txt;
  const void* theta;
  const void* U;
  const void* mu;
  void* out;
  int B, H_kv, G, R, m, ms, n, T, T_cap;   // m, ms: key rows per block = length of a compressed score row, and its pitch
  int mv, msv;         // value rows per block = length of a weight row, and its pitch (= m, ms unless one side is verbatim)
  int Ts;              // row stride of s_txt
  int passthrough;
  int id_theta, id_U;  // the score expansion / the re-projection is the identity (verbatim keys / verbatim values)
  float* S;            // fp32 scores (CUDA-core expansion)
  __nv_bfloat16* Sb;   // bf16 scores (tensor-core expansion); exactly one of S / Sb is used
  float* s_txt;
  float* W;
  float2* wstat;
  float* Wcomb;
  float4* statc;
  float* ypart;
  float2* ystat;
  int* cnt;
  unsigned long long* fcnt;   // arrival words of the one-kernel path
  unsigned int token;         // this call's token (never 0)
  const int* R_b;      // per-sequence block counts (<= R) and text lengths (<= T), device arrays; nullptr: R and T for all
  const int* T_b;
  int* status;         // device status word (0 = ok, else a kvc_status), cleared by the first kernel of the call
  float* fpart_y;      // partials of the one-kernel path
  float2* fpart_ml;
  void* split_base;    // regions of the three-kernel bf16 path
  void* resident_base; // regions of the resident-parameter bf16 path
  int early_capsules;  // the capsule store has not been written since the handle's last decode call began: kernels may read it early
  WsLayout ws;
};

#ifdef __CUDACC__
// blocks and text rows sequence b takes part with (clamped to the call's bounds; the first kernel reports a clamp)
__device__ __forceinline__ int seq_R(const DecodeArgs& a, int b) {
  if (!a.R_b) return a.R;
  const int r = a.R_b[b];
  return r < 0 ? 0 : (r > a.R ? a.R : r);
}
__device__ __forceinline__ int seq_T(const DecodeArgs& a, int b) {
  if (!a.T_b) return a.T;
  const int t = a.T_b[b];
  return t < 0 ? 0 : (t > a.T ? a.T : t);
}
// after the status word has been cleared: lengths outside [0, R] x [0, T] are reported (and clamped by seq_R / seq_T)
__device__ __forceinline__ void check_seq_lengths(const DecodeArgs& a, int tid, int nthreads) {
  if (!a.R_b && !a.T_b) return;
  for (int b = tid; b < a.B; b += nthreads) {
    const bool bad = (a.R_b && (a.R_b[b] < 0 || a.R_b[b] > a.R)) || (a.T_b && (a.T_b[b] < 0 || a.T_b[b] > a.T));
    if (bad) atomicExch(a.status, (int)KVC_ERR_BOUNDS);
  }
}
#endif

// validation + the three launches of one decode call; `workspace` is any 256-byte aligned device
// scratch of ws_layout(L, B, R, T).total bytes
int decode_common(const kvc_layer* L, const void* q, const void* capsules, int B, int R, const void* K_txt,
                  const void* V_txt, int T, int T_cap, void* out, void* workspace, cudaStream_t st,
                  const int* R_b = nullptr, const int* T_b = nullptr);

// Raises a kernel's dynamic shared-memory limit to at least `bytes` on the current device.  The attribute is per device
// (and per kernel), so the record of what has been set is keyed by (kernel, device ordinal); safe from several host threads.
cudaError_t ensure_dynamic_smem(const void* kernel, size_t bytes);

// optional event brackets around a launch (kvc_profile_*)
bool prof_begin(int kernel_id, cudaStream_t st);
void prof_end(cudaStream_t st);
struct ProfScope {
  cudaStream_t st; bool on;
  ProfScope(int kernel_id, cudaStream_t s) : st(s), on(prof_begin(kernel_id, s)) {}
  ~ProfScope() { if (on) prof_end(st); }
};

// Launch with programmatic stream serialisation: the kernel may begin while the preceding kernel of
// the stream is still running, and must execute griddepcontrol.wait before touching anything that
// kernel (or anything before it) writes.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// launchers (each returns a cudaError_t from the launch)
cudaError_t launch_scores(const DecodeArgs& a, int dtype, cudaStream_t st);
cudaError_t launch_expand(const DecodeArgs& a, int dtype, cudaStream_t st);
// dynamic shared memory of the tensor-core expansion kernel for rows of `ms` retained positions cut into column groups of `cgw`
size_t expand_mma_smem_bytes(int ms, int cgw);
cudaError_t launch_expand_mma(const DecodeArgs& a, cudaStream_t st);
cudaError_t launch_output(const DecodeArgs& a, int dtype, cudaStream_t st);
// one-kernel path; *encoded == false (and nothing launched) if the tensor maps could not be built
cudaError_t launch_fused(const kvc_layer* L, const DecodeArgs& a, const FusedPlan& p, cudaStream_t st, bool* encoded);
// theta[h] = W1[h] W2[h] (m x k times k x n), fp32 accumulation, one rounding to the storage type
cudaError_t launch_collapse_theta(const void* W1, const void* W2, void* theta, int H_kv, int m, int k, int n, int dtype,
                                  cudaStream_t st);
cudaError_t launch_export_groups(int32_t* d_out, int R, int n, cudaStream_t st);   // (block, offset) of every vision token
int static_scratch(void** out);     // device address of the fixed scratch array on the current device (kvc_static.cu)
void launch_wait_selftest(int* status, cudaStream_t st);   // one warp, a wait that runs out: *status = KVC_ERR_TIMEOUT
kvc_map_cache* map_cache_create();
void map_cache_destroy(kvc_map_cache* c);
cudaError_t compute_usum(const kvc_layer* L, float* usum);
cudaError_t launch_project_values_tc(const kvc_layer* L, const void* V_vis, int B, int R, void* Vc, cudaStream_t st, bool* used);
cudaError_t launch_project_values_mma(const kvc_layer* L, const void* V_vis, int B, int R, void* Vc, cudaStream_t st, bool* used);
cudaError_t launch_compress_ragged(const kvc_layer* L, const void* K_vis, const void* V_vis, int B, int N_cap,
                                   const int* N_v, int R_max, void* Kc, void* Vc, void* K_tail, void* V_tail, int T_cap,
                                   int* R_b, int* T_b, cudaStream_t st);
cudaError_t launch_compress_keys(const kvc_layer* L, const void* K_vis, int B, int R, void* Kc, cudaStream_t st);
cudaError_t launch_compress_values(const kvc_layer* L, const void* V_vis, int B, int R, void* Vc, cudaStream_t st);

}  // namespace kvc
