// Host side of the C ABI: validation, layer handles, workspace layout, kernel sequencing.
#include <atomic>
#include <map>
#include <mutex>
#include <new>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "kvc_internal.cuh"
#include "kvc_split.cuh"
#include "kvc_resident.cuh"

namespace kvc {

static size_t elem_bytes(int dtype) { return dtype == KVC_BF16 ? 2 : 4; }

WsLayout ws_layout(const kvc_layer* L, int B, int R, int T_cap) {
  WsLayout w{};
  const int H_kv = L->desc.H_kv, G = L->G, n = L->desc.n;
  const int ms = (L->mk + 15) / 16 * 16, msv = (L->mv + 15) / 16 * 16;
  const int rows_h = B * G * R;
  // tensor-core expansion: bf16 storage and 16-byte aligned rows of theta / U
  w.use_mma = (!L->passthrough && L->mode == KVC_MODE_KV && L->desc.dtype == KVC_BF16 && n % 8 == 0) ? 1 : 0;
  w.CG = 1;
  w.cgw = ms;
  int row_tiles;
  if (w.use_mma) {
    w.CG = ceil_div(ms, 256);
    w.cgw = (int)align_up((size_t)ceil_div(ms, w.CG), 16);
    // the kernel keeps a 64-row score tile and a chunk of theta over all retained positions in shared memory: past about 720
    // of them (n = 1024 at ratios below 0.3) that no longer fits, and the fp32 expansion takes over
    if (expand_mma_smem_bytes(ms, w.cgw) > 227u * 1024u) { w.use_mma = 0; w.CG = 1; w.cgw = ms; }
  }
  if (w.use_mma) {
    row_tiles = ceil_div(rows_h, 64) * H_kv * w.CG;
  } else {
    row_tiles = ceil_div(rows_h, EXP_ROWS) * H_kv;
  }
  if (L->passthrough || rows_h == 0) {
    w.NS = 1;
    w.IR = (int)align_up(n, EXP_IC);
  } else {
    int ns = ceil_div(EXP_TARGET_CTAS, row_tiles);
    ns = ns < 1 ? 1 : ns;
    int max_ns = ceil_div(n, EXP_IC);
    max_ns = max_ns > MAX_NS ? MAX_NS : max_ns;
    ns = ns > max_ns ? max_ns : ns;
    w.IR = (int)align_up((size_t)ceil_div(n, ns), EXP_IC);
    w.NS = ceil_div(n, w.IR);
  }
  w.cpb = ceil_div(L->mv, OUT_CHUNK);
  w.ct = ceil_div(T_cap, OUT_CHUNK);
  w.chunks_per_bh = R * w.cpb + w.ct;
  w.GT = G == 1 ? 1 : (G == 2 ? 2 : (G <= 4 ? 4 : 8));
  {
    const long long total = (long long)B * H_kv * w.chunks_per_bh;
    const int per_sm = w.GT <= 2 ? 3 : 2;
    long long ctas = (long long)(L->num_sms > 0 ? L->num_sms : 148) * per_sm;
    if (ctas > total) ctas = total;
    if (ctas < 1) ctas = 1;
    w.cpc = (int)((total + ctas - 1) / ctas);
    if (w.cpc < 1) w.cpc = 1;
    w.out_ctas = (int)((total + w.cpc - 1) / w.cpc);
  }
  {
    // a (sequence, KV head) spans chunks_per_bh <= cpc * ctas / (B*H_kv) chunks, hence at most that many + 1 CTAs;
    // the bound does not depend on T, so a workspace sized for T_cap fits every T <= T_cap
    const long long ctas_max = (long long)(L->num_sms > 0 ? L->num_sms : 148) * (w.GT <= 2 ? 3 : 2);
    const long long bh = (long long)B * H_kv;
    w.nsplit = (int)((ctas_max + (bh > 0 ? bh : 1) - 1) / (bh > 0 ? bh : 1)) + 2;
  }
  w.Ts = (int)align_up((size_t)(T_cap > 0 ? T_cap : 1), 4);
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  w.off_cnt = take(sizeof(int) * ((size_t)B * H_kv + 1));
  w.off_S = take((w.use_mma ? sizeof(__nv_bfloat16) : sizeof(float)) * (size_t)H_kv * rows_h * ms);
  w.off_stxt = take(sizeof(float) * (size_t)B * H_kv * G * w.Ts);
  w.off_W = take(sizeof(float) * (size_t)w.NS * H_kv * rows_h * msv);
  w.off_wstat = take(sizeof(float2) * (size_t)w.NS * H_kv * rows_h);
  w.off_Wc = take(sizeof(float) * (size_t)H_kv * rows_h * msv);
  w.off_statc = take(sizeof(float4) * (size_t)H_kv * rows_h);
  w.off_ypart = take(sizeof(float) * (size_t)B * H_kv * G * w.nsplit * D);
  w.off_ystat = take(sizeof(float2) * (size_t)B * H_kv * G * w.nsplit);
  {
    // partial outputs of the one-kernel path: per (sequence, KV head) one per unit along the block axis, or, without
    // vision blocks, one per slice of the text rows (at most 16, whatever T is)
    size_t np = 0;
    if (B > 0 && R > 0) {
      const FusedPlan fp = plan_fused(L, B, R);
      if (fp.ok && L->mode == KVC_MODE_KV && fp.nrg > 1) np = (size_t)B * H_kv * fp.nrg * G;
    }
    if ((R == 0 || L->passthrough) && B > 0 && R * n + T_cap > 0 && plan_fused_text(L, B, R * n + T_cap).ok) {
      const size_t np_plain = (size_t)B * H_kv * 16 * G;
      np = np > np_plain ? np : np_plain;
    }
    w.off_fpy = take(sizeof(float) * np * D);
    w.off_fpml = take(sizeof(float2) * np);
    w.off_fcnt = take(sizeof(unsigned long long) * (np ? (size_t)B * H_kv : 0));
  }
  {
    size_t sb = 0;
    if (B > 0 && R > 0) {
      const SplitPlan sp = plan_split(L, B, R);
      if (sp.ok && L->mode == KVC_MODE_KV) sb = split_ws(L, sp, B, R, T_cap).bytes;
    }
    w.off_split = take(sb);
  }
  w.off_resident = take(B > 0 && R > 0 && plan_resident(L, B, R, 0).ok ? resident_ws(L, B).bytes : 0);
  w.total = off;
  return w;
}

}  // namespace kvc

using namespace kvc;

namespace kvc {
cudaError_t ensure_dynamic_smem(const void* kernel, size_t bytes) {
  static std::mutex mu;
  static std::map<std::pair<const void*, int>, size_t> set_to;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  std::lock_guard<std::mutex> lock(mu);
  size_t& have = set_to[std::make_pair(kernel, dev)];
  if (have >= bytes) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) have = bytes;
  return e;
}

static thread_local cudaError_t g_last_cuda = cudaSuccess;
// KVC_OK, or KVC_ERR_CUDA after remembering the error for kvc_last_cuda_error (the runtime's own slot is cleared)
int cuda_status(cudaError_t e) {
  if (e == cudaSuccess) return KVC_OK;
  g_last_cuda = e;
  cudaGetLastError();
  return KVC_ERR_CUDA;
}
}  // namespace kvc

extern "C" {

const char* kvc_last_cuda_error(void) { return cudaGetErrorString(g_last_cuda); }

int kvc_retained_len(int n, int ratio_permille) {
  if (n <= 0 || ratio_permille < 0 || ratio_permille >= 1000) return -1;
  return (int)(((long long)n * (1000 - ratio_permille) + 999) / 1000);
}

const char* kvc_strerror(int s) {
  switch (s) {
    case KVC_OK: return "ok";
    case KVC_ERR_ARG: return "invalid argument (null pointer or negative size)";
    case KVC_ERR_SHAPE: return "unsupported or inconsistent shape";
    case KVC_ERR_DTYPE: return "unknown dtype";
    case KVC_ERR_NO_PARAMS: return "theta / U / mu / idx missing for a compression ratio > 0";
    case KVC_ERR_WORKSPACE: return "workspace null, not 256-byte aligned, or static scratch too small for this shape";
    case KVC_ERR_CUDA: return "CUDA runtime error";
    case KVC_ERR_TIMEOUT: return "bounded device-side wait gave up";
    case KVC_ERR_BOUNDS: return "index set entry out of range or not strictly increasing";
    default: return "unknown status";
  }
}

int kvc_layer_create(const kvc_layer_desc* desc, kvc_layer** out) {
  if (!desc || !out) return KVC_ERR_ARG;
  *out = nullptr;
  if (desc->dtype != KVC_F32 && desc->dtype != KVC_BF16) return KVC_ERR_DTYPE;
  if (desc->d != D || desc->H_q <= 0 || desc->H_kv <= 0 || desc->H_q % desc->H_kv != 0 ||
      desc->H_q / desc->H_kv > MAX_G || desc->n <= 0)
    return KVC_ERR_SHAPE;
  const int m = kvc_retained_len(desc->n, desc->ratio_permille);
  if (m < 1) return KVC_ERR_SHAPE;
  const bool pass = desc->ratio_permille == 0;
  const int mode = pass ? KVC_MODE_KV : desc->mode;
  if (mode != KVC_MODE_KV && mode != KVC_MODE_K_ONLY && mode != KVC_MODE_V_ONLY) return KVC_ERR_ARG;
  const bool key_side = mode != KVC_MODE_V_ONLY, value_side = mode != KVC_MODE_K_ONLY;   // sides that are compressed
  if (!pass && ((key_side && (!desc->idx || !desc->theta)) || (value_side && (!desc->U || !desc->mu)))) return KVC_ERR_NO_PARAMS;

  std::vector<int32_t> idx((size_t)desc->H_kv * m);
  for (int h = 0; h < desc->H_kv; ++h)
    for (int j = 0; j < m; ++j) {
      const int32_t v = (pass || !key_side) ? j : desc->idx[(desc->idx_per_head ? (size_t)h * m : 0) + j];
      if (v < 0 || v >= desc->n || (j > 0 && v <= idx[(size_t)h * m + j - 1])) return KVC_ERR_BOUNDS;
      idx[(size_t)h * m + j] = v;
    }

  kvc_layer* L = new (std::nothrow) kvc_layer();
  if (!L) return KVC_ERR_ARG;
  L->desc = *desc;
  L->desc.idx = nullptr;
  L->m = m;
  L->ms = (m + 15) / 16 * 16;
  L->G = desc->H_q / desc->H_kv;
  L->passthrough = pass ? 1 : 0;
  L->capsules_fresh = 1;
  L->mode = mode;
  L->mk = key_side ? m : desc->n;
  L->mv = value_side ? m : desc->n;
  L->d_idx = nullptr;
  L->d_cstatus = nullptr;
  L->d_usum = nullptr;
  L->maps = map_cache_create();
  L->num_sms = 0;
  {
    const char* ex = std::getenv("KVC_EXPANSION");
    L->use_tc = !ex ? 0 : (std::strcmp(ex, "tcgen05") == 0 ? 1 : (std::strcmp(ex, "pair") == 0 ? 2 : (std::strcmp(ex, "mma") == 0 ? -1 : (std::strcmp(ex, "phases") == 0 ? -2 : (std::strcmp(ex, "split") == 0 ? 3 : (std::strcmp(ex, "resident") == 0 ? 4 : 0))))));
  }
  if (cudaGetDevice(&L->device) != cudaSuccess ||
      cudaDeviceGetAttribute(&L->num_sms, cudaDevAttrMultiProcessorCount, L->device) != cudaSuccess ||
      cudaMalloc(&L->d_idx, idx.size() * sizeof(int32_t)) != cudaSuccess ||
      cudaMemcpy(L->d_idx, idx.data(), idx.size() * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMalloc(&L->d_cstatus, sizeof(int)) != cudaSuccess ||
      cudaMemset(L->d_cstatus, 0, sizeof(int)) != cudaSuccess ||
      (!pass && value_side && (cudaMalloc(&L->d_usum, idx.size() * sizeof(float)) != cudaSuccess ||
                 compute_usum(L, L->d_usum) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess))) {
    if (L->d_idx) cudaFree(L->d_idx);
    if (L->d_cstatus) cudaFree(L->d_cstatus);
    if (L->d_usum) cudaFree(L->d_usum);
    map_cache_destroy(L->maps);
    delete L;
    cudaGetLastError();
    return KVC_ERR_CUDA;
  }
  *out = L;
  return KVC_OK;
}

int kvc_layer_destroy(kvc_layer* L) {
  if (!L) return KVC_OK;
  if (L->d_idx) cudaFree(L->d_idx);
  if (L->d_cstatus) cudaFree(L->d_cstatus);
  if (L->d_usum) cudaFree(L->d_usum);
  map_cache_destroy(L->maps);
  delete L;
  return KVC_OK;
}

int kvc_layer_capsules_written(kvc_layer* L) {
  if (!L) return KVC_ERR_ARG;
  L->capsules_fresh = 1;
  return KVC_OK;
}

int kvc_layer_m(const kvc_layer* L) { return L ? L->m : -1; }

int kvc_layer_rows(const kvc_layer* L, int* key_rows, int* value_rows) {
  if (!L) return KVC_ERR_ARG;
  if (key_rows) *key_rows = L->mk;
  if (value_rows) *value_rows = L->mv;
  return KVC_OK;
}

// bytes of the key part of a capsule store (the value part follows it)
static size_t key_part_bytes(const kvc_layer* L, int B, int R) {
  return (size_t)B * L->desc.H_kv * R * L->mk * D * elem_bytes(L->desc.dtype);
}

size_t kvc_capsule_bytes(const kvc_layer* L, int B, int R) {
  if (!L || B < 0 || R < 0) return 0;
  return (size_t)B * L->desc.H_kv * R * ((size_t)L->mk + L->mv) * D * elem_bytes(L->desc.dtype);
}

size_t kvc_workspace_bytes(const kvc_layer* L, int B, int R, int T_cap) {
  if (!L || B < 0 || R < 0 || T_cap < 0) return 0;
  return ws_layout(L, B, R, T_cap).total;
}

int kvc_compress(const kvc_layer* L, const void* K_vis, const void* V_vis, int B, int R, void* capsules,
                 void* stream) {
  if (!L || B < 0 || R < 0) return KVC_ERR_ARG;
  if (B == 0 || R == 0) return KVC_OK;
  if (!K_vis || !V_vis || !capsules) return KVC_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t kbytes = key_part_bytes(L, B, R), vbytes = kvc_capsule_bytes(L, B, R) - kbytes;
  void* Kc = capsules;
  void* Vc = static_cast<char*>(capsules) + kbytes;
  const_cast<kvc_layer*>(L)->capsules_fresh = 1;
  cudaError_t e = cudaMemsetAsync(L->d_cstatus, 0, sizeof(int), st);   // status word of this compress call
  if (e != cudaSuccess) return cuda_status(e);
  // a side kept verbatim (rho = 0, or the one-sided modes) is a plain copy of its n rows per block
  if (L->passthrough || L->mode == KVC_MODE_V_ONLY) e = cudaMemcpyAsync(Kc, K_vis, kbytes, cudaMemcpyDeviceToDevice, st);
  else e = launch_compress_keys(L, K_vis, B, R, Kc, st);
  if (e != cudaSuccess) return cuda_status(e);
  if (L->passthrough || L->mode == KVC_MODE_K_ONLY) e = cudaMemcpyAsync(Vc, V_vis, vbytes, cudaMemcpyDeviceToDevice, st);
  else e = launch_compress_values(L, V_vis, B, R, Vc, st);
  return cuda_status(e);
}

}  // extern "C"

namespace kvc {
// Which bf16 shapes take the three-kernel path (the others take the one-kernel path).  Measured on B200 over batch 1-64,
// 2-32 blocks and ratios 0.2-0.8 at n = 1024, G = 7: ahead of the one-kernel variants at 31 of 33 points (by 1.0-2.1 x;
// behind by at most 12 % at ratio 0.8 with few rows); behind them for short blocks (n = 256: 35 vs 21 us, n = 576: 74 vs
// 41 us at the 7B shapes), where the logits of a unit fit the registers of the one-kernel path.
// KVC_EXPANSION=split forces it where its plan applies, any other value of the variable keeps it off.
static bool use_split(const kvc_layer* L, int B, int R) {
  if (L->use_tc != 3 && !(L->use_tc == 0 && L->desc.n > 640)) return false;
  return plan_split(L, B, R).ok != 0;
}

// One token per decode call, process-wide: never 0 and never one of the byte patterns a caller is likely to have
// filled a fresh workspace with, so that stale workspace contents cannot pass for arrivals of this call.
static unsigned int next_token() {
  static std::atomic<unsigned int> counter{0x1000u};
  for (;;) {
    const unsigned int t = counter.fetch_add(1u, std::memory_order_relaxed) + 1u;
    const unsigned int b0 = t & 0xffu;
    const bool uniform = ((t >> 8) & 0xffu) == b0 && ((t >> 16) & 0xffu) == b0 && (t >> 24) == b0;
    if (t != 0u && !uniform) return t;
  }
}

int decode_common(const kvc_layer* L, const void* q, const void* capsules, int B, int R, const void* K_txt,
                  const void* V_txt, int T, int T_cap, void* out, void* workspace, cudaStream_t st, const int* R_b,
                  const int* T_b) {
  if (!L || B < 0 || R < 0 || T < 0 || T_cap < T) return KVC_ERR_ARG;
  if (B == 0) return KVC_OK;
  if (R == 0 && T == 0) return KVC_ERR_SHAPE;
  if (!q || !out || (R > 0 && !capsules) || (T > 0 && (!K_txt || !V_txt))) return KVC_ERR_ARG;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255)) return KVC_ERR_WORKSPACE;

  DecodeArgs a{};
  a.ws = ws_layout(L, B, R, T);
  char* ws = static_cast<char*>(workspace);
  a.q = q;
  a.Kc = capsules;
  a.Vc = capsules ? static_cast<const char*>(capsules) + key_part_bytes(L, B, R) : nullptr;
  a.K_txt = K_txt; a.V_txt = V_txt;
  a.theta = L->desc.theta; a.U = L->desc.U; a.mu = L->desc.mu;
  a.out = out;
  a.B = B; a.H_kv = L->desc.H_kv; a.G = L->G; a.R = R; a.m = L->mk; a.ms = (L->mk + 15) / 16 * 16; a.n = L->desc.n;
  a.mv = L->mv; a.msv = (L->mv + 15) / 16 * 16;
  a.id_theta = L->mode == KVC_MODE_V_ONLY; a.id_U = L->mode == KVC_MODE_K_ONLY;
  a.T = T; a.T_cap = T_cap > 0 ? T_cap : 1; a.Ts = a.ws.Ts;
  a.passthrough = L->passthrough;
  a.S = reinterpret_cast<float*>(ws + a.ws.off_S);
  a.Sb = reinterpret_cast<__nv_bfloat16*>(ws + a.ws.off_S);
  a.s_txt = reinterpret_cast<float*>(ws + a.ws.off_stxt);
  a.W = reinterpret_cast<float*>(ws + a.ws.off_W);
  a.wstat = reinterpret_cast<float2*>(ws + a.ws.off_wstat);
  a.Wcomb = reinterpret_cast<float*>(ws + a.ws.off_Wc);
  a.statc = reinterpret_cast<float4*>(ws + a.ws.off_statc);
  a.ypart = reinterpret_cast<float*>(ws + a.ws.off_ypart);
  a.ystat = reinterpret_cast<float2*>(ws + a.ws.off_ystat);
  a.cnt = reinterpret_cast<int*>(ws + a.ws.off_cnt);
  a.fcnt = reinterpret_cast<unsigned long long*>(ws + a.ws.off_fcnt);
  a.token = next_token();
  a.status = a.cnt + (size_t)B * L->desc.H_kv;
  a.fpart_y = reinterpret_cast<float*>(ws + a.ws.off_fpy);
  a.fpart_ml = reinterpret_cast<float2*>(ws + a.ws.off_fpml);
  a.split_base = ws + a.ws.off_split;
  a.resident_base = ws + a.ws.off_resident;
  a.R_b = R_b; a.T_b = T_b;
  a.early_capsules = L->capsules_fresh ? 0 : 1;
  const_cast<kvc_layer*>(L)->capsules_fresh = 0;

  // bf16 storage with TMA-compatible shapes and pointers: the whole of Algorithm 1 in one kernel
  {
    // R == 0 (text rows only, the uncompressed comparator): the same kernel with text stages only
    // rho = 0 stores K and V verbatim: vision rows and text rows are attended as plain rows by the text-only mode
    const bool plain = R == 0 || L->passthrough;
    // one-sided modes are served by the three-phase kernels below; so are per-sequence lengths, except on the shapes the
    // resident-parameter kernel takes (it reads the lengths itself)
    const bool ragged = R_b != nullptr || T_b != nullptr;
    const bool one_sided = (R > 0 && L->mode != KVC_MODE_KV) || ragged;
    const uintptr_t align = reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(capsules) |
                            reinterpret_cast<uintptr_t>(out) | (T > 0 ? reinterpret_cast<uintptr_t>(K_txt) |
                            reinterpret_cast<uintptr_t>(V_txt) : 0) | reinterpret_cast<uintptr_t>(L->desc.mu);
    // Short blocks whose theta and U fit shared memory (n <= 256, m <= 128, G <= 8) take the resident-parameter kernel: on
    // the n = 256, G = 7, m = 103 shape it ran ahead of the other one-kernel variants at every batch measured (1, 4, 16:
    // 19.2 / 19.5 / 42.4 us against 22.4 / 23.5 / 83.7 us).  KVC_EXPANSION=resident forces it, any other value keeps it off.
    if (!plain && L->mode == KVC_MODE_KV && (align & 15) == 0 && (L->use_tc == 4 || L->use_tc == 0)) {
      const ResidentPlan rp = plan_resident(L, B, R, T);
      if (rp.ok) {
        bool encoded = false;
        const cudaError_t re = launch_resident(L, a, rp, st, &encoded);
        if (encoded) return cuda_status(re);
      }
    }
    if (!plain && !one_sided && (align & 15) == 0 && T <= 64 * SP_OUT_ROWS * SP_TEXT_CHUNK && use_split(L, B, R)) {
      const SplitPlan sp = plan_split(L, B, R);
      bool encoded = false;
      const cudaError_t se = launch_split(L, a, sp, st, &encoded);
      if (encoded) return cuda_status(se);
    }
    FusedPlan fp = plain ? plan_fused_text(L, B, R * L->desc.n + T) : plan_fused(L, B, R);
    if (one_sided) fp.ok = 0;
    if (fp.ok && (align & 15) == 0) {
      bool encoded = false;
      const cudaError_t fe = launch_fused(L, a, fp, st, &encoded);
      if (encoded) return cuda_status(fe);
    }
  }

  cudaError_t e = launch_scores(a, L->desc.dtype, st);
  if (e == cudaSuccess) e = launch_expand(a, L->desc.dtype, st);
  if (e == cudaSuccess) e = launch_output(a, L->desc.dtype, st);
  return cuda_status(e);
}
}  // namespace kvc

extern "C" {

int kvc_decode_attend(const kvc_layer* L, const void* q, const void* capsules, int B, int R, const void* K_txt,
                      const void* V_txt, int T, int T_cap, void* out, void* workspace, void* stream) {
  return decode_common(L, q, capsules, B, R, K_txt, V_txt, T, T_cap, out, workspace,
                       static_cast<cudaStream_t>(stream));
}

int kvc_decode_attend_ragged(const kvc_layer* L, const void* q, const void* capsules, int B, int R_max, const int* R_b,
                             const void* K_txt, const void* V_txt, int T_max, const int* T_b, int T_cap, void* out,
                             void* workspace, void* stream) {
  return decode_common(L, q, capsules, B, R_max, K_txt, V_txt, T_max, T_cap, out, workspace,
                       static_cast<cudaStream_t>(stream), R_b, T_b);
}

int kvc_compress_ragged(const kvc_layer* L, const void* K_vis, const void* V_vis, int B, int N_cap, const int* N_v,
                        int R_max, void* capsules, void* K_tail, void* V_tail, int T_cap, int* R_b, int* T_b, void* stream) {
  if (!L || B < 0 || N_cap < 0 || R_max < 0 || T_cap < 0) return KVC_ERR_ARG;
  if (B == 0) return KVC_OK;
  if (!N_v || !R_b || !T_b || (N_cap > 0 && (!K_vis || !V_vis)) || (R_max > 0 && !capsules) ||
      (T_cap > 0 && (!K_tail || !V_tail)))
    return KVC_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const_cast<kvc_layer*>(L)->capsules_fresh = 1;
  cudaError_t e = cudaMemsetAsync(L->d_cstatus, 0, sizeof(int), st);
  if (e != cudaSuccess) return cuda_status(e);
  void* Vc = capsules ? static_cast<char*>(capsules) + key_part_bytes(L, B, R_max) : nullptr;
  return cuda_status(launch_compress_ragged(L, K_vis, V_vis, B, N_cap, N_v, R_max, capsules, Vc, K_tail, V_tail, T_cap,
                                            R_b, T_b, st));
}

int kvc_attend_full(const kvc_layer* L, const void* q, const void* K, const void* V, int B, int S, int S_cap,
                    void* out, void* workspace, void* stream) {
  return decode_common(L, q, nullptr, B, 0, K, V, S, S_cap, out, workspace, static_cast<cudaStream_t>(stream));
}

int kvc_collapse_theta(const void* W1, const void* W2, int H_kv, int m, int k, int n, kvc_dtype dtype, void* theta_out,
                       void* stream) {
  if (!W1 || !W2 || !theta_out) return KVC_ERR_ARG;
  if (H_kv < 1 || m < 1 || k < 1 || n < 1 || H_kv > 65535 || (m + 63) / 64 > 65535) return KVC_ERR_SHAPE;
  if (dtype != KVC_F32 && dtype != KVC_BF16) return KVC_ERR_DTYPE;
  return cuda_status(kvc::launch_collapse_theta(W1, W2, theta_out, H_kv, m, k, n, (int)dtype, static_cast<cudaStream_t>(stream)));
}

int kvc_selftest_bounded_wait(void* stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int* d_status = nullptr;
  cudaError_t e = cudaMalloc(&d_status, sizeof(int));
  if (e != cudaSuccess) return cuda_status(e);
  int h_status = KVC_ERR_CUDA;
  e = cudaMemsetAsync(d_status, 0, sizeof(int), st);
  if (e == cudaSuccess) {
    kvc::launch_wait_selftest(d_status, st);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(&h_status, d_status, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  cudaFree(d_status);
  if (e != cudaSuccess) return cuda_status(e);
  return h_status;
}

int kvc_read_device_status(const kvc_layer* L, int B, int R, int T, const void* workspace, int* status_out) {
  if (!L || !status_out || B < 0 || R < 0 || T < 0) return KVC_ERR_ARG;
  if (!workspace) {                           // the fixed scratch array of kvc_decode_attend_static on this device
    void* p = nullptr;
    const int s = kvc::static_scratch(&p);
    if (s != KVC_OK) return s;
    workspace = p;
  }
  const WsLayout w = ws_layout(L, B, R, T);
  const char* p = static_cast<const char*>(workspace) + w.off_cnt + sizeof(int) * (size_t)B * L->desc.H_kv;
  return cudaMemcpy(status_out, p, sizeof(int), cudaMemcpyDeviceToHost) == cudaSuccess ? KVC_OK : KVC_ERR_CUDA;
}

int kvc_read_compress_status(const kvc_layer* L, int* status_out) {
  if (!L || !status_out) return KVC_ERR_ARG;
  return cudaMemcpy(status_out, L->d_cstatus, sizeof(int), cudaMemcpyDeviceToHost) == cudaSuccess ? KVC_OK : KVC_ERR_CUDA;
}

int kvc_export_maps(const kvc_layer* L, int R, int32_t* idx_out, int32_t* group_out) {
  if (!L || R < 0) return KVC_ERR_ARG;
  if (idx_out) {
    if (cudaMemcpy(idx_out, L->d_idx, (size_t)L->desc.H_kv * L->m * sizeof(int32_t), cudaMemcpyDeviceToHost) !=
        cudaSuccess)
      return KVC_ERR_CUDA;
  }
  if (group_out && R > 0) {
    // written by a kernel with the row arithmetic of the key selection (block r, offset i -> row r*n + i)
    const size_t bytes = (size_t)R * L->desc.n * 2 * sizeof(int32_t);
    int32_t* d = nullptr;
    if (cudaMalloc(&d, bytes) != cudaSuccess) return cuda_status(cudaGetLastError());
    cudaError_t e = cudaMemset(d, 0xff, bytes);
    if (e == cudaSuccess) e = kvc::launch_export_groups(d, R, L->desc.n, nullptr);
    if (e == cudaSuccess) e = cudaMemcpy(group_out, d, bytes, cudaMemcpyDeviceToHost);
    cudaFree(d);
    if (e != cudaSuccess) return cuda_status(e);
  }
  return KVC_OK;
}

}  // extern "C"
