// Host side of the three-kernel bf16 decode path: launch plan, workspace regions, tensor maps, the three launches.
#include "kvc_split.cuh"

namespace kvc {

cudaError_t launch_split_scores(const CUtensorMap& tmK, const SplitArgs& a, const SplitPlan& p, cudaStream_t st);
cudaError_t launch_split_expand(const CUtensorMap* tm, const SplitArgs& a, const SplitPlan& p, cudaStream_t st);
cudaError_t launch_split_output(const CUtensorMap* tm, const SplitArgs& a, const SplitPlan& p, cudaStream_t st);

constexpr uint32_t SP_SMEM_LIMIT = 232448;      // 227 KB per CTA on sm_100

SplitPlan plan_split(const kvc_layer* L, int B, int R) {
  SplitPlan p{};
  const int G = L->G, n = L->desc.n, m = L->m, H_kv = L->desc.H_kv;
  if (L->desc.dtype != KVC_BF16 || L->passthrough || R < 1 || B < 1 || n % 64 != 0 || G > 16) return p;
  if ((reinterpret_cast<uintptr_t>(L->desc.theta) | reinterpret_cast<uintptr_t>(L->desc.U)) & 15) return p;
  const int sms = L->num_sms > 0 ? L->num_sms : 148;
  p.rows_h = B * R * G;
  p.ntile = ceil_div(p.rows_h, SP_TILE_ROWS);
  p.ms = (m + 7) & ~7;
  p.nk1 = ceil_div(m, 64);
  // ranges of the n axis: widths of 64..256 columns that divide n; the fewest ranges that still give most SMs a CTA
  const int ncg = n / 64;
  p.NS = 0;
  for (int ns = 1; ns <= ncg; ++ns) {
    if (ncg % ns != 0 || n / ns > 256) continue;
    p.NS = ns;
    if ((long long)H_kv * p.ntile * ns >= (sms * 2) / 3) break;
  }
  if (p.NS == 0) return p;
  p.NW = n / p.NS;
  if ((long long)R * p.NS > 128) return p;            // the output kernel keeps a factor per (block, range, head) in shared memory
  // passes over the weights: at most 512 tensor-memory columns each, cut into one or two boxes of rows of U
  const int mpad = (m + 15) & ~15;
  p.npass = ceil_div(mpad, 512);
  // one pass: whole 32-column steps; several: whole 64-column tiles, so that no pass stores into the next one's columns
  p.prow = p.npass == 1 ? ((mpad + 31) & ~31) : ((ceil_div(mpad, p.npass) + 63) & ~63);
  p.nbox = p.prow > 256 ? 2 : 1;
  p.brow = p.prow / p.nbox;
  int cols = p.prow > p.NW ? p.prow : p.NW;
  p.tmem_cols = 32;
  while (p.tmem_cols < cols) p.tmem_cols <<= 1;
  p.e_p_bytes = (uint32_t)p.NW * 256u;
  const uint32_t st1 = 16384u + (uint32_t)(p.NW / 64) * 8192u, st2 = (uint32_t)p.prow * 128u;
  p.e_stage_bytes = ((st1 > st2 ? st1 : st2) + 1023u) & ~1023u;
  p.e_stages = (int)((SP_SMEM_LIMIT - 5120u - p.e_p_bytes) / p.e_stage_bytes);
  if (p.e_stages > 4) p.e_stages = 4;
  if (p.e_stages < 2) return p;
  p.e_smem = (size_t)p.e_p_bytes + (size_t)p.e_stages * p.e_stage_bytes + 1024;
  p.e_grid = H_kv * p.ntile * p.NS;
  // score kernel
  p.s_tiles_bh = ceil_div(R * m, SP_TILE_ROWS);
  p.s_stages = 6;
  p.s_smem = (size_t)p.s_stages * 32768 + 1024;
  {
    const long long items = (long long)B * H_kv * p.s_tiles_bh;
    p.s_grid = (int)(items < sms ? items : sms);
  }
  // output kernel
  p.vt = ceil_div(m, SP_OUT_ROWS);
  p.o_w_bytes = (uint32_t)(p.NS * G) * 128u;
  p.o_stage_bytes = (16384u + p.o_w_bytes + 1023u) & ~1023u;
  {
    // CTAs per (sequence, KV head): as many as the SMs allow (the same for every pair), at most one per value tile
    const long long bh = (long long)B * H_kv;
    const long long vb = (long long)R * p.vt;
    long long cpb = sms / bh;
    if (cpb < 1) cpb = 1;
    if (cpb > vb) cpb = vb;
    p.o_cpb = (int)cpb;
    p.o_grid = (int)(cpb > 1 ? bh * cpb : (bh < sms ? bh : sms));
  }
  {
    const int NH = G > 8 ? 2 : 1;
    uint32_t off = 0;
    auto take = [&](uint32_t bytes) { uint32_t o = off; off = (off + bytes + 127u) & ~127u; return o; };
    p.o_off_q = take(16u * (uint32_t)D * 4u);                       // summed accumulators of a pair
    p.o_off_fac = take((uint32_t)(R * p.NS) * (uint32_t)SO_FAC_PITCH * 8u);
    p.o_off_red = take(8u * NH * 8u * (uint32_t)D * 4u);
    p.o_off_stat = take((uint32_t)(32 + 2 * (p.o_cpb + 64) * 16) * 4u);   // up to 64 text chunks (16384 text rows)
    if (off + 2048u + 2 * p.o_stage_bytes > SP_SMEM_LIMIT) return p;
    p.o_stages = (int)((SP_SMEM_LIMIT - 2048u - off) / p.o_stage_bytes);
    if (p.o_stages > SP_MAX_STAGES) p.o_stages = SP_MAX_STAGES;
    const uint32_t ring = (uint32_t)p.o_stages * p.o_stage_bytes;
    p.o_off_q += ring; p.o_off_fac += ring; p.o_off_red += ring; p.o_off_stat += ring;
    p.o_smem = (size_t)ring + off + 1024;
  }
  p.ok = 1;
  return p;
}

SplitWs split_ws(const kvc_layer* L, const SplitPlan& p, int B, int R, int T) {
  SplitWs w{};
  (void)R;
  const int H_kv = L->desc.H_kv, G = L->G;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  w.off_S = take(sizeof(__nv_bfloat16) * (size_t)H_kv * p.rows_h * p.ms);
  w.off_Wp = take(sizeof(__nv_bfloat16) * (size_t)H_kv * p.NS * p.rows_h * p.ms);
  w.off_stat = take(sizeof(float2) * (size_t)H_kv * p.NS * p.rows_h);
  const size_t nslot = (size_t)p.o_cpb;          // one slot per CTA of a pair; a pair served by one CTA still parks its part there
  w.off_py = take(sizeof(float) * (size_t)B * H_kv * nslot * G * D);
  w.off_pml = take(sizeof(float2) * (size_t)B * H_kv * nslot * G);
  w.off_cnt = take(sizeof(int) * (size_t)B * H_kv);
  const size_t nct = (size_t)ceil_div(ceil_div(T > 0 ? T : 0, SP_OUT_ROWS), SP_TEXT_CHUNK);
  w.off_tpy = take(sizeof(float) * (size_t)B * H_kv * nct * G * D);
  w.off_tpml = take(sizeof(float2) * (size_t)B * H_kv * nct * G);
  w.bytes = off;
  return w;
}

cudaError_t launch_split(const kvc_layer* L, const DecodeArgs& a, const SplitPlan& p, cudaStream_t st, bool* encoded) {
  const int H_kv = a.H_kv, m = a.m, n = a.n, R = a.R, B = a.B, G = a.G;
  *encoded = false;
  char* ws = reinterpret_cast<char*>(a.split_base);
  const SplitWs w = split_ws(L, p, B, R, a.T);
  CUtensorMap tmK, tmS, tmTh, tmU, tmWs, tmO[4];
  {
    // K_tilde as (64 channels, R m rows of a pair, channel half, pairs): a box lands as [half][128 rows][64]; rows past the
    // pair's last are zero-filled, not read
    const uint64_t dims[4] = {64ull, (uint64_t)R * m, 2ull, (uint64_t)B * H_kv};
    const uint64_t str[3] = {256ull, 128ull, (uint64_t)R * m * 256};
    const uint32_t box[4] = {64u, (uint32_t)SP_TILE_ROWS, 2u, 1u};
    if (!encode_tensor_map_bf16(&tmK, a.Kc, 4, dims, str, box)) return cudaSuccess;
  }
  {
    const uint64_t dims[3] = {(uint64_t)m, (uint64_t)p.rows_h, (uint64_t)H_kv};
    const uint64_t str[2] = {(uint64_t)p.ms * 2, (uint64_t)p.rows_h * p.ms * 2};
    const uint32_t box[3] = {64u, (uint32_t)SP_TILE_ROWS, 1u};
    if (!encode_tensor_map_bf16(&tmS, ws + w.off_S, 3, dims, str, box)) return cudaSuccess;
  }
  {
    // theta [H_kv][m][n] viewed as (64 columns, m rows, n/64 column groups, H_kv): a box lands as [group][row][64]
    const uint64_t dims[4] = {64ull, (uint64_t)m, (uint64_t)(n / 64), (uint64_t)H_kv};
    const uint64_t str[3] = {(uint64_t)n * 2, 128ull, (uint64_t)m * n * 2};
    const uint32_t box[4] = {64u, 64u, (uint32_t)(p.NW / 64), 1u};
    if (!encode_tensor_map_bf16(&tmTh, a.theta, 4, dims, str, box)) return cudaSuccess;
  }
  {
    const uint64_t dims[3] = {(uint64_t)n, (uint64_t)m, (uint64_t)H_kv};
    const uint64_t str[2] = {(uint64_t)n * 2, (uint64_t)m * n * 2};
    const uint32_t box[3] = {64u, (uint32_t)p.brow, 1u};
    if (!encode_tensor_map_bf16(&tmU, a.U, 3, dims, str, box)) return cudaSuccess;
  }
  {
    // V_tilde as (64 channels, m rows of a block, channel half, blocks of all pairs): a box lands as [half][64 rows][64]
    const uint64_t dims[4] = {64ull, (uint64_t)m, 2ull, (uint64_t)B * H_kv * R};
    const uint64_t str[3] = {256ull, 128ull, (uint64_t)m * 256};
    const uint32_t box[4] = {64u, (uint32_t)SP_OUT_ROWS, 2u, 1u};
    if (!encode_tensor_map_bf16(&tmO[0], a.Vc, 4, dims, str, box)) return cudaSuccess;
  }
  if (a.T > 0) {
    // the text rows as (64 channels, T rows, channel half, H_kv, B): a box lands as [half][64 rows][64]
    const uint64_t dims[5] = {64ull, (uint64_t)a.T, 2ull, (uint64_t)H_kv, (uint64_t)B};
    const uint64_t str[4] = {256ull, 128ull, (uint64_t)a.T_cap * 256, (uint64_t)H_kv * a.T_cap * 256};
    const uint32_t box[5] = {64u, (uint32_t)SP_OUT_ROWS, 2u, 1u, 1u};
    if (!encode_tensor_map_bf16(&tmO[1], a.K_txt, 5, dims, str, box)) return cudaSuccess;
    if (!encode_tensor_map_bf16(&tmO[2], a.V_txt, 5, dims, str, box)) return cudaSuccess;
  } else {
    tmO[1] = tmO[0];
    tmO[2] = tmO[0];
  }
  {
    // partial weights as (m columns, expansion rows, ranges, H_kv): a box = 64 columns of the G rows of a block, all ranges
    const uint64_t dims[4] = {(uint64_t)m, (uint64_t)p.rows_h, (uint64_t)p.NS, (uint64_t)H_kv};
    const uint64_t str[3] = {(uint64_t)p.ms * 2, (uint64_t)p.rows_h * p.ms * 2, (uint64_t)p.NS * p.rows_h * p.ms * 2};
    const uint32_t box[4] = {64u, (uint32_t)G, (uint32_t)p.NS, 1u};
    if (!encode_tensor_map_bf16(&tmO[3], ws + w.off_Wp, 4, dims, str, box, false)) return cudaSuccess;
    // the same tensor as the expansion kernel stores it: 64 columns of the 128 rows of a tile, swizzled rows
    const uint32_t sbox[4] = {64u, (uint32_t)SP_TILE_ROWS, 1u, 1u};
    if (!encode_tensor_map_bf16(&tmWs, ws + w.off_Wp, 4, dims, str, sbox)) return cudaSuccess;
  }
  *encoded = true;

  SplitArgs sa{};
  sa.q = static_cast<const __nv_bfloat16*>(a.q);
  sa.mu = static_cast<const __nv_bfloat16*>(a.mu);
  sa.out = static_cast<__nv_bfloat16*>(a.out);
  sa.S = reinterpret_cast<__nv_bfloat16*>(ws + w.off_S);
  sa.Wp = reinterpret_cast<__nv_bfloat16*>(ws + w.off_Wp);
  sa.stat = reinterpret_cast<float2*>(ws + w.off_stat);
  sa.py = reinterpret_cast<float*>(ws + w.off_py);
  sa.pml = reinterpret_cast<float2*>(ws + w.off_pml);
  sa.cnt = reinterpret_cast<int*>(ws + w.off_cnt);
  sa.tpy = reinterpret_cast<float*>(ws + w.off_tpy);
  sa.tpml = reinterpret_cast<float2*>(ws + w.off_tpml);
  sa.status = a.status;
  sa.early = a.early_capsules;
  sa.B = B; sa.H_kv = H_kv; sa.G = G; sa.R = R; sa.m = m; sa.n = n; sa.T = a.T;
  sa.rows_h = p.rows_h; sa.ntile = p.ntile; sa.NS = p.NS; sa.NW = p.NW; sa.ms = p.ms; sa.nk1 = p.nk1;
  sa.npass = p.npass; sa.prow = p.prow; sa.nbox = p.nbox; sa.brow = p.brow; sa.tmem_cols = p.tmem_cols;
  sa.e_stages = p.e_stages; sa.e_stage_bytes = p.e_stage_bytes;
  sa.s_tiles_bh = p.s_tiles_bh; sa.s_stages = p.s_stages;
  sa.vt = p.vt; sa.o_stages = p.o_stages; sa.o_stage_bytes = p.o_stage_bytes;
  sa.o_cpb = p.o_cpb;
  sa.o_off_q = p.o_off_q; sa.o_off_fac = p.o_off_fac; sa.o_off_red = p.o_off_red; sa.o_off_stat = p.o_off_stat;

  sa.e_grid = p.e_grid;
  {
    // text CTAs: the SMs the expansion CTAs leave idle in their last wave (a dozen at least), one item each at most
    const int sms = L->num_sms > 0 ? L->num_sms : 148;
    const long long items = (long long)B * H_kv * ceil_div(ceil_div(a.T, SP_OUT_ROWS), SP_TEXT_CHUNK);
    int idle = sms - p.e_grid % sms;
    if (idle < 12) idle = 12;
    sa.tx_grid = a.T > 0 ? (int)(items < idle ? items : idle) : 0;
  }
  const CUtensorMap tmE[6] = {tmS, tmTh, tmU, tmWs, tmO[1], tmO[2]};
  cudaError_t e = launch_split_scores(tmK, sa, p, st);
  if (e == cudaSuccess) e = launch_split_expand(tmE, sa, p, st);
  if (e == cudaSuccess) e = launch_split_output(tmO, sa, p, st);
  return e;
}

}  // namespace kvc
