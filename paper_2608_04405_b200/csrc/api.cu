// C-ABI entry points: argument validation, context life cycle, stream plumbing.
#include <new>
#include <stdlib.h>
#include <string.h>
#include "common.cuh"
#include "sched_host.h"

cudaError_t bpc_launch_decode_bf16(bpc_ctx*, const DecodeParams&, cudaStream_t);
cudaError_t bpc_launch_decode_f32(bpc_ctx*, const DecodeParams&, cudaStream_t);
cudaError_t bpc_decode_limits_bf16(const bpc_ctx*, int, int*, int*, size_t*);
cudaError_t bpc_decode_limits_f32(const bpc_ctx*, int, int*, int*, size_t*);
cudaError_t bpc_launch_decode_bf16_eas(bpc_ctx*, const DecodeParams&, cudaStream_t);
cudaError_t bpc_launch_decode_f32_eas(bpc_ctx*, const DecodeParams&, cudaStream_t);
cudaError_t bpc_decode_limits_bf16_eas(const bpc_ctx*, int, int*, int*, size_t*);
cudaError_t bpc_decode_limits_f32_eas(const bpc_ctx*, int, int*, int*, size_t*);
cudaError_t bpc_launch_decode_bf16_stream(bpc_ctx*, const DecodeParams&, cudaStream_t);
cudaError_t bpc_launch_decode_f32_stream(bpc_ctx*, const DecodeParams&, cudaStream_t);
cudaError_t bpc_launch_decode_bf16_k8(bpc_ctx*, const DecodeParams&, cudaStream_t);
cudaError_t bpc_launch_decode_f32_k8(bpc_ctx*, const DecodeParams&, cudaStream_t);
cudaError_t bpc_decode_limits_bf16_k8(const bpc_ctx*, int, int*, int*, size_t*);
cudaError_t bpc_decode_limits_f32_k8(const bpc_ctx*, int, int*, int*, size_t*);
cudaError_t bpc_launch_decode_bf16_w7(bpc_ctx*, const DecodeParams&, cudaStream_t);
cudaError_t bpc_launch_decode_f32_w7(bpc_ctx*, const DecodeParams&, cudaStream_t);
cudaError_t bpc_decode_limits_bf16_w7(const bpc_ctx*, int, int*, int*, size_t*);
cudaError_t bpc_decode_limits_f32_w7(const bpc_ctx*, int, int*, int*, size_t*);

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bpc_status check_cfg(const bpc_config* c) {
  if (c == nullptr) return BPC_ERR_INVALID_ARG;
  if (c->batch < 1 || c->n_kv_heads < 1 || c->n_q_heads < 1 || c->n_max < 1) return BPC_ERR_INVALID_ARG;
  if (c->head_dim != BPC_D) return BPC_ERR_UNSUPPORTED;
  if (c->code_bits != 32 && c->code_bits != 64 && c->code_bits != 128 && c->code_bits != 256) return BPC_ERR_UNSUPPORTED;
  if (c->code_bits == 32 && c->n_max % 4 != 0) return BPC_ERR_INVALID_ARG;   // 16-byte aligned code rows per unit
  if (c->n_q_heads % c->n_kv_heads != 0) return BPC_ERR_INVALID_ARG;
  if (c->n_q_heads / c->n_kv_heads > BPC_MAX_GROUP) return BPC_ERR_UNSUPPORTED;
  if (c->kv_dtype != BPC_BF16 && c->kv_dtype != BPC_F32) return BPC_ERR_UNSUPPORTED;
  if (c->score_mode != BPC_SCORE_HAMMING && c->score_mode != BPC_SCORE_WEIGHTED7) return BPC_ERR_INVALID_ARG;
  // weighted scores are kept as 16-bit keys, shifted right by up to two bits when the largest possible score
  // 127 * G * b needs more (the dropped bits are recovered for the keys at the threshold)
  if (c->score_mode == BPC_SCORE_WEIGHTED7 && 127LL * (c->n_q_heads / c->n_kv_heads) * c->code_bits > 4LL * 65535) return BPC_ERR_UNSUPPORTED;
  const long long units = (long long)c->batch * c->n_kv_heads;
  if (c->hash_sets != units && c->hash_sets != c->n_kv_heads) return BPC_ERR_INVALID_ARG;
  if (c->residual_correction != 0 && c->residual_correction != 1) return BPC_ERR_INVALID_ARG;
  if (!(c->sm_scale >= 0.f)) return BPC_ERR_INVALID_ARG;
  if (c->kv_row_stride != 0 && (c->kv_row_stride < c->head_dim || c->kv_row_stride % 8 != 0)) return BPC_ERR_INVALID_ARG;
  if (c->eas_ppm < 0 || c->eas_ppm > 1000000) return BPC_ERR_INVALID_ARG;
  if (c->fit_power_iters < 0 || c->fit_power_iters > 8) return BPC_ERR_INVALID_ARG;
  if (c->eas_ppm > 0 && (c->residual_correction == 0 || c->score_mode != BPC_SCORE_HAMMING)) return BPC_ERR_UNSUPPORTED;
  if (c->eas_ppm > 0 && ((long long)c->n_max * c->eas_ppm + 999999) / 1000000 > 16384) return BPC_ERR_UNSUPPORTED;
  if (c->n_max % 2 != 0) return BPC_ERR_INVALID_ARG;   // keeps every unit's code rows 16-byte aligned at 64 bits
  if (c->n_max > (1 << 26)) return BPC_ERR_UNSUPPORTED; // far above what a cluster's shared memory holds; keeps index math in 32 bits
  return BPC_OK;
}

bpc_status cuda_fail(bpc_ctx* ctx, cudaError_t e) {
  if (ctx) ctx->last_cuda_error = (int32_t)e;
  (void)cudaGetLastError();
  return BPC_ERR_CUDA;
}

// Largest score key (sum of |A_j| after removing the common factor), the shift that maps keys to at most 2048
// histogram bins, and the number of bins.
int max_score_key(const bpc_ctx* ctx) {
  const int G = ctx->group, b = ctx->cfg.code_bits;
  if (ctx->cfg.score_mode == BPC_SCORE_WEIGHTED7) return 127 * G * b;
  return (G * b) >> ((G % 2 == 0) ? 1 : 0);
}
// (the histogram is taken over the stored keys, which are at most 16 bits wide)
int max_stored_key(const bpc_ctx* ctx) { const int m = max_score_key(ctx); return m > 65535 ? 65535 : m; }
int hist_shift(const bpc_ctx* ctx) {
  int s = 0;
  while ((max_stored_key(ctx) >> s) >= 2048) ++s;
  return s;
}
int hist_bins(const bpc_ctx* ctx) { return (max_stored_key(ctx) >> hist_shift(ctx)) + 1; }

cudaError_t decode_limits(const bpc_ctx* ctx, int /*unused*/, int* max_cluster, int* chunk_cap, size_t* smem) {
  const int nbins = hist_bins(ctx);
  if (ctx->cfg.score_mode == BPC_SCORE_WEIGHTED7)
    return ctx->cfg.kv_dtype == BPC_BF16 ? bpc_decode_limits_bf16_w7(ctx, nbins, max_cluster, chunk_cap, smem)
                                         : bpc_decode_limits_f32_w7(ctx, nbins, max_cluster, chunk_cap, smem);
  if (ctx->cfg.eas_ppm > 0)
    return ctx->cfg.kv_dtype == BPC_BF16 ? bpc_decode_limits_bf16_eas(ctx, nbins, max_cluster, chunk_cap, smem)
                                         : bpc_decode_limits_f32_eas(ctx, nbins, max_cluster, chunk_cap, smem);
  return ctx->cfg.kv_dtype == BPC_BF16 ? bpc_decode_limits_bf16(ctx, nbins, max_cluster, chunk_cap, smem)
                                       : bpc_decode_limits_f32(ctx, nbins, max_cluster, chunk_cap, smem);
}

// keys per block the kernel may assign (the larger of its plain and its fused-launch split), rounded to 64
int chunk_for(int n_max, int cs) {
  const int plain = (((n_max + cs - 1) / cs) + 63) & ~63;
  if (cs == 1) return plain;
  const int fused = bpc_fused_chunk(n_max, cs);
  return fused > plain ? fused : plain;
}

// Cluster size of the decode launch.  Candidates run from the smallest cluster whose blocks can hold n_max scores to
// the largest the device schedules, as long as a block keeps at least 1024 keys.  The phases of a block are bound by
// what one SM can have in flight, so more SMs per unit win until the grid no longer fits the device at once.  The
// estimate, in units of "time to scan one code", is
//   (waves of resident clusters) x (keys per block + 600 per block of the cluster for the merges across blocks
//                                   + 4000 per eight-row attention tile of a warp + 20 000 for hash and selection),
// with the attention tiles counted for a nominal budget of 2 % of n_max, at least 1024 keys (the budget itself is an
// argument of each call); the cheapest candidate is taken.  Measured on B200: 8 units pick 8 blocks at 32K keys and
// 10 at 128K; 16 units pick 6, 24 units 5, 40 units 3 at 128K.
int choose_cluster(const bpc_ctx* ctx, int chunk_cap, int max_cluster) {
  int cs = 1;
  while (cs <= max_cluster && (ctx->max_active[cs] < 1 || chunk_for(ctx->cfg.n_max, cs) > chunk_cap)) ++cs;
  if (cs > max_cluster) return 0;
  long long k_nom = ((long long)ctx->cfg.n_max * 20000 + 999999) / 1000000;
  if (k_nom < 1024) k_nom = 1024;
  if (k_nom > ctx->cfg.n_max) k_nom = ctx->cfg.n_max;
  int best = cs;
  long long best_cost = -1;
  for (int c = cs; c <= max_cluster; ++c) {
    if (ctx->max_active[c] < 1) continue;
    const int chunk = chunk_for(ctx->cfg.n_max, c);
    if (c > cs && chunk < 1024) break;
    const long long waves = (ctx->units + ctx->max_active[c] - 1) / ctx->max_active[c];
    const long long rows_per_warp = ((k_nom + c - 1) / c + 15) / 16;
    const long long tiles = (rows_per_warp + 7) / 8;
    const long long cost = waves * (chunk + 600LL * c + 4000LL * tiles + 20000LL);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = c; }
  }
  return best;
}


// ---- work-item decode kernel: which contexts it serves, its geometry and its scratch
bool sched_covers(const bpc_config& c) {
  return c.kv_dtype == BPC_BF16 && c.score_mode == BPC_SCORE_HAMMING && c.eas_ppm == 0 &&
         (long long)c.batch * c.n_kv_heads <= bpcdev::kSchedMaxUnits;
}

int round_up(long long x, int g) { return (int)(((x + g - 1) / g) * g); }

// keys per SCAN item: about 3.5 items per resident block over all units, a multiple of the granule, at most
// kSchedMaxRanges items per unit and at most 32768 keys (range histogram counts are 16-bit)
int sched_auto_ch(const bpc_ctx* ctx) {
  const long long total = (long long)ctx->units * ctx->cfg.n_max;
  long long ch = (long long)((double)total / (3.5 * ctx->sched_grid_max));
  ch = round_up(ch < 1 ? 1 : ch, ctx->sched_gran);
  int floor_ch = round_up((ctx->cfg.n_max + bpcdev::kSchedMaxRanges - 1) / bpcdev::kSchedMaxRanges, ctx->sched_gran);
  if (ch < floor_ch) ch = floor_ch;
  const int cap = (32768 / ctx->sched_gran) * ctx->sched_gran;
  if (ch > cap) ch = cap;
  return (int)ch;
}

cudaError_t sched_setup(bpc_ctx* ctx) {
  ctx->sched_ok = false;
  const bpc_config& c = ctx->cfg;
  if (!sched_covers(c)) return cudaSuccess;
  const int nbins = hist_bins(ctx);
  int per_sm = 0;
  cudaError_t e = bpc_sched_configure(ctx->group, c.code_bits, nbins, ctx->units, ctx->device, &ctx->sched_smem, &per_sm);
  if (e != cudaSuccess) { (void)cudaGetLastError(); return cudaSuccess; }   // not schedulable here: the cluster kernel serves
  if (per_sm < 1) return cudaSuccess;
  ctx->sched_grid_max = per_sm * ctx->sm_count;
  ctx->sched_gran = bpc_sched_granule(c.code_bits);
  ctx->sched_ch = sched_auto_ch(ctx);
  if ((c.n_max + ctx->sched_ch - 1) / ctx->sched_ch > bpcdev::kSchedMaxRanges) return cudaSuccess;   // context too long
  // scratch rows are sized for the smallest range length a caller may ask for
  int r_alloc = (c.n_max + ctx->sched_gran - 1) / ctx->sched_gran;
  if (r_alloc > bpcdev::kSchedMaxRanges) r_alloc = bpcdev::kSchedMaxRanges;
  ctx->sched_r_alloc = r_alloc;
  // attention slices per unit: one or more per range, at most ranges + ceil(k / rows per slice) <= ranges + 64 + ...
  int na = (c.n_max + bpcdev::kSchedListCap - 1) / bpcdev::kSchedListCap;
  ctx->sched_na_cap = r_alloc + (na < 64 ? 64 : na) + 1;
  ctx->sched_sc_stride = (c.n_max + 7) & ~7;
  const int gp = bpc_sched_padded_group(ctx->group);
  const int w32 = c.code_bits / 32;
  const int np = gp <= 2 ? 1 : (gp == 4 ? 2 : 3);
  ctx->sched_qp_words = (w32 * (2 + np) + 3) & ~3;
  const size_t U = (size_t)ctx->units;
  const size_t sync_words = bpcdev::kSchedSyncHead + U * bpcdev::kSchedSyncPerUnit;
  e = cudaMalloc(&ctx->sc_scores, U * ctx->sched_sc_stride * 2);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->sc_hist, U * r_alloc * (size_t)nbins * 2);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->sc_table, U * (r_alloc + 1) * sizeof(int4));
  if (e == cudaSuccess) e = cudaMalloc(&ctx->sc_planes, U * ctx->sched_qp_words * 4);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->sc_partials, U * ctx->sched_na_cap * (size_t)gp * (BPC_D + 2) * 4);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->sc_sync, sync_words * 4);
  if (e == cudaSuccess) e = cudaMemset(ctx->sc_sync, 0, sync_words * 4);
  if (e != cudaSuccess) return e;
  ctx->sched_ok = true;
  return cudaSuccess;
}

}  // namespace

cudaError_t bpc_plan_decode_geometry(bpc_ctx* ctx) {
  int mc[BPC_MAX_CLUSTER + 1] = {1}, cap = 0;
  cudaError_t e = decode_limits(ctx, 0, mc, &cap, nullptr);
  if (e != cudaSuccess) return e;
  ctx->max_cluster = mc[0];
  ctx->max_active[0] = 0;
  for (int i = 1; i <= BPC_MAX_CLUSTER; ++i) ctx->max_active[i] = mc[i];
  ctx->chunk_cap_limit = cap;
  ctx->cluster_size = choose_cluster(ctx, cap, ctx->max_cluster);
  ctx->streaming = false;
  ctx->byte_keys = false;
  // Byte score keys (Hamming scores with at most 256 distinct values, no safeguard): a block holds 2.5 times the keys,
  // so contexts of a million keys and more fit clusters that are all resident at once.  Taken when the 16-bit plan
  // would need the streaming selection or more waves of clusters than the byte plan (same kernel resources: the
  // occupancy answers of the plain variant are reused).
  if (ctx->cfg.score_mode == BPC_SCORE_HAMMING && ctx->cfg.eas_ppm == 0 && hist_shift(ctx) == 0 && hist_bins(ctx) <= 256 &&
      ctx->force_byte_keys >= 0 && !ctx->force_streaming) {
    int cap8 = 0;
    e = ctx->cfg.kv_dtype == BPC_BF16 ? bpc_decode_limits_bf16_k8(ctx, hist_bins(ctx), nullptr, &cap8, nullptr)
                                      : bpc_decode_limits_f32_k8(ctx, hist_bins(ctx), nullptr, &cap8, nullptr);
    if (e != cudaSuccess) return e;
    const int cs8 = choose_cluster(ctx, cap8, ctx->max_cluster);
    auto waves = [&](int cs) { return (ctx->units + ctx->max_active[cs] - 1) / ctx->max_active[cs]; };
    if (cs8 > 0 && (ctx->force_byte_keys > 0 || ctx->cluster_size == 0 || waves(cs8) < waves(ctx->cluster_size))) {
      ctx->byte_keys = true;
      ctx->cluster_size = cs8;
      ctx->chunk_cap_limit = cap8;
    }
  }
  const bool forced = ctx->force_streaming;                 // diagnostic switch: two-pass selection at any size
  if ((ctx->cluster_size == 0 || forced) && ctx->cfg.score_mode == BPC_SCORE_HAMMING && ctx->cfg.eas_ppm == 0) {
    // Units too long for the largest cluster's shared memory: no score is stored, the codes are read twice.  The
    // largest cluster size that still runs all units in one wave is used (at least the largest schedulable one).
    int cs = forced && ctx->cluster_size > 0 ? ctx->cluster_size : ctx->max_cluster;
    if (!(forced && ctx->cluster_size > 0))
      while (cs > 1 && ctx->units > ctx->max_active[cs]) --cs;
    ctx->cluster_size = cs;
    ctx->streaming = true;
  }
  return cudaSuccess;
}

extern "C" {
#pragma GCC visibility push(default)

const char* bpc_version(void) { return "bpc 0.1 (sm_100a)"; }

size_t bpc_codes_bytes(const bpc_config* c) {
  if (check_cfg(c) != BPC_OK) return 0;
  return (size_t)c->batch * c->n_kv_heads * (size_t)c->n_max * (c->code_bits / 8);
}

size_t bpc_fit_workspace_bytes(const bpc_config* c) {
  if (check_cfg(c) != BPC_OK) return 0;
  return bpc_fit_workspace_bytes_impl(c);
}

size_t bpc_fit_codes_offset(const bpc_config* c) {
  if (check_cfg(c) != BPC_OK) return 0;
  return bpc_fit_codes_offset_impl(c);
}

int64_t bpc_max_context(const bpc_config* c) {
  if (check_cfg(c) != BPC_OK) return 0;
  bpc_ctx tmp;
  memset(&tmp, 0, sizeof(tmp));
  tmp.cfg = *c;
  tmp.group = c->n_q_heads / c->n_kv_heads;
  if (cudaGetDevice(&tmp.device) != cudaSuccess) return 0;
  if (bpc_plan_decode_geometry(&tmp) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
  if (c->score_mode == BPC_SCORE_HAMMING && c->eas_ppm == 0) return (int64_t)1 << 26;   // streaming selection: no per-unit limit
  return (int64_t)tmp.max_cluster * tmp.chunk_cap_limit;
}

bpc_status bpc_create(const bpc_config* cfg, bpc_ctx** out) {
  if (out == nullptr) return BPC_ERR_INVALID_ARG;
  *out = nullptr;
  bpc_status s = check_cfg(cfg);
  if (s != BPC_OK) return s;
  bpc_ctx* ctx = new (std::nothrow) bpc_ctx;
  if (ctx == nullptr) return BPC_ERR_INVALID_ARG;
  memset(ctx, 0, sizeof(*ctx));
  ctx->cfg = *cfg;
  ctx->sm_scale_d = cfg->sm_scale == 0.f ? 0.08838834764831845 : (double)cfg->sm_scale;   // default 1/sqrt(128)
  ctx->units = cfg->batch * cfg->n_kv_heads;
  ctx->group = cfg->n_q_heads / cfg->n_kv_heads;
  ctx->use_pdl = true;
  ctx->row_stride = cfg->kv_row_stride == 0 ? cfg->head_dim : cfg->kv_row_stride;
  cudaError_t e = cudaGetDevice(&ctx->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device);
  const size_t b = cfg->code_bits, hs = cfg->hash_sets;
  const size_t esz = cfg->kv_dtype == BPC_BF16 ? 2 : 4;
  if (e == cudaSuccess) e = cudaMalloc(&ctx->P, hs * b * BPC_D * 4);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->P_h, hs * b * BPC_D * esz);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->P_hf, hs * b * BPC_D * 4);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->gram, hs * b * b * 4);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->unit_lens, (size_t)ctx->units * 4);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->sel_scratch, (size_t)ctx->units * cfg->n_max * 4);
  if (cfg->eas_ppm > 0) {
    ctx->eas_cap = (int)(((long long)cfg->n_max * cfg->eas_ppm + 999999) / 1000000);
    if (e == cudaSuccess) e = cudaMalloc(&ctx->key_err, (size_t)ctx->units * cfg->n_max * 4);
    if (e == cudaSuccess) e = cudaMalloc(&ctx->eas_idx, (size_t)ctx->units * ctx->eas_cap * 4);
    if (e == cudaSuccess) e = cudaMalloc(&ctx->eas_cnt, (size_t)ctx->units * 4);
    if (e == cudaSuccess) e = cudaMemset(ctx->eas_cnt, 0, (size_t)ctx->units * 4);
    if (e == cudaSuccess) e = cudaMemset(ctx->key_err, 0, (size_t)ctx->units * cfg->n_max * 4);
  }
  if (e == cudaSuccess) e = cudaMalloc(&ctx->dev_err, 4);
  if (e == cudaSuccess) e = cudaMemset(ctx->dev_err, 0, 4);
  if (e == cudaSuccess) e = cudaMemset(ctx->unit_lens, 0, (size_t)ctx->units * 4);
  if (e == cudaSuccess) e = cudaMallocHost(&ctx->lens_staging, (size_t)BPC_LENS_SLOTS * ctx->units * 4);
  for (int i = 0; i < BPC_LENS_SLOTS && e == cudaSuccess; ++i)
    e = cudaEventCreateWithFlags(&ctx->lens_event[i], cudaEventDisableTiming);
  ctx->host_lens = new (std::nothrow) int32_t[cfg->batch];
  if (ctx->host_lens) memset(ctx->host_lens, 0, sizeof(int32_t) * cfg->batch);
  if (e != cudaSuccess || ctx->host_lens == nullptr) {
    bpc_destroy(ctx);
    (void)cudaGetLastError();
    return BPC_ERR_CUDA;
  }
  e = bpc_plan_decode_geometry(ctx);
  if (e != cudaSuccess) { bpc_destroy(ctx); (void)cudaGetLastError(); return BPC_ERR_CUDA; }
  if (hist_bins(ctx) > 2048 || hist_shift(ctx) > 5) { bpc_destroy(ctx); return BPC_ERR_UNSUPPORTED; }
  if (ctx->cluster_size == 0) { bpc_destroy(ctx); return BPC_ERR_UNSUPPORTED; }
  *out = ctx;
  return BPC_OK;
}

bpc_status bpc_destroy(bpc_ctx* ctx) {
  if (ctx == nullptr) return BPC_ERR_INVALID_ARG;
  cudaFree(ctx->P); cudaFree(ctx->P_h); cudaFree(ctx->P_hf); cudaFree(ctx->gram);
  cudaFree(ctx->unit_lens); cudaFree(ctx->sel_scratch); cudaFree(ctx->dev_err);
  cudaFree(ctx->key_err); cudaFree(ctx->eas_idx); cudaFree(ctx->eas_cnt);
  cudaFree(ctx->sc_scores); cudaFree(ctx->sc_hist); cudaFree(ctx->sc_table); cudaFree(ctx->sc_planes);
  cudaFree(ctx->sc_partials); cudaFree(ctx->sc_sync);
  if (ctx->lens_staging) cudaFreeHost(ctx->lens_staging);
  for (int i = 0; i < BPC_LENS_SLOTS; ++i)
    if (ctx->lens_event[i]) cudaEventDestroy(ctx->lens_event[i]);
  delete[] ctx->host_lens;
  delete ctx;
  (void)cudaGetLastError();
  return BPC_OK;
}

bpc_status bpc_set_cluster_size(bpc_ctx* ctx, int32_t cs) {
  if (ctx == nullptr) return BPC_ERR_INVALID_ARG;
  const int cap = ctx->chunk_cap_limit, mc = ctx->max_cluster;
  if (cs == 0) {                                           // back to the library's own choice of geometry
    if (ctx->streaming) return BPC_OK;                     // keeps the size chosen at creation
    cs = choose_cluster(ctx, cap, mc);
    if (cs < 1) return BPC_ERR_UNSUPPORTED;
    ctx->cluster_size = cs;
    return BPC_OK;
  }
  if (cs < 1 || cs > mc || ctx->max_active[cs] < 1) return BPC_ERR_UNSUPPORTED;
  if (!ctx->streaming && chunk_for(ctx->cfg.n_max, cs) > cap) return BPC_ERR_UNSUPPORTED;
  ctx->cluster_size = cs;
  return BPC_OK;
}

int32_t bpc_plan_cluster_size(const bpc_config* cfg, const int32_t* max_active, int32_t chunk_cap) {
  if (check_cfg(cfg) != BPC_OK || max_active == nullptr || chunk_cap < 0) return 0;
  bpc_ctx tmp;
  memset(&tmp, 0, sizeof(tmp));
  tmp.cfg = *cfg;
  tmp.units = cfg->batch * cfg->n_kv_heads;
  tmp.group = cfg->n_q_heads / cfg->n_kv_heads;
  int mc = 0;
  for (int c = 1; c <= BPC_MAX_CLUSTER; ++c) {
    tmp.max_active[c] = max_active[c] > 0 ? max_active[c] : 0;
    if (tmp.max_active[c] > 0) mc = c;
  }
  if (mc == 0) return 0;
  return choose_cluster(&tmp, chunk_cap, mc);
}

int32_t bpc_get_cluster_size(bpc_ctx* ctx) { return ctx ? ctx->cluster_size : 0; }
int32_t bpc_uses_streaming(bpc_ctx* ctx) { return (ctx && ctx->streaming) ? 1 : 0; }

bpc_status bpc_set_seq_lens(bpc_ctx* ctx, const int32_t* host_lens, void* stream) {
  if (ctx == nullptr || host_lens == nullptr) return BPC_ERR_INVALID_ARG;
  const bpc_config& c = ctx->cfg;
  for (int i = 0; i < c.batch; ++i)
    if (host_lens[i] < 0 || host_lens[i] > c.n_max) return BPC_ERR_CAPACITY;
  // The per-unit lengths are staged in pinned memory owned by the context and copied asynchronously on `stream`: the
  // call does not wait for the stream.  A ring of staging slots, each guarded by an event recorded after its copy,
  // lets several calls be in flight; only a call that finds its slot's previous copy unfinished waits for that copy.
  const int slot = ctx->lens_slot;
  ctx->lens_slot = (slot + 1) % BPC_LENS_SLOTS;
  cudaError_t e = cudaEventSynchronize(ctx->lens_event[slot]);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  int32_t* tmp = ctx->lens_staging + (size_t)slot * ctx->units;
  for (int i = 0; i < c.batch; ++i) {
    ctx->host_lens[i] = host_lens[i];
    for (int h = 0; h < c.n_kv_heads; ++h) tmp[i * c.n_kv_heads + h] = host_lens[i];
  }
  e = cudaMemcpyAsync(ctx->unit_lens, tmp, (size_t)ctx->units * 4, cudaMemcpyHostToDevice, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaEventRecord(ctx->lens_event[slot], (cudaStream_t)stream);
  return e == cudaSuccess ? BPC_OK : cuda_fail(ctx, e);
}

bpc_status bpc_get_seq_lens(bpc_ctx* ctx, int32_t* host_out) {
  if (ctx == nullptr || host_out == nullptr) return BPC_ERR_INVALID_ARG;
  for (int i = 0; i < ctx->cfg.batch; ++i) host_out[i] = ctx->host_lens[i];
  return BPC_OK;
}

bpc_status bpc_set_projection(bpc_ctx* ctx, const float* P, void* stream) {
  if (ctx == nullptr || P == nullptr) return BPC_ERR_INVALID_ARG;
  const bpc_config& c = ctx->cfg;
  cudaError_t e = cudaMemcpyAsync(ctx->P, P, (size_t)c.hash_sets * c.code_bits * BPC_D * 4, cudaMemcpyDeviceToDevice,
                                  (cudaStream_t)stream);
  if (e == cudaSuccess) e = bpc_launch_finalize_projection(ctx, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  ctx->fitted = true;
  return BPC_OK;
}

bpc_status bpc_get_projection(bpc_ctx* ctx, float* P_out, float* Ph_out, float* gram_out, void* stream) {
  if (ctx == nullptr) return BPC_ERR_INVALID_ARG;
  if (!ctx->fitted) return BPC_ERR_NOT_FITTED;
  const bpc_config& c = ctx->cfg;
  const size_t pb = (size_t)c.hash_sets * c.code_bits * BPC_D * 4;
  cudaError_t e = cudaSuccess;
  if (P_out) e = cudaMemcpyAsync(P_out, ctx->P, pb, cudaMemcpyDeviceToDevice, (cudaStream_t)stream);
  if (e == cudaSuccess && Ph_out) e = cudaMemcpyAsync(Ph_out, ctx->P_hf, pb, cudaMemcpyDeviceToDevice, (cudaStream_t)stream);
  if (e == cudaSuccess && gram_out)
    e = cudaMemcpyAsync(gram_out, ctx->gram, (size_t)c.hash_sets * c.code_bits * c.code_bits * 4, cudaMemcpyDeviceToDevice,
                        (cudaStream_t)stream);
  return e == cudaSuccess ? BPC_OK : cuda_fail(ctx, e);
}

bpc_status bpc_fit(bpc_ctx* ctx, const void* k_cache, const float* v_star, void* workspace, size_t workspace_bytes,
                   void* stream) {
  if (ctx == nullptr || k_cache == nullptr || v_star == nullptr || workspace == nullptr) return BPC_ERR_INVALID_ARG;
  if (!aligned16(k_cache) || !aligned16(v_star) || !aligned16(workspace)) return BPC_ERR_INVALID_ARG;
  if (ctx->cfg.hash_sets != ctx->units) return BPC_ERR_UNSUPPORTED;
  if (workspace_bytes < bpc_fit_workspace_bytes_impl(&ctx->cfg)) return BPC_ERR_INVALID_ARG;
  int launches = 0;
  cudaError_t e = bpc_launch_fit(ctx, k_cache, v_star, workspace, (cudaStream_t)stream, &launches);
  ctx->launches += launches;
  if (e == cudaSuccess) e = bpc_launch_finalize_projection(ctx, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  ctx->fitted = true;
  return BPC_OK;
}

bpc_status bpc_encode_keys(bpc_ctx* ctx, const void* k_cache, uint64_t* codes, void* stream) {
  if (ctx == nullptr || k_cache == nullptr || codes == nullptr) return BPC_ERR_INVALID_ARG;
  if (!aligned16(k_cache) || !aligned16(codes)) return BPC_ERR_INVALID_ARG;
  if (!ctx->fitted) return BPC_ERR_NOT_FITTED;
  cudaError_t e = bpc_launch_encode_tc(ctx, k_cache, codes, (cudaStream_t)stream);
  if (e == cudaErrorNotSupported) {
    (void)cudaGetLastError();
    e = bpc_launch_encode_simple(ctx, k_cache, codes, (cudaStream_t)stream);
  }
  return e == cudaSuccess ? BPC_OK : cuda_fail(ctx, e);
}

int32_t bpc_eas_capacity(const bpc_config* c) {
  if (check_cfg(c) != BPC_OK || c->eas_ppm <= 0) return 0;
  return (int32_t)(((long long)c->n_max * c->eas_ppm + 999999) / 1000000);
}

bpc_status bpc_build_eas(bpc_ctx* ctx, void* stream) {
  if (ctx == nullptr) return BPC_ERR_INVALID_ARG;
  if (ctx->cfg.eas_ppm <= 0) return BPC_ERR_UNSUPPORTED;
  if (!ctx->fitted) return BPC_ERR_NOT_FITTED;
  cudaError_t e = bpc_launch_build_eas(ctx, (cudaStream_t)stream);
  return e == cudaSuccess ? BPC_OK : cuda_fail(ctx, e);
}

bpc_status bpc_exact_topk(bpc_ctx* ctx, const void* q, const void* k_cache, int32_t budget_ppm, int32_t budget_count,
                          float* scores, int32_t* sel_out, int32_t* count_out, void* stream) {
  if (ctx == nullptr || q == nullptr || k_cache == nullptr || scores == nullptr || sel_out == nullptr || count_out == nullptr)
    return BPC_ERR_INVALID_ARG;
  if (budget_count < 0 || (budget_count == 0 && (budget_ppm < 0 || budget_ppm > 1000000))) return BPC_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k_cache)) & 15u) return BPC_ERR_INVALID_ARG;
  cudaError_t e = bpc_launch_exact_topk(ctx, q, k_cache, budget_ppm, budget_count, scores, sel_out, count_out, (cudaStream_t)stream);
  return e == cudaSuccess ? BPC_OK : cuda_fail(ctx, e);
}

bpc_status bpc_get_eas(bpc_ctx* ctx, float* sq_err_out, int32_t* set_out, int32_t* count_out, void* stream) {
  if (ctx == nullptr) return BPC_ERR_INVALID_ARG;
  if (ctx->cfg.eas_ppm <= 0) return BPC_ERR_UNSUPPORTED;
  cudaError_t e = cudaSuccess;
  if (sq_err_out) e = cudaMemcpyAsync(sq_err_out, ctx->key_err, (size_t)ctx->units * ctx->cfg.n_max * 4, cudaMemcpyDeviceToDevice, (cudaStream_t)stream);
  if (e == cudaSuccess && set_out) e = cudaMemcpyAsync(set_out, ctx->eas_idx, (size_t)ctx->units * ctx->eas_cap * 4, cudaMemcpyDeviceToDevice, (cudaStream_t)stream);
  if (e == cudaSuccess && count_out) e = cudaMemcpyAsync(count_out, ctx->eas_cnt, (size_t)ctx->units * 4, cudaMemcpyDeviceToDevice, (cudaStream_t)stream);
  return e == cudaSuccess ? BPC_OK : cuda_fail(ctx, e);
}

bpc_status bpc_append(bpc_ctx* ctx, const void* k_new, const void* v_new, void* k_cache, void* v_cache, uint64_t* codes,
                      void* stream) {
  if (ctx == nullptr || k_new == nullptr || v_new == nullptr || k_cache == nullptr || v_cache == nullptr || codes == nullptr)
    return BPC_ERR_INVALID_ARG;
  if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(codes))
    return BPC_ERR_INVALID_ARG;
  if (!ctx->fitted) return BPC_ERR_NOT_FITTED;
  for (int i = 0; i < ctx->cfg.batch; ++i)
    if (ctx->host_lens[i] >= ctx->cfg.n_max) return BPC_ERR_CAPACITY;
  cudaError_t e = bpc_launch_append(ctx, k_new, v_new, k_cache, v_cache, codes, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  for (int i = 0; i < ctx->cfg.batch; ++i) ctx->host_lens[i] += 1;
  return BPC_OK;
}

static bpc_status decode_common(bpc_ctx* ctx, const void* k_new, const void* v_new, void* k_cache_w, void* v_cache_w,
                                uint64_t* codes_w, const void* q, const void* k_cache, const void* v_cache,
                                const uint64_t* codes, int32_t budget_ppm, int32_t budget_count, float* out,
                                int32_t* sel_idx, void* stream) {
  if (ctx == nullptr || q == nullptr || k_cache == nullptr || v_cache == nullptr || codes == nullptr || out == nullptr)
    return BPC_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(codes) || !aligned16(out))
    return BPC_ERR_INVALID_ARG;
  if (sel_idx != nullptr && !aligned16(sel_idx)) return BPC_ERR_INVALID_ARG;
  if (budget_ppm < 0 || budget_ppm > 1000000 || budget_count < 0) return BPC_ERR_INVALID_ARG;
  if (budget_ppm == 0 && budget_count == 0) return BPC_ERR_INVALID_ARG;
  if (!ctx->fitted) return BPC_ERR_NOT_FITTED;
  const bpc_config& c = ctx->cfg;
  const bool forced_stream_env = ctx->streaming && ctx->cluster_size > 0 && chunk_for(c.n_max, ctx->cluster_size) <= ctx->chunk_cap_limit;
  (void)forced_stream_env;
  const bool want_sched = ctx->sched_ok && ctx->decode_path == 2;   // measured slower than the cluster kernel: on request only
  if (want_sched) {
    bpcdev::SchedParams sp;
    memset(&sp, 0, sizeof(sp));
    sp.q = q; sp.k_cache = k_cache; sp.v_cache = v_cache; sp.codes = reinterpret_cast<const uint32_t*>(codes);
    sp.P_h = ctx->P_h; sp.gram = ctx->gram; sp.unit_lens = ctx->unit_lens; sp.unit_lens_w = ctx->unit_lens;
    sp.k_new = k_new; sp.v_new = v_new; sp.k_cache_w = k_cache_w; sp.v_cache_w = v_cache_w;
    sp.codes_w = reinterpret_cast<uint32_t*>(codes_w);
    sp.out = out; sp.sel = sel_idx;
    sp.scores = ctx->sc_scores; sp.hist_rows = ctx->sc_hist; sp.table = reinterpret_cast<int4*>(ctx->sc_table);
    sp.qplanes = ctx->sc_planes; sp.partials = ctx->sc_partials; sp.sync = ctx->sc_sync; sp.err = ctx->dev_err;
    sp.dbg_scores = ctx->dbg_scores; sp.dbg_qweights = ctx->dbg_qweights; sp.dbg_trace = ctx->dbg_trace;
    sp.units = ctx->units; sp.n_kv_heads = c.n_kv_heads; sp.group = ctx->group; sp.n_max = c.n_max;
    sp.row_stride = ctx->row_stride; sp.shared_sets = c.hash_sets != ctx->units;
    sp.budget_ppm = budget_ppm; sp.budget_count = budget_count; sp.residual_correction = c.residual_correction;
    sp.ch = ctx->sched_ch_user > 0 ? ctx->sched_ch_user : ctx->sched_ch;
    sp.r_max = (c.n_max + sp.ch - 1) / sp.ch;
    const int k_max = bpcdev::sched_budget(c.n_max, budget_ppm, budget_count);
    // rows per attention slice: a slice lies in one key range; twice the rows a range selects on average, so that
    // most ranges are one slice, within [128, kSchedListCap] and never fewer than k/64 (bounds the slices per unit)
    int rpa = ctx->sched_rpa_user;
    if (rpa <= 0) {
      rpa = (int)((2LL * k_max * sp.ch + c.n_max - 1) / c.n_max);
      if (rpa < 128) rpa = 128;
    }
    if (rpa < (k_max + 63) / 64) rpa = (k_max + 63) / 64;
    if (rpa > bpcdev::kSchedListCap) rpa = bpcdev::kSchedListCap;
    sp.rpa = rpa;
    sp.na_cap = ctx->sched_na_cap;
    const int group_items = 2 * sp.r_max + (k_max + rpa - 1) / rpa;   // a unit's SCAN items plus (at most) its ATTEND items
    if (sp.r_max + (k_max + rpa - 1) / rpa > sp.na_cap) return BPC_ERR_UNSUPPORTED;
    sp.delta = 0;
    sp.nbins = hist_bins(ctx);
    sp.qp_words = ctx->sched_qp_words;
    sp.sc_stride = ctx->sched_sc_stride;
    sp.sm_scale_d = ctx->sm_scale_d;
    long long items = (long long)ctx->units * (group_items + 2 + c.code_bits / 32);
    const int grid = (int)(items < ctx->sched_grid_max ? items : ctx->sched_grid_max);
    cudaError_t es = bpc_sched_launch(ctx->group, c.code_bits, sp, grid, ctx->sched_smem, ctx->use_pdl, (cudaStream_t)stream);
    if (es != cudaSuccess) return cuda_fail(ctx, es);
    ctx->launches += 1;
    return BPC_OK;
  }
  if (ctx->cluster_size == 0) return BPC_ERR_UNSUPPORTED;
  const int cap = ctx->chunk_cap_limit;
  cudaError_t e;
  DecodeParams p;
  memset(&p, 0, sizeof(p));
  p.q = q; p.k_cache = k_cache; p.v_cache = v_cache; p.codes = codes; p.P_h = ctx->P_h;
  p.unit_lens = ctx->unit_lens; p.out = out;
  p.k_new = k_new; p.v_new = v_new; p.k_cache_w = k_cache_w; p.v_cache_w = v_cache_w; p.codes_w = codes_w;
  p.unit_lens_w = ctx->unit_lens; p.gram = ctx->gram; p.residual_correction = c.residual_correction;
  p.eas_idx = ctx->eas_idx; p.eas_cnt = ctx->eas_cnt; p.eas_cap = ctx->eas_cap;
  p.sel = sel_idx != nullptr ? sel_idx : ctx->sel_scratch;
  p.dbg_scores = ctx->dbg_scores; p.dbg_qweights = ctx->dbg_qweights; p.dbg_times = ctx->dbg_times;
  p.err = ctx->dev_err;
  p.n_kv_heads = c.n_kv_heads; p.group = ctx->group; p.n_max = c.n_max; p.row_stride = ctx->row_stride;
  p.shared_sets = c.hash_sets != ctx->units;
  p.budget_ppm = budget_ppm; p.budget_count = budget_count; p.sm_scale_d = ctx->sm_scale_d;
  const int chunk = chunk_for(c.n_max, ctx->cluster_size);
  if (!ctx->streaming && chunk > cap) return BPC_ERR_UNSUPPORTED;
  p.chunk_cap = ctx->streaming ? 0 : chunk;               // shared memory is sized for the largest possible unit
  p.nbins = hist_bins(ctx);
  p.hist_shift = hist_shift(ctx);
  p.key_shift_min = ctx->key_shift_min;
  if (ctx->streaming)
    e = c.kv_dtype == BPC_BF16 ? bpc_launch_decode_bf16_stream(ctx, p, (cudaStream_t)stream)
                               : bpc_launch_decode_f32_stream(ctx, p, (cudaStream_t)stream);
  else if (ctx->byte_keys)
    e = c.kv_dtype == BPC_BF16 ? bpc_launch_decode_bf16_k8(ctx, p, (cudaStream_t)stream)
                               : bpc_launch_decode_f32_k8(ctx, p, (cudaStream_t)stream);
  else if (c.score_mode == BPC_SCORE_WEIGHTED7)
    e = c.kv_dtype == BPC_BF16 ? bpc_launch_decode_bf16_w7(ctx, p, (cudaStream_t)stream)
                               : bpc_launch_decode_f32_w7(ctx, p, (cudaStream_t)stream);
  else if (c.eas_ppm > 0)
    e = c.kv_dtype == BPC_BF16 ? bpc_launch_decode_bf16_eas(ctx, p, (cudaStream_t)stream)
                               : bpc_launch_decode_f32_eas(ctx, p, (cudaStream_t)stream);
  else
    e = c.kv_dtype == BPC_BF16 ? bpc_launch_decode_bf16(ctx, p, (cudaStream_t)stream)
                               : bpc_launch_decode_f32(ctx, p, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  ctx->launches += 1;
  return BPC_OK;
}

bpc_status bpc_decode_attn(bpc_ctx* ctx, const void* q, const void* k_cache, const void* v_cache, const uint64_t* codes,
                           int32_t budget_ppm, int32_t budget_count, float* out, int32_t* sel_idx, void* stream) {
  return decode_common(ctx, nullptr, nullptr, nullptr, nullptr, nullptr, q, k_cache, v_cache, codes, budget_ppm,
                       budget_count, out, sel_idx, stream);
}

bpc_status bpc_append_decode_attn(bpc_ctx* ctx, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                                  uint64_t* codes, const void* q, int32_t budget_ppm, int32_t budget_count, float* out,
                                  int32_t* sel_idx, void* stream) {
  if (ctx == nullptr || k_new == nullptr || v_new == nullptr || k_cache == nullptr || v_cache == nullptr || codes == nullptr)
    return BPC_ERR_INVALID_ARG;
  if (!aligned16(k_new) || !aligned16(v_new)) return BPC_ERR_INVALID_ARG;
  for (int i = 0; i < ctx->cfg.batch; ++i)
    if (ctx->host_lens[i] >= ctx->cfg.n_max) return BPC_ERR_CAPACITY;
  bpc_status s = decode_common(ctx, k_new, v_new, k_cache, v_cache, codes, q, k_cache, v_cache, codes, budget_ppm,
                               budget_count, out, sel_idx, stream);
  if (s != BPC_OK) return s;
  for (int i = 0; i < ctx->cfg.batch; ++i) ctx->host_lens[i] += 1;
  return BPC_OK;
}

bpc_status bpc_debug_set_buffers(bpc_ctx* ctx, int32_t* scores, int32_t* qweights) {
  if (ctx == nullptr) return BPC_ERR_INVALID_ARG;
  ctx->dbg_scores = scores;
  ctx->dbg_qweights = qweights;
  return BPC_OK;
}

bpc_status bpc_debug_set_phase_timer(bpc_ctx* ctx, uint64_t* stamps) {
  if (ctx == nullptr) return BPC_ERR_INVALID_ARG;
  ctx->dbg_times = reinterpret_cast<unsigned long long*>(stamps);
  return BPC_OK;
}

bpc_status bpc_debug_set_pdl(bpc_ctx* ctx, int32_t on) {
  if (ctx == nullptr) return BPC_ERR_INVALID_ARG;
  ctx->use_pdl = on != 0;
  return BPC_OK;
}

bpc_status bpc_debug_force_key_shift(bpc_ctx* ctx, int32_t shift) {
  if (ctx == nullptr || shift < 0 || shift > 2) return BPC_ERR_INVALID_ARG;
  if (ctx->cfg.score_mode != BPC_SCORE_WEIGHTED7) return BPC_ERR_UNSUPPORTED;
  ctx->key_shift_min = shift;
  return BPC_OK;
}

bpc_status bpc_debug_set_tensor_core_encode(bpc_ctx* ctx, int32_t on) {
  if (ctx == nullptr) return BPC_ERR_INVALID_ARG;
  ctx->no_tc_encode = on == 0;
  return BPC_OK;
}

bpc_status bpc_debug_force_streaming(bpc_ctx* ctx, int32_t on) {
  if (ctx == nullptr) return BPC_ERR_INVALID_ARG;
  if (on != 0 && (ctx->cfg.score_mode != BPC_SCORE_HAMMING || ctx->cfg.eas_ppm != 0)) return BPC_ERR_UNSUPPORTED;
  ctx->force_streaming = on != 0;
  ctx->decode_smem_set = 0;                                 // another kernel variant: its function attributes are set at its first launch
  cudaError_t e = bpc_plan_decode_geometry(ctx);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  return ctx->cluster_size > 0 ? BPC_OK : BPC_ERR_UNSUPPORTED;
}

bpc_status bpc_debug_force_byte_keys(bpc_ctx* ctx, int32_t mode) {
  if (ctx == nullptr || mode < -1 || mode > 1) return BPC_ERR_INVALID_ARG;
  ctx->force_byte_keys = mode;
  ctx->decode_smem_set = 0;                                 // possibly another kernel variant: attributes at its first launch
  cudaError_t e = bpc_plan_decode_geometry(ctx);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  if (ctx->cluster_size == 0) return BPC_ERR_UNSUPPORTED;
  return (mode > 0 && !ctx->byte_keys) ? BPC_ERR_UNSUPPORTED : BPC_OK;
}

int32_t bpc_uses_byte_keys(bpc_ctx* ctx) { return (ctx != nullptr && ctx->byte_keys) ? 1 : 0; }

bpc_status bpc_status_of_device_error(int32_t error_word) { return error_word == 0 ? BPC_OK : BPC_ERR_DEVICE; }

bpc_status bpc_debug_set_decode_path(bpc_ctx* ctx, int32_t path) {
  if (ctx == nullptr || path < 0 || path > 2) return BPC_ERR_INVALID_ARG;
  if (path == 2 && !ctx->sched_ok) {                        // first request: plan the geometry, allocate the scratch
    cudaError_t e = sched_setup(ctx);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
  }
  if (path == 2 && !ctx->sched_ok) return BPC_ERR_UNSUPPORTED;
  if (path == 1 && ctx->cluster_size == 0) return BPC_ERR_UNSUPPORTED;
  ctx->decode_path = path;
  return BPC_OK;
}

int32_t bpc_uses_work_items(bpc_ctx* ctx) { return (ctx != nullptr && ctx->sched_ok && ctx->decode_path == 2) ? 1 : 0; }

bpc_status bpc_debug_set_work_item_geometry(bpc_ctx* ctx, int32_t keys_per_scan_item, int32_t rows_per_attend_item) {
  if (ctx == nullptr || !ctx->sched_ok) return ctx == nullptr ? BPC_ERR_INVALID_ARG : BPC_ERR_UNSUPPORTED;
  if (keys_per_scan_item < 0 || rows_per_attend_item < 0) return BPC_ERR_INVALID_ARG;
  if (keys_per_scan_item > 0) {
    if (keys_per_scan_item % ctx->sched_gran != 0 || keys_per_scan_item > 32768) return BPC_ERR_INVALID_ARG;
    if ((ctx->cfg.n_max + keys_per_scan_item - 1) / keys_per_scan_item > ctx->sched_r_alloc) return BPC_ERR_INVALID_ARG;
  }
  if (rows_per_attend_item > bpcdev::kSchedListCap) return BPC_ERR_INVALID_ARG;
  ctx->sched_ch_user = keys_per_scan_item;
  ctx->sched_rpa_user = rows_per_attend_item;
  return BPC_OK;
}

bpc_status bpc_debug_set_work_item_trace(bpc_ctx* ctx, uint64_t* trace) {
  if (ctx == nullptr) return BPC_ERR_INVALID_ARG;
  ctx->dbg_trace = reinterpret_cast<unsigned long long*>(trace);
  return BPC_OK;
}

int32_t bpc_work_item_grid(bpc_ctx* ctx) { return (ctx && ctx->sched_ok) ? ctx->sched_grid_max : 0; }

bpc_status bpc_last_device_error(bpc_ctx* ctx, int32_t* host_out, void* stream) {
  if (ctx == nullptr || host_out == nullptr) return BPC_ERR_INVALID_ARG;
  cudaError_t e = cudaMemcpyAsync(host_out, ctx->dev_err, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  return bpc_status_of_device_error(*host_out);
}

int32_t bpc_last_cuda_error(bpc_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }
int64_t bpc_launch_count(bpc_ctx* ctx) { return ctx ? ctx->launches : 0; }

#pragma GCC visibility pop
}  // extern "C"
