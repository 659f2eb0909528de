// C-ABI entry points: argument validation, context life cycle, stream plumbing.
#include <new>
#include <stdlib.h>
#include <string.h>
#include "common.cuh"

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
  // weighted scores are kept as 16-bit keys: the largest possible score 127 * G * b must fit
  if (c->score_mode == BPC_SCORE_WEIGHTED7 && 127LL * (c->n_q_heads / c->n_kv_heads) * c->code_bits > 65535) return BPC_ERR_UNSUPPORTED;
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
int hist_shift(const bpc_ctx* ctx) {
  int s = 0;
  while ((max_score_key(ctx) >> s) >= 2048) ++s;
  return s;
}
int hist_bins(const bpc_ctx* ctx) { return (max_score_key(ctx) >> hist_shift(ctx)) + 1; }

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
  const char* force = getenv("BPC_FORCE_STREAMING");        // diagnostic switch: two-pass selection at any size
  const bool forced = force != nullptr && force[0] == '1';
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
  {
    const char* no_pdl = getenv("BPC_NO_PDL");          // diagnostic switch: plain stream-ordered launches
    ctx->use_pdl = !(no_pdl != nullptr && no_pdl[0] == '1');
  }
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
  ctx->host_lens = new (std::nothrow) int32_t[cfg->batch];
  if (ctx->host_lens) memset(ctx->host_lens, 0, sizeof(int32_t) * cfg->batch);
  if (e != cudaSuccess || ctx->host_lens == nullptr) {
    bpc_destroy(ctx);
    (void)cudaGetLastError();
    return BPC_ERR_CUDA;
  }
  e = bpc_plan_decode_geometry(ctx);
  if (e != cudaSuccess) { bpc_destroy(ctx); (void)cudaGetLastError(); return BPC_ERR_CUDA; }
  if (ctx->cluster_size == 0) { bpc_destroy(ctx); return BPC_ERR_UNSUPPORTED; }
  if (hist_bins(ctx) > 2048 || hist_shift(ctx) > 5) { bpc_destroy(ctx); return BPC_ERR_UNSUPPORTED; }
  *out = ctx;
  return BPC_OK;
}

bpc_status bpc_destroy(bpc_ctx* ctx) {
  if (ctx == nullptr) return BPC_ERR_INVALID_ARG;
  cudaFree(ctx->P); cudaFree(ctx->P_h); cudaFree(ctx->P_hf); cudaFree(ctx->gram);
  cudaFree(ctx->unit_lens); cudaFree(ctx->sel_scratch); cudaFree(ctx->dev_err);
  cudaFree(ctx->key_err); cudaFree(ctx->eas_idx); cudaFree(ctx->eas_cnt);
  delete[] ctx->host_lens;
  delete ctx;
  (void)cudaGetLastError();
  return BPC_OK;
}

bpc_status bpc_set_cluster_size(bpc_ctx* ctx, int32_t cs) {
  if (ctx == nullptr) return BPC_ERR_INVALID_ARG;
  const int cap = ctx->chunk_cap_limit, mc = ctx->max_cluster;
  if (cs == 0 && ctx->streaming) return BPC_OK;            // keeps the size chosen at creation
  if (cs == 0) cs = choose_cluster(ctx, cap, mc);
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
  // expand to per-unit lengths through a small pageable staging array: the copy is synchronous with
  // respect to the host buffer, so the temporary can be released on return
  int32_t* tmp = new (std::nothrow) int32_t[ctx->units];
  if (tmp == nullptr) return BPC_ERR_INVALID_ARG;
  for (int i = 0; i < c.batch; ++i) {
    ctx->host_lens[i] = host_lens[i];
    for (int h = 0; h < c.n_kv_heads; ++h) tmp[i * c.n_kv_heads + h] = host_lens[i];
  }
  cudaError_t e = cudaMemcpyAsync(ctx->unit_lens, tmp, (size_t)ctx->units * 4, cudaMemcpyHostToDevice, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
  delete[] tmp;
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
  if (ctx->streaming)
    e = c.kv_dtype == BPC_BF16 ? bpc_launch_decode_bf16_stream(ctx, p, (cudaStream_t)stream)
                               : bpc_launch_decode_f32_stream(ctx, p, (cudaStream_t)stream);
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

bpc_status bpc_last_device_error(bpc_ctx* ctx, int32_t* host_out, void* stream) {
  if (ctx == nullptr || host_out == nullptr) return BPC_ERR_INVALID_ARG;
  cudaError_t e = cudaMemcpyAsync(host_out, ctx->dev_err, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
  return e == cudaSuccess ? BPC_OK : cuda_fail(ctx, e);
}

int32_t bpc_last_cuda_error(bpc_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }
int64_t bpc_launch_count(bpc_ctx* ctx) { return ctx ? ctx->launches : 0; }

#pragma GCC visibility pop
}  // extern "C"
