// Quality yard-sticks: the exact-score top-k selector (appendix "Baseline Methods", TOPK (Oracle)).  Evaluation aids,
// not part of the decode path: exact scores of every cached key for every query head, then a per-head top-k by a
// radix select.  (Dense attention, the other yard-stick, is the decode call with a budget of all keys.)
#include "common.cuh"

namespace {

constexpr int kScoreThreads = 256;
constexpr int kScoreRows = 2048;          // key rows per block

// scores[(seq * n_q_heads + head) * n_max + r] = q_head . k_r   (fp32: exact bf16 products, fp32 sums)
template <typename KV>
__global__ void __launch_bounds__(kScoreThreads)
exact_scores_kernel(const KV* __restrict__ q, const KV* __restrict__ k_cache, float* __restrict__ scores,
                    const int32_t* __restrict__ unit_lens, int n_kv_heads, int group, int n_max, int row_stride) {
  const int unit = blockIdx.y, seq = unit / n_kv_heads, kvh = unit % n_kv_heads;
  const int n = min(unit_lens[unit], n_max);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_q_heads = n_kv_heads * group;
  float qv[BPC_MAX_GROUP][4];
#pragma unroll
  for (int g = 0; g < BPC_MAX_GROUP; ++g) {
#pragma unroll
    for (int c = 0; c < 4; ++c)
      qv[g][c] = g < group ? to_float(q[((size_t)seq * n_q_heads + kvh * group + g) * BPC_D + 4 * lane + c]) : 0.f;
  }
  const int row0 = blockIdx.x * kScoreRows, row_end = min(n, row0 + kScoreRows);
  for (int r = row0 + warp; r < row_end; r += kScoreThreads / 32) {
    const KV* kr = k_cache + ((size_t)unit * n_max + r) * row_stride + 4 * lane;
    const float x0 = to_float(kr[0]), x1 = to_float(kr[1]), x2 = to_float(kr[2]), x3 = to_float(kr[3]);
#pragma unroll
    for (int g = 0; g < BPC_MAX_GROUP; ++g) {
      if (g < group) {
        float t = x0 * qv[g][0];
        t = fmaf(x1, qv[g][1], t); t = fmaf(x2, qv[g][2], t); t = fmaf(x3, qv[g][3], t);
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (lane == 0) scores[((size_t)seq * n_q_heads + kvh * group + g) * n_max + r] = t;
      }
    }
  }
}

// order-preserving map of a float's bits to an unsigned integer
__device__ __forceinline__ uint32_t ordered_bits(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kSelThreads = 1024;

// One block per (sequence, query head): the k largest scores, ties to the lowest index, ascending index order.
// A 4-pass radix select (8 bits per pass) over the ordered bit patterns finds the k-th largest, one ordered pass compacts.
__global__ void __launch_bounds__(kSelThreads)
exact_topk_kernel(const float* __restrict__ scores, const int32_t* __restrict__ unit_lens, int32_t* __restrict__ sel,
                  int32_t* __restrict__ sel_cnt, int n_kv_heads, int group, int n_max, int budget_ppm, int budget_count) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t wsum[kSelThreads / 32];
  __shared__ uint32_t s_prefix, s_need, s_run_gt, s_run_eq;
  const int head = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_q_heads = n_kv_heads * group;
  const int seq = head / n_q_heads, kvh = (head % n_q_heads) / group;
  const int n = min(unit_lens[seq * n_kv_heads + kvh], n_max);
  long long kk = budget_count > 0 ? (long long)budget_count : ((long long)n * budget_ppm + 999999LL) / 1000000LL;
  const int k = (int)(kk < 0 ? 0 : (kk < n ? kk : n));
  const float* e = scores + (size_t)head * n_max;
  int32_t* out = sel + (size_t)head * n_max;
  if (tid == 0) sel_cnt[head] = k;
  if (k <= 0) return;
  if (tid == 0) { s_prefix = 0u; s_need = (uint32_t)k; }
  __syncthreads();
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0u;
    __syncthreads();
    const uint32_t prefix = s_prefix, himask = shift == 24 ? 0u : ~((1u << (shift + 8)) - 1u);
    for (int i = tid; i < n; i += kSelThreads) {
      const uint32_t v = ordered_bits(e[i]);
      if ((v & himask) == prefix) atomicAdd(&hist[(v >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      uint32_t need = s_need, acc = 0;
      int d = 255;
      for (; d > 0; --d) { if (acc + hist[d] >= need) break; acc += hist[d]; }
      s_need = need - acc;
      s_prefix = prefix | ((uint32_t)d << shift);
    }
    __syncthreads();
  }
  const uint32_t thr = s_prefix, need_eq = s_need;           // every v > thr and the first need_eq with v == thr
  if (tid == 0) { s_run_gt = 0u; s_run_eq = 0u; }
  __syncthreads();
  for (int i0 = 0; i0 < n; i0 += kSelThreads) {
    const int i = i0 + tid;
    const uint32_t v = i < n ? ordered_bits(e[i]) : 0u;
    const bool gt = i < n && v > thr, eq = i < n && v == thr;
    const uint32_t bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
    if (lane == 0) wsum[warp] = (uint32_t)__popc(bg) | ((uint32_t)__popc(be) << 16);
    __syncthreads();
    uint32_t before = 0, total = 0;
    for (int w = 0; w < kSelThreads / 32; ++w) { if (w < warp) before += wsum[w]; total += wsum[w]; }
    const uint32_t lt = (1u << lane) - 1u;
    const uint32_t gt_before = s_run_gt + (before & 0xffffu) + (uint32_t)__popc(bg & lt);
    const uint32_t eq_before = s_run_eq + (before >> 16) + (uint32_t)__popc(be & lt);
    if (gt || (eq && eq_before < need_eq)) out[gt_before + min(eq_before, need_eq)] = i;
    __syncthreads();
    if (tid == 0) { s_run_gt += total & 0xffffu; s_run_eq += total >> 16; }
    __syncthreads();
  }
}

}  // namespace

cudaError_t bpc_launch_exact_topk(bpc_ctx* ctx, const void* q, const void* k_cache, int budget_ppm, int budget_count,
                                  float* scores, int32_t* sel, int32_t* sel_cnt, cudaStream_t stream) {
  const bpc_config& c = ctx->cfg;
  const dim3 grid((c.n_max + kScoreRows - 1) / kScoreRows, ctx->units);
  if (c.kv_dtype == BPC_BF16)
    exact_scores_kernel<__nv_bfloat16><<<grid, kScoreThreads, 0, stream>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k_cache, scores,
                                                                            ctx->unit_lens, c.n_kv_heads, ctx->group, c.n_max, ctx->row_stride);
  else
    exact_scores_kernel<float><<<grid, kScoreThreads, 0, stream>>>((const float*)q, (const float*)k_cache, scores, ctx->unit_lens,
                                                                   c.n_kv_heads, ctx->group, c.n_max, ctx->row_stride);
  exact_topk_kernel<<<c.batch * c.n_q_heads, kSelThreads, 0, stream>>>(scores, ctx->unit_lens, sel, sel_cnt, c.n_kv_heads, ctx->group,
                                                                       c.n_max, budget_ppm, budget_count);
  ctx->launches += 2;
  return cudaGetLastError();
}
