// Tensor-core pass of Algorithm 1 (bf16 caches): one pass over the keys per bit.
//
// Per bit i the pass needs, for every key row, the decision value
//     t = R_row . d = K_row . d - sum_{j<i} u_j (v_j . d)
// (the residual is never stored: the earlier signs u_j are the code words written so far), the new sign u_i = sign(t),
// and over all rows the sums  sum_rows u_i K_row  (128 channels) and the agreement counts of u_i with every earlier
// bit, from which a small kernel forms the new projection row.  The CUDA-core pass spends about 60 warp instructions
// per row on that and is bound by instruction issue.  Here both contractions with the key rows run on the tensor
// cores, on tiles of 128 keys:
//   * K_tile (128 keys x 128 channels, bf16, the 128-byte-swizzled K-major layout)  x  d  (three bf16 terms of the fp32
//     direction as rows 0..2 of a 16-row operand)  ->  128 x 16 accumulator, one key per tensor-memory lane; the
//     thread that owns the key adds the three columns;
//   * K_tile read the other way round (MN-major descriptor: M = channel, K = key)  x  u  (the tile's 128 new signs as a
//     bf16 +-1 row of a 16-row operand, 0 for rows past the end)  ->  128 x 16 accumulator with one CHANNEL per lane,
//     accumulated over the tiles of a warpgroup; every kFlushTiles tiles the running sums move into fp64 registers, so
//     that the fp32 accumulation in tensor memory never spans more than 1024 rows (as the CUDA-core pass's block sums).
// What stays on the CUDA cores is per key, not per (key, channel): the table look-up of sum_j u_j (v_j . d) four bits
// at a time (the same table as the CUDA-core pass), the sign, one code-word store, and the agreement counters (bit-sliced,
// one key per thread and tile).  A block holds three warpgroups with their own double-buffered key tiles, accumulators
// and barriers; blocks take long contiguous row ranges (a few waves of blocks in total), so the per-block sums and
// counts are few and the counters are reduced once per block.
//
// Waits on MMA-completion barriers are bounded; on expiry the block raises the device error word, still releases its
// tensor memory and returns.
#include <stdlib.h>
#include "common.cuh"
#include "umma.cuh"

namespace {
using namespace umma;

constexpr int kTileKeys = 128;
constexpr int kGroupThreads = 128;
constexpr int kGroups = 3;
constexpr int kThreads = kGroupThreads * kGroups;
constexpr int kFlushTiles = 8;  // tiles whose channel sums accumulate in tensor memory before moving to fp64
constexpr int kPlanWaves = 1;        // waves of blocks the row ranges are planned from
constexpr int kPlanes = 8;           // bit-sliced agreement counters: up to 255 tiles per warpgroup and block
constexpr int kTileBytes = kTileKeys * 256;
constexpr int kSmallOp = 16 * 128 * 2;   // a [16 x 128] bf16 operand (direction terms / new signs)

__device__ __forceinline__ void group_sync(int g) { asm volatile("bar.sync %0, %1;" ::"r"(1 + g), "r"(kGroupThreads) : "memory"); }

// 16 consecutive accumulator columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                 "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
               : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// element (row n, k) of a [16 x 128] bf16 operand, K-major without swizzle (core matrices of 8 rows x 16 bytes)
__device__ __forceinline__ size_t small_off(int n, int k) { return (size_t)(k >> 3) * 256 + (size_t)(n >> 3) * 128 + (size_t)(n & 7) * 16 + (size_t)(k & 7) * 2; }

template <int WORDS>
__global__ void __launch_bounds__(kThreads, 1)
fit_pass_tc_kernel(const __nv_bfloat16* __restrict__ k_cache, uint32_t* __restrict__ hfit, const float* __restrict__ dir,
                   const float* __restrict__ dots, float* __restrict__ partials, int32_t* __restrict__ agree,
                   const int32_t* __restrict__ unit_lens, int32_t* __restrict__ err, int n_max, int row_stride, int it,
                   int blocks_per_unit, int rows_per_block) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // swizzled tiles: 1024-byte alignment
  constexpr int b = WORDS * 32, NIB = WORDS * 8;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int grp = tid / kGroupThreads, gtid = tid % kGroupThreads;
  unsigned char* a_g = smem + (size_t)grp * 2 * kTileBytes;            // this warpgroup's two key-tile buffers
  unsigned char* bd_s = smem + (size_t)kGroups * 2 * kTileBytes;       // direction: rows 0..2 = its three bf16 terms
  unsigned char* bu_s = bd_s + kSmallOp + (size_t)grp * kSmallOp;      // this warpgroup's new signs: row 0
  float* lut = reinterpret_cast<float*>(bd_s + (size_t)(1 + kGroups) * kSmallOp);   // [NIB][16]
  int* cnt_s = reinterpret_cast<int*>(lut + NIB * 16);                 // [b] agreement counts of the block
  double* red = reinterpret_cast<double*>(cnt_s + b);                  // [kGroups][128] channel sums of the warpgroups
  __shared__ unsigned long long bar1_s[kGroups], bar2_s[kGroups];
  __shared__ uint32_t tmem_base_s;
  __shared__ int timed_out_g[kGroups];

  const int unit = blockIdx.y;
  const int n = min(unit_lens[unit], n_max);
  const int row0_blk = blockIdx.x * rows_per_block;
  const int row_end = min(n, row0_blk + rows_per_block);
  float* part_out = partials + ((size_t)unit * blocks_per_unit + blockIdx.x) * BPC_D;
  int32_t* agree_out = agree + ((size_t)unit * blocks_per_unit + blockIdx.x) * b;
  if (row0_blk >= n) {                                               // no rows: (uniform over the block) nothing to set up
    if (tid < BPC_D) part_out[tid] = 0.f;
    for (int j = tid; j < b; j += kThreads) agree_out[j] = 0;
    return;
  }
  const int ntile = (row_end - row0_blk + kTileKeys - 1) / kTileKeys;

  // ---- one-time set-up
  if (tid == 0) {
    for (int g = 0; g < kGroups; ++g) { mbar_init(&bar1_s[g], 1); mbar_init(&bar2_s[g], 1); timed_out_g[g] = 0; }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(128) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  for (int i = tid; i < (1 + kGroups) * kSmallOp / 16; i += kThreads) reinterpret_cast<uint4*>(bd_s)[i] = make_uint4(0u, 0u, 0u, 0u);
  for (int j = tid; j < b; j += kThreads) cnt_s[j] = 0;
  // sum_j u_j (v_j . d) four bits at a time: lut[nibble][pattern] (inner products of bits >= it are zero)
  for (int e = tid; e < NIB * 16; e += kThreads) {
    const int m = e & 15, nb = e >> 4;
    float v = 0.f;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float d = dots[(size_t)unit * b + 4 * nb + q];
      v += ((m >> q) & 1) ? d : -d;
    }
    lut[e] = v;
  }
  __syncthreads();
  if (tid < BPC_D) {                                                 // the direction as three bf16 terms (24 mantissa bits)
    const float d = dir[(size_t)unit * BPC_D + tid];
    const __nv_bfloat16 t1 = __float2bfloat16_rn(d);
    const float r1 = d - __bfloat162float(t1);
    const __nv_bfloat16 t2 = __float2bfloat16_rn(r1);
    const __nv_bfloat16 t3 = __float2bfloat16_rn(r1 - __bfloat162float(t2));
    *reinterpret_cast<__nv_bfloat16*>(bd_s + small_off(0, tid)) = t1;
    *reinterpret_cast<__nv_bfloat16*>(bd_s + small_off(1, tid)) = t2;
    *reinterpret_cast<__nv_bfloat16*>(bd_s + small_off(2, tid)) = t3;
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_all = tmem_base_s;
  const uint32_t lane_off = (uint32_t)(32 * (warp & 3)) << 16;        // a warp reaches the lanes of its quarter
  const uint32_t tm_d1 = tmem_all + (uint32_t)(grp * 32);            // decision values: lane = key of the tile
  const uint32_t tm_d2 = tm_d1 + 16;                                 // channel sums: lane = channel
  unsigned long long* bar1 = &bar1_s[grp];
  unsigned long long* bar2 = &bar2_s[grp];

  const unsigned char* kbase = reinterpret_cast<const unsigned char*>(k_cache) + (size_t)unit * n_max * (size_t)row_stride * 2;
  auto load_tile = [&](int tile, int buf) {                          // rows past the end are zero-filled
    const int r0 = row0_blk + tile * kTileKeys;
    unsigned char* a = a_g + (size_t)buf * kTileBytes;
    for (int c = gtid; c < kTileKeys * 16; c += kGroupThreads) {
      const int r = c >> 4, ch = c & 15;
      unsigned char* d = a + sw128_offset(kTileKeys, r, ch);
      if (r0 + r < row_end) cp_async16(d, kbase + (size_t)(r0 + r) * row_stride * 2 + ch * 16);
      else *reinterpret_cast<uint4*>(d) = make_uint4(0u, 0u, 0u, 0u);
    }
    cp_async_commit();
  };
  const uint32_t idesc = umma_idesc_bf16(kTileKeys, 16);
  auto issue_dot = [&](const unsigned char* a) {                     // keys x channels times the direction terms
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      const size_t aoff = (size_t)(ks >> 2) * (kTileKeys * 128) + (size_t)(ks & 3) * 32;
      umma_bf16(tm_d1, umma_desc_sw128(a + aoff), umma_desc_nosw(bd_s + (size_t)ks * 512, 256, 128), idesc, ks > 0 ? 1u : 0u);
    }
    umma_commit(bar1);
  };
  auto issue_sum = [&](const unsigned char* a, bool accumulate) {    // channels x keys times the new signs
#pragma unroll
    for (int ks = 0; ks < 8; ++ks)
      umma_bf16(tm_d2, umma_desc_sw128_mn(a + (size_t)ks * 2048, 16384, 1024), umma_desc_nosw(bu_s + (size_t)ks * 512, 256, 128),
                idesc | kIdescAMnMajor, (accumulate || ks > 0) ? 1u : 0u);
    umma_commit(bar2);
  };

  // ---- tiles of this warpgroup: grp, grp + kGroups, ... of the block's row range.  All threads of a warpgroup take
  // the same branches, so its hardware barrier is always reached by all 128 of them.
  unsigned ph1 = 0, ph2 = 0;                                         // phases the next waits on the two barriers refer to
  bool pend2 = false;                                                // a channel-sum MMA has been committed and not waited for
  int since_flush = 0;
  double vacc = 0.0;                                                 // sum over rows of u_i * K[row][channel gtid]
  uint32_t pl[kPlanes][WORDS];                                       // bit-sliced counts: agreements of u_i with each earlier bit
#pragma unroll
  for (int k = 0; k < kPlanes; ++k)
#pragma unroll
    for (int w = 0; w < WORDS; ++w) pl[k][w] = 0u;
  // code words of a key: requested one turn ahead, so that the global load is not on the turn's critical path
  auto load_words = [&](uint32_t (&v)[WORDS], int r) {
#pragma unroll
    for (int w = 0; w < WORDS; ++w) v[w] = 0u;
    if (it > 0 && r < row_end) {
      const uint32_t* src = hfit + ((size_t)unit * n_max + r) * WORDS;
      if constexpr (WORDS == 8) {
        const uint4 q = *reinterpret_cast<const uint4*>(src), q2 = *reinterpret_cast<const uint4*>(src + 4);
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w; v[4] = q2.x; v[5] = q2.y; v[6] = q2.z; v[7] = q2.w;
      } else if constexpr (WORDS == 4) { const uint4 q = *reinterpret_cast<const uint4*>(src); v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w; }
      else if constexpr (WORDS == 2) { const uint2 q = *reinterpret_cast<const uint2*>(src); v[0] = q.x; v[1] = q.y; }
      else v[0] = src[0];
    }
  };
  uint32_t nxt[WORDS];
  load_words(nxt, row0_blk + grp * kTileKeys + gtid);
  if (grp < ntile) load_tile(grp, 0);
  int idx = 0;
  for (int tl = grp; tl < ntile; tl += kGroups, ++idx) {
    const int buf = idx & 1;
    const unsigned char* a = a_g + (size_t)buf * kTileBytes;
    const int row = row0_blk + tl * kTileKeys + gtid;
    const bool live = row < row_end;
    uint32_t* hrow = hfit + ((size_t)unit * n_max + (live ? row : row0_blk)) * WORDS;
    uint32_t mine[WORDS];                                            // the key's earlier bits (bits >= it are zero: the fit clears the code words first)
#pragma unroll
    for (int w = 0; w < WORDS; ++w) mine[w] = nxt[w];                // (requested one turn ago)
    load_words(nxt, row + kGroups * kTileKeys);
    cp_async_wait_all();
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    group_sync(grp);                                                 // the tile has landed for all 128 threads
    if (timed_out_g[grp]) break;                                     // (set before the barrier, so all 128 threads agree)
    if (gtid == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      issue_dot(a);
    }
    // The channel-sum MMA of the previous tile runs ahead of this tile's dot product in the tensor pipe; once it has
    // completed, its operands (the sign row and the other tile buffer) are free: the next tile's copy starts as early
    // as possible, because the buffer count, not the arithmetic, bounds this kernel.
    if (pend2) {
      if (!mbar_wait(bar2, ph2)) timed_out_g[grp] = 1;
      ph2 ^= 1u;
      pend2 = false;
    }
    if (tl + kGroups < ntile) load_tile(tl + kGroups, buf ^ 1);
    // sum_j u_j (v_j . d) from the table, four partial sums in a fixed order
    float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int nb = 0; nb < NIB; ++nb) s4[nb & 3] += lut[nb * 16 + ((mine[nb >> 3] >> (4 * (nb & 7))) & 15u)];
    const float tc = (s4[0] + s4[1]) + (s4[2] + s4[3]);
    if (!mbar_wait(bar1, ph1)) timed_out_g[grp] = 1;
    ph1 ^= 1u;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    float d1[16];
    tmem_ld16(tm_d1 + lane_off, d1);
    const float tk = (d1[0] + d1[1]) + d1[2];                        // K_row . d: the three terms of d
    const bool pos = (tk - tc) >= 0.f;
    *reinterpret_cast<uint16_t*>(bu_s + small_off(0, gtid)) = live ? (pos ? (uint16_t)0x3F80u : (uint16_t)0xBF80u) : (uint16_t)0u;
    if (live) {
      hrow[it >> 5] = mine[it >> 5] | ((pos ? 1u : 0u) << (it & 31));
#pragma unroll
      for (int w = 0; w < WORDS; ++w) {
        uint32_t carry = pos ? mine[w] : ~mine[w];                   // bit e: u_j agrees with u_i
#pragma unroll
        for (int k = 0; k < kPlanes; ++k) {
          const uint32_t nc = pl[k][w] & carry;
          pl[k][w] ^= carry;
          carry = nc;
        }
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the sign row -> visible to the tensor core
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");  // (and this tile's accumulator reads are done)
    group_sync(grp);
    if (gtid == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      issue_sum(a, since_flush > 0);
    }
    pend2 = true;
    ++since_flush;
    if (since_flush == kFlushTiles || tl + kGroups >= ntile) {       // move the running channel sums to fp64
      if (!mbar_wait(bar2, ph2)) timed_out_g[grp] = 1;
      ph2 ^= 1u;
      pend2 = false;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      float d2[16];
      tmem_ld16(tm_d2 + lane_off, d2);
      vacc += (double)d2[0];
      since_flush = 0;
    }
  }
  if (timed_out_g[grp] && gtid == 0) atomicOr(err, BPC_DEVERR_TIMEOUT);
  cp_async_wait_all();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  red[grp * BPC_D + gtid] = vacc;
  // agreement counts: bit-sliced addition across the 32 lanes of a warp (the planes grow by one per step), then lane l
  // adds the totals of bits l, 32 + l, ... to the block's counters
  {
    constexpr int PT = kPlanes + 5;
#pragma unroll
    for (int w = 0; w < WORDS; ++w) {                                // one code word at a time (registers)
      uint32_t s[PT];
#pragma unroll
      for (int k = 0; k < PT; ++k) s[k] = k < kPlanes ? pl[k][w] : 0u;
#pragma unroll
      for (int st = 0; st < 5; ++st) {
        uint32_t carry = 0u;
#pragma unroll
        for (int k = 0; k < kPlanes + st + 1; ++k) {
          const uint32_t o = __shfl_xor_sync(0xffffffffu, s[k], 1 << st);
          const uint32_t x = s[k];
          s[k] = x ^ o ^ carry;
          carry = (x & o) | (carry & (x ^ o));
        }
      }
      int c = 0;
#pragma unroll
      for (int k = 0; k < PT; ++k) c += (int)((s[k] >> lane) & 1u) << k;
      if (c) atomicAdd(&cnt_s[32 * w + lane], c);
    }
  }
  __syncthreads();                                                   // all warpgroups are done with tensor memory
  if (tid < BPC_D) part_out[tid] = (float)((red[tid] + red[BPC_D + tid]) + red[2 * BPC_D + tid]);
  for (int j = tid; j < b; j += kThreads) agree_out[j] = cnt_s[j];
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_all), "r"(128) : "memory");
  }
}

// Row range of a block: from about two blocks per SM over all units, the first count whose last wave of one-block-per-SM
// is at least 90 % full (32 units on 148 SMs: 23 blocks per unit = 4.97 waves; fewer, longer blocks were measured slower,
// above all on ragged batches where a block is the unit of balance), never
// more tiles per warpgroup than the agreement counters hold and never fewer rows than the CUDA-core pass's blocks
// (the workspace is sized for those).
void plan(const bpc_ctx* ctx, int* bpu_out, int* rows_out) {
  const int n_max = ctx->cfg.n_max;
  int bpu = (kPlanWaves * ctx->sm_count + ctx->units - 1) / ctx->units;
  if (bpu < 1) bpu = 1;
  for (int tries = 0; tries < 16; ++tries) {
    const int rem = (int)(((long long)ctx->units * bpu) % ctx->sm_count);
    if (rem == 0 || rem * 10 >= ctx->sm_count * 9) break;
    ++bpu;
  }
  int rows = ((n_max + bpu - 1) / bpu + kTileKeys - 1) / kTileKeys * kTileKeys;
  const int rows_cap = 255 * kGroups * kTileKeys;
  if (rows > rows_cap) rows = rows_cap;
  if (rows < 1024) rows = 1024;
  *rows_out = rows;
  *bpu_out = (n_max + rows - 1) / rows;
}

}  // namespace

bool bpc_fit_tc_covers(const bpc_ctx* ctx) {
  return ctx->cfg.kv_dtype == BPC_BF16 && !ctx->no_tc_encode;
}

void bpc_fit_tc_geometry(const bpc_ctx* ctx, int* blocks_per_unit, int* rows_per_block) { plan(ctx, blocks_per_unit, rows_per_block); }

cudaError_t bpc_launch_fit_pass_tc(bpc_ctx* ctx, const void* k_cache, uint32_t* hfit, const float* dir, const float* dots,
                                   float* partials, int32_t* agree, int it, cudaStream_t stream) {
  int bpu = 0, rows = 0;
  plan(ctx, &bpu, &rows);
  const bpc_config& c = ctx->cfg;
  const int b = c.code_bits;
  const size_t smem = (size_t)kGroups * 2 * kTileBytes + (size_t)(1 + kGroups) * kSmallOp + (size_t)(b / 4) * 16 * 4 + (size_t)b * 4 +
                      (size_t)kGroups * BPC_D * 8 + 1024;
  const dim3 grid(bpu, ctx->units);
#define BPC_FIT_TC(W)                                                                                                      \
  do {                                                                                                                    \
    cudaError_t e = cudaFuncSetAttribute(fit_pass_tc_kernel<W>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
    if (e != cudaSuccess) return e;                                                                                      \
    fit_pass_tc_kernel<W><<<grid, kThreads, smem, stream>>>((const __nv_bfloat16*)k_cache, hfit, dir, dots, partials, agree, \
                                                            ctx->unit_lens, ctx->dev_err, c.n_max, ctx->row_stride, it, bpu, rows); \
  } while (0)
  if (b == 32) BPC_FIT_TC(1); else if (b == 64) BPC_FIT_TC(2); else if (b == 128) BPC_FIT_TC(4); else if (b == 256) BPC_FIT_TC(8); else return cudaErrorNotSupported;
#undef BPC_FIT_TC
  return cudaGetLastError();
}
