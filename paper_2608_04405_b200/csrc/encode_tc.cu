// Tensor-core encode: Algorithm 2 for all cached keys of bf16 caches.
//
// The decision values before any correction are a dense contraction T = K P_h^T (keys x channels times
// channels x bits).  It runs on the 5th-generation tensor cores: per warpgroup, tiles of 128 keys (M = 128) against
// the unit's b projection rows (N = b: 32, 64 or 128) over the 128 channels (eight tcgen05.mma steps of K = 16), bf16
// operands in shared memory in the 128-byte-swizzled K-major layout, fp32 accumulator in tensor memory with one
// key per TMEM lane.  Algorithm 2's greedy sweep in its Gram form,
//     u_i = sign(t_i);  t_j -= u_i * G_ij  (j > i),   G = P_h P_h^T,
// (equal to updating the residual r <- r - u_i P_i and testing r . P_{i+1}) is blocked by 32 bits.  Inside a block the
// 32 sign decisions are sequential: each thread pulls its key's 32 decision values out of tensor memory (tcgen05.ld)
// and sweeps them in registers (496 FMAs).  The corrections of all LATER blocks by those 32 signs are again a dense
// contraction, T[:, later] -= U (128 keys x 32 signs) G[block, later], and go to the tensor cores too: the signs are
// written to shared memory as a bf16 operand (+-1 is exact), the Gram rows are kept as three bf16 terms whose sum
// carries 24 mantissa bits (so the products are exact and the fp32 accumulation in tensor memory sees what an fp32
// FMA chain would see up to rounding), and six small MMAs (three terms x two K = 16 steps) accumulate straight into
// the accumulator columns that still wait for their decisions.  That leaves 1 984 of the 8 128 sign-dependent FMAs per
// key (128 bits) on the CUDA cores.  The small operands use the K-major layout without swizzle (8-row x 16-byte core
// matrices; leading-dimension offset = distance between core matrices along K, stride offset = 128 bytes along M/N).
// A block holds three warpgroups, which share the projection rows and the Gram operands in shared memory and otherwise
// run independent pipelines (own key tile, own accumulator columns, own mbarrier, own hardware barrier), so one
// warpgroup's sweep covers the others' MMA round trips; the next key tile of a warpgroup is copied in while it sweeps.
//
// Waits on the MMA-completion mbarrier are bounded: on expiry the block raises the device error word, still
// releases its tensor memory and returns.
#include <stdlib.h>
#include "common.cuh"
#include "umma.cuh"

namespace {
using namespace umma;

constexpr int kTileKeys = 128;
constexpr int kGroupThreads = 128;   // one warpgroup sweeps one key tile (a TMEM lane per thread)
constexpr int kGroups = 3;           // warpgroups per block, each with its own tile, accumulator columns and barrier
constexpr int kPair = 1;             // key tiles a warpgroup sweeps together (one key of each per thread)
// 256-bit codes run as two launches over 128 bits each.  HALF = 0: the code is NBITS long.  HALF = 1: bits 0..127 of a
// 256-bit code (projection rows 0..127, Gram block G[0:128, 0:128], code words 0..3 of 8).  HALF = 2: bits 128..255; their
// decision values start from P_h[128 + j] . k - sum_{i < 128} u_i G[i][128 + j], and that sum over the first half's signs
// (read back from the code words the first launch wrote) is one more contraction on the tensor cores, U1 (128 keys x
// 128 signs) times -G[0:128, 128:256] as three bf16 terms (96 KB of shared memory: one warpgroup per block then).
constexpr int kCrossBytes = 3 * 128 * 128 * 2;

// barrier among the 128 threads of one warpgroup (hardware barriers 1 .. kGroups; 0 is __syncthreads)
__device__ __forceinline__ void group_sync(int g) { asm volatile("bar.sync %0, %1;" ::"r"(1 + g), "r"(kGroupThreads) : "memory"); }

// 32 consecutive accumulator columns of this thread's TMEM lane, into t[OFF .. OFF+31]
template <int OFF, int N>
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[N]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr + OFF));
#pragma unroll
  for (int i = 0; i < 32; ++i) v[OFF + i] = __uint_as_float(r[i]);
}

// Greedy sweep of one 32-bit column block held in registers (every index a compile-time constant), for the kPair
// keys of a thread at once.  On entry t[q][j] already carries the corrections of all earlier blocks; on exit word[q]
// holds the 32 signs of key q.  Each key sees exactly the operations of a sweep on its own.
template <int I>
struct DiagSweep {
  static __device__ __forceinline__ void run(float (&t)[kPair][32], uint32_t (&word)[kPair], float (&abs_sum)[kPair],
                                             const float* g_diag, int ld, int rc) {
    float u[kPair];
#pragma unroll
    for (int q = 0; q < kPair; ++q) {
      const bool pos = t[q][I] >= 0.f;
      word[q] |= (pos ? 1u : 0u) << I;
      abs_sum[q] += fabsf(t[q][I]);
      u[q] = pos ? 1.f : -1.f;
    }
    if (rc) {
      // row I of the diagonal block, columns after I: 16-byte broadcast reads (the reads, not the FMAs, bound the sweep)
      const float4* gi4 = reinterpret_cast<const float4*>(g_diag + I * ld);
#pragma unroll
      for (int j4 = (I + 1) / 4; j4 < 8; ++j4) {
        const float4 gv = gi4[j4];
        const float ge[4] = {gv.x, gv.y, gv.z, gv.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (4 * j4 + e > I) {
#pragma unroll
            for (int q = 0; q < kPair; ++q) t[q][4 * j4 + e] = fmaf(-u[q], ge[e], t[q][4 * j4 + e]);
          }
        }
      }
    }
    DiagSweep<I + 1>::run(t, word, abs_sum, g_diag, ld, rc);
  }
};
template <>
struct DiagSweep<32> {
  static __device__ __forceinline__ void run(float (&)[kPair][32], uint32_t (&)[kPair], float (&)[kPair], const float*, int, int) {}
};

template <int NBITS, int GROUPS, int HALF>
__global__ void __launch_bounds__(kGroupThreads * GROUPS, 1)
encode_tc_kernel(const __nv_bfloat16* __restrict__ k_cache, const __nv_bfloat16* __restrict__ Ph, const float* __restrict__ gram,
                 const int32_t* __restrict__ unit_lens, uint64_t* __restrict__ codes, int32_t* __restrict__ err,
                 int n_kv_heads, int n_max, int row_stride, int shared_sets, int residual_correction, int blocks_per_unit,
                 float* __restrict__ key_err) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // the swizzled operand tiles need 1024-byte alignment in the shared address space
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  constexpr int kGroups = GROUPS;                          // (shadows the default of the single-launch code lengths)
  constexpr int kThreads = kGroupThreads * GROUPS;
  static_assert(HALF == 0 || NBITS == 128, "the two-launch form is for 256-bit codes");
  constexpr int TOTAL = HALF == 0 ? NBITS : 256;           // bits of a whole code
  constexpr int ROW0 = HALF == 2 ? 128 : 0;                // first projection row (= first bit) of this launch
  constexpr int NB = NBITS / 32;                           // 32-bit column blocks of this launch
  constexpr int NWK = TOTAL / 32;                          // code words per key
  constexpr int A_BYTES = kTileKeys * 256;                 // one key tile (128 rows x 128 bf16)
  constexpr int B_BYTES = NBITS * 256;                     // the projection rows
  constexpr int GD_BYTES = NB * 32 * 32 * 4;               // diagonal 32 x 32 blocks of the Gram matrix, fp32
  constexpr int U_BYTES = kTileKeys * 64;                  // the 32 signs of one block for 128 keys, bf16 operand [128 x 32]
  // one bf16 term of -G[rows of block pb][columns after block pb] is an operand [NBITS - 32 (pb + 1) x 32]; the three
  // terms of block pb start at gb_off(pb)
  constexpr unsigned U_LBO = (kTileKeys / 8) * 128;        // bytes between core matrices along K
  const int tid = threadIdx.x, warp = tid >> 5;
  const int grp = tid / kGroupThreads, gtid = tid % kGroupThreads;   // warpgroup and thread within it
  unsigned char* a_t = smem + (size_t)grp * A_BYTES;       // this warpgroup's key tile (one buffer: see the loop)
  unsigned char* b_s = smem + kGroups * A_BYTES;
  float* gd_s = reinterpret_cast<float*>(b_s + B_BYTES);   // [NB][32][32]
  unsigned char* u_s = reinterpret_cast<unsigned char*>(gd_s) + GD_BYTES + (size_t)grp * U_BYTES;
  unsigned char* gb_s = reinterpret_cast<unsigned char*>(gd_s) + GD_BYTES + kGroups * U_BYTES;
  constexpr size_t GB_BYTES = (size_t)3 * 64 * ((NB - 1) * NBITS - 16 * (NB - 1) * NB);
  unsigned char* x_s = gb_s + GB_BYTES;                    // HALF == 2: the three bf16 terms of -G[0:128, 128:256], operands [128 x 128]
  auto gb_cols = [](int pb) { return NBITS - 32 * (pb + 1); };                     // columns after block pb
  auto gb_off = [](int pb) { return (size_t)3 * 64 * (size_t)(pb * NBITS - 16 * pb * (pb + 1)); };   // 3 * 64 * sum_{p<pb} cols(p)
  __shared__ unsigned long long mma_bar_s[kGroups];
  __shared__ uint32_t tmem_base_s;
  __shared__ int timed_out_g[kGroups];
  unsigned long long* mma_bar = &mma_bar_s[grp];
  constexpr int kAccCols = kGroups * NBITS;                // fp32 accumulator columns of the tiles in flight
  constexpr int kTmemCols = kAccCols <= 32 ? 32 : kAccCols <= 64 ? 64 : kAccCols <= 128 ? 128 : kAccCols <= 256 ? 256 : 512;   // a power of two >= 32
  static_assert(kAccCols <= 512, "accumulators exceed tensor memory");

  const int unit = blockIdx.y;
  const int n = min(unit_lens[unit], n_max);
  const int ntiles = (n + kTileKeys - 1) / kTileKeys;
  const int set = shared_sets ? unit % n_kv_heads : unit;

  // ---- one-time set-up: barrier, tensor memory, projection and Gram operands in shared memory
  if (tid == 0) {
    for (int g = 0; g < kGroups; ++g) { mbar_init(&mma_bar_s[g], 1); timed_out_g[g] = 0; }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  {
    const unsigned char* psrc = reinterpret_cast<const unsigned char*>(Ph + ((size_t)set * TOTAL + ROW0) * BPC_D);
    for (int c = tid; c < NBITS * 16; c += kThreads) {
      const int r = c >> 4, ch = c & 15;
      *reinterpret_cast<uint4*>(b_s + sw128_offset(NBITS, r, ch)) = *reinterpret_cast<const uint4*>(psrc + (size_t)r * 256 + ch * 16);
    }
    const float* gfull = gram + (size_t)set * TOTAL * TOTAL;
    const float* gsrc = gfull + (size_t)ROW0 * TOTAL + ROW0;  // this launch's diagonal block of the Gram matrix, row stride TOTAL
    for (int c = tid; c < NB * 32 * 32; c += kThreads) {     // diagonal blocks, kept in fp32 for the in-register sweep
      const int d = c >> 10, i = (c >> 5) & 31, j = c & 31;
      gd_s[c] = gsrc[(size_t)(32 * d + i) * TOTAL + 32 * d + j];
    }
    if constexpr (HALF == 2) {
      // -G[i][128 + j] for the first half's bits i, as three bf16 terms; operand rows j, K index i, [128 x 128] each
      for (int c = tid; c < 128 * 128; c += kThreads) {
        const int i = c >> 7, j = c & 127;
        const float g = -gfull[(size_t)i * TOTAL + 128 + j];
        const __nv_bfloat16 t1 = __float2bfloat16_rn(g);
        const float r1 = g - __bfloat162float(t1);
        const __nv_bfloat16 t2 = __float2bfloat16_rn(r1);
        const __nv_bfloat16 t3 = __float2bfloat16_rn(r1 - __bfloat162float(t2));
        unsigned char* base = x_s + nosw_offset(128, j, i);
        *reinterpret_cast<__nv_bfloat16*>(base) = t1;
        *reinterpret_cast<__nv_bfloat16*>(base + 32768) = t2;
        *reinterpret_cast<__nv_bfloat16*>(base + 65536) = t3;
      }
    }
    // -G[32 pb + i][j], j after block pb, as three bf16 terms (g = t1 + t2 + t3 up to 2^-24 |g|); operand rows j, K index i
    for (int c = tid; c < (NB - 1) * 32 * NBITS; c += kThreads) {
      const int pb = c / (32 * NBITS), i = (c / NBITS) & 31, j = c % NBITS;
      const int j0 = 32 * (pb + 1);
      if (j < j0) continue;
      const float g = -gsrc[(size_t)(32 * pb + i) * TOTAL + j];
      const __nv_bfloat16 t1 = __float2bfloat16_rn(g);
      const float r1 = g - __bfloat162float(t1);
      const __nv_bfloat16 t2 = __float2bfloat16_rn(r1);
      const __nv_bfloat16 t3 = __float2bfloat16_rn(r1 - __bfloat162float(t2));
      const size_t part = (size_t)gb_cols(pb) * 64;
      unsigned char* base = gb_s + gb_off(pb) + nosw_offset(gb_cols(pb), j - j0, i);
      *reinterpret_cast<__nv_bfloat16*>(base) = t1;
      *reinterpret_cast<__nv_bfloat16*>(base + part) = t2;
      *reinterpret_cast<__nv_bfloat16*>(base + 2 * part) = t3;
    }
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the tensor core
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_all = tmem_base_s;
  const uint32_t tmem_base = tmem_all + (uint32_t)(grp * NBITS);   // this warpgroup's accumulator columns
  float trace_g = 0.f;                                       // trace of the whole Gram matrix (added by the launch that finishes the code)
  if (key_err != nullptr && HALF != 1) {
    if constexpr (HALF == 2)
      for (int i = 0; i < 128; ++i) trace_g += gram[(size_t)set * TOTAL * TOTAL + (size_t)i * TOTAL + i];
    for (int i = 0; i < NBITS; ++i) trace_g += gd_s[(i >> 5) * 1024 + (i & 31) * 33];
  }

  const unsigned char* kbase = reinterpret_cast<const unsigned char*>(k_cache) + (size_t)unit * n_max * (size_t)row_stride * 2;
  auto load_tile = [&](int tile) {                           // rows past n are zero-filled
    const int r0 = tile * kTileKeys;
    for (int c = gtid; c < kTileKeys * 16; c += kGroupThreads) {
      const int r = c >> 4, ch = c & 15;
      unsigned char* d = a_t + sw128_offset(kTileKeys, r, ch);
      if (r0 + r < n) cp_async16(d, kbase + (size_t)(r0 + r) * row_stride * 2 + ch * 16);
      else *reinterpret_cast<uint4*>(d) = make_uint4(0u, 0u, 0u, 0u);
    }
    cp_async_commit();
  };
  const uint32_t idesc = umma_idesc_bf16(kTileKeys, NBITS);
  auto issue_gemm = [&]() {                                 // one thread: 8 steps of K = 16 over the 128 channels
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      const size_t aoff = (size_t)(ks >> 2) * (kTileKeys * 128) + (size_t)(ks & 3) * 32;
      const size_t boff = (size_t)(ks >> 2) * (NBITS * 128) + (size_t)(ks & 3) * 32;
      umma_bf16(tmem_base, umma_desc_sw128(a_t + aoff), umma_desc_sw128(b_s + boff), idesc, ks > 0 ? 1u : 0u);
    }
    umma_commit(mma_bar);                                    // arrives when all MMAs issued so far have completed
  };
  // corrections of the columns after block pb by the block's 32 signs: T[:, j0..] += U x (-G[block rows, j0..]),
  // three bf16 terms x two K steps, accumulated into the columns that still wait for their decisions
  auto issue_corrections = [&](int pb) {
    const int j0 = 32 * (pb + 1);
    const uint32_t idc = umma_idesc_bf16(kTileKeys, NBITS - j0);
#pragma unroll
    for (int part = 0; part < 3; ++part) {
#pragma unroll
      for (int ks = 0; ks < 2; ++ks) {
        const unsigned lbo = (unsigned)(gb_cols(pb) >> 3) * 128;
        const unsigned char* ap = u_s + (size_t)ks * 2 * U_LBO;
        const unsigned char* bp = gb_s + gb_off(pb) + (size_t)part * gb_cols(pb) * 64 + (size_t)ks * 2 * lbo;
        umma_bf16(tmem_base + (uint32_t)j0, umma_desc_nosw(ap, U_LBO, 128), umma_desc_nosw(bp, lbo, 128), idc, 1u);
      }
    }
    umma_commit(mma_bar);
  };

  // HALF == 2: T[:, 0..127] += U1 x (-G[0:128, 128:256]); U1 sits in the key-tile buffer (the projection has completed),
  // three bf16 terms x eight K steps
  auto issue_cross = [&]() {
#pragma unroll
    for (int part = 0; part < 3; ++part) {
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const unsigned char* ap = a_t + (size_t)ks * 2 * U_LBO;
        const unsigned char* bp = x_s + (size_t)part * 32768 + (size_t)ks * 2 * U_LBO;
        umma_bf16(tmem_base, umma_desc_nosw(ap, U_LBO, 128), umma_desc_nosw(bp, U_LBO, 128), idesc, 1u);
      }
    }
    umma_commit(mma_bar);
  };

  // Tiles of this warpgroup: kGroups * blockIdx.x + grp, then every kGroups * blocks_per_unit-th.  The warpgroups
  // run independent pipelines (own tile, own accumulator columns, own MMA barrier, own hardware barrier); all threads
  // of a warpgroup take the same branches, so its barrier is always reached by all 128 of them.
  const int tile_step = kGroups * blocks_per_unit;
  int tl = kGroups * blockIdx.x + grp;
  unsigned ph = 0;                                           // phase of the MMA barrier the next wait refers to
  if (tl < ntiles) {
    load_tile(tl);
    cp_async_wait_all();
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    group_sync(grp);
    if (gtid == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      issue_gemm();
    }
  }
  for (; tl < ntiles; tl += tile_step) {
    const int next = tl + tile_step;
    // decision values of this tile: wait for the MMAs, then one TMEM lane (one key) per thread
    if (!mbar_wait(mma_bar, ph)) timed_out_g[grp] = 1;
    ph ^= 1u;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // The MMAs are the only readers of the key tile (besides the key norms below), and they have completed: the
    // buffer is refilled with the warpgroup's next tile right away, under the sweep.
    const int key = tl * kTileKeys + gtid;
    float k2 = 0.f;
    if (key_err != nullptr && HALF != 2) {                   // squared norm of this thread's key, from the operand tile
      if (key < n) {
#pragma unroll
        for (int ch = 0; ch < 16; ++ch) {
          const uint4 w = *reinterpret_cast<const uint4*>(a_t + sw128_offset(kTileKeys, gtid, ch));
          const float f0 = bf16_lo(w.x), f1 = bf16_hi(w.x), f2 = bf16_lo(w.y), f3 = bf16_hi(w.y);
          const float f4 = bf16_lo(w.z), f5 = bf16_hi(w.z), f6 = bf16_lo(w.w), f7 = bf16_hi(w.w);
          k2 += (f0 * f0 + f1 * f1) + (f2 * f2 + f3 * f3) + (f4 * f4 + f5 * f5) + (f6 * f6 + f7 * f7);
        }
      }
      group_sync(grp);                                       // every thread has read its row before the refill starts
    }
    const uint32_t* kwords = reinterpret_cast<const uint32_t*>(codes) + ((size_t)unit * n_max + (key < n ? key : 0)) * NWK;
    if (HALF == 2 && residual_correction) {
      // the first half's 128 signs of this thread's key as row gtid of the bf16 operand U1, written over the key tile
      // (no reader of the tile is left: the MMAs have completed and this launch computes no key norms)
      const uint4 cw = *reinterpret_cast<const uint4*>(kwords);
      const uint32_t w4[4] = {cw.x, cw.y, cw.z, cw.w};
#pragma unroll
      for (int c = 0; c < 16; ++c) {                         // chunk c: signs 8c .. 8c+7
        uint32_t h[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const uint32_t lo = ((w4[c >> 2] >> (8 * (c & 3) + 2 * e)) & 1u) ? 0x3F80u : 0xBF80u;
          const uint32_t hi = ((w4[c >> 2] >> (8 * (c & 3) + 2 * e + 1)) & 1u) ? 0x3F80u : 0xBF80u;
          h[e] = lo | (hi << 16);
        }
        *reinterpret_cast<uint4*>(a_t + (size_t)c * U_LBO + (size_t)(gtid >> 3) * 128 + (size_t)(gtid & 7) * 16) =
            make_uint4(h[0], h[1], h[2], h[3]);
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      group_sync(grp);
      if (gtid == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        issue_cross();
      }
      if (!mbar_wait(mma_bar, ph)) timed_out_g[grp] = 1;     // the decision values now carry the first half's corrections
      ph ^= 1u;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    }
    if (next < ntiles) load_tile(next);
    const uint32_t taddr = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16);   // a warp reaches the lanes of its quarter
    uint32_t words[NB];
    float abs_sum[kPair] = {0.f};                            // sum of |t_i| at decision time (for Eq. 8)
#pragma unroll
    for (int cb = 0; cb < NB; ++cb) {
      if (cb > 0 && residual_correction) {                   // the corrections by block cb - 1 (and all before it) have landed
        if (!mbar_wait(mma_bar, ph)) timed_out_g[grp] = 1;
        ph ^= 1u;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      }
      float t[kPair][32];
      tmem_ld32<0>(taddr + (uint32_t)(32 * cb), t[0]);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      uint32_t word[kPair] = {0u};
      DiagSweep<0>::run(t, word, abs_sum, gd_s + (size_t)cb * 1024, 32, residual_correction);
      words[cb] = word[0];
      if (cb + 1 < NB && residual_correction) {
        // this key's 32 signs as a row of the bf16 operand U (+1 = 0x3F80, -1 = 0xBF80), 8 per 16-byte chunk
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t h[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const uint32_t lo = ((word[0] >> (8 * c + 2 * e)) & 1u) ? 0x3F80u : 0xBF80u;
            const uint32_t hi = ((word[0] >> (8 * c + 2 * e + 1)) & 1u) ? 0x3F80u : 0xBF80u;
            h[e] = lo | (hi << 16);
          }
          *reinterpret_cast<uint4*>(u_s + (size_t)c * U_LBO + (size_t)(gtid >> 3) * 128 + (size_t)(gtid & 7) * 16) =
              make_uint4(h[0], h[1], h[2], h[3]);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        group_sync(grp);                                     // all 128 rows of U are written (and the block's TMEM reads are done)
        if (gtid == 0) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          issue_corrections(cb);
        }
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    if (next < ntiles) {
      cp_async_wait_all();
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    group_sync(grp);                                         // the accumulators have been read by the whole warpgroup; its next tile has landed
    if (timed_out_g[grp]) break;                             // (written only by this warpgroup, before the barrier)
    if (next < ntiles && gtid == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      issue_gemm();
    }
    // squared reconstruction error (Eq. 8) from the sweep: ||k - hP||^2 = ||k||^2 - 2 sum|t_i| + trace(G)
    // (256-bit codes: the first launch leaves ||k||^2 - 2 sum|t_i| of its bits, the second adds its own sum and the trace)
    if (key_err != nullptr && key < n) {
      float* ke = key_err + (size_t)unit * n_max + key;
      if (HALF == 0) *ke = fmaxf(0.f, k2 - 2.f * abs_sum[0] + trace_g);
      else if (HALF == 1) *ke = k2 - 2.f * abs_sum[0];
      else *ke = fmaxf(0.f, *ke - 2.f * abs_sum[0] + trace_g);
    }
    if (key < n) {
      uint32_t* dst = reinterpret_cast<uint32_t*>(codes) + ((size_t)unit * n_max + key) * NWK + (HALF == 2 ? 4 : 0);
      if (NB == 1) {
        dst[0] = words[0];
      } else if (NB == 2) {
        *reinterpret_cast<uint2*>(dst) = make_uint2(words[0], words[1]);
      } else {
#pragma unroll
        for (int w = 0; w + 3 < NB; w += 4) *reinterpret_cast<uint4*>(dst + w) = make_uint4(words[w], words[w + 1], words[w + 2], words[w + 3]);
      }
    }
  }
  if (timed_out_g[grp] && gtid == 0) atomicOr(err, BPC_DEVERR_TIMEOUT);
  cp_async_wait_all();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();                                           // both warpgroups are done with tensor memory
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_all), "r"(kTmemCols) : "memory");
  }
}

template <int NBITS, int GROUPS, int HALF>
cudaError_t launch(bpc_ctx* ctx, const void* k_cache, uint64_t* codes, cudaStream_t stream) {
  const bpc_config& c = ctx->cfg;
  constexpr int NB = NBITS / 32;
  const size_t smem = (size_t)GROUPS * kTileKeys * 256 + (size_t)NBITS * 256 + (size_t)NB * 4096 + (size_t)GROUPS * kTileKeys * 64 +
                      (size_t)3 * 64 * ((NB - 1) * NBITS - 16 * (NB - 1) * NB) +            // (Gram terms: columns after each block)
                      (HALF == 2 ? (size_t)kCrossBytes : 0) + 1024;
  cudaError_t e = cudaFuncSetAttribute(encode_tc_kernel<NBITS, GROUPS, HALF>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int tiles_max = ((c.n_max + kTileKeys - 1) / kTileKeys + GROUPS - 1) / GROUPS;   // a block takes GROUPS tiles at a time
  // Blocks per unit.  One block fits an SM (shared memory), so the grid runs in waves of sm_count blocks and a last,
  // partly filled wave costs as much as a full one: starting from about four waves, take the first count whose last
  // wave is at least 90 % full (32 units on 148 SMs: 23 blocks per unit = 736 blocks = 4.97 waves).
  int bpu = (4 * ctx->sm_count + ctx->units - 1) / ctx->units;
  if (bpu < 1) bpu = 1;
  for (int tries = 0; tries < 16; ++tries) {
    const int rem = (int)(((long long)ctx->units * bpu) % ctx->sm_count);
    if (rem == 0 || rem * 10 >= ctx->sm_count * 9) break;
    ++bpu;
  }
  if (bpu > tiles_max) bpu = tiles_max;
  const dim3 grid(bpu, ctx->units);
  encode_tc_kernel<NBITS, GROUPS, HALF><<<grid, kGroupThreads * GROUPS, smem, stream>>>(
      (const __nv_bfloat16*)k_cache, (const __nv_bfloat16*)ctx->P_h, ctx->gram, ctx->unit_lens, codes, ctx->dev_err,
      c.n_kv_heads, c.n_max, ctx->row_stride, c.hash_sets != ctx->units, c.residual_correction, bpu, ctx->key_err);
  return cudaGetLastError();
}

}  // namespace

// bf16 caches run on the tensor cores: 32-, 64- and 128-bit codes in one launch, 256-bit codes in two (the bf16 terms of
// a 256 x 256 Gram matrix do not fit shared memory next to the operands, those of its 128 x 128 blocks do).  fp32 caches
// report "not supported" and the caller falls back to the CUDA-core kernel (they have no bf16 operands).
cudaError_t bpc_launch_encode_tc(bpc_ctx* ctx, const void* k_cache, uint64_t* codes, cudaStream_t stream) {
  if (ctx->cfg.kv_dtype != BPC_BF16) return cudaErrorNotSupported;
  if (ctx->no_tc_encode) return cudaErrorNotSupported;     // diagnostic switch: the CUDA-core kernel is asked for
  cudaError_t e;
  if (ctx->cfg.code_bits == 32) e = launch<32, kGroups, 0>(ctx, k_cache, codes, stream);
  else if (ctx->cfg.code_bits == 64) e = launch<64, kGroups, 0>(ctx, k_cache, codes, stream);
  else if (ctx->cfg.code_bits == 128) e = launch<128, kGroups, 0>(ctx, k_cache, codes, stream);
  else if (ctx->cfg.code_bits == 256) {
    e = launch<128, kGroups, 1>(ctx, k_cache, codes, stream);
    if (e == cudaSuccess) {
      ctx->launches += 1;
      e = launch<128, 1, 2>(ctx, k_cache, codes, stream);
    }
  } else return cudaErrorNotSupported;
  if (e == cudaSuccess) ctx->launches += 1;
  return e;
}
