// Tensor-core encode: Algorithm 2 for all cached keys of bf16 caches.
//
// The decision values before any correction are a dense contraction T = K P_h^T (keys x channels times
// channels x bits).  It runs on the 5th-generation tensor cores: per block, tiles of 128 keys (M = 128) against
// the unit's b projection rows (N = b, 64 or 128) over the 128 channels (eight tcgen05.mma steps of K = 16), bf16
// operands in shared memory in the 128-byte-swizzled K-major layout, fp32 accumulator in tensor memory with one
// key per TMEM lane.  Each of the 128 threads of a warpgroup then pulls its key's b decision values out of tensor
// memory (tcgen05.ld) into registers and runs the greedy sweep of Algorithm 2 in its Gram form
//     u_i = sign(t_i);  t_j -= u_i * G_ij  (j > i),   G = P_h P_h^T,
// which equals updating the residual r <- r - u_i P_i and testing r . P_{i+1}.  While the threads sweep tile i,
// the asynchronous copy of tile i+1 is already in flight.  A block holds two such warpgroups, which share the
// projection rows and the Gram matrix in shared memory and otherwise run independent pipelines, and every warpgroup
// works on two key tiles at once, one key of each per thread: the sweep is a chain of dependent FMAs per key fed by
// broadcast reads of the Gram matrix, so one warp per scheduler cannot keep the FP32 pipe busy, and with one key per
// thread the shared-memory reads (one 16-byte read per four FMAs) bound it.
//
// Waits on the MMA-completion mbarrier are bounded: on expiry the block raises the device error word, still
// releases its tensor memory and returns.
#include <stdlib.h>
#include "common.cuh"

namespace {

constexpr int kTileKeys = 128;
constexpr int kGroupThreads = 128;   // one warpgroup sweeps one key tile (a TMEM lane per thread)
constexpr int kGroups = 2;           // warpgroups per block, each with its own tiles, accumulator columns and barrier
constexpr int kPair = 2;             // key tiles a warpgroup sweeps together, one key of each per thread: every Gram
                                     // value read from shared memory then feeds two FMAs (the loads bound the sweep)
constexpr int kThreads = kGroupThreads * kGroups;

__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
// barrier among the 128 threads of one warpgroup (hardware barriers 1 .. kGroups; 0 is __syncthreads)
__device__ __forceinline__ void group_sync(int g) { asm volatile("bar.sync %0, %1;" ::"r"(1 + g), "r"(kGroupThreads) : "memory"); }

// Shared-memory operand descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw128(const void* smem_ptr) {
  const uint64_t addr = (uint64_t)(smem_u32(smem_ptr) & 0x3FFFF) >> 4;
  uint64_t d = addr;                       // bits [0,14): start address / 16
  d |= (uint64_t)1 << 16;                  // bits [16,30): leading-dimension byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;        // bits [32,46): stride between 8-row groups / 16
  d |= (uint64_t)1 << 46;                  // bits [46,48): descriptor version of this architecture
  d |= (uint64_t)2 << 61;                  // bits [61,64): 128-byte swizzle
  return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, N and M.
__device__ __forceinline__ uint32_t umma_idesc_bf16(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}\n"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
// bounded wait on an mbarrier phase; false when the iteration budget runs out
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity) {
  for (int it = 0; it < 20000000; ++it) {
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    if (ok) return true;
  }
  return false;
}
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
      const float* gi = g_diag + I * ld;
#pragma unroll
      for (int j = I + 1; j < 32; ++j) {
        const float g = gi[j];
#pragma unroll
        for (int q = 0; q < kPair; ++q) t[q][j] = fmaf(-u[q], g, t[q][j]);
      }
    }
    DiagSweep<I + 1>::run(t, word, abs_sum, g_diag, ld, rc);
  }
};
template <>
struct DiagSweep<32> {
  static __device__ __forceinline__ void run(float (&)[kPair][32], uint32_t (&)[kPair], float (&)[kPair], const float*, int, int) {}
};

// byte offset of 16-byte chunk `ch` (0..15) of row `r` inside a [rows x 128 channels] bf16 operand tile:
// two column blocks of 64 channels (128 bytes per row each), chunks XOR-swizzled by the row number
__device__ __forceinline__ size_t sw128_offset(int rows, int r, int ch) {
  return (size_t)(ch >> 3) * ((size_t)rows * 128) + (size_t)r * 128 + (size_t)(((ch & 7) ^ (r & 7)) << 4);
}

template <int NBITS>
__global__ void __launch_bounds__(kThreads, 1)
encode_tc_kernel(const __nv_bfloat16* __restrict__ k_cache, const __nv_bfloat16* __restrict__ Ph, const float* __restrict__ gram,
                 const int32_t* __restrict__ unit_lens, uint64_t* __restrict__ codes, int32_t* __restrict__ err,
                 int n_kv_heads, int n_max, int row_stride, int shared_sets, int residual_correction, int blocks_per_unit,
                 float* __restrict__ key_err) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // the swizzled operand tiles need 1024-byte alignment in the shared address space
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  constexpr int A_BYTES = kTileKeys * 256;                 // one key tile (128 rows x 128 bf16)
  constexpr int B_BYTES = NBITS * 256;                     // the projection rows
  const int tid = threadIdx.x, warp = tid >> 5;
  const int grp = tid / kGroupThreads, gtid = tid % kGroupThreads;   // warpgroup and thread within it
  unsigned char* a_t = smem + (size_t)(grp * kPair) * A_BYTES;   // this warpgroup's kPair key tiles (one buffer each: see the loop)
  unsigned char* b_s = smem + kGroups * kPair * A_BYTES;
  float* g_s = reinterpret_cast<float*>(smem + kGroups * kPair * A_BYTES + B_BYTES);   // [NBITS][NBITS]
  __shared__ unsigned long long mma_bar_s[kGroups];
  __shared__ uint32_t tmem_base_s;
  __shared__ int timed_out_g[kGroups];
  unsigned long long* mma_bar = &mma_bar_s[grp];
  constexpr int kAccCols = kGroups * kPair * NBITS;        // fp32 accumulator columns of all tiles in flight
  constexpr int kTmemCols = kAccCols <= 32 ? 32 : kAccCols <= 64 ? 64 : kAccCols <= 128 ? 128 : kAccCols <= 256 ? 256 : 512;   // a power of two >= 32
  static_assert(kAccCols <= 512, "accumulators exceed tensor memory");

  const int unit = blockIdx.y;
  const int n = min(unit_lens[unit], n_max);
  const int ntiles = (n + kTileKeys - 1) / kTileKeys;
  const int set = shared_sets ? unit % n_kv_heads : unit;

  // ---- one-time set-up: barrier, tensor memory, projection and Gram matrix in shared memory
  if (tid == 0) {
    for (int g = 0; g < kGroups; ++g) { mbar_init(&mma_bar_s[g], 1); timed_out_g[g] = 0; }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  {
    const unsigned char* psrc = reinterpret_cast<const unsigned char*>(Ph + (size_t)set * NBITS * BPC_D);
    for (int c = tid; c < NBITS * 16; c += kThreads) {
      const int r = c >> 4, ch = c & 15;
      *reinterpret_cast<uint4*>(b_s + sw128_offset(NBITS, r, ch)) = *reinterpret_cast<const uint4*>(psrc + (size_t)r * 256 + ch * 16);
    }
    const float4* gsrc = reinterpret_cast<const float4*>(gram + (size_t)set * NBITS * NBITS);
    for (int c = tid; c < NBITS * NBITS / 4; c += kThreads) reinterpret_cast<float4*>(g_s)[c] = gsrc[c];
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_all = tmem_base_s;
  const uint32_t tmem_base = tmem_all + (uint32_t)(grp * kPair * NBITS);   // this warpgroup's accumulator columns (tile q at + q * NBITS)
  float trace_g = 0.f;
  if (key_err != nullptr)
    for (int i = 0; i < NBITS; ++i) trace_g += g_s[i * NBITS + i];

  const unsigned char* kbase = reinterpret_cast<const unsigned char*>(k_cache) + (size_t)unit * n_max * (size_t)row_stride * 2;
  auto load_tile = [&](int tile, unsigned char* dst) {
    const int r0 = tile * kTileKeys;
    for (int c = gtid; c < kTileKeys * 16; c += kGroupThreads) {
      const int r = c >> 4, ch = c & 15;
      unsigned char* d = dst + sw128_offset(kTileKeys, r, ch);
      if (r0 + r < n) cp_async16(d, kbase + (size_t)(r0 + r) * row_stride * 2 + ch * 16);
      else *reinterpret_cast<uint4*>(d) = make_uint4(0u, 0u, 0u, 0u);
    }
    cp_async_commit();
  };
  const uint32_t idesc = umma_idesc_bf16(kTileKeys, NBITS);
  auto issue_mma = [&]() {                                  // one thread: per tile 8 steps of K = 16 over the 128 channels
#pragma unroll
    for (int q = 0; q < kPair; ++q) {
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const size_t aoff = (size_t)q * A_BYTES + (size_t)(ks >> 2) * (kTileKeys * 128) + (size_t)(ks & 3) * 32;
        const size_t boff = (size_t)(ks >> 2) * (NBITS * 128) + (size_t)(ks & 3) * 32;
        umma_bf16(tmem_base + (uint32_t)(q * NBITS), umma_desc_sw128(a_t + aoff), umma_desc_sw128(b_s + boff), idesc, ks > 0 ? 1u : 0u);
      }
    }
    umma_commit(mma_bar);                                    // arrives when all MMAs issued so far have completed
  };
  auto load_pair = [&](int pr) {                             // tiles kPair * pr + q; rows past n are zero-filled
#pragma unroll
    for (int q = 0; q < kPair; ++q) load_tile(kPair * pr + q, a_t + (size_t)q * A_BYTES);
  };

  // Tile pairs of this warpgroup: kGroups * blockIdx.x + grp, then every kGroups * blocks_per_unit-th.  The warpgroups
  // run independent pipelines (own tiles, own accumulator columns, own MMA barrier, own hardware barrier); all threads
  // of a warpgroup take the same branches, so its barrier is always reached by all 128 of them.
  const int npairs = (ntiles + kPair - 1) / kPair;
  const int pair_step = kGroups * blocks_per_unit;
  int pr = kGroups * blockIdx.x + grp;
  int it = 0;
  if (pr < npairs) {
    load_pair(pr);
    cp_async_wait_all();
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the tensor core
    group_sync(grp);
    if (gtid == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      issue_mma();
    }
  }
  for (; pr < npairs; pr += pair_step, ++it) {
    const int next = pr + pair_step;
    // decision values of these tiles: wait for the MMAs, then one TMEM lane (one key of each tile) per thread
    bool ok = mbar_wait(mma_bar, (unsigned)(it & 1));
    if (!ok) timed_out_g[grp] = 1;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // The MMAs are the only readers of the key tiles (besides the key norms below), and they have completed: the
    // buffers are refilled with the warpgroup's next tiles right away, under the sweep, which is many times longer
    // than the copy.
    int key[kPair];
    float k2[kPair];
#pragma unroll
    for (int q = 0; q < kPair; ++q) { key[q] = (kPair * pr + q) * kTileKeys + gtid; k2[q] = 0.f; }
    if (key_err != nullptr) {                                // squared norms of this thread's keys, from the operand tiles
#pragma unroll
      for (int q = 0; q < kPair; ++q) {
        if (key[q] < n) {
#pragma unroll
          for (int ch = 0; ch < 16; ++ch) {
            const uint4 w = *reinterpret_cast<const uint4*>(a_t + (size_t)q * A_BYTES + sw128_offset(kTileKeys, gtid, ch));
            const float f0 = bf16_lo(w.x), f1 = bf16_hi(w.x), f2 = bf16_lo(w.y), f3 = bf16_hi(w.y);
            const float f4 = bf16_lo(w.z), f5 = bf16_hi(w.z), f6 = bf16_lo(w.w), f7 = bf16_hi(w.w);
            k2[q] += (f0 * f0 + f1 * f1) + (f2 * f2 + f3 * f3) + (f4 * f4 + f5 * f5) + (f6 * f6 + f7 * f7);
          }
        }
      }
      group_sync(grp);                                       // every thread has read its rows before the refill starts
    }
    if (next < npairs) load_pair(next);
    const uint32_t taddr = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16);   // a warp reaches the lanes of its quarter
    // Column blocks of 32 bits: pull the block out of tensor memory, apply the corrections of all earlier
    // bits (t_j -= u_i G_ij, G rows are broadcast reads from shared memory), then sweep the block itself.
    uint32_t words[kPair][NBITS / 32];
    float abs_sum[kPair];                                    // sum of |t_i| at decision time (for Eq. 8)
#pragma unroll
    for (int q = 0; q < kPair; ++q) {
      abs_sum[q] = 0.f;
#pragma unroll
      for (int w = 0; w < NBITS / 32; ++w) words[q][w] = 0u;
    }
#pragma unroll 1
    for (int cb = 0; cb < NBITS / 32; ++cb) {
      float t[kPair][32];
#pragma unroll
      for (int q = 0; q < kPair; ++q) tmem_ld32<0>(taddr + (uint32_t)(q * NBITS + 32 * cb), t[q]);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      if (residual_correction) {
#pragma unroll 1
        for (int pb = 0; pb < cb; ++pb) {
          uint32_t wprev[kPair];                             // words[q][pb], selected without indexing registers
#pragma unroll
          for (int q = 0; q < kPair; ++q) {
            wprev[q] = words[q][0];
#pragma unroll
            for (int w = 1; w < NBITS / 32; ++w) wprev[q] = pb == w ? words[q][w] : wprev[q];
          }
#pragma unroll 4
          for (int i = 0; i < 32; ++i) {
            float mu[kPair];                                 // minus the sign of bit 32 pb + i
#pragma unroll
            for (int q = 0; q < kPair; ++q) mu[q] = ((wprev[q] >> i) & 1u) ? -1.f : 1.f;
            const float4* gi = reinterpret_cast<const float4*>(g_s + (size_t)(32 * pb + i) * NBITS + 32 * cb);
#pragma unroll
            for (int j4 = 0; j4 < 8; ++j4) {
              const float4 gv = gi[j4];
#pragma unroll
              for (int q = 0; q < kPair; ++q) {
                t[q][4 * j4] = fmaf(mu[q], gv.x, t[q][4 * j4]);
                t[q][4 * j4 + 1] = fmaf(mu[q], gv.y, t[q][4 * j4 + 1]);
                t[q][4 * j4 + 2] = fmaf(mu[q], gv.z, t[q][4 * j4 + 2]);
                t[q][4 * j4 + 3] = fmaf(mu[q], gv.w, t[q][4 * j4 + 3]);
              }
            }
          }
        }
      }
      uint32_t word[kPair];
#pragma unroll
      for (int q = 0; q < kPair; ++q) word[q] = 0u;
      DiagSweep<0>::run(t, word, abs_sum, g_s + (size_t)(32 * cb) * NBITS + 32 * cb, NBITS, residual_correction);
#pragma unroll
      for (int q = 0; q < kPair; ++q) {
#pragma unroll
        for (int w = 0; w < NBITS / 32; ++w) words[q][w] = cb == w ? word[q] : words[q][w];
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    if (next < npairs) {
      cp_async_wait_all();
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    group_sync(grp);                                         // the accumulators have been read by the whole warpgroup; its next tiles have landed
    if (timed_out_g[grp]) break;                             // (written only by this warpgroup, before the barrier)
    if (next < npairs && gtid == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      issue_mma();
    }
#pragma unroll
    for (int q = 0; q < kPair; ++q) {
      // squared reconstruction error (Eq. 8) from the sweep: ||k - hP||^2 = ||k||^2 - 2 sum|t_i| + trace(G)
      if (key_err != nullptr && key[q] < n) key_err[(size_t)unit * n_max + key[q]] = fmaxf(0.f, k2[q] - 2.f * abs_sum[q] + trace_g);
      if (key[q] < n) {
        uint32_t* dst = reinterpret_cast<uint32_t*>(codes + ((size_t)unit * n_max + key[q]) * (NBITS / 64));
        if (NBITS == 64) {
          *reinterpret_cast<uint2*>(dst) = make_uint2(words[q][0], words[q][1]);
        } else {
#pragma unroll
          for (int w = 0; w < NBITS / 32; w += 4) *reinterpret_cast<uint4*>(dst + w) = make_uint4(words[q][w], words[q][w + 1], words[q][w + 2], words[q][w + 3]);
        }
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

template <int NBITS>
cudaError_t launch(bpc_ctx* ctx, const void* k_cache, uint64_t* codes, cudaStream_t stream) {
  const bpc_config& c = ctx->cfg;
  const size_t smem = (size_t)kGroups * kPair * kTileKeys * 256 + (size_t)NBITS * 256 + (size_t)NBITS * NBITS * 4 + 1024;
  cudaError_t e = cudaFuncSetAttribute(encode_tc_kernel<NBITS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int tiles_max = ((c.n_max + kTileKeys - 1) / kTileKeys + kGroups * kPair - 1) / (kGroups * kPair);   // a block takes kGroups * kPair tiles at a time
  // Blocks per unit.  One block fits an SM (shared memory), so the grid runs in waves of sm_count blocks and a last,
  // partly filled wave costs as much as a full one: starting from about four waves, take the first count whose last
  // wave is at least 90 % full (32 units on 148 SMs: 23 blocks per unit = 736 blocks = 4.97 waves; the 10 used before
  // gave 2.16 waves, i.e. three rounds for two rounds' worth of work).
  int bpu = (4 * ctx->sm_count + ctx->units - 1) / ctx->units;
  if (bpu < 1) bpu = 1;
  for (int tries = 0; tries < 16; ++tries) {
    const int rem = (int)(((long long)ctx->units * bpu) % ctx->sm_count);
    if (rem == 0 || rem * 10 >= ctx->sm_count * 9) break;
    ++bpu;
  }
  if (bpu > tiles_max) bpu = tiles_max;
  const dim3 grid(bpu, ctx->units);
  encode_tc_kernel<NBITS><<<grid, kThreads, smem, stream>>>(
      (const __nv_bfloat16*)k_cache, (const __nv_bfloat16*)ctx->P_h, ctx->gram, ctx->unit_lens, codes, ctx->dev_err,
      c.n_kv_heads, c.n_max, ctx->row_stride, c.hash_sets != ctx->units, c.residual_correction, bpu, ctx->key_err);
  return cudaGetLastError();
}

}  // namespace

// bf16 caches with 64- or 128-bit codes run on the tensor cores; other shapes report "not supported" and the
// caller falls back to the CUDA-core kernel (fp32 caches have no bf16 operands; at 256 bits the Gram matrix no
// longer fits next to the operands in shared memory).
cudaError_t bpc_launch_encode_tc(bpc_ctx* ctx, const void* k_cache, uint64_t* codes, cudaStream_t stream) {
  if (ctx->cfg.kv_dtype != BPC_BF16) return cudaErrorNotSupported;
  if (ctx->no_tc_encode) return cudaErrorNotSupported;     // diagnostic switch: the CUDA-core kernel is asked for
  cudaError_t e;
  if (ctx->cfg.code_bits == 64) e = launch<64>(ctx, k_cache, codes, stream);
  else if (ctx->cfg.code_bits == 128) e = launch<128>(ctx, k_cache, codes, stream);
  else return cudaErrorNotSupported;
  if (e == cudaSuccess) ctx->launches += 1;
  return e;
}
