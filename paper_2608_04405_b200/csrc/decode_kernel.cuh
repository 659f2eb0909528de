// Fused decode step: query hash -> code scan -> top-k -> gathered softmax attention, one thread-block
// cluster per (sequence, KV head) unit.
//
// Section 3.2 "Retrieval Phase" and Algorithm 3 define the score c = (q P^T) h^T on the quantised
// projection; the appendix "CUDA Optimizations on Bitwise Operations" evaluates it with XOR, AND and
// popcount on bit planes.  Here the query heads of one KV head are first collapsed into a single
// integer weight vector A = sum_g s_g * a_g, whose sign word and magnitude bit planes play the role
// of the paper's eight packed query words; the score of key h is <A, h>.
//
// Phases of a cluster of CS blocks working on one unit with n cached keys:
//   0  every block hashes the group's queries (identical arithmetic in all blocks)
//   1  block r scans keys [r*chunk, (r+1)*chunk): 128-bit code loads, LOP3 (+ carry-save compression) and
//      POPC score, 16-bit score key into shared memory, shared-memory histogram.  In a launch that also appends
//      a key, the last warp of the block that owns the new key codes it (Algorithm 2) meanwhile.
//   2  every block stores its histogram into its peers' shared memory; cluster barrier; the threshold key T
//      and the per-block output offsets follow from one block scan; each block emits its selected indices in
//      ascending order (score > T, then the lowest-index ties at T) into the unit's index list
//   3  cluster barrier; block r runs online-softmax attention over rows [k*r/CS, k*(r+1)/CS) of the
//      list.  Rows are gathered into per-warp shared-memory rings with 16-byte asynchronous copies; bf16 caches
//      use warp-level tensor-core MMAs (q K^T, then P V with P split in two bf16 halves), fp32 caches use
//      fp64 arithmetic on the CUDA cores.  Partial (m, l, acc) are merged inside the block, stored into the
//      shared memory of the block that owns each output, and finished there after one more cluster barrier.
// Scores and gathered rows never touch global memory.
#pragma once
#include <type_traits>
#include <cooperative_groups.h>
#include "common.cuh"

namespace bpcdev {
namespace cg = cooperative_groups;

constexpr int kSegKeys = 32;        // score keys per shared-memory segment
constexpr int kSegSlots = 40;       // 16-bit slots per segment (80 B: conflict-free 16-byte reads)
constexpr int kMaxBins = 2048;      // histogram bins (score keys are 0..nbins-1)
constexpr int kIdxTile = 1024;      // selected indices staged at a time (fp32 path, long lists)
constexpr int kMaxPlanes = 10;
constexpr int kEasMax = 16384;      // largest error-aware safeguard set per unit
constexpr int kUnrolledSweepKeys = 16384;   // key ranges shorter than this take the unrolled sign sweep of the appended key
constexpr int kEasLocal = 1024;     // safeguard keys of one block kept in shared memory (larger slices stay in global)

template <int GP, int MODE> struct PlaneCount {
  static constexpr int value = MODE == 0 ? (GP <= 2 ? 1 : (GP == 4 ? 2 : 3))
                                         : (GP == 1 ? 7 : (GP == 2 ? 8 : (GP == 4 ? 9 : 10)));
};

struct SmallState {
  uint32_t signw[8];
  uint32_t mask[kMaxPlanes][8];
  uint32_t gt[BPC_MAX_CLUSTER];
  uint32_t eq[BPC_MAX_CLUSTER];
  uint32_t wgt[32], weq[32];             // streaming selection: per-warp numbers of keys above / at the threshold
  uint32_t wscan[64];                    // block scans: two alternating buffers of 2 x 16 warp totals (16-byte aligned)
  double pmax[BPC_MAX_GROUP];
  int T, cnt_gt, my_take, my_base, rsum, e0, e1, pad;
  uint32_t newcode[8];                   // code of the key appended by this launch
  int32_t eas_s[kEasLocal];              // this block's slice of the safeguard set (when it fits)
  uint8_t stage_valid[32][4];            // per warp and gather stage: which of the 8 rows are real
};

template <typename KV> struct IsBf16 { static constexpr bool value = false; };
template <> struct IsBf16<__nv_bfloat16> { static constexpr bool value = true; };

// Shared-memory plan of one block, computed identically on host and device.
template <typename KV, int GP, int W32>
struct DecodeSmem {
  typedef typename KvTraits<KV>::acc_t acc_t;
  static constexpr bool kMma = IsBf16<KV>::value;
  static constexpr int NT = kMma ? 512 : (GP <= 2 ? 512 : 256);
  static constexpr int NW = NT / 32;
  static constexpr int B = W32 * 32;
  static constexpr int kRowBytes = BPC_D * (int)sizeof(KV);
  // gather staging: bf16 tiles hold 8 rows per warp (K rows, then V rows, 16-byte chunks XOR-swizzled);
  // fp32 tiles hold 32 rows, each K row followed by its V row
  static constexpr int kTileRows = kMma ? 8 * NW : 32;
  static constexpr int kStageBytes = kTileRows * 2 * kRowBytes;
  __host__ __device__ static constexpr size_t a16(size_t x) { return (x + 15) & ~(size_t)15; }
  __host__ __device__ static constexpr size_t part_bytes() { return (size_t)NW * GP * (BPC_D + 2) * sizeof(acc_t); }
  static constexpr int GV = GP + 1;      // vectors projected in phase 0: the group's queries and the appended key
  __host__ __device__ static constexpr size_t hashpart_bytes() { return (size_t)NT * GV * 8; }

  size_t off_hist, off_tot, off_qf, off_pd, off_idx, off_cta, off_small, off_union, total;
  // bytes of the score keys of a block: 16-bit keys in padded 32-key segments, or (key_bytes == 1) plain bytes
  __host__ __device__ static constexpr size_t score_bytes(int chunk_cap, int key_bytes) {
    return key_bytes == 1 ? (size_t)((chunk_cap + kSegKeys - 1) / kSegKeys) * kSegKeys
                          : (size_t)((chunk_cap + kSegKeys - 1) / kSegKeys) * kSegSlots * 2;
  }
  __host__ __device__ DecodeSmem(int chunk_cap, int nbins, int stages, int key_bytes = 2) {
    const size_t nb = a16((size_t)nbins * 4);
    off_hist = 0;
    off_tot = off_hist + nb;
    off_qf = off_tot + nb;                                           // float[GP+1][128]
    off_pd = off_qf + (size_t)GV * BPC_D * 4;                        // double[GP+1][B]
    off_idx = off_pd + (size_t)GV * B * 8;                           // int32[kIdxTile]
    off_cta = off_idx + kIdxTile * 4;                                // merge inbox: acc_t[GP * (128 + 2 * 16) + 16]
    off_small = a16(off_cta + ((size_t)GP * (BPC_D + 2 * BPC_MAX_CLUSTER) + BPC_MAX_CLUSTER) * sizeof(acc_t));
    off_union = a16(off_small + sizeof(SmallState));
    size_t u = score_bytes(chunk_cap, key_bytes);                                  // score keys
    if (u < part_bytes()) u = part_bytes();                                      // block-level merge
    if (u < hashpart_bytes()) u = hashpart_bytes();                              // query-hash partial sums
    if (u < (size_t)stages * kStageBytes) u = (size_t)stages * kStageBytes;      // gather ring
    total = off_union + a16(u);
  }
};

__device__ __forceinline__ int score_slot(int i) { return (i >> 5) * kSegSlots + (i & 31); }

// Exclusive prefix sum over the NT threads of a block; *total receives the block sum.  One barrier per call: the warp
// totals come from a warp reduction and are posted before each warp scans its own lanes, and consecutive calls
// alternate between two buffers (ph, the number of calls so far, is uniform over the block), so a warp that is early
// for the next call cannot overwrite totals that a late warp still reads.  wscan holds 2 x 2 x 16 words.
template <int NT>
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* wscan, int& ph, uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t* buf = wscan + (ph & 1) * 32;
  ++ph;
  const uint32_t wt = __reduce_add_sync(0xffffffffu, v);
  if (lane == 0) buf[warp] = wt;
  uint32_t inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();
  uint32_t wbase = 0, tot = 0;
#pragma unroll
  for (int w4 = 0; w4 < NT / 128; ++w4) {
    const uint4 q = reinterpret_cast<const uint4*>(buf)[w4];
    const uint32_t e[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (4 * w4 + i < warp) wbase += e[i];
      tot += e[i];
    }
  }
  *total = tot;
  return wbase + inc - v;
}

// the same for two values at once
template <int NT>
__device__ __forceinline__ void block_excl_scan2(uint32_t a, uint32_t b, uint32_t* wscan, int& ph, uint32_t& ea, uint32_t& eb) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t* buf = wscan + (ph & 1) * 32;
  ++ph;
  const uint32_t wa = __reduce_add_sync(0xffffffffu, a), wb = __reduce_add_sync(0xffffffffu, b);
  if (lane == 0) { buf[warp] = wa; buf[16 + warp] = wb; }
  uint32_t ia = a, ib = b;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t ta = __shfl_up_sync(0xffffffffu, ia, o), tb = __shfl_up_sync(0xffffffffu, ib, o);
    if (lane >= o) { ia += ta; ib += tb; }
  }
  __syncthreads();
  uint32_t ba = 0, bb = 0;
#pragma unroll
  for (int w4 = 0; w4 < NT / 128; ++w4) {
    const uint4 qa = reinterpret_cast<const uint4*>(buf)[w4], qb = reinterpret_cast<const uint4*>(buf + 16)[w4];
    const uint32_t xa[4] = {qa.x, qa.y, qa.z, qa.w}, xb[4] = {qb.x, qb.y, qb.z, qb.w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (4 * w4 + i < warp) { ba += xa[i]; bb += xb[i]; }
  }
  ea = ba + ia - a;
  eb = bb + ib - b;
}

template <typename T> __device__ __forceinline__ T fast_exp2(T x);
template <> __device__ __forceinline__ float fast_exp2<float>(float x) { return exp2f(x); }
template <> __device__ __forceinline__ double fast_exp2<double>(double x) { return exp2(x); }

// 16-byte asynchronous global->shared copy (bypasses L1 and registers) and its group bookkeeping
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// ---- warp-level tensor-core helpers (legacy mma.sync path; M = 16 is padded query heads)
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* smem_row) {
  const unsigned a = (unsigned)__cvta_generic_to_shared(smem_row);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem_row) {
  const unsigned a = (unsigned)__cvta_generic_to_shared(smem_row);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
// D(16x8,f32) += A(16x16,bf16,row) * B(16x8,bf16,col); rows 8..15 of A are zero here (a1 = a3 = 0)
__device__ __forceinline__ void mma_qk(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  const uint32_t z = 0u;
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(z), "r"(a2), "r"(z), "r"(b0), "r"(b1));
}
// D(16x8,f32) += A(16x8,bf16,row) * B(8x8,bf16,col)
__device__ __forceinline__ void mma_pv(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(b0));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// carry-save adder on 32 bit positions at once
__device__ __forceinline__ void csa(uint32_t a, uint32_t b, uint32_t c, uint32_t& sum, uint32_t& carry) {
  sum = a ^ b ^ c;
  carry = (a & b) | (a & c) | (b & c);
}
// ---- score key of one code: sum over planes of weight * popc(agree & mask); agree = ~(h ^ sign)
template <int W32, int NP>
__device__ __forceinline__ int score_key(const uint32_t (&h)[W32], const uint32_t (&sg)[W32], const uint32_t (&mk)[NP][W32]) {
  int key = 0;
  if constexpr (NP >= 3 && W32 >= 2) {
    // Three or more planes (weighted scores; Hamming scores with five to eight query heads per KV head, where it took
    // config 4's step from 46.7 to 44.7 us): one population count per masked word would keep the 16-lane pipe busy for most
    // of the scan.  A full adder per pair of masked words adds them to a carry word handed down from the plane below
    // (a + b + c = (a ^ b ^ c) + 2 maj(a, b, c), bit by bit), which halves the counts: W32/2 per plane plus W32/2 for
    // the last carries.  Each adder is three three-input logic operations, the masks included:
    // t = a ^ c, s = b ^ t, maj(a, b, c) = c ^ (t & (b ^ c)) with b ^ c = s ^ t ^ c.
    constexpr int C = W32 / 2;
    uint32_t cy[C], x[W32];
#pragma unroll
    for (int f = 0; f < C; ++f) cy[f] = 0u;
#pragma unroll
    for (int w = 0; w < W32; ++w) x[w] = ~(h[w] ^ sg[w]);
#pragma unroll
    for (int pl = 0; pl < NP; ++pl) {
      int c = 0;
#pragma unroll
      for (int f = 0; f < C; ++f) {
        const uint32_t t = (x[2 * f] & mk[pl][2 * f]) ^ cy[f];
        const uint32_t s = (x[2 * f + 1] & mk[pl][2 * f + 1]) ^ t;
        cy[f] = cy[f] ^ (t & (s ^ t ^ cy[f]));
        c += __popc(s);
      }
      key += c << pl;
    }
    int c = 0;
#pragma unroll
    for (int f = 0; f < C; ++f) c += __popc(cy[f]);
    key += c << NP;
    return key;
  }
#pragma unroll
  for (int pl = 0; pl < NP; ++pl) {
    int c = 0;
#pragma unroll
    for (int w = 0; w < W32; ++w) c += __popc(~(h[w] ^ sg[w]) & mk[pl][w]);
    key += c << pl;
  }
  return key;
}
// 128-bit codes with two planes (weights 1 and 2): carry-save adders fold the eight masked words into five
// before the population counts, which run on the 16-lane pipe
template <>
__device__ __forceinline__ int score_key<4, 2>(const uint32_t (&h)[4], const uint32_t (&sg)[4], const uint32_t (&mk)[2][4]) {
  uint32_t x0[4], x1[4];
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    const uint32_t agree = ~(h[w] ^ sg[w]);
    x0[w] = agree & mk[0][w];
    x1[w] = agree & mk[1][w];
  }
  uint32_t s0, c0, s1, c1, s2, c2;
  csa(x0[0], x0[1], x0[2], s0, c0);       // ones -> one ones word + one twos word
  csa(c0, x1[0], x1[1], s1, c1);          // twos -> twos + fours
  csa(s1, x1[2], x1[3], s2, c2);
  return __popc(s0) + __popc(x0[3]) + 2 * __popc(s2) + 4 * (__popc(c1) + __popc(c2));
}

// Weighted scores of U codes at once, planes in the outer loop.  The plane masks (up to ten planes of W32 words) are
// read from shared memory one plane at a time (the whole warp reads one address: a broadcast) instead of living in
// registers, which leaves the registers to the U codes and their carry words: U independent dependency chains per
// thread instead of two, so that the logic and population-count pipes stay busy.  Same arithmetic as score_key.
template <int W32, int NP, int U>
__device__ __forceinline__ void score_keys_plane_outer(const uint32_t (&h)[U][W32], const uint32_t (&sg)[W32],
                                                       const uint32_t (*mask)[8], int (&key)[U]) {
  static_assert(W32 >= 2 && W32 % 2 == 0, "pairs of words");
  constexpr int C = W32 / 2;
  uint32_t x[U][W32], cy[U][C];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    key[u] = 0;
#pragma unroll
    for (int f = 0; f < C; ++f) cy[u][f] = 0u;
#pragma unroll
    for (int w = 0; w < W32; ++w) x[u][w] = ~(h[u][w] ^ sg[w]);
  }
#pragma unroll
  for (int pl = 0; pl < NP; ++pl) {
    uint32_t m[W32];
    if constexpr (W32 % 4 == 0) {
#pragma unroll
      for (int w = 0; w < W32; w += 4) {
        const uint4 v = *reinterpret_cast<const uint4*>(&mask[pl][w]);
        m[w] = v.x; m[w + 1] = v.y; m[w + 2] = v.z; m[w + 3] = v.w;
      }
    } else {
      const uint2 v = *reinterpret_cast<const uint2*>(&mask[pl][0]);
      m[0] = v.x; m[1] = v.y;
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      int c = 0;
#pragma unroll
      for (int f = 0; f < C; ++f) {
        const uint32_t t = (x[u][2 * f] & m[2 * f]) ^ cy[u][f];
        const uint32_t s2 = (x[u][2 * f + 1] & m[2 * f + 1]) ^ t;
        cy[u][f] = cy[u][f] ^ (t & (s2 ^ t ^ cy[u][f]));
        c += __popc(s2);
      }
      key[u] += c << pl;
    }
  }
#pragma unroll
  for (int u = 0; u < U; ++u) {
    int c = 0;
#pragma unroll
    for (int f = 0; f < C; ++f) c += __popc(cy[u][f]);
    key[u] += c << NP;
  }
}

// K/V row fragment of 8 consecutive dims held by one lane (fp32 caches; read from the staging ring)
struct RowFragF32 {
  uint4 a, b;
  __device__ __forceinline__ void load(const unsigned char* row, int hl) {
    a = *reinterpret_cast<const uint4*>(row + 32 * hl); b = *reinterpret_cast<const uint4*>(row + 32 * hl + 16);
  }
  __device__ __forceinline__ void get(double* f) const {
    f[0] = __uint_as_float(a.x); f[1] = __uint_as_float(a.y); f[2] = __uint_as_float(a.z); f[3] = __uint_as_float(a.w);
    f[4] = __uint_as_float(b.x); f[5] = __uint_as_float(b.y); f[6] = __uint_as_float(b.z); f[7] = __uint_as_float(b.w);
  }
};

// Exact score key of one code from the query planes kept in shared memory (sign words, then mask planes).  Used
// only for the few keys whose stored 16-bit key equals the threshold when weighted scores need more than 16 bits;
// kept out of line so that its registers do not weigh on the loops that call it.
template <int W32, int NP>
__device__ __noinline__ int rescore_key(const uint32_t* code, const uint32_t* signw, const uint32_t (*mask)[8]) {
  uint32_t h[W32], sg[W32], mk[NP][W32];
#pragma unroll
  for (int w = 0; w < W32; ++w) {
    h[w] = code[w]; sg[w] = signw[w];
#pragma unroll
    for (int pl = 0; pl < NP; ++pl) mk[pl][w] = mask[pl][w];
  }
  return score_key<W32, NP>(h, sg, mk);
}

// VAR selects what is compiled in besides the plain path (VAR = 0): 1 = the error-aware safeguard (a static
// hard-to-hash set that is always attended); 2 = the streaming selection for units whose scores do not fit the
// cluster's shared memory (no score is stored: the scan keeps one histogram per warp over that warp's contiguous key
// range, and after the threshold is known every warp reads its codes a second time and emits its selection in order);
// 3 = byte score keys: Hamming scores with at most 256 distinct keys are stored one byte per key, unpadded, so that a
// block holds 2.5 times as many (contexts of a million keys and more in clusters that are all resident at once).
template <typename KV, int GP, int W32, int MODE, int VAR>
__global__ void __launch_bounds__((DecodeSmem<KV, GP, W32>::NT), 1)
bpc_decode_kernel(const DecodeParams p) {
  constexpr int EAS = VAR == 1 ? 1 : 0;
  constexpr bool STREAM = VAR == 2;
  constexpr bool K8 = VAR == 3;
  static_assert(!K8 || MODE == 0, "byte keys are for Hamming scores");
  typedef DecodeSmem<KV, GP, W32> L;
  typedef typename L::acc_t acc_t;
  constexpr int NT = L::NT, NW = L::NW, B = L::B;
  constexpr int NP = PlaneCount<GP, MODE>::value;
  // Hamming scores whose largest key fits one histogram bin per thread: only the one-pass threshold search is compiled
  constexpr bool kFastOnly = MODE == 0 && L::B * ((1 << NP) - 1) + 1 <= L::NT;
  constexpr int ROWB = L::kRowBytes;
  extern __shared__ __align__(16) unsigned char smem[];

  cg::cluster_group cluster = cg::this_cluster();
  const int CS = (int)cluster.num_blocks();
  const int rank = (int)cluster.block_rank();
  const int unit = blockIdx.x / CS;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = p.group;
  const int kvh = unit % p.n_kv_heads;
  const int seq = unit / p.n_kv_heads;

  // Programmatic dependent launch: when this grid was launched early (while its predecessor in the stream
  // was still running) nothing of the predecessor's output may be read before this point; afterwards the
  // successor's blocks may be scheduled as ours drain.  Both are no-ops for an ordinary launch.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // The rows of the projection are requested first of all after the dependency wait (the kernel before this one in
  // the stream may be the one that wrote them: bpc_fit, bpc_set_projection).
  constexpr int HPARTS = NT / B;                 // slices per projection row in the query hash
  constexpr int HDS = BPC_D / HPARTS;            // channels per slice (a multiple of 8)
  constexpr int HV = HDS * (int)sizeof(KV) / 16; // 16-byte vectors per slice
  uint4 prow[HV];
  {
    const int j = tid % B, part = tid / B;
    const uint4* row = reinterpret_cast<const uint4*>(reinterpret_cast<const KV*>(p.P_h) +
                                                      ((size_t)(p.shared_sets ? kvh : unit) * B + j) * BPC_D + part * HDS);
#pragma unroll
    for (int v = 0; v < HV; ++v) prow[v] = row[v];
  }

  // The queries do not depend on the sequence length: their loads overlap the length read and the set-up below.
  const KV* qg = reinterpret_cast<const KV*>(p.q) + ((size_t)seq * p.n_kv_heads + kvh) * (size_t)G * BPC_D;
  KV qreg[(GP * BPC_D + NT - 1) / NT];
#pragma unroll
  for (int v = 0; v < (GP * BPC_D + NT - 1) / NT; ++v) {
    const int i = tid + v * NT;
    qreg[v] = (i < GP * BPC_D && (i >> 7) < G) ? qg[i] : (KV)0.f;
  }

  int n = p.unit_lens[unit];
  n = max(0, min(n, p.n_max));
  // Fused cache write: this launch also appends one (k, v) row per unit at position n, codes it and counts it.
  bool fused = p.k_new != nullptr;
  if (fused && n >= p.n_max) {                               // full: nothing is written, the step runs on n keys
    if (tid == 0 && rank == 0) atomicOr(p.err, BPC_DEVERR_APPEND_CAP);
    fused = false;
  }
  if (fused) n += 1;
  long long kk = p.budget_count > 0 ? (long long)p.budget_count
                                    : ((long long)n * (long long)p.budget_ppm + 999999LL) / 1000000LL;
  if (kk < 0) kk = 0;
  const int k = (int)(kk < (long long)n ? kk : (long long)n);
  // Error-aware safeguard: the first `me` keys of the unit's static set S_err are always attended, the hash search
  // fills the remaining kh = k - me places.
  const int32_t* eas_u = nullptr;
  int me_rt = 0;
  if (EAS && p.eas_idx != nullptr) {
    me_rt = min(min(p.eas_cnt[unit], p.eas_cap), min(k, kEasMax));
    eas_u = p.eas_idx + (size_t)unit * p.eas_cap;
  }
  const int me = EAS ? me_rt : 0;                            // a compile-time zero without the safeguard
  const int kh = k - me;
  // Keys per block.  In a fused launch the appending block (the last one with keys) scans with one warp less, so
  // it is given a smaller share (bpc_fused_chunk).
  const int chunk = (fused && CS > 1) ? bpc_fused_chunk(n, CS) : (((n + CS - 1) / CS) + 63) & ~63;
  float* out_u = p.out + ((size_t)seq * p.n_kv_heads + kvh) * (size_t)G * BPC_D;

  // Both early exits depend only on values every block of the cluster sees identically, so either all
  // blocks of a cluster leave here (before any cluster barrier) or none does.
  if (!STREAM && chunk > p.chunk_cap) {
    if (tid == 0) atomicOr(p.err, BPC_DEVERR_CHUNK_CAP);
    return;
  }
  if (k == 0) {
    if (rank == 0)
      for (int o = tid; o < G * BPC_D; o += NT) out_u[o] = 0.f;
    return;
  }

  const int nbins = p.nbins;
  const int hsh = p.hist_shift;                              // histogram bin = score key >> hsh (0 in Hamming mode)
  const L plan(p.chunk_cap, nbins, p.stages, K8 ? 1 : 2);
  uint32_t* hist = reinterpret_cast<uint32_t*>(smem + plan.off_hist);
  uint32_t* tot = reinterpret_cast<uint32_t*>(smem + plan.off_tot);
  float* qf_s = reinterpret_cast<float*>(smem + plan.off_qf);
  double* pd = reinterpret_cast<double*>(smem + plan.off_pd);
  int32_t* idx_s = reinterpret_cast<int32_t*>(smem + plan.off_idx);
  // Inbox of the cluster-level merge: row r holds block r's partial sums for the outputs this block owns, then its
  // running maxima and denominators of all heads (peers store them here before the last cluster barrier).
  acc_t* inbox = reinterpret_cast<acc_t*>(smem + plan.off_cta);
  SmallState* st = reinterpret_cast<SmallState*>(smem + plan.off_small);
  unsigned char* uni = smem + plan.off_union;
  uint16_t* sc = reinterpret_cast<uint16_t*>(uni);
  [[maybe_unused]] uint8_t* sc8 = uni;                       // (byte-key variant: key i of the block at byte i)
  // Phase stamps (debug): slots 0 and 7 hold the global timer at block start and end, slots 15 and 14 the SM's cycle
  // counter at the same two points, every other slot the cycle counter (cheap to read) at that phase boundary.
#define BPC_STAMP(i) do { if (p.dbg_times != nullptr && tid == 0) p.dbg_times[(size_t)blockIdx.x * 16 + (i)] = (unsigned long long)clock64(); } while (0)
  if (p.dbg_times != nullptr && tid == 0) p.dbg_times[(size_t)blockIdx.x * 16] = global_timer_ns();
  BPC_STAMP(15);
  // the block whose key range holds the appended key (index n-1) does the append work in its last warp
  const bool appender = fused && rank == (n - 1) / chunk;

  // The appending block stages the Gram matrix in the part of the shared-memory union that the score keys do
  // not reach (free until the gather ring starts), so that the sequential sign decisions of Algorithm 2 cost a
  // shuffle and a few FMAs each.  Shapes where it does not fit read it from global memory instead.
  const float* gsm = nullptr;
  if (appender && p.residual_correction != 0) {
    const size_t union_bytes = plan.total - plan.off_union;
    const size_t score_bytes = STREAM ? (size_t)NW * nbins * 4      // (streaming: the per-warp histograms sit there)
                                      : L::score_bytes(p.chunk_cap, K8 ? 1 : 2);
    constexpr size_t kGramPad = 0;
    if (score_bytes + (size_t)B * B * 4 + kGramPad <= union_bytes && L::hashpart_bytes() + (size_t)B * B * 4 + kGramPad <= union_bytes) {
      float* dstg = reinterpret_cast<float*>(uni + union_bytes - (size_t)B * B * 4 - kGramPad);
      const float* Gs = p.gram + (size_t)(p.shared_sets ? kvh : unit) * B * B;
      for (int c = tid; c < B * B / 4; c += NT) cp_async16(dstg + 4 * c, Gs + 4 * c);
      gsm = dstg;
    }
  }
  cp_async_commit();

  // ---- scan set-up, hoisted above the query hash so that the first batch of codes is already in flight
  const int c0 = min(n, rank * chunk), c1 = min(n, c0 + chunk);
  // In the appending block the last warp codes the new key while the other warps scan; the new key's code is
  // not in memory yet, so the scan stops one key short and the key is scored separately below.
  const int nts = appender ? NT - 32 : NT;
  const int c1s = appender ? c1 - 1 : c1;
  const uint32_t* cu = reinterpret_cast<const uint32_t*>(p.codes) + (size_t)unit * (size_t)p.n_max * W32;
  int32_t* dbg = p.dbg_scores != nullptr ? p.dbg_scores + (size_t)unit * p.n_max : nullptr;
  // codes in flight per thread and buffer: the Hamming scan is bound by memory latency and wants many; the weighted
  // scan is bound by its arithmetic and scores a whole batch plane by plane (masks read from shared memory), so its
  // batch is as large as the registers for the codes and their carry words allow
  constexpr int U = MODE == 1 ? (W32 <= 1 ? 4 : W32 == 2 ? 8 : W32 == 4 ? 4 : 2) : (W32 <= 4 ? 8 : 4);
  auto load_code = [&](uint32_t (&h)[W32], int i) {
    const uint32_t* src = cu + (size_t)i * W32;
    if (W32 == 1) {
      h[0] = ld_stream_u32(src);
    } else if (W32 == 2) {
      const uint2 v = ld_stream_v2(src); h[0] = v.x; h[1] = v.y;
    } else {
#pragma unroll
      for (int w = 0; w < W32; w += 4) {
        const uint4 v = ld_stream_v4(src + w);
        h[w] = v.x; h[w + 1] = v.y; h[w + 2] = v.z; h[w + 3] = v.w;
      }
    }
  };
  auto load_batch = [&](uint32_t (&h)[U][W32], int base) {
#pragma unroll
    for (int u = 0; u < U; ++u) load_code(h[u], base + u * nts + tid);
  };
  uint32_t ha[U][W32], hb[U][W32];
  const bool pipelined = tid < nts && c0 + nts * U <= c1s;   // at least one full batch
  if (!STREAM && pipelined) load_batch(ha, c0);

  // ------------------------------------------------------------------ phase 0: query hash
  // p[g][j] = P_h[j] . q_g.  Thread (part, j) covers a slice of the 128 channels of row j: products are
  // summed eight at a time in fp32 (exact products for bf16 inputs) and the groups are added in fp64; the
  // slices are then added in fp64 in a fixed order.  Every block of the cluster gets identical bits.
#pragma unroll
  for (int v = 0; v < (GP * BPC_D + NT - 1) / NT; ++v) {
    const int i = tid + v * NT;
    if (i < GP * BPC_D) qf_s[i] = to_float(qreg[v]);
  }
  if (tid < BPC_D)                                           // slot GP: the appended key (its decision values P_h k)
    qf_s[GP * BPC_D + tid] = appender ? to_float(reinterpret_cast<const KV*>(p.k_new)[(size_t)unit * BPC_D + tid]) : 0.f;
  for (int i = tid; i < nbins; i += NT) hist[i] = 0u;
  if (tid < BPC_MAX_CLUSTER) { st->gt[tid] = 0u; st->eq[tid] = 0u; }
  if (tid == 0) { st->rsum = 0; st->T = 0; st->cnt_gt = 0; st->my_take = 0; st->my_base = 0; st->e0 = 0; st->e1 = 0; }
  // Safeguard keys inside this block's key range: the set is sorted, so their list positions [e0, e1) are the numbers
  // of entries below the range's two ends.  A set of at most kEasLocal keys is copied to shared memory asynchronously
  // now and searched after the hash (nothing needs e0, e1 before the selection); a larger one stays in global
  // memory and is counted by the whole block right away.
  const bool eas_local = EAS && me > 0 && me <= kEasLocal;
  if (eas_local) {
    for (int i = tid; i < me; i += NT) {
      const unsigned d = (unsigned)__cvta_generic_to_shared(&st->eas_s[i]);
      asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(d), "l"(eas_u + i) : "memory");
    }
    cp_async_commit();
  }
  __syncthreads();
  if (EAS && me > kEasLocal) {
    const int lo_key = min(n, rank * chunk), hi_key = min(n, lo_key + chunk);
    int c_lo = 0, c_hi = 0;
    for (int i = tid; i < me; i += NT) {
      const int v = eas_u[i];
      c_lo += v < lo_key;
      c_hi += v < hi_key;
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
      c_lo += __shfl_xor_sync(0xffffffffu, c_lo, o);
      c_hi += __shfl_xor_sync(0xffffffffu, c_hi, o);
    }
    if (lane == 0 && (c_lo | c_hi)) { atomicAdd(&st->e0, c_lo); atomicAdd(&st->e1, c_hi); }
  }
  {
    constexpr int PARTS = HPARTS, DS = HDS;
    const int j = tid % B, part = tid / B;
    constexpr int GV = L::GV;
    double acc[GV];
#pragma unroll
    for (int g = 0; g < GV; ++g) acc[g] = 0.0;
#pragma unroll
    for (int c0 = 0; c0 < DS; c0 += 8) {
      float pv[8];
      if (L::kMma) {
        const uint4 w = prow[c0 / 8];
        pv[0] = bf16_lo(w.x); pv[1] = bf16_hi(w.x); pv[2] = bf16_lo(w.y); pv[3] = bf16_hi(w.y);
        pv[4] = bf16_lo(w.z); pv[5] = bf16_hi(w.z); pv[6] = bf16_lo(w.w); pv[7] = bf16_hi(w.w);
      } else {
        const uint4 w0 = prow[c0 / 4], w1 = prow[c0 / 4 + 1];
        pv[0] = __uint_as_float(w0.x); pv[1] = __uint_as_float(w0.y); pv[2] = __uint_as_float(w0.z); pv[3] = __uint_as_float(w0.w);
        pv[4] = __uint_as_float(w1.x); pv[5] = __uint_as_float(w1.y); pv[6] = __uint_as_float(w1.z); pv[7] = __uint_as_float(w1.w);
      }
#pragma unroll
      for (int g = 0; g < GV; ++g) {
        const float4 q0 = *reinterpret_cast<const float4*>(qf_s + g * BPC_D + part * DS + c0);
        const float4 q1 = *reinterpret_cast<const float4*>(qf_s + g * BPC_D + part * DS + c0 + 4);
        float s0 = pv[0] * q0.x, s1 = pv[1] * q0.y;
        s0 = fmaf(pv[2], q0.z, s0); s1 = fmaf(pv[3], q0.w, s1);
        s0 = fmaf(pv[4], q1.x, s0); s1 = fmaf(pv[5], q1.y, s1);
        s0 = fmaf(pv[6], q1.z, s0); s1 = fmaf(pv[7], q1.w, s1);
        acc[g] += (double)s0 + (double)s1;
      }
    }
    double* hp = reinterpret_cast<double*>(uni);   // [PARTS][GV][B]
#pragma unroll
    for (int g = 0; g < GV; ++g) hp[((size_t)part * GV + g) * B + j] = acc[g];
    __syncthreads();
    for (int i = tid; i < GV * B; i += NT) {       // i = g * B + j
      double s = 0.0;
#pragma unroll
      for (int pt = 0; pt < PARTS; ++pt) s += hp[(size_t)pt * GV * B + i];
      pd[i] = s;
    }
  }
  __syncthreads();
  if (MODE == 1) {
    if (warp < G) {
      double mx = 0.0;
      for (int j = lane; j < B; j += 32) mx = fmax(mx, fabs(pd[warp * B + j]));
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      if (lane == 0) st->pmax[warp] = mx;
    }
    __syncthreads();
  }
  const int cs = (MODE == 0 && (G & 1) == 0) ? 1 : 0;      // common factor 2^cs of every |A_j|
  if (tid < B) {                                           // B is a multiple of 32: whole warps
    int A = 0;
    for (int g = 0; g < G; ++g) {
      const double pv = pd[g * B + tid];
      int a = 1;
      if (MODE == 1) {
        const double pm = st->pmax[g];
        a = pm > 0.0 ? (int)fmin(127.0, rint((127.0 * fabs(pv)) / pm)) : 0;
      }
      A += pv >= 0.0 ? a : -a;
    }
    const int absA = A < 0 ? -A : A;
    const uint32_t sw = __ballot_sync(0xffffffffu, A >= 0);
    if (lane == 0) st->signw[warp] = sw;
#pragma unroll
    for (int pl = 0; pl < NP; ++pl) {
      const uint32_t mw = __ballot_sync(0xffffffffu, (absA >> (pl + cs)) & 1);
      if (lane == 0) st->mask[pl][warp] = mw;
    }
    int rs = absA >> cs;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) rs += __shfl_xor_sync(0xffffffffu, rs, o);
    if (lane == 0) atomicAdd(&st->rsum, rs);
    if (p.dbg_qweights != nullptr && rank == 0) p.dbg_qweights[(size_t)unit * B + tid] = A;
  }
  cp_async_wait<0>();                                        // Gram staging (appending block only) has landed
  __syncthreads();
  // Weighted scores reach sum_j |A_j| <= 127 G b, which can exceed 16 bits (seven or eight query heads per KV head at
  // 128 bits, 256-bit codes).  The stored key is then the score key shifted right by ksh (0, 1 or 2, from this query's
  // own sum), the selection runs on the stored keys as before, and the keys whose stored key equals the threshold are
  // scored again from their codes to order them by the bits the shift dropped.
  int ksh = 0;
  if (MODE == 1) {
    const int rs = st->rsum;
    ksh = rs > 0xffff ? (rs > 0x1ffff ? 2 : 1) : 0;
    ksh = max(ksh, p.key_shift_min);
  }
  if (eas_local && (tid == 0 || tid == 32)) {                // lower bounds of the block's two range ends in the set
    const int lo_key = min(n, rank * chunk);
    const int bound = tid == 0 ? lo_key : min(n, lo_key + chunk);
    int a = 0, b2 = me;
    while (a < b2) {
      const int mid = (a + b2) >> 1;
      if (st->eas_s[mid] < bound) a = mid + 1; else b2 = mid;
    }
    if (tid == 0) st->e0 = a; else st->e1 = a;              // read after the cluster barrier that ends the scan
  }

  BPC_STAMP(1);
  // ------------------------------------------------------------------ phase 1: scan
  if (tid < nts) {
    // weighted scores of codes of two or more words: the plane masks stay in shared memory (score_keys_plane_outer)
    constexpr bool kPlaneOuter = MODE == 1 && W32 >= 2;
    uint32_t sg[W32], mk[kPlaneOuter ? 1 : NP][W32];
#pragma unroll
    for (int w = 0; w < W32; ++w) {
      sg[w] = st->signw[w];
      if constexpr (!kPlaneOuter) {
#pragma unroll
        for (int pl = 0; pl < NP; ++pl) mk[pl][w] = st->mask[pl][w];
      }
    }
    const int rfull = st->rsum << cs;                       // sum_j |A_j|
    auto score_batch = [&](const uint32_t (&h)[U][W32], int base) {
      if constexpr (kPlaneOuter) {
        int keys[U];
        score_keys_plane_outer<W32, NP, U>(h, sg, st->mask, keys);
#pragma unroll
        for (int u = 0; u < U; ++u) {
          sc[score_slot(base - c0 + u * nts + tid)] = (uint16_t)(keys[u] >> ksh);
          atomicAdd(&hist[(keys[u] >> ksh) >> hsh], 1u);
        }
      } else {
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int key = score_key<W32, NP>(h[u], sg, mk);
          if constexpr (K8) sc8[base - c0 + u * nts + tid] = (uint8_t)key;
          else sc[score_slot(base - c0 + u * nts + tid)] = (uint16_t)(key >> ksh);
          atomicAdd(&hist[(key >> ksh) >> hsh], 1u);
        }
      }
    };
    [[maybe_unused]] const int STEP = nts * U;
    if (dbg != nullptr) {                                    // score export (tests): a plain loop, one key at a time
#pragma unroll 1
      for (int i = c0 + tid; i < c1s; i += nts) {
        uint32_t h[W32];
        load_code(h, i);
        if constexpr (kPlaneOuter) dbg[i] = ((2 * rescore_key<W32, NP>(h, st->signw, st->mask)) << cs) - rfull;
        else dbg[i] = ((2 * score_key<W32, NP>(h, sg, mk)) << cs) - rfull;
      }
    }
    if constexpr (STREAM) {
      // Streaming selection, first pass: warp w owns the contiguous keys [w0, w1) and counts their score keys in its
      // own histogram (no score is stored).  A batch is U codes per lane, 32 keys apart.
      uint32_t* whist = reinterpret_cast<uint32_t*>(uni) + (size_t)warp * nbins;
      for (int i = lane; i < nbins; i += 32) whist[i] = 0u;
      __syncwarp();
      const int nw = nts >> 5;
      const int wlen = (((c1s - c0) + nw - 1) / nw + 31) & ~31;
      const int w0 = min(c1s, c0 + warp * wlen), w1 = min(c1s, w0 + wlen);
      constexpr int WSTEP = 32 * U;
      auto wload = [&](uint32_t (&h)[U][W32], int base) {    // indices past the range are clamped (their scores are dropped)
#pragma unroll
        for (int u = 0; u < U; ++u) load_code(h[u], min(base + 32 * u + lane, w1 - 1));
      };
      auto wcount = [&](const uint32_t (&h)[U][W32], int base) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int key = score_key<W32, NP>(h[u], sg, mk);
          if (base + 32 * u + lane < w1) atomicAdd(&whist[key], 1u);
        }
      };
      if (w0 < w1) wload(ha, w0);
#pragma unroll 1
      for (int base = w0; base < w1; base += 2 * WSTEP) {    // two register buffers: one batch in flight while one is scored
        if (base + WSTEP < w1) wload(hb, base + WSTEP);
        wcount(ha, base);
        if (base + WSTEP >= w1) break;
        if (base + 2 * WSTEP < w1) wload(ha, base + 2 * WSTEP);
        wcount(hb, base + WSTEP);
      }
    } else {
    int i0 = c0;
    if (pipelined) {
      // Full batches without bounds checks, software-pipelined over two register buffers so that the
      // loads of the next batch are in flight while the current one is scored (a warp's 32 keys share one
      // score segment).  The first batch was requested before the query hash.
#pragma unroll 1
      for (;;) {
        const bool more_b = i0 + 2 * STEP <= c1s;
        if (more_b) load_batch(hb, i0 + STEP);
        score_batch(ha, i0);
        i0 += STEP;
        if (!more_b) break;
        const bool more_a = i0 + 2 * STEP <= c1s;
        if (more_a) load_batch(ha, i0 + STEP);
        score_batch(hb, i0);
        i0 += STEP;
        if (!more_a) break;
      }
    }
    // ragged tail (less than one batch): the same batch with per-key bounds checks, loads in flight together
    if (i0 < c1s) {
      uint32_t h[U][W32];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = i0 + u * nts + tid;
        if (i < c1s) {
          load_code(h[u], i);
        } else {
#pragma unroll
          for (int w = 0; w < W32; ++w) h[u][w] = 0u;
        }
      }
      if constexpr (kPlaneOuter) {
        int keys[U];
        score_keys_plane_outer<W32, NP, U>(h, sg, st->mask, keys);
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int i = i0 + u * nts + tid;
          if (i < c1s) {
            sc[score_slot(i - c0)] = (uint16_t)(keys[u] >> ksh);
            atomicAdd(&hist[(keys[u] >> ksh) >> hsh], 1u);
          }
        }
      } else {
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int i = i0 + u * nts + tid;
          if (i < c1s) {
            const int key = score_key<W32, NP>(h[u], sg, mk);
            if constexpr (K8) sc8[i - c0] = (uint8_t)key;
            else sc[score_slot(i - c0)] = (uint16_t)(key >> ksh);
            atomicAdd(&hist[(key >> ksh) >> hsh], 1u);
          }
        }
      }
    }
    }
    if (p.dbg_times != nullptr && tid == 0) p.dbg_times[(size_t)blockIdx.x * 16 + 13] = (unsigned long long)clock64();
  } else {
    // ---- appending warp (Algorithm 2 on the new key, Gram form): cache rows, sign sweep, code words.
    // Lane l holds the decision values of bits l, 32+l, ...; bit i is decided by a shuffle from its owner
    // lane and every later column is corrected with G[i][.].
    const size_t rstride_e = (size_t)p.row_stride;
    const KV* kn = reinterpret_cast<const KV*>(p.k_new) + (size_t)unit * BPC_D;
    const KV* vn = reinterpret_cast<const KV*>(p.v_new) + (size_t)unit * BPC_D;
    KV* krow = reinterpret_cast<KV*>(p.k_cache_w) + ((size_t)unit * p.n_max + (n - 1)) * rstride_e;
    KV* vrow = reinterpret_cast<KV*>(p.v_cache_w) + ((size_t)unit * p.n_max + (n - 1)) * rstride_e;
    constexpr int CPL = ROWB / 16 / 16;                      // 16-byte chunks per lane and row (1 bf16, 2 fp32)
#pragma unroll
    for (int c = 0; c < CPL; ++c) {
      const int chn = (lane & 15) * CPL + c;
      if (lane < 16) reinterpret_cast<uint4*>(krow)[chn] = reinterpret_cast<const uint4*>(kn)[chn];
      else           reinterpret_cast<uint4*>(vrow)[chn] = reinterpret_cast<const uint4*>(vn)[chn];
    }
    constexpr int NB = W32;                                  // 32-bit column blocks
    float t[NB];
#pragma unroll
    for (int c = 0; c < NB; ++c) t[c] = (float)pd[GP * B + 32 * c + lane];
    const float* Gs = p.gram + (size_t)(p.shared_sets ? kvh : unit) * B * B;
    const bool rc = p.residual_correction != 0;
    uint32_t* code_dst = reinterpret_cast<uint32_t*>(p.codes_w) + ((size_t)unit * p.n_max + (n - 1)) * W32;
    if (p.dbg_times != nullptr && lane == 0) p.dbg_times[(size_t)blockIdx.x * 16 + 12] = (unsigned long long)clock64();
    {
      // The b sign decisions are taken eight at a time: every lane collects the eight
      // decision values of the group and decides them on its own copy (their 8 x 8 Gram block is read at one address
      // by the whole warp: no cross-lane traffic inside the dependency chain), then the eight signs correct all later
      // columns, one column per lane and 32-bit word.  Every value sees the same fp32 operations in the same order
      // as a one-bit-at-a-time sweep.
      // Two compilations of the same loops.  Unrolled in full, the word index is known at compile time, the corrections
      // of the words carry no run-time condition and the loads of all rows of a group are issued together instead of
      // one conditional block after the other (one warp alone: 7500 -> 3200 cycles for 128 bits); that is used when the
      // block's key range is short and the other warps would wait for this one.  With a long range the scan outlasts
      // the sweep anyway, and the rolled loops (a quarter of the code, a lower issue rate) disturb the scanning warps
      // of the block less (config 2: 39.6 us per step against 39.9).
      const float* gq = gsm != nullptr ? gsm : Gs;             // Gram matrix: staged in shared memory when it fits
      auto sweep = [&](auto unrolled_tag) {
      constexpr bool kUnrolled = decltype(unrolled_tag)::value;
#pragma unroll (kUnrolled ? NB : 1)
      for (int bi = 0; bi < NB; ++bi) {
        uint32_t wbits = 0u;
        if (!rc) {
          float tb = t[0];
#pragma unroll
          for (int c = 1; c < NB; ++c) tb = bi == c ? t[c] : tb;
          wbits = __ballot_sync(0xffffffffu, tb >= 0.f);
        } else {
#pragma unroll (kUnrolled ? 4 : 1)
          for (int sub = 0; sub < 4; ++sub) {
            float tb = t[0];
#pragma unroll
            for (int c = 1; c < NB; ++c) tb = bi == c ? t[c] : tb;
            float w[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) w[e] = __shfl_sync(0xffffffffu, tb, 8 * sub + e);
            const int r0 = 32 * bi + 8 * sub;
            const float* gd = gq + (size_t)r0 * B + r0;         // the group's 8 x 8 diagonal block
            float nu[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const bool pos = w[e] >= 0.f;
              wbits |= pos ? (1u << (8 * sub + e)) : 0u;
              nu[e] = pos ? -1.f : 1.f;
              const float4 g0 = *reinterpret_cast<const float4*>(gd + (size_t)e * B);
              const float4 g1 = *reinterpret_cast<const float4*>(gd + (size_t)e * B + 4);
              const float gr[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
              for (int f = e + 1; f < 8; ++f) w[f] = fmaf(nu[e], gr[f], w[f]);
            }
#pragma unroll
            for (int c = 0; c < NB; ++c) {
              if (c >= bi) {                                     // decided columns of word bi are corrected too: never read again
                const float* gc = gq + (size_t)r0 * B + 32 * c + lane;
#pragma unroll
                for (int e = 0; e < 8; ++e) t[c] = fmaf(nu[e], gc[(size_t)e * B], t[c]);
              }
            }
          }
        }
        if (lane == 0) { st->newcode[bi] = wbits; code_dst[bi] = wbits; }
      }
      };
      if (c1 - c0 < kUnrolledSweepKeys) sweep(std::true_type()); else sweep(std::false_type());
    }
    if (p.dbg_times != nullptr && lane == 0) p.dbg_times[(size_t)blockIdx.x * 16 + 11] = (unsigned long long)clock64();
  }
  int newkey = -1;                                           // streaming: score key of the key appended by this launch
  if constexpr (STREAM) {
    __syncthreads();                                         // every warp's histogram is complete (and the new code is known)
    if (appender) {
      uint32_t sg[W32], mk[NP][W32], h[W32];
#pragma unroll
      for (int w = 0; w < W32; ++w) {
        sg[w] = st->signw[w]; h[w] = st->newcode[w];
#pragma unroll
        for (int pl = 0; pl < NP; ++pl) mk[pl][w] = st->mask[pl][w];
      }
      newkey = score_key<W32, NP>(h, sg, mk);
      if (tid == 0 && p.dbg_scores != nullptr) p.dbg_scores[(size_t)unit * p.n_max + (n - 1)] = ((2 * newkey) << cs) - (st->rsum << cs);
    }
    const uint32_t* wh = reinterpret_cast<const uint32_t*>(uni);
    const int nw = nts >> 5;
    for (int bin = tid; bin < nbins; bin += NT) {
      uint32_t sum = bin == newkey ? 1u : 0u;
      for (int w = 0; w < nw; ++w) sum += wh[(size_t)w * nbins + bin];
      hist[bin] = sum;
    }
  }
  if (!STREAM && appender) {
    __syncthreads();                                         // the new code is in shared memory; the scan is done
    if (tid == 0) {
      uint32_t sg[W32], mk[NP][W32], h[W32];
#pragma unroll
      for (int w = 0; w < W32; ++w) {
        sg[w] = st->signw[w]; h[w] = st->newcode[w];
#pragma unroll
        for (int pl = 0; pl < NP; ++pl) mk[pl][w] = st->mask[pl][w];
      }
      const int key = score_key<W32, NP>(h, sg, mk);
      if constexpr (K8) sc8[n - 1 - c0] = (uint8_t)key;
      else sc[score_slot(n - 1 - c0)] = (uint16_t)(key >> ksh);
      atomicAdd(&hist[(key >> ksh) >> hsh], 1u);
      if (p.dbg_scores != nullptr) p.dbg_scores[(size_t)unit * p.n_max + (n - 1)] = ((2 * key) << cs) - (st->rsum << cs);
    }
  }

  BPC_STAMP(2);
  // ------------------------------------------------------------------ phase 2: threshold and ordered selection
  // With one bin per thread, every block first stores its finished histogram into a slot of every peer's shared memory
  // (behind the score keys), so that after the barrier all CS histograms are local reads.
  const bool fast_sel = kFastOnly || (nbins <= NT && hsh == 0);
  uint32_t* pushed = nullptr;
  {
    const size_t union_bytes = plan.total - plan.off_union;
    size_t push_off = STREAM ? (size_t)NW * nbins * 4 : L::score_bytes(p.chunk_cap, K8 ? 1 : 2);
    if (push_off < L::hashpart_bytes()) push_off = L::hashpart_bytes();   // a peer may still be hashing
    push_off = (push_off + 15) & ~(size_t)15;
    if (fast_sel && CS > 1 && push_off + (size_t)CS * nbins * 4 + (size_t)B * B * 4 <= union_bytes)
      pushed = reinterpret_cast<uint32_t*>(uni + push_off);
  }
  if (pushed != nullptr) {
    __syncthreads();                                         // this block's histogram is complete
    if (tid < nbins) {
      const uint32_t v = hist[tid];
#pragma unroll
      for (int r = 0; r < BPC_MAX_CLUSTER; ++r)
        if (r < CS) cluster.map_shared_rank(pushed, r)[rank * nbins + tid] = v;
    }
  }
  cluster.sync();                                            // every block's histogram is complete (and delivered)
  BPC_STAMP(8);
  const int e0 = (EAS && me > 0) ? st->e0 : 0, e1 = (EAS && me > 0) ? st->e1 : 0;
  if (appender && tid == 0) p.unit_lens_w[unit] = n;         // every block of the cluster has read the old length
  // Threshold key T (the k-th largest score key) and this block's share of the output.
  int T;
  int scan_calls = 0;                                        // block scans so far (selects their buffer)
  if (fast_sel) {
    // Common case, one histogram bin per thread: thread t owns bin nbins-1-t, reads that bin from every block of
    // the cluster (distributed shared memory) and a two-value block scan yields, for every bin, the number of keys
    // in higher bins (cluster-wide, and in the blocks of lower rank).  The thread whose bin holds the k-th key
    // then knows everything this block needs: T, how many ties it may take and where its output starts
    // (ties are granted to blocks in rank order, which is index order).
    const int bin = nbins - 1 - tid;
    uint32_t s_all = 0, s_low = 0, mine = 0;
    {
      const int bq = max(bin, 0);
      if (pushed != nullptr) {
#pragma unroll 1
        for (int r = 0; r < CS; ++r) {
          const uint32_t v = bin >= 0 ? pushed[r * nbins + bq] : 0u;
          s_all += v;
          if (r < rank) s_low += v;
          if (r == rank) mine = v;
        }
      } else {
#pragma unroll 1
        for (int r = 0; r < CS; ++r) {
          const uint32_t v = bin >= 0 ? cluster.map_shared_rank(hist, r)[bq] : 0u;
          s_all += v;
          if (r < rank) s_low += v;
          if (r == rank) mine = v;
        }
      }
    }
    uint32_t above_all, above_low;
    block_excl_scan2<NT>(s_all, s_low, st->wscan, scan_calls, above_all, above_low);
    if (bin >= 0 && above_all < (uint32_t)kh && above_all + s_all >= (uint32_t)kh) {
      const int need = kh - (int)above_all;                   // ties to take, cluster-wide (>= 1)
      const int lower_take = min(need, (int)s_low);          // ties granted to blocks of lower rank
      st->T = bin;
      st->cnt_gt = (int)above_all;
      st->my_take = min(max(need - (int)s_low, 0), (int)mine);
      st->my_base = (int)above_low + lower_take;
    }
    __syncthreads();
    T = st->T;
    BPC_STAMP(9);
  } else if constexpr (!kFastOnly) {
    // Total histogram through distributed shared memory.  With at most one bin per thread (the common case)
    // the per-block counts of that bin stay in registers and are reused for the per-block offsets below.
    const bool one_bin = nbins <= NT;
    uint32_t myv[BPC_MAX_CLUSTER];
#pragma unroll
    for (int r = 0; r < BPC_MAX_CLUSTER; ++r) myv[r] = 0u;
    if (one_bin) {
      if (tid < nbins) {
        uint32_t s = 0;
#pragma unroll
        for (int r = 0; r < BPC_MAX_CLUSTER; ++r)
          if (r < CS) { myv[r] = cluster.map_shared_rank(hist, r)[tid]; s += myv[r]; }
        tot[tid] = s;
      }
    } else {
      for (int bin = tid; bin < nbins; bin += NT) {
        uint32_t s = 0;
        for (int r = 0; r < CS; ++r) s += cluster.map_shared_rank(hist, r)[bin];
        tot[bin] = s;
      }
    }
    __syncthreads();
    {
      const int bpt = (nbins + NT - 1) / NT;                   // bins per thread; thread 0 owns the highest bins
      const int hi = nbins - tid * bpt;
      const int lo = max(0, hi - bpt);
      uint32_t local = 0;
      for (int bin = hi - 1; bin >= lo; --bin) local += tot[bin];
      uint32_t total;
      uint32_t above = block_excl_scan<NT>(local, st->wscan, scan_calls, &total);
      for (int bin = hi - 1; bin >= lo; --bin) {
        const uint32_t c = tot[bin];
        if (above < (uint32_t)kh && above + c >= (uint32_t)kh) { st->T = bin; st->cnt_gt = (int)above; }
        above += c;
      }
    }
    __syncthreads();
    T = st->T;
    BPC_STAMP(9);
    if (one_bin) {
      if (tid < nbins && tid >= T) {
#pragma unroll
        for (int r = 0; r < BPC_MAX_CLUSTER; ++r) {
          if (r < CS) {
            if (tid == T) st->eq[r] = myv[r];
            else if (myv[r]) atomicAdd(&st->gt[r], myv[r]);
          }
        }
      }
    } else {
      for (int bin = T + 1 + tid; bin < nbins; bin += NT) {
        if (tot[bin] == 0u) continue;
        for (int r = 0; r < CS; ++r) {
          const uint32_t v = cluster.map_shared_rank(hist, r)[bin];
          if (v) atomicAdd(&st->gt[r], v);
        }
      }
      if (tid < CS) st->eq[tid] = cluster.map_shared_rank(hist, tid)[T];
    }
    __syncthreads();
  }
  int T_exact = T;
  if (MODE == 1 && hsh > 0 && kh > 0) {
    // Weighted scores have more distinct values than histogram bins: the search above found the coarse bin
    // that holds the k-th score.  A second, small histogram over the low bits of the keys inside that bin (again
    // summed across the cluster) yields the exact threshold and corrects the per-block counts.
    const int FB = 1 << hsh;                                 // at most 32 fine bins
    uint32_t* fine = tot;
    if (tid < FB) fine[tid] = 0u;
    __syncthreads();
    {
      const int len = c1 - c0;
      for (int i = tid; i < len; i += NT) {
        const int key = (int)sc[score_slot(i)];
        if ((key >> hsh) == T) atomicAdd(&fine[key & (FB - 1)], 1u);
      }
    }
    cluster.sync();                                          // every block's fine histogram is complete
    if (warp == 0) {
      uint32_t fr[BPC_MAX_CLUSTER];
      uint32_t f = 0;
#pragma unroll
      for (int r = 0; r < BPC_MAX_CLUSTER; ++r) {
        fr[r] = (r < CS && lane < FB) ? cluster.map_shared_rank(fine, r)[lane] : 0u;
        f += fr[r];
      }
      // suffix sums over lanes: above = number of keys of the coarse bin with larger low bits
      uint32_t incl = f;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_down_sync(0xffffffffu, incl, o);
        if (lane + o < 32) incl += v;
      }
      const uint32_t above = incl - f;
      const uint32_t need_c = (uint32_t)(kh - st->cnt_gt);    // keys still to take from the coarse bin (>= 1)
      const bool mine = above < need_c && above + f >= need_c;
      const int vstar = __ffs(__ballot_sync(0xffffffffu, mine)) - 1;
      const uint32_t above_star = __shfl_sync(0xffffffffu, above, vstar);
#pragma unroll
      for (int r = 0; r < BPC_MAX_CLUSTER; ++r) {
        if (r < CS) {
          // per block: keys of the coarse bin strictly above the exact threshold, and ties at it
          uint32_t g = lane > vstar ? fr[r] : 0u;
#pragma unroll
          for (int o = 16; o >= 1; o >>= 1) g += __shfl_xor_sync(0xffffffffu, g, o);
          const uint32_t e = __shfl_sync(0xffffffffu, fr[r], vstar);
          if (lane == 0) { st->gt[r] += g; st->eq[r] = e; }
        }
      }
      if (lane == 0) { st->T = (T << hsh) | vstar; st->cnt_gt += (int)above_star; }
    }
    __syncthreads();
    T_exact = st->T;
  }
  // exact key of key i of this block's range (weighted scores with shifted keys only)
  auto exact_key = [&](int i) -> int {
    const bool is_new = fused && c0 + i == n - 1;            // the key appended by this launch: its code is in shared memory
    const uint32_t* code = is_new ? st->newcode : cu + (size_t)(c0 + i) * W32;
    return rescore_key<W32, NP>(code, st->signw, st->mask);
  };
  int T_low = 0;
  if (MODE == 1 && ksh > 0 && kh > 0) {
    // Stored keys are score keys shifted right by ksh: the class of stored keys equal to the threshold found above is
    // split once more by the dropped bits (2 or 4 values), from exact scores recomputed for the members of the class
    // (a handful of keys per block).  Same procedure as for the coarse bin: counts summed across the cluster, the
    // exact threshold, and the per-block numbers of keys above it and at it.
    const int FB = 1 << ksh;
    uint32_t* fine = st->wgt;                                // (32 words the weighted mode does not use otherwise; the array of the
                                                             //  previous level may still be read by a peer)
    if (tid < 32) fine[tid] = 0u;
    __syncthreads();
    {
      const int len = c1 - c0;
      for (int i = tid; i < len; i += NT)
        if ((int)sc[score_slot(i)] == T_exact) atomicAdd(&fine[exact_key(i) & (FB - 1)], 1u);
    }
    cluster.sync();
    if (warp == 0) {
      uint32_t fr[BPC_MAX_CLUSTER];
      uint32_t f = 0;
#pragma unroll
      for (int r = 0; r < BPC_MAX_CLUSTER; ++r) {
        fr[r] = (r < CS && lane < FB) ? cluster.map_shared_rank(fine, r)[lane] : 0u;
        f += fr[r];
      }
      uint32_t incl = f;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_down_sync(0xffffffffu, incl, o);
        if (lane + o < 32) incl += v;
      }
      const uint32_t above = incl - f;
      const uint32_t need_c = (uint32_t)(kh - st->cnt_gt);    // keys still to take from the class (>= 1)
      const bool mine = above < need_c && above + f >= need_c;
      const int vstar = __ffs(__ballot_sync(0xffffffffu, mine)) - 1;
      const uint32_t above_star = __shfl_sync(0xffffffffu, above, vstar);
#pragma unroll
      for (int r = 0; r < BPC_MAX_CLUSTER; ++r) {
        if (r < CS) {
          uint32_t g = lane > vstar ? fr[r] : 0u;
#pragma unroll
          for (int o = 16; o >= 1; o >>= 1) g += __shfl_xor_sync(0xffffffffu, g, o);
          const uint32_t e = __shfl_sync(0xffffffffu, fr[r], vstar);
          if (lane == 0) { st->gt[r] += g; st->eq[r] = e; }
        }
      }
      if (lane == 0) { st->e0 = vstar; st->cnt_gt += (int)above_star; }   // (e0 is free here: the safeguard is Hamming-only)
    }
    __syncthreads();
    T_low = st->e0;
  }
  if (!kFastOnly && !fast_sel && tid == 0) {
    const int need = kh - st->cnt_gt;                        // ties to take, cluster-wide (>= 1)
    int tie_base = 0, out_base = 0;
    for (int r = 0; r < CS; ++r) {
      int take = need - tie_base;
      take = take < 0 ? 0 : (take > (int)st->eq[r] ? (int)st->eq[r] : take);
      if (r == rank) { st->my_take = take; st->my_base = out_base; }
      out_base += (int)st->gt[r] + take;
      tie_base += (int)st->eq[r];
    }
  }
  if (!kFastOnly && !fast_sel) __syncthreads();                            // (the fast path published its values before its own barrier)
  int32_t* sel_u = p.sel + (size_t)unit * p.n_max;
  BPC_STAMP(10);
  if constexpr (STREAM) {
    // Streaming selection, second pass.  Per-warp numbers of keys above and at the threshold come from the warps'
    // histograms; a warp's output starts after the keys of the warps before it (ties are granted in warp order, which
    // is index order), and inside the warp one ballot per 32 keys keeps the order.
    const int my_take = st->my_take, my_base = st->my_base, Tk = T_exact;
    const uint32_t* whist = reinterpret_cast<const uint32_t*>(uni) + (size_t)warp * nbins;
    const int nw = nts >> 5;
    if (tid < nts) {
      uint32_t g = 0;
      for (int bin = Tk + 1 + lane; bin < nbins; bin += 32) g += whist[bin];
      g = __reduce_add_sync(0xffffffffu, g);
      if (lane == 0) { st->wgt[warp] = g; st->weq[warp] = whist[Tk]; }
    }
    __syncthreads();
    if (tid < nts && kh > 0) {
      int gt_before = 0, eq_before = 0;
      for (int w = 0; w < warp; ++w) { gt_before += (int)st->wgt[w]; eq_before += (int)st->weq[w]; }
      const int take_w = min(max(my_take - eq_before, 0), (int)st->weq[warp]);
      int pos = my_base + gt_before + min(eq_before, my_take);
      int run_eq = 0;
      uint32_t sg[W32], mk[NP][W32];
#pragma unroll
      for (int w = 0; w < W32; ++w) {
        sg[w] = st->signw[w];
#pragma unroll
        for (int pl = 0; pl < NP; ++pl) mk[pl][w] = st->mask[pl][w];
      }
      const int wlen = (((c1s - c0) + nw - 1) / nw + 31) & ~31;
      const int w0 = min(c1s, c0 + warp * wlen), w1 = min(c1s, w0 + wlen);
      const uint32_t lt = (1u << lane) - 1u;
      constexpr int WSTEP = 32 * U;
      auto wload = [&](uint32_t (&h)[U][W32], int base) {
#pragma unroll
        for (int u = 0; u < U; ++u) load_code(h[u], min(base + 32 * u + lane, w1 - 1));
      };
      auto wemit = [&](const uint32_t (&h)[U][W32], int base) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int i = base + 32 * u + lane;
          const int key = score_key<W32, NP>(h[u], sg, mk);
          const bool valid = i < w1;
          const uint32_t be = __ballot_sync(0xffffffffu, valid && key == Tk);
          const bool takes = valid && (key > Tk || (key == Tk && run_eq + __popc(be & lt) < take_w));
          const uint32_t bs = __ballot_sync(0xffffffffu, takes);
          if (takes) sel_u[pos + __popc(bs & lt)] = i;
          pos += __popc(bs);
          run_eq += __popc(be);
        }
      };
      if (w0 < w1) wload(ha, w0);
#pragma unroll 1
      for (int base = w0; base < w1; base += 2 * WSTEP) {
        if (base + WSTEP < w1) wload(hb, base + WSTEP);
        wemit(ha, base);
        if (base + WSTEP >= w1) break;
        if (base + 2 * WSTEP < w1) wload(ha, base + 2 * WSTEP);
        wemit(hb, base + WSTEP);
      }
    }
    if (appender && tid == 0 && kh > 0) {                    // the appended key is the last key of this block's range
      int gt_all = 0, eq_all = 0;
      for (int w = 0; w < nw; ++w) { gt_all += (int)st->wgt[w]; eq_all += (int)st->weq[w]; }
      if (newkey > Tk || (newkey == Tk && eq_all < my_take)) sel_u[my_base + gt_all + min(eq_all, my_take)] = n - 1;
    }
  } else {
    // Each thread owns whole 32-key segments, in ascending order within a pass.  Two keys share a 32-bit
    // word; adding (0x8000 - T) to both halves raises bit 15 / bit 31 exactly for keys >= T (keys < 2048),
    // which is shifted into a 32-bit candidate mask without branches.  Only the few candidates are looked
    // at again (re-read from shared memory) to tell "greater" from "tie".
    const int len = c1 - c0;
    const int nseg = (len + kSegKeys - 1) / kSegKeys;
    const int my_take = st->my_take;
    const int T = T_exact;                                   // shadows the coarse bin: from here on the exact key
    const uint32_t cge = (uint32_t)(0x8000 - T) * 0x10001u;
    constexpr int SPT = 4;                                   // most consecutive segments one thread takes per pass
    const int spt = min(SPT, (nseg + NT - 1) / NT);
    int run_gt = 0, run_eq = 0;
    // With the safeguard, every thread also leaves the mask of the keys it selected in the padding of each of its
    // segments (slots 32, 33), where the safeguard keys of this block look themselves up afterwards: a key chosen
    // by both sources is attended once.
    for (int s0 = 0; s0 < nseg && kh > 0; s0 += NT * spt) {
      uint32_t M[SPT], Mgt[SPT];                             // bit j: key j of the segment is >= T / > T
      int cgt = 0, ceq = 0;
#pragma unroll
      for (int q = 0; q < SPT; ++q) {
        M[q] = 0u; Mgt[q] = 0u;
        const int seg = s0 + tid * spt + q;
        if (q < spt && seg < nseg) {
          uint32_t kw[16];
          if constexpr (K8) {                                // 32 byte keys: two 16-byte reads
            const uint4* src = reinterpret_cast<const uint4*>(sc8 + (size_t)seg * kSegKeys);
#pragma unroll
            for (int v = 0; v < 2; ++v) {
              const uint4 x = src[v];
              kw[4 * v] = x.x; kw[4 * v + 1] = x.y; kw[4 * v + 2] = x.z; kw[4 * v + 3] = x.w;
            }
          } else {
          const uint4* src = reinterpret_cast<const uint4*>(sc + (size_t)seg * kSegSlots);
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            const uint4 x = src[v];
            kw[4 * v] = x.x; kw[4 * v + 1] = x.y; kw[4 * v + 2] = x.z; kw[4 * v + 3] = x.w;
          }
          }
          uint32_t m = 0;
          if constexpr (K8) {
            // four keys per word: a per-byte unsigned compare leaves 0xFF where key >= T; one multiplication moves the
            // four flags (bits 0, 8, 16, 24 after masking) next to each other: (y * 0x01020408) >> 24
            const uint32_t T4 = (uint32_t)T * 0x01010101u;
#pragma unroll
            for (int w = 0; w < 8; ++w) {
              const uint32_t ge = __vcmpgeu4(kw[w], T4) & 0x01010101u;
              m |= (((ge * 0x01020408u) >> 24) & 15u) << (4 * w);
            }
          } else {
#pragma unroll
          for (int w = 0; w < 16; ++w) {
            if (MODE == 0) {                                 // keys < 2048: both halves compared with one addition
              const uint32_t gq = kw[w] + cge;
              m |= (2 * w <= 15 ? (gq >> (15 - 2 * w)) : (gq << (2 * w - 15))) & (1u << (2 * w));
              m |= (gq >> (30 - 2 * w)) & (2u << (2 * w));
            } else {                                         // keys up to 65535: compare the halves separately
              m |= ((int)(kw[w] & 0xffffu) >= T ? 1u : 0u) << (2 * w);
              m |= ((int)(kw[w] >> 16) >= T ? 2u : 0u) << (2 * w);
            }
          }
          }
          const int valid = len - seg * kSegKeys;
          if (valid < kSegKeys) m &= (1u << valid) - 1u;     // slots past the end of the chunk hold stale bytes
          uint32_t rem = m, mg = 0;
          while (rem) {
            const int j = __ffs(rem) - 1;
            rem &= rem - 1;
            if constexpr (K8) {
              if ((int)sc8[(size_t)seg * kSegKeys + j] > T) mg |= 1u << j;
            } else
            if ((int)sc[(size_t)seg * kSegSlots + j] > T) mg |= 1u << j;
            else if (MODE == 1 && ksh > 0) {                 // stored key == threshold: the dropped bits decide
              const int low = exact_key(seg * kSegKeys + j) & ((1 << ksh) - 1);
              if (low > T_low) mg |= 1u << j;
              else if (low < T_low) m &= ~(1u << j);
            }
          }
          M[q] = m; Mgt[q] = mg;
          cgt += __popc(mg);
          ceq += __popc(m) - __popc(mg);
        }
      }
      uint32_t total;
      const uint32_t ex = block_excl_scan<NT>((uint32_t)cgt | ((uint32_t)ceq << 16), st->wscan, scan_calls, &total);
      uint32_t TK[SPT];                                      // bit j: key j of the segment was selected
#pragma unroll
      for (int q = 0; q < SPT; ++q) TK[q] = 0u;
      if (cgt | ceq) {
        int eqb = run_eq + (int)(ex >> 16);
        int pos = st->my_base + run_gt + (int)(ex & 0xffffu) + min(eqb, my_take);
#pragma unroll
        for (int q = 0; q < SPT; ++q) {
          const int seg = s0 + tid * spt + q;
          uint32_t rem = M[q];
          while (rem) {
            const int j = __ffs(rem) - 1;
            rem &= rem - 1;
            const int gi = c0 + seg * kSegKeys + j;
            bool takes = true;
            if (!((Mgt[q] >> j) & 1u)) { takes = eqb < my_take; ++eqb; }
            if (takes) {
              sel_u[pos++] = gi;
              if (EAS) TK[q] |= 1u << j;
            }
          }
        }
      }
      if (EAS && me > 0) {
#pragma unroll
        for (int q = 0; q < SPT; ++q) {
          const int seg = s0 + tid * spt + q;
          if (q < spt && seg < nseg) *reinterpret_cast<uint32_t*>(sc + (size_t)seg * kSegSlots + kSegKeys) = TK[q];
        }
      }
      run_gt += (int)(total & 0xffffu);
      run_eq += (int)(total >> 16);
    }
  }
  // this block attends rows [lo, hi) of the hash list and the safeguard keys that lie in its own key range
  const int lo = (int)(((unsigned)kh * (unsigned)rank) / (unsigned)CS), hi = (int)(((unsigned)kh * (unsigned)(rank + 1)) / (unsigned)CS);   // kh * 16 < 2^31
  const int nh = hi - lo, ne = e1 - e0;                      // rows from the two sources
  if (me > 0) {
    __syncthreads();                                         // the selection masks of this block are written
    for (int t = tid; t < e1 - e0; t += NT) {
      const int v = eas_local ? st->eas_s[e0 + t] : eas_u[e0 + t];
      const int rel = v - c0;                                // the key's position in this block's range
      const bool dup = kh > 0 && ((*reinterpret_cast<const uint32_t*>(sc + (size_t)(rel >> 5) * kSegSlots + kSegKeys) >> (rel & 31)) & 1u);
      sel_u[kh + e0 + t] = dup ? -1 : v;
    }
  }
  BPC_STAMP(3);
  cluster.sync();                                            // release/acquire at cluster scope: the unit's index list
                                                             // (global memory, written by all blocks) is complete and visible
  BPC_STAMP(4);

  // ------------------------------------------------------------------ phase 3: gathered attention
  // The list was written by other SMs during this launch: it is read at L2 (ld.global.cg), never through this SM's L1.
  auto row_index = [&](int qrow) -> int {                    // qrow in [0, nh + ne): cache row, or -1 for a duplicate
    if (!EAS) return __ldcg(sel_u + lo + qrow);
    return qrow < nh ? __ldcg(sel_u + lo + qrow) : __ldcg(sel_u + kh + e0 + (qrow - nh));
  };
  const size_t rstride = (size_t)p.row_stride * sizeof(KV);   // bytes between consecutive cache rows
  const unsigned char* Ku = reinterpret_cast<const unsigned char*>(p.k_cache) + (size_t)unit * (size_t)p.n_max * rstride;
  const unsigned char* Vu = reinterpret_cast<const unsigned char*>(p.v_cache) + (size_t)unit * (size_t)p.n_max * rstride;
  constexpr int TR = L::kTileRows, CPR = ROWB / 16;
  const int NS = p.stages;
  unsigned char* stg = uni;
  acc_t* part = reinterpret_cast<acc_t*>(uni);               // [NW][GP][130]; aliases the ring (used after it)
  const float scale2 = (float)(p.sm_scale_d * 1.4426950408889634);   // logits in base-2 exponent units

  if constexpr (L::kMma) {
    // ---- bf16: tensor-core path.  Warp w owns rows 8w..8w+7 of every tile.
    //   S^T[head][key] = Q (16 x 128, rows >= G zero) . K_tile^T : 8 MMAs m16n8k16 per 8 keys
    //   O[head][dim]  += P (16 x 8; rows 0-7 = bf16(p), rows 8-15 = bf16(p - bf16(p))) . V_tile : 16 MMAs m16n8k8
    // Lane (g = lane/4, t = lane%4) holds the logits of head g for keys 2t, 2t+1 and, in every 8-dim output
    // tile, dims 2t, 2t+1 of head g (high part in d[0..1], low part in d[2..3]).
    const int g = lane >> 2, t = lane & 3;
    uint32_t qa0[8], qa2[8];
    {
      const uint32_t* qw = reinterpret_cast<const uint32_t*>(qg + (size_t)g * BPC_D);
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        qa0[s] = g < G ? qw[8 * s + t] : 0u;                 // dims 16s + 2t, +1
        qa2[s] = g < G ? qw[8 * s + 4 + t] : 0u;             // dims 16s + 8 + 2t, +1
      }
    }
    float o[16][4];
#pragma unroll
    for (int j = 0; j < 16; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
    float m_run = -1e30f, l_run = 0.f;
    const int lrow = lane & 7, lmat = lane >> 3;             // ldmatrix: lane supplies row lrow of matrix lmat

    // Every warp runs its own gather ring (no block barriers): it owns the 8-row blocks warp, warp+NW, ... of
    // the block's slice, copies a block's K and V rows with one 16-byte asynchronous copy per lane and row
    // (lanes 0-15 the K row, lanes 16-31 the V row; chunks XOR-swizzled by the row number so that ldmatrix
    // reads are conflict-free), keeps NS-1 blocks in flight and multiplies the oldest one.
    constexpr int WSTG = 8 * 2 * ROWB;                       // bytes of one 8-row stage (K rows, then V rows)
    unsigned char* wst = stg + (size_t)warp * NS * WSTG;
    // the block's rows are split evenly over the warps (contiguous ranges; the last 8-row block of a warp may be short)
    const int nrows_b = nh + ne;
    const int r0w = (int)(((long long)nrows_b * warp) / NW), r1w = (int)(((long long)nrows_b * (warp + 1)) / NW);
    const int nrows = r1w - r0w;
    const int nblk = (nrows + 7) >> 3;
    const int isv = lane >> 4, ch = lane & 15;
    const unsigned char* srcbase = (isv ? Vu : Ku) + (size_t)ch * 16;
    // a warp's first 64 list entries are fetched once (one coalesced read), later ones block by block
    int pre0 = -1, pre1 = -1;
    if (lane < nrows) pre0 = row_index(r0w + lane);
    if (32 + lane < nrows) pre1 = row_index(r0w + 32 + lane);
    auto issue = [&](int bi) {
      if (bi < nblk) {
        const int rbase = 8 * bi;
        int myidx = -1;
        if (bi < 8) {                                        // warp-uniform
          const int v = __shfl_sync(0xffffffffu, bi < 4 ? pre0 : pre1, (rbase & 31) + (lane & 7));
          if (lane < 8) myidx = v;
        } else if (lane < 8 && rbase + lane < nrows) {
          myidx = row_index(r0w + rbase + lane);
        }
        if (myidx >= 0) myidx = min(myidx, p.n_max - 1);
        if (EAS) {   // which of the 8 rows are real (not past the end, not a duplicate of a hash-selected key)
          const uint32_t vm = __ballot_sync(0xffffffffu, myidx >= 0) & 0xffu;
          if (lane == 0) st->stage_valid[warp][bi % NS] = (uint8_t)vm;
        }
        unsigned char* dst = wst + (size_t)(bi % NS) * WSTG + (size_t)isv * (8 * ROWB);
#pragma unroll
        for (int it = 0; it < 8; ++it) {
          const int idx = __shfl_sync(0xffffffffu, myidx, it);
          unsigned char* d = dst + it * ROWB + ((ch ^ it) << 4);
          if (idx >= 0) {
            cp_async16(d, srcbase + (size_t)idx * rstride);
          } else {
            // rows past the end of the list get zeros: their probabilities are zero, and 0 * stale NaN
            // must not reach the accumulators
            *reinterpret_cast<uint4*>(d) = make_uint4(0u, 0u, 0u, 0u);
          }
        }
      }
      cp_async_commit();
    };
    for (int tt = 0; tt < NS; ++tt) issue(tt);              // every stage of the ring starts in flight
    for (int bi = 0; bi < nblk; ++bi) {
      if (NS == 2) cp_async_wait<1>(); else cp_async_wait<2>();   // this lane's copies for block bi have landed
      __syncwarp();                                          // ... and every lane's
      const int rbase_c = 8 * bi;
      const uint32_t vmask = EAS ? (uint32_t)st->stage_valid[warp][bi % NS]
                                 : (rbase_c + 8 <= nrows ? 0xffu : ((1u << (nrows - rbase_c)) - 1u));
      const unsigned char* ks = wst + (size_t)(bi % NS) * WSTG;
      const unsigned char* vs = ks + 8 * ROWB;
      float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {                       // 32 dims per ldmatrix.x4: chunks 4jj .. 4jj+3
        uint32_t b[4];
        ldmatrix_x4(b, ks + (size_t)lrow * ROWB + (((4 * jj + lmat) ^ lrow) << 4));
        mma_qk(s, qa0[2 * jj], qa2[2 * jj], b[0], b[1]);
        mma_qk(s, qa0[2 * jj + 1], qa2[2 * jj + 1], b[2], b[3]);
      }
      const bool v0 = (vmask >> (2 * t)) & 1u, v1 = (vmask >> (2 * t + 1)) & 1u;
      const float s0 = v0 ? s[0] * scale2 : -1e30f, s1 = v1 ? s[1] * scale2 : -1e30f;
      float tmax = fmaxf(s0, s1);
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
      if (__any_sync(0xffffffffu, tmax > m_run)) {
        if (tmax > m_run) {
          const float corr = exp2f(m_run - tmax);
          l_run *= corr;
#pragma unroll
          for (int j = 0; j < 16; ++j) { o[j][0] *= corr; o[j][1] *= corr; o[j][2] *= corr; o[j][3] *= corr; }
          m_run = tmax;
        }
      }
      const float p0 = v0 ? exp2f(s0 - m_run) : 0.f, p1 = v1 ? exp2f(s1 - m_run) : 0.f;
      l_run += p0 + p1;
      const __nv_bfloat162 hi2 = __floats2bfloat162_rn(p0, p1);
      const float r0f = p0 - __low2float(hi2), r1f = p1 - __high2float(hi2);
      const uint32_t pa0 = *reinterpret_cast<const uint32_t*>(&hi2);
      const uint32_t pa1 = pack_bf16x2(r0f, r1f);
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        uint32_t b[4];
        ldmatrix_x4_trans(b, vs + (size_t)lrow * ROWB + (((4 * jj + lmat) ^ lrow) << 4));
        mma_pv(o[4 * jj], pa0, pa1, b[0]);
        mma_pv(o[4 * jj + 1], pa0, pa1, b[1]);
        mma_pv(o[4 * jj + 2], pa0, pa1, b[2]);
        mma_pv(o[4 * jj + 3], pa0, pa1, b[3]);
      }
      __syncwarp();                                          // every lane is done with this stage:
      issue(bi + NS);                                        // refill it
    }
    cp_async_wait<0>();
    // lanes of one head (same g) hold partial sums of l over their keys
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    __syncthreads();                                         // the ring is no longer read: reuse it for the merge
    if (g < GP) {
      acc_t* dst = part + ((size_t)warp * GP + g) * (BPC_D + 2);
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        dst[8 * j + 2 * t] = o[j][0] + o[j][2];
        dst[8 * j + 2 * t + 1] = o[j][1] + o[j][3];
      }
      if (t == 0) { dst[BPC_D] = m_run; dst[BPC_D + 1] = l_run; }
    }
  } else {
    // ---- fp32 caches: fp64 logits and averages on the CUDA cores, half a warp per row
    const int hl = lane & 15, half = lane >> 4;
    acc_t qf[GP][8], acc[GP][8], m_run[GP], l_run[GP];
#pragma unroll
    for (int gg = 0; gg < GP; ++gg) {
#pragma unroll
      for (int c = 0; c < 8; ++c) { qf[gg][c] = (acc_t)qf_s[gg * BPC_D + 8 * hl + c] * (acc_t)(p.sm_scale_d * 1.4426950408889634); acc[gg][c] = (acc_t)0; }
      m_run[gg] = (acc_t)-1e30; l_run[gg] = (acc_t)0;
    }
    auto process = [&](const RowFragF32& kf, const RowFragF32& vf, bool valid) {
      acc_t kv8[8], s[GP];
      kf.get(kv8);
#pragma unroll
      for (int gg = 0; gg < GP; ++gg) {
        acc_t d = qf[gg][0] * kv8[0];
#pragma unroll
        for (int c = 1; c < 8; ++c) d = fma(qf[gg][c], kv8[c], d);
        s[gg] = d;
      }
#pragma unroll
      for (int o = 8; o >= 1; o >>= 1) {
#pragma unroll
        for (int gg = 0; gg < GP; ++gg) s[gg] += __shfl_xor_sync(0xffffffffu, s[gg], o);
      }
      if (valid) {                                           // rows past the tile's end hold stale bytes
#pragma unroll
        for (int gg = 0; gg < GP; ++gg) {
          if (s[gg] > m_run[gg]) {
            const acc_t corr = fast_exp2<acc_t>(m_run[gg] - s[gg]);
            l_run[gg] *= corr;
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[gg][c] *= corr;
            m_run[gg] = s[gg];
          }
        }
        vf.get(kv8);
#pragma unroll
        for (int gg = 0; gg < GP; ++gg) {
          const acc_t pr = fast_exp2<acc_t>(s[gg] - m_run[gg]);
          l_run[gg] += pr;
#pragma unroll
          for (int c = 0; c < 8; ++c) acc[gg][c] = fma(pr, kv8[c], acc[gg][c]);
        }
      }
    };
    for (int t0 = 0; t0 < nh + ne; t0 += kIdxTile) {         // virtual rows: hash slice, then own safeguard keys
      const int tn = min(kIdxTile, nh + ne - t0);
      __syncthreads();
      for (int i = tid; i < tn; i += NT) {
        const int v = row_index(t0 + i);
        idx_s[i] = v < 0 ? -1 : min(v, p.n_max - 1);
      }
      __syncthreads();
      const int ntile = (tn + TR - 1) / TR;
      auto issue = [&](int tile) {
        if (tile < ntile) {
          unsigned char* dst = stg + (size_t)(tile % NS) * L::kStageBytes;
          const int r0 = tile * TR;
          for (int c = tid; c < TR * 2 * CPR; c += NT) {
            const int row = c / (2 * CPR), within = c % (2 * CPR);
            const int isv = within / CPR, ch = within % CPR;
            if (r0 + row < tn && idx_s[r0 + row] >= 0) {
              const size_t off = (size_t)idx_s[r0 + row] * rstride + (size_t)ch * 16;
              cp_async16(dst + (size_t)row * 2 * ROWB + isv * ROWB + ch * 16, (isv ? Vu : Ku) + off);
            }
          }
        }
        cp_async_commit();
      };
      for (int tt = 0; tt < NS - 1; ++tt) issue(tt);
      for (int tile = 0; tile < ntile; ++tile) {
        if (NS == 2) cp_async_wait<0>(); else cp_async_wait<1>();
        __syncthreads();
        issue(tile + NS - 1);
        const unsigned char* src = stg + (size_t)(tile % NS) * L::kStageBytes;
        const int r0 = tile * TR;
        for (int rp = warp; 2 * rp < TR; rp += NW) {
          const int r = 2 * rp + half;
          RowFragF32 kf, vf;
          kf.load(src + (size_t)r * 2 * ROWB, hl);
          vf.load(src + (size_t)r * 2 * ROWB + ROWB, hl);
          process(kf, vf, r0 + r < tn && idx_s[r0 + r] >= 0);
        }
      }
      cp_async_wait<0>();
    }
    // merge the two half warps
#pragma unroll
    for (int gg = 0; gg < GP; ++gg) {
      const acc_t om = __shfl_xor_sync(0xffffffffu, m_run[gg], 16);
      const acc_t ol = __shfl_xor_sync(0xffffffffu, l_run[gg], 16);
      const acc_t mm = om > m_run[gg] ? om : m_run[gg];
      const acc_t ws = fast_exp2<acc_t>(m_run[gg] - mm), wo = fast_exp2<acc_t>(om - mm);
      l_run[gg] = l_run[gg] * ws + ol * wo;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const acc_t oa = __shfl_xor_sync(0xffffffffu, acc[gg][c], 16);
        acc[gg][c] = acc[gg][c] * ws + oa * wo;
      }
      m_run[gg] = mm;
    }
    __syncthreads();                                         // the ring is no longer read: reuse it for the merge
    if (half == 0) {
#pragma unroll
      for (int gg = 0; gg < GP; ++gg) {
        acc_t* dst = part + ((size_t)warp * GP + gg) * (BPC_D + 2);
#pragma unroll
        for (int c = 0; c < 8; ++c) dst[8 * hl + c] = acc[gg][c];
        if (hl == 0) { dst[BPC_D] = m_run[gg]; dst[BPC_D + 1] = l_run[gg]; }
      }
    }
  }
  BPC_STAMP(5);
  __syncthreads();
  // Block-level merge of the warps' partials; every result goes straight to the block of the cluster that owns that
  // output (outputs are split evenly over the ranks), its maximum and denominator to every block.
  const int nout = G * BPC_D;
  const int per = (nout + CS - 1) / CS;                      // outputs owned by one rank
  const int istride = per + 2 * GP;                          // one inbox row
  for (int o = tid; o < GP * BPC_D; o += NT) {
    const int g = o >> 7, d = o & 127;
    acc_t mm = (acc_t)-1e30;
    for (int w = 0; w < NW; ++w) {
      const acc_t v = part[((size_t)w * GP + g) * (BPC_D + 2) + BPC_D];
      mm = v > mm ? v : mm;
    }
    acc_t num = 0, den = 0;
    for (int w = 0; w < NW; ++w) {
      const acc_t* src = part + ((size_t)w * GP + g) * (BPC_D + 2);
      const acc_t wt = fast_exp2<acc_t>(src[BPC_D] - mm);
      num = fma(src[d], wt, num);
      den = fma(src[BPC_D + 1], wt, den);
    }
    if (o < nout) {
      const int owner = o / per;
      cluster.map_shared_rank(inbox, owner)[rank * istride + (o - owner * per)] = num;
    }
    if (d == 0 && g < G) {
#pragma unroll 1
      for (int r = 0; r < CS; ++r) {
        acc_t* row = cluster.map_shared_rank(inbox, r) + rank * istride + per;
        row[g] = mm;
        row[GP + g] = den;
      }
    }
  }
  BPC_STAMP(6);
  cluster.sync();                                            // every block's partial results have been delivered
  {
    // cluster-level merge of the outputs this block owns, from its own shared memory; nothing remote is read after
    // the barrier, so a block may exit as soon as it has written its outputs
    const int o_end = min(nout, (rank + 1) * per);
    for (int o = rank * per + tid; o < o_end; o += NT) {
      const int g = o >> 7, j = o - rank * per;
      acc_t mm = (acc_t)-1e30;
      for (int r = 0; r < CS; ++r) {
        const acc_t v = inbox[r * istride + per + g];
        mm = v > mm ? v : mm;
      }
      acc_t num = 0, den = 0;
      for (int r = 0; r < CS; ++r) {
        const acc_t wt = fast_exp2<acc_t>(inbox[r * istride + per + g] - mm);
        num = fma(inbox[r * istride + j], wt, num);
        den = fma(inbox[r * istride + per + GP + g], wt, den);
      }
      out_u[o] = (float)(num / den);
    }
  }
  BPC_STAMP(14);
  if (p.dbg_times != nullptr && tid == 0) p.dbg_times[(size_t)blockIdx.x * 16 + 7] = global_timer_ns();
#undef BPC_STAMP
}

}  // namespace bpcdev
