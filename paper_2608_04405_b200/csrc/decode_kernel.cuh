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
//   0  every block hashes the group's queries (fp64 projection, identical in all blocks)
//   1  block r scans keys [r*chunk, (r+1)*chunk): 128-bit code loads, LOP3+POPC score, 16-bit score
//      key into shared memory, shared-memory histogram
//   2  cluster barrier; histograms are summed through distributed shared memory; the threshold key T
//      and the per-block output offsets follow; each block emits its selected indices in ascending
//      order (score > T, then the lowest-index ties at T) into the unit's index list
//   3  cluster barrier; block r runs online-softmax attention over rows [k*r/CS, k*(r+1)/CS) of the
//      list, gathering K and V rows with 16-byte loads; partial (m, l, acc) are merged inside the
//      block, then across the cluster through distributed shared memory
// Scores and gathered rows never touch global memory.
#pragma once
#include <cooperative_groups.h>
#include "common.cuh"

namespace bpcdev {
namespace cg = cooperative_groups;

constexpr int kSegKeys = 32;        // score keys per shared-memory segment
constexpr int kSegSlots = 40;       // 16-bit slots per segment (80 B: conflict-free 16-byte reads)
constexpr int kMaxBins = 2048;      // histogram bins (score keys are 0..nbins-1)
constexpr int kIdxTile = 1024;      // selected indices staged per attention tile
constexpr int kMaxPlanes = 10;

template <int GP, int MODE> struct PlaneCount {
  static constexpr int value = MODE == 0 ? (GP <= 2 ? 1 : (GP == 4 ? 2 : 3))
                                         : (GP == 1 ? 7 : (GP == 2 ? 8 : (GP == 4 ? 9 : 10)));
};

struct SmallState {
  uint32_t signw[8];
  uint32_t mask[kMaxPlanes][8];
  uint32_t gt[BPC_MAX_CLUSTER];
  uint32_t eq[BPC_MAX_CLUSTER];
  uint32_t wscan[32];
  double pmax[BPC_MAX_GROUP];
  int T, cnt_gt, my_take, my_base, rsum, pad[3];
};

template <typename KV, int GP, int W32>
struct DecodeSmem {
  typedef typename KvTraits<KV>::acc_t acc_t;
  static constexpr int NT = (GP <= 4) ? 512 : 256;
  static constexpr int NW = NT / 32;
  static constexpr int B = W32 * 32;
  // offsets in bytes
  __host__ __device__ static constexpr size_t a16(size_t x) { return (x + 15) & ~(size_t)15; }
  __host__ __device__ static constexpr size_t part_bytes() { return (size_t)NW * GP * (BPC_D + 2) * sizeof(acc_t); }
  __host__ __device__ static size_t scores_bytes(int chunk_cap) {
    size_t s = (size_t)((chunk_cap + kSegKeys - 1) / kSegKeys) * kSegSlots * 2;
    return a16(s > part_bytes() ? s : part_bytes());
  }
  static constexpr size_t off_hist = 0;                                    // uint32[kMaxBins]
  static constexpr size_t off_tot = off_hist + kMaxBins * 4;               // uint32[kMaxBins]
  static constexpr size_t off_qd = off_tot + kMaxBins * 4;                 // double[GP][128]
  static constexpr size_t off_pd = off_qd + (size_t)GP * BPC_D * 8;        // double[GP][B]
  static constexpr size_t off_idx = off_pd + (size_t)GP * B * 8;           // int32[kIdxTile]
  static constexpr size_t off_cta = off_idx + kIdxTile * 4;                // acc_t[GP][130]
  static constexpr size_t off_small = a16(off_cta + (size_t)GP * (BPC_D + 2) * sizeof(acc_t));
  static constexpr size_t off_scores = a16(off_small + sizeof(SmallState));
  __host__ __device__ static size_t total(int chunk_cap) { return off_scores + scores_bytes(chunk_cap); }
};

__device__ __forceinline__ int score_slot(int i) { return (i >> 5) * kSegSlots + (i & 31); }

// exclusive prefix sum over the NT threads of a block; *total receives the block sum
template <int NT>
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* wscan, uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();                       // wscan may still be read from a previous call
  if (lane == 31) wscan[warp] = inc;
  __syncthreads();
  uint32_t wbase = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < NT / 32; ++w) {
    uint32_t t = wscan[w];
    if (w < warp) wbase += t;
    tot += t;
  }
  *total = tot;
  return wbase + inc - v;
}

template <typename T> __device__ __forceinline__ T fast_exp2(T x);
template <> __device__ __forceinline__ float fast_exp2<float>(float x) { return exp2f(x); }
template <> __device__ __forceinline__ double fast_exp2<double>(double x) { return exp2(x); }

// K/V row fragment of 8 consecutive dims held by one lane
template <typename KV> struct RowFrag;
template <> struct RowFrag<__nv_bfloat16> {
  uint4 w;
  __device__ __forceinline__ void load(const __nv_bfloat16* row, int hl) { w = ld_stream_v4(row + 8 * hl); }
  __device__ __forceinline__ void get(float* f) const {
    f[0] = bf16_lo(w.x); f[1] = bf16_hi(w.x); f[2] = bf16_lo(w.y); f[3] = bf16_hi(w.y);
    f[4] = bf16_lo(w.z); f[5] = bf16_hi(w.z); f[6] = bf16_lo(w.w); f[7] = bf16_hi(w.w);
  }
};
template <> struct RowFrag<float> {
  uint4 a, b;
  __device__ __forceinline__ void load(const float* row, int hl) {
    a = ld_stream_v4(row + 8 * hl); b = ld_stream_v4(row + 8 * hl + 4);
  }
  __device__ __forceinline__ void get(double* f) const {
    f[0] = __uint_as_float(a.x); f[1] = __uint_as_float(a.y); f[2] = __uint_as_float(a.z); f[3] = __uint_as_float(a.w);
    f[4] = __uint_as_float(b.x); f[5] = __uint_as_float(b.y); f[6] = __uint_as_float(b.z); f[7] = __uint_as_float(b.w);
  }
};

template <typename KV, int GP, int W32, int MODE>
__global__ void __launch_bounds__((GP <= 4) ? 512 : 256, 1)
bpc_decode_kernel(const DecodeParams p) {
  typedef DecodeSmem<KV, GP, W32> L;
  typedef typename L::acc_t acc_t;
  constexpr int NT = L::NT, NW = L::NW, B = L::B;
  constexpr int NP = PlaneCount<GP, MODE>::value;
  extern __shared__ __align__(16) unsigned char smem[];

  cg::cluster_group cluster = cg::this_cluster();
  const int CS = (int)cluster.num_blocks();
  const int rank = (int)cluster.block_rank();
  const int unit = blockIdx.x / CS;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = p.group;
  const int kvh = unit % p.n_kv_heads;
  const int seq = unit / p.n_kv_heads;

  int n = p.unit_lens[unit];
  n = max(0, min(n, p.n_max));
  long long kk = p.budget_count > 0 ? (long long)p.budget_count
                                    : ((long long)n * (long long)p.budget_ppm + 999999LL) / 1000000LL;
  if (kk < 0) kk = 0;
  const int k = (int)(kk < (long long)n ? kk : (long long)n);
  const int chunk = (((n + CS - 1) / CS) + 63) & ~63;
  float* out_u = p.out + ((size_t)seq * p.n_kv_heads + kvh) * (size_t)G * BPC_D;

  // Both early exits depend only on values every block of the cluster sees identically, so either all
  // blocks of a cluster leave here (before any cluster barrier) or none does.
  if (chunk > p.chunk_cap) {
    if (tid == 0) atomicOr(p.err, BPC_DEVERR_CHUNK_CAP);
    return;
  }
  if (k == 0) {
    if (rank == 0)
      for (int o = tid; o < G * BPC_D; o += NT) out_u[o] = 0.f;
    return;
  }

  uint32_t* hist = reinterpret_cast<uint32_t*>(smem + L::off_hist);
  uint32_t* tot = reinterpret_cast<uint32_t*>(smem + L::off_tot);
  double* qd = reinterpret_cast<double*>(smem + L::off_qd);
  double* pd = reinterpret_cast<double*>(smem + L::off_pd);
  int32_t* idx_s = reinterpret_cast<int32_t*>(smem + L::off_idx);
  acc_t* cta_acc = reinterpret_cast<acc_t*>(smem + L::off_cta);        // [GP][128], then m[GP], l[GP]
  acc_t* cta_m = cta_acc + GP * BPC_D;
  acc_t* cta_l = cta_m + GP;
  SmallState* st = reinterpret_cast<SmallState*>(smem + L::off_small);
  uint16_t* sc = reinterpret_cast<uint16_t*>(smem + L::off_scores);
  const int nbins = p.nbins;

  // ------------------------------------------------------------------ phase 0: query hash
  const KV* qg = reinterpret_cast<const KV*>(p.q) + ((size_t)seq * p.n_kv_heads + kvh) * (size_t)G * BPC_D;
  for (int i = tid; i < GP * BPC_D; i += NT) qd[i] = (i >> 7) < G ? (double)to_float(qg[i]) : 0.0;
  for (int i = tid; i < nbins; i += NT) hist[i] = 0u;
  if (tid < BPC_MAX_CLUSTER) { st->gt[tid] = 0u; st->eq[tid] = 0u; }
  if (tid == 0) { st->rsum = 0; st->T = 0; st->cnt_gt = 0; }
  __syncthreads();
  {
    const KV* Ph = reinterpret_cast<const KV*>(p.P_h) + (size_t)(p.shared_sets ? kvh : unit) * B * BPC_D;
#pragma unroll 4
    for (int j = warp; j < B; j += NW) {
      const KV* row = Ph + (size_t)j * BPC_D + 4 * lane;
      double pv[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) pv[c] = (double)to_float(row[c]);
#pragma unroll
      for (int g = 0; g < GP; ++g) {
        const double* qq = qd + g * BPC_D + 4 * lane;
        double s = pv[0] * qq[0];
        s = fma(pv[1], qq[1], s); s = fma(pv[2], qq[2], s); s = fma(pv[3], qq[3], s);
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) pd[g * B + j] = s;
      }
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
  __syncthreads();

  // ------------------------------------------------------------------ phase 1: scan
  const int c0 = min(n, rank * chunk), c1 = min(n, c0 + chunk);
  {
    uint32_t sg[W32], mk[NP][W32];
#pragma unroll
    for (int w = 0; w < W32; ++w) {
      sg[w] = st->signw[w];
#pragma unroll
      for (int pl = 0; pl < NP; ++pl) mk[pl][w] = st->mask[pl][w];
    }
    const int rfull = st->rsum << cs;                       // sum_j |A_j|
    const uint32_t* cu = reinterpret_cast<const uint32_t*>(p.codes) + (size_t)unit * (size_t)p.n_max * W32;
    int32_t* dbg = p.dbg_scores != nullptr ? p.dbg_scores + (size_t)unit * p.n_max : nullptr;
    constexpr int U = 4;
    for (int i0 = c0; i0 < c1; i0 += NT * U) {
      uint32_t h[U][W32];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = i0 + u * NT + tid;
        if (i < c1) {
          const uint32_t* src = cu + (size_t)i * W32;
          if (W32 == 2) {
            const uint2 v = ld_stream_v2(src); h[u][0] = v.x; h[u][1] = v.y;
          } else {
#pragma unroll
            for (int w = 0; w < W32; w += 4) {
              const uint4 v = ld_stream_v4(src + w);
              h[u][w] = v.x; h[u][w + 1] = v.y; h[u][w + 2] = v.z; h[u][w + 3] = v.w;
            }
          }
        } else {
#pragma unroll
          for (int w = 0; w < W32; ++w) h[u][w] = 0u;
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = i0 + u * NT + tid;
        if (i < c1) {
          int key = 0;
#pragma unroll
          for (int pl = 0; pl < NP; ++pl) {
            int c = 0;
#pragma unroll
            for (int w = 0; w < W32; ++w) c += __popc(~(h[u][w] ^ sg[w]) & mk[pl][w]);
            key += c << pl;
          }
          sc[score_slot(i - c0)] = (uint16_t)key;
          atomicAdd(&hist[key], 1u);
          if (dbg != nullptr) dbg[i] = ((2 * key) << cs) - rfull;
        }
      }
    }
  }

  // ------------------------------------------------------------------ phase 2: threshold and ordered selection
  cluster.sync();                                            // every block's histogram is complete
  for (int bin = tid; bin < nbins; bin += NT) {
    uint32_t s = 0;
    for (int r = 0; r < CS; ++r) s += cluster.map_shared_rank(hist, r)[bin];
    tot[bin] = s;
  }
  __syncthreads();
  {
    const int bpt = (nbins + NT - 1) / NT;                   // bins per thread; thread 0 owns the highest bins
    const int hi = nbins - tid * bpt;
    const int lo = max(0, hi - bpt);
    uint32_t local = 0;
    for (int bin = hi - 1; bin >= lo; --bin) local += tot[bin];
    uint32_t total;
    uint32_t above = block_excl_scan<NT>(local, st->wscan, &total);
    for (int bin = hi - 1; bin >= lo; --bin) {
      const uint32_t c = tot[bin];
      if (above < (uint32_t)k && above + c >= (uint32_t)k) { st->T = bin; st->cnt_gt = (int)above; }
      above += c;
    }
  }
  __syncthreads();
  const int T = st->T;
  for (int bin = T + 1 + tid; bin < nbins; bin += NT) {
    if (tot[bin] == 0u) continue;
    for (int r = 0; r < CS; ++r) {
      const uint32_t v = cluster.map_shared_rank(hist, r)[bin];
      if (v) atomicAdd(&st->gt[r], v);
    }
  }
  if (tid < CS) st->eq[tid] = cluster.map_shared_rank(hist, tid)[T];
  __syncthreads();
  if (tid == 0) {
    const int need = k - st->cnt_gt;                         // ties to take, cluster-wide (>= 1)
    int tie_base = 0, out_base = 0;
    for (int r = 0; r < CS; ++r) {
      int take = need - tie_base;
      take = take < 0 ? 0 : (take > (int)st->eq[r] ? (int)st->eq[r] : take);
      if (r == rank) { st->my_take = take; st->my_base = out_base; }
      out_base += (int)st->gt[r] + take;
      tie_base += (int)st->eq[r];
    }
  }
  __syncthreads();
  int32_t* sel_u = p.sel + (size_t)unit * p.n_max;
  {
    const int len = c1 - c0;
    const int nseg = (len + kSegKeys - 1) / kSegKeys;
    const int my_take = st->my_take;
    int run_gt = 0, run_eq = 0;
    for (int s0 = 0; s0 < nseg; s0 += NT) {
      const int seg = s0 + tid;
      uint32_t kw[16];
      int cgt = 0, ceq = 0;
      if (seg < nseg) {
        const uint4* src = reinterpret_cast<const uint4*>(sc + (size_t)seg * kSegSlots);
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const uint4 x = src[v];
          kw[4 * v] = x.x; kw[4 * v + 1] = x.y; kw[4 * v + 2] = x.z; kw[4 * v + 3] = x.w;
        }
        const int valid = min(kSegKeys, len - seg * kSegKeys);
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int key = (int)((kw[j >> 1] >> ((j & 1) * 16)) & 0xffffu);
          if (j < valid) { cgt += key > T; ceq += key == T; }
        }
      }
      uint32_t total;
      const uint32_t ex = block_excl_scan<NT>((uint32_t)cgt | ((uint32_t)ceq << 16), st->wscan, &total);
      if (seg < nseg && (cgt | ceq)) {
        int eqb = run_eq + (int)(ex >> 16);
        int pos = st->my_base + run_gt + (int)(ex & 0xffffu) + min(eqb, my_take);
        const int valid = min(kSegKeys, len - seg * kSegKeys);
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int key = (int)((kw[j >> 1] >> ((j & 1) * 16)) & 0xffffu);
          if (j < valid) {
            if (key > T) {
              sel_u[pos++] = c0 + seg * kSegKeys + j;
            } else if (key == T) {
              if (eqb < my_take) sel_u[pos++] = c0 + seg * kSegKeys + j;
              ++eqb;
            }
          }
        }
      }
      run_gt += (int)(total & 0xffffu);
      run_eq += (int)(total >> 16);
    }
  }
  __threadfence();
  cluster.sync();                                            // the unit's index list is complete and visible

  // ------------------------------------------------------------------ phase 3: gathered attention
  const int hl = lane & 15, half = lane >> 4;
  const int lo = (int)(((long long)k * rank) / CS), hi = (int)(((long long)k * (rank + 1)) / CS);
  acc_t qf[GP][8], acc[GP][8], m_run[GP], l_run[GP];
  {
    const double scale = (double)p.sm_scale * 1.4426950408889634;   // logits in base-2 exponent units
#pragma unroll
    for (int g = 0; g < GP; ++g) {
#pragma unroll
      for (int c = 0; c < 8; ++c) { qf[g][c] = (acc_t)(qd[g * BPC_D + 8 * hl + c] * scale); acc[g][c] = (acc_t)0; }
      m_run[g] = (acc_t)-1e30; l_run[g] = (acc_t)0;
    }
  }
  const KV* Ku = reinterpret_cast<const KV*>(p.k_cache) + (size_t)unit * (size_t)p.n_max * BPC_D;
  const KV* Vu = reinterpret_cast<const KV*>(p.v_cache) + (size_t)unit * (size_t)p.n_max * BPC_D;

  auto process = [&](const RowFrag<KV>& kf, const RowFrag<KV>& vf, bool valid) {
    acc_t kv8[8], s[GP];
    kf.get(kv8);
#pragma unroll
    for (int g = 0; g < GP; ++g) {
      acc_t d = qf[g][0] * kv8[0];
#pragma unroll
      for (int c = 1; c < 8; ++c) d = fma(qf[g][c], kv8[c], d);
      s[g] = d;
    }
#pragma unroll
    for (int o = 8; o >= 1; o >>= 1) {
#pragma unroll
      for (int g = 0; g < GP; ++g) s[g] += __shfl_xor_sync(0xffffffffu, s[g], o);
    }
    bool grow = false;
#pragma unroll
    for (int g = 0; g < GP; ++g) grow |= (s[g] > m_run[g]);
    grow &= valid;
    if (__any_sync(0xffffffffu, grow)) {
      if (valid) {
#pragma unroll
        for (int g = 0; g < GP; ++g) {
          if (s[g] > m_run[g]) {
            const acc_t corr = fast_exp2<acc_t>(m_run[g] - s[g]);
            l_run[g] *= corr;
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[g][c] *= corr;
            m_run[g] = s[g];
          }
        }
      }
    }
    vf.get(kv8);
#pragma unroll
    for (int g = 0; g < GP; ++g) {
      const acc_t pr = valid ? fast_exp2<acc_t>(s[g] - m_run[g]) : (acc_t)0;
      l_run[g] += pr;
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[g][c] = fma(pr, kv8[c], acc[g][c]);
    }
  };

  for (int t0 = lo; t0 < hi; t0 += kIdxTile) {
    const int tn = min(kIdxTile, hi - t0);
    __syncthreads();
    for (int i = tid; i < tn; i += NT) idx_s[i] = sel_u[t0 + i];
    __syncthreads();
    // a warp handles two rows per pass (one per half warp), two passes per iteration
    for (int rp = warp; 2 * rp < tn; rp += 2 * NW) {
      const int r0 = 2 * rp + half, r1 = 2 * (rp + NW) + half;
      const bool v0 = r0 < tn, v1 = r1 < tn;
      const int i0 = min(max(idx_s[v0 ? r0 : 0], 0), p.n_max - 1);
      const int i1 = min(max(idx_s[v1 ? r1 : 0], 0), p.n_max - 1);
      RowFrag<KV> k0, vv0, k1, vv1;
      k0.load(Ku + (size_t)i0 * BPC_D, hl); vv0.load(Vu + (size_t)i0 * BPC_D, hl);
      k1.load(Ku + (size_t)i1 * BPC_D, hl); vv1.load(Vu + (size_t)i1 * BPC_D, hl);
      process(k0, vv0, v0);
      process(k1, vv1, v1);
    }
  }

  // merge the two half warps, then the warps of the block
  acc_t* part = reinterpret_cast<acc_t*>(sc);                // [NW][GP][130]: the score storage is free now
#pragma unroll
  for (int g = 0; g < GP; ++g) {
    const acc_t om = __shfl_xor_sync(0xffffffffu, m_run[g], 16);
    const acc_t ol = __shfl_xor_sync(0xffffffffu, l_run[g], 16);
    const acc_t mm = om > m_run[g] ? om : m_run[g];
    const acc_t ws = fast_exp2<acc_t>(m_run[g] - mm), wo = fast_exp2<acc_t>(om - mm);
    l_run[g] = l_run[g] * ws + ol * wo;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const acc_t oa = __shfl_xor_sync(0xffffffffu, acc[g][c], 16);
      acc[g][c] = acc[g][c] * ws + oa * wo;
    }
    m_run[g] = mm;
  }
  __syncthreads();                                           // all reads of the score storage are done
  if (half == 0) {
#pragma unroll
    for (int g = 0; g < GP; ++g) {
      acc_t* dst = part + ((size_t)warp * GP + g) * (BPC_D + 2);
#pragma unroll
      for (int c = 0; c < 8; ++c) dst[8 * hl + c] = acc[g][c];
      if (hl == 0) { dst[BPC_D] = m_run[g]; dst[BPC_D + 1] = l_run[g]; }
    }
  }
  __syncthreads();
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
    cta_acc[o] = num;
    if (d == 0) { cta_m[g] = mm; cta_l[g] = den; }
  }
  cluster.sync();                                            // every block's partial result is published
  {
    const int nout = G * BPC_D;
    const int per = (nout + CS - 1) / CS;
    const int o_end = min(nout, (rank + 1) * per);
    for (int o = rank * per + tid; o < o_end; o += NT) {
      const int g = o >> 7;
      acc_t mm = (acc_t)-1e30;
      for (int r = 0; r < CS; ++r) {
        const acc_t v = cluster.map_shared_rank(cta_m, r)[g];
        mm = v > mm ? v : mm;
      }
      acc_t num = 0, den = 0;
      for (int r = 0; r < CS; ++r) {
        const acc_t wt = fast_exp2<acc_t>(cluster.map_shared_rank(cta_m, r)[g] - mm);
        num = fma(cluster.map_shared_rank(cta_acc, r)[o], wt, num);
        den = fma(cluster.map_shared_rank(cta_l, r)[g], wt, den);
      }
      out_u[o] = (float)(num / den);
    }
  }
  cluster.sync();                                            // keep shared memory alive until all peers have read it
}

}  // namespace bpcdev
