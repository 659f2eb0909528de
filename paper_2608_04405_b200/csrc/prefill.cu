// Prefill-side and cache-write kernels: projection finalisation, Algorithm 1 (fit), Algorithm 2 on CUDA
// cores (fp32 caches and shapes the tensor-core encode does not cover), and the per-step append.
#include "common.cuh"

namespace {

// --------------------------------------------------------------------------- projection finalisation
// P (float) -> P_h in the cache dtype (the hash function is defined on these rounded values),
// the same values as float, and the Gram matrix G = P_h P_h^T used by the Gram form of Algorithm 2:
// t_i = k.P_i - sum_{j<i} u_j G_ji is the decision value r.P_i of the residual form.
template <typename KV>
__global__ void round_projection_kernel(const float* __restrict__ P, KV* __restrict__ Ph, float* __restrict__ Phf, size_t n) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    KV v = (KV)P[i];
    Ph[i] = v;
    Phf[i] = to_float(v);
  }
}
template <> __global__ void round_projection_kernel<__nv_bfloat16>(const float* __restrict__ P, __nv_bfloat16* __restrict__ Ph,
                                                                   float* __restrict__ Phf, size_t n) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    __nv_bfloat16 v = __float2bfloat16_rn(P[i]);
    Ph[i] = v;
    Phf[i] = __bfloat162float(v);
  }
}

__global__ void gram_kernel(const float* __restrict__ Phf, float* __restrict__ gram, int b) {
  // grid (b, hash_sets); thread j computes G[i][j] with fp64 accumulation
  const int i = blockIdx.x, s = blockIdx.y;
  const float* base = Phf + (size_t)s * b * BPC_D;
  __shared__ float ri[BPC_D];
  for (int c = threadIdx.x; c < BPC_D; c += blockDim.x) ri[c] = base[(size_t)i * BPC_D + c];
  __syncthreads();
  for (int j = threadIdx.x; j < b; j += blockDim.x) {
    const float* rj = base + (size_t)j * BPC_D;
    double acc = 0.0;
    for (int c = 0; c < BPC_D; ++c) acc = fma((double)ri[c], (double)rj[c], acc);
    gram[((size_t)s * b + i) * b + j] = (float)acc;
  }
}

// --------------------------------------------------------------------------- Algorithm 2 on CUDA cores
// One thread per key.  Decision values t = k P_h^T are accumulated in fp64 and kept as fp32 in shared
// memory ([bit][thread]); the greedy sweep u_i = sign(t_i), t_j -= u_i G_ij (j > i) then runs per thread.
constexpr int kEncThreads = 128;

template <typename KV>
__global__ void __launch_bounds__(kEncThreads)
encode_simple_kernel(const KV* __restrict__ k_cache, const float* __restrict__ Phf, const float* __restrict__ gram,
                     const int32_t* __restrict__ unit_lens, uint64_t* __restrict__ codes, int n_kv_heads, int n_max,
                     int row_stride, int b, int shared_sets, int residual_correction, float* __restrict__ key_err) {
  extern __shared__ __align__(16) unsigned char smem[];
  float* ps = reinterpret_cast<float*>(smem);                       // [128 rows of P][128]
  float* ts = ps + 128 * BPC_D;                                      // [b][kEncThreads]
  const int unit = blockIdx.y;
  const int n = min(unit_lens[unit], n_max);
  const int key = blockIdx.x * kEncThreads + threadIdx.x;
  if (blockIdx.x * kEncThreads >= n) return;                         // whole block beyond the unit: uniform
  const int set = shared_sets ? unit % n_kv_heads : unit;
  const float* Pset = Phf + (size_t)set * b * BPC_D;
  const float* Gset = gram + (size_t)set * b * b;
  const bool live = key < n;
  float kr[BPC_D];
  {
    const KV* row = k_cache + ((size_t)unit * n_max + (live ? key : 0)) * row_stride;
#pragma unroll
    for (int c = 0; c < BPC_D; ++c) kr[c] = to_float(row[c]);
  }
  for (int jb = 0; jb < b; jb += 128) {
    const int rows = min(128, b - jb);
    __syncthreads();
    for (int i = threadIdx.x; i < rows * BPC_D; i += kEncThreads) ps[i] = Pset[(size_t)jb * BPC_D + i];
    __syncthreads();
    for (int j = 0; j < rows; ++j) {
      const float4* pr = reinterpret_cast<const float4*>(ps + j * BPC_D);
      double a0 = 0, a1 = 0, a2 = 0, a3 = 0;
#pragma unroll
      for (int c4 = 0; c4 < BPC_D / 4; ++c4) {
        const float4 pv = pr[c4];
        a0 = fma((double)kr[4 * c4], (double)pv.x, a0);
        a1 = fma((double)kr[4 * c4 + 1], (double)pv.y, a1);
        a2 = fma((double)kr[4 * c4 + 2], (double)pv.z, a2);
        a3 = fma((double)kr[4 * c4 + 3], (double)pv.w, a3);
      }
      ts[(size_t)(jb + j) * kEncThreads + threadIdx.x] = (float)((a0 + a1) + (a2 + a3));
    }
  }
  uint32_t* dst = reinterpret_cast<uint32_t*>(codes) + ((size_t)unit * n_max + (live ? key : 0)) * (b / 32);
  uint32_t word = 0;
  double abs_sum = 0.0;                                              // sum of |t_i| at decision time
  for (int i = 0; i < b; ++i) {
    const float ti = ts[(size_t)i * kEncThreads + threadIdx.x];
    const bool pos = ti >= 0.f;
    abs_sum += (double)fabsf(ti);
    word |= (pos ? 1u : 0u) << (i & 31);
    if ((i & 31) == 31) {
      if (live) dst[i >> 5] = word;
      word = 0;
    }
    if (residual_correction) {
      const float u = pos ? 1.f : -1.f;
      const float* gi = Gset + (size_t)i * b;
      for (int j = i + 1; j < b; ++j) ts[(size_t)j * kEncThreads + threadIdx.x] -= u * __ldg(gi + j);
    }
  }
  if (key_err != nullptr && live) {
    // squared reconstruction error (Eq. 8) from the sweep: ||k - hP||^2 = ||k||^2 - 2 sum|t_i| + trace(G)
    double k2 = 0.0, trg = 0.0;
#pragma unroll
    for (int c = 0; c < BPC_D; ++c) k2 = fma((double)kr[c], (double)kr[c], k2);
    for (int i = 0; i < b; ++i) trg += (double)__ldg(Gset + (size_t)i * b + i);
    key_err[(size_t)unit * n_max + key] = (float)fmax(0.0, k2 - 2.0 * abs_sum + trg);
  }
}

// --------------------------------------------------------------------------- append (cache write + Algorithm 2 on one key)
// One block per unit.  The decision values come from a warp-cooperative fp32 mat-vec; the greedy sweep is
// split in 32-bit column blocks: warp B owns columns 32B..32B+31, sweeps its diagonal block with register
// shuffles, publishes its 32 signs, and the later warps apply that rank-32 update.
constexpr int kAppThreads = 256;

template <typename KV>
__global__ void __launch_bounds__(kAppThreads)
append_kernel(const KV* __restrict__ k_new, const KV* __restrict__ v_new, KV* __restrict__ k_cache, KV* __restrict__ v_cache,
              uint64_t* __restrict__ codes, const KV* __restrict__ Ph, const float* __restrict__ gram,
              int32_t* __restrict__ unit_lens, int32_t* __restrict__ err, int n_kv_heads, int n_max, int row_stride,
              int b, int shared_sets, int residual_correction) {
  extern __shared__ __align__(16) unsigned char smem[];
  // the 32 x 32 blocks of the Gram matrix on and to the right of the diagonal (the only ones the sweep reads), block
  // (r, c) at slot r * nb - r (r - 1) / 2 + (c - r): 144 KB at 256 bits
  float* gs = reinterpret_cast<float*>(smem);
  __shared__ float t_s[256];
  __shared__ float k_s[BPC_D];
  __shared__ uint32_t ubits_s[8];
  const int unit = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = unit_lens[unit];
  if (n >= n_max || n < 0) {
    if (tid == 0) atomicOr(err, BPC_DEVERR_APPEND_CAP);
    return;
  }
  const int set = shared_sets ? unit % n_kv_heads : unit;
  const float* Gset = gram + (size_t)set * b * b;
  const int nb = b / 32;
  if (residual_correction) {
    float4* dst = reinterpret_cast<float4*>(gs);
    int slot = 0;
    for (int r = 0; r < nb; ++r) {
      for (int c = r; c < nb; ++c, ++slot) {                         // one block per pass of the 256 threads: row tid / 8, four columns
        const int i = tid >> 3, l4 = tid & 7;
        dst[slot * 256 + tid] = *reinterpret_cast<const float4*>(Gset + (size_t)(32 * r + i) * b + 32 * c + 4 * l4);
      }
    }
  }
  const KV* kn = k_new + (size_t)unit * BPC_D;
  const KV* vn = v_new + (size_t)unit * BPC_D;
  if (tid < BPC_D) {
    const KV kv = kn[tid];
    k_s[tid] = to_float(kv);
    k_cache[((size_t)unit * n_max + n) * row_stride + tid] = kv;
  } else if (tid < 2 * BPC_D) {
    v_cache[((size_t)unit * n_max + n) * row_stride + (tid - BPC_D)] = vn[tid - BPC_D];
  }
  __syncthreads();
  // t_j = P_h[j] . k
  {
    const KV* Pset = Ph + (size_t)set * b * BPC_D;
    const float k0 = k_s[4 * lane], k1 = k_s[4 * lane + 1], k2 = k_s[4 * lane + 2], k3 = k_s[4 * lane + 3];
#pragma unroll 4
    for (int j = warp; j < b; j += kAppThreads / 32) {
      const KV* row = Pset + (size_t)j * BPC_D + 4 * lane;
      float s = to_float(row[0]) * k0;
      s = fmaf(to_float(row[1]), k1, s);
      s = fmaf(to_float(row[2]), k2, s);
      s = fmaf(to_float(row[3]), k3, s);
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) t_s[j] = s;
    }
  }
  __syncthreads();
  auto gblock = [&](int r, int c) { return gs + (size_t)(r * nb - r * (r - 1) / 2 + (c - r)) * 1024; };
  float t = warp < nb ? t_s[32 * warp + lane] : 0.f;
  float gd[32];                                                      // diagonal block column of this lane
  if (warp < nb && residual_correction) {
    const float* gb = gblock(warp, warp);
#pragma unroll
    for (int i = 0; i < 32; ++i) gd[i] = gb[32 * i + lane];
  }
  for (int blk = 0; blk < nb; ++blk) {
    if (warp == blk) {
      uint32_t bits = 0;
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float ti = __shfl_sync(0xffffffffu, t, i);
        const bool pos = ti >= 0.f;
        bits |= (pos ? 1u : 0u) << i;
        if (residual_correction && lane > i) t -= pos ? gd[i] : -gd[i];
      }
      if (lane == 0) {
        ubits_s[blk] = bits;
        (reinterpret_cast<uint32_t*>(codes) + ((size_t)unit * n_max + n) * (b / 32))[blk] = bits;
      }
    }
    __syncthreads();
    if (residual_correction && warp > blk && warp < nb) {
      const uint32_t bits = ubits_s[blk];
      const float* gcol = gblock(blk, warp) + lane;
      float a = 0.f;
#pragma unroll 8
      for (int i = 0; i < 32; ++i) {
        const float g = gcol[32 * i];
        a += ((bits >> i) & 1u) ? g : -g;
      }
      t -= a;
    }
  }
  if (tid == 0) unit_lens[unit] = n + 1;
}

// --------------------------------------------------------------------------- Algorithm 1 (fit)
// The residual is never stored.  With the signs u_j of the earlier bits kept as packed code words (the codes H that
// Algorithm 1 itself produces) and P_j = v_j, a row's residual is R_row = K_row - sum_j u_j v_j, hence
//   t = R_row . d        = K_row . d - sum_{j<i} u_j (v_j . d)          (d = the direction of bit i)
//   u_i R = u_i K - sum_{j<i} (u_i . u_j) v_j                            (u_i . u_j = 2 * agreements - N, an integer)
// Iteration i therefore reads the key row and its code words (272 bytes per row instead of 1 KB of fp32 residual read and
// written back), writes one bit, and leaves per block a partial sum of +-K rows and the per-bit agreement counts; a
// small kernel before the pass prepares d and the b inner products v_j . d, a small one after it forms v_i.
constexpr int kFitThreads = 256;
constexpr int kFitRowsPerBlock = 1024;

// before the pass of bit `it`: dir[unit] = direction (the caller's draw, unless the power-iteration kernel already
// wrote one), dots[unit][j] = v_j . dir for j < it and 0 for the other bits
__global__ void __launch_bounds__(BPC_D)
fit_prep_kernel(const float* __restrict__ P, const float* __restrict__ v_star, float* __restrict__ dir, float* __restrict__ dots,
                int b, int it, int have_dir) {
  const int unit = blockIdx.x, tid = threadIdx.x;
  __shared__ float d_s[BPC_D];
  float dv = have_dir ? dir[(size_t)unit * BPC_D + tid] : v_star[((size_t)unit * b + it) * BPC_D + tid];
  d_s[tid] = dv;
  if (!have_dir) dir[(size_t)unit * BPC_D + tid] = dv;
  __syncthreads();
  for (int j = tid; j < b; j += BPC_D) {
    double acc = 0.0;
    if (j < it) {
      const float* pj = P + ((size_t)unit * b + j) * BPC_D;
      for (int c = 0; c < BPC_D; ++c) acc += (double)pj[c] * (double)d_s[c];
    }
    dots[(size_t)unit * b + j] = (float)acc;
  }
}

// Eight lanes share a row (16 channels and b/8 earlier bits each), so a warp works on four rows at once.
template <typename KV, int JPL>          // JPL = b / 8 bits per lane
__global__ void __launch_bounds__(kFitThreads, 4)   // latency-bound: four blocks (32 warps) per SM
fit_pass_kernel(const KV* __restrict__ k_cache, uint32_t* __restrict__ hfit, const float* __restrict__ dir,
                const float* __restrict__ dots, float* __restrict__ partials, int32_t* __restrict__ agree,
                const int32_t* __restrict__ unit_lens, int n_max, int row_stride, int it, int blocks_per_unit) {
  constexpr int b = JPL * 8, WORDS = b / 32;
  constexpr int CPLN = 16;                                    // channels per lane
  const int unit = blockIdx.y;
  const int n = min(unit_lens[unit], n_max);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sub = lane & 7, grp = lane >> 3;                  // lane within the row's group, row within the warp's four
  const int row0 = blockIdx.x * kFitRowsPerBlock;
  float dv[CPLN];
#pragma unroll
  for (int c = 0; c < CPLN; ++c) dv[c] = dir[(size_t)unit * BPC_D + sub * CPLN + c];
  // sum_j u_j (v_j . d) over a lane's bits is looked up four bits at a time: lut[sub][nibble][pattern] = sum over the
  // nibble's bits of +-(v_j . d) (the inner products of bits >= it are zero, so later bits add nothing)
  constexpr int NIB = JPL / 4;
  __shared__ float lut[8][NIB][16];
  for (int e = tid; e < 8 * NIB * 16; e += kFitThreads) {
    const int m = e & 15, nb = (e >> 4) % NIB, sb = e / (16 * NIB);
    float v = 0.f;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float d = dots[(size_t)unit * b + sb * JPL + 4 * nb + q];
      v += ((m >> q) & 1) ? d : -d;
    }
    lut[sb][nb][m] = v;
  }
  __syncthreads();
  const int my_word = (sub * JPL) >> 5, my_shift = (sub * JPL) & 31;
  float acc[CPLN];
#pragma unroll
  for (int c = 0; c < CPLN; ++c) acc[c] = 0.f;
  // agreements with the earlier bits are counted in six bit-sliced counter planes (at most 32 rows per lane group)
  uint32_t pl[6] = {0u, 0u, 0u, 0u, 0u, 0u};
  const int row_end = min(n, row0 + kFitRowsPerBlock);
  constexpr int ROWS_PER_ITER = (kFitThreads / 32) * 4;
  // Rows reach the lanes through a small ring in shared memory filled by asynchronous copies, NSTG - 1 row sets ahead
  // (the pass is bound by memory latency).  Every lane copies and later reads only its own 16-byte pieces, so the ring
  // needs no barrier.
  constexpr int NV = CPLN * (int)sizeof(KV) / 16;            // 16-byte vectors per lane and row
  constexpr int NSTG = sizeof(KV) == 2 ? 4 : 2;
  __shared__ uint4 ring[NSTG][kFitThreads][NV];
  __shared__ uint32_t ringw[NSTG][kFitThreads];
  auto issue = [&](int slot, int rb) {
    const int r = rb + warp * 4 + grp;
    if (r < row_end) {
      const uint4* kr = reinterpret_cast<const uint4*>(k_cache + ((size_t)unit * n_max + r) * row_stride + sub * CPLN);
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        const unsigned d = (unsigned)__cvta_generic_to_shared(&ring[slot][tid][v]);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(kr + v) : "memory");
      }
      if (it > 0) {
        const unsigned d = (unsigned)__cvta_generic_to_shared(&ringw[slot][tid]);
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(d), "l"(hfit + ((size_t)unit * n_max + r) * WORDS + my_word) : "memory");
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
#pragma unroll
  for (int s0 = 0; s0 < NSTG - 1; ++s0) issue(s0, row0 + s0 * ROWS_PER_ITER);
  int slot = 0;
  for (int rb = row0; rb < row_end; rb += ROWS_PER_ITER) {   // uniform trip count: the shuffles below need whole warps
    issue(slot == 0 ? NSTG - 1 : slot - 1, rb + (NSTG - 1) * ROWS_PER_ITER);
    asm volatile("cp.async.wait_group %0;" ::"n"(NSTG - 1) : "memory");
    const int r = rb + warp * 4 + grp;
    const bool live = r < row_end;
    float x[CPLN];
    if (sizeof(KV) == 2) {
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        const uint4 q = ring[slot][tid][v];
        const uint32_t ww[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) { x[8 * v + 2 * c] = __uint_as_float(ww[c] << 16); x[8 * v + 2 * c + 1] = __uint_as_float(ww[c] & 0xffff0000u); }
      }
    } else {
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        const uint4 q = ring[slot][tid][v];
        x[4 * v] = __uint_as_float(q.x); x[4 * v + 1] = __uint_as_float(q.y); x[4 * v + 2] = __uint_as_float(q.z); x[4 * v + 3] = __uint_as_float(q.w);
      }
    }
    if (!live) {                                             // nothing was copied for this lane: keep the arithmetic finite
#pragma unroll
      for (int c = 0; c < CPLN; ++c) x[c] = 0.f;
    }
    const uint32_t mine = (it > 0 && live) ? (ringw[slot][tid] >> my_shift) : 0u;       // this lane's JPL earlier bits
    slot = slot + 1 == NSTG ? 0 : slot + 1;
    float tk = 0.f;
#pragma unroll
    for (int c = 0; c < CPLN; ++c) tk = fmaf(x[c], dv[c], tk);
    float tc = 0.f;
#pragma unroll
    for (int nb = 0; nb < NIB; ++nb) tc += lut[sub][nb][(mine >> (4 * nb)) & 15u];
    double t = (double)tk - (double)tc;
#pragma unroll
    for (int o = 4; o >= 1; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    const bool pos = t >= 0.0;
    if (live) {
      if (sub == 0) {
        uint32_t* w = hfit + ((size_t)unit * n_max + r) * WORDS + (it >> 5);
        const uint32_t prev = (it & 31) ? *w : 0u;
        *w = prev | ((pos ? 1u : 0u) << (it & 31));
      }
      const float sg = pos ? 1.f : -1.f;
#pragma unroll
      for (int c = 0; c < CPLN; ++c) acc[c] = fmaf(sg, x[c], acc[c]);
      uint32_t carry = pos ? mine : ~mine;                                              // bit e: u_j agrees with u_i
#pragma unroll
      for (int k = 0; k < 6; ++k) {
        const uint32_t nc = pl[k] & carry;
        pl[k] ^= carry;
        carry = nc;
      }
    }
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();                                           // the ring is free: it now holds the block's partial sums
  float (*red)[BPC_D] = reinterpret_cast<float (*)[BPC_D]>(&ring[0][0][0]);
  int32_t (*redc)[b] = reinterpret_cast<int32_t (*)[b]>(reinterpret_cast<unsigned char*>(&ring[0][0][0]) + (kFitThreads / 32) * BPC_D * 4);
  // the four row groups of a warp hold partial sums for the same channels and bits
#pragma unroll
  for (int c = 0; c < CPLN; ++c) {
    acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], 8);
    acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], 16);
  }
  int cnt[JPL];
#pragma unroll
  for (int e = 0; e < JPL; ++e) {
    int c = 0;
#pragma unroll
    for (int k = 0; k < 6; ++k) c += (int)((pl[k] >> e) & 1u) << k;
    c += __shfl_xor_sync(0xffffffffu, c, 8);
    c += __shfl_xor_sync(0xffffffffu, c, 16);
    cnt[e] = c;
  }
  if (grp == 0) {
#pragma unroll
    for (int c = 0; c < CPLN; ++c) red[warp][sub * CPLN + c] = acc[c];
#pragma unroll
    for (int e = 0; e < JPL; ++e) redc[warp][sub * JPL + e] = cnt[e];
  }
  __syncthreads();
  if (tid < BPC_D) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kFitThreads / 32; ++w) s += red[w][tid];
    partials[((size_t)unit * blocks_per_unit + blockIdx.x) * BPC_D + tid] = s;
  }
  for (int j = tid; j < b; j += kFitThreads) {
    int c = 0;
#pragma unroll
    for (int w = 0; w < kFitThreads / 32; ++w) c += redc[w][j];
    agree[((size_t)unit * blocks_per_unit + blockIdx.x) * b + j] = c;
  }
}

// v_i = (sum of the blocks' +-K partial sums - sum_{j<i} (2 * agreements_j - N) v_j) / N.  Four thread groups split
// the blocks and the earlier bits; every sum is formed in a fixed order (group partials added 0..3).
constexpr int kRedGroups = 4;
__global__ void __launch_bounds__(BPC_D * kRedGroups)
fit_reduce_kernel(const float* __restrict__ partials, const int32_t* __restrict__ agree, float* __restrict__ P,
                  const int32_t* __restrict__ unit_lens, int n_max, int b, int it, int blocks_per_unit, int rows_per_block) {
  const int unit = blockIdx.x, c = threadIdx.x & (BPC_D - 1), q = threadIdx.x / BPC_D;
  const int n = min(unit_lens[unit], n_max);
  const int nblk = (n + rows_per_block - 1) / rows_per_block;
  __shared__ double corr[256];                               // u_i . u_j for j < it
  __shared__ double part[kRedGroups][BPC_D];
  __shared__ int agp[kRedGroups][256];
  // agreement counts: group q adds the blocks k = q, q + 4, ... (eight loads in flight per thread), then the groups are added
  for (int j = c; j < it; j += BPC_D) {
    int a8[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    int k = q;
    for (; k + 7 * kRedGroups < nblk; k += 8 * kRedGroups) {
#pragma unroll
      for (int e = 0; e < 8; ++e) a8[e] += agree[((size_t)unit * blocks_per_unit + k + e * kRedGroups) * b + j];
    }
    for (; k < nblk; k += kRedGroups) a8[0] += agree[((size_t)unit * blocks_per_unit + k) * b + j];
    agp[q][j] = ((a8[0] + a8[1]) + (a8[2] + a8[3])) + ((a8[4] + a8[5]) + (a8[6] + a8[7]));
  }
  __syncthreads();
  for (int j = threadIdx.x; j < it; j += BPC_D * kRedGroups) {
    const long long a = (long long)agp[0][j] + agp[1][j] + agp[2][j] + agp[3][j];
    corr[j] = (double)(2 * a - (long long)n);
  }
  __syncthreads();
  double s = 0.0;
  {
    double s8[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    int k = q;
    for (; k + 7 * kRedGroups < nblk; k += 8 * kRedGroups) {
#pragma unroll
      for (int e = 0; e < 8; ++e) s8[e] += (double)partials[((size_t)unit * blocks_per_unit + k + e * kRedGroups) * BPC_D + c];
    }
    for (; k < nblk; k += kRedGroups) s8[0] += (double)partials[((size_t)unit * blocks_per_unit + k) * BPC_D + c];
    s = ((s8[0] + s8[1]) + (s8[2] + s8[3])) + ((s8[4] + s8[5]) + (s8[6] + s8[7]));
  }
  {
    double t8[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    int j = q;
    for (; j + 7 * kRedGroups < it; j += 8 * kRedGroups) {
#pragma unroll
      for (int e = 0; e < 8; ++e) t8[e] += corr[j + e * kRedGroups] * (double)P[((size_t)unit * b + j + e * kRedGroups) * BPC_D + c];
    }
    for (; j < it; j += kRedGroups) t8[0] += corr[j] * (double)P[((size_t)unit * b + j) * BPC_D + c];
    s -= ((t8[0] + t8[1]) + (t8[2] + t8[3])) + ((t8[4] + t8[5]) + (t8[6] + t8[7]));
  }
  part[q][c] = s;
  __syncthreads();
  if (q == 0) {
    double t = 0.0;
#pragma unroll
    for (int g = 0; g < kRedGroups; ++g) t += part[g][c];
    P[((size_t)unit * b + it) * BPC_D + c] = n > 0 ? (float)(t / (double)n) : 0.f;
  }
}

// --------------------------------------------------------------------------- power-iteration fit
// u = sign((R R^T)^n R v*^T) = sign(R z) with z = (R^T R)^n v*^T.  C = R^T R (D x D, fp64) is formed once from the keys
// and then follows the residual through C <- C - N v^T v (u R = N v and u u^T = N make the cross terms collapse), so
// a power-iteration fit costs one extra pass over the keys and a D x D product per bit.
constexpr int kGramRows = 8192;          // key rows per block of the initial Gram pass

// One block per (row slab, unit): its 256 threads own 8 x 8 tiles of the D x D partial sum.  Rows are staged 32 at a
// time in shared memory; a tile of 32 rows is summed in fp32 and added to fp64 accumulators.
template <typename KV>
__global__ void __launch_bounds__(256, 1)
fit_gram0_kernel(const KV* __restrict__ k_cache, double* __restrict__ cpart, const int32_t* __restrict__ unit_lens,
                 int n_max, int row_stride, int slabs_per_unit) {
  const int unit = blockIdx.y, tid = threadIdx.x;
  const int n = min(unit_lens[unit], n_max);
  const int row0 = blockIdx.x * kGramRows, row_end = min(n, row0 + kGramRows);
  __shared__ float tile[32][BPC_D + 4];
  const int i0 = (tid >> 4) * 8, j0 = (tid & 15) * 8;
  double acc[8][8];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[a][c] = 0.0;
  for (int r0 = row0; r0 < row_end; r0 += 32) {
    __syncthreads();
    for (int e = tid; e < 32 * BPC_D; e += 256) {
      const int r = e >> 7, c = e & 127;
      tile[r][c] = (r0 + r < row_end) ? to_float(k_cache[((size_t)unit * n_max + r0 + r) * row_stride + c]) : 0.f;
    }
    __syncthreads();
    float part[8][8];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
      for (int c = 0; c < 8; ++c) part[a][c] = 0.f;
#pragma unroll 4
    for (int r = 0; r < 32; ++r) {
      float xa[8], xb[8];
#pragma unroll
      for (int a = 0; a < 8; ++a) { xa[a] = tile[r][i0 + a]; xb[a] = tile[r][j0 + a]; }
#pragma unroll
      for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int c = 0; c < 8; ++c) part[a][c] = fmaf(xa[a], xb[c], part[a][c]);
    }
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[a][c] += (double)part[a][c];
  }
  double* dst = cpart + ((size_t)unit * slabs_per_unit + blockIdx.x) * BPC_D * BPC_D;
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int c = 0; c < 8; ++c) dst[(size_t)(i0 + a) * BPC_D + j0 + c] = acc[a][c];
}

// C[unit] = sum of the slabs' partial sums, in slab order
__global__ void fit_gram0_reduce_kernel(const double* __restrict__ cpart, double* __restrict__ C,
                                        const int32_t* __restrict__ unit_lens, int n_max, int slabs_per_unit) {
  const int unit = blockIdx.y, e = blockIdx.x * blockDim.x + threadIdx.x;
  const int n = min(unit_lens[unit], n_max);
  const int nslab = (n + kGramRows - 1) / kGramRows;
  double s = 0.0;
  for (int k = 0; k < nslab; ++k) s += cpart[((size_t)unit * slabs_per_unit + k) * BPC_D * BPC_D + e];
  C[(size_t)unit * BPC_D * BPC_D + e] = s;
}

// One block of D threads per unit, before the pass of bit `it`: apply the previous bit's downdate C -= N v v^T (v = row
// it-1 of P), then z = C^n v*_it with a rescale between the products, written as the pass's direction (fp32).
__global__ void __launch_bounds__(BPC_D)
fit_direction_kernel(double* __restrict__ C, const float* __restrict__ P, const float* __restrict__ v_star,
                     float* __restrict__ dir, const int32_t* __restrict__ unit_lens, int n_max, int b, int it, int power_iters) {
  const int unit = blockIdx.x, j = threadIdx.x;
  const int n = min(unit_lens[unit], n_max);
  double* Cu = C + (size_t)unit * BPC_D * BPC_D;
  __shared__ double z[BPC_D];
  __shared__ double red[BPC_D / 32];
  __shared__ float vprev[BPC_D];
  if (it > 0) {
    vprev[j] = P[((size_t)unit * b + (it - 1)) * BPC_D + j];
    __syncthreads();
    const double nv = (double)n * (double)vprev[j];
    for (int c = 0; c < BPC_D; ++c) Cu[(size_t)c * BPC_D + j] -= nv * (double)vprev[c];   // column j (C is symmetric)
  }
  z[j] = (double)v_star[((size_t)unit * b + it) * BPC_D + j];
  __syncthreads();
  for (int k = 0; k < power_iters; ++k) {
    double s = 0.0;
    for (int c = 0; c < BPC_D; ++c) s += Cu[(size_t)c * BPC_D + j] * z[c];                // (C z)_j, reading column j
    double q = s * s;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
    __syncthreads();                                        // everyone has read z
    if ((j & 31) == 0) red[j >> 5] = q;
    __syncthreads();
    double nrm = 0.0;
#pragma unroll
    for (int w = 0; w < BPC_D / 32; ++w) nrm += red[w];
    nrm = sqrt(nrm);
    z[j] = nrm > 0.0 ? s / nrm : s;
    __syncthreads();
  }
  dir[(size_t)unit * BPC_D + j] = (float)z[j];
}

// --------------------------------------------------------------------------- error-aware safeguard set
// One block per unit: the m keys with the largest squared reconstruction error, ties to the lowest index, written
// in ascending index order.  The errors are non-negative floats, so their bit patterns order like unsigned
// integers: a 4-pass radix select (8 bits per pass) finds the m-th largest pattern, then one ordered pass compacts.
constexpr int kEasThreads = 1024;

__global__ void __launch_bounds__(kEasThreads)
build_eas_kernel(const float* __restrict__ key_err, const int32_t* __restrict__ unit_lens, int32_t* __restrict__ eas_idx,
                 int32_t* __restrict__ eas_cnt, int n_max, int eas_ppm, int eas_cap) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t wsum[kEasThreads / 32];
  __shared__ uint32_t s_prefix, s_need, s_run_gt, s_run_eq;
  const int unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = min(unit_lens[unit], n_max);
  int m = (int)(((long long)n * eas_ppm + 999999) / 1000000);
  m = min(min(m, n), eas_cap);
  const uint32_t* e = reinterpret_cast<const uint32_t*>(key_err + (size_t)unit * n_max);
  if (m <= 0) { if (tid == 0) eas_cnt[unit] = 0; return; }
  if (tid == 0) { s_prefix = 0u; s_need = (uint32_t)m; }
  __syncthreads();
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0u;
    __syncthreads();
    const uint32_t prefix = s_prefix, himask = shift == 24 ? 0u : ~((1u << (shift + 8)) - 1u);
    for (int i = tid; i < n; i += kEasThreads) {
      const uint32_t v = e[i];
      if ((v & himask) == prefix) atomicAdd(&hist[(v >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {                                          // 256 bins: a serial walk from the top is cheap enough
      uint32_t need = s_need, acc = 0;
      int d = 255;
      for (; d > 0; --d) { if (acc + hist[d] >= need) break; acc += hist[d]; }
      s_need = need - acc;                                   // still to take among values with this digit
      s_prefix = prefix | ((uint32_t)d << shift);
    }
    __syncthreads();
  }
  const uint32_t thr = s_prefix, need_eq = s_need;           // take every v > thr and the first need_eq with v == thr
  if (tid == 0) { s_run_gt = 0u; s_run_eq = 0u; }
  __syncthreads();
  int32_t* out = eas_idx + (size_t)unit * eas_cap;
  for (int i0 = 0; i0 < n; i0 += kEasThreads) {
    const int i = i0 + tid;
    const uint32_t v = i < n ? e[i] : 0u;
    const bool gt = i < n && v > thr, eq = i < n && v == thr;
    const uint32_t bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
    if (lane == 0) wsum[warp] = (uint32_t)__popc(bg) | ((uint32_t)__popc(be) << 16);
    __syncthreads();
    uint32_t before = 0, total = 0;
    for (int w = 0; w < kEasThreads / 32; ++w) { if (w < warp) before += wsum[w]; total += wsum[w]; }
    const uint32_t lt = (1u << lane) - 1u;
    const uint32_t gt_before = s_run_gt + (before & 0xffffu) + (uint32_t)__popc(bg & lt);
    const uint32_t eq_before = s_run_eq + (before >> 16) + (uint32_t)__popc(be & lt);
    if (gt || (eq && eq_before < need_eq)) out[gt_before + min(eq_before, need_eq)] = i;
    __syncthreads();
    if (tid == 0) { s_run_gt += total & 0xffffu; s_run_eq += total >> 16; }
    __syncthreads();
  }
  if (tid == 0) eas_cnt[unit] = m;
}

}  // namespace

// =========================================================================== host launchers
cudaError_t bpc_launch_finalize_projection(bpc_ctx* ctx, cudaStream_t stream) {
  const bpc_config& c = ctx->cfg;
  const size_t n = (size_t)c.hash_sets * c.code_bits * BPC_D;
  const int th = 256;
  const unsigned blocks = (unsigned)((n + th - 1) / th);
  if (c.kv_dtype == BPC_BF16)
    round_projection_kernel<__nv_bfloat16><<<blocks, th, 0, stream>>>(ctx->P, (__nv_bfloat16*)ctx->P_h, ctx->P_hf, n);
  else
    round_projection_kernel<float><<<blocks, th, 0, stream>>>(ctx->P, (float*)ctx->P_h, ctx->P_hf, n);
  gram_kernel<<<dim3(c.code_bits, c.hash_sets), 128, 0, stream>>>(ctx->P_hf, ctx->gram, c.code_bits);
  ctx->launches += 2;
  return cudaGetLastError();
}

cudaError_t bpc_launch_encode_simple(bpc_ctx* ctx, const void* k_cache, uint64_t* codes, cudaStream_t stream) {
  const bpc_config& c = ctx->cfg;
  const int b = c.code_bits;
  const size_t smem = (size_t)128 * BPC_D * 4 + (size_t)b * kEncThreads * 4;
  const dim3 grid((c.n_max + kEncThreads - 1) / kEncThreads, ctx->units);
  const int shared_sets = c.hash_sets != ctx->units;
  cudaError_t e;
  if (c.kv_dtype == BPC_BF16) {
    e = cudaFuncSetAttribute(encode_simple_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    encode_simple_kernel<__nv_bfloat16><<<grid, kEncThreads, smem, stream>>>(
        (const __nv_bfloat16*)k_cache, ctx->P_hf, ctx->gram, ctx->unit_lens, codes, c.n_kv_heads, c.n_max, ctx->row_stride, b, shared_sets,
        c.residual_correction, ctx->key_err);
  } else {
    e = cudaFuncSetAttribute(encode_simple_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    encode_simple_kernel<float><<<grid, kEncThreads, smem, stream>>>(
        (const float*)k_cache, ctx->P_hf, ctx->gram, ctx->unit_lens, codes, c.n_kv_heads, c.n_max, ctx->row_stride, b, shared_sets,
        c.residual_correction, ctx->key_err);
  }
  ctx->launches += 1;
  return cudaGetLastError();
}

cudaError_t bpc_launch_append(bpc_ctx* ctx, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                              uint64_t* codes, cudaStream_t stream) {
  const bpc_config& c = ctx->cfg;
  const int b = c.code_bits;
  const size_t smem = (size_t)(b / 32) * (b / 32 + 1) / 2 * 4096;   // Gram blocks on and right of the diagonal
  const int shared_sets = c.hash_sets != ctx->units;
  cudaError_t e;
  if (c.kv_dtype == BPC_BF16) {
    e = cudaFuncSetAttribute(append_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    append_kernel<__nv_bfloat16><<<ctx->units, kAppThreads, smem, stream>>>(
        (const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new, (__nv_bfloat16*)k_cache, (__nv_bfloat16*)v_cache, codes,
        (const __nv_bfloat16*)ctx->P_h, ctx->gram, ctx->unit_lens, ctx->dev_err, c.n_kv_heads, c.n_max, ctx->row_stride, b, shared_sets,
        c.residual_correction);
  } else {
    e = cudaFuncSetAttribute(append_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    append_kernel<float><<<ctx->units, kAppThreads, smem, stream>>>(
        (const float*)k_new, (const float*)v_new, (float*)k_cache, (float*)v_cache, codes, (const float*)ctx->P_h,
        ctx->gram, ctx->unit_lens, ctx->dev_err, c.n_kv_heads, c.n_max, ctx->row_stride, b, shared_sets,
        c.residual_correction);
  }
  ctx->launches += 1;
  return cudaGetLastError();
}

static inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// extra workspace of the power-iteration fit, placed after the fitted codes: C, the slabs' partial sums, the directions
static size_t fit_power_bytes(const bpc_config* c) {
  if (c->fit_power_iters <= 0) return 0;
  const size_t units = (size_t)c->batch * c->n_kv_heads;
  const size_t slabs = ((size_t)c->n_max + kGramRows - 1) / kGramRows;
  return align256(units * BPC_D * BPC_D * 8) + align256(units * slabs * BPC_D * BPC_D * 8) + align256(units * BPC_D * 4);
}

// workspace layout: fitted codes H | per-block partial sums | per-block agreement counts | direction | inner products
// | (power-iteration fit) C, its slab partial sums
static size_t fit_off_partials(const bpc_config* c) {
  const size_t units = (size_t)c->batch * c->n_kv_heads;
  return align256(units * c->n_max * (c->code_bits / 8));
}
static size_t fit_off_agree(const bpc_config* c) {
  const size_t units = (size_t)c->batch * c->n_kv_heads;
  const size_t bpu = ((size_t)c->n_max + kFitRowsPerBlock - 1) / kFitRowsPerBlock;
  return fit_off_partials(c) + align256(units * bpu * BPC_D * 4);
}
static size_t fit_off_dir(const bpc_config* c) {
  const size_t units = (size_t)c->batch * c->n_kv_heads;
  const size_t bpu = ((size_t)c->n_max + kFitRowsPerBlock - 1) / kFitRowsPerBlock;
  return fit_off_agree(c) + align256(units * bpu * c->code_bits * 4);
}
static size_t fit_off_power(const bpc_config* c) {
  const size_t units = (size_t)c->batch * c->n_kv_heads;
  return fit_off_dir(c) + align256(units * BPC_D * 4) + align256(units * c->code_bits * 4);
}

size_t bpc_fit_workspace_bytes_impl(const bpc_config* c) { return fit_off_power(c) + fit_power_bytes(c); }

size_t bpc_fit_codes_offset_impl(const bpc_config* c) { (void)c; return 0; }

cudaError_t bpc_launch_fit(bpc_ctx* ctx, const void* k_cache, const float* v_star, void* workspace,
                           cudaStream_t stream, int* launches) {
  const bpc_config& c = ctx->cfg;
  const size_t units = (size_t)ctx->units;
  int bpu = (c.n_max + kFitRowsPerBlock - 1) / kFitRowsPerBlock;
  int rows_per_block = kFitRowsPerBlock;
  // bf16 caches: the pass runs on the tensor cores, with longer row ranges per block (never
  // more blocks than the workspace was sized for)
  const bool tc_pass = bpc_fit_tc_covers(ctx);
  if (tc_pass) bpc_fit_tc_geometry(ctx, &bpu, &rows_per_block);
  unsigned char* ws = (unsigned char*)workspace;
  uint32_t* hfit = (uint32_t*)ws;
  float* partials = (float*)(ws + fit_off_partials(&c));
  int32_t* agree = (int32_t*)(ws + fit_off_agree(&c));
  float* dir = (float*)(ws + fit_off_dir(&c));
  float* dots = (float*)(ws + fit_off_dir(&c) + align256(units * BPC_D * 4));
  const dim3 grid(bpu, ctx->units);
  if (tc_pass) {
    // the tensor-core pass ORs each new bit into its code word and reads the earlier bits back: the words must not
    // carry anything an earlier fit left in the workspace (masking them in the pass instead was measured: 15 % slower)
    cudaError_t e = cudaMemsetAsync(hfit, 0, units * (size_t)c.n_max * (size_t)(c.code_bits / 8), stream);
    if (e != cudaSuccess) return e;
  }
  const int npow = c.fit_power_iters;
  double* Cm = nullptr;
  if (npow > 0) {
    const int slabs = (c.n_max + kGramRows - 1) / kGramRows;
    unsigned char* pw = ws + fit_off_power(&c);
    Cm = (double*)pw;
    double* cpart = (double*)(pw + align256(units * BPC_D * BPC_D * 8));
    const dim3 g0(slabs, ctx->units);
    if (c.kv_dtype == BPC_BF16)
      fit_gram0_kernel<__nv_bfloat16><<<g0, 256, 0, stream>>>((const __nv_bfloat16*)k_cache, cpart, ctx->unit_lens, c.n_max, ctx->row_stride, slabs);
    else
      fit_gram0_kernel<float><<<g0, 256, 0, stream>>>((const float*)k_cache, cpart, ctx->unit_lens, c.n_max, ctx->row_stride, slabs);
    fit_gram0_reduce_kernel<<<dim3(BPC_D * BPC_D / 256, ctx->units), 256, 0, stream>>>(cpart, Cm, ctx->unit_lens, c.n_max, slabs);
    *launches += 2;
  }
  for (int it = 0; it < c.code_bits; ++it) {
    if (npow > 0) {
      fit_direction_kernel<<<ctx->units, BPC_D, 0, stream>>>(Cm, ctx->P, v_star, dir, ctx->unit_lens, c.n_max, c.code_bits, it, npow);
      *launches += 1;
    }
    fit_prep_kernel<<<ctx->units, BPC_D, 0, stream>>>(ctx->P, v_star, dir, dots, c.code_bits, it, npow > 0 ? 1 : 0);
#define BPC_FIT_PASS(KV, JPL)                                                                                          \
    fit_pass_kernel<KV, JPL><<<grid, kFitThreads, 0, stream>>>((const KV*)k_cache, hfit, dir, dots, partials, agree,   \
                                                                ctx->unit_lens, c.n_max, ctx->row_stride, it, bpu)
    if (tc_pass) {
      cudaError_t e = bpc_launch_fit_pass_tc(ctx, k_cache, hfit, dir, dots, partials, agree, it, stream);
      if (e != cudaSuccess) return e;
    } else if (c.kv_dtype == BPC_BF16) {
      if (c.code_bits == 32) BPC_FIT_PASS(__nv_bfloat16, 4); else if (c.code_bits == 64) BPC_FIT_PASS(__nv_bfloat16, 8); else if (c.code_bits == 128) BPC_FIT_PASS(__nv_bfloat16, 16); else BPC_FIT_PASS(__nv_bfloat16, 32);
    } else {
      if (c.code_bits == 32) BPC_FIT_PASS(float, 4); else if (c.code_bits == 64) BPC_FIT_PASS(float, 8); else if (c.code_bits == 128) BPC_FIT_PASS(float, 16); else BPC_FIT_PASS(float, 32);
    }
#undef BPC_FIT_PASS
    fit_reduce_kernel<<<ctx->units, BPC_D * kRedGroups, 0, stream>>>(partials, agree, ctx->P, ctx->unit_lens, c.n_max, c.code_bits, it, bpu, rows_per_block);
    *launches += 3;
  }
  return cudaGetLastError();
}

cudaError_t bpc_launch_build_eas(bpc_ctx* ctx, cudaStream_t stream) {
  build_eas_kernel<<<ctx->units, kEasThreads, 0, stream>>>(ctx->key_err, ctx->unit_lens, ctx->eas_idx, ctx->eas_cnt,
                                                           ctx->cfg.n_max, ctx->cfg.eas_ppm, ctx->eas_cap);
  ctx->launches += 1;
  return cudaGetLastError();
}
