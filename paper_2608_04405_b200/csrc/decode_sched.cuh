// Decode step as a persistent grid of work items: query hash -> code scan -> top-k -> gathered softmax attention.
//
// Section 3.2 "Retrieval Phase" and Algorithm 3 define what a step computes (see decode_kernel.cuh for the score
// arithmetic, which is shared); this file changes only how the work is spread over the device.  Instead of one
// thread-block cluster per (sequence, KV head) unit, every thread block of a grid that fills the device takes work
// items from one global ticket counter:
//
//   APPEND(u)      cache write of the step's new (k, v) row of unit u and Algorithm 2 on the new key (fused calls only)
//   HASH(u, w)     rows 32w .. 32w+31 of p_g = P_h q_g for the unit's query heads -> word w of the sign word and of the
//                  magnitude planes of the collapsed integer weights A
//   SCAN(u, r)     score keys [r*CH, (r+1)*CH) of unit u: 128-bit streaming loads, two register buffers per thread (the
//                  block's producer warp asked for the range with one bulk L2 prefetch when it claimed the ticket, an
//                  item ahead); the 16-bit score keys go to a scratch array (they stay in L2), the range's histogram
//                  to a scratch row.
//   THRESH(u)      after a unit's last range: the threshold key T from the summed histograms and, per range, the
//                  selected keys before it, its tie quota and its ATTEND items.
//   ATTEND(u, j)   the j-th slice of the unit's selection (ascending index order; a slice is at most RPA selected keys
//                  of ONE key range): the block re-reads that range's score keys, compacts them in order, gathers the
//                  K/V rows and runs online-softmax attention; the partial (m, l, acc) goes to scratch.
//   MERGE(u)       after a unit's last slice: the slices' partials merged in slice order -> output.
//
// Two cursors hand out the work.  A ticket counter runs through APPEND, HASH and then the SCAN items in unit order;
// a SCAN item waits only for its unit's HASH (and, for the range that holds the appended key, APPEND) items, which have
// smaller tickets, so it always waits for work that a running block already holds.  A slice cursor (unit, slice) is
// advanced by compare-and-swap and only while the unit's threshold is known, so an ATTEND item can start the moment
// it is taken; blocks look there first and take a SCAN item otherwise.  No co-residency of blocks is assumed, and
// every wait is bounded (on expiry the device error word gets BPC_DEVERR_TIMEOUT and all waits end).
// THRESH and MERGE items carry no ticket: the producer warp of the block whose item was a unit's last SCAN / ATTEND
// hands them to its own scoring warps next.  The producer warp also does all signalling: when the scoring warps have
// finished an item it issues the device-scope fence and the counter update while they already work on the next item.
// Different units are in different phases at any time, so the code stream of one unit overlaps the row gather of
// another and the short serial phases (hash, threshold, merges) of a third.
#pragma once
#include "decode_kernel.cuh"
#include "sched_host.h"

namespace bpcdev {

// ---- mbarrier / bulk-copy helpers
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* b, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* b, unsigned parity) {
  unsigned ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait(uint64_t* b, unsigned parity) {
  unsigned ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
  return ok != 0;
}
// Bulk asynchronous copy global -> shared memory, completion counted in bytes on an mbarrier.  Both addresses are
// 16-byte aligned and the size is a multiple of 16 bytes (the callers guarantee it).
__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ int ld_acquire(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(int32_t* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_relaxed(const int32_t* p) {
  int v;
  asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// D(16x8,f32) += A(16x16,bf16,row) * B(16x8,bf16,col) with rows 8..15 of A zero: columns 0-7 of A hold the bf16
// value of the eight probabilities, columns 8-15 their bf16 remainders, and both halves of B hold the same eight V
// rows, so one accumulator pair per lane receives (hi + lo) . V.  The two accumulator registers of the zero rows
// are shared by all calls.
__device__ __forceinline__ void mma_pv16(float& d0, float& d1, float& z0, float& z1, uint32_t a_hi, uint32_t a_lo, uint32_t b) {
  const uint32_t z = 0u;
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d0), "+f"(d1), "+f"(z0), "+f"(z1) : "r"(a_hi), "r"(z), "r"(a_lo), "r"(z), "r"(b), "r"(b));
}

// Shared-memory plan of one block, computed identically on host and device.
template <int GP, int W32, int NC>
struct SchedSmem {
  static constexpr int NCW = NC / 32;
  static constexpr int B = W32 * 32;
  static constexpr int U = W32 <= 4 ? 8 : 4;      // codes per thread and register buffer in the scan
  static constexpr int STEP = NC * U;             // keys of one scan batch
  // X: gather rings (per warp NS stages of eight K|V row pairs), or the Gram matrix of the cache-write item
  static constexpr int NS = 3;                    // gather ring depth per warp
  static constexpr int XB = (NCW * NS * 8 * 512) > (B <= 128 ? B * B * 4 : 0) ? (NCW * NS * 8 * 512) : (B * B * 4);
  static_assert(NCW >= 4, "the query hash uses four warps");
  __host__ __device__ static constexpr size_t a128(size_t x) { return (x + 127) & ~(size_t)127; }
  size_t off_x, off_list, off_hist, off_misc, off_tab, off_small, total;
  __host__ __device__ SchedSmem(int nbins, int units, int delta) {
    off_x = 0;
    off_list = off_x + XB;
    off_hist = off_list + (size_t)kSchedListCap * 4;
    off_misc = a128(off_hist + (size_t)nbins * 4);
    // misc: float[GP][128] queries (or the new key), then double[B] decision values of the new key
    off_tab = a128(off_misc + (size_t)GP * BPC_D * 4 + (size_t)B * 8);
    // tab: int n[units], int sb[units + 1]
    (void)delta;
    off_small = a128(off_tab + (size_t)(2 * units + 2) * 4);
    total = off_small + 1024;
  }
};

struct SchedItem {
  int type, unit, idx, T;            // idx: HASH word / SCAN range / ATTEND range
  int slot, part, base, take;        // ATTEND: slice number in the unit, slice number in the range, selected keys before
  int sel, na, pad0, pad1;           //         the range, the range's tie quota, its selected keys; na: the unit's slices
};
struct SchedMeta { int type, unit, aux, pad; };

struct SchedSmall {
  uint64_t qfull[kSchedNQ], qempty[kSchedNQ];
  SchedItem items[kSchedNQ];
  SchedMeta meta[kSchedNQ];             // what the producer warp signals when the item in the slot is finished
  SchedMeta cont[4];                    // THRESH / MERGE items waiting to be handed over (producer warp only)
  uint32_t wscan[64];
  int T, cnt_gt, abort_seen, pad1;
};
static_assert(sizeof(SchedSmall) <= 1024, "small state");

template <int NC> __device__ __forceinline__ void cbar() { asm volatile("bar.sync 1, %0;" ::"n"(NC) : "memory"); }

// Exclusive prefix sum over the NC scoring threads (named barrier 1); see block_excl_scan.
template <int NC>
__device__ __forceinline__ uint32_t cons_excl_scan(uint32_t v, uint32_t* wscan, int& ph, uint32_t* total) {
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
  cbar<NC>();
  uint32_t wbase = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < NC / 32; ++w) {
    const uint32_t e = buf[w];
    if (w < warp) wbase += e;
    tot += e;
  }
  *total = tot;
  return wbase + inc - v;
}

// Algorithm 2 on one key in the Gram form, one warp: lane l holds the decision values of bits l, 32+l, ...; the bits
// are decided eight at a time on lane-redundant copies (their 8 x 8 Gram block is read at one address by the whole
// warp), then the eight signs correct all later columns.  Returns the code words through `out` (lane 0 writes).
template <int W32, bool kUnrolled>
__device__ __forceinline__ void sign_sweep_warp(float (&t)[W32], const float* gq, bool rc, uint32_t* out, int lane) {
  constexpr int NB = W32, B = W32 * 32;
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
        for (int e2 = 0; e2 < 8; ++e2) w[e2] = __shfl_sync(0xffffffffu, tb, 8 * sub + e2);
        const int r0 = 32 * bi + 8 * sub;
        const float* gd = gq + (size_t)r0 * B + r0;
        float nu[8];
#pragma unroll
        for (int e2 = 0; e2 < 8; ++e2) {
          const bool pos = w[e2] >= 0.f;
          wbits |= pos ? (1u << (8 * sub + e2)) : 0u;
          nu[e2] = pos ? -1.f : 1.f;
          const float4 g0 = *reinterpret_cast<const float4*>(gd + (size_t)e2 * B);
          const float4 g1 = *reinterpret_cast<const float4*>(gd + (size_t)e2 * B + 4);
          const float gr[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
          for (int f = e2 + 1; f < 8; ++f) w[f] = fmaf(nu[e2], gr[f], w[f]);
        }
#pragma unroll
        for (int c = 0; c < NB; ++c) {
          if (c >= bi) {
            const float* gc = gq + (size_t)r0 * B + 32 * c + lane;
#pragma unroll
            for (int e2 = 0; e2 < 8; ++e2) t[c] = fmaf(nu[e2], gc[(size_t)e2 * B], t[c]);
          }
        }
      }
    }
    if (lane == 0) out[bi] = wbits;
  }
}

// ------------------------------------------------------------------------------------------------ the kernel
template <int GP, int W32, int NC, int MINB>
__global__ void __launch_bounds__(NC + 32, MINB)
bpc_decode_sched_kernel(const SchedParams p) {
  typedef __nv_bfloat16 KV;
  typedef SchedSmem<GP, W32, NC> L;
  constexpr int NCW = L::NCW, B = L::B, U = L::U, STEP = L::STEP;
  constexpr int NP = PlaneCount<GP, 0>::value;
  constexpr int ROWB = BPC_D * 2;
  extern __shared__ __align__(16) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int NU = p.units, G = p.group;
  const L plan(p.nbins, NU, p.delta);
  unsigned char* X = smem + plan.off_x;
  int32_t* list = reinterpret_cast<int32_t*>(smem + plan.off_list);
  uint32_t* hist = reinterpret_cast<uint32_t*>(smem + plan.off_hist);
  float* qf_s = reinterpret_cast<float*>(smem + plan.off_misc);
  int* un = reinterpret_cast<int*>(smem + plan.off_tab);          // keys of every unit in this step
  int* gb = un + NU;                                              // SCAN items of the units before each unit
  SchedSmall* st = reinterpret_cast<SchedSmall*>(smem + plan.off_small);
  const bool fused = p.k_new != nullptr;
  const int cs = (G & 1) == 0 ? 1 : 0;                            // common factor 2^cs of every |A_j| (Hamming scores)
  int32_t* sy = p.sync;
  int32_t* abortw = sy + 2;

  // Programmatic dependent launch: nothing the previous kernel of the stream wrote is read before this point.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (tid == 0) {
#pragma unroll
    for (int i = 0; i < kSchedNQ; ++i) { mbar_init(&st->qfull[i], 1); mbar_init(&st->qempty[i], 1); }
    st->abort_seen = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // unit table: keys per unit in this step (after the fused cache write), then the ticket layout
  for (int u = tid; u < NU; u += NC + 32) {
    int n = p.unit_lens[u];
    n = max(0, min(n, p.n_max));
    if (fused && n < p.n_max) n += 1;
    un[u] = n;
  }
  __syncthreads();
  auto ranges_of = [&](int u) { return (un[u] + p.ch - 1) / p.ch; };
  if (warp == 0) {                                              // sb[u] = SCAN items of the units before u
    int carry = 0;
    for (int g0 = 0; g0 <= NU; g0 += 32) {
      const int g = g0 + lane;
      const int sz = g < NU ? ranges_of(g) : 0;
      int inc = sz;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      if (g <= NU) gb[g] = carry + inc - sz;
      carry += __shfl_sync(0xffffffffu, inc, 31);
    }
  }
  __syncthreads();
  const int nC = fused ? NU : 0;
  const int nH = NU * W32;
  const int total_tickets = nC + nH + gb[NU];
  const uint64_t pol_ef = l2_evict_first_policy();

  // Bounded waits.  A flag set by another block is polled by one thread; an mbarrier of this block by every waiting
  // thread.  Either gives up after kSchedWaitNs, records BPC_DEVERR_TIMEOUT and raises the abort flag, which ends
  // every other wait of the launch early (results are then undefined, the error word says so, and the counters
  // are still reset at the end so that the context stays usable).
  auto give_up = [&]() {
    atomicOr(p.err, BPC_DEVERR_TIMEOUT);
    atomicExch(abortw, 1);
    st->abort_seen = 1;
  };
  auto wait_flag = [&](const int32_t* f, int want) -> bool {
    if (ld_acquire(f) >= want) return true;
    const unsigned long long t0 = global_timer_ns();
    for (unsigned it = 0;; ++it) {
      if (ld_acquire(f) >= want) return true;
      __nanosleep(it < 16 ? 32 : 200);
      if ((it & 15) == 15) {
        if (ld_relaxed(abortw) != 0) { st->abort_seen = 1; return false; }
        if (global_timer_ns() - t0 > kSchedWaitNs) break;
      }
    }
    give_up();
    return false;
  };
  auto wait_mbar = [&](uint64_t* b, unsigned parity) -> bool {
    if (mbar_try_wait(b, parity)) return true;                 // (try_wait suspends the thread for a bounded time itself)
    const unsigned long long t0 = global_timer_ns();
    for (unsigned it = 0;; ++it) {
      if (mbar_try_wait(b, parity)) return true;
      if ((it & 7) == 7) {
        if (ld_relaxed(abortw) != 0) return false;
        if (global_timer_ns() - t0 > kSchedWaitNs) break;
      }
    }
    give_up();
    return false;
  };

  if (warp == NCW) {
    // ================================================================== producer warp
    // Lane 0 claims tickets and hands items to the scoring warps through a two-slot queue; when the scoring warps have
    // finished an item (its slot's "empty" barrier), lane 0 issues the device-scope fence and updates the unit's
    // counter or flag, so the scoring warps never wait for their stores to drain.  An item that turns out to be a
    // unit's last SCAN (ATTEND) makes this block's next item the unit's THRESH (MERGE).  The whole warp resolves an
    // ATTEND slot to its key range in one round trip.  While lane 0 waits for another block's flag it keeps
    // signalling its own block's finished items (the flag may depend on them).
    unsigned e_pub = 0, e_done = 0;                               // items handed over / items signalled (lane 0)
    int cont_n = 0;
    bool ended = false;
    bool a_done = false;                                          // every unit's slices have been taken
    unsigned long long idle_t0 = 0;
    auto complete = [&](unsigned e) {                             // lane 0: signal item e
      const SchedMeta m = st->meta[e % kSchedNQ];
      int32_t* syu = sy + kSchedSyncHead + m.unit * kSchedSyncPerUnit;
      if (m.type == IT_MERGE) return;
      __threadfence();          // the scoring warps' stores (ordered before this point by their barrier and the slot's
                                // mbarrier) become visible device-wide before the update below
      if (m.type == IT_HASH) atomicAdd(&syu[SY_HASH], 1);
      else if (m.type == IT_APPEND) st_release(&syu[SY_CODE], 1);
      else if (m.type == IT_THRESH) st_release(&syu[SY_READY], 1);
      else if (m.type == IT_SCAN || m.type == IT_ATTEND) {
        const int old = atomicAdd(&syu[m.type == IT_SCAN ? SY_SCAN : SY_ATT], 1);
        if (old == m.aux - 1) {                                   // the unit's last one: its follow-up item runs here
          __threadfence();
          SchedMeta c;
          c.type = m.type == IT_SCAN ? IT_THRESH : IT_MERGE; c.unit = m.unit; c.aux = m.aux; c.pad = 0;
          st->cont[cont_n++] = c;
        }
      }
    };
    auto service = [&]() -> bool {                                // lane 0: signal the oldest item if it is finished
      if (e_done < e_pub && mbar_test_wait(&st->qempty[e_done % kSchedNQ], (e_done / kSchedNQ) & 1)) {
        complete(e_done);
        ++e_done;
        return true;
      }
      return false;
    };
    int a_cur = 0;                                                // (warp-uniform) lowest unit that may still have slices
    for (;;) {
      int type = -1, unit = 0, idx = 0, aux = 0, slot = 0;
      if (lane == 0) {
        while (e_pub - e_done >= (unsigned)kSchedNQ) {            // both slots in use: wait for the older item
          wait_mbar(&st->qempty[e_done % kSchedNQ], (e_done / kSchedNQ) & 1);
          complete(e_done);
          ++e_done;
        }
        slot = (int)(e_pub % kSchedNQ);
        if (cont_n > 0) {
          const SchedMeta c = st->cont[--cont_n];
          type = c.type; unit = c.unit; aux = c.aux;
        }
      }
      type = __shfl_sync(0xffffffffu, type, 0);
      if (type == -1) {
        // Attention slices first.  The 32 lanes look at the next 32 units at once: a unit offers work when its threshold
        // is known and its slice counter is below its number of slices; the lowest such unit's counter is advanced
        // by lane 0 (an atomic add, so blocks never retry against each other), and the slice is taken if the counter
        // was still in range.  A block therefore never holds work that cannot start.
        if (!a_done) {
          const int cu = a_cur + lane;
          bool exhausted = true, offers = false;
          int na_l = 0;
          if (cu < NU && sched_budget(un[cu], p.budget_ppm, p.budget_count) > 0) {
            int32_t* syc = sy + kSchedSyncHead + cu * kSchedSyncPerUnit;
            exhausted = false;
            if (ld_acquire(&syc[SY_READY]) >= 1) {
              na_l = __ldcg(&syc[SY_NA]);
              exhausted = ld_relaxed(&syc[SY_ACLAIM]) >= na_l;
              offers = !exhausted;
            }
          }
          const unsigned exm = __ballot_sync(0xffffffffu, exhausted), ofm = __ballot_sync(0xffffffffu, offers);
          const int lead = exm == 0xffffffffu ? 32 : __ffs(~exm) - 1;   // leading units with nothing left
          if (ofm) {
            const int src = __ffs(ofm) - 1;
            const int na_c = __shfl_sync(0xffffffffu, na_l, src);
            int j = 0;
            if (lane == 0) j = atomicAdd(&sy[kSchedSyncHead + (a_cur + src) * kSchedSyncPerUnit + SY_ACLAIM], 1);
            j = __shfl_sync(0xffffffffu, j, 0);
            if (j < na_c) { type = IT_ATTEND; unit = a_cur + src; idx = j; aux = na_c; }
          }
          a_cur += lead;
          if (a_cur >= NU) a_done = true;
        }
        if (lane == 0 && type == -1) {
          if (!ended) {
            int t = atomicAdd(&sy[0], 1);
            if (t >= total_tickets || ld_relaxed(abortw) != 0) ended = true;
            else if (t < nC) { type = IT_APPEND; unit = t; }
            else if (t < nC + nH) { type = IT_HASH; unit = (t - nC) / W32; idx = (t - nC) % W32; }
            else {
              t -= nC + nH;
              int lo = 0, hi = NU;                               // gb[lo] <= t < gb[hi]
              while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (gb[mid] <= t) lo = mid; else hi = mid;
              }
              type = IT_SCAN; unit = lo; idx = t - gb[lo]; aux = ranges_of(lo);
            }
          }
          if (type == -1) {
            if (ended && (a_done || ld_relaxed(abortw) != 0)) {
              if (e_done < e_pub) {                               // drain: a finished item may still need its follow-up
                wait_mbar(&st->qempty[e_done % kSchedNQ], (e_done / kSchedNQ) & 1);
                complete(e_done);
                ++e_done;
                type = -2;
              } else if (cont_n > 0) {
                type = -2;
              } else {
                type = IT_DONE;
              }
            } else {
              // no scan range left and no unit offers a slice yet: signal finished items, then look again
              if (idle_t0 == 0) idle_t0 = global_timer_ns();
              if (!service()) __nanosleep(200);
              if (global_timer_ns() - idle_t0 > kSchedWaitNs) { give_up(); ended = true; a_done = true; }
              type = -2;
            }
          } else {
            idle_t0 = 0;
          }
        }
        a_done = __shfl_sync(0xffffffffu, (int)a_done, 0) != 0;    // (lane 0 may have given up)
      }
      type = __shfl_sync(0xffffffffu, type, 0);
      if (type == -2) continue;
      unit = __shfl_sync(0xffffffffu, unit, 0);
      idx = __shfl_sync(0xffffffffu, idx, 0);
      aux = __shfl_sync(0xffffffffu, aux, 0);
      slot = __shfl_sync(0xffffffffu, slot, 0);
      __syncwarp();
      int32_t* syu = sy + kSchedSyncHead + unit * kSchedSyncPerUnit;
      SchedItem it;
      it.type = type; it.unit = unit; it.idx = idx; it.T = 0;
      it.slot = 0; it.part = 0; it.base = 0; it.take = 0; it.sel = 0; it.na = aux; it.pad0 = 0; it.pad1 = 0;
      bool skip = false;
      if (type == IT_SCAN) {
        if (lane == 0) {
          // ask for the range's first codes now: they reach L2 while the scoring warps are still busy with the item before
          const int n = un[unit];
          const int k0 = idx * p.ch;
          const int k1 = min(n, k0 + p.ch);
          const unsigned bytes = ((unsigned)min(k1 - k0, STEP) * (W32 * 4)) & ~15u;   // (the first scan batch)
          const unsigned char* src = reinterpret_cast<const unsigned char*>(p.codes) + ((size_t)unit * p.n_max + k0) * (W32 * 4);
          if (bytes) asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
        }
      } else if (type == IT_ATTEND) {
        // slice idx of the unit: the range whose ATTEND items include it (the unit's table holds, per range, the
        // number of slices before it)
        const int R = ranges_of(unit);
        const int4* tb = p.table + (size_t)unit * (p.r_max + 1);
        const int na = min(aux, p.na_cap);
        int found = -1;
        int4 e0 = make_int4(0, 0, 0, 0), e1 = e0;
        if (idx < na) {
          for (int r0 = 0; r0 < R && found < 0; r0 += 32) {
            const int rr = r0 + lane;
            bool hit = false;
            if (rr < R) {
              e0 = __ldcg(tb + rr);
              e1 = __ldcg(tb + rr + 1);
              hit = e0.z <= idx && idx < e1.z;
            }
            const unsigned bal = __ballot_sync(0xffffffffu, hit);
            if (bal) found = __ffs(bal) - 1;
            if (found >= 0) {
              it.idx = r0 + found;
              it.base = __shfl_sync(0xffffffffu, e0.x, found);
              it.take = __shfl_sync(0xffffffffu, e0.y, found);
              it.part = idx - __shfl_sync(0xffffffffu, e0.z, found);
              it.sel = __shfl_sync(0xffffffffu, e1.x, found) - it.base;
            }
          }
        }
        skip = found < 0;
        it.slot = idx;
        it.na = na;
        aux = na;
        it.T = __ldcg(&syu[SY_T]);
      }
      __syncwarp();
      if (skip) continue;                                         // (no slot of the hand-over queue was used)
      if (lane == 0) {
        SchedMeta m;
        m.type = type; m.unit = unit; m.aux = aux; m.pad = 0;
        if (ld_relaxed(abortw) != 0) it.pad0 = 1;               // the launch was aborted: the item is handed over to be skipped
        st->meta[slot] = m;
        st->items[slot] = it;
        mbar_arrive(&st->qfull[slot]);                           // (release: the slot's contents are visible to waiters)
        ++e_pub;
      }
      if (type == IT_DONE) break;
    }
    __syncwarp();
  } else {
    // ================================================================== scoring / attention warps
    const float scale2 = (float)(p.sm_scale_d * 1.4426950408889634);
    int scan_ph = 0;
    int trace_n = 0;
    for (unsigned e = 0;; ++e) {
      const int slot = (int)(e % kSchedNQ);
      wait_mbar(&st->qfull[slot], (e / kSchedNQ) & 1);
      const SchedItem it = st->items[slot];
      if (it.type == IT_DONE) break;
      const int u = it.unit;
      const int kvh = u % p.n_kv_heads, seq_i = u / p.n_kv_heads;
      int32_t* syu = sy + kSchedSyncHead + u * kSchedSyncPerUnit;
      const int n = un[u];
      const int k = sched_budget(n, p.budget_ppm, p.budget_count);
      // item trace (diagnostic): stamps go straight to the trace row
      const bool tracing = p.dbg_trace != nullptr && tid == 0 && trace_n < 64;
#define BPC_TS(i) do { if (tracing) p.dbg_trace[((size_t)blockIdx.x * 64 + trace_n) * 12 + 3 + (i)] = global_timer_ns(); } while (0)
      if (tracing) {
        unsigned long long* tr = p.dbg_trace + ((size_t)blockIdx.x * 64 + trace_n) * 12;
        tr[0] = ((unsigned long long)it.type << 40) | ((unsigned long long)(it.unit & 0xffff) << 24) | (unsigned long long)(it.idx & 0xffffff);
        tr[1] = global_timer_ns();
      }

      if (it.pad0 != 0 || st->abort_seen != 0) {
        // the launch was aborted after a bounded wait ran out: nothing more is computed (the error word says so)
      } else if (it.type == IT_HASH) {
        // ---------------------------------------------------------------- 32 rows of P_h times the unit's queries
        const int w = it.idx;
        float* out_u = p.out + ((size_t)seq_i * p.n_kv_heads + kvh) * (size_t)G * BPC_D;
        if (k == 0) {
          if (w == 0)
            for (int o = tid; o < G * BPC_D; o += NC) out_u[o] = 0.f;
        } else {
          // thread (slice = warp, row = lane): 32 channels of one row times every query; eight exact products are
          // summed in fp32, the groups of eight in fp64, the four slices in fp64 in a fixed order
          uint4 prow[4];
          if (warp < 4) {
            const uint4* row = reinterpret_cast<const uint4*>(reinterpret_cast<const KV*>(p.P_h) +
                                                              ((size_t)(p.shared_sets ? kvh : u) * B + 32 * w + lane) * BPC_D + 32 * warp);
#pragma unroll
            for (int v = 0; v < 4; ++v) prow[v] = row[v];
          }
          const KV* qg = reinterpret_cast<const KV*>(p.q) + ((size_t)seq_i * p.n_kv_heads + kvh) * (size_t)G * BPC_D;
          for (int i = tid; i < GP * BPC_D; i += NC) qf_s[i] = (i >> 7) < G ? to_float(qg[i]) : 0.f;
          BPC_TS(0);
          cbar<NC>();
          BPC_TS(1);
          double* hp = reinterpret_cast<double*>(X);             // [4][GP][32]
          if (warp < 4) {
            double acc[GP];
#pragma unroll
            for (int g = 0; g < GP; ++g) acc[g] = 0.0;
#pragma unroll
            for (int c0 = 0; c0 < 32; c0 += 8) {
              const uint4 wv = prow[c0 / 8];
              const float pv[8] = {bf16_lo(wv.x), bf16_hi(wv.x), bf16_lo(wv.y), bf16_hi(wv.y),
                                   bf16_lo(wv.z), bf16_hi(wv.z), bf16_lo(wv.w), bf16_hi(wv.w)};
#pragma unroll
              for (int g = 0; g < GP; ++g) {
                const float4 q0 = *reinterpret_cast<const float4*>(qf_s + g * BPC_D + 32 * warp + c0);
                const float4 q1 = *reinterpret_cast<const float4*>(qf_s + g * BPC_D + 32 * warp + c0 + 4);
                float s0 = pv[0] * q0.x, s1 = pv[1] * q0.y;
                s0 = fmaf(pv[2], q0.z, s0); s1 = fmaf(pv[3], q0.w, s1);
                s0 = fmaf(pv[4], q1.x, s0); s1 = fmaf(pv[5], q1.y, s1);
                s0 = fmaf(pv[6], q1.z, s0); s1 = fmaf(pv[7], q1.w, s1);
                acc[g] += (double)s0 + (double)s1;
              }
            }
#pragma unroll
            for (int g = 0; g < GP; ++g) hp[((size_t)warp * GP + g) * 32 + lane] = acc[g];
          }
          BPC_TS(2);
          cbar<NC>();
          if (warp == 0) {
            // collapsed weights A_j = sum_g sign(p_gj) -> word w of the sign word and of the planes of |A_j| >> cs
            int A = 0;
            for (int g = 0; g < G; ++g) {
              const double pv = (hp[(0 * GP + g) * 32 + lane] + hp[(1 * GP + g) * 32 + lane]) +
                                (hp[(2 * GP + g) * 32 + lane] + hp[(3 * GP + g) * 32 + lane]);
              A += pv >= 0.0 ? 1 : -1;
            }
            const int absA = A < 0 ? -A : A;
            const uint32_t sw = __ballot_sync(0xffffffffu, A >= 0);
            uint32_t* qp = p.qplanes + (size_t)u * p.qp_words;
            if (lane == 0) qp[w] = sw;
#pragma unroll
            for (int pl = 0; pl < NP; ++pl) {
              const uint32_t mw = __ballot_sync(0xffffffffu, (absA >> (pl + cs)) & 1);
              if (lane == 0) qp[W32 + pl * W32 + w] = mw;
            }
            int rs = absA >> cs;
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) rs += __shfl_xor_sync(0xffffffffu, rs, o);
            if (lane == 0) qp[W32 * (1 + NP) + w] = (uint32_t)rs;
            if (p.dbg_qweights != nullptr) p.dbg_qweights[(size_t)u * B + 32 * w + lane] = A;
          }
          BPC_TS(3);
        }
      } else if (it.type == IT_APPEND) {
        // ---------------------------------------------------------------- cache write + Algorithm 2 on the new key
        const int n_old = p.unit_lens[u];
        if (!(n_old >= 0 && n_old < p.n_max)) {
          if (tid == 0) atomicOr(p.err, BPC_DEVERR_APPEND_CAP);
        } else {
          const KV* kn = reinterpret_cast<const KV*>(p.k_new) + (size_t)u * BPC_D;
          const KV* vn = reinterpret_cast<const KV*>(p.v_new) + (size_t)u * BPC_D;
          const float* Gs = p.gram + (size_t)(p.shared_sets ? kvh : u) * B * B;
          const float* gq = Gs;
          if (p.residual_correction != 0 && (size_t)B * B * 4 <= (size_t)L::XB) {
            // the Gram matrix goes to shared memory so that the sequential sign decisions cost a shuffle and a few FMAs
            float* dstg = reinterpret_cast<float*>(X);
            for (int c = tid; c < B * B / 4; c += NC) cp_async16(dstg + 4 * c, Gs + 4 * c);
            gq = dstg;
          }
          cp_async_commit();
          if (tid < BPC_D) qf_s[tid] = to_float(kn[tid]);
          if (warp == 1) {                                       // the two cache rows
            const size_t rs = (size_t)p.row_stride;
            KV* krow = reinterpret_cast<KV*>(p.k_cache_w) + ((size_t)u * p.n_max + n_old) * rs;
            KV* vrow = reinterpret_cast<KV*>(p.v_cache_w) + ((size_t)u * p.n_max + n_old) * rs;
            const int chn = lane & 15;
            if (lane < 16) reinterpret_cast<uint4*>(krow)[chn] = reinterpret_cast<const uint4*>(kn)[chn];
            else           reinterpret_cast<uint4*>(vrow)[chn] = reinterpret_cast<const uint4*>(vn)[chn];
          }
          BPC_TS(0);
          cbar<NC>();
          // decision values t_j = P_h[j] . k: one row per thread (fp32 sums of eight exact products, fp64 across groups)
          double* pd = reinterpret_cast<double*>(qf_s + GP * BPC_D);   // [B]
          for (int j = tid; j < B; j += NC) {
            const uint4* row = reinterpret_cast<const uint4*>(reinterpret_cast<const KV*>(p.P_h) +
                                                              ((size_t)(p.shared_sets ? kvh : u) * B + j) * BPC_D);
            double acc = 0.0;
#pragma unroll 8
            for (int c0 = 0; c0 < BPC_D; c0 += 8) {
              const uint4 wv = row[c0 / 8];
              const float4 q0 = *reinterpret_cast<const float4*>(qf_s + c0);
              const float4 q1 = *reinterpret_cast<const float4*>(qf_s + c0 + 4);
              float s0 = bf16_lo(wv.x) * q0.x, s1 = bf16_hi(wv.x) * q0.y;
              s0 = fmaf(bf16_lo(wv.y), q0.z, s0); s1 = fmaf(bf16_hi(wv.y), q0.w, s1);
              s0 = fmaf(bf16_lo(wv.z), q1.x, s0); s1 = fmaf(bf16_hi(wv.z), q1.y, s1);
              s0 = fmaf(bf16_lo(wv.w), q1.z, s0); s1 = fmaf(bf16_hi(wv.w), q1.w, s1);
              acc += (double)s0 + (double)s1;
            }
            pd[j] = acc;
          }
          cp_async_wait<0>();
          BPC_TS(1);
          cbar<NC>();
          BPC_TS(2);
          if (warp == 0) {
            float t[W32];
#pragma unroll
            for (int c = 0; c < W32; ++c) t[c] = (float)pd[32 * c + lane];
            uint32_t* code_dst = p.codes_w + ((size_t)u * p.n_max + n_old) * W32;
            sign_sweep_warp<W32, false>(t, gq, p.residual_correction != 0, code_dst, lane);
          }
          BPC_TS(3);
        }
      } else if (it.type == IT_SCAN) {
        // ---------------------------------------------------------------- code scan of one key range
        const int r = it.idx;
        const int k0 = r * p.ch, k1 = min(n, k0 + p.ch);
        const bool has_new = fused && k1 == n && p.unit_lens[u] < p.n_max;
        const int send = has_new ? k1 - 1 : k1;                 // the appended key has no code in memory yet
        const uint32_t* cu = p.codes + (size_t)u * (size_t)p.n_max * W32;
        auto load_code = [&](uint32_t (&h)[W32], int i) {
          const uint32_t* src = cu + (size_t)i * W32;
          if (W32 == 1) {
            h[0] = ld_stream_u32_ef(src, pol_ef);
          } else if (W32 == 2) {
            const uint2 v = ld_stream_v2_ef(src, pol_ef); h[0] = v.x; h[1] = v.y;
          } else {
#pragma unroll
            for (int w = 0; w < W32; w += 4) {
              const uint4 v = ld_stream_v4_ef(src + w, pol_ef);
              h[w] = v.x; h[w + 1] = v.y; h[w + 2] = v.z; h[w + 3] = v.w;
            }
          }
        };
        // a batch is U codes per thread, NC keys apart; indices past the range's end are clamped (and not scored)
        auto load_batch = [&](uint32_t (&h)[U][W32], int base) {
          if (base + STEP <= send) {
#pragma unroll
            for (int uu = 0; uu < U; ++uu) load_code(h[uu], base + uu * NC + tid);
          } else {
#pragma unroll
            for (int uu = 0; uu < U; ++uu) load_code(h[uu], min(base + uu * NC + tid, send - 1));
          }
        };
        uint32_t ha[U][W32], hb[U][W32];
        // the first two batches are requested before anything else: their latency covers the wait for the query hash
        if (k0 < send) load_batch(ha, k0);
        if (k0 + STEP < send) load_batch(hb, k0 + STEP);
        for (int i = tid; i < p.nbins; i += NC) hist[i] = 0u;
        if (tid == 0) wait_flag(&syu[SY_HASH], W32);
        cbar<NC>();
        const bool live = st->abort_seen == 0;                   // (false only after a wait ran out: the range is skipped)
        uint32_t sg[W32], mk[NP][W32];
        const uint32_t* qp = p.qplanes + (size_t)u * p.qp_words;
#pragma unroll
        for (int w = 0; w < W32; ++w) {
          sg[w] = __ldcg(qp + w);
#pragma unroll
          for (int pl = 0; pl < NP; ++pl) mk[pl][w] = __ldcg(qp + W32 + pl * W32 + w);
        }
        uint16_t* sc_u = p.scores + (size_t)u * p.sc_stride;
        int32_t* dbg = p.dbg_scores != nullptr ? p.dbg_scores + (size_t)u * p.n_max : nullptr;
        int rfull = 0;
        if (dbg != nullptr) {
#pragma unroll
          for (int w = 0; w < W32; ++w) rfull += (int)__ldcg(qp + W32 * (1 + NP) + w);
          rfull <<= cs;
        }
        BPC_TS(0);
        auto score_batch = [&](const uint32_t (&h)[U][W32], int base) {
#pragma unroll
          for (int uu = 0; uu < U; ++uu) {
            const int i = base + uu * NC + tid;
            if (i < send) {
              const int key = score_key<W32, NP>(h[uu], sg, mk);
              sc_u[i] = (uint16_t)key;
              atomicAdd(&hist[key], 1u);
              if (dbg != nullptr) dbg[i] = ((2 * key) << cs) - rfull;
            }
          }
        };
#pragma unroll 1
        for (int base = k0; base < send && live; base += 2 * STEP) {
          score_batch(ha, base);
          if (base + 2 * STEP < send) load_batch(ha, base + 2 * STEP);
          if (base + STEP >= send) break;
          score_batch(hb, base + STEP);
          if (base + 3 * STEP < send) load_batch(hb, base + 3 * STEP);
        }
        if (has_new && tid == 0 && live && wait_flag(&syu[SY_CODE], 1)) {
          // the key appended by this launch: its code comes from the APPEND item of the unit
          uint32_t h[W32];
          const uint32_t* src = p.codes_w + ((size_t)u * p.n_max + (n - 1)) * W32;
#pragma unroll
          for (int w = 0; w < W32; ++w) h[w] = __ldcg(src + w);
          const int key = score_key<W32, NP>(h, sg, mk);
          sc_u[n - 1] = (uint16_t)key;
          atomicAdd(&hist[key], 1u);
          if (dbg != nullptr) dbg[n - 1] = ((2 * key) << cs) - rfull;
        }
        BPC_TS(1);
        cbar<NC>();
        BPC_TS(2);
        uint16_t* row = p.hist_rows + ((size_t)u * p.r_max + r) * p.nbins;
        for (int i = tid; i < p.nbins; i += NC) row[i] = (uint16_t)hist[i];
        BPC_TS(3);
      } else if (it.type == IT_THRESH) {
        // ---------------------------------------------------------------- threshold key, per-range offsets and slices
        const int R = (n + p.ch - 1) / p.ch;
        const uint16_t* rows = p.hist_rows + (size_t)u * p.r_max * p.nbins;
        uint32_t* tot = reinterpret_cast<uint32_t*>(X);                 // [nbins]
        int* gt_s = reinterpret_cast<int*>(X) + p.nbins;                // [R]
        int* eq_s = gt_s + R;                                           // [R]
        for (int b = tid; b < p.nbins; b += NC) {
          uint32_t s = 0;
          for (int rr = 0; rr < R; ++rr) s += (uint32_t)__ldcg(rows + (size_t)rr * p.nbins + b);
          tot[b] = s;
        }
        if (tid == 0) { st->T = 0; st->cnt_gt = 0; }
        cbar<NC>();
        BPC_TS(0);
        {
          const int bpt = (p.nbins + NC - 1) / NC;               // bins per thread; thread 0 owns the highest bins
          const int hi = p.nbins - tid * bpt;
          const int lo = max(0, hi - bpt);
          uint32_t local = 0;
          for (int b = hi - 1; b >= lo; --b) local += tot[b];
          uint32_t total;
          uint32_t above = cons_excl_scan<NC>(local, st->wscan, scan_ph, &total);
          for (int b = hi - 1; b >= lo; --b) {
            const uint32_t c = tot[b];
            if (above < (uint32_t)k && above + c >= (uint32_t)k) { st->T = b; st->cnt_gt = (int)above; }
            above += c;
          }
        }
        cbar<NC>();
        BPC_TS(1);
        const int T = st->T;
        const int need = k - st->cnt_gt;                         // ties to take, unit-wide (>= 1)
        for (int rr = warp; rr < R; rr += NCW) {
          const uint16_t* rw = rows + (size_t)rr * p.nbins;
          int g = 0;
          for (int b = T + 1 + lane; b < p.nbins; b += 32) g += (int)__ldcg(rw + b);
          g = __reduce_add_sync(0xffffffffu, g);
          if (lane == 0) { gt_s[rr] = g; eq_s[rr] = (int)__ldcg(rw + T); }
        }
        cbar<NC>();
        BPC_TS(2);
        int4* tb = p.table + (size_t)u * (p.r_max + 1);
        int eq_carry = 0, sel_carry = 0, part_carry = 0;
        for (int r0 = 0; r0 < R; r0 += NC) {                     // ties are granted to ranges in index order
          const int rr = r0 + tid;
          const int eqr = rr < R ? eq_s[rr] : 0, gtr = rr < R ? gt_s[rr] : 0;
          uint32_t tot_e, tot_s, tot_p;
          const int eb = eq_carry + (int)cons_excl_scan<NC>((uint32_t)eqr, st->wscan, scan_ph, &tot_e);
          const int take = min(max(need - eb, 0), eqr);
          const int selr = gtr + take;
          const int sb = sel_carry + (int)cons_excl_scan<NC>((uint32_t)selr, st->wscan, scan_ph, &tot_s);
          const int parts = (selr + p.rpa - 1) / p.rpa;
          const int pb = part_carry + (int)cons_excl_scan<NC>((uint32_t)parts, st->wscan, scan_ph, &tot_p);
          if (rr < R) tb[rr] = make_int4(sb, take, pb, 0);
          eq_carry += (int)tot_e;
          sel_carry += (int)tot_s;
          part_carry += (int)tot_p;
        }
        if (tid == 0) { tb[R] = make_int4(k, 0, part_carry, 0); syu[SY_T] = T; syu[SY_NA] = part_carry; }
        BPC_TS(3);
      } else if (it.type == IT_ATTEND) {
        // ---------------------------------------------------------------- attention over one slice of the selection
        const int r = it.idx, T = it.T;
        const int lo = it.part * p.rpa, hi = min(it.sel, lo + p.rpa), nr = hi - lo;   // ranks inside the range
        const uint16_t* sc_u = p.scores + (size_t)u * p.sc_stride;
        int32_t* sel_u = p.sel != nullptr ? p.sel + (size_t)u * p.n_max : nullptr;
        {
          // Ordered compaction of the range's score keys.  Thread t owns the consecutive 4-key words [t*upt, (t+1)*upt).
          // Two keys share a 32-bit word; adding (0x8000 - T) to both halves raises bit 15 / bit 31 exactly for keys
          // >= T (keys are below 0x8000), likewise with T + 1 for keys > T, so a word costs a few integer operations
          // and only words that hold a candidate are looked at again.
          const int kb = r * p.ch, len = min(n, kb + p.ch) - kb;
          const int upt = (p.ch / 4 + NC - 1) / NC;
          const uint32_t cge = (uint32_t)(0x8000 - T) * 0x10001u, cgt = (uint32_t)(0x8000 - (T + 1)) * 0x10001u;
          const uint2* src = reinterpret_cast<const uint2*>(sc_u + kb) + (size_t)tid * upt;
          auto masks_from = [&](uint2 v, int i0, uint32_t& mge, uint32_t& mgt) {   // 4-bit masks of one word
            const int nv = len - i0;                               // valid keys in the word (>= 1)
            const uint32_t vx = nv >= 2 ? 0x80008000u : 0x00008000u;
            const uint32_t vy = nv >= 4 ? 0x80008000u : (nv == 3 ? 0x00008000u : 0u);
            const uint32_t gex = (v.x + cge) & vx, gey = (v.y + cge) & vy;
            const uint32_t gtx = (v.x + cgt) & vx, gty = (v.y + cgt) & vy;
            mge = ((gex >> 15) & 1u) | ((gex >> 30) & 2u) | ((gey >> 13) & 4u) | ((gey >> 28) & 8u);
            mgt = ((gtx >> 15) & 1u) | ((gtx >> 30) & 2u) | ((gty >> 13) & 4u) | ((gty >> 28) & 8u);
          };
          uint32_t pge = 0u, pgt = 0u;                               // masks of the first eight words, 4 bits each
          int cgtn = 0, cgen = 0;
          {
            uint2 vb[8];                                             // the first eight words: all loads in flight at once
#pragma unroll
            for (int w = 0; w < 8; ++w) {
              vb[w] = make_uint2(0u, 0u);
              if (w < upt && (tid * upt + w) * 4 < len) vb[w] = __ldcg(src + w);
            }
#pragma unroll
            for (int w = 0; w < 8; ++w) {
              const int i0 = (tid * upt + w) * 4;
              if (w < upt && i0 < len) {
                uint32_t mge, mgt;
                masks_from(vb[w], i0, mge, mgt);
                cgen += __popc(mge); cgtn += __popc(mgt);
                pge |= mge << (4 * w); pgt |= mgt << (4 * w);
              }
            }
          }
          for (int w = 8; w < upt; ++w) {
            const int i0 = (tid * upt + w) * 4;
            if (i0 < len) {
              uint32_t mge, mgt;
              masks_from(__ldcg(src + w), i0, mge, mgt);
              cgen += __popc(mge); cgtn += __popc(mgt);
            }
          }
          const int ceqn = cgen - cgtn;
          uint32_t totp;
          const uint32_t ex = cons_excl_scan<NC>((uint32_t)cgtn | ((uint32_t)ceqn << 16), st->wscan, scan_ph, &totp);
          if (cgen) {
            int gtb = (int)(ex & 0xffffu), eqb = (int)(ex >> 16);
            for (int w = 0; w < upt; ++w) {
              const int i0 = (tid * upt + w) * 4;
              uint32_t mge = 0u, mgt = 0u;
              if (w < 8) { mge = (pge >> (4 * w)) & 15u; mgt = (pgt >> (4 * w)) & 15u; }
              else if (i0 < len) masks_from(__ldcg(src + w), i0, mge, mgt);
              while (mge) {
                const int c = __ffs(mge) - 1;
                mge &= mge - 1;
                bool takes;
                int rank;
                if ((mgt >> c) & 1u) { takes = true; rank = gtb + min(eqb, it.take); ++gtb; }
                else { takes = eqb < it.take; rank = gtb + eqb; ++eqb; }
                if (takes && rank >= lo && rank < hi) {
                  list[rank - lo] = kb + i0 + c;
                  if (sel_u != nullptr) sel_u[it.base + rank] = kb + i0 + c;
                }
              }
            }
          }
        }
        cbar<NC>();
        BPC_TS(1);
        // ---- gathered attention: warp w owns rows [nr*w/NCW, nr*(w+1)/NCW) of the slice (see decode_kernel.cuh)
        const size_t rstride = (size_t)p.row_stride * 2;
        const unsigned char* Ku = reinterpret_cast<const unsigned char*>(p.k_cache) + (size_t)u * (size_t)p.n_max * rstride;
        const unsigned char* Vu = reinterpret_cast<const unsigned char*>(p.v_cache) + (size_t)u * (size_t)p.n_max * rstride;
        const KV* qg = reinterpret_cast<const KV*>(p.q) + ((size_t)seq_i * p.n_kv_heads + kvh) * (size_t)G * BPC_D;
        const int g = lane >> 2, t = lane & 3;
        uint32_t qa0[8], qa2[8];
        {
          const uint32_t* qw = reinterpret_cast<const uint32_t*>(qg + (size_t)g * BPC_D);
#pragma unroll
          for (int s = 0; s < 8; ++s) {
            qa0[s] = g < G ? qw[8 * s + t] : 0u;
            qa2[s] = g < G ? qw[8 * s + 4 + t] : 0u;
          }
        }
        float o[16][2], oz0 = 0.f, oz1 = 0.f;
#pragma unroll
        for (int jj = 0; jj < 16; ++jj) { o[jj][0] = o[jj][1] = 0.f; }
        float m_run = -1e30f, l_run = 0.f;
        const int lrow = lane & 7, lmat = lane >> 3;
        constexpr int NS = L::NS;
        constexpr int WSTG = 8 * 2 * ROWB;
        unsigned char* wst = X + (size_t)warp * NS * WSTG;
        const int r0w = (int)(((long long)nr * warp) / NCW), r1w = (int)(((long long)nr * (warp + 1)) / NCW);
        const int nrows = r1w - r0w;
        const int nblk = (nrows + 7) >> 3;
        const int isv = lane >> 4, chn = lane & 15;
        const unsigned char* srcbase = (isv ? Vu : Ku) + (size_t)chn * 16;
        auto issue_rows = [&](int bi) {
          if (bi < nblk) {
            const int rbase = 8 * bi;
            int myidx = -1;
            if (lane < 8 && rbase + lane < nrows) myidx = min(list[r0w + rbase + lane], p.n_max - 1);
            unsigned char* dst = wst + (size_t)(bi % NS) * WSTG + (size_t)isv * (8 * ROWB);
#pragma unroll
            for (int itr = 0; itr < 8; ++itr) {
              const int idx = __shfl_sync(0xffffffffu, myidx, itr);
              unsigned char* d = dst + itr * ROWB + ((chn ^ itr) << 4);
              if (idx >= 0) cp_async16_ef(d, srcbase + (size_t)idx * rstride, pol_ef);
              else *reinterpret_cast<uint4*>(d) = make_uint4(0u, 0u, 0u, 0u);
            }
          }
          cp_async_commit();
        };
        for (int tt = 0; tt < NS; ++tt) issue_rows(tt);
        for (int bi = 0; bi < nblk; ++bi) {
          cp_async_wait<NS - 1>();
          __syncwarp();
          const int rbase_c = 8 * bi;
          const uint32_t vmask = rbase_c + 8 <= nrows ? 0xffu : ((1u << (nrows - rbase_c)) - 1u);
          const unsigned char* ks = wst + (size_t)(bi % NS) * WSTG;
          const unsigned char* vs = ks + 8 * ROWB;
          float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
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
              for (int jj = 0; jj < 16; ++jj) { o[jj][0] *= corr; o[jj][1] *= corr; }
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
            mma_pv16(o[4 * jj][0], o[4 * jj][1], oz0, oz1, pa0, pa1, b[0]);
            mma_pv16(o[4 * jj + 1][0], o[4 * jj + 1][1], oz0, oz1, pa0, pa1, b[1]);
            mma_pv16(o[4 * jj + 2][0], o[4 * jj + 2][1], oz0, oz1, pa0, pa1, b[2]);
            mma_pv16(o[4 * jj + 3][0], o[4 * jj + 3][1], oz0, oz1, pa0, pa1, b[3]);
          }
          __syncwarp();
          issue_rows(bi + NS);
        }
        cp_async_wait<0>();
        BPC_TS(2);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
        cbar<NC>();                                               // the rings are no longer read: reuse them for the merge
        float* part = reinterpret_cast<float*>(X);                // [NCW][GP][130]
        if (g < GP) {
          float* dst = part + ((size_t)warp * GP + g) * (BPC_D + 2);
#pragma unroll
          for (int jj = 0; jj < 16; ++jj) {
            dst[8 * jj + 2 * t] = o[jj][0];
            dst[8 * jj + 2 * t + 1] = o[jj][1];
          }
          if (t == 0) { dst[BPC_D] = m_run; dst[BPC_D + 1] = l_run; }
        }
        cbar<NC>();
        // block-level merge of the warps' partials -> this slice's partial in scratch
        float* gpart = p.partials + ((size_t)u * p.na_cap + it.slot) * (size_t)GP * (BPC_D + 2);
        for (int oi = tid; oi < GP * BPC_D; oi += NC) {
          const int gg = oi >> 7, d = oi & 127;
          float mm = -1e30f;
#pragma unroll
          for (int w = 0; w < NCW; ++w) mm = fmaxf(mm, part[((size_t)w * GP + gg) * (BPC_D + 2) + BPC_D]);
          float num = 0.f, den = 0.f;
#pragma unroll
          for (int w = 0; w < NCW; ++w) {
            const float* srcp = part + ((size_t)w * GP + gg) * (BPC_D + 2);
            const float wt = exp2f(srcp[BPC_D] - mm);
            num = fmaf(srcp[d], wt, num);
            den = fmaf(srcp[BPC_D + 1], wt, den);
          }
          gpart[(size_t)gg * (BPC_D + 2) + d] = num;
          if (d == 0) { gpart[(size_t)gg * (BPC_D + 2) + BPC_D] = mm; gpart[(size_t)gg * (BPC_D + 2) + BPC_D + 1] = den; }
        }
        BPC_TS(3);
      } else if (it.type == IT_MERGE && it.na <= p.na_cap) {
        // ---------------------------------------------------------------- the unit's slices merged in slice order
        float* out_u = p.out + ((size_t)seq_i * p.n_kv_heads + kvh) * (size_t)G * BPC_D;
        const float* up = p.partials + (size_t)u * p.na_cap * (size_t)GP * (BPC_D + 2);
        for (int oi = tid; oi < G * BPC_D; oi += NC) {
          const int gg = oi >> 7, d = oi & 127;
          float mm = -1e30f;
          for (int a = 0; a < it.na; ++a) mm = fmaxf(mm, __ldcg(up + ((size_t)a * GP + gg) * (BPC_D + 2) + BPC_D));
          float num = 0.f, den = 0.f;
          for (int a = 0; a < it.na; ++a) {
            const float* srcp = up + ((size_t)a * GP + gg) * (BPC_D + 2);
            const float wt = exp2f(__ldcg(srcp + BPC_D) - mm);
            num = fmaf(__ldcg(srcp + d), wt, num);
            den = fmaf(__ldcg(srcp + BPC_D + 1), wt, den);
          }
          out_u[oi] = num / den;
        }
      }
      if (tracing) p.dbg_trace[((size_t)blockIdx.x * 64 + trace_n) * 12 + 2] = global_timer_ns();
      if (p.dbg_trace != nullptr) ++trace_n;
#undef BPC_TS
      cbar<NC>();                                                 // every scoring thread is done with the item (and with X)
      if (tid == 0) mbar_arrive(&st->qempty[slot]);               // -> the producer warp signals it
    }
  }

  // ---- exit: the last block to leave resets the counters for the next launch and advances the lengths
  __syncthreads();
  __shared__ int s_last;
  if (tid == 0) {
    __threadfence();
    s_last = (atomicAdd(&sy[1], 1) == (int)gridDim.x - 1) ? 1 : 0;
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    const int words = kSchedSyncHead + NU * kSchedSyncPerUnit;
    for (int i = tid; i < words; i += NC + 32) sy[i] = 0;
    if (fused)
      for (int u = tid; u < NU; u += NC + 32) p.unit_lens_w[u] = un[u];
  }
}

}  // namespace bpcdev
