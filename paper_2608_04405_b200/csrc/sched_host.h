// Host interface between api.cu and the work-item decode kernel's translation unit: launch parameters, limits,
// and the functions decode_sched.cu exports.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace bpcdev {

constexpr int kSchedNQ = 2;             // item slots between the producer warp and the scoring warps
constexpr int kSchedMaxUnits = 512;
constexpr int kSchedMaxRanges = 1024;   // SCAN items per unit
constexpr int kSchedListCap = 512;      // rows of one ATTEND item
constexpr int kSchedSyncHead = 8;       // words before the per-unit counters
constexpr int kSchedSyncPerUnit = 8;
constexpr unsigned long long kSchedWaitNs = 250000000ull;   // longest any single wait may last (0.25 s)

enum { IT_DONE = 0, IT_APPEND = 1, IT_HASH = 2, IT_SCAN = 3, IT_ATTEND = 4, IT_THRESH = 5, IT_MERGE = 6 };
enum { SY_HASH = 0, SY_CODE = 1, SY_SCAN = 2, SY_READY = 3, SY_ATT = 4, SY_T = 5, SY_NA = 6, SY_ACLAIM = 7 };   // per-unit words of `sync`

struct SchedParams {
  const void* q;
  const void* k_cache;
  const void* v_cache;
  const uint32_t* codes;
  const void* P_h;
  const float* gram;
  const int32_t* unit_lens;
  int32_t* unit_lens_w;
  const void* k_new;          // fused cache write (null: decode only)
  const void* v_new;
  void* k_cache_w;
  void* v_cache_w;
  uint32_t* codes_w;
  float* out;
  int32_t* sel;               // [units][n_max] or null
  // scratch owned by the context
  uint16_t* scores;           // [units][n_max]
  uint16_t* hist_rows;        // [units][r_max][nbins]
  int4* table;                // [units][r_max + 1]: (selected keys before the range, ties the range may take,
                              //  ATTEND items before the range, unused); entry r_u holds the unit's totals
  uint32_t* qplanes;          // [units][qp_words]
  float* partials;            // [units][na_cap][GP][130]: one slot per ATTEND item
  int32_t* sync;              // ticket, exit counter, abort flag, then kSchedSyncPerUnit words per unit
  int32_t* err;
  int32_t* dbg_scores;
  int32_t* dbg_qweights;
  unsigned long long* dbg_trace;   // [blocks][64][12]: item type << 40 | unit << 24 | index, start ns, end ns, six stamps, unused
  int units, n_kv_heads, group, n_max, row_stride, shared_sets, budget_ppm, budget_count, residual_correction;
  int ch;                     // keys per SCAN item
  int r_max;                  // ceil(n_max / ch)
  int rpa;                    // most rows of one ATTEND item (an item's rows lie in one key range)
  int na_cap;                 // partial slots per unit
  int delta;                  // unused
  int nbins;
  int qp_words;
  int sc_stride;              // score keys per unit in the scratch array (n_max rounded up to 8)
  double sm_scale_d;
};

__host__ __device__ inline int sched_budget(int n, int ppm, int count) {
  long long kk = count > 0 ? (long long)count : ((long long)n * (long long)ppm + 999999LL) / 1000000LL;
  if (kk < 0) kk = 0;
  return (int)(kk < (long long)n ? kk : (long long)n);
}


}  // namespace bpcdev

int bpc_sched_threads(void);                     // scoring threads per block
int bpc_sched_padded_group(int group);           // query heads per KV head the kernel is instantiated for
int bpc_sched_granule(int code_bits);            // keys per SCAN item must be a multiple of this
cudaError_t bpc_sched_configure(int group, int code_bits, int nbins, int units, int device, size_t* smem, int* blocks_per_sm);
cudaError_t bpc_sched_launch(int group, int code_bits, const bpcdev::SchedParams& p, int grid, size_t smem, bool pdl,
                             cudaStream_t stream);
