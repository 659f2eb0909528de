// Shared declarations of the BinaryPC CUDA library (device helpers, context, launch parameters).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "../../include/bpc.h"

#define BPC_D 128            // head_dim (the paper's models all use 128)
#define BPC_MAX_GROUP 8
#define BPC_MAX_CLUSTER 16
#define BPC_LENS_SLOTS 8      // pinned staging slots of bpc_set_seq_lens

// Device error word bits.
#define BPC_DEVERR_CHUNK_CAP   1   // a unit does not fit the cluster's score storage
#define BPC_DEVERR_APPEND_CAP  2   // append at n_max
#define BPC_DEVERR_TIMEOUT     4   // a bounded wait gave up

// In a launch that also appends, the block that codes the new key scans with fewer resources (one warp runs
// Algorithm 2's sign sweep); it is given (16 - BPC_APPEND_LOSS16)/16 of the other blocks' key share.
#define BPC_APPEND_LOSS16 2
__host__ __device__ inline int bpc_fused_chunk(int n, int cs) {
  // n <= 2^26 (bpc_create rejects larger n_max), so 32-bit arithmetic is exact here; a 64-bit division by a run-time
  // divisor would cost every thread of the kernel some hundred instructions
  return ((int)(((unsigned)n * 16u + 16u * (unsigned)cs - (unsigned)BPC_APPEND_LOSS16 - 1u) / (16u * (unsigned)cs - (unsigned)BPC_APPEND_LOSS16)) + 63) & ~63;
}

struct bpc_ctx {
  bpc_config cfg;
  int device;
  int units;                // batch * n_kv_heads
  int group;                // query heads per KV head
  int row_stride;           // cache elements between consecutive rows
  int cluster_size;         // decode: thread blocks per cluster
  int max_cluster;          // largest cluster size the device schedules for the decode kernel
  int max_active[BPC_MAX_CLUSTER + 1];   // [cs]: clusters of size cs that can be resident at once (0 = not schedulable)
  int sm_count;
  bool fitted;
  bool use_pdl;             // launch the decode kernel with programmatic stream serialization
  bool streaming;           // the scores of a full unit do not fit the largest cluster: two-pass (streaming) selection
  float* P;                 // [hash_sets][b][D] float
  void*  P_h;               // [hash_sets][b][D] cache dtype (the hash function)
  float* P_hf;              // P_h as float values
  float* gram;              // [hash_sets][b][b] float, P_h P_h^T
  int32_t* unit_lens;       // [units] device
  int32_t* host_lens;       // [batch] host shadow
  int32_t* lens_staging;    // pinned, [BPC_LENS_SLOTS][units]: per-unit lengths on their way to the device
  cudaEvent_t lens_event[BPC_LENS_SLOTS];
  int lens_slot;
  bool byte_keys;           // Hamming scores stored as byte keys (kernel variant 3): 2.5 times the keys per block
  int force_byte_keys;      // diagnostic switch: 0 = the library decides, 1 = byte keys wherever they are possible, -1 = never
  bool force_streaming;     // diagnostic switch: streaming selection at any size
  bool no_tc_encode;        // diagnostic switch: CUDA-core encode kernel
  int key_shift_min;        // diagnostic switch: weighted scores stored with at least this right shift
  int32_t* sel_scratch;     // [units][n_max] int32
  int32_t* dev_err;         // device error word
  float* key_err;           // [units][n_max] squared reconstruction errors (error-aware safeguard), or null
  int32_t* eas_idx;         // [units][eas_cap] hard-to-hash set, ascending
  int32_t* eas_cnt;         // [units] its size (0 until bpc_build_eas)
  int eas_cap;
  int32_t* dbg_scores;      // caller buffers (may be null)
  int32_t* dbg_qweights;
  unsigned long long* dbg_times;
  int32_t last_cuda_error;
  int64_t launches;
  int chunk_cap_limit;      // keys one decode block can hold with all opt-in shared memory
  double sm_scale_d;        // softmax scale in double (exact 1/sqrt(head_dim) by default)
  size_t decode_smem_set;   // non-zero once the decode kernel's function attributes have been set
  // ---- work-item decode kernel (decode_sched.cuh): geometry and scratch, set up by bpc_create when the shape is covered
  bool sched_ok;            // the work-item kernel serves this context's decode calls
  int decode_path;          // 0 = automatic, 1 = cluster kernel, 2 = work-item kernel (diagnostic switch)
  int sched_grid_max;       // resident blocks (SMs x blocks per SM)
  size_t sched_smem;
  int sched_gran;           // keys per SCAN item are a multiple of this
  int sched_ch;             // keys per SCAN item (automatic choice)
  int sched_r_alloc;        // SCAN items per unit the scratch rows are sized for
  int sched_na_cap;         // ATTEND items per unit the partial slots are sized for
  int sched_ch_user, sched_rpa_user;   // diagnostic overrides (0 = automatic)
  int sched_sc_stride;
  int sched_qp_words;
  uint16_t* sc_scores;
  uint16_t* sc_hist;
  void* sc_table;
  uint32_t* sc_planes;
  float* sc_partials;
  int32_t* sc_sync;
  unsigned long long* dbg_trace;
};

struct DecodeParams {
  const void* q;
  const void* k_cache;
  const void* v_cache;
  const uint64_t* codes;
  const void* P_h;
  const int32_t* unit_lens;
  // fused cache write (all null / unused when the launch only decodes)
  const void* k_new;
  const void* v_new;
  void* k_cache_w;
  void* v_cache_w;
  uint64_t* codes_w;
  int32_t* unit_lens_w;
  const float* gram;
  int residual_correction;
  const int32_t* eas_idx;    // error-aware safeguard set (null when disabled)
  const int32_t* eas_cnt;
  int eas_cap;
  float* out;
  int32_t* sel;              // [units][n_max]
  int32_t* dbg_scores;
  int32_t* dbg_qweights;
  unsigned long long* dbg_times;   // [blocks][8] phase time stamps (ns), or null
  int32_t* err;
  int n_kv_heads;
  int group;
  int n_max;
  int row_stride;            // cache elements between consecutive rows
  int shared_sets;           // 1: projection shared per KV head, 0: one per unit
  int budget_ppm;
  int budget_count;
  double sm_scale_d;         // softmax scale
  int stages;                // gather ring depth (2 or 3)
  int chunk_cap;             // keys whose scores one thread block can hold
  int nbins;                 // histogram bins
  int hist_shift;            // histogram bin = stored score key >> hist_shift
  int key_shift_min;         // weighted scores: smallest right shift of the stored 16-bit keys (diagnostic; normally 0)
};

// ---- launchers implemented in the per-dtype translation units

// ---- launch geometry (api.cu): fills max_cluster, max_active, chunk_cap_limit and picks cluster_size (0 = none fits)
cudaError_t bpc_plan_decode_geometry(bpc_ctx* ctx);

// ---- prefill-side launchers (prefill.cu)
cudaError_t bpc_launch_finalize_projection(bpc_ctx* ctx, cudaStream_t stream);
cudaError_t bpc_launch_encode_simple(bpc_ctx* ctx, const void* k_cache, uint64_t* codes, cudaStream_t stream);
cudaError_t bpc_launch_append(bpc_ctx* ctx, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                              uint64_t* codes, cudaStream_t stream);
cudaError_t bpc_launch_fit(bpc_ctx* ctx, const void* k_cache, const float* v_star, void* workspace,
                           cudaStream_t stream, int* launches);
size_t bpc_fit_workspace_bytes_impl(const bpc_config* cfg);
// tensor-core pass of Algorithm 1 (fit_tc.cu)
bool bpc_fit_tc_covers(const bpc_ctx* ctx);
void bpc_fit_tc_geometry(const bpc_ctx* ctx, int* blocks_per_unit, int* rows_per_block);
cudaError_t bpc_launch_fit_pass_tc(bpc_ctx* ctx, const void* k_cache, uint32_t* hfit, const float* dir, const float* dots,
                                   float* partials, int32_t* agree, int it, cudaStream_t stream);
size_t bpc_fit_codes_offset_impl(const bpc_config* cfg);

// ---- error-aware safeguard set construction (prefill.cu)
cudaError_t bpc_launch_build_eas(bpc_ctx* ctx, cudaStream_t stream);
cudaError_t bpc_launch_exact_topk(bpc_ctx* ctx, const void* q, const void* k_cache, int budget_ppm, int budget_count,
                                  float* scores, int32_t* sel, int32_t* sel_cnt, cudaStream_t stream);

// ---- tensor-core encode (encode_tc.cu); returns cudaErrorNotSupported when the shape is not covered
cudaError_t bpc_launch_encode_tc(bpc_ctx* ctx, const void* k_cache, uint64_t* codes, cudaStream_t stream);

// --------------------------------------------------------------------------- device helpers
#ifdef __CUDACC__
__device__ __forceinline__ float bf16_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }

// 16-byte streaming load that does not allocate in L1 (data read once per step).
__device__ __forceinline__ uint4 ld_stream_v4(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  return r;
}
__device__ __forceinline__ uint32_t ld_stream_u32(const void* p) {
  uint32_t r;
  asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(r) : "l"(p));
  return r;
}
__device__ __forceinline__ uint2 ld_stream_v2(const void* p) {
  uint2 r;
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(r.x), "=r"(r.y) : "l"(p));
  return r;
}

// Streaming data (packed codes, gathered K/V rows) is read once per step: it is marked "evict first" in L2 so that it
// does not push out what the step reuses (the kernel's own instructions, score keys, histograms, partials).
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint4 ld_stream_v4_ef(const void* p, uint64_t pol) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p), "l"(pol));
  return r;
}
__device__ __forceinline__ uint2 ld_stream_v2_ef(const void* p, uint64_t pol) {
  uint2 r;
  asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v2.u32 {%0,%1}, [%2], %3;" : "=r"(r.x), "=r"(r.y) : "l"(p), "l"(pol));
  return r;
}
__device__ __forceinline__ uint32_t ld_stream_u32_ef(const void* p, uint64_t pol) {
  uint32_t r;
  asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.u32 %0, [%1], %2;" : "=r"(r) : "l"(p), "l"(pol));
  return r;
}
__device__ __forceinline__ void cp_async16_ef(void* smem_dst, const void* gsrc, uint64_t pol) {
  const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(d), "l"(gsrc), "l"(pol) : "memory");
}


template <typename T> struct KvTraits;
template <> struct KvTraits<__nv_bfloat16> {
  typedef float acc_t;                 // bf16 products are exact in fp32
  static constexpr int kBytes = 2;
};
template <> struct KvTraits<float> {
  typedef double acc_t;                // fp32 caches: logits and averages in fp64 (1e-5 output tolerance)
  static constexpr int kBytes = 4;
};

__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_float(float v) { return v; }
#endif
