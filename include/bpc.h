/*
 * bpc.h - C-ABI of the BinaryPC decode-time sparse-attention library (single GPU, sm_100a).
 *
 * The library implements the per-token hot path of "Training-Free Hashing-Based Attention via
 * Binary Principal Components": fit the per-head hash projection (Algorithm 1), encode cached keys
 * (Algorithm 2), append a code on every cache write, and per decode step hash the query, score it
 * against every packed key code (Algorithm 3), keep the top-k keys per KV head and run softmax
 * attention over those rows only (Section 3.2, "Retrieval Phase").
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer owned by the caller unless its name starts with host_.
 *     The library allocates device memory only inside bpc_create (state of the context) and frees
 *     it in bpc_destroy.  No entry point copies, resizes or keeps caller buffers beyond the call.
 *     The small per-step arrays q, k_new, v_new and out of bpc_decode_attn / bpc_append /
 *     bpc_append_decode_attn may instead be pinned (page-locked) host memory that the device can
 *     address at its host address (cudaHostAlloc / cudaHostRegister under unified addressing):
 *     the kernels then read the step's inputs and write its result across the bus themselves,
 *     which saves the copies of a host-driven decode loop.  Caches, codes and projections must be
 *     device memory.
 *   - Every compute call is asynchronous on `stream` (a cudaStream_t passed as void*; NULL is the
 *     legacy default stream) and returns a bpc_status; nothing aborts, traps or prints.  Only
 *     bpc_last_device_error waits for the stream.
 *   - Layouts (row-major, contiguous):
 *       k_cache, v_cache : [batch][n_kv_heads][n_max] rows of head_dim kv_dtype values, base 16-byte
 *                          aligned; consecutive rows are kv_row_stride elements apart (head_dim when the
 *                          caches are separate arrays; 2*head_dim with v_cache = k_cache + head_dim for the
 *                          interleaved layout, where a token's K and V rows are adjacent in memory and one
 *                          gather touches 4*head_dim contiguous bytes instead of two separate rows)
 *       codes            : [batch][n_kv_heads][n_max][code_bits/64] uint64 (code_bits/8 bytes per key; with
 *                          32-bit codes one uint32 per key, the array still passed as uint64_t*)
 *                          bit j of a key (Algorithm 2 iteration j+1) is word j/64, bit j%64,
 *                          least significant first; 1 means the component is +1 (decision value >= 0)
 *       q                : [batch][n_q_heads][head_dim]            kv_dtype
 *       out              : [batch][n_q_heads][head_dim]            float
 *       k_new, v_new     : [batch][n_kv_heads][head_dim]           kv_dtype
 *       projection P     : [hash_sets][code_bits][head_dim]        float
 *     Query head hq belongs to KV head hq / (n_q_heads / n_kv_heads).  A "unit" is one
 *     (sequence, KV head) pair, unit = sequence * n_kv_heads + kv_head.
 *   - Limits: head_dim == 128; code_bits in {32,64,128,256}; n_q_heads a multiple of n_kv_heads with
 *     at most 8 query heads per KV head; n_max <= bpc_max_context(cfg).
 */
#ifndef BPC_H_
#define BPC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  BPC_OK = 0,
  BPC_ERR_INVALID_ARG = 1,   /* null / misaligned pointer, bad size */
  BPC_ERR_UNSUPPORTED = 2,   /* shape or mode outside the limits above */
  BPC_ERR_CAPACITY = 3,      /* a sequence would exceed n_max; nothing was written */
  BPC_ERR_NOT_FITTED = 4,    /* a call needs the projection before bpc_fit / bpc_set_projection */
  BPC_ERR_CUDA = 5,          /* a CUDA runtime call failed (see bpc_last_cuda_error) */
  BPC_ERR_DEVICE = 6,        /* a kernel reported an internal error through the device error word */
  BPC_ERR_SCRATCH_LIMIT = 7  /* bpc_decode_attn_static only: the shape needs more than the built-in scratch array */
} bpc_status;

typedef enum { BPC_BF16 = 0, BPC_F32 = 1 } bpc_dtype;

/* Algorithm 3 with one magnitude plane (all magnitudes 1: Hamming similarity) or the paper's
 * sign + seven magnitude planes. */
typedef enum { BPC_SCORE_HAMMING = 0, BPC_SCORE_WEIGHTED7 = 1 } bpc_score_mode;

typedef struct {
  int32_t batch;
  int32_t n_q_heads;
  int32_t n_kv_heads;
  int32_t head_dim;             /* 128 */
  int32_t code_bits;            /* 32 | 64 | 128 | 256 (with 32, n_max must be a multiple of 4) */
  int32_t n_max;                /* rows per unit in the caches and the code array */
  int32_t kv_dtype;             /* bpc_dtype */
  int32_t score_mode;           /* bpc_score_mode */
  float   sm_scale;             /* softmax scale; 0 selects 1/sqrt(head_dim) */
  int32_t hash_sets;            /* batch*n_kv_heads (one projection per unit) or n_kv_heads (shared per KV head) */
  int32_t residual_correction;  /* 1: Algorithm 2 (default). 0: plain sign(k P^T), for comparison only */
  int32_t kv_row_stride;        /* elements between consecutive cache rows; 0 selects head_dim */
  int32_t eas_ppm;              /* error-aware safeguard: size of the hard-to-hash set as parts per million of the
                                   keys cached when bpc_build_eas runs (0 = no safeguard; at most 16384 keys per unit) */
  int32_t fit_power_iters;      /* bpc_fit: n in u = sign((R R^T)^n R v*^T), 0..8; 0 is Algorithm 1 as printed */
} bpc_config;

typedef struct bpc_ctx bpc_ctx;

/* Context life cycle.  bpc_create validates cfg, allocates the projection, Gram matrix, per-unit
 * lengths, a selected-index scratch list and the device error word on the current device. */
bpc_status bpc_create(const bpc_config* host_cfg, bpc_ctx** host_out);
bpc_status bpc_destroy(bpc_ctx* ctx);

/* Sizes the caller needs: bytes of the code array, bytes of the workspace bpc_fit needs, the largest
 * n_max this build supports for cfg, and the most keys a decode step can select per unit (= n_max).  Normally the
 * scores of one unit are kept in the shared memory of one thread block cluster (up to about 1.3 M keys per unit);
 * longer units are served, for Hamming scores without the safeguard, by a streaming selection that stores no scores
 * and reads the codes twice (n_max up to 2^26); the weighted score mode and the safeguard keep the cluster limit. */
size_t  bpc_codes_bytes(const bpc_config* host_cfg);
size_t  bpc_fit_workspace_bytes(const bpc_config* host_cfg);
/* Byte offset inside the fit workspace at which bpc_fit leaves the codes H that Algorithm 1 itself
 * assigns to the fitted keys ([units][n_max][code_bits/64] uint64, same bit layout as `codes`).  They are a
 * diagnostic: the cache codes always come from Algorithm 2 (bpc_encode_keys). */
size_t  bpc_fit_codes_offset(const bpc_config* host_cfg);
int64_t bpc_max_context(const bpc_config* host_cfg);

/* Current number of cached keys of every sequence (host array [batch]).  Setting it stages the per-unit lengths in
 * pinned memory owned by the context and copies them to the device asynchronously on `stream` (no wait for the stream;
 * host_lens may be reused as soon as the call returns).  Eight calls can be in flight; a ninth waits for the first
 * one's copy.  The context keeps a host shadow that bpc_append advances, so capacity errors are raised before any
 * launch. */
bpc_status bpc_set_seq_lens(bpc_ctx* ctx, const int32_t* host_lens, void* stream);
bpc_status bpc_get_seq_lens(bpc_ctx* ctx, int32_t* host_lens_out);

/* Algorithm 1 (Section 3.2, "Binary Principal Components Finding"): for every unit, run code_bits
 * greedy iterations on its first seq_len keys of k_cache.  v_star [hash_sets][code_bits][head_dim]
 * float are the Gaussian directions the algorithm samples (supplied by the caller so that a run is
 * reproducible).  workspace must hold bpc_fit_workspace_bytes(cfg).  Requires hash_sets ==
 * batch*n_kv_heads.  Leaves P, P rounded to the cache precision (the hash function proper) and
 * its Gram matrix in the context.  With cfg.fit_power_iters = n > 0 the binary component comes from the power
 * iteration the same section starts from, u = sign((R R^T)^n R v*^T) = sign(R (R^T R)^n v*^T): the head_dim x head_dim
 * matrix R^T R is formed once (one extra pass over the keys) and then follows the residual by the rank-one change
 * -N v^T v per iteration, so the passes over R stay one per bit. */
bpc_status bpc_fit(bpc_ctx* ctx, const void* k_cache, const float* v_star,
                   void* workspace, size_t workspace_bytes, void* stream);

/* Offline-calibrated projection (Section 3.2, "Offline Projection Calibration"): install a caller
 * supplied P [hash_sets][code_bits][head_dim] float instead of fitting. */
bpc_status bpc_set_projection(bpc_ctx* ctx, const float* P, void* stream);

/* Copy out the projection (float), its cache-precision rounding as float values, and the Gram
 * matrix [hash_sets][code_bits][code_bits] float.  Any pointer may be NULL. */
bpc_status bpc_get_projection(bpc_ctx* ctx, float* P_out, float* P_hash_out, float* gram_out, void* stream);

/* Algorithm 2 for the first seq_len keys of every unit: codes[unit][0..seq_len). */
bpc_status bpc_encode_keys(bpc_ctx* ctx, const void* k_cache, uint64_t* codes, void* stream);

/* Error-Aware Safeguard (Section 3.2, Eqs. 8-9).  With cfg.eas_ppm > 0, bpc_encode_keys also records every
 * key's reconstruction error ||k - h P_h||_2 (squared), and bpc_build_eas, called once after it, keeps per unit the
 * m = ceil(seq_len * eas_ppm / 1e6) keys with the largest error (ties to the lowest index) as the static set S_err.
 * From then on a decode step with budget k always attends the first min(m, k) keys of S_err and lets the hash search
 * fill the other k - min(m, k) places; keys found by both are attended once.  With sel_idx given, entries
 * [0, k - min(m,k)) are the hash-selected keys (ascending) and the following min(m, k) entries are S_err in ascending
 * order with -1 in place of keys the hash search already selected.  Keys appended later never join S_err.
 * Requires residual_correction = 1 and Hamming scores.  bpc_get_eas copies out the squared errors [units][n_max] float, the set
 * [units][eas_capacity] int32 and its sizes [units] int32 (any pointer may be NULL). */
bpc_status bpc_build_eas(bpc_ctx* ctx, void* stream);
bpc_status bpc_get_eas(bpc_ctx* ctx, float* sq_err_out, int32_t* set_out, int32_t* count_out, void* stream);
int32_t    bpc_eas_capacity(const bpc_config* host_cfg);

/* Cache write of one new (k, v) row per unit at position seq_len, Algorithm 2 on the new key, its
 * code stored beside the others, seq_len += 1 (on the device and in the host shadow).
 * Returns BPC_ERR_CAPACITY, with nothing written, if any sequence is already at n_max. */
bpc_status bpc_append(bpc_ctx* ctx, const void* k_new, const void* v_new,
                      void* k_cache, void* v_cache, uint64_t* codes, void* stream);

/* One decode step (Section 3.2 "Retrieval Phase", Algorithm 3, Appendix "CUDA Optimizations"):
 * hash the queries of each KV head, score every cached key of the unit, keep the k keys with the
 * highest score (ties to the lowest index) and write softmax(sm_scale q K_S^T) V_S for every query
 * head.  k = budget_count if > 0 else ceil(seq_len * budget_ppm / 1e6), never more than seq_len;
 * it is computed on the device from the device-side lengths.  sel_idx, if not NULL, receives the
 * selected indices of each unit in ascending order, [units][n_max] int32 (first k entries). */
bpc_status bpc_decode_attn(bpc_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                           const uint64_t* codes, int32_t budget_ppm, int32_t budget_count,
                           float* out, int32_t* sel_idx, void* stream);

/* bpc_append followed by bpc_decode_attn as ONE launch (the two calls of a decode step, fused): the block of
 * each unit's cluster that owns the new position writes the (k, v) rows, codes the new key in one of its warps
 * while the other warps scan the old codes, scores it, and advances the length; the step's selection and
 * attention then see n+1 keys exactly as after a separate bpc_append.  Same arguments, layouts, limits and
 * errors as the two calls it replaces (BPC_ERR_CAPACITY, with nothing launched, if any sequence is at n_max). */
bpc_status bpc_append_decode_attn(bpc_ctx* ctx, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                                  uint64_t* codes, const void* q, int32_t budget_ppm, int32_t budget_count,
                                  float* out, int32_t* sel_idx, void* stream);

/* The same decode step for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this is a property of the library, not of the method.)
 *
 * Who needs it: a plug-in inside a serving process whose memory pool has already taken the whole device, or
 * code that may run while another thread has a stream capture open; neither can call cudaMalloc, so neither
 * can use bpc_create.  This call takes no context, makes no cudaMalloc / cudaFree / allocating library call,
 * and keeps the two things the regular call gets from its context - the selected-index list and the device
 * error word - in a fixed array compiled into the library (4 MiB + 256 B, held by every device that loads the
 * library until the process exits).
 *
 * The caller passes every input and the output: cfg (host; same meaning and limits as for bpc_create, Hamming
 * scores only), q, k_cache, v_cache, codes, out as for bpc_decode_attn; P_hash = the hash projection rounded to
 * the cache dtype, [hash_sets][code_bits][head_dim] kv_dtype (what bpc_get_projection reports as P_hash_out,
 * stored in kv_dtype); unit_lens = number of cached keys per unit, [batch*n_kv_heads] int32 on the device.
 * cfg.eas_ppm must be 0 (the safeguard set belongs to a context).
 *
 * Limits and hazards
 *   - batch * n_kv_heads * n_max must not exceed bpc_static_scratch_entries() (1 Mi index entries); larger
 *     shapes return BPC_ERR_SCRATCH_LIMIT and launch nothing.
 *   - All calls on one device share the array.  Calls that can overlap on the GPU (different streams without
 *     an ordering between them) race on it; order them on one stream or with events.
 *   - The array keeps the previous call's contents.  The call clears the error word itself (asynchronously, on
 *     `stream`) before launching; the index list needs no clearing because each unit's entries are written
 *     before they are read.
 *   - The first call on each device looks up the array's device address and sets the kernel's launch
 *     attributes; make that first call outside any stream capture. */
bpc_status bpc_decode_attn_static(const bpc_config* host_cfg, const void* q, const void* k_cache, const void* v_cache,
                                  const uint64_t* codes, const void* P_hash, const int32_t* unit_lens,
                                  int32_t budget_ppm, int32_t budget_count, float* out, void* stream);
size_t     bpc_static_scratch_entries(void);
/* The error word of the last bpc_decode_attn_static call on the current device (it lives in the same built-in array):
 * copies it to *host_out, waits for `stream`, and returns BPC_ERR_DEVICE when it is non-zero.  Allocates nothing. */
bpc_status bpc_static_last_device_error(int32_t* host_out, void* stream);

/* Quality yard-stick: the exact-score selector (appendix "Baseline Methods", TOPK (Oracle)).  For every query head,
 * scores[(seq * n_q_heads + head)][i] = q_head . k_i over the cached keys (fp32) and the k keys with the largest
 * scores (k from the budget as in bpc_decode_attn; ties to the lowest index) in ascending index order in
 * sel_out[(seq * n_q_heads + head)][0..k), with k in count_out[seq * n_q_heads + head].  scores (float) and sel_out
 * (int32) are device arrays [batch * n_q_heads][n_max], count_out int32 [batch * n_q_heads]; q and k_cache as for
 * bpc_decode_attn.  An evaluation aid: it reads every key row.  The other yard-stick, dense attention over all cached
 * keys, is bpc_decode_attn with budget_ppm = 1000000. */
bpc_status bpc_exact_topk(bpc_ctx* ctx, const void* q, const void* k_cache, int32_t budget_ppm, int32_t budget_count,
                          float* scores, int32_t* sel_out, int32_t* count_out, void* stream);

/* Parity aids.  When set (non-NULL), the next bpc_decode_attn calls also write the integer hash
 * score of every cached key (scores [units][n_max] int32) and the collapsed integer query weights
 * A = sum over the group's heads of sign*magnitude (qweights [units][code_bits] int32). */
bpc_status bpc_debug_set_buffers(bpc_ctx* ctx, int32_t* scores, int32_t* qweights);

/* Tracing aid.  When set (non-NULL), every thread block of the next bpc_decode_attn calls writes time stamps at
 * its phase boundaries into a row of 16 slots.  Slots 0 and 7 hold %globaltimer (ns) at the block's start and end,
 * slots 15 and 14 the SM cycle counter at the same two points (which gives the block's ns per cycle); every other
 * slot holds the cycle counter: 1 query hash done, 2 scan done, 8 histograms complete (cluster barrier passed),
 * 9 threshold known, 10 output offsets known, 3 selection done, 4 index list visible, 5 attention done, 6 block
 * merge done; in the block that appends a key also 12 / 11 sign sweep started / finished and 13 its scanning warps
 * done.  stamps [units * cluster_size][16] uint64. */
bpc_status bpc_debug_set_phase_timer(bpc_ctx* ctx, uint64_t* stamps);

/* Launch geometry of the decode kernel: thread blocks per cluster, any size from 1 to 16 that the device schedules
 * (0 = choose automatically: the largest size that keeps all units' clusters resident at once).
 * Returns BPC_ERR_UNSUPPORTED if n_max does not fit that many blocks or the device cannot schedule the size. */
bpc_status bpc_set_cluster_size(bpc_ctx* ctx, int32_t cluster_size);
/* The automatic choice as a pure host function (no device is touched): the cluster size bpc_create would take for
 * `cfg` on a device whose limits are given by the caller.  max_active (host, 17 entries) holds at index c = 1 .. 16 how
 * many clusters of c blocks the device keeps resident at once (0 = size not schedulable; entry 0 is ignored);
 * chunk_cap = score keys one block's shared memory holds.  Candidates are the sizes whose blocks hold n_max scores
 * and, above the smallest such size, keep at least 1024 keys per block; the result minimises
 * waves x (keys per block + 600 x size + 4000 x eight-row attention tiles per warp at a nominal budget of
 * max(2 % of n_max, 1024) + 20000), waves = ceil(units / max_active[size]).  Returns 0 when no size fits (the
 * streaming selection then applies) or an argument is invalid. */
int32_t    bpc_plan_cluster_size(const bpc_config* cfg, const int32_t* max_active, int32_t chunk_cap);
int32_t    bpc_get_cluster_size(bpc_ctx* ctx);
/* 1 when this context's decode calls use the streaming selection (units longer than a cluster's shared memory holds). */
int32_t    bpc_uses_streaming(bpc_ctx* ctx);

/* A second decode kernel, kept as an alternative that can be selected per context.  (The paper has no counterpart: it is
 * a different schedule for the same step.)  For bf16 caches with Hamming scores and no safeguard (at most 512 units) a
 * decode call can run as ONE launch of a persistent grid (two blocks per SM) whose blocks take work items from global
 * counters: per unit one cache-write item (fused call) and one query-hash item per 32 code bits, then code-scan items
 * of a fixed number of keys and attention items over at most a fixed number of selected rows of one key range.
 * Scores (2 bytes per cached key), range histograms, per-range offsets and attention partials of a step live in
 * scratch memory that the first bpc_debug_set_decode_path(ctx, 2) allocates.  The selection is identical to the
 * cluster kernel's and the output equal up to the summation order of the attention partials; any context length up to
 * 2^25 keys is covered without the streaming selection.  On B200 it is slower than the cluster kernel on every
 * configuration measured (hand-overs between items go through L2), so it is never chosen automatically.
 * bpc_debug_set_decode_path: 0 or 1 = cluster kernel (default), 2 = work-item kernel (BPC_ERR_UNSUPPORTED if the
 * context is not covered).  bpc_uses_work_items: 1 when this context's decode calls take that kernel.
 * bpc_work_item_grid: its resident blocks.
 * bpc_debug_set_work_item_geometry: keys per scan item (a multiple of 1792; 0 = automatic) and the most selected rows
 * per attention item (<= 512; 0 = automatic).
 * bpc_debug_set_work_item_trace: when set (non-NULL), every block records the items it ran: trace [blocks][64][12] uint64
 * = (item type << 40 | unit << 24 | index, start ns, end ns, six time stamps inside the item, unused), types 1 cache
 * write, 2 query hash, 3 scan, 4 attention, 5 threshold, 6 merge. */
int32_t    bpc_uses_work_items(bpc_ctx* ctx);
int32_t    bpc_work_item_grid(bpc_ctx* ctx);
bpc_status bpc_debug_set_decode_path(bpc_ctx* ctx, int32_t path);
bpc_status bpc_debug_set_work_item_geometry(bpc_ctx* ctx, int32_t keys_per_scan_item, int32_t rows_per_attend_item);
bpc_status bpc_debug_set_work_item_trace(bpc_ctx* ctx, uint64_t* trace);

/* Diagnostics.  bpc_last_device_error copies the device error word to *host_out; it is the one call that waits for
 * `stream` (it returns a host value), and it returns BPC_ERR_DEVICE when the word is non-zero (bit 0: a unit did not
 * fit the cluster's score storage, bit 1: append at n_max, bit 2: a bounded wait inside a kernel gave up), BPC_OK
 * otherwise.  bpc_status_of_device_error is that mapping as a pure function.  Then: last CUDA error code seen by the
 * context, number of kernels this context has launched so far.
 * Diagnostic switches (explicit calls; the library reads no environment variable): bpc_debug_set_pdl(ctx, 0) launches
 * the decode kernel without programmatic dependent launch; bpc_debug_set_tensor_core_encode(ctx, 0) makes
 * bpc_encode_keys and the passes of bpc_fit take the CUDA-core kernels instead of the tensor-core ones; bpc_debug_force_streaming(ctx, 1) selects the streaming selection at any
 * context length (Hamming scores without the safeguard only) and re-plans the launch geometry;
 * bpc_debug_force_key_shift(ctx, s) with s in 0..2 stores weighted score keys shifted right by at least s bits (the
 * library does that by itself only when a query's largest possible score exceeds 16 bits), so that the exact
 * re-scoring of the keys at the threshold can be exercised at any shape. */
bpc_status bpc_status_of_device_error(int32_t error_word);
bpc_status bpc_debug_set_pdl(bpc_ctx* ctx, int32_t on);
bpc_status bpc_debug_force_key_shift(bpc_ctx* ctx, int32_t shift);
bpc_status bpc_debug_set_tensor_core_encode(bpc_ctx* ctx, int32_t on);
bpc_status bpc_debug_force_streaming(bpc_ctx* ctx, int32_t on);
/* Byte score keys.  Hamming scores with at most 256 distinct values (G*b/2 <= 255 for an even number G of query heads
 * per KV head, G*b <= 255 for an odd one; no safeguard) can be kept one byte per key in shared memory, which lets a
 * thread block hold 2.5 times as many keys.  The library takes that kernel variant by itself when the 16-bit keys
 * would need the streaming selection or more waves of clusters (bpc_uses_byte_keys reports the choice); the result is
 * the same bit for bit.  bpc_debug_force_byte_keys(ctx, 1) takes it wherever it is possible (BPC_ERR_UNSUPPORTED
 * where it is not), -1 never, 0 leaves the choice to the library; each call re-plans the launch geometry. */
int32_t bpc_uses_byte_keys(bpc_ctx* ctx);
bpc_status bpc_debug_force_byte_keys(bpc_ctx* ctx, int32_t mode);
bpc_status bpc_last_device_error(bpc_ctx* ctx, int32_t* host_out, void* stream);
int32_t    bpc_last_cuda_error(bpc_ctx* ctx);
int64_t    bpc_launch_count(bpc_ctx* ctx);
const char* bpc_version(void);

#ifdef __cplusplus
}
#endif
#endif /* BPC_H_ */
