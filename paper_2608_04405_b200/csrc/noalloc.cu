// bpc_decode_attn_static: the decode step for callers that must not allocate device memory.
//
// The regular bpc_decode_attn keeps its selected-index list and its device error word in buffers that
// bpc_create obtained with cudaMalloc.  A plug-in that lives inside a serving process whose memory pool has
// already claimed the whole device, or code that may run while some other thread has a stream capture open
// (an allocation would break that capture), cannot create such a context.  This entry point needs no context:
// the caller hands in every input (including the hash projection and the per-unit lengths) and the output,
// and the index list plus the error word live in a fixed array that is part of the library image itself.
//
// Consequences of the fixed array, all documented in bpc.h: there is one array per device, every call on that
// device uses it, so two calls that can overlap on the GPU (different streams, no dependency) race; shapes
// whose index list does not fit are refused; the array keeps whatever the previous call left in it.
#include <string.h>
#include "common.cuh"

cudaError_t bpc_launch_decode_bf16(bpc_ctx*, const DecodeParams&, cudaStream_t);
cudaError_t bpc_launch_decode_f32(bpc_ctx*, const DecodeParams&, cudaStream_t);

#define BPC_STATIC_HEADER_BYTES 256                       // error word, padded to the array's alignment
#define BPC_STATIC_LIST_BYTES (4u << 20)                  // index list: up to 1 Mi int32 entries (units * n_max)

// Held by every device that loads the library, until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[BPC_STATIC_HEADER_BYTES + BPC_STATIC_LIST_BYTES];

namespace {

constexpr int kMaxDevices = 64;
// Device address of g_static_scratch per device ordinal.  In host code the symbol's name is only a handle for
// the runtime, never a pointer a kernel could use: the address has to be asked for, with that device current.
void* g_scratch_addr[kMaxDevices] = {};

cudaError_t scratch_for_current_device(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
  if (g_scratch_addr[device] == nullptr) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[device] = p;
  }
  *out = g_scratch_addr[device];
  return cudaSuccess;
}

// keys per block the kernel may assign (the larger of its plain and its fused-launch split), rounded to 64
int chunk_for(int n_max, int cs) {
  const int plain = (((n_max + cs - 1) / cs) + 63) & ~63;
  if (cs == 1) return plain;
  const int fused = bpc_fused_chunk(n_max, cs);
  return fused > plain ? fused : plain;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

size_t bpc_static_scratch_entries(void) { return BPC_STATIC_LIST_BYTES / 4; }

bpc_status bpc_decode_attn_static(const bpc_config* cfg, const void* q, const void* k_cache, const void* v_cache,
                                  const uint64_t* codes, const void* P_hash, const int32_t* unit_lens,
                                  int32_t budget_ppm, int32_t budget_count, float* out, void* stream) {
  if (cfg == nullptr || q == nullptr || k_cache == nullptr || v_cache == nullptr || codes == nullptr ||
      P_hash == nullptr || unit_lens == nullptr || out == nullptr)
    return BPC_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(codes) || !aligned16(P_hash) ||
      !aligned16(out) || (reinterpret_cast<uintptr_t>(unit_lens) & 3u) != 0)
    return BPC_ERR_INVALID_ARG;
  if (cfg->batch < 1 || cfg->n_kv_heads < 1 || cfg->n_q_heads < 1 || cfg->n_max < 1 || cfg->n_max % 2 != 0)
    return BPC_ERR_INVALID_ARG;
  if (cfg->head_dim != BPC_D) return BPC_ERR_UNSUPPORTED;
  if (cfg->code_bits != 32 && cfg->code_bits != 64 && cfg->code_bits != 128 && cfg->code_bits != 256) return BPC_ERR_UNSUPPORTED;
  if (cfg->code_bits == 32 && cfg->n_max % 4 != 0) return BPC_ERR_INVALID_ARG;   // 16-byte aligned code rows per unit
  if (cfg->eas_ppm != 0) return BPC_ERR_UNSUPPORTED;        // the safeguard set lives in a context
  if (cfg->n_q_heads % cfg->n_kv_heads != 0) return BPC_ERR_INVALID_ARG;
  const int group = cfg->n_q_heads / cfg->n_kv_heads;
  if (group > BPC_MAX_GROUP) return BPC_ERR_UNSUPPORTED;
  if (cfg->kv_dtype != BPC_BF16 && cfg->kv_dtype != BPC_F32) return BPC_ERR_UNSUPPORTED;
  if (cfg->score_mode != BPC_SCORE_HAMMING) return BPC_ERR_UNSUPPORTED;
  const long long units = (long long)cfg->batch * cfg->n_kv_heads;
  if (cfg->hash_sets != units && cfg->hash_sets != cfg->n_kv_heads) return BPC_ERR_INVALID_ARG;
  if (cfg->kv_row_stride != 0 && (cfg->kv_row_stride < cfg->head_dim || cfg->kv_row_stride % 8 != 0))
    return BPC_ERR_INVALID_ARG;
  if (!(cfg->sm_scale >= 0.f)) return BPC_ERR_INVALID_ARG;
  if (budget_ppm < 0 || budget_ppm > 1000000 || budget_count < 0 || (budget_ppm == 0 && budget_count == 0))
    return BPC_ERR_INVALID_ARG;
  // the index list of all units must fit the fixed array
  if (units * (long long)cfg->n_max > (long long)(BPC_STATIC_LIST_BYTES / 4)) return BPC_ERR_SCRATCH_LIMIT;

  // a context on the stack: nothing in it is allocated, it only carries the launch geometry
  bpc_ctx tmp;
  memset(&tmp, 0, sizeof(tmp));
  tmp.cfg = *cfg;
  tmp.units = (int)units;
  tmp.group = group;
  tmp.row_stride = cfg->kv_row_stride == 0 ? cfg->head_dim : cfg->kv_row_stride;
  tmp.sm_scale_d = cfg->sm_scale == 0.f ? 0.08838834764831845 : (double)cfg->sm_scale;
  cudaError_t e = cudaGetDevice(&tmp.device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&tmp.sm_count, cudaDevAttrMultiProcessorCount, tmp.device);
  void* scratch = nullptr;
  if (e == cudaSuccess) e = scratch_for_current_device(tmp.device, &scratch);
  if (e != cudaSuccess) { (void)cudaGetLastError(); return BPC_ERR_CUDA; }

  const int nbins = ((group * cfg->code_bits) >> ((group % 2 == 0) ? 1 : 0)) + 1;
  if (nbins > 2048) return BPC_ERR_UNSUPPORTED;
  tmp.force_byte_keys = -1;                                 // this entry point launches the 16-bit-key kernel only
  e = bpc_plan_decode_geometry(&tmp);                       // occupancy queries only; nothing is allocated
  if (e != cudaSuccess) { (void)cudaGetLastError(); return BPC_ERR_CUDA; }
  // only the plain kernel is launched here: contexts too long for a cluster's shared memory (which a context would
  // serve with the streaming selection) are refused
  if (tmp.cluster_size == 0 || tmp.streaming || tmp.byte_keys) return BPC_ERR_UNSUPPORTED;
  const int cs = tmp.cluster_size;
  if (chunk_for(cfg->n_max, cs) > tmp.chunk_cap_limit) return BPC_ERR_UNSUPPORTED;

  // the error word accumulates with atomicOr, so it has to start at zero; the list is overwritten before use
  e = cudaMemsetAsync(scratch, 0, BPC_STATIC_HEADER_BYTES, (cudaStream_t)stream);
  if (e != cudaSuccess) { (void)cudaGetLastError(); return BPC_ERR_CUDA; }

  DecodeParams p;
  memset(&p, 0, sizeof(p));
  p.q = q; p.k_cache = k_cache; p.v_cache = v_cache; p.codes = codes; p.P_h = P_hash;
  p.unit_lens = unit_lens; p.out = out;
  p.err = reinterpret_cast<int32_t*>(scratch);
  p.sel = reinterpret_cast<int32_t*>(static_cast<unsigned char*>(scratch) + BPC_STATIC_HEADER_BYTES);
  p.n_kv_heads = cfg->n_kv_heads; p.group = group; p.n_max = cfg->n_max; p.row_stride = tmp.row_stride;
  p.shared_sets = cfg->hash_sets != units;
  p.budget_ppm = budget_ppm; p.budget_count = budget_count; p.sm_scale_d = tmp.sm_scale_d;
  p.chunk_cap = chunk_for(cfg->n_max, cs);
  p.nbins = nbins;
  e = cfg->kv_dtype == BPC_BF16 ? bpc_launch_decode_bf16(&tmp, p, (cudaStream_t)stream)
                                : bpc_launch_decode_f32(&tmp, p, (cudaStream_t)stream);
  if (e != cudaSuccess) { (void)cudaGetLastError(); return BPC_ERR_CUDA; }
  return BPC_OK;
}

bpc_status bpc_static_last_device_error(int32_t* host_out, void* stream) {
  if (host_out == nullptr) return BPC_ERR_INVALID_ARG;
  int device = 0;
  cudaError_t e = cudaGetDevice(&device);
  void* scratch = nullptr;
  if (e == cudaSuccess) e = scratch_for_current_device(device, &scratch);
  if (e == cudaSuccess) e = cudaMemcpyAsync(host_out, scratch, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) { (void)cudaGetLastError(); return BPC_ERR_CUDA; }
  return *host_out == 0 ? BPC_OK : BPC_ERR_DEVICE;
}

#pragma GCC visibility pop
}  // extern "C"
