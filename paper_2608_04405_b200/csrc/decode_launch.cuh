// Host-side dispatch of the fused decode kernel for one cache dtype (included by decode_bf16.cu / decode_f32.cu).
#pragma once
#include "decode_kernel.cuh"

#include <atomic>

namespace bpcdev {

// The shared-memory ceiling is always raised to the device's opt-in maximum, so contexts with different
// n_max can share one kernel instance.
template <typename KV, int GP, int W32, int MODE, int EAS>
static cudaError_t configure_kernel(int device) {
  auto kern = bpc_decode_kernel<KV, GP, W32, MODE, EAS>;
  int optin = 0;
  cudaError_t e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, optin);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
}

template <typename KV, int GP, int W32, int MODE, int EAS>
static cudaError_t launch_one(bpc_ctx* ctx, const DecodeParams& p_in, cudaStream_t stream) {
  typedef DecodeSmem<KV, GP, W32> L;
  DecodeParams p = p_in;
  int optin = 0;
  cudaError_t e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, ctx->device);
  if (e != cudaSuccess) return e;
  constexpr int kKeyBytes = EAS == 3 ? 1 : 2;               // (variant 3 stores byte score keys)
  p.stages = L(p.chunk_cap, p.nbins, 3, kKeyBytes).total <= (size_t)optin ? 3 : 2;
  const size_t smem = L(p.chunk_cap, p.nbins, p.stages, kKeyBytes).total;
  if (smem > (size_t)optin) return cudaErrorInvalidConfiguration;
  if (ctx->decode_smem_set == 0) {                          // function attributes are sticky: set them once
    e = configure_kernel<KV, GP, W32, MODE, EAS>(ctx->device);
    if (e != cudaSuccess) return e;
    ctx->decode_smem_set = 1;
  }
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3((unsigned)(ctx->units * ctx->cluster_size), 1, 1);
  lc.blockDim = dim3(L::NT, 1, 1);
  lc.dynamicSmemBytes = smem;
  lc.stream = stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)ctx->cluster_size;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  // let the grid be scheduled while the previous kernel of the stream drains (the kernel waits for that
  // kernel's completion itself before it reads anything)
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = ctx->use_pdl ? 2 : 1;
  return cudaLaunchKernelEx(&lc, bpc_decode_kernel<KV, GP, W32, MODE, EAS>, p);
}

// Largest cluster size the device can schedule with a full-size block, and the number of score keys one block can
// hold next to a two-stage gather ring.
template <typename KV, int GP, int W32, int MODE, int EAS>
static cudaError_t limits_one(const bpc_ctx* ctx, int nbins, int* max_cluster, int* chunk_cap, size_t* smem_bytes) {
  typedef DecodeSmem<KV, GP, W32> L;
  int dev = ctx->device, optin = 0;
  cudaError_t e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  const size_t fixed = L(0, nbins, 2).off_union;
  const size_t avail = (size_t)optin > fixed + 64 ? (size_t)optin - fixed - 64 : 0;
  constexpr int kKeyBytes = EAS == 3 ? 1 : 2;
  int cap = kKeyBytes == 1 ? (int)(avail > 0x3fffffff ? 0x3fffffff : avail) : (int)((avail / (kSegSlots * 2)) * kSegKeys);
  cap &= ~63;
  if (L(cap, nbins, 2, kKeyBytes).total > (size_t)optin) cap = 0;
  if (chunk_cap) *chunk_cap = cap;
  if (smem_bytes) *smem_bytes = (size_t)optin;
  if (max_cluster) {
    // max_cluster[0] = largest schedulable cluster size; max_cluster[cs] = clusters of size cs that can be resident
    // at once (a grid with more clusters than that runs in several waves), cs = 1 .. BPC_MAX_CLUSTER
    // The answers depend on the kernel and the device only: they are kept per instantiation for the first device
    // asked about (published with a release store once complete), so that contexts and the allocation-free entry
    // point do not repeat the sixteen occupancy queries.
    static std::atomic<int> cached_dev(-1);
    static int cached[BPC_MAX_CLUSTER + 1];
    if (cached_dev.load(std::memory_order_acquire) == dev) {
      for (int i = 0; i <= BPC_MAX_CLUSTER; ++i) max_cluster[i] = cached[i];
      return cudaSuccess;
    }
    int best = 1;
    e = configure_kernel<KV, GP, W32, MODE, EAS>(dev);
    if (e != cudaSuccess) return e;
    for (int cs = 1; cs <= BPC_MAX_CLUSTER; ++cs) {
      cudaLaunchConfig_t lc = {};
      lc.gridDim = dim3((unsigned)cs, 1, 1);
      lc.blockDim = dim3(L::NT, 1, 1);
      lc.dynamicSmemBytes = (size_t)optin;
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = (unsigned)cs; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
      lc.attrs = at; lc.numAttrs = 1;
      int nclusters = 0;
      cudaError_t q = cudaOccupancyMaxActiveClusters(&nclusters, bpc_decode_kernel<KV, GP, W32, MODE, EAS>, &lc);
      if (q != cudaSuccess) { (void)cudaGetLastError(); nclusters = 0; }
      max_cluster[cs] = nclusters;
      if (nclusters >= 1) best = cs;
    }
    max_cluster[0] = best;
    static std::atomic<int> claimed(0);
    if (claimed.exchange(1) == 0) {                           // the first caller publishes
      for (int i = 0; i <= BPC_MAX_CLUSTER; ++i) cached[i] = max_cluster[i];
      cached_dev.store(dev, std::memory_order_release);
    }
  }
  return cudaSuccess;
}

#define BPC_DISPATCH_W(KV, GP, MODE, EAS, FN, ...)                                   \
  switch (ctx->cfg.code_bits) {                                                      \
    case 32:  return FN<KV, GP, 1, MODE, EAS>(__VA_ARGS__);                          \
    case 64:  return FN<KV, GP, 2, MODE, EAS>(__VA_ARGS__);                          \
    case 128: return FN<KV, GP, 4, MODE, EAS>(__VA_ARGS__);                          \
    case 256: return FN<KV, GP, 8, MODE, EAS>(__VA_ARGS__);                          \
    default:  return cudaErrorInvalidValue;                                          \
  }

#define BPC_DISPATCH_G(KV, MODE, EAS, FN, ...)                                       \
  if (ctx->group == 1)      { BPC_DISPATCH_W(KV, 1, MODE, EAS, FN, __VA_ARGS__) }    \
  else if (ctx->group == 2) { BPC_DISPATCH_W(KV, 2, MODE, EAS, FN, __VA_ARGS__) }    \
  else if (ctx->group <= 4) { BPC_DISPATCH_W(KV, 4, MODE, EAS, FN, __VA_ARGS__) }    \
  else                      { BPC_DISPATCH_W(KV, 8, MODE, EAS, FN, __VA_ARGS__) }

// One translation unit per (cache dtype, score mode): MODE 0 = Hamming, MODE 1 = sign + 7 magnitude planes.
template <typename KV, int MODE, int EAS>
static cudaError_t launch_dtype(bpc_ctx* ctx, const DecodeParams& p, cudaStream_t stream) {
  BPC_DISPATCH_G(KV, MODE, EAS, launch_one, ctx, p, stream)
}
template <typename KV, int MODE, int EAS>
static cudaError_t limits_dtype(const bpc_ctx* ctx, int nbins, int* max_cluster, int* chunk_cap, size_t* smem) {
  BPC_DISPATCH_G(KV, MODE, EAS, limits_one, ctx, nbins, max_cluster, chunk_cap, smem)
}

}  // namespace bpcdev
