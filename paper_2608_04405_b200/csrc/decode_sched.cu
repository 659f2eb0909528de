// Host side of the work-item decode kernel (decode_sched.cuh): geometry, scratch sizes, launch.  bf16 caches,
// Hamming scores.
#include "decode_sched.cuh"
#include "sched_host.h"

namespace bpcdev {

// Eight warps per block (seven that score and attend, one producer), two blocks per SM: four warps per scheduler is
// the most that leaves every thread 128 registers (the register file is split over the four schedulers), which the
// attention items need, and two independent blocks per SM hide each other's serial latencies (fences, L2 round trips,
// block barriers).
#ifndef BPC_SCHED_NC
#define BPC_SCHED_NC 224
#endif
constexpr int kNC = BPC_SCHED_NC;                 // scoring threads per block (plus one producer warp)
constexpr int kMinBlocks = kNC >= 384 ? 1 : 2;    // blocks per SM the register budget is sized for

template <int GP, int W32>
static cudaError_t sched_configure(int device, size_t smem, int* blocks_per_sm) {
  auto kern = bpc_decode_sched_kernel<GP, W32, kNC, kMinBlocks>;
  int optin = 0;
  cudaError_t e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
  if (e != cudaSuccess) return e;
  if (smem > (size_t)optin) return cudaErrorInvalidConfiguration;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int nb = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, kern, kNC + 32, smem);
  if (e != cudaSuccess) return e;
  *blocks_per_sm = nb;
  return cudaSuccess;
}

template <int GP, int W32>
static cudaError_t sched_launch(const SchedParams& p, int grid, size_t smem, bool pdl, cudaStream_t stream) {
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3((unsigned)grid, 1, 1);
  lc.blockDim = dim3(kNC + 32, 1, 1);
  lc.dynamicSmemBytes = smem;
  lc.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&lc, bpc_decode_sched_kernel<GP, W32, kNC, kMinBlocks>, p);
}

template <int GP, int W32>
static size_t sched_smem(int nbins, int units) {
  return SchedSmem<GP, W32, kNC>(nbins, units, 0).total;
}

#define SCHED_DISPATCH_W(GP, FN, ...)                     \
  switch (w32) {                                          \
    case 1: return FN<GP, 1>(__VA_ARGS__);                \
    case 2: return FN<GP, 2>(__VA_ARGS__);                \
    case 4: return FN<GP, 4>(__VA_ARGS__);                \
    case 8: return FN<GP, 8>(__VA_ARGS__);                \
    default: break;                                       \
  }
#define SCHED_DISPATCH(FN, FAIL, ...)                                      \
  if (group == 1)      { SCHED_DISPATCH_W(1, FN, __VA_ARGS__) }            \
  else if (group == 2) { SCHED_DISPATCH_W(2, FN, __VA_ARGS__) }            \
  else if (group <= 4) { SCHED_DISPATCH_W(4, FN, __VA_ARGS__) }            \
  else                 { SCHED_DISPATCH_W(8, FN, __VA_ARGS__) }            \
  return FAIL;

static cudaError_t dispatch_configure(int group, int w32, int device, size_t smem, int* nb) {
  SCHED_DISPATCH(sched_configure, cudaErrorInvalidValue, device, smem, nb)
}
static cudaError_t dispatch_launch(int group, int w32, const SchedParams& p, int grid, size_t smem, bool pdl, cudaStream_t s) {
  SCHED_DISPATCH(sched_launch, cudaErrorInvalidValue, p, grid, smem, pdl, s)
}
static size_t dispatch_smem(int group, int w32, int nbins, int units) {
  SCHED_DISPATCH(sched_smem, 0, nbins, units)
}

}  // namespace bpcdev

int bpc_sched_threads(void) { return bpcdev::kNC; }

int bpc_sched_padded_group(int group) { return group == 1 ? 1 : (group == 2 ? 2 : (group <= 4 ? 4 : 8)); }

int bpc_sched_granule(int code_bits) {
  (void)code_bits;
  return bpcdev::kNC * 8;                         // two scan batches of 256-bit codes, one of shorter codes
}

cudaError_t bpc_sched_configure(int group, int code_bits, int nbins, int units, int device, size_t* smem, int* blocks_per_sm) {
  *smem = bpcdev::dispatch_smem(group, code_bits / 32, nbins, units);
  if (*smem == 0) return cudaErrorInvalidValue;
  return bpcdev::dispatch_configure(group, code_bits / 32, device, *smem, blocks_per_sm);
}

cudaError_t bpc_sched_launch(int group, int code_bits, const bpcdev::SchedParams& p, int grid, size_t smem, bool pdl,
                             cudaStream_t stream) {
  return bpcdev::dispatch_launch(group, code_bits / 32, p, grid, smem, pdl, stream);
}
