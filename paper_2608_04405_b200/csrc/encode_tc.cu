// Tensor-core encode (Algorithm 2 as a tcgen05 GEMM plus greedy sweep).  Placeholder until the kernel lands:
// reports "not supported" so that bpc_encode_keys takes the CUDA-core path.
#include "common.cuh"
cudaError_t bpc_launch_encode_tc(bpc_ctx*, const void*, uint64_t*, cudaStream_t) { return cudaErrorNotSupported; }
