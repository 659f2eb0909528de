// Fused decode kernel instantiations: bf16 caches, Hamming scores, streaming selection (units whose scores do not fit
// the cluster's shared memory).
#include "decode_launch.cuh"
cudaError_t bpc_launch_decode_bf16_stream(bpc_ctx* ctx, const DecodeParams& p, cudaStream_t stream) {
  return bpcdev::launch_dtype<__nv_bfloat16, 0, 2>(ctx, p, stream);
}
cudaError_t bpc_decode_limits_bf16_stream(const bpc_ctx* ctx, int nbins, int* max_cluster, int* chunk_cap, size_t* smem) {
  return bpcdev::limits_dtype<__nv_bfloat16, 0, 2>(ctx, nbins, max_cluster, chunk_cap, smem);
}
