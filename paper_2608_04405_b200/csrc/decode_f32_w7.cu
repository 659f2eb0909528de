// Fused decode kernel instantiations: f32 caches, weighted scores (sign + seven magnitude planes, Algorithm 3).
#include "decode_launch.cuh"
cudaError_t bpc_launch_decode_f32_w7(bpc_ctx* ctx, const DecodeParams& p, cudaStream_t stream) {
  return bpcdev::launch_dtype<float, 1, 0>(ctx, p, stream);
}
cudaError_t bpc_decode_limits_f32_w7(const bpc_ctx* ctx, int nbins, int* max_cluster, int* chunk_cap, size_t* smem) {
  return bpcdev::limits_dtype<float, 1, 0>(ctx, nbins, max_cluster, chunk_cap, smem);
}
