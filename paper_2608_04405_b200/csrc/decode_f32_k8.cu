// Fused decode kernel instantiations: f32 caches, Hamming scores kept as byte keys (at most 256 distinct scores), for
// contexts whose 16-bit keys would not fit clusters that are all resident at once.
#include "decode_launch.cuh"
cudaError_t bpc_launch_decode_f32_k8(bpc_ctx* ctx, const DecodeParams& p, cudaStream_t stream) {
  return bpcdev::launch_dtype<float, 0, 3>(ctx, p, stream);
}
cudaError_t bpc_decode_limits_f32_k8(const bpc_ctx* ctx, int nbins, int* max_cluster, int* chunk_cap, size_t* smem) {
  return bpcdev::limits_dtype<float, 0, 3>(ctx, nbins, max_cluster, chunk_cap, smem);
}
