// Fused decode kernel instantiations for bf16 caches.
#include "decode_launch.cuh"
cudaError_t bpc_launch_decode_bf16(bpc_ctx* ctx, const DecodeParams& p, cudaStream_t stream) {
  return bpcdev::launch_dtype<__nv_bfloat16>(ctx, p, stream);
}
cudaError_t bpc_decode_limits_bf16(const bpc_ctx* ctx, int cs, int* max_cluster, int* chunk_cap, size_t* smem) {
  return bpcdev::limits_dtype<__nv_bfloat16>(ctx, cs, max_cluster, chunk_cap, smem);
}
