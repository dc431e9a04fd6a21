// Placeholder until the tensor-core kernels land: nothing is supported yet.
#include "tc_kernels.cuh"
bool lorc_tc_decode_supported(const lorc_ctx*, const LorcLayer&, const CacheView&) { return false; }
bool lorc_tc_append_supported(const lorc_ctx*, const LorcLayer&, const CacheView&, int) { return false; }
size_t lorc_tc_workspace_bytes(const lorc_ctx*, int, int) { return 0; }
cudaError_t lorc_tc_decode(lorc_ctx*, int, const LorcLayer&, const CacheView&, const bf16*, bf16*, int, void*, size_t, cudaStream_t, int*) { return cudaErrorNotSupported; }
cudaError_t lorc_tc_append(lorc_ctx*, int, const LorcLayer&, const CacheView&, const bf16*, int, cudaStream_t, int*) { return cudaErrorNotSupported; }
void lorc_tc_invalidate_layer(lorc_ctx*, int) {}
void lorc_tc_release(lorc_ctx*) {}
