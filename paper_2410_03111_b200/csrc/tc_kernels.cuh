// Tensor-core (tcgen05 / TMA) kernels of the library: interface used by the C ABI.
#pragma once

#include "common.cuh"

// Whether the tensor-core kernels cover this layer / cache combination.
bool lorc_tc_decode_supported(const lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv);
bool lorc_tc_append_supported(const lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, int T);

// Scratch bytes the tensor-core decode path needs for (batch, max_seq_len), any layer.
size_t lorc_tc_workspace_bytes(const lorc_ctx* ctx, int batch, int max_seq_len);

cudaError_t lorc_tc_decode(lorc_ctx* ctx, int layer, const LorcLayer& L, const CacheView& cv,
                           const bf16* q, bf16* out, int n_splits, void* ws, size_t ws_bytes,
                           cudaStream_t st, int* launches);
cudaError_t lorc_tc_append(lorc_ctx* ctx, int layer, const LorcLayer& L, const CacheView& cv,
                           const bf16* x, int T, cudaStream_t st, int* launches);

// Merge of split partials + value up-projection for LATENT layers with d_head = 128
// (same inputs and result as lorc_generic_combine).
cudaError_t lorc_fast_combine(const lorc_ctx* ctx, const LorcLayer& L, int batch, int n_splits,
                              const float* part_ml, const float* part_o, bf16* out, cudaStream_t st,
                              int* launches);

// Drop cached per-layer state (tensor maps) when factors are reloaded / the context dies.
void lorc_tc_invalidate_layer(lorc_ctx* ctx, int layer);
void lorc_tc_release(lorc_ctx* ctx);
