// Tensor-core (tcgen05 / TMA) kernels of the library: interface used by the C ABI.
#pragma once

#include <cuda.h>

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

// Softmax + P.C_V and value up-projection (tc_pv.cu).  scores [b, H_q, n_pad] (log2 units) and
// rowmax [b, H_q] (exact row maxima as order-preserving keys, see lorc_float_key; the PV kernel zeroes them again)
// come from the score kernel.
// mapCV: C_V cache in 64-column x 128-row (or page-sized) swizzled boxes; mapBVT: B_V^T [n, r_v] in swizzled
// boxes of 64 latent columns x 32 rows.  Launches the PV kernel and the up-projection kernel that writes `out`.
size_t lorc_tc_pv_scratch_bytes(const lorc_ctx* ctx, int batch, int max_seq_len);
cudaError_t lorc_tc_pv_launch(lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, const CUtensorMap& mapCV,
                              const CUtensorMap& mapBVT, const float* scores, unsigned* rowmax, int n_pad, int tiles,
                              int n_splits_hint, void* scratch, size_t scratch_bytes, bf16* out, cudaStream_t st,
                              int* launches);

// A_cat [D, R] (row-major) -> fragment order [R/8][D/32][32 lanes][8] used by the fast append kernel.  The first
// pair_cols columns (uncompressed mode with half-split rotary pairs: the key columns; otherwise 0) are laid out with the
// two members of each rotary pair side by side.
cudaError_t lorc_fast_retile_factor(const bf16* A_cat, bf16* A_tiled, int D, int R, int pair_cols, int d_head,
                                    cudaStream_t st);

// Drop cached per-layer state (tensor maps) when factors are reloaded / the context dies.
void lorc_tc_invalidate_layer(lorc_ctx* ctx, int layer);
void lorc_tc_release(lorc_ctx* ctx);

// Order-preserving map from finite floats (and infinities) to unsigned integers: a < b  <=>  key(a) < key(b).  No float
// maps to 0, so 0 can stand for "nothing yet" under an atomic maximum.
__device__ __forceinline__ unsigned lorc_float_key(float f) {
    const unsigned b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float lorc_key_float(unsigned k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
