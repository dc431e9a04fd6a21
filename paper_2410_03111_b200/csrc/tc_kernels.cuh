// Tensor-core (tcgen05 / TMA) kernels of the library: interface used by the C ABI.
#pragma once

#include <cuda.h>

#include "common.cuh"

// Whether the tensor-core kernels cover this layer / cache combination.
bool lorc_tc_decode_supported(const lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv);
bool lorc_tc_append_supported(const lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, int T);

// Scratch bytes the tensor-core decode path needs for (batch, max_seq_len), any layer.
size_t lorc_tc_workspace_bytes(const lorc_ctx* ctx, int batch, int max_seq_len);

// latent_out: `out` receives the normalised latent output [b, H_q, r_v] instead of the up-projected one.
// pos0, q_pos / ml_out: context shards (see lorc_decode_attn_shard): per sequence the position of the first cached row
// and of the query, and where to leave (reference, denominator) [b, H_q, 2] of the softmax over this shard.
cudaError_t lorc_tc_decode(lorc_ctx* ctx, int layer, const LorcLayer& L, const CacheView& cv,
                           const bf16* q, bf16* out, int n_splits, void* ws, size_t ws_bytes,
                           cudaStream_t st, int* launches, bool latent_out = false, const int32_t* pos0 = nullptr,
                           const int32_t* q_pos = nullptr, float* ml_out = nullptr);
cudaError_t lorc_tc_append(lorc_ctx* ctx, int layer, const LorcLayer& L, const CacheView& cv,
                           const bf16* x, int T, cudaStream_t st, int* launches);
// Cache write of compressed layers as a tcgen05 GEMM (tc_append.cu), for launches of at least 128 tokens.
bool lorc_tc_append_gemm_supported(const lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, int T);
cudaError_t lorc_tc_append_gemm(lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, const bf16* x, int T,
                                cudaStream_t st, int* launches);

// Bytes of one probability tile image (128 tokens of one sequence, all query heads): the bf16 numerators as the PV
// kernel's swizzled MMA operand, then float m[4][H_q] and float l[4][H_q] (reference and sum per 32-token quarter).
__host__ __device__ inline int lorc_tc_image_bytes(int n_q_heads) { return 2 * n_q_heads * 64 * 2 + 8 * n_q_heads * 4; }

// Score kernel (tc_score.cu): key reconstruction, rotation, q.k and the softmax numerators; writes one tile image per
// 128 tokens into pimg [b, tiles, image] and raises the row maxima (integers, as order-preserving keys).  rope_tile:
// the in-tile rotation table (33 x 32 float4, lorc_tc_rope_tile_fill).  Its first block clears zero[0 .. n_zero).
#define LORC_SCORE_MAX_BATCH 64      // sequences per launch (larger batches take several launches)
cudaError_t lorc_tc_score_set_attrs();
cudaError_t lorc_tc_rope_tile_fill(float2* table, double theta, cudaStream_t st);
cudaError_t lorc_tc_score_launch(lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, const CUtensorMap& mapCK,
                                 const CUtensorMap& mapBKT, const bf16* q, uint8_t* pimg, unsigned* rowmax,
                                 const float4* rope_tile, int tiles, int* zero, int n_zero, const int32_t* pos0,
                                 const int32_t* q_pos, cudaStream_t st, int* launches);

// Score kernel of layers without rotation (tc_absorbed.cu): the key up-projection is absorbed into the query
// (q~ = B_K q, written to `qabs`, lorc_tc_absorbed_scratch_bytes of scratch), the scores are a skinny GEMM over the
// latent keys.  Same outputs as lorc_tc_score_launch.
size_t lorc_tc_absorbed_scratch_bytes(const lorc_ctx* ctx, int batch);
cudaError_t lorc_tc_absorbed_set_attrs();
cudaError_t lorc_tc_score_absorbed_launch(lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, const CUtensorMap& mapCK,
                                          const bf16* q, bf16* qabs, uint8_t* pimg, unsigned* rowmax, int tiles, int* zero,
                                          int n_zero, cudaStream_t st, int* launches);

// P.C_V and value up-projection (tc_pv.cu).  mapCV: C_V cache in 64-column x 128-row (or page-sized) swizzled boxes;
// mapBVT: B_V^T [n, r_v] in swizzled boxes of 64 latent columns x 32 rows.  The plan says how a launch splits the
// work and where its pieces of scratch lie; the `done` words (plan.n_blk * batch ints at off_done) must be zero when
// the PV kernel starts.  The up-projection kernel writes `out` and leaves the row maxima empty again.
struct LorcPvPlan {
    int n_blk, n_csplit;
    bool fits;
    size_t off_on, off_done;
};
size_t lorc_tc_pv_scratch_bytes(const lorc_ctx* ctx, int batch, int max_seq_len);
cudaError_t lorc_tc_pv_set_attrs();
void lorc_tc_pv_plan(const lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, int n_splits_hint, size_t scratch_bytes,
                     LorcPvPlan* plan);
cudaError_t lorc_tc_pv_launch(lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, const CUtensorMap& mapCV,
                              const CUtensorMap& mapBVT, const uint8_t* pimg, unsigned* rowmax, int tiles,
                              const LorcPvPlan& plan, void* scratch, bf16* out, bool latent_out, float* ml_out,
                              cudaStream_t st, int* launches);

// Prompt processing (tc_prefill.cu): attention of the T newest tokens of every sequence (q, out [b, T, H_q, 128]) over
// the latent cache, causal inside the chunk.  Keys and values are reconstructed once into `scratch`
// (lorc_tc_prefill_scratch_bytes), then a flash-attention kernel runs over them.  mapBKT / mapBVT128: B_K^T, B_V^T
// [n, r] in swizzled boxes of 64 latent columns x 128 rows.
bool lorc_tc_prefill_supported(const lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv);
size_t lorc_tc_prefill_scratch_bytes(const lorc_ctx* ctx, int batch, int max_seq_len, int T);
cudaError_t lorc_tc_prefill_set_attrs();
cudaError_t lorc_tc_prefill_launch(lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, const CUtensorMap& mapCK,
                                   const CUtensorMap& mapCV, const CUtensorMap& mapBKT, const CUtensorMap& mapBVT128,
                                   const bf16* q, bf16* out, int T, void* scratch, cudaStream_t st, int* launches);
cudaError_t lorc_tc_prefill(lorc_ctx* ctx, int layer, const LorcLayer& L, const CacheView& cv, const bf16* q, bf16* out,
                            int T, void* ws, size_t ws_bytes, cudaStream_t st, int* launches);

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
