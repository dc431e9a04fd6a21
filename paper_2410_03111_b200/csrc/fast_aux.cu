// Bandwidth-bound helper of the fast path: latent cache write for a handful of tokens (decode) or chunks of tokens (prefill):
//     C = x [A_K | A_V], a skinny GEMM whose cost is streaming the factor once.  Warp-level
//     mma.sync (M = 16 tokens) is the natural tile here: a 128-row tcgen05 tile would be
//     7/8 padding at decode batch sizes, and the kernel is bound by the weight stream.
#include "common.cuh"
#include "sm100_ptx.cuh"
#include "tc_kernels.cuh"

namespace {

// ---------------------------------------------------------------------------------------------
// append: grid (R/8, token tiles of 16); 8 warps = 8 slices of D for one tile of 8 columns.
// Operands: x [n_tok, D] row-major and the factor in fragment order A_tiled[R/8][D/32][lane][8]: for the
// tile of 8 columns n0.. and the block of 32 k values kb, lane (g = lane/4, t = lane%4) owns the 8
// consecutive k = 32 kb + 8 t .. of column n0 + g, so a warp reads one contiguous 512-byte block per
// step.  Those 8 values fill the fragment slots of two m16n8k16 steps; x is loaded with the same slot
// order, so the contraction is unchanged.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// FULL (uncompressed mode): the factor is [W_K | W_V] and keys are cached rotated.  The key columns of the tiled
// factor are permuted (see retile_factor_kernel) so that the two accumulator columns a thread ends up with are the two
// members of one rotary pair: the rotation needs no exchange between threads.
template <bool FULL>
__global__ void __launch_bounds__(256, 2)
append_mma_kernel(const bf16* __restrict__ x, const bf16* __restrict__ A_tiled, CacheView cv, int D, int r_k,
                  int r_v, int T, int max_pos, int* status, int d_head, int rope_style,
                  const float2* __restrict__ rope_table) {
    __shared__ float red[8][32][4];
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int g = lane >> 2, t = lane & 3;
    const int R = r_k + r_v;
    const int kq = warp;
    const int n0 = blockIdx.x * 8;
    const long long m0 = (long long)blockIdx.y * 16;
    const long long n_tok = (long long)cv.batch * T;
    float c[4] = {0.f, 0.f, 0.f, 0.f};
    if (n0 < R) {
        const int kspan = D / 8;
        const int k_begin = kq * kspan;
        const bool row_lo = (m0 + g) < n_tok, row_hi = (m0 + g + 8) < n_tok;
        const uint4* xa = reinterpret_cast<const uint4*>(x + (m0 + g) * D + k_begin) + t;
        const uint4* xb = reinterpret_cast<const uint4*>(x + (m0 + g + 8) * D + k_begin) + t;
        const uint4* wb = reinterpret_cast<const uint4*>(A_tiled) + ((long long)blockIdx.x * (D / 32) + k_begin / 32) * 32 + lane;
        const uint4 zero = make_uint4(0, 0, 0, 0);
        // The factor comes from HBM and nothing else in the kernel takes long: up to 16 steps' worth of it (8 KiB per
        // warp) is requested before the first MMA (volatile asm keeps the loads together, ahead of their uses).
        const int steps = kspan / 32;
        for (int kb0 = 0; kb0 < steps; kb0 += 16) {
            uint4 w[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                w[i] = zero;
                if (kb0 + i < steps) {
                    const uint4* src = wb + (kb0 + i) * 32;
                    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(w[i].x), "=r"(w[i].y), "=r"(w[i].z), "=r"(w[i].w)
                                 : "l"(src));
                }
            }
#pragma unroll
            for (int i0 = 0; i0 < 16; i0 += 8) {
                uint4 lo[8], hi[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    lo[i] = zero;
                    hi[i] = zero;
                    if (kb0 + i0 + i < steps) {
                        if (row_lo)
                            asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];"
                                         : "=r"(lo[i].x), "=r"(lo[i].y), "=r"(lo[i].z), "=r"(lo[i].w)
                                         : "l"(xa + (kb0 + i0 + i) * 4));
                        if (row_hi)
                            asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];"
                                         : "=r"(hi[i].x), "=r"(hi[i].y), "=r"(hi[i].z), "=r"(hi[i].w)
                                         : "l"(xb + (kb0 + i0 + i) * 4));
                    }
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (kb0 + i0 + i < steps) {
                        mma_bf16_16816(c, lo[i].x, hi[i].x, lo[i].y, hi[i].y, w[i0 + i].x, w[i0 + i].y);
                        mma_bf16_16816(c, lo[i].z, hi[i].z, lo[i].w, hi[i].w, w[i0 + i].z, w[i0 + i].w);
                    }
                }
            }
        }
    }
    red[warp][lane][0] = c[0];
    red[warp][lane][1] = c[1];
    red[warp][lane][2] = c[2];
    red[warp][lane][3] = c[3];
    __syncthreads();
    if (kq != 0 || n0 >= R) return;
#pragma unroll
    for (int i = 0; i < 4; ++i)
        c[i] = ((red[0][lane][i] + red[1][lane][i]) + (red[2][lane][i] + red[3][lane][i])) +
               ((red[4][lane][i] + red[5][lane][i]) + (red[6][lane][i] + red[7][lane][i]));
    const int col = n0 + 2 * t;          // columns col, col + 1
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        const long long tok = m0 + g + half * 8;
        if (tok >= n_tok) continue;
        const int s = (int)(tok / T);
        const int i = (int)(tok - (long long)s * T);
        const int pos = cv.seq_lens[s] - T + i;
        const long long row = lorc_row_index(cv, s, pos);
        if (row < 0 || pos >= max_pos) {
            lorc_set_status(status, LORC_ERR_CAPACITY);
            continue;
        }
        __nv_bfloat162 v = __floats2bfloat162_rn(c[half * 2], c[half * 2 + 1]);
        if (FULL && col < r_k) {
            const int hd = d_head / 2, head = col / d_head, j = (col - head * d_head) >> 1;
            const float2 cs = rope_table[(long long)pos * hd + j];
            const float a = c[half * 2], b = c[half * 2 + 1];
            const float ka = a * cs.x - b * cs.y, kb = a * cs.y + b * cs.x;
            bf16* krow = cv.k + row * cv.w_k;
            if (rope_style == LORC_ROPE_HALF_SPLIT) {
                krow[head * d_head + j] = __float2bfloat16_rn(ka);
                krow[head * d_head + j + hd] = __float2bfloat16_rn(kb);
            } else {
                *reinterpret_cast<__nv_bfloat162*>(krow + col) = __floats2bfloat162_rn(ka, kb);
            }
        } else if (col < r_k)
            *reinterpret_cast<__nv_bfloat162*>(cv.k + row * cv.w_k + col) = v;
        else
            *reinterpret_cast<__nv_bfloat162*>(cv.v + row * cv.w_v + (col - r_k)) = v;
    }
}

// The first `pair_cols` columns (0: none) are taken in rotary-pair order: tiled column head * d_head + 2 j + e is the
// factor's column head * d_head + j + e * d_head / 2, so that a pair (j, j + d_head / 2) sits in adjacent columns.
__global__ void retile_factor_kernel(const bf16* __restrict__ A_cat, bf16* __restrict__ A_tiled, int D, int R,
                                     int pair_cols, int d_head) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)D * R) return;
    const int e = (int)(i & 7), lane = (int)((i >> 3) & 31);
    const long long blk = i >> 8;                       // (column tile, k block)
    const int kb = (int)(blk % (D / 32)), nt = (int)(blk / (D / 32));
    int col = nt * 8 + (lane >> 2);
    const int k = kb * 32 + (lane & 3) * 8 + e;
    if (col < pair_cols) {
        const int head = col / d_head, w = col - head * d_head;
        col = head * d_head + (w >> 1) + (w & 1) * (d_head / 2);
    }
    A_tiled[i] = A_cat[(long long)k * R + col];
}

}  // namespace

cudaError_t lorc_fast_retile_factor(const bf16* A_cat, bf16* A_tiled, int D, int R, int pair_cols, int d_head,
                                    cudaStream_t st) {
    const long long total = (long long)D * R;
    retile_factor_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(A_cat, A_tiled, D, R, pair_cols, d_head);
    return cudaGetLastError();
}

bool lorc_tc_append_supported(const lorc_ctx* ctx, const LorcLayer& L, const CacheView&, int) {
    return ctx->desc.d_model % 256 == 0 && L.A_tiled != nullptr;
}

cudaError_t lorc_tc_append(lorc_ctx* ctx, int, const LorcLayer& L, const CacheView& cv, const bf16* x, int T,
                           cudaStream_t st, int* launches) {
    const int R = L.r_k + L.r_v;
    const long long n_tok = (long long)cv.batch * T;
    dim3 grid((R + 7) / 8, (unsigned)((n_tok + 15) / 16));
    if (L.mode == LORC_MODE_FULL)
        append_mma_kernel<true><<<grid, 256, 0, st>>>(x, L.A_tiled, cv, ctx->desc.d_model, L.r_k, L.r_v, T,
                                                      ctx->desc.max_pos, ctx->status_dev, ctx->desc.d_head,
                                                      ctx->pair_style, ctx->rope_table);
    else
        append_mma_kernel<false><<<grid, 256, 0, st>>>(x, L.A_tiled, cv, ctx->desc.d_model, L.r_k, L.r_v, T,
                                                       ctx->desc.max_pos, ctx->status_dev, ctx->desc.d_head,
                                                       ctx->pair_style, ctx->rope_table);
    *launches += 1;
    return cudaGetLastError();
}
