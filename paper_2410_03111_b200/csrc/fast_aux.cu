// Bandwidth-bound helpers of the fast path:
//   * latent cache write for a handful of tokens (decode) or chunks of tokens (prefill):
//     C = x [A_K | A_V], a skinny GEMM whose cost is streaming the factor once.  Warp-level
//     mma.sync (M = 16 tokens) is the natural tile here: a 128-row tcgen05 tile would be
//     7/8 padding at decode batch sizes, and the kernel is bound by the weight stream.
//   * merge of the context-split partials + value up-projection out = (O_lat / l) B_V[:, g].
#include "common.cuh"
#include "tc_kernels.cuh"

namespace {

// ---------------------------------------------------------------------------------------------
// append: grid (R/8, token tiles of 16); 8 warps = 8 slices of D for one tile of 8 columns.
// Operands: x [n_tok, D] row-major, A_catT [R, D] (K contiguous).  K is consumed in blocks of 32:
// lane (g = lane/4, t = lane%4) loads 8 consecutive k (16 bytes) of its rows and uses them as the
// fragment slots of two m16n8k16 steps; both operands use the same slot order, so the contraction
// is unchanged.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__global__ void __launch_bounds__(256)
append_mma_kernel(const bf16* __restrict__ x, const bf16* __restrict__ A_catT, CacheView cv, int D, int r_k,
                  int r_v, int T, int max_pos, int* status) {
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
        const uint4* wb = reinterpret_cast<const uint4*>(A_catT + (long long)(n0 + g) * D + k_begin) + t;
        const uint4 zero = make_uint4(0, 0, 0, 0);
#pragma unroll 8
        for (int kb = 0; kb < kspan / 32; ++kb) {
            const uint4 w = __ldg(wb + kb * 4);
            const uint4 lo = row_lo ? __ldg(xa + kb * 4) : zero;
            const uint4 hi = row_hi ? __ldg(xb + kb * 4) : zero;
            mma_bf16_16816(c, lo.x, hi.x, lo.y, hi.y, w.x, w.y);
            mma_bf16_16816(c, lo.z, hi.z, lo.w, hi.w, w.z, w.w);
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
        if (col < r_k)
            *reinterpret_cast<__nv_bfloat162*>(cv.k + row * cv.w_k + col) = v;
        else
            *reinterpret_cast<__nv_bfloat162*>(cv.v + row * cv.w_v + (col - r_k)) = v;
    }
}

// ---------------------------------------------------------------------------------------------
// merge + up-projection: grid (n_kv_heads, batch); 512 threads.  A block owns the G query heads of
// one KV head of one sequence, so the B_V slice [r_v, 128] is read once per block.
// ---------------------------------------------------------------------------------------------
template <int G>
__global__ void __launch_bounds__(512)
combine_fast_kernel(const float* __restrict__ part_ml, const float* __restrict__ part_o,
                    const bf16* __restrict__ B_v, bf16* __restrict__ out, int H_q, int W, int n, int n_splits,
                    int* status) {
    extern __shared__ float sh[];
    float* o_lat = sh;                               // [W][G]
    float* w_s = sh + (size_t)W * G;                 // [G][n_splits]   merge weight / L
    float* red = w_s + G * n_splits;                 // [3][128][G]
    const int tid = threadIdx.x;
    const int g = blockIdx.x, s = blockIdx.y;
    if (tid < G) {
        const int h = g * G + tid;
        float* w = w_s + tid * n_splits;
        const long long unit0 = ((long long)s * H_q + h) * n_splits;
        float M = -INFINITY;
        for (int c = 0; c < n_splits; ++c)
            if (part_ml[(unit0 + c) * 2 + 1] > 0.f) M = fmaxf(M, part_ml[(unit0 + c) * 2]);
        float L = 0.f;
        for (int c = 0; c < n_splits; ++c) {
            const float l = part_ml[(unit0 + c) * 2 + 1];
            const float ww = (l > 0.f) ? __expf(part_ml[(unit0 + c) * 2] - M) : 0.f;
            w[c] = ww;
            L += ww * l;
        }
        const float inv = (L > 0.f) ? 1.f / L : 0.f;
        if (!(L > 0.f)) lorc_set_status(status, LORC_ERR_EMPTY);
        for (int c = 0; c < n_splits; ++c) w[c] *= inv;
    }
    __syncthreads();
    // merged, normalised latent outputs [rho][row]; every load is issued unconditionally so that many are in flight
    for (int idx = tid; idx < G * W; idx += 512) {
        const int row = idx / W, rho = idx - row * W;
        const float* po = part_o + (((long long)s * H_q + g * G + row) * n_splits) * W + rho;
        const float* w = w_s + row * n_splits;
        float a = 0.f;
        int c = 0;
        for (; c + 4 <= n_splits; c += 4) {
            const float v0 = po[(long long)c * W], v1 = po[(long long)(c + 1) * W];
            const float v2 = po[(long long)(c + 2) * W], v3 = po[(long long)(c + 3) * W];
            const float w0 = w[c], w1 = w[c + 1], w2 = w[c + 2], w3 = w[c + 3];
            a += (w0 != 0.f ? w0 * v0 : 0.f) + (w1 != 0.f ? w1 * v1 : 0.f) + (w2 != 0.f ? w2 * v2 : 0.f) +
                 (w3 != 0.f ? w3 * v3 : 0.f);
        }
        for (; c < n_splits; ++c) {
            const float v = po[(long long)c * W], ww = w[c];
            a += (ww != 0.f ? ww * v : 0.f);
        }
        o_lat[rho * G + row] = a;
    }
    __syncthreads();
    // out[row][j] = sum_rho o_lat[rho][row] * B_V[rho][g*128 + j]; four quarters of rho per column
    const int j = tid & 127, part = tid >> 7;
    float acc[G];
#pragma unroll
    for (int r = 0; r < G; ++r) acc[r] = 0.f;
    const int per = (W + 3) / 4;
    const int rho_end = min(W, (part + 1) * per);
    const bf16* bp = B_v + (long long)g * 128 + j;
#pragma unroll 8
    for (int rho = part * per; rho < rho_end; ++rho) {
        const float b = __bfloat162float(bp[(long long)rho * n]);
        const float4* ol = reinterpret_cast<const float4*>(o_lat + rho * G);
#pragma unroll
        for (int r4 = 0; r4 < G / 4; ++r4) {
            const float4 o = ol[r4];
            acc[r4 * 4 + 0] = fmaf(o.x, b, acc[r4 * 4 + 0]);
            acc[r4 * 4 + 1] = fmaf(o.y, b, acc[r4 * 4 + 1]);
            acc[r4 * 4 + 2] = fmaf(o.z, b, acc[r4 * 4 + 2]);
            acc[r4 * 4 + 3] = fmaf(o.w, b, acc[r4 * 4 + 3]);
        }
    }
    if (part > 0) {
#pragma unroll
        for (int r = 0; r < G; ++r) red[((part - 1) * 128 + j) * G + r] = acc[r];
    }
    __syncthreads();
    if (part == 0) {
#pragma unroll
        for (int r = 0; r < G; ++r) {
            const float v = acc[r] + red[j * G + r] + red[(128 + j) * G + r] + red[(256 + j) * G + r];
            out[((long long)s * H_q + g * G + r) * 128 + j] = __float2bfloat16_rn(v);
        }
    }
}

}  // namespace

bool lorc_tc_append_supported(const lorc_ctx* ctx, const LorcLayer& L, const CacheView&, int) {
    return L.mode == LORC_MODE_LATENT && ctx->desc.d_model % 256 == 0 && L.A_catT != nullptr;
}

cudaError_t lorc_tc_append(lorc_ctx* ctx, int, const LorcLayer& L, const CacheView& cv, const bf16* x, int T,
                           cudaStream_t st, int* launches) {
    const int R = L.r_k + L.r_v;
    const long long n_tok = (long long)cv.batch * T;
    dim3 grid((R + 7) / 8, (unsigned)((n_tok + 15) / 16));
    append_mma_kernel<<<grid, 256, 0, st>>>(x, L.A_catT, cv, ctx->desc.d_model, L.r_k, L.r_v, T, ctx->desc.max_pos,
                                            ctx->status_dev);
    *launches += 1;
    return cudaGetLastError();
}

// Merge + up-projection for LATENT layers with d_head = 128 and 4 or 8 query heads per KV head.
cudaError_t lorc_fast_combine(const lorc_ctx* ctx, const LorcLayer& L, int batch, int n_splits,
                              const float* part_ml, const float* part_o, bf16* out, cudaStream_t st,
                              int* launches) {
    const lorc_model_desc& d = ctx->desc;
    const int G = ctx->group, W = L.r_v;
    dim3 grid(d.n_kv_heads, batch);
    size_t smem = ((size_t)W * G + (size_t)G * n_splits + 3 * 128 * G) * sizeof(float);
    static bool attr = false;
    if (!attr) {
        cudaError_t e = cudaFuncSetAttribute(combine_fast_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             100 * 1024);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(combine_fast_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
        if (e != cudaSuccess) return e;
        attr = true;
    }
    if (smem > 100 * 1024 || (G != 4 && G != 8))
        return lorc_generic_combine(ctx, L, batch, n_splits, part_ml, part_o, out, st, launches);
    LorcStageTimer timer(ctx, LORC_STAGE_COMBINE, st);
    if (G == 4)
        combine_fast_kernel<4><<<grid, 512, smem, st>>>(part_ml, part_o, L.B_v, out, d.n_q_heads, W, ctx->n, n_splits,
                                                       ctx->status_dev);
    else
        combine_fast_kernel<8><<<grid, 512, smem, st>>>(part_ml, part_o, L.B_v, out, d.n_q_heads, W, ctx->n, n_splits,
                                                       ctx->status_dev);
    *launches += 1;
    return cudaGetLastError();
}
