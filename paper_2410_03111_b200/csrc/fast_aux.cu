// Bandwidth-bound helpers of the fast path:
//   * latent cache write for a handful of tokens (decode) or chunks of tokens (prefill):
//     C = x [A_K | A_V], a skinny GEMM whose cost is streaming the factor once.  Warp-level
//     mma.sync (M = 16 tokens) is the natural tile here: a 128-row tcgen05 tile would be
//     7/8 padding at decode batch sizes, and the kernel is bound by the weight stream.
//   * merge of the context-split partials + value up-projection out = (O_lat / l) B_V[:, g].
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

__global__ void __launch_bounds__(256)
append_mma_kernel(const bf16* __restrict__ x, const bf16* __restrict__ A_tiled, CacheView cv, int D, int r_k,
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
        const uint4* wb = reinterpret_cast<const uint4*>(A_tiled) + ((long long)blockIdx.x * (D / 32) + k_begin / 32) * 32 + lane;
        const uint4 zero = make_uint4(0, 0, 0, 0);
#pragma unroll 8
        for (int kb = 0; kb < kspan / 32; ++kb) {
            const uint4 w = __ldg(wb + kb * 32);
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
// merge + up-projection: grid (n_kv_heads, batch); 16 compute warps + 1 TMA warp.  A block owns the
// G query heads of one KV head of one sequence.  The B_V slice [r_v, 128] of that KV head is streamed
// by TMA through a ring of 64-row slices while the split partials are being merged, so the
// up-projection loop never waits on a global load.
// ---------------------------------------------------------------------------------------------
constexpr int CB_SLOTS = 6;
constexpr int CB_THREADS = 544;

template <int G>
__global__ void __launch_bounds__(CB_THREADS)
combine_fast_kernel(const __grid_constant__ CUtensorMap mapBV, const float* __restrict__ part_ml,
                    const float* __restrict__ part_o, bf16* __restrict__ out, int H_q, int W, int n_splits,
                    int* status) {
    extern __shared__ uint8_t craw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(craw) + 127) & ~uintptr_t(127));
    bf16* BV = reinterpret_cast<bf16*>(base);                                  // [CB_SLOTS][64][128]
    uint64_t* full = reinterpret_cast<uint64_t*>(base + CB_SLOTS * 64 * 128 * 2);
    uint64_t* empty = full + CB_SLOTS;
    float* o_lat = reinterpret_cast<float*>(empty + CB_SLOTS);                 // [W][G]
    float* w_s = o_lat + (size_t)W * G;                                        // [G][n_splits]
    float* red = w_s + G * n_splits;                                           // [3][128][G], first used as (m, l) staging
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = blockIdx.x, s = blockIdx.y;
    const int n_bv = (W + 63) / 64;
    if (tid == 0) {
        for (int i = 0; i < CB_SLOTS; ++i) {
            sm100::mbar_init(&full[i], 1);
            sm100::mbar_init(&empty[i], 16);
        }
        sm100::fence_barrier_init();
    }
    __syncthreads();
    if (warp == 16) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            for (int c = 0; c < n_bv; ++c) {
                const int slot = c % CB_SLOTS;
                if (!sm100::mbar_wait(&empty[slot], ((c / CB_SLOTS) & 1) ^ 1)) {
                    lorc_set_status(status, LORC_ERR_TIMEOUT);
                    break;
                }
                sm100::mbar_arrive_expect_tx(&full[slot], 64 * 128 * 2);
                sm100::tma_load_2d(BV + slot * 64 * 128, &mapBV, &full[slot], g * 128, c * 64);
            }
        }
    } else {
        // (m, l) of every (row, split): one load per thread, then a short serial pass per row in shared memory
        float2* ml_sh = reinterpret_cast<float2*>(red);      // [G][n_splits]
        for (int idx = tid; idx < G * n_splits; idx += 512) {
            const int row = idx / n_splits, c = idx - row * n_splits;
            ml_sh[idx] = *reinterpret_cast<const float2*>(part_ml + (((long long)s * H_q + g * G + row) * n_splits + c) * 2);
        }
        asm volatile("bar.sync 1, 512;" ::: "memory");
        if (tid < G) {
            float* w = w_s + tid * n_splits;
            const float2* ml = ml_sh + tid * n_splits;
            float M = -INFINITY;
            for (int c = 0; c < n_splits; ++c)
                if (ml[c].y > 0.f) M = fmaxf(M, ml[c].x);
            float L = 0.f;
            for (int c = 0; c < n_splits; ++c) {
                const float ww = (ml[c].y > 0.f) ? __expf(ml[c].x - M) : 0.f;
                w[c] = ww;
                L += ww * ml[c].y;
            }
            const float inv = (L > 0.f) ? 1.f / L : 0.f;
            if (!(L > 0.f)) lorc_set_status(status, LORC_ERR_EMPTY);
            for (int c = 0; c < n_splits; ++c) w[c] *= inv;
        }
        asm volatile("bar.sync 1, 512;" ::: "memory");
        // merged, normalised latent outputs [rho][row].  One 16-byte load per (row, 4 rho, split); the loads of
        // eight splits are issued before any is used, so a thread waits for memory only a couple of times.
        const int W4 = W >> 2;
        for (int idx = tid; idx < G * W4; idx += 512) {
            const int row = idx / W4, r4 = idx - row * W4;
            const float4* po = reinterpret_cast<const float4*>(
                                   part_o + (((long long)s * H_q + g * G + row) * n_splits) * W) + r4;
            const float* w = w_s + row * n_splits;
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int c0 = 0; c0 < n_splits; c0 += 8) {
                float4 v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    v[u] = (c0 + u < n_splits) ? __ldg(po + (long long)(c0 + u) * W4) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const float ww = (c0 + u < n_splits) ? w[c0 + u] : 0.f;
                    if (ww != 0.f) {
                        a.x = fmaf(ww, v[u].x, a.x);
                        a.y = fmaf(ww, v[u].y, a.y);
                        a.z = fmaf(ww, v[u].z, a.z);
                        a.w = fmaf(ww, v[u].w, a.w);
                    }
                }
            }
            o_lat[(r4 * 4 + 0) * G + row] = a.x;
            o_lat[(r4 * 4 + 1) * G + row] = a.y;
            o_lat[(r4 * 4 + 2) * G + row] = a.z;
            o_lat[(r4 * 4 + 3) * G + row] = a.w;
        }
        asm volatile("bar.sync 1, 512;" ::: "memory");
        // out[row][j] = sum_rho o_lat[rho][row] * B_V[rho][g*128 + j]; each 64-row slice is shared by 4 thread groups
        const int j = tid & 127, part = tid >> 7;
        float acc[G];
#pragma unroll
        for (int r = 0; r < G; ++r) acc[r] = 0.f;
        bool ok = true;
        for (int c = 0; c < n_bv; ++c) {
            const int slot = c % CB_SLOTS;
            if (!sm100::mbar_wait(&full[slot], (c / CB_SLOTS) & 1)) { ok = false; break; }
            const bf16* bv = BV + slot * 64 * 128 + (part * 16) * 128 + j;
            const int rho0 = c * 64 + part * 16;
            const int rows = min(16, W - rho0);
#pragma unroll 4
            for (int r = 0; r < rows; ++r) {
                const float b = __bfloat162float(bv[r * 128]);
                const float4* ol = reinterpret_cast<const float4*>(o_lat + (rho0 + r) * G);
#pragma unroll
                for (int r4 = 0; r4 < G / 4; ++r4) {
                    const float4 o = ol[r4];
                    acc[r4 * 4 + 0] = fmaf(o.x, b, acc[r4 * 4 + 0]);
                    acc[r4 * 4 + 1] = fmaf(o.y, b, acc[r4 * 4 + 1]);
                    acc[r4 * 4 + 2] = fmaf(o.z, b, acc[r4 * 4 + 2]);
                    acc[r4 * 4 + 3] = fmaf(o.w, b, acc[r4 * 4 + 3]);
                }
            }
            __syncwarp();
            if (lane == 0) sm100::mbar_arrive(&empty[slot]);
        }
        if (!ok && lane == 0) lorc_set_status(status, LORC_ERR_TIMEOUT);
        if (part > 0) {
#pragma unroll
            for (int r = 0; r < G; ++r) red[((part - 1) * 128 + j) * G + r] = acc[r];
        }
        asm volatile("bar.sync 1, 512;" ::: "memory");
        if (part == 0) {
#pragma unroll
            for (int r = 0; r < G; ++r) {
                const float v = acc[r] + red[j * G + r] + red[(128 + j) * G + r] + red[(256 + j) * G + r];
                out[((long long)s * H_q + g * G + r) * 128 + j] = __float2bfloat16_rn(v);
            }
        }
    }
}

__global__ void retile_factor_kernel(const bf16* __restrict__ A_cat, bf16* __restrict__ A_tiled, int D, int R) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)D * R) return;
    const int e = (int)(i & 7), lane = (int)((i >> 3) & 31);
    const long long blk = i >> 8;                       // (column tile, k block)
    const int kb = (int)(blk % (D / 32)), nt = (int)(blk / (D / 32));
    const int col = nt * 8 + (lane >> 2), k = kb * 32 + (lane & 3) * 8 + e;
    A_tiled[i] = A_cat[(long long)k * R + col];
}

}  // namespace

cudaError_t lorc_fast_retile_factor(const bf16* A_cat, bf16* A_tiled, int D, int R, cudaStream_t st) {
    const long long total = (long long)D * R;
    retile_factor_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(A_cat, A_tiled, D, R);
    return cudaGetLastError();
}

bool lorc_tc_append_supported(const lorc_ctx* ctx, const LorcLayer& L, const CacheView&, int) {
    return L.mode == LORC_MODE_LATENT && ctx->desc.d_model % 256 == 0 && L.A_tiled != nullptr;
}

cudaError_t lorc_tc_append(lorc_ctx* ctx, int, const LorcLayer& L, const CacheView& cv, const bf16* x, int T,
                           cudaStream_t st, int* launches) {
    const int R = L.r_k + L.r_v;
    const long long n_tok = (long long)cv.batch * T;
    dim3 grid((R + 7) / 8, (unsigned)((n_tok + 15) / 16));
    append_mma_kernel<<<grid, 256, 0, st>>>(x, L.A_tiled, cv, ctx->desc.d_model, L.r_k, L.r_v, T, ctx->desc.max_pos,
                                            ctx->status_dev);
    *launches += 1;
    return cudaGetLastError();
}

// Merge + up-projection for LATENT layers with d_head = 128 and 4 or 8 query heads per KV head.
// mapBV: B_V [r_v, n] as a 2-D tensor map with plain 64 x 128 boxes.
cudaError_t lorc_fast_combine(const lorc_ctx* ctx, const LorcLayer& L, const CUtensorMap* mapBV, int batch,
                              int n_splits, const float* part_ml, const float* part_o, bf16* out, cudaStream_t st,
                              int* launches) {
    const lorc_model_desc& d = ctx->desc;
    const int G = ctx->group, W = L.r_v;
    dim3 grid(d.n_kv_heads, batch);
    const size_t red_floats = (size_t)(3 * 128 * G > 2 * G * n_splits ? 3 * 128 * G : 2 * G * n_splits);
    size_t smem = 128 + (size_t)CB_SLOTS * 64 * 128 * 2 + 2 * CB_SLOTS * sizeof(uint64_t) +
                  ((size_t)W * G + (size_t)G * n_splits + red_floats) * sizeof(float);
    static bool attr = false;
    if (!attr) {
        cudaError_t e = cudaFuncSetAttribute(combine_fast_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             200 * 1024);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(combine_fast_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        attr = true;
    }
    if (!mapBV || smem > 200 * 1024 || (G != 4 && G != 8))
        return lorc_generic_combine(ctx, L, batch, n_splits, part_ml, part_o, out, st, launches);
    LorcStageTimer timer(ctx, LORC_STAGE_COMBINE, st);
    if (G == 4)
        combine_fast_kernel<4><<<grid, CB_THREADS, smem, st>>>(*mapBV, part_ml, part_o, out, d.n_q_heads, W, n_splits,
                                                              ctx->status_dev);
    else
        combine_fast_kernel<8><<<grid, CB_THREADS, smem, st>>>(*mapBV, part_ml, part_o, out, d.n_q_heads, W, n_splits,
                                                              ctx->status_dev);
    *launches += 1;
    return cudaGetLastError();
}
