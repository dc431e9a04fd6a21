// Decode attention of the uncompressed reference mode (ordinary KV cache: keys stored rotated, values as they are)
// on the warp-level tensor cores.  The work is one pass over 2 n bf16 numbers per token and is bound by HBM, so the
// kernel is shaped for streaming: a CTA owns one (sequence, KV head, context share), each of its four warps owns
// 16 of every 64 tokens with its own running softmax (no block-wide synchronisation inside the loop), and the G
// query heads of the KV head are the rows of one m16n8k16 tile (rows G..15 are padding).
//
//   S[16 x 16 tok]  = Q^[16 x 128] . K[16 tok x 128]^T     q^ = RoPE(q, N-1)/sqrt(d_h) split into bf16 hi + lo parts,
//                                                           so the scores keep fp32-level accuracy
//   p = exp(S - m) rounded to bf16 (the same rounded value enters the denominator)
//   O[16 x 128]    += P[16 x 16 tok] . V[16 tok x 128]      V staged in the warp's own shared-memory slice
//
// Each CTA leaves (m, l, un-normalised O) per query head for the merge kernel of the plain family.
#include <math.h>

#include "common.cuh"

namespace {

constexpr int FD_DH = 128;
constexpr int FD_TILE = 64;          // tokens per CTA iteration (16 per warp)
constexpr int FD_VPAD = 8;           // bf16 elements of padding per staged value row (keeps ldmatrix conflict-free)

__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem_row) {
    const uint32_t addr = (uint32_t)__cvta_generic_to_shared(smem_row);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

struct FdSmem {
    float qs[8][FD_DH];                              // rotated, scaled queries of the G heads (rows G..7 zero)
    union {
        bf16 v[4][16][FD_DH + FD_VPAD];              // per warp: its 16 value rows
        float o[4][8][FD_DH];                        // after the loop: every warp's un-normalised output
    } u;
    float m[4][8], l[4][8];
};

__global__ void __launch_bounds__(128)
full_decode_mma_kernel(const bf16* __restrict__ q, CacheView cv, int G, int n_splits, int rope_style,
                       const float2* __restrict__ rope_table, int max_pos, float* __restrict__ part_ml,
                       float* __restrict__ part_o, int* status) {
    __shared__ __align__(16) FdSmem sm;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;            // fragment row / column group of this lane
    const int split = blockIdx.x, kvh = blockIdx.y, s = blockIdx.z;
    const int H_q = G * (int)gridDim.y;
    int len = cv.seq_lens[s];
    if (len > max_pos) {
        if (tid == 0) lorc_set_status(status, LORC_ERR_CAPACITY);
        len = 0;
    }
    if (len < 0) len = 0;
    // this CTA's share of the context, in whole 64-token tiles
    const int tiles = (len + FD_TILE - 1) / FD_TILE;
    const int tps = (tiles + n_splits - 1) / n_splits;
    const int t_begin = min(len, split * tps * FD_TILE), t_end = min(len, (split + 1) * tps * FD_TILE);

    // q^ = RoPE(q, N - 1) / sqrt(d_h) for the G heads of this KV head
    for (int i = tid; i < 8 * (FD_DH / 2); i += 128) {
        const int h = i / (FD_DH / 2), jj = i - h * (FD_DH / 2);
        const int ia = (rope_style == LORC_ROPE_HALF_SPLIT) ? jj : 2 * jj;
        const int ib = (rope_style == LORC_ROPE_HALF_SPLIT) ? jj + FD_DH / 2 : 2 * jj + 1;
        float ra = 0.f, rb = 0.f;
        if (h < G && len > 0) {
            const bf16* qp = q + ((long long)s * H_q + kvh * G + h) * FD_DH;
            const float a = __bfloat162float(qp[ia]), b = __bfloat162float(qp[ib]);
            const float2 cs = rope_table[(long long)(len - 1) * (FD_DH / 2) + jj];
            const float scale = rsqrtf((float)FD_DH);
            ra = (a * cs.x - b * cs.y) * scale;
            rb = (a * cs.y + b * cs.x) * scale;
        }
        sm.qs[h][ia] = ra;
        sm.qs[h][ib] = rb;
    }
    __syncthreads();

    // Query fragments.  The contraction index of an MMA may be numbered freely as long as both operands agree: k-step
    // 2j / 2j+1 of lane (g, t) covers the dimensions 32 j + 8 t + {0..3} / {4..7}, so a lane's key operand for two
    // k-steps is one 16-byte load of 8 consecutive dimensions.  Rows 8..15 of the tile are padding (zero operands).
    uint32_t qhi[8][2], qlo[8][2];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        const int d0 = 32 * (ks >> 1) + 8 * t + 4 * (ks & 1);
        float v[4], hi[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            v[e] = g < 8 ? sm.qs[g][d0 + e] : 0.f;
            hi[e] = __bfloat162float(__float2bfloat16_rn(v[e]));
        }
        qhi[ks][0] = pack_bf16(hi[0], hi[1]);
        qhi[ks][1] = pack_bf16(hi[2], hi[3]);
        qlo[ks][0] = pack_bf16(v[0] - hi[0], v[1] - hi[1]);
        qlo[ks][1] = pack_bf16(v[2] - hi[2], v[3] - hi[3]);
    }

    float o[16][4];                                   // O[rows g, g + 8][dims 8 dt + 2 t, + 1]
#pragma unroll
    for (int dt = 0; dt < 16; ++dt)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[dt][e] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;             // running maximum and (per-lane partial) denominator of row g

    const int col0 = kvh * FD_DH;
    for (int t0 = t_begin + warp * 16; t0 < t_end; t0 += FD_TILE) {
        // rows of this warp's 16 tokens (lane i < 16 looks token i up; -1: past the end or no such row)
        long long my_row = -1;
        if (lane < 16 && t0 + lane < t_end) {
            my_row = lorc_row_index(cv, s, t0 + lane);
            if (my_row < 0) lorc_set_status(status, LORC_ERR_CAPACITY);
        }
        // keys: tokens g and g + 8, four 16-byte pieces each
        uint4 kf[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            const long long row = __shfl_sync(0xffffffffu, my_row, nt * 8 + g);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                kf[nt][j] = make_uint4(0, 0, 0, 0);
                if (row >= 0) kf[nt][j] = __ldg(reinterpret_cast<const uint4*>(cv.k + row * cv.w_k + col0 + 32 * j + 8 * t));
            }
        }
        // values: two rows per step, staged in this warp's slice (rows that do not exist are zero)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = 2 * i + (lane >> 4);
            const long long row = __shfl_sync(0xffffffffu, my_row, r);
            uint4 val = make_uint4(0, 0, 0, 0);
            if (row >= 0) val = __ldg(reinterpret_cast<const uint4*>(cv.v + row * cv.w_v + col0) + (lane & 15));
            *reinterpret_cast<uint4*>(&sm.u.v[warp][r][(lane & 15) * 8]) = val;
        }
        __syncwarp();

        // scores of rows g (and padding rows g + 8) against tokens nt * 8 + 2 t, + 1
        float sc[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) sc[nt][e] = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                mma_16816(sc[nt], qhi[2 * j][0], 0u, qhi[2 * j][1], 0u, kf[nt][j].x, kf[nt][j].y);
                mma_16816(sc[nt], qhi[2 * j + 1][0], 0u, qhi[2 * j + 1][1], 0u, kf[nt][j].z, kf[nt][j].w);
                mma_16816(sc[nt], qlo[2 * j][0], 0u, qlo[2 * j][1], 0u, kf[nt][j].x, kf[nt][j].y);
                mma_16816(sc[nt], qlo[2 * j + 1][0], 0u, qlo[2 * j + 1][1], 0u, kf[nt][j].z, kf[nt][j].w);
            }
        }
        // running softmax of row g over this warp's tokens
        float mx = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int tok = nt * 8 + 2 * t + e;
                const long long row = __shfl_sync(0xffffffffu, my_row, tok);
                if (row < 0) sc[nt][e] = -INFINITY;
                mx = fmaxf(mx, sc[nt][e]);
            }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run, mx);
        float alpha = 1.f;
        uint32_t pa[2] = {0u, 0u};
        if (m_new != -INFINITY) {
            alpha = (m_run == -INFINITY) ? 0.f : expf(m_run - m_new);
            float p[2][2];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e)
                    p[nt][e] = __bfloat162float(__float2bfloat16_rn(expf(sc[nt][e] - m_new)));
            l_run = l_run * alpha + (p[0][0] + p[0][1]) + (p[1][0] + p[1][1]);
            pa[0] = pack_bf16(p[0][0], p[0][1]);
            pa[1] = pack_bf16(p[1][0], p[1][1]);
        }
        m_run = m_new;
        // O = alpha O + P V   (alpha of a lane's row; the padding rows carry zeros)
#pragma unroll
        for (int dp = 0; dp < 8; ++dp) {
            uint32_t vb[4];
            const int mi = lane >> 3;                 // which 8 x 8 matrix this lane addresses
            ldmatrix_x4_trans(vb, &sm.u.v[warp][(mi & 1) * 8 + (lane & 7)][8 * (2 * dp + (mi >> 1))]);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                float (&acc)[4] = o[2 * dp + half];
                acc[0] *= alpha;
                acc[1] *= alpha;
                mma_16816(acc, pa[0], 0u, pa[1], 0u, vb[2 * half], vb[2 * half + 1]);
            }
        }
        __syncwarp();                                 // the slice is rewritten in the next iteration
    }

    // merge the four warps of the CTA
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    __syncthreads();                                  // every warp is done with its value slice (the union is reused)
    if (g < 8) {
        if (t == 0) {
            sm.m[warp][g] = m_run;
            sm.l[warp][g] = l_run;
        }
#pragma unroll
        for (int dt = 0; dt < 16; ++dt) {
            sm.u.o[warp][g][8 * dt + 2 * t] = o[dt][0];
            sm.u.o[warp][g][8 * dt + 2 * t + 1] = o[dt][1];
        }
    }
    __syncthreads();
    for (int h = 0; h < G; ++h) {
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < 4; ++w)
            if (sm.l[w][h] > 0.f) M = fmaxf(M, sm.m[w][h]);
        float L = 0.f, acc = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float wgt = (sm.l[w][h] > 0.f) ? expf(sm.m[w][h] - M) : 0.f;
            L += wgt * sm.l[w][h];
            acc += wgt * sm.u.o[w][h][tid];
        }
        const long long unit = ((long long)s * H_q + kvh * G + h) * n_splits + split;
        if (tid == 0) {
            part_ml[unit * 2 + 0] = M;
            part_ml[unit * 2 + 1] = L;
        }
        part_o[unit * FD_DH + tid] = acc;
    }
}

}  // namespace

bool lorc_full_decode_supported(const lorc_ctx* ctx, const LorcLayer& L) {
    return L.mode == LORC_MODE_FULL && ctx->desc.d_head == FD_DH && ctx->group >= 1 && ctx->group <= 8 &&
           !(ctx->desc.flags & LORC_FLAG_DEBUG_FP32);
}

cudaError_t lorc_full_decode(const lorc_ctx* ctx, const CacheView& cv, const bf16* q, int n_splits, float* part_ml,
                             float* part_o, cudaStream_t st, int* launches) {
    const lorc_model_desc& d = ctx->desc;
    dim3 grid(n_splits, d.n_kv_heads, cv.batch);
    full_decode_mma_kernel<<<grid, 128, 0, st>>>(q, cv, ctx->group, n_splits, d.rope_style, ctx->rope_table, d.max_pos,
                                                 part_ml, part_o, ctx->status_dev);
    *launches += 1;
    return cudaGetLastError();
}
