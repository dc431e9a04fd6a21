// Decode attention of the uncompressed reference mode (ordinary KV cache: keys stored rotated, values as they are)
// on the warp-level tensor cores.  The work is one pass over 2 n bf16 numbers per token and is bound by HBM, so the
// kernel is shaped for streaming: a CTA owns one (sequence, KV head, context share), each of its four warps owns
// 16 of every 64 tokens with its own running softmax (no block-wide synchronisation inside the loop), and the G
// query heads of the KV head are the rows of one m16n8k16 tile (rows G..15 are padding).
//
//   S[16 x 16 tok]  = Q^[16 x 128] . K[16 tok x 128]^T     q^ = RoPE(q, N-1)/sqrt(d_h) split into bf16 hi + lo parts,
//                                                           so the scores keep fp32-level accuracy
//   p = exp(S - m) rounded to bf16 (the same rounded value enters the denominator)
//   O[16 x 128]    += P[16 x 16 tok] . V[16 tok x 128]
// Keys and values of a warp's 16 tokens are staged in its own double-buffered shared-memory slice by asynchronous
// copies (the next tile is in flight while the current one is worked on) and read with ldmatrix.
//
// Each CTA leaves (m, l, un-normalised O) per query head for the merge kernel of the plain family.
#include <math.h>

#include "common.cuh"

namespace {

constexpr int FD_DH = 128;
constexpr int FD_TILE = 64;          // tokens per CTA iteration (16 per warp)
constexpr int FD_VPAD = 8;           // bf16 elements of padding per staged value row (keeps ldmatrix conflict-free)

// m16n8k16 bf16 MMA whose A rows 8..15 are zero (operands a1, a3 = 0): c0, c1 belong to row lane / 4; the
// padding row's results are discarded.
__device__ __forceinline__ void mma_16816_lo(float& c0, float& c1, uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    asm volatile(
        "{\n\t"
        ".reg .f32 d2, d3;\n\t"          // results of the padding rows: zero, never read
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,d2,d3}, {%2,%3,%4,%3}, {%5,%6}, {%0,%1,%7,%7};\n\t"
        "}\n"
        : "+f"(c0), "+f"(c1)
        : "r"(a0), "r"(0u), "r"(a2), "r"(b0), "r"(b1), "f"(0.f));
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

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* smem_row) {
    const uint32_t addr = (uint32_t)__cvta_generic_to_shared(smem_row);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

// 16-byte asynchronous copy global -> shared (bypassing L1), grouped with commit / wait
__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gsrc) {
    const uint32_t addr = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(addr), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

constexpr int FD_ROW = FD_DH + FD_VPAD;              // staged row length in bf16 elements (272 bytes)

struct FdSmem {
    float qs[8][FD_DH];                              // rotated, scaled queries of the G heads (rows G..7 zero)
    float m[4][8], l[4][8];
    union {
        bf16 kv[4][2][2][16][FD_ROW];                // [warp][buffer][keys | values][token][dimension]
        float o[4][8][FD_DH];                        // after the loop: every warp's un-normalised output
    } u;
};

__global__ void __launch_bounds__(128, 3)
full_decode_mma_kernel(const bf16* __restrict__ q, CacheView cv, int G, int n_splits, int rope_style,
                       const float2* __restrict__ rope_table, int max_pos, float* __restrict__ part_ml,
                       float* __restrict__ part_o, int* status) {
    extern __shared__ __align__(16) uint8_t fd_raw[];
    FdSmem& sm = *reinterpret_cast<FdSmem*>(fd_raw);
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
    const int col0 = kvh * FD_DH;

    // Stage the 16 key rows and 16 value rows of the warp's tile that starts at token t0 into buffer `buf`
    // (asynchronous 16-byte copies, two rows per step; rows that do not exist are zero).  Returns, in lanes 0..15,
    // the cache row of token t0 + lane (-1: none).
    auto stage = [&](int t0, int buf) -> long long {
        long long my_row = -1;
        if (lane < 16 && t0 + lane < t_end) {
            my_row = lorc_row_index(cv, s, t0 + lane);
            if (my_row < 0) lorc_set_status(status, LORC_ERR_CAPACITY);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = 2 * i + (lane >> 4);
            const long long row = __shfl_sync(0xffffffffu, my_row, r);
            bf16* kd = &sm.u.kv[warp][buf][0][r][(lane & 15) * 8];
            bf16* vd = &sm.u.kv[warp][buf][1][r][(lane & 15) * 8];
            if (row >= 0) {
                cp_async_16(kd, reinterpret_cast<const uint4*>(cv.k + row * cv.w_k + col0) + (lane & 15));
                cp_async_16(vd, reinterpret_cast<const uint4*>(cv.v + row * cv.w_v + col0) + (lane & 15));
            } else {
                *reinterpret_cast<uint4*>(kd) = make_uint4(0, 0, 0, 0);
                *reinterpret_cast<uint4*>(vd) = make_uint4(0, 0, 0, 0);
            }
        }
        cp_async_commit();
        return my_row;
    };

    // the first tile is on its way while the query is prepared
    const int t_first = t_begin + warp * 16;
    long long row_cur = -1;
    if (t_first < t_end) row_cur = stage(t_first, 0);

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

    // Query fragments of row g (rows 8..15 of the tile are padding): k-step ks covers the dimensions 16 ks .. + 15,
    // split into bf16 hi + lo parts.
    uint32_t qhi[8][2], qlo[8][2];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int d0 = 16 * ks + 8 * half + 2 * t;
            const float v0 = sm.qs[g][d0], v1 = sm.qs[g][d0 + 1];
            const float h0 = __bfloat162float(__float2bfloat16_rn(v0)), h1 = __bfloat162float(__float2bfloat16_rn(v1));
            qhi[ks][half] = pack_bf16(h0, h1);
            qlo[ks][half] = pack_bf16(v0 - h0, v1 - h1);
        }
    }

    float o[16][2];                                   // O[row g][dims 8 dt + 2 t, + 1]
#pragma unroll
    for (int dt = 0; dt < 16; ++dt) o[dt][0] = o[dt][1] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;             // running maximum and (per-lane partial) denominator of row g

    const int mi = lane >> 3;                         // which 8 x 8 matrix of an ldmatrix.x4 this lane addresses
    int it = 0;
    for (int t0 = t_first; t0 < t_end; t0 += FD_TILE, ++it) {
        const int buf = it & 1;
        // next tile into the other buffer, then wait for this one
        long long row_next = -1;
        const bool has_next = t0 + FD_TILE < t_end;
        if (has_next) {
            row_next = stage(t0 + FD_TILE, buf ^ 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncwarp();

        // scores of row g against tokens nt * 8 + 2 t, + 1
        float sc[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            uint32_t kb[4];       // (tokens 0..7, dims 16 ks..+7), (0..7, +8..15), (tokens 8..15, ...), (8..15, ...)
            ldmatrix_x4(kb, &sm.u.kv[warp][buf][0][(mi >> 1) * 8 + (lane & 7)][16 * ks + 8 * (mi & 1)]);
            mma_16816_lo(sc[0][0], sc[0][1], qhi[ks][0], qhi[ks][1], kb[0], kb[1]);
            mma_16816_lo(sc[1][0], sc[1][1], qhi[ks][0], qhi[ks][1], kb[2], kb[3]);
            mma_16816_lo(sc[0][0], sc[0][1], qlo[ks][0], qlo[ks][1], kb[0], kb[1]);
            mma_16816_lo(sc[1][0], sc[1][1], qlo[ks][0], qlo[ks][1], kb[2], kb[3]);
        }
        // running softmax of row g over this warp's tokens
        float mx = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const long long row = __shfl_sync(0xffffffffu, row_cur, nt * 8 + 2 * t + e);
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
        // O = alpha O + P V
#pragma unroll
        for (int dp = 0; dp < 8; ++dp) {
            uint32_t vb[4];       // (tokens 0..7 | 8..15) x (dims 16 dp..+7 | +8..15), transposed on the way in
            ldmatrix_x4_trans(vb, &sm.u.kv[warp][buf][1][(mi & 1) * 8 + (lane & 7)][8 * (2 * dp + (mi >> 1))]);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                float (&acc)[2] = o[2 * dp + half];
                acc[0] *= alpha;
                acc[1] *= alpha;
                mma_16816_lo(acc[0], acc[1], pa[0], pa[1], vb[2 * half], vb[2 * half + 1]);
            }
        }
        __syncwarp();                                 // this buffer is refilled two tiles from now
        row_cur = row_next;
    }

    // merge the four warps of the CTA
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    __syncthreads();                                  // every warp is done with its staging buffers (the union is reused)
    if (t == 0) {
        sm.m[warp][g] = m_run;
        sm.l[warp][g] = l_run;
    }
#pragma unroll
    for (int dt = 0; dt < 16; ++dt) {
        sm.u.o[warp][g][8 * dt + 2 * t] = o[dt][0];
        sm.u.o[warp][g][8 * dt + 2 * t + 1] = o[dt][1];
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
    // the attribute belongs to a device's copy of the kernel: one flag per device (devices beyond the table set it
    // on every call, which is only slower)
    static bool attr[64] = {false};
    const bool known = ctx->device >= 0 && ctx->device < 64;
    if (!known || !attr[ctx->device]) {
        cudaError_t e = cudaFuncSetAttribute(full_decode_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)sizeof(FdSmem));
        if (e != cudaSuccess) return e;
        if (known) attr[ctx->device] = true;
    }
    full_decode_mma_kernel<<<grid, 128, sizeof(FdSmem), st>>>(q, cv, ctx->group, n_splits, ctx->pair_style, ctx->rope_table, d.max_pos,
                                                 part_ml, part_o, ctx->status_dev);
    *launches += 1;
    return cudaGetLastError();
}
