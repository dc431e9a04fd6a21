// Softmax + P.C_V, split by LATENT COLUMNS, and the value up-projection, both on the tensor cores.
//
// PV kernel.  A CTA owns one 128-column block of C_V (rho in [128 blk, 128 blk + 128)) of one sequence
// and one share of its context.  A block of latent columns is disjoint from every other block, so the
// CTA's accumulator O_lat^T[128 rho, H_q] (fp32 in TMEM) needs no merge with other column blocks; and
// every CTA uses the same exact row maximum (from the quarter-tile maxima the score kernel leaves
// behind), so the context shares of a block simply add.  Each CTA writes its 128 x H_q piece of the
// un-normalised latent output and, for block 0, its share of the softmax denominator.
//
//   per tile of 128 tokens:  p = 2^(s - m) (bf16, K-major in shared memory)        softmax warps
//                            O_lat^T += C_V[tile, block]^T . P^T                    tcgen05, MN-major A
//
// Up-projection kernel.  One CTA per (KV head g, 128 output rows = 128 / G sequences): builds the
// normalised latent rows o[(s, i), rho] = sum_shares O_lat / l in bf16, 64 columns at a time, and
// multiplies by B_V[:, g] (TMA-staged from a transposed copy): out = o . B_V[:, g] in TMEM, then bf16.
#include <math.h>

#include "sm100_ptx.cuh"
#include "tc_kernels.cuh"

using namespace sm100;

namespace {

constexpr int TILE = 128;
constexpr int KC = 64;
constexpr int P_STAGES = 2;          // 2 x 32 KiB: two CTAs fit on an SM
constexpr int P_THREADS = 192;       // warp 0 TMA, warp 1 MMA, warps 2..5 softmax / epilogue
constexpr int P_SOFT = 128;

// read-only global load that the compiler keeps in program order with the other volatile asm of this file
__device__ __forceinline__ float ldg_nc_f32(const float* p) {
    float v;
    asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}

template <int HQ>
struct Pv2Smem {
    bf16 V[P_STAGES][2][TILE * KC];       // C_V block: two 64-column halves of [128 tokens][64]; 32 KiB / stage
    bf16 P[2][2][HQ * KC];                // probabilities [HQ][128 tokens] as two 64-token chunks, 128-byte swizzle
    float m_s[HQ];
    float red[4][HQ];
    uint64_t full[P_STAGES], empty[P_STAGES], p_full[2], p_empty[2], o_full;
    uint32_t tmem_base;
};

struct Pv2Params {
    const float* scores;           // [b, H_q, n_pad]      log2 units
    const float* tmax;             // [b, H_q, tiles, 4]   maxima of every 32-token quarter tile
    float* o_part;                 // [b, n_csplit, H_q, r_pad]   un-normalised latent output, r_pad = 128 n_blk
    float* l_part;                 // [b, n_csplit, H_q]
    const int32_t* seq_lens;
    const int32_t* page_table;
    int* status;
    int batch, H_q, n_kv, r_v, n_pad, tiles, n_blk, n_csplit, max_pos;
    int page_size, max_pages_per_seq, n_pages;
};

template <int HQ>
__global__ void __launch_bounds__(P_THREADS, 2)
lorc_pv2_kernel(const __grid_constant__ CUtensorMap mapCV, const Pv2Params p) {
    extern __shared__ uint8_t raw[];
    typedef Pv2Smem<HQ> S;
    S& sm = *reinterpret_cast<S*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    constexpr uint32_t TM_COLS = HQ <= 32 ? 32 : 64;
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int blk = blockIdx.x, cs = blockIdx.y, s = blockIdx.z;

    int len = p.seq_lens[s];
    if (len > p.max_pos) {
        if (tid == 0) lorc_set_status(p.status, LORC_ERR_CAPACITY);
        len = 0;
    }
    if (len < 0) len = 0;
    // this CTA's share of the context: whole 128-token tiles, dealt evenly over the context shares
    const int tiles_s = (len + TILE - 1) / TILE;
    const int per = (tiles_s + p.n_csplit - 1) / p.n_csplit;
    const int tile_lo = min(tiles_s, cs * per), tile_hi = min(tiles_s, tile_lo + per);
    const int ntiles = tile_hi - tile_lo;
    const int t_begin = tile_lo * TILE, t_end = min(len, tile_hi * TILE);
    const int rho0 = blk * 128;

    if (tid == 0) {
        for (int i = 0; i < P_STAGES; ++i) {
            mbar_init(&sm.full[i], 1);
            mbar_init(&sm.empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sm.p_full[i], P_SOFT);
            mbar_init(&sm.p_empty[i], 1);
        }
        mbar_init(&sm.o_full, 1);
        fence_barrier_init();
        prefetch_tensormap(&mapCV);
    }
    if (warp == 1) {
        tmem_alloc(&sm.tmem_base, TM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    bool ok = true;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            for (int i = 0; i < ntiles && ok; ++i) {
                const int n0 = t_begin + i * TILE;
                const int st = i % P_STAGES;
                if (!mbar_wait(&sm.empty[st], ((i / P_STAGES) & 1) ^ 1)) { ok = false; break; }
                mbar_arrive_expect_tx(&sm.full[st], 2 * TILE * KC * 2);
                if (p.page_table == nullptr) {
                    tma_load_3d(sm.V[st][0], &mapCV, &sm.full[st], rho0, n0, s);
                    tma_load_3d(sm.V[st][1], &mapCV, &sm.full[st], rho0 + 64, n0, s);
                } else {
                    // One box per page.  Pages past the end of the sequence (or with a bad table entry) are read
                    // from page 0 instead: their probabilities are zero, but the rows must hold finite numbers,
                    // which stale shared memory would not guarantee.
                    const int ppt = TILE / p.page_size;
                    for (int pg = 0; pg < ppt; ++pg) {
                        const int lp = n0 / p.page_size + pg;
                        int page = 0;
                        if (lp * p.page_size < len && lp < p.max_pages_per_seq) {
                            page = p.page_table[(long long)s * p.max_pages_per_seq + lp];
                            if (page < 0 || page >= p.n_pages) {
                                lorc_set_status(p.status, LORC_ERR_CAPACITY);
                                page = 0;
                            }
                        }
                        tma_load_3d(sm.V[st][0] + pg * p.page_size * KC, &mapCV, &sm.full[st], rho0, 0, page);
                        tma_load_3d(sm.V[st][1] + pg * p.page_size * KC, &mapCV, &sm.full[st], rho0 + 64, 0, page);
                    }
                }
            }
            if (!ok) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && ntiles > 0) {
            const uint32_t idesc = make_idesc_bf16(128, HQ, 1, 0);
            for (int i = 0; i < ntiles && ok; ++i) {
                const int buf = i & 1, st = i % P_STAGES;
                if (!mbar_wait(&sm.p_full[buf], (i >> 1) & 1)) { ok = false; break; }
                if (!mbar_wait(&sm.full[st], (i / P_STAGES) & 1)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t p0 = smem_u32(sm.P[buf][0]), v0 = smem_u32(sm.V[st][0]);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    // A: C_V^T block (MN-major): 16 token rows per step, the two 64-column halves 16 KiB apart
                    const uint64_t ad = make_smem_desc_sw128(v0 + k * 2048, TILE * KC * 2, 1024);
                    // B: P [HQ][128 tokens] (K-major), 64-token chunks of HQ*128 bytes
                    const uint64_t bd = make_smem_desc_sw128(p0 + (k >> 2) * (HQ * KC * 2) + (k & 3) * 32, 0, 1024);
                    tc_mma_bf16(tmem, ad, bd, idesc, (i | k) != 0);
                }
                tc_commit(&sm.empty[st]);
                tc_commit(&sm.p_empty[buf]);
            }
            tc_commit(&sm.o_full);
            if (!ok) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
        }
    } else {
        // ------------------------------------------------------------------ softmax, then up-projection
        const int t = tid - 64;                   // token inside the tile; later output column j
        const int wq = warp - 2;
        float l[HQ];
#pragma unroll
        for (int h = 0; h < HQ; ++h) l[h] = 0.f;
        // exact maximum of every head over the WHOLE sequence, from the quarter-tile maxima the score kernel wrote
        // ([tile][4 quarters] per head: one 16-byte load per tile, eight tiles in flight per thread)
        for (int idx = t; idx < HQ * 4; idx += P_SOFT) {          // (head, tile phase)
            const int h = idx >> 2, ph = idx & 3;
            const float4* tp = reinterpret_cast<const float4*>(p.tmax + ((long long)s * p.H_q + h) * (4 * p.tiles));
            float v = -INFINITY;
            int i = ph;
            for (; i + 28 < tiles_s; i += 32) {
                float4 q[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) q[u] = tp[i + 4 * u];
#pragma unroll
                for (int u = 0; u < 8; ++u) v = fmaxf(v, fmaxf(fmaxf(q[u].x, q[u].y), fmaxf(q[u].z, q[u].w)));
            }
            for (; i < tiles_s; i += 4) {
                const float4 q = tp[i];
                v = fmaxf(v, fmaxf(fmaxf(q.x, q.y), fmaxf(q.z, q.w)));
            }
            sm.red[ph][h] = v;
        }
        asm volatile("bar.sync 2, 128;" ::: "memory");
        if (t < HQ) sm.m_s[t] = fmaxf(fmaxf(sm.red[0][t], sm.red[1][t]), fmaxf(sm.red[2][t], sm.red[3][t]));
        asm volatile("bar.sync 2, 128;" ::: "memory");

        // Scores of a tile are loaded one tile ahead, all heads at once.  The loads and the shared-memory stores are
        // volatile asm, which keeps them in program order: loads of tile i + 1, then stores of tile i.
        float sv[HQ];
        {
            const int n = t_begin + t;
            const float* sp = p.scores + (long long)s * p.H_q * p.n_pad + n;
#pragma unroll
            for (int h = 0; h < HQ; ++h) sv[h] = (ntiles > 0 && n < t_end) ? ldg_nc_f32(sp + (long long)h * p.n_pad) : 0.f;
        }
        for (int i = 0; i < ntiles; ++i) {
            const int buf = i & 1;
            if (!mbar_wait(&sm.p_empty[buf], ((i >> 1) & 1) ^ 1)) { ok = false; break; }
            const bool valid = t_begin + i * TILE + t < t_end;
            // p = 2^(s - m), rounded to bf16 (the same rounded value enters the denominator)
            bf16 pr[HQ];
            float ssum = 0.f;
#pragma unroll
            for (int h = 0; h < HQ; ++h) {
                ssum += sv[h];
                pr[h] = __float2bfloat16_rn(valid ? exp2f(sv[h] - sm.m_s[h]) : 0.f);
                l[h] += __bfloat162float(pr[h]);
            }
            // a NaN among the scores means non-finite numbers in the cache, the factors or the query
            if (ssum != ssum) lorc_set_status(p.status, LORC_ERR_ARG);
            {
                const int nn = t_begin + (i + 1) * TILE + t;
                const float* sp = p.scores + (long long)s * p.H_q * p.n_pad + nn;
#pragma unroll
                for (int h = 0; h < HQ; ++h) sv[h] = (i + 1 < ntiles && nn < t_end) ? ldg_nc_f32(sp + (long long)h * p.n_pad) : 0.f;
            }
            const uint32_t pb = smem_u32(sm.P[buf][t >> 6]);
            const int tc = t & 63;
#pragma unroll
            for (int h = 0; h < HQ; ++h) {
                const int off = h * 128 + ((((tc >> 3) ^ (h & 7)) << 4) | ((tc & 7) << 1));
                asm volatile("st.shared.b16 [%0], %1;" ::"r"(pb + off), "h"(__bfloat16_as_ushort(pr[h])));
            }
            fence_proxy_async_smem();
            mbar_arrive(&sm.p_full[buf]);
        }
        // softmax denominator of this context share (written once per share, by the CTA of block 0)
#pragma unroll
        for (int h = 0; h < HQ; ++h) {
            float v = l[h];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == 0) sm.red[wq][h] = v;
        }
        asm volatile("bar.sync 2, 128;" ::: "memory");
        if (blk == 0 && t < HQ)
            p.l_part[((long long)s * p.n_csplit + cs) * p.H_q + t] =
                (ntiles > 0 && ok) ? sm.red[0][t] + sm.red[1][t] + sm.red[2][t] + sm.red[3][t] : 0.f;

        // this CTA's piece of the un-normalised latent output: TMEM lane = latent row of the block
        if (ntiles > 0 && ok) {
            if (!mbar_wait(&sm.o_full, 0)) ok = false;
        }
        {
            const int quarter = warp % 4;
            const int r_pad = p.n_blk * 128;
            float* op = p.o_part + (((long long)s * p.n_csplit + cs) * p.H_q) * r_pad + rho0 + quarter * 32 + lane;
            if (ntiles > 0 && ok) tc_fence_after_sync();
#pragma unroll
            for (int c0 = 0; c0 < HQ; c0 += 32) {
                uint32_t r[32];
                if (ntiles > 0 && ok) {
                    tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + c0, r);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = 0u;
                }
#pragma unroll
                for (int i = 0; i < 32; ++i) op[(long long)(c0 + i) * r_pad] = __uint_as_float(r[i]);
            }
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, TM_COLS);
}

}  // namespace

namespace {

// ------------------------------------------------------------------------------------------------
// value up-projection: out[(s, h), :] = (sum_shares O_lat[s, share, h, :] / l[s, h]) . B_V[:, g(h)]
// grid (n_kv_heads, ceil(batch * G / 128)); warp 0 TMA (B_V^T slices), warp 1 MMA, warps 2..5 build
// the A operand (one output row per thread) and write the result.
// ------------------------------------------------------------------------------------------------
constexpr int U_BSTAGES = 4;
constexpr int U_THREADS = 192;

struct UpSmem {
    bf16 A[2][128 * KC];                  // normalised latent rows [128 rows][64 rho], K-major, 128-byte swizzle
    bf16 B[U_BSTAGES][128 * KC];          // B_V^T slice [128 columns j][64 rho] by TMA
    uint64_t a_full[2], a_empty[2], b_full[U_BSTAGES], b_empty[U_BSTAGES], d_full;
    uint32_t tmem_base;
};

struct UpParams {
    const float* o_part;           // [b, n_csplit, H_q, r_pad]
    const float* l_part;           // [b, n_csplit, H_q]
    bf16* out;                     // [b, H_q, 128]
    int* status;
    int batch, H_q, G, r_v, r_pad, n_csplit;
};

__global__ void __launch_bounds__(U_THREADS, 1)
lorc_upproj_kernel(const __grid_constant__ CUtensorMap mapBVT, const UpParams p) {
    extern __shared__ uint8_t raw[];
    UpSmem& sm = *reinterpret_cast<UpSmem*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int g = blockIdx.x, chunk = blockIdx.y;
    const int nkc = (p.r_v + KC - 1) / KC;
    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sm.a_full[i], 128);
            mbar_init(&sm.a_empty[i], 1);
        }
        for (int i = 0; i < U_BSTAGES; ++i) {
            mbar_init(&sm.b_full[i], 1);
            mbar_init(&sm.b_empty[i], 1);
        }
        mbar_init(&sm.d_full, 1);
        fence_barrier_init();
        prefetch_tensormap(&mapBVT);
    }
    if (warp == 1) {
        tmem_alloc(&sm.tmem_base, 128);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    bool ok = true;

    if (warp == 0) {
        if (lane == 0) {
            for (int kc = 0; kc < nkc; ++kc) {
                const int st = kc % U_BSTAGES;
                if (!mbar_wait(&sm.b_empty[st], ((kc / U_BSTAGES) & 1) ^ 1)) { ok = false; break; }
                mbar_arrive_expect_tx(&sm.b_full[st], 128 * KC * 2);
                tma_load_2d(sm.B[st], &mapBVT, &sm.b_full[st], kc * KC, g * 128);
            }
            if (!ok) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(128, 128, 0, 0);
            for (int kc = 0; kc < nkc; ++kc) {
                const int sa = kc & 1, sb = kc % U_BSTAGES;
                if (!mbar_wait(&sm.a_full[sa], (kc >> 1) & 1)) { ok = false; break; }
                if (!mbar_wait(&sm.b_full[sb], (kc / U_BSTAGES) & 1)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t a0 = smem_u32(sm.A[sa]), b0 = smem_u32(sm.B[sb]);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    tc_mma_bf16(tmem, make_smem_desc_sw128(a0 + k * 32, 0, 1024), make_smem_desc_sw128(b0 + k * 32, 0, 1024),
                                idesc, (kc | k) != 0);
                tc_commit(&sm.a_empty[sa]);
                tc_commit(&sm.b_empty[sb]);
            }
            tc_commit(&sm.d_full);
            if (!ok) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
        }
    } else {
        const int t = tid - 64;                        // output row inside this CTA
        const int R = chunk * 128 + t;                 // (sequence, head of the group)
        const int s = R / p.G, i = R - s * p.G;
        const int h = g * p.G + i;
        const bool live = s < p.batch;
        float inv = 0.f;
        if (live) {
            float L = 0.f;
            for (int c = 0; c < p.n_csplit; ++c) L += p.l_part[((long long)s * p.n_csplit + c) * p.H_q + h];
            if (L > 0.f) inv = 1.f / L;
            else if (i == 0) lorc_set_status(p.status, LORC_ERR_EMPTY);
        }
        const float* orow = p.o_part + ((long long)s * p.n_csplit * p.H_q + h) * p.r_pad;
        const long long share_stride = (long long)p.H_q * p.r_pad;
        for (int kc = 0; kc < nkc; ++kc) {
            const int sa = kc & 1;
            // the 64 latent columns of this row, summed over the context shares (loads first, then the wait)
            float4 v[16];
#pragma unroll
            for (int q4 = 0; q4 < 16; ++q4) v[q4] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (live && inv != 0.f) {
                for (int c = 0; c < p.n_csplit; ++c) {
                    const float4* src = reinterpret_cast<const float4*>(orow + c * share_stride + kc * KC);
#pragma unroll
                    for (int q4 = 0; q4 < 16; ++q4) {
                        const float4 x = __ldg(src + q4);
                        v[q4].x += x.x; v[q4].y += x.y; v[q4].z += x.z; v[q4].w += x.w;
                    }
                }
            }
            if (!mbar_wait(&sm.a_empty[sa], ((kc >> 1) & 1) ^ 1)) { ok = false; break; }
            const uint32_t arow = smem_u32(sm.A[sa]) + t * 128;
#pragma unroll
            for (int c8 = 0; c8 < 8; ++c8) {           // 16-byte chunks of the 128-byte row
                const float4 x = v[2 * c8], y = v[2 * c8 + 1];
                __nv_bfloat162 b0 = __floats2bfloat162_rn(x.x * inv, x.y * inv), b1 = __floats2bfloat162_rn(x.z * inv, x.w * inv);
                __nv_bfloat162 b2 = __floats2bfloat162_rn(y.x * inv, y.y * inv), b3 = __floats2bfloat162_rn(y.z * inv, y.w * inv);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(arow + ((c8 ^ (t & 7)) << 4)),
                             "r"(*reinterpret_cast<uint32_t*>(&b0)), "r"(*reinterpret_cast<uint32_t*>(&b1)),
                             "r"(*reinterpret_cast<uint32_t*>(&b2)), "r"(*reinterpret_cast<uint32_t*>(&b3)));
            }
            fence_proxy_async_smem();
            mbar_arrive(&sm.a_full[sa]);
        }
        if (ok && !mbar_wait(&sm.d_full, 0)) ok = false;
        if (ok) {
            tc_fence_after_sync();
            const int quarter = warp % 4;
            // TMEM lane = output row; the warp's lane quarter decides which rows it can read
            const int row = quarter * 32 + lane;
            const int R2 = chunk * 128 + row;
            const int s2 = R2 / p.G, h2 = g * p.G + (R2 - s2 * p.G);
#pragma unroll
            for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + c0, r);
                tmem_wait_ld();
                if (s2 < p.batch) {
                    uint4* dst = reinterpret_cast<uint4*>(p.out + ((long long)s2 * p.H_q + h2) * 128 + c0);
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(r[q4 * 8 + 2 * e]),
                                                                     __uint_as_float(r[q4 * 8 + 2 * e + 1]));
                            w[e] = *reinterpret_cast<uint32_t*>(&b);
                        }
                        dst[q4] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 128);
}

// Column blocks and context shares of one PV launch: two CTAs fit on an SM, so aim at filling those slots once.
void pv_plan(const lorc_ctx* ctx, const LorcLayer& L, int batch, int max_seq_len, int n_splits_hint, int* n_blk,
             int* n_csplit) {
    const int tiles = (max_seq_len + TILE - 1) / TILE;
    *n_blk = (L.r_v + 127) / 128;
    const int slots = 2 * ctx->sm_count;
    int cs = n_splits_hint > 0 ? n_splits_hint : slots / (batch * *n_blk);
    if (cs > tiles) cs = tiles;
    if (cs > 64) cs = 64;
    if (cs < 1) cs = 1;
    *n_csplit = cs;
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
size_t lorc_tc_pv_scratch_bytes(const lorc_ctx* ctx, int batch, int max_seq_len) {
    // the planned number of context shares for the narrowest layer (one column block), which is the largest
    const int tiles = (max_seq_len + TILE - 1) / TILE;
    int cs = 2 * ctx->sm_count / batch;
    if (cs > tiles) cs = tiles;
    if (cs > 64) cs = 64;
    if (cs < 1) cs = 1;
    const size_t r_pad = (size_t)((ctx->n + 127) / 128) * 128;
    return lorc_align_up((size_t)batch * cs * ctx->desc.n_q_heads * r_pad * sizeof(float), 256) +
           lorc_align_up((size_t)batch * cs * ctx->desc.n_q_heads * sizeof(float), 256);
}

cudaError_t lorc_tc_pv_launch(lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, const CUtensorMap& mapCV,
                              const CUtensorMap& mapBVT, const float* scores, const float* tmax, int n_pad, int tiles,
                              int n_splits_hint, void* scratch, size_t scratch_bytes, bf16* out, cudaStream_t st,
                              int* launches) {
    const lorc_model_desc& d = ctx->desc;
    static bool attr = false;
    if (!attr) {
        cudaError_t e = cudaFuncSetAttribute(lorc_pv2_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)sizeof(Pv2Smem<32>) + 1024);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(lorc_pv2_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)sizeof(Pv2Smem<64>) + 1024);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(lorc_upproj_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)sizeof(UpSmem) + 1024);
        if (e != cudaSuccess) return e;
        attr = true;
    }
    int n_blk, n_csplit;
    pv_plan(ctx, L, cv.batch, cv.max_seq_len, n_splits_hint, &n_blk, &n_csplit);
    const int r_pad = n_blk * 128;
    size_t part_bytes, l_bytes;
    for (;; --n_csplit) {
        part_bytes = lorc_align_up((size_t)cv.batch * n_csplit * d.n_q_heads * r_pad * sizeof(float), 256);
        l_bytes = lorc_align_up((size_t)cv.batch * n_csplit * d.n_q_heads * sizeof(float), 256);
        if (part_bytes + l_bytes <= scratch_bytes) break;
        if (n_csplit == 1) return cudaErrorMemoryAllocation;
    }
    Pv2Params p;
    p.scores = scores; p.tmax = tmax;
    p.o_part = (float*)scratch;
    p.l_part = (float*)((char*)scratch + part_bytes);
    p.seq_lens = cv.seq_lens; p.page_table = cv.page_table; p.status = ctx->status_dev;
    p.batch = cv.batch; p.H_q = d.n_q_heads; p.n_kv = d.n_kv_heads; p.r_v = L.r_v; p.n_pad = n_pad; p.tiles = tiles;
    p.n_blk = n_blk; p.n_csplit = n_csplit; p.max_pos = d.max_pos;
    p.page_size = cv.page_size; p.max_pages_per_seq = cv.max_pages_per_seq; p.n_pages = cv.n_pages;
    dim3 grid(n_blk, n_csplit, cv.batch);
    {
        LorcStageTimer timer(ctx, LORC_STAGE_PV, st);
        if (d.n_q_heads == 32)
            lorc_pv2_kernel<32><<<grid, P_THREADS, sizeof(Pv2Smem<32>) + 1024, st>>>(mapCV, p);
        else
            lorc_pv2_kernel<64><<<grid, P_THREADS, sizeof(Pv2Smem<64>) + 1024, st>>>(mapCV, p);
    }
    *launches += 1;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    UpParams u;
    u.o_part = p.o_part; u.l_part = p.l_part; u.out = out; u.status = ctx->status_dev;
    u.batch = cv.batch; u.H_q = d.n_q_heads; u.G = ctx->group; u.r_v = L.r_v; u.r_pad = r_pad; u.n_csplit = n_csplit;
    {
        LorcStageTimer timer(ctx, LORC_STAGE_COMBINE, st);
        dim3 ugrid(d.n_kv_heads, (cv.batch * ctx->group + 127) / 128);
        lorc_upproj_kernel<<<ugrid, U_THREADS, sizeof(UpSmem) + 1024, st>>>(mapBVT, u);
    }
    *launches += 1;
    return cudaGetLastError();
}
