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
// normalise: o_norm[s, h, rho] = bf16( sum_shares O_lat[s, share, h, rho] / sum_shares l[s, share, h] )
// one thread per 4 latent columns
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
lorc_normalize_kernel(const float* __restrict__ o_part, const float* __restrict__ l_part, bf16* __restrict__ o_norm,
                      int H_q, int r_pad, int n_csplit, long long total4, int* status) {
    const long long i4 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i4 >= total4) return;
    const int r4n = r_pad >> 2;
    const long long row = i4 / r4n;                   // s * H_q + h
    const int r4 = (int)(i4 - row * r4n);
    const int s = (int)(row / H_q), h = (int)(row - (long long)s * H_q);
    const long long share_stride4 = (long long)H_q * r4n;
    const float4* src = reinterpret_cast<const float4*>(o_part) + ((long long)s * n_csplit * H_q + h) * r4n + r4;
    const float* lp = l_part + (long long)s * n_csplit * H_q + h;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    float L = 0.f;
    int c = 0;
    for (; c + 4 <= n_csplit; c += 4) {
        float4 v[4];
        float l[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            v[u] = __ldg(src + (c + u) * share_stride4);
            l[u] = __ldg(lp + (long long)(c + u) * H_q);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            a.x += v[u].x; a.y += v[u].y; a.z += v[u].z; a.w += v[u].w;
            L += l[u];
        }
    }
    for (; c < n_csplit; ++c) {
        const float4 v = __ldg(src + c * share_stride4);
        a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
        L += __ldg(lp + (long long)c * H_q);
    }
    float inv = 0.f;
    if (L > 0.f) inv = 1.f / L;
    else if (r4 == 0) lorc_set_status(status, LORC_ERR_EMPTY);
    __nv_bfloat162 b0 = __floats2bfloat162_rn(a.x * inv, a.y * inv), b1 = __floats2bfloat162_rn(a.z * inv, a.w * inv);
    uint2 w = make_uint2(*reinterpret_cast<uint32_t*>(&b0), *reinterpret_cast<uint32_t*>(&b1));
    reinterpret_cast<uint2*>(o_norm)[i4] = w;
}

// ------------------------------------------------------------------------------------------------
// value up-projection: out[(s, h), :] = o_norm[s, h, :] . B_V[:, g(h)], a plain TMA-fed tcgen05 GEMM.
// grid (n_kv_heads, ceil(batch * G / 128)): 128 output rows (s, i) x 128 columns, K = r_v in slices of 64.
// ------------------------------------------------------------------------------------------------
constexpr int U_STAGES = 6;
constexpr int U_THREADS = 192;

struct UpSmem {
    bf16 A[U_STAGES][128 * KC];           // o_norm rows [128 rows (s, i)][64 rho]
    bf16 B[U_STAGES][128 * KC];           // B_V^T slice [128 columns j][64 rho]
    uint64_t full[U_STAGES], empty[U_STAGES], d_full;
    uint32_t tmem_base;
};

struct UpParams {
    bf16* out;                     // [b, H_q, 128]
    int* status;
    int batch, H_q, G, r_v;
};

__global__ void __launch_bounds__(U_THREADS, 1)
lorc_upproj_kernel(const __grid_constant__ CUtensorMap mapON, const __grid_constant__ CUtensorMap mapBVT,
                   const UpParams p) {
    extern __shared__ uint8_t raw[];
    UpSmem& sm = *reinterpret_cast<UpSmem*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int g = blockIdx.x, chunk = blockIdx.y;
    const int nkc = (p.r_v + KC - 1) / KC;
    const int seqs_per_cta = 128 / p.G;
    if (tid == 0) {
        for (int i = 0; i < U_STAGES; ++i) {
            mbar_init(&sm.full[i], 1);
            mbar_init(&sm.empty[i], 1);
        }
        mbar_init(&sm.d_full, 1);
        fence_barrier_init();
        prefetch_tensormap(&mapON);
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
                const int st = kc % U_STAGES;
                if (!mbar_wait(&sm.empty[st], ((kc / U_STAGES) & 1) ^ 1)) { ok = false; break; }
                mbar_arrive_expect_tx(&sm.full[st], 2 * 128 * KC * 2);
                // rows (s, i): box of G heads x 128/G sequences (sequences past the batch read as zero)
                tma_load_3d(sm.A[st], &mapON, &sm.full[st], kc * KC, g * p.G, chunk * seqs_per_cta);
                tma_load_2d(sm.B[st], &mapBVT, &sm.full[st], kc * KC, g * 128);
            }
            if (!ok) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(128, 128, 0, 0);
            for (int kc = 0; kc < nkc; ++kc) {
                const int st = kc % U_STAGES;
                if (!mbar_wait(&sm.full[st], (kc / U_STAGES) & 1)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t a0 = smem_u32(sm.A[st]), b0 = smem_u32(sm.B[st]);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    tc_mma_bf16(tmem, make_smem_desc_sw128(a0 + k * 32, 0, 1024), make_smem_desc_sw128(b0 + k * 32, 0, 1024),
                                idesc, (kc | k) != 0);
                tc_commit(&sm.empty[st]);
            }
            tc_commit(&sm.d_full);
            if (!ok) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
        }
    } else {
        if (!mbar_wait(&sm.d_full, 0)) ok = false;
        if (ok) {
            tc_fence_after_sync();
            // TMEM lane = output row (s_local * G + i); the warp's lane quarter decides which rows it reads
            const int quarter = warp % 4;
            const int row = quarter * 32 + lane;
            const int s = chunk * seqs_per_cta + row / p.G, h = g * p.G + row % p.G;
#pragma unroll
            for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + c0, r);
                tmem_wait_ld();
                if (s < p.batch) {
                    uint4* dst = reinterpret_cast<uint4*>(p.out + ((long long)s * p.H_q + h) * 128 + c0);
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
           lorc_align_up((size_t)batch * cs * ctx->desc.n_q_heads * sizeof(float), 256) +
           lorc_align_up((size_t)batch * ctx->desc.n_q_heads * r_pad * sizeof(bf16), 256);
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
    const size_t on_bytes = lorc_align_up((size_t)cv.batch * d.n_q_heads * r_pad * sizeof(bf16), 256);
    for (;; --n_csplit) {
        part_bytes = lorc_align_up((size_t)cv.batch * n_csplit * d.n_q_heads * r_pad * sizeof(float), 256);
        l_bytes = lorc_align_up((size_t)cv.batch * n_csplit * d.n_q_heads * sizeof(float), 256);
        if (part_bytes + l_bytes + on_bytes <= scratch_bytes) break;
        if (n_csplit == 1) return cudaErrorMemoryAllocation;
    }
    bf16* o_norm = (bf16*)((char*)scratch + part_bytes + l_bytes);
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
    LorcStageTimer timer(ctx, LORC_STAGE_COMBINE, st);
    const long long total4 = (long long)cv.batch * d.n_q_heads * (r_pad / 4);
    lorc_normalize_kernel<<<(unsigned)((total4 + 255) / 256), 256, 0, st>>>(p.o_part, p.l_part, o_norm, d.n_q_heads, r_pad,
                                                                        n_csplit, total4, ctx->status_dev);
    *launches += 1;
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    // o_norm [b, H_q, r_pad] as (rho, head, sequence) with boxes of 64 rho x G heads x 128/G sequences
    CUtensorMap mapON;
    {
        uint64_t dims[3] = {(uint64_t)r_pad, (uint64_t)d.n_q_heads, (uint64_t)cv.batch};
        uint64_t str[2] = {(uint64_t)r_pad * 2, (uint64_t)d.n_q_heads * r_pad * 2};
        uint32_t box[3] = {KC, (uint32_t)ctx->group, (uint32_t)(128 / ctx->group)};
        if (!lorc_make_tmap_bf16(&mapON, o_norm, 3, dims, str, box)) return cudaErrorInvalidValue;
    }
    UpParams u;
    u.out = out; u.status = ctx->status_dev;
    u.batch = cv.batch; u.H_q = d.n_q_heads; u.G = ctx->group; u.r_v = L.r_v;
    dim3 ugrid(d.n_kv_heads, (cv.batch * ctx->group + 127) / 128);
    lorc_upproj_kernel<<<ugrid, U_THREADS, sizeof(UpSmem) + 1024, st>>>(mapON, mapBVT, u);
    *launches += 1;
    return cudaGetLastError();
}
