// Softmax + P.C_V + value up-projection on the tensor cores, split by LATENT COLUMNS.
//
// A CTA owns one 128-column block of C_V (rho in [128 blk, 128 blk + 128)) of one sequence and one
// share of its context.  Because a block of latent columns is disjoint from every other block, the
// CTA's accumulator O_lat^T[128 rho, H_q] (fp32 in TMEM) needs no merge with other column blocks;
// and because every CTA uses the same exact row maximum (taken from the quarter-tile maxima the score
// kernel leaves behind), context shares of the same block add up directly.  The CTA therefore
// finishes its own piece of the output, out_part[h, :] = sum_rho O_lat[h, rho] B_V[rho, g(h)], against
// the 128 rows of B_V it owns, and writes 16 KiB (H_q = 32) instead of a full latent-space partial.
// A small kernel adds the pieces in a fixed order and divides by the softmax denominator, so results
// do not depend on scheduling.
//
//   per tile of 128 tokens:  p = 2^(s - m) (bf16, K-major in shared memory)        softmax warps
//                            O_lat^T += C_V[tile, block]^T . P^T                    tcgen05, MN-major A
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
constexpr int BV_SLOTS = 5;           // B_V pieces of 64 rows (16 KiB): four in the C_V stages, one in the P buffers

// read-only global load that the compiler keeps in program order with the other volatile asm of this file
__device__ __forceinline__ float ldg_nc_f32(const float* p) {
    float v;
    asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}

template <int HQ>
struct Pv2Smem {
    bf16 V[P_STAGES][2][TILE * KC];       // C_V block: two 64-column halves of [128 tokens][64]; 32 KiB / stage.
                                          // After the last MMA: ring of B_V pieces [64 rho][128 columns of one KV head]
    bf16 P[2][2][HQ * KC];                // probabilities [HQ][128 tokens] as two 64-token chunks, 128-byte swizzle
    float o_sm[128][HQ];                  // O_lat block [rho][head] after the last MMA
    float m_s[HQ];
    float red[4][HQ];
    uint64_t full[P_STAGES], empty[P_STAGES], p_full[2], p_empty[2], o_full, bv_full[BV_SLOTS], bv_empty[BV_SLOTS];
    uint32_t tmem_base;
};

struct Pv2Params {
    const float* scores;           // [b, H_q, n_pad]      log2 units
    const float* tmax;             // [b, H_q, tiles, 4]   maxima of every 32-token quarter tile
    float* out_part;               // [b, n_blk * n_csplit, H_q, 128]
    float* l_part;                 // [b, n_csplit, H_q]
    const int32_t* seq_lens;
    const int32_t* page_table;
    int* status;
    int batch, H_q, n_kv, r_v, n_pad, tiles, n_blk, n_csplit, max_pos;
    int page_size, max_pages_per_seq, n_pages;
};

template <int HQ>
__global__ void __launch_bounds__(P_THREADS, 2)
lorc_pv2_kernel(const __grid_constant__ CUtensorMap mapCV, const __grid_constant__ CUtensorMap mapBV,
                const Pv2Params p) {
    extern __shared__ uint8_t raw[];
    typedef Pv2Smem<HQ> S;
    S& sm = *reinterpret_cast<S*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    constexpr int G_MAX = 8;
    constexpr uint32_t TM_COLS = HQ <= 32 ? 32 : 64;
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int blk = blockIdx.x, cs = blockIdx.y, s = blockIdx.z;
    const int G = HQ / p.n_kv;

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
    const int rows_valid = min(128, p.r_v - rho0);       // latent rows of this block that exist
    const int n_bv = (ntiles > 0) ? 2 * p.n_kv : 0;      // B_V pieces to stream: (KV head, half of the block's rows)

    if (tid == 0) {
        for (int i = 0; i < P_STAGES; ++i) {
            mbar_init(&sm.full[i], 1);
            mbar_init(&sm.empty[i], 1);
        }
        for (int i = 0; i < BV_SLOTS; ++i) {
            mbar_init(&sm.bv_full[i], 1);
            mbar_init(&sm.bv_empty[i], P_SOFT);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sm.p_full[i], P_SOFT);
            mbar_init(&sm.p_empty[i], 1);
        }
        mbar_init(&sm.o_full, 1);
        fence_barrier_init();
        prefetch_tensormap(&mapCV);
        prefetch_tensormap(&mapBV);
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
            // the rows of B_V this block multiplies with, in pieces of 64 rows x 128 columns (one KV head), through a
            // ring that reuses the C_V stages and the P buffers (all free once every MMA has retired)
            if (n_bv > 0 && ok && !mbar_wait(&sm.o_full, 0)) ok = false;
            for (int c = 0; c < n_bv && ok; ++c) {
                const int slot = c % BV_SLOTS;
                if (!mbar_wait(&sm.bv_empty[slot], ((c / BV_SLOTS) & 1) ^ 1)) { ok = false; break; }
                bf16* dst = (slot < 4) ? (&sm.V[0][0][0] + slot * 64 * 128) : &sm.P[0][0][0];
                mbar_arrive_expect_tx(&sm.bv_full[slot], 64 * 128 * 2);
                tma_load_2d(dst, &mapBV, &sm.bv_full[slot], (c >> 1) * 128, rho0 + (c & 1) * 64);
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

        float* op = p.out_part + (((long long)s * (p.n_blk * p.n_csplit) + blk * p.n_csplit + cs) * p.H_q) * 128;
        if (ntiles > 0 && ok) {
            if (!mbar_wait(&sm.o_full, 0)) ok = false;
        }
        if (ntiles > 0 && ok) {
            tc_fence_after_sync();
            // TMEM lane = latent row of the block; this warp reads lane quarter (warp % 4)
            const int quarter = warp % 4;
            const int row = quarter * 32 + lane;
#pragma unroll
            for (int c0 = 0; c0 < HQ; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + c0, r);
                tmem_wait_ld();
#pragma unroll
                for (int i4 = 0; i4 < 8; ++i4)
                    *reinterpret_cast<float4*>(&sm.o_sm[row][c0 + i4 * 4]) =
                        make_float4(__uint_as_float(r[i4 * 4]), __uint_as_float(r[i4 * 4 + 1]),
                                    __uint_as_float(r[i4 * 4 + 2]), __uint_as_float(r[i4 * 4 + 3]));
            }
        }
        asm volatile("bar.sync 2, 128;" ::: "memory");
        // out_part[h][j] = sum_rho O_lat[rho][h] * B_V[rho0 + rho][g(h) * 128 + j], thread = column j
        {
            float acc[G_MAX];
            for (int c = 0; c < n_bv; ++c) {
                const int slot = c % BV_SLOTS, g = c >> 1, half = c & 1;
                if (half == 0) {
#pragma unroll
                    for (int i = 0; i < G_MAX; ++i) acc[i] = 0.f;
                }
                if (ok && !mbar_wait(&sm.bv_full[slot], (c / BV_SLOTS) & 1)) ok = false;
                if (ok) {
                    const bf16* bv = ((slot < 4) ? (&sm.V[0][0][0] + slot * 64 * 128) : &sm.P[0][0][0]) + t;
                    const int r_lo = half * 64;
                    const int rows = max(0, min(64, rows_valid - r_lo));
                    if (G == 4) {
#pragma unroll 8
                        for (int r = 0; r < rows; ++r) {
                            const float b = __bfloat162float(bv[r * 128]);
                            const float4 o = *reinterpret_cast<const float4*>(&sm.o_sm[r_lo + r][g * 4]);
                            acc[0] = fmaf(o.x, b, acc[0]);
                            acc[1] = fmaf(o.y, b, acc[1]);
                            acc[2] = fmaf(o.z, b, acc[2]);
                            acc[3] = fmaf(o.w, b, acc[3]);
                        }
                    } else {
#pragma unroll 4
                        for (int r = 0; r < rows; ++r) {
                            const float b = __bfloat162float(bv[r * 128]);
                            const float4 o0 = *reinterpret_cast<const float4*>(&sm.o_sm[r_lo + r][g * 8]);
                            const float4 o1 = *reinterpret_cast<const float4*>(&sm.o_sm[r_lo + r][g * 8 + 4]);
                            acc[0] = fmaf(o0.x, b, acc[0]);
                            acc[1] = fmaf(o0.y, b, acc[1]);
                            acc[2] = fmaf(o0.z, b, acc[2]);
                            acc[3] = fmaf(o0.w, b, acc[3]);
                            acc[4] = fmaf(o1.x, b, acc[4]);
                            acc[5] = fmaf(o1.y, b, acc[5]);
                            acc[6] = fmaf(o1.z, b, acc[6]);
                            acc[7] = fmaf(o1.w, b, acc[7]);
                        }
                    }
                    mbar_arrive(&sm.bv_empty[slot]);
                }
                if (half == 1)
                    for (int i = 0; i < G; ++i) op[(long long)(g * G + i) * 128 + t] = ok ? acc[i] : 0.f;
            }
        }
        if (ntiles == 0) {
            for (int h = 0; h < HQ; ++h) op[(long long)h * 128 + t] = 0.f;
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, TM_COLS);
}

}  // namespace

namespace {

// out[s][h][:] = (sum over pieces of out_part) / (sum over context shares of l), pieces added in index order.
// grid (H_q / 4, batch), 512 threads = 4 heads x 128 columns.
__global__ void __launch_bounds__(512)
lorc_pv_finalize_kernel(const float* __restrict__ out_part, const float* __restrict__ l_part, bf16* __restrict__ out,
                        int H_q, int n_parts, int n_csplit, int* status) {
    const int s = blockIdx.y;
    const int h = blockIdx.x * 4 + (threadIdx.x >> 7), j = threadIdx.x & 127;
    float L = 0.f;
    for (int c = 0; c < n_csplit; ++c) L += l_part[((long long)s * n_csplit + c) * H_q + h];
    const float* op = out_part + ((long long)s * n_parts * H_q + h) * 128 + j;
    float a = 0.f;
    int c = 0;
    for (; c + 8 <= n_parts; c += 8) {
        float v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = op[(long long)(c + u) * H_q * 128];
#pragma unroll
        for (int u = 0; u < 8; ++u) a += v[u];
    }
    for (; c < n_parts; ++c) a += op[(long long)c * H_q * 128];
    if (!(L > 0.f)) {
        if (j == 0) lorc_set_status(status, LORC_ERR_EMPTY);
        a = 0.f;
        L = 1.f;
    }
    out[((long long)s * H_q + h) * 128 + j] = __float2bfloat16_rn(a / L);
}

// Column blocks and context shares of one launch: two CTAs fit on an SM, so aim at filling those slots once.
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
    // any layer (up to n / 128 column blocks) with the number of context shares the plan picks for it, or a
    // forced share count as far as it fits (the launch lowers the count until the pieces fit)
    const int tiles = (max_seq_len + TILE - 1) / TILE;
    const int n_blk_max = (ctx->n + 127) / 128;
    int cs = 2 * ctx->sm_count / batch;          // n_blk * n_csplit <= slots / batch for every n_blk
    if (cs < n_blk_max) cs = n_blk_max;
    int cs_l = tiles < 64 ? tiles : 64;
    return lorc_align_up((size_t)batch * cs * ctx->desc.n_q_heads * 128 * sizeof(float), 256) +
           lorc_align_up((size_t)batch * cs_l * ctx->desc.n_q_heads * sizeof(float), 256);
}

cudaError_t lorc_tc_pv_launch(lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, const CUtensorMap& mapCV,
                              const CUtensorMap& mapBV, const float* scores, const float* tmax, int n_pad, int tiles,
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
        if (e != cudaSuccess) return e;
        attr = true;
    }
    int n_blk, n_csplit;
    pv_plan(ctx, L, cv.batch, cv.max_seq_len, n_splits_hint, &n_blk, &n_csplit);
    size_t part_bytes, l_bytes;
    for (;; --n_csplit) {
        part_bytes = lorc_align_up((size_t)cv.batch * n_blk * n_csplit * d.n_q_heads * 128 * sizeof(float), 256);
        l_bytes = lorc_align_up((size_t)cv.batch * n_csplit * d.n_q_heads * sizeof(float), 256);
        if (part_bytes + l_bytes <= scratch_bytes) break;
        if (n_csplit == 1) return cudaErrorMemoryAllocation;
    }
    Pv2Params p;
    p.scores = scores; p.tmax = tmax;
    p.out_part = (float*)scratch;
    p.l_part = (float*)((char*)scratch + part_bytes);
    p.seq_lens = cv.seq_lens; p.page_table = cv.page_table; p.status = ctx->status_dev;
    p.batch = cv.batch; p.H_q = d.n_q_heads; p.n_kv = d.n_kv_heads; p.r_v = L.r_v; p.n_pad = n_pad; p.tiles = tiles;
    p.n_blk = n_blk; p.n_csplit = n_csplit; p.max_pos = d.max_pos;
    p.page_size = cv.page_size; p.max_pages_per_seq = cv.max_pages_per_seq; p.n_pages = cv.n_pages;
    dim3 grid(n_blk, n_csplit, cv.batch);
    {
        LorcStageTimer timer(ctx, LORC_STAGE_PV, st);
        if (d.n_q_heads == 32)
            lorc_pv2_kernel<32><<<grid, P_THREADS, sizeof(Pv2Smem<32>) + 1024, st>>>(mapCV, mapBV, p);
        else
            lorc_pv2_kernel<64><<<grid, P_THREADS, sizeof(Pv2Smem<64>) + 1024, st>>>(mapCV, mapBV, p);
    }
    *launches += 1;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    {
        LorcStageTimer timer(ctx, LORC_STAGE_COMBINE, st);
        lorc_pv_finalize_kernel<<<dim3(d.n_q_heads / 4, cv.batch), 512, 0, st>>>(
            p.out_part, p.l_part, out, d.n_q_heads, n_blk * n_csplit, n_csplit, ctx->status_dev);
    }
    *launches += 1;
    return cudaGetLastError();
}
