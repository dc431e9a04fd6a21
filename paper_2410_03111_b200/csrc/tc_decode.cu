// Tensor-core decode attention over the latent cache (sm_100a: TMA + tcgen05 + TMEM).
//
// Two kernels per layer, followed by the merge / value-up-projection kernel:
//
//  score kernel   persistent CTAs walk (sequence, 128-token tile, KV-head pair) units.  Per unit the
//                 key tile of two KV heads is reconstructed on the tensor cores,
//                     K[128 tokens, 256] = C_K[tile, :] . B_K[:, pair]          (fp32 in TMEM),
//                 from TMA-staged 64-wide slices of the latent tile and of B_K^T.  Eight epilogue warps
//                 (thread = token row) read the accumulator, rotate each key at its position and dot it
//                 with the G rotated queries of its KV head; the scores (log2 units) go to scratch.
//                 RoPE is split as R(n0 + t) = R(n0) R(t): R(t), t < 128, is a constant table in shared
//                 memory and R(n0) is folded into the query once per unit (q' = R(m - n0) q).
//  PV kernel      one CTA per (sequence, context split): exact row max of the split, p = 2^(s - m) as
//                 bf16 into shared memory, and O_lat^T[r_V, H_q] += C_V^T . P^T on the tensor cores with
//                 C_V consumed straight from its row-major TMA tiles (MN-major operand).
//                 Partials (m, l, O_lat) go to scratch.
//  combine        merges the splits and applies B_V (fast_aux.cu).
//
// Keys and values never exist in memory; only the 4*H_q bytes of scores per token are written.
#include <math.h>

#include "sm100_ptx.cuh"
#include "tc_kernels.cuh"

using namespace sm100;

namespace {

constexpr int TILE = 128;            // tokens per tile
constexpr int KC = 64;               // latent columns per pipeline stage
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

// ------------------------------------------------------------------------------------------------
// score kernel
// ------------------------------------------------------------------------------------------------
constexpr int S_STAGES = 3;
constexpr int S_THREADS = 320;       // warp 0 TMA, warp 1 MMA, warps 2..9 epilogue
constexpr int S_EPI = 256;

struct ScoreSmem {
    bf16 A[S_STAGES][TILE * KC];          // latent slice  [128 tokens][64]       16 KiB
    bf16 B[S_STAGES][256 * KC];           // B_K^T slice   [256 features][64]     32 KiB
    float2 trigT[64][TILE];               // (cos, sin)(t * theta_j), [j][t]      64 KiB
    float qrot[2][2][64][16];             // [buffer][head of pair][pair j][qa_0..qa_G-1, qb_0..qb_G-1]  16 KiB
    uint64_t full[S_STAGES], empty[S_STAGES], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};

struct ScoreParams {
    const bf16* q;                 // [b, H_q, 128]
    float* scores;                 // [b, H_q, n_pad]
    const int32_t* seq_lens;
    const int32_t* page_table;     // NULL: contiguous
    const float2* rope_table;      // [max_pos][64]
    const float2* rope_tile;       // [64][128]  (cos, sin)(t * theta_j)
    int* status;
    int batch, H_q, n_hp, r_k, n_pad, tiles_per_seq, max_pos;
    int page_size, max_pages_per_seq, n_pages;
};

struct Unit {
    int s, tile, hp, len;
};

__device__ __forceinline__ bool decode_unit(const ScoreParams& p, int u, Unit& un) {
    un.hp = u % p.n_hp;
    int r = u / p.n_hp;
    un.tile = r % p.tiles_per_seq;
    un.s = r / p.tiles_per_seq;
    un.len = p.seq_lens[un.s];
    return un.len > 0 && un.len <= p.max_pos && un.tile * TILE < un.len;
}

template <int G>
__global__ void __launch_bounds__(S_THREADS, 1)
lorc_score_kernel(const __grid_constant__ CUtensorMap mapCK, const __grid_constant__ CUtensorMap mapBKT,
                  const ScoreParams p) {
    extern __shared__ uint8_t raw[];
    ScoreSmem& sm = *reinterpret_cast<ScoreSmem*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int total_units = p.batch * p.tiles_per_seq * p.n_hp;
    const int nkc = (p.r_k + KC - 1) / KC;

    if (tid == 0) {
        for (int i = 0; i < S_STAGES; ++i) {
            mbar_init(&sm.full[i], 1);
            mbar_init(&sm.empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sm.acc_full[i], 1);
            mbar_init(&sm.acc_empty[i], S_EPI);
        }
        sm.abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&mapCK);
        prefetch_tensormap(&mapBKT);
    }
    if (warp == 1) {
        tmem_alloc(&sm.tmem_base, 512);
        tmem_relinquish();
    }
    // constant in-tile rotation table
    for (int i = tid; i < 64 * TILE; i += S_THREADS) (&sm.trigT[0][0])[i] = p.rope_tile[i];
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
                Unit un;
                if (!decode_unit(p, u, un)) continue;
                for (int kc = 0; kc < nkc; ++kc, ++it) {
                    const int st = it % S_STAGES;
                    const uint32_t ph = (it / S_STAGES) & 1;
                    if (!mbar_wait(&sm.empty[st], ph ^ 1)) { ok = false; break; }
                    if (p.page_table == nullptr) {
                        mbar_arrive_expect_tx(&sm.full[st], (TILE + 256) * KC * 2);
                        tma_load_3d(sm.A[st], &mapCK, &sm.full[st], kc * KC, un.tile * TILE, un.s);
                    } else {
                        const int ppt = TILE / p.page_size;          // pages per tile
                        int pages[8];
                        uint32_t bytes = 256 * KC * 2;
                        for (int pg = 0; pg < ppt; ++pg) {
                            int lp = un.tile * ppt + pg;
                            int page = -1;
                            if (lp * p.page_size < un.len && lp < p.max_pages_per_seq) {
                                page = p.page_table[(long long)un.s * p.max_pages_per_seq + lp];
                                if (page < 0 || page >= p.n_pages) {
                                    lorc_set_status(p.status, LORC_ERR_CAPACITY);
                                    page = -1;
                                }
                            }
                            pages[pg] = page;
                            if (page >= 0) bytes += p.page_size * KC * 2;
                        }
                        mbar_arrive_expect_tx(&sm.full[st], bytes);
                        for (int pg = 0; pg < ppt; ++pg)
                            if (pages[pg] >= 0)
                                tma_load_3d(sm.A[st] + pg * p.page_size * KC, &mapCK, &sm.full[st], kc * KC, 0,
                                            pages[pg]);
                    }
                    tma_load_2d(sm.B[st], &mapBKT, &sm.full[st], kc * KC, un.hp * 256);
                }
            }
            if (!ok) {
                lorc_set_status(p.status, LORC_ERR_TIMEOUT);
                sm.abort_flag = 1;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(128, 256, 0, 0);
            uint32_t it = 0, uc = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
                Unit un;
                if (!decode_unit(p, u, un)) continue;
                const int buf = uc & 1;
                if (!mbar_wait(&sm.acc_empty[buf], ((uc >> 1) & 1) ^ 1)) { ok = false; break; }
                tc_fence_after_sync();
                for (int kc = 0; kc < nkc; ++kc, ++it) {
                    const int st = it % S_STAGES;
                    if (!mbar_wait(&sm.full[st], (it / S_STAGES) & 1)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t a0 = smem_u32(sm.A[st]), b0 = smem_u32(sm.B[st]);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        tc_mma_bf16(tmem + buf * 256, make_smem_desc_sw128(a0 + k * 32, 0, 1024),
                                    make_smem_desc_sw128(b0 + k * 32, 0, 1024), idesc, (kc | k) != 0);
                    }
                    tc_commit(&sm.empty[st]);
                }
                if (!ok) break;
                tc_commit(&sm.acc_full[buf]);
                ++uc;
            }
            if (!ok) {
                lorc_set_status(p.status, LORC_ERR_TIMEOUT);
                sm.abort_flag = 1;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: RoPE + scores
        const int te = tid - 64;                  // 0..255
        const int grp = te / 128;                 // which head of the pair
        const int quarter = warp % 4;             // TMEM lane quarter this warp may read
        const int t = quarter * 32 + lane;        // token row inside the tile
        const float scale = rsqrtf(128.f) * LOG2E;
        uint32_t uc = 0;
        bool ok = true;
        for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
            Unit un;
            if (!decode_unit(p, u, un)) continue;
            const int buf = uc & 1, qb = uc & 1;
            const int n0 = un.tile * TILE;
            const int delta = un.len - 1 - n0;    // query position relative to the tile start
            for (int idx = te; idx < 2 * G * 64; idx += S_EPI) {
                const int hh = idx >> 6, j = idx & 63;
                const int hip = hh / G, g = hh - hip * G;
                const int h = (un.hp * 2 + hip) * G + g;
                const float2 cs = p.rope_table[(long long)delta * 64 + j];
                const bf16* qp = p.q + ((long long)un.s * p.H_q + h) * 128;
                const float a = __bfloat162float(qp[j]), b = __bfloat162float(qp[j + 64]);
                sm.qrot[qb][hip][j][g] = (a * cs.x - b * cs.y) * scale;
                sm.qrot[qb][hip][j][G + g] = (a * cs.y + b * cs.x) * scale;
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (!mbar_wait(&sm.acc_full[buf], (uc >> 1) & 1)) { ok = false; break; }
            tc_fence_after_sync();
            float acc[G];
#pragma unroll
            for (int g = 0; g < G; ++g) acc[g] = 0.f;
            const uint32_t tbase = tmem + ((uint32_t)(quarter * 32) << 16) + buf * 256 + grp * 128;
#pragma unroll 1
            for (int jc = 0; jc < 2; ++jc) {
                uint32_t ra[32], rb[32];
                tmem_ld32(tbase + jc * 32, ra);
                tmem_ld32(tbase + 64 + jc * 32, rb);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int j = jc * 32 + i;
                    const float2 cs = sm.trigT[j][t];
                    const float a = __uint_as_float(ra[i]), b = __uint_as_float(rb[i]);
                    const float ka = a * cs.x - b * cs.y;
                    const float kb = a * cs.y + b * cs.x;
                    const float4* qv = reinterpret_cast<const float4*>(sm.qrot[qb][grp][j]);
                    float qa[G], qbv[G];
#pragma unroll
                    for (int g4 = 0; g4 < G / 4; ++g4) {
                        const float4 x = qv[g4], y = qv[G / 4 + g4];
                        qa[g4 * 4 + 0] = x.x; qa[g4 * 4 + 1] = x.y; qa[g4 * 4 + 2] = x.z; qa[g4 * 4 + 3] = x.w;
                        qbv[g4 * 4 + 0] = y.x; qbv[g4 * 4 + 1] = y.y; qbv[g4 * 4 + 2] = y.z; qbv[g4 * 4 + 3] = y.w;
                    }
#pragma unroll
                    for (int g = 0; g < G; ++g) acc[g] = fmaf(qbv[g], kb, fmaf(qa[g], ka, acc[g]));
                }
            }
            tc_fence_before_sync();
            mbar_arrive(&sm.acc_empty[buf]);
            const int n = n0 + t;
            if (n < p.n_pad) {
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const int h = (un.hp * 2 + grp) * G + g;
                    p.scores[((long long)un.s * p.H_q + h) * p.n_pad + n] = acc[g];
                }
            }
            ++uc;
        }
        if (!ok && lane == 0) {
            lorc_set_status(p.status, LORC_ERR_TIMEOUT);
            sm.abort_flag = 1;
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------------------------
// PV kernel
// ------------------------------------------------------------------------------------------------
constexpr int V_STAGES = 4;
constexpr int V_THREADS = 192;       // warp 0 TMA, warp 1 MMA, warps 2..5 softmax
constexpr int V_SOFT = 128;

template <int HQ>
struct PvSmem {
    bf16 V[V_STAGES][2][TILE * KC];       // C_V slice: two 64-column blocks of [128 tokens][64]   32 KiB/stage
    bf16 P[2][2][HQ * KC];                // probabilities [HQ heads][128 tokens] as two 64-token chunks
    float red[4][HQ];
    float m_s[HQ];
    uint64_t full[V_STAGES], empty[V_STAGES], p_full[2], p_empty[2], o_full;
    uint32_t tmem_base;
    int abort_flag;
};

struct PvParams {
    const float* scores;           // [b, H_q, n_pad]  (log2 units)
    float* part_ml;                // [b, H_q, S, 2]   (max in natural-log units, sum)
    float* part_o;                 // [b, H_q, S, r_v]
    const int32_t* seq_lens;
    const int32_t* page_table;
    int* status;
    int batch, H_q, r_v, n_pad, n_splits, tiles_per_split, max_pos;
    int page_size, max_pages_per_seq, n_pages;
};

template <int HQ>
__global__ void __launch_bounds__(V_THREADS, 1)
lorc_pv_kernel(const __grid_constant__ CUtensorMap mapCV, const PvParams p) {
    extern __shared__ uint8_t raw[];
    typedef PvSmem<HQ> S;
    S& sm = *reinterpret_cast<S*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int split = blockIdx.x, s = blockIdx.y;
    const int nblk = (p.r_v + 127) / 128;
    constexpr uint32_t TM_COLS = (HQ * 8 <= 256) ? 256 : 512;

    int len = p.seq_lens[s];
    if (len > p.max_pos) {
        if (tid == 0) lorc_set_status(p.status, LORC_ERR_CAPACITY);
        len = 0;
    }
    if (len < 0) len = 0;
    const int t_begin = min(len, split * p.tiles_per_split * TILE);
    const int t_end = min(len, (split + 1) * p.tiles_per_split * TILE);
    const int ntiles = (t_end - t_begin + TILE - 1) / TILE;

    if (tid == 0) {
        for (int i = 0; i < V_STAGES; ++i) {
            mbar_init(&sm.full[i], 1);
            mbar_init(&sm.empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sm.p_full[i], V_SOFT);
            mbar_init(&sm.p_empty[i], 1);
        }
        mbar_init(&sm.o_full, 1);
        sm.abort_flag = 0;
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

    if (warp == 0) {
        if (lane == 0 && ntiles > 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int i = 0; i < ntiles && ok; ++i) {
                const int n0 = t_begin + i * TILE;
                for (int blk = 0; blk < nblk; ++blk, ++it) {
                    const int st = it % V_STAGES;
                    if (!mbar_wait(&sm.empty[st], ((it / V_STAGES) & 1) ^ 1)) { ok = false; break; }
                    if (p.page_table == nullptr) {
                        mbar_arrive_expect_tx(&sm.full[st], 2 * TILE * KC * 2);
                        tma_load_3d(sm.V[st][0], &mapCV, &sm.full[st], blk * 128, n0, s);
                        tma_load_3d(sm.V[st][1], &mapCV, &sm.full[st], blk * 128 + 64, n0, s);
                    } else {
                        const int ppt = TILE / p.page_size;
                        int pages[8];
                        uint32_t bytes = 0;
                        for (int pg = 0; pg < ppt; ++pg) {
                            int lp = n0 / p.page_size + pg;
                            int page = -1;
                            if (lp * p.page_size < len && lp < p.max_pages_per_seq) {
                                page = p.page_table[(long long)s * p.max_pages_per_seq + lp];
                                if (page < 0 || page >= p.n_pages) {
                                    lorc_set_status(p.status, LORC_ERR_CAPACITY);
                                    page = -1;
                                }
                            }
                            pages[pg] = page;
                            if (page >= 0) bytes += 2 * p.page_size * KC * 2;
                        }
                        if (bytes == 0) {
                            mbar_arrive(&sm.full[st]);
                        } else {
                            mbar_arrive_expect_tx(&sm.full[st], bytes);
                            for (int pg = 0; pg < ppt; ++pg)
                                if (pages[pg] >= 0) {
                                    tma_load_3d(sm.V[st][0] + pg * p.page_size * KC, &mapCV, &sm.full[st], blk * 128,
                                                0, pages[pg]);
                                    tma_load_3d(sm.V[st][1] + pg * p.page_size * KC, &mapCV, &sm.full[st],
                                                blk * 128 + 64, 0, pages[pg]);
                                }
                        }
                    }
                }
            }
            if (!ok) {
                lorc_set_status(p.status, LORC_ERR_TIMEOUT);
                sm.abort_flag = 1;
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && ntiles > 0) {
            const uint32_t idesc = make_idesc_bf16(128, HQ, 1, 0);
            uint32_t it = 0;
            bool ok = true;
            for (int i = 0; i < ntiles && ok; ++i) {
                const int buf = i & 1;
                if (!mbar_wait(&sm.p_full[buf], (i >> 1) & 1)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t p0 = smem_u32(sm.P[buf][0]);
                for (int blk = 0; blk < nblk; ++blk, ++it) {
                    const int st = it % V_STAGES;
                    if (!mbar_wait(&sm.full[st], (it / V_STAGES) & 1)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t v0 = smem_u32(sm.V[st][0]);
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        // A: C_V^T block, MN-major: 16 token rows per step, two 64-column blocks 16 KiB apart
                        const uint64_t ad = make_smem_desc_sw128(v0 + k * 2048, TILE * KC * 2, 1024);
                        // B: P [HQ][128 tokens], K-major: 64-token chunks of HQ*128 bytes
                        const uint64_t bd =
                            make_smem_desc_sw128(p0 + (k >> 2) * (HQ * KC * 2) + (k & 3) * 32, 0, 1024);
                        tc_mma_bf16(tmem + blk * HQ, ad, bd, idesc, (i | k) != 0);
                    }
                    tc_commit(&sm.empty[st]);
                }
                if (!ok) break;
                tc_commit(&sm.p_empty[buf]);
            }
            tc_commit(&sm.o_full);
            if (!ok) {
                lorc_set_status(p.status, LORC_ERR_TIMEOUT);
                sm.abort_flag = 1;
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax warps
        const int t = tid - 64;                   // 0..127: token inside the tile, and TMEM lane later
        const int wq = warp - 2;                  // 0..3 == warp % 4 - 2 .. careful below
        float l[HQ];
#pragma unroll
        for (int h = 0; h < HQ; ++h) l[h] = 0.f;
        bool ok = true;
        if (ntiles > 0) {
            // phase A: exact maximum of every head over this split
            {
                float mx[HQ];
#pragma unroll
                for (int h = 0; h < HQ; ++h) mx[h] = -INFINITY;
                // (two tiles per iteration: twice as many independent loads in flight)
                int n = t_begin + t;
                for (; n + TILE < t_end; n += 2 * TILE) {
                    const float* sp = p.scores + (long long)s * p.H_q * p.n_pad + n;
#pragma unroll
                    for (int h = 0; h < HQ; ++h)
                        mx[h] = fmaxf(mx[h], fmaxf(sp[(long long)h * p.n_pad], sp[(long long)h * p.n_pad + TILE]));
                }
                if (n < t_end) {
                    const float* sp = p.scores + (long long)s * p.H_q * p.n_pad + n;
#pragma unroll
                    for (int h = 0; h < HQ; ++h) mx[h] = fmaxf(mx[h], sp[(long long)h * p.n_pad]);
                }
#pragma unroll
                for (int h = 0; h < HQ; ++h) {
                    float v = mx[h];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
                    if (lane == 0) sm.red[wq][h] = v;
                }
                asm volatile("bar.sync 2, 128;" ::: "memory");
                if (t < HQ) sm.m_s[t] = fmaxf(fmaxf(sm.red[0][t], sm.red[1][t]), fmaxf(sm.red[2][t], sm.red[3][t]));
                asm volatile("bar.sync 2, 128;" ::: "memory");
            }
            // phase B: probabilities of each tile into shared memory (bf16, K-major, 128-byte swizzle)
            for (int i = 0; i < ntiles; ++i) {
                const int buf = i & 1;
                if (!mbar_wait(&sm.p_empty[buf], ((i >> 1) & 1) ^ 1)) { ok = false; break; }
                const int n = t_begin + i * TILE + t;
                const bool valid = n < t_end;
                const float* sp = p.scores + (long long)s * p.H_q * p.n_pad + n;
                uint8_t* pb = reinterpret_cast<uint8_t*>(sm.P[buf][t >> 6]);
                const int tc = t & 63;
#pragma unroll
                for (int h = 0; h < HQ; ++h) {
                    float pv = 0.f;
                    if (valid) pv = exp2f(sp[(long long)h * p.n_pad] - sm.m_s[h]);
                    const bf16 pr = __float2bfloat16_rn(pv);
                    l[h] += __bfloat162float(pr);
                    const int off = h * 128 + ((((tc >> 3) ^ (h & 7)) << 4) | ((tc & 7) << 1));
                    *reinterpret_cast<bf16*>(pb + off) = pr;
                }
                fence_proxy_async_smem();
                mbar_arrive(&sm.p_full[buf]);
            }
        }
        // sum of probabilities per head over the CTA
        float lsum = 0.f;
#pragma unroll
        for (int h = 0; h < HQ; ++h) {
            float v = l[h];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == 0) sm.red[wq][h] = v;
        }
        asm volatile("bar.sync 2, 128;" ::: "memory");
        if (t < HQ) {
            lsum = sm.red[0][t] + sm.red[1][t] + sm.red[2][t] + sm.red[3][t];
            const long long unit = ((long long)s * p.H_q + t) * p.n_splits + split;
            p.part_ml[unit * 2 + 0] = (ntiles > 0) ? sm.m_s[t] * LN2 : -INFINITY;
            p.part_ml[unit * 2 + 1] = (ntiles > 0 && ok) ? lsum : 0.f;
        }
        if (ntiles > 0 && ok) {
            if (mbar_wait(&sm.o_full, 0)) {
                tc_fence_after_sync();
                // TMEM lane = latent row inside a 128-row block; this warp may read quarter (warp % 4)
                const int quarter = warp % 4;
                const int row = quarter * 32 + lane;
                for (int blk = 0; blk < nblk; ++blk) {
                    const int rr = blk * 128 + row;
#pragma unroll
                    for (int c0 = 0; c0 < HQ; c0 += 32) {
                        uint32_t r[32];
                        tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + blk * HQ + c0, r);
                        tmem_wait_ld();
                        if (rr < p.r_v) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                const long long unit = ((long long)s * p.H_q + c0 + i) * p.n_splits + split;
                                p.part_o[unit * p.r_v + rr] = __uint_as_float(r[i]);
                            }
                        }
                    }
                }
            } else {
                ok = false;
            }
        }
        if (!ok && lane == 0) {
            lorc_set_status(p.status, LORC_ERR_TIMEOUT);
            sm.abort_flag = 1;
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, TM_COLS);
}

// constant table (cos, sin)(t * theta_j) laid out [j][t], t < 128
__global__ void rope_tile_kernel(float2* out, double theta) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 64 * TILE) return;
    int j = i / TILE, t = i % TILE;
    double inv = pow(theta, -(double)j / 64.0);
    double sn, cs;
    sincos((double)t * inv, &sn, &cs);
    out[i] = make_float2((float)cs, (float)sn);
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
struct LorcTcLayer {
    bool has_bkt = false;
    CUtensorMap mapBKT, mapBV;          // B_K^T in 64 x 256 swizzled boxes; B_V in plain 64-row x 128-column boxes
    // cache maps are rebuilt only when the cache geometry or pointers change
    const void* k_ptr = nullptr;
    const void* v_ptr = nullptr;
    long long key_dims[6] = {0, 0, 0, 0, 0, 0};
    CUtensorMap mapCK, mapCV;
};

struct LorcTcState {
    float2* rope_tile = nullptr;
    std::vector<LorcTcLayer> layers;
    bool attrs_set = false;
};

static LorcTcState* tc_state(lorc_ctx* ctx) {
    if (!ctx->tc) {
        ctx->tc = new LorcTcState();
        ctx->tc->layers.resize(ctx->desc.n_layers);
    }
    return ctx->tc;
}

void lorc_tc_release(lorc_ctx* ctx) {
    if (ctx->tc) {
        cudaFree(ctx->tc->rope_tile);
        delete ctx->tc;
        ctx->tc = nullptr;
    }
}

void lorc_tc_invalidate_layer(lorc_ctx* ctx, int layer) {
    if (ctx->tc && layer >= 0 && layer < (int)ctx->tc->layers.size()) ctx->tc->layers[layer] = LorcTcLayer();
}

static bool tc_shape_ok(const lorc_ctx* ctx) {
    const lorc_model_desc& d = ctx->desc;
    return d.d_head == 128 && d.rope_style == LORC_ROPE_HALF_SPLIT && (d.n_kv_heads % 2) == 0 &&
           (ctx->group == 4 || ctx->group == 8) && (d.n_q_heads == 32 || d.n_q_heads == 64);
}

bool lorc_tc_decode_supported(const lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv) {
    if (!tc_shape_ok(ctx) || L.mode != LORC_MODE_LATENT) return false;
    if (cv.page_table) {
        int ps = cv.page_size;
        if (!(ps == 16 || ps == 32 || ps == 64 || ps == 128)) return false;
    }
    if (L.r_k % 8 || L.r_v % 8) return false;
    return lorc_get_tmap_encode() != nullptr;
}

static int tc_tiles_per_split(int max_seq_len, int n_splits_hint) {
    int tiles = (max_seq_len + TILE - 1) / TILE;
    if (n_splits_hint > 0) {
        int S = n_splits_hint < tiles ? n_splits_hint : tiles;
        return (tiles + S - 1) / S;
    }
    return tiles < 4 ? tiles : 4;
}

static size_t tc_scores_bytes(const lorc_ctx* ctx, int batch, int max_seq_len) {
    size_t n_pad = (size_t)((max_seq_len + TILE - 1) / TILE) * TILE;
    return lorc_align_up((size_t)batch * ctx->desc.n_q_heads * n_pad * sizeof(float), 256);
}

size_t lorc_tc_workspace_bytes(const lorc_ctx* ctx, int batch, int max_seq_len) {
    if (!tc_shape_ok(ctx)) return 0;
    // worst case over split hints: one tile per split
    int tiles = (max_seq_len + TILE - 1) / TILE;
    int S = (tiles + 3) / 4;
    size_t units = (size_t)batch * ctx->desc.n_q_heads * S;
    return tc_scores_bytes(ctx, batch, max_seq_len) + lorc_align_up(units * 2 * sizeof(float), 256) +
           lorc_align_up(units * (size_t)ctx->n * sizeof(float), 256);
}

static bool build_cache_maps(LorcTcLayer& T, const LorcLayer& L, const CacheView& cv) {
    long long key[6] = {cv.page_table ? 1 : 0, cv.seq_stride, cv.batch, cv.page_size, cv.n_pages, L.r_k * 4096LL + L.r_v};
    bool same = T.k_ptr == cv.k && T.v_ptr == cv.v;
    for (int i = 0; i < 6; ++i) same = same && key[i] == T.key_dims[i];
    if (same) return true;
    uint64_t dims[3], str[2];
    uint32_t box[3];
    for (int which = 0; which < 2; ++which) {
        const int r = which ? L.r_v : L.r_k;
        const void* base = which ? (const void*)cv.v : (const void*)cv.k;
        if (cv.page_table == nullptr) {
            dims[0] = r; dims[1] = (uint64_t)cv.seq_stride; dims[2] = cv.batch;
            str[0] = (uint64_t)r * 2; str[1] = (uint64_t)cv.seq_stride * r * 2;
            box[0] = KC; box[1] = TILE; box[2] = 1;
        } else {
            dims[0] = r; dims[1] = cv.page_size; dims[2] = cv.n_pages;
            str[0] = (uint64_t)r * 2; str[1] = (uint64_t)cv.page_size * r * 2;
            box[0] = KC; box[1] = cv.page_size; box[2] = 1;
        }
        if (!lorc_make_tmap_bf16(which ? &T.mapCV : &T.mapCK, base, 3, dims, str, box)) return false;
    }
    T.k_ptr = cv.k;
    T.v_ptr = cv.v;
    for (int i = 0; i < 6; ++i) T.key_dims[i] = key[i];
    return true;
}

cudaError_t lorc_tc_decode(lorc_ctx* ctx, int layer, const LorcLayer& L, const CacheView& cv, const bf16* q,
                           bf16* out, int n_splits, void* ws, size_t ws_bytes, cudaStream_t st, int* launches) {
    LorcTcState* T = tc_state(ctx);
    LorcTcLayer& TL = T->layers[layer];
    const lorc_model_desc& d = ctx->desc;
    if (!T->rope_tile) {
        cudaError_t e = cudaMalloc(&T->rope_tile, sizeof(float2) * 64 * TILE);
        if (e != cudaSuccess) return e;
        rope_tile_kernel<<<(64 * TILE + 255) / 256, 256, 0, st>>>(T->rope_tile, d.rope_theta);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    if (!T->attrs_set) {
        cudaError_t e;
        e = cudaFuncSetAttribute(lorc_score_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ScoreSmem) + 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(lorc_score_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ScoreSmem) + 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(lorc_pv_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(PvSmem<32>) + 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(lorc_pv_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(PvSmem<64>) + 1024);
        if (e != cudaSuccess) return e;
        T->attrs_set = true;
    }
    if (!TL.has_bkt) {
        uint64_t dims[2] = {(uint64_t)L.r_k, (uint64_t)ctx->n}, str[1] = {(uint64_t)L.r_k * 2};
        uint32_t box[2] = {KC, 256};
        if (!lorc_make_tmap_bf16(&TL.mapBKT, L.B_kT, 2, dims, str, box)) return cudaErrorInvalidValue;
        uint64_t d2[2] = {(uint64_t)ctx->n, (uint64_t)L.r_v}, s2[1] = {(uint64_t)ctx->n * 2};
        uint32_t b2[2] = {128, 64};
        if (!lorc_make_tmap_bf16(&TL.mapBV, L.B_v, 2, d2, s2, b2, false)) return cudaErrorInvalidValue;
        TL.has_bkt = true;
    }
    if (!build_cache_maps(TL, L, cv)) return cudaErrorInvalidValue;

    const int tiles = (cv.max_seq_len + TILE - 1) / TILE;
    const int n_pad = tiles * TILE;
    int tps = tc_tiles_per_split(cv.max_seq_len, n_splits);
    const size_t sc_bytes = tc_scores_bytes(ctx, cv.batch, cv.max_seq_len);
    int S;
    size_t units, ml_bytes, o_bytes;
    // fewer, longer splits until the partial results fit the workspace and the merge kernel's limit
    for (;; ++tps) {
        S = (tiles + tps - 1) / tps;
        units = (size_t)cv.batch * d.n_q_heads * S;
        ml_bytes = lorc_align_up(units * 2 * sizeof(float), 256);
        o_bytes = lorc_align_up(units * (size_t)L.r_v * sizeof(float), 256);
        if (S <= LORC_MAX_SPLITS && sc_bytes + ml_bytes + o_bytes <= ws_bytes) break;
        if (S == 1) return cudaErrorMemoryAllocation;
    }
    float* scores = (float*)ws;
    float* part_ml = (float*)((char*)ws + sc_bytes);
    float* part_o = (float*)((char*)ws + sc_bytes + ml_bytes);

    ScoreParams sp;
    sp.q = q; sp.scores = scores; sp.seq_lens = cv.seq_lens; sp.page_table = cv.page_table;
    sp.rope_table = ctx->rope_table; sp.rope_tile = T->rope_tile; sp.status = ctx->status_dev;
    sp.batch = cv.batch; sp.H_q = d.n_q_heads; sp.n_hp = d.n_kv_heads / 2; sp.r_k = L.r_k; sp.n_pad = n_pad;
    sp.tiles_per_seq = tiles; sp.max_pos = d.max_pos;
    sp.page_size = cv.page_size; sp.max_pages_per_seq = cv.max_pages_per_seq; sp.n_pages = cv.n_pages;
    const int total_units = cv.batch * tiles * sp.n_hp;
    int grid1 = total_units < ctx->sm_count ? total_units : ctx->sm_count;
    const size_t smem1 = sizeof(ScoreSmem) + 1024;
    {
        LorcStageTimer timer(ctx, LORC_STAGE_SCORE, st);
        if (ctx->group == 4)
            lorc_score_kernel<4><<<grid1, S_THREADS, smem1, st>>>(TL.mapCK, TL.mapBKT, sp);
        else
            lorc_score_kernel<8><<<grid1, S_THREADS, smem1, st>>>(TL.mapCK, TL.mapBKT, sp);
    }
    *launches += 1;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;

    PvParams pp;
    pp.scores = scores; pp.part_ml = part_ml; pp.part_o = part_o; pp.seq_lens = cv.seq_lens;
    pp.page_table = cv.page_table; pp.status = ctx->status_dev;
    pp.batch = cv.batch; pp.H_q = d.n_q_heads; pp.r_v = L.r_v; pp.n_pad = n_pad; pp.n_splits = S;
    pp.tiles_per_split = tps; pp.max_pos = d.max_pos;
    pp.page_size = cv.page_size; pp.max_pages_per_seq = cv.max_pages_per_seq; pp.n_pages = cv.n_pages;
    dim3 grid2(S, cv.batch);
    {
        LorcStageTimer timer(ctx, LORC_STAGE_PV, st);
        if (d.n_q_heads == 32)
            lorc_pv_kernel<32><<<grid2, V_THREADS, sizeof(PvSmem<32>) + 1024, st>>>(TL.mapCV, pp);
        else
            lorc_pv_kernel<64><<<grid2, V_THREADS, sizeof(PvSmem<64>) + 1024, st>>>(TL.mapCV, pp);
    }
    *launches += 1;
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return lorc_fast_combine(ctx, L, &TL.mapBV, cv.batch, S, part_ml, part_o, out, st, launches);
}
