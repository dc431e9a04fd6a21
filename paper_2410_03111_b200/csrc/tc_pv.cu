// Softmax, P.C_V split by LATENT COLUMNS, and the value up-projection; the two contractions run on the tensor cores.
//
// Probability kernel.  One CTA per (sequence, group of 128-token tiles): reads the exact row maximum of every head
// over the whole sequence (one word per head, raised by the score kernel with atomic maxima), turns the scores of its
// tiles into p = 2^(s - m) rounded to bf16 -- stored tile by tile as the 128-byte-swizzled K-major image the PV
// kernel's MMA reads, so that kernel fetches a tile with one bulk copy -- and writes its share of the softmax
// denominator.  The probabilities are computed once, not once per column block.
//
// PV kernel.  A CTA owns one 128-column block of C_V (rho in [128 blk, 128 blk + 128)) of one sequence and one share
// of its context.  A block of latent columns is disjoint from every other block, so the CTA's accumulator
// O_lat^T[128 rho, H_q] (fp32 in TMEM) needs no merge with other column blocks; and every tile uses the same exact
// row maximum, so the context shares of a block simply add.  Per tile of 128 tokens
//       O_lat^T += C_V[tile, block]^T . P^T                    tcgen05, MN-major A
// and at the end the CTA writes its 128 x H_q piece of the un-normalised latent output.
//
// Up-projection.  A small kernel adds the context shares, divides by the denominator and rounds to bf16; then one
// CTA per (KV head g, 128 output rows = 128 / G sequences) multiplies those rows by B_V[:, g] (TMA-staged from a
// transposed copy): out = o . B_V[:, g] in TMEM, then bf16.
#include <math.h>

#include "sm100_ptx.cuh"
#include "tc_kernels.cuh"

using namespace sm100;

namespace {

constexpr int TILE = 128;
constexpr int KC = 64;
// one CTA per SM; 5 stages x 40 KiB with 32 query heads (200 KiB in flight), 4 x 48 KiB with 64
template <int HQ>
struct PvStages { static constexpr int value = HQ <= 32 ? 5 : 4; };
constexpr int P_THREADS = 192;       // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue

// read-only global load that the compiler keeps in program order with the other volatile asm of this file
__device__ __forceinline__ float ldg_nc_f32(const float* p) {
    float v;
    asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}

// ------------------------------------------------------------------------------------------------
// probability kernel
// ------------------------------------------------------------------------------------------------
struct ProbParams {
    const float* scores;           // [b, H_q, n_pad]      log2 units
    const unsigned* rowmax;        // [b, H_q]   exact row maxima as order-preserving keys (0: no token seen)
    bf16* probs;                   // [b, tiles, 2 chunks of 64 tokens, H_q, 64]   swizzled tile images
    float* l_part;                 // [b, n_groups, H_q]
    int* done;                     // [b, n_blk]  arrival counters of the PV kernel's context shares, zeroed here
    const int32_t* seq_lens;
    int* status;
    int H_q, n_pad, tiles, tiles_per_group, n_groups, n_blk, max_pos;
};

// byte offset of (head h, token tc < 64) inside a 64-token chunk image: rows of 128 bytes, 16-byte pieces XOR-ed with
// the row number (the 128-byte swizzle of the shared-memory matrix descriptors)
__device__ __forceinline__ int prob_image_offset(int h, int tc) {
    return h * 128 + ((((tc >> 3) ^ (h & 7)) << 4) | ((tc & 7) << 1));
}

// 256 threads: thread = (token of the tile, half of the heads).
template <int HQ>
__global__ void __launch_bounds__(256, 3)
lorc_prob_kernel(const ProbParams p) {
    constexpr int NH = HQ / 2;                        // heads per thread
    __shared__ float m_s[HQ];
    __shared__ float red[8][HQ];
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int t = tid & 127, hh = tid >> 7, h0 = hh * NH;
    const int grp = blockIdx.x, s = blockIdx.y;
    grid_dep_wait();                                 // the scores come from the kernel before this one
    grid_dep_launch();
    int len = p.seq_lens[s];
    if (len > p.max_pos || len < 0) len = 0;        // the score kernel reports the capacity error
    const int tiles_s = (len + TILE - 1) / TILE;
    const int tile_lo = min(tiles_s, grp * p.tiles_per_group), tile_hi = min(tiles_s, tile_lo + p.tiles_per_group);
    if (grp == 0 && tid < p.n_blk) p.done[s * p.n_blk + tid] = 0;
    float l[NH];
#pragma unroll
    for (int i = 0; i < NH; ++i) l[i] = 0.f;
    if (tile_lo < tile_hi) {
        // the scores of the first tile are requested before the maxima, so the two round trips overlap
        float sv[NH];
        const float* sbase = p.scores + ((long long)s * p.H_q + h0) * p.n_pad + t;
        {
            const int n = tile_lo * TILE + t;
#pragma unroll
            for (int i = 0; i < NH; ++i) sv[i] = n < len ? ldg_nc_f32(sbase + (long long)i * p.n_pad + tile_lo * TILE) : 0.f;
        }
        // exact maximum of every head over the WHOLE sequence
        if (tid < HQ) {
            const unsigned key = p.rowmax[(long long)s * p.H_q + tid];
            m_s[tid] = key ? lorc_key_float(key) : 0.f;
        }
        __syncthreads();
        for (int tile = tile_lo; tile < tile_hi; ++tile) {
            const bool valid = tile * TILE + t < len;
            uint8_t* img = reinterpret_cast<uint8_t*>(p.probs) +
                           (((long long)s * p.tiles + tile) * 2 + (t >> 6)) * (HQ * KC * 2);
            const int tc = t & 63;
            float ssum = 0.f;
            bf16 pr[NH];
#pragma unroll
            for (int i = 0; i < NH; ++i) {
                ssum += sv[i];
                // p = 2^(s - m), rounded to bf16 (the same rounded value enters the denominator)
                pr[i] = __float2bfloat16_rn(valid ? exp2f(sv[i] - m_s[h0 + i]) : 0.f);
                l[i] += __bfloat162float(pr[i]);
            }
            // a NaN among the scores means non-finite numbers in the cache, the factors or the query
            if (ssum != ssum) lorc_set_status(p.status, LORC_ERR_ARG);
            if (tile + 1 < tile_hi) {
                const int n = (tile + 1) * TILE + t;
#pragma unroll
                for (int i = 0; i < NH; ++i)
                    sv[i] = n < len ? ldg_nc_f32(sbase + (long long)i * p.n_pad + (tile + 1) * TILE) : 0.f;
            }
#pragma unroll
            for (int i = 0; i < NH; ++i) *reinterpret_cast<bf16*>(img + prob_image_offset(h0 + i, tc)) = pr[i];
        }
    }
    // This group's share of the softmax denominator (zero for a group past the end of the sequence).  A warp holds
    // 32 tokens x NH heads; each exchange step halves the heads a lane carries, so NH - 1 (+1) shuffles add them all.
    __syncthreads();
    {
        int n = NH;
#pragma unroll
        for (int step = 16; step >= 1; step >>= 1) {
            if (n > 1) {
                const bool upper = (lane & step) != 0;
#pragma unroll
                for (int i = 0; i < NH / 2; ++i) {
                    if (i < n / 2) {
                        const float keep = upper ? l[i + n / 2] : l[i];
                        const float send = upper ? l[i] : l[i + n / 2];
                        l[i] = keep + __shfl_xor_sync(0xffffffffu, send, step);
                    }
                }
                n >>= 1;
            } else {
                l[0] += __shfl_xor_sync(0xffffffffu, l[0], step);
            }
        }
        // the lane now holds head (lane * NH / 32) of its half
        if ((lane & (32 / NH - 1)) == 0) red[warp & 3][h0 + lane * NH / 32] = l[0];
    }
    __syncthreads();
    if (tid < HQ) p.l_part[((long long)s * p.n_groups + grp) * p.H_q + tid] = red[0][tid] + red[1][tid] + red[2][tid] + red[3][tid];
}

// ------------------------------------------------------------------------------------------------
// PV kernel
// ------------------------------------------------------------------------------------------------
template <int HQ>
struct Pv2Smem {
    static constexpr int P_STAGES = PvStages<HQ>::value;
    bf16 V[P_STAGES][2][TILE * KC];       // C_V block: two 64-column halves of [128 tokens][64]; 32 KiB / stage
    bf16 P[P_STAGES][2][HQ * KC];         // probabilities [HQ][128 tokens] as two 64-token chunks, 128-byte swizzle
    float red[128 / HQ][HQ];
    float l_inv[HQ];
    uint64_t full[P_STAGES], empty[P_STAGES], o_full, red_full;
    uint32_t tmem_base;
    int last;
};

struct Pv2Params {
    const bf16* probs;             // [b, tiles, 2, H_q, 64]   swizzled tile images
    float* o_part;                 // [b, n_blk, n_csplit, H_q, 128]   un-normalised latent output of every context share
    const float* l_part;           // [b, n_groups, H_q]   shares of the softmax denominator
    unsigned* rowmax;              // [b, H_q]   row maxima of the softmax: zeroed here for the next call
    bf16* o_norm;                  // [b, H_q, r_pad]      normalised latent output
    int* done;                     // [b, n_blk]           context shares of a column block that have finished
    const int32_t* seq_lens;
    const int32_t* page_table;
    int* status;
    int batch, H_q, n_kv, r_v, tiles, n_blk, n_csplit, n_groups, max_pos;
    int page_size, max_pages_per_seq, n_pages;
};

template <int HQ>
__global__ void __launch_bounds__(P_THREADS, 1)
lorc_pv2_kernel(const __grid_constant__ CUtensorMap mapCV, const Pv2Params p) {
    extern __shared__ uint8_t raw[];
    typedef Pv2Smem<HQ> S;
    constexpr int P_STAGES = PvStages<HQ>::value;
    S& sm = *reinterpret_cast<S*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    constexpr uint32_t TM_COLS = HQ <= 32 ? 32 : 64;
    constexpr uint32_t P_BYTES = 2 * HQ * KC * 2;
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
    const int rho0 = blk * 128;

    if (tid == 0) {
        for (int i = 0; i < P_STAGES; ++i) {
            mbar_init(&sm.full[i], 1);
            mbar_init(&sm.empty[i], 1);
        }
        mbar_init(&sm.o_full, 1);
        mbar_init(&sm.red_full, 1);
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
        // The whole warp walks the loop and one elected lane issues: the asynchronous instructions take their
        // operands from uniform registers, which the compiler only uses in warp-uniform code.
        // The kernel before this one only writes the probabilities and denominators; the latent values were complete
        // before IT could start.  So the first stages' C_V boxes are requested right away, and only the probability
        // tiles wait for that kernel to finish.
        {
            for (int i = 0; i < ntiles && ok; ++i) {
                const int tile = tile_lo + i;
                const int n0 = tile * TILE;
                const int st = i % P_STAGES;
                if (i == P_STAGES) {
                    // probability tiles of the stages whose C_V boxes went out before the wait
                    grid_dep_wait();
                    if (elect_one()) {
                        for (int j = 0; j < P_STAGES; ++j)
                            bulk_load(sm.P[j][0], p.probs + ((long long)s * p.tiles + tile_lo + j) * (2 * HQ * KC), P_BYTES,
                                      &sm.full[j]);
                    }
                    __syncwarp();
                }
                if (!mbar_wait(&sm.empty[st], ((i / P_STAGES) & 1) ^ 1)) { ok = false; break; }
                if (elect_one()) {
                mbar_arrive_expect_tx(&sm.full[st], 2 * TILE * KC * 2 + P_BYTES);
                if (i >= P_STAGES)
                    bulk_load(sm.P[st][0], p.probs + ((long long)s * p.tiles + tile) * (2 * HQ * KC), P_BYTES, &sm.full[st]);
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
                __syncwarp();
            }
            if (ntiles <= P_STAGES) {
                grid_dep_wait();
                if (elect_one()) {
                    for (int j = 0; j < ntiles; ++j)
                        bulk_load(sm.P[j][0], p.probs + ((long long)s * p.tiles + tile_lo + j) * (2 * HQ * KC), P_BYTES,
                                  &sm.full[j]);
                }
                __syncwarp();
            }
            if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (warp-uniform, elected lane)
        if (ntiles > 0) {
            const uint32_t idesc = make_idesc_bf16(128, HQ, 1, 0);
            for (int i = 0; i < ntiles && ok; ++i) {
                const int st = i % P_STAGES;
                if (!mbar_wait(&sm.full[st], (i / P_STAGES) & 1)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t p0 = smem_u32(sm.P[st][0]), v0 = smem_u32(sm.V[st][0]);
                if (elect_one()) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        // A: C_V^T block (MN-major): 16 token rows per step, the two 64-column halves 16 KiB apart
                        const uint64_t ad = make_smem_desc_sw128(v0 + k * 2048, TILE * KC * 2, 1024);
                        // B: P [HQ][128 tokens] (K-major), 64-token chunks of HQ*128 bytes
                        const uint64_t bd = make_smem_desc_sw128(p0 + (k >> 2) * (HQ * KC * 2) + (k & 3) * 32, 0, 1024);
                        tc_mma_bf16(tmem, ad, bd, idesc, (i | k) != 0);
                    }
                    tc_commit(&sm.empty[st]);
                }
                __syncwarp();
            }
            if (elect_one()) tc_commit(&sm.o_full);
            __syncwarp();
            if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int t = tid - 64;
        const int quarter = warp % 4;
        const int row = quarter * 32 + lane;              // TMEM lane = latent row of the block
        const int r_pad = p.n_blk * 128;
        grid_dep_wait();                              // denominators come from the kernel before this one
        grid_dep_launch();
        // the probability kernel has read the row maxima: leave them empty for the next call's score kernel
        if (blk == 0 && cs == 0 && t < HQ) p.rowmax[(long long)s * p.H_q + t] = 0u;
        // while the tiles stream: the reciprocal softmax denominator of every head (all shares of the sequence)
        {
            constexpr int PARTS = 128 / HQ;
            const int h = t % HQ, part = t / HQ;
            const float* lp = p.l_part + (long long)s * p.n_groups * p.H_q + h;
            float L = 0.f;
            for (int g = part; g < p.n_groups; g += PARTS) L += __ldg(lp + (long long)g * p.H_q);
            sm.red[part][h] = L;
            __syncwarp();   // a named barrier counts a warp once only if the warp arrives converged
            asm volatile("bar.sync 2, 128;" ::: "memory");
            if (t < HQ) {
                float Ls = 0.f;
#pragma unroll
                for (int i = 0; i < PARTS; ++i) Ls += sm.red[i][t];
                sm.l_inv[t] = Ls > 0.f ? 1.f / Ls : 0.f;
                if (!(Ls > 0.f) && blk == 0 && cs == 0) lorc_set_status(p.status, LORC_ERR_EMPTY);
            }
        }
        if (ntiles > 0) {
            if (!mbar_wait(&sm.o_full, 0)) ok = false;
        }
        float acc[HQ];
        if (ntiles > 0 && ok) {
            tc_fence_after_sync();
#pragma unroll
            for (int c0 = 0; c0 < HQ; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + c0, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) acc[c0 + i] = __uint_as_float(r[i]);
            }
        } else {
#pragma unroll
            for (int h = 0; h < HQ; ++h) acc[h] = 0.f;
        }
        bool finish = true;
        if (p.n_csplit > 1) {
            // publish this share (a contiguous [H_q][128] block); the share that arrives last adds them all up (in
            // share order, so the result does not depend on which one that is)
            constexpr int SHARE_FLOATS = HQ * 128;
            float* blk_base = p.o_part + ((long long)s * p.n_blk + blk) * p.n_csplit * SHARE_FLOATS;
            float* op = blk_base + (long long)cs * SHARE_FLOATS + row;
#pragma unroll
            for (int h = 0; h < HQ; ++h) op[h * 128] = acc[h];
            __threadfence();
            __syncwarp();   // a named barrier counts a warp once only if the warp arrives converged
            asm volatile("bar.sync 2, 128;" ::: "memory");
            if (t == 0) sm.last = atomicAdd(p.done + s * p.n_blk + blk, 1) == p.n_csplit - 1;
            __syncwarp();   // a named barrier counts a warp once only if the warp arrives converged
            asm volatile("bar.sync 2, 128;" ::: "memory");
            finish = sm.last != 0;
            if (finish) {
                __threadfence();
                // The shares come in by bulk copy, a batch at a time, into the C_V stages (every MMA that read them has
                // completed: o_full): one round trip per batch instead of one per share.
                constexpr int PER = (P_STAGES * 2 * TILE * KC * 2) / (SHARE_FLOATS * 4);
                float* stage = reinterpret_cast<float*>(&sm.V[0][0][0]);
#pragma unroll
                for (int h = 0; h < HQ; ++h) acc[h] = 0.f;
                uint32_t par = 0;
                for (int c0 = 0; c0 < p.n_csplit && ok; c0 += PER) {
                    const int nb = min(PER, p.n_csplit - c0);
                    if (c0 > 0) {
                        __syncwarp();
                        asm volatile("bar.sync 2, 128;" ::: "memory");   // everyone has added the previous batch
                    }
                    if (t == 0) {
                        fence_proxy_async_all();     // the other shares' stores (seen through the counter) before the copies
                        mbar_arrive_expect_tx(&sm.red_full, (uint32_t)(nb * SHARE_FLOATS * 4));
                        for (int j = 0; j < nb; ++j)
                            bulk_load(stage + j * SHARE_FLOATS, blk_base + (long long)(c0 + j) * SHARE_FLOATS,
                                      SHARE_FLOATS * 4, &sm.red_full);
                    }
                    if (!mbar_wait(&sm.red_full, par)) { ok = false; break; }
                    par ^= 1;
                    for (int j = 0; j < nb; ++j) {
#pragma unroll
                        for (int h = 0; h < HQ; ++h) acc[h] += stage[(j * HQ + h) * 128 + row];
                    }
                }
            }
        } else {
            __syncwarp();   // a named barrier counts a warp once only if the warp arrives converged
            asm volatile("bar.sync 2, 128;" ::: "memory");     // l_inv is complete
        }
        if (finish) {
            bf16* on = p.o_norm + (long long)s * p.H_q * r_pad + rho0 + row;
#pragma unroll
            for (int h = 0; h < HQ; ++h) on[(long long)h * r_pad] = __float2bfloat16_rn(acc[h] * sm.l_inv[h]);
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
// value up-projection: out[(s, h), :] = o_norm[s, h, :] . B_V[:, g(h)], a plain TMA-fed tcgen05 GEMM.
// grid (n_kv_heads, ceil(batch * G / 128), 4): 128 output rows (s, i) x 32 of the head's 128 columns, K = r_v in
// slices of 64.  (Splitting the columns gives four times the CTAs and small stages, so a whole rank is in flight.)
// ------------------------------------------------------------------------------------------------
constexpr int U_STAGES = 10;         // 10 x 20 KiB: most ranks fit in one round of loads
constexpr int U_THREADS = 192;
constexpr int U_NCOL = 32;           // output columns per CTA (a quarter of a head)

struct UpSmem {
    bf16 A[U_STAGES][128 * KC];           // o_norm rows [128 rows (s, i)][64 rho]
    bf16 B[U_STAGES][U_NCOL * KC];        // B_V^T slice [32 columns j][64 rho]
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
    const int g = blockIdx.x, chunk = blockIdx.y, cq = blockIdx.z;     // KV head, block of 128 rows, column quarter
    const int nkc = (p.r_v + KC - 1) / KC;
    const int seqs_per_cta = 128 / p.G;
    constexpr uint32_t STAGE_BYTES = (128 + U_NCOL) * KC * 2;
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
        tmem_alloc(&sm.tmem_base, 32);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    bool ok = true;

    if (warp == 0) {
        // (warp-uniform loops, one elected lane issues)
        // The factor slices of the first stages do not depend on the kernel before this one: they are requested
        // before the wait, the latent rows after it.
        const int npre = nkc < U_STAGES ? nkc : U_STAGES;
        if (elect_one()) {
            for (int kc = 0; kc < npre; ++kc) {
                mbar_arrive_expect_tx(&sm.full[kc], STAGE_BYTES);
                tma_load_2d(sm.B[kc], &mapBVT, &sm.full[kc], kc * KC, g * 128 + cq * U_NCOL);
            }
        }
        __syncwarp();
        grid_dep_wait();                             // the normalised latent rows come from the kernel before
        grid_dep_launch();
        for (int kc = 0; kc < nkc; ++kc) {
            const int st = kc % U_STAGES;
            if (kc >= npre && !mbar_wait(&sm.empty[st], ((kc / U_STAGES) & 1) ^ 1)) { ok = false; break; }
            if (elect_one()) {
                if (kc >= npre) {
                    mbar_arrive_expect_tx(&sm.full[st], STAGE_BYTES);
                    tma_load_2d(sm.B[st], &mapBVT, &sm.full[st], kc * KC, g * 128 + cq * U_NCOL);
                }
                // rows (s, i): box of G heads x 128/G sequences (sequences past the batch read as zero)
                tma_load_3d(sm.A[st], &mapON, &sm.full[st], kc * KC, g * p.G, chunk * seqs_per_cta);
            }
            __syncwarp();
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    } else if (warp == 1) {
        const uint32_t idesc = make_idesc_bf16(128, U_NCOL, 0, 0);
        for (int kc = 0; kc < nkc; ++kc) {
            const int st = kc % U_STAGES;
            if (!mbar_wait(&sm.full[st], (kc / U_STAGES) & 1)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t a0 = smem_u32(sm.A[st]), b0 = smem_u32(sm.B[st]);
            if (elect_one()) {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    tc_mma_bf16(tmem, make_smem_desc_sw128(a0 + k * 32, 0, 1024), make_smem_desc_sw128(b0 + k * 32, 0, 1024),
                                idesc, (kc | k) != 0);
                tc_commit(&sm.empty[st]);
            }
            __syncwarp();
        }
        if (elect_one()) tc_commit(&sm.d_full);
        __syncwarp();
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    } else {
        grid_dep_wait();
        if (!mbar_wait(&sm.d_full, 0)) ok = false;
        if (ok) {
            tc_fence_after_sync();
            // TMEM lane = output row (s_local * G + i); the warp's lane quarter decides which rows it reads
            const int quarter = warp % 4;
            const int row = quarter * 32 + lane;
            const int s = chunk * seqs_per_cta + row / p.G, h = g * p.G + row % p.G;
            {
                uint32_t r[32];
                tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16), r);
                tmem_wait_ld();
                if (s < p.batch) {
                    uint4* dst = reinterpret_cast<uint4*>(p.out + ((long long)s * p.H_q + h) * 128 + cq * U_NCOL);
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
    if (warp == 1) tmem_dealloc(tmem, 32);
}

// Column blocks and context shares of one PV launch: one CTA per SM, and as few context shares as fill the SMs once
// (a CTA with four stages in flight pulls its share of the HBM bandwidth alone; fewer shares mean longer streams per
// CTA and, at one share, no share reduction at all).
void pv_plan(const lorc_ctx* ctx, const LorcLayer& L, int batch, int max_seq_len, int n_splits_hint, int* n_blk,
             int* n_csplit) {
    const int tiles = (max_seq_len + TILE - 1) / TILE;
    *n_blk = (L.r_v + 127) / 128;
    const int slots = ctx->sm_count;
    int cs = n_splits_hint > 0 ? n_splits_hint : slots / (batch * *n_blk);
    if (cs > tiles) cs = tiles;
    if (cs > 64) cs = 64;
    if (cs < 1) cs = 1;
    *n_csplit = cs;
}

// Tiles per CTA of the probability kernel: about four CTAs per SM over the whole batch (every CTA first reduces the
// row maxima of its sequence, so very many tiny CTAs would repeat that too often).
void prob_plan(const lorc_ctx* ctx, int batch, int tiles, int* tiles_per_group, int* n_groups) {
    int tpg = (int)(((long long)tiles * batch + 4LL * ctx->sm_count - 1) / (4LL * ctx->sm_count));
    if (tpg < 1) tpg = 1;
    *tiles_per_group = tpg;
    *n_groups = (tiles + tpg - 1) / tpg;
}

struct PvScratch {
    size_t part_bytes, l_bytes, on_bytes, prob_bytes, done_bytes;
};

PvScratch pv_scratch_layout(const lorc_ctx* ctx, int batch, int tiles, int n_csplit, int n_groups, size_t r_pad) {
    PvScratch z;
    const size_t hq = (size_t)ctx->desc.n_q_heads;
    z.part_bytes = lorc_align_up((size_t)batch * n_csplit * hq * r_pad * sizeof(float), 256);   // [b][n_blk][n_csplit][H_q][128]
    z.l_bytes = lorc_align_up((size_t)batch * n_groups * hq * sizeof(float), 256);
    z.on_bytes = lorc_align_up((size_t)batch * hq * r_pad * sizeof(bf16), 256);
    z.prob_bytes = lorc_align_up((size_t)batch * tiles * hq * TILE * sizeof(bf16), 256);
    z.done_bytes = lorc_align_up((size_t)batch * (r_pad / 128) * sizeof(int), 256);
    return z;
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
    int tpg, n_groups;
    prob_plan(ctx, batch, tiles, &tpg, &n_groups);
    const size_t r_pad = (size_t)((ctx->n + 127) / 128) * 128;
    const PvScratch z = pv_scratch_layout(ctx, batch, tiles, cs, n_groups, r_pad);
    return z.part_bytes + z.l_bytes + z.on_bytes + z.prob_bytes + z.done_bytes;
}

cudaError_t lorc_tc_pv_launch(lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, const CUtensorMap& mapCV,
                              const CUtensorMap& mapBVT, const float* scores, unsigned* rowmax, int n_pad, int tiles,
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
    int n_blk, n_csplit, tpg, n_groups;
    pv_plan(ctx, L, cv.batch, cv.max_seq_len, n_splits_hint, &n_blk, &n_csplit);
    prob_plan(ctx, cv.batch, tiles, &tpg, &n_groups);
    const int r_pad = n_blk * 128;
    PvScratch z;
    for (;; --n_csplit) {
        z = pv_scratch_layout(ctx, cv.batch, tiles, n_csplit, n_groups, (size_t)r_pad);
        if (z.part_bytes + z.l_bytes + z.on_bytes + z.prob_bytes + z.done_bytes <= scratch_bytes) break;
        if (n_csplit == 1) return cudaErrorMemoryAllocation;
    }
    float* o_part = (float*)scratch;
    float* l_part = (float*)((char*)scratch + z.part_bytes);
    bf16* o_norm = (bf16*)((char*)scratch + z.part_bytes + z.l_bytes);
    bf16* probs = (bf16*)((char*)scratch + z.part_bytes + z.l_bytes + z.on_bytes);
    int* done = (int*)((char*)scratch + z.part_bytes + z.l_bytes + z.on_bytes + z.prob_bytes);
    cudaError_t e;
    {
        LorcStageTimer timer(ctx, LORC_STAGE_PV, st);
        ProbParams q;
        q.scores = scores; q.rowmax = rowmax; q.probs = probs; q.l_part = l_part; q.done = done; q.seq_lens = cv.seq_lens;
        q.status = ctx->status_dev; q.H_q = d.n_q_heads; q.n_pad = n_pad; q.tiles = tiles; q.tiles_per_group = tpg;
        q.n_groups = n_groups; q.n_blk = n_blk; q.max_pos = d.max_pos;
        dim3 pgrid(n_groups, cv.batch);
        if (d.n_q_heads == 32)
            e = lorc_launch_dependent(lorc_prob_kernel<32>, pgrid, dim3(256), 0, st, q);
        else
            e = lorc_launch_dependent(lorc_prob_kernel<64>, pgrid, dim3(256), 0, st, q);
        *launches += 1;
        if (e != cudaSuccess) return e;

        Pv2Params p;
        p.probs = probs; p.o_part = o_part; p.l_part = l_part; p.rowmax = rowmax; p.o_norm = o_norm; p.done = done;
        p.seq_lens = cv.seq_lens; p.page_table = cv.page_table; p.status = ctx->status_dev;
        p.batch = cv.batch; p.H_q = d.n_q_heads; p.n_kv = d.n_kv_heads; p.r_v = L.r_v; p.tiles = tiles;
        p.n_blk = n_blk; p.n_csplit = n_csplit; p.n_groups = n_groups; p.max_pos = d.max_pos;
        p.page_size = cv.page_size; p.max_pages_per_seq = cv.max_pages_per_seq; p.n_pages = cv.n_pages;
        dim3 grid(n_blk, n_csplit, cv.batch);
        if (d.n_q_heads == 32)
            e = lorc_launch_dependent(lorc_pv2_kernel<32>, grid, dim3(P_THREADS), sizeof(Pv2Smem<32>) + 1024, st, mapCV, p);
        else
            e = lorc_launch_dependent(lorc_pv2_kernel<64>, grid, dim3(P_THREADS), sizeof(Pv2Smem<64>) + 1024, st, mapCV, p);
        *launches += 1;
        if (e != cudaSuccess) return e;
    }
    LorcStageTimer timer(ctx, LORC_STAGE_COMBINE, st);
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
    dim3 ugrid(d.n_kv_heads, (cv.batch * ctx->group + 127) / 128, 128 / U_NCOL);
    e = lorc_launch_dependent(lorc_upproj_kernel, ugrid, dim3(U_THREADS), sizeof(UpSmem) + 1024, st, mapON, mapBVT, u);
    *launches += 1;
    return e;
}
