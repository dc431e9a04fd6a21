// P.C_V split by LATENT COLUMNS, and the value up-projection; both contractions run on the tensor cores.
//
// PV kernel.  A CTA owns one 128-column block of C_V (rho in [128 blk, 128 blk + 128)) of one sequence and one share
// of its context.  A block of latent columns is disjoint from every other block, so the CTA's accumulator
// O_lat^T[128 rho, H_q] (fp32 in TMEM) needs no merge with other column blocks.  The score kernel left, per tile of
// 128 tokens, the softmax numerators p = bf16(2^(s - m)) against an integer reference m per 32-token quarter and head
// (as the swizzled K-major image the MMA reads), m itself and the sums of p.  While the tile sits in shared memory the
// epilogue warps multiply it by 2^(m - M), M the reference of the whole sequence (exact: only the exponent changes),
// and add up the denominator; then
//       O_lat^T += C_V[tile, block]^T . P^T                    tcgen05, MN-major A
// and at the end the CTA writes its 128 x H_q piece of the latent output, normalised, as bf16 (with several context
// shares, the share that finishes last adds the others' pieces and denominators first).
//
// Up-projection.  One CTA per (KV head g, 64 output rows = 64 / G sequences, quarter of the head's columns)
// multiplies those rows by B_V[:, g] (TMA-staged from a transposed copy): out = o . B_V[:, g] in TMEM, then bf16.
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

// ------------------------------------------------------------------------------------------------
// PV kernel
// ------------------------------------------------------------------------------------------------
// Tile image written by the score kernel, fetched with one bulk copy per tile:
//   [2 chunks of 64 tokens][HQ rows of 128 bytes]   p = bf16(2^(s - m)), 128-byte swizzle (the MMA's B operand)
//   float m[4][HQ]   integer reference of every 32-token quarter and head (log2 units; -inf: no token)
//   float l[4][HQ]   sum of the quarter's rounded p
template <int HQ>
struct Pv2Smem {
    static constexpr int P_STAGES = PvStages<HQ>::value;
    static constexpr int IMG = 2 * HQ * KC * 2 + 8 * HQ * 4;
    // tile images (IMG is a multiple of 1 KiB).  They come first: with 32 heads the MMA's 64-row A operand runs
    // 4 KiB past a chunk of the image, into the next image or into V, never past the allocation
    uint8_t P[P_STAGES][IMG];
    bf16 V[P_STAGES][2][TILE * KC];       // C_V block: two 64-column halves of [128 tokens][64]; 32 KiB / stage
    float red[128 / HQ][HQ];
    float m_row[HQ];                      // row maximum over the whole sequence
    float l_inv[HQ];
    uint64_t vfull[P_STAGES], pfull[P_STAGES], fixed[P_STAGES], empty[P_STAGES], o_full, red_full;
    uint32_t tmem_base;
    int last;
};

struct Pv2Params {
    const uint8_t* pimg;           // [b, tiles, image]
    float* o_part;                 // [b, n_blk, n_csplit, H_q * 128 + H_q]   un-normalised latent output and denominator of every context share
    unsigned* rowmax;              // [b, H_q]   row maxima of the softmax (order-preserving keys of integers)
    bf16* o_norm;                  // [b, H_q, r_pad]      normalised latent output
    int* done;                     // [b, n_blk]           context shares of a column block that have finished (zero on entry)
    float* ml_out;                 // NULL, or [b, H_q, 2]: reference M (log2 units) and denominator sum_n 2^(s_n - M)
    const int32_t* seq_lens;
    const int32_t* page_table;
    int* status;
    int batch, H_q, n_kv, r_v, tiles, n_blk, n_csplit, max_pos;
    int page_size, max_pages_per_seq, n_pages;
};

// Biased exponent of 2^d for an integer-valued d <= 0 (0, i.e. the number zero, below 2^-126 and for d = -inf).
__device__ __forceinline__ uint32_t pow2_exponent(float d) { return d >= -126.f ? (uint32_t)(127 + (int)d) : 0u; }

template <int HQ>
__global__ void __launch_bounds__(P_THREADS, 1)
lorc_pv2_kernel(const __grid_constant__ CUtensorMap mapCV, const Pv2Params p) {
    extern __shared__ uint8_t raw[];
    typedef Pv2Smem<HQ> S;
    constexpr int P_STAGES = PvStages<HQ>::value;
    S& sm = *reinterpret_cast<S*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    constexpr uint32_t TM_COLS = 128;
    constexpr uint32_t P_BYTES = S::IMG;
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int blk = blockIdx.x, cs = blockIdx.y, s = blockIdx.z;

    int len = p.seq_lens[s];
    if (len > p.max_pos || len > p.tiles * TILE) len = 0;     // the score kernel reports the capacity error
    if (len < 0) len = 0;
    // this CTA's share of the context: whole 128-token tiles, dealt evenly over the context shares
    const int tiles_s = (len + TILE - 1) / TILE;
    const int per = (tiles_s + p.n_csplit - 1) / p.n_csplit;
    const int tile_lo = min(tiles_s, cs * per), tile_hi = min(tiles_s, tile_lo + per);
    const int ntiles = tile_hi - tile_lo;
    const int rho0 = blk * 128;

    if (tid == 0) {
        for (int i = 0; i < P_STAGES; ++i) {
            mbar_init(&sm.vfull[i], 1);
            mbar_init(&sm.pfull[i], 1);
            mbar_init(&sm.fixed[i], 4);
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
        // The kernel before this one only writes the tile images; the latent values were complete before IT could
        // start.  So the first stages' C_V boxes are requested right away, and only the images wait for that kernel
        // to finish.
        {
            for (int i = 0; i < ntiles && ok; ++i) {
                const int tile = tile_lo + i;
                const int n0 = tile * TILE;
                const int st = i % P_STAGES;
                if (i == P_STAGES) {
                    // images of the stages whose C_V boxes went out before the wait
                    grid_dep_wait();
                    if (elect_one()) {
                        for (int j = 0; j < P_STAGES; ++j) {
                            mbar_arrive_expect_tx(&sm.pfull[j], P_BYTES);
                            bulk_load(sm.P[j], p.pimg + ((long long)s * p.tiles + tile_lo + j) * P_BYTES, P_BYTES, &sm.pfull[j]);
                        }
                    }
                    __syncwarp();
                }
                if (!mbar_wait(&sm.empty[st], ((i / P_STAGES) & 1) ^ 1)) { ok = false; break; }
                if (elect_one()) {
                // the image (from L2, where the score kernel just left it) and the C_V block (from HBM) are counted on
                // barriers of their own: the exponent shift of the image runs while the block is still in flight
                if (i >= P_STAGES) {
                    mbar_arrive_expect_tx(&sm.pfull[st], P_BYTES);
                    bulk_load(sm.P[st], p.pimg + ((long long)s * p.tiles + tile) * P_BYTES, P_BYTES, &sm.pfull[st]);
                }
                mbar_arrive_expect_tx(&sm.vfull[st], 2 * TILE * KC * 2);
                if (p.page_table == nullptr) {
                    tma_load_3d(sm.V[st][0], &mapCV, &sm.vfull[st], rho0, n0, s);
                    tma_load_3d(sm.V[st][1], &mapCV, &sm.vfull[st], rho0 + 64, n0, s);
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
                        tma_load_3d(sm.V[st][0] + pg * p.page_size * KC, &mapCV, &sm.vfull[st], rho0, 0, page);
                        tma_load_3d(sm.V[st][1] + pg * p.page_size * KC, &mapCV, &sm.vfull[st], rho0 + 64, 0, page);
                    }
                }
                }
                __syncwarp();
            }
            if (ntiles <= P_STAGES) {
                grid_dep_wait();
                if (elect_one()) {
                    for (int j = 0; j < ntiles; ++j) {
                        mbar_arrive_expect_tx(&sm.pfull[j], P_BYTES);
                        bulk_load(sm.P[j], p.pimg + ((long long)s * p.tiles + tile_lo + j) * P_BYTES, P_BYTES, &sm.pfull[j]);
                    }
                }
                __syncwarp();
            }
            if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (warp-uniform, elected lane)
        if (ntiles > 0) {
            // O_lat[64 rows (heads; 32 of them unused with 32 heads), 128 rho] += P[heads, 16 tokens] . C_V[16 tokens, 128 rho]:
            // the heads are the M side (a small M costs few cycles per MMA), the latent columns the N side
            const uint32_t idesc = make_idesc_bf16(64, 128, 0, 1);
            for (int i = 0; i < ntiles && ok; ++i) {
                const int st = i % P_STAGES;
                if (!mbar_wait(&sm.fixed[st], (i / P_STAGES) & 1)) { ok = false; break; }
                if (!mbar_wait(&sm.vfull[st], (i / P_STAGES) & 1)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t p0 = smem_u32(sm.P[st]), v0 = smem_u32(sm.V[st][0]);
                if (elect_one()) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        // A: P [heads][128 tokens] (K-major), 64-token chunks of HQ*128 bytes
                        const uint64_t ad = make_smem_desc_sw128(p0 + (k >> 2) * (HQ * KC * 2) + (k & 3) * 32, 0, 1024);
                        // B: C_V block (MN-major: a token's 64 latent columns are contiguous): 16 token rows per step,
                        // the two 64-column halves 16 KiB apart
                        const uint64_t bd = make_smem_desc_sw128(v0 + k * 2048, TILE * KC * 2, 1024);
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
        // ------------------------------------------------------------------ exponent shift, then epilogue
        const int t = tid - 64;
        const int quarter = warp % 4;
        const int r_pad = p.n_blk * 128;
        constexpr int PARTS = 128 / HQ;                   // threads per head in the denominator sums
        grid_dep_wait();                                  // images and row maxima come from the kernel before this one
        grid_dep_launch();
        if (t < HQ) {
            const unsigned key = p.rowmax[(long long)s * p.H_q + t];
            sm.m_row[t] = key ? lorc_key_float(key) : 0.f;
        }
        __syncwarp();   // a named barrier counts a warp once only if the warp arrives converged
        asm volatile("bar.sync 2, 128;" ::: "memory");
        // While the tiles stream: every tile image holds p against the integer reference m of its own 32-token
        // quarter; multiplying by 2^(m - M), M the reference of the whole sequence, is exact in bf16 (a change of the
        // exponent) unless the product is too small to matter.  Thread t owns 2 HQ bytes of the image: with 32 heads
        // half a row (one head, one quarter), with 64 heads a whole row (one head, both quarters of a chunk).
        const int frow = (t * 2 * HQ) >> 7;               // row of the image: chunk * HQ + head
        const int fchunk = frow / HQ, fh = frow % HQ;
        const int fpiece0 = ((t * 2 * HQ) & 127) >> 4;    // first 16-byte piece (physical) of this thread
        const int frot = HQ == 32 ? (t >> 1) & 3 : t & 7;  // rotation of the order in which it takes its pieces
        const float m_mine = sm.m_row[fh];
        const int lh = t % HQ, lpart = t / HQ;            // denominator: head, and which quarters of a tile
        const float m_l = sm.m_row[lh];
        float lacc = 0.f;
        for (int i = 0; i < ntiles && ok; ++i) {
            const int st = i % P_STAGES;
            if (!mbar_wait(&sm.pfull[st], (i / P_STAGES) & 1)) { ok = false; break; }
            const float* mt = reinterpret_cast<const float*>(sm.P[st] + 2 * HQ * KC * 2);
            const float* lt = mt + 4 * HQ;
#pragma unroll
            for (int qq = 0; qq < 4 / PARTS; ++qq) {
                const int qrt = lpart * (4 / PARTS) + qq;
                lacc += lt[qrt * HQ + lh] * __uint_as_float(pow2_exponent(mt[qrt * HQ + lh] - m_l) << 23);
            }
            // 2^(m - M) of the quarter(s) this thread's pieces belong to, as a bf16 pair (built from the exponent: m and M
            // are integers).  A piece's quarter is bit 2 of its logical index, physical index xor (head & 7).
            uint32_t scb[2];
#pragma unroll
            for (int hq = 0; hq < 2; ++hq) {
                const uint32_t e = pow2_exponent(mt[(fchunk * 2 + hq) * HQ + fh] - m_mine) << 7;
                scb[hq] = e | (e << 16);
            }
            uint4* prow = reinterpret_cast<uint4*>(sm.P[st] + frow * 128);
            constexpr int NP = (2 * HQ) / 16;                 // 16-byte pieces per thread: 4 or 8
            uint4 v[NP];
            // (the pieces are taken in an order rotated by the thread index: the threads of a quarter warp, whose
            // pieces lie 64 or 128 bytes apart, then touch different banks)
#pragma unroll
            for (int j = 0; j < NP; ++j) v[j] = prow[fpiece0 + ((j + frot) & (NP - 1))];
#pragma unroll
            for (int j = 0; j < NP; ++j) {
                const int pp = fpiece0 + ((j + frot) & (NP - 1));
                const uint32_t sb = scb[((pp ^ (fh & 7)) >> 2) & 1];
                const __nv_bfloat162 sc = *reinterpret_cast<const __nv_bfloat162*>(&sb);
                __nv_bfloat162* e = reinterpret_cast<__nv_bfloat162*>(&v[j]);
#pragma unroll
                for (int k = 0; k < 4; ++k) e[k] = __hmul2(e[k], sc);
                prow[pp] = v[j];
            }
            fence_proxy_async_smem();      // the MMA reads the image through the asynchronous proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.fixed[st]);
        }
        // this share's part of the softmax denominator
        sm.red[lpart][lh] = lacc;
        __syncwarp();
        asm volatile("bar.sync 2, 128;" ::: "memory");
        float l_share = 0.f;
        if (t < HQ) {
#pragma unroll
            for (int i = 0; i < PARTS; ++i) l_share += sm.red[i][t];
        }
        if (ntiles > 0 && ok) {
            if (!mbar_wait(&sm.o_full, 0)) ok = false;
        }
        // The accumulator holds head 16 q + i (i < 16) in lane i of lane quarter q, 128 latent columns wide.
        const int hrow = quarter * 16 + lane;             // the head this thread reads (lanes 16..31 of a warp: none)
        const bool has_row = lane < 16 && hrow < HQ;
        constexpr int SHARE_FLOATS = HQ * 128 + HQ;
        if (p.n_csplit == 1) {
            if (t < HQ) {
                sm.l_inv[t] = l_share > 0.f ? 1.f / l_share : 0.f;
                if (!(l_share > 0.f) && blk == 0 && !p.ml_out) lorc_set_status(p.status, LORC_ERR_EMPTY);
                if (p.ml_out && blk == 0) {
                    p.ml_out[((long long)s * p.H_q + t) * 2] = sm.m_row[t];
                    p.ml_out[((long long)s * p.H_q + t) * 2 + 1] = l_share;
                }
            }
            __syncwarp();
            asm volatile("bar.sync 2, 128;" ::: "memory");
            const float li = has_row ? sm.l_inv[hrow] : 0.f;
            bf16* on = p.o_norm + ((long long)s * p.H_q + (has_row ? hrow : 0)) * r_pad + rho0;
#pragma unroll
            for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t r[32];
                if (ntiles > 0 && ok) {
                    tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + c0, r);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = 0u;
                }
                if (has_row) {
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(r[q4 * 8 + 2 * e]) * li,
                                                                            __uint_as_float(r[q4 * 8 + 2 * e + 1]) * li);
                            w[e] = *reinterpret_cast<const uint32_t*>(&b2);
                        }
                        *reinterpret_cast<uint4*>(on + c0 + q4 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
        } else {
            // publish this share (a contiguous block: [H_q][128] outputs, then [H_q] denominators); the share that
            // arrives last adds them all up (in share order, so the result does not depend on which one that is)
            float* blk_base = p.o_part + ((long long)s * p.n_blk + blk) * p.n_csplit * SHARE_FLOATS;
            float* op = blk_base + (long long)cs * SHARE_FLOATS;
#pragma unroll
            for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t r[32];
                if (ntiles > 0 && ok) {
                    tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + c0, r);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = 0u;
                }
                if (has_row) {
#pragma unroll
                    for (int q4 = 0; q4 < 8; ++q4)
                        *reinterpret_cast<uint4*>(op + hrow * 128 + c0 + q4 * 4) =
                            make_uint4(r[q4 * 4], r[q4 * 4 + 1], r[q4 * 4 + 2], r[q4 * 4 + 3]);
                }
            }
            if (t < HQ) op[HQ * 128 + t] = l_share;
            __threadfence();
            __syncwarp();   // a named barrier counts a warp once only if the warp arrives converged
            asm volatile("bar.sync 2, 128;" ::: "memory");
            if (t == 0) sm.last = atomicAdd(p.done + s * p.n_blk + blk, 1) == p.n_csplit - 1;
            __syncwarp();   // a named barrier counts a warp once only if the warp arrives converged
            asm volatile("bar.sync 2, 128;" ::: "memory");
            if (sm.last != 0) {
                __threadfence();
                // The shares come in by bulk copy, a batch at a time, into the C_V stages (every MMA that read them has
                // completed: o_full): one round trip per batch instead of one per share.  Thread = latent column.
                constexpr int PER = (P_STAGES * 2 * TILE * KC * 2) / (SHARE_FLOATS * 4);
                float* stage = reinterpret_cast<float*>(&sm.V[0][0][0]);
                float acc[HQ];
#pragma unroll
                for (int h = 0; h < HQ; ++h) acc[h] = 0.f;
                l_share = 0.f;
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
                        for (int h = 0; h < HQ; ++h) acc[h] += stage[j * SHARE_FLOATS + h * 128 + t];
                        if (t < HQ) l_share += stage[j * SHARE_FLOATS + HQ * 128 + t];
                    }
                }
                if (t < HQ) {
                    sm.l_inv[t] = l_share > 0.f ? 1.f / l_share : 0.f;
                    if (!(l_share > 0.f) && blk == 0 && !p.ml_out) lorc_set_status(p.status, LORC_ERR_EMPTY);
                    if (p.ml_out && blk == 0) {
                        p.ml_out[((long long)s * p.H_q + t) * 2] = sm.m_row[t];
                        p.ml_out[((long long)s * p.H_q + t) * 2 + 1] = l_share;
                    }
                }
                __syncwarp();
                asm volatile("bar.sync 2, 128;" ::: "memory");
                bf16* on = p.o_norm + (long long)s * p.H_q * r_pad + rho0 + t;
#pragma unroll
                for (int h = 0; h < HQ; ++h) on[(long long)h * r_pad] = __float2bfloat16_rn(acc[h] * sm.l_inv[h]);
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
// value up-projection: out[(s, h), :] = o_norm[s, h, :] . B_V[:, g(h)], a plain TMA-fed tcgen05 GEMM.
// grid (n_kv_heads, ceil(batch * G / 64), 4): 64 output rows (s, i) x 32 of the head's 128 columns, K = r_v in
// slices of 64.  (Splitting the columns gives four times the CTAs and small stages, so a whole rank is in flight.)
// ------------------------------------------------------------------------------------------------
constexpr int U_STAGES = 16;         // 16 x 12 KiB: every rank up to 1024 fits in one round of loads
constexpr int U_THREADS = 192;
constexpr int U_NCOL = 32;           // output columns per CTA (a quarter of a head)
constexpr int U_ROWS = 64;           // output rows (sequence, head of the KV head) per CTA: the M of the MMA

struct UpSmem {
    bf16 A[U_STAGES][U_ROWS * KC];        // o_norm rows [64 rows (s, i)][64 rho]
    bf16 B[U_STAGES][U_NCOL * KC];        // B_V^T slice [32 columns j][64 rho]
    uint64_t full[U_STAGES], empty[U_STAGES], d_full;
    uint32_t tmem_base;
};

struct UpParams {
    bf16* out;                     // [b, H_q, 128]
    unsigned* rowmax;              // [b, H_q]   left empty for the next call's score kernel
    int* status;
    int batch, H_q, G, r_v;
};

__global__ void __launch_bounds__(U_THREADS, 1)
lorc_upproj_kernel(const __grid_constant__ CUtensorMap mapON, const __grid_constant__ CUtensorMap mapBVT,
                   const UpParams p) {
    extern __shared__ uint8_t raw[];
    UpSmem& sm = *reinterpret_cast<UpSmem*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int g = blockIdx.x, chunk = blockIdx.y, cq = blockIdx.z;     // KV head, block of 64 rows, column quarter
    const int nkc = (p.r_v + KC - 1) / KC;
    const int seqs_per_cta = U_ROWS / p.G;
    constexpr uint32_t STAGE_BYTES = (U_ROWS + U_NCOL) * KC * 2;
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
        const uint32_t idesc = make_idesc_bf16(U_ROWS, U_NCOL, 0, 0);    // 64 rows: half the cycles of a 128-row MMA
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
        // every reader of the row maxima (the kernel before this one) has completed
        if (g == 0 && chunk == 0 && cq == 0)
            for (int i = tid - 64; i < p.batch * p.H_q; i += 128) p.rowmax[i] = 0u;
        if (!mbar_wait(&sm.d_full, 0)) ok = false;
        if (ok) {
            tc_fence_after_sync();
            // A 64-row accumulator keeps row 16 q + i (i < 16) in lane i of lane quarter q; row = s_local * G + i
            const int quarter = warp % 4;
            const int row = quarter * 16 + (lane & 15);
            const bool has_row = lane < 16;
            const int s = chunk * seqs_per_cta + row / p.G, h = g * p.G + row % p.G;
            {
                uint32_t r[32];
                tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16), r);
                tmem_wait_ld();
                if (has_row && s < p.batch) {
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

// Result of lorc_decode_attn_latent_out: the normalised latent output without the padding columns, and the row maxima
// left empty for the next call (what the up-projection kernel does otherwise).
__global__ void latent_out_kernel(const bf16* __restrict__ o_norm, bf16* __restrict__ o_lat, unsigned* rowmax, int rows,
                                  int r_v, int r_pad) {
    grid_dep_wait();
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < rows) rowmax[i] = 0u;
    const int vec = r_v / 8;                              // r_v is a multiple of 8: 16-byte pieces
    if (i < (long long)rows * vec) {
        const long long row = i / vec, c = i % vec;
        reinterpret_cast<uint4*>(o_lat + row * r_v)[c] = reinterpret_cast<const uint4*>(o_norm + row * r_pad)[c];
    }
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

struct PvScratch {
    size_t part_bytes, on_bytes, done_bytes;
};

PvScratch pv_scratch_layout(const lorc_ctx* ctx, int batch, int n_csplit, size_t r_pad) {
    PvScratch z;
    const size_t hq = (size_t)ctx->desc.n_q_heads;
    // [b][n_blk][n_csplit][H_q * 128 + H_q]
    z.part_bytes = n_csplit > 1 ? lorc_align_up((size_t)batch * (r_pad / 128) * n_csplit * (hq * 128 + hq) * sizeof(float), 256) : 256;
    z.on_bytes = lorc_align_up((size_t)batch * hq * r_pad * sizeof(bf16), 256);
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
    const size_t r_pad = (size_t)((ctx->n + 127) / 128) * 128;
    size_t worst = 0;
    // the share area grows with (column blocks x shares), which the plan keeps near the number of SMs
    for (int n_blk = 1; n_blk <= (int)(r_pad / 128); ++n_blk) {
        int c = ctx->sm_count / (batch * n_blk);
        if (c > cs) c = cs;
        if (c < 1) c = 1;
        const PvScratch z = pv_scratch_layout(ctx, batch, c, (size_t)n_blk * 128);
        if (z.part_bytes > worst) worst = z.part_bytes;
    }
    const PvScratch z = pv_scratch_layout(ctx, batch, 1, r_pad);
    return worst + z.on_bytes + z.done_bytes;
}

cudaError_t lorc_tc_pv_set_attrs() {
    cudaError_t e = cudaFuncSetAttribute(lorc_pv2_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)sizeof(Pv2Smem<32>) + 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(lorc_pv2_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)sizeof(Pv2Smem<64>) + 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(lorc_upproj_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)sizeof(UpSmem) + 1024);
    return e;
}

void lorc_tc_pv_plan(const lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, int n_splits_hint, size_t scratch_bytes,
                     LorcPvPlan* plan) {
    int n_blk, n_csplit;
    pv_plan(ctx, L, cv.batch, cv.max_seq_len, n_splits_hint, &n_blk, &n_csplit);
    PvScratch z;
    for (;; --n_csplit) {
        z = pv_scratch_layout(ctx, cv.batch, n_csplit, (size_t)n_blk * 128);
        if (z.part_bytes + z.on_bytes + z.done_bytes <= scratch_bytes || n_csplit == 1) break;
    }
    plan->n_blk = n_blk;
    plan->n_csplit = n_csplit;
    plan->fits = z.part_bytes + z.on_bytes + z.done_bytes <= scratch_bytes;
    plan->off_on = z.part_bytes;
    plan->off_done = z.part_bytes + z.on_bytes;
}

// scratch: [o_part | o_norm | done]; `done` (plan.n_blk * batch words) must be zero when the PV kernel starts (the
// score kernel clears it).
cudaError_t lorc_tc_pv_launch(lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, const CUtensorMap& mapCV,
                              const CUtensorMap& mapBVT, const uint8_t* pimg, unsigned* rowmax, int tiles,
                              const LorcPvPlan& plan, void* scratch, bf16* out, bool latent_out, float* ml_out,
                              cudaStream_t st, int* launches) {
    const lorc_model_desc& d = ctx->desc;
    const int n_blk = plan.n_blk, n_csplit = plan.n_csplit;
    const int r_pad = n_blk * 128;
    float* o_part = (float*)scratch;
    bf16* o_norm = (bf16*)((char*)scratch + plan.off_on);
    int* done = (int*)((char*)scratch + plan.off_done);
    cudaError_t e;
    {
        LorcStageTimer timer(ctx, LORC_STAGE_PV, st);
        Pv2Params p;
        p.pimg = pimg; p.o_part = o_part; p.rowmax = rowmax; p.o_norm = o_norm; p.done = done; p.ml_out = ml_out;
        p.seq_lens = cv.seq_lens; p.page_table = cv.page_table; p.status = ctx->status_dev;
        p.batch = cv.batch; p.H_q = d.n_q_heads; p.n_kv = d.n_kv_heads; p.r_v = L.r_v; p.tiles = tiles;
        p.n_blk = n_blk; p.n_csplit = n_csplit; p.max_pos = d.max_pos;
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
    if (latent_out) {
        const int rows = cv.batch * d.n_q_heads;
        const long long work = (long long)rows * (L.r_v / 8);
        e = lorc_launch_dependent(latent_out_kernel, dim3((unsigned)((work + 255) / 256)), dim3(256), 0, st,
                                  (const bf16*)o_norm, out, rowmax, rows, L.r_v, r_pad);
        *launches += 1;
        return e;
    }
    // o_norm [b, H_q, r_pad] as (rho, head, sequence) with boxes of 64 rho x G heads x 64/G sequences
    CUtensorMap mapON;
    {
        uint64_t dims[3] = {(uint64_t)r_pad, (uint64_t)d.n_q_heads, (uint64_t)cv.batch};
        uint64_t str[2] = {(uint64_t)r_pad * 2, (uint64_t)d.n_q_heads * r_pad * 2};
        uint32_t box[3] = {KC, (uint32_t)ctx->group, (uint32_t)(U_ROWS / ctx->group)};
        if (!lorc_make_tmap_bf16(&mapON, o_norm, 3, dims, str, box)) return cudaErrorInvalidValue;
    }
    UpParams u;
    u.out = out; u.rowmax = rowmax; u.status = ctx->status_dev;
    u.batch = cv.batch; u.H_q = d.n_q_heads; u.G = ctx->group; u.r_v = L.r_v;
    dim3 ugrid(d.n_kv_heads, (cv.batch * ctx->group + U_ROWS - 1) / U_ROWS, 128 / U_NCOL);
    e = lorc_launch_dependent(lorc_upproj_kernel, ugrid, dim3(U_THREADS), sizeof(UpSmem) + 1024, st, mapON, mapBVT, u);
    *launches += 1;
    return e;
}
