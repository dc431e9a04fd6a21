// Prompt processing on the tensor cores (sm_100a): attention of the T newest tokens of every sequence over its latent
// cache, the cached prefix in full and the new chunk causally (Preliminary section's Attention(Q, K, V) with the usual
// mask; keys and values reconstructed from the latents of Sec. 3.1, rotation at attention time as in the appendix).
//
// With many queries per key the reconstruction is worth keeping: every key and value of the layer is rebuilt ONCE into
// a transient fp16 buffer (the decode path rebuilds them per query and never stores them), then a flash-attention
// kernel runs over that buffer.
//
//   reconstruct kernel  K^[tile, head] = RoPE(C_K[tile, :] . B_K[:, head]),  V[tile, head] = C_V[tile, :] . B_V[:, head]
//                       persistent CTA pairs over (two 128-token tiles, pair of KV heads): TMA-staged 64-wide slices,
//                       tcgen05 cta_group::2 (M = 256 tokens, N = 256), rotation in the epilogue (thread = token row)
//                       under the next unit's MMAs, 16-bit rows to the buffer: keys as
//                       fp16 (the scores are then exact to 2^-11 of |q| |k|, four times closer than with bf16 keys),
//                       values as fp16 too (a reconstructed element must stay below 65504 in magnitude)
//   attention kernel    one CTA per two blocks of 128 query rows (128 / G positions x G heads of one KV head each); the
//                       rows are rotated at their positions and scaled in shared memory, Q^ = RoPE(q) log2(e) / sqrt(d_h)
//                       as fp16, before the first MMA; for
//                       every 128-key tile and block   S = Q^ K^^T (tcgen05, fp32 in TMEM)  ->  online softmax, thread =
//                       query row; the probabilities go back into tensor memory as fp16 over the scores  ->  O += P V
//                       with P read from tensor memory.  The two blocks alternate, so the tensor pipe works on one
//                       while the other's softmax runs.  The running reference of a row is only raised when a tile
//                       exceeds it by more than 2^8 (the accumulator is rescaled then), so most tiles need no pass over O.
#include <cuda_fp16.h>
#include <math.h>

#include "sm100_pair.cuh"
#include "sm100_ptx.cuh"
#include "tc_kernels.cuh"

using namespace sm100;

namespace {

constexpr int TILE = 128;
constexpr int KC = 64;
constexpr float LOG2E = 1.4426950408889634f;

// ------------------------------------------------------------------------------------------------
// reconstruction of keys (rotated) or values into [b, n_rows, n] fp16
// ------------------------------------------------------------------------------------------------
// Persistent CTA PAIRS (clusters of two, cta_group::2 MMAs) walk units (sequence, pair of 128-token tiles, pair of KV
// heads), the head pair running fastest (the pairs that work on the same latent rows at the same time share them in
// L2).  Per unit  acc[256 tokens, 256 features] = C[tiles, :] . B[:, 2 heads]  in 64-wide slices: each CTA stages its
// own 128 tokens and HALF of the factor slice (what a CTA can take in through TMA, not the MMA rate, bounds a
// single CTA with the whole slice); the accumulator is double-buffered in tensor memory, so the epilogue of one unit
// (rotation, rounding, 512-byte row stores of the CTA's own tokens) runs under the MMAs of the next.
constexpr int R_STAGES = 6;
constexpr int R_THREADS = 192;       // warp 0 TMA, warp 1 MMA (leader CTA issues), warps 2..5 epilogue
constexpr int R_N = 256;             // features per unit: two KV heads

struct RecSmem {
    bf16 A[R_STAGES][TILE * KC];          // latent slice of this CTA's tile [128 tokens][64]
    bf16 B[R_STAGES][TILE * KC];          // this CTA's half of the factor slice [128 features][64]
    uint64_t full[R_STAGES], empty[R_STAGES], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
};

struct RecParams {
    bf16* out;                     // [b, n_rows, n]
    const int32_t* seq_lens;
    const int32_t* page_table;
    const float2* rope_table;      // [max_pos][64]
    int* status;
    int r, n, n_rows, max_pos, batch, tile_pairs, n_hp;
    int page_size, max_pages_per_seq, n_pages;
};

template <bool ROPE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(R_THREADS, 1)
lorc_reconstruct_kernel(const __grid_constant__ CUtensorMap mapC, const __grid_constant__ CUtensorMap mapBT, const RecParams p) {
    extern __shared__ uint8_t raw[];
    RecSmem& sm = *reinterpret_cast<RecSmem*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int rank = (int)cluster_ctarank();           // 0 = leader (issues the MMAs, owns the full / acc_empty barriers)
    const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int nkc = (p.r + KC - 1) / KC;
    const int total = p.batch * p.tile_pairs * p.n_hp;
    // unit -> (sequence, tile pair, head pair); a unit whose first tile lies past the sequence's cached tokens is
    // skipped by both CTAs and every role alike (sequences beyond the buffer are reported by the attention kernel)
    auto decode = [&](int u, int& s, int& tp, int& hp, int& len) -> bool {
        hp = u % p.n_hp;
        const int st = u / p.n_hp;
        tp = st % p.tile_pairs;
        s = st / p.tile_pairs;
        len = p.seq_lens[s];
        if (len > p.max_pos || len > p.n_rows) len = 0;
        return 2 * tp * TILE < len;
    };

    if (tid == 0) {
        for (int i = 0; i < R_STAGES; ++i) {
            mbar_init(&sm.full[i], 1);
            mbar_init(&sm.empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sm.acc_full[i], 1);
            mbar_init(&sm.acc_empty[i], 2 * 4);             // one arrival per epilogue warp, both CTAs
        }
        fence_barrier_init();
        prefetch_tensormap(&mapC);
        prefetch_tensormap(&mapBT);
    }
    if (warp == 1) {
        tmem_alloc_pair(&sm.tmem_base, 512);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_arrive_release();                            // the peer's barriers are initialised before anyone signals them
    cluster_wait_acquire();
    tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    bool ok = true;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        const uint32_t a_base = smem_u32(sm.A[0]), b_base = smem_u32(sm.B[0]);
        const uint32_t empty0 = smem_u32(&sm.empty[0]), full0 = smem_u32(&sm.full[0]);
        const uint32_t lead_full0 = mapa_shared(full0, 0);   // all bytes of a stage are counted on the leader's barrier
        uint32_t st = 0, par = 1;
        for (int u = pair_id; u < total && ok; u += n_pairs) {
            int s, tp, hp, len;
            if (!decode(u, s, tp, hp, len)) continue;
            const int tile = 2 * tp + rank;
            for (int kc = 0; kc < nkc; ++kc) {
                if (!mbar_wait_addr(empty0 + st * 8, par)) { ok = false; break; }
                const uint32_t lead_bar = lead_full0 + st * 8;
                const uint32_t a_dst = a_base + st * (TILE * KC * 2);
                if (elect_one()) {
                    if (rank == 0) mbar_arrive_expect_tx_addr(full0 + st * 8, 2 * 2 * TILE * KC * 2);
                    if (p.page_table == nullptr) {
                        // (a tile past the buffer's rows reads as zero)
                        tma_load_3d_pair_addr(a_dst, &mapC, lead_bar, kc * KC, tile * TILE, s);
                    } else {
                        // one box per page; pages past the end of the sequence (or with a bad table entry) come from page 0
                        const int ppt = TILE / p.page_size;
                        for (int pg = 0; pg < ppt; ++pg) {
                            const int lp = tile * ppt + pg;
                            int page = 0;
                            if ((long long)lp * p.page_size < len && lp < p.max_pages_per_seq) {
                                page = p.page_table[(long long)s * p.max_pages_per_seq + lp];
                                if (page < 0 || page >= p.n_pages) {
                                    lorc_set_status(p.status, LORC_ERR_CAPACITY);
                                    page = 0;
                                }
                            }
                            tma_load_3d_pair_addr(a_dst + pg * p.page_size * KC * 2, &mapC, lead_bar, kc * KC, 0, page);
                        }
                    }
                    tma_load_2d_pair_addr(b_base + st * (TILE * KC * 2), &mapBT, lead_bar, kc * KC, hp * R_N + rank * 128);
                }
                __syncwarp();
                if (++st == R_STAGES) { st = 0; par ^= 1; }
            }
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (rank == 0) {
            const uint32_t idesc = make_idesc_bf16(256, R_N, 0, 0);
            const int nk_last = (p.r - (nkc - 1) * KC + 15) >> 4;     // 16-column steps the last stage really holds
            const uint64_t da0 = make_smem_desc_sw128(smem_u32(sm.A[0]), 0, 1024);
            const uint64_t db0 = make_smem_desc_sw128(smem_u32(sm.B[0]), 0, 1024);
            const uint32_t a_lo0 = (uint32_t)da0, a_hi = (uint32_t)(da0 >> 32);
            const uint32_t b_lo0 = (uint32_t)db0, b_hi = (uint32_t)(db0 >> 32);
            const uint32_t empty0 = smem_u32(&sm.empty[0]), full0 = smem_u32(&sm.full[0]);
            uint32_t st = 0, par = 0, uc = 0;
            for (int u = pair_id; u < total && ok; u += n_pairs) {
                int s, tp, hp, len;
                if (!decode(u, s, tp, hp, len)) continue;
                const int buf = uc & 1;
                if (!mbar_wait(&sm.acc_empty[buf], ((uc >> 1) & 1) ^ 1)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d = tmem + buf * R_N;
                for (int kc = 0; kc < nkc; ++kc) {
                    if (!mbar_wait_addr(full0 + st * 8, par)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t a_lo = a_lo0 + st * (TILE * KC * 2 / 16), b_lo = b_lo0 + st * (TILE * KC * 2 / 16);
                    if (elect_one()) {
                        if (kc == 0)
                            tc_mma_bf16_pair_set(d, a_lo, a_hi, b_lo, b_hi, idesc);
                        else
                            tc_mma_bf16_pair_acc(d, a_lo, a_hi, b_lo, b_hi, idesc);
                        const int nk = (kc + 1 < nkc) ? 4 : nk_last;
                        if (nk > 1) tc_mma_bf16_pair_acc(d, a_lo + 2, a_hi, b_lo + 2, b_hi, idesc);
                        if (nk > 2) tc_mma_bf16_pair_acc(d, a_lo + 4, a_hi, b_lo + 4, b_hi, idesc);
                        if (nk > 3) tc_mma_bf16_pair_acc(d, a_lo + 6, a_hi, b_lo + 6, b_hi, idesc);
                        tc_commit_pair_addr(empty0 + st * 8);        // frees the stage in both CTAs
                    }
                    __syncwarp();
                    if (++st == R_STAGES) { st = 0; par ^= 1; }
                }
                if (!ok) break;
                if (elect_one()) tc_commit_pair(&sm.acc_full[buf]);   // both CTAs' epilogues may read their accumulators
                __syncwarp();
                ++uc;
            }
            if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
        }
    } else {
        // ------------------------------------------------------------------ epilogue (both CTAs): this CTA's 128 tokens
        const int quarter = warp % 4;
        const int row = quarter * 32 + lane;                         // token of the tile = TMEM lane
        const uint32_t lead_acc_empty[2] = {mapa_shared(smem_u32(&sm.acc_empty[0]), 0),
                                            mapa_shared(smem_u32(&sm.acc_empty[1]), 0)};
        uint32_t uc = 0;
        for (int u = pair_id; u < total && ok; u += n_pairs) {
            int s, tp, hp, len;
            if (!decode(u, s, tp, hp, len)) continue;
            const int buf = uc & 1;
            if (!mbar_wait(&sm.acc_full[buf], (uc >> 1) & 1)) { ok = false; break; }
            tc_fence_after_sync();
            const int pos = (2 * tp + rank) * TILE + row;
            const float2* cs = p.rope_table + (long long)min(pos, p.max_pos - 1) * 64;
#pragma unroll 1
            for (int hd = 0; hd < 2; ++hd) {
                bf16* dst = p.out + ((long long)s * p.n_rows + pos) * p.n + (hp * 2 + hd) * 128;
                const uint32_t tcol = tmem + ((uint32_t)(quarter * 32) << 16) + buf * R_N + hd * 128;
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t ra[32], rb[32];
                    tmem_ld32(tcol + c0, ra);          // elements c0 .. c0 + 31 of the head
                    tmem_ld32(tcol + 64 + c0, rb);     // their partners in the second half
                    tmem_wait_ld();
                    if (pos < p.n_rows) {
                        uint32_t wa[16], wb[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            float a0 = __uint_as_float(ra[2 * i]), a1 = __uint_as_float(ra[2 * i + 1]);
                            float b0 = __uint_as_float(rb[2 * i]), b1 = __uint_as_float(rb[2 * i + 1]);
                            if (ROPE) {
                                const float4 t = __ldg(reinterpret_cast<const float4*>(cs + c0 + 2 * i));   // (cos, sin) x 2
                                const float x0 = a0 * t.x - b0 * t.y, y0 = a0 * t.y + b0 * t.x;
                                const float x1 = a1 * t.z - b1 * t.w, y1 = a1 * t.w + b1 * t.z;
                                a0 = x0; b0 = y0; a1 = x1; b1 = y1;
                            }
                            {                    // keys and values alike: fp16
                                const __half2 pa = __floats2half2_rn(a0, a1), pb = __floats2half2_rn(b0, b1);
                                wa[i] = *reinterpret_cast<const uint32_t*>(&pa);
                                wb[i] = *reinterpret_cast<const uint32_t*>(&pb);
                            }
                        }
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            reinterpret_cast<uint4*>(dst + c0)[v] = make_uint4(wa[4 * v], wa[4 * v + 1], wa[4 * v + 2], wa[4 * v + 3]);
                            reinterpret_cast<uint4*>(dst + 64 + c0)[v] = make_uint4(wb[4 * v], wb[4 * v + 1], wb[4 * v + 2], wb[4 * v + 3]);
                        }
                    }
                }
            }
            // this warp has read its part of the accumulator
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(lead_acc_empty[buf]);
            ++uc;
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    }
    // both CTAs are done with tensor memory and with each other's barriers before either lets go
    tc_fence_before_sync();
    __syncthreads();
    cluster_arrive_release();
    cluster_wait_acquire();
    if (warp == 1) tmem_dealloc_pair(tmem, 512);
}

// ------------------------------------------------------------------------------------------------
// attention over the reconstructed keys and values
// ------------------------------------------------------------------------------------------------
// A CTA owns TWO blocks of 128 query rows (block b: 128 / G positions x the G heads of one KV head) and walks the key
// tiles once for both.  The blocks alternate on the tensor pipe: while the softmax warps of one block turn its scores
// into probabilities, the pipe multiplies the other block's probabilities into its output and computes its next
// scores.  Tensor memory: scores / probabilities of block b at column 128 b, its output at column 256 + 128 b.
constexpr int F_THREADS = 320;       // warp 0 TMA, warp 1 MMA, warps 2..5 softmax of block 0, warps 6..9 of block 1
constexpr int F_STAGES = 2;
constexpr float F_RAISE = 8.f;       // a row's reference is raised only when a tile exceeds it by more than this (log2 units)

struct FaSmem {
    bf16 Q[2][2][TILE * KC];              // [block][64-element half][128 rows]
    bf16 K[F_STAGES][2][TILE * KC];       // key tile [128 keys][two halves]
    bf16 V[F_STAGES][2][TILE * KC];       // value tile [128 keys][two halves]
    uint64_t q_full, q_ready, k_full[F_STAGES], v_full[F_STAGES], k_empty[F_STAGES], v_empty[F_STAGES];
    uint64_t s_full[2], p_half[2], p_ready[2], o_done;
    uint32_t tmem_base;
};

struct FaParams {
    bf16* out;                     // [b, T, H_q, 128]
    const int32_t* seq_lens;
    const float2* rope_table;      // [max_pos][64]
    int* status;
    int T, H_q, G, n_rows, max_pos;
};

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 32 scores of a row -> probabilities 2^(s - m), rounded to fp16 and packed two per column at tensor-memory address
// taddr (16 columns); their unrounded sums are added to l0 / l1.  (Packed fp32 adds for the subtraction and the sums
// were measured 2.5 % slower than these scalar ones: the pack / unpack moves cost more than the adds they save.)
__device__ __forceinline__ void probs_chunk(const uint32_t (&r)[32], float m, uint32_t taddr, float& l0, float& l1) {
    uint32_t w[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float e0 = ex2_approx(__uint_as_float(r[2 * i]) - m), e1 = ex2_approx(__uint_as_float(r[2 * i + 1]) - m);
        l0 += e0;
        l1 += e1;
        const __half2 pr = __floats2half2_rn(e0, e1);
        w[i] = *reinterpret_cast<const uint32_t*>(&pr);
    }
    tmem_st16(taddr, w);
}

__global__ void __launch_bounds__(F_THREADS, 1)
lorc_prefill_attn_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                         const __grid_constant__ CUtensorMap mapV, const FaParams p) {
    extern __shared__ uint8_t raw[];
    FaSmem& sm = *reinterpret_cast<FaSmem*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int g = blockIdx.y, s = blockIdx.z;
    const int qp = TILE / p.G;                                // query positions per block of 128 rows
    // the CTAs with the latest positions see the most keys: they go first
    const int t0 = ((int)gridDim.x - 1 - (int)blockIdx.x) * 2 * qp;   // first position (inside the chunk) of this CTA
    int len = p.seq_lens[s];
    if (len > p.max_pos || len > p.n_rows) {
        if (tid == 0) lorc_set_status(p.status, LORC_ERR_CAPACITY);
        len = 0;
    }
    if (len < p.T) {                                          // the chunk is not in the cache: nothing to attend
        if (tid == 0 && len > 0) lorc_set_status(p.status, LORC_ERR_ARG);
        len = 0;
    }
    const int t_last = min(p.T, t0 + 2 * qp) - 1;             // last query position of the CTA
    const int n_tiles = len > 0 ? (len - p.T + t_last) / TILE + 1 : 0;

    if (tid == 0) {
        mbar_init(&sm.q_full, 1);
        mbar_init(&sm.q_ready, 8);
        for (int i = 0; i < F_STAGES; ++i) {
            mbar_init(&sm.k_full[i], 1);
            mbar_init(&sm.v_full[i], 1);
            mbar_init(&sm.k_empty[i], 1);
            mbar_init(&sm.v_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sm.s_full[i], 1);
            mbar_init(&sm.p_half[i], 4);
            mbar_init(&sm.p_ready[i], 4);
        }
        mbar_init(&sm.o_done, 1);
        fence_barrier_init();
        prefetch_tensormap(&mapQ);
        prefetch_tensormap(&mapK);
        prefetch_tensormap(&mapV);
    }
    if (warp == 1) {
        tmem_alloc(&sm.tmem_base, 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    bool ok = true;

    if (warp == 0) {
        if (n_tiles > 0) {
            if (elect_one()) {
                // rows of a block: (position, head i of the KV head) -> row (position - first) * G + i; positions past the
                // chunk read as zero
                mbar_arrive_expect_tx(&sm.q_full, 4 * TILE * KC * 2);
                for (int b = 0; b < 2; ++b) {
                    tma_load_4d(sm.Q[b][0], &mapQ, &sm.q_full, 0, g * p.G, t0 + b * qp, s);
                    tma_load_4d(sm.Q[b][1], &mapQ, &sm.q_full, 64, g * p.G, t0 + b * qp, s);
                }
            }
            __syncwarp();
            for (int j = 0; j < n_tiles && ok; ++j) {
                const int st = j % F_STAGES;
                const uint32_t par = ((j / F_STAGES) & 1) ^ 1;
                if (!mbar_wait(&sm.k_empty[st], par)) { ok = false; break; }
                if (elect_one()) {
                    mbar_arrive_expect_tx(&sm.k_full[st], 2 * TILE * KC * 2);
                    tma_load_3d(sm.K[st][0], &mapK, &sm.k_full[st], g * 128, j * TILE, s);
                    tma_load_3d(sm.K[st][1], &mapK, &sm.k_full[st], g * 128 + 64, j * TILE, s);
                }
                __syncwarp();
                if (!mbar_wait(&sm.v_empty[st], par)) { ok = false; break; }
                if (elect_one()) {
                    mbar_arrive_expect_tx(&sm.v_full[st], 2 * TILE * KC * 2);
                    tma_load_3d(sm.V[st][0], &mapV, &sm.v_full[st], g * 128, j * TILE, s);
                    tma_load_3d(sm.V[st][1], &mapV, &sm.v_full[st], g * 128 + 64, j * TILE, s);
                }
                __syncwarp();
            }
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    } else if (warp == 1) {
        if (n_tiles > 0) {
            const uint32_t idesc_s = make_idesc_f16(128, 128);            // S = Q K^T: fp16 operands, both K-major
            const uint32_t idesc_o = make_idesc_f16(128, 128, 0, 1);      // O += P V: fp16 too, V MN-major (a key's elements are contiguous)
            // The MMAs of one thread run in the order they were issued, and a commit covers everything issued before it:
            // when s_full[b] fires for tile j + 1, block b's P V of tile j has also finished with the probabilities that
            // these scores overwrite and with the output a softmax warp may rescale.
            auto scores = [&](int b, int st) {
                const uint32_t q0 = smem_u32(sm.Q[b][0]), k0 = smem_u32(sm.K[st][0]);
                if (elect_one()) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const uint32_t off = (k >> 2) * (TILE * KC * 2) + (k & 3) * 32;
                        tc_mma_bf16(tmem + b * 128, make_smem_desc_sw128(q0 + off, 0, 1024),
                                    make_smem_desc_sw128(k0 + off, 0, 1024), idesc_s, k != 0);
                    }
                    tc_commit(&sm.s_full[b]);
                    if (b == 1) tc_commit(&sm.k_empty[st]);
                }
                __syncwarp();
            };
            if (!mbar_wait(&sm.q_ready, 0)) ok = false;          // the query rows, rotated and scaled in place
            if (ok && !mbar_wait(&sm.k_full[0], 0)) ok = false;
            if (ok) {
                tc_fence_after_sync();
                scores(0, 0);
                scores(1, 0);
            }
            for (int j = 0; j < n_tiles && ok; ++j) {
                const int st = j % F_STAGES, st1 = (j + 1) % F_STAGES;
                const uint32_t v0 = smem_u32(sm.V[st][0]);
#pragma unroll 1
                for (int b = 0; b < 2 && ok; ++b) {
                    // the softmax warps of block b replace its scores by probabilities (and rescale its output first if
                    // needed); they report the first 64 keys' worth and then the rest, so the first half of P V runs
                    // while the second half of the exponentials is still being computed
                    if (!mbar_wait(&sm.p_half[b], j & 1)) { ok = false; break; }
                    if (b == 0 && !mbar_wait(&sm.v_full[st], (j / F_STAGES) & 1)) { ok = false; break; }
                    tc_fence_after_sync();
                    if (elect_one()) {
#pragma unroll
                        for (int k = 0; k < 4; ++k)      // 16 keys per step: 8 columns of packed probabilities, 16 rows of V
                            tc_mma_bf16_ts(tmem + 256 + b * 128, tmem + b * 128 + k * 8,
                                           make_smem_desc_sw128(v0 + k * 2048, TILE * KC * 2, 1024), idesc_o, (j | k) != 0);
                    }
                    __syncwarp();
                    if (!mbar_wait(&sm.p_ready[b], j & 1)) { ok = false; break; }
                    tc_fence_after_sync();
                    if (elect_one()) {
#pragma unroll
                        for (int k = 4; k < 8; ++k)
                            tc_mma_bf16_ts(tmem + 256 + b * 128, tmem + b * 128 + k * 8,
                                           make_smem_desc_sw128(v0 + k * 2048, TILE * KC * 2, 1024), idesc_o, 1);
                        if (b == 1) tc_commit(&sm.v_empty[st]);
                        if (b == 1 && j + 1 == n_tiles) tc_commit(&sm.o_done);
                    }
                    __syncwarp();
                    if (j + 1 < n_tiles) {
                        if (b == 0 && !mbar_wait(&sm.k_full[st1], ((j + 1) / F_STAGES) & 1)) { ok = false; break; }
                        tc_fence_after_sync();
                        scores(b, st1);
                    }
                }
            }
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    } else {
        const int b = (warp - 2) >> 2;                           // block of this softmax warp
        const int quarter = warp % 4;                            // the 32 lanes of tensor memory this warp may touch
        const int row = quarter * 32 + lane;
        const int tt = b * qp + row / p.G, hi = row % p.G;
        const bool live = len > 0 && t0 + tt < p.T;
        const int pq = live ? len - p.T + t0 + tt : -1;          // this row's position: it sees keys 0 .. pq
        const uint32_t trow = tmem + ((uint32_t)(quarter * 32) << 16) + b * 128;   // scores / probabilities
        const uint32_t orow = tmem + ((uint32_t)(quarter * 32) << 16) + 256 + b * 128;
        float m_ref = -INFINITY, l0 = 0.f, l1 = 0.f;      // l0 + l1: sum of the row's probabilities
        if (n_tiles > 0) {
            // Q^ = RoPE(q, position) * log2(e) / sqrt(d_h), fp16, in place: this thread's row of the block, 16 bytes at a
            // time.  The two 64-element halves of a row have the same swizzled layout, so a rotary pair (j, j + 64) sits
            // at the same offset of both; elements 8 lc ... 8 lc + 7 of row r are its physical 16-byte piece lc ^ (r & 7).
            if (!mbar_wait(&sm.q_full, 0)) ok = false;
            if (ok) {
                const float scale = rsqrtf(128.f) * LOG2E;
                const float2* cs = p.rope_table + (long long)min(max(pq, 0), p.max_pos - 1) * 64;
                uint4* h0 = reinterpret_cast<uint4*>(sm.Q[b][0]) + row * 8;
                uint4* h1 = reinterpret_cast<uint4*>(sm.Q[b][1]) + row * 8;
#pragma unroll
                for (int lc = 0; lc < 8; ++lc) {
                    // logical piece lc of every row at once: the rows of a quarter warp then touch all eight physical
                    // pieces (no shared-memory bank conflict)
                    const int pc = lc ^ (row & 7), j0 = 8 * lc;
                    uint4 a = h0[pc], c = h1[pc];
                    uint32_t* aw = reinterpret_cast<uint32_t*>(&a);
                    uint32_t* cw = reinterpret_cast<uint32_t*>(&c);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float4 t = __ldg(reinterpret_cast<const float4*>(cs + j0 + 2 * e));   // (cos, sin) x 2
                        const float a0 = __uint_as_float(aw[e] << 16), a1 = __uint_as_float(aw[e] & 0xffff0000u);
                        const float b0 = __uint_as_float(cw[e] << 16), b1 = __uint_as_float(cw[e] & 0xffff0000u);
                        const __half2 x = __floats2half2_rn((a0 * t.x - b0 * t.y) * scale, (a1 * t.z - b1 * t.w) * scale);
                        const __half2 y = __floats2half2_rn((a0 * t.y + b0 * t.x) * scale, (a1 * t.w + b1 * t.z) * scale);
                        aw[e] = *reinterpret_cast<const uint32_t*>(&x);
                        cw[e] = *reinterpret_cast<const uint32_t*>(&y);
                    }
                    h0[pc] = a;
                    h1[pc] = c;
                }
                fence_proxy_async_smem();      // the MMA reads the rows through the asynchronous proxy
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.q_ready);
            }
        }
        for (int j = 0; j < n_tiles && ok; ++j) {
            if (!mbar_wait(&sm.s_full[b], j & 1)) { ok = false; break; }
            tc_fence_after_sync();
            const int n0 = j * TILE;
            // the whole row of scores in registers
            uint32_t r0[32], r1[32], r2[32], r3[32];
            tmem_ld32(trow, r0);
            tmem_ld32(trow + 32, r1);
            tmem_ld32(trow + 64, r2);
            tmem_ld32(trow + 96, r3);
            tmem_wait_ld();
            // keys past the row's own position (tiles on the diagonal, rows past the chunk) count as -inf
            if (__any_sync(0xffffffffu, n0 + TILE - 1 > pq)) {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    if (n0 + i > pq) r0[i] = 0xff800000u;
                    if (n0 + 32 + i > pq) r1[i] = 0xff800000u;
                    if (n0 + 64 + i > pq) r2[i] = 0xff800000u;
                    if (n0 + 96 + i > pq) r3[i] = 0xff800000u;
                }
            }
            // the row maximum: four independent chains
            float mt0 = -INFINITY, mt1 = -INFINITY, mt2 = -INFINITY, mt3 = -INFINITY;
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                mt0 = max3(mt0, __uint_as_float(r0[i]), __uint_as_float(r0[i + 1]));
                mt1 = max3(mt1, __uint_as_float(r1[i]), __uint_as_float(r1[i + 1]));
                mt2 = max3(mt2, __uint_as_float(r2[i]), __uint_as_float(r2[i + 1]));
                mt3 = max3(mt3, __uint_as_float(r3[i]), __uint_as_float(r3[i + 1]));
            }
            const float mt = fmaxf(fmaxf(mt0, mt1), fmaxf(mt2, mt3));
            // raise the reference?  (the accesses to tensor memory below are warp-wide: the warp rescales if any of its
            // rows must, the other rows by a factor of one)
            const bool raise = mt > m_ref + F_RAISE || (m_ref == -INFINITY && mt > -INFINITY);
            if (__any_sync(0xffffffffu, raise)) {
                // what has been accumulated so far shrinks by 2^(old - new)
                const float alpha = !raise ? 1.f : (m_ref == -INFINITY ? 0.f : exp2f(m_ref - mt));
                l0 *= alpha;
                l1 *= alpha;
                if (j > 0) {
#pragma unroll 1
                    for (int c0 = 0; c0 < TILE; c0 += 16) {
                        uint32_t o[16];
                        tmem_ld16(orow + c0, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st16(orow + c0, o);
                    }
                }
                if (raise) m_ref = mt;
            }
            // probabilities (at most 2^8), rounded to fp16, packed two per column over the scores they came from
            const float m_use = m_ref == -INFINITY ? 0.f : m_ref;     // a row that has seen nothing yet: 2^(-inf) = 0
            probs_chunk(r0, m_use, trow, l0, l1);
            probs_chunk(r1, m_use, trow + 16, l0, l1);
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.p_half[b]);
            probs_chunk(r2, m_use, trow + 32, l0, l1);
            probs_chunk(r3, m_use, trow + 48, l0, l1);
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.p_ready[b]);
        }
        if (n_tiles > 0 && ok) {
            if (!mbar_wait(&sm.o_done, 0)) ok = false;
        }
        if (ok) {
            tc_fence_after_sync();
            const bool has_out = t0 + tt < p.T;                // (rows past the chunk still take part in the warp-wide loads)
            const float l = l0 + l1;
            const float inv = l > 0.f ? 1.f / l : 0.f;
            // a NaN means non-finite numbers in the cache, the factors or the query (or a key beyond the fp16 range)
            if (has_out && l != l) lorc_set_status(p.status, LORC_ERR_ARG);
            if (has_out && !(l > 0.f) && l == l && hi == 0 && g == 0 && t0 + tt == 0) lorc_set_status(p.status, LORC_ERR_EMPTY);
            bf16* dst = p.out + (((long long)s * p.T + (has_out ? t0 + tt : 0)) * p.H_q + g * p.G + hi) * 128;
#pragma unroll
            for (int c0 = 0; c0 < TILE; c0 += 32) {
                uint32_t o[32];
                if (n_tiles > 0) {
                    tmem_ld32(orow + c0, o);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = 0u;
                }
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(o[v * 8 + 2 * e]) * inv,
                                                                        __uint_as_float(o[v * 8 + 2 * e + 1]) * inv);
                        w[e] = *reinterpret_cast<const uint32_t*>(&b2);
                    }
                    if (has_out) reinterpret_cast<uint4*>(dst + c0)[v] = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
// scratch: [K^ | V], rows of the key / value buffers rounded up to whole tiles
static size_t prefill_rows(int max_seq_len) { return (size_t)((max_seq_len + TILE - 1) / TILE) * TILE; }

size_t lorc_tc_prefill_scratch_bytes(const lorc_ctx* ctx, int batch, int max_seq_len, int T) {
    (void)T;
    const size_t kv = lorc_align_up((size_t)batch * prefill_rows(max_seq_len) * ctx->n * sizeof(bf16), 256);
    return 2 * kv;
}

cudaError_t lorc_tc_prefill_set_attrs() {
    cudaError_t e = cudaFuncSetAttribute(lorc_reconstruct_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)sizeof(RecSmem) + 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(lorc_reconstruct_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)sizeof(RecSmem) + 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(lorc_prefill_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)sizeof(FaSmem) + 1024);
    return e;
}

cudaError_t lorc_tc_prefill_launch(lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, const CUtensorMap& mapCK,
                                   const CUtensorMap& mapCV, const CUtensorMap& mapBKT, const CUtensorMap& mapBVT128,
                                   const bf16* q, bf16* out, int T, void* scratch, cudaStream_t st, int* launches) {
    const lorc_model_desc& d = ctx->desc;
    const size_t rows = prefill_rows(cv.max_seq_len);
    const size_t kv_bytes = lorc_align_up((size_t)cv.batch * rows * ctx->n * sizeof(bf16), 256);
    bf16* khat = (bf16*)scratch;
    bf16* vbuf = (bf16*)((char*)scratch + kv_bytes);
    const int tiles = (int)(rows / TILE);
    cudaError_t e;

    RecParams rp;
    rp.seq_lens = cv.seq_lens; rp.page_table = cv.page_table; rp.rope_table = ctx->rope_table; rp.status = ctx->status_dev;
    rp.n = ctx->n; rp.n_rows = (int)rows; rp.max_pos = d.max_pos;
    rp.page_size = cv.page_size; rp.max_pages_per_seq = cv.max_pages_per_seq; rp.n_pages = cv.n_pages;
    rp.batch = cv.batch; rp.tile_pairs = (tiles + 1) / 2; rp.n_hp = d.n_kv_heads / 2;
    const int units = cv.batch * rp.tile_pairs * rp.n_hp;
    const int pairs = units < ctx->sm_count / 2 ? units : ctx->sm_count / 2;
    dim3 rgrid(2 * pairs);
    rp.out = khat; rp.r = L.r_k;
    lorc_reconstruct_kernel<true><<<rgrid, R_THREADS, sizeof(RecSmem) + 1024, st>>>(mapCK, mapBKT, rp);
    *launches += 1;
    rp.out = vbuf; rp.r = L.r_v;
    lorc_reconstruct_kernel<false><<<rgrid, R_THREADS, sizeof(RecSmem) + 1024, st>>>(mapCV, mapBVT128, rp);
    *launches += 1;
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;

    CUtensorMap mapQ, mapK, mapV;
    {
        // q [b, T, H_q, 128]: box = 64 elements x G heads x 128 / G positions
        uint64_t dims[4] = {128, (uint64_t)d.n_q_heads, (uint64_t)T, (uint64_t)cv.batch};
        uint64_t str[3] = {128 * 2, (uint64_t)d.n_q_heads * 128 * 2, (uint64_t)T * d.n_q_heads * 128 * 2};
        uint32_t box[4] = {KC, (uint32_t)ctx->group, (uint32_t)(TILE / ctx->group), 1};
        if (!lorc_make_tmap_bf16(&mapQ, q, 4, dims, str, box)) return cudaErrorInvalidValue;
        uint64_t kd[3] = {(uint64_t)ctx->n, (uint64_t)rows, (uint64_t)cv.batch};
        uint64_t ks[2] = {(uint64_t)ctx->n * 2, (uint64_t)rows * ctx->n * 2};
        uint32_t kb[3] = {KC, TILE, 1};
        if (!lorc_make_tmap_bf16(&mapK, khat, 3, kd, ks, kb)) return cudaErrorInvalidValue;
        if (!lorc_make_tmap_bf16(&mapV, vbuf, 3, kd, ks, kb)) return cudaErrorInvalidValue;
    }
    FaParams fp;
    fp.out = out; fp.seq_lens = cv.seq_lens; fp.rope_table = ctx->rope_table; fp.status = ctx->status_dev;
    fp.T = T; fp.H_q = d.n_q_heads; fp.G = ctx->group; fp.n_rows = (int)rows; fp.max_pos = d.max_pos;
    const int qp = 2 * TILE / ctx->group;                      // query positions per CTA (two blocks of 128 rows)
    dim3 fgrid((T + qp - 1) / qp, d.n_kv_heads, cv.batch);
    lorc_prefill_attn_kernel<<<fgrid, F_THREADS, sizeof(FaSmem) + 1024, st>>>(mapQ, mapK, mapV, fp);
    *launches += 1;
    return cudaGetLastError();
}
