// Score kernel of the tensor-core decode path (sm_100a: TMA + tcgen05 + TMEM).
//
// Persistent CTA PAIRS (clusters of two, cta_group::2 MMAs) walk units.  The 128-token tiles of all sequences of the
// batch form one flat list; a unit is two consecutive tiles of that list (one per CTA of the pair, possibly of
// different sequences) and one pair of KV heads.  Per unit
//   1. key reconstruction   K[256 tokens, 256] = C_K[tiles, :] . B_K[:, head pair]       (fp32 in both CTAs' TMEM)
//      from TMA-staged 64-wide slices of the latent tiles and of B_K^T (each CTA holds its own 128 tokens and half
//      of the B_K^T slice, which halves the shared-memory fill per FLOP);
//   2. eight epilogue warps per CTA (thread = token row) read the accumulator, rotate every key at its position and
//      dot it with the G rotated queries of its KV head.  RoPE is split as R(n0 + t) = R(n0) R(t): R(t), t < 128, is a
//      constant table in shared memory and R(n0) is folded into the query (q' = R(m - n0) q), which a warp of its own
//      prepares one unit ahead;
//   3. softmax numerators.  Every warp holds the scores of 32 tokens x G heads.  It takes their maximum, rounds it up
//      to an integer m (log2 units) and writes p = bf16(2^(s - m)) straight into the 128-byte-swizzled tile image the
//      PV kernel's MMA reads, together with m and the sum of the rounded p.  Because m is an integer, changing the
//      reference later (to the maximum over the whole sequence) only shifts exponents: the PV kernel does that exactly,
//      so the result equals a softmax with the exact row maximum, and no fp32 score ever goes to memory.
// Keys never exist in memory; per token the kernel writes 2*H_q bytes of probabilities.
#include <math.h>

#include "sm100_pair.cuh"
#include "sm100_ptx.cuh"
#include "tc_kernels.cuh"

using namespace sm100;

namespace {

constexpr int TILE = 128;            // tokens per tile
constexpr int KC = 64;               // latent columns per pipeline stage
constexpr float LOG2E = 1.4426950408889634f;

constexpr int Q_STAGES = 6;
constexpr int Q_THREADS = 352;       // warp 0 TMA, warp 1 MMA, warps 2..9 epilogue, warp 10 query
constexpr int Q_EPI_WARPS = 8;

struct ScoreSmem {
    bf16 A[Q_STAGES][TILE * KC];          // latent slice  [128 tokens][64]                                   16 KiB
    bf16 B[Q_STAGES][128 * KC];           // this CTA's half of the B_K^T slice [128 features][64]            16 KiB
    float4 trig[33][32];                  // in-tile rotation table, see rope_tile_kernel                     16.5 KiB
    float qrot[2][2][1024];               // [buffer][head of pair][rotated, scaled query; see qrot_index]    16 KiB
    uint64_t full[Q_STAGES], empty[Q_STAGES], acc_full[2], acc_empty[2], q_full[2], q_empty[2], trig_full;
    uint32_t tmem_base;
    int32_t tile_start[LORC_SCORE_MAX_BATCH + 1];   // first flat tile of every sequence
    int32_t lens[LORC_SCORE_MAX_BATCH];             // checked sequence lengths (0: nothing to do)
    int32_t qrel[LORC_SCORE_MAX_BATCH];             // query position relative to the first cached row
};

struct ScoreParams {
    const bf16* q;                 // [b, H_q, 128]          (already offset to the first sequence of this launch)
    uint8_t* pimg;                 // [b, tiles, image]      probability tile images, see lorc_tc_image_bytes
    unsigned* rowmax;              // [b, H_q]  running row maximum (an integer, as an order-preserving key; 0: none yet)
    const int32_t* seq_lens;
    const int32_t* pos0;           // NULL, or per sequence the position of the first cached row and the position of the
    const int32_t* q_pos;          // query (context shards: the rows of this cache start at some later position than 0)
    const int32_t* page_table;     // NULL: contiguous
    const float2* rope_table;      // [max_pos][64]
    const float4* rope_tile;       // [33][32]   in-tile rotation table in its shared-memory layout
    int* zero;                     // words the first block clears for the kernels that follow
    int* status;
    int batch, seq0, H_q, n_hp, r_k, tiles, n_zero, max_pos;
    int page_size, max_pages_per_seq, n_pages;
};

struct Unit {
    int s, tile, len, hp;
    bool valid;           // false: the flat list ended before this CTA's tile (the pair still needs finite operands)
};

// Walk over the units u = first, first + stride, ... of a CTA pair, u = fp * n_hp + hp (fp: pair of flat tiles),
// by additions with carry; `s` follows the flat tile index, which never decreases.
struct Walk {
    int u, fp, hp, s;
    int d_fp, d_hp, stride, n_hp;
    __device__ __forceinline__ Walk(int first, int stride_, int n_hp_) {
        stride = stride_; n_hp = n_hp_;
        u = first; hp = first % n_hp; fp = first / n_hp;
        d_hp = stride % n_hp; d_fp = stride / n_hp;
        s = 0;
    }
    __device__ __forceinline__ void next() {
        u += stride;
        hp += d_hp;
        const int carry = hp >= n_hp;
        hp -= carry ? n_hp : 0;
        fp += d_fp + carry;
    }
};

__device__ __forceinline__ void decode_unit(const ScoreSmem& sm, Walk& w, int rank, int n_flat, int batch, Unit& un) {
    int f = 2 * w.fp + rank;
    un.valid = f < n_flat;
    if (!un.valid) f = n_flat - 1;
    while (w.s + 1 < batch && f >= sm.tile_start[w.s + 1]) ++w.s;
    un.s = w.s;
    un.tile = f - sm.tile_start[w.s];
    un.len = sm.lens[w.s];
    un.hp = w.hp;
}

// Epilogue work split.  A warp reads its 32 accumulator lanes (tokens) with 16-lane x 256-bit loads, so lane
// (r = lane / 4, c = lane % 4) holds, per 32-column chunk jc, the tokens r + 8m (m = 0..3) and the rotary pairs
// j = 32 jc + 8k + 2c + e (k = 0..3, e = 0..1): four tokens share every query operand the thread loads, and the four
// lanes of equal r add their partial dots at the end.
//
// Float index of query head g, pair j, component `half` (0: first half of the head, 1: second) in qrot[][].  One
// 16-byte piece holds two heads x the thread's two adjacent pairs (e = j & 1), i.e. two packed-fp32 operands; the four
// c of equal (kk, half, g / 2) are neighbouring pieces, one conflict-free shared-memory access.
// 2^x for x <= 0 on the special-function unit (relative error 2^-22; the result is rounded to bf16 anyway).
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int G>
__device__ __forceinline__ int qrot_index(int j, int half, int g) {
    const int kk = j >> 3, c = (j >> 1) & 3, e = j & 1;
    return ((((kk * 2 + half) * (G / 2) + (g >> 1)) * 4 + c) << 2) + ((g & 1) << 1) + e;
}

template <int G>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(Q_THREADS, 1)
lorc_score_kernel(const __grid_constant__ CUtensorMap mapCK, const __grid_constant__ CUtensorMap mapBKT,
                  const ScoreParams p) {
    extern __shared__ uint8_t raw[];
    ScoreSmem& sm = *reinterpret_cast<ScoreSmem*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int rank = (int)cluster_ctarank();           // 0 = leader (issues the MMAs, owns the full / acc_empty barriers)
    const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int nkc = (p.r_k + KC - 1) / KC;
    const int img_bytes = lorc_tc_image_bytes(p.H_q);

    if (tid == 0) {
        for (int i = 0; i < Q_STAGES; ++i) {
            mbar_init(&sm.full[i], 1);
            mbar_init(&sm.empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sm.acc_full[i], 1);
            mbar_init(&sm.acc_empty[i], 2 * Q_EPI_WARPS);        // one arrival per epilogue warp, both CTAs
            mbar_init(&sm.q_full[i], 1);
            mbar_init(&sm.q_empty[i], Q_EPI_WARPS);
        }
        mbar_init(&sm.trig_full, 1);
        fence_barrier_init();
        prefetch_tensormap(&mapCK);
        prefetch_tensormap(&mapBKT);
        // constant in-tile rotation table: does not depend on earlier work in the stream
        mbar_arrive_expect_tx(&sm.trig_full, (uint32_t)sizeof(sm.trig));
        bulk_load(&sm.trig[0][0], p.rope_tile, (uint32_t)sizeof(sm.trig), &sm.trig_full);
    }
    // Everything above may overlap the tail of the previous kernel in the stream; inputs are read, results written
    // and tensor memory claimed only once that kernel has completed.
    grid_dep_wait();
    if (blockIdx.x == 0)
        for (int i = tid; i < p.n_zero; i += Q_THREADS) p.zero[i] = 0;
    for (int i = tid; i < p.batch; i += Q_THREADS) {
        int len = p.seq_lens[i];
        if (len > p.max_pos || len > p.tiles * TILE) {   // beyond what the tables or the scratch were sized for
            lorc_set_status(p.status, LORC_ERR_CAPACITY);
            len = 0;
        }
        int qr = p.q_pos ? p.q_pos[i] - p.pos0[i] : len - 1;
        if (qr < len - 1 || qr >= p.max_pos || (p.q_pos && (p.pos0[i] < 0 || p.q_pos[i] >= p.max_pos))) {
            // the query may not precede a cached key, nor leave the tables
            lorc_set_status(p.status, LORC_ERR_CAPACITY);
            len = 0;
        }
        sm.lens[i] = len > 0 ? len : 0;
        sm.qrel[i] = qr;
    }
    if (warp == 1) {
        tmem_alloc_pair(&sm.tmem_base, 512);
        tmem_relinquish_pair();
    }
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        for (int i = 0; i < p.batch; ++i) {
            sm.tile_start[i] = acc;
            acc += (sm.lens[i] + TILE - 1) / TILE;
        }
        sm.tile_start[p.batch] = acc;
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_arrive_release();                            // the peer's barriers are initialised before anyone signals them
    cluster_wait_acquire();
    tc_fence_after_sync();
    grid_dep_launch();
    const uint32_t tmem = sm.tmem_base;
    const int n_flat = sm.tile_start[p.batch];
    const int total_units = ((n_flat + 1) >> 1) * p.n_hp;

    // The two single-thread loops below share their schedulers with epilogue warps that keep them busy, so they are
    // written to need few issue slots per stage: stage index and phase advance incrementally, shared-memory
    // addresses and descriptor words are base + stage * constant.
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        // (whole warp in the loop, one elected lane issues: the asynchronous instructions take their operands from
        // uniform registers, which the compiler only uses in warp-uniform code)
        const uint32_t a_base = smem_u32(sm.A[0]), b_base = smem_u32(sm.B[0]);
        const uint32_t empty0 = smem_u32(&sm.empty[0]), full0 = smem_u32(&sm.full[0]);
        const uint32_t lead_full0 = mapa_shared(full0, 0);   // all bytes of a stage are counted on the leader's barrier
        const bool paged = p.page_table != nullptr;
        const int b_row = rank * 128;
        uint32_t st = 0, par = 1;                            // stage and the parity its empty barrier is waited with
        bool ok = true;
        for (Walk w(pair_id, n_pairs, p.n_hp); w.u < total_units && ok; w.next()) {
            Unit un;
            decode_unit(sm, w, rank, n_flat, p.batch, un);
            const int row0 = un.tile * TILE, brow = un.hp * 256 + b_row, sg = p.seq0 + un.s;
            for (int x = 0; x < nkc * KC; x += KC) {
                if (!mbar_wait_addr(empty0 + st * 8, par)) { ok = false; break; }
                const uint32_t lead_bar = lead_full0 + st * 8;
                const uint32_t a_dst = a_base + st * (TILE * KC * 2);
                if (elect_one()) {
                    if (rank == 0) mbar_arrive_expect_tx_addr(full0 + st * 8, 2 * 2 * TILE * KC * 2);
                    if (!paged) {
                        tma_load_3d_pair_addr(a_dst, &mapCK, lead_bar, x, row0, sg);
                    } else {
                        // one box per page; pages past the end of the sequence (or with a bad table entry) are
                        // read from page 0: those rows are masked, but every box must deliver its bytes
                        const int ppt = TILE / p.page_size;
                        for (int pg = 0; pg < ppt; ++pg) {
                            const int lp = un.tile * ppt + pg;
                            int page = 0;
                            if ((long long)lp * p.page_size < un.len && lp < p.max_pages_per_seq) {
                                page = p.page_table[(long long)sg * p.max_pages_per_seq + lp];
                                if (page < 0 || page >= p.n_pages) {
                                    lorc_set_status(p.status, LORC_ERR_CAPACITY);
                                    page = 0;
                                }
                            }
                            tma_load_3d_pair_addr(a_dst + pg * p.page_size * KC * 2, &mapCK, lead_bar, x, 0, page);
                        }
                    }
                    tma_load_2d_pair_addr(b_base + st * (128 * KC * 2), &mapBKT, lead_bar, x, brow);
                }
                __syncwarp();
                if (++st == Q_STAGES) { st = 0; par ^= 1; }
            }
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        // The whole warp walks the loop (so the compiler can keep addresses and descriptor words in uniform
        // registers, which is what the MMA instruction takes); one elected lane issues.
        if (rank == 0) {
            const uint32_t idesc = make_idesc_bf16(256, 256, 0, 0);
            const int nk_last = (p.r_k - (nkc - 1) * KC + 15) >> 4;   // 16-column steps the last stage really holds
            // descriptor words of stage 0, k-step 0; a stage adds its byte offset >> 4 to the low word, a k-step
            // (16 columns = 32 bytes inside the 128-byte swizzle row) adds 2
            const uint64_t da0 = make_smem_desc_sw128(smem_u32(sm.A[0]), 0, 1024);
            const uint64_t db0 = make_smem_desc_sw128(smem_u32(sm.B[0]), 0, 1024);
            const uint32_t a_lo0 = (uint32_t)da0, a_hi = (uint32_t)(da0 >> 32);
            const uint32_t b_lo0 = (uint32_t)db0, b_hi = (uint32_t)(db0 >> 32);
            const uint32_t empty0 = smem_u32(&sm.empty[0]), full0 = smem_u32(&sm.full[0]);
            uint32_t st = 0, par = 0, uc = 0;
            bool ok = true;
            for (int u = pair_id; u < total_units && ok; u += n_pairs) {
                const int buf = uc & 1;
                if (!mbar_wait(&sm.acc_empty[buf], ((uc >> 1) & 1) ^ 1)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d = tmem + buf * 256;
                for (int kc = 0; kc < nkc; ++kc) {
                    if (!mbar_wait_addr(full0 + st * 8, par)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t a_lo = a_lo0 + st * (TILE * KC * 2 / 16), b_lo = b_lo0 + st * (128 * KC * 2 / 16);
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
                    if (++st == Q_STAGES) { st = 0; par ^= 1; }
                }
                if (!ok) break;
                if (elect_one()) tc_commit_pair(&sm.acc_full[buf]);   // both CTAs' epilogues may read their accumulators
                __syncwarp();
                ++uc;
            }
            if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
        }
    } else if (warp == 10) {
        // ------------------------------------------------------------------ query of the unit, one unit ahead (both CTAs)
        // Lane l owns the rotary pairs j = 2 l, 2 l + 1 of the 2 G query heads of the unit's two KV heads:
        // q' = R(m - n0) q / sqrt(d_h) * log2(e), m the query's position, n0 the first token of this CTA's tile.
        const float scale = rsqrtf(128.f) * LOG2E;
        uint32_t uc = 0;
        bool ok = true;
        for (Walk w(pair_id, n_pairs, p.n_hp); w.u < total_units && ok; w.next(), ++uc) {
            Unit un;
            decode_unit(sm, w, rank, n_flat, p.batch, un);
            const int buf = uc & 1;
            const int delta = max(sm.qrel[un.s] - un.tile * TILE, 0);
            const float4 cs = __ldg(reinterpret_cast<const float4*>(p.rope_table + (long long)delta * 64) + lane);
            uint32_t qa[2 * G], qb[2 * G];
#pragma unroll
            for (int i = 0; i < 2 * G; ++i) {
                const int h = un.hp * 2 * G + i;
                const uint32_t* qp = reinterpret_cast<const uint32_t*>(p.q + ((long long)un.s * p.H_q + h) * 128);
                qa[i] = __ldg(qp + lane);
                qb[i] = __ldg(qp + 32 + lane);
            }
            // the epilogue warps are done with the unit that used this buffer before
            if (!mbar_wait(&sm.q_empty[buf], ((uc >> 1) & 1) ^ 1)) { ok = false; break; }
#pragma unroll
            for (int i = 0; i < 2 * G; ++i) {
                const int hd = i / G, g = i % G;
                const float a0 = __uint_as_float(qa[i] << 16), a1 = __uint_as_float(qa[i] & 0xffff0000u);
                const float b0 = __uint_as_float(qb[i] << 16), b1 = __uint_as_float(qb[i] & 0xffff0000u);
                float* dst = sm.qrot[buf][hd];
                // pairs 2 l and 2 l + 1 are neighbours in the layout (e = 0, 1): one 8-byte store per half
                *reinterpret_cast<float2*>(dst + qrot_index<G>(2 * lane, 0, g)) =
                    make_float2((a0 * cs.x - b0 * cs.y) * scale, (a1 * cs.z - b1 * cs.w) * scale);
                *reinterpret_cast<float2*>(dst + qrot_index<G>(2 * lane, 1, g)) =
                    make_float2((a0 * cs.y + b0 * cs.x) * scale, (a1 * cs.w + b1 * cs.z) * scale);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.q_full[buf]);
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    } else {
        // ------------------------------------------------------------------ epilogue: RoPE, scores, softmax numerators
        const int te = tid - 64;                  // 0..255
        const int grp = te / 128;                 // which head of the pair
        const int quarter = warp % 4;             // TMEM lane quarter this warp may read
        const int r = lane >> 2, c = lane & 3;
        uint32_t uc = 0;
        bool ok = mbar_wait(&sm.trig_full, 0);
        const uint32_t lead_acc_empty[2] = {mapa_shared(smem_u32(&sm.acc_empty[0]), 0),
                                            mapa_shared(smem_u32(&sm.acc_empty[1]), 0)};
        const ulonglong2* tr2 = reinterpret_cast<const ulonglong2*>(&sm.trig[quarter * 8 + r][0]);  // first token
        const ulonglong2* tw2 = reinterpret_cast<const ulonglong2*>(&sm.trig[32][0]) + c;           // 8-position step
        const int tswz = (r & 1) << 2;                      // odd rows of the table swap 64-byte halves
        const uint64_t minus1 = f2_pack(-1.f, -1.f);
        for (Walk w(pair_id, n_pairs, p.n_hp); w.u < total_units && ok; w.next(), ++uc) {
            Unit un;
            decode_unit(sm, w, rank, n_flat, p.batch, un);
            const int buf = uc & 1;
            if (!mbar_wait(&sm.q_full[buf], (uc >> 1) & 1)) { ok = false; break; }
            if (!mbar_wait(&sm.acc_full[buf], (uc >> 1) & 1)) { ok = false; break; }
            tc_fence_after_sync();
            // Packed fp32: every operation below acts on the thread's two adjacent rotary pairs (columns 2c, 2c + 1
            // of the 8-column step) at once, which halves the instructions the epilogue issues.  acc2[m][g] holds the
            // partial dots of the even and the odd pairs; they are added at the end.
            uint64_t acc2[4][G];
#pragma unroll
            for (int m = 0; m < 4; ++m)
#pragma unroll
                for (int g = 0; g < G; ++g) acc2[m][g] = 0ull;
            const uint32_t tbase = tmem + ((uint32_t)(quarter * 32) << 16) + buf * 256 + grp * 128;
            const ulonglong2* q2 = reinterpret_cast<const ulonglong2*>(sm.qrot[buf][grp]) + c;
            // One 8-column step at a time.  Unrolled, so that the loads and the dependent fp32 chains of several steps
            // overlap (a scheduler has only two epilogue warps to switch between).
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                uint32_t ra[2][4], rb[2][4];
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    tmem_ld16x256_x1(tbase + ((uint32_t)(hf * 16) << 16) + kk * 8, ra[hf]);
                    tmem_ld16x256_x1(tbase + ((uint32_t)(hf * 16) << 16) + 64 + kk * 8, rb[hf]);
                }
                // (cos, -sin) of this thread's first token for its two rotary pairs, and (cos, sin) of the 8-position
                // step that leads to its other three tokens (r + 8, r + 16, r + 24): angle addition instead of a table
                // row per token
                const ulonglong2 t0 = tr2[(kk * 4 + c) ^ tswz];
                const ulonglong2 tw = tw2[kk * 4];
                uint64_t cs = t0.x, ns = t0.y;                 // (cos_e0, cos_e1), (-sin_e0, -sin_e1)
                const uint64_t wc = tw.x, ws = tw.y, nws = f2_mul(tw.y, minus1);
                uint64_t qa[G], qbv[G];
#pragma unroll
                for (int gp = 0; gp < G / 2; ++gp) {
                    const ulonglong2 x = q2[((kk * 2 + 0) * (G / 2) + gp) * 4];
                    const ulonglong2 y = q2[((kk * 2 + 1) * (G / 2) + gp) * 4];
                    qa[2 * gp] = x.x; qa[2 * gp + 1] = x.y;
                    qbv[2 * gp] = y.x; qbv[2 * gp + 1] = y.y;
                }
                tmem_wait_ld();
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    const uint64_t a = f2_pack(__uint_as_float(ra[m >> 1][2 * (m & 1)]), __uint_as_float(ra[m >> 1][2 * (m & 1) + 1]));
                    const uint64_t b = f2_pack(__uint_as_float(rb[m >> 1][2 * (m & 1)]), __uint_as_float(rb[m >> 1][2 * (m & 1) + 1]));
                    const uint64_t na = f2_mul(a, minus1);
                    const uint64_t ka = f2_fma(b, ns, f2_mul(a, cs));       // a cos - b sin
                    const uint64_t kb = f2_fma(b, cs, f2_mul(na, ns));      // a sin + b cos
#pragma unroll
                    for (int g = 0; g < G; ++g) acc2[m][g] = f2_fma(qbv[g], kb, f2_fma(qa[g], ka, acc2[m][g]));
                    if (m < 3) {
                        const uint64_t nc = f2_fma(ns, ws, f2_mul(cs, wc));   // cos cos' - sin sin'
                        ns = f2_fma(ns, wc, f2_mul(cs, nws));                 // -(cos sin' + sin cos')
                        cs = nc;
                    }
                }
            }
            float acc[4][G];
#pragma unroll
            for (int m = 0; m < 4; ++m)
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    float x, y;
                    f2_unpack(acc2[m][g], x, y);
                    acc[m][g] = x + y;
                }
            // one arrival per warp: every lane has its accumulator values in registers (tmem_wait_ld above) and has
            // read its query operands
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive_cluster(lead_acc_empty[buf]);
                mbar_arrive(&sm.q_empty[buf]);
            }
            // add the four lanes' partial dots; lane c ends with the heads g = 4i + c
            float tot[4][G / 4];
#pragma unroll
            for (int m = 0; m < 4; ++m) {
                float h1[G / 2];
#pragma unroll
                for (int i = 0; i < G / 2; ++i) {
                    const float keep = (c & 1) ? acc[m][2 * i + 1] : acc[m][2 * i];
                    const float send = (c & 1) ? acc[m][2 * i] : acc[m][2 * i + 1];
                    h1[i] = keep + __shfl_xor_sync(0xffffffffu, send, 1);
                }
#pragma unroll
                for (int i = 0; i < G / 4; ++i) {
                    const float keep = (c & 2) ? h1[2 * i + 1] : h1[2 * i];
                    const float send = (c & 2) ? h1[2 * i] : h1[2 * i + 1];
                    tot[m][i] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
                }
            }
            if (!un.valid) continue;
            // softmax numerators of this warp's 32 tokens (a quarter of the tile) against their own integer reference
            uint8_t* img = p.pimg + ((long long)un.s * p.tiles + un.tile) * img_bytes;
            uint8_t* chunk_img = img + (quarter >> 1) * (p.H_q * KC * 2);
            float* m_out = reinterpret_cast<float*>(img + 2 * p.H_q * KC * 2) + quarter * p.H_q;
            float* l_out = m_out + 4 * p.H_q;
            const int n_first = un.tile * TILE + quarter * 32 + r;
            const int tc0 = (quarter & 1) * 32 + r;
#pragma unroll
            for (int i = 0; i < G / 4; ++i) {
                const int h = (un.hp * 2 + grp) * G + 4 * i + c;
                float mxv = -INFINITY, ssum = 0.f;
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    ssum += tot[m][i];
                    if (n_first + 8 * m < un.len) mxv = fmaxf(mxv, tot[m][i]);
                }
                // a NaN among the scores means non-finite numbers in the cache, the factors or the query
                if (ssum != ssum) lorc_set_status(p.status, LORC_ERR_ARG);
#pragma unroll
                for (int o = 4; o < 32; o <<= 1) mxv = fmaxf(mxv, __shfl_xor_sync(0xffffffffu, mxv, o));
                const float mref = ceilf(mxv);                 // -inf: no token of the sequence in this quarter
                float lsum = 0.f;
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    const bool valid = n_first + 8 * m < un.len;
                    // p = 2^(s - m), rounded to bf16 (the same rounded value enters the denominator)
                    const bf16 pr = __float2bfloat16_rn(valid ? ex2_approx(tot[m][i] - mref) : 0.f);
                    lsum += __bfloat162float(pr);
                    const int tc = tc0 + 8 * m;
                    *reinterpret_cast<bf16*>(chunk_img + h * 128 + ((((tc >> 3) ^ (h & 7)) << 4) | ((tc & 7) << 1))) = pr;
                }
#pragma unroll
                for (int o = 4; o < 32; o <<= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
                if (r == 0) {
                    m_out[h] = mref;
                    l_out[h] = lsum;
                    if (mxv > -INFINITY) atomicMax(p.rowmax + (long long)un.s * p.H_q + h, lorc_float_key(mref));
                }
            }
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

// Constant in-tile rotation table in the layout the score kernel keeps in shared memory: 33 rows of 32 pieces of
// 16 bytes.  Row 8 q + r (q < 4, r < 8) holds (cos, sin)(t theta_j) for the token t = 32 q + r, piece
// (j / 2) ^ (4 (r & 1)) = (cos_j, cos_j+1, -sin_j, -sin_j+1) for even j (the swap of 64-byte halves on odd rows spreads
// the epilogue's accesses over all banks); row 32 holds the same for a step of 8 positions, unswizzled.  The other
// tokens of a tile follow by angle addition: t + 8 m.
__global__ void rope_tile_kernel(float2* out, double theta) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 33 * 64) return;
    int row = i / 64, j = i % 64;
    const int t = row < 32 ? (row >> 3) * 32 + (row & 7) : 8;
    const int swz = row < 32 ? (row & 1) << 2 : 0;
    double inv = pow(theta, -(double)j / 64.0);
    double sn, cs;
    sincos((double)t * inv, &sn, &cs);
    // piece = (cos_j, cos_j+1, -sin_j, -sin_j+1) in the token rows, (cos, cos, +sin, +sin) in the step row
    float* piece = reinterpret_cast<float*>(out) + (row * 32 + ((j >> 1) ^ swz)) * 4;
    piece[j & 1] = (float)cs;
    piece[2 + (j & 1)] = row < 32 ? -(float)sn : (float)sn;
}

}  // namespace

cudaError_t lorc_tc_score_set_attrs() {
    cudaError_t e = cudaFuncSetAttribute(lorc_score_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)sizeof(ScoreSmem) + 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(lorc_score_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)sizeof(ScoreSmem) + 1024);
    return e;
}

cudaError_t lorc_tc_rope_tile_fill(float2* table, double theta, cudaStream_t st) {
    rope_tile_kernel<<<(64 * 33 + 255) / 256, 256, 0, st>>>(table, theta);
    return cudaGetLastError();
}

// One launch per block of LORC_SCORE_MAX_BATCH sequences (the kernel keeps the block's lengths and tile offsets in
// shared memory).  The first launch clears `zero[0 .. n_zero)` for the kernels that follow it in the stream.
cudaError_t lorc_tc_score_launch(lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, const CUtensorMap& mapCK,
                                 const CUtensorMap& mapBKT, const bf16* q, uint8_t* pimg, unsigned* rowmax,
                                 const float4* rope_tile, int tiles, int* zero, int n_zero, const int32_t* pos0,
                                 const int32_t* q_pos, cudaStream_t st, int* launches) {
    const lorc_model_desc& d = ctx->desc;
    const size_t img_bytes = (size_t)lorc_tc_image_bytes(d.n_q_heads);
    for (int s0 = 0; s0 < cv.batch; s0 += LORC_SCORE_MAX_BATCH) {
        const int nb = cv.batch - s0 < LORC_SCORE_MAX_BATCH ? cv.batch - s0 : LORC_SCORE_MAX_BATCH;
        ScoreParams sp;
        sp.q = q + (size_t)s0 * d.n_q_heads * 128;
        sp.pimg = pimg + (size_t)s0 * tiles * img_bytes;
        sp.rowmax = rowmax + (size_t)s0 * d.n_q_heads;
        sp.seq_lens = cv.seq_lens + s0;
        sp.pos0 = pos0 ? pos0 + s0 : nullptr;
        sp.q_pos = q_pos ? q_pos + s0 : nullptr;
        sp.page_table = cv.page_table;
        sp.rope_table = ctx->rope_table;
        sp.rope_tile = rope_tile;
        sp.zero = zero;
        sp.n_zero = s0 == 0 ? n_zero : 0;
        sp.status = ctx->status_dev;
        sp.batch = nb; sp.seq0 = s0; sp.H_q = d.n_q_heads; sp.n_hp = d.n_kv_heads / 2; sp.r_k = L.r_k;
        sp.tiles = tiles; sp.max_pos = d.max_pos;
        sp.page_size = cv.page_size; sp.max_pages_per_seq = cv.max_pages_per_seq; sp.n_pages = cv.n_pages;
        // units if every sequence were full: an upper bound that only caps the grid
        const long long max_units = ((long long)nb * tiles + 1) / 2 * sp.n_hp;
        int n_pairs = ctx->sm_count / 2;
        if (max_units < n_pairs) n_pairs = (int)max_units;
        if (n_pairs < 1) n_pairs = 1;
        const size_t smem = sizeof(ScoreSmem) + 1024;
        cudaError_t e;
        if (ctx->group == 4)
            e = lorc_launch_dependent(lorc_score_kernel<4>, dim3(2 * n_pairs), dim3(Q_THREADS), smem, st, mapCK, mapBKT, sp);
        else
            e = lorc_launch_dependent(lorc_score_kernel<8>, dim3(2 * n_pairs), dim3(Q_THREADS), smem, st, mapCK, mapBKT, sp);
        *launches += 1;
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}
