// Tensor-core decode attention over the latent cache (sm_100a: TMA + tcgen05 + TMEM).
//
// Two kernels per layer, followed by a small kernel that adds up the output pieces:
//
//  score kernel   persistent CTA PAIRS (clusters of two, cta_group::2 MMAs) walk (sequence, two consecutive
//                 128-token tiles, KV-head pair) units.  Per unit the key tiles of two KV heads are
//                 reconstructed on the tensor cores, each CTA holding its own 128 tokens and HALF of the
//                 B_K^T slice (the pair shares it, which halves the shared-memory traffic per FLOP),
//                     K[256 tokens, 256] = C_K[tiles, :] . B_K[:, pair]         (fp32 in both CTAs' TMEM),
//                 from TMA-staged 64-wide slices of the latent tile and of B_K^T.  Eight epilogue warps
//                 (thread = token row) read the accumulator, rotate each key at its position and dot it
//                 with the G rotated queries of its KV head; the scores (log2 units) go to scratch.
//                 RoPE is split as R(n0 + t) = R(n0) R(t): R(t), t < 128, is a constant table in shared
//                 memory and R(n0) is folded into the query once per unit (q' = R(m - n0) q).
//                 It also folds the maximum of every 32-token quarter tile into one word per (sequence, head)
//                 with an atomic maximum, so that the next kernel knows the exact row maximum of the softmax
//                 without a pass over the scores.
//  PV kernel      softmax + P.C_V + value up-projection, split by latent columns (tc_pv.cu).
//
// Keys and values never exist in memory; only the 4*H_q bytes of scores per token are written.
#include <math.h>

#include "sm100_pair.cuh"
#include "sm100_ptx.cuh"
#include "tc_kernels.cuh"

using namespace sm100;

namespace {

constexpr int TILE = 128;            // tokens per tile
constexpr int KC = 64;               // latent columns per pipeline stage
constexpr float LOG2E = 1.4426950408889634f;

// ------------------------------------------------------------------------------------------------
// score kernel
// ------------------------------------------------------------------------------------------------
constexpr int S_STAGES = 6;
constexpr int S_THREADS = 320;       // warp 0 TMA, warp 1 MMA, warps 2..9 epilogue
constexpr int S_EPI = 256;
constexpr int S_LENS = 96;

struct ScoreSmem {
    bf16 A[S_STAGES][TILE * KC];          // latent slice  [128 tokens][64]       16 KiB
    bf16 B[S_STAGES][128 * KC];           // this CTA's half of the B_K^T slice [128 features][64]   16 KiB
    float4 trig[33][32];                  // in-tile rotation table, see rope_tile_kernel                     16.5 KiB
    float qrot[2][2][1024];               // [buffer][head of pair][rotated, scaled query; see qrot_index]    16 KiB
    uint64_t full[S_STAGES], empty[S_STAGES], acc_full[2], acc_empty[2], trig_full;
    uint32_t tmem_base;
    int32_t lens[S_LENS];                 // sequence lengths of the first S_LENS sequences (the rest are read from global)
};

struct ScoreParams {
    const bf16* q;                 // [b, H_q, 128]
    float* scores;                 // [b, H_q, n_pad]
    unsigned* rowmax;              // [b, H_q]  running row maximum as an order-preserving key (0: none yet)
    const int32_t* seq_lens;
    const int32_t* page_table;     // NULL: contiguous
    const float2* rope_table;      // [max_pos][64]
    const float4* rope_tile;       // [33][32]   in-tile rotation table in its shared-memory layout
    int* status;
    int batch, H_q, n_hp, r_k, n_pad, tiles_per_seq, tile_pairs, max_pos;
    int page_size, max_pages_per_seq, n_pages;
};

struct Unit {
    int s, tile, hp, len;     // tile = this CTA's own 128-token tile of the pair's two
};

// Walk over the units u = first, first + stride, ... of a CTA pair, u = (s * tile_pairs + tp) * n_hp + hp, keeping
// (s, tp, hp) up to date by additions with carry: the divisions are done once per kernel, not once per unit (every
// role decodes every unit, and at low ranks the decode sat on the epilogue's critical path).
struct UnitWalk {
    int u, hp, tp, s;
    int d_hp, d_tp, d_s, stride, n_hp, tile_pairs;
    __device__ __forceinline__ UnitWalk(const ScoreParams& p, int first, int stride_) {
        stride = stride_; n_hp = p.n_hp; tile_pairs = p.tile_pairs;
        u = first;
        hp = first % n_hp;
        int r = first / n_hp;
        tp = r % tile_pairs;
        s = r / tile_pairs;
        d_hp = stride % n_hp;
        r = stride / n_hp;
        d_tp = r % tile_pairs;
        d_s = r / tile_pairs;
    }
    __device__ __forceinline__ void next() {
        u += stride;
        hp += d_hp;
        int carry = hp >= n_hp;
        hp -= carry ? n_hp : 0;
        tp += d_tp + carry;
        carry = tp >= tile_pairs;
        tp -= carry ? tile_pairs : 0;
        s += d_s + carry;
    }
};

// The unit the walk stands on: (sequence, tile pair, KV-head pair).  Valid when the pair's first tile starts inside
// the sequence; the second CTA's tile may lie past the end (its rows are then masked or not written at all).
__device__ __forceinline__ bool decode_unit(const ScoreParams& p, const int32_t* lens_sm, const UnitWalk& w, int rank,
                                            Unit& un) {
    un.hp = w.hp;
    un.s = w.s;
    un.tile = 2 * w.tp + rank;
    // a shared-memory copy spares every role a global round trip at each unit boundary
    un.len = un.s < S_LENS ? lens_sm[un.s] : p.seq_lens[un.s];
    return un.len > 0 && un.len <= p.max_pos && 2 * w.tp * TILE < un.len;
}

// Epilogue work split.  A warp reads its 32 accumulator lanes (tokens) with 16-lane x 256-bit loads, so lane
// (r = lane / 4, c = lane % 4) holds, per 32-column chunk jc, the tokens r + 8m (m = 0..3) and the rotary pairs
// j = 32 jc + 8k + 2c + e (k = 0..3, e = 0..1): four tokens share every query operand the thread loads, and the four
// lanes of equal r add their partial dots at the end.
//
// Float index of query head g, pair j, component `half` (0: first half of the head, 1: second) in qrot[][].  One
// 16-byte piece holds two heads x the thread's two adjacent pairs (e = j & 1), i.e. two packed-fp32 operands; the four
// c of equal (kk, half, g / 2) are neighbouring pieces, one conflict-free shared-memory access.
template <int G>
__device__ __forceinline__ int qrot_index(int j, int half, int g) {
    const int kk = j >> 3, c = (j >> 1) & 3, e = j & 1;
    return ((((kk * 2 + half) * (G / 2) + (g >> 1)) * 4 + c) << 2) + ((g & 1) << 1) + e;
}

template <int G>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(S_THREADS, 1)
lorc_score_kernel(const __grid_constant__ CUtensorMap mapCK, const __grid_constant__ CUtensorMap mapBKT,
                  const ScoreParams p) {
    extern __shared__ uint8_t raw[];
    ScoreSmem& sm = *reinterpret_cast<ScoreSmem*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int rank = (int)cluster_ctarank();           // 0 = leader (issues the MMAs, owns the full / acc_empty barriers)
    const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int total_units = p.batch * p.tile_pairs * p.n_hp;
    const int nkc = (p.r_k + KC - 1) / KC;

    if (tid == 0) {
        for (int i = 0; i < S_STAGES; ++i) {
            mbar_init(&sm.full[i], 1);
            mbar_init(&sm.empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sm.acc_full[i], 1);
            mbar_init(&sm.acc_empty[i], 2 * S_EPI / 32); // one arrival per epilogue warp, both CTAs
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
    for (int i = tid; i < S_LENS && i < p.batch; i += S_THREADS) sm.lens[i] = p.seq_lens[i];
    if (warp == 1) {
        tmem_alloc_pair(&sm.tmem_base, 512);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_arrive_release();                            // the peer's barriers are initialised before anyone signals them
    cluster_wait_acquire();
    tc_fence_after_sync();
    grid_dep_launch();
    const uint32_t tmem = sm.tmem_base;

    // The two single-thread loops below share their schedulers with epilogue warps that keep them busy, so they are
    // written to need few issue slots per stage: stage index and phase advance incrementally, shared-memory
    // addresses and descriptor words are base + stage * constant.
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        // (whole warp in the loop, one elected lane issues: see the MMA warp below)
        {
            const uint32_t a_base = smem_u32(sm.A[0]), b_base = smem_u32(sm.B[0]);
            const uint32_t empty0 = smem_u32(&sm.empty[0]), full0 = smem_u32(&sm.full[0]);
            const uint32_t lead_full0 = mapa_shared(full0, 0);   // all bytes of a stage are counted on the leader's barrier
            const bool paged = p.page_table != nullptr;
            const int b_row = rank * 128;
            uint32_t st = 0, par = 1;                            // stage and the parity its empty barrier is waited with
            bool ok = true;
            for (UnitWalk w(p, pair_id, n_pairs); w.u < total_units && ok; w.next()) {
                Unit un;
                if (!decode_unit(p, sm.lens, w, rank, un)) continue;
                const int row0 = un.tile * TILE, brow = un.hp * 256 + b_row;
                for (int x = 0; x < nkc * KC; x += KC) {
                    if (!mbar_wait_addr(empty0 + st * 8, par)) { ok = false; break; }
                    const uint32_t lead_bar = lead_full0 + st * 8;
                    const uint32_t a_dst = a_base + st * (TILE * KC * 2);
                    if (elect_one()) {
                        if (rank == 0) mbar_arrive_expect_tx_addr(full0 + st * 8, 2 * 2 * TILE * KC * 2);
                        if (!paged) {
                            tma_load_3d_pair_addr(a_dst, &mapCK, lead_bar, x, row0, un.s);
                        } else {
                            // one box per page; pages past the end of the sequence (or with a bad table entry) are
                            // read from page 0: those rows are masked, but every box must deliver its bytes
                            const int ppt = TILE / p.page_size;
                            for (int pg = 0; pg < ppt; ++pg) {
                                const int lp = un.tile * ppt + pg;
                                int page = 0;
                                if ((long long)lp * p.page_size < un.len && lp < p.max_pages_per_seq) {
                                    page = p.page_table[(long long)un.s * p.max_pages_per_seq + lp];
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
                    if (++st == S_STAGES) { st = 0; par ^= 1; }
                }
            }
            if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
        }
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
            for (UnitWalk w(p, pair_id, n_pairs); w.u < total_units && ok; w.next()) {
                Unit un;
                if (!decode_unit(p, sm.lens, w, rank, un)) continue;
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
                    if (++st == S_STAGES) { st = 0; par ^= 1; }
                }
                if (!ok) break;
                if (elect_one()) tc_commit_pair(&sm.acc_full[buf]);   // both CTAs' epilogues may read their accumulators
                __syncwarp();
                ++uc;
            }
            if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
        }
    } else {
        // ------------------------------------------------------------------ epilogue: RoPE + scores
        const int te = tid - 64;                  // 0..255
        const int grp = te / 128;                 // which head of the pair
        const int quarter = warp % 4;             // TMEM lane quarter this warp may read
        const int r = lane >> 2, c = lane & 3;
        const float scale = rsqrtf(128.f) * LOG2E;
        constexpr int QL = 2 * G * 64 / S_EPI;    // (head, pair) items of the query rotation per thread
        uint32_t uc = 0;
        bool ok = mbar_wait(&sm.trig_full, 0);
        const uint32_t lead_acc_empty[2] = {mapa_shared(smem_u32(&sm.acc_empty[0]), 0),
                                            mapa_shared(smem_u32(&sm.acc_empty[1]), 0)};
        // The query of the NEXT unit is fetched while this unit's accumulators are processed: the loads below are
        // only issued here (raw bits, volatile asm), nothing touches their results before the next unit's rotation.
        uint32_t q_a[QL], q_b[QL];
        float2 q_cs[QL];
        auto fetch_query = [&](const Unit& un) {
            // query position relative to the tile start (a tile wholly past the sequence is masked anyway)
            const int delta = max(un.len - 1 - un.tile * TILE, 0);
#pragma unroll
            for (int i = 0; i < QL; ++i) {
                const int idx = te + i * S_EPI;
                const int hh = idx >> 6, j = idx & 63;
                const int h = un.hp * 2 * G + hh;
                const bf16* qp = p.q + ((long long)un.s * p.H_q + h) * 128;
                const float2* cp = p.rope_table + (long long)delta * 64 + j;
                asm volatile("ld.global.nc.v2.f32 {%0, %1}, [%2];" : "=f"(q_cs[i].x), "=f"(q_cs[i].y) : "l"(cp));
                asm volatile("ld.global.nc.u16 %0, [%1];" : "=r"(q_a[i]) : "l"(qp + j));
                asm volatile("ld.global.nc.u16 %0, [%1];" : "=r"(q_b[i]) : "l"(qp + j + 64));
            }
        };
        Unit un;
        UnitWalk w(p, pair_id, n_pairs);
        while (w.u < total_units && !decode_unit(p, sm.lens, w, rank, un)) w.next();
        if (w.u < total_units) fetch_query(un);
        while (w.u < total_units && ok) {
            const int buf = uc & 1, qb = uc & 1;
            const int n0 = un.tile * TILE;
#pragma unroll
            for (int i = 0; i < QL; ++i) {
                const int idx = te + i * S_EPI;
                const int hh = idx >> 6, j = idx & 63;
                const int hip = hh / G, g = hh - hip * G;
                const float qa_ = __uint_as_float(q_a[i] << 16), qb_ = __uint_as_float(q_b[i] << 16);
                sm.qrot[qb][hip][qrot_index<G>(j, 0, g)] = (qa_ * q_cs[i].x - qb_ * q_cs[i].y) * scale;
                sm.qrot[qb][hip][qrot_index<G>(j, 1, g)] = (qa_ * q_cs[i].y + qb_ * q_cs[i].x) * scale;
            }
            __syncwarp();   // a named barrier counts a warp once only if the warp arrives converged
            asm volatile("bar.sync 1, 256;" ::: "memory");
            // next unit of this pair
            Unit un_next;
            w.next();
            while (w.u < total_units && !decode_unit(p, sm.lens, w, rank, un_next)) w.next();
            if (w.u < total_units) fetch_query(un_next);

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
            const ulonglong2* q2 = reinterpret_cast<const ulonglong2*>(sm.qrot[qb][grp]) + c;
            const ulonglong2* tr2 = reinterpret_cast<const ulonglong2*>(&sm.trig[quarter * 8 + r][0]);  // first token
            const ulonglong2* tw2 = reinterpret_cast<const ulonglong2*>(&sm.trig[32][0]) + c;           // 8-position step
            const int tswz = (r & 1) << 2;                      // odd rows of the table swap 64-byte halves
            const uint64_t minus1 = f2_pack(-1.f, -1.f);
            // One 8-column step at a time.  Unrolled, so that the loads and the dependent fp32 chains of several steps
            // overlap (a scheduler has only two epilogue warps to switch between): measured per unit at rank 256,
            // 4.1 k clk not unrolled, 3.1 k by two, 2.8 k fully (165 registers, no spills, with four or eight query
            // heads per KV head).
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
            // one arrival per warp (512 arrivals per unit on one barrier, half of them remote, cost about 2 % at low
            // ranks): every lane has its accumulator values in registers (tmem_wait_ld above)
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(lead_acc_empty[buf]);
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
#pragma unroll
            for (int i = 0; i < G / 4; ++i) {
                const int h = (un.hp * 2 + grp) * G + 4 * i + c;
                float* srow = p.scores + ((long long)un.s * p.H_q + h) * p.n_pad;
                // maximum over the 32 tokens of this warp (tokens past the end of the sequence do not count)
                float mxv = -INFINITY;
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    const int n = n0 + quarter * 32 + r + 8 * m;
                    if (n < p.n_pad) srow[n] = tot[m][i];
                    if (n < un.len) mxv = fmaxf(mxv, tot[m][i]);
                }
#pragma unroll
                for (int o = 4; o < 32; o <<= 1) mxv = fmaxf(mxv, __shfl_xor_sync(0xffffffffu, mxv, o));
                if (r == 0 && mxv > -INFINITY) atomicMax(p.rowmax + (long long)un.s * p.H_q + h, lorc_float_key(mxv));
            }
            ++uc;
            un = un_next;
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

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
struct LorcTcLayer {
    bool has_bkt = false;
    CUtensorMap mapBKT, mapBVT;         // B_K^T in 64 x 128 swizzled boxes; B_V^T in 64 x 32 swizzled boxes
    // cache maps are rebuilt only when the cache geometry or pointers change
    const void* k_ptr = nullptr;
    const void* v_ptr = nullptr;
    long long key_dims[6] = {0, 0, 0, 0, 0, 0};
    CUtensorMap mapCK, mapCV;
};

struct LorcTcState {
    float2* rope_tile = nullptr;
    unsigned* rowmax = nullptr;         // [rowmax_cap] row maxima of the softmax, see lorc_tc_decode
    size_t rowmax_cap = 0;
    bool rowmax_dirty = true;
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
        cudaFree(ctx->tc->rowmax);
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

static size_t tc_scores_bytes(const lorc_ctx* ctx, int batch, int max_seq_len) {
    size_t n_pad = (size_t)((max_seq_len + TILE - 1) / TILE) * TILE;
    return lorc_align_up((size_t)batch * ctx->desc.n_q_heads * n_pad * sizeof(float), 256);
}

size_t lorc_tc_workspace_bytes(const lorc_ctx* ctx, int batch, int max_seq_len) {
    if (!tc_shape_ok(ctx)) return 0;
    return tc_scores_bytes(ctx, batch, max_seq_len) + lorc_tc_pv_scratch_bytes(ctx, batch, max_seq_len);
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
        cudaError_t e = cudaMalloc(&T->rope_tile, sizeof(float2) * 64 * 33);
        if (e != cudaSuccess) return e;
        rope_tile_kernel<<<(64 * 33 + 255) / 256, 256, 0, st>>>(T->rope_tile, d.rope_theta);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    if (!T->attrs_set) {
        cudaError_t e;
        e = cudaFuncSetAttribute(lorc_score_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ScoreSmem) + 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(lorc_score_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ScoreSmem) + 1024);
        if (e != cudaSuccess) return e;
        T->attrs_set = true;
    }
    if (!TL.has_bkt) {
        uint64_t dims[2] = {(uint64_t)L.r_k, (uint64_t)ctx->n}, str[1] = {(uint64_t)L.r_k * 2};
        uint32_t box[2] = {KC, 128};
        if (!lorc_make_tmap_bf16(&TL.mapBKT, L.B_kT, 2, dims, str, box)) return cudaErrorInvalidValue;
        uint64_t d2[2] = {(uint64_t)L.r_v, (uint64_t)ctx->n}, s2[1] = {(uint64_t)L.r_v * 2};
        uint32_t b2[2] = {KC, 32};          // the up-projection takes a quarter of a head's columns per CTA
        if (!lorc_make_tmap_bf16(&TL.mapBVT, L.B_vT, 2, d2, s2, b2)) return cudaErrorInvalidValue;
        TL.has_bkt = true;
    }
    if (!build_cache_maps(TL, L, cv)) return cudaErrorInvalidValue;

    const int tiles = (cv.max_seq_len + TILE - 1) / TILE;
    const int n_pad = tiles * TILE;
    const size_t sc_bytes = tc_scores_bytes(ctx, cv.batch, cv.max_seq_len);
    if (sc_bytes >= ws_bytes) return cudaErrorMemoryAllocation;
    float* scores = (float*)ws;
    void* pv_scratch = (char*)ws + sc_bytes;
    const size_t pv_bytes = ws_bytes - sc_bytes;
    // Row maxima [batch, H_q]: all zero between calls (the PV kernel clears what the score kernel raised).  Owned by
    // the library because that invariant must hold from the first call on; grown when a larger batch shows up, and
    // cleared again after a call that did not get as far as launching the PV kernel.
    const size_t rm_need = (size_t)cv.batch * d.n_q_heads;
    if (rm_need > T->rowmax_cap) {
        cudaError_t e = cudaFree(T->rowmax);
        T->rowmax = nullptr;
        T->rowmax_cap = 0;
        if (e == cudaSuccess) e = cudaMalloc(&T->rowmax, rm_need * sizeof(unsigned));
        if (e != cudaSuccess) return e;
        T->rowmax_cap = rm_need;
        T->rowmax_dirty = true;
    }
    if (T->rowmax_dirty) {
        cudaError_t e = cudaMemsetAsync(T->rowmax, 0, T->rowmax_cap * sizeof(unsigned), st);
        if (e != cudaSuccess) return e;
    }
    T->rowmax_dirty = true;

    ScoreParams sp;
    sp.q = q; sp.scores = scores; sp.rowmax = T->rowmax; sp.seq_lens = cv.seq_lens; sp.page_table = cv.page_table;
    sp.rope_table = ctx->rope_table; sp.rope_tile = reinterpret_cast<const float4*>(T->rope_tile); sp.status = ctx->status_dev;
    sp.batch = cv.batch; sp.H_q = d.n_q_heads; sp.n_hp = d.n_kv_heads / 2; sp.r_k = L.r_k; sp.n_pad = n_pad;
    sp.tiles_per_seq = tiles; sp.tile_pairs = (tiles + 1) / 2; sp.max_pos = d.max_pos;
    sp.page_size = cv.page_size; sp.max_pages_per_seq = cv.max_pages_per_seq; sp.n_pages = cv.n_pages;
    const int total_units = cv.batch * sp.tile_pairs * sp.n_hp;          // units of a CTA pair
    int n_pairs = ctx->sm_count / 2;
    if (total_units < n_pairs) n_pairs = total_units;
    const int grid1 = 2 * n_pairs;
    const size_t smem1 = sizeof(ScoreSmem) + 1024;
    {
        LorcStageTimer timer(ctx, LORC_STAGE_SCORE, st);
        cudaError_t e;
        if (ctx->group == 4)
            e = lorc_launch_dependent(lorc_score_kernel<4>, dim3(grid1), dim3(S_THREADS), smem1, st, TL.mapCK, TL.mapBKT, sp);
        else
            e = lorc_launch_dependent(lorc_score_kernel<8>, dim3(grid1), dim3(S_THREADS), smem1, st, TL.mapCK, TL.mapBKT, sp);
        *launches += 1;
        if (e != cudaSuccess) return e;
    }
    const cudaError_t e2 = lorc_tc_pv_launch(ctx, L, cv, TL.mapCV, TL.mapBVT, scores, T->rowmax, n_pad, tiles, n_splits,
                                             pv_scratch, pv_bytes, out, st, launches);
    if (e2 == cudaSuccess) T->rowmax_dirty = false;
    return e2;
}
