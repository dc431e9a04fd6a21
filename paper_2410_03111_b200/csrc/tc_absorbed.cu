// Score kernel for layers whose keys take no rotation at attention time (LORC_ROPE_NONE): the paper's absorbed form.
//
// Without a position-dependent rotation between the key up-projection and the dot product, the up-projection moves to
// the query side (Sec. 3.1, the W_q' equation):
//     s[h, n] = q_h . (B_K[:, g]^T c_n) / sqrt(d_h) = (B_K[:, g] q_h) . c_n / sqrt(d_h) = q~_h . c_n,
// so the keys are never reconstructed and the scores are one skinny GEMM over the latent rows: 2 H_q r FLOP per
// 2 r bytes of C_K, far below the machine balance, i.e. bound by the HBM stream of C_K.
//
//   absorb kernel   q~[s, h, :] = B_K[:, g(h)] q[s, h, :] * log2(e) / sqrt(d_h) for all heads, split into a bf16 high
//                   part and a bf16 remainder (so the scores keep fp32-level accuracy), stored as the K-major rows the
//                   MMA reads;
//   score kernel    persistent CTAs walk the flat list of 128-token tiles.  Per tile
//                       S[heads, 128 tokens] = Q~hi . C_K[tile]^T + Q~lo . C_K[tile]^T      (tcgen05, fp32 in TMEM)
//                   with the heads on the M side (64 rows) and the tokens on the N side, from TMA-staged 64-wide slices
//                   of the latent tile and of q~; then the same softmax numerators as the rotating score kernel:
//                   per 32-token quarter and head an integer reference m, p = bf16(2^(s - m)) written into the PV
//                   kernel's operand image, m and the sum of p beside it, the row maxima raised by atomic maxima.
#include <math.h>

#include "sm100_ptx.cuh"
#include "tc_kernels.cuh"

using namespace sm100;

namespace {

constexpr int TILE = 128;
constexpr int KC = 64;
constexpr float LOG2E = 1.4426950408889634f;
constexpr int A_THREADS = 192;       // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
constexpr int A_ROWS = 64;           // rows of the query operand (heads; rows beyond H_q are padding)

// q~ in memory, r_ld = r_k rounded up to 64:
//   64 query heads: [sequence][part: 0 high, 1 remainder][64 rows = heads][r_ld] bf16 (two 64-row operands);
//   32 query heads: [sequence][64 rows: 32 high parts, then 32 remainders][r_ld] (one 64-row operand).
// One block per (64 latent columns, KV head g, 64 rows (sequence, head of g)): the block's 128 x 64 piece of B_K^T is
// read once and serves all 64 rows; thread = (latent column, group of 16 rows), the queries sit transposed in shared
// memory so that a thread fetches four rows' values with one 16-byte load.
__global__ void __launch_bounds__(256)
absorb_query_kernel(const bf16* __restrict__ q, const bf16* __restrict__ B_kT, bf16* __restrict__ qabs,
                    int batch, int H_q, int G, int r_k, int r_ld) {
    __shared__ __align__(16) float qT[128][64];            // [j][row]
    __shared__ __align__(16) bf16 Bs[128][64];             // the block's piece of B_K^T: [j][latent column]
    const int g = blockIdx.y, row0 = blockIdx.z * 64, rows = batch * G;
    const int tid = threadIdx.x;
    {
        // 128 rows of 128 bytes, eight 16-byte vectors each: all of a thread's loads are in flight at once
        // (r_k is a multiple of 8, so a vector lies wholly inside or wholly outside the rank)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int v = tid + i * 256, j = v >> 3, c8 = (v & 7) * 8;
            const int rho = blockIdx.x * 64 + c8;
            uint4 w = make_uint4(0u, 0u, 0u, 0u);
            if (rho < r_k) w = __ldg(reinterpret_cast<const uint4*>(B_kT + ((long long)g * 128 + j) * r_k + rho));
            *reinterpret_cast<uint4*>(&Bs[j][c8]) = w;
        }
    }
    {
        // thread = (row, quarter of j): consecutive lanes hold consecutive rows, so the transposed stores do not collide
        const int row = tid & 63, jq = tid >> 6;
        const int R = row0 + row;
        if (R < rows) {
            const int s = R / G, h = g * G + R % G;
            const uint4* src = reinterpret_cast<const uint4*>(q + ((long long)s * H_q + h) * 128 + jq * 32);
#pragma unroll
            for (int v4 = 0; v4 < 4; ++v4) {
                const uint4 w = __ldg(src + v4);
                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    qT[jq * 32 + v4 * 8 + 2 * e][row] = __uint_as_float(ww[e] << 16);
                    qT[jq * 32 + v4 * 8 + 2 * e + 1][row] = __uint_as_float(ww[e] & 0xffff0000u);
                }
            }
        } else {
            for (int j = 0; j < 32; ++j) qT[jq * 32 + j][row] = 0.f;
        }
    }
    __syncthreads();
    const int rho = blockIdx.x * 64 + (tid & 63), rg = tid >> 6;     // latent column, rows 16 rg .. 16 rg + 15 of the block
    float acc[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0.f;
    {
#pragma unroll 8
        for (int j = 0; j < 128; ++j) {
            const float bv = __bfloat162float(Bs[j][tid & 63]);
            const float4* qv = reinterpret_cast<const float4*>(&qT[j][rg * 16]);
#pragma unroll
            for (int i4 = 0; i4 < 4; ++i4) {
                const float4 x = qv[i4];
                acc[4 * i4 + 0] = fmaf(x.x, bv, acc[4 * i4 + 0]);
                acc[4 * i4 + 1] = fmaf(x.y, bv, acc[4 * i4 + 1]);
                acc[4 * i4 + 2] = fmaf(x.z, bv, acc[4 * i4 + 2]);
                acc[4 * i4 + 3] = fmaf(x.w, bv, acc[4 * i4 + 3]);
            }
        }
    }
    const float scale = rsqrtf(128.f) * LOG2E;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const int R = row0 + rg * 16 + i;
        if (R >= rows) break;
        const int s = R / G, h = g * G + R % G;
        const float x = acc[i] * scale;                     // zero in the padding columns r_k .. r_ld
        const bf16 a = __float2bfloat16_rn(x);
        const bf16 lo = __float2bfloat16_rn(x - __bfloat162float(a));
        if (H_q == 32) {
            qabs[((long long)s * A_ROWS + h) * r_ld + rho] = a;
            qabs[((long long)s * A_ROWS + 32 + h) * r_ld + rho] = lo;
        } else {
            qabs[(((long long)s * 2 + 0) * A_ROWS + h) * r_ld + rho] = a;
            qabs[(((long long)s * 2 + 1) * A_ROWS + h) * r_ld + rho] = lo;
        }
    }
}

// 64 heads: a stage holds the latent slice and two query operands (high parts, remainders), two MMAs per k-step add
// them in the accumulator.  32 heads: one query operand carries both (rows 0..31 high parts, rows 32..63 remainders),
// one MMA per k-step, and the warps that hold the remainder rows hand their values to the warps of the high-part rows.
template <int HQ>
struct AbsSmem {
    static constexpr int NQ = HQ == 64 ? 2 : 1;          // query operands per stage
    static constexpr int STAGES = HQ == 64 ? 6 : 8;
    bf16 C[STAGES][TILE * KC];            // latent slice [128 tokens][64]                16 KiB
    bf16 Q[STAGES][NQ][A_ROWS * KC];      // q~ operand(s) [64 rows][64]                   8 KiB each
    float4 xch[2][16][32];                // remainder-row scores on their way to the high-part rows (32 heads)
    uint64_t full[STAGES], empty[STAGES], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    int32_t tile_start[LORC_SCORE_MAX_BATCH + 1];
    int32_t lens[LORC_SCORE_MAX_BATCH];
};

struct AbsParams {
    uint8_t* pimg;                 // [b, tiles, image]
    unsigned* rowmax;              // [b, H_q]
    const int32_t* seq_lens;
    const int32_t* page_table;
    int* zero;
    int* status;
    int batch, seq0, H_q, r_k, tiles, n_zero, max_pos;
    int page_size, max_pages_per_seq, n_pages;
};

// sequence and tile index of flat tile f (s only moves forward)
template <class Smem>
__device__ __forceinline__ void locate_tile(const Smem& sm, int f, int batch, int& s, int& tile) {
    while (s + 1 < batch && f >= sm.tile_start[s + 1]) ++s;
    tile = f - sm.tile_start[s];
}

template <int HQ>
__global__ void __launch_bounds__(A_THREADS, 1)
lorc_score_absorbed_kernel(const __grid_constant__ CUtensorMap mapCK, const __grid_constant__ CUtensorMap mapQ,
                           const AbsParams p) {
    extern __shared__ uint8_t raw[];
    typedef AbsSmem<HQ> S;
    S& sm = *reinterpret_cast<S*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    constexpr int A_STAGES = S::STAGES, NQ = S::NQ;
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int nkc = (p.r_k + KC - 1) / KC;
    const int img_bytes = lorc_tc_image_bytes(HQ);
    constexpr int EPI_WARPS = 4;                         // every lane quarter of the accumulator holds rows in use

    if (tid == 0) {
        for (int i = 0; i < A_STAGES; ++i) {
            mbar_init(&sm.full[i], 1);
            mbar_init(&sm.empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sm.acc_full[i], 1);
            mbar_init(&sm.acc_empty[i], EPI_WARPS);
        }
        fence_barrier_init();
        prefetch_tensormap(&mapCK);
        prefetch_tensormap(&mapQ);
    }
    grid_dep_wait();                                     // q~ comes from the kernel before this one
    if (blockIdx.x == 0)
        for (int i = tid; i < p.n_zero; i += A_THREADS) p.zero[i] = 0;
    for (int i = tid; i < p.batch; i += A_THREADS) {
        int len = p.seq_lens[i];
        if (len > p.max_pos || len > p.tiles * TILE) {
            lorc_set_status(p.status, LORC_ERR_CAPACITY);
            len = 0;
        }
        sm.lens[i] = len > 0 ? len : 0;
    }
    if (warp == 1) {
        tmem_alloc(&sm.tmem_base, 256);
        tmem_relinquish();
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
    tc_fence_after_sync();
    grid_dep_launch();
    const uint32_t tmem = sm.tmem_base;
    const int n_flat = sm.tile_start[p.batch];
    bool ok = true;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (warp-uniform, elected lane)
        const bool paged = p.page_table != nullptr;
        uint32_t st = 0, par = 1;
        int s = 0;
        for (int f = blockIdx.x; f < n_flat && ok; f += gridDim.x) {
            int tile;
            locate_tile(sm, f, p.batch, s, tile);
            const int sg = p.seq0 + s, len = sm.lens[s];
            for (int kc = 0; kc < nkc; ++kc) {
                if (!mbar_wait(&sm.empty[st], par)) { ok = false; break; }
                if (elect_one()) {
                    mbar_arrive_expect_tx(&sm.full[st], (TILE + NQ * A_ROWS) * KC * 2);
                    if (!paged) {
                        tma_load_3d(sm.C[st], &mapCK, &sm.full[st], kc * KC, tile * TILE, sg);
                    } else {
                        // one box per page; pages past the end of the sequence (or with a bad table entry) are read
                        // from page 0: those tokens are masked, but every box must deliver its bytes
                        const int ppt = TILE / p.page_size;
                        for (int pg = 0; pg < ppt; ++pg) {
                            const int lp = tile * ppt + pg;
                            int page = 0;
                            if ((long long)lp * p.page_size < len && lp < p.max_pages_per_seq) {
                                page = p.page_table[(long long)sg * p.max_pages_per_seq + lp];
                                if (page < 0 || page >= p.n_pages) {
                                    lorc_set_status(p.status, LORC_ERR_CAPACITY);
                                    page = 0;
                                }
                            }
                            tma_load_3d(sm.C[st] + pg * p.page_size * KC, &mapCK, &sm.full[st], kc * KC, 0, page);
                        }
                    }
#pragma unroll
                    for (int part = 0; part < NQ; ++part)
                        tma_load_3d(sm.Q[st][part], &mapQ, &sm.full[st], kc * KC, 0, NQ * s + part);
                }
                __syncwarp();
                if (++st == A_STAGES) { st = 0; par ^= 1; }
            }
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (warp-uniform, elected lane)
        const uint32_t idesc = make_idesc_bf16(A_ROWS, TILE, 0, 0);
        const int nk_last = (p.r_k - (nkc - 1) * KC + 15) >> 4;       // 16-column steps the last slice really holds
        uint32_t st = 0, par = 0, uc = 0;
        for (int f = blockIdx.x; f < n_flat && ok; f += gridDim.x, ++uc) {
            const int buf = uc & 1;
            if (!mbar_wait(&sm.acc_empty[buf], ((uc >> 1) & 1) ^ 1)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t d = tmem + buf * 128;
            for (int kc = 0; kc < nkc; ++kc) {
                if (!mbar_wait(&sm.full[st], par)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t c0 = smem_u32(sm.C[st]), q0 = smem_u32(sm.Q[st][0]);
                if (elect_one()) {
                    const int nk = (kc + 1 < nkc) ? 4 : nk_last;
                    for (int k = 0; k < nk; ++k) {
                        const uint64_t bd = make_smem_desc_sw128(c0 + k * 32, 0, 1024);
                        tc_mma_bf16(d, make_smem_desc_sw128(q0 + k * 32, 0, 1024), bd, idesc, (kc | k) != 0);
                        if (NQ == 2)
                            tc_mma_bf16(d, make_smem_desc_sw128(q0 + A_ROWS * KC * 2 + k * 32, 0, 1024), bd, idesc, 1u);
                    }
                    tc_commit(&sm.empty[st]);
                }
                __syncwarp();
                if (++st == A_STAGES) { st = 0; par ^= 1; }
            }
            if (!ok) break;
            if (elect_one()) tc_commit(&sm.acc_full[buf]);
            __syncwarp();
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    } else {
        // ------------------------------------------------------------------ epilogue: softmax numerators
        // A 64-row accumulator keeps head 16 q + i (i < 16) in lane i of lane quarter q.  With 16-lane x 256-bit loads
        // lane (r = lane / 4, c = lane % 4) holds, per 8-token group k, the heads 16 q + r and 16 q + r + 8 and the tokens
        // 8 k + 2 c, 8 k + 2 c + 1: all 32 lanes work, and the four lanes of equal r share a head.
        const int quarter = warp % 4;
        {
            const int r = lane >> 2, c = lane & 3;
            uint32_t uc = 0;
            int s = 0;
            for (int f = blockIdx.x; f < n_flat && ok; f += gridDim.x, ++uc) {
                int tile;
                locate_tile(sm, f, p.batch, s, tile);
                const int len = sm.lens[s], buf = uc & 1;
                if (!mbar_wait(&sm.acc_full[buf], (uc >> 1) & 1)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t tbase = tmem + ((uint32_t)(quarter * 32) << 16) + buf * 128;
                uint32_t v[16][4];                                // [8-token group][head r: tokens 2c, 2c+1 | head r+8: same]
#pragma unroll
                for (int k = 0; k < 16; ++k) tmem_ld16x256_x1(tbase + k * 8, v[k]);
                tmem_wait_ld();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.acc_empty[buf]);
                if (HQ == 32) {
                    // lane quarters 2 and 3 hold the remainder rows of the heads of quarters 0 and 1, in the same layout
                    if (quarter >= 2) {
#pragma unroll
                        for (int k = 0; k < 16; ++k)
                            sm.xch[quarter - 2][k][lane] = make_float4(__uint_as_float(v[k][0]), __uint_as_float(v[k][1]),
                                                                       __uint_as_float(v[k][2]), __uint_as_float(v[k][3]));
                    }
                    __syncwarp();   // a named barrier counts a warp once only if the warp arrives converged
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (quarter < 2) {
#pragma unroll
                        for (int k = 0; k < 16; ++k) {
                            const float4 x = sm.xch[quarter][k][lane];
                            v[k][0] = __float_as_uint(__uint_as_float(v[k][0]) + x.x);
                            v[k][1] = __float_as_uint(__uint_as_float(v[k][1]) + x.y);
                            v[k][2] = __float_as_uint(__uint_as_float(v[k][2]) + x.z);
                            v[k][3] = __float_as_uint(__uint_as_float(v[k][3]) + x.w);
                        }
                    }
                    __syncwarp();
                    asm volatile("bar.sync 2, 128;" ::: "memory");   // the values have been taken: the next tile may overwrite them
                    if (quarter >= 2) continue;
                }
                uint8_t* img = p.pimg + ((long long)s * p.tiles + tile) * img_bytes;
                float* m_out = reinterpret_cast<float*>(img + 2 * HQ * KC * 2);
                float* l_out = m_out + 4 * HQ;
#pragma unroll
                for (int qt = 0; qt < 4; ++qt) {                  // 32-token quarter of the tile
                    uint8_t* chunk_img = img + (qt >> 1) * (HQ * KC * 2);
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const int h = quarter * 16 + r + 8 * hh;
                        float sc[4][2];
                        float mxv = -INFINITY, ssum = 0.f;
#pragma unroll
                        for (int k = 0; k < 4; ++k)
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                sc[k][e] = __uint_as_float(v[qt * 4 + k][2 * hh + e]);
                                ssum += sc[k][e];
                                if (tile * TILE + qt * 32 + 8 * k + 2 * c + e < len) mxv = fmaxf(mxv, sc[k][e]);
                            }
                        // a NaN among the scores means non-finite numbers in the cache, the factors or the query
                        if (ssum != ssum) lorc_set_status(p.status, LORC_ERR_ARG);
                        mxv = fmaxf(mxv, __shfl_xor_sync(0xffffffffu, mxv, 1));
                        mxv = fmaxf(mxv, __shfl_xor_sync(0xffffffffu, mxv, 2));
                        const float mref = ceilf(mxv);            // -inf: no token of the sequence in this quarter
                        float lsum = 0.f;
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int t0 = qt * 32 + 8 * k + 2 * c;              // token inside the tile
                            const bool v0 = tile * TILE + t0 < len, v1 = tile * TILE + t0 + 1 < len;
                            const __nv_bfloat162 pr = __floats2bfloat162_rn(v0 ? exp2f(sc[k][0] - mref) : 0.f,
                                                                            v1 ? exp2f(sc[k][1] - mref) : 0.f);
                            lsum += __low2float(pr) + __high2float(pr);
                            const int tc = t0 & 63;
                            *reinterpret_cast<__nv_bfloat162*>(chunk_img + h * 128 + ((((tc >> 3) ^ (h & 7)) << 4) | ((tc & 7) << 1))) = pr;
                        }
                        lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
                        lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
                        if (c == 0) {
                            m_out[qt * HQ + h] = mref;
                            l_out[qt * HQ + h] = lsum;
                            if (mxv > -INFINITY) atomicMax(p.rowmax + (long long)s * HQ + h, lorc_float_key(mref));
                        }
                    }
                }
            }
            if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 256);
}

}  // namespace

size_t lorc_tc_absorbed_scratch_bytes(const lorc_ctx* ctx, int batch) {
    const size_t r_ld = (size_t)((ctx->n + KC - 1) / KC) * KC;
    const size_t parts = ctx->desc.n_q_heads == 64 ? 2 : 1;
    return lorc_align_up((size_t)batch * parts * A_ROWS * r_ld * sizeof(bf16), 256);
}

cudaError_t lorc_tc_absorbed_set_attrs() {
    cudaError_t e = cudaFuncSetAttribute(lorc_score_absorbed_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)sizeof(AbsSmem<32>) + 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(lorc_score_absorbed_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)sizeof(AbsSmem<64>) + 1024);
    return e;
}

// qabs: scratch of lorc_tc_absorbed_scratch_bytes.  Launches the absorb kernel and the score kernel (one pair per
// block of LORC_SCORE_MAX_BATCH sequences); outputs as lorc_tc_score_launch.
cudaError_t lorc_tc_score_absorbed_launch(lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, const CUtensorMap& mapCK,
                                          const bf16* q, bf16* qabs, uint8_t* pimg, unsigned* rowmax, int tiles, int* zero,
                                          int n_zero, cudaStream_t st, int* launches) {
    const lorc_model_desc& d = ctx->desc;
    const int r_ld = (L.r_k + KC - 1) / KC * KC;
    const size_t img_bytes = (size_t)lorc_tc_image_bytes(d.n_q_heads);
    for (int s0 = 0; s0 < cv.batch; s0 += LORC_SCORE_MAX_BATCH) {
        const int nb = cv.batch - s0 < LORC_SCORE_MAX_BATCH ? cv.batch - s0 : LORC_SCORE_MAX_BATCH;
        const int parts = d.n_q_heads == 64 ? 2 : 1;
        bf16* qa = qabs + (size_t)s0 * parts * A_ROWS * r_ld;
        absorb_query_kernel<<<dim3(r_ld / KC, d.n_kv_heads, (nb * ctx->group + 63) / 64), 256, 0, st>>>(
            q + (size_t)s0 * d.n_q_heads * 128, L.B_kT, qa, nb, d.n_q_heads, ctx->group, L.r_k, r_ld);
        cudaError_t e = cudaGetLastError();
        *launches += 1;
        if (e != cudaSuccess) return e;
        CUtensorMap mapQ;
        {
            uint64_t dims[3] = {(uint64_t)L.r_k, (uint64_t)A_ROWS, (uint64_t)nb * parts};
            uint64_t str[2] = {(uint64_t)r_ld * 2, (uint64_t)A_ROWS * r_ld * 2};
            uint32_t box[3] = {KC, A_ROWS, 1};
            if (!lorc_make_tmap_bf16(&mapQ, qa, 3, dims, str, box)) return cudaErrorInvalidValue;
        }
        AbsParams ap;
        ap.pimg = pimg + (size_t)s0 * tiles * img_bytes;
        ap.rowmax = rowmax + (size_t)s0 * d.n_q_heads;
        ap.seq_lens = cv.seq_lens + s0;
        ap.page_table = cv.page_table;
        ap.zero = zero;
        ap.n_zero = s0 == 0 ? n_zero : 0;
        ap.status = ctx->status_dev;
        ap.batch = nb; ap.seq0 = s0; ap.H_q = d.n_q_heads; ap.r_k = L.r_k; ap.tiles = tiles; ap.max_pos = d.max_pos;
        ap.page_size = cv.page_size; ap.max_pages_per_seq = cv.max_pages_per_seq; ap.n_pages = cv.n_pages;
        const long long max_tiles = (long long)nb * tiles;
        const int grid = (int)(max_tiles < ctx->sm_count ? max_tiles : ctx->sm_count);
        if (d.n_q_heads == 32)
            e = lorc_launch_dependent(lorc_score_absorbed_kernel<32>, dim3(grid), dim3(A_THREADS), sizeof(AbsSmem<32>) + 1024,
                                      st, mapCK, mapQ, ap);
        else
            e = lorc_launch_dependent(lorc_score_absorbed_kernel<64>, dim3(grid), dim3(A_THREADS), sizeof(AbsSmem<64>) + 1024,
                                      st, mapCK, mapQ, ap);
        *launches += 1;
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}
