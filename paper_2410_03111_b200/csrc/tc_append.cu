// Cache write for prompt-sized token counts on the tensor cores (sm_100a: TMA + tcgen05 + TMEM).
//
// C_K, C_V[new tokens] = bf16(x . [A_K | A_V])  (Sec. 3.1: the cache keeps X times the Sigma-carrying factor), one GEMM
// with M = tokens, N = r_k + r_v, K = D.  At decode (a token per sequence) the call is bound by the factor stream and
// runs on the warp-level kernel; from 128 tokens per launch on it is a dense contraction and runs here:
//   one CTA per (128 tokens, 256 columns of [A_K | A_V]); K = D in 64-wide TMA stages; x rows are the K-major A
//   operand, the factor rows (D index) with their contiguous columns are the MN-major B operand, so the factor needs
//   no transposed copy; fp32 accumulation in TMEM; the epilogue (thread = token) rounds once to bf16 and writes each
//   token's slice to its row of the contiguous or paged cache.
#include <math.h>

#include "sm100_ptx.cuh"
#include "tc_kernels.cuh"

using namespace sm100;

namespace {

constexpr int TILE = 128;            // tokens per CTA
constexpr int KC = 64;               // D elements per stage
constexpr int NB = 256;              // columns of [A_K | A_V] per CTA
constexpr int W_STAGES = 4;
constexpr int W_THREADS = 192;       // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue

struct AppSmem {
    bf16 X[W_STAGES][TILE * KC];          // [128 tokens][64]                    16 KiB
    bf16 A[W_STAGES][4][KC * KC];         // four blocks of [64 D rows][64 cols]  32 KiB
    uint64_t full[W_STAGES], empty[W_STAGES], d_full;
    uint32_t tmem_base;
};

struct AppParams {
    CacheView cv;
    int D, r_k, r_v, T, n_tok, max_pos;
    int* status;
};

__global__ void __launch_bounds__(W_THREADS, 1)
lorc_append_tc_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapA, const AppParams p) {
    extern __shared__ uint8_t raw[];
    AppSmem& sm = *reinterpret_cast<AppSmem*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int col0 = blockIdx.x * NB, tok0 = blockIdx.y * TILE;
    const int R = p.r_k + p.r_v;
    const int nkc = p.D / KC;
    const int nblk = min(4, (R - col0 + KC - 1) / KC);        // 64-column blocks of the factor that exist here

    if (tid == 0) {
        for (int i = 0; i < W_STAGES; ++i) {
            mbar_init(&sm.full[i], 1);
            mbar_init(&sm.empty[i], 1);
        }
        mbar_init(&sm.d_full, 1);
        fence_barrier_init();
        prefetch_tensormap(&mapX);
        prefetch_tensormap(&mapA);
    }
    if (warp == 1) {
        tmem_alloc(&sm.tmem_base, NB);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    bool ok = true;

    if (warp == 0) {
        for (int kc = 0; kc < nkc && ok; ++kc) {
            const int st = kc % W_STAGES;
            if (!mbar_wait(&sm.empty[st], ((kc / W_STAGES) & 1) ^ 1)) { ok = false; break; }
            if (elect_one()) {
                // columns past r_k + r_v and token rows past the batch read as zero, but still deliver their bytes
                mbar_arrive_expect_tx(&sm.full[st], (TILE + 4 * KC) * KC * 2);
                tma_load_2d(sm.X[st], &mapX, &sm.full[st], kc * KC, tok0);
#pragma unroll
                for (int b = 0; b < 4; ++b) tma_load_2d(sm.A[st][b], &mapA, &sm.full[st], col0 + b * KC, kc * KC);
            }
            __syncwarp();
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    } else if (warp == 1) {
        // A: x rows (K-major).  B: factor block (MN-major: a D row's 64 columns are contiguous), 64-column blocks 8 KiB
        // apart, 16 D rows (one k-step) 2 KiB apart.
        const uint32_t idesc = make_idesc_bf16(TILE, NB, 0, 1);
        for (int kc = 0; kc < nkc && ok; ++kc) {
            const int st = kc % W_STAGES;
            if (!mbar_wait(&sm.full[st], (kc / W_STAGES) & 1)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t x0 = smem_u32(sm.X[st]), a0 = smem_u32(sm.A[st][0]);
            if (elect_one()) {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    tc_mma_bf16(tmem, make_smem_desc_sw128(x0 + k * 32, 0, 1024),
                                make_smem_desc_sw128(a0 + k * 2048, KC * KC * 2, 1024), idesc, (kc | k) != 0);
                tc_commit(&sm.empty[st]);
            }
            __syncwarp();
        }
        if (ok) {
            if (elect_one()) tc_commit(&sm.d_full);
            __syncwarp();
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    } else {
        if (!mbar_wait(&sm.d_full, 0)) ok = false;
        if (ok) {
            tc_fence_after_sync();
            const int quarter = warp % 4;
            const int tok = tok0 + quarter * 32 + lane;               // token of the launch = TMEM lane
            // where this token's rows live: token i of sequence s goes to position seq_lens[s] - T + i
            long long row = -1;
            if (tok < p.n_tok) {
                const int s = tok / p.T, i = tok - s * p.T;
                const int pos = p.cv.seq_lens[s] - p.T + i;
                if (pos >= 0 && pos < p.max_pos) row = lorc_row_index(p.cv, s, pos);
                if (row < 0) lorc_set_status(p.status, LORC_ERR_CAPACITY);
            }
#pragma unroll 1
            for (int b = 0; b < nblk; ++b) {
#pragma unroll
                for (int c0 = 0; c0 < KC; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + b * KC + c0, r);
                    tmem_wait_ld();
                    if (row < 0) continue;
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        const int col = col0 + b * KC + c0 + v * 8;   // eight columns: ranks are multiples of eight, so a
                        if (col >= R) break;                          // piece lies wholly in C_K or wholly in C_V
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(r[v * 8 + 2 * e]),
                                                                            __uint_as_float(r[v * 8 + 2 * e + 1]));
                            w[e] = *reinterpret_cast<const uint32_t*>(&b2);
                        }
                        bf16* dst = col < p.r_k ? p.cv.k + row * p.cv.w_k + col : p.cv.v + row * p.cv.w_v + (col - p.r_k);
                        *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
        }
        if (!ok && lane == 0) lorc_set_status(p.status, LORC_ERR_TIMEOUT);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, NB);
}

}  // namespace

bool lorc_tc_append_gemm_supported(const lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, int T) {
    return L.mode == LORC_MODE_LATENT && (long long)cv.batch * T >= TILE && ctx->desc.d_model % KC == 0 &&
           L.r_k % 8 == 0 && L.r_v % 8 == 0 && lorc_get_tmap_encode() != nullptr;
}

cudaError_t lorc_tc_append_gemm(lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv, const bf16* x, int T,
                                cudaStream_t st, int* launches) {
    static bool attr[64] = {false};
    const bool known = ctx->device >= 0 && ctx->device < 64;
    if (!known || !attr[ctx->device]) {
        cudaError_t e = cudaFuncSetAttribute(lorc_append_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)sizeof(AppSmem) + 1024);
        if (e != cudaSuccess) return e;
        if (known) attr[ctx->device] = true;
    }
    const int D = ctx->desc.d_model, R = L.r_k + L.r_v;
    const long long n_tok = (long long)cv.batch * T;
    CUtensorMap mapX, mapA;
    {
        uint64_t xd[2] = {(uint64_t)D, (uint64_t)n_tok}, xs[1] = {(uint64_t)D * 2};
        uint32_t xb[2] = {KC, TILE};
        if (!lorc_make_tmap_bf16(&mapX, x, 2, xd, xs, xb)) return cudaErrorInvalidValue;
        uint64_t ad[2] = {(uint64_t)R, (uint64_t)D}, as[1] = {(uint64_t)R * 2};
        uint32_t ab[2] = {KC, KC};
        if (!lorc_make_tmap_bf16(&mapA, L.A_cat, 2, ad, as, ab)) return cudaErrorInvalidValue;
    }
    AppParams p;
    p.cv = cv; p.D = D; p.r_k = L.r_k; p.r_v = L.r_v; p.T = T; p.n_tok = (int)n_tok; p.max_pos = ctx->desc.max_pos;
    p.status = ctx->status_dev;
    dim3 grid((R + NB - 1) / NB, (unsigned)((n_tok + TILE - 1) / TILE));
    lorc_append_tc_kernel<<<grid, W_THREADS, sizeof(AppSmem) + 1024, st>>>(mapX, mapA, p);
    *launches += 1;
    return cudaGetLastError();
}
