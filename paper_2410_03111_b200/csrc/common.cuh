// Shared declarations of the latent-KV decode-attention library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "lorc.h"

typedef __nv_bfloat16 bf16;

// Device status word values mirror the LORC_ERR_* codes; the first error wins.
__device__ __forceinline__ void lorc_set_status(int* status, int code) {
    atomicCAS(status, 0, code);
}

// Per-layer factor storage owned by the library (device memory).
struct LorcLayer {
    int loaded = 0;
    int mode = LORC_MODE_LATENT;
    int r_k = 0, r_v = 0;      // FULL mode: both equal n
    bf16* A_cat = nullptr;     // [D, r_k + r_v]   columns of A_K then A_V (FULL: W_k then W_v)
    bf16* A_tiled = nullptr;   // [(r_k+r_v)/8][D/32][32 lanes][8]: A_cat in mma fragment order (fast append), D % 32 == 0
    bf16* B_k = nullptr;       // [r_k, n]   (LATENT)
    bf16* B_v = nullptr;       // [r_v, n]   (LATENT)
    bf16* B_kT = nullptr;      // [n, r_k]   transposed copy (K-major operand of the key reconstruction)
    bf16* B_vT = nullptr;      // [n, r_v]   transposed copy (K-major operand of the value up-projection)
};

struct LorcTcState;            // tensor-core path's private per-context state

// Event pairs recorded around kernels when LORC_FLAG_PROFILE is set.
struct LorcProfile {
    struct Rec { int stage; cudaEvent_t e0, e1; };
    std::vector<Rec> pending;
    std::vector<cudaEvent_t> pool;
    cudaEvent_t get() {
        if (!pool.empty()) { cudaEvent_t e = pool.back(); pool.pop_back(); return e; }
        cudaEvent_t e = nullptr;
        cudaEventCreate(&e);
        return e;
    }
};

struct lorc_ctx {
    lorc_model_desc desc;
    int device = 0;
    int n = 0;                 // n_kv_heads * d_head
    int group = 0;             // n_q_heads / n_kv_heads
    int pair_style = LORC_ROPE_HALF_SPLIT;   // how the kernels pair the elements of a head (LORC_ROPE_NONE: half split,
                                              // with a rotation table that holds the identity)
    int sm_count = 0;
    std::vector<LorcLayer> layers;
    float2* rope_table = nullptr;   // [max_pos][d_head/2] (cos, sin)
    int* status_dev = nullptr;
    void* ws = nullptr;
    size_t ws_bytes = 0;
    std::string err;
    int last_path = 0;
    int64_t launches = 0;
    LorcTcState* tc = nullptr;
    LorcProfile* prof = nullptr;   // event bookkeeping, created on first use
    bool prof_on = false;          // LORC_FLAG_PROFILE or lorc_profile_enable
};

// RAII bracket: records an event pair around the launches issued in its scope (no-op unless profiling).
struct LorcStageTimer {
    LorcProfile* p;
    LorcProfile::Rec rec;
    cudaStream_t st;
    LorcStageTimer(const lorc_ctx* ctx, int stage, cudaStream_t stream)
        : p(ctx->prof_on ? ctx->prof : nullptr), st(stream) {
        if (!p) return;
        rec.stage = stage;
        rec.e0 = p->get();
        rec.e1 = p->get();
        cudaEventRecord(rec.e0, st);
    }
    ~LorcStageTimer() {
        if (!p) return;
        cudaEventRecord(rec.e1, st);
        p->pending.push_back(rec);
    }
};

// Where rows of a cache live: contiguous or paged (mirrors lorc_cache, device-usable).
struct CacheView {
    bf16* k;
    bf16* v;
    const int32_t* page_table;
    const int32_t* seq_lens;
    int batch;
    int max_seq_len;
    int page_size;
    int max_pages_per_seq;
    int n_pages;
    long long seq_stride;
    int w_k, w_v;              // row widths (elements)
    long long capacity;        // rows per sequence that exist
};

// Row index (in rows of the pool / of the contiguous array) of token `pos` of
// sequence `s`, or -1 when the position or the page is out of range.
__device__ __forceinline__ long long lorc_row_index(const CacheView& c, int s, int pos) {
    if (pos < 0 || (long long)pos >= c.capacity) return -1;
    if (c.page_table == nullptr) return (long long)s * c.seq_stride + pos;
    int lp = pos / c.page_size;
    int page = c.page_table[(long long)s * c.max_pages_per_seq + lp];
    if (page < 0 || page >= c.n_pages) return -1;
    return (long long)page * c.page_size + (pos - lp * c.page_size);
}

static inline size_t lorc_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- plain fp32 CUDA-core kernels: generic_kernels.cu ------------------------
cudaError_t lorc_generic_build_rope_table(float2* table, int max_pos, int d_head, double theta,
                                          cudaStream_t st);
cudaError_t lorc_generic_transpose(const bf16* in, bf16* out, int rows, int cols, cudaStream_t st);
cudaError_t lorc_generic_append(const lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv,
                                const bf16* x, int T, cudaStream_t st, int* launches);
// Uncompressed mode, 128-wide heads, bf16 path: streaming decode kernel on mma.sync (full_decode.cu).  Leaves the same
// per-split partial results as the plain kernel, for lorc_generic_combine.
bool lorc_full_decode_supported(const lorc_ctx* ctx, const LorcLayer& L);
cudaError_t lorc_full_decode(const lorc_ctx* ctx, const CacheView& cv, const bf16* q, int n_splits, float* part_ml,
                             float* part_o, cudaStream_t st, int* launches);
// latent_out: stop before the value up-projection and write the normalised latent output [b, H_q, r_v] to `out`.
// T > 1: T queries per sequence (q, out [b, T, H_q, d_head]; partial results for b * T units), query t of a sequence
// at position seq_lens[s] - T + t, attending to the tokens up to its own.
cudaError_t lorc_generic_decode(const lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv,
                                const bf16* q, bf16* out, int n_splits, float* part_ml,
                                float* part_o, cudaStream_t st, int* launches, bool latent_out = false, int T = 1,
                                const int32_t* pos0 = nullptr, const int32_t* q_pos = nullptr, float* ml_out = nullptr);
// Merge of the results of context shards (lorc_merge_shards).
cudaError_t lorc_generic_merge_shards(const lorc_ctx* ctx, int n_shards, const bf16* outs, const float* mls, bf16* out,
                                      int batch, cudaStream_t st, int* launches);
// Merge of split partials + value up-projection (also used by the tensor-core path):
// part_ml [b, H_q, S, 2] (running max in natural-log units, sum), part_o [b, H_q, S, W].
cudaError_t lorc_generic_combine(const lorc_ctx* ctx, const LorcLayer& L, int batch, int n_splits,
                                 const float* part_ml, const float* part_o, bf16* out,
                                 cudaStream_t st, int* launches, bool latent_out = false, float* ml_out = nullptr);
// token granularity of a split in the plain decode kernel
#define LORC_GENERIC_TILE 32
#define LORC_MAX_SPLITS 256
