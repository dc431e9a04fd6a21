// Decode attention for callers that may not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at all: an inference server
// that hands the whole GPU to its own pool at start-up and treats any later
// driver allocation as a bug (it would fail, or stall every stream while the
// driver maps memory), or a plug-in that is given tensors but no allocator.
// lorc_decode_attn needs scratch for the per-split partial results and expects
// the caller to lend it (lorc_set_workspace); lorc_decode_attn_static instead
// keeps that scratch in a fixed array inside the library image, so the call
// needs nothing but its inputs and outputs.
#include "common.cuh"

// The scratch itself: LORC_STATIC_SCRATCH_BYTES of device memory that every GPU
// loading the library holds until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[LORC_STATIC_SCRATCH_BYTES];

namespace {

// g_static_scratch is only a host-side handle here; the address kernels can use
// is asked from the runtime once per device and remembered.
constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {nullptr};

int static_fail(lorc_ctx* ctx, int code, const char* msg) {
    if (ctx) ctx->err = msg;
    return code;
}

size_t partial_bytes(int batch, int n_q_heads, int S, int W) {
    size_t units = (size_t)batch * n_q_heads * S;
    return lorc_align_up(units * 2 * sizeof(float), 256) + lorc_align_up(units * (size_t)W * sizeof(float), 256);
}

}  // namespace

extern "C" int lorc_decode_attn_static(lorc_ctx* ctx, int layer, const lorc_cache* c, const void* q,
                                       void* out, int n_splits, void* stream) {
    if (!ctx) return LORC_ERR_ARG;
    if (layer < 0 || layer >= ctx->desc.n_layers || !ctx->layers[layer].loaded)
        return static_fail(ctx, LORC_ERR_LAYER, "decode_attn_static: bad layer or no factors loaded");
    const LorcLayer& L = ctx->layers[layer];
    if (!q || !out || !c || !c->k || !c->v || !c->seq_lens)
        return static_fail(ctx, LORC_ERR_ARG, "decode_attn_static: null pointer");
    if (((uintptr_t)q & 15) || ((uintptr_t)out & 15) || ((uintptr_t)c->k & 15) || ((uintptr_t)c->v & 15))
        return static_fail(ctx, LORC_ERR_ARG, "decode_attn_static: pointers must be 16-byte aligned");
    if (n_splits < 0 || c->batch <= 0 || c->max_seq_len <= 0 || c->max_seq_len > ctx->desc.max_pos)
        return static_fail(ctx, LORC_ERR_ARG, "decode_attn_static: bad batch, max_seq_len or n_splits");
    long long capacity;
    if (c->page_table) {
        if (c->page_size <= 0 || c->page_size % 16 != 0 || c->max_pages_per_seq <= 0 || c->n_pages <= 0)
            return static_fail(ctx, LORC_ERR_ARG, "decode_attn_static: bad paging parameters");
        capacity = (long long)c->page_size * c->max_pages_per_seq;
    } else {
        if (c->seq_stride <= 0) return static_fail(ctx, LORC_ERR_ARG, "decode_attn_static: bad seq_stride");
        capacity = c->seq_stride;
    }
    if ((long long)c->max_seq_len > capacity)
        return static_fail(ctx, LORC_ERR_ARG, "decode_attn_static: max_seq_len exceeds the cache capacity");

    // set-up, once per device, with that device current
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices || dev != ctx->device) {
        ctx->err = "decode_attn_static: the context's device must be the current device";
        return LORC_ERR_CUDA;
    }
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) {
            ctx->err = std::string("decode_attn_static: cudaGetSymbolAddress: ") + cudaGetErrorString(e);
            return LORC_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }

    const bool latent = (L.mode == LORC_MODE_LATENT);
    const int W = latent ? L.r_v : ctx->desc.d_head;
    int S = n_splits > 0 ? n_splits : (c->max_seq_len + 511) / 512;
    int tiles = (c->max_seq_len + LORC_GENERIC_TILE - 1) / LORC_GENERIC_TILE;
    if (S > tiles) S = tiles;
    if (S > LORC_MAX_SPLITS) S = LORC_MAX_SPLITS;
    if (S < 1) S = 1;
    // fewer splits need less scratch; below one split nothing more can be saved
    while (S > 1 && partial_bytes(c->batch, ctx->desc.n_q_heads, S, W) > (size_t)LORC_STATIC_SCRATCH_BYTES) --S;
    if (partial_bytes(c->batch, ctx->desc.n_q_heads, S, W) > (size_t)LORC_STATIC_SCRATCH_BYTES)
        return static_fail(ctx, LORC_ERR_WORKSPACE,
                           "decode_attn_static: batch * n_q_heads * (2 + accumulator width) * 4 bytes exceeds "
                           "LORC_STATIC_SCRATCH_BYTES; use lorc_decode_attn with a workspace");

    CacheView cv;
    cv.k = (bf16*)c->k;
    cv.v = (bf16*)c->v;
    cv.page_table = c->page_table;
    cv.seq_lens = c->seq_lens;
    cv.batch = c->batch;
    cv.max_seq_len = c->max_seq_len;
    cv.page_size = c->page_table ? c->page_size : 0;
    cv.max_pages_per_seq = c->max_pages_per_seq;
    cv.n_pages = c->n_pages;
    cv.seq_stride = c->seq_stride;
    cv.w_k = L.r_k;
    cv.w_v = L.r_v;
    cv.capacity = capacity;

    // Every partial slot of this call's (batch, head, split) grid is written by the
    // attention kernel before the merge kernel reads it, so stale contents of the
    // shared array from an earlier call are never observed and nothing needs zeroing.
    size_t units = (size_t)c->batch * ctx->desc.n_q_heads * S;
    float* part_ml = (float*)g_scratch_addr[dev];
    float* part_o = (float*)((char*)g_scratch_addr[dev] + lorc_align_up(units * 2 * sizeof(float), 256));
    int launches = 0;
    e = lorc_generic_decode(ctx, L, cv, (const bf16*)q, (bf16*)out, S, part_ml, part_o, (cudaStream_t)stream,
                            &launches);
    ctx->launches += launches;
    ctx->last_path = lorc_full_decode_supported(ctx, L) ? 3 : 1;
    if (e != cudaSuccess) {
        ctx->err = std::string("decode_attn_static: ") + cudaGetErrorString(e);
        return LORC_ERR_CUDA;
    }
    return LORC_OK;
}
