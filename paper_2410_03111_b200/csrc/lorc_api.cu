// C ABI of the library: context, factor storage, argument checks and dispatch.
#include <stdio.h>
#include <string.h>

#include <new>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "tc_kernels.cuh"

namespace {

int fail(lorc_ctx* ctx, int code, const char* msg) {
    if (ctx) ctx->err = msg;
    return code;
}

int fail_cuda(lorc_ctx* ctx, cudaError_t e, const char* where) {
    if (ctx) ctx->err = std::string(where) + ": " + cudaGetErrorString(e);
    return LORC_ERR_CUDA;
}

void free_layer(LorcLayer& L) {
    cudaFree(L.A_cat);
    cudaFree(L.A_tiled);
    cudaFree(L.B_k);
    cudaFree(L.B_v);
    cudaFree(L.B_kT);
    cudaFree(L.B_vT);
    L = LorcLayer();
}

// Default number of context splits of the plain kernels: about 512 tokens each.
int generic_default_splits(int max_seq_len) {
    int s = (max_seq_len + 511) / 512;
    if (s < 1) s = 1;
    if (s > LORC_MAX_SPLITS) s = LORC_MAX_SPLITS;
    return s;
}

struct WsLayout {
    size_t off_ml, off_o, total;
};

// Partial-result area of the plain kernels for `batch` sequences, S splits and
// accumulator width W; it starts at the front of the workspace.
WsLayout ws_layout(const lorc_ctx* ctx, int batch, int S, int W) {
    WsLayout w;
    size_t units = (size_t)batch * ctx->desc.n_q_heads * S;
    size_t o = 0;
    w.off_ml = o;
    o = lorc_align_up(o + units * 2 * sizeof(float), 256);
    w.off_o = o;
    o = lorc_align_up(o + units * (size_t)W * sizeof(float), 256);
    w.total = o;
    return w;
}

// Staging of the host-buffer entry point: x, q and out of one step, carved from
// the END of the workspace so that it never overlaps partial results.
size_t staging_bytes(const lorc_ctx* ctx, int batch) {
    const lorc_model_desc& d = ctx->desc;
    size_t xb = (size_t)batch * d.d_model * sizeof(bf16);
    size_t qb = (size_t)batch * d.n_q_heads * d.d_head * sizeof(bf16);
    return lorc_align_up(xb, 256) + 2 * lorc_align_up(qb, 256);
}

int check_cache(lorc_ctx* ctx, const lorc_cache* c, const LorcLayer& L, CacheView* cv) {
    if (!c || !c->k || !c->v || !c->seq_lens) return fail(ctx, LORC_ERR_ARG, "cache: null pointer");
    if (c->batch <= 0) return fail(ctx, LORC_ERR_ARG, "cache: batch must be positive");
    if (c->max_seq_len <= 0) return fail(ctx, LORC_ERR_ARG, "cache: max_seq_len must be positive");
    if (c->max_seq_len > ctx->desc.max_pos)
        return fail(ctx, LORC_ERR_ARG, "cache: max_seq_len exceeds the context's max_pos");
    long long capacity;
    if (c->page_table) {
        if (c->page_size <= 0 || c->page_size % 16 != 0 || c->max_pages_per_seq <= 0 || c->n_pages <= 0)
            return fail(ctx, LORC_ERR_ARG,
                        "cache: bad paging parameters (page_size must be a positive multiple of 16)");
        capacity = (long long)c->page_size * c->max_pages_per_seq;
    } else {
        if (c->seq_stride <= 0) return fail(ctx, LORC_ERR_ARG, "cache: seq_stride must be positive");
        capacity = c->seq_stride;
    }
    if ((long long)c->max_seq_len > capacity)
        return fail(ctx, LORC_ERR_ARG, "cache: max_seq_len exceeds the cache capacity");
    if (((uintptr_t)c->k & 15) || ((uintptr_t)c->v & 15))
        return fail(ctx, LORC_ERR_ARG, "cache: k and v must be 16-byte aligned");
    cv->k = (bf16*)c->k;
    cv->v = (bf16*)c->v;
    cv->page_table = c->page_table;
    cv->seq_lens = c->seq_lens;
    cv->batch = c->batch;
    cv->max_seq_len = c->max_seq_len;
    cv->page_size = c->page_table ? c->page_size : 0;
    cv->max_pages_per_seq = c->max_pages_per_seq;
    cv->n_pages = c->n_pages;
    cv->seq_stride = c->seq_stride;
    cv->w_k = L.r_k;
    cv->w_v = L.r_v;
    cv->capacity = capacity;
    return LORC_OK;
}

int get_layer(lorc_ctx* ctx, int layer, LorcLayer** L) {
    if (!ctx) return LORC_ERR_ARG;
    if (layer < 0 || layer >= ctx->desc.n_layers) return fail(ctx, LORC_ERR_LAYER, "layer index out of range");
    if (!ctx->layers[layer].loaded) return fail(ctx, LORC_ERR_LAYER, "no factors loaded for this layer");
    *L = &ctx->layers[layer];
    return LORC_OK;
}

}  // namespace

extern "C" {

int lorc_create(const lorc_model_desc* desc, lorc_ctx** out) {
    if (!desc || !out) return LORC_ERR_ARG;
    *out = nullptr;
    if (desc->n_layers <= 0 || desc->d_model <= 0 || desc->n_q_heads <= 0 || desc->n_kv_heads <= 0 ||
        desc->max_pos <= 0 || !(desc->rope_theta > 0.0))
        return LORC_ERR_ARG;
    if (desc->n_q_heads % desc->n_kv_heads != 0) return LORC_ERR_ARG;
    if (desc->n_q_heads / desc->n_kv_heads > 8) return LORC_ERR_UNSUPPORTED;
    if (desc->d_head != 64 && desc->d_head != 128) return LORC_ERR_UNSUPPORTED;
    if (desc->rope_style != LORC_ROPE_HALF_SPLIT && desc->rope_style != LORC_ROPE_INTERLEAVED &&
        desc->rope_style != LORC_ROPE_NONE)
        return LORC_ERR_ARG;
    if (desc->d_model % 8 != 0) return LORC_ERR_ARG;
    lorc_ctx* ctx = new (std::nothrow) lorc_ctx();
    if (!ctx) return LORC_ERR_ARG;
    ctx->desc = *desc;
    ctx->n = desc->n_kv_heads * desc->d_head;
    ctx->group = desc->n_q_heads / desc->n_kv_heads;
    ctx->pair_style = desc->rope_style == LORC_ROPE_NONE ? LORC_ROPE_HALF_SPLIT : desc->rope_style;
    ctx->layers.resize(desc->n_layers);
    if (desc->flags & LORC_FLAG_PROFILE) {
        ctx->prof = new (std::nothrow) LorcProfile();
        ctx->prof_on = ctx->prof != nullptr;
    }
    cudaError_t e = cudaGetDevice(&ctx->device);
    if (e == cudaSuccess)
        e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device);
    if (e == cudaSuccess) e = cudaMalloc(&ctx->status_dev, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(ctx->status_dev, 0, sizeof(int));
    size_t tbytes = (size_t)desc->max_pos * (desc->d_head / 2) * sizeof(float2);
    if (e == cudaSuccess) e = cudaMalloc(&ctx->rope_table, tbytes);
    if (e == cudaSuccess)
        e = lorc_generic_build_rope_table(ctx->rope_table, desc->max_pos, desc->d_head,
                                          desc->rope_style == LORC_ROPE_NONE ? 0.0 : desc->rope_theta, 0);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        cudaFree(ctx->status_dev);
        cudaFree(ctx->rope_table);
        delete ctx->prof;
        delete ctx;
        return LORC_ERR_CUDA;
    }
    *out = ctx;
    return LORC_OK;
}

int lorc_destroy(lorc_ctx* ctx) {
    if (!ctx) return LORC_ERR_ARG;
    for (auto& L : ctx->layers) free_layer(L);
    lorc_tc_release(ctx);
    if (ctx->prof) {
        for (auto& r : ctx->prof->pending) {
            cudaEventDestroy(r.e0);
            cudaEventDestroy(r.e1);
        }
        for (auto e : ctx->prof->pool) cudaEventDestroy(e);
        delete ctx->prof;
    }
    cudaFree(ctx->status_dev);
    cudaFree(ctx->rope_table);
    delete ctx;
    return LORC_OK;
}

int lorc_load_factors(lorc_ctx* ctx, int layer, int mode, int r_k, int r_v, const void* A_k,
                      const void* B_k, const void* A_v, const void* B_v, void* stream) {
    if (!ctx) return LORC_ERR_ARG;
    if (layer < 0 || layer >= ctx->desc.n_layers) return fail(ctx, LORC_ERR_LAYER, "layer index out of range");
    if (mode != LORC_MODE_LATENT && mode != LORC_MODE_FULL) return fail(ctx, LORC_ERR_ARG, "unknown layer mode");
    const int D = ctx->desc.d_model, n = ctx->n;
    if (!A_k || !A_v) return fail(ctx, LORC_ERR_ARG, "load_factors: A_k / A_v is null");
    if (mode == LORC_MODE_LATENT) {
        if (!B_k || !B_v) return fail(ctx, LORC_ERR_ARG, "load_factors: B_k / B_v is null");
        if (r_k < 8 || r_v < 8 || r_k > n || r_v > n || r_k % 8 || r_v % 8)
            return fail(ctx, LORC_ERR_ARG,
                        "load_factors: ranks must be multiples of 8 in [8, n_kv_heads*d_head]");
    } else {
        r_k = r_v = n;
    }
    cudaStream_t st = (cudaStream_t)stream;
    LorcLayer& L = ctx->layers[layer];
    free_layer(L);
    lorc_tc_invalidate_layer(ctx, layer);
    const int R = r_k + r_v;
    cudaError_t e = cudaMalloc(&L.A_cat, (size_t)D * R * sizeof(bf16));
    if (e == cudaSuccess && D % 32 == 0) e = cudaMalloc(&L.A_tiled, (size_t)D * R * sizeof(bf16));
    if (e == cudaSuccess && mode == LORC_MODE_LATENT) {
        e = cudaMalloc(&L.B_k, (size_t)r_k * n * sizeof(bf16));
        if (e == cudaSuccess) e = cudaMalloc(&L.B_v, (size_t)r_v * n * sizeof(bf16));
        if (e == cudaSuccess) e = cudaMalloc(&L.B_kT, (size_t)r_k * n * sizeof(bf16));
        if (e == cudaSuccess) e = cudaMalloc(&L.B_vT, (size_t)r_v * n * sizeof(bf16));
    }
    if (e == cudaSuccess)
        e = cudaMemcpy2DAsync(L.A_cat, (size_t)R * sizeof(bf16), A_k, (size_t)r_k * sizeof(bf16),
                              (size_t)r_k * sizeof(bf16), D, cudaMemcpyDeviceToDevice, st);
    if (e == cudaSuccess)
        e = cudaMemcpy2DAsync(L.A_cat + r_k, (size_t)R * sizeof(bf16), A_v, (size_t)r_v * sizeof(bf16),
                              (size_t)r_v * sizeof(bf16), D, cudaMemcpyDeviceToDevice, st);
    if (e == cudaSuccess && L.A_tiled) {
        const bool pairs = mode == LORC_MODE_FULL && ctx->pair_style == LORC_ROPE_HALF_SPLIT;
        e = lorc_fast_retile_factor(L.A_cat, L.A_tiled, D, R, pairs ? r_k : 0, ctx->desc.d_head, st);
    }
    if (e == cudaSuccess && mode == LORC_MODE_LATENT) {
        e = cudaMemcpyAsync(L.B_k, B_k, (size_t)r_k * n * sizeof(bf16), cudaMemcpyDeviceToDevice, st);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(L.B_v, B_v, (size_t)r_v * n * sizeof(bf16), cudaMemcpyDeviceToDevice, st);
        if (e == cudaSuccess) e = lorc_generic_transpose(L.B_k, L.B_kT, r_k, n, st);
        if (e == cudaSuccess) e = lorc_generic_transpose(L.B_v, L.B_vT, r_v, n, st);
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) {
        free_layer(L);
        return fail_cuda(ctx, e, "lorc_load_factors");
    }
    L.loaded = 1;
    L.mode = mode;
    L.r_k = r_k;
    L.r_v = r_v;
    return LORC_OK;
}

size_t lorc_workspace_bytes(const lorc_ctx* ctx, int batch, int max_seq_len) {
    if (!ctx || batch <= 0 || max_seq_len <= 0) return 0;
    int S = generic_default_splits(max_seq_len);
    size_t gen = ws_layout(ctx, batch, S, ctx->n).total;
    size_t tc = lorc_align_up(lorc_tc_workspace_bytes(ctx, batch, max_seq_len), 256);
    return (gen > tc ? gen : tc) + staging_bytes(ctx, batch) + 256;
}

int lorc_set_workspace(lorc_ctx* ctx, void* workspace, size_t bytes) {
    if (!ctx) return LORC_ERR_ARG;
    if (workspace && ((uintptr_t)workspace & 255))
        return fail(ctx, LORC_ERR_ARG, "workspace must be 256-byte aligned");
    ctx->ws = workspace;
    ctx->ws_bytes = workspace ? bytes : 0;
    return LORC_OK;
}

int lorc_append(lorc_ctx* ctx, int layer, const lorc_cache* cache, const void* x, int T, void* stream) {
    LorcLayer* L;
    int rc = get_layer(ctx, layer, &L);
    if (rc) return rc;
    if (!x || T <= 0) return fail(ctx, LORC_ERR_ARG, "append: null x or non-positive T");
    if ((uintptr_t)x & 15) return fail(ctx, LORC_ERR_ARG, "append: x must be 16-byte aligned");
    CacheView cv;
    rc = check_cache(ctx, cache, *L, &cv);
    if (rc) return rc;
    if (T > cv.max_seq_len) return fail(ctx, LORC_ERR_ARG, "append: T exceeds max_seq_len");
    cudaStream_t st = (cudaStream_t)stream;
    int launches = 0;
    cudaError_t e;
    int path = 1;
    LorcStageTimer timer(ctx, LORC_STAGE_APPEND, st);
    if (!(ctx->desc.flags & LORC_FLAG_DEBUG_FP32) && lorc_tc_append_gemm_supported(ctx, *L, cv, T)) {
        // prompt-sized launch: a dense contraction, on tcgen05
        e = lorc_tc_append_gemm(ctx, *L, cv, (const bf16*)x, T, st, &launches);
        path = 2;
    } else if (!(ctx->desc.flags & LORC_FLAG_DEBUG_FP32) && lorc_tc_append_supported(ctx, *L, cv, T)) {
        e = lorc_tc_append(ctx, layer, *L, cv, (const bf16*)x, T, st, &launches);
        path = 2;
    } else {
        e = lorc_generic_append(ctx, *L, cv, (const bf16*)x, T, st, &launches);
    }
    ctx->launches += launches;
    ctx->last_path = path;
    if (e != cudaSuccess) return fail_cuda(ctx, e, "lorc_append");
    return LORC_OK;
}

static int decode_attn_impl(lorc_ctx* ctx, int layer, const lorc_cache* cache, const void* q, void* out,
                            int n_splits, void* stream, bool latent_out, const int32_t* pos0 = nullptr,
                            const int32_t* q_pos = nullptr, float* ml_out = nullptr) {
    LorcLayer* L;
    int rc = get_layer(ctx, layer, &L);
    if (rc) return rc;
    if (!q || !out) return fail(ctx, LORC_ERR_ARG, "decode_attn: null q or out");
    if (((uintptr_t)q & 15) || ((uintptr_t)out & 15))
        return fail(ctx, LORC_ERR_ARG, "decode_attn: q and out must be 16-byte aligned");
    if (n_splits < 0) return fail(ctx, LORC_ERR_ARG, "decode_attn: negative n_splits");
    if (latent_out && L->mode != LORC_MODE_LATENT)
        return fail(ctx, LORC_ERR_UNSUPPORTED, "decode_attn_latent_out: the layer is not compressed");
    if (q_pos && L->mode != LORC_MODE_LATENT)
        return fail(ctx, LORC_ERR_UNSUPPORTED, "decode_attn_shard: the layer is not compressed");
    CacheView cv;
    rc = check_cache(ctx, cache, *L, &cv);
    if (rc) return rc;
    if (!ctx->ws) return fail(ctx, LORC_ERR_WORKSPACE, "decode_attn: no workspace set");
    cudaStream_t st = (cudaStream_t)stream;
    const bool latent = (L->mode == LORC_MODE_LATENT);
    const int W = latent ? L->r_v : ctx->desc.d_head;
    int launches = 0;
    cudaError_t e;

    if (!(ctx->desc.flags & LORC_FLAG_DEBUG_FP32) && lorc_tc_decode_supported(ctx, *L, cv)) {
        size_t tc = lorc_tc_workspace_bytes(ctx, cv.batch, cv.max_seq_len);
        if (tc > ctx->ws_bytes) return fail(ctx, LORC_ERR_WORKSPACE, "decode_attn: workspace too small");
        e = lorc_tc_decode(ctx, layer, *L, cv, (const bf16*)q, (bf16*)out, n_splits, ctx->ws,
                           ctx->ws_bytes, st, &launches, latent_out, pos0, q_pos, ml_out);
        ctx->launches += launches;
        ctx->last_path = 2;
        if (e != cudaSuccess) return fail_cuda(ctx, e, "lorc_decode_attn (tensor-core path)");
        return LORC_OK;
    }

    int S = n_splits > 0 ? n_splits : generic_default_splits(cv.max_seq_len);
    int tiles = (cv.max_seq_len + LORC_GENERIC_TILE - 1) / LORC_GENERIC_TILE;
    if (S > tiles) S = tiles;
    if (S > LORC_MAX_SPLITS) S = LORC_MAX_SPLITS;
    // shrink the split count until the partial results fit the workspace
    while (S > 1 && ws_layout(ctx, cv.batch, S, W).total > ctx->ws_bytes) --S;
    WsLayout w = ws_layout(ctx, cv.batch, S, W);
    if (w.total > ctx->ws_bytes) return fail(ctx, LORC_ERR_WORKSPACE, "decode_attn: workspace too small");
    float* part_ml = (float*)((char*)ctx->ws + w.off_ml);
    float* part_o = (float*)((char*)ctx->ws + w.off_o);
    e = lorc_generic_decode(ctx, *L, cv, (const bf16*)q, (bf16*)out, S, part_ml, part_o, st, &launches, latent_out, 1,
                            pos0, q_pos, ml_out);
    ctx->launches += launches;
    ctx->last_path = lorc_full_decode_supported(ctx, *L) ? 3 : 1;
    if (e != cudaSuccess) return fail_cuda(ctx, e, "lorc_decode_attn");
    return LORC_OK;
}

int lorc_decode_attn(lorc_ctx* ctx, int layer, const lorc_cache* cache, const void* q, void* out,
                     int n_splits, void* stream) {
    return decode_attn_impl(ctx, layer, cache, q, out, n_splits, stream, false);
}

int lorc_decode_attn_latent_out(lorc_ctx* ctx, int layer, const lorc_cache* cache, const void* q, void* o_lat,
                                int n_splits, void* stream) {
    return decode_attn_impl(ctx, layer, cache, q, o_lat, n_splits, stream, true);
}

int lorc_decode_attn_shard(lorc_ctx* ctx, int layer, const lorc_cache* cache, const void* q, const int32_t* pos0,
                           const int32_t* q_pos, void* out, float* ml, int n_splits, void* stream) {
    if (!ctx) return LORC_ERR_ARG;
    if (!pos0 || !q_pos || !ml) return fail(ctx, LORC_ERR_ARG, "decode_attn_shard: null pos0, q_pos or ml");
    return decode_attn_impl(ctx, layer, cache, q, out, n_splits, stream, false, pos0, q_pos, ml);
}

int lorc_merge_shards(lorc_ctx* ctx, int n_shards, const void* outs, const float* mls, void* out, int batch, void* stream) {
    if (!ctx) return LORC_ERR_ARG;
    if (!outs || !mls || !out || batch <= 0 || n_shards <= 0 || n_shards > 64)
        return fail(ctx, LORC_ERR_ARG, "merge_shards: null pointer, or batch / n_shards out of range (1..64 shards)");
    int launches = 0;
    cudaError_t e = lorc_generic_merge_shards(ctx, n_shards, (const bf16*)outs, mls, (bf16*)out, batch, (cudaStream_t)stream,
                                              &launches);
    ctx->launches += launches;
    if (e != cudaSuccess) return fail_cuda(ctx, e, "lorc_merge_shards");
    return LORC_OK;
}

size_t lorc_prefill_workspace_bytes(const lorc_ctx* ctx, int batch, int max_seq_len, int T) {
    if (!ctx || batch <= 0 || max_seq_len <= 0 || T <= 0) return 0;
    int S = generic_default_splits(max_seq_len);
    size_t gen = ws_layout(ctx, batch * T, S, ctx->n).total;
    size_t tc = lorc_tc_workspace_bytes(ctx, batch, max_seq_len) ? lorc_tc_prefill_scratch_bytes(ctx, batch, max_seq_len, T) : 0;
    return (gen > tc ? gen : tc) + 256;
}

int lorc_prefill_attn(lorc_ctx* ctx, int layer, const lorc_cache* cache, const void* q, void* out, int T, void* stream) {
    LorcLayer* L;
    int rc = get_layer(ctx, layer, &L);
    if (rc) return rc;
    if (!q || !out || T <= 0) return fail(ctx, LORC_ERR_ARG, "prefill_attn: null q or out, or non-positive T");
    if (((uintptr_t)q & 15) || ((uintptr_t)out & 15))
        return fail(ctx, LORC_ERR_ARG, "prefill_attn: q and out must be 16-byte aligned");
    CacheView cv;
    rc = check_cache(ctx, cache, *L, &cv);
    if (rc) return rc;
    if (T > cv.max_seq_len) return fail(ctx, LORC_ERR_ARG, "prefill_attn: T exceeds max_seq_len");
    if (!ctx->ws) return fail(ctx, LORC_ERR_WORKSPACE, "prefill_attn: no workspace set");
    cudaStream_t st = (cudaStream_t)stream;
    int launches = 0;
    cudaError_t e;
    if (!(ctx->desc.flags & LORC_FLAG_DEBUG_FP32) && lorc_tc_prefill_supported(ctx, *L, cv)) {
        if (lorc_tc_prefill_scratch_bytes(ctx, cv.batch, cv.max_seq_len, T) > ctx->ws_bytes)
            return fail(ctx, LORC_ERR_WORKSPACE, "prefill_attn: workspace too small (see lorc_prefill_workspace_bytes)");
        LorcStageTimer timer(ctx, LORC_STAGE_SCORE, st);
        e = lorc_tc_prefill(ctx, layer, *L, cv, (const bf16*)q, (bf16*)out, T, ctx->ws, ctx->ws_bytes, st, &launches);
        ctx->launches += launches;
        ctx->last_path = 2;
        if (e != cudaSuccess) return fail_cuda(ctx, e, "lorc_prefill_attn (tensor-core path)");
        return LORC_OK;
    }
    // plain kernels: every (sequence, query) is a decode query over the sequence cut after its own token
    const bool latent = (L->mode == LORC_MODE_LATENT);
    const int W = latent ? L->r_v : ctx->desc.d_head;
    int S = generic_default_splits(cv.max_seq_len);
    int tiles = (cv.max_seq_len + LORC_GENERIC_TILE - 1) / LORC_GENERIC_TILE;
    if (S > tiles) S = tiles;
    while (S > 1 && ws_layout(ctx, cv.batch * T, S, W).total > ctx->ws_bytes) --S;
    WsLayout w = ws_layout(ctx, cv.batch * T, S, W);
    if (w.total > ctx->ws_bytes)
        return fail(ctx, LORC_ERR_WORKSPACE, "prefill_attn: workspace too small (see lorc_prefill_workspace_bytes)");
    float* part_ml = (float*)((char*)ctx->ws + w.off_ml);
    float* part_o = (float*)((char*)ctx->ws + w.off_o);
    e = lorc_generic_decode(ctx, *L, cv, (const bf16*)q, (bf16*)out, S, part_ml, part_o, st, &launches, false, T);
    ctx->launches += launches;
    ctx->last_path = 1;
    if (e != cudaSuccess) return fail_cuda(ctx, e, "lorc_prefill_attn");
    return LORC_OK;
}

int lorc_decode_step_host(lorc_ctx* ctx, int layer, const lorc_cache* cache, const void* x_host,
                          const void* q_host, void* out_host, int n_splits, void* stream) {
    LorcLayer* L;
    int rc = get_layer(ctx, layer, &L);
    if (rc) return rc;
    if (!x_host || !q_host || !out_host) return fail(ctx, LORC_ERR_ARG, "decode_step_host: null host buffer");
    if (!cache || cache->batch <= 0) return fail(ctx, LORC_ERR_ARG, "decode_step_host: bad cache");
    if (!ctx->ws) return fail(ctx, LORC_ERR_WORKSPACE, "decode_step_host: no workspace set");
    const lorc_model_desc& d = ctx->desc;
    size_t xb = (size_t)cache->batch * d.d_model * sizeof(bf16);
    size_t qb = (size_t)cache->batch * d.n_q_heads * d.d_head * sizeof(bf16);
    if (ctx->ws_bytes < staging_bytes(ctx, cache->batch) + 256)
        return fail(ctx, LORC_ERR_WORKSPACE, "decode_step_host: workspace too small");
    char* end = (char*)ctx->ws + (ctx->ws_bytes / 256) * 256;
    char* out_d = end - lorc_align_up(qb, 256);
    char* q_d = out_d - lorc_align_up(qb, 256);
    char* x_d = q_d - lorc_align_up(xb, 256);
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = cudaMemcpyAsync(x_d, x_host, xb, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(q_d, q_host, qb, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "decode_step_host: host to device copy");
    // lend the attention call only the part of the workspace in front of the staging
    size_t saved = ctx->ws_bytes;
    ctx->ws_bytes = (size_t)(x_d - (char*)ctx->ws);
    rc = lorc_append(ctx, layer, cache, x_d, 1, stream);
    if (rc == LORC_OK) rc = lorc_decode_attn(ctx, layer, cache, q_d, out_d, n_splits, stream);
    ctx->ws_bytes = saved;
    if (rc) return rc;
    e = cudaMemcpyAsync(out_host, out_d, qb, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "decode_step_host: device to host copy");
    return LORC_OK;
}

// ---------------------------------------------------------------------------------------------------------------
// Self-test of the bounded wait: one thread waits, with the library's own wait routine, on a barrier that nothing
// ever signals; when the (short) limit runs out it reports LORC_ERR_TIMEOUT through the status word like any kernel
// of the library would, and returns.
// ---------------------------------------------------------------------------------------------------------------
__global__ void wait_expiry_kernel(unsigned long long limit_ns, int* status) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        sm100::mbar_init(&bar, 1);
        sm100::fence_barrier_init();
        if (!sm100::mbar_wait_for(&bar, 0, limit_ns)) lorc_set_status(status, LORC_ERR_TIMEOUT);
    }
}

int lorc_selftest_wait_expiry(lorc_ctx* ctx, unsigned long long limit_ns, void* stream) {
    if (!ctx) return LORC_ERR_ARG;
    if (limit_ns == 0 || limit_ns > 1000000000ull)
        return fail(ctx, LORC_ERR_ARG, "selftest_wait_expiry: the limit must be between 1 ns and 1 s");
    wait_expiry_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(limit_ns, ctx->status_dev);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail_cuda(ctx, e, "lorc_selftest_wait_expiry");
    ctx->launches += 1;
    return LORC_OK;
}

int lorc_sync_status(lorc_ctx* ctx, void* stream) {
    if (!ctx) return LORC_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return fail_cuda(ctx, e, "lorc_sync_status: synchronize");
    int code = 0;
    e = cudaMemcpy(&code, ctx->status_dev, sizeof(int), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && code != 0) e = cudaMemset(ctx->status_dev, 0, sizeof(int));
    if (e != cudaSuccess) return fail_cuda(ctx, e, "lorc_sync_status: status read");
    if (code != 0) {
        static const char* names[] = {"ok",
                                      "bad argument",
                                      "bad layer",
                                      "cache capacity exceeded or page index out of range",
                                      "attention over an empty sequence",
                                      "device-side wait timed out",
                                      "cuda error",
                                      "unsupported",
                                      "workspace"};
        ctx->err = std::string("device status: ") + ((code > 0 && code < 9) ? names[code] : "unknown");
    }
    return code;
}

const char* lorc_last_error(const lorc_ctx* ctx) { return ctx ? ctx->err.c_str() : "null context"; }

int lorc_last_path(const lorc_ctx* ctx) { return ctx ? ctx->last_path : 0; }

int lorc_profile_read(lorc_ctx* ctx, float* ms, int64_t* launches) {
    if (!ctx) return LORC_ERR_ARG;
    float acc[LORC_N_STAGES] = {0.f, 0.f, 0.f, 0.f};
    int64_t cnt[LORC_N_STAGES] = {0, 0, 0, 0};
    if (ctx->prof) {
        for (auto& r : ctx->prof->pending) {
            float t = 0.f;
            cudaError_t e = cudaEventSynchronize(r.e1);
            if (e == cudaSuccess) e = cudaEventElapsedTime(&t, r.e0, r.e1);
            if (e != cudaSuccess) return fail_cuda(ctx, e, "lorc_profile_read");
            if (r.stage >= 0 && r.stage < LORC_N_STAGES) {
                acc[r.stage] += t;
                cnt[r.stage] += 1;
            }
            ctx->prof->pool.push_back(r.e0);
            ctx->prof->pool.push_back(r.e1);
        }
        ctx->prof->pending.clear();
    }
    for (int i = 0; i < LORC_N_STAGES; ++i) {
        if (ms) ms[i] = acc[i];
        if (launches) launches[i] = cnt[i];
    }
    return LORC_OK;
}

int lorc_profile_enable(lorc_ctx* ctx, int on) {
    if (!ctx) return LORC_ERR_ARG;
    if (on && !ctx->prof) {
        ctx->prof = new (std::nothrow) LorcProfile();
        if (!ctx->prof) return fail(ctx, LORC_ERR_CUDA, "lorc_profile_enable: out of host memory");
    }
    ctx->prof_on = on != 0;
    return LORC_OK;
}

int64_t lorc_launch_count(const lorc_ctx* ctx) { return ctx ? ctx->launches : 0; }

}  // extern "C"
