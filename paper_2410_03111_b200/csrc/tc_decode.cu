// Tensor-core decode attention over the latent cache (sm_100a: TMA + tcgen05 + TMEM): host side.
//
// Three kernels per layer, chained by programmatic dependent launch:
//   score kernel    (tc_score.cu)  key reconstruction on tcgen05, RoPE and q.k in its epilogue, softmax numerators
//                                  against per-quarter-tile integer references, written as the PV kernel's MMA operand;
//   PV kernel       (tc_pv.cu)     exact change of reference, P.C_V on tcgen05 split by latent column blocks;
//   up-projection   (tc_pv.cu)     out = o_lat . B_V on tcgen05.
// Keys and values never exist in memory.
#include <math.h>

#include "sm100_ptx.cuh"
#include "tc_kernels.cuh"

namespace {
constexpr int TILE = 128;            // tokens per tile
constexpr int KC = 64;               // latent columns per TMA box
}  // namespace

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
struct LorcTcLayer {
    bool has_bkt = false;
    CUtensorMap mapBKT, mapBVT;         // B_K^T in 64 x 128 swizzled boxes; B_V^T in 64 x 32 swizzled boxes
    CUtensorMap mapBVT128;              // B_V^T in 64 x 128 boxes (reconstruction of values for prompt processing)
    // cache maps are rebuilt only when the cache geometry or pointers change
    const void* k_ptr = nullptr;
    const void* v_ptr = nullptr;
    long long key_dims[6] = {0, 0, 0, 0, 0, 0};
    CUtensorMap mapCK, mapCV;
};

struct LorcTcState {
    float2* rope_tile = nullptr;
    unsigned* rowmax = nullptr;         // [rowmax_cap] row maxima of the softmax, see lorc_tc_decode
    std::vector<unsigned*> retired;     // smaller tables of earlier calls, freed with the context
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
        for (unsigned* r : ctx->tc->retired) cudaFree(r);
        delete ctx->tc;
        ctx->tc = nullptr;
    }
}

void lorc_tc_invalidate_layer(lorc_ctx* ctx, int layer) {
    if (ctx->tc && layer >= 0 && layer < (int)ctx->tc->layers.size()) ctx->tc->layers[layer] = LorcTcLayer();
}

static bool tc_shape_ok(const lorc_ctx* ctx) {
    const lorc_model_desc& d = ctx->desc;
    return d.d_head == 128 && (d.rope_style == LORC_ROPE_HALF_SPLIT || d.rope_style == LORC_ROPE_NONE) && (d.n_kv_heads % 2) == 0 &&
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

static size_t tc_image_area_bytes(const lorc_ctx* ctx, int batch, int max_seq_len) {
    const size_t tiles = (size_t)((max_seq_len + TILE - 1) / TILE);
    return lorc_align_up((size_t)batch * tiles * lorc_tc_image_bytes(ctx->desc.n_q_heads), 256);
}

// the absorbed query of layers without rotation sits between the images and the PV scratch
static size_t tc_absorbed_bytes(const lorc_ctx* ctx, int batch) {
    return ctx->desc.rope_style == LORC_ROPE_NONE ? lorc_tc_absorbed_scratch_bytes(ctx, batch) : 0;
}

size_t lorc_tc_workspace_bytes(const lorc_ctx* ctx, int batch, int max_seq_len) {
    if (!tc_shape_ok(ctx)) return 0;
    return tc_image_area_bytes(ctx, batch, max_seq_len) + tc_absorbed_bytes(ctx, batch) +
           lorc_tc_pv_scratch_bytes(ctx, batch, max_seq_len);
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

// One-time tables and attributes of the context, the layer's factor maps, and the cache maps for this call.
static cudaError_t tc_prepare(lorc_ctx* ctx, LorcTcState* T, LorcTcLayer& TL, const LorcLayer& L, const CacheView& cv,
                              cudaStream_t st) {
    const lorc_model_desc& d = ctx->desc;
    if (!T->rope_tile) {
        cudaError_t e = cudaMalloc(&T->rope_tile, sizeof(float2) * 64 * 33);
        if (e == cudaSuccess) e = lorc_tc_rope_tile_fill(T->rope_tile, d.rope_theta, st);
        if (e != cudaSuccess) return e;
    }
    if (!T->attrs_set) {
        // per context, hence per device: the attribute belongs to the device's copy of the kernel
        cudaError_t e = lorc_tc_score_set_attrs();
        if (e == cudaSuccess) e = lorc_tc_pv_set_attrs();
        if (e == cudaSuccess) e = lorc_tc_absorbed_set_attrs();
        if (e == cudaSuccess) e = lorc_tc_prefill_set_attrs();
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
        uint32_t b3[2] = {KC, 128};
        if (!lorc_make_tmap_bf16(&TL.mapBVT128, L.B_vT, 2, d2, s2, b3)) return cudaErrorInvalidValue;
        TL.has_bkt = true;
    }
    if (!build_cache_maps(TL, L, cv)) return cudaErrorInvalidValue;

    return cudaSuccess;
}

cudaError_t lorc_tc_decode(lorc_ctx* ctx, int layer, const LorcLayer& L, const CacheView& cv, const bf16* q,
                           bf16* out, int n_splits, void* ws, size_t ws_bytes, cudaStream_t st, int* launches,
                           bool latent_out, const int32_t* pos0, const int32_t* q_pos, float* ml_out) {
    LorcTcState* T = tc_state(ctx);
    LorcTcLayer& TL = T->layers[layer];
    const lorc_model_desc& d = ctx->desc;
    {
        cudaError_t e0 = tc_prepare(ctx, T, TL, L, cv, st);
        if (e0 != cudaSuccess) return e0;
    }
    const int tiles = (cv.max_seq_len + TILE - 1) / TILE;
    const size_t img_area = tc_image_area_bytes(ctx, cv.batch, cv.max_seq_len);
    const size_t abs_area = tc_absorbed_bytes(ctx, cv.batch);
    if (img_area + abs_area >= ws_bytes) return cudaErrorMemoryAllocation;
    uint8_t* pimg = (uint8_t*)ws;
    bf16* qabs = (bf16*)((char*)ws + img_area);
    void* pv_scratch = (char*)ws + img_area + abs_area;
    LorcPvPlan plan;
    lorc_tc_pv_plan(ctx, L, cv, n_splits, ws_bytes - img_area - abs_area, &plan);
    if (!plan.fits) return cudaErrorMemoryAllocation;
    // Row maxima [batch, H_q]: all zero between calls (the up-projection kernel clears what the score kernel raised).
    // Owned by the library because that invariant must hold from the first call on.  The table only ever grows, and a
    // block that was handed to earlier launches is kept until the context dies (a captured graph may still name it).
    const size_t rm_need = (size_t)cv.batch * d.n_q_heads;
    if (rm_need > T->rowmax_cap) {
        unsigned* fresh = nullptr;
        cudaError_t e = cudaMalloc(&fresh, rm_need * sizeof(unsigned));
        if (e != cudaSuccess) return e;
        if (T->rowmax) T->retired.push_back(T->rowmax);
        T->rowmax = fresh;
        T->rowmax_cap = rm_need;
        T->rowmax_dirty = true;
    }
    if (T->rowmax_dirty) {
        cudaError_t e = cudaMemsetAsync(T->rowmax, 0, T->rowmax_cap * sizeof(unsigned), st);
        if (e != cudaSuccess) return e;
    }
    T->rowmax_dirty = true;
    {
        LorcStageTimer timer(ctx, LORC_STAGE_SCORE, st);
        int* zero = (int*)((char*)pv_scratch + plan.off_done);
        cudaError_t e;
        if (d.rope_style == LORC_ROPE_NONE)
            // no rotation between the key up-projection and the dot product: the up-projection moves to the query
            e = lorc_tc_score_absorbed_launch(ctx, L, cv, TL.mapCK, q, qabs, pimg, T->rowmax, tiles, zero,
                                              cv.batch * plan.n_blk, st, launches);
        else
            e = lorc_tc_score_launch(ctx, L, cv, TL.mapCK, TL.mapBKT, q, pimg, T->rowmax,
                                     reinterpret_cast<const float4*>(T->rope_tile), tiles, zero, cv.batch * plan.n_blk, pos0,
                                     q_pos, st, launches);
        if (e != cudaSuccess) return e;
    }
    const cudaError_t e2 = lorc_tc_pv_launch(ctx, L, cv, TL.mapCV, TL.mapBVT, pimg, T->rowmax, tiles, plan, pv_scratch,
                                             out, latent_out, ml_out, st, launches);
    if (e2 == cudaSuccess) T->rowmax_dirty = false;
    return e2;
}

bool lorc_tc_prefill_supported(const lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv) {
    return lorc_tc_decode_supported(ctx, L, cv);
}

cudaError_t lorc_tc_prefill(lorc_ctx* ctx, int layer, const LorcLayer& L, const CacheView& cv, const bf16* q, bf16* out,
                            int T_new, void* ws, size_t ws_bytes, cudaStream_t st, int* launches) {
    LorcTcState* T = tc_state(ctx);
    LorcTcLayer& TL = T->layers[layer];
    cudaError_t e = tc_prepare(ctx, T, TL, L, cv, st);
    if (e != cudaSuccess) return e;
    if (lorc_tc_prefill_scratch_bytes(ctx, cv.batch, cv.max_seq_len, T_new) > ws_bytes) return cudaErrorMemoryAllocation;
    return lorc_tc_prefill_launch(ctx, L, cv, TL.mapCK, TL.mapCV, TL.mapBKT, TL.mapBVT128, q, out, T_new, ws, st, launches);
}
