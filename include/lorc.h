/*
 * lorc.h - C ABI of the B200 (sm_100a) latent-KV decode-attention library.
 *
 * The library implements the run-time half of LoRC (arXiv 2410.03111): the KV
 * cache of every layer holds rank-r latents C_K = X A_K, C_V = X A_V instead of
 * keys and values, where W_k ~= A_K B_K and W_v ~= A_V B_V are truncated-SVD
 * factorisations (A = U_r Sigma_r, B = V_r^T; Sec. 3.1, Algorithm 1), and decode
 * attention runs directly on the latents.
 *
 * Conventions
 *   - Row-vector convention K = X W (Preliminary section).  D = d_model,
 *     n = n_kv_heads * d_head, query head h reads KV head h / (n_q_heads / n_kv_heads)
 *     (Sec. 3.3).
 *   - All tensors are dense, row-major, bfloat16 unless stated.  "device" pointers
 *     are CUDA device memory owned by the caller; the library never frees or
 *     reallocates caller memory.  "host" pointers are ordinary host memory.
 *   - `stream` arguments are a cudaStream_t passed as void* (NULL = default stream).
 *     Calls enqueue work on that stream and return without synchronising unless
 *     stated.
 *   - Every function returns LORC_OK (0) or a positive LORC_ERR_* code; nothing
 *     throws, aborts or traps.  lorc_last_error() gives a text for the last failure
 *     on that context.  Problems only a kernel can see (a page index outside the
 *     pool, a position beyond the capacity, a bounded wait that ran out) set a
 *     device status word that lorc_sync_status() returns.
 *   - Positions are 0-based.  RoPE angle for pair j at position p is
 *     p * rope_theta^(-2j/d_head).
 */
#ifndef LORC_H_
#define LORC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* status codes */
#define LORC_OK 0
#define LORC_ERR_ARG 1          /* null pointer, bad size, bad alignment */
#define LORC_ERR_LAYER 2        /* layer index out of range or factors not loaded */
#define LORC_ERR_CAPACITY 3     /* position beyond cache capacity / page index outside the pool */
#define LORC_ERR_EMPTY 4        /* a sequence with zero cached tokens was attended */
#define LORC_ERR_TIMEOUT 5      /* a bounded device-side wait expired */
#define LORC_ERR_CUDA 6         /* a CUDA runtime / driver call failed */
#define LORC_ERR_UNSUPPORTED 7  /* shape outside what the kernels implement */
#define LORC_ERR_WORKSPACE 8    /* workspace missing or too small */

/* layer modes */
#define LORC_MODE_LATENT 0      /* compressed layer: cache holds rank-r latents */
#define LORC_MODE_FULL 1        /* layer skipped by the compression schedule: ordinary KV cache */

/* RoPE pairing */
#define LORC_ROPE_HALF_SPLIT 0  /* pair (j, j + d_head/2) */
#define LORC_ROPE_INTERLEAVED 1 /* pair (2j, 2j + 1)      */
#define LORC_ROPE_NONE 2        /* no rotation at attention time: a model without rotary embedding, or one whose
                                   rotation does not touch the compressed keys.  The scores then take the absorbed
                                   form of Sec. 3.1 (the W_q' equation), s = (B_K q) . c: keys are never reconstructed */

/* context flags */
#define LORC_FLAG_DEBUG_FP32 1  /* run the plain fp32 CUDA-core kernels everywhere (debug path) */
#define LORC_FLAG_PROFILE 2     /* bracket every kernel with CUDA events (see lorc_profile_read) */

/* stages reported by lorc_profile_read */
#define LORC_STAGE_APPEND 0     /* cache write */
#define LORC_STAGE_SCORE 1      /* tensor-core path: key reconstruction + RoPE + scores + softmax numerators;
                                   plain kernels: the whole split-context attention kernel */
#define LORC_STAGE_PV 2         /* tensor-core path: change of softmax reference + P.C_V */
#define LORC_STAGE_COMBINE 3    /* value up-projection (plain kernels: split merge + up-projection) */
#define LORC_N_STAGES 4

typedef struct lorc_ctx lorc_ctx;

/* Model geometry, fixed for the life of a context.  Shapes follow the paper's
 * "Model Architectures" table (layers, heads, KV heads, head dimension, model
 * dimension).  max_pos bounds every position used with this context (the
 * library builds a cos/sin table of max_pos rows at creation). */
typedef struct lorc_model_desc {
    int32_t n_layers;
    int32_t d_model;
    int32_t n_q_heads;
    int32_t n_kv_heads;
    int32_t d_head;      /* 64 or 128 */
    int32_t rope_style;  /* LORC_ROPE_* */
    int32_t max_pos;     /* positions are in [0, max_pos) */
    int32_t flags;       /* LORC_FLAG_* */
    double rope_theta;
} lorc_model_desc;

/* One layer's cache for a batch of sequences.  The cache-size model of the
 * Preliminary section (b x N x h x d per layer) becomes b x N x r here.
 *
 * Contiguous layout (page_table == NULL):
 *     k = C_K[batch][seq_stride][r_k], v = C_V[batch][seq_stride][r_v]
 * Paged layout (page_table != NULL):
 *     k = pool_K[n_pages][page_size][r_k], v = pool_V[n_pages][page_size][r_v],
 *     page_table[batch][max_pages_per_seq] (device int32) gives the physical page
 *     of each logical page of each sequence.
 * In LORC_MODE_FULL layers the row width is n = n_kv_heads*d_head for both, and
 * k holds keys already rotated at their positions.
 *
 * seq_lens[batch] (device int32, caller-owned, never written by the library) is
 * the number of cached tokens of each sequence.  max_seq_len is a host-side upper
 * bound on seq_lens used to size launches and scratch; it must not exceed the
 * capacity (seq_stride, or max_pages_per_seq*page_size).  The kernels enforce
 * seq_lens[s] <= max_seq_len (rounded up to a multiple of 128 on the tensor-core
 * path) and seq_lens[s] <= max_pos: a longer sequence is treated as empty and the
 * status word is set to LORC_ERR_CAPACITY; nothing is read or written out of
 * bounds.  Rows at positions >= seq_lens[s] may be read by tile loads; they must
 * hold finite numbers (zero the cache once when allocating it). */
typedef struct lorc_cache {
    void* k;                      /* device */
    void* v;                      /* device */
    const int32_t* page_table;    /* device, or NULL for the contiguous layout */
    const int32_t* seq_lens;      /* device */
    int32_t batch;
    int32_t max_seq_len;
    int32_t page_size;            /* paged: tokens per page (multiple of 16) */
    int32_t max_pages_per_seq;    /* paged */
    int32_t n_pages;              /* paged: pages in the pool */
    int32_t reserved;
    int64_t seq_stride;           /* contiguous: rows between consecutive sequences */
} lorc_cache;

/* Create / destroy a context.  Creation allocates only library-owned tables
 * (the cos/sin table of max_pos x d_head/2 pairs and a status word; per-layer
 * factor copies come later, in lorc_load_factors).  Uses the current CUDA device.
 * Errors: ARG (null, non-positive sizes, n_q_heads not a multiple of
 * n_kv_heads), UNSUPPORTED (d_head not 64/128, more than 8 query heads per KV
 * head), CUDA. */
int lorc_create(const lorc_model_desc* desc, lorc_ctx** out);
int lorc_destroy(lorc_ctx* ctx);

/* Hand the factors of one layer to the library (Sec. 3.1; Algorithm 1, the two
 * "Matrix Compression" blocks).  Setup call: it allocates library-owned device
 * copies in the layouts the kernels want and synchronises `stream` before it
 * returns, so the caller's buffers may be released afterwards.
 *   mode LATENT: A_k [D, r_k], B_k [r_k, n], A_v [D, r_v], B_v [r_v, n], device bf16.
 *                r_k, r_v in [8, n], multiples of 8.
 *   mode FULL  : A_k = W_k [D, n], A_v = W_v [D, n]; B_k, B_v, r_k, r_v ignored
 *                (a layer the schedule leaves uncompressed, Algorithm 1 "skip").
 * Errors: ARG, LAYER, CUDA. */
int lorc_load_factors(lorc_ctx* ctx, int layer, int mode, int r_k, int r_v,
                      const void* A_k, const void* B_k, const void* A_v, const void* B_v,
                      void* stream);

/* Scratch memory for decode attention (split-context partial results) and for
 * the host-buffer entry point (staging).  The caller allocates `bytes` of device
 * memory (256-byte aligned) and lends it to the context until replaced or the
 * context is destroyed.  lorc_workspace_bytes returns a size sufficient for any
 * layer of this context with the given batch and max_seq_len. */
size_t lorc_workspace_bytes(const lorc_ctx* ctx, int batch, int max_seq_len);
int lorc_set_workspace(lorc_ctx* ctx, void* workspace, size_t bytes);

/* Cache write (Sec. 3.1: the cache stores X times the Sigma-carrying factor;
 * Appendix "Adjusted Position Embedding": compressed keys are stored un-rotated).
 *   x [batch, T, D] device bf16: T new tokens for every sequence of the cache.
 *   seq_lens must already count the new tokens: token i of sequence s is written
 *   at position seq_lens[s] - T + i.
 * LATENT layers write C_K = x A_K, C_V = x A_V (fp32 accumulation, one rounding
 * to bf16).  FULL layers write RoPE(x W_k) and x W_v.
 * Errors: ARG, LAYER, UNSUPPORTED; CAPACITY through the status word. */
int lorc_append(lorc_ctx* ctx, int layer, const lorc_cache* cache, const void* x, int T,
                void* stream);

/* Decode attention for one layer (Preliminary section's Attention(Q,K,V) with the
 * GQA repeat of Sec. 3.3 and the rotation placement of the appendix):
 *   q   [batch, n_q_heads, d_head] device bf16, un-rotated, one query per sequence
 *       at position seq_lens[s] - 1;
 *   out [batch, n_q_heads, d_head] device bf16.
 * For every sequence s and head h (g = KV head of h):
 *   k_n = B_K[:, g]^T C_K[n], rotated at n;  q^ = RoPE(q, seq_lens[s]-1);
 *   p = softmax_n(q^ . k_n / sqrt(d_head)),  out = (sum_n p_n C_V[n]) B_V[:, g]
 * over n in [0, seq_lens[s]).  Keys and values are never written to memory.
 * n_splits = 0 lets the library choose how many CTAs share one sequence's context;
 * a positive value asks for that many shares (context splits of the plain kernels
 * and of the uncompressed mode; context shares per latent column block of the
 * tensor-core path), clamped to what the workspace holds.  Uses the workspace.
 * A sequence with seq_lens[s] <= 0 gets a row of zeros and sets status EMPTY.
 * The first call on a context, and the first call with a larger batch than any
 * before, sets up small library-owned tables (an in-tile rotation table, one word
 * per sequence and head for the softmax row maxima) with cudaMalloc: make those
 * calls outside any stream capture.  A table handed to earlier calls is kept until
 * lorc_destroy, so CUDA graphs captured before a larger batch showed up stay valid.
 * Calls on one context must not overlap on the GPU (they share the workspace and
 * those tables).
 * Errors: ARG, LAYER, WORKSPACE, UNSUPPORTED. */
int lorc_decode_attn(lorc_ctx* ctx, int layer, const lorc_cache* cache, const void* q, void* out,
                     int n_splits, void* stream);

/* Prompt processing: attention of the T newest tokens of every sequence (a whole prompt, or one chunk of it) over the
 * latent cache.  Preliminary section's Attention(Q, K, V) with the usual causal mask; keys and values come from the
 * cached latents as in lorc_decode_attn (Sec. 3.1), rotated at attention time (appendix).
 *   q   [batch, T, n_q_heads, d_head] device bf16, un-rotated; out the same shape.
 *   The T tokens must already be in the cache (lorc_append first) and counted in seq_lens: query t of sequence s sits
 *   at position seq_lens[s] - T + t and attends to positions 0 .. seq_lens[s] - T + t (the cached prefix in full, the
 *   new chunk causally).  With T = 1 the result equals lorc_decode_attn's.
 * On the tensor-core path every key and value of the layer is reconstructed once into the workspace (a transient
 * fp16 buffer: the method's saving is in the cache, not in this scratch; a reconstructed key or value element must
 * stay below 65504 in magnitude), then attended with a flash-attention
 * kernel; every call reconstructs the whole cached sequence, so chunks should be large.  Needs a workspace of
 * lorc_prefill_workspace_bytes(ctx, batch, max_seq_len, T).  A sequence with seq_lens[s] < T sets status ARG.
 * Errors: ARG, LAYER, WORKSPACE; CAPACITY / EMPTY through the status word. */
size_t lorc_prefill_workspace_bytes(const lorc_ctx* ctx, int batch, int max_seq_len, int T);
int lorc_prefill_attn(lorc_ctx* ctx, int layer, const lorc_cache* cache, const void* q, void* out, int T, void* stream);

/* Decode attention that stops before the value up-projection (Sec. 3.1, the W_o' equation: the orthonormal value
 * factor can be folded into the output projection, W_o' = B_V,g W_o,h stacked over the heads).  Same arguments as
 * lorc_decode_attn except the result:
 *   o_lat [batch, n_q_heads, r_v] device bf16,  o_lat[s, h, :] = sum_n p_n C_V[n, :]  (softmax as in lorc_decode_attn),
 * so that lorc_decode_attn's out[s, h, :] = o_lat[s, h, :] B_V[:, g(h)].  Compressed (LATENT) layers only.
 * Errors: as lorc_decode_attn, UNSUPPORTED for an uncompressed layer. */
int lorc_decode_attn_latent_out(lorc_ctx* ctx, int layer, const lorc_cache* cache, const void* q, void* o_lat,
                                int n_splits, void* stream);

/* Context-sharded decode: one sequence's cache split over several GPUs by position, every GPU attending to its own
 * shard, and the per-shard results merged.  (The method shards by sequence without any exchange; splitting ONE long
 * context is the case that needs one, and a small one: d_head + 2 numbers per sequence and head.)
 *
 * lorc_decode_attn_shard: like lorc_decode_attn, but the cache of this call holds the tokens of sequence s at positions
 * pos0[s] .. pos0[s] + seq_lens[s] - 1 (device int32 [batch]) and the query sits at position q_pos[s] (device int32
 * [batch]; not before the shard's last token, below max_pos).  Results:
 *   out [batch, n_q_heads, d_head] bf16   the attention output over this shard alone (zeros for an empty shard);
 *   ml  [batch, n_q_heads, 2] fp32        M, a reference for the scores in log2 units, and L = sum_n 2^(s_n - M).
 * An empty shard (seq_lens[s] = 0) is not an error here: it reports L = 0.  Compressed (LATENT) layers only.
 *
 * lorc_merge_shards: outs [n_shards, batch, n_q_heads, d_head] bf16 and mls [n_shards, batch, n_q_heads, 2] fp32 (the
 * shards' results, gathered on this GPU, e.g. with an NCCL all-gather) ->
 *   out = sum_r w_r out_r / sum_r w_r,  w_r = L_r 2^(M_r - max_r M_r),
 * the softmax over the union of the shards.  n_shards <= 64.  Status EMPTY when no shard held a token. */
int lorc_decode_attn_shard(lorc_ctx* ctx, int layer, const lorc_cache* cache, const void* q, const int32_t* pos0,
                           const int32_t* q_pos, void* out, float* ml, int n_splits, void* stream);
int lorc_merge_shards(lorc_ctx* ctx, int n_shards, const void* outs, const float* mls, void* out, int batch, void* stream);

/* Decode attention without any caller-provided or freshly allocated scratch.
 * (The paper has no counterpart to this call; it exists for deployment reasons.)
 * Meant for hosts that cannot allocate device memory when they call in: a server
 * that gave the whole GPU to its own memory pool at start-up, or a plug-in that
 * receives tensors but no allocator.  Same arguments, meaning and result as
 * lorc_decode_attn, computed by the split-context kernels (the plain CUDA-core
 * ones; for an uncompressed layer with 128-wide heads the mma.sync streaming
 * kernel, as lorc_last_path reports), but the per-split
 * partial results live in a fixed array of LORC_STATIC_SCRATCH_BYTES inside the
 * library (each GPU that loads the library holds that much until the process
 * ends).  The call performs no cudaMalloc/cudaFree and ignores the workspace.
 *   - Limit: batch * n_q_heads * n_splits * (2 + w) * 4 bytes must fit, w = r_v
 *     of the layer (d_head for FULL layers).  The split count is lowered
 *     automatically to fit; if one split still does not fit the call returns
 *     LORC_ERR_WORKSPACE and runs nothing.
 *   - The first call on each device looks up the array's device address
 *     (a short host-side set-up step); make that first call outside any stream
 *     capture.  The context's device must be current.
 *   - All calls, on every context and stream, share the one array per GPU.  It
 *     keeps whatever the previous call left; this call overwrites every slot it
 *     later reads, so no clearing is needed.  Two calls whose kernels may overlap
 *     on the GPU (different streams without ordering) race on the array: order
 *     them. */
#define LORC_STATIC_SCRATCH_BYTES (8u << 20)
int lorc_decode_attn_static(lorc_ctx* ctx, int layer, const lorc_cache* cache, const void* q, void* out,
                            int n_splits, void* stream);

/* One decode step of one layer from HOST buffers: copies x_host [batch, D] and
 * q_host [batch, n_q_heads, d_head] to staging at the end of the workspace, runs
 * lorc_append (T = 1) and lorc_decode_attn, and copies the result to out_host
 * [batch, n_q_heads, d_head]; all on `stream`, asynchronously when the host
 * buffers are pinned.  The caller synchronises the stream before reading
 * out_host.  The cache stays on the device. */
int lorc_decode_step_host(lorc_ctx* ctx, int layer, const lorc_cache* cache, const void* x_host,
                          const void* q_host, void* out_host, int n_splits, void* stream);

/* Synchronise `stream`, then read and clear the device status word.  Returns
 * LORC_OK or the first error a kernel recorded since the last call. */
int lorc_sync_status(lorc_ctx* ctx, void* stream);

/* Text of the last error reported on this context (never NULL). */
const char* lorc_last_error(const lorc_ctx* ctx);

/* Which kernel family the last lorc_decode_attn / lorc_append call on this
 * context used: 0 = none yet, 1 = plain fp32 CUDA-core kernels, 2 = tensor-core
 * (tcgen05) kernels of the latent mode, 3 = warp-level tensor-core (mma.sync) kernel of
 * the uncompressed mode.  For tests and benchmarks. */
int lorc_last_path(const lorc_ctx* ctx);

/* Contexts created with LORC_FLAG_PROFILE record a CUDA event before and after every
 * kernel they launch (do not use together with stream capture).  This call waits for the
 * recorded events, adds up the device time per stage since the previous call and writes
 * ms[LORC_N_STAGES] (milliseconds) and launches[LORC_N_STAGES]; either may be NULL.
 * Without the flag it returns zeros. */
int lorc_profile_read(lorc_ctx* ctx, float* ms, int64_t* launches);

/* Self-test of the device-side bounded waits.  Every wait of every kernel of the library (on a shared-memory barrier
 * that a copy or a tensor-core operation completes) runs through one routine with a time limit; when the limit runs out
 * the kernel stops issuing work, sets the status word to LORC_ERR_TIMEOUT and returns.  This call launches a one-thread
 * kernel that waits with that routine, with the limit given here (1 ns .. 1 s), on a barrier that nothing signals: the
 * next lorc_sync_status returns LORC_ERR_TIMEOUT and the context stays usable.  Asynchronous on `stream`. */
int lorc_selftest_wait_expiry(lorc_ctx* ctx, unsigned long long limit_ns, void* stream);

/* Switches the event bracketing of LORC_FLAG_PROFILE on (on != 0) or off for the calls that
 * follow, on any context; while it is off the launches carry no events and may be captured
 * into a CUDA graph.  Events still pending are kept for the next lorc_profile_read.
 * Returns LORC_ERR_ARG for a NULL context, LORC_ERR_CUDA when the bookkeeping cannot be set up. */
int lorc_profile_enable(lorc_ctx* ctx, int on);

/* Number of kernel launches the library has enqueued on this context so far. */
int64_t lorc_launch_count(const lorc_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* LORC_H_ */
