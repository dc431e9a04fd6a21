// Plain fp32 CUDA-core kernels: the debug path of the library and the handler of
// shapes the tensor-core kernels do not cover.  Everything is computed the
// direct way: latent projection as a dot product per output element, key tiles
// reconstructed as C_K . B_K, rotated with a table of exact-to-fp32 cos/sin,
// online softmax per head, P . C_V accumulated in latent space, and the value
// up-projection applied once per (sequence, head) in the combine kernel.
#include <math.h>

#include "common.cuh"

// ---------------------------------------------------------------------------
// RoPE table: (cos, sin)(pos * theta^(-2j/d_head)), angles in fp64.  theta <= 0 stands for "no rotation": every entry
// is (1, 0), and the kernels that rotate by the table leave keys and queries as they are.
// ---------------------------------------------------------------------------
__global__ void rope_table_kernel(float2* table, int max_pos, int half, double theta) {
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    long long total = (long long)max_pos * half;
    if (i >= total) return;
    int pos = (int)(i / half);
    int j = (int)(i - (long long)pos * half);
    if (!(theta > 0.0)) {
        table[i] = make_float2(1.f, 0.f);
        return;
    }
    double inv_freq = pow(theta, -(double)j / (double)half);   // theta^(-2j/d_head)
    double s, c;
    sincos((double)pos * inv_freq, &s, &c);
    table[i] = make_float2((float)c, (float)s);
}

cudaError_t lorc_generic_build_rope_table(float2* table, int max_pos, int d_head, double theta,
                                          cudaStream_t st) {
    int half = d_head / 2;
    long long total = (long long)max_pos * half;
    int threads = 256;
    long long blocks = (total + threads - 1) / threads;
    rope_table_kernel<<<(unsigned)blocks, threads, 0, st>>>(table, max_pos, half, theta);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// out[c][r] = in[r][c]
// ---------------------------------------------------------------------------
__global__ void transpose_kernel(const bf16* __restrict__ in, bf16* __restrict__ out, int rows,
                                 int cols) {
    __shared__ bf16 tile[32][33];
    int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    for (int i = threadIdx.y; i < 32; i += blockDim.y) {
        int r = r0 + i, c = c0 + threadIdx.x;
        if (r < rows && c < cols) tile[i][threadIdx.x] = in[(long long)r * cols + c];
    }
    __syncthreads();
    for (int i = threadIdx.y; i < 32; i += blockDim.y) {
        int c = c0 + i, r = r0 + threadIdx.x;
        if (r < rows && c < cols) out[(long long)c * rows + r] = tile[threadIdx.x][i];
    }
}

cudaError_t lorc_generic_transpose(const bf16* in, bf16* out, int rows, int cols, cudaStream_t st) {
    dim3 grid((cols + 31) / 32, (rows + 31) / 32), block(32, 8);
    transpose_kernel<<<grid, block, 0, st>>>(in, out, rows, cols);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Append: latent rows C = x A for TT tokens per block, 128 output columns per block.
// A_cat is [D, R] with R = r_k + r_v; column c < r_k goes to the K cache.
// FULL layers rotate the K part before storing.
// ---------------------------------------------------------------------------
#define APPEND_TT 8
#define APPEND_DCHUNK 512

template <bool FULL>
__global__ void __launch_bounds__(128)
append_generic_kernel(const bf16* __restrict__ x, const bf16* __restrict__ A_cat, CacheView cv, int D,
                      int r_k, int r_v, int T, int d_head, int rope_style,
                      const float2* __restrict__ rope_table, int max_pos, int* status) {
    __shared__ float xs[APPEND_TT][APPEND_DCHUNK];
    __shared__ float ex[APPEND_TT][128];
    const int R = r_k + r_v;
    const int tid = threadIdx.x;
    const int col = blockIdx.x * 128 + tid;
    const long long tok0 = (long long)blockIdx.y * APPEND_TT;
    const long long n_tok = (long long)cv.batch * T;
    float acc[APPEND_TT];
#pragma unroll
    for (int t = 0; t < APPEND_TT; ++t) acc[t] = 0.f;

    for (int d0 = 0; d0 < D; d0 += APPEND_DCHUNK) {
        int dn = min(APPEND_DCHUNK, D - d0);
        for (int i = tid; i < APPEND_TT * APPEND_DCHUNK; i += 128) {
            int t = i / APPEND_DCHUNK, d = i - t * APPEND_DCHUNK;
            float v = 0.f;
            if (tok0 + t < n_tok && d < dn) v = __bfloat162float(x[(tok0 + t) * D + d0 + d]);
            xs[t][d] = v;
        }
        __syncthreads();
        if (col < R) {
            const bf16* ap = A_cat + (long long)d0 * R + col;
            for (int d = 0; d < dn; ++d) {
                float a = __bfloat162float(ap[(long long)d * R]);
#pragma unroll
                for (int t = 0; t < APPEND_TT; ++t) acc[t] = fmaf(xs[t][d], a, acc[t]);
            }
        }
        __syncthreads();
    }

    if (FULL) {
        // rotation partner of a key column lives in the same 128-column block
#pragma unroll
        for (int t = 0; t < APPEND_TT; ++t) ex[t][tid] = acc[t];
        __syncthreads();
    }

#pragma unroll
    for (int t = 0; t < APPEND_TT; ++t) {
        long long tok = tok0 + t;
        if (tok >= n_tok || col >= R) continue;
        int s = (int)(tok / T);
        int i = (int)(tok - (long long)s * T);
        int len = cv.seq_lens[s];
        int pos = len - T + i;
        long long row = lorc_row_index(cv, s, pos);
        if (row < 0 || pos >= max_pos) {
            lorc_set_status(status, LORC_ERR_CAPACITY);
            continue;
        }
        float val = acc[t];
        if (col < r_k) {
            if (FULL) {
                const int half = d_head / 2;
                const int j = col % d_head;
                if (rope_style == LORC_ROPE_HALF_SPLIT) {
                    float2 cs = rope_table[(long long)pos * half + (j % half)];
                    float partner = (j < half) ? ex[t][tid + half] : ex[t][tid - half];
                    val = (j < half) ? val * cs.x - partner * cs.y : val * cs.x + partner * cs.y;
                } else {
                    float2 cs = rope_table[(long long)pos * half + (j / 2)];
                    float partner = (j & 1) ? ex[t][tid - 1] : ex[t][tid + 1];
                    val = (j & 1) ? val * cs.x + partner * cs.y : val * cs.x - partner * cs.y;
                }
            }
            cv.k[row * cv.w_k + col] = __float2bfloat16_rn(val);
        } else {
            cv.v[row * cv.w_v + (col - r_k)] = __float2bfloat16_rn(val);
        }
    }
}

cudaError_t lorc_generic_append(const lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv,
                                const bf16* x, int T, cudaStream_t st, int* launches) {
    const int R = L.r_k + L.r_v;
    long long n_tok = (long long)cv.batch * T;
    dim3 grid((R + 127) / 128, (unsigned)((n_tok + APPEND_TT - 1) / APPEND_TT));
    if (L.mode == LORC_MODE_FULL) {
        append_generic_kernel<true><<<grid, 128, 0, st>>>(
            x, L.A_cat, cv, ctx->desc.d_model, L.r_k, L.r_v, T, ctx->desc.d_head,
            ctx->pair_style, ctx->rope_table, ctx->desc.max_pos, ctx->status_dev);
    } else {
        append_generic_kernel<false><<<grid, 128, 0, st>>>(
            x, L.A_cat, cv, ctx->desc.d_model, L.r_k, L.r_v, T, ctx->desc.d_head,
            ctx->pair_style, ctx->rope_table, ctx->desc.max_pos, ctx->status_dev);
    }
    *launches += 1;
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Decode attention, one block per (context split, KV head, sequence).
// ---------------------------------------------------------------------------
#define GEN_TILE LORC_GENERIC_TILE
#define GEN_GMAX 8          // query heads per KV head supported
#define GEN_NC 8            // accumulator columns per thread: 8 * 128 = 1024 >= r_v

template <int DH, bool LATENT>
__global__ void __launch_bounds__(128)
decode_generic_kernel(const bf16* __restrict__ q, CacheView cv, const bf16* __restrict__ B_k, int r_k,
                      int r_v, int n, int G, int n_splits, int rope_style,
                      const float2* __restrict__ rope_table, int max_pos, float* __restrict__ part_ml,
                      float* __restrict__ part_o, int* status, int T, const int32_t* __restrict__ pos0,
                      const int32_t* __restrict__ q_pos) {
    constexpr int HALF = DH / 2;
    constexpr int SUB = 128 / DH;            // token subsets when DH < 128
    constexpr int TPS = GEN_TILE / SUB;      // tokens per thread in the reconstruction
    __shared__ float qs[GEN_GMAX][DH];
    __shared__ float Kt[GEN_TILE][DH + 1];
    __shared__ float Cs[GEN_TILE][33];
    __shared__ float Bs[32][DH];
    __shared__ float Ps[GEN_GMAX][GEN_TILE];
    __shared__ float m_s[GEN_GMAX], l_s[GEN_GMAX], alpha_s[GEN_GMAX];
    __shared__ long long row_s[GEN_TILE];

    const int tid = threadIdx.x;
    // With T queries per sequence (prompt processing) blockIdx.z runs over (sequence, query): query t of a chunk of T
    // sits at position seq_lens[s] - T + t and sees the tokens up to its own, i.e. it is the decode query of the
    // sequence cut after that token.  sq indexes queries, partial results and outputs; s the cache.
    const int split = blockIdx.x, g = blockIdx.y, sq = blockIdx.z, s = sq / T;
    const int H_q = G * (int)gridDim.y;
    const int W = LATENT ? r_v : DH;         // width of the output accumulator
    int len = cv.seq_lens[s];
    if (T > 1) len = len >= T ? len - (T - 1 - sq % T) : 0;
    // context shards: the cached rows sit at positions p0 .. p0 + len - 1, the query at qpos (not before the last row)
    const int p0 = pos0 ? pos0[s] : 0;
    int qpos_abs = q_pos ? q_pos[s] : p0 + len - 1;
    if (len > 0 && (p0 < 0 || qpos_abs < p0 + len - 1 || qpos_abs >= max_pos)) {
        if (threadIdx.x == 0) lorc_set_status(status, LORC_ERR_CAPACITY);
        len = 0;
    }

    // token range of this split
    int tiles = (len + GEN_TILE - 1) / GEN_TILE;
    int tps = (tiles + n_splits - 1) / n_splits;
    int t_begin = min(len, split * tps * GEN_TILE);
    int t_end = min(len, (split + 1) * tps * GEN_TILE);
    if (len <= 0) t_begin = t_end = 0;

    float acc[GEN_GMAX][GEN_NC];
#pragma unroll
    for (int h = 0; h < GEN_GMAX; ++h)
#pragma unroll
        for (int c = 0; c < GEN_NC; ++c) acc[h][c] = 0.f;

    // rotated, scaled query of the G heads of this KV head
    if (len > 0 && len <= max_pos) {
        const float scale = rsqrtf((float)DH);
        const int qpos = qpos_abs;
        for (int i = tid; i < G * HALF; i += 128) {
            int h = i / HALF, jj = i - h * HALF;
            int ia = (rope_style == LORC_ROPE_HALF_SPLIT) ? jj : 2 * jj;
            int ib = (rope_style == LORC_ROPE_HALF_SPLIT) ? jj + HALF : 2 * jj + 1;
            const bf16* qp = q + ((long long)sq * H_q + g * G + h) * DH;
            float a = __bfloat162float(qp[ia]), b = __bfloat162float(qp[ib]);
            float2 cs = rope_table[(long long)qpos * HALF + jj];
            qs[h][ia] = (a * cs.x - b * cs.y) * scale;
            qs[h][ib] = (a * cs.y + b * cs.x) * scale;
        }
    } else if (len > max_pos) {
        if (tid == 0) lorc_set_status(status, LORC_ERR_CAPACITY);
        t_begin = t_end = 0;
    }
    if (tid < GEN_GMAX) {
        m_s[tid] = -INFINITY;
        l_s[tid] = 0.f;
        alpha_s[tid] = 1.f;
    }
    __syncthreads();

    for (int t0 = t_begin; t0 < t_end; t0 += GEN_TILE) {
        if (tid < GEN_TILE) {
            int pos = t0 + tid;
            long long row = -1;
            if (pos < t_end) {
                row = lorc_row_index(cv, s, pos);
                if (row < 0) lorc_set_status(status, LORC_ERR_CAPACITY);
            }
            row_s[tid] = row;
        }
        __syncthreads();

        if (LATENT) {
            // key reconstruction: Kt[t][j] = sum_k C_K[t][k] * B_K[k][g*DH + j]
            const int j = tid % DH, sub = tid / DH;
            float kacc[TPS];
#pragma unroll
            for (int t = 0; t < TPS; ++t) kacc[t] = 0.f;
            for (int k0 = 0; k0 < r_k; k0 += 32) {
                for (int i = tid; i < GEN_TILE * 32; i += 128) {
                    int t = i / 32, kk = i - t * 32;
                    float v = 0.f;
                    long long row = row_s[t];
                    if (row >= 0 && k0 + kk < r_k) v = __bfloat162float(cv.k[row * cv.w_k + k0 + kk]);
                    Cs[t][kk] = v;
                }
                for (int i = tid; i < 32 * DH; i += 128) {
                    int kk = i / DH, jj = i - kk * DH;
                    float v = 0.f;
                    if (k0 + kk < r_k) v = __bfloat162float(B_k[(long long)(k0 + kk) * n + g * DH + jj]);
                    Bs[kk][jj] = v;
                }
                __syncthreads();
#pragma unroll 4
                for (int kk = 0; kk < 32; ++kk) {
                    float b = Bs[kk][j];
#pragma unroll
                    for (int t = 0; t < TPS; ++t) kacc[t] = fmaf(Cs[sub * TPS + t][kk], b, kacc[t]);
                }
                __syncthreads();
            }
#pragma unroll
            for (int t = 0; t < TPS; ++t) Kt[sub * TPS + t][j] = kacc[t];
            __syncthreads();
            // rotate each key at its own position
            for (int i = tid; i < GEN_TILE * HALF; i += 128) {
                int t = i / HALF, jj = i - t * HALF;
                int pos = t0 + t;
                if (pos >= t_end) continue;
                int ia = (rope_style == LORC_ROPE_HALF_SPLIT) ? jj : 2 * jj;
                int ib = (rope_style == LORC_ROPE_HALF_SPLIT) ? jj + HALF : 2 * jj + 1;
                float2 cs = rope_table[(long long)(p0 + pos) * HALF + jj];
                float a = Kt[t][ia], b = Kt[t][ib];
                Kt[t][ia] = a * cs.x - b * cs.y;
                Kt[t][ib] = a * cs.y + b * cs.x;
            }
        } else {
            // uncompressed cache: keys are stored rotated
            for (int i = tid; i < GEN_TILE * DH; i += 128) {
                int t = i / DH, j = i - t * DH;
                long long row = row_s[t];
                Kt[t][j] = (row >= 0) ? __bfloat162float(cv.k[row * cv.w_k + g * DH + j]) : 0.f;
            }
        }
        __syncthreads();

        // scores
        for (int i = tid; i < G * GEN_TILE; i += 128) {
            int h = i / GEN_TILE, t = i - h * GEN_TILE;
            float sc = -INFINITY;
            if (t0 + t < t_end && row_s[t] >= 0) {
                float d = 0.f;
#pragma unroll 8
                for (int j = 0; j < DH; ++j) d = fmaf(qs[h][j], Kt[t][j], d);
                sc = d;
            }
            Ps[h][t] = sc;
        }
        __syncthreads();

        // online softmax bookkeeping, one thread per head
        if (tid < G) {
            float m_old = m_s[tid], m_new = m_old;
            for (int t = 0; t < GEN_TILE; ++t) m_new = fmaxf(m_new, Ps[tid][t]);
            float alpha = 1.f, sum = 0.f;
            if (m_new == -INFINITY) {
                for (int t = 0; t < GEN_TILE; ++t) Ps[tid][t] = 0.f;
            } else {
                alpha = (m_old == -INFINITY) ? 0.f : expf(m_old - m_new);
                for (int t = 0; t < GEN_TILE; ++t) {
                    float p = expf(Ps[tid][t] - m_new);
                    Ps[tid][t] = p;
                    sum += p;
                }
            }
            m_s[tid] = m_new;
            l_s[tid] = l_s[tid] * alpha + sum;
            alpha_s[tid] = alpha;
        }
        __syncthreads();

        // O[h][col] = O[h][col]*alpha + sum_t p[h][t] * V[t][col]
#pragma unroll
        for (int c = 0; c < GEN_NC; ++c) {
            int col = tid + c * 128;
            if (col >= W) break;
#pragma unroll
            for (int h = 0; h < GEN_GMAX; ++h)
                if (h < G) acc[h][c] *= alpha_s[h];
            for (int t = 0; t < GEN_TILE; ++t) {
                long long row = row_s[t];
                if (row < 0) continue;
                float v = LATENT ? __bfloat162float(cv.v[row * cv.w_v + col])
                                 : __bfloat162float(cv.v[row * cv.w_v + g * DH + col]);
#pragma unroll
                for (int h = 0; h < GEN_GMAX; ++h)
                    if (h < G) acc[h][c] = fmaf(Ps[h][t], v, acc[h][c]);
            }
        }
        __syncthreads();
    }

    // partial results of this split
#pragma unroll
    for (int h = 0; h < GEN_GMAX; ++h) {
        if (h >= G) break;
        long long unit = ((long long)sq * H_q + g * G + h) * n_splits + split;
        if (tid == 0) {
            part_ml[unit * 2 + 0] = m_s[h];
            part_ml[unit * 2 + 1] = l_s[h];
        }
#pragma unroll
        for (int c = 0; c < GEN_NC; ++c) {
            int col = tid + c * 128;
            if (col < W) part_o[unit * W + col] = acc[h][c];
        }
    }
}

// Merge the splits of one (sequence, head) and apply the value up-projection.
template <bool LATENT>
__global__ void __launch_bounds__(128)
combine_generic_kernel(const float* __restrict__ part_ml, const float* __restrict__ part_o,
                       const bf16* __restrict__ B_v, bf16* __restrict__ out, int W, int n, int DH, int G,
                       int n_splits, int* status, float* __restrict__ ml_out) {
    extern __shared__ float o_lat[];     // [W]
    __shared__ float w_s[LORC_MAX_SPLITS];
    __shared__ float L_s;
    const int h = blockIdx.x, s = blockIdx.y, H_q = gridDim.x, tid = threadIdx.x;
    const long long unit0 = ((long long)s * H_q + h) * n_splits;
    if (tid == 0) {
        float M = -INFINITY;
        for (int c = 0; c < n_splits; ++c) {
            float l = part_ml[(unit0 + c) * 2 + 1];
            if (l > 0.f) M = fmaxf(M, part_ml[(unit0 + c) * 2]);
        }
        double L = 0.0;
        for (int c = 0; c < n_splits; ++c) {
            float m = part_ml[(unit0 + c) * 2], l = part_ml[(unit0 + c) * 2 + 1];
            float w = (l > 0.f) ? expf(m - M) : 0.f;
            w_s[c] = w;
            L += (double)w * (double)l;
        }
        L_s = (float)L;
        if (ml_out) {
            // reference in log2 units and the denominator relative to it (a shard of a context may be empty)
            ml_out[((long long)s * H_q + h) * 2] = L > 0.0 ? M * 1.4426950408889634f : 0.f;
            ml_out[((long long)s * H_q + h) * 2 + 1] = (float)L;
        } else if (!(L > 0.0)) {
            lorc_set_status(status, LORC_ERR_EMPTY);
        }
    }
    __syncthreads();
    const float L = L_s;
    const float inv = (L > 0.f) ? 1.f / L : 0.f;
    for (int col = tid; col < W; col += 128) {
        float a = 0.f;
        for (int c = 0; c < n_splits; ++c) {
            float w = w_s[c];
            if (w != 0.f) a = fmaf(w, part_o[(unit0 + c) * W + col], a);
        }
        o_lat[col] = a * inv;
    }
    __syncthreads();
    bf16* op = out + ((long long)s * H_q + h) * DH;
    if (LATENT) {
        const int g = h / G;
        for (int j = tid; j < DH; j += 128) {
            float a = 0.f;
            for (int k = 0; k < W; ++k)
                a = fmaf(o_lat[k], __bfloat162float(B_v[(long long)k * n + g * DH + j]), a);
            op[j] = __float2bfloat16_rn(a);
        }
    } else {
        for (int j = tid; j < DH; j += 128) op[j] = __float2bfloat16_rn(o_lat[j]);
    }
}

cudaError_t lorc_generic_combine(const lorc_ctx* ctx, const LorcLayer& L, int batch, int n_splits,
                                 const float* part_ml, const float* part_o, bf16* out,
                                 cudaStream_t st, int* launches, bool latent_out, float* ml_out) {
    const lorc_model_desc& d = ctx->desc;
    const bool latent = (L.mode == LORC_MODE_LATENT);
    const int W = latent ? L.r_v : d.d_head;
    dim3 cgrid(d.n_q_heads, batch);
    size_t smem = (size_t)W * sizeof(float);
    LorcStageTimer timer(ctx, LORC_STAGE_COMBINE, st);
    if (latent && latent_out)
        // merge only: the normalised latent output [b, H_q, r_v] is the result (rows of width W instead of d_head)
        combine_generic_kernel<false><<<cgrid, 128, smem, st>>>(part_ml, part_o, nullptr, out, W, ctx->n, W, ctx->group,
                                                               n_splits, ctx->status_dev, ml_out);
    else if (latent)
        combine_generic_kernel<true><<<cgrid, 128, smem, st>>>(part_ml, part_o, L.B_v, out, W, ctx->n,
                                                              d.d_head, ctx->group, n_splits,
                                                              ctx->status_dev, ml_out);
    else
        combine_generic_kernel<false><<<cgrid, 128, smem, st>>>(part_ml, part_o, nullptr, out, W, ctx->n,
                                                               d.d_head, ctx->group, n_splits,
                                                               ctx->status_dev, ml_out);
    *launches += 1;
    return cudaGetLastError();
}

cudaError_t lorc_generic_decode(const lorc_ctx* ctx, const LorcLayer& L, const CacheView& cv,
                                const bf16* q, bf16* out, int n_splits, float* part_ml,
                                float* part_o, cudaStream_t st, int* launches, bool latent_out, int T,
                                const int32_t* pos0, const int32_t* q_pos, float* ml_out) {
    const lorc_model_desc& d = ctx->desc;
    const int G = ctx->group;
    const bool latent = (L.mode == LORC_MODE_LATENT);
    dim3 grid(n_splits, d.n_kv_heads, cv.batch * T);
    if (T == 1 && lorc_full_decode_supported(ctx, L)) {
        // uncompressed mode with 128-wide heads: the streaming kernel on the warp-level tensor cores
        {
            LorcStageTimer timer(ctx, LORC_STAGE_SCORE, st);
            cudaError_t e = lorc_full_decode(ctx, cv, q, n_splits, part_ml, part_o, st, launches);
            if (e != cudaSuccess) return e;
        }
        return lorc_generic_combine(ctx, L, cv.batch, n_splits, part_ml, part_o, out, st, launches, false, nullptr);
    }
    {
    LorcStageTimer timer(ctx, LORC_STAGE_SCORE, st);
#define LAUNCH_DEC(DHV, LAT)                                                                      \
    decode_generic_kernel<DHV, LAT><<<grid, 128, 0, st>>>(                                        \
        q, cv, L.B_k, L.r_k, L.r_v, ctx->n, G, n_splits, ctx->pair_style, ctx->rope_table, d.max_pos, \
        part_ml, part_o, ctx->status_dev, T, pos0, q_pos)
    if (d.d_head == 128) {
        if (latent) LAUNCH_DEC(128, true); else LAUNCH_DEC(128, false);
    } else {
        if (latent) LAUNCH_DEC(64, true); else LAUNCH_DEC(64, false);
    }
#undef LAUNCH_DEC
    }
    *launches += 1;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return lorc_generic_combine(ctx, L, cv.batch * T, n_splits, part_ml, part_o, out, st, launches, latent_out, ml_out);
}

// ---------------------------------------------------------------------------
// Merge of context shards: out = sum_r w_r out_r / sum_r w_r,  w_r = L_r 2^(M_r - M),  M = max_r M_r.
// ---------------------------------------------------------------------------
__global__ void merge_shards_kernel(const bf16* __restrict__ outs, const float* __restrict__ mls, bf16* __restrict__ out,
                                    int n_shards, long long rows, int DH, int* status) {
    const long long row = blockIdx.x;                    // (sequence, head)
    __shared__ float w_s[64];
    __shared__ float inv_s;
    if (threadIdx.x == 0) {
        float M = -INFINITY;
        for (int r = 0; r < n_shards; ++r)
            if (mls[((long long)r * rows + row) * 2 + 1] > 0.f) M = fmaxf(M, mls[((long long)r * rows + row) * 2]);
        float tot = 0.f;
        for (int r = 0; r < n_shards; ++r) {
            const float l = mls[((long long)r * rows + row) * 2 + 1];
            const float w = l > 0.f ? l * exp2f(mls[((long long)r * rows + row) * 2] - M) : 0.f;
            w_s[r] = w;
            tot += w;
        }
        inv_s = tot > 0.f ? 1.f / tot : 0.f;
        if (!(tot > 0.f)) lorc_set_status(status, LORC_ERR_EMPTY);
    }
    __syncthreads();
    for (int j = threadIdx.x; j < DH; j += blockDim.x) {
        float a = 0.f;
        for (int r = 0; r < n_shards; ++r)
            if (w_s[r] != 0.f) a = fmaf(w_s[r], __bfloat162float(outs[((long long)r * rows + row) * DH + j]), a);
        out[row * DH + j] = __float2bfloat16_rn(a * inv_s);
    }
}

cudaError_t lorc_generic_merge_shards(const lorc_ctx* ctx, int n_shards, const bf16* outs, const float* mls, bf16* out,
                                      int batch, cudaStream_t st, int* launches) {
    const long long rows = (long long)batch * ctx->desc.n_q_heads;
    merge_shards_kernel<<<(unsigned)rows, 128, 0, st>>>(outs, mls, out, n_shards, rows, ctx->desc.d_head, ctx->status_dev);
    *launches += 1;
    return cudaGetLastError();
}
