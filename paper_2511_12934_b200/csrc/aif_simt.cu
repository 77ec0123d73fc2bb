// CUDA-core kernels of libaif: table scatter / gather, the general scoring kernel (any storage type, all
// interaction blocks, fp32 arithmetic) and the user-side network.  The tensor-core kernels live in aif_tc.cu.
#include <type_traits>

#include "aif_internal.h"
#include "aif_device.cuh"

namespace aif {

std::atomic<uint64_t> g_launches{0};

// ------------------------------------------------------------------------------------------------
// item table: scatter (nearline refresh) and gather
// ------------------------------------------------------------------------------------------------
template <typename V>
__global__ void k_scatter_rows(V *__restrict__ table, const V *__restrict__ rows, const int32_t *__restrict__ ids,
                               int64_t n, int vec_per_row, int64_t M, uint32_t *status)
{
    const int64_t total = n * vec_per_row;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / vec_per_row;
        const int c = (int)(i - r * vec_per_row);
        const int64_t dst = ids ? (int64_t)ids[r] : r;
        if (dst < 0 || dst >= M) {
            if (c == 0) atomicOr(status, AIF_STATUS_BAD_ID);
            continue;
        }
        table[dst * vec_per_row + c] = rows[i];
    }
}

// rows_out[i] = table[ids[i]]; 16 bytes per thread and four independent rows in flight per thread.
__global__ void __launch_bounds__(256) k_gather_rows(const uint4 *__restrict__ table, const int32_t *__restrict__ ids,
                                                     int64_t n, int vec_per_row, int64_t M, uint4 *__restrict__ out,
                                                     uint32_t *status)
{
    const int64_t total = n * vec_per_row;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i < total; i += 4 * stride) {
        uint4 v[4];
        bool ok[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t ii = i + u * stride;
            ok[u] = false;
            v[u] = make_uint4(0, 0, 0, 0);
            if (ii < total) {
                const int64_t r = ii / vec_per_row;
                const int c = (int)(ii - r * vec_per_row);
                const int64_t src = ids[r];
                ok[u] = true;
                if (src >= 0 && src < M) v[u] = __ldg(table + src * vec_per_row + c);
                else if (c == 0) atomicOr(status, AIF_STATUS_BAD_ID);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (ok[u]) out[i + u * stride] = v[u];
    }
}

// Copies candidate ids from page-locked host memory that is mapped into the device's address space.
__global__ void __launch_bounds__(256) k_stage_ids(const int32_t *__restrict__ src, int32_t *__restrict__ dst, int n)
{
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) dst[i] = src[i];
}

cudaError_t launch_stage_ids(const int32_t *mapped_src, int32_t *dst, int n, cudaStream_t st)
{
    const int grid = (n + 255) / 256 < 148 ? (n + 255) / 256 : 148;
    k_stage_ids<<<grid, 256, 0, st>>>(mapped_src, dst, n);
    count_launch();
    return cudaGetLastError();
}

static int grid_for(int64_t items, int per_block, int cap)
{
    int64_t g = (items + per_block - 1) / per_block;
    if (g < 1) g = 1;
    return (int)(g > cap ? cap : g);
}

template <typename V>
static cudaError_t scatter_typed(void *table, const void *rows, const int32_t *ids, int64_t n, size_t row_bytes, int64_t M,
                                 uint32_t *status, cudaStream_t st)
{
    const int vpr = (int)(row_bytes / sizeof(V));
    k_scatter_rows<V><<<grid_for(n * vpr, 256, 148 * 32), 256, 0, st>>>((V *)table, (const V *)rows, ids, n, vpr, M, status);
    count_launch();
    return cudaGetLastError();
}

static cudaError_t scatter_bytes(void *table, const void *rows, const int32_t *ids, int64_t n, size_t row_bytes, int64_t M,
                                 uint32_t *status, cudaStream_t st)
{
    if (row_bytes % 16 == 0) return scatter_typed<uint4>(table, rows, ids, n, row_bytes, M, status, st);
    if (row_bytes % 8 == 0) return scatter_typed<uint2>(table, rows, ids, n, row_bytes, M, status, st);
    if (row_bytes % 4 == 0) return scatter_typed<uint32_t>(table, rows, ids, n, row_bytes, M, status, st);
    return scatter_typed<uint16_t>(table, rows, ids, n, row_bytes, M, status, st);
}

cudaError_t launch_scatter_rows(const aif_ctx *ctx, const int32_t *ids, int64_t n, const void *rows, const void *bea_w,
                                const uint8_t *sig, cudaStream_t st)
{
    const aif_config &c = ctx->cfg;
    cudaError_t e = scatter_bytes(ctx->E, rows, ids, n, (size_t)c.d * ctx->el, c.M, ctx->status, st);
    if (e != cudaSuccess) return e;
    if (ctx->bea_w) {
        e = scatter_bytes(ctx->bea_w, bea_w, ids, n, (size_t)c.n_bridge * ctx->el, c.M, ctx->status, st);
        if (e != cudaSuccess) return e;
    }
    if (ctx->sig) e = scatter_bytes(ctx->sig, sig, ids, n, (size_t)c.lsh_bits / 8, c.M, ctx->status, st);
    return e;
}

// The same for rows of VPR 16-byte vectors with VPR a divisor of 32 (128 to 512 bytes: every benchmark shape).  A warp
// takes 8 x (32 / VPR) consecutive output rows per step: their ids arrive with one coalesced load and are handed round by
// shuffles, every lane then has eight independent 16-byte loads in flight, each instruction covering whole rows, and no
// division or second dependent load stands between a lane and its data.
template <int VPR>
__global__ void __launch_bounds__(256) k_gather_rows_w(const uint4 *__restrict__ table, const int32_t *__restrict__ ids, int64_t n, int64_t M,
                                                       uint4 *__restrict__ out, uint32_t *status)
{
    constexpr int RPI = 32 / VPR, RPS = 8 * RPI;   // rows per instruction, rows per step of a warp
    const int lane = threadIdx.x & 31, sub = lane / VPR, c = lane % VPR;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5, n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t r0 = warp * RPS; r0 < n; r0 += n_warps * RPS) {
        int my = -1;
        if (lane < RPS && r0 + lane < n) {
            my = ids[r0 + lane];
            if (my < 0 || (int64_t)my >= M) {
                my = -1;
                atomicOr(status, AIF_STATUS_BAD_ID);
            }
        }
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int src = __shfl_sync(0xffffffffu, my, u * RPI + sub);
            v[u] = src >= 0 ? __ldg(table + (int64_t)src * VPR + c) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int64_t r = r0 + u * RPI + sub;
            if (r < n) out[r * VPR + c] = v[u];
        }
    }
}

cudaError_t launch_gather_rows(const aif_ctx *ctx, const int32_t *ids, int64_t n, void *out, cudaStream_t st)
{
    const int vpr = (int)((size_t)ctx->cfg.d * ctx->el / 16);
    if (vpr == 8 || vpr == 16 || vpr == 32) {
        const int rps = 8 * (32 / vpr);
        const int64_t warps = (n + rps - 1) / rps;
        const int grid = (int)((warps + 7) / 8 < 148 * 16 ? (warps + 7) / 8 : 148 * 16);
        if (vpr == 8) k_gather_rows_w<8><<<grid, 256, 0, st>>>((const uint4 *)ctx->E, ids, n, ctx->cfg.M, (uint4 *)out, ctx->status);
        else if (vpr == 16) k_gather_rows_w<16><<<grid, 256, 0, st>>>((const uint4 *)ctx->E, ids, n, ctx->cfg.M, (uint4 *)out, ctx->status);
        else k_gather_rows_w<32><<<grid, 256, 0, st>>>((const uint4 *)ctx->E, ids, n, ctx->cfg.M, (uint4 *)out, ctx->status);
        count_launch();
        return cudaGetLastError();
    }
    const int64_t total = n * vpr;
    const int grid = grid_for((total + 3) / 4, 256, 148 * 16);
    k_gather_rows<<<grid, 256, 0, st>>>((const uint4 *)ctx->E, ids, n, vpr, ctx->cfg.M, (uint4 *)out, ctx->status);
    count_launch();
    return cudaGetLastError();
}

// out[i] = table[ids[i]] for narrow rows (BEA weights, signatures): one thread per 4 bytes.
__global__ void __launch_bounds__(256) k_gather_words(const uint32_t *__restrict__ table, const int32_t *__restrict__ ids, int64_t n,
                                                      int words_per_row, int64_t M, uint32_t *__restrict__ out, uint32_t *status)
{
    const int64_t total = n * words_per_row;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / words_per_row;
        const int c = (int)(i - r * words_per_row);
        const int64_t src = ids[r];
        uint32_t v = 0u;
        if (src >= 0 && src < M) v = __ldg(table + src * words_per_row + c);
        else if (c == 0) atomicOr(status, AIF_STATUS_BAD_ID);
        out[i] = v;
    }
}

cudaError_t launch_gather_sidecars(const aif_ctx *ctx, const int32_t *ids, int64_t n, void *bea_w_out, uint8_t *sig_out, cudaStream_t st)
{
    const aif_config &c = ctx->cfg;
    if (bea_w_out) {
        const int words = (int)((size_t)c.n_bridge * ctx->el / 4);
        k_gather_words<<<grid_for(n * words, 256, 148 * 16), 256, 0, st>>>((const uint32_t *)ctx->bea_w, ids, n, words, c.M,
                                                                           (uint32_t *)bea_w_out, ctx->status);
        count_launch();
    }
    if (sig_out) {
        const int words = c.lsh_bits / 32;
        k_gather_words<<<grid_for(n * words, 256, 148 * 16), 256, 0, st>>>((const uint32_t *)ctx->sig, ids, n, words, c.M,
                                                                           (uint32_t *)sig_out, ctx->status);
        count_launch();
    }
    return cudaGetLastError();
}

template <typename T>
__global__ void k_transpose(const T *__restrict__ in, T *__restrict__ out, int rows, int cols)
{
    __shared__ T tile[32][33];
    const int bx = blockIdx.x * 32, by = blockIdx.y * 32;
    for (int r = threadIdx.y; r < 32; r += blockDim.y) {
        const int y = by + r, x = bx + threadIdx.x;
        if (y < rows && x < cols) tile[r][threadIdx.x] = in[(size_t)y * cols + x];
    }
    __syncthreads();
    for (int r = threadIdx.y; r < 32; r += blockDim.y) {
        const int x = bx + r, y = by + threadIdx.x;
        if (y < rows && x < cols) out[(size_t)x * rows + y] = tile[threadIdx.x][r];
    }
}

// out [cols x rows] = in [rows x cols]^T
cudaError_t launch_transpose(const void *in, void *out, int rows, int cols, size_t el, cudaStream_t st)
{
    dim3 grid((cols + 31) / 32, (rows + 31) / 32), block(32, 8);
    if (el == 4) k_transpose<float><<<grid, block, 0, st>>>((const float *)in, (float *)out, rows, cols);
    else k_transpose<uint16_t><<<grid, block, 0, st>>>((const uint16_t *)in, (uint16_t *)out, rows, cols);
    count_launch();
    return cudaGetLastError();
}

int simt_tiles_for(const aif_ctx *ctx, int n) { return tiles_of(n, kSimtTile, ctx->cfg.mini_batch); }

// ------------------------------------------------------------------------------------------------
// general scoring kernel: one block = one tile of kSimtTile candidates, one warp per candidate for the
// interaction blocks, then all threads for the MLP with the decomposed first layer.
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kSimtThreads) k_score_simt(ModelDev md, ScoreLaunch sl, int max_h)
{
    constexpr int TM = kSimtTile;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *xs = reinterpret_cast<float *>(smem_raw);        // [k1][TM]   candidate-dependent input, transposed
    float *ha = xs + (size_t)md.k1 * TM;                     // [max_h][TM]
    float *hb = ha + (size_t)max_h * TM;                     // [max_h][TM]
    float *qv = hb + (size_t)max_h * TM;                     // [TM][d]    item vectors as fp32 rows (queries)
    uint32_t *sigq = reinterpret_cast<uint32_t *>(qv + (size_t)TM * md.d);   // [TM][8]
    int *tiers = reinterpret_cast<int *>(sigq + TM * 8);     // [TM][16]
    int *bkt = tiers + TM * 16;                              // [TM][F]
    int *id_s = bkt + TM * md.F;                             // [TM]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const ReqDev rq = find_request(sl, blockIdx.x);
    int start, cnt;
    tile_range(blockIdx.x - rq.tile_begin, rq.n, TM, md.mini_batch, start, cnt);
    const SlotDev slot = sl.slots[rq.slot];
    const int32_t *ids = sl.ids + rq.off + start;
    float *logits = sl.logits + rq.off + start;
    const int d = md.d, dq = d >> 5;

    if (tid < TM) {
        int id = -1;
        if (tid < cnt) {
            id = ids[tid];
            if (id < 0 || (int64_t)id >= md.M) {
                id = -1;
                atomicOr(sl.status, AIF_STATUS_BAD_ID);
            }
        }
        id_s[tid] = id;
    }
    for (int i = tid; i < md.k1 * TM; i += kSimtThreads) xs[i] = 0.f;
    for (int i = tid; i < TM * 16; i += kSimtThreads) tiers[i] = 0;
    __syncthreads();

    // ---- stage A: interaction blocks, warp c <-> candidate c
    {
        const int c = warp;
        const int id = id_s[c];
        if (id >= 0) {
            const T *e = reinterpret_cast<const T *>(md.E) + (size_t)id * d;
            int col = 0;
            for (int k = lane; k < d; k += 32) {
                const float v = to_f(e[k]);
                qv[c * d + k] = v;
                xs[(col + k) * TM + c] = v;
            }
            col += d;
            const bool do_att = md.blocks & AIF_BLK_ATT, do_din = md.blocks & AIF_BLK_LSH_DIN,
                       do_tier = md.blocks & AIF_BLK_SIMTIER, do_lsh = do_din || do_tier;
            if (do_lsh && lane < (md.lsh_bits >> 5))
                sigq[c * 8 + lane] = reinterpret_cast<const uint32_t *>(md.sig + (size_t)id * (md.lsh_bits >> 3))[lane];
            if (md.blocks & AIF_BLK_CROSS)
                for (int f = lane; f < md.F; f += 32) bkt[c * md.F + f] = bucket_of(id, f, md.B, md.bucket_mode);
            __syncwarp();
            float att[8], din[8];
            if (do_att || do_lsh)
                warp_interact<T>(qv + c * d, reinterpret_cast<const T *>(slot.S), slot.L, d, rsqrtf((float)d), do_att,
                                 do_lsh, do_tier, sigq + c * 8, slot.sigS, md.lsh_bits, md.n_tiers, tiers + c * 16, att,
                                 din);
            if (do_att) {
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    if (q < dq) xs[(col + lane + 32 * q) * TM + c] = att[q];
                col += d;
            }
            if (md.blocks & AIF_BLK_CROSS) {
                const T *Tt = reinterpret_cast<const T *>(slot.T);
                const int fdc = md.F * md.dc;
                for (int i = lane; i < fdc; i += 32) {
                    const int f = i / md.dc, k = i - f * md.dc;
                    xs[(col + i) * TM + c] = to_f(Tt[((size_t)f * md.B + bkt[c * md.F + f]) * md.dc + k]);
                }
                col += fdc;
            }
            if (md.blocks & AIF_BLK_BEA) {
                const T *wh = reinterpret_cast<const T *>(md.bea_w) + (size_t)id * md.n_bridge;
                const T *V = reinterpret_cast<const T *>(slot.V);
                for (int k = lane; k < d; k += 32) {
                    float acc = 0.f;
                    for (int b = 0; b < md.n_bridge; ++b) acc = fmaf(to_f(wh[b]), to_f(V[(size_t)b * d + k]), acc);
                    xs[(col + k) * TM + c] = acc;
                }
                col += d;
            }
            if (do_din) {
                const float nrm = md.lsh_din_norm == AIF_NORM_MEAN ? 1.0f / (float)slot.L : 1.0f;
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    if (q < dq) xs[(col + lane + 32 * q) * TM + c] = din[q] * nrm;
                col += d;
            }
            if (do_tier) {
                __syncwarp();
                const float nrm = md.simtier_norm == AIF_NORM_MEAN ? 1.0f / (float)slot.L : 1.0f;
                if (lane < md.n_tiers) xs[(col + lane) * TM + c] = (float)tiers[c * 16 + lane] * nrm;
            }
        }
    }
    __syncthreads();

    // ---- stage B: MLP.  First layer = cached user partial + candidate-dependent columns.
    const float *in_act = xs;
    float *out_act = ha;
    int in_w = md.k1;
    for (int layer = 0; layer < md.n_hidden; ++layer) {
        const int H = md.hidden[layer];
        const T *W = reinterpret_cast<const T *>(md.Wt[layer]) + (layer == 0 ? (size_t)d * H : 0);
        const float *bias = layer == 0 ? slot.p_u : md.b[layer];
        for (int j = tid; j < H; j += kSimtThreads) {
            float acc[TM];
            const float b0 = bias[j];
#pragma unroll
            for (int c = 0; c < TM; ++c) acc[c] = b0;
            // weights in batches of 32 independent loads (the accumulation order over k stays sequential): after an L2
            // flush every weight comes from HBM, and one load per iteration would expose that latency 32 times as often
            auto step = [&](int k, float w) {
                const float4 a = *reinterpret_cast<const float4 *>(in_act + k * TM);
                const float4 b = *reinterpret_cast<const float4 *>(in_act + k * TM + 4);
                acc[0] = fmaf(w, a.x, acc[0]);
                acc[1] = fmaf(w, a.y, acc[1]);
                acc[2] = fmaf(w, a.z, acc[2]);
                acc[3] = fmaf(w, a.w, acc[3]);
                acc[4] = fmaf(w, b.x, acc[4]);
                acc[5] = fmaf(w, b.y, acc[5]);
                acc[6] = fmaf(w, b.z, acc[6]);
                acc[7] = fmaf(w, b.w, acc[7]);
            };
            int k = 0;
            for (; k + 32 <= in_w; k += 32) {
                float w[32];
#pragma unroll
                for (int u = 0; u < 32; ++u) w[u] = to_f(W[(size_t)(k + u) * H + j]);
#pragma unroll
                for (int u = 0; u < 32; ++u) step(k + u, w[u]);
            }
            for (; k < in_w; ++k) step(k, to_f(W[(size_t)k * H + j]));
#pragma unroll
            for (int c = 0; c < TM; ++c) out_act[j * TM + c] = fmaxf(acc[c], 0.f);
        }
        __syncthreads();
        in_act = out_act;
        out_act = (out_act == ha) ? hb : ha;
        in_w = H;
    }
    // ---- output layer: warp c reduces candidate c in a fixed order
    {
        const int c = warp;
        if (c < cnt) {
            const T *wo = reinterpret_cast<const T *>(md.w_out);
            float acc = 0.f;
            for (int j = lane; j < in_w; j += 32) acc = fmaf(to_f(wo[j]), in_act[j * TM + c], acc);
            acc = warp_sum(acc);
            if (lane == 0) {
                float logit = acc + md.b_out[0];
                if (md.emit_sigmoid) logit = 1.0f / (1.0f + expf(-logit));
                logits[c] = id_s[c] >= 0 ? logit : __int_as_float(0x7fc00000);
            }
        }
    }
}

static size_t simt_smem_bytes(const aif_ctx *ctx, int &max_h)
{
    const aif_config &c = ctx->cfg;
    max_h = 0;
    for (int k = 0; k < c.n_hidden; ++k) max_h = c.hidden[k] > max_h ? c.hidden[k] : max_h;
    const int k1 = ctx->input_width - c.d;
    size_t fl = (size_t)(k1 + 2 * max_h + c.d) * kSimtTile;
    size_t ints = (size_t)kSimtTile * (8 + 16 + c.F + 1);
    return (fl + ints) * 4 + 16;
}

cudaError_t launch_score_simt(const aif_ctx *ctx, const ScoreLaunch &sl, cudaStream_t st)
{
    if (sl.n_tiles <= 0) return cudaSuccess;
    int max_h;
    const size_t smem = simt_smem_bytes(ctx, max_h);
    const ModelDev md = make_model(ctx);
    cudaError_t e;
    timing_begin(ctx, st);
    if (ctx->cfg.dtype == AIF_F32) {
        e = cudaFuncSetAttribute(k_score_simt<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k_score_simt<float><<<sl.n_tiles, kSimtThreads, smem, st>>>(md, sl, max_h);
    } else {
        e = cudaFuncSetAttribute(k_score_simt<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k_score_simt<__nv_bfloat16><<<sl.n_tiles, kSimtThreads, smem, st>>>(md, sl, max_h);
    }
    count_launch();
    timing_mark(ctx, "score_simt", st);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// user-side network (eqs. 1-3), fp32 arithmetic on storage-type inputs
// ------------------------------------------------------------------------------------------------

// eq. 1.  blockIdx.x < L: one sequence row -> S (storage type).  blockIdx.x == L: the profile -> prof_hat (fp32).
template <typename T>
__global__ void k_user_project(const T *__restrict__ seq, const T *__restrict__ profile, const T *__restrict__ Wseq_t,
                               const T *__restrict__ Wprof_t, int L, int dU, int d, T *__restrict__ S,
                               float *__restrict__ prof_hat)
{
    extern __shared__ float row[];
    const bool is_prof = (int)blockIdx.x == L;
    const T *src = is_prof ? profile : seq + (size_t)blockIdx.x * dU;
    const T *W = is_prof ? Wprof_t : Wseq_t;
    for (int k = threadIdx.x; k < dU; k += blockDim.x) row[k] = to_f(src[k]);
    __syncthreads();
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        float acc = 0.f;
        for (int k = 0; k < dU; ++k) acc = fmaf(row[k], to_f(W[(size_t)k * d + j]), acc);
        if (is_prof) prof_hat[j] = acc;
        else from_f(S[(size_t)blockIdx.x * d + j], acc);
    }
}

// eq. 2.  Warp g handles rows g, g + n_warps, ...: attention over the whole sequence, FFN, and a running sum
// for the mean pooling; partial[g] holds the warp's sum (summed later in a fixed order).  att_rows != nullptr: the
// attention rows softmax(S S^T / sqrt(d)) S were already computed by the tensor-core attention kernel.
template <typename T>
__global__ void __launch_bounds__(256) k_user_self(const T *__restrict__ S, int L, int d, const T *__restrict__ Wa_t,
                                                   const float *__restrict__ b_a, const T *__restrict__ Wb_t,
                                                   const float *__restrict__ b_b, float *__restrict__ partial,
                                                   int n_warps, const T *__restrict__ att_rows)
{
    extern __shared__ float sm[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = blockIdx.x * 8 + warp, dq = d >> 5;
    float *q = sm + (size_t)warp * 3 * d, *ctx = q + d;
    float pooled[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) pooled[c] = 0.f;
    const float scale = rsqrtf((float)d);
    for (int i = g; i < L; i += n_warps) {
        if (att_rows) {
            for (int k = lane; k < d; k += 32) ctx[k] = to_f(att_rows[(size_t)i * d + k]);
        } else {
            for (int k = lane; k < d; k += 32) q[k] = to_f(S[(size_t)i * d + k]);
            __syncwarp();
            float att[8], din[8];
            warp_interact<T>(q, S, L, d, scale, true, false, false, nullptr, nullptr, 0, 0, nullptr, att, din);
#pragma unroll
            for (int c = 0; c < 8; ++c)
                if (c < dq) ctx[lane + 32 * c] = att[c];
        }
        __syncwarp();
#pragma unroll
        for (int c = 0; c < 8; ++c)
            if (c < dq) {
                const int j = lane + 32 * c;
                float acc = b_a[j];
                for (int k = 0; k < d; ++k) acc = fmaf(ctx[k], to_f(Wa_t[(size_t)k * d + j]), acc);
                // the second FFN layer is linear, so it commutes with the mean pooling: pool the hidden activations
                // here and apply W_b once, in k_user_finish
                pooled[c] += fmaxf(acc, 0.f);
            }
        __syncwarp();
    }
    if (g < n_warps) {
#pragma unroll
        for (int c = 0; c < 8; ++c)
            if (c < dq) partial[(size_t)g * d + lane + 32 * c] = pooled[c];
    }
}

// eq. 3 in slices: warp g attends the profile query to keys [g * slice, (g + 1) * slice) and leaves its unnormalised
// output row with the slice's maximum and sum; k_user_finish merges the slices.
template <typename T>
__global__ void __launch_bounds__(256) k_user_prof(const T *__restrict__ S, int L, int d, const float *__restrict__ prof_hat,
                                                   int slice, float *__restrict__ ppart)
{
    __shared__ float q[256];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = blockIdx.x * 8 + warp, dq = d >> 5;
    for (int k = threadIdx.x; k < d; k += 256) q[k] = prof_hat[k];
    __syncthreads();
    float *out = ppart + (size_t)g * (d + 2);
    const int start = g * slice, len = min(slice, L - start);
    if (len <= 0) {
        if (lane == 0) out[d] = -INFINITY, out[d + 1] = 0.f;
        return;
    }
    float att[8], din[8];
    warp_interact<T>(q, S + (size_t)start * d, len, d, rsqrtf((float)d), true, false, false, nullptr, nullptr, 0, 0, nullptr, att,
                     din, out + d);
#pragma unroll
    for (int c = 0; c < 8; ++c)
        if (c < dq) out[lane + 32 * c] = att[c];
}

// eq. 3, the combined vector, and the cached first-layer partial product p_u = W1[:, 0:d] u + b1.
// raw = 1: u = mean-pooled self-attention + profile attention.  raw = 0: u is given (u_in, storage type).
template <typename T>
__global__ void __launch_bounds__(256) k_user_finish(int raw, const T *__restrict__ S, int L, int d,
                                                     const float *__restrict__ prof_hat,
                                                     const float *__restrict__ partial, int n_warps,
                                                     const T *__restrict__ u_in, T *__restrict__ u_out,
                                                     float *__restrict__ u32, const T *__restrict__ W1t,
                                                     const float *__restrict__ b1, int H1, float *__restrict__ p_u,
                                                     __nv_bfloat16 *__restrict__ pu_hl, const T *__restrict__ Wb_t, const float *__restrict__ b_b,
                                                     const float *__restrict__ ppart)
{
    __shared__ float q[256], uprof[256], us[256], wgt[kProfParts], red[256];
    static_assert(kProfParts == 256, "one thread per key slice");
    const int tid = threadIdx.x;
    if (raw) {
        // merge the key slices of the profile attention: softmax over all keys from per-slice maxima and sums.  One
        // thread per slice for the weights 2^(m_g - m) (kProfParts = blockDim), then one thread per output column.
        {
            const float m_g = ppart[(size_t)tid * (d + 2) + d], l_g = ppart[(size_t)tid * (d + 2) + d + 1];
            red[tid] = l_g > 0.f ? m_g : -INFINITY;
            __syncthreads();
            for (int o = 128; o > 0; o >>= 1) {
                if (tid < o) red[tid] = fmaxf(red[tid], red[tid + o]);
                __syncthreads();
            }
            const float m_all = red[0];
            __syncthreads();
            const float w = l_g > 0.f ? expf(m_g - m_all) : 0.f;
            wgt[tid] = w;
            red[tid] = w * l_g;
            __syncthreads();
            for (int o = 128; o > 0; o >>= 1) {   // fixed tree: the same sum in every run
                if (tid < o) red[tid] += red[tid + o];
                __syncthreads();
            }
            const float den = red[0];
            for (int k = tid; k < d; k += 256) {
                float n4[4] = {0.f, 0.f, 0.f, 0.f};
                for (int g = 0; g < kProfParts; g += 4) {   // four independent loads in flight
#pragma unroll
                    for (int u = 0; u < 4; ++u) n4[u] = fmaf(wgt[g + u], ppart[(size_t)(g + u) * (d + 2) + k], n4[u]);
                }
                uprof[k] = ((n4[0] + n4[1]) + (n4[2] + n4[3])) / den;
            }
        }
        __syncthreads();
        // mean over the sequence of the hidden FFN activations: the warps' partial sums in a fixed order, 256 / d threads
        // per column over interleaved slices of the partials, eight loads in flight per thread
        {
            const int parts = 256 / d > 0 ? 256 / d : 1;
            const int k = tid % d, part = tid / d;
            float a8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            if (part < parts && k < d) {
                int g = part;
                for (; g + 7 * parts < n_warps; g += 8 * parts) {
#pragma unroll
                    for (int u = 0; u < 8; ++u) a8[u] += partial[(size_t)(g + u * parts) * d + k];
                }
                for (; g < n_warps; g += parts) a8[0] += partial[(size_t)g * d + k];
            }
            red[tid] = ((a8[0] + a8[1]) + (a8[2] + a8[3])) + ((a8[4] + a8[5]) + (a8[6] + a8[7]));
            __syncthreads();
            for (int kk = tid; kk < d; kk += 256) {
                float acc = 0.f;
                for (int pp = 0; pp < parts; ++pp) acc += red[pp * d + kk];
                q[kk] = acc / (float)L;
            }
        }
        __syncthreads();
        // ... through the second FFN layer, plus the profile attention: the combined user vector
        for (int k = tid; k < d; k += 256) {
            float acc = b_b[k];
            for (int j = 0; j < d; ++j) acc = fmaf(q[j], to_f(Wb_t[(size_t)j * d + k]), acc);
            const float u = acc + uprof[k];
            us[k] = u;
            u32[k] = u;
            from_f(u_out[k], u);
        }
    } else {
        for (int k = tid; k < d; k += 256) {
            const float u = to_f(u_in[k]);
            us[k] = u;
            u32[k] = u;
        }
    }
    __syncthreads();
    for (int j = tid; j < H1; j += 256) {
        float acc = b1[j];
        for (int k = 0; k < d; ++k) acc = fmaf(us[k], to_f(W1t[(size_t)k * H1 + j]), acc);
        p_u[j] = acc;
        // the same partial as two bf16 values (high part, remainder): the form in which the tensor cores add it
        const __nv_bfloat16 hi = __float2bfloat16_rn(acc);
        pu_hl[j] = hi;
        pu_hl[H1 + j] = __float2bfloat16_rn(acc - __bfloat162float(hi));
    }
}

// the slot's length, and its key-norm bound back to zero (k_row_norm_max raises it once the rows are written)
__global__ void k_set_slot_len(SlotDev *slots, int index, int L)
{
    slots[index].L = L;
    *const_cast<float *>(slots[index].k_norm) = 0.f;
}

// Largest Euclidean norm over a set of rows, one warp per row.  Norms are non-negative, so their bit patterns order like
// integers; a NaN row yields a pattern above every finite one and stays.
template <typename T>
__global__ void __launch_bounds__(256) k_row_norm_max(const T *__restrict__ rows, const int32_t *__restrict__ ids, int64_t n, int64_t M, int d,
                                                      float *__restrict__ out)
{
    const int lane = threadIdx.x & 31;
    const int64_t w0 = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5), stride = (int64_t)gridDim.x * 8;
    int best = 0;
    for (int64_t i = w0; i < n; i += stride) {
        const int64_t r = ids ? (int64_t)ids[i] : i;
        if (r < 0 || r >= M) continue;
        const T *row = rows + (size_t)r * d;
        float acc = 0.f;
        for (int c = lane; c < d; c += 32) {
            const float v = to_f(row[c]);
            acc = fmaf(v, v, acc);
        }
        acc = warp_sum(acc);
        best = max(best, __float_as_int(sqrtf(acc)) & 0x7fffffff);
    }
    if (lane == 0 && best > 0) atomicMax(reinterpret_cast<int *>(out), best);
}

cudaError_t launch_row_norm_max(const aif_ctx *ctx, const void *rows, const int32_t *ids, int64_t n, int64_t M, float *out, cudaStream_t st)
{
    if (n <= 0 || !out) return cudaSuccess;
    const int64_t want = (n + 7) / 8;
    const int grid = (int)(want < 148 * 8 ? want : 148 * 8);
    if (ctx->cfg.dtype == AIF_F32) k_row_norm_max<float><<<grid, 256, 0, st>>>((const float *)rows, ids, n, M, ctx->cfg.d, out);
    else k_row_norm_max<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16 *)rows, ids, n, M, ctx->cfg.d, out);
    count_launch();
    return cudaGetLastError();
}

// partial[g][k] = sum over rows g, g + n_parts, ... of rows[i][k] (bf16 rows, fp32 sums in a fixed order): the mean pooling of
// eq. 2 over hidden FFN activations that a tensor-core layer has written
__global__ void __launch_bounds__(256) k_pool_rows(const __nv_bfloat16 *__restrict__ rows, int L, int d, int n_parts, float *__restrict__ partial)
{
    const int lane = threadIdx.x & 31, g = blockIdx.x * 8 + (threadIdx.x >> 5), dq = d >> 5;
    if (g >= n_parts) return;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int i = g; i < L; i += n_parts) {
#pragma unroll
        for (int c = 0; c < 8; ++c)
            if (c < dq) acc[c] += __bfloat162float(rows[(size_t)i * d + lane + 32 * c]);
    }
#pragma unroll
    for (int c = 0; c < 8; ++c)
        if (c < dq) partial[(size_t)g * d + lane + 32 * c] = acc[c];
}

template <typename T>
static cudaError_t user_network_typed(const aif_ctx *ctx, HostSlot &hs, int slot_index, const aif_user_inputs *in, int L,
                                      cudaStream_t st)
{
    const aif_config &c = ctx->cfg;
    const int d = c.d, H1 = c.hidden[0];
    cudaError_t e;
    T *S = (T *)hs.dev.S;
    const bool raw = in->mode == AIF_USER_RAW;
    // Long sequences on bf16 tensor-core contexts: eq. 1's sequence projection and the first FFN layer of eq. 2 are dense
    // layers over L rows and run through the scoring MLP's layer kernel (tcgen05); shorter ones stay on the CUDA cores,
    // where a launch of this size is latency, not throughput.
    const bool tc_user = raw && std::is_same<T, __nv_bfloat16>::value && ctx->tensor_path && ctx->tc_att_plan && L >= 1024 &&
                         c.dU % 64 == 0 && d % 64 == 0;
    if (raw && tc_user) {
        DenseLayer lay{};
        lay.A = in->seq, lay.W = ctx->Wseq_k, lay.bias = ctx->zero_bias, lay.out = S, lay.in_w = c.dU, lay.H = d, lay.relu = 0, lay.sign_bits = 0;
        if ((e = tc_dense_layer(ctx, lay, L, st)) != cudaSuccess) return e;
        // the profile row alone (block index L of the projection kernel, launched with no sequence rows)
        k_user_project<T><<<1, 128, c.dU * sizeof(float), st>>>((const T *)in->seq, (const T *)in->profile, (const T *)ctx->Wseq_t,
                                                                 (const T *)ctx->Wprofile_t, 0, c.dU, d, S, hs.prof_hat);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    } else if (raw) {
        k_user_project<T><<<L + 1, 128, c.dU * sizeof(float), st>>>((const T *)in->seq, (const T *)in->profile,
                                                                    (const T *)ctx->Wseq_t, (const T *)ctx->Wprofile_t, L,
                                                                    c.dU, d, S, hs.prof_hat);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    } else {
        if ((e = cudaMemcpyAsync(S, in->seq, (size_t)L * d * sizeof(T), cudaMemcpyDeviceToDevice, st)) != cudaSuccess) return e;
        if ((e = cudaMemcpyAsync((void *)hs.dev.u, in->profile, (size_t)d * sizeof(T), cudaMemcpyDeviceToDevice, st)) !=
            cudaSuccess)
            return e;
    }
    {   // zero the rows between L and the end of the last 128-key block, so that block-wise readers see no stale rows
        const int L_pad = (L + 127) / 128 * 128 < c.L_max ? (L + 127) / 128 * 128 : c.L_max;
        if (L_pad > L && (e = cudaMemsetAsync(S + (size_t)L * d, 0, (size_t)(L_pad - L) * d * sizeof(T), st)) != cudaSuccess) return e;
    }
    // the slot's length is set here already: the tensor-core self-attention below reads it like any scoring launch
    k_set_slot_len<<<1, 1, 0, st>>>(ctx->slots_dev, slot_index, L);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if ((e = launch_row_norm_max(ctx, S, nullptr, L, L, const_cast<float *>(hs.dev.k_norm), st)) != cudaSuccess) return e;
    if (raw) {
        // eq. 2: the attention rows on the tensor cores where the shape allows, else inside k_user_self
        const T *att_rows = nullptr;
        if (std::is_same<T, __nv_bfloat16>::value && ctx->tc_att_plan) {
            const void *rows = nullptr;
            if ((e = launch_self_att_tc(ctx, slot_index, L, st, &rows)) != cudaSuccess) return e;
            att_rows = static_cast<const T *>(rows);
        }
        const int slice = ((L + kProfParts - 1) / kProfParts + 31) / 32 * 32;
        k_user_prof<T><<<kProfParts / 8, 256, 0, st>>>(S, L, d, hs.prof_hat, slice, hs.ppart);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        const int n_warps = kUserPartials;
        if (tc_user && att_rows) {
            // hidden = ReLU(attention rows W_a^T + b_a) as a dense layer, then the pooling sums (the second FFN layer is
            // linear and is applied once to the pooled row, in k_user_finish)
            DenseLayer lay{};
            lay.A = att_rows, lay.W = ctx->Wa_k, lay.bias = ctx->b_a, lay.out = ctx->ffn_rows, lay.in_w = d, lay.H = d, lay.relu = 1, lay.sign_bits = 0;
            if ((e = tc_dense_layer(ctx, lay, L, st)) != cudaSuccess) return e;
            k_pool_rows<<<n_warps / 8, 256, 0, st>>>((const __nv_bfloat16 *)ctx->ffn_rows, L, d, n_warps, hs.partial);
        } else {
            k_user_self<T><<<n_warps / 8, 256, 8 * 3 * d * sizeof(float), st>>>(S, L, d, (const T *)ctx->Wa_t, ctx->b_a,
                                                                                (const T *)ctx->Wb_t, ctx->b_b, hs.partial,
                                                                                n_warps, att_rows);
        }
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    k_user_finish<T><<<1, 256, 0, st>>>(raw ? 1 : 0, S, L, d, hs.prof_hat, hs.partial, kUserPartials,
                                        (const T *)in->profile, (T *)hs.dev.u, (float *)hs.dev.u32, (const T *)ctx->Wt[0],
                                        ctx->b[0], H1, (float *)hs.dev.p_u, (__nv_bfloat16 *)hs.dev.pu_hl, (const T *)ctx->Wb_t, ctx->b_b, hs.ppart);
    count_launch();
    return cudaGetLastError();
}

// Algorithm 1 steps 1-2 for one user, one block: W = Softmax(B U^T / sqrt(d)) per bridge, A_k = sum_j W_kj U_j,
// V_k = W_f A_k.  Shared memory: W [n x m] and A [n x d] in fp32.
template <typename T>
__global__ void __launch_bounds__(256) k_bea_user(const T *__restrict__ Bm, const T *__restrict__ U, const T *__restrict__ Wf, int n, int m,
                                                  int d, T *__restrict__ V)
{
    extern __shared__ float sm_bea[];
    float *W = sm_bea, *A = sm_bea + n * m;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float scale = rsqrtf((float)d);
    for (int p = warp; p < n * m; p += 8) {   // one warp per (bridge, feature) pair
        const int k = p / m, j = p - k * m;
        float acc = 0.f;
        for (int c = lane; c < d; c += 32) acc = fmaf(to_f(Bm[(size_t)k * d + c]), to_f(U[(size_t)j * d + c]), acc);
        acc = warp_sum(acc);
        if (lane == 0) W[p] = acc * scale;
    }
    __syncthreads();
    for (int k = warp; k < n; k += 8) {       // one warp per bridge: softmax over the m features
        float mx = -INFINITY;
        for (int j = lane; j < m; j += 32) mx = fmaxf(mx, W[k * m + j]);
        mx = warp_max(mx);
        float den = 0.f;
        for (int j = lane; j < m; j += 32) den += expf(W[k * m + j] - mx);
        den = warp_sum(den);
        for (int j = lane; j < m; j += 32) W[k * m + j] = expf(W[k * m + j] - mx) / den;
    }
    __syncthreads();
    for (int p = tid; p < n * d; p += 256) {
        const int k = p / d, c = p - k * d;
        float acc = 0.f;
        for (int j = 0; j < m; ++j) acc = fmaf(W[k * m + j], to_f(U[(size_t)j * d + c]), acc);
        A[p] = acc;
    }
    __syncthreads();
    for (int p = tid; p < n * d; p += 256) {
        const int k = p / d, r = p - k * d;
        float acc = 0.f;
        for (int c = 0; c < d; ++c) acc = fmaf(to_f(Wf[(size_t)r * d + c]), A[k * d + c], acc);
        from_f(V[p], acc);
    }
}

cudaError_t launch_user_network(const aif_ctx *ctx, HostSlot &hs, int slot_index, const aif_user_inputs *in, int L,
                                cudaStream_t st)
{
    const aif_config &c = ctx->cfg;
    cudaError_t e;
    if (c.blocks & AIF_BLK_CROSS) {
        e = cudaMemcpyAsync((void *)hs.dev.T, in->cross_raw, (size_t)c.F * c.B * c.dc * ctx->el, cudaMemcpyDeviceToDevice, st);
        if (e != cudaSuccess) return e;
    }
    if ((c.blocks & AIF_BLK_BEA) && in->bea_V) {
        e = cudaMemcpyAsync((void *)hs.dev.V, in->bea_V, (size_t)c.n_bridge * c.d * ctx->el, cudaMemcpyDeviceToDevice, st);
        if (e != cudaSuccess) return e;
    } else if (c.blocks & AIF_BLK_BEA) {
        const size_t smem = (size_t)(c.n_bridge * in->bea_m + c.n_bridge * c.d) * 4;
        if (smem > 48 * 1024) {   // up to 80 KB at n_bridge = 16, bea_m = 1024, d = 256: beyond the default limit of a launch
            e = c.dtype == AIF_F32 ? cudaFuncSetAttribute(k_bea_user<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                                   : cudaFuncSetAttribute(k_bea_user<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
        }
        if (c.dtype == AIF_F32)
            k_bea_user<float><<<1, 256, smem, st>>>((const float *)ctx->bridges, (const float *)in->bea_U, (const float *)ctx->W_f, c.n_bridge,
                                                    in->bea_m, c.d, (float *)hs.dev.V);
        else
            k_bea_user<__nv_bfloat16><<<1, 256, smem, st>>>((const __nv_bfloat16 *)ctx->bridges, (const __nv_bfloat16 *)in->bea_U,
                                                            (const __nv_bfloat16 *)ctx->W_f, c.n_bridge, in->bea_m, c.d,
                                                            (__nv_bfloat16 *)hs.dev.V);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    if (c.blocks & (AIF_BLK_LSH_DIN | AIF_BLK_SIMTIER)) {
        e = cudaMemcpyAsync((void *)hs.dev.sigS, in->seq_sig, (size_t)L * (c.lsh_bits / 8), cudaMemcpyDeviceToDevice, st);
        if (e != cudaSuccess) return e;
        // the form the tensor-core LSH kernel multiplies: one +-1 byte per signature bit
        if (ctx->tc_lsh_plan && (e = launch_expand_signatures(ctx, in->seq_sig, L, const_cast<uint8_t *>(hs.dev.sigE), st)) != cudaSuccess) return e;
    }
    if (c.dtype == AIF_F32) return user_network_typed<float>(ctx, hs, slot_index, in, L, st);
    return user_network_typed<__nv_bfloat16>(ctx, hs, slot_index, in, L, st);
}

}  // namespace aif
