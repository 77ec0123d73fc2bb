// Item side of the nearline pipeline as a compute call (Section 3.2 eq. 4, Algorithm 1 step 3, Section 4.2 eq. 5):
// raw item features -> item vectors, BEA weight rows and LSH signatures, written into the item table.
//
// bf16 contexts whose widths fit run on the tensor cores: the tower as one kernel with its hidden activations in tensor
// memory (aif_tc_tower.cu; hidden width <= 256, d <= 128) or as two launches of the scoring MLP's layer kernel over dense
// rows (tc_dense_layer, linear-output epilogue), the hash projections as one such launch with a sign-bit epilogue; every
// other case runs the CUDA-core kernels below.  The BEA weights are 2 n d flop per item against d element reads: a
// warp per item on CUDA cores.  Items are processed in passes of at most kPassRows rows so that the scratch
// (hidden activations; for incremental updates also the rows before their scatter) stays bounded.
#include <new>

#include "aif_device.cuh"
#include "aif_internal.h"

namespace aif {
namespace {

constexpr int64_t kPassRows = 1 << 20;

struct NearlinePlan {
    int dI = 0, hI = 0, d_mm = 0;
    bool ready = false, tensor = false;
    bool fused_tower = false;             // both tower layers in one kernel (hidden activations in tensor memory)
    void *W0 = nullptr, *W1 = nullptr, *bridges = nullptr, *W_hash = nullptr;
    float *b0 = nullptr, *b1 = nullptr, *zeros = nullptr;
    int64_t cap = 0;                      // rows per pass the scratch has room for
    void *hidden = nullptr;               // [cap x hI] bf16 (tensor path)
    void *rows = nullptr, *bea = nullptr; // incremental updates: computed rows before the scatter
    uint8_t *sig = nullptr;
};

NearlinePlan *plan_of(const aif_ctx *ctx) { return reinterpret_cast<NearlinePlan *>(ctx->nearline_plan); }

// eq. 4 on CUDA cores: one warp per item; x and the hidden activations in shared memory.
template <typename T>
__global__ void __launch_bounds__(256) k_item_tower(const T *__restrict__ I_raw, int64_t n, int dI, int hI, int d, const T *__restrict__ W0,
                                                    const float *__restrict__ b0, const T *__restrict__ W1,
                                                    const float *__restrict__ b1, T *__restrict__ out)
{
    extern __shared__ float sm_f[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float *x = sm_f + (size_t)warp * (dI + hI), *h = x + dI;
    for (int64_t i = (int64_t)blockIdx.x * 8 + warp; i < n; i += (int64_t)gridDim.x * 8) {
        for (int c = lane; c < dI; c += 32) x[c] = to_f(I_raw[i * dI + c]);
        __syncwarp();
        for (int j = lane; j < hI; j += 32) {
            float acc = b0[j];
            const T *w = W0 + (size_t)j * dI;
            for (int c = 0; c < dI; ++c) acc = fmaf(to_f(w[c]), x[c], acc);
            h[j] = fmaxf(acc, 0.f);
        }
        __syncwarp();
        for (int k = lane; k < d; k += 32) {
            float acc = b1[k];
            const T *w = W1 + (size_t)k * hI;
            for (int j = 0; j < hI; ++j) acc = fmaf(to_f(w[j]), h[j], acc);
            from_f(out[i * d + k], acc);
        }
        __syncwarp();
    }
}

// Algorithm 1 step 3: w^ = Softmax(I_id B^T / sqrt(d)), one warp per item, n_bridge <= 32.
template <typename T>
__global__ void __launch_bounds__(256) k_item_bridge_weights(const T *__restrict__ I_id, int64_t n, int d, int nb, const T *__restrict__ Bm,
                                                             T *__restrict__ out)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float scale = rsqrtf((float)d);
    for (int64_t i = (int64_t)blockIdx.x * 8 + warp; i < n; i += (int64_t)gridDim.x * 8) {
        float mine = -INFINITY;   // lane k ends up with the score of bridge k
        for (int k = 0; k < nb; ++k) {
            float acc = 0.f;
            for (int c = lane; c < d; c += 32) acc = fmaf(to_f(I_id[i * d + c]), to_f(Bm[(size_t)k * d + c]), acc);
            acc = warp_sum(acc) * scale;
            if (lane == k) mine = acc;
        }
        const float mx = warp_max(mine);
        const float e = lane < nb ? expf(mine - mx) : 0.f;
        const float den = warp_sum(e);
        if (lane < nb) from_f(out[i * nb + lane], e / den);
    }
}

// eq. 5 on CUDA cores: one warp per item, 32 bits per round; eight bits per byte, first bit most significant.
template <typename T>
__global__ void __launch_bounds__(256) k_item_signatures(const T *__restrict__ M_mm, int64_t n, int d_mm, int bits, const T *__restrict__ W_hash,
                                                         uint8_t *__restrict__ sig)
{
    extern __shared__ float sm_f[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float *x = sm_f + (size_t)warp * d_mm;
    for (int64_t i = (int64_t)blockIdx.x * 8 + warp; i < n; i += (int64_t)gridDim.x * 8) {
        for (int c = lane; c < d_mm; c += 32) x[c] = to_f(M_mm[i * d_mm + c]);
        __syncwarp();
        for (int k0 = 0; k0 < bits; k0 += 32) {
            const T *w = W_hash + (size_t)(k0 + lane) * d_mm;
            float acc = 0.f;
            for (int c = 0; c < d_mm; ++c) acc = fmaf(to_f(w[c]), x[c], acc);
            const uint32_t ballot = __ballot_sync(0xffffffffu, acc > 0.f);   // lane j -> bit j
            // lane 0's bit must become the top bit of the first byte in memory
            const uint32_t word = __byte_perm(__brev(ballot), 0u, 0x0123);
            if (lane == 0) *reinterpret_cast<uint32_t *>(sig + i * (bits >> 3) + (k0 >> 3)) = word;
        }
        __syncwarp();
    }
}

cudaError_t take(aif_ctx *ctx, void **p, size_t bytes)
{
    bytes = (bytes + 255) / 256 * 256;
    cudaError_t e = cudaMalloc(p, bytes);
    if (e != cudaSuccess) return e;
    ctx->allocations.push_back(*p);
    ctx->device_bytes += (int64_t)bytes;
    return cudaMemset(*p, 0, bytes);
}

int grid_for_items(int64_t n) { return (int)((n + 7) / 8 < 148 * 8 ? (n + 7) / 8 : 148 * 8); }

template <typename T>
cudaError_t run_pass(aif_ctx *ctx, NearlinePlan *pl, int64_t m, const void *I_raw, const void *I_id, const void *M_mm, void *rows_out,
                     void *bea_out, uint8_t *sig_out, cudaStream_t st)
{
    const aif_config &c = ctx->cfg;
    cudaError_t e;
    if (pl->tensor && pl->fused_tower) {
        // the kernel also raises the table's norm bound from the rows it writes
        if ((e = launch_item_tower_tc(ctx, I_raw, pl->W0, pl->b0, pl->W1, pl->b1, rows_out, m, pl->dI, pl->hI, ctx->e_norm, st)) != cudaSuccess) return e;
    } else if (pl->tensor) {
        DenseLayer l0{I_raw, pl->W0, pl->b0, pl->hidden, pl->dI, pl->hI, 1, 0};
        if ((e = tc_dense_layer(ctx, l0, m, st)) != cudaSuccess) return e;
        DenseLayer l1{pl->hidden, pl->W1, pl->b1, rows_out, pl->hI, c.d, 0, 0};
        if ((e = tc_dense_layer(ctx, l1, m, st)) != cudaSuccess) return e;
    } else {
        k_item_tower<T><<<grid_for_items(m), 256, (size_t)8 * (pl->dI + pl->hI) * 4, st>>>(
            (const T *)I_raw, m, pl->dI, pl->hI, c.d, (const T *)pl->W0, pl->b0, (const T *)pl->W1, pl->b1, (T *)rows_out);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    // the table's norm bound from the rows just computed (whether or not their ids turn out to lie in the table)
    if (!(pl->tensor && pl->fused_tower) && (e = launch_row_norm_max(ctx, rows_out, nullptr, m, m, ctx->e_norm, st)) != cudaSuccess) return e;
    if (c.blocks & AIF_BLK_BEA) {
        k_item_bridge_weights<T><<<grid_for_items(m), 256, 0, st>>>((const T *)(I_id ? I_id : rows_out), m, c.d, c.n_bridge,
                                                                    (const T *)pl->bridges, (T *)bea_out);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    if (c.blocks & (AIF_BLK_LSH_DIN | AIF_BLK_SIMTIER)) {
        if (pl->tensor) {
            DenseLayer lh{M_mm, pl->W_hash, pl->zeros, sig_out, pl->d_mm, c.lsh_bits, 0, 1};
            if ((e = tc_dense_layer(ctx, lh, m, st)) != cudaSuccess) return e;
        } else {
            k_item_signatures<T><<<grid_for_items(m), 256, (size_t)8 * pl->d_mm * 4, st>>>((const T *)M_mm, m, pl->d_mm, c.lsh_bits,
                                                                                          (const T *)pl->W_hash, sig_out);
            count_launch();
            if ((e = cudaGetLastError()) != cudaSuccess) return e;
        }
    }
    return cudaSuccess;
}

}  // namespace

int nearline_load_weights(aif_ctx *ctx, const aif_item_weights *w, cudaStream_t st)
{
    const aif_config &c = ctx->cfg;
    const bool bea = c.blocks & AIF_BLK_BEA, lsh = c.blocks & (AIF_BLK_LSH_DIN | AIF_BLK_SIMTIER);
    if (!w->W_i0 || !w->b_i0 || !w->W_i1 || !w->b_i1 || (bea && !w->bridges) || (lsh && !w->W_hash)) return AIF_ERR_ARG;
    if (w->dI < 4 || w->hI < 4 || w->dI % 4 || w->hI % 4 || (lsh && (w->d_mm < 4 || w->d_mm % 4 || c.lsh_bits % 32))) return AIF_ERR_SHAPE;
    if (bea && c.n_bridge > 32) return AIF_ERR_SHAPE;
    if ((size_t)(w->dI + w->hI) * 32 > 48 * 1024 || (size_t)w->d_mm * 32 > 48 * 1024) return AIF_ERR_SHAPE;   // CUDA-core kernels' shared memory
    NearlinePlan *pl = plan_of(ctx);
    if (pl && (pl->dI != w->dI || pl->hI != w->hI || pl->d_mm != w->d_mm)) return AIF_ERR_SHAPE;   // widths are fixed by the first call
    const size_t el = ctx->el;
    if (!pl) {
        pl = new (std::nothrow) NearlinePlan();
        if (!pl) return AIF_ERR_OOM;
        ctx->nearline_plan = pl;
        pl->dI = w->dI, pl->hI = w->hI, pl->d_mm = w->d_mm;
        const int H = w->hI;
        pl->tensor = ctx->tensor_path && w->dI % 64 == 0 && H % 64 == 0 && (H <= 256 || H % 256 == 0) && w->dI <= 4096 && H <= 4096 &&
                     c.d % 32 == 0 && c.d <= 256 && (!lsh || (w->d_mm % 64 == 0 && w->d_mm <= 4096 && c.lsh_bits <= 256));
        pl->fused_tower = pl->tensor && tc_tower_supported(w->dI, H, c.d) && tc_tower_prepare() == cudaSuccess;
        pl->cap = c.M < kPassRows ? c.M : kPassRows;
        cudaError_t e = cudaSuccess;
        auto need = [&](void **p, size_t bytes) {
            if (e == cudaSuccess) e = take(ctx, p, bytes);
        };
        need(&pl->W0, (size_t)w->hI * w->dI * el);
        need(&pl->W1, (size_t)c.d * w->hI * el);
        need((void **)&pl->b0, (size_t)w->hI * 4);
        need((void **)&pl->b1, (size_t)c.d * 4);
        need((void **)&pl->zeros, 4096 * 4);
        if (bea) need(&pl->bridges, (size_t)c.n_bridge * c.d * el);
        if (lsh) need(&pl->W_hash, (size_t)c.lsh_bits * w->d_mm * el);
        if (pl->tensor && !pl->fused_tower) need(&pl->hidden, (size_t)(pl->cap + kTcTile) * w->hI * 2);
        need(&pl->rows, (size_t)(pl->cap + kTcTile) * c.d * el);
        if (bea) need(&pl->bea, (size_t)pl->cap * c.n_bridge * el);
        if (lsh) need((void **)&pl->sig, (size_t)(pl->cap + kTcTile) * c.lsh_bits / 8);
        if (e != cudaSuccess) {
            cudaGetLastError();
            set_last_error("item-side weights: out of device memory");
            return AIF_ERR_OOM;
        }
    }
    auto copy = [&](void *dst, const void *src, size_t bytes) { return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, st); };
    cudaError_t e = copy(pl->W0, w->W_i0, (size_t)w->hI * w->dI * el);
    if (e == cudaSuccess) e = copy(pl->W1, w->W_i1, (size_t)c.d * w->hI * el);
    if (e == cudaSuccess) e = copy(pl->b0, w->b_i0, (size_t)w->hI * 4);
    if (e == cudaSuccess) e = copy(pl->b1, w->b_i1, (size_t)c.d * 4);
    if (e == cudaSuccess && bea) e = copy(pl->bridges, w->bridges, (size_t)c.n_bridge * c.d * el);
    if (e == cudaSuccess && lsh) e = copy(pl->W_hash, w->W_hash, (size_t)c.lsh_bits * w->d_mm * el);
    if (e != cudaSuccess) {
        set_last_error(cudaGetErrorString(e));
        return AIF_ERR_CUDA;
    }
    pl->ready = true;
    return AIF_OK;
}

int nearline_compute(aif_ctx *ctx, const int32_t *ids, int64_t n, const void *I_raw, const void *I_id, const void *M_mm, cudaStream_t st)
{
    NearlinePlan *pl = plan_of(ctx);
    if (!pl || !pl->ready) return AIF_ERR_NOT_READY;
    const aif_config &c = ctx->cfg;
    const bool bea = c.blocks & AIF_BLK_BEA, lsh = c.blocks & (AIF_BLK_LSH_DIN | AIF_BLK_SIMTIER);
    const size_t el = ctx->el;
    for (int64_t off = 0; off < n; off += pl->cap) {
        const int64_t m = n - off < pl->cap ? n - off : pl->cap;
        const char *raw = (const char *)I_raw + (size_t)off * pl->dI * el;
        const char *iid = I_id ? (const char *)I_id + (size_t)off * c.d * el : nullptr;
        const char *mm = lsh ? (const char *)M_mm + (size_t)off * pl->d_mm * el : nullptr;
        // a full refresh writes straight into the table; an incremental one goes through scratch and the scatter kernel
        void *rows_out = ids ? pl->rows : (char *)ctx->E + (size_t)off * c.d * el;
        void *bea_out = !bea ? nullptr : ids ? pl->bea : (char *)ctx->bea_w + (size_t)off * c.n_bridge * el;
        uint8_t *sig_out = !lsh ? nullptr : ids ? pl->sig : ctx->sig + (size_t)off * c.lsh_bits / 8;
        cudaError_t e = el == 4 ? run_pass<float>(ctx, pl, m, raw, iid, mm, rows_out, bea_out, sig_out, st)
                                : run_pass<__nv_bfloat16>(ctx, pl, m, raw, iid, mm, rows_out, bea_out, sig_out, st);
        if (e == cudaSuccess && ids) e = launch_scatter_rows(ctx, ids + off, m, rows_out, bea_out, sig_out, st);
        if (e != cudaSuccess) {
            set_last_error(cudaGetErrorString(e));
            return AIF_ERR_CUDA;
        }
    }
    return AIF_OK;
}

void nearline_destroy(aif_ctx *ctx)
{
    delete plan_of(ctx);
    ctx->nearline_plan = nullptr;
}

}  // namespace aif
