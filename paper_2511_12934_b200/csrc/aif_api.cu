// Host side of libaif: context, arena, weight copies, and the extern "C" entry points.
#include <cstdio>
#include <cstring>
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "aif_internal.h"

using namespace aif;

namespace {

thread_local char g_last_error[256] = "";

int cuda_fail(cudaError_t e, const char *what)
{
    snprintf(g_last_error, sizeof(g_last_error), "%s: %s", what, cudaGetErrorString(e));
    cudaGetLastError();   // clear the sticky-free error state
    return AIF_ERR_CUDA;
}

#define AIF_CUDA(call)                                     \
    do {                                                   \
        cudaError_t e__ = (call);                          \
        if (e__ != cudaSuccess) return cuda_fail(e__, #call); \
    } while (0)

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

int dev_alloc(aif_ctx *ctx, void **p, size_t bytes, bool zero)
{
    bytes = align_up(bytes ? bytes : 1, 256);
    cudaError_t e = cudaMalloc(p, bytes);
    if (e != cudaSuccess) {
        cudaGetLastError();
        snprintf(g_last_error, sizeof(g_last_error), "cudaMalloc(%zu): %s", bytes, cudaGetErrorString(e));
        return AIF_ERR_OOM;
    }
    ctx->allocations.push_back(*p);
    ctx->device_bytes += (int64_t)bytes;
    if (zero) AIF_CUDA(cudaMemset(*p, 0, bytes));
    return AIF_OK;
}

bool mult(int v, int m) { return v > 0 && v % m == 0; }

int check_config(const aif_config *c)
{
    if (!c || c->struct_size != sizeof(aif_config)) return AIF_ERR_ARG;
    if (c->dtype != AIF_F32 && c->dtype != AIF_BF16) return AIF_ERR_ARG;
    if (c->M <= 0 || c->M >= (int64_t)1 << 31) return AIF_ERR_SHAPE;
    if (!mult(c->d, 32) || c->d > 256) return AIF_ERR_SHAPE;
    if (!mult(c->dU, 4) || c->L_max < 1) return AIF_ERR_SHAPE;
    if (c->n_hidden < 1 || c->n_hidden > 4) return AIF_ERR_SHAPE;
    for (int k = 0; k < c->n_hidden; ++k)
        if (!mult(c->hidden[k], 8) || c->hidden[k] > 1024) return AIF_ERR_SHAPE;
    if (c->blocks & ~(AIF_BLK_ATT | AIF_BLK_CROSS | AIF_BLK_BEA | AIF_BLK_LSH_DIN | AIF_BLK_SIMTIER)) return AIF_ERR_ARG;
    if (c->blocks & AIF_BLK_CROSS) {
        if (c->F < 1 || c->F > 256 || c->B < 1 || !mult(c->dc, 8)) return AIF_ERR_SHAPE;
        if (c->bucket_mode != AIF_BUCKET_MOD && c->bucket_mode != AIF_BUCKET_HASH) return AIF_ERR_ARG;
    }
    if ((c->blocks & AIF_BLK_BEA) && (c->n_bridge < 1 || c->n_bridge > 16)) return AIF_ERR_SHAPE;
    if (c->blocks & (AIF_BLK_LSH_DIN | AIF_BLK_SIMTIER)) {
        if (!mult(c->lsh_bits, 32) || c->lsh_bits > 256) return AIF_ERR_SHAPE;
        if ((c->blocks & AIF_BLK_SIMTIER) && (c->n_tiers < 1 || c->n_tiers > 16)) return AIF_ERR_SHAPE;
    }
    if (c->max_user_states < 1 || c->mini_batch < 0 || c->max_batch_candidates < 1) return AIF_ERR_SHAPE;
    if (c->path < AIF_PATH_AUTO || c->path > AIF_PATH_TENSOR) return AIF_ERR_ARG;
    if (c->n_categories < 0 || c->n_categories > 4096) return AIF_ERR_SHAPE;
    if (c->versioned_table != 0 && c->versioned_table != 1) return AIF_ERR_ARG;
    if (c->n_categories > 0 && c->bucket_mode != AIF_BUCKET_MOD && c->bucket_mode != AIF_BUCKET_HASH) return AIF_ERR_ARG;
    return AIF_OK;
}

cudaStream_t as_stream(aif_stream s) { return reinterpret_cast<cudaStream_t>(s); }

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) ok = false;
        else if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard()
    {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

int state_check(aif_ctx *ctx, const aif_user_state *st)
{
    if (!ctx || !st || st->ctx != ctx || st->index < 0 || st->index >= (int)ctx->slots.size()) return AIF_ERR_ARG;
    const HostSlot &hs = ctx->slots[st->index];
    if (!hs.in_use || !hs.ready) return AIF_ERR_NOT_READY;
    if (hs.model_version != ctx->model_version) return AIF_ERR_VERSION;
    return AIF_OK;
}

int tiles_for(const aif_ctx *ctx, int n) { return ctx->tensor_path ? tc_tiles_for(ctx, n) : simt_tiles_for(ctx, n); }

int run_score(aif_ctx *ctx, const ScoreLaunch &sl, int64_t total, cudaStream_t st)
{
    cudaError_t e = ctx->tensor_path ? launch_score_tc(ctx, sl, total, st) : launch_score_simt(ctx, sl, st);
    if (e != cudaSuccess) return cuda_fail(e, "score launch");
    ctx->stats.score_calls += 1;
    ctx->stats.candidates_scored += (uint64_t)total;
    return AIF_OK;
}

}  // namespace

namespace aif {

int check_user_state(aif_ctx *ctx, const aif_user_state *st) { return state_check(ctx, st); }

cudaError_t wait_table_ready(const aif_ctx *ctx, cudaStream_t st)
{
    if (!ctx->table_ev_pending) return cudaSuccess;
    const cudaError_t q = cudaEventQuery(ctx->table_ev);
    if (q == cudaSuccess) {
        ctx->table_ev_pending = false;
        return cudaSuccess;
    }
    if (q != cudaErrorNotReady) return q;
    (void)cudaGetLastError();
    return cudaStreamWaitEvent(st, ctx->table_ev, 0);
}

// Versioned table, full refresh: the spare copy becomes the one every writer and (from now on) every reader addresses;
// rows the refresh does not cover are carried over from the copy that was live.
static cudaError_t begin_full_refresh(aif_ctx *ctx, int64_t n, cudaStream_t st)
{
    const aif_config &c = ctx->cfg;
    // the copies are written on `st`: it must be behind the previous full refresh, whose copy is the source of the rows carried over
    cudaError_t e = wait_table_ready(ctx, st);
    if (e != cudaSuccess) return e;
    std::swap(ctx->E, ctx->E_alt), std::swap(ctx->bea_w, ctx->bea_w_alt), std::swap(ctx->sig, ctx->sig_alt);
    if (n < c.M) {
        const size_t rest = (size_t)(c.M - n);
        e = cudaMemcpyAsync((char *)ctx->E + (size_t)n * c.d * ctx->el, (const char *)ctx->E_alt + (size_t)n * c.d * ctx->el, rest * c.d * ctx->el,
                            cudaMemcpyDeviceToDevice, st);
        if (e == cudaSuccess && ctx->bea_w)
            e = cudaMemcpyAsync((char *)ctx->bea_w + (size_t)n * c.n_bridge * ctx->el, (const char *)ctx->bea_w_alt + (size_t)n * c.n_bridge * ctx->el,
                                rest * c.n_bridge * ctx->el, cudaMemcpyDeviceToDevice, st);
        if (e == cudaSuccess && ctx->sig)
            e = cudaMemcpyAsync(ctx->sig + (size_t)n * c.lsh_bits / 8, ctx->sig_alt + (size_t)n * c.lsh_bits / 8, rest * c.lsh_bits / 8,
                                cudaMemcpyDeviceToDevice, st);
    }
    return e;
}

static cudaError_t end_full_refresh(aif_ctx *ctx, cudaStream_t st)
{
    const cudaError_t e = cudaEventRecord(ctx->table_ev, st);
    ctx->table_ev_pending = e == cudaSuccess;
    return e;
}

StageRange::StageRange(const char *name) { nvtxRangePushA(name); }
StageRange::~StageRange() { nvtxRangePop(); }

void set_last_error(const char *text) { snprintf(g_last_error, sizeof(g_last_error), "%s", text); }

void timing_begin(const aif_ctx *ctx, cudaStream_t st)
{
    KernelTiming &t = ctx->timing;
    if (!t.on) return;
    t.n = 0;
    cudaEventRecord(t.ev[0], st);
}

void timing_mark(const aif_ctx *ctx, const char *name, cudaStream_t st)
{
    KernelTiming &t = ctx->timing;
    if (!t.on || t.n >= KernelTiming::kMax) return;
    t.names[t.n] = name;
    t.n += 1;
    cudaEventRecord(t.ev[t.n], st);
}

ModelDev make_model(const aif_ctx *ctx)
{
    const aif_config &c = ctx->cfg;
    ModelDev m{};
    m.d = c.d, m.F = c.F, m.B = c.B, m.dc = c.dc, m.n_hidden = c.n_hidden;
    for (int k = 0; k < kMaxHidden; ++k) {
        m.hidden[k] = c.hidden[k];
        m.Wt[k] = ctx->Wt[k];
        m.b[k] = ctx->b[k];
    }
    m.bucket_mode = c.bucket_mode, m.blocks = c.blocks, m.n_bridge = c.n_bridge, m.lsh_bits = c.lsh_bits;
    m.n_tiers = c.n_tiers, m.lsh_din_norm = c.lsh_din_norm, m.simtier_norm = c.simtier_norm;
    m.emit_sigmoid = c.emit_sigmoid, m.k1 = ctx->input_width - c.d, m.mini_batch = c.mini_batch, m.M = c.M;
    m.E = ctx->E, m.bea_w = ctx->bea_w, m.sig = ctx->sig, m.w_out = ctx->w_out, m.b_out = ctx->b_out;
    return m;
}

}  // namespace aif

extern "C" {

int aif_input_width(const aif_config *c)
{
    if (!c) return AIF_ERR_ARG;
    int w = 2 * c->d;
    if (c->blocks & AIF_BLK_ATT) w += c->d;
    if (c->blocks & AIF_BLK_CROSS) w += c->F * c->dc;
    if (c->blocks & AIF_BLK_BEA) w += c->d;
    if (c->blocks & AIF_BLK_LSH_DIN) w += c->d;
    if (c->blocks & AIF_BLK_SIMTIER) w += c->n_tiers;
    return w;
}

int64_t aif_category(int64_t id, int32_t n_categories, int32_t bucket_mode)
{
    if (n_categories < 1) return 0;
    if (bucket_mode == AIF_BUCKET_MOD) return id % n_categories;
    return (int64_t)(aif_mix64((uint64_t)id, (uint64_t)AIF_CATEGORY_FIELD) % (uint64_t)n_categories);
}

uint64_t aif_mix64(uint64_t id, uint64_t field)
{
    uint64_t z = id * 0x9E3779B97F4A7C15ull + field;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

int aif_create(const aif_config *cfg, aif_ctx **out)
{
    if (!out) return AIF_ERR_ARG;
    *out = nullptr;
    int rc = check_config(cfg);
    if (rc != AIF_OK) return rc;
    aif_ctx *ctx = new (std::nothrow) aif_ctx();
    if (!ctx) return AIF_ERR_OOM;
    ctx->cfg = *cfg;
    const aif_config &c = ctx->cfg;
    ctx->el = c.dtype == AIF_F32 ? 4 : 2;
    ctx->input_width = aif_input_width(cfg);
    if (cudaGetDevice(&ctx->device) != cudaSuccess) {
        delete ctx;
        return cuda_fail(cudaGetLastError(), "cudaGetDevice");
    }
    if (c.path == AIF_PATH_TENSOR && !tc_supported(c)) {
        delete ctx;
        return AIF_ERR_SHAPE;
    }
    ctx->tensor_path = c.path != AIF_PATH_SIMT && tc_supported(c);
    if (c.n_categories > 0) {
        // sub-sequences by category are a feature of the tensor-core kernels: every sequence block that is on must be one
        // of theirs
        const bool att_ok = !(c.blocks & AIF_BLK_ATT) || tc_att_supported(c);
        const bool lsh_ok = !(c.blocks & (AIF_BLK_LSH_DIN | AIF_BLK_SIMTIER)) || tc_lsh_supported(c);
        if (!ctx->tensor_path || !att_ok || !lsh_ok) {
            delete ctx;
            set_last_error("n_categories > 0 needs bf16 storage and d = 128 or 256 (tensor-core attention and LSH kernels)");
            return AIF_ERR_SHAPE;
        }
        ctx->grouped_rows = sim_grouped_rows(c.L_max, c.n_categories);
    }

#define TRY(x)                 \
    do {                       \
        rc = (x);              \
        if (rc != AIF_OK) {    \
            aif_destroy(ctx);  \
            return rc;         \
        }                      \
    } while (0)

    const size_t el = ctx->el;
    TRY(dev_alloc(ctx, &ctx->E, (size_t)c.M * c.d * el, true));
    if (c.blocks & AIF_BLK_BEA) TRY(dev_alloc(ctx, &ctx->bea_w, (size_t)c.M * c.n_bridge * el, true));
    if (c.blocks & (AIF_BLK_LSH_DIN | AIF_BLK_SIMTIER)) TRY(dev_alloc(ctx, (void **)&ctx->sig, (size_t)c.M * c.lsh_bits / 8, true));
    TRY(dev_alloc(ctx, (void **)&ctx->e_norm, 4, true));
    if (c.versioned_table) {
        TRY(dev_alloc(ctx, &ctx->E_alt, (size_t)c.M * c.d * el, true));
        if (ctx->bea_w) TRY(dev_alloc(ctx, &ctx->bea_w_alt, (size_t)c.M * c.n_bridge * el, true));
        if (ctx->sig) TRY(dev_alloc(ctx, (void **)&ctx->sig_alt, (size_t)c.M * c.lsh_bits / 8, true));
        if (cudaEventCreateWithFlags(&ctx->table_ev, cudaEventDisableTiming) != cudaSuccess) {
            aif_destroy(ctx);
            return cuda_fail(cudaGetLastError(), "cudaEventCreate");
        }
    }
    TRY(dev_alloc(ctx, (void **)&ctx->status, 256, true));

    // weights
    int in_w = ctx->input_width;
    for (int k = 0; k < c.n_hidden; ++k) {
        TRY(dev_alloc(ctx, &ctx->Wt[k], (size_t)in_w * c.hidden[k] * el, true));
        TRY(dev_alloc(ctx, (void **)&ctx->b[k], (size_t)c.hidden[k] * 4, true));
        in_w = c.hidden[k];
    }
    TRY(dev_alloc(ctx, &ctx->w_out, (size_t)in_w * el, true));
    TRY(dev_alloc(ctx, (void **)&ctx->b_out, 4, true));
    TRY(dev_alloc(ctx, &ctx->Wprofile_t, (size_t)c.dU * c.d * el, true));
    TRY(dev_alloc(ctx, &ctx->Wseq_t, (size_t)c.dU * c.d * el, true));
    TRY(dev_alloc(ctx, &ctx->Wa_t, (size_t)c.d * c.d * el, true));
    TRY(dev_alloc(ctx, &ctx->Wb_t, (size_t)c.d * c.d * el, true));
    TRY(dev_alloc(ctx, &ctx->Wseq_k, (size_t)c.dU * c.d * el, true));
    TRY(dev_alloc(ctx, &ctx->Wa_k, (size_t)c.d * c.d * el, true));
    TRY(dev_alloc(ctx, (void **)&ctx->zero_bias, 256 * 4, true));
    if (ctx->tensor_path) TRY(dev_alloc(ctx, &ctx->ffn_rows, ((size_t)c.L_max + 128) * c.d * 2, true));
    TRY(dev_alloc(ctx, (void **)&ctx->b_a, (size_t)c.d * 4, true));
    TRY(dev_alloc(ctx, (void **)&ctx->b_b, (size_t)c.d * 4, true));

    // user-state arena: fixed-size slots in one allocation
    struct Off { size_t u, u32, S, T, V, sig, sigE, pu, pu_hl, prof, partial, ppart, Sg, sigEg, cat_off, cat_len, cat_map, cat_hist, k_norm, end; } o{};
    size_t p = 0;
    auto take = [&](size_t bytes) { size_t at = p; p += align_up(bytes ? bytes : 16, 256); return at; };
    o.u = take((size_t)c.d * el);
    o.u32 = take((size_t)c.d * 4);
    o.S = take((size_t)c.L_max * c.d * el);
    o.T = take((c.blocks & AIF_BLK_CROSS) ? (size_t)c.F * c.B * c.dc * el : 0);
    o.V = take((c.blocks & AIF_BLK_BEA) ? (size_t)c.n_bridge * c.d * el : 0);
    o.sig = take((c.blocks & (AIF_BLK_LSH_DIN | AIF_BLK_SIMTIER)) ? (size_t)c.L_max * c.lsh_bits / 8 : 0);
    const bool lsh_tc = ctx->tensor_path && tc_lsh_supported(c);
    o.sigE = take(lsh_tc ? (size_t)c.L_max * c.lsh_bits : 0);
    o.pu = take((size_t)c.hidden[0] * 4);
    o.pu_hl = take((size_t)c.hidden[0] * 2 * 2);
    o.prof = take((size_t)c.d * 4);
    o.partial = take((size_t)kUserPartials * c.d * 4);
    o.ppart = take((size_t)kProfParts * (c.d + 2) * 4);
    const bool sim = c.n_categories > 0;
    o.Sg = take(sim ? ctx->grouped_rows * c.d * el : 0);
    o.sigEg = take(sim && lsh_tc ? ctx->grouped_rows * c.lsh_bits : 0);
    o.cat_off = take(sim ? (size_t)c.n_categories * 4 : 0);
    o.cat_len = take(sim ? (size_t)c.n_categories * 4 : 0);
    o.cat_map = take(sim ? (size_t)c.L_max * 4 : 0);
    o.cat_hist = take(sim ? (size_t)((c.L_max + 1023) / 1024) * c.n_categories * 4 : 0);
    o.k_norm = take(4);
    o.end = p;
    ctx->slot_bytes = o.end;
    TRY(dev_alloc(ctx, (void **)&ctx->arena, ctx->slot_bytes * (size_t)c.max_user_states, true));
    TRY(dev_alloc(ctx, (void **)&ctx->slots_dev, sizeof(SlotDev) * (size_t)c.max_user_states, true));
    ctx->slots.resize((size_t)c.max_user_states);
    ctx->handles.resize((size_t)c.max_user_states);
    std::vector<SlotDev> host_slots((size_t)c.max_user_states);
    for (int i = 0; i < c.max_user_states; ++i) {
        char *base = ctx->arena + (size_t)i * ctx->slot_bytes;
        HostSlot &hs = ctx->slots[(size_t)i];
        hs.dev.u = base + o.u, hs.dev.u32 = (const float *)(base + o.u32), hs.dev.S = base + o.S;
        hs.dev.T = base + o.T, hs.dev.V = base + o.V, hs.dev.sigS = (const uint8_t *)(base + o.sig);
        hs.dev.sigE = lsh_tc ? (const uint8_t *)(base + o.sigE) : nullptr;
        hs.dev.p_u = (const float *)(base + o.pu), hs.dev.pu_hl = base + o.pu_hl, hs.dev.L = 0;
        hs.dev.k_norm = (const float *)(base + o.k_norm);
        hs.prof_hat = (float *)(base + o.prof), hs.partial = (float *)(base + o.partial), hs.ppart = (float *)(base + o.ppart);
        if (sim) {
            hs.dev.Sg = base + o.Sg, hs.dev.sigEg = lsh_tc ? (const uint8_t *)(base + o.sigEg) : nullptr;
            hs.dev.cat_off = (const int32_t *)(base + o.cat_off), hs.dev.cat_len = (const int32_t *)(base + o.cat_len);
            hs.cat_map = (int32_t *)(base + o.cat_map), hs.cat_hist = (int32_t *)(base + o.cat_hist);
        }
        cudaError_t e = cudaEventCreateWithFlags(&hs.ev, cudaEventDisableTiming);
        if (e != cudaSuccess) {
            aif_destroy(ctx);
            return cuda_fail(e, "cudaEventCreate");
        }
        host_slots[(size_t)i] = hs.dev;
        ctx->handles[(size_t)i] = aif_user_state{ctx, i};
    }
    {
        cudaError_t e = cudaMemcpy(ctx->slots_dev, host_slots.data(), sizeof(SlotDev) * host_slots.size(), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            aif_destroy(ctx);
            return cuda_fail(e, "cudaMemcpy slots");
        }
    }

    // scratch
    TRY(dev_alloc(ctx, (void **)&ctx->ids_stage, (size_t)c.max_batch_candidates * 4, false));
    TRY(dev_alloc(ctx, (void **)&ctx->logits_stage, (size_t)c.max_batch_candidates * 4, false));
    if (ctx->tensor_path) {
        cudaError_t e = tc_prepare_context(ctx);
        if (e != cudaSuccess) {
            aif_destroy(ctx);
            return e == cudaErrorMemoryAllocation ? AIF_ERR_OOM : cuda_fail(e, "tensor-path setup");
        }
    }

    // pinned ring for the request table of aif_score_batch
    ctx->ring.capacity = c.max_user_states;
    for (int i = 0; i < PinnedRing::kSlots; ++i) {
        cudaError_t e = cudaMallocHost((void **)&ctx->ring.host[i], sizeof(ReqDev) * (size_t)ctx->ring.capacity);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ring.ev[i], cudaEventDisableTiming);
        if (e != cudaSuccess) {
            aif_destroy(ctx);
            return cuda_fail(e, "pinned ring");
        }
        TRY(dev_alloc(ctx, (void **)&ctx->ring.dev[i], sizeof(ReqDev) * (size_t)ctx->ring.capacity, true));
    }
#undef TRY
    AIF_CUDA(cudaDeviceSynchronize());
    *out = ctx;
    return AIF_OK;
}

int aif_destroy(aif_ctx *ctx)
{
    if (!ctx) return AIF_ERR_ARG;
    DeviceGuard g(ctx->device);
    cudaDeviceSynchronize();
    for (auto &hs : ctx->slots)
        if (hs.ev) cudaEventDestroy(hs.ev);
    if (ctx->table_ev) cudaEventDestroy(ctx->table_ev);
    for (int i = 0; i <= KernelTiming::kMax; ++i)
        if (ctx->timing.ev[i]) cudaEventDestroy(ctx->timing.ev[i]);
    for (int i = 0; i < PinnedRing::kSlots; ++i) {
        if (ctx->ring.host[i]) cudaFreeHost(ctx->ring.host[i]);
        if (ctx->ring.ev[i]) cudaEventDestroy(ctx->ring.ev[i]);
    }
    if (ctx->sim_plan) sim_destroy(ctx);
    if (ctx->tc_plan) tc_destroy_context(ctx);
    if (ctx->nearline_plan) nearline_destroy(ctx);
    for (void *p : ctx->allocations) cudaFree(p);
    cudaGetLastError();
    delete ctx;
    return AIF_OK;
}

int aif_load_weights(aif_ctx *ctx, const aif_weights *w, aif_stream stream)
{
    if (!ctx || !w || w->struct_size != sizeof(aif_weights)) return AIF_ERR_ARG;
    const aif_config &c = ctx->cfg;
    for (int k = 0; k < c.n_hidden; ++k)
        if (!w->W[k] || !w->b[k]) return AIF_ERR_ARG;
    if (!w->w_out || !w->b_out) return AIF_ERR_ARG;
    DeviceGuard g(ctx->device);
    cudaStream_t st = as_stream(stream);
    const size_t el = ctx->el;
    int in_w = ctx->input_width;
    for (int k = 0; k < c.n_hidden; ++k) {
        AIF_CUDA(launch_transpose(w->W[k], ctx->Wt[k], c.hidden[k], in_w, el, st));
        AIF_CUDA(cudaMemcpyAsync(ctx->b[k], w->b[k], (size_t)c.hidden[k] * 4, cudaMemcpyDeviceToDevice, st));
        in_w = c.hidden[k];
    }
    AIF_CUDA(cudaMemcpyAsync(ctx->w_out, w->w_out, (size_t)in_w * el, cudaMemcpyDeviceToDevice, st));
    AIF_CUDA(cudaMemcpyAsync(ctx->b_out, w->b_out, 4, cudaMemcpyDeviceToDevice, st));
    ctx->user_weights = w->W_profile && w->W_seq && w->W_a && w->W_b && w->b_a && w->b_b;
    if (ctx->user_weights) {
        AIF_CUDA(launch_transpose(w->W_profile, ctx->Wprofile_t, c.d, c.dU, el, st));
        AIF_CUDA(launch_transpose(w->W_seq, ctx->Wseq_t, c.d, c.dU, el, st));
        AIF_CUDA(launch_transpose(w->W_a, ctx->Wa_t, c.d, c.d, el, st));
        AIF_CUDA(cudaMemcpyAsync(ctx->Wseq_k, w->W_seq, (size_t)c.d * c.dU * el, cudaMemcpyDeviceToDevice, st));
        AIF_CUDA(cudaMemcpyAsync(ctx->Wa_k, w->W_a, (size_t)c.d * c.d * el, cudaMemcpyDeviceToDevice, st));
        AIF_CUDA(launch_transpose(w->W_b, ctx->Wb_t, c.d, c.d, el, st));
        AIF_CUDA(cudaMemcpyAsync(ctx->b_a, w->b_a, (size_t)c.d * 4, cudaMemcpyDeviceToDevice, st));
        AIF_CUDA(cudaMemcpyAsync(ctx->b_b, w->b_b, (size_t)c.d * 4, cudaMemcpyDeviceToDevice, st));
    }
    ctx->bea_user_weights = false;
    if ((c.blocks & AIF_BLK_BEA) && w->bridges && w->W_f) {
        if (!ctx->bridges) {
            int rc = dev_alloc(ctx, &ctx->bridges, (size_t)c.n_bridge * c.d * el, true);
            if (rc == AIF_OK) rc = dev_alloc(ctx, &ctx->W_f, (size_t)c.d * c.d * el, true);
            if (rc != AIF_OK) return rc;
        }
        AIF_CUDA(cudaMemcpyAsync(ctx->bridges, w->bridges, (size_t)c.n_bridge * c.d * el, cudaMemcpyDeviceToDevice, st));
        AIF_CUDA(cudaMemcpyAsync(ctx->W_f, w->W_f, (size_t)c.d * c.d * el, cudaMemcpyDeviceToDevice, st));
        ctx->bea_user_weights = true;
    }
    if (ctx->tensor_path) AIF_CUDA(tc_prepare_weights(ctx, w, st));
    if (ctx->tensor_path && ctx->tc_fused_plan) AIF_CUDA(tc_fused_prepare_weights(ctx, st));
    ctx->weights_loaded = true;
    ctx->model_version += 1;
    ctx->stats.model_version = ctx->model_version;
    return AIF_OK;
}

int aif_item_nearline_refresh(aif_ctx *ctx, const int32_t *ids, int64_t n, const void *rows, const void *bea_w,
                              const uint8_t *lsh_sig, aif_stream stream)
{
    StageRange range("aif_item_nearline_refresh");
    if (!ctx || !rows || n < 0) return AIF_ERR_ARG;
    if (ctx->bea_w && !bea_w) return AIF_ERR_ARG;
    if (ctx->sig && !lsh_sig) return AIF_ERR_ARG;
    if (!ids && n > ctx->cfg.M) return AIF_ERR_SHAPE;
    if (n == 0) return AIF_OK;
    DeviceGuard g(ctx->device);
    const bool versioned = ctx->cfg.versioned_table && !ids;
    if (versioned) AIF_CUDA(begin_full_refresh(ctx, n, as_stream(stream)));
    else AIF_CUDA(wait_table_ready(ctx, as_stream(stream)));
    AIF_CUDA(launch_scatter_rows(ctx, ids, n, rows, bea_w, lsh_sig, as_stream(stream)));
    AIF_CUDA(launch_row_norm_max(ctx, ctx->E, ids, n, ctx->cfg.M, ctx->e_norm, as_stream(stream)));
    if (versioned) AIF_CUDA(end_full_refresh(ctx, as_stream(stream)));
    ctx->table_version += 1;
    ctx->stats.table_version = ctx->table_version;
    ctx->stats.refresh_calls += 1;
    ctx->stats.rows_refreshed += (uint64_t)n;
    return AIF_OK;
}

int aif_load_item_weights(aif_ctx *ctx, const aif_item_weights *w, aif_stream stream)
{
    if (!ctx || !w || w->struct_size != sizeof(aif_item_weights)) return AIF_ERR_ARG;
    DeviceGuard g(ctx->device);
    return nearline_load_weights(ctx, w, as_stream(stream));
}

int aif_item_nearline_compute(aif_ctx *ctx, const int32_t *ids, int64_t n, const void *I_raw, const void *I_id, const void *M_mm,
                              aif_stream stream)
{
    StageRange range("aif_item_nearline_compute");
    if (!ctx || !I_raw || n < 0) return AIF_ERR_ARG;
    if (ctx->sig && !M_mm) return AIF_ERR_ARG;
    if (!ids && n > ctx->cfg.M) return AIF_ERR_SHAPE;
    if (!ctx->nearline_plan) return AIF_ERR_NOT_READY;
    if (n == 0) return AIF_OK;
    DeviceGuard g(ctx->device);
    const bool versioned = ctx->cfg.versioned_table && !ids;
    if (versioned) AIF_CUDA(begin_full_refresh(ctx, n, as_stream(stream)));
    else AIF_CUDA(wait_table_ready(ctx, as_stream(stream)));
    const int rc = nearline_compute(ctx, ids, n, I_raw, I_id, M_mm, as_stream(stream));
    if (rc != AIF_OK) return rc;
    if (versioned) AIF_CUDA(end_full_refresh(ctx, as_stream(stream)));
    ctx->table_version += 1;
    ctx->stats.table_version = ctx->table_version;
    ctx->stats.refresh_calls += 1;
    ctx->stats.rows_refreshed += (uint64_t)n;
    return AIF_OK;
}

int aif_user_precompute(aif_ctx *ctx, uint64_t request_key, const aif_user_inputs *in, int32_t L, aif_user_state **out,
                        aif_stream side_stream)
{
    StageRange range("aif_user_precompute");
    if (!ctx || !in || !out || in->struct_size != sizeof(aif_user_inputs)) return AIF_ERR_ARG;
    *out = nullptr;
    const aif_config &c = ctx->cfg;
    if (!ctx->weights_loaded) return AIF_ERR_NOT_READY;
    if (in->mode != AIF_USER_RAW && in->mode != AIF_USER_PROJECTED) return AIF_ERR_ARG;
    if (in->mode == AIF_USER_RAW && !ctx->user_weights) return AIF_ERR_NOT_READY;
    if (L < 1 || L > c.L_max) return AIF_ERR_SHAPE;
    if (!in->profile || !in->seq) return AIF_ERR_ARG;
    if ((c.blocks & AIF_BLK_CROSS) && !in->cross_raw) return AIF_ERR_ARG;
    if ((c.blocks & AIF_BLK_BEA) && !in->bea_V) {
        if (!in->bea_U) return AIF_ERR_ARG;
        if (in->bea_m < 1 || in->bea_m > 1024) return AIF_ERR_SHAPE;
        if (!ctx->bea_user_weights) return AIF_ERR_NOT_READY;
    }
    if ((c.blocks & (AIF_BLK_LSH_DIN | AIF_BLK_SIMTIER)) && !in->seq_sig) return AIF_ERR_ARG;
    if (c.n_categories > 0 && !in->seq_cat) return AIF_ERR_ARG;
    int idx = -1;
    for (int i = 0; i < (int)ctx->slots.size(); ++i)
        if (!ctx->slots[(size_t)i].in_use) {
            idx = i;
            break;
        }
    if (idx < 0) return AIF_ERR_OOM;
    DeviceGuard g(ctx->device);
    HostSlot &hs = ctx->slots[(size_t)idx];
    cudaStream_t st = as_stream(side_stream);
    AIF_CUDA(launch_user_network(ctx, hs, idx, in, L, st));
    if (c.n_categories > 0) AIF_CUDA(sim_group_sequence(ctx, hs, in->seq_cat, L, st));
    AIF_CUDA(cudaEventRecord(hs.ev, st));
    hs.ev_seen_done = false;
    hs.in_use = true, hs.ready = true, hs.L = L, hs.key = request_key, hs.model_version = ctx->model_version;
    hs.dev.L = L;
    ctx->stats.precompute_calls += 1;
    ctx->stats.user_states_in_use += 1;
    if (ctx->stats.user_states_in_use > ctx->stats.user_states_high_water)
        ctx->stats.user_states_high_water = ctx->stats.user_states_in_use;
    *out = &ctx->handles[(size_t)idx];
    return AIF_OK;
}

int aif_user_release(aif_ctx *ctx, aif_user_state *state)
{
    if (!ctx || !state || state->ctx != ctx || state->index < 0 || state->index >= (int)ctx->slots.size()) return AIF_ERR_ARG;
    HostSlot &hs = ctx->slots[(size_t)state->index];
    if (!hs.in_use) return AIF_ERR_ARG;
    hs.in_use = false, hs.ready = false;
    ctx->stats.user_states_in_use -= 1;
    return AIF_OK;
}

uint64_t aif_user_request_key(const aif_user_state *state)
{
    if (!state || !state->ctx) return 0;
    return state->ctx->slots[(size_t)state->index].key;
}

int aif_user_state_export(aif_ctx *ctx, const aif_user_state *state, float *u_out, void *S_out, float *pu_out,
                          aif_stream stream)
{
    int rc = state_check(ctx, state);
    if (rc != AIF_OK) return rc;
    DeviceGuard g(ctx->device);
    const HostSlot &hs = ctx->slots[(size_t)state->index];
    cudaStream_t st = as_stream(stream);
    AIF_CUDA(cudaStreamWaitEvent(st, hs.ev, 0));
    const aif_config &c = ctx->cfg;
    if (u_out) AIF_CUDA(cudaMemcpyAsync(u_out, hs.dev.u32, (size_t)c.d * 4, cudaMemcpyDeviceToDevice, st));
    if (S_out) AIF_CUDA(cudaMemcpyAsync(S_out, hs.dev.S, (size_t)hs.L * c.d * ctx->el, cudaMemcpyDeviceToDevice, st));
    if (pu_out) AIF_CUDA(cudaMemcpyAsync(pu_out, hs.dev.p_u, (size_t)c.hidden[0] * 4, cudaMemcpyDeviceToDevice, st));
    return AIF_OK;
}

// Orders `st` behind the user-side call that filled the slot.  Once that call is known to have finished, no wait is
// enqueued any more: a wait between two scoring calls of a stream costs device time and keeps the second call's
// set-up from overlapping the first call's tail.
static cudaError_t wait_user_ready(const HostSlot &hs, cudaStream_t st)
{
    if (hs.ev_seen_done) return cudaSuccess;
    const cudaError_t q = cudaEventQuery(hs.ev);
    if (q == cudaSuccess) {
        hs.ev_seen_done = true;
        return cudaSuccess;
    }
    if (q != cudaErrorNotReady) return q;
    (void)cudaGetLastError();   // "not ready" is an answer, not a failure: keep it out of later launch checks
    return cudaStreamWaitEvent(st, hs.ev, 0);
}

int aif_user_state_export_bea(aif_ctx *ctx, const aif_user_state *state, void *V_out, aif_stream stream)
{
    int rc = state_check(ctx, state);
    if (rc != AIF_OK) return rc;
    if (!(ctx->cfg.blocks & AIF_BLK_BEA) || !V_out) return AIF_ERR_ARG;
    DeviceGuard g(ctx->device);
    const HostSlot &hs = ctx->slots[(size_t)state->index];
    cudaStream_t st = as_stream(stream);
    AIF_CUDA(cudaStreamWaitEvent(st, hs.ev, 0));
    AIF_CUDA(cudaMemcpyAsync(V_out, hs.dev.V, (size_t)ctx->cfg.n_bridge * ctx->cfg.d * ctx->el, cudaMemcpyDeviceToDevice, st));
    return AIF_OK;
}

int aif_score(aif_ctx *ctx, const aif_user_state *state, const int32_t *cand_ids, int32_t n, float *logits, aif_stream stream)
{
    StageRange range("aif_score");
    int rc = state_check(ctx, state);
    if (rc != AIF_OK) return rc;
    if (n < 0) return AIF_ERR_SHAPE;
    if (n == 0) return AIF_OK;
    if (!cand_ids || !logits) return AIF_ERR_ARG;
    if ((int64_t)n > ctx->cfg.max_batch_candidates) return AIF_ERR_SHAPE;
    DeviceGuard g(ctx->device);
    cudaStream_t st = as_stream(stream);
    const HostSlot &hs = ctx->slots[(size_t)state->index];
    AIF_CUDA(wait_user_ready(hs, st));
    AIF_CUDA(wait_table_ready(ctx, st));
    ScoreLaunch sl{};
    sl.slots = ctx->slots_dev, sl.reqs = nullptr, sl.n_req = 1;
    sl.single = ReqDev{state->index, n, 0, 0, 0};
    sl.n_tiles = tiles_for(ctx, n);
    sl.total = n, sl.max_L = hs.L;
    sl.ids = cand_ids, sl.logits = logits, sl.status = ctx->status;
    return run_score(ctx, sl, n, st);
}

int aif_score_batch(aif_ctx *ctx, int32_t n_req, const aif_user_state *const *states, const int32_t *cand_ids,
                    const int64_t *offsets, float *logits, aif_stream stream)
{
    StageRange range("aif_score_batch");
    if (!ctx || !states || !offsets || n_req < 0) return AIF_ERR_ARG;
    if (n_req == 0) return AIF_OK;
    if (n_req > ctx->ring.capacity) return AIF_ERR_SHAPE;
    if (offsets[0] != 0) return AIF_ERR_ARG;
    for (int r = 0; r < n_req; ++r) {
        int rc = state_check(ctx, states[r]);
        if (rc != AIF_OK) return rc;
        const int64_t n = offsets[r + 1] - offsets[r];
        if (n < 0 || n > 0x7fffffff) return AIF_ERR_SHAPE;
    }
    const int64_t total = offsets[n_req];
    if (total > ctx->cfg.max_batch_candidates) return AIF_ERR_SHAPE;
    if (total == 0) return AIF_OK;
    if (!cand_ids || !logits) return AIF_ERR_ARG;
    DeviceGuard g(ctx->device);
    cudaStream_t st = as_stream(stream);
    PinnedRing &ring = ctx->ring;
    const int slot = ring.next;
    ring.next = (ring.next + 1) % PinnedRing::kSlots;
    if (ring.used[slot]) AIF_CUDA(cudaEventSynchronize(ring.ev[slot]));
    AIF_CUDA(wait_table_ready(ctx, st));
    int tiles = 0, max_L = 0;
    for (int r = 0; r < n_req; ++r) {
        const int n = (int)(offsets[r + 1] - offsets[r]);
        if (ctx->slots[(size_t)states[r]->index].L > max_L) max_L = ctx->slots[(size_t)states[r]->index].L;
        ring.host[slot][r] = ReqDev{states[r]->index, n, offsets[r], tiles, 0};
        tiles += tiles_for(ctx, n);
        AIF_CUDA(wait_user_ready(ctx->slots[(size_t)states[r]->index], st));
    }
    if (ctx->tensor_path && ctx->cfg.n_categories == 0 && (size_t)tiles > tc_tile_capacity(ctx)) {
        snprintf(g_last_error, sizeof(g_last_error), "aif_score_batch: %d tiles exceed the tile table's %zu entries", tiles,
                 tc_tile_capacity(ctx));
        return AIF_ERR_SHAPE;
    }
    AIF_CUDA(cudaMemcpyAsync(ring.dev[slot], ring.host[slot], sizeof(ReqDev) * (size_t)n_req, cudaMemcpyHostToDevice, st));
    ScoreLaunch sl{};
    sl.slots = ctx->slots_dev, sl.reqs = ring.dev[slot], sl.n_req = n_req, sl.n_tiles = tiles, sl.total = total, sl.max_L = max_L;
    sl.ids = cand_ids, sl.logits = logits, sl.status = ctx->status;
    int rc = run_score(ctx, sl, total, st);
    if (rc != AIF_OK) return rc;
    AIF_CUDA(cudaEventRecord(ring.ev[slot], st));
    ring.used[slot] = true;
    return AIF_OK;
}

int aif_score_host(aif_ctx *ctx, const aif_user_state *state, const int32_t *host_ids, int32_t n, float *host_logits,
                   aif_stream stream)
{
    StageRange range("aif_score_host");
    int rc = state_check(ctx, state);
    if (rc != AIF_OK) return rc;
    if (n < 0 || (int64_t)n > ctx->cfg.max_batch_candidates) return AIF_ERR_SHAPE;
    if (n == 0) return AIF_OK;
    if (!host_ids || !host_logits) return AIF_ERR_ARG;
    DeviceGuard g(ctx->device);
    cudaStream_t st = as_stream(stream);
    // Page-locked buffers that are mapped into the device's address space need no copy engine: a small kernel pulls
    // the ids over, and the last scoring kernel writes the logits straight into the host buffer.
    auto mapped = [](const void *hp) -> void * {
        cudaPointerAttributes a{};
        if (cudaPointerGetAttributes(&a, hp) != cudaSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        return a.type == cudaMemoryTypeHost ? a.devicePointer : nullptr;
    };
    void *d_ids = mapped(host_ids), *d_out = mapped(host_logits);
    if (d_ids && d_out) {
        AIF_CUDA(launch_stage_ids(static_cast<const int32_t *>(d_ids), ctx->ids_stage, n, st));
        rc = aif_score(ctx, state, ctx->ids_stage, n, static_cast<float *>(d_out), stream);
        if (rc != AIF_OK) return rc;
    } else {
        AIF_CUDA(cudaMemcpyAsync(ctx->ids_stage, host_ids, (size_t)n * 4, cudaMemcpyHostToDevice, st));
        rc = aif_score(ctx, state, ctx->ids_stage, n, ctx->logits_stage, stream);
        if (rc != AIF_OK) return rc;
        AIF_CUDA(cudaMemcpyAsync(host_logits, ctx->logits_stage, (size_t)n * 4, cudaMemcpyDeviceToHost, st));
    }
    AIF_CUDA(cudaStreamSynchronize(st));
    return AIF_OK;
}

int aif_score_batch_host(aif_ctx *ctx, int32_t n_req, const aif_user_state *const *states, const int32_t *host_ids,
                         const int64_t *offsets, float *host_logits, aif_stream stream)
{
    StageRange range("aif_score_batch_host");
    if (!ctx || !states || !offsets || n_req < 0) return AIF_ERR_ARG;
    if (n_req == 0) return AIF_OK;
    const int64_t total = offsets[n_req];
    if (total < 0 || total > ctx->cfg.max_batch_candidates) return AIF_ERR_SHAPE;
    if (total == 0) return AIF_OK;
    if (!host_ids || !host_logits) return AIF_ERR_ARG;
    DeviceGuard g(ctx->device);
    cudaStream_t st = as_stream(stream);
    AIF_CUDA(cudaMemcpyAsync(ctx->ids_stage, host_ids, (size_t)total * 4, cudaMemcpyHostToDevice, st));
    const int rc = aif_score_batch(ctx, n_req, states, ctx->ids_stage, offsets, ctx->logits_stage, stream);
    if (rc != AIF_OK) return rc;
    AIF_CUDA(cudaMemcpyAsync(host_logits, ctx->logits_stage, (size_t)total * 4, cudaMemcpyDeviceToHost, st));
    AIF_CUDA(cudaStreamSynchronize(st));
    return AIF_OK;
}

int aif_gather_rows(aif_ctx *ctx, const int32_t *ids, int64_t n, void *rows_out, aif_stream stream)
{
    if (!ctx || n < 0) return AIF_ERR_ARG;
    if (n == 0) return AIF_OK;
    if (!ids || !rows_out) return AIF_ERR_ARG;
    DeviceGuard g(ctx->device);
    AIF_CUDA(wait_table_ready(ctx, as_stream(stream)));
    AIF_CUDA(launch_gather_rows(ctx, ids, n, rows_out, as_stream(stream)));
    return AIF_OK;
}

int aif_gather_sidecars(aif_ctx *ctx, const int32_t *ids, int64_t n, void *bea_w_out, uint8_t *sig_out, aif_stream stream)
{
    if (!ctx || n < 0) return AIF_ERR_ARG;
    if ((bea_w_out && !ctx->bea_w) || (sig_out && !ctx->sig)) return AIF_ERR_ARG;
    if (bea_w_out && ((size_t)ctx->cfg.n_bridge * ctx->el) % 4 != 0) return AIF_ERR_SHAPE;
    if (sig_out && ctx->cfg.lsh_bits % 32 != 0) return AIF_ERR_SHAPE;
    if (n == 0 || (!bea_w_out && !sig_out)) return AIF_OK;
    if (!ids) return AIF_ERR_ARG;
    DeviceGuard g(ctx->device);
    AIF_CUDA(wait_table_ready(ctx, as_stream(stream)));
    AIF_CUDA(launch_gather_sidecars(ctx, ids, n, bea_w_out, sig_out, as_stream(stream)));
    return AIF_OK;
}

int aif_poll_status(aif_ctx *ctx, uint32_t *bits)
{
    if (!ctx || !bits) return AIF_ERR_ARG;
    DeviceGuard g(ctx->device);
    AIF_CUDA(cudaDeviceSynchronize());
    AIF_CUDA(cudaMemcpy(bits, ctx->status, 4, cudaMemcpyDeviceToHost));
    AIF_CUDA(cudaMemset(ctx->status, 0, 4));
    if (*bits & AIF_STATUS_BAD_ID) ctx->stats.bad_id_events += 1;
    if (*bits & AIF_STATUS_TIMEOUT) ctx->stats.timeout_events += 1;
    return AIF_OK;
}

int aif_get_stats(aif_ctx *ctx, aif_stats *out)
{
    if (!ctx || !out) return AIF_ERR_ARG;
    ctx->stats.device_bytes = ctx->device_bytes;
    ctx->stats.tensor_path = ctx->tensor_path ? 1 : 0;
    *out = ctx->stats;
    return AIF_OK;
}

int aif_set_kernel_timing(aif_ctx *ctx, int on)
{
    if (!ctx) return AIF_ERR_ARG;
    DeviceGuard g(ctx->device);
    KernelTiming &t = ctx->timing;
    if (on && !t.ev[0])
        for (int i = 0; i <= KernelTiming::kMax; ++i) AIF_CUDA(cudaEventCreate(&t.ev[i]));
    t.on = on != 0;
    t.n = 0;
    return AIF_OK;
}

int aif_get_kernel_timing(aif_ctx *ctx, int32_t *n, const char **names, float *ms)
{
    if (!ctx || !n || !names || !ms) return AIF_ERR_ARG;
    DeviceGuard g(ctx->device);
    KernelTiming &t = ctx->timing;
    *n = 0;
    if (!t.on || t.n == 0) return AIF_OK;
    AIF_CUDA(cudaEventSynchronize(t.ev[t.n]));
    for (int i = 0; i < t.n; ++i) {
        AIF_CUDA(cudaEventElapsedTime(&ms[i], t.ev[i], t.ev[i + 1]));
        names[i] = t.names[i];
    }
    *n = t.n;
    return AIF_OK;
}

uint64_t aif_kernel_launches(void) { return g_launches.load(); }

int aif_selftest_bounded_wait(aif_ctx *ctx, int64_t limit_cycles, aif_stream stream)
{
    if (!ctx || limit_cycles < 1 || limit_cycles > 2000000000ll) return AIF_ERR_ARG;
    DeviceGuard g(ctx->device);
    AIF_CUDA(launch_wait_selftest(ctx, (long long)limit_cycles, as_stream(stream)));
    return AIF_OK;
}

const char *aif_strerror(int code)
{
    switch (code) {
        case AIF_OK: return "ok";
        case AIF_ERR_ARG: return "bad argument";
        case AIF_ERR_SHAPE: return "unsupported shape or size";
        case AIF_ERR_OOM: return "out of device memory or user-state slots";
        case AIF_ERR_CUDA: return "CUDA runtime error";
        case AIF_ERR_VERSION: return "user state computed under other weights";
        case AIF_ERR_NOT_READY: return "weights or user state not ready";
        case AIF_ERR_BAD_ID: return "id outside the item table";
        case AIF_ERR_TIMEOUT: return "bounded device wait ran out";
        default: return "unknown error";
    }
}

const char *aif_last_error(void) { return g_last_error; }

}  // extern "C"
