// aif_score_noalloc: the tensor-core scoring chain with its intermediate activations in a fixed device array that
// is part of the library image, for callers that must not allocate.
#include <cstdio>
#include <mutex>

#include "aif_internal.h"

using namespace aif;

namespace {

constexpr int kMaxCandidates = AIF_NOALLOC_MAX_CANDIDATES;
constexpr int kRowBytes = AIF_NOALLOC_ROW_BYTES;
constexpr size_t kRows = (size_t)kMaxCandidates + kTcTile;   // the kernels address whole 128-row tiles

// The scratch itself.  Every GPU that loads the library carries it until the process exits (4.5 MiB).
static __device__ __align__(256) unsigned char g_scratch[kRows * kRowBytes];

// In host code `g_scratch` only names the symbol; the address the kernels need comes from cudaGetSymbolAddress,
// asked once per device with that device current.
constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char *g_dev_ptr[kMaxDevices] = {};

int scratch_for_current_device(int device, unsigned char **out)
{
    if (device < 0 || device >= kMaxDevices) {
        set_last_error("aif_score_noalloc: device ordinal out of range");
        return AIF_ERR_ARG;
    }
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_dev_ptr[device]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_scratch);
        if (e != cudaSuccess || !p) {
            char msg[200];
            snprintf(msg, sizeof(msg), "aif_score_noalloc: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
            set_last_error(msg);
            cudaGetLastError();
            return AIF_ERR_CUDA;
        }
        g_dev_ptr[device] = static_cast<unsigned char *>(p);
    }
    *out = g_dev_ptr[device];
    return AIF_OK;
}

}  // namespace

extern "C" int aif_score_noalloc(aif_ctx *ctx, const aif_user_state *state, const int32_t *cand_ids, int32_t n, float *logits,
                                 aif_stream stream)
{
    int rc = check_user_state(ctx, state);
    if (rc != AIF_OK) return rc;
    if (n < 0) return AIF_ERR_SHAPE;
    if (n == 0) return AIF_OK;
    if (!cand_ids || !logits) return AIF_ERR_ARG;
    if (n > kMaxCandidates) {
        char msg[200];
        snprintf(msg, sizeof(msg), "aif_score_noalloc: n = %d exceeds AIF_NOALLOC_MAX_CANDIDATES = %d", n, kMaxCandidates);
        set_last_error(msg);
        return AIF_ERR_SHAPE;
    }
    if (!ctx->tensor_path) {
        set_last_error("aif_score_noalloc: this context runs the CUDA-core kernel, which has no scratch; use aif_score");
        return AIF_ERR_SHAPE;
    }
    if (ctx->cfg.n_categories > 0) {
        set_last_error("aif_score_noalloc: contexts with category sub-sequences group their candidates in allocated scratch; use aif_score");
        return AIF_ERR_SHAPE;
    }
    if (tc_scratch_row_bytes(ctx) > (size_t)kRowBytes) {
        char msg[200];
        snprintf(msg, sizeof(msg), "aif_score_noalloc: model needs %zu scratch bytes per candidate, limit is %d",
                 tc_scratch_row_bytes(ctx), kRowBytes);
        set_last_error(msg);
        return AIF_ERR_SHAPE;
    }
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return AIF_ERR_CUDA;
    if (prev != ctx->device && cudaSetDevice(ctx->device) != cudaSuccess) return AIF_ERR_CUDA;
    unsigned char *base = nullptr;
    rc = scratch_for_current_device(ctx->device, &base);
    if (rc == AIF_OK) {
        cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
        const HostSlot &hs = ctx->slots[(size_t)state->index];
        cudaError_t e = cudaStreamWaitEvent(st, hs.ev, 0);
        if (e == cudaSuccess) e = wait_table_ready(ctx, st);
        if (e == cudaSuccess) {
            TcScratch sc;
            tc_scratch_layout(ctx, base, kRows, &sc);
            ScoreLaunch sl{};
            sl.slots = ctx->slots_dev, sl.reqs = nullptr, sl.n_req = 1;
            sl.single = ReqDev{state->index, n, 0, 0, 0};
            sl.n_tiles = tc_tiles_for(ctx, n);
            sl.total = n, sl.max_L = hs.L;
            sl.ids = cand_ids, sl.logits = logits, sl.status = ctx->status;
            e = launch_score_tc_scratch(ctx, sl, st, sc);
        }
        if (e != cudaSuccess) {
            set_last_error(cudaGetErrorString(e));
            cudaGetLastError();
            rc = AIF_ERR_CUDA;
        } else {
            ctx->stats.score_calls += 1;
            ctx->stats.candidates_scored += (uint64_t)n;
        }
    }
    if (prev != ctx->device) cudaSetDevice(prev);
    return rc;
}
