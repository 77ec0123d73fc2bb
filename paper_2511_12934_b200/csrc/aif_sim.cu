// Category sub-sequences (Section 3.3, SIM-hard): the long-term sequence is kept as <user, category, sub-sequence>, and a
// candidate interacts only with the sub-sequence of its own category.
//
// User side (in parallel with retrieval): the projected sequence and its +-1 signatures are laid out a second time,
// grouped by category, every sub-sequence starting on a multiple of 128 rows and padded with zero rows to the next one.
// This is the pre-cache of parsed sub-sequences for all of the user's categories.
//
// Real time: the candidates of a launch are grouped by (request, category); every group becomes tiles of up to 128
// candidates that carry their sub-sequence's key range, and the tensor-core kernels walk those tiles.  The number of
// tiles depends on the data, so it is left in device memory for the kernels to read; logits go back to the caller's
// order through an index.
#include "aif_device.cuh"
#include "aif_internal.h"

namespace aif {
namespace {

constexpr int kCatBlock = 1024;   // sequence items per block of the grouping passes

__device__ __forceinline__ int category_of(int id, int n_cat, int mode)
{
    if (mode == AIF_BUCKET_MOD) return id % n_cat;
    return (int)(mix64((uint64_t)id, (uint64_t)AIF_CATEGORY_FIELD) % (uint64_t)n_cat);
}

// ---- user side ------------------------------------------------------------------------------------------------
// hist[b][c] = items of category c among the block's 1024 sequence items
__global__ void __launch_bounds__(kCatBlock) k_cat_hist(const int32_t *__restrict__ cat, int L, int n_cat, int32_t *__restrict__ hist,
                                                        uint32_t *status)
{
    extern __shared__ int h_s[];
    for (int c = threadIdx.x; c < n_cat; c += kCatBlock) h_s[c] = 0;
    __syncthreads();
    const int j = blockIdx.x * kCatBlock + threadIdx.x;
    if (j < L) {
        const int c = cat[j];
        if (c >= 0 && c < n_cat) atomicAdd(&h_s[c], 1);
        else atomicOr(status, AIF_STATUS_BAD_ID);
    }
    __syncthreads();
    for (int c = threadIdx.x; c < n_cat; c += kCatBlock) hist[(size_t)blockIdx.x * n_cat + c] = h_s[c];
}

// One block: hist[b][c] becomes the number of items of category c in earlier blocks; cat_len[c] the total; cat_off[c]
// the first row of the sub-sequence, sub-sequences following each other on multiples of 128 rows.
__global__ void __launch_bounds__(kCatBlock) k_cat_scan(int n_blocks, int n_cat, int32_t *__restrict__ hist, int32_t *__restrict__ cat_off,
                                                        int32_t *__restrict__ cat_len)
{
    __shared__ int32_t carry;
    __shared__ int32_t part[kCatBlock];
    for (int c = threadIdx.x; c < n_cat; c += kCatBlock) {
        int run = 0;
        for (int b = 0; b < n_blocks; ++b) {
            const int v = hist[(size_t)b * n_cat + c];
            hist[(size_t)b * n_cat + c] = run;
            run += v;
        }
        cat_len[c] = run;
    }
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    // exclusive scan of the padded lengths, 1024 categories at a time
    for (int c0 = 0; c0 < n_cat; c0 += kCatBlock) {
        const int c = c0 + threadIdx.x;
        const int v = c < n_cat ? (cat_len[c] + 127) / 128 * 128 : 0;
        part[threadIdx.x] = v;
        __syncthreads();
        for (int o = 1; o < kCatBlock; o <<= 1) {
            const int add = (int)threadIdx.x >= o ? part[threadIdx.x - o] : 0;
            __syncthreads();
            part[threadIdx.x] += add;
            __syncthreads();
        }
        if (c < n_cat) cat_off[c] = carry + part[threadIdx.x] - v;
        __syncthreads();
        if (threadIdx.x == kCatBlock - 1) carry += part[kCatBlock - 1];
        __syncthreads();
    }
}

// map[j] = row of sequence item j in the grouped sequence: its sub-sequence's first row + items of its category in
// earlier blocks + items of its category before it in this block (counted, not raced for: the order inside a
// sub-sequence is the order of the sequence, the same in every run).  -1 for a category outside the range.
__global__ void __launch_bounds__(kCatBlock) k_cat_place(const int32_t *__restrict__ cat, int L, int n_cat, const int32_t *__restrict__ hist,
                                                         const int32_t *__restrict__ cat_off, int32_t *__restrict__ map)
{
    __shared__ int32_t c_s[kCatBlock];
    const int j = blockIdx.x * kCatBlock + threadIdx.x;
    const int c = j < L ? cat[j] : -1;
    c_s[threadIdx.x] = c;
    __syncthreads();
    if (j >= L) return;
    if (c < 0 || c >= n_cat) {
        map[j] = -1;
        return;
    }
    int rank = 0;
    for (int i = 0; i < (int)threadIdx.x; ++i) rank += c_s[i] == c;
    map[j] = cat_off[c] + hist[(size_t)blockIdx.x * n_cat + c] + rank;
}

// dst[map[j]] = src[j], rows of row_bytes (a multiple of 16)
__global__ void __launch_bounds__(256) k_group_rows(const uint4 *__restrict__ src, const int32_t *__restrict__ map, int L, int vec_per_row,
                                                    uint4 *__restrict__ dst)
{
    const int64_t total = (int64_t)L * vec_per_row;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int j = (int)(i / vec_per_row), v = (int)(i - (int64_t)j * vec_per_row);
        const int r = map[j];
        if (r >= 0) dst[(int64_t)r * vec_per_row + v] = src[i];
    }
}

// ---- real time ------------------------------------------------------------------------------------------------
__device__ __forceinline__ int request_of(const ScoreLaunch &sl, int64_t pos, ReqDev &rq)
{
    if (sl.reqs == nullptr) {
        rq = sl.single;
        return 0;
    }
    int lo = 0, hi = sl.n_req - 1;
    while (lo < hi) {   // last request that begins at or before pos (empty requests share their successor's start)
        const int mid = (lo + hi + 1) >> 1;
        if (sl.reqs[mid].off <= pos) lo = mid;
        else hi = mid - 1;
    }
    rq = sl.reqs[lo];
    return lo;
}

// group of a candidate: request index * n_cat + category (category 0 for an id outside the table: its logit is NaN anyway)
__device__ __forceinline__ int group_of(const ScoreLaunch &sl, int64_t pos, int64_t M, int n_cat, int mode, int &id_out)
{
    ReqDev rq;
    const int r = request_of(sl, pos, rq);
    const int id = sl.ids[pos];
    id_out = id;
    const int c = (id >= 0 && (int64_t)id < M) ? category_of(id, n_cat, mode) : 0;
    return r * n_cat + c;
}

__global__ void __launch_bounds__(256) k_sim_count(ScoreLaunch sl, int64_t M, int n_cat, int mode, int32_t *__restrict__ grp_cnt)
{
    for (int64_t pos = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; pos < sl.total; pos += (int64_t)gridDim.x * blockDim.x) {
        int id;
        atomicAdd(&grp_cnt[group_of(sl, pos, M, n_cat, mode, id)], 1);
    }
}

// One block over the groups: first grouped position of every group (exclusive scan of the counts), the tile records, the
// number of tiles; the counts are turned into cursors (zero) for the placement.  Tiles are laid out by the size of their
// sub-sequence, longest first (in classes of powers of two): a tile's cost is its number of key blocks, the kernels hand
// tile t to CTA t mod grid, and a long tile that started late would be what everything else waits for.
__global__ void __launch_bounds__(1024) k_sim_tiles(ScoreLaunch sl, int n_groups, int n_cat, int32_t *__restrict__ grp_cnt,
                                                    int32_t *__restrict__ grp_start, TileDev *__restrict__ tiles, int tile_cap,
                                                    int32_t *__restrict__ n_tiles_out)
{
    constexpr int kClasses = 32;
    __shared__ int32_t part_c[1024];
    __shared__ int32_t carry_c;
    __shared__ int32_t cls_tiles[kClasses], cls_base[kClasses];
    if (threadIdx.x == 0) carry_c = 0;
    if (threadIdx.x < kClasses) cls_tiles[threadIdx.x] = 0;
    __syncthreads();
    auto group_info = [&](int g, int &slot, int &len, int &key0) {
        const int r = g / n_cat, c = g - r * n_cat;
        slot = sl.reqs ? sl.reqs[r].slot : sl.single.slot;
        const SlotDev *sd = sl.slots + slot;
        len = sd->cat_len[c], key0 = sd->cat_off[c];
    };
    auto class_of = [](int len) { return len > 0 ? 32 - __clz(len) : 0; };   // 0: empty sub-sequence, else floor(log2) + 1
    // pass 1: grouped positions (scan of the counts) and tiles per size class
    for (int g0 = 0; g0 < n_groups; g0 += 1024) {
        const int g = g0 + threadIdx.x;
        const int cnt = g < n_groups ? grp_cnt[g] : 0;
        part_c[threadIdx.x] = cnt;
        __syncthreads();
        for (int o = 1; o < 1024; o <<= 1) {
            const int ac = (int)threadIdx.x >= o ? part_c[threadIdx.x - o] : 0;
            __syncthreads();
            part_c[threadIdx.x] += ac;
            __syncthreads();
        }
        if (g < n_groups) {
            grp_start[g] = carry_c + part_c[threadIdx.x] - cnt;
            if (cnt > 0) {
                int slot, len, key0;
                group_info(g, slot, len, key0);
                atomicAdd(&cls_tiles[class_of(len)], (cnt + kTcTile - 1) / kTcTile);
            }
        }
        __syncthreads();
        if (threadIdx.x == 1023) carry_c += part_c[1023];
        __syncthreads();
    }
    // first tile of every class, longest sub-sequences first
    if (threadIdx.x == 0) {
        int run = 0;
        for (int k = kClasses - 1; k >= 0; --k) {
            cls_base[k] = run;
            run += cls_tiles[k];
            cls_tiles[k] = 0;   // from here on the class's cursor
        }
        *n_tiles_out = min(run, tile_cap);
    }
    __syncthreads();
    // pass 2: the tile records; the counts become the placement cursors
    for (int g = threadIdx.x; g < n_groups; g += 1024) {
        const int cnt = grp_cnt[g];
        grp_cnt[g] = 0;
        if (cnt == 0) continue;
        int slot, len, key0;
        group_info(g, slot, len, key0);
        const int nt = (cnt + kTcTile - 1) / kTcTile, k = class_of(len);
        const int t0 = cls_base[k] + atomicAdd(&cls_tiles[k], nt);
        const int start = grp_start[g];
        for (int i = 0; i < nt; ++i) {
            if (t0 + i >= tile_cap) break;   // cannot happen for a launch within the context's limits (sim_prepare)
            TileDev t;
            t.slot = slot, t.cnt = min(kTcTile, cnt - i * kTcTile), t.pos0 = (int64_t)start + (int64_t)i * kTcTile;
            t.L = len, t.key0 = key0, t.pad_[0] = t.pad_[1] = 0;
            tiles[t0 + i] = t;
        }
    }
}

// grouped ids and, for every grouped position, where its logit belongs
__global__ void __launch_bounds__(256) k_sim_place(ScoreLaunch sl, int64_t M, int n_cat, int mode, const int32_t *__restrict__ grp_start,
                                                   int32_t *__restrict__ cursor, int32_t *__restrict__ ids_out, int32_t *__restrict__ out_index)
{
    for (int64_t pos = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; pos < sl.total; pos += (int64_t)gridDim.x * blockDim.x) {
        int id;
        const int g = group_of(sl, pos, M, n_cat, mode, id);
        const int p = grp_start[g] + atomicAdd(&cursor[g], 1);
        ids_out[p] = id;
        out_index[p] = (int32_t)pos;
    }
}

struct SimPlan {
    int n_groups_max = 0;
    size_t tile_cap = 0, cap = 0;
    int32_t *grp_cnt = nullptr, *grp_start = nullptr, *ids_sorted = nullptr, *out_index = nullptr, *n_tiles_dev = nullptr;
    TileDev *tiles = nullptr;
};

SimPlan *plan_of(const aif_ctx *ctx) { return reinterpret_cast<SimPlan *>(ctx->sim_plan); }

}  // namespace

// rows of a slot's grouped sequence: every sub-sequence rounded up to 128 rows
size_t sim_grouped_rows(int L_max, int n_categories) { return ((size_t)L_max + 127) / 128 * 128 + (size_t)n_categories * 128; }

cudaError_t sim_prepare(aif_ctx *ctx)
{
    const aif_config &c = ctx->cfg;
    SimPlan *pl = new SimPlan();
    ctx->sim_plan = pl;
    pl->n_groups_max = c.max_user_states * c.n_categories;
    pl->cap = (size_t)c.max_batch_candidates;
    // a group of n candidates is ceil(n / 128) tiles: at most candidates / 128 tiles plus one per non-empty group
    const size_t groups = (size_t)pl->n_groups_max < pl->cap ? (size_t)pl->n_groups_max : pl->cap;
    pl->tile_cap = pl->cap / kTcTile + groups + 1;
    auto alloc = [&](void **p, size_t bytes) -> cudaError_t {
        bytes = (bytes + 255) / 256 * 256;
        cudaError_t e = cudaMalloc(p, bytes);
        if (e != cudaSuccess) return e;
        ctx->allocations.push_back(*p);
        ctx->device_bytes += (int64_t)bytes;
        return cudaMemset(*p, 0, bytes);
    };
    cudaError_t e;
    if ((e = alloc((void **)&pl->grp_cnt, (size_t)pl->n_groups_max * 4)) != cudaSuccess) return e;
    if ((e = alloc((void **)&pl->grp_start, (size_t)pl->n_groups_max * 4)) != cudaSuccess) return e;
    if ((e = alloc((void **)&pl->ids_sorted, (pl->cap + kTcTile) * 4)) != cudaSuccess) return e;
    if ((e = alloc((void **)&pl->out_index, (pl->cap + kTcTile) * 4)) != cudaSuccess) return e;
    if ((e = alloc((void **)&pl->n_tiles_dev, 256)) != cudaSuccess) return e;
    if ((e = alloc((void **)&pl->tiles, pl->tile_cap * sizeof(TileDev))) != cudaSuccess) return e;
    return cudaSuccess;
}

void sim_destroy(aif_ctx *ctx)
{
    delete plan_of(ctx);
    ctx->sim_plan = nullptr;
}

size_t sim_tile_capacity(const aif_ctx *ctx) { return plan_of(ctx)->tile_cap; }

cudaError_t sim_group_sequence(const aif_ctx *ctx, HostSlot &hs, const int32_t *seq_cat, int L, cudaStream_t st)
{
    const aif_config &c = ctx->cfg;
    const int nb = (L + kCatBlock - 1) / kCatBlock;
    cudaError_t e;
    k_cat_hist<<<nb, kCatBlock, (size_t)c.n_categories * 4, st>>>(seq_cat, L, c.n_categories, hs.cat_hist, ctx->status);
    k_cat_scan<<<1, kCatBlock, 0, st>>>(nb, c.n_categories, hs.cat_hist, const_cast<int32_t *>(hs.dev.cat_off),
                                        const_cast<int32_t *>(hs.dev.cat_len));
    k_cat_place<<<nb, kCatBlock, 0, st>>>(seq_cat, L, c.n_categories, hs.cat_hist, hs.dev.cat_off, hs.cat_map);
    count_launch(3);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    // zero rows everywhere (the padding of every sub-sequence), then the items at their places
    const size_t row_bytes = (size_t)c.d * ctx->el;
    if ((e = cudaMemsetAsync(const_cast<void *>(hs.dev.Sg), 0, ctx->grouped_rows * row_bytes, st)) != cudaSuccess) return e;
    const int64_t vecs = (int64_t)L * (int64_t)(row_bytes / 16);
    k_group_rows<<<(int)((vecs + 255) / 256 < 1184 ? (vecs + 255) / 256 : 1184), 256, 0, st>>>(
        (const uint4 *)hs.dev.S, hs.cat_map, L, (int)(row_bytes / 16), (uint4 *)const_cast<void *>(hs.dev.Sg));
    count_launch();
    if (hs.dev.sigEg) {
        if ((e = cudaMemsetAsync(const_cast<uint8_t *>(hs.dev.sigEg), 0, ctx->grouped_rows * (size_t)c.lsh_bits, st)) != cudaSuccess) return e;
        const int64_t v2 = (int64_t)L * (c.lsh_bits / 16);
        k_group_rows<<<(int)((v2 + 255) / 256 < 1184 ? (v2 + 255) / 256 : 1184), 256, 0, st>>>(
            (const uint4 *)hs.dev.sigE, hs.cat_map, L, c.lsh_bits / 16, (uint4 *)const_cast<uint8_t *>(hs.dev.sigEg));
        count_launch();
    }
    return cudaGetLastError();
}

cudaError_t sim_group_candidates(const aif_ctx *ctx, ScoreLaunch &sl, cudaStream_t st)
{
    const aif_config &c = ctx->cfg;
    SimPlan *pl = plan_of(ctx);
    const int n_groups = sl.n_req * c.n_categories;
    cudaError_t e = cudaMemsetAsync(pl->grp_cnt, 0, (size_t)n_groups * 4, st);
    if (e != cudaSuccess) return e;
    const int grid = (int)((sl.total + 255) / 256 < 1184 ? (sl.total + 255) / 256 : 1184);
    k_sim_count<<<grid, 256, 0, st>>>(sl, c.M, c.n_categories, c.bucket_mode, pl->grp_cnt);
    k_sim_tiles<<<1, 1024, 0, st>>>(sl, n_groups, c.n_categories, pl->grp_cnt, pl->grp_start, pl->tiles, (int)pl->tile_cap, pl->n_tiles_dev);
    k_sim_place<<<grid, 256, 0, st>>>(sl, c.M, c.n_categories, c.bucket_mode, pl->grp_start, pl->grp_cnt, pl->ids_sorted, pl->out_index);
    count_launch(3);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    const int64_t groups = (int64_t)n_groups < sl.total ? (int64_t)n_groups : sl.total;
    sl.n_tiles = (int32_t)(sl.total / kTcTile + groups + 1 < (int64_t)pl->tile_cap ? sl.total / kTcTile + groups + 1 : (int64_t)pl->tile_cap);
    sl.ids = pl->ids_sorted;
    sl.tiles = pl->tiles;
    sl.n_tiles_dev = pl->n_tiles_dev;
    sl.out_index = pl->out_index;
    sl.grouped = 1;
    return cudaSuccess;
}

}  // namespace aif
