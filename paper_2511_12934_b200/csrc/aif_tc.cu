// Tensor-core scoring path for sm_100a (bf16 storage): the scoring MLP as tcgen05 GEMMs with a fused gather
// prologue and fused epilogues.
//
// One layer = one persistent kernel (k_layer_tc<MODE>).  A work item is one or two 128-candidate tiles times one or two
// 256-wide slices of the layer's outputs (LayerCfg below).  Roles inside a CTA (one accumulator: 320 threads, two: 576):
//   epilogue   4 warps per accumulator: read the fp32 accumulator from TMEM (tcgen05.ld), add the bias (for the first
//              layer the request's cached user partial p_u), ReLU, then either store bf16 activations for the next
//              layer (through a staging slab and a TMA tile store), reduce against w_out and write the logit, or (item
//              side of the nearline pipeline) store without ReLU / pack the sign bits of the outputs
//   MMA        one warp allocates TMEM; one lane issues tcgen05.mma (M=128, N<=256, K=16, bf16 in, fp32 accumulate)
//   A producer 4 warps per tile: gather the tile's input rows chunk by chunk (64 columns = 128 bytes per row) with
//              16-byte cp.async into the 128B-swizzled K-major layout the MMA reads: item-table rows by candidate
//              id, cross-feature rows by (field, bucket) from the request's pre-cache with the bucket looked up in
//              the table k_cross_buckets wrote; dense rows (attention output, previous activations, raw item
//              features) come by position as one TMA tile per chunk.
//              Ids of the next item and the sources of the next chunk are fetched ahead of their use.
//   B producer one lane streams the weight slice with TMA (cp.async.bulk.tensor, 128B swizzle)
// Shared-memory rings (mbarriers) decouple producers from the MMA.  Two TMEM accumulators of 256 columns: with one
// accumulator per item they alternate so that the epilogue of one item overlaps the main loop of the next; with two,
// each tile (or output slice) of the item owns one.  Every wait is bounded: on expiry the CTA raises
// AIF_STATUS_TIMEOUT, all roles leave their loops, TMEM is freed and the kernel returns.
#include <cuda.h>

#include "aif_device.cuh"
#include "aif_internal.h"
#include "aif_tc_ptx.cuh"

namespace aif {
namespace {

constexpr int kABytes = kTcTile * 128;    // one A chunk of one tile: 128 rows x 64 bf16
constexpr int kBBytes = 256 * 128;        // one B chunk: up to 256 weight rows x 64 bf16
constexpr int kMaxChunks = 64;
constexpr int kFusedMaxTiles = 148;

enum { SRC_ITEM = 0, SRC_DENSE = 1, SRC_CROSS = 2 };
enum { EPI_STORE = 0, EPI_DOT = 1, EPI_SIGN = 2 };

struct ChunkSrc {
    int32_t kind;
    int32_t off;   // ITEM / DENSE: byte offset inside the source row; CROSS: first cross column of the chunk
};

struct LayerParams {
    ScoreLaunch sl;
    int32_t n_nchunks, n_cols, n_k, mini_batch;
    // A sources
    const uint8_t *E;
    int64_t M;
    int32_t e_row_bytes;
    int32_t x_row_bytes;
    const uint8_t *X;             // dense rows, indexed by candidate position in the launch
    const uint16_t *xb;           // cross-feature buckets [positions x F], written by k_cross_buckets
    int32_t F, B, dc;
    int32_t check_ids;            // first layer: flag ids outside the table
    // epilogue
    int32_t epi, bias_from_slot, emit_sigmoid, out_stride;
    int32_t linear_out;           // EPI_STORE without the ReLU (output layer of the item-side tower)
    uint8_t *sig_out;             // EPI_SIGN: [positions x out_stride / 8] packed sign bits of the outputs
    const float *bias;
    __nv_bfloat16 *out;           // EPI_STORE: [positions x out_stride]
    const __nv_bfloat16 *w_out;
    const float *b_out;
    ChunkSrc src[kMaxChunks];
};

// Geometry of the layer kernel.  A work item fills one or two 256-column TMEM accumulators:
//   MODE 0  one tile, one 256-wide output slice; the two accumulators alternate between consecutive items so that the
//           epilogue of one overlaps the main loop of the next (small launches, every item on its own SM)
//   MODE 1  two tiles, one slice: one weight chunk in shared memory feeds both tiles, which halves the weight traffic
//           per candidate (large launches)
//   MODE 2  one tile, two slices: one gathered A chunk feeds both slices, so the tile's rows are gathered once instead
//           of once per slice (launches that would otherwise need a second round of items)
//   MODE 3  as MODE 1 with a deeper A ring and a shallower B ring, for the first layer: its cross-feature rows come
//           from per-request tables that may live in HBM, the weights from L2
// A and B have rings of their own: gathered rows have the longer latency and the smaller chunks.
template <int MODE>
struct LayerCfg {
    static constexpr int G = (MODE == 1 || MODE == 3) ? 2 : 1;   // tiles per work item
    static constexpr int NB = MODE == 2 ? 2 : 1;         // output slices per work item
    static constexpr int kAcc = G * NB;                  // accumulators a work item fills
    static constexpr int kStagesA = MODE == 1 ? 3 : 4;
    static constexpr int kStagesB = MODE == 0 ? 4 : (MODE == 1 ? 3 : 2);
    static constexpr int kAStage = G * kABytes, kBStage = NB * kBBytes;
    static constexpr int kEpiWarps = 4 * kAcc;
    static constexpr int kMmaWarp = kEpiWarps;
    static constexpr int kProdWarp0 = kEpiWarps + 1;
    static constexpr int kProdThreads = 128 * G;    // 128 producer threads per tile of the group, 8 rows each
    static constexpr int kBWarp = kProdWarp0 + 4 * G;
    static constexpr int kThreads = (kBWarp + 1) * 32;
    static constexpr int kSlabs = MODE == 0 ? 2 : 1;    // output staging slabs (2 KB) per epilogue warp
    static_assert(1024 + kStagesA * kAStage + kStagesB * kBStage + kEpiWarps * kSlabs * 2048 + 8192 <= 227 * 1024, "shared memory");
    static constexpr size_t kSmem = 1024 + (size_t)kStagesA * kAStage + (size_t)kStagesB * kBStage + (2 * kStagesA + 2 * kStagesB + 4) * 8 +
                                    32 + 2 * kAcc * 256 * 4 + kEpiWarps * kSlabs * 2048 + 2 * G * 128 * 4;
};

struct TileInfo {
    ReqDev rq;
    int start, cnt;
    int64_t pos0;   // position of the tile's first candidate in the launch (ids / logits / dense rows)
};

__device__ __forceinline__ TileInfo decode_tile(const LayerParams &p, int tile, int n_tiles)
{
    TileInfo t;
    if (tile >= n_tiles) {   // the second tile of the last group may not exist
        t.rq = ReqDev{0, 0, 0, 0, 0};
        t.start = 0, t.cnt = 0, t.pos0 = 0;
        return t;
    }
    if (p.sl.tiles) {   // looked up once per launch
        const int4 v = *reinterpret_cast<const int4 *>(p.sl.tiles + tile);   // slot, cnt, pos0
        t.rq = ReqDev{v.x, 0, 0, 0, 0};
        t.start = 0, t.cnt = v.y;
        t.pos0 = ((int64_t)(uint32_t)v.w << 32) | (int64_t)(uint32_t)v.z;
        return t;
    }
    t.rq = find_request(p.sl, tile);
    tile_range(tile - t.rq.tile_begin, t.rq.n, kTcTile, p.mini_batch, t.start, t.cnt);
    t.pos0 = t.rq.off + t.start;
    return t;
}

// Cross-feature index generation for a whole launch (Section 3.3, "real-time generation" from the candidate's
// attribute): xb[pos][f] = bucket of candidate pos in field f, or kNoBucket for an id outside the item table.  Done
// once per call so that the layer kernel's gather threads only look the bucket up.
constexpr uint32_t kNoBucket = 0xFFFFu;
__global__ void __launch_bounds__(256) k_cross_buckets(const int32_t *__restrict__ ids, int64_t total, int64_t M, int F, int B,
                                                        int b_mask, int mode, uint16_t *__restrict__ xb)
{
    grid_dep_launch();
    grid_dep_wait();
    // eight threads per candidate, each taking every eighth field: the id is read once per thread, nothing is divided,
    // and a warp's stores cover four candidates' rows of F entries
    const int sub = threadIdx.x & 7;
    for (int64_t pos = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 3; pos < total; pos += ((int64_t)gridDim.x * blockDim.x) >> 3) {
        const int id = ids[pos];
        const bool good = id >= 0 && (int64_t)id < M;
        uint16_t *row = xb + pos * F;
        for (int f = sub; f < F; f += 8) {
            uint32_t bk = kNoBucket;
            if (good) {
                if (mode == AIF_BUCKET_MOD) bk = (uint32_t)(id % B);
                else {
                    const uint64_t h = mix64((uint64_t)id, (uint64_t)f);
                    bk = b_mask >= 0 ? (uint32_t)(h & (uint64_t)b_mask) : (uint32_t)(h % (uint64_t)B);
                }
            }
            row[f] = (uint16_t)bk;
        }
    }
}

// Tile table of a launch over several requests: one thread per tile does the search of the request table that every
// role of every kernel would otherwise repeat per tile (a chain of dependent loads on the critical path of the MMA
// issuers).
__global__ void __launch_bounds__(256) k_tile_table(ScoreLaunch sl, int mini_batch, TileDev *__restrict__ out)
{
    grid_dep_launch();
    grid_dep_wait();
    const int tile = blockIdx.x * blockDim.x + threadIdx.x;
    if (tile >= sl.n_tiles) return;
    const ReqDev rq = find_request(sl, tile);
    int start, cnt;
    tile_range(tile - rq.tile_begin, rq.n, kTcTile, mini_batch, start, cnt);
    TileDev t;
    t.slot = rq.slot, t.cnt = cnt, t.pos0 = rq.off + start, t.L = sl.slots[rq.slot].L;
    t.pad_[0] = t.pad_[1] = t.pad_[2] = 0;
    out[tile] = t;
}

// ---- the layer kernel -----------------------------------------------------------------------------------------
template <int MODE>
__global__ void __launch_bounds__(LayerCfg<MODE>::kThreads, 1) k_layer_tc(const __grid_constant__ CUtensorMap tmapB,
                                                                          const __grid_constant__ CUtensorMap tmapOut,
                                                                          const __grid_constant__ CUtensorMap tmapA, const LayerParams p)
{
    using C = LayerCfg<MODE>;
    constexpr int G = C::G, NB = C::NB, kAcc = C::kAcc, kSA = C::kStagesA, kSB = C::kStagesB;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char *base = reinterpret_cast<unsigned char *>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    // A ring (per stage: one chunk per tile of the group), B ring (per stage: one chunk per output slice), the output
    // staging slabs (2 KB each) of the epilogue warps, then barriers and small arrays
    unsigned char *smA = base, *smB = base + kSA * C::kAStage;
    unsigned char *out_stage = smB + kSB * C::kBStage;
    uint64_t *bars = reinterpret_cast<uint64_t *>(out_stage + C::kEpiWarps * C::kSlabs * 2048);
    uint64_t *full_a = bars, *empty_a = full_a + kSA, *full_b = empty_a + kSA, *empty_b = full_b + kSB;
    uint64_t *acc_full = empty_b + kSB, *acc_empty = acc_full + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    float *bias_s = reinterpret_cast<float *>(((uintptr_t)(tmem_slot + 4) + 15) & ~(uintptr_t)15);   // [kAcc][256]
    float *wout_s = bias_s + kAcc * 256;                         // [kAcc][256]
    int *ids_s = reinterpret_cast<int *>(wout_s + kAcc * 256);   // [2][G][128] validated ids of the current / next item

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < kSA; ++s) {
            mbar_init(smem_u32(full_a + s), C::kProdThreads);
            mbar_init(smem_u32(empty_a + s), 1);
        }
        for (int s = 0; s < kSB; ++s) {
            mbar_init(smem_u32(full_b + s), 1);
            mbar_init(smem_u32(empty_b + s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(acc_full + b), 1);
            mbar_init(smem_u32(acc_empty + b), 4);
        }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == C::kMmaWarp) tmem_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    grid_dep_launch();
    grid_dep_wait();   // everything above overlapped the tail of the previous kernel; from here on its results are read
    // tiles formed on the device (candidates grouped by category): their number is read here
    const int n_tiles = p.sl.n_tiles_dev ? *p.sl.n_tiles_dev : p.sl.n_tiles;
    const int n_groups = (n_tiles + G - 1) / G;
    const int n_ncg = p.n_nchunks / NB;             // groups of output slices
    const int n_items = n_groups * n_ncg;

    if (warp < C::kEpiWarps) {
        // ===================== epilogue =====================
        const int a = warp >> 2;                     // accumulator this warp quartet serves
        const int g = G == 2 ? a : 0;                // its tile of the group
        const int row = (warp & 3) * 32 + lane;      // TMEM lane = candidate row of the tile
        float *bs = bias_s + a * 256, *ws = wout_s + a * 256;
        // staging slabs of 32 rows x 64 bytes, 64-byte swizzle (the layout tmapOut expects)
        unsigned char *stg = out_stage + warp * (C::kSlabs * 2048);
        uint32_t slab = 0;
        int it = 0;
        // a wait that ran out in an earlier kernel of this call left its outputs unwritten: logits computed from them are
        // replaced by NaN
        const bool poisoned = p.epi == EPI_DOT && (*reinterpret_cast<volatile const uint32_t *>(p.sl.status) & AIF_STATUS_TIMEOUT) != 0u;
        for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++it) {
            const int grp = item / n_ncg, nc = (item - grp * n_ncg) * NB + (NB == 2 ? a : 0), n0 = nc * p.n_cols;
            const int buf = kAcc == 1 ? (it & 1) : a;
            const uint32_t ph = kAcc == 1 ? (uint32_t)((it >> 1) & 1) : (uint32_t)(it & 1);
            const TileInfo t = decode_tile(p, grp * G + g, n_tiles);
            if (t.cnt > 0) {
                const float *bias = p.bias_from_slot ? p.sl.slots[t.rq.slot].p_u : p.bias;
                for (int j = row; j < p.n_cols; j += 128) {
                    bs[j] = bias[n0 + j];
                    if (p.epi == EPI_DOT) ws[j] = __bfloat162float(p.w_out[n0 + j]);
                }
            }
            named_bar_sync(1 + a, 128);
            // a wait that ran out is carried to the barrier at the end of the item, so that the four warps of an
            // accumulator leave together and none is left waiting there
            const bool got = __all_sync(0xffffffffu, mbar_wait(smem_u32(acc_full + buf), ph, abort_flag));
            tc_fence_after();
            const bool valid = row < t.cnt;
            const uint32_t taddr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(buf * 256);
            float dot = 0.f;
            const float floor_v = p.linear_out ? -INFINITY : 0.f;
            if (got && t.cnt > 0 && p.epi == EPI_STORE) {
                // Activations of a hidden layer.  The accumulator is read in the 16x256b shape: a thread then owns two
                // columns (per group of eight) over four rows, needs eight bias values per 32 columns instead of all 32,
                // and the bias reads, which every row thread used to repeat, no longer fill the shared memory's return
                // path.  Three instructions per pair of outputs: bias added to both (f32x2), rounded to bf16, ReLU on
                // the rounded pair (rounding is monotonic and keeps zero: the same result in either order).
                const int l4 = lane & 3, r8 = lane >> 2;
                const __nv_bfloat162 floor2 = __float2bfloat162_rn(floor_v);
                const int wrow0 = (warp & 3) * 32;
                for (int c0 = 0; c0 < p.n_cols; c0 += 32) {
                    uint32_t ra[16], rb[16];
                    tmem_ld16x256(taddr + (uint32_t)c0, ra);                    // rows 0..15 of this warp's 32
                    tmem_ld16x256(taddr + (16u << 16) + (uint32_t)c0, rb);      // rows 16..31
                    uint64_t bias2[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) bias2[j] = *reinterpret_cast<const uint64_t *>(bs + c0 + 8 * j + 2 * l4);
                    tmem_ld_wait();
                    // through a staging slab (32 rows x 64 bytes, 64-byte swizzle): the rows of a full slab leave with one
                    // asynchronous tile store, a ragged slab (last tile of a request or mini-batch) with guarded stores
                    unsigned char *sb = stg + slab * 2048;
                    if (lane == 0) bulk_wait_read<C::kSlabs - 1>();   // the store that last read this slab is done with it
                    __syncwarp();
                    auto emit = [&](const uint32_t (&r)[16], int row_h) {
#pragma unroll
                        for (int j = 0; j < 4; ++j)
#pragma unroll
                            for (int q = 0; q < 2; ++q) {
                                float x0, x1;
                                unpack_f32x2(add_f32x2(pack_f32x2(__uint_as_float(r[4 * j + 2 * q]), __uint_as_float(r[4 * j + 2 * q + 1])), bias2[j]), x0, x1);
                                const __nv_bfloat162 h = __hmax2(__floats2bfloat162_rn(x0, x1), floor2);
                                const int rr = row_h + r8 + 8 * q;
                                *reinterpret_cast<uint32_t *>(sb + rr * 64 + ((j ^ ((rr >> 1) & 3)) << 4) + 4 * l4) = *reinterpret_cast<const uint32_t *>(&h);
                            }
                    };
                    emit(ra, 0);
                    emit(rb, 16);
                    if (wrow0 + 32 <= t.cnt) {
                        fence_proxy_async();
                        __syncwarp();
                        if (lane == 0) {
                            tma_store_2d(&tmapOut, smem_u32(sb), n0 + c0, (int)(t.pos0 + wrow0));
                            bulk_commit();
                        }
                    } else {
                        __syncwarp();
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int rr = 8 * j + (lane >> 2), q = lane & 3;
                            const uint4 v = *reinterpret_cast<const uint4 *>(sb + rr * 64 + ((q ^ ((rr >> 1) & 3)) << 4));
                            if (wrow0 + rr < t.cnt)
                                *reinterpret_cast<uint4 *>(p.out + (size_t)(t.pos0 + wrow0 + rr) * p.out_stride + n0 + c0 + q * 8) = v;
                        }
                        __syncwarp();
                    }
                    slab = (slab + 1u) % (uint32_t)C::kSlabs;
                }
            } else if (got && t.cnt > 0 && p.epi == EPI_DOT) {
                // Last hidden layer: ReLU(x + b) . w_out per row, in the same 16x256b shape (eight bias and eight output
                // weights per thread and 32 columns).  A thread sums its column pairs for its four rows; the four
                // threads of a row are joined by shuffles at the end, and the row's own thread takes the result.
                const int l4 = lane & 3;
                uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};   // rows r8, r8 + 8, r8 + 16, r8 + 24 (r8 = lane / 4), two columns each
                for (int c0 = 0; c0 < p.n_cols; c0 += 32) {
                    uint32_t ra[16], rb[16];
                    tmem_ld16x256(taddr + (uint32_t)c0, ra);
                    tmem_ld16x256(taddr + (16u << 16) + (uint32_t)c0, rb);
                    // the last width may end in the middle of these 32 columns (a multiple of 16): the rest is skipped
                    const int n_j = (p.n_cols - c0) >> 3;
                    uint64_t bias2[4], w2[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int col = c0 + 8 * (j < n_j ? j : 0) + 2 * l4;
                        bias2[j] = *reinterpret_cast<const uint64_t *>(bs + col);
                        w2[j] = *reinterpret_cast<const uint64_t *>(ws + col);
                    }
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 4; ++j)
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            if (j >= n_j) continue;   // columns no product wrote
                            float x0, x1, y0, y1;
                            unpack_f32x2(add_f32x2(pack_f32x2(__uint_as_float(ra[4 * j + 2 * q]), __uint_as_float(ra[4 * j + 2 * q + 1])), bias2[j]), x0, x1);
                            unpack_f32x2(add_f32x2(pack_f32x2(__uint_as_float(rb[4 * j + 2 * q]), __uint_as_float(rb[4 * j + 2 * q + 1])), bias2[j]), y0, y1);
                            acc[q] = fma_f32x2(pack_f32x2(fmaxf(x0, 0.f), fmaxf(x1, 0.f)), w2[j], acc[q]);
                            acc[2 + q] = fma_f32x2(pack_f32x2(fmaxf(y0, 0.f), fmaxf(y1, 0.f)), w2[j], acc[2 + q]);
                        }
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float lo, hi;
                    unpack_f32x2(acc[i], lo, hi);
                    float v = lo + hi;
                    v += __shfl_xor_sync(0xffffffffu, v, 1);
                    v += __shfl_xor_sync(0xffffffffu, v, 2);
                    // row 8 i + r8 of this warp's 32 belongs to lane 8 i + r8; lane 4 r8 (among others) holds its sum
                    v = __shfl_sync(0xffffffffu, v, 4 * (lane & 7));
                    if ((lane >> 3) == i) dot = v;
                }
            } else if (got && t.cnt > 0) {
                for (int c0 = 0; c0 < p.n_cols; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld32(taddr + (uint32_t)c0, r);
                    tmem_ld_wait();
                    if (p.epi == EPI_SIGN) {
                        // eq. 5: one bit per output, set where the projection is positive; eight bits per byte, first bit
                        // most significant
                        uint32_t word = 0u;
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            word |= (__uint_as_float(r[i]) > 0.f ? 1u : 0u) << (8 * (i >> 3) + 7 - (i & 7));
                        if (valid) *reinterpret_cast<uint32_t *>(p.sig_out + (size_t)(t.pos0 + row) * (p.out_stride >> 3) + ((n0 + c0) >> 3)) = word;
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (got && lane == 0) mbar_arrive(smem_u32(acc_empty + buf));
            if (p.epi == EPI_DOT && valid) {
                float logit = dot + p.b_out[0];
                if (p.emit_sigmoid) logit = 1.0f / (1.0f + expf(-logit));
                const int id = p.sl.ids[t.pos0 + row];
                // no number for an id outside the table, nor for a tile whose inputs never arrived (here or in an
                // earlier kernel of the call: the status word says so)
                if (id < 0 || (int64_t)id >= p.M || !got || poisoned) logit = __int_as_float(0x7fc00000);
                p.sl.logits[p.sl.out_index ? (int64_t)p.sl.out_index[t.pos0 + row] : t.pos0 + row] = logit;
            }
            if (named_bar_or(1 + a, 128, !got)) break;
        }
        if (lane == 0) bulk_wait<0>();   // all tile stores of this warp have reached global memory
    } else if (warp == C::kMmaWarp) {
        // ===================== MMA issuer =====================
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(kTcTile, p.n_cols);
            const int n_k = p.n_k;
            // descriptors of stage 0 of each ring; stage s lies s stage sizes further (the address field counts 16 bytes)
            const uint64_t bdesc0 = umma_desc_sw128(smem_u32(smB));
            uint64_t adesc0[G];
#pragma unroll
            for (int g = 0; g < G; ++g) adesc0[g] = umma_desc_sw128(smem_u32(smA + g * kABytes));
            int it = 0, sa = 0, sb = 0;
            uint32_t pha = 0, phb = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x, ++it) {
                for (int kc = 0; kc < n_k; ++kc) {
                    if (!mbar_wait(smem_u32(full_a + sa), pha, abort_flag) || !mbar_wait(smem_u32(full_b + sb), phb, abort_flag)) {
                        ok = false;
                        break;
                    }
                    // the A chunk was written by cp.async (generic proxy) and is read by the MMA (async proxy)
                    fence_proxy_async();
                    tc_fence_after();
                    const uint64_t aoff = (uint64_t)(uint32_t)(sa * (C::kAStage >> 4)), boff = (uint64_t)(uint32_t)(sb * (C::kBStage >> 4));
#pragma unroll
                    for (int a = 0; a < kAcc; ++a) {
                        const int buf = kAcc == 1 ? (it & 1) : a;
                        if (kc == 0) {   // the accumulator must have been drained by the epilogue of its previous use
                            const uint32_t eph = (kAcc == 1 ? (uint32_t)((it >> 1) & 1) : (uint32_t)(it & 1)) ^ 1u;
                            if (!mbar_wait(smem_u32(acc_empty + buf), eph, abort_flag)) {
                                ok = false;
                                break;
                            }
                            tc_fence_after();
                        }
                        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * 256);
                        const uint64_t adesc = adesc0[G == 2 ? a : 0] + aoff;
                        const uint64_t bdesc = bdesc0 + boff + (uint64_t)(NB == 2 ? a * (kBBytes >> 4) : 0);
                        // 4 x K=16 inside the 64-column chunk: +32 bytes (2 units) per step
                        umma_bf16(d_tmem, adesc, bdesc, idesc, kc != 0 ? 1u : 0u);
                        umma_bf16_acc(d_tmem, adesc + 2, bdesc + 2, idesc);
                        umma_bf16_acc(d_tmem, adesc + 4, bdesc + 4, idesc);
                        umma_bf16_acc(d_tmem, adesc + 6, bdesc + 6, idesc);
                        if (kc == n_k - 1) umma_commit(smem_u32(acc_full + buf));
                    }
                    if (!ok) break;
                    umma_commit(smem_u32(empty_a + sa));
                    umma_commit(smem_u32(empty_b + sb));
                    if (++sa == kSA) sa = 0, pha ^= 1u;
                    if (++sb == kSB) sb = 0, phb ^= 1u;
                }
            }
        }
        __syncwarp();
    } else if (warp < C::kBWarp) {
        // ===================== A producer (128 threads per tile of the group) =====================
        const int pt = tid - C::kProdWarp0 * 32;
        const int gt = pt >> 7, lp = pt & 127;   // tile of the group this thread serves; its index among that tile's threads
        const int sub = lp & 7;                  // 16-byte slot inside the 128-byte row chunk
        const int r0 = lp >> 3;                  // rows r0, r0+16, ...
        const uint32_t a_off = (uint32_t)(gt * kABytes + r0 * 128) + (uint32_t)((sub ^ (r0 & 7)) << 4);
        const bool deep = p.n_k >= 2;            // bucket look-ups run two chunks ahead (needs the next item at most)

        // The tile of the current / next item: registers hold where it lies, shared memory its validated ids
        // (ids_s[buffer][tile][row], -1 for rows beyond the tile and for ids outside the table).
        struct Rows {
            uint32_t rowmask;        // bit i: row r0 + 16 i lies inside the tile
            uint32_t pos0;
            const uint8_t *Tt;
            const uint16_t *xb;      // bucket row of this thread's first row
        };
        const uint32_t xb_step = (uint32_t)(16 * p.F);   // elements between the bucket rows of rows r0 + 16 i and r0 + 16 (i + 1)
        auto load_rows = [&](int item, Rows &R, int &pend) {
            const TileInfo t = decode_tile(p, (item / n_ncg) * G + gt, n_tiles);
            const int nrows = t.cnt > r0 ? (t.cnt - r0 + 15) >> 4 : 0;
            R.rowmask = (1u << nrows) - 1u, R.pos0 = (uint32_t)t.pos0;
            R.Tt = t.cnt > 0 ? reinterpret_cast<const uint8_t *>(p.sl.slots[t.rq.slot].T) : p.E;
            R.xb = p.xb + (size_t)(t.pos0 + r0) * p.F;
            int id = -1;
            if (lp < t.cnt) {   // this thread fetches the id of row lp; the others read it from shared memory
                id = p.sl.ids ? p.sl.ids[t.pos0 + lp] : 0;   // no id array: a launch over dense rows only
                if (id < 0 || (int64_t)id >= p.M) {
                    id = -1;
                    if (p.check_ids) atomicOr(p.sl.status, AIF_STATUS_BAD_ID);
                }
            }
            pend = id;
        };
        // returns true if some producer thread's wait ran out: they all learn it here and leave together, so that none
        // is left waiting at this barrier
        auto publish = [&](int buf, int pend, bool failed) {
            const bool any = named_bar_or(9, C::kProdThreads, failed);   // every producer thread is done reading what this buffer held
            ids_s[(buf * G + gt) * 128 + lp] = pend;
            named_bar_sync(9, C::kProdThreads);
            return any;
        };
        // bucket of this thread's rows in the field its slot of chunk kc belongs to (cross chunks only); rows outside
        // the tile read other candidates' entries or stale scratch, which rowmask discards
        auto fetch = [&](int kc, const Rows &R, uint32_t (&raw)[8]) {
            const ChunkSrc src = p.src[kc];
            if (src.kind != SRC_CROSS) return;
            const uint16_t *xb = R.xb + (src.off + sub * 8) / p.dc;
#pragma unroll
            for (int i = 0; i < 8; ++i) raw[i] = (uint32_t)__ldg(xb + i * xb_step);
        };
        // global sources of chunk kc: a base pointer and, per row, an offset in 16-byte units; rows whose bit in `mask`
        // is clear are zero-filled
        // (dense chunks: consecutive rows of X / the previous activations, fetched as one TMA tile by the tile's first
        // producer thread; tma_x < 0 marks every other kind)
        auto resolve = [&](int kc, const Rows &R, const int *ids, uint32_t (&raw)[8], bool have_raw, const uint8_t *&bp,
                           uint32_t (&off)[8], uint32_t &mask, int &tma_x, int &tma_y) {
            const ChunkSrc src = p.src[kc];
            tma_x = -1;
            if (src.kind == SRC_DENSE) {
                // rows beyond the tile bring other candidates' values along; their results are never stored
                tma_x = R.rowmask != 0u || lp != 0 ? src.off >> 1 : -2;   // -2: the tile does not exist, nothing to fetch
                tma_y = (int)R.pos0;
                mask = 0;
            } else if (src.kind == SRC_ITEM) {
                const uint32_t row16 = (uint32_t)(p.e_row_bytes >> 4), c16 = (uint32_t)(src.off >> 4) + sub;
                bp = p.E;
                mask = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int id = ids[r0 + 16 * i];
                    off[i] = (uint32_t)(id >= 0 ? id : 0) * row16 + c16;
                    if (id >= 0) mask |= 1u << i;
                }
            } else {
                const int col = src.off + sub * 8;
                const int f = col / p.dc, kin = col - f * p.dc;
                const uint32_t row16 = (uint32_t)(p.dc >> 3), base16 = (uint32_t)(f * p.B) * row16 + (uint32_t)(kin >> 3);
                bp = R.Tt;
                if (!have_raw) {
                    const uint16_t *xb = R.xb + f;
#pragma unroll
                    for (int i = 0; i < 8; ++i) raw[i] = (uint32_t)__ldg(xb + i * xb_step);
                }
                mask = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (raw[i] != kNoBucket) mask |= 1u << i;
                    off[i] = raw[i] * row16 + base16;
                }
                mask &= R.rowmask;
            }
        };

        int s = 0, buf = 0;
        uint32_t ph = 0;
        bool ok = true;
        Rows cur, nxt;
        int pend = -1;
        const uint8_t *bp = p.E;
        uint32_t off[8], raw[8], mask = 0;
        int tma_x = -1, tma_y = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) off[i] = 0, raw[i] = 0;
        if ((int)blockIdx.x < n_items) {
            load_rows(blockIdx.x, cur, pend);
            publish(0, pend, false);
            resolve(0, cur, ids_s + gt * 128, raw, false, bp, off, mask, tma_x, tma_y);
            if (deep) fetch(1, cur, raw);
        }
        nxt = cur;
        for (int item = blockIdx.x; item < n_items; item += gridDim.x, buf ^= 1) {
            const int next_item = item + gridDim.x;
            const bool has_next = next_item < n_items;
            const int *ids_cur = ids_s + (buf * G + gt) * 128, *ids_nxt = ids_s + ((buf ^ 1) * G + gt) * 128;
            if (has_next) load_rows(next_item, nxt, pend);   // the id load lands while chunk 0 is copied
            bool all_out = false;
            for (int kc = 0; kc < p.n_k; ++kc) {
                // a thread whose wait ran out keeps walking (no copies, no arrivals) until the next publish barrier
                if (ok && !mbar_wait(smem_u32(empty_a + s), ph ^ 1u, abort_flag)) ok = false;
                if (!ok) {
                    if (kc == 0 && has_next) all_out = publish(buf ^ 1, pend, true);
                    if (all_out) break;
                    continue;
                }
                if (tma_x == -1) {
                    const uint32_t dst0 = smem_u32(smA + s * C::kAStage) + a_off;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const bool on = (mask >> i) & 1u;
                        cp_async16(dst0 + (uint32_t)(i * 16 * 128), on ? bp + ((size_t)off[i] << 4) : p.E, on ? 16u : 0u);
                    }
                } else if (lp == 0 && tma_x >= 0) {
                    mbar_expect_tx_only(smem_u32(full_a + s), (uint32_t)kABytes);
                    tma_load_2d(smem_u32(smA + s * C::kAStage + gt * kABytes), &tmapA, smem_u32(full_a + s), tma_x, tma_y);
                }
                // the stage's barrier receives this thread's arrival when its copies have landed: no thread waits for them
                cp_async_arrive_noinc(smem_u32(full_a + s));
                if (++s == kSA) s = 0, ph ^= 1u;
                if (kc == 0 && has_next && publish(buf ^ 1, pend, false)) {
                    all_out = true;
                    break;
                }
                // sources of the next chunk from the buckets fetched one iteration ago; then start the fetch for the
                // chunk after it, so that its latency is covered by a whole iteration
                if (kc + 1 < p.n_k) resolve(kc + 1, cur, ids_cur, raw, deep, bp, off, mask, tma_x, tma_y);
                else if (has_next) resolve(0, nxt, ids_nxt, raw, deep, bp, off, mask, tma_x, tma_y);
                if (deep) {
                    if (kc + 2 < p.n_k) fetch(kc + 2, cur, raw);
                    else if (has_next) fetch(kc + 2 - p.n_k, nxt, raw);
                }
            }
            if (all_out) break;
            cur = nxt;
        }
        cp_async_wait_all();
    } else {
        // ===================== B producer (TMA) =====================
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            const uint32_t bytes = (uint32_t)p.n_cols * 128u;
            for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
                const int grp = item / n_ncg, nc0 = (item - grp * n_ncg) * NB;
                for (int kc = 0; kc < p.n_k; ++kc) {
                    if (!mbar_wait(smem_u32(empty_b + s), ph ^ 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    mbar_expect_tx(smem_u32(full_b + s), NB * bytes);
#pragma unroll
                    for (int nb = 0; nb < NB; ++nb)
                        tma_load_2d(smem_u32(smB + s * C::kBStage + nb * kBBytes), &tmapB, smem_u32(full_b + s), kc * 64,
                                    (nc0 + nb) * p.n_cols);
                    if (++s == kSB) s = 0, ph ^= 1u;
                }
            }
        }
        __syncwarp();
    }

    // ---- teardown: everybody arrives here, also after an abort
    if (*abort_flag) {
        if (tid == 0) atomicOr(p.sl.status, AIF_STATUS_TIMEOUT);
        // let copies and MMAs that are still in flight land before shared memory and TMEM go away
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == C::kMmaWarp) tmem_dealloc(tmem_base, 512);
}

// ---- interaction blocks that feed dense columns (CUDA cores; one warp per candidate) ---------------------------
// Writes, per candidate position, a bf16 row [ att (d) | v_bea (d) | lsh_din (d) | simtier (64, first n_tiers used) ]
// holding only the enabled blocks.
__global__ void __launch_bounds__(256) k_interact_x(ModelDev md, ScoreLaunch sl, __nv_bfloat16 *X, int x_stride, int att_done, int lsh_done)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *qv = reinterpret_cast<float *>(smem_raw);                         // [8][d]
    uint32_t *sigq = reinterpret_cast<uint32_t *>(qv + 8 * md.d);            // [8][8]
    int *tiers = reinterpret_cast<int *>(sigq + 64);                         // [8][16]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, d = md.d, dq = d >> 5;
    grid_dep_launch();
    grid_dep_wait();
    // the tile: from the launch's tile table when it has one that was formed on the device, else from the request table
    int slot_index, cnt;
    int64_t pos0;
    if (sl.n_tiles_dev) {
        if ((int)blockIdx.x >= *sl.n_tiles_dev) return;
        const TileDev t = sl.tiles[blockIdx.x];
        slot_index = t.slot, cnt = t.cnt, pos0 = t.pos0;
    } else {
        const ReqDev rq = find_request(sl, blockIdx.x);
        int start;
        tile_range(blockIdx.x - rq.tile_begin, rq.n, kTcTile, md.mini_batch, start, cnt);
        slot_index = rq.slot, pos0 = rq.off + start;
    }
    const SlotDev slot = sl.slots[slot_index];
    // att_done / lsh_done: those columns were already written by the tensor-core attention / LSH kernels
    const bool has_att = md.blocks & AIF_BLK_ATT, do_att = has_att && !att_done, do_bea = md.blocks & AIF_BLK_BEA;
    const bool has_din = md.blocks & AIF_BLK_LSH_DIN, has_tier = md.blocks & AIF_BLK_SIMTIER;
    const bool do_din = has_din && !lsh_done, do_tier = has_tier && !lsh_done, do_lsh = do_din || do_tier;
    const int col_bea = has_att ? d : 0, col_din = col_bea + (do_bea ? d : 0), col_tier = col_din + (has_din ? d : 0);
    using T = __nv_bfloat16;
    for (int c = warp; c < cnt; c += 8) {
        const int64_t pos = pos0 + c;
        const int id = sl.ids[pos];
        T *xrow = X + (size_t)pos * x_stride;
        if (id < 0 || (int64_t)id >= md.M) {
            // zero the columns this kernel owns; the tensor-core kernels zero theirs
            const __nv_bfloat16 z = __float2bfloat16_rn(0.f);
            for (int k = lane; k < d; k += 32) {
                if (do_att) xrow[k] = z;
                if (do_bea) xrow[col_bea + k] = z;
                if (do_din) xrow[col_din + k] = z;
            }
            if (do_tier)
                for (int k = lane; k < 64; k += 32) xrow[col_tier + k] = z;
            continue;
        }
        const T *e = reinterpret_cast<const T *>(md.E) + (size_t)id * d;
        for (int k = lane; k < d; k += 32) qv[warp * d + k] = to_f(e[k]);
        if (do_lsh && lane < (md.lsh_bits >> 5))
            sigq[warp * 8 + lane] = reinterpret_cast<const uint32_t *>(md.sig + (size_t)id * (md.lsh_bits >> 3))[lane];
        if (lane < 16) tiers[warp * 16 + lane] = 0;
        __syncwarp();
        float att[8], din[8];
        if (do_att || do_lsh)
            warp_interact<T>(qv + warp * d, reinterpret_cast<const T *>(slot.S), slot.L, d, rsqrtf((float)d), do_att, do_lsh,
                             do_tier, sigq + warp * 8, slot.sigS, md.lsh_bits, md.n_tiers, tiers + warp * 16, att, din);
        int col = 0;
        if (do_att) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (q < dq) xrow[col + lane + 32 * q] = __float2bfloat16_rn(att[q]);
        }
        if (has_att) col += d;
        if (do_bea) {
            const T *wh = reinterpret_cast<const T *>(md.bea_w) + (size_t)id * md.n_bridge;
            const T *V = reinterpret_cast<const T *>(slot.V);
            for (int k = lane; k < d; k += 32) {
                float acc = 0.f;
                for (int b = 0; b < md.n_bridge; ++b) acc = fmaf(to_f(wh[b]), to_f(V[(size_t)b * d + k]), acc);
                xrow[col + k] = __float2bfloat16_rn(acc);
            }
            col += d;
        }
        if (do_din) {
            const float nrm = md.lsh_din_norm == AIF_NORM_MEAN ? 1.0f / (float)slot.L : 1.0f;
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (q < dq) xrow[col + lane + 32 * q] = __float2bfloat16_rn(din[q] * nrm);
        }
        if (has_din) col += d;
        if (do_tier) {
            __syncwarp();
            const float nrm = md.simtier_norm == AIF_NORM_MEAN ? 1.0f / (float)slot.L : 1.0f;
            for (int k = lane; k < 64; k += 32)
                xrow[col + k] = __float2bfloat16_rn(k < md.n_tiers ? (float)tiers[warp * 16 + k] * nrm : 0.f);
        }
        __syncwarp();
    }
}

// Self-test of the bounded wait: one thread waits, with a short limit, on an mbarrier that nobody arrives on.  The wait
// gives up, raises the status bit and the kernel returns normally: this is the path a scoring kernel takes when a
// producer never delivers, exercised without any fault.
__global__ void k_wait_selftest(uint32_t *status, long long limit_cycles)
{
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const bool done = mbar_try_wait(smem_u32(&bar), 0u, 1000u) || mbar_wait_slow(smem_u32(&bar), 0u, &abort_flag, limit_cycles);
        if (!done && abort_flag) atomicOr(status, AIF_STATUS_TIMEOUT);
    }
}

// W1 [H1 x Din] -> [H1 x k1pad]: user columns dropped, zero padding at the end.
__global__ void k_pack_w1(const __nv_bfloat16 *W1, __nv_bfloat16 *out, int H1, int din, int d, int k1, int k1pad)
{
    const int64_t total = (int64_t)H1 * k1pad;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int j = (int)(i / k1pad), c = (int)(i - (int64_t)j * k1pad);
        out[i] = c < k1 ? W1[(size_t)j * din + d + c] : __float2bfloat16_rn(0.f);
    }
}

// ---- host side ------------------------------------------------------------------------------------------------
struct TcPlan {
    int n_layers = 0;
    int k1 = 0, k1pad = 0, x_cols = 0;
    int n_k[kMaxHidden] = {}, n_cols[kMaxHidden] = {}, n_nchunks[kMaxHidden] = {};
    ChunkSrc src0[kMaxChunks] = {};
    CUtensorMap tmap[kMaxHidden];
    size_t cap_rows = 0;                 // rows of the context's own scratch arrays
    __nv_bfloat16 *W[kMaxHidden] = {};
    __nv_bfloat16 *H[kMaxHidden] = {};   // activations after layer k (k < last)
    __nv_bfloat16 *X = nullptr;
    uint16_t *xb = nullptr;              // cross-feature buckets [positions x F]
    TileDev *tiles = nullptr;            // tile table of a launch over several requests
    size_t tiles_cap = 0;                // its entries
    bool maps_ready = false;
};

int dense_cols(const aif_config &c)
{
    int x = 0;
    if (c.blocks & AIF_BLK_ATT) x += c.d;
    if (c.blocks & AIF_BLK_BEA) x += c.d;
    if (c.blocks & AIF_BLK_LSH_DIN) x += c.d;
    if (c.blocks & AIF_BLK_SIMTIER) x += 64;
    return x;
}

}  // namespace

bool tc_supported(const aif_config &c)
{
    if (c.dtype != AIF_BF16 || c.d % 64 != 0) return false;
    if ((uint64_t)c.M * (uint64_t)c.d * 2 / 16 >= (1ull << 32)) return false;        // row offsets are 32-bit, in 16-byte units
    if ((uint64_t)(c.max_batch_candidates + kTcTile) * 4096 / 16 >= (1ull << 32)) return false;   // same for dense rows
    if (c.blocks & AIF_BLK_CROSS) {
        if ((c.F * c.dc) % 64 != 0 || c.dc % 8 != 0 || c.B >= 65535) return false;
        if (64 % c.dc != 0 && c.dc % 64 != 0) return false;
    }
    for (int k = 0; k < c.n_hidden; ++k) {
        const int H = c.hidden[k];
        if (H <= 256 ? H % 16 != 0 : H % 256 != 0) return false;
        if (k + 1 < c.n_hidden && H % 64 != 0) return false;
    }
    if (c.hidden[c.n_hidden - 1] > 256) return false;
    aif_config tmp = c;
    const int k1 = aif_input_width(&tmp) - c.d;
    if ((k1 + 63) / 64 > kMaxChunks) return false;
    return encode_fn() != nullptr;
}

int tc_tiles_for(const aif_ctx *ctx, int n) { return tiles_of(n, kTcTile, ctx->cfg.mini_batch); }

size_t tc_tile_capacity(const aif_ctx *ctx) { return reinterpret_cast<const TcPlan *>(ctx->tc_plan)->tiles_cap; }

static TcPlan *plan_of(const aif_ctx *ctx) { return reinterpret_cast<TcPlan *>(ctx->tc_plan); }

// Allocates the tensor-path buffers (called from aif_create through tc_prepare_context).
cudaError_t tc_prepare_context(aif_ctx *ctx)
{
    const aif_config &c = ctx->cfg;
    TcPlan *pl = new TcPlan();
    ctx->tc_plan = pl;
    pl->n_layers = c.n_hidden;
    pl->k1 = ctx->input_width - c.d;
    pl->x_cols = dense_cols(c);
    // chunk list of the first layer, in the column order [e | att | cross | bea | din | simtier]
    int n = 0, xoff = 0;
    auto add = [&](int kind, int off) { pl->src0[n].kind = kind, pl->src0[n].off = off, ++n; };
    for (int o = 0; o < c.d; o += 64) add(SRC_ITEM, o * 2);
    if (c.blocks & AIF_BLK_ATT) {
        for (int o = 0; o < c.d; o += 64) add(SRC_DENSE, (xoff + o) * 2);
        xoff += c.d;
    }
    if (c.blocks & AIF_BLK_CROSS)
        for (int o = 0; o < c.F * c.dc; o += 64) add(SRC_CROSS, o);
    if (c.blocks & AIF_BLK_BEA) {
        for (int o = 0; o < c.d; o += 64) add(SRC_DENSE, (xoff + o) * 2);
        xoff += c.d;
    }
    if (c.blocks & AIF_BLK_LSH_DIN) {
        for (int o = 0; o < c.d; o += 64) add(SRC_DENSE, (xoff + o) * 2);
        xoff += c.d;
    }
    if (c.blocks & AIF_BLK_SIMTIER) add(SRC_DENSE, xoff * 2);
    pl->k1pad = n * 64;
    const size_t cap = (size_t)c.max_batch_candidates + kTcTile;
    pl->cap_rows = cap;
    auto alloc = [&](void **p, size_t bytes) -> cudaError_t {
        bytes = (bytes + 255) / 256 * 256;
        cudaError_t e = cudaMalloc(p, bytes);
        if (e != cudaSuccess) return e;
        ctx->allocations.push_back(*p);
        ctx->device_bytes += (int64_t)bytes;
        return cudaMemset(*p, 0, bytes);
    };
    cudaError_t e;
    int in_w = pl->k1pad;
    for (int k = 0; k < c.n_hidden; ++k) {
        const int H = c.hidden[k];
        pl->n_k[k] = in_w / 64;
        pl->n_cols[k] = H <= 256 ? H : 256;
        pl->n_nchunks[k] = H / pl->n_cols[k];
        if ((e = alloc((void **)&pl->W[k], (size_t)H * in_w * 2)) != cudaSuccess) return e;
        if (k + 1 < c.n_hidden && (e = alloc((void **)&pl->H[k], cap * H * 2)) != cudaSuccess) return e;
        in_w = H;
    }
    if (pl->x_cols && (e = alloc((void **)&pl->X, cap * pl->x_cols * 2)) != cudaSuccess) return e;
    if ((c.blocks & AIF_BLK_CROSS) && (e = alloc((void **)&pl->xb, cap * c.F * 2)) != cudaSuccess) return e;
    {
        // Tiles never straddle a mini-batch, so every mini-batch rounds up by itself: a mini-batch of mb candidates is
        // ceil(mb / 128) tiles, and the tail of every request adds at most as many again.
        const size_t mb = (size_t)c.mini_batch;
        const size_t tpm = mb ? (mb + kTcTile - 1) / kTcTile : 0;
        const size_t body = mb ? ((size_t)c.max_batch_candidates / mb + 1) * tpm : (size_t)c.max_batch_candidates / kTcTile + 1;
        pl->tiles_cap = body + (size_t)c.max_user_states * (mb ? tpm : 1) + 64;
        if ((e = alloc((void **)&pl->tiles, pl->tiles_cap * sizeof(TileDev))) != cudaSuccess) return e;
    }
    e = cudaFuncSetAttribute(k_layer_tc<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LayerCfg<0>::kSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_layer_tc<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LayerCfg<1>::kSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_layer_tc<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LayerCfg<2>::kSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_layer_tc<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LayerCfg<3>::kSmem);
    if (e != cudaSuccess) return e;
    // tensor maps over the packed weights: [H x in_w] bf16, box = 64 columns x n_cols rows, 128-byte swizzle
    EncodeFn enc = encode_fn();
    if (!enc) return cudaErrorNotSupported;
    in_w = pl->k1pad;
    for (int k = 0; k < c.n_hidden; ++k) {
        const cuuint64_t dims[2] = {(cuuint64_t)in_w, (cuuint64_t)c.hidden[k]};
        const cuuint64_t strides[1] = {(cuuint64_t)in_w * 2};
        const cuuint32_t box[2] = {64, (cuuint32_t)pl->n_cols[k]};
        const cuuint32_t estr[2] = {1, 1};
        CUresult r = enc(&pl->tmap[k], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, pl->W[k], dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
        in_w = c.hidden[k];
    }
    pl->maps_ready = true;
    if (tc_att_supported(c) && (e = tc_att_prepare(ctx)) != cudaSuccess) return e;
    if (tc_fused_supported(c) && (e = tc_fused_prepare(ctx)) != cudaSuccess) return e;
    if (tc_lsh_supported(c) && (e = tc_lsh_prepare(ctx)) != cudaSuccess) return e;
    if (c.n_categories > 0 && (e = sim_prepare(ctx)) != cudaSuccess) return e;
    return cudaSuccess;
}

const void *tc_weight_tmap(const aif_ctx *ctx, int k) { return &plan_of(ctx)->tmap[k]; }

void tc_destroy_context(aif_ctx *ctx)
{
    if (ctx->tc_att_plan) tc_att_destroy(ctx);
    if (ctx->tc_lsh_plan) tc_lsh_destroy(ctx);
    delete plan_of(ctx);
    ctx->tc_plan = nullptr;
}

cudaError_t tc_prepare_weights(aif_ctx *ctx, const aif_weights *w, cudaStream_t st)
{
    const aif_config &c = ctx->cfg;
    TcPlan *pl = plan_of(ctx);
    k_pack_w1<<<296, 256, 0, st>>>((const __nv_bfloat16 *)w->W[0], pl->W[0], c.hidden[0], ctx->input_width, c.d, pl->k1,
                                   pl->k1pad);
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    for (int k = 1; k < c.n_hidden; ++k) {
        e = cudaMemcpyAsync(pl->W[k], w->W[k], (size_t)c.hidden[k] * c.hidden[k - 1] * 2, cudaMemcpyDeviceToDevice, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_wait_selftest(const aif_ctx *ctx, long long limit_cycles, cudaStream_t st)
{
    k_wait_selftest<<<1, 32, 0, st>>>(ctx->status, limit_cycles);
    count_launch();
    return cudaGetLastError();
}

size_t tc_scratch_row_bytes(const aif_ctx *ctx)
{
    const aif_config &c = ctx->cfg;
    size_t cols = (size_t)plan_of(ctx)->x_cols;
    for (int k = 0; k + 1 < c.n_hidden; ++k) cols += (size_t)c.hidden[k];
    if (c.blocks & AIF_BLK_CROSS) cols += (size_t)c.F;
    return cols * 2;
}

void tc_scratch_layout(const aif_ctx *ctx, void *base, size_t rows, TcScratch *out)
{
    const aif_config &c = ctx->cfg;
    unsigned char *p = reinterpret_cast<unsigned char *>(base);
    out->X = p;
    p += rows * (size_t)plan_of(ctx)->x_cols * 2;
    for (int k = 0; k < kMaxHidden; ++k) {
        out->H[k] = nullptr;
        if (k + 1 < c.n_hidden) {
            out->H[k] = p;
            p += rows * (size_t)c.hidden[k] * 2;
        }
    }
    out->xb = (c.blocks & AIF_BLK_CROSS) ? p : nullptr;
    out->tiles = nullptr;
    out->rows = rows;
}

// One dense layer over `rows` consecutive rows of a row-major bf16 matrix, with the layer kernel: out = act(A W^T + b)
// (bf16), or the packed sign bits of A W^T.  Used by the item side of the nearline pipeline.
cudaError_t tc_dense_layer(const aif_ctx *ctx, const DenseLayer &L, int64_t rows, cudaStream_t st)
{
    if (rows <= 0) return cudaSuccess;
    EncodeFn enc = encode_fn();
    if (!enc) return cudaErrorNotSupported;
    LayerParams p{};
    p.sl.slots = ctx->slots_dev, p.sl.reqs = nullptr, p.sl.n_req = 1;
    p.sl.single = ReqDev{0, (int32_t)rows, 0, 0, 0};
    p.sl.n_tiles = (int32_t)((rows + kTcTile - 1) / kTcTile), p.sl.total = rows, p.sl.max_L = 0;
    p.sl.ids = nullptr, p.sl.logits = nullptr, p.sl.status = ctx->status;
    p.n_cols = L.H <= 256 ? L.H : 256, p.n_nchunks = L.H / p.n_cols, p.n_k = L.in_w / 64, p.mini_batch = 0;
    p.E = (const uint8_t *)ctx->E, p.M = ctx->cfg.M, p.e_row_bytes = ctx->cfg.d * 2;
    p.X = (const uint8_t *)L.A, p.x_row_bytes = L.in_w * 2;
    p.B = 1, p.dc = 8, p.F = 0, p.xb = nullptr, p.check_ids = 0;
    for (int i = 0; i < p.n_k; ++i) p.src[i].kind = SRC_DENSE, p.src[i].off = i * 128;
    p.epi = L.sign_bits ? EPI_SIGN : EPI_STORE;
    p.bias_from_slot = 0, p.bias = L.bias, p.emit_sigmoid = 0, p.linear_out = L.relu ? 0 : 1;
    p.out = (__nv_bfloat16 *)L.out, p.out_stride = L.H, p.sig_out = (uint8_t *)L.out;
    p.w_out = nullptr, p.b_out = nullptr;
    const cuuint32_t estr[2] = {1, 1};
    CUtensorMap tmap_b, tmap_a, tmap_out;
    {
        const cuuint64_t dims[2] = {(cuuint64_t)L.in_w, (cuuint64_t)L.H};
        const cuuint64_t strides[1] = {(cuuint64_t)L.in_w * 2};
        const cuuint32_t box[2] = {64, (cuuint32_t)p.n_cols};
        if (enc(&tmap_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(L.W), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        const cuuint64_t dims[2] = {(cuuint64_t)L.in_w, (cuuint64_t)rows};
        const cuuint64_t strides[1] = {(cuuint64_t)L.in_w * 2};
        const cuuint32_t box[2] = {64, 128};
        if (enc(&tmap_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(L.A), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    tmap_out = tmap_b;
    if (!L.sign_bits) {
        const cuuint64_t dims[2] = {(cuuint64_t)L.H, (cuuint64_t)rows};
        const cuuint64_t strides[1] = {(cuuint64_t)L.H * 2};
        const cuuint32_t box[2] = {32, 32};
        if (enc(&tmap_out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L.out, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    const int single = p.sl.n_tiles * p.n_nchunks;
    const bool pair = ((p.sl.n_tiles + 1) / 2) * p.n_nchunks >= 2 * 148;
    const bool wide = !pair && p.n_nchunks % 2 == 0 && single > 148;
    const int items = pair ? ((p.sl.n_tiles + 1) / 2) * p.n_nchunks : wide ? single / 2 : single;
    const int grid = items < 148 ? items : 148;
    cudaError_t e;
    if (pair) e = launch_pdl(k_layer_tc<1>, dim3(grid), dim3(LayerCfg<1>::kThreads), LayerCfg<1>::kSmem, st, tmap_b, tmap_out, tmap_a, p);
    else if (wide) e = launch_pdl(k_layer_tc<2>, dim3(grid), dim3(LayerCfg<2>::kThreads), LayerCfg<2>::kSmem, st, tmap_b, tmap_out, tmap_a, p);
    else e = launch_pdl(k_layer_tc<0>, dim3(grid), dim3(LayerCfg<0>::kThreads), LayerCfg<0>::kSmem, st, tmap_b, tmap_out, tmap_a, p);
    count_launch();
    return e;
}

cudaError_t launch_score_tc(const aif_ctx *ctx, const ScoreLaunch &sl, int64_t, cudaStream_t st)
{
    TcPlan *pl = plan_of(ctx);
    TcScratch sc;
    sc.X = pl->X;
    sc.xb = pl->xb;
    sc.tiles = pl->tiles;
    sc.rows = pl->cap_rows;
    for (int k = 0; k < kMaxHidden; ++k) sc.H[k] = pl->H[k];
    return launch_score_tc_scratch(ctx, sl, st, sc);
}

cudaError_t launch_score_tc_scratch(const aif_ctx *ctx, const ScoreLaunch &sl_in, cudaStream_t st, const TcScratch &sc)
{
    if (sl_in.n_tiles <= 0) return cudaSuccess;
    ScoreLaunch sl = sl_in;
    sl.tiles = nullptr;
    const aif_config &c = ctx->cfg;
    TcPlan *pl = plan_of(ctx);
    const ModelDev md = make_model(ctx);
    timing_begin(ctx, st);
    // a launch that fits the machine in one round of tiles: the whole pass in one kernel, one CTA per tile
    if (c.n_categories == 0 && sl.n_tiles <= kFusedMaxTiles && sl.max_L <= 256 && tc_fused_supported(c)) {
        StageRange range("aif score_fused");
        cudaError_t e = launch_request_fused(ctx, sl, st);
        timing_mark(ctx, "score_fused", st);
        return e;
    }
    if (c.n_categories > 0) {
        // candidates grouped by (request, category): tiles, grouped ids and the way back to the caller's order
        if (sc.rows < (size_t)sl.total + kTcTile || !ctx->sim_plan) return cudaErrorInvalidValue;
        StageRange range("aif group");
        cudaError_t e = sim_group_candidates(ctx, sl, st);
        timing_mark(ctx, "group", st);
        if (e != cudaSuccess) return e;
    } else if (sl.reqs && sc.tiles) {   // several requests: look every tile up once
        cudaError_t e = launch_pdl(k_tile_table, dim3((sl.n_tiles + 255) / 256), dim3(256), 0, st, sl, c.mini_batch, (TileDev *)sc.tiles);
        count_launch();
        if (e != cudaSuccess) return e;
        sl.tiles = (const TileDev *)sc.tiles;
    }
    if (c.blocks & AIF_BLK_CROSS) {
        StageRange range("aif buckets");
        const int64_t n = sl.total * 8;   // eight threads per candidate
        const int grid = (int)((n + 255) / 256 < 148 * 16 ? (n + 255) / 256 : 148 * 16);
        cudaError_t e = launch_pdl(k_cross_buckets, dim3(grid), dim3(256), 0, st, sl.ids, sl.total, c.M, c.F, c.B,
                                   (c.B & (c.B - 1)) == 0 ? c.B - 1 : -1, c.bucket_mode, (uint16_t *)sc.xb);
        count_launch();
        timing_mark(ctx, "buckets", st);
        if (e != cudaSuccess) return e;
    }
    const bool att_tc = ctx->tc_att_plan != nullptr;
    if (att_tc) {
        StageRange range("aif attention");
        cudaError_t e = launch_att_tc(ctx, sl, st, sc.X, pl->x_cols, sc.rows);
        timing_mark(ctx, "attention", st);
        if (e != cudaSuccess) return e;
    }
    const int lsh_blocks = c.blocks & (AIF_BLK_LSH_DIN | AIF_BLK_SIMTIER);
    const bool lsh_tc = lsh_blocks && ctx->tc_lsh_plan != nullptr;
    if (lsh_tc) {
        // columns of X: [ att | v_bea | lsh_din | simtier (64) ], enabled blocks only
        int col = 0;
        if (c.blocks & AIF_BLK_ATT) col += c.d;
        if (c.blocks & AIF_BLK_BEA) col += c.d;
        const int x_din = (c.blocks & AIF_BLK_LSH_DIN) ? col : -1;
        if (c.blocks & AIF_BLK_LSH_DIN) col += c.d;
        const int x_tier = (c.blocks & AIF_BLK_SIMTIER) ? col : -1;
        StageRange range("aif lsh");
        cudaError_t e = launch_lsh_tc(ctx, sl, st, sc.X, pl->x_cols, sc.rows, x_din, x_tier);
        timing_mark(ctx, "lsh", st);
        if (e != cudaSuccess) return e;
    }
    const bool need_att = (c.blocks & AIF_BLK_ATT) && !att_tc, need_lsh = lsh_blocks && !lsh_tc;
    if (pl->x_cols && (need_att || need_lsh || (c.blocks & AIF_BLK_BEA))) {
        StageRange range("aif interact");
        const size_t smem = (size_t)8 * c.d * 4 + 64 * 4 + 128 * 4;
        cudaError_t e = launch_pdl(k_interact_x, dim3(sl.n_tiles), dim3(256), smem, st, md, sl, (__nv_bfloat16 *)sc.X, pl->x_cols,
                                   att_tc ? 1 : 0, lsh_tc ? 1 : 0);
        count_launch();
        timing_mark(ctx, "interact", st);
        if (e != cudaSuccess) return e;
    }
    static const char *names[kMaxHidden] = {"layer1", "layer2", "layer3", "layer4"};
    static const char *range_names[kMaxHidden] = {"aif layer1", "aif layer2", "aif layer3", "aif layer4"};
    for (int k = 0; k < c.n_hidden; ++k) {
        StageRange range(range_names[k]);
        LayerParams p{};
        p.sl = sl;
        p.n_nchunks = pl->n_nchunks[k], p.n_cols = pl->n_cols[k], p.n_k = pl->n_k[k], p.mini_batch = c.mini_batch;
        p.E = (const uint8_t *)ctx->E, p.M = c.M, p.e_row_bytes = c.d * 2;
        p.B = c.B > 0 ? c.B : 1, p.dc = c.dc > 0 ? c.dc : 8, p.F = c.F, p.xb = (const uint16_t *)sc.xb;
        p.check_ids = k == 0;
        if (k == 0) {
            p.X = (const uint8_t *)sc.X, p.x_row_bytes = pl->x_cols * 2;
            for (int i = 0; i < p.n_k; ++i) p.src[i] = pl->src0[i];
        } else {
            p.X = (const uint8_t *)sc.H[k - 1], p.x_row_bytes = c.hidden[k - 1] * 2;
            for (int i = 0; i < p.n_k; ++i) p.src[i].kind = SRC_DENSE, p.src[i].off = i * 128;
        }
        const bool last = k + 1 == c.n_hidden;
        // store target of the epilogue: the activation array as a [rows x hidden[k]] tensor, 32 x 32 boxes, 64-byte swizzle
        CUtensorMap tmap_out = pl->tmap[k];
        if (!last) {
            const cuuint64_t dims[2] = {(cuuint64_t)c.hidden[k], (cuuint64_t)sc.rows};
            const cuuint64_t strides[1] = {(cuuint64_t)c.hidden[k] * 2};
            const cuuint32_t box[2] = {32, 32};
            const cuuint32_t estr[2] = {1, 1};
            CUresult r = encode_fn()(&tmap_out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, sc.H[k], dims, strides, box, estr,
                                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
        }
        p.epi = last ? EPI_DOT : EPI_STORE;
        p.bias_from_slot = k == 0, p.bias = ctx->b[k], p.emit_sigmoid = c.emit_sigmoid;
        p.out = (__nv_bfloat16 *)sc.H[k], p.out_stride = c.hidden[k];
        p.w_out = (const __nv_bfloat16 *)ctx->w_out, p.b_out = ctx->b_out;
        // two tiles per item once that still leaves every SM at least two items; else, if single items would need a
        // second round on some SMs, one tile with two output slices per item
        const int single = sl.n_tiles * p.n_nchunks;
        const bool pair = ((sl.n_tiles + 1) / 2) * p.n_nchunks >= 2 * 148;
        const bool wide = !pair && p.n_nchunks % 2 == 0 && single > 148;
        const int items = pair ? ((sl.n_tiles + 1) / 2) * p.n_nchunks : wide ? single / 2 : single;
        const int grid = items < 148 ? items : 148;
        // load source of the dense chunks: X (layer 1) or the previous activations, 64-column x 128-row tiles
        CUtensorMap tmap_a = pl->tmap[k];
        const int dense_w = k == 0 ? pl->x_cols : c.hidden[k - 1];
        if (dense_w > 0) {
            const cuuint64_t dims[2] = {(cuuint64_t)dense_w, (cuuint64_t)sc.rows};
            const cuuint64_t strides[1] = {(cuuint64_t)dense_w * 2};
            const cuuint32_t box[2] = {64, 128};
            const cuuint32_t estr[2] = {1, 1};
            CUresult r = encode_fn()(&tmap_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<uint8_t *>(p.X), dims, strides, box, estr,
                                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
        }
        cudaError_t e;
        if (pair && k == 0 && (c.blocks & AIF_BLK_CROSS))
            e = launch_pdl(k_layer_tc<3>, dim3(grid), dim3(LayerCfg<3>::kThreads), LayerCfg<3>::kSmem, st, pl->tmap[k], tmap_out, tmap_a, p);
        else if (pair) e = launch_pdl(k_layer_tc<1>, dim3(grid), dim3(LayerCfg<1>::kThreads), LayerCfg<1>::kSmem, st, pl->tmap[k], tmap_out, tmap_a, p);
        else if (wide) e = launch_pdl(k_layer_tc<2>, dim3(grid), dim3(LayerCfg<2>::kThreads), LayerCfg<2>::kSmem, st, pl->tmap[k], tmap_out, tmap_a, p);
        else e = launch_pdl(k_layer_tc<0>, dim3(grid), dim3(LayerCfg<0>::kThreads), LayerCfg<0>::kSmem, st, pl->tmap[k], tmap_out, tmap_a, p);
        count_launch();
        timing_mark(ctx, names[k], st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace aif
