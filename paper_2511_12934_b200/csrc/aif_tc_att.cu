// Dense target attention on the tensor cores (sm_100a): att_i = softmax(e_i S^T / sqrt(d)) S for tiles of 128
// candidates against the request's projected behaviour sequence S [L x d] (Section 4.2, first paragraph: similarity
// of the target item with every historical item, then pooling; here in its dense softmax form).
//
// One CTA per SM walks over the tiles blockIdx.x, blockIdx.x + gridDim.x, ... (or one CTA per tile when no SM has two).
// Warps at d = 128 (512 threads; d = 256 in brackets, 256 threads):
//   0-7 [0-3]  softmax: per key block read the score row from TMEM into registers, exponentials in fp32, and write the
//              probabilities back into the same TMEM columns as packed bf16 pairs (the A operand of P V is read from
//              tensor memory and never crosses shared memory).  A thread owns a candidate row; at d = 128 two warps
//              share each quarter of the rows, each with half of a block's keys, and agree on the block maximum through
//              shared memory.  At the end of a tile: hand the row sums to the output warps (d = 128) or normalise O and
//              store the attention rows themselves (d = 256)
//   8  [4]     allocates TMEM; one lane issues scores = Q K^T (both K-major) up to two blocks ahead of the softmax
//   9  [5]     one lane streams key/value blocks of S with TMA (3-D tensor map over the user-state arena)
//   10 [6]     gathers the item rows of the next tile (the queries) with cp.async while the current tile is processed
//              (two query buffers)
//   11 [7]     one lane issues O += P V, with V read from the very same shared-memory tile as K, as an MN-major B operand
//   12-15      d = 128 only: normalise the finished tile's O accumulator and store its rows while the other warps are
//              on the next tile (two O accumulators fill the 512 tensor-memory columns)
// TMEM: two score buffers (so the softmax of block j overlaps Q K^T of block j+1) and the O accumulator.
// The running maximum is only raised when a row's block maximum exceeds it by more than 8 (in the log2 domain);
// then the warp rescales its 32 rows of O in TMEM.  Until then probabilities stay below 2^8, which fp32 sums and
// bf16 operands hold without loss of accuracy.  Every wait is bounded.
#include <type_traits>

#include "aif_device.cuh"
#include "aif_internal.h"
#include "aif_tc_ptx.cuh"

namespace aif {
namespace {


struct AttParams {
    ScoreLaunch sl;
    const uint8_t *E;
    int64_t M;
    int32_t mini_batch;
    int32_t x_stride;        // elements per row of X
    __nv_bfloat16 *X;        // attention rows go to columns [0, d)
    float scale_log2;        // log2(e) / sqrt(d)
    const float *q_norm;     // device: upper bound on the Euclidean norm of a query row, or nullptr (none known)
};

// A request whose scores are bounded by this many powers of two on either side (|q| |k| log2(e) / sqrt(d), from the norm
// bounds kept with the table and with the slot) needs no running maximum: softmax does not depend on the exponent's
// offset, 2^+-50 is far inside the range of fp32 sums and of bf16 probabilities, whose relative precision does not
// depend on the magnitude.  Without the maximum a block costs its warps no reduction, no exchange between the two
// warps of a row quarter and no barrier, so the two run out of step and one's exponentials cover the other's loads.
constexpr float kNoMaxBound = 50.0f;

template <int D, int BN>
struct AttCfg {
    static constexpr int kQChunks = D / 64;             // 64-column (128-byte) chunks of a row
    static constexpr int kQBytes = kQChunks * 128 * 128;
    static constexpr int kQBufs = 2;                    // query buffers
    static constexpr int kKvStages = D <= 128 ? 4 : 3;
    static constexpr int kKvChunkBytes = BN * 128;      // one 64-column chunk of a key block
    static constexpr int kKvBytes = kQChunks * kKvChunkBytes;
    // tensor memory: two score buffers of BN columns | two probability buffers of BN / 2 columns (packed bf16 pairs) | O.
    // The probabilities have columns of their own: a score buffer is free for the scores of block j + 2 as soon as the
    // softmax warps have read block j out of it, not only once P V of block j has run.
    static constexpr int kTmemP = 2 * BN;
    static constexpr int kTmemO = 3 * BN;
    // d = 128: four more warps normalise and store a finished tile while the softmax warps and the Q K^T products are
    // already on the next one (its first P V waits until they have read the accumulator)
    static constexpr bool kSplitEpi = D <= 128;
    // softmax warps per quarter of the rows, each with its share of a block's keys: one warp alone leaves its scheduler
    // idle through every tensor-memory round trip and hand-over
    static constexpr int kHalves = D <= 128 ? 2 : 1;
    static constexpr int kSoftWarps = 4 * kHalves;
    static constexpr int kMmaWarp = kSoftWarps, kTmaWarp = kSoftWarps + 1, kGatherWarp = kSoftWarps + 2;
    static constexpr int kPvWarp = kSoftWarps + 3;     // issues the P V products (kMmaWarp: Q K^T, and owns tensor memory)
    static constexpr int kEpiWarp0 = kSoftWarps + 4;   // first of the four output warps (kSplitEpi)
    static constexpr int kThreads = (kSoftWarps + 4 + (kSplitEpi ? 4 : 0)) * 32;
    // barriers and the tensor-memory slot; row sums [2 tiles][kHalves][128]; block maxima [2 blocks][2][128]
    static constexpr int kMisc = 512 + (kSplitEpi ? 2 * kHalves * 512 : 0) + (kHalves == 2 ? 2048 : 0);
    static constexpr size_t kSmem = 1024 + kQBufs * kQBytes + kKvStages * kKvBytes + kMisc;
};

// One tile of the launch as every role needs it.
struct AttTile {
    int slot, cnt, nb, L;
    int key0;   // first key row: 0, or where the tile's category's sub-sequence begins in the grouped sequence
    int64_t pos0;
};

template <int BN>
__device__ __forceinline__ AttTile att_tile(const AttParams &p, int tile)
{
    AttTile t;
    if (p.sl.tiles) {   // looked up once per launch (k_tile_table)
        const int4 v = *reinterpret_cast<const int4 *>(p.sl.tiles + tile);   // slot, cnt, pos0
        t.slot = v.x, t.cnt = v.y;
        t.pos0 = ((int64_t)(uint32_t)v.w << 32) | (int64_t)(uint32_t)v.z;
        t.L = p.sl.tiles[tile].L, t.key0 = p.sl.tiles[tile].key0;
        // an empty sub-sequence still walks one key block, every column of it masked: the roles' hand-overs stay the same
        t.nb = t.L > 0 ? (t.L + BN - 1) / BN : 1;
        return t;
    }
    const ReqDev rq = find_request(p.sl, tile);
    int start, cnt;
    tile_range(tile - rq.tile_begin, rq.n, kTcTile, p.mini_batch, start, cnt);
    t.slot = rq.slot, t.cnt = cnt, t.pos0 = rq.off + start;
    t.L = p.sl.slots[rq.slot].L, t.key0 = 0;
    t.nb = (t.L + BN - 1) / BN;
    return t;
}

template <int D, int BN>
__global__ void __launch_bounds__((AttCfg<D, BN>::kThreads), 1) k_att_tc(const __grid_constant__ CUtensorMap tmapS,
                                                           const __grid_constant__ CUtensorMap tmapX, const AttParams p)
{
    using C = AttCfg<D, BN>;
    constexpr int kS = C::kKvStages, kQB = C::kQBufs;
    constexpr bool kSplit = C::kSplitEpi;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char *base = reinterpret_cast<unsigned char *>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    unsigned char *smQ = base;
    unsigned char *smKV = smQ + kQB * C::kQBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smKV + kS * C::kKvBytes);
    uint64_t *kv_full = bars, *kv_empty = bars + kS;
    uint64_t *s_full = bars + 2 * kS, *p_full = s_full + 2, *pv_done = p_full + 2;
    uint64_t *q_full = pv_done + 2, *q_empty = q_full + 2, *o_final = q_empty + 2, *o_free = o_final + 2, *l_ready = o_free + 2;
    uint64_t *q_first = l_ready + 2, *s_free = q_first + 1;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(s_free + 2);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    float *l_s = reinterpret_cast<float *>(tmem_slot + 4);   // [2][kHalves][128] row sums handed to the output warps
    float *mx_s = l_s + (kSplit ? 2 * C::kHalves * 128 : 0);    // [2][2][128] block maxima exchanged between partner warps

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < kS; ++s) {
            mbar_init(smem_u32(kv_full + s), 1);
            mbar_init(smem_u32(kv_empty + s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(s_full + b), 1);
            mbar_init(smem_u32(p_full + b), C::kSoftWarps * 32);
            mbar_init(smem_u32(pv_done + b), 1);
            mbar_init(smem_u32(s_free + b), C::kSoftWarps);
            mbar_init(smem_u32(q_full + b), 32);
            mbar_init(smem_u32(q_empty + b), 5);   // the last Q K^T of the tenant, and the four softmax warps' output staging
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(o_final + b), 1);
            mbar_init(smem_u32(o_free + b), 128);
            mbar_init(smem_u32(l_ready + b), C::kSoftWarps * 32);
        }
        mbar_init(smem_u32(q_first), C::kSoftWarps * 32);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == C::kMmaWarp) tmem_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    grid_dep_launch();
    grid_dep_wait();   // the set-up above overlapped the previous kernel; the request table and slots are read from here on

    const int n_tiles = p.sl.n_tiles_dev ? *p.sl.n_tiles_dev : p.sl.n_tiles;

    // Normalises a finished tile's O accumulator and stores the attention rows.  Run by the softmax warps themselves
    // (d = 256) or by the epilogue warps (d = 128); wq = the warp's quarter of the TMEM lanes.
    auto tile_epilogue = [&](int k, const AttTile &t, float l_sum, int wq, int lane) {
        const int row = wq * 32 + lane;
        const uint32_t lane_base = tmem_base + ((uint32_t)(wq * 32) << 16);
        const uint32_t o_col = (uint32_t)C::kTmemO;
        uint64_t *o_free_k = o_free + (kSplit ? (k & 1) : 0);
        const float inv = l_sum > 0.f ? 1.0f / l_sum : 0.f;   // no key at all (an empty sub-sequence): a zero row
        bool good = false;
        if (row < t.cnt) {
            const int id = p.sl.ids[t.pos0 + row];
            good = id >= 0 && (int64_t)id < p.M;
        }
        // Output rows leave through shared memory and asynchronous tile stores: a thread owns a row, so direct stores
        // are 32 scattered half-used sectors per instruction, which cost several thousand cycles per tile.  The
        // staging slabs (2 x 2 KB per warp, 64-byte swizzle) live in the tile's own query buffer: every Q K^T of the
        // tile is complete, and the gather of the buffer's next tenant waits for these warps as well.
        const int qb_out = k % kQB;
        unsigned char *stg = smQ + qb_out * C::kQBytes + wq * 4096;
        const bool whole = wq * 32 + 32 <= t.cnt;   // ragged last tiles keep the guarded direct stores
        uint32_t slab = 0;
        auto emit = [&](const uint32_t (&r)[32], int c0) {
            uint32_t packed[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const __nv_bfloat162 h = __floats2bfloat162_rn(good ? __uint_as_float(r[2 * i]) * inv : 0.f,
                                                               good ? __uint_as_float(r[2 * i + 1]) * inv : 0.f);
                packed[i] = *reinterpret_cast<const uint32_t *>(&h);
            }
            if (whole) {
                unsigned char *sb = stg + slab * 2048;
                if (lane == 0) bulk_wait_read<1>();   // the store that last read this slab is done with it
                __syncwarp();
                const int swz = (lane >> 1) & 3;
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    *reinterpret_cast<uint4 *>(sb + lane * 64 + ((q ^ swz) << 4)) =
                        make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(&tmapX, smem_u32(sb), c0, (int)(t.pos0 + wq * 32));
                    bulk_commit();
                }
                slab ^= 1u;
            } else if (row < t.cnt) {
                uint4 *dst = reinterpret_cast<uint4 *>(p.X + (size_t)(t.pos0 + row) * p.x_stride + c0);
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    dst[q] = make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
            }
        };
        // two chunks of 32 columns per round; the load of the next chunk is in flight while one is converted and staged
        uint32_t ra[32], rb[32];
        tmem_ld32(lane_base + o_col, ra);
#pragma unroll 1
        for (int c0 = 0; c0 < D; c0 += 64) {
            tmem_ld_wait();
            tmem_ld32(lane_base + o_col + (uint32_t)(c0 + 32), rb);
            emit(ra, c0);
            tmem_ld_wait();
            if (c0 + 64 < D) tmem_ld32(lane_base + o_col + (uint32_t)(c0 + 64), ra);
            else {   // O is in registers: the next tile's first P V may overwrite the accumulator
                tc_fence_before();
                mbar_arrive(smem_u32(o_free_k));
            }
            emit(rb, c0 + 32);
        }
        if (lane == 0) {
            bulk_wait_read<0>();   // the staging is no longer read: the query buffer may take its next tenant
            mbar_arrive(smem_u32(q_empty + qb_out));
        }
    };

    if (warp < C::kSoftWarps) {
        // ===================== softmax, output =====================
        // kH warps share a quarter of the rows (the tensor-memory lanes 32 wq ...): each takes CW of a block's BN keys.
        constexpr int kH = C::kHalves, CW = BN / kH;
        const int wq = warp & 3, half = warp >> 2;
        const int row = wq * 32 + lane;
        const uint32_t lane_base = tmem_base + ((uint32_t)(wq * 32) << 16);
        const float k2 = p.scale_log2;
        bool ok = true;
        bool late = false;   // kH = 2: a wait failed where the partner warp cannot see it; both leave at the next pair barrier
        uint32_t gb = 0;     // key blocks processed so far by this CTA (all tiles): selects score / P buffers and phases
        int k = 0;           // tiles processed so far
        if ((int)blockIdx.x < n_tiles) {
            // The CTA's first tile has nobody to prefetch it: these warps, idle until the first scores arrive, gather
            // its queries (8 threads per row, 16 bytes each per 128-byte chunk); later tiles come from the gather warp.
            const AttTile t = att_tile<BN>(p, blockIdx.x);
            const int sub = tid & 7, r0 = tid >> 3;
#pragma unroll
            for (int i = 0; i < 8 / kH; ++i) {
                const int r = r0 + 16 * kH * i;
                int id = -1;
                if (r < t.cnt) {
                    id = p.sl.ids[t.pos0 + r];
                    if (id < 0 || (int64_t)id >= p.M) id = -1;
                }
                const uint8_t *g = p.E + (id >= 0 ? (size_t)id * (D * 2) + sub * 16 : 0);
                const uint32_t dst = smem_u32(smQ) + (uint32_t)(r * 128) + (uint32_t)((sub ^ (r & 7)) << 4);
#pragma unroll
                for (int c = 0; c < C::kQChunks; ++c) cp_async16(dst + c * 16384, g + c * 128, id >= 0 ? 16u : 0u);
            }
            cp_async_arrive_noinc(smem_u32(q_first));
        }
        for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x, ++k) {
            const AttTile t = att_tile<BN>(p, tile);
            const int L = t.L;
            // Decided once per tile and agreed on by the warps that meet at a barrier in the other mode: two warps
            // reading a bound that a refresh is raising meanwhile must not come to different answers.
            const float bound = p.q_norm ? *p.q_norm * *p.sl.slots[t.slot].k_norm * k2 : INFINITY;
            bool fast = bound <= kNoMaxBound;    // NaN: false
            if (kH == 2) fast = !named_bar_or(1 + wq, 64, !fast || late);
            else fast = __all_sync(0xffffffffu, fast);
            float m_used = fast ? 0.f : -INFINITY, l_sum = 0.f;
            for (int j = 0; j < t.nb; ++j, ++gb) {
                const int b = (int)(gb & 1u);
                const int valid_cols = min(BN, L - j * BN);
                const int vc = min(CW, valid_cols - half * CW);   // this warp's keys of the block that exist (may be <= 0)
                const bool got = __all_sync(0xffffffffu, mbar_wait(smem_u32(s_full + b), (gb >> 1) & 1u, abort_flag));
                const uint32_t ts = lane_base + (uint32_t)(b * BN);
                // the row's CW scores: all loads first, one wait
                uint32_t sc[CW];
                float mt = -INFINITY;
                if (got) {
                    tc_fence_after();
#pragma unroll
                    for (int c0 = 0; c0 < CW; c0 += 32)
                        tmem_ld32(ts + (uint32_t)(half * CW + c0), *reinterpret_cast<uint32_t(*)[32]>(&sc[c0]));
                }
                // the probability buffer's previous reader, P V of block gb - 2, must be done with it (long since, as a rule)
                const bool p_free = gb < 2 || __all_sync(0xffffffffu, mbar_wait(smem_u32(pv_done + b), ((gb - 2) >> 1) & 1u, abort_flag));
                if (got) {
                    tmem_ld_wait();
                    // the scores are in registers: the buffer may take the scores of block gb + 2
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(s_free + b));
                }
                if (fast) {
                    if (!got || !p_free) {   // nobody waits for this warp inside the block: it goes on empty-handed to the next meeting point
                        if (kH == 2) {
                            late = true;
                            continue;
                        }
                        ok = false;
                        break;
                    }
                } else {
                if (got) {
                    // block maximum of the row (four independent chains)
                    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                    if (vc == CW) {
#pragma unroll
                        for (int i = 0; i < CW; i += 8) {   // three-input maxima: two scores per instruction
                            mx4[0] = fmax3(mx4[0], __uint_as_float(sc[i]), __uint_as_float(sc[i + 1]));
                            mx4[1] = fmax3(mx4[1], __uint_as_float(sc[i + 2]), __uint_as_float(sc[i + 3]));
                            mx4[2] = fmax3(mx4[2], __uint_as_float(sc[i + 4]), __uint_as_float(sc[i + 5]));
                            mx4[3] = fmax3(mx4[3], __uint_as_float(sc[i + 6]), __uint_as_float(sc[i + 7]));
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < CW; ++i)
                            if (i < vc) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(sc[i]));
                    }
                    mt = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * k2;
                }
                if (kH == 2) {
                    // The two warps of a row quarter agree on the block maximum through shared memory (two buffers: the
                    // partner may still read block gb - 1's value).
                    float *mx = mx_s + (gb & 1u) * 256;
                    mx[half * 128 + row] = mt;
                    tc_fence_before();
                    const bool bad = named_bar_or(1 + wq, 64, !got || !p_free || late);
                    tc_fence_after();
                    if (bad) {
                        ok = false;
                        break;
                    }
                    mt = fmaxf(mt, mx[(half ^ 1) * 128 + row]);
                } else if (!got || !p_free) {
                    ok = false;
                    break;
                }
                if (j == 0) {
                    m_used = mt;
                } else {
                    const bool need = mt > m_used + 8.0f;
                    if (__any_sync(0xffffffffu, need)) {
                        // raise the running maximum and rescale this warp's share of its rows of O (rare)
                        const float m_new = need ? mt : m_used;
                        const float f = fast_exp2(m_used - m_new);
                        l_sum *= f;
                        m_used = m_new;
                        const bool pv = __all_sync(0xffffffffu, mbar_wait(smem_u32(pv_done + ((gb - 1) & 1u)),
                                                                           ((gb - 1) >> 1) & 1u, abort_flag));
                        if (!pv) {
                            if (kH == 2) {
                                late = true;
                            } else {
                                ok = false;
                                break;
                            }
                        } else {
                            tc_fence_after();
#pragma unroll 1
                            for (int c0 = half * (D / kH); c0 < (half + 1) * (D / kH); c0 += 32) {
                                uint32_t r[32];
                                const uint32_t oc = (uint32_t)(C::kTmemO + c0);
                                tmem_ld32(lane_base + oc, r);
                                tmem_ld_wait();
#pragma unroll
                                for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
                                tmem_st32(lane_base + oc, r);
                            }
                            tmem_st_wait();
                        }
                    }
                }
                }
                // probabilities -> packed bf16 pairs in the block's probability buffer
                // The loop is bound by issue slots, so exponent and row sum are formed two at a time (f32x2), and the
                // masking of keys past the end of the sequence exists only in the copy a ragged last block runs.
                const uint64_t k2p = pack_f32x2(k2, k2), mneg = pack_f32x2(-m_used, -m_used);
                uint64_t ls2[2] = {0ull, 0ull};
                auto probabilities = [&](auto masked) {
#pragma unroll
                    for (int c0 = 0; c0 < CW; c0 += 64) {
                        uint32_t packed[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            float p0, p1;
                            unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sc[c0 + 2 * i]), __uint_as_float(sc[c0 + 2 * i + 1])), k2p, mneg), p0, p1);
                            p0 = fast_exp2(p0), p1 = fast_exp2(p1);
                            if (decltype(masked)::value) {
                                if (c0 + 2 * i >= vc) p0 = 0.f;
                                if (c0 + 2 * i + 1 >= vc) p1 = 0.f;
                            }
                            ls2[i & 1] = add_f32x2(ls2[i & 1], pack_f32x2(p0, p1));
                            const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                            packed[i] = *reinterpret_cast<const uint32_t *>(&h);
                        }
                        tmem_st32(lane_base + (uint32_t)(C::kTmemP + b * (BN / 2) + ((half * CW + c0) >> 1)), packed);
                    }
                };
                if (vc == CW) probabilities(std::false_type{});
                else probabilities(std::true_type{});
                tmem_st_wait();
                {
                    float a0, a1, b0, b1;
                    unpack_f32x2(ls2[0], a0, a1), unpack_f32x2(ls2[1], b0, b1);
                    l_sum += (a0 + a1) + (b0 + b1);
                }
                tc_fence_before();
                mbar_arrive(smem_u32(p_full + b));
            }
            if (!ok) break;
            if (kSplit) {
                // hand the row sums to the output warps and go on with the next tile.  l_s[k & 1] was last read by the
                // output of tile k - 2, before it released that O accumulator.
                if (k >= 2 && !__all_sync(0xffffffffu, mbar_wait(smem_u32(o_free + (k & 1)), (uint32_t)(((k - 2) >> 1) & 1), abort_flag))) {
                    if (kH == 2) {
                        late = true;
                        continue;
                    }
                    ok = false;
                    break;
                }
                l_s[((k & 1) * kH + half) * 128 + row] = l_sum;
                mbar_arrive(smem_u32(l_ready + (k & 1)));
            } else {
                if (!mbar_wait(smem_u32(o_final), (uint32_t)(k & 1), abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                tile_epilogue(k, t, l_sum, warp, lane);
            }
        }
        if (lane == 0) bulk_wait<0>();   // all tile stores of this warp have reached global memory
    } else if (warp == C::kMmaWarp || warp == C::kPvWarp) {
        // ===================== MMA issuers =====================
        // One lane of one warp issues the Q K^T products, one lane of another the P V products: a single issuer spends
        // more time in its waits, fences and commits than the sixteen products of a key block take, and the tensor pipe
        // idles meanwhile.  Each walks the flat sequence of key blocks of this CTA's tiles with a cursor of its own.
        if (lane == 0) {
            constexpr uint32_t idesc_qk = umma_idesc_bf16(kTcTile, BN);
            constexpr uint32_t idesc_pv = umma_idesc_bf16_bmn(kTcTile, D);
            struct Cursor {
                int tile, k, j, nb;
                uint32_t gb;
                int nb_next;   // key blocks of the tile after this one, fetched a whole tile ahead of its use
            };
            auto blocks_of = [&](int tile) { return tile < n_tiles ? att_tile<BN>(p, tile).nb : 0; };
            auto open_tile = [&](Cursor &c) {
                c.nb = c.nb_next;
                c.nb_next = blocks_of(c.tile + (int)gridDim.x);
            };
            auto advance = [&](Cursor &c) {
                ++c.gb;
                if (++c.j == c.nb) {
                    c.j = 0, c.tile += gridDim.x, ++c.k;
                    open_tile(c);
                }
            };
            Cursor c{(int)blockIdx.x, 0, 0, 0, 0u, 0};
            c.nb_next = blocks_of(c.tile);
            open_tile(c);
            bool ok = true;
            if (warp == C::kMmaWarp) {
                // scores of block gb into buffer gb & 1, up to two blocks ahead of the softmax
                // operand descriptors of buffer / stage 0; the others lie a fixed number of 16-byte units further
                const uint64_t qdesc0 = umma_desc_sw128(smem_u32(smQ)), kdesc0 = umma_desc_sw128(smem_u32(smKV));
                while (ok && c.tile < n_tiles) {
                    const int qb = c.k % kQB;
                    if (c.j == 0) {   // first block of a tile: its queries must have landed (cp.async, generic proxy)
                        ok = c.k == 0 ? mbar_wait(smem_u32(q_first), 0u, abort_flag)
                                      : mbar_wait(smem_u32(q_full + qb), (uint32_t)(((c.k - 1) / kQB) & 1), abort_flag);
                        if (!ok) break;
                        fence_proxy_async();
                    }
                    const int s = (int)(c.gb % kS);
                    if (!mbar_wait(smem_u32(kv_full + s), (c.gb / kS) & 1u, abort_flag)) break;
                    // the buffer's previous content, the scores of block gb - 2, must have been read by every softmax warp
                    if (c.gb >= 2 && !mbar_wait(smem_u32(s_free + (c.gb & 1u)), ((c.gb - 2) >> 1) & 1u, abort_flag)) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + (uint32_t)((c.gb & 1u) * BN);
                    const uint64_t qd = qdesc0 + (uint64_t)(uint32_t)(qb * (C::kQBytes >> 4));
                    const uint64_t kd = kdesc0 + (uint64_t)(uint32_t)(s * (C::kKvBytes >> 4));
                    umma_bf16(d_tmem, qd, kd, idesc_qk, 0u);
#pragma unroll
                    for (int kk = 1; kk < D / 16; ++kk)
                        umma_bf16_acc(d_tmem, qd + (uint64_t)((kk >> 2) * (16384 >> 4) + 2 * (kk & 3)),
                                      kd + (uint64_t)((kk >> 2) * (C::kKvChunkBytes >> 4) + 2 * (kk & 3)), idesc_qk);
                    umma_commit(smem_u32(s_full + (c.gb & 1u)));
                    if (c.j == c.nb - 1) umma_commit(smem_u32(q_empty + qb));   // the tile's queries are no longer needed
                    advance(c);
                }
            } else {
                // O += P V of block gb as soon as its probabilities are in tensor memory
                const uint64_t vdesc0 = umma_desc_mn_sw128(smem_u32(smKV), C::kKvChunkBytes);
                while (ok && c.tile < n_tiles) {
                    if (!mbar_wait(smem_u32(p_full + (c.gb & 1u)), (c.gb >> 1) & 1u, abort_flag)) break;
                    // the first P V of a tile overwrites O: the output of the accumulator's previous tile must have been read
                    if (c.j == 0 && c.k > 0 &&
                        !(kSplit ? mbar_wait(smem_u32(o_free + ((c.k - 1) & 1)), (uint32_t)(((c.k - 1) >> 1) & 1), abort_flag)
                                 : mbar_wait(smem_u32(o_free), (uint32_t)((c.k - 1) & 1), abort_flag)))
                        break;
                    tc_fence_after();
                    const int s = (int)(c.gb % kS);
                    const uint32_t o_tmem = tmem_base + (uint32_t)C::kTmemO;
                    const uint32_t p_tmem = tmem_base + (uint32_t)(C::kTmemP + (c.gb & 1u) * (BN / 2));   // P: 8 columns per 16 keys
                    const uint64_t vd = vdesc0 + (uint64_t)(uint32_t)(s * (C::kKvBytes >> 4));
#pragma unroll
                    for (int kk = 0; kk < BN / 16; ++kk)   // V: 16 keys further = 16 rows x 128 bytes
                        umma_bf16_ts(o_tmem, p_tmem + (uint32_t)(kk * 8), vd + (uint64_t)(kk * (2048 >> 4)), idesc_pv,
                                     (c.j > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(smem_u32(pv_done + (c.gb & 1u)));
                    umma_commit(smem_u32(kv_empty + s));   // Q K^T of the block, the stage's other reader, completed long ago
                    if (c.j == c.nb - 1) umma_commit(smem_u32(o_final + (kSplit ? (c.k & 1) : 0)));
                    advance(c);
                }
            }
        }
        __syncwarp();
    } else if (warp == C::kTmaWarp) {
        // ===================== key/value producer (TMA) =====================
        if (lane == 0) {
            uint32_t gb = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x) {
                const AttTile t = att_tile<BN>(p, tile);
                for (int j = 0; j < t.nb; ++j, ++gb) {
                    const int s = (int)(gb % kS);
                    if (!mbar_wait(smem_u32(kv_empty + s), ((gb / kS) & 1u) ^ 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    mbar_expect_tx(smem_u32(kv_full + s), (uint32_t)C::kKvBytes);
#pragma unroll
                    for (int c = 0; c < C::kQChunks; ++c)
                        tma_load_3d(smem_u32(smKV + s * C::kKvBytes + c * C::kKvChunkBytes), &tmapS, smem_u32(kv_full + s), c * 64,
                                    t.key0 + j * BN, t.slot);
                }
            }
        }
        __syncwarp();
    } else if (kSplit && warp >= C::kEpiWarp0) {
        // ===================== output of finished tiles (d = 128: 128 threads) =====================
        const int wq = warp & 3;   // the quarter of the tensor-memory lanes this warp may read
        int k = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++k) {
            const AttTile t = att_tile<BN>(p, tile);
            const int b = k & 1;
            const uint32_t parity = (uint32_t)((k >> 1) & 1);
            if (!mbar_wait(smem_u32(l_ready + b), parity, abort_flag)) break;
            float l_sum = 0.f;
#pragma unroll
            for (int h = 0; h < C::kHalves; ++h) l_sum += l_s[(b * C::kHalves + h) * 128 + wq * 32 + lane];
            if (!mbar_wait(smem_u32(o_final + b), parity, abort_flag)) break;
            tc_fence_after();
            tile_epilogue(k, t, l_sum, wq, lane);
        }
        if (lane == 0) bulk_wait<0>();   // all tile stores of this warp have reached global memory
    } else if (warp == C::kGatherWarp) {
        // ===================== query gather (32 threads) =====================
        // 8 threads per row (16 bytes each per 128-byte chunk), rows lane / 8 + 4 i, 128B-swizzled K-major chunks
        const int sub = lane & 7, r0 = lane >> 3;
        int k = 1;
        for (int tile = blockIdx.x + gridDim.x; tile < n_tiles; tile += gridDim.x, ++k) {
            const int qb = k % kQB;
            // the buffer's previous tenant is tile k - kQB (the first tile, tenant of buffer 0, included)
            if (k >= kQB && !mbar_wait(smem_u32(q_empty + qb), (uint32_t)(((k - kQB) / kQB) & 1), abort_flag)) break;
            const AttTile t = att_tile<BN>(p, tile);
            unsigned char *q = smQ + qb * C::kQBytes;
            // the tile's 128 ids with four coalesced loads per lane (rows lane, lane + 32, ...); -1 = zero row
            int idv[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int r = lane + 32 * u;
                int id = -1;
                if (r < t.cnt) {
                    id = p.sl.ids[t.pos0 + r];
                    if (id < 0 || (int64_t)id >= p.M) id = -1;
                }
                idv[u] = id;
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int r = r0 + 4 * i;                                   // row r: register r / 32 of lane r % 32
                const int id = __shfl_sync(0xffffffffu, idv[i >> 3], r0 + 4 * (i & 7));
                const uint8_t *g = p.E + (id >= 0 ? (size_t)id * (D * 2) + sub * 16 : 0);
                const uint32_t dst = smem_u32(q) + (uint32_t)(r * 128) + (uint32_t)((sub ^ (r & 7)) << 4);
#pragma unroll
                for (int c = 0; c < C::kQChunks; ++c) cp_async16(dst + c * 16384, g + c * 128, id >= 0 ? 16u : 0u);
            }
            cp_async_arrive_noinc(smem_u32(q_full + qb));
        }
        cp_async_wait_all();
    }

    if (*abort_flag) {
        if (tid == 0) atomicOr(p.sl.status, AIF_STATUS_TIMEOUT);
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == C::kMmaWarp) tmem_dealloc(tmem_base, 512);
}

struct AttPlan {
    CUtensorMap tmap;
    CUtensorMap tmap_g;                   // categories on: over the grouped sequences
    int bn = 0;
    __nv_bfloat16 *self_rows = nullptr;   // [L_max + 128][d]: attention rows of eq. 2 for the user state being computed
    int32_t *iota = nullptr;              // 0, 1, 2, ...: the "candidate ids" of that launch are the sequence positions
};

__global__ void k_iota(int32_t *out, int n)
{
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) out[i] = i;
}

}  // namespace

bool tc_att_supported(const aif_config &c)
{
    return c.dtype == AIF_BF16 && (c.blocks & AIF_BLK_ATT) && (c.d == 128 || c.d == 256) && encode_fn() != nullptr;
}

// Tensor map over the S regions of all user-state slots: [n_slots][L_max][d] with the slot stride of the arena.
cudaError_t tc_att_prepare(aif_ctx *ctx)
{
    const aif_config &c = ctx->cfg;
    AttPlan *pl = new AttPlan();
    ctx->tc_att_plan = pl;
    pl->bn = c.d == 128 ? 128 : 64;
    EncodeFn enc = encode_fn();
    if (!enc) return cudaErrorNotSupported;
    const cuuint64_t dims[3] = {(cuuint64_t)c.d, (cuuint64_t)c.L_max, (cuuint64_t)c.max_user_states};
    const cuuint64_t strides[2] = {(cuuint64_t)c.d * 2, (cuuint64_t)ctx->slot_bytes};
    const cuuint32_t box[3] = {64, (cuuint32_t)pl->bn, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    void *base = const_cast<void *>(ctx->slots[0].dev.S);
    CUresult r = enc(&pl->tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    if (c.n_categories > 0) {
        const cuuint64_t gdims[3] = {(cuuint64_t)c.d, (cuuint64_t)ctx->grouped_rows, (cuuint64_t)c.max_user_states};
        r = enc(&pl->tmap_g, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ctx->slots[0].dev.Sg), gdims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    cudaError_t e;
    {   // scratch of the user-side self-attention
        const size_t rows = (size_t)c.L_max + kTcTile;
        void *ptr = nullptr;
        if ((e = cudaMalloc(&ptr, rows * c.d * 2)) != cudaSuccess) return e;
        ctx->allocations.push_back(ptr), ctx->device_bytes += (int64_t)(rows * c.d * 2);
        pl->self_rows = static_cast<__nv_bfloat16 *>(ptr);
        if ((e = cudaMemset(ptr, 0, rows * c.d * 2)) != cudaSuccess) return e;
        if ((e = cudaMalloc(&ptr, rows * 4)) != cudaSuccess) return e;
        ctx->allocations.push_back(ptr), ctx->device_bytes += (int64_t)(rows * 4);
        pl->iota = static_cast<int32_t *>(ptr);
        k_iota<<<64, 256>>>(pl->iota, (int)rows);
        count_launch();
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    if (c.d == 128)
        e = cudaFuncSetAttribute(k_att_tc<128, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AttCfg<128, 128>::kSmem);
    else
        e = cudaFuncSetAttribute(k_att_tc<256, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AttCfg<256, 64>::kSmem);
    return e;
}

const void *tc_att_tmap(const aif_ctx *ctx) { return &reinterpret_cast<const AttPlan *>(ctx->tc_att_plan)->tmap; }

void tc_att_destroy(aif_ctx *ctx)
{
    delete reinterpret_cast<AttPlan *>(ctx->tc_att_plan);
    ctx->tc_att_plan = nullptr;
}

// Rows a user state's S must have zeroed beyond L so that the last key block reads no stale values.
int tc_att_key_block(const aif_ctx *ctx)
{
    const AttPlan *pl = reinterpret_cast<const AttPlan *>(ctx->tc_att_plan);
    return pl ? pl->bn : 0;
}

// Store target of the attention rows: X as a [rows x x_stride] bf16 tensor, 32 x 32 boxes, 64-byte swizzle.
static cudaError_t encode_x_map(CUtensorMap *m, void *X, int x_stride, size_t rows)
{
    const cuuint64_t dims[2] = {(cuuint64_t)x_stride, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)x_stride * 2};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                             CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t launch_att_tc(const aif_ctx *ctx, const ScoreLaunch &sl, cudaStream_t st, void *X, int x_stride, size_t x_rows)
{
    const aif_config &c = ctx->cfg;
    const AttPlan *pl = reinterpret_cast<const AttPlan *>(ctx->tc_att_plan);
    CUtensorMap tmap_x;
    cudaError_t ex = encode_x_map(&tmap_x, X, x_stride, x_rows);
    if (ex != cudaSuccess) return ex;
    AttParams p{};
    p.sl = sl, p.E = (const uint8_t *)ctx->E, p.M = c.M, p.mini_batch = c.mini_batch;
    p.x_stride = x_stride, p.X = (__nv_bfloat16 *)X;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)c.d);
    p.q_norm = ctx->e_norm;
    // One CTA per SM walking over its tiles hides a tile's query gather and output behind its neighbours' key blocks:
    // 22 k against 31 k cycles per 8-block tile, which outweighs the static assignment's rounding (8.5 tiles per SM cost
    // 9 tile times) as soon as some SM has two tiles.
    const int grid = sl.n_tiles > 148 ? 148 : sl.n_tiles;
    cudaError_t e;
    const CUtensorMap &tm = sl.grouped ? pl->tmap_g : pl->tmap;
    if (c.d == 128)
        e = launch_pdl(k_att_tc<128, 128>, dim3(grid), dim3(AttCfg<128, 128>::kThreads), AttCfg<128, 128>::kSmem, st, tm, tmap_x, p);
    else
        e = launch_pdl(k_att_tc<256, 64>, dim3(grid), dim3(AttCfg<256, 64>::kThreads), AttCfg<256, 64>::kSmem, st, tm, tmap_x, p);
    count_launch();
    return e;
}

cudaError_t launch_self_att_tc(const aif_ctx *ctx, int slot_index, int L, cudaStream_t st, const void **rows_out)
{
    const aif_config &c = ctx->cfg;
    const AttPlan *pl = reinterpret_cast<const AttPlan *>(ctx->tc_att_plan);
    ScoreLaunch sl{};
    sl.slots = ctx->slots_dev, sl.reqs = nullptr, sl.n_req = 1;
    sl.single = ReqDev{slot_index, L, 0, 0, 0};
    sl.n_tiles = (L + kTcTile - 1) / kTcTile, sl.total = L, sl.max_L = L;
    sl.ids = pl->iota, sl.logits = nullptr, sl.status = ctx->status;
    AttParams p{};
    p.sl = sl, p.E = reinterpret_cast<const uint8_t *>(ctx->slots[(size_t)slot_index].dev.S), p.M = L, p.mini_batch = 0;
    p.x_stride = c.d, p.X = pl->self_rows;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)c.d);
    p.q_norm = ctx->slots[(size_t)slot_index].dev.k_norm;   // the queries are the sequence rows themselves
    CUtensorMap tmap_x;
    cudaError_t ex = encode_x_map(&tmap_x, pl->self_rows, c.d, (size_t)c.L_max + kTcTile);
    if (ex != cudaSuccess) return ex;
    const int grid = sl.n_tiles > 148 ? 148 : sl.n_tiles;
    cudaError_t e;
    if (c.d == 128)
        e = launch_pdl(k_att_tc<128, 128>, dim3(grid), dim3(AttCfg<128, 128>::kThreads), AttCfg<128, 128>::kSmem, st, pl->tmap, tmap_x, p);
    else
        e = launch_pdl(k_att_tc<256, 64>, dim3(grid), dim3(AttCfg<256, 64>::kThreads), AttCfg<256, 64>::kSmem, st, pl->tmap, tmap_x, p);
    count_launch();
    *rows_out = pl->self_rows;
    return e;
}

}  // namespace aif
