// LSH similarity, LSH-DIN and SimTier on the tensor cores (sm_100a; Section 4.2, eqs. 6-9) for tiles of 128 candidates
// against the request's behaviour sequence.
//
// eq. 6 counts the signature bits on which a candidate and a sequence item agree.  With every bit written as +1 / -1 the
// dot product of two signatures is matches - mismatches = 2 matches - d', so the whole match-count matrix of a tile
// against a key block is one [128 x d'] . [d' x BN] product of +-1 operands (fp8 E4M3, exact in fp32 accumulation): the
// xor + population count per pair becomes tensor work at twice the bf16 rate, and what is left for the CUDA cores per pair
// is one conversion and the tier bookkeeping.  eq. 8 is then the [128 x BN] . [BN x d] product of those counts (2 matches,
// exact in bf16 up to 512) with the projected sequence, accumulated in fp32 over the key blocks; the factor 1 / (2 d')
// (and 1 / L for the mean form) is applied once, when the tile's rows are written.  eq. 9's histogram is counted from the
// same scores in integer arithmetic, tier = min(N - 1, floor(matches N / d')), exactly as the definition has it.
//
// The +-1 form of the sequence signatures is written once per user state (k_expand_signatures, user side); the +-1 form
// of a tile's item signatures is built in shared memory by the CTA that scores the tile.
//
// One CTA per SM walks over the tiles blockIdx.x, blockIdx.x + gridDim.x, ...  Warps at d = 128 (512 threads; d = 256 in
// brackets, 256 threads):
//   0-7 [0-3]  per key block: read the score row from tensor memory, write 2 matches as packed bf16 pairs into the P
//              buffer (A operand of the second product, never in shared memory), count the tiers.  A thread owns a
//              candidate row; at d = 128 two warps share each quarter of the rows and take alternate key blocks.  At the
//              end of a tile the SimTier columns are written.
//   8  [4]     allocates tensor memory; one lane issues the signature products, up to two blocks ahead
//   9  [5]     one lane streams the key blocks with TMA, the +-1 signatures (ahead) and the rows of S through rings of their own
//   10 [6]     expands the item signatures of the next tile into one of two operand buffers
//   11 [7]     one lane issues O += P S
//   12-15      d = 128 only: scale the finished tile's O accumulator and store the LSH-DIN rows while the other warps are
//              on the next tile's first blocks
// Tensor memory: two score buffers, two P buffers, one O accumulator.  P has columns of its own, so that the signature
// product of block j + 2 waits only until the scores of block j are in registers and not for the product that reads P_j:
// with P written over the scores, a block's period was the sum of both products, both conversions' latencies and four
// barrier round trips, divided by two buffers (1470 cycles per 128-key block at d = 128 with next to no conversion work).
// Every wait is bounded.
#include "aif_device.cuh"
#include "aif_internal.h"
#include "aif_tc_ptx.cuh"

namespace aif {
namespace {

constexpr int kTierSlots = 16;   // n_tiers <= 16

struct LshParams {
    ScoreLaunch sl;
    const uint8_t *sig;      // item signatures [M x D / 8], first bit = most significant bit of byte 0
    int64_t M;
    int32_t mini_batch;
    int32_t x_stride;        // elements per row of X
    int32_t x_din;           // first LSH-DIN column of X, or -1: block off
    int32_t x_tier;          // first SimTier column of X (64 columns, the first n_tiers used), or -1
    int32_t n_tiers;
    int32_t din_mean, tier_mean;   // divide by the sequence length
    __nv_bfloat16 *X;
};

template <int D, int BN>
struct LshCfg {
    static constexpr int kQChunks = D / 128;             // 128-byte chunks of a +-1 signature row (one byte per bit)
    static constexpr int kQBytes = kQChunks * 128 * 128;
    static constexpr int kQBufs = 2;
    // key blocks arrive through two rings: the +-1 signatures (needed two blocks ahead, by the first product) and the rows
    // of S (needed by the second product, and held until it completes)
    static constexpr int kStagesG = D <= 128 ? 4 : 3, kStagesV = 3;
    static constexpr int kVChunks = D / 64;              // 64-column (128-byte) chunks of a row of S
    static constexpr int kVChunkBytes = BN * 128;
    static constexpr int kVBytes = kVChunks * kVChunkBytes;
    static constexpr int kGChunkBytes = BN * 128;        // one 128-bit chunk of a key block's signatures
    static constexpr int kGBytes = kQChunks * kGChunkBytes;
    // tensor memory: two score buffers, two P buffers of their own (BN / 2 columns of packed bf16 pairs each: the next
    // signature product only waits until the scores are in registers, not for the product that reads P), one O accumulator
    static constexpr int kTmemP = 2 * BN;
    static constexpr int kTmemO = D <= 128 ? 384 : 256;
    static_assert(kTmemP + BN <= kTmemO && kTmemO + D <= 512, "tensor memory");
    static constexpr bool kSplitEpi = D <= 128;
    static constexpr int kHalves = D <= 128 ? 2 : 1;
    static constexpr int kConvWarps = 4 * kHalves;
    static constexpr int kMmaWarp = kConvWarps, kTmaWarp = kConvWarps + 1, kGatherWarp = kConvWarps + 2, kPvWarp = kConvWarps + 3;
    static constexpr int kEpiWarp0 = kConvWarps + 4;
    static constexpr int kThreads = (kConvWarps + 4 + (kSplitEpi ? 4 : 0)) * 32;
    // tier counters [tile parity][half][tier][row] (two parities only where two warps share a row)
    static constexpr int kTierBufs = kHalves == 2 ? 2 : 1;
    static constexpr int kTierBytes = kTierBufs * kHalves * kTierSlots * 128 * 4;
    static constexpr size_t kSmem = 1024 + kQBufs * kQBytes + kStagesG * kGBytes + kStagesV * kVBytes + 512 + kTierBytes;
    static_assert(kSmem <= 227 * 1024, "shared memory");
    static_assert(kQBytes >= 16384, "output staging lives in the signature buffer");
};

struct LshTile {
    int slot, cnt, nb, L;
    int key0;   // first key row: 0, or where the tile's category's sub-sequence begins in the grouped sequence
    int64_t pos0;
};

template <int BN>
__device__ __forceinline__ LshTile lsh_tile(const LshParams &p, int tile)
{
    LshTile t;
    if (p.sl.tiles) {
        const int4 v = *reinterpret_cast<const int4 *>(p.sl.tiles + tile);
        t.slot = v.x, t.cnt = v.y;
        t.pos0 = ((int64_t)(uint32_t)v.w << 32) | (int64_t)(uint32_t)v.z;
        t.L = p.sl.tiles[tile].L, t.key0 = p.sl.tiles[tile].key0;
        // an empty sub-sequence still walks one key block (its outputs are forced to zero): the hand-overs stay the same
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

// Sixteen signature bits (two bytes, first bit = most significant bit of b0) as sixteen E4M3 bytes: +1.0 (0x38) for a set
// bit, -1.0 (0xB8) for a clear one.
__device__ __forceinline__ uint4 expand16(uint32_t b0, uint32_t b1)
{
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t nib = ~((i < 2 ? b0 : b1) >> (4 - 4 * (i & 1))) & 0xFu;   // inverted bits 4 i .. 4 i + 3, first one in bit 3
        w[i] = 0x38383838u | ((nib & 8u) << 4) | ((nib & 4u) << 13) | ((nib & 2u) << 22) | ((nib & 1u) << 31);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}

// A chunk of a candidate row's scores against a key block: 32 scores (2 matches - d', exact integers in fp32) -> P = 2 matches as packed
// bf16 pairs, and the tier counts in 8-bit counters (tier t in byte t & 3 of cnt[t >> 2]), 32 keys at a time.
//
// Tier of a pair (eq. 9, equal-width tiers, the last one closed): n = floor(matches N / d').  d' is a power of two here, so
// 2 matches * (N / 2 d') is exact in fp32 and a fused multiply-add that rounds towards minus infinity onto 1.5 * 2^23 leaves
// n in the low mantissa bits (fp32 counts in ones between 2^23 and 2^24).  An integer multiply by 0x1111 copies n into the
// four low nibbles.  Up to eight tiers: adding 0x0123 makes nibble p equal to n + 3 - p, which is 3 exactly where p = n and 7
// where p + 4 = n, never carries (n <= 8) and has bit 3 set (the byte permute's sign-replicating mode: zero for these
// pools) when it is 8 or more; byte permutes with that selector over a pool whose byte 3, or byte 7, is 0x01 yield the
// increments 1 << 8 n of the two packed counters.  More than eight tiers: the nibbles are xor-ed with their positions
// instead (p ^ n is zero only where p = n) and n is capped at 15.  matches = d' gives n = N, one past the last tier: those
// pairs land in no counted slot and the last tier is derived from the total.  The per-thread work here is what bounds
// the kernel (about seven instructions per pair with SimTier on), so every instruction counts.
template <int D, bool TIERS, bool WIDE>
__device__ __forceinline__ void lsh_convert(const uint32_t (&sc)[32], float c1, float n_cap, uint32_t p_col, uint32_t (&cnt)[4])
{
    uint32_t packed[16];
    // the offset and the rounding multiply-add take two scores per instruction (f32x2)
    const uint64_t d2 = pack_f32x2((float)D, (float)D), c2 = pack_f32x2(c1, c1), magic2 = pack_f32x2(12582912.0f, 12582912.0f);
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        const uint64_t pp = add_f32x2(pack_f32x2(__uint_as_float(sc[i]), __uint_as_float(sc[i + 1])), d2);   // 2 matches
        float p0, p1;
        unpack_f32x2(pp, p0, p1);
        if (TIERS) {
            float w0, w1;
            unpack_f32x2(fma_rm_f32x2(pp, c2, magic2), w0, w1);
            if (WIDE) {
                w0 = fminf(w0, n_cap), w1 = fminf(w1, n_cap);
                const uint32_t r0 = __float_as_uint(w0) * 0x1111u, r1 = __float_as_uint(w1) * 0x1111u;
                cnt[0] += prmt(1u, 0u, r0 ^ 0x3210u) + prmt(1u, 0u, r1 ^ 0x3210u);
                cnt[1] += prmt(0u, 1u, r0 ^ 0x3210u) + prmt(0u, 1u, r1 ^ 0x3210u);
                cnt[2] += prmt(1u, 0u, r0 ^ 0xBA98u) + prmt(1u, 0u, r1 ^ 0xBA98u);
                cnt[3] += prmt(0u, 1u, r0 ^ 0xBA98u) + prmt(0u, 1u, r1 ^ 0xBA98u);
            } else {
                const uint32_t s0 = __float_as_uint(w0) * 0x1111u + 0x0123u, s1 = __float_as_uint(w1) * 0x1111u + 0x0123u;
                cnt[0] += prmt(0x01000000u, 0u, s0) + prmt(0x01000000u, 0u, s1);
                cnt[1] += prmt(0u, 0x01000000u, s0) + prmt(0u, 0x01000000u, s1);
            }
        }
        const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
        packed[i >> 1] = *reinterpret_cast<const uint32_t *>(&h);
    }
    tmem_st16(p_col, packed);
}

// One key block of a candidate row: BN scores from the score buffer at s_col -> P at p_col and the packed tier counts,
// 32 columns at a time with the load of the next chunk in flight while one is converted.  Returns after the last load
// has landed and `s_free` has been told so; the stores may still be in flight.
// Columns beyond the sequence need no special case: their signatures and their rows of S are zero (the user side pads
// both to the key block), so they add nothing to O, and their score of 0 (matches = d' / 2) lands in tier floor(N / 2),
// from which the caller takes them out again.
template <int D, int BN, bool TIERS, bool WIDE>
__device__ __forceinline__ void lsh_block(uint32_t s_col, uint32_t p_col, float c1, float n_cap, uint32_t s_free_bar, uint32_t (&cnt)[4])
{
    uint32_t ra[32], rb[32];
    tmem_ld32(s_col, ra);
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += 64) {
        tmem_ld_wait();
        tmem_ld32(s_col + (uint32_t)(c0 + 32), rb);
        lsh_convert<D, TIERS, WIDE>(ra, c1, n_cap, p_col + (uint32_t)(c0 >> 1), cnt);
        tmem_ld_wait();
        if (c0 + 64 < BN) tmem_ld32(s_col + (uint32_t)(c0 + 64), ra);
        else {   // all scores are in registers: the signature product of block gb + 2 may overwrite the buffer
            tc_fence_before();
            mbar_arrive(s_free_bar);
        }
        lsh_convert<D, TIERS, WIDE>(rb, c1, n_cap, p_col + (uint32_t)((c0 + 32) >> 1), cnt);
    }
}

template <int D, int BN>
__global__ void __launch_bounds__((LshCfg<D, BN>::kThreads), 1) k_lsh_tc(const __grid_constant__ CUtensorMap tmapS,
                                                                         const __grid_constant__ CUtensorMap tmapG,
                                                                         const __grid_constant__ CUtensorMap tmapX, const LshParams p)
{
    using C = LshCfg<D, BN>;
    constexpr int kSG = C::kStagesG, kSV = C::kStagesV, kQB = C::kQBufs;
    constexpr bool kSplit = C::kSplitEpi;
    constexpr int kH = C::kHalves;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char *base = reinterpret_cast<unsigned char *>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    unsigned char *smQ = base;
    unsigned char *smV = smQ + kQB * C::kQBytes;
    unsigned char *smG = smV + kSV * C::kVBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smG + kSG * C::kGBytes);
    uint64_t *v_full = bars, *v_empty = bars + kSV, *g_full = v_empty + kSV, *g_empty = g_full + kSG;
    uint64_t *s_full = g_empty + kSG, *p_full = s_full + 2, *pv_done = p_full + 2, *s_free = pv_done + 2;
    uint64_t *q_full = s_free + 2, *q_empty = q_full + 2, *o_final = q_empty + 2, *o_free = o_final + 2;
    uint64_t *q_first = o_free + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(q_first + 1);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    uint32_t *tier_s = reinterpret_cast<uint32_t *>(reinterpret_cast<unsigned char *>(bars) + 512);   // [bufs][halves][16][128]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < kSV; ++s) {
            mbar_init(smem_u32(v_full + s), 1);
            mbar_init(smem_u32(v_empty + s), 1);
        }
        for (int s = 0; s < kSG; ++s) {
            mbar_init(smem_u32(g_full + s), 1);
            mbar_init(smem_u32(g_empty + s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(s_full + b), 1);
            mbar_init(smem_u32(p_full + b), 128);
            mbar_init(smem_u32(pv_done + b), 1);
            mbar_init(smem_u32(s_free + b), 128);
            mbar_init(smem_u32(q_full + b), 32);
            mbar_init(smem_u32(q_empty + b), 5);   // the tenant's last signature product, and the four output warps' staging
            mbar_init(smem_u32(o_final + b), 1);
            mbar_init(smem_u32(o_free + b), 128);
        }
        mbar_init(smem_u32(q_first), C::kConvWarps * 32);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < C::kTierBytes / 4; i += C::kThreads) tier_s[i] = 0u;
    if (warp == C::kMmaWarp) tmem_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    grid_dep_launch();
    grid_dep_wait();

    const int n_tiles = p.sl.n_tiles_dev ? *p.sl.n_tiles_dev : p.sl.n_tiles;

    // A row's item signature as +-1 bytes in the operand layout (128-byte swizzled K-major chunks): 8 threads per row,
    // 16 bits (two signature bytes) each per 128-bit chunk.
    auto expand_row = [&](unsigned char *q, int r, int sub, int id) {
#pragma unroll
        for (int c = 0; c < C::kQChunks; ++c) {
            uint4 v = make_uint4(0u, 0u, 0u, 0u);   // rows beyond the tile and ids outside the table: zeros
            if (id >= 0) {
                const uint32_t two = *reinterpret_cast<const uint16_t *>(p.sig + (size_t)id * (D / 8) + c * 16 + sub * 2);
                v = expand16(two & 0xFFu, two >> 8);
            }
            *reinterpret_cast<uint4 *>(q + c * 16384 + r * 128 + ((sub ^ (r & 7)) << 4)) = v;
        }
    };

    // Scales a finished tile's O accumulator and stores the LSH-DIN rows.  wq = the warp's quarter of the TMEM lanes.
    auto tile_epilogue = [&](int k, const LshTile &t, int wq, int lane) {
        const int row = wq * 32 + lane;
        const uint32_t lane_base = tmem_base + ((uint32_t)(wq * 32) << 16);
        const uint32_t o_col = (uint32_t)C::kTmemO;
        uint64_t *o_free_k = o_free;
        const float scale = (0.5f / (float)D) * (p.din_mean ? 1.0f / (float)t.L : 1.0f);
        bool good = false;
        if (row < t.cnt && t.L > 0) {   // an empty sub-sequence gives zero rows
            const int id = p.sl.ids[t.pos0 + row];
            good = id >= 0 && (int64_t)id < p.M;
        }
        const int qb_out = k % kQB;
        if (p.x_din >= 0) {
            // through staging slabs (2 x 2 KB per warp, 64-byte swizzle) in the tile's own signature buffer and asynchronous
            // tile stores: every signature product of the tile is complete, and the buffer's next tenant waits for these warps
            unsigned char *stg = smQ + qb_out * C::kQBytes + wq * 4096;
            const bool whole = wq * 32 + 32 <= t.cnt;
            uint32_t slab = 0;
            auto emit = [&](const uint32_t (&r)[32], int c0) {
                uint32_t packed[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const __nv_bfloat162 h = __floats2bfloat162_rn(good ? __uint_as_float(r[2 * i]) * scale : 0.f,
                                                                   good ? __uint_as_float(r[2 * i + 1]) * scale : 0.f);
                    packed[i] = *reinterpret_cast<const uint32_t *>(&h);
                }
                if (whole) {
                    unsigned char *sb = stg + slab * 2048;
                    if (lane == 0) bulk_wait_read<1>();
                    __syncwarp();
                    const int swz = (lane >> 1) & 3;
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        *reinterpret_cast<uint4 *>(sb + lane * 64 + ((q ^ swz) << 4)) =
                            make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&tmapX, smem_u32(sb), p.x_din + c0, (int)(t.pos0 + wq * 32));
                        bulk_commit();
                    }
                    slab ^= 1u;
                } else if (row < t.cnt) {
                    uint4 *dst = reinterpret_cast<uint4 *>(p.X + (size_t)(t.pos0 + row) * p.x_stride + p.x_din + c0);
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        dst[q] = make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
                }
            };
            uint32_t ra[32], rb[32];
            tmem_ld32(lane_base + o_col, ra);
#pragma unroll 1
            for (int c0 = 0; c0 < D; c0 += 64) {
                tmem_ld_wait();
                tmem_ld32(lane_base + o_col + (uint32_t)(c0 + 32), rb);
                emit(ra, c0);
                tmem_ld_wait();
                if (c0 + 64 < D) tmem_ld32(lane_base + o_col + (uint32_t)(c0 + 64), ra);
                else {   // O is in registers: the next tile's first product may overwrite the accumulator
                    tc_fence_before();
                    mbar_arrive(smem_u32(o_free_k));
                }
                emit(rb, c0 + 32);
            }
        } else {
            tc_fence_before();
            mbar_arrive(smem_u32(o_free_k));
        }
        if (lane == 0) {
            bulk_wait_read<0>();
            mbar_arrive(smem_u32(q_empty + qb_out));
        }
    };

    if (warp < C::kConvWarps) {
        // ===================== match counts -> P, tiers =====================
        const int wq = warp & 3, half = warp >> 2;
        const int row = wq * 32 + lane;
        const uint32_t lane_base = tmem_base + ((uint32_t)(wq * 32) << 16);
        const bool tiers = p.x_tier >= 0, wide = p.n_tiers > 8;
        // constants of the tier arithmetic (lsh_convert)
        const float tc1 = (float)p.n_tiers / (float)(2 * D), n_cap = 12582912.0f + 15.0f;
        bool ok = true;
        uint32_t gb = 0;
        int k = 0;
        if ((int)blockIdx.x < n_tiles) {
            // the CTA's first tile has nobody to prefetch it: these warps build its signature operand
            const LshTile t = lsh_tile<BN>(p, blockIdx.x);
            const int sub = tid & 7, r0 = tid >> 3;
#pragma unroll
            for (int i = 0; i < 8 / kH; ++i) {
                const int r = r0 + 16 * kH * i;
                int id = -1;
                if (r < t.cnt) {
                    id = p.sl.ids[t.pos0 + r];
                    if (id < 0 || (int64_t)id >= p.M) id = -1;
                }
                expand_row(smQ, r, sub, id);
            }
            fence_proxy_async();   // read by the MMA through the async proxy
            mbar_arrive(smem_u32(q_first));
        }
        for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x, ++k) {
            const LshTile t = lsh_tile<BN>(p, tile);
            const int L = t.L;
            uint32_t *tc = tier_s + (((kH == 2 ? (k & 1) * kH : 0) + half) * kTierSlots) * 128 + row;   // this thread's counters, stride 128
            int n_valid = 0, n_pad = 0;   // keys this thread has counted, and columns beyond the sequence it has converted
            for (int j = 0; j < t.nb; ++j, ++gb) {
                // d = 128: the two warps of a row quarter take alternate key blocks (block gb, and with it score and P buffer
                // gb & 1, belongs to warp half gb & 1), so that one converts while the other sits in its waits
                if (kH == 2 && (int)(gb & 1u) != half) continue;
                const int b = (int)(gb & 1u);
                const int vc = min(BN, L - j * BN);   // keys of the block that exist
                if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(s_full + b), (gb >> 1) & 1u, abort_flag))) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                // P buffer b was last read by the product of block gb - 2
                if (gb >= 2 && !__all_sync(0xffffffffu, mbar_wait(smem_u32(pv_done + b), ((gb - 2) >> 1) & 1u, abort_flag))) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t s_col = lane_base + (uint32_t)(b * BN), p_col = lane_base + (uint32_t)(C::kTmemP + b * (BN / 2));
                uint32_t cnt[4] = {0u, 0u, 0u, 0u};
                if (!tiers) lsh_block<D, BN, false, false>(s_col, p_col, tc1, n_cap, smem_u32(s_free + b), cnt);
                else if (!wide) lsh_block<D, BN, true, false>(s_col, p_col, tc1, n_cap, smem_u32(s_free + b), cnt);
                else lsh_block<D, BN, true, true>(s_col, p_col, tc1, n_cap, smem_u32(s_free + b), cnt);
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(smem_u32(p_full + b));
                n_valid += vc, n_pad += BN - vc;
                // the block's packed counts (at most 128 per slot) into the tile's 32-bit counters
                if (tiers) {
#pragma unroll
                    for (int t4 = 0; t4 < 4; ++t4) {
                        tc[t4 * 128] += (cnt[0] >> (8 * t4)) & 0xFFu;
                        tc[(4 + t4) * 128] += (cnt[1] >> (8 * t4)) & 0xFFu;
                    }
                    if (wide) {
#pragma unroll
                        for (int t4 = 0; t4 < 4; ++t4) {
                            tc[(8 + t4) * 128] += (cnt[2] >> (8 * t4)) & 0xFFu;
                            tc[(12 + t4) * 128] += (cnt[3] >> (8 * t4)) & 0xFFu;
                        }
                    }
                }
            }
            // ---- SimTier columns of the tile (eq. 9): 64 bf16 per row, the first n_tiers used
            if (p.x_tier >= 0) {
                if (kH == 2) {
                    // the two warps of a row quarter meet here once per tile; a failed wait is carried through the barrier so
                    // that both leave together
                    // slot 15 is free (the last tier is derived from the total): this warp's totals for its partner
                    tc[15 * 128] = (uint32_t)n_valid | ((uint32_t)n_pad << 24);
                    if (named_bar_or(1 + wq, 64, !ok)) {
                        ok = false;
                        break;
                    }
                } else if (!ok)
                    break;
                if (half == 0) {
                    uint32_t *tc1 = tc + kTierSlots * 128;   // the partner's counters
                    int total = n_valid, pads = n_pad;
                    if (kH == 2) total += (int)(tc1[15 * 128] & 0xFFFFFFu), pads += (int)(tc1[15 * 128] >> 24);
                    bool good = false;
                    if (row < t.cnt && L > 0) {
                        const int id = p.sl.ids[t.pos0 + row];
                        good = id >= 0 && (int64_t)id < p.M;
                    }
                    const float nrm = p.tier_mean ? 1.0f / (float)L : 1.0f;
                    uint32_t outw[32];
                    int below = 0;
                    float prev = 0.f;
#pragma unroll
                    for (int tt = 0; tt < 16; ++tt) {
                        int cnt_t = (int)tc[tt * 128] + (kH == 2 ? (int)tc1[tt * 128] : 0);
                        tc[tt * 128] = 0u;
                        if (kH == 2) tc1[tt * 128] = 0u;
                        if (tt == (p.n_tiers >> 1)) cnt_t -= pads;        // columns beyond the sequence scored 0: matches = d' / 2
                        if (tt == p.n_tiers - 1) cnt_t = total - below;   // the closed last tier takes matches = d' as well
                        below += cnt_t;
                        const float v = (good && tt < p.n_tiers) ? (float)cnt_t * nrm : 0.f;
                        if (tt & 1) {
                            const __nv_bfloat162 h = __floats2bfloat162_rn(prev, v);
                            outw[tt >> 1] = *reinterpret_cast<const uint32_t *>(&h);
                        } else
                            prev = v;
                    }
#pragma unroll
                    for (int i = 8; i < 32; ++i) outw[i] = 0u;
                    if (row < t.cnt) {
                        uint4 *dst = reinterpret_cast<uint4 *>(p.X + (size_t)(t.pos0 + row) * p.x_stride + p.x_tier);
#pragma unroll
                        for (int q = 0; q < 8; ++q) dst[q] = make_uint4(outw[4 * q], outw[4 * q + 1], outw[4 * q + 2], outw[4 * q + 3]);
                    }
                }
            }
            if (!ok) break;
            if (!kSplit) {
                if (!mbar_wait(smem_u32(o_final), (uint32_t)(k & 1), abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                tile_epilogue(k, t, warp, lane);
            }
        }
        if (lane == 0) bulk_wait<0>();
    } else if (warp == C::kMmaWarp || warp == C::kPvWarp) {
        // ===================== MMA issuers =====================
        if (lane == 0) {
            constexpr uint32_t idesc_sig = umma_idesc_e4m3(kTcTile, BN);
            constexpr uint32_t idesc_pv = umma_idesc_bf16_bmn(kTcTile, D);
            struct Cursor {
                int tile, k, j, nb;
                uint32_t gb;
                int nb_next;
            };
            auto blocks_of = [&](int tile) { return tile < n_tiles ? lsh_tile<BN>(p, tile).nb : 0; };
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
                // scores of block gb (2 matches - d') into buffer gb & 1
                const uint64_t qdesc0 = umma_desc_sw128(smem_u32(smQ)), gdesc0 = umma_desc_sw128(smem_u32(smG));
                while (ok && c.tile < n_tiles) {
                    const int qb = c.k % kQB;
                    if (c.j == 0) {
                        ok = c.k == 0 ? mbar_wait(smem_u32(q_first), 0u, abort_flag)
                                      : mbar_wait(smem_u32(q_full + qb), (uint32_t)(((c.k - 1) / kQB) & 1), abort_flag);
                        if (!ok) break;
                    }
                    const int s = (int)(c.gb % kSG);
                    if (!mbar_wait(smem_u32(g_full + s), (c.gb / kSG) & 1u, abort_flag)) break;
                    // the buffer's previous content, the scores of block gb - 2, must have been read
                    if (c.gb >= 2 && !mbar_wait(smem_u32(s_free + (c.gb & 1u)), ((c.gb - 2) >> 1) & 1u, abort_flag)) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + (uint32_t)((c.gb & 1u) * BN);
                    const uint64_t qd = qdesc0 + (uint64_t)(uint32_t)(qb * (C::kQBytes >> 4));
                    const uint64_t gd = gdesc0 + (uint64_t)(uint32_t)(s * (C::kGBytes >> 4));
#pragma unroll
                    for (int kk = 0; kk < D / 32; ++kk)   // K = 32 signature bits per instruction, 32 bytes of a chunk row
                        umma_e4m3(d_tmem, qd + (uint64_t)((kk >> 2) * (16384 >> 4) + 2 * (kk & 3)),
                                  gd + (uint64_t)((kk >> 2) * (C::kGChunkBytes >> 4) + 2 * (kk & 3)), idesc_sig, kk > 0 ? 1u : 0u);
                    umma_commit(smem_u32(s_full + (c.gb & 1u)));
                    umma_commit(smem_u32(g_empty + s));
                    if (c.j == c.nb - 1) umma_commit(smem_u32(q_empty + qb));
                    advance(c);
                }
            } else {
                // O += P S of block gb as soon as its counts are in tensor memory
                const uint64_t vdesc0 = umma_desc_mn_sw128(smem_u32(smV), C::kVChunkBytes);
                while (ok && c.tile < n_tiles) {
                    const int s = (int)(c.gb % kSV);
                    if (!mbar_wait(smem_u32(v_full + s), (c.gb / kSV) & 1u, abort_flag)) break;
                    if (!mbar_wait(smem_u32(p_full + (c.gb & 1u)), (c.gb >> 1) & 1u, abort_flag)) break;
                    // the first product of a tile overwrites O: the previous tile's rows must have been read
                    if (c.j == 0 && c.k > 0 && !mbar_wait(smem_u32(o_free), (uint32_t)((c.k - 1) & 1), abort_flag)) break;
                    tc_fence_after();
                    const uint32_t o_tmem = tmem_base + (uint32_t)C::kTmemO;
                    const uint32_t p_tmem = tmem_base + (uint32_t)(C::kTmemP + (c.gb & 1u) * (BN / 2));
                    const uint64_t vd = vdesc0 + (uint64_t)(uint32_t)(s * (C::kVBytes >> 4));
#pragma unroll
                    for (int kk = 0; kk < BN / 16; ++kk)
                        umma_bf16_ts(o_tmem, p_tmem + (uint32_t)(kk * 8), vd + (uint64_t)(kk * (2048 >> 4)), idesc_pv,
                                     (c.j > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(smem_u32(pv_done + (c.gb & 1u)));
                    umma_commit(smem_u32(v_empty + s));
                    if (c.j == c.nb - 1) umma_commit(smem_u32(o_final));
                    advance(c);
                }
            }
        }
        __syncwarp();
    } else if (warp == C::kTmaWarp) {
        // ===================== key blocks: rows of S and +-1 signatures (TMA) =====================
        if (lane == 0) {
            // two cursors over the same sequence of key blocks: the signature stream runs up to three blocks ahead of the
            // stream of S rows, which is held back by the products that still read its stages
            struct Stream {
                int tile, j, nb, slot, key0;
                uint32_t gb;
            };
            auto open = [&](Stream &c) {
                if (c.tile < n_tiles) {
                    const LshTile t = lsh_tile<BN>(p, c.tile);
                    c.nb = t.nb, c.slot = t.slot, c.key0 = t.key0;
                }
            };
            auto step = [&](Stream &c) {
                ++c.gb;
                if (++c.j == c.nb) {
                    c.j = 0, c.tile += gridDim.x;
                    open(c);
                }
            };
            Stream g{(int)blockIdx.x, 0, 0, 0, 0, 0u}, v{(int)blockIdx.x, 0, 0, 0, 0, 0u};
            open(g), open(v);
            bool ok = true;
            while (ok && v.tile < n_tiles) {
                while (ok && g.tile < n_tiles && g.gb < v.gb + (uint32_t)(kSG - 1)) {
                    const int s = (int)(g.gb % kSG);
                    if (!mbar_wait(smem_u32(g_empty + s), ((g.gb / kSG) & 1u) ^ 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    mbar_expect_tx(smem_u32(g_full + s), (uint32_t)C::kGBytes);
#pragma unroll
                    for (int c = 0; c < C::kQChunks; ++c)
                        tma_load_3d(smem_u32(smG + s * C::kGBytes + c * C::kGChunkBytes), &tmapG, smem_u32(g_full + s), c * 128,
                                    g.key0 + g.j * BN, g.slot);
                    step(g);
                }
                if (!ok) break;
                const int s = (int)(v.gb % kSV);
                if (!mbar_wait(smem_u32(v_empty + s), ((v.gb / kSV) & 1u) ^ 1u, abort_flag)) break;
                mbar_expect_tx(smem_u32(v_full + s), (uint32_t)C::kVBytes);
#pragma unroll
                for (int c = 0; c < C::kVChunks; ++c)
                    tma_load_3d(smem_u32(smV + s * C::kVBytes + c * C::kVChunkBytes), &tmapS, smem_u32(v_full + s), c * 64,
                                v.key0 + v.j * BN, v.slot);
                step(v);
            }
        }
        __syncwarp();
    } else if (kSplit && warp >= C::kEpiWarp0) {
        // ===================== output of finished tiles (d = 128) =====================
        const int wq = warp & 3;
        int k = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++k) {
            const LshTile t = lsh_tile<BN>(p, tile);
            if (!mbar_wait(smem_u32(o_final), (uint32_t)(k & 1), abort_flag)) break;
            tc_fence_after();
            tile_epilogue(k, t, wq, lane);
        }
        if (lane == 0) bulk_wait<0>();
    } else if (warp == C::kGatherWarp) {
        // ===================== signature operand of the next tile (32 threads) =====================
        const int sub = lane & 7, r0 = lane >> 3;
        int k = 1;
        for (int tile = blockIdx.x + gridDim.x; tile < n_tiles; tile += gridDim.x, ++k) {
            const int qb = k % kQB;
            if (k >= kQB && !mbar_wait(smem_u32(q_empty + qb), (uint32_t)(((k - kQB) / kQB) & 1), abort_flag)) break;
            const LshTile t = lsh_tile<BN>(p, tile);
            unsigned char *q = smQ + qb * C::kQBytes;
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
                const int r = r0 + 4 * i;
                const int id = __shfl_sync(0xffffffffu, idv[i >> 3], r0 + 4 * (i & 7));
                expand_row(q, r, sub, id);
            }
            fence_proxy_async();
            mbar_arrive(smem_u32(q_full + qb));
        }
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

// Sequence signatures of a user state as +-1 bytes: out[j][b] = +1.0 (E4M3) where bit b of signature j is set, else -1.0.
__global__ void __launch_bounds__(256) k_expand_signatures(const uint8_t *__restrict__ sig, int L, int bits, uint8_t *__restrict__ out)
{
    const int per_row = bits >> 4;   // 16-bit pieces per signature
    const int64_t total = (int64_t)L * per_row;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t two = *reinterpret_cast<const uint16_t *>(sig + i * 2);
        *reinterpret_cast<uint4 *>(out + i * 16) = expand16(two & 0xFFu, two >> 8);
    }
}

struct LshPlan {
    CUtensorMap tmap_s, tmap_g;
    CUtensorMap tmap_sg, tmap_gg;   // categories on: the same over the grouped sequences
    int bn = 0;
};

}  // namespace

bool tc_lsh_supported(const aif_config &c)
{
    return c.dtype == AIF_BF16 && (c.blocks & (AIF_BLK_LSH_DIN | AIF_BLK_SIMTIER)) && (c.d == 128 || c.d == 256) && c.lsh_bits == c.d &&
           encode_fn() != nullptr;
}

// Tensor maps over the S regions and the +-1 signature regions of all user-state slots.
cudaError_t tc_lsh_prepare(aif_ctx *ctx)
{
    const aif_config &c = ctx->cfg;
    LshPlan *pl = new LshPlan();
    ctx->tc_lsh_plan = pl;
    pl->bn = c.d == 128 ? 128 : 64;
    EncodeFn enc = encode_fn();
    if (!enc) return cudaErrorNotSupported;
    const cuuint32_t estr[3] = {1, 1, 1};
    {
        const cuuint64_t dims[3] = {(cuuint64_t)c.d, (cuuint64_t)c.L_max, (cuuint64_t)c.max_user_states};
        const cuuint64_t strides[2] = {(cuuint64_t)c.d * 2, (cuuint64_t)ctx->slot_bytes};
        const cuuint32_t box[3] = {64, (cuuint32_t)pl->bn, 1};
        if (enc(&pl->tmap_s, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ctx->slots[0].dev.S), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        const cuuint64_t dims[3] = {(cuuint64_t)c.lsh_bits, (cuuint64_t)c.L_max, (cuuint64_t)c.max_user_states};
        const cuuint64_t strides[2] = {(cuuint64_t)c.lsh_bits, (cuuint64_t)ctx->slot_bytes};
        const cuuint32_t box[3] = {128, (cuuint32_t)pl->bn, 1};
        if (enc(&pl->tmap_g, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<uint8_t *>(ctx->slots[0].dev.sigE), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    if (c.n_categories > 0) {
        const cuuint64_t dims[3] = {(cuuint64_t)c.d, (cuuint64_t)ctx->grouped_rows, (cuuint64_t)c.max_user_states};
        const cuuint64_t strides[2] = {(cuuint64_t)c.d * 2, (cuuint64_t)ctx->slot_bytes};
        const cuuint32_t box[3] = {64, (cuuint32_t)pl->bn, 1};
        if (enc(&pl->tmap_sg, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ctx->slots[0].dev.Sg), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
        const cuuint64_t gdims[3] = {(cuuint64_t)c.lsh_bits, (cuuint64_t)ctx->grouped_rows, (cuuint64_t)c.max_user_states};
        const cuuint64_t gstrides[2] = {(cuuint64_t)c.lsh_bits, (cuuint64_t)ctx->slot_bytes};
        const cuuint32_t gbox[3] = {128, (cuuint32_t)pl->bn, 1};
        if (enc(&pl->tmap_gg, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<uint8_t *>(ctx->slots[0].dev.sigEg), gdims, gstrides, gbox, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    if (c.d == 128) return cudaFuncSetAttribute(k_lsh_tc<128, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LshCfg<128, 128>::kSmem);
    return cudaFuncSetAttribute(k_lsh_tc<256, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LshCfg<256, 64>::kSmem);
}

void tc_lsh_destroy(aif_ctx *ctx)
{
    delete reinterpret_cast<LshPlan *>(ctx->tc_lsh_plan);
    ctx->tc_lsh_plan = nullptr;
}

cudaError_t launch_expand_signatures(const aif_ctx *ctx, const uint8_t *sig, int L, uint8_t *out, cudaStream_t st)
{
    const int64_t total = (int64_t)L * (ctx->cfg.lsh_bits >> 4);
    const int grid = (int)((total + 255) / 256 < 592 ? (total + 255) / 256 : 592);
    k_expand_signatures<<<grid, 256, 0, st>>>(sig, L, ctx->cfg.lsh_bits, out);
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    // zero bytes from the sequence's end to the end of its last 128-key block: the kernel relies on a score of exactly 0
    // for the columns beyond the sequence (rows beyond L_max are zero-filled by the tensor map)
    const int L_pad = (L + 127) / 128 * 128 < ctx->cfg.L_max ? (L + 127) / 128 * 128 : ctx->cfg.L_max;
    if (L_pad > L) e = cudaMemsetAsync(out + (size_t)L * ctx->cfg.lsh_bits, 0, (size_t)(L_pad - L) * ctx->cfg.lsh_bits, st);
    return e;
}

// LSH-DIN rows into columns [x_din, x_din + d) and SimTier rows into [x_tier, x_tier + 64) of X; a negative column turns
// that output off.
cudaError_t launch_lsh_tc(const aif_ctx *ctx, const ScoreLaunch &sl, cudaStream_t st, void *X, int x_stride, size_t x_rows, int x_din,
                          int x_tier)
{
    const aif_config &c = ctx->cfg;
    const LshPlan *pl = reinterpret_cast<const LshPlan *>(ctx->tc_lsh_plan);
    CUtensorMap tmap_x;
    {
        const cuuint64_t dims[2] = {(cuuint64_t)x_stride, (cuuint64_t)x_rows};
        const cuuint64_t strides[1] = {(cuuint64_t)x_stride * 2};
        const cuuint32_t box[2] = {32, 32};
        const cuuint32_t estr[2] = {1, 1};
        if (encode_fn()(&tmap_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    LshParams p{};
    p.sl = sl, p.sig = ctx->sig, p.M = c.M, p.mini_batch = c.mini_batch;
    p.x_stride = x_stride, p.x_din = x_din, p.x_tier = x_tier, p.X = (__nv_bfloat16 *)X;
    p.n_tiers = (c.blocks & AIF_BLK_SIMTIER) ? c.n_tiers : 1;
    p.din_mean = c.lsh_din_norm == AIF_NORM_MEAN, p.tier_mean = c.simtier_norm == AIF_NORM_MEAN;
    const int grid = sl.n_tiles > 148 ? 148 : sl.n_tiles;
    cudaError_t e;
    const CUtensorMap &ts = sl.grouped ? pl->tmap_sg : pl->tmap_s, &tg = sl.grouped ? pl->tmap_gg : pl->tmap_g;
    if (c.d == 128)
        e = launch_pdl(k_lsh_tc<128, 128>, dim3(grid), dim3(LshCfg<128, 128>::kThreads), LshCfg<128, 128>::kSmem, st, ts, tg, tmap_x, p);
    else
        e = launch_pdl(k_lsh_tc<256, 64>, dim3(grid), dim3(LshCfg<256, 64>::kThreads), LshCfg<256, 64>::kSmem, st, ts, tg, tmap_x, p);
    count_launch();
    return e;
}

}  // namespace aif
