// Whole scoring pass of one 128-candidate tile in one CTA (sm_100a, bf16 storage): gather, cross-feature
// generation, dense target attention, decomposed first layer, second layer, logit (Section 3.1 "Real-Time
// Prediction Phase", Sections 3.3 and 4.2).  This is the latency form of the kernel chain: a single request of ~10^4
// candidates is fewer tiles than the GPU has SMs, so nothing is gained by spreading a layer over the machine, while
// every separate launch, and every trip of the activations through global memory, lengthens the request.  One launch,
// one CTA per tile, nothing but the logits written.
//
// Shape: d = 128, blocks = attention + cross features, behaviour sequences of at most 256 items, two hidden layers of
// 512 and <= 256 units.  Other shapes and large batches take the kernel-per-layer path.
//
// 448 threads:
//   warps 0-7   two groups of four warps, one thread per candidate row (TMEM lane) in each.  Softmax: group g takes
//               the scores of key block g, writes the probabilities into tensor memory as packed bf16 (A operand of
//               P V) and exchanges its row sums with the other group through shared memory; then it normalises O into
//               the attention chunks of the first layer's input (group g: columns [64 g, 64 g + 64)).  While layer 1
//               runs, the groups build the bias operands in shared memory: both layers' biases (for layer 1 the
//               request's cached user partial p_u) are added by the tensor cores.  Layer-1 epilogue: ReLU on output
//               slice g, bf16 activations written back into tensor memory over accumulator columns already read (A
//               operand of layer 2).  Layer-2 epilogue: ReLU and the dot with w_out, half of the units per group.
//   warp 8      allocates tensor memory; one lane issues every tcgen05.mma
//   warps 9-12  gather the tile's item rows (queries of the attention and first K chunks of layer 1) and, chunk by
//               chunk, its cross-feature rows from the request's pre-cache, with 16-byte cp.async into 128B-swizzled
//               K-major chunks; buckets are hashed one chunk ahead of their use; last, the tile of ones that multiplies
//               the bias operands
//   warp 13     one lane streams key/value blocks, then first- and second-layer weights with TMA
//
// Tensor memory (512 columns): attention uses [0, 256) for the scores of up to two key blocks, [256, 384) for O and
// [384, 512) for the probabilities (packed bf16, 64 columns per key block).  Layer 1 then fills two 256-column
// accumulators [0, 256) and [256, 512); its activations are packed over them into [0, 128) and [384, 512); layer 2
// accumulates into the freed columns [128, 384).
// Shared memory: item tile 32 KB, later the bias operands and the output weights | key/value blocks 64 KB, later the
// attention chunks and two more stages of the cross-feature ring | two cross-feature stages 32 KB | weight ring
// 3 x 32 KB | barriers and the exchange array.
// Every wait is bounded: on expiry the CTA raises AIF_STATUS_TIMEOUT, every role skips its remaining work, tensor
// memory is freed and the kernel returns.
#include <cuda.h>

#include "aif_device.cuh"
#include "aif_internal.h"
#include "aif_tc_ptx.cuh"

namespace aif {
namespace {

constexpr int kFThreads = 448;
constexpr int kFMmaWarp = 8, kFProdWarp0 = 9, kFBWarp = 13;
constexpr int kChunk = 16384;                  // 128 rows x 64 bf16
constexpr int kOffKV = 32768, kOffA01 = 98304, kOffB = 131072, kOffMisc = 229376;
constexpr int kBStage = 32768, kBStages = 3, kAStages = 4;
constexpr size_t kFSmem = 1024 + kOffMisc + 2048;
constexpr int kMaxCross = 8;                   // cross-feature chunks (64 columns each)
constexpr int kH1 = 512;

enum {
    BAR_E_FULL = 0, BAR_KV_FULL, BAR_S_FULL = BAR_KV_FULL + 2, BAR_P_FULL, BAR_O_FINAL, BAR_ATT_FULL, BAR_E_FREE, BAR_ACC1_FULL,
    BAR_H1_FULL, BAR_ACC2_FULL, BAR_BIAS_FULL, BAR_FULL_A, BAR_EMPTY_A = BAR_FULL_A + kAStages, BAR_FULL_B = BAR_EMPTY_A + kAStages,
    BAR_EMPTY_B = BAR_FULL_B + kBStages, BAR_COUNT = BAR_EMPTY_B + kBStages
};
static_assert(BAR_COUNT * 8 + 16 + 2 * 128 * 4 <= 2048, "misc area");

struct FusedParams {
    ScoreLaunch sl;
    const uint8_t *E;
    int64_t M;
    int32_t mini_batch;
    int32_t B, dc, b_mask, bucket_mode, n_cross;
    int32_t H2, emit_sigmoid;
    float scale_log2;       // log2(e) / sqrt(d)
    const __nv_bfloat16 *b2_hl;   // [2][H2]: second-layer bias, high parts then remainders
    const __nv_bfloat16 *w_out;
    const float *b_out;
};

__global__ void __launch_bounds__(kFThreads, 1) k_request_fused(const __grid_constant__ CUtensorMap tmapS,
                                                                const __grid_constant__ CUtensorMap tmapW1,
                                                                const __grid_constant__ CUtensorMap tmapW2, const FusedParams p)
{
    extern __shared__ unsigned char smem_dyn[];
    unsigned char *base = reinterpret_cast<unsigned char *>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    unsigned char *smE = base, *smKV = base + kOffKV, *smAtt = smKV, *smB = base + kOffB;
    uint64_t *bars = reinterpret_cast<uint64_t *>(base + kOffMisc);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + BAR_COUNT);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    float *xs = reinterpret_cast<float *>(tmem_slot + 4);   // [2][128]: row maxima, later row sums, of the two softmax groups
    auto bar = [&](int i) { return smem_u32(bars + i); };
    auto a_stage = [&](int s) { return s < 2 ? base + kOffA01 + s * kChunk : smKV + 32768 + (s - 2) * kChunk; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        mbar_init(bar(BAR_E_FULL), 128);
        mbar_init(bar(BAR_KV_FULL), 1);
        mbar_init(bar(BAR_KV_FULL + 1), 1);
        mbar_init(bar(BAR_S_FULL), 1);
        mbar_init(bar(BAR_P_FULL), 256);
        mbar_init(bar(BAR_O_FINAL), 1);
        mbar_init(bar(BAR_ATT_FULL), 256);
        mbar_init(bar(BAR_E_FREE), 1);
        mbar_init(bar(BAR_ACC1_FULL), 1);
        mbar_init(bar(BAR_H1_FULL), 256);
        mbar_init(bar(BAR_ACC2_FULL), 1);
        mbar_init(bar(BAR_BIAS_FULL), 256);
        for (int s = 0; s < kAStages; ++s) {
            mbar_init(bar(BAR_FULL_A + s), 128);
            mbar_init(bar(BAR_EMPTY_A + s), 1);
        }
        for (int s = 0; s < kBStages; ++s) {
            mbar_init(bar(BAR_FULL_B + s), 1);
            mbar_init(bar(BAR_EMPTY_B + s), 1);
        }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // The gather threads fetch their candidate ids while barriers and tensor memory are being set up: the ids head the
    // longest chain of dependent memory accesses of the kernel (ids -> item rows -> scores).
    int id[8];
    if (warp >= kFProdWarp0 && warp < kFBWarp) {
        grid_dep_wait();
        const ReqDev rq0 = find_request(p.sl, blockIdx.x);
        int start0, cnt0;
        tile_range(blockIdx.x - rq0.tile_begin, rq0.n, kTcTile, p.mini_batch, start0, cnt0);
        const int r0 = (tid - kFProdWarp0 * 32) >> 3;
#pragma unroll
        for (int i = 0; i < 8; ++i) id[i] = r0 + 16 * i < cnt0 ? p.sl.ids[rq0.off + start0 + r0 + 16 * i] : -1;
    }
    if (warp == kFMmaWarp) tmem_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    grid_dep_launch();
    grid_dep_wait();

    // the tile
    const ReqDev rq = find_request(p.sl, blockIdx.x);
    int start, cnt;
    tile_range(blockIdx.x - rq.tile_begin, rq.n, kTcTile, p.mini_batch, start, cnt);
    const int64_t pos0 = rq.off + start;
    const SlotDev *slot = p.sl.slots + rq.slot;
    const int L = slot->L;
    const int nb = L > 128 ? 2 : 1;
    const int n_k1 = 4 + p.n_cross;

    if (warp < 8) {
        // ===================== softmax, epilogues =====================
        const int g = warp >> 2, wq = warp & 3, row = wq * 32 + lane;
        const uint32_t lane_base = tmem_base + ((uint32_t)(wq * 32) << 16);
        const float k2 = p.scale_log2;
        bool ok = true;
        // a wait of the whole warp: the tensor-memory loads and stores that follow need every lane to take the same branch
        auto wait = [&](int b) {
            const bool got = ok && mbar_wait(bar(b), 0u, abort_flag);
            ok = __all_sync(0xffffffffu, got);
        };
        const float b_out = p.b_out[0];
        bool good = false;
        if (row < cnt) {
            const int id = p.sl.ids[pos0 + row];
            good = id >= 0 && (int64_t)id < p.M;
        }
        // ---- attention: scores of key block g -> probabilities
        // Softmax is invariant to the offset subtracted in the exponent, and bf16 keeps its relative precision over the
        // whole fp32 exponent range.  The first attempt therefore subtracts nothing, p = 2^(s k2), and saves the pass
        // over the scores that finds the row maxima; a row sum outside [2^-80, 2^80] (scores far from zero: overflow,
        // or every term flushed to zero) makes the whole CTA repeat the step with the exact row maxima.  The
        // probabilities go to columns of their own, so the scores are still there for the repeat.
        const bool act = g < nb;
        const int valid_cols = L - g * 128 < 128 ? L - g * 128 : 128;
        const uint32_t p_col = 384u + (uint32_t)(g * 64);
        auto probabilities = [&](float mt) {   // P = 2^(s k2 - mt) as packed bf16; returns the row sum over this block
            float lsum = 0.f;
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {
                uint32_t sc[64];
                tmem_ld32(lane_base + (uint32_t)(g * 128 + 64 * h), *reinterpret_cast<uint32_t(*)[32]>(&sc[0]));
                tmem_ld32(lane_base + (uint32_t)(g * 128 + 64 * h + 32), *reinterpret_cast<uint32_t(*)[32]>(&sc[32]));
                tmem_ld_wait();
                uint32_t packed[32];
                float ls4[4] = {0.f, 0.f, 0.f, 0.f};
                const int left = valid_cols - 64 * h;   // valid columns among these 64
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    float p0 = fast_exp2(fmaf(__uint_as_float(sc[2 * i]), k2, -mt));
                    float p1 = fast_exp2(fmaf(__uint_as_float(sc[2 * i + 1]), k2, -mt));
                    if (2 * i >= left) p0 = 0.f;
                    if (2 * i + 1 >= left) p1 = 0.f;
                    ls4[i & 3] += p0 + p1;
                    const __nv_bfloat162 hh = __floats2bfloat162_rn(p0, p1);
                    packed[i] = *reinterpret_cast<const uint32_t *>(&hh);
                }
                tmem_st32(lane_base + p_col + (uint32_t)(32 * h), packed);
                lsum += (ls4[0] + ls4[1]) + (ls4[2] + ls4[3]);
            }
            tmem_st_wait();
            return lsum;
        };
        float lsum = 0.f;
        if (act) {
            wait(BAR_S_FULL);
            tc_fence_after();
            if (ok) lsum = probabilities(0.f);
        }
        xs[g * 128 + row] = lsum;
        const bool off_range = act && ok && !(lsum > 0x1p-80f && lsum < 0x1p80f);
        float l_other;
        if (named_bar_or(1, 256, off_range)) {
            // exact form: row maxima over both key blocks first
            float mx = -INFINITY;
            if (act && ok) {
#pragma unroll 1
                for (int c0 = 0; c0 < 128; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld32(lane_base + (uint32_t)(g * 128 + c0), r);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (c0 + i < valid_cols) mx = fmaxf(mx, __uint_as_float(r[i]));
                }
            }
            xs[g * 128 + row] = mx;
            named_bar_sync(1, 256);
            const float mt = fmaxf(mx, xs[(g ^ 1) * 128 + row]) * k2;   // an inactive group has published -inf
            named_bar_sync(1, 256);                                    // both maxima are read: xs may now take the sums
            lsum = act && ok ? probabilities(mt) : 0.f;
            xs[g * 128 + row] = lsum;
            named_bar_sync(1, 256);
        }
        l_other = xs[(g ^ 1) * 128 + row];
        tc_fence_before();
        mbar_arrive(bar(BAR_P_FULL));
        const float l_all = lsum + l_other;
        // ---- O -> attention chunk g of the first layer's input (64 columns, 128B-swizzled K-major)
        wait(BAR_O_FINAL);
        tc_fence_after();
        if (ok) {
            const float inv = good ? 1.0f / l_all : 0.f;
            unsigned char *dst = smAtt + g * kChunk + row * 128;
#pragma unroll 1
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(lane_base + (uint32_t)(256 + 64 * g + c0), r);
                tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint32_t w[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(r[8 * q + 2 * i]) * inv,
                                                                        __uint_as_float(r[8 * q + 2 * i + 1]) * inv);
                        w[i] = *reinterpret_cast<const uint32_t *>(&hh);
                    }
                    const int slot16 = (c0 >> 3) + q;
                    *reinterpret_cast<uint4 *>(dst + ((slot16 ^ (row & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        }
        fence_proxy_async();   // the MMA reads these chunks through the async proxy
        tc_fence_before();
        mbar_arrive(bar(BAR_ATT_FULL));
        // ---- bias operands into the item tile's memory once layer 1 has consumed it.  The biases are added by the
        // tensor cores: one more K step whose A operand is a tile of ones in columns 0 and 1 and whose B operand holds,
        // per output unit, the bias split into two bf16 values (high part, remainder) in K rows 0 and 1 (fp32
        // accumulation restores the bias to about 2^-17 of its magnitude).  Reading biases from shared memory in the
        // epilogue would cost one shared-memory cycle per element and warp, more than everything else there.
        // Layout: MN-major 128B-swizzled groups of 64 units x 16 K rows (2 KB each): layer 1 at smE, layer 2 behind it.
        wait(BAR_E_FREE);
        __nv_bfloat16 *wout_s = reinterpret_cast<__nv_bfloat16 *>(smE + 24576);
        float *dot_s = reinterpret_cast<float *>(smE + 25600);
        {
            const int t = warp * 32 + lane;
            const uint4 *hl1 = reinterpret_cast<const uint4 *>(slot->pu_hl);   // [2][512] bf16
            const uint4 *hl2 = reinterpret_cast<const uint4 *>(p.b2_hl);       // [2][H2] bf16
            const int n1 = kH1 / 64 * 128, n2 = p.H2 / 64 * 128;              // 16-byte slots of the two operands
            for (int sidx = t; sidx < n1 + n2; sidx += 256) {
                const bool second = sidx >= n1;
                const int q = second ? sidx - n1 : sidx;
                const int grp = q >> 7, k = (q >> 3) & 15, j = (q & 7) ^ (k & 7);
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (k < 2) v = second ? hl2[(k * p.H2 + grp * 64 + j * 8) >> 3] : hl1[(k * kH1 + grp * 64 + j * 8) >> 3];
                *reinterpret_cast<uint4 *>(smE + (second ? 16384 : 0) + q * 16) = v;
            }
            if (t < p.H2 / 8) reinterpret_cast<uint4 *>(wout_s)[t] = reinterpret_cast<const uint4 *>(p.w_out)[t];
        }
        fence_proxy_async();
        mbar_arrive(bar(BAR_BIAS_FULL));
        named_bar_sync(1, 256);
        // ---- layer-1 epilogue: slice g, ReLU, 32 accumulator columns -> 16 columns of packed bf16, over accumulator
        // columns already read; the load of the next chunk is in flight meanwhile
        wait(BAR_ACC1_FULL);
        tc_fence_after();
        if (ok) {
            uint32_t ra[32], rb[32];
            const uint32_t col0 = lane_base + (uint32_t)(g * 256);
            auto finish = [&](const uint32_t (&r)[32], int c) {
                uint32_t packed[16];
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                    const __nv_bfloat162 h0 = __floats2bfloat162_rn(fmaxf(__uint_as_float(r[2 * q]), 0.f), fmaxf(__uint_as_float(r[2 * q + 1]), 0.f));
                    packed[q] = *reinterpret_cast<const uint32_t *>(&h0);
                }
                tmem_st16(lane_base + (uint32_t)((g ? 384 : 0) + 16 * c), packed);
            };
            // slice 0 is read upwards and packed into [0, 128), slice 1 downwards and packed into [384, 512): either way
            // a packed piece lands on columns that have been read, and the 256 columns in between become free
            auto chunk_of = [&](int i) { return g ? 7 - i : i; };
            tmem_ld32(col0 + (uint32_t)(32 * chunk_of(0)), ra);
#pragma unroll 1
            for (int i = 0; i < 8; i += 2) {
                tmem_ld_wait();
                tmem_ld32(col0 + (uint32_t)(32 * chunk_of(i + 1)), rb);
                finish(ra, chunk_of(i));
                tmem_ld_wait();
                if (i + 2 < 8) tmem_ld32(col0 + (uint32_t)(32 * chunk_of(i + 2)), ra);
                finish(rb, chunk_of(i + 1));
            }
            tmem_st_wait();
        }
        tc_fence_before();
        mbar_arrive(bar(BAR_H1_FULL));
        // ---- layer-2 epilogue: half g of the units, ReLU, reduced against w_out
        wait(BAR_ACC2_FULL);
        tc_fence_after();
        float dot = 0.f;
        if (ok) {
            const int hn = p.H2 >> 1;
            const uint32_t col0 = lane_base + 128u + (uint32_t)(g * hn);
            float d4[4] = {0.f, 0.f, 0.f, 0.f};
            uint32_t ra[32], rb[32];
            auto reduce = [&](const uint32_t (&r)[32], int c0) {
                const uint4 *w8 = reinterpret_cast<const uint4 *>(wout_s + g * hn + c0);   // eight bf16 weights per load
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint4 ww = w8[q];
                    const float2 w0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&ww.x));
                    const float2 w1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&ww.y));
                    const float2 w2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&ww.z));
                    const float2 w3 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&ww.w));
                    d4[0] = fmaf(fmaxf(__uint_as_float(r[8 * q]), 0.f), w0.x, d4[0]);
                    d4[1] = fmaf(fmaxf(__uint_as_float(r[8 * q + 1]), 0.f), w0.y, d4[1]);
                    d4[2] = fmaf(fmaxf(__uint_as_float(r[8 * q + 2]), 0.f), w1.x, d4[2]);
                    d4[3] = fmaf(fmaxf(__uint_as_float(r[8 * q + 3]), 0.f), w1.y, d4[3]);
                    d4[0] = fmaf(fmaxf(__uint_as_float(r[8 * q + 4]), 0.f), w2.x, d4[0]);
                    d4[1] = fmaf(fmaxf(__uint_as_float(r[8 * q + 5]), 0.f), w2.y, d4[1]);
                    d4[2] = fmaf(fmaxf(__uint_as_float(r[8 * q + 6]), 0.f), w3.x, d4[2]);
                    d4[3] = fmaf(fmaxf(__uint_as_float(r[8 * q + 7]), 0.f), w3.y, d4[3]);
                }
            };
            tmem_ld32(col0, ra);
#pragma unroll 1
            for (int c0 = 0; c0 < hn; c0 += 64) {   // hn is a multiple of 32
                tmem_ld_wait();
                if (c0 + 32 < hn) tmem_ld32(col0 + (uint32_t)(c0 + 32), rb);
                reduce(ra, c0);
                if (c0 + 32 < hn) {
                    tmem_ld_wait();
                    if (c0 + 64 < hn) tmem_ld32(col0 + (uint32_t)(c0 + 64), ra);
                    reduce(rb, c0 + 32);
                }
            }
            dot = (d4[0] + d4[1]) + (d4[2] + d4[3]);
        }
        if (g == 1) dot_s[row] = dot;
        const bool all_ok = !named_bar_or(1, 256, !ok);   // also orders dot_s; a wait that ran out anywhere in these warps
        if (g == 0 && row < cnt) {
            float logit = dot + dot_s[row] + b_out;
            if (p.emit_sigmoid) logit = 1.0f / (1.0f + expf(-logit));
            if (!good || !all_ok) logit = __int_as_float(0x7fc00000);   // no number for a bad id, nor for a tile whose wait ran out
            p.sl.logits[pos0 + row] = logit;
        }
    } else if (warp == kFMmaWarp) {
        // ===================== MMA issuer =====================
        if (lane == 0) {
            constexpr uint32_t idesc_qk = umma_idesc_bf16(kTcTile, 128);
            constexpr uint32_t idesc_pv = umma_idesc_bf16_bmn(kTcTile, 128);
            constexpr uint32_t idesc1 = umma_idesc_bf16(kTcTile, 256);
            const uint32_t idesc2 = umma_idesc_bf16(kTcTile, p.H2);
            bool ok = mbar_wait(bar(BAR_E_FULL), 0u, abort_flag);
            fence_proxy_async();   // the item rows were written by cp.async
            // scores = Q K^T, one key block after the other
            const uint64_t qd = umma_desc_sw128(smem_u32(smE));
            for (int j = 0; ok && j < nb; ++j) {
                ok = mbar_wait(bar(BAR_KV_FULL + j), 0u, abort_flag);
                tc_fence_after();
                if (!ok) break;
                const uint64_t kd = umma_desc_sw128(smem_u32(smKV + j * 32768));
                const uint32_t d_tmem = tmem_base + (uint32_t)(j * 128);
                umma_bf16(d_tmem, qd, kd, idesc_qk, 0u);
#pragma unroll
                for (int kk = 1; kk < 8; ++kk) {
                    const uint64_t o = (uint64_t)((kk >> 2) * (kChunk >> 4) + 2 * (kk & 3));
                    umma_bf16_acc(d_tmem, qd + o, kd + o, idesc_qk);
                }
            }
            if (ok) umma_commit(bar(BAR_S_FULL));
            // O = P V: the probabilities from tensor memory, V = the key blocks read MN-major
            ok = ok && mbar_wait(bar(BAR_P_FULL), 0u, abort_flag);
            tc_fence_after();
            if (ok) {
                for (int j = 0; j < nb; ++j) {
                    const uint64_t vd = umma_desc_mn_sw128(smem_u32(smKV + j * 32768), kChunk);
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        umma_bf16_ts(tmem_base + 256u, tmem_base + (uint32_t)(384 + j * 64 + kk * 8), vd + (uint64_t)(kk * (2048 >> 4)), idesc_pv,
                                     (j > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(bar(BAR_O_FINAL));
            }
            // layer 1: K chunks [ item 0-1 | attention 2-3 | cross 4.. ], two 256-column output slices per chunk
            ok = ok && mbar_wait(bar(BAR_ATT_FULL), 0u, abort_flag);
            tc_fence_after();
            int qb = 0;
            for (int kc = 0; ok && kc < n_k1; ++kc) {
                uint64_t ad;
                int sa = -1;
                if (kc < 2) ad = umma_desc_sw128(smem_u32(smE + kc * kChunk));
                else if (kc < 4) ad = umma_desc_sw128(smem_u32(smAtt + (kc - 2) * kChunk));
                else {
                    const int i = kc - 4;
                    sa = i % kAStages;
                    ok = mbar_wait(bar(BAR_FULL_A + sa), (uint32_t)((i / kAStages) & 1), abort_flag);
                    if (!ok) break;
                    fence_proxy_async();
                    ad = umma_desc_sw128(smem_u32(a_stage(sa)));
                }
                for (int sl = 0; sl < 2; ++sl, ++qb) {
                    const int sb = qb % kBStages;
                    ok = mbar_wait(bar(BAR_FULL_B + sb), (uint32_t)((qb / kBStages) & 1), abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t bd = umma_desc_sw128(smem_u32(smB + sb * kBStage));
                    const uint32_t d_tmem = tmem_base + (uint32_t)(sl * 256);
                    umma_bf16(d_tmem, ad, bd, idesc1, kc != 0 ? 1u : 0u);
                    umma_bf16_acc(d_tmem, ad + 2, bd + 2, idesc1);
                    umma_bf16_acc(d_tmem, ad + 4, bd + 4, idesc1);
                    umma_bf16_acc(d_tmem, ad + 6, bd + 6, idesc1);
                    umma_commit(bar(BAR_EMPTY_B + sb));
                }
                if (!ok) break;
                if (sa >= 0) umma_commit(bar(BAR_EMPTY_A + sa));
                if (kc == 1) umma_commit(bar(BAR_E_FREE));
            }
            // the cached user partial p_u (first-layer bias of this request): ones x [high; remainder]
            const int s_ones = p.n_cross % kAStages;
            uint64_t ones_d = 0;
            if (ok) ok = mbar_wait(bar(BAR_FULL_A + s_ones), (uint32_t)((p.n_cross / kAStages) & 1), abort_flag) &&
                         mbar_wait(bar(BAR_BIAS_FULL), 0u, abort_flag);
            if (ok) {
                fence_proxy_async();
                tc_fence_after();
                ones_d = umma_desc_sw128(smem_u32(a_stage(s_ones)));
                constexpr uint32_t idesc_b1 = umma_idesc_bf16_bmn(kTcTile, 256);
                umma_bf16(tmem_base, ones_d, umma_desc_mn_sw128(smem_u32(smE), 2048), idesc_b1, 1u);
                umma_bf16(tmem_base + 256u, ones_d, umma_desc_mn_sw128(smem_u32(smE + 8192), 2048), idesc_b1, 1u);
                umma_commit(bar(BAR_ACC1_FULL));
            }
            // layer 2: A = the packed activations in tensor memory
            ok = ok && mbar_wait(bar(BAR_H1_FULL), 0u, abort_flag);
            tc_fence_after();
            for (int kc = 0; ok && kc < kH1 / 64; ++kc, ++qb) {
                const int sb = qb % kBStages;
                ok = mbar_wait(bar(BAR_FULL_B + sb), (uint32_t)((qb / kBStages) & 1), abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint64_t bd = umma_desc_sw128(smem_u32(smB + sb * kBStage));
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const int k16 = kc * 4 + kk;   // 16 activations = 8 packed columns
                    const uint32_t a_tmem = tmem_base + (uint32_t)(k16 < 16 ? 8 * k16 : 384 + 8 * (k16 - 16));
                    umma_bf16_ts(tmem_base + 128u, a_tmem, bd + (uint64_t)(2 * kk), idesc2, (kc > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(bar(BAR_EMPTY_B + sb));
            }
            if (ok) {
                const uint32_t idesc_b2 = umma_idesc_bf16_bmn(kTcTile, p.H2);
                umma_bf16(tmem_base + 128u, ones_d, umma_desc_mn_sw128(smem_u32(smE + 16384), 2048), idesc_b2, 1u);
                umma_commit(bar(BAR_ACC2_FULL));
            }
        }
        __syncwarp();
    } else if (warp < kFBWarp) {
        // ===================== item-row and cross-feature gather (128 threads) =====================
        const int pt = tid - kFProdWarp0 * 32;
        const int sub = pt & 7, r0 = pt >> 3;   // 16-byte slot of the 128-byte chunk row; rows r0, r0 + 16, ...
        const uint32_t row_off = (uint32_t)(r0 * 128) + (uint32_t)((sub ^ (r0 & 7)) << 4);
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (r0 + 16 * i < cnt && (id[i] < 0 || (int64_t)id[i] >= p.M)) {
                id[i] = -1;
                if (sub == 0) atomicOr(p.sl.status, AIF_STATUS_BAD_ID);
            }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint8_t *gsrc = p.E + (id[i] >= 0 ? (size_t)id[i] * 256 + sub * 16 : 0);
            const uint32_t dst = smem_u32(smE) + row_off + (uint32_t)(i * 16 * 128);
            cp_async16(dst, gsrc, id[i] >= 0 ? 16u : 0u);
            cp_async16(dst + kChunk, gsrc + 128, id[i] >= 0 ? 16u : 0u);
        }
        cp_async_arrive_noinc(bar(BAR_E_FULL));
        // cross features (Section 3.3): the row of field f's user-side table that the candidate's bucket selects
        const uint8_t *Tt = reinterpret_cast<const uint8_t *>(slot->T);
        uint32_t src16[8];   // offsets of this thread's eight copies of the coming chunk, in 16-byte units; ~0: zero fill
        auto resolve = [&](int i) {
            const int col = 64 * i + 8 * sub;
            const int f = col / p.dc, kin = col - f * p.dc;
            const uint32_t row16 = (uint32_t)(p.dc >> 3), base16 = (uint32_t)(f * p.B) * row16 + (uint32_t)(kin >> 3);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                uint32_t bk;
                if (p.bucket_mode == AIF_BUCKET_MOD) bk = (uint32_t)(id[j] % p.B);
                else {
                    const uint64_t h = mix64((uint64_t)id[j], (uint64_t)f);
                    bk = p.b_mask >= 0 ? (uint32_t)(h & (uint64_t)p.b_mask) : (uint32_t)(h % (uint64_t)p.B);
                }
                src16[j] = id[j] >= 0 ? bk * row16 + base16 : 0xFFFFFFFFu;
            }
        };
        bool ok = true;
        if (p.n_cross > 0) resolve(0);
        for (int i = 0; ok && i < p.n_cross; ++i) {
            const int s = i % kAStages;
            ok = mbar_wait(bar(BAR_EMPTY_A + s), (uint32_t)(((i / kAStages) & 1) ^ 1), abort_flag);
            // stages 2 and 3 lie where the second key block was: P V must be done with it
            if (ok && s >= 2 && i < kAStages && nb == 2) ok = mbar_wait(bar(BAR_O_FINAL), 0u, abort_flag);
            if (!ok) break;
            const uint32_t dst0 = smem_u32(a_stage(s)) + row_off;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const bool on = src16[j] != 0xFFFFFFFFu;
                cp_async16(dst0 + (uint32_t)(j * 16 * 128), on ? Tt + ((size_t)src16[j] << 4) : p.E, on ? 16u : 0u);
            }
            cp_async_arrive_noinc(bar(BAR_FULL_A + s));
            if (i + 1 < p.n_cross) resolve(i + 1);
        }
        // the tile of ones that carries the biases: one more stage of the ring, columns 0 and 1 of row pt
        if (ok) {
            const int i = p.n_cross, s = i % kAStages;
            ok = mbar_wait(bar(BAR_EMPTY_A + s), (uint32_t)(((i / kAStages) & 1) ^ 1), abort_flag);
            if (ok && s >= 2 && i < kAStages && nb == 2) ok = mbar_wait(bar(BAR_O_FINAL), 0u, abort_flag);
            if (ok) {
                unsigned char *rowp = a_stage(s) + pt * 128;
                *reinterpret_cast<uint4 *>(rowp + ((0 ^ (pt & 7)) << 4)) = make_uint4(0x3F803F80u, 0u, 0u, 0u);
                *reinterpret_cast<uint4 *>(rowp + ((1 ^ (pt & 7)) << 4)) = make_uint4(0u, 0u, 0u, 0u);
                fence_proxy_async();
                mbar_arrive(bar(BAR_FULL_A + s));
            }
        }
        cp_async_wait_all();
    } else {
        // ===================== key/value blocks and weights (TMA) =====================
        if (lane == 0) {
            for (int j = 0; j < nb; ++j) {
                mbar_expect_tx(bar(BAR_KV_FULL + j), 32768u);
                tma_load_3d(smem_u32(smKV + j * 32768), &tmapS, bar(BAR_KV_FULL + j), 0, j * 128, rq.slot);
                tma_load_3d(smem_u32(smKV + j * 32768 + kChunk), &tmapS, bar(BAR_KV_FULL + j), 64, j * 128, rq.slot);
            }
            bool ok = true;
            int qb = 0;
            for (int kc = 0; ok && kc < n_k1; ++kc)
                for (int sl = 0; sl < 2; ++sl, ++qb) {
                    const int sb = qb % kBStages;
                    ok = mbar_wait(bar(BAR_EMPTY_B + sb), (uint32_t)(((qb / kBStages) & 1) ^ 1), abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(bar(BAR_FULL_B + sb), 32768u);
                    tma_load_2d(smem_u32(smB + sb * kBStage), &tmapW1, bar(BAR_FULL_B + sb), kc * 64, sl * 256);
                }
            for (int kc = 0; ok && kc < kH1 / 64; ++kc, ++qb) {
                const int sb = qb % kBStages;
                ok = mbar_wait(bar(BAR_EMPTY_B + sb), (uint32_t)(((qb / kBStages) & 1) ^ 1), abort_flag);
                if (!ok) break;
                mbar_expect_tx(bar(BAR_FULL_B + sb), (uint32_t)p.H2 * 128u);
                tma_load_2d(smem_u32(smB + sb * kBStage), &tmapW2, bar(BAR_FULL_B + sb), kc * 64, 0);
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
    if (warp == kFMmaWarp) tmem_dealloc(tmem_base, 512);
}

// bias [n] fp32 -> [2][n] bf16: high parts, then the remainders bias - high
__global__ void k_split_bias(const float *__restrict__ b, int n, __nv_bfloat16 *__restrict__ out)
{
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const __nv_bfloat16 hi = __float2bfloat16_rn(b[i]);
        out[i] = hi;
        out[n + i] = __float2bfloat16_rn(b[i] - __bfloat162float(hi));
    }
}

}  // namespace

bool tc_fused_supported(const aif_config &c)
{
    if (c.dtype != AIF_BF16 || c.d != 128) return false;
    if (c.blocks != (AIF_BLK_ATT | AIF_BLK_CROSS)) return false;
    if (c.n_hidden != 2 || c.hidden[0] != kH1 || c.hidden[1] > 256 || c.hidden[1] % 64 != 0) return false;
    const int cross_cols = c.F * c.dc;
    if (cross_cols % 64 != 0 || cross_cols / 64 > kMaxCross || c.dc % 8 != 0) return false;
    return tc_supported(c) && tc_att_supported(c);
}

cudaError_t tc_fused_prepare(aif_ctx *ctx)
{
    void *ptr = nullptr;   // the second layer's bias as the tensor cores take it: [2][hidden[1]] bf16
    cudaError_t e = cudaMalloc(&ptr, 2 * 256 * 2);
    if (e != cudaSuccess) return e;
    ctx->allocations.push_back(ptr), ctx->device_bytes += 2 * 256 * 2;
    ctx->tc_fused_plan = ptr;
    return cudaFuncSetAttribute(k_request_fused, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFSmem);
}

cudaError_t tc_fused_prepare_weights(aif_ctx *ctx, cudaStream_t st)
{
    k_split_bias<<<1, 256, 0, st>>>(ctx->b[1], ctx->cfg.hidden[1], reinterpret_cast<__nv_bfloat16 *>(ctx->tc_fused_plan));
    count_launch();
    return cudaGetLastError();
}

// One launch for the whole call; the caller has checked tc_fused_supported and that no sequence is longer than 256.
cudaError_t launch_request_fused(const aif_ctx *ctx, const ScoreLaunch &sl, cudaStream_t st)
{
    const aif_config &c = ctx->cfg;
    FusedParams p{};
    p.sl = sl, p.E = (const uint8_t *)ctx->E, p.M = c.M, p.mini_batch = c.mini_batch;
    p.B = c.B, p.dc = c.dc, p.b_mask = (c.B & (c.B - 1)) == 0 ? c.B - 1 : -1, p.bucket_mode = c.bucket_mode;
    p.n_cross = c.F * c.dc / 64;
    p.H2 = c.hidden[1], p.emit_sigmoid = c.emit_sigmoid;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)c.d);
    p.b2_hl = reinterpret_cast<const __nv_bfloat16 *>(ctx->tc_fused_plan), p.w_out = (const __nv_bfloat16 *)ctx->w_out, p.b_out = ctx->b_out;
    const CUtensorMap *ms = reinterpret_cast<const CUtensorMap *>(tc_att_tmap(ctx));
    const CUtensorMap *m1 = reinterpret_cast<const CUtensorMap *>(tc_weight_tmap(ctx, 0));
    const CUtensorMap *m2 = reinterpret_cast<const CUtensorMap *>(tc_weight_tmap(ctx, 1));
    cudaError_t e = launch_pdl(k_request_fused, dim3(sl.n_tiles), dim3(kFThreads), kFSmem, st, *ms, *m1, *m2, p);
    count_launch();
    return e;
}

}  // namespace aif
