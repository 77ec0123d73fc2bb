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
//               the scores of key block g; the groups exchange row maxima and sums through shared memory, write the
//               probabilities back into tensor memory as packed bf16 (A operand of P V), then normalise O into the
//               attention chunks of the first layer's input (group g: columns [64 g, 64 g + 64)).  Layer-1 epilogue:
//               group g adds the request's cached user partial p_u to output slice g, applies ReLU and writes the bf16
//               activations back into tensor memory over the accumulator it has just read (A operand of layer 2).
//               Layer-2 epilogue: bias, ReLU and the dot with w_out, half of the units per group.
//   warp 8      allocates tensor memory; one lane issues every tcgen05.mma
//   warps 9-12  gather the tile's item rows (queries of the attention and first K chunks of layer 1) and, chunk by
//               chunk, its cross-feature rows from the request's pre-cache, with 16-byte cp.async into 128B-swizzled
//               K-major chunks; buckets are hashed one chunk ahead of their use
//   warp 13     one lane streams key/value blocks, then first- and second-layer weights with TMA
//
// Tensor memory (512 columns): attention uses [0, 256) for the scores of up to two key blocks (probabilities packed
// over the first half of each block's own columns) and [256, 384) for O.  Layer 1 then fills two 256-column
// accumulators [0, 256) and [256, 512); its activations are packed in place into [0, 128) and [256, 384); layer 2
// accumulates its two halves into the freed columns [128, 256) and [384, 512).
// Shared memory: item tile 32 KB | key/value blocks 64 KB, later the attention chunks and two more stages of the
// cross-feature ring | two cross-feature stages 32 KB | weight ring 3 x 32 KB | barriers and exchange arrays.
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
    BAR_H1_FULL, BAR_ACC2_FULL, BAR_FULL_A, BAR_EMPTY_A = BAR_FULL_A + kAStages, BAR_FULL_B = BAR_EMPTY_A + kAStages,
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
    const float *b2;
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
        bool good = false;
        if (row < cnt) {
            const int id = p.sl.ids[pos0 + row];
            good = id >= 0 && (int64_t)id < p.M;
        }
        // ---- attention: scores of key block g -> probabilities
        const bool act = g < nb;
        const int valid_cols = L - g * 128 < 128 ? L - g * 128 : 128;
        float mx = -INFINITY;
        if (act) {
            wait(BAR_S_FULL);
            tc_fence_after();
            if (ok) {
#pragma unroll 1
                for (int c0 = 0; c0 < 128; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld32(lane_base + (uint32_t)(g * 128 + c0), r);
                    tmem_ld_wait();
                    float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (c0 + i < valid_cols) m4[i & 3] = fmaxf(m4[i & 3], __uint_as_float(r[i]));
                    mx = fmaxf(mx, fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])));
                }
            }
        }
        xs[g * 128 + row] = mx;
        named_bar_sync(1, 256);
        const float mt = fmaxf(mx, xs[(g ^ 1) * 128 + row]) * k2;   // an inactive group has published -inf
        named_bar_sync(1, 256);                                    // both maxima are read: xs may now take the sums
        float lsum = 0.f;
        if (act && ok) {
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {
                uint32_t sc[64];
                tmem_ld32(lane_base + (uint32_t)(g * 128 + 64 * h), *reinterpret_cast<uint32_t(*)[32]>(&sc[0]));
                tmem_ld32(lane_base + (uint32_t)(g * 128 + 64 * h + 32), *reinterpret_cast<uint32_t(*)[32]>(&sc[32]));
                tmem_ld_wait();
                uint32_t packed[32];
                float ls4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    float p0 = fast_exp2(fmaf(__uint_as_float(sc[2 * i]), k2, -mt));
                    float p1 = fast_exp2(fmaf(__uint_as_float(sc[2 * i + 1]), k2, -mt));
                    if (64 * h + 2 * i >= valid_cols) p0 = 0.f;
                    if (64 * h + 2 * i + 1 >= valid_cols) p1 = 0.f;
                    ls4[i & 3] += p0 + p1;
                    const __nv_bfloat162 hh = __floats2bfloat162_rn(p0, p1);
                    packed[i] = *reinterpret_cast<const uint32_t *>(&hh);
                }
                // over columns this thread has already read: [64 h, 64 h + 64) of the block -> [32 h, 32 h + 32)
                tmem_st32(lane_base + (uint32_t)(g * 128 + 32 * h), packed);
                lsum += (ls4[0] + ls4[1]) + (ls4[2] + ls4[3]);
            }
            tmem_st_wait();
        }
        xs[g * 128 + row] = lsum;
        tc_fence_before();
        mbar_arrive(bar(BAR_P_FULL));
        named_bar_sync(1, 256);
        const float l_all = lsum + xs[(g ^ 1) * 128 + row];
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
        // ---- biases into the item tile's memory once layer 1 has consumed it
        wait(BAR_E_FREE);
        float *bias1 = reinterpret_cast<float *>(smE), *b2_s = bias1 + kH1, *wout_s = b2_s + 256, *dot_s = wout_s + 256;
        {
            const int t = warp * 32 + lane;
            bias1[t] = slot->p_u[t];
            bias1[t + 256] = slot->p_u[t + 256];
            if (t < p.H2) {
                b2_s[t] = p.b2[t];
                wout_s[t] = __bfloat162float(p.w_out[t]);
            }
        }
        named_bar_sync(1, 256);
        // ---- layer-1 epilogue: slice g, 64 accumulator columns -> 32 columns of packed bf16, in place
        wait(BAR_ACC1_FULL);
        tc_fence_after();
        if (ok) {
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t r[64];
                tmem_ld32(lane_base + (uint32_t)(g * 256 + 64 * c), *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
                tmem_ld32(lane_base + (uint32_t)(g * 256 + 64 * c + 32), *reinterpret_cast<uint32_t(*)[32]>(&r[32]));
                tmem_ld_wait();
                const float4 *b4 = reinterpret_cast<const float4 *>(bias1 + g * 256 + 64 * c);
                uint32_t packed[32];
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                    const float4 bb = b4[q];
                    const __nv_bfloat162 h0 = __floats2bfloat162_rn(fmaxf(__uint_as_float(r[4 * q]) + bb.x, 0.f),
                                                                    fmaxf(__uint_as_float(r[4 * q + 1]) + bb.y, 0.f));
                    const __nv_bfloat162 h1 = __floats2bfloat162_rn(fmaxf(__uint_as_float(r[4 * q + 2]) + bb.z, 0.f),
                                                                    fmaxf(__uint_as_float(r[4 * q + 3]) + bb.w, 0.f));
                    packed[2 * q] = *reinterpret_cast<const uint32_t *>(&h0);
                    packed[2 * q + 1] = *reinterpret_cast<const uint32_t *>(&h1);
                }
                tmem_st32(lane_base + (uint32_t)(g * 256 + 32 * c), packed);
            }
            tmem_st_wait();
        }
        tc_fence_before();
        mbar_arrive(bar(BAR_H1_FULL));
        // ---- layer-2 epilogue: half g of the units, reduced against w_out
        wait(BAR_ACC2_FULL);
        tc_fence_after();
        float dot = 0.f;
        if (ok) {
            const int hn = p.H2 >> 1;
            for (int c0 = 0; c0 < hn; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(lane_base + (uint32_t)((g ? 384 : 128) + c0), r);
                tmem_ld_wait();
                const float4 *b4 = reinterpret_cast<const float4 *>(b2_s + g * hn + c0);
                const float4 *w4 = reinterpret_cast<const float4 *>(wout_s + g * hn + c0);
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const float4 bb = b4[q], ww = w4[q];
                    dot = fmaf(fmaxf(__uint_as_float(r[4 * q]) + bb.x, 0.f), ww.x, dot);
                    dot = fmaf(fmaxf(__uint_as_float(r[4 * q + 1]) + bb.y, 0.f), ww.y, dot);
                    dot = fmaf(fmaxf(__uint_as_float(r[4 * q + 2]) + bb.z, 0.f), ww.z, dot);
                    dot = fmaf(fmaxf(__uint_as_float(r[4 * q + 3]) + bb.w, 0.f), ww.w, dot);
                }
            }
        }
        if (g == 1) dot_s[row] = dot;
        named_bar_sync(1, 256);
        if (g == 0 && ok && row < cnt) {
            float logit = dot + dot_s[row] + p.b_out[0];
            if (p.emit_sigmoid) logit = 1.0f / (1.0f + expf(-logit));
            if (!good) logit = __int_as_float(0x7fc00000);
            p.sl.logits[pos0 + row] = logit;
        }
    } else if (warp == kFMmaWarp) {
        // ===================== MMA issuer =====================
        if (lane == 0) {
            constexpr uint32_t idesc_qk = umma_idesc_bf16(kTcTile, 128);
            constexpr uint32_t idesc_pv = umma_idesc_bf16_bmn(kTcTile, 128);
            constexpr uint32_t idesc1 = umma_idesc_bf16(kTcTile, 256);
            const uint32_t idesc2 = umma_idesc_bf16(kTcTile, p.H2 >> 1);
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
                        umma_bf16_ts(tmem_base + 256u, tmem_base + (uint32_t)(j * 128 + kk * 8), vd + (uint64_t)(kk * (2048 >> 4)), idesc_pv,
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
            if (ok) umma_commit(bar(BAR_ACC1_FULL));
            // layer 2: A = the packed activations in tensor memory, two halves of the output units
            ok = ok && mbar_wait(bar(BAR_H1_FULL), 0u, abort_flag);
            tc_fence_after();
            const uint64_t half_off = (uint64_t)(((p.H2 >> 1) * 128) >> 4);
            for (int kc = 0; ok && kc < kH1 / 64; ++kc, ++qb) {
                const int sb = qb % kBStages;
                ok = mbar_wait(bar(BAR_FULL_B + sb), (uint32_t)((qb / kBStages) & 1), abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint64_t bd0 = umma_desc_sw128(smem_u32(smB + sb * kBStage));
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const uint32_t d_tmem = tmem_base + (hf ? 384u : 128u);
                    const uint64_t bd = bd0 + (hf ? half_off : 0ull);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const int k16 = kc * 4 + kk;   // 16 activations = 8 packed columns
                        const uint32_t a_tmem = tmem_base + (uint32_t)(k16 < 16 ? 8 * k16 : 256 + 8 * (k16 - 16));
                        umma_bf16_ts(d_tmem, a_tmem, bd + (uint64_t)(2 * kk), idesc2, (kc > 0 || kk > 0) ? 1u : 0u);
                    }
                }
                umma_commit(bar(BAR_EMPTY_B + sb));
            }
            if (ok) umma_commit(bar(BAR_ACC2_FULL));
        }
        __syncwarp();
    } else if (warp < kFBWarp) {
        // ===================== item-row and cross-feature gather (128 threads) =====================
        const int pt = tid - kFProdWarp0 * 32;
        const int sub = pt & 7, r0 = pt >> 3;   // 16-byte slot of the 128-byte chunk row; rows r0, r0 + 16, ...
        const uint32_t row_off = (uint32_t)(r0 * 128) + (uint32_t)((sub ^ (r0 & 7)) << 4);
        int id[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = r0 + 16 * i;
            int v = -1;
            if (r < cnt) {
                v = p.sl.ids[pos0 + r];
                if (v < 0 || (int64_t)v >= p.M) {
                    v = -1;
                    if (sub == 0) atomicOr(p.sl.status, AIF_STATUS_BAD_ID);
                }
            }
            id[i] = v;
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

cudaError_t tc_fused_prepare(aif_ctx *)
{
    return cudaFuncSetAttribute(k_request_fused, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFSmem);
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
    p.b2 = ctx->b[1], p.w_out = (const __nv_bfloat16 *)ctx->w_out, p.b_out = ctx->b_out;
    const CUtensorMap *ms = reinterpret_cast<const CUtensorMap *>(tc_att_tmap(ctx));
    const CUtensorMap *m1 = reinterpret_cast<const CUtensorMap *>(tc_weight_tmap(ctx, 0));
    const CUtensorMap *m2 = reinterpret_cast<const CUtensorMap *>(tc_weight_tmap(ctx, 1));
    cudaError_t e = launch_pdl(k_request_fused, dim3(sl.n_tiles), dim3(kFThreads), kFSmem, st, *ms, *m1, *m2, p);
    count_launch();
    return e;
}

}  // namespace aif
