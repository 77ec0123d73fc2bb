// Item-side tower of the nearline pipeline (Section 3.2 eq. 4) in one kernel: I^ = W1 ReLU(W0 I + b0) + b1 for rows of
// raw item features, bf16 in, fp32 accumulate, with the hidden activations kept in tensor memory.  Run as two launches
// of the layer kernel the call is bound by the hidden activations' trip through HBM (512 B written and read per item
// against 1.25 KB of input and output); here they never leave the SM.
//
// Persistent: a CTA walks over pairs of 128-row tiles; both tiles of a pair are fed from the same weight chunks, which
// halves the weight bytes an SM takes in per item.  320 threads:
//   warps 0-7  two groups of four warps, group g = tile g of the pair, one thread per row.  After layer 1: bias, ReLU,
//              bf16, packed back into tensor memory over accumulator columns already read (A operand of layer 2).
//              After layer 2: bias, bf16, through a staging slab and a TMA tile store into the output rows.
//   warp 8     allocates tensor memory; one lane issues tcgen05.mma
//   warp 9     one lane streams the raw rows (two 128 x 64 boxes per K chunk) and the weights with TMA
// Tensor memory per tile g: layer-1 accumulator [256 g, 256 g + hI), packed activations [256 g, 256 g + hI / 2), layer-2
// accumulator [256 g + 128, 256 g + 128 + d).  Shapes: dI a multiple of 64; hI in {64, 128, 192, 256}; d <= 128, a
// multiple of 32.  Every wait is bounded (AIF_STATUS_TIMEOUT on expiry, tensor memory freed, normal return).
#include <cuda.h>

#include "aif_device.cuh"
#include "aif_internal.h"
#include "aif_tc_ptx.cuh"

namespace aif {
namespace {

constexpr int kTThreads = 320, kTMmaWarp = 8;   // warp 9 streams rows and weights
constexpr int kTStagesA = 3, kTStagesB = 3, kTAStage = 32768, kTBStage = 32768;
constexpr int kTOffB = kTStagesA * kTAStage, kTOffSlab = kTOffB + kTStagesB * kTBStage, kTOffMisc = kTOffSlab + 8 * 2048;
constexpr size_t kTSmem = 1024 + kTOffMisc + 2048;

enum { TB_FULL_A = 0, TB_EMPTY_A = TB_FULL_A + kTStagesA, TB_FULL_B = TB_EMPTY_A + kTStagesA, TB_EMPTY_B = TB_FULL_B + kTStagesB,
       TB_ACC1 = TB_EMPTY_B + kTStagesB, TB_H_FULL, TB_ACC2, TB_TM_FREE, TB_COUNT };

struct TowerParams {
    int64_t n;            // rows
    int32_t n_pairs, n_k1, hI, d;
    const float *b0, *b1;
    __nv_bfloat16 *out;   // [n x d]
    float *norm_max;      // raised to the largest Euclidean norm of an output row (an upper bound: taken before rounding, widened by 2^-8)
    uint32_t *status;
};

__global__ void __launch_bounds__(kTThreads, 1) k_item_tower_tc(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapW0,
                                                                const __grid_constant__ CUtensorMap tmapW1,
                                                                const __grid_constant__ CUtensorMap tmapOut, const TowerParams p)
{
    extern __shared__ unsigned char smem_dyn[];
    unsigned char *base = reinterpret_cast<unsigned char *>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    unsigned char *smA = base, *smB = base + kTOffB, *slabs = base + kTOffSlab;
    uint64_t *bars = reinterpret_cast<uint64_t *>(base + kTOffMisc);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + TB_COUNT);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    float *b0_s = reinterpret_cast<float *>(tmem_slot + 4), *b1_s = b0_s + 256;   // [256], [128]
    auto bar = [&](int i) { return smem_u32(bars + i); };
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < kTStagesA; ++s) mbar_init(bar(TB_FULL_A + s), 1), mbar_init(bar(TB_EMPTY_A + s), 1);
        for (int s = 0; s < kTStagesB; ++s) mbar_init(bar(TB_FULL_B + s), 1), mbar_init(bar(TB_EMPTY_B + s), 1);
        mbar_init(bar(TB_ACC1), 1);
        mbar_init(bar(TB_H_FULL), 256);
        mbar_init(bar(TB_ACC2), 1);
        mbar_init(bar(TB_TM_FREE), 256);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kTMmaWarp) tmem_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    grid_dep_launch();
    grid_dep_wait();
    const int n_k2 = p.hI >> 6;

    if (warp < 8) {
        // ===================== epilogues =====================
        const int g = warp >> 2, wq = warp & 3, row = wq * 32 + lane;
        const uint32_t col0 = tmem_base + ((uint32_t)(wq * 32) << 16) + (uint32_t)(g * 256);
        for (int j = tid; j < 256; j += 256) b0_s[j] = j < p.hI ? p.b0[j] : 0.f;
        if (tid < 128) b1_s[tid] = tid < p.d ? p.b1[tid] : 0.f;
        named_bar_sync(1, 256);
        unsigned char *sb = slabs + warp * 2048;
        bool ok = true;
        auto wait = [&](int b, uint32_t parity) {
            const bool got = ok && mbar_wait(bar(b), parity, abort_flag);
            ok = __all_sync(0xffffffffu, got);
        };
        int it = 0;
        for (int pair = blockIdx.x; pair < p.n_pairs; pair += gridDim.x, ++it) {
            const uint32_t ph = (uint32_t)(it & 1);
            const int64_t row0 = ((int64_t)pair * 2 + g) * kTcTile;   // first row of this group's tile
            // ---- after layer 1: bias, ReLU, 32 columns -> 16 packed columns over columns already read
            wait(TB_ACC1, ph);
            tc_fence_after();
            if (!ok) break;
            {
                uint32_t ra[32], rb[32];
                auto finish = [&](const uint32_t (&r)[32], int c) {
                    const float4 *b4 = reinterpret_cast<const float4 *>(b0_s + 32 * c);
                    uint32_t packed[16];
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const float4 bb = b4[q];
                        const __nv_bfloat162 h0 = __floats2bfloat162_rn(fmaxf(__uint_as_float(r[4 * q]) + bb.x, 0.f),
                                                                        fmaxf(__uint_as_float(r[4 * q + 1]) + bb.y, 0.f));
                        const __nv_bfloat162 h1 = __floats2bfloat162_rn(fmaxf(__uint_as_float(r[4 * q + 2]) + bb.z, 0.f),
                                                                        fmaxf(__uint_as_float(r[4 * q + 3]) + bb.w, 0.f));
                        packed[2 * q] = *reinterpret_cast<const uint32_t *>(&h0);
                        packed[2 * q + 1] = *reinterpret_cast<const uint32_t *>(&h1);
                    }
                    tmem_st16(col0 + (uint32_t)(16 * c), packed);
                };
                const int nc = p.hI >> 5;   // even
                tmem_ld32(col0, ra);
#pragma unroll 1
                for (int c = 0; c < nc; c += 2) {
                    tmem_ld_wait();
                    tmem_ld32(col0 + (uint32_t)(32 * (c + 1)), rb);
                    finish(ra, c);
                    tmem_ld_wait();
                    if (c + 2 < nc) tmem_ld32(col0 + (uint32_t)(32 * (c + 2)), ra);
                    finish(rb, c + 1);
                }
                tmem_st_wait();
            }
            tc_fence_before();
            mbar_arrive(bar(TB_H_FULL));
            // ---- after layer 2: bias, bf16, out
            wait(TB_ACC2, ph);
            tc_fence_after();
            if (!ok) break;
            const bool whole = row0 + wq * 32 + 32 <= p.n;
            float ss = 0.f;   // squared norm of this thread's output row
            for (int c0 = 0; c0 < p.d; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(col0 + (uint32_t)(128 + c0), r);
                tmem_ld_wait();
                if (c0 + 32 >= p.d) {   // the accumulators of this pair are in registers: the next pair may overwrite them
                    tc_fence_before();
                    mbar_arrive(bar(TB_TM_FREE));
                }
                const float4 *b4 = reinterpret_cast<const float4 *>(b1_s + c0);
                uint32_t packed[16];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const float4 bb = b4[q];
                    const float x0 = __uint_as_float(r[4 * q]) + bb.x, x1 = __uint_as_float(r[4 * q + 1]) + bb.y;
                    const float x2 = __uint_as_float(r[4 * q + 2]) + bb.z, x3 = __uint_as_float(r[4 * q + 3]) + bb.w;
                    ss = fmaf(x0, x0, fmaf(x1, x1, fmaf(x2, x2, fmaf(x3, x3, ss))));
                    const __nv_bfloat162 h0 = __floats2bfloat162_rn(x0, x1);
                    const __nv_bfloat162 h1 = __floats2bfloat162_rn(x2, x3);
                    packed[2 * q] = *reinterpret_cast<const uint32_t *>(&h0);
                    packed[2 * q + 1] = *reinterpret_cast<const uint32_t *>(&h1);
                }
                if (whole) {
                    if (lane == 0) bulk_wait_read<0>();   // the store that last read the slab is done with it
                    __syncwarp();
                    const int swz = (lane >> 1) & 3;
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        *reinterpret_cast<uint4 *>(sb + lane * 64 + ((q ^ swz) << 4)) =
                            make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&tmapOut, smem_u32(sb), c0, (int)(row0 + wq * 32));
                        bulk_commit();
                    }
                } else if (row0 + row < p.n) {
                    uint4 *dst = reinterpret_cast<uint4 *>(p.out + (size_t)(row0 + row) * p.d + c0);
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        dst[q] = make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
                }
            }
            if (p.norm_max) {
                // non-negative floats order like their bit patterns; a NaN row gives a pattern above every finite one
                const int bits = row0 + row < p.n ? (__float_as_int(sqrtf(ss) * 1.00390625f) & 0x7fffffff) : 0;
                const int best = __reduce_max_sync(0xffffffffu, bits);
                if (lane == 0 && best > 0) atomicMax(reinterpret_cast<int *>(p.norm_max), best);
            }
        }
        if (lane == 0) bulk_wait<0>();
    } else if (warp == kTMmaWarp) {
        // ===================== MMA issuer =====================
        if (lane == 0) {
            const uint32_t idesc1 = umma_idesc_bf16(kTcTile, p.hI), idesc2 = umma_idesc_bf16(kTcTile, p.d);
            int sa = 0, sb = 0, it = 0;
            uint32_t pha = 0, phb = 0;
            bool ok = true;
            for (int pair = blockIdx.x; ok && pair < p.n_pairs; pair += gridDim.x, ++it) {
                // tensor memory of the previous pair must have been read out
                if (it > 0) ok = mbar_wait(bar(TB_TM_FREE), (uint32_t)((it - 1) & 1), abort_flag);
                tc_fence_after();
                for (int kc = 0; ok && kc < p.n_k1; ++kc) {
                    ok = mbar_wait(bar(TB_FULL_A + sa), pha, abort_flag) && mbar_wait(bar(TB_FULL_B + sb), phb, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t bd = umma_desc_sw128(smem_u32(smB + sb * kTBStage));
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        const uint64_t ad = umma_desc_sw128(smem_u32(smA + sa * kTAStage + g * 16384));
                        const uint32_t d_tmem = tmem_base + (uint32_t)(g * 256);
                        umma_bf16(d_tmem, ad, bd, idesc1, kc != 0 ? 1u : 0u);
                        umma_bf16_acc(d_tmem, ad + 2, bd + 2, idesc1);
                        umma_bf16_acc(d_tmem, ad + 4, bd + 4, idesc1);
                        umma_bf16_acc(d_tmem, ad + 6, bd + 6, idesc1);
                    }
                    umma_commit(bar(TB_EMPTY_A + sa));
                    umma_commit(bar(TB_EMPTY_B + sb));
                    if (++sa == kTStagesA) sa = 0, pha ^= 1u;
                    if (++sb == kTStagesB) sb = 0, phb ^= 1u;
                }
                if (!ok) break;
                umma_commit(bar(TB_ACC1));
                ok = mbar_wait(bar(TB_H_FULL), (uint32_t)(it & 1), abort_flag);
                tc_fence_after();
                for (int kc = 0; ok && kc < n_k2; ++kc) {
                    ok = mbar_wait(bar(TB_FULL_B + sb), phb, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t bd = umma_desc_sw128(smem_u32(smB + sb * kTBStage));
#pragma unroll
                    for (int g = 0; g < 2; ++g)
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)   // 16 activations = 8 packed columns
                            umma_bf16_ts(tmem_base + (uint32_t)(g * 256 + 128), tmem_base + (uint32_t)(g * 256 + 8 * (kc * 4 + kk)),
                                         bd + (uint64_t)(2 * kk), idesc2, (kc > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(bar(TB_EMPTY_B + sb));
                    if (++sb == kTStagesB) sb = 0, phb ^= 1u;
                }
                if (ok) umma_commit(bar(TB_ACC2));
            }
        }
        __syncwarp();
    } else {
        // ===================== rows and weights (TMA) =====================
        if (lane == 0) {
            int sa = 0, sb = 0;
            uint32_t pha = 0, phb = 0;
            bool ok = true;
            for (int pair = blockIdx.x; ok && pair < p.n_pairs; pair += gridDim.x) {
                for (int kc = 0; ok && kc < p.n_k1; ++kc) {
                    ok = mbar_wait(bar(TB_EMPTY_A + sa), pha ^ 1u, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(bar(TB_FULL_A + sa), 32768u);   // rows beyond the last one arrive as zeros
                    tma_load_2d(smem_u32(smA + sa * kTAStage), &tmapA, bar(TB_FULL_A + sa), kc * 64, pair * 256);
                    tma_load_2d(smem_u32(smA + sa * kTAStage + 16384), &tmapA, bar(TB_FULL_A + sa), kc * 64, pair * 256 + 128);
                    if (++sa == kTStagesA) sa = 0, pha ^= 1u;
                    ok = mbar_wait(bar(TB_EMPTY_B + sb), phb ^ 1u, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(bar(TB_FULL_B + sb), (uint32_t)p.hI * 128u);
                    tma_load_2d(smem_u32(smB + sb * kTBStage), &tmapW0, bar(TB_FULL_B + sb), kc * 64, 0);
                    if (++sb == kTStagesB) sb = 0, phb ^= 1u;
                }
                for (int kc = 0; ok && kc < n_k2; ++kc) {
                    ok = mbar_wait(bar(TB_EMPTY_B + sb), phb ^ 1u, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(bar(TB_FULL_B + sb), (uint32_t)p.d * 128u);
                    tma_load_2d(smem_u32(smB + sb * kTBStage), &tmapW1, bar(TB_FULL_B + sb), kc * 64, 0);
                    if (++sb == kTStagesB) sb = 0, phb ^= 1u;
                }
            }
        }
        __syncwarp();
    }

    if (*abort_flag) {
        if (tid == 0) atomicOr(p.status, AIF_STATUS_TIMEOUT);
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kTMmaWarp) tmem_dealloc(tmem_base, 512);
}

cudaError_t encode2d(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint32_t box_c, uint32_t box_r, CUtensorMapSwizzle sw)
{
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {box_c, box_r};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

}  // namespace

bool tc_tower_supported(int dI, int hI, int d)
{
    return dI % 64 == 0 && dI <= 4096 && hI % 64 == 0 && hI >= 64 && hI <= 256 && d % 32 == 0 && d >= 32 && d <= 128 && encode_fn() != nullptr;
}

cudaError_t tc_tower_prepare() { return cudaFuncSetAttribute(k_item_tower_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTSmem); }

// out [n x d] = W1 ReLU(W0 I_raw^T + b0) + b1 for n rows of I_raw [n x dI]; all matrices bf16 row-major, biases fp32.
cudaError_t launch_item_tower_tc(const aif_ctx *ctx, const void *I_raw, const void *W0, const float *b0, const void *W1, const float *b1,
                                 void *out, int64_t n, int dI, int hI, float *norm_max, cudaStream_t st)
{
    if (n <= 0) return cudaSuccess;
    const int d = ctx->cfg.d;
    CUtensorMap ma, m0, m1, mo;
    cudaError_t e;
    if ((e = encode2d(&ma, I_raw, (uint64_t)dI, (uint64_t)n, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B)) != cudaSuccess) return e;
    if ((e = encode2d(&m0, W0, (uint64_t)dI, (uint64_t)hI, 64, (uint32_t)hI, CU_TENSOR_MAP_SWIZZLE_128B)) != cudaSuccess) return e;
    if ((e = encode2d(&m1, W1, (uint64_t)hI, (uint64_t)d, 64, (uint32_t)d, CU_TENSOR_MAP_SWIZZLE_128B)) != cudaSuccess) return e;
    if ((e = encode2d(&mo, out, (uint64_t)d, (uint64_t)n, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B)) != cudaSuccess) return e;
    TowerParams p{};
    p.n = n, p.n_pairs = (int)((n + 2 * kTcTile - 1) / (2 * kTcTile)), p.n_k1 = dI / 64, p.hI = hI, p.d = d;
    p.b0 = b0, p.b1 = b1, p.out = (__nv_bfloat16 *)out, p.norm_max = norm_max, p.status = ctx->status;
    const int grid = p.n_pairs < 148 ? p.n_pairs : 148;
    e = launch_pdl(k_item_tower_tc, dim3(grid), dim3(kTThreads), kTSmem, st, ma, m0, m1, mo, p);
    count_launch();
    return e;
}

}  // namespace aif
