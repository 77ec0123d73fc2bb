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
        const int l4 = lane & 3, r8 = lane >> 2;
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
                // The accumulator is read in the 16x256b shape (a thread owns two adjacent columns of every eight over
                // four rows): eight bias values per thread and 32 columns instead of all 32, which every row thread used
                // to fetch through the shared memory's return path.  The packed pairs go back in the matching 16x128b
                // shape.  A chunk's pairs land on columns the whole warp has read (its loads are complete before any
                // of its stores is issued, and the chunk in flight lies further right).
                uint32_t ra[2][16], rb[2][16];
                auto fetch = [&](uint32_t (&r)[2][16], int c) {
                    tmem_ld16x256(col0 + (uint32_t)(32 * c), r[0]);
                    tmem_ld16x256(col0 + (16u << 16) + (uint32_t)(32 * c), r[1]);
                };
                auto finish = [&](const uint32_t (&r)[2][16], int c) {
                    uint64_t bias2[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) bias2[j] = *reinterpret_cast<const uint64_t *>(b0_s + 32 * c + 8 * j + 2 * l4);
                    const __nv_bfloat162 zero2 = __float2bfloat162_rn(0.f);
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        uint32_t packed[8];
#pragma unroll
                        for (int k = 0; k < 8; ++k) {   // k = 2 j + q
                            float x0, x1;
                            unpack_f32x2(add_f32x2(pack_f32x2(__uint_as_float(r[hh][2 * k]), __uint_as_float(r[hh][2 * k + 1])), bias2[k >> 1]), x0, x1);
                            const __nv_bfloat162 h = __hmax2(__floats2bfloat162_rn(x0, x1), zero2);   // ReLU on the rounded pair: same result
                            packed[k] = *reinterpret_cast<const uint32_t *>(&h);
                        }
                        tmem_st16x128(col0 + ((uint32_t)(16 * hh) << 16) + (uint32_t)(16 * c), packed);
                    }
                };
                const int nc = p.hI >> 5;   // even
                fetch(ra, 0);
#pragma unroll 1
                for (int c = 0; c < nc; c += 2) {
                    tmem_ld_wait();
                    fetch(rb, c + 1);
                    finish(ra, c);
                    tmem_ld_wait();
                    if (c + 2 < nc) fetch(ra, c + 2);
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
            // the same shape: rows r8 + 8 i (i = 0..3) of this warp's 32, two columns of every eight; the 32 x 32 block goes
            // through the staging slab (64-byte swizzle, 4-byte stores, conflict-free) and leaves as one tile store
            float ss[4] = {0.f, 0.f, 0.f, 0.f};   // this thread's share of the squared norms of its four rows
            for (int c0 = 0; c0 < p.d; c0 += 32) {
                uint32_t r[2][16];
                tmem_ld16x256(col0 + (uint32_t)(128 + c0), r[0]);
                tmem_ld16x256(col0 + (16u << 16) + (uint32_t)(128 + c0), r[1]);
                uint64_t bias2[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) bias2[j] = *reinterpret_cast<const uint64_t *>(b1_s + c0 + 8 * j + 2 * l4);
                tmem_ld_wait();
                if (c0 + 32 >= p.d) {   // the accumulators of this pair are in registers: the next pair may overwrite them
                    tc_fence_before();
                    mbar_arrive(bar(TB_TM_FREE));
                }
                if (lane == 0) bulk_wait_read<0>();   // the store that last read the slab is done with it
                __syncwarp();
#pragma unroll
                for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                    for (int k = 0; k < 8; ++k) {   // k = 2 j + q
                        float x0, x1;
                        unpack_f32x2(add_f32x2(pack_f32x2(__uint_as_float(r[hh][2 * k]), __uint_as_float(r[hh][2 * k + 1])), bias2[k >> 1]), x0, x1);
                        ss[2 * hh + (k & 1)] = fmaf(x0, x0, fmaf(x1, x1, ss[2 * hh + (k & 1)]));
                        const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
                        const int rr = 16 * hh + r8 + 8 * (k & 1), j = k >> 1;
                        *reinterpret_cast<uint32_t *>(sb + rr * 64 + ((j ^ ((rr >> 1) & 3)) << 4) + 4 * l4) = *reinterpret_cast<const uint32_t *>(&h);
                    }
                if (whole) {
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&tmapOut, smem_u32(sb), c0, (int)(row0 + wq * 32));
                        bulk_commit();
                    }
                } else {
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int rr = 8 * j + (lane >> 2), q = lane & 3;
                        const uint4 v = *reinterpret_cast<const uint4 *>(sb + rr * 64 + ((q ^ ((rr >> 1) & 3)) << 4));
                        if (row0 + wq * 32 + rr < p.n) *reinterpret_cast<uint4 *>(p.out + (size_t)(row0 + wq * 32 + rr) * p.d + c0 + q * 8) = v;
                    }
                    __syncwarp();
                }
            }
            if (p.norm_max) {
                // non-negative floats order like their bit patterns; a NaN row gives a pattern above every finite one
                int best = 0;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float v = ss[i];
                    v += __shfl_xor_sync(0xffffffffu, v, 1);
                    v += __shfl_xor_sync(0xffffffffu, v, 2);
                    const int rr = 16 * (i >> 1) + r8 + 8 * (i & 1);
                    if (row0 + wq * 32 + rr < p.n) best = max(best, __float_as_int(sqrtf(v) * 1.00390625f) & 0x7fffffff);
                }
                best = __reduce_max_sync(0xffffffffu, best);
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
