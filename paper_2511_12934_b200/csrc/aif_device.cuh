// Device-side helpers shared by the CUDA-core and the tensor-core kernels of libaif.
#pragma once

#include "aif_internal.h"

namespace aif {

// ------------------------------------------------------------------------------------------------
// small device helpers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void from_f(float &dst, float v) { dst = v; }
__device__ __forceinline__ void from_f(__nv_bfloat16 &dst, float v) { dst = __float2bfloat16_rn(v); }

// Cross-feature bucket hash: splitmix64 output function of id * golden + field (Section 3.3 leaves the
// candidate attribute open; the id-derived bucket stands in for the category).
__device__ __forceinline__ uint64_t mix64(uint64_t id, uint64_t field)
{
    uint64_t z = id * 0x9E3779B97F4A7C15ull + field;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__device__ __forceinline__ int bucket_of(int id, int f, int B, int mode)
{
    if (mode == AIF_BUCKET_MOD) return id % B;
    return (int)(mix64((uint64_t)id, (uint64_t)f) % (uint64_t)B);
}

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// row (storage type, global) . q (fp32, shared), d a multiple of 8
__device__ __forceinline__ float dot_row(const float *row, const float *q, int d)
{
    float acc = 0.f;
    const float4 *r4 = reinterpret_cast<const float4 *>(row);
    const float4 *q4 = reinterpret_cast<const float4 *>(q);
    for (int k = 0; k < d / 4; ++k) {
        float4 r = __ldg(r4 + k), w = q4[k];
        acc = fmaf(r.x, w.x, acc);
        acc = fmaf(r.y, w.y, acc);
        acc = fmaf(r.z, w.z, acc);
        acc = fmaf(r.w, w.w, acc);
    }
    return acc;
}

__device__ __forceinline__ float dot_row(const __nv_bfloat16 *row, const float *q, int d)
{
    float acc = 0.f;
    const uint4 *r4 = reinterpret_cast<const uint4 *>(row);
    const float4 *q4 = reinterpret_cast<const float4 *>(q);
    for (int k = 0; k < d / 8; ++k) {
        uint4 r = __ldg(r4 + k);
        float4 a = q4[2 * k], b = q4[2 * k + 1];
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&r);
        float2 f0 = __bfloat1622float2(h[0]), f1 = __bfloat1622float2(h[1]);
        float2 f2 = __bfloat1622float2(h[2]), f3 = __bfloat1622float2(h[3]);
        acc = fmaf(f0.x, a.x, acc);
        acc = fmaf(f0.y, a.y, acc);
        acc = fmaf(f1.x, a.z, acc);
        acc = fmaf(f1.y, a.w, acc);
        acc = fmaf(f2.x, b.x, acc);
        acc = fmaf(f2.y, b.y, acc);
        acc = fmaf(f3.x, b.z, acc);
        acc = fmaf(f3.y, b.w, acc);
    }
    return acc;
}

// One warp, one query: streams over the L rows of S in chunks of 32 keys.
//   att  = softmax(q S^T * scale) S      (online softmax; dense target attention and eqs. 2-3)
//   din  = sum_j sim_j S_j, sim_j = matches(sig_q, sigS_j) / lsh_bits      (eqs. 6-8)
//   tiers[t] += #{ j : tier(matches_j) = t }                               (eq. 9; shared-memory counters)
// Lane owns columns lane, lane+32, ... of the outputs (d <= 256).
template <typename T>
__device__ void warp_interact(const float *q, const T *S, int L, int d, float scale, bool do_att, bool do_lsh,
                              bool do_tiers, const uint32_t *sig_q, const uint8_t *sigS, int lsh_bits, int n_tiers,
                              int *tiers, float att[8], float din[8], float *ml_out = nullptr)
{
    const int lane = threadIdx.x & 31, dq = d >> 5, words = lsh_bits >> 5;
    float m = -INFINITY, l = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) att[c] = 0.f, din[c] = 0.f;
    const float inv_bits = do_lsh ? 1.0f / (float)lsh_bits : 0.f;
    for (int j0 = 0; j0 < L; j0 += 32) {
        const int j = j0 + lane;
        const bool valid = j < L;
        float s = -INFINITY, simv = 0.f;
        if (valid) {
            if (do_att) s = dot_row(S + (size_t)j * d, q, d) * scale;
            if (do_lsh) {
                const uint32_t *sj = reinterpret_cast<const uint32_t *>(sigS + (size_t)j * (lsh_bits >> 3));
                int diff = 0;
                for (int w = 0; w < words; ++w) diff += __popc(sig_q[w] ^ __ldg(sj + w));
                const int matches = lsh_bits - diff;
                simv = (float)matches * inv_bits;
                if (do_tiers) {
                    int t = (matches * n_tiers) / lsh_bits;
                    atomicAdd(&tiers[t < n_tiers - 1 ? t : n_tiers - 1], 1);
                }
            }
        }
        float p = 0.f;
        if (do_att) {
            const float m_new = fmaxf(m, warp_max(s));
            const float sc = expf(m - m_new);
            p = valid ? expf(s - m_new) : 0.f;
            l = l * sc + warp_sum(p);
            m = m_new;
#pragma unroll
            for (int c = 0; c < 8; ++c) att[c] *= sc;
        }
        const int cnt = min(32, L - j0);
        for (int jj = 0; jj < cnt; ++jj) {
            const float pj = __shfl_sync(0xffffffffu, p, jj);
            const float sj = __shfl_sync(0xffffffffu, simv, jj);
            const T *row = S + (size_t)(j0 + jj) * d + lane;
#pragma unroll
            for (int c = 0; c < 8; ++c)
                if (c < dq) {
                    const float v = to_f(row[32 * c]);
                    att[c] = fmaf(pj, v, att[c]);
                    din[c] = fmaf(sj, v, din[c]);
                }
        }
    }
    if (do_att) {
        if (ml_out) {   // partial result over a slice of the keys: left unnormalised, with its maximum and sum
            if (lane == 0) ml_out[0] = m, ml_out[1] = l;
        } else {
            const float inv = 1.0f / l;
#pragma unroll
            for (int c = 0; c < 8; ++c) att[c] *= inv;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// tiles of a request: kTile candidates, never across a mini-batch boundary
// ------------------------------------------------------------------------------------------------
__host__ __device__ inline int tiles_of(int n, int tile, int mb)
{
    if (mb <= 0) return (n + tile - 1) / tile;
    const int tpm = (mb + tile - 1) / tile;
    const int full = n / mb, rem = n - full * mb;
    return full * tpm + (rem + tile - 1) / tile;
}

__device__ inline void tile_range(int lt, int n, int tile, int mb, int &start, int &cnt)
{
    if (mb <= 0) {
        start = lt * tile;
        cnt = min(tile, n - start);
        return;
    }
    const int tpm = (mb + tile - 1) / tile;
    const int b = lt / tpm, w = lt - b * tpm;
    start = b * mb + w * tile;
    const int end = min(min(start + tile, (b + 1) * mb), n);
    cnt = end - start;
}

__device__ inline ReqDev find_request(const ScoreLaunch &sl, int t)
{
    if (sl.reqs == nullptr) return sl.single;
    int lo = 0, hi = sl.n_req - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (sl.reqs[mid].tile_begin <= t) lo = mid;
        else hi = mid - 1;
    }
    return sl.reqs[lo];
}


}  // namespace aif
