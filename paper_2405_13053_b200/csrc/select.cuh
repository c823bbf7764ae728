// Warp-level top-k selection with softmax over the selected logits (Sec. 3.1, Eq. 3; temperature App. A.5),
// and the selection of one token from the stacked shrink.
#pragma once

#include <math_constants.h>

#include "common.cuh"

namespace meteora {

// Logits per lane: lane l holds logit l, l + 32, l + 64, l + 96 (METEORA_MAX_N = 128 adapters).
constexpr int kSelVals = METEORA_MAX_N / 32;

// v[i] = logit[lane + 32 i]; entries at or beyond N are ignored.
// On return lane j < k holds pick j (index and softmax weight).  Every lane runs the same code.
__device__ __forceinline__ void warp_topk_softmax(float (&v)[kSelVals], int N, int k, float inv_tau, int lane,
                                                  int& my_idx, float& my_w) {
    bool taken[kSelVals];
#pragma unroll
    for (int i = 0; i < kSelVals; ++i) {
        taken[i] = lane + 32 * i >= N;
        if (!(v[i] > -CUDART_INF_F)) v[i] = -CUDART_INF_F;  // NaN never wins a comparison; treat it as -inf
        v[i] += 0.f;                                        // -0 becomes +0: equal as floats, and equal as the keys below
    }
    float first = 0.f, sum = 0.f, my_e = 0.f;
    my_idx = 0;
    for (int j = 0; j < k; ++j) {
        float bv = -CUDART_INF_F;
        int bi = 0x7FFFFFFF;
#pragma unroll
        for (int i = 0; i < kSelVals; ++i)                   // ascending index: a later equal value does not replace
            if (!taken[i] && (bi == 0x7FFFFFFF || v[i] > bv)) { bv = v[i]; bi = lane + 32 * i; }
        // Warp-wide arg-max by two reductions instead of a five-step butterfly of shuffles (a third of the latency):
        // the largest value through an order-preserving integer key, then the lowest index among the lanes that hold it.
        const uint32_t bits = __float_as_uint(bv);
        const uint32_t key = (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
        const uint32_t kmax = __reduce_max_sync(0xFFFFFFFFu, key);
        bi = __reduce_min_sync(0xFFFFFFFFu, key == kmax ? bi : 0x7FFFFFFF);
        bv = __uint_as_float((kmax & 0x80000000u) ? (kmax & 0x7FFFFFFFu) : ~kmax);
        bi = min(bi, N - 1);
#pragma unroll
        for (int i = 0; i < kSelVals; ++i)
            if (bi == lane + 32 * i) taken[i] = true;
        if (j == 0) first = bv;
        const float e = expf((bv - first) * inv_tau);
        sum += e;
        if (lane == j) { my_idx = bi; my_e = e; }
    }
    my_w = my_e / sum;
}

// Loads of the stacked-shrink partials: through L1 normally, bypassing it (.cg) when the partials were written
// earlier in the same kernel by other CTAs.
template <bool kCoherent>
__device__ __forceinline__ float ld_part(const float* p) { return kCoherent ? __ldcg(p) : *p; }
template <bool kCoherent>
__device__ __forceinline__ float4 ld_part4(const float4* p) { return kCoherent ? __ldcg(p) : *p; }

// Selection for one token with at most ZMAX partial copies: lane n owns logit n and reads it from every slice,
// the loads issued together (one memory round trip); the slices are added in slice order.
template <bool kCoherent, int ZMAX>
__device__ __forceinline__ void select_token_few(const float* row, int col_logits, int zsplits, size_t zstride,
                                                 int t, int N, int r, int k, float inv_tau, int lane,
                                                 int32_t* topk_idx, float* topk_w, float* uw) {
    float v[kSelVals];
#pragma unroll
    for (int i = 0; i < kSelVals; ++i) {
        v[i] = 0.f;
        if (32 * i < N) {                                   // uniform across the warp
            float part[ZMAX];
#pragma unroll
            for (int z = 0; z < ZMAX; ++z)
                part[z] = (z < zsplits && lane + 32 * i < N) ? ld_part<kCoherent>(row + z * zstride + col_logits + lane + 32 * i) : 0.f;
#pragma unroll
            for (int z = 0; z < ZMAX; ++z) v[i] += part[z];
        }
    }
    int idx;
    float w;
    warp_topk_softmax(v, N, k, inv_tau, lane, idx, w);
    if (lane < k) {
        topk_idx[(size_t)t * k + lane] = idx;
        topk_w[(size_t)t * k + lane] = w;
    }
    for (int c0 = 0; c0 < k * r; c0 += 32) {
        const int c = c0 + lane;
        const int j = min(c / r, k - 1), q = c - j * r;
        const int ij = __shfl_sync(0xFFFFFFFFu, idx, j);
        const float wj = __shfl_sync(0xFFFFFFFFu, w, j);
        float pu[ZMAX];
#pragma unroll
        for (int z = 0; z < ZMAX; ++z)
            pu[z] = (z < zsplits && c < k * r) ? ld_part<kCoherent>(row + z * zstride + ij * r + q) : 0.f;
        float u = 0.f;
#pragma unroll
        for (int z = 0; z < ZMAX; ++z) u += pu[z];
        if (c < k * r) uw[(size_t)t * k * r + c] = wj * u;
    }
}

// Selection for one token (one warp): row t of u_all holds A_i x for every adapter (N*r values) and, from
// column col_logits on, the N gate logits; u_all comes as `zsplits` partial copies (slices of the contraction
// axis, zstride floats apart).  Writes the picks, their weights and uw[t,j,:] = w_j * (A_{i_j} x).
template <bool kCoherent>
__device__ __forceinline__ void select_token(const float* u_all, int ld_u, int col_logits, int zsplits,
                                             size_t zstride, int t, int N, int r, int k, float inv_tau, int lane,
                                             int32_t* topk_idx, float* topk_w, float* uw) {
    const float* row = u_all + (size_t)t * ld_u;
    if (zsplits <= 8) {
        select_token_few<kCoherent, 8>(row, col_logits, zsplits, zstride, t, N, r, k, inv_tau, lane, topk_idx, topk_w, uw);
        return;
    }
    if (zsplits <= 16) {
        select_token_few<kCoherent, 16>(row, col_logits, zsplits, zstride, t, N, r, k, inv_tau, lane, topk_idx, topk_w, uw);
        return;
    }
    if (zsplits <= 32 && r == 8 && k <= 4) {
        // Many partial copies: lane z reads slice z, so all loads of a phase are in flight at once (one
        // memory round trip instead of one per slice); the slices are then added across lanes by a
        // butterfly, the same order for every token and every run.
        const float* mine = row + (size_t)min(lane, zsplits - 1) * zstride;
        const bool live = lane < zsplits;
        float v[kSelVals];
#pragma unroll
        for (int i = 0; i < kSelVals; ++i) v[i] = 0.f;
#pragma unroll
        for (int n0 = 0; n0 < 32 * kSelVals; n0 += 32) {
            if (n0 >= N) break;
            float vals[32];
#pragma unroll
            for (int n = 0; n < 32; ++n) vals[n] = (live && n0 + n < N) ? ld_part<kCoherent>(mine + col_logits + n0 + n) : 0.f;
#pragma unroll
            for (int n = 0; n < 32; ++n) {
                if (n0 + n < N) {                       // uniform across the warp
                    const float sum = warp_sum(vals[n]);
                    if (lane == n) v[n0 / 32] = sum;
                }
            }
        }
        int idx;
        float w;
        warp_topk_softmax(v, N, k, inv_tau, lane, idx, w);
        if (lane < k) {
            topk_idx[(size_t)t * k + lane] = idx;
            topk_w[(size_t)t * k + lane] = w;
        }
        float4 part[4][2];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int ij = __shfl_sync(0xFFFFFFFFu, idx, j);
            const float4* src = reinterpret_cast<const float4*>(mine + ij * 8);
            const bool on = live && j < k;
            part[j][0] = on ? ld_part4<kCoherent>(src) : make_float4(0.f, 0.f, 0.f, 0.f);
            part[j][1] = on ? ld_part4<kCoherent>(src + 1) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        float out = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (j < k) {                                // uniform across the warp
                const float wj = __shfl_sync(0xFFFFFFFFu, w, j);
                const float e[8] = {part[j][0].x, part[j][0].y, part[j][0].z, part[j][0].w,
                                    part[j][1].x, part[j][1].y, part[j][1].z, part[j][1].w};
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const float sum = warp_sum(e[q]);
                    if (lane == j * 8 + q) out = wj * sum;
                }
            }
        }
        if (lane < k * 8) uw[(size_t)t * k * 8 + lane] = out;
        return;
    }
    float v[kSelVals];
#pragma unroll
    for (int i = 0; i < kSelVals; ++i) v[i] = 0.f;
    for (int z = 0; z < zsplits; ++z) {
#pragma unroll
        for (int i = 0; i < kSelVals; ++i)
            if (lane + 32 * i < N) v[i] += ld_part<kCoherent>(row + z * zstride + col_logits + lane + 32 * i);
    }
    int idx;
    float w;
    warp_topk_softmax(v, N, k, inv_tau, lane, idx, w);
    if (lane < k) {
        topk_idx[(size_t)t * k + lane] = idx;
        topk_w[(size_t)t * k + lane] = w;
    }
    for (int c0 = 0; c0 < k * r; c0 += 32) {
        const int c = c0 + lane;
        const int j = min(c / r, k - 1), p = c - j * r;
        const int ij = __shfl_sync(0xFFFFFFFFu, idx, j);
        const float wj = __shfl_sync(0xFFFFFFFFu, w, j);
        if (c < k * r) {
            float u = 0.f;
            for (int z = 0; z < zsplits; ++z) u += ld_part<kCoherent>(row + z * zstride + ij * r + p);
            uw[(size_t)t * k * r + c] = wj * u;
        }
    }
}

}  // namespace meteora
