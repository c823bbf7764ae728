// Low-rank shrink (x A_i) and expand ((x A_i) B_i, weighted and summed over the picks) of Eq. 2
// on CUDA cores.  The shrink has two forms:
//   - adapter by adapter over the grouped slots (Sec. 3.3 grouping from meteora_route): a CTA
//     takes up to kSegSlots slots of ONE adapter, stages that adapter's A_i in shared memory
//     chunk by chunk and reuses it for all its slots;
//   - slot by slot in token order (one warp per (token, pick)), used by the plain forward path.
// The expand is token-major and sums the k picks in pick order, so it needs no atomics.
#include "common.cuh"

namespace meteora {

constexpr int kSegSlots = 32;    // slots of one adapter per CTA
constexpr int kSegWarps = 8;
constexpr int kSegSlotsPerWarp = kSegSlots / kSegWarps;
constexpr int kSegRows = 8;      // adapter rows (rank entries) staged at a time
constexpr int kSegChunkBytes = 32 * 1024;

template <typename TI>
__global__ void __launch_bounds__(kSegWarps * 32)
k_shrink_segments(const TI* __restrict__ x, const TI* __restrict__ A, const int32_t* __restrict__ offsets,
                  const int32_t* __restrict__ perm, int d_in, int N, int r, int k, float* __restrict__ u) {
    constexpr int DC = kSegChunkBytes / (kSegRows * (int)sizeof(TI));  // elements of d_in per staged chunk
    __shared__ __align__(16) TI sA[kSegRows][DC];
    __shared__ int s_tile[3];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (tid == 0) {  // which (adapter, tile of its group) is this CTA?
        int b = blockIdx.x, e = 0;
        for (; e < N; ++e) {
            const int c = offsets[e + 1] - offsets[e];
            const int nt = (c + kSegSlots - 1) / kSegSlots;
            if (b < nt) break;
            b -= nt;
        }
        s_tile[0] = e < N ? e : -1;
        if (e < N) {
            s_tile[1] = offsets[e] + b * kSegSlots;
            s_tile[2] = min(offsets[e + 1], s_tile[1] + kSegSlots);
        }
    }
    __syncthreads();
    const int e = s_tile[0];
    if (e < 0) return;
    const int p_begin = s_tile[1], p_end = s_tile[2];
    const bool vec = (d_in % 8) == 0;

    int slot[kSegSlotsPerWarp];
#pragma unroll
    for (int i = 0; i < kSegSlotsPerWarp; ++i) {
        const int p = p_begin + warp + i * kSegWarps;
        slot[i] = p < p_end ? perm[p] : -1;
    }

    for (int r0 = 0; r0 < r; r0 += kSegRows) {
        const int rows = min(kSegRows, r - r0);
        float acc[kSegSlotsPerWarp][kSegRows];
#pragma unroll
        for (int i = 0; i < kSegSlotsPerWarp; ++i)
#pragma unroll
            for (int q = 0; q < kSegRows; ++q) acc[i][q] = 0.f;

        for (int d0 = 0; d0 < d_in; d0 += DC) {
            const int len = min(DC, d_in - d0);
            __syncthreads();  // previous chunk fully consumed
            const TI* src = A + ((size_t)e * r + r0) * d_in + d0;
            if (vec) {
                const int vec_per_row = len / 8;
                for (int v = tid; v < rows * vec_per_row; v += kSegWarps * 32) {
                    const int q = v / vec_per_row, c = v - q * vec_per_row;
                    if (sizeof(TI) == 2) {
                        *reinterpret_cast<uint4*>(&sA[q][c * 8]) =
                            *reinterpret_cast<const uint4*>(src + (size_t)q * d_in + c * 8);
                    } else {
                        *reinterpret_cast<float4*>(&sA[q][c * 8]) =
                            *reinterpret_cast<const float4*>(src + (size_t)q * d_in + c * 8);
                        *reinterpret_cast<float4*>(&sA[q][c * 8 + 4]) =
                            *reinterpret_cast<const float4*>(src + (size_t)q * d_in + c * 8 + 4);
                    }
                }
            } else {
                for (int v = tid; v < rows * len; v += kSegWarps * 32) {
                    const int q = v / len, c = v - q * len;
                    sA[q][c] = src[(size_t)q * d_in + c];
                }
            }
            __syncthreads();
#pragma unroll
            for (int i = 0; i < kSegSlotsPerWarp; ++i) {
                if (slot[i] < 0) continue;
                const TI* xt = x + (size_t)(slot[i] / k) * d_in + d0;
                if (vec) {
                    // all of the slot's x values of this chunk first (one round trip to memory instead of one
                    // per 256 columns), then the products against the staged rows
                    constexpr int NV = DC / 256;
                    float xv[NV][8];
#pragma unroll
                    for (int v = 0; v < NV; ++v) {
                        const int d = lane * 8 + v * 256;
                        if (d < len) {
                            load8(xt + d, xv[v]);
                        } else {
#pragma unroll
                            for (int c = 0; c < 8; ++c) xv[v][c] = 0.f;
                        }
                    }
#pragma unroll
                    for (int v = 0; v < NV; ++v) {
                        const int d = lane * 8 + v * 256;
                        if (d < len) {
#pragma unroll
                            for (int q = 0; q < kSegRows; ++q) {
                                if (q < rows) {
                                    float av[8];
                                    load8(&sA[q][d], av);
#pragma unroll
                                    for (int c = 0; c < 8; ++c) acc[i][q] = fmaf(av[c], xv[v][c], acc[i][q]);
                                }
                            }
                        }
                    }
                } else {
                    for (int d = lane; d < len; d += 32) {
                        const float xv = to_f32(xt[d]);
#pragma unroll
                        for (int q = 0; q < kSegRows; ++q)
                            if (q < rows) acc[i][q] = fmaf(to_f32(sA[q][d]), xv, acc[i][q]);
                    }
                }
            }
        }
#pragma unroll
        for (int i = 0; i < kSegSlotsPerWarp; ++i) {
#pragma unroll
            for (int q = 0; q < kSegRows; ++q) {
                const float v = warp_sum(acc[i][q]);
                if (lane == 0 && slot[i] >= 0 && q < rows) u[(size_t)slot[i] * r + r0 + q] = v;
            }
        }
    }
}

// One warp per slot (t, j): uw[t,j,:] = w[t,j] * A[idx[t,j]] x[t].
template <typename TI>
__global__ void __launch_bounds__(256)
k_shrink_tokens(const TI* __restrict__ x, const TI* __restrict__ A, const int32_t* __restrict__ topk_idx,
                const float* __restrict__ topk_w, int S, int d_in, int N, int r, int k, float* __restrict__ uw) {
    const int lane = threadIdx.x & 31;
    const int s = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (s >= S) return;
    const int e = min(max(topk_idx[s], 0), N - 1);
    const float w = topk_w[s];
    const bool vec = (d_in % 8) == 0;
    const TI* xt = x + (size_t)(s / k) * d_in;
    for (int p = 0; p < r; ++p) {
        const float v = warp_dot(xt, A + ((size_t)e * r + p) * d_in, d_in, lane, vec);
        if (lane == 0) uw[(size_t)s * r + p] = w * v;
    }
}

// delta[t,o] = sum_j w[t,j] * sum_p B[idx[t,j], o, p] * u[t*k + j, p].   One thread per output row o,
// kExpTokens tokens per CTA so that the B rows of an adapter picked by several of them stay in L1.
constexpr int kExpTokens = 8;
constexpr int kExpThreads = 256;

template <typename TI>
__global__ void __launch_bounds__(kExpThreads)
k_expand(const TI* __restrict__ B, const int32_t* __restrict__ topk_idx, const float* __restrict__ topk_w,
         const float* __restrict__ u, int T, int d_out, int N, int r, int k, float* __restrict__ delta) {
    __shared__ int s_idx[kExpTokens * METEORA_MAX_K];
    __shared__ float s_w[kExpTokens * METEORA_MAX_K];
    __shared__ float s_u[kExpTokens * METEORA_MAX_K * METEORA_MAX_R];
    const int t0 = blockIdx.x * kExpTokens;
    const int nt = min(kExpTokens, T - t0);
    for (int i = threadIdx.x; i < nt * k; i += kExpThreads) {
        s_idx[i] = min(max(topk_idx[(size_t)t0 * k + i], 0), N - 1);
        s_w[i] = topk_w[(size_t)t0 * k + i];
    }
    for (int i = threadIdx.x; i < nt * k * r; i += kExpThreads) s_u[i] = u[(size_t)t0 * k * r + i];
    __syncthreads();
    const int o = blockIdx.y * kExpThreads + threadIdx.x;
    if (o >= d_out) return;
    const bool vec = (r % 8) == 0;
    for (int tt = 0; tt < nt; ++tt) {
        float out = 0.f;
        for (int j = 0; j < k; ++j) {
            const TI* brow = B + ((size_t)s_idx[tt * k + j] * d_out + o) * r;
            const float* uj = &s_u[(tt * k + j) * r];
            float acc = 0.f;
            if (vec) {
                for (int p = 0; p < r; p += 8) {
                    float bv[8];
                    load8(brow + p, bv);
#pragma unroll
                    for (int c = 0; c < 8; ++c) acc = fmaf(bv[c], uj[p + c], acc);
                }
            } else {
                for (int p = 0; p < r; ++p) acc = fmaf(to_f32(brow[p]), uj[p], acc);
            }
            out = fmaf(s_w[tt * k + j], acc, out);
        }
        delta[(size_t)(t0 + tt) * d_out + o] = out;
    }
}

int launch_shrink_segments(const void* x, const void* A, const int32_t* offsets, const int32_t* perm,
                           const meteora_shape_t& s, float* u, cudaStream_t st) {
    if (s.T == 0) return METEORA_OK;
    const int S = s.T * s.k;
    const int blocks = (S + kSegSlots - 1) / kSegSlots + s.N;  // upper bound of sum_e ceil(count_e / kSegSlots)
    if (s.dtype == METEORA_BF16)
        k_shrink_segments<__nv_bfloat16><<<blocks, kSegWarps * 32, 0, st>>>(
            (const __nv_bfloat16*)x, (const __nv_bfloat16*)A, offsets, perm, s.d_in, s.N, s.r, s.k, u);
    else
        k_shrink_segments<float><<<blocks, kSegWarps * 32, 0, st>>>((const float*)x, (const float*)A, offsets, perm,
                                                                    s.d_in, s.N, s.r, s.k, u);
    return last_launch_status();
}

int launch_shrink_tokens(const void* x, const void* A, const int32_t* topk_idx, const float* topk_w,
                         const meteora_shape_t& s, float* uw, cudaStream_t st) {
    if (s.T == 0) return METEORA_OK;
    const int S = s.T * s.k;
    const int blocks = (S + 7) / 8;
    if (s.dtype == METEORA_BF16)
        k_shrink_tokens<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)A,
                                                                topk_idx, topk_w, S, s.d_in, s.N, s.r, s.k, uw);
    else
        k_shrink_tokens<float><<<blocks, 256, 0, st>>>((const float*)x, (const float*)A, topk_idx, topk_w, S, s.d_in,
                                                        s.N, s.r, s.k, uw);
    return last_launch_status();
}

int launch_expand(const void* B, const int32_t* topk_idx, const float* topk_w, const float* u,
                  const meteora_shape_t& s, float* delta, cudaStream_t st) {
    if (s.T == 0) return METEORA_OK;
    dim3 grid((s.T + kExpTokens - 1) / kExpTokens, (s.d_out + kExpThreads - 1) / kExpThreads);
    if (s.dtype == METEORA_BF16)
        k_expand<__nv_bfloat16><<<grid, kExpThreads, 0, st>>>((const __nv_bfloat16*)B, topk_idx, topk_w, u, s.T,
                                                               s.d_out, s.N, s.r, s.k, delta);
    else
        k_expand<float><<<grid, kExpThreads, 0, st>>>((const float*)B, topk_idx, topk_w, u, s.T, s.d_out, s.N, s.r,
                                                       s.k, delta);
    return last_launch_status();
}

}  // namespace meteora
