// Token -> adapter grouping (Sec. 3.3): histogram, exclusive prefix sum and the stable
// permutation of the T*k (token, pick) slots by adapter index.  Integer work only.
//
// One CTA walks the slots in tiles of 1024.  Inside a tile the rank of a slot among the
// slots with the same key is: (slots with that key in earlier tiles) + (in earlier warps
// of this tile) + (in lower lanes of this warp, from __match_any_sync).  All three terms
// count slots with a smaller slot number, so equal keys keep ascending slot order.
#include "common.cuh"

namespace meteora {

constexpr int kRouteThreads = 1024;
constexpr int kRouteWarps = kRouteThreads / 32;

__global__ void __launch_bounds__(kRouteThreads)
k_route(const int32_t* __restrict__ topk_idx, int S, int N, int32_t* __restrict__ counts,
        int32_t* __restrict__ offsets, int32_t* __restrict__ perm) {
    __shared__ int hist[METEORA_MAX_N];
    __shared__ int running[METEORA_MAX_N];                // next free position of every adapter's group
    __shared__ int warp_cnt[kRouteWarps][METEORA_MAX_N];  // per tile: count, then base, per (warp, key)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (tid < METEORA_MAX_N) hist[tid] = 0;
    __syncthreads();
    for (int s = tid; s < S; s += kRouteThreads) {
        const int key = min(max(topk_idx[s], 0), N - 1);
        atomicAdd(&hist[key], 1);
    }
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        for (int e = 0; e < N; ++e) {
            counts[e] = hist[e];
            offsets[e] = acc;
            running[e] = acc;
            acc += hist[e];
        }
        offsets[N] = acc;
    }
    __syncthreads();

    for (int base = 0; base < S; base += kRouteThreads) {
        const int s = base + tid;
        const bool live = s < S;
        const int key = live ? min(max(topk_idx[s], 0), N - 1) : -1 - lane;  // dead lanes match nobody
        for (int e = lane; e < N; e += 32) warp_cnt[warp][e] = 0;
        __syncwarp();
        const unsigned peers = __match_any_sync(0xFFFFFFFFu, key);
        const int rank_in_warp = __popc(peers & ((1u << lane) - 1u));
        if (live && rank_in_warp == 0) warp_cnt[warp][key] = __popc(peers);
        __syncthreads();
        if (tid < N) {
            int acc = running[tid];
            for (int w = 0; w < kRouteWarps; ++w) {
                const int c = warp_cnt[w][tid];
                warp_cnt[w][tid] = acc;
                acc += c;
            }
            running[tid] = acc;
        }
        __syncthreads();
        if (live) perm[warp_cnt[warp][key] + rank_in_warp] = s;
        __syncthreads();
    }
}

int launch_route(const int32_t* topk_idx, int T, int k, int N, int32_t* counts, int32_t* offsets, int32_t* perm,
                 cudaStream_t st) {
    k_route<<<1, kRouteThreads, 0, st>>>(topk_idx, T * k, N, counts, offsets, perm);
    return last_launch_status();
}

}  // namespace meteora
