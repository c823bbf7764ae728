// Gate logits, top-k selection and softmax over the selected logits (Sec. 3.1, Eq. 3; temperature App. A.5).
//
// One warp owns one token.  Lane l holds the logits l, l + 32, l + 64, l + 96; the k picks are
// taken by k rounds of a warp-wide arg-max whose ordering is (logit descending, index ascending),
// so equal logits always resolve to the lower adapter index.
#include <math_constants.h>

#include "common.cuh"
#include "select.cuh"

namespace meteora {

constexpr int kGateWarps = 8;

template <typename TI>
__global__ void __launch_bounds__(kGateWarps * 32)
k_gate_topk(const TI* __restrict__ x, const TI* __restrict__ Wg, int T, int d_in, int N, int k, float inv_tau,
            int32_t* __restrict__ topk_idx, float* __restrict__ topk_w, float* __restrict__ logits) {
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * kGateWarps + (threadIdx.x >> 5);
    if (t >= T) return;
    const bool vec = (d_in % 8) == 0;
    const TI* xt = x + (size_t)t * d_in;
    float v[kSelVals];
#pragma unroll
    for (int i = 0; i < kSelVals; ++i) v[i] = 0.f;
    for (int n = 0; n < N; ++n) {
        const float l = warp_dot(xt, Wg + (size_t)n * d_in, d_in, lane, vec);
#pragma unroll
        for (int i = 0; i < kSelVals; ++i)
            if (n == lane + 32 * i) v[i] = l;
    }
    if (logits) {
#pragma unroll
        for (int i = 0; i < kSelVals; ++i)
            if (lane + 32 * i < N) logits[(size_t)t * N + lane + 32 * i] = v[i];
    }
    int idx;
    float w;
    warp_topk_softmax(v, N, k, inv_tau, lane, idx, w);
    if (lane < k) {
        topk_idx[(size_t)t * k + lane] = idx;
        topk_w[(size_t)t * k + lane] = w;
    }
}

// The same gate for long rows (d_in a multiple of 8, at least 512): a block of 8 warps owns TT tokens and cuts the
// contraction axis into chunks of 256 elements dealt to the warps, so that a decode batch of 128 tokens fills 128 SMs
// instead of 16 (one warp per token left most of the machine idle: 63 us at 4096 -> 28 logits, 128 tokens) and a row
// of Wg is read once per TT tokens.  Per-warp partial logits meet in shared memory and are added in warp order by
// the warp that then selects for the token.
template <typename TI, int TT>
__global__ void __launch_bounds__(kGateWarps * 32)
k_gate_topk_split(const TI* __restrict__ x, const TI* __restrict__ Wg, int T, int d_in, int N, int k, float inv_tau,
                  int32_t* __restrict__ topk_idx, float* __restrict__ topk_w, float* __restrict__ logits) {
    __shared__ float part[TT][kGateWarps][METEORA_MAX_N];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t0 = blockIdx.x * TT;
    for (int n = 0; n < N; ++n) {
        float acc[TT];
#pragma unroll
        for (int tt = 0; tt < TT; ++tt) acc[tt] = 0.f;
        const TI* wrow = Wg + (size_t)n * d_in;
        for (int d = warp * 256 + lane * 8; d < d_in; d += kGateWarps * 256) {
            float wv[8];
            load8(wrow + d, wv);
#pragma unroll
            for (int tt = 0; tt < TT; ++tt) {
                if (t0 + tt < T) {
                    float xv[8];
                    load8(x + (size_t)(t0 + tt) * d_in + d, xv);
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[tt] = fmaf(wv[i], xv[i], acc[tt]);
                }
            }
        }
#pragma unroll
        for (int tt = 0; tt < TT; ++tt) {
            const float sum = warp_sum(acc[tt]);
            if (lane == 0) part[tt][warp][n] = sum;
        }
    }
    __syncthreads();
    if (warp >= TT || t0 + warp >= T) return;
    const int t = t0 + warp;
    float v[kSelVals];
#pragma unroll
    for (int i = 0; i < kSelVals; ++i) {
        v[i] = 0.f;
        if (lane + 32 * i < N)
            for (int q = 0; q < kGateWarps; ++q) v[i] += part[warp][q][lane + 32 * i];
    }
    if (logits) {
#pragma unroll
        for (int i = 0; i < kSelVals; ++i)
            if (lane + 32 * i < N) logits[(size_t)t * N + lane + 32 * i] = v[i];
    }
    int idx;
    float w;
    warp_topk_softmax(v, N, k, inv_tau, lane, idx, w);
    if (lane < k) {
        topk_idx[(size_t)t * k + lane] = idx;
        topk_w[(size_t)t * k + lane] = w;
    }
}

// Selection from the stacked shrink: row t of u_all holds A_i x for every adapter (N*r values)
// and, from column col_logits on, the N gate logits.  u_all comes as `zsplits` partial copies (slices
// of the contraction axis, zstride floats apart) that are added here in slice order.  Besides the picks and weights this writes
// uw[t,j,:] = w_j * (A_{i_j} x), the activations the base product's epilogue expands.
__global__ void __launch_bounds__(kGateWarps * 32)
k_select_from_stacked(const float* __restrict__ u_all, int ld_u, int col_logits, int zsplits, size_t zstride, int T,
                      int N, int r, int k,
                      float inv_tau, int32_t* __restrict__ topk_idx, float* __restrict__ topk_w,
                      float* __restrict__ uw, int pdl) {
    if (pdl) {
        // Let the dependent launch (the base product) start streaming weights now; wait for the
        // stacked shrink, which produced u_all, before reading it.
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * kGateWarps + (threadIdx.x >> 5);
    if (t >= T) return;
    select_token<false>(u_all, ld_u, col_logits, zsplits, zstride, t, N, r, k, inv_tau, lane, topk_idx, topk_w, uw);
}

int launch_gate_topk(const void* x, const void* Wg, const meteora_shape_t& s, int32_t* topk_idx, float* topk_w,
                     float* logits, cudaStream_t st) {
    if (s.T == 0) return METEORA_OK;
    const int blocks = (s.T + kGateWarps - 1) / kGateWarps;
    const float inv_tau = 1.0f / s.temperature;
    if (s.d_in % 8 == 0 && s.d_in >= 512) {
        // long rows: 8 warps share a token's contraction axis; from 1024 tokens up a block takes 4 tokens per row of Wg
        const bool many = s.T >= 1024;
        const int grid = many ? (s.T + 3) / 4 : s.T;
        if (s.dtype == METEORA_BF16) {
            const __nv_bfloat16 *xb = (const __nv_bfloat16*)x, *gb = (const __nv_bfloat16*)Wg;
            if (many)
                k_gate_topk_split<__nv_bfloat16, 4><<<grid, kGateWarps * 32, 0, st>>>(xb, gb, s.T, s.d_in, s.N, s.k, inv_tau,
                                                                                   topk_idx, topk_w, logits);
            else
                k_gate_topk_split<__nv_bfloat16, 1><<<grid, kGateWarps * 32, 0, st>>>(xb, gb, s.T, s.d_in, s.N, s.k, inv_tau,
                                                                                   topk_idx, topk_w, logits);
        } else {
            const float *xf = (const float*)x, *gf = (const float*)Wg;
            if (many)
                k_gate_topk_split<float, 4><<<grid, kGateWarps * 32, 0, st>>>(xf, gf, s.T, s.d_in, s.N, s.k, inv_tau, topk_idx,
                                                                           topk_w, logits);
            else
                k_gate_topk_split<float, 1><<<grid, kGateWarps * 32, 0, st>>>(xf, gf, s.T, s.d_in, s.N, s.k, inv_tau, topk_idx,
                                                                           topk_w, logits);
        }
        return last_launch_status();
    }
    if (s.dtype == METEORA_BF16)
        k_gate_topk<__nv_bfloat16><<<blocks, kGateWarps * 32, 0, st>>>(
            (const __nv_bfloat16*)x, (const __nv_bfloat16*)Wg, s.T, s.d_in, s.N, s.k, inv_tau, topk_idx, topk_w, logits);
    else
        k_gate_topk<float><<<blocks, kGateWarps * 32, 0, st>>>((const float*)x, (const float*)Wg, s.T, s.d_in, s.N,
                                                               s.k, inv_tau, topk_idx, topk_w, logits);
    return last_launch_status();
}

int launch_select_from_stacked(const float* u_all, int ld_u, int col_logits, int zsplits, const meteora_shape_t& s,
                               int32_t* topk_idx, float* topk_w, float* uw, bool pdl, cudaStream_t st) {
    if (s.T == 0) return METEORA_OK;
    const int blocks = (s.T + kGateWarps - 1) / kGateWarps;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(kGateWarps * 32);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    const float inv_tau = 1.0f / s.temperature;
    cudaError_t e = cudaLaunchKernelEx(&cfg, k_select_from_stacked, u_all, ld_u, col_logits, zsplits,
                                       (size_t)s.T * ld_u, s.T, s.N, s.r, s.k,
                                       inv_tau, topk_idx, topk_w, uw, pdl ? 1 : 0);
    return cuda_status(e);
}

}  // namespace meteora
