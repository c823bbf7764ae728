// Gradient of the gate weights Wg through Eq. 3 (softmax over the selected logits, temperature of App. A.5) and
// Eq. 2 (Sec. 3.2: the base model and the adapters are fixed, only the gating networks are trained).
//
//   g[t,j]      = < dy_t, B_e (A_e x_t) > = < B_e^T dy_t, A_e x_t >,  e = topk_idx[t,j]     (two rank-r vectors)
//   dlogit[t,j] = w[t,j] * (g[t,j] - sum_m w[t,m] g[t,m]) / tau
//   dWg[e,:]    = sum over the slots (t,j) that picked e of dlogit[t,j] * x_t
//
// Three kernels: a warp per slot for g; a thread per token for dlogit; then, with the slots bucketed by adapter
// (meteora_route's stable permutation, Sec. 3.3), a CTA per (adapter, 256 columns of d_in) adds its bucket in
// permutation order, so the result does not depend on scheduling and needs no atomics.
#include "common.cuh"

namespace meteora {

// g of one slot per warp.  Both rank-r vectors are built 8 entries at a time.
template <typename TI>
__global__ void __launch_bounds__(256)
k_gate_grad_slots(const TI* __restrict__ x, const TI* __restrict__ A, const TI* __restrict__ B,
                  const TI* __restrict__ dy, const int32_t* __restrict__ topk_idx, int S, int d_in, int d_out, int N,
                  int r, int k, float* __restrict__ g) {
    const int lane = threadIdx.x & 31;
    const int s = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (s >= S) return;
    const int e = min(max(topk_idx[s], 0), N - 1);
    const int t = s / k;
    const TI* xt = x + (size_t)t * d_in;
    const TI* dyt = dy + (size_t)t * d_out;
    const TI* Ae = A + (size_t)e * r * d_in;
    const TI* Be = B + (size_t)e * d_out * r;
    const bool vec_in = (d_in % 8) == 0;
    float total = 0.f;
    for (int p0 = 0; p0 < r; p0 += 8) {
        const int np = min(8, r - p0);
        // z[p] = sum_o B_e[o, p0 + p] * dy_t[o]: lanes stride over the output rows
        float z[8];
#pragma unroll
        for (int p = 0; p < 8; ++p) z[p] = 0.f;
        for (int o = lane; o < d_out; o += 32) {
            const float dv = to_f32(dyt[o]);
            const TI* brow = Be + (size_t)o * r + p0;
            if ((r & 7) == 0) {                                  // whole 8-entry chunks: one or two 128-bit loads
                float bv[8];
                load8(brow, bv);
#pragma unroll
                for (int p = 0; p < 8; ++p) z[p] = fmaf(bv[p], dv, z[p]);
            } else {
#pragma unroll
                for (int p = 0; p < 8; ++p)
                    if (p < np) z[p] = fmaf(to_f32(brow[p]), dv, z[p]);
            }
        }
#pragma unroll
        for (int p = 0; p < 8; ++p) z[p] = warp_sum(z[p]);
        // u[p] = A_e[p0 + p, :] . x_t
        for (int p = 0; p < np; ++p) {
            const float u = warp_dot(xt, Ae + (size_t)(p0 + p) * d_in, d_in, lane, vec_in);
            total = fmaf(u, z[p], total);
        }
    }
    if (lane == 0) g[s] = total;
}

// dlogit[t,j] = w_j (g_j - sum_m w_m g_m) / tau; one thread per token.
__global__ void k_gate_dlogit(const float* __restrict__ g, const float* __restrict__ topk_w, int T, int k,
                              float inv_tau, float* __restrict__ dlogit) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    float mean = 0.f;
    for (int j = 0; j < k; ++j) mean = fmaf(topk_w[(size_t)t * k + j], g[(size_t)t * k + j], mean);
    for (int j = 0; j < k; ++j)
        dlogit[(size_t)t * k + j] = topk_w[(size_t)t * k + j] * (g[(size_t)t * k + j] - mean) * inv_tau;
}

// dWg[e, d] = sum over the adapter's bucket, in permutation order, of dlogit[slot] * x[token(slot), d].
template <typename TI>
__global__ void __launch_bounds__(256)
k_gate_dwg(const TI* __restrict__ x, const float* __restrict__ dlogit, const int32_t* __restrict__ offsets,
           const int32_t* __restrict__ perm, int d_in, int k, float* __restrict__ dWg) {
    const int e = blockIdx.x;
    const int d = blockIdx.y * 256 + threadIdx.x;
    if (d >= d_in) return;
    const int p0 = offsets[e], p1 = offsets[e + 1];
    float acc = 0.f;
    for (int p = p0; p < p1; ++p) {
        const int s = perm[p];
        acc = fmaf(dlogit[s], to_f32(x[(size_t)(s / k) * d_in + d]), acc);
    }
    dWg[(size_t)e * d_in + d] = acc;
}

int launch_gate_backward(const void* x, const void* A, const void* B, const void* dy, const int32_t* topk_idx,
                         const float* topk_w, const meteora_shape_t& s, float* g, float* dlogit, int32_t* counts,
                         int32_t* offsets, int32_t* perm, float* dWg, cudaStream_t st) {
    const int S = s.T * s.k;
    int rc;
    if (s.T == 0) return cuda_status(cudaMemsetAsync(dWg, 0, (size_t)s.N * s.d_in * sizeof(float), st));
    if (s.dtype == METEORA_BF16)
        k_gate_grad_slots<__nv_bfloat16><<<(S + 7) / 8, 256, 0, st>>>(
            (const __nv_bfloat16*)x, (const __nv_bfloat16*)A, (const __nv_bfloat16*)B, (const __nv_bfloat16*)dy,
            topk_idx, S, s.d_in, s.d_out, s.N, s.r, s.k, g);
    else
        k_gate_grad_slots<float><<<(S + 7) / 8, 256, 0, st>>>((const float*)x, (const float*)A, (const float*)B,
                                                               (const float*)dy, topk_idx, S, s.d_in, s.d_out, s.N,
                                                               s.r, s.k, g);
    if ((rc = last_launch_status()) != METEORA_OK) return rc;
    k_gate_dlogit<<<(s.T + 255) / 256, 256, 0, st>>>(g, topk_w, s.T, s.k, 1.0f / s.temperature, dlogit);
    if ((rc = last_launch_status()) != METEORA_OK) return rc;
    if ((rc = launch_route(topk_idx, s.T, s.k, s.N, counts, offsets, perm, st)) != METEORA_OK) return rc;
    const dim3 grid(s.N, (s.d_in + 255) / 256);
    if (s.dtype == METEORA_BF16)
        k_gate_dwg<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)x, dlogit, offsets, perm, s.d_in, s.k, dWg);
    else
        k_gate_dwg<float><<<grid, 256, 0, st>>>((const float*)x, dlogit, offsets, perm, s.d_in, s.k, dWg);
    return last_launch_status();
}

}  // namespace meteora
