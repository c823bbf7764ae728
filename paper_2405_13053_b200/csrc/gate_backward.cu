// Gradient of the gate weights Wg through Eq. 3 (softmax over the selected logits, temperature of App. A.5) and
// Eq. 2 (Sec. 3.2: the base model and the adapters are fixed, only the gating networks are trained).
//
//   g[t,j]      = < dy_t, B_e (A_e x_t) > = < B_e^T dy_t, A_e x_t >,  e = topk_idx[t,j]     (two rank-r vectors)
//   dlogit[t,j] = w[t,j] * (g[t,j] - sum_m w[t,m] g[t,m]) / tau
//   dWg[e,:]    = sum over the slots (t,j) that picked e of dlogit[t,j] * x_t
//
// The slots are bucketed by adapter first (meteora_route's stable permutation, Sec. 3.3).  With B transposed,
// B_e^T dy_t is the same product as the shrink A_e x_t, so both rank-r vectors come from one kernel run twice:
//   - bf16 layers the tensor cores take: the stacked shrink of the forward pass ([A_0..A_{N-1}] x for ALL adapters
//     as one dense product, Sec. 3.3), once on (x, A) and once on (dy, B^T); the slots then read their adapter's
//     r columns.  The dense product does N / k times the needed flops and is still several times faster than
//     gathering, as in the forward pass;
//   - otherwise the grouped shrink kernel of the LoRA term (a CTA stages one adapter's rows in shared memory for
//     up to 32 of its slots).
// A warp per token applies the softmax Jacobian, and a CTA per (adapter, 256 columns of d_in) adds its bucket in
// permutation order, so the result does not depend on scheduling and needs no atomics.
//
// Small batches (up to 2048 slots; a decode batch) are bound by the number of dependent launches, not by any of
// them, so they take fewer: no bucketing (each CTA of the last kernel scans the batch's routing for its adapter,
// in token order, which is the bucket's order), both stacked shrinks as one launch, and B^T from the caller when
// it was transposed beforehand (the adapters are fixed, Sec. 3.2: once per model, not once per step).
#include "common.cuh"

#include <algorithm>

namespace meteora {

// Bt[n, p, o] = B[n, o, p]: with the rank entry as the row, B_e^T dy is the same product as the shrink A_e x
// and runs on the same kernel.
template <typename TI>
__global__ void k_transpose_b(const TI* __restrict__ B, TI* __restrict__ Bt, int N, int d_out, int r) {
    const size_t total = (size_t)N * d_out * r;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const size_t n = i / ((size_t)d_out * r), rem = i - n * (size_t)d_out * r;
        const size_t p = rem / d_out, o = rem - p * d_out;          // consecutive threads write consecutive o
        Bt[i] = B[(n * d_out + o) * r + p];
    }
}

// g[t,j] = < B_e^T dy_t, A_e x_t > from the two shrink outputs, then
// dlogit[t,j] = w_j (g_j - sum_m w_m g_m) / tau; one warp per token.  The shrink outputs are either per slot
// (`dense` = 0: u[(t*k + j)*r + p]) or the stacked shrink's rows (`dense` = 1: u[q][t][e*r + p], `zsplits` partial
// copies `zstride` floats apart, row pitch `ld`).  The copies are added in a fixed order: when the rank divides 32,
// lane l adds the copies q = l / r, l / r + 32 / r, .. of entry l % r and the lanes of an entry are then added by
// a butterfly; otherwise each lane adds all copies of its entries in slice order.
__global__ void __launch_bounds__(256)
k_gate_dlogit(const float* __restrict__ u, const float* __restrict__ z, const int32_t* __restrict__ topk_idx,
              const float* __restrict__ topk_w, int T, int N, int k, int r, float inv_tau, int dense, int ld,
              int zsplits_u, int zsplits_z, size_t zstride, float* __restrict__ dlogit, float* __restrict__ dlogit2) {
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * 8 + (threadIdx.x >> 5);
    // launched ahead of the end of the shrinks, and lets the last kernel become resident in turn (no-ops without
    // the launch attribute)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const bool spread = r <= 32 && (32 % r) == 0;
    const int nq = spread ? 32 / r : 1, qg = spread ? lane / r : 0;
    // every load of the token goes out before the first reduction: the picks' adapters and weights (inputs of the
    // call: read while the shrinks still run), then the copies of both shrink outputs for all picks (the kernel is
    // a chain of dependent loads otherwise)
    int e[METEORA_MAX_K];
    float w[METEORA_MAX_K], g[METEORA_MAX_K];
#pragma unroll
    for (int j = 0; j < METEORA_MAX_K; ++j) {
        const bool live = j < k && t < T;
        e[j] = live ? min(max(topk_idx[(size_t)t * k + j], 0), N - 1) : 0;
        w[j] = live ? topk_w[(size_t)t * k + j] : 0.f;
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (t >= T) return;
#pragma unroll
    for (int j = 0; j < METEORA_MAX_K; ++j) {
        g[j] = 0.f;
        if (j >= k) continue;
        const size_t row = dense ? (size_t)t * ld + (size_t)e[j] * r : ((size_t)t * k + j) * r;
        if (spread) {
            const int p = lane - qg * r;
            float uv = 0.f, zv = 0.f;
            for (int q = qg; q < zsplits_u; q += nq) uv += u[q * zstride + row + p];
            for (int q = qg; q < zsplits_z; q += nq) zv += z[q * zstride + row + p];
            for (int o = r; o < 32; o <<= 1) {
                uv += __shfl_xor_sync(0xFFFFFFFFu, uv, o);
                zv += __shfl_xor_sync(0xFFFFFFFFu, zv, o);
            }
            g[j] = qg == 0 ? uv * zv : 0.f;
        } else {
            for (int p = lane; p < r; p += 32) {
                float uv = 0.f, zv = 0.f;
                for (int q = 0; q < zsplits_u; ++q) uv += u[q * zstride + row + p];
                for (int q = 0; q < zsplits_z; ++q) zv += z[q * zstride + row + p];
                g[j] = fmaf(uv, zv, g[j]);
            }
        }
    }
    float mean = 0.f;
#pragma unroll
    for (int j = 0; j < METEORA_MAX_K; ++j) {
        if (j >= k) continue;
        g[j] = warp_sum(g[j]);
        mean = fmaf(w[j], g[j], mean);
    }
    if (lane == 0)
#pragma unroll
        for (int j = 0; j < METEORA_MAX_K; ++j) {
            if (j >= k) continue;
            const float v = w[j] * (g[j] - mean) * inv_tau;
            dlogit[(size_t)t * k + j] = v;
            if (dlogit2) dlogit2[(size_t)t * k + j] = v;
        }
}

// dWg[e, d] = sum over the adapter's bucket of dlogit[slot] * x[token(slot), d].  A CTA owns 256 columns of one
// adapter: warp w adds the bucket's entries w, w + 8, w + 16, ... in that order (8 columns per lane, 128-bit
// loads when the row pitch allows), and the eight partial sums of a column are added in warp order: a fixed
// order whatever the scheduling.
template <typename TI>
__global__ void __launch_bounds__(256)
k_gate_dwg(const TI* __restrict__ x, const float* __restrict__ dlogit, const int32_t* __restrict__ offsets,
           const int32_t* __restrict__ perm, int d_in, int k, float* __restrict__ dWg) {
    __shared__ float part[8][256];
    const int e = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int d0 = blockIdx.y * 256 + lane * 8;
    asm volatile("griddepcontrol.wait;" ::: "memory");               // dlogit comes from the grid before
    const int p0 = offsets[e], p1 = offsets[e + 1];
    const bool vec = (d_in % 8) == 0;
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    for (int p = p0 + warp; p < p1; p += 8) {
        const int s = perm[p];
        const float dl = dlogit[s];
        const TI* row = x + (size_t)(s / k) * d_in + d0;
        if (vec && d0 + 8 <= d_in) {
            float xv[8];
            load8(row, xv);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = fmaf(dl, xv[i], acc[i]);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (d0 + i < d_in) acc[i] = fmaf(dl, to_f32(row[i]), acc[i]);
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) part[warp][lane * 8 + i] = acc[i];
    __syncthreads();
    const int d = blockIdx.y * 256 + threadIdx.x;
    if (d < d_in) {
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) sum += part[w][threadIdx.x];
        dWg[(size_t)e * d_in + d] = sum;
    }
}

// The same sum without the bucketing, for small batches: the CTA of (adapter e, 256 columns) walks the batch's
// routing itself.  Warp w takes the slots [32c, 32c + 32) for c = w, w + 8, ..: each lane reads one slot's adapter,
// a ballot marks those that picked e, and the warp adds them in slot order; the eight partial sums are added in
// warp order.
template <typename TI>
__global__ void __launch_bounds__(256)
k_gate_dwg_scan(const TI* __restrict__ x, const float* __restrict__ dlogit, const int32_t* __restrict__ topk_idx,
                int T, int d_in, int k, float* __restrict__ dWg) {
    __shared__ float part[8][256];
    const int e = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int d0 = blockIdx.y * 256 + lane * 8;
    const bool vec = (d_in % 8) == 0;
    const int slots = T * k;
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    // the routing is an input of the call; dlogit comes from the grid before
    for (int c = warp * 32; c < slots; c += 8 * 32) {
        const int s_lane = c + lane;
        unsigned m = __ballot_sync(0xFFFFFFFFu, s_lane < slots && topk_idx[s_lane] == e);
        if (c == warp * 32) asm volatile("griddepcontrol.wait;" ::: "memory");
        while (m) {
            const int s = c + __ffs(m) - 1;
            m &= m - 1;
            const float dl = dlogit[s];
            const TI* row = x + (size_t)(s / k) * d_in + d0;
            if (vec && d0 + 8 <= d_in) {
                float xv[8];
                load8(row, xv);
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[i] = fmaf(dl, xv[i], acc[i]);
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (d0 + i < d_in) acc[i] = fmaf(dl, to_f32(row[i]), acc[i]);
            }
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");               // (warps without a slot of their own)
#pragma unroll
    for (int i = 0; i < 8; ++i) part[warp][lane * 8 + i] = acc[i];
    __syncthreads();
    const int d = blockIdx.y * 256 + threadIdx.x;
    if (d < d_in) {
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) sum += part[w][threadIdx.x];
        dWg[(size_t)e * d_in + d] = sum;
    }
}

int launch_transpose_b(const void* B, const meteora_shape_t& s, void* Bt, cudaStream_t st) {
    if (s.dtype == METEORA_BF16)
        k_transpose_b<__nv_bfloat16><<<296, 256, 0, st>>>((const __nv_bfloat16*)B, (__nv_bfloat16*)Bt, s.N, s.d_out, s.r);
    else
        k_transpose_b<float><<<296, 256, 0, st>>>((const float*)B, (float*)Bt, s.N, s.d_out, s.r);
    return last_launch_status();
}

// Slots up to which the last kernel scans the routing instead of reading buckets.
constexpr size_t kScanSlots = 2048;

// B == nullptr: Bt already holds the transposed adapters (launch_transpose_b).  dlogit_out: optional second copy.
int launch_gate_backward(const void* x, const void* A, const void* B, const void* dy, const int32_t* topk_idx,
                         const float* topk_w, const meteora_shape_t& s, void* Bt, float* u, float* z, float* dlogit,
                         float* dlogit_out, int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* status,
                         float* dWg, cudaStream_t st) {
    int rc;
    if (s.T == 0) return cuda_status(cudaMemsetAsync(dWg, 0, (size_t)s.N * s.d_in * sizeof(float), st));
    const bool dense = gate_backward_dense(s);
    const bool scan = dense && (size_t)s.T * s.k <= kScanSlots;   // the grouped shrink kernel needs the buckets
    if (!scan && (rc = launch_route(topk_idx, s.T, s.k, s.N, counts, offsets, perm, st)) != METEORA_OK) return rc;
    if (B && (rc = launch_transpose_b(B, s, Bt, st)) != METEORA_OK) return rc;
    meteora_shape_t sb = s;
    sb.d_in = s.d_out;                                           // the contraction of B_e^T dy runs over d_out
    int ld = 0, zs_u = 1, zs_z = 1;
    if (dense && stacked_dual_supported(s)) {
        // u = [A_0; ..; A_{N-1}] x and z = [B_0^T; ..; B_{N-1}^T] dy as one launch: z's columns follow u's
        // (u and z are one contiguous buffer here)
        if ((rc = launch_stacked_dual_tc(x, A, dy, Bt, s, u, status, st)) != METEORA_OK) return rc;
        const int half = (s.N * s.r + 127) / 128 * 128;
        ld = 2 * half;
        z = u + half;
        zs_u = zs_z = stacked_dual_zsplits(s);
    } else if (dense) {
        // each on the tensor cores for every adapter.  The kernel also wants a gate matrix of N rows: the first N
        // rows of the stacked operand stand in, and the N columns they produce are not read.
        Workspace wu = {}, wz = {};
        wu.status = wz.status = status;
        wu.ld_u = wz.ld_u = ld = tc_stacked_pitch(s, &wu.col_logits);
        wz.col_logits = wu.col_logits;
        wu.u_all = u;
        wz.u_all = z;
        if ((rc = launch_stacked_shrink_tc(x, A, A, s, wu, st)) != METEORA_OK) return rc;
        if ((rc = launch_stacked_shrink_tc(dy, Bt, Bt, sb, wz, st)) != METEORA_OK) return rc;
        zs_u = tc_stacked_zsplits(s);
        zs_z = tc_stacked_zsplits(sb);
    } else {
        // adapter by adapter over the bucketed slots
        if ((rc = launch_shrink_segments(x, A, offsets, perm, s, u, st)) != METEORA_OK) return rc;
        if ((rc = launch_shrink_segments(dy, Bt, offsets, perm, sb, z, st)) != METEORA_OK) return rc;
    }
    // The last two kernels are launched programmatically dependent: resident while their predecessor still runs,
    // they wait for it (griddepcontrol.wait) before their first read.
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = tuning().pdl ? 1 : 0;
    cfg.gridDim = dim3((s.T + 7) / 8);
    const float inv_tau = 1.0f / s.temperature;
    const int dense_i = dense ? 1 : 0;
    const size_t zstride = (size_t)s.T * ld;
    const float* uc = u;
    const float* zc = z;
    if ((rc = cuda_status(cudaLaunchKernelEx(&cfg, k_gate_dlogit, uc, zc, topk_idx, topk_w, s.T, s.N, s.k, s.r, inv_tau,
                                             dense_i, ld, zs_u, zs_z, zstride, dlogit, dlogit_out))) != METEORA_OK)
        return rc;
    cfg.gridDim = dim3(s.N, (s.d_in + 255) / 256);
    const float* dlc = dlogit;
    const int32_t* offc = offsets;
    const int32_t* permc = perm;
    if (s.dtype == METEORA_BF16) {
        const __nv_bfloat16* xb = (const __nv_bfloat16*)x;
        return cuda_status(scan ? cudaLaunchKernelEx(&cfg, k_gate_dwg_scan<__nv_bfloat16>, xb, dlc, topk_idx, s.T, s.d_in, s.k, dWg)
                                : cudaLaunchKernelEx(&cfg, k_gate_dwg<__nv_bfloat16>, xb, dlc, offc, permc, s.d_in, s.k, dWg));
    }
    const float* xf = (const float*)x;
    return cuda_status(scan ? cudaLaunchKernelEx(&cfg, k_gate_dwg_scan<float>, xf, dlc, topk_idx, s.T, s.d_in, s.k, dWg)
                            : cudaLaunchKernelEx(&cfg, k_gate_dwg<float>, xf, dlc, offc, permc, s.d_in, s.k, dWg));
}

// Both products of the gate gradient as dense stacked shrinks on the tensor cores?
bool gate_backward_dense(const meteora_shape_t& s) {
    meteora_shape_t sb = s;
    sb.d_in = s.d_out;
    return tc_path_supported(s) && tc_path_supported(sb);
}

// Floats of each of the two shrink outputs: per slot, or the stacked shrink's partial copies.
size_t gate_backward_shrink_floats(const meteora_shape_t& s) {
    const size_t slots = (size_t)s.T * s.k * s.r;
    if (!gate_backward_dense(s)) return slots;
    return std::max(slots, (size_t)s.T * tc_stacked_pitch(s, nullptr) * stacked_zsplits_bound(s.T));
}

}  // namespace meteora
