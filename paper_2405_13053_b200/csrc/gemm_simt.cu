// Plain CUDA-core path for the base product of Eq. 2 with the LoRA expand fused in its epilogue:
//   y[t,o] = sum_d W0[o,d] x[t,d] + sum_j sum_p B[idx[t,j], o, p] * uw[t,j,p]       (uw already holds w_j * A x)
// It serves fp32 layers (the tensor cores would round fp32 inputs to tf32) and every shape the
// TMA/tcgen05 path does not take.  fp32 accumulation throughout, one rounding of y.
#include "common.cuh"

namespace meteora {

constexpr int kTile = 64;   // tokens x outputs per CTA
constexpr int kBK = 16;

__device__ __forceinline__ void store_out(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

template <typename TI>
__global__ void __launch_bounds__(256)
k_gemm_simt(const TI* __restrict__ x, const TI* __restrict__ W0, const TI* __restrict__ B,
            const int32_t* __restrict__ topk_idx, const float* __restrict__ uw, int T, int d_in, int d_out, int N,
            int r, int k, TI* __restrict__ y) {
    __shared__ float sx[kBK][kTile + 4];
    __shared__ float sw[kBK][kTile + 4];
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;   // tx: outputs, ty: tokens
    const int t0 = blockIdx.x * kTile, o0 = blockIdx.y * kTile;
    float acc[4][4] = {};

    for (int d0 = 0; d0 < d_in; d0 += kBK) {
        for (int i = tid; i < kTile * kBK; i += 256) {
            const int row = i / kBK, c = i - row * kBK;
            const int d = d0 + c;
            const int t = t0 + row, o = o0 + row;
            sx[c][row] = (t < T && d < d_in) ? to_f32(x[(size_t)t * d_in + d]) : 0.f;
            sw[c][row] = (o < d_out && d < d_in) ? to_f32(W0[(size_t)o * d_in + d]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int c = 0; c < kBK; ++c) {
            float xv[4], wv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                xv[i] = sx[c][ty * 4 + i];
                wv[i] = sw[c][tx * 4 + i];
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(xv[i], wv[j], acc[i][j]);
        }
        __syncthreads();
    }

    for (int i = 0; i < 4; ++i) {
        const int t = t0 + ty * 4 + i;
        if (t >= T) continue;
        for (int j = 0; j < 4; ++j) {
            const int o = o0 + tx * 4 + j;
            if (o >= d_out) continue;
            float out = acc[i][j];
            for (int q = 0; q < k; ++q) {
                const int e = min(max(topk_idx[(size_t)t * k + q], 0), N - 1);
                const TI* brow = B + ((size_t)e * d_out + o) * r;
                const float* uq = uw + ((size_t)t * k + q) * r;
                float d = 0.f;
                for (int p = 0; p < r; ++p) d = fmaf(to_f32(brow[p]), uq[p], d);
                out += d;
            }
            store_out(&y[(size_t)t * d_out + o], out);
        }
    }
}

int launch_gemm_simt(const void* x, const void* W0, const void* B, const int32_t* topk_idx, const float* uw,
                     const meteora_shape_t& s, void* y, cudaStream_t st) {
    if (s.T == 0) return METEORA_OK;
    dim3 grid((s.T + kTile - 1) / kTile, (s.d_out + kTile - 1) / kTile);
    if (s.dtype == METEORA_BF16)
        k_gemm_simt<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)W0,
                                                          (const __nv_bfloat16*)B, topk_idx, uw, s.T, s.d_in, s.d_out,
                                                          s.N, s.r, s.k, (__nv_bfloat16*)y);
    else
        k_gemm_simt<float><<<grid, 256, 0, st>>>((const float*)x, (const float*)W0, (const float*)B, topk_idx, uw, s.T,
                                                  s.d_in, s.d_out, s.N, s.r, s.k, (float*)y);
    return last_launch_status();
}

}  // namespace meteora
