// Shared declarations of the MeteoRA CUDA library (internal; the public C ABI is include/meteora.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "meteora.h"

namespace meteora {

// ---------------------------------------------------------------------------------------------
// Workspace layout.  Every region starts on a 256-byte boundary.
// ---------------------------------------------------------------------------------------------
constexpr size_t kHeaderBytes = 4096;    // zero-initialised head of every workspace
constexpr int kMaxFusedRowTiles = 960;   // tile counters that fit into the header

struct Workspace {
    int32_t* status;    // [64]  word 0: error flag of bounded device waits; words 1..: where it gave up
    int32_t* topk_idx;  // [T,k]
    float* topk_w;      // [T,k]
    float* uw;          // [T,k,r]   w_j * (A_{i_j} x): the shrunk, gate-weighted activations
    float* u_all;       // [Z][T,ld_u]  stacked shrink: every adapter's A_i x, then the gate logits; Z partial
                        //           copies (slices of the contraction axis) that the selection kernel adds up
    int ld_u;           // row pitch of u_all in floats
    int col_logits;     // first logit column inside a u_all row
    float* part_g;      // fused decode: fp32 partial accumulator tiles of the base product (T <= 256 only)
    int32_t* tile_ctr;  // fused decode: one counter per 128-row tile of d_out (inside the header)
    void* A_pad;        // bf16 layers whose rank is no multiple of 8: A and B zero-padded to the next multiple,
    void* B_pad;        //           [N,r8,d_in] and [N,d_out,r8], rewritten by every call (nullptr otherwise)
    void* x_dev;        // [T,d_in]  staging for the host-buffer entry point
    void* y_dev;        // [T,d_out]
    size_t bytes;       // total
};

Workspace carve_workspace(const meteora_shape_t& s, void* base);

// A bf16 layer whose rank is no multiple of 8 runs on the tensor-core paths with its adapters zero-padded to
// the next multiple of 8 (the padded rank entries contribute exact zeros to Eq. 2).
inline bool rank_pad_applies(const meteora_shape_t& s) {
    return s.dtype == METEORA_BF16 && s.d_in % 8 == 0 && s.r > 0 && s.r % 8 != 0;
}
inline meteora_shape_t rank_padded(const meteora_shape_t& s) {
    meteora_shape_t e = s;
    if (rank_pad_applies(s)) e.r = (s.r + 7) / 8 * 8;
    return e;
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline size_t elem_size(meteora_dtype_t t) { return t == METEORA_BF16 ? 2 : 4; }

// ---------------------------------------------------------------------------------------------
// Kernel launchers (each returns a meteora_status_t).  All pointers are device pointers.
// ---------------------------------------------------------------------------------------------
// gate_topk.cu
int launch_gate_topk(const void* x, const void* Wg, const meteora_shape_t& s, int32_t* topk_idx, float* topk_w,
                     float* logits, cudaStream_t st);
int launch_select_from_stacked(const float* u_all, int ld_u, int col_logits, int zsplits, const meteora_shape_t& s,
                               int32_t* topk_idx, float* topk_w, float* uw, bool pdl, cudaStream_t st);
// route.cu
int launch_gate_backward(const void* x, const void* A, const void* B, const void* dy, const int32_t* topk_idx,
                         const float* topk_w, const meteora_shape_t& s, void* Bt, float* u, float* z, float* dlogit,
                         float* dlogit_out, int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* status,
                         float* dWg, cudaStream_t st);
int launch_transpose_b(const void* B, const meteora_shape_t& s, void* Bt, cudaStream_t st);
bool gate_backward_dense(const meteora_shape_t& s);            // both shrinks as dense products on the tensor cores
size_t gate_backward_shrink_floats(const meteora_shape_t& s);  // floats of each of the two shrink outputs
int launch_route(const int32_t* topk_idx, int T, int k, int N, int32_t* counts, int32_t* offsets, int32_t* perm,
                 cudaStream_t st);
// lora.cu
int launch_shrink_segments(const void* x, const void* A, const int32_t* offsets, const int32_t* perm,
                           const meteora_shape_t& s, float* u, cudaStream_t st);
int launch_shrink_tokens(const void* x, const void* A, const int32_t* topk_idx, const float* topk_w,
                         const meteora_shape_t& s, float* uw, cudaStream_t st);
int launch_expand(const void* B, const int32_t* topk_idx, const float* topk_w, const float* u,
                  const meteora_shape_t& s, float* delta, cudaStream_t st);
// gemm_simt.cu
int launch_gemm_simt(const void* x, const void* W0, const void* B, const int32_t* topk_idx, const float* uw,
                     const meteora_shape_t& s, void* y, cudaStream_t st);
// wgemm_tcgen05.cu
bool tc_path_supported(const meteora_shape_t& s);
int tc_stacked_pitch(const meteora_shape_t& s, int* col_logits);  // row pitch (floats) of u_all
int stacked_zsplits_bound(int T);                                  // upper bound of those copies, sizes the workspace
bool stacked_dual_supported(const meteora_shape_t& s);            // both shrinks of the gate gradient in one launch?
int stacked_dual_zsplits(const meteora_shape_t& s);               // copies of its output
int launch_stacked_dual_tc(const void* x, const void* A, const void* dy, const void* Bt, const meteora_shape_t& s,
                           float* out, int32_t* status, cudaStream_t st);
int tc_stacked_zsplits(const meteora_shape_t& s);                 // copies of u_all the stacked shrink writes (<= 4)
int launch_stacked_shrink_tc(const void* x, const void* A, const void* Wg, const meteora_shape_t& s,
                             const Workspace& ws, cudaStream_t st);
int launch_base_lora_tc(const void* x, const void* W0, const void* B, const meteora_shape_t& s, const Workspace& ws,
                        void* y, bool pdl, cudaStream_t st);

// fused decode kernel (wgemm_tcgen05.cu + decode_fused.cuh)
bool decode_fused_supported(const meteora_shape_t& s);
constexpr int kMaxGroupModules = 4;   // modules per group call (= kMaxGroup of the decode kernel)
// Several modules that share x (their own W0, A, B, Wg, y, d_out and routing scratch) in one launch of the decode kernel.
struct GroupModule {
    const void* W0;
    const void* A;
    const void* B;
    const void* Wg;
    void* y;
    int d_out;
    Workspace ws;       // topk_idx, topk_w, uw, u_all, ld_u, col_logits of this module
};
bool decode_group_supported(const meteora_shape_t& s, const int* d_outs, int n_modules);
int launch_decode_group(const void* x, const GroupModule* mods, int n_modules, const meteora_shape_t& s,
                        int32_t* status, float* part_g, int32_t* tile_ctr, cudaStream_t st);
int describe_plan(const meteora_shape_t& s, char* buf, size_t n);
int set_wait_limit_us(int us);   // limit of the bounded device-side waits on the current device (0: default)
int launch_decode_fused(const void* x, const void* W0, const void* A, const void* B, const void* Wg,
                        const meteora_shape_t& s, const Workspace& ws, void* y, cudaStream_t st);
// streamed decode kernel (wgemm_tcgen05.cu + decode_stream.cuh): up to 128 tokens, two launches resident at a time
bool decode_cluster_supported(const meteora_shape_t& s);
int launch_decode_cluster(const void* x, const void* W0, const void* A, const void* B, const void* Wg,
                          const meteora_shape_t& s, const Workspace& ws, void* y, cudaStream_t st);
bool decode_stream_supported(const meteora_shape_t& s);
int launch_decode_stream(const void* x, const void* W0, const void* A, const void* B, const void* Wg,
                         const meteora_shape_t& s, const Workspace& ws, void* y, cudaStream_t st);

struct Tuning {
    int splits = 0;
    int stages = 0;
    int tile_tokens = 0;
    int kc = 0;
    int no_tma_store = 0;  // 1: write y with plain stores even where the TMA store applies
    int zmax = 0;          // cap on the contraction slices of the decode-batch stacked shrink (0: automatic)
    int stacked_direct = 0;  // 1: decode-batch stacked shrink without clusters, slices stored directly
    int simt_expand = 0;   // 1: keep the LoRA expand on CUDA cores even for rank 8
    int force_simt = 0;
    int pdl = 1;
    int stream = 1;          // streamed decode kernel: 0 never, 1 the planner's choice of one or two CTAs per SM,
                             // 2 / 4 always one CTA per SM (deep ring), 3 two per SM wherever they fit
    int group_pairs = 0;     // prefill on pairs of SMs: row pairs per scheduling group (0: planner's choice; a large value = row-major order)
    int pair_decode = 0;     // streamed decode kernel, main CTAs in pairs (two-CTA MMA): 0 never (measured slower), 1 from 64 tokens up, 2 from 17
    int bulk_deliver = 0;    // streamed decode kernel: partial tiles leave through shared memory and bulk copies (1: where the row slices are equal; default plain stores)
    int own_local = 1;       // streamed decode kernel: a CTA keeps its own row slice of its accumulator in shared memory
    int pf = 0;              // its L2 prefetch of the weights beyond the ring: 0 planner's cap, -1 none, n > 0 cap in MB
    int fused = 1;           // 0: never use the single-launch decode kernel
    int coop = 1;            // 0 (measurement only): launch it without the co-residency guarantee
    int pair = 1;            // prefill base product on pairs of SMs (256 x 256 tiles, two-CTA MMA): 0 never, 1 where
                             // the pairs cover enough SMs, 2 wherever the shape allows
    int unit_split = 0;      // decode kernel's main CTAs: 0 planner's choice, 1 even unit ranges over all free SMs, 2 whole row tiles per CTA group
    int aux_ctas = 0;        // > 0: budget of aux CTAs of the decode kernel (the planner's own: 20, or 4 per stacked-shrink tile)
    int no_hold = 0;         // decode kernel, head start of the aux CTAs: 0 planner's choice, 1 none, 64 counter wait, other = nanoseconds
    int hold_after = 0;      // decode kernel: ring stages of W0 the main CTAs request before the aux CTAs' head start (0: planner, -1: none)
    int narrow_select = 0;   // decode kernel's selection: 0 by batch size, 1 always two narrow round trips, -1 always one wide one
    int tail_carve = 0;      // prefill on pairs of SMs: 0 = the planner carves a nearly empty last wave out, -1 = never, n = n row pairs
    int aux_plain = 1;       // streamed kernel: the aux CTAs' partial tiles leave as plain stores (0: staged, one bulk copy)
    int cluster_decode = 0;  // decode batches on clusters that exchange through distributed shared memory (0: never)
    int pdl_decode = 1;      // the decode kernel is launched with programmatic stream serialization as well (0: not)
    int pdl_decode_refused = 0;   // launches the driver refused with both attributes (repeated without it)
    int fused_refused = 0;   // cooperative launches the driver refused (the chain ran instead)
};
Tuning& tuning();

// ---------------------------------------------------------------------------------------------
// Device helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

// 8 consecutive elements as fp32, from a 16-byte aligned address.
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 q = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
    const float4 a = *reinterpret_cast<const float4*>(p);
    const float4 b = *reinterpret_cast<const float4*>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Dot product of two length-n vectors, spread over a warp; every lane returns the sum.
// vec: n % 8 == 0 and both rows 16-byte aligned (128-bit loads); otherwise element by element.
template <typename TI>
__device__ __forceinline__ float warp_dot(const TI* __restrict__ a, const TI* __restrict__ b, int n, int lane,
                                          bool vec) {
    float acc = 0.f;
    if (vec) {
        for (int d = lane * 8; d < n; d += 256) {
            float xa[8], xb[8];
            load8(a + d, xa);
            load8(b + d, xb);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc = fmaf(xa[i], xb[i], acc);
        }
    } else {
        for (int d = lane; d < n; d += 32) acc = fmaf(to_f32(a[d]), to_f32(b[d]), acc);
    }
    return warp_sum(acc);
}

inline int cuda_status(cudaError_t e) { return e == cudaSuccess ? METEORA_OK : METEORA_ERR_CUDA; }
// Internal (never returned through the C ABI): the driver refused a launch CONFIGURATION (co-residency, attributes,
// resources), as opposed to any other CUDA error; only this lets a caller fall back to another launch plan.
constexpr int kLaunchRefused = -100;
inline bool launch_config_refused(cudaError_t e) {
    return e == cudaErrorCooperativeLaunchTooLarge || e == cudaErrorNotSupported || e == cudaErrorInvalidConfiguration ||
           e == cudaErrorInvalidValue || e == cudaErrorLaunchOutOfResources;
}
inline int last_launch_status() { return cuda_status(cudaGetLastError()); }

}  // namespace meteora
