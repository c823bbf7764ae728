// C ABI of the library (declared in include/meteora.h): argument validation, workspace carve-up,
// dispatch between the tensor-core path and the plain CUDA-core path.
#include <stdio.h>
#include <string.h>

#include <vector>

#include "common.cuh"

namespace meteora {

Tuning& tuning() {
    static Tuning t;
    return t;
}

Workspace carve_workspace(const meteora_shape_t& s_in, void* base) {
    const meteora_shape_t s = rank_padded(s_in);                 // scratch is sized for the padded rank
    Workspace ws;
    uint8_t* p = (uint8_t*)base;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        uint8_t* q = p ? p + off : nullptr;
        off += align_up(bytes, 256);
        return q;
    };
    const size_t T = (size_t)s.T, es = elem_size(s.dtype);
    int col_logits = 0;
    ws.ld_u = tc_stacked_pitch(s, &col_logits);
    ws.col_logits = col_logits;
    ws.status = (int32_t*)take(kHeaderBytes);   // status words [0,64), fused-decode tile counters [64,1024)
    ws.tile_ctr = ws.status ? ws.status + 64 : nullptr;
    ws.topk_idx = (int32_t*)take(T * s.k * sizeof(int32_t));
    ws.topk_w = (float*)take(T * s.k * sizeof(float));
    ws.uw = (float*)take(T * s.k * s.r * sizeof(float));
    ws.u_all = (float*)take(T * ws.ld_u * sizeof(float) * (size_t)stacked_zsplits_bound(s.T));   // one copy per slice of the contraction axis
    // decode kernel scratch: one partial tile of 128 x BN fp32 per (main CTA, row tile it touches), in slot
    // row tile + main CTA: fewer than row tiles + 148 slots
    const size_t row_tiles = ((size_t)s.d_out + 127) / 128;
    const size_t bn = (T + 15) / 16 * 16;
    const size_t part_tiles = s.T <= 256 ? row_tiles + 148 : 0;
    ws.part_g = (float*)take(part_tiles * bn * 128 * sizeof(float));
    ws.x_dev = take(T * s.d_in * es);
    ws.y_dev = take(T * s.d_out * es);
    const bool pad = rank_pad_applies(s_in);
    ws.A_pad = pad ? take((size_t)s.N * s.r * s.d_in * es) : nullptr;
    ws.B_pad = pad ? take((size_t)s.N * s.d_out * s.r * es) : nullptr;
    ws.bytes = off;
    return ws;
}

// A[N,r,d_in] -> Ap[N,r8,d_in] and B[N,d_out,r] -> Bp[N,d_out,r8], the new rank entries zero.
__global__ void k_pad_rank(const __nv_bfloat16* __restrict__ A, const __nv_bfloat16* __restrict__ B,
                           __nv_bfloat16* __restrict__ Ap, __nv_bfloat16* __restrict__ Bp, int N, int r, int r8,
                           int d_in, int d_out) {
    const size_t vec_per_row = (size_t)d_in / 8;                 // d_in % 8 == 0: rows of A move as 16-byte vectors
    const size_t total_a = (size_t)N * r8 * vec_per_row, total_b = (size_t)N * d_out;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total_a; i += stride) {
        const size_t row = i / vec_per_row, v = i - row * vec_per_row;
        const size_t n = row / r8, q = row - n * r8;
        uint4 val = make_uint4(0u, 0u, 0u, 0u);
        if (q < (size_t)r) val = __ldg(reinterpret_cast<const uint4*>(A + (n * r + q) * d_in) + v);
        reinterpret_cast<uint4*>(Ap)[i] = val;
    }
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total_b; i += stride) {
        const __nv_bfloat16* src = B + i * r;
        __nv_bfloat16* dst = Bp + i * r8;
        for (int q = 0; q < r8; ++q) dst[q] = q < r ? src[q] : __float2bfloat16_rn(0.f);
    }
}

static int check_shape(const meteora_shape_t* s, bool need_out, bool need_r) {
    if (!s) return METEORA_ERR_INVALID_ARG;
    if (s->dtype != METEORA_F32 && s->dtype != METEORA_BF16) return METEORA_ERR_INVALID_ARG;
    if (s->T < 0 || s->d_in <= 0 || s->N <= 0 || s->k <= 0 || s->k > s->N) return METEORA_ERR_INVALID_ARG;
    if (!(s->temperature > 0.f)) return METEORA_ERR_INVALID_ARG;
    if (need_out && s->d_out <= 0) return METEORA_ERR_INVALID_ARG;
    if (need_r && s->r <= 0) return METEORA_ERR_INVALID_ARG;
    if (s->N > METEORA_MAX_N || s->k > METEORA_MAX_K) return METEORA_ERR_UNSUPPORTED_SHAPE;
    if (need_r && s->r > METEORA_MAX_R) return METEORA_ERR_UNSUPPORTED_SHAPE;
    if ((long long)s->T * s->k >= (1LL << 31)) return METEORA_ERR_UNSUPPORTED_SHAPE;
    return METEORA_OK;
}

// Optional timing of the dominant kernel (the base product with its LoRA epilogue): while a profile is
// open every forward records a CUDA event pair around that launch on the caller's stream.
struct Profile {
    std::vector<cudaEvent_t> ev;   // 2 * capacity events
    int used = 0;                  // pairs recorded
    bool open = false;
};
static Profile& profile() {
    static Profile p;
    return p;
}

static bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

static int forward_device(const void* x, const void* W0, const void* A, const void* B, const void* Wg,
                          const meteora_shape_t& s, void* y, const Workspace& ws, cudaStream_t st) {
    int rc;
    if (rank_pad_applies(s) && !tuning().force_simt && ws.A_pad && ws.B_pad) {
        const meteora_shape_t e = rank_padded(s);
        k_pad_rank<<<296, 256, 0, st>>>((const __nv_bfloat16*)A, (const __nv_bfloat16*)B, (__nv_bfloat16*)ws.A_pad,
                                        (__nv_bfloat16*)ws.B_pad, s.N, s.r, e.r, s.d_in, s.d_out);
        if ((rc = last_launch_status()) != METEORA_OK) return rc;
        return forward_device(x, W0, ws.A_pad, ws.B_pad, Wg, e, y, ws, st);
    }
    Profile& pf = profile();
    const bool timed = pf.open && 2 * (pf.used + 1) <= (int)pf.ev.size();
    if (decode_cluster_supported(s)) {
        if (timed) cudaEventRecord(pf.ev[2 * pf.used], st);
        rc = launch_decode_cluster(x, W0, A, B, Wg, s, ws, y, st);
        if (rc != kLaunchRefused) {
            if (timed) cudaEventRecord(pf.ev[2 * pf.used++ + 1], st);
            return rc;
        }
        tuning().fused_refused += 1;   // the cluster launch was refused: the streamed kernel takes the call
    }
    if (decode_stream_supported(s)) {
        if (timed) cudaEventRecord(pf.ev[2 * pf.used], st);
        rc = launch_decode_stream(x, W0, A, B, Wg, s, ws, y, st);
        if (timed) cudaEventRecord(pf.ev[2 * pf.used++ + 1], st);
        return rc;
    }
    if (decode_fused_supported(s)) {
        if (timed) cudaEventRecord(pf.ev[2 * pf.used], st);
        rc = launch_decode_fused(x, W0, A, B, Wg, s, ws, y, st);
        if (rc != kLaunchRefused) {
            if (timed) cudaEventRecord(pf.ev[2 * pf.used++ + 1], st);
            return rc;
        }
        tuning().fused_refused += 1;   // the cooperative launch was refused (not all CTAs can be resident): use the chain
    }
    if (tc_path_supported(s)) {
        const bool pdl = tuning().pdl != 0;
        if ((rc = launch_stacked_shrink_tc(x, A, Wg, s, ws, st)) != METEORA_OK) return rc;
        if ((rc = launch_select_from_stacked(ws.u_all, ws.ld_u, ws.col_logits, tc_stacked_zsplits(s), s, ws.topk_idx,
                                             ws.topk_w, ws.uw, pdl, st)) != METEORA_OK)
            return rc;
        if (timed) cudaEventRecord(pf.ev[2 * pf.used], st);
        rc = launch_base_lora_tc(x, W0, B, s, ws, y, pdl && !timed, st);
        if (timed) cudaEventRecord(pf.ev[2 * pf.used++ + 1], st);
        return rc;
    }
    if ((rc = launch_gate_topk(x, Wg, s, ws.topk_idx, ws.topk_w, nullptr, st)) != METEORA_OK) return rc;
    if ((rc = launch_shrink_tokens(x, A, ws.topk_idx, ws.topk_w, s, ws.uw, st)) != METEORA_OK) return rc;
    return launch_gemm_simt(x, W0, B, ws.topk_idx, ws.uw, s, y, st);
}

// Workspace of a group call: the modules' own workspaces one after the other (module 0's header serves the
// group: status word, counters), then the partial tiles of the one-launch decode kernel for all row tiles.
struct GroupWorkspace {
    Workspace mod[kMaxGroupModules];
    float* part_g;
    size_t bytes;
};
static GroupWorkspace carve_group(const meteora_shape_t& s, const int* d_outs, int G, void* base) {
    GroupWorkspace gw = {};
    uint8_t* p = (uint8_t*)base;
    size_t off = 0, tiles = 0;
    for (int m = 0; m < G; ++m) {
        meteora_shape_t sm = s;
        sm.d_out = d_outs[m];
        gw.mod[m] = carve_workspace(sm, p ? p + off : nullptr);
        off += align_up(gw.mod[m].bytes, 256);
        tiles += ((size_t)d_outs[m] + 127) / 128;
    }
    const size_t bn = ((size_t)s.T + 15) / 16 * 16;
    const size_t part_tiles = s.T <= 256 ? tiles + 148 : 0;
    gw.part_g = (float*)(p ? p + off : nullptr);
    off += align_up(part_tiles * bn * 128 * sizeof(float), 256);
    gw.bytes = off;
    return gw;
}

static int check_group(const meteora_shape_t* shape, const int* d_out, int n_modules) {
    if (!shape || !d_out || n_modules < 1) return METEORA_ERR_INVALID_ARG;
    if (n_modules > kMaxGroupModules) return METEORA_ERR_UNSUPPORTED_SHAPE;
    for (int m = 0; m < n_modules; ++m) {
        meteora_shape_t sm = *shape;
        sm.d_out = d_out[m];
        const int rc = check_shape(&sm, true, true);
        if (rc != METEORA_OK) return rc;
    }
    return METEORA_OK;
}

}  // namespace meteora

using namespace meteora;

extern "C" {

int meteora_gate_topk(const void* x, const void* Wg, const meteora_shape_t* shape, int32_t* topk_idx,
                      float* topk_w, float* logits, void* stream) {
    int rc = check_shape(shape, false, false);
    if (rc != METEORA_OK) return rc;
    if (shape->T == 0) return METEORA_OK;
    if (!x || !Wg || !topk_idx || !topk_w) return METEORA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(Wg)) return METEORA_ERR_MISALIGNED;
    return launch_gate_topk(x, Wg, *shape, topk_idx, topk_w, logits, (cudaStream_t)stream);
}

int meteora_route(const int32_t* topk_idx, int T, int k, int N, int32_t* counts, int32_t* offsets,
                  int32_t* perm, void* stream) {
    if (T < 0 || k <= 0 || N <= 0 || k > N) return METEORA_ERR_INVALID_ARG;
    if (N > METEORA_MAX_N || k > METEORA_MAX_K || (long long)T * k >= (1LL << 31))
        return METEORA_ERR_UNSUPPORTED_SHAPE;
    if (!counts || !offsets || (T > 0 && (!topk_idx || !perm))) return METEORA_ERR_INVALID_ARG;
    return launch_route(topk_idx, T, k, N, counts, offsets, perm, (cudaStream_t)stream);
}

int meteora_lora_delta(const void* x, const void* A, const void* B, const int32_t* topk_idx,
                       const float* topk_w, const int32_t* offsets, const int32_t* perm,
                       const meteora_shape_t* shape, float* delta, void* workspace, size_t workspace_bytes,
                       void* stream) {
    int rc = check_shape(shape, true, true);
    if (rc != METEORA_OK) return rc;
    if (shape->T == 0) return METEORA_OK;
    if (!x || !A || !B || !topk_idx || !topk_w || !offsets || !perm || !delta || !workspace)
        return METEORA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(A) || !aligned16(B) || !aligned16(delta) || !aligned16(workspace))
        return METEORA_ERR_MISALIGNED;
    const Workspace ws = carve_workspace(*shape, workspace);
    if (workspace_bytes < ws.bytes) return METEORA_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    if ((rc = launch_shrink_segments(x, A, offsets, perm, *shape, ws.uw, st)) != METEORA_OK) return rc;
    return launch_expand(B, topk_idx, topk_w, ws.uw, *shape, delta, st);
}

int meteora_linear_forward(const void* x, const void* W0, const void* A, const void* B, const void* Wg,
                           const meteora_shape_t* shape, void* y, void* workspace, size_t workspace_bytes,
                           void* stream) {
    int rc = check_shape(shape, true, true);
    if (rc != METEORA_OK) return rc;
    if (shape->T == 0) return METEORA_OK;
    if (!x || !W0 || !A || !B || !Wg || !y || !workspace) return METEORA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(W0) || !aligned16(A) || !aligned16(B) || !aligned16(Wg) || !aligned16(y) ||
        !aligned16(workspace))
        return METEORA_ERR_MISALIGNED;
    const Workspace ws = carve_workspace(*shape, workspace);
    if (workspace_bytes < ws.bytes) return METEORA_ERR_WORKSPACE_TOO_SMALL;
    return forward_device(x, W0, A, B, Wg, *shape, y, ws, (cudaStream_t)stream);
}

size_t meteora_group_workspace_bytes(const meteora_shape_t* shape, const int* d_out, int n_modules) {
    if (check_group(shape, d_out, n_modules) != METEORA_OK) return 0;
    return carve_group(*shape, d_out, n_modules, nullptr).bytes;
}

int meteora_group_plan(const meteora_shape_t* shape, const int* d_out, int n_modules) {
    const int rc = check_group(shape, d_out, n_modules);
    if (rc != METEORA_OK) return rc;
    return n_modules > 1 && decode_group_supported(*shape, d_out, n_modules) ? 1 : 0;
}

int meteora_group_workspace_routing(const meteora_shape_t* shape, const int* d_out, int n_modules, int module,
                                    void* workspace, int32_t** topk_idx, float** topk_w) {
    const int rc = check_group(shape, d_out, n_modules);
    if (rc != METEORA_OK) return rc;
    if (!workspace || module < 0 || module >= n_modules) return METEORA_ERR_INVALID_ARG;
    const GroupWorkspace gw = carve_group(*shape, d_out, n_modules, workspace);
    if (topk_idx) *topk_idx = gw.mod[module].topk_idx;
    if (topk_w) *topk_w = gw.mod[module].topk_w;
    return METEORA_OK;
}

int meteora_linear_forward_group(const void* x, const void* const* W0, const void* const* A, const void* const* B,
                                 const void* const* Wg, const int* d_out, int n_modules,
                                 const meteora_shape_t* shape, void* const* y, void* workspace,
                                 size_t workspace_bytes, void* stream) {
    int rc = check_group(shape, d_out, n_modules);
    if (rc != METEORA_OK) return rc;
    if (shape->T == 0) return METEORA_OK;
    if (!x || !W0 || !A || !B || !Wg || !y || !workspace) return METEORA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(workspace)) return METEORA_ERR_MISALIGNED;
    for (int m = 0; m < n_modules; ++m) {
        if (!W0[m] || !A[m] || !B[m] || !Wg[m] || !y[m]) return METEORA_ERR_INVALID_ARG;
        if (!aligned16(W0[m]) || !aligned16(A[m]) || !aligned16(B[m]) || !aligned16(Wg[m]) || !aligned16(y[m]))
            return METEORA_ERR_MISALIGNED;
    }
    GroupWorkspace gw = carve_group(*shape, d_out, n_modules, workspace);
    if (workspace_bytes < gw.bytes) return METEORA_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    // one status word and one set of counters for the whole group: module 0's header
    for (int m = 1; m < n_modules; ++m) {
        gw.mod[m].status = gw.mod[0].status;
        gw.mod[m].tile_ctr = gw.mod[0].tile_ctr;
    }
    if (n_modules > 1 && decode_group_supported(*shape, d_out, n_modules)) {
        GroupModule gm[kMaxGroupModules];
        for (int m = 0; m < n_modules; ++m) gm[m] = GroupModule{W0[m], A[m], B[m], Wg[m], y[m], d_out[m], gw.mod[m]};
        rc = launch_decode_group(x, gm, n_modules, *shape, gw.mod[0].status, gw.part_g, gw.mod[0].tile_ctr, st);
        if (rc != kLaunchRefused) return rc;
        tuning().fused_refused += 1;   // the cooperative launch was refused: one call per module instead
    }
    for (int m = 0; m < n_modules; ++m) {
        meteora_shape_t sm = *shape;
        sm.d_out = d_out[m];
        if ((rc = forward_device(x, W0[m], A[m], B[m], Wg[m], sm, y[m], gw.mod[m], st)) != METEORA_OK) return rc;
    }
    return METEORA_OK;
}

size_t meteora_gate_backward_workspace_bytes(const meteora_shape_t* shape) {
    if (check_shape(shape, true, true) != METEORA_OK) return 0;
    const size_t S = (size_t)shape->T * shape->k, r = (size_t)shape->r;
    return kHeaderBytes + 2 * align_up(S * 4, 256) + 2 * align_up(gate_backward_shrink_floats(*shape) * 4, 256) +
           2 * align_up(((size_t)shape->N + 1) * 4, 256) +
           align_up((size_t)shape->N * shape->d_out * r * elem_size(shape->dtype), 256);
}

// B != nullptr: transposed into the workspace first; else Bt_ready holds the transposed adapters.
static int gate_backward_impl(const void* x, const void* A, const void* B, const void* Bt_ready, const void* dy,
                              const int32_t* topk_idx, const float* topk_w, const meteora_shape_t* shape,
                              float* dlogit, float* dWg, void* workspace, size_t workspace_bytes, void* stream) {
    int rc = check_shape(shape, true, true);
    if (rc != METEORA_OK) return rc;
    if (!dWg || !workspace) return METEORA_ERR_INVALID_ARG;
    const void* b_any = B ? B : Bt_ready;
    if (shape->T > 0 && (!x || !A || !b_any || !dy || !topk_idx || !topk_w)) return METEORA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(A) || !aligned16(b_any) || !aligned16(dy) || !aligned16(workspace))
        return METEORA_ERR_MISALIGNED;
    if (workspace_bytes < meteora_gate_backward_workspace_bytes(shape)) return METEORA_ERR_WORKSPACE_TOO_SMALL;
    const size_t S = (size_t)shape->T * shape->k, r = (size_t)shape->r;
    uint8_t* p = (uint8_t*)workspace + kHeaderBytes;
    auto take = [&](size_t bytes) {
        uint8_t* q = p;
        p += align_up(bytes, 256);
        return q;
    };
    float* dl = (float*)take(S * 4);
    int32_t* perm = (int32_t*)take(S * 4);
    const size_t shrink_bytes = gate_backward_shrink_floats(*shape) * 4;
    float* u = (float*)take(shrink_bytes);               // u and z are contiguous: the one-launch pair of stacked
    float* z = (float*)take(shrink_bytes);               // shrinks writes both into the space of the two
    int32_t* counts = (int32_t*)take(((size_t)shape->N + 1) * 4);
    int32_t* offsets = (int32_t*)take(((size_t)shape->N + 1) * 4);
    void* Bt = take((size_t)shape->N * shape->d_out * r * elem_size(shape->dtype));
    cudaStream_t st = (cudaStream_t)stream;
    // the header's first words take the error flags of the tensor-core kernels
    if (cudaMemsetAsync(workspace, 0, 256, st) != cudaSuccess) return METEORA_ERR_CUDA;
    return launch_gate_backward(x, A, B, dy, topk_idx, topk_w, *shape, B ? Bt : const_cast<void*>(Bt_ready), u, z, dl,
                                S > 0 ? dlogit : nullptr, counts, offsets, perm, (int32_t*)workspace, dWg, st);
}

int meteora_gate_backward(const void* x, const void* A, const void* B, const void* dy, const int32_t* topk_idx,
                          const float* topk_w, const meteora_shape_t* shape, float* dlogit, float* dWg,
                          void* workspace, size_t workspace_bytes, void* stream) {
    if (shape && shape->T > 0 && !B) return METEORA_ERR_INVALID_ARG;
    return gate_backward_impl(x, A, B, nullptr, dy, topk_idx, topk_w, shape, dlogit, dWg, workspace, workspace_bytes,
                              stream);
}

int meteora_pad_adapters_bytes(const meteora_shape_t* shape, size_t* a_bytes, size_t* b_bytes) {
    if (check_shape(shape, true, true) != METEORA_OK || !rank_pad_applies(*shape)) return 0;
    const meteora_shape_t e = rank_padded(*shape);
    if (a_bytes) *a_bytes = (size_t)e.N * e.r * e.d_in * 2;
    if (b_bytes) *b_bytes = (size_t)e.N * e.d_out * e.r * 2;
    return e.r;
}

int meteora_pad_adapters(const void* A, const void* B, const meteora_shape_t* shape, void* A_pad, void* B_pad,
                         void* stream) {
    int rc = check_shape(shape, true, true);
    if (rc != METEORA_OK) return rc;
    if (!A || !B || !A_pad || !B_pad) return METEORA_ERR_INVALID_ARG;
    if (!rank_pad_applies(*shape)) return METEORA_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(A) || !aligned16(A_pad) || !aligned16(B_pad)) return METEORA_ERR_MISALIGNED;
    const meteora_shape_t e = rank_padded(*shape);
    k_pad_rank<<<296, 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)A, (const __nv_bfloat16*)B,
                                                      (__nv_bfloat16*)A_pad, (__nv_bfloat16*)B_pad, shape->N, shape->r,
                                                      e.r, shape->d_in, shape->d_out);
    return last_launch_status();
}

size_t meteora_adapters_bt_bytes(const meteora_shape_t* shape) {
    if (check_shape(shape, true, true) != METEORA_OK) return 0;
    return (size_t)shape->N * shape->d_out * shape->r * elem_size(shape->dtype);
}

int meteora_transpose_adapters_b(const void* B, const meteora_shape_t* shape, void* Bt, void* stream) {
    int rc = check_shape(shape, true, true);
    if (rc != METEORA_OK) return rc;
    if (!B || !Bt) return METEORA_ERR_INVALID_ARG;
    if (!aligned16(B) || !aligned16(Bt)) return METEORA_ERR_MISALIGNED;
    return launch_transpose_b(B, *shape, Bt, (cudaStream_t)stream);
}

int meteora_gate_backward_bt(const void* x, const void* A, const void* Bt, const void* dy, const int32_t* topk_idx,
                             const float* topk_w, const meteora_shape_t* shape, float* dlogit, float* dWg,
                             void* workspace, size_t workspace_bytes, void* stream) {
    if (shape && shape->T > 0 && !Bt) return METEORA_ERR_INVALID_ARG;
    return gate_backward_impl(x, A, nullptr, Bt, dy, topk_idx, topk_w, shape, dlogit, dWg, workspace, workspace_bytes,
                              stream);
}

int meteora_linear_forward_host(const void* x_host, const void* W0, const void* A, const void* B,
                                const void* Wg, const meteora_shape_t* shape, void* y_host, void* workspace,
                                size_t workspace_bytes, void* stream) {
    int rc = check_shape(shape, true, true);
    if (rc != METEORA_OK) return rc;
    if (shape->T == 0) return METEORA_OK;
    if (!x_host || !W0 || !A || !B || !Wg || !y_host || !workspace) return METEORA_ERR_INVALID_ARG;
    if (!aligned16(W0) || !aligned16(A) || !aligned16(B) || !aligned16(Wg) || !aligned16(workspace))
        return METEORA_ERR_MISALIGNED;
    const Workspace ws = carve_workspace(*shape, workspace);
    if (workspace_bytes < ws.bytes) return METEORA_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t es = elem_size(shape->dtype);
    if (cudaMemcpyAsync(ws.x_dev, x_host, (size_t)shape->T * shape->d_in * es, cudaMemcpyHostToDevice, st) !=
        cudaSuccess)
        return METEORA_ERR_CUDA;
    if ((rc = forward_device(ws.x_dev, W0, A, B, Wg, *shape, ws.y_dev, ws, st)) != METEORA_OK) return rc;
    if (cudaMemcpyAsync(y_host, ws.y_dev, (size_t)shape->T * shape->d_out * es, cudaMemcpyDeviceToHost, st) !=
        cudaSuccess)
        return METEORA_ERR_CUDA;
    return METEORA_OK;
}

size_t meteora_workspace_bytes(const meteora_shape_t* shape) {
    if (check_shape(shape, true, true) != METEORA_OK) return 0;
    return carve_workspace(*shape, nullptr).bytes;
}

int meteora_workspace_routing(const meteora_shape_t* shape, void* workspace, int32_t** topk_idx, float** topk_w) {
    int rc = check_shape(shape, true, true);
    if (rc != METEORA_OK) return rc;
    if (!workspace || !topk_idx || !topk_w) return METEORA_ERR_INVALID_ARG;
    const Workspace ws = carve_workspace(*shape, workspace);
    *topk_idx = ws.topk_idx;
    *topk_w = ws.topk_w;
    return METEORA_OK;
}

int meteora_workspace_init(void* workspace, void* stream) {
    if (!workspace) return METEORA_ERR_INVALID_ARG;
    return cuda_status(cudaMemsetAsync(workspace, 0, kHeaderBytes, (cudaStream_t)stream));
}

int meteora_workspace_status(void* workspace, void* stream) {
    if (!workspace) return METEORA_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    int32_t word = 0;
    if (cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return METEORA_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return METEORA_ERR_CUDA;
    if (word != 0) {
        if (cudaMemsetAsync(workspace, 0, kHeaderBytes, st) != cudaSuccess) return METEORA_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return METEORA_ERR_CUDA;
        return METEORA_ERR_TIMEOUT;
    }
    return METEORA_OK;
}

int meteora_profile_begin(int max_launches) {
    Profile& pf = profile();
    if (max_launches <= 0 || max_launches > (1 << 20)) return METEORA_ERR_INVALID_ARG;
    while ((int)pf.ev.size() < 2 * max_launches) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) return METEORA_ERR_CUDA;
        pf.ev.push_back(e);
    }
    pf.used = 0;
    pf.open = true;
    return METEORA_OK;
}

int meteora_profile_end(float* total_ms, int* launches) {
    Profile& pf = profile();
    if (!total_ms || !launches) return METEORA_ERR_INVALID_ARG;
    pf.open = false;
    float sum = 0.f;
    for (int i = 0; i < pf.used; ++i) {
        float ms = 0.f;
        if (cudaEventSynchronize(pf.ev[2 * i + 1]) != cudaSuccess ||
            cudaEventElapsedTime(&ms, pf.ev[2 * i], pf.ev[2 * i + 1]) != cudaSuccess)
            return METEORA_ERR_CUDA;
        sum += ms;
    }
    *total_ms = sum;
    *launches = pf.used;
    pf.used = 0;
    return METEORA_OK;
}

int meteora_describe_plan(const meteora_shape_t* shape, char* buf, size_t buf_bytes) {
    int rc = check_shape(shape, true, true);
    if (rc != METEORA_OK) return rc;
    if (!buf || buf_bytes == 0) return METEORA_ERR_INVALID_ARG;
    char tmp[512];
    const bool pad = rank_pad_applies(*shape) && !tuning().force_simt;
    describe_plan(pad ? rank_padded(*shape) : *shape, tmp, sizeof(tmp));
    snprintf(buf, buf_bytes, "%s%s fused_refused=%d pdl_decode=%d pdl_decode_refused=%d", tmp,
             pad ? " rank_padded_to_multiple_of_8" : "", tuning().fused_refused, tuning().pdl_decode,
             tuning().pdl_decode_refused);
    return METEORA_OK;
}

int meteora_set_tuning(const char* name, int value) {
    if (!name) return METEORA_ERR_INVALID_ARG;
    Tuning& t = tuning();
    if (!strcmp(name, "splits")) t.splits = value;
    else if (!strcmp(name, "stages")) t.stages = value;
    else if (!strcmp(name, "tile_tokens")) t.tile_tokens = value;
    else if (!strcmp(name, "kc")) t.kc = value;
    else if (!strcmp(name, "no_tma_store")) t.no_tma_store = value;
    else if (!strcmp(name, "zmax")) t.zmax = value;
    else if (!strcmp(name, "stacked_direct")) t.stacked_direct = value;
    else if (!strcmp(name, "simt_expand")) t.simt_expand = value;
    else if (!strcmp(name, "force_simt")) t.force_simt = value;
    else if (!strcmp(name, "pdl")) t.pdl = value;
    else if (!strcmp(name, "fused")) t.fused = value;
    else if (!strcmp(name, "stream")) t.stream = value;
    else if (!strcmp(name, "pf")) t.pf = value;
    else if (!strcmp(name, "own_local")) t.own_local = value;
    else if (!strcmp(name, "group_pairs")) t.group_pairs = value;
    else if (!strcmp(name, "bulk_deliver")) t.bulk_deliver = value;
    else if (!strcmp(name, "pair_decode")) t.pair_decode = value;
    else if (!strcmp(name, "cluster_decode")) t.cluster_decode = value;
    else if (!strcmp(name, "aux_plain")) t.aux_plain = value;
    else if (!strcmp(name, "tail_carve")) t.tail_carve = value;
    else if (!strcmp(name, "wait_limit_us")) return set_wait_limit_us(value);
    else if (!strcmp(name, "coop")) t.coop = value;
    else if (!strcmp(name, "no_hold")) t.no_hold = value;
    else if (!strcmp(name, "unit_split")) t.unit_split = value;
    else if (!strcmp(name, "aux_ctas")) t.aux_ctas = value;
    else if (!strcmp(name, "pair")) t.pair = value;
    else if (!strcmp(name, "pdl_decode")) t.pdl_decode = value;
    else if (!strcmp(name, "hold_after")) t.hold_after = value;
    else if (!strcmp(name, "narrow_select")) t.narrow_select = value;
    else return METEORA_ERR_INVALID_ARG;
    return METEORA_OK;
}

const char* meteora_status_string(int status) {
    switch (status) {
        case METEORA_OK: return "ok";
        case METEORA_ERR_INVALID_ARG: return "invalid argument";
        case METEORA_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case METEORA_ERR_MISALIGNED: return "pointer not 16-byte aligned";
        case METEORA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case METEORA_ERR_CUDA: return "CUDA error";
        case METEORA_ERR_TIMEOUT: return "bounded device wait expired";
        default: return "unknown status";
    }
}

}  // extern "C"
