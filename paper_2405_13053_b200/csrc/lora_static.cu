// meteora_lora_delta_static: the LoRA term of the layer for callers that cannot hand the library any scratch.
//
// meteora_lora_delta keeps the shrunk activations u[T*k, r] (fp32) in a caller-provided workspace.  Some
// callers cannot provide one: a plug-in that runs inside another framework's memory-pool critical section, a
// real-time serving loop whose allocator is frozen after start-up, a driver written in a language binding
// that exposes launches but no allocator.  For them this file keeps that scratch in a
// file-scope device array of fixed size.  Every GPU that loads the library holds the array (256 KB) until the
// process exits.
#include <atomic>

#include "common.cuh"

namespace meteora {

// u[slot, p] for up to METEORA_STATIC_SCRATCH_FLOATS values of T * k * r.
static __device__ __align__(256) float g_static_u[METEORA_STATIC_SCRATCH_FLOATS];

// In host code `g_static_u` is only a handle for the runtime, not a device address; the address a kernel can
// use comes from cudaGetSymbolAddress, once per device, with that device current (the caller's stream must
// belong to that device).  The lookup can load the module (driver memory, a synchronisation), which is why
// the first call per device belongs at start-up.  Threads may race to the first lookup: they store the same
// address, through an atomic.
static int static_scratch(float** out) {
    static std::atomic<float*> ptr[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return METEORA_ERR_CUDA;
    if (dev < 0 || dev >= 64) return METEORA_ERR_UNSUPPORTED_SHAPE;
    float* cached = ptr[dev].load(std::memory_order_acquire);
    if (!cached) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_u) != cudaSuccess || !p) return METEORA_ERR_CUDA;
        cached = static_cast<float*>(p);
        ptr[dev].store(cached, std::memory_order_release);
    }
    *out = cached;
    return METEORA_OK;
}

}  // namespace meteora

using namespace meteora;

extern "C" int meteora_lora_delta_static(const void* x, const void* A, const void* B, const int32_t* topk_idx,
                                         const float* topk_w, const int32_t* offsets, const int32_t* perm,
                                         const meteora_shape_t* s, float* delta, void* stream) {
    if (!s) return METEORA_ERR_INVALID_ARG;
    if (s->dtype != METEORA_F32 && s->dtype != METEORA_BF16) return METEORA_ERR_INVALID_ARG;
    if (s->T < 0 || s->d_in <= 0 || s->d_out <= 0 || s->N <= 0 || s->r <= 0 || s->k <= 0 || s->k > s->N)
        return METEORA_ERR_INVALID_ARG;
    if (s->N > METEORA_MAX_N || s->k > METEORA_MAX_K || s->r > METEORA_MAX_R) return METEORA_ERR_UNSUPPORTED_SHAPE;
    if ((long long)s->T * s->k * s->r > (long long)METEORA_STATIC_SCRATCH_FLOATS)
        return METEORA_ERR_UNSUPPORTED_SHAPE;            // beyond the built-in scratch: use meteora_lora_delta
    if (s->T == 0) return METEORA_OK;
    if (!x || !A || !B || !topk_idx || !topk_w || !offsets || !perm || !delta) return METEORA_ERR_INVALID_ARG;
    const uintptr_t bits = (uintptr_t)x | (uintptr_t)A | (uintptr_t)B | (uintptr_t)delta;
    if (bits & 15u) return METEORA_ERR_MISALIGNED;
    float* u = nullptr;
    int rc = static_scratch(&u);
    if (rc != METEORA_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // Nothing in the scratch has to start at zero: the shrink writes u[slot, :] for every slot of the
    // permutation before the expand reads it, so what an earlier call left there is never seen.
    if ((rc = launch_shrink_segments(x, A, offsets, perm, *s, u, st)) != METEORA_OK) return rc;
    return launch_expand(B, topk_idx, topk_w, u, *s, delta, st);
}
