// Tensor-core path (sm_100a): the dense contractions of the layer on tcgen05 with TMEM accumulators,
// operands staged by TMA.
//
// Both contractions of the forward have the same form  D[row, t] = sum_d W[row, d] * x[t, d]  with the
// weight rows on the MMA's M axis (128 TMEM lanes) and the tokens on its N axis (TMEM columns):
//   - stacked shrink + gate: W = [A_0; ...; A_{N-1}] (N*r rows) followed by Wg (N rows).  One pass over x
//     yields A_i x for every adapter and the gate logits G(x) (Sec. 3.1), written as fp32 to u_all[t, :].
//   - base product: W = W0.  The epilogue adds the gate-weighted LoRA expand
//     sum_j B[idx_j][row, :] . uw[t, j, :]  (Eq. 2) in fp32 and rounds y once to bf16.
// With the weights on M, a decode batch of 1..256 tokens is a single N tile (UMMA N = 16..256), so the
// weight matrix streams from HBM exactly once; when there are fewer row tiles than SMs the contraction
// axis is split over a thread-block cluster and the partial accumulators are summed through distributed
// shared memory in a fixed order (deterministic, no global scratch).
//
// Warp roles (320 threads): warp 0 lane 0 issues TMA loads into a ring of shared-memory stages, warp 1
// owns the TMEM allocation and lane 0 issues tcgen05.mma, warps 2-9 run the epilogue (TMEM lane quarter
// = warp id % 4, two warps per quarter sharing the columns).  Every mbarrier wait is bounded; on expiry the kernel records it in the status word
// and drains instead of hanging.
#include <cuda.h>

#include <stdio.h>

#include <mutex>
#include <vector>

#include "common.cuh"
#include "select.cuh"

namespace meteora {

constexpr int kBM = 128;       // weight rows per tile (UMMA M)
constexpr int kBK = 64;        // contraction elements per stage: one 128-byte swizzled row of bf16
constexpr int kUmmaK = 16;     // contraction elements per tcgen05.mma (32 bytes of bf16)
constexpr int kThreads = 320;      // warp 0: TMA, warp 1: MMA + TMEM, warps 2-9: epilogue
constexpr int kEpiThreads = 256;
constexpr int kWTileBytes = kBM * kBK * 2;
constexpr long long kDefaultWaitLimitCycles = 2000000000LL;  // about a second
// Limit of every bounded device-side wait in SM clock cycles (knob wait_limit_us; one value per device).
__device__ long long g_wait_limit_cycles = kDefaultWaitLimitCycles;
constexpr int kMaxZSplits = 32;

enum { MODE_STACKED = 0, MODE_LORA = 1 };

// Optional device timeline for tuning: built with -DMETEORA_TRACE, CTA 0 of a base-product launch writes the
// low 31 bits of %globaltimer (ns) into status words 32 + slot at a few points.  Compiled out otherwise.
#ifdef METEORA_TRACE
#define METEORA_STAMP(p, slot)                                                      \
    do {                                                                            \
        if (blockIdx.x == 0 && blockIdx.y == 0 && (p).mode == MODE_LORA) {          \
            unsigned long long t_;                                                  \
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                  \
            (p).status[32 + (slot)] = (int)(t_ & 0x7FFFFFFF);                       \
        }                                                                           \
    } while (0)
#else
#define METEORA_STAMP(p, slot) do { } while (0)
#endif

struct WGemmParams {
    int T, K;            // tokens, contraction length
    int BN;              // tokens per tile (multiple of 16, <= 256)
    int splits;          // cluster size along the contraction axis
    int zsplits;         // gridDim.z: further split of the contraction axis; slice z writes its own u_all copy
    size_t u_all_zstride;   // floats between the u_all copies
    int ksteps;          // ceil(K / kBK)
    int stages;          // depth of the TMA ring
    int kc;              // k-steps (64-element chunks) per stage; > 1 only with the 3-D tensor maps
    int maps3d;          // tensor maps are (64, rows, K/64) views: one TMA instruction fetches kc chunks
    int tmem_cols;       // power of two >= max(32, BN)
    int split_tile;      // row tiles >= split_tile read tensor map 1 (their rows restart at 0)
    int rows0, rows1;    // valid rows under tensor map 0 / 1
    int mode;
    float* u_all;        // MODE_STACKED: out[t * ld_u + col]
    int ld_u, col1;      //   col = row (map 0) or col1 + row (map 1)
    const int32_t* topk_idx;   // MODE_LORA
    const float* uw;
    const __nv_bfloat16* B;
    __nv_bfloat16* y;
    int d_out, N, r, k;
    int epi_off;         // byte offset of the epilogue staging area behind the ring
    int uw_off, slab_off;   // byte offsets of s_uw and the B slab inside that area
    int slab_q;          // slab entries held in shared memory (0: read B from global memory)
    int per_slot;        // slab indexed by slot t*k+j instead of by adapter
    // LoRA expand on the tensor cores (rank 8): CTA `split` of a tile owns adapters [split*na, split*na + na)
    // and adds  sum_e B_e[rows, :] . U_e[:, tokens]  to its accumulator with na/2 extra MMAs.
    int lora_mma;        // 1: the expand runs as MMAs, the epilogue only reduces and stores
    int na;              // adapters per split, even (two 8-wide adapters per K = 16 MMA)
    int us_in_ring;      // the token-side operand is too big for the staging area: build it in the idle ring
    int us_off;          // byte offset of the token-side operand inside the staging area (slab at slab_off)
    int idx_off;         // single-launch decode kernel: byte offset of the staged adapter indices (weights at uw_off)
    int tma_store;       // 1: the finished tile is rounded to bf16 in shared memory and leaves by one TMA store
    int32_t* status;
    int pdl_wait;        // epilogue waits for the preceding grid before reading its results
    int pdl_trigger;     // let the dependent grid start as soon as this one is resident
    int row_tile0, tok_base;   // the launch covers row tiles from row_tile0 and tokens from tok_base (a rectangle of y)
    int x_alt;           // MODE_STACKED: row tiles >= split_tile multiply the tokens of the FOURTH tensor map over
    int ksteps1;         //   ksteps1 k-steps (two stacked products with different token operands in one launch)
};

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within the wait limit.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64(), limit = g_wait_limit_cycles;
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try(bar, parity)) return true;
        if ((spin & 0x3FF) == 0 && clock64() - t0 > limit) return false;
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"((uint64_t)tm), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"((uint64_t)tm), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
// Shared memory -> global tensor tile; the calling thread waits until the copy has completed.
__device__ __forceinline__ void tma_store_2d_and_wait(const CUtensorMap* tm, uint32_t src, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"((uint64_t)tm), "r"(src), "r"(c0), "r"(c1)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes, 128-byte swizzled
// (the layout TMA writes with CU_TENSOR_MAP_SWIZZLE_128B): start address, leading byte offset unused
// (1), stride byte offset 1024 (eight rows), descriptor version 1, swizzle mode 2 (128 B).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Shared-memory matrix descriptor of an un-swizzled K-major bf16 operand made of 8-row x 16-byte core
// matrices (128 contiguous bytes each): kstride = bytes between core matrices adjacent along K (leading
// byte offset), mnstride = bytes between core matrices adjacent along M/N (stride byte offset).
__device__ __forceinline__ uint64_t smem_desc_plain(uint32_t addr, uint32_t kstride, uint32_t mnstride) {
    uint64_t d = (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((kstride >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((mnstride >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;
    return d;
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, both operands K-major, M = 128, N = bn.
__device__ __forceinline__ uint32_t instr_desc_bf16(int bn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}

// ------------------------------------------------------------------------------------------------
// Epilogue.  The accumulator tile is parked in shared memory as part[t][row] (row fastest) by the four
// epilogue warps; CTA `split` of the cluster then owns rows [128*split/S, 128*(split+1)/S) of the tile
// and sums, in rank order, the S partial tiles of the cluster for those rows (its own through shared
// memory, its peers' through distributed shared memory).  A thread finishes two adjacent rows of one
// token at a time, so y is written as packed bf16 pairs, 4 bytes per thread, contiguous across lanes.
//
// What the LoRA expand needs is staged in shared memory while the main loop still streams W0:
//   s_e[t][j]   adapter picked by token t at rank j,
//   s_uw[t][j][:] = w_j * (A_e x_t)  (fp32, from the selection kernel),
//   slab[q][row][:]  the B rows of this CTA's row slice, q = adapter (all N of them) or, when the tile
//                    holds fewer (token, pick) slots than there are adapters, q = slot t*k+j.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float2 ld_part2(uint32_t local_addr, uint32_t rank, bool remote) {
    float2 v;
    if (remote) {
        uint32_t a;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(local_addr), "r"(rank));
        asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(a));
    } else {
        asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(local_addr));
    }
    return v;
}

__device__ __forceinline__ void fma8(const uint4& b, const float4& u0, const float4& u1, float& acc) {
    acc = fmaf(__uint_as_float(b.x << 16), u0.x, acc);
    acc = fmaf(__uint_as_float(b.x & 0xFFFF0000u), u0.y, acc);
    acc = fmaf(__uint_as_float(b.y << 16), u0.z, acc);
    acc = fmaf(__uint_as_float(b.y & 0xFFFF0000u), u0.w, acc);
    acc = fmaf(__uint_as_float(b.z << 16), u1.x, acc);
    acc = fmaf(__uint_as_float(b.z & 0xFFFF0000u), u1.y, acc);
    acc = fmaf(__uint_as_float(b.w << 16), u1.z, acc);
    acc = fmaf(__uint_as_float(b.w & 0xFFFF0000u), u1.w, acc);
}

// Stage s_e, s_uw and the B slab of rows [row0, row0 + nrows) (epilogue threads only).  All global loads of
// a batch are issued before any shared-memory store, so the arrays cost one memory round trip together
// instead of one each (the loads queue behind the W0 stream and see microseconds of latency).
__device__ __forceinline__ void stage_lora_operands(const WGemmParams& p, uint8_t* epi, int tok0, int ntok, int row0,
                                                    int nrows, int etid) {
    int* s_e = reinterpret_cast<int*>(epi);
    float4* s_uw4 = reinterpret_cast<float4*>(epi + p.uw_off);
    uint4* slab = reinterpret_cast<uint4*>(epi + p.slab_off);
    const int slots = ntok * p.k;
    const int n4 = slots * p.r / 4;
    const float4* uw4 = reinterpret_cast<const float4*>(p.uw + (size_t)tok0 * p.k * p.r);
    const int32_t* idx = p.topk_idx + (size_t)tok0 * p.k;
    const int vpr = p.r >> 3;                      // 16-byte vectors per B row
    const int vpe = nrows * vpr;                   // vectors per slab entry
    const int nq = p.per_slot ? slots : p.N;
    const int total = p.slab_q > 0 ? nq * vpe : 0;
    const uint4* Bv = reinterpret_cast<const uint4*>(p.B);
    constexpr int UE = 2, UU = 4, UB = 4;
    int e_reg[UE];
    float4 u_reg[UU];
    uint4 b_reg[UB];
#pragma unroll
    for (int u = 0; u < UE; ++u) {
        const int i = etid + u * kEpiThreads;
        e_reg[u] = i < slots ? __ldg(idx + i) : 0;
    }
#pragma unroll
    for (int u = 0; u < UU; ++u) {
        const int i = etid + u * kEpiThreads;
        u_reg[u] = i < n4 ? __ldg(uw4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    auto load_b = [&](int v) {
        uint4 val = make_uint4(0u, 0u, 0u, 0u);
        if (v < total) {
            const int q = v / vpe, w = v - q * vpe;
            const int rr = w / vpr;
            const int e = p.per_slot ? min(max(__ldg(idx + q), 0), p.N - 1) : q;
            if (row0 + rr < p.d_out) val = __ldg(Bv + ((size_t)e * p.d_out + row0) * vpr + w);
        }
        return val;
    };
#pragma unroll
    for (int u = 0; u < UB; ++u) b_reg[u] = load_b(etid + u * kEpiThreads);
#pragma unroll
    for (int u = 0; u < UE; ++u) {
        const int i = etid + u * kEpiThreads;
        if (i < slots) s_e[i] = min(max(e_reg[u], 0), p.N - 1);
    }
#pragma unroll
    for (int u = 0; u < UU; ++u) {
        const int i = etid + u * kEpiThreads;
        if (i < n4) s_uw4[i] = u_reg[u];
    }
#pragma unroll
    for (int u = 0; u < UB; ++u) {
        const int v = etid + u * kEpiThreads;
        if (v < total) slab[v] = b_reg[u];
    }
    // whatever did not fit into the first batch
    for (int i = etid + UE * kEpiThreads; i < slots; i += kEpiThreads) s_e[i] = min(max(__ldg(idx + i), 0), p.N - 1);
    for (int i = etid + UU * kEpiThreads; i < n4; i += kEpiThreads) s_uw4[i] = __ldg(uw4 + i);
    for (int v0 = etid + UB * kEpiThreads; v0 < total; v0 += UB * kEpiThreads) {
#pragma unroll
        for (int u = 0; u < UB; ++u) b_reg[u] = load_b(v0 + u * kEpiThreads);
#pragma unroll
        for (int u = 0; u < UB; ++u) {
            const int v = v0 + u * kEpiThreads;
            if (v < total) slab[v] = b_reg[u];
        }
    }
}

// Operands of the tensor-core expand (rank 8), both K-major without swizzle, K = adapter-major (8 elements
// = 16 bytes per adapter):
//   slab[a][row 0..127][8]   = B[a0 + a][tile rows]  -- in global memory the 8 rows x 16 bytes of a core
//                              matrix are already 128 contiguous bytes, so this is a plain copy;
//   us[a][t 0..BN)[8]        = bf16(w_j * A_e x_t) if token t picked adapter e = a0 + a at rank j, else 0.
__device__ __forceinline__ void stage_slab_mma(const WGemmParams& p, uint8_t* epi, int a0, int tile_row0, int etid) {
    uint4* slab = reinterpret_cast<uint4*>(epi + p.slab_off);
    const uint4* Bv = reinterpret_cast<const uint4*>(p.B);
    const int total = p.na * kBM;
    constexpr int U = 4;
    for (int v0 = etid; v0 < total; v0 += U * kEpiThreads) {
        uint4 val[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * kEpiThreads;
            const int a = v / kBM, row = v - a * kBM;
            val[u] = make_uint4(0u, 0u, 0u, 0u);
            if (v < total && a0 + a < p.N && tile_row0 + row < p.d_out)
                val[u] = __ldg(Bv + (size_t)(a0 + a) * p.d_out + tile_row0 + row);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = v0 + u * kEpiThreads;
            if (v < total) slab[v] = val[u];
        }
    }
}

__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }

__device__ __forceinline__ void stage_us_mma(const WGemmParams& p, uint4* us, int a0, int tok0, int ntok, int etid) {
    const int total = p.na * p.BN;
    for (int v = etid; v < total; v += kEpiThreads) us[v] = make_uint4(0u, 0u, 0u, 0u);
    epi_barrier();
    const int slots = ntok * p.k;
    const int32_t* idx = p.topk_idx + (size_t)tok0 * p.k;
    const float4* uw4 = reinterpret_cast<const float4*>(p.uw + (size_t)tok0 * p.k * 8);
    for (int i = etid; i < slots; i += kEpiThreads) {
        const int a = __ldg(idx + i) - a0;
        if (a >= 0 && a < p.na) {
            const float4 lo = __ldg(uw4 + 2 * i), hi = __ldg(uw4 + 2 * i + 1);
            const __nv_bfloat162 q0 = __floats2bfloat162_rn(lo.x, lo.y), q1 = __floats2bfloat162_rn(lo.z, lo.w);
            const __nv_bfloat162 q2 = __floats2bfloat162_rn(hi.x, hi.y), q3 = __floats2bfloat162_rn(hi.z, hi.w);
            uint4 val;
            val.x = *reinterpret_cast<const uint32_t*>(&q0);
            val.y = *reinterpret_cast<const uint32_t*>(&q1);
            val.z = *reinterpret_cast<const uint32_t*>(&q2);
            val.w = *reinterpret_cast<const uint32_t*>(&q3);
            us[a * p.BN + i / p.k] = val;
        }
    }
}

// One (row pair, token) result: add the LoRA expand and store.
__device__ __forceinline__ void finish_pair(const WGemmParams& p, const uint8_t* epi, int tile_m, int row_in_tile,
                                            int nrows, int pr, int t, int token, float a0, float a1) {
    if (p.mode == MODE_STACKED) {
        int row = tile_m * kBM + row_in_tile, limit = p.rows0, col = row;
        if (tile_m >= p.split_tile) {
            row = (tile_m - p.split_tile) * kBM + row_in_tile;
            limit = p.rows1;
            col = p.col1 + row;
        }
        float* dst = p.u_all + (size_t)blockIdx.z * p.u_all_zstride + (size_t)token * p.ld_u + col;
        if (row + 1 < limit) {
            *reinterpret_cast<float2*>(dst) = make_float2(a0, a1);
        } else if (row < limit) {
            dst[0] = a0;
        }
        return;
    }
    const int* s_e = reinterpret_cast<const int*>(epi);
    const float4* s_uw4 = reinterpret_cast<const float4*>(epi + p.uw_off);
    const uint4* slab = reinterpret_cast<const uint4*>(epi + p.slab_off);
    const int vpr = p.r >> 3;
    const int o = tile_m * kBM + row_in_tile;
    for (int j = 0; j < (p.lora_mma ? 0 : p.k); ++j) {
        const int slot = t * p.k + j;
        const int e = s_e[slot];
        for (int c = 0; c < vpr; ++c) {
            uint4 b0, b1;
            if (p.slab_q > 0) {
                const int q = p.per_slot ? slot : e;
                b0 = slab[(q * nrows + 2 * pr) * vpr + c];
                b1 = slab[(q * nrows + 2 * pr + 1) * vpr + c];
            } else {
                const uint4* Bv = reinterpret_cast<const uint4*>(p.B) + ((size_t)e * p.d_out + o) * vpr + c;
                b0 = o < p.d_out ? __ldg(Bv) : make_uint4(0u, 0u, 0u, 0u);
                b1 = o + 1 < p.d_out ? __ldg(Bv + vpr) : make_uint4(0u, 0u, 0u, 0u);
            }
            const float4 u0 = s_uw4[(slot * p.r >> 2) + 2 * c];
            const float4 u1 = s_uw4[(slot * p.r >> 2) + 2 * c + 1];
            fma8(b0, u0, u1, a0);
            fma8(b1, u0, u1, a1);
        }
    }
    __nv_bfloat16* dst = p.y + (size_t)token * p.d_out + o;
    if (o + 1 < p.d_out && (p.d_out & 1) == 0) {
        *reinterpret_cast<__nv_bfloat162*>(dst) = __floats2bfloat162_rn(a0, a1);
    } else {
        if (o < p.d_out) dst[0] = __float2bfloat16_rn(a0);
        if (o + 1 < p.d_out) dst[1] = __float2bfloat16_rn(a1);
    }
}

template <int S>
__device__ __forceinline__ void reduce_and_finish(const WGemmParams& p, uint32_t ring, const uint8_t* epi, int tile_m,
                                                  int split, int tok0, int ntok, int etid) {
    constexpr int P = 64 / S;                 // row pairs of this CTA's slice
    constexpr int TPP = kEpiThreads / P;      // tokens handled per pass of the epilogue threads
    constexpr int NROWS = kBM / S;
    constexpr int U = S >= 8 ? 4 : 8;         // tokens in flight per thread: their partial loads go out together
    const int pr = etid % P, tg = etid / P;
    const int row_in_tile = NROWS * split + 2 * pr;

    for (int t0 = tg; t0 < ntok; t0 += U * TPP) {
        float2 part[U][S];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int t = min(t0 + u * TPP, ntok - 1);
            const uint32_t addr = ring + (uint32_t)((t * kBM + row_in_tile) * 4);
#pragma unroll
            for (int q = 0; q < S; ++q) part[u][q] = ld_part2(addr, (uint32_t)q, S > 1);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int t = t0 + u * TPP;
            if (t >= ntok) break;
            float a0 = 0.f, a1 = 0.f;
#pragma unroll
            for (int q = 0; q < S; ++q) {
                a0 += part[u][q].x;
                a1 += part[u][q].y;
            }
            finish_pair(p, epi, tile_m, row_in_tile, NROWS, pr, t, tok0 + t, a0, a1);
        }
    }
}

__global__ void __launch_bounds__(kThreads)
k_wgemm(const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
        const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmY, const WGemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;                 // 1024-byte aligned for the 128-byte swizzle
    uint8_t* ring_ptr = smem_raw + (ring - raw);
    const uint32_t x_tile_bytes = p.BN * 128;
    const uint32_t stage_bytes = p.kc * (kWTileBytes + x_tile_bytes);   // [kc W tiles][kc x tiles]
    const uint32_t ring_bytes = p.stages * stage_bytes;
    const uint32_t bar_base = ring + ring_bytes;                 // full[stages], empty[stages], acc (8 bytes each)
    const uint32_t bar_acc = bar_base + 2 * p.stages * 8;       // accumulators complete
    const uint32_t bar_main = bar_acc + 8;                      // main-loop MMAs complete: the ring is idle
    const uint32_t bar_us = bar_acc + 16;                       // operands of the tensor-core expand are staged
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ring_ptr + ring_bytes + (2 * p.stages + 3) * 8);
    uint8_t* epi = ring_ptr + ring_bytes + p.epi_off;             // staging of the LoRA operands

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = p.splits;
    const int split = (int)cluster_rank();
    const int tile_m = p.row_tile0 + blockIdx.x / S;
    const int tok0 = p.tok_base + blockIdx.y * p.BN;
    const int ntok = min(p.BN, p.T - tok0);
    // contraction range of this CTA: first cut by grid z, then by cluster rank
    const bool second_x = p.x_alt && tile_m >= p.split_tile;
    const int ksteps_here = second_x ? p.ksteps1 : p.ksteps;
    const int kz0 = (int)(((long long)ksteps_here * blockIdx.z) / p.zsplits);
    const int kz1 = (int)(((long long)ksteps_here * (blockIdx.z + 1)) / p.zsplits);
    const int ks0 = kz0 + (int)(((long long)(kz1 - kz0) * split) / S);
    const int ks1 = kz0 + (int)(((long long)(kz1 - kz0) * (split + 1)) / S);
    const int nks = ks1 - ks0;
    const int niter = nks / p.kc;             // the host picks kc so that it divides every CTA's k-step count

    if (p.pdl_trigger && threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) METEORA_STAMP(p, 0);      // start

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(bar_base + s * 8, 1);
            mbar_init(bar_base + (p.stages + s) * 8, 1);
        }
        mbar_init(bar_acc, 1);
        mbar_init(bar_main, 1);
        mbar_init(bar_us, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"((uint32_t)p.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_slot);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const bool second = tile_m >= p.split_tile;
            const CUtensorMap* tmW = second ? &tmW1 : &tmW0;
            const CUtensorMap* tmT = second_x ? &tmY : &tmX;
            const int row0 = (second ? tile_m - p.split_tile : tile_m) * kBM;
            int issued = 0;
            bool ok = true;
            for (int i = 0; i < niter; ++i) {
                const int s = i % p.stages, round = i / p.stages;
                if (round > 0) ok = mbar_wait(bar_base + (p.stages + s) * 8, (round & 1) ^ 1);
                if (!ok) break;
                const uint32_t full = bar_base + s * 8;
                const uint32_t dst = ring + s * stage_bytes;
                const int kstep = ks0 + i * p.kc;
                mbar_expect_tx(full, stage_bytes);
                if (p.maps3d) {      // one instruction per operand brings kc consecutive 64-element chunks
                    tma_load_3d(dst, tmW, 0, row0, kstep, full);
                    tma_load_3d(dst + p.kc * kWTileBytes, tmT, 0, tok0, kstep, full);
                } else {
                    tma_load_2d(dst, tmW, kstep * kBK, row0, full);
                    tma_load_2d(dst + kWTileBytes, tmT, kstep * kBK, tok0, full);
                }
                issued = i + 1;
            }
            if (!ok) {
                atomicExch(p.status, 1);
                atomicExch(p.status + 1, 100 + issued);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = instr_desc_bf16(p.BN);
            bool ok = true;
            for (int i = 0; i < niter; ++i) {
                const int s = i % p.stages, round = i / p.stages;
                ok = mbar_wait(bar_base + s * 8, round & 1);
                if (!ok) break;
                tc_fence_after();
                const uint32_t wa = ring + s * stage_bytes, xa = wa + p.kc * kWTileBytes;
                for (int c = 0; c < p.kc; ++c) {
                    const uint64_t da = smem_desc_sw128(wa + c * kWTileBytes);
                    const uint64_t db = smem_desc_sw128(xa + c * x_tile_bytes);
#pragma unroll
                    for (int kk = 0; kk < kBK / kUmmaK; ++kk)
                        umma_bf16(tmem_base, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (i | c | kk) != 0);
                }
                umma_commit(bar_base + (p.stages + s) * 8);   // stage reusable once these MMAs have read it
            }
            if (p.lora_mma && ok) {
                // LoRA expand as a K extension of the same accumulation: na/2 MMAs of K = 16 (two adapters)
                umma_commit(bar_main);
                ok = mbar_wait(bar_us, 0);
                if (ok) {
                    tc_fence_after();
                    const uint32_t slab_a = smem_u32(epi + p.slab_off);
                    const uint32_t us_a = p.us_in_ring ? ring : smem_u32(epi + p.us_off);
                    const uint32_t ka = kBM * 16, kb = p.BN * 16;      // bytes from one adapter to the next
                    for (int m = 0; m < p.na / 2; ++m)
                        umma_bf16(tmem_base, smem_desc_plain(slab_a + 2 * m * ka, ka, 128),
                                  smem_desc_plain(us_a + 2 * m * kb, kb, 128), idesc, (niter | m) != 0);
                }
            }
            umma_commit(bar_acc);                              // accumulators complete
            METEORA_STAMP(p, 1);                                // all MMAs issued
            if (!ok) {
                atomicExch(p.status, 1);
                atomicExch(p.status + 2, 200);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps, part 1
        const int quad = warp & 3;                    // TMEM lanes 32*quad .. 32*quad+31 belong to this warp
        const int etid = threadIdx.x - 64;
        if (p.pdl_wait) asm volatile("griddepcontrol.wait;" ::: "memory");
        if (p.mode == MODE_LORA && p.lora_mma) {
            const int a0 = split * p.na;
            stage_slab_mma(p, epi, a0, tile_m * kBM, etid);
            bool ring_ok = true;
            if (p.us_in_ring) {                                 // the token-side operand goes where the ring was
                ring_ok = mbar_wait(bar_main, 0);
                if (!ring_ok && lane == 0) {
                    atomicExch(p.status, 1);
                    atomicExch(p.status + 4, 350);
                }
            }
            uint4* us = reinterpret_cast<uint4*>(p.us_in_ring ? ring_ptr : epi + p.us_off);
            stage_us_mma(p, us, a0, tok0, ntok, etid);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> tensor-core reads
            epi_barrier();
            if (etid == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_us) : "memory");
        } else if (p.mode == MODE_LORA) {
            stage_lora_operands(p, epi, tok0, ntok, tile_m * kBM + (kBM / S) * split, kBM / S, etid);
        }
        if (etid == 0) METEORA_STAMP(p, 2);                     // LoRA operands staged
        bool acc_ok = true;
        if (nks > 0 || p.lora_mma) {
            acc_ok = mbar_wait(bar_acc, 0);
            if (!acc_ok && lane == 0) {
                atomicExch(p.status, 1);
                atomicExch(p.status + 3, 300);
            }
        }
        acc_ok = __all_sync(0xFFFFFFFFu, acc_ok);   // keep the warp-collective TMEM loads convergent
        if (etid == 0) METEORA_STAMP(p, 3);                     // accumulators ready
        tc_fence_after();
        // Park the accumulators in the ring, which is idle now: every load has landed and every MMA that
        // read it has completed.  (The stacked shrink without split-K stores them straight to u_all: lane =
        // row = column of u_all, so a warp writes 128 contiguous bytes per token.)
        float* part = reinterpret_cast<float*>(ring_ptr);
        const int row_in_tile = quad * 32 + lane;
        const int half = ((p.BN / 16 + 1) / 2) * 16;            // warps 2-5 take columns [0, half), warps 6-9 the rest
        const int c_begin = warp < 6 ? 0 : half, c_end = warp < 6 ? half : p.BN;
        if (p.mode == MODE_STACKED && S == 1) {
            int row = tile_m * kBM + row_in_tile, limit = p.rows0, col = row;
            if (tile_m >= p.split_tile) {
                row = (tile_m - p.split_tile) * kBM + row_in_tile;
                limit = p.rows1;
                col = p.col1 + row;
            }
            float* dst = p.u_all + (size_t)blockIdx.z * p.u_all_zstride + (size_t)tok0 * p.ld_u + col;
            for (int c = c_begin; c < c_end; c += 16) {
                float v[16];
                if (nks > 0 && acc_ok) {
                    tmem_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + c, v);
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = 0.f;
                }
                if (row < limit) {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (c + i < ntok) dst[(size_t)(c + i) * p.ld_u] = v[i];
                }
            }
        } else
        for (int c = c_begin; c < c_end; c += 16) {
            float v[16];
            if ((nks > 0 || p.lora_mma) && acc_ok) {
                tmem_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + c, v);
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = 0.f;
            }
            if (p.tma_store) {
                // final values already (the expand ran as MMAs): round once and stage as ystage[t][row]
                __nv_bfloat16* ystage = reinterpret_cast<__nv_bfloat16*>(ring_ptr);
#pragma unroll
                for (int i = 0; i < 16; ++i) ystage[(c + i) * kBM + row_in_tile] = __float2bfloat16_rn(v[i]);
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) part[(c + i) * kBM + row_in_tile] = v[i];
            }
        }
        if (p.tma_store) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> TMA read
    }
    if (threadIdx.x == 64) METEORA_STAMP(p, 4);                 // accumulators parked
    __syncwarp();
    if (S > 1) cluster_sync(); else __syncthreads();
    if (threadIdx.x == 64) METEORA_STAMP(p, 5);                 // partials of the cluster visible

    if (p.tma_store) {
        // one copy moves the whole 128 x BN tile; rows beyond d_out and tokens beyond T are clipped by the map
        if (threadIdx.x == 64) tma_store_2d_and_wait(&tmY, ring, tile_m * kBM, tok0);
    } else if (warp >= 2 && !(p.mode == MODE_STACKED && S == 1)) {
        const int etid = threadIdx.x - 64;
        switch (S) {
            case 1: reduce_and_finish<1>(p, ring, epi, tile_m, split, tok0, ntok, etid); break;
            case 2: reduce_and_finish<2>(p, ring, epi, tile_m, split, tok0, ntok, etid); break;
            case 4: reduce_and_finish<4>(p, ring, epi, tile_m, split, tok0, ntok, etid); break;
            default: reduce_and_finish<8>(p, ring, epi, tile_m, split, tok0, ntok, etid); break;
        }
    }
    if (threadIdx.x == 64) METEORA_STAMP(p, 6);                 // this thread's outputs stored
    __syncwarp();
    if (S > 1) cluster_sync();   // nobody leaves while a peer may still read its partials
    if (threadIdx.x == 64) METEORA_STAMP(p, 7);

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                     "r"((uint32_t)p.tmem_cols)
                     : "memory");
    }
}

}  // namespace meteora

#include "decode_fused.cuh"
#include "wgemm_pair.cuh"
#include "decode_stream.cuh"
#include "decode_cluster.cuh"

namespace meteora {

// ------------------------------------------------------------------------------------------------
// Host side: tensor maps, planning, launches
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        return (EncodeTiledFn)sym;
    }();
    return fn;
}

struct MapKey {
    const void* ptr;
    int K, rows, box_rows, depth;   // depth 0: 2-D map; depth >= 1: 3-D map whose box holds `depth` chunks
    bool operator==(const MapKey& o) const {
        return ptr == o.ptr && K == o.K && rows == o.rows && box_rows == o.box_rows && depth == o.depth;
    }
};
struct MapEntry {
    MapKey key;
    CUtensorMap map;
};

// Tensor map of a [rows, K] row-major bf16 matrix, 128-byte swizzled, out-of-range elements read as zero.
//   depth == 0: 2-D (K, rows), box = 64 elements (128 bytes) x box_rows.
//   depth >= 1: 3-D view (64, rows, K/64) with strides (K*2, 128) bytes, box = 64 x box_rows x depth, so a
//               single copy lands `depth` consecutive k-chunks as `depth` consecutive [box_rows][128 B]
//               tiles.  Needs K % 64 == 0 (a ragged last chunk would run into the next row).
// Encoded maps are cached by (pointer, shape).
static int get_tensor_map(const void* ptr, int K, int rows, int box_rows, int depth, CUtensorMap* out) {
    static std::mutex mu;
    static std::vector<MapEntry> cache;
    static size_t next_evict = 0;
    const MapKey key{ptr, K, rows, box_rows, depth};
    std::lock_guard<std::mutex> lock(mu);
    for (const MapEntry& e : cache)
        if (e.key == key) {
            *out = e.map;
            return METEORA_OK;
        }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return METEORA_ERR_CUDA;
    MapEntry e;
    e.key = key;
    CUresult r;
    if (depth == 0) {
        const cuuint64_t gdim[2] = {(cuuint64_t)K, (cuuint64_t)rows};
        const cuuint64_t gstride[1] = {(cuuint64_t)K * 2};
        const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
        const cuuint32_t estride[2] = {1, 1};
        r = fn(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstride, box, estride,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
        const cuuint64_t gdim[3] = {(cuuint64_t)kBK, (cuuint64_t)rows, (cuuint64_t)(K / kBK)};
        const cuuint64_t gstride[2] = {(cuuint64_t)K * 2, (cuuint64_t)kBK * 2};
        const cuuint32_t box[3] = {(cuuint32_t)kBK, (cuuint32_t)box_rows, (cuuint32_t)depth};
        const cuuint32_t estride[3] = {1, 1, 1};
        r = fn(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), gdim, gstride, box, estride,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (r != CUDA_SUCCESS) return METEORA_ERR_CUDA;
    if (cache.size() < 256) {
        cache.push_back(e);
    } else {
        cache[next_evict] = e;
        next_evict = (next_evict + 1) % cache.size();
    }
    *out = e.map;
    return METEORA_OK;
}

// Tensor map of y[T, d_out] (bf16, row-major) for storing a tile of 128 outputs x box_tokens tokens from
// shared memory laid out [token][128 outputs]; not swizzled.  Needs d_out % 8 == 0 (16-byte row pitch).
static int get_store_map(const void* y, int d_out, int T, int box_tokens, CUtensorMap* out) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return METEORA_ERR_CUDA;
    const cuuint64_t gdim[2] = {(cuuint64_t)d_out, (cuuint64_t)T};
    const cuuint64_t gstride[1] = {(cuuint64_t)d_out * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBM, (cuuint32_t)box_tokens};
    const cuuint32_t estride[2] = {1, 1};
    const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(y), gdim, gstride, box, estride,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? METEORA_OK : METEORA_ERR_CUDA;
}

static int sm_count() {
    static int n = []() {
        int dev = 0, v = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
        return v > 0 ? v : 148;
    }();
    return n;
}

bool tc_path_supported(const meteora_shape_t& s) {
    return s.dtype == METEORA_BF16 && s.d_in % 8 == 0 && s.r % 8 == 0 && s.T > 0 && !tuning().force_simt;
}

// u_all row: columns [0, N*r) hold A_i x, padded to whole 128-row tiles; the logits follow.
int tc_stacked_pitch(const meteora_shape_t& s, int* col_logits) {
    const int a_tiles = (s.N * s.r + kBM - 1) / kBM;
    if (col_logits) *col_logits = a_tiles * kBM;
    return a_tiles * kBM + (int)align_up((size_t)s.N, 32);
}

struct Plan;
static Plan make_plan(int row_tiles, int T, int K, bool lora, int N, int r, int k, bool fused_epi = false,
                      int bn_force = 0, bool no_mma_expand = false, int K2 = 0, int splits_force = 0, int zcap_force = 0);

struct Plan {
    int BN, n_tiles, splits, zsplits, stages, kc, maps3d, tmem_cols;
    int epi_off, uw_off, slab_off, slab_q, per_slot, lora_mma, na, us_in_ring, us_off, idx_off;
    size_t smem;
};

// Tile shape, split-K factor and shared-memory budget of one launch.
//   - tokens per tile: the whole batch when it fits one UMMA N (<= 256), else 256;
//   - split-K cluster size S in {1,2,4,8}: the largest that keeps one CTA per SM; if that leaves more
//     than a quarter of the SMs idle, the next one (two CTAs per SM share the shared memory);
//   - ring depth: whatever the shared memory left after the epilogue staging allows.
// Upper bound of the contraction slices (copies of u_all) the stacked shrink may use for T tokens: 32 for a
// decode batch; for larger batches as many as it takes to reach one CTA per SM with 256-token tiles.
int stacked_zsplits_bound(int T) {
    if (T <= 256) return kMaxZSplits;
    // prefill: one pair of CTAs (or three single CTAs) per 256 tokens; slices until about one CTA per SM
    const int tiles = 2 * ((T + 255) / 256);
    return std::min(kMaxZSplits, std::max(1, 148 / tiles));
}

// K2 > 0: part of the row tiles contracts over K2 instead of K (two stacked products in one launch); the plan is
// made for the shorter of the two and its k-steps per stage divide both.  splits_force / zcap_force: cluster size and
// bound of the grid-z slices chosen by the caller (the tuning knobs still win).
static Plan make_plan(int row_tiles, int T, int K, bool lora, int N, int r, int k, bool fused_epi, int bn_force,
                      bool no_mma_expand, int K2, int splits_force, int zcap_force) {
    const Tuning& tn = tuning();
    Plan pl = {};
    const int ksteps_long = (std::max(K, K2) + kBK - 1) / kBK;
    if (K2 > 0 && K2 < K) std::swap(K, K2);
    const int ksteps = (K + kBK - 1) / kBK;
    // tokens per tile: a decode batch is one tile; a prefill batch uses 256-token tiles (never split along the
    // contraction axis while they fill the SMs: summing 128 x 256 partial tiles across a cluster costs more than it
    // gains there).
    int bn = tn.tile_tokens > 0 ? tn.tile_tokens : (T <= 256 ? (T + 15) / 16 * 16 : 256);
    // A prefill grid that leaves SMs idle with 256-token tiles: over a long contraction axis (from 8192) two CTAs
    // share a 256-token tile's axis when that still fits the SMs, else 128-token tiles (and two CTAs per tile
    // while those fill less than half of the SMs).  Measured on B200, whole layer: 14336 -> 4096 at 512 tokens 100.8 us
    // with 128-token tiles, 82.4 with 256-token tiles on two CTAs each (106 on pairs of SMs); 4096 -> 1024 at 512
    // tokens 31.7 -> 26.8 us and at 1024 tokens 39.4 -> 34.8 with two CTAs per 128-token tile; 4096 -> 4096 at 512
    // tokens stays on 128-token tiles (33.6 us against 41.2).
    bool prefill_split2 = false;
    if (tn.tile_tokens == 0 && T > 256 && row_tiles * ((T + 255) / 256) < sm_count()) {
        if (lora && K >= 8192 && row_tiles * ((T + 255) / 256) * 2 <= sm_count()) {
            prefill_split2 = true;
        } else {
            bn = 128;
            prefill_split2 = lora && row_tiles * ((T + 127) / 128) * 2 <= sm_count();
        }
    }
    if (bn_force > 0) bn = bn_force;
    bn = std::min(256, std::max(16, (bn + 15) / 16 * 16));
    pl.BN = bn;
    pl.n_tiles = (T + bn - 1) / bn;
    const int tiles = row_tiles * pl.n_tiles;
    const int sms = sm_count();
    int splits = 1;
    if (tn.splits > 0 || splits_force > 0) {
        const int want = tn.splits > 0 ? tn.splits : splits_force;
        splits = want >= 8 ? 8 : want >= 4 ? 4 : want >= 2 ? 2 : 1;
    } else if (pl.n_tiles == 1) {
        while (splits < 8 && tiles * splits * 2 <= sms) splits *= 2;
        if (splits < 8 && tiles * splits * 4 < sms * 3 && tiles * splits * 2 <= 2 * sms) splits *= 2;
    } else if (prefill_split2 && bn_force == 0) {
        splits = 2;
    }
    while (splits > 1 && splits > ksteps) splits /= 2;
    pl.splits = splits;
    // The stacked shrink of a decode batch has only a handful of row tiles: cut its contraction axis
    // further over grid z (every slice keeps at least two k-steps); the selection kernel adds the slices.
    pl.zsplits = 1;
    if (!lora && pl.n_tiles == 1) {
        // Decode-batch stacked shrink (a handful of row tiles): cut the contraction axis further over grid z,
        // every slice keeping at least two k-steps; the selection kernel adds the slices.  With the
        // "stacked_direct" knob there is no cluster at all: up to 32 slices, each stored straight to u_all[z].
        if (tn.stacked_direct) {
            splits = tn.splits > 0 ? splits : 1;
            pl.splits = splits;
        }
        const int zcap = tn.zmax > 0 ? std::min(tn.zmax, kMaxZSplits)
                         : zcap_force > 0 ? std::min(zcap_force, kMaxZSplits) : (tn.stacked_direct ? kMaxZSplits : 4);
        pl.zsplits = std::min(zcap, std::max(1, ksteps / splits / 2));
    } else if (!lora) {
        // Stacked shrink of a prefill batch: never a cluster (summing 128 x 256 partial tiles through
        // distributed shared memory costs more than the product itself); if the tiles leave SMs idle, slices
        // of the contraction axis over grid z, stored straight to u_all[z] and added by the selection kernel
        // (same bound as the workspace: stacked_zsplits_bound).
        splits = 1;
        pl.splits = 1;
        const int zcap = tn.zmax > 0 ? std::min(tn.zmax, kMaxZSplits) : kMaxZSplits;
        const int fill = std::max(1, sms / tiles);
        pl.zsplits = std::min(std::min(zcap, std::min(fill, stacked_zsplits_bound(T))), std::max(1, ksteps / 4));
    }
    const int ksteps_cta = std::max(1, ksteps / (splits * pl.zsplits));
    const bool two_per_sm = tiles * splits * pl.zsplits > sms;
    const size_t total_budget = two_per_sm ? 112 * 1024 : 226 * 1024;

    // epilogue staging (LoRA mode): s_e, s_uw, B slab of this CTA's 128/S rows
    const int tile_tokens = std::min(T, bn);
    size_t epi_bytes = 0;
    size_t us_bytes = 0;
    if (lora && fused_epi) {
        // single-launch decode kernel: B rows of the CTA's slice of the tile for every adapter, then the routing
        pl.slab_off = 0;
        pl.uw_off = (int)align_up((size_t)N * (kBM / splits) * 16, 16);
        pl.idx_off = pl.uw_off + bn * k * r * 4;
        epi_bytes = (size_t)pl.idx_off + (size_t)bn * k * 4;
    } else if (lora && r == 8 && !tn.simt_expand && !no_mma_expand) {
        // expand on the tensor cores: B rows of this split's adapters for all 128 rows, and the masked,
        // gate-weighted shrink outputs of the tile's tokens as the other operand
        pl.lora_mma = 1;
        pl.na = ((N + splits - 1) / splits + 1) / 2 * 2;
        pl.slab_off = 0;
        const size_t slab_bytes = (size_t)pl.na * kBM * 16;
        us_bytes = (size_t)pl.na * bn * 16;
        pl.us_in_ring = us_bytes > 32 * 1024 ? 1 : 0;
        pl.us_off = (int)slab_bytes;
        epi_bytes = slab_bytes + (pl.us_in_ring ? 0 : us_bytes);
    } else if (lora) {
        pl.uw_off = (int)align_up((size_t)bn * k * 4, 16);
        pl.slab_off = pl.uw_off + bn * k * r * 4;
        pl.per_slot = tile_tokens * k <= N ? 1 : 0;
        const int q = pl.per_slot ? tile_tokens * k : N;
        const size_t slab_bytes = (size_t)q * (kBM / splits) * r * 2;
        pl.slab_q = slab_bytes <= 64 * 1024 ? q : 0;
        epi_bytes = pl.slab_off + (pl.slab_q > 0 ? slab_bytes : 0);
    }
    const size_t chunk_bytes = kWTileBytes + (size_t)bn * 128;   // one k-step of both operands
    const size_t part_bytes = (size_t)bn * kBM * 4;           // accumulators parked in the idle ring
    const size_t fixed = 1024 + 256 + epi_bytes;               // alignment slack + barriers + staging
    const size_t avail = total_budget > fixed ? total_budget - fixed : 0;
    // k-steps per stage: issuing a TMA copy costs about as much as moving 16 KB, so with the 3-D maps one
    // instruction per operand fetches up to 4 consecutive k-steps, as long as that count divides every
    // CTA's share of the contraction axis and at least two stages still fit.
    pl.maps3d = (K % kBK) == 0 && (K2 % kBK) == 0 ? 1 : 0;
    int kc = 1;
    const int parts = splits * pl.zsplits;
    if (pl.maps3d && ksteps % parts == 0 && ksteps_long % parts == 0) {
        const int per = ksteps / parts, per2 = ksteps_long / parts;
        for (int cand = 4; cand > 1; cand /= 2)
            if (per % cand == 0 && per2 % cand == 0 && (size_t)std::max(2, tn.stages) * cand * chunk_bytes <= avail) {
                kc = cand;
                break;
            }
        if (tn.kc > 0 && per % tn.kc == 0 && per2 % tn.kc == 0) kc = tn.kc;
    }
    pl.kc = kc;
    const size_t stage_bytes = kc * chunk_bytes;
    const int niter = (std::max(ksteps_cta, ksteps_long / (splits * pl.zsplits)) + kc - 1) / kc + 1;
    int stages;
    if (tn.stages > 0) {
        stages = tn.stages;
    } else {
        stages = (int)std::min<size_t>((size_t)niter, avail / stage_bytes);
    }
    stages = std::max(stages, 2);
    while ((size_t)stages * stage_bytes < part_bytes) ++stages;
    if (pl.us_in_ring)
        while ((size_t)stages * stage_bytes < us_bytes) ++stages;
    pl.stages = stages;
    int cols = 32;
    while (cols < bn) cols *= 2;
    pl.tmem_cols = cols;
    pl.epi_off = (int)align_up((size_t)(2 * std::max(stages, 16) + 3) * 8 + 16, 128);
    pl.smem = 1024 + (size_t)stages * stage_bytes + pl.epi_off + epi_bytes;
    // Large ranks with the expand on CUDA cores stage k * r floats per token: if that does not leave room for two
    // ring stages, take fewer tokens per tile.
    if (pl.smem > 227 * 1024 && bn_force == 0 && tn.tile_tokens == 0) {
        for (int cand = 128; cand >= 16; cand /= 2) {
            if (cand >= bn) continue;
            const Plan q = make_plan(row_tiles, T, K, lora, N, r, k, fused_epi, cand, no_mma_expand);
            if (q.smem <= 227 * 1024) return q;
        }
    }
    // Many adapters (from about 100 at rank 8): the B rows of all of them for 128 output rows no longer fit
    // beside the ring, so the expand of this kernel runs on CUDA cores, B rows read through L1.
    if (pl.smem > 227 * 1024 && pl.lora_mma && bn_force == 0)
        return make_plan(row_tiles, T, K, lora, N, r, k, fused_epi, 0, true);
    return pl;
}

static int launch_wgemm(const CUtensorMap& m0, const CUtensorMap& m1, const CUtensorMap& mx, const CUtensorMap& my,
                        WGemmParams& p,
                        int row_tiles, const Plan& pl, bool pdl_attr, cudaStream_t st) {
    if (pl.smem > 227 * 1024) return METEORA_ERR_UNSUPPORTED_SHAPE;
    static int smem_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return METEORA_ERR_CUDA;
    if (dev < 0 || dev >= 64) return METEORA_ERR_UNSUPPORTED_SHAPE;
    if (smem_set[dev] < (int)pl.smem) {
        if (cudaFuncSetAttribute(k_wgemm, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
            return METEORA_ERR_CUDA;
        smem_set[dev] = 227 * 1024;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(row_tiles * pl.splits, pl.n_tiles, pl.zsplits);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int na = 0;
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = pl.splits;
    attr[na].val.clusterDim.y = 1;
    attr[na].val.clusterDim.z = 1;
    ++na;
    if (pdl_attr) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    return cuda_status(cudaLaunchKernelEx(&cfg, k_wgemm, m0, m1, mx, my, p));
}

static int stacked_row_tiles(const meteora_shape_t& s) { return (s.N * s.r + kBM - 1) / kBM + 1; }

// Stacked shrink of a prefill batch on pairs of SMs (k_stacked_pair).
struct StackedPairPlan {
    bool ok;
    int a_tiles, aux_tiles, gate_tile, gate_row0, zsplits, stages;
    size_t smem;
};
static StackedPairPlan make_stacked_pair_plan(const meteora_shape_t& s) {
    StackedPairPlan sp = {};
    if (!tuning().pair || tuning().stacked_direct || !tc_path_supported(s) || s.r != 8 || s.T <= 256) return sp;
    // measured: below about a thousand tokens the pairs' set-up (cluster launch, two cluster barriers) costs
    // 2 - 3 us more than it saves
    if (tuning().pair == 1 && s.T < 1024) return sp;
    sp.a_tiles = (s.N * s.r + kBM - 1) / kBM;
    const int tail_rows = s.N * s.r - (sp.a_tiles - 1) * kBM;
    const bool merged = tail_rows % 8 == 0 && tail_rows + s.N <= kBM;
    sp.aux_tiles = merged ? sp.a_tiles : sp.a_tiles + 1;
    sp.gate_tile = sp.aux_tiles - 1;
    sp.gate_row0 = merged ? tail_rows : 0;
    const int ksteps = (s.d_in + kBK - 1) / kBK;
    const int pairs = ((sp.aux_tiles + 1) / 2) * ((s.T + kPairTokens - 1) / kPairTokens);
    const int zcap = tuning().zmax > 0 ? std::min(tuning().zmax, kMaxZSplits) : kMaxZSplits;
    const int fill = std::max(1, sm_count() / (2 * pairs));
    sp.zsplits = std::min(std::min(zcap, std::min(fill, stacked_zsplits_bound(s.T))), std::max(1, ksteps / 4));
    sp.stages = std::min(6, std::max(2, (ksteps + sp.zsplits - 1) / sp.zsplits));
    sp.smem = 1024 + (size_t)sp.stages * (kWTileBytes + kPairHalf * 128) + 256;
    sp.ok = true;
    return sp;
}

static int launch_stacked_shrink_pair(const void* x, const void* A, const void* Wg, const meteora_shape_t& s,
                                      const Workspace& ws, const StackedPairPlan& sp, cudaStream_t st) {
    CUtensorMap mA, mAt, mG, mX;
    int rc;
    const int tail_box = sp.gate_row0 > 0 ? sp.gate_row0 : kBM, gate_box = kBM - sp.gate_row0;
    if ((rc = get_tensor_map(A, s.d_in, s.N * s.r, kBM, 0, &mA)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(A, s.d_in, s.N * s.r, tail_box, 0, &mAt)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(Wg, s.d_in, s.N, gate_box, 0, &mG)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(x, s.d_in, s.T, kPairHalf, 0, &mX)) != METEORA_OK) return rc;
    StackedPairParams p = {};
    p.T = s.T;
    p.ksteps = (s.d_in + kBK - 1) / kBK;
    p.stages = sp.stages;
    p.zsplits = sp.zsplits;
    p.a_tiles = sp.a_tiles;
    p.a_rows = s.N * s.r;
    p.aux_tiles = sp.aux_tiles;
    p.gate_tile = sp.gate_tile;
    p.gate_row0 = sp.gate_row0;
    p.N = s.N;
    p.u_all = ws.u_all;
    p.zstride = (size_t)s.T * ws.ld_u;
    p.ld_u = ws.ld_u;
    p.col_logits = ws.col_logits;
    p.status = ws.status;
    p.pdl_trigger = tuning().pdl ? 1 : 0;
    static int smem_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return METEORA_ERR_CUDA;
    if (dev < 0 || dev >= 64) return METEORA_ERR_UNSUPPORTED_SHAPE;
    if (!smem_set[dev]) {
        if (cudaFuncSetAttribute(k_stacked_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
            return METEORA_ERR_CUDA;
        smem_set[dev] = 1;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * ((sp.aux_tiles + 1) / 2), (s.T + kPairTokens - 1) / kPairTokens, sp.zsplits);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = sp.smem;
    cfg.stream = st;
    return cuda_status(cudaLaunchKernelEx(&cfg, k_stacked_pair, mA, mAt, mG, mX, p));
}

int tc_stacked_zsplits(const meteora_shape_t& s) {
    const StackedPairPlan sp = make_stacked_pair_plan(s);
    if (sp.ok) return sp.zsplits;
    return make_plan(stacked_row_tiles(s), s.T, s.d_in, false, s.N, s.r, s.k).zsplits;
}

static void fill_common(WGemmParams& p, const Plan& pl, int T, int K, int32_t* status) {
    p.T = T;
    p.K = K;
    p.BN = pl.BN;
    p.splits = pl.splits;
    p.zsplits = pl.zsplits;
    p.ksteps = (K + kBK - 1) / kBK;
    p.stages = pl.stages;
    p.kc = pl.kc;
    p.maps3d = pl.maps3d;
    p.tmem_cols = pl.tmem_cols;
    p.epi_off = pl.epi_off;
    p.uw_off = pl.uw_off;
    p.slab_off = pl.slab_off;
    p.slab_q = pl.slab_q;
    p.per_slot = pl.per_slot;
    p.lora_mma = pl.lora_mma;
    p.na = pl.na;
    p.us_in_ring = pl.us_in_ring;
    p.us_off = pl.us_off;
    p.idx_off = pl.idx_off;
    p.status = status;
}

int launch_stacked_shrink_tc(const void* x, const void* A, const void* Wg, const meteora_shape_t& s,
                             const Workspace& ws, cudaStream_t st) {
    const StackedPairPlan sp = make_stacked_pair_plan(s);
    if (sp.ok) return launch_stacked_shrink_pair(x, A, Wg, s, ws, sp, st);
    const int a_rows = s.N * s.r;
    const int a_tiles = (a_rows + kBM - 1) / kBM;
    const int row_tiles = a_tiles + 1;
    const Plan pl = make_plan(row_tiles, s.T, s.d_in, false, s.N, s.r, s.k);
    CUtensorMap mA, mG, mX;
    int rc;
    if ((rc = get_tensor_map(A, s.d_in, a_rows, kBM, pl.maps3d ? pl.kc : 0, &mA)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(Wg, s.d_in, s.N, kBM, pl.maps3d ? pl.kc : 0, &mG)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(x, s.d_in, s.T, pl.BN, pl.maps3d ? pl.kc : 0, &mX)) != METEORA_OK) return rc;
    WGemmParams p = {};
    fill_common(p, pl, s.T, s.d_in, ws.status);
    p.split_tile = a_tiles;
    p.rows0 = a_rows;
    p.rows1 = s.N;
    p.mode = MODE_STACKED;
    p.u_all = ws.u_all;
    p.u_all_zstride = (size_t)s.T * ws.ld_u;
    p.ld_u = ws.ld_u;
    p.col1 = ws.col_logits;
    p.pdl_wait = 0;
    p.pdl_trigger = tuning().pdl ? 1 : 0;
    return launch_wgemm(mA, mG, mX, mX, p, row_tiles, pl, false, st);
}

// Two stacked shrinks with different token operands as ONE launch, for the gate gradient of a decode batch:
// out[z][t][col] with col = e*r + p for [A_0; ..; A_{N-1}] x (contraction over d_in) and col = half + e*r + p for
// [Bt_0; ..; Bt_{N-1}] dy (contraction over d_out), half = the A rows padded to whole 128-row tiles, row pitch
// 2 * half.  Batches of one token tile only (T <= 256).
bool stacked_dual_supported(const meteora_shape_t& s) {
    meteora_shape_t sb = s;
    sb.d_in = s.d_out;
    return s.T <= 256 && !tuning().stacked_direct && tc_path_supported(s) && tc_path_supported(sb);
}

static Plan make_dual_plan(const meteora_shape_t& s) {
    const int a_tiles = (s.N * s.r + kBM - 1) / kBM;
    // Measured on B200 (4096 -> 4096, 128 tokens; the whole gradient per call): clusters of 8 with 4 slices 30.6 us,
    // clusters of 4: 23.5, of 2 with 16 slices: 24.0, no cluster and 16 slices, each stored straight to its copy of
    // the output: 21.9 (32 slices: 25.5).
    return make_plan(2 * a_tiles, s.T, s.d_in, false, s.N, s.r, s.k, false, 0, false, s.d_out, 1, 16);
}

int stacked_dual_zsplits(const meteora_shape_t& s) { return make_dual_plan(s).zsplits; }

int launch_stacked_dual_tc(const void* x, const void* A, const void* dy, const void* Bt, const meteora_shape_t& s,
                           float* out, int32_t* status, cudaStream_t st) {
    const int a_rows = s.N * s.r;
    const int a_tiles = (a_rows + kBM - 1) / kBM;
    const Plan pl = make_dual_plan(s);
    if (pl.n_tiles != 1) return METEORA_ERR_UNSUPPORTED_SHAPE;
    CUtensorMap mA, mB, mX, mD;
    int rc;
    if ((rc = get_tensor_map(A, s.d_in, a_rows, kBM, pl.maps3d ? pl.kc : 0, &mA)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(Bt, s.d_out, a_rows, kBM, pl.maps3d ? pl.kc : 0, &mB)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(x, s.d_in, s.T, pl.BN, pl.maps3d ? pl.kc : 0, &mX)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(dy, s.d_out, s.T, pl.BN, pl.maps3d ? pl.kc : 0, &mD)) != METEORA_OK) return rc;
    WGemmParams p = {};
    fill_common(p, pl, s.T, s.d_in, status);
    p.split_tile = a_tiles;
    p.rows0 = p.rows1 = a_rows;
    p.mode = MODE_STACKED;
    p.u_all = out;
    p.ld_u = 2 * a_tiles * kBM;
    p.u_all_zstride = (size_t)s.T * p.ld_u;
    p.col1 = a_tiles * kBM;
    p.x_alt = 1;
    p.ksteps1 = (s.d_out + kBK - 1) / kBK;
    p.pdl_trigger = 1;                      // the kernel that follows waits for this grid before it reads
    return launch_wgemm(mA, mB, mX, mD, p, 2 * a_tiles, pl, false, st);
}

// Prefill batches on pairs of SMs (wgemm_pair.cuh): 256 x 256 tiles, ranks that are multiples of 8, y stored by TMA.
struct PairPlan {
    bool ok;
    int stages, nblk, rb, epi_off;   // blocks of 8 expand columns (adapter, 8 rank entries): all, per round
    size_t smem;
};
static PairPlan make_pair_plan(const meteora_shape_t& s) {
    PairPlan pp = {};
    if (!tuning().pair || tuning().simt_expand || tuning().no_tma_store || tuning().tile_tokens || tuning().splits > 1)
        return pp;
    if (!tc_path_supported(s) || s.r % 8 != 0 || s.T <= 256 || s.d_out % 8 != 0) return pp;
    // Measured on B200: ahead of the one-CTA tiles (by 8 - 17 %, and by more where those fall back to 128-token
    // tiles) as soon as the pairs cover a quarter of the SMs; below that too few SMs work at all.
    const int pairs = ((s.d_out + 2 * kBM - 1) / (2 * kBM)) * ((s.T + kPairTokens - 1) / kPairTokens);
    if (tuning().pair == 1 && pairs * 4 < sm_count()) return pp;
    pp.nblk = s.N * (s.r / 8);
    pp.rb = std::min((pp.nblk + 1) / 2 * 2, 28);                  // 28 blocks: 56 KB of B rows, 56 KB of us per round
    const size_t slab = (size_t)pp.rb * kBM * 16, us = (size_t)pp.rb * kPairHalf * 16;
    const size_t ystage = (size_t)kPairTokens * kBM * 2, stage = kWTileBytes + kPairHalf * 128;
    for (int stages = 6; stages >= 2; --stages) {
        const size_t epi_off = align_up((size_t)(2 * stages + 3) * 8 + 16, 128);
        const size_t smem = 1024 + stages * stage + epi_off + slab;
        if (smem <= 226 * 1024 && stages * stage >= std::max(us, ystage)) {
            pp.stages = tuning().stages > 1 && tuning().stages < stages ? tuning().stages : stages;
            pp.epi_off = (int)align_up((size_t)(2 * pp.stages + 3) * 8 + 16, 128);
            pp.smem = 1024 + pp.stages * stage + pp.epi_off + slab;
            pp.ok = pp.stages * stage >= std::max(us, ystage);
            return pp;
        }
    }
    return pp;
}

static int launch_base_lora_pair(const void* x, const void* W0, const void* B, const meteora_shape_t& s,
                                 const Workspace& ws, void* y, const PairPlan& pp, bool pdl, cudaStream_t st,
                                 int skip_rp0, int skip_tt0) {
    const int row_tiles = (s.d_out + kBM - 1) / kBM;
    CUtensorMap mW, mX, mY;
    int rc;
    if ((rc = get_tensor_map(W0, s.d_in, s.d_out, kBM, 0, &mW)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(x, s.d_in, s.T, kPairHalf, 0, &mX)) != METEORA_OK) return rc;
    if ((rc = get_store_map(y, s.d_out, s.T, kPairTokens, &mY)) != METEORA_OK) return rc;
    PairParams p = {};
    p.T = s.T;
    p.K = s.d_in;
    p.ksteps = (s.d_in + kBK - 1) / kBK;
    p.stages = pp.stages;
    p.d_out = s.d_out;
    p.N = s.N;
    p.k = s.k;
    p.r = s.r;
    p.nblk = pp.nblk;
    p.rb = pp.rb;
    p.row_tiles = row_tiles;
    {
        // row pairs per scheduling group: the pairs resident at one time (one per two SMs) cover all token tiles of a group
        const int tok_tiles = (s.T + kPairTokens - 1) / kPairTokens, row_pairs = (row_tiles + 1) / 2;
        const int resident = std::max(1, sm_count() / 2);
        // (measured at 4096 -> 14336, 2048 tokens: row-major 258.9 us per call, groups of 9 / 4 / 2 row pairs 246.3 / 243.8 / 243.4)
        int gp = std::max(1, (resident / tok_tiles + 1) / 2);
        if (tuning().group_pairs > 0) gp = tuning().group_pairs;
        p.group_pairs = std::min(gp, row_pairs);
    }
    p.epi_off = pp.epi_off;
    p.slab_off = 0;
    p.topk_idx = ws.topk_idx;
    p.uw = ws.uw;
    p.B = (const __nv_bfloat16*)B;
    p.status = ws.status;
    p.pdl_wait = pdl ? 1 : 0;
    p.skip_rp0 = skip_rp0;
    p.skip_tt0 = skip_tt0;
    p.pdl_trigger = skip_rp0 != 0x7FFFFFFF && tuning().pdl ? 1 : 0;
    static int smem_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return METEORA_ERR_CUDA;
    if (dev < 0 || dev >= 64) return METEORA_ERR_UNSUPPORTED_SHAPE;
    if (!smem_set[dev]) {
        if (cudaFuncSetAttribute(k_wgemm_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
            return METEORA_ERR_CUDA;
        smem_set[dev] = 1;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * ((row_tiles + 1) / 2), (s.T + kPairTokens - 1) / kPairTokens, 1);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = pp.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cuda_status(cudaLaunchKernelEx(&cfg, k_wgemm_pair, mW, mX, mY, p));
}

// Base product + LoRA expand of the rectangle of y [row tiles row_tile0 .. + n_row_tiles) x [tokens tok_base .. + n_tok) on
// k_wgemm (one CTA, or a cluster along the contraction axis, per tile); bn_force > 0 fixes the tokens per tile.
static int launch_base_lora_rect(const void* x, const void* W0, const void* B, const meteora_shape_t& s,
                                 const Workspace& ws, void* y, int row_tile0, int n_row_tiles, int tok_base, int n_tok,
                                 int bn_force, bool pdl, cudaStream_t st) {
    const int row_tiles = n_row_tiles;
    // a carved-out rectangle of small tiles: clusters along the contraction axis until the tiles fill the SMs (a
    // 128 x 64 tile alone takes in 1.5 MB over 64 k-steps, 23 us on one SM)
    int splits_force = 0;
    if (bn_force > 0) {
        const int tiles = row_tiles * ((n_tok + bn_force - 1) / bn_force);
        splits_force = 1;
        while (splits_force < 8 && tiles * splits_force * 2 <= sm_count()) splits_force *= 2;
    }
    const Plan pl = make_plan(row_tiles, n_tok, s.d_in, true, s.N, s.r, s.k, false, bn_force, false, 0, splits_force);
    CUtensorMap mW, mX;
    int rc;
    if ((rc = get_tensor_map(W0, s.d_in, s.d_out, kBM, pl.maps3d ? pl.kc : 0, &mW)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(x, s.d_in, s.T, pl.BN, pl.maps3d ? pl.kc : 0, &mX)) != METEORA_OK) return rc;
    WGemmParams p = {};
    fill_common(p, pl, s.T, s.d_in, ws.status);
    p.split_tile = 0x7FFFFFFF;
    p.rows0 = s.d_out;
    p.rows1 = 0;
    p.mode = MODE_LORA;
    p.topk_idx = ws.topk_idx;
    p.uw = ws.uw;
    p.B = (const __nv_bfloat16*)B;
    p.y = (__nv_bfloat16*)y;
    p.d_out = s.d_out;
    p.N = s.N;
    p.r = s.r;
    p.k = s.k;
    p.pdl_wait = pdl ? 1 : 0;
    p.pdl_trigger = 0;
    p.row_tile0 = row_tile0;
    p.tok_base = tok_base;
    CUtensorMap mY = mX;
    p.tma_store = 0;
    if (pl.splits == 1 && pl.lora_mma && s.d_out % 8 == 0 && !tuning().no_tma_store) {
        if ((rc = get_store_map(y, s.d_out, s.T, pl.BN, &mY)) != METEORA_OK) return rc;
        p.tma_store = 1;
    }
    return launch_wgemm(mW, mW, mX, mY, p, row_tiles, pl, pdl, st);
}

// A last wave that is nearly empty costs a whole tile time: 448 pair tiles on 74 pairs of SMs are 6 waves and 4 tiles.
// Those tiles (the last token tile of the last `rem` row pairs) are carved out of the pair launch and follow as 128 x 64
// tiles of k_wgemm, which take a fraction of a pair tile's time on a few SMs.  Returns the row pairs to carve.
static int pair_tail_carve(const meteora_shape_t& s) {
    const int row_tiles = (s.d_out + kBM - 1) / kBM, row_pairs = (row_tiles + 1) / 2;
    const int tok_tiles = (s.T + kPairTokens - 1) / kPairTokens;
    const int resident = std::max(1, sm_count() / 2), tiles = row_pairs * tok_tiles;
    const int rem = tiles % resident;
    const int knob = tuning().tail_carve;                        // 0: planner, -1: never, n > 0: carve n row pairs
    int carve = 0;
    if (knob >= 0 && tiles > resident && rem > 0 && rem <= row_pairs && 4 * rem <= resident) carve = rem;
    if (knob > 0) carve = std::min(knob, row_pairs);
    if (tok_tiles < 2) carve = 0;
    return carve;
}

int launch_base_lora_tc(const void* x, const void* W0, const void* B, const meteora_shape_t& s, const Workspace& ws,
                        void* y, bool pdl, cudaStream_t st) {
    const PairPlan pp = make_pair_plan(s);
    if (pp.ok) {
        const int row_tiles = (s.d_out + kBM - 1) / kBM, row_pairs = (row_tiles + 1) / 2;
        const int tok_tiles = (s.T + kPairTokens - 1) / kPairTokens;
        const int carve = pair_tail_carve(s);
        int rc = launch_base_lora_pair(x, W0, B, s, ws, y, pp, pdl, st, carve > 0 ? row_pairs - carve : 0x7FFFFFFF,
                                       tok_tiles - 1);
        if (rc != METEORA_OK || carve == 0) return rc;
        const int row_tile0 = 2 * (row_pairs - carve), tok_base = (tok_tiles - 1) * kPairTokens;
        // (launched programmatically dependent: its main loops run on the SMs the pair launch's last wave frees first;
        // its epilogue waits for the pair launch, and with it for the routing, before it reads the routing)
        return launch_base_lora_rect(x, W0, B, s, ws, y, row_tile0, row_tiles - row_tile0, tok_base, s.T - tok_base, 64,
                                     tuning().pdl != 0, st);
    }
    return launch_base_lora_rect(x, W0, B, s, ws, y, 0, (s.d_out + kBM - 1) / kBM, 0, s.T, 0, pdl, st);
}

// ------------------------------------------------------------------------------------------------
// Fused decode launch: base product + stacked shrink + selection in one cooperative kernel.
// ------------------------------------------------------------------------------------------------
// How many CTAs of the fused kernel with `smem` bytes of dynamic shared memory fit on the device at once.
static int max_resident_ctas(size_t smem) {
    static std::mutex mu;
    static std::vector<std::pair<size_t, int>> cache;
    const size_t key = (smem + 1023) / 1024;
    std::lock_guard<std::mutex> lock(mu);
    for (auto& e : cache)
        if (e.first == key) return e.second;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(k_decode_fused, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
            cudaSuccess)
            cudaGetLastError();
        attr_set = true;
    }
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_decode_fused, kThreads, smem) != cudaSuccess) {
        cudaGetLastError();
        per_sm = 0;
    }
    const int n = per_sm * sm_count();
    cache.push_back({key, n});
    return n;
}

struct FusedPlan {
    bool ok;
    int why;   // why not: 1 knob/shape, 2 more row tiles than main CTAs, 4 residency, 5 shared memory
    Plan main; // BN, stages, kc, maps3d, tmem_cols, staging offsets, smem of the decode kernel
    int row_tiles, n_main, upt, n_aux, a_tiles, aux_tiles, gate_tile, gate_row0, aux_slices, aux_stages, slab_rows, segs;
    size_t w0_bytes;
};

// Launch plan of the single-launch decode kernel, for one module or a group of modules that share x.  Main CTAs: as many as the SMs the aux CTAs leave, at most 14
// per row tile (16 partial tiles is the most the last step sums) and at least one per row tile (a CTA's unit
// range then spans at most two tiles).  Aux CTAs: about 20, the row tiles of the stacked shrink times up to 16
// slices of the contraction axis.
static FusedPlan make_fused_plan(const meteora_shape_t& s, const int* d_outs, int G) {
    const Tuning& tn = tuning();
    FusedPlan fp = {};
    fp.why = 1;
    if (G < 1 || G > kMaxGroup) return fp;
    // Measured on B200 (4096 -> 4096): the single launch is ahead of the three-launch chain at every decode
    // batch size (15.7 vs 16.5 us at T = 1, 19.5 vs 25 us at T = 128).
    if (!tn.fused) return fp;
    if (!tc_path_supported(s) || s.T > 256 || s.r % 8 != 0 || tn.simt_expand) return fp;
    fp.row_tiles = 0;                                            // of all modules of the group together
    size_t w0_bytes = 0;
    for (int m = 0; m < G; ++m) {
        if (d_outs[m] <= 0) return fp;
        fp.row_tiles += (d_outs[m] + kBM - 1) / kBM;
        w0_bytes += (size_t)d_outs[m] * s.d_in * 2;
    }
    fp.w0_bytes = w0_bytes;
    if (fp.row_tiles > kMaxFusedRowTiles) return fp;
    Plan& pl = fp.main;
    const int sms = std::min(sm_count(), 148);                   // the workspace holds partial tiles for 148 CTAs
    const int ksteps = (s.d_in + kBK - 1) / kBK;
    pl.BN = std::min(256, (s.T + 15) / 16 * 16);
    pl.n_tiles = 1;
    pl.splits = 1;
    pl.zsplits = 1;
    pl.maps3d = (s.d_in % kBK) == 0 ? 1 : 0;
    pl.kc = (pl.maps3d && ksteps % 2 == 0) ? 2 : 1;
    if (tn.kc > 0 && pl.maps3d && ksteps % tn.kc == 0 && tn.kc <= 4) pl.kc = tn.kc;
    {
        // staging of the last step (B rows, routing) comes first; with 256-token tiles two k-steps per stage
        // would leave room for one stage only
        const size_t staged = (size_t)s.N * kBM * s.r * 2 + 2 * (size_t)pl.BN * s.k * (s.r * 4 + 4) + 2048;
        const size_t one = kWTileBytes + (size_t)pl.BN * 128;
        while (pl.kc > 1 && staged + 2 * pl.kc * one > 226 * 1024) pl.kc /= 2;
    }
    fp.upt = ksteps / pl.kc;
    // aux CTAs
    fp.a_tiles = (s.N * s.r + kBM - 1) / kBM;
    // Wg rides behind A's last rows when the tile has room for it (N * r = 224, N = 28: rows 96..123 of tile 1)
    const int tail_rows = s.N * s.r - (fp.a_tiles - 1) * kBM;
    const bool merged = tail_rows % 8 == 0 && tail_rows + s.N <= kBM;
    fp.aux_tiles = merged ? fp.a_tiles : fp.a_tiles + 1;
    fp.gate_tile = fp.aux_tiles - 1;
    fp.gate_row0 = merged ? tail_rows : 0;
    fp.why = 2;
    const int group_tiles = G * fp.aux_tiles;                    // every module has its own stacked shrink
    if (group_tiles + 8 > sms) return fp;
    int aux_budget = std::min(std::max(std::max(20, 4 * group_tiles), group_tiles), sms - 8);
    if (tn.aux_ctas > 0) aux_budget = std::min(std::max(tn.aux_ctas, group_tiles), sms - 8);
    fp.aux_slices = std::min(std::min(aux_budget / group_tiles, ksteps), 16);   // 16: the selection reads all slices at once
    if (fp.aux_slices < 1) return fp;
    fp.n_aux = group_tiles * fp.aux_slices;
    const long long units = (long long)fp.row_tiles * fp.upt;
    // Main CTAs: at most 8 per row tile share a tile's rows in the last step.  A multiple of the row tiles keeps
    // every CTA inside one tile (one accumulator, one finishing duty); it is taken unless it idles more than a
    // tenth of the CTAs an uneven split would use (6 per tile keep any tile within 8 unit ranges).
    const int m_max = sms - fp.n_aux;
    if (m_max < 1) return fp;
    const int m_even = fp.row_tiles * std::min(8, m_max / fp.row_tiles);
    int n_main = std::min(m_max, 6 * fp.row_tiles);
    // (measured at 5120 -> 13824 and 4096 -> 14336, 84 % and 88 %: the even unit ranges win by 4 - 8 % up to 192
    // tokens; with 256-token tiles, whose partial tiles are 128 KB each, the whole tiles win by 11 %)
    if (m_even > 0 && m_even * 10 >= n_main * (s.T > 192 ? 8 : 9)) n_main = m_even;
    // an uneven split makes a CTA finish up to 128 rows: if the B rows of 128 rows of every adapter (large ranks)
    // would crowd out the ring, stay with whole tiles per CTA group
    if (m_even > 0 && n_main % fp.row_tiles != 0 && (size_t)s.N * kBM * s.r * 2 > 64 * 1024) n_main = m_even;
    if (tn.unit_split == 1) n_main = std::min(m_max, 6 * fp.row_tiles);
    if (tn.unit_split == 2 && m_even > 0) n_main = m_even;
    if (tn.splits > 0 && tn.splits * fp.row_tiles <= m_max) n_main = std::min(tn.splits, 8) * fp.row_tiles;
    n_main = (int)std::min<long long>(n_main, units);
    if (n_main < 1 || (units + 1) * (n_main + 1) >= (1LL << 31)) return fp;   // 32-bit unit arithmetic on the device
    // SMs the main CTAs leave idle anyway (narrow layers: 8 row tiles use 64 main CTAs) go to the stacked shrink
    // as further slices: its loads are the head of the chain that ends in the routing.  Measured at 4096 -> 1024
    // and 5120 -> 1024, 20 -> 32 aux CTAs: 11.9 -> 11.3 / 13.4 -> 12.8 / 16.0 -> 15.5 us at T = 1 / 32 / 128.  (Where
    // the aux CTAs would take SMs from the main CTAs, 4096 -> 2048 and wider, more of them lose at 128 tokens.)
    // A few spare SMs do not pay: 120 main CTAs + 8 more aux CTAs (14 slices instead of 10) cost 0.2 - 0.5 us at
    // 5120 -> 5120 and 13824 -> 5120 (more partial copies for the selection to add), so only the full 16 slices are taken.
    if (tn.aux_ctas == 0) {
        const int spare = sms - n_main - fp.n_aux;
        const int full = std::min(ksteps, 16);
        if (fp.aux_slices < full && fp.aux_slices + spare / group_tiles >= full) {
            fp.aux_slices = full;
            fp.n_aux = group_tiles * fp.aux_slices;
        }
    }
    // Row tiles a CTA's unit range can touch: 1 for whole tiles per CTA group, 2 while a range is no longer than a
    // tile's units, more beyond that (one TMEM accumulator of BN columns each: at most 4, and 512 columns in all).
    const long long range = (units + n_main - 1) / n_main;
    const int segs = n_main % fp.row_tiles == 0 ? 1 : (int)std::max<long long>(2, (range - 2) / fp.upt + 2);
    if (segs > kMaxSeg || segs * pl.BN > 512) return fp;
    // Measured (gate/up of LLaMA3-8B, 224 row tiles, T = 64): a group whose CTAs finish three tiles one after the
    // other takes 83 us in one launch against 2 x 36 us as two calls, so groups stay within two tiles per CTA.
    if (G > 1 && segs > 2) return fp;
    // A single layer with more row tiles than CTAs (4096 -> 32000, three tiles per CTA): 75 us here against 61 us
    // for the three launches at T = 1, 89 against 96 us at T = 64: taken from 32 tokens up.
    if (segs > 2 && s.T < 32 && tn.fused != 2) return fp;
    fp.segs = segs;
    fp.n_main = n_main;
    // shared memory: staged B rows (at most 128 rows of every adapter), routing, barriers, ring
    fp.why = 5;
    pl.slab_off = 0;
    // rows a CTA finishes: 128 / c when every tile belongs to exactly c CTAs, up to 128 (two tiles) otherwise
    const bool whole = n_main % fp.row_tiles == 0;
    const int own_rows = whole ? 4 * ((32 + n_main / fp.row_tiles - 1) / (n_main / fp.row_tiles)) : kBM;
    // the routing once per tile a CTA finishes rows of (one tile, or two that may belong to two modules)
    const int duties = segs;
    fp.slab_rows = own_rows;
    pl.uw_off = (int)align_up((size_t)s.N * own_rows * s.r * 2, 16);
    pl.idx_off = pl.uw_off + duties * pl.BN * s.k * s.r * 4;
    const size_t epi_bytes = (size_t)pl.idx_off + (size_t)duties * pl.BN * s.k * 4;
    pl.epi_off = (int)align_up((size_t)(2 * 16 + kMaxSeg + 1) * 8 + 16, 128);
    const size_t fixed = 1024 + pl.epi_off + epi_bytes;
    if (fixed + 48 * 1024 > 226 * 1024) return fp;
    const size_t chunk = kWTileBytes + (size_t)pl.BN * 128;      // one k-step of both operands
    const size_t stage_bytes = pl.kc * chunk;
    const size_t avail = 226 * 1024 - fixed;
    int stages = tn.stages > 0 ? tn.stages : (int)std::min<size_t>(avail / stage_bytes, 4);
    stages = std::min(stages, 16);
    if (stages < 2 || (size_t)stages * stage_bytes > avail) return fp;
    pl.stages = stages;
    const size_t ring_bytes = (size_t)stages * stage_bytes;
    // the accumulator tiles leave through the idle ring (128 rows x BN tokens of fp32)
    if (ring_bytes < (size_t)pl.BN * kBM * 4) return fp;
    // the aux CTAs' selection keeps one summed row of the stacked shrink per warp in the idle ring
    int col_logits = 0;
    if (ring_bytes < (size_t)(kThreads / 32) * tc_stacked_pitch(s, &col_logits) * sizeof(float)) return fp;
    int cols = 32;
    while (cols < std::max(2, segs) * pl.BN) cols *= 2;           // one accumulator per row tile a unit range can touch
    pl.tmem_cols = cols;
    pl.smem = 1024 + ring_bytes + pl.epi_off + epi_bytes;
    const int nks_aux = (ksteps + fp.aux_slices - 1) / fp.aux_slices;
    fp.aux_stages = (int)std::min<size_t>(std::min<size_t>(ring_bytes / chunk, 16), (size_t)std::max(nks_aux, 1));
    fp.why = 4;
    if (max_resident_ctas(pl.smem) < fp.n_main + fp.n_aux) return fp;
    fp.why = 0;
    fp.ok = true;
    return fp;
}

static FusedPlan make_fused_plan(const meteora_shape_t& s) { return make_fused_plan(s, &s.d_out, 1); }

bool decode_fused_supported(const meteora_shape_t& s) { return make_fused_plan(s).ok; }

bool decode_group_supported(const meteora_shape_t& s, const int* d_outs, int G) {
    return make_fused_plan(s, d_outs, G).ok;
}

// (module, token) items from which the selection reads in two narrow round trips.  Measured, narrow against wide, us
// per call at T = 1 / 16 / 32 / 64 / 128 / 256: 4096 -> 4096 +0.25 / -0.25 / -0.1 / -0.4 / -0.35 / -1.05; 4096 -> 1024
// 0 / -0.2 / -0.1 / -0.4 / -0.4 / -0.4; 5120 -> 5120 0 / -0.4 / -0.2 / 0 / +0.1 / +0.2; 13824 -> 5120 within +-0.2.
constexpr int kNarrowSelectTokens = 16;

int launch_decode_group(const void* x, const GroupModule* mods, int G, const meteora_shape_t& s, int32_t* status,
                        float* part_g, int32_t* tile_ctr, cudaStream_t st) {
    int d_outs[kMaxGroup] = {};
    if (G < 1 || G > kMaxGroup) return METEORA_ERR_UNSUPPORTED_SHAPE;
    for (int m = 0; m < G; ++m) d_outs[m] = mods[m].d_out;
    const FusedPlan fp = make_fused_plan(s, d_outs, G);
    if (!fp.ok) return METEORA_ERR_UNSUPPORTED_SHAPE;
    const Plan& pl = fp.main;
    const int depth = pl.maps3d ? pl.kc : 0, depth1 = pl.maps3d ? 1 : 0;
    DecodeMaps maps;
    CUtensorMap mX, mX1;
    int rc;
    const int tail_box = fp.gate_row0 > 0 ? fp.gate_row0 : kBM, gate_box = kBM - fp.gate_row0;
    if ((rc = get_tensor_map(x, s.d_in, s.T, pl.BN, depth, &mX)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(x, s.d_in, s.T, pl.BN, depth1, &mX1)) != METEORA_OK) return rc;
    DecodeParams d = {};
    fill_common(d.main, pl, s.T, s.d_in, status);
    d.main.split_tile = 0x7FFFFFFF;
    d.main.mode = MODE_LORA;
    d.main.N = s.N;
    d.main.r = s.r;
    d.main.k = s.k;
    d.n_mod = G;
    int tile0 = 0;
    for (int m = 0; m < kMaxGroup; ++m) {
        const GroupModule& gm = mods[m < G ? m : 0];             // unused slots repeat module 0's (valid) maps
        if ((rc = get_tensor_map(gm.W0, s.d_in, gm.d_out, kBM, depth, &maps.W0[m])) != METEORA_OK) return rc;
        if ((rc = get_tensor_map(gm.A, s.d_in, s.N * s.r, kBM, depth1, &maps.A[m])) != METEORA_OK) return rc;
        if ((rc = get_tensor_map(gm.A, s.d_in, s.N * s.r, tail_box, depth1, &maps.At[m])) != METEORA_OK) return rc;
        if ((rc = get_tensor_map(gm.Wg, s.d_in, s.N, gate_box, depth1, &maps.G[m])) != METEORA_OK) return rc;
        if (m >= G) continue;
        DecodeModule& mo = d.mod[m];
        mo.B = (const __nv_bfloat16*)gm.B;
        mo.y = (__nv_bfloat16*)gm.y;
        mo.d_out = gm.d_out;
        mo.tile0 = tile0;
        mo.topk_idx = gm.ws.topk_idx;
        mo.topk_w = gm.ws.topk_w;
        mo.uw = gm.ws.uw;
        mo.u_part = gm.ws.u_all;
        tile0 += (gm.d_out + kBM - 1) / kBM;
    }
    d.n_main = fp.n_main;
    d.upt = fp.upt;
    d.units = fp.row_tiles * fp.upt;
    d.n_aux = fp.n_aux;
    d.a_tiles = fp.a_tiles;
    d.a_rows = s.N * s.r;
    d.aux_tiles = fp.aux_tiles;
    d.gate_tile = fp.gate_tile;
    d.gate_row0 = fp.gate_row0;
    d.aux_slices = fp.aux_slices;
    d.aux_stages = fp.aux_stages;
    d.bar_stages = std::max(fp.aux_stages, pl.stages);
    d.ld_u = mods[0].ws.ld_u;
    d.col_logits = mods[0].ws.col_logits;
    d.inv_tau = 1.0f / s.temperature;
    // A head start for the aux CTAs' loads pays only while the base product is short.  Measured, us per call at
    // T = 1 / 32 / 128 with none, 1.3, 1.7, 2.1 us: 4096 -> 4096 (34 MB) 15.8 / 15.2 / 15.2 / 15.5, 17.8 / 17.3 /
    // 16.5 / 16.9, 20.1 / 19.7 / 19.5 / 19.8; 4096 -> 5120 (42 MB) is best without one at T = 1 and 128 (15.9 against
    // 16.7 - 17.0, 22.3 against 22.9 - 23.2), and so is 5120 -> 5120 (52 MB): there the routing is ready long before
    // it is needed either way.  Knob no_hold: 1 = none, 64 = wait for the aux CTAs' counter, any other value =
    // that many nanoseconds.
    {
        const int nh = tuning().no_hold;
        const bool is_short = fp.w0_bytes < ((size_t)40 << 20);
        d.hold = nh == 1 ? 0 : nh == 64 ? 1 : nh > 1 ? nh : is_short ? 1800 : 0;
        // The first ring stage of W0 may go out before that head start: measured with 1 stage ahead, 4096 -> 4096
        // (34 MB) 14.0 -> 13.6 / 14.8 -> 14.6 / 17.9 -> 17.5 us at T = 1 / 32 / 128, 4096 -> 1024 (8 MB) 11.8 -> 12.0 /
        // 13.1 -> 13.4 / 15.4 -> 15.9 us; two stages ahead lose the gain again.  Taken from 20 MB of W0 up.
        // Knob hold_after: 0 = this choice, -1 = none, n > 0 = n stages.
        const int ha = tuning().hold_after;
        d.hold_after = ha > 0 ? ha : ha < 0 ? 0 : (d.hold > 0 && fp.w0_bytes >= ((size_t)20 << 20)) ? 1 : 0;
    }
    {
        // knob narrow_select: 0 = by batch size, 1 = always, -1 = never
        const int ns = tuning().narrow_select;
        d.narrow_select = ns > 0 ? 1 : ns < 0 ? 0 : (G * s.T >= kNarrowSelectTokens ? 1 : 0);
    }
    d.ctr = status + 16;
    d.part_g = part_g;
    d.tile_ctr = tile_ctr;
    d.row_tiles = fp.row_tiles;
    d.slab_rows = fp.slab_rows;
    if (pl.smem > 227 * 1024) return METEORA_ERR_UNSUPPORTED_SHAPE;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(fp.n_main + fp.n_aux);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (tuning().coop) {
        attr[na].id = cudaLaunchAttributeCooperative;     // the CTAs wait on one another: all must be resident
        attr[na].val.cooperative = 1;
        ++na;
    }
    // Programmatic dependent launch on top (knob pdl_decode): the next launch is processed under this kernel's tail.
    // If the driver does not take the two attributes together, the kernel is launched without it from then on.
    static bool pdl_accepted = true;
    const bool want_pdl = tuning().pdl_decode != 0 && pdl_accepted;
    if (want_pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    d.pdl = want_pdl ? 1 : 0;
#ifdef METEORA_TRACE
    static int trace_calls = 0;
    d.trace_call = trace_calls++;
#endif
    cudaError_t err = cudaLaunchKernelEx(&cfg, k_decode_fused, maps, mX, mX1, d);
    if (launch_config_refused(err) && want_pdl) {                // the two attributes together: try without the second
        cudaGetLastError();
        pdl_accepted = false;
        tuning().pdl_decode_refused += 1;
        cfg.numAttrs = na - 1;
        d.pdl = 0;
        err = cudaLaunchKernelEx(&cfg, k_decode_fused, maps, mX, mX1, d);
    }
    if (launch_config_refused(err)) {                            // the caller may take the three-launch chain instead
        cudaGetLastError();
        return kLaunchRefused;
    }
    return cuda_status(err);                                     // any other error is reported, not worked around
}

int launch_decode_fused(const void* x, const void* W0, const void* A, const void* B, const void* Wg,
                        const meteora_shape_t& s, const Workspace& ws, void* y, cudaStream_t st) {
    GroupModule gm = {W0, A, B, Wg, y, s.d_out, ws};
    return launch_decode_group(x, &gm, 1, s, ws.status, ws.part_g, ws.tile_ctr, st);
}


// ------------------------------------------------------------------------------------------------
// Streamed decode launch (decode_stream.cuh): one launch per call, two launches resident at a time.
// ------------------------------------------------------------------------------------------------
struct StreamPlan {
    bool ok;
    int why;       // why not: 1 knob/shape, 2 more row tiles than SMs, 5 shared memory
    int BN, kc, stages, aux_stages, tmem_cols, S, n_main, row_tiles;
    int n_aux, a_tiles, aux_tiles, gate_tile, gate_row0, aux_slices;
    int pf_main, pf_aux, slab_off, ring_bytes, ctas_per_sm;
    int pair;      // main CTAs in pairs (clusters of two, two-CTA MMA): each loads half of the token tile
    size_t smem;
};
constexpr int kStreamBarSlots = 16;
constexpr size_t kTwoPerSmBytes = 113 * 1024;    // dynamic shared memory with which two CTAs share an SM

static StreamPlan make_stream_plan_with(const meteora_shape_t& s, int aux_budget_forced) {
    const Tuning& tn = tuning();
    StreamPlan sp = {};
    sp.why = 1;
    if (!tn.fused || !tn.stream || tn.simt_expand) return sp;
    if (!tc_path_supported(s) || s.T > 128 || s.r % 8 != 0 || s.d_in % kBK != 0 || s.d_out <= 0) return sp;
    const int sms = std::min(sm_count(), 148);                   // the workspace holds partial tiles for 148 CTAs
    const int ksteps = s.d_in / kBK;
    sp.row_tiles = (s.d_out + kBM - 1) / kBM;
    if (sp.row_tiles > kMaxFusedRowTiles) return sp;
    // stacked shrink: tiles of [A; Wg] (Wg behind A's last rows when the tile has room), slices of the contraction axis
    sp.a_tiles = (s.N * s.r + kBM - 1) / kBM;
    const int tail_rows = s.N * s.r - (sp.a_tiles - 1) * kBM;
    const bool merged = tail_rows % 8 == 0 && tail_rows + s.N <= kBM;
    sp.aux_tiles = merged ? sp.a_tiles : sp.a_tiles + 1;
    sp.gate_tile = sp.aux_tiles - 1;
    sp.gate_row0 = merged ? tail_rows : 0;
    sp.why = 2;
    int aux_budget = std::max(20, 4 * sp.aux_tiles);
    if (aux_budget_forced > 0) aux_budget = std::max(aux_budget_forced, sp.aux_tiles);
    if (tn.aux_ctas > 0) aux_budget = std::max(tn.aux_ctas, sp.aux_tiles);
    aux_budget = std::min(aux_budget, sms - 8);
    sp.aux_slices = std::min(std::min(aux_budget / sp.aux_tiles, ksteps), 16);
    if (sp.aux_slices < 1) return sp;
    sp.n_aux = sp.aux_tiles * sp.aux_slices;
    sp.kc = 1;
    if (tn.kc > 0 && tn.kc <= 4 && ksteps % tn.kc == 0) sp.kc = tn.kc;
    const int nst = ksteps / sp.kc;
    // Pairs of main CTAs (knob pair_decode: 0 never, the default; 1 from 64 tokens up; 2 from 17 tokens up): each CTA of
    // a pair loads half of the token tile, which at 128 tokens is as large as the W0 tile, and the ring gets a fourth
    // stage.  Measured at 4096 -> 4096: the main loop ends no earlier (8.6 against 8.3 us after the call ahead at 128
    // tokens, 8.4 against 8.0 at 64) and a call takes 18.1 against 16.9 us and 15.4 against 14.6: the loop waits for W0's
    // lines, not for the token tile, and the pair adds two cluster barriers.  Kept as a knob, off by default.
    sp.pair = tn.pair_decode == 0 ? 0 : (s.T >= (tn.pair_decode >= 2 ? 17 : 64) ? 1 : 0);
    const int tiles_padded = sp.pair ? (sp.row_tiles + 1) / 2 * 2 : sp.row_tiles;
    if (sp.pair) sp.n_aux = (sp.n_aux + 1) / 2 * 2;              // whole clusters of two
    int S = std::min(8, (sms - sp.n_aux) / tiles_padded);
    if (tn.splits > 0) S = std::min(tn.splits, 8);
    S = std::min(S, nst);
    // at most two CTAs per SM in all, and the workspace holds row tiles + 148 partial tiles
    if (S < 1 || tiles_padded * S + sp.n_aux > 2 * sms || sp.row_tiles * S > sp.row_tiles + 148) return sp;
    sp.S = S;
    sp.n_main = tiles_padded * S;
    // narrow layers leave SMs idle: give them to the stacked shrink as further slices (all 16 or none)
    if (tn.aux_ctas == 0) {
        const int spare = sms - sp.n_main - sp.n_aux;
        const int full = std::min(ksteps, 16);
        if (sp.aux_slices < full && sp.aux_slices + spare / sp.aux_tiles >= full) {
            sp.aux_slices = full;
            sp.n_aux = sp.aux_tiles * sp.aux_slices;
            if (sp.pair) sp.n_aux = (sp.n_aux + 1) / 2 * 2;
        }
    }
    sp.why = 5;
    sp.BN = sp.pair ? (s.T + 31) / 32 * 32 : (s.T + 15) / 16 * 16;
    int cols = 32;
    while (cols < sp.BN) cols *= 2;
    sp.tmem_cols = cols;
    const int cpa = s.r / 8;
    const int nq_max = (32 + S - 1) / S;
    const size_t slab_bytes = (size_t)s.N * cpa * 4 * nq_max * 16;
    sp.slab_off = (int)align_up((size_t)(2 * kStreamBarSlots + 4) * 8 + 16, 128);
    const size_t stage_bytes = (size_t)sp.kc * (kWTileBytes + (size_t)sp.BN * (sp.pair ? 64 : 128));
    const size_t aux_stage_bytes = kWTileBytes + (size_t)sp.BN * 128;
    const int ntok = s.T;
    // what the last step fetches into the idle ring: S row slices of partial tiles (or the CTA's own tile), the
    // adapter indices and uw of every token; the aux CTAs stage their accumulator tile there
    // (S blocks of partials and one of the expand, each a row slice of at most 4 nq_max rows for all tokens)
    const size_t parts = (size_t)(S + 1) * ((size_t)sp.BN * 4 * nq_max * 4);   // (blocks hold the padded token count)
    const size_t landing = parts + align_up(align_up((size_t)ntok * s.k * 4, 16), 128) + (size_t)ntok * s.k * s.r * 4;
    // an aux CTA stages its accumulator tile there, later its tokens' rows of every partial tile of the stacked shrink
    // (and the summed rows of those tokens behind them)
    const size_t aux_rows = (size_t)(sp.n_aux + sp.aux_tiles) * ((s.T + sp.n_aux - 1) / sp.n_aux) * kBM * 4;
    const size_t ring_need = std::max(std::max(landing, (size_t)sp.BN * kBM * 4), aux_rows);
    const int n_it_max = (nst + S - 1) / S;
    const int nks_aux = (ksteps + sp.aux_slices - 1) / sp.aux_slices;
    // Two CTAs per SM (the next call's CTAs resident under this call) or one with twice the ring?  Two hide the set-up
    // and load the first tiles under the call ahead, but the in-order ring stalls on its slowest line and five
    // stages run at 3.3 - 4 TB/s where eleven reach HBM's rate: the longer the stream, the more the deeper ring counts.
    // Measured per call, two / one per SM (us): 4096 -> 4096 (34 MB of W0) 12.2 / 13.1 at 1 token, 12.4 / 13.2 at 8,
    // 14.3 / 13.8 at 64, 16.6 / 16.4 at 128; 5120 -> 5120 (52 MB) 15.3 / 15.9 at 1, 15.4 / 16.1 at 16, 19.1 / 17.1 at 64;
    // 4096 -> 1024 (8 MB) 10.3 / 10.3 at 1, 12.1 / 11.8 at 64; 4096 -> 14336 (117 MB) 30.3 / 26.7 at 1, 31.2 / 31.5 at 64;
    // 5120 -> 13824 (142 MB) 36.5 / 31.8 at 1.  So: two per SM for 16 - 56 MB of W0 and up to 32 tokens, else one.
    // (Knob stream: 2 or 4 always one per SM, 3 always two where they fit.)
    const size_t w0_bytes = (size_t)s.d_out * s.d_in * 2;
    // (later, at 4096 -> 4096: 12.9 / 13.3 at 48 tokens, 13.4 / 13.5 at 64, 14.4 / 14.3 at 80; at 5120 -> 5120 16.8 / 16.6 at 48
    // and 18.6 / 16.8 at 64: up to 64 tokens for the layers up to 40 MB.)
    const int two_tokens = w0_bytes <= ((size_t)40 << 20) ? 64 : 32;
    const bool want_two = tn.stream == 3 || (tn.stream == 1 && s.T <= two_tokens && w0_bytes >= ((size_t)16 << 20) &&
                                             w0_bytes <= ((size_t)56 << 20));
    for (int per_sm = 2; per_sm >= 1; --per_sm) {
        if (per_sm == 2 && !want_two) continue;
        const size_t budget = per_sm == 2 ? kTwoPerSmBytes : 226 * 1024;
        // all CTAs wait for one another through the workspace: they must all be resident (a forced split can ask for
        // more CTAs than one per SM holds)
        if (sp.n_main + sp.n_aux > per_sm * sms) continue;
        const size_t fixed = 1024 + sp.slab_off + slab_bytes;
        if (fixed + ring_need > budget || fixed + 2 * stage_bytes > budget) continue;
        const size_t avail = budget - fixed;
        int stages = (int)std::min<size_t>(avail / stage_bytes, (size_t)std::min(kStreamBarSlots, std::max(n_it_max, 2)));
        if (tn.stages > 0) stages = std::min(tn.stages, (int)std::min<size_t>(avail / stage_bytes, kStreamBarSlots));
        if (stages < 2) continue;
        const size_t ring_bytes = align_up(std::max((size_t)stages * stage_bytes, ring_need), 128);
        if (fixed + ring_bytes > budget) continue;
        sp.stages = stages;
        sp.aux_stages = (int)std::min<size_t>(std::min<size_t>(ring_bytes / aux_stage_bytes, kStreamBarSlots),
                                              (size_t)std::max(nks_aux, 1));
        sp.ring_bytes = (int)ring_bytes;
        sp.smem = fixed + ring_bytes;
        sp.ctas_per_sm = per_sm;
        break;
    }
    if (sp.ctas_per_sm == 0) return sp;
    // L2 prefetch of the weights beyond the ring, issued before the wait for the kernel ahead: everything up to a
    // cap (the L2 holds this call's weights and the next call's at the same time).  Knob pf: -1 none, n > 0 cap in MB.
    // (measured at 4096 -> 4096: with the prefetch a call takes 20.2 us at 128 tokens and 13.9 at one, without it 18.1
    // and 13.0; a prefetch 4 - 8 ring stages ahead of the loads inside the main loop costs 0.6 - 1.4 us as well: the
    // prefetches take the TMA engine's and the memory system's time without shortening the loads' latency.  Off by default.)
    const size_t cap = tn.pf > 0 ? (size_t)tn.pf << 20 : 0;
    const size_t per_stage_all = (size_t)sp.n_main * sp.kc * kWTileBytes;
    sp.pf_main = (int)std::min<size_t>((size_t)std::max(0, n_it_max - sp.stages), cap / per_stage_all);
    sp.pf_aux = cap > 0 ? std::max(0, nks_aux - sp.aux_stages) : 0;
    sp.why = 0;
    sp.ok = true;
    return sp;
}

// Large ranks (64 at N = 28): with the usual four aux CTAs per stacked tile the main CTAs are few, each has many output
// rows, and the B rows of all adapters for them do not fit beside the ring.  One aux CTA per stacked tile leaves more
// main CTAs with fewer rows each (measured at 4096 -> 4096, 32 tokens, rank 64: 34.4 us against 41.6 on the three-launch
// chain; an expand that reads the picked adapters' rows from L2 instead of staging them took 68 - 78 us).
static StreamPlan make_stream_plan(const meteora_shape_t& s) {
    StreamPlan sp = make_stream_plan_with(s, 0);
    if (!sp.ok && sp.why == 5 && tuning().aux_ctas == 0) sp = make_stream_plan_with(s, 20);
    return sp;
}

bool decode_stream_supported(const meteora_shape_t& s) { return make_stream_plan(s).ok; }

int launch_decode_stream(const void* x, const void* W0, const void* A, const void* B, const void* Wg,
                         const meteora_shape_t& s, const Workspace& ws, void* y, cudaStream_t st) {
    const StreamPlan sp = make_stream_plan(s);
    if (!sp.ok) return METEORA_ERR_UNSUPPORTED_SHAPE;
    CUtensorMap mW, mA, mAt, mG, mX, mX1;
    int rc;
    const int tail_box = sp.gate_row0 > 0 ? sp.gate_row0 : kBM, gate_box = kBM - sp.gate_row0;
    if ((rc = get_tensor_map(W0, s.d_in, s.d_out, kBM, sp.kc, &mW)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(A, s.d_in, s.N * s.r, kBM, 1, &mA)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(A, s.d_in, s.N * s.r, tail_box, 1, &mAt)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(Wg, s.d_in, s.N, gate_box, 1, &mG)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(x, s.d_in, s.T, sp.pair ? sp.BN / 2 : sp.BN, sp.kc, &mX)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(x, s.d_in, s.T, sp.BN, 1, &mX1)) != METEORA_OK) return rc;
    StreamParams d = {};
    d.T = s.T;
    d.BN = sp.BN;
    d.ksteps = s.d_in / kBK;
    d.stages = sp.stages;
    d.kc = sp.kc;
    d.aux_stages = sp.aux_stages;
    d.tmem_cols = sp.tmem_cols;
    d.N = s.N;
    d.r = s.r;
    d.k = s.k;
    d.d_out = s.d_out;
    d.row_tiles = sp.row_tiles;
    d.S = sp.S;
    d.n_main = sp.n_main;
    d.n_aux = sp.n_aux;
    d.aux_tiles = sp.aux_tiles;
    d.aux_slices = sp.aux_slices;
    d.a_tiles = sp.a_tiles;
    d.gate_tile = sp.gate_tile;
    d.gate_row0 = sp.gate_row0;
    d.pf_main = sp.pf_main;
    d.pf_aux = sp.pf_aux;
    d.slab_off = sp.slab_off;
    d.ring_bytes = sp.ring_bytes;
    d.bar_slots = kStreamBarSlots;
    d.inv_tau = 1.0f / s.temperature;
    d.B = (const __nv_bfloat16*)B;
    d.y = (__nv_bfloat16*)y;
    d.topk_idx = ws.topk_idx;
    d.topk_w = ws.topk_w;
    d.uw = ws.uw;
    d.u_part = ws.u_all;
    d.part_g = ws.part_g;
    d.ctr = ws.status + 16;
    d.tile_ctr = ws.tile_ctr;
    d.status = ws.status;
    // Knob bulk_deliver = 1: the partial tiles leave through shared memory and one bulk copy per row slice (where all
    // slices have the same size) instead of plain stores.  Measured at 4096 -> 4096: the same 2.2 - 2.6 us from the
    // accumulator to the counter at 128 tokens either way, 0.3 us slower at one token; off by default.
    d.bulk_deliver = sp.S > 1 && 32 % sp.S == 0 && tuning().bulk_deliver > 0 ? 1 : 0;
    d.aux_plain = tuning().aux_plain ? 1 : 0;
    d.own_local = tuning().own_local && sp.S > 1 ? 1 : 0;
    if (d.bulk_deliver) d.own_local = 1;
    if (sp.S == 1) d.own_local = 1;                             // the tile is the CTA's alone: nothing goes through scratch
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return METEORA_ERR_CUDA;
    if (dev < 0 || dev >= 64) return METEORA_ERR_UNSUPPORTED_SHAPE;
    if (!attr_set[dev]) {
        // the whole shared-memory / L1 array as shared memory, so that two CTAs of 113 KB fit
        if (cudaFuncSetAttribute(k_decode_stream<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
            cudaFuncSetAttribute(k_decode_stream<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
            cudaFuncSetAttribute(k_decode_stream<false>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 cudaSharedmemCarveoutMaxShared) != cudaSuccess ||
            cudaFuncSetAttribute(k_decode_stream<true>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 cudaSharedmemCarveoutMaxShared) != cudaSuccess)
            return METEORA_ERR_CUDA;
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sp.n_main + sp.n_aux);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = sp.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    const bool want_pdl = tuning().pdl_decode != 0;
    int na = 0;
    if (sp.pair) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = 2;
        attr[na].val.clusterDim.y = 1;
        attr[na].val.clusterDim.z = 1;
        ++na;
    }
    if (want_pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    d.pdl = want_pdl ? 1 : 0;
#ifdef METEORA_TRACE
    static int trace_calls = 0;
    d.trace_call = trace_calls++;
#endif
    if (sp.pair) return cuda_status(cudaLaunchKernelEx(&cfg, k_decode_stream<true>, mW, mA, mAt, mG, mX, mX1, d));
    return cuda_status(cudaLaunchKernelEx(&cfg, k_decode_stream<false>, mW, mA, mAt, mG, mX, mX1, d));
}

// ------------------------------------------------------------------------------------------------
// Clustered decode launch (decode_cluster.cuh): the CTAs of a row tile exchange through distributed shared memory.
// ------------------------------------------------------------------------------------------------
struct ClusterPlan {
    bool ok;
    int why;       // why not: 1 knob/shape, 2 clusters do not fit the device, 5 shared memory
    int BN, stages, tmem_cols, acc2_col, S, row_tiles, n_cta;
    int a_tiles, aux_tiles, gate_tile, gate_row0, SL, n_sel;
    int slab_off, recv_off, delta_off, route_off, ring_bytes;
    size_t smem;
};

// How many clusters of `S` CTAs with `smem` bytes of dynamic shared memory the device holds at once (0: unknown).
static int cluster_capacity(int S, size_t smem) {
    static int cache[64][9][2] = {};                             // [device][S][smem above / below 113 KB]
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64 || S < 1 || S > 8) return 0;
    int& slot = cache[dev][S][smem > kTwoPerSmBytes ? 0 : 1];
    if (slot != 0) return slot;
    if (cudaFuncSetAttribute(k_decode_cluster, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
        return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S * 148);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem > kTwoPerSmBytes ? 226 * 1024 : kTwoPerSmBytes;   // the most a plan of that class may ask for
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, k_decode_cluster, &cfg) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    slot = n > 0 ? n : -1;
    return slot;
}

static ClusterPlan make_cluster_plan(const meteora_shape_t& s) {
    const Tuning& tn = tuning();
    ClusterPlan cp = {};
    cp.why = 1;
    if (!tn.fused || !tn.cluster_decode || tn.simt_expand) return cp;
    if (!tc_path_supported(s) || s.T > 128 || s.r % 8 != 0 || s.d_in % kBK != 0 || s.d_out <= 0) return cp;
    const int sms = std::min(sm_count(), 148);
    const int ksteps = s.d_in / kBK;
    cp.row_tiles = (s.d_out + kBM - 1) / kBM;
    cp.a_tiles = (s.N * s.r + kBM - 1) / kBM;
    const int tail_rows = s.N * s.r - (cp.a_tiles - 1) * kBM;
    const bool merged = tail_rows % 8 == 0 && tail_rows + s.N <= kBM;
    cp.aux_tiles = merged ? cp.a_tiles : cp.a_tiles + 1;
    cp.gate_tile = cp.aux_tiles - 1;
    cp.gate_row0 = merged ? tail_rows : 0;
    if (cp.row_tiles < cp.aux_tiles || cp.row_tiles > sms) return cp;       // every stacked tile needs a cluster
    cp.SL = std::min(std::min(cp.row_tiles / cp.aux_tiles, 16), ksteps);
    if (cp.SL * cp.aux_tiles > kEpiThreads) return cp;                      // one thread issues each partial's copy
    cp.BN = (s.T + 15) / 16 * 16;
    int cols = 32;
    while (cols < cp.BN) cols *= 2;
    cp.acc2_col = cols;
    cp.tmem_cols = 2 * cols;
    cp.why = 2;
    // cluster size: as many CTAs per row tile as the SMs allow (at most 8), and the device must hold all clusters at once
    int S = tn.splits > 0 ? std::min(tn.splits, 8) : std::min(8, sms / cp.row_tiles);
    S = std::min(S, ksteps);
    for (; S >= 1; --S) {
        const int cap = cluster_capacity(S, 226 * 1024);
        if (cap >= cp.row_tiles) break;
    }
    if (S < 1) return cp;
    cp.S = S;
    cp.n_cta = cp.row_tiles * S;
    cp.n_sel = std::min(s.T, cp.n_cta);
    cp.why = 5;
    const int cpa = s.r / 8;
    const int nq_max = (32 + S - 1) / S;
    const size_t slab_bytes = (size_t)s.N * cpa * 4 * nq_max * 16;
    const size_t blk_max = (size_t)cp.BN * 4 * nq_max * 4;
    // what the selection puts into the receive blocks: its tokens' rows of all partials and their sums behind them
    const int ntl_max = (s.T + cp.n_cta - 1) / cp.n_cta;
    const size_t sel_bytes = (size_t)(cp.SL * cp.aux_tiles + cp.aux_tiles) * ntl_max * kBM * 4;
    const size_t recv_bytes = align_up(std::max((size_t)S * blk_max, sel_bytes), 128);
    const size_t route_bytes = align_up(align_up((size_t)s.T * s.k * 4, 16), 128) + (size_t)s.T * s.k * s.r * 4;
    cp.slab_off = (int)align_up((size_t)(2 * kStreamBarSlots + 7) * 8 + 16, 128);
    cp.recv_off = (int)align_up(cp.slab_off + slab_bytes, 128);
    cp.delta_off = (int)(cp.recv_off + recv_bytes);
    cp.route_off = (int)align_up(cp.delta_off + blk_max, 128);
    const size_t tail_bytes = cp.route_off + align_up(route_bytes, 128);
    const size_t stage_bytes = kWTileBytes + (size_t)cp.BN * 128;
    const size_t budget = 226 * 1024;
    if (1024 + tail_bytes + 2 * stage_bytes > budget) return cp;
    const int n_it_max = (ksteps + S - 1) / S + (ksteps / S + cp.SL - 1) / cp.SL + 1;
    int stages = (int)std::min<size_t>((budget - 1024 - tail_bytes) / stage_bytes, (size_t)std::min(kStreamBarSlots, n_it_max));
    if (tn.stages > 0) stages = std::min(tn.stages, stages);
    if (stages < 2) return cp;
    cp.stages = stages;
    cp.ring_bytes = (int)(stages * stage_bytes);
    cp.smem = 1024 + cp.ring_bytes + tail_bytes;
    cp.why = 0;
    cp.ok = true;
    return cp;
}

bool decode_cluster_supported(const meteora_shape_t& s) { return make_cluster_plan(s).ok; }

int launch_decode_cluster(const void* x, const void* W0, const void* A, const void* B, const void* Wg,
                          const meteora_shape_t& s, const Workspace& ws, void* y, cudaStream_t st) {
    const ClusterPlan cp = make_cluster_plan(s);
    if (!cp.ok) return METEORA_ERR_UNSUPPORTED_SHAPE;
    CUtensorMap mW, mA, mAt, mG, mX;
    int rc;
    const int tail_box = cp.gate_row0 > 0 ? cp.gate_row0 : kBM, gate_box = kBM - cp.gate_row0;
    if ((rc = get_tensor_map(W0, s.d_in, s.d_out, kBM, 1, &mW)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(A, s.d_in, s.N * s.r, kBM, 1, &mA)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(A, s.d_in, s.N * s.r, tail_box, 1, &mAt)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(Wg, s.d_in, s.N, gate_box, 1, &mG)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(x, s.d_in, s.T, cp.BN, 1, &mX)) != METEORA_OK) return rc;
    ClusterParams d = {};
    d.T = s.T;
    d.BN = cp.BN;
    d.ksteps = s.d_in / kBK;
    d.stages = cp.stages;
    d.tmem_cols = cp.tmem_cols;
    d.acc2_col = cp.acc2_col;
    d.N = s.N;
    d.r = s.r;
    d.k = s.k;
    d.d_out = s.d_out;
    d.row_tiles = cp.row_tiles;
    d.S = cp.S;
    d.aux_tiles = cp.aux_tiles;
    d.a_tiles = cp.a_tiles;
    d.gate_tile = cp.gate_tile;
    d.gate_row0 = cp.gate_row0;
    d.SL = cp.SL;
    d.n_stk = cp.SL * cp.aux_tiles * cp.S;
    d.n_sel = cp.n_sel;
    d.ring_bytes = cp.ring_bytes;
    d.bar_slots = kStreamBarSlots;
    d.slab_off = cp.slab_off;
    d.recv_off = cp.recv_off;
    d.delta_off = cp.delta_off;
    d.route_off = cp.route_off;
    d.inv_tau = 1.0f / s.temperature;
    d.B = (const __nv_bfloat16*)B;
    d.y = (__nv_bfloat16*)y;
    d.topk_idx = ws.topk_idx;
    d.topk_w = ws.topk_w;
    d.uw = ws.uw;
    d.u_part = ws.u_all;
    d.ctr = ws.status + 16;
    d.status = ws.status;
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return METEORA_ERR_CUDA;
    if (dev < 0 || dev >= 64) return METEORA_ERR_UNSUPPORTED_SHAPE;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(k_decode_cluster, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
            cudaFuncSetAttribute(k_decode_cluster, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 cudaSharedmemCarveoutMaxShared) != cudaSuccess)
            return METEORA_ERR_CUDA;
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cp.n_cta);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = cp.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    const bool want_pdl = tuning().pdl_decode != 0;
    int na = 0;
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = cp.S;
    attr[na].val.clusterDim.y = 1;
    attr[na].val.clusterDim.z = 1;
    ++na;
    if (want_pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    d.pdl = want_pdl ? 1 : 0;
#ifdef METEORA_TRACE
    static int trace_calls = 0;
    d.trace_call = trace_calls++;
#endif
    const cudaError_t err = cudaLaunchKernelEx(&cfg, k_decode_cluster, mW, mA, mAt, mG, mX, d);
    if (err != cudaSuccess && launch_config_refused(err)) {
        cudaGetLastError();
        return kLaunchRefused;
    }
    return cuda_status(err);
}

// Human-readable launch plan of meteora_linear_forward for this shape (for logs and benchmark records).
int describe_plan(const meteora_shape_t& s, char* buf, size_t n) {
    if (!tc_path_supported(s)) return snprintf(buf, n, "path=simt");
    const ClusterPlan cp = make_cluster_plan(s);
    if (cp.ok)
        return snprintf(buf, n,
                        "path=cluster_decode launches=1 ctas=%d row_tiles=%d cluster=%d stacked_tiles=%d stacked_slices=%d "
                        "tile_tokens=%d stages=%d smem=%zu",
                        cp.n_cta, cp.row_tiles, cp.S, cp.aux_tiles, cp.SL, cp.BN, cp.stages, cp.smem);
    const StreamPlan sp = make_stream_plan(s);
    if (sp.ok)
        return snprintf(buf, n,
                        "path=stream_decode launches=1 main_ctas=%d row_tiles=%d ctas_per_tile=%d aux_ctas=%d aux_slices=%d "
                        "tile_tokens=%d stages=%d kc=%d smem=%zu ctas_per_sm=%d pairs=%d l2_prefetch_stages=%d",
                        sp.n_main, sp.row_tiles, sp.S, sp.n_aux, sp.aux_slices, sp.BN, sp.stages, sp.kc, sp.smem,
                        sp.ctas_per_sm, sp.pair, sp.pf_main);
    const FusedPlan fp = make_fused_plan(s);
    if (fp.ok)
        return snprintf(buf, n,
                        "path=fused_decode launches=1 main_ctas=%d row_tiles=%d units_per_cta=%.1f aux_ctas=%d "
                        "aux_slices=%d tile_tokens=%d stages=%d kc=%d smem=%zu resident_ctas=%d",
                        fp.n_main, fp.row_tiles, (double)fp.row_tiles * fp.upt / fp.n_main, fp.n_aux, fp.aux_slices,
                        fp.main.BN, fp.main.stages, fp.main.kc, fp.main.smem, max_resident_ctas(fp.main.smem));
    const int row_tiles = (s.d_out + kBM - 1) / kBM;
    const PairPlan pp = make_pair_plan(s);
    if (pp.ok)
        return snprintf(buf, n,
                        "path=chain(not fused: reason %d) launches=%d base=pairs_of_ctas pairs=%d tile=256x256 stages=%d "
                        "smem=%zu expand=mma tail_pairs_as_small_tiles=%d",
                        fp.why, pair_tail_carve(s) > 0 ? 4 : 3,
                        (row_tiles + 1) / 2 * ((s.T + kPairTokens - 1) / kPairTokens) - pair_tail_carve(s), pp.stages,
                        pp.smem, pair_tail_carve(s));
    const Plan pl = make_plan(row_tiles, s.T, s.d_in, true, s.N, s.r, s.k);
    return snprintf(buf, n,
                    "path=chain(not fused: reason %d) launches=3 base_ctas=%d cluster=%d tile_tokens=%d stages=%d kc=%d "
                    "smem=%zu expand=%s",
                    fp.why, row_tiles * pl.splits * pl.n_tiles, pl.splits, pl.BN, pl.stages, pl.kc, pl.smem,
                    pl.lora_mma ? "mma" : "simt");
}

// Knob wait_limit_us: the limit of the bounded device-side waits on the current device (0: the default, about a second).
int set_wait_limit_us(int us) {
    const long long cycles = us > 0 ? (long long)us * 2000LL : kDefaultWaitLimitCycles;   // ~2 GHz SM clock
    return cuda_status(cudaMemcpyToSymbol(g_wait_limit_cycles, &cycles, sizeof(cycles)));
}

}  // namespace meteora

#ifdef METEORA_TRACE
// Trace build only: copy the device-side time stamps of the decode kernel to the host.
extern "C" int meteora_trace_read(unsigned long long* host, size_t count) {
    const size_t total = (size_t)meteora::kTraceCalls * meteora::kTraceCtas * meteora::kTraceSlots;
    if (count > total) count = total;
    return cudaMemcpyFromSymbol(host, meteora::g_fused_trace, count * sizeof(unsigned long long)) == cudaSuccess ? 0 : -5;
}
#endif
