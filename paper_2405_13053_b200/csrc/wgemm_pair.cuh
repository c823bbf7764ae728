// Base product W0 x with the LoRA expand (Eq. 2) for prefill batches on PAIRS of SMs.
// Included by wgemm_tcgen05.cu after the device helpers it uses.
//
// A 128 x 256 tile per SM reads 48 KB of operands per k-step for 4.2 MFLOP, and the L2 -> SM path cannot feed
// the tensor cores at that ratio.  Here a cluster of two CTAs computes a 256 (rows of W0) x 256 (tokens) tile
// with tcgen05.mma.cta_group::2: each CTA loads ITS 128 rows of W0 and ITS 128 of the 256 tokens (32 KB per
// k-step), the tensor cores of both SMs read both halves of the token operand, and each CTA ends up with the
// accumulators of its own 128 rows for all 256 tokens in its own TMEM.  No load is multicast.
//
//   warp 0 (both CTAs)  TMA producer: own W0 rows and own token half into the own ring; every copy signals the
//                       LEADER's (cluster rank 0) full barrier, whose expected byte count covers both CTAs.
//   warp 1              TMEM allocation (both CTAs, pair-wide form); MMA issue by the leader only.  A stage is
//                       released, and completion is announced, by tcgen05.commit multicast to both CTAs.
//   warps 2-9 (both)    stage the B rows of the own 128 rows for every adapter while the main loop runs; when
//                       the ring is idle, stage the masked, gate-weighted shrink outputs of the own 128 tokens
//                       there and tell the leader; it then issues more MMAs of K = 16 into the same
//                       accumulators.  The expand's contraction axis is cut into blocks of 8 (adapter a, rank
//                       entries 8c..8c+7): N * r / 8 blocks, two per MMA, at most 28 blocks (56 KB of B rows) per
//                       round; rank 8 with 28 adapters is one round, larger ranks take several, each staged
//                       after the previous round's MMAs have completed.  Finally TMEM -> bf16 -> shared
//                       memory -> one TMA store of the own 128 x 256 tile of y.
// Every wait is bounded; the pair leaves together (cluster barrier) so that no signal arrives in a CTA that is gone.
#pragma once

namespace meteora {

constexpr int kPairTokens = 256;   // tokens per pair tile (UMMA N)
constexpr int kPairHalf = 128;     // tokens each CTA loads

__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
    uint32_t a;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(local_addr), "r"(rank));
    return a;
}
// 2-D tile load whose completion bytes go to a barrier that may live in the peer CTA of the pair.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* tm, int c0, int c1,
                                                 uint32_t cluster_bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"((uint64_t)tm), "r"(c0), "r"(c1), "r"(cluster_bar)
        : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrives, once the MMAs issued so far have completed, on the barrier at this offset in BOTH CTAs of the pair.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"((uint16_t)3)
        : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait on a barrier that threads of the peer CTA arrive on.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity) {
    if (mbar_try_cluster(bar, parity)) return true;
    const long long t0 = clock64(), limit = g_wait_limit_cycles;
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try_cluster(bar, parity)) return true;
        if ((spin & 0x3FF) == 0 && clock64() - t0 > limit) return false;
    }
}
// fp32 accumulate, bf16 x bf16, both operands K-major, M = 256 over the pair, N = 256.
__device__ __forceinline__ uint32_t instr_desc_bf16_pair() {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kPairTokens >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

struct PairParams {
    int T, K, ksteps, stages;
    int d_out, N, k, r;           // rank r: a multiple of 8
    int nblk, rb;                 // blocks of 8 expand columns: N * r / 8 in all, rb (even) per round
    int row_tiles;
    int group_pairs;              // row pairs per scheduling group (see the kernel: which tile a pair of CTAs takes)
    int epi_off, slab_off;        // staging area behind the barriers; the B rows sit at slab_off inside it
    const int32_t* topk_idx;
    const float* uw;
    const __nv_bfloat16* B;
    int32_t* status;
    int pdl_wait;
    int skip_rp0, skip_tt0;       // tiles with row pair >= skip_rp0 AND token tile >= skip_tt0 are another launch's
    int pdl_trigger;              // that launch follows: let it become resident as this launch's last wave drains
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads)
k_wgemm_pair(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
             const __grid_constant__ CUtensorMap tmY, const PairParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;
    uint8_t* ring_ptr = smem_raw + (ring - raw);
    constexpr uint32_t kXHalfBytes = kPairHalf * 128;             // 128 tokens x 64 bf16
    constexpr uint32_t kStageBytes = kWTileBytes + kXHalfBytes;   // per CTA
    const uint32_t ring_bytes = p.stages * kStageBytes;
    const uint32_t bar_base = ring + ring_bytes;                  // full[stages], empty[stages], acc, main, us
    const uint32_t bar_acc = bar_base + 2 * p.stages * 8;
    const uint32_t bar_main = bar_acc + 8;
    const uint32_t bar_us = bar_acc + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ring_ptr + ring_bytes + (2 * p.stages + 3) * 8);
    uint8_t* epi = ring_ptr + ring_bytes + p.epi_off;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const bool leader = rank == 0;
    // Which tile this pair takes.  Pairs are dispatched in the order of p = blockIdx.y * (gridDim.x / 2) + blockIdx.x / 2;
    // taken row-major (all row pairs of one token tile, then the next token tile) every token tile streams the whole of
    // W0 again, and once W0 is about as large as the L2 each pass comes from HBM: 764 MB of DRAM reads per launch at
    // 4096 -> 14336 with 2048 tokens, 6.5 times W0.  Instead the row pairs are cut into groups of `group_pairs`, and a
    // group's row pairs run over ALL token tiles before the next group starts: the pairs resident at one time then
    // share a few row pairs of W0 (read from HBM once, found in L2 by the other token tiles) and all of x (small).
    const int row_pairs = (int)gridDim.x >> 1, tok_tiles = (int)gridDim.y;
    const int lin = (int)blockIdx.y * row_pairs + ((int)blockIdx.x >> 1);
    const int per_group = p.group_pairs * tok_tiles;
    const int grp = lin / per_group, rem = lin - grp * per_group;
    const int in_grp = min(p.group_pairs, row_pairs - grp * p.group_pairs);     // the last group may be smaller
    const int tok_tile = rem / in_grp, row_pair = grp * p.group_pairs + rem - tok_tile * in_grp;
    // The tiles of a last, nearly empty wave are carved out of this launch (a launch of small tiles takes them): both
    // CTAs of such a pair leave before they touch a barrier or TMEM.
    if (row_pair >= p.skip_rp0 && tok_tile >= p.skip_tt0) return;
    const int tile_m = row_pair * 2 + (int)rank;                  // own 128 rows of W0 / y
    const int tok0 = tok_tile * kPairTokens;                      // the pair's 256 tokens
    const int tokh = tok0 + (int)rank * kPairHalf;                // own half of them
    const int niter = p.ksteps;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(bar_base + s * 8, 1);                       // the leader's expect-tx arrival
            mbar_init(bar_base + (p.stages + s) * 8, 1);          // one multicast commit
        }
        mbar_init(bar_acc, 1);
        mbar_init(bar_main, 1);
        mbar_init(bar_us, 2);                                     // one arrival from each CTA's epilogue warps
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"((uint32_t)kPairTokens)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncwarp();
    cluster_sync();                                               // both CTAs' barriers exist before anyone signals
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_slot);
    if (p.pdl_trigger && threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            bool ok = true;
            int issued = 0;
            for (int i = 0; i < niter; ++i) {
                const int s = i % p.stages, round = i / p.stages;
                if (round > 0) ok = mbar_wait(bar_base + (p.stages + s) * 8, (round & 1) ^ 1);
                if (!ok) break;
                const uint32_t full = bar_base + s * 8;
                const uint32_t full_leader = map_to_cta(full, 0);
                const uint32_t dst = ring + s * kStageBytes;
                if (leader) mbar_expect_tx(full, 2 * kStageBytes);
                tma_load_2d_pair(dst, &tmW, i * kBK, tile_m * kBM, full_leader);
                tma_load_2d_pair(dst + kWTileBytes, &tmX, i * kBK, tokh, full_leader);
                issued = i + 1;
            }
            if (!ok) {
                atomicExch(p.status, 1);
                atomicExch(p.status + 1, 1100 + issued);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader only)
        if (lane == 0 && leader) {
            const uint32_t idesc = instr_desc_bf16_pair();
            bool ok = true;
            for (int i = 0; i < niter; ++i) {
                const int s = i % p.stages, round = i / p.stages;
                ok = mbar_wait(bar_base + s * 8, round & 1);
                if (!ok) break;
                tc_fence_after();
                const uint32_t wa = ring + s * kStageBytes, xa = wa + kWTileBytes;
                const uint64_t da = smem_desc_sw128(wa), db = smem_desc_sw128(xa);
#pragma unroll
                for (int kk = 0; kk < kBK / kUmmaK; ++kk)
                    umma_bf16_pair(tmem_base, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (i | kk) != 0);
                umma_commit_pair(bar_base + (p.stages + s) * 8);  // both rings may refill this stage
            }
            umma_commit_pair(bar_main);                            // both rings are idle
            // LoRA expand as a K extension of the same accumulation, round by round: rb/2 MMAs of K = 16 (two
            // blocks of 8 expand columns) over un-swizzled core matrices, 2 KB per block and operand
            const int rounds = (p.nblk + p.rb - 1) / p.rb;
            for (int rho = 0; rho < rounds && ok; ++rho) {
                ok = mbar_wait_cluster(bar_us, rho & 1);           // both CTAs have staged this round's operands
                if (!ok) break;
                tc_fence_after();
                const uint32_t slab_a = smem_u32(epi + p.slab_off), us_a = ring;
                const uint32_t ka = kBM * 16, kb = kPairHalf * 16;   // bytes from one block to the next
                const int nb = min(p.rb, (p.nblk - rho * p.rb + 1) / 2 * 2);
                for (int m = 0; m < nb / 2; ++m)
                    umma_bf16_pair(tmem_base, smem_desc_plain(slab_a + 2 * m * ka, ka, 128),
                                   smem_desc_plain(us_a + 2 * m * kb, kb, 128), idesc, (niter | rho | m) != 0);
                if (rho + 1 < rounds) umma_commit_pair(bar_main);  // staging buffers free for the next round
            }
            umma_commit_pair(bar_acc);                             // accumulators complete in both CTAs
            if (!ok) {
                atomicExch(p.status, 1);
                atomicExch(p.status + 2, 1200);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps (both CTAs)
        const int quad = warp & 3;
        const int etid = threadIdx.x - 64;
        // Round by round: B rows of the own 128 output rows (block q = adapter q / (r/8), rank entries 8 (q % (r/8)) ..,
        // 16 bytes per row: un-swizzled K-major core matrices) and us[q][t 0..128)[8] = bf16(w_j * (A_a x_t)[8c..])
        // where own token t picked adapter a at rank j, else 0.  Round 0's B rows are staged while the main loop
        // runs; everything else waits until the MMAs that read the buffers before have completed.
        const int cpa = p.r >> 3;                                   // blocks per adapter
        const int rounds = (p.nblk + p.rb - 1) / p.rb;
        const int ntok = max(0, min(kPairHalf, p.T - tokh));
        bool ring_ok = true;
        for (int rho = 0; rho < rounds; ++rho) {
            const int q0 = rho * p.rb, nb = min(p.rb, (p.nblk - q0 + 1) / 2 * 2);
            if (rho > 0) {
                ring_ok = ring_ok && mbar_wait(bar_main, rho & 1);   // previous round's MMAs done
            }
            {
                uint4* slab = reinterpret_cast<uint4*>(epi + p.slab_off);
                const uint4* Bv = reinterpret_cast<const uint4*>(p.B);
                const int total = nb * kBM;
                constexpr int U = 4;
                for (int v0 = etid; v0 < total; v0 += U * kEpiThreads) {
                    uint4 val[U];
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const int v = v0 + u * kEpiThreads;
                        const int q = q0 + v / kBM, row = v % kBM;
                        const int a = q / cpa, c = q - a * cpa;
                        val[u] = make_uint4(0u, 0u, 0u, 0u);
                        if (v < total && a < p.N && tile_m * kBM + row < p.d_out)
                            val[u] = __ldg(Bv + ((size_t)a * p.d_out + tile_m * kBM + row) * cpa + c);
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const int v = v0 + u * kEpiThreads;
                        if (v < total) slab[v] = val[u];
                    }
                }
            }
            if (rho == 0) {
                if (p.pdl_wait) asm volatile("griddepcontrol.wait;" ::: "memory");   // the routing comes from the previous kernel
                ring_ok = mbar_wait(bar_main, 0);                   // main loop done: the ring is idle
            }
            if (!ring_ok && lane == 0) {
                atomicExch(p.status, 1);
                atomicExch(p.status + 4, 1350);
            }
            {
                uint4* us = reinterpret_cast<uint4*>(ring_ptr);
                const int total = nb * kPairHalf;
                for (int v = etid; v < total; v += kEpiThreads) us[v] = make_uint4(0u, 0u, 0u, 0u);
                epi_barrier();
                const int items = ntok * p.k * cpa;                  // (token, pick, chunk of 8 rank entries)
                const int32_t* idx = p.topk_idx + (size_t)tokh * p.k;
                const float4* uw4 = reinterpret_cast<const float4*>(p.uw + (size_t)tokh * p.k * p.r);
                for (int i = etid; i < items; i += kEpiThreads) {
                    const int slot = i / cpa, c = i - slot * cpa;
                    const int a = __ldg(idx + slot);
                    const int q = a * cpa + c - q0;
                    if (a >= 0 && a < p.N && q >= 0 && q < nb) {
                        const float4 lo = __ldg(uw4 + 2 * i), hi = __ldg(uw4 + 2 * i + 1);
                        const __nv_bfloat162 h0 = __floats2bfloat162_rn(lo.x, lo.y), h1 = __floats2bfloat162_rn(lo.z, lo.w);
                        const __nv_bfloat162 h2 = __floats2bfloat162_rn(hi.x, hi.y), h3 = __floats2bfloat162_rn(hi.z, hi.w);
                        uint4 val;
                        val.x = *reinterpret_cast<const uint32_t*>(&h0);
                        val.y = *reinterpret_cast<const uint32_t*>(&h1);
                        val.z = *reinterpret_cast<const uint32_t*>(&h2);
                        val.w = *reinterpret_cast<const uint32_t*>(&h3);
                        us[q * kPairHalf + slot / p.k] = val;
                    }
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> tensor-core reads
            epi_barrier();
            if (etid == 0) mbar_arrive_cluster(map_to_cta(bar_us, 0));
        }
        bool acc_ok = mbar_wait(bar_acc, 0);
        if (!acc_ok && lane == 0) {
            atomicExch(p.status, 1);
            atomicExch(p.status + 3, 1300);
        }
        acc_ok = __all_sync(0xFFFFFFFFu, acc_ok);
        tc_fence_after();
        // own 128 rows x 256 tokens: round once and stage as ystage[t][row] in the idle ring
        __nv_bfloat16* ystage = reinterpret_cast<__nv_bfloat16*>(ring_ptr);
        const int row_in_tile = quad * 32 + lane;
        const int c_begin = warp < 6 ? 0 : kPairTokens / 2, c_end = warp < 6 ? kPairTokens / 2 : kPairTokens;
        for (int c = c_begin; c < c_end; c += 16) {
            float v[16];
            if (acc_ok) {
                tmem_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + c, v);
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = 0.f;
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) ystage[(c + i) * kBM + row_in_tile] = __float2bfloat16_rn(v[i]);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> TMA read
    }
    __syncwarp();
    __syncthreads();
    // one copy moves the whole 128 x 256 tile; rows beyond d_out and tokens beyond T are clipped by the map
    if (threadIdx.x == 64 && tile_m < p.row_tiles) tma_store_2d_and_wait(&tmY, ring, tile_m * kBM, tok0);
    tc_fence_before();
    __syncwarp();
    cluster_sync();                                               // nobody leaves while the peer may still signal it
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                     "r"((uint32_t)kPairTokens)
                     : "memory");
    }
}

// ------------------------------------------------------------------------------------------------
// Stacked shrink [A_0..A_{N-1}; Wg] x for prefill batches on pairs of SMs: the 256 rows of a pair tile are two
// 128-row tiles of the stacked matrix (for N = 28, rank 8 that is all of it: A's rows 0..127 in the leader,
// A's rows 128..223 followed by the 28 rows of Wg in its peer), the 256 tokens are split as above.  Slices of
// the contraction axis go over grid z; each writes its fp32 partial straight from TMEM to u_all[z].
// ------------------------------------------------------------------------------------------------
struct StackedPairParams {
    int T, ksteps, stages, zsplits;
    int a_tiles, a_rows, aux_tiles, gate_tile, gate_row0, N;
    float* u_all;
    size_t zstride;
    int ld_u, col_logits;
    int32_t* status;
    int pdl_trigger;
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads)
k_stacked_pair(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmAt,
               const __grid_constant__ CUtensorMap tmG, const __grid_constant__ CUtensorMap tmX,
               const StackedPairParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;
    uint8_t* ring_ptr = smem_raw + (ring - raw);
    constexpr uint32_t kXHalfBytes = kPairHalf * 128;
    constexpr uint32_t kStageBytes = kWTileBytes + kXHalfBytes;
    const uint32_t ring_bytes = p.stages * kStageBytes;
    const uint32_t bar_base = ring + ring_bytes;                  // full[stages], empty[stages], acc
    const uint32_t bar_acc = bar_base + 2 * p.stages * 8;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ring_ptr + ring_bytes + (2 * p.stages + 1) * 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const bool leader = rank == 0;
    const int tile = (blockIdx.x >> 1) * 2 + (int)rank;           // own 128 rows of the stacked matrix
    const int tok0 = blockIdx.y * kPairTokens;
    const int tokh = tok0 + (int)rank * kPairHalf;
    const int ks0 = (int)(((long long)p.ksteps * blockIdx.z) / p.zsplits);
    const int ks1 = (int)(((long long)p.ksteps * (blockIdx.z + 1)) / p.zsplits);
    const int niter = ks1 - ks0;

    if (p.pdl_trigger && threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(bar_base + s * 8, 1);
            mbar_init(bar_base + (p.stages + s) * 8, 1);
        }
        mbar_init(bar_acc, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"((uint32_t)kPairTokens)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncwarp();
    cluster_sync();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_slot);

    if (warp == 0) {
        if (lane == 0) {
            // Own tile of the stacked matrix: rows of A (the last A tile through the map whose box stops at A's
            // last row when Wg follows in the same tile), rows of Wg, or nothing but zero fill (a tile past
            // the end reads A out of range).  Every stage is 16 KB of weights + 16 KB of tokens whatever the tile.
            const bool has_a = tile < p.a_tiles || tile != p.gate_tile;
            const bool merged_tail = tile == p.a_tiles - 1 && tile == p.gate_tile;
            const CUtensorMap* mA = merged_tail ? &tmAt : &tmA;
            bool ok = true;
            int issued = 0;
            for (int i = 0; i < niter; ++i) {
                const int s = i % p.stages, round = i / p.stages;
                if (round > 0) ok = mbar_wait(bar_base + (p.stages + s) * 8, (round & 1) ^ 1);
                if (!ok) break;
                const uint32_t full = bar_base + s * 8;
                const uint32_t full_leader = map_to_cta(full, 0);
                const uint32_t dst = ring + s * kStageBytes;
                const int c0 = (ks0 + i) * kBK;
                if (leader) mbar_expect_tx(full, 2 * kStageBytes);
                if (has_a) tma_load_2d_pair(dst, mA, c0, tile * kBM, full_leader);
                if (tile == p.gate_tile) tma_load_2d_pair(dst + (uint32_t)p.gate_row0 * 128u, &tmG, c0, 0, full_leader);
                tma_load_2d_pair(dst + kWTileBytes, &tmX, c0, tokh, full_leader);
                issued = i + 1;
            }
            if (!ok) {
                atomicExch(p.status, 1);
                atomicExch(p.status + 1, 2100 + issued);
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && leader) {
            const uint32_t idesc = instr_desc_bf16_pair();
            bool ok = true;
            for (int i = 0; i < niter; ++i) {
                const int s = i % p.stages, round = i / p.stages;
                ok = mbar_wait(bar_base + s * 8, round & 1);
                if (!ok) break;
                tc_fence_after();
                const uint32_t wa = ring + s * kStageBytes, xa = wa + kWTileBytes;
                const uint64_t da = smem_desc_sw128(wa), db = smem_desc_sw128(xa);
#pragma unroll
                for (int kk = 0; kk < kBK / kUmmaK; ++kk)
                    umma_bf16_pair(tmem_base, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (i | kk) != 0);
                umma_commit_pair(bar_base + (p.stages + s) * 8);
            }
            umma_commit_pair(bar_acc);
            if (!ok) {
                atomicExch(p.status, 1);
                atomicExch(p.status + 2, 2200);
            }
        }
    } else {
        const int quad = warp & 3;
        bool acc_ok = mbar_wait(bar_acc, 0);
        if (!acc_ok && lane == 0) {
            atomicExch(p.status, 1);
            atomicExch(p.status + 3, 2300);
        }
        acc_ok = __all_sync(0xFFFFFFFFu, acc_ok);
        tc_fence_after();
        // accumulators straight to u_all[z]: lane = row of the tile = column of u_all, 128 contiguous bytes per warp
        const int trow = quad * 32 + lane;
        int col = -1;                                                        // -1: padding row
        if (tile < p.a_tiles && tile * kBM + trow < p.a_rows && !(tile == p.gate_tile && trow >= p.gate_row0))
            col = tile * kBM + trow;
        if (tile == p.gate_tile && trow >= p.gate_row0 && trow < p.gate_row0 + p.N)
            col = p.col_logits + trow - p.gate_row0;
        float* dst = p.u_all + (size_t)blockIdx.z * p.zstride + (size_t)tok0 * p.ld_u + max(col, 0);
        const int ntok = min(kPairTokens, p.T - tok0);
        const int c_begin = warp < 6 ? 0 : kPairTokens / 2, c_end = warp < 6 ? kPairTokens / 2 : kPairTokens;
        for (int c = c_begin; c < c_end; c += 16) {
            float v[16];
            if (acc_ok && niter > 0) {
                tmem_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + c, v);
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = 0.f;
            }
            if (col >= 0) {
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    if (c + i < ntok) dst[(size_t)(c + i) * p.ld_u] = v[i];
            }
        }
    }
    tc_fence_before();
    __syncwarp();
    cluster_sync();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                     "r"((uint32_t)kPairTokens)
                     : "memory");
    }
}

}  // namespace meteora
