// Whole MeteoRA linear forward for a decode batch (one token tile, T <= 256, rank 8) as ONE kernel launch.
// Included by wgemm_tcgen05.cu after the device helpers it uses.
//
// The grid holds two kinds of CTAs, all resident at the same time (cooperative launch, no clusters):
//   - main CTAs, S per 128-row tile of W0 along the contraction axis: stream W0 through TMA + tcgen05 into
//     TMEM, add the LoRA expand of their share of the adapters as extra MMAs (Eq. 2), write the partial
//     accumulator tile to an fp32 scratch (it stays in L2) and, once the tile's S partials are in, each sums
//     its slice of the rows in split order and stores y;
//   - a few aux CTAs on the SMs the main CTAs leave free: each computes a slice of the stacked shrink
//     [A_0..A_{N-1}; Wg] x (every adapter's A_i x and the gate logits, Sec. 3.1) on the same main loop and
//     writes it as an fp32 partial; once all partials are in, the aux CTAs share the tokens and run the
//     top-k selection and the softmax over the selected logits (Eq. 3), publishing topk_idx, topk_w, uw.
// The main CTAs hold their first loads back until the aux CTAs have issued theirs, so the 2 MB of the shrink
// are ahead of the 33 MB of W0 in the memory queues; they need the routing only for the expand at the end of
// their main loop.  Every wait is bounded; on expiry the status word is set and the kernel drains.  The
// counters live in the workspace header and are re-armed by the last CTA to exit.
#pragma once

namespace meteora {

struct DecodeParams {
    WGemmParams main;      // base product (MODE_LORA, lora_mma): ring geometry, staging offsets, outputs
    int n_main;            // main CTAs = row tiles * S
    int n_aux;             // aux CTAs; they take the lowest block indices so that they are scheduled first
    int a_tiles, a_rows;   // row tiles / rows of the stacked A matrix (N * r rows); one more tile holds Wg
    int aux_slices;        // contraction slices per aux row tile; active aux CTAs = (a_tiles + 1) * aux_slices
    int aux_stages;        // ring depth of the aux main loop (one k-step per stage)
    int bar_stages;        // barriers are laid out for max(main stages, aux stages) ring slots
    float* u_part;         // [aux_slices][T][ld_u] partial stacked shrink
    int ld_u, col_logits;
    int32_t* topk_idx;     // selection results, written by aux CTAs, read by main CTAs
    float* topk_w;
    float* uw;
    float inv_tau;
    int32_t* ctr;          // [0] aux partials written, [1] selections published, [2] CTAs exited, [3] aux loads issued
    float* part_g;         // [row tile][split][BN][128] fp32 partial accumulator tiles of the base product
    int32_t* tile_ctr;     // [row tiles] partials written per tile
    int row_tiles;
    int overlap;           // launched with programmatic stream serialization: prefetch weights, then wait
};

__device__ __forceinline__ int ld_acquire(const int32_t* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Bounded wait until *ctr >= target; false if it did not happen within kWaitLimitCycles.
__device__ __forceinline__ bool wait_counter(const int32_t* ctr, int target) {
    const long long t0 = clock64();
    while (ld_acquire(ctr) < target) {
        if (clock64() - t0 > kWaitLimitCycles) return false;
        __nanosleep(32);
    }
    return true;
}

// Token-side operand of the tensor-core expand: the caller has zeroed it; scatter bf16(w_j * A_e x_t) of the
// slots whose adapter belongs to this CTA, reading the routing with loads that bypass L1 (it was written
// by other CTAs of this same kernel).
__device__ __forceinline__ void scatter_us_mma_coherent(const WGemmParams& p, uint4* us, int a0, int ntok, int etid) {
    const int slots = ntok * p.k;
    const float4* uw4 = reinterpret_cast<const float4*>(p.uw);
    for (int i = etid; i < slots; i += kEpiThreads) {
        const int a = __ldcg(p.topk_idx + i) - a0;
        if (a >= 0 && a < p.na) {
            const float4 lo = __ldcg(uw4 + 2 * i), hi = __ldcg(uw4 + 2 * i + 1);
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

#ifdef METEORA_TRACE
#define FUSED_STAMP(p, base, slot)                                                  \
    do {                                                                            \
        unsigned long long t_;                                                      \
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                      \
        (p).status[(base) + (slot)] = (int)(t_ & 0x7FFFFFFF);                       \
    } while (0)
#else
#define FUSED_STAMP(p, base, slot) do { } while (0)
#endif

__device__ __forceinline__ void flag_error(const WGemmParams& p, int word, int code) {
    atomicExch(p.status, 1);
    atomicExch(p.status + word, code);
}

// Ring geometry of one main loop: stage layout [kc weight tiles of 128 x 64][kc token tiles of BN x 64].
struct RingGeom {
    uint32_t ring, bar_base, x_tile_bytes, stage_bytes;
    int stages, kc, maps3d;
};

// Producer side of a main loop (one thread).  `first_batch_done`, if not null, is bumped once the loads
// that fit into the ring without waiting have been issued.
__device__ __forceinline__ bool fused_producer(const RingGeom& g, const CUtensorMap* tmW, const CUtensorMap* tmXp,
                                               int row0, int ks0, int niter, int32_t* first_batch_done) {
    bool ok = true;
    for (int i = 0; i < niter; ++i) {
        const int s = i % g.stages, round = i / g.stages;
        if (i == g.stages && first_batch_done) {
            atomicAdd(first_batch_done, 1);
            first_batch_done = nullptr;
        }
        if (round > 0) ok = mbar_wait(g.bar_base + (g.stages + s) * 8, (round & 1) ^ 1);
        if (!ok) break;
        const uint32_t full = g.bar_base + s * 8;
        const uint32_t dst = g.ring + s * g.stage_bytes;
        const int kstep = ks0 + i * g.kc;
        mbar_expect_tx(full, g.stage_bytes);
        if (g.maps3d) {
            tma_load_3d(dst, tmW, 0, row0, kstep, full);
            tma_load_3d(dst + g.kc * kWTileBytes, tmXp, 0, 0, kstep, full);
        } else {
            tma_load_2d(dst, tmW, kstep * kBK, row0, full);
            tma_load_2d(dst + kWTileBytes, tmXp, kstep * kBK, 0, full);
        }
    }
    if (first_batch_done) atomicAdd(first_batch_done, 1);
    return ok;
}

// MMA side of a main loop (one thread); does not commit the accumulator barrier.
__device__ __forceinline__ bool fused_mma(const RingGeom& g, uint32_t tmem_base, uint32_t idesc, int niter) {
    bool ok = true;
    for (int i = 0; i < niter; ++i) {
        const int s = i % g.stages, round = i / g.stages;
        ok = mbar_wait(g.bar_base + s * 8, round & 1);
        if (!ok) break;
        tc_fence_after();
        const uint32_t wa = g.ring + s * g.stage_bytes, xa = wa + g.kc * kWTileBytes;
        for (int c = 0; c < g.kc; ++c) {
            const uint64_t da = smem_desc_sw128(wa + c * kWTileBytes);
            const uint64_t db = smem_desc_sw128(xa + c * g.x_tile_bytes);
#pragma unroll
            for (int kk = 0; kk < kBK / kUmmaK; ++kk)
                umma_bf16(tmem_base, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (i | c | kk) != 0);
        }
        umma_commit(g.bar_base + (g.stages + s) * 8);
    }
    return ok;
}

__global__ void __launch_bounds__(kThreads)
k_decode_fused(const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmX,
               const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmG,
               const __grid_constant__ CUtensorMap tmX1, const DecodeParams d) {
    const WGemmParams& p = d.main;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;
    uint8_t* ring_ptr = smem_raw + (ring - raw);
    const uint32_t x_tile_bytes = p.BN * 128;
    const uint32_t stage_bytes = p.kc * (kWTileBytes + x_tile_bytes);
    const uint32_t ring_bytes = p.stages * stage_bytes;
    const uint32_t bar_base = ring + ring_bytes;
    const int nbar = 2 * d.bar_stages + 3;           // sized for the deeper of the two rings
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ring_ptr + ring_bytes + nbar * 8);
    uint8_t* epi = ring_ptr + ring_bytes + p.epi_off;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool is_aux = (int)blockIdx.x < d.n_aux;
    const int main_id = (int)blockIdx.x - d.n_aux;
    const int n_active = (d.a_tiles + 1) * d.aux_slices;

    if (threadIdx.x == 0) {
        for (int s = 0; s < nbar; ++s) mbar_init(bar_base + s * 8, 1);
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
    const uint32_t idesc = instr_desc_bf16(p.BN);
    const int quad = warp & 3;
    const int etid = threadIdx.x - 64;
    const int ntok = min(p.BN, p.T);
    const int half = ((p.BN / 16 + 1) / 2) * 16;
    const int c_begin = warp < 6 ? 0 : half, c_end = warp < 6 ? half : p.BN;
    const bool tr_main = main_id == 0, tr_aux = blockIdx.x == 0;

    if (d.overlap) {
        // Overlap with the previous kernel of the stream: it may still be running.  Until it has completed
        // (griddepcontrol.wait) nothing it could have written is read and nothing is written; the weights of
        // this CTA are only pulled into L2, which changes no value anyone can observe.
        if (threadIdx.x == 0) {
            asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
            if (is_aux) {
                if ((int)blockIdx.x < n_active) {
                    const int tile = blockIdx.x % (d.a_tiles + 1), slice = blockIdx.x / (d.a_tiles + 1);
                    const int k0 = (int)(((long long)p.ksteps * slice) / d.aux_slices);
                    const int k1 = (int)(((long long)p.ksteps * (slice + 1)) / d.aux_slices);
                    const bool is_gate = tile >= d.a_tiles;
                    for (int ks = k0; ks < k1; ++ks) {
                        if (p.maps3d) tma_prefetch_3d(is_gate ? &tmG : &tmA, 0, is_gate ? 0 : tile * kBM, ks);
                        else tma_prefetch_2d(is_gate ? &tmG : &tmA, ks * kBK, is_gate ? 0 : tile * kBM);
                    }
                }
            } else {
                const int S = p.splits, split = main_id % S, tile_m = main_id / S;
                const int k0 = (int)(((long long)p.ksteps * split) / S);
                const int k1 = (int)(((long long)p.ksteps * (split + 1)) / S);
                for (int ks = k0; ks < k1; ks += p.kc) {
                    if (p.maps3d) tma_prefetch_3d(&tmW0, 0, tile_m * kBM, ks);
                    else tma_prefetch_2d(&tmW0, ks * kBK, tile_m * kBM);
                }
                // B rows of this split's adapters for the tile's 128 output rows (2 KB per adapter)
                const int row0 = tile_m * kBM, rows = min(kBM, p.d_out - row0);
                for (int a = split * p.na; a < min(p.N, (split + 1) * p.na); ++a)
                    bulk_prefetch_l2(p.B + ((size_t)a * p.d_out + row0) * 8, (uint32_t)rows * 16u);
            }
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }
    if (threadIdx.x == 0 && tr_main) FUSED_STAMP(p, 32, 0);
    if (threadIdx.x == 0 && tr_aux) FUSED_STAMP(p, 48, 0);

    if (is_aux) {
        // ================================================================== aux CTA
        const int aux_id = blockIdx.x;
        const bool active = aux_id < n_active;
        const int tile = aux_id % (d.a_tiles + 1), slice = aux_id / (d.a_tiles + 1);
        const int ks0 = active ? (int)(((long long)p.ksteps * slice) / d.aux_slices) : 0;
        const int ks1 = active ? (int)(((long long)p.ksteps * (slice + 1)) / d.aux_slices) : 0;
        const int niter = ks1 - ks0;
        const RingGeom geom = {ring, bar_base, x_tile_bytes, kWTileBytes + x_tile_bytes, d.aux_stages, 1, p.maps3d};
        const uint32_t bar_acc = bar_base + 2 * d.aux_stages * 8;
        if (warp == 0) {
            if (lane == 0 && active) {
                const bool is_gate = tile >= d.a_tiles;
                if (!fused_producer(geom, is_gate ? &tmG : &tmA, &tmX1, is_gate ? 0 : tile * kBM, ks0, niter,
                                    d.ctr + 3))
                    flag_error(p, 1, 400);
            }
        } else if (warp == 1) {
            if (lane == 0 && active) {
                if (!fused_mma(geom, tmem_base, idesc, niter)) flag_error(p, 2, 500);
                umma_commit(bar_acc);
                if (tr_aux) FUSED_STAMP(p, 48, 1);
            }
        } else if (active) {
            bool acc_ok = mbar_wait(bar_acc, 0);
            if (!acc_ok && lane == 0) flag_error(p, 3, 600);
            acc_ok = __all_sync(0xFFFFFFFFu, acc_ok);
            tc_fence_after();
            // accumulators straight to the partial buffer: lane = row, a warp writes 128 contiguous bytes
            const int row = tile < d.a_tiles ? tile * kBM + quad * 32 + lane : quad * 32 + lane;
            const int limit = tile < d.a_tiles ? d.a_rows : p.N;
            const int col = tile < d.a_tiles ? row : d.col_logits + row;
            float* dst = d.u_part + (size_t)slice * p.T * d.ld_u + col;
            for (int c = c_begin; c < c_end; c += 16) {
                float v[16];
                if (acc_ok) {
                    tmem_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + c, v);
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = 0.f;
                }
                if (row < limit) {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (c + i < p.T) dst[(size_t)(c + i) * d.ld_u] = v[i];
                }
            }
        }
        __syncwarp();
        __syncthreads();
        if (active) {
            if (threadIdx.x == 0) {
                if (tr_aux) FUSED_STAMP(p, 48, 2);
                __threadfence();
                atomicAdd(d.ctr + 0, 1);
                if (!wait_counter(d.ctr + 0, n_active)) flag_error(p, 4, 700);   // every slice of every tile is in
                if (tr_aux) FUSED_STAMP(p, 48, 3);
            }
            __syncthreads();
            const int nwarps = kThreads / 32;                                    // tokens dealt round-robin
            for (int t = aux_id * nwarps + warp; t < p.T; t += n_active * nwarps)
                select_token<true>(d.u_part, d.ld_u, d.col_logits, d.aux_slices, (size_t)p.T * d.ld_u, t, p.N, p.r,
                                   p.k, d.inv_tau, lane, d.topk_idx, d.topk_w, d.uw);
            __syncthreads();
            if (threadIdx.x == 0) {
                __threadfence();
                atomicAdd(d.ctr + 1, 1);
                if (tr_aux) FUSED_STAMP(p, 48, 4);
            }
        }
    } else {
        // ================================================================== main CTA
        const int S = p.splits;
        const int split = main_id % S;
        const int tile_m = main_id / S;
        const int ks0 = (int)(((long long)p.ksteps * split) / S);
        const int ks1 = (int)(((long long)p.ksteps * (split + 1)) / S);
        const int niter = (ks1 - ks0) / p.kc;
        const RingGeom geom = {ring, bar_base, x_tile_bytes, stage_bytes, p.stages, p.kc, p.maps3d};
        const uint32_t bar_acc = bar_base + 2 * p.stages * 8, bar_us = bar_acc + 16;
        const size_t part_stride = (size_t)p.BN * kBM;                       // floats per partial tile
        float* my_part = d.part_g + ((size_t)tile_m * S + split) * part_stride;
        if (warp == 0) {
            if (lane == 0) {
                // let the stacked shrink get its loads into the memory queues first
                bool ok = wait_counter(d.ctr + 3, n_active);
                if (tr_main) FUSED_STAMP(p, 32, 1);
                ok = fused_producer(geom, &tmW0, &tmX, tile_m * kBM, ks0, niter, nullptr) && ok;
                if (!ok) flag_error(p, 1, 100);
            }
        } else if (warp == 1) {
            if (lane == 0) {
                bool ok = fused_mma(geom, tmem_base, idesc, niter);
                if (tr_main) FUSED_STAMP(p, 32, 2);
                if (ok) ok = mbar_wait(bar_us, 0);                            // operands of the expand staged
                if (ok) {
                    tc_fence_after();
                    const uint32_t slab_a = smem_u32(epi + p.slab_off), us_a = smem_u32(epi + p.us_off);
                    const uint32_t ka = kBM * 16, kb = p.BN * 16;
                    for (int m = 0; m < p.na / 2; ++m)
                        umma_bf16(tmem_base, smem_desc_plain(slab_a + 2 * m * ka, ka, 128),
                                  smem_desc_plain(us_a + 2 * m * kb, kb, 128), idesc, (niter | m) != 0);
                }
                umma_commit(bar_acc);
                if (!ok) flag_error(p, 2, 200);
            }
        } else {
            const int a0 = split * p.na;
            stage_slab_mma(p, epi, a0, tile_m * kBM, etid);                   // B rows: no routing needed
            uint4* us = reinterpret_cast<uint4*>(epi + p.us_off);
            for (int v = etid; v < p.na * p.BN; v += kEpiThreads) us[v] = make_uint4(0u, 0u, 0u, 0u);
            if (etid == 0 && tr_main) FUSED_STAMP(p, 32, 3);
            if (etid == 0 && !wait_counter(d.ctr + 1, n_active)) flag_error(p, 4, 800);   // routing published
            if (etid == 0 && tr_main) FUSED_STAMP(p, 32, 4);
            epi_barrier();
            scatter_us_mma_coherent(p, us, a0, ntok, etid);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            epi_barrier();
            if (etid == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_us) : "memory");
            bool acc_ok = mbar_wait(bar_acc, 0);
            if (!acc_ok && lane == 0) flag_error(p, 3, 300);
            acc_ok = __all_sync(0xFFFFFFFFu, acc_ok);
            tc_fence_after();
            if (etid == 0 && tr_main) FUSED_STAMP(p, 32, 5);
            // Accumulators out of TMEM: to the fp32 scratch when the tile is split over several CTAs (lane =
            // row, a warp writes 128 contiguous bytes per token), else to the idle ring.
            float* part = S > 1 ? my_part : reinterpret_cast<float*>(ring_ptr);
            const int row_in_tile = quad * 32 + lane;
            for (int c = c_begin; c < c_end; c += 16) {
                float v[16];
                if (acc_ok) {
                    tmem_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + c, v);
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = 0.f;
                }
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    if (S == 1 || c + i < ntok) part[(c + i) * kBM + row_in_tile] = v[i];
            }
            epi_barrier();
            if (S > 1 && etid == 0) {
                __threadfence();
                atomicAdd(d.tile_ctr + tile_m, 1);
                if (!wait_counter(d.tile_ctr + tile_m, S)) flag_error(p, 4, 900);   // all partials of the tile in
            }
            if (etid == 0 && tr_main) FUSED_STAMP(p, 32, 6);
            epi_barrier();
            // sum the slice of rows this CTA owns over the S partials, in split order, and store y
            const int P = 64 / S, TPP = kEpiThreads / P, NROWS = kBM / S;
            const int pr = etid % P, tg = etid / P;
            const int rit = NROWS * split + 2 * pr;
            const int o = tile_m * kBM + rit;
            const float* src = S > 1 ? d.part_g + (size_t)tile_m * S * part_stride : part;
            for (int t0 = tg; t0 < ntok; t0 += 4 * TPP) {
                float2 acc[4], v[4][8];
                // all partial loads of four tokens first (one L2 round trip), then the sums in split order
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int t = min(t0 + u * TPP, ntok - 1);
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        v[u][q] = make_float2(0.f, 0.f);
                        if (q < S) {
                            const float2* a = reinterpret_cast<const float2*>(src + q * part_stride + t * kBM + rit);
                            v[u][q] = S > 1 ? __ldcg(a) : *a;
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    acc[u] = make_float2(0.f, 0.f);
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        if (q < S) {
                            acc[u].x += v[u][q].x;
                            acc[u].y += v[u][q].y;
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int t = t0 + u * TPP;
                    if (t >= ntok) break;
                    __nv_bfloat16* dst = p.y + (size_t)t * p.d_out + o;
                    if (o + 1 < p.d_out && (p.d_out & 1) == 0) {
                        *reinterpret_cast<__nv_bfloat162*>(dst) = __floats2bfloat162_rn(acc[u].x, acc[u].y);
                    } else {
                        if (o < p.d_out) dst[0] = __float2bfloat16_rn(acc[u].x);
                        if (o + 1 < p.d_out) dst[1] = __float2bfloat16_rn(acc[u].y);
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && tr_main) FUSED_STAMP(p, 32, 7);
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                     "r"((uint32_t)p.tmem_cols)
                     : "memory");
    }
    if (threadIdx.x == 0) {
        // the last CTA out re-arms the counters for the next call on this workspace
        if (atomicAdd(d.ctr + 2, 1) == (int)gridDim.x - 1) {
            d.ctr[0] = 0;
            d.ctr[1] = 0;
            d.ctr[3] = 0;
            for (int i = 0; i < d.row_tiles; ++i) d.tile_ctr[i] = 0;
            __threadfence();
            d.ctr[2] = 0;
        }
    }
}

}  // namespace meteora
