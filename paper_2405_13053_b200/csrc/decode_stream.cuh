// Whole MeteoRA linear forward (Eq. 2 with Eq. 3) for a decode batch of up to 128 tokens as ONE kernel launch
// whose CTAs are small enough that TWO launches fit on the SMs at the same time, so that under programmatic
// dependent launch the next call's CTAs are resident while this call still runs.
// Included by wgemm_tcgen05.cu after decode_fused.cuh, whose device helpers it shares.
//
// What a resident CTA of the NEXT call does before the call ahead of it has completed touches only weights,
// which never depend on an earlier kernel: it fills its ring with the first tiles of W0 (or of [A; Wg]), asks
// the TMA engine to prefetch the rest of its share into L2, and stages the B rows of its output rows.  HBM
// therefore streams the next layer's weights while this layer exchanges partial tiles and stores y, and once
// the call ahead has completed (griddepcontrol.wait) the CTA only adds the x tiles and runs from L2.
//
// Work split (no clusters, no co-residency requirement beyond "lower block indices are placed first"):
//   - aux CTAs (the lowest block indices): one 128-row tile of the stacked matrix [A_0..A_{N-1}; Wg] times one
//     slice of the contraction axis each; the fp32 partial tile goes to scratch as one bulk copy; after a counter
//     barrier among the aux CTAs a warp per token adds the slices in order, selects the top-k, applies the
//     softmax over the picks (Eq. 3) and publishes topk_idx, topk_w, uw = w_j * (A_{i_j} x).
//   - main CTAs: row tile i of W0 belongs to S CTAs, CTA j of them multiplies k-steps [K j / S, K (j+1) / S) and
//     writes its fp32 accumulator to scratch cut into S row slices (its own slice stays in shared memory); when all
//     S have delivered, CTA j fetches row slice j of the other partials (one bulk copy each, contiguous by
//     construction) into the idle ring.  While those are on their way the epilogue threads compute the LoRA expand
//     of the slice from the staged B rows and the routing (fetched the same way by the idle producer thread);
//     then partials in CTA order + expand, one rounding to bf16, store.  The epilogue threads never poll a
//     counter: warp 0 waits for the routing, warp 1 for the tile.
// Every wait is bounded; on expiry the status word is set and the CTA drains.  The workspace counters are
// re-armed by the last CTA to stop reading them.
#pragma once

namespace meteora {

struct StreamParams {
    int T, BN, ksteps;
    int stages, kc;            // main ring: stages of kc k-steps, [kc W tiles][kc x tiles]
    int aux_stages;            // aux ring: one k-step per stage
    int tmem_cols;
    int N, r, k, d_out;
    int row_tiles, S, n_main;  // S main CTAs per 128-row tile of W0
    int n_aux, aux_tiles, aux_slices, a_tiles, gate_tile, gate_row0;
    int pf_main, pf_aux;       // stages beyond the ring whose weights are prefetched into L2 before the wait
    int slab_off;              // byte offset of the staged B rows behind the barriers
    int ring_bytes;            // ring of both kinds of CTA; later the landing area of the last step
    int bar_slots;             // ring slots the barrier area is laid out for
    float inv_tau;
    const __nv_bfloat16* B;
    __nv_bfloat16* y;
    int32_t* topk_idx;
    float* topk_w;
    float* uw;
    float* u_part;             // [aux_slices][aux_tiles][T][128] partial stacked shrink
    float* part_g;             // [row tile * S + j][BN * 128] partial accumulator tiles, cut into S row slices
    int32_t* ctr;              // [0] aux partials in, [1] routing published, [2] CTAs counted out
    int32_t* tile_ctr;         // [row tiles] partials delivered
    int32_t* status;
    int bulk_deliver;          // the other CTAs' row slices leave through shared memory and bulk copies instead of plain stores
    int aux_plain;             // the aux CTAs' partial tiles leave as plain stores instead of one bulk copy
    int own_local;             // the CTA's own row slice of its accumulator stays in shared memory (else through scratch like the others)
    int pdl;
    int trace_call;
};

__device__ __forceinline__ void mbar_expect_tx_only(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_prefetch_l2_3d(const CUtensorMap* tm, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"((uint64_t)tm), "r"(c0),
                 "r"(c1), "r"(c2)
                 : "memory");
}
// One contiguous block from global to shared memory by the TMA engine; completion is counted on `bar`.
__device__ __forceinline__ void bulk_load_block(uint32_t smem_dst, const void* gsrc, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_dst),
                 "l"(gsrc), "r"(bytes), "r"(bar)
                 : "memory");
}

// TMEM -> registers, 16 columns of this warp's 32 lanes, WITHOUT waiting: several of these go out back to back and
// one tmem_ld_wait() covers them all (a load and its wait take about half a microsecond; four in a row, each
// waited for, cost the epilogue 2 us at 128 tokens).
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// The accumulator columns [c_begin, c_end) of this warp's 32 rows (whole chunks of 16 columns, at most 64 per round) to
// column * pitch floats behind a shared-memory address or a global pointer; `valid` false stores zeros (a wait gave
// up).  No store is predicated: columns beyond the last token hold zeros (the token tile's rows past T are zero-filled)
// and every destination is sized for the padded token count.  (Bounds checked per store, or stores through a
// pointer that may be shared or global, made this loop five times slower: 2.4 us for 64 columns.)
__device__ __forceinline__ void tmem_rows_out(uint32_t taddr, int c_begin, int c_end, bool valid, float* dst,
                                              uint32_t dst_shared, bool to_shared, int pitch,
                                              unsigned long long* t_ld = nullptr) {
    for (int c0 = c_begin; c0 < c_end; c0 += 64) {
        uint32_t r[4][16];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (valid && c0 + 16 * q < c_end) {                          // warp-uniform
                tmem_ld16_issue(taddr + (uint32_t)(c0 + 16 * q), r[q]);
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) r[q][i] = 0u;
            }
        }
        tmem_ld_wait();
        if (t_ld) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(*t_ld));
        const int nchunks = min(4, (c_end - c0) / 16);
        if (to_shared) {
            const uint32_t a0 = dst_shared + (uint32_t)(c0 * pitch * 4);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (q < nchunks) {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        asm volatile("st.shared.b32 [%0], %1;" ::"r"(a0 + (uint32_t)((16 * q + i) * pitch * 4)), "r"(r[q][i])
                                     : "memory");
                }
            }
        } else {
            float* g0 = dst + (size_t)c0 * pitch;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (q < nchunks) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) g0[(size_t)(16 * q + i) * pitch] = __uint_as_float(r[q][i]);
                }
            }
        }
    }
}

// 3-D tile load of a CTA pair: the completion bytes go to a barrier that may live in the pair's other CTA.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2,
                                                 uint32_t cluster_bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"((uint64_t)tm), "r"(c0), "r"(c1), "r"(c2), "r"(cluster_bar)
        : "memory");
}

// Bounded wait until *ctr >= target with a longer pause between looks than wait_counter: over a hundred CTAs watch
// the same cache line that others add to, and every look is a request to that line.
__device__ __forceinline__ bool wait_counter_slow(const int32_t* ctr, int target, unsigned pause_ns) {
    const long long t0 = clock64(), limit = g_wait_limit_cycles;
    while (ld_acquire(ctr) < target) {
        if (clock64() - t0 > limit) return false;
        __nanosleep(pause_ns);
    }
    return true;
}

__device__ __forceinline__ void stream_flag_error(const StreamParams& d, int word, int code) {
    atomicExch(d.status, 1);
    atomicExch(d.status + word, code);
}

// Counts this CTA out (one thread, after its last look at a workspace counter); the last one re-arms them.
__device__ __forceinline__ void stream_count_out(const StreamParams& d) {
    if (atomicAdd(d.ctr + 2, 1) == (int)gridDim.x - 1) {
        d.ctr[0] = 0;
        d.ctr[1] = 0;
        for (int i = 0; i < d.row_tiles; ++i) d.tile_ctr[i] = 0;
        d.ctr[2] = 0;
    }
}

#ifdef METEORA_TRACE
#define STREAM_STAMP(slot)                                                                                        \
    do {                                                                                                          \
        unsigned long long t_;                                                                                    \
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                                                    \
        if (blockIdx.x < kTraceCtas)                                                                              \
            g_fused_trace[((d.trace_call % kTraceCalls) * kTraceCtas + blockIdx.x) * kTraceSlots + (slot)] = t_;  \
    } while (0)
#else
#define STREAM_STAMP(slot) do { } while (0)
#endif

// Selection for one token from its summed row of the stacked shrink in shared memory (row[R] for stacked row R of
// [A_0 .. A_{N-1}], logit n at row[gate_tile * 128 + gate_row0 + n]): top-k, softmax over the picks (Eq. 3), uw.
__device__ __forceinline__ void select_token_row(const float* row, int gate_tile, int gate_row0, int t, int N, int r, int k,
                                                 float inv_tau, int lane, int32_t* topk_idx, float* topk_w, float* uw) {
    float v[kSelVals];
#pragma unroll
    for (int i = 0; i < kSelVals; ++i)
        v[i] = lane + 32 * i < N ? row[gate_tile * kBM + gate_row0 + lane + 32 * i] : 0.f;
    int idx;
    float w;
    warp_topk_softmax(v, N, k, inv_tau, lane, idx, w);
    if (lane < k) {
        topk_idx[(size_t)t * k + lane] = idx;
        topk_w[(size_t)t * k + lane] = w;
    }
    for (int c0 = 0; c0 < k * r; c0 += 32) {
        const int c = min(c0 + lane, k * r - 1);
        const int j = c / r, q = c - j * r;
        const int ij = __shfl_sync(0xFFFFFFFFu, idx, j);
        const float wj = __shfl_sync(0xFFFFFFFFu, w, j);
        if (c0 + lane < k * r) uw[(size_t)t * k * r + c0 + lane] = wj * row[ij * r + q];
    }
}

// Row slice of contributor j of S: groups of 4 rows [32 j / S, 32 (j + 1) / S).
__device__ __forceinline__ void row_slice(int j, int S, int& q0, int& nq) {
    q0 = 32 * j / S;
    nq = 32 * (j + 1) / S - q0;
}

// kPair: the grid runs in clusters of two CTAs and a pair of main CTAs multiplies TWO row tiles of W0 (one each) with
// the same slice of the contraction axis by tcgen05.mma.cta_group::2: each CTA loads its own 128 rows of W0 but only
// HALF of the token tile, and the tensor cores of both SMs read both halves.  At 128 tokens the token tile is as large
// as the W0 tile, so this takes a quarter off what an SM takes in and lets the ring hold four stages instead of three.
// No load is multicast; every copy of the pair signals the leader's barrier, which expects both CTAs' bytes; the
// leader alone issues MMAs and releases stages by commits that arrive in both CTAs.  Aux CTAs work alone as before.
template <bool kPair>
__global__ void __launch_bounds__(kThreads, 2)
k_decode_stream(const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmA,
                const __grid_constant__ CUtensorMap tmAt, const __grid_constant__ CUtensorMap tmG,
                const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmX1,
                const StreamParams d) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;
    uint8_t* ring_ptr = smem_raw + (ring - raw);
    const uint32_t aux_x_bytes = d.BN * 128;                                  // an aux CTA takes the whole token tile
    const uint32_t x_tile_bytes = kPair ? d.BN * 64 : d.BN * 128;             // a main CTA of a pair half of it
    const uint32_t stage_bytes = d.kc * (kWTileBytes + x_tile_bytes);
    const uint32_t aux_stage_bytes = kWTileBytes + aux_x_bytes;
    const uint32_t ring_bytes = (uint32_t)d.ring_bytes;
    const uint32_t bar_base = ring + ring_bytes;              // full[slots], empty[slots], acc, land, route, deliv
    const uint32_t bar_acc = bar_base + 2 * d.bar_slots * 8;
    const uint32_t bar_land = bar_acc + 8;
    const uint32_t bar_route = bar_acc + 16;
    const uint32_t bar_deliv = bar_acc + 24;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ring_ptr + ring_bytes + (2 * d.bar_slots + 4) * 8);
    uint8_t* slab_ptr = ring_ptr + ring_bytes + d.slab_off;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool is_aux = (int)blockIdx.x < d.n_aux;
    const int n_active = d.aux_tiles * d.aux_slices;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2 * d.bar_slots + 4; ++s) mbar_init(bar_base + s * 8, 1);
        tmem_slot[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        if (kPair && !is_aux) {                                               // the pair-wide form, by both CTAs
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                         "r"((uint32_t)d.tmem_cols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                         "r"((uint32_t)d.tmem_cols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    if (kPair) {
        __syncwarp();
        cluster_sync();                                                       // both CTAs' barriers exist before anyone signals
    } else {
        __syncthreads();
    }
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_slot);
    // The next launch on the stream may become resident from here on (it only touches weights until this
    // kernel has completed).
    if (d.pdl && threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) STREAM_STAMP(0);

    const uint32_t idesc = instr_desc_bf16(d.BN);
    const int quad = warp & 3;
    const int etid = threadIdx.x - 64;
    const int ntok = min(d.BN, d.T);
    const int half = ((d.BN / 16 + 1) / 2) * 16;
    const int c_begin = warp < 6 ? 0 : half, c_end = warp < 6 ? half : d.BN;

    if (is_aux) {
        // ================================================================== aux CTA
        const int aux_id = blockIdx.x;
        const bool active = aux_id < n_active;
        const int tile = aux_id % d.aux_tiles, slice = aux_id / d.aux_tiles;
        const int ks0 = active ? (d.ksteps * slice) / d.aux_slices : 0;
        const int ks1 = active ? (d.ksteps * (slice + 1)) / d.aux_slices : 0;
        const int niter = ks1 - ks0;
        if (warp == 0) {
            if (lane == 0 && active) {
                // A's last tile has its own map (its box stops at A's last row when Wg follows in the same tile)
                const CUtensorMap* mA = tile >= d.a_tiles ? nullptr : tile == d.a_tiles - 1 ? &tmAt : &tmA;
                const CUtensorMap* mG = tile == d.gate_tile ? &tmG : nullptr;
                const uint32_t g_off = (uint32_t)d.gate_row0 * 128u;
                const int pre = min(niter, d.aux_stages);
                // weights first: they do not depend on the kernel ahead
                for (int i = 0; i < pre; ++i) {
                    const uint32_t full = bar_base + i * 8, dst = ring + i * aux_stage_bytes;
                    mbar_expect_tx_only(full, kWTileBytes);
                    if (mA) tma_load_3d(dst, mA, 0, tile * kBM, ks0 + i, full);
                    if (mG) tma_load_3d(dst + g_off, mG, 0, 0, ks0 + i, full);
                }
                for (int i = pre; i < min(niter, pre + d.pf_aux); ++i) {
                    if (mA) tma_prefetch_l2_3d(mA, 0, tile * kBM, ks0 + i);
                    if (mG) tma_prefetch_l2_3d(mG, 0, 0, ks0 + i);
                }
                if (d.pdl) asm volatile("griddepcontrol.wait;" ::: "memory");
                STREAM_STAMP(1);
                for (int i = 0; i < pre; ++i) {
                    const uint32_t full = bar_base + i * 8, dst = ring + i * aux_stage_bytes;
                    mbar_expect_tx(full, aux_x_bytes);
                    tma_load_3d(dst + kWTileBytes, &tmX1, 0, 0, ks0 + i, full);
                }
                bool ok = true;
                for (int i = pre; i < niter; ++i) {
                    const int s = i % d.aux_stages, round = i / d.aux_stages;
                    ok = mbar_wait(bar_base + (d.bar_slots + s) * 8, (round & 1) ^ 1);
                    if (!ok) break;
                    const uint32_t full = bar_base + s * 8, dst = ring + s * aux_stage_bytes;
                    mbar_expect_tx(full, aux_stage_bytes);
                    if (mA) tma_load_3d(dst, mA, 0, tile * kBM, ks0 + i, full);
                    if (mG) tma_load_3d(dst + g_off, mG, 0, 0, ks0 + i, full);
                    tma_load_3d(dst + kWTileBytes, &tmX1, 0, 0, ks0 + i, full);
                }
                if (!ok) stream_flag_error(d, 1, 400);
            }
        } else if (warp == 1) {
            if (lane == 0 && active) {
                bool ok = true;
                for (int i = 0; i < niter; ++i) {
                    const int s = i % d.aux_stages, round = i / d.aux_stages;
                    ok = mbar_wait(bar_base + s * 8, round & 1);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t wa = ring + s * aux_stage_bytes, xa = wa + kWTileBytes;
                    const uint64_t da = smem_desc_sw128(wa), db = smem_desc_sw128(xa);
#pragma unroll
                    for (int kk = 0; kk < kBK / kUmmaK; ++kk)
                        umma_bf16(tmem_base, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (i | kk) != 0);
                    umma_commit(bar_base + (d.bar_slots + s) * 8);
                }
                umma_commit(bar_acc);
                if (!ok) stream_flag_error(d, 2, 500);
                STREAM_STAMP(2);
            }
        } else if (active) {
            bool acc_ok = mbar_wait(bar_acc, 0);
            if (!acc_ok && lane == 0) stream_flag_error(d, 3, 600);
            acc_ok = __all_sync(0xFFFFFFFFu, acc_ok);
            tc_fence_after();
            // the accumulator tile as it is, [token][128 rows] fp32
            const int trow = quad * 32 + lane;
            if (d.aux_plain) {
                // straight from registers: lane = row, a warp writes 128 contiguous bytes per token (the scratch holds
                // BN token rows per tile, so nothing is predicated)
                if (d.pdl) asm volatile("griddepcontrol.wait;" ::: "memory");
                float* dst = d.u_part + (((size_t)slice * d.aux_tiles + tile) * d.T) * kBM + trow;
                for (int c0 = c_begin; c0 < c_end; c0 += 16) {
                    float v[16];
                    if (acc_ok && niter > 0) {
                        tmem_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)c0, v);
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = 0.f;
                    }
                    if (c0 + 16 <= d.T) {                                      // warp-uniform: whole chunks unpredicated
#pragma unroll
                        for (int i = 0; i < 16; ++i) dst[(size_t)(c0 + i) * kBM] = v[i];
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (c0 + i < d.T) dst[(size_t)(c0 + i) * kBM] = v[i];
                    }
                }
            } else {
                // through the idle ring and one bulk copy (all BN columns are written: the copy moves T of them)
                tmem_rows_out(tmem_base + ((uint32_t)(quad * 32) << 16), c_begin, c_end, acc_ok && niter > 0, nullptr,
                              ring + (uint32_t)trow * 4u, true, kBM);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
        }
        __syncwarp();
        __syncthreads();
        if (active) {
            if (d.pdl) asm volatile("griddepcontrol.wait;" ::: "memory");     // every thread below touches the scratch
            if (threadIdx.x == 0) {
                float* dst = d.u_part + (((size_t)slice * d.aux_tiles + tile) * d.T) * kBM;
                if (!d.aux_plain) bulk_store_block(dst, ring, (uint32_t)d.T * kBM * 4u);
                __threadfence();
                atomicAdd(d.ctr + 0, 1);
                STREAM_STAMP(3);
                if (!wait_counter(d.ctr + 0, n_active)) stream_flag_error(d, 4, 700);
                STREAM_STAMP(4);
            }
            // This CTA's share of the tokens: their rows of every partial tile into the idle ring (one bulk copy per
            // tile and slice, a token range is contiguous there), then a warp per token selects from shared memory.
            const int t0 = d.T * aux_id / n_active, t1 = d.T * (aux_id + 1) / n_active, ntl = t1 - t0;
            const uint32_t rows_bytes = (uint32_t)(n_active * ntl * kBM * 4);
            __syncthreads();                                         // thread 0 has seen all partials; its staged tile has left the ring
            if (ntl > 0) {
                // one copy per (slice, tile), each issued by a thread of its own (twenty issued by one thread took over a microsecond)
                if (threadIdx.x == 0) mbar_expect_tx(bar_land, rows_bytes);
                if ((int)threadIdx.x < n_active)
                    bulk_load_block(ring + (uint32_t)((int)threadIdx.x * ntl * kBM * 4),
                                    d.u_part + ((size_t)threadIdx.x * d.T + t0) * kBM, (uint32_t)(ntl * kBM * 4), bar_land);
                bool ok = mbar_wait(bar_land, 0);
                if (!ok && lane == 0) stream_flag_error(d, 4, 750);
                ok = __all_sync(0xFFFFFFFFu, ok);                   // the selection is warp-collective
                if (threadIdx.x == 0) STREAM_STAMP(6);
                // All threads add the slices of the CTA's tokens' rows, four columns per item, every slice of an item in
                // flight together, in slice order (the same sums in the same order as select_token_narrow: same bits); a
                // warp per token then selects from the summed row.  (One warp doing both for its token took 1.7 us.)
                const float4* sm4 = reinterpret_cast<const float4*>(ring_ptr);
                float4* rows4 = reinterpret_cast<float4*>(ring_ptr + rows_bytes);      // [ntl][tiles * 128] floats
                const int per_tok = d.aux_tiles * 32, zs4 = d.aux_tiles * ntl * 32;
                for (int it = threadIdx.x; it < ntl * per_tok && ok; it += kThreads) {
                    const int tl = it / per_tok, rem = it - tl * per_tok, tile = rem >> 5, l4 = rem & 31;
                    const float4* src = sm4 + (tile * ntl + tl) * 32 + l4;
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
                    for (int z = 0; z < d.aux_slices; ++z) {
                        const float4 v = src[z * zs4];
                        acc.x += v.x;
                        acc.y += v.y;
                        acc.z += v.z;
                        acc.w += v.w;
                    }
                    rows4[it] = acc;
                }
                if (threadIdx.x == 0) STREAM_STAMP(10);
                __syncthreads();
                if (threadIdx.x == 0) STREAM_STAMP(11);
                const int nwarps = kThreads / 32;
                for (int tl = warp; tl < ntl && ok; tl += nwarps)
                    select_token_row(reinterpret_cast<const float*>(rows4 + tl * per_tok), d.gate_tile, d.gate_row0, t0 + tl, d.N,
                                     d.r, d.k, d.inv_tau, lane, d.topk_idx, d.topk_w, d.uw);
                if (threadIdx.x == 0) STREAM_STAMP(7);
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                STREAM_STAMP(8);
                __threadfence();
                STREAM_STAMP(9);
                atomicAdd(d.ctr + 1, 1);
                STREAM_STAMP(5);
            }
        }
        if (threadIdx.x == 0) {
            if (d.pdl) asm volatile("griddepcontrol.wait;" ::: "memory");
            stream_count_out(d);
        }
    } else {
        // ================================================================== main CTA
        const int main_id = (int)blockIdx.x - d.n_aux;
        const int S = d.S;
        // alone: CTA = (tile, slice j); in pairs: pair = (two adjacent tiles, slice j), the CTA's rank picks the tile
        const uint32_t rank = kPair ? cluster_rank() : 0u;
        const bool leader = rank == 0;
        const int tile = kPair ? 2 * ((main_id >> 1) / S) + (int)rank : main_id / S;
        const int j = kPair ? (main_id >> 1) % S : main_id - tile * S;
        const bool live = tile < d.row_tiles;                       // an odd tile count leaves the last pair's second CTA without rows
        const int slot_id = tile * S + j;                            // this CTA's partial tile in the scratch
        const int nst = d.ksteps / d.kc;                             // stages of the whole contraction axis
        const int it0 = nst * j / S, it1 = nst * (j + 1) / S;
        const int n_it = it1 - it0;
        const int row0 = tile * kBM;
        int q0, nq;
        row_slice(j, S, q0, nq);
        const int cpa = d.r >> 3;
        uint4* slab = reinterpret_cast<uint4*>(slab_ptr);
        // Landing area in the idle ring: block c = row slice j of partial c ([token][4 nq rows] fp32; block j is
        // written by this CTA's own threads), then one block for the LoRA expand of the slice, then the routing.
        // (blocks hold the padded token count BN: the accumulator leaves in whole chunks of 16 token columns)
        const uint32_t blk_bytes = (uint32_t)(d.BN * 4 * nq * 4);
        const uint32_t delta_off = S * blk_bytes;
        const uint32_t idx_bytes = ((uint32_t)(ntok * d.k * 4) + 15u) & ~15u;
        const uint32_t uw_bytes = (uint32_t)(ntok * d.k * d.r * 4);
        const uint32_t idx_off = delta_off + blk_bytes, uw_off = idx_off + ((idx_bytes + 127u) & ~127u);
        int* s_done = reinterpret_cast<int*>(tmem_slot) + 1;          // warps 0 and 1: who is last counts the CTA out
        if (warp == 0) {
            if (lane == 0) {
                const uint32_t w_bytes = d.kc * kWTileBytes, xs_bytes = d.kc * x_tile_bytes;
                const uint32_t both = kPair ? 2u : 1u;               // the leader's barrier expects both CTAs' bytes
                const int tok0 = kPair ? (int)rank * (d.BN / 2) : 0;  // own half of the token tile
                const int pre = min(n_it, d.stages);
                auto full_bar = [&](int s_) {                        // where this CTA's copies report: the leader's barrier
                    const uint32_t local = bar_base + s_ * 8;
                    return kPair ? map_to_cta(local, 0) : local;
                };
                auto load_w = [&](uint32_t dst, int it, uint32_t bar) {
                    if (kPair) tma_load_3d_pair(dst, &tmW0, 0, row0, it * d.kc, bar);
                    else tma_load_3d(dst, &tmW0, 0, row0, it * d.kc, bar);
                };
                auto load_x = [&](uint32_t dst, int it, uint32_t bar) {
                    if (kPair) tma_load_3d_pair(dst, &tmX, 0, tok0, it * d.kc, bar);
                    else tma_load_3d(dst, &tmX, 0, tok0, it * d.kc, bar);
                };
                for (int i = 0; i < pre; ++i) {
                    if (leader) mbar_expect_tx_only(bar_base + i * 8, both * w_bytes);
                    load_w(ring + i * stage_bytes, it0 + i, full_bar(i));
                }
                for (int i = pre; i < min(n_it, pre + d.pf_main); ++i) tma_prefetch_l2_3d(&tmW0, 0, row0, (it0 + i) * d.kc);
                if (d.pdl) asm volatile("griddepcontrol.wait;" ::: "memory");
                STREAM_STAMP(1);
                for (int i = 0; i < pre; ++i) {
                    if (leader) mbar_expect_tx(bar_base + i * 8, both * xs_bytes);
                    load_x(ring + i * stage_bytes + w_bytes, it0 + i, full_bar(i));
                }
                bool ok = true;
                int st = pre == d.stages ? 0 : pre, round = pre == d.stages ? 1 : 0;
                for (int i = pre; i < n_it; ++i) {
                    ok = mbar_wait(bar_base + (d.bar_slots + st) * 8, (round & 1) ^ 1);
                    if (!ok) break;
                    const uint32_t dst = ring + st * stage_bytes;
                    if (leader) mbar_expect_tx(bar_base + st * 8, both * stage_bytes);
                    load_w(dst, it0 + i, full_bar(st));
                    load_x(dst + w_bytes, it0 + i, full_bar(st));
                    if (++st == d.stages) {
                        st = 0;
                        ++round;
                    }
                }
                if (!ok) stream_flag_error(d, 1, 100);
                STREAM_STAMP(2);
                // The routing into the landing area, as soon as the ring is idle and the aux CTAs have published it.
                ok = mbar_wait(bar_acc, 0);
                if (ok) ok = wait_counter_slow(d.ctr + 1, n_active, 200);
                if (!ok) stream_flag_error(d, 4, 800);
                STREAM_STAMP(7);
                mbar_expect_tx(bar_route, idx_bytes + uw_bytes);
                bulk_load_block(ring + idx_off, d.topk_idx, idx_bytes, bar_route);
                bulk_load_block(ring + uw_off, d.uw, uw_bytes, bar_route);
                if (atomicAdd_block(s_done, 1) == 1) stream_count_out(d);   // the CTA reads no workspace counter any more
                mbar_wait(bar_route, 0);    // own copies have landed before the CTA may leave (the epilogue may have given up)
            }
        } else if (warp == 1) {
            if (lane == 0) {
                bool ok = true;
                if (leader) {                                        // of a pair, the leader alone issues the MMAs
                    const uint32_t idesc_main =
                        kPair ? (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(d.BN >> 3) << 17) | ((uint32_t)(256 >> 4) << 24)
                              : idesc;
                    int st = 0, round = 0;
                    for (int i = 0; i < n_it; ++i) {
                        ok = mbar_wait(bar_base + st * 8, round & 1);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t wa = ring + st * stage_bytes, xa = wa + d.kc * kWTileBytes;
                        for (int c = 0; c < d.kc; ++c) {
                            const uint64_t da = smem_desc_sw128(wa + c * kWTileBytes);
                            const uint64_t db = smem_desc_sw128(xa + c * x_tile_bytes);
#pragma unroll
                            for (int kk = 0; kk < kBK / kUmmaK; ++kk) {
                                if (kPair)
                                    umma_bf16_pair(tmem_base, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc_main,
                                                   (i | c | kk) != 0);
                                else
                                    umma_bf16(tmem_base, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc_main,
                                              (i | c | kk) != 0);
                            }
                        }
                        if (kPair) umma_commit_pair(bar_base + (d.bar_slots + st) * 8);   // both rings may refill the stage
                        else umma_commit(bar_base + (d.bar_slots + st) * 8);
                        if (++st == d.stages) {
                            st = 0;
                            ++round;
                        }
                    }
                    if (kPair) umma_commit_pair(bar_acc);            // accumulators complete in both CTAs
                    else umma_commit(bar_acc);
                    if (!ok) stream_flag_error(d, 2, 200);
                }
                STREAM_STAMP(3);
                // The other CTAs' partials of this CTA's row slice into the landing area, once the ring is idle and
                // all S CTAs of the tile have delivered (this CTA's own delivery included).
                ok = mbar_wait(bar_deliv, 0);                      // not before this CTA's own partial is out
                if (d.pdl) asm volatile("griddepcontrol.wait;" ::: "memory");
                if (ok && S > 1 && live) ok = wait_counter_slow(d.tile_ctr + tile, S, 100);
                if (!ok) stream_flag_error(d, 4, 900);
                STREAM_STAMP(6);
                const uint32_t one = blk_bytes;
                mbar_expect_tx(bar_land, live ? (uint32_t)(d.own_local ? S - 1 : S) * one : 0u);
                for (int c = 0; c < S && live; ++c)
                    if (c != j || !d.own_local)
                        bulk_load_block(ring + c * blk_bytes,
                                        d.part_g + (size_t)(tile * S + c) * ((size_t)d.BN * kBM) + (size_t)d.BN * 4 * q0, one,
                                        bar_land);
                if (atomicAdd_block(s_done, 1) == 1) stream_count_out(d);
                mbar_wait(bar_land, 0);     // own copies have landed before the CTA may leave
            }
        } else {
            // B rows of this CTA's row slice for every adapter: weights, staged before the wait
            if (live) stage_slab_rows(d.B, d.d_out, d.N, cpa, slab, row0 + 4 * q0, 4 * nq, etid);
            // Where this thread's accumulator row goes (worked out before the accumulator is ready): the accumulator
            // is cut into the S row slices, each stored [token][rows of the slice] so that the CTA that finishes a
            // slice fetches it as one contiguous block: the own slice straight into the landing area, the others to scratch.
            const int row_in_tile = quad * 32 + lane;
            float* land = reinterpret_cast<float*>(ring_ptr);          // the ring is idle once the accumulator is complete
            int sj = 0, sq0 = 0, snq = 32;                             // the slice this thread's row belongs to
            for (int c = 0; c < S; ++c) {
                int a, b;
                row_slice(c, S, a, b);
                if (row_in_tile / 4 >= a) {
                    sj = c;
                    sq0 = a;
                    snq = b;
                }
            }
            // (bulk_deliver: the slices for the other CTAs are staged where their counterparts will land later, block c of
            // the landing area, and leave as one bulk copy each; the host takes this only where all slices have equal size)
            const bool part_shared = (sj == j && d.own_local) || d.bulk_deliver;
            const uint32_t part_s = ring + (uint32_t)sj * blk_bytes + (uint32_t)(row_in_tile - 4 * sq0) * 4u;
            float* part = d.part_g + (size_t)slot_id * ((size_t)d.BN * kBM) + (size_t)d.BN * 4 * sq0 + (row_in_tile - 4 * sq0);
            (void)land;
            if (d.pdl) asm volatile("griddepcontrol.wait;" ::: "memory");
            bool acc_ok = mbar_wait(bar_acc, 0);
            if (!acc_ok && lane == 0) stream_flag_error(d, 3, 300);
            acc_ok = __all_sync(0xFFFFFFFFu, acc_ok);
            tc_fence_after();
            if (etid == 0) STREAM_STAMP(4);
            {
                const int pitch = 4 * snq;
#ifdef METEORA_TRACE
                unsigned long long t_ld = 0;
                if (live)
                    tmem_rows_out(tmem_base + ((uint32_t)(quad * 32) << 16), c_begin, c_end, acc_ok && n_it > 0, part, part_s,
                                  part_shared, pitch, &t_ld);
                if (etid == 0 && blockIdx.x < kTraceCtas)
                    g_fused_trace[((d.trace_call % kTraceCalls) * kTraceCtas + blockIdx.x) * kTraceSlots + 14] = t_ld;
#else
                if (live)
                    tmem_rows_out(tmem_base + ((uint32_t)(quad * 32) << 16), c_begin, c_end, acc_ok && n_it > 0, part, part_s,
                                  part_shared, pitch);
#endif
                if (etid == 0) STREAM_STAMP(11);
                if (d.bulk_deliver) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> bulk copy reads
                epi_barrier();                                         // also orders the own slice for the threads below
                if (etid == 0) {
                    STREAM_STAMP(12);
                    if (d.bulk_deliver && S > 1 && live) {
                        const uint32_t one = blk_bytes;
                        for (int c = 0; c < S; ++c)
                            if (c != j) {
                                int a, b;
                                row_slice(c, S, a, b);
                                float* dst = d.part_g + (size_t)slot_id * ((size_t)d.BN * kBM) + (size_t)d.BN * 4 * a;
                                asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst),
                                             "r"(ring + c * blk_bytes), "r"(one)
                                             : "memory");
                            }
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
                    }
                    if (S > 1 && live) {
                        __threadfence();
                        STREAM_STAMP(13);
                        atomicAdd(d.tile_ctr + tile, 1);
                    }
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_deliv) : "memory");
                    STREAM_STAMP(5);
                }
            }
            // LoRA expand of the slice (Eq. 2) while the partials are on their way: routing and B rows are here.
            bool ok = mbar_wait(bar_route, 0);
            if (etid == 0) STREAM_STAMP(15);
            if (!ok && lane == 0) stream_flag_error(d, 4, 850);
            const int* s_idx = reinterpret_cast<const int*>(ring_ptr + idx_off);
            const float4* s_uw4 = reinterpret_cast<const float4*>(ring_ptr + uw_off);
            float4* dblk = reinterpret_cast<float4*>(ring_ptr + delta_off);
            const int items = live ? nq * ntok : 0, slab_rows = 4 * nq;
            for (int it = etid; it < items && ok; it += kEpiThreads) {
                const int t = it / nq, ql = it - t * nq;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int jj = 0; jj < d.k; ++jj) {
                    const int slot = t * d.k + jj;
                    const int e = min(max(s_idx[slot], 0), d.N - 1);
                    for (int ch = 0; ch < cpa; ++ch) {               // 8 rank entries at a time
                        const float4 u0 = s_uw4[2 * (slot * cpa + ch)], u1 = s_uw4[2 * (slot * cpa + ch) + 1];
                        const uint4* b = slab + (size_t)(e * cpa + ch) * slab_rows + ql;
                        fma8(b[0], u0, u1, acc.x);
                        fma8(b[nq], u0, u1, acc.y);
                        fma8(b[2 * nq], u0, u1, acc.z);
                        fma8(b[3 * nq], u0, u1, acc.w);
                    }
                }
                dblk[it] = acc;                                      // read back by the same thread below
            }
            if (etid == 0) STREAM_STAMP(8);
            if (S > 1 && live) ok = mbar_wait(bar_land, 0) && ok;
            if (!ok && lane == 0) stream_flag_error(d, 4, 950);
            if (etid == 0) STREAM_STAMP(9);
            const int blk4 = (int)(blk_bytes / 16);
            for (int it = etid; it < items && ok; it += kEpiThreads) {
                const int t = it / nq, ql = it - t * nq;
                const float4* p4 = reinterpret_cast<const float4*>(land) + it;
                float4 acc = p4[0];
                for (int c = 1; c < S; ++c) {                        // partials in CTA order: the same sum every run
                    const float4 v = p4[c * blk4];
                    acc.x += v.x;
                    acc.y += v.y;
                    acc.z += v.z;
                    acc.w += v.w;
                }
                const float4 dl = dblk[it];
                acc.x += dl.x;
                acc.y += dl.y;
                acc.z += dl.z;
                acc.w += dl.w;
                const int o = row0 + (q0 + ql) * 4;
                __nv_bfloat16* dst = d.y + (size_t)t * d.d_out + o;
                if ((d.d_out & 3) == 0 && o + 3 < d.d_out) {
                    const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
                    uint2 pk;
                    pk.x = *reinterpret_cast<const uint32_t*>(&lo);
                    pk.y = *reinterpret_cast<const uint32_t*>(&hi);
                    *reinterpret_cast<uint2*>(dst) = pk;
                } else {
                    const float f[4] = {acc.x, acc.y, acc.z, acc.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (o + i < d.d_out) dst[i] = __float2bfloat16_rn(f[i]);
                }
            }
            if (etid == 0) STREAM_STAMP(10);
        }
    }

    tc_fence_before();
    if (kPair) {
        __syncwarp();
        cluster_sync();                     // nobody leaves while the pair's other CTA may still signal it
    } else {
        __syncthreads();
    }
    if (warp == 1) {
        if (kPair && !is_aux)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)d.tmem_cols)
                         : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)d.tmem_cols)
                         : "memory");
    }
}

}  // namespace meteora
