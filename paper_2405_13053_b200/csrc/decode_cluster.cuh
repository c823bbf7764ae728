// Whole MeteoRA linear forward (Eq. 2 with Eq. 3) for a decode batch of up to 128 tokens as ONE kernel launch of
// thread-block CLUSTERS: the S CTAs that share a 128-row tile of W0 (each multiplies one slice of the contraction
// axis) form a cluster and add their partial tiles through distributed shared memory instead of through L2, and
// there are no CTAs set aside for the stacked shrink: every CTA multiplies a few k-steps of one tile of
// [A_0 .. A_{N-1}; Wg] FIRST, so that the routing is known before the stream of W0 ends.
// Included by wgemm_tcgen05.cu after decode_stream.cuh, whose device helpers it shares.
//
// A CTA (row tile i = its cluster, slice j = its rank) runs two products through the same TMA ring:
//   1. stacked: tile a = i mod (tiles of the stacked matrix), the k-steps k0 + c, k0 + c + SL, .. of its own slice
//      [k0, k1) where c = i div (tiles) is the cluster's place among the SL clusters that share tile a; into a second
//      TMEM accumulator.  The S partial tiles of a cluster are reduce-scattered by row slices through distributed
//      shared memory (each CTA stores slice s of its accumulator straight into CTA s's receive blocks, then arrives
//      on CTA s's barrier); CTA j adds the S blocks of its slice and writes [token][rows of the slice] of the
//      cluster's partial to scratch (u_part[c][a]), fence, counter.  When all partials are in, every CTA selects for
//      its share of the tokens (fetch of the tokens' rows of all partials by bulk copies, slices added in order,
//      top-k, softmax over the picks, uw = w_j * A_{i_j} x) and publishes; when all tokens are published every CTA
//      fetches the routing and computes the LoRA expand of its row slice from the B rows it staged at the start.
//   2. main: W0 rows of tile i times k-steps [k0, k1); the accumulator is reduce-scattered the same way (same
//      receive blocks: every peer has told this CTA that it is done reading them), and CTA j adds the S blocks and
//      the expand, rounds once to bf16 and stores its row slice of y.
// The epilogue warps run step 1's exchange and the selection while the producer and MMA threads stream W0.
// Every wait is bounded; on expiry the status word is set and the CTA goes on without computing (its arrivals
// still happen, so that no peer waits for it in vain).  All CTAs must be resident at once (they wait for one
// another through scratch counters): the host launches only as many clusters as the device reports it can hold.
#pragma once

namespace meteora {

struct ClusterParams {
    int T, BN, ksteps;
    int stages;
    int tmem_cols, acc2_col;       // the stacked product accumulates at TMEM column acc2_col
    int N, r, k, d_out;
    int row_tiles, S;
    int aux_tiles, a_tiles, gate_tile, gate_row0;
    int SL;                        // clusters (= slices of the contraction axis) per tile of the stacked matrix
    int n_stk;                     // CTAs that deliver a piece of the stacked shrink: SL * aux_tiles * S
    int n_sel;                     // CTAs that select for at least one token
    int ring_bytes, bar_slots;
    int slab_off, recv_off, delta_off, route_off;   // byte offsets behind the ring
    float inv_tau;
    const __nv_bfloat16* B;
    __nv_bfloat16* y;
    int32_t* topk_idx;
    float* topk_w;
    float* uw;
    float* u_part;                 // [SL][aux_tiles][T][128] partial stacked shrink
    int32_t* ctr;                  // [0] stacked pieces in, [1] selections published, [2] CTAs counted out
    int32_t* status;
    int pdl;
    int trace_call;
};

#ifdef METEORA_TRACE
#define CL_STAMP(slot)                                                                                            \
    do {                                                                                                          \
        unsigned long long t_;                                                                                    \
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                                                    \
        if (blockIdx.x < kTraceCtas)                                                                              \
            g_fused_trace[((d.trace_call % kTraceCalls) * kTraceCtas + blockIdx.x) * kTraceSlots + (slot)] = t_;  \
    } while (0)
#else
#define CL_STAMP(slot) do { } while (0)
#endif

__device__ __forceinline__ void cluster_flag_error(const ClusterParams& d, int word, int code) {
    atomicExch(d.status, 1);
    atomicExch(d.status + word, code);
}

// Accumulator columns [c_begin, c_end) of this warp's 32 rows to column * pitch floats behind an address in the
// CLUSTER's shared memory window (another CTA's receive block, or this CTA's own); unpredicated as tmem_rows_out.
__device__ __forceinline__ void tmem_rows_to_cluster(uint32_t taddr, int c_begin, int c_end, bool valid, uint32_t dst,
                                                     int pitch) {
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
        const int nchunks = min(4, (c_end - c0) / 16);
        const uint32_t a0 = dst + (uint32_t)(c0 * pitch * 4);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (q < nchunks) {
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(a0 + (uint32_t)((16 * q + i) * pitch * 4)),
                                 "r"(r[q][i])
                                 : "memory");
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1)
k_decode_cluster(const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmA,
                 const __grid_constant__ CUtensorMap tmAt, const __grid_constant__ CUtensorMap tmG,
                 const __grid_constant__ CUtensorMap tmX, const ClusterParams d) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;
    uint8_t* ring_ptr = smem_raw + (ring - raw);
    const uint32_t x_tile_bytes = d.BN * 128;
    const uint32_t stage_bytes = kWTileBytes + x_tile_bytes;
    const uint32_t ring_bytes = (uint32_t)d.ring_bytes;
    // barriers behind the ring: full[slots], empty[slots], then the seven below, then the TMEM slot
    const uint32_t bar_base = ring + ring_bytes;
    const uint32_t bar_acc = bar_base + 2 * d.bar_slots * 8;   // main accumulator complete
    const uint32_t bar_acc2 = bar_acc + 8;                     // stacked accumulator complete
    const uint32_t bar_stk = bar_acc + 16;                     // S CTAs have stored their stacked slices here
    const uint32_t bar_mainx = bar_acc + 24;                   // S CTAs have stored their main slices here
    const uint32_t bar_free = bar_acc + 32;                    // the S - 1 peers no longer read their receive blocks
    const uint32_t bar_sel = bar_acc + 40;                     // the tokens' rows of the stacked shrink have landed
    const uint32_t bar_route = bar_acc + 48;                   // the routing has landed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ring_ptr + ring_bytes + (2 * d.bar_slots + 7) * 8);
    uint8_t* tail = ring_ptr + ring_bytes;                     // offsets below count from here
    const uint32_t tail_u32 = ring + ring_bytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = d.S;
    const int j = (int)cluster_rank();
    const int tile = (int)blockIdx.x / S;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2 * d.bar_slots + 2; ++s) mbar_init(bar_base + s * 8, 1);
        mbar_init(bar_stk, (uint32_t)S);
        mbar_init(bar_mainx, (uint32_t)S);
        mbar_init(bar_free, (uint32_t)max(S - 1, 1));
        mbar_init(bar_sel, 1);
        mbar_init(bar_route, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"((uint32_t)d.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncwarp();
    cluster_sync();                                            // every CTA's barriers exist before anyone signals them
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_slot);
    if (d.pdl && threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) CL_STAMP(0);

    const uint32_t idesc = instr_desc_bf16(d.BN);
    const int quad = warp & 3;
    const int etid = threadIdx.x - 64;
    const int ntok = min(d.BN, d.T);
    const int half = ((d.BN / 16 + 1) / 2) * 16;
    const int c_begin = warp < 6 ? 0 : half, c_end = warp < 6 ? half : d.BN;

    // this CTA's slice of the contraction axis, and its k-steps of the stacked product
    const int k0 = d.ksteps * j / S, k1 = d.ksteps * (j + 1) / S;
    const int n_it = k1 - k0;
    const int a_tile = tile % d.aux_tiles, c_slice = tile / d.aux_tiles;
    const bool stk_cluster = c_slice < d.SL;                   // the same for the whole cluster
    const int ns = stk_cluster && c_slice < n_it ? (n_it - c_slice + d.SL - 1) / d.SL : 0;
    const int n_all = ns + n_it;
    const int row0 = tile * kBM;
    int q0, nq;
    row_slice(j, S, q0, nq);
    const int cpa = d.r >> 3;
    const uint32_t blk_bytes = (uint32_t)(d.BN * 4 * nq * 4);  // a receive block: [token][rows of this CTA's slice] fp32

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------------------------ TMA producer
            const CUtensorMap* mA = a_tile >= d.a_tiles ? nullptr : a_tile == d.a_tiles - 1 ? &tmAt : &tmA;
            const CUtensorMap* mG = a_tile == d.gate_tile ? &tmG : nullptr;
            const uint32_t g_off = (uint32_t)d.gate_row0 * 128u;
            auto load_w = [&](uint32_t dst, int i, uint32_t bar) {        // iteration i: stacked first, then W0
                if (i < ns) {
                    const int ks = k0 + c_slice + i * d.SL;
                    if (mA) tma_load_3d(dst, mA, 0, a_tile * kBM, ks, bar);
                    if (mG) tma_load_3d(dst + g_off, mG, 0, 0, ks, bar);
                } else {
                    tma_load_3d(dst, &tmW0, 0, row0, k0 + i - ns, bar);
                }
            };
            auto load_x = [&](uint32_t dst, int i, uint32_t bar) {
                tma_load_3d(dst, &tmX, 0, 0, i < ns ? k0 + c_slice + i * d.SL : k0 + i - ns, bar);
            };
            const int pre = min(n_all, d.stages);
            for (int i = 0; i < pre; ++i) {                               // weights do not depend on the kernel ahead
                mbar_expect_tx_only(bar_base + i * 8, kWTileBytes);
                load_w(ring + i * stage_bytes, i, bar_base + i * 8);
            }
            if (d.pdl) asm volatile("griddepcontrol.wait;" ::: "memory");
            CL_STAMP(1);
            for (int i = 0; i < pre; ++i) {
                mbar_expect_tx(bar_base + i * 8, x_tile_bytes);
                load_x(ring + i * stage_bytes + kWTileBytes, i, bar_base + i * 8);
            }
            bool ok = true;
            int st = pre == d.stages ? 0 : pre, round = pre == d.stages ? 1 : 0;
            for (int i = pre; i < n_all; ++i) {
                ok = mbar_wait(bar_base + (d.bar_slots + st) * 8, (round & 1) ^ 1);
                if (!ok) break;
                const uint32_t dst = ring + st * stage_bytes;
                mbar_expect_tx(bar_base + st * 8, stage_bytes);
                load_w(dst, i, bar_base + st * 8);
                load_x(dst + kWTileBytes, i, bar_base + st * 8);
                if (++st == d.stages) {
                    st = 0;
                    ++round;
                }
            }
            if (!ok) cluster_flag_error(d, 1, 1100);
            CL_STAMP(2);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ------------------------------------------------------------------ MMA issuer
            bool ok = true;
            int st = 0, round = 0;
            for (int i = 0; i < n_all; ++i) {
                ok = mbar_wait(bar_base + st * 8, round & 1);
                if (!ok) break;
                tc_fence_after();
                const uint32_t wa = ring + st * stage_bytes, xa = wa + kWTileBytes;
                const uint64_t da = smem_desc_sw128(wa), db = smem_desc_sw128(xa);
                const uint32_t acc = i < ns ? tmem_base + (uint32_t)d.acc2_col : tmem_base;
                const int first = i < ns ? i : i - ns;
#pragma unroll
                for (int kk = 0; kk < kBK / kUmmaK; ++kk)
                    umma_bf16(acc, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (first | kk) != 0);
                umma_commit(bar_base + (d.bar_slots + st) * 8);
                if (i == ns - 1) umma_commit(bar_acc2);
                if (++st == d.stages) {
                    st = 0;
                    ++round;
                }
            }
            umma_commit(bar_acc);
            if (!ok) cluster_flag_error(d, 2, 1200);
            CL_STAMP(3);
        }
    } else {
        // ---------------------------------------------------------------------- epilogue warps
        uint4* slab = reinterpret_cast<uint4*>(tail + d.slab_off);
        stage_slab_rows(d.B, d.d_out, d.N, cpa, slab, row0 + 4 * q0, 4 * nq, etid);     // weights: before the wait
        // where this thread's accumulator row goes: slice sj of the tile, rows [4 sq0, 4 (sq0 + snq))
        const int row_in_tile = quad * 32 + lane;
        int sj = 0, sq0 = 0, snq = 32;
        for (int c = 0; c < S; ++c) {
            int a, b;
            row_slice(c, S, a, b);
            if (row_in_tile / 4 >= a) {
                sj = c;
                sq0 = a;
                snq = b;
            }
        }
        // block j of CTA sj's receive area, this row's column; the same offsets in every CTA of the cluster
        const uint32_t push_dst = map_to_cta(tail_u32 + (uint32_t)d.recv_off + (uint32_t)j * (uint32_t)(d.BN * 16 * snq) +
                                                 (uint32_t)(row_in_tile - 4 * sq0) * 4u,
                                             (uint32_t)sj);
        const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16);
        float* recv = reinterpret_cast<float*>(tail + d.recv_off);
        const int blk4 = (int)(blk_bytes / 16);
        const int items = nq * ntok;
        if (d.pdl) asm volatile("griddepcontrol.wait;" ::: "memory");     // everything below touches scratch or x's products
        bool ok = true;

        // ---- step 1: the cluster's piece of the stacked shrink, reduce-scattered by row slices
        if (stk_cluster) {
            bool a_ok = ns > 0 ? mbar_wait(bar_acc2, 0) : true;
            if (!a_ok && lane == 0) cluster_flag_error(d, 3, 1300);
            a_ok = __all_sync(0xFFFFFFFFu, a_ok);
            tc_fence_after();
            if (etid == 0) CL_STAMP(4);
            tmem_rows_to_cluster(taddr + (uint32_t)d.acc2_col, c_begin, c_end, a_ok && ns > 0, push_dst, 4 * snq);
            epi_barrier();
            if (etid < S) mbar_arrive_cluster(map_to_cta(bar_stk, (uint32_t)etid));
            if (etid == 0) CL_STAMP(5);
            ok = mbar_wait_cluster(bar_stk, 0) && a_ok;
            if (etid == 0) CL_STAMP(6);
            if (!ok && lane == 0) cluster_flag_error(d, 4, 1350);
            // sum of the S blocks in rank order -> [token][128] rows of the cluster's partial, columns of this slice
            float* up = d.u_part + (((size_t)c_slice * d.aux_tiles + a_tile) * d.T) * kBM + 4 * q0;
            for (int it = etid; it < items && ok; it += kEpiThreads) {
                const int t = it / nq, ql = it - t * nq;
                const float4* p4 = reinterpret_cast<const float4*>(recv) + it;
                float4 acc = p4[0];
                for (int c = 1; c < S; ++c) {
                    const float4 v = p4[c * blk4];
                    acc.x += v.x;
                    acc.y += v.y;
                    acc.z += v.z;
                    acc.w += v.w;
                }
                *reinterpret_cast<float4*>(up + (size_t)t * kBM + 4 * ql) = acc;
            }
            epi_barrier();
            if (etid == 0) {
                __threadfence();
                atomicAdd(d.ctr + 0, 1);
                CL_STAMP(7);
            }
        }

        // ---- selection for this CTA's share of the tokens, from the summed partials of all clusters
        const int g = (int)blockIdx.x, n_cta = (int)gridDim.x;
        const int t0 = d.T * g / n_cta, t1 = d.T * (g + 1) / n_cta, ntl = t1 - t0;
        const int n_active = d.SL * d.aux_tiles;
        const uint32_t recv_u32 = tail_u32 + (uint32_t)d.recv_off;
        if (ntl > 0) {
            const uint32_t rows_bytes = (uint32_t)(n_active * ntl * kBM * 4);
            if (etid == 0) {
                if (!wait_counter_slow(d.ctr + 0, d.n_stk, 100)) {
                    cluster_flag_error(d, 4, 1400);
                    ok = false;
                }
                tmem_slot[1] = ok ? 1u : 0u;                               // what thread 0 found, for the other threads
                mbar_expect_tx(bar_sel, ok ? rows_bytes : 0u);
                CL_STAMP(8);
            }
            epi_barrier();                    // thread 0 has seen all pieces; nobody reads the receive blocks any more
            const bool go = *reinterpret_cast<volatile uint32_t*>(tmem_slot + 1) != 0u;
            if (etid < n_active && go)
                bulk_load_block(recv_u32 + (uint32_t)(etid * ntl * kBM * 4), d.u_part + ((size_t)etid * d.T + t0) * kBM,
                                (uint32_t)(ntl * kBM * 4), bar_sel);
            bool s_ok = go ? mbar_wait(bar_sel, 0) : false;
            if (!s_ok && lane == 0) cluster_flag_error(d, 4, 1450);
            s_ok = __all_sync(0xFFFFFFFFu, s_ok);                          // the selection is warp-collective
            const float4* sm4 = reinterpret_cast<const float4*>(recv);
            float4* rows4 = reinterpret_cast<float4*>(tail + d.recv_off + rows_bytes);   // [ntl][tiles * 128] floats
            const int per_tok = d.aux_tiles * 32, zs4 = d.aux_tiles * ntl * 32;
            for (int it = etid; it < ntl * per_tok && s_ok; it += kEpiThreads) {
                const int tl = it / per_tok, rem = it - tl * per_tok, tl_tile = rem >> 5, l4 = rem & 31;
                const float4* src = sm4 + (tl_tile * ntl + tl) * 32 + l4;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
                for (int z = 0; z < d.SL; ++z) {                          // slices in order: the same sum every run
                    const float4 v = src[z * zs4];
                    acc.x += v.x;
                    acc.y += v.y;
                    acc.z += v.z;
                    acc.w += v.w;
                }
                rows4[it] = acc;
            }
            epi_barrier();
            for (int tl = warp - 2; tl < ntl && s_ok; tl += kEpiThreads / 32)
                select_token_row(reinterpret_cast<const float*>(rows4 + tl * per_tok), d.gate_tile, d.gate_row0, t0 + tl, d.N,
                                 d.r, d.k, d.inv_tau, lane, d.topk_idx, d.topk_w, d.uw);
            epi_barrier();
            if (etid == 0) {
                __threadfence();
                atomicAdd(d.ctr + 1, 1);
                CL_STAMP(9);
            }
            ok = ok && s_ok;
        }
        // the peers may store their main slices into this CTA's receive blocks from here on
        if (S > 1 && etid < S && etid != j) mbar_arrive_cluster(map_to_cta(bar_free, (uint32_t)etid));

        // ---- the routing of all tokens, then the LoRA expand of this CTA's row slice (Eq. 2)
        const uint32_t idx_bytes = ((uint32_t)(ntok * d.k * 4) + 15u) & ~15u;
        const uint32_t uw_bytes = (uint32_t)(ntok * d.k * d.r * 4);
        const uint32_t idx_off = (uint32_t)d.route_off, uw_off = idx_off + ((idx_bytes + 127u) & ~127u);
        if (etid == 0) {
            bool r_ok = wait_counter_slow(d.ctr + 1, d.n_sel, 100);
            if (!r_ok) cluster_flag_error(d, 4, 1500);
            CL_STAMP(10);
            tmem_slot[2] = r_ok ? 1u : 0u;
            mbar_expect_tx(bar_route, r_ok ? idx_bytes + uw_bytes : 0u);
            if (r_ok) {
                bulk_load_block(tail_u32 + idx_off, d.topk_idx, idx_bytes, bar_route);
                bulk_load_block(tail_u32 + uw_off, d.uw, uw_bytes, bar_route);
            }
            // the CTA reads no scratch counter any more: count it out; the last one re-arms the counters
            if (atomicAdd(d.ctr + 2, 1) == n_cta - 1) {
                d.ctr[0] = 0;
                d.ctr[1] = 0;
                d.ctr[2] = 0;
            }
        }
        bool r_ok = mbar_wait(bar_route, 0);
        if (etid == 0) CL_STAMP(11);
        if (*reinterpret_cast<volatile uint32_t*>(tmem_slot + 2) == 0u) r_ok = false;   // written before the arrival above
        ok = ok && r_ok;
        const int* s_idx = reinterpret_cast<const int*>(tail + idx_off);
        const float4* s_uw4 = reinterpret_cast<const float4*>(tail + uw_off);
        float4* dblk = reinterpret_cast<float4*>(tail + d.delta_off);
        const int slab_rows = 4 * nq;
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

        if (etid == 0) CL_STAMP(12);
        // ---- step 2: the main accumulator, reduce-scattered by row slices; partials + expand, one rounding, y
        bool m_ok = mbar_wait(bar_acc, 0);
        if (!m_ok && lane == 0) cluster_flag_error(d, 3, 1600);
        if (S > 1 && !mbar_wait_cluster(bar_free, 0)) {
            if (lane == 0) cluster_flag_error(d, 4, 1650);
            m_ok = false;
        }
        m_ok = __all_sync(0xFFFFFFFFu, m_ok);
        tc_fence_after();
        if (etid == 0) CL_STAMP(13);
        tmem_rows_to_cluster(taddr, c_begin, c_end, m_ok && n_it > 0, push_dst, 4 * snq);
        epi_barrier();
        if (etid < S) mbar_arrive_cluster(map_to_cta(bar_mainx, (uint32_t)etid));
        if (!mbar_wait_cluster(bar_mainx, 0)) {
            if (lane == 0) cluster_flag_error(d, 4, 1700);
            ok = false;
        }
        if (etid == 0) CL_STAMP(14);
        ok = ok && m_ok;
        for (int it = etid; it < items && ok; it += kEpiThreads) {
            const int t = it / nq, ql = it - t * nq;
            const float4* p4 = reinterpret_cast<const float4*>(recv) + it;
            float4 acc = p4[0];
            for (int c = 1; c < S; ++c) {                        // partials in rank order: the same sum every run
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
        if (etid == 0) CL_STAMP(15);
    }

    tc_fence_before();
    __syncwarp();
    cluster_sync();                     // nobody leaves while a peer may still store into it or signal it
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)d.tmem_cols)
                     : "memory");
}

}  // namespace meteora
