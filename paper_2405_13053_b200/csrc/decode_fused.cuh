// Whole MeteoRA linear forward for a decode batch (one token tile, T <= 256, rank a multiple of 8) as ONE kernel
// launch, for one module or for up to four modules that share x.
// Included by wgemm_tcgen05.cu after the device helpers it uses.
//
// The grid holds two kinds of CTAs, all resident at the same time (cooperative launch, no clusters):
//   - main CTAs.  The base product W0 x is cut into units of one 128-row tile of W0 times kc k-steps, numbered
//     tile by tile, and main CTA i takes the units [U*i/M, U*(i+1)/M): every SM streams the same number of
//     bytes whatever the shape, and a CTA's range covers the tail of one tile and the head of the next, or up
//     to kMaxSeg tiles when a layer has more row tiles than CTAs (the host checks).  Each segment runs through
//     TMA + tcgen05 into its own TMEM accumulator and goes to an fp32 scratch (it stays in L2).  When all the
//     CTAs that share a tile have delivered, each of them sums its slice of the tile's rows in CTA order, adds
//     the LoRA expand of those rows (Eq. 2: the B rows of every adapter wait in shared memory, the routing
//     arrives from the aux CTAs) and stores y;
//   - a few aux CTAs on the SMs the main CTAs leave free: each computes a slice of the stacked shrink
//     [A_0..A_{N-1}; Wg] x (every adapter's A_i x and the gate logits, Sec. 3.1) on the same main loop and
//     sends its fp32 accumulator tile to scratch as one bulk copy; once all partials are in, the aux CTAs share
//     the tokens and run the top-k selection and the softmax over the selected logits (Eq. 3), publishing
//     topk_idx, topk_w, uw.
// While the base product is short (W0 below 40 MB) the main CTAs give the aux CTAs a head start of 1.8
// microseconds, so the 2 MB of the shrink are ahead of W0 in the memory queues (measured: a fixed delay does
// as well as waiting for a counter the aux CTAs bump, without the round trip); they need the routing only after
// their main loop and the exchange of the partial tiles.  Every wait is bounded; on expiry the status word is
// set and the kernel drains.  The counters live in the workspace header and are re-armed by the last CTA to exit.
#pragma once

namespace meteora {

constexpr int kMaxSeg = 4;     // row tiles a main CTA's unit range may touch (one TMEM accumulator each)
constexpr int kMaxGroup = kMaxGroupModules;   // modules one launch can serve (they share x: q/k/v, gate/up)

// What differs between the modules of a group: weights come through the tensor maps, the rest is here.
struct DecodeModule {
    const __nv_bfloat16* B;
    __nv_bfloat16* y;
    int d_out;
    int tile0;             // first row tile of the module in the group-wide numbering of 128-row tiles
    int32_t* topk_idx;     // selection results, written by aux CTAs, read by main CTAs
    float* topk_w;
    float* uw;
    float* u_part;         // [aux_slices][aux_tiles][T][128] partial stacked shrink, tile by tile as accumulated
};
struct DecodeMaps {
    CUtensorMap W0[kMaxGroup], A[kMaxGroup], At[kMaxGroup], G[kMaxGroup];
};

struct DecodeParams {
    WGemmParams main;      // base product: ring geometry, staging offsets (B, y, d_out, topk_idx, uw unused here)
    int n_mod;             // modules of the group; their row tiles are numbered one after the other
    DecodeModule mod[kMaxGroup];
    int n_main;            // main CTAs (M)
    int upt;               // units per row tile = k-steps / kc
    int units;             // row tiles * upt (U); U * M stays below 2^31 (checked by the host)
    int n_aux;             // aux CTAs; they take the lowest block indices so that they are scheduled first
    int a_tiles, a_rows;   // row tiles / rows of the stacked A matrix (N * r rows)
    int aux_tiles;         // row tiles of the stacked shrink: a_tiles, plus one for Wg unless it fits behind A's last rows
    int gate_tile;         // the tile that holds the N rows of Wg, from tile row gate_row0 on
    int gate_row0;
    int aux_slices;        // contraction slices per aux row tile; active aux CTAs = aux_tiles * aux_slices
    int aux_stages;        // ring depth of the aux main loop (one k-step per stage)
    int bar_stages;        // barriers are laid out for max(main stages, aux stages) ring slots
    int ld_u, col_logits;
    float inv_tau;
    int hold_after;        // ring stages the main CTAs request before that head start (0: none)
    int hold;              // 1: main CTAs start loading only after the aux CTAs have issued their first loads; > 1: after that many nanoseconds
    int32_t* ctr;          // [0] aux partials written, [1] selections published, [2] CTAs exited, [3] aux loads issued
    float* part_g;         // [row tile + main CTA][BN][128] fp32 partial accumulator tiles of the base product
    int32_t* tile_ctr;     // [row tiles] partials delivered per tile
    int row_tiles;         // of all modules together
    int slab_rows;         // rows of B (of every adapter) the staging buffer of a main CTA holds
    int trace_call;        // trace builds: which record of the trace buffer this launch fills
    int narrow_select;     // selection in two round trips (logits, then the picks' shrink values) instead of one wide one
    int pdl;               // launched with programmatic stream serialization: trigger the next launch, wait for the previous
};

__device__ __forceinline__ int ld_acquire(const int32_t* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// One contiguous block from shared memory to global memory as a single bulk copy of the TMA engine (both
// addresses 16-byte aligned, `bytes` a multiple of 16); returns when the writes are complete.  The data were
// written to shared memory by ordinary stores: every writer ran fence.proxy.async before the barrier that
// precedes this call.
__device__ __forceinline__ void bulk_store_block(void* gdst, uint32_t smem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_src), "r"(bytes)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// Bounded wait until *ctr >= target; false if it did not happen within the wait limit.
__device__ __forceinline__ bool wait_counter(const int32_t* ctr, int target) {
    const long long t0 = clock64(), limit = g_wait_limit_cycles;
    while (ld_acquire(ctr) < target) {
        if (clock64() - t0 > limit) return false;
        __nanosleep(32);
    }
    return true;
}

// Selection for one token by one warp, every partial copy of the token's row read in ONE round trip: the
// N*r shrink values and the N logits are summed over the `zsplits` copies in slice order (two 16-byte columns
// per lane, all loads in flight together) into `wbuf` (shared memory, ld_u floats), then top-k, softmax over
// the picks (Eq. 3) and uw[t,j,:] = w_j * (A_{i_j} x) come from there.  The rank r is a multiple of 4; 256 floats
// per 32 lanes and pass, further passes for more columns.
// The partials are laid out as the aux CTAs' accumulator tiles, u_part[slice][tile][T][128]: stacked row R of
// [A; Wg] sits in tile R / 128 at R % 128, logit n in the gate tile at gate_row0 + n.
__device__ __forceinline__ void select_token_wide(const float* u_part, int T, int tiles, int gate_tile, int gate_row0,
                                                  int col_logits, int zsplits, int t, int N, int r, int k,
                                                  float inv_tau, int lane, float* wbuf, int32_t* topk_idx,
                                                  float* topk_w, float* uw) {
    constexpr int ZMAX = 16;
    const int n_a4 = N * r / 4, n_c4 = n_a4 + (N + 3) / 4;         // 16-byte chunks: shrink values, then logits
    const size_t zstride = (size_t)tiles * T * kBM;
    for (int c0 = 0; c0 < n_c4; c0 += 64) {
        float4 acc[2];
        float4 v[2][ZMAX];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            // No branch around the loads (the compiler would wait for each one before taking the next): a chunk
            // or a slice past the end is clamped to the last one, read again and left out of the sum below.
            const int c4 = min(c0 + h * 32 + lane, n_c4 - 1);
            const int tile = c4 < n_a4 ? (4 * c4) / kBM : gate_tile;
            const int within = c4 < n_a4 ? (4 * c4) % kBM : gate_row0 + 4 * (c4 - n_a4);
            const float* src = u_part + ((size_t)tile * T + t) * kBM + within;
#pragma unroll
            for (int z = 0; z < ZMAX; ++z)
                v[h][z] = __ldcg(reinterpret_cast<const float4*>(src + (size_t)min(z, zsplits - 1) * zstride));
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            acc[h] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int z = 0; z < ZMAX; ++z) {
                acc[h].x += z < zsplits ? v[h][z].x : 0.f;
                acc[h].y += z < zsplits ? v[h][z].y : 0.f;
                acc[h].z += z < zsplits ? v[h][z].z : 0.f;
                acc[h].w += z < zsplits ? v[h][z].w : 0.f;
            }
            const int c4 = c0 + h * 32 + lane;
            const int col = c4 < n_a4 ? 4 * c4 : col_logits + 4 * (c4 - n_a4);
            if (c4 < n_c4) *reinterpret_cast<float4*>(wbuf + col) = acc[h];
        }
    }
    __syncwarp();
    float v[kSelVals];
#pragma unroll
    for (int i = 0; i < kSelVals; ++i) v[i] = lane + 32 * i < N ? wbuf[col_logits + lane + 32 * i] : 0.f;
    int idx;
    float w;
    warp_topk_softmax(v, N, k, inv_tau, lane, idx, w);
    if (lane < k) {
        topk_idx[(size_t)t * k + lane] = idx;
        topk_w[(size_t)t * k + lane] = w;
    }
    for (int c0 = 0; c0 < k * r; c0 += 32) {
        const int c = c0 + lane;
        const int j = min(c / r, k - 1), q = c - j * r;
        const int ij = __shfl_sync(0xFFFFFFFFu, idx, j);
        const float wj = __shfl_sync(0xFFFFFFFFu, w, j);
        if (c < k * r) uw[(size_t)t * k * r + c] = wj * wbuf[ij * r + q];
    }
    __syncwarp();
}

// The same selection in two round trips that move far less: first the N logits of the token from every slice
// (lane n owns logit n, n + 32, ...), top-k and softmax, then only the k * r shrink values of the picks.  A token
// costs (N + k r) * slices floats instead of the whole stacked row (N r + N) * slices: 1.8 KB instead of 10 KB
// at N = 28, r = 8, k = 2 and 10 slices, which is what counts once every aux warp has a token (the aux SMs
// take in the partial copies at 50 - 60 GB/s each).  Same sums in the same slice order as select_token_wide.
__device__ __forceinline__ void select_token_narrow(const float* u_part, int T, int tiles, int gate_tile, int gate_row0,
                                                    int zsplits, int t, int N, int r, int k, float inv_tau, int lane,
                                                    int32_t* topk_idx, float* topk_w, float* uw) {
    constexpr int ZMAX = 16;
    const size_t zstride = (size_t)tiles * T * kBM;
    float v[kSelVals];
    const float* grow = u_part + ((size_t)gate_tile * T + t) * kBM + gate_row0;
#pragma unroll
    for (int i = 0; i < kSelVals; ++i) {
        v[i] = 0.f;
        if (32 * i < N) {                                   // uniform across the warp
            const float* src = grow + min(lane + 32 * i, N - 1);
            float part[ZMAX];
#pragma unroll
            for (int z = 0; z < ZMAX; ++z) part[z] = __ldcg(src + (size_t)min(z, zsplits - 1) * zstride);
#pragma unroll
            for (int z = 0; z < ZMAX; ++z) v[i] += z < zsplits ? part[z] : 0.f;
        }
    }
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
        const int R = ij * r + q;                           // row of the stacked matrix [A_0 .. A_{N-1}]
        const float* src = u_part + ((size_t)(R / kBM) * T + t) * kBM + (R % kBM);
        float part[ZMAX];
#pragma unroll
        for (int z = 0; z < ZMAX; ++z) part[z] = __ldcg(src + (size_t)min(z, zsplits - 1) * zstride);
        float u = 0.f;
#pragma unroll
        for (int z = 0; z < ZMAX; ++z) u += z < zsplits ? part[z] : 0.f;
        if (c0 + lane < k * r) uw[(size_t)t * k * r + c0 + lane] = wj * u;
    }
}

// B rows [row0, row0 + nrows) of every adapter (8 bf16 = 16 bytes each) as slab[e][row % 4][row / 4], so that
// threads owning consecutive groups of 4 rows read consecutive 16-byte words; rows past d_out are zero.
// (For ranks above 8 a row has cpa = r / 8 such 16-byte words: slab[e][chunk][row % 4][row / 4].)
__device__ __forceinline__ void stage_slab_rows(const __nv_bfloat16* B, int d_out, int N, int cpa, uint4* slab,
                                                int row0, int nrows, int etid) {
    const uint4* Bg = reinterpret_cast<const uint4*>(B);
    const int per_e = nrows * cpa, total = N * per_e, nq = nrows / 4;
    for (int i = etid; i < total; i += kEpiThreads) {
        const int e = i / per_e, w = i - e * per_e, rl = w / cpa, c = w - rl * cpa, o = row0 + rl;
        slab[(e * cpa + c) * nrows + (rl & 3) * nq + (rl >> 2)] =
            o < d_out ? __ldg(Bg + ((size_t)e * d_out + o) * cpa + c) : make_uint4(0u, 0u, 0u, 0u);
    }
}

// Last step of a main CTA for one tile: rows [4*q0, 4*(q0+nq)) of the tile, all tokens.  Work items are
// (token, group of 4 rows); a thread keeps U items in flight: the values of the C partial tiles first (one round
// trip to L2; `parts` in CTA order, the first `c` are real), then their sum in that order, the expand of Eq. 2
// from the staged B rows and the routing in shared memory, one rounding to bf16 and the store.  The routing is
// staged by warp 0, which arrives on named barrier 2 when it is in shared memory; the threads here join that
// barrier once (`routing_pending`), after issuing their first loads.  `nthr` threads (etid = 0 .. nthr-1) share
// the tile: all 256 epilogue threads, or half of them when the CTA finishes rows of two tiles at once.
template <int C, int U>
__device__ __forceinline__ void finish_rows(__nv_bfloat16* y, int d_out, int k, int cpa, const float* const (&parts)[C], int c,
                                            int tile_row0, int q0, int nq, int ntok, const uint4* slab,
                                            const float* s_uw, const int* s_idx, int etid, int nthr,
                                            bool& routing_pending) {
    const int items = nq * ntok, slab_rows = 4 * nq;
    const float4* s_uw4 = reinterpret_cast<const float4*>(s_uw);
    for (int base = 0; base < items; base += nthr * U) {
        float4 v[U][C];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int it = min(base + etid + u * nthr, items - 1);
            const int t = it / nq, ql = it - t * nq;
            const size_t off = (size_t)t * kBM + (q0 + ql) * 4;
#pragma unroll
            for (int q = 0; q < C; ++q)                // no branch: parts[q] repeats the last real tile for q >= c
                v[u][q] = __ldcg(reinterpret_cast<const float4*>(parts[q] + off));
        }
        if (routing_pending) {
            asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads + 32) : "memory");
            routing_pending = false;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int it = base + etid + u * nthr;
            if (it >= items) break;
            const int t = it / nq, ql = it - t * nq;
            float4 acc = v[u][0];
#pragma unroll
            for (int q = 1; q < C; ++q) {
                acc.x += q < c ? v[u][q].x : 0.f;
                acc.y += q < c ? v[u][q].y : 0.f;
                acc.z += q < c ? v[u][q].z : 0.f;
                acc.w += q < c ? v[u][q].w : 0.f;
            }
            for (int j = 0; j < k; ++j) {
                const int slot = t * k + j;
                for (int ch = 0; ch < cpa; ++ch) {               // 8 rank entries at a time
                    const float4 u0 = s_uw4[2 * (slot * cpa + ch)], u1 = s_uw4[2 * (slot * cpa + ch) + 1];
                    const uint4* b = slab + (size_t)(s_idx[slot] * cpa + ch) * slab_rows + ql;
                    fma8(b[0], u0, u1, acc.x);
                    fma8(b[nq], u0, u1, acc.y);
                    fma8(b[2 * nq], u0, u1, acc.z);
                    fma8(b[3 * nq], u0, u1, acc.w);
                }
            }
            const int o = tile_row0 + (q0 + ql) * 4;
            __nv_bfloat16* dst = y + (size_t)t * d_out + o;
            if ((d_out & 3) == 0 && o + 3 < d_out) {
                const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
                uint2 pk;
                pk.x = *reinterpret_cast<const uint32_t*>(&lo);
                pk.y = *reinterpret_cast<const uint32_t*>(&hi);
                *reinterpret_cast<uint2*>(dst) = pk;
            } else {
                const float f[4] = {acc.x, acc.y, acc.z, acc.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (o + i < d_out) dst[i] = __float2bfloat16_rn(f[i]);
            }
        }
    }
}

// Rows of row tile `tile` that main CTA `main_id` finishes.  The tile is shared by the main CTAs owner(first
// unit) .. owner(last unit), `c` of them from `first` on; contributor j takes the groups of 4 rows
// [32 j / c, 32 (j + 1) / c).  Unit u belongs to main CTA ceil((u + 1) M / U) - 1.
__device__ __forceinline__ void tile_share(int tile, int upt, int M, unsigned U, int main_id, int& first, int& c,
                                           int& q0, int& nq) {
    const unsigned x0 = (unsigned)(tile * upt), x1 = x0 + (unsigned)upt - 1u;
    first = (int)(((x0 + 1u) * (unsigned)M + U - 1u) / U) - 1;
    const int last = (int)(((x1 + 1u) * (unsigned)M + U - 1u) / U) - 1;
    c = last - first + 1;
    const int j = main_id - first;
    q0 = 32 * j / c;
    nq = 32 * (j + 1) / c - q0;
}

// A main CTA finishes its (one or two) tiles side by side, all B rows staged at once, if they fit the staging
// buffer together; else tile after tile.  Both the epilogue warps and warp 0 ask.
__device__ __forceinline__ bool finishes_side_by_side(int tile_a, int nseg, int upt, int M, unsigned U, int main_id,
                                                      int N, int cpa, int slab_rows) {
    if (nseg > 2) return false;
    int words = 0;
    for (int sg = 0; sg < nseg; ++sg) {
        int first, c, q0, nq;
        tile_share(tile_a + sg, upt, M, U, main_id, first, c, q0, nq);
        words += N * cpa * 4 * nq;
    }
    return words <= N * cpa * slab_rows;
}

// Module that owns a row tile of the group-wide numbering.
__device__ __forceinline__ int module_of_tile(const DecodeModule* mod, int n_mod, int tile) {
    int m = 0;
    for (int i = 1; i < n_mod; ++i)
        if (tile >= mod[i].tile0) m = i;
    return m;
}

template <int C, int U>
__device__ __forceinline__ void finish_tile(__nv_bfloat16* y, int d_out, int k, int cpa, int tile_row0, const float* part_g,
                                            size_t part_stride, int units, int M, int upt, int tile, int first_cta, int c,
                                            int q0, int nq, int ntok, const uint4* slab, const float* s_uw,
                                            const int* s_idx, int etid, int nthr, bool& routing_pending) {
    // The partial of main CTA i for row tile t sits in slot t + i: unit ranges are ordered, so no two (CTA, tile)
    // pairs share a slot, and at most row tiles + main CTAs slots are in use.
    const float* parts[C];
#pragma unroll
    for (int q = 0; q < C; ++q) parts[q] = part_g + (size_t)(tile + first_cta + min(q, c - 1)) * part_stride;
    finish_rows<C, U>(y, d_out, k, cpa, parts, c, tile_row0, q0, nq, ntok, slab, s_uw, s_idx, etid, nthr, routing_pending);
}

#ifdef METEORA_TRACE
// Trace build only: every CTA stamps the global nanosecond timer at the points of interest.
constexpr int kTraceCalls = 32, kTraceCtas = 256, kTraceSlots = 16;
__device__ unsigned long long g_fused_trace[kTraceCalls * kTraceCtas * kTraceSlots];
#define FUSED_STAMP(p, base, slot)                                                                   \
    do {                                                                                             \
        unsigned long long t_;                                                                       \
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                                       \
        if (blockIdx.x < kTraceCtas)                                                                 \
            g_fused_trace[((d.trace_call % kTraceCalls) * kTraceCtas + blockIdx.x) * kTraceSlots + (slot)] = t_; \
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
// A second weight map `tmW2` (or the only one, when tmW is null) lands `w2_off` bytes into the weight tile: the
// rows of Wg behind the last rows of A.
__device__ __forceinline__ bool fused_producer(const RingGeom& g, const CUtensorMap* tmW, const CUtensorMap* tmXp,
                                               int row0, int ks0, int niter, int32_t* first_batch_done,
                                               const CUtensorMap* tmW2 = nullptr, uint32_t w2_off = 0) {
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
            if (tmW) tma_load_3d(dst, tmW, 0, row0, kstep, full);
            if (tmW2) tma_load_3d(dst + w2_off, tmW2, 0, 0, kstep, full);
            tma_load_3d(dst + g.kc * kWTileBytes, tmXp, 0, 0, kstep, full);
        } else {
            if (tmW) tma_load_2d(dst, tmW, kstep * kBK, row0, full);
            if (tmW2) tma_load_2d(dst + w2_off, tmW2, kstep * kBK, 0, full);
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

// One thread per CTA, once the CTA has read the workspace counters for the last time: counts the CTA out; the
// last one re-arms the counters for the next call on this workspace.  (No fence between the stores: nobody
// reads them before the next kernel, and the kernel boundary orders them.)
__device__ __forceinline__ void count_cta_out(const DecodeParams& d) {
    if (atomicAdd(d.ctr + 2, 1) == (int)gridDim.x - 1) {
        d.ctr[0] = 0;
        d.ctr[1] = 0;
        d.ctr[3] = 0;
        for (int i = 0; i < d.row_tiles; ++i) d.tile_ctr[i] = 0;
        d.ctr[2] = 0;
    }
}

__global__ void __launch_bounds__(kThreads)
k_decode_fused(const __grid_constant__ DecodeMaps maps, const __grid_constant__ CUtensorMap tmX,
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
    const int nbar = 2 * d.bar_stages + kMaxSeg + 1;  // full / empty for the deeper of the two rings, one per segment
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ring_ptr + ring_bytes + nbar * 8);
    uint8_t* epi = ring_ptr + ring_bytes + p.epi_off;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool is_aux = (int)blockIdx.x < d.n_aux;
    const int main_id = (int)blockIdx.x - d.n_aux;
    const int n_active = d.n_mod * d.aux_tiles * d.aux_slices;
    bool counted_out = false;                      // thread 0: this CTA has been counted out before the end

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
    if (d.pdl) {
        // Programmatic dependent launch: the next kernel on the stream is launched and runs its own set-up
        // (barriers, TMEM) under this kernel's tail; up to here this kernel has touched no global memory, and it
        // touches none before the kernel ahead of it has completed.
        if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }
    const uint32_t idesc = instr_desc_bf16(p.BN);
    const int quad = warp & 3;
    const int etid = threadIdx.x - 64;
    const int ntok = min(p.BN, p.T);
    const int half = ((p.BN / 16 + 1) / 2) * 16;
    const int c_begin = warp < 6 ? 0 : half, c_end = warp < 6 ? half : p.BN;
#ifdef METEORA_TRACE
    const bool tr_main = !is_aux, tr_aux = is_aux;
#else
    const bool tr_main = main_id == 0, tr_aux = blockIdx.x == 0;
#endif

    if (threadIdx.x == 0 && tr_main) FUSED_STAMP(p, 32, 8);
    if (threadIdx.x == 0 && tr_aux) FUSED_STAMP(p, 48, 5);
    if (threadIdx.x == 0 && tr_main) FUSED_STAMP(p, 32, 0);
    if (threadIdx.x == 0 && tr_aux) FUSED_STAMP(p, 48, 0);

    if (is_aux) {
        // ================================================================== aux CTA
        const int aux_id = blockIdx.x;
        const bool active = aux_id < n_active;
        const int group_tiles = d.n_mod * d.aux_tiles;                       // (module, tile) pairs of the stacked shrinks
        const int am = active ? (aux_id % group_tiles) / d.aux_tiles : 0;    // module
        const int tile = (aux_id % group_tiles) % d.aux_tiles, slice = aux_id / group_tiles;
        // (k-steps x slices stays far below 2^31: 32-bit divisions, this is on the way to the first load)
        const int ks0 = active ? (p.ksteps * slice) / d.aux_slices : 0;
        const int ks1 = active ? (p.ksteps * (slice + 1)) / d.aux_slices : 0;
        const int niter = ks1 - ks0;
        const RingGeom geom = {ring, bar_base, x_tile_bytes, kWTileBytes + x_tile_bytes, d.aux_stages, 1, p.maps3d};
        const uint32_t bar_acc = bar_base + 2 * d.aux_stages * 8;
        if (warp == 0) {
            if (lane == 0 && active) {
                // A's last tile has its own map (its box stops at A's last row when Wg follows in the same tile)
                const CUtensorMap* mA = tile >= d.a_tiles ? nullptr : tile == d.a_tiles - 1 ? &maps.At[am] : &maps.A[am];
                const CUtensorMap* mG = tile == d.gate_tile ? &maps.G[am] : nullptr;
                if (tr_aux) FUSED_STAMP(p, 48, 6);
                if (!fused_producer(geom, mA, &tmX1, tile * kBM, ks0, niter, d.ctr + 3, mG, (uint32_t)d.gate_row0 * 128u))
                    flag_error(p, 1, 400);
                if (tr_aux) FUSED_STAMP(p, 48, 7);
            }
        } else if (warp == 1) {
            if (lane == 0 && active) {
#ifdef METEORA_TRACE
                if (niter > 0) mbar_wait(bar_base, 0);                          // first stage landed
                FUSED_STAMP(p, 48, 8);
#endif
                if (!fused_mma(geom, tmem_base, idesc, niter)) flag_error(p, 2, 500);
                umma_commit(bar_acc);
                if (tr_aux) FUSED_STAMP(p, 48, 1);
            }
        } else if (active) {
            bool acc_ok = mbar_wait(bar_acc, 0);
            if (!acc_ok && lane == 0) flag_error(p, 3, 600);
            acc_ok = __all_sync(0xFFFFFFFFu, acc_ok);
            tc_fence_after();
            if (etid == 0 && tr_aux) FUSED_STAMP(p, 48, 9);
            // The accumulator tile goes out as it is, [token][128 rows] fp32: staged in the idle ring (lane = row:
            // a warp writes 128 contiguous bytes of shared memory), then ONE bulk copy by thread 0 below.  (Plain
            // 4-byte stores straight to global memory took 2.7 us for the 64 KB of a 128-token tile.)
            const int trow = quad * 32 + lane;                                   // row of the tile
            float* stage = reinterpret_cast<float*>(ring_ptr);
            for (int c = c_begin; c < c_end; c += 16) {
                float v[16];
                if (acc_ok) {
                    tmem_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + c, v);
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = 0.f;
                }
#pragma unroll
                for (int i = 0; i < 16; ++i) stage[(c + i) * kBM + trow] = v[i];
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");         // generic writes -> bulk copy reads
            if (etid == 0 && tr_aux) FUSED_STAMP(p, 48, 10);
        }
        __syncwarp();
        __syncthreads();
        if (active) {
            if (threadIdx.x == 0) {
                float* dst = d.mod[am].u_part + (((size_t)slice * d.aux_tiles + tile) * p.T) * kBM;
                bulk_store_block(dst, ring, (uint32_t)p.T * kBM * 4u);
                if (tr_aux) FUSED_STAMP(p, 48, 2);
                __threadfence();
                atomicAdd(d.ctr + 0, 1);
                if (!wait_counter(d.ctr + 0, n_active)) flag_error(p, 4, 700);   // every slice of every tile is in
                if (tr_aux) FUSED_STAMP(p, 48, 3);
            }
            __syncthreads();
            const int nwarps = kThreads / 32;                                    // (module, token) items dealt round-robin
            float* wbuf = reinterpret_cast<float*>(ring_ptr) + warp * d.ld_u;     // the ring is idle by now
            for (int it = aux_id * nwarps + warp; it < d.n_mod * p.T; it += n_active * nwarps) {
                const int sm = it / p.T, t = it - sm * p.T;
                const DecodeModule& mo = d.mod[sm];
                if (d.narrow_select)
                    select_token_narrow(mo.u_part, p.T, d.aux_tiles, d.gate_tile, d.gate_row0, d.aux_slices, t, p.N, p.r,
                                        p.k, d.inv_tau, lane, mo.topk_idx, mo.topk_w, mo.uw);
                else
                    select_token_wide(mo.u_part, p.T, d.aux_tiles, d.gate_tile, d.gate_row0, d.col_logits, d.aux_slices, t,
                                      p.N, p.r, p.k, d.inv_tau, lane, wbuf, mo.topk_idx, mo.topk_w, mo.uw);
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                __threadfence();
                atomicAdd(d.ctr + 1, 1);
                if (tr_aux) FUSED_STAMP(p, 48, 4);
            }
        }
    } else {
        // ================================================================== main CTA
        const int M = d.n_main, upt = d.upt;
        const unsigned U = (unsigned)d.units;
        const int u0 = (int)(U * (unsigned)main_id / (unsigned)M);                   // M <= U: never empty
        const int u1 = (int)(U * (unsigned)(main_id + 1) / (unsigned)M);
        const int n_it = u1 - u0;
        const int tile_a = u0 / upt, tile_b = (u1 - 1) / upt;
        const int nseg = tile_b - tile_a + 1;                                        // 1 .. kMaxSeg (host-checked)
        const RingGeom geom = {ring, bar_base, x_tile_bytes, stage_bytes, p.stages, p.kc, p.maps3d};
        const uint32_t bar_acc = bar_base + 2 * p.stages * 8;                        // [0 .. kMaxSeg): one per segment
        const size_t part_stride = (size_t)p.BN * kBM;                               // floats per partial tile
        if (warp == 0) {
            if (lane == 0) {
                // let the stacked shrink get its loads into the memory queues first
                bool ok = true;
                unsigned long long t0 = 0;
                if (d.hold > 1) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
                if (tr_main) FUSED_STAMP(p, 32, 1);
                int cur_tile = -1, row0 = 0;
                const CUtensorMap* tmW0 = &maps.W0[0];
                int tile = tile_a, kpos = u0 - tile_a * upt, st = 0, round = 0;
                for (int it = 0; it < n_it && ok; ++it) {
                    if (it == d.hold_after) {                    // the first hold_after stages go out at once
                        if (d.hold == 1) {
                            ok = wait_counter(d.ctr + 3, n_active);
                            if (!ok) break;
                        } else if (d.hold > 1) {                 // a fixed head start for the aux CTAs, in nanoseconds
                            unsigned long long t1;
                            int spins = 0;                         // bounded like every other wait: 4096 x 64 ns at most
                            do {
                                __nanosleep(64);
                                asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
                            } while (t1 - t0 < (unsigned long long)d.hold && ++spins < 4096);
                        }
                    }
                    if (round > 0) ok = mbar_wait(bar_base + (geom.stages + st) * 8, (round & 1) ^ 1);
                    if (!ok) break;
                    const uint32_t full = bar_base + st * 8, dst = ring + st * stage_bytes;
                    const int kstep = kpos * p.kc;
                    if (tile != cur_tile) {                      // rows of which module's W0
                        const int wm = module_of_tile(d.mod, d.n_mod, tile);
                        cur_tile = tile;
                        tmW0 = &maps.W0[wm];
                        row0 = (tile - d.mod[wm].tile0) * kBM;
                    }
                    mbar_expect_tx(full, stage_bytes);
                    if (p.maps3d) {
                        tma_load_3d(dst, tmW0, 0, row0, kstep, full);
                        tma_load_3d(dst + p.kc * kWTileBytes, &tmX, 0, 0, kstep, full);
                    } else {
                        tma_load_2d(dst, tmW0, kstep * kBK, row0, full);
                        tma_load_2d(dst + kWTileBytes, &tmX, kstep * kBK, 0, full);
                    }
                    if (++kpos == upt) {
                        kpos = 0;
                        ++tile;
                    }
                    if (++st == geom.stages) {
                        st = 0;
                        ++round;
                    }
                }
                if (!ok) flag_error(p, 1, 100);
                if (!wait_counter(d.ctr + 1, n_active)) flag_error(p, 4, 800);              // routing published
                if (tr_main) FUSED_STAMP(p, 32, 4);
            }
            __syncwarp();
            // The routing into shared memory for the epilogue warps, once per tile this CTA finishes rows of (two
            // tiles may belong to two modules of a group); it was written by other CTAs of this kernel: loads
            // that bypass L1.  Then named barrier 2.
            {
                const int slots = ntok * p.k;
                for (int sg = 0; sg < nseg; ++sg) {
                    const DecodeModule& mo = d.mod[module_of_tile(d.mod, d.n_mod, tile_a + sg)];
                    int* s_idx = reinterpret_cast<int*>(epi + p.idx_off) + sg * p.BN * p.k;
                    float4* s_uw4 = reinterpret_cast<float4*>(epi + p.uw_off) + sg * p.BN * p.k * (p.r / 4);
                    const float4* uw4 = reinterpret_cast<const float4*>(mo.uw);
                    // Batches of 8 loads per lane with NO branch in them: an index past the end is clamped to the
                    // last element (those lanes copy it again, the same value to the same place), so the compiler
                    // can issue a batch's loads together: one round trip to L2 per batch at any token count.  (A
                    // loop unrolled by 8 ran its remainder one dependent load at a time, and a bound checked by
                    // `if` does the same for every element: 3 - 5 us at 112 tokens against 1.4 at 128.)
                    const int n_uw = slots * (p.r / 4);
                    for (int b0 = 0; b0 < slots; b0 += 8 * 32) {
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const int i = min(b0 + u * 32 + lane, slots - 1);
                            s_idx[i] = min(max(__ldcg(mo.topk_idx + i), 0), p.N - 1);
                        }
                    }
                    for (int b0 = 0; b0 < n_uw; b0 += 8 * 32) {
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const int i = min(b0 + u * 32 + lane, n_uw - 1);
                            s_uw4[i] = __ldcg(uw4 + i);
                        }
                    }
                }
                __syncwarp();
                // Side by side, every epilogue thread reaches barrier 2 after its last look at a tile counter,
                // and this warp has seen the routing counter: from there on the CTA reads no counter, so it is
                // counted out here, under the last step, instead of after it (the atomic's round trip and the
                // re-arming by the last CTA then end before y is stored; at the end of the kernel they cost
                // 1.5 - 2 us per call).  Tile after tile the later waits come after barrier 2: counted out at the end.
                if (finishes_side_by_side(tile_a, nseg, upt, M, U, main_id, p.N, p.r >> 3, d.slab_rows)) {
                    asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads + 32) : "memory");
                    if (lane == 0) {
                        if (tr_main) FUSED_STAMP(p, 32, 9);
                        __threadfence();
                        count_cta_out(d);
                        counted_out = true;
                    }
                } else {
                    asm volatile("bar.arrive 2, %0;" ::"n"(kEpiThreads + 32) : "memory");
                    if (lane == 0 && tr_main) FUSED_STAMP(p, 32, 9);
                }
            }
        } else if (warp == 1) {
            if (lane == 0) {
                bool ok = true;
                int committed = 0;                                                  // segments announced so far
                int sg = 0, kpos = u0 - tile_a * upt, st = 0, round = 0;            // no divisions in this loop: it paces the tensor cores
                for (int it = 0; it < n_it; ++it) {
                    ok = mbar_wait(bar_base + st * 8, round & 1);
                    if (!ok) break;
                    tc_fence_after();
                    const bool fresh = it == 0 || kpos == 0;                        // first MMA of a segment overwrites
                    const uint32_t acc = tmem_base + (uint32_t)(sg * p.BN);
                    const uint32_t wa = ring + st * stage_bytes, xa = wa + p.kc * kWTileBytes;
                    for (int c = 0; c < p.kc; ++c) {
                        const uint64_t da = smem_desc_sw128(wa + c * kWTileBytes);
                        const uint64_t db = smem_desc_sw128(xa + c * x_tile_bytes);
#pragma unroll
                        for (int kk = 0; kk < kBK / kUmmaK; ++kk)
                            umma_bf16(acc, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, !fresh || (c | kk) != 0);
                    }
                    umma_commit(bar_base + (geom.stages + st) * 8);
                    ++kpos;
                    if (it + 1 == n_it || kpos == upt) {                            // the segment is complete
                        umma_commit(bar_acc + 8 * sg);
                        committed = sg + 1;
                    }
                    if (kpos == upt) {
                        kpos = 0;
                        ++sg;
                    }
                    if (++st == geom.stages) {
                        st = 0;
                        ++round;
                    }
                }
                if (tr_main) FUSED_STAMP(p, 32, 2);
                for (int sg = committed; sg < nseg; ++sg) umma_commit(bar_acc + 8 * sg);   // only after a failed wait
                if (!ok) flag_error(p, 2, 200);
            }
        } else {
            // Which rows of which tile this CTA finishes: tile `t` is shared by the CTAs owner(first unit) ..
            // owner(last unit), in that order; contributor j of c takes the groups of 4 rows [32j/c, 32(j+1)/c).
            int d_tile[kMaxSeg], d_first[kMaxSeg], d_c[kMaxSeg], d_q0[kMaxSeg], d_nq[kMaxSeg], d_mod[kMaxSeg],
                d_row0[kMaxSeg];
            const int cpa = p.r >> 3;                                        // 16-byte words per B row
            uint4* slab = reinterpret_cast<uint4*>(epi + p.slab_off);
            uint4* d_slab[kMaxSeg];
            int slab_words = 0;
            for (int sg = 0; sg < nseg; ++sg) {
                const int tile = tile_a + sg;
                d_tile[sg] = tile;
                tile_share(tile, upt, M, U, main_id, d_first[sg], d_c[sg], d_q0[sg], d_nq[sg]);
                d_slab[sg] = slab + slab_words;
                d_mod[sg] = module_of_tile(d.mod, d.n_mod, tile);
                d_row0[sg] = (tile - d.mod[d_mod[sg]].tile0) * kBM;          // the tile's first row inside its module
                slab_words += p.N * cpa * 4 * d_nq[sg];
            }
            // side by side only if both tiles' rows fit the staging buffer together (a range longer than a
            // tile's units can own one tile entirely and share another); else the tiles are finished one after
            // the other, B rows staged each time
            const bool side_by_side = finishes_side_by_side(tile_a, nseg, upt, M, U, main_id, p.N, cpa, d.slab_rows);
            if (side_by_side) {
                // B rows of the CTA's slices for every adapter: no routing needed yet
                for (int sg = 0; sg < nseg; ++sg)
                    stage_slab_rows(d.mod[d_mod[sg]].B, d.mod[d_mod[sg]].d_out, p.N, cpa, d_slab[sg],
                                    d_row0[sg] + 4 * d_q0[sg], 4 * d_nq[sg], etid);
            }
            if (etid == 0 && tr_main) FUSED_STAMP(p, 32, 3);
            // Accumulators out of TMEM to the fp32 scratch, segment by segment (lane = row, a warp writes 128
            // contiguous bytes per token); each delivery bumps the tile's counter.
            const int row_in_tile = quad * 32 + lane;
            for (int sg = 0; sg < nseg; ++sg) {
                bool acc_ok = mbar_wait(bar_acc + 8 * sg, 0);
                if (!acc_ok && lane == 0) flag_error(p, 3, 300);
                acc_ok = __all_sync(0xFFFFFFFFu, acc_ok);
                tc_fence_after();
                if (etid == 0 && tr_main && sg == nseg - 1) FUSED_STAMP(p, 32, 5);
                float* part = d.part_g + (size_t)(d_tile[sg] + main_id) * part_stride;
                // (plain stores: routed through the idle ring and one bulk copy, as the aux CTAs' tiles are, the
                // delivery was 0 - 1.4 us slower at every shape and batch size measured: the copy's completion has
                // to be awaited before the counter moves, while these stores drain behind the fence)
                for (int c = c_begin; c < c_end; c += 16) {
                    float v[16];
                    if (acc_ok) {
                        tmem_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(sg * p.BN + c), v);
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = 0.f;
                    }
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (c + i < ntok) part[(c + i) * kBM + row_in_tile] = v[i];
                }
                epi_barrier();
                if (etid == 0) {
                    __threadfence();
                    atomicAdd(d.tile_ctr + d_tile[sg], 1);
                }
            }
            // Two tiles to finish: half of the epilogue threads each, side by side (one round trip to L2 for both).
            bool routing_pending = true;
            if (side_by_side) {
                const int nthr = nseg > 1 ? kEpiThreads / 2 : kEpiThreads;
                const int sg = nseg > 1 ? etid / nthr : 0, gtid = etid - sg * nthr;
                if (gtid == 0) {
                    if (!wait_counter(d.tile_ctr + d_tile[sg], d_c[sg])) flag_error(p, 4, 900);   // all partials of the tile in
                    if (tr_main && sg == nseg - 1) FUSED_STAMP(p, 32, 6);
                }
                asm volatile("bar.sync %0, %1;" ::"r"(3 + sg), "r"(nthr) : "memory");
                const int c = d_c[sg];
                const DecodeModule& mo = d.mod[d_mod[sg]];
                const float* s_uw = reinterpret_cast<const float*>(epi + p.uw_off) + sg * p.BN * p.k * p.r;
                const int* s_idx = reinterpret_cast<const int*>(epi + p.idx_off) + sg * p.BN * p.k;
                if (c <= 1)
                    finish_tile<1, 4>(mo.y, mo.d_out, p.k, cpa, d_row0[sg], d.part_g, part_stride, d.units, M, upt, d_tile[sg], d_first[sg], c, d_q0[sg], d_nq[sg], ntok, d_slab[sg], s_uw, s_idx, gtid, nthr, routing_pending);
                else if (c <= 2)
                    finish_tile<2, 4>(mo.y, mo.d_out, p.k, cpa, d_row0[sg], d.part_g, part_stride, d.units, M, upt, d_tile[sg], d_first[sg], c, d_q0[sg], d_nq[sg], ntok, d_slab[sg], s_uw, s_idx, gtid, nthr, routing_pending);
                else if (c <= 4)
                    finish_tile<4, 4>(mo.y, mo.d_out, p.k, cpa, d_row0[sg], d.part_g, part_stride, d.units, M, upt, d_tile[sg], d_first[sg], c, d_q0[sg], d_nq[sg], ntok, d_slab[sg], s_uw, s_idx, gtid, nthr, routing_pending);
                else if (c <= 8)
                    finish_tile<8, 2>(mo.y, mo.d_out, p.k, cpa, d_row0[sg], d.part_g, part_stride, d.units, M, upt, d_tile[sg], d_first[sg], c, d_q0[sg], d_nq[sg], ntok, d_slab[sg], s_uw, s_idx, gtid, nthr, routing_pending);
                else
                    finish_tile<16, 1>(mo.y, mo.d_out, p.k, cpa, d_row0[sg], d.part_g, part_stride, d.units, M, upt, d_tile[sg], d_first[sg], c, d_q0[sg], d_nq[sg], ntok, d_slab[sg], s_uw, s_idx, gtid, nthr, routing_pending);
            } else {
                // More than two tiles (a range longer than a tile's units): one after the other with all epilogue
                // threads, the single staging buffer refilled with each tile's B rows.
                for (int sg = 0; sg < nseg; ++sg) {
                    const DecodeModule& mo = d.mod[d_mod[sg]];
                    epi_barrier();                                                   // the buffer's previous readers are done
                    stage_slab_rows(mo.B, mo.d_out, p.N, cpa, slab, d_row0[sg] + 4 * d_q0[sg], 4 * d_nq[sg], etid);
                    if (etid == 0) {
                        if (!wait_counter(d.tile_ctr + d_tile[sg], d_c[sg])) flag_error(p, 4, 900);
                        if (tr_main && sg == nseg - 1) FUSED_STAMP(p, 32, 6);
                    }
                    epi_barrier();
                    const int c = d_c[sg];
                    const float* s_uw = reinterpret_cast<const float*>(epi + p.uw_off) + sg * p.BN * p.k * p.r;
                    const int* s_idx = reinterpret_cast<const int*>(epi + p.idx_off) + sg * p.BN * p.k;
                    if (c <= 1)
                        finish_tile<1, 4>(mo.y, mo.d_out, p.k, cpa, d_row0[sg], d.part_g, part_stride, d.units, M, upt, d_tile[sg], d_first[sg], c, d_q0[sg], d_nq[sg], ntok, slab, s_uw, s_idx, etid, kEpiThreads, routing_pending);
                    else if (c <= 2)
                        finish_tile<2, 4>(mo.y, mo.d_out, p.k, cpa, d_row0[sg], d.part_g, part_stride, d.units, M, upt, d_tile[sg], d_first[sg], c, d_q0[sg], d_nq[sg], ntok, slab, s_uw, s_idx, etid, kEpiThreads, routing_pending);
                    else if (c <= 4)
                        finish_tile<4, 4>(mo.y, mo.d_out, p.k, cpa, d_row0[sg], d.part_g, part_stride, d.units, M, upt, d_tile[sg], d_first[sg], c, d_q0[sg], d_nq[sg], ntok, slab, s_uw, s_idx, etid, kEpiThreads, routing_pending);
                    else if (c <= 8)
                        finish_tile<8, 2>(mo.y, mo.d_out, p.k, cpa, d_row0[sg], d.part_g, part_stride, d.units, M, upt, d_tile[sg], d_first[sg], c, d_q0[sg], d_nq[sg], ntok, slab, s_uw, s_idx, etid, kEpiThreads, routing_pending);
                    else
                        finish_tile<16, 1>(mo.y, mo.d_out, p.k, cpa, d_row0[sg], d.part_g, part_stride, d.units, M, upt, d_tile[sg], d_first[sg], c, d_q0[sg], d_nq[sg], ntok, slab, s_uw, s_idx, etid, kEpiThreads, routing_pending);
                }
            }
            if (routing_pending) asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads + 32) : "memory");
            if (etid == 0 && tr_main) FUSED_STAMP(p, 32, 10);
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
    if (threadIdx.x == 0 && !counted_out) count_cta_out(d);
}

}  // namespace meteora
