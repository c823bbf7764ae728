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
// Warp roles (192 threads): warp 0 lane 0 issues TMA loads into a ring of shared-memory stages, warp 1
// owns the TMEM allocation and lane 0 issues tcgen05.mma, warps 2-5 run the epilogue (TMEM lane quarter
// = warp id % 4).  Every mbarrier wait is bounded; on expiry the kernel records it in the status word
// and drains instead of hanging.
#include <cuda.h>

#include <mutex>
#include <vector>

#include "common.cuh"

namespace meteora {

constexpr int kBM = 128;       // weight rows per tile (UMMA M)
constexpr int kBK = 64;        // contraction elements per stage: one 128-byte swizzled row of bf16
constexpr int kUmmaK = 16;     // contraction elements per tcgen05.mma (32 bytes of bf16)
constexpr int kThreads = 192;
constexpr int kEpiThreads = 128;
constexpr int kWTileBytes = kBM * kBK * 2;
constexpr long long kWaitLimitCycles = 2000000000LL;  // about a second

enum { MODE_STACKED = 0, MODE_LORA = 1 };

struct WGemmParams {
    int T, K;            // tokens, contraction length
    int BN;              // tokens per tile (multiple of 16, <= 256)
    int splits;          // cluster size along the contraction axis
    int ksteps;          // ceil(K / kBK)
    int stages;          // depth of the TMA ring
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
    int32_t* status;
    int pdl_wait;        // epilogue waits for the preceding grid before reading its results
    int pdl_trigger;     // let the dependent grid start as soon as this one is resident
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
// Bounded wait: false if the phase did not complete within kWaitLimitCycles.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try(bar, parity)) return true;
        if ((spin & 0x3FF) == 0 && clock64() - t0 > kWaitLimitCycles) return false;
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"((uint64_t)tm), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
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
__device__ __forceinline__ float ld_peer_f32(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
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
// Instruction descriptor: fp32 accumulate, bf16 x bf16, both operands K-major, M = 128, N = bn.
__device__ __forceinline__ uint32_t instr_desc_bf16(int bn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}

// ------------------------------------------------------------------------------------------------
// Epilogue of one accumulator element: row of the launch's row space, token index, fp32 sum.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void finish_element(const WGemmParams& p, int tile_m, int row_in_tile, int token,
                                               float acc) {
    if (token >= p.T) return;
    if (p.mode == MODE_STACKED) {
        int row, col;
        if (tile_m < p.split_tile) {
            row = tile_m * kBM + row_in_tile;
            if (row >= p.rows0) return;
            col = row;
        } else {
            row = (tile_m - p.split_tile) * kBM + row_in_tile;
            if (row >= p.rows1) return;
            col = p.col1 + row;
        }
        p.u_all[(size_t)token * p.ld_u + col] = acc;
    } else {
        const int o = tile_m * kBM + row_in_tile;
        if (o >= p.d_out) return;
        const int32_t* ti = p.topk_idx + (size_t)token * p.k;
        const float* uq = p.uw + (size_t)token * p.k * p.r;
        for (int j = 0; j < p.k; ++j) {
            const int e = min(max(__ldg(ti + j), 0), p.N - 1);
            const __nv_bfloat16* brow = p.B + ((size_t)e * p.d_out + o) * p.r;
            for (int q = 0; q < p.r; q += 8) {
                float bv[8];
                load8(brow + q, bv);
                const float4 u0 = __ldg(reinterpret_cast<const float4*>(uq + j * p.r + q));
                const float4 u1 = __ldg(reinterpret_cast<const float4*>(uq + j * p.r + q + 4));
                acc = fmaf(bv[0], u0.x, acc); acc = fmaf(bv[1], u0.y, acc);
                acc = fmaf(bv[2], u0.z, acc); acc = fmaf(bv[3], u0.w, acc);
                acc = fmaf(bv[4], u1.x, acc); acc = fmaf(bv[5], u1.y, acc);
                acc = fmaf(bv[6], u1.z, acc); acc = fmaf(bv[7], u1.w, acc);
            }
        }
        p.y[(size_t)token * p.d_out + o] = __float2bfloat16_rn(acc);
    }
}

__global__ void __launch_bounds__(kThreads)
k_wgemm(const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
        const __grid_constant__ CUtensorMap tmX, const WGemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;                 // 1024-byte aligned for the 128-byte swizzle
    uint8_t* ring_ptr = smem_raw + (ring - raw);
    const uint32_t stage_bytes = kWTileBytes + p.BN * 128;
    const uint32_t ring_bytes = p.stages * stage_bytes;
    const uint32_t bar_base = ring + ring_bytes;                 // full[stages], empty[stages], acc (8 bytes each)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ring_ptr + ring_bytes + (2 * p.stages + 1) * 8);
    const uint32_t bar_acc = bar_base + 2 * p.stages * 8;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = p.splits;
    const int split = (int)cluster_rank();
    const int tile_m = blockIdx.x / S;
    const int tok0 = blockIdx.y * p.BN;
    const int ks0 = (int)(((long long)p.ksteps * split) / S);
    const int ks1 = (int)(((long long)p.ksteps * (split + 1)) / S);
    const int nks = ks1 - ks0;

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
            const int row0 = (second ? tile_m - p.split_tile : tile_m) * kBM;
            int issued = 0;
            bool ok = true;
            for (int i = 0; i < nks && ok; ++i) {
                const int s = i % p.stages, round = i / p.stages;
                if (round > 0) ok = mbar_wait(bar_base + (p.stages + s) * 8, (round & 1) ^ 1);
                if (!ok) break;
                const uint32_t full = bar_base + s * 8;
                const uint32_t dst = ring + s * stage_bytes;
                mbar_expect_tx(full, stage_bytes);
                tma_load_2d(dst, tmW, (ks0 + i) * kBK, row0, full);
                tma_load_2d(dst + kWTileBytes, &tmX, (ks0 + i) * kBK, tok0, full);
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
            for (int i = 0; i < nks; ++i) {
                const int s = i % p.stages, round = i / p.stages;
                ok = mbar_wait(bar_base + s * 8, round & 1);
                if (!ok) break;
                tc_fence_after();
                const uint32_t wa = ring + s * stage_bytes;
                const uint64_t da = smem_desc_sw128(wa), db = smem_desc_sw128(wa + kWTileBytes);
#pragma unroll
                for (int kk = 0; kk < kBK / kUmmaK; ++kk)
                    umma_bf16(tmem_base, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (i | kk) != 0);
                umma_commit(bar_base + (p.stages + s) * 8);   // stage reusable once these MMAs have read it
            }
            umma_commit(bar_acc);                              // accumulators complete
            if (!ok) {
                atomicExch(p.status, 1);
                atomicExch(p.status + 2, 200);
            }
        }
    }
    __syncwarp();

    // ---------------------------------------------------------------------- epilogue
    const bool epi = warp >= 2;
    const int quad = warp & 3;                    // TMEM lanes 32*quad .. 32*quad+31 belong to this warp
    const int etid = threadIdx.x - 64;            // 0..127 among the epilogue threads
    bool acc_ok = true;
    if (epi) {
        if (p.pdl_wait) asm volatile("griddepcontrol.wait;" ::: "memory");
        if (nks > 0) {
            acc_ok = mbar_wait(bar_acc, 0);
            if (!acc_ok && lane == 0) {
                atomicExch(p.status, 1);
                atomicExch(p.status + 3, 300);
            }
        }
        acc_ok = __all_sync(0xFFFFFFFFu, acc_ok);   // keep the warp-collective TMEM loads convergent
        tc_fence_after();
    }

    if (S == 1) {
        if (epi) {
            const int row_in_tile = quad * 32 + lane;
            for (int c = 0; c < p.BN; c += 16) {
                float v[16];
                if (nks > 0 && acc_ok) {
                    tmem_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + c, v);
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = 0.f;
                }
                if (acc_ok) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) finish_element(p, tile_m, row_in_tile, tok0 + c + i, v[i]);
                }
            }
        }
    } else {
        // Partial accumulators go to shared memory (the ring is idle now: every load has landed and every
        // MMA that read it has completed), then each CTA of the cluster sums one slice of the 128 rows
        // over all partials, in rank order, reading its peers through distributed shared memory.
        float* part = reinterpret_cast<float*>(ring_ptr);          // part[t][row], row fastest
        if (epi) {
            const int row_in_tile = quad * 32 + lane;
            for (int c = 0; c < p.BN; c += 16) {
                float v[16];
                if (nks > 0 && acc_ok) {
                    tmem_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + c, v);
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = 0.f;
                }
#pragma unroll
                for (int i = 0; i < 16; ++i) part[(c + i) * kBM + row_in_tile] = v[i];
            }
        }
        cluster_sync();
        if (epi && acc_ok) {
            const int lo = (kBM * split) / S, hi = (kBM * (split + 1)) / S;
            const int nrows = hi - lo;
            const int items = nrows * p.BN;
            for (int it = etid; it < items; it += kEpiThreads) {
                const int t = it / nrows, rl = it - t * nrows;
                const uint32_t addr = ring + (uint32_t)((t * kBM + lo + rl) * 4);
                float acc = 0.f;
                for (int q = 0; q < S; ++q) acc += ld_peer_f32(addr, (uint32_t)q);
                finish_element(p, tile_m, lo + rl, tok0 + t, acc);
            }
        }
        cluster_sync();   // nobody leaves while a peer may still read its partials
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                     "r"((uint32_t)p.tmem_cols)
                     : "memory");
    }
}

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
    int K, rows, box_rows;
    bool operator==(const MapKey& o) const {
        return ptr == o.ptr && K == o.K && rows == o.rows && box_rows == o.box_rows;
    }
};
struct MapEntry {
    MapKey key;
    CUtensorMap map;
};

// A [rows, K] row-major bf16 matrix as a 2-D tensor map whose box is kBK (128 bytes) x box_rows, 128-byte
// swizzled; out-of-range rows and columns read as zero.  Encoded maps are cached by (pointer, shape).
static int get_tensor_map(const void* ptr, int K, int rows, int box_rows, CUtensorMap* out) {
    static std::mutex mu;
    static std::vector<MapEntry> cache;
    static size_t next_evict = 0;
    const MapKey key{ptr, K, rows, box_rows};
    std::lock_guard<std::mutex> lock(mu);
    for (const MapEntry& e : cache)
        if (e.key == key) {
            *out = e.map;
            return METEORA_OK;
        }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return METEORA_ERR_CUDA;
    const cuuint64_t gdim[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
    const cuuint32_t estride[2] = {1, 1};
    MapEntry e;
    e.key = key;
    const CUresult r = fn(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstride, box,
                          estride, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
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

struct Plan {
    int BN, n_tiles, splits, stages, tmem_cols;
    size_t smem;
};

static Plan make_plan(int row_tiles, int T, int K) {
    const Tuning& tn = tuning();
    Plan pl;
    const int ksteps = (K + kBK - 1) / kBK;
    int bn = tn.tile_tokens > 0 ? tn.tile_tokens : (T <= 256 ? (T + 15) / 16 * 16 : 256);
    bn = std::min(256, std::max(16, (bn + 15) / 16 * 16));
    pl.BN = bn;
    pl.n_tiles = (T + bn - 1) / bn;
    const int tiles = row_tiles * pl.n_tiles;
    int splits = tn.splits > 0 ? tn.splits : std::max(1, sm_count() / tiles);
    splits = std::min(std::min(splits, 8), ksteps);
    pl.splits = splits;
    const int nks = (ksteps + splits - 1) / splits;
    const size_t stage_bytes = kWTileBytes + (size_t)bn * 128;
    const size_t budget = (splits == 1 && tiles > sm_count()) ? 98 * 1024 : 200 * 1024;  // two CTAs per SM when tiles queue up
    int stages = tn.stages > 0 ? tn.stages : (int)std::min<size_t>((size_t)nks, budget / stage_bytes);
    stages = std::max(stages, 2);
    if (splits > 1)   // the partial accumulators (bn * 512 bytes) are parked in the idle ring
        while ((size_t)stages * stage_bytes < (size_t)bn * 512) ++stages;
    pl.stages = stages;
    int cols = 32;
    while (cols < bn) cols *= 2;
    pl.tmem_cols = cols;
    pl.smem = 1024 + (size_t)stages * stage_bytes + (2 * stages + 1) * 8 + 16;
    return pl;
}

static int launch_wgemm(const CUtensorMap& m0, const CUtensorMap& m1, const CUtensorMap& mx, WGemmParams& p,
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
    cfg.gridDim = dim3(row_tiles * pl.splits, pl.n_tiles);
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
    return cuda_status(cudaLaunchKernelEx(&cfg, k_wgemm, m0, m1, mx, p));
}

static void fill_common(WGemmParams& p, const Plan& pl, int T, int K, int32_t* status) {
    p.T = T;
    p.K = K;
    p.BN = pl.BN;
    p.splits = pl.splits;
    p.ksteps = (K + kBK - 1) / kBK;
    p.stages = pl.stages;
    p.tmem_cols = pl.tmem_cols;
    p.status = status;
}

int launch_stacked_shrink_tc(const void* x, const void* A, const void* Wg, const meteora_shape_t& s,
                             const Workspace& ws, cudaStream_t st) {
    const int a_rows = s.N * s.r;
    const int a_tiles = (a_rows + kBM - 1) / kBM;
    const int row_tiles = a_tiles + 1;
    const Plan pl = make_plan(row_tiles, s.T, s.d_in);
    CUtensorMap mA, mG, mX;
    int rc;
    if ((rc = get_tensor_map(A, s.d_in, a_rows, kBM, &mA)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(Wg, s.d_in, s.N, kBM, &mG)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(x, s.d_in, s.T, pl.BN, &mX)) != METEORA_OK) return rc;
    WGemmParams p = {};
    fill_common(p, pl, s.T, s.d_in, ws.status);
    p.split_tile = a_tiles;
    p.rows0 = a_rows;
    p.rows1 = s.N;
    p.mode = MODE_STACKED;
    p.u_all = ws.u_all;
    p.ld_u = ws.ld_u;
    p.col1 = ws.col_logits;
    p.pdl_wait = 0;
    p.pdl_trigger = tuning().pdl ? 1 : 0;
    return launch_wgemm(mA, mG, mX, p, row_tiles, pl, false, st);
}

int launch_base_lora_tc(const void* x, const void* W0, const void* B, const meteora_shape_t& s, const Workspace& ws,
                        void* y, bool pdl, cudaStream_t st) {
    const int row_tiles = (s.d_out + kBM - 1) / kBM;
    const Plan pl = make_plan(row_tiles, s.T, s.d_in);
    CUtensorMap mW, mX;
    int rc;
    if ((rc = get_tensor_map(W0, s.d_in, s.d_out, kBM, &mW)) != METEORA_OK) return rc;
    if ((rc = get_tensor_map(x, s.d_in, s.T, pl.BN, &mX)) != METEORA_OK) return rc;
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
    return launch_wgemm(mW, mW, mX, p, row_tiles, pl, pdl, st);
}

}  // namespace meteora
