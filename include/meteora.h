/*
 * meteora.h -- C ABI of the B200 (sm_100a) MeteoRA linear-layer forward.
 *
 * The layer (MeteoRA paper, Sec. 3.1, Eq. 2 and Eq. 3): every token x picks the k
 * of N embedded LoRA adapters with the highest gate logits G(x) = Wg x, weighs them
 * by a softmax over the k selected logits, and the output is
 *
 *     y = W0 x + sum_{i in topk(x)} w_i(x) * B_i (A_i x).
 *
 * Storage (all row-major, contiguous; the transposes of the paper's (n,d,r) and
 * (n,r,h) adapter tensors of Sec. 3.3 so that every contraction runs along the
 * contiguous axis):
 *     x[T,d_in]  W0[d_out,d_in]  A[N,r,d_in]  B[N,d_out,r]  Wg[N,d_in]  y[T,d_out]
 * in the element type named by meteora_shape_t::dtype (fp32, or bf16 with fp32
 * accumulation and a single rounding of y).  No bias anywhere.  The LoRA scale
 * alpha/r is folded into B by the caller (Eq. 1-2 carry no scale).
 *
 * Conventions for every entry point
 *   - All tensor arguments are DEVICE pointers owned by the caller, 16-byte aligned,
 *     unless an argument is explicitly marked "host".  The library allocates nothing,
 *     keeps no pointer after a call returns, launches on `stream` (a cudaStream_t cast
 *     to void*, NULL = default stream) and never synchronises, except where stated.
 *   - Return value: METEORA_OK (0) or a negative meteora_status_t.  Arguments are
 *     validated on the host before anything is launched; invalid arguments never reach
 *     the device.  There is no CPU fallback and no other backend.
 *   - Limits: 1 <= k <= METEORA_MAX_K, k <= N <= METEORA_MAX_N, 1 <= r <= METEORA_MAX_R,
 *     T >= 0 (T == 0 is a no-op), T*k < 2^31, temperature > 0.
 *   - Same inputs give bit-identical outputs from run to run (no floating-point atomics).
 *   - Behaviour for NaN/Inf inputs is undefined but memory-safe (indices stay < N).
 */
#ifndef METEORA_H_
#define METEORA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define METEORA_MAX_N 128
#define METEORA_MAX_K 8
#define METEORA_MAX_R 64
#define METEORA_STATIC_SCRATCH_FLOATS 65536 /* capacity of meteora_lora_delta_static: T * k * r may not exceed it */

typedef enum { METEORA_F32 = 0, METEORA_BF16 = 1 } meteora_dtype_t;

typedef enum {
    METEORA_OK = 0,
    METEORA_ERR_INVALID_ARG = -1,         /* null pointer, non-positive size, k > N, temperature <= 0 ... */
    METEORA_ERR_UNSUPPORTED_SHAPE = -2,   /* a limit above is exceeded */
    METEORA_ERR_MISALIGNED = -3,          /* a base pointer is not 16-byte aligned */
    METEORA_ERR_WORKSPACE_TOO_SMALL = -4, /* workspace_bytes < meteora_workspace_bytes(shape) */
    METEORA_ERR_CUDA = -5,                /* a CUDA runtime/driver call or a launch failed */
    METEORA_ERR_TIMEOUT = -6              /* a bounded device-side wait expired (see meteora_workspace_status) */
} meteora_status_t;

typedef struct {
    int T;               /* tokens (batch * sequence; tokens are independent, Sec. 3.3) */
    int d_in;            /* input width  (paper: d) */
    int d_out;           /* output width (paper: h) */
    int N;               /* embedded adapters (paper: n) */
    int r;               /* LoRA rank */
    int k;               /* adapters selected per token */
    meteora_dtype_t dtype;
    float temperature;   /* divides the selected logits before the softmax (App. A.5); 1.0f = Eq. 3 as written */
} meteora_shape_t;

/*
 * Gate, selection and weights (Sec. 3.1: G(x) = Wg x, the k highest logits form I(x);
 * Eq. 3: softmax over the selected logits; App. A.1: k = 1 gives weight exactly 1).
 *   x[T,d_in], Wg[N,d_in] in shape->dtype.  d_out and r of the shape are ignored.
 *   topk_idx[T,k] int32: adapters by descending logit; equal logits keep the lower index first.
 *   topk_w[T,k]   fp32 : the matching weights.
 *   logits[T,N]   fp32 : optional (may be NULL).
 * Logits are accumulated in fp32.
 */
int meteora_gate_topk(const void* x, const void* Wg, const meteora_shape_t* shape, int32_t* topk_idx,
                      float* topk_w, float* logits, void* stream);

/*
 * Token -> adapter grouping (Sec. 3.3: the tokens that picked adapter i are gathered into one
 * group per adapter).  Slot s = t*k + j has key topk_idx[s].
 *   counts[N]    : slots per adapter.
 *   offsets[N+1] : exclusive prefix sum of counts.
 *   perm[T*k]    : slot numbers sorted by key, equal keys in ascending slot order (stable); the
 *                  group of adapter e is perm[offsets[e] .. offsets[e+1]).
 * Pure integer work; bit-exact.  Keys outside [0,N) are out of contract (clamped on the device).
 */
int meteora_route(const int32_t* topk_idx, int T, int k, int N, int32_t* counts, int32_t* offsets,
                  int32_t* perm, void* stream);

/*
 * The LoRA term of Eq. 2 alone, for a given routing:
 *   delta[t,:] = sum_j topk_w[t,j] * B[topk_idx[t,j]] (A[topk_idx[t,j]] x[t]).
 * The shrink (x A_i) runs adapter by adapter over the grouped slots (offsets, perm from
 * meteora_route), the expand and weighted sum run token by token.
 *   delta[T,d_out] fp32.  workspace: device scratch of at least meteora_workspace_bytes(shape).
 */
int meteora_lora_delta(const void* x, const void* A, const void* B, const int32_t* topk_idx,
                       const float* topk_w, const int32_t* offsets, const int32_t* perm,
                       const meteora_shape_t* shape, float* delta, void* workspace, size_t workspace_bytes,
                       void* stream);

/*
 * meteora_lora_delta without a workspace.  (The paper has no counterpart: this entry point exists for the
 * way the library is embedded, not for the method.)
 *
 * Who it is for: callers that cannot allocate device memory at the point where they need the LoRA term,
 * and so have no workspace to pass: code running while another framework holds its allocator lock,
 * serving loops whose memory pool is frozen after start-up, bindings that can launch but not allocate.  The scratch that meteora_lora_delta takes from its workspace (the shrunk activations, T*k*r
 * floats) lives here in a fixed device array inside the library, METEORA_STATIC_SCRATCH_FLOATS floats
 * (256 KB) on every GPU that loads the library, for the life of the process.  The call allocates nothing
 * and frees nothing.
 *
 * Arguments, layouts and result are those of meteora_lora_delta (inputs and delta[T,d_out] fp32 are still
 * the caller's).  Differences:
 *   - T * k * r > METEORA_STATIC_SCRATCH_FLOATS returns METEORA_ERR_UNSUPPORTED_SHAPE and launches nothing;
 *     larger problems need meteora_lora_delta and a workspace.
 *   - The first call on each device looks up the device address of the built-in array (a runtime query,
 *     with that device current; it may make the runtime load the module, which can allocate driver memory
 *     and synchronise).  Make that first call at start-up, in a warm-up step: outside any stream capture
 *     and outside the region in which allocation is forbidden.  Later calls on that device only launch.
 *   - `stream` must belong to the device that is current when the call is made: the array's address is
 *     looked up for the current device.
 *   - All calls on a device share the one array and it keeps whatever the previous call left in it.  No
 *     part of it needs clearing (every value is written before it is read within a call), but two calls
 *     whose kernels can overlap on the GPU (different streams, no ordering between them) race on it: keep
 *     calls on one device ordered.
 */
int meteora_lora_delta_static(const void* x, const void* A, const void* B, const int32_t* topk_idx,
                              const float* topk_w, const int32_t* offsets, const int32_t* perm,
                              const meteora_shape_t* shape, float* delta, void* stream);

/*
 * The whole layer, Eq. 2 with Eq. 3: gate, top-k, softmax over the selected, base product,
 * gate-weighted LoRA sum, one rounding of y.
 *   y[T,d_out] in shape->dtype.  workspace: device scratch of at least
 *   meteora_workspace_bytes(shape); calls that share a workspace must not overlap in time.
 * After the call the workspace holds the routing that was used (meteora_workspace_routing).
 * bf16 shapes with d_in % 8 == 0 and r % 8 == 0 run on the tensor-core paths (TMA + tcgen05):
 * decode batches (T <= 256, rank a multiple of 8 whose staged rows of B fit shared memory) as ONE cooperative
 * kernel launch in which the CTAs exchange partial results through the workspace, everything else as three launches
 * (stacked shrink [A; Wg] x, selection, base product with the LoRA expand; for prefill batches of
 * ranks that are multiples of 8 on pairs of SMs with two-CTA MMAs).  A bf16 layer whose rank is no multiple of 8 takes the same
 * paths with A and B zero-padded to the next multiple of 8 inside the workspace (rewritten by every call).  Every other shape
 * runs on a plain CUDA-core path with the same results up to rounding order.  The workspace header
 * must have been zeroed once (meteora_workspace_init) before its first use; the kernels leave it
 * ready for the next call.  meteora_describe_plan tells which path a shape takes.
 */
int meteora_linear_forward(const void* x, const void* W0, const void* A, const void* B, const void* Wg,
                           const meteora_shape_t* shape, void* y, void* workspace, size_t workspace_bytes,
                           void* stream);

/*
 * Several MeteoRA linears that read the SAME x (Sec. 3.2: every linear of a decoder block carries its own gate
 * and adapters; q/k/v share their input, gate/up share theirs), Eq. 2 with Eq. 3 for each of them:
 *   y[m][T, d_out[m]] = W0[m] x + sum over module m's own top-k picks.
 * W0, A, B, Wg, y are HOST arrays of n_modules DEVICE pointers (1 <= n_modules <= METEORA_MAX_GROUP), d_out a host
 * array; T, d_in, N, r, k, dtype, temperature come from `shape` (its d_out is ignored).  Results per module are
 * those of meteora_linear_forward up to the rounding order of fp32 sums.  Decode batches (T <= 256, rank a
 * multiple of 8, bf16, all modules together at most about 120 row tiles of 128) run as ONE kernel launch for the whole group;
 * anything else runs module by module.  workspace: meteora_group_workspace_bytes(shape, d_out, n_modules) bytes of
 * device memory, its first 4 KB zeroed once (meteora_workspace_init); meteora_workspace_status reads the group's
 * status word.  meteora_group_workspace_routing returns where module `module` left its routing;
 * meteora_group_plan returns 1 if the group runs as one launch, 0 if module by module, or an error code.
 */
#define METEORA_MAX_GROUP 4
size_t meteora_group_workspace_bytes(const meteora_shape_t* shape, const int* d_out, int n_modules);
int meteora_group_plan(const meteora_shape_t* shape, const int* d_out, int n_modules);
int meteora_group_workspace_routing(const meteora_shape_t* shape, const int* d_out, int n_modules, int module,
                                    void* workspace, int32_t** topk_idx, float** topk_w);
int meteora_linear_forward_group(const void* x, const void* const* W0, const void* const* A, const void* const* B,
                                 const void* const* Wg, const int* d_out, int n_modules,
                                 const meteora_shape_t* shape, void* const* y, void* workspace,
                                 size_t workspace_bytes, void* stream);

/*
 * Gradient of the gate weights (Sec. 3.2: the base model and the adapters stay fixed, only the gating networks
 * are trained; with top-k > 1 the token loss reaches them through the weights of Eq. 3).  Given dy = dL/dy
 * [T,d_out] (shape->dtype) and the routing a forward left (topk_idx, topk_w; meteora_workspace_routing):
 *   g[t,j]      = < dy[t], B_e (A_e x[t]) >,  e = topk_idx[t,j]
 *   dlogit[t,j] = topk_w[t,j] * (g[t,j] - sum_m topk_w[t,m] g[t,m]) / temperature
 *   dWg[e,:]    = sum over the slots (t,j) that picked e of dlogit[t,j] * x[t]          fp32 [N,d_in], overwritten
 * Adapters nobody picked get a zero row; top-1 gives all zeros (the weight is the constant 1, App. A.1).  The
 * cross-entropy term of the gate loss (Eq. 4) is the caller's: it needs labels this library does not see.
 * dlogit: optional fp32 [T,k] output (may be null).  fp32 accumulation, sums in a fixed order (bit-identical
 * from run to run).  workspace: device scratch of meteora_gate_backward_workspace_bytes(shape) bytes; it may be
 * the forward's workspace once its routing has been copied out or is passed here as topk_idx / topk_w from a
 * DIFFERENT buffer (the call overwrites the start of the workspace).
 */
size_t meteora_gate_backward_workspace_bytes(const meteora_shape_t* shape);
int meteora_gate_backward(const void* x, const void* A, const void* B, const void* dy, const int32_t* topk_idx,
                          const float* topk_w, const meteora_shape_t* shape, float* dlogit, float* dWg,
                          void* workspace, size_t workspace_bytes, void* stream);

/*
 * Zero-padding of the adapters' rank to the next multiple of 8, made ONCE instead of by every forward: a bf16 layer
 * whose rank is no multiple of 8 (rank 4, say) runs on the tensor-core paths with A and B padded, and
 * meteora_linear_forward pads them into its workspace on every call.  The adapters are fixed (Sec. 3.2), so a
 * caller pads them once: A_pad[N, r8, d_in] and B_pad[N, d_out, r8] (bf16, device memory owned by the caller, 16-byte
 * aligned, *a_bytes and *b_bytes from meteora_pad_adapters_bytes, which returns r8 = the padded rank, or 0 where
 * the shape needs no padding or is invalid), then calls the forward with shape->r = r8 and the padded arrays: the
 * added rank entries are zero in A (rows) and in B (columns), so y, the routing and every sum are bit-identical.
 * Asynchronous on `stream`; reads N, r, d_in, d_out and dtype of the shape.
 */
int meteora_pad_adapters_bytes(const meteora_shape_t* shape, size_t* a_bytes, size_t* b_bytes);
int meteora_pad_adapters(const void* A, const void* B, const meteora_shape_t* shape, void* A_pad, void* B_pad,
                         void* stream);

/*
 * The same gradient with the adapters' B matrices transposed beforehand.  The adapters are fixed while the gates
 * train (Sec. 3.2), so Bt[n, p, o] = B[n, o, p] (shape->dtype, [N, r, d_out], device memory of
 * meteora_adapters_bt_bytes(shape) bytes, 16-byte aligned, owned by the caller) is made once per module with
 * meteora_transpose_adapters_b (asynchronous on `stream`; only N, d_out, r and dtype of the shape are read) and
 * every step then calls meteora_gate_backward_bt, which is meteora_gate_backward without its transposition of B
 * (same arguments, results bit-identical to it, same workspace size).
 */
size_t meteora_adapters_bt_bytes(const meteora_shape_t* shape);
int meteora_transpose_adapters_b(const void* B, const meteora_shape_t* shape, void* Bt, void* stream);
int meteora_gate_backward_bt(const void* x, const void* A, const void* Bt, const void* dy, const int32_t* topk_idx,
                             const float* topk_w, const meteora_shape_t* shape, float* dlogit, float* dWg,
                             void* workspace, size_t workspace_bytes, void* stream);

/*
 * Same as meteora_linear_forward with the activations in HOST memory: x_host[T,d_in] is copied to
 * the device, the layer runs, y_host[T,d_out] is copied back, all on `stream` (pinned host memory
 * makes the copies asynchronous).  Weights and workspace stay device pointers.  The call does not
 * synchronise: y_host is valid once `stream` has been synchronised by the caller.
 */
int meteora_linear_forward_host(const void* x_host, const void* W0, const void* A, const void* B,
                                const void* Wg, const meteora_shape_t* shape, void* y_host, void* workspace,
                                size_t workspace_bytes, void* stream);

/* Upper bound of the scratch any of the calls above needs for this shape (0 on invalid shape). */
size_t meteora_workspace_bytes(const meteora_shape_t* shape);

/*
 * Where meteora_linear_forward left its routing inside `workspace`: *topk_idx -> int32[T,k],
 * *topk_w -> fp32[T,k] (device pointers into the workspace; valid until the workspace is reused).
 */
int meteora_workspace_routing(const meteora_shape_t* shape, void* workspace, int32_t** topk_idx, float** topk_w);

/*
 * Clears the 4 KB header of a freshly allocated workspace (status words and the counters the
 * single-launch decode kernel synchronises on), asynchronously on `stream`.  Call once before the
 * workspace's first use; memory that is already zero needs no call.
 */
int meteora_workspace_init(void* workspace, void* stream);

/*
 * Reads the workspace's device status word (SYNCHRONISES `stream`): METEORA_OK, or
 * METEORA_ERR_TIMEOUT if a bounded wait inside a kernel (an mbarrier of the TMA/tensor-core
 * pipeline, or a counter another CTA of the decode kernel bumps) gave up, in which case the
 * outputs of that call are invalid.  The word is cleared; after a timeout call
 * meteora_workspace_init again before the workspace's next use (the counters may be mid-count).
 */
int meteora_workspace_status(void* workspace, void* stream);

/*
 * Timing of the base-product launch (the dominant kernel of the three-launch path) for roofline
 * reports.  Between meteora_profile_begin and meteora_profile_end every meteora_linear_forward
 * that takes the three-launch tensor-core path
 * records a CUDA event pair around that one launch on the caller's stream (up to max_launches
 * pairs; the launch is not overlapped with its predecessor while timed).  meteora_profile_end
 * SYNCHRONISES on the recorded events and returns the summed kernel time and the launch count.
 * The events are created on first use and kept for the life of the process; not thread-safe; not
 * to be used during stream capture.
 */
int meteora_profile_begin(int max_launches);
int meteora_profile_end(float* total_ms, int* launches);

/*
 * Writes a one-line description of how meteora_linear_forward will run this shape (path, launches,
 * CTAs, split factor, tile, ring depth) into buf, followed by the number of single-launch decode
 * kernels the driver has refused so far in this process.  Host-only; for logs and benchmark records.
 */
int meteora_describe_plan(const meteora_shape_t* shape, char* buf, size_t buf_bytes);

/*
 * Tuning knobs for measurements (process-wide, not thread-safe; 0 = automatic unless stated):
 *   "splits"         split-K cluster size of the three-launch base product (1, 2, 4, 8); main CTAs
 *                    per 128-row tile of the decode kernel
 *   "stages"         TMA ring depth
 *   "tile_tokens"    tokens per tile of the three-launch path
 *   "kc"             64-element k-chunks fetched per TMA copy: 1, 2 or 4
 *   "zmax"           cap on the contraction slices of the stacked shrink
 *   "stacked_direct" 1 = decode-batch stacked shrink without clusters
 *   "simt_expand"    1 = LoRA expand of the three-launch path on CUDA cores even for rank 8
 *   "no_tma_store"   1 = plain stores of y where the TMA store would apply
 *   "force_simt"     1 = never take a tensor-core path
 *   "pdl"            default 1 = the three launches of a call overlap by programmatic dependent launch
 *   "fused"          default 1; 0 = never use the single-launch decode kernel; 2 = also where the planner
 *                    prefers the three launches (layers with several row tiles per CTA below 32 tokens)
 *   "coop"           default 1; 0 = launch the decode kernel without the co-residency guarantee
 *   "unit_split"     decode kernel's main CTAs: 0 = planner's choice, 1 = even unit ranges over all free SMs,
 *                    2 = whole row tiles per group of CTAs (falls back to the choice that fits)
 *   "aux_ctas"       > 0 = how many CTAs of the decode kernel the stacked shrink and the selection may take
 *   "no_hold"        head start of the decode kernel's aux CTAs: 0 = planner's choice (1800 ns for layers below
 *                    40 MB, none above), 1 = none, 64 = main CTAs wait for a counter, other = nanoseconds
 *   "hold_after"     ring stages of W0 the decode kernel's main CTAs request before that head start: 0 = planner's
 *                    choice (one stage for layers of 20 to 40 MB, none otherwise), -1 = none, n > 0 = n stages
 *   "narrow_select"  selection inside the decode kernel: 0 = by batch size (from 16 tokens up the logits are read
 *                    first and then only the picks' shrink values, below that the whole stacked row at once),
 *                    1 = always the former, -1 = always the latter; same results bit for bit
 *   "pdl_decode"     default 1 = the decode kernel is launched with programmatic stream serialization on top of
 *                    the co-residency guarantee: the next launch is processed and its CTAs set up under this
 *                    kernel's tail (the kernel touches no global memory before the launch ahead of it has
 *                    completed); 0 = plain stream order.  If the driver refuses the pair of attributes
 *                    the kernel is launched without it (pdl_decode_refused in the plan string counts these).
 *   "pair"           default 1 = prefill base product on pairs of SMs (two-CTA MMA, 256 x 256 tiles)
 *                    where the pairs cover a quarter of the SMs; 0 = never; 2 = wherever the shape allows
 *   "stream"         decode batches up to 128 tokens on the streamed one-launch kernel: default 1 = planner's
 *                    choice of one or two CTAs per SM, 0 = never (the cooperative kernel takes them), 2 = always one
 *                    CTA per SM with a deep ring, 3 = two per SM wherever they fit
 *   "pf"             L2 prefetch of the weights beyond the streamed kernel's ring: default 0 / -1 = none, n > 0 = cap in MB
 *   "own_local"      default 1 = a CTA's own row slice of its partial tile stays in shared memory; 0 = through scratch
 *   "bulk_deliver"   1 = the partial tiles leave through shared memory and bulk copies instead of plain stores
 *   "aux_plain"      default 1 = the stacked shrink's partial tiles leave the aux CTAs as plain stores; 0 = staged in
 *                    shared memory and sent as one bulk copy each
 *   "pair_decode"    streamed kernel on pairs of CTAs (two-CTA MMA, half a token tile each): default 0 = never,
 *                    1 = from 64 tokens up, 2 = from 17 tokens up
 *   "cluster_decode" decode batches on the clustered one-launch kernel (the CTAs of a row tile exchange their partial
 *                    tiles through distributed shared memory, the stacked shrink is spread over all CTAs):
 *                    default 0 = never (measured slower than the streamed kernel except for the largest layers),
 *                    other = wherever the device can hold all clusters at once
 *   "group_pairs"    > 0 = row pairs per scheduling group of the prefill kernel on pairs of SMs (0 = planner's choice)
 *   "tail_carve"     prefill on pairs of SMs: 0 = the planner carves the tiles of a nearly empty last wave out of the
 *                    pair launch (they follow as a launch of small tiles), -1 = never, n > 0 = the last token tile of n row pairs
 *   "wait_limit_us"  > 0 = limit of every bounded device-side wait in microseconds (0 = the default of about a second)
 * Unknown names return METEORA_ERR_INVALID_ARG.  The defaults are what the benchmarks measure.
 */
int meteora_set_tuning(const char* name, int value);

const char* meteora_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* METEORA_H_ */
