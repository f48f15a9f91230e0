/*
 * linfusion_attn.h — C ABI of the B200 (sm_100a) normalized non-causal linear attention.
 *
 * The operation is the token mixer of the LinFusion module (Sec. 2.3, Prop. 2 / Prop. 3,
 * with the normalization of Sec. 2.2 / Eq. 5 in its non-causal form).  For every
 * (batch, head) slab, with Q = f'(X), K = g'(X), V = X W_V already computed by the caller:
 *
 *     S   = sum_j phi(K_j)^T V_j          d x d state      (g'(X)^T X of Prop. 2)
 *     z   = sum_j phi(K_j)                1 x d normalizer (Z of Eq. 5, scan replaced by the sum)
 *     Y_i = phi(Q_i) S / (phi(Q_i) . z + eps)
 *
 * phi is the non-negative activation of Sec. 2.2 (the paper gives no closed form; this
 * library implements phi(x) = elu(x) + 1, and the identity for callers whose features are
 * already non-negative).  eps is this library's guard on the denominator; the paper has none.
 *
 * Unless a function says otherwise, tensor arguments are DEVICE pointers to dense row-major
 * bf16 (or fp16: LINFUSION_DTYPE_FP16) [B, H, N, d] (token rows of d contiguous channels, one slab of N rows per (b, h)),
 * 16-byte aligned.  Y must not overlap Q, K or V.  The caller owns Q, K, V, Y and the stream.
 * The handle owns an fp32 workspace on its device unless the caller lends one (set_workspace).
 *
 * Every function returns a status code; nothing throws or aborts across this boundary.
 * forward() only enqueues work on the given stream and returns without synchronizing; it
 * allocates nothing.  Results are bit-identical from call to call for identical inputs
 * (fixed split of N, fixed summation order, no floating-point atomics).
 * One forward may be in flight per handle at a time (the workspace is shared).
 */
#ifndef LINFUSION_ATTN_H
#define LINFUSION_ATTN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct linfusion_attn linfusion_attn_t; /* opaque handle */

typedef enum {
    LINFUSION_OK = 0,
    LINFUSION_ERR_INVALID_ARG = 1, /* null / misaligned pointer, non-positive size, bad eps   */
    LINFUSION_ERR_UNSUPPORTED = 2, /* head dim, phi, flags or device this build cannot serve  */
    LINFUSION_ERR_ALLOC = 3,       /* device workspace could not be allocated / is too small   */
    LINFUSION_ERR_CUDA = 4,        /* a CUDA runtime or driver call failed                     */
    LINFUSION_ERR_TIMEOUT = 5      /* a bounded device-side wait expired (see status())        */
} linfusion_status_t;

typedef enum {
    LINFUSION_PHI_ELU_PLUS_ONE = 0, /* phi(x) = x + 1 (x > 0), exp(x) (x <= 0)  */
    LINFUSION_PHI_IDENTITY = 1      /* phi(x) = x: inputs are non-negative features already */
} linfusion_phi_t;

/* flags: kernel-variant selection.  0 lets the library choose from (N, d, B*H). */
#define LINFUSION_VARIANT_AUTO 0u
#define LINFUSION_VARIANT_SPLIT 1u   /* three launches: split-N state, reduction, apply (any supported d) */
#define LINFUSION_VARIANT_STREAM 2u  /* TMA-pipelined persistent tcgen05 kernels (d = 64 only): two launches, the
                                        apply kernel sums the partial states itself (three when slabs > SMs) */
#define LINFUSION_VARIANT_CLUSTER 3u /* one launch, thread-block cluster per slab (small N); one CTA per slab for N <= 192 */
#define LINFUSION_VARIANT_FUSED 4u   /* one launch, persistent TMA + tcgen05 kernel with per-slab counters: d = 64, and
                                        d = 40 / 80 / 160 (d' = d) when N <= 65536 * max(1, SMs / (B*H)) */
#define LINFUSION_VARIANT_MASK 0xFu
/*
 * flags: memory layout of Q, K, V and Y.  Default (bit clear): head-major [B, H, N, d].  Bit set:
 * token-major [B, N, H, d] — the [B, N, C] tensor a UNet block holds, with C = H*d split into
 * heads in place — so that the caller needs no transpose before or after the attention (a
 * transpose pass would move twice the attention's own minimum traffic).  Every entry point that
 * takes a descriptor or a handle follows it.  The split and cluster variants do the same arithmetic
 * in the same order in both layouts (same bits); the stream variant uses another fixed split of N
 * in this layout (the same number of CTAs on every slab, which keeps the heads of a token in step),
 * so its last bits may differ from the head-major result, reproducibly.
 */
#define LINFUSION_LAYOUT_TOKEN_MAJOR 0x10u

/*
 * flags: the operator without its normalizer.  Bit set: Y_i = phi(Q_i) S, i.e. Y = f'(X) g'(X)^T X of
 * Prop. 2 before the division of Eq. 5 is applied (the "without normalization" rows of the
 * ablation in Tab. 2).  eps is then unused; z is still accumulated and read_state() returns it.
 * |Y| grows with N in this form (the paper's reason for the normalizer); outputs are still 16-bit.
 */
#define LINFUSION_FLAG_UNNORMALIZED 0x20u
/*
 * flags: storage type of Q, K, V and Y.  Default (bit clear): bf16.  Bit set: fp16 (IEEE half), the
 * precision the paper's implementation runs in.  Accumulation is fp32 either way.  With fp16 the
 * state S | z, whose entries grow with N, is handed to the apply step's tensor-core operand scaled
 * by 2^-ceil(log2 N) so that it fits the format (the scale cancels in Eq. 5's quotient; eps is
 * scaled with it); read_state() returns the unscaled fp32 state.  The un-normalized operator's
 * output itself grows like sqrt(N) and must fit fp16's range (65504) in that case.
 */
#define LINFUSION_DTYPE_FP16 0x40u

typedef struct {
    int32_t B;      /* batch                                   > 0 */
    int32_t H;      /* heads                                   > 0; B*H <= 65535 (one grid row per slab) */
    int32_t N;      /* tokens per slab                         > 0 */
    int32_t d;      /* head dim: one of 32, 40, 64, 80, 128, 160   */
    int32_t phi;    /* linfusion_phi_t                             */
    float eps;      /* finite, >= 0; added once to phi(Q_i) . z    */
    int32_t device; /* CUDA device ordinal the handle lives on     */
    uint32_t flags; /* LINFUSION_VARIANT_* | LINFUSION_LAYOUT_*      */
    int32_t d_qk;   /* feature width d' of Q and K when it differs from d (Prop. 3); 0 = d.
                       Supported pairs (d', d): (128, 64), (80, 40), (32, 64)              */
} linfusion_attn_desc_t;

/*
 * Two widths (Prop. 3).  The proposition lets f' and g' map a token to d' features while the values
 * keep d channels: Q and K are then [B, H, N, d'] (token-major: [B, N, H, d']), V and Y stay
 * [B, H, N, d], the state S is d' x d and z has d' entries:
 *
 *     S = sum_j phi(K_j)^T V_j  (d' x d),   z = sum_j phi(K_j)  (d'),   Y_i = phi(Q_i) S / (phi(Q_i) . z + eps)
 *
 * desc.d is the value width d, desc.d_qk the feature width d' (0: the same as d, the released
 * model's case).  The three-launch split path and the cluster kernel serve d' != d; the TMA +
 * tcgen05 variants are for d' = d: STREAM at 64, FUSED at 40, 64, 80 and 160.  Everywhere this header says [.., d] for Q
 * or K, or d x d for S, or d for z, read d' for the feature side.
 */

/*
 * Create a handle for one problem shape (Prop. 2's token mixer at fixed B, H, N, d).
 * Validates the descriptor, checks that `device` is compute capability 10.x, fixes the
 * split of N and allocates the workspace (cudaMalloc) on that device.
 * Errors: INVALID_ARG (null pointers, sizes <= 0, eps negative or not finite),
 * UNSUPPORTED (d, phi, variant, unknown flag bits, B*H > 65535, device architecture), ALLOC, CUDA.
 * *out is NULL on error.  create() and set_workspace() return only when the workspace has been
 * cleared, so a forward() may follow at once on any stream.
 */
linfusion_status_t linfusion_attn_create(const linfusion_attn_desc_t* desc, linfusion_attn_t** out);

/*
 * Enqueue Y = norm-linear-attention(Q, K, V) on `cuda_stream` (a cudaStream_t / CUstream;
 * NULL is the legacy default stream).  q, k, v: const bf16 (or fp16) [B,H,N,d] device memory;
 * y: the same type, [B,H,N,d] device memory, written in full, rounded to nearest even from fp32.
 * Steps: split-N state reduction (S_p, z_p per chunk p of the tokens; Prop. 2 and Eq. 5),
 * fixed-order reduction to (S, z), apply — or all three in one launch (CLUSTER, FUSED).
 * Errors: INVALID_ARG (null handle or pointer, pointer not 16-byte aligned, y overlapping an
 * input), CUDA (launch or tensor-map encoding failed).  A bounded device-side wait that
 * expired is reported by status(), not here.
 */
linfusion_status_t linfusion_attn_forward(linfusion_attn_t* h, const void* q, const void* k,
                                          const void* v, void* y, void* cuda_stream);

/*
 * The same operation for callers whose tensors live in HOST memory (pinned memory makes the
 * copies asynchronous): copies K, V, Q to device staging buffers owned by the handle, runs
 * forward() on them and copies Y back, ordered after the earlier work and before the later work
 * of `cuda_stream`.  Large problems are cut into up to 20 groups of (b, h) slabs so that the upload
 * of one group, the kernels of the previous one and the download of the one before overlap (two
 * internal copy streams); each group then has its own fixed split of N, so Y may differ from
 * forward()'s in the last bits while staying bit-identical from call to call.  The staging
 * buffers (4 x B*H*N*d*2 bytes), the group handle, the streams and the events are created by
 * the first call on a handle and freed by destroy().  y_host is valid after `cuda_stream` has
 * been synchronized.  Errors: INVALID_ARG, ALLOC, CUDA.
 */
linfusion_status_t linfusion_attn_forward_host(linfusion_attn_t* h, const void* q_host,
                                               const void* k_host, const void* v_host, void* y_host,
                                               void* cuda_stream);

/* Free the handle, the workspace it owns and its staging buffers.  destroy(NULL) is OK. */
linfusion_status_t linfusion_attn_destroy(linfusion_attn_t* h);

/* Static, NUL-terminated description of a status code. */
const char* linfusion_status_string(linfusion_status_t s);

/*
 * Bytes of device workspace a handle for `desc` needs, for callers that want to own it:
 * fp32 partial states S_p | z_p of the split of N, the reduced state S | z per slab, and one
 * status word.  Pure host computation (no CUDA call) for a given SM count; `sm_count` <= 0
 * means 148 (B200).  Errors: INVALID_ARG, UNSUPPORTED.
 */
linfusion_status_t linfusion_attn_workspace_bytes(const linfusion_attn_desc_t* desc, int sm_count,
                                                  size_t* bytes);

/*
 * What a handle for `desc` would run on a device with `sm_count` SMs (<= 0: 148), without creating
 * one: *variant receives the LINFUSION_VARIANT_* that desc.flags resolves to (AUTO resolved from
 * (N, d, B*H) as create() does it, before any fall-back create() may take when a cluster cannot be
 * scheduled), *launches the kernel launches per forward, *ctas the grid size of its largest kernel
 * (0 for the split and cluster variants, whose grids are two-dimensional).  Pure host computation (no
 * CUDA call); any of the three pointers may be NULL.  Errors: INVALID_ARG, UNSUPPORTED.
 */
linfusion_status_t linfusion_attn_plan(const linfusion_attn_desc_t* desc, int sm_count, int32_t* variant,
                                       int32_t* launches, int32_t* ctas);

/*
 * Lend a device workspace (256-byte aligned, at least workspace_bytes) to the handle, which
 * stops using — and frees — its own.  The caller keeps ownership and must keep it alive
 * until the handle is destroyed.  Errors: INVALID_ARG, ALLOC (too small).
 */
linfusion_status_t linfusion_attn_set_workspace(linfusion_attn_t* h, void* dev_ptr, size_t bytes);

/*
 * Synchronize the handle's last stream and read the device status word: OK, or TIMEOUT if
 * a kernel gave up on a bounded wait (its outputs are then undefined), or CUDA.
 */
linfusion_status_t linfusion_attn_status(linfusion_attn_t* h);

/*
 * Self-test of the failure reporting (the paper has no counterpart): runs a one-warp kernel that
 * waits on a barrier nothing will ever complete, exactly as the attention kernels wait, on the
 * handle's last stream.  The wait must give up after its time bound (a quarter of a second), the
 * kernel must end normally and the device status word must be set.  Returns TIMEOUT when all of
 * that happened (the expected result), OK if the wait claimed to have succeeded, or CUDA; the
 * status word is cleared again, so the handle and the context stay usable.  *waited_ms (may be NULL)
 * receives the kernel's duration.
 */
linfusion_status_t linfusion_attn_selftest_wait(linfusion_attn_t* h, float* waited_ms);
/*
 * The same self-test for the other kind of bounded wait: the single-launch variant
 * (LINFUSION_VARIANT_FUSED) lets the CTAs that apply a slab wait, by polling a counter in global
 * memory, until every CTA that contributes a partial state of that slab (Prop. 2's sum over tokens,
 * split over CTAs) has delivered it.  This runs one warp that polls a counter nothing advances.
 * Results as for selftest_wait().
 */
linfusion_status_t linfusion_attn_selftest_counter_wait(linfusion_attn_t* h, float* waited_ms);

/*
 * Copy the reduced state of the last forward to HOST buffers (fp32): S [B*H][d][d] (row =
 * feature c of K, column = channel e of V) and z [B*H][d].  Synchronizes the handle's last
 * stream.  Either pointer may be NULL.  This is the c' x c quantity that the paper's
 * distributed inference exchanges between devices (Sec. 4.3).  Errors: INVALID_ARG, CUDA.
 */
linfusion_status_t linfusion_attn_read_state(linfusion_attn_t* h, float* S_host, float* z_host);

/*
 * Token-sharded (sequence-parallel) use — the distributed inference of Sec. 4.3: every device
 * owns a run of the tokens of Q, K, V and Y (desc.N is the local token count), and the only
 * quantity exchanged is the state S | z, whose size does not depend on N.  Per layer:
 *
 *   1. linfusion_attn_state(h, k_local, v_local, stream)   S, z of the local K/V tokens
 *                                                           (split-N kernel + fixed-order reduction)
 *   2. the caller sums the fp32 buffer returned by linfusion_attn_state_buffer() over all devices,
 *      in place, on the same stream (e.g. an NCCL all-reduce; the state is additive over token
 *      shards, Prop. 2)
 *   3. linfusion_attn_apply(h, q_local, y_local, stream)    Y of the local Q tokens from the
 *                                                           summed state
 *
 * state_buffer: *dev_ptr is the device address of [B*H][d*d S (row = feature c of K, column =
 * channel e of V), then d z] fp32, *floats its length; it stays valid until the handle is
 * destroyed or its workspace is replaced.  Handles that resolved to a single-launch variant
 * (CLUSTER, FUSED; AUTO picks CLUSTER for N <= 192, FUSED for many small slabs of head dim 64 and for
 * head dims 40 / 80 / 160 wherever that kernel applies) cannot be split in two:
 * state() and apply() return UNSUPPORTED for them (create the handle with LINFUSION_VARIANT_SPLIT
 * or _STREAM).  Other errors as for forward().
 */
linfusion_status_t linfusion_attn_state(linfusion_attn_t* h, const void* k, const void* v,
                                        void* cuda_stream);
linfusion_status_t linfusion_attn_apply(linfusion_attn_t* h, const void* q, void* y, void* cuda_stream);

/*
 * Steps 2 and 3 in one: the apply half that sums the devices' states itself (Sec. 4.3's exchange of
 * the c' x c quantity, done by the kernel that needs it instead of a separate collective).
 * peer_states is a HOST array of n_peers (1 .. LINFUSION_MAX_PEERS) DEVICE addresses, entry r the
 * state_buffer() of rank r's handle (this rank's own included), each readable from this handle's
 * device: the caller maps peers' buffers (peer access, CUDA IPC or symmetric memory) and passes
 * the same list, in the same order, on every rank.  A small kernel adds the n states element by
 * element in list order with plain loads (over NVLink for peers' entries; 4*B*H*d*(d+1) bytes
 * from each) into this handle's 16-bit operand image, and the apply kernel follows on the same
 * stream.  Same list => same summation order => the same bits of S | z on every rank.  Nobody's
 * state buffer is written, so ranks may run this concurrently; read_state() keeps returning the
 * local, unsummed state.
 * Synchronization is the caller's: every rank's linfusion_attn_state() must have completed, and
 * no rank may start its next linfusion_attn_state() on these handles before all ranks' apply_peers
 * kernels have read its buffer (e.g. a stream-ordered barrier on either side).
 * With fp16 storage the operand scale 2^-ceil(log2 N) is derived from the LOCAL token count, while
 * the summed z is about 1.2 * N_local * n_peers: the scaled z stays below 1.2 * n_peers (well
 * inside fp16's 65504 for any n_peers <= LINFUSION_MAX_PEERS), S keeps its relative size.
 * Errors: INVALID_ARG (null / misaligned pointers, n_peers out of range), UNSUPPORTED (cluster
 * handle), CUDA.
 */
#define LINFUSION_MAX_PEERS 16
linfusion_status_t linfusion_attn_apply_peers(linfusion_attn_t* h, const void* q, void* y,
                                              const float* const* peer_states, int32_t n_peers,
                                              void* cuda_stream);
linfusion_status_t linfusion_attn_state_buffer(linfusion_attn_t* h, float** dev_ptr, size_t* floats);

/*
 * Per-kernel timing for benchmarks.  enable(h, slots > 0) creates `slots` sets of CUDA events;
 * from then on every forward() brackets each of its kernels with event records on its stream
 * (set = call index modulo slots).  enable(h, 0) turns it off.  kernel_times() synchronizes the
 * handle's last stream and returns, for the calls recorded since the last kernel_times()
 * (at most `slots`), the summed milliseconds of each kernel in launch order — ms_sum[0] the
 * state kernel (or the single clustered kernel), ms_sum[1] the reduction, ms_sum[2] the apply —
 * and the number of calls summed.  Errors: INVALID_ARG, ALLOC, CUDA.
 */
linfusion_status_t linfusion_attn_enable_kernel_timing(linfusion_attn_t* h, int32_t slots);
linfusion_status_t linfusion_attn_kernel_times(linfusion_attn_t* h, float* ms_sum, int32_t* calls);
/*
 * Sample the timing: only every `stride`-th forward (the first one after enable() included) is
 * bracketed with events; the others are enqueued exactly as without timing.  An event record between
 * two kernels keeps the second from being scheduled behind the first (the kernels of a forward
 * are chained by programmatic dependent launch), so timing every call slows the calls it times;
 * a stride keeps most of a timed region undisturbed.  Default 1.  Errors: INVALID_ARG (stride < 1).
 */
linfusion_status_t linfusion_attn_set_kernel_timing_stride(linfusion_attn_t* h, int32_t stride);

/*
 * The attention without a handle and without any allocation.  (The paper has no counterpart to
 * this call; it exists for how the library gets embedded.)
 *
 * Some hosts cannot let a library allocate device memory: an inference server that hands all of
 * its device memory to its own arena at start-up, so that a later cudaMalloc from inside a
 * library either fails or breaks the memory budget it promised; or a latency-bound pipeline that
 * cannot afford the device-wide synchronization cudaMalloc and cudaFree imply.  create() and the
 * first forward_host() both allocate, so such callers use this entry point instead.  It runs the
 * three-launch split path (split-N state, fixed-order reduction, apply; any supported head dim)
 * and keeps the partial states and the reduced state in a fixed 16 MiB array that is part of the
 * library's device image: every GPU that loads the library holds those 16 MiB until the process
 * exits.  (With CUDA's default lazy module loading the driver commits the library's device image,
 * these 16 MiB included, when the library is first used on a device — the first call of this
 * function, if nothing else came before; with CUDA_MODULE_LOADING=EAGER, when the library is
 * loaded.  A host that gives all remaining device memory to its arena must make that first call,
 * or load eagerly, before it does so.)  It calls no cudaMalloc, cudaFree or other allocating
 * routine, creates no streams or events, and keeps no per-call host state.
 *
 * desc: as for create(); flags must be AUTO or SPLIT.  q, k, v, y, cuda_stream: as for forward().
 * The split of N uses as many chunks as fit in the array; a problem whose state alone does not
 * fit — 2 * B*H * d*(d+1) * 4 bytes + 512 above 16 MiB, e.g. d = 160 with more than 81 slabs — is
 * rejected with LINFUSION_ERR_ALLOC and nothing is launched.  Other errors: INVALID_ARG,
 * UNSUPPORTED (as for create(), B*H > 65535 included), CUDA, as for create() and forward().
 *
 * The first call on each device looks up the array's device address, and the first call for each
 * (device, head dim, phi, storage type) raises the two kernels' shared-memory limits; later calls
 * make no CUDA call besides the three launches.  Make those first calls before starting any
 * stream capture.  First calls from several host threads at once are safe (the set-up is
 * serialized); the array's contents are what concurrent calls race on, see below.
 * Every call on a device shares the one array, which keeps whatever the last call left in it.
 * Nothing in it needs clearing between calls (each call writes every element before reading it),
 * but two calls whose kernels overlap on the GPU — different streams, or several host threads —
 * race on it and corrupt each other's state: order such calls on one stream, or with events.
 * Output is bit-identical from call to call for identical inputs on the same device.
 */
linfusion_status_t linfusion_attn_forward_noalloc(const linfusion_attn_desc_t* desc, const void* q,
                                                  const void* k, const void* v, void* y,
                                                  void* cuda_stream);

/*
 * Where forward_noalloc() would put a problem in its fixed array, without touching a device (the
 * paper has no counterpart): *chunks = partial states per slab that the split of N uses on a GPU
 * with `sm_count` SMs (<= 0: 148), cut down to what leaves room for the state; *state_offset = byte
 * offset of the reduced state (the partials start at 0); *bytes_used = end of the state;
 * *capacity = size of the array.  Any output pointer may be NULL.  bytes_used <= capacity whenever
 * OK is returned.  Errors: INVALID_ARG, UNSUPPORTED, ALLOC (does not fit), as forward_noalloc().
 */
linfusion_status_t linfusion_attn_noalloc_layout(const linfusion_attn_desc_t* desc, int sm_count,
                                                 int32_t* chunks, size_t* state_offset,
                                                 size_t* bytes_used, size_t* capacity);

/*
 * The attention fed from the layer input X instead of from Q, K, V (Sec. 3.1, implementation details;
 * Eq. 2).  In the module, Q = f'(X), K = g'(X) and V = X W_V, with
 *
 *     f'(X) = X W_Q + LeakyReLU(LayerNorm(X W_1q + b_1q)),     g'(X) likewise with its own weights:
 *
 * a linear branch plus one Linear-LayerNorm-LeakyReLU block, summed.  The entry points below run the
 * projections on the tensor cores inside the kernels that consume them, so that K, V and Q are never
 * written to or read from device memory.
 *
 * They need a handle with head dim 64 (d_qk = 0), LINFUSION_VARIANT_STREAM and
 * LINFUSION_LAYOUT_TOKEN_MAJOR (else UNSUPPORTED).  x: device, 16-bit, [B, N, C] with C = H * 64 (the
 * heads of a token side by side, which is what [B, N, H, d] is).  Every weight matrix: device, 16-bit
 * (the handle's storage type), [C][C] row-major with row = input channel, column = output channel
 * (out = x W), 16-byte aligned.
 *
 * state_x: S | z of the slabs from X — per 128-token tile and head, [K | V] = X [W_K,h | W_V,h] into
 * tensor memory, K (+ t_k) through phi, both rounded to 16 bits into shared memory, then the split-N
 * state accumulation and the fixed-order reduction exactly as in linfusion_attn_state().  t_k (may be
 * NULL) is the output of g's non-linear branch, LeakyReLU(LayerNorm(X W_1k + b_1k)), 16-bit [B, N, C];
 * NULL means the branch contributes nothing (the paper's initialization).  Afterwards state_buffer(),
 * read_state(), apply() and apply_peers() work as after linfusion_attn_state().
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA.
 */
linfusion_status_t linfusion_attn_state_x(linfusion_attn_t* h, const void* x, const void* w_k,
                                          const void* w_v, const void* t_k, void* cuda_stream);
/*
 * apply_x: Y of the local tokens from X and the handle's current state (Prop. 2's output with Eq. 5's
 * division) — per 128-token tile and head, Q = X W_Q,h into tensor memory, Q (+ t_q) through phi and back
 * into tensor memory as the A operand of phi(Q) [S | z], rows divided by their denominator, Y tile
 * stored with TMA.  t_q (may be NULL): output of f's non-linear branch, as t_k above.  y: device, 16-bit,
 * [B, N, C], written in full; must not overlap x.  The fp32 state is re-read (it may have been summed
 * over devices since state_x(), Sec. 4.3), so state_x() / all-reduce / apply_x() is the token-sharded
 * forward from X.  Errors: INVALID_ARG, UNSUPPORTED, CUDA.
 */
linfusion_status_t linfusion_attn_apply_x(linfusion_attn_t* h, const void* x, const void* w_q,
                                          const void* t_q, void* y, void* cuda_stream);

/*
 * branch_x: the output of one non-linear branch, T = LeakyReLU(LayerNorm(X W_1 + b_1; gamma, beta)), into
 * t_out [B, N, C] (device, 16-bit, must not overlap x).  w_1: [C][C] as the other weights; b_1 (may be
 * NULL: no bias), gamma, beta: [C], 16-bit.  LayerNorm runs over a token's whole feature vector (all
 * heads), biased variance, ln_eps inside the root; leaky_slope is LeakyReLU's negative slope.  Two
 * launches: the projection on the tensor cores, which also leaves every row's mean and
 * 1 / sqrt(variance + ln_eps) (sums taken in fp32 before U is rounded to 16 bits), and the
 * element-wise normalization in place.  The first call on a handle allocates the row-statistics
 * buffer (8 bytes per token; freed by destroy()).  C <= 2048.
 * Errors: INVALID_ARG, UNSUPPORTED, ALLOC, CUDA.
 */
linfusion_status_t linfusion_attn_branch_x(linfusion_attn_t* h, const void* x, const void* w_1,
                                           const void* b_1, const void* gamma, const void* beta,
                                           float ln_eps, float leaky_slope, void* t_out,
                                           void* cuda_stream);

/* The parameters of f' or g': out = x w_lin + LeakyReLU(LayerNorm(x w_1 + b_1; gamma, beta)). */
typedef struct {
    const void* w_lin; /* [C][C] linear branch (initialized from W_Q / W_K in the paper)     */
    const void* w_1;   /* [C][C] the block's Linear; NULL: the non-linear branch is absent   */
    const void* b_1;   /* [C] its bias; may be NULL                                          */
    const void* gamma; /* [C] LayerNorm scale                                                */
    const void* beta;  /* [C] LayerNorm shift                                                */
} linfusion_mlp_weights_t;

typedef struct {
    linfusion_mlp_weights_t q; /* f' */
    linfusion_mlp_weights_t k; /* g' */
    const void* w_v;           /* [C][C], Eq. 2 */
    float ln_eps;              /* LayerNorm's epsilon          */
    float leaky_slope;         /* LeakyReLU's negative slope   */
} linfusion_module_weights_t;

/*
 * forward_x: the whole module from the layer input, Y = attention(f'(X), g'(X), X W_V): the non-linear
 * branches that are present (branch_x into buffers of B*N*C*2 bytes each that the handle allocates on
 * first use and frees in destroy()), then state_x and apply_x.  x, y: [B, N, C] as above.
 * Errors: INVALID_ARG, UNSUPPORTED, ALLOC, CUDA.
 */
linfusion_status_t linfusion_attn_forward_x(linfusion_attn_t* h, const void* x,
                                            const linfusion_module_weights_t* w, void* y,
                                            void* cuda_stream);

/*
 * The bounds-checked debugging build (the paper has no counterpart; it stands in for a memory checker).
 * The same sources compiled with -DLF_CHECKED give a second library in which forward(), forward_noalloc(),
 * state(), apply() and apply_peers() of the SPLIT and CLUSTER variants first tell the device which byte
 * ranges the call may touch (Q, K, V, Y, the workspace, peers' states), and every global-memory address
 * these kernels compute is compared with them: an access that does not lie wholly inside one range is
 * counted and skipped (loads return zero) — nothing traps or faults, the call completes.  One range table
 * per device: checked calls on different streams must not overlap in time.
 *   checked_build():       1 in that library, 0 in the normal one.
 *   checked_violations():  synchronizes `device` and returns the number of skipped accesses since the
 *                          last reset in *count (reset != 0 clears it).  UNSUPPORTED in the normal build
 *                          (*count = 0).  Errors: INVALID_ARG, CUDA.
 *   checked_shrink_y():    self-test of the check itself: from now on the registered range of Y is cut
 *                          short by `bytes` at its end, so that the (valid) stores to the last rows of Y
 *                          are reported and skipped and those rows keep what they held; 0 restores the
 *                          full range.  No access leaves its buffer either way.  UNSUPPORTED in the
 *                          normal build.
 */
int32_t linfusion_attn_checked_build(void);
linfusion_status_t linfusion_attn_checked_violations(int32_t device, uint32_t* count, int32_t reset);
linfusion_status_t linfusion_attn_checked_shrink_y(size_t bytes);

/* Name of the kernel variant the handle resolved to ("split", "stream", "cluster", "fused"). */
const char* linfusion_attn_variant_name(const linfusion_attn_t* h);

/* Number of kernel launches one forward() enqueues for this handle. */
int32_t linfusion_attn_launches_per_forward(const linfusion_attn_t* h);

#ifdef __cplusplus
}
#endif
#endif /* LINFUSION_ATTN_H */
