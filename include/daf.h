/*
 * daf.h -- C ABI of the B200 (sm_100a) activation compress / decompress library.
 *
 * The library implements the data-parallel hot path of the Dynamic Activation
 * Framework: saved activations are quantized group by group after the forward
 * pass and dequantized before the backward pass (Sec. 2.3 of the paper).
 *
 * Conventions for every entry point
 *   - Pointers named d_* are DEVICE pointers owned by the caller; h_* are HOST
 *     pointers.  The library never allocates or frees device memory: inputs,
 *     outputs and scratch ("workspace") all belong to the caller.
 *   - `stream` is a cudaStream_t passed as void*.  GPU work is enqueued on it
 *     and the call returns without waiting; outputs are valid once the stream
 *     has reached that point.
 *   - The return value is a daf_status.  Argument errors are detected on the
 *     host before anything is launched.  Errors that only the device can see
 *     (packed buffer too small, a bounded wait that ran out) are recorded in a
 *     status word inside the workspace and read back with daf_poll_status; the
 *     kernels never store out of bounds, trap or spin without limit.
 *   - Device pointers must be 16-byte aligned unless stated otherwise.
 *   - No entry point throws.  State the library keeps between calls: a table, one entry per
 *     (kernel, device), of how many CTAs of that kernel the device holds at once, filled at
 *     the first launch on each device and guarded by a mutex; and the scratch array of
 *     daf_compress_static.  Entry points may be called from several threads and on several
 *     devices at once (work goes to the device that is current in the calling thread) as
 *     long as calls that overlap on the GPU use different workspaces.  daf_pool and
 *     daf_store objects are not thread safe: one thread at a time per object.
 *
 * Data layout (all tensors are flat, contiguous, row-major)
 *   group   : G consecutive elements (G a power of two, 32 <= G <= window_elems)
 *   window  : window_elems consecutive elements = the unit over which the
 *             average bit budget is enforced and the unit of parallel work
 *   packed  : for group g, G*b_g/8 bytes at byte offset sum_{h<g} G*b_h/8; code i
 *             of the group occupies bits [i*b_g, (i+1)*b_g) of that byte string,
 *             least significant bit first (little-endian 32-bit words with
 *             code i at shift (i*b_g) mod 32); no padding anywhere
 *   bits    : one byte per group, the width b_g itself
 *   min, scale : one float per group (binary32 for every input dtype)
 *   window_offsets : n_windows+1 uint64 byte offsets of each window's first
 *             group in `packed`; the last entry is the total packed size
 */
#ifndef DAF_H
#define DAF_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum daf_status {
    DAF_OK = 0,
    DAF_ERR_INVALID_ARG = 1,  /* null / misaligned pointer, bad group or window size, bad mask */
    DAF_ERR_SHAPE = 2,        /* numel is zero or not a multiple of the group size            */
    DAF_ERR_BUDGET = 3,       /* bit budget below the smallest allowed width                   */
    DAF_ERR_CAPACITY = 4,     /* packed buffer or workspace too small                          */
    DAF_ERR_CUDA = 5,         /* a CUDA runtime call failed                                    */
    DAF_ERR_TIMEOUT = 6,      /* a bounded device-side wait ran out                            */
    DAF_ERR_UNSUPPORTED = 7   /* valid request this build does not implement                   */
} daf_status;

typedef enum daf_dtype { DAF_F32 = 0, DAF_F16 = 1, DAF_BF16 = 2 } daf_dtype;
typedef enum daf_round { DAF_ROUND_STOCHASTIC = 0, DAF_ROUND_NEAREST = 1 } daf_round;

typedef void *daf_stream;     /* a cudaStream_t */

/* Description of one tensor and of how it is (was) compressed. */
typedef struct daf_params {
    uint32_t struct_size;     /* sizeof(daf_params), for ABI checking                               */
    uint32_t dtype;           /* daf_dtype of the input of compress / the output of decompress      */
    uint64_t numel;           /* elements; a positive multiple of group_size                        */
    uint32_t group_size;      /* G: power of two, 32 <= G <= window_elems                           */
    uint32_t window_elems;    /* 0 means 16384; supported: 4096, 8192, 16384                        */
    uint32_t width_mask;      /* bit b set <=> width b allowed; non-empty subset of {1,2,4,8}       */
    float    bit_budget;      /* average bits per element per window; floor(budget*256)/256 is used */
    uint32_t rounding;        /* daf_round                                                          */
    uint32_t flags;           /* 0, or DAF_FLAG_* values or'ed together (launch policy, diagnostics) */
    uint64_t seed;            /* Philox key                                                         */
    uint64_t elem_index_base; /* global index of element 0 (a multiple of 8); 0 unless the tensor
                                 is a shard of a larger one compressed with the same seed          */
} daf_params;

/* daf_params.flags.  None of them changes a result.
 *   DAF_FLAG_STREAM_ALWAYS / _NEVER : daf_compress first runs a streaming kernel that assumes windows
 *       of one width, or of two neighbouring widths (see daf_compress), unless the call is small or the
 *       parameters rule such windows out; ALWAYS drops the size rule, NEVER goes to the general kernel directly (e.g. for data known
 *       to mix widths).  Giving both is an error.
 *   DAF_FLAG_ONE_PASS / _TWO_PASS : windows of mixed widths are handled either by the general kernel (one pass
 *       over the input; CTAs that wait for one another's window offsets) or by the two-pass kernels (widths first,
 *       then offsets, then quantize + pack: the input is read twice, nothing waits).  The library chooses by
 *       element type and group size; these flags force one or the other where both exist (two-pass: groups of 128
 *       to 1024 elements, default window, no fused activation).  Giving both is an error.
 *   DAF_FLAG_KEEP_WORKSPACE : diagnostic.  The workspace is not cleared on entry: the caller has
 *       prepared it (all zero, except what a test of the failure paths has planted there).
 *   DAF_FLAG_POLL_LIMIT(n)  : diagnostic.  Bounded device-side waits give up after n polls
 *       (1 <= n < 2^24) instead of the default 2^20.
 */
#define DAF_FLAG_STREAM_ALWAYS  0x1u
#define DAF_FLAG_STREAM_NEVER   0x2u
#define DAF_FLAG_KEEP_WORKSPACE 0x4u
#define DAF_FLAG_ONE_PASS       0x8u
#define DAF_FLAG_TWO_PASS       0x10u
#define DAF_FLAG_POLL_LIMIT(n)  ((uint32_t)(n) << 8)

/*
 * Sizes that follow from the parameters (host only, launches nothing).
 *   n_groups = numel / G, n_windows = ceil(n_groups / (window_elems / G)),
 *   packed_capacity_bytes = sum over windows of floor(beta_q8 * n / 256) * G / 8 with n the
 *   window's group count and beta_q8 = floor(bit_budget * 256): an upper bound on the packed
 *   size that the budget guarantees,
 *   workspace_bytes = scratch needed by daf_compress / daf_decompress for this tensor.
 * Any output pointer may be NULL.  Errors: INVALID_ARG, SHAPE, BUDGET, UNSUPPORTED.
 */
daf_status daf_sizes(const daf_params *params, uint64_t *n_groups, uint64_t *n_windows,
                     uint64_t *packed_capacity_bytes, uint64_t *workspace_bytes);

/*
 * Sharding (host only).  The path has no exchange step: a tensor is cut at window boundaries, every rank (GPU)
 * compresses its slice with the same seed and with elem_index_base moved to the slice's first element, and the results
 * are exactly the pieces of the unsharded result (widths, minima, scales, packed bytes; window offsets restart at 0 in
 * every slice).  daf_shard fills *shard with the parameters of the slice of rank `rank` among `world` ranks -- whole
 * windows, as even as possible, in order -- and *first_elem (may be NULL) with the slice's first element.  A rank
 * beyond the number of windows gets shard->numel == 0: nothing to do.  Errors: those of daf_sizes for `whole`;
 * INVALID_ARG for a null shard, world == 0 or rank >= world.
 */
daf_status daf_shard(const daf_params *whole, uint32_t rank, uint32_t world, daf_params *shard, uint64_t *first_elem);

/*
 * Compress one tensor (Eq. 1 applied per group; widths chosen greedily per window by
 * importance per bit under the budget, Sec. 3.4.1; codes packed compactly, Sec. 3.3).
 *   d_in             in : numel elements of params->dtype; 32-byte aligned for DAF_F32 (a lane reads
 *                          eight elements at once), 16-byte aligned otherwise
 *   d_packed         out: packed codes, at most packed_capacity bytes are written
 *   d_bits           out: n_groups bytes        d_min, d_scale  out: n_groups floats each
 *   d_window_offsets out: n_windows + 1 uint64
 *   d_workspace          : workspace_bytes of scratch, contents irrelevant on entry; also
 *                          holds the device status word afterwards (see daf_poll_status)
 * The call enqueues, in this order: a streaming kernel, which assumes that in every window
 * all groups end at one and the same width (the one the budget gives a window of equal
 * groups) and writes every output on that assumption while it records what is needed to
 * check it; a small kernel that checks it for every window and writes the window offsets;
 * and a fallback, which returns at once unless the check failed somewhere and then redoes the
 * whole call with the window-by-window greedy choice.  Where the budget lies between two
 * allowed widths (groups of 256 to 1024 elements, default window) the streaming kernel is
 * another one: it assumes that in every window the groups end at those two widths, the k
 * groups with the largest ranges at the larger one (k follows from the budget alone), checks
 * that itself window by window, and asks for the fallback where the assumption fails.  The fallback is the general kernel
 * (one launch; the input is read once), or, for calls of more than 4096 windows on 16-bit
 * elements with groups of 128 to 1024 elements, three kernels that read the input twice:
 * widths and metadata of every window, window offsets, quantize + pack.  A call of at most
 * 4096 windows, or one whose parameters rule out one-width windows, goes to the fallback
 * alone; params->flags can force each of these choices.  All routes give the same bytes.
 * Every output is final when the call's work on the stream is done.  If the packed output
 * of a window would pass packed_capacity, nothing of that window is stored and the status
 * word becomes DAF_ERR_CAPACITY.  Inputs must be finite; behaviour on NaN / Inf is unspecified but
 * memory safe.  Calls sharing a workspace must not overlap on the GPU.
 */
daf_status daf_compress(const daf_params *params, const void *d_in, void *d_packed,
                        uint64_t packed_capacity, uint8_t *d_bits, float *d_min, float *d_scale,
                        uint64_t *d_window_offsets, void *d_workspace, uint64_t workspace_bytes,
                        daf_stream stream);

/* Fused producer (Sec. 3.2.3, kernel fusion: the statistics are taken where the activation is
 * produced, so it crosses HBM once).  Computes act = max(x, +0) element-wise (ReLU; -0 and
 * negative values give +0), writes it to d_act in the input's type, and compresses act exactly
 * as daf_compress would: every other output is that of daf_compress(params, d_act, ...).
 * d_act (device, numel elements, 32-byte aligned) may be d_in itself.  Default window only
 * (window_elems 0 or 16384; DAF_ERR_UNSUPPORTED otherwise); other arguments, ownership and
 * errors as for daf_compress.
 */
daf_status daf_relu_compress(const daf_params *params, const void *d_in, void *d_act, void *d_packed,
                             uint64_t packed_capacity, uint8_t *d_bits, float *d_min, float *d_scale,
                             uint64_t *d_window_offsets, void *d_workspace, uint64_t workspace_bytes,
                             daf_stream stream);

/*
 * Decompress (Sec. 2.3: stored activations are dequantized to their original precision
 * for the gradient computation): x_hat = fma(code, scale, min), rounded to nearest even
 * into params->dtype.  Inputs are the outputs of daf_compress for the same params;
 * d_out receives numel elements; it must be 32-byte aligned for DAF_F32 (a lane stores eight
 * elements at once), 16-byte aligned otherwise.  The workspace is not used by this version and may be NULL.
 */
daf_status daf_decompress(const daf_params *params, const void *d_packed, const uint8_t *d_bits,
                          const float *d_min, const float *d_scale,
                          const uint64_t *d_window_offsets, void *d_out, void *d_workspace,
                          uint64_t workspace_bytes, daf_stream stream);

/* The same for other activations.  act:
 *   DAF_ACT_RELU   as daf_relu_compress.
 *   DAF_ACT_RELU6  act = min(max(x, +0), 6), written to d_act and compressed.
 *   DAF_ACT_GELU   d_act receives GELU(x) = x/2 * (1 + erf(x / sqrt 2)), computed in binary32 and rounded to the
 *                  input's type (before that rounding, within 8 units in the last place of binary32 plus
 *                  2^-24 |x| of the exact value: the far negative tail is noise around 0); what is COMPRESSED is x itself, because the backward pass of a GELU
 *                  needs its input: every other output is that of daf_compress(params, d_in, ...).  d_act must
 *                  not be (or overlap) d_in.
 * Any other value of act: DAF_ERR_INVALID_ARG.
 */
typedef enum daf_act { DAF_ACT_RELU = 1, DAF_ACT_RELU6 = 2, DAF_ACT_GELU = 3 } daf_act;
daf_status daf_act_compress(const daf_params *params, uint32_t act, const void *d_in, void *d_act, void *d_packed,
                            uint64_t packed_capacity, uint8_t *d_bits, float *d_min, float *d_scale,
                            uint64_t *d_window_offsets, void *d_workspace, uint64_t workspace_bytes,
                            daf_stream stream);

/* Fused consumer (Sec. 3.2.3): the backward pass of a ReLU whose output was stored compressed.
 * d_grad_in[i] = d_grad_out[i] where the restored activation (exactly what daf_decompress would
 * store, in params->dtype) is > 0, else +0; the restored activation itself is never written.
 * d_grad_out, d_grad_in: device, numel elements of params->dtype, aligned like d_out of
 * daf_decompress; they may be the same buffer.  Other arguments and errors as for daf_decompress.
 */
daf_status daf_decompress_relu_grad(const daf_params *params, const void *d_packed, const uint8_t *d_bits,
                                    const float *d_min, const float *d_scale, const uint64_t *d_window_offsets,
                                    const void *d_grad_out, void *d_grad_in, daf_stream stream);

/* The consumer for the activations of daf_act_compress, r being the restored value in params->dtype:
 *   DAF_ACT_RELU   d_grad_in = d_grad_out where r > 0, else +0
 *   DAF_ACT_RELU6  d_grad_in = d_grad_out where 0 < r < 6, else +0
 *   DAF_ACT_GELU   d_grad_in = d_grad_out * (Phi(r) + r phi(r)), r the restored INPUT of the GELU; the factor is
 *                  computed in binary32 (within 2^-20 of the exact one), the product rounded to params->dtype
 * Arguments and errors as for daf_decompress_relu_grad.
 */
daf_status daf_decompress_act_grad(const daf_params *params, uint32_t act, const void *d_packed, const uint8_t *d_bits,
                                   const float *d_min, const float *d_scale, const uint64_t *d_window_offsets,
                                   const void *d_grad_out, void *d_grad_in, daf_stream stream);

/*
 * Device-wide exclusive prefix sum of the group byte lengths G*b_g/8 ("layout
 * concatenation", Sec. 3.3): d_offsets[g] = sum_{h<g} G*bits[h]/8 for g = 0..n_groups.
 * Single pass with a bounded decoupled look-back.  d_ws: daf_group_offsets_workspace(n_groups)
 * bytes of scratch.  d_bits needs no alignment; d_offsets must be 8-byte aligned.
 */
daf_status daf_group_offsets(const uint8_t *d_bits, uint64_t n_groups, uint32_t group_size,
                             uint64_t *d_offsets, void *d_ws, uint64_t ws_bytes, daf_stream stream);
uint64_t   daf_group_offsets_workspace(uint64_t n_groups);
/* The same with diagnostic flags (DAF_FLAG_KEEP_WORKSPACE, DAF_FLAG_POLL_LIMIT(n); any other bit is an error): for
 * tests of the bounded wait.  With KEEP_WORKSPACE the caller has prepared d_ws: all zero, except for what the test
 * plants there (the tile counter is the second 32-bit word, one 64-bit look-back descriptor per tile of 8192 groups
 * starts at byte 256; state in the top two bits: 0 empty, 1 tile sum, 2 prefix, 3 poison). */
daf_status daf_group_offsets_diag(const uint8_t *d_bits, uint64_t n_groups, uint32_t group_size,
                                  uint64_t *d_offsets, void *d_ws, uint64_t ws_bytes, uint32_t flags,
                                  daf_stream stream);

/*
 * Wait for `stream` and return the device status word of a workspace that was last used by
 * daf_compress, daf_compress_batch or daf_group_offsets: DAF_OK, DAF_ERR_CAPACITY or
 * DAF_ERR_TIMEOUT (DAF_ERR_CUDA if the copy itself fails).
 */
daf_status daf_poll_status(const void *d_workspace, daf_stream stream);

/*
 * Batched forms for sets of activations (one launch per up to DAF_BATCH_MAX tensors): the
 * result for tensor i is exactly that of the single-tensor call with params[i] and the i-th
 * pointers.  All arrays are HOST arrays of n entries holding device pointers / capacities;
 * every tensor of a batch must share dtype, group_size, window_elems, width_mask, bit_budget
 * and rounding (seed and elem_index_base may differ).  One workspace serves the whole batch:
 * daf_batch_workspace(n, params) bytes.
 */
#define DAF_BATCH_MAX 64   /* tensors per batched call */
uint64_t   daf_batch_workspace(uint32_t n, const daf_params *params);
daf_status daf_compress_batch(uint32_t n, const daf_params *params, const void *const *d_in,
                              void *const *d_packed, const uint64_t *packed_capacity,
                              uint8_t *const *d_bits, float *const *d_min, float *const *d_scale,
                              uint64_t *const *d_window_offsets, void *d_workspace,
                              uint64_t workspace_bytes, daf_stream stream);
daf_status daf_decompress_batch(uint32_t n, const daf_params *params, const void *const *d_packed,
                                const uint8_t *const *d_bits, const float *const *d_min,
                                const float *const *d_scale,
                                const uint64_t *const *d_window_offsets, void *const *d_out,
                                daf_stream stream);

/*
 * daf_compress without a caller-supplied workspace.  (The paper has no counterpart: this entry
 * point exists for callers of this library, not for the method.)
 *
 * Some callers cannot hand the library scratch memory because they cannot allocate any at the
 * point where activations are compressed: a training job that has given every free byte of the
 * device to its own preallocated arena, so that a further cudaMalloc fails; code running inside
 * a framework allocator's out-of-memory or free-memory callback, where asking that allocator
 * for a workspace tensor would re-enter it; paths that cannot afford the device-wide
 * synchronisation an allocation may imply.  For them the scratch of the compress kernel (the
 * 256-byte header with ticket and status word, and one 64-bit look-back descriptor per window)
 * lives in a fixed array inside the library's device image: two descriptors per window up to DAF_STATIC_MAX_WINDOWS,
 * 1 MiB + 256 B, held by every GPU that loads the library until the process exits.
 *
 * Arguments as for daf_compress, minus the workspace.  d_status (device, 4-byte aligned, may be
 * NULL) receives the device status word (a daf_status) once the stream reaches that point.
 *   - Tensors with more than DAF_STATIC_MAX_WINDOWS windows (2^30 elements at the default window
 *     of 16384) are rejected with DAF_ERR_CAPACITY before anything is enqueued.
 *   - The call allocates and frees nothing, on host or device.  The first call on each device
 *     looks up the array's device address (with that device current); make that first call
 *     outside any stream capture.
 *   - Every call uses the same array.  The part a call needs is cleared on the stream first, so
 *     stale contents of an earlier call never matter, but two calls that overlap on the GPU (on
 *     different streams, or from different threads) race on it: serialise them.
 */
#define DAF_STATIC_MAX_WINDOWS 65536
daf_status daf_compress_static(const daf_params *params, const void *d_in, void *d_packed,
                               uint64_t packed_capacity, uint8_t *d_bits, float *d_min,
                               float *d_scale, uint64_t *d_window_offsets, uint32_t *d_status,
                               daf_stream stream);

/*
 * Per-tensor statistics and per-tensor quantization: Eq. 1 at the granularity the paper states it (one min, max and
 * width per activation tensor; the group-wise calls above are the refinement the library is built around), with the
 * collective reduction of Sec. 3.2.1-3.2.2 behind it: tree reduction inside a CTA, one integer atomic per CTA and
 * statistic across CTAs (the paper's hybrid of both; its compare-and-swap loop on floats is replaced by a native
 * atomic max on a monotone integer key).  No workspace; nothing is allocated.
 *
 *   d_in / d_out : numel elements of dtype (a daf_dtype); numel a positive multiple of 8 (DAF_ERR_SHAPE otherwise);
 *                  32-byte aligned for DAF_F32, 16 otherwise.
 *   d_stats      : device, 32 bytes, 16-byte aligned.  daf_tensor_minmax writes float words [0] min, [1] max (under the
 *                  order in which -0 < +0), [2] range = max - min, or 0 when that is below 2^-118 (the tensor then
 *                  counts as constant); words 4-7 are scratch.  daf_tensor_compress reads words 0 and 2.
 *   d_packed     : numel * width / 8 bytes, 16-byte aligned; code i occupies bits [i*width, (i+1)*width), LSB first.
 *   d_min_scale  : device, two floats: the minimum and scale = range / (2^width - 1) (0 for a constant tensor),
 *                  written by daf_tensor_compress, read by daf_tensor_decompress.
 *   width in {1,2,4,8}; rounding, seed, elem_index_base (a multiple of 8) as in daf_params: element i draws the 16-bit
 *   lane (elem_index_base + i) & 7 of Philox block (elem_index_base + i) >> 3, exactly as the group-wise path does.
 * The code of element i is min((RNE((x_i - min) * fl(L / range) * 2^15) + r15) >> 15, L) with L = 2^width - 1, i.e. the
 * group-wise arithmetic with the whole tensor as the one group; decompress gives fma(code, scale, min) rounded to dtype.
 * Errors: INVALID_ARG (null or misaligned pointer, bad dtype / width / rounding / base), SHAPE, CUDA.
 */
daf_status daf_tensor_minmax(uint32_t dtype, const void *d_in, uint64_t numel, void *d_stats, daf_stream stream);
daf_status daf_tensor_compress(uint32_t dtype, const void *d_in, uint64_t numel, uint32_t width, uint32_t rounding,
                               uint64_t seed, uint64_t elem_index_base, const void *d_stats, void *d_packed,
                               float *d_min_scale, daf_stream stream);
daf_status daf_tensor_decompress(uint32_t dtype, const void *d_packed, uint64_t numel, uint32_t width,
                                 const float *d_min_scale, void *d_out, daf_stream stream);

/*
 * Host-side page pool for packed buffers (Sec. 3.4.2: one preallocated contiguous arena,
 * page-granular first-fit allocation; Sec. 3.4.3: every allocation carries an importance,
 * and the least important one is evicted first).  The pool does bookkeeping only: it never
 * touches the arena's memory, which the caller allocates (device or host) and describes by
 * its size.  Not thread safe.  Handles are positive; 0 means "no allocation".
 */
typedef struct daf_pool daf_pool;
typedef struct daf_pool_stats {
    uint64_t arena_bytes, page_bytes, pages_total, pages_used, live_allocations,
             bytes_requested, largest_free_run_pages, evictions;
} daf_pool_stats;
daf_pool  *daf_pool_create(uint64_t arena_bytes, uint64_t page_bytes /* 0 => 65536 */);
void       daf_pool_destroy(daf_pool *pool);
/* Returns a handle and the byte offset of the run inside the arena, or 0 if no run fits. */
uint64_t   daf_pool_alloc(daf_pool *pool, uint64_t bytes, double importance, uint64_t *offset);
daf_status daf_pool_free(daf_pool *pool, uint64_t handle);
/* Frees the live allocation with the lowest importance per byte; returns its handle (0 if none). */
uint64_t   daf_pool_evict_lowest(daf_pool *pool);
daf_status daf_pool_get_stats(const daf_pool *pool, daf_pool_stats *stats);

/*
 * Importance-aware store: which saved activations are kept, at which width, and where in a paged
 * arena (Sec. 3.4).  Host bookkeeping only, like daf_pool: the caller owns the arena, compresses
 * into the offsets the store hands out, and performs the moves a shrinking budget asks for.
 *
 *   Sec. 3.4.1  Greedy choice across activations under a memory AND a time budget: while a budget
 *               is exceeded, the constraint with the smaller remaining proportion is the tighter
 *               one, and the activation worth least per unit of that resource gives way (ties:
 *               least per unit of the other resource).  Width 0 = the activation is not stored.
 *   Alg. 3      Two ordered indices (red-black trees) over the same activations, keyed
 *               importance / size and importance / time, always updated together.  Under memory
 *               pressure an activation not yet placed this iteration gives way by going one width
 *               down (below the smallest allowed width it is dropped); one that already occupies
 *               pages is evicted; under time pressure the victim is always evicted.  The paper
 *               does not say at which end of an index the victim sits; here it is the entry with
 *               the LEAST importance per unit.
 *   Sec. 3.4.2  First fit over the free pages.
 *   Sec. 3.4.4  The arena starts at one step (step_bytes, 100 MB when 0), grows by a step (never
 *               past the memory budget) when an allocation finds no run, and shrinks in steps when
 *               daf_store_set_budget lowers the budget: allocations beyond the new end move to the
 *               first fit below it (reported as moves) or are evicted.
 *
 * Sizes: an activation of numel elements at width b counts daf_store_bytes(numel, G, b) bytes: its
 * window offsets (8*(ceil(numel/16384)+1)), min and scale (4*numel/G each), codes (numel*b/8) and widths
 * (numel/G), in this order, each part rounded up to 16 bytes; the sum is rounded up to pages.
 * Time: the caller's estimate of what storing the activation costs per iteration (compress +
 * decompress), in any unit; it counts while the activation is kept, at any width.
 *
 * Per iteration: daf_store_estimate for every activation (Alg. 3, pre-iteration estimation, with
 * the moving-average importance), then, in forward order, daf_store_admit when the activation and
 * its measured importance arrive (returns the width to compress at and the arena offset), and
 * daf_store_release once the backward pass has consumed it.
 * daf_store_estimate, daf_store_admit and daf_store_set_budget report the ids that lost their place in
 * the call (the id itself included when it was dropped): what an evicted id held in the arena is no
 * longer the caller's, the pages may be handed out again at once.
 * Errors: DAF_ERR_INVALID_ARG for null handles, unknown ids, negative or NaN importance / time,
 * numel not a multiple of group_size, an activation admitted twice.  Output arrays: *n on entry is
 * the array's capacity, on return the number of items there were (items beyond the capacity are
 * not written).
 */
typedef struct daf_store daf_store;
typedef struct daf_store_config {
    uint64_t mem_budget_bytes;   /* B_mem: upper bound on the arena                          */
    double   time_budget;        /* B_time, in the unit of the time costs                     */
    uint64_t page_bytes;         /* 0 => 65536                                                */
    uint64_t step_bytes;         /* arena growth / shrink step; 0 => 100 MB (100 * 2^20)      */
    uint32_t width_mask;         /* allowed widths, as in daf_params                          */
    uint32_t reserved;           /* 0                                                         */
} daf_store_config;
typedef struct daf_store_move { uint64_t id, from_offset, to_offset, bytes; } daf_store_move;
typedef struct daf_store_stats {
    uint64_t arena_bytes, mem_budget_bytes, used_bytes, planned_bytes;
    double   time_budget, used_time;
    uint64_t entries, kept, evictions, resizes, grows, shrinks, moves;
} daf_store_stats;
uint64_t   daf_store_bytes(uint64_t numel, uint32_t group_size, uint32_t width);
daf_store *daf_store_create(const daf_store_config *config);       /* NULL on bad config */
void       daf_store_destroy(daf_store *store);
daf_status daf_store_estimate(daf_store *store, uint64_t id, uint64_t numel, uint32_t group_size,
                              double importance, double time_cost, uint32_t *width,
                              uint64_t *evicted_ids, uint32_t *n_evicted);
daf_status daf_store_admit(daf_store *store, uint64_t id, double importance, uint32_t *width,
                           uint64_t *offset /* UINT64_MAX when not stored */,
                           uint64_t *evicted_ids, uint32_t *n_evicted);
/* Current width (0 = dropped) and offset (UINT64_MAX = not in pages) of an activation. */
daf_status daf_store_width(const daf_store *store, uint64_t id, uint32_t *width, uint64_t *offset);
daf_status daf_store_release(daf_store *store, uint64_t id);
daf_status daf_store_set_budget(daf_store *store, uint64_t mem_budget_bytes, double time_budget,
                                daf_store_move *moves, uint32_t *n_moves,
                                uint64_t *evicted_ids, uint32_t *n_evicted);
daf_status daf_store_get_stats(const daf_store *store, daf_store_stats *stats);

const char *daf_status_string(daf_status status);
uint32_t    daf_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DAF_H */
