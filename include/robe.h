/*
 * robe.h - C ABI of the B200 (sm_100a) ROBE-Z embedding library.
 *
 * ROBE (Random Offset Block Embedding array, arXiv 2108.02191) replaces all
 * embedding tables of a recommendation model by ONE circular array M of m learned
 * scalars.  The d-dimensional embedding of token x of table e is assembled from
 * ceil(d/Z) blocks of Z consecutive array elements; block c starts at the
 * universal-hash offset h(e,x,c) and wraps around the end of the array
 * (Section 3.1 "ROBE-D", Section 3.2 "ROBE-Z").  The backward pass adds the
 * output gradients back into the slots they were read from (Section 3.1,
 * backward equation).
 *
 * Conventions shared by every entry point
 *   - All sizes are in ELEMENTS unless a name says bytes.
 *   - "device pointer" = memory of the CUDA device that is current when the call
 *     is made; "host pointer" = ordinary host memory.  The library never
 *     allocates or frees device memory, and never synchronises, except where an
 *     entry point says otherwise.
 *   - Bags are sample-major.  With T tables and a batch of B samples there are
 *     B*T bags; bag k = n*T + e belongs to sample n and table e = k mod T and
 *     covers indices[offsets[k] .. offsets[k+1]).  offsets == NULL means one id
 *     per bag (one-hot): bag k is indices[k] and nnz must equal B*T.
 *   - Output / output-gradient element (n, e, i) lives at ((n*T + e)*d + i).
 *   - Every function returns a robe_status; invalid arguments launch nothing.
 *     No exception, abort or device trap crosses this boundary.
 *   - Launches are asynchronous on the given stream (a cudaStream_t passed as
 *     void*; NULL is the legacy default stream).
 */
#ifndef ROBE_H_
#define ROBE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct robe_ctx* robe_handle_t; /* opaque; host memory owned by the library */

typedef enum {
    ROBE_OK = 0,
    ROBE_ERR_INVALID_ARG = -1, /* null pointer, zero size, d > M, Z > d not a multiple of d, M + d > 2^32, ... */
    ROBE_ERR_NO_ARRAY = -2,    /* forward/backward before robe_attach_array            */
    ROBE_ERR_WORKSPACE = -3,   /* deterministic backward: workspace missing/too small  */
    ROBE_ERR_CUDA = -4,        /* the CUDA runtime reported an error at launch         */
    ROBE_ERR_UNSUPPORTED = -5  /* valid request that this build does not implement     */
} robe_status;

/* array element types */
#define ROBE_F32 0
#define ROBE_BF16 1

/* option keys for robe_set_option */
#define ROBE_OPT_SIGN 1     /* 0 (default) | 1: multiply by the sign hash g(e,x,i)        */
#define ROBE_OPT_BWD_MODE 2 /* ROBE_BWD_ATOMIC (default) | ROBE_BWD_DETERMINISTIC | ROBE_BWD_BINNED */
#define ROBE_OPT_VALIDATE 3 /* 0 (default) | 1: range-check ids/offsets on the device and
                               record the first violation in a status word instead of
                               using the bad value.  The word is sticky: while it is
                               non-zero EVERY kernel of EVERY later call on the handle
                               returns at once - robe_forward leaves `out` as it was
                               (not overwritten), robe_forward_keep keeps nothing, the
                               backward calls add nothing - and the host call still
                               returns ROBE_OK.  Read it with robe_last_device_status
                               and zero it yourself before going on.                      */
#define ROBE_OPT_FWD_KERNEL 4 /* forward kernel; every variant gives the same bits.
                                 0 automatic (default): the lane-hashed kernel for Z <= 2 on arrays of
                                   up to 192 MB, the staged kernel for rows of up to 128 elements, else
                                   the direct kernel
                                 1 direct: any (Z, d); every lane hashes its element's chunk per id
                                 2 staged: d <= 128; block starts of a batch of ids through shared
                                   memory, 4-byte loads, lanes on consecutive slots of a block
                                 3 vector: 16-byte loads of the aligned pieces around a block, shifted
                                   in registers; fp32 array, d, Z and M multiples of 4, d <= 128, sign
                                   off (measured slower than 2 on every workload; kept for comparison)
                                 4 lane-hashed: d <= 128, Z <= d, sign off; chunks hashed in registers by
                                   the lane that owns the element, persistent warps
                                 A variant asked for a call it cannot take returns
                                 ROBE_ERR_UNSUPPORTED and launches nothing.                          */
#define ROBE_OPT_BWD_KERNEL 5 /* kernel of the ATOMIC backward (all within the atomic bound):
                                 0 automatic (default): staged for d <= 128, else direct
                                 1 direct   2 staged (scalar red.global.add.f32, lanes on consecutive slots)
                                 3 vector: red.global.add.v4.f32 on the aligned middle of a block,
                                   scalar head and tail; d, Z, M multiples of 4, d <= 128, sign off
                                   (measured slower than 2; kept for comparison)
                                 4 vector, repeats of an id inside a staged batch merged first
                                 5 merged rows: one-hot input, sign off, d <= 128; a warp takes up to 64
                                   rows of ONE table, sums the gradient rows of repeated ids in
                                   registers and issues one reduction per element for all of them -
                                   pays for skewed (Zipf) ids with long blocks (Z = 128: 1.34 x), costs
                                   10-40 % on uniform ids, so it is the caller's choice
                                 6 lane-hashed: d <= 128, Z <= d, sign off (the reductions, not the
                                   hashing, bound this pass: measured no faster than 2)              */

#define ROBE_OPT_INDEX_TYPE 6 /* ROBE_I64 (default) | ROBE_I32: element type of `indices` in the
                                 calls that follow (offsets stay int64)                   */

#define ROBE_OPT_BAG_LAYOUT 7 /* ROBE_BAGS_SAMPLE_MAJOR (default): bag k = n*T + e, out and grad_out are
                                 [batch, T, d];  ROBE_BAGS_TABLE_MAJOR: bag k = e*batch + n - the ids of
                                 table 0 for all samples, then table 1, ... (per-table id lists laid end
                                 to end) - and out and grad_out are [T, batch, d].  Applies to the calls
                                 that follow; offsets index bags in the chosen order.              */
#define ROBE_BAGS_SAMPLE_MAJOR 0
#define ROBE_BAGS_TABLE_MAJOR 1

#define ROBE_OPT_ARRAY_L2_KEEP 8 /* 0 (default) on | 1 off: the reductions of the atomic and the binned
                                    backward carry the L2 cache policy "evict these lines last"
                                    (createpolicy ... L2::evict_last), so that a gradient target about
                                    the size of the L2 stays there next to the streamed ids and gradient
                                    rows: 19-35 % faster on a 100 MB array, no slower elsewhere.  Results
                                    are unchanged.  (The same policy on the forward's loads measured no
                                    effect and is not offered.)                                      */

/* index element types */
#define ROBE_I64 0
#define ROBE_I32 1

#define ROBE_BWD_ATOMIC 0
#define ROBE_BWD_DETERMINISTIC 1
#define ROBE_BWD_BINNED 2

/* values of the device status word (robe_last_device_status) */
#define ROBE_DEV_OK 0
#define ROBE_DEV_BAD_INDEX 1  /* an id was negative                         */
#define ROBE_DEV_BAD_OFFSETS 2 /* offsets not monotone or out of [0, nnz]   */

/*
 * robe_create - make a handle for one ROBE array shape (Section 3.2).
 *   out         host pointer receiving the handle.
 *   M           array length m = |M| in elements; 1 <= d <= M and M + d <= 2^32.
 *   Z           block size.  1 <= Z <= d: Z = d is ROBE-D (one block per embedding,
 *               Section 3.1); Z = 1 hashes every element on its own (Section 3.3); if Z
 *               does not divide d the last block is short.  Z > d (Section 3.2, last
 *               paragraph: several embeddings clubbed into one chunk): Z must be a
 *               multiple of d and <= M; rows floor(x/R) R .. + R-1 of a table, R = Z/d,
 *               then share the block that starts at h(e, floor(x/R), 0), row x being the
 *               piece [(x mod R) d, (x mod R) d + d) of it.
 *   d           embedding dimension (one d per handle; several handles may share
 *               one array, Section 3.1 "Multiple embedding tables").
 *   num_tables  T >= 1; the table id e of bag k is k mod T (k / batch after
 *               ROBE_OPT_BAG_LAYOUT = ROBE_BAGS_TABLE_MAJOR).
 *   hash_seed   seeds the draw of the hash constants: P = 2^61 - 1 and, from a
 *               SplitMix64 stream, A_h B_h C_h D_h A_g B_g C_g D_g (61-bit draws,
 *               redrawn when outside [1,P-1] for multipliers / [0,P-1] for the
 *               additive terms), as the paper's hash family requires.
 * A handle holds options and, after the first deterministic backward, a CUDA stream and two
 * events of its own (no device memory) on the device that was current at that call; a
 * deterministic backward made later with another device current runs in the caller's stream
 * alone.  Calls on ONE handle must not overlap in time on the host; different handles are
 * independent.
 * Errors: ROBE_ERR_INVALID_ARG.
 */
int robe_create(robe_handle_t* out, uint64_t M, uint32_t Z, uint32_t d, uint32_t num_tables,
                uint64_t hash_seed);

/* robe_destroy - free the host handle (waits for the handle's own stream, if it has one).  Device
 * buffers stay the caller's. */
int robe_destroy(robe_handle_t h);

/* robe_set_option - see the ROBE_OPT_* keys.  ROBE_ERR_INVALID_ARG on a bad key/value. */
int robe_set_option(robe_handle_t h, int key, int64_t value);

/*
 * robe_attach_array - name the parameter array M (Section 3: the one array that holds the
 * learned parameters of all tables).
 *   dev_array  device pointer to M elements of `dtype`, 16-byte aligned, owned by the
 *              caller, read by forward and updated in place by the fused-SGD backward.
 *   dtype      ROBE_F32 or ROBE_BF16 (bf16 is read-only: widened exactly to fp32).
 */
int robe_attach_array(robe_handle_t h, void* dev_array, int dtype);

/*
 * robe_get_hash_constants - copy out {P, A_h, B_h, C_h, D_h, A_g, B_g, C_g, D_g}
 * (host pointer to 9 words) so that a checker can be handed numbers, not code.
 *   h(e,x,c) = ((A_h e + B_h x + C_h c + D_h) mod P) mod M           (Section 3.2)
 *   g(e,x,i) = 2 (((A_g e + B_g x + C_g i + D_g) mod P) mod 2) - 1   (Section 3.1)
 */
int robe_get_hash_constants(robe_handle_t h, uint64_t out[9]);

/*
 * robe_forward - embedding lookup with optional sum pooling (Section 3.2 forward).
 *   out[n,e,i] = sum over ids x_p of bag (n,e), in bag order, sequentially in fp32
 *                (first term initialises), of g(e,x_p,i) * M[(h(e,x_p,i/Z) + i%Z) mod M]
 *   indices  device pointer, int64 [nnz] (int32 [nnz] after ROBE_OPT_INDEX_TYPE = ROBE_I32),
 *            ids >= 0.
 *   offsets  device pointer, int64 [batch*T + 1], offsets[0] = 0, non-decreasing,
 *            offsets[batch*T] = nnz; or NULL for one-hot (then nnz == batch*T).
 *   batch    number of samples B >= 0;  nnz >= 0 total ids.
 *   out      device pointer, fp32 [batch, T, d] ([T, batch, d] with ROBE_BAGS_TABLE_MAJOR), fully
 *            overwritten; an empty bag gives +0.
 * Errors: ROBE_ERR_INVALID_ARG, ROBE_ERR_NO_ARRAY, ROBE_ERR_CUDA.
 */
int robe_forward(robe_handle_t h, const void* indices, const int64_t* offsets, int64_t batch,
                 int64_t nnz, float* out, void* stream);

/*
 * robe_backward_workspace_bytes - bytes of caller-provided device scratch that
 * robe_backward needs in the handle's current backward mode for a call of this
 * size (0 in atomic mode; binned and deterministic mode need the same).  Returns 0 for a
 * bad handle.
 */
size_t robe_backward_workspace_bytes(robe_handle_t h, int64_t batch, int64_t nnz);

/*
 * robe_backward - scatter-add of the output gradient (Section 3.1 backward equation):
 *   delta[j] = sum over (p, i) with idx(e, x_p, i) = j of g(e,x_p,i) * grad_out[bag(p), i]
 * every occurrence of an id contributes, duplicates included.
 *   grad_out    device pointer, fp32 [batch, T, d].
 *   grad_array  device pointer, fp32 [M]: delta is ADDED to it (the caller zeroes it
 *               when a plain gradient is wanted).  NULL selects the fused SGD step
 *               M[j] <- M[j] - lr * delta[j] applied in place to the attached fp32
 *               array (the paper trains its DLRM with plain SGD, Section 5).
 *   lr          learning rate, used only when grad_array == NULL.
 *   workspace   device pointer to workspace_bytes bytes, 256-byte aligned; may be NULL
 *               in atomic mode.
 * Atomic mode adds with red.global (fp32, order not fixed).  Binned mode does the same adds
 * after grouping the blocks by array region (one radix pass on the top bits of the block
 * start), so that the read-modify-write of an array much larger than the L2 happens in L2; it
 * needs the workspace of the deterministic mode and gives atomic-mode accuracy, not
 * reproducible bits.  Deterministic mode sorts
 * the blocks by start offset (stable) and lets each array slot sum its terms in that
 * order in fp32 from +0, then applies ONE add (dense) or ONE fma (SGD) per touched
 * slot: results are bit-reproducible.
 * Errors: ROBE_ERR_INVALID_ARG (also: fused SGD on a bf16 array), ROBE_ERR_NO_ARRAY,
 * ROBE_ERR_WORKSPACE, ROBE_ERR_CUDA.
 */
int robe_backward(robe_handle_t h, const float* grad_out, const void* indices,
                  const int64_t* offsets, int64_t batch, int64_t nnz, float* grad_array, float lr,
                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * robe_forward_keep / robe_backward_kept - the forward and backward of one training step on
 * the same ids, sharing the hash work.  The block starts h(e, x_p, c) that the forward computes
 * (Section 3.2) are what the binned and the deterministic backward sort by; robe_forward_keep
 * is robe_forward that also stores them in `workspace`, and robe_backward_kept is
 * robe_backward that takes them from there instead of hashing every id again.  The paper has
 * no counterpart: it is a fusion across the two passes, results are those of robe_forward and
 * robe_backward bit for bit (deterministic mode) or within the same bound (binned mode).
 *   workspace  device pointer, 256-byte aligned, at least robe_backward_workspace_bytes(h,
 *              batch, nnz) bytes; owned by the caller, who leaves it untouched between the two
 *              calls.  The backward consumes what was kept: one robe_backward_kept per
 *              robe_forward_keep.
 *   The two calls get the same indices, offsets, batch and nnz, with the handle's sign,
 *   index-type and backward-mode options unchanged in between.  The backward trusts what the
 *   workspace holds: after anything else (other sizes, a workspace written to in between, no
 *   robe_forward_keep before) its behaviour is undefined, as for a wrong pointer.
 * In atomic mode nothing is sorted: the two calls are then robe_forward and robe_backward, and
 * workspace may be NULL.
 * Errors: those of robe_forward and robe_backward; ROBE_ERR_UNSUPPORTED and
 * ROBE_ERR_WORKSPACE already from robe_forward_keep.
 */
int robe_forward_keep(robe_handle_t h, const void* indices, const int64_t* offsets, int64_t batch,
                      int64_t nnz, float* out, void* workspace, size_t workspace_bytes, void* stream);
int robe_backward_kept(robe_handle_t h, const float* grad_out, const void* indices,
                       const int64_t* offsets, int64_t batch, int64_t nnz, float* grad_array, float lr,
                       void* workspace, size_t workspace_bytes, void* stream);

/*
 * robe_backward_adam - deterministic backward with the Adam step fused in (the paper trains
 * five of its six Criteo-Kaggle models with Adam, Section 5; the update is Algorithm 1 of
 * Kingma & Ba, "Adam: a method for stochastic optimization").  For every array slot j that
 * receives at least one gradient term, with delta[j] summed in the deterministic order of
 * robe_backward:
 *     m1[j] = beta1 m1[j] + (1 - beta1) delta[j]
 *     m2[j] = beta2 m2[j] + (1 - beta2) delta[j]^2
 *     M[j]  = M[j] - lr * (m1[j] / (1 - beta1^step)) / (sqrt(m2[j] / (1 - beta2^step)) + eps)
 * each operation a separate round-to-nearest fp32 one; slots without a term keep M, m1 and m2
 * as they are (the "lazy" form that sparse embedding updates use).  Bit-reproducible.
 *   m1, m2   device pointers, fp32 [M], caller-owned, zeroed by the caller before step 1.
 *   step     t >= 1, the number of this update (used for the bias corrections only).
 *   workspace / workspace_bytes  as for robe_backward in deterministic mode; size it with
 *            robe_backward_workspace_bytes after ROBE_OPT_BWD_MODE = ROBE_BWD_DETERMINISTIC.
 * The handle's ROBE_OPT_BWD_MODE is not consulted.  The attached array must be fp32.
 * Errors: as robe_backward; ROBE_ERR_INVALID_ARG also for null moments, step < 1, beta outside
 * [0, 1) or eps < 0.
 */
int robe_backward_adam(robe_handle_t h, const float* grad_out, const void* indices,
                       const int64_t* offsets, int64_t batch, int64_t nnz, float* m1, float* m2,
                       float lr, float beta1, float beta2, float eps, int64_t step, void* workspace,
                       size_t workspace_bytes, void* stream);

/*
 * robe_backward_adagrad - deterministic backward with the Adagrad step fused in (Duchi, Hazan, Singer,
 * "Adaptive subgradient methods ..."; the optimizer recommendation models are commonly trained with,
 * beside the SGD and Adam of the paper's Section 5).  Embedding tables usually keep ONE accumulator
 * per row ("row-wise Adagrad"); the ROBE array has no rows - a slot is shared by elements of many
 * rows of many tables - so the accumulator is per slot.  For every array slot j that receives at
 * least one gradient term, with delta[j] summed in the deterministic order of robe_backward:
 *     sum_sq[j] = sum_sq[j] + delta[j]^2
 *     M[j]      = M[j] - lr * delta[j] / (sqrt(sum_sq[j]) + eps)
 * each operation a separate round-to-nearest fp32 one; other slots keep M and sum_sq.  Bit-reproducible.
 *   sum_sq   device pointer, fp32 [M], caller-owned, zeroed by the caller before the first step.
 *   workspace / workspace_bytes  as for robe_backward in deterministic mode.
 * The handle's ROBE_OPT_BWD_MODE is not consulted.  The attached array must be fp32.
 * Errors: as robe_backward; ROBE_ERR_INVALID_ARG also for a null sum_sq or eps < 0.
 */
int robe_backward_adagrad(robe_handle_t h, const float* grad_out, const void* indices,
                          const int64_t* offsets, int64_t batch, int64_t nnz, float* sum_sq, float lr,
                          float eps, void* workspace, size_t workspace_bytes, void* stream);

/*
 * robe_apply_sgd - the dense SGD apply of a data-parallel training step (Section 1 of the
 * paper, implications of the compression: the whole model fits every GPU, so training is plain
 * data-parallel and the ranks exchange one gradient the size of the array; Section 5: SGD).
 * A rank runs robe_backward with a dense grad_array on its shard of the batch, the caller
 * sums grad_array over the ranks (an all-reduce: 4 M bytes), and this call applies the sum
 *     M[j] <- fma(-lr, grad_array[j], M[j])       for every j < M
 * to the attached fp32 array in one streaming pass.  On one rank it gives the bits of the
 * fused step (robe_backward with grad_array == NULL) when grad_array held +0 before the
 * deterministic backward ran.
 *   grad_array  device pointer, fp32 [M], 16-byte aligned; with zero_grad = 1 it is left
 *               holding +0 everywhere, ready for the next step's robe_backward.
 *   zero_grad   0 or 1.
 * Errors: ROBE_ERR_INVALID_ARG (null or misaligned pointer, bf16 array), ROBE_ERR_NO_ARRAY,
 * ROBE_ERR_CUDA.
 */
int robe_apply_sgd(robe_handle_t h, float* grad_array, float lr, int zero_grad, void* stream);

/*
 * robe_backward_deterministic_static - the deterministic robe_backward for callers that
 * cannot supply scratch memory.  (The paper has no counterpart: this is a convenience of
 * this library, not part of the method.)
 *
 * Who needs it: code that runs where device allocation is off the table - for example a
 * serving process whose memory pool already owns the whole device, so a cudaMalloc would
 * fail or stall every stream while it synchronises the device, or an operator plugged
 * into a host framework that hands it input and output buffers and nothing else.  Such a
 * caller has no way to come up with the workspace robe_backward asks for in
 * deterministic mode.  Here the workspace is a fixed array of ROBE_STATIC_SCRATCH_BYTES
 * that is part of the library image itself: every device that loads librobe.so carries
 * it from load until the process exits, whether or not this function is ever called.
 *
 * Arguments and result are those of robe_backward in ROBE_BWD_DETERMINISTIC mode (the
 * handle's ROBE_OPT_BWD_MODE is ignored), minus workspace/workspace_bytes: the caller
 * still passes grad_out, indices, offsets and grad_array (or NULL for the fused SGD step),
 * and gets bit-identical output.  The function calls no cudaMalloc, cudaFree or other
 * allocating routine.
 *
 * Limit: the call must fit the fixed array, i.e. the value robe_backward_workspace_bytes
 * reports for it in deterministic mode (about 19 bytes per block, nnz * ceil(d/Z) blocks,
 * plus 4 bytes per id, 0.7 MB of counters and lists, and the window bounds of the array:
 * M/57 bytes for arrays under 2 M slots, M/228 bytes above) must not exceed
 * ROBE_STATIC_SCRATCH_BYTES; a larger call returns ROBE_ERR_WORKSPACE and launches nothing.
 *
 * First call on a device: the function looks up the device address of the array once per
 * device (with that device current) and remembers it.  Make that first call during
 * set-up, before any stream capture is begun.
 *
 * Sharing: all handles, streams and threads of the process use the same array on a given
 * device, and it keeps whatever the previous call left in it.  The function re-initialises
 * the parts that must start from zero on every call, so back-to-back calls on ONE stream
 * are safe; two calls that may overlap on the GPU (different streams without an ordering
 * between them) race on the array and give undefined results - order them yourself.
 *
 * Errors: as robe_backward, plus ROBE_ERR_WORKSPACE for a call beyond the limit and
 * ROBE_ERR_CUDA if the address lookup fails.
 */
#define ROBE_STATIC_SCRATCH_BYTES (32u << 20) /* 32 MiB per device */
int robe_backward_deterministic_static(robe_handle_t h, const float* grad_out,
                                       const void* indices, const int64_t* offsets,
                                       int64_t batch, int64_t nnz, float* grad_array, float lr,
                                       void* stream);

/*
 * robe_set_status_word - give the handle a device int32 (caller-owned, zeroed by the
 * caller) that kernels write a ROBE_DEV_* code into when ROBE_OPT_VALIDATE is on.  Only the
 * first violation is recorded (compare-and-swap from ROBE_DEV_OK), and a non-zero word turns
 * all later launches on the handle into no-ops until the caller zeroes it (see
 * ROBE_OPT_VALIDATE).
 * robe_last_device_status - synchronise `stream`, read that word (device-to-host copy)
 * and return it (>= 0), or a negative robe_status.
 */
int robe_set_status_word(robe_handle_t h, int32_t* dev_word);
int robe_last_device_status(robe_handle_t h, void* stream);

/*
 * robe_debug_status / robe_debug_selftest - the index-check build (librobe_debug.so: the same
 * sources compiled with -DROBE_DEBUG; it stands in for a memory checker on machines where none can
 * be run).  In that build every computed index of every kernel - array slots, sorted positions,
 * shared-memory offsets, positions in grad_out, window and hand-over record numbers - is compared
 * with its bound before use; a violation records a ROBE_DBG_* code (the first one sticks) and the
 * access is skipped: nothing traps, the context stays usable.  robe_debug_status synchronises
 * `stream`, returns the recorded code (0 = none; see the ROBE_DBG_* values below) and clears it.
 * robe_debug_selftest launches one kernel that fails a check on purpose WITHOUT touching memory
 * (code 99), to show that the reporting path works.  The release library performs no check and
 * returns ROBE_ERR_UNSUPPORTED from both.
 */
#define ROBE_DBG_ARRAY_SLOT 1
#define ROBE_DBG_SORT_POS 2
#define ROBE_DBG_SHARED 3
#define ROBE_DBG_GRAD_POS 4
#define ROBE_DBG_WINDOW 5
#define ROBE_DBG_LONG_WALK 6
#define ROBE_DBG_SELFTEST 99
int robe_debug_status(void* stream);
int robe_debug_selftest(void* stream);

/* robe_status_string - static host string for a robe_status value. */
const char* robe_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* ROBE_H_ */
