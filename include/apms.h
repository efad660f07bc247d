/*
 * apms.h - C ABI of the APMSqueeze compressed-step library for NVIDIA B200 (sm_100a).
 *
 * The library runs the data-parallel hot path of APMSqueeze on ONE GPU, with the n
 * data-parallel workers simulated as n device-resident buffer sets and the two exchanges
 * of the Gather-Scatter AllReduce (Figure 1) replaced by direct indexing of device memory:
 *
 *   warmup phase       full-precision Adam with bias correction on the worker-averaged
 *                      gradient (Algorithm 1 line 2; Section 3.2);
 *   phase switch       the variance v is frozen, all compression errors start at zero
 *                      (Section 3.3, first paragraph; Algorithm 1 initialisation);
 *   compression phase  per step, for every chunk: every worker forms its local momentum,
 *                      adds its compression error, compresses to sign bits + one scale and
 *                      keeps the new error; the chunk's server averages the n decompressed
 *                      messages, adds its own error, recompresses and keeps its new error;
 *                      every worker replaces its momentum by the decompressed server message
 *                      and updates the model with the frozen variance
 *                      (Section 3.3 steps 1-6 = Algorithm 1 lines 4-11; Supplement A).
 *
 * Compressor (Section 5.1): sign bits + scale = ||z||_2 / sqrt(L) per chunk of L elements,
 * so that the decompressed chunk has the l2 norm of the compensated chunk z.
 *
 * Conventions
 *   - All state is binary32; sums of squares are accumulated in binary64.  Every operation
 *     is rounded once (no fused contraction except the momentum update's single fma).
 *   - A chunk is `chunk` consecutive elements of the flat parameter vector (a positive
 *     multiple of 32); the last chunk may be shorter and is scaled by its true length.
 *     C = ceil(d / chunk) chunks, W = ceil(d / 32) sign words.
 *   - Sign words: uint32 word w, bit j (LSB = bit 0) holds element 32*w + j; 1 means
 *     value >= 0 (so +0.0 and -0.0 give 1, NaN gives 0); bits past d are 0.
 *   - Scales: float[C] in chunk order.
 *   - "dev" pointers are device pointers valid on the context's device; "host" pointers
 *     are ordinary host memory.  Gradient arrays are HOST arrays of n pointers.
 *   - Every call enqueues its work on the context's stream and returns without a host
 *     synchronisation unless stated otherwise.  The library never traps or aborts; every
 *     failure is a status code and a message available from apms_last_error().
 *   - The library has no CPU fallback: without a CUDA device every device call fails with
 *     APMS_ERR_CUDA.
 *   - The step functions that take device gradients enqueue kernels and nothing else, so a
 *     step can be recorded by CUDA stream capture on the context's stream and replayed as a
 *     graph (not the first step of the COMPRESSED phase, which differs from the later ones, and
 *     not with timing on).  A replay repeats the device work only: the host-side counters
 *     (apms_get_step, apms_launch_count) count the capture, not the replays.
 *   - One context must not be used from two host threads at once.
 */
#ifndef APMS_H
#define APMS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct apms_ctx apms_ctx;

typedef enum {
    APMS_OK = 0,
    APMS_ERR_INVALID_ARG = 1,   /* null / misaligned pointer, size out of range            */
    APMS_ERR_BAD_STATE = 2,     /* call not allowed in the context's current phase         */
    APMS_ERR_CUDA = 3,          /* a CUDA runtime call failed; see apms_last_error()       */
    APMS_ERR_OOM = 4,           /* workspace too small, or allocation failed               */
    APMS_ERR_TIMEOUT = 5,       /* a bounded device-side wait gave up (reported by the next
                                   synchronising call; the context's state is then undefined) */
    APMS_ERR_BOUNDS = 6         /* apms_check_guards found guard bytes overwritten, or a checked
                                   accessor of the checked build refused an access          */
} apms_status;

/* Phases of Algorithm 1. */
typedef enum {
    APMS_PHASE_CREATED = 0,     /* no parameters yet                                       */
    APMS_PHASE_WARMUP = 1,      /* Adam steps (Algorithm 1 line 2)                         */
    APMS_PHASE_COMPRESSED = 2   /* v frozen, 1-bit steps (Algorithm 1 lines 3-12)          */
} apms_phase;

/* State arrays readable / writable through apms_get_state / apms_set_state. */
typedef enum {
    APMS_STATE_X = 0,              /* float[d]   model x                                   */
    APMS_STATE_V = 1,              /* float[d]   variance v (frozen after the switch)      */
    APMS_STATE_M = 2,              /* float[d]   momentum m shared by all workers          */
    APMS_STATE_WORKER_ERR = 3,     /* float[d]   worker compression error delta^(i)        */
    APMS_STATE_WORKER_BITS = 4,    /* uint32[W]  sign words worker i sent last step        */
    APMS_STATE_WORKER_SCALES = 5,  /* float[C]   scales worker i sent last step            */
    APMS_STATE_SERVER_ERR = 6,     /* float[d]   server compression error delta-bar        */
    APMS_STATE_SERVER_BITS = 7,    /* uint32[W]  sign words the servers broadcast          */
    APMS_STATE_SERVER_SCALES = 8   /* float[C]   scales the servers broadcast              */
} apms_state_id;

/* Kernels of the path, for apms_kernel_time(). */
typedef enum {
    APMS_KERNEL_WARMUP_ADAM = 0,   /* Section 3.2                                           */
    APMS_KERNEL_WORKER = 1,        /* Section 3.3 steps 1-2 (momentum + EC compression)     */
    APMS_KERNEL_SERVER = 2,        /* Section 3.3 step 4 (average + EC recompression)       */
    APMS_KERNEL_APPLY = 3,         /* Section 3.3 steps 5-6 (momentum replace + model update) */
    APMS_KERNEL_COUNT = 4
} apms_kernel_id;

/* Element type of the gradient arrays given to the *_typed step functions.  Section 5.1 counts
 * the compressor's saving for float32 and for float16 training; with 16-bit gradients a step reads
 * 2 instead of 4 bytes per worker and element.  A 16-bit gradient is widened to binary32 exactly
 * before its first use; all state and all arithmetic stay binary32 as stated above. */
typedef enum {
    APMS_GRAD_F32 = 0,    /* IEEE binary32 */
    APMS_GRAD_BF16 = 1,   /* bfloat16: the upper 16 bits of a binary32 */
    APMS_GRAD_F16 = 2     /* IEEE binary16 */
} apms_grad_type;

/* The "magnitude" in the scaling factor of Section 5.1.  The default reads it as the paper's norm:
 * scale = ||z||_2 / sqrt(L), so that the decompressed chunk has the l2 norm of the compensated one.
 * The other common reading, the mean of |z| (the least-squares scale of a sign vector), is offered as
 * a switch; it applies to the worker and the server compressor of the following steps (and runs on
 * the library's general kernels, not on the forms tuned for the default). */
typedef enum {
    APMS_SCALE_L2 = 0,
    APMS_SCALE_L1_MEAN = 1
} apms_scale_kind;

/* The compression operator C (Section 5.1 describes two).  ONEBIT is the default and the one all of the
 * above describes.  TOPK keeps, per chunk of L elements, the K = ceil(fraction * L) elements (at least one)
 * of largest absolute value and sends nothing for the others, which decompress to 0; equal magnitudes are
 * resolved in favour of the lower index; magnitudes are compared through the bit pattern of |z|.
 * In TOPK mode the context keeps, in place of the sign words, a selection mask per worker and for the
 * server (APMS_STATE_*_BITS return it: bit j = element j was sent), in place of the scales the magnitude
 * of the K-th (smallest sent) element of each chunk (APMS_STATE_*_SCALES; the next step uses it to guess
 * where its own threshold lies).  The momentum m = C[zbar] is not stored separately while it can be read
 * as (server mask ? server compensated vector : 0); APMS_STATE_M returns it spelled out.  An element
 * that the server does not keep is left untouched by the model update when that is exact (lr >= +0,
 * eps > 0, no negative or NaN entry in v); otherwise every element is updated.  Chosen with
 * apms_set_compressor until the first compression-phase step has run; TOPK works with the momentum
 * variant and the l2 scale setting, through the whole-step functions and the apms_topk_* phase-wise calls. */
typedef enum {
    APMS_COMPRESSOR_ONEBIT = 0,
    APMS_COMPRESSOR_TOPK = 1
} apms_compressor;

/* What the workers compress.  MOMENTUM is the method (Section 3.3).  GRADIENT is the comparison variant
 * "APGSqueeze" of Section 5.3 (Implementations and setups, item 4): error-compensated compression of the
 * gradient g_t instead of the momentum; per chunk
 *   worker i:  z_i = g_i + delta_i ;  s_i, bits_i, delta_i as in apms_compressed_step
 *   server:    as in apms_compressed_step; its message is a gradient ghat = +-S
 *   workers:   m <- b1 m + (1-b1) ghat  (binary32, never compressed) ;  x <- x - (lr m) / (sqrt(v) + eps)
 * All step functions of the compression phase follow the context's variant. */
typedef enum {
    APMS_VARIANT_MOMENTUM = 0,
    APMS_VARIANT_GRADIENT = 1
} apms_variant;

/* How threads are grouped on a tile of a chunk in the worker and server kernels. */
typedef enum {
    APMS_TEAM_AUTO = 0,   /* the library's choice for the shape (the forms below, per kernel)      */
    APMS_TEAM_CTA = 1,    /* always one CTA (8 warps) per tile, operands loaded by the threads      */
    APMS_TEAM_WARP = 2,   /* always one warp per tile, eight tiles per CTA                          */
    APMS_TEAM_STAGED = 3  /* one CTA per tile fed by bulk asynchronous copies through shared memory
                             wherever the shape allows it (chunk a multiple of 2048), else as AUTO  */
} apms_team_mode;

#define APMS_MAX_WORKERS 64

/* Bytes of device workspace a context of this shape needs (pure function; 0 if the shape
 * is invalid).  Covers x, v, m, the n worker and one server compensated vectors, all sign
 * words and scales, two d-float staging buffers for the host-gradient entry point, and the
 * kernels' scratch (partial sums of squares, the error monitor's sums, a status word). */
size_t apms_workspace_bytes(int64_t d, int n, int64_t chunk);

/* Create a context on the current CUDA device for d parameters and n simulated workers
 * (Problem Setting: n workers, one shared x).  beta1, beta2, eps (Adam's constant, also
 * added to sqrt(v) in the compression phase) and lr (gamma_t, changeable with
 * apms_set_lr) are the hyper-parameters of Algorithm 1.  Requires d >= 1,
 * 1 <= n <= APMS_MAX_WORKERS, chunk a positive multiple of 32.  No device memory is
 * touched until apms_bind() or the first call that needs the workspace.
 * On failure *out is NULL and apms_last_error(NULL) describes why. */
apms_status apms_create(apms_ctx** out, int64_t d, int n, float beta1, float beta2,
                        float eps, float lr, int64_t chunk);

/* Give the context caller-owned device memory (>= apms_workspace_bytes, 256-byte aligned)
 * and a CUDA stream (a cudaStream_t passed as void*; NULL = the legacy default stream).
 * The caller keeps ownership and must keep both alive until apms_destroy().  If never
 * called, the context allocates its own workspace with cudaMalloc on first use and works
 * on the default stream; workspace_dev == NULL with bytes == 0 sets the stream alone and
 * leaves the workspace to the library.  Must be called before apms_set_params(). */
apms_status apms_bind(apms_ctx* ctx, void* workspace_dev, size_t bytes, void* cuda_stream);

/* x <- x0, m <- 0, v <- 0, t <- 0 (Algorithm 1 initialisation); phase becomes WARMUP.
 * x0 holds d floats, on the device if src_is_device != 0, else on the host (the call then
 * synchronises the stream before returning). */
apms_status apms_set_params(apms_ctx* ctx, const float* x0, int src_is_device);

/* gamma_t for the following steps (Algorithm 1 takes a per-step learning rate). */
apms_status apms_set_lr(apms_ctx* ctx, float lr);

/* One Adam step (Section 3.2) on gbar = (1/n) sum_i g_i, summed in worker order:
 *   m <- b1 m + (1-b1) gbar ; v <- b2 v + (1-b2) gbar^2 ;
 *   x <- x - lr (m / (1-b1^t)) / (sqrt(v / (1-b2^t)) + eps),  t = 1 for the first call.
 * grads_dev: host array of n device pointers, each d floats, 16-byte aligned, read-only,
 * valid until the stream has passed this step.  Phase must be WARMUP. */
apms_status apms_warmup_step(apms_ctx* ctx, const float* const* grads_dev);

/* End of warmup (Section 3.3: v is no longer updated): phase becomes COMPRESSED, every
 * worker error and the server error are zero, Adam's raw m carries over. */
apms_status apms_freeze_v(apms_ctx* ctx);

/* One compression-phase step (Section 3.3 steps 1-6), for every chunk c of length L:
 *   worker i:  z_i = (b1 m + (1-b1) g_i) + delta_i ;  s_i = ||z_i||_2 / sqrt(L) ;
 *              bits_i = (z_i >= 0) ;  delta_i <- z_i - (+-s_i)
 *   server:    zbar = (1/n) sum_i (+-s_i) + dbar ;  S = ||zbar||_2 / sqrt(L) ;
 *              bits = (zbar >= 0) ;  dbar <- zbar - (+-S)
 *   workers:   m <- +-S ;  x <- x - (lr m) / (sqrt(v) + eps)
 * Same gradient-array contract as apms_warmup_step.  Phase must be COMPRESSED. */
apms_status apms_compressed_step(apms_ctx* ctx, const float* const* grads_dev);

/* The same step with the n gradients in HOST memory (pinned memory gives asynchronous
 * copies): worker i's gradient is copied to a device staging buffer while worker i-1 is
 * being compressed.  If x_out_host is not NULL the updated x (d floats) is copied back.
 * Synchronises the stream before returning. */
apms_status apms_compressed_step_host(apms_ctx* ctx, const float* const* grads_host,
                                      float* x_out_host);

/* The three step functions for gradients of another element type: the same operations on
 * g_i widened to binary32.  grads_*: host array of n pointers to d elements of `type` each,
 * aligned to 16 bytes (binary32) or 8 bytes (16-bit types).  apms_warmup_step(ctx, g) is
 * apms_warmup_step_typed(ctx, g, APMS_GRAD_F32), and so on. */
apms_status apms_warmup_step_typed(apms_ctx* ctx, const void* const* grads_dev, apms_grad_type type);
apms_status apms_compressed_step_typed(apms_ctx* ctx, const void* const* grads_dev, apms_grad_type type);
apms_status apms_compressed_step_host_typed(apms_ctx* ctx, const void* const* grads_host, apms_grad_type type,
                                            float* x_out_host);

/* A compression-phase step in its phases, for callers that carry out the two exchanges of the
 * Gather-Scatter AllReduce themselves (Figure 1; Section 3.3 steps 3 and 5) - one process per
 * GPU, each context holding its GPU's workers and serving a range of chunks:
 *
 *   apms_worker_phase   steps 1-2 for the context's n workers: leaves worker i's message (sign
 *                       words of the whole vector, one scale per chunk) where apms_get_message
 *                       points;
 *   [exchange 1: every process sends, of each of its workers' messages, the part that belongs
 *    to the chunks a peer serves, to that peer]
 *   apms_server_phase   step 4 for chunks [chunk_begin, chunk_end) from `rows` received
 *                       messages, averaged in row order: row j occupies row_words sign words
 *                       starting at bits_rows_dev + j * row_words - its word 0 is the first word
 *                       of chunk chunk_begin - and row_scales scales starting at
 *                       scale_rows_dev + j * row_scales.  row_words must be a multiple of 4 that
 *                       covers the range's words rounded up to 4; bits_rows_dev 16-byte aligned.
 *                       Writes that range of the server's message (apms_get_message(ctx, -1)).
 *                       May be called for several ranges in one step.
 *   [exchange 2: every process sends its range of the server's message to all peers, so that
 *    each holds the whole of it]
 *   apms_apply_phase    steps 5-6 over the whole vector from the server's message; ends the step.
 *
 * With rows = the total number of workers in global worker order and the ranges covering every
 * chunk once, the result equals apms_compressed_step of one context that holds all workers.
 * apms_get_message: device addresses of worker i's message (worker = -1: the server's), valid
 * while the workspace lives; the buffers hold W words / C scales, rows padded to 256 bytes. */
apms_status apms_worker_phase(apms_ctx* ctx, const void* const* grads_dev, apms_grad_type type);
/* The worker phase over chunks [chunk_begin, chunk_end) only (Section 3.3 steps 1-2 are independent per
 * chunk): after the call - in stream order - that part of every worker's message is final, so the caller
 * can hand it to the process that serves those chunks while the rest of the vector is still being
 * compressed (Section 3.3 step 3, Figure 1a).  One step's calls must cover every chunk exactly once, in any
 * order, with the same gradients; the server phases may follow once they do.  apms_worker_phase is the
 * call for [0, C). */
apms_status apms_worker_phase_range(apms_ctx* ctx, const void* const* grads_dev, apms_grad_type type,
                                    int64_t chunk_begin, int64_t chunk_end);
apms_status apms_get_message(apms_ctx* ctx, int worker, uint32_t** bits_dev, float** scales_dev);
apms_status apms_server_phase(apms_ctx* ctx, const uint32_t* bits_rows_dev, int64_t row_words,
                              const float* scale_rows_dev, int64_t row_scales, int rows,
                              int64_t chunk_begin, int64_t chunk_end);
apms_status apms_apply_phase(apms_ctx* ctx);

/* The phase-wise step with the top-k compressor (Section 5.1, second item; the compressor the paper runs on 8 GPUs
 * for ResNet-18).  On the wire a top-k message is a selection mask (one bit per element, the layout of the sign
 * words) plus the kept values in index order: K = ceil(fraction * L) values per chunk of L elements, stored
 * apms_topk_values_per_chunk() = ceil(fraction * chunk) apart (the last, shorter chunk fills fewer).  Inside a
 * context the values stay where they are (the compensated vectors); these calls pack and unpack them:
 *
 *   apms_worker_phase       (whole vector) steps 1-2; worker i's mask is its message's sign-word buffer
 *                           (apms_get_message);
 *   apms_topk_pack_values   writes the kept values of worker `worker` (-1: of the server's message, after the
 *                           server phase) for chunks [chunk_begin, chunk_end) to vals_dev (device,
 *                           (chunk_end - chunk_begin) * values_per_chunk floats);
 *   [exchange 1: masks and packed values of the chunks a peer serves go to that peer]
 *   apms_topk_server_phase  step 4 and, for the kept elements of these chunks, steps 5-6: `rows` received messages
 *                           (row j: row_words mask words from mask_rows_dev + j * row_words, word 0 = first word of
 *                           chunk chunk_begin; row_vals packed values from val_rows_dev + j * row_vals), summed in
 *                           row order.  scratch_dev: caller-owned device memory of
 *                           apms_topk_server_scratch_bytes(ctx, rows, chunk_begin, chunk_end) bytes, 16-byte aligned
 *                           (the rows are spread out there); may be reused by the next call;
 *   [exchange 2: every process's range of the server's message - mask words (apms_get_message(ctx, -1)) and packed
 *    values (apms_topk_pack_values(ctx, -1, ...)) - goes to all peers]
 *   apms_topk_put_server_range  takes over a range computed elsewhere: mask words (word 0 = first word of chunk
 *                           chunk_begin), the kept values to their places, steps 5-6 for them;
 *   apms_apply_phase        ends the step.
 *
 * The phase-wise top-k step needs the conditions under which an element that is not kept does not move (lr >= +0,
 * eps > 0, no negative or NaN entry in v; APMS_ERR_BAD_STATE otherwise).  With rows in global worker order and the
 * ranges covering every chunk once the result equals apms_compressed_step of one context holding all workers. */
int64_t     apms_topk_values_per_chunk(const apms_ctx* ctx);
/* Diagnostics of the top-k kernels (no counterpart in the paper; the selection is exact on every route): how many
 * (worker, chunk) and server chunk selections, since the last call, were settled [0] by the list of keys around the
 * threshold predicted from the earlier steps (the chunk is read once), [1] by two passes over the chunk, [2] by the
 * general radix select; and how many predictions missed (those chunks then took route 1 or 2) because the K-th key
 * lay [3] above or [4] below the listed keys or [5] the list overflowed.  Synchronises the stream and resets the
 * counters. */
apms_status apms_topk_route_counts(apms_ctx* ctx, int64_t worker_routes[6], int64_t server_routes[6]);
apms_status apms_topk_pack_values(apms_ctx* ctx, int worker, int64_t chunk_begin, int64_t chunk_end, float* vals_dev);
size_t      apms_topk_server_scratch_bytes(const apms_ctx* ctx, int rows, int64_t chunk_begin, int64_t chunk_end);
apms_status apms_topk_server_phase(apms_ctx* ctx, const uint32_t* mask_rows_dev, int64_t row_words,
                                   const float* val_rows_dev, int64_t row_vals, int rows,
                                   int64_t chunk_begin, int64_t chunk_end, void* scratch_dev, size_t scratch_bytes);
apms_status apms_topk_put_server_range(apms_ctx* ctx, const uint32_t* mask_words_dev, const float* vals_dev,
                                       int64_t chunk_begin, int64_t chunk_end);

/* The same step with the exchanges done by the GPUs themselves, for processes on one node whose
 * GPUs reach each other's memory (NVLink / NVSwitch peers): every process maps its peers' workspaces
 * (apms_ipc_export / apms_ipc_open), and
 *
 *   exchange 1 is the server kernel reading: apms_server_phase_rows takes one pair of device
 *     pointers per sender - bits_rows[j] the address of row j's sign word of the first element of
 *     chunk chunk_begin (inside a message buffer padded as the library's are; the kernel that
 *     streams the rows with bulk copies runs when all rows lie at the same distance from a 16-byte
 *     boundary, as rows of equally shaped contexts do), scale_rows[j] the address of its scale of
 *     chunk chunk_begin - and loads
 *     the rows where they lie, this GPU's memory or a mapped peer's.  A
 *     peer worker's row is (mapped base of its process) + apms_message_offsets(worker) + the range's
 *     offset; contexts created with the same d, n, chunk have the same offsets.  Both arrays are
 *     HOST arrays of `rows` pointers, read during the call.  Rows are averaged in array order.
 *   exchange 2 is a store: apms_put_server_range copies chunks [chunk_begin, chunk_end) of this
 *     context's server message into a peer's server-message buffers (dst_* = the START of the
 *     peer's sign-word / scale buffers, i.e. mapped base + apms_message_offsets(-1)), on the
 *     context's stream.
 *
 * The caller orders the phases across processes (the library has no device-side waits on other
 * GPUs): all workers' messages must be complete before any server phase reads them, and all
 * server ranges stored before any apply phase - a stream synchronisation and a host barrier at
 * each of the two points.  The paper's description of the exchanges: Section 3.3 steps 3 and 5,
 * Figure 1.  apms_ipc_export: writes APMS_IPC_HANDLE_BYTES bytes naming this context's workspace,
 * which must be the library's own allocation (no apms_bind); APMS_ERR_BAD_STATE otherwise.
 * apms_ipc_open: maps the workspace named by a handle made in ANOTHER process and returns its base
 * address in this process; apms_ipc_close unmaps it.  An exported context must outlive every
 * mapping of it: destroy it only after all processes that opened its handle have closed it.
 * apms_ipc_open and apms_ipc_close take no context; on failure apms_last_error(NULL) describes why. */
#define APMS_IPC_HANDLE_BYTES 64
apms_status apms_server_phase_rows(apms_ctx* ctx, const uint32_t* const* bits_rows, const float* const* scale_rows,
                                   int rows, int64_t chunk_begin, int64_t chunk_end);
apms_status apms_put_server_range(apms_ctx* ctx, uint32_t* dst_bits_dev, float* dst_scales_dev,
                                  int64_t chunk_begin, int64_t chunk_end);
apms_status apms_message_offsets(apms_ctx* ctx, int worker, size_t* bits_offset, size_t* scales_offset);
apms_status apms_ipc_export(apms_ctx* ctx, void* handle_out);
apms_status apms_ipc_open(const void* handle, void** base_dev);
apms_status apms_ipc_close(void* base_dev);

/* Copy x (d floats) to dst: device memory if dst_is_device != 0 (stream-ordered), else
 * host memory (synchronises the stream). */
apms_status apms_get_params(apms_ctx* ctx, float* dst, int dst_is_device);

/* Copy one state array to host memory (synchronises).  `worker` is ignored for arrays
 * that are not per worker.  Errors and momentum are produced from the stored form: the
 * library keeps, per worker and for the server, the compensated vector z and the chunk
 * scales, from which delta = z - (+-scale) and m = +-scale follow exactly. */
apms_status apms_get_state(apms_ctx* ctx, apms_state_id which, int worker, void* dst_host);

/* The same for elements [first, first + count) of the array (count floats or words). */
apms_status apms_get_state_slice(apms_ctx* ctx, apms_state_id which, int worker, int64_t first,
                                 int64_t count, void* dst_host);

/* Overwrite X, V, M, WORKER_ERR or SERVER_ERR from host memory (teacher forcing, restoring
 * a checkpoint).  Setting an error array resets that side's stored scales to zero (they
 * read as 0 until the next step); sign words and scales themselves cannot be set.
 * Synchronises. */
apms_status apms_set_state(apms_ctx* ctx, apms_state_id which, int worker, const void* src_host);

/* Restore the Adam step counter and phase of a checkpoint (t = Adam steps taken so far; it sets the
 * bias correction of the next warmup step).  Going to COMPRESSED from WARMUP freezes v as apms_freeze_v
 * does; going back to WARMUP while the momentum is held as a server message first writes it out in
 * binary32, which is what the Adam step reads.  A phase-wise step in progress is abandoned.
 * The schedule's step counter is restored separately with apms_set_step. */
apms_status apms_restore(apms_ctx* ctx, int t, apms_phase phase);

/* Algorithm 1 end to end: T_w Adam steps, then compression-phase steps, with the learning rate
 * gamma_t of the paper's BERT runs (Section 5.2: linear increase to the peak over the first
 * steps, then multiplied by a constant factor after every so many steps).  Step k = 0, 1, ...:
 *   k <  lr_ramp_steps :  lr = peak_lr * (k + 1) / lr_ramp_steps
 *   k >= lr_ramp_steps :  lr = peak_lr * lr_decay ^ floor((k - lr_ramp_steps) / lr_decay_every)
 * (lr_ramp_steps = 0: no ramp; lr_decay_every = 0: no decay), evaluated in binary64 and rounded
 * once.  The paper's BERT-Large values would be {23000, 4e-4f, 12500, 0.99f, 520}. */
typedef struct {
    int64_t warmup_steps;     /* T_w: Adam steps before v is frozen                  */
    float   peak_lr;
    int64_t lr_ramp_steps;
    float   lr_decay;
    int64_t lr_decay_every;
} apms_schedule;

/* gamma_k of a schedule (pure function; 0 for a NULL schedule or k < 0). */
float apms_schedule_lr(const apms_schedule* schedule, int64_t step);

/* Attach a schedule (copied) for apms_step; NULL detaches it. */
apms_status apms_set_schedule(apms_ctx* ctx, const apms_schedule* schedule);

/* One step of Algorithm 1 under the attached schedule: sets gamma_k, runs a warmup step while
 * fewer than T_w steps have been taken, calls apms_freeze_v when T_w is reached, and a
 * compression-phase step from then on.  Same gradient contract as the *_typed functions.
 * The step counter starts at 0 at apms_set_params and counts only successful apms_step calls. */
apms_status apms_step(apms_ctx* ctx, const void* const* grads_dev, apms_grad_type type);
int64_t     apms_get_step(const apms_ctx* ctx);

/* Set the step counter of apms_step (what apms_get_step returned when a checkpoint was taken), so that
 * a restored context continues the schedule - the learning-rate ramp and decay of Section 5.2 and the
 * T_w warmup steps of Algorithm 1 - where the saved one stopped instead of from step 0.  Call it after
 * apms_restore: in the COMPRESSED phase the steps beyond t count as compression-phase steps taken,
 * which fixes the variant and the compressor as they do in an uninterrupted run. */
apms_status apms_set_step(apms_ctx* ctx, int64_t steps);

/* Monitor for Assumption 1 (the compression errors stay bounded): squared l2 norms of the n
 * worker errors delta^(i) (worker_sq_host, n doubles, may be NULL) and of the server error
 * delta-bar (server_sq_host, may be NULL), summed in binary64 in a fixed order.  Reads every
 * compensated vector once ((n+1) d floats) and synchronises.  Phase must be COMPRESSED.  Not part of
 * a step; call it as often as wanted.  With the top-k compressor the error of an element is its
 * compensated value where it was not sent and zero where it was. */
apms_status apms_error_norms(apms_ctx* ctx, double* worker_sq_host, double* server_sq_host);

apms_phase  apms_get_phase(const apms_ctx* ctx);
int         apms_get_t(const apms_ctx* ctx);

/* Choose the compressor (see apms_compressor); topk_fraction in (0, 1] is used for TOPK only. */
apms_status apms_set_compressor(apms_ctx* ctx, apms_compressor kind, double topk_fraction);

/* Choose the variant (see apms_variant); allowed until the first compression-phase step has run. */
apms_status apms_set_variant(apms_ctx* ctx, apms_variant variant);

/* "APMSqueeze (Uncompressed)" of Section 5.3 (item 3): a step with v frozen and nothing compressed,
 *   m <- (1/n) sum_i (b1 m + (1-b1) g_i)  (worker order) ;  x <- x - (lr m) / (sqrt(v) + eps).
 * Phase must be COMPRESSED.  Compression errors are neither read nor changed; if the momentum is held
 * as a server message it is first written out in binary32.  Counted under APMS_KERNEL_WARMUP_ADAM by
 * apms_kernel_time.  Same gradient contract as the *_typed functions. */
apms_status apms_uncompressed_step_typed(apms_ctx* ctx, const void* const* grads_dev, apms_grad_type type);

/* Choose the scale definition (see apms_scale_kind); any phase, takes effect from the next step. */
apms_status apms_set_scale_kind(apms_ctx* ctx, apms_scale_kind kind);

/* Launch-shape override (tuning and tests); results do not depend on it except for the order
 * of the binary64 additions inside a chunk's sum of squares. */
apms_status apms_set_team_mode(apms_ctx* ctx, apms_team_mode mode);

/* Guard bytes (a debugging aid that stands in for a memory checker).  apms_set_guard_bytes(b) is a
 * process-wide switch read by apms_create and apms_workspace_bytes: contexts created while b > 0 (a multiple
 * of 256, at most 1 MiB) lay out their workspace with at least b bytes that belong to no array behind every
 * row of every array (each worker's compensated vector, sign words, scales, partial sums, ...) and before the
 * first; apms_set_params and apms_freeze_v fill them with a fixed pattern.  apms_check_guards synchronises the
 * stream, reads all guard bytes back and compares: APMS_OK if untouched, APMS_ERR_BOUNDS otherwise, with the
 * workspace offset of the first changed byte in *bad_offset (may be NULL) and the array it follows named in
 * apms_last_error.  Results of steps do not depend on the switch.  b = 0 restores the ordinary layout for
 * contexts created afterwards. */
apms_status apms_set_guard_bytes(size_t bytes);
apms_status apms_check_guards(apms_ctx* ctx, int64_t* bad_offset);

/* The checked build of the library (compiled with -DAPMS_BOUNDS_CHECK, `libapms_checked.so`; the debugging aid
 * that goes with the guard bytes): every global store of the 1-bit step's kernels, of the Adam, update and
 * finalize kernels, their streaming loads and the sources of their bulk copies are validated on the device
 * against the live contexts' workspaces and guard regions.  An access that would leave its array is skipped and
 * recorded; the next synchronising call (and apms_check_guards) returns APMS_ERR_BOUNDS with the offset in
 * apms_last_error.  Nothing traps or faults.  (Not covered: the top-k kernels and the monitor.)
 * apms_build_is_checked: 1 in that build, 0 in the ordinary one, where the accessors compile to nothing.
 * apms_selftest_bounds: checked build with the guard layout only - issues one checked store aimed into the guard
 * bytes behind x and returns APMS_OK iff it was refused, reported and the guard bytes are untouched; clears the
 * report.  APMS_ERR_BAD_STATE in the ordinary build. */
int         apms_build_is_checked(void);
apms_status apms_selftest_bounds(apms_ctx* ctx);

/* Kernel timing: when enabled, every kernel launch is bracketed by CUDA events on the
 * context's stream.  apms_kernel_time() synchronises the stream, returns the total time
 * and launch count of one kernel since the last call for that kernel, and resets them. */
apms_status apms_set_timing(apms_ctx* ctx, int enabled);
apms_status apms_kernel_time(apms_ctx* ctx, apms_kernel_id which, double* total_ms, int64_t* launches);

/* Self-test of the report path of bounded device-side waits.  Every wait inside the library's kernels
 * (they wait only for their own asynchronous copies) gives up after about a second, records that in a
 * status word and ends its CTA; the next synchronising call then returns APMS_ERR_TIMEOUT.  This call
 * runs a one-CTA kernel that waits, with a bound of about a millisecond, for a barrier that nothing
 * completes, and checks that the status word reads "gave up": APMS_OK if so.  With leave_reported != 0
 * the word stays set, so that the next synchronising call returns APMS_ERR_TIMEOUT (apms_set_params
 * clears it); otherwise it is cleared again.  Synchronises.  Harmless: no fault, no hang, no state touched. */
apms_status apms_selftest_wait_report(apms_ctx* ctx, int leave_reported);

/* Kernels launched by this context since creation. */
int64_t     apms_launch_count(const apms_ctx* ctx);

/* Message of the last failure on this context (ctx == NULL: of the last failed
 * apms_create, apms_ipc_open or apms_ipc_close on this thread).  Never NULL. */
const char* apms_last_error(const apms_ctx* ctx);

/* Free the context (and its workspace if it allocated one).  NULL is ignored. */
void        apms_destroy(apms_ctx* ctx);

/* Allocation-free compression of a flat vector.  (The paper has no counterpart: this entry
 * point exists for callers, not for the algorithm.)
 *
 * Who needs it: code that runs where device memory may not be allocated or freed - inside a
 * region of a framework that forbids allocator calls (a step function that must not disturb a
 * caching allocator or its memory accounting), a plugin that is handed a fixed set of buffers
 * and a stream and nothing else, a latency-critical loop in which cudaMalloc's implicit
 * device-wide synchronisation is unacceptable.  Such a caller cannot create a context with its
 * own workspace and has no spare buffer to bind one to.
 *
 * What it does: the 1-bit compressor of Section 5.1 on every chunk of z, as the worker side of
 * apms_compressed_step does for a vector z = m_i + delta_i that is already formed:
 *   scales_dev[c] = ||z_c||_2 / sqrt(L_c),   bit j of bits_dev = (z[j] >= 0),
 * with the sign-word and scale layout stated at the top of this file.  z is not modified.
 *   z_dev       device, d floats, 16-byte aligned, read-only
 *   bits_dev    device, ceil(d/32) uint32, written (padding bits 0)
 *   scales_dev  device, ceil(d/chunk) floats, written
 *   cuda_stream a cudaStream_t passed as void* (NULL = the legacy default stream) on the
 *               current device; the call enqueues two kernels and returns without synchronising
 * The caller owns all three buffers.  The only memory the kernels use beyond them is one
 * binary64 partial sum of squares per 32768-element tile of a chunk; it lives in a fixed array
 * of APMS_NOALLOC_MAX_TILES doubles (128 KiB) that is part of the library's device image, so
 * every GPU that loads the library holds those 128 KiB until the process exits.  The call makes
 * no cudaMalloc / cudaFree and calls no allocating routine of any library.
 *
 * Limits and rules
 *   - ceil(d/chunk) * ceil(chunk/32768) must not exceed APMS_NOALLOC_MAX_TILES (for chunks up
 *     to 32768 elements that is d <= 2^29); larger shapes, d < 1, or a chunk that is not a
 *     positive multiple of 32 return APMS_ERR_INVALID_ARG before anything is launched.
 *   - The first call on each device looks up the device address of the fixed array (once per
 *     device, with that device current).  Make that first call before any stream capture.
 *   - All calls on a device share the one array.  It needs no clearing - every tile's slot is
 *     overwritten before it is read - but it keeps the last call's contents, and two calls
 *     whose kernels may overlap on the GPU (different streams without an ordering between
 *     them, or different host threads) race on it and give wrong scales.  Calls on one stream
 *     are safe back to back.
 *   - There is no context: the message of a failure is read with apms_last_error(NULL) on the
 *     calling thread. */
#define APMS_NOALLOC_MAX_TILES 16384
apms_status apms_compress_noalloc(const float* z_dev, int64_t d, int64_t chunk,
                                  uint32_t* bits_dev, float* scales_dev, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* APMS_H */
